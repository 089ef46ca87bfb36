"""Test helpers: build synthetic LoPRo layers once, hand the same bytes to the CPU oracle (as fp64)
and to the CUDA library (as device tensors).  Holds none of the method's arithmetic."""
import numpy as np
import torch

from oracle import lopro_oracle as o
from paper_2601_19675_b200 import synth


def random_layer_np(d_in, d_out, bits, group_size, rank, seed=0):
    """Stored tensors of one layer as numpy bit patterns (cfg2-style recipe)."""
    return synth.random_layer(d_in, d_out, bits, group_size, rank, seed)


def oracle_args(layer, group_size, b_i, b_h, rows=None):
    """Keyword arguments of oracle.forward_* decoded to fp64 (optionally a subset of output rows)."""
    sel = slice(None) if rows is None else np.asarray(rows)
    a = o.f16_bits_to_f64(layer["A"])[sel] if layer["A"].size else np.zeros((layer["codes"][sel].shape[0], 0))
    b = o.f16_bits_to_f64(layer["B"]) if layer["B"].size else np.zeros((0, layer["codes"].shape[1]))
    return dict(codes=layer["codes"][sel], scales=o.f16_bits_to_f64(layer["scales"])[sel],
                zeros=o.f16_bits_to_f64(layer["zeros"])[sel], perm=layer["perm"], a=a, b=b, g=group_size,
                b_i=b_i, b_h=b_h)


def to_device(layer, device="cuda"):
    """numpy bit patterns -> device tensors with the dtypes the binding expects."""
    def t16(a):
        return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to(device)
    out = dict(codes=torch.from_numpy(np.ascontiguousarray(layer["codes"])).to(device),
               scales=t16(layer["scales"]), zeros=t16(layer["zeros"]),
               perm=torch.from_numpy(np.ascontiguousarray(layer["perm"], dtype=np.int32)).to(device))
    out["A"] = t16(layer["A"]) if layer["A"].size else None
    out["B"] = t16(layer["B"]) if layer["B"].size else None
    return out


def bf16_bits_to_device(bits, device="cuda"):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(device).view(torch.bfloat16)


def device_bf16_to_f64(t):
    """Device bf16 tensor -> fp64 numpy via its bit patterns (no torch arithmetic)."""
    bits = t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    return o.bf16_bits_to_f64(bits)
