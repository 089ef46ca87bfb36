"""Forward of the experts of a mixture layer: every expert's rows against the fp64 oracle of Eq. 8 and against the
single-layer entry point called on those rows."""
import numpy as np
import pytest
import torch

from oracle import lopro_oracle as o
from paper_2601_19675_b200 import lopro, synth
from tests.test_gpu_forward import _gate_b_with_ties
from tests._layers import bf16_bits_to_device, device_bf16_to_f64, oracle_args, random_layer_np, to_device

pytestmark = pytest.mark.gpu


def _experts(n, m, bits, g, b, r, n_experts, seed):
    d = lopro.make_desc(n, m, bits, g, b, rank=r)
    layers, blobs = [], []
    for e in range(n_experts):
        layer = random_layer_np(n, m, bits, g, r, seed=seed + 17 * e)          # own codes, perm, A, B per expert
        dev = to_device(layer)
        blobs.append(lopro.pack(d, dev["codes"], dev["scales"], dev["zeros"], dev["perm"], dev["A"], dev["B"]))
        layers.append(layer)
    return d, layers, blobs


def _check_experts(d, layers, blobs, counts, seed, shared=None, rows=None, bit_equal=True):
    offs = [0]
    for c in counts:
        offs.append(offs[-1] + c)
    total = offs[-1]
    x_bits = synth.activations(max(total, 1), d.d_in, seed=seed, outlier_frac=0.01)[:total]
    x = bf16_bits_to_device(x_bits) if total else torch.zeros((0, d.d_in), dtype=torch.bfloat16, device="cuda")
    path, launches = lopro.linear_fwd_experts_path(d, offs)
    if shared is not None:
        assert (path == 2) == shared
        if shared:
            assert launches == 2 * ((sum(c > 0 for c in counts) + 7) // 8)
    ws = torch.zeros(max(lopro.experts_workspace_bytes(d, len(blobs), max(counts + [1])), 256), dtype=torch.uint8, device="cuda")
    y_bf = lopro.linear_fwd_experts(d, blobs, offs, x, lopro.OUT_BF16, workspace=ws).clone()
    y_f32 = lopro.linear_fwd_experts(d, blobs, offs, x, lopro.OUT_F32, workspace=ws)
    torch.cuda.synchronize()
    assert lopro.workspace_status(ws) == lopro.OK
    x64 = o.bf16_bits_to_f64(x_bits)
    sel = slice(None) if rows is None else rows
    for e, layer in enumerate(layers):
        r0, r1 = offs[e], offs[e + 1]
        if r1 == r0:
            continue
        args = oracle_args(layer, d.group_size, d.identity_cols, d.block_size, rows=None if rows is None else rows)
        exact = o.forward_exact(x64[r0:r1], **args)
        mirrored = o.forward_mirrored(x64[r0:r1], **args, round_w=False, round_t="f16", out="f32")
        assert o.max_rel_err(device_bf16_to_f64(y_bf[r0:r1])[:, sel], exact) <= 2e-2
        got_f32 = y_f32[r0:r1].cpu().numpy().astype(np.float64)[:, sel]
        err_b = o.max_rel_err(got_f32, mirrored)
        if err_b > 1e-3:    # a rotated entry on a bf16 rounding boundary: either side is a valid rounding
            err_b = _gate_b_with_ties(x64[r0:r1], args, False, mirrored, got_f32)
        assert err_b <= 1e-3
        alone = lopro.linear_fwd(d, blobs[e], x[r0:r1], lopro.OUT_F32)
        if bit_equal and r1 - r0 == max(counts):
            # the launch is shaped for the largest row count: that expert runs the very kernel variant of its single call
            assert torch.equal(alone, y_f32[r0:r1])
        else:   # another kernel variant (token tile), or other runs of row tiles per CTA: fp32 summation order differs
            assert (alone - y_f32[r0:r1]).abs().max().item() <= 2e-5 * alone.abs().max().item()


@pytest.mark.parametrize("bits,g", [(4, 128), (2, 64), (3, 64)])
@pytest.mark.parametrize("counts", [[3, 1, 8, 2], [1, 1, 1, 1, 1, 1, 1, 1], [0, 5, 0, 32, 7, 0, 0, 16], [9] * 10, [0, 0, 4]])
def test_experts_share_launches(bits, g, counts):
    n, m, r = 1024, 272, 16
    d, layers, blobs = _experts(n, m, bits, g, 128, r, len(counts), seed=bits + len(counts))
    _check_experts(d, layers, blobs, counts, seed=5 + bits, shared=True)


def test_experts_through_the_persistent_kernel():
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    n, m, r = 512, 16 * (2 * sms + 5), 16
    d, layers, blobs = _experts(n, m, 4, 128, 128, r, 5, seed=2)
    assert lopro.linear_fwd_path(d, 8)[0] == lopro.PATH_TALL
    _check_experts(d, layers, blobs, [8, 0, 3, 20, 1], seed=9, shared=True, bit_equal=False)


def test_experts_with_many_rows_run_one_after_the_other():
    n, m, r = 1024, 256, 16
    d, layers, blobs = _experts(n, m, 4, 128, 128, r, 3, seed=4)
    _check_experts(d, layers, blobs, [40, 2, 0], seed=6, shared=False)
    _check_experts(d, layers, blobs, [0, 0, 0], seed=6)               # nothing to do


@pytest.mark.parametrize("counts", [[8] * 8, [1, 0, 3, 0, 0, 2, 0, 2]])
def test_experts_at_the_shapes_of_a_mixture_model(counts):
    # eight experts 4096 -> 14336 (the up projection of a Mixtral-style block), 2-bit g64, block 256, rank 16
    n, m = 4096, 14336
    d, layers, blobs = _experts(n, m, 2, 64, 256, 16, 8, seed=11)
    rows = np.unique(np.concatenate([[0, 15, 16, m - 1, m // 2], np.random.default_rng(3).integers(0, m, size=24)]))
    _check_experts(d, layers, blobs, counts, seed=12, shared=True, rows=rows, bit_equal=False)


def test_experts_argument_errors():
    d, layers, blobs = _experts(512, 64, 4, 128, 64, 0, 2, seed=5)
    x = torch.zeros((4, 512), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(lopro.LoproError) as e:
        lopro.linear_fwd_experts(d, blobs, [0, 3, 2], x)                        # offsets must not decrease
    assert e.value.status == lopro.ERR_INVALID_ARG
    with pytest.raises(lopro.LoproError) as e:
        lopro.linear_fwd_experts(d, blobs, [0, 2, 4], x, workspace=torch.zeros(256, dtype=torch.uint8, device="cuda"))
    assert e.value.status == lopro.ERR_BUFFER_TOO_SMALL
    assert lopro.linear_fwd_experts_path(d, [1, 2, 3])[0] == 0                 # offsets start at 0
