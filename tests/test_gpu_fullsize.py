"""Parity at the full sizes of the benchmark workloads, in the launch configuration bench.py times,
on sampled output rows the oracle computes one by one (configurations 2, 3 and 4, and the three linear
shapes of the stack of configuration 5)."""
import numpy as np
import pytest
import torch

from oracle import lopro_oracle as o
from paper_2601_19675_b200 import lopro, synth
from tests._layers import bf16_bits_to_device, device_bf16_to_f64, oracle_args, random_layer_np, to_device

pytestmark = pytest.mark.gpu


def _sampled(cfg, T, n_rows=48, seed=0, layout=lopro.LAYOUT_FRAGMENT):
    c = synth.CONFIGS[cfg] if isinstance(cfg, str) else cfg
    n, m = c["d_in"], c["d_out"]
    layer = random_layer_np(n, m, c["bits"], c["group_size"], c["rank"], seed=seed)
    d = lopro.make_desc(n, m, c["bits"], c["group_size"], c["block_size"], c["identity_cols"], c["rank"], layout=layout)
    dev = to_device(layer)
    blob = lopro.pack(d, dev["codes"], dev["scales"], dev["zeros"], dev["perm"], dev["A"], dev["B"])
    del dev
    x_bits = synth.activations(T, n, seed=seed, outlier_frac=c.get("outlier_frac", 0.0),
                               outlier_scale=c.get("outlier_scale", 20.0))
    x = bf16_bits_to_device(x_bits)
    ws = torch.zeros(lopro.workspace_bytes(d, T), dtype=torch.uint8, device="cuda")
    y_bf = lopro.linear_fwd(d, blob, x, lopro.OUT_BF16, workspace=ws)
    y_f32 = lopro.linear_fwd(d, blob, x, lopro.OUT_F32, workspace=ws)
    torch.cuda.synchronize()
    assert lopro.workspace_status(ws) == lopro.OK
    rng = np.random.default_rng(seed + 17)
    rows = np.unique(np.concatenate([[0, 15, 16, m - 1, m - 16, m // 2], rng.integers(0, m, size=n_rows)]))
    toks = np.unique(np.concatenate([[0, T - 1], rng.integers(0, T, size=min(T, 24))]))
    args = oracle_args(layer, d.group_size, d.identity_cols, d.block_size, rows=rows)
    x64 = o.bf16_bits_to_f64(x_bits[toks])
    exact = o.forward_exact(x64, **args)
    mirrored = o.forward_mirrored(x64, **args, round_w=lopro.linear_fwd_path(d, T)[0] == lopro.PATH_PREFILL, round_t="f16", out="f32")
    # error relative to the rms of the sampled entries of each token's row
    got_bf = device_bf16_to_f64(y_bf[torch.from_numpy(toks).cuda()])[:, rows]
    got_f32 = y_f32[torch.from_numpy(toks).cuda()].cpu().numpy().astype(np.float64)[:, rows]
    assert o.max_rel_err(got_bf, exact) <= 2e-2
    assert o.max_rel_err(got_f32, mirrored) <= 1e-3
    assert torch.isfinite(y_f32).all()


LAYOUTS = [lopro.LAYOUT_FRAGMENT, lopro.LAYOUT_ROWBLOCK]


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("T", [1, 8])
def test_cfg2_decode(T, layout):
    _sampled("cfg2", T, layout=layout)


@pytest.mark.parametrize("layout", LAYOUTS)
def test_cfg3_prefill(layout):
    _sampled("cfg3", 2048, n_rows=32, layout=layout)


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("T", [16, 4096])
def test_cfg4_large_layer(T, layout):
    _sampled("cfg4", T, n_rows=24, layout=layout)


# the three linear shapes of the 32-layer stack configuration (hidden 4096, MLP 11008; 4-bit, g = 128, rank 32,
# block 128): attention projections, gate/up, and down -- whose 11008 input columns are neither a multiple of
# 1024 (ragged last stage of the streaming kernels) nor of 256 x 8
_STACK = dict(bits=4, group_size=128, block_size=128, identity_cols=128, rank=32)


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("T", [1, 32])
@pytest.mark.parametrize("n,m", [(4096, 4096), (4096, 11008), (11008, 4096)])
def test_stack_linear_shapes(n, m, T, layout):
    _sampled(dict(d_in=n, d_out=m, **_STACK), T, n_rows=32, seed=n // 64 + T, layout=layout)
