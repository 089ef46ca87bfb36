"""Grouped forward of sibling layers (the q/k/v or gate/up projections of a decoder block read the same activations):
every sibling against the fp64 oracle of Eq. 8, and against the layer-by-layer entry point."""
import numpy as np
import pytest
import torch

from oracle import lopro_oracle as o
from paper_2601_19675_b200 import lopro, synth
from tests._layers import bf16_bits_to_device, device_bf16_to_f64, oracle_args, random_layer_np, to_device

pytestmark = pytest.mark.gpu


def _siblings(n, ms, bits, g, b, r, seed, ranks=None):
    layers, descs, blobs = [], [], []
    for i, m in enumerate(ms):
        rk = r if ranks is None else ranks[i]
        layer = random_layer_np(n, m, bits, g, rk, seed=seed + 31 * i)       # own codes, perm, A, B per sibling
        d = lopro.make_desc(n, m, bits, g, b, rank=rk)
        dev = to_device(layer)
        blobs.append(lopro.pack(d, dev["codes"], dev["scales"], dev["zeros"], dev["perm"], dev["A"], dev["B"]))
        layers.append(layer)
        descs.append(d)
    return layers, descs, blobs


def _check_group(layers, descs, blobs, x_bits, rows=None, shared=None, bit_equal=True):
    T = x_bits.shape[0]
    x = bf16_bits_to_device(x_bits)
    path, launches = lopro.linear_fwd_group_path(descs, T)
    if shared is not None:
        assert (path == 2) == shared
        if shared:
            assert launches == 2
    ws = torch.zeros(lopro.group_workspace_bytes(descs, T), dtype=torch.uint8, device="cuda")
    ys_bf = lopro.linear_fwd_group(descs, blobs, x, lopro.OUT_BF16, workspace=ws)
    ys_bf = [y.clone() for y in ys_bf]
    ys_f32 = lopro.linear_fwd_group(descs, blobs, x, lopro.OUT_F32, workspace=ws)
    torch.cuda.synchronize()
    assert lopro.workspace_status(ws) == lopro.OK
    x64 = o.bf16_bits_to_f64(x_bits)
    for layer, d, blob, y_bf, y_f32 in zip(layers, descs, blobs, ys_bf, ys_f32):
        sel = slice(None) if rows is None else rows[rows < d.d_out]
        args = oracle_args(layer, d.group_size, d.identity_cols, d.block_size, rows=None if rows is None else sel)
        exact = o.forward_exact(x64, **args)
        mirrored = o.forward_mirrored(x64, **args, round_w=False, round_t="f16", out="f32")
        got_bf = device_bf16_to_f64(y_bf)[:, sel]
        got_f32 = y_f32.cpu().numpy().astype(np.float64)[:, sel]
        assert o.max_rel_err(got_bf, exact) <= 2e-2
        assert o.max_rel_err(got_f32, mirrored) <= 1e-3
        # the same kernels sum the same products in the same order as the layer-by-layer call
        alone = lopro.linear_fwd(d, blob, x, lopro.OUT_F32)
        if bit_equal:
            assert torch.equal(alone, y_f32)
        else:
            # persistent kernel: a layer's CTAs own other runs of row tiles than in the single-layer launch, and
            # the split of K inside a run's last tiles depends on the run -- equal up to fp32 summation order
            scale = alone.abs().max().item()
            assert (alone - y_f32).abs().max().item() <= 2e-5 * scale


@pytest.mark.parametrize("T", [1, 5, 8, 16, 32])
@pytest.mark.parametrize("bits,g,ms", [(4, 128, (256, 272, 144)), (2, 64, (528, 64)), (3, 64, (96, 96, 96, 160))])
def test_sibling_layers_share_two_launches(T, bits, g, ms):
    n, r = 2048, 17
    layers, descs, blobs = _siblings(n, ms, bits, g, 128, r, seed=T + bits)
    _check_group(layers, descs, blobs, synth.activations(T, n, seed=T + 40, outlier_frac=0.01), shared=True)


def test_groups_that_cannot_share_run_layer_by_layer():
    n = 1024
    # different ranks: no shared launches, same results
    layers, descs, blobs = _siblings(n, (128, 160), 4, 128, 128, 0, seed=3, ranks=(16, 32))
    _check_group(layers, descs, blobs, synth.activations(8, n, seed=9), shared=False)
    # more than 32 tokens
    layers, descs, blobs = _siblings(n, (128, 160), 4, 128, 128, 16, seed=4)
    _check_group(layers, descs, blobs, synth.activations(40, n, seed=10), shared=False)
    # a single layer is a group too
    _check_group(layers[:1], descs[:1], blobs[:1], synth.activations(8, n, seed=11), shared=False)


@pytest.mark.parametrize("T", [1, 8, 32])
def test_attention_projections_of_the_stack_at_full_size(T):
    # q, k, v of the 32-layer stack configuration: three 4096 x 4096 layers, 4-bit g128, block 128, rank 32
    n = 4096
    layers, descs, blobs = _siblings(n, (4096, 4096, 4096), 4, 128, 128, 32, seed=T)
    rows = np.unique(np.concatenate([[0, 15, 16, 4095, 2048], np.random.default_rng(T).integers(0, 4096, size=24)]))
    # together the three projections make more than one wave of the per-group kernel, so the group runs through the
    # persistent kernel while each layer alone does not: same products, another order of summation
    _check_group(layers, descs, blobs, synth.activations(T, n, seed=T + 1), rows=rows, shared=True, bit_equal=False)
    with lopro.configured(lopro.OPT_NO_TALL, 1):
        _check_group(layers, descs, blobs, synth.activations(T, n, seed=T + 1), rows=rows, shared=True)


def _persistent_rows(extra_tiles):
    # more than two 16-row tiles per SM: the layer runs through the persistent kernel
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    return 16 * (2 * sms + extra_tiles)


@pytest.mark.parametrize("T", [1, 8, 16, 32])
@pytest.mark.parametrize("bits,g,extra", [(4, 128, (1, 1)), (2, 64, (7, 130)), (3, 64, (3, 40, 90))])
def test_sibling_layers_through_the_persistent_kernel(T, bits, g, extra):
    n, r = 512, 16
    ms = tuple(_persistent_rows(e) for e in extra)
    layers, descs, blobs = _siblings(n, ms, bits, g, 128, r, seed=T + bits)
    assert all(lopro.linear_fwd_path(d, T)[0] == lopro.PATH_TALL for d in descs)
    _check_group(layers, descs, blobs, synth.activations(T, n, seed=T + 50, outlier_frac=0.01), shared=True, bit_equal=False)


@pytest.mark.parametrize("T", [1, 32])
def test_mlp_projections_of_the_stack_at_full_size(T):
    # gate, up of the 32-layer stack configuration: two 4096 -> 11008 layers, 4-bit g128, block 128, rank 32
    n = 4096
    layers, descs, blobs = _siblings(n, (11008, 11008), 4, 128, 128, 32, seed=T + 7)
    rows = np.unique(np.concatenate([[0, 15, 16, 11007, 5504], np.random.default_rng(T).integers(0, 11008, size=24)]))
    _check_group(layers, descs, blobs, synth.activations(T, n, seed=T + 2), rows=rows, shared=True, bit_equal=False)


def test_group_argument_errors():
    n = 512
    layers, descs, blobs = _siblings(n, (64, 64), 4, 128, 64, 0, seed=5)
    x = torch.zeros((4, n), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(lopro.LoproError) as e:
        lopro.linear_fwd_group(descs, blobs, x, workspace=torch.zeros(256, dtype=torch.uint8, device="cuda"))
    assert e.value.status == lopro.ERR_BUFFER_TOO_SMALL
    other = lopro.make_desc(1024, 64, 4, 128, 64, rank=0)          # siblings must read the same x
    with pytest.raises(lopro.LoproError) as e:
        lopro.linear_fwd_group([descs[0], other], blobs, x)
    assert e.value.status == lopro.ERR_INVALID_ARG
