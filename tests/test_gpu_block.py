"""Decoder-block operations between the quantized linears (RMS norm with residual, rotary embedding with cache append,
attention of one new token over a key/value cache, SiLU gating) against their fp64 definitions.  Inputs and outputs are
bf16: the tolerance is the output rounding (2^-8 relative) plus fp32 accumulation."""
import numpy as np
import pytest
import torch

from oracle import glue_oracle as g
from oracle import lopro_oracle as o
from paper_2601_19675_b200 import lopro, synth
from tests._layers import bf16_bits_to_device, device_bf16_to_f64

pytestmark = pytest.mark.gpu


def _bits(shape, seed, scale=1.0):
    n = int(np.prod(shape))
    return (synth.activations(1, n, seed=seed)[0]).reshape(shape) if scale == 1.0 else \
        synth.f32_to_bf16_bits(o.bf16_bits_to_f64(synth.activations(1, n, seed=seed)[0]).astype(np.float32) * np.float32(scale)).reshape(shape)


def _status():
    return torch.zeros(1, dtype=torch.int32, device="cuda")


@pytest.mark.parametrize("T,d,with_y", [(1, 4096, False), (5, 4096, True), (32, 4096, True), (3, 64, True), (2, 11008, False)])
def test_add_rmsnorm(T, d, with_y):
    hb, yb, wb = _bits((T, d), 1), _bits((T, d), 2, 0.5), _bits((d,), 3)
    h = bf16_bits_to_device(hb)
    y = bf16_bits_to_device(yb) if with_y else None
    out = lopro.block_add_rmsnorm(h, y, bf16_bits_to_device(wb), 1e-5)
    torch.cuda.synchronize()
    h64 = o.bf16_bits_to_f64(hb)
    if with_y:
        h64 = o.round_bf16(h64 + o.bf16_bits_to_f64(yb))          # the residual stream is stored in bf16
        np.testing.assert_array_equal(device_bf16_to_f64(h), h64)
    ref = g.rmsnorm(h64, o.bf16_bits_to_f64(wb), 1e-5)
    got = device_bf16_to_f64(out)
    assert np.max(np.abs(got - ref) / (np.abs(ref) + 1e-3)) <= 2.0 ** -8 + 1e-5


@pytest.mark.parametrize("T,H,hd,ctx_max", [(1, 32, 128, 2049), (4, 2, 64, 16), (32, 32, 128, 130)])
def test_rope_append(T, H, hd, ctx_max):
    qb, kb, vb = _bits((T, H * hd), 4), _bits((T, H * hd), 5), _bits((T, H * hd), 6)
    pos = np.array([(ctx_max - 1) if t == 0 else (7 * t) % ctx_max for t in range(T)], dtype=np.int32)
    q, k, v = bf16_bits_to_device(qb), bf16_bits_to_device(kb), bf16_bits_to_device(vb)
    kc = torch.zeros((T, H, ctx_max, hd), dtype=torch.bfloat16, device="cuda")
    vc = torch.zeros_like(kc)
    st = _status()
    lopro.block_rope_append(q, k, v, torch.from_numpy(pos).cuda(), kc, vc, 10000.0, st)
    torch.cuda.synchronize()
    assert int(st.item()) == lopro.OK
    q_ref = g.rope(o.bf16_bits_to_f64(qb).reshape(T, H, hd), pos)
    k_ref = g.rope(o.bf16_bits_to_f64(kb).reshape(T, H, hd), pos)
    tol = lambda ref: 2.0 ** -8 * np.abs(ref) + 2.0 ** -7 * 2.0 ** -8 * np.abs(ref).max() + 1e-6
    got_q = device_bf16_to_f64(q).reshape(T, H, hd)
    assert np.all(np.abs(got_q - q_ref) <= tol(q_ref))
    kc64, vc64 = device_bf16_to_f64(kc), device_bf16_to_f64(vc)
    for t in range(T):
        assert np.all(np.abs(kc64[t, :, pos[t]] - k_ref[t]) <= tol(k_ref[t]))
        np.testing.assert_array_equal(vc64[t, :, pos[t]], o.bf16_bits_to_f64(vb).reshape(T, H, hd)[t])    # values are copied
        mask = np.ones(ctx_max, dtype=bool)
        mask[pos[t]] = False
        assert np.all(kc64[t][:, mask] == 0.0) and np.all(vc64[t][:, mask] == 0.0)                        # nothing else is touched


def test_rope_append_reports_a_position_outside_the_cache():
    T, H, hd, ctx_max = 2, 2, 64, 8
    q = bf16_bits_to_device(_bits((T, H * hd), 1))
    kc = torch.zeros((T, H, ctx_max, hd), dtype=torch.bfloat16, device="cuda")
    vc = torch.zeros_like(kc)
    st = _status()
    lopro.block_rope_append(q, q.clone(), q.clone(), torch.tensor([3, 8], dtype=torch.int32, device="cuda"), kc, vc, 10000.0, st)
    torch.cuda.synchronize()
    assert int(st.item()) == lopro.ERR_INVALID_DATA
    assert torch.all(kc[1] == 0)


@pytest.mark.parametrize("T,H,ctx_max,ctx", [(1, 32, 2049, [2049]), (3, 4, 700, [1, 256, 513]), (32, 32, 300, None), (2, 2, 256, [255, 256])])
def test_attention_decode(T, H, ctx_max, ctx):
    hd = 128
    if ctx is None:
        ctx = [1 + (37 * t) % ctx_max for t in range(T)]
    ctx = np.array(ctx, dtype=np.int32)
    qb = _bits((T, H * hd), 7)
    kb, vb = _bits((T, H, ctx_max, hd), 8), _bits((T, H, ctx_max, hd), 9)
    scale = 1.0 / np.sqrt(hd)
    q, kc, vc = bf16_bits_to_device(qb), bf16_bits_to_device(kb), bf16_bits_to_device(vb)
    ws = torch.empty(lopro.block_attention_workspace_bytes(T, H, hd, ctx_max), dtype=torch.uint8, device="cuda")
    st = _status()
    out = lopro.block_attention_decode(q, kc, vc, torch.from_numpy(ctx).cuda(), float(scale), ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == lopro.OK
    ref = g.attention_decode(o.bf16_bits_to_f64(qb).reshape(T, H, hd), o.bf16_bits_to_f64(kb), o.bf16_bits_to_f64(vb), ctx, scale)
    got = device_bf16_to_f64(out).reshape(T, H, hd)
    # bf16 output rounding plus the fast exponential (2 ulp of fp32 on arguments up to a few tens)
    assert np.max(np.abs(got - ref)) <= 2.0 ** -8 * np.abs(ref).max() + 1e-4


def test_attention_reports_a_bad_context_length():
    T, H, hd, ctx_max = 2, 2, 128, 64
    q = bf16_bits_to_device(_bits((T, H * hd), 1))
    kc = bf16_bits_to_device(_bits((T, H, ctx_max, hd), 2))
    ws = torch.empty(lopro.block_attention_workspace_bytes(T, H, hd, ctx_max), dtype=torch.uint8, device="cuda")
    st = _status()
    out = lopro.block_attention_decode(q, kc, kc, torch.tensor([5, 65], dtype=torch.int32, device="cuda"), 0.1, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == lopro.ERR_INVALID_DATA
    assert torch.all(out[1] == 0)


@pytest.mark.parametrize("T,d", [(1, 11008), (32, 11008), (3, 64)])
def test_silu_mul(T, d):
    gb, ub = _bits((T, d), 10, 3.0), _bits((T, d), 11)
    out = lopro.block_silu_mul(bf16_bits_to_device(gb), bf16_bits_to_device(ub))
    torch.cuda.synchronize()
    ref = g.silu_mul(o.bf16_bits_to_f64(gb), o.bf16_bits_to_f64(ub))
    got = device_bf16_to_f64(out)
    assert np.max(np.abs(got - ref) / (np.abs(ref) + 1e-6)) <= 2.0 ** -8 + 1e-5


def test_block_argument_errors():
    x = torch.zeros((2, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(lopro.LoproError) as e:
        lopro.block_add_rmsnorm(torch.zeros((2, 60), dtype=torch.bfloat16, device="cuda"), None, x[0, :60].contiguous(), 1e-5)
    assert e.value.status == lopro.ERR_INVALID_ARG
    assert lopro.block_attention_workspace_bytes(1, 1, 64, 16) == 0      # head size the attention kernels are not written for
