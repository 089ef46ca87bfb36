"""Offline side on the GPU (Algorithm 1 without calibration): rank-1 sketch with deflation, residual, R' = R P Q and the
round-to-nearest group grid, against the oracle.  Integer results (codes, zero-points, fp16 steps) are compared bit for
bit where both sides take the decision in single precision on the same fp32 input; floating-point stages within
tolerances derived from single-precision rounding."""
import numpy as np
import pytest
import torch

from oracle import lopro_oracle as o
from paper_2601_19675_b200 import lopro, synth
from tests._layers import bf16_bits_to_device, device_bf16_to_f64

pytestmark = pytest.mark.gpu


def _dev(a, dtype=None):
    return torch.from_numpy(np.ascontiguousarray(a if dtype is None else a.astype(dtype))).cuda()


def _f16(t):
    return t.cpu().numpy().view(np.float16).astype(np.float64)


def _rotated_residual(m, n, g, seed):
    """fp32 rows with the structure the quantizer meets: Gaussian bulk, a few outliers, constant groups (positive,
    negative, zero), a group of two values, tiny and large magnitudes."""
    rng = np.random.Generator(np.random.Philox(key=[seed, 77]))
    v = (rng.standard_normal((m, n)) * 0.02).astype(np.float32)
    v[rng.integers(0, m, 40), rng.integers(0, n, 40)] *= np.float32(25.0)
    v[0, :g] = np.float32(0.0)
    v[1, :g] = np.float32(0.375)
    v[2, :g] = np.float32(-0.0123)
    v[3, :g] = np.where(np.arange(g) % 2 == 0, np.float32(1.0), np.float32(-1.0))
    v[4] *= np.float32(1e-3)
    v[5] *= np.float32(300.0)
    return v


@pytest.mark.parametrize("bits,g,n", [(4, 128, 512), (3, 64, 1152), (2, 64, 512), (2, 256, 1024), (4, 64, 8192)])
def test_rtn_kernel_bit_exact_against_the_single_precision_oracle(bits, g, n):
    m = 48
    d = lopro.make_desc(n, m, bits, g, 64, rank=0)
    v = _rotated_residual(m, n, g, seed=bits + n)
    codes, scales, zeros, status = lopro.rtn_quantize(d, _dev(v))
    torch.cuda.synchronize()
    assert int(status.item()) == lopro.OK
    c_ref, s_ref, z_ref = o.rtn_quantize(v, bits, g, dtype=np.float32)
    np.testing.assert_array_equal(codes.cpu().numpy(), c_ref)
    np.testing.assert_array_equal(_f16(scales), s_ref)
    np.testing.assert_array_equal(_f16(zeros), z_ref)


def test_rtn_kernel_reports_bad_input():
    d = lopro.make_desc(256, 16, 4, 64, 64, rank=0)
    v = _rotated_residual(16, 256, 64, seed=1)
    v[7, 100] = np.float32(np.inf)
    *_, status = lopro.rtn_quantize(d, _dev(v))
    torch.cuda.synchronize()
    assert int(status.item()) == lopro.ERR_INVALID_DATA
    v = _rotated_residual(16, 256, 64, seed=1)
    v[9, 64:128] = np.linspace(0.0, 1e-9, 64, dtype=np.float32)      # range / 15 underflows fp16
    *_, status = lopro.rtn_quantize(d, _dev(v))
    torch.cuda.synchronize()
    assert int(status.item()) == lopro.ERR_INVALID_DATA


@pytest.mark.parametrize("n,b_i,b_h,rank", [(512, 64, 64, 16), (1024, 0, 1024, 0), (768, 256, 256, 5), (4096, 128, 128, 32),
                                           (11008, 128, 128, 32), (640, 640, 64, 3), (256, 0, 2, 1)])
def test_residual_rotate_against_the_oracle(n, b_i, b_h, rank):
    m = 32
    d = lopro.make_desc(n, m, 4, 64, b_h, identity_cols=b_i, rank=rank)
    w = synth.weights(m, n, seed=n + rank)
    a_bits, b_bits = synth.factors(m, n, max(rank, 1), seed=n, std=0.05)
    af = o.f16_bits_to_f64(a_bits)[:, :rank]
    bf = o.f16_bits_to_f64(b_bits)[:rank]
    perm = synth.permutation(n, seed=n + 1)
    got, status = lopro.residual_rotate(d, _dev(w), _dev(af, np.float32) if rank else None,
                                        _dev(bf, np.float32) if rank else None, _dev(perm))
    torch.cuda.synchronize()
    assert int(status.item()) == lopro.OK
    resid = w.astype(np.float64) - af @ bf
    ref = o.partial_block_rotate(o.permute_columns(resid, perm), b_i, b_h)
    # fp32: rank fused multiply-adds, log2(b_h) butterfly levels, one scaling -- a few ulp of the largest entry of a block
    tol = 2.0 ** -23 * (4 + rank + np.log2(b_h)) * np.abs(ref).max()
    assert np.max(np.abs(got.cpu().numpy().astype(np.float64) - ref)) <= tol
    # the untouched prefix is the gathered residual itself, to fp32 rounding of the rank terms
    if rank == 0 and b_i:
        np.testing.assert_array_equal(got.cpu().numpy()[:, :b_i], w[:, perm[:b_i]])


def test_residual_rotate_reports_an_index_out_of_range():
    n, m = 256, 16
    d = lopro.make_desc(n, m, 4, 64, 64, rank=0)
    perm = synth.permutation(n, seed=3).copy()
    perm[17] = n + 5
    _, status = lopro.residual_rotate(d, _dev(synth.weights(m, n, seed=1)), None, None, _dev(perm))
    torch.cuda.synchronize()
    assert int(status.item()) == lopro.ERR_INVALID_DATA


@pytest.mark.parametrize("m,n,r,it", [(256, 384, 6, 4), (512, 256, 4, 8), (128, 128, 3, 0)])
def test_r1svd_against_the_oracle(m, n, r, it):
    w = synth.weights(m, n, seed=m + it, spikes=r + 2)
    sk = synth.sketches(r, n, seed=5).astype(np.float32)
    wd = _dev(w.copy())
    U, sigma, V = lopro.r1svd(wd, r, it, _dev(sk))
    torch.cuda.synchronize()
    u_ref, s_ref, v_ref = o.r1svd(w.astype(np.float64), r, it, sk.astype(np.float64))
    np.testing.assert_allclose(sigma.cpu().numpy(), s_ref, rtol=2e-4)
    # unit vectors: absolute tolerance; the product U Sigma V and the deflated remainder in the Frobenius norm
    assert np.max(np.abs(U.cpu().numpy() - u_ref)) <= 5e-4
    assert np.max(np.abs(V.cpu().numpy() - v_ref)) <= 5e-4
    rem_ref = w.astype(np.float64) - (u_ref * s_ref[None, :]) @ v_ref
    assert np.linalg.norm(wd.cpu().numpy() - rem_ref) <= 1e-4 * np.linalg.norm(w)


def test_r1svd_recovers_a_low_rank_matrix():
    # Eq. 10-12 make each step a projection deflation: a rank-3 matrix is exhausted after three ranks, for any sketch
    m, n, k = 192, 320, 3
    rng = np.random.Generator(np.random.Philox(key=[9, 9]))
    w = (rng.standard_normal((m, k)) @ rng.standard_normal((k, n))).astype(np.float32)
    wd = _dev(w.copy())
    U, sigma, V = lopro.r1svd(wd, k, 2, _dev(synth.sketches(k, n, seed=2).astype(np.float32)))
    torch.cuda.synchronize()
    rec = (U.cpu().numpy().astype(np.float64) * sigma.cpu().numpy()[None, :]) @ V.cpu().numpy()
    assert np.linalg.norm(rec - w) <= 2e-5 * np.linalg.norm(w)
    assert np.linalg.norm(wd.cpu().numpy()) <= 2e-5 * np.linalg.norm(w)


def test_r1svd_with_the_fp8_cast_inside_the_loop():
    m, n, r, it = 256, 256, 8, 4
    w = synth.weights(m, n, seed=21, spikes=10)
    sk = synth.sketches(r, n, seed=6).astype(np.float32)
    wd = _dev(w.copy())
    U, sigma, V = lopro.r1svd(wd, r, it, _dev(sk), cast=True)
    torch.cuda.synchronize()
    u, v = U.cpu().numpy().astype(np.float64), V.cpu().numpy().astype(np.float64)
    # every stored entry is an fp8 e4m3 number
    np.testing.assert_array_equal(o.round_e4m3(u), u)
    np.testing.assert_array_equal(o.round_e4m3(v), v)
    u_ref, s_ref, v_ref = o.r1svd(w.astype(np.float64), r, it, sk.astype(np.float64), cast=o.round_e4m3)
    # rank 0 saw the same matrix on both sides: entries differ only where fp32 and fp64 fall on different sides of an
    # fp8 rounding boundary (one step of 2^-3 relative at most), and rarely
    d0 = np.abs(u[:, 0] - u_ref[:, 0])
    assert np.mean(d0 > 0) <= 0.02 and np.all(d0 <= 0.126 * np.abs(u_ref[:, 0]) + 2.0 ** -9)
    # later ranks inherit those differences through the deflation; the approximation they reach is the same
    np.testing.assert_allclose(sigma.cpu().numpy(), s_ref, rtol=2e-2)
    rem_ref = w.astype(np.float64) - (u_ref * s_ref[None, :]) @ v_ref
    assert abs(np.linalg.norm(wd.cpu().numpy()) / np.linalg.norm(rem_ref) - 1.0) <= 5e-3


def _effective_error(w, q, perm, g, b_i, b_h, lowrank):
    """|| W - (low-rank part + Q(R') Q^T P^T) ||_F / || W ||_F of a quantized record, evaluated by the oracle."""
    a, b = lowrank
    w_eff = o.effective_weight(q["codes"], q["scales"], q["zeros"], perm, a, b, g, b_i, b_h)
    return np.linalg.norm(w_eff - w) / np.linalg.norm(w)


def _gpu_record(out, fp8):
    rec = dict(codes=out["codes"].cpu().numpy(), scales=_f16(out["scales"]), zeros=_f16(out["zeros"]))
    if fp8:
        u = o.e4m3_bits_to_f64(out["U"].cpu().numpy())
        v = o.e4m3_bits_to_f64(out["V"].cpu().numpy())
        sig, s = _f16(out["sigma"]), _f16(out["s"])
        return rec, (u * sig[None, :], v / s[None, :]), dict(U=u, V=v, sigma=sig, s=s)
    a, b = _f16(out["A"]), _f16(out["B"])
    return rec, (a, b), dict(A=a, B=b)


@pytest.mark.parametrize("cfg", [dict(n=512, m=512, bits=4, g=128, b=64, r=16, it=8),            # configuration 1
                                 dict(n=1024, m=768, bits=2, g=64, b=256, r=8, it=4),
                                 dict(n=768, m=256, bits=3, g=64, b=128, r=0, it=0)])
def test_quantize_layer_folded_record_against_the_oracle(cfg):
    n, m, bits, g, b, r, it = (cfg[k] for k in ("n", "m", "bits", "g", "b", "r", "it"))
    d = lopro.make_desc(n, m, bits, g, b, rank=r)
    w = synth.weights(m, n, seed=n, spikes=r + 4 if r else 0)
    perm = synth.permutation(n, seed=n + 2)
    sk = synth.sketches(max(r, 1), n, seed=3).astype(np.float32)
    out = lopro.quantize_layer(d, _dev(w), _dev(perm), _dev(sk) if r else None, it=it)
    torch.cuda.synchronize()
    assert lopro.workspace_status(out["workspace"]) == lopro.OK
    ref = o.lopro_quantize(w.astype(np.float64), perm, b, b, r, bits, g, method="r1svd", it=it, sketches=sk.astype(np.float64))
    rec, lowrank, fac = _gpu_record(out, fp8=False) if r else (dict(codes=out["codes"].cpu().numpy(), scales=_f16(out["scales"]),
                                                                    zeros=_f16(out["zeros"])), (np.zeros((m, 0)), np.zeros((0, n))), {})
    if r:
        # fp16 factors: equal except where fp32 and fp64 intermediate values fall on different sides of an fp16 boundary
        assert np.mean(fac["A"] != ref["A"]) <= 0.02 and np.max(np.abs(fac["A"] - ref["A"])) <= 2.0 ** -10 * np.abs(ref["A"]).max()
        assert np.mean(fac["B"] != ref["B"]) <= 0.02 and np.max(np.abs(fac["B"] - ref["B"])) <= 2.0 ** -10 * np.abs(ref["B"]).max()
    # the grid: steps equal up to one fp16 ulp, codes equal up to one level, and nearly all of them identical
    assert np.mean(rec["scales"] != ref["scales"]) <= 0.02
    assert np.max(np.abs(rec["scales"] - ref["scales"]) / ref["scales"]) <= 2.0 ** -10
    dc = np.abs(rec["codes"].astype(np.int32) - ref["codes"].astype(np.int32))
    assert dc.max() <= 1 and np.mean(dc != 0) <= (0.01 if r else 1e-4)
    # what matters: the record reproduces W as well as the oracle's does
    e_gpu = _effective_error(w.astype(np.float64), rec, perm, g, b, b, lowrank)
    e_ref = _effective_error(w.astype(np.float64), ref, perm, g, b, b, (ref["A"], ref["B"]))
    assert abs(e_gpu / e_ref - 1.0) <= 5e-3


def test_quantize_layer_paper_format_record_then_pack_and_forward():
    # Algorithm 1's record (U, V fp8; Sigma, s fp16) produced on the GPU, packed, and run through the forward: the output
    # approximates W x as well as the oracle's record does.
    n, m, bits, g, b, r, it, T = 512, 512, 4, 128, 64, 16, 8, 8
    d = lopro.make_desc(n, m, bits, g, b, rank=r, lowrank_format=lopro.LOWRANK_FP8)
    w = synth.weights(m, n, seed=4, spikes=20)
    perm = synth.permutation(n, seed=6)
    sk = synth.sketches(r, n, seed=8).astype(np.float32)
    s = np.abs(synth.weights(1, n, seed=10, std=0.5)[0]) + np.float32(0.5)
    out = lopro.quantize_layer(d, _dev(w), _dev(perm), _dev(sk), it=it, s=_dev(s))
    torch.cuda.synchronize()
    assert lopro.workspace_status(out["workspace"]) == lopro.OK
    ref = o.lopro_quantize_unfolded(w.astype(np.float64), perm, b, b, r, bits, g, s.astype(np.float64), it, sk.astype(np.float64))
    rec, lowrank, fac = _gpu_record(out, fp8=True)
    np.testing.assert_array_equal(fac["s"], ref["s"])
    np.testing.assert_allclose(fac["sigma"], ref["sigma"], rtol=2e-2)
    w64 = w.astype(np.float64)
    e_gpu = _effective_error(w64, rec, perm, g, b, b, lowrank)
    e_ref = _effective_error(w64, ref, perm, g, b, b, (ref["U"] * ref["sigma"][None, :], ref["V"] / ref["s"][None, :]))
    assert abs(e_gpu / e_ref - 1.0) <= 2e-2
    blob = lopro.pack_lr8(d, out["codes"], out["scales"], out["zeros"], _dev(perm), out["U"], out["V"], out["sigma"], out["s"])
    x_bits = synth.activations(T, n, seed=12)
    y = lopro.linear_fwd(d, blob, bf16_bits_to_device(x_bits), lopro.OUT_F32)
    torch.cuda.synchronize()
    x64 = o.bf16_bits_to_f64(x_bits)
    exact = x64 @ w64.T
    got = y.cpu().numpy().astype(np.float64)
    # the forward of the GPU's own record against the oracle's forward of the same record
    mine = o.forward_exact_unfolded(x64, rec["codes"], rec["scales"], rec["zeros"], perm, fac["U"], fac["sigma"], fac["V"],
                                    fac["s"], g, b, b)
    assert o.max_rel_err(got, mine) <= 2e-2
    # and against W x: the quantization error of a 4-bit grid, as small as with the oracle's record
    theirs = o.forward_exact_unfolded(x64, ref["codes"], ref["scales"], ref["zeros"], perm, ref["U"], ref["sigma"], ref["V"],
                                      ref["s"], g, b, b)
    err_gpu = np.linalg.norm(got - exact) / np.linalg.norm(exact)
    err_ref = np.linalg.norm(theirs - exact) / np.linalg.norm(exact)
    assert err_gpu <= 1.05 * err_ref + 1e-3


def test_quantize_layer_at_the_size_of_a_decoder_projection():
    # 4096 x 4096, the paper's defaults (rank 16, 8 iterations, 2-bit g64... here 4-bit g128 as in configuration 2)
    n = m = 4096
    bits, g, b, r, it = 4, 128, 128, 16, 8
    d = lopro.make_desc(n, m, bits, g, b, rank=r)
    w = synth.weights(m, n, seed=1, spikes=24)
    perm = synth.permutation(n, seed=2)
    sk = synth.sketches(r, n, seed=3).astype(np.float32)
    out = lopro.quantize_layer(d, _dev(w), _dev(perm), _dev(sk), it=it)
    torch.cuda.synchronize()
    assert lopro.workspace_status(out["workspace"]) == lopro.OK
    ref = o.lopro_quantize(w.astype(np.float64), perm, b, b, r, bits, g, method="r1svd", it=it, sketches=sk.astype(np.float64))
    codes = out["codes"].cpu().numpy()
    dc = np.abs(codes.astype(np.int32) - ref["codes"].astype(np.int32))
    assert dc.max() <= 1 and np.mean(dc != 0) <= 0.01
    assert np.mean(_f16(out["scales"]) != ref["scales"]) <= 0.02
    assert np.mean(_f16(out["A"]) != ref["A"]) <= 0.02 and np.mean(_f16(out["B"]) != ref["B"]) <= 0.02


def test_quantize_argument_errors():
    d = lopro.make_desc(512, 64, 4, 128, 64, rank=4)
    w = torch.zeros((64, 512), dtype=torch.float32, device="cuda")
    perm = _dev(synth.permutation(512, seed=1))
    sk = torch.zeros((4, 512), dtype=torch.float32, device="cuda")
    with pytest.raises(lopro.LoproError) as e:
        lopro.quantize_layer(d, w, perm, sk, workspace=torch.zeros(1024, dtype=torch.uint8, device="cuda"))
    assert e.value.status == lopro.ERR_BUFFER_TOO_SMALL
    with pytest.raises(lopro.LoproError) as e:
        lopro.quantize_layer(d, w, perm, None)                  # rank > 0 needs sketches
    assert e.value.status == lopro.ERR_INVALID_ARG
    with pytest.raises(lopro.LoproError) as e:
        lopro.r1svd(w, 0, 2, sk)
    assert e.value.status == lopro.ERR_INVALID_ARG
