"""Pins for the low-rank side of the oracle (Eq. 4, Eq. 10-12, Algorithm 1) and for the
layer quantizer built from it.  CPU only."""
import numpy as np

from oracle import lopro_oracle as o
from paper_2601_19675_b200 import synth


def _rank_k(m, n, k, seed):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((m, k)) @ rng.standard_normal((k, n))


def test_truncated_svd_eckart_young():
    rng = np.random.default_rng(0)
    w = rng.standard_normal((20, 30))
    sv = np.linalg.svd(w, compute_uv=False)
    for r in (1, 4, 20):
        u, s, v = o.svd_lowrank(w, r)
        resid = w - (u * s) @ v
        np.testing.assert_allclose(np.sum(resid ** 2), np.sum(sv[r:] ** 2), rtol=1e-10, atol=1e-20)
        np.testing.assert_allclose(u.T @ u, np.eye(r), atol=1e-12)
        np.testing.assert_allclose(v @ v.T, np.eye(r), atol=1e-12)


def test_lowrank_exact_when_rank_le_r():
    w = _rank_k(24, 40, 3, 1)
    u, s, v = o.svd_lowrank(w, 4)
    np.testing.assert_allclose((u * s) @ v, w, atol=1e-12)
    # R1SVD: every step is a projection deflation (A - U U^T A), so a rank-k matrix is
    # reproduced in k steps for any iteration count and any generic sketch
    for it in (0, 1, 8):
        u, s, v = o.r1svd(w, 4, it, synth.sketches(4, 40, seed=it))
        np.testing.assert_allclose((u * s) @ v, w, atol=1e-9)
        assert s[3] == 0.0 or abs(s[3]) < 1e-9     # fourth component finds nothing left
    # rank-1 matrix in one step
    w1 = _rank_k(10, 12, 1, 2)
    u, s, v = o.r1svd(w1, 1, 0, synth.sketches(1, 12, seed=5))
    np.testing.assert_allclose(s[0] * np.outer(u[:, 0], v[0]), w1, atol=1e-12)


def test_r1svd_step_formulas_eq_10_12():
    # One step against the closed forms of Eq. 12 written out with explicit matrix powers.
    rng = np.random.default_rng(3)
    a = rng.standard_normal((7, 9))
    sk = rng.standard_normal((1, 9))
    it = 2
    u, s, v = o.r1svd(a, 1, it, sk)
    big = np.linalg.matrix_power(a @ a.T, it) @ a @ sk[0]
    row = sk[0] @ a.T @ np.linalg.matrix_power(a @ a.T, it) @ a
    np.testing.assert_allclose(u[:, 0], big / np.linalg.norm(big), atol=1e-12)
    np.testing.assert_allclose(v[0], row / np.linalg.norm(row), atol=1e-12)
    np.testing.assert_allclose(s[0], np.linalg.norm(row) / np.linalg.norm(big), rtol=1e-12)
    # deflation is the projection (I - U U^T) A
    resid = a - s[0] * np.outer(u[:, 0], v[0])
    np.testing.assert_allclose(resid, a - np.outer(u[:, 0], u[:, 0]) @ a, atol=1e-12)


def test_r1svd_converges_to_top_singular_triple():
    rng = np.random.default_rng(4)
    q1, _ = np.linalg.qr(rng.standard_normal((12, 12)))
    q2, _ = np.linalg.qr(rng.standard_normal((15, 15)))
    sv = np.array([5.0, 2.0, 1.0, 0.5] + [0.1] * 8)
    a = (q1 * sv) @ q2[:12, :]
    u, s, v = o.r1svd(a, 2, 30, synth.sketches(2, 15, seed=1))
    us, ss, vs = o.svd_lowrank(a, 2)
    for j in range(2):
        np.testing.assert_allclose(s[j], ss[j], rtol=1e-8)
        np.testing.assert_allclose(abs(u[:, j] @ us[:, j]), 1.0, atol=1e-8)
        np.testing.assert_allclose(abs(v[j] @ vs[j]), 1.0, atol=1e-8)


def test_r1svd_fp8_cast_is_compensated_by_later_ranks():
    # Sec. 3.3: the precision lost by casting U_1, V_1 is picked up by the following
    # deflation steps, so the residual keeps shrinking with the rank.
    w = _rank_k(32, 48, 6, 6)
    prev = np.linalg.norm(w)
    for r in (2, 4, 8):
        u, s, v = o.r1svd(w, r, 4, synth.sketches(r, 48, seed=2), cast=o.round_e4m3)
        assert np.all(o.round_e4m3(u) == u) and np.all(o.round_e4m3(v) == v)
        res = np.linalg.norm(w - (u * s) @ v)
        assert res < prev
        prev = res


def test_scaled_svd_folding_eq4():
    # W_r = (U Sigma)(V alpha^-1) approximates W itself, with the error weighted by alpha.
    rng = np.random.default_rng(8)
    w = _rank_k(16, 24, 2, 8)
    alpha = rng.uniform(0.5, 2.0, size=24)
    u, s, v = o.svd_lowrank(w * alpha, 2)
    np.testing.assert_allclose((u * s) @ (v / alpha), w, atol=1e-12)


def test_lopro_quantize_layer_reconstruction_and_forward():
    m, n, T = 64, 256, 4
    w = synth.weights(m, n, seed=0).astype(np.float64)
    # plant a rank-2 component so that the low-rank branch has something to catch
    w += 0.05 * _rank_k(m, n, 2, 9) / np.sqrt(n)
    perm = synth.permutation(n, seed=0)
    x = o.bf16_bits_to_f64(synth.activations(T, n, seed=0))
    errs = {}
    for bits in (2, 3, 4):
        L = o.lopro_quantize(w, perm, 64, 64, 4, bits, 64)
        w_eff = o.effective_weight(L["codes"], L["scales"], L["zeros"], perm, L["A"], L["B"], 64, 64, 64)
        errs[bits] = np.linalg.norm(w_eff - w) / np.linalg.norm(w)
        y = o.forward_exact(x, L["codes"], L["scales"], L["zeros"], perm, L["A"], L["B"], 64, 64, 64)
        np.testing.assert_allclose(y, x @ w_eff.T, atol=1e-10)
        assert np.all(o.round_f16(L["A"]) == L["A"]) and np.all(o.round_f16(L["scales"]) == L["scales"])
        # Q is orthogonal, so the weight error equals the quantisation error of R'
        resid = w - L["A"] @ L["B"]
        rp = o.partial_block_rotate(o.permute_columns(resid, perm), 64, 64)
        qerr = np.linalg.norm(o.dequant(L["codes"], L["scales"], L["zeros"], 64) - rp)
        np.testing.assert_allclose(np.linalg.norm(w_eff - w), qerr, rtol=1e-9)
    assert errs[4] < errs[3] < errs[2] < 0.5
    # r1svd route gives a layer of comparable quality
    L2 = o.lopro_quantize(w, perm, 64, 64, 4, 4, 64, method="r1svd", it=8, sketches=synth.sketches(4, n, seed=0))
    w2 = o.effective_weight(L2["codes"], L2["scales"], L2["zeros"], perm, L2["A"], L2["B"], 64, 64, 64)
    assert np.linalg.norm(w2 - w) / np.linalg.norm(w) < 1.2 * errs[4]


def test_synth_generators_are_seeded_and_typed():
    a1 = synth.activations(3, 64, seed=1, outlier_frac=0.05)
    a2 = synth.activations(3, 64, seed=1, outlier_frac=0.05)
    np.testing.assert_array_equal(a1, a2)
    assert a1.dtype == np.uint16 and synth.permutation(8).dtype == np.int32
    assert not np.array_equal(a1, synth.activations(3, 64, seed=2, outlier_frac=0.05))
    # the generator's bf16 conversion agrees with the oracle's own rounding
    x = np.random.default_rng(0).standard_normal(1000).astype(np.float32)
    np.testing.assert_array_equal(o.bf16_bits_to_f64(synth.f32_to_bf16_bits(x)), o.round_bf16(x.astype(np.float64)))
    L = synth.random_layer(**{k: v for k, v in synth.CONFIGS["cfg1"].items() if k != "T"})
    assert L["codes"].max() == 15 and o.is_permutation(L["perm"])
    s = o.f16_bits_to_f64(L["scales"])
    assert s.min() >= 0.005 - 1e-5 and s.max() <= 0.02 + 1e-5


def _unfolded_layer(seed, m=8, n=32, g=8, bits=3, b_i=8, b_h=8, r=3, T=4, dyadic=False):
    rng = np.random.default_rng(seed)
    codes = rng.integers(0, 2 ** bits, size=(m, n)).astype(np.uint8)
    scales = o.round_f16(rng.uniform(0.01, 0.1, size=(m, n // g)))
    zeros = o.round_f16(rng.uniform(0, 2 ** bits - 1, size=(m, n // g)))
    perm = rng.permutation(n).astype(np.int32)
    if dyadic:   # every product and sum below is exact in fp64
        u = rng.integers(-8, 9, size=(m, r)) / 8.0
        v = rng.integers(-8, 9, size=(r, n)) / 8.0
        sigma = 2.0 ** rng.integers(-2, 3, size=r)
        s = 2.0 ** rng.integers(-1, 2, size=n)
        x = rng.integers(-16, 17, size=(T, n)) / 4.0
    else:
        u = o.round_e4m3(rng.standard_normal((m, r)) / np.sqrt(m))
        v = o.round_e4m3(rng.standard_normal((r, n)) / np.sqrt(n))
        sigma = o.round_f16(rng.uniform(0.5, 2.0, size=r))
        s = o.round_f16(rng.uniform(0.5, 2.0, size=n))
        x = o.round_bf16(rng.standard_normal((T, n)))
    return dict(x=x, codes=codes, scales=scales, zeros=zeros, perm=perm, u=u, sigma=sigma, v=v, s=s, g=g, b_i=b_i, b_h=b_h)


def _folded(L):
    F = {k: L[k] for k in ("x", "codes", "scales", "zeros", "perm", "g", "b_i", "b_h")}
    F["a"] = L["u"] * L["sigma"][None, :]             # W_L = U Sigma
    F["b"] = L["v"] / L["s"][None, :]                 # W_R = V alpha^-1, alpha = diag(s)  (Eq. 4)
    return F


def test_unfolded_forward_equals_the_folded_one_on_exact_factors():
    # with dyadic factors U Sigma and V / s are exact, so the stored form of Algorithm 1's record and the folded form
    # of Eq. 4 describe the same numbers and every partial sum is exact: the low-rank parts must agree bit for bit
    L = _unfolded_layer(5, dyadic=True)
    F = _folded(L)
    zero_q = dict(L, codes=np.zeros_like(L["codes"]), zeros=np.zeros_like(L["zeros"]))
    zero_f = dict(F, codes=np.zeros_like(F["codes"]), zeros=np.zeros_like(F["zeros"]))
    np.testing.assert_array_equal(o.forward_exact_unfolded(**zero_q), o.forward_exact(**zero_f))
    np.testing.assert_allclose(o.forward_exact_unfolded(**L), o.forward_exact(**F), rtol=0, atol=1e-12)


def test_unfolded_forward_equals_dense_eq8():
    # Eq. 8 literally: W_eff = U Sigma V diag(s)^-1 + W^ Q^T P^T, y = W_eff x
    L = _unfolded_layer(6)
    n = L["x"].shape[1]
    w_hat = o.dequant(L["codes"], L["scales"], L["zeros"], L["g"])
    w_eff = L["u"] @ np.diag(L["sigma"]) @ L["v"] @ np.diag(1.0 / L["s"]) \
        + w_hat @ o.q_matrix(n, L["b_i"], L["b_h"]).T @ o.p_matrix(L["perm"]).T
    np.testing.assert_allclose(o.forward_exact_unfolded(**L), L["x"] @ w_eff.T, atol=1e-12)
    # the mirrored variant differs only by its declared roundings, and with none left (rotation off, no t rounding)
    # it is the fp32 rounding of the exact result
    Li = dict(L, b_i=n)
    np.testing.assert_array_equal(o.forward_mirrored_unfolded(**Li, round_t="none"),
                                  o.forward_exact_unfolded(**Li).astype(np.float32).astype(np.float64))
    e = o.max_rel_err(o.forward_mirrored_unfolded(**L), o.forward_exact_unfolded(**L))
    assert 0.0 < e < 2e-2


def test_e4m3_bit_patterns_round_trip_and_match_the_library_cast():
    import torch
    allbits = np.arange(256, dtype=np.uint8)
    finite = allbits[(allbits & 0x7F) != 0x7F]                       # 0x7F / 0xFF are NaN in the finite-only format
    vals = o.e4m3_bits_to_f64(finite)
    ref = torch.from_numpy(finite.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    np.testing.assert_array_equal(vals, ref)
    back = o.f64_to_e4m3_bits(vals)
    np.testing.assert_array_equal(back & 0x7F, finite & 0x7F)        # (the sign of zero aside, covered below)
    np.testing.assert_array_equal(o.e4m3_bits_to_f64(back), vals)
    np.testing.assert_array_equal(o.round_e4m3(vals), vals)          # representable values are fixed points


def test_unfolded_quantizer_absorbs_the_fp8_rounding_in_the_residual():
    # Algorithm 1 with the casts of Sec. 3.3: the quantized part sees R = W - U Sigma V / s with the STORED factors,
    # so the layer reproduces W up to the RTN grid alone (same bound as with exact factors)
    rng = np.random.default_rng(8)
    m, n, r, g, bits = 32, 64, 4, 16, 4
    w = rng.standard_normal((m, n)) * 0.05
    s = rng.uniform(0.5, 2.0, size=n)
    perm = rng.permutation(n).astype(np.int32)
    q = o.lopro_quantize_unfolded(w, perm, 16, 16, r, bits, g, s, it=4, sketches=rng.standard_normal((r, n)))
    np.testing.assert_array_equal(o.round_e4m3(q["U"]), q["U"])
    np.testing.assert_array_equal(o.round_e4m3(q["V"]), q["V"])
    np.testing.assert_array_equal(o.round_f16(q["sigma"]), q["sigma"])
    x = np.eye(n)
    w_back = o.forward_exact_unfolded(x, q["codes"], q["scales"], q["zeros"], perm, q["U"], q["sigma"], q["V"], q["s"], g, 16, 16).T
    resid = w - (q["U"] * q["sigma"][None, :]) @ (q["V"] / q["s"][None, :])
    rp = o.partial_block_rotate(o.permute_columns(resid, perm), 16, 16)
    step = np.repeat(q["scales"], g, axis=1)
    err_rot = o.partial_block_rotate(o.permute_columns(w - w_back, perm), 16, 16)   # error in the rotated basis
    assert np.all(np.abs(err_rot) <= 0.5 * step + 1e-3 * np.abs(rp).max())
    # and the low-rank part carries most of the weight of the leading directions: the residual is smaller than W
    assert np.linalg.norm(resid) < np.linalg.norm(w)
