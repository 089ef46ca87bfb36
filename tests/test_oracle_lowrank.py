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
