"""Pins for the quantized part and the forward of the oracle (Eq. 8, Eq. 13, Appendix
A.2/A.3): dense-matrix evaluation, brute-force loops, the zero-quantization-error
construction, packing, size accounting, and the hand-written rounding helpers
against independent library casts.  CPU only."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import lopro_oracle as o


def _tiny_layer(seed, m=6, n=16, g=8, bits=3, b_i=4, b_h=4, r=2, T=3):
    rng = np.random.default_rng(seed)
    codes = rng.integers(0, 2 ** bits, size=(m, n)).astype(np.uint8)
    scales = o.round_f16(rng.uniform(0.01, 0.1, size=(m, n // g)))
    zeros = o.round_f16(rng.uniform(0, 2 ** bits - 1, size=(m, n // g)))
    perm = rng.permutation(n).astype(np.int32)
    a = o.round_f16(rng.standard_normal((m, r)) * 0.1)
    b = o.round_f16(rng.standard_normal((r, n)) * 0.1)
    x = o.round_bf16(rng.standard_normal((T, n)))
    return dict(x=x, codes=codes, scales=scales, zeros=zeros, perm=perm, a=a, b=b, g=g, b_i=b_i, b_h=b_h)


def _bruteforce_forward(L):
    """Eq. 8 with scalar Python loops only (no numpy linear algebra)."""
    x, codes, scales, zeros, perm = L["x"], L["codes"], L["scales"], L["zeros"], L["perm"]
    a, b, g, b_i, b_h = L["a"], L["b"], L["g"], L["b_i"], L["b_h"]
    T, n = x.shape
    m = codes.shape[0]
    r = a.shape[1]
    y = [[0.0] * m for _ in range(T)]
    for t in range(T):
        xp = [float(x[t][int(perm[k])]) for k in range(n)]
        xt = list(xp)
        for s in range(b_i, n, b_h):
            for i in range(b_h):
                acc = 0.0
                for j in range(b_h):
                    sign = -1.0 if bin(i & j).count("1") & 1 else 1.0
                    acc += sign * xp[s + j]
                xt[s + i] = acc / math.sqrt(b_h)
        tt = [sum(float(b[j][k]) * float(x[t][k]) for k in range(n)) for j in range(r)]
        for i in range(m):
            acc = 0.0
            for k in range(n):
                w = float(scales[i][k // g]) * (float(codes[i][k]) - float(zeros[i][k // g]))
                acc += w * xt[k]
            for j in range(r):
                acc += float(a[i][j]) * tt[j]
            y[t][i] = acc
    return np.array(y)


@pytest.mark.parametrize("seed,kw", [(0, {}), (1, dict(bits=2, b_i=0, b_h=8, g=4)), (2, dict(bits=4, b_i=8, b_h=8, r=3)),
                                     (3, dict(n=32, g=16, b_i=16, b_h=16, r=0))])
def test_forward_exact_equals_dense_and_bruteforce(seed, kw):
    L = _tiny_layer(seed, **kw)
    y = o.forward_exact(**L)
    np.testing.assert_allclose(y, o.forward_dense(**L), atol=1e-12)
    np.testing.assert_allclose(y, _bruteforce_forward(L), atol=1e-12)
    Lw = {k: v for k, v in L.items() if k != "x"}
    np.testing.assert_allclose(y, L["x"] @ o.effective_weight(**Lw).T, atol=1e-12)


def test_forward_invariant_under_consistent_relabelling():
    # Renaming the input channels (x and the rows of B permuted by sigma, perm composed
    # with sigma^-1) must not change y: the layer only ever sees x through perm and B.
    L = _tiny_layer(7)
    n = L["x"].shape[1]
    rng = np.random.default_rng(70)
    sigma = rng.permutation(n)
    inv_sigma = o.invert_permutation(sigma)
    L2 = dict(L)
    L2["x"] = L["x"][:, sigma]                      # x'[j] = x[sigma[j]]
    L2["b"] = L["b"][:, sigma]
    L2["perm"] = inv_sigma[L["perm"]]                # x'[perm'[k]] = x[perm[k]]
    np.testing.assert_allclose(o.forward_exact(**L2), o.forward_exact(**L), atol=1e-12)


def test_forward_reduces_to_plain_matmul_when_nothing_is_rotated():
    # b_I = n and identity perm: Q = I, P = I, so y = x (W^ + A B)^T, a textbook product.
    L = _tiny_layer(9, b_i=16, b_h=4)
    L["perm"] = np.arange(16, dtype=np.int32)
    w_hat = o.dequant(L["codes"], L["scales"], L["zeros"], L["g"])
    np.testing.assert_allclose(o.forward_exact(**L), L["x"] @ (w_hat + L["a"] @ L["b"]).T, atol=1e-12)


def test_dequant_bruteforce_all_codes():
    for bits in (2, 3, 4):
        for s, z in [(0.0123, 0.0), (0.5, 3.0), (0.0078125, 2.5), (1.5, 7.25)]:
            codes = np.arange(2 ** bits, dtype=np.uint8)[None, :]
            g = 2 ** bits
            w = o.dequant(codes, [[s]], [[z]], g)
            for c in range(2 ** bits):
                assert w[0, c] == s * (c - z)
    # group indexing: second group uses the second scale/zero
    w = o.dequant(np.array([[1, 1, 1, 1]], dtype=np.uint8), [[1.0, 2.0]], [[0.0, 3.0]], 2)
    np.testing.assert_array_equal(w, [[1.0, 1.0, -4.0, -4.0]])


def test_zero_quantization_error_reconstructs_w_exactly():
    # Dyadic construction: power-of-two scales, integer zeros, every group holds code 0 and
    # code 2^q - 1, b_H in {4, 16, 64} so that 1/sqrt(b_H) is dyadic: all arithmetic exact.
    rng = np.random.default_rng(11)
    for bits, b_h, g, n, b_i in [(4, 4, 8, 24, 8), (2, 16, 16, 64, 16), (3, 64, 32, 192, 64), (4, 16, 8, 48, 0)]:
        m, r = 8, 2
        qmax = 2 ** bits - 1
        codes = rng.integers(0, qmax + 1, size=(m, n)).astype(np.uint8)
        codes.reshape(m, n // g, g)[:, :, 0] = 0
        codes.reshape(m, n // g, g)[:, :, 1] = qmax
        scales = 2.0 ** rng.integers(-6, -2, size=(m, n // g))
        zeros = rng.integers(0, qmax + 1, size=(m, n // g)).astype(np.float64)
        perm = rng.permutation(n).astype(np.int32)
        a = rng.integers(-4, 5, size=(m, r)) / 8.0
        b = rng.integers(-4, 5, size=(r, n)) / 8.0
        w = o.effective_weight(codes, scales, zeros, perm, a, b, g, b_i, b_h)
        # quantize the residual against the same (exactly representable) factors
        resid = w - a @ b
        rp = o.partial_block_rotate(o.permute_columns(resid, perm), b_i, b_h)
        np.testing.assert_array_equal(rp, o.dequant(codes, scales, zeros, g))   # R' recovered exactly
        for dtype in (np.float64, np.float32):      # every operation is exact here, so the precision cannot matter
            c2, s2, z2 = o.rtn_quantize(rp, bits, g, dtype=dtype)
            np.testing.assert_array_equal(c2, codes)
            np.testing.assert_array_equal(s2, scales)
            np.testing.assert_array_equal(z2, zeros)
        w2 = o.effective_weight(c2, s2, z2, perm, a, b, g, b_i, b_h)
        assert np.max(np.abs(w2 - w)) == 0.0


def test_rtn_error_bound_and_degenerate_groups():
    rng = np.random.default_rng(12)
    v = rng.standard_normal((16, 64)) * 0.02
    for bits in (2, 3, 4):
        codes, s, z = o.rtn_quantize(v, bits, 32)
        assert codes.max() <= 2 ** bits - 1
        err = np.abs(o.dequant(codes, s, z, 32) - v)
        # half a step plus the fp16 rounding of the step (relative 2^-11 over <= 2^q steps)
        bound = np.repeat(s, 32, axis=1) * (0.5 + 2.0 ** -11 * 2 ** bits + 1e-9)
        assert np.all(err <= bound)
    # constant groups dequantize to the constant (positive, negative, zero)
    for c in (0.25, -0.25, 0.0):
        codes, s, z = o.rtn_quantize(np.full((1, 8), c), 4, 8)
        np.testing.assert_array_equal(o.dequant(codes, s, z, 8), np.full((1, 8), c))


def test_rtn_precision_switch_worked_by_hand():
    # 2-bit group {2^-30, 3t, a, 1/2} with t = 1 + 3/2048, the midpoint of the fp16 neighbours 1 + 1/1024 and 1 + 2/1024.
    # Double precision: hi - lo = 3t - 2^-30 exactly, a third of it lies just below t, so the step rounds DOWN to
    # 1 + 1/1024.  Single precision: 2^-30 is far below half an ulp of 3t (2^-23), the difference rounds to 3t, the
    # quotient is t itself, and the tie goes to the even mantissa, 1 + 2/1024.  a = 1 + 1029/2048 then lands on
    # a / step = 1.50098 (code 2) in double and 1.49951 (code 1) in single; the zero-point is rne(-2^-30 / step) = 0.
    t = 1.0 + 3.0 / 2048.0
    a = 1.0 + 1029.0 / 2048.0
    v = np.array([[2.0 ** -30, 3.0 * t, a, 0.5]])
    assert np.all(v.astype(np.float32).astype(np.float64) == v)          # the inputs are single-precision numbers
    c64, s64, z64 = o.rtn_quantize(v, 2, 4)
    c32, s32, z32 = o.rtn_quantize(v, 2, 4, dtype=np.float32)
    assert s64[0, 0] == 1.0 + 1.0 / 1024.0 and s32[0, 0] == 1.0 + 2.0 / 1024.0
    assert z64[0, 0] == 0.0 and z32[0, 0] == 0.0
    np.testing.assert_array_equal(c64, [[0, 3, 2, 0]])
    np.testing.assert_array_equal(c32, [[0, 3, 1, 0]])


def test_pack_canonical_bit_stream():
    # 4-bit: word = sum_j c_j 16^j, low nibble first
    c = np.array([[1, 2, 3, 4, 5, 6, 7, 8]], dtype=np.uint8)
    assert o.pack_canonical(c, 4)[0, 0] == sum(int(v) << (4 * j) for j, v in enumerate(c[0]))
    assert o.pack_canonical(c, 4)[0, 0] == 0x87654321
    # independent check through Python big integers for every bit width, with straddling 3-bit codes
    rng = np.random.default_rng(13)
    for bits in (2, 3, 4):
        codes = rng.integers(0, 2 ** bits, size=(3, 64)).astype(np.uint8)
        words = o.pack_canonical(codes, bits)
        assert words.dtype == np.uint32 and words.shape == (3, 64 * bits // 32)
        for i in range(3):
            big = sum(int(v) << (bits * k) for k, v in enumerate(codes[i]))
            ref = [(big >> (32 * w)) & 0xFFFFFFFF for w in range(64 * bits // 32)]
            assert [int(t) for t in words[i]] == ref
        np.testing.assert_array_equal(o.unpack_canonical(words, bits, 64), codes)
    # walking one: code k = 1 sets exactly bit k*q
    for bits in (2, 3, 4):
        for k in (0, 5, 10, 11, 21, 31):
            codes = np.zeros((1, 32), dtype=np.uint8)
            codes[0, k] = 1
            words = o.pack_canonical(codes, bits)
            pos = k * bits
            expect = np.zeros(32 * bits // 32, dtype=np.uint32)
            expect[pos // 32] = 1 << (pos % 32)
            np.testing.assert_array_equal(words[0], expect)
    with pytest.raises(ValueError):
        o.pack_canonical(np.array([[4] * 16], dtype=np.uint8), 2)


def _golden_bits(golden_dir):
    out = {}
    with open(os.path.join(golden_dir, "avg_bits.txt")) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                k, v, tol, _src = line.split()
                out[k] = (float(v), float(tol))
    return out


def test_size_accounting_reproduces_printed_figures(golden_dir):
    gold = _golden_bits(golden_dir)
    shapes = {"7b": [(4096, 4096)] * 4 + [(11008, 4096)] * 2 + [(4096, 11008)],
              "13b": [(5120, 5120)] * 4 + [(13824, 5120)] * 2 + [(5120, 13824)]}
    for model, sh in shapes.items():
        for r in (8, 16, 32, 64):
            val, tol = gold[f"rbit_{model}_r{r}"]
            assert abs(o.lowrank_bits(sh, r, 8) - val) <= tol
    for q in (2, 3):
        val, tol = gold[f"bits_gptq_{q}"]
        assert abs((q + 16 / 128) - val) <= tol
        assert abs(o.average_bits(10 ** 9, 10 ** 9, q, 16, 128, 0, 8) - val) <= tol
        val, tol = gold[f"bits_lopro_{q}"]
        assert abs(q + 16 / 128 + o.lowrank_bits(shapes["7b"], 16, 8) - val) <= tol
    # Eq. 13 term by term on a square layer
    m = n = 4096
    d = o.average_bits(m, n, 2, 16, 128, 16, 8)
    assert abs(d - (2 + 16 / 128 + 16 * 8 / n + 16 * 8 / m + 2 * 16 / n + 16 * 16 / (m * n))) < 1e-15
    # for one matrix the U, V terms of Eq. 13 equal the parameter-weighted formula
    assert abs(o.lowrank_bits([(m, n)], 16, 8) - (16 * 8 / n + 16 * 8 / m)) < 1e-15


def test_rounding_helpers_against_library_casts():
    rng = np.random.default_rng(14)
    x = np.concatenate([rng.standard_normal(20000) * 10.0 ** rng.integers(-9, 5, size=20000),
                        [0.0, 1.0, -1.0, 65504.0, 65519.9, 65520.0, 1e-8, 2.0 ** -24, 2.0 ** -25, 3 * 2.0 ** -25,
                         1.00390625, 1.01171875, 256.5, 257.5]])
    with np.errstate(over="ignore"):
        np.testing.assert_array_equal(o.round_f16(x), x.astype(np.float16).astype(np.float64))
    xb = x[np.abs(x) < 1e30]
    # torch casts fp64 -> bf16 directly (one rounding)
    ref_bf16 = torch.from_numpy(xb).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(o.round_bf16(xb), ref_bf16)
    np.testing.assert_array_equal(o.round_f32(x), x.astype(np.float32).astype(np.float64))
    x8 = np.concatenate([rng.uniform(-1, 1, 5000), rng.standard_normal(5000) * 50, [0.0, 448.0, 2.0 ** -9, 2.0 ** -10,
                                                                                 3 * 2.0 ** -10, 0.0146484375]])
    x8 = x8[np.abs(x8) <= 448.0]
    ref8 = torch.from_numpy(x8).to(torch.float32).to(torch.float8_e4m3fn).to(torch.float64).numpy()
    x8_single = x8.astype(np.float32).astype(np.float64)   # torch's cast starts from fp32
    np.testing.assert_array_equal(o.round_e4m3(x8_single), ref8)
    # bit-pattern decoders
    assert o.bf16_bits_to_f64(np.array([0x3F80, 0xC000, 0x4300], dtype=np.uint16)).tolist() == [1.0, -2.0, 128.0]
    assert o.f16_bits_to_f64(np.array([0x3C00, 0xC000, 0x7BFF], dtype=np.uint16)).tolist() == [1.0, -2.0, 65504.0]
    np.testing.assert_array_equal(o.f64_to_bf16_bits(np.array([1.0, -2.0, 128.0])), [0x3F80, 0xC000, 0x4300])
    np.testing.assert_array_equal(o.f64_to_f16_bits(np.array([1.0, -2.0, 65504.0])), [0x3C00, 0xC000, 0x7BFF])


def test_mirrored_close_to_exact_and_roundings_are_visible():
    L = _tiny_layer(21, m=32, n=256, g=64, bits=4, b_i=64, b_h=64, r=4, T=8)
    y = o.forward_exact(**L)
    for kw in (dict(), dict(round_w=True), dict(out="bf16"), dict(round_t="bf16", round_w=True, out="bf16")):
        ym = o.forward_mirrored(**L, **kw)
        e = o.max_rel_err(ym, y)
        assert 0.0 < e < 2e-2, (kw, e)     # declared roundings stay inside the bf16 gate
    # the mirrored fp32 path differs from exact only at rounding level
    assert o.max_rel_err(o.forward_mirrored(**L), y) < 1e-2


def test_max_rel_err_definition():
    y_ref = np.array([[3.0, 4.0, 0.0, 0.0]])      # rms = 2.5
    y = np.array([[3.3, 4.0, 0.25, 0.0]])
    # |0.3| / 3 = 0.1 ; |0.25| / max(0, 2.5) = 0.1
    assert abs(o.max_rel_err(y, y_ref) - 0.1) < 1e-12


def _lib_bf16(a):
    """fp64 -> bf16 values by torch's cast (independent of the oracle's rounding helpers)."""
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float64)).to(torch.bfloat16).to(torch.float64).numpy()


def _mirrored_by_hand(L, round_w, round_t, out):
    """Eq. 8 with the declared roundings written out step by step: explicit dense P and Q, scalar loops for the
    dequantization, library casts (torch bfloat16, numpy float16 / float32) for every rounding."""
    x, codes, scales, zeros, perm = L["x"], L["codes"], L["scales"], L["zeros"], L["perm"]
    a, b, g, b_i, b_h = L["a"], L["b"], L["g"], L["b_i"], L["b_h"]
    T, n = x.shape
    m = codes.shape[0]
    p = np.zeros((n, n))
    for k in range(n):
        p[int(perm[k]), k] = 1.0                       # (x P)[k] = x[perm[k]]
    q = np.zeros((n, n))
    for k in range(b_i):
        q[k, k] = 1.0
    for s in range(b_i, n, b_h):
        for i in range(b_h):
            for j in range(b_h):
                q[s + i, s + j] = (-1.0 if bin(i & j).count("1") & 1 else 1.0) / math.sqrt(b_h)
    xt = _lib_bf16(x @ p @ q)                          # rotated activations, stored as bf16
    w = np.zeros((m, n))
    for i in range(m):
        for k in range(n):
            w[i, k] = float(scales[i, k // g]) * (float(codes[i, k]) - float(zeros[i, k // g]))
    if round_w:
        w = _lib_bf16(w.astype(np.float32).astype(np.float64))   # fp32 product, then one rounding to bf16
    t = x @ b.T
    if round_t == "f16":
        t = t.astype(np.float16).astype(np.float64)
    elif round_t == "bf16":
        t = _lib_bf16(t)
    y = xt @ w.T + t @ a.T
    return _lib_bf16(y) if out == "bf16" else y.astype(np.float32).astype(np.float64)


@pytest.mark.parametrize("round_w", [False, True])
@pytest.mark.parametrize("round_t", ["f16", "bf16", "none"])
@pytest.mark.parametrize("out", ["f32", "bf16"])
def test_forward_mirrored_equals_the_steps_written_out(round_w, round_t, out):
    # every product and partial sum of this tiny layer is exact in fp64 (8-bit activations, 11-bit scales and
    # factors, a narrow exponent range), so the two evaluations may differ in nothing but a misplaced rounding
    L = _tiny_layer(31, m=8, n=64, g=16, bits=4, b_i=16, b_h=16, r=3, T=5)
    got = o.forward_mirrored(**L, round_w=round_w, round_t=round_t, out=out)
    np.testing.assert_array_equal(got, _mirrored_by_hand(L, round_w, round_t, out))


def test_each_switch_of_forward_mirrored_touches_only_the_operand_it_names():
    L = _tiny_layer(32, m=8, n=64, g=16, bits=4, b_i=16, b_h=16, r=3, T=5)
    base = o.forward_mirrored(**L, round_w=False, round_t="none", out="f32")
    # weights that are bf16 values already (power-of-two scales, integer zero-points): round_w changes nothing,
    # while with generic fp16 scales it does
    Lp = dict(L)
    Lp["scales"] = np.full_like(L["scales"], 2.0 ** -5)
    Lp["zeros"] = np.rint(L["zeros"])
    np.testing.assert_array_equal(o.forward_mirrored(**Lp, round_w=True, round_t="none"),
                                  o.forward_mirrored(**Lp, round_w=False, round_t="none"))
    assert not np.array_equal(o.forward_mirrored(**L, round_w=True, round_t="none"), base)
    # no low-rank branch: round_t changes nothing; with one it does, and by exactly A (round(t) - t)
    L0 = dict(L)
    L0["a"], L0["b"] = np.zeros((8, 0)), np.zeros((0, 64))
    np.testing.assert_array_equal(o.forward_mirrored(**L0, round_t="f16"), o.forward_mirrored(**L0, round_t="none"))
    t = L["x"] @ L["b"].T
    d_t = (t.astype(np.float16).astype(np.float64) - t) @ L["a"].T
    full = o.forward_mirrored(**L, round_w=False, round_t="f16", out="f32")
    np.testing.assert_allclose(full - base, d_t, atol=2e-6)       # both sides carry one fp32 rounding of y
    assert np.abs(d_t).max() > 0.0
    # activations: always rounded -- x~ that is bf16 already (rotation off, b_I = n) makes mirrored == exact
    Li = dict(L)
    Li["b_i"] = 64
    y_exact = o.forward_exact(**Li)
    np.testing.assert_array_equal(o.forward_mirrored(**Li, round_t="none"), y_exact.astype(np.float32).astype(np.float64))
    # out: the bf16 result is one rounding of the fp64 sum, not of the fp32 result
    np.testing.assert_array_equal(o.forward_mirrored(**Li, round_t="none", out="bf16"), _lib_bf16(y_exact))
