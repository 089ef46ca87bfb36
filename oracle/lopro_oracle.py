"""Plain fp64 oracle of the LoPRo quantize-and-forward definitions.

TEST INFRASTRUCTURE ONLY -- never imported by the CUDA library or its binding.

Notation follows the paper: W in R^{m x n} (m = d_out, n = d_in), X holds one
token per row here (the paper writes tokens as columns of X in R^{n x b}),
W_r = A B the rank-r part (A = U Sigma, B = V alpha^-1, Eq. 4), R = W - W_r the
residual, P the permutation matrix built from the index vector `perm`, Q the
partial block Walsh-Hadamard matrix (Eq. 6), Qz(.) the group quantizer, and

    W X = W_r X + Qz(R') Q^T P^T X,      R' = R P Q            (Eq. 8, Eq. 6)

Every function states the passage it follows.  Nothing here is blocked, fused
or reordered beyond what the cited definition states.

Readings taken where the paper is silent or inconsistent:
  * permutation direction: gather, (P^T x)[k] = x[perm[k]], i.e. P[perm[k], k] = 1,
    which is the reading under which "sort(...).idx" moves the selected columns
    to the front (Eq. 5 and the sentence after it);
  * Hadamard ordering: the Sylvester/Kronecker recursion of Eq. 2, natural order,
    no random signs;
  * quantization grid: asymmetric, w = scale * (code - zero), fp16 scale and fp16
    zero per group of g consecutive (rotated) columns, round-to-nearest-even.

Pinned by tests/test_oracle_*.py against: the printed H_2 and the hand-expanded
H_4 (Eq. 2), H H^T = I with entries +-1/sqrt(b) (Notation 4), P^T P = I (text
after Eq. 5), Q^T Q = I and the untouched identity prefix (Eq. 6 and its text),
Eq. 8 evaluated with explicit dense P and Q, brute-force Python loops on tiny
layers, a zero-quantization-error construction, exact recovery of rank <= r
matrices by both low-rank routines (Eq. 10-12 make each step a projection
deflation), the Eckart-Young residual of the truncated SVD, and the printed
average-bit figures (Eq. 13, 0.05 / 0.04 bit for r = 16, the r.bit column of
the rank ablation).  The rounding helpers are pinned against independent
library casts (numpy float16, torch bfloat16 / float8_e4m3fn).
"""
from __future__ import annotations

import numpy as np

# --------------------------------------------------------------------------
# number formats: decoding stored bit patterns, and hand-written rounding
# --------------------------------------------------------------------------


def bf16_bits_to_f64(bits):
    """uint16 bfloat16 bit patterns -> float64 (exact)."""
    b = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def f16_bits_to_f64(bits):
    """uint16 IEEE half bit patterns -> float64 (exact)."""
    return np.asarray(bits, dtype=np.uint16).view(np.float16).astype(np.float64)


def round_to_format(x, mant_bits, emin, max_finite):
    """Round fp64 values to a binary float format, nearest-even, one rounding.

    mant_bits = explicit mantissa bits, emin = exponent of the smallest normal
    (values below it keep the fixed spacing 2^(emin - mant_bits), i.e. gradual
    underflow), max_finite = largest finite value; results beyond it saturate to
    +-inf.  Returns fp64 holding exactly representable values.
    """
    x = np.asarray(x, dtype=np.float64)
    out = np.zeros_like(x)
    fin = np.isfinite(x) & (x != 0.0)
    m, e = np.frexp(x[fin])  # x = m * 2^e, 0.5 <= |m| < 1  ->  exponent of leading bit = e-1
    lead = e - 1
    lead = np.maximum(lead, emin)  # subnormal range: fixed quantum
    quantum_exp = lead - mant_bits
    q = np.rint(np.ldexp(x[fin], -quantum_exp))  # np.rint is round-half-even
    r = np.ldexp(q, quantum_exp)
    r = np.where(np.abs(r) > max_finite, np.copysign(np.inf, r), r)
    out[fin] = r
    out[~np.isfinite(x)] = x[~np.isfinite(x)]
    return out


def round_bf16(x):
    """fp64 -> nearest bfloat16 value (8-bit significand, fp32 exponent range)."""
    return round_to_format(x, 7, -126, float.fromhex("0x1.fep127"))


def round_f16(x):
    """fp64 -> nearest IEEE half value."""
    return round_to_format(x, 10, -14, 65504.0)


def round_f32(x):
    """fp64 -> nearest IEEE single value."""
    return round_to_format(x, 23, -126, float.fromhex("0x1.fffffep127"))


def round_e4m3(x):
    """fp64 -> nearest fp8 e4m3 value (the format the paper stores U, V in; Sec. 3.3,
    implementation details).  Finite-only variant: max 448, values beyond saturate
    to +-448 as storage casts of unit vectors never get there."""
    r = round_to_format(x, 3, -6, 1e30)
    return np.clip(r, -448.0, 448.0)


def f64_to_bf16_bits(x):
    """Exactly-representable fp64 values -> bfloat16 bit patterns (uint16)."""
    f = np.asarray(x, dtype=np.float64).astype(np.float32)
    return (f.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def f64_to_f16_bits(x):
    return np.asarray(round_f16(x)).astype(np.float16).view(np.uint16)


# --------------------------------------------------------------------------
# rotation side: Eq. 2 (Hadamard), Eq. 5 (permutation), Eq. 6 (partial block Q)
# --------------------------------------------------------------------------


def hadamard_matrix(b):
    """Normalised Walsh-Hadamard matrix by the recursion of Eq. 2:
    H_2 = [[1, 1], [1, -1]] / sqrt(2),  H_{2^k} = H_2 (x) H_{2^{k-1}}."""
    if b < 1 or (b & (b - 1)):
        raise ValueError("Hadamard size must be a power of two")
    h2 = np.array([[1.0, 1.0], [1.0, -1.0]]) / np.sqrt(2.0)
    h = np.array([[1.0]])
    while h.shape[0] < b:
        h = np.kron(h2, h)
    return h


def fwht(v):
    """Fast Walsh-Hadamard transform of the last axis (length a power of two),
    normalised so that it equals v @ hadamard_matrix(b) (H is symmetric).
    log2(b) butterfly stages of b/2 add/sub pairs each (Appendix A.3)."""
    v = np.array(v, dtype=np.float64)
    b = v.shape[-1]
    if b & (b - 1):
        raise ValueError("block length must be a power of two")
    h = 1
    while h < b:
        w = v.reshape(v.shape[:-1] + (b // (2 * h), 2, h))
        lo = w[..., 0, :] + w[..., 1, :]
        hi = w[..., 0, :] - w[..., 1, :]
        v = np.stack([lo, hi], axis=-2).reshape(v.shape)
        h *= 2
    return v / np.sqrt(float(b))


def fwht_counted(vec):
    """Pure-Python butterfly on one block; returns (result, number of add/sub).
    Used to check the O(n log b_H) operation count of Appendix A.3."""
    a = [float(t) for t in vec]
    b = len(a)
    ops = 0
    h = 1
    while h < b:
        for start in range(0, b, 2 * h):
            for j in range(start, start + h):
                u, w = a[j], a[j + h]
                a[j], a[j + h] = u + w, u - w
                ops += 2
        h *= 2
    s = 1.0 / np.sqrt(float(b))
    return [t * s for t in a], ops


def check_block_params(n, b_i, b_h):
    if b_h < 1 or (b_h & (b_h - 1)):
        raise ValueError("b_H must be a power of two")
    if b_i < 0 or b_i > n or (n - b_i) % b_h:
        raise ValueError("(n - b_I) must be a non-negative multiple of b_H")


def q_matrix(n, b_i, b_h):
    """Dense Q = diag(I_{b_I}, H_wal, ..., H_wal) of Eq. 6."""
    check_block_params(n, b_i, b_h)
    q = np.zeros((n, n))
    q[:b_i, :b_i] = np.eye(b_i)
    h = hadamard_matrix(b_h)
    for s in range(b_i, n, b_h):
        q[s:s + b_h, s:s + b_h] = h
    return q


def p_matrix(perm):
    """Dense permutation matrix with P[perm[k], k] = 1, so that (R P)[:, k] = R[:, perm[k]]
    and (P^T x)[k] = x[perm[k]] (gather reading of Eq. 5; P^T P = I)."""
    perm = np.asarray(perm)
    n = perm.shape[0]
    p = np.zeros((n, n))
    p[perm, np.arange(n)] = 1.0
    return p


def is_permutation(perm):
    perm = np.asarray(perm)
    return perm.ndim == 1 and np.array_equal(np.sort(perm), np.arange(perm.shape[0]))


def invert_permutation(perm):
    perm = np.asarray(perm)
    inv = np.empty_like(perm)
    inv[perm] = np.arange(perm.shape[0], dtype=perm.dtype)
    return inv


def permute_columns(x, perm):
    """P^T applied to token rows: out[t, k] = x[t, perm[k]] (Appendix A.3, O(nb))."""
    return np.asarray(x)[..., np.asarray(perm)]


def partial_block_rotate(xp, b_i, b_h):
    """Q^T applied to token rows (Q is symmetric): the first b_I entries are kept,
    every following length-b_H block is replaced by its Walsh-Hadamard transform
    (Eq. 6; Appendix A.3)."""
    xp = np.asarray(xp, dtype=np.float64)
    n = xp.shape[-1]
    check_block_params(n, b_i, b_h)
    out = xp.copy()
    if n > b_i:
        blocks = xp[..., b_i:].reshape(xp.shape[:-1] + ((n - b_i) // b_h, b_h))
        out[..., b_i:] = fwht(blocks).reshape(xp.shape[:-1] + (n - b_i,))
    return out


def rotate(x, perm, b_i, b_h):
    """x~ = Q^T P^T x for every token row (the activation-side transform of Eq. 8)."""
    return partial_block_rotate(permute_columns(np.asarray(x, dtype=np.float64), perm), b_i, b_h)


def perm_from_stats(diag_h, r):
    """Eq. 5: perm = sort(diag(H) / amean(R, axis=0)).idx.  Reading: descending
    (large ratio first, as the prose after Eq. 5 and Appendix A.4 describe),
    stable, ties to the lower index."""
    ratio = np.asarray(diag_h, dtype=np.float64) / np.mean(np.abs(np.asarray(r, dtype=np.float64)), axis=0)
    return np.argsort(-ratio, kind="stable").astype(np.int32)


def activation_scale(x_calib):
    """Algorithm 1: Xbar = mean(|X|, axis=0); s = Xbar^2.5 / sqrt(max(Xbar) * min(Xbar))."""
    xbar = np.mean(np.abs(np.asarray(x_calib, dtype=np.float64)), axis=0)
    return xbar ** 2.5 / np.sqrt(xbar.max() * xbar.min())


# --------------------------------------------------------------------------
# quantized part: group grid, dequantisation, canonical bit stream
# --------------------------------------------------------------------------


def dequant(codes, scales, zeros, g):
    """W^[i, k] = scale[i, k // g] * (code[i, k] - zero[i, k // g]) (Appendix A.2/A.3:
    d_q-bit codes with one scale entry per group of g; zero-point per the
    asymmetric grid).  codes uint8 [m][n]; scales, zeros fp64 [m][n/g]."""
    codes = np.asarray(codes).astype(np.float64)
    s = np.repeat(np.asarray(scales, dtype=np.float64), g, axis=1)
    z = np.repeat(np.asarray(zeros, dtype=np.float64), g, axis=1)
    return s * (codes - z)


def rtn_quantize(rp, bits, g, dtype=np.float64):
    """Round-to-nearest asymmetric min/max group quantizer (the RTN row of the
    component ablation).  Per (row, group of g consecutive columns):
    scale = fp16((hi - lo) / (2^q - 1)), zero = fp16(rne(-lo / scale)),
    code = clamp(rne(v / scale) + zero, 0, 2^q - 1).  Degenerate group hi == lo = v:
    scale = |v| (1 if v == 0), zero = 1 if v < 0 else 0, code = 1 if v > 0 else 0.
    `dtype` is the precision every operation is carried out and rounded in (IEEE, nearest-even):
    float64 for the definition; float32 where the integer decisions (codes, zero-points) have to
    be taken in the precision of an implementation that computes in single.
    Returns (codes uint8, scales fp64 holding fp16 values, zeros likewise)."""
    rp = np.asarray(rp, dtype=dtype)
    m, n = rp.shape
    if n % g:
        raise ValueError("group size must divide n")
    qmax = dtype(2 ** bits - 1)
    one, nil = dtype(1.0), dtype(0.0)
    v = rp.reshape(m, n // g, g)
    lo = v.min(axis=2)
    hi = v.max(axis=2)
    degenerate = hi == lo
    scale = round_f16(np.where(degenerate, np.where(lo != nil, np.abs(lo), one), (hi - lo) / qmax)).astype(dtype)
    if np.any(scale == nil):
        raise ValueError("group range underflows fp16")
    zero = round_f16(np.where(degenerate, np.where(lo < nil, one, nil), np.rint(-lo / scale))).astype(dtype)
    code = np.clip(np.rint(v / scale[..., None]) + zero[..., None], nil, qmax)
    return code.reshape(m, n).astype(np.uint8), scale.astype(np.float64), zero.astype(np.float64)


def pack_canonical(codes, bits):
    """Canonical interchange format: per row, code k occupies bits [k q, (k+1) q) of a
    little-endian bit stream stored as uint32 words (4-bit: 8 codes per word, low
    nibble first; 2-bit: 16 per word; 3-bit: 32 codes per 3 words)."""
    codes = np.asarray(codes, dtype=np.uint8)
    m, n = codes.shape
    if (n * bits) % 32:
        raise ValueError("row bit length must be a multiple of 32")
    if np.any(codes >> bits):
        raise ValueError("code out of range")
    bitplane = ((codes[:, :, None] >> np.arange(bits, dtype=np.uint8)) & 1).reshape(m, n * bits)
    weights = (np.uint64(1) << np.arange(32, dtype=np.uint64))
    words = (bitplane.reshape(m, -1, 32).astype(np.uint64) * weights).sum(axis=2)
    return words.astype(np.uint32)


def unpack_canonical(words, bits, n):
    words = np.asarray(words, dtype=np.uint32)
    m = words.shape[0]
    bitplane = ((words[:, :, None] >> np.arange(32, dtype=np.uint32)) & 1).astype(np.uint8).reshape(m, -1)
    b = bitplane[:, : n * bits].reshape(m, n, bits)
    return (b << np.arange(bits, dtype=np.uint8)).sum(axis=2).astype(np.uint8)


def average_bits(m, n, d_q, d_o, g, r, d_r):
    """Eq. 13: d_C = d_q + d_o/g + r d_r/n + r d_r/m + 2 d_o/n + r d_o/(m n)."""
    return d_q + d_o / g + r * d_r / n + r * d_r / m + 2.0 * d_o / n + r * d_o / (m * n)


def lowrank_bits(shapes, r, d_r):
    """Parameter-weighted storage of the U, V factors over a list of (m, n) shapes,
    in bits per weight: sum r d_r (m + n) / sum m n (the 'r.bit' column)."""
    num = sum(r * d_r * (m + n) for m, n in shapes)
    den = sum(m * n for m, n in shapes)
    return num / den


# --------------------------------------------------------------------------
# low-rank part: Eq. 4 (scaled SVD) and Eq. 10-12 / Algorithm 1 (R1SVD)
# --------------------------------------------------------------------------


def svd_lowrank(w_s, r):
    """Truncated SVD of the scaled weight (Eq. 4).  Returns U [m][r], sigma [r], V [r][n]
    with W_s ~= U diag(sigma) V."""
    u, s, vt = np.linalg.svd(np.asarray(w_s, dtype=np.float64), full_matrices=False)
    return u[:, :r], s[:r], vt[:r, :]


def r1svd(w_s, r, it, sketches, cast=None):
    """Rank-1 randomized sketch with deflation (Sec. 3.3, Eq. 10-12; Algorithm 1 inner
    loop).  Per rank: y = (W W^T)^it W v, p = W^T y, U_1 = y / |y|, V_1 = p / |p|,
    sigma = |p| / |y|, optionally cast U_1, V_1 (cast(x) -> x), then W <- W - sigma U_1 V_1.
    `sketches` [r][n] are the random vectors v, passed in so that the routine itself
    draws nothing.  Returns U [m][r], sigma [r], V [r][n]."""
    w = np.array(w_s, dtype=np.float64)
    m, n = w.shape
    us = np.zeros((m, r))
    vs = np.zeros((r, n))
    sig = np.zeros(r)
    for j in range(r):
        y = w @ np.asarray(sketches[j], dtype=np.float64)
        for _ in range(it):
            y = w @ (w.T @ y)
        p = w.T @ y
        ny, npn = np.linalg.norm(y), np.linalg.norm(p)
        if ny == 0.0 or npn == 0.0:
            break  # matrix already exhausted (rank < r)
        u1, v1, s1 = y / ny, p / npn, npn / ny
        if cast is not None:
            u1, v1 = cast(u1), cast(v1)
        us[:, j], vs[j, :], sig[j] = u1, v1, s1
        w = w - s1 * np.outer(u1, v1)
    return us, sig, vs


def lopro_quantize(w, perm, b_i, b_h, r, bits, g, s=None, method="svd", it=8, sketches=None):
    """Calibration-free subset of Algorithm 1 for one linear layer.

    1. W_s = W diag(s) (s defaults to ones); rank-r part of W_s by `method`;
       A = fp16(U Sigma), B = fp16(V diag(s)^-1)                       (Eq. 4)
    2. R = W - A B with the stored (rounded) factors                    (Eq. 3 ii, Eq. 5)
    3. R' = R P Q                                                       (Eq. 6)
    4. RTN group quantisation of R'                                     (ablation row 'RTN')
    Returns dict(codes, scales, zeros, A, B) with fp64 arrays holding fp16 values."""
    w = np.asarray(w, dtype=np.float64)
    m, n = w.shape
    s = np.ones(n) if s is None else np.asarray(s, dtype=np.float64)
    w_s = w * s[None, :]
    if r > 0:
        if method == "svd":
            u, sig, v = svd_lowrank(w_s, r)
        elif method == "r1svd":
            u, sig, v = r1svd(w_s, r, it, sketches)
        else:
            raise ValueError(method)
        a = round_f16(u * sig[None, :])
        b = round_f16(v / s[None, :])
    else:
        a = np.zeros((m, 0))
        b = np.zeros((0, n))
    resid = w - a @ b
    rp = partial_block_rotate(permute_columns(resid, perm), b_i, b_h)  # rows of R P Q (Q symmetric)
    codes, scales, zeros = rtn_quantize(rp, bits, g)
    return dict(codes=codes, scales=scales, zeros=zeros, A=a, B=b)


# --------------------------------------------------------------------------
# forward: Eq. 8
# --------------------------------------------------------------------------


def forward_exact(x, codes, scales, zeros, perm, a, b, g, b_i, b_h):
    """y = A (B x) + W^ (Q^T P^T x), steps in the order of Appendix A.3, all in fp64,
    no intermediate rounding.  x [T][n] -> y [T][m]."""
    x = np.asarray(x, dtype=np.float64)
    xt = rotate(x, perm, b_i, b_h)                 # permutation + FWHT   O(n b log b_H)
    w_hat = dequant(codes, scales, zeros, g)       # Dequant(W_q)
    y_q = xt @ w_hat.T                             # main product         O(b n^2)
    t = x @ np.asarray(b, dtype=np.float64).T      # Y = V X  (folded: B x)
    y_lr = t @ np.asarray(a, dtype=np.float64).T   # O = U (Sigma Y)  (folded: A t)
    return y_q + y_lr


def forward_dense(x, codes, scales, zeros, perm, a, b, g, b_i, b_h):
    """Eq. 8 evaluated literally with dense matrices: W_eff = A B + W^ Q^T P^T,
    y = W_eff x.  For tiny layers only (builds n x n matrices)."""
    x = np.asarray(x, dtype=np.float64)
    n = x.shape[-1]
    w_hat = dequant(codes, scales, zeros, g)
    w_eff = np.asarray(a, dtype=np.float64) @ np.asarray(b, dtype=np.float64) \
        + w_hat @ q_matrix(n, b_i, b_h).T @ p_matrix(perm).T
    return x @ w_eff.T


def effective_weight(codes, scales, zeros, perm, a, b, g, b_i, b_h):
    """The matrix the quantized layer represents: A B + W^ Q^T P^T (Eq. 8), built by
    un-rotating and un-permuting the rows of W^ rather than with dense P, Q."""
    w_hat = dequant(codes, scales, zeros, g)
    unrot = partial_block_rotate(w_hat, b_i, b_h)           # W^ Q^T  (Q symmetric, block-diagonal)
    w_q = np.empty_like(unrot)
    w_q[:, np.asarray(perm)] = unrot                        # (. P^T)[:, perm[k]] = .[:, k]
    return np.asarray(a, dtype=np.float64) @ np.asarray(b, dtype=np.float64) + w_q


def forward_mirrored(x, codes, scales, zeros, perm, a, b, g, b_i, b_h,
                     round_w=False, round_t="f16", out="f32"):
    """Same steps as forward_exact with fp64 accumulation, but with the roundings a
    bf16-activation implementation declares applied by the hand-written rounding
    functions: x~ -> bf16 (always: it is the rotated activation tensor that is
    stored), optionally W^ -> bf16 (fp32 product s*(q-z) then one rounding), t -> fp16
    (or bf16 / none), y -> fp32 or bf16."""
    x = np.asarray(x, dtype=np.float64)
    xt = round_bf16(rotate(x, perm, b_i, b_h))
    w_hat = dequant(codes, scales, zeros, g)
    if round_w:
        w_hat = round_bf16(round_f32(w_hat))
    y_q = xt @ w_hat.T
    t = x @ np.asarray(b, dtype=np.float64).T
    if round_t == "f16":
        t = round_f16(t)
    elif round_t == "bf16":
        t = round_bf16(t)
    y = y_q + t @ np.asarray(a, dtype=np.float64).T
    return round_bf16(y) if out == "bf16" else round_f32(y)


def forward_exact_unfolded(x, codes, scales, zeros, perm, u, sigma, v, s, g, b_i, b_h):
    """Eq. 8 with the low-rank branch in the form Algorithm 1 saves, the record (W_q, U, V, Sigma, p, s):
    y = U (Sigma (V (x / s))) + W^ (Q^T P^T x), i.e. W_r = U Sigma V diag(s)^-1 (Eq. 4 with alpha = diag(s); Sec. 3.3
    keeps s apart so that the fp8 factors U, V stay unit vectors).  u [m][r], sigma [r], v [r][n], s [n]; all fp64,
    no intermediate rounding."""
    x = np.asarray(x, dtype=np.float64)
    xt = rotate(x, perm, b_i, b_h)
    y_q = xt @ dequant(codes, scales, zeros, g).T
    t = (x / np.asarray(s, dtype=np.float64)[None, :]) @ np.asarray(v, dtype=np.float64).T   # Y = V (X / s)
    t = t * np.asarray(sigma, dtype=np.float64)[None, :]                                    # Sigma Y
    return y_q + t @ np.asarray(u, dtype=np.float64).T                                      # O = U (Sigma Y)


def forward_mirrored_unfolded(x, codes, scales, zeros, perm, u, sigma, v, s, g, b_i, b_h, round_t="f16", out="f32"):
    """forward_exact_unfolded with the declared roundings: x~ -> bf16, t = Sigma V (x / s) -> fp16 (or none),
    y -> fp32 or bf16."""
    x = np.asarray(x, dtype=np.float64)
    xt = round_bf16(rotate(x, perm, b_i, b_h))
    y_q = xt @ dequant(codes, scales, zeros, g).T
    t = ((x / np.asarray(s, dtype=np.float64)[None, :]) @ np.asarray(v, dtype=np.float64).T) * np.asarray(sigma, dtype=np.float64)[None, :]
    if round_t == "f16":
        t = round_f16(t)
    y = y_q + t @ np.asarray(u, dtype=np.float64).T
    return round_bf16(y) if out == "bf16" else round_f32(y)


def lopro_quantize_unfolded(w, perm, b_i, b_h, r, bits, g, s, it, sketches):
    """Algorithm 1 for one layer with the low-rank factors kept as the paper stores them: W_s = W diag(s); R1SVD of
    W_s with U_1, V_1 cast to fp8 e4m3 inside the loop (Sec. 3.3), Sigma rounded to fp16; the residual is taken against
    the STORED factors, R = W - U Sigma V diag(s)^-1, then R' = R P Q and RTN group quantization as in lopro_quantize.
    Returns dict(codes, scales, zeros, U, sigma, V, s) (fp64 arrays holding e4m3 / fp16 values; s rounded to fp16)."""
    w = np.asarray(w, dtype=np.float64)
    s = round_f16(np.asarray(s, dtype=np.float64))
    u, sig, v = r1svd(w * s[None, :], r, it, sketches, cast=round_e4m3)
    sig = round_f16(sig)
    resid = w - (u * sig[None, :]) @ (v / s[None, :])
    rp = partial_block_rotate(permute_columns(resid, perm), b_i, b_h)
    codes, scales, zeros = rtn_quantize(rp, bits, g)
    return dict(codes=codes, scales=scales, zeros=zeros, U=u, sigma=sig, V=v, s=s)


def f64_to_e4m3_bits(x):
    """Exactly representable fp64 values -> fp8 e4m3 bit patterns (uint8): sign, 4 exponent bits (bias 7), 3 mantissa
    bits; subnormals below 2^-6; no infinities (the finite-only format of the ML fp8 proposal)."""
    x = np.asarray(x, dtype=np.float64)
    sign = (np.signbit(x)).astype(np.uint8) << 7
    a = np.abs(x)
    out = np.zeros(x.shape, dtype=np.uint8)
    nz = a > 0
    m, e = np.frexp(a[nz])                    # a = m 2^e, 0.5 <= m < 1  ->  a = (2m) 2^(e-1)
    exp = e - 1
    normal = exp >= -6
    bits = np.zeros(m.shape, dtype=np.int64)
    bits[normal] = ((exp[normal] + 7) << 3) | np.rint((2.0 * m[normal] - 1.0) * 8.0).astype(np.int64)
    bits[~normal] = np.rint(a[nz][~normal] * 2.0 ** 9).astype(np.int64)       # subnormal: k 2^-9, k = 1..7
    out[nz] = bits.astype(np.uint8)
    return out | sign


def e4m3_bits_to_f64(b):
    b = np.asarray(b, dtype=np.uint8).astype(np.int64)
    sign = np.where(b & 0x80, -1.0, 1.0)
    exp, man = (b >> 3) & 15, b & 7
    return sign * np.where(exp == 0, man * 2.0 ** -9, (1.0 + man / 8.0) * 2.0 ** (exp - 7.0))


# --------------------------------------------------------------------------
# vector-quantized residual (the LoPRo_v variant, Appendix "implementation details")
# --------------------------------------------------------------------------
# Reading (the paper names a randomly initialised codebook, 4-D at 2 bits, 2-D at 3 bits, no block-wise scaling, no
# learned codebooks, and leaves every format detail to the vector quantizer it calls): the rotated residual R' is cut
# into groups of cb_rows rows x cb_cols columns; a group has ONE codebook of 2^(dim * q) centroids of dimension dim;
# a centroid stands for dim consecutive (rotated) columns of one row; no scale.  With 4-D / 8-bit indices, bf16
# centroids and groups of 512 x 256 the codebook costs 256 * 4 * 16 / (512 * 256) = 0.125 bit per weight -- the
# figure the results table implies (2.17 = 2 + 0.125 + the 0.05 of the rank-16 factors).


def vq_dequant(idx, codebooks, dim, cb_rows, cb_cols):
    """W^[i, dim v + e] = C[i // cb_rows][(dim v) // cb_cols][idx[i, v]][e].
    idx [m][n / dim] integer; codebooks [ceil(m / cb_rows)][n / cb_cols][K][dim] fp64."""
    idx = np.asarray(idx)
    m, nv = idx.shape
    out = np.empty((m, nv * dim))
    for i in range(m):
        for v in range(nv):
            out[i, dim * v:dim * (v + 1)] = codebooks[i // cb_rows][(dim * v) // cb_cols][idx[i, v]]
    return out


def vq_quantize(rp, dim, index_bits, cb_rows, cb_cols, picks):
    """Vector quantization of R' with a randomly initialised codebook: the centroids of a group are 2^index_bits of the
    group's own vectors -- `picks` [row groups][column groups][2^index_bits] indexes the group's vectors in row-major
    order (row within the group, then vector within the row) and is passed in, so that the routine draws nothing --
    rounded to bf16; every vector takes the nearest centroid in the Euclidean norm (the loss of Eq. "rotate loss"
    with H' = I), ties to the lower index.  Returns (idx uint16 [m][n / dim], codebooks fp64 holding bf16 values)."""
    rp = np.asarray(rp, dtype=np.float64)
    m, n = rp.shape
    if n % cb_cols or cb_cols % dim:
        raise ValueError("codebook columns must divide n and hold whole vectors")
    k = 2 ** index_bits
    n_rg, n_cg, vpg = -(-m // cb_rows), n // cb_cols, cb_cols // dim
    idx = np.zeros((m, n // dim), dtype=np.uint16)
    books = np.zeros((n_rg, n_cg, k, dim))
    for rg in range(n_rg):
        r0, r1 = rg * cb_rows, min(m, (rg + 1) * cb_rows)
        for cg in range(n_cg):
            vecs = rp[r0:r1, cg * cb_cols:(cg + 1) * cb_cols].reshape(-1, dim)        # row-major: (row, vector)
            cb = round_bf16(vecs[np.asarray(picks[rg][cg]) % vecs.shape[0]])
            d2 = ((vecs[:, None, :] - cb[None, :, :]) ** 2).sum(axis=2)
            idx[r0:r1, cg * vpg:(cg + 1) * vpg] = np.argmin(d2, axis=1).reshape(r1 - r0, vpg)
            books[rg, cg] = cb
    return idx, books


def forward_exact_vq(x, idx, codebooks, perm, a, b, dim, cb_rows, cb_cols, b_i, b_h):
    """Eq. 8 with the vector-quantized residual: y = x B^T A^T + rotate(x) W^_vq^T, fp64, no rounding."""
    x = np.asarray(x, dtype=np.float64)
    w_hat = vq_dequant(idx, codebooks, dim, cb_rows, cb_cols)
    y = rotate(x, perm, b_i, b_h) @ w_hat.T
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    if a.shape[1]:
        y = y + (x @ b.T) @ a.T
    return y


def vq_average_bits(m, n, dim, index_bits, d_c, cb_rows, cb_cols, r, d_r):
    """Average bits per weight of the vector-quantized record: index bits per weight, the codebooks (d_c bits per
    centroid entry), and the rank-r factors with d_r bits per entry (the last term of Eq. 13)."""
    n_books = -(-m // cb_rows) * (n // cb_cols)
    return index_bits / dim + n_books * (2 ** index_bits) * dim * d_c / (m * n) + r * d_r * (m + n) / (m * n)


def max_rel_err(y, y_ref):
    """Element-wise error relative to max(|y_ref[t, i]|, rms_i y_ref[t, :]): the
    'max relative error' of the acceptance gates, floored at the row RMS so that
    outputs that cancel to ~0 do not dominate."""
    y = np.asarray(y, dtype=np.float64)
    y_ref = np.asarray(y_ref, dtype=np.float64)
    rms = np.sqrt(np.mean(y_ref ** 2, axis=-1, keepdims=True))
    denom = np.maximum(np.abs(y_ref), rms)
    denom = np.where(denom == 0.0, 1.0, denom)
    return float(np.max(np.abs(y - y_ref) / denom))
