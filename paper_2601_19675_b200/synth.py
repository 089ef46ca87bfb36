"""Seeded synthetic inputs for the LoPRo linear-layer workloads.

This module only draws random tensors and converts them to the storage formats of
the C ABI (bf16 / fp16 bit patterns, uint8 codes, int32 indices).  It contains none
of the method's arithmetic (no permutation, rotation, quantisation, packing or
matmul) and imports neither the CUDA binding nor the CPU oracle, so both sides can
be fed the same bytes.

Generator: numpy's counter-based Philox, one independent stream per tensor, keyed by
(seed, tensor tag).

Workloads (stand-ins for the LLM layers the paper quantizes; real weights and
calibration data are not available):
  cfg1  512 x 512, T=16, 4-bit g128, b_I=b_H=64, r=16, weights ~ N(0, 0.02) to be
        quantized by the caller
  cfg2  4096 x 4096 decode, T in {1, 8}, 4-bit g128, b=128, r=32
  cfg3  4096 -> 11008 prefill, T=2048, 3-bit g64, b=128, r=64, 1 % outlier columns x20
  cfg4  8192 -> 28672, T in {16, 4096}, 2-bit g64, b=256, r=128
Codes are uniform on [0, 2^q), scales ~ U(0.005, 0.02), zeros ~ U(0, 2^q - 1) (code
units), low-rank factors ~ N(0, 0.01), activations ~ N(0, 1), permutation uniform.
"""
from __future__ import annotations

import numpy as np

_TAGS = {"x": 1, "perm": 2, "codes": 3, "scales": 4, "zeros": 5, "A": 6, "B": 7, "W": 8,
         "outliers": 9, "sketch": 10, "U": 11, "V": 12, "sigma": 13, "s": 14}

CONFIGS = {
    "cfg1": dict(d_in=512, d_out=512, bits=4, group_size=128, block_size=64, identity_cols=64, rank=16, T=(16,)),
    "cfg2": dict(d_in=4096, d_out=4096, bits=4, group_size=128, block_size=128, identity_cols=128, rank=32, T=(1, 8)),
    "cfg3": dict(d_in=4096, d_out=11008, bits=3, group_size=64, block_size=128, identity_cols=128, rank=64, T=(2048,),
                 outlier_frac=0.01, outlier_scale=20.0),
    "cfg4": dict(d_in=8192, d_out=28672, bits=2, group_size=64, block_size=256, identity_cols=256, rank=128,
                 T=(16, 4096)),
}


def _rng(seed, tag):
    return np.random.Generator(np.random.Philox(key=[int(seed), _TAGS[tag]]))


def f32_to_bf16_bits(a):
    """float32 -> bfloat16 bit patterns, round-to-nearest-even (storage conversion)."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def f32_to_f16_bits(a):
    return np.asarray(a, dtype=np.float32).astype(np.float16).view(np.uint16)


def f32_to_e4m3_bits(a):
    """float32 -> fp8 e4m3 bit patterns (finite-only format: 4 exponent bits, bias 7, 3 mantissa bits, subnormals
    below 2^-6, largest value 448), round-to-nearest-even, magnitudes beyond 448 clamped (storage conversion)."""
    a = np.asarray(a, dtype=np.float32).astype(np.float64)
    sign = np.signbit(a).astype(np.uint8) << 7
    mag = np.minimum(np.abs(a), 448.0)
    m, e = np.frexp(mag)                                   # mag = m 2^e, 0.5 <= m < 1
    exp = np.maximum(e - 1, -6)                            # exponent of the leading bit, clamped to the subnormal range
    q = np.rint(np.ldexp(mag, 3 - exp)).astype(np.int64)   # significand in units of 2^(exp - 3): 8..16 (0..8 below 2^-6)
    exp = np.where(q == 16, exp + 1, exp)                  # rounding carried into the next binade
    q = np.where(q == 16, 8, q)
    normal = q >= 8
    bits = np.where(normal, ((exp + 7) << 3) | (q - 8), q)
    return (bits.astype(np.uint8) | sign).astype(np.uint8)


def lowrank_record(m, n, r, seed=0):
    """The low-rank record (U, V, Sigma, s) in its stored formats: U [m][r], V [r][n] as e4m3 bit patterns of entries
    ~ N(0, 1/dim) (unit-vector scale), Sigma [r] ~ U(0.05, 0.5) and the activation scale s [n] ~ U(0.5, 2) as fp16 bits."""
    u = _rng(seed, "U").standard_normal((m, r), dtype=np.float32) / np.float32(np.sqrt(m))
    v = _rng(seed, "V").standard_normal((r, n), dtype=np.float32) / np.float32(np.sqrt(n))
    sigma = _rng(seed, "sigma").uniform(0.05, 0.5, size=r).astype(np.float32)
    s = _rng(seed, "s").uniform(0.5, 2.0, size=n).astype(np.float32)
    return dict(U=f32_to_e4m3_bits(u), V=f32_to_e4m3_bits(v), sigma=f32_to_f16_bits(sigma), s=f32_to_f16_bits(s))


def activations(T, n, seed=0, outlier_frac=0.0, outlier_scale=20.0):
    """bf16 bit patterns [T][n] of N(0,1) activations; a seeded fraction of the columns
    is scaled up to imitate the few dominant channels of LLM activations."""
    x = _rng(seed, "x").standard_normal((T, n), dtype=np.float32)
    if outlier_frac > 0.0:
        k = max(1, int(round(outlier_frac * n)))
        cols = _rng(seed, "outliers").choice(n, size=k, replace=False)
        x[:, cols] *= np.float32(outlier_scale)
    return f32_to_bf16_bits(x)


def permutation(n, seed=0):
    return _rng(seed, "perm").permutation(n).astype(np.int32)


def codes(m, n, bits, seed=0):
    return _rng(seed, "codes").integers(0, 2 ** bits, size=(m, n), dtype=np.uint8)


def scales(m, n_groups, seed=0, lo=0.005, hi=0.02):
    return f32_to_f16_bits(_rng(seed, "scales").uniform(lo, hi, size=(m, n_groups)).astype(np.float32))


def zeros(m, n_groups, bits, seed=0):
    return f32_to_f16_bits(_rng(seed, "zeros").uniform(0.0, 2 ** bits - 1, size=(m, n_groups)).astype(np.float32))


def factors(m, n, r, seed=0, std=0.01):
    a = _rng(seed, "A").standard_normal((m, r), dtype=np.float32) * np.float32(std)
    b = _rng(seed, "B").standard_normal((r, n), dtype=np.float32) * np.float32(std)
    return f32_to_f16_bits(a), f32_to_f16_bits(b)


def weights(m, n, seed=0, std=0.02, spikes=0, spike_gain=24.0):
    """fp32 weight matrix ~ N(0, std); `spikes` > 0 adds that many rank-1 terms with geometrically decaying weights
    (separated leading singular values, as trained LLM weights have)."""
    w = _rng(seed, "W").standard_normal((m, n), dtype=np.float32) * np.float32(std)
    if spikes:
        a = _rng(seed, "A").standard_normal((m, spikes), dtype=np.float32)
        b = _rng(seed, "B").standard_normal((spikes, n), dtype=np.float32)
        gains = (np.float32(spike_gain * std) * np.float32(0.75) ** np.arange(spikes, dtype=np.float32)) / np.float32(np.sqrt(min(m, n)))
        w = w + (a * gains[None, :]) @ b
    return w.astype(np.float32)


def sketches(r, n, seed=0):
    return _rng(seed, "sketch").standard_normal((r, n))


def random_layer(d_in, d_out, bits, group_size, rank, seed=0, **_unused):
    """All stored tensors of one synthetic quantized layer (cfg2-style recipe)."""
    ng = d_in // group_size
    a, b = factors(d_out, d_in, rank, seed)
    return dict(codes=codes(d_out, d_in, bits, seed), scales=scales(d_out, ng, seed),
                zeros=zeros(d_out, ng, bits, seed), perm=permutation(d_in, seed), A=a, B=b)
