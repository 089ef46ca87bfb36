"""Plain fp64 definitions of the decoder-block operations that sit BETWEEN the quantized linear layers of the
32-layer stack workload: RMS normalisation, rotary position embedding, causal soft-max attention of one new token per
sequence over a key/value cache, SiLU gating and the residual sum.

TEST INFRASTRUCTURE ONLY -- never imported by the CUDA library or its binding.

None of these is part of the quantization method (the paper's Eq. 8 covers the linear layers only; its latency table
measures them inside a LLaMA decoder).  They are the textbook operations of that architecture, written out as their
definitions, one token per row:

  rmsnorm(x, w, eps)[t, i] = x[t, i] * w[i] / sqrt(mean_i(x[t, i]^2) + eps)
  rope(x, pos, theta)      : the head's dimensions form pairs (2i, 2i+1); pair i of the token at position p is
                             rotated by the angle p * theta^(-2i/d)   (the original rotary formulation; pairing
                             (i, i + d/2) instead is the same map after a fixed re-ordering of the dimensions)
  attention_decode         : out[t, h] = sum_j softmax_j(q[t, h] . K[t, h, j] * scale) V[t, h, j],  j < ctx[t]
  silu_mul(g, u)           = g * sigmoid(g) * u
Pinned by tests/test_oracle_glue.py against closed forms (unit-variance rows, zero angle, norm preservation, the
relative-position property of the rotary map, uniform attention of a zero query, a single key, a dominant key,
tabulated values of the logistic function).
"""
from __future__ import annotations

import numpy as np


def rmsnorm(x, w, eps):
    x = np.asarray(x, dtype=np.float64)
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x * np.asarray(w, dtype=np.float64) / np.sqrt(ms + eps)


def rope(x, pos, theta=10000.0):
    """x [T][H][d] (d even), pos [T] integer positions: every head's pair (2i, 2i+1) rotated by pos * theta^(-2i/d)."""
    x = np.asarray(x, dtype=np.float64)
    T, H, d = x.shape
    i = np.arange(d // 2, dtype=np.float64)
    ang = np.asarray(pos, dtype=np.float64)[:, None] * theta ** (-2.0 * i / d)[None, :]      # [T][d/2]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    out = np.empty_like(x)
    out[..., 0::2] = x[..., 0::2] * c - x[..., 1::2] * s
    out[..., 1::2] = x[..., 0::2] * s + x[..., 1::2] * c
    return out


def attention_decode(q, k_cache, v_cache, ctx, scale):
    """q [T][H][d]: one new token per sequence; k_cache, v_cache [T][H][C][d]: the sequence's keys and values (the new
    token's own among them); ctx [T]: how many cache entries of sequence t are valid.  Returns [T][H][d]."""
    q = np.asarray(q, dtype=np.float64)
    T, H, d = q.shape
    out = np.zeros((T, H, d))
    for t in range(T):
        n = int(ctx[t])
        for h in range(H):
            s = np.asarray(k_cache[t, h, :n], dtype=np.float64) @ q[t, h] * scale
            p = np.exp(s - s.max())
            p /= p.sum()
            out[t, h] = p @ np.asarray(v_cache[t, h, :n], dtype=np.float64)
    return out


def silu_mul(gate, up):
    g = np.asarray(gate, dtype=np.float64)
    return g / (1.0 + np.exp(-g)) * np.asarray(up, dtype=np.float64)
