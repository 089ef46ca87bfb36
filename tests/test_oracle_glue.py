"""Pins of the decoder-block operations of oracle/glue_oracle.py against closed forms and invariants."""
import numpy as np

from oracle import glue_oracle as g


def test_rmsnorm_closed_forms():
    # a row of +-a has mean square a^2: the output is sign * w (eps = 0)
    x = np.array([[3.0, -3.0, 3.0, -3.0], [0.5, 0.5, -0.5, 0.5]])
    w = np.array([1.0, 2.0, -1.0, 0.25])
    np.testing.assert_allclose(g.rmsnorm(x, w, 0.0), np.sign(x) * w, rtol=1e-15)
    # hand-worked: x = (1, 2, 2, 4): mean square 25/4, rms 5/2
    np.testing.assert_allclose(g.rmsnorm(np.array([[1.0, 2.0, 2.0, 4.0]]), np.ones(4), 0.0), [[0.4, 0.8, 0.8, 1.6]], rtol=1e-15)
    # eps enters under the root: a zero row stays zero, and x = (2, 2) with eps = 5 has denominator 3
    assert np.all(g.rmsnorm(np.zeros((1, 8)), np.ones(8), 1e-6) == 0.0)
    np.testing.assert_allclose(g.rmsnorm(np.array([[2.0, 2.0]]), np.ones(2), 5.0), [[2.0 / 3.0, 2.0 / 3.0]], rtol=1e-15)
    # scale invariance (eps = 0) and unit mean square of the unweighted output
    rng = np.random.default_rng(1)
    x = rng.standard_normal((5, 64))
    np.testing.assert_allclose(g.rmsnorm(7.5 * x, w=np.ones(64), eps=0.0), g.rmsnorm(x, np.ones(64), 0.0), rtol=1e-13)
    np.testing.assert_allclose(np.mean(g.rmsnorm(x, np.ones(64), 0.0) ** 2, axis=1), 1.0, rtol=1e-13)


def test_rope_closed_forms():
    rng = np.random.default_rng(2)
    x = rng.standard_normal((6, 3, 8))
    # position 0 is the identity
    np.testing.assert_array_equal(g.rope(x, np.zeros(6, dtype=np.int64)), x)
    # pair 0 turns by exactly pos radians (theta^0 = 1): (1, 0) at position p becomes (cos p, sin p)
    e = np.zeros((1, 1, 8))
    e[0, 0, 0] = 1.0
    out = g.rope(e, np.array([3]))
    np.testing.assert_allclose(out[0, 0, :2], [np.cos(3.0), np.sin(3.0)], rtol=1e-15)
    assert np.all(out[0, 0, 2:] == 0.0)
    # pair i turns by pos * theta^(-2i/d): d = 8, theta = 16 -> pair 2 has frequency 16^(-1/2) = 1/4
    e = np.zeros((1, 1, 8))
    e[0, 0, 5] = 1.0
    out = g.rope(e, np.array([2]), theta=16.0)
    np.testing.assert_allclose(out[0, 0, 4:6], [-np.sin(0.5), np.cos(0.5)], rtol=1e-15)
    # a rotation: norms of pairs are preserved
    pos = np.array([0, 1, 5, 17, 100, 2047])
    y = g.rope(x, pos)
    np.testing.assert_allclose(y[..., 0::2] ** 2 + y[..., 1::2] ** 2, x[..., 0::2] ** 2 + x[..., 1::2] ** 2, rtol=1e-12)
    # relative-position property: <rope(q, m), rope(k, n)> depends on m - n only
    q, k = rng.standard_normal((1, 1, 8)), rng.standard_normal((1, 1, 8))
    a = np.sum(g.rope(q, np.array([9])) * g.rope(k, np.array([4])))
    b = np.sum(g.rope(q, np.array([105])) * g.rope(k, np.array([100])))
    np.testing.assert_allclose(a, b, rtol=1e-11)


def test_attention_closed_forms():
    rng = np.random.default_rng(3)
    T, H, C, d = 3, 2, 7, 4
    k, v = rng.standard_normal((T, H, C, d)), rng.standard_normal((T, H, C, d))
    ctx = np.array([7, 1, 4])
    # a zero query attends uniformly: the mean of the valid values
    out = g.attention_decode(np.zeros((T, H, d)), k, v, ctx, 0.5)
    for t in range(T):
        np.testing.assert_allclose(out[t], v[t, :, :ctx[t]].mean(axis=1), rtol=1e-14)
    # a single valid key returns its value whatever the query
    out = g.attention_decode(rng.standard_normal((T, H, d)), k, v, ctx, 0.5)
    np.testing.assert_allclose(out[1], v[1, :, 0], rtol=1e-14)
    # two keys with scores s and 0: weights are the logistic function of s
    q = np.array([[[2.0, 0.0]]])
    kk = np.array([[[[1.5, 0.0], [0.0, 1.0]]]])
    vv = np.array([[[[1.0, 0.0], [0.0, 1.0]]]])
    out = g.attention_decode(q, kk, vv, np.array([2]), 1.0)
    p = 1.0 / (1.0 + np.exp(-3.0))
    np.testing.assert_allclose(out[0, 0], [p, 1.0 - p], rtol=1e-14)
    # the scale multiplies the scores; a dominant key wins; large scores do not overflow
    out = g.attention_decode(q, kk * 1000.0, vv, np.array([2]), 1.0)
    np.testing.assert_allclose(out[0, 0], [1.0, 0.0], atol=1e-300)
    # entries beyond ctx are ignored
    k2, v2 = k.copy(), v.copy()
    k2[2, :, 4:], v2[2, :, 4:] = 1e6, 1e6
    qq = rng.standard_normal((T, H, d))
    np.testing.assert_array_equal(g.attention_decode(qq, k2, v2, ctx, 0.5)[2], g.attention_decode(qq, k, v, ctx, 0.5)[2])


def test_silu_mul_values():
    # x sigmoid(x): 0 at 0, x/2 slope... tabulated logistic values: sigma(ln 3) = 3/4, sigma(-ln 3) = 1/4
    x = np.array([0.0, np.log(3.0), -np.log(3.0), 40.0, -40.0])
    u = np.array([5.0, 2.0, 2.0, 1.0, 1.0])
    ref = np.array([0.0, np.log(3.0) * 0.75 * 2.0, -np.log(3.0) * 0.25 * 2.0, 40.0, -40.0 * np.exp(-40.0)])
    np.testing.assert_allclose(g.silu_mul(x, u), ref, rtol=1e-13, atol=1e-300)
    # odd part: silu(x) - silu(-x) = x
    z = np.linspace(-6.0, 6.0, 25)
    np.testing.assert_allclose(g.silu_mul(z, np.ones_like(z)) - g.silu_mul(-z, np.ones_like(z)), z, rtol=1e-13, atol=1e-15)
