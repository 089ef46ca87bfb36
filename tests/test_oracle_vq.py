"""Pins of the vector-quantized residual of oracle/lopro_oracle.py (the LoPRo_v variant)."""
import numpy as np

from oracle import lopro_oracle as o


def _golden():
    import os
    out = {}
    for line in open(os.path.join(os.path.dirname(__file__), "golden", "avg_bits.txt")):
        if line.strip() and not line.startswith("#"):
            k, v, tol, _ = line.split()
            out[k] = (float(v), float(tol))
    return out


def test_vq_dequant_is_a_table_lookup():
    # two row groups x two column groups, 2-D centroids: every entry written out by hand
    books = np.zeros((2, 2, 4, 2))
    for rg in range(2):
        for cg in range(2):
            for k in range(4):
                books[rg, cg, k] = [100 * rg + 10 * cg + k, -(100 * rg + 10 * cg + k)]
    idx = np.array([[0, 1, 2, 3], [3, 3, 0, 0], [1, 0, 0, 2]])            # 3 rows, 4 vectors = 8 columns
    w = o.vq_dequant(idx, books, dim=2, cb_rows=2, cb_cols=4)
    exp = np.array([[0, 0, 1, -1, 12, -12, 13, -13],
                    [3, -3, 3, -3, 10, -10, 10, -10],
                    [101, -101, 100, -100, 110, -110, 112, -112]], dtype=np.float64)
    np.testing.assert_array_equal(w, exp)


def test_vq_quantize_picks_the_nearest_centroid_brute_force():
    rng = np.random.default_rng(3)
    m, n, dim, bits, cr, cc = 6, 16, 4, 3, 4, 8
    rp = rng.standard_normal((m, n))
    picks = [[rng.integers(0, 1000, size=2 ** bits) for _ in range(n // cc)] for _ in range(2)]
    idx, books = o.vq_quantize(rp, dim, bits, cr, cc, picks)
    np.testing.assert_array_equal(books, o.round_bf16(books))            # centroids are bf16 numbers
    for i in range(m):
        for v in range(n // dim):
            cb = books[i // cr][(dim * v) // cc]
            d = [float(np.sum((rp[i, dim * v:dim * v + dim] - c) ** 2)) for c in cb]
            assert idx[i, v] == int(np.argmin(d))                        # ties go to the lower index (argmin's rule)
    # a group whose every vector is among its centroids (and is a bf16 number) is reproduced exactly
    base = o.round_bf16(rng.standard_normal((8, dim)))
    rp2 = base[rng.integers(0, 8, size=(4 * 2,))].reshape(4, 2 * dim)
    rp2[0], rp2[1] = np.concatenate([base[0], base[1]]), np.concatenate([base[2], base[3]])
    rp2[2], rp2[3] = np.concatenate([base[4], base[5]]), np.concatenate([base[6], base[7]])
    idx2, books2 = o.vq_quantize(rp2, dim, 3, 4, 2 * dim, [[np.arange(8)]])
    np.testing.assert_array_equal(o.vq_dequant(idx2, books2, dim, 4, 2 * dim), rp2)


def test_forward_vq_equals_a_plain_product_with_the_effective_matrix():
    rng = np.random.default_rng(5)
    m, n, dim, bits, cr, cc, b, r, T = 8, 32, 4, 4, 4, 16, 8, 2, 3
    idx = rng.integers(0, 2 ** bits, size=(m, n // dim))
    books = o.round_bf16(rng.standard_normal((m // cr, n // cc, 2 ** bits, dim)))
    perm = rng.permutation(n).astype(np.int32)
    a, bb = rng.standard_normal((m, r)), rng.standard_normal((r, n))
    x = rng.standard_normal((T, n))
    y = o.forward_exact_vq(x, idx, books, perm, a, bb, dim, cr, cc, b, b)
    # Eq. 8 with explicit dense P and Q
    w_hat = o.vq_dequant(idx, books, dim, cr, cc)
    P, Q = o.p_matrix(perm), o.q_matrix(n, b, b)
    np.testing.assert_allclose(y, x @ (a @ bb + w_hat @ Q.T @ P.T).T, atol=1e-12)


def test_vq_storage_matches_the_printed_average_bits():
    # 4-D codebook, 8-bit indices, bf16 centroids, one codebook per 512 x 256 weights: 2 + 0.125 bits; with the rank-16
    # fp8 factors on the 7B shapes the results table's 2.17 for the vector-quantized variant
    gold = _golden()
    shapes = [(4096, 4096)] * 4 + [(11008, 4096)] * 2 + [(4096, 11008)]
    total = sum(m * n for m, n in shapes)
    bits = sum(o.vq_average_bits(m, n, 4, 8, 16, 512, 256, 16, 8) * m * n for m, n in shapes) / total
    val, _ = gold["bits_lopro_2"]
    # 2.1757: the 11008-row matrices end in a partial group of 256 rows that still carries a whole codebook (+0.0017);
    # the table's 2.17 is this figure with the third decimal cut, as in its rank-ablation rows
    assert 0.0 <= bits - val <= 0.0081
    assert o.vq_average_bits(4096, 4096, 4, 8, 16, 512, 256, 0, 8) == 2.125
    assert abs(o.vq_average_bits(4096, 4096, 4, 8, 16, 512, 256, 16, 8) - (2.125 + 2 * 16 * 8 / 4096)) < 1e-15
    # the 3-bit form: 2-D centroids, 6-bit indices, 64 centroids per group of 512 x 256 -- 3 + 64 * 2 * 16 / 131072 bits
    assert o.vq_average_bits(4096, 4096, 2, 6, 16, 512, 256, 0, 8) == 3.015625
    assert abs(o.vq_average_bits(4096, 4096, 2, 6, 16, 512, 256, 16, 8) - (3.015625 + 2 * 16 * 8 / 4096)) < 1e-15


def test_vq_quantize_with_two_dimensional_centroids_brute_force():
    rng = np.random.default_rng(11)
    m, n, dim, bits, cr, cc = 5, 12, 2, 6, 4, 6
    rp = rng.standard_normal((m, n))
    picks = [[rng.integers(0, 1000, size=2 ** bits) for _ in range(n // cc)] for _ in range(2)]
    idx, books = o.vq_quantize(rp, dim, bits, cr, cc, picks)
    assert idx.max() < 64 and books.shape == (2, 2, 64, 2)
    for i in range(m):
        for v in range(n // dim):
            cb = books[i // cr][(dim * v) // cc]
            d = [float(np.sum((rp[i, dim * v:dim * v + dim] - c) ** 2)) for c in cb]
            assert idx[i, v] == int(np.argmin(d))

