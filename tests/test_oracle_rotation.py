"""Pins for the rotation side of the oracle (Eq. 2, Eq. 5, Eq. 6, Appendix A.3):
printed / hand-expanded Hadamard matrices, orthogonality, structure of Q, and the
permutation convention.  CPU only."""
import os

import numpy as np
import pytest

from oracle import lopro_oracle as o


def _read_golden_hadamard(golden_dir):
    mats, cur, size = {}, [], None
    with open(os.path.join(golden_dir, "hadamard_eq2.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            if line.startswith("H "):
                if size is not None:
                    mats[size] = np.array(cur, dtype=np.float64)
                size, cur = int(line.split()[1]), []
            else:
                cur.append([1.0 if c == "+" else -1.0 for c in line.split()])
    mats[size] = np.array(cur, dtype=np.float64)
    return mats


def test_hadamard_matches_printed_h2_and_hand_expanded(golden_dir):
    mats = _read_golden_hadamard(golden_dir)
    assert set(mats) == {2, 4, 8}
    for b, signs in mats.items():
        assert signs.shape == (b, b)
        np.testing.assert_allclose(o.hadamard_matrix(b), signs / np.sqrt(b), rtol=0, atol=1e-15)


@pytest.mark.parametrize("b", [1, 2, 4, 16, 64, 128, 256])
def test_hadamard_orthogonal_entries_and_popcount_form(b):
    h = o.hadamard_matrix(b)
    np.testing.assert_allclose(h @ h.T, np.eye(b), atol=1e-12)
    np.testing.assert_allclose(np.abs(h), 1.0 / np.sqrt(b), atol=1e-15)
    np.testing.assert_allclose(h, h.T, atol=0)
    i, j = np.meshgrid(np.arange(b), np.arange(b), indexing="ij")
    pop = np.array([[bin(a & c).count("1") for c in range(b)] for a in range(b)])
    np.testing.assert_allclose(h, (-1.0) ** pop / np.sqrt(b), atol=1e-15)


@pytest.mark.parametrize("b", [2, 4, 8, 64, 256])
def test_butterfly_equals_dense_product(b):
    rng = np.random.default_rng(b)
    v = rng.standard_normal((5, b))
    np.testing.assert_allclose(o.fwht(v), v @ o.hadamard_matrix(b), atol=1e-12)
    # involution, norm preservation, H e_0 = constant vector
    np.testing.assert_allclose(o.fwht(o.fwht(v)), v, atol=1e-12)
    np.testing.assert_allclose(np.linalg.norm(o.fwht(v), axis=1), np.linalg.norm(v, axis=1), rtol=1e-12)
    e0 = np.zeros(b)
    e0[0] = 1.0
    np.testing.assert_allclose(o.fwht(e0), np.full(b, 1 / np.sqrt(b)), atol=1e-15)


def test_butterfly_distinguishes_natural_from_other_orderings():
    # e_1 must map to the second ROW of the Sylvester matrix: + - + - ...
    e1 = np.zeros(8)
    e1[1] = 1.0
    np.testing.assert_allclose(o.fwht(e1) * np.sqrt(8), [1, -1, 1, -1, 1, -1, 1, -1], atol=1e-15)
    e4 = np.zeros(8)
    e4[4] = 1.0
    np.testing.assert_allclose(o.fwht(e4) * np.sqrt(8), [1, 1, 1, 1, -1, -1, -1, -1], atol=1e-15)


def test_fwht_counted_matches_and_counts_n_log_b():
    rng = np.random.default_rng(1)
    for b in (2, 8, 64):
        v = rng.standard_normal(b)
        res, ops = o.fwht_counted(v)
        np.testing.assert_allclose(res, o.fwht(v), atol=1e-12)
        assert ops == b * int(np.log2(b))  # b/2 pairs x 2 ops x log2(b) stages (Appendix A.3)


@pytest.mark.parametrize("n,b_i,b_h", [(16, 0, 4), (24, 8, 4), (64, 32, 16), (12, 4, 8), (32, 32, 8), (192, 64, 64)])
def test_q_structure(n, b_i, b_h):
    q = o.q_matrix(n, b_i, b_h)
    np.testing.assert_allclose(q.T @ q, np.eye(n), atol=1e-12)
    np.testing.assert_allclose(q[:b_i, :b_i], np.eye(b_i), atol=0)
    rng = np.random.default_rng(n)
    x = rng.standard_normal((3, n))
    xr = o.partial_block_rotate(x, b_i, b_h)
    np.testing.assert_allclose(xr, x @ q, atol=1e-12)          # row form of Q^T x, Q symmetric
    np.testing.assert_array_equal(xr[:, :b_i], x[:, :b_i])     # identity prefix untouched
    # block independence: perturbing one rotated block changes that block only
    if n > b_i:
        x2 = x.copy()
        x2[:, b_i:b_i + b_h] += 1.0
        d = o.partial_block_rotate(x2, b_i, b_h) - xr
        assert np.all(d[:, :b_i] == 0) and np.all(np.abs(d[:, b_i + b_h:]) < 1e-13)
        assert np.any(np.abs(d[:, b_i:b_i + b_h]) > 0.1)


def test_block_param_validation():
    with pytest.raises(ValueError):
        o.q_matrix(20, 0, 8)
    with pytest.raises(ValueError):
        o.q_matrix(24, 0, 6)
    with pytest.raises(ValueError):
        o.fwht(np.zeros(12))


def test_permutation_convention_and_orthogonality():
    rng = np.random.default_rng(3)
    n = 12
    perm = rng.permutation(n).astype(np.int32)
    p = o.p_matrix(perm)
    np.testing.assert_array_equal(p.T @ p, np.eye(n))
    x = rng.standard_normal((2, n))
    # gather reading: (P^T x)[k] = x[perm[k]]
    np.testing.assert_array_equal(o.permute_columns(x, perm), x @ p)
    for k in range(n):
        assert o.permute_columns(x, perm)[0, k] == x[0, perm[k]]
    # columns of a matrix: (R P)[:, k] = R[:, perm[k]]
    r = rng.standard_normal((4, n))
    np.testing.assert_array_equal(r @ p, r[:, perm])
    # round trip with the inverse index vector
    inv = o.invert_permutation(perm)
    np.testing.assert_array_equal(o.permute_columns(o.permute_columns(x, perm), inv), x)
    assert o.is_permutation(perm) and not o.is_permutation(np.array([0, 0, 1]))
    # a hand-written case: perm = [2, 0, 1] brings old column 2 to the front
    np.testing.assert_array_equal(o.permute_columns(np.array([[10.0, 20.0, 30.0]]), [2, 0, 1]), [[30.0, 10.0, 20.0]])


def test_perm_from_stats_moves_large_ratio_first():
    diag_h = np.array([1.0, 4.0, 1.0, 2.0])
    r = np.array([[1.0, 1.0, 0.5, 1.0], [-1.0, 1.0, -0.5, -1.0]])   # amean = 1, 1, .5, 1 -> ratio 1, 4, 2, 2
    np.testing.assert_array_equal(o.perm_from_stats(diag_h, r), [1, 2, 3, 0])


def test_activation_scale_worked_by_hand():
    # Algorithm 1: Xbar = column means of |X| = (2, 2, 4); max * min = 8, so s = Xbar^2.5 / sqrt(8):
    # 2^2.5 / 2^1.5 = 2 and 4^2.5 / 2^1.5 = 32 / (2 sqrt 2) = 8 sqrt 2 -- numbers worked out on paper
    x = np.array([[1.0, -2.0, 4.0], [3.0, 2.0, -4.0]])
    s = o.activation_scale(x)
    np.testing.assert_allclose(s, [2.0, 2.0, 11.313708498984761], rtol=1e-14)
    # homogeneous of degree 1.5 in X (2.5 - 2 / 2): scaling the calibration data by 4 scales s by 8
    np.testing.assert_allclose(o.activation_scale(4.0 * x), 8.0 * s, rtol=1e-14)


def test_rotate_is_orthogonal_map_of_x():
    rng = np.random.default_rng(5)
    n, b_i, b_h = 96, 32, 32
    perm = rng.permutation(n)
    x = rng.standard_normal((4, n))
    xt = o.rotate(x, perm, b_i, b_h)
    np.testing.assert_allclose(np.linalg.norm(xt, axis=1), np.linalg.norm(x, axis=1), rtol=1e-12)
    np.testing.assert_allclose(xt, x @ o.p_matrix(perm) @ o.q_matrix(n, b_i, b_h), atol=1e-12)
