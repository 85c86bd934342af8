"""Pins of the CPU update oracle (scatter, factorised box blur, divide; Section 3.4) against what
the paper and the mathematics fix: a hand-computed case, the band-matrix form of the truncated
box passes, closed forms for special inputs, and the stated edge rules."""
import os

import numpy as np
import pytest

from oracle import som_update_oracle as uorc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "update_handbuilt.txt")


def _csr(rows_list):
    indptr = np.zeros(len(rows_list) + 1, np.int32)
    indptr[1:] = np.cumsum([len(r) for r in rows_list])
    indices = np.concatenate([np.asarray(r, np.int32) for r in rows_list]) if rows_list else np.zeros(0, np.int32)
    return indptr, indices.astype(np.int32)


def _band(E, r):
    i = np.arange(E)
    return (np.abs(i[:, None] - i[None, :]) <= r).astype(np.float64)


def test_handbuilt_case_from_fixture():
    cases, cur = {}, None
    for line in open(GOLDEN):
        tok = line.split()
        if not tok or tok[0].startswith("#"):
            continue
        if tok[0] == "passes":
            cur = cases.setdefault(int(tok[1]), {})
        else:
            cur[tok[0]] = np.array([float(t) for t in tok[1:]])
    indptr, indices = _csr([[0], [1], [1]])
    bmu = np.array([0, 3, 3], np.int32)
    W_old = np.full(2 * 4, 7.0, np.float32)
    for passes, f in cases.items():
        W = uorc.update(W_old, 2, 1, 4, indptr, indices, bmu, 1, passes).reshape(2, 4)
        np.testing.assert_array_equal(W[0], f["num0"] / f["den"])
        np.testing.assert_array_equal(W[1], f["num1"] / f["den"])
        np.testing.assert_array_equal(uorc.blur(np.array([1.0, 0, 0, 2]), 1, 4, 1, passes)[0], f["den"])


@pytest.mark.parametrize("rows,cols,radius", [(5, 7, 1), (8, 8, 3), (6, 4, 2), (9, 3, 5), (1, 10, 2)])
def test_blur_equals_band_matrix_powers(rows, cols, radius):
    """A truncated, unnormalised box pass along an axis is multiplication by the 0/1 band matrix
    |i - j| <= radius; three passes per axis are its cube on either side."""
    rng = np.random.default_rng(rows * 100 + cols)
    P = rng.integers(0, 5, size=(rows, cols)).astype(np.float64)
    A_r = np.linalg.matrix_power(_band(rows, radius), 3)
    A_c = np.linalg.matrix_power(_band(cols, radius), 3)
    np.testing.assert_allclose(uorc.blur(P, rows, cols, radius, 3), A_r @ P @ A_c.T, rtol=1e-13)
    # one pass, and the two axes separately
    np.testing.assert_allclose(uorc.blur(P, rows, cols, radius, 1), _band(rows, radius) @ P @ _band(cols, radius), rtol=1e-13)


def _random_problem(seed, V, rows, cols, n):
    rng = np.random.default_rng(seed)
    M = rows * cols
    samples = [np.sort(rng.choice(V, size=int(rng.integers(1, 6)), replace=False)) for _ in range(n)]
    indptr, indices = _csr(samples)
    bmu = rng.integers(0, M, size=n).astype(np.int32)
    W_old = rng.random(V * M).astype(np.float32)
    return samples, indptr, indices, bmu, W_old


def test_update_equals_dense_matrix_form():
    """Whole update against numpy: scatter by dense one-hot products, blur by band matrices."""
    V, rows, cols, n, radius = 13, 6, 5, 60, 1
    samples, indptr, indices, bmu, W_old = _random_problem(1, V, rows, cols, n)
    M = rows * cols
    X = np.zeros((n, V))
    for s, f in enumerate(samples):
        X[s, f] = 1.0
    C = np.zeros((n, M))
    C[np.arange(n), bmu] = 1.0
    num = X.T @ C          # [V, M] sum of the samples of every cell
    den = C.sum(0)         # [M]
    A_r = np.linalg.matrix_power(_band(rows, radius), 3)
    A_c = np.linalg.matrix_power(_band(cols, radius), 3)
    den_b = (A_r @ den.reshape(rows, cols) @ A_c.T).reshape(M)
    num_b = np.stack([(A_r @ num[v].reshape(rows, cols) @ A_c.T).reshape(M) for v in range(V)])
    want = np.where(den_b > 0, num_b / np.where(den_b > 0, den_b, 1.0), W_old.reshape(V, M).astype(np.float64))
    got = uorc.update(W_old, V, rows, cols, indptr, indices, bmu, radius).reshape(V, M)
    np.testing.assert_allclose(got, want, rtol=1e-13, atol=0)


def test_feature_of_every_sample_becomes_one_and_absent_feature_zero():
    """num and den receive the identical kernel (unnormalised sums cancel): a feature that every
    sample has gives exactly num = den, a feature no sample has gives 0."""
    V, rows, cols, n = 6, 7, 7, 40
    rng = np.random.default_rng(3)
    samples = [np.unique(np.concatenate([[0], rng.choice(np.arange(1, V - 1), size=2, replace=False)])) for _ in range(n)]
    indptr, indices = _csr(samples)
    bmu = rng.integers(0, rows * cols, size=n).astype(np.int32)
    W_old = np.full(V * rows * cols, 0.5, np.float32)
    W = uorc.update(W_old, V, rows, cols, indptr, indices, bmu, 2).reshape(V, rows * cols)
    assert np.all(W[0] == 1.0)          # radius 2 x 3 passes reaches every cell of a 7 x 7 lattice
    assert np.all(W[V - 1] == 0.0)
    assert np.all((W >= 0.0) & (W <= 1.0))  # a weighted mean of binary samples


def test_cells_outside_every_support_keep_their_prototype():
    """Blurred denominator zero -> prototype unchanged; the support of three radius-1 passes is the
    Chebyshev ball of radius 3, truncated at the edge (clamped, not toroidal)."""
    V, rows, cols = 4, 12, 12
    indptr, indices = _csr([[1, 2]])
    bmu = np.array([0], np.int32)  # the corner cell
    W_old = (np.arange(V * rows * cols) % 17 / 17.0).astype(np.float32)
    W = uorc.update(W_old, V, rows, cols, indptr, indices, bmu, 1).reshape(V, rows, cols)
    old = W_old.reshape(V, rows, cols).astype(np.float64)
    rr, cc = np.meshgrid(np.arange(rows), np.arange(cols), indexing="ij")
    inside = np.maximum(rr, cc) <= 3
    for v in range(V):
        np.testing.assert_array_equal(W[v][~inside], old[v][~inside])
        np.testing.assert_array_equal(W[v][inside], 1.0 if v in (1, 2) else 0.0)
    assert np.all(W[:, rows - 1, :] == old[:, rows - 1, :])  # nothing wraps around


def test_radius_covering_the_lattice_gives_the_global_mean():
    """With radius >= the lattice edge every pass sums whole lines, so every neuron becomes the
    mean of all samples."""
    V, rows, cols, n = 9, 4, 6, 50
    samples, indptr, indices, bmu, W_old = _random_problem(5, V, rows, cols, n)
    W = uorc.update(W_old, V, rows, cols, indptr, indices, bmu, 6).reshape(V, rows * cols)
    freq = np.bincount(indices, minlength=V) / n
    np.testing.assert_allclose(W, np.repeat(freq[:, None], rows * cols, 1), rtol=1e-14)


def test_no_samples_leaves_the_codebook():
    V, rows, cols = 3, 4, 4
    W_old = np.linspace(0, 1, V * rows * cols).astype(np.float32)
    W = uorc.update(W_old, V, rows, cols, np.zeros(1, np.int32), np.zeros(0, np.int32), np.zeros(0, np.int32), 2)
    np.testing.assert_array_equal(W, W_old.astype(np.float64))
