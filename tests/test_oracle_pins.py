"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU).

Each test is chosen so that a plausible mistake in the oracle (dropped |S| or norm term,
wrong sign or factor on the dot product, transposed layout, wrong tie direction, off-by-one
in the CSR walk) makes at least one of them fail.
"""
import os

import numpy as np
import pytest

from oracle import som_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "handbuilt_cases.txt")


def _random_problem(rng, V, M, n, max_nnz):
    W = rng.random((V, M)).astype(np.float32)  # feature-major [V, M]
    rows = []
    for _ in range(n):
        k = int(rng.integers(0, min(max_nnz, V) + 1))
        rows.append(np.sort(rng.choice(V, size=k, replace=False)).astype(np.int32))
    indptr = np.zeros(n + 1, np.int32)
    indptr[1:] = np.cumsum([len(r) for r in rows])
    indices = np.concatenate(rows).astype(np.int32) if n else np.zeros(0, np.int32)
    return W, indptr, indices, rows


def _dense_brute_force(W, rows):
    """sum_v (x_v - w_iv)^2 on the densified 0/1 vector: the left side of Eq. 1."""
    V, M = W.shape
    Wd = W.astype(np.float64)
    out = np.empty((len(rows), M))
    for s, r in enumerate(rows):
        x = np.zeros(V)
        x[r] = 1.0
        out[s] = ((x[:, None] - Wd) ** 2).sum(axis=0)
    return out


@pytest.mark.parametrize("seed,V,M,n", [(0, 8, 3, 40), (1, 64, 32, 200), (2, 17, 1, 20), (3, 33, 7, 64)])
def test_distance_identity_vs_dense_brute_force(seed, V, M, n):
    """Eq. 1: the sparse form equals the dense squared distance; same argmin."""
    rng = np.random.default_rng(seed)
    W, indptr, indices, rows = _random_problem(rng, V, M, n, 12)
    D = orc.all_distances(W, V, M, indptr, indices)
    B = _dense_brute_force(W, rows)
    np.testing.assert_allclose(D, B, rtol=1e-12, atol=1e-12)
    t = orc.bmu(W, V, M, indptr, indices)
    np.testing.assert_array_equal(t.b1, B.argmin(axis=1))  # numpy argmin: first minimum
    np.testing.assert_allclose(t.d1, B.min(axis=1), rtol=1e-12, atol=1e-12)
    if M > 1:
        second = np.sort(B, axis=1)[:, 1]
        np.testing.assert_allclose(t.d2, second, rtol=1e-12, atol=1e-12)
        assert np.all(t.b2 != t.b1)
        np.testing.assert_allclose(B[np.arange(n), t.b2], t.d2, rtol=1e-12, atol=1e-12)
    else:
        assert np.all(t.b2 == -1) and np.all(np.isinf(t.d2))


def test_adversarial_dense_rows_and_extreme_ids():
    """Samples that use feature 0, feature V-1, all features, one feature, none."""
    rng = np.random.default_rng(7)
    V, M = 40, 9
    W = (rng.random((V, M)) * 2 - 0.5).astype(np.float32)  # negative weights allowed
    rows = [np.array([0], np.int32), np.array([V - 1], np.int32), np.arange(V, dtype=np.int32),
            np.zeros(0, np.int32), np.array([0, V - 1], np.int32)]
    indptr = np.zeros(len(rows) + 1, np.int32)
    indptr[1:] = np.cumsum([len(r) for r in rows])
    indices = np.concatenate(rows)
    D = orc.all_distances(W, V, M, indptr, indices)
    np.testing.assert_allclose(D, _dense_brute_force(W, rows), rtol=1e-12, atol=1e-12)


def test_layout_invariance():
    """Section 3.2 / 3.4: node-major and feature-major storage give identical results."""
    rng = np.random.default_rng(11)
    V, M, n = 50, 24, 150
    W, indptr, indices, _ = _random_problem(rng, V, M, n, 15)
    Wn = np.ascontiguousarray(W.T)  # node-major [M, V]
    a = orc.bmu(W, V, M, indptr, indices, layout=orc.FEATURE_MAJOR)
    b = orc.bmu(Wn, V, M, indptr, indices, layout=orc.NODE_MAJOR)
    np.testing.assert_array_equal(a.b1, b.b1)
    np.testing.assert_array_equal(a.b2, b.b2)
    np.testing.assert_array_equal(a.d1, b.d1)  # same summation order: bit-identical
    np.testing.assert_array_equal(a.d2, b.d2)
    np.testing.assert_array_equal(orc.norms(W, V, M), orc.norms(Wn, V, M, orc.NODE_MAJOR))


def test_layout_flag_is_not_ignored():
    """A square codebook read with the wrong flag is the transposed codebook: results differ."""
    rng = np.random.default_rng(12)
    V = M = 16
    W, indptr, indices, rows = _random_problem(rng, V, M, 60, 6)
    a = orc.all_distances(W, V, M, indptr, indices, layout=orc.FEATURE_MAJOR)
    b = orc.all_distances(W, V, M, indptr, indices, layout=orc.NODE_MAJOR)
    np.testing.assert_allclose(b, _dense_brute_force(np.ascontiguousarray(W.T), rows), rtol=1e-12)
    assert np.abs(a - b).max() > 1e-3


def _parse_golden():
    cases, cur = [], None
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        tok = line.split()
        if tok[0] == "case":
            cur = {"name": tok[1], "V": int(tok[2]), "M": int(tok[3]), "w": {}, "x": []}
            cases.append(cur)
        elif tok[0] == "w":
            cur["w"][int(tok[1])] = [float(t) for t in tok[3:]]
        elif tok[0] == "x":
            left, right = line[1:].split("|")
            ids = [int(t) for t in left.replace(":", " ").split()]
            r = right.split()
            cur["x"].append((ids, int(r[0]), float(r[1]), int(r[2]), float(r[3])))
    return cases


@pytest.mark.parametrize("case", _parse_golden(), ids=lambda c: c["name"])
def test_handbuilt_cases(case):
    """Known nearest neuron, exact distances, lowest-index ties (Eq. 1, Section 3.1)."""
    V, M = case["V"], case["M"]
    Wn = np.array([case["w"][i] for i in range(M)], np.float32)  # node vectors [M, V]
    assert Wn.shape == (M, V)
    W = np.ascontiguousarray(Wn.T)  # feature-major
    rows = [np.array(x[0], np.int32) for x in case["x"]]
    indptr = np.zeros(len(rows) + 1, np.int32)
    indptr[1:] = np.cumsum([len(r) for r in rows])
    indices = np.concatenate(rows) if rows else np.zeros(0, np.int32)
    for layout, Wl in ((orc.FEATURE_MAJOR, W), (orc.NODE_MAJOR, Wn)):
        t = orc.bmu(Wl, V, M, indptr, indices, layout=layout)
        for s, (_, b1, d1, b2, d2) in enumerate(case["x"]):
            assert t.b1[s] == b1 and t.b2[s] == b2, (case["name"], s, t.b1[s], t.b2[s])
            assert t.d1[s] == d1 and t.d2[s] == d2, (case["name"], s, t.d1[s], t.d2[s])


def test_norms_closed_form():
    """Constant codebook c: ||w||^2 = V*c^2 exactly for power-of-two c."""
    V, M = 3000, 5
    for c in (0.5, 0.25, 2.0):
        W = np.full((V, M), c, np.float32)
        np.testing.assert_array_equal(orc.norms(W, V, M), np.full(M, V * c * c))
    # one-hot columns: norm is the single squared entry
    W = np.zeros((V, M), np.float32)
    for i in range(M):
        W[17 * i + 1, i] = np.float32(i + 1)
    np.testing.assert_array_equal(orc.norms(W, V, M), np.arange(1, M + 1, dtype=np.float64) ** 2)


def test_empty_sample_returns_smallest_norm():
    rng = np.random.default_rng(5)
    V, M = 30, 12
    W = rng.random((V, M)).astype(np.float32)
    indptr = np.array([0, 0, 0], np.int32)
    t = orc.bmu(W, V, M, indptr, np.zeros(0, np.int32))
    nn = (W.astype(np.float64) ** 2).sum(0)
    assert np.all(t.b1 == nn.argmin())
    np.testing.assert_allclose(t.d1, nn.min(), rtol=1e-14)


def test_indptr_base_offset_and_row_walk():
    """Rows are read from indptr[s]..indptr[s+1]; an off-by-one shows up as a changed row."""
    rng = np.random.default_rng(9)
    V, M, n = 25, 6, 30
    W, indptr, indices, rows = _random_problem(rng, V, M, n, 8)
    full = orc.bmu(W, V, M, indptr, indices)
    # take rows 10..19 through an indptr slice that does not start at 0
    sub = orc.bmu(W, V, M, indptr[10:21], indices)
    np.testing.assert_array_equal(sub.b1, full.b1[10:20])
    np.testing.assert_array_equal(sub.d1, full.d1[10:20])


def test_slab_merge_equals_whole():
    """Scanning neuron slabs in ascending order and merging equals one scan."""
    rng = np.random.default_rng(13)
    V, M, n = 40, 37, 120
    W, indptr, indices, _ = _random_problem(rng, V, M, n, 10)
    W[:, 20] = W[:, 3]  # a duplicate across slabs: tie must go to neuron 3
    whole = orc.bmu(W, V, M, indptr, indices)
    run = None
    for m0 in range(0, M, 8):
        m1 = min(M, m0 + 8)
        slab = np.ascontiguousarray(W[:, m0:m1])
        run = orc.bmu(slab, V, m1 - m0, indptr, indices, m_offset=m0, running=run)
    np.testing.assert_array_equal(run.b1, whole.b1)
    np.testing.assert_array_equal(run.b2, whole.b2)
    np.testing.assert_array_equal(run.d1, whole.d1)
    np.testing.assert_array_equal(run.d2, whole.d2)
    assert not np.any(whole.b1 == 20)  # neuron 3 is identical and has the lower index


def test_dist_at_matches_matrix():
    rng = np.random.default_rng(17)
    V, M, n = 30, 11, 50
    W, indptr, indices, _ = _random_problem(rng, V, M, n, 9)
    D = orc.all_distances(W, V, M, indptr, indices)
    pick = rng.integers(0, M, size=n)
    np.testing.assert_array_equal(orc.dist_at(W, V, M, indptr, indices, pick), D[np.arange(n), pick])


def test_argmin_invariant_to_common_shift_of_sample():
    """||x||^2 is constant across neurons (Eq. 1): dropping it changes no argmin."""
    rng = np.random.default_rng(19)
    V, M, n = 45, 20, 80
    W, indptr, indices, rows = _random_problem(rng, V, M, n, 10)
    D = orc.all_distances(W, V, M, indptr, indices)
    nn = orc.norms(W, V, M)
    Wd = W.astype(np.float64)
    for s, r in enumerate(rows):
        score = nn - 2.0 * Wd[r].sum(axis=0)
        assert score.argmin() == D[s].argmin()
        np.testing.assert_allclose(score + len(r), D[s], rtol=1e-12, atol=1e-12)


def test_second_best_parity_rule_on_brute_force():
    """The band rule for the second-best unit, against an explicit ranking of all fp64 distances:
    the true second passes, the third-best fails wherever it lies outside the band, a repeat of
    the best unit always fails, and swapped near-tied leaders pass."""
    from oracle import parity
    rng = np.random.default_rng(11)
    V, M, n = 40, 12, 300
    W = rng.random((V, M)).astype(np.float32)
    rows = [np.sort(rng.choice(V, size=int(rng.integers(1, 9)), replace=False)).astype(np.int32) for _ in range(n)]
    indptr = np.zeros(n + 1, np.int32)
    indptr[1:] = np.cumsum([len(r) for r in rows])
    indices = np.concatenate(rows)
    D = orc.all_distances(W.reshape(-1), V, M, indptr, indices)
    order = np.argsort(D, axis=1, kind="stable")
    t = orc.bmu(W.reshape(-1), V, M, indptr, indices)
    ar = np.arange(n)
    np.testing.assert_array_equal(order[:, 0], t.b1)
    np.testing.assert_array_equal(order[:, 1], t.b2)
    good = parity.check_second(t.b1, t.b2, D[ar, t.b2], t, D[ar, t.b2], M)
    assert good.ok and good.differs_from_oracle == 0
    third = order[:, 2]
    far = (D[ar, third] - t.d2) > parity.GAP_REL * t.d2
    assert far.sum() > n // 2
    bad = parity.check_second(t.b1, third, D[ar, third], t, D[ar, third], M)
    assert not bad.ok and bad.outside_band == int(far.sum())
    rep = parity.check_second(t.b1, t.b1, t.d1, t, t.d1, M)
    assert not rep.ok and rep.same_as_best == n
    swapped = parity.check_second(t.b2, t.b1, t.d1, t, t.d1, M)  # leaders the other way round
    assert swapped.ok
    wrong_dist = parity.check_second(t.b1, t.b2, D[ar, t.b2] * (1 + 1e-4), t, D[ar, t.b2], M)
    assert wrong_dist.dist_violations == n


def test_first_unit_parity_rule_rejects_wrong_outputs():
    """The rule every GPU parity test stands on (oracle.parity.check), against an explicit ranking
    of all fp64 distances: the true answer passes; the second-best unit given as the best fails
    wherever the two are outside the band; a distance off by 1e-4 relative fails; an index out of
    range fails; a near-tied unit just inside the band passes and one just outside it fails."""
    from oracle import parity
    rng = np.random.default_rng(23)
    V, M, n = 40, 12, 300
    W = rng.random((V, M)).astype(np.float32)
    rows = [np.sort(rng.choice(V, size=int(rng.integers(1, 9)), replace=False)).astype(np.int32) for _ in range(n)]
    indptr = np.zeros(n + 1, np.int32)
    indptr[1:] = np.cumsum([len(r) for r in rows])
    indices = np.concatenate(rows)
    D = orc.all_distances(W.reshape(-1), V, M, indptr, indices)
    order = np.argsort(D, axis=1, kind="stable")
    t = orc.bmu(W.reshape(-1), V, M, indptr, indices)
    ar = np.arange(n)
    good = parity.check(t.b1, D[ar, t.b1].astype(np.float32), t, D[ar, t.b1], M)
    assert good.ok and good.index_mismatch_unambiguous == 0 and good.histogram_equal
    # the oracle's second unit in place of the first
    far = (t.d2 - t.d1) > parity.GAP_REL * t.d1
    assert far.sum() > n // 2
    second = parity.check(t.b2, D[ar, t.b2].astype(np.float32), t, D[ar, t.b2], M)
    assert not second.ok and second.index_mismatch_unambiguous == int(far.sum())
    assert not second.histogram_equal
    # right units, distances off by 1e-4 relative (ten times the tolerance)
    off = parity.check(t.b1, (D[ar, t.b1] * (1 + 1e-4)).astype(np.float32), t, D[ar, t.b1], M)
    assert not off.ok and off.dist_violations == n and off.index_mismatch_unambiguous == 0
    # distances inside the tolerance pass: 2e-6 relative
    near = parity.check(t.b1, D[ar, t.b1] * (1 + 2e-6), t, D[ar, t.b1], M)
    assert near.ok
    # an index out of range, on an unambiguous and on a near-tied sample
    bad = t.b1.copy()
    bad[0] = M
    bad[1] = -1
    safe = np.clip(bad, 0, M - 1)
    rep = parity.check(bad, D[ar, safe].astype(np.float32), t, D[ar, safe], M)
    assert not rep.ok
    # hand-made near ties: two units whose distances differ by a chosen relative gap
    top = orc.Top2(np.array([3, 3, 3]), np.array([10.0, 10.0, 10.0]), np.array([5, 5, 5]),
                   np.array([10.0 + 5e-4, 10.0 + 5e-4, 10.0 + 2e-3]))
    # sample 0: near tie, unit 5 reported, its distance inside the band -> accepted and counted
    # sample 1: near tie, a third unit reported whose distance is just outside the band -> rejected
    # sample 2: unambiguous (gap 2e-4 relative), unit 5 reported -> rejected
    g = np.array([5, 7, 5])
    d_at = np.array([10.0 + 5e-4, 10.0 + 1.1e-3, 10.0 + 2e-3])
    rep = parity.check(g, d_at.astype(np.float32), top, d_at, M)
    assert rep.near_ties == 2 and rep.unambiguous == 1
    assert rep.near_tie_outside_band == 1 and rep.index_mismatch_unambiguous == 1
    ok_only = parity.check(g[:1], d_at[:1].astype(np.float32),
                           orc.Top2(top.b1[:1], top.d1[:1], top.b2[:1], top.d2[:1]), d_at[:1], M)
    assert ok_only.ok and ok_only.near_ties == 1


def test_real_valued_samples_against_dense_brute_force():
    """Sparse real-valued samples: ||x||^2 - 2<x,w> + ||w||^2 against sum_v (x_v - w_iv)^2 on the
    densified vector (numpy); all-ones values reduce to the binary search; a neuron equal to the
    sample is at distance zero."""
    rng = np.random.default_rng(21)
    V, M, n = 48, 19, 120
    W = rng.normal(size=(V, M)).astype(np.float32)
    rows = [np.sort(rng.choice(V, size=int(rng.integers(0, 10)), replace=False)).astype(np.int32) for _ in range(n)]
    indptr = np.zeros(n + 1, np.int32)
    indptr[1:] = np.cumsum([len(r) for r in rows])
    indices = np.concatenate(rows).astype(np.int32)
    values = rng.normal(size=indices.size).astype(np.float32)
    X = np.zeros((n, V))
    for s_, r in enumerate(rows):
        X[s_, r] = values[indptr[s_]:indptr[s_ + 1]].astype(np.float64)
    D = ((X[:, :, None] - W.astype(np.float64)[None, :, :]) ** 2).sum(1)
    t = orc.bmu_values(W.reshape(-1), V, M, indptr, indices, values)
    order = np.argsort(D, axis=1, kind="stable")
    np.testing.assert_array_equal(t.b1, order[:, 0])
    np.testing.assert_array_equal(t.b2, order[:, 1])
    np.testing.assert_allclose(t.d1, D[np.arange(n), t.b1], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(orc.dist_at_values(W.reshape(-1), V, M, indptr, indices, values, t.b2),
                               D[np.arange(n), t.b2], rtol=1e-12, atol=1e-12)
    ones = np.ones_like(values)
    tb, tv = orc.bmu(W.reshape(-1), V, M, indptr, indices), orc.bmu_values(W.reshape(-1), V, M, indptr, indices, ones)
    np.testing.assert_array_equal(tb.b1, tv.b1)
    np.testing.assert_allclose(tb.d1, tv.d1, rtol=1e-13, atol=1e-13)
    W2 = W.copy()
    W2[:, 7] = X[3].astype(np.float32)  # neuron 7 becomes sample 3
    t2 = orc.bmu_values(W2.reshape(-1), V, M, indptr, indices, values)
    assert t2.b1[3] == 7 and abs(t2.d1[3]) < 1e-5
