"""GPU parity tests of the two-best search (som_bmu2) against the CPU oracle's second-best unit.

The best unit and its distance must be bit-identical to som_bmu's; the second-best unit follows
the band rule of ``oracle.parity.check_second``.
"""
import os

import numpy as np
import pytest
import torch

from oracle import parity
from oracle import som_oracle as orc
from paper_2608_24067_b200 import synth

pytestmark = pytest.mark.gpu

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "handbuilt_cases.txt")


@pytest.fixture(scope="module")
def som_mod():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_24067_b200 import som
    som.load_library()  # fail loudly when the extension is missing
    return som


def _run_both(som_mod, W_dev, V, M, indptr_dev, indices_dev, variant=None, options=()):
    h = som_mod.Som(V, M, W_dev)
    if variant is not None:
        h.set_option(0, variant)
    for key, value in options:
        h.set_option(key, value)
    h.norms()
    one = h.bmu(indptr_dev, indices_dev)
    two = h.bmu2(indptr_dev, indices_dev)
    again = h.bmu2(indptr_dev, indices_dev)
    torch.cuda.synchronize()
    # the best unit does not depend on whether the second is tracked; outputs repeat bit for bit
    assert torch.equal(one[0], two[0]) and torch.equal(one[1].view(torch.int32), two[1].view(torch.int32))
    for a, b in zip(two, again):
        assert torch.equal(a.view(torch.int32), b.view(torch.int32))
    return [t.cpu().numpy() for t in two]


def _subset(indptr, indices, rows):
    indptr = np.asarray(indptr, dtype=np.int64)
    lens = indptr[rows + 1] - indptr[rows]
    out_ptr = np.zeros(len(rows) + 1, np.int32)
    out_ptr[1:] = np.cumsum(lens)
    out_idx = np.concatenate([indices[indptr[r]:indptr[r + 1]] for r in rows]).astype(np.int32)
    return out_ptr, out_idx


def _check(W_host, V, M, indptr, indices, out, rows=None):
    g1, gd1, g2, gd2 = out
    indptr, indices = np.asarray(indptr), np.asarray(indices)
    if rows is not None:
        indptr, indices = _subset(indptr, indices, rows)
        g1, gd1, g2, gd2 = g1[rows], gd1[rows], g2[rows], gd2[rows]
    nn = orc.norms(W_host, V, M)
    top2 = orc.bmu(W_host, V, M, indptr, indices, norms_=nn)
    d_at1 = orc.dist_at(W_host, V, M, indptr, indices, np.clip(g1.astype(np.int64), 0, M - 1), norms_=nn)
    rep1 = parity.check(g1, gd1, top2, d_at1, M)
    assert rep1.ok, str(rep1)
    d_at2 = orc.dist_at(W_host, V, M, indptr, indices, np.clip(g2.astype(np.int64), 0, M - 1), norms_=nn)
    rep2 = parity.check_second(g1, g2, gd2, top2, d_at2, M)
    assert rep2.ok, str(rep2)
    return rep2


@pytest.mark.parametrize("variant", [1, 2, 0])
@pytest.mark.parametrize("kind", ["zipf", "uniform"])
def test_top2_config1_full(som_mod, kind, variant):
    """Tiny 16x16 configuration, every sample, both kernels."""
    w = synth.CONFIGS[0]
    W = synth.fill_codebook(w.V, w.M, w.seed, device="cuda")
    b = synth.sample_csr(w.N, w.V, w.lam, w.seed, device="cuda", zipf_s=0.0 if kind == "uniform" else w.zipf_s)
    out = _run_both(som_mod, W, w.V, w.M, b.indptr, b.indices, variant)
    rep = _check(W.cpu().numpy(), w.V, w.M, b.indptr.cpu().numpy(), b.indices.cpu().numpy(), out)
    assert rep.differs_from_oracle < 0.01 * w.N


@pytest.mark.parametrize("variant", [1, 2])
def test_top2_config2_sampled_rows(som_mod, variant):
    """64x64 map, one million samples on the GPU; every 40th row against the oracle."""
    w = synth.CONFIGS[1]
    W = synth.fill_codebook(w.V, w.M, w.seed, device="cuda")
    b = synth.sample_csr(w.N, w.V, w.lam, w.seed, device="cuda")
    out = _run_both(som_mod, W, w.V, w.M, b.indptr, b.indices, variant)
    assert out[2].min() >= 0 and out[2].max() < w.M and np.all(out[2] != out[0])
    rows = np.concatenate([np.arange(0, w.N, 40), [w.N - 1]])
    rep = _check(W.cpu().numpy(), w.V, w.M, b.indptr.cpu().numpy(), b.indices.cpu().numpy(), out, rows)
    assert rep.differs_from_oracle < 0.05 * rows.size


@pytest.mark.parametrize("lane_neurons,threads", [(4, 1024), (8, 640), (16, 512)])
def test_top2_row_table_geometries(som_mod, lane_neurons, threads):
    V, M, n = 30_000, 1_024, 60_000
    W = synth.fill_codebook(V, M, 3, device="cuda")
    b = synth.sample_csr(n, V, 11.0, 3, device="cuda", permute_ids=True)
    out = _run_both(som_mod, W, V, M, b.indptr, b.indices, 2, options=((3, lane_neurons), (2, threads)))
    _check(W.cpu().numpy(), V, M, b.indptr.cpu().numpy(), b.indices.cpu().numpy(), out, np.arange(0, n, 7))


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


@pytest.mark.parametrize("variant", [1, 2, 0])
@pytest.mark.parametrize("case", _parse_golden(), ids=lambda c: c["name"])
def test_top2_handbuilt_cases(som_mod, case, variant):
    """Exactly representable weights: both units and both distances must be exact, ties (also
    between the best and the second) broken to the lowest index."""
    V, M = case["V"], case["M"]
    Wn = np.array([case["w"][i] for i in range(M)], np.float32)
    W = torch.from_numpy(np.ascontiguousarray(Wn.T)).cuda().reshape(-1)
    rows = [np.array(x[0], np.int32) for x in case["x"]]
    indptr = np.zeros(len(rows) + 1, np.int32)
    indptr[1:] = np.cumsum([len(r) for r in rows])
    indices = np.concatenate(rows) if rows else np.zeros(0, np.int32)
    idx_dev = torch.from_numpy(indices).cuda() if indices.size else torch.zeros(1, dtype=torch.int32, device="cuda")
    g1, gd1, g2, gd2 = _run_both(som_mod, W, V, M, torch.from_numpy(indptr).cuda(), idx_dev, variant)
    for s, (_, b1, d1, b2, d2) in enumerate(case["x"]):
        assert g1[s] == b1 and gd1[s] == np.float32(d1), (case["name"], s, g1[s], gd1[s])
        assert g2[s] == b2 and gd2[s] == np.float32(d2), (case["name"], s, g2[s], gd2[s])


@pytest.mark.parametrize("variant", [1, 2, 0])
@pytest.mark.parametrize("V,M,n", [(64, 37, 200), (97, 130, 300), (40, 4, 64), (40, 2, 64),
                                   (300, 260, 500), (1000, 1028, 700)])
def test_top2_ragged_shapes(som_mod, V, M, n, variant):
    rng = np.random.default_rng(V * 1000 + M)
    W = rng.random((V, M)).astype(np.float32)
    rows = []
    for s in range(n):
        k = int(rng.integers(0, min(V, 45) + 1))  # includes empty rows and rows longer than 32
        rows.append(np.sort(rng.choice(V, size=k, replace=False)).astype(np.int32))
    indptr = np.zeros(n + 1, np.int32)
    indptr[1:] = np.cumsum([len(r) for r in rows])
    indices = np.concatenate(rows).astype(np.int32)
    out = _run_both(som_mod, torch.from_numpy(W).cuda().reshape(-1), V, M,
                    torch.from_numpy(indptr).cuda(), torch.from_numpy(indices).cuda(), variant)
    _check(W, V, M, indptr, indices, out)


def test_top2_single_neuron_has_no_second(som_mod):
    V, M, n = 50, 1, 30
    rng = np.random.default_rng(5)
    W = rng.random((V, M)).astype(np.float32)
    indptr = np.arange(0, 3 * (n + 1), 3, dtype=np.int32)
    indices = np.concatenate([np.sort(rng.choice(V, 3, replace=False)) for _ in range(n)]).astype(np.int32)
    g1, gd1, g2, gd2 = _run_both(som_mod, torch.from_numpy(W).cuda().reshape(-1), V, M,
                                 torch.from_numpy(indptr).cuda(), torch.from_numpy(indices).cuda())
    assert np.all(g1 == 0) and np.all(g2 == -1) and np.all(np.isinf(gd2))


def test_top2_rejects_null_outputs(som_mod):
    import ctypes
    w = synth.CONFIGS[0]
    W = synth.fill_codebook(w.V, w.M, w.seed, device="cuda")
    b = synth.sample_csr(100, w.V, w.lam, w.seed, device="cuda")
    h = som_mod.Som(w.V, w.M, W)
    h.norms()
    o1 = torch.empty(100, dtype=torch.int32, device="cuda")
    o2 = torch.empty(100, dtype=torch.float32, device="cuda")
    rc = h._lib.som_bmu2(h._h, b.indptr.data_ptr(), b.indices.data_ptr(), 100, o1.data_ptr(), o2.data_ptr(),
                         None, None, ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
    assert rc == 1  # SOM_ERR_INVALID_ARG
