"""GPU parity tests: the CUDA library (through its C ABI) against the CPU oracle.

Index work must match exactly outside the stated near-tie band, distances within 1e-5
relative, histograms of unambiguous winners bit-exact, outputs bit-identical run to run.
"""
import os

import numpy as np
import pytest
import torch

from oracle import parity
from oracle import som_oracle as orc
from paper_2608_24067_b200 import synth

import largemap

pytestmark = pytest.mark.gpu

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "handbuilt_cases.txt")


@pytest.fixture(scope="module")
def som_mod():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_24067_b200 import som
    som.load_library()  # fail loudly when the extension is missing
    return som


def _run_gpu(som_mod, W_dev, V, M, indptr_dev, indices_dev, variant=None):
    h = som_mod.Som(V, M, W_dev)
    if variant is not None:
        h.set_option(0, variant)
    h.norms()
    bmu, dist = h.bmu(indptr_dev, indices_dev)
    torch.cuda.synchronize()
    return h, bmu.cpu().numpy(), dist.cpu().numpy()


def _subset_csr(indptr, indices, rows):
    """Host CSR of the chosen rows (numpy)."""
    indptr = np.asarray(indptr, dtype=np.int64)
    lens = indptr[rows + 1] - indptr[rows]
    out_ptr = np.zeros(len(rows) + 1, np.int32)
    out_ptr[1:] = np.cumsum(lens)
    parts = [indices[indptr[r]:indptr[r + 1]] for r in rows]
    out_idx = np.concatenate(parts).astype(np.int32) if len(parts) else np.zeros(0, np.int32)
    return out_ptr, out_idx


def _check_against_oracle(W_host, V, M, indptr, indices, g_bmu, g_dist, rows=None):
    indptr = np.asarray(indptr)
    indices = np.asarray(indices)
    if rows is not None:
        indptr, indices = _subset_csr(indptr, indices, rows)
        g_bmu, g_dist = g_bmu[rows], g_dist[rows]
    nn = orc.norms(W_host, V, M)
    top2 = orc.bmu(W_host, V, M, indptr, indices, norms_=nn)
    safe = np.clip(g_bmu.astype(np.int64), 0, M - 1)
    d_at = orc.dist_at(W_host, V, M, indptr, indices, safe, norms_=nn)
    rep = parity.check(g_bmu, g_dist, top2, d_at, M)
    assert rep.ok, str(rep)
    return rep


@pytest.mark.parametrize("variant", [1, 2, 0])
@pytest.mark.parametrize("kind", ["zipf", "permuted", "uniform"])
def test_config1_full(som_mod, kind, variant):
    """Tiny 16x16 configuration, every sample checked."""
    w = synth.CONFIGS[0]
    W = synth.fill_codebook(w.V, w.M, w.seed, device="cuda")
    b = synth.sample_csr(w.N, w.V, w.lam, w.seed, device="cuda",
                         zipf_s=0.0 if kind == "uniform" else w.zipf_s,
                         permute_ids=(kind == "permuted"))
    h, g_bmu, g_dist = _run_gpu(som_mod, W, w.V, w.M, b.indptr, b.indices, variant)
    assert h.validate_csr(b.indptr, b.indices)
    rep = _check_against_oracle(W.cpu().numpy(), w.V, w.M, b.indptr.cpu().numpy(),
                                b.indices.cpu().numpy(), g_bmu, g_dist)
    assert rep.near_ties < 0.01 * w.N
    # norms against the oracle's fp64 norms
    nn = orc.norms(W.cpu().numpy(), w.V, w.M)
    np.testing.assert_allclose(h.get_norms().cpu().numpy().astype(np.float64), nn, rtol=2e-7)


@pytest.mark.parametrize("variant", [1, 2, 0])
def test_config2_sampled_rows(som_mod, variant):
    """64x64 map, one million samples on the GPU; every 40th row against the oracle."""
    w = synth.CONFIGS[1]
    W = synth.fill_codebook(w.V, w.M, w.seed, device="cuda")
    b = synth.sample_csr(w.N, w.V, w.lam, w.seed, device="cuda")
    h, g_bmu, g_dist = _run_gpu(som_mod, W, w.V, w.M, b.indptr, b.indices, variant)
    rows = np.arange(0, w.N, 40)
    rows = np.concatenate([rows, [w.N - 1]])
    rep = _check_against_oracle(W.cpu().numpy(), w.V, w.M, b.indptr.cpu().numpy(),
                                b.indices.cpu().numpy(), g_bmu, g_dist, rows)
    assert rep.near_ties < 0.05 * rows.size
    # run-to-run determinism on the full batch
    bmu2, dist2 = h.bmu(b.indptr, b.indices)
    torch.cuda.synchronize()
    assert np.array_equal(bmu2.cpu().numpy(), g_bmu)
    assert np.array_equal(dist2.cpu().numpy().view(np.uint32), g_dist.view(np.uint32))


@pytest.mark.parametrize("lane_neurons,threads", [(4, 1024), (4, 768), (8, 512), (8, 768), (8, 640), (16, 512),
                                                  (16, 576)])
def test_row_table_geometries(som_mod, lane_neurons, threads):
    """The lane widths of the row-table kernel (32-, 64- and 128-neuron ranges) and block sizes,
    with permuted feature ids so that the hot features are not the low ids."""
    V, M, n = 30_000, 1_024, 60_000
    W = synth.fill_codebook(V, M, 3, device="cuda")
    b = synth.sample_csr(n, V, 11.0, 3, device="cuda", permute_ids=True)
    h = som_mod.Som(V, M, W)
    h.set_option(0, 2)
    h.set_option(3, lane_neurons)
    h.set_option(2, threads)
    h.norms()
    bmu, dist = h.bmu(b.indptr, b.indices)
    torch.cuda.synchronize()
    rows = np.arange(0, n, 7)
    _check_against_oracle(W.cpu().numpy(), V, M, b.indptr.cpu().numpy(), b.indices.cpu().numpy(),
                          bmu.cpu().numpy(), dist.cpu().numpy(), rows)


@pytest.mark.parametrize("mask_bits", [1, 5, 9, 16])
def test_mask_feature_counts(som_mod, mask_bits):
    """How many of the batch's most frequent features the plan handles as mask bits (the rest of the 16
    become ordinary hot rows) is a matter of speed only: every split matches the oracle, on fp32 and on the
    wide fp16 layout (permuted feature ids, so that the frequent features are not the low ids)."""
    V, M, n = 30_000, 1_024, 50_000
    b = synth.sample_csr(n, V, 11.0, 4, device="cuda", permute_ids=True)
    rows = np.arange(0, n, 9)
    for dtype in (torch.float32, torch.float16):
        W = synth.fill_codebook(V, M, 4, device="cuda").to(dtype)
        h = som_mod.Som(V, M, W)
        h.set_option(0, 2)
        h.set_option(8, mask_bits)
        h.norms()
        bmu, dist = h.bmu(b.indptr, b.indices)
        torch.cuda.synchronize()
        _check_against_oracle(W.float().cpu().numpy(), V, M, b.indptr.cpu().numpy(), b.indices.cpu().numpy(),
                              bmu.cpu().numpy(), dist.cpu().numpy(), rows)
        assert h.device_flags() == 0


@pytest.mark.parametrize("lane_neurons", [4, 8, 16])
@pytest.mark.parametrize("codebook", ["recipe", "smooth", "constant", "negative"])
def test_pruning_by_range_maxima_changes_nothing(som_mod, lane_neurons, codebook):
    """The row-table kernel may skip a sample's tail rows for a neuron range whose scores cannot reach the
    sample's key (bounds from the per-range maxima that som_norms writes).  Forced on (by default it runs on
    maps of 32 ranges of 128 neurons and more; this map has 16), its outputs are bit-identical to those of the full search and match the
    oracle: on the benchmark's codebook recipe, on a smooth map (nearly everything is skipped), on a map of
    equal neurons (nothing can be skipped: every range ties) and on weights of both signs."""
    V, M, n = 30_000, 2_048, 40_000
    W = synth.fill_codebook(V, M, 5, device="cuda")
    if codebook == "smooth":
        ramp = torch.linspace(0.0, 1.0, M, device="cuda")
        W = (W.view(V, M) * 0.2 + ramp[None, :] * torch.rand(V, 1, device="cuda")).reshape(-1).contiguous()
    elif codebook == "constant":
        W = W.view(V, M)[:, :1].repeat(1, M).reshape(-1).contiguous()
    elif codebook == "negative":
        W = (W - 0.3).contiguous()
    b = synth.sample_csr(n, V, 11.0, 5, device="cuda", permute_ids=True)
    outs = []
    for prune in (2, 1):
        h = som_mod.Som(V, M, W)
        h.set_option(0, 2)
        h.set_option(3, lane_neurons)
        h.set_option(10, prune)
        h.norms()
        bmu, dist = h.bmu(b.indptr, b.indices)
        b1, d1, b2, d2 = h.bmu2(b.indptr, b.indices)
        torch.cuda.synchronize()
        assert h.device_flags() == 0
        outs.append([t.cpu().numpy() for t in (bmu, dist, b1, d1, b2, d2)])
    for full, pruned in zip(*outs):
        assert np.array_equal(full.view(np.uint32) if full.dtype == np.float32 else full,
                              pruned.view(np.uint32) if pruned.dtype == np.float32 else pruned)
    rows = np.arange(0, n, 11)
    _check_against_oracle(W.cpu().numpy(), V, M, b.indptr.cpu().numpy(), b.indices.cpu().numpy(),
                          outs[1][0], outs[1][1], rows)


@pytest.mark.parametrize("mode", ["f16-8", "f16-16", "two-stage"])  # (the 8-neuron fp16 layout does not prune)
@pytest.mark.parametrize("codebook", ["recipe", "smooth", "negative"])
def test_pruning_with_fp16_rows(som_mod, mode, codebook):
    """The same for an fp16-stored codebook (maxima of the stored halves, both fp16 layouts) and with the
    two-stage search switched on over an fp32 codebook (its first pass over the fp16 copy does not prune; the
    plain fallback and the option's bookkeeping must not be disturbed by the maxima)."""
    V, M, n = 30_000, 2_048, 40_000
    W = synth.fill_codebook(V, M, 6, device="cuda")
    if codebook == "smooth":
        ramp = torch.linspace(0.0, 1.0, M, device="cuda")
        W = (W.view(V, M) * 0.2 + ramp[None, :] * torch.rand(V, 1, device="cuda")).reshape(-1).contiguous()
    elif codebook == "negative":
        W = (W - 0.3).contiguous()
    if mode != "two-stage":
        W = W.half()
    b = synth.sample_csr(n, V, 11.0, 6, device="cuda", permute_ids=True)
    outs = []
    for prune in (2, 1):
        h = som_mod.Som(V, M, W)
        h.set_option(0, 2)
        if mode == "two-stage":
            h.set_option(7, 1)
        else:
            h.set_option(3, int(mode.split("-")[1]))
        h.set_option(10, prune)
        h.norms()
        bmu, dist = h.bmu(b.indptr, b.indices)
        b1, d1, b2, d2 = h.bmu2(b.indptr, b.indices)
        torch.cuda.synchronize()
        outs.append([t.cpu().numpy() for t in (bmu, dist, b1, d1, b2, d2)])
    for full, pruned in zip(*outs):
        assert np.array_equal(full.view(np.uint32) if full.dtype == np.float32 else full,
                              pruned.view(np.uint32) if pruned.dtype == np.float32 else pruned)
    rows = np.arange(0, n, 11)
    _check_against_oracle(W.float().cpu().numpy(), V, M, b.indptr.cpu().numpy(), b.indices.cpu().numpy(),
                          outs[1][0], outs[1][1], rows)


def test_config3_full_size_sampled_rows(som_mod):
    """128x128 map at its full size (4M samples, the benchmark's launch configuration);
    a strided sample of rows against the oracle, plus properties that hold for all rows."""
    w = synth.CONFIGS[2]
    W = synth.fill_codebook(w.V, w.M, w.seed, device="cuda")
    b = synth.sample_csr(w.N, w.V, w.lam, w.seed, device="cuda")
    h, g_bmu, g_dist = _run_gpu(som_mod, W, w.V, w.M, b.indptr, b.indices)
    assert g_bmu.min() >= 0 and g_bmu.max() < w.M
    assert np.isfinite(g_dist).all() and g_dist.min() >= 0
    rows = np.concatenate([np.arange(0, w.N, 2000), [w.N - 1]])
    _check_against_oracle(W.cpu().numpy(), w.V, w.M, b.indptr.cpu().numpy(), b.indices.cpu().numpy(),
                          g_bmu, g_dist, rows)


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
            cur["x"].append((ids, int(r[0]), float(r[1])))
    return cases


@pytest.mark.parametrize("variant", [1, 2, 0])
@pytest.mark.parametrize("case", _parse_golden(), ids=lambda c: c["name"])
def test_handbuilt_cases_on_gpu(som_mod, case, variant):
    """Exactly representable weights: winner and distance must be exact, ties to the lowest index."""
    V, M = case["V"], case["M"]
    Wn = np.array([case["w"][i] for i in range(M)], np.float32)
    W = torch.from_numpy(np.ascontiguousarray(Wn.T)).cuda().reshape(-1)
    rows = [np.array(x[0], np.int32) for x in case["x"]]
    indptr = np.zeros(len(rows) + 1, np.int32)
    indptr[1:] = np.cumsum([len(r) for r in rows])
    indices = np.concatenate(rows) if rows else np.zeros(0, np.int32)
    idx_dev = torch.from_numpy(indices).cuda() if indices.size else torch.zeros(1, dtype=torch.int32, device="cuda")
    _, g_bmu, g_dist = _run_gpu(som_mod, W, V, M, torch.from_numpy(indptr).cuda(), idx_dev, variant)
    for s, (_, b1, d1) in enumerate(case["x"]):
        assert g_bmu[s] == b1 and g_dist[s] == np.float32(d1), (case["name"], s, g_bmu[s], g_dist[s])


@pytest.mark.parametrize("variant", [1, 2, 0])
@pytest.mark.parametrize("V,M,n", [(50, 1, 30), (64, 37, 200), (97, 130, 300), (40, 4, 64),
                                   (300, 260, 500), (1000, 1028, 700)])
def test_ragged_shapes(som_mod, V, M, n, variant):
    """Neuron counts that are not multiples of the vector width or of a block, tiny maps."""
    rng = np.random.default_rng(V * 1000 + M)
    W = rng.random((V, M)).astype(np.float32)
    rows = []
    for s in range(n):
        k = int(rng.integers(0, min(V, 45) + 1))  # includes empty rows and rows longer than 32
        rows.append(np.sort(rng.choice(V, size=k, replace=False)).astype(np.int32))
    indptr = np.zeros(n + 1, np.int32)
    indptr[1:] = np.cumsum([len(r) for r in rows])
    indices = np.concatenate(rows).astype(np.int32)
    _, g_bmu, g_dist = _run_gpu(som_mod, torch.from_numpy(W).cuda().reshape(-1), V, M,
                                torch.from_numpy(indptr).cuda(), torch.from_numpy(indices).cuda(), variant)
    _check_against_oracle(W, V, M, indptr, indices, g_bmu, g_dist)


def test_indptr_with_base_offset(som_mod):
    """d_indptr[0] may be any offset into d_indices (a batch cut out of a longer stream)."""
    w = synth.CONFIGS[0]
    W = synth.fill_codebook(w.V, w.M, w.seed, device="cuda")
    b = synth.sample_csr(3000, w.V, w.lam, w.seed, device="cuda")
    h = som_mod.Som(w.V, w.M, W)
    h.norms()
    full_bmu, full_dist = h.bmu(b.indptr, b.indices)
    part_bmu, part_dist = h.bmu(b.indptr[1000:2001].contiguous(), b.indices)
    torch.cuda.synchronize()
    assert torch.equal(part_bmu, full_bmu[1000:2000])
    assert torch.equal(part_dist, full_dist[1000:2000])


def test_host_entry_point_matches_device_entry_point(som_mod):
    w = synth.CONFIGS[0]
    W = synth.fill_codebook(w.V, w.M, w.seed, device="cuda")
    b = synth.sample_csr(5000, w.V, w.lam, w.seed, device="cpu")
    h = som_mod.Som(w.V, w.M, W)
    h.norms()
    d_bmu, d_dist = h.bmu(b.indptr.cuda(), b.indices.cuda())
    hb = torch.empty(b.n, dtype=torch.int32).pin_memory()
    hd = torch.empty(b.n, dtype=torch.float32).pin_memory()
    h.bmu_host(b.indptr.pin_memory(), b.indices.pin_memory(), hb, hd)
    assert torch.equal(hb, d_bmu.cpu()) and torch.equal(hd, d_dist.cpu())


def test_status_codes_and_noops(som_mod):
    w = synth.CONFIGS[0]
    W = synth.fill_codebook(w.V, w.M, w.seed, device="cuda")
    b = synth.sample_csr(100, w.V, w.lam, w.seed, device="cuda")
    h = som_mod.Som(w.V, w.M, W)
    with pytest.raises(som_mod.SomError) as e:
        h.bmu(b.indptr, b.indices)  # norms not computed yet
    assert e.value.status == 2
    h.norms()
    # n = 0 is a successful no-op
    out_b, out_d = h.bmu(b.indptr[:1].contiguous(), b.indices)
    assert out_b.numel() == 0 and out_d.numel() == 0
    # validator: unsorted row, out-of-range id
    bad = b.indices.clone()
    bad[0], bad[1] = b.indices[1], b.indices[0]
    if int(b.indptr[1]) >= 2:
        assert not h.validate_csr(b.indptr, bad)
    bad = b.indices.clone()
    bad[-1] = w.V
    assert not h.validate_csr(b.indptr, bad)
    assert h.validate_csr(b.indptr, b.indices)
    # invalid arguments at creation
    with pytest.raises(som_mod.SomError):
        som_mod.Som(0, 0, W[:0])
    lib = som_mod.load_library()
    assert lib.som_status_string(5) == b"SOM_ERR_BAD_CSR"
    assert lib.som_destroy(None) == 0


def test_norms_follow_codebook_update(som_mod):
    """After an in-place codebook update som_norms must be rerun; then results follow the new weights."""
    V, M, n = 200, 64, 400
    rng = np.random.default_rng(3)
    W = torch.from_numpy(rng.random((V, M)).astype(np.float32)).cuda().reshape(-1)
    b = synth.sample_csr(n, V, 7.0, seed=1, device="cuda")
    h = som_mod.Som(V, M, W)
    h.norms()
    h.bmu(b.indptr, b.indices)
    W.mul_(0.5)
    W[5::M] += 0.25
    h.norms()
    g_bmu, g_dist = h.bmu(b.indptr, b.indices)
    torch.cuda.synchronize()
    _check_against_oracle(W.cpu().numpy(), V, M, b.indptr.cpu().numpy(), b.indices.cpu().numpy(),
                          g_bmu.cpu().numpy(), g_dist.cpu().numpy())


@pytest.mark.parametrize("cfg", [3, 4])
def test_large_configs_full_size_sampled_rows(som_mod, cfg):
    """512x512 (31.5 GB codebook) and 1024x1024 (125.8 GB, resident in HBM): all four batches of the
    configuration at the batch size the benchmark uses.  More than 20 000 rows (5 000 per batch, evenly
    spread, the first and last row of every batch among them) are checked against the oracle, which
    reads the device codebook slab by slab; their hit-count histogram is compared inside the parity
    rule.  For every sample of every batch the reported distance must be the fp64 distance to the
    reported neuron (Eq. 1, from the stored weights and the oracle's norms) within 1e-5 relative."""
    w = synth.CONFIGS[cfg]
    import gc
    gc.collect()  # handles and tensors of earlier tests
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    need = w.V * w.M * 4 + (8 << 30)
    if free < need:
        pytest.skip("needs %.0f GB of free device memory" % (need / 1e9))
    W = torch.empty(w.V * w.M, dtype=torch.float32, device="cuda")
    synth.fill_codebook(w.V, w.M, w.seed, out=W)
    h = som_mod.Som(w.V, w.M, W)
    h.norms()
    n_batches = w.N // w.batch
    assert n_batches == 4
    per_batch = 5000
    sub_ptr, sub_idx, sub_bmu, sub_dist, full = [], [], [], [], []
    for bi in range(n_batches):
        b = synth.sample_csr(w.batch, w.V, w.lam, w.seed, device="cuda", first_sample=bi * w.batch)
        bmu, dist = h.bmu(b.indptr, b.indices)
        torch.cuda.synchronize()
        g_bmu, g_dist = bmu.cpu().numpy(), dist.cpu().numpy()
        assert g_bmu.min() >= 0 and g_bmu.max() < w.M
        assert np.isfinite(g_dist).all() and g_dist.min() >= 0
        ip, ix = b.indptr.cpu().numpy(), b.indices.cpu().numpy()
        rows = largemap.sample_rows(w.batch, per_batch)
        assert rows[0] == 0 and rows[-1] == w.batch - 1
        p, x = largemap.subset_csr(ip, ix, rows)
        sub_ptr.append(p)
        sub_idx.append(x)
        sub_bmu.append(g_bmu[rows])
        sub_dist.append(g_dist[rows])
        full.append((ip, ix, g_bmu, g_dist))
        del b, bmu, dist
    # one oracle pass over the union of the sampled rows
    ptr = np.zeros(1, np.int64)
    for p in sub_ptr:
        ptr = np.concatenate([ptr, ptr[-1] + p[1:].astype(np.int64)])
    ptr = ptr.astype(np.int32)
    idx = np.concatenate(sub_idx)
    g_sub, gd_sub = np.concatenate(sub_bmu), np.concatenate(sub_dist)
    assert g_sub.size >= 20000
    top2, norms = largemap.oracle_top2_slabbed(W, w.V, w.M, ptr, idx)
    d_at = largemap.dist_to_named_neuron(W, w.V, w.M, ptr, idx, g_sub, norms)
    rep = parity.check(g_sub, gd_sub, top2, d_at, w.M)
    assert rep.ok, str(rep)
    assert rep.unambiguous > 0.9 * g_sub.size
    # every sample of every batch: reported distance == fp64 distance to the reported neuron
    for ip, ix, g_bmu, g_dist in full:
        d_all = largemap.dist_to_named_neuron(W, w.V, w.M, ip, ix, g_bmu, norms)
        err = np.abs(g_dist.astype(np.float64) - d_all)
        assert np.all(err <= parity.DIST_REL * np.abs(d_all) + parity.DIST_ABS), float(err.max())
    # norms of the library against the oracle's, all neurons
    np.testing.assert_allclose(h.get_norms().cpu().numpy().astype(np.float64), norms, rtol=2e-7)
    h.destroy()
    del W
    torch.cuda.empty_cache()


@pytest.mark.parametrize("variant", [1, 2, 0])
def test_batch_of_empty_samples(som_mod, variant):
    """Every sample empty (nnz = 0, no index array needed): each gets argmin ||w_i||^2 and that norm."""
    V, M, n = 500, 1_024, 100_000
    W = synth.fill_codebook(V, M, 8, device="cuda")
    indptr = torch.zeros(n + 1, dtype=torch.int32, device="cuda")
    indices = torch.zeros(1, dtype=torch.int32, device="cuda")
    h = som_mod.Som(V, M, W)
    h.set_option(0, variant)
    h.norms()
    bmu, dist = h.bmu(indptr, indices)
    torch.cuda.synchronize()
    nn = orc.norms(W.cpu().numpy(), V, M)
    best = int(np.argmin(nn.astype(np.float32)))
    assert np.all(bmu.cpu().numpy() == best)
    np.testing.assert_allclose(dist.cpu().numpy(), np.float32(nn[best]), rtol=1e-6)


def test_streamed_host_entry_point(som_mod):
    """som_bmu_host_async over a stream of different batches equals som_bmu on each of them."""
    w = synth.CONFIGS[0]
    W = synth.fill_codebook(w.V, w.M, w.seed, device="cuda")
    h = som_mod.Som(w.V, w.M, W)
    h.norms()
    batches = [synth.sample_csr(4000 + 500 * k, w.V, w.lam, w.seed, device="cpu", first_sample=10_000 * k)
               for k in range(5)]
    pinned = [(b.indptr.pin_memory(), b.indices.pin_memory()) for b in batches]
    outs = [(torch.empty(b.n, dtype=torch.int32).pin_memory(), torch.empty(b.n, dtype=torch.float32).pin_memory())
            for b in batches]
    for (ip, ix), (ob, od) in zip(pinned, outs):
        h.bmu_host_async(ip, ix, ob, od)
    h.host_sync()
    for b, (ob, od) in zip(batches, outs):
        d_bmu, d_dist = h.bmu(b.indptr.cuda(), b.indices.cuda())
        torch.cuda.synchronize()
        assert torch.equal(ob, d_bmu.cpu()) and torch.equal(od.view(torch.int32), d_dist.cpu().view(torch.int32))


@pytest.mark.parametrize("variant", [0, 1, 2])
def test_reusable_plan_matches_som_bmu(som_mod, variant):
    """A plan built once serves several epochs: after each in-place change of the codebook (and
    som_norms) the planned search equals som_bmu bit for bit, and both obey the oracle."""
    V, M, n = 30_000, 1_024, 60_000
    W = synth.fill_codebook(V, M, 4, device="cuda")
    b = synth.sample_csr(n, V, 11.0, 4, device="cuda")
    h = som_mod.Som(V, M, W)
    h.set_option(0, variant)
    plan = h.plan(b.indptr, b.indices)
    for epoch in range(3):
        if epoch:
            W.mul_(0.9)
            W[epoch::7] += 0.01
        h.norms()
        p_bmu, p_dist = plan.bmu()
        d_bmu, d_dist = h.bmu(b.indptr, b.indices)
        torch.cuda.synchronize()
        assert torch.equal(p_bmu, d_bmu) and torch.equal(p_dist.view(torch.int32), d_dist.view(torch.int32))
    _check_against_oracle(W.cpu().numpy(), V, M, b.indptr.cpu().numpy(), b.indices.cpu().numpy(),
                          p_bmu.cpu().numpy(), p_dist.cpu().numpy(), np.arange(0, n, 9))
    plan.destroy()
    # a plan is tied to its handle
    other = som_mod.Som(V, M, W)
    other.norms()
    plan2 = h.plan(b.indptr, b.indices)
    rc = other._lib.som_bmu_planned(other._h, plan2._p, p_bmu.data_ptr(), p_dist.data_ptr(), None)
    assert rc == 1  # SOM_ERR_INVALID_ARG


@pytest.mark.parametrize("variant,store,two_stage", [(1, "f32", False), (2, "f32", False), (2, "f16", False),
                                                      (2, "f32", True)])
def test_search_on_a_smoothed_map(som_mod, variant, store, two_stage):
    """A map right after a batch update with a wide blur (built by the update ORACLE from random
    assignments): neighbouring units are nearly equal, so near ties abound.  Every kernel must stay
    inside the parity rule there, and the two-stage search must fall back to exact scores."""
    from oracle import som_update_oracle as uorc
    V, rows, cols, n = 2_000, 32, 32, 70_000
    M = rows * cols
    rng = np.random.default_rng(21)
    b = synth.sample_csr(n, V, 7.0, 6, device="cpu")
    ip, ix = b.indptr.numpy(), b.indices.numpy()
    W0 = synth.fill_codebook(V, M, 6, device="cpu").numpy()
    assign = rng.integers(0, M, size=n).astype(np.int32)
    W_host = uorc.update(W0, V, rows, cols, ip, ix, assign, 5).astype(np.float32)
    if store == "f16":
        W_dev = torch.from_numpy(W_host).cuda().half()
        W_host = W_dev.float().cpu().numpy()  # the oracle sees the stored values
    else:
        W_dev = torch.from_numpy(W_host).cuda()
    h = som_mod.Som(V, M, W_dev)
    h.set_option(0, variant)
    if two_stage:
        h.set_option(7, 1)
    h.norms()
    g_bmu, g_dist = h.bmu(b.indptr.cuda(), b.indices.cuda())
    torch.cuda.synchronize()
    if two_stage:
        assert h.last_uncertain() > n // 5
    rep = _check_against_oracle(W_host, V, M, ip, ix, g_bmu.cpu().numpy(), g_dist.cpu().numpy(), np.arange(0, n, 7))
    assert rep.near_ties > 0
