"""GPU parity tests of the fp16-stored codebook (som_create_f16: fp16 storage, fp32 accumulation).

The oracle is given the same weights widened to fp32 (exact), so the rule and the tolerances are
those of the fp32 path.
"""
import numpy as np
import pytest
import torch

from oracle import parity
from oracle import som_oracle as orc
from paper_2608_24067_b200 import synth

import largemap

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def som_mod():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_24067_b200 import som
    som.load_library()  # fail loudly when the extension is missing
    return som


def _subset(indptr, indices, rows):
    indptr = np.asarray(indptr, dtype=np.int64)
    lens = indptr[rows + 1] - indptr[rows]
    out_ptr = np.zeros(len(rows) + 1, np.int32)
    out_ptr[1:] = np.cumsum(lens)
    out_idx = np.concatenate([indices[indptr[r]:indptr[r + 1]] for r in rows]).astype(np.int32)
    return out_ptr, out_idx


def _run_and_check(som_mod, W16, V, M, indptr_dev, indices_dev, variant=None, options=(), rows=None,
                   check_norms=True):
    """W16: fp16 CUDA tensor.  Runs som_bmu2 (and som_bmu, which must agree on the best unit) and
    checks both units against the oracle on the widened weights."""
    h = som_mod.Som(V, M, W16)
    if variant is not None:
        h.set_option(0, variant)
    for key, value in options:
        h.set_option(key, value)
    h.norms()
    one = h.bmu(indptr_dev, indices_dev)
    two = h.bmu2(indptr_dev, indices_dev)
    torch.cuda.synchronize()
    assert torch.equal(one[0], two[0]) and torch.equal(one[1].view(torch.int32), two[1].view(torch.int32))
    g1, gd1, g2, gd2 = [t.cpu().numpy() for t in two]
    W_host = W16.float().cpu().numpy()
    indptr, indices = indptr_dev.cpu().numpy(), indices_dev.cpu().numpy()
    if rows is not None:
        indptr, indices = _subset(indptr, indices, rows)
        g1, gd1, g2, gd2 = g1[rows], gd1[rows], g2[rows], gd2[rows]
    nn = orc.norms(W_host, V, M)
    if check_norms:
        np.testing.assert_allclose(h.get_norms().cpu().numpy().astype(np.float64), nn, rtol=2e-7)
    top2 = orc.bmu(W_host, V, M, indptr, indices, norms_=nn)
    d_at1 = orc.dist_at(W_host, V, M, indptr, indices, np.clip(g1.astype(np.int64), 0, M - 1), norms_=nn)
    rep1 = parity.check(g1, gd1, top2, d_at1, M)
    assert rep1.ok, str(rep1)
    if M >= 2:
        d_at2 = orc.dist_at(W_host, V, M, indptr, indices, np.clip(g2.astype(np.int64), 0, M - 1), norms_=nn)
        rep2 = parity.check_second(g1, g2, gd2, top2, d_at2, M)
        assert rep2.ok, str(rep2)
    return rep1


@pytest.mark.parametrize("variant", [1, 2, 0])
@pytest.mark.parametrize("kind", ["zipf", "permuted", "uniform"])
def test_f16_config1_full(som_mod, kind, variant):
    """Tiny 16x16 configuration, every sample, both kernels."""
    w = synth.CONFIGS[0]
    W16 = synth.fill_codebook(w.V, w.M, w.seed, device="cuda").half()
    b = synth.sample_csr(w.N, w.V, w.lam, w.seed, device="cuda",
                         zipf_s=0.0 if kind == "uniform" else w.zipf_s, permute_ids=(kind == "permuted"))
    rep = _run_and_check(som_mod, W16, w.V, w.M, b.indptr, b.indices, variant)
    assert rep.near_ties < 0.01 * w.N


@pytest.mark.parametrize("variant", [1, 2, 0])
def test_f16_config2_sampled_rows(som_mod, variant):
    """64x64 map, one million samples on the GPU; every 40th row against the oracle."""
    w = synth.CONFIGS[1]
    W16 = synth.fill_codebook(w.V, w.M, w.seed, device="cuda").half()
    b = synth.sample_csr(w.N, w.V, w.lam, w.seed, device="cuda")
    rows = np.concatenate([np.arange(0, w.N, 40), [w.N - 1]])
    rep = _run_and_check(som_mod, W16, w.V, w.M, b.indptr, b.indices, variant, rows=rows)
    assert rep.near_ties < 0.05 * rows.size


@pytest.mark.parametrize("lane_neurons,threads", [(8, 640), (8, 896), (8, 1024), (16, 512), (16, 640)])
def test_f16_row_table_geometries(som_mod, lane_neurons, threads):
    """Both fp16 layouts of the row-table kernel (64- and 128-neuron ranges) and block sizes."""
    V, M, n = 30_000, 1_024, 60_000
    W16 = synth.fill_codebook(V, M, 3, device="cuda").half()
    b = synth.sample_csr(n, V, 11.0, 3, device="cuda", permute_ids=True)
    _run_and_check(som_mod, W16, V, M, b.indptr, b.indices, 2, options=((3, lane_neurons), (2, threads)),
                   rows=np.arange(0, n, 7))


@pytest.mark.parametrize("variant", [1, 2, 0])
@pytest.mark.parametrize("V,M,n", [(50, 1, 30), (64, 37, 200), (97, 130, 300), (40, 4, 64), (40, 8, 64),
                                   (300, 264, 500), (500, 320, 700), (1000, 1028, 700)])
def test_f16_ragged_shapes(som_mod, V, M, n, variant):
    """Neuron counts that are not multiples of the vector widths (2, 4, 8, 64), tiny maps."""
    rng = np.random.default_rng(V * 1000 + M)
    W16 = torch.from_numpy(rng.random((V, M)).astype(np.float32)).cuda().half().reshape(-1)
    rows = []
    for s in range(n):
        k = int(rng.integers(0, min(V, 45) + 1))  # includes empty rows and rows longer than 32
        rows.append(np.sort(rng.choice(V, size=k, replace=False)).astype(np.int32))
    indptr = np.zeros(n + 1, np.int32)
    indptr[1:] = np.cumsum([len(r) for r in rows])
    indices = np.concatenate(rows).astype(np.int32)
    _run_and_check(som_mod, W16, V, M, torch.from_numpy(indptr).cuda(), torch.from_numpy(indices).cuda(), variant)


def test_f16_matches_fp32_handle_on_the_same_values(som_mod):
    """Widening is exact, so an fp32 handle over the widened weights ranks the neurons by the same
    real-valued scores; the two handles may differ only inside the near-tie band (their fp32
    summation orders differ), and both reported distances come from the same fp64 recomputation."""
    w = synth.CONFIGS[0]
    W16 = synth.fill_codebook(w.V, w.M, w.seed, device="cuda").half()
    W32 = W16.float()
    b = synth.sample_csr(w.N, w.V, w.lam, w.seed, device="cuda")
    h16, h32 = som_mod.Som(w.V, w.M, W16), som_mod.Som(w.V, w.M, W32)
    h16.norms(); h32.norms()
    assert torch.equal(h16.get_norms(), h32.get_norms())
    b16, d16 = h16.bmu(b.indptr, b.indices)
    b32, d32 = h32.bmu(b.indptr, b.indices)
    torch.cuda.synchronize()
    same = (b16 == b32)
    assert same.float().mean().item() > 0.99
    assert torch.equal(d16[same], d32[same])


def test_f16_largest_map_full_size_sampled_rows(som_mod):
    """1024x1024 map stored in fp16 (62.9 GB, resident in HBM) at the batch size the benchmark
    uses, through som_bmu2, all four batches: 5 000 rows per batch (first and last among them) are
    checked against the oracle, which reads the device codebook slab by slab; for every sample both
    reported distances must be the fp64 distances to the reported neurons within 1e-5 relative."""
    w = synth.CONFIGS[4]
    import gc
    gc.collect()  # handles and tensors of earlier tests
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    need = w.V * w.M * 2 + (8 << 30)
    if free < need:
        pytest.skip("needs %.0f GB of free device memory" % (need / 1e9))
    W16 = torch.empty(w.V * w.M, dtype=torch.float16, device="cuda")
    synth.fill_codebook(w.V, w.M, w.seed, out=W16)
    h = som_mod.Som(w.V, w.M, W16)
    h.norms()
    subs, full = [], []
    for bi in range(w.N // w.batch):
        b = synth.sample_csr(w.batch, w.V, w.lam, w.seed, device="cuda", first_sample=bi * w.batch)
        g1, gd1, g2, gd2 = [t.cpu().numpy() for t in h.bmu2(b.indptr, b.indices)]
        assert g1.min() >= 0 and g1.max() < w.M and g2.min() >= 0 and g2.max() < w.M
        assert np.all(g1 != g2) and np.isfinite(gd1).all() and np.isfinite(gd2).all()
        ip, ix = b.indptr.cpu().numpy(), b.indices.cpu().numpy()
        rows = largemap.sample_rows(w.batch, 5000)
        p, x = largemap.subset_csr(ip, ix, rows)
        subs.append((p, x, g1[rows], gd1[rows], g2[rows], gd2[rows]))
        full.append((ip, ix, g1, gd1, g2, gd2))
        del b
    ptr = np.zeros(1, np.int64)
    for s_ in subs:
        ptr = np.concatenate([ptr, ptr[-1] + s_[0][1:].astype(np.int64)])
    ptr = ptr.astype(np.int32)
    idx = np.concatenate([s_[1] for s_ in subs])
    sg1, sd1, sg2, sd2 = [np.concatenate([s_[k] for s_ in subs]) for k in (2, 3, 4, 5)]
    assert sg1.size >= 20000
    top2, norms = largemap.oracle_top2_slabbed(W16, w.V, w.M, ptr, idx)
    rep1 = parity.check(sg1, sd1, top2, largemap.dist_to_named_neuron(W16, w.V, w.M, ptr, idx, sg1, norms), w.M)
    assert rep1.ok, str(rep1)
    rep2 = parity.check_second(sg1, sg2, sd2, top2,
                               largemap.dist_to_named_neuron(W16, w.V, w.M, ptr, idx, sg2, norms), w.M)
    assert rep2.ok, str(rep2)
    for ip, ix, g1, gd1, g2, gd2 in full:
        for g, gd in ((g1, gd1), (g2, gd2)):
            d_all = largemap.dist_to_named_neuron(W16, w.V, w.M, ip, ix, g, norms)
            err = np.abs(gd.astype(np.float64) - d_all)
            assert np.all(err <= parity.DIST_REL * np.abs(d_all) + parity.DIST_ABS), float(err.max())
    np.testing.assert_allclose(h.get_norms().cpu().numpy().astype(np.float64), norms, rtol=2e-7)
    h.destroy()
    del W16
    torch.cuda.empty_cache()
