"""GPU parity tests of the batch update (som_update) against the CPU update oracle.

Tolerance: the fields between the six box passes are stored in fp32 (five roundings of 2^-24
each in numerator and denominator), the running sums are fp64 and the quotient is rounded once
to the storage type, so the new weights agree with the fp64 oracle within 1e-6 relative
(plus one fp16 ulp, 2^-11 relative, when the codebook is stored in fp16).  Prototypes of
neurons outside the reach of every sample must be bit-identical to the old ones.
"""
import numpy as np
import pytest
import torch

from oracle import som_update_oracle as uorc
from paper_2608_24067_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def som_mod():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_24067_b200 import som
    som.load_library()  # fail loudly when the extension is missing
    return som


def _problem(seed, V, rows, cols, n, spread=None):
    rng = np.random.default_rng(seed)
    M = rows * cols
    samples = [np.sort(rng.choice(V, size=int(rng.integers(1, min(V, 9) + 1)), replace=False)).astype(np.int32)
               for _ in range(n)]
    indptr = np.zeros(n + 1, np.int32)
    indptr[1:] = np.cumsum([len(r) for r in samples])
    indices = np.concatenate(samples).astype(np.int32) if n else np.zeros(0, np.int32)
    if spread is None:
        bmu = rng.integers(0, M, size=n).astype(np.int32)
    else:  # samples confined to the top-left spread x spread cells
        bmu = (rng.integers(0, spread, size=n) * cols + rng.integers(0, spread, size=n)).astype(np.int32)
    W_old = rng.random(V * M).astype(np.float32)
    return indptr, indices, bmu, W_old


def _run(som_mod, W_old, V, rows, cols, indptr, indices, bmu, radius, dtype=torch.float32, options=()):
    W = torch.from_numpy(W_old).cuda().to(dtype)
    h = som_mod.Som(V, rows * cols, W)
    for k, v in options:
        h.set_option(k, v)
    idx = torch.from_numpy(indices).cuda() if indices.size else torch.zeros(1, dtype=torch.int32, device="cuda")
    bm = torch.from_numpy(bmu).cuda() if bmu.size else torch.zeros(1, dtype=torch.int32, device="cuda")
    h.update(rows, cols, torch.from_numpy(indptr).cuda(), idx, bm, radius)
    torch.cuda.synchronize()
    if indptr.size > 1:
        with pytest.raises(som_mod.SomError):  # the norms are stale after an update
            h.bmu(torch.from_numpy(indptr).cuda(), idx)
    return W.float().cpu().numpy().astype(np.float64)


def _check(got, W_old_stored, V, rows, cols, indptr, indices, bmu, radius, rtol):
    want = uorc.update(W_old_stored, V, rows, cols, indptr, indices, bmu, radius)
    np.testing.assert_allclose(got, want, rtol=rtol, atol=1e-12)
    # neurons outside every sample's reach: bit-identical old prototypes
    occ = np.zeros((rows, cols))
    if bmu.size:
        occ[bmu // cols, bmu % cols] = 1
    reach = uorc.blur(occ, rows, cols, 3 * radius, 1).reshape(-1) > 0
    got2, old2 = got.reshape(V, -1), W_old_stored.astype(np.float64).reshape(V, -1)
    assert np.array_equal(got2[:, ~reach], old2[:, ~reach])
    return int((~reach).sum())


@pytest.mark.parametrize("V,rows,cols,n,radius", [
    (40, 8, 8, 300, 1), (64, 16, 16, 2000, 2), (33, 12, 20, 500, 3), (50, 32, 32, 5000, 5),
    (20, 7, 5, 100, 1), (17, 16, 16, 400, 16), (25, 1, 40, 200, 2), (25, 40, 1, 200, 2),
    (30, 9, 9, 0, 1), (12, 64, 64, 3000, 0), (70, 33, 65, 4000, 4),
    # more than 4096 cells: fp32 plane buffers in shared memory; more than 16384: the passes go
    # through device memory
    (6, 72, 80, 3000, 3), (5, 66, 64, 2000, 70), (4, 300, 20, 1500, 2), (3, 128, 128, 4000, 9),
    (3, 130, 130, 2000, 4), (2, 2000, 9, 1500, 2),
    # the strip route (rows, then column strips, through shared memory): square and oblong lattices,
    # windows shorter and much longer than a thread's segment, a radius beyond the lattice
    (2, 512, 512, 20000, 37), (2, 512, 512, 3000, 1), (2, 40, 1000, 3000, 5), (1, 3000, 11, 2000, 3),
    (2, 256, 300, 5000, 128), (1, 1024, 1024, 50000, 200), (2, 200, 150, 4000, 400),
    # shapes beyond the strip route's shared memory: the passes through device memory
    (1, 5000, 8, 3000, 2), (1, 3, 30000, 3000, 6)])
def test_update_matches_oracle(som_mod, V, rows, cols, n, radius):
    indptr, indices, bmu, W_old = _problem(V * 7 + rows, V, rows, cols, n)
    got = _run(som_mod, W_old, V, rows, cols, indptr, indices, bmu, radius)
    _check(got, W_old, V, rows, cols, indptr, indices, bmu, radius, rtol=1e-6)


@pytest.mark.parametrize("radius", [1, 2])
def test_update_leaves_unreached_neurons(som_mod, radius):
    """All samples in one corner of a 40 x 40 lattice: most neurons keep their prototype."""
    V, rows, cols, n = 30, 40, 40, 500
    indptr, indices, bmu, W_old = _problem(9, V, rows, cols, n, spread=4)
    got = _run(som_mod, W_old, V, rows, cols, indptr, indices, bmu, radius)
    untouched = _check(got, W_old, V, rows, cols, indptr, indices, bmu, radius, rtol=1e-6)
    assert untouched > rows * cols // 2


def test_update_in_slabs_equals_single_slab(som_mod):
    """A small workspace budget makes the update walk the features in several slabs."""
    V, rows, cols, n, radius = 300, 64, 64, 20000, 3
    indptr, indices, bmu, W_old = _problem(4, V, rows, cols, n)
    whole = _run(som_mod, W_old, V, rows, cols, indptr, indices, bmu, radius)
    slabs = _run(som_mod, W_old, V, rows, cols, indptr, indices, bmu, radius, options=((6, 1),))  # 1 MiB: 32 planes
    assert np.array_equal(whole, slabs)
    _check(whole, W_old, V, rows, cols, indptr, indices, bmu, radius, rtol=1e-6)


def test_update_of_fp16_codebook_on_a_large_lattice(som_mod):
    V, rows, cols, n, radius = 3, 192, 160, 6000, 7
    indptr, indices, bmu, W_old = _problem(16, V, rows, cols, n)
    W_old16 = torch.from_numpy(W_old).half().float().numpy()
    got = _run(som_mod, W_old16, V, rows, cols, indptr, indices, bmu, radius, dtype=torch.float16)
    _check(got, W_old16, V, rows, cols, indptr, indices, bmu, radius, rtol=2.0 ** -11 + 1e-6)


def test_update_of_fp16_codebook(som_mod):
    V, rows, cols, n, radius = 60, 16, 16, 3000, 2
    indptr, indices, bmu, W_old = _problem(6, V, rows, cols, n, spread=6)
    W_old16 = torch.from_numpy(W_old).half().float().numpy()  # what the fp16 codebook holds
    got = _run(som_mod, W_old16, V, rows, cols, indptr, indices, bmu, radius, dtype=torch.float16)
    _check(got, W_old16, V, rows, cols, indptr, indices, bmu, radius, rtol=2.0 ** -11 + 1e-6)


def test_epoch_on_synthetic_workload(som_mod):
    """One epoch of the tiny configuration end to end: search, update, norms, search again.  The
    update is driven by the ORACLE's assignment (no oracle input comes from the CUDA path; the
    GPU's own assignment is checked against it first), and compared with the update oracle."""
    from oracle import parity
    from oracle import som_oracle as orc
    w = synth.CONFIGS[0]
    rows = cols = 16
    W = synth.fill_codebook(w.V, w.M, w.seed, device="cuda")
    W_old = W.cpu().numpy().copy()
    b = synth.sample_csr(w.N, w.V, w.lam, w.seed, device="cuda")
    ip, ix = b.indptr.cpu().numpy(), b.indices.cpu().numpy()
    h = som_mod.Som(w.V, w.M, W)
    h.norms()
    bmu, dist = h.bmu(b.indptr, b.indices)
    torch.cuda.synchronize()
    nn = orc.norms(W_old, w.V, w.M)
    top2 = orc.bmu(W_old, w.V, w.M, ip, ix, norms_=nn)
    g = bmu.cpu().numpy()
    rep = parity.check(g, dist.cpu().numpy(), top2, orc.dist_at(W_old, w.V, w.M, ip, ix, g.astype(np.int64), norms_=nn), w.M)
    assert rep.ok, str(rep)
    assign = top2.b1.astype(np.int32)
    h.update(rows, cols, b.indptr, b.indices, torch.from_numpy(assign).cuda(), 4)
    h.norms()
    bmu2, dist2 = h.bmu(b.indptr, b.indices)
    torch.cuda.synchronize()
    want = uorc.update(W_old, w.V, rows, cols, ip, ix, assign, 4)
    np.testing.assert_allclose(W.cpu().numpy().astype(np.float64), want, rtol=1e-6, atol=1e-12)
    assert np.isfinite(dist2.cpu().numpy()).all()


@pytest.mark.parametrize("mib", [0, 1])
def test_update_with_frequent_features_counted_on_chip(som_mod, mib):
    """Many samples on a small lattice with Zipf-shaped features: the most frequent features take the
    shared-memory counting path; with a 1 MiB budget they are spread over four feature slabs."""
    w = synth.CONFIGS[0]
    rows = cols = 16
    rng = np.random.default_rng(12)
    W_old = rng.random(w.V * w.M).astype(np.float32)
    b = synth.sample_csr(60_000, w.V, w.lam, 4, device="cpu")
    bmu = rng.integers(0, w.M, size=b.n).astype(np.int32)
    got = _run(som_mod, W_old, w.V, rows, cols, b.indptr.numpy(), b.indices.numpy(), bmu, 2,
               options=((6, mib),) if mib else ())
    _check(got, W_old, w.V, rows, cols, b.indptr.numpy(), b.indices.numpy(), bmu, 2, rtol=1e-6)


def test_update_with_frequent_features_on_the_strip_route(som_mod):
    """A 130 x 130 lattice (above the on-chip blur, so the strip kernels run, which take the counts in neuron
    order) with enough Zipf-shaped samples for the frequent features' shared-memory counting path: both
    scatters must write the order the strips read."""
    V, rows, cols = 300, 130, 130
    rng = np.random.default_rng(21)
    W_old = rng.random(V * rows * cols).astype(np.float32)
    b = synth.sample_csr(150_000, V, 6.0, 8, device="cpu")
    bmu = rng.integers(0, rows * cols, size=b.n).astype(np.int32)
    got = _run(som_mod, W_old, V, rows, cols, b.indptr.numpy(), b.indices.numpy(), bmu, 5)
    _check(got, W_old, V, rows, cols, b.indptr.numpy(), b.indices.numpy(), bmu, 5, rtol=1e-6)


def test_update_at_benchmark_shape(som_mod):
    """The shape the benchmark times: a 64 x 64 lattice, V = 30 000, one million Zipf-shaped samples,
    radius 16 (edge / 4).  The frequent features take the on-chip counting path, the blur runs fused
    in shared memory; every one of the 122 880 000 new weights is compared with the update oracle."""
    w = synth.CONFIGS[1]
    rows = cols = 64
    rng = np.random.default_rng(31)
    W_old = synth.fill_codebook(w.V, w.M, w.seed, device="cpu").numpy()
    b = synth.sample_csr(w.batch, w.V, w.lam, w.seed, device="cpu")
    assert b.n >= 1_000_000
    ip, ix = b.indptr.numpy(), b.indices.numpy()
    bmu = rng.integers(0, w.M, size=b.n).astype(np.int32)
    got = _run(som_mod, W_old, w.V, rows, cols, ip, ix, bmu, 16)
    want = uorc.update(W_old, w.V, rows, cols, ip, ix, bmu, 16)
    np.testing.assert_allclose(got, want, rtol=1e-6, atol=1e-12)


def test_update_with_a_huge_radius_equals_a_radius_that_spans_the_lattice(som_mod):
    V, rows, cols, n = 9, 12, 20, 300
    indptr, indices, bmu, W_old = _problem(2, V, rows, cols, n)
    huge = _run(som_mod, W_old, V, rows, cols, indptr, indices, bmu, 2 ** 30)
    spans = _run(som_mod, W_old, V, rows, cols, indptr, indices, bmu, 20)
    assert np.array_equal(huge, spans)
    _check(spans, W_old, V, rows, cols, indptr, indices, bmu, 20, rtol=1e-6)


def test_update_rejects_bad_lattice(som_mod):
    V, rows, cols = 10, 4, 4
    W = torch.zeros(V * rows * cols, device="cuda")
    h = som_mod.Som(V, rows * cols, W)
    z = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(som_mod.SomError):
        h.update(rows, cols + 1, z, z, z, 1)
    with pytest.raises(som_mod.SomError):
        h.update(rows, cols, z, z, z, -1)
