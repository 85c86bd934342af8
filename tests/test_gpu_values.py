"""GPU parity tests of the search for sparse real-valued samples (som_bmu_values) against the oracle.

Parity rule as for the binary search: exact best unit outside the 1e-4 relative near-tie band,
distance within 1e-5 relative of the fp64 distance to the reported unit."""
import numpy as np
import pytest
import torch

from oracle import parity
from oracle import som_oracle as orc
from paper_2608_24067_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def som_mod():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_24067_b200 import som
    som.load_library()  # fail loudly when the extension is missing
    return som


def _values_for(b, seed, signed):
    """Seeded sample values: tf-idf-like positive weights, or signed ones."""
    g = torch.Generator(device="cpu").manual_seed(seed)
    x = torch.rand(b.indices.numel(), generator=g) * 1.5 + 0.25
    if signed:
        x = x * (torch.randint(0, 2, x.shape, generator=g) * 2 - 1)
    return x.float()


def _check(W_host, V, M, indptr, indices, values, g_bmu, g_dist):
    nn = orc.norms(W_host, V, M)
    top2 = orc.bmu_values(W_host, V, M, indptr, indices, values, norms_=nn)
    d_at = orc.dist_at_values(W_host, V, M, indptr, indices, values, np.clip(g_bmu.astype(np.int64), 0, M - 1), norms_=nn)
    rep = parity.check(g_bmu, g_dist, top2, d_at, M)
    assert rep.ok, str(rep)
    return rep


@pytest.mark.parametrize("dtype", [torch.float32, torch.float16])
@pytest.mark.parametrize("signed", [False, True])
def test_values_config1_full(som_mod, signed, dtype):
    w = synth.CONFIGS[0]
    W = synth.fill_codebook(w.V, w.M, w.seed, device="cuda").to(dtype)
    b = synth.sample_csr(w.N, w.V, w.lam, w.seed, device="cpu")
    x = _values_for(b, 3, signed)
    h = som_mod.Som(w.V, w.M, W)
    h.norms()
    bmu, dist = h.bmu_values(b.indptr.cuda(), b.indices.cuda(), x.cuda())
    again = h.bmu_values(b.indptr.cuda(), b.indices.cuda(), x.cuda())
    torch.cuda.synchronize()
    assert torch.equal(bmu, again[0]) and torch.equal(dist.view(torch.int32), again[1].view(torch.int32))
    rep = _check(W.float().cpu().numpy(), w.V, w.M, b.indptr.numpy(), b.indices.numpy(), x.numpy(),
                 bmu.cpu().numpy(), dist.cpu().numpy())
    assert rep.near_ties < 0.02 * w.N


def test_values_all_ones_equal_the_binary_search(som_mod):
    w = synth.CONFIGS[0]
    W = synth.fill_codebook(w.V, w.M, w.seed, device="cuda")
    b = synth.sample_csr(w.N, w.V, w.lam, w.seed, device="cuda")
    h = som_mod.Som(w.V, w.M, W)
    h.set_option(0, 1)  # the direct-load kernel: same summation order as the valued search
    h.norms()
    b1, d1 = h.bmu(b.indptr, b.indices)
    b2, d2 = h.bmu_values(b.indptr, b.indices, torch.ones(b.indices.numel(), device="cuda"))
    torch.cuda.synchronize()
    assert torch.equal(b1, b2) and torch.equal(d1.view(torch.int32), d2.view(torch.int32))


@pytest.mark.parametrize("V,M,n", [(50, 1, 30), (64, 37, 200), (97, 130, 300), (300, 260, 500), (1000, 1028, 400)])
def test_values_ragged_shapes(som_mod, V, M, n):
    rng = np.random.default_rng(V + M)
    W = rng.normal(size=(V, M)).astype(np.float32)
    rows = [np.sort(rng.choice(V, size=int(rng.integers(0, min(V, 45) + 1)), replace=False)).astype(np.int32)
            for _ in range(n)]
    indptr = np.zeros(n + 1, np.int32)
    indptr[1:] = np.cumsum([len(r) for r in rows])
    indices = np.concatenate(rows).astype(np.int32)
    values = rng.normal(size=indices.size).astype(np.float32)
    h = som_mod.Som(V, M, torch.from_numpy(W).cuda().reshape(-1))
    h.norms()
    bmu, dist = h.bmu_values(torch.from_numpy(indptr).cuda(), torch.from_numpy(indices).cuda(),
                             torch.from_numpy(values).cuda())
    torch.cuda.synchronize()
    _check(W, V, M, indptr, indices, values, bmu.cpu().numpy(), dist.cpu().numpy())


def test_values_64x64_sampled_rows(som_mod):
    w = synth.CONFIGS[1]
    n = 200_000
    W = synth.fill_codebook(w.V, w.M, w.seed, device="cuda")
    b = synth.sample_csr(n, w.V, w.lam, w.seed, device="cpu")
    x = _values_for(b, 5, False)
    h = som_mod.Som(w.V, w.M, W)
    h.norms()
    bmu, dist = h.bmu_values(b.indptr.cuda(), b.indices.cuda(), x.cuda())
    torch.cuda.synchronize()
    rows = np.arange(0, n, 25)
    ip = b.indptr.numpy().astype(np.int64)
    lens = ip[rows + 1] - ip[rows]
    op = np.zeros(len(rows) + 1, np.int32)
    op[1:] = np.cumsum(lens)
    oi = np.concatenate([b.indices.numpy()[ip[r]:ip[r + 1]] for r in rows]).astype(np.int32)
    ov = np.concatenate([x.numpy()[ip[r]:ip[r + 1]] for r in rows]).astype(np.float32)
    _check(W.cpu().numpy(), w.V, w.M, op, oi, ov, bmu.cpu().numpy()[rows], dist.cpu().numpy()[rows])
