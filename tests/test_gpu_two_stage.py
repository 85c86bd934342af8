"""GPU parity tests of the two-stage search (option 7): certified first pass over an fp16 copy of
an fp32 codebook, exact fp32 second pass for the uncertain samples.  The result must satisfy the
same parity rule as the plain fp32 search, and certified samples must have the plain search's unit."""
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


def _subset(indptr, indices, rows):
    indptr = np.asarray(indptr, dtype=np.int64)
    lens = indptr[rows + 1] - indptr[rows]
    out_ptr = np.zeros(len(rows) + 1, np.int32)
    out_ptr[1:] = np.cumsum(lens)
    out_idx = np.concatenate([indices[indptr[r]:indptr[r + 1]] for r in rows]).astype(np.int32)
    return out_ptr, out_idx


def _run(som_mod, W, V, M, b, two_stage, variant=2, lane_neurons=0):
    h = som_mod.Som(V, M, W)
    h.set_option(0, variant)
    if lane_neurons:
        h.set_option(3, lane_neurons)
    if two_stage:
        h.set_option(7, 1)
    h.norms()
    bmu, dist = h.bmu(b.indptr, b.indices)
    again = h.bmu(b.indptr, b.indices)
    torch.cuda.synchronize()
    assert torch.equal(bmu, again[0]) and torch.equal(dist.view(torch.int32), again[1].view(torch.int32))
    return h, bmu.cpu().numpy(), dist.cpu().numpy()


def _check(W_host, V, M, b, g_bmu, g_dist, rows):
    ip, ix = _subset(b.indptr.cpu().numpy(), b.indices.cpu().numpy(), rows)
    nn = orc.norms(W_host, V, M)
    top2 = orc.bmu(W_host, V, M, ip, ix, norms_=nn)
    d_at = orc.dist_at(W_host, V, M, ip, ix, np.clip(g_bmu[rows].astype(np.int64), 0, M - 1), norms_=nn)
    rep = parity.check(g_bmu[rows], g_dist[rows], top2, d_at, M)
    assert rep.ok, str(rep)
    return rep


@pytest.mark.parametrize("scale", [1.0, 37.0, 1.0 / 64.0, 1e-6, 1e5])
def test_two_stage_matches_oracle_and_plain_search(som_mod, scale):
    """The error bound scales with the largest weight, so the certificate must hold for scaled codebooks."""
    V, M, n = 30_000, 1_024, 80_000
    W = synth.fill_codebook(V, M, 5, device="cuda") * scale
    b = synth.sample_csr(n, V, 11.0, 5, device="cuda")
    h2, bmu2, dist2 = _run(som_mod, W, V, M, b, True)
    h1, bmu1, dist1 = _run(som_mod, W, V, M, b, False)
    unc = h2.last_uncertain()
    if 1e-3 < scale < 1e3:
        assert 0 < unc < n // 2  # most samples are certified, some are not
    # (weights of 1e-6 fall into fp16's subnormal range, weights of 1e5 overflow it: the bound
    # then certifies little or nothing and the exact pass does the work)
    differ = np.flatnonzero(bmu1 != bmu2)
    assert differ.size <= unc  # only samples of the exact pass can differ (near ties, other summation order)
    same = bmu1 == bmu2
    assert np.array_equal(dist1[same].view(np.uint32), dist2[same].view(np.uint32))
    rows = np.unique(np.concatenate([np.arange(0, n, 9), differ]))
    _check(W.cpu().numpy(), V, M, b, bmu2, dist2, rows)


def test_two_stage_config2_sampled_rows(som_mod):
    w = synth.CONFIGS[1]
    W = synth.fill_codebook(w.V, w.M, w.seed, device="cuda")
    b = synth.sample_csr(w.N, w.V, w.lam, w.seed, device="cuda")
    h, bmu, dist = _run(som_mod, W, w.V, w.M, b, True, variant=0)
    assert 0 < h.last_uncertain() < w.N // 4
    rows = np.concatenate([np.arange(0, w.N, 40), [w.N - 1]])
    _check(W.cpu().numpy(), w.V, w.M, b, bmu, dist, rows)


def test_two_stage_with_duplicate_neurons_sends_everything_to_the_exact_pass(som_mod):
    """Two identical halves of the map: every best unit has an exact twin, no sample can be certified,
    and the lowest index must win."""
    V, half, n = 2_000, 1_024, 40_000
    Wh = synth.fill_codebook(V, half, 2, device="cuda").view(V, half)
    W = torch.cat([Wh, Wh], dim=1).contiguous().view(-1)
    M = 2 * half
    b = synth.sample_csr(n, V, 7.0, 2, device="cuda")
    h, bmu, dist = _run(som_mod, W, V, M, b, True)
    assert h.last_uncertain() == n
    assert bmu.max() < half
    _check(W.cpu().numpy(), V, M, b, bmu, dist, np.arange(0, n, 11))


def test_two_stage_needs_its_shadow_from_norms(som_mod):
    """Switching the option on invalidates the norms: the next som_norms has to write the copy."""
    V, M, n = 2_000, 1_024, 30_000
    W = synth.fill_codebook(V, M, 1, device="cuda")
    b = synth.sample_csr(n, V, 7.0, 1, device="cuda")
    h = som_mod.Som(V, M, W)
    h.norms()
    h.set_option(7, 1)
    with pytest.raises(som_mod.SomError):
        h.bmu(b.indptr, b.indices)
    h.norms()
    # after an in-place change of the codebook the copy follows at the next som_norms
    W.mul_(0.5)
    h.norms()
    bmu, dist = h.bmu(b.indptr, b.indices)
    torch.cuda.synchronize()
    _check(W.cpu().numpy(), V, M, b, bmu.cpu().numpy(), dist.cpu().numpy(), np.arange(0, n, 13))


def _run2(som_mod, W, V, M, b, two_stage, variant=2, lane_neurons=0):
    h = som_mod.Som(V, M, W)
    h.set_option(0, variant)
    if lane_neurons:
        h.set_option(3, lane_neurons)
    if two_stage:
        h.set_option(7, 1)
    h.norms()
    out = h.bmu2(b.indptr, b.indices)
    again = h.bmu2(b.indptr, b.indices)
    torch.cuda.synchronize()
    for a, c in zip(out, again):
        assert torch.equal(a.view(torch.int32), c.view(torch.int32))
    return h, [t.cpu().numpy() for t in out]


def _check2(W_host, V, M, b, out, rows):
    g1, gd1, g2, gd2 = [x[rows] for x in out]
    ip, ix = _subset(b.indptr.cpu().numpy(), b.indices.cpu().numpy(), rows)
    nn = orc.norms(W_host, V, M)
    top2 = orc.bmu(W_host, V, M, ip, ix, norms_=nn)
    rep1 = parity.check(g1, gd1, top2, orc.dist_at(W_host, V, M, ip, ix, np.clip(g1.astype(np.int64), 0, M - 1), norms_=nn), M)
    assert rep1.ok, str(rep1)
    rep2 = parity.check_second(g1, g2, gd2, top2,
                               orc.dist_at(W_host, V, M, ip, ix, np.clip(g2.astype(np.int64), 0, M - 1), norms_=nn), M)
    assert rep2.ok, str(rep2)


@pytest.mark.parametrize("scale", [1.0, 37.0, 1.0 / 64.0, 1e-6, 1e5])
def test_two_stage_two_best_matches_oracle_and_plain_search(som_mod, scale):
    """som_bmu2 with the option: three best of the first pass, both gaps certified."""
    V, M, n = 30_000, 1_024, 80_000
    W = synth.fill_codebook(V, M, 5, device="cuda") * scale
    b = synth.sample_csr(n, V, 11.0, 5, device="cuda")
    hs, staged = _run2(som_mod, W, V, M, b, True)
    hp, plain = _run2(som_mod, W, V, M, b, False)
    unc = hs.last_uncertain()
    if 1e-3 < scale < 1e3:
        assert 0 < unc < n // 2
    differ = np.flatnonzero((plain[0] != staged[0]) | (plain[2] != staged[2]))
    assert differ.size <= unc  # only samples of the exact pass can differ (near ties, other summation order)
    same = (plain[0] == staged[0]) & (plain[2] == staged[2])
    assert np.array_equal(plain[1][same].view(np.uint32), staged[1][same].view(np.uint32))
    assert np.array_equal(plain[3][same].view(np.uint32), staged[3][same].view(np.uint32))
    assert np.all(staged[2] != staged[0]) and staged[2].min() >= 0 and staged[2].max() < M
    rows = np.unique(np.concatenate([np.arange(0, n, 9), differ]))
    _check2(W.cpu().numpy(), V, M, b, staged, rows)


def test_two_stage_two_best_config2_sampled_rows(som_mod):
    w = synth.CONFIGS[1]
    W = synth.fill_codebook(w.V, w.M, w.seed, device="cuda")
    b = synth.sample_csr(w.N, w.V, w.lam, w.seed, device="cuda")
    h, out = _run2(som_mod, W, w.V, w.M, b, True, variant=0)
    assert 0 < h.last_uncertain() < w.N // 3
    rows = np.concatenate([np.arange(0, w.N, 40), [w.N - 1]])
    _check2(W.cpu().numpy(), w.V, w.M, b, out, rows)


def test_two_stage_two_best_with_duplicate_neurons(som_mod):
    """Two identical halves of the map: the best unit's twin is the second best at the same distance;
    nothing can be certified and the lower index comes first."""
    V, half, n = 2_000, 1_024, 40_000
    Wh = synth.fill_codebook(V, half, 2, device="cuda").view(V, half)
    W = torch.cat([Wh, Wh], dim=1).contiguous().view(-1)
    M = 2 * half
    b = synth.sample_csr(n, V, 7.0, 2, device="cuda")
    h, out = _run2(som_mod, W, V, M, b, True)
    assert h.last_uncertain() == n
    assert out[0].max() < half
    assert np.array_equal(out[2], out[0] + half)
    assert np.array_equal(out[1].view(np.uint32), out[3].view(np.uint32))
    _check2(W.cpu().numpy(), V, M, b, out, np.arange(0, n, 11))


def test_two_stage_option_leaves_the_other_entry_points_alone(som_mod):
    """An fp16-stored codebook has no use for the option and a forced direct-load kernel overrides
    it: both must give what they give without the option."""
    V, M, n = 2_000, 1_024, 30_000
    W = synth.fill_codebook(V, M, 9, device="cuda")
    b = synth.sample_csr(n, V, 7.0, 9, device="cuda")
    plain, staged = som_mod.Som(V, M, W), som_mod.Som(V, M, W)
    staged.set_option(7, 1)
    plain.norms(); staged.norms()
    plain.set_option(0, 1); staged.set_option(0, 1)
    for a, c in zip(plain.bmu(b.indptr, b.indices), staged.bmu(b.indptr, b.indices)):
        assert torch.equal(a.view(torch.int32), c.view(torch.int32))
    for a, c in zip(plain.bmu2(b.indptr, b.indices), staged.bmu2(b.indptr, b.indices)):
        assert torch.equal(a.view(torch.int32), c.view(torch.int32))
    W16 = W.half()
    h16a, h16b = som_mod.Som(V, M, W16), som_mod.Som(V, M, W16)
    h16b.set_option(7, 1)
    h16a.norms(); h16b.norms()
    for a, c in zip(h16a.bmu(b.indptr, b.indices), h16b.bmu(b.indptr, b.indices)):
        assert torch.equal(a.view(torch.int32), c.view(torch.int32))
    for a, c in zip(h16a.bmu2(b.indptr, b.indices), h16b.bmu2(b.indptr, b.indices)):
        assert torch.equal(a.view(torch.int32), c.view(torch.int32))
    torch.cuda.synchronize()


def test_two_stage_with_a_reusable_plan(som_mod):
    """The planned search takes the two-stage route like som_bmu and gives the same bits, epoch after epoch."""
    V, M, n = 30_000, 1_024, 60_000
    W = synth.fill_codebook(V, M, 4, device="cuda")
    b = synth.sample_csr(n, V, 11.0, 4, device="cuda")
    h = som_mod.Som(V, M, W)
    h.set_option(0, 2)
    h.set_option(7, 1)
    plan = h.plan(b.indptr, b.indices)
    for epoch in range(3):
        if epoch:
            W.mul_(0.9)
            W[epoch::7] += 0.01
        h.norms()
        p_bmu, p_dist = plan.bmu()
        torch.cuda.synchronize()  # (the count travels back unwaited for: read it once the stream is done)
        unc_planned = h.last_uncertain()
        d_bmu, d_dist = h.bmu(b.indptr, b.indices)
        torch.cuda.synchronize()
        assert 0 < unc_planned < n // 2 and unc_planned == h.last_uncertain()
        assert torch.equal(p_bmu, d_bmu) and torch.equal(p_dist.view(torch.int32), d_dist.view(torch.int32))
    _check(W.cpu().numpy(), V, M, b, p_bmu.cpu().numpy(), p_dist.cpu().numpy(), np.arange(0, n, 9))
    plan.destroy()


def test_two_stage_probe_sends_a_smooth_map_to_the_plain_search(som_mod):
    """Units that differ by less than fp16 resolves: the probe (one sample in 256 of a batch of at least
    65536) fails the certificate nearly everywhere and the call takes the plain search on the same plan,
    whose bits it must then reproduce (the plain search with 8 neurons per lane: the layout whose table
    matches the first pass's plan); a smaller batch is not probed and goes through the exact pass."""
    V, M, n = 4_000, 1_024, 100_000
    base = synth.fill_codebook(V, 1, 3, device="cuda").view(V, 1)
    noise = synth.fill_codebook(V, M, 8, device="cuda").view(V, M)
    W = (base + 1e-5 * noise).contiguous().view(-1)
    b = synth.sample_csr(n, V, 9.0, 3, device="cuda")
    hs, bs, ds = _run(som_mod, W, V, M, b, True)
    hp, bp, dp = _run(som_mod, W, V, M, b, False, lane_neurons=8)
    assert hs.last_uncertain() == n
    assert np.array_equal(bs, bp) and np.array_equal(ds.view(np.uint32), dp.view(np.uint32))
    _check(W.cpu().numpy(), V, M, b, bs, ds, np.arange(0, n, 23))
    hs2, out_s = _run2(som_mod, W, V, M, b, True)
    hp2, out_p = _run2(som_mod, W, V, M, b, False, lane_neurons=8)
    assert hs2.last_uncertain() == n
    for a, c in zip(out_s, out_p):
        assert np.array_equal(a.view(np.uint32), c.view(np.uint32))
    small = synth.sample_csr(20_000, V, 9.0, 4, device="cuda")
    h3, b3, d3 = _run(som_mod, W, V, M, small, True)
    assert h3.last_uncertain() > 15_000
    _check(W.cpu().numpy(), V, M, small, b3, d3, np.arange(0, 20_000, 7))
