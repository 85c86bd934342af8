"""The synthetic workload generators: structure, distributions and reproducibility (CPU)."""
import numpy as np
import torch

from paper_2608_24067_b200 import synth


def _row_lengths(b):
    ip = b.indptr.long()
    return ip[1:] - ip[:-1]


def test_csr_structure_sorted_distinct_in_range():
    b = synth.sample_csr(5000, 2000, 7.0, seed=0)
    cnt = _row_lengths(b)
    assert b.indptr.dtype == torch.int32 and b.indices.dtype == torch.int32
    assert int(b.indptr[0]) == 0 and int(b.indptr[-1]) == b.nnz
    assert int(cnt.min()) >= 1 and int(cnt.max()) <= 40
    idx = b.indices.long()
    assert int(idx.min()) >= 0 and int(idx.max()) < 2000
    row = torch.repeat_interleave(torch.arange(b.n), cnt)
    same = row[1:] == row[:-1]
    assert bool(((idx[1:] - idx[:-1])[same] > 0).all())


def test_csr_statistics_match_recipe():
    """nnz = min(40, 1 + Poisson(11)); Zipf(1.1) head coverage as measured for the recipe."""
    b = synth.sample_csr(60000, 30000, 11.0, seed=0)
    cnt = _row_lengths(b).double()
    assert abs(cnt.mean().item() - 12.0) < 0.08
    assert abs(cnt.var().item() - 11.0) < 0.5
    q = torch.bincount(b.indices.long(), minlength=30000).double() / b.n
    assert abs(q[0].item() - 0.84) < 0.02 and abs(q[1].item() - 0.60) < 0.02
    cover = torch.cumsum(q, 0) / q.sum()
    assert abs(cover[15].item() - 0.34) < 0.02
    assert abs(cover[1023].item() - 0.76) < 0.02


def test_csr_reproducible_and_batchable():
    a = synth.sample_csr(3000, 500, 7.0, seed=3)
    b = synth.sample_csr(3000, 500, 7.0, seed=3, chunk=777)
    assert torch.equal(a.indptr, b.indptr) and torch.equal(a.indices, b.indices)
    c = synth.sample_csr(1000, 500, 7.0, seed=3, first_sample=2000)
    lo = int(a.indptr[2000])
    assert torch.equal(c.indices, a.indices[lo:])
    d = synth.sample_csr(3000, 500, 7.0, seed=4)
    assert not torch.equal(a.indices[:100], d.indices[:100])


def test_csr_variants():
    u = synth.sample_csr(20000, 1000, 7.0, seed=0, zipf_s=0.0)
    q = torch.bincount(u.indices.long(), minlength=1000).double() / u.n
    assert q.max().item() < 3 * q.mean().item()  # uniform: no heavy head
    p = synth.sample_csr(20000, 1000, 7.0, seed=0, permute_ids=True)
    z = synth.sample_csr(20000, 1000, 7.0, seed=0)
    assert torch.equal(_row_lengths(p), _row_lengths(z))
    qp = torch.bincount(p.indices.long(), minlength=1000)
    qz = torch.bincount(z.indices.long(), minlength=1000)
    assert torch.equal(torch.sort(qp)[0], torch.sort(qz)[0])  # same multiset of frequencies
    assert int(qp.argmax()) != 0 or int(qz.argmax()) != 0
    cnt = _row_lengths(p)
    row = torch.repeat_interleave(torch.arange(p.n), cnt)
    same = row[1:] == row[:-1]
    idx = p.indices.long()
    assert bool(((idx[1:] - idx[:-1])[same] > 0).all())
    e = synth.sample_csr(0, 100, 7.0)
    assert e.n == 0 and e.indptr.numel() == 1 and e.nnz == 0


def test_small_vocabulary_caps_row_length():
    b = synth.sample_csr(500, 5, 7.0, seed=1)
    assert int(_row_lengths(b).max()) <= 5


def test_codebook_recipe():
    V, M = 2000, 256
    W = synth.fill_codebook(V, M, seed=0).view(V, M)
    spikes = W >= 0.3
    base = W[~spikes]
    assert float(base.min()) >= 0.0 and float(base.max()) < 0.05
    assert abs(float(base.mean()) - 0.025) < 5e-4
    per_neuron = spikes.sum(0)
    assert int(per_neuron.max()) <= 20 and int(per_neuron.min()) >= 17
    sv = W[spikes]
    assert float(sv.min()) >= 0.3 and float(sv.max()) < 1.0
    assert abs(float(sv.mean()) - 0.65) < 0.01
    # spikes are uniform over V, not concentrated on the frequent (low) ids
    assert abs(float(spikes.nonzero()[:, 0].double().mean()) - V / 2) < 0.03 * V


def test_codebook_reproducible_chunking_and_rows():
    V, M = 300, 64
    a = synth.fill_codebook(V, M, seed=5)
    b = synth.fill_codebook(V, M, seed=5, chunk_elems=1000)
    assert torch.equal(a, b)
    rows = torch.tensor([0, 17, 299])
    assert torch.equal(synth.codebook_rows(V, M, rows, seed=5), a.view(V, M)[rows])
    assert not torch.equal(a, synth.fill_codebook(V, M, seed=6))
    assert torch.equal(synth.codebook_slab(V, M, 8, 40, seed=5, chunk_elems=500), a.view(V, M)[:, 8:40])
    assert torch.equal(synth.codebook_slab(V, M, 0, M, seed=5), a.view(V, M))


def test_configs_table():
    c = synth.CONFIGS
    assert [w.M for w in c] == [256, 4096, 16384, 262144, 1048576]
    assert [w.N for w in c] == [20000, 10 ** 6, 4 * 10 ** 6, 4 * 10 ** 6, 10 ** 6]
    assert c[3].batch == 10 ** 6 and c[4].batch == 250000
    assert np.isclose(c[4].V * c[4].M * 4 / 1e9, 125.8, atol=0.1)
