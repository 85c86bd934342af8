"""Helpers of the GPU parity tests on maps whose codebook lives on the device only (31 to 126 GB).

Test code: the oracle consumes the device codebook in neuron slabs copied to the host; distances
to named neurons are formed in fp64 from the stored weights gathered off the device (Eq. 1).
"""
import numpy as np
import torch

from oracle import som_oracle as orc


def subset_csr(indptr, indices, rows):
    """Host CSR of the chosen rows (numpy)."""
    indptr = np.asarray(indptr, dtype=np.int64)
    rows = np.asarray(rows, dtype=np.int64)
    lens = indptr[rows + 1] - indptr[rows]
    out_ptr = np.zeros(len(rows) + 1, np.int32)
    out_ptr[1:] = np.cumsum(lens)
    take = np.repeat(indptr[rows] - out_ptr[:-1], lens) + np.arange(int(out_ptr[-1]))
    return out_ptr, np.asarray(indices)[take].astype(np.int32)


def sample_rows(n, count):
    """`count` evenly spread rows of a batch of n, its first and last row included."""
    return np.unique(np.concatenate([np.linspace(0, n - 1, count).astype(np.int64), [0, n - 1]]))


def oracle_top2_slabbed(W_dev, V, M, indptr, indices, slab_neurons=16384):
    """Oracle best/second best over a codebook that lives on the device (fp32 or fp16 storage),
    consumed in neuron slabs (ascending) widened and copied to the host; also returns the oracle's
    fp64 norms of all neurons."""
    W2 = W_dev.view(V, M)
    run = None
    norms = np.empty(M, np.float64)
    for m0 in range(0, M, slab_neurons):
        m1 = min(M, m0 + slab_neurons)
        slab = W2[:, m0:m1].float().contiguous().cpu().numpy()
        nn = orc.norms(slab, V, m1 - m0)
        norms[m0:m1] = nn
        run = orc.bmu(slab, V, m1 - m0, indptr, indices, norms_=nn, m_offset=m0, running=run)
        del slab
    return run, norms


def dist_to_named_neuron(W_dev, V, M, indptr, indices, neuron, norms):
    """fp64 squared distance |S| - 2 sum_{v in S} w(v, g) + ||w_g||^2 of every sample to its named
    neuron g (Eq. 1): the stored weights are gathered on the device (one gather, exact values),
    summed in fp64 on the host.  indptr / indices: host CSR with indptr[0] == 0; norms: fp64 [M]."""
    indptr = np.asarray(indptr, dtype=np.int64)
    n = indptr.size - 1
    lens = indptr[1:] - indptr[:-1]
    g = np.asarray(neuron, dtype=np.int64)
    if indptr[-1] == 0:
        return lens.astype(np.float64) + norms[g]
    col = torch.from_numpy(np.repeat(g, lens)).cuda()
    row = torch.from_numpy(np.asarray(indices[:indptr[-1]], dtype=np.int64)).cuda()
    w = W_dev[row * M + col].double().cpu().numpy()
    del col, row
    dot = np.zeros(n, np.float64)
    nz = lens > 0
    dot[nz] = np.add.reduceat(w, indptr[:-1][nz])
    return lens.astype(np.float64) - 2.0 * dot + norms[g]
