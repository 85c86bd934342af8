"""Seeded synthetic workloads shaped like the paper's MeSH corpus (Section 4.2, Table 1).

Everything here is *data generation only*: a counter-based integer hash turned into
uniform numbers, a codebook fill, and a sparse-binary CSR batch sampler.  None of the
search arithmetic (distances, norms, argmin) lives in this module, so both the CPU
oracle's tests and the CUDA tests may draw their inputs from it.

All generators are written with torch integer ops only, so the same call gives
bit-identical results on ``device="cpu"`` and ``device="cuda"``; that is what lets a
126 GB codebook be filled in place on the GPU while a test regenerates any slab of it
on the host.

Workload recipes (the five benchmark configurations):

* codebook: fp32, feature-major ``W[v*M+i]``; every entry U[0, 0.05); then for each
  neuron 20 feature ids drawn uniformly over V are overwritten with U[0.3, 1).
* samples: binary CSR, int32 sorted indices, ``nnz = min(40, 1 + Poisson(lam))``,
  features drawn without replacement from Zipf(s) over V (probability of id v
  proportional to (v+1)^-s, successive iid draws with repeats discarded).
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np
import torch

_M32 = 0xFFFFFFFF

# stream constants: separate hash streams for separate purposes
_STREAM_BASE = 0x243F6A88
_STREAM_SPIKE_POS = 0x85A308D3
_STREAM_SPIKE_VAL = 0x13198A2E
_STREAM_NNZ = 0x03707344
_STREAM_DRAW_HI = 0xA4093822
_STREAM_DRAW_LO = 0x299F31D0
_STREAM_PERM = 0x082EFA98


def _mix32(x: torch.Tensor) -> torch.Tensor:
    """32-bit avalanche mix on int64 tensors holding unsigned 32-bit values."""
    x = x & _M32
    x = ((x ^ (x >> 16)) * 0x7FEB352D) & _M32
    x = ((x ^ (x >> 15)) * 0x846CA68B) & _M32
    x = x ^ (x >> 16)
    return x


def hash32(seed: int, stream: int, a: torch.Tensor, b) -> torch.Tensor:
    """Counter-based hash of (seed, stream, a, b) -> uint32 stored in int64.

    ``a`` may exceed 32 bits (it is folded as two words); ``b`` is a tensor or int
    below 2^32.
    """
    s = ((seed & _M32) * 0x9E3779B1 + stream) & _M32
    a_lo = a & _M32
    a_hi = (a >> 32) & _M32
    h = _mix32(a_lo ^ s)
    h = _mix32(h + a_hi * 0x9E3779B1 + 0x7F4A7C15)
    h = _mix32(h ^ ((b * 0x85EBCA77) & _M32))
    return h


def _u24_to_f32(h: torch.Tensor, lo: float, width: float) -> torch.Tensor:
    """uint32 hash -> fp32 in [lo, lo+width) using the top 24 bits (exact steps)."""
    u = (h >> 8).to(torch.float32)  # exact: < 2^24
    out = u * np.float32(width / 16777216.0)
    if lo != 0.0:
        out = out + np.float32(lo)
    return out


def fill_codebook(V: int, M: int, seed: int = 0, device="cpu", out: torch.Tensor | None = None,
                  spikes_per_neuron: int = 20, chunk_elems: int = 1 << 26) -> torch.Tensor:
    """Feature-major fp32 codebook of V*M weights (flat, element (v,i) at v*M+i).

    Base fill U[0,0.05) keyed on the flat offset; then ``spikes_per_neuron`` feature
    ids per neuron, uniform over V, are overwritten with U[0.3,1).  A spike's value is
    keyed on (v,i) and not on the draw number, so a repeated pick writes the same value
    twice and the result does not depend on write order.  ``out`` may be a float16 tensor: each
    fp32 value is then rounded to the nearest fp16 on store (the fp16-stored codebook).
    """
    total = V * M
    if out is None:
        out = torch.empty(total, dtype=torch.float32, device=device)
    assert out.numel() == total and out.dtype in (torch.float32, torch.float16)
    dev = out.device
    rows_per_chunk = max(1, chunk_elems // M)
    for v0 in range(0, V, rows_per_chunk):
        v1 = min(V, v0 + rows_per_chunk)
        off = torch.arange(v0 * M, v1 * M, dtype=torch.int64, device=dev)
        out[v0 * M:v1 * M] = _u24_to_f32(hash32(seed, _STREAM_BASE, off, 0), 0.0, 0.05)
        del off
    # spikes, processed in neuron chunks
    n_chunk = max(1, chunk_elems // max(1, spikes_per_neuron))
    for i0 in range(0, M, n_chunk):
        i1 = min(M, i0 + n_chunk)
        i = torch.arange(i0, i1, dtype=torch.int64, device=dev)
        for k in range(spikes_per_neuron):
            v = hash32(seed, _STREAM_SPIKE_POS, i, k) % V
            flat = v * M + i
            val = _u24_to_f32(hash32(seed, _STREAM_SPIKE_VAL, flat, 0), 0.3, 0.7)
            out[flat] = val.to(out.dtype)
    return out


def codebook_rows(V: int, M: int, rows: torch.Tensor, seed: int = 0,
                  spikes_per_neuron: int = 20) -> torch.Tensor:
    """Regenerate selected feature rows of ``fill_codebook`` on the CPU: [len(rows), M]."""
    rows = rows.to(torch.int64).cpu()
    r = rows.numel()
    out = torch.empty(r, M, dtype=torch.float32)
    i = torch.arange(M, dtype=torch.int64)
    for j in range(r):
        v = int(rows[j])
        out[j] = _u24_to_f32(hash32(seed, _STREAM_BASE, v * M + i, 0), 0.0, 0.05)
    pos = {int(v): j for j, v in enumerate(rows.tolist())}
    for k in range(spikes_per_neuron):
        v = hash32(seed, _STREAM_SPIKE_POS, i, k) % V
        for vv, j in pos.items():
            sel = (v == vv).nonzero().flatten()
            if sel.numel():
                flat = vv * M + sel
                out[j, sel] = _u24_to_f32(hash32(seed, _STREAM_SPIKE_VAL, flat, 0), 0.3, 0.7)
    return out


def codebook_slab(V: int, M: int, m0: int, m1: int, seed: int = 0, device="cpu",
                  spikes_per_neuron: int = 20, chunk_elems: int = 1 << 24) -> torch.Tensor:
    """Columns [m0, m1) of ``fill_codebook`` as a dense [V, m1-m0] fp32 tensor (same values)."""
    dev = torch.device(device)
    ms = m1 - m0
    out = torch.empty(V, ms, dtype=torch.float32, device=dev)
    i = torch.arange(m0, m1, dtype=torch.int64, device=dev)
    rows_per_chunk = max(1, chunk_elems // max(1, ms))
    for v0 in range(0, V, rows_per_chunk):
        v1 = min(V, v0 + rows_per_chunk)
        v = torch.arange(v0, v1, dtype=torch.int64, device=dev)
        off = (v[:, None] * M + i[None, :]).reshape(-1)
        out[v0:v1] = _u24_to_f32(hash32(seed, _STREAM_BASE, off, 0), 0.0, 0.05).view(v1 - v0, ms)
    for k in range(spikes_per_neuron):
        v = hash32(seed, _STREAM_SPIKE_POS, i, k) % V
        val = _u24_to_f32(hash32(seed, _STREAM_SPIKE_VAL, v * M + i, 0), 0.3, 0.7)
        out[v, i - m0] = val
    return out


def zipf_cdf(V: int, s: float) -> np.ndarray:
    """Cumulative distribution (float64, host) of p(v) ~ (v+1)^-s over v in [0,V)."""
    p = np.power(np.arange(1, V + 1, dtype=np.float64), -float(s))
    c = np.cumsum(p)
    c /= c[-1]
    c[-1] = 1.0
    return c


def poisson_cdf(lam: float, kmax: int = 200) -> np.ndarray:
    k = np.arange(kmax + 1, dtype=np.float64)
    logp = -lam + k * math.log(lam) - np.array([math.lgamma(x + 1.0) for x in k])
    c = np.cumsum(np.exp(logp))
    c[-1] = 1.0
    return c


def _uniform53(seed: int, a: torch.Tensor, b) -> torch.Tensor:
    hi = hash32(seed, _STREAM_DRAW_HI, a, b)
    lo = hash32(seed, _STREAM_DRAW_LO, a, b)
    return ((hi << 21) | (lo >> 11)).to(torch.float64) * (1.0 / 9007199254740992.0)


@dataclass
class CsrBatch:
    """Sparse-binary CSR batch: row pointers and sorted column ids, values implicit 1."""
    indptr: torch.Tensor   # int32 [n+1]
    indices: torch.Tensor  # int32 [nnz_total], ascending and distinct inside each row
    n: int
    V: int

    @property
    def nnz(self) -> int:
        return int(self.indices.numel())


def sample_csr(N: int, V: int, lam: float, seed: int = 0, zipf_s: float = 1.1, nnz_cap: int = 40,
               device="cpu", first_sample: int = 0, permute_ids: bool = False,
               chunk: int = 1 << 17) -> CsrBatch:
    """N sparse-binary samples; sample ids run from ``first_sample`` so that batches of one
    long stream can be produced independently.

    Row n holds the first k_n distinct values of an iid Zipf(zipf_s) stream keyed on
    (seed, n, draw number), with k_n = min(nnz_cap, 1 + Poisson(lam)), sorted ascending.
    ``zipf_s = 0`` gives features uniform over V.  ``permute_ids`` relabels feature ids by
    a seeded permutation, so that the frequent features are not the low ids.
    """
    dev = torch.device(device)
    cdf = torch.from_numpy(zipf_cdf(V, zipf_s)).to(dev)
    pcdf = torch.from_numpy(poisson_cdf(lam)).to(dev)
    perm = None
    if permute_ids:
        hv = hash32(seed, _STREAM_PERM, torch.arange(V, dtype=torch.int64, device=dev), 0)
        perm = torch.argsort(hv * V + torch.arange(V, dtype=torch.int64, device=dev))
    big = V + 1
    rows_idx, rows_cnt = [], []
    for c0 in range(0, N, chunk):
        c1 = min(N, c0 + chunk)
        n_ids = torch.arange(first_sample + c0, first_sample + c1, dtype=torch.int64, device=dev)
        un = hash32(seed, _STREAM_NNZ, n_ids, 0).to(torch.float64) * (1.0 / 4294967296.0)
        k = 1 + torch.searchsorted(pcdf, un, right=True)
        k = torch.clamp(k, max=min(nnz_cap, V))
        D = 64
        pending = torch.arange(c1 - c0, device=dev)
        vals_out = torch.full((c1 - c0, nnz_cap), big, dtype=torch.int64, device=dev)
        while pending.numel():
            ids = n_ids[pending]
            kk = k[pending]
            j = torch.arange(D, dtype=torch.int64, device=dev)
            u = _uniform53(seed, ids[:, None].expand(-1, D).contiguous(), j[None, :])
            draws = torch.searchsorted(cdf, u, right=True).clamp_(max=V - 1)
            sv, sp = torch.sort(draws, dim=1, stable=True)
            dup_s = torch.zeros_like(sv, dtype=torch.bool)
            dup_s[:, 1:] = sv[:, 1:] == sv[:, :-1]
            dup = torch.zeros_like(dup_s)
            dup.scatter_(1, sp, dup_s)
            fresh = ~dup
            rank = torch.cumsum(fresh.to(torch.int64), dim=1)
            ok = rank[:, -1] >= kk
            sel = fresh & (rank <= kk[:, None])
            cand = torch.where(sel, draws, torch.full_like(draws, big))
            cand, _ = torch.sort(cand, dim=1)
            good = ok.nonzero().flatten()
            vals_out[pending[good]] = cand[good, :nnz_cap]
            pending = pending[(~ok).nonzero().flatten()]
            D *= 8
            if D > 64 * 8 ** 4:
                raise RuntimeError("sample_csr: could not draw enough distinct features")
        keep = torch.arange(nnz_cap, device=dev)[None, :] < k[:, None]
        flat = vals_out[keep]
        if perm is not None:
            # relabel, then restore ascending order inside each row
            relab = torch.full_like(vals_out, big)
            relab[keep] = perm[flat]
            relab, _ = torch.sort(relab, dim=1)
            flat = relab[keep]
        rows_idx.append(flat.to(torch.int32))
        rows_cnt.append(k)
    if N == 0:
        return CsrBatch(torch.zeros(1, dtype=torch.int32, device=dev),
                        torch.zeros(0, dtype=torch.int32, device=dev), 0, V)
    cnt = torch.cat(rows_cnt)
    indptr = torch.zeros(N + 1, dtype=torch.int64, device=dev)
    indptr[1:] = torch.cumsum(cnt, 0)
    assert int(indptr[-1]) < 2 ** 31
    return CsrBatch(indptr.to(torch.int32), torch.cat(rows_idx), N, V)


@dataclass(frozen=True)
class Workload:
    """One benchmark configuration (map size, sample count, batch size)."""
    name: str
    V: int
    M: int
    N: int
    batch: int
    lam: float
    seed: int = 0
    zipf_s: float = 1.1


CONFIGS = [
    Workload("tiny-16x16", 2_000, 256, 20_000, 20_000, 7.0),
    Workload("64x64", 30_000, 4_096, 1_000_000, 1_000_000, 11.0),
    Workload("128x128", 30_000, 16_384, 4_000_000, 4_000_000, 11.0),
    Workload("512x512", 30_000, 262_144, 4_000_000, 1_000_000, 11.0),
    Workload("1024x1024", 30_000, 1_048_576, 1_000_000, 250_000, 11.0),
]
