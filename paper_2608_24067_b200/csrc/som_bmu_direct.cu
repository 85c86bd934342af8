// Direct-load BMU search kernel, winner finalisation and CSR validation.
//
// k_bmu_direct is the simplest complete statement of the fused search (Section 3.3):
// a warp owns one sample at a time and a block of 32*VEC neurons; every lane keeps VEC
// score accumulators in registers, seeded with ||w_i||^2 / 2, and for each active feature v
// subtracts the contiguous segment W[v*M + i0 .. i0+VEC) fetched with one 128-bit load
// (feature-major layout: the warp's 32 loads cover 512 contiguous bytes), four features at a
// time so that their loads are in flight together.  The per-block
// argmin is a warp-shuffle reduction on (score, index) with ties to the lower index, and
// the cross-block combine is a 64-bit atomicMin on an order-preserving packed key, which is
// commutative and associative and therefore deterministic.  No N x M score block is ever
// written.  It serves every shape (any M, any row length) and is the fallback of the
// faster row-table kernel.
#include "som_internal.cuh"

namespace {

constexpr int DIRECT_THREADS = 256;
constexpr int DIRECT_WARPS = DIRECT_THREADS / 32;
constexpr int DIRECT_SAMPLES_PER_WARP = 16;

// (score, index) order: smaller score first, then lower index
__device__ __forceinline__ bool before(float a, uint32_t ai, float b, uint32_t bi)
{
    return a < b || (a == b && ai < bi);
}

// four adjacent weights of one feature row with one vector load (16 bytes of fp32, 8 of fp16)
__device__ __forceinline__ void load4(const float* p, float (&w)[4])
{
    const float4 v = __ldg(reinterpret_cast<const float4*>(p));
    w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
}
__device__ __forceinline__ void load4(const __half* p, float (&w)[4])
{
    const uint2 v = __ldg(reinterpret_cast<const uint2*>(p));
    const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&v.x));
    const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&v.y));
    w[0] = a.x; w[1] = a.y; w[2] = b.x; w[3] = b.y;
}

// TOP2 also keeps the second-best unit in keys2 (Algorithm 2 keeps the two best units).
// ST is the storage type of the codebook (float, or __half widened exactly before the fp32 add).
// VALUED: sparse real-valued samples (a values array parallel to the indices; the paper's outlook,
// Section 7): the gather-sum becomes a gather-multiply, score = ||w||^2/2 - sum_k x_k * w[idx_k].
template <int VEC, bool TOP2, typename ST, bool VALUED = false>
__global__ void __launch_bounds__(DIRECT_THREADS)
k_bmu_direct(const ST* __restrict__ W, const float* __restrict__ hnorm, int64_t M,
             const int32_t* __restrict__ indptr, const int32_t* __restrict__ indices, int64_t n,
             unsigned long long* __restrict__ keys, unsigned long long* __restrict__ keys2,
             int64_t neuron_off, const int32_t* __restrict__ sample_list,
             const float* __restrict__ values = nullptr)
{
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int64_t i0 = neuron_off + ((int64_t)blockIdx.y * 32 + lane) * VEC;
    const float inf = __int_as_float(0x7f800000);

    float seed[VEC];
#pragma unroll
    for (int k = 0; k < VEC; ++k) seed[k] = (i0 + k < M) ? hnorm[i0 + k] : inf;
    const bool live = i0 < M;  // with VEC >= 4, M % VEC == 0: all of the lane's neurons or none
    const ST* W_lane = W + (live ? i0 : 0);

    const int64_t s0 = ((int64_t)blockIdx.x * DIRECT_WARPS + warp) * DIRECT_SAMPLES_PER_WARP;
    const int64_t s1 = min(n, s0 + DIRECT_SAMPLES_PER_WARP);
    for (int64_t s = s0; s < s1; ++s) {
        // with a sample list, position s of the list (and of the key arrays) is sample list[s]
        const int64_t sid = sample_list ? (int64_t)sample_list[s] : s;
        const int beg = indptr[sid];
        const int end = indptr[sid + 1];
        float acc[VEC];
#pragma unroll
        for (int k = 0; k < VEC; ++k) acc[k] = seed[k];
        for (int base = beg; base < end; base += 32) {
            const int mine = (base + lane < end) ? indices[base + lane] : 0;
            const float mine_x = (VALUED && base + lane < end) ? values[base + lane] : 1.f;
            const int cnt = min(32, end - base);
            int j = 0;
            // four features at a time: their row segments are in flight together, the
            // subtractions keep the ascending feature order
            for (; j + 4 <= cnt; j += 4) {
                int v[4];
                float x[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    v[u] = __shfl_sync(0xffffffffu, mine, j + u);
                    x[u] = VALUED ? __shfl_sync(0xffffffffu, mine_x, j + u) : 1.f;
                }
                if (live) {
                    float w[4][VEC];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const ST* p = W_lane + (int64_t)v[u] * M;
                        if (VEC >= 4) {
#pragma unroll
                            for (int g = 0; g < VEC / 4; ++g) {
                                float t[4];
                                load4(p + 4 * g, t);
#pragma unroll
                                for (int k = 0; k < 4; ++k) w[u][(4 * g + k) % VEC] = t[k];
                            }
                        } else {
                            w[u][0] = som_weight(p);
                        }
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u)
#pragma unroll
                        for (int k = 0; k < VEC; ++k)
                            acc[k] = VALUED ? fmaf(-x[u], w[u][k], acc[k]) : acc[k] - w[u][k];
                }
            }
            for (; j < cnt; ++j) {
                const int v = __shfl_sync(0xffffffffu, mine, j);
                const float x = VALUED ? __shfl_sync(0xffffffffu, mine_x, j) : 1.f;
                if (live) {
                    const ST* p = W_lane + (int64_t)v * M;
                    if (VEC >= 4) {
#pragma unroll
                        for (int g = 0; g < VEC / 4; ++g) {
                            float t[4];
                            load4(p + 4 * g, t);
#pragma unroll
                            for (int k = 0; k < 4; ++k)
                                acc[(4 * g + k) % VEC] = VALUED ? fmaf(-x, t[k], acc[(4 * g + k) % VEC])
                                                                : acc[(4 * g + k) % VEC] - t[k];
                        }
                    } else {
                        acc[0] = VALUED ? fmaf(-x, som_weight(p), acc[0]) : acc[0] - som_weight(p);
                    }
                }
            }
        }
        float best = acc[0];
        uint32_t bi = (uint32_t)i0;
        float second = inf;            // TOP2: the lane's, then the warp's, second best
        uint32_t si = 0xffffffffu;
#pragma unroll
        for (int k = 1; k < VEC; ++k) {
            const uint32_t ik = (uint32_t)(i0 + k);
            if (acc[k] < best) {
                if (TOP2) { second = best; si = bi; }
                best = acc[k];
                bi = ik;
            } else if (TOP2 && before(acc[k], ik, second, si)) {
                second = acc[k];
                si = ik;
            }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float ob = __shfl_down_sync(0xffffffffu, best, off);
            const uint32_t oi = __shfl_down_sync(0xffffffffu, bi, off);
            if (TOP2) {
                // merge two sorted pairs into the best two of the four
                const float os = __shfl_down_sync(0xffffffffu, second, off);
                const uint32_t osi = __shfl_down_sync(0xffffffffu, si, off);
                if (before(ob, oi, best, bi)) {
                    if (before(best, bi, os, osi)) { second = best; si = bi; }
                    else { second = os; si = osi; }
                    best = ob;
                    bi = oi;
                } else if (before(ob, oi, second, si)) {
                    second = ob;
                    si = oi;
                }
            } else {
                if (ob < best || (ob == best && oi < bi)) { best = ob; bi = oi; }
            }
        }
        if (lane == 0) {
            const unsigned long long c1 = som_pack_key(best, bi);
            if (!TOP2) {
                atomicMin(&keys[s], c1);
            } else {
                // keys ends as the minimum of all candidates; each other candidate reaches
                // keys2 exactly once (directly, or when a smaller one displaces it from keys)
                const unsigned long long old = atomicMin(&keys[s], c1);
                atomicMin(&keys2[s], old > c1 ? old : c1);
                if (si != 0xffffffffu) atomicMin(&keys2[s], som_pack_key(second, si));
            }
        }
    }
}

// One thread per sample: unpack the winner and recompute its full squared distance
// |S| - 2*dot + ||w||^2 (left side of Eq. 1) in fp64, ascending feature order.
template <typename ST>
__global__ void k_finalize(const ST* __restrict__ W, const double* __restrict__ norm64, int64_t M,
                           const int32_t* __restrict__ indptr, const int32_t* __restrict__ indices,
                           int64_t n, const unsigned long long* __restrict__ keys,
                           int32_t* __restrict__ bmu, float* __restrict__ dist,
                           const int32_t* __restrict__ sample_list, const float* __restrict__ values = nullptr)
{
    const int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= n) return;
    const int64_t s = sample_list ? (int64_t)sample_list[k] : k;
    const uint32_t idx = (uint32_t)(keys[k] & 0xffffffffull);
    if (idx >= M) {  // only a second-best key can be empty: fewer than two neurons
        bmu[s] = -1;
        dist[s] = __int_as_float(0x7f800000);
        return;
    }
    const int beg = indptr[s];
    const int end = indptr[s + 1];
    double dot = 0.0, xx = (double)(end - beg);
    if (values) {
        xx = 0.0;
        for (int j = beg; j < end; ++j) {
            const double x = (double)values[j];
            xx += x * x;
            dot += x * (double)som_weight(W + (int64_t)indices[j] * M + idx);
        }
    } else {
        for (int j = beg; j < end; ++j) dot += (double)som_weight(W + (int64_t)indices[j] * M + idx);
    }
    bmu[s] = (int32_t)idx;
    dist[s] = (float)(xx - 2.0 * dot + norm64[idx]);
}

__global__ void k_validate(const int32_t* __restrict__ indptr, const int32_t* __restrict__ indices,
                           int64_t n, int V, int* __restrict__ flag)
{
    const int64_t s = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= n) return;
    const int beg = indptr[s];
    const int end = indptr[s + 1];
    bool bad = end < beg || beg < 0;
    if (!bad) {
        int prev = -1;
        for (int j = beg; j < end; ++j) {
            const int v = indices[j];
            if (v <= prev || v >= V) { bad = true; break; }
            prev = v;
        }
    }
    if (bad) atomicExch(flag, 1);
}

}  // namespace

int som_launch_bmu_direct(som_handle* h, const int32_t* indptr, const int32_t* indices, int64_t n,
                          unsigned long long* keys, unsigned long long* keys2, const int32_t* sample_list,
                          cudaStream_t st)
{
    const int vec = (h->M % 4 == 0) ? 4 : 1;
    const int64_t per_block = (int64_t)DIRECT_WARPS * DIRECT_SAMPLES_PER_WARP;
    const int64_t gx = (n + per_block - 1) / per_block;
    const int64_t neurons_per_block = 32 * vec;
    int64_t gy = (h->M + neurons_per_block - 1) / neurons_per_block;
    // gridDim.y is limited to 65535: walk the neuron axis in slices
    const int64_t max_gy = 65535;
    for (int64_t y0 = 0; y0 < gy; y0 += max_gy) {
        const int64_t ny = (gy - y0 < max_gy) ? gy - y0 : max_gy;
        dim3 grid((unsigned)gx, (unsigned)ny);
        const int64_t neuron_off = y0 * neurons_per_block;
#define SOM_DIRECT(VEC_, TOP2_, ST_, W_)                                                          \
    k_bmu_direct<VEC_, TOP2_, ST_><<<grid, DIRECT_THREADS, 0, st>>>(W_, h->hnorm, h->M, indptr, indices, n, \
                                                                    keys, keys2, neuron_off, sample_list)
        if (h->Wh) {
            if (vec == 4 && !keys2) SOM_DIRECT(4, false, __half, h->Wh);
            else if (vec == 4) SOM_DIRECT(4, true, __half, h->Wh);
            else if (!keys2) SOM_DIRECT(1, false, __half, h->Wh);
            else SOM_DIRECT(1, true, __half, h->Wh);
        } else {
            if (vec == 4 && !keys2) SOM_DIRECT(4, false, float, h->W);
            else if (vec == 4) SOM_DIRECT(4, true, float, h->W);
            else if (!keys2) SOM_DIRECT(1, false, float, h->W);
            else SOM_DIRECT(1, true, float, h->W);
        }
#undef SOM_DIRECT
        SOM_CK(h, cudaGetLastError());
        h->launches += 1;
    }
    return SOM_OK;
}

// Sparse real-valued samples: always the direct-load kernel, best unit only.
int som_launch_bmu_values(som_handle* h, const int32_t* indptr, const int32_t* indices, const float* values,
                          int64_t n, unsigned long long* keys, cudaStream_t st)
{
    const int vec = (h->M % 4 == 0) ? 4 : 1;
    const int64_t per_block = (int64_t)DIRECT_WARPS * DIRECT_SAMPLES_PER_WARP;
    const int64_t gx = (n + per_block - 1) / per_block;
    const int64_t neurons_per_block = 32 * vec;
    const int64_t gy = (h->M + neurons_per_block - 1) / neurons_per_block;
    const int64_t max_gy = 65535;
    for (int64_t y0 = 0; y0 < gy; y0 += max_gy) {
        const int64_t ny = (gy - y0 < max_gy) ? gy - y0 : max_gy;
        dim3 grid((unsigned)gx, (unsigned)ny);
        const int64_t neuron_off = y0 * neurons_per_block;
#define SOM_VALUED(VEC_, ST_, W_)                                                                     \
    k_bmu_direct<VEC_, false, ST_, true><<<grid, DIRECT_THREADS, 0, st>>>(W_, h->hnorm, h->M, indptr, indices, n, \
                                                                          keys, nullptr, neuron_off, nullptr, values)
        if (h->Wh) {
            if (vec == 4) SOM_VALUED(4, __half, h->Wh);
            else SOM_VALUED(1, __half, h->Wh);
        } else {
            if (vec == 4) SOM_VALUED(4, float, h->W);
            else SOM_VALUED(1, float, h->W);
        }
#undef SOM_VALUED
        SOM_CK(h, cudaGetLastError());
        h->launches += 1;
    }
    return SOM_OK;
}

int som_launch_finalize_values(som_handle* h, const int32_t* indptr, const int32_t* indices, const float* values,
                               int64_t n, const unsigned long long* keys, int32_t* bmu, float* dist,
                               cudaStream_t st)
{
    const int64_t blocks = (n + 255) / 256;
    if (h->Wh)
        k_finalize<__half><<<(unsigned)blocks, 256, 0, st>>>(h->Wh, h->norm64, h->M, indptr, indices, n, keys,
                                                             bmu, dist, nullptr, values);
    else
        k_finalize<float><<<(unsigned)blocks, 256, 0, st>>>(h->W, h->norm64, h->M, indptr, indices, n, keys,
                                                            bmu, dist, nullptr, values);
    SOM_CK(h, cudaGetLastError());
    h->launches += 1;
    return SOM_OK;
}

int som_launch_finalize(som_handle* h, const int32_t* indptr, const int32_t* indices, int64_t n,
                        const unsigned long long* keys, int32_t* bmu, float* dist, const int32_t* sample_list,
                        cudaStream_t st)
{
    const int64_t blocks = (n + 255) / 256;
    if (h->Wh)
        k_finalize<__half><<<(unsigned)blocks, 256, 0, st>>>(h->Wh, h->norm64, h->M, indptr, indices, n, keys,
                                                             bmu, dist, sample_list);
    else
        k_finalize<float><<<(unsigned)blocks, 256, 0, st>>>(h->W, h->norm64, h->M, indptr, indices, n, keys,
                                                            bmu, dist, sample_list);
    SOM_CK(h, cudaGetLastError());
    h->launches += 1;
    return SOM_OK;
}

int som_launch_validate(som_handle* h, const int32_t* indptr, const int32_t* indices, int64_t n,
                        int* d_flag, cudaStream_t st)
{
    const int64_t blocks = (n + 255) / 256;
    k_validate<<<(unsigned)blocks, 256, 0, st>>>(indptr, indices, n, h->V, d_flag);
    SOM_CK(h, cudaGetLastError());
    h->launches += 1;
    return SOM_OK;
}
