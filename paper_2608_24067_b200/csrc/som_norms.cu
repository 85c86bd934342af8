// Per-neuron squared norms ||w_i||^2 of a feature-major codebook (the norm term of Eq. 1).
//
// HBM-bound streaming pass: each thread owns VEC adjacent neurons and walks down the
// feature rows with 128-bit loads (a warp reads 512 contiguous bytes of one row), several
// rows in flight.  Squares are accumulated in fp64.  The V axis is split across blockIdx.y
// so that small maps still fill 148 SMs; the per-split partial sums are combined in a second
// kernel in ascending split order, which keeps the result independent of scheduling.
#include "som_internal.cuh"

namespace {

constexpr int NORM_THREADS = 128;
constexpr int NORM_UNROLL = 8;

// four floats -> four halves (round to nearest even), one 64-bit store
__device__ __forceinline__ void store_half4(__half* dst, const float4 w)
{
    const __half2 a = __floats2half2_rn(w.x, w.y);
    const __half2 b = __floats2half2_rn(w.z, w.w);
    uint2 v;
    v.x = *reinterpret_cast<const uint32_t*>(&a);
    v.y = *reinterpret_cast<const uint32_t*>(&b);
    *reinterpret_cast<uint2*>(dst) = v;
}

// SHADOW (VEC == 4 only): the pass also writes an fp16 copy of the codebook and the largest
// |weight| (as float bits, through atomicMax: non-negative floats order like their bits), which
// the two-stage search uses for its first pass and its error bound.
// RMAX (VEC == 4 and M % 128 == 0 only): the pass also writes, for every feature row and every range of 128
// neurons (the 128 neurons a warp holds), the largest weight of the row in each of the range's four groups of
// 32 neurons: range_max[(range * V + v) * 4 + group].  The row-table search uses them to bound what a sample's
// rows can still take off the scores of a range (see k_bmu_table).
__device__ __forceinline__ void store_range_max(float* __restrict__ dst, float m)
{
    // max over each group of eight lanes (32 neurons) in one instruction: floats ordered as signed integers
    int key = __float_as_int(m);
    key ^= (key >> 31) & 0x7fffffff;
    const unsigned int lane = threadIdx.x & 31;
    key = __reduce_max_sync(0xffu << (lane & 24), key);
    key ^= (key >> 31) & 0x7fffffff;
    if ((lane & 7) == 0) dst[lane >> 3] = __int_as_float(key);
}

template <int VEC, bool SHADOW, bool RMAX>
__global__ void __launch_bounds__(NORM_THREADS)
k_norms_partial(const float* __restrict__ W, int64_t M, int V, int rows_per_split,
                double* __restrict__ partial, __half* __restrict__ shadow, unsigned int* __restrict__ wmax_bits,
                float* __restrict__ range_max)
{
    const int64_t i = ((int64_t)blockIdx.x * NORM_THREADS + threadIdx.x) * VEC;
    if (i >= M) return;
    const int v0 = blockIdx.y * rows_per_split;
    const int v1 = min(V, v0 + rows_per_split);
    double acc[VEC];
#pragma unroll
    for (int k = 0; k < VEC; ++k) acc[k] = 0.0;
    const float* p = W + (int64_t)v0 * M + i;
    __half* ps = SHADOW ? shadow + (int64_t)v0 * M + i : nullptr;
    float wmax = 0.f, wmin = 0.f;
    // (RMAX: M % 128 == 0, so a warp is all inside M and holds exactly range i / 128)
    float* pr = RMAX ? range_max + ((i / 128) * (int64_t)V + v0) * 4 : nullptr;
    int v = v0;
    if (VEC == 4) {
        for (; v + NORM_UNROLL <= v1; v += NORM_UNROLL) {
            float4 w[NORM_UNROLL];
#pragma unroll
            for (int u = 0; u < NORM_UNROLL; ++u)
                w[u] = __ldcs(reinterpret_cast<const float4*>(p + (int64_t)u * M));
#pragma unroll
            for (int u = 0; u < NORM_UNROLL; ++u) {
                if (SHADOW) {
                    store_half4(ps + (int64_t)u * M, w[u]);
                    wmax = fmaxf(wmax, fmaxf(fmaxf(fabsf(w[u].x), fabsf(w[u].y)), fmaxf(fabsf(w[u].z), fabsf(w[u].w))));
                    wmin = fminf(wmin, fminf(fminf(w[u].x, w[u].y), fminf(w[u].z, w[u].w)));
                }
                if (RMAX) store_range_max(pr + 4 * u, fmaxf(fmaxf(w[u].x, w[u].y), fmaxf(w[u].z, w[u].w)));
                acc[0] = fma((double)w[u].x, (double)w[u].x, acc[0]);
                acc[1 % VEC] = fma((double)w[u].y, (double)w[u].y, acc[1 % VEC]);
                acc[2 % VEC] = fma((double)w[u].z, (double)w[u].z, acc[2 % VEC]);
                acc[3 % VEC] = fma((double)w[u].w, (double)w[u].w, acc[3 % VEC]);
            }
            p += (int64_t)NORM_UNROLL * M;
            if (SHADOW) ps += (int64_t)NORM_UNROLL * M;
            if (RMAX) pr += 4 * NORM_UNROLL;
        }
        for (; v < v1; ++v) {
            float4 w = __ldcs(reinterpret_cast<const float4*>(p));
            if (SHADOW) {
                store_half4(ps, w);
                wmax = fmaxf(wmax, fmaxf(fmaxf(fabsf(w.x), fabsf(w.y)), fmaxf(fabsf(w.z), fabsf(w.w))));
                wmin = fminf(wmin, fminf(fminf(w.x, w.y), fminf(w.z, w.w)));
                ps += M;
            }
            if (RMAX) {
                store_range_max(pr, fmaxf(fmaxf(w.x, w.y), fmaxf(w.z, w.w)));
                pr += 4;
            }
            acc[0] = fma((double)w.x, (double)w.x, acc[0]);
            acc[1 % VEC] = fma((double)w.y, (double)w.y, acc[1 % VEC]);
            acc[2 % VEC] = fma((double)w.z, (double)w.z, acc[2 % VEC]);
            acc[3 % VEC] = fma((double)w.w, (double)w.w, acc[3 % VEC]);
            p += M;
        }
    } else {
        for (; v < v1; ++v) {
            float w = __ldcs(p);
            acc[0] = fma((double)w, (double)w, acc[0]);
            p += M;
        }
    }
    double* out = partial + (int64_t)blockIdx.y * M + i;
#pragma unroll
    for (int k = 0; k < VEC; ++k) out[k] = acc[k];
    if (SHADOW) {
        // one atomic per warp (lanes past the last neuron have left: reduce over the active ones);
        // NaN weights are outside the preconditions, fmaxf drops them
        const unsigned int active = __activemask();
        const unsigned int best = __reduce_max_sync(active, __float_as_uint(wmax));
        if ((threadIdx.x & 31) == (__ffs(active) - 1)) atomicMax(wmax_bits, best);
        if (wmin < 0.f) wmax_bits[SOM_AUX_HAS_NEGATIVE] = 1u;  // (every writer stores the same value)
    }
}

// The same pass over an fp16-stored codebook: VEC = 8 neurons per thread (one 128-bit load of
// eight halves per row) or 1; every weight is widened exactly and squared in fp64.
// RMAX (VEC == 8, M % 128 == 0): a half-warp (16 threads x 8 neurons) holds one range of 128, four threads a group of 32
// neurons; its largest weight of every row goes to range_max[range * V + v] (see k_norms_partial).
__device__ __forceinline__ void store_range_max_half(float* __restrict__ dst, float m)
{
    // a thread holds 8 neurons, four threads a group of 32, a half-warp the range of 128
    int key = __float_as_int(m);
    key ^= (key >> 31) & 0x7fffffff;
    const unsigned int lane = threadIdx.x & 31;
    key = __reduce_max_sync(0xfu << (lane & 28), key);
    key ^= (key >> 31) & 0x7fffffff;
    if ((lane & 3) == 0) dst[(lane & 15) >> 2] = __int_as_float(key);
}

template <int VEC, bool RMAX>
__global__ void __launch_bounds__(NORM_THREADS)
k_norms_partial_h(const __half* __restrict__ W, int64_t M, int V, int rows_per_split,
                  double* __restrict__ partial, float* __restrict__ range_max)
{
    const int64_t i = ((int64_t)blockIdx.x * NORM_THREADS + threadIdx.x) * VEC;
    if (i >= M) return;
    const int v0 = blockIdx.y * rows_per_split;
    const int v1 = min(V, v0 + rows_per_split);
    double acc[VEC];
#pragma unroll
    for (int k = 0; k < VEC; ++k) acc[k] = 0.0;
    const __half* p = W + (int64_t)v0 * M + i;
    // (RMAX: M % 128 == 0, so a half-warp, 16 threads x 8 neurons, is all inside M and holds range i / 128)
    float* pr = RMAX ? range_max + ((i / 128) * (int64_t)V + v0) * 4 : nullptr;
    int v = v0;
    if (VEC == 8) {
        for (; v + NORM_UNROLL <= v1; v += NORM_UNROLL) {
            uint4 w[NORM_UNROLL];
#pragma unroll
            for (int u = 0; u < NORM_UNROLL; ++u)
                w[u] = __ldcs(reinterpret_cast<const uint4*>(p + (int64_t)u * M));
#pragma unroll
            for (int u = 0; u < NORM_UNROLL; ++u) {
                const uint32_t word[4] = {w[u].x, w[u].y, w[u].z, w[u].w};
                float wm = -3.0e38f;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&word[k]));
                    if (RMAX) wm = fmaxf(wm, fmaxf(f.x, f.y));
                    acc[(2 * k) % VEC] = fma((double)f.x, (double)f.x, acc[(2 * k) % VEC]);
                    acc[(2 * k + 1) % VEC] = fma((double)f.y, (double)f.y, acc[(2 * k + 1) % VEC]);
                }
                if (RMAX) store_range_max_half(pr + 4 * u, wm);
            }
            p += (int64_t)NORM_UNROLL * M;
            if (RMAX) pr += 4 * NORM_UNROLL;
        }
        for (; v < v1; ++v) {
            const uint4 w = __ldcs(reinterpret_cast<const uint4*>(p));
            const uint32_t word[4] = {w.x, w.y, w.z, w.w};
            float wm = -3.0e38f;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&word[k]));
                if (RMAX) wm = fmaxf(wm, fmaxf(f.x, f.y));
                acc[(2 * k) % VEC] = fma((double)f.x, (double)f.x, acc[(2 * k) % VEC]);
                acc[(2 * k + 1) % VEC] = fma((double)f.y, (double)f.y, acc[(2 * k + 1) % VEC]);
            }
            if (RMAX) {
                store_range_max_half(pr, wm);
                pr += 4;
            }
            p += M;
        }
    } else {
        for (; v < v1; ++v) {
            const float w = __half2float(__ldcs(p));
            acc[0] = fma((double)w, (double)w, acc[0]);
            p += M;
        }
    }
    double* out = partial + (int64_t)blockIdx.y * M + i;
#pragma unroll
    for (int k = 0; k < VEC; ++k) out[k] = acc[k];
}

// 32 neurons x 8 groups of splits per block: group g adds splits g, g + 8, ... in order, then
// the eight group sums are added in order (a fixed order: the result does not depend on the run)
constexpr int COMBINE_GROUPS = 8;
__global__ void k_norms_combine(const double* __restrict__ partial, int64_t M, int splits,
                                double* __restrict__ norm64, float* __restrict__ norm32,
                                float* __restrict__ hnorm, unsigned int* __restrict__ hmax_bits)
{
    __shared__ double sh[COMBINE_GROUPS][33];
    const int64_t i = (int64_t)blockIdx.x * 32 + threadIdx.x;
    double s = 0.0;
    if (i < M)
        for (int k = threadIdx.y; k < splits; k += COMBINE_GROUPS) s += partial[(int64_t)k * M + i];
    sh[threadIdx.y][threadIdx.x] = s;
    __syncthreads();
    if (threadIdx.y != 0 || i >= M) return;
    s = sh[0][threadIdx.x];
#pragma unroll
    for (int g = 1; g < COMBINE_GROUPS; ++g) s += sh[g][threadIdx.x];
    norm64[i] = s;
    norm32[i] = (float)s;
    hnorm[i] = (float)(0.5 * s);
    // largest ||w||^2 / 2 over the map (non-negative: its float bits order like unsigned integers)
    if (hmax_bits) atomicMax(hmax_bits, __float_as_uint((float)(0.5 * s)));
}

// The 128-neuron ranges ordered by their smallest ||w||^2 / 2 (one block; bitonic sort in shared memory of up to
// 8192 ranges, ties by range number): the search kernel visits them in this order when it prunes.
constexpr int ORDER_MAX_RANGES = 8192;
__global__ void __launch_bounds__(1024)
k_range_order(const float* __restrict__ hnorm, int n_ranges, int32_t* __restrict__ order)
{
    extern __shared__ unsigned long long okeys[];  // (ordered float bits << 32) | range
    int n_pow = 1;
    while (n_pow < n_ranges) n_pow *= 2;
    for (int r = threadIdx.x; r < n_pow; r += 1024) {
        unsigned long long k = ~0ull;
        if (r < n_ranges) {
            float m = 3.0e38f;
            for (int j = 0; j < 128; ++j) m = fminf(m, hnorm[(int64_t)r * 128 + j]);
            unsigned int b = __float_as_uint(m);  // (norms are non-negative: their bits order like unsigned integers)
            k = ((unsigned long long)b << 32) | (unsigned int)r;
        }
        okeys[r] = k;
    }
    __syncthreads();
    for (int size = 2; size <= n_pow; size *= 2)
        for (int stride = size / 2; stride > 0; stride /= 2) {
            for (int i = threadIdx.x; i < n_pow; i += 1024) {
                const int j = i ^ stride;
                if (j > i) {
                    const bool up = (i & size) == 0;
                    const unsigned long long a = okeys[i], b = okeys[j];
                    if ((a > b) == up) {
                        okeys[i] = b;
                        okeys[j] = a;
                    }
                }
            }
            __syncthreads();
        }
    for (int r = threadIdx.x; r < n_ranges; r += 1024) order[r] = (int32_t)(okeys[r] & 0xffffffffull);
}

struct NormPlan {
    int vec;
    int splits;
    int rows_per_split;
    int64_t col_blocks;
};

NormPlan plan_norms(const som_handle* h)
{
    NormPlan p;
    p.vec = h->Wh ? ((h->M % 8 == 0) ? 8 : 1) : ((h->M % 4 == 0) ? 4 : 1);
    const int64_t col_threads = (h->M + p.vec - 1) / p.vec;
    p.col_blocks = (col_threads + NORM_THREADS - 1) / NORM_THREADS;
    // aim for ~16 resident blocks per SM worth of work, at least 16 rows per split
    int64_t want = ((int64_t)h->sm_count * 16 + p.col_blocks - 1) / p.col_blocks;
    int64_t max_splits = (h->V + 15) / 16;
    if (want > max_splits) want = max_splits;
    if (want < 1) want = 1;
    if (want > 65535) want = 65535;
    p.rows_per_split = (int)((h->V + want - 1) / want);
    p.splits = (h->V + p.rows_per_split - 1) / p.rows_per_split;
    return p;
}

}  // namespace

size_t som_norms_workspace_bytes(const som_handle* h)
{
    NormPlan p = plan_norms(h);
    return (size_t)p.splits * (size_t)h->M * sizeof(double);
}

int som_launch_norms(som_handle* h, cudaStream_t st)
{
    NormPlan p = plan_norms(h);
    double* partial = reinterpret_cast<double*>(h->ws);
    dim3 grid((unsigned)p.col_blocks, (unsigned)p.splits);
    if (h->Wh && p.vec == 8 && h->range_max)
        k_norms_partial_h<8, true><<<grid, NORM_THREADS, 0, st>>>(h->Wh, h->M, h->V, p.rows_per_split, partial,
                                                                  h->range_max);
    else if (h->Wh && p.vec == 8)
        k_norms_partial_h<8, false><<<grid, NORM_THREADS, 0, st>>>(h->Wh, h->M, h->V, p.rows_per_split, partial, nullptr);
    else if (h->Wh)
        k_norms_partial_h<1, false><<<grid, NORM_THREADS, 0, st>>>(h->Wh, h->M, h->V, p.rows_per_split, partial, nullptr);
    else if (p.vec == 4 && h->shadow) {
        SOM_CK(h, cudaMemsetAsync(h->wmax_bits, 0, 4 * sizeof(unsigned int), st));
        if (h->range_max)
            k_norms_partial<4, true, true><<<grid, NORM_THREADS, 0, st>>>(h->W, h->M, h->V, p.rows_per_split, partial,
                                                                          h->shadow, h->wmax_bits, h->range_max);
        else
            k_norms_partial<4, true, false><<<grid, NORM_THREADS, 0, st>>>(h->W, h->M, h->V, p.rows_per_split, partial,
                                                                           h->shadow, h->wmax_bits, nullptr);
    } else if (p.vec == 4 && h->range_max)
        k_norms_partial<4, false, true><<<grid, NORM_THREADS, 0, st>>>(h->W, h->M, h->V, p.rows_per_split, partial,
                                                                       nullptr, nullptr, h->range_max);
    else if (p.vec == 4)
        k_norms_partial<4, false, false><<<grid, NORM_THREADS, 0, st>>>(h->W, h->M, h->V, p.rows_per_split, partial,
                                                                        nullptr, nullptr, nullptr);
    else
        k_norms_partial<1, false, false><<<grid, NORM_THREADS, 0, st>>>(h->W, h->M, h->V, p.rows_per_split, partial,
                                                                        nullptr, nullptr, nullptr);
    SOM_CK(h, cudaGetLastError());
    const int64_t blocks = (h->M + 31) / 32;
    k_norms_combine<<<(unsigned)blocks, dim3(32, COMBINE_GROUPS), 0, st>>>(
        partial, h->M, p.splits, h->norm64, h->norm32, h->hnorm,
        (p.vec == 4 && h->shadow && !h->Wh) ? h->wmax_bits + SOM_AUX_HMAX : nullptr);
    SOM_CK(h, cudaGetLastError());
    h->launches += 2;
    if (h->range_order) {
        const int n_ranges = (int)(h->M / 128);
        int n_pow = 1;
        while (n_pow < n_ranges) n_pow *= 2;
        SOM_CK(h, cudaFuncSetAttribute(k_range_order, cudaFuncAttributeMaxDynamicSharedMemorySize, n_pow * 8));
        k_range_order<<<1, 1024, (size_t)n_pow * 8, st>>>(h->hnorm, n_ranges, h->range_order);
        SOM_CK(h, cudaGetLastError());
        h->launches += 1;
    }
    return SOM_OK;
}
