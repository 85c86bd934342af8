// Direct-load BMU search kernel, winner finalisation and CSR validation.
//
// k_bmu_direct is the simplest complete statement of the fused search (Section 3.3):
// a warp owns one sample at a time and up to 512 adjacent neurons (TILES tiles of 32*VEC);
// every lane keeps TILES*VEC score accumulators in registers, seeded with ||w_i||^2 / 2, and for
// each active feature v subtracts the contiguous segment W[v*M + i .. i+VEC) of each tile, fetched
// with one vector load (feature-major layout: the warp's 32 loads cover 512 contiguous bytes of
// fp32), four features at a time so that their loads are in flight together.  The argmin over the
// warp's neurons is a shuffle reduction on (score, index) with ties to the lower index, and
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

// A lane's VEC adjacent weights of one feature row, as loaded (one vector load), and the
// accumulation of such a segment into the lane's scores.  NEG: the scores are held negated,
// sum(rows) - ||w||^2/2, because fp16 weights enter through the mixed-precision add
// (add.rn.f32.f16 widens the weight exactly and rounds once, like the fp32 subtraction, but only
// adds); (-a) - w and -(a + w) round identically, so the scores are those of the subtracting form.
template <typename ST, int VEC> struct Seg;
template <> struct Seg<float, 1> {
    float v;
    static constexpr bool NEG = false;
    __device__ __forceinline__ void load(const float* p) { v = __ldg(p); }
    template <bool VALUED>
    __device__ __forceinline__ void apply(float (&acc)[1], float x) const
    {
        acc[0] = VALUED ? fmaf(-x, v, acc[0]) : acc[0] - v;
    }
};
template <> struct Seg<float, 4> {
    float4 v;
    static constexpr bool NEG = false;
    __device__ __forceinline__ void load(const float* p) { v = __ldg(reinterpret_cast<const float4*>(p)); }
    template <bool VALUED>
    __device__ __forceinline__ void apply(float (&acc)[4], float x) const
    {
        acc[0] = VALUED ? fmaf(-x, v.x, acc[0]) : acc[0] - v.x;
        acc[1] = VALUED ? fmaf(-x, v.y, acc[1]) : acc[1] - v.y;
        acc[2] = VALUED ? fmaf(-x, v.z, acc[2]) : acc[2] - v.z;
        acc[3] = VALUED ? fmaf(-x, v.w, acc[3]) : acc[3] - v.w;
    }
};
template <> struct Seg<__half, 1> {
    float v;
    static constexpr bool NEG = false;
    __device__ __forceinline__ void load(const __half* p) { v = __half2float(__ldg(p)); }
    template <bool VALUED>
    __device__ __forceinline__ void apply(float (&acc)[1], float x) const
    {
        acc[0] = VALUED ? fmaf(-x, v, acc[0]) : acc[0] - v;
    }
};
// two fp16 weights of one 32-bit word added to two (negated) scores
__device__ __forceinline__ void add_h2(float& d0, float& d1, uint32_t w)
{
    asm("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %2;\n\t"
        "add.rn.f32.f16 %0, l, %0;\n\tadd.rn.f32.f16 %1, h, %1;\n\t}"
        : "+f"(d0), "+f"(d1) : "r"(w));
}
__device__ __forceinline__ void fma_h2(float& d0, float& d1, float x, uint32_t w)
{
    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w));
    d0 = fmaf(-x, f.x, d0);
    d1 = fmaf(-x, f.y, d1);
}
template <> struct Seg<__half, 4> {
    uint2 v;
    static constexpr bool NEG = true;  // (only without values: real-valued samples multiply in fp32)
    __device__ __forceinline__ void load(const __half* p) { v = __ldg(reinterpret_cast<const uint2*>(p)); }
    template <bool VALUED>
    __device__ __forceinline__ void apply(float (&acc)[4], float x) const
    {
        if (VALUED) { fma_h2(acc[0], acc[1], x, v.x); fma_h2(acc[2], acc[3], x, v.y); }
        else { add_h2(acc[0], acc[1], v.x); add_h2(acc[2], acc[3], v.y); }
    }
};
template <> struct Seg<__half, 8> {
    uint4 v;
    static constexpr bool NEG = true;
    __device__ __forceinline__ void load(const __half* p) { v = __ldg(reinterpret_cast<const uint4*>(p)); }
    template <bool VALUED>
    __device__ __forceinline__ void apply(float (&acc)[8], float x) const
    {
        if (VALUED) {
            fma_h2(acc[0], acc[1], x, v.x); fma_h2(acc[2], acc[3], x, v.y);
            fma_h2(acc[4], acc[5], x, v.z); fma_h2(acc[6], acc[7], x, v.w);
        } else {
            add_h2(acc[0], acc[1], v.x); add_h2(acc[2], acc[3], v.y);
            add_h2(acc[4], acc[5], v.z); add_h2(acc[6], acc[7], v.w);
        }
    }
};

// TOP2 also keeps the second-best unit in keys2 (Algorithm 2 keeps the two best units).
// ST is the storage type of the codebook (float, or __half widened exactly before the fp32 add).
// VALUED: sparse real-valued samples (a values array parallel to the indices; the paper's outlook,
// Section 7): the gather-sum becomes a gather-multiply, score = ||w||^2/2 - sum_k x_k * w[idx_k].
// TILES: a warp covers TILES adjacent tiles of 32*VEC neurons per sample, so that the feature
// broadcast, the row address and the shuffle argmin are paid once per TILES tiles.
// WALK: the block walks the sample groups blockIdx.x, blockIdx.x + gridDim.x, ... instead of taking one
// (launches that mostly return at once, or whose sample count only the device knows, come with a small grid).
template <int VEC, int TILES, bool TOP2, typename ST, bool VALUED = false, bool WALK = false>
__global__ void __launch_bounds__(DIRECT_THREADS, 2)
k_bmu_direct(const ST* __restrict__ W, const float* __restrict__ hnorm, int64_t M, uint32_t row_bytes,
             const int32_t* __restrict__ indptr, const int32_t* __restrict__ indices, int64_t n,
             unsigned long long* __restrict__ keys, unsigned long long* __restrict__ keys2,
             int64_t neuron_off, const int32_t* __restrict__ sample_list,
             const float* __restrict__ values = nullptr, const int* __restrict__ gate = nullptr, int gate_want = 0,
             int sample_groups = 0, const int* __restrict__ n_dev = nullptr)
{
    if constexpr (WALK) {  // (gates and device-side sample counts come with the walking form only)
        if (som_gated_off(gate, gate_want)) return;
        if (n_dev) n = *n_dev;  // length of a sample list that lives on the device
    }
    constexpr int TILE = 32 * VEC;  // neurons per tile
    // features whose row segments are in flight together (fp16 rows are half as long: twice as many)
    constexpr int FEATS = sizeof(ST) == 2 ? 8 : 4;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int64_t i0 = neuron_off + (int64_t)blockIdx.y * (TILES * TILE) + lane * VEC;
    const float inf = __int_as_float(0x7f800000);

    constexpr bool NEG = Seg<ST, VEC>::NEG && !VALUED;  // scores held negated
    float seed[TILES][VEC];
    bool live[TILES];  // with VEC >= 4, M % VEC == 0: all of the lane's neurons of a tile or none
#pragma unroll
    for (int t = 0; t < TILES; ++t) {
        live[t] = i0 + t * TILE < M;
#pragma unroll
        for (int k = 0; k < VEC; ++k) {
            const float hn = (i0 + t * TILE + k < M) ? hnorm[i0 + t * TILE + k] : inf;
            seed[t][k] = NEG ? -hn : hn;
        }
    }
    // byte address of the lane's first neuron in feature row 0; row v is row_bytes * v further on
    const char* W_lane = reinterpret_cast<const char*>(W + (live[0] ? i0 : 0));

    int bx = blockIdx.x;
    if (WALK && bx >= sample_groups) return;
    do {
    const int64_t s0 = ((int64_t)bx * DIRECT_WARPS + warp) * DIRECT_SAMPLES_PER_WARP;
    const int n_mine = (int)min((int64_t)DIRECT_SAMPLES_PER_WARP, n - s0);
    if (n_mine <= 0) break;  // (later groups lie further on)
    // lane q holds the row bounds of the warp's q-th sample
    // (with a sample list, position s of the list and of the key arrays is sample list[s])
    int beg_l = 0, end_l = 0;
    if (lane < n_mine) {
        const int64_t sid = sample_list ? (int64_t)sample_list[s0 + lane] : s0 + lane;
        beg_l = indptr[sid];
        end_l = indptr[sid + 1];
    }
    int beg = __shfl_sync(0xffffffffu, beg_l, 0);
    int end = __shfl_sync(0xffffffffu, end_l, 0);
    int first = (beg + lane < end) ? indices[beg + lane] : 0;
    float first_x = (VALUED && beg + lane < end) ? values[beg + lane] : 1.f;
    // The key a sample's candidates are tested against before any index is tracked: its best so
    // far, or with TOP2 its second best so far (a stale, larger value only lets more through).
    // Lane q reads the key of the warp's q-th sample; volatile: other blocks lower it meanwhile.
    const unsigned long long* filter_keys = TOP2 ? keys2 : keys;
    unsigned long long key_l = ~0ull;
    if (lane < n_mine) key_l = *reinterpret_cast<const volatile unsigned long long*>(filter_keys + s0 + lane);

    for (int q = 0; q < n_mine; ++q) {
        // the next sample's first 32 features are fetched while this one is searched
        const int nbeg = __shfl_sync(0xffffffffu, beg_l, (q + 1) & 31);
        const int nend = (q + 1 < n_mine) ? __shfl_sync(0xffffffffu, end_l, (q + 1) & 31) : nbeg;
        const int next = (nbeg + lane < nend) ? indices[nbeg + lane] : 0;
        const float next_x = (VALUED && nbeg + lane < nend) ? values[nbeg + lane] : 1.f;

        float acc[TILES][VEC];
#pragma unroll
        for (int t = 0; t < TILES; ++t)
#pragma unroll
            for (int k = 0; k < VEC; ++k) acc[t][k] = seed[t][k];
        for (int base = beg; base < end; base += 32) {
            int mine = first;
            float mine_x = first_x;
            if (base != beg) {
                mine = (base + lane < end) ? indices[base + lane] : 0;
                mine_x = (VALUED && base + lane < end) ? values[base + lane] : 1.f;
            }
            const int cnt = min(32, end - base);
            int j = 0;
            // FEATS features at a time; the subtractions keep the ascending feature order
            for (; j + FEATS <= cnt; j += FEATS) {
                const char* p[FEATS];
                float x[FEATS];
#pragma unroll
                for (int u = 0; u < FEATS; ++u) {
                    p[u] = W_lane + (uint64_t)(uint32_t)__shfl_sync(0xffffffffu, mine, j + u) * row_bytes;
                    x[u] = VALUED ? __shfl_sync(0xffffffffu, mine_x, j + u) : 1.f;
                }
#pragma unroll
                for (int t = 0; t < TILES; ++t) {
                    if (!live[t]) continue;
                    Seg<ST, VEC> w[FEATS];
#pragma unroll
                    for (int u = 0; u < FEATS; ++u) w[u].load(reinterpret_cast<const ST*>(p[u]) + t * TILE);
#pragma unroll
                    for (int u = 0; u < FEATS; ++u) w[u].template apply<VALUED>(acc[t], x[u]);
                }
            }
            for (; j < cnt; ++j) {
                const char* p = W_lane + (uint64_t)(uint32_t)__shfl_sync(0xffffffffu, mine, j) * row_bytes;
                const float x = VALUED ? __shfl_sync(0xffffffffu, mine_x, j) : 1.f;
#pragma unroll
                for (int t = 0; t < TILES; ++t) {
                    if (!live[t]) continue;
                    Seg<ST, VEC> w;
                    w.load(reinterpret_cast<const ST*>(p) + t * TILE);
                    w.template apply<VALUED>(acc[t], x);
                }
            }
        }
        if (NEG) {
#pragma unroll
            for (int t = 0; t < TILES; ++t)
#pragma unroll
                for (int k = 0; k < VEC; ++k) acc[t][k] = -acc[t][k];
        }
        // Most visits change nothing: unless some lane's smallest score reaches the sample's
        // current key, the indices, the shuffles and the atomics are skipped.
        {
            float mn = acc[0][0];
#pragma unroll
            for (int e = 1; e < TILES * VEC; ++e) mn = fminf(mn, acc[e / VEC][e % VEC]);
            const uint32_t cu = (uint32_t)(__shfl_sync(0xffffffffu, key_l, q) >> 32);
            const float cs = __uint_as_float((cu & 0x80000000u) ? (cu ^ 0x80000000u) : ~cu);  // NaN for an empty key
            if (!__any_sync(0xffffffffu, !(mn > cs))) {
                beg = nbeg;
                end = nend;
                first = next;
                first_x = next_x;
                continue;
            }
        }
        // the lane's best (and second best) in ascending neuron order, then across the warp
        float best = acc[0][0];
        uint32_t bi = (uint32_t)i0;
        float second = inf;            // TOP2: the lane's, then the warp's, second best
        uint32_t si = 0xffffffffu;
#pragma unroll
        for (int e = 1; e < TILES * VEC; ++e) {
            const float a = acc[e / VEC][e % VEC];
            const uint32_t ie = (uint32_t)(i0 + (e / VEC) * TILE + e % VEC);
            if (a < best) {
                if (TOP2) { second = best; si = bi; }
                best = a;
                bi = ie;
            } else if (TOP2 && before(a, ie, second, si)) {
                second = a;
                si = ie;
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
            const int64_t s = s0 + q;
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
        beg = nbeg;
        end = nend;
        first = next;
        first_x = next_x;
    }
    } while (WALK && (bx += (int)gridDim.x) < sample_groups);
}

// One thread per sample: unpack the winner and recompute its full squared distance
// |S| - 2*dot + ||w||^2 (left side of Eq. 1) in fp64, ascending feature order.
template <typename ST>
__global__ void k_finalize(const ST* __restrict__ W, const double* __restrict__ norm64, int64_t M,
                           const int32_t* __restrict__ indptr, const int32_t* __restrict__ indices,
                           int64_t n, const unsigned long long* __restrict__ keys,
                           int32_t* __restrict__ bmu, float* __restrict__ dist,
                           const int32_t* __restrict__ sample_list, const float* __restrict__ values = nullptr,
                           const int* __restrict__ gate = nullptr, int gate_want = 0,
                           const int* __restrict__ n_dev = nullptr)
{
    if (som_gated_off(gate, gate_want)) return;
    if (n_dev) n = *n_dev;  // length of a sample list that lives on the device
    for (int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; k < n; k += (int64_t)gridDim.x * blockDim.x) {
    const int64_t s = sample_list ? (int64_t)sample_list[k] : k;
    const uint32_t idx = (uint32_t)(keys[k] & 0xffffffffull);
    if (idx >= M) {  // only a second-best key can be empty: fewer than two neurons
        bmu[s] = -1;
        dist[s] = __int_as_float(0x7f800000);
        continue;
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

// Neurons per lane and tile (one vector load: 16 bytes of fp32, 8 or 16 of fp16) and tiles per
// warp: 512 neurons per warp and sample, fewer on maps that have fewer (measured at 64x64: four
// tiles with four features in flight beat one and two tiles on Zipf and on uniform features alike).
static int direct_vec(int64_t M, bool half) { return (half && M % 8 == 0) ? 8 : (M % 4 == 0 ? 4 : 1); }
static int direct_tiles(int64_t M, int vec)
{
    const int64_t tile = 32 * vec;
    const int most = vec == 8 ? 2 : 4;
    int tiles = 1;
    while (tiles < most && M > tiles * tile) tiles *= 2;
    return tiles;
}

template <int VEC, int TILES, typename ST>
static void launch_direct(dim3 grid, cudaStream_t st, const ST* W, som_handle* h, const int32_t* indptr,
                          const int32_t* indices, int64_t n, unsigned long long* keys,
                          unsigned long long* keys2, int64_t neuron_off, const int32_t* sample_list,
                          const float* values, int sample_groups, bool walk)
{
    const uint32_t row_bytes = (uint32_t)(h->M * (int64_t)sizeof(ST));
#define SOM_DIRECT_GO(TOP2_, VALUED_, WALK_, K2_, SL_, VAL_)                                                      \
    k_bmu_direct<VEC, TILES, TOP2_, ST, VALUED_, WALK_><<<grid, DIRECT_THREADS, 0, st>>>(                         \
        W, h->hnorm, h->M, row_bytes, indptr, indices, n, keys, K2_, neuron_off, SL_, VAL_, h->gate, h->gate_want, \
        sample_groups, h->list_len_dev)
    if (values) SOM_DIRECT_GO(false, true, false, nullptr, nullptr, values);
    else if (keys2 && walk) SOM_DIRECT_GO(true, false, true, keys2, sample_list, nullptr);
    else if (keys2) SOM_DIRECT_GO(true, false, false, keys2, sample_list, nullptr);
    else if (walk) SOM_DIRECT_GO(false, false, true, nullptr, sample_list, nullptr);
    else SOM_DIRECT_GO(false, false, false, nullptr, sample_list, nullptr);
#undef SOM_DIRECT_GO
}

template <typename ST>
static int launch_direct_any(som_handle* h, const ST* W, const int32_t* indptr, const int32_t* indices,
                             const float* values, int64_t n, unsigned long long* keys,
                             unsigned long long* keys2, const int32_t* sample_list, cudaStream_t st)
{
    if (h->M * (int64_t)sizeof(ST) > 0xffffffffll) return SOM_ERR_INVALID_ARG;  // 32-bit row pitch
    const int vec = direct_vec(h->M, sizeof(ST) == 2);
    const int tiles = direct_tiles(h->M, vec);
    const int64_t per_block = (int64_t)DIRECT_WARPS * DIRECT_SAMPLES_PER_WARP;
    const int64_t gx = (n + per_block - 1) / per_block;
    const int64_t neurons_per_block = (int64_t)32 * vec * tiles;
    const int64_t gy = (h->M + neurons_per_block - 1) / neurons_per_block;
    // gridDim.y is limited to 65535: walk the neuron axis in slices
    const int64_t max_gy = 65535;
    for (int64_t y0 = 0; y0 < gy; y0 += max_gy) {
        const int64_t ny = (gy - y0 < max_gy) ? gy - y0 : max_gy;
        // a gated launch returns at once on most calls: keep it to about 2048 blocks, each of which walks
        // several sample groups when it does run
        int64_t gx_launch = gx;
        // gated launches and launches over a device-side list take the walking form of the kernel; those
        // expected to be idle, and the lists (short), come with a small grid
        const bool walk = (h->gate || h->list_len_dev) && !values;
        if ((h->gate_small_grid || h->list_len_dev) && walk && gx * ny > 2048) gx_launch = 2048 / ny > 1 ? 2048 / ny : 1;
        dim3 grid((unsigned)gx_launch, (unsigned)ny);
        const int64_t neuron_off = y0 * neurons_per_block;
#define SOM_DIRECT(VEC_, TILES_) \
    launch_direct<VEC_, TILES_, ST>(grid, st, W, h, indptr, indices, n, keys, keys2, neuron_off, sample_list, values, (int)gx, walk)
        if constexpr (sizeof(ST) == 2) {
            if (vec == 8 && tiles == 2) SOM_DIRECT(8, 2);
            else if (vec == 8) SOM_DIRECT(8, 1);
        }
        if (vec == 8) {}
        else if (vec == 4 && tiles == 4) SOM_DIRECT(4, 4);
        else if (vec == 4 && tiles == 2) SOM_DIRECT(4, 2);
        else if (vec == 4) SOM_DIRECT(4, 1);
        else if (tiles == 4) SOM_DIRECT(1, 4);
        else if (tiles == 2) SOM_DIRECT(1, 2);
        else SOM_DIRECT(1, 1);
#undef SOM_DIRECT
        SOM_CK(h, cudaGetLastError());
        h->launches += 1;
    }
    return SOM_OK;
}

int som_launch_bmu_direct(som_handle* h, const int32_t* indptr, const int32_t* indices, int64_t n,
                          unsigned long long* keys, unsigned long long* keys2, const int32_t* sample_list,
                          cudaStream_t st)
{
    if (h->Wh) return launch_direct_any(h, h->Wh, indptr, indices, nullptr, n, keys, keys2, sample_list, st);
    return launch_direct_any(h, h->W, indptr, indices, nullptr, n, keys, keys2, sample_list, st);
}

// Sparse real-valued samples: always the direct-load kernel, best unit only.
int som_launch_bmu_values(som_handle* h, const int32_t* indptr, const int32_t* indices, const float* values,
                          int64_t n, unsigned long long* keys, cudaStream_t st)
{
    if (h->Wh) return launch_direct_any(h, h->Wh, indptr, indices, values, n, keys, nullptr, nullptr, st);
    return launch_direct_any(h, h->W, indptr, indices, values, n, keys, nullptr, nullptr, st);
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
    int64_t blocks = (n + 255) / 256;
    if (h->list_len_dev && blocks > 64) blocks = 64;  // a list whose (short) length lives on the device
    if (h->Wh)
        k_finalize<__half><<<(unsigned)blocks, 256, 0, st>>>(h->Wh, h->norm64, h->M, indptr, indices, n, keys,
                                                             bmu, dist, sample_list, nullptr, h->gate, h->gate_want,
                                                             h->list_len_dev);
    else
        k_finalize<float><<<(unsigned)blocks, 256, 0, st>>>(h->W, h->norm64, h->M, indptr, indices, n, keys,
                                                            bmu, dist, sample_list, nullptr, h->gate, h->gate_want,
                                                            h->list_len_dev);
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
