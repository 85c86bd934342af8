// Per-batch plan of the row-table BMU kernel: the merged feature lists of a sample tile
// (Section 3.3), pushed from one tile to the whole batch.
//
//   1. feature histogram of the batch                      (k_feat_hist)
//   2. pick the 16 most frequent features ("mask" features) and the next H ("hot" features);
//      give each a slot in the shared-memory row table      (k_select_hot, one block)
//   3. classify each sample: 16-bit mask of mask features, number of hot / tail features,
//      and count sort bins keyed on (mask, length class)    (k_classify)
//   4. exclusive scan of the bins                           (k_scan_*)
//   5. scatter every sample to its sorted position and write its fixed-size slot there:
//      hot features as byte offsets of their table row, tail features as feature ids
//      (k_scatter_slots); the rare sample that does not fit a slot is marked and listed, and the
//      direct-load kernel searches that list after the row-table kernel.
//
// Samples that share a mask end up adjacent, so the search kernel keeps
// ||w||^2/2 - sum(mask rows) in registers across them (the corpus-clustering lever of
// Section 7 of the paper, which shrinks a tile's feature union, taken to the register level).
// Nothing here depends on the neuron range, so the plan is built once per batch.
#include "som_internal.cuh"
#include "som_plan.cuh"

namespace {

constexpr int PLAN_THREADS = 256;

__device__ __forceinline__ int warp_incl_scan(int v, int lane)
{
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

// Exclusive scan of one int per thread over a 1024-thread block; returns the exclusive prefix,
// *total receives the block sum.  warp_sums must hold 32 ints of shared memory.
__device__ int block_excl_scan_1024(int v, int* warp_sums, int* total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int incl = warp_incl_scan(v, lane);
    __syncthreads();
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int s = warp_sums[lane];
        int si = warp_incl_scan(s, lane);
        warp_sums[lane] = si - s;
        if (lane == 31) *total = si;
    }
    __syncthreads();
    return warp_sums[warp] + incl - v;
}

// ---- 1. feature histogram --------------------------------------------------------------------
__global__ void __launch_bounds__(1024)
k_feat_hist(const int32_t* __restrict__ indptr, const int32_t* __restrict__ indices, int64_t n, int V,
            int use_smem, uint32_t* __restrict__ feat_count, int* __restrict__ flags)
{
    // a feature id outside [0, V) is skipped here and in the later plan kernels, and noted in the
    // handle's flag word (the search itself keeps sorted, distinct, in-range ids as a precondition)
    bool bad = false;
    extern __shared__ uint32_t sh_hist[];
    const int64_t beg = indptr[0], end = indptr[n];
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    if (use_smem) {
        for (int v = threadIdx.x; v < V; v += blockDim.x) sh_hist[v] = 0;
        __syncthreads();
        for (int64_t p = beg + (int64_t)blockIdx.x * blockDim.x + threadIdx.x; p < end; p += stride) {
            const int v = indices[p];
            if ((unsigned)v < (unsigned)V) atomicAdd(&sh_hist[v], 1u);
            else bad = true;
        }
        __syncthreads();
        for (int v = threadIdx.x; v < V; v += blockDim.x) {
            const uint32_t c = sh_hist[v];
            if (c) atomicAdd(&feat_count[v], c);
        }
    } else {
        for (int64_t p = beg + (int64_t)blockIdx.x * blockDim.x + threadIdx.x; p < end; p += stride) {
            const int v = indices[p];
            if ((unsigned)v < (unsigned)V) atomicAdd(&feat_count[v], 1u);
            else bad = true;
        }
    }
    if (bad) atomicOr(flags, SOM_FLAG_BAD_INDEX);
}

// Adds 1 to bins[bin] with one atomic per distinct bin in the warp; returns this thread's
// rank inside the bin's increment (0-based) plus the old value.
__device__ __forceinline__ uint32_t warp_agg_inc(uint32_t* bins, uint32_t bin, bool active)
{
    const unsigned act = __ballot_sync(0xffffffffu, active);
    uint32_t res = 0;
    if (active) {
        const unsigned peers = __match_any_sync(act, bin);
        const int lane = threadIdx.x & 31;
        const int leader = __ffs(peers) - 1;
        uint32_t old = 0;
        if (lane == leader) old = atomicAdd(&bins[bin], (uint32_t)__popc(peers));
        old = __shfl_sync(peers, old, leader);
        res = old + (uint32_t)__popc(peers & ((1u << lane) - 1u));
    }
    return res;
}

// ---- 2. hot-set selection --------------------------------------------------------------------
// K-th largest count by a 4-pass radix select.  thr = that count, n_greater = how many counts
// are strictly larger.  All threads of the 1024-thread block call it.
__device__ void kth_largest(const uint32_t* __restrict__ c, int V, int K, uint32_t* sh_hist,
                            uint32_t* sh_state, int* scan_ws, uint32_t* thr, int* n_greater)
{
    if (threadIdx.x == 0) { sh_state[0] = 0; sh_state[1] = (uint32_t)K; sh_state[2] = 0; }
    __syncthreads();
    for (int shift = 24; shift >= 0; shift -= 8) {
        if (threadIdx.x < 256) sh_hist[threadIdx.x] = 0;
        __syncthreads();
        const uint32_t prefix = sh_state[0];
        const uint32_t hi_mask = (shift == 24) ? 0u : (0xffffffffu << (shift + 8));
        // (nearly all counts share their high bytes: one atomic per distinct digit and warp)
        for (int v0 = 0; v0 < V; v0 += blockDim.x) {
            const int v = v0 + threadIdx.x;
            const uint32_t x = v < V ? c[v] : 0u;
            warp_agg_inc(sh_hist, (x >> shift) & 255u, v < V && (x & hi_mask) == prefix);
        }
        __syncthreads();
        // the digit d whose bin holds the K-th largest: the counts above it (an exclusive scan
        // over the digits in descending order) stay below `need`, with bin d they reach it;
        // digit 0 when even all bins together do not (fewer counts than K)
        {
            const uint32_t need = sh_state[1];
            const int d = 255 - (int)threadIdx.x;
            const uint32_t mine = d >= 0 ? sh_hist[d] : 0u;
            int total;
            const uint32_t above = (uint32_t)block_excl_scan_1024((int)mine, scan_ws, &total);
            if (d >= 0 && ((above < need && need <= above + mine) || (d == 0 && above + mine < need))) {
                sh_state[2] += above;
                sh_state[1] = need - above;
                sh_state[0] = prefix | ((uint32_t)d << shift);
            }
        }
        __syncthreads();
    }
    *thr = sh_state[0];
    *n_greater = (int)sh_state[2];
    __syncthreads();
}

__global__ void __launch_bounds__(1024)
k_select_hot(const uint32_t* __restrict__ feat_count_g, int V, int n_mask, int n_hot, int use_smem,
             int32_t* __restrict__ feat_slot, int32_t* __restrict__ slot_feat, int32_t* __restrict__ n_slots,
             const int32_t* __restrict__ indptr, int64_t n, int cover_pct)
{
    // the counts are walked thirteen times: keep them in shared memory when they fit
    extern __shared__ uint32_t sh_counts[];
    const uint32_t* feat_count = feat_count_g;
    if (use_smem) {
        for (int v = threadIdx.x; v < V; v += blockDim.x) sh_counts[v] = feat_count_g[v];
        feat_count = sh_counts;
        __syncthreads();
    }
    __shared__ uint32_t sh_hist[256];
    __shared__ uint32_t sh_state[4];
    __shared__ int warp_sums[32];
    __shared__ int sh_total;
    uint32_t thr_m, thr_a;
    int gr_m, gr_a;
    kth_largest(feat_count, V, n_mask, sh_hist, sh_state, warp_sums, &thr_m, &gr_m);
    kth_largest(feat_count, V, n_mask + n_hot, sh_hist, sh_state, warp_sums, &thr_a, &gr_a);
    const int need_m = n_mask - gr_m;            // ties at thr_m to take (lowest ids first)
    const int need_a = n_mask + n_hot - gr_a;    // ties at thr_a to take
    // Every thread owns a contiguous range of feature ids, so ranks in id order are "offset of my
    // range (one block scan) + position inside it".  Pass 1 ranks the ties at the two thresholds
    // (the lowest ids are taken), pass 2 decides mask / hot and counts them, pass 3 writes the
    // slots: four block scans in all, whatever V is.
    const int per = (V + 1023) / 1024;
    const int v_lo = min(V, (int)threadIdx.x * per), v_hi = min(V, v_lo + per);
    int my_em = 0, my_ea = 0;
    for (int v = v_lo; v < v_hi; ++v) {
        const uint32_t c = feat_count[v];
        my_em += (c == thr_m && c > 0);
        my_ea += (c == thr_a && c > 0);
    }
    const int off_em = block_excl_scan_1024(my_em, warp_sums, &sh_total);
    const int off_ea = block_excl_scan_1024(my_ea, warp_sums, &sh_total);
    int my_mask = 0, my_hot = 0, seen_m = off_em, seen_a = off_ea;
    for (int v = v_lo; v < v_hi; ++v) {
        const uint32_t c = feat_count[v];
        const bool e_m = c == thr_m && c > 0, e_a = c == thr_a && c > 0;
        const bool is_mask = c > thr_m || (e_m && seen_m < need_m);
        const bool is_sel = c > thr_a || (e_a && seen_a < need_a);
        seen_m += e_m;
        seen_a += e_a;
        my_mask += is_mask;
        my_hot += is_sel && !is_mask;
    }
    int slot_m = block_excl_scan_1024(my_mask, warp_sums, &sh_total);
    const int mask_assigned = sh_total;
    int slot_h = block_excl_scan_1024(my_hot, warp_sums, &sh_total);
    const int hot_assigned = sh_total;
    seen_m = off_em;
    seen_a = off_ea;
    int covered = 0;
    for (int v = v_lo; v < v_hi; ++v) {
        const uint32_t c = feat_count[v];
        const bool e_m = c == thr_m && c > 0, e_a = c == thr_a && c > 0;
        const bool is_mask = c > thr_m || (e_m && seen_m < need_m);
        const bool is_sel = c > thr_a || (e_a && seen_a < need_a);
        seen_m += e_m;
        seen_a += e_a;
        int slot = -1;
        if (is_mask) slot = slot_m++;
        else if (is_sel) slot = n_mask + slot_h++;
        feat_slot[v] = slot;
        if (slot >= 0) {
            slot_feat[slot] = v;
            covered += (int)c;  // instances the table will serve
        }
    }
    if (covered) atomicAdd(&n_slots[SOM_PLAN_COVERED], covered);
    // unused slots (fewer distinct features than slots) point at no feature
    for (int s = threadIdx.x; s < n_mask + n_hot; s += blockDim.x) {
        const bool used = (s < n_mask) ? (s < mask_assigned) : (s - n_mask < hot_assigned);
        if (!used) slot_feat[s] = -1;
    }
    // The kernel choice of the automatic mode, made here so that the host never waits for it: the row
    // table pays when its features serve at least cover_pct percent of the batch's feature instances.
    __syncthreads();  // every thread's share of the covered count has been added
    if (threadIdx.x == 0) {
        n_slots[0] = mask_assigned;
        n_slots[1] = hot_assigned;
        const int64_t nnz = (int64_t)indptr[n] - (int64_t)indptr[0];
        const int64_t cov = *reinterpret_cast<volatile int32_t*>(&n_slots[SOM_PLAN_COVERED]);
        n_slots[SOM_PLAN_USE_TABLE] = (cov * 100 >= (int64_t)cover_pct * nnz) ? 1 : 0;
    }
}

// ---- 3. classify ----------------------------------------------------------------------------
// Samples are grouped by mask, then by hot count, then by tail count, so that the four samples
// of a search round share the register-resident prefix and the trip counts of both row loops.
__device__ __forceinline__ uint32_t sort_bin(uint32_t mask, uint32_t n_hot, uint32_t n_tail)
{
    const uint32_t ch = n_hot > 15u ? 15u : n_hot;
    const uint32_t ct = n_tail > 7u ? 7u : n_tail;
    return (mask << SOM_PLAN_LEN_BITS) | (ch << 3) | ct;
}

__global__ void __launch_bounds__(PLAN_THREADS)
k_classify(const int32_t* __restrict__ indptr, const int32_t* __restrict__ indices, int64_t n, int V,
           const int32_t* __restrict__ feat_slot, int n_mask, uint32_t* __restrict__ pk,
           uint32_t* __restrict__ ntail, uint32_t* __restrict__ bin_count, const int* __restrict__ gate,
           int gate_want)
{
    if (som_gated_off(gate, gate_want)) return;
    const int64_t s = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const bool active = s < n;
    uint32_t mask = 0, nh = 0, nt = 0;
    if (active) {
        const int beg = indptr[s], end = indptr[s + 1];
        for (int j = beg; j < end; ++j) {
            const int v = indices[j];
            if ((unsigned)v >= (unsigned)V) continue;  // skipped (k_feat_hist has noted it)
            const int slot = feat_slot[v];
            if (slot < 0) ++nt;
            else if (slot < n_mask) mask |= 1u << slot;
            else ++nh;
        }
        // hot features beyond a slot's twelve go with the tail features (their rows are then read from the
        // codebook like any tail row) as long as those have room: far fewer samples are left to the list
        if (nh > (uint32_t)SOM_SLOT_MAX_HOT && nt + (nh - SOM_SLOT_MAX_HOT) <= (uint32_t)SOM_SLOT_MAX_TAIL) {
            nt += nh - SOM_SLOT_MAX_HOT;
            nh = SOM_SLOT_MAX_HOT;
        }
        pk[s] = mask | (nh << 16);
        ntail[s] = nt;
    }
    warp_agg_inc(bin_count, sort_bin(mask, nh, nt), active);
}

// ---- 4. exclusive scan of the sort bins (three kernels) ----------------------------------------
constexpr int SCAN_ITEMS = 4;
constexpr int SCAN_BLOCK = 1024 * SCAN_ITEMS;

__global__ void __launch_bounds__(1024)
k_scan_reduce(const uint32_t* __restrict__ in, int n, uint32_t* __restrict__ block_sums)
{
    __shared__ int warp_sums[32];
    __shared__ int sh_total;
    const int base = blockIdx.x * SCAN_BLOCK + threadIdx.x * SCAN_ITEMS;
    int sum = 0;
    if (base + SCAN_ITEMS <= n) {
        const uint4 v = *reinterpret_cast<const uint4*>(in + base);
        sum = (int)(v.x + v.y + v.z + v.w);
    } else {
        for (int u = 0; u < SCAN_ITEMS; ++u)
            if (base + u < n) sum += (int)in[base + u];
    }
    block_excl_scan_1024(sum, warp_sums, &sh_total);
    if (threadIdx.x == 0) block_sums[blockIdx.x] = (uint32_t)sh_total;
}

__global__ void __launch_bounds__(1024)
k_scan_block_sums(uint32_t* __restrict__ block_sums, int n_blocks)
{
    __shared__ int warp_sums[32];
    __shared__ int sh_total;
    int carry = 0;
    for (int b0 = 0; b0 < n_blocks; b0 += 1024) {
        const int b = b0 + threadIdx.x;
        const int v = (b < n_blocks) ? (int)block_sums[b] : 0;
        const int ex = block_excl_scan_1024(v, warp_sums, &sh_total);
        if (b < n_blocks) block_sums[b] = (uint32_t)(carry + ex);
        carry += sh_total;
        __syncthreads();
    }
}

__global__ void __launch_bounds__(1024)
k_scan_apply(const uint32_t* __restrict__ in, int n, const uint32_t* __restrict__ block_sums,
             uint32_t* __restrict__ out)
{
    __shared__ int warp_sums[32];
    __shared__ int sh_total;
    const int base = blockIdx.x * SCAN_BLOCK + threadIdx.x * SCAN_ITEMS;
    int v[SCAN_ITEMS];
    int sum = 0;
#pragma unroll
    for (int u = 0; u < SCAN_ITEMS; ++u) {
        v[u] = (base + u < n) ? (int)in[base + u] : 0;
        sum += v[u];
    }
    int run = block_excl_scan_1024(sum, warp_sums, &sh_total) + (int)block_sums[blockIdx.x];
#pragma unroll
    for (int u = 0; u < SCAN_ITEMS; ++u) {
        if (base + u < n) out[base + u] = (uint32_t)run;
        run += v[u];
    }
}

// ---- 5. scatter + slots ----------------------------------------------------------------------
__global__ void __launch_bounds__(PLAN_THREADS)
k_scatter_slots(const int32_t* __restrict__ indptr, const int32_t* __restrict__ indices, int64_t n, int V,
                const int32_t* __restrict__ feat_slot, int n_mask, int zero_row,
                const uint32_t* __restrict__ pk, const uint32_t* __restrict__ ntail,
                uint32_t* __restrict__ bin_cursor /* starts as bin_start */,
                uint32_t* __restrict__ slots, uint32_t* __restrict__ order, int32_t* __restrict__ rare_list,
                int32_t* __restrict__ rare_count,
                const int* __restrict__ gate, int gate_want)
{
    if (som_gated_off(gate, gate_want)) return;
    const int64_t s = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const bool active = s < n;
    uint32_t mask = 0, nh = 0, nt = 0, p = 0;
    if (active) {
        p = pk[s];
        mask = p & 0xffffu;
        nh = p >> 16;
        nt = ntail[s];
    }
    const uint32_t pos = warp_agg_inc(bin_cursor, sort_bin(mask, nh, nt), active);
    if (!active) return;
    const bool fits = nh <= SOM_SLOT_MAX_HOT && nt <= SOM_SLOT_MAX_TAIL;
    // The slot is assembled in registers and written with three 128-bit stores.  Unused hot
    // codes point at the all-zero row that follows the table; unused tail codes are feature 0.
    const uint32_t zz = (uint32_t)zero_row | ((uint32_t)zero_row << 16);
    uint32_t w[SOM_SLOT_WORDS];
    w[0] = fits ? (mask | (nh << 16) | (nt << 24)) : (mask | (SOM_SLOT_NT_OVERFLOW << 24));  // (zero hot codes)
    w[1] = 0u;  // tail codes 8..9
#pragma unroll
    for (int i = 2; i < 8; ++i) w[i] = zz;
#pragma unroll
    for (int i = 8; i < 12; ++i) w[i] = 0u;
    const int beg = indptr[s], end = indptr[s + 1];
    if (fits) {
        uint32_t ih = 0, it = 0;
        for (int j = beg; j < end; ++j) {
            const int v = indices[j];
            if ((unsigned)v >= (unsigned)V) continue;
            const int fs = feat_slot[v];
            if (fs < 0 || (fs >= n_mask && ih >= (uint32_t)SOM_SLOT_MAX_HOT)) {  // tail feature, or a hot one too many
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if ((it >> 1) == (uint32_t)i)
                        w[8 + i] = (it & 1u) ? (w[8 + i] | ((uint32_t)v << 16)) : (uint32_t)v;
                if (it == 8u) w[1] = (uint32_t)v;
                if (it == 9u) w[1] |= (uint32_t)v << 16;
                ++it;
            } else if (fs >= n_mask) {
#pragma unroll
                for (int i = 0; i < 6; ++i)
                    if ((ih >> 1) == (uint32_t)i)
                        w[2 + i] = (ih & 1u) ? ((w[2 + i] & 0xffffu) | ((uint32_t)fs << 16))
                                             : ((w[2 + i] & 0xffff0000u) | (uint32_t)fs);
                ++ih;
            }
        }
    } else {
        // a sample that does not fit a slot goes on the list that the direct-load kernel searches
        rare_list[atomicAdd(rare_count, 1)] = (int32_t)s;
    }
    order[pos] = (uint32_t)s;
    uint4* slot = reinterpret_cast<uint4*>(slots + (size_t)pos * SOM_SLOT_WORDS);
    slot[0] = make_uint4(w[0], w[1], w[2], w[3]);
    slot[1] = make_uint4(w[4], w[5], w[6], w[7]);
    slot[2] = make_uint4(w[8], w[9], w[10], w[11]);
}

// The slot array is padded to whole rounds with copies of the last slot.
__global__ void k_pad_slots(uint4* __restrict__ slots, int64_t n, int64_t n_pad)
{
    const int64_t extra = (n_pad - n) * (SOM_SLOT_WORDS / 4);
    if (threadIdx.x < extra) {
        const int64_t dst = n * (SOM_SLOT_WORDS / 4) + threadIdx.x;
        slots[dst] = slots[(n - 1) * (SOM_SLOT_WORDS / 4) + threadIdx.x % (SOM_SLOT_WORDS / 4)];
    }
}

}  // namespace

size_t som_plan_head_bytes(int32_t V, int n_slots_max, SomPlanBuffers* b)
{
    size_t off = 0;
    auto take = [&](size_t bytes) {
        const size_t o = off;
        off = som_align_up(off + bytes, 256);
        return o;
    };
    b->feat_count = take((size_t)V * 4);
    b->feat_slot = take((size_t)V * 4);
    b->slot_feat = take((size_t)n_slots_max * 4);
    b->n_slots = take(SOM_PLAN_N_SLOTS_INTS * 4);
    return off;
}

size_t som_plan_workspace_bytes(int64_t n, SomPlanBuffers* b)
{
    size_t off = 0;
    auto take = [&](size_t bytes) {
        const size_t o = off;
        off = som_align_up(off + bytes, 256);
        return o;
    };
    b->keys = take((size_t)(n + 16) * 8);
    b->keys2 = take((size_t)(n + 16) * 8);
    b->keys3 = take((size_t)(n + 16) * 8);
    b->pk = take((size_t)n * 4);
    b->ntail = take((size_t)n * 4);
    b->bin_count = take((size_t)SOM_PLAN_BINS * 4);
    b->bin_start = take((size_t)SOM_PLAN_BINS * 4);
    b->block_sums = take((size_t)(SOM_PLAN_BINS / SCAN_BLOCK + 2) * 4);
    b->slots = take((size_t)(n + 16) * SOM_SLOT_WORDS * 4);
    b->order = take((size_t)(n + 16) * 4);
    b->uncertain = take((size_t)n * 4);
    b->ukeys = take((size_t)(n + 16) * 8);
    b->ukeys2 = take((size_t)(n + 16) * 8);
    b->slots2 = take((size_t)(n + 16) * SOM_SLOT_WORDS * 4);
    b->rare_list = take((size_t)n * 4);
    b->rare_keys = take((size_t)(n + 16) * 8);
    b->rare_keys2 = take((size_t)(n + 16) * 8);
    return off;
}

int som_launch_pad_slots(som_handle* h, char* ws, size_t slots_offset, int64_t n, cudaStream_t st)
{
    const int64_t n_pad = (n + 3) / 4 * 4;
    if (n_pad > n && n > 0) {
        k_pad_slots<<<1, 32, 0, st>>>(reinterpret_cast<uint4*>(ws + slots_offset), n, n_pad);
        SOM_CK(h, cudaGetLastError());
        h->launches += 1;
    }
    return SOM_OK;
}

// How many of the table's first SOM_PLAN_MASK_FEATURES rows are handled as mask bits (the others are
// ordinary hot rows).  A mask feature costs a sample nothing while its mask equals that of the sample its
// team handled before (four positions earlier in the sorted list), and a rebuild of the whole prefix,
// which stalls the other three teams of the warp, when it does not.  The sorted list has one run per
// distinct mask, so the smaller the batch, the shorter the runs and the fewer bits pay.  Measured on the
// MeSH-shaped batches, whole call, fp32: 250k samples on the 1024 x 1024 map 430 ms with 16 bits, 379 with 9
// (the optimum: 387 with 7, 386 with 11); 1M samples on 512 x 512: 359 / 337 (10 or 11 bits); 4M samples
// on 128 x 128: 82.0 / 80.4 (12 or 13 bits).  fp16 storage moves the same way (269 -> 226 ms at 9 bits).
static void plan_split(const som_handle* h, int64_t n, int* n_mask, int* n_hot)
{
    int bits = (int)h->opt_mask_bits;
    if (bits == 0) {
        int lg = 0;
        while (lg < 40 && ((int64_t)1 << (lg + 1)) <= n) ++lg;  // floor(log2 n)
        bits = lg - 8;                                            // 250k -> 9, 1M -> 11, 4M -> 13
        // Where the search prunes (som_table_prunes; not the first pass of the two-stage search) few samples reach
        // the search rounds of a range, the more ranges the fewer, and the shared prefixes serve less: fewer mask
        // features measure faster, by floor((floor(log2 ranges) - 3) / 2), at most 4.  Search phase, fp32: 1M
        // samples on 64 x 64 3.62 -> 3.56 ms (10 bits), 4M on 128 x 128 43.8 -> 42.4 (11), 1M on 512 x 512
        // 96.3 -> 87.8 (7; 88.8 with 4, 92.3 with 10), 250k on 1024 x 1024 107.6 -> 98.3 (5; 100.1 with 3 or 7).
        if (som_table_prunes(h) && h->opt_two_stage != 1) {
            int lr = 0;
            const int64_t ranges = (h->M + 127) / 128;
            while (lr < 40 && ((int64_t)1 << (lr + 1)) <= ranges) ++lr;  // floor(log2 ranges)
            int less = (lr - 3) / 2;
            bits -= less < 0 ? 0 : (less > 4 ? 4 : less);
        }
        if (bits < 4) bits = 4;
    }
    if (bits > *n_mask) bits = *n_mask;
    *n_hot += *n_mask - bits;
    *n_mask = bits;
}

int som_launch_plan_select(som_handle* h, const int32_t* indptr, const int32_t* indices, int64_t n,
                           char* head, const SomPlanBuffers& b, int n_mask, int n_hot, cudaStream_t st)
{
    uint32_t* feat_count = reinterpret_cast<uint32_t*>(head + b.feat_count);
    int32_t* feat_slot = reinterpret_cast<int32_t*>(head + b.feat_slot);
    int32_t* slot_feat = reinterpret_cast<int32_t*>(head + b.slot_feat);
    int32_t* n_slots = reinterpret_cast<int32_t*>(head + b.n_slots);
    plan_split(h, n, &n_mask, &n_hot);

    SOM_CK(h, cudaMemsetAsync(feat_count, 0, (size_t)h->V * 4, st));
    SOM_CK(h, cudaMemsetAsync(n_slots, 0, SOM_PLAN_N_SLOTS_INTS * 4, st));

    // 1. histogram
    {
        const size_t sh = (size_t)h->V * 4;
        const int use_smem = sh <= (size_t)160 * 1024;
        int blocks = h->sm_count;
        if (use_smem) {
            if (!h->plan_attr_set) {
                SOM_CK(h, cudaFuncSetAttribute(k_feat_hist, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024));
                h->plan_attr_set = 1;
            }
        } else {
            blocks = h->sm_count * 2;
        }
        k_feat_hist<<<blocks, 1024, use_smem ? sh : 0, st>>>(indptr, indices, n, h->V, use_smem, feat_count, h->dev_flags);
        SOM_CK(h, cudaGetLastError());
    }
    // 2. select
    const size_t counts_sh = (size_t)h->V * 4;
    const int counts_fit = counts_sh <= 200 * 1024;
    if (counts_fit)
        SOM_CK(h, cudaFuncSetAttribute(k_select_hot, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)counts_sh));
    k_select_hot<<<1, 1024, counts_fit ? counts_sh : 0, st>>>(feat_count, h->V, n_mask, n_hot, counts_fit, feat_slot,
                                                             slot_feat, n_slots, indptr, n,
                                                             (int)(h->opt_cover > 0 ? h->opt_cover : (h->opt_cover < 0 ? 0 : 60)));
    SOM_CK(h, cudaGetLastError());
    h->launches += 2;
    return SOM_OK;
}

int som_launch_plan_sort(som_handle* h, const int32_t* indptr, const int32_t* indices, int64_t n,
                         char* head, char* ws, const SomPlanBuffers& b, int n_mask, int n_hot,
                         cudaStream_t st)
{
    int32_t* feat_slot = reinterpret_cast<int32_t*>(head + b.feat_slot);
    uint32_t* pk = reinterpret_cast<uint32_t*>(ws + b.pk);
    uint32_t* ntail = reinterpret_cast<uint32_t*>(ws + b.ntail);
    uint32_t* bin_count = reinterpret_cast<uint32_t*>(ws + b.bin_count);
    uint32_t* bin_start = reinterpret_cast<uint32_t*>(ws + b.bin_start);
    uint32_t* slots = reinterpret_cast<uint32_t*>(ws + b.slots);
    plan_split(h, n, &n_mask, &n_hot);

    SOM_CK(h, cudaMemsetAsync(bin_count, 0, (size_t)SOM_PLAN_BINS * 4, st));
    // 3. classify
    const unsigned sblocks = (unsigned)((n + PLAN_THREADS - 1) / PLAN_THREADS);
    k_classify<<<sblocks, PLAN_THREADS, 0, st>>>(indptr, indices, n, h->V, feat_slot, n_mask, pk, ntail, bin_count,
                                                 h->gate, h->gate_want);
    SOM_CK(h, cudaGetLastError());
    // 4. scan bins
    {
        uint32_t* block_sums = reinterpret_cast<uint32_t*>(ws + b.block_sums);
        const int scan_blocks = (SOM_PLAN_BINS + SCAN_BLOCK - 1) / SCAN_BLOCK;
        k_scan_reduce<<<scan_blocks, 1024, 0, st>>>(bin_count, SOM_PLAN_BINS, block_sums);
        SOM_CK(h, cudaGetLastError());
        k_scan_block_sums<<<1, 1024, 0, st>>>(block_sums, scan_blocks);
        SOM_CK(h, cudaGetLastError());
        k_scan_apply<<<scan_blocks, 1024, 0, st>>>(bin_count, SOM_PLAN_BINS, block_sums, bin_start);
        SOM_CK(h, cudaGetLastError());
    }
    // 5. scatter + slots (bin_start doubles as the running cursor)
    k_scatter_slots<<<sblocks, PLAN_THREADS, 0, st>>>(indptr, indices, n, h->V, feat_slot, n_mask, n_mask + n_hot, pk, ntail,
                                                      bin_start, slots, reinterpret_cast<uint32_t*>(ws + b.order),
                                                      reinterpret_cast<int32_t*>(ws + b.rare_list),
                                                      reinterpret_cast<int32_t*>(head + b.n_slots) + SOM_PLAN_RARE,
                                                      h->gate, h->gate_want);
    SOM_CK(h, cudaGetLastError());
    const int64_t n_pad = (n + 3) / 4 * 4;
    if (n_pad > n) {
        k_pad_slots<<<1, 32, 0, st>>>(reinterpret_cast<uint4*>(slots), n, n_pad);
        SOM_CK(h, cudaGetLastError());
        h->launches += 1;
    }
    h->launches += 5;
    return SOM_OK;
}
