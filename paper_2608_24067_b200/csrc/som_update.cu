// Batch update of the codebook (Section 3.4 of the paper; Algorithm 2, steps 8-9): scatter the
// batch onto the lattice (per cell the sum of the assigned binary samples, num, and their count,
// den), blur both fields with three unnormalised box passes per lattice axis whose window is
// truncated at the edge, and replace every prototype by num / den where den > 0.
//
// Layout and order of work.  The codebook is feature-major, so the field of one feature (a
// "plane": rows x cols cells, neuron i at row i / cols, column i % cols) is contiguous, and the
// planes are independent.  They are processed in slabs of as many planes as fit a bounded
// workspace (two buffers), so the update needs no second V x M array beside the codebook:
//   1. scatter the slab's features into buffer A in TRANSPOSED cell order (col-major), so that
//   2. three box passes along the slow index, one thread per (plane, fast index) walking a line
//      with coalesced loads and a running window sum (add the entering element, subtract the
//      leaving one: O(1) per cell whatever the radius), are the passes along the lattice rows;
//   3. a tiled transpose back to neuron order;
//   4. three more such passes, now along the lattice columns, the last one fused with the
//      division and the write of the new weights (fp32 or fp16 storage; rounding happens only at
//      this final write).
// Box passes along different axes commute, so three per axis in this order equal the paper's
// (row, column) x 3.  The running sums are carried in fp64 (the paper carries fp32); the fields
// between passes are fp32.  Whether a neuron's blurred denominator is zero is decided exactly,
// from an integer box count of the occupied cells over the reach of three passes (3 * radius):
// a running sum that subtracts can leave a rounding residue where the exact sum is zero.
// Lattices of up to 128 x 128 cells replace steps 2-4 by one kernel that blurs a plane in shared
// memory (k_upd_blur_fused): one read and one write of the plane instead of seven.  Larger lattices
// scatter in neuron order and take two strip kernels through shared memory (k_upd_strip), as long as
// a strip of eight lines fits there; only shapes beyond that walk steps 1-4 through device memory.
#include "som_internal.cuh"

namespace {

constexpr int UPD_THREADS = 256;

// Count of samples per cell into den_t (TRANSPOSED cell order) and the occupancy flags.  Small
// lattices take a per-block histogram in shared memory first (a million samples on a few
// thousand cells would otherwise queue on a handful of L2 atomic units); counts are exact in fp32.
// A best-unit index outside [0, M) (a stale buffer, the -1 of a missing second unit) is skipped and
// noted in the handle's flag word, here and in the scatters below.
__global__ void k_upd_count(const int32_t* __restrict__ bmu, int64_t n, int rows, int cols, int use_smem,
                            float* __restrict__ den_t, int32_t* __restrict__ occ, int* __restrict__ flags)
{
    extern __shared__ unsigned int hist[];
    const int M = rows * cols;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    if (use_smem) {
        for (int c = threadIdx.x; c < M; c += blockDim.x) hist[c] = 0u;
        __syncthreads();
        bool bad = false;
        for (int64_t s = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; s < n; s += stride) {
            const int c = bmu[s];
            if ((unsigned)c < (unsigned)M) atomicAdd(&hist[c], 1u);
            else bad = true;
        }
        if (bad) atomicOr(flags, SOM_FLAG_BAD_UNIT);
        __syncthreads();
        for (int c = threadIdx.x; c < M; c += blockDim.x) {
            const unsigned int k = hist[c];
            if (k) {
                const int r = c / cols, q = c - r * cols;
                atomicAdd(&den_t[(int64_t)q * rows + r], (float)k);
                occ[c] = 1;
            }
        }
    } else {
        for (int64_t s = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; s < n; s += stride) {
            const int c = bmu[s];
            if ((unsigned)c >= (unsigned)M) {
                atomicOr(flags, SOM_FLAG_BAD_UNIT);
                continue;
            }
            const int r = c / cols, q = c - r * cols;
            atomicAdd(&den_t[(int64_t)q * rows + r], 1.0f);
            occ[c] = 1;
        }
    }
}

// one thread per sample: its features inside [v0, v1) add 1 to the cell of its best unit
__global__ void k_upd_scatter(const int32_t* __restrict__ indptr, const int32_t* __restrict__ indices,
                              int64_t n, const int32_t* __restrict__ bmu, int v0, int v1, int rows, int cols,
                              const int32_t* __restrict__ hot_slot, float* __restrict__ num_t, int natural_order)
{
    const int64_t s = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= n) return;
    const int c = bmu[s];
    const int64_t M = (int64_t)rows * cols;
    if ((unsigned)c >= (unsigned)M) return;  // skipped; k_upd_count has noted it
    const int r = c / cols, q = c - r * cols;
    // transposed cell order for the routes that blur along the lattice rows first with walks along the
    // slow index; neuron order for the strip route
    const int64_t cell_t = natural_order ? (int64_t)c : (int64_t)q * rows + r;
    const int beg = indptr[s], end = indptr[s + 1];
    for (int j = beg; j < end; ++j) {
        const int v = indices[j];
        if (v >= v1) break;  // ids ascend inside a row
        if (v >= v0 && !(hot_slot && hot_slot[v] >= 0)) atomicAdd(&num_t[(int64_t)(v - v0) * M + cell_t], 1.0f);
    }
}

// The planes of the most frequent features take most of the batch's increments (a feature that
// 84 % of a million samples carry puts 200 atomic adds on every cell of one 4096-cell plane, and
// same-address atomics queue in L2).  k_upd_hot_mask notes per sample which of the (at most 16) hot
// features it has; block (slice, group) of k_upd_scatter_hot then counts the increments of its group
// of hot features over its slice of the samples in shared memory, reading only mask and best unit of
// a sample, and adds each non-zero count to the plane once.  hot_slot[v] = rank of feature v among the
// hot ones or -1; slot_feat is its inverse.
__global__ void k_upd_hot_mask(const int32_t* __restrict__ indptr, const int32_t* __restrict__ indices, int64_t n,
                               int V, const int32_t* __restrict__ hot_slot, uint32_t* __restrict__ mask,
                               int* __restrict__ flags)
{
    const int64_t s = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= n) return;
    uint32_t m = 0;
    const int beg = indptr[s], end = indptr[s + 1];
    for (int j = beg; j < end; ++j) {
        const int v = indices[j];
        if ((unsigned)v >= (unsigned)V) {  // skipped and noted
            atomicOr(flags, SOM_FLAG_BAD_INDEX);
            continue;
        }
        const int slot = hot_slot[v];
        if (slot >= 0) m |= 1u << slot;
    }
    mask[s] = m;
}

__global__ void k_upd_scatter_hot(const uint32_t* __restrict__ mask, int64_t n, const int32_t* __restrict__ bmu,
                                  int v0, int v1, int rows, int cols, const int32_t* __restrict__ slot_feat,
                                  int n_slots, int planes_per_block, float* __restrict__ num_t, int natural_order)
{
    extern __shared__ unsigned int cnt[];
    const int M = rows * cols;
    const int slot0 = blockIdx.y * planes_per_block;
    for (int e = threadIdx.x; e < planes_per_block * M; e += blockDim.x) cnt[e] = 0u;
    // the group's slots whose feature lies in this slab
    uint32_t group = 0;
    for (int p = 0; p < planes_per_block && slot0 + p < n_slots; ++p) {
        const int f = slot_feat[slot0 + p];
        if (f >= v0 && f < v1) group |= 1u << (slot0 + p);
    }
    __syncthreads();
    const int64_t per = (n + gridDim.x - 1) / gridDim.x;
    const int64_t s_lo = (int64_t)blockIdx.x * per, s_hi = min(n, s_lo + per);
    if (group) {
        for (int64_t s = s_lo + threadIdx.x; s < s_hi; s += blockDim.x) {
            uint32_t m = mask[s] & group;
            if (!m) continue;
            const int c = bmu[s];
            if ((unsigned)c >= (unsigned)M) continue;  // skipped; k_upd_count has noted it
            const int r = c / cols, q = c - r * cols;
            const int cell_t = natural_order ? c : q * rows + r;  // (transposed cell order unless the strip route follows)
            while (m) {
                const int slot = __ffs(m) - 1;
                m &= m - 1;
                atomicAdd(&cnt[(slot - slot0) * M + cell_t], 1u);
            }
        }
    }
    __syncthreads();
    for (int p = 0; p < planes_per_block && slot0 + p < n_slots; ++p) {
        if (!((group >> (slot0 + p)) & 1u)) continue;  // unused slot, or a feature of another slab
        float* plane = num_t + (int64_t)(slot_feat[slot0 + p] - v0) * M;
        for (int e = threadIdx.x; e < M; e += blockDim.x) {
            const unsigned int k = cnt[p * M + e];
            if (k) atomicAdd(&plane[e], (float)k);
        }
    }
}

// Box pass along the slow index of planes laid out [plane][len][width]: thread (plane, f) walks
// i = 0..len-1 at fixed fast index f.  out = sum of in over [i - radius, i + radius] clipped to
// the line.  T = float (fields) or int32 (the occupancy count).
template <typename T, typename ACC>
__global__ void k_box_pass(const T* __restrict__ in, T* __restrict__ out, int64_t planes, int len, int width,
                           int radius)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= planes * width) return;
    const int64_t p = t / width;
    const int f = (int)(t - p * width);
    const T* src = in + p * (int64_t)len * width + f;
    T* dst = out + p * (int64_t)len * width + f;
    ACC sum = 0;
    const int first = radius < len - 1 ? radius : len - 1;
    for (int j = 0; j <= first; ++j) sum += (ACC)src[(int64_t)j * width];
    dst[0] = (T)sum;
    for (int i = 1; i < len; ++i) {
        if (i + radius < len) sum += (ACC)src[(int64_t)(i + radius) * width];
        if (i - radius - 1 >= 0) sum -= (ACC)src[(int64_t)(i - radius - 1) * width];
        dst[(int64_t)i * width] = (T)sum;
    }
}

// The last pass, along the lattice columns of planes in neuron order, fused with the division
// (a multiplication by the reciprocal of the blurred denominator, both in fp64) and the write of
// the new weights of features v0 + plane.  A zero reciprocal marks a neuron out of every
// sample's reach: its prototype stays.
// 1 / blurred denominator in fp64 where the cell is within reach of a sample, else 0 (= keep)
__global__ void k_upd_reciprocal(const float* __restrict__ den_b, const int32_t* __restrict__ reach, int64_t M,
                                 double* __restrict__ rden)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < M) rden[i] = reach[i] > 0 ? 1.0 / (double)den_b[i] : 0.0;
}

template <typename ST>
__global__ void k_box_pass_divide(const float* __restrict__ in, int64_t planes, int rows, int cols, int radius,
                                  const double* __restrict__ rden, ST* __restrict__ W, int v0)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= planes * cols) return;
    const int64_t p = t / cols;
    const int f = (int)(t - p * cols);
    const int64_t M = (int64_t)rows * cols;
    const float* src = in + p * M + f;
    ST* dst = W + (int64_t)(v0 + p) * M + f;
    double sum = 0.0;
    const int first = radius < rows - 1 ? radius : rows - 1;
    for (int j = 0; j <= first; ++j) sum += (double)src[(int64_t)j * cols];
    for (int i = 0; i < rows; ++i) {
        if (i > 0) {
            if (i + radius < rows) sum += (double)src[(int64_t)(i + radius) * cols];
            if (i - radius - 1 >= 0) sum -= (double)src[(int64_t)(i - radius - 1) * cols];
        }
        const double rd = rden[(int64_t)i * cols + f];
        if (rd != 0.0) dst[(int64_t)i * cols] = (ST)(float)(sum * rd);
    }
}

// Small lattices: the whole blur of a plane in shared memory.  A block takes one plane at a time:
// it loads the scattered counts (transposed cell order) into an fp64 buffer, runs the three box
// passes along each axis between two fp64 buffers (counts and their window sums are integers, so
// fp64 holds them exactly up to 2^53 and the order of the passes does not matter), multiplies by
// the reciprocal denominator and writes the new weights: one read and one write of the plane
// instead of seven trips through DRAM.  A line is cut into `seg` segments, each walked by its own
// thread with a running window sum started from a plain sum over its first window, so that a
// 64 x 64 plane keeps 256 threads busy; the row pitch is odd (in doubles), which keeps the walks
// along either axis at the two shared-memory wavefronts a warp's 64-bit accesses need anyway.
constexpr int FUSED_THREADS = 256;
constexpr int FUSED_THREADS_WIDE = 1024;

constexpr int FUSED_PREFETCH = 16;  // cells per thread held in registers: planes of up to 4096 cells

// lines of `len` cells: cell j of line l at buf[l * line_stride + j * cell_stride]
// All threads of the block call it; n_lines * seg <= blockDim.x, so a thread has at most one
// segment.  With use_totals (worth it when the window is much longer than a segment; it costs
// one block synchronisation) a segment's first window sum is put together from the totals of the
// segments that lie wholly inside the window (each thread sums its own segment first; `tot` holds
// one double per thread) and the few cells at the window's two ends; else from the window's cells.
template <bool use_totals, typename BT>
__device__ __forceinline__ void box_lines(const BT* __restrict__ in, BT* __restrict__ out, int n_lines,
                                          int len, int line_stride, int cell_stride, int radius, int seg,
                                          double* __restrict__ tot)
{
    const int seg_len = (len + seg - 1) / seg;
    const int job = threadIdx.x;
    const bool busy = job < n_lines * seg;
    const int line = busy ? job % n_lines : 0;
    const int g = busy ? job / n_lines : 0;
    const int a = g * seg_len;
    const int b = min(len, a + seg_len);
    const BT* src = in + line * line_stride;
    if (busy && use_totals) {
        double t0 = 0.0, t1 = 0.0;
        const BT* p = src + a * cell_stride;
        int j = a;
        for (; j + 1 < b; j += 2, p += 2 * cell_stride) {
            t0 += (double)p[0];
            t1 += (double)p[cell_stride];
        }
        if (j < b) t0 += (double)p[0];
        tot[job] = t0 + t1;  // (an empty segment, a >= b, holds 0)
    }
    if (use_totals) __syncthreads();  // (the same for every thread of the block)
    if (!busy || a >= b) return;
    BT* dst = out + line * line_stride;
    const int lo = max(0, a - radius), hi = min(len - 1, a + radius);
    // segments g_lo .. g_hi lie wholly inside [lo, hi]
    const int g_lo = (lo + seg_len - 1) / seg_len;
    int g_hi = (hi + 1) / seg_len - 1;
    if (hi == len - 1) g_hi = (len - 1) / seg_len;  // the last segment may be short; it ends at len - 1
    double sum = 0.0;
    int left_end = hi + 1, right_begin = hi + 1;  // cells [lo, left_end) and [right_begin, hi] are added singly
    if (use_totals && g_lo <= g_hi) {
        for (int q = g_lo; q <= g_hi; ++q) sum += tot[line + n_lines * q];
        left_end = g_lo * seg_len;
        right_begin = min(len, (g_hi + 1) * seg_len);
    }
    for (int j = lo; j < left_end; ++j) sum += (double)src[j * cell_stride];
    for (int j = right_begin; j <= hi; ++j) sum += (double)src[j * cell_stride];
    BT* pd = dst + a * cell_stride;
    *pd = (BT)sum;
    pd += cell_stride;
    const BT* pe = src + (a + 1 + radius) * cell_stride;  // the cell entering the window
    const BT* pl = src + (a - radius) * cell_stride;      // the cell leaving it
    // i < len - radius: a cell enters; i > radius: a cell leaves
    for (int i = a + 1; i < b; ++i, pe += cell_stride, pl += cell_stride, pd += cell_stride) {
        const double enter = (i < len - radius) ? (double)*pe : 0.0;
        const double leave = (i > radius) ? (double)*pl : 0.0;
        sum += enter - leave;
        *pd = (BT)sum;
    }
}

// Lattices too large for one plane to be blurred on chip (more than 16384 cells) take the blur in two
// strip kernels through shared memory instead of seven trips through device memory.  A box pass
// along one lattice axis never mixes the lines of the other, so a block can take a strip of `tc`
// adjacent lines over their whole length, run the three passes of that axis between two fp32 tiles
// [line][cell] with fp64 running sums (the fields between passes are rounded to fp32, as on the
// device-memory route) and write once:
//   first launch  (ROWS = true):  a line is a lattice row, contiguous in memory; in and out in neuron order;
//   second launch (ROWS = false): a line is a lattice column (cell i of line f at i * width + f); the result
//                 is multiplied by the reciprocal blurred denominator and written as the new weights of
//                 features v0 + plane (a zero reciprocal keeps the prototype).
// A plane crosses device memory five times in all (scatter, in, out, in, weights out).
//
// One thread walks a segment of 16 cells: the window sum at the segment's first cell is put together from
// the totals of the segments that lie wholly inside the window (fp64, one per segment, kept in shared memory)
// and the few cells at the window's two ends; then every step adds the entering cell and subtracts the
// leaving one.  The totals of the next pass's input are summed on the way (the thread has just produced
// those 16 cells).  What counts is the instruction budget: the first version of this kernel spent 58
// instructions per cell and pass (generic strides, bounds tests and pointer updates per cell, a totals
// pass of its own, three fp32 <-> fp64 conversions per cell on the 16-lane conversion unit); here the walk of
// a segment whose window stays inside the line is fully unrolled with immediate offsets, the other
// segments clamp their indices into a zero cell instead of testing bounds, and the widening of the value
// just rounded goes through integer instructions instead of the conversion unit.
// Layout: the line pitch is 1 modulo 32 words and a warp holds 16 lines x 2 neighbouring segments (or 32 lines
// x 1), so every access of a walk touches 32 different banks.  Cells [len, pitch) of every line and the word
// before the first line stay zero: they are what out-of-range window ends read.
constexpr int STRIP_THREADS = 512;
constexpr int STRIP_SEG = 16;
constexpr int STRIP_MAX_ITERS = 4;  // segments of a strip per thread, at most

// A window sum rounded to the 24 significant bits of the fp32 field it is stored in, still as an fp64 value
// (Veltkamp's splitting with 2^29 + 1: one multiplication and two additions on the fp64 pipe, result the
// nearest 24-bit value).  The thread stores it (its conversion to fp32 is then exact) and adds the same
// value to the total of the next pass's input, so cells and totals agree bit for bit without widening the
// stored value again: the conversion unit (16 lanes per SM) sees three conversions per cell, not four, and
// an integer emulation of the widening cost seven instructions per cell.
__device__ __forceinline__ double strip_round24(double x)
{
    // (intrinsics: the compiler must not contract the product into the subtraction)
    const double gamma = __dmul_rn(x, 536870913.0);  // 2^29 + 1
    const double delta = __dsub_rn(x, gamma);
    return __dadd_rn(gamma, delta);
}

// The walk of one segment: y[k] = window sum at cell a + k for k = 1 .. 15, given the sum at cell a.
// ENTER / LEAVE say whether the segment's steps have an entering / a leaving cell at all (they have all or none
// on these paths; pe[k] enters and pl[k] leaves at step k); returns the fp64 total of the rounded outputs.
template <bool ENTER, bool LEAVE>
__device__ __forceinline__ double strip_walk(const float* __restrict__ pe, const float* __restrict__ pl,
                                             float* __restrict__ y, double sum, double t_next)
{
#pragma unroll
    for (int k = 1; k < STRIP_SEG; ++k) {
        if (ENTER && LEAVE) sum += (double)pe[k] - (double)pl[k];
        else if (ENTER) sum += (double)pe[k];
        else if (LEAVE) sum -= (double)pl[k];
        const double o = strip_round24(sum);
        y[k] = (float)o;
        t_next += o;
    }
    return t_next;
}

// in: plane-major; ROWS: cell i of line f at f * len + i, else at i * width + f.  The block's strip is lines
// f0 .. f0 + tc - 1 (tc a power of two).  Shared memory: the segment totals tot[tc][n_seg | 1] and their
// running sums cum[tc][(n_seg + 1) | 1] (fp64), then 1 + 2 * tc * pitch floats.
template <typename ST, bool ROWS>
__global__ void __launch_bounds__(STRIP_THREADS, 3)
k_upd_strip(const float* __restrict__ in, float* __restrict__ out, int64_t planes, int len, int width, int radius,
            int tc, int tc_shift, int pitch, const double* __restrict__ rden, ST* __restrict__ W, int v0)
{
    extern __shared__ __align__(16) unsigned char strip_raw[];
    const int n_seg = (len + STRIP_SEG - 1) / STRIP_SEG;
    const int len_pad = n_seg * STRIP_SEG;
    const int n_jobs = n_seg << tc_shift;
    const int tot_pitch = n_seg | 1, cum_pitch = (n_seg + 1) | 1;  // odd: 16 lines at one segment, 32 banks
    double* tot = reinterpret_cast<double*>(strip_raw);
    double* cum = tot + tc * tot_pitch;
    float* A = reinterpret_cast<float*>(cum + tc * cum_pitch) + 1;
    float* B = A + (size_t)tc * pitch;
    for (int c = threadIdx.x; c < 1 + 2 * tc * pitch; c += STRIP_THREADS) A[c - 1] = 0.f;
    const int64_t M = (int64_t)len * width;
    const int groups = (width + tc - 1) / tc;
    const int64_t items = planes * groups;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // Column strips (ROWS = false) are moved with line f = thread % tc and walk index col_first, col_first +
    // 512 / tc, ...  A warp of up to 32 lines holds 32 / tc walk indices; they are taken tc apart, so that the
    // warp's 32 tile cells [f][i] (bank f + i) fall into 32 banks; the sweep of the block still covers
    // 512 / tc consecutive indices.
    const int col_first = tc <= 32 ? (lane >> tc_shift) * tc + (warp & (tc - 1)) + 32 * (warp >> tc_shift)
                                   : threadIdx.x >> tc_shift;
    __syncthreads();
    for (int64_t it = blockIdx.x; it < items; it += gridDim.x) {
        const int64_t plane = it / groups;
        const int f0 = (int)(it - plane * groups) * tc;
        const int nf = min(tc, width - f0);
        // ---- load the strip -------------------------------------------------------------------------
        if (ROWS) {
            for (int f = warp; f < nf; f += STRIP_THREADS / 32) {
                const float* s = in + plane * M + (int64_t)(f0 + f) * len + lane;
                float* d = A + f * pitch + lane;
                int i = lane;
                for (; i + 96 < len; i += 128, s += 128, d += 128) {  // four loads in flight
                    const float v0 = s[0], v1 = s[32], v2 = s[64], v3 = s[96];
                    d[0] = v0;
                    d[32] = v1;
                    d[64] = v2;
                    d[96] = v3;
                }
                for (; i < len; i += 32, s += 32, d += 32) d[0] = s[0];
            }
        } else {
            const int f = threadIdx.x & (tc - 1);
            const int step = STRIP_THREADS >> tc_shift;
            if (f < nf) {
                int i = col_first;
                const float* s = in + plane * M + f0 + (int64_t)i * width + f;
                const int64_t hop = (int64_t)step * width;
                float* d = A + f * pitch + i;
                for (; i + 3 * step < len; i += 4 * step, s += 4 * hop, d += 4 * step) {
                    const float v0 = s[0], v1 = s[hop], v2 = s[2 * hop], v3 = s[3 * hop];
                    d[0] = v0;
                    d[step] = v1;
                    d[2 * step] = v2;
                    d[3 * step] = v3;
                }
                for (; i < len; i += step, s += hop, d += step) d[0] = s[0];
            }
        }
        __syncthreads();
        // ---- totals of the first pass's input -------------------------------------------------------
#pragma unroll 1
        for (int job = threadIdx.x; job < n_jobs; job += STRIP_THREADS) {
            {
                const int line = job & (tc - 1), g = job >> tc_shift;
                const float* x = A + line * pitch + g * STRIP_SEG;
                double t0 = 0.0, t1 = 0.0;
#pragma unroll
                for (int k = 0; k < STRIP_SEG; k += 2) {
                    t0 += (double)x[k];
                    t1 += (double)x[k + 1];
                }
                tot[line * tot_pitch + g] = t0 + t1;
            }
        }
        // ---- three passes --------------------------------------------------------------------------
        float* X = A;
        float* Y = B;
#pragma unroll 1
        for (int pass = 0; pass < 3; ++pass) {
            __syncthreads();  // the totals of this pass's input are written
            // running sums of a line's totals, a warp per line: cum[q] = tot[0] + ... + tot[q - 1]
            for (int line = warp; line < tc; line += STRIP_THREADS / 32) {
                double carry = 0.0;
                for (int q0 = 0; q0 < n_seg; q0 += 32) {
                    const int q = q0 + lane;
                    double v = q < n_seg ? tot[line * tot_pitch + q] : 0.0;
#pragma unroll
                    for (int d = 1; d < 32; d *= 2) {
                        const double up = __shfl_up_sync(0xffffffffu, v, d);
                        if (lane >= d) v += up;
                    }
                    if (q < n_seg) cum[line * cum_pitch + q + 1] = carry + v;
                    carry += __shfl_sync(0xffffffffu, v, 31);
                }
                if (lane == 0) cum[line * cum_pitch] = 0.0;
            }
            __syncthreads();
#pragma unroll 1
            for (int job = threadIdx.x; job < n_jobs; job += STRIP_THREADS) {
                {
                    const int line = job & (tc - 1), g = job >> tc_shift;
                    const int a = g * STRIP_SEG;
                    const float* x = X + line * pitch;
                    // window sum at the segment's first cell: whole segments from the running sums, the
                    // cells at the window's two ends singly
                    const int lo = max(0, a - radius), hi = min(len_pad - 1, a + radius);
                    const int q_lo = (lo + STRIP_SEG - 1) / STRIP_SEG, q_hi = (hi + 1) / STRIP_SEG - 1;
                    int left_end = hi + 1, right_begin = hi + 1;  // cells [lo, left_end) and [right_begin, hi] singly
                    double sum = 0.0;
                    if (q_lo <= q_hi) {
                        const double* cl = cum + line * cum_pitch;
                        sum = cl[q_hi + 1] - cl[q_lo];
                        left_end = q_lo * STRIP_SEG;
                        right_begin = (q_hi + 1) * STRIP_SEG;
                    }
                    for (int j = lo; j < left_end; ++j) sum += (double)x[j];
                    for (int j = right_begin; j <= hi; ++j) sum += (double)x[j];
                    float* y = Y + line * pitch + a;
                    double t_next = a < len ? strip_round24(sum) : 0.0;
                    y[0] = (float)t_next;
                    const float* pe = x + a + radius;      // pe[k] enters at cell a + k
                    const float* pl = x + a - radius - 1;  // pl[k] leaves
                    const bool whole = a + STRIP_SEG <= len;
                    const bool e_all = a + STRIP_SEG - 1 + radius <= len_pad;  // (cells [len, len_pad] are zero)
                    const bool e_none = a + 1 + radius >= len;
                    const bool l_all = a >= radius;
                    const bool l_none = a + STRIP_SEG - 1 <= radius;
                    if (whole && e_all && l_all) t_next = strip_walk<true, true>(pe, pl, y, sum, t_next);
                    else if (whole && e_all && l_none) t_next = strip_walk<true, false>(pe, pl, y, sum, t_next);
                    else if (whole && e_none && l_all) t_next = strip_walk<false, true>(pe, pl, y, sum, t_next);
                    else if (whole && e_none && l_none) t_next = strip_walk<false, false>(pe, pl, y, sum, t_next);
                    else {
                        // a window end crosses the line's end inside the segment: indices are clamped into a zero cell
#pragma unroll 5
                        for (int k = 1; k < STRIP_SEG; ++k) {
                            const int i = a + k;
                            const float enter = x[min(i + radius, len_pad)];  // (cell len_pad is zero)
                            const float leave = x[max(i - radius - 1, -1)];   // (so is cell -1)
                            sum += (double)enter - (double)leave;
                            const double o = i < len ? strip_round24(sum) : 0.0;
                            y[k] = (float)o;
                            t_next += o;
                        }
                    }
                    tot[line * tot_pitch + g] = t_next;
                }
            }
            float* t = X; X = Y; Y = t;
        }
        __syncthreads();
        // ---- write (X holds the result) --------------------------------------------------------------
        if (ROWS) {
            for (int f = warp; f < nf; f += STRIP_THREADS / 32) {
                float* d = out + plane * M + (int64_t)(f0 + f) * len + lane;
                const float* s = X + f * pitch + lane;
                int i = lane;
                for (; i + 96 < len; i += 128, s += 128, d += 128) {
                    d[0] = s[0];
                    d[32] = s[32];
                    d[64] = s[64];
                    d[96] = s[96];
                }
                for (; i < len; i += 32, s += 32, d += 32) d[0] = s[0];
            }
        } else {
            // (len = rows, width = cols: cell i of line f0 + f is neuron i * width + f0 + f)
            ST* dst = W + (int64_t)(v0 + plane) * M + f0;
            const double* rd_base = rden + f0;
            const int f = threadIdx.x & (tc - 1);
            if (f < nf)
                for (int i = col_first; i < len; i += STRIP_THREADS >> tc_shift) {
                    const double rd = rd_base[(int64_t)i * width + f];
                    if (rd != 0.0) dst[(int64_t)i * width + f] = (ST)(float)((double)X[f * pitch + i] * rd);
                }
        }
        __syncthreads();
    }
}

// BT: type of the two plane buffers (double: exact; float: rounded between passes like the
// device-memory route, for planes too large for two fp64 buffers); running sums are fp64 either way.
template <typename ST, typename BT, int THREADS, bool TOTALS>
__global__ void __launch_bounds__(THREADS)
k_upd_blur_fused(const float* __restrict__ slab, int planes, int rows, int cols, int radius, int seg_r, int seg_c,
                 const double* __restrict__ rden, ST* __restrict__ W, int v0)
{
    extern __shared__ __align__(16) unsigned char fused_raw[];
    __shared__ double tot[THREADS];
    const int pitch = cols | 1;  // odd, in cells
    const int M = rows * cols;   // <= FUSED_PREFETCH * THREADS
    BT* A = reinterpret_cast<BT*>(fused_raw);
    BT* B = A + rows * pitch;
    // the next plane's counts wait in registers while the current plane is blurred
    float pre[FUSED_PREFETCH];
    if ((int)blockIdx.x < planes) {
        const float* src = slab + (int64_t)blockIdx.x * M;
#pragma unroll
        for (int k = 0; k < FUSED_PREFETCH; ++k) {
            const int g = threadIdx.x + k * THREADS;
            pre[k] = g < M ? __ldg(src + g) : 0.f;
        }
    }
    // cell (r, c) of this thread's k-th element, in transposed order (g = c * rows + r) and in
    // neuron order (i = r * cols + c): advanced by THREADS per element without divisions
    const int t_c0 = threadIdx.x / rows, t_r0 = threadIdx.x % rows;
    const int t_dc = THREADS / rows, t_dr = THREADS % rows;
    const int n_r0 = threadIdx.x / cols, n_c0 = threadIdx.x % cols;
    const int n_dr = THREADS / cols, n_dc = THREADS % cols;
    for (int plane = blockIdx.x; plane < planes; plane += gridDim.x) {
        {
            int r = t_r0, c = t_c0;
#pragma unroll
            for (int k = 0; k < FUSED_PREFETCH; ++k) {
                if ((int)threadIdx.x + k * THREADS < M) A[r * pitch + c] = (BT)pre[k];
                r += t_dr; c += t_dc;
                if (r >= rows) { r -= rows; c += 1; }
            }
        }
        __syncthreads();
        if (plane + (int)gridDim.x < planes) {
            const float* src = slab + (int64_t)(plane + gridDim.x) * M;
#pragma unroll
            for (int k = 0; k < FUSED_PREFETCH; ++k) {
                const int g = threadIdx.x + k * THREADS;
                pre[k] = g < M ? __ldg(src + g) : 0.f;
            }
        }
        BT* x = A;
        BT* y = B;
        for (int pass = 0; pass < 3; ++pass) {  // along the lattice rows: a line is a row
            box_lines<TOTALS>(x, y, rows, cols, pitch, 1, radius, seg_r, tot);
            __syncthreads();
            BT* t = x; x = y; y = t;
        }
        for (int pass = 0; pass < 3; ++pass) {  // along the lattice columns: a line is a column
            box_lines<TOTALS>(x, y, cols, rows, 1, pitch, radius, seg_c, tot);
            __syncthreads();
            BT* t = x; x = y; y = t;
        }
        ST* dst = W + (int64_t)(v0 + plane) * M;
        {
            int r = n_r0, c = n_c0;
            for (int i = threadIdx.x; i < M; i += THREADS) {
                const double rd = rden[i];
                if (rd != 0.0) dst[i] = (ST)(float)((double)x[r * pitch + c] * rd);
                r += n_dr; c += n_dc;
                if (c >= cols) { c -= cols; r += 1; }
            }
        }
        __syncthreads();
    }
}

// The denominator's route on a small lattice, one block: blur the sample counts (transposed cell
// order) like a numerator plane, count the occupied cells within the reach of three passes
// (3 * radius) along each axis with the same box walk (the counts are integers, exact in fp64), and
// write the reciprocal of the blurred denominator where the reach is not empty, else 0 (= keep).
__global__ void __launch_bounds__(FUSED_THREADS)
k_upd_den_fused(const float* __restrict__ den_t, const int32_t* __restrict__ occ, int rows, int cols, int radius,
                int seg_r, int seg_c, double* __restrict__ rden)
{
    extern __shared__ __align__(16) unsigned char fused_raw[];
    __shared__ double tot[FUSED_THREADS];
    const int pitch = cols | 1;
    const int M = rows * cols;
    double* A = reinterpret_cast<double*>(fused_raw);
    double* B = A + rows * pitch;
    double* C = A + 2 * rows * pitch;
    for (int g = threadIdx.x; g < M; g += blockDim.x) {
        const int c = g / rows, r = g - c * rows;
        A[r * pitch + c] = (double)den_t[g];
    }
    __syncthreads();
    double* x = A;
    double* y = B;
    for (int pass = 0; pass < 3; ++pass) {
        box_lines<false>(x, y, rows, cols, pitch, 1, radius, seg_r, tot);
        __syncthreads();
        double* t = x; x = y; y = t;
    }
    for (int pass = 0; pass < 3; ++pass) {
        box_lines<false>(x, y, cols, rows, 1, pitch, radius, seg_c, tot);
        __syncthreads();
        double* t = x; x = y; y = t;
    }
    for (int i = threadIdx.x; i < M; i += blockDim.x) {
        const int r = i / cols, c = i - r * cols;
        C[r * pitch + c] = x[r * pitch + c];
    }
    __syncthreads();
    for (int i = threadIdx.x; i < M; i += blockDim.x) {
        const int r = i / cols, c = i - r * cols;
        A[r * pitch + c] = occ[i] > 0 ? 1.0 : 0.0;
    }
    __syncthreads();
    box_lines<false>(A, B, rows, cols, pitch, 1, 3 * radius, seg_r, tot);
    __syncthreads();
    box_lines<false>(B, A, cols, rows, 1, pitch, 3 * radius, seg_c, tot);
    __syncthreads();
    for (int i = threadIdx.x; i < M; i += blockDim.x) {
        const int r = i / cols, c = i - r * cols;
        rden[i] = A[r * pitch + c] > 0.0 ? 1.0 / C[r * pitch + c] : 0.0;
    }
}

// [plane][a][b] -> [plane][b][a] through 32 x 32 shared-memory tiles
template <typename T>
__global__ void k_transpose(const T* __restrict__ in, T* __restrict__ out, int a, int b)
{
    __shared__ T tile[32][33];
    const int64_t plane = blockIdx.z;
    const T* src = in + plane * (int64_t)a * b;
    T* dst = out + plane * (int64_t)a * b;
    const int b0 = blockIdx.x * 32, a0 = blockIdx.y * 32;
    for (int j = threadIdx.y; j < 32; j += blockDim.y) {
        const int ia = a0 + j, ib = b0 + threadIdx.x;
        if (ia < a && ib < b) tile[j][threadIdx.x] = src[(int64_t)ia * b + ib];
    }
    __syncthreads();
    for (int j = threadIdx.y; j < 32; j += blockDim.y) {
        const int ib = b0 + j, ia = a0 + threadIdx.x;
        if (ia < a && ib < b) dst[(int64_t)ib * a + ia] = tile[threadIdx.x][j];
    }
}

inline unsigned blocks_for(int64_t threads) { return (unsigned)((threads + UPD_THREADS - 1) / UPD_THREADS); }

// three passes along the slow index, ping-ponging between x and y; returns where the result is
template <typename T, typename ACC>
T* three_passes(som_handle* h, T* x, T* y, int64_t planes, int len, int width, int radius, cudaStream_t st)
{
    for (int pass = 0; pass < 3; ++pass) {
        k_box_pass<T, ACC><<<blocks_for(planes * width), UPD_THREADS, 0, st>>>(x, y, planes, len, width, radius);
        h->launches += 1;
        T* t = x; x = y; y = t;
    }
    return x;
}

template <typename T>
void transpose(som_handle* h, const T* in, T* out, int64_t planes, int a, int b, cudaStream_t st)
{
    for (int64_t p0 = 0; p0 < planes; p0 += 65535) {
        const int64_t np = planes - p0 < 65535 ? planes - p0 : 65535;
        dim3 grid((unsigned)((b + 31) / 32), (unsigned)((a + 31) / 32), (unsigned)np);
        k_transpose<T><<<grid, dim3(32, 8), 0, st>>>(in + p0 * (int64_t)a * b, out + p0 * (int64_t)a * b, a, b);
        h->launches += 1;
    }
}

}  // namespace

size_t som_update_workspace_bytes(const som_handle* h, int64_t budget_bytes, int* planes_per_slab)
{
    const int64_t M = h->M;
    int64_t planes = budget_bytes / (2 * M * 4);
    if (planes < 1) planes = 1;
    if (planes > h->V) planes = h->V;
    *planes_per_slab = (int)planes;
    // den (2 buffers), occupancy and reach (3 int buffers, 1 spare), reciprocal (fp64), then the two slab buffers
    return som_align_up((size_t)M * 4, 256) * 8 + 2 * som_align_up((size_t)planes * M * 4, 256);
}

int som_launch_update(som_handle* h, int rows, int cols, const int32_t* indptr, const int32_t* indices,
                      int64_t n, const int32_t* bmu, int radius, int planes_per_slab, const int32_t* hot_slot,
                      const int32_t* slot_feat, int n_hot_slots, cudaStream_t st, cudaStream_t aux,
                      cudaEvent_t ev_join)
{
    // The denominator's route (single-block kernels) and the clearing of the first slab run on the
    // side stream `aux`, which the caller has made wait for `st`; `st` joins it before the scatter.
    // Meanwhile `st` runs the selection of the frequent features and their masks.
    cudaStream_t main_st = st;
    if (aux) st = aux;
    const int64_t M = h->M;
    const size_t mb = som_align_up((size_t)M * 4, 256);
    char* ws = reinterpret_cast<char*>(h->ws);
    float* den_a = reinterpret_cast<float*>(ws);
    float* den_b = reinterpret_cast<float*>(ws + mb);
    int32_t* occ_a = reinterpret_cast<int32_t*>(ws + 2 * mb);
    int32_t* occ_b = reinterpret_cast<int32_t*>(ws + 3 * mb);
    int32_t* occ_c = reinterpret_cast<int32_t*>(ws + 4 * mb);
    float* slab_a = reinterpret_cast<float*>(ws + 8 * mb);
    float* slab_b = reinterpret_cast<float*>(ws + 8 * mb + som_align_up((size_t)planes_per_slab * M * 4, 256));

    // ---- denominator and the exact reach of the blur --------------------------------------------
    SOM_CK(h, cudaMemsetAsync(den_a, 0, (size_t)M * 4, st));
    SOM_CK(h, cudaMemsetAsync(occ_a, 0, (size_t)M * 4, st));
    if (n > 0) {
        const int use_smem = M * 4 <= 96 * 1024;
        if (use_smem) {
            SOM_CK(h, cudaFuncSetAttribute(k_upd_count, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024));
            k_upd_count<<<h->sm_count * 2, 1024, (size_t)M * 4, st>>>(bmu, n, rows, cols, 1, den_a, occ_a, h->dev_flags);
        } else {
            k_upd_count<<<h->sm_count * 8, UPD_THREADS, 0, st>>>(bmu, n, rows, cols, 0, den_a, occ_a, h->dev_flags);
        }
        h->launches += 1;
    }
    double* rden = reinterpret_cast<double*>(ws + 6 * mb);
    // planes of up to 4096 cells are blurred on chip in fp64 buffers by 256 threads, planes of up to
    // 16384 cells in fp32 buffers by 1024 threads; larger ones take the passes through device memory
    const int wide = M > FUSED_PREFETCH * FUSED_THREADS;
    const int f_threads = wide ? FUSED_THREADS_WIDE : FUSED_THREADS;
    const bool fused = M <= FUSED_PREFETCH * f_threads && rows <= f_threads && cols <= f_threads;
    const int seg_r = f_threads / rows > 1 ? f_threads / rows : 1;  // segments per lattice row
    const int seg_c = f_threads / cols > 1 ? f_threads / cols : 1;  // segments per lattice column
    const size_t plane_sh = (size_t)rows * (cols | 1) * (wide ? sizeof(float) : sizeof(double));
    if (fused && !wide) {
        SOM_CK(h, cudaFuncSetAttribute(k_upd_den_fused, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)(3 * plane_sh)));
        k_upd_den_fused<<<1, FUSED_THREADS, 3 * plane_sh, st>>>(den_a, occ_a, rows, cols, radius, seg_r, seg_c, rden);
        h->launches += 1;
    } else {
        float* d = three_passes<float, double>(h, den_a, den_b, 1, cols, rows, radius, st);  // along the lattice rows
        float* d_other = (d == den_a) ? den_b : den_a;
        transpose<float>(h, d, d_other, 1, cols, rows, st);
        float* den_blurred = three_passes<float, double>(h, d_other, d, 1, rows, cols, radius, st);
        // occupied cells within 3 * radius along each axis (exact integer counts; the count of a cell
        // is at most M, so int32 suffices)
        const int reach_r = 3 * radius;
        k_box_pass<int32_t, int32_t><<<blocks_for(cols), UPD_THREADS, 0, st>>>(occ_a, occ_b, 1, rows, cols, reach_r);
        transpose<int32_t>(h, occ_b, occ_c, 1, rows, cols, st);
        k_box_pass<int32_t, int32_t><<<blocks_for(rows), UPD_THREADS, 0, st>>>(occ_c, occ_b, 1, cols, rows, reach_r);
        transpose<int32_t>(h, occ_b, occ_c, 1, cols, rows, st);  // occ_c: reach count in neuron order
        k_upd_reciprocal<<<blocks_for(M), UPD_THREADS, 0, st>>>(den_blurred, occ_c, M, rden);
        h->launches += 3;
    }
    SOM_CK(h, cudaGetLastError());

    if (aux) {
        const int64_t first = planes_per_slab < h->V ? planes_per_slab : h->V;
        SOM_CK(h, cudaMemsetAsync(slab_a, 0, (size_t)first * M * 4, aux));
        SOM_CK(h, cudaEventRecord(ev_join, aux));
        st = main_st;
    }
    // Larger lattices: the strip route wherever a strip of at least eight lines over the whole length of
    // either axis fits in shared memory twice over (fp32); else the passes through device memory.
    struct StripGeom { int tc, shift, pitch; size_t sh; };
    auto strip_geom = [&](int len, int width) {
        StripGeom g = {0, 0, 0, 0};
        const int n_seg = (len + STRIP_SEG - 1) / STRIP_SEG;
        const int pitch = (n_seg * STRIP_SEG + 31) / 32 * 32 + 1;  // > the padded length, 1 modulo 32
        auto bytes = [&](int tc) {
            return (size_t)tc * ((n_seg | 1) + ((n_seg + 1) | 1)) * 8 + (size_t)(2 * tc * pitch + 1) * 4;
        };
        // as many lines as give every thread one or two segments, three blocks per SM where that leaves at
        // least 16 lines (a warp then covers 32 banks), never fewer than 8 lines
        int tc = 256;
        while (tc > 8 && (tc * n_seg > 2 * STRIP_THREADS || bytes(tc) > (size_t)80 * 1024)) tc /= 2;
        while (tc > 8 && tc / 2 >= width) tc /= 2;  // few lines: all of them in one strip
        if (tc * n_seg > STRIP_MAX_ITERS * STRIP_THREADS || bytes(tc) > (size_t)200 * 1024) return g;
        g.tc = tc;
        while ((1 << g.shift) < tc) ++g.shift;
        g.pitch = pitch;
        g.sh = bytes(tc);
        return g;
    };
    const StripGeom sg_r = fused ? StripGeom{0, 0, 0, 0} : strip_geom(cols, rows);  // walk along a lattice row
    const StripGeom sg_c = fused ? StripGeom{0, 0, 0, 0} : strip_geom(rows, cols);  // walk down a lattice column
    const bool strip = !fused && sg_r.tc > 0 && sg_c.tc > 0;
    // ---- numerator, slab by slab ------------------------------------------------------------------
    // (the per-sample masks of the hot features live behind the two slab buffers)
    uint32_t* hot_mask = reinterpret_cast<uint32_t*>(ws + 8 * mb + 2 * som_align_up((size_t)planes_per_slab * M * 4, 256));
    if (hot_slot && n > 0) {
        k_upd_hot_mask<<<blocks_for(n), UPD_THREADS, 0, st>>>(indptr, indices, n, h->V, hot_slot, hot_mask, h->dev_flags);
        h->launches += 1;
    }
    for (int v0 = 0; v0 < h->V; v0 += planes_per_slab) {
        const int v1 = (v0 + planes_per_slab < h->V) ? v0 + planes_per_slab : h->V;
        const int64_t planes = v1 - v0;
        if (aux && v0 == 0) SOM_CK(h, cudaStreamWaitEvent(st, ev_join, 0));  // first slab cleared, denominator ready
        else SOM_CK(h, cudaMemsetAsync(slab_a, 0, (size_t)planes * M * 4, st));
        if (n > 0) {
            k_upd_scatter<<<blocks_for(n), UPD_THREADS, 0, st>>>(indptr, indices, n, bmu, v0, v1, rows, cols, hot_slot,
                                                                 slab_a, strip ? 1 : 0);
            h->launches += 1;
            if (hot_slot) {
                int ppb = (int)((160 * 1024) / (M * 4));
                if (ppb > n_hot_slots) ppb = n_hot_slots;
                const int groups = (n_hot_slots + ppb - 1) / ppb;
                int slices = h->sm_count / groups;
                slices = slices < 1 ? 1 : (slices > 16 ? 16 : slices);
                const size_t sh = (size_t)ppb * M * 4;
                SOM_CK(h, cudaFuncSetAttribute(k_upd_scatter_hot, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sh));
                k_upd_scatter_hot<<<dim3(slices, groups), 1024, sh, st>>>(hot_mask, n, bmu, v0, v1, rows, cols, slot_feat,
                                                                        n_hot_slots, ppb, slab_a, strip ? 1 : 0);
                h->launches += 1;
            }
        }
        // small lattices: everything after the scatter in one kernel, a plane at a time on chip
        const size_t fused_sh = 2 * plane_sh;
        if (fused) {
            // segment totals for the first window sums where the window spans more than three segments
            const bool totals = 2 * radius + 1 > 3 * ((cols + seg_r - 1) / seg_r) &&
                                2 * radius + 1 > 3 * ((rows + seg_c - 1) / seg_c);
            const int per_sm = (int)((size_t)216 * 1024 / (fused_sh + 1024));
            int64_t grid = (int64_t)h->sm_count * per_sm;
            if (grid > planes) grid = planes;
#define SOM_FUSED(ST_, BT_, THREADS_, TOT_, W_)                                                                 \
    do {                                                                                                        \
        SOM_CK(h, cudaFuncSetAttribute(k_upd_blur_fused<ST_, BT_, THREADS_, TOT_>,                              \
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)fused_sh));            \
        k_upd_blur_fused<ST_, BT_, THREADS_, TOT_><<<(unsigned)grid, THREADS_, fused_sh, st>>>(                 \
            slab_a, (int)planes, rows, cols, radius, seg_r, seg_c, rden, W_, v0);                               \
    } while (0)
#define SOM_FUSED_T(ST_, BT_, THREADS_, W_)                                                                     \
    do {                                                                                                        \
        if (totals) SOM_FUSED(ST_, BT_, THREADS_, true, W_);                                                    \
        else SOM_FUSED(ST_, BT_, THREADS_, false, W_);                                                          \
    } while (0)
            if (h->Wh && wide) SOM_FUSED_T(__half, float, FUSED_THREADS_WIDE, const_cast<__half*>(h->Wh));
            else if (h->Wh) SOM_FUSED_T(__half, double, FUSED_THREADS, const_cast<__half*>(h->Wh));
            else if (wide) SOM_FUSED_T(float, float, FUSED_THREADS_WIDE, const_cast<float*>(h->W));
            else SOM_FUSED_T(float, double, FUSED_THREADS, const_cast<float*>(h->W));
#undef SOM_FUSED_T
#undef SOM_FUSED
            h->launches += 1;
            SOM_CK(h, cudaGetLastError());
            continue;
        }
        if (strip) {
            // slab_a holds the counts in neuron order
            auto grid_for = [&](size_t sh, int64_t items) {
                int per_sm = (int)((size_t)226 * 1024 / (sh + 1024));
                per_sm = per_sm < 1 ? 1 : (per_sm > 3 ? 3 : per_sm);  // (the kernel's launch bound: three blocks)
                const int64_t g = (int64_t)h->sm_count * per_sm;
                return (unsigned)(g < items ? g : items);
            };
            const int64_t items_r = planes * ((rows + sg_r.tc - 1) / sg_r.tc);
            const int64_t items_c = planes * ((cols + sg_c.tc - 1) / sg_c.tc);
#define SOM_STRIP(ST_, ROWS_, IN_, OUT_, LEN_, WIDTH_, G_, ITEMS_, W_)                                           \
    do {                                                                                                         \
        SOM_CK(h, cudaFuncSetAttribute(k_upd_strip<ST_, ROWS_>, cudaFuncAttributeMaxDynamicSharedMemorySize,     \
                                       (int)(G_).sh));                                                           \
        k_upd_strip<ST_, ROWS_><<<grid_for((G_).sh, ITEMS_), STRIP_THREADS, (G_).sh, st>>>(                      \
            IN_, OUT_, planes, LEN_, WIDTH_, radius, (G_).tc, (G_).shift, (G_).pitch, rden, W_, v0);            \
    } while (0)
            float* none_w = nullptr;
            SOM_STRIP(float, true, slab_a, slab_b, cols, rows, sg_r, items_r, none_w);
            if (h->Wh) SOM_STRIP(__half, false, slab_b, nullptr, rows, cols, sg_c, items_c, const_cast<__half*>(h->Wh));
            else SOM_STRIP(float, false, slab_b, nullptr, rows, cols, sg_c, items_c, const_cast<float*>(h->W));
#undef SOM_STRIP
            h->launches += 2;
            SOM_CK(h, cudaGetLastError());
            continue;
        }
        float* x = three_passes<float, double>(h, slab_a, slab_b, planes, cols, rows, radius, st);
        float* y = (x == slab_a) ? slab_b : slab_a;
        transpose<float>(h, x, y, planes, cols, rows, st);  // y: neuron order
        for (int pass = 0; pass < 2; ++pass) {
            k_box_pass<float, double><<<blocks_for(planes * cols), UPD_THREADS, 0, st>>>(y, x, planes, rows, cols, radius);
            h->launches += 1;
            float* t = x; x = y; y = t;
        }
        if (h->Wh)
            k_box_pass_divide<__half><<<blocks_for(planes * cols), UPD_THREADS, 0, st>>>(
                y, planes, rows, cols, radius, rden, const_cast<__half*>(h->Wh), v0);
        else
            k_box_pass_divide<float><<<blocks_for(planes * cols), UPD_THREADS, 0, st>>>(
                y, planes, rows, cols, radius, rden, const_cast<float*>(h->W), v0);
        h->launches += 1;
        SOM_CK(h, cudaGetLastError());
    }
    return SOM_OK;
}
