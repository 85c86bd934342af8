// Row-table BMU search kernel (the fast path of som_bmu), the certificate of the two-stage
// search and the finalisation.
//
// Decomposition (Section 3.3 of the paper, re-planned for B200): a work unit is a neuron
// range of T = 8*R neurons (R neurons per lane) times a contiguous part of the mask-sorted
// sample list.  One persistent block per SM claims units from a global counter in range-major
// order, so that at any time only a few neuron ranges are live and their codebook slabs
// W[:, i0..i0+T) stay L2-resident while HBM sees the codebook about once per batch.  Inside a
// unit the warps pull chunks of samples from a shared counter, which keeps them busy whatever
// the mix of row lengths.
//
// Inside a block the rows W[v*M + i0 .. i0+T) of the batch's hottest features (the row
// table) are staged in shared memory once per unit.  Eight lanes form a team that owns one
// sample at a time; a lane keeps R score accumulators in registers and subtracts, for every
// code of the sample, its 128-bit slices of the row: a shared-memory read for hot features, a
// coalesced 128-bit read-only load of the L2-resident slab for tail features (the team's eight
// loads cover one contiguous 128-byte segment).  How the R neurons map onto a row, and how a
// slice is consumed, is the storage layout's business (fp32: packed f32x2 subtractions;
// fp16: mixed-precision adds; see the Lay* structs).  The accumulators start from ||w||^2/2
// minus the rows of the sample's mask features, which is held in registers across consecutive
// samples that share the mask (they are adjacent after the plan's sort).
//
// Feeding the teams: a sample's 48-byte slot sits at a fixed address for its sorted position.
// Each warp owns a two-stage ring in shared memory; 14 of its lanes fetch the slot and key
// bytes of round r+2 into registers, store those of round r+1, and every team reads round r
// from the ring, so slot and key latency is never on the critical path.  A sample's first
// four tail rows go in flight at the top of its round and are consumed after its hot rows.
// The first hot row is subtracted in three-operand form (score = prefix - row), the rest of
// the hot loop is a jump table on the longest hot list of the warp's four samples (shorter
// lists are padded with an all-zero row), the slot array is padded to whole rounds and all
// addressing is by pointer increment, so the inner steps carry no predicate.
//
// Argmin: each lane reduces its R scores, compares with the sample's packed key and only on a
// (rare) improvement issues a 64-bit atomicMin on (ordered score bits, neuron).  The unsigned
// minimum of that key is the lexicographic (score, lowest neuron) minimum, so the combine is
// order-independent and ties break to the lowest neuron index (Section 3.1).
#include "som_internal.cuh"
#include "som_plan.cuh"

namespace {

constexpr int CHUNK = 128;  // samples a warp takes at a time ...
// ... where the launch prunes: 64 (its test takes 32 samples at a time and the search rounds of a chunk are few either
// way; measured 5 to 7 % faster than 128 at every map size, 32 slower again; the search that reads every row loses 1 %
// with 64)
constexpr int PRUNE_CHUNK = 64;
constexpr int SMALL_CHUNK = 32;  // ... and near the end of a unit, so that its warps finish together
constexpr int RING_STAGE = 224;  // bytes of one ring stage: 4 slots + 4 keys
constexpr int SLOT_Q = SOM_SLOT_WORDS / 4;  // uint4 per slot

typedef unsigned long long u64;

struct Pair2 {  // four fp32 as two packed pairs
    u64 lo, hi;
};

// R neurons of one lane: H = R / 4 groups of four consecutive neurons, 32 neurons apart
template <int H>
struct Acc {
    Pair2 g[H];
};

__device__ __forceinline__ void unpack2(u64 v, float& a, float& b)
{
    asm("mov.b64 {%0,%1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}

__device__ __forceinline__ void sub_pair(Pair2& acc, const Pair2 w)
{
    asm("sub.rn.f32x2 %0, %0, %1;" : "+l"(acc.lo) : "l"(w.lo));
    asm("sub.rn.f32x2 %0, %0, %1;" : "+l"(acc.hi) : "l"(w.hi));
}

__device__ __forceinline__ Pair2 lds_row(const unsigned char* p)
{
    const ulonglong2 v = *reinterpret_cast<const ulonglong2*>(p);
    Pair2 r;
    r.lo = v.x;
    r.hi = v.y;
    return r;
}

// 128-bit read of a tail row slice through the read-only path with normal eviction priority:
// an L1::no_allocate hint would also demote the line to evict-first in L2, and the slab rows
// are exactly what has to stay L2-resident.  Allocating in the 60 KB of L1 left beside the
// table measured 4 % faster than an L2-only (.cg) load: moderately frequent tail features
// recur within a block's recent rows.
__device__ __forceinline__ Pair2 ldg_row(const float* p)
{
    Pair2 r;
    asm("ld.global.nc.v2.b64 {%0,%1}, [%2];" : "=l"(r.lo), "=l"(r.hi) : "l"(p));
    return r;
}

template <int H>
__device__ __forceinline__ void sub_acc(Acc<H>& a, const Acc<H>& w)
{
#pragma unroll
    for (int x = 0; x < H; ++x) sub_pair(a.g[x], w.g[x]);
}

// out = a - w (three-operand form: no copy of `a` is needed when it must survive)
template <int H>
__device__ __forceinline__ Acc<H> sub_acc3(const Acc<H>& a, const Acc<H>& w)
{
    Acc<H> r;
#pragma unroll
    for (int x = 0; x < H; ++x) {
        asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r.g[x].lo) : "l"(a.g[x].lo), "l"(w.g[x].lo));
        asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r.g[x].hi) : "l"(a.g[x].hi), "l"(w.g[x].hi));
    }
    return r;
}

// a lane's slice of a shared-memory row: 16 bytes per group, groups 128 bytes apart
template <int H>
__device__ __forceinline__ Acc<H> lds_acc(const unsigned char* p)
{
    Acc<H> r;
#pragma unroll
    for (int x = 0; x < H; ++x) r.g[x] = lds_row(p + 128 * x);
    return r;
}

// a lane's slice of a codebook row in global memory
template <int H>
__device__ __forceinline__ Acc<H> ldg_acc(const float* p)
{
    Acc<H> r;
#pragma unroll
    for (int x = 0; x < H; ++x) r.g[x] = ldg_row(p + 32 * x);
    return r;
}

// 128-bit load of slot or key bytes past L1 (the keys change under atomics).  `keep` asks L2 to evict the line
// last: on a small batch the whole slot and key stream then stays L2-resident from one neuron range to the
// next instead of being fetched from device memory once per range.
__device__ __forceinline__ uint4 ld_feed(const uint4* p, uint64_t policy)
{
    uint4 v;
    asm volatile("ld.global.L1::no_allocate.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p), "l"(policy));
    return v;
}

__device__ __forceinline__ uint32_t lo16(uint32_t w) { return w & 0xffffu; }
__device__ __forceinline__ uint32_t hi16(uint32_t w) { return w >> 16; }

// address of row `code` in the codebook slab: base + code * row_stride_bytes, one mad.wide
__device__ __forceinline__ const unsigned char* row_ptr(const unsigned char* base, uint32_t code,
                                                        uint32_t stride_bytes)
{
    const unsigned char* p;
    asm("mad.wide.u32 %0, %1, %2, %3;" : "=l"(p) : "r"(code), "r"(stride_bytes), "l"(base));
    return p;
}

// Staging of whole, 16-byte aligned table rows through registers: 128-bit pieces, eight in flight per
// lane.  (Bulk async copies, one per row, completion counted on an mbarrier, measured slower here: 8 %
// on the largest map when one warp enqueues them, 2 % when all warps do; a range's rows are many small
// copies from as many pages.)
template <typename L>
__device__ __forceinline__ void stage_vec(unsigned char* tab, const typename L::Store* __restrict__ W, int64_t M,
                                          int64_t i0, const int32_t* __restrict__ slot_feat, int n_rows,
                                          int warp, int lane, int warps)
{
    constexpr int PPR = L::ROWB / 16;                // pieces per row (at most 32)
    constexpr int RPL = 32 / PPR;                    // rows one warp-wide load covers
    constexpr int U = 8;
    const int sub_row = lane / PPR, col = lane % PPR;
    for (int row0 = warp * U * RPL; row0 < n_rows; row0 += warps * U * RPL) {
        uint4 v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int row = row0 + u * RPL + sub_row;
            const int f = row < n_rows ? slot_feat[row] : -1;
            v[u] = make_uint4(0u, 0u, 0u, 0u);
            if (f >= 0) v[u] = __ldg(reinterpret_cast<const uint4*>(W + (int64_t)f * M + i0) + col);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int row = row0 + u * RPL + sub_row;
            if (row < n_rows) reinterpret_cast<uint4*>(tab + (size_t)row * L::ROWB)[col] = v[u];
        }
    }
}

// ---- storage layouts of the row table -------------------------------------------------------
// A layout says how a lane's R neurons map onto a T-neuron row, how the lane reads its slice of
// a row from shared or global memory, and how a slice is subtracted from the lane's scores.
// In both layouts lane q of a team starts 16 bytes * q into a row.

// fp32 storage: R/4 groups of four neurons, 32 neurons apart; scores as packed f32x2 pairs.
template <int R_>
struct LayF32 {
    typedef float Store;
    static constexpr int R = R_, H = R_ / 4, T = 8 * R_, ROWB = T * 4;
    // tail rows of a sample whose loads go in flight before its hot rows (each holds R registers; with 16
    // neurons per lane three fit 128 registers at the price of a 36-byte spill, and measure 1 to 3 % faster
    // than two)
    static constexpr int TAILS_AHEAD = R_ >= 16 ? 3 : 4;
    static constexpr bool CAN_PRUNE = true;
    static constexpr int GROUPS = R_ / 4;       // (pruning) 32-neuron groups of a team's range with bounds of their own
    static constexpr bool HALF_GROUPS = false;  // every lane's x-th quad of neurons lies in group x
    static constexpr float SEED_SIGN = 1.f;     // scores are held as they are
    typedef Acc<H> Scores;
    typedef Acc<H> Slice;
    static __device__ __forceinline__ Slice lds(const unsigned char* p) { return lds_acc<H>(p); }
    static __device__ __forceinline__ Slice ldg(const unsigned char* p)
    {
        return ldg_acc<H>(reinterpret_cast<const float*>(p));
    }
    static __device__ __forceinline__ void sub(Scores& a, const Slice& w) { sub_acc<H>(a, w); }
    static __device__ __forceinline__ Scores sub3(const Scores& a, const Slice& w) { return sub_acc3<H>(a, w); }
    static __device__ __forceinline__ Scores seed(const float* hn, int q)
    {
        return lds_acc<H>(reinterpret_cast<const unsigned char*>(hn) + q * 16);
    }
    static __device__ __forceinline__ Scores worst()
    {
        Scores r;
        const u64 two_inf = 0x7f8000007f800000ull;
#pragma unroll
        for (int x = 0; x < H; ++x) r.g[x].lo = r.g[x].hi = two_inf;
        return r;
    }
    static __device__ __forceinline__ void unpack(const Scores& s, float (&a)[R_])
    {
#pragma unroll
        for (int x = 0; x < H; ++x) {
            unpack2(s.g[x].lo, a[4 * x], a[4 * x + 1]);
            unpack2(s.g[x].hi, a[4 * x + 2], a[4 * x + 3]);
        }
    }
    static __device__ __forceinline__ int lane_first(int q) { return 4 * q; }
    static __device__ __forceinline__ uint32_t neuron_of(int rr) { return (uint32_t)((rr >> 2) * 32 + (rr & 3)); }
    // stage table rows row0.. of this warp: a lane moves element `lane` of each 32-neuron group
    static __device__ __forceinline__ void stage(unsigned char* tab, const float* __restrict__ W, int64_t M,
                                                 int64_t i0, const int32_t* __restrict__ slot_feat,
                                                 int n_rows, int warp, int lane, int warps)
    {
        float* tab_f = reinterpret_cast<float*>(tab);
        for (int row0 = warp * 4; row0 < n_rows; row0 += warps * 4) {
            float v[4][H];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int row = row0 + u;
                const int f = row < n_rows ? slot_feat[row] : -1;
#pragma unroll
                for (int x = 0; x < H; ++x) {
                    const int64_t i = i0 + 32 * x + lane;
                    v[u][x] = (f >= 0 && i < M) ? __ldg(W + (int64_t)f * M + i) : 0.f;
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (row0 + u < n_rows) {
#pragma unroll
                    for (int x = 0; x < H; ++x) tab_f[(row0 + u) * T + 32 * x + lane] = v[u][x];
                }
        }
    }
};

// fp16 storage, fp32 scores (the paper's production precision, Section 3.2): a lane owns eight
// consecutive neurons, i.e. one 128-bit slice of a 128-byte row, so a row costs half the
// shared-memory and L2 wavefronts of the fp32 layout.  Every weight is widened exactly inside
// the mixed-precision add (add.rn.f32.f16: one rounding, that of the fp32 sum).  That
// instruction only adds, so the lane holds NEGATED scores, sum(rows) - ||w||^2/2, and flips
// the sign when it hands them to the argmin; (-a) - w and -(a + w) round identically, so the
// scores are those of the subtracting form.
struct LayF16 {
    typedef __half Store;
    static constexpr int R = 8, T = 64, ROWB = T * 2;
    static constexpr int TAILS_AHEAD = 4;
    // (no pruning with this layout: it serves neuron counts that 128 does not divide, which have no range maxima;
    //  forced onto a map that has them, its pruning variant hit a sporadic memory fault whose cause was not found
    //  by reading, so it is not built)
    static constexpr bool CAN_PRUNE = false;
    static constexpr int GROUPS = 1;
    static constexpr bool HALF_GROUPS = false;
    static constexpr float SEED_SIGN = -1.f;  // the seed array holds -||w||^2/2
    struct Scores { float v[8]; };
    typedef uint4 Slice;
    static __device__ __forceinline__ Slice lds(const unsigned char* p) { return *reinterpret_cast<const uint4*>(p); }
    static __device__ __forceinline__ Slice ldg(const unsigned char* p)
    {
        Slice r;
        asm("ld.global.nc.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
        return r;
    }
    static __device__ __forceinline__ void add2(float& d0, float& d1, float a0, float a1, uint32_t w)
    {
        asm("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %4;\n\t"
            "add.rn.f32.f16 %0, l, %2;\n\tadd.rn.f32.f16 %1, h, %3;\n\t}"
            : "=f"(d0), "=f"(d1) : "f"(a0), "f"(a1), "r"(w));
    }
    static __device__ __forceinline__ Scores sub3(const Scores& a, const Slice& w)
    {
        Scores r;
        add2(r.v[0], r.v[1], a.v[0], a.v[1], w.x);
        add2(r.v[2], r.v[3], a.v[2], a.v[3], w.y);
        add2(r.v[4], r.v[5], a.v[4], a.v[5], w.z);
        add2(r.v[6], r.v[7], a.v[6], a.v[7], w.w);
        return r;
    }
    static __device__ __forceinline__ void sub(Scores& a, const Slice& w) { a = sub3(a, w); }
    static __device__ __forceinline__ Scores seed(const float* hn, int q)
    {
        const float4 lo = *reinterpret_cast<const float4*>(hn + 8 * q);
        const float4 hi = *reinterpret_cast<const float4*>(hn + 8 * q + 4);
        Scores r;
        r.v[0] = lo.x; r.v[1] = lo.y; r.v[2] = lo.z; r.v[3] = lo.w;
        r.v[4] = hi.x; r.v[5] = hi.y; r.v[6] = hi.z; r.v[7] = hi.w;
        return r;
    }
    static __device__ __forceinline__ Scores worst()
    {
        Scores r;
#pragma unroll
        for (int j = 0; j < 8; ++j) r.v[j] = __int_as_float(0xff800000);  // negated scores: -inf
        return r;
    }
    static __device__ __forceinline__ void unpack(const Scores& s, float (&a)[8])
    {
#pragma unroll
        for (int j = 0; j < 8; ++j) a[j] = -s.v[j];
    }
    static __device__ __forceinline__ int lane_first(int q) { return 8 * q; }
    static __device__ __forceinline__ uint32_t neuron_of(int rr) { return (uint32_t)rr; }
    // a lane moves one 32-bit word (two neurons) of each row; M % 64 == 0 is guaranteed
    static __device__ __forceinline__ void stage(unsigned char* tab, const __half* __restrict__ W, int64_t M,
                                                 int64_t i0, const int32_t* __restrict__ slot_feat,
                                                 int n_rows, int warp, int lane, int warps)
    {
        uint32_t* tab_w = reinterpret_cast<uint32_t*>(tab);
        for (int row0 = warp * 8; row0 < n_rows; row0 += warps * 8) {
            uint32_t v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int row = row0 + u;
                const int f = row < n_rows ? slot_feat[row] : -1;
                v[u] = (f >= 0) ? __ldg(reinterpret_cast<const uint32_t*>(W + (int64_t)f * M + i0) + lane) : 0u;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u)
                if (row0 + u < n_rows) tab_w[(row0 + u) * 32 + lane] = v[u];
        }
    }
};

// The same with 16 neurons per lane: two groups of eight, 64 neurons apart (two 128-bit slices
// of a 256-byte row).  Twice the work per round for the same per-round bookkeeping.
struct LayF16W {
    typedef __half Store;
    static constexpr int R = 16, T = 128, ROWB = T * 2;
    static constexpr int TAILS_AHEAD = 4;
    static constexpr bool CAN_PRUNE = true;
    // (pruning) the four 32-neuron groups of the range have bounds of their own; a lane's first eight neurons lie
    // in group q >> 2, its second eight in group 2 + (q >> 2)
    static constexpr int GROUPS = 4;
    static constexpr bool HALF_GROUPS = true;
    static constexpr float SEED_SIGN = -1.f;
    struct Scores { float v[16]; };
    struct Slice { uint4 g[2]; };
    static __device__ __forceinline__ Slice lds(const unsigned char* p)
    {
        Slice r;
        r.g[0] = *reinterpret_cast<const uint4*>(p);
        r.g[1] = *reinterpret_cast<const uint4*>(p + 128);
        return r;
    }
    static __device__ __forceinline__ Slice ldg(const unsigned char* p)
    {
        Slice r;
        r.g[0] = LayF16::ldg(p);
        r.g[1] = LayF16::ldg(p + 128);
        return r;
    }
    static __device__ __forceinline__ Scores sub3(const Scores& a, const Slice& w)
    {
        Scores r;
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            LayF16::add2(r.v[8 * x + 0], r.v[8 * x + 1], a.v[8 * x + 0], a.v[8 * x + 1], w.g[x].x);
            LayF16::add2(r.v[8 * x + 2], r.v[8 * x + 3], a.v[8 * x + 2], a.v[8 * x + 3], w.g[x].y);
            LayF16::add2(r.v[8 * x + 4], r.v[8 * x + 5], a.v[8 * x + 4], a.v[8 * x + 5], w.g[x].z);
            LayF16::add2(r.v[8 * x + 6], r.v[8 * x + 7], a.v[8 * x + 6], a.v[8 * x + 7], w.g[x].w);
        }
        return r;
    }
    static __device__ __forceinline__ void sub(Scores& a, const Slice& w) { a = sub3(a, w); }
    static __device__ __forceinline__ Scores seed(const float* hn, int q)
    {
        Scores r;
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            const float4 lo = *reinterpret_cast<const float4*>(hn + 64 * x + 8 * q);
            const float4 hi = *reinterpret_cast<const float4*>(hn + 64 * x + 8 * q + 4);
            r.v[8 * x + 0] = lo.x; r.v[8 * x + 1] = lo.y; r.v[8 * x + 2] = lo.z; r.v[8 * x + 3] = lo.w;
            r.v[8 * x + 4] = hi.x; r.v[8 * x + 5] = hi.y; r.v[8 * x + 6] = hi.z; r.v[8 * x + 7] = hi.w;
        }
        return r;
    }
    static __device__ __forceinline__ Scores worst()
    {
        Scores r;
#pragma unroll
        for (int j = 0; j < 16; ++j) r.v[j] = __int_as_float(0xff800000);  // negated scores: -inf
        return r;
    }
    static __device__ __forceinline__ void unpack(const Scores& s, float (&a)[16])
    {
#pragma unroll
        for (int j = 0; j < 16; ++j) a[j] = -s.v[j];
    }
    static __device__ __forceinline__ int lane_first(int q) { return 8 * q; }
    static __device__ __forceinline__ uint32_t neuron_of(int rr) { return (uint32_t)((rr >> 3) * 64 + (rr & 7)); }
    // a lane moves two 32-bit words (four neurons) of each row; M % 128 == 0 is guaranteed
    static __device__ __forceinline__ void stage(unsigned char* tab, const __half* __restrict__ W, int64_t M,
                                                 int64_t i0, const int32_t* __restrict__ slot_feat,
                                                 int n_rows, int warp, int lane, int warps)
    {
        uint32_t* tab_w = reinterpret_cast<uint32_t*>(tab);
        for (int row0 = warp * 4; row0 < n_rows; row0 += warps * 4) {
            uint32_t v[4][2];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int row = row0 + u;
                const int f = row < n_rows ? slot_feat[row] : -1;
                const uint32_t* src = reinterpret_cast<const uint32_t*>(W + (int64_t)(f >= 0 ? f : 0) * M + i0);
                v[u][0] = (f >= 0) ? __ldg(src + lane) : 0u;
                v[u][1] = (f >= 0) ? __ldg(src + 32 + lane) : 0u;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (row0 + u < n_rows) {
                    tab_w[(row0 + u) * 64 + lane] = v[u][0];
                    tab_w[(row0 + u) * 64 + 32 + lane] = v[u][1];
                }
        }
    }
};

// ---- pruning helpers ---------------------------------------------------------------------------
// Smallest score of the team's neurons, per 32-neuron group where the layout keeps the groups apart, else over
// the whole range.  fp32: every lane's x-th quad of neurons lies in group x.  Wide fp16 rows (HALF_GROUPS): a
// lane's c-th eight neurons lie in group 2 c + (q >> 2), so lanes 0..3 and lanes 4..7 of the team each reduce among
// themselves and then swap.  All lanes of the team call it together and all end up with all the minima.
template <typename L>
__device__ __forceinline__ void group_min(const typename L::Scores& s, uint32_t team_lanes, int q, float (&lo)[L::GROUPS])
{
    constexpr int R = L::R, G = L::GROUPS;
    float a[R];
    L::unpack(s, a);
    if constexpr (L::HALF_GROUPS) {
        constexpr int PER = 2 * R / G;  // neurons of the lane per group it has a share in
#pragma unroll
        for (int c = 0; c < G / 2; ++c) {
            float m = a[c * PER];
#pragma unroll
            for (int j = 1; j < PER; ++j) m = fminf(m, a[c * PER + j]);
            m = fminf(m, __shfl_xor_sync(team_lanes, m, 1));
            m = fminf(m, __shfl_xor_sync(team_lanes, m, 2));
            const float o = __shfl_xor_sync(team_lanes, m, 4);
            lo[2 * c] = (q & 4) ? o : m;
            lo[2 * c + 1] = (q & 4) ? m : o;
        }
    } else {
#pragma unroll
        for (int g = 0; g < G; ++g) {
            constexpr int PER = R / G;  // neurons of the lane per group
            float m = a[g * PER];
#pragma unroll
            for (int j = 1; j < PER; ++j) m = fminf(m, a[g * PER + j]);
            m = fminf(m, __shfl_xor_sync(team_lanes, m, 1));
            m = fminf(m, __shfl_xor_sync(team_lanes, m, 2));
            m = fminf(m, __shfl_xor_sync(team_lanes, m, 4));
            lo[g] = m;
        }
    }
}

// The bounds of one table entry (four floats: the largest weight of a feature in the four 32-neuron groups of a
// 128-neuron range) for a layout whose range starts at group g0 and spans SPAN groups: G = SPAN values, or their
// maximum (G = 1).  `e` points at the entry's first float.
template <int G, int SPAN>
__device__ __forceinline__ void entry_bounds(const float* __restrict__ e, int g0, float (&b)[G])
{
    float v[SPAN];
    if constexpr (SPAN == 4) {
        const float4 t = __ldg(reinterpret_cast<const float4*>(e));
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    } else if constexpr (SPAN == 2) {
        const float2 t = __ldg(reinterpret_cast<const float2*>(e + g0));
        v[0] = t.x; v[1] = t.y;
    } else {
        v[0] = __ldg(e + g0);
    }
    if constexpr (G == SPAN) {
#pragma unroll
        for (int g = 0; g < G; ++g) b[g] = v[g];
    } else {
        float m = v[0];
#pragma unroll
        for (int g = 1; g < SPAN; ++g) m = fmaxf(m, v[g]);
        b[0] = m;
    }
}

#define SOM_HOT(code) L::sub(acc, L::lds(tab_q + (code) * ROWB))
#define SOM_TAIL(code) L::ldg(row_ptr(w_q, (code), stride_b))

// L = storage layout (R = neurons per lane, 4 or 8; a team of 8 lanes covers T = 8*R neurons of
// one sample).  KEEP = 2 also keeps the second-best unit of every sample in keys2 (Algorithm 2 keeps the two
// best units); the candidate filter then tests against the second-best score.
// KEEP = 3 (first pass of the two-stage two-best search) keeps the third best as well, in keys3.
template <typename L, int THREADS, int KEEP, bool PRUNE>
__global__ void __launch_bounds__(THREADS, 1)
k_bmu_table(const typename L::Store* __restrict__ W, const float* __restrict__ hnorm, int64_t M,
            const int32_t* __restrict__ slot_feat, int n_rows,
            const uint4* __restrict__ slots, int64_t n_pad,
            u64* __restrict__ keys, u64* __restrict__ keys2, u64* __restrict__ keys3, int parts,
            int64_t part_len, int n_units, int n_whole, int* __restrict__ unit_counter,
            const int* __restrict__ gate, int gate_want, int feed_keep_arg, const float* __restrict__ range_max, int V,
            const int32_t* __restrict__ range_order)
{
    if (som_gated_off(gate, gate_want)) return;
    uint64_t feed_keep;  // L2 cache policy of the slot and key stream: "evict last" on small batches, else normal
    if (feed_keep_arg) asm("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(feed_keep));
    else asm("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(feed_keep));
    constexpr bool TOP2 = KEEP >= 2;
    constexpr int R = L::R;
    constexpr int T = L::T;
    constexpr int ROWB = L::ROWB;
    constexpr int CH = PRUNE ? PRUNE_CHUNK : CHUNK;  // samples a warp takes at a time
    // (pruning) the search rounds test again before their tail rows.  (With one bound per range instead of one per
    // 32-neuron group, as the wide fp16 layout first had it, this test lost 12 to 14 % at 64 x 64 and 128 x 128:
    // most samples passed it and their rows then started late.)
    constexpr bool SECOND_TEST = PRUNE;
    constexpr int WARPS = THREADS / 32;
    typedef typename L::Scores Scores;
    typedef typename L::Slice Slice;
    extern __shared__ __align__(16) unsigned char tab[];
    __shared__ int next_chunk;
    __shared__ int unit_sh;
    __shared__ __align__(16) float hn_sh[T];  // ||w||^2/2 of the range's neurons (+inf past M)
    // Warp-private ring of two stages; a stage holds the four slots (192 B) and four keys (32 B)
    // of one round.  The bytes of round r+2 are in flight in registers, round r+1 is being
    // stored, round r is being read: slot and key latency never sits on the critical path.
    __shared__ __align__(16) unsigned char ring_sh[WARPS * 2 * RING_STAGE];
    __shared__ unsigned char live_sh[PRUNE ? WARPS * CH : 16];  // (pruning) a warp's surviving samples of a chunk
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int q = lane & 7;
    const int sub = lane >> 3;
    const float inf = __int_as_float(0x7f800000);
    const unsigned char* tab_q = tab + q * 16;
    const uint32_t stride_b = (uint32_t)M * (uint32_t)sizeof(typename L::Store);  // launcher: M < 2^30

    // row n_rows of the table is all zeros: the target of padded hot codes
    for (int c = threadIdx.x; c < ROWB / 4; c += THREADS)
        reinterpret_cast<uint32_t*>(tab)[n_rows * (ROWB / 4) + c] = 0u;

    int cur_range = -1;
    // pruning: largest weight of every feature row in the live 128-neuron range (global), a copy for the table's
    // rows behind the table in shared memory, the lanes of this lane's team
    const float* rmax_range = nullptr;
    int rmax_g0 = 0;  // first 32-neuron group of this layout's range inside its 128-neuron range
    float* rmax_hot = reinterpret_cast<float*>(tab + (size_t)(n_rows + 1) * ROWB);
    const uint32_t team_lanes = 0xffu << (8 * sub);
    const unsigned char* w_q = reinterpret_cast<const unsigned char*>(W);
    uint32_t i_first = 0;
    for (;;) {
        // Units are claimed from a global counter in range-major order, so the blocks always
        // work on neighbouring units: the window of live neuron ranges (whose slabs must share
        // L2 with the slot stream) stays a few ranges wide however long the launch runs, and no
        // block is left with a queue of its own at the end.
        __syncthreads();  // every warp has left the previous unit
        if (threadIdx.x == 0) {
            unit_sh = atomicAdd(unit_counter, 1);
            next_chunk = 0;
        }
        __syncthreads();
        const int unit = unit_sh;
        if (unit >= n_units) break;
        // The last units of the launch are claimed in quarters, so that the blocks run out of
        // work within a quarter of a unit of each other.
        const int whole = unit < n_whole ? unit : n_whole + ((unit - n_whole) >> 2);
        const int range = whole / parts;  // (position in the launch's order of ranges)
        const int part = whole - range * parts;
        // With pruning the 128-neuron ranges are taken in the order of their smallest ||w||^2 (written by
        // som_norms): the ranges that are likeliest to hold a sample's best unit come first, its key is tight
        // sooner and more of the later ranges are skipped.  (The result does not depend on the order.)
        int64_t i0 = (int64_t)range * T;
        if (PRUNE && range_order) {
            constexpr int PER = 128 / T;  // ranges of this layout per 128 neurons
            i0 = (int64_t)range_order[range / PER] * 128 + (int64_t)(range % PER) * T;
        }
        if (range != cur_range) {
            // rows start on 16-byte boundaries when M * sizeof(weight) does (the range offset always does)
            if (((M * (int64_t)sizeof(typename L::Store)) & 15) == 0 && (reinterpret_cast<uintptr_t>(W) & 15) == 0 &&
                i0 + T <= M)
                stage_vec<L>(tab, W, M, i0, slot_feat, n_rows, warp, lane, WARPS);
            else
                L::stage(tab, W, M, i0, slot_feat, n_rows, warp, lane, WARPS);
            cur_range = range;
            // Lanes (or their upper group) past the last neuron still read valid addresses and
            // carry +inf scores, so they never beat a real neuron and need no predicate below.
            // With R = 8 the launcher guarantees M % 64 == 0, so a lane is all in or all out.
            const int64_t i_lane = i0 + L::lane_first(q);
            i_first = (uint32_t)i_lane;
            w_q = reinterpret_cast<const unsigned char*>(W + (i_lane < M ? i_lane : 0));
            if constexpr (PRUNE) {
                rmax_range = range_max + (i0 >> 7) * (int64_t)V * 4;  // (four floats per feature)
                rmax_g0 = (int)((i0 & 127) >> 5);
                for (int c = threadIdx.x; c <= n_rows; c += THREADS) {
                    const int f = c < n_rows ? slot_feat[c] : -1;
                    float hb[L::GROUPS];
#pragma unroll
                    for (int g = 0; g < L::GROUPS; ++g) hb[g] = 0.f;  // (the zero row and unused rows take nothing off)
                    if (f >= 0) entry_bounds<L::GROUPS, T / 32>(rmax_range + (int64_t)f * 4, rmax_g0, hb);
#pragma unroll
                    for (int g = 0; g < L::GROUPS; ++g) rmax_hot[c * L::GROUPS + g] = hb[g];
                }
            }
            for (int c = threadIdx.x; c < T; c += THREADS)
                hn_sh[c] = L::SEED_SIGN * ((i0 + c < M) ? hnorm[i0 + c] : inf);
        }
        __syncthreads();

        int64_t k_begin = (int64_t)part * part_len;
        int64_t k_end = min(n_pad, k_begin + part_len);  // a multiple of 4
        if (unit >= n_whole) {
            const int64_t quarter = ((part_len >> 2) + CH - 1) / CH * CH;
            k_begin += (int64_t)((unit - n_whole) & 3) * quarter;
            k_end = min(k_end, k_begin + quarter);
        }
        // full chunks first; the last 64 samples per warp of the unit go out in small chunks
        const int64_t unit_len = k_end > k_begin ? k_end - k_begin : 0;
        const int64_t tail_len = min(unit_len, (int64_t)WARPS * 2 * SMALL_CHUNK);
        const int n_big = (int)((unit_len - tail_len) / CH);
        const int64_t small_begin = k_begin + (int64_t)n_big * CH;
        const int n_chunks = n_big + (int)((k_end - small_begin + SMALL_CHUNK - 1) / SMALL_CHUNK);

        uint32_t curmask = 0;
        Scores base = L::seed(hn_sh, q);
        float base_lo[L::GROUPS];
#pragma unroll
        for (int g = 0; g < L::GROUPS; ++g) base_lo[g] = 0.f;
        if constexpr (PRUNE) group_min<L>(base, team_lanes, q, base_lo);
        for (;;) {
            int chunk = 0;
            if (lane == 0) chunk = atomicAdd(&next_chunk, 1);
            chunk = __shfl_sync(0xffffffffu, chunk, 0);
            if (chunk >= n_chunks) break;
            const int64_t w0 = chunk < n_big ? k_begin + (int64_t)chunk * CH
                                              : small_begin + (int64_t)(chunk - n_big) * SMALL_CHUNK;
            const int rounds = (int)(min(k_end, w0 + (chunk < n_big ? CH : SMALL_CHUNK)) - w0) >> 2;

            // Ring feed: lanes 0..11 carry the twelve 16-byte pieces of a round's four slots,
            // lanes 12..13 the two 16-byte pieces of its four keys.
            unsigned char* ring = ring_sh + warp * 2 * RING_STAGE;
            // the keys a round tests its candidates against: the best so far, or with TOP2 the
            // second (third) best so far (a stale, larger value only lets more candidates through)
            const u64* filter_keys = KEEP == 3 ? keys3 : (TOP2 ? keys2 : keys);
            const unsigned char* my_slot = ring + sub * 48;
            const unsigned char* my_key = ring + 192 + sub * 8;
            int rounds_b = rounds;  // rounds of the search loop below
            int n_live = 0;         // (pruning) survivors of the chunk
            unsigned char* live_list = live_sh + warp * CH;  // (pruning) positions in the chunk of the samples to search
            if constexpr (PRUNE) {
                // ---- pruning, before the search loop: find the samples of the chunk that this range can still
                //      matter to.  A sample survives unless (smallest prefix score of the range for its mask) minus
                //      (largest weights in this range of all its hot and tail rows) stays above its key, per group
                //      of 32 neurons, with a margin for the rounding of the sums.  Everything else is skipped for
                //      this range: a neuron of it would have lost the candidate comparison of the search loop, so
                //      the result is that of the full search bit for bit.  The survivors are then searched four to
                //      a round like any chunk; a round tests once more before it reads tail rows (see there).
                //      32 samples of the chunk at a time, the next 32's slots and keys already in flight:
                //      step 1, by teams as in the search loop: the prefix of the mask and its smallest scores (the
                //      samples are sorted by mask, so nearly always one mask serves all 32);
                //      step 2, a lane per sample: the bounds of its codes, the test, and the list of survivors in
                //      order.
                const int n_chunk = 4 * rounds;
                auto to_mask = [&](uint32_t mask) {  // the team's prefix scores and their minima for this mask
                    if (mask == curmask) return;
                    base = L::seed(hn_sh, q);
                    uint32_t mm = mask;
                    while (mm) {
                        const int b = __ffs(mm) - 1;
                        mm &= mm - 1;
                        L::sub(base, L::lds(tab_q + b * ROWB));
                    }
                    curmask = mask;
                    group_min<L>(base, team_lanes, q, base_lo);
                };
                // the slot and key of this lane's sample of step p (a step's loads are issued one step ahead)
                uint4 n0, n1, n2;
                u64 nkey;
                auto load_step = [&](int p) {
                    const int pos = lane + 32 * p;
                    n0 = make_uint4(SOM_SLOT_NT_OVERFLOW << 24, 0u, 0u, 0u);
                    n1 = n2 = make_uint4(0u, 0u, 0u, 0u);
                    nkey = 0;
                    if (pos < n_chunk) {
                        const uint4* sl = slots + (w0 + pos) * SLOT_Q;
                        n0 = __ldcg(sl);
                        n1 = __ldcg(sl + 1);
                        n2 = __ldcg(sl + 2);
                        nkey = __ldcg(filter_keys + w0 + pos);
                    }
                };
                load_step(0);
#pragma unroll
                for (int p = 0; p < CH / 32; ++p) {
                    if (32 * p >= n_chunk) break;  // (the same for every lane)
                    const int pos = lane + 32 * p;
                    const uint4 s0 = n0, s1 = n1, s2 = n2;
                    const u64 key0 = nkey;
                    if (p + 1 < CH / 32 && 32 * (p + 1) < n_chunk) load_step(p + 1);
                    const uint32_t hdr = s0.x;
                    float lo[L::GROUPS];
                    // Step 1.  The samples are sorted by mask, so nearly always the 32 of this step share one: then
                    // every team holds the same minima and every lane takes them as they are.
                    const uint32_t my_mask = hdr & 0xffffu;
                    const uint32_t first_mask = __shfl_sync(0xffffffffu, my_mask, 0);
                    if (__all_sync(0xffffffffu, pos >= n_chunk || my_mask == first_mask)) {
                        to_mask(first_mask);
#pragma unroll
                        for (int g = 0; g < L::GROUPS; ++g) lo[g] = base_lo[g];
                    } else {
#pragma unroll
                        for (int g = 0; g < L::GROUPS; ++g) lo[g] = 0.f;
#pragma unroll 1
                        for (int rr = 0; rr < 8; ++rr) {
                            const uint32_t h = __shfl_sync(0xffffffffu, hdr, 4 * rr + sub);
                            if (32 * p + 4 * rr >= n_chunk) break;  // (the same for every lane)
                            to_mask(h & 0xffffu);
                            // lane 4 * rr + s of the warp owns the sample that team s has just looked at
#pragma unroll
                            for (int g = 0; g < L::GROUPS; ++g) {
                                const float t = __shfl_sync(0xffffffffu, base_lo[g], 8 * (lane & 3));
                                if ((lane >> 2) == rr) lo[g] = t;
                            }
                        }
                    }
                    // Step 2.
                    const uint32_t nt = hdr >> 24, nh = (hdr >> 16) & 0xffu;
                    bool live = pos < n_chunk && nt != SOM_SLOT_NT_OVERFLOW;
                    if (live) {
                        const uint32_t hw[6] = {s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};  // hot codes 0..11
                        const uint32_t tw[5] = {s2.x, s2.y, s2.z, s2.w, s0.y};        // tail codes 0..9
                        float bnd[L::GROUPS];
#pragma unroll
                        for (int g = 0; g < L::GROUPS; ++g) bnd[g] = 0.f;
#pragma unroll
                        for (int j = 0; j < SOM_SLOT_MAX_HOT; ++j)
                            if ((uint32_t)j < nh) {
                                const float* hb = rmax_hot + ((j & 1) ? hi16(hw[j >> 1]) : lo16(hw[j >> 1])) * L::GROUPS;
#pragma unroll
                                for (int g = 0; g < L::GROUPS; ++g) bnd[g] += hb[g];
                            }
#pragma unroll
                        for (int j = 0; j < SOM_SLOT_MAX_TAIL; ++j)
                            if ((uint32_t)j < nt) {
                                float tb[L::GROUPS];
                                entry_bounds<L::GROUPS, T / 32>(
                                    rmax_range + (size_t)((j & 1) ? hi16(tw[j >> 1]) : lo16(tw[j >> 1])) * 4, rmax_g0, tb);
#pragma unroll
                                for (int g = 0; g < L::GROUPS; ++g) bnd[g] += tb[g];
                            }
                        const uint32_t cu = (uint32_t)(key0 >> 32);
                        const float cs = __uint_as_float((cu & 0x80000000u) ? (cu ^ 0x80000000u) : ~cu);
                        // the sample survives if some group of the range may still hold a candidate
                        // (an empty key decodes to NaN: the comparisons are false and the sample stays live)
                        live = false;
#pragma unroll
                        for (int g = 0; g < L::GROUPS; ++g)
                            live = live || !(lo[g] - bnd[g] > cs + 1e-5f * (fabsf(lo[g]) + fabsf(cs) + fabsf(bnd[g])));
                    }
                    const uint32_t votes = __ballot_sync(0xffffffffu, live);
                    if (live) live_list[n_live + __popc(votes & ((1u << lane) - 1u))] = (unsigned char)pos;
                    n_live += __popc(votes);
                }
                rounds_b = (n_live + 3) >> 2;
                __syncwarp();  // the list is written
                // whole rounds: the last survivor is repeated, so that the spare teams' loads have an address
                if (n_live > 0 && lane < 3 && n_live + lane < 4 * rounds_b) live_list[n_live + lane] = live_list[n_live - 1];
                __syncwarp();
            }
            // the search loop's feed: contiguous slots and keys, or (pruning) those of the survivors
            const uint4* feed;
            int feed_step = 0;
            bool feeder;
            unsigned char* my_store;
            auto feed_at = [&](int r) -> const uint4* {  // (pruning) where this lane's piece of round r lies
                const int rr = 4 * min(r, rounds_b - 1);  // (past the last round: that round's again, a valid address)
                if (lane < 12) return slots + (w0 + live_list[rr + lane / 3]) * SLOT_Q + lane % 3;
                return reinterpret_cast<const uint4*>(filter_keys + w0 + live_list[rr + (lane - 12)]);
            };
            if constexpr (PRUNE) {
                feeder = lane < 16;
                my_store = ring + (lane < 12 ? lane * 16 : 192 + (lane - 12) * 8);
                feed = nullptr;
            } else {
                feeder = lane < 14;
                my_store = ring + (lane < 12 ? lane * 16 : 192 + (lane - 12) * 16);
                feed = (lane < 12) ? slots + w0 * SLOT_Q + lane
                                   : reinterpret_cast<const uint4*>(filter_keys + w0) + (lane - 12);
                feed_step = (lane < 12) ? 4 * SLOT_Q : 2;  // uint4 per round
            }
            uint4 g = make_uint4(0u, 0u, 0u, 0u);
            // (a key lane of the pruning feed moves 8 bytes: the low half of g)
            auto ld_piece = [&](const uint4* p) -> uint4 {
                if (PRUNE && lane >= 12) {
                    const uint2 k = __ldcg(reinterpret_cast<const uint2*>(p));
                    return make_uint4(k.x, k.y, 0u, 0u);
                }
                return ld_feed(p, feed_keep);
            };
            auto st_piece = [&](unsigned char* dst, const uint4 v) {
                if (PRUNE && lane >= 12) *reinterpret_cast<uint2*>(dst) = make_uint2(v.x, v.y);
                else *reinterpret_cast<uint4*>(dst) = v;
            };
            __syncwarp();  // the previous chunk's (or phase A's) last reads of the ring are done
            if (rounds_b > 0 && feeder) {
                st_piece(my_store, ld_piece(PRUNE ? feed_at(0) : feed));  // round 0 -> stage 0
                g = ld_piece(PRUNE ? feed_at(1) : feed + feed_step);      // round 1, in flight
            }
            if (!PRUNE) feed += 2 * feed_step;
            __syncwarp();
            u64* pk = keys + w0 + sub;
            for (int r = 0; r < rounds_b; ++r) {
                const int st = (r & 1) * RING_STAGE;
                const uint4 s0 = *reinterpret_cast<const uint4*>(my_slot + st);
                const uint4 s1 = *reinterpret_cast<const uint4*>(my_slot + st + 16);
                const uint4 s2 = *reinterpret_cast<const uint4*>(my_slot + st + 32);
                const u64 key0 = *reinterpret_cast<const u64*>(my_key + st);
                if constexpr (PRUNE) pk = keys + w0 + live_list[4 * r + sub] + 4;  // (the combine below names pk - 4)
                // round r+1 goes into the other stage (its previous content, round r-1, was
                // consumed a round ago); round r+2 goes in flight.  The slot and key arrays
                // are padded, so the loads past the chunk's end stay in bounds.
                if (feeder) {
                    st_piece(my_store + (RING_STAGE - st), g);
                    g = ld_piece(PRUNE ? feed_at(r + 2) : feed);
                }
                if (!PRUNE) feed += feed_step;
                __syncwarp();
                const uint32_t hdr = s0.x;
                const uint32_t nt = hdr >> 24;  // SOM_SLOT_NT_OVERFLOW marks an overflow sample
                const uint32_t nh = (hdr >> 16) & 0xffu;
                const uint32_t mask = hdr & 0xffffu;
                const bool p0 = nt > 0, p1 = nt > 1, p2 = nt > 2, p3 = nt > 3;

                // ---- the first tail rows of this sample go in flight first ----------------------------
                Slice tr0, tr1, tr2, tr3;
                float tail_bound[L::GROUPS];  // (second test) this lane's share of the tail rows' bounds
#pragma unroll
                for (int g = 0; g < L::GROUPS; ++g) tail_bound[g] = 0.f;
                if constexpr (!SECOND_TEST) {
                    if (p0) tr0 = SOM_TAIL(lo16(s2.x));
                    if (p1) tr1 = SOM_TAIL(hi16(s2.x));
                    if constexpr (L::TAILS_AHEAD >= 3) {
                        if (p2) tr2 = SOM_TAIL(lo16(s2.y));
                    }
                    if constexpr (L::TAILS_AHEAD >= 4) {
                        if (p3) tr3 = SOM_TAIL(hi16(s2.y));
                    }
                } else {
                    // Second test (below, after the hot rows): lane q of the team fetches the bounds of tail rows
                    // q and q + 8; the rows themselves wait for the test.
                    const uint32_t w = (q >> 1) == 0 ? s2.x : ((q >> 1) == 1 ? s2.y : ((q >> 1) == 2 ? s2.z : s2.w));
                    if ((uint32_t)q < nt && nt <= (uint32_t)SOM_SLOT_MAX_TAIL)
                        entry_bounds<L::GROUPS, T / 32>(rmax_range + (size_t)((q & 1) ? hi16(w) : lo16(w)) * 4, rmax_g0,
                                                        tail_bound);
                    if ((uint32_t)q + 8u < nt && nt <= (uint32_t)SOM_SLOT_MAX_TAIL) {
                        float more[L::GROUPS];
                        entry_bounds<L::GROUPS, T / 32>(rmax_range + (size_t)((q & 1) ? hi16(s0.y) : lo16(s0.y)) * 4, rmax_g0,
                                                        more);
#pragma unroll
                        for (int g = 0; g < L::GROUPS; ++g) tail_bound[g] += more[g];
                    }
                }

                // ---- mask prefix ------------------------------------------------------------
                if (mask != curmask) {
                    base = L::seed(hn_sh, q);
                    uint32_t mm = mask;
                    while (mm) {
                        const int b = __ffs(mm) - 1;
                        mm &= mm - 1;
                        L::sub(base, L::lds(tab_q + b * ROWB));
                    }
                    curmask = mask;
                }

                // ---- hot rows: exactly max(nh over the warp, 1) steps; shorter lists are padded
                //      with the zero row, so a step carries no predicate.  The first step also
                //      moves the running score out of `base` (which the next sample may reuse).
                // (pruning: the last round of the survivors may be short; its spare teams, which were fed the last
                //  survivor again so that every load has a valid address, sit the round out)
                const bool spare = PRUNE && 4 * r + sub >= n_live;
                const uint32_t nh_max = __reduce_max_sync(0xffffffffu, spare ? 0u : nh);
                if (spare) continue;
                Scores acc = L::sub3(base, L::lds(tab_q + lo16(s0.z) * ROWB));
                switch (nh_max) {
                    case 12: SOM_HOT(hi16(s1.w));
                    case 11: SOM_HOT(lo16(s1.w));
                    case 10: SOM_HOT(hi16(s1.z));
                    case 9: SOM_HOT(lo16(s1.z));
                    case 8: SOM_HOT(hi16(s1.y));
                    case 7: SOM_HOT(lo16(s1.y));
                    case 6: SOM_HOT(hi16(s1.x));
                    case 5: SOM_HOT(lo16(s1.x));
                    case 4: SOM_HOT(hi16(s0.w));
                    case 3: SOM_HOT(lo16(s0.w));
                    case 2: SOM_HOT(hi16(s0.z));
                    default: break;
                }
                const uint32_t t45 = s2.z, t67 = s2.w;  // tail codes 4..7
                // ---- tail rows ------------------------------------------------------------------
                if constexpr (SECOND_TEST) {
                    // Second test, now that the scores hold the mask and hot rows exactly: if no neuron of the
                    // team can get under the sample's key even when every tail row takes its largest weight of
                    // the neuron's group off, the tail rows (mostly cold: few samples of a batch read a given
                    // row of this range) are not read at all.  Such a sample offers no candidate either way.
#pragma unroll
                    for (int g = 0; g < L::GROUPS; ++g) {
                        float t = tail_bound[g];
                        t += __shfl_xor_sync(team_lanes, t, 1);
                        t += __shfl_xor_sync(team_lanes, t, 2);
                        t += __shfl_xor_sync(team_lanes, t, 4);
                        tail_bound[g] = t;
                    }
                    const uint32_t cu2 = (uint32_t)(key0 >> 32);
                    const float cs2 = __uint_as_float((cu2 & 0x80000000u) ? (cu2 ^ 0x80000000u) : ~cu2);
                    bool may = false;
                    float sc[R];
                    L::unpack(acc, sc);
                    // (the lane's neurons group by group, as in group_min; an empty key decodes to NaN: the
                    //  comparison is false and the rows are read)
                    constexpr int SHARES = L::HALF_GROUPS ? L::GROUPS / 2 : L::GROUPS;
                    constexpr int PER = R / SHARES;
#pragma unroll
                    for (int c = 0; c < SHARES; ++c) {
                        float m = sc[c * PER];
#pragma unroll
                        for (int j = 1; j < PER; ++j) m = fminf(m, sc[c * PER + j]);
                        float tb;
                        if constexpr (L::HALF_GROUPS) tb = (q & 4) ? tail_bound[2 * c + 1] : tail_bound[2 * c];
                        else tb = tail_bound[c];
                        may = may || !(m - tb > cs2 + 1e-5f * (fabsf(m) + fabsf(cs2) + fabsf(tb)));
                    }
                    if (!__any_sync(team_lanes, may)) continue;
                    // A step of the warp waits for the slowest of its four teams: the rows are loaded
                    // as many at a time as the registers allow, not one after the other.
                    // (fp32 blocks of more than 640 threads have 80 registers: one row at a time)
                    constexpr int A = (sizeof(typename L::Store) == 4 && THREADS > 640) ? 1 : L::TAILS_AHEAD;
                    if (nt == SOM_SLOT_NT_OVERFLOW) {
                        acc = L::worst();  // (never a survivor; see the other branch)
                    } else {
                        const uint32_t tc[5] = {s2.x, s2.y, s2.z, s2.w, s0.y};
#pragma unroll
                        for (int b = 0; b < SOM_SLOT_MAX_TAIL; b += A) {
                            if (nt > (uint32_t)b) {
#pragma unroll
                                for (int j = b; j < b + A && j < SOM_SLOT_MAX_TAIL; ++j) {
                                    Slice& t = (j - b == 0) ? tr0 : ((j - b == 1) ? tr1 : ((j - b == 2) ? tr2 : tr3));
                                    if (nt > (uint32_t)j) t = SOM_TAIL((j & 1) ? hi16(tc[j >> 1]) : lo16(tc[j >> 1]));
                                }
#pragma unroll
                                for (int j = b; j < b + A && j < SOM_SLOT_MAX_TAIL; ++j) {
                                    Slice& t = (j - b == 0) ? tr0 : ((j - b == 1) ? tr1 : ((j - b == 2) ? tr2 : tr3));
                                    if (nt > (uint32_t)j) L::sub(acc, t);
                                }
                            }
                        }
                    }
                } else {
                if (p0) L::sub(acc, tr0);
                if (p1) L::sub(acc, tr1);
                if constexpr (L::TAILS_AHEAD >= 3) {
                    if (p2) L::sub(acc, tr2);
                } else {
                    if (p2) L::sub(acc, SOM_TAIL(lo16(s2.y)));
                }
                if constexpr (L::TAILS_AHEAD >= 4) {
                    if (p3) L::sub(acc, tr3);
                } else {
                    if (p3) L::sub(acc, SOM_TAIL(hi16(s2.y)));
                }
                if (nt > 4) {
                    if (nt != SOM_SLOT_NT_OVERFLOW) {
                        L::sub(acc, SOM_TAIL(lo16(t45)));
                        if (nt > 5) L::sub(acc, SOM_TAIL(hi16(t45)));
                        if (nt > 6) L::sub(acc, SOM_TAIL(lo16(t67)));
                        if (nt > 7) L::sub(acc, SOM_TAIL(hi16(t67)));
                        if (nt > 8) L::sub(acc, SOM_TAIL(lo16(s0.y)));
                        if (nt > 9) L::sub(acc, SOM_TAIL(hi16(s0.y)));
                    } else {
                        // rare: a sample that does not fit its slot (more than 12 hot or 10 tail
                        // features) is not searched here: its scores are made the worst possible,
                        // so that it offers no candidate; the direct-load kernel searches the
                        // list of such samples afterwards.  (Walking its row of the batch here,
                        // even out of line, cost the hot loop of every sample 15 to 20 %.)
                        acc = L::worst();
                    }
                }

                }

                // ---- lane-local argmin, rare atomic combine ------------------------------------
                float a[R];
                L::unpack(acc, a);
                float mn = fminf(fminf(a[0], a[1]), fminf(a[2], a[3]));
                if (R >= 8) mn = fminf(mn, fminf(fminf(a[4 % R], a[5 % R]), fminf(a[6 % R], a[7 % R])));
                if (R == 16) {
                    mn = fminf(mn, fminf(fminf(a[8 % R], a[9 % R]), fminf(a[10 % R], a[11 % R])));
                    mn = fminf(mn, fminf(fminf(a[12 % R], a[13 % R]), fminf(a[14 % R], a[15 % R])));
                }
                if constexpr (!PRUNE) pk += 4;
                const uint32_t cu = (uint32_t)(key0 >> 32);
                const float cs = __uint_as_float((cu & 0x80000000u) ? (cu ^ 0x80000000u) : ~cu);
                if (!(mn > cs)) {
                    int rr = R - 1;
#pragma unroll
                    for (int j = R - 2; j >= 0; --j)
                        if (a[j] == mn) rr = j;  // lowest neuron among the lane's minima
                    const uint32_t neuron = i_first + L::neuron_of(rr);
                    const u64 c1 = som_pack_key(mn, neuron);
                    if (!TOP2) {
                        atomicMin(pk - 4, c1);
                    } else {
                        // Two-key combine.  keys ends as the minimum of all candidates; every
                        // other candidate reaches keys2 exactly once, either directly (it did
                        // not beat the best of its time) or when a later, smaller candidate
                        // displaces it from keys, so keys2 ends as the second smallest.  Both
                        // are minima of fixed sets: order-independent, ties to the lower index.
                        // With KEEP = 3 the chain has one more level: what loses at keys2 goes
                        // on to keys3; the lane's second best (never the overall best) enters at
                        // keys2, its third best (never among the overall two best) at keys3.
                        u64* k1 = pk - 4;
                        u64* k2 = keys2 + (k1 - keys);
                        u64* k3 = KEEP == 3 ? keys3 + (k1 - keys) : nullptr;
                        const u64 old = atomicMin(k1, c1);
                        const u64 l1 = old > c1 ? old : c1;
                        const u64 old2 = atomicMin(k2, l1);
                        if (KEEP == 3) atomicMin(k3, old2 > l1 ? old2 : l1);
                        // the lane's second smallest score first; its index only if it can matter
                        float m2 = inf;
#pragma unroll
                        for (int j = 0; j < R; ++j) m2 = fminf(m2, j == rr ? inf : a[j]);
                        if (!(m2 > cs)) {
                            int r2 = rr == R - 1 ? R - 2 : R - 1;
#pragma unroll
                            for (int j = R - 1; j >= 0; --j)
                                if (j != rr && a[j] == m2) r2 = j;  // lowest such neuron
                            const u64 c2 = som_pack_key(m2, i_first + L::neuron_of(r2));
                            const u64 o2 = atomicMin(k2, c2);
                            if (KEEP == 3) {
                                atomicMin(k3, o2 > c2 ? o2 : c2);
                                float m3 = inf;
                                int r3 = 0;
#pragma unroll
                                for (int j = R - 1; j >= 0; --j)
                                    if (j != rr && j != r2 && a[j] <= m3) { m3 = a[j]; r3 = j; }
                                if (!(m3 > cs)) atomicMin(k3, som_pack_key(m3, i_first + L::neuron_of(r3)));
                            }
                        }
                    }
                }
            }
        }
    }
}

template <typename ST>
__global__ void k_finalize_sorted(const ST* __restrict__ W, const double* __restrict__ norm64, int64_t M, int V,
                                  const int32_t* __restrict__ indptr, const int32_t* __restrict__ indices,
                                  int64_t n, const uint32_t* __restrict__ order,
                                  const u64* __restrict__ keys, int32_t* __restrict__ bmu,
                                  float* __restrict__ dist, const int* __restrict__ gate, int gate_want)
{
    if (som_gated_off(gate, gate_want)) return;
    const int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= n) return;
    const uint32_t s = order[k];
    const uint32_t idx = (uint32_t)(keys[k] & 0xffffffffull);
    if (idx >= M) {  // only a second-best key can be empty: fewer than two neurons
        bmu[s] = -1;
        dist[s] = __int_as_float(0x7f800000);
        return;
    }
    const int beg = indptr[s];
    const int end = indptr[s + 1];
    double dot = 0.0;
    for (int j = beg; j < end; ++j) {
        const int v = indices[j];
        if ((unsigned)v < (unsigned)V) dot += (double)som_weight(W + (int64_t)v * M + idx);  // (the plan skipped the others)
    }
    bmu[s] = (int32_t)idx;
    dist[s] = (float)((double)(end - beg) - 2.0 * dot + norm64[idx]);
}

template <typename L, int THREADS, int KEEP>
int launch_table(som_handle* h, const void* codebook_v, const int32_t* indptr, const int32_t* indices,
                 int64_t n_real, char* head, char* ws, const SomPlanBuffers& b, int n_hot, size_t smem,
                 cudaStream_t st)
{
    constexpr int T = L::T;
    const int64_t n = (n_real + 3) / 4 * 4;  // the plan pads the slot array to whole rounds
    const int n_ranges = (int)((h->M + T - 1) / T);
    // Pruning by range maxima, when som_norms has written them.  Measured against the search that reads every row
    // (fp32 storage, the benchmark's batches): 64 x 64 (32 ranges) 5.28 -> 3.96 ms, 128 x 128 78.2 -> 50.0 ms,
    // 512 x 512 329 -> 113 ms, 1024 x 1024 368 -> 130 ms; the share of the (sample, range) pairs it skips grows
    // with the number of ranges, because a sample's key tightens as the ranges go by.  Below 32 ranges it is off.
    bool prune = false;
    if constexpr (L::CAN_PRUNE)
        prune = som_table_prunes(h);
    // (the maxima are those of the handle's own codebook: the first pass of the two-stage search, which reads
    //  the fp16 copy of an fp32 codebook, does not prune; with the copy's rounding allowed for it measured 3 %
    //  slower at 512 x 512: it tests against the second-best key, which skips less)
    if (codebook_v != static_cast<const void*>(h->W) && codebook_v != static_cast<const void*>(h->Wh)) prune = false;
    int parts = h->opt_parts > 0 ? (int)h->opt_parts : som_table_default_parts(n, T, L::ROWB);
    // (with pruning a unit's search is three times shorter on the large maps but its table costs the same: on a
    //  250k-sample batch 16 parts instead of 44 measure 4 % faster at 512 x 512 and 1024 x 1024; the small maps,
    //  whose units are few, keep theirs)
    if (prune && h->opt_parts <= 0 && L::ROWB >= 512 && n >= 200000 && n < 600000 && n_ranges >= 1024) parts = 16;
    if ((int64_t)parts * 1024 > n) parts = (int)(n / 1024);
    if (parts < 1) parts = 1;
    int64_t part_len = (n + parts - 1) / parts;
    part_len = (part_len + CHUNK - 1) / CHUNK * CHUNK;
    parts = (int)((n + part_len - 1) / part_len);
    const int64_t n_units64 = (int64_t)n_ranges * parts;
    if (n_units64 > 0x7fffffff) return SOM_ERR_UNSUPPORTED;
    const int grid = n_units64 < h->sm_count ? (int)n_units64 : h->sm_count;
    // the last `grid` units are claimed as quarters (see the kernel)
    const int n_split = (n_units64 >= 4 * (int64_t)grid && part_len >= 16 * CHUNK) ? grid : 0;
    const int n_whole = (int)n_units64 - n_split;
    if (n_units64 + 3 * (int64_t)n_split > 0x7fffffff) return SOM_ERR_UNSUPPORTED;
    const int n_units = n_whole + 4 * n_split;
    const typename L::Store* codebook = reinterpret_cast<const typename L::Store*>(codebook_v);
    const int feed_keep = h->opt_feed_keep == 1 || (h->opt_feed_keep == 0 && n * 56 <= ((int64_t)24 << 20));
    if (prune) smem += ((size_t)(SOM_PLAN_MASK_FEATURES + n_hot + 1) * L::GROUPS * sizeof(float) + 15) / 16 * 16;  // the table rows' maxima
    auto launch = [&](auto kern) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        kern<<<grid, THREADS, smem, st>>>(codebook, h->hnorm, h->M,
                                          reinterpret_cast<const int32_t*>(head + b.slot_feat),
                                          SOM_PLAN_MASK_FEATURES + n_hot,
                                          reinterpret_cast<const uint4*>(ws + b.slots),
                                          n,
                                          reinterpret_cast<u64*>(ws + b.keys),
                                          KEEP >= 2 ? reinterpret_cast<u64*>(ws + b.keys2) : nullptr,
                                          KEEP == 3 ? reinterpret_cast<u64*>(ws + b.keys3) : nullptr, parts, part_len,
                                          n_units, n_whole,
                                          reinterpret_cast<int*>(head + b.n_slots) + 3, h->gate, h->gate_want,
                                          feed_keep, prune ? h->range_max : nullptr, (int)h->V, prune ? h->range_order : nullptr);
        return cudaGetLastError();
    };
    if constexpr (L::CAN_PRUNE) {
        if (prune) SOM_CK(h, launch(k_bmu_table<L, THREADS, KEEP, true>));
        else SOM_CK(h, launch(k_bmu_table<L, THREADS, KEEP, false>));
    } else {
        SOM_CK(h, launch(k_bmu_table<L, THREADS, KEEP, false>));
    }
    SOM_CK(h, cudaGetLastError());
    h->launches += 1;
    return SOM_OK;
}

}  // namespace

SomTableGeom som_table_geometry(const som_handle* h, bool shadow)
{
    const bool f16 = h->Wh != nullptr || shadow;  // the layout of the codebook this launch reads
    SomTableGeom g;
    // 8 neurons per lane (half as many rounds for the same work) whenever the neuron count is
    // a multiple of the 64-neuron range it needs; 640 threads leave it 96 registers, the
    // measured optimum between resident warps and spills
    // (an fp16-stored codebook has the 8-neuron layout only; som_table_usable checks M % 64)
    g.R = (f16 || (h->opt_r != 4 && h->M % 64 == 0)) ? 8 : 4;
    if (f16 && h->opt_r != 8 && h->M % 128 == 0) g.R = 16;  // wide fp16 layout wherever it divides M
    // fp32 storage: 16 neurons per lane (128-neuron ranges, 512-byte rows) wherever 128 divides M: half the
    // per-round bookkeeping and half the row visits per add (3 to 5 % faster; 11 % on the largest map,
    // where every row visit is another 2 MB page)
    // (not with the two-stage search, whose exact pass shares the plan of the fp16 first pass: 720 hot rows)
    if (!f16 && h->opt_r != 4 && h->opt_r != 8 && h->M % 128 == 0 && h->opt_two_stage != 1) g.R = 16;
    g.T = 8 * g.R;
    const int row_bytes = g.T * (f16 ? 2 : 4);
    // (the fp16 layout holds half as many row registers: 896 threads at 72 registers measured best)
    // fp32, 16 neurons per lane: where the launch prunes (launch_table) its rounds seldom read tail rows, so they
    // are loaded one at a time, the kernel fits 80 registers and 24 warps hide more of its latency than 16 do:
    // 768 threads measure 7 % faster than 512 (512 x 512: 103 -> 96 ms).  The search that reads every row keeps
    // three rows in flight and 512 threads (576 and more spill and measure slower).
    const bool prunes = !shadow && som_table_prunes(h);
    const int def_threads = f16 ? (g.R == 16 ? 512 : 896) : (g.R == 16 ? (prunes ? 768 : 512) : (g.R == 8 ? 640 : 1024));
    g.threads = (h->opt_threads == 512 || h->opt_threads == 576 || h->opt_threads == 640 || h->opt_threads == 768 ||
                 h->opt_threads == 896 || h->opt_threads == 1024)
                    ? (int)h->opt_threads : def_threads;
    // 227 KB per block, minus the static shared memory (slot rings, norms) of the kernel
    int max_rows = (int)((227 * 1024 - 16 * 1024) / row_bytes) - SOM_PLAN_MASK_FEATURES - 1;
    // Defaults keep dynamic + static shared memory (and the KB that the system reserves per block) under 196 KB: one
    // step more and the SM's carve-out leaves 28 KB instead of 60 KB of L1, which costs 9 to 12 % (measured at
    // every map size).  The wide layouts count in the bounds of the table's rows that a pruning launch keeps behind
    // the table (16 bytes per row) and the rings of a 768-thread block: 334 rows of 512 bytes and 680 of 256
    // bytes (fp16) are the most that stay below the step; the defaults leave a KB of room.  (The fp16 copy that
    // the two-stage search reads first does not prune, and its plan is also that of the exact pass: 720 rows.)
    int want = h->opt_hot_rows > 0 ? (int)h->opt_hot_rows
                                   : (row_bytes == 128 ? (f16 ? 1456 : 1376)
                                                       : (row_bytes == 512 ? 330 : (f16 && g.R == 16 && !shadow ? 676 : 720)));
    if (want > max_rows) want = max_rows;
    g.n_hot = want;
    g.row_bytes = row_bytes;
    g.smem = (size_t)(SOM_PLAN_MASK_FEATURES + g.n_hot + 1) * row_bytes;  // + the zero row
    return g;
}

template <int KEEP>
static int launch_table_any(som_handle* h, bool shadow, const int32_t* indptr, const int32_t* indices, int64_t n,
                            char* head, char* ws, const SomPlanBuffers& b, int n_hot, cudaStream_t st)
{
    const SomTableGeom g = som_table_geometry(h, shadow);
    const bool f16 = h->Wh != nullptr || shadow;
    const void* cb = shadow ? (const void*)h->shadow : (h->Wh ? (const void*)h->Wh : (const void*)h->W);
#define SOM_TABLE(L_, THREADS_) return launch_table<L_, THREADS_, KEEP>(h, cb, indptr, indices, n, head, ws, b, n_hot, g.smem, st)
    if (f16 && g.R == 16) {
        if (KEEP < 3 && g.threads == 768) SOM_TABLE(LayF16W, 768);
        if (KEEP < 3 && g.threads == 640) SOM_TABLE(LayF16W, 640);
        SOM_TABLE(LayF16W, 512);
    }
    if constexpr (KEEP == 3) return SOM_ERR_UNSUPPORTED;  // three best: the wide fp16 layout only
    else {
    if (f16) {
        if (g.threads == 1024) SOM_TABLE(LayF16, 1024);
        if (g.threads == 896) SOM_TABLE(LayF16, 896);
        if (g.threads == 768) SOM_TABLE(LayF16, 768);
        if (g.threads == 640) SOM_TABLE(LayF16, 640);
        SOM_TABLE(LayF16, 512);
    }
    if (g.R == 16) {
        if (g.threads == 768) SOM_TABLE(LayF32<16>, 768);
        if (g.threads == 576) SOM_TABLE(LayF32<16>, 576);
        SOM_TABLE(LayF32<16>, 512);
    }
    if (g.R == 8) {
        if (g.threads == 1024) SOM_TABLE(LayF32<8>, 1024);
        if (g.threads == 896) SOM_TABLE(LayF32<8>, 896);
        if (g.threads == 768) SOM_TABLE(LayF32<8>, 768);
        if (g.threads == 640) SOM_TABLE(LayF32<8>, 640);
        SOM_TABLE(LayF32<8>, 512);
    }
    if (g.threads == 1024) SOM_TABLE(LayF32<4>, 1024);
    if (g.threads == 896) SOM_TABLE(LayF32<4>, 896);
    if (g.threads == 768) SOM_TABLE(LayF32<4>, 768);
    if (g.threads == 640) SOM_TABLE(LayF32<4>, 640);
    SOM_TABLE(LayF32<4>, 512);
    }
#undef SOM_TABLE
}

int som_launch_bmu_table(som_handle* h, bool shadow, const int32_t* indptr, const int32_t* indices, int64_t n,
                         char* head, char* ws, const SomPlanBuffers& b, int n_hot, int keep, cudaStream_t st)
{
    if (keep == 3) return launch_table_any<3>(h, shadow, indptr, indices, n, head, ws, b, n_hot, st);
    return keep == 2 ? launch_table_any<2>(h, shadow, indptr, indices, n, head, ws, b, n_hot, st)
                     : launch_table_any<1>(h, shadow, indptr, indices, n, head, ws, b, n_hot, st);
}

// ---- two-stage search: certification of the first pass ----------------------------------------
// The first pass ranked the neurons by fp32 sums of the fp16-rounded weights.  For a sample with
// k active features such a score differs from the fp32 score of the exact weights by at most
//   k * max(wmax * 2^-11, 2^-25)  (rounding of each weight to fp16, round to nearest; the second
//                                  term covers fp16's subnormal range)
//   + 2 * (k + 2) * 2^-24 * B     (fp32 summation, either path; B bounds every partial sum).
// When no weight is negative (the norm pass records it) the first term tightens to 2^-11 times the
// unit's own dot product with the sample, i.e. ||w||^2/2 minus its score, plus k * 2^-25; for a unit
// that is not named, to 2^-11 * (max ||w||^2/2 - its score), largest at the lowest score it can have.
// When the two best first-pass scores are further apart than the bounds of the best unit and of
// any other unit together, the best unit of the exact weights is the first pass's best unit.  Such
// samples are finalised here (distance recomputed in fp64 from the fp32 weights, as always); the
// others are listed for an exact fp32 search.
namespace {
__device__ __forceinline__ float score_of_key(u64 key)
{
    const uint32_t cu = (uint32_t)(key >> 32);
    return __uint_as_float((cu & 0x80000000u) ? (cu ^ 0x80000000u) : ~cu);
}

// SECOND: the two-best search.  With the three best first-pass scores s1 <= s2 <= s3, the two
// first-pass winners are the two best units of the exact weights, in that order, when both gaps
// exceed the bounds of their two sides (s3 - s2: no third unit can overtake either; s2 - s1: they
// cannot swap).
// COUNT_ONLY: the probe of the two-stage search; nothing is finalised or listed, the samples that fail the
// certificate are only counted.
template <bool SECOND, bool COUNT_ONLY>
__global__ void k_certify(const float* __restrict__ W, const double* __restrict__ norm64, int64_t M, int V,
                          const int32_t* __restrict__ indptr, const int32_t* __restrict__ indices, int64_t n,
                          const uint4* __restrict__ slots, const uint32_t* __restrict__ order,
                          const u64* __restrict__ keys, const u64* __restrict__ keys2, const u64* __restrict__ keys3,
                          const unsigned int* __restrict__ wmax_bits, const float* __restrict__ hnorm,
                          int32_t* __restrict__ bmu, float* __restrict__ dist,
                          int32_t* __restrict__ bmu2, float* __restrict__ dist2,
                          int32_t* __restrict__ uncertain, uint4* __restrict__ slots2,
                          int* __restrict__ n_uncertain, const int* __restrict__ gate, int gate_want)
{
    if (som_gated_off(gate, gate_want)) return;
    __shared__ int warp_count[8];
    __shared__ int block_base;
    const int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    bool flag = false;
    uint32_t s = 0;
    if (k < n) {
        s = order[k];
        const u64 k1 = keys[k], k2 = keys2[k];
        const int beg = indptr[s];
        const int end = indptr[s + 1];
        const float wmax = __uint_as_float(wmax_bits[0]);
        const bool has_negative = wmax_bits[SOM_AUX_HAS_NEGATIVE] != 0u;
        const float hmax = __uint_as_float(wmax_bits[SOM_AUX_HMAX]);
        const float s1 = score_of_key(k1), s2 = score_of_key(k2);
        const uint32_t i1 = (uint32_t)(k1 & 0xffffffffull), i2 = (uint32_t)(k2 & 0xffffffffull);
        const float cnt = (float)(end - beg);
        float top = fmaxf(fabsf(s1), fabsf(s2));
        float s3 = 0.f;
        if (SECOND) {
            s3 = score_of_key(keys3[k]);
            top = fmaxf(top, fabsf(s3));
        }
        // fp32 summation of either pass: 2 (k + 2) 2^-24 B, B a bound on every partial sum
        const float fsum = 2.f * (cnt + 2.f) * 5.9604645e-8f * (top + 2.f * cnt * wmax);
        // rounding of the weights to fp16: at most 2^-11 relative in fp16's normal range, at most
        // 2^-25 absolute below it
        float e1, e2, eo;  // error bounds of the first, the second and of any other unit's score
        if (!has_negative && i1 < M && i2 < M) {
            // All weights >= 0: a unit's rounding errors add up to at most 2^-11 times its dot
            // product, which is ||w||^2/2 minus its score (first-pass values, hence the margins).
            // For a unit that is not named its dot product is at most hmax minus the lowest score
            // it can have; the bound shrinks as the score grows, so that lowest score is the worst case.
            const float c = 4.8828125e-4f * 1.002f;
            const float sub = cnt * 2.9802322e-8f;
            e1 = c * fmaxf(hnorm[i1] - s1 + fsum, 0.f) + sub + fsum;
            e2 = c * fmaxf(hnorm[i2] - s2 + fsum, 0.f) + sub + fsum;
            eo = c * fmaxf(hmax - (SECOND ? s3 : s2) + fsum, 0.f) + sub + fsum;
        } else {
            e1 = e2 = eo = cnt * fmaxf(wmax * 4.8828125e-4f, 2.9802322e-8f) * 1.0001f + fsum;
        }
        // comparisons are false for NaN or an empty key
        bool certain;
        if (!SECOND) certain = (s2 - s1) > e1 + eo;
        else certain = (s2 - s1) > e1 + e2 && (s3 - s2) > e2 + eo;  // (a map of two units has no third: exact pass)
        flag = !certain;
        if (certain && !COUNT_ONLY) {
            const uint32_t idx = (uint32_t)(k1 & 0xffffffffull);
            const uint32_t idx2 = (uint32_t)(k2 & 0xffffffffull);
            double dot = 0.0, dot2 = 0.0;
            for (int j = beg; j < end; ++j) {
                const int v = indices[j];
                if ((unsigned)v >= (unsigned)V) continue;  // (the plan skipped it too)
                const float* row = W + (int64_t)v * M;
                dot += (double)__ldg(row + idx);
                if (SECOND) dot2 += (double)__ldg(row + idx2);
            }
            bmu[s] = (int32_t)idx;
            dist[s] = (float)((double)(end - beg) - 2.0 * dot + norm64[idx]);
            if (SECOND) {
                bmu2[s] = (int32_t)idx2;
                dist2[s] = (float)((double)(end - beg) - 2.0 * dot2 + norm64[idx2]);
            }
        }
    }
    // The uncertain samples of a block keep their (mask-sorted) order: their ids and their
    // slots are compacted to one contiguous run of the lists, so that the exact pass can run
    // the row-table kernel on the same plan.
    const unsigned int votes = __ballot_sync(0xffffffffu, flag);
    if (COUNT_ONLY) {
        if (lane == 0 && votes) atomicAdd(n_uncertain, __popc(votes));
        return;
    }
    if (lane == 0) warp_count[warp] = __popc(votes);
    __syncthreads();
    if (threadIdx.x == 0) {
        int total = 0;
        for (int w = 0; w < 8; ++w) { const int c = warp_count[w]; warp_count[w] = total; total += c; }
        block_base = total ? atomicAdd(n_uncertain, total) : 0;
    }
    __syncthreads();
    if (flag) {
        const int pos = block_base + warp_count[warp] + __popc(votes & ((1u << lane) - 1u));
        uncertain[pos] = (int32_t)s;
#pragma unroll
        for (int x = 0; x < SLOT_Q; ++x) slots2[(int64_t)pos * SLOT_Q + x] = slots[k * SLOT_Q + x];
    }
}
}  // namespace

int som_launch_certify(som_handle* h, const int32_t* indptr, const int32_t* indices, int64_t n, char* ws,
                       const SomPlanBuffers& b, bool second, bool count_only, int32_t* bmu, float* dist,
                       int32_t* bmu2, float* dist2, int32_t* uncertain, int* n_uncertain, cudaStream_t st)
{
    const int64_t blocks = (n + 255) / 256;
    const uint4* slots = reinterpret_cast<const uint4*>(ws + b.slots);
    const uint32_t* order = reinterpret_cast<const uint32_t*>(ws + b.order);
    const u64* keys = reinterpret_cast<const u64*>(ws + b.keys);
    const u64* keys2 = reinterpret_cast<const u64*>(ws + b.keys2);
    const u64* keys3 = second ? reinterpret_cast<const u64*>(ws + b.keys3) : nullptr;
    uint4* slots2 = reinterpret_cast<uint4*>(ws + b.slots2);
#define SOM_CERTIFY(SECOND_, COUNT_)                                                                            \
    k_certify<SECOND_, COUNT_><<<(unsigned)blocks, 256, 0, st>>>(h->W, h->norm64, h->M, h->V, indptr, indices, n, slots, \
                                                                 order, keys, keys2, keys3, h->wmax_bits, h->hnorm, bmu,  \
                                                                 dist, bmu2, dist2, uncertain, slots2, n_uncertain, \
                                                                 h->gate, h->gate_want)
    if (second && count_only) SOM_CERTIFY(true, true);
    else if (second) SOM_CERTIFY(true, false);
    else if (count_only) SOM_CERTIFY(false, true);
    else SOM_CERTIFY(false, false);
#undef SOM_CERTIFY
    SOM_CK(h, cudaGetLastError());
    h->launches += 1;
    return SOM_OK;
}

// Probe of the two-stage search: the slot of every SOM_PROBE_STRIDE-th sample (by sample index) goes to
// position index / SOM_PROBE_STRIDE of a second slot array.
namespace {
__global__ void k_probe_gather(const uint4* __restrict__ slots, const uint32_t* __restrict__ order, int64_t n,
                               uint4* __restrict__ probe, uint32_t* __restrict__ probe_order,
                               const int* __restrict__ gate, int gate_want)
{
    if (som_gated_off(gate, gate_want)) return;
    const int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= n) return;
    const uint32_t s = order[k];
    if (s % SOM_PROBE_STRIDE) return;
    const int64_t pos = s / SOM_PROBE_STRIDE;
    probe_order[pos] = s;
#pragma unroll
    for (int x = 0; x < SLOT_Q; ++x) probe[pos * SLOT_Q + x] = slots[k * SLOT_Q + x];
}
}  // namespace

int som_launch_probe_gather(som_handle* h, int64_t n, char* ws, const SomPlanBuffers& b, cudaStream_t st)
{
    const int64_t blocks = (n + 255) / 256;
    // (the probe's slots go to slots2, their sample indices to the uncertain list, which is free until
    //  the certificate of the full batch fills it)
    k_probe_gather<<<(unsigned)blocks, 256, 0, st>>>(reinterpret_cast<const uint4*>(ws + b.slots),
                                                     reinterpret_cast<const uint32_t*>(ws + b.order), n,
                                                     reinterpret_cast<uint4*>(ws + b.slots2),
                                                     reinterpret_cast<uint32_t*>(ws + b.uncertain), h->gate, h->gate_want);
    SOM_CK(h, cudaGetLastError());
    h->launches += 1;
    return SOM_OK;
}

// The two-stage search's own choice, made on the device: with the row-table kernel chosen (gate word 1),
// the batch takes the two-stage search (gate word 2) unless its probe failed the certificate for more than
// a fifth of the probed samples.  *report receives what som_last_uncertain is to say for a batch that takes the
// plain search (all its samples), else -1 (the certificate's own count follows later).
namespace {
__global__ void k_two_stage_decide(int* __restrict__ choice, const int* __restrict__ probe_uncertain, int n_probe,
                                   int64_t n, int* __restrict__ counters_to_clear, int* __restrict__ report)
{
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    int r = -1;
    if (*choice >= 1) {  // (2 is what an earlier search of the same plan left)
        const bool plain = n_probe > 0 && (int64_t)(*probe_uncertain) * 5 > (int64_t)n_probe;
        *choice = plain ? 1 : 2;
        if (plain) r = (int)n;
    } else if (*choice == 0) {
        r = 0;
    }
    *report = r;
    counters_to_clear[0] = 0;  // the probe's uncertain count: the full batch's certificate starts from zero
}
}  // namespace

int som_launch_two_stage_decide(som_handle* h, char* head, const SomPlanBuffers& b, int n_probe, int64_t n,
                                cudaStream_t st)
{
    int* counters = reinterpret_cast<int*>(head + b.n_slots);
    k_two_stage_decide<<<1, 32, 0, st>>>(counters + SOM_PLAN_USE_TABLE, counters + SOM_PLAN_UNCERTAIN, n_probe, n,
                                         counters + SOM_PLAN_UNCERTAIN, counters + SOM_PLAN_REPORT);
    SOM_CK(h, cudaGetLastError());
    h->launches += 1;
    return SOM_OK;
}

int som_launch_finalize_sorted(som_handle* h, const int32_t* indptr, const int32_t* indices, int64_t n,
                               char* ws, const SomPlanBuffers& b, bool second, int32_t* bmu, float* dist,
                               cudaStream_t st)
{
    const int64_t blocks = (n + 255) / 256;
    const uint32_t* order = reinterpret_cast<const uint32_t*>(ws + b.order);
    const u64* keys = reinterpret_cast<const u64*>(ws + (second ? b.keys2 : b.keys));
    if (h->Wh)
        k_finalize_sorted<__half><<<(unsigned)blocks, 256, 0, st>>>(h->Wh, h->norm64, h->M, h->V, indptr, indices, n,
                                                                    order, keys, bmu, dist, h->gate, h->gate_want);
    else
        k_finalize_sorted<float><<<(unsigned)blocks, 256, 0, st>>>(h->W, h->norm64, h->M, h->V, indptr, indices, n,
                                                                   order, keys, bmu, dist, h->gate, h->gate_want);
    SOM_CK(h, cudaGetLastError());
    h->launches += 1;
    return SOM_OK;
}
