// Densified hot-feature tile on the 5th-generation tensor cores (tcgen05): a measured probe.
//
// The fused search is a gather-accumulate (Section 3.3 of the paper), bound on this GPU by the bytes
// every executed add pulls through the SM's load/store pipe.  For the batch's H most frequent
// features the gather can be written as a small dense contraction instead: a tile of 128 samples
// becomes a 0/1 matrix A [128 x H] (one row per sample, a one where the sample has the feature),
// the rows W[v, i0..i0+64) of those features a matrix B [H x 64], and A x B is the samples' partial
// dot products with 64 neurons.  This file runs exactly that piece on tcgen05.mma, with everything
// the fused kernel would have to do around it, so that its cost can be set against the shared-memory
// reads it replaces:
//   * builder warps expand each sample's H-bit membership word into its fp16 row of A in shared
//     memory (K-major, no swizzle: 8 x 16-byte core matrices);
//   * one thread issues the MMAs of a tile: fp32 weights enter as TERMS fp16 terms (1 = rounded to
//     fp16; 2 = hi + lo, |w - hi - lo| <= 2^-22 |w|), the same A tile against each term, plus one
//     16-wide K step that adds the seed ||w||^2 / 2 (three fp16 terms, A columns of ones); B is
//     negated by the instruction descriptor, so the accumulator holds the partial SCORE
//     ||w||^2/2 - sum of the dense rows, in fp32, in tensor memory (128 lanes x 64 columns);
//   * consumer warps drain the accumulator with tcgen05.ld (16 lanes x 256 bits: four threads per
//     sample), optionally redistribute it by shuffles to the eight-threads-per-sample layout that the
//     row-table kernel's conflict-free shared-memory reads need, and reduce it.
// A tiles and accumulators are double-buffered; the stages hand over through mbarriers.  Every wait
// is bounded: a wait that gives up sets a status word and every role leaves its loop.
#include "som_internal.cuh"

namespace {

constexpr int TP_NEURONS = 64;            // N of the MMA = neurons of a range
constexpr int TP_SAMPLES = 128;           // M of the MMA = samples of a tile
constexpr int TP_BUILD_WARPS = 4;
constexpr int TP_DRAIN_WARPS = 4;
constexpr int TP_THREADS = 32 * (1 + TP_BUILD_WARPS + TP_DRAIN_WARPS);
constexpr long long TP_WAIT_CYCLES = 400000000ll;  // about 0.2 s: far beyond any legitimate wait

__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// Waits for the phase with the given parity to complete; gives up after TP_WAIT_CYCLES or when another
// thread has raised *abort.  Returns false when it gave up (and raises *abort itself).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag)
{
    const long long t0 = clock64();
    for (;;) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(smem_u32(bar)), "r"(parity)
            : "memory");
        if (done) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > TP_WAIT_CYCLES) {
            *abort_flag = 1;
            return false;
        }
    }
}

// shared-memory matrix descriptor, K-major, no swizzle: rows of a core matrix 16 bytes apart,
// groups of 8 rows `sbo` bytes apart, the two 8-element K chunks of one MMA `lbo` bytes apart
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo)
{
    return (uint64_t)((addr >> 4) & 0x3fffu) | ((uint64_t)((lbo >> 4) & 0x3fffu) << 16) |
           ((uint64_t)((sbo >> 4) & 0x3fffu) << 32) | (1ull << 46);
}

// D[tmem] (+)= A[smem] * (-B[smem]); fp16 operands, fp32 accumulation, M = 128, N = 64, K = 16
__device__ __forceinline__ void mma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t accumulate)
{
    constexpr uint32_t idesc = (1u << 4) /* D fp32 */ | (1u << 14) /* negate B */ |
                               ((uint32_t)(TP_NEURONS >> 3) << 17) | ((uint32_t)(TP_SAMPLES >> 4) << 24);
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        :
        : "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

__device__ __forceinline__ void mma_commit(uint64_t* bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

// two membership bits -> two fp16 values (1.0 = 0x3c00) in one word
__device__ __forceinline__ uint32_t two_halves(uint32_t bits)
{
    const uint32_t x = (bits | (bits << 15)) & 0x00010001u;
    return x * 0x3c00u;
}

struct TcProbeArgs {
    const float* W;           // [H][64] fp32: the dense features' rows of one neuron range
    const float* hnorm;       // [64] ||w||^2 / 2
    const uint32_t* bits;     // [n_tiles * 128][H / 32] membership words, bit f of word f / 32
    int H;                    // dense features: 32, 64, 96, ... (multiple of 32, at most 256)
    int terms;                // fp16 terms per weight: 1 or 2
    int n_tiles;
    int mode;                 // bit 0 build A every tile, bit 1 issue the MMAs, bit 2 drain, bit 3 redistribute,
                              // bit 4 the drain warps also stream 128-bit shared-memory reads (contention test)
    int repeats;
    float* out;               // [128][64] scores of the first tile (block 0 only)
    float* mins;              // [gridDim.x][128] per-sample minimum over the last tile
    long long* cycles;        // [gridDim.x]
    int* status;              // set to 1 if a wait gave up
};

__global__ void __launch_bounds__(TP_THREADS, 1) k_tc_probe(const __grid_constant__ TcProbeArgs a)
{
    extern __shared__ __align__(1024) unsigned char tp_smem[];
    __shared__ __align__(8) uint64_t a_full[2], a_empty[2], d_full[2], d_empty[2], all_done;
    __shared__ uint32_t tmem_base_sh;
    __shared__ int abort_sh;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int H = a.H;
    const int KD = H + 16;                     // K of one term's pass plus the seed step
    const int chunks_a = KD / 8;               // 16-byte K chunks of an A row
    const uint32_t a_bytes = (uint32_t)chunks_a * TP_SAMPLES * 16;
    const uint32_t b_term_bytes = (uint32_t)(H / 8) * TP_NEURONS * 16;
    unsigned char* sA[2] = {tp_smem, tp_smem + a_bytes};
    unsigned char* sB = tp_smem + 2 * a_bytes;               // terms x [H/8][64][8] halves, then the seed chunk pair
    unsigned char* sSeed = sB + (uint32_t)a.terms * b_term_bytes;  // [2][64][8] halves

    if (threadIdx.x == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(&a_full[i], TP_BUILD_WARPS * 32);
            mbar_init(&a_empty[i], 1);
            mbar_init(&d_full[i], 1);
            mbar_init(&d_empty[i], TP_DRAIN_WARPS * 32);
        }
        mbar_init(&all_done, 1);
        abort_sh = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {  // one warp allocates 128 columns of tensor memory: two accumulators of 64 columns
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_sh)),
                     "r"(128u)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // B: every weight as `terms` fp16 terms, K-major [H/8][64][8]; element (feature k, neuron n)
    for (int e = threadIdx.x; e < (H / 8) * TP_NEURONS; e += TP_THREADS) {
        const int c = e / TP_NEURONS, n = e % TP_NEURONS;
        __half hi[8], lo[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float w = a.W[(size_t)(c * 8 + j) * TP_NEURONS + n];
            hi[j] = __float2half_rn(w);
            lo[j] = __float2half_rn(w - __half2float(hi[j]));
        }
        *reinterpret_cast<uint4*>(sB + (size_t)e * 16) = *reinterpret_cast<const uint4*>(hi);
        if (a.terms > 1) *reinterpret_cast<uint4*>(sB + b_term_bytes + (size_t)e * 16) = *reinterpret_cast<const uint4*>(lo);
    }
    // seed step: K rows 0..2 hold -(||w||^2/2) in three fp16 terms (B is negated by the descriptor)
    for (int e = threadIdx.x; e < 2 * TP_NEURONS; e += TP_THREADS) {
        const int c = e / TP_NEURONS, n = e % TP_NEURONS;
        __half v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = __float2half_rn(0.f);
        if (c == 0) {
            const float h = -a.hnorm[n];
            v[0] = __float2half_rn(h);
            const float r1 = h - __half2float(v[0]);
            v[1] = __float2half_rn(r1);
            v[2] = __float2half_rn(r1 - __half2float(v[1]));
        }
        *reinterpret_cast<uint4*>(sSeed + (size_t)e * 16) = *reinterpret_cast<const uint4*>(v);
    }
    // the seed columns of both A buffers: ones in K positions H..H+2, zeros up to H+15
    for (int e = threadIdx.x; e < 2 * 2 * TP_SAMPLES; e += TP_THREADS) {
        const int buf = e / (2 * TP_SAMPLES), c = (e / TP_SAMPLES) & 1, r = e % TP_SAMPLES;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (c == 0) {
            v.x = 0x3c003c00u;
            v.y = 0x00003c00u;
        }
        *reinterpret_cast<uint4*>(sA[buf] + ((size_t)(H / 8 + c) * TP_SAMPLES + r) * 16) = v;
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_sh;
    volatile int* abort_flag = &abort_sh;

    const int total = a.n_tiles * a.repeats;
    const bool do_build = a.mode & 1, do_mma = a.mode & 2, do_drain = a.mode & 4, do_redist = a.mode & 8;
    const bool do_lds = a.mode & 16;
    const long long t_begin = clock64();

    if (warp == 0) {
        // ---- MMA issuer (one thread) --------------------------------------------------------------
        if (lane == 0) {
            for (int it = 0; it < total; ++it) {
                const int buf = it & 1;
                const uint32_t ph = (uint32_t)(it >> 1) & 1u;
                if (!mbar_wait(&a_full[buf], ph, abort_flag)) break;
                if (it >= 2 && !mbar_wait(&d_empty[buf], ((uint32_t)(it >> 1) - 1u) & 1u, abort_flag)) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                if (do_mma) {
                    const uint32_t d_tmem = tmem_base + (uint32_t)buf * TP_NEURONS;
                    const uint32_t a_addr = smem_u32(sA[buf]);
                    uint32_t acc = 0;
                    for (int t = 0; t < a.terms; ++t) {
                        const uint32_t b_addr = smem_u32(sB) + (uint32_t)t * b_term_bytes;
                        for (int ks = 0; ks < H / 16; ++ks) {
                            mma_f16(d_tmem, smem_desc(a_addr + (uint32_t)ks * 2 * TP_SAMPLES * 16, TP_SAMPLES * 16, 128),
                                    smem_desc(b_addr + (uint32_t)ks * 2 * TP_NEURONS * 16, TP_NEURONS * 16, 128), acc);
                            acc = 1;
                        }
                    }
                    mma_f16(d_tmem, smem_desc(a_addr + (uint32_t)(H / 8) * TP_SAMPLES * 16, TP_SAMPLES * 16, 128),
                            smem_desc(smem_u32(sSeed), TP_NEURONS * 16, 128), acc);
                }
                mma_commit(&a_empty[buf]);  // the tile's MMAs have read A
                mma_commit(&d_full[buf]);   // and written the accumulator
            }
            mma_commit(&all_done);
            mbar_wait(&all_done, 0, abort_flag);
        }
    } else if (warp <= TP_BUILD_WARPS) {
        // ---- A builders: thread r writes sample r's row --------------------------------------------
        const int r = threadIdx.x - 32;
        for (int it = 0; it < total; ++it) {
            const int buf = it & 1;
            if (it >= 2 && !mbar_wait(&a_empty[buf], ((uint32_t)(it >> 1) - 1u) & 1u, abort_flag)) break;
            if (do_build || it < 2) {
                const int tile = it % a.n_tiles;
                const uint32_t* my = a.bits + ((size_t)tile * TP_SAMPLES + r) * (H / 32);
                for (int wd = 0; wd < H / 32; ++wd) {
                    const uint32_t m = __ldg(my + wd);
#pragma unroll
                    for (int c = 0; c < 4; ++c) {  // four chunks of 8 features per word
                        const uint32_t b8 = m >> (8 * c);
                        uint4 v;
                        v.x = two_halves(b8 & 3u);
                        v.y = two_halves((b8 >> 2) & 3u);
                        v.z = two_halves((b8 >> 4) & 3u);
                        v.w = two_halves((b8 >> 6) & 3u);
                        *reinterpret_cast<uint4*>(sA[buf] + ((size_t)(wd * 4 + c) * TP_SAMPLES + r) * 16) = v;
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            }
            mbar_arrive(&a_full[buf]);
        }
    } else {
        // ---- drain: warp q of the group owns accumulator lanes 32 q .. 32 q + 31 -------------------
        const int q = warp & 3;  // (a warp may only touch the tensor-memory lanes of its own quarter)
        float keep = __int_as_float(0x7f800000);
        for (int it = 0; it < total; ++it) {
            const int buf = it & 1;
            if (!mbar_wait(&d_full[buf], (uint32_t)(it >> 1) & 1u, abort_flag)) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (do_drain) {
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    uint32_t v[32];
                    const uint32_t taddr = tmem_base + (uint32_t)buf * TP_NEURONS + ((uint32_t)(32 * q + 16 * hh) << 16);
                    asm volatile(
                        "tcgen05.ld.sync.aligned.16x256b.x8.b32 "
                        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]),
                          "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]),
                          "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]),
                          "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                        : "r"(taddr)
                        : "memory");
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    // register 4 g + 2 j + e = (lane 32 q + 16 hh + lane / 4 + 8 j, column 8 g + 2 (lane % 4) + e)
                    if (it == 0 && blockIdx.x == 0 && a.out) {
#pragma unroll
                        for (int g = 0; g < 8; ++g)
#pragma unroll
                            for (int j = 0; j < 2; ++j)
#pragma unroll
                                for (int e = 0; e < 2; ++e)
                                    a.out[(size_t)(32 * q + 16 * hh + (lane >> 2) + 8 * j) * TP_NEURONS + 8 * g +
                                          2 * (lane & 3) + e] = __uint_as_float(v[4 * g + 2 * j + e]);
                    }
                    if (do_redist) {
                        // to eight threads per sample: a thread keeps half of each of its two samples'
                        // sixteen neurons and trades the other half with the thread sixteen lanes away
                        // (whose samples are four slots on), as the fused kernel's 128-byte reads need
#pragma unroll
                        for (int g = 0; g < 8; g += 2) {
#pragma unroll
                            for (int j = 0; j < 2; ++j)
#pragma unroll
                                for (int e = 0; e < 2; ++e) {
                                    const bool upper = lane & 16;
                                    const uint32_t give = upper ? v[4 * g + 2 * j + e] : v[4 * (g + 1) + 2 * j + e];
                                    const uint32_t got = __shfl_xor_sync(0xffffffffu, give, 16);
                                    if (upper) v[4 * g + 2 * j + e] = got;
                                    else v[4 * (g + 1) + 2 * j + e] = got;
                                }
                        }
                    }
                    float m0 = __uint_as_float(v[0]), m1 = __uint_as_float(v[2]);
#pragma unroll
                    for (int g = 0; g < 8; ++g) {
                        m0 = fminf(m0, fminf(__uint_as_float(v[4 * g]), __uint_as_float(v[4 * g + 1])));
                        m1 = fminf(m1, fminf(__uint_as_float(v[4 * g + 2]), __uint_as_float(v[4 * g + 3])));
                    }
                    keep = fminf(keep, fminf(m0, m1));
                    if (it == total - 1 && a.mins && !do_redist) {
                        // per-sample minimum over the 64 neurons: combine the four threads of a sample
                        m0 = fminf(m0, __shfl_xor_sync(0xffffffffu, m0, 1));
                        m0 = fminf(m0, __shfl_xor_sync(0xffffffffu, m0, 2));
                        m1 = fminf(m1, __shfl_xor_sync(0xffffffffu, m1, 1));
                        m1 = fminf(m1, __shfl_xor_sync(0xffffffffu, m1, 2));
                        if ((lane & 3) == 0) {
                            a.mins[(size_t)blockIdx.x * TP_SAMPLES + 32 * q + 16 * hh + (lane >> 2)] = m0;
                            a.mins[(size_t)blockIdx.x * TP_SAMPLES + 32 * q + 16 * hh + (lane >> 2) + 8] = m1;
                        }
                    }
                }
            }
            if (do_lds) {
                // The row-table kernel's shared-memory traffic, in its access pattern: eight lanes read one
                // contiguous 128-byte row segment; 64 such 128-bit reads per thread and tile, i.e. 1024
                // wavefronts per tile from the four warps.  Run beside the MMAs, it shows whether the
                // tensor core's operand fetch and the load/store pipe draw on the same shared-memory cycles.
                const unsigned char* base = sB + (lane & 7) * 16;
                uint32_t rows_mask = 1;  // (a power of two of 128-byte rows inside B, less one)
                while (2 * rows_mask <= (uint32_t)a.terms * b_term_bytes / 128) rows_mask *= 2;
                rows_mask -= 1;
                const uint32_t r0 = (uint32_t)(it * 37 + (threadIdx.x >> 3) * 11);
                uint4 s4 = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll 16
                for (int k = 0; k < 64; ++k) {
                    const uint32_t rr = (r0 + (uint32_t)k * 29u) & rows_mask;  // independent addresses: all in flight
                    const uint4 x = *reinterpret_cast<const uint4*>(base + (size_t)rr * 128);
                    s4.x ^= x.x; s4.y ^= x.y; s4.z ^= x.z; s4.w ^= x.w;
                }
                keep = fminf(keep, __uint_as_float((s4.x ^ s4.y ^ s4.z ^ s4.w) | 0x40000000u));
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            mbar_arrive(&d_empty[buf]);
        }
        if (keep == -1.2345f && a.mins) a.mins[0] = keep;  // keeps the reductions alive
    }
    const long long t_end = clock64();
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x == 0) {
        a.cycles[blockIdx.x] = t_end - t_begin;
        if (abort_sh) *a.status = 1;
    }
    if (warp == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(128u) : "memory");
    }
}

}  // namespace

extern "C" int som_tc_probe(const float* d_rows, const float* d_hnorm, const uint32_t* d_bits, int32_t H, int32_t terms,
                            int32_t n_tiles, int32_t mode, int32_t repeats, int32_t blocks, float* d_out,
                            float* d_mins, long long* d_cycles, int* d_status, void* stream)
{
    if (!d_rows || !d_hnorm || !d_bits || !d_cycles || !d_status) return SOM_ERR_INVALID_ARG;
    if (H < 32 || H > 256 || H % 32 != 0 || (terms != 1 && terms != 2) || n_tiles < 1 || repeats < 1 || blocks < 1)
        return SOM_ERR_INVALID_ARG;
    const size_t smem = (size_t)2 * ((H + 16) / 8) * TP_SAMPLES * 16 + (size_t)terms * (H / 8) * TP_NEURONS * 16 +
                        2 * TP_NEURONS * 16;
    if (smem > 220 * 1024) return SOM_ERR_UNSUPPORTED;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (cudaFuncSetAttribute(k_tc_probe, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return SOM_ERR_CUDA;
    TcProbeArgs a;
    a.W = d_rows;
    a.hnorm = d_hnorm;
    a.bits = d_bits;
    a.H = H;
    a.terms = terms;
    a.n_tiles = n_tiles;
    a.mode = mode;
    a.repeats = repeats;
    a.out = d_out;
    a.mins = d_mins;
    a.cycles = d_cycles;
    a.status = d_status;
    if (cudaMemsetAsync(d_status, 0, sizeof(int), st) != cudaSuccess) return SOM_ERR_CUDA;
    k_tc_probe<<<blocks, TP_THREADS, smem, st>>>(a);
    return cudaGetLastError() == cudaSuccess ? SOM_OK : SOM_ERR_CUDA;
}
