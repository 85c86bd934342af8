// Microbenchmarks of the units that bound the search: the plain FP32 add pipe, and the two paths an add's
// operand takes into a register (shared memory; L2 through the load/store pipe or the texture unit).
// The search executes adds and no multiplies (Section 5.7 of the paper says the same of its
// kernel), so its roofline is SMs x 128 lanes x clock adds per second; this kernel measures what
// the device delivers when nothing but independent add chains is issued.
#include "som_internal.cuh"
#include <new>

namespace {

constexpr int UB_THREADS = 1024;
constexpr int UB_CHAINS = 8;

__global__ void __launch_bounds__(UB_THREADS, 2)
k_fadd_peak(float* __restrict__ out, int iters, float step)
{
    float a[UB_CHAINS];
#pragma unroll
    for (int j = 0; j < UB_CHAINS; ++j) a[j] = (float)(threadIdx.x + j);
    // eight independent chains per thread, 64 warps per SM: the adds of a warp never wait
    for (int i = 0; i < iters; ++i) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
#pragma unroll
            for (int j = 0; j < UB_CHAINS; ++j) a[j] += step;
        }
    }
    float s = 0.f;
#pragma unroll
    for (int j = 0; j < UB_CHAINS; ++j) s += a[j];
    out[(size_t)blockIdx.x * UB_THREADS + threadIdx.x] = s;
}

// ---- operand paths -----------------------------------------------------------------------------------
// One block of 512 threads per SM; eight lanes read one 512-byte row as four 128-bit pieces 128 bytes apart,
// the access pattern of the row-table search kernel's wide fp32 layout: rows of a 180 KB table in shared
// memory (bit 0 of mode), rows of an L2-resident buffer with read-only global loads (bit 1), the same rows
// through a linear texture (bit 2).  Row numbers come from a per-team generator, so nothing is reused.
constexpr int OP_THREADS = 512;
constexpr int OP_ROWS_SHARED = 360;

__global__ void __launch_bounds__(OP_THREADS, 1)
k_operand_paths(const float4* __restrict__ rows, uint32_t n_rows, cudaTextureObject_t tex, int mode, int iters,
                float* __restrict__ out, long long* __restrict__ cycles)
{
    extern __shared__ float4 op_table[];
    for (int i = threadIdx.x; i < OP_ROWS_SHARED * 32; i += OP_THREADS) op_table[i] = make_float4((float)i, 1.f, 2.f, 3.f);
    __syncthreads();
    const int q = threadIdx.x & 7;
    uint32_t rng = ((uint32_t)blockIdx.x * OP_THREADS + threadIdx.x) / 8u * 2654435761u + 12345u;  // one per team
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    const long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
        rng = rng * 1664525u + 1013904223u;
        const uint32_t rs = (rng >> 8) % OP_ROWS_SHARED, rg = (rng >> 4) % n_rows;
        if (mode & 1) {
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const float4 v = op_table[rs * 32 + x * 8 + q];
                acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
            }
        }
        if (mode & 2) {
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const float4 v = __ldg(rows + (size_t)rg * 32 + x * 8 + q);
                acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
            }
        }
        if (mode & 4) {
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const float4 v = tex1Dfetch<float4>(tex, (int)(rg * 32 + x * 8 + q));
                acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
            }
        }
    }
    const long long t1 = clock64();
    out[(size_t)blockIdx.x * OP_THREADS + threadIdx.x] = acc.x + acc.y + acc.z + acc.w;
    if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

}  // namespace

extern "C" int som_measure_operand_paths(double* bytes_per_clk, int n_out, const void* d_rows, int64_t rows_bytes,
                                         float* d_scratch, int64_t scratch_elems, void* stream)
{
    if (!bytes_per_clk || n_out < 4 || !d_rows || !d_scratch) return SOM_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(d_rows) & 511) != 0 || rows_bytes < 512 || rows_bytes > ((int64_t)1 << 31))
        return SOM_ERR_INVALID_ARG;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return SOM_ERR_NO_DEVICE;
    // scratch: one float per thread, then one 64-bit cycle count per block
    if (scratch_elems < (int64_t)sms * OP_THREADS + 2 * (int64_t)sms + 2) return SOM_ERR_INVALID_ARG;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const uint32_t n_rows = (uint32_t)(rows_bytes / 512);
    cudaResourceDesc rd = {};
    rd.resType = cudaResourceTypeLinear;
    rd.res.linear.devPtr = const_cast<void*>(d_rows);
    rd.res.linear.desc = cudaCreateChannelDesc<float4>();
    rd.res.linear.sizeInBytes = (size_t)n_rows * 512;
    cudaTextureDesc td = {};
    td.readMode = cudaReadModeElementType;
    td.filterMode = cudaFilterModePoint;
    td.addressMode[0] = cudaAddressModeClamp;
    cudaTextureObject_t tex = 0;
    if (cudaCreateTextureObject(&tex, &rd, &td, nullptr) != cudaSuccess) return SOM_ERR_CUDA;
    const size_t shb = (size_t)OP_ROWS_SHARED * 512;
    int rc = SOM_OK;
    if (cudaFuncSetAttribute(k_operand_paths, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)shb) != cudaSuccess)
        rc = SOM_ERR_CUDA;
    long long* d_cycles = reinterpret_cast<long long*>(
        (reinterpret_cast<uintptr_t>(d_scratch + (size_t)sms * OP_THREADS) + 7) & ~(uintptr_t)7);
    long long* h_cycles = new (std::nothrow) long long[sms];
    if (!h_cycles) rc = SOM_ERR_CUDA;
    const int iters = 6000;  // about 3 ms per launch at the slowest path
    const int modes[4] = {1, 2, 3, 4};  // shared memory, L2, both streams in one loop, texture
    for (int m = 0; m < 4 && rc == SOM_OK; ++m) {
        for (int rep = 0; rep < 2; ++rep)  // (the first launch warms L2)
            k_operand_paths<<<sms, OP_THREADS, shb, st>>>(reinterpret_cast<const float4*>(d_rows), n_rows, tex, modes[m],
                                                          iters, d_scratch, d_cycles);
        if (cudaMemcpyAsync(h_cycles, d_cycles, (size_t)sms * 8, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
            cudaStreamSynchronize(st) != cudaSuccess || cudaGetLastError() != cudaSuccess) {
            rc = SOM_ERR_CUDA;
            break;
        }
        double mean = 0.0;
        for (int i = 0; i < sms; ++i) mean += (double)h_cycles[i];
        mean /= sms;
        // per SM and iteration: 16 warps x 4 teams x 512 bytes per stream
        const double streams = modes[m] == 3 ? 2.0 : 1.0;
        bytes_per_clk[m] = mean > 0.0 ? streams * 16.0 * 4.0 * 512.0 * iters / mean : 0.0;
    }
    delete[] h_cycles;
    cudaDestroyTextureObject(tex);
    return rc;
}

extern "C" int som_measure_fadd_peak(double* adds_per_s, float* d_scratch, int64_t scratch_elems, void* stream)
{
    if (!adds_per_s || !d_scratch) return SOM_ERR_INVALID_ARG;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return SOM_ERR_NO_DEVICE;
    const int blocks = sms * 2;
    if (scratch_elems < (int64_t)blocks * UB_THREADS) return SOM_ERR_INVALID_ARG;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return SOM_ERR_CUDA;
    const int iters = 20000;  // 8 x 8 adds per iteration and thread: about 10 ms per launch
    double best = 0.0;
    int rc = SOM_OK;
    for (int rep = 0; rep < 4 && rc == SOM_OK; ++rep) {  // the first launch warms up
        cudaEventRecord(e0, st);
        k_fadd_peak<<<blocks, UB_THREADS, 0, st>>>(d_scratch, iters, 1.0f + (float)rep);
        cudaEventRecord(e1, st);
        if (cudaEventSynchronize(e1) != cudaSuccess || cudaGetLastError() != cudaSuccess) {
            rc = SOM_ERR_CUDA;
            break;
        }
        float ms = 0.f;
        cudaEventElapsedTime(&ms, e0, e1);
        const double adds = (double)blocks * UB_THREADS * UB_CHAINS * 8.0 * (double)iters;
        if (rep > 0 && ms > 0.f && adds / (ms * 1e-3) > best) best = adds / (ms * 1e-3);
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    *adds_per_s = best;
    return rc;
}
