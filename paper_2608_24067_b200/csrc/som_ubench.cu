// Microbenchmark of the unit whose peak bounds the search: the plain FP32 add pipe.
// The search executes adds and no multiplies (Section 5.7 of the paper says the same of its
// kernel), so its roofline is SMs x 128 lanes x clock adds per second; this kernel measures what
// the device delivers when nothing but independent add chains is issued.
#include "som_internal.cuh"

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

}  // namespace

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
