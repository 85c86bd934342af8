// som_norms_noalloc: the per-neuron norm pass for callers that must not allocate device memory.
//
// The regular som_norms keeps its per-split partial sums in a workspace that the handle
// obtains from cudaMalloc.  Some callers cannot afford that call: a process that has already
// handed the whole device to its own memory pool (a raw cudaMalloc there can fail or fragment
// the pool), or a latency-critical loop in which cudaMalloc's implicit device-wide
// synchronisation is not acceptable.  For them this file keeps the partial sums in a
// file-scope __device__ array of fixed size; the caller supplies the codebook and the output.
//
// Cost and limits: every GPU that loads this library holds the 4 MiB array until the process
// exits.  The array bounds the problem size: splits * M doubles must fit, so M may not exceed
// SOM_NOALLOC_MAX_M.  All calls on a device share the array and it keeps the previous call's
// contents; two calls that overlap on the GPU (different streams, no ordering) race on it.
// Nothing in it has to start at zero: each call's first kernel overwrites every element that
// its second kernel reads.
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "../../include/som.h"

namespace {

constexpr int64_t SCRATCH_DOUBLES = 512 * 1024;  // 4 MiB
constexpr int NA_THREADS = 128;
constexpr int NA_MAX_DEVICES = 64;

static __device__ __align__(256) double g_norm_scratch[SCRATCH_DOUBLES];

// In host code `g_norm_scratch` is only a handle for the runtime, not a device address; the
// address a kernel can use comes from cudaGetSymbolAddress, once per device.
double* g_scratch_addr[NA_MAX_DEVICES];
bool g_scratch_ready[NA_MAX_DEVICES];
std::mutex g_setup_mutex;

template <int VEC>
__global__ void __launch_bounds__(NA_THREADS)
k_na_partial(const float* __restrict__ W, int64_t M, int V, int rows_per_split, double* __restrict__ partial)
{
    const int64_t i = ((int64_t)blockIdx.x * NA_THREADS + threadIdx.x) * VEC;
    if (i >= M) return;
    const int v0 = blockIdx.y * rows_per_split;
    const int v1 = min(V, v0 + rows_per_split);
    double acc[VEC];
#pragma unroll
    for (int k = 0; k < VEC; ++k) acc[k] = 0.0;
    const float* p = W + (int64_t)v0 * M + i;
    for (int v = v0; v < v1; ++v, p += M) {
        if (VEC == 4) {
            const float4 w = __ldcs(reinterpret_cast<const float4*>(p));
            acc[0] = fma((double)w.x, (double)w.x, acc[0]);
            acc[1 % VEC] = fma((double)w.y, (double)w.y, acc[1 % VEC]);
            acc[2 % VEC] = fma((double)w.z, (double)w.z, acc[2 % VEC]);
            acc[3 % VEC] = fma((double)w.w, (double)w.w, acc[3 % VEC]);
        } else {
            const float w = __ldcs(p);
            acc[0] = fma((double)w, (double)w, acc[0]);
        }
    }
    double* out = partial + (int64_t)blockIdx.y * M + i;
#pragma unroll
    for (int k = 0; k < VEC; ++k) out[k] = acc[k];
}

__global__ void k_na_combine(const double* __restrict__ partial, int64_t M, int splits, float* __restrict__ norms)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= M) return;
    double s = 0.0;
    for (int k = 0; k < splits; ++k) s += partial[(int64_t)k * M + i];
    norms[i] = (float)s;
}

}  // namespace

extern "C" int som_norms_noalloc(int32_t V, int64_t M, const float* d_codebook, float* d_norms, void* stream)
{
    if (V <= 0 || M <= 0 || !d_codebook || !d_norms) return SOM_ERR_INVALID_ARG;
    if (M > SOM_NOALLOC_MAX_M) return SOM_ERR_UNSUPPORTED;  // the static scratch cannot hold one split
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return SOM_ERR_NO_DEVICE;
    if (dev < 0 || dev >= NA_MAX_DEVICES) return SOM_ERR_UNSUPPORTED;
    double* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_setup_mutex);
        if (!g_scratch_ready[dev]) {
            void* p = nullptr;
            if (cudaGetSymbolAddress(&p, g_norm_scratch) != cudaSuccess || !p) return SOM_ERR_CUDA;
            g_scratch_addr[dev] = static_cast<double*>(p);
            g_scratch_ready[dev] = true;
        }
        scratch = g_scratch_addr[dev];
    }
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return SOM_ERR_CUDA;

    const int vec = (M % 4 == 0 && (reinterpret_cast<uintptr_t>(d_codebook) & 15u) == 0) ? 4 : 1;
    const int64_t col_threads = (M + vec - 1) / vec;
    const int64_t col_blocks = (col_threads + NA_THREADS - 1) / NA_THREADS;
    int64_t splits = ((int64_t)sms * 16 + col_blocks - 1) / col_blocks;  // enough blocks to fill the GPU
    const int64_t fit = SCRATCH_DOUBLES / M;                           // what the static array can hold
    if (splits > fit) splits = fit;
    if (splits > (V + 15) / 16) splits = (V + 15) / 16;
    if (splits > 65535) splits = 65535;
    if (splits < 1) splits = 1;
    const int rows_per_split = (int)((V + splits - 1) / splits);
    const int n_splits = (V + rows_per_split - 1) / rows_per_split;

    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    dim3 grid((unsigned)col_blocks, (unsigned)n_splits);
    if (vec == 4)
        k_na_partial<4><<<grid, NA_THREADS, 0, st>>>(d_codebook, M, V, rows_per_split, scratch);
    else
        k_na_partial<1><<<grid, NA_THREADS, 0, st>>>(d_codebook, M, V, rows_per_split, scratch);
    if (cudaGetLastError() != cudaSuccess) return SOM_ERR_CUDA;
    k_na_combine<<<(unsigned)((M + 255) / 256), 256, 0, st>>>(scratch, M, n_splits, d_norms);
    if (cudaGetLastError() != cudaSuccess) return SOM_ERR_CUDA;
    return SOM_OK;
}
