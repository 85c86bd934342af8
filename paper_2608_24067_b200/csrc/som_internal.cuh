// Internal declarations shared by the translation units of the BMU library (sm_100a).
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/som.h"

#define SOM_EV_PER_CALL 6
#define SOM_EV_RING 32
#define SOM_N_EVENTS (SOM_EV_PER_CALL * SOM_EV_RING)

// which choices of the device-side gate a launch belongs to (bit number = value of the gate word)
#define SOM_GATE_DIRECT 1      /* choice 0 */
#define SOM_GATE_TABLE_PLAIN 2 /* choice 1 */
#define SOM_GATE_TABLE_TS 4    /* choice 2 */
#define SOM_GATE_TABLE 6       /* choice 1 or 2: the plan, the rare pass */

// bits of som_handle::dev_flags
#define SOM_FLAG_BAD_INDEX 1 /* a feature id outside [0, V) was skipped */
#define SOM_FLAG_BAD_UNIT 2  /* a best-unit index outside [0, M) was skipped */

#define SOM_AUX_HAS_NEGATIVE 1
#define SOM_AUX_HMAX 2

struct som_handle {
    int device;
    int sm_count;
    int32_t V;
    int64_t M;
    const float* W;    // borrowed, feature-major fp32 codebook (nullptr when stored as fp16)
    const __half* Wh;  // borrowed, feature-major fp16 codebook (som_create_f16), else nullptr
    float* range_max;  // owned, [M / 128][V][4]: per feature row, 128-neuron range and 32-neuron group the largest weight (written by
                       // som_norms when M % 128 == 0; nullptr = none); bounds for the search's pruning
    int32_t* range_order;  // owned, [M / 128]: the 128-neuron ranges by ascending smallest ||w||^2 (nullptr = none)
    __half* shadow;    // owned fp16 copy of an fp32 codebook for the two-stage search (nullptr = none)
    unsigned int* wmax_bits;  // device, written by som_norms with the shadow: [0] float bits of max |weight|,
                              // [SOM_AUX_HAS_NEGATIVE] 1 if a weight is negative, [SOM_AUX_HMAX] float bits of max ||w||^2/2
    int shadow_valid;         // the last som_norms wrote the shadow
    int64_t last_uncertain;   // samples the last two-stage search sent to its exact pass

    double* norm64;  // [M] ||w_i||^2 in fp64
    float* norm32;   // [M] the same rounded to fp32
    float* hnorm;    // [M] 0.5 * ||w_i||^2, the seed of every score accumulator
    int norms_valid;

    void* ws;  // grow-only device workspace shared by som_norms / som_bmu
    size_t ws_bytes;
    void* stage;  // grow-only device staging for som_bmu_host
    size_t stage_bytes;
    // pipelined host entry point (som_bmu_host_async): copy stream, two staging buffers, events
    cudaStream_t copy_stream, back_stream;  // host-to-device and device-to-host
    cudaStream_t aux_stream;                // som_update: side stream of the denominator's route
    cudaEvent_t ev_fork, ev_join;
    cudaEvent_t ev_h2d[2], ev_searched[2], ev_d2h[2];
    void* pipe_stage[2];
    size_t pipe_stage_bytes[2];
    int64_t pipe_calls;
    void* head;  // small plan arrays that the selection phase fills before nnz is known
    size_t head_bytes;

    int last_cuda_error;
    int timing;
    int events_made;
    cudaEvent_t ev[SOM_N_EVENTS];
    int64_t ev_norms_calls;  // calls recorded since timing was switched on
    int64_t ev_bmu_calls;
    int64_t launches;
    int64_t opt_variant;   // 0 auto, 1 direct-load kernel, 2 row-table kernel
    int64_t opt_hot_rows;  // 0 = default number of hot rows in shared memory
    int64_t opt_threads;   // block size of the row-table kernel: 0 (default 512), 512 or 1024
    int64_t opt_r;         // neurons per lane of the row-table kernel: 0 = default, 4, 8 or 16
    int64_t opt_parts;     // row-table kernel: sample parts per neuron range (0 = default)
    int64_t opt_feed_keep; // row-table kernel: slot stream kept in L2 (0 = by batch size, 1 = always, 2 = never)
    int64_t opt_prune;     // row-table kernel: skip a sample's tail rows for ranges that cannot hold its best unit
                           // (0 = where range_max exists and the map has at least 32 ranges of 128 neurons, 1 = wherever range_max exists, 2 = off)
    int64_t opt_mask_bits; // plan: features handled as mask bits (0 = default by batch size, else 1..16)
    int plan_attr_set;
    int64_t opt_update_mib;  // som_update: workspace budget for its slab buffers in MiB (0 = 4096)
    int64_t opt_two_stage;  // 0 = off, 1 = on where it applies (fp32 storage, M % 128 == 0, memory for the shadow)
    int64_t opt_cover;     // auto selection: least percentage of instances the row table must cover (0 = 60)
    // Kernel choice made on the device: the launchers hand `gate` / `gate_want` to the kernels of every
    // search path, and a kernel returns at once unless bit *gate of gate_want is set (SOM_GATE_* masks).
    // *gate is 0 = direct-load kernel, 1 = row-table kernel, 2 = row-table kernel with the two-stage search.
    const int* gate;       // device, nullptr = no gate
    int gate_want;
    int gate_small_grid;   // the gated launch in hand is expected to return at once: give it a small grid
    // Length of a sample list that only the device knows (the samples that do not fit a slot of the
    // row-table plan): while set, the direct-load kernel and its finalisation read their sample count
    // from it and are launched with small grids that walk the list.
    const int* list_len_dev;
    int* dev_flags;        // device, sticky: SOM_FLAG_* bits set by kernels that skipped a bad entry
    int32_t* host_pair;    // pinned, 4 ints: read-back of indptr[0], indptr[n], covered instances, uncertain samples
};

// pruning by range maxima in the row-table search: on from this many ranges of 128 neurons (option 10 = 0)
constexpr int SOM_PRUNE_MIN_RANGES = 32;
// whether the row-table search over the handle's own codebook prunes (the launcher also wants a layout that can)
static inline bool som_table_prunes(const som_handle* h)
{
    return h->range_max != nullptr &&
           (h->opt_prune == 1 || (h->opt_prune == 0 && (h->M + 127) / 128 >= SOM_PRUNE_MIN_RANGES));
}


// event slots
enum { EV_NORMS_BEGIN = 0, EV_NORMS_END, EV_BMU_BEGIN, EV_BMU_PLAN_END, EV_BMU_SEARCH_END, EV_BMU_END };

#define SOM_CK(h, call)                                   \
    do {                                                  \
        cudaError_t e__ = (call);                         \
        if (e__ != cudaSuccess) {                         \
            (h)->last_cuda_error = (int)e__;              \
            return SOM_ERR_CUDA;                          \
        }                                                 \
    } while (0)

static inline size_t som_align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Order-preserving map of an fp32 value to uint32 (smaller float -> smaller uint).
__device__ __forceinline__ uint32_t som_ordered_bits(float f)
{
    uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// (score, neuron) packed so that an unsigned 64-bit min is the lexicographic
// (smallest score, then lowest neuron index) min.
__device__ __forceinline__ unsigned long long som_pack_key(float score, uint32_t neuron)
{
    return ((unsigned long long)som_ordered_bits(score) << 32) | (unsigned long long)neuron;
}

// One stored weight as fp32 (exact for both storage types).
__device__ __forceinline__ float som_weight(const float* p) { return __ldg(p); }
__device__ __forceinline__ float som_weight(const __half* p) { return __half2float(__ldg(p)); }

// kernels' host launchers (each returns a som_status)
int som_launch_norms(som_handle* h, cudaStream_t st);
int som_launch_bmu_direct(som_handle* h, const int32_t* indptr, const int32_t* indices, int64_t n,
                          unsigned long long* keys, unsigned long long* keys2, const int32_t* sample_list,
                          cudaStream_t st);
int som_launch_finalize(som_handle* h, const int32_t* indptr, const int32_t* indices, int64_t n,
                        const unsigned long long* keys, int32_t* bmu, float* dist, const int32_t* sample_list,
                        cudaStream_t st);
int som_launch_bmu_values(som_handle* h, const int32_t* indptr, const int32_t* indices, const float* values,
                          int64_t n, unsigned long long* keys, cudaStream_t st);
int som_launch_finalize_values(som_handle* h, const int32_t* indptr, const int32_t* indices, const float* values,
                               int64_t n, const unsigned long long* keys, int32_t* bmu, float* dist,
                               cudaStream_t st);
int som_launch_validate(som_handle* h, const int32_t* indptr, const int32_t* indices, int64_t n,
                        int* d_flag, cudaStream_t st);
size_t som_norms_workspace_bytes(const som_handle* h);
size_t som_update_workspace_bytes(const som_handle* h, int64_t budget_bytes, int* planes_per_slab);
int som_launch_update(som_handle* h, int rows, int cols, const int32_t* indptr, const int32_t* indices,
                      int64_t n, const int32_t* bmu, int radius, int planes_per_slab, const int32_t* hot_slot,
                      const int32_t* slot_feat, int n_hot_slots, cudaStream_t st, cudaStream_t aux,
                      cudaEvent_t ev_join);

// true when this launch belongs to the search path that the plan's selection did not choose
__device__ __forceinline__ bool som_gated_off(const int* gate, int want_mask)
{
    return gate != nullptr && !((want_mask >> *reinterpret_cast<const volatile int*>(gate)) & 1);
}

// records a skipped entry in the handle's flag word (one atomic per warp that saw any)
__device__ __forceinline__ void som_raise(int* flags, bool bad, int bit)
{
    if (__any_sync(__activemask(), bad) && bad) atomicOr(flags, bit);
}
