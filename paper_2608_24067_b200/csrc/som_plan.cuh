// Layout of the per-batch plan in the handle's workspace, shared by the plan kernels and the
// row-table search kernel.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

struct som_handle;

#define SOM_PLAN_MASK_FEATURES 16
#define SOM_PLAN_LEN_BITS 7 /* hot count (4 bits) and tail count (3 bits) */
#define SOM_PLAN_BINS (1 << (SOM_PLAN_MASK_FEATURES + SOM_PLAN_LEN_BITS))

// One 48-byte slot per sample, at a fixed address for its sorted position k (slots[k]), so
// that the search kernel can load it one round ahead without chasing an offset.  As 12 words:
//   w0        mask of mask features (bits 0-15) | hot codes (16-23) | tail codes (24-31);
//             a tail count of SOM_SLOT_NT_OVERFLOW marks a sample that does not fit a slot
//   w1        tail codes 8..9
//   w2..w7    hot codes 0..11, 16 bits each: row of the feature in the shared-memory table;
//             unused ones hold the index of the all-zero row that follows the table
//   w8..w11   tail codes 0..7, 16 bits each: feature id
// (the sample index of a sorted position lives in a separate array, `order`: only the
// finalisation needs it).
// A sample fits when it has at most 12 hot and 10 tail features; for the rare others the slot
// holds only the mask and the sample index (hot codes all zero-row, tail codes feature 0): the
// row-table kernel gives such a sample no candidate, and its index goes on a list (rare_list)
// that the direct-load kernel searches afterwards, writing its outputs last.
// 16-bit codes require V <= 65536 and at most 65536 table rows.
// The slot array is padded to a multiple of 4 samples with copies of the last slot, so the
// search kernel always runs whole rounds; the duplicates redo the same idempotent atomicMin.
#define SOM_SLOT_WORDS 12
#define SOM_SLOT_MAX_HOT 12
#define SOM_SLOT_MAX_TAIL 10
#define SOM_SLOT_NT_OVERFLOW 255u

// Byte offsets of the plan's arrays.  The first four live in the small "head" buffer, sized by V;
// the others live in the handle's workspace, sized by the number of samples alone (the host never
// needs the batch's nnz, which lives on the device).
struct SomPlanBuffers {
    // head buffer
    size_t feat_count;  // u32 [V]
    size_t feat_slot;   // i32 [V]      table slot of a feature, -1 = tail
    size_t slot_feat;   // i32 [slots]  feature of a table slot, -1 = unused
    size_t n_slots;     // i32 [8]      mask slots used, hot slots used, length of rare_list, search unit counter,
                        //              feature instances covered by the table, uncertain samples, the gate
                        //              word (SOM_PLAN_USE_TABLE), the two-stage report (SOM_PLAN_REPORT)
    // workspace
    size_t keys;        // u64 [n]      packed (score, neuron) per sorted position
    size_t keys2;       // u64 [n]      the same for the second-best unit (two-best search only)
    size_t keys3;       // u64 [n]      and for the third best (first pass of the two-stage two-best search)
    size_t pk;          // u32 [n]      mask | n_hot << 16, by sample
    size_t ntail;       // u32 [n]
    size_t bin_count;   // u32 [bins]
    size_t bin_start;   // u32 [bins]
    size_t block_sums;  // u32 [scan blocks]
    size_t slots;       // 48 B [n + 16]
    size_t order;       // u32 [n + 16]  sample index of every sorted position
    size_t uncertain;   // i32 [n]      samples the two-stage search sends to its exact pass
    size_t ukeys;       // u64 [n + 16] their packed keys, by position in that list
    size_t ukeys2;      // u64 [n + 16] and their second-best keys (two-best search)
    size_t slots2;      // 48 B [n + 16] their slots, compacted in list order
    size_t rare_list;   // i32 [n]      samples that do not fit a slot (searched by the direct-load kernel)
    size_t rare_keys;   // u64 [n + 16] their packed keys, by position in that list
    size_t rare_keys2;  // u64 [n + 16] and their second-best keys (two-best search)
};
#define SOM_PLAN_N_SLOTS_INTS 8
#define SOM_PLAN_RARE 2 /* index into n_slots: length of rare_list */
#define SOM_PLAN_COVERED 4 /* index into n_slots */
#define SOM_PLAN_UNCERTAIN 5 /* index into n_slots: length of the two-stage search's uncertain list */
#define SOM_PLAN_USE_TABLE 6 /* index into n_slots: the device-side choice (the gate word): 0 direct-load kernel,
                                1 row-table kernel, 2 row-table kernel with the two-stage search */
#define SOM_PLAN_REPORT 7    /* index into n_slots: the two-stage search's report (see k_two_stage_decide) */

// Sample parts per neuron range of the row-table kernel.  More parts mean fewer ranges live at
// once (their slabs must share L2 with the slot stream) but smaller units, each of which
// rebuilds the row table.  Measured on 250k to 4M-sample batches:
//   64-neuron ranges (fp32, 256-byte rows): flat optimum at about 20,000 samples per unit, at most 32 parts;
//   128-neuron ranges of the wide fp16 layout (256-byte rows): half as many ranges, smaller units;
//   128-neuron ranges of the wide fp32 layout (512-byte rows, slabs of 15 MB): the fewer ranges are
//     live the better - 40 to 48 parts on a 250k-sample batch (units of 6,000 samples) are 10 % faster
//     than 16 on the largest map, 64 to 80 are best on 1M samples, 96 to 128 on 4M samples.
//     (Those are the figures of the search that reads every row; where it prunes, the launcher takes 16 parts
//     for batches of that size on the large maps, see launch_table.)
static inline int som_table_default_parts(int64_t n, int range_neurons, int row_bytes)
{
    if (row_bytes >= 512) return n < 48 * 1024 ? (n < 1024 ? 1 : (int)(n / 1024)) : (n < 600000 ? 44 : (n < 2500000 ? 64 : 96));
    const bool wide = range_neurons >= 128;
    const int64_t parts = n / (wide ? 15000 : 20000);
    const int64_t cap = wide ? 64 : 32;
    return parts < 1 ? 1 : (parts > cap ? (int)cap : (int)parts);
}

size_t som_plan_head_bytes(int32_t V, int n_slots_max, SomPlanBuffers* b);
size_t som_plan_workspace_bytes(int64_t n, SomPlanBuffers* b);

// Phase 1 (needs no workspace): feature histogram and choice of the mask and hot features;
// leaves the number of feature instances they cover in n_slots[SOM_PLAN_COVERED].
int som_launch_plan_select(som_handle* h, const int32_t* indptr, const int32_t* indices, int64_t n,
                           char* head, const SomPlanBuffers& b, int n_mask, int n_hot, cudaStream_t st);
// Phase 2: classify, sort and re-encode the samples into slots.
int som_launch_plan_sort(som_handle* h, const int32_t* indptr, const int32_t* indices, int64_t n,
                         char* head, char* ws, const SomPlanBuffers& b, int n_mask, int n_hot,
                         cudaStream_t st);

// shadow = read the handle's fp16 shadow of an fp32 codebook (first pass of the two-stage search);
// keep = how many best units per sample are kept (1, 2; 3 with the shadow's wide layout only)
int som_launch_bmu_table(som_handle* h, bool shadow, const int32_t* indptr, const int32_t* indices, int64_t n,
                         char* head, char* ws, const SomPlanBuffers& b, int n_hot, int keep, cudaStream_t st);

// pads a slot array of n slots to a multiple of four with copies of the last one
int som_launch_pad_slots(som_handle* h, char* ws, size_t slots_offset, int64_t n, cudaStream_t st);

// second: the two-best search (needs the three best first-pass keys); count_only: only count the
// samples that fail the certificate into *n_uncertain (the probe; no outputs are touched)
int som_launch_certify(som_handle* h, const int32_t* indptr, const int32_t* indices, int64_t n, char* ws,
                       const SomPlanBuffers& b, bool second, bool count_only, int32_t* bmu, float* dist,
                       int32_t* bmu2, float* dist2, int32_t* uncertain, int* n_uncertain, cudaStream_t st);

// The two-stage search first tries its certificate on one sample in SOM_PROBE_STRIDE (by sample index, so
// the choice depends on the batch alone); batches below SOM_PROBE_MIN_BATCH samples are not probed.
#define SOM_PROBE_STRIDE 256
#define SOM_PROBE_MIN_BATCH 65536
int som_launch_probe_gather(som_handle* h, int64_t n, char* ws, const SomPlanBuffers& b, cudaStream_t st);
int som_launch_two_stage_decide(som_handle* h, char* head, const SomPlanBuffers& b, int n_probe, int64_t n,
                                cudaStream_t st);

int som_launch_finalize_sorted(som_handle* h, const int32_t* indptr, const int32_t* indices, int64_t n,
                               char* ws, const SomPlanBuffers& b, bool second, int32_t* bmu, float* dist,
                               cudaStream_t st);

// Geometry of the row-table kernel for this handle: neurons per range, hot rows that fit.
struct SomTableGeom {
    int R;        // neurons per lane (4, 8 or 16)
    int T;        // neurons per range = 8 * R
    int n_hot;    // hot rows held in shared memory
    int threads;  // block size
    int row_bytes;  // bytes of a table row (T neurons in the storage type)
    size_t smem;  // dynamic shared memory bytes
};
SomTableGeom som_table_geometry(const som_handle* h, bool shadow = false);
