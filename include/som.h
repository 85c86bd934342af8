/*
 * som.h - C ABI of the B200 best-matching-unit (BMU) search for sparse-binary
 * self-organizing maps with a feature-major codebook.
 *
 * The operation (paper, Section 3.1, Eq. 1): for a binary sample x with active feature
 * set S and M prototypes w_i,
 *
 *     BMU(x) = argmin_i ||x - w_i||^2 = argmin_i ( ||w_i||^2 - 2 * sum_{v in S} w_i[v] ),
 *
 * ties broken to the lowest neuron index (Section 3.1).  The codebook is stored
 * feature-major (Section 3.2): weight (v, i) lives at W[v*M + i], so the M weights of one
 * feature are contiguous.  Samples arrive as sparse-binary CSR (Section 4.2): a row-pointer
 * array and one concatenated array of ascending column ids, values implicit 1.
 *
 * Conventions
 *   - Every function returns an int status (SOM_OK == 0).  Nothing throws, prints or exits.
 *   - "device pointer" = memory of the CUDA device that was current in som_create;
 *     "host pointer" = ordinary process memory.  The library never takes ownership of a
 *     caller's buffer.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     som_norms / som_bmu / som_bmu2 only enqueue work on it and return without waiting for
 *     the device: the batch's nnz, the choice of the table's features and, in automatic mode,
 *     the choice between the two search kernels all stay on the device (the kernels of both
 *     paths are enqueued; those of the path not chosen return at once).  Exceptions: growing
 *     the handle's workspace (first call, or a larger batch than any before) allocates device
 *     memory, which may synchronise the device once.
 *   - Thread safety: one handle must not be used from two host threads at once, and two
 *     calls on the same handle must not overlap on the GPU (they share the workspace);
 *     issue them on one stream or order the streams yourself.
 */
#ifndef SOM_B200_H
#define SOM_B200_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct som_handle som_handle; /* opaque */

enum som_status {
    SOM_OK = 0,
    SOM_ERR_INVALID_ARG = 1, /* null pointer, V <= 0, M <= 0, n < 0, misaligned codebook */
    SOM_ERR_NORMS_STALE = 2, /* som_bmu called before som_norms                           */
    SOM_ERR_UNSUPPORTED = 3, /* size outside what the kernels index (see som_create)      */
    SOM_ERR_CUDA = 4,        /* a CUDA call failed; see som_last_cuda_error               */
    SOM_ERR_BAD_CSR = 5,     /* som_validate_csr found a malformed batch                  */
    SOM_ERR_NO_DEVICE = 6    /* no CUDA device / device is not sm_100                     */
};

/*
 * som_create - bind a handle to a codebook (Section 3.2, the feature-major codebook).
 *   out         host pointer; receives the handle.
 *   V           number of features, 1 <= V < 2^31.
 *   M           number of neurons,  1 <= M < 2^31.
 *   d_codebook  DEVICE pointer, fp32, V*M elements, element (v,i) at v*M + i, 16-byte
 *               aligned.  BORROWED: the caller keeps ownership, must keep it alive while
 *               the handle lives, and may rewrite it in place between calls; after any
 *               rewrite som_norms must run again before the next som_bmu.
 * M need not be a multiple of 4, but only then do the 128-bit vector paths apply; other
 * M take a scalar-load kernel.  Allocates M*8 bytes of device memory for the norms.
 */
int som_create(som_handle** out, int32_t V, int64_t M, const float* d_codebook);

/*
 * som_create_f16 - som_create for a codebook STORED in fp16 and accumulated in fp32, the paper's
 * production precision (Section 3.2): half the codebook bytes in HBM, L2 and shared memory
 * (the 1024x1024 map takes 63 GB instead of 126 GB).
 *   d_codebook_f16  DEVICE pointer, IEEE binary16, V*M elements, element (v,i) at v*M + i, 16-byte
 *                   aligned, borrowed like som_create's.
 * Every later call behaves as with som_create: each stored weight is widened exactly to fp32
 * before it is used, scores are accumulated in fp32, norms and reported distances in fp64, so the
 * results are those of som_create on the same values held as fp32.  The vector paths need
 * M % 8 == 0 (norms), M % 4 == 0 (direct-load kernel) and M % 64 == 0 (row-table kernel); other M
 * take the scalar-load kernels.
 */
int som_create_f16(som_handle** out, int32_t V, int64_t M, const void* d_codebook_f16);

/*
 * som_norms - recompute ||w_i||^2 for all M neurons (the norm term of Eq. 1; the separate norm
 * pass whose cost Section 5.7 reports as negligible).  One streaming read of the codebook; squares are
 * accumulated in fp64 in a fixed order (deterministic) and stored as fp32.
 * Must be called once after som_create and again after every codebook update.
 * With M % 128 == 0 the same read also records, for every feature and every range of 128
 * neurons, the largest weight in each of the range's four groups of 32 neurons (V * M / 32 floats, allocated by
 * the first call; if that memory cannot be had the call carries on without them), and the order of the ranges by
 * their smallest norm.  The search uses them to skip rows that cannot change a sample's result (som_bmu below);
 * writing them makes the pass about a fifth longer on the largest map (18 -> 22 ms at 1024 x 1024).
 */
int som_norms(som_handle* h, void* stream);

/*
 * som_bmu - BMU search for one batch (Section 3.3; Algorithm 2, steps 4-7, best unit only).
 *   d_indptr    DEVICE pointer, int32 [n_samples+1]; row s owns indices
 *               [d_indptr[s], d_indptr[s+1]) of d_indices.  d_indptr[0] may be any offset.
 *   d_indices   DEVICE pointer, int32; inside each row ascending, distinct, in [0, V).
 *               These are preconditions (the paper sorts ascending, Section 3.1) and are
 *               NOT checked here; som_validate_csr checks them.  (The batch-plan kernels skip
 *               an id outside [0, V) and record it, see som_device_flags; the search kernels
 *               themselves rely on the precondition.)  May be NULL only when every row is empty.
 *   n_samples   0 <= n_samples < 2^31; 0 is a successful no-op.
 *   d_bmu       DEVICE pointer, int32 [n_samples]  out: index of the nearest neuron,
 *               lowest index among exact fp32 ties.
 *   d_min_dist  DEVICE pointer, fp32 [n_samples]   out: the full squared Euclidean distance
 *               ||x - w_bmu||^2 = |S| - 2*sum_{v in S} w_bmu[v] + ||w_bmu||^2 (left side of
 *               Eq. 1, no square root), recomputed for the winner in fp64 and rounded once.
 * A sample with no active feature gets argmin ||w_i||^2 and that norm.
 * Scores are accumulated in fp32 in a fixed order, so outputs are bit-identical from run
 * to run for the same inputs (same batch, same options).  That order is fixed per BATCH, not
 * per sample: which features the row table holds, and which kernel the automatic mode takes,
 * follow from the batch's feature histogram.  So one sample searched inside two different
 * batches (or by the two kernels) gets fp32 scores that may differ in the last bits, and its
 * best unit may differ between the two calls when its two best units are nearer to each other
 * than that rounding (about 1e-6 of the score; Section 3.1 reports the same effect of the
 * summation order, about one assignment in 1e5 at 256x256).  Wherever the two best units are
 * further apart than 1e-4 of the best squared distance the unit is the same in every batch.
 * The reported distance is always the fp64 one of the reported unit.
 * Not every row of the sparse x dense product is formed: where som_norms has recorded the per-range
 * maxima (M % 128 == 0; by default on maps of at least 4096 neurons), the kernel leaves a sample out
 * of the search of a range of 128 neurons when even the range's smallest partial score over the sample's
 * most frequent features, lowered by the largest weights in the range of its other features, stays above
 * the sample's best score so far, with a margin for fp32 rounding: no neuron of the range can then be
 * the best unit.  A sample that stays in is tested once more, with the partial scores of its frequent
 * features exact for every neuron, before any row of its rare features is read.  The outputs are bit for bit
 * those of the search that forms every row (tests/test_gpu_parity.py forces it both ways).
 */
int som_bmu(som_handle* h, const int32_t* d_indptr, const int32_t* d_indices, int64_t n_samples,
            int32_t* d_bmu, float* d_min_dist, void* stream);

/*
 * som_bmu2 - som_bmu that also returns the second-best unit, found in the same sweep (the
 * paper's search kernel keeps the two best units of every sample: Section 3.3; Algorithm 2,
 * step 7; the second one feeds the topographic error, Section 3.5).
 *   d_bmu, d_min_dist   as in som_bmu.
 *   d_bmu2     DEVICE pointer, int32 [n_samples]  out: the neuron that comes second in the order
 *              (fp32 score, neuron index), i.e. the nearest neuron other than d_bmu, lowest
 *              index among exact fp32 ties; -1 when the map has a single neuron.
 *   d_dist2    DEVICE pointer, fp32 [n_samples]   out: its full squared distance, recomputed in
 *              fp64 and rounded once like d_min_dist; +inf when d_bmu2 is -1.
 * Same preconditions, asynchrony and determinism as som_bmu; with the two-stage search off (the
 * default) d_bmu/d_min_dist are bit-identical to som_bmu's for the same inputs (with option 7 the
 * two calls may send different samples to the exact pass, whose kernel sums in another order).
 */
int som_bmu2(som_handle* h, const int32_t* d_indptr, const int32_t* d_indices, int64_t n_samples,
             int32_t* d_bmu, float* d_min_dist, int32_t* d_bmu2, float* d_dist2, void* stream);

/*
 * som_plan_create / som_bmu_planned / som_plan_destroy - a reusable batch plan for epoch loops.
 * The per-batch preparation inside som_bmu (feature histogram, choice of the table's features, sort of the
 * samples, re-encoded index lists: the merged feature lists of a sample tile, Section 3.3) depends on the batch
 * alone, not on the codebook.  Training searches the same batches every epoch (Algorithm 2, step 2), so a
 * caller can build each batch's plan once:
 *   som_plan_create   builds the plan of the device-resident CSR batch (arguments as in som_bmu) in
 *                     device memory of its own (about 220 bytes per sample plus 70 MB, scratch of the
 *                     search included) and synchronises `stream`.
 *                     The plan BORROWS d_indptr / d_indices: they must stay valid and unchanged while
 *                     the plan lives.  It is tied to the handle and to the handle's options and
 *                     storage type at this moment.
 *   som_bmu_planned   som_bmu for the plan's batch: same outputs (bit-identical to som_bmu's on the same
 *                     batch with the same options), but only enqueues work on `stream` (no host
 *                     synchronisation, no allocation); it takes the two-stage search (option 7) like som_bmu.
 *                     Two searches with the same plan must not overlap on the GPU.
 *   som_plan_destroy  frees the plan (NULL is accepted); destroy plans before their handle.
 */
typedef struct som_plan som_plan; /* opaque */
int som_plan_create(som_handle* h, const int32_t* d_indptr, const int32_t* d_indices, int64_t n_samples,
                    som_plan** out, void* stream);
int som_bmu_planned(som_handle* h, som_plan* plan, int32_t* d_bmu, float* d_min_dist, void* stream);
int som_plan_destroy(som_plan* plan);

/*
 * som_bmu_values - the search for sparse REAL-VALUED samples (the paper's outlook, Section 7: a values
 * array beside the feature indices and the sample's own squared norm; its SparseFloat variant, Table 6):
 *   d_values   DEVICE pointer, fp32, parallel to d_indices: sample s has value d_values[k] at feature
 *              d_indices[k] for k in [d_indptr[s], d_indptr[s+1]) and 0 elsewhere.
 * BMU = argmin_i (||w_i||^2 - 2 * sum_k x_k * w_i[idx_k]), ties to the lowest index; d_min_dist is
 * ||x||^2 - 2<x,w> + ||w||^2, recomputed in fp64 for the winner.  With all values 1 the result is
 * som_bmu's.  The gather-sum becomes a gather-multiply (fused multiply-add, fp32), run by the
 * direct-load kernel only (the row-table plan is specific to binary samples); other arguments,
 * preconditions, asynchrony and determinism as in som_bmu.
 */
int som_bmu_values(som_handle* h, const int32_t* d_indptr, const int32_t* d_indices, const float* d_values,
                   int64_t n_samples, int32_t* d_bmu, float* d_min_dist, void* stream);

/*
 * som_update - the batch update that follows the search in an epoch (Section 3.4; Algorithm 2,
 * steps 8-9): scatter the samples onto the lattice (per cell the sum of its assigned samples
 * and their count), blur both fields with three unnormalised box passes per lattice axis of
 * half-width `radius` whose window is truncated at the lattice edge, and REPLACE every prototype
 * by the ratio; a neuron whose blurred count is zero keeps its prototype.  No learning rate.
 *   rows, cols   lattice shape, rows * cols == M; neuron i sits at row i / cols, column i % cols.
 *   d_indptr, d_indices, n_samples   the epoch's samples as in som_bmu (DEVICE CSR); an epoch
 *                searched in several batches passes their concatenation.
 *   d_bmu        DEVICE pointer, int32 [n_samples]: the best unit of every sample (som_bmu's output).
 *   radius       box half-width in cells, >= 0; the paper uses the schedule's sigma rounded to whole
 *                cells and never smaller than one (the caller applies the schedule).
 * WRITES the codebook the handle borrows, in place (fp32, or fp16 for som_create_f16: sums and the
 * blur are carried in fp32/fp64 and rounded to the storage type only at this final write), so
 * som_norms must run again before the next search.  Work is enqueued on `stream`; the features are
 * processed in slabs through the handle's workspace (option 6 bounds it), so no second V x M array
 * is needed.  The window sums are running sums (add the entering cell, subtract the leaving one):
 * constant work per cell whatever the radius, but a cell whose exact sum is many orders of
 * magnitude below the largest sum of its line inherits that line's rounding error (2^-53 relative
 * to the largest; the sums are carried in fp64).
 */
int som_update(som_handle* h, int32_t rows, int32_t cols, const int32_t* d_indptr, const int32_t* d_indices,
               int64_t n_samples, const int32_t* d_bmu, int32_t radius, void* stream);

/*
 * som_bmu_host - the same search with HOST buffers: copies the CSR batch to device staging
 * memory owned by the handle, runs som_bmu, copies both outputs back, all enqueued on
 * `stream`, then synchronises that stream before returning.  h_* pointers are host memory
 * (pinned memory makes the copies asynchronous and faster); h_indptr[0] must be 0.
 * The paper has the corpus stream from host memory into the kernels (Section 4.2).
 */
int som_bmu_host(som_handle* h, const int32_t* h_indptr, const int32_t* h_indices, int64_t n_samples,
                 int32_t* h_bmu, float* h_min_dist, void* stream);

/*
 * som_bmu_host_async / som_host_sync - som_bmu_host for a STREAM of batches: the call returns once the
 * batch's work is enqueued (it waits only for the staging buffer it reuses, i.e. for the results of
 * the call before the previous one to have left the device), and h_bmu / h_min_dist hold the results after som_host_sync(h).  The handle
 * keeps two staging buffers and two copy streams of its own, so the host-to-device copy of one batch
 * overlaps the search of the previous one and the results travel back while the next search runs
 * (the paper streams the corpus from host memory, Section 4.2).  The search itself runs on `stream`.
 * h_indptr / h_indices must stay unchanged until the NEXT call on the handle has returned (or
 * som_host_sync); the output buffers of up to two calls are in flight at a time.  Use pinned host
 * memory: pageable buffers make the copies synchronous and the overlap is lost.
 */
int som_bmu_host_async(som_handle* h, const int32_t* h_indptr, const int32_t* h_indices, int64_t n_samples,
                       int32_t* h_bmu, float* h_min_dist, void* stream);
int som_host_sync(som_handle* h);

/*
 * som_validate_csr - check the preconditions of som_bmu on a device-resident batch:
 * non-decreasing row pointers, ids in [0, V), strictly ascending inside each row
 * (Section 4.2, the sparse-binary CSR container).  Synchronises `stream`.
 * Returns SOM_OK or SOM_ERR_BAD_CSR.
 */
int som_validate_csr(som_handle* h, const int32_t* d_indptr, const int32_t* d_indices,
                     int64_t n_samples, void* stream);

/*
 * som_device_flags - what earlier calls on this handle skipped on the device.  (No counterpart in the
 * paper: error reporting of this library.)  Kernels never fault on a bad index they can see cheaply;
 * they skip the entry and set a sticky bit in a flag word on the device:
 *   - a feature id outside [0, V) met by the batch-plan kernels of som_bmu / som_plan_create or by
 *     som_update's frequent-feature pass             -> SOM_ERR_BAD_CSR
 *   - a best-unit index outside [0, M) in som_update's d_bmu (a stale buffer, the -1 that som_bmu2
 *     writes for a missing second unit): the sample is left out of the update -> SOM_ERR_INVALID_ARG
 * This call copies the word back, clears it, synchronises `stream` and returns SOM_OK or the
 * status above (SOM_ERR_BAD_CSR first when both bits are set).
 */
int som_device_flags(som_handle* h, void* stream);

/*
 * som_get_norms - copy the M fp32 norms computed by the last som_norms into a DEVICE buffer
 * (enqueued on `stream`).  For tests and for callers that want ||w_i||^2 (Eq. 1).
 */
int som_get_norms(som_handle* h, float* d_out, void* stream);

/*
 * som_norms_noalloc - ||w_i||^2 for all M neurons without a handle and without allocating.
 * (No counterpart in the paper: an integration convenience of this library.)
 *
 * For callers that must not call cudaMalloc: a process whose device memory already belongs
 * to its own pool, where a raw allocation can fail or fragment that pool, or a
 * latency-critical loop that cannot take the device-wide synchronisation an allocation may
 * imply.  som_norms keeps per-split partial sums in an allocated workspace; this variant
 * keeps them in a fixed 4 MiB array built into the library, which every GPU that loads the
 * library holds until the process exits.
 *   V, M        as in som_create, with M <= SOM_NOALLOC_MAX_M; a larger M returns
 *               SOM_ERR_UNSUPPORTED and nothing runs.
 *   d_codebook  DEVICE pointer, fp32, feature-major, V*M elements (borrowed, read only).
 *   d_norms     DEVICE pointer, fp32 [M], out: squared norms, fp64 accumulation rounded once.
 *   stream      the two kernels are enqueued on it; the call does not synchronise.
 * The first call on each device looks up the array's device address; make that first call
 * outside any stream capture.  All calls on a device share the array, which keeps the last
 * call's contents (nothing in it needs clearing: each call overwrites what it reads), so two
 * calls that may overlap on the GPU must be ordered by the caller or they race.
 * The device must be the current one; allocates nothing on host or device.
 */
#define SOM_NOALLOC_MAX_M 524288
int som_norms_noalloc(int32_t V, int64_t M, const float* d_codebook, float* d_norms, void* stream);

/* som_destroy - free the handle, its norms and workspace.  NULL is accepted. */
int som_destroy(som_handle* h);

/* Human-readable name of a status code (static storage). */
const char* som_status_string(int status);

/* cudaError_t value of the last failed CUDA call on this handle (0 if none). */
int som_last_cuda_error(const som_handle* h);

/*
 * Instrumentation (no paper counterpart; used by the benchmark).
 * som_set_timing(h, 1) makes each som_norms / som_bmu record CUDA events around its
 * phases on the caller's stream (switching it on or off restarts the record).
 * som_get_timing, called after the stream has been synchronised, returns the mean over the
 * calls recorded since then (the most recent 32 of each kind at most):
 *   out_ms[0] som_norms total, out_ms[1] som_bmu total, out_ms[2] som_bmu plan phase,
 *   out_ms[3] som_bmu search kernel(s), out_ms[4] som_bmu finalize.
 * som_launch_count returns how many kernels this handle has launched since creation.
 * som_set_option sets a per-handle option (SOM_ERR_INVALID_ARG for an unknown key or value):
 *   key 0  search kernel: 0 automatic (default), 1 direct-load kernel, 2 shared-memory row-table kernel (where
 *          M % 4 == 0 and V <= 65536).
 *   key 5  automatic selection: least percentage of the batch's feature instances that the row table's
 *          features must cover for the row-table kernel to be taken (0 = default 60; batches below it go to
 *          the direct-load kernel).
 *   key 6  workspace budget of som_update's slab buffers in MiB (0 = default 4096).
 *   key 7  two-stage search for fp32 storage (0 = off, the default; 1 = on): som_norms then also keeps an fp16
 *          copy of the codebook (V*M*2 more bytes of device memory, allocated by this call, which fails with
 *          SOM_ERR_CUDA if they cannot be had), the largest |weight|, the largest ||w||^2 and whether any weight
 *          is negative; som_bmu ranks the neurons by a first pass over that copy, keeps the result for every
 *          sample whose two best first-pass scores are further apart than a bound on what the fp16 rounding and
 *          the fp32 summation can change (then the best unit of the exact weights is provably the same one; the
 *          bound is tighter when no weight is negative), and searches the other samples again with the fp32
 *          weights.  som_bmu2 does the same with the three best first-pass scores (both units and their order
 *          certified).  Reported distances always come from the fp32 weights.  It pays on maps whose units are
 *          distinct at fp16 resolution (random initialisation, small final radius); on a map that a wide blur
 *          has just smoothed most samples fail the certificate.  A batch of at least 65536 samples is therefore
 *          probed first (one sample in 256, chosen by sample index): if more
 *          than a fifth of those fail, the call runs the plain search instead (on the same plan, i.e. with 8
 *          neurons per lane: bit-identical to a plain call with key 3 = 8).  Needs M % 128 == 0 and the
 *          row-table kernel.  A two-stage call only enqueues, like any other: the probe's verdict, the choice
 *          between the two-stage path and the plain search and the length of the second pass's list all stay on
 *          the device (the kernels of both paths are enqueued; those of the path not taken return at once; the
 *          second pass is run by the direct-load kernel, which reads the list's length on the device).
 *          som_last_uncertain returns how many samples the last two-stage search sent to its second pass (all
 *          of them when the probe chose the plain search); the figure travels back unwaited for and is valid
 *          once the call's stream has been synchronised.
 *   keys 1 to 4 and 8 to 10 are tunables of the row-table kernel and its plan for benchmarking (hot rows in shared
 *          memory, block size, neurons per lane, sample parts per neuron range, mask features, L2 policy of the slot stream, pruning by range maxima; 0 = the measured
 *          default): described in
 *          paper_2608_24067_b200/csrc/som_tuning.h.  Callers need not touch them; a plan (som_plan_create) is
 *          tied to their values at its creation.
 */
/*
 * som_measure_fadd_peak - measure the device's FP32 add rate (no counterpart in the paper: the
 * denominator of this library's roofline, measured instead of derived).  Launches a kernel of
 * independent add chains (eight per thread, 64 warps per SM) four times on `stream`, times the last
 * three with CUDA events and returns the best rate in *adds_per_s.  Synchronises.
 *   d_scratch      DEVICE pointer, fp32, at least 2048 * (number of SMs) elements; written.
 *   scratch_elems  its length.
 */
int som_measure_fadd_peak(double* adds_per_s, float* d_scratch, int64_t scratch_elems, void* stream);

/*
 * som_measure_operand_paths - measure how many bytes per clock and SM reach registers along the paths that an
 * add's operand takes in the row-table search kernel (no counterpart in the paper; Section 5.7 only says that
 * its kernel executes adds and no multiplies: what bounds such a kernel is operand delivery).  One block of 512
 * threads per SM reads 512-byte rows, eight lanes per row, as that kernel's wide fp32 layout does:
 *   bytes_per_clk[0]  rows of a 180 KB table in shared memory,
 *   bytes_per_clk[1]  rows of the caller's buffer with read-only global loads (L2-resident when the buffer is a
 *                     few tens of MB),
 *   bytes_per_clk[2]  both streams in one loop (the sum of both streams' bytes over the loop's time),
 *   bytes_per_clk[3]  the buffer's rows through a linear texture.
 * Times with the SM cycle counter, mean over the blocks.  Synchronises.
 *   n_out          length of bytes_per_clk, at least 4.
 *   d_rows         DEVICE pointer, 512-byte aligned, rows_bytes bytes (512 .. 2^31) of finite fp32 values; read.
 *   d_scratch      DEVICE pointer, fp32, at least 514 * (number of SMs) + 2 elements; written.
 */
int som_measure_operand_paths(double* bytes_per_clk, int n_out, const void* d_rows, int64_t rows_bytes,
                              float* d_scratch, int64_t scratch_elems, void* stream);

/*
 * som_tc_probe - measured probe of a densified hot-feature tile on the tensor cores (no counterpart in
 * the paper, whose kernels run on plain CUDA cores; Section 3.3 is the gather it restates).  For the H
 * most frequent features of a batch the gather-sum of a tile of 128 samples over 64 neurons is the dense
 * product of the samples' 0/1 membership matrix with those features' rows.  The probe runs that product on
 * tcgen05.mma (fp16 operands, fp32 accumulation in tensor memory) with the steps a fused search kernel
 * would need around it - building the 0/1 tile in shared memory from membership bits, the MMAs, draining
 * the accumulator into registers - and reports the clock cycles, so that the cost can be compared with the
 * shared-memory reads the product would replace.  The accumulator is seeded with ||w||^2 / 2 and the rows
 * are subtracted, i.e. it holds the samples' partial scores.
 *   d_rows     DEVICE, fp32 [H][64]: rows of the H dense features for one range of 64 neurons.
 *   d_hnorm    DEVICE, fp32 [64]: ||w||^2 / 2 of those neurons.
 *   d_bits     DEVICE, uint32 [n_tiles * 128][H / 32]: bit f % 32 of word f / 32 = sample has feature f.
 *   H          32 ... 256, a multiple of 32.   terms: fp16 terms per weight, 1 (rounded) or 2 (hi + lo).
 *   mode       bit 0 build the 0/1 tile for every tile (else only the first two), bit 1 issue the MMAs,
 *              bit 2 drain the accumulators, bit 3 also redistribute the drained values by shuffles to
 *              eight threads per sample, bit 4 the drain warps also stream 1024 wavefronts of 128-bit
 *              shared-memory reads per tile (to see whether they and the MMAs' operand fetch contend).
 *   repeats    every block walks the n_tiles tiles this many times; blocks: thread blocks (one per SM).
 *   d_out      DEVICE, fp32 [128][64] or NULL: partial scores of the first tile (written by block 0).
 *   d_mins     DEVICE, fp32 [blocks][128] or NULL: per-sample minimum score of the last tile walked.
 *   d_cycles   DEVICE, int64 [blocks]: clock cycles of each block's loop.
 *   d_status   DEVICE, int: 0, or 1 if a bounded wait inside the kernel gave up (results invalid).
 * Enqueues one kernel on `stream`; does not synchronise.
 */
int som_tc_probe(const float* d_rows, const float* d_hnorm, const uint32_t* d_bits, int32_t H, int32_t terms,
                 int32_t n_tiles, int32_t mode, int32_t repeats, int32_t blocks, float* d_out, float* d_mins,
                 long long* d_cycles, int* d_status, void* stream);

int som_set_timing(som_handle* h, int enable);
int som_get_timing(som_handle* h, float* out_ms, int n_out);
int64_t som_launch_count(const som_handle* h);
int64_t som_last_uncertain(const som_handle* h);
int som_set_option(som_handle* h, int key, int64_t value);

#ifdef __cplusplus
}
#endif
#endif /* SOM_B200_H */
