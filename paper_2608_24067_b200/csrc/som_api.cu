// Host side of the C ABI declared in include/som.h: handle life cycle, argument checks,
// workspace management, phase timing and kernel selection.  All compute is in the kernels.
#include <new>

#include "som_internal.cuh"
#include "som_plan.cuh"

namespace {

struct DeviceGuard {
    int prev;
    bool switched;
    explicit DeviceGuard(int dev) : prev(-1), switched(false)
    {
        if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) {
            cudaSetDevice(dev);
            switched = true;
        }
    }
    ~DeviceGuard()
    {
        if (switched) cudaSetDevice(prev);
    }
};

int ensure_bytes(som_handle* h, void** buf, size_t* have, size_t need)
{
    if (need <= *have) return SOM_OK;
    if (*buf) {
        SOM_CK(h, cudaFree(*buf));  // synchronises: earlier work using the buffer is done
        *buf = nullptr;
        *have = 0;
    }
    need = som_align_up(need + need / 8, 1 << 20);
    SOM_CK(h, cudaMalloc(buf, need));
    *have = need;
    return SOM_OK;
}

int ensure_events(som_handle* h)
{
    if (h->events_made) return SOM_OK;
    for (int i = 0; i < SOM_N_EVENTS; ++i) SOM_CK(h, cudaEventCreate(&h->ev[i]));
    h->events_made = 1;
    return SOM_OK;
}

// Events live in a ring of SOM_EV_RING calls so that the mean over a timed region can be read
// after one synchronisation at its end.
inline int mark(som_handle* h, int64_t call, int slot, cudaStream_t st)
{
    if (!h->timing) return SOM_OK;
    SOM_CK(h, cudaEventRecord(h->ev[(call % SOM_EV_RING) * SOM_EV_PER_CALL + slot], st));
    return SOM_OK;
}

// Hands the device-side kernel choice to the launchers for the length of a scope.
struct GateScope {
    som_handle* h;
    GateScope(som_handle* h_, const int* gate) : h(h_)
    {
        h->gate = gate;
        h->gate_want = SOM_GATE_TABLE;
    }
    ~GateScope()
    {
        h->gate = nullptr;
        h->gate_want = 0;
    }
};

}  // namespace

extern "C" {

static int create_impl(som_handle** out, int32_t V, int64_t M, const void* d_codebook, bool f16)
{
    if (!out) return SOM_ERR_INVALID_ARG;
    *out = nullptr;
    if (V <= 0 || M <= 0 || !d_codebook) return SOM_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(d_codebook) & 15u) != 0) return SOM_ERR_INVALID_ARG;
    if (M >= (int64_t)1 << 31) return SOM_ERR_UNSUPPORTED;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return SOM_ERR_NO_DEVICE;
    int major = 0, sms = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return SOM_ERR_NO_DEVICE;
    if (major != 10) return SOM_ERR_NO_DEVICE;  // the kernels are built for sm_100a only

    som_handle* h = new (std::nothrow) som_handle();
    if (!h) return SOM_ERR_INVALID_ARG;
    h->device = dev;
    h->sm_count = sms;
    h->V = V;
    h->M = M;
    h->W = f16 ? nullptr : static_cast<const float*>(d_codebook);
    h->Wh = f16 ? static_cast<const __half*>(d_codebook) : nullptr;
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&h->norm64), (size_t)M * sizeof(double));
    if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&h->norm32), (size_t)M * sizeof(float));
    if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&h->hnorm), (size_t)M * sizeof(float));
    if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&h->dev_flags), 256);
    if (e == cudaSuccess) e = cudaMemset(h->dev_flags, 0, 256);
    if (e != cudaSuccess) {
        som_destroy(h);
        return SOM_ERR_CUDA;
    }
    *out = h;
    return SOM_OK;
}

int som_create(som_handle** out, int32_t V, int64_t M, const float* d_codebook)
{
    return create_impl(out, V, M, d_codebook, false);
}

int som_create_f16(som_handle** out, int32_t V, int64_t M, const void* d_codebook_f16)
{
    return create_impl(out, V, M, d_codebook_f16, true);
}

int som_destroy(som_handle* h)
{
    if (!h) return SOM_OK;
    DeviceGuard g(h->device);
    cudaFree(h->norm64);
    cudaFree(h->norm32);
    cudaFree(h->hnorm);
    cudaFree(h->dev_flags);
    cudaFree(h->ws);
    cudaFree(h->stage);
    cudaFree(h->head);
    cudaFree(h->shadow);
    cudaFree(h->range_max);
    cudaFree(h->range_order);
    if (h->aux_stream) {
        cudaStreamSynchronize(h->aux_stream);
        cudaEventDestroy(h->ev_fork);
        cudaEventDestroy(h->ev_join);
        cudaStreamDestroy(h->aux_stream);
    }
    if (h->copy_stream) {
        cudaStreamSynchronize(h->copy_stream);
        cudaStreamSynchronize(h->back_stream);
        for (int t = 0; t < 2; ++t) {
            cudaEventDestroy(h->ev_h2d[t]);
            cudaEventDestroy(h->ev_searched[t]);
            cudaEventDestroy(h->ev_d2h[t]);
            cudaFree(h->pipe_stage[t]);
        }
        cudaStreamDestroy(h->copy_stream);
        cudaStreamDestroy(h->back_stream);
    }
    cudaFree(h->wmax_bits);
    if (h->host_pair) cudaFreeHost(h->host_pair);
    if (h->events_made)
        for (int i = 0; i < SOM_N_EVENTS; ++i) cudaEventDestroy(h->ev[i]);
    delete h;
    return SOM_OK;
}

int som_norms(som_handle* h, void* stream)
{
    if (!h) return SOM_ERR_INVALID_ARG;
    DeviceGuard g(h->device);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    int rc = ensure_bytes(h, &h->ws, &h->ws_bytes, som_norms_workspace_bytes(h));
    if (rc) return rc;
    if (h->timing && (rc = ensure_events(h))) return rc;
    // per-range maxima of the feature rows for the search's pruning (M % 128 == 0): V * M / 32
    // floats, allocated by the first call; without the memory the search simply does not prune
    if (!h->range_max && h->M % 128 == 0 && h->opt_prune != 2) {
        if (cudaMalloc(reinterpret_cast<void**>(&h->range_max), (size_t)h->V * (size_t)(h->M / 32) * sizeof(float)) !=
            cudaSuccess) {
            h->range_max = nullptr;
            (void)cudaGetLastError();
        } else if (h->M / 128 <= 8192 &&  // (the order of the ranges: what one block sorts in shared memory)
                   cudaMalloc(reinterpret_cast<void**>(&h->range_order), (size_t)(h->M / 128) * sizeof(int32_t)) !=
                       cudaSuccess) {
            h->range_order = nullptr;
            (void)cudaGetLastError();
        }
    }
    if ((rc = mark(h, h->ev_norms_calls, EV_NORMS_BEGIN, st))) return rc;
    if ((rc = som_launch_norms(h, st))) return rc;
    h->shadow_valid = h->shadow != nullptr && h->M % 4 == 0;
    if ((rc = mark(h, h->ev_norms_calls, EV_NORMS_END, st))) return rc;
    if (h->timing) h->ev_norms_calls += 1;
    h->norms_valid = 1;
    return SOM_OK;
}

// Samples that do not fit a slot of the row-table plan (more than 10 tail features, counting the hot features beyond 12 among them; the plan
// lists them, the row-table kernel skips them): the direct-load kernel searches the list, whose length
// only the device knows, and their outputs are written last.  Two small launches that return at once
// when the list is empty.
static int rare_pass(som_handle* h, const int32_t* indptr, const int32_t* indices, int64_t n, char* head, char* ws,
                     const SomPlanBuffers& pb, int32_t* bmu, float* dist, int32_t* bmu2, float* dist2,
                     cudaStream_t st)
{
    const bool top2 = bmu2 != nullptr;
    unsigned long long* rk = reinterpret_cast<unsigned long long*>(ws + pb.rare_keys);
    unsigned long long* rk2 = top2 ? reinterpret_cast<unsigned long long*>(ws + pb.rare_keys2) : nullptr;
    const int32_t* list = reinterpret_cast<const int32_t*>(ws + pb.rare_list);
    const size_t kb = (size_t)(n + 16) * sizeof(unsigned long long);
    SOM_CK(h, cudaMemsetAsync(rk, 0xFF, kb, st));
    if (top2) SOM_CK(h, cudaMemsetAsync(rk2, 0xFF, kb, st));
    h->list_len_dev = reinterpret_cast<const int*>(head + pb.n_slots) + SOM_PLAN_RARE;
    int rc = som_launch_bmu_direct(h, indptr, indices, n, rk, rk2, list, st);
    if (!rc) rc = som_launch_finalize(h, indptr, indices, n, rk, bmu, dist, list, st);
    if (!rc && top2) rc = som_launch_finalize(h, indptr, indices, n, rk2, bmu2, dist2, list, st);
    h->list_len_dev = nullptr;
    return rc;
}

// The two-stage search on a batch whose plan (slots in ws, table features in head) is ready: first
// pass over the fp16 shadow keeping the two (som_bmu2: three) best units, certificate, exact fp32
// pass for the samples it leaves open.  Everything is enqueued; nothing is read back.  `gate` is the
// device word that says which path this batch takes: the probe and the decision kernel may raise it from
// 1 (row-table kernel) to 2 (row-table kernel, two-stage search); the kernels enqueued here for the
// two-stage path run only then, and the caller enqueues the plain search for the other case.
// Key arrays (keys, keys2, keys3) must have been cleared by the caller.
static int two_stage_enqueue(som_handle* h, const int32_t* indptr, const int32_t* indices, int64_t n, char* head,
                             char* ws, const SomPlanBuffers& pb, int n_hot, int32_t* bmu, float* dist,
                             int32_t* bmu2, float* dist2, cudaStream_t st)
{
    int rc = SOM_OK;
    const bool top2 = bmu2 != nullptr;
    int* counters = reinterpret_cast<int*>(head + pb.n_slots);
    int32_t* uncertain = reinterpret_cast<int32_t*>(ws + pb.uncertain);
    int* n_unc_dev = counters + SOM_PLAN_UNCERTAIN;
    SOM_CK(h, cudaMemsetAsync(counters + 3, 0, sizeof(int), st));   // search unit counter
    SOM_CK(h, cudaMemsetAsync(n_unc_dev, 0, sizeof(int), st));      // length of the uncertain list

    // Probe.  On a map whose neighbouring units differ by less than fp16 resolves (one that a wide
    // blur has just smoothed) most samples fail the certificate, and a first pass over the whole
    // batch is wasted.  So one sample in SOM_PROBE_STRIDE goes through first pass and certificate
    // first (count only); the decision kernel sends the batch to the plain fp32 search if more than a
    // fifth of those fail.
    int n_probe = 0;
    h->gate_want = SOM_GATE_TABLE;
    if (n >= SOM_PROBE_MIN_BATCH) {
        n_probe = (int)((n + SOM_PROBE_STRIDE - 1) / SOM_PROBE_STRIDE);
        const size_t pkb = (size_t)(n_probe + 16) * sizeof(unsigned long long);
        SomPlanBuffers pp = pb;
        pp.slots = pb.slots2;
        pp.order = pb.uncertain;
        pp.keys = pb.ukeys;
        pp.keys2 = pb.ukeys2;
        pp.keys3 = pb.rare_keys;  // (free until the rare pass at the end of the call)
        SOM_CK(h, cudaMemsetAsync(ws + pp.keys, 0xFF, pkb, st));
        SOM_CK(h, cudaMemsetAsync(ws + pp.keys2, 0xFF, pkb, st));
        if (top2) SOM_CK(h, cudaMemsetAsync(ws + pp.keys3, 0xFF, pkb, st));
        if ((rc = som_launch_probe_gather(h, n, ws, pb, st))) return rc;
        if ((rc = som_launch_pad_slots(h, ws, pb.slots2, n_probe, st))) return rc;
        // (enough sample parts per neuron range that the short launch still occupies every SM)
        const SomTableGeom first = som_table_geometry(h, true);
        const int64_t n_ranges = (h->M + first.T - 1) / first.T;
        const int64_t saved_parts = h->opt_parts;
        h->opt_parts = (2 * (int64_t)h->sm_count + n_ranges - 1) / n_ranges;
        rc = som_launch_bmu_table(h, true, indptr, indices, n_probe, head, ws, pp, n_hot, top2 ? 3 : 2, st);
        h->opt_parts = saved_parts;
        if (rc) return rc;
        if ((rc = som_launch_certify(h, indptr, indices, n_probe, ws, pp, top2, true, nullptr, nullptr, nullptr,
                                     nullptr, nullptr, n_unc_dev, st)))
            return rc;
    }
    if ((rc = som_launch_two_stage_decide(h, head, pb, n_probe, n, st))) return rc;
    SOM_CK(h, cudaMemsetAsync(counters + 3, 0, sizeof(int), st));

    // ---- the two-stage path proper: runs when the gate word is 2 -------------------------------------
    h->gate_want = SOM_GATE_TABLE_TS;
    if ((rc = som_launch_bmu_table(h, true, indptr, indices, n, head, ws, pb, n_hot, top2 ? 3 : 2, st))) return rc;
    // certificate; certain samples are finalised, the others listed
    if ((rc = som_launch_certify(h, indptr, indices, n, ws, pb, top2, false, bmu, dist, bmu2, dist2, uncertain,
                                 n_unc_dev, st)))
        return rc;
    // exact pass over the listed samples: fp32 weights, all neurons, by the direct-load kernel, which reads
    // the length of the list on the device
    unsigned long long* ukeys = reinterpret_cast<unsigned long long*>(ws + pb.ukeys);
    unsigned long long* ukeys2 = top2 ? reinterpret_cast<unsigned long long*>(ws + pb.ukeys2) : nullptr;
    const size_t ub = (size_t)(n + 16) * sizeof(unsigned long long);
    SOM_CK(h, cudaMemsetAsync(ukeys, 0xFF, ub, st));
    if (top2) SOM_CK(h, cudaMemsetAsync(ukeys2, 0xFF, ub, st));
    h->list_len_dev = n_unc_dev;
    rc = som_launch_bmu_direct(h, indptr, indices, n, ukeys, ukeys2, uncertain, st);
    if (!rc) rc = som_launch_finalize(h, indptr, indices, n, ukeys, bmu, dist, uncertain, st);
    if (!rc && top2) rc = som_launch_finalize(h, indptr, indices, n, ukeys2, bmu2, dist2, uncertain, st);
    h->list_len_dev = nullptr;
    if (rc) return rc;
    // what som_last_uncertain reports travels to pinned host words, unwaited for
    SOM_CK(h, cudaMemcpyAsync(h->host_pair, counters + SOM_PLAN_REPORT, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    SOM_CK(h, cudaMemcpyAsync(h->host_pair + 1, n_unc_dev, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    h->last_uncertain = -1;  // (read from the pinned words on demand)
    return SOM_OK;
}

// The search behind som_bmu (d_bmu2 == nullptr) and som_bmu2 (both second-best outputs given).
static int bmu_impl(som_handle* h, const int32_t* d_indptr, const int32_t* d_indices, int64_t n_samples,
                    int32_t* d_bmu, float* d_min_dist, int32_t* d_bmu2, float* d_dist2, void* stream)
{
    if (!h || n_samples < 0) return SOM_ERR_INVALID_ARG;
    if (n_samples == 0) return SOM_OK;
    if (!d_indptr || !d_bmu || !d_min_dist) return SOM_ERR_INVALID_ARG;
    const bool top2 = d_bmu2 != nullptr;
    // (d_indices may be null only for a batch whose rows are all empty: no kernel dereferences it then)
    if (n_samples >= (int64_t)1 << 31) return SOM_ERR_UNSUPPORTED;
    if (!h->norms_valid) return SOM_ERR_NORMS_STALE;
    DeviceGuard g(h->device);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);

    int rc = SOM_OK;
    if (h->timing && (rc = ensure_events(h))) return rc;

    // Two-stage search (option 7, fp32 storage): a first pass over the fp16 shadow of the
    // codebook with the wide fp16 layout, a certificate per sample, an exact fp32 pass for the
    // samples that fail it.  It needs the shadow written by the last som_norms and the row-table
    // kernel; the two-best search keeps the three best of the first pass (the certificate for the
    // second unit needs the third).
    const bool two_stage_ok = h->opt_two_stage == 1 && h->shadow && h->shadow_valid && !h->Wh &&
                              h->M % 128 == 0;
    // Kernel selection.  The row-table kernel needs 128-bit aligned row segments (M % 4 == 0;
    // M % 64 == 0 with fp16 storage), feature ids that fit its 16-bit codes (V <= 65536) and
    // enough (neuron range x sample part) units to occupy every SM; everything else goes to
    // the direct-load kernel.  So do, in automatic mode, batches whose most frequent features
    // cover too few feature instances for a shared-memory table to pay: there the direct-load
    // kernel, bound by L2 bandwidth alone, is faster (measured cross-over: between a half and
    // two thirds of the instances).
    const SomTableGeom geom = som_table_geometry(h, two_stage_ok);
    bool use_table = h->opt_variant != 1 && (h->M % (h->Wh ? 64 : 4) == 0) && h->V <= 65536 &&
                     h->M < ((int64_t)1 << 30);
    if (use_table && h->opt_variant == 0) {
        const int64_t parts = som_table_default_parts(n_samples, geom.T, geom.row_bytes);
        const int64_t units = ((h->M + geom.T - 1) / geom.T) * parts;
        if (units < 2 * (int64_t)h->sm_count) use_table = false;
    }
    SomPlanBuffers pb;
    char* head = nullptr;
    bool begun = false;
    const int* gate = nullptr;  // device-side choice between the search paths
    bool table_hint = true;     // what an earlier call's batch chose (automatic mode)
    if (use_table) {
        const size_t head_need = som_plan_head_bytes(h->V, SOM_PLAN_MASK_FEATURES + geom.n_hot, &pb);
        if ((rc = ensure_bytes(h, &h->head, &h->head_bytes, head_need))) return rc;
        head = reinterpret_cast<char*>(h->head);
        if (!h->host_pair) {
            SOM_CK(h, cudaMallocHost(reinterpret_cast<void**>(&h->host_pair), 4 * sizeof(int32_t)));
            h->host_pair[0] = h->host_pair[1] = 0;
            h->host_pair[2] = 1;
        }
        if ((rc = mark(h, h->ev_bmu_calls, EV_BMU_BEGIN, st))) return rc;
        begun = true;
        // The selection phase of the plan: feature histogram, choice of the table's features and of the
        // kernel (in automatic mode the table must serve enough of the batch's feature instances; a forced
        // row-table kernel always gets 1), written to the gate word on the device.
        const int64_t saved_cover = h->opt_cover;
        if (h->opt_variant == 2) h->opt_cover = -1;  // (coverage threshold of zero percent)
        rc = som_launch_plan_select(h, d_indptr, d_indices, n_samples, head, pb, SOM_PLAN_MASK_FEATURES, geom.n_hot, st);
        h->opt_cover = saved_cover;
        if (rc) return rc;
        const int32_t* counters = reinterpret_cast<const int32_t*>(head + pb.n_slots);
        // Everything stays on the device: the kernels of every path are enqueued, and those of the paths
        // not chosen return at once.  The host never waits for the batch.  (A forced row-table kernel
        // without the two-stage search has one path only and needs no gate.)
        if (h->opt_variant == 0 || two_stage_ok) gate = counters + SOM_PLAN_USE_TABLE;
        if (h->opt_variant == 0) {
            // The choice also travels to a pinned host word, unwaited for: a later call reads what an
            // earlier call chose (batches of one stream mostly agree) and gives the launch it expects to
            // be idle a small grid.  Only the cost of a wrong guess depends on it, never the result.
            table_hint = *reinterpret_cast<volatile int32_t*>(h->host_pair + 2) != 0;
            SOM_CK(h, cudaMemcpyAsync(h->host_pair + 2, counters + SOM_PLAN_USE_TABLE, sizeof(int32_t),
                                      cudaMemcpyDeviceToHost, st));
        }
    }

    if (!use_table) {
        const size_t key_bytes = som_align_up((size_t)n_samples * sizeof(unsigned long long), 256);
        if ((rc = ensure_bytes(h, &h->ws, &h->ws_bytes, 2 * key_bytes))) return rc;
        unsigned long long* keys = reinterpret_cast<unsigned long long*>(h->ws);
        unsigned long long* keys2 = top2 ? keys + key_bytes / sizeof(unsigned long long) : nullptr;
        if (!begun && (rc = mark(h, h->ev_bmu_calls, EV_BMU_BEGIN, st))) return rc;
        SOM_CK(h, cudaMemsetAsync(keys, 0xFF, top2 ? 2 * key_bytes : key_bytes, st));
        if ((rc = mark(h, h->ev_bmu_calls, EV_BMU_PLAN_END, st))) return rc;
        if ((rc = som_launch_bmu_direct(h, d_indptr, d_indices, n_samples, keys, keys2, nullptr, st))) return rc;
        if ((rc = mark(h, h->ev_bmu_calls, EV_BMU_SEARCH_END, st))) return rc;
        if ((rc = som_launch_finalize(h, d_indptr, d_indices, n_samples, keys, d_bmu, d_min_dist, nullptr, st)))
            return rc;
        if (top2 &&
            (rc = som_launch_finalize(h, d_indptr, d_indices, n_samples, keys2, d_bmu2, d_dist2, nullptr, st)))
            return rc;
    } else {
        const size_t need = som_plan_workspace_bytes(n_samples, &pb);
        if ((rc = ensure_bytes(h, &h->ws, &h->ws_bytes, need))) return rc;
        char* ws = reinterpret_cast<char*>(h->ws);
        unsigned long long* keys = reinterpret_cast<unsigned long long*>(ws + pb.keys);
        unsigned long long* keys2 = reinterpret_cast<unsigned long long*>(ws + pb.keys2);
        const size_t kb = (size_t)(n_samples + 16) * sizeof(unsigned long long);
        SOM_CK(h, cudaMemsetAsync(keys, 0xFF, kb, st));
        if (top2 || two_stage_ok) SOM_CK(h, cudaMemsetAsync(keys2, 0xFF, kb, st));
        if (top2 && two_stage_ok) SOM_CK(h, cudaMemsetAsync(ws + pb.keys3, 0xFF, kb, st));
        GateScope scope(h, gate);  // the plan: runs when a row-table path is chosen (or there is no gate)
        if ((rc = som_launch_plan_sort(h, d_indptr, d_indices, n_samples, head, ws, pb, SOM_PLAN_MASK_FEATURES,
                                       geom.n_hot, st)))
            return rc;
        if ((rc = mark(h, h->ev_bmu_calls, EV_BMU_PLAN_END, st))) return rc;
        if (two_stage_ok &&
            (rc = two_stage_enqueue(h, d_indptr, d_indices, n_samples, head, ws, pb, geom.n_hot, d_bmu, d_min_dist,
                                    d_bmu2, d_dist2, st)))
            return rc;
        // plain row-table search (with the two-stage search enabled: only when the gate word stayed at 1)
        h->gate_want = two_stage_ok ? SOM_GATE_TABLE_PLAIN : SOM_GATE_TABLE;
        if ((rc = som_launch_bmu_table(h, false, d_indptr, d_indices, n_samples, head, ws, pb, geom.n_hot,
                                       top2 ? 2 : 1, st)))
            return rc;
        if (gate && h->opt_variant == 0) {
            // direct-load path on the same key arrays (indexed by sample there): runs when the choice is 0
            h->gate_want = SOM_GATE_DIRECT;
            h->gate_small_grid = table_hint ? 1 : 0;
            rc = som_launch_bmu_direct(h, d_indptr, d_indices, n_samples, keys, top2 ? keys2 : nullptr, nullptr, st);
            h->gate_small_grid = 0;
            if (rc) return rc;
        }
        if ((rc = mark(h, h->ev_bmu_calls, EV_BMU_SEARCH_END, st))) return rc;
        h->gate_want = two_stage_ok ? SOM_GATE_TABLE_PLAIN : SOM_GATE_TABLE;
        if ((rc = som_launch_finalize_sorted(h, d_indptr, d_indices, n_samples, ws, pb, false, d_bmu,
                                             d_min_dist, st)))
            return rc;
        if (top2 && (rc = som_launch_finalize_sorted(h, d_indptr, d_indices, n_samples, ws, pb, true, d_bmu2,
                                                     d_dist2, st)))
            return rc;
        h->gate_want = SOM_GATE_TABLE;
        if ((rc = rare_pass(h, d_indptr, d_indices, n_samples, head, ws, pb, d_bmu, d_min_dist, d_bmu2, d_dist2, st)))
            return rc;
        if (gate && h->opt_variant == 0) {
            h->gate_want = SOM_GATE_DIRECT;
            if ((rc = som_launch_finalize(h, d_indptr, d_indices, n_samples, keys, d_bmu, d_min_dist, nullptr, st)))
                return rc;
            if (top2 &&
                (rc = som_launch_finalize(h, d_indptr, d_indices, n_samples, keys2, d_bmu2, d_dist2, nullptr, st)))
                return rc;
        }
    }
    if ((rc = mark(h, h->ev_bmu_calls, EV_BMU_END, st))) return rc;
    if (h->timing) h->ev_bmu_calls += 1;
    return SOM_OK;
}

int som_bmu(som_handle* h, const int32_t* d_indptr, const int32_t* d_indices, int64_t n_samples,
            int32_t* d_bmu, float* d_min_dist, void* stream)
{
    return bmu_impl(h, d_indptr, d_indices, n_samples, d_bmu, d_min_dist, nullptr, nullptr, stream);
}

int som_bmu2(som_handle* h, const int32_t* d_indptr, const int32_t* d_indices, int64_t n_samples,
             int32_t* d_bmu, float* d_min_dist, int32_t* d_bmu2, float* d_dist2, void* stream)
{
    if (n_samples > 0 && (!d_bmu2 || !d_dist2)) return SOM_ERR_INVALID_ARG;
    return bmu_impl(h, d_indptr, d_indices, n_samples, d_bmu, d_min_dist, d_bmu2, d_dist2, stream);
}

int som_bmu_values(som_handle* h, const int32_t* d_indptr, const int32_t* d_indices, const float* d_values,
                   int64_t n_samples, int32_t* d_bmu, float* d_min_dist, void* stream)
{
    if (!h || n_samples < 0) return SOM_ERR_INVALID_ARG;
    if (n_samples == 0) return SOM_OK;
    if (!d_indptr || !d_indices || !d_values || !d_bmu || !d_min_dist) return SOM_ERR_INVALID_ARG;
    if (n_samples >= (int64_t)1 << 31) return SOM_ERR_UNSUPPORTED;
    if (!h->norms_valid) return SOM_ERR_NORMS_STALE;
    DeviceGuard g(h->device);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const size_t key_bytes = som_align_up((size_t)n_samples * sizeof(unsigned long long), 256);
    int rc = ensure_bytes(h, &h->ws, &h->ws_bytes, key_bytes);
    if (rc) return rc;
    unsigned long long* keys = reinterpret_cast<unsigned long long*>(h->ws);
    if (h->timing && (rc = ensure_events(h))) return rc;
    if ((rc = mark(h, h->ev_bmu_calls, EV_BMU_BEGIN, st))) return rc;
    SOM_CK(h, cudaMemsetAsync(keys, 0xFF, key_bytes, st));
    if ((rc = mark(h, h->ev_bmu_calls, EV_BMU_PLAN_END, st))) return rc;
    if ((rc = som_launch_bmu_values(h, d_indptr, d_indices, d_values, n_samples, keys, st))) return rc;
    if ((rc = mark(h, h->ev_bmu_calls, EV_BMU_SEARCH_END, st))) return rc;
    if ((rc = som_launch_finalize_values(h, d_indptr, d_indices, d_values, n_samples, keys, d_bmu, d_min_dist, st)))
        return rc;
    if ((rc = mark(h, h->ev_bmu_calls, EV_BMU_END, st))) return rc;
    if (h->timing) h->ev_bmu_calls += 1;
    return SOM_OK;
}

// ---- reusable batch plan ---------------------------------------------------------------------
// The plan of a batch (hot set, sort, slots) depends on the batch alone, not on the codebook, so an
// epoch loop that searches the same batches every epoch builds each plan once.
struct som_plan {
    som_handle* h;
    int device;              // its own copy: the plan may outlive the handle until it is destroyed
    const int32_t* indptr;   // borrowed
    const int32_t* indices;  // borrowed
    int64_t n, nnz;
    int use_table;
    int n_hot;
    int f16;                 // storage layout the plan was built for
    SomPlanBuffers pb;
    char* head;
    char* ws;                // table path: the plan's arrays; direct path: the keys
};

int som_plan_destroy(som_plan* p)
{
    if (!p) return SOM_OK;
    DeviceGuard g(p->device);
    cudaFree(p->head);
    cudaFree(p->ws);
    delete p;
    return SOM_OK;
}

int som_plan_create(som_handle* h, const int32_t* d_indptr, const int32_t* d_indices, int64_t n_samples,
                    som_plan** out, void* stream)
{
    if (!out) return SOM_ERR_INVALID_ARG;
    *out = nullptr;
    if (!h || n_samples <= 0 || !d_indptr) return SOM_ERR_INVALID_ARG;
    if (n_samples >= (int64_t)1 << 31) return SOM_ERR_UNSUPPORTED;
    DeviceGuard g(h->device);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    som_plan* p = new (std::nothrow) som_plan();
    if (!p) return SOM_ERR_INVALID_ARG;
    p->h = h;
    p->device = h->device;
    p->indptr = d_indptr;
    p->indices = d_indices;
    p->n = n_samples;
    p->f16 = h->Wh != nullptr;
    int rc = SOM_OK;
    // the same choice of kernel as som_bmu makes (see there)
    const SomTableGeom geom = som_table_geometry(h, false);
    p->n_hot = geom.n_hot;
    bool use_table = h->opt_variant != 1 && (h->M % (h->Wh ? 64 : 4) == 0) && h->V <= 65536 &&
                     h->M < ((int64_t)1 << 30);
    if (use_table && h->opt_variant == 0) {
        const int64_t units = ((h->M + geom.T - 1) / geom.T) * som_table_default_parts(n_samples, geom.T, geom.row_bytes);
        if (units < 2 * (int64_t)h->sm_count) use_table = false;
    }
    if (!h->host_pair && cudaMallocHost(reinterpret_cast<void**>(&h->host_pair), 4 * sizeof(int32_t)) != cudaSuccess)
        rc = SOM_ERR_CUDA;
    if (!rc && use_table) {
        const size_t head_need = som_plan_head_bytes(h->V, SOM_PLAN_MASK_FEATURES + geom.n_hot, &p->pb);
        if (cudaMalloc(reinterpret_cast<void**>(&p->head), head_need) != cudaSuccess) rc = SOM_ERR_CUDA;
        if (!rc) rc = som_launch_plan_select(h, d_indptr, d_indices, n_samples, p->head, p->pb,
                                             SOM_PLAN_MASK_FEATURES, geom.n_hot, st);
    }
    if (!rc) {
        cudaError_t e = cudaMemcpyAsync(h->host_pair, d_indptr, sizeof(int32_t), cudaMemcpyDeviceToHost, st);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(h->host_pair + 1, d_indptr + n_samples, sizeof(int32_t), cudaMemcpyDeviceToHost, st);
        h->host_pair[2] = 0;
        if (e == cudaSuccess && use_table)
            e = cudaMemcpyAsync(h->host_pair + 2,
                                reinterpret_cast<const int32_t*>(p->head + p->pb.n_slots) + SOM_PLAN_COVERED,
                                sizeof(int32_t), cudaMemcpyDeviceToHost, st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
        if (e != cudaSuccess) rc = SOM_ERR_CUDA;
    }
    if (!rc) {
        p->nnz = (int64_t)h->host_pair[1] - (int64_t)h->host_pair[0];
        if (p->nnz < 0 || (p->nnz > 0 && !d_indices)) rc = SOM_ERR_INVALID_ARG;
    }
    if (!rc && use_table) {
        const int64_t cover_pct = h->opt_cover > 0 ? h->opt_cover : 60;
        if (h->opt_variant == 0 && (int64_t)h->host_pair[2] * 100 < cover_pct * p->nnz) use_table = false;
    }
    if (!rc) {
        p->use_table = use_table ? 1 : 0;
        const size_t need = use_table ? som_plan_workspace_bytes(n_samples, &p->pb)
                                      : som_align_up((size_t)n_samples * sizeof(unsigned long long), 256);
        if (cudaMalloc(reinterpret_cast<void**>(&p->ws), need) != cudaSuccess) rc = SOM_ERR_CUDA;
        if (!rc && use_table)
            rc = som_launch_plan_sort(h, d_indptr, d_indices, n_samples, p->head, p->ws, p->pb,
                                      SOM_PLAN_MASK_FEATURES, geom.n_hot, st);
    }
    if (rc) {
        if (rc == SOM_ERR_CUDA && !h->last_cuda_error) h->last_cuda_error = (int)cudaGetLastError();
        som_plan_destroy(p);
        return rc;
    }
    *out = p;
    return SOM_OK;
}

int som_bmu_planned(som_handle* h, som_plan* p, int32_t* d_bmu, float* d_min_dist, void* stream)
{
    if (!h || !p || p->h != h || !d_bmu || !d_min_dist) return SOM_ERR_INVALID_ARG;
    if (!h->norms_valid) return SOM_ERR_NORMS_STALE;
    if (p->f16 != (h->Wh != nullptr)) return SOM_ERR_INVALID_ARG;
    DeviceGuard g(h->device);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    int rc = SOM_OK;
    if (h->timing && (rc = ensure_events(h))) return rc;
    if ((rc = mark(h, h->ev_bmu_calls, EV_BMU_BEGIN, st))) return rc;
    if (!p->use_table) {
        unsigned long long* keys = reinterpret_cast<unsigned long long*>(p->ws);
        SOM_CK(h, cudaMemsetAsync(keys, 0xFF, (size_t)p->n * sizeof(unsigned long long), st));
        if ((rc = mark(h, h->ev_bmu_calls, EV_BMU_PLAN_END, st))) return rc;
        if ((rc = som_launch_bmu_direct(h, p->indptr, p->indices, p->n, keys, nullptr, nullptr, st))) return rc;
        if ((rc = mark(h, h->ev_bmu_calls, EV_BMU_SEARCH_END, st))) return rc;
        if ((rc = som_launch_finalize(h, p->indptr, p->indices, p->n, keys, d_bmu, d_min_dist, nullptr, st)))
            return rc;
    } else {
        // the plan was built for a table of p->n_hot rows: the handle's options must still give it
        if (som_table_geometry(h, false).n_hot != p->n_hot) return SOM_ERR_INVALID_ARG;
        // two-stage search (option 7), as in som_bmu, when the shadow's layout holds the same table
        if (h->opt_two_stage == 1 && h->shadow && h->shadow_valid && !h->Wh && h->M % 128 == 0 &&
            som_table_geometry(h, true).n_hot == p->n_hot) {
            // as in som_bmu: both the two-stage path and the plain search are enqueued, the gate word (set
            // to 1 here: this plan takes the row-table kernel) is raised to 2 on the device unless the probe
            // sends the batch to the plain search
            static const int32_t one = 1;
            int* counters = reinterpret_cast<int*>(p->head + p->pb.n_slots);
            if (!h->host_pair) {
                SOM_CK(h, cudaMallocHost(reinterpret_cast<void**>(&h->host_pair), 4 * sizeof(int32_t)));
                h->host_pair[0] = h->host_pair[1] = 0;
                h->host_pair[2] = 1;
            }
            SOM_CK(h, cudaMemcpyAsync(counters + SOM_PLAN_USE_TABLE, &one, sizeof(int32_t), cudaMemcpyHostToDevice, st));
            const size_t kb = (size_t)(p->n + 16) * sizeof(unsigned long long);
            SOM_CK(h, cudaMemsetAsync(p->ws + p->pb.keys, 0xFF, kb, st));
            SOM_CK(h, cudaMemsetAsync(p->ws + p->pb.keys2, 0xFF, kb, st));
            if ((rc = mark(h, h->ev_bmu_calls, EV_BMU_PLAN_END, st))) return rc;
            GateScope scope(h, counters + SOM_PLAN_USE_TABLE);
            if ((rc = two_stage_enqueue(h, p->indptr, p->indices, p->n, p->head, p->ws, p->pb, p->n_hot, d_bmu,
                                        d_min_dist, nullptr, nullptr, st)))
                return rc;
            h->gate_want = SOM_GATE_TABLE_PLAIN;
            if ((rc = som_launch_bmu_table(h, false, p->indptr, p->indices, p->n, p->head, p->ws, p->pb, p->n_hot, 1,
                                           st)))
                return rc;
            if ((rc = mark(h, h->ev_bmu_calls, EV_BMU_SEARCH_END, st))) return rc;
            if ((rc = som_launch_finalize_sorted(h, p->indptr, p->indices, p->n, p->ws, p->pb, false, d_bmu,
                                                 d_min_dist, st)))
                return rc;
            h->gate_want = SOM_GATE_TABLE;
            if ((rc = rare_pass(h, p->indptr, p->indices, p->n, p->head, p->ws, p->pb, d_bmu, d_min_dist, nullptr,
                                nullptr, st)))
                return rc;
            if ((rc = mark(h, h->ev_bmu_calls, EV_BMU_END, st))) return rc;
            if (h->timing) h->ev_bmu_calls += 1;
            return SOM_OK;
        }
        SOM_CK(h, cudaMemsetAsync(p->ws + p->pb.keys, 0xFF, (size_t)(p->n + 16) * sizeof(unsigned long long), st));
        SOM_CK(h, cudaMemsetAsync(reinterpret_cast<int*>(p->head + p->pb.n_slots) + 3, 0, sizeof(int), st));
        if ((rc = mark(h, h->ev_bmu_calls, EV_BMU_PLAN_END, st))) return rc;
        if ((rc = som_launch_bmu_table(h, false, p->indptr, p->indices, p->n, p->head, p->ws, p->pb, p->n_hot, 1, st)))
            return rc;
        if ((rc = mark(h, h->ev_bmu_calls, EV_BMU_SEARCH_END, st))) return rc;
        if ((rc = som_launch_finalize_sorted(h, p->indptr, p->indices, p->n, p->ws, p->pb, false, d_bmu,
                                             d_min_dist, st)))
            return rc;
        if ((rc = rare_pass(h, p->indptr, p->indices, p->n, p->head, p->ws, p->pb, d_bmu, d_min_dist, nullptr,
                            nullptr, st)))
            return rc;
    }
    if ((rc = mark(h, h->ev_bmu_calls, EV_BMU_END, st))) return rc;
    if (h->timing) h->ev_bmu_calls += 1;
    return SOM_OK;
}

int som_update(som_handle* h, int32_t rows, int32_t cols, const int32_t* d_indptr, const int32_t* d_indices,
               int64_t n_samples, const int32_t* d_bmu, int32_t radius, void* stream)
{
    if (!h || n_samples < 0 || rows <= 0 || cols <= 0 || radius < 0) return SOM_ERR_INVALID_ARG;
    if ((int64_t)rows * cols != h->M) return SOM_ERR_INVALID_ARG;
    if (n_samples > 0 && (!d_indptr || !d_bmu)) return SOM_ERR_INVALID_ARG;
    if (n_samples >= (int64_t)1 << 31) return SOM_ERR_UNSUPPORTED;
    DeviceGuard g(h->device);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    // a window that already spans the lattice along both axes does not grow any more
    if (radius > (rows > cols ? rows : cols)) radius = rows > cols ? rows : cols;
    int planes = 1;
    const int64_t budget = (h->opt_update_mib > 0 ? h->opt_update_mib : 4096) << 20;
    // (n_samples more words: the per-sample masks of the most frequent features, see below)
    const size_t need = som_update_workspace_bytes(h, budget, &planes) + som_align_up((size_t)n_samples * 4, 256);
    int rc = ensure_bytes(h, &h->ws, &h->ws_bytes, need);
    if (rc) return rc;
    h->norms_valid = 0;  // the codebook changes: som_norms must run before the next search
    // a side stream for the denominator's route, forked from `stream` here and joined inside
    if (!h->aux_stream) {
        SOM_CK(h, cudaStreamCreateWithFlags(&h->aux_stream, cudaStreamNonBlocking));
        SOM_CK(h, cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming));
        SOM_CK(h, cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming));
    }
    SOM_CK(h, cudaEventRecord(h->ev_fork, st));
    SOM_CK(h, cudaStreamWaitEvent(h->aux_stream, h->ev_fork, 0));
    // On small lattices with many samples the planes of the most frequent features are counted
    // in shared memory (see k_upd_scatter_hot); the plan's selection phase names those features.
    const int32_t* hot_slot = nullptr;
    const int32_t* slot_feat = nullptr;
    const int n_hot_slots = 16;
    if (h->M * 4 <= 80 * 1024 && n_samples >= 8 * h->M && d_indices) {
        SomPlanBuffers pb;
        const size_t head_need = som_plan_head_bytes(h->V, n_hot_slots, &pb);
        if ((rc = ensure_bytes(h, &h->head, &h->head_bytes, head_need))) return rc;
        char* head = reinterpret_cast<char*>(h->head);
        if ((rc = som_launch_plan_select(h, d_indptr, d_indices, n_samples, head, pb, n_hot_slots, 0, st))) return rc;
        hot_slot = reinterpret_cast<const int32_t*>(head + pb.feat_slot);
        slot_feat = reinterpret_cast<const int32_t*>(head + pb.slot_feat);
    }
    return som_launch_update(h, rows, cols, d_indptr, d_indices, n_samples, d_bmu, radius, planes, hot_slot,
                             slot_feat, n_hot_slots, st, h->aux_stream, h->ev_join);
}

int som_bmu_host(som_handle* h, const int32_t* h_indptr, const int32_t* h_indices, int64_t n_samples,
                 int32_t* h_bmu, float* h_min_dist, void* stream)
{
    if (!h || n_samples < 0) return SOM_ERR_INVALID_ARG;
    if (n_samples == 0) return SOM_OK;
    if (!h_indptr || !h_bmu || !h_min_dist) return SOM_ERR_INVALID_ARG;
    if (h_indptr[0] != 0 || h_indptr[n_samples] < 0) return SOM_ERR_INVALID_ARG;
    const int64_t nnz = h_indptr[n_samples];
    if (nnz > 0 && !h_indices) return SOM_ERR_INVALID_ARG;
    if (!h->norms_valid) return SOM_ERR_NORMS_STALE;
    DeviceGuard g(h->device);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);

    const size_t b_ptr = som_align_up((size_t)(n_samples + 1) * 4, 256);
    const size_t b_idx = som_align_up((size_t)(nnz > 0 ? nnz : 1) * 4, 256);
    const size_t b_out = som_align_up((size_t)n_samples * 4, 256);
    int rc = ensure_bytes(h, &h->stage, &h->stage_bytes, b_ptr + b_idx + 2 * b_out);
    if (rc) return rc;
    char* base = reinterpret_cast<char*>(h->stage);
    int32_t* d_ptr = reinterpret_cast<int32_t*>(base);
    int32_t* d_idx = reinterpret_cast<int32_t*>(base + b_ptr);
    int32_t* d_bmu = reinterpret_cast<int32_t*>(base + b_ptr + b_idx);
    float* d_dist = reinterpret_cast<float*>(base + b_ptr + b_idx + b_out);
    SOM_CK(h, cudaMemcpyAsync(d_ptr, h_indptr, (size_t)(n_samples + 1) * 4, cudaMemcpyHostToDevice, st));
    if (nnz > 0)
        SOM_CK(h, cudaMemcpyAsync(d_idx, h_indices, (size_t)nnz * 4, cudaMemcpyHostToDevice, st));
    rc = som_bmu(h, d_ptr, d_idx, n_samples, d_bmu, d_dist, stream);
    if (rc) return rc;
    SOM_CK(h, cudaMemcpyAsync(h_bmu, d_bmu, (size_t)n_samples * 4, cudaMemcpyDeviceToHost, st));
    SOM_CK(h, cudaMemcpyAsync(h_min_dist, d_dist, (size_t)n_samples * 4, cudaMemcpyDeviceToHost, st));
    SOM_CK(h, cudaStreamSynchronize(st));
    return SOM_OK;
}

// Pipelined host entry point: two staging buffers and two copy streams of the handle's own (one
// per direction: a single in-order stream would hold the next batch's upload behind the previous
// batch's download, which waits for its search), so that the host-to-device copy of one batch
// overlaps the search of the previous one and the results travel back while the next search runs.
static int pipe_setup(som_handle* h)
{
    if (h->copy_stream) return SOM_OK;
    SOM_CK(h, cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking));
    SOM_CK(h, cudaStreamCreateWithFlags(&h->back_stream, cudaStreamNonBlocking));
    for (int t = 0; t < 2; ++t) {
        SOM_CK(h, cudaEventCreateWithFlags(&h->ev_h2d[t], cudaEventDisableTiming));
        SOM_CK(h, cudaEventCreateWithFlags(&h->ev_searched[t], cudaEventDisableTiming));
        SOM_CK(h, cudaEventCreateWithFlags(&h->ev_d2h[t], cudaEventDisableTiming));
    }
    return SOM_OK;
}

int som_bmu_host_async(som_handle* h, const int32_t* h_indptr, const int32_t* h_indices, int64_t n_samples,
                       int32_t* h_bmu, float* h_min_dist, void* stream)
{
    if (!h || n_samples < 0) return SOM_ERR_INVALID_ARG;
    if (n_samples == 0) return SOM_OK;
    if (!h_indptr || !h_bmu || !h_min_dist) return SOM_ERR_INVALID_ARG;
    if (h_indptr[0] != 0 || h_indptr[n_samples] < 0) return SOM_ERR_INVALID_ARG;
    const int64_t nnz = h_indptr[n_samples];
    if (nnz > 0 && !h_indices) return SOM_ERR_INVALID_ARG;
    if (!h->norms_valid) return SOM_ERR_NORMS_STALE;
    DeviceGuard g(h->device);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    int rc = pipe_setup(h);
    if (rc) return rc;
    const int t = (int)(h->pipe_calls & 1);
    // the buffer's previous batch (two calls ago) must have left it
    if (h->pipe_calls >= 2) SOM_CK(h, cudaEventSynchronize(h->ev_d2h[t]));

    const size_t b_ptr = som_align_up((size_t)(n_samples + 1) * 4, 256);
    const size_t b_idx = som_align_up((size_t)(nnz > 0 ? nnz : 1) * 4, 256);
    const size_t b_out = som_align_up((size_t)n_samples * 4, 256);
    if ((rc = ensure_bytes(h, &h->pipe_stage[t], &h->pipe_stage_bytes[t], b_ptr + b_idx + 2 * b_out))) return rc;
    char* base = reinterpret_cast<char*>(h->pipe_stage[t]);
    int32_t* d_ptr = reinterpret_cast<int32_t*>(base);
    int32_t* d_idx = reinterpret_cast<int32_t*>(base + b_ptr);
    int32_t* d_bmu = reinterpret_cast<int32_t*>(base + b_ptr + b_idx);
    float* d_dist = reinterpret_cast<float*>(base + b_ptr + b_idx + b_out);
    SOM_CK(h, cudaMemcpyAsync(d_ptr, h_indptr, (size_t)(n_samples + 1) * 4, cudaMemcpyHostToDevice, h->copy_stream));
    if (nnz > 0)
        SOM_CK(h, cudaMemcpyAsync(d_idx, h_indices, (size_t)nnz * 4, cudaMemcpyHostToDevice, h->copy_stream));
    SOM_CK(h, cudaEventRecord(h->ev_h2d[t], h->copy_stream));
    SOM_CK(h, cudaStreamWaitEvent(st, h->ev_h2d[t], 0));
    rc = som_bmu(h, d_ptr, d_idx, n_samples, d_bmu, d_dist, stream);
    if (rc) return rc;
    SOM_CK(h, cudaEventRecord(h->ev_searched[t], st));
    SOM_CK(h, cudaStreamWaitEvent(h->back_stream, h->ev_searched[t], 0));
    SOM_CK(h, cudaMemcpyAsync(h_bmu, d_bmu, (size_t)n_samples * 4, cudaMemcpyDeviceToHost, h->back_stream));
    SOM_CK(h, cudaMemcpyAsync(h_min_dist, d_dist, (size_t)n_samples * 4, cudaMemcpyDeviceToHost, h->back_stream));
    SOM_CK(h, cudaEventRecord(h->ev_d2h[t], h->back_stream));
    h->pipe_calls += 1;
    return SOM_OK;
}

int som_host_sync(som_handle* h)
{
    if (!h) return SOM_ERR_INVALID_ARG;
    if (!h->copy_stream) return SOM_OK;
    DeviceGuard g(h->device);
    SOM_CK(h, cudaStreamSynchronize(h->copy_stream));
    SOM_CK(h, cudaStreamSynchronize(h->back_stream));
    return SOM_OK;
}

int som_validate_csr(som_handle* h, const int32_t* d_indptr, const int32_t* d_indices,
                     int64_t n_samples, void* stream)
{
    if (!h || n_samples < 0) return SOM_ERR_INVALID_ARG;
    if (n_samples == 0) return SOM_OK;
    if (!d_indptr) return SOM_ERR_INVALID_ARG;
    DeviceGuard g(h->device);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    int rc = ensure_bytes(h, &h->stage, &h->stage_bytes, 256);
    if (rc) return rc;
    int* d_flag = reinterpret_cast<int*>(h->stage);
    SOM_CK(h, cudaMemsetAsync(d_flag, 0, sizeof(int), st));
    if ((rc = som_launch_validate(h, d_indptr, d_indices, n_samples, d_flag, st))) return rc;
    int flag = 0;
    SOM_CK(h, cudaMemcpyAsync(&flag, d_flag, sizeof(int), cudaMemcpyDeviceToHost, st));
    SOM_CK(h, cudaStreamSynchronize(st));
    return flag ? SOM_ERR_BAD_CSR : SOM_OK;
}

int som_device_flags(som_handle* h, void* stream)
{
    if (!h) return SOM_ERR_INVALID_ARG;
    DeviceGuard g(h->device);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    int flags = 0;
    SOM_CK(h, cudaMemcpyAsync(&flags, h->dev_flags, sizeof(int), cudaMemcpyDeviceToHost, st));
    SOM_CK(h, cudaMemsetAsync(h->dev_flags, 0, sizeof(int), st));
    SOM_CK(h, cudaStreamSynchronize(st));
    if (flags & SOM_FLAG_BAD_INDEX) return SOM_ERR_BAD_CSR;
    if (flags & SOM_FLAG_BAD_UNIT) return SOM_ERR_INVALID_ARG;
    return SOM_OK;
}

int som_get_norms(som_handle* h, float* d_out, void* stream)
{
    if (!h || !d_out) return SOM_ERR_INVALID_ARG;
    if (!h->norms_valid) return SOM_ERR_NORMS_STALE;
    DeviceGuard g(h->device);
    SOM_CK(h, cudaMemcpyAsync(d_out, h->norm32, (size_t)h->M * sizeof(float), cudaMemcpyDeviceToDevice,
                              reinterpret_cast<cudaStream_t>(stream)));
    return SOM_OK;
}

const char* som_status_string(int status)
{
    switch (status) {
        case SOM_OK: return "SOM_OK";
        case SOM_ERR_INVALID_ARG: return "SOM_ERR_INVALID_ARG";
        case SOM_ERR_NORMS_STALE: return "SOM_ERR_NORMS_STALE";
        case SOM_ERR_UNSUPPORTED: return "SOM_ERR_UNSUPPORTED";
        case SOM_ERR_CUDA: return "SOM_ERR_CUDA";
        case SOM_ERR_BAD_CSR: return "SOM_ERR_BAD_CSR";
        case SOM_ERR_NO_DEVICE: return "SOM_ERR_NO_DEVICE";
        default: return "SOM_ERR_UNKNOWN";
    }
}

int som_last_cuda_error(const som_handle* h) { return h ? h->last_cuda_error : 0; }

int som_set_timing(som_handle* h, int enable)
{
    if (!h) return SOM_ERR_INVALID_ARG;
    h->timing = enable ? 1 : 0;
    h->ev_norms_calls = h->ev_bmu_calls = 0;
    return SOM_OK;
}

int som_get_timing(som_handle* h, float* out_ms, int n_out)
{
    if (!h || !out_ms || n_out < 0) return SOM_ERR_INVALID_ARG;
    float v[5] = {0, 0, 0, 0, 0};
    DeviceGuard g(h->device);
    auto ev = [&](int64_t call, int slot) { return h->ev[(call % SOM_EV_RING) * SOM_EV_PER_CALL + slot]; };
    auto span = [&](int64_t call, int a, int b, float* acc) -> cudaError_t {
        float ms = 0.f;
        cudaError_t e = cudaEventElapsedTime(&ms, ev(call, a), ev(call, b));
        *acc += ms;
        return e;
    };
    {
        const int64_t c1 = h->ev_norms_calls, c0 = c1 > SOM_EV_RING ? c1 - SOM_EV_RING : 0;
        for (int64_t c = c0; c < c1; ++c) SOM_CK(h, span(c, EV_NORMS_BEGIN, EV_NORMS_END, &v[0]));
        if (c1 > c0) v[0] /= (float)(c1 - c0);
    }
    {
        const int64_t c1 = h->ev_bmu_calls, c0 = c1 > SOM_EV_RING ? c1 - SOM_EV_RING : 0;
        for (int64_t c = c0; c < c1; ++c) {
            SOM_CK(h, span(c, EV_BMU_BEGIN, EV_BMU_END, &v[1]));
            SOM_CK(h, span(c, EV_BMU_BEGIN, EV_BMU_PLAN_END, &v[2]));
            SOM_CK(h, span(c, EV_BMU_PLAN_END, EV_BMU_SEARCH_END, &v[3]));
            SOM_CK(h, span(c, EV_BMU_SEARCH_END, EV_BMU_END, &v[4]));
        }
        if (c1 > c0)
            for (int i = 1; i < 5; ++i) v[i] /= (float)(c1 - c0);
    }
    for (int i = 0; i < n_out && i < 5; ++i) out_ms[i] = v[i];
    return SOM_OK;
}

int64_t som_last_uncertain(const som_handle* h)
{
    if (!h) return 0;
    if (h->last_uncertain >= 0 || !h->host_pair) return h->last_uncertain < 0 ? 0 : h->last_uncertain;
    // the last two-stage call left its report in pinned host words (valid once its stream has been waited for):
    // word 0 = all samples when the probe sent the batch to the plain search, else -1; word 1 = the length of
    // the certificate's list
    const int32_t report = *reinterpret_cast<volatile int32_t*>(h->host_pair);
    return report >= 0 ? (int64_t)report : (int64_t) * reinterpret_cast<volatile int32_t*>(h->host_pair + 1);
}

int64_t som_launch_count(const som_handle* h) { return h ? h->launches : 0; }

int som_set_option(som_handle* h, int key, int64_t value)
{
    if (!h) return SOM_ERR_INVALID_ARG;
    if (key == 0) {
        if (value < 0 || value > 2) return SOM_ERR_INVALID_ARG;
        h->opt_variant = value;
        return SOM_OK;
    }
    if (key == 1) {
        if (value < 0 || value > 65000) return SOM_ERR_INVALID_ARG;
        h->opt_hot_rows = value;
        return SOM_OK;
    }
    if (key == 4) {
        if (value < 0 || value > 1024) return SOM_ERR_INVALID_ARG;
        h->opt_parts = value;
        return SOM_OK;
    }
    if (key == 10) {
        if (value < 0 || value > 2) return SOM_ERR_INVALID_ARG;
        h->opt_prune = value;
        return SOM_OK;
    }
    if (key == 9) {
        if (value < 0 || value > 2) return SOM_ERR_INVALID_ARG;
        h->opt_feed_keep = value;
        return SOM_OK;
    }
    if (key == 8) {
        if (value < 0 || value > SOM_PLAN_MASK_FEATURES) return SOM_ERR_INVALID_ARG;
        h->opt_mask_bits = value;
        return SOM_OK;
    }
    if (key == 7) {
        if (value != 0 && value != 1) return SOM_ERR_INVALID_ARG;
        if (value == 1 && !h->shadow && !h->Wh) {
            DeviceGuard g(h->device);
            // the fp16 shadow of the codebook: half its size again in device memory
            SOM_CK(h, cudaMalloc(reinterpret_cast<void**>(&h->shadow), (size_t)h->V * (size_t)h->M * sizeof(__half)));
            SOM_CK(h, cudaMalloc(reinterpret_cast<void**>(&h->wmax_bits), 256));
            h->shadow_valid = 0;
            h->norms_valid = 0;  // the next som_norms writes the shadow
        }
        h->opt_two_stage = value;
        return SOM_OK;
    }
    if (key == 6) {
        if (value < 0 || value > (1 << 20)) return SOM_ERR_INVALID_ARG;
        h->opt_update_mib = value;
        return SOM_OK;
    }
    if (key == 5) {
        if (value < 0 || value > 100) return SOM_ERR_INVALID_ARG;
        h->opt_cover = value;
        return SOM_OK;
    }
    if (key == 3) {
        if (value != 0 && value != 4 && value != 8 && value != 16) return SOM_ERR_INVALID_ARG;
        h->opt_r = value;
        return SOM_OK;
    }
    if (key == 2) {
        if (value != 0 && value != 512 && value != 576 && value != 640 && value != 768 &&
            value != 896 && value != 1024)
            return SOM_ERR_INVALID_ARG;
        h->opt_threads = value;
        return SOM_OK;
    }
    return SOM_ERR_INVALID_ARG;
}

}  // extern "C"
