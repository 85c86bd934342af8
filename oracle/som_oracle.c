/*
 * CPU oracle for the best-matching-unit search of a sparse-binary self-organizing map.
 *
 * THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, fp64 statement of what the search
 * computes, used only by the tests, the smoke check and the CPU-baseline leg of the
 * benchmark.  It shares no code with the CUDA library and the library never calls it.
 *
 * What it computes (Section 3.1, Eq. 1 of the paper): for a binary sample x with active
 * feature set S (sorted ascending) and every neuron i with prototype w_i,
 *
 *     d(x, i) = ||x - w_i||^2 = |S| - 2 * sum_{v in S} w_i[v] + sum_{v < V} w_i[v]^2
 *
 * and BMU(x) = argmin_i d(x, i), ties broken to the lowest neuron index (Section 3.1).
 * The sum over S runs in ascending feature order, the norm in ascending v, both in
 * double precision from the stored fp32 weights.  The argmin is a linear scan with a
 * strict "<", which is exactly the lowest-index tie rule.  The second-best unit (the
 * paper's bmu2, Algorithm 2 step 7) is tracked in the same scan.
 *
 * The codebook layout flag changes the address of weight (v, i) and nothing else
 * (Section 3.2): feature-major W[v*M + i], node-major W[i*V + v].
 *
 * Parity pins (tests, "not gpu"): dense brute force sum_v (x_v - w_iv)^2 on tiny inputs,
 * layout invariance, hand-built cases with a known unique nearest neuron, closed-form
 * norms, duplicate-neuron ties, slab merging.  The paper prints no worked numeric
 * example, so numeric parity with the paper's own runs is unpinned.
 */
#include <stdint.h>
#include <stdlib.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define SOM_ORACLE_FEATURE_MAJOR 0
#define SOM_ORACLE_NODE_MAJOR 1

static inline double weight(const float* W, int layout, int64_t V, int64_t M, int64_t v, int64_t i)
{
    return layout == SOM_ORACLE_FEATURE_MAJOR ? (double)W[v * M + i] : (double)W[i * V + v];
}

int som_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ||w_i||^2 for every neuron of the slab, ascending v, fp64. */
void som_oracle_norms(const float* W, int layout, int64_t V, int64_t M, double* norms)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < M; ++i) {
        double s = 0.0;
        for (int64_t v = 0; v < V; ++v) {
            double w = weight(W, layout, V, M, v, i);
            s += w * w;
        }
        norms[i] = s;
    }
}

/* d(x_n, i) for one sample and one neuron. */
static double distance(const float* W, int layout, int64_t V, int64_t M, const double* norms,
                       const int32_t* idx, int64_t nnz, int64_t i)
{
    double dot = 0.0;
    for (int64_t k = 0; k < nnz; ++k)
        dot += weight(W, layout, V, M, (int64_t)idx[k], i);
    return (double)nnz - 2.0 * dot + norms[i];
}

/*
 * Best and second-best unit of every sample over the M neurons of this codebook slab.
 * m_offset is the global index of the slab's neuron 0.  With merge == 0 the outputs are
 * initialised (b = -1, d = +inf); with merge != 0 the slab is merged into the running
 * best / second best already in the outputs.  Slabs must be visited in ascending neuron
 * order for the strict "<" to keep the lowest-index rule across slabs.
 */
void som_oracle_bmu(const float* W, int layout, int64_t V, int64_t M, const double* norms,
                    const int32_t* indptr, const int32_t* indices, int64_t n,
                    int64_t m_offset, int merge,
                    int64_t* b1, double* d1, int64_t* b2, double* d2)
{
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t s = 0; s < n; ++s) {
        const int32_t* idx = indices + indptr[s];
        int64_t nnz = (int64_t)indptr[s + 1] - (int64_t)indptr[s];
        int64_t bb1 = -1, bb2 = -1;
        double dd1 = INFINITY, dd2 = INFINITY;
        if (merge) { bb1 = b1[s]; dd1 = d1[s]; bb2 = b2[s]; dd2 = d2[s]; }
        for (int64_t i = 0; i < M; ++i) {
            double d = distance(W, layout, V, M, norms, idx, nnz, i);
            if (d < dd1) { dd2 = dd1; bb2 = bb1; dd1 = d; bb1 = m_offset + i; }
            else if (d < dd2) { dd2 = d; bb2 = m_offset + i; }
        }
        b1[s] = bb1; d1[s] = dd1; b2[s] = bb2; d2[s] = dd2;
    }
}

/* d(x_n, neuron[n]) for given (sample, neuron) pairs; neuron ids are slab-local. */
void som_oracle_dist_at(const float* W, int layout, int64_t V, int64_t M, const double* norms,
                        const int32_t* indptr, const int32_t* indices, int64_t n,
                        const int64_t* neuron, double* d)
{
#pragma omp parallel for schedule(static)
    for (int64_t s = 0; s < n; ++s) {
        const int32_t* idx = indices + indptr[s];
        int64_t nnz = (int64_t)indptr[s + 1] - (int64_t)indptr[s];
        d[s] = distance(W, layout, V, M, norms, idx, nnz, neuron[s]);
    }
}

/*
 * Sparse real-valued samples (the paper's outlook, Section 7: a values array beside the feature
 * indices and the sample's own squared norm): x has value val[k] at feature idx[k] and 0 elsewhere, and
 *   d(x, w_i) = ||x - w_i||^2 = sum_k val[k]^2 - 2 * sum_k val[k] * w_i[idx[k]] + ||w_i||^2.
 */
static double distance_values(const float* W, int layout, int64_t V, int64_t M, const double* norms,
                              const int32_t* idx, const float* val, int64_t nnz, int64_t i)
{
    double xx = 0.0, dot = 0.0;
    for (int64_t k = 0; k < nnz; ++k) {
        const double x = (double)val[k];
        xx += x * x;
        dot += x * weight(W, layout, V, M, (int64_t)idx[k], i);
    }
    return xx - 2.0 * dot + norms[i];
}

/* som_oracle_bmu for sparse real-valued samples (values[] runs parallel to indices[]). */
void som_oracle_bmu_values(const float* W, int layout, int64_t V, int64_t M, const double* norms,
                           const int32_t* indptr, const int32_t* indices, const float* values, int64_t n,
                           int64_t* b1, double* d1, int64_t* b2, double* d2)
{
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t s = 0; s < n; ++s) {
        const int32_t* idx = indices + indptr[s];
        const float* val = values + indptr[s];
        int64_t nnz = (int64_t)indptr[s + 1] - (int64_t)indptr[s];
        int64_t bb1 = -1, bb2 = -1;
        double dd1 = INFINITY, dd2 = INFINITY;
        for (int64_t i = 0; i < M; ++i) {
            double d = distance_values(W, layout, V, M, norms, idx, val, nnz, i);
            if (d < dd1) { dd2 = dd1; bb2 = bb1; dd1 = d; bb1 = i; }
            else if (d < dd2) { dd2 = d; bb2 = i; }
        }
        b1[s] = bb1; d1[s] = dd1; b2[s] = bb2; d2[s] = dd2;
    }
}

void som_oracle_dist_at_values(const float* W, int layout, int64_t V, int64_t M, const double* norms,
                               const int32_t* indptr, const int32_t* indices, const float* values,
                               int64_t n, const int64_t* neuron, double* d)
{
#pragma omp parallel for schedule(static)
    for (int64_t s = 0; s < n; ++s)
        d[s] = distance_values(W, layout, V, M, norms, indices + indptr[s], values + indptr[s],
                               (int64_t)indptr[s + 1] - (int64_t)indptr[s], neuron[s]);
}

/* Full n x M distance matrix (row-major), for tiny inputs only. */
void som_oracle_all_distances(const float* W, int layout, int64_t V, int64_t M, const double* norms,
                              const int32_t* indptr, const int32_t* indices, int64_t n, double* out)
{
    for (int64_t s = 0; s < n; ++s) {
        const int32_t* idx = indices + indptr[s];
        int64_t nnz = (int64_t)indptr[s + 1] - (int64_t)indptr[s];
        for (int64_t i = 0; i < M; ++i)
            out[s * M + i] = distance(W, layout, V, M, norms, idx, nnz, i);
    }
}
