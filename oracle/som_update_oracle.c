/*
 * som_update_oracle.c - plain CPU restatement of the batch update of the sparse-binary SOM.
 *
 * TEST INFRASTRUCTURE ONLY: used by tests/ to check the CUDA update path.  It shares no code
 * with the CUDA library.
 *
 * What it computes (paper, Section 3.4 "Factorised box-blur update"; Algorithm 2, steps 8-9):
 *   1. scatter: for every sample s assigned to lattice cell c = bmu[s], den[c] += 1 and, for
 *      every active feature v of s, num[v][c] += 1 (the per-cell sum of the assigned binary
 *      samples and their count);
 *   2. blur: every field (each feature plane of num, and den) is filtered by `passes` box
 *      passes per lattice axis (the paper fixes three).  A box pass replaces a cell by the
 *      UNNORMALISED sum of the cells within `radius` of it along that axis; at the lattice edge
 *      the window is truncated (clamped, not toroidal), identically for num and den;
 *   3. divide: W[v][i] = num_b[v][i] / den_b[i] wherever den_b[i] > 0; a neuron whose blurred
 *      denominator is zero keeps its old prototype.
 * The update is a pure replacement (no learning rate).  Neuron i sits at lattice row i / cols,
 * column i % cols.  Everything is fp64 and each window sum is written out as the plain sum over
 * the window (no running sums), so the code can be checked against the text by eye.  The
 * codebook is feature-major: weight (v, i) at W[v*M + i], M = rows * cols.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* one box pass along the column index (within each lattice row) */
static void pass_along_row(const double* in, double* out, int64_t rows, int64_t cols, int64_t radius)
{
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c) {
            int64_t lo = c - radius < 0 ? 0 : c - radius;
            int64_t hi = c + radius > cols - 1 ? cols - 1 : c + radius;
            double s = 0.0;
            for (int64_t j = lo; j <= hi; ++j) s += in[r * cols + j];
            out[r * cols + c] = s;
        }
}

/* one box pass along the row index (within each lattice column) */
static void pass_along_col(const double* in, double* out, int64_t rows, int64_t cols, int64_t radius)
{
    for (int64_t r = 0; r < rows; ++r) {
        int64_t lo = r - radius < 0 ? 0 : r - radius;
        int64_t hi = r + radius > rows - 1 ? rows - 1 : r + radius;
        for (int64_t c = 0; c < cols; ++c) {
            double s = 0.0;
            for (int64_t j = lo; j <= hi; ++j) s += in[j * cols + c];
            out[r * cols + c] = s;
        }
    }
}

/* `passes` times: a pass along the rows followed by one along the columns (Section 3.4).
 * field is overwritten; tmp holds rows*cols doubles. */
void som_oracle_blur(double* field, double* tmp, int64_t rows, int64_t cols, int64_t radius, int passes)
{
    for (int p = 0; p < passes; ++p) {
        pass_along_row(field, tmp, rows, cols, radius);
        pass_along_col(tmp, field, rows, cols, radius);
    }
}

/*
 * W_old [V*M] fp32 feature-major; bmu [n] lattice cell of every sample; out [V*M] fp64: the new
 * codebook (unrounded quotient, or the old weight where the blurred denominator is zero).
 * Returns 0, or 1 if memory could not be had.
 */
int som_oracle_update(const float* W_old, int64_t V, int64_t rows, int64_t cols, const int32_t* indptr,
                      const int32_t* indices, int64_t n, const int32_t* bmu, int64_t radius, int passes,
                      double* out)
{
    const int64_t M = rows * cols;
    double* num = (double*)calloc((size_t)(V * M), sizeof(double));
    double* den = (double*)calloc((size_t)M, sizeof(double));
    double* tmp = (double*)malloc((size_t)M * sizeof(double));
    if (!num || !den || !tmp) {
        free(num); free(den); free(tmp);
        return 1;
    }
    for (int64_t s = 0; s < n; ++s) {
        const int64_t c = bmu[s];
        den[c] += 1.0;
        for (int64_t j = indptr[s]; j < indptr[s + 1]; ++j) num[(int64_t)indices[j] * M + c] += 1.0;
    }
    som_oracle_blur(den, tmp, rows, cols, radius, passes);
    for (int64_t v = 0; v < V; ++v) {
        double* plane = num + v * M;
        som_oracle_blur(plane, tmp, rows, cols, radius, passes);
        for (int64_t i = 0; i < M; ++i)
            out[v * M + i] = den[i] > 0.0 ? plane[i] / den[i] : (double)W_old[v * M + i];
    }
    free(num); free(den); free(tmp);
    return 0;
}
