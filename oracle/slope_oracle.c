/*
 * slope_oracle.c -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, fp64 CPU statement of what the SLoPe 2:4-sparse linear layer
 * computes (thesis chapter "SLoPe: Double-Pruned Sparse Plus Lazy Low-Rank
 * Adapter Pretraining of LLMs").  Only the tests, the smoke check and the
 * benchmark's cpu_baseline / reference arm may call it.  It shares no code
 * with the CUDA library: no headers, no tables, no helpers.
 *
 * Every matrix is dense row-major.  bf16 values travel as raw uint16 bit
 * patterns; all arithmetic is done in double after an exact widening.
 *
 * Pins (see tests/test_oracle_pins.py): brute-force pair enumeration for the
 * selection rule, structural invariants, Lemma 1's closed form (9.375 % extra
 * zeros for 2:4), numpy fp64 matmul on the masked dense matrices, central
 * finite differences on tiny inputs, and the fused-adapter identity of
 * Eq. (concat).  The general N:M passes (O9, O10) are pinned by subset
 * enumeration on tie-heavy groups, by agreement with the 2:4 path, and by
 * Eq. (sparsity_ratio) for seven (N, M) patterns on Gaussian data.
 *
 * Conventions
 *   W  [d_out x d_in]   weight (Sec. "Sparse Plus Low-rank Pretraining")
 *   X  [b x d_in], Y [b x d_out], dY [b x d_out], dX [b x d_in]
 *   L  [d_in x r], R [r x d_out]  (orientation of Eq. (concat): Y = (X L) R + X W^T)
 *   mask bit of element (i, j): bit (j mod 8), LSB first, of byte mask[i][j/8],
 *   always in W's orientation (also for the second-pass mask).
 *   nibble of a group = p0 | p1 << 2 with p0 < p1 the kept positions.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double bf16_to_double(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

static int mask_get(const uint8_t *mask, long row_bytes, long i, long j) {
    return (mask[i * row_bytes + (j >> 3)] >> (j & 7)) & 1;
}

/* Choose the two largest of four 15-bit magnitudes; among equal magnitudes the
 * lower position wins.  Returns the kept positions p0 < p1. */
static void top2_of_4(const uint32_t key[4], int *p0, int *p1) {
    int first = 0;
    for (int t = 1; t < 4; ++t)
        if (key[t] > key[first]) first = t;            /* strict: lower index wins ties */
    int second = -1;
    for (int t = 0; t < 4; ++t) {
        if (t == first) continue;
        if (second < 0 || key[t] > key[second]) second = t;
    }
    *p0 = first < second ? first : second;
    *p1 = first < second ? second : first;
}

/* O1 -- first pass: 2:4 magnitude selection along d_in (the reduction dimension
 * of Eq. (sparse_forward)), compression to values + positions
 * (supplementary "cuSPARSELt Initialization Overhead": copy the non-zeros into a
 * contiguous layout and generate indices). */
void slope_oracle_prune24(const uint16_t *W, int d_out, int d_in,
                          uint16_t *vals, uint8_t *nib, uint8_t *mask1)
{
    long mrow = d_in / 8;
    memset(mask1, 0, (size_t)d_out * mrow);
    for (long i = 0; i < d_out; ++i) {
        for (long g = 0; g < d_in / 4; ++g) {
            uint32_t key[4];
            for (int t = 0; t < 4; ++t) key[t] = W[i * d_in + 4 * g + t] & 0x7FFFu;
            int p0, p1;
            top2_of_4(key, &p0, &p1);
            vals[i * (d_in / 2) + 2 * g + 0] = W[i * d_in + 4 * g + p0];
            vals[i * (d_in / 2) + 2 * g + 1] = W[i * d_in + 4 * g + p1];
            nib[i * (d_in / 4) + g] = (uint8_t)(p0 | (p1 << 2));
            long j0 = 4 * g + p0, j1 = 4 * g + p1;
            mask1[i * mrow + (j0 >> 3)] |= (uint8_t)(1u << (j0 & 7));
            mask1[i * mrow + (j1 >> 3)] |= (uint8_t)(1u << (j1 & 7));
        }
    }
}

/* O2 -- second pass (double pruning): transpose the already 2:4 matrix W^R and
 * impose 2:4 again, now along d_out (the reduction dimension of
 * Eq. (sparse_backward_input)).  Entries removed by the first pass enter with
 * magnitude zero and value +0.  Output is the compressed transposed copy. */
void slope_oracle_double_prune(const uint16_t *W, const uint8_t *mask1, int d_out, int d_in,
                               uint16_t *valsT, uint8_t *nibT, uint8_t *mask2)
{
    long mrow = d_in / 8;
    memset(mask2, 0, (size_t)d_out * mrow);
    for (long j = 0; j < d_in; ++j) {
        for (long h = 0; h < d_out / 4; ++h) {
            uint32_t key[4];
            uint16_t v[4];
            int kept1[4];
            for (int t = 0; t < 4; ++t) {
                long i = 4 * h + t;
                kept1[t] = mask_get(mask1, mrow, i, j);
                v[t] = kept1[t] ? W[i * d_in + j] : (uint16_t)0;
                key[t] = v[t] & 0x7FFFu;
            }
            int q0, q1;
            top2_of_4(key, &q0, &q1);
            valsT[j * (d_out / 2) + 2 * h + 0] = v[q0];
            valsT[j * (d_out / 2) + 2 * h + 1] = v[q1];
            nibT[j * (d_out / 4) + h] = (uint8_t)(q0 | (q1 << 2));
            if (kept1[q0]) mask2[(4 * h + q0) * mrow + (j >> 3)] |= (uint8_t)(1u << (j & 7));
            if (kept1[q1]) mask2[(4 * h + q1) * mrow + (j >> 3)] |= (uint8_t)(1u << (j & 7));
        }
    }
}

/* Canonical metadata: four consecutive groups of a row share one little-endian
 * uint16, group g at bits 4*(g mod 4). */
void slope_oracle_pack_canonical(const uint8_t *nib, int rows, int cols, uint16_t *canon)
{
    long groups = cols / 4;
    for (long i = 0; i < rows; ++i)
        for (long u = 0; u < groups / 4; ++u) {
            uint16_t w = 0;
            for (int t = 0; t < 4; ++t) w |= (uint16_t)(nib[i * groups + 4 * u + t] << (4 * t));
            canon[i * (groups / 4) + u] = w;
        }
}

/* Sparse-MMA operand order of the metadata (Eq. (index_bits) counts 3 bits per
 * group; the tensor-core operand stores 2 bits per kept element = 4 bits).
 * The matrix is cut into blocks of 128 rows x 128 columns, block (rb, cb) at
 * byte offset ((rb * (cols/128)) + cb) * 2048.  Inside a block a 16-bit unit
 * (4 groups = 16 columns) of row rr and 16-column slot cs sits in 32-bit word
 *   word = (16*(rr/16) + 8*(cs%2) + rr%8) * 4 + cs/2
 * in its low half when (rr/8)%2 == 0, else in its high half. */
void slope_oracle_canonical_to_hw(const uint16_t *canon, int rows, int cols, uint8_t *hw)
{
    long units_per_row = cols / 16;
    long cblocks = cols / 128;
    for (long i = 0; i < rows; ++i)
        for (long u = 0; u < units_per_row; ++u) {
            long rb = i / 128, rr = i % 128;
            long cb = u / 8, cs = u % 8;
            long word = (16 * (rr / 16) + 8 * (cs % 2) + rr % 8) * 4 + cs / 2;
            long half = (rr / 8) % 2;
            long off = (rb * cblocks + cb) * 2048 + word * 4 + half * 2;
            uint16_t w = canon[i * units_per_row + u];
            hw[off] = (uint8_t)(w & 0xFF);
            hw[off + 1] = (uint8_t)(w >> 8);
        }
}

/* Rebuild the dense masked matrix from values + positions (doubles). */
void slope_oracle_decompress(const uint16_t *vals, const uint8_t *nib, int rows, int cols, double *dense)
{
    memset(dense, 0, sizeof(double) * (size_t)rows * cols);
    for (long i = 0; i < rows; ++i)
        for (long g = 0; g < cols / 4; ++g) {
            int n = nib[i * (cols / 4) + g];
            dense[i * cols + 4 * g + (n & 3)] = bf16_to_double(vals[i * (cols / 2) + 2 * g]);
            dense[i * cols + 4 * g + ((n >> 2) & 3)] = bf16_to_double(vals[i * (cols / 2) + 2 * g + 1]);
        }
}

/* O3 -- Eq. (sparse_forward) plus the adapter path of Eq. (concat):
 *   Y[n][i] = sum_j X[n][j] W^R[i][j] + sum_k (sum_j X[n][j] L[j][k]) R[k][i]
 * for the listed token rows.  r == 0 leaves the adapter out. */
void slope_oracle_fwd_rows(const uint16_t *X, const uint16_t *W, const uint8_t *mask1,
                           int b, int d_out, int d_in,
                           const uint16_t *L, const uint16_t *R, int r,
                           const int *rows, int nrows, double *Y)
{
    (void)b;
    long mrow = d_in / 8;
#pragma omp parallel for schedule(dynamic, 1)
    for (int s = 0; s < nrows; ++s) {
        long n = rows[s];
        double *x = (double *)malloc(sizeof(double) * d_in);
        double *t = (double *)malloc(sizeof(double) * (r > 0 ? r : 1));
        for (long j = 0; j < d_in; ++j) x[j] = bf16_to_double(X[n * d_in + j]);
        for (int k = 0; k < r; ++k) {
            double acc = 0.0;
            for (long j = 0; j < d_in; ++j) acc += x[j] * bf16_to_double(L[j * r + k]);
            t[k] = acc;
        }
        for (long i = 0; i < d_out; ++i) {
            double acc = 0.0;
            for (long j = 0; j < d_in; ++j)
                if (mask_get(mask1, mrow, i, j)) acc += x[j] * bf16_to_double(W[i * d_in + j]);
            double lr = 0.0;
            for (int k = 0; k < r; ++k) lr += t[k] * bf16_to_double(R[(long)k * d_out + i]);
            Y[(long)s * d_out + i] = acc + lr;
        }
        free(x);
        free(t);
    }
}

/* O4 -- Eq. (sparse_backward_input) with the double-pruned weight, plus the
 * exact chain-rule adapter term:
 *   dX[n][j] = sum_i dY[n][i] W^{R,C}[i][j] + sum_k (sum_i dY[n][i] R[k][i]) L[j][k] */
void slope_oracle_dx_rows(const uint16_t *dY, const uint16_t *W, const uint8_t *mask2,
                          int b, int d_out, int d_in,
                          const uint16_t *L, const uint16_t *R, int r,
                          const int *rows, int nrows, double *dX)
{
    (void)b;
    long mrow = d_in / 8;
#pragma omp parallel for schedule(dynamic, 1)
    for (int s = 0; s < nrows; ++s) {
        long n = rows[s];
        double *g = (double *)malloc(sizeof(double) * d_out);
        double *dt = (double *)malloc(sizeof(double) * (r > 0 ? r : 1));
        for (long i = 0; i < d_out; ++i) g[i] = bf16_to_double(dY[n * d_out + i]);
        for (int k = 0; k < r; ++k) {
            double acc = 0.0;
            for (long i = 0; i < d_out; ++i) acc += g[i] * bf16_to_double(R[(long)k * d_out + i]);
            dt[k] = acc;
        }
        for (long j = 0; j < d_in; ++j) {
            double acc = 0.0;
            for (long i = 0; i < d_out; ++i)
                if (mask_get(mask2, mrow, i, j)) acc += g[i] * bf16_to_double(W[i * d_in + j]);
            double lr = 0.0;
            for (int k = 0; k < r; ++k) lr += dt[k] * bf16_to_double(L[j * r + k]);
            dX[(long)s * d_in + j] = acc + lr;
        }
        free(g);
        free(dt);
    }
}

/* O5 -- Eq. (sparse_backward_weight) followed by Algorithm 1's pruneAndCompress:
 * the weight gradient restricted to the first-pass mask, kept entries of each
 * group in ascending column order, output [d_out x d_in/2].  Listed rows only. */
void slope_oracle_dw_rows(const uint16_t *dY, const uint16_t *X, const uint8_t *mask1,
                          int b, int d_out, int d_in,
                          const int *orows, int n_orows, double *dWc)
{
    long mrow = d_in / 8;
#pragma omp parallel for schedule(dynamic, 1)
    for (int s = 0; s < n_orows; ++s) {
        long i = orows[s];
        long *cols = (long *)malloc(sizeof(long) * (d_in / 2));
        long c = 0;
        for (long j = 0; j < d_in; ++j)
            if (mask_get(mask1, mrow, i, j)) cols[c++] = j;
        double *acc = dWc + (long)s * (d_in / 2);
        for (long q = 0; q < d_in / 2; ++q) acc[q] = 0.0;
        for (long n = 0; n < b; ++n) {
            double gy = bf16_to_double(dY[n * d_out + i]);
            for (long q = 0; q < c; ++q) acc[q] += gy * bf16_to_double(X[n * d_in + cols[q]]);
        }
        free(cols);
    }
}

/* T = X L for the listed token rows (first half of Eq. (concat)). */
void slope_oracle_adapter_T_rows(const uint16_t *X, const uint16_t *L, int b, int d_in, int r,
                                 const int *rows, int nrows, double *T)
{
    (void)b;
#pragma omp parallel for schedule(static)
    for (int s = 0; s < nrows; ++s) {
        long n = rows[s];
        for (int k = 0; k < r; ++k) {
            double acc = 0.0;
            for (long j = 0; j < d_in; ++j)
                acc += bf16_to_double(X[n * d_in + j]) * bf16_to_double(L[j * r + k]);
            T[(long)s * r + k] = acc;
        }
    }
}

/* dT = dY R^T for the listed token rows (chain rule through Y = T R + ...). */
void slope_oracle_adapter_dT_rows(const uint16_t *dY, const uint16_t *R, int b, int d_out, int r,
                                  const int *rows, int nrows, double *dT)
{
    (void)b;
#pragma omp parallel for schedule(static)
    for (int s = 0; s < nrows; ++s) {
        long n = rows[s];
        for (int k = 0; k < r; ++k) {
            double acc = 0.0;
            for (long i = 0; i < d_out; ++i)
                acc += bf16_to_double(dY[n * d_out + i]) * bf16_to_double(R[(long)k * d_out + i]);
            dT[(long)s * r + k] = acc;
        }
    }
}

/* O6 -- dL[j][k] = sum_n X[n][j] dT[n][k] with dT = dY R^T kept in fp64, for
 * the listed d_in rows j. */
void slope_oracle_adapter_dL_rows(const uint16_t *X, const uint16_t *dY, const uint16_t *R,
                                  int b, int d_out, int d_in, int r,
                                  const int *jrows, int njrows, double *dL)
{
    double *dT = (double *)malloc(sizeof(double) * (size_t)b * r);
#pragma omp parallel for schedule(static)
    for (long n = 0; n < b; ++n)
        for (int k = 0; k < r; ++k) {
            double acc = 0.0;
            for (long i = 0; i < d_out; ++i)
                acc += bf16_to_double(dY[n * d_out + i]) * bf16_to_double(R[(long)k * d_out + i]);
            dT[n * r + k] = acc;
        }
#pragma omp parallel for schedule(static)
    for (int s = 0; s < njrows; ++s) {
        long j = jrows[s];
        for (int k = 0; k < r; ++k) {
            double acc = 0.0;
            for (long n = 0; n < b; ++n) acc += bf16_to_double(X[n * d_in + j]) * dT[n * r + k];
            dL[(long)s * r + k] = acc;
        }
    }
    free(dT);
}

/* O6 -- dR[k][i] = sum_n T[n][k] dY[n][i] with T = X L kept in fp64, for the
 * listed d_out columns i; output [r x nicols]. */
void slope_oracle_adapter_dR_cols(const uint16_t *X, const uint16_t *L, const uint16_t *dY,
                                  int b, int d_out, int d_in, int r,
                                  const int *icols, int nicols, double *dR)
{
    double *T = (double *)malloc(sizeof(double) * (size_t)b * r);
#pragma omp parallel for schedule(static)
    for (long n = 0; n < b; ++n)
        for (int k = 0; k < r; ++k) {
            double acc = 0.0;
            for (long j = 0; j < d_in; ++j)
                acc += bf16_to_double(X[n * d_in + j]) * bf16_to_double(L[j * r + k]);
            T[n * r + k] = acc;
        }
#pragma omp parallel for schedule(static)
    for (int k = 0; k < r; ++k)
        for (int s = 0; s < nicols; ++s) {
            long i = icols[s];
            double acc = 0.0;
            for (long n = 0; n < b; ++n) acc += T[n * r + k] * bf16_to_double(dY[n * d_out + i]);
            dR[(long)k * nicols + s] = acc;
        }
    free(T);
}

/* O7 -- Algorithm 1 "sparseAdd" (supplementary "Sparse matrix addition"): beta*A + gamma*B for
 * two compressed value arrays sharing one sparsity pattern, e.g. (1/gamma_scale) * dW + alpha * W
 * for weight decay under gradient scaling.  Element-wise, so the pattern never enters. */
void slope_oracle_sparse_add(const uint16_t *A, const uint16_t *B, double beta, double gamma,
                             long count, double *out)
{
    for (long e = 0; e < count; ++e) out[e] = beta * bf16_to_double(A[e]) + gamma * bf16_to_double(B[e]);
}

/* O8 -- Algorithm 1 "updateSparseMatrix" for the transposed copy: after the optimizer wrote new
 * values Wc_new (same first-pass pattern, [d_out x d_in/2]), rebuild the values of the
 * compressed (W^{R,C})^T under the static masks.  Slot t of group h of row j of the
 * transposed copy holds W_new[4h + q_t][j] when that element survived both passes, else +0;
 * W_new[i][j] sits in Wc_new at the rank of column j among the kept columns of its group. */
void slope_oracle_update_transposed(const uint16_t *Wc_new, const uint8_t *mask1, const uint8_t *mask2,
                                    const uint8_t *nibT, int d_out, int d_in, uint16_t *valsT)
{
    long mrow = d_in / 8;
    for (long j = 0; j < d_in; ++j)
        for (long h = 0; h < d_out / 4; ++h) {
            int n = nibT[j * (d_out / 4) + h];
            int q[2] = {n & 3, (n >> 2) & 3};
            for (int t = 0; t < 2; ++t) {
                long i = 4 * h + q[t];
                uint16_t v = 0;
                if (mask_get(mask2, mrow, i, j)) {
                    long g = j / 4;
                    int rank = 0;
                    for (long c = 4 * g; c < j; ++c) rank += mask_get(mask1, mrow, i, c);
                    v = Wc_new[i * (d_in / 2) + 2 * g + rank];
                }
                valsT[j * (d_out / 2) + 2 * h + t] = v;
            }
        }
}

/* Choose the n largest of m 15-bit magnitudes, one at a time: each round takes the
 * largest magnitude not taken yet, the lowest position among equals.  taken[t] = 1
 * for the kept positions. */
static void topn_of_m(const uint32_t *key, int n, int m, int *taken) {
    for (int t = 0; t < m; ++t) taken[t] = 0;
    for (int round = 0; round < n; ++round) {
        int best = -1;
        for (int t = 0; t < m; ++t) {
            if (taken[t]) continue;
            if (best < 0 || key[t] > key[best]) best = t;     /* strict: lower index wins ties */
        }
        taken[best] = 1;
    }
}

/* O9 -- general N:M first pass (Lemma 1's "row-wise N:M pruned" A^R; the accuracy
 * experiments emulate N:M by pruning the dense weight): in every group of m
 * consecutive entries of a row keep the n of largest magnitude.  Output is the
 * dense matrix with the pruned entries set to +0, and the bit mask. */
void slope_oracle_prune_nm(const uint16_t *W, int d_out, int d_in, int n, int m,
                           uint16_t *WR, uint8_t *mask1)
{
    long mrow = d_in / 8;
    memset(mask1, 0, (size_t)d_out * mrow);
    for (long i = 0; i < d_out; ++i)
        for (long g = 0; g < d_in / m; ++g) {
            uint32_t key[64];
            int taken[64];
            for (int t = 0; t < m; ++t) key[t] = W[i * d_in + m * g + t] & 0x7FFFu;
            topn_of_m(key, n, m, taken);
            for (int t = 0; t < m; ++t) {
                long j = m * g + t;
                WR[i * d_in + j] = taken[t] ? W[i * d_in + j] : (uint16_t)0;
                if (taken[t]) mask1[i * mrow + (j >> 3)] |= (uint8_t)(1u << (j & 7));
            }
        }
}

/* O10 -- general N:M second pass (Lemma 1's A^{R,C}): on the row-wise pruned
 * matrix, in every group of m consecutive entries of a COLUMN keep the n of
 * largest magnitude; entries the first pass removed enter with magnitude zero.
 * Output is dense, in W's orientation; mask2 = kept by both passes. */
void slope_oracle_double_prune_nm(const uint16_t *W, const uint8_t *mask1, int d_out, int d_in,
                                  int n, int m, uint16_t *WRC, uint8_t *mask2)
{
    long mrow = d_in / 8;
    memset(mask2, 0, (size_t)d_out * mrow);
    for (long j = 0; j < d_in; ++j)
        for (long h = 0; h < d_out / m; ++h) {
            uint32_t key[64];
            uint16_t v[64];
            int kept1[64], taken[64];
            for (int t = 0; t < m; ++t) {
                long i = m * h + t;
                kept1[t] = mask_get(mask1, mrow, i, j);
                v[t] = kept1[t] ? W[i * d_in + j] : (uint16_t)0;
                key[t] = v[t] & 0x7FFFu;
            }
            topn_of_m(key, n, m, taken);
            for (int t = 0; t < m; ++t) {
                long i = m * h + t;
                WRC[i * d_in + j] = taken[t] ? v[t] : (uint16_t)0;
                if (taken[t] && kept1[t]) mask2[i * mrow + (j >> 3)] |= (uint8_t)(1u << (j & 7));
            }
        }
}

/* O11 -- mask difference (supplementary "Comparison with Dynamic Sparsity: SR-STE":
 * the number of mask elements in which the mask of an iteration differs from the
 * converged one): count of element positions whose mask bits differ. */
long long slope_oracle_mask_difference(const uint8_t *mask_a, const uint8_t *mask_b, int rows, int cols)
{
    long long diff = 0;
    long mrow = cols / 8;
    for (long i = 0; i < rows; ++i)
        for (long j = 0; j < cols; ++j)
            diff += mask_get(mask_a, mrow, i, j) != mask_get(mask_b, mrow, i, j);
    return diff;
}

int slope_oracle_max_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
