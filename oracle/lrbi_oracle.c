/*
 * CPU oracle for inference with a layer pruned by a tiled low-rank binary index.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * hot path computes.  It is used by the tests, by the smoke check and by the
 * timed CPU-baseline leg of the benchmark, and by nothing else.  It shares no
 * code, header, table or helper with the CUDA library and never sees the packed
 * factor format of that library: every bit here is one byte (0 or 1).
 *
 * What it follows
 *   - Eq. 3 of the paper: (Ia)[i,j] = OR_{l=1..k} ( Ip[i,l] AND Iz[l,j] ).
 *   - Section 3.1 (tile-based factorisation): the index matrix is cut into
 *     equal blocks; every block has its own Ip (tm x k) and Iz (k x tn) of the
 *     same rank and is decoded on its own.
 *   - Section 2 (Eq. 1-2) and Section 2.2: a 1 in the index keeps the weight, a
 *     0 prunes it to zero; the decoded index Ia is the masking layer of the
 *     layer, so the layer output is Y = X * (W .* Ia)^T.
 *
 * Precision: weights and activations arrive as bf16 bit patterns (already
 * rounded once by the input generator).  They are widened exactly to double and
 * every sum is a sequential fp64 sum in index order.  A pruned position is
 * skipped (select), never multiplied by zero, so a NaN or Inf stored in a pruned
 * weight cannot reach the output.
 *
 * Threads (OpenMP) split the OUTER loop only; the arithmetic order inside one
 * output element never depends on the thread count.
 *
 * All entry points are pinned by tests that do not use this file to make
 * their expected values (the paper's printed worked example, brute-force
 * enumeration on tiny tiles, closed-form special cases, numpy's fp64 matmul for
 * the all-ones mask).  Nothing here is "parity unpinned".
 */
#include <stdint.h>
#include <string.h>

static double bf16_bits_to_double(uint16_t h)
{
    uint32_t u = ((uint32_t)h) << 16;   /* bf16 is the upper half of an IEEE fp32 */
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;                   /* fp32 -> fp64 is exact */
}

/* Eq. 3 on one tile, one output bit. ip_row: k bytes. iz_tile: k x tn bytes. */
static uint8_t boolean_dot(const uint8_t *ip_row, const uint8_t *iz_tile,
                           int64_t k, int64_t tn, int64_t j)
{
    uint8_t acc = 0;
    for (int64_t l = 0; l < k; ++l)
        acc |= (uint8_t)(ip_row[l] & iz_tile[l * tn + j]);
    return acc;
}

/*
 * Tiled Boolean product (Eq. 3 per tile, Section 3.1).
 *   Ip : [GR][GC][tm][k] bytes,  Iz : [GR][GC][k][tn] bytes,
 *   GR = ceil(rows/tm), GC = ceil(cols/tn);  M : [rows][cols] bytes.
 * Rows/columns of an edge tile that fall outside the matrix are ignored.
 */
void lrbi_oracle_decode(int64_t rows, int64_t cols, int64_t tm, int64_t tn, int64_t k,
                        const uint8_t *Ip, const uint8_t *Iz, uint8_t *M)
{
    const int64_t GC = (cols + tn - 1) / tn;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        const int64_t tr = r / tm, i = r % tm;
        for (int64_t c = 0; c < cols; ++c) {
            const int64_t tc = c / tn, j = c % tn;
            const int64_t tile = tr * GC + tc;
            const uint8_t *ip_row = Ip + (tile * tm + i) * k;
            const uint8_t *iz_tile = Iz + tile * k * tn;
            M[r * cols + c] = boolean_dot(ip_row, iz_tile, k, tn, j);
        }
    }
}

/*
 * The same product when every tile has its own rank (Section 3.1, last paragraph: each submatrix may
 * choose a different rank).  The factors are stored with room for kmax = the largest rank,
 *   Ip : [GR][GC][tm][kmax] bytes,  Iz : [GR][GC][kmax][tn] bytes,  ranks : [GR*GC],
 * and tile t uses its first ranks[t] columns of Ip / rows of Iz only: whatever lies beyond is ignored.
 */
void lrbi_oracle_decode_ranks(int64_t rows, int64_t cols, int64_t tm, int64_t tn, int64_t kmax,
                              const int32_t *ranks, const uint8_t *Ip, const uint8_t *Iz, uint8_t *M)
{
    const int64_t GC = (cols + tn - 1) / tn;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        const int64_t tr = r / tm, i = r % tm;
        for (int64_t c = 0; c < cols; ++c) {
            const int64_t tc = c / tn, j = c % tn;
            const int64_t tile = tr * GC + tc;
            const uint8_t *ip_row = Ip + (tile * tm + i) * kmax;
            const uint8_t *iz_tile = Iz + tile * kmax * tn;
            uint8_t acc = 0;
            for (int64_t l = 0; l < ranks[tile]; ++l)            /* Eq. 3 with k = the tile's own rank */
                acc |= (uint8_t)(ip_row[l] & iz_tile[l * tn + j]);
            M[r * cols + c] = acc;
        }
    }
}

/*
 * Masked layer forward:  Y[b][o] = sum_i  M[o][i] ? X[b][i] * W[o][i] : nothing.
 *   W : [N][K] bf16 bits, M : [N][K] bytes, X : [B][K] bf16 bits, Y : [B][N] fp64.
 */
void lrbi_oracle_masked_gemm(int64_t B, int64_t N, int64_t K,
                             const uint16_t *W, const uint8_t *M,
                             const uint16_t *X, double *Y)
{
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t b = 0; b < B; ++b) {
        for (int64_t o = 0; o < N; ++o) {
            double s = 0.0;
            for (int64_t i = 0; i < K; ++i) {
                if (M[o * K + i])
                    s += bf16_bits_to_double(X[b * K + i]) * bf16_bits_to_double(W[o * K + i]);
            }
            Y[b * N + o] = s;
        }
    }
}

/*
 * Backward pass of the masked layer (Section 2.2: the pruned network is retrained with the index Ia as its
 * masking layer, so gradients flow through kept weights only).  With Y = X (W .* Ia)^T and dY = dL/dY:
 *   dX[b][i] = sum_o  Ia[o][i] ? dY[b][o] * W[o][i] : nothing
 *   dW[o][i] = Ia[o][i] ? sum_b dY[b][o] * X[b][i] : 0          (a pruned weight gets no gradient)
 *   W : [N][K], M : [N][K] bytes, X : [B][K], dY : [B][N] (bf16 bits);  dX : [B][K], dW : [N][K] fp64.
 */
void lrbi_oracle_masked_backward(int64_t B, int64_t N, int64_t K, const uint16_t *W, const uint8_t *M,
                                 const uint16_t *X, const uint16_t *dY, double *dX, double *dW)
{
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t b = 0; b < B; ++b) {
        for (int64_t i = 0; i < K; ++i) {
            double s = 0.0;
            for (int64_t o = 0; o < N; ++o)
                if (M[o * K + i]) s += bf16_bits_to_double(dY[b * N + o]) * bf16_bits_to_double(W[o * K + i]);
            dX[b * K + i] = s;
        }
    }
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t o = 0; o < N; ++o) {
        for (int64_t i = 0; i < K; ++i) {
            double s = 0.0;
            if (M[o * K + i])
                for (int64_t b = 0; b < B; ++b)
                    s += bf16_bits_to_double(dY[b * N + o]) * bf16_bits_to_double(X[b * K + i]);
            dW[o * K + i] = s;
        }
    }
}

/*
 * The same two definitions restricted to chosen outputs, for layers too large to
 * evaluate in full: for sample s the mask row o = o_idx[s] is decoded from its
 * tiles' factors (Eq. 3), then Y[b_idx[s]][o] is summed as above.
 */
void lrbi_oracle_masked_gemm_samples(int64_t N, int64_t K, int64_t tm, int64_t tn, int64_t k,
                                     const uint16_t *W, const uint8_t *Ip, const uint8_t *Iz,
                                     const uint16_t *X, int64_t n_samples,
                                     const int64_t *b_idx, const int64_t *o_idx, double *out)
{
    const int64_t GC = (K + tn - 1) / tn;
    (void)N;
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t s = 0; s < n_samples; ++s) {
        const int64_t b = b_idx[s], o = o_idx[s];
        const int64_t tr = o / tm, i = o % tm;
        double acc = 0.0;
        for (int64_t c = 0; c < K; ++c) {
            const int64_t tc = c / tn, j = c % tn;
            const int64_t tile = tr * GC + tc;
            if (boolean_dot(Ip + (tile * tm + i) * k, Iz + tile * k * tn, k, tn, j))
                acc += bf16_bits_to_double(X[b * K + c]) * bf16_bits_to_double(W[o * K + c]);
        }
        out[s] = acc;
    }
}

/* Exact widening of bf16 bit patterns, exposed so tests can pin it. */
void lrbi_oracle_bf16_to_f64(int64_t n, const uint16_t *in, double *out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = bf16_bits_to_double(in[i]);
}

/* Number of threads the outer loops will use (reported beside timings). */
#ifdef _OPENMP
#include <omp.h>
int lrbi_oracle_threads(void) { return omp_get_max_threads(); }
#else
int lrbi_oracle_threads(void) { return 1; }
#endif
