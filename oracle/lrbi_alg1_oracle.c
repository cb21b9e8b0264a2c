/*
 * CPU oracle for the inner loop of Algorithm 1 (binary pruning-index-data matrix factorisation).
 *
 * TEST INFRASTRUCTURE ONLY, like lrbi_oracle.c: plain loops, one byte per bit, fp64 sums, no code
 * shared with the CUDA library.
 *
 * What it follows (Section 2.1 of the paper)
 *   - binary conversion of the NMF factors: (Ip)[i,j] = 1 if (Mp)[i,j] >= T_p, else 0, and the same
 *     for Iz with T_z (the sentence under Eq. 4; Eq. 4 -> Eq. 5 is its printed example);
 *   - the magnitude matrix M[i,j] = |W[i,j]| (first step of Algorithm 1) and the pruning index
 *     I[i,j] = 1 if |W[i,j]| >= theta (Eq. 1 -> Eq. 2, threshold 0.7 in the example);
 *   - the sparsity of a binary matrix = the fraction of its zeros (S, S_a, S_p, S_z above Eq. 7);
 *   - Cost = sum of M[i,j] over the positions with I[i,j] = 1 and (Ia)[i,j] = 0, the magnitude of
 *     the weights that the factorisation prunes unintentionally (the cost line of Algorithm 1).
 * Each tile of a tiled layer is its own factorisation problem (Section 3.1), so every count and
 * cost is reported per tile, tiles in row-major grid order.
 *
 * Precision: factor values are fp32 and are compared as they are; weights are bf16 bit patterns,
 * widened exactly; theta is an fp32 value; the cost is a sequential fp64 sum in index order.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

static double bf16_to_double(uint16_t h)
{
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/*
 * Binary conversion with one threshold per tile: values [ntiles][per_tile], T [ntiles],
 * out [ntiles][per_tile] bytes.  out = 1 iff value >= threshold.
 */
void lrbi_oracle_threshold(int64_t ntiles, int64_t per_tile, const float *values, const float *T, uint8_t *out)
{
    for (int64_t t = 0; t < ntiles; ++t)
        for (int64_t e = 0; e < per_tile; ++e)
            out[t * per_tile + e] = values[t * per_tile + e] >= T[t] ? 1 : 0;
}

/*
 * Per tile: kept_i = number of ones of I, kept_a = number of ones of Ia, lost = number of
 * positions with I = 1 and Ia = 0, cost = sum of |W| over those positions.
 *   W : [rows][cols] bf16 bits, Ia : [rows][cols] bytes, outputs [GR*GC].
 */
void lrbi_oracle_index_cost(int64_t rows, int64_t cols, int64_t tm, int64_t tn, const uint16_t *W, float theta,
                            const uint8_t *Ia, int64_t *kept_i, int64_t *kept_a, int64_t *lost, double *cost)
{
    const int64_t GR = (rows + tm - 1) / tm, GC = (cols + tn - 1) / tn;
    for (int64_t t = 0; t < GR * GC; ++t) { kept_i[t] = 0; kept_a[t] = 0; lost[t] = 0; cost[t] = 0.0; }
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t c = 0; c < cols; ++c) {
            const int64_t t = (r / tm) * GC + c / tn;
            const double m = fabs(bf16_to_double(W[r * cols + c]));   /* M = |W| */
            const int i = m >= (double)theta;                        /* I */
            const int a = Ia[r * cols + c] != 0;                      /* Ia */
            kept_i[t] += i;
            kept_a[t] += a;
            if (i && !a) { lost[t] += 1; cost[t] += m; }
        }
    }
}
