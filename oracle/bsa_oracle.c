/*
 * CPU oracle for block-sparse masked attention.  TEST INFRASTRUCTURE ONLY:
 * the product (CUDA) path never links, imports or calls anything in this
 * directory, and this file shares no code with it.
 *
 * What it computes is the paper's definition of masked attention (Section 2.1,
 * Eq. 1): for one head, O_M = softmax(Q K^T / sqrt(d) + B_M) V, where
 * B_M(i,j) = 0 when the token pair (i,j) lies in an active logical block of
 * the mask M (the effective interaction set E(M)) and -inf otherwise.
 *
 * The mask is expanded to token pairs directly: query token i belongs to
 * block row i / B_Q, key token j to block column j / B_KV, and the pair is
 * active iff M[h][i / B_Q][j / B_KV] != 0.  No tiles, no merging, no
 * splitting, no online softmax: each row takes its scores over all reachable
 * keys, subtracts their maximum, exponentiates, sums and normalises, in fp64.
 *
 * Readings where the paper is silent (listed in the design notes):
 *  - a row with no reachable key gives O = 0 and LSE = -inf;
 *  - LSE = max + ln(sum of exp(score - max)), natural log;
 *  - N need not be a multiple of the block sizes: the last block is ragged and
 *    keys >= N do not exist.
 *
 * Section 2.1 gives Q as N_q x d and K, V as N_kv x d: the number of query
 * tokens (N) and of key tokens (N_kv) are separate arguments.
 *
 * Inputs are bf16 bit patterns (the same rounded values the GPU sees),
 * widened exactly to double; with fp16 != 0 they are IEEE half bit patterns
 * instead (the tensor type is a request property, Section 4.4).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static inline double bf16_to_double(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* IEEE 754 binary16: 1 sign, 5 exponent (bias 15), 10 fraction bits. */
static inline double f16_to_double(uint16_t h) {
    const int sign = h >> 15, e = (h >> 10) & 31, m = h & 1023;
    double v;
    if (e == 0) v = ldexp((double)m, -24);                 /* zero and subnormals: m * 2^-24 */
    else if (e == 31) v = m ? NAN : INFINITY;
    else v = ldexp((double)(1024 + m), e - 25);            /* (1 + m/1024) * 2^(e-15) */
    return sign ? -v : v;
}

static inline double in_to_double(uint16_t b, int fp16) { return fp16 ? f16_to_double(b) : bf16_to_double(b); }

int bsa_oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Evaluate n_sel query blocks.  Selected block s is (sel_head[s], sel_qblock[s]);
 * its rows are tokens sel_qblock[s]*B_Q ... (+B_Q-1), clipped to N; keys are tokens 0 ... N_kv-1.
 * row_step > 1 evaluates only every row_step-th row of each block (rows are
 * independent; used to bound oracle time on very dense requests); rows not
 * evaluated are left untouched in the outputs.
 *
 * mask : uint8 [H][nQb][nKb], nonzero = active
 * Q    : bf16 (or fp16) bits [H][N][d]        K,V: the same, [H][N_kv][d]
 * O    : double [n_sel][B_Q][d]     LSE: double [n_sel][B_Q]
 * pairs_out (optional): number of active token pairs evaluated.
 * Returns 0, or -1 on allocation failure.
 */
int bsa_oracle_blocks(const uint8_t* mask, int H, int nQb, int nKb, int B_Q, int B_KV, int64_t N, int64_t N_kv, int d,
                      int fp16,
                      const uint16_t* Q, const uint16_t* K, const uint16_t* V,
                      int n_sel, const int32_t* sel_head, const int32_t* sel_qblock, int row_step,
                      double* O, double* LSE, int64_t* pairs_out) {
    const double inv_sqrt_d = 1.0 / sqrt((double)d);
    int64_t pairs_total = 0;
    int failed = 0;
    (void)H;
    if (row_step < 1) row_step = 1;
#pragma omp parallel reduction(+ : pairs_total)
    {
        double* s = (double*)malloc(sizeof(double) * (size_t)(N_kv > 0 ? N_kv : 1));
        double* q = (double*)malloc(sizeof(double) * (size_t)d);
        double* acc = (double*)malloc(sizeof(double) * (size_t)d);
        if (!s || !q || !acc) {
#pragma omp atomic write
            failed = 1;
        } else {
#pragma omp for schedule(dynamic, 1)
            for (int sidx = 0; sidx < n_sel; ++sidx) {
                const int h = sel_head[sidx];
                const int bi = sel_qblock[sidx];
                const uint8_t* mrow = mask + ((size_t)h * nQb + bi) * nKb;
                const uint16_t* Kh = K + (size_t)h * N_kv * d;
                const uint16_t* Vh = V + (size_t)h * N_kv * d;
                for (int r = 0; r < B_Q; r += row_step) {
                    const int64_t i = (int64_t)bi * B_Q + r;
                    if (i >= N) break;
                    double* o_out = O + ((size_t)sidx * B_Q + r) * d;
                    const uint16_t* qi = Q + ((size_t)h * N + i) * d;
                    for (int c = 0; c < d; ++c) q[c] = in_to_double(qi[c], fp16);
                    /* scores over the reachable keys J(h,i) */
                    int64_t cnt = 0;
                    double m = -INFINITY;
                    for (int bj = 0; bj < nKb; ++bj) {
                        if (!mrow[bj]) continue;
                        int64_t j0 = (int64_t)bj * B_KV, j1 = j0 + B_KV;
                        if (j1 > N_kv) j1 = N_kv;
                        for (int64_t j = j0; j < j1; ++j) {
                            const uint16_t* kj = Kh + (size_t)j * d;
                            double dot = 0.0;
                            for (int c = 0; c < d; ++c) dot += q[c] * in_to_double(kj[c], fp16);
                            dot *= inv_sqrt_d;
                            s[j] = dot;
                            if (dot > m) m = dot;
                            ++cnt;
                        }
                    }
                    pairs_total += cnt;
                    for (int c = 0; c < d; ++c) acc[c] = 0.0;
                    if (cnt == 0) {
                        for (int c = 0; c < d; ++c) o_out[c] = 0.0;
                        LSE[(size_t)sidx * B_Q + r] = -INFINITY;
                        continue;
                    }
                    double l = 0.0;
                    for (int bj = 0; bj < nKb; ++bj) {
                        if (!mrow[bj]) continue;
                        int64_t j0 = (int64_t)bj * B_KV, j1 = j0 + B_KV;
                        if (j1 > N_kv) j1 = N_kv;
                        for (int64_t j = j0; j < j1; ++j) {
                            const double p = exp(s[j] - m);
                            l += p;
                            const uint16_t* vj = Vh + (size_t)j * d;
                            for (int c = 0; c < d; ++c) acc[c] += p * in_to_double(vj[c], fp16);
                        }
                    }
                    for (int c = 0; c < d; ++c) o_out[c] = acc[c] / l;
                    LSE[(size_t)sidx * B_Q + r] = m + log(l);
                }
            }
        }
        free(s);
        free(q);
        free(acc);
    }
    if (pairs_out) *pairs_out = pairs_total;
    return failed ? -1 : 0;
}
