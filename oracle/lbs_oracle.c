/*
 * CPU oracle for the local block shuffle (test infrastructure, not product code).
 *
 * Follows the paper's Algorithm 1 ("Channel Shuffle") after its first line: the
 * permuted channels are cut into blocks of m positions (Section "Information
 * Reorder - Channel Shuffle", m = 256), and inside each block the pair of
 * channels whose exchange improves the retained metric the most is swapped,
 * again and again, until no exchange improves it.  The quantity maximised is
 * the simplified objective (Eq. 5): the sum, over all rows and all groups of 4
 * consecutive permuted channels, of the 2 largest metric values
 * xi[j,c] = |W[j,c]| * s_c  (Eq. 3 with s_c = IR_c + alpha * AM_c).
 *
 * Arithmetic of one group's retained sum V(c0,c1,c2,c3):
 *   kept(j,k)  : slot k is among the 2 largest xi of row j (ties: lower slot wins)
 *   A_k        = sum_j kept(j,k) * |W[j,c_k]|          exact, as integers in units of 2^-24
 *   V          = ((s_c0*a0 + s_c1*a1) + s_c2*a2) + s_c3*a3,  a_k = A_k * 2^-24, fp64, no FMA
 * The row sum is therefore independent of the order rows are visited in.
 *
 * Nothing here is shared with the CUDA path; only tests and the benchmark's CPU
 * baseline call it.  Plain loops; OpenMP only across independent table entries.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

static inline double half_abs_value(uint16_t h)
{
    int e = (h >> 10) & 31;
    int m = h & 1023;
    if (e == 0) return ldexp((double)m, -24);
    return ldexp((double)(1024 + m), e - 25);
}

static inline int64_t half_abs_fixed(uint16_t h) /* |h| in units of 2^-24 */
{
    int e = (h >> 10) & 31;
    int64_t m = h & 1023;
    if (e == 0) return m;
    return (1024 + m) << (e - 1);
}

/* Retained metric sum of one group of 4 channels over all rows. */
static double group_value(const uint16_t *W, int No, long ldw, const double *s, const int32_t ch[4])
{
    int64_t A[4] = {0, 0, 0, 0};
    for (int j = 0; j < No; ++j) {
        const uint16_t *row = W + (long)j * ldw;
        double xi[4];
        for (int k = 0; k < 4; ++k) xi[k] = half_abs_value(row[ch[k]]) * s[ch[k]];
        for (int k = 0; k < 4; ++k) {
            int ahead = 0;
            for (int q = 0; q < 4; ++q) {
                if (q == k) continue;
                if (xi[q] > xi[k] || (xi[q] == xi[k] && q < k)) ++ahead;
            }
            if (ahead < 2) A[k] += half_abs_fixed(row[ch[k]]);
        }
    }
    double t0 = s[ch[0]] * ldexp((double)A[0], -24);
    double t1 = s[ch[1]] * ldexp((double)A[1], -24);
    double t2 = s[ch[2]] * ldexp((double)A[2], -24);
    double t3 = s[ch[3]] * ldexp((double)A[3], -24);
    return ((t0 + t1) + t2) + t3;
}

double lbs_oracle_group_value(const uint16_t *W, int No, long ldw, const double *s, const int32_t *ch)
{
    return group_value(W, No, ldw, s, ch);
}

/* Sum of group values over all groups of theta (the Eq. 5 objective). */
double lbs_oracle_objective(const uint16_t *W, int No, int C, long ldw, const double *s, const int32_t *theta)
{
    double total = 0.0;
    for (int g = 0; g < C / 4; ++g) total += group_value(W, No, ldw, s, theta + 4 * g);
    return total;
}

/*
 * theta: in = order after the global shuffle, out = order after the block shuffle.
 * incremental != 0 keeps a table S[g][slot][x] = V(group g with its slot replaced by
 * block channel x) and refreshes only the two touched groups after a swap;
 * incremental == 0 re-evaluates every candidate pair from the weights each iteration.
 * Both take the same decisions.
 * swaps_per_block / near_tie_swaps may be NULL.  Returns total swaps, or -1 on bad arguments.
 */
long long lbs_oracle_run(const uint16_t *W, int No, int C, long ldw, const double *s, int32_t *theta,
                         int block, int max_swaps, int incremental,
                         long long *swaps_per_block, long long *near_tie_swaps)
{
    if (C % 4 != 0 || block % 4 != 0 || block <= 0) return -1;
    long long total_swaps = 0;
    long long near = 0;
    int nblocks = (C + block - 1) / block;
    for (int b = 0; b < nblocks; ++b) {
        int p0 = b * block;
        int m = (C - p0 < block) ? (C - p0) : block; /* positions in this block */
        int G = m / 4;
        int32_t *pos2x = (int32_t *)malloc(sizeof(int32_t) * m);   /* position -> local channel id */
        int32_t *chan = (int32_t *)malloc(sizeof(int32_t) * m);    /* local channel id -> channel  */
        double *base = (double *)malloc(sizeof(double) * G);
        double *S = NULL;
        for (int p = 0; p < m; ++p) { pos2x[p] = p; chan[p] = theta[p0 + p]; }
        if (incremental) S = (double *)malloc(sizeof(double) * (size_t)G * 4 * m);

#define GROUP_CH(g, out) do { for (int k_ = 0; k_ < 4; ++k_) (out)[k_] = chan[pos2x[4 * (g) + k_]]; } while (0)
        for (int g = 0; g < G; ++g) { int32_t ch[4]; GROUP_CH(g, ch); base[g] = group_value(W, No, ldw, s, ch); }
        if (incremental) {
#pragma omp parallel for schedule(dynamic, 64)
            for (long e = 0; e < (long)G * 4 * m; ++e) {
                int x = (int)(e % m), slot = (int)((e / m) % 4), g = (int)(e / (4L * m));
                int32_t ch[4]; GROUP_CH(g, ch); ch[slot] = chan[x];
                S[e] = group_value(W, No, ldw, s, ch);
            }
        }
        long long swaps = 0;
        for (;;) {
            if (max_swaps > 0 && swaps >= max_swaps) break;
            double best = -INFINITY, second = -INFINITY;
            int bi = -1, bj = -1;
            if (incremental) {
                for (int i = 0; i < m; ++i) {
                    int gi = i / 4, si = i % 4;
                    for (int j = i + 1; j < m; ++j) {
                        int gj = j / 4, sj = j % 4;
                        if (gi == gj) continue;
                        double after = S[((long)gi * 4 + si) * m + pos2x[j]] + S[((long)gj * 4 + sj) * m + pos2x[i]];
                        double gain = after - (base[gi] + base[gj]);
                        if (gain > best) { second = best; best = gain; bi = i; bj = j; }
                        else if (gain > second) second = gain;
                    }
                }
            } else {
                long npairs = (long)m * m;
                double *gains = (double *)malloc(sizeof(double) * npairs);
#pragma omp parallel for schedule(dynamic, 8)
                for (long e = 0; e < npairs; ++e) {
                    int i = (int)(e / m), j = (int)(e % m);
                    gains[e] = -INFINITY;
                    if (j <= i || i / 4 == j / 4) continue;
                    int gi = i / 4, gj = j / 4;
                    int32_t ci[4], cj[4];
                    GROUP_CH(gi, ci); GROUP_CH(gj, cj);
                    int32_t t = ci[i % 4]; ci[i % 4] = cj[j % 4]; cj[j % 4] = t;
                    double after = group_value(W, No, ldw, s, ci) + group_value(W, No, ldw, s, cj);
                    gains[e] = after - (base[gi] + base[gj]);
                }
                for (long e = 0; e < npairs; ++e) {
                    int i = (int)(e / m), j = (int)(e % m);
                    if (j <= i || i / 4 == j / 4) continue;
                    double gain = gains[e];
                    if (gain > best) { second = best; best = gain; bi = i; bj = j; }
                    else if (gain > second) second = gain;
                }
                free(gains);
            }
            if (!(best > 0.0)) break;
            if (second > -INFINITY && (best - second) < 1e-6 * fabs(best)) ++near;
            int32_t t = pos2x[bi]; pos2x[bi] = pos2x[bj]; pos2x[bj] = t;
            ++swaps;
            int touched[2] = { bi / 4, bj / 4 };
            for (int q = 0; q < 2; ++q) {
                int g = touched[q];
                int32_t ch[4]; GROUP_CH(g, ch);
                base[g] = group_value(W, No, ldw, s, ch);
                if (incremental) {
#pragma omp parallel for schedule(dynamic, 64)
                    for (long e = 0; e < 4L * m; ++e) {
                        int x = (int)(e % m), slot = (int)(e / m);
                        int32_t c2[4]; GROUP_CH(g, c2); c2[slot] = chan[x];
                        S[((long)g * 4 + slot) * m + x] = group_value(W, No, ldw, s, c2);
                    }
                }
            }
        }
#undef GROUP_CH
        for (int p = 0; p < m; ++p) theta[p0 + p] = chan[pos2x[p]];
        if (swaps_per_block) swaps_per_block[b] = swaps;
        total_swaps += swaps;
        free(pos2x); free(chan); free(base); free(S);
    }
    if (near_tie_swaps) *near_tie_swaps = near;
    return total_swaps;
}
