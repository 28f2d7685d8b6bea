/*
 * CPU oracle for block selection in unaligned block-wise pruning.
 *
 * TEST INFRASTRUCTURE ONLY. Nothing in the product path may call into this
 * file; it shares no code, header, table or helper with the library.
 *
 * What is here, and the passage each function follows:
 *   orc_block_scores   S_k = l1 norm of W[i:i+N, j, :, :], k = i + c_out*j,
 *                      -inf where the block would leave the weights      (Eq. 1)
 *   orc_bed_expand     block expansion: m times take the arg max of the
 *                      remaining score list, re-score the N-1 entries to its
 *                      left as if the chosen block's kernels were gone, drop
 *                      the N entries that start inside the chosen block, keep
 *                      the original index of the chosen entry        (Algorithm 1)
 *   orc_bed_divide     block division: sort the kept indices and re-cut
 *                      expanded blocks every N positions              (Algorithm 2)
 *   orc_greedy_select  best score first; the 2N-1 overlapping candidates of a
 *                      chosen block drop to -inf                          (Eq. 3)
 *   orc_optimal_select dynamic programme over (first k candidates, n chosen)
 *                                                                       (Eq. 4)
 *   orc_starts_to_mask kept blocks -> 0/1 mask over [c_out][c_in]
 *
 * Arithmetic. The scores decide an arg max, so the precision is part of the
 * result: scores, and the re-scoring S[k-n] <- (S[k-n] + S[k-n+N]) - S[k], are
 * single precision, evaluated in exactly that order; a kernel's l1 norm is the
 * sum of |w| over its taps in storage order, a block's score the sum of its N
 * kernels' norms in row order. Ties in an arg max go to the lowest position.
 * The dynamic programme is double precision (it is only compared by value).
 * Pins for every function live in the CPU test-suite (the paper's eight-weight
 * example, a brute-force restatement by window sums, exhaustive search on tiny
 * inputs, the aligned special case, invariants); none is "parity unpinned".
 */
#include <stdint.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

#define ORC_OK 0
#define ORC_E_ARG (-1)
#define ORC_E_SPACE (-3)

/* Eq. 1. W is [M][C][R] row-major (M = c_out, C = c_in, R = taps); S is [C*M], k = i + M*j. */
int orc_block_scores(const float *W, int M, int C, int R, int Nb, float *S)
{
    if (!W || !S || M < 1 || C < 1 || R < 1 || Nb < 1) return ORC_E_ARG;
    for (int j = 0; j < C; ++j)
        for (int i = 0; i < M; ++i) {
            float s = -INFINITY;
            if (i + Nb - 1 < M) {
                s = 0.0f;
                for (int t = 0; t < Nb; ++t) {
                    const float *w = W + ((size_t)(i + t) * C + j) * R;
                    float a = 0.0f;
                    for (int r = 0; r < R; ++r) a += fabsf(w[r]);
                    s += a;
                }
            }
            S[(size_t)i + (size_t)M * j] = s;
        }
    return ORC_OK;
}

static int64_t first_max(const float *S, int64_t len)
{
    int64_t k = 0;
    for (int64_t q = 1; q < len; ++q)
        if (S[q] > S[k]) k = q;
    return k;
}

/*
 * Algorithm 1. S_in holds the b scores; at most m indices are written to Ibar
 * (original candidate indices, in the order chosen) and optionally their
 * scores at the moment they were chosen. Returns how many were chosen: fewer
 * than m when no finite score is left. Positions k-n below the start of the
 * list do not exist and are skipped; a score past its end counts as -inf.
 */
int64_t orc_bed_expand(const float *S_in, int64_t b, int Nb, int64_t m, int64_t *Ibar, float *chosen_score)
{
    if (!S_in || !Ibar || b < 1 || Nb < 1 || m < 0) return ORC_E_ARG;
    float *S = (float *)malloc((size_t)b * sizeof(float));
    int64_t *Rl = (int64_t *)malloc((size_t)b * sizeof(int64_t));
    if (!S || !Rl) { free(S); free(Rl); return ORC_E_SPACE; }
    memcpy(S, S_in, (size_t)b * sizeof(float));
    for (int64_t q = 0; q < b; ++q) Rl[q] = q;
    int64_t len = b, cnt = 0;
    for (int64_t it = 0; it < m && len > 0; ++it) {
        const int64_t k = first_max(S, len);
        const float Sk = S[k];
        if (!(Sk > -INFINITY)) break;
        for (int n = 1; n < Nb; ++n) {
            if (k - n < 0) continue;
            const float right = (k - n + Nb < len) ? S[k - n + Nb] : -INFINITY;
            S[k - n] = (S[k - n] + right) - Sk;
        }
        Ibar[cnt] = Rl[k];
        if (chosen_score) chosen_score[cnt] = Sk;
        ++cnt;
        int64_t drop = Nb;
        if (k + drop > len) drop = len - k;
        memmove(S + k, S + k + drop, (size_t)(len - k - drop) * sizeof(float));
        memmove(Rl + k, Rl + k + drop, (size_t)(len - k - drop) * sizeof(int64_t));
        len -= drop;
    }
    free(S);
    free(Rl);
    return cnt;
}

static int cmp_i64(const void *a, const void *b)
{
    const int64_t x = *(const int64_t *)a, y = *(const int64_t *)b;
    return (x > y) - (x < y);
}

/*
 * Block division (Algorithm 2). Ibar (cnt chosen indices of the expansion, any order) -> I (cnt block start
 * indices, ascending). Seen on the original index axis, the kernels the expansion removed form runs: a chosen index
 * that lies at or beyond everything placed so far opens a run at its own position, and every further chosen index that
 * falls inside what the run already covers lengthens the run by one block. Division places the t-th block of a run at
 * run start + t * Nb, i.e. cuts each run every Nb positions from its first one.
 */
int orc_bed_divide(const int64_t *Ibar, int64_t cnt, int Nb, int64_t *I)
{
    if (cnt < 0 || Nb < 1 || (cnt > 0 && (!Ibar || !I))) return ORC_E_ARG;
    int64_t *sorted = (int64_t *)malloc((size_t)(cnt > 0 ? cnt : 1) * sizeof(int64_t));
    if (!sorted) return ORC_E_SPACE;
    memcpy(sorted, Ibar, (size_t)cnt * sizeof(int64_t));
    qsort(sorted, (size_t)cnt, sizeof(int64_t), cmp_i64);
    int64_t q = 0;
    while (q < cnt) {
        const int64_t run_start = sorted[q];
        int64_t blocks = 0;                           /* blocks of this run placed so far */
        do {
            I[q] = run_start + blocks * Nb;
            ++blocks;
            ++q;
        } while (q < cnt && sorted[q] < run_start + blocks * Nb);
    }
    free(sorted);
    return ORC_OK;
}

/*
 * Eq. 3, as the text describes it: candidates sorted by score (best first, lowest index among equals), walked in
 * that order; a candidate is taken unless an earlier choice set it to -inf, and taking k sets k-N+1 .. k+N-1 to
 * -inf. Returns the number chosen (fewer than m when nothing finite is left); I in the order chosen.
 */
static const float *g_sort_scores;
static int cmp_score_desc(const void *a, const void *b)
{
    const int64_t x = *(const int64_t *)a, y = *(const int64_t *)b;
    const float sx = g_sort_scores[x], sy = g_sort_scores[y];
    if (sx > sy) return -1;
    if (sx < sy) return 1;
    return (x > y) - (x < y);
}

int64_t orc_greedy_select(const float *S_in, int64_t b, int Nb, int64_t m, int64_t *I)
{
    if (!S_in || !I || b < 1 || Nb < 1 || m < 0) return ORC_E_ARG;
    int64_t *ord = (int64_t *)malloc((size_t)b * sizeof(int64_t));
    uint8_t *gone = (uint8_t *)calloc((size_t)b, 1);
    if (!ord || !gone) { free(ord); free(gone); return ORC_E_SPACE; }
    for (int64_t q = 0; q < b; ++q) ord[q] = q;
    g_sort_scores = S_in;
    qsort(ord, (size_t)b, sizeof(int64_t), cmp_score_desc);
    int64_t cnt = 0;
    for (int64_t q = 0; q < b && cnt < m; ++q) {
        const int64_t k = ord[q];
        if (!(S_in[k] > -INFINITY)) break;
        if (gone[k]) continue;
        I[cnt++] = k;
        for (int64_t n = -(int64_t)Nb + 1; n < Nb; ++n)
            if (k + n >= 0 && k + n < b) gone[k + n] = 1;
    }
    free(ord);
    free(gone);
    return cnt;
}

/*
 * Eq. 4. T[k][n] = best total of n non-overlapping blocks among the first k
 * candidates (indices 0..k-1); taking candidate k-1 leaves the first k-N.
 * Writes the chosen indices (ascending) to I and the total to *total; returns
 * the number chosen, m, or -1 when m blocks cannot be placed.
 */
int64_t orc_optimal_select(const float *S, int64_t b, int Nb, int64_t m, int64_t *I, double *total)
{
    if (!S || b < 1 || Nb < 1 || m < 0) return ORC_E_ARG;
    const size_t w = (size_t)m + 1;
    double *T = (double *)malloc((size_t)(b + 1) * w * sizeof(double));
    if (!T) return ORC_E_SPACE;
    for (int64_t k = 0; k <= b; ++k)
        for (int64_t n = 0; n <= m; ++n) {
            double v;
            if (n == 0) v = 0.0;
            else if (k == 0) v = -INFINITY;
            else {
                const int64_t kp = k - Nb < 0 ? 0 : k - Nb;
                /* with fewer than N candidates before it, the block can only be the first one chosen */
                const double prev = (k - Nb < 0 && n > 1) ? -INFINITY : T[(size_t)kp * w + (size_t)(n - 1)];
                const double take = prev + (double)S[k - 1];
                const double skip = T[(size_t)(k - 1) * w + (size_t)n];
                v = take > skip ? take : skip;
            }
            T[(size_t)k * w + (size_t)n] = v;
        }
    const double best = T[(size_t)b * w + (size_t)m];
    if (total) *total = best;
    int64_t got = -1;
    if (best > -INFINITY) {
        int64_t k = b, n = m;
        while (n > 0 && k > 0) {
            if (T[(size_t)k * w + (size_t)n] > T[(size_t)(k - 1) * w + (size_t)n]) {
                if (I) I[n - 1] = k - 1;
                k = k - Nb < 0 ? 0 : k - Nb;
                --n;
            } else {
                --k;
            }
        }
        got = (n == 0) ? m : -1;
    }
    free(T);
    return got;
}

/* Blocks with linear start index k = i + M*j -> mask[M][C] (row-major); -1 if a block leaves its column or overlaps. */
int orc_starts_to_mask(const int64_t *I, int64_t cnt, int M, int C, int Nb, uint8_t *mask)
{
    if (!mask || M < 1 || C < 1 || Nb < 1 || cnt < 0) return ORC_E_ARG;
    memset(mask, 0, (size_t)M * C);
    for (int64_t q = 0; q < cnt; ++q) {
        const int64_t k = I[q];
        if (k < 0 || k >= (int64_t)M * C) return ORC_E_ARG;
        const int64_t i = k % M, j = k / M;
        if (i + Nb > M) return ORC_E_ARG;
        for (int t = 0; t < Nb; ++t) {
            uint8_t *p = mask + (size_t)(i + t) * C + j;
            if (*p) return ORC_E_ARG;
            *p = 1;
        }
    }
    return ORC_OK;
}
