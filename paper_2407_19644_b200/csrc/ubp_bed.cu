// Block selection by expansion and division (Section 4.1, Algorithms 1 and 2) on the device.
//
// The paper's procedure is sequential over one score list of length b = c_out * c_in: m times take the arg max,
// re-score the N-1 entries to its left, drop N entries. Two facts make it data-parallel without changing a bit of
// its result:
//   * a candidate's score is the l1 mass of the next N remaining kernels of ITS input channel (or -inf when fewer
//     remain), so choosing a block only changes scores inside the same input channel: the columns evolve
//     independently and meet only in the global arg max;
//   * inside a column the chosen scores never increase (a re-scored entry is at most the maximum just removed,
//     also in rounded arithmetic, because rounding is monotonic), so the global order of choices is the merge of
//     the per-column sequences by (score descending, input channel ascending, position in the sequence ascending)
//     -- lowest-index tie-breaking of the global arg max, restated.
// So: every column runs the expansion to exhaustion (one warp per column, the score list in shared memory), the
// m-th largest chosen score over all columns is found by a radix select, ties at that score are given to the
// lowest input channels first, and the mask is the set of kernels a column removed before its cut. Cutting the
// resulting runs of ones every N rows (Algorithm 2) is what ubp_pack does when it decodes the mask.
//
// Arithmetic (part of the result, because it decides an arg max): single precision throughout; a kernel's norm is
// the sum of |w| over its taps in storage order, a block's score the sum of its N kernels' norms in row order
// (Eq. 1), and a re-scored entry is (S[k-n] + S[k-n+N]) - S[k] in that order (Algorithm 1).
#include <cuda_runtime.h>

#include <cstdint>

#include "ubp_internal.h"

namespace ubp {
namespace bed {

constexpr uint16_t NONE = 0xFFFFu;
constexpr int MAX_M = 16384;

constexpr int FINE_SHIFT = 19;      // fine histogram bin = score bits >> 19 (below 4096 for finite scores)
constexpr int COARSE_SHIFT = 24;    // coarse histogram bin = score bits >> 24 = 32 fine bins

struct SelState {
    unsigned int coarse[128];    // chosen scores so far, by sign and the top seven exponent bits
    unsigned int fine[4096];     // and by sign, exponent and the top four mantissa bits
    unsigned int hist[4][256];   // radix-select histograms, one per pass
    unsigned int tau_lb;         // bits of a lower bound on the m-th largest chosen score (only ever rises)
    unsigned int pad;
    long long nsel;              // blocks selected in the end
};

struct Workspace {
    float *aT;        // [C][M] l1 norm of kernel (i, j)
    float *S;         // [C][M] Eq. 1 scores
    float *ev;        // [T][C] score of the t-th block chosen in column j
    uint16_t *order;  // [C][M] iteration at which kernel (i, j) left the list, NONE if it never did
    int *nev;         // [C] blocks chosen in column j
    int *cut;         // [C] how many of them are selected
    SelState *sel;
    size_t bytes;
};

static inline size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }

static Workspace carve(void *base, int M, int C, int Nb)
{
    Workspace w;
    const size_t mc = (size_t)M * C, T = (size_t)(M / Nb);
    size_t off = 0;
    auto take = [&](size_t n) { size_t o = off; off += up256(n); return reinterpret_cast<char *>(reinterpret_cast<uintptr_t>(base) + o); };
    w.aT = (float *)take(mc * 4);
    w.S = (float *)take(mc * 4);
    w.ev = (float *)take((T > 0 ? T : 1) * C * 4);
    w.order = (uint16_t *)take(mc * 2);
    w.nev = (int *)take((size_t)C * 4);
    w.cut = (int *)take((size_t)C * 4);
    w.sel = (SelState *)take(sizeof(SelState));
    w.bytes = off;
    return w;
}

// ---------------------------------------------------------------------------------------------------------------
// Eq. 1, part one: aT[j][i] = sum over taps of |W[i][j][r]| (storage order), written transposed so that an input
// channel's column is contiguous.
__global__ void __launch_bounds__(256) bed_norm_kernel(const float *__restrict__ W, int M, int C, int R, float *__restrict__ aT)
{
    __shared__ float tile[32][33];
    const int j0 = blockIdx.x * 32, i0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int ii = ty; ii < 32; ii += 8) {
        const int i = i0 + ii, j = j0 + tx;
        float a = 0.0f;
        if (i < M && j < C) {
            const float *w = W + ((size_t)i * C + j) * R;
            for (int r = 0; r < R; ++r) a += fabsf(w[r]);
        }
        tile[ii][tx] = a;
    }
    __syncthreads();
    for (int jj = ty; jj < 32; jj += 8) {
        const int j = j0 + jj, i = i0 + tx;
        if (i < M && j < C) aT[(size_t)j * M + i] = tile[tx][jj];
    }
}

// Eq. 1, part two: S[j][i] = aT[j][i] + ... + aT[j][i+N-1] in that order, -inf when the block would leave the column.
__global__ void __launch_bounds__(256) bed_window_kernel(const float *__restrict__ aT, int M, int C, int Nb, float *__restrict__ S)
{
    const size_t idx = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (idx >= (size_t)M * C) return;
    const int i = (int)(idx % (size_t)M);
    float s = __int_as_float(0xff800000);
    if (i + Nb <= M) {
        const float *a = aT + idx;
        s = a[0];
        for (int t = 1; t < Nb; ++t) s += a[t];
    }
    S[idx] = s;
}

// ---------------------------------------------------------------------------------------------------------------
// A lower bound on the m-th largest chosen score, shared by all columns while they run: every chosen score is
// counted in two histograms of its bit pattern (128 bins by sign and the top seven exponent bits; 4096 bins by
// sign, exponent and four mantissa bits), and the lower edge of the highest fine bin with at least m scores at or
// above it can only rise. A column whose best remaining score is below the bound stops: nothing it could still
// choose can be among the m best (its later scores are no larger).
// Warp-collective: lane l holds coarse bins [4 l, 4 l + 4), then fine bin l of the coarse bin where the count crosses m.
__device__ __forceinline__ void refresh_bound(SelState *st, unsigned long long m, int lane)
{
    const uint4 v = __ldcg(reinterpret_cast<const uint4 *>(st->coarse) + lane);
    const unsigned int c4[4] = {v.x, v.y, v.z, v.w};
    const unsigned long long t = (unsigned long long)v.x + v.y + v.z + v.w;
    unsigned long long incl = t;                 // sum over lanes >= lane
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const unsigned long long o = __shfl_down_sync(0xffffffffu, incl, off);
        if (lane + off < 32) incl += o;
    }
    unsigned long long above = incl - t;
    const bool mine = above < m && incl >= m;
    int cb = 0;
    if (mine) {
        bool found = false;
#pragma unroll
        for (int b = 3; b >= 0; --b)
            if (!found) {
                if (above + c4[b] >= m) { cb = lane * 4 + b; found = true; }
                else above += c4[b];
            }
    }
    const unsigned int who = __ballot_sync(0xffffffffu, mine);
    if (who == 0u) return;                       // fewer than m scores so far
    const int src = __ffs(who) - 1;
    cb = __shfl_sync(0xffffffffu, cb, src);
    above = __shfl_sync(0xffffffffu, above, src);    // scores in coarse bins above cb
    const unsigned long long f = __ldcg(st->fine + cb * 32 + lane);
    unsigned long long fin = f;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const unsigned long long o = __shfl_down_sync(0xffffffffu, fin, off);
        if (lane + off < 32) fin += o;
    }
    // the highest fine bin with at least m scores at or above it (the counts may have grown since the first look,
    // which only makes the bound found here lower than it could be)
    const unsigned int ok = __ballot_sync(0xffffffffu, above + fin >= m);
    if (ok != 0u && lane == 0) atomicMax(&st->tau_lb, (unsigned int)(cb * 32 + (31 - __clz(ok))) << FINE_SHIFT);
}

__device__ __forceinline__ void flush_counts(SelState *st, unsigned int bin, unsigned int cnt)
{
    if (cnt) {
        atomicAdd(&st->fine[bin], cnt);
        atomicAdd(&st->coarse[bin >> (COARSE_SHIFT - FINE_SHIFT)], cnt);
    }
}

// Algorithm 1 for one input channel per warp. Shared memory per warp: the scores (padded with -inf to a multiple
// of 128), a doubly linked list over the entries still in the list (entry M = end marker), and the positions met
// while walking N steps to either side of the chosen entry. Lane l owns the entries of the float4 groups
// l, l + 32, ... and keeps their maximum in registers; after a choice only the lanes that own a changed entry
// look at their entries again.
// NS > 0: the block size, known at compile time and small: lane 0 alone walks the list, re-scores and drops (its
// loops unroll and their operands stay in registers); NS = 0: any block size, the lanes share that work through a
// scratch array.
template <int NS>
__global__ void __launch_bounds__(32) bed_expand_kernel(const float *__restrict__ S, int M, int C, int Nb, int Mpad, int T,
                                                        unsigned long long m, SelState *st,
                                                        float *__restrict__ ev, uint16_t *__restrict__ order,
                                                        int *__restrict__ nev)
{
    extern __shared__ __align__(16) unsigned char smem[];
    float *s = reinterpret_cast<float *>(smem);
    uint16_t *nxt = reinterpret_cast<uint16_t *>(s + Mpad);
    uint16_t *prv = nxt + (M + 1);
    uint16_t *wk = prv + (M + 1);                  // [2][Nb + 1]: successors, predecessors
    const int lane = threadIdx.x;
    const int j = blockIdx.x;
    const float NEG = __int_as_float(0xff800000);
    const float *Sj = S + (size_t)j * M;
    uint16_t *oj = order + (size_t)j * M;
    for (int i = lane; i < Mpad; i += 32) s[i] = i < M ? Sj[i] : NEG;
    for (int i = lane; i <= M; i += 32) {
        nxt[i] = (uint16_t)(i < M ? i + 1 : M);
        prv[i] = (uint16_t)(i > 0 ? i - 1 : NONE);
    }
    for (int i = lane; i < M; i += 32) oj[i] = NONE;
    __syncwarp();

    const float4 *s4 = reinterpret_cast<const float4 *>(s);
    const int G = Mpad >> 7;                        // float4 groups per lane
    float lbest;
    int lidx;
    // maximum of this lane's entries and the lowest position that holds it: the first float4 group that reaches the
    // maximum, then the first component of that group
    auto rescan = [&]() {
        float mx = NEG;
        int gb = 0;
#pragma unroll 4
        for (int g = 0; g < G; ++g) {
            const float4 v = s4[lane + 32 * g];
            const float m4 = fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w));
            if (m4 > mx) { mx = m4; gb = g; }
        }
        const float4 v = s4[lane + 32 * gb];
        const int base = (lane + 32 * gb) << 2;
        lidx = v.x == mx ? base : v.y == mx ? base + 1 : v.z == mx ? base + 2 : base + 3;
        lbest = mx;
    };
    rescan();

    unsigned int tau_next = __ldcg(&st->tau_lb);
    unsigned int pend_bin = 0, pend_cnt = 0;        // lane 0: chosen scores not yet added to the shared histograms
    float *evp = ev + j;
    int it = 0;
    for (; it < T; ++it) {
        // arg max, lowest position among equals. Scores are finite and >= 0 (or -inf), so their order is the
        // order of their bit patterns; bits + 1 leaves 0 for -inf.
        const unsigned int kb = lbest > NEG ? __float_as_uint(lbest) + 1u : 0u;
        const unsigned int mk = __reduce_max_sync(0xffffffffu, kb);
        if (mk == 0u) break;
        const int bidx = (int)__reduce_min_sync(0xffffffffu, kb == mk ? (unsigned int)lidx : 0x7fffffffu);
        const float best = __uint_as_float(mk - 1u);
        if (__float_as_uint(best) < tau_next) break;        // below the m-th largest score of the whole layer
        tau_next = __ldcg(&st->tau_lb);                      // looked at in the next round
        const int k = bidx;
        unsigned int dirty = 0;
        if constexpr (NS > 0) {
            if (lane == 0) {
                unsigned succ[NS + 1], pred[NS];
                unsigned cur = (unsigned)k;
#pragma unroll
                for (int t = 1; t <= NS; ++t) { cur = nxt[cur]; succ[t] = cur; }       // succ[NS] may be the end marker
                cur = (unsigned)k;
#pragma unroll
                for (int n = 1; n < NS; ++n) { cur = cur == NONE ? NONE : prv[cur]; pred[n] = cur; }
                const unsigned p1 = NS > 1 ? pred[NS > 1 ? 1 : 0] : (unsigned)prv[k];
                float sv[NS];
#pragma unroll
                for (int t = 1; t < NS; ++t) sv[t] = s[succ[t]];
                // entry n to the left now spans n kernels before the block and N-n after it
#pragma unroll
                for (int n = 1; n < NS; ++n)
                    if (pred[n] != NONE) {
                        s[pred[n]] = (s[pred[n]] + sv[NS - n]) - best;
                        dirty |= 1u << ((pred[n] >> 2) & 31u);
                    }
                s[k] = NEG;
                oj[k] = (uint16_t)it;
                dirty |= 1u << (((unsigned)k >> 2) & 31u);
#pragma unroll
                for (int t = 1; t < NS; ++t) {
                    s[succ[t]] = NEG;
                    oj[succ[t]] = (uint16_t)it;
                    dirty |= 1u << ((succ[t] >> 2) & 31u);
                }
                if (p1 != NONE) nxt[p1] = (uint16_t)succ[NS];
                prv[succ[NS]] = (uint16_t)p1;
                *evp = best;
                evp += C;
                // count it; a column's scores fall, so equal bins come in runs: one update per run
                const unsigned int bin = __float_as_uint(best) >> FINE_SHIFT;
                if (bin != pend_bin) {
                    flush_counts(st, pend_bin, pend_cnt);
                    pend_bin = bin;
                    pend_cnt = 0;
                }
                ++pend_cnt;
            }
            dirty = __shfl_sync(0xffffffffu, dirty, 0);
            __syncwarp();
        } else {
            // the N entries after k (lane 0) and before it (lane 1) that are still in the list
            if (lane < 2) {
                const uint16_t *link = lane == 0 ? nxt : prv;
                uint16_t *out = wk + lane * (Nb + 1);
                unsigned cur = (unsigned)k;
                for (int t = 1; t <= Nb; ++t) {
                    cur = cur == NONE ? NONE : link[cur];
                    out[t] = (uint16_t)cur;
                }
            }
            __syncwarp();
            // entry n to the left now spans n kernels before the block and N-n after it
            for (int n = 1 + lane; n < Nb; n += 32) {
                const unsigned p = wk[(Nb + 1) + n];
                if (p != NONE) {
                    const unsigned r = wk[Nb - n];
                    s[p] = (s[p] + s[r]) - best;
                    dirty |= 1u << ((p >> 2) & 31u);
                }
            }
            __syncwarp();
            for (int t = lane; t < Nb; t += 32) {
                const unsigned idx = t == 0 ? (unsigned)k : wk[t];
                s[idx] = NEG;
                oj[idx] = (uint16_t)it;
                dirty |= 1u << ((idx >> 2) & 31u);
            }
            if (lane == 0) {
                const unsigned p1 = wk[(Nb + 1) + 1], sN = wk[Nb];
                if (p1 != NONE) nxt[p1] = (uint16_t)sN;
                prv[sN] = (uint16_t)p1;
                *evp = best;
                evp += C;
                // count it; a column's scores fall, so equal bins come in runs: one update per run
                const unsigned int bin = __float_as_uint(best) >> FINE_SHIFT;
                if (bin != pend_bin) {
                    flush_counts(st, pend_bin, pend_cnt);
                    pend_bin = bin;
                    pend_cnt = 0;
                }
                ++pend_cnt;
            }
            dirty = __reduce_or_sync(0xffffffffu, dirty);
            __syncwarp();
        }
        if ((dirty >> lane) & 1u) rescan();
        if ((it & 15) == 15) {
            if (lane == 0) { flush_counts(st, pend_bin, pend_cnt); pend_cnt = 0; }
            refresh_bound(st, m, lane);
        }
    }
    if (lane == 0) {
        flush_counts(st, pend_bin, pend_cnt);
        nev[j] = it;
    }
}

// ---------------------------------------------------------------------------------------------------------------
// The m-th largest chosen score over all columns: radix select over the bit patterns (scores are finite and >= 0,
// so unsigned order of the bits is the order of the values), 8 bits per pass from the top. The digit a pass settles
// is read off its histogram by whoever needs it next (warp-collective; lane l holds bins [8 l, 8 l + 8)).
__device__ __forceinline__ void settle_digit(const unsigned int *hist_row, int shift, unsigned int &prefix,
                                             unsigned long long &rank, int lane)
{
    unsigned int v[8];
    unsigned long long t = 0;
#pragma unroll
    for (int b = 0; b < 8; ++b) { v[b] = __ldcg(hist_row + lane * 8 + b); t += v[b]; }
    unsigned long long incl = t;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const unsigned long long o = __shfl_down_sync(0xffffffffu, incl, off);
        if (lane + off < 32) incl += o;
    }
    const unsigned long long above = incl - t;
    const bool mine = above < rank && incl >= rank;
    unsigned int d = 0;
    unsigned long long nr = 0;
    if (mine) {
        unsigned long long cum = above;
#pragma unroll
        for (int b = 7; b >= 0; --b) {
            if (nr == 0) {
                if (cum + v[b] >= rank) { d = (unsigned)(lane * 8 + b); nr = rank - cum; }
                else cum += v[b];
            }
        }
    }
    const unsigned int who = __ballot_sync(0xffffffffu, mine);
    const int src = who ? __ffs(who) - 1 : 0;
    d = __shfl_sync(0xffffffffu, d, src);
    nr = __shfl_sync(0xffffffffu, nr, src);
    prefix |= d << shift;
    rank = nr;
}

// (prefix, rank) after `passes` settled digits; rank = 0 means there is nothing to select. Warp-collective.
__device__ __forceinline__ void settled(const SelState *st, int passes, unsigned long long m, unsigned int &prefix,
                                        unsigned long long &rank, int lane)
{
    prefix = 0;
    rank = 0;
    if (passes == 0) return;
    unsigned long long t = 0;
    for (int b = lane; b < 256; b += 32) t += __ldcg(&st->hist[0][b]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) t += __shfl_xor_sync(0xffffffffu, t, off);
    rank = m < t ? m : t;
    if (rank == 0) return;
    for (int p = 0; p < passes; ++p) settle_digit(st->hist[p], 24 - 8 * p, prefix, rank, lane);
}

__global__ void __launch_bounds__(256) bed_hist_kernel(const float *__restrict__ ev, const int *__restrict__ nev, int T, int C,
                                                       int pass, unsigned long long m, SelState *st)
{
    __shared__ unsigned int h[256];
    __shared__ unsigned int prefix_s;
    __shared__ unsigned long long rank_s;
    h[threadIdx.x] = 0;
    if (threadIdx.x < 32) {
        unsigned int prefix;
        unsigned long long rank;
        settled(st, pass, m, prefix, rank, threadIdx.x);
        if (threadIdx.x == 0) { prefix_s = prefix; rank_s = rank; }
    }
    __syncthreads();
    if (pass > 0 && rank_s == 0) return;
    const int shift = 24 - 8 * pass;
    const unsigned int prefix = prefix_s;
    const size_t total = (size_t)T * C;
    for (size_t idx = (size_t)blockIdx.x * 256 + threadIdx.x; idx < total; idx += (size_t)gridDim.x * 256) {
        const int j = (int)(idx % (size_t)C), t = (int)(idx / (size_t)C);
        if (t < nev[j]) {
            const unsigned int key = __float_as_uint(ev[idx]);
            if (pass == 0 || (key >> (shift + 8)) == (prefix >> (shift + 8))) atomicAdd(&h[(key >> shift) & 255u], 1u);
        }
    }
    __syncthreads();
    if (h[threadIdx.x]) atomicAdd(&st->hist[pass][threadIdx.x], h[threadIdx.x]);
}

// Per column: how many of its chosen blocks score above the threshold, how many exactly at it; ties are handed out
// to the lowest input channels first. One CTA, columns in chunks of 1024 with a running carry.
__global__ void __launch_bounds__(1024) bed_cut_kernel(const float *__restrict__ ev, const int *__restrict__ nev, int C,
                                                        unsigned long long m, SelState *st, int *__restrict__ cut,
                                                        long long *nsel_out)
{
    __shared__ unsigned long long warp_sum[32];
    __shared__ unsigned long long carry_s;
    __shared__ long long nsel_s;
    __shared__ unsigned int tau_s;
    __shared__ unsigned long long r_s;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    if (tid == 0) { carry_s = 0; nsel_s = 0; }
    if (wid == 0) {
        unsigned int prefix;
        unsigned long long rank;
        settled(st, 4, m, prefix, rank, lane);
        if (lane == 0) { tau_s = prefix; r_s = rank; }
    }
    __syncthreads();
    const unsigned int tau = tau_s;
    const unsigned long long r = r_s;
    const bool none = r == 0;
    for (int j0 = 0; j0 < C; j0 += 1024) {
        const int j = j0 + tid;
        int gt = 0, eq = 0;
        if (j < C && !none) {
            const int n = nev[j];
            int lo = 0, hi = n;                     // first position whose score is <= tau
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if (__float_as_uint(ev[(size_t)mid * C + j]) > tau) lo = mid + 1; else hi = mid;
            }
            gt = lo;
            hi = n;                                 // first position whose score is < tau
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if (__float_as_uint(ev[(size_t)mid * C + j]) >= tau) lo = mid + 1; else hi = mid;
            }
            eq = lo - gt;
        }
        // exclusive prefix sum of eq over the chunk
        unsigned long long incl = (unsigned long long)eq;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned long long o = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += o;
        }
        if (lane == 31) warp_sum[wid] = incl;
        __syncthreads();
        if (wid == 0) {
            unsigned long long w = warp_sum[lane];
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const unsigned long long o = __shfl_up_sync(0xffffffffu, w, off);
                if (lane >= off) w += o;
            }
            warp_sum[lane] = w;                     // inclusive over warps
        }
        __syncthreads();
        const unsigned long long before = carry_s + (wid > 0 ? warp_sum[wid - 1] : 0ull) + incl - (unsigned long long)eq;
        int c = 0;
        if (j < C && !none) {
            const unsigned long long left = r > before ? r - before : 0ull;
            c = gt + (int)((unsigned long long)eq < left ? (unsigned long long)eq : left);
        }
        if (j < C) cut[j] = c;
        long long cs = c;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) cs += __shfl_xor_sync(0xffffffffu, cs, off);
        __syncthreads();
        if (lane == 0 && cs) atomicAdd((unsigned long long *)&nsel_s, (unsigned long long)cs);
        if (tid == 0) carry_s += warp_sum[31];
        __syncthreads();
    }
    if (tid == 0) {
        st->nsel = nsel_s;
        if (nsel_out) *nsel_out = nsel_s;
    }
}

// mask[i][j] = 1 when kernel (i, j) left its column's list before the column's cut.
__global__ void __launch_bounds__(256) bed_mask_kernel(const uint16_t *__restrict__ order, const int *__restrict__ cut, int M, int C,
                                                       uint8_t *__restrict__ mask)
{
    __shared__ uint8_t tile[32][33];
    const int i0 = blockIdx.x * 32, j0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int jj = ty; jj < 32; jj += 8) {
        const int j = j0 + jj, i = i0 + tx;
        uint8_t v = 0;
        if (i < M && j < C) v = (int)order[(size_t)j * M + i] < cut[j] ? 1 : 0;
        tile[jj][tx] = v;
    }
    __syncthreads();
    for (int ii = ty; ii < 32; ii += 8) {
        const int i = i0 + ii, j = j0 + tx;
        if (i < M && j < C) mask[(size_t)i * C + j] = tile[tx][ii];
    }
}

static int check(cudaError_t e)
{
    if (e == cudaSuccess) return UBP_OK;
    set_last_cuda_error((int)e);
    return UBP_E_CUDA;
}

static int check_dims(int M, int C, int R, int Nb)
{
    if (M < 1 || C < 1 || R < 1 || Nb < 1 || Nb > M) return UBP_E_ARG;
    if (M > MAX_M || (int64_t)M * C >= ((int64_t)1 << 31)) return UBP_E_UNSUPPORTED;
    return UBP_OK;
}

static int launch_scores(const float *W, int M, int C, int R, int Nb, float *aT, float *S, cudaStream_t st)
{
    dim3 g1((unsigned)((C + 31) / 32), (unsigned)((M + 31) / 32));
    bed_norm_kernel<<<g1, 256, 0, st>>>(W, M, C, R, aT);
    const size_t mc = (size_t)M * C;
    bed_window_kernel<<<(unsigned)((mc + 255) / 256), 256, 0, st>>>(aT, M, C, Nb, S);
    return check(cudaGetLastError());
}

}  // namespace bed
}  // namespace ubp

using namespace ubp::bed;

extern "C" {

int ubp_bed_workspace_size(int M, int C, int Nb, size_t *dev_bytes)
{
    if (!dev_bytes) return UBP_E_ARG;
    if (int rc = check_dims(M, C, 1, Nb)) return rc;
    *dev_bytes = carve(nullptr, M, C, Nb).bytes;
    return UBP_OK;
}

int ubp_block_scores(const float *W, int M, int C, int R, int Nb, void *workspace, size_t workspace_bytes,
                     float *S, void *stream)
{
    if (!W || !workspace || !S) return UBP_E_ARG;
    if (int rc = check_dims(M, C, R, Nb)) return rc;
    if (((uintptr_t)workspace & 255u) != 0) return UBP_E_ARG;
    Workspace w = carve(workspace, M, C, Nb);
    if (workspace_bytes < w.bytes) return UBP_E_SPACE;
    return launch_scores(W, M, C, R, Nb, w.aT, S, (cudaStream_t)stream);
}

int ubp_bed_select(const float *W, int M, int C, int R, int Nb, int64_t m, void *workspace, size_t workspace_bytes,
                   uint8_t *mask, int64_t *n_selected, void *stream)
{
    if (!W || !workspace || !mask || m < 0) return UBP_E_ARG;
    if (int rc = check_dims(M, C, R, Nb)) return rc;
    if (((uintptr_t)workspace & 255u) != 0) return UBP_E_ARG;
    Workspace w = carve(workspace, M, C, Nb);
    if (workspace_bytes < w.bytes) return UBP_E_SPACE;
    cudaStream_t st = (cudaStream_t)stream;
    if (int rc = launch_scores(W, M, C, R, Nb, w.aT, w.S, st)) return rc;

    const int Mpad = (M + 127) & ~127;
    const size_t smem = (size_t)Mpad * 4 + (size_t)(M + 1) * 4 + (size_t)(Nb + 1) * 4;
    using ExpandFn = void (*)(const float *, int, int, int, int, int, unsigned long long, SelState *, float *, uint16_t *, int *);
    const ExpandFn expand = Nb == 1 ? bed_expand_kernel<1> : Nb == 2 ? bed_expand_kernel<2> : Nb == 4 ? bed_expand_kernel<4>
                            : Nb == 8 ? bed_expand_kernel<8> : bed_expand_kernel<0>;
    if (smem > 48 * 1024)
        if (int rc = check(cudaFuncSetAttribute(expand, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)))
            return rc;
    if (int rc = check(cudaMemsetAsync(w.sel, 0, sizeof(SelState), st))) return rc;
    const int T = M / Nb;
    expand<<<(unsigned)C, 32, smem, st>>>(w.S, M, C, Nb, Mpad, m > 0 ? T : 0, (unsigned long long)m, w.sel,
                                                     w.ev, w.order, w.nev);
    if (int rc = check(cudaGetLastError())) return rc;
    const size_t total = (size_t)T * C;
    unsigned hb = (unsigned)((total + 255) / 256);
    if (hb > 1184) hb = 1184;
    if (hb < 1) hb = 1;
    for (int pass = 0; pass < 4; ++pass)
        bed_hist_kernel<<<hb, 256, 0, st>>>(w.ev, w.nev, T, C, pass, (unsigned long long)m, w.sel);
    bed_cut_kernel<<<1, 1024, 0, st>>>(w.ev, w.nev, C, (unsigned long long)m, w.sel, w.cut, (long long *)n_selected);
    dim3 gm((unsigned)((M + 31) / 32), (unsigned)((C + 31) / 32));
    bed_mask_kernel<<<gm, 256, 0, st>>>(w.order, w.cut, M, C, mask);
    return check(cudaGetLastError());
}

}  // extern "C"
