// CUDA kernels (sm_100a) for Y = act(Wm X + bias) on unaligned block-wise
// pruned weights, and their launchers.
//
// Dataflow (the output-stationary idea of Section 4.2, re-organised for SIMT):
// a warp owns a panel of P output rows x (32 lanes x 4V columns) and keeps it in
// registers for the whole reduction over input channels; the CTA's warps share
// one staged activation tile X[k0:k0+KT, strip] per pipeline stage. Blocks are
// consumed from the plan, bucketed by start offset inside the panel, and the
// kernel is statically unrolled over that offset, so every accumulator index is
// a compile-time constant (registers cannot be indexed at run time; this plays
// the role the weight rotation plays on the paper's SIMD register file).
//
// Staging: per pipeline stage one thread issues a TMA tensor copy of the X tile
// and a bulk copy of the plan group into shared memory, completing on an
// mbarrier; the warps wait on it, compute, and release the stage through a
// second mbarrier. All waits are bounded; a wait that runs out sets the plan's
// status word and the CTA drains and exits.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdio>
#include <mutex>

#include "ubp_internal.h"
#include "ubp_tc_common.cuh"

namespace ubp {

// ------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait. Returns false if the wait ran out or another thread of the CTA
// already gave up (abort flag in shared memory).
__device__ __forceinline__ uint64_t global_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag)
{
    constexpr uint64_t kLimitNs = 1000ull * 1000ull * 1000ull;   // one second, then give up
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_ns();
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 0u) {
            if (*abort_flag) return false;
            if (global_ns() - t0 > kLimitNs) break;
        }
    }
    *abort_flag = 1;
    return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *tm, int c0, int c1, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) { return __ffma2_rn(a, b, c); }

template <int N>
__device__ __forceinline__ void load_floats(float (&w)[N], const float *p)
{
    if constexpr (N == 1) {
        w[0] = p[0];
    } else if constexpr (N == 2) {
        const float2 t = *reinterpret_cast<const float2 *>(p);
        w[0] = t.x; w[1] = t.y;
    } else {
        static_assert(N % 4 == 0, "entry weights are loaded as float4");
#pragma unroll
        for (int q = 0; q < N / 4; ++q) {
            const float4 t = *reinterpret_cast<const float4 *>(p + 4 * q);
            w[4 * q] = t.x; w[4 * q + 1] = t.y; w[4 * q + 2] = t.z; w[4 * q + 3] = t.w;
        }
    }
}

// ------------------------------------------------------------------ main 1x1 kernel
// One fragment = all entries of this (panel, tile) whose first row sits at
// offset S inside the panel (S may be negative for an entry that started in the
// panel above). Rows outside [0, P) are clipped at compile time.
//
// The entry stream of a panel is contiguous across fragments, so the loads of
// entry e+1 (activation row, weights) and the channel index of entry e+2 are
// issued before the multiply-adds of entry e: a two-deep software pipeline
// that runs straight through fragment boundaries.
template <int V, int WF>
struct EntryRegs {
    float4 x[V];
    float w[WF];
};

template <int V, int WF, int XROW_BYTES>
__device__ __forceinline__ void fetch_entry(EntryRegs<V, WF> &r, const uint8_t *xs_lane, uint32_t j,
                                            const float *wv, int e)
{
    const uint8_t *xp = xs_lane + j * (uint32_t)XROW_BYTES;
#pragma unroll
    for (int v = 0; v < V; ++v) r.x[v] = *reinterpret_cast<const float4 *>(xp + v * 512);
    load_floats<WF>(r.w, wv + (size_t)e * WF);
}

template <int NBK, int P, int V, int S, bool DUPW>
__device__ __forceinline__ void fma_entry(float2 (&acc)[P][2 * V], const EntryRegs<V, NBK * (DUPW ? 2 : 1)> &r)
{
    constexpr int R_LO = (S < 0) ? -S : 0;
    constexpr int R_HI = (S + NBK > P) ? (P - S) : NBK;
#pragma unroll
    for (int q = R_LO; q < R_HI; ++q) {
        const float2 w2 = DUPW ? make_float2(r.w[2 * q], r.w[2 * q + 1]) : make_float2(r.w[q], r.w[q]);
#pragma unroll
        for (int v = 0; v < V; ++v) {
            acc[S + q][2 * v] = fma2(w2, make_float2(r.x[v].x, r.x[v].y), acc[S + q][2 * v]);
            acc[S + q][2 * v + 1] = fma2(w2, make_float2(r.x[v].z, r.x[v].w), acc[S + q][2 * v + 1]);
        }
    }
}

// Pipeline state carried across fragments: `cur` holds the next entry to be
// consumed (already loaded), jn the channel of the entry after it; wp / jp point
// at the weights / channel index of the entry in `cur`.
template <int V, int WF>
struct PipeState {
    EntryRegs<V, WF> cur;
    uint32_t jn;
    const float *wp;
    const uint16_t *jp;
};

// fragment offsets are held in registers as packed 16-bit pairs
template <int FOW>
__device__ __forceinline__ int fo_at(const uint32_t (&fw)[FOW], int f)
{
    return (f & 1) ? (int)(fw[f >> 1] >> 16) : (int)(fw[f >> 1] & 0xffffu);
}

template <int NBK, int P, int V, bool DUPW, int XROW_BYTES, int FOW, int F0, int F1>
struct FragmentLoop {
    static constexpr int WF = NBK * (DUPW ? 2 : 1);
    __device__ __forceinline__ static void run(float2 (&acc)[P][2 * V], PipeState<V, WF> &ps, const uint8_t *xs_lane,
                                               const uint32_t (&fw)[FOW])
    {
        if constexpr (F0 < F1) {
            constexpr int S = F0 - (NBK - 1);
            int cnt = fo_at<FOW>(fw, F0 + 1) - fo_at<FOW>(fw, F0);
            EntryRegs<V, WF> nxt;
            while (cnt >= 2) {
                fetch_entry<V, WF, XROW_BYTES>(nxt, xs_lane, ps.jn, ps.wp, 1);
                const uint32_t j2 = ps.jp[2];
                fma_entry<NBK, P, V, S, DUPW>(acc, ps.cur);
                fetch_entry<V, WF, XROW_BYTES>(ps.cur, xs_lane, j2, ps.wp, 2);
                ps.jn = ps.jp[3];
                fma_entry<NBK, P, V, S, DUPW>(acc, nxt);
                ps.wp += 2 * WF;
                ps.jp += 2;
                cnt -= 2;
            }
            if (cnt) {
                // odd tail: consume `cur`, then refill it in place (no register copies)
                const uint32_t j2 = ps.jp[2];
                fma_entry<NBK, P, V, S, DUPW>(acc, ps.cur);
                fetch_entry<V, WF, XROW_BYTES>(ps.cur, xs_lane, ps.jn, ps.wp, 1);
                ps.jn = j2;
                ps.wp += WF;
                ps.jp += 1;
            }
            FragmentLoop<NBK, P, V, DUPW, XROW_BYTES, FOW, F0 + 1, F1>::run(acc, ps, xs_lane, fw);
        }
    }
};

// ------------------------------------------------------------------ the other block orientation (K-runs)
// Plan entries of a configuration of kind 5: a run of NB consecutive input channels of ONE output row (fragment =
// the row inside the panel, so the accumulator is a compile-time constant again): one channel index, NB weights
// and NB activation rows of the staged tile per entry.
template <int NB, int P, int V, int XROW_BYTES, int FOW, int F0, int F1>
struct KrunLoop {
    __device__ __forceinline__ static void run(float2 (&acc)[P][2 * V], const uint8_t *xs_lane, const uint16_t *jl,
                                               const float *wv, const uint32_t (&fw)[FOW])
    {
        if constexpr (F0 < F1) {
            const int e1 = fo_at<FOW>(fw, F0 + 1);
#pragma unroll 2
            for (int e = fo_at<FOW>(fw, F0); e < e1; ++e) {
                const uint8_t *xp = xs_lane + (uint32_t)jl[e] * (uint32_t)XROW_BYTES;
                float w[NB];
                load_floats<NB>(w, wv + (size_t)e * NB);
                constexpr int TG = NB < 4 ? NB : 4;          // activation rows in flight at once
#pragma unroll
                for (int t0 = 0; t0 < NB; t0 += TG) {
                    float4 x[TG][V];
#pragma unroll
                    for (int t = 0; t < TG; ++t)
#pragma unroll
                        for (int v = 0; v < V; ++v)
                            x[t][v] = *reinterpret_cast<const float4 *>(xp + (t0 + t) * XROW_BYTES + v * 512);
#pragma unroll
                    for (int t = 0; t < TG; ++t) {
                        const float2 w2 = make_float2(w[t0 + t], w[t0 + t]);
#pragma unroll
                        for (int v = 0; v < V; ++v) {
                            acc[F0][2 * v] = fma2(w2, make_float2(x[t][v].x, x[t][v].y), acc[F0][2 * v]);
                            acc[F0][2 * v + 1] = fma2(w2, make_float2(x[t][v].z, x[t][v].w), acc[F0][2 * v + 1]);
                        }
                    }
                }
            }
            KrunLoop<NB, P, V, XROW_BYTES, FOW, F0 + 1, F1>::run(acc, xs_lane, jl, wv, fw);
        }
    }
};

struct SpmmArgs {
    const uint8_t *plan;     // device plan image
    const float *bias;       // [M] or null
    float *Y;
    int64_t ldy;
    int64_t Nc;
    int M;
    int nkt, NG;
    int nstrips;             // column strips of the product (a CTA walks every gridDim.y-th of them)
    int stages;
    uint32_t stage_bytes;    // X tile + largest plan group, 128-byte multiple
    int relu;
};

// All warps of the CTA compute; thread 0 also feeds the pipeline: before it starts on step `it` it issues the
// copies for step it + D (D = stages - 2) into the stage that every warp released two steps ago, so that wait
// almost never blocks. Each stage has a "full" mbarrier (completed by the copies' byte count) and an "empty"
// one (one arrival per warp).
template <int NBK, int P, int V, int WR, int WC, int KT, bool DUPW, bool KRUN>
__global__ void __launch_bounds__(WR * WC * 32, WR * WC <= 8 ? 2 : 1)
ubp_spmm_kernel(const __grid_constant__ CUtensorMap tmX, const SpmmArgs a)
{
    constexpr int CS = WC * 128 * V;               // columns per CTA
    constexpr int XT_BYTES = KT * CS * 4;
    constexpr int F = KRUN ? P : P + NBK - 1;      // fragments: rows of the panel (K-runs) or start offsets
    constexpr int NCW = WR * WC;                   // warps
    constexpr int FO_BYTES = ((F + 1) * 2 + 15) & ~15;
    constexpr int WF = NBK * (DUPW ? 2 : 1);
    constexpr int MAX_STAGES = 8;

    extern __shared__ __align__(1024) uint8_t smem[];
    __shared__ __align__(8) uint64_t bar_full[MAX_STAGES];
    __shared__ __align__(8) uint64_t bar_empty[MAX_STAGES];
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = blockIdx.x;                      // row group
    // The CTA is persistent over column strips blockIdx.y, blockIdx.y + gridDim.y, ...: the copy pipeline runs
    // straight across strip boundaries, so the loads of the next strip fly while this one computes and stores.
    const int my_strips = (a.nstrips - (int)blockIdx.y + (int)gridDim.y - 1) / (int)gridDim.y;
    const int total = my_strips * a.nkt;           // (strip, channel tile) steps of this CTA
    const int S = a.stages;
    const int D = S > 2 ? S - 2 : 1;               // steps in flight ahead of the one being computed
    const uint32_t *gtab = reinterpret_cast<const uint32_t *>(a.plan + 256);

    // Launched with programmatic stream serialisation: the next kernel in the stream may become resident while this one
    // drains, and this one sets its barriers up while its predecessor drains; nothing global is touched before the wait.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < S; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), NCW);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    __syncthreads();

    int issued = 0;                                // steps whose copies thread 0 has issued
    int iss_kt = 0, iss_strip = blockIdx.y;        // (channel tile, strip) of the next step to issue
    auto issue_step = [&]() -> bool {              // thread 0 only
        const int it = issued, st = it % S;
        if (it >= S && !mbar_wait(smem_u32(&bar_empty[st]), ((it / S) - 1) & 1, &abort_flag)) return false;
        const uint32_t o0 = gtab[(size_t)iss_kt * a.NG + g], o1 = gtab[(size_t)iss_kt * a.NG + g + 1];
        const uint32_t gbytes = (o1 - o0) * 16u;
        const uint32_t bar = smem_u32(&bar_full[st]);
        uint8_t *stage = smem + (size_t)st * a.stage_bytes;
        mbar_expect_tx(bar, (uint32_t)XT_BYTES + gbytes);
        tma_load_2d(smem_u32(stage), &tmX, iss_strip * CS, iss_kt * KT, bar);
        bulk_load(smem_u32(stage + XT_BYTES), a.plan + (size_t)o0 * 16u, gbytes, bar);
        ++issued;
        if (++iss_kt == a.nkt) { iss_kt = 0; iss_strip += gridDim.y; }
        return true;
    };
    if (threadIdx.x == 0)
        for (int it = 0; it < D && it < total; ++it) issue_step();

    const int wr = warp / WC, wc = warp % WC;
    const int panel = g * WR + wr;
    float2 acc[P][2 * V];

    bool ok = true;
    int kt = 0, strip = blockIdx.y;
    for (int it = 0; it < total; ++it) {
        if (threadIdx.x == 0 && it + D < total) ok = issue_step();
        if (kt == 0) {
#pragma unroll
            for (int r = 0; r < P; ++r)
#pragma unroll
                for (int q = 0; q < 2 * V; ++q) acc[r][q] = make_float2(0.f, 0.f);
        }
        const int st = it % S;
        ok = ok && mbar_wait(smem_u32(&bar_full[st]), (it / S) & 1, &abort_flag);
        if (!ok) break;
        const uint8_t *stage = smem + (size_t)st * a.stage_bytes;
        const uint8_t *grp = stage + XT_BYTES;
        const uint32_t po = reinterpret_cast<const uint32_t *>(grp)[wr];
        uint32_t pn = reinterpret_cast<const uint32_t *>(grp)[wr + 1];
#ifdef UBP_DEBUG
        {
            // checked build: the stage lies inside the CTA's shared memory; the panel's lists lie inside the stage, have
            // exactly the length their entry count implies and ascending fragment offsets; every entry names a channel
            // (K-runs: NBK channels) of the staged tile. A panel that fails is skipped.
            int *status = reinterpret_cast<int *>(const_cast<uint8_t *>(a.plan));
            bool good = UBP_CHK_SMEM((uint64_t)(st + 1) * a.stage_bytes <= tc::dbg_dynamic_smem() && po <= pn &&
                                     pn <= a.stage_bytes - (uint32_t)XT_BYTES, status);
            if (good && pn > po) {
                const uint16_t *fo = reinterpret_cast<const uint16_t *>(grp + po);
                const uint32_t n = fo[F];
                good = UBP_CHK_SMEM(pn - po == (uint32_t)FO_BYTES + ((2u * (n + 4) + 15u) & ~15u) + ((4u * (n + 2) * WF + 15u) & ~15u), status);
                for (int f = 0; good && f < F; ++f) good = UBP_CHK_SMEM(fo[f] <= fo[f + 1], status);
                const uint16_t *jl = reinterpret_cast<const uint16_t *>(grp + po + FO_BYTES);
                for (uint32_t e = lane; good && e < n; e += 32) good = UBP_CHK_SMEM((int)jl[e] + (KRUN ? NBK : 1) <= KT, status);
                good = __all_sync(0xffffffffu, good);
            }
            if (!good) pn = po;
        }
#endif
        if (pn > po) {                               // panel exists in this group
            constexpr int FOW = FO_BYTES / 4;
            uint32_t fw[FOW];
#pragma unroll
            for (int q = 0; q < FOW / 4; ++q) {
                const uint4 t = *reinterpret_cast<const uint4 *>(grp + po + 16 * q);
                fw[4 * q] = t.x; fw[4 * q + 1] = t.y; fw[4 * q + 2] = t.z; fw[4 * q + 3] = t.w;
            }
            const int n = fo_at<FOW>(fw, F);
            const uint8_t *xs_lane = stage + (wc * 128 * V + lane * 4) * 4;
            if constexpr (KRUN) {
                KrunLoop<NBK, P, V, CS * 4, FOW, 0, F>::run(acc, xs_lane, reinterpret_cast<const uint16_t *>(grp + po + FO_BYTES),
                                                            reinterpret_cast<const float *>(grp + po + FO_BYTES + ((2 * (n + 4) + 15) & ~15)), fw);
            } else {
            // the plan pads jl with 4 zero entries and w with 2 zero entries, so the pipeline may read ahead
            PipeState<V, WF> ps;
            ps.jp = reinterpret_cast<const uint16_t *>(grp + po + FO_BYTES);
            ps.wp = reinterpret_cast<const float *>(grp + po + FO_BYTES + ((2 * (n + 4) + 15) & ~15));
            fetch_entry<V, WF, CS * 4>(ps.cur, xs_lane, ps.jp[0], ps.wp, 0);
            ps.jn = ps.jp[1];
            FragmentLoop<NBK, P, V, DUPW, CS * 4, FOW, 0, F>::run(acc, ps, xs_lane, fw);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bar_empty[st]));
        if (++kt < a.nkt) continue;

        // ---------------- strip finished: bias, activation, one 128-bit store per lane and column group
        const int64_t col0 = (int64_t)strip * CS + wc * 128 * V + lane * 4;
#pragma unroll
        for (int r = 0; r < P; ++r) {
            const int row = panel * P + r;
            if (row < a.M) {
                const float b = a.bias ? __ldg(a.bias + row) : 0.f;
                float *yrow = a.Y + (size_t)row * a.ldy;
#pragma unroll
                for (int v = 0; v < V; ++v) {
                    const int64_t col = col0 + v * 128;
                    float4 o = make_float4(acc[r][2 * v].x + b, acc[r][2 * v].y + b,
                                           acc[r][2 * v + 1].x + b, acc[r][2 * v + 1].y + b);
                    if (a.relu) { o.x = fmaxf(o.x, 0.f); o.y = fmaxf(o.y, 0.f); o.z = fmaxf(o.z, 0.f); o.w = fmaxf(o.w, 0.f); }
                    if (!UBP_CHK_GMEM(col >= 0 && (col >= a.Nc || (size_t)row * a.ldy + col < (size_t)(a.M - 1) * a.ldy + a.Nc),
                                      reinterpret_cast<int *>(const_cast<uint8_t *>(a.plan)))) continue;
                    if (col + 3 < a.Nc) {
                        *reinterpret_cast<float4 *>(yrow + col) = o;
                    } else {
                        if (col < a.Nc) yrow[col] = o.x;
                        if (col + 1 < a.Nc) yrow[col + 1] = o.y;
                        if (col + 2 < a.Nc) yrow[col + 2] = o.z;
                    }
                }
            }
        }
        kt = 0;
        strip += gridDim.y;
    }
    if (!ok) {
        // A bounded wait ran out somewhere in this CTA: report through the plan's status word and stop
        // storing. Thread 0 first gives the copies it has in flight a bounded chance to land.
        if (threadIdx.x == 0) {
            const int first = issued > S ? issued - S : 0;
            for (int it = first; it < issued; ++it)
                for (uint32_t w = 0; w < (1u << 16); ++w)
                    if (mbar_try_wait(smem_u32(&bar_full[it % S]), (it / S) & 1)) break;
        }
        if (lane == 0) atomicExch(reinterpret_cast<int *>(const_cast<uint8_t *>(a.plan)), 1);
    }
}

// ------------------------------------------------------------------ fallback 1x1 kernel
// Any alignment, any leading dimension: one lane per output column, plan and
// activations read straight from global memory. Same plan, same summation
// order per output as the main kernel.
template <int NBK, int P, int S>
__device__ __forceinline__ void simple_fragment(float (&acc)[P], const float *xcol, int64_t ldx, bool live,
                                                const uint16_t *jl, const float *wv, int wstride, int wdup,
                                                int e0, int e1)
{
    constexpr int R_LO = (S < 0) ? -S : 0;
    constexpr int R_HI = (S + NBK > P) ? (P - S) : NBK;
    for (int e = e0; e < e1; ++e) {
        const float x = live ? xcol[(size_t)jl[e] * ldx] : 0.f;
#pragma unroll
        for (int r = R_LO; r < R_HI; ++r) acc[S + r] = fmaf(wv[(size_t)e * wstride + r * wdup], x, acc[S + r]);
    }
}
template <int NBK, int P, int F0, int F1>
struct SimpleLoop {
    __device__ __forceinline__ static void run(float (&acc)[P], const float *xcol, int64_t ldx, bool live,
                                               const uint16_t *fo, const uint16_t *jl, const float *wv,
                                               int wstride, int wdup, int e0)
    {
        if constexpr (F0 < F1) {
            const int e1 = fo[F0 + 1];
            simple_fragment<NBK, P, F0 - (NBK - 1)>(acc, xcol, ldx, live, jl, wv, wstride, wdup, e0, e1);
            SimpleLoop<NBK, P, F0 + 1, F1>::run(acc, xcol, ldx, live, fo, jl, wv, wstride, wdup, e1);
        }
    }
};

template <int NBK, int P>
__global__ void __launch_bounds__(128)
ubp_spmm_simple_kernel(const uint8_t *plan, const float *X, int64_t ldx, int64_t Nc, const float *bias, int relu,
                       float *Y, int64_t ldy, int M, int NP, int nkt, int NG, int WR, int KT, int dupw)
{
    constexpr int F = P + NBK - 1;
    constexpr int FO_BYTES = ((F + 1) * 2 + 15) & ~15;
    const int panel = blockIdx.y;
    const int64_t col = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const bool live = col < Nc;
    if (panel >= NP) return;
    const int g = panel / WR, wr = panel % WR;
    const uint32_t *gtab = reinterpret_cast<const uint32_t *>(plan + 256);
    float acc[P];
#pragma unroll
    for (int r = 0; r < P; ++r) acc[r] = 0.f;
    const int wdup = dupw ? 2 : 1;
    for (int kt = 0; kt < nkt; ++kt) {
        const uint8_t *grp = plan + (size_t)gtab[(size_t)kt * NG + g] * 16u;
        const uint32_t po = reinterpret_cast<const uint32_t *>(grp)[wr];
        const uint16_t *fo = reinterpret_cast<const uint16_t *>(grp + po);
        const int n = fo[F];
        const uint16_t *jl = reinterpret_cast<const uint16_t *>(grp + po + FO_BYTES);
        const float *wv = reinterpret_cast<const float *>(grp + po + FO_BYTES + ((2 * (n + 4) + 15) & ~15));
        const float *xcol = X + (size_t)kt * KT * ldx + (live ? col : 0);
        SimpleLoop<NBK, P, 0, F>::run(acc, xcol, ldx, live, fo, jl, wv, NBK * wdup, wdup, 0);
    }
    if (!live) return;
#pragma unroll
    for (int r = 0; r < P; ++r) {
        const int row = panel * P + r;
        if (row < M) {
            float o = acc[r] + (bias ? bias[row] : 0.f);
            if (relu) o = fmaxf(o, 0.f);
            Y[(size_t)row * ldy + col] = o;
        }
    }
}

// The same for K-run plans (kind 5): an entry is NB consecutive channels of one output row.
template <int NB, int P>
__global__ void __launch_bounds__(128)
ubp_spmm_krun_simple_kernel(const uint8_t *plan, const float *X, int64_t ldx, int64_t Nc, const float *bias, int relu,
                            float *Y, int64_t ldy, int M, int C, int NP, int nkt, int NG, int WR, int KT)
{
    constexpr int FO_BYTES = ((P + 1) * 2 + 15) & ~15;
    const int panel = blockIdx.y;
    const int64_t col = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (panel >= NP || col >= Nc) return;
    const int g = panel / WR, wr = panel % WR;
    const uint32_t *gtab = reinterpret_cast<const uint32_t *>(plan + 256);
    float acc[P];
#pragma unroll
    for (int r = 0; r < P; ++r) acc[r] = 0.f;
    for (int kt = 0; kt < nkt; ++kt) {
        const uint8_t *grp = plan + (size_t)gtab[(size_t)kt * NG + g] * 16u;
        const uint32_t po = reinterpret_cast<const uint32_t *>(grp)[wr];
        const uint16_t *fo = reinterpret_cast<const uint16_t *>(grp + po);
        const int n = fo[P];
        const uint16_t *jl = reinterpret_cast<const uint16_t *>(grp + po + FO_BYTES);
        const float *wv = reinterpret_cast<const float *>(grp + po + FO_BYTES + ((2 * (n + 4) + 15) & ~15));
#pragma unroll
        for (int r = 0; r < P; ++r)
            for (int e = fo[r]; e < fo[r + 1]; ++e) {
                const int c0 = kt * KT + jl[e];
#pragma unroll
                for (int t = 0; t < NB; ++t)      // channels past the layer's last one carry zero weights: skip the read
                    if (c0 + t < C) acc[r] = fmaf(wv[(size_t)e * NB + t], X[(size_t)(c0 + t) * ldx + col], acc[r]);
            }
    }
#pragma unroll
    for (int r = 0; r < P; ++r) {
        const int row = panel * P + r;
        if (row < M) {
            float o = acc[r] + (bias ? bias[row] : 0.f);
            if (relu) o = fmaxf(o, 0.f);
            Y[(size_t)row * ldy + col] = o;
        }
    }
}

// ------------------------------------------------------------------ 3x3 implicit kernel (first version)
// One lane per output pixel n = (b, y, x); the nine taps of an entry read the
// input plane in place (zero outside the image), so the lowered K = 9*C matrix
// never exists. Entry weights are [nbk][9].
template <int NBK, int P, int S>
__device__ __forceinline__ void conv_fragment(float (&acc)[P], const float *inb, int64_t isc, int y, int x, int H, int Wd,
                                              bool live, const uint16_t *jl, const float *wv, int kt_base, int e0, int e1)
{
    constexpr int R_LO = (S < 0) ? -S : 0;
    constexpr int R_HI = (S + NBK > P) ? (P - S) : NBK;
    for (int e = e0; e < e1; ++e) {
        const float *plane = inb + (size_t)(kt_base + jl[e]) * isc;
        const float *w = wv + (size_t)e * NBK * 9;
#pragma unroll
        for (int dy = 0; dy < 3; ++dy)
#pragma unroll
            for (int dx = 0; dx < 3; ++dx) {
                const int yy = y + dy - 1, xx = x + dx - 1;
                const bool in = live && yy >= 0 && yy < H && xx >= 0 && xx < Wd;
                const float xv = in ? __ldg(plane + (size_t)yy * Wd + xx) : 0.f;
#pragma unroll
                for (int r = R_LO; r < R_HI; ++r) acc[S + r] = fmaf(w[r * 9 + dy * 3 + dx], xv, acc[S + r]);
            }
    }
}
template <int NBK, int P, int F0, int F1>
struct ConvLoop {
    __device__ __forceinline__ static void run(float (&acc)[P], const float *inb, int64_t isc, int y, int x, int H, int Wd,
                                               bool live, const uint16_t *fo, const uint16_t *jl, const float *wv,
                                               int kt_base, int e0)
    {
        if constexpr (F0 < F1) {
            const int e1 = fo[F0 + 1];
            conv_fragment<NBK, P, F0 - (NBK - 1)>(acc, inb, isc, y, x, H, Wd, live, jl, wv, kt_base, e0, e1);
            ConvLoop<NBK, P, F0 + 1, F1>::run(acc, inb, isc, y, x, H, Wd, live, fo, jl, wv, kt_base, e1);
        }
    }
};

template <int NBK, int P>
__global__ void __launch_bounds__(128)
ubp_conv3x3_simple_kernel(const uint8_t *plan, const float *in, int B, int H, int Wd, int64_t isb, int64_t isc,
                          const float *bias, int relu, float *out, int64_t osb, int64_t osc,
                          int M, int NP, int nkt, int NG, int WR, int KT, int stride)
{
    constexpr int F = P + NBK - 1;
    constexpr int FO_BYTES = ((F + 1) * 2 + 15) & ~15;
    const int panel = blockIdx.y;
    const int64_t n = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int Ho = (H - 1) / stride + 1, Wo = (Wd - 1) / stride + 1;   // pad 1, 3x3: output pixel (yo, xo) is centred
    const int64_t total = (int64_t)B * Ho * Wo;                         // on input pixel (yo * stride, xo * stride)
    const bool live = n < total;
    const int64_t nn = live ? n : 0;
    const int b = (int)(nn / (Ho * Wo));
    const int pix = (int)(nn % (Ho * Wo));
    const int y = (pix / Wo) * stride, x = (pix % Wo) * stride;
    const int g = panel / WR, wr = panel % WR;
    const uint32_t *gtab = reinterpret_cast<const uint32_t *>(plan + 256);
    const float *inb = in + (size_t)b * isb;
    float acc[P];
#pragma unroll
    for (int r = 0; r < P; ++r) acc[r] = 0.f;
    for (int kt = 0; kt < nkt; ++kt) {
        const uint8_t *grp = plan + (size_t)gtab[(size_t)kt * NG + g] * 16u;
        const uint32_t po = reinterpret_cast<const uint32_t *>(grp)[wr];
        const uint16_t *fo = reinterpret_cast<const uint16_t *>(grp + po);
        const int cnt = fo[F];
        const uint16_t *jl = reinterpret_cast<const uint16_t *>(grp + po + FO_BYTES);
        const float *wv = reinterpret_cast<const float *>(grp + po + FO_BYTES + ((2 * (cnt + 4) + 15) & ~15));
        ConvLoop<NBK, P, 0, F>::run(acc, inb, isc, y, x, H, Wd, live, fo, jl, wv, kt * KT, 0);
    }
    if (!live) return;
#pragma unroll
    for (int r = 0; r < P; ++r) {
        const int row = panel * P + r;
        if (row < M) {
            float o = acc[r] + (bias ? bias[row] : 0.f);
            if (relu) o = fmaxf(o, 0.f);
            out[(size_t)b * osb + (size_t)row * osc + pix] = o;
        }
    }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

static int check(cudaError_t e)
{
    if (e == cudaSuccess) return UBP_OK;
    set_last_cuda_error((int)e);
    return UBP_E_CUDA;
}

constexpr size_t kSmemBudget = 227 * 1024 - 1024;   // dynamic shared memory we allow ourselves per CTA

template <int NBK, int P, int V, int WR, int WC, int KT, bool DUPW, bool KRUN>
static int launch_main(const ubp_plan *pl, const float *X, int64_t ldx, int64_t Nc, const float *bias, int relu,
                       float *Y, int64_t ldy, cudaStream_t stream)
{
    constexpr int CS = WC * 128 * V;
    constexpr size_t XT = (size_t)KT * CS * 4;
    const size_t stage_bytes = (XT + pl->img.max_group_bytes + 127) & ~(size_t)127;
    int stages = (int)(kSmemBudget / stage_bytes);
    if (stages < 2) return UBP_E_UNSUPPORTED;
    if (stages > 5) stages = 5;
    // Eight-warp configurations (layers of at most 64 rows): two CTAs per SM with three stages each hide the latency of
    // the entry loop and of the stores better than one CTA with five.
    constexpr bool kTwoPerSm = WR * WC <= 8;
    if (kTwoPerSm && stages >= 3 && 3 * stage_bytes <= 110 * 1024) stages = 3;

    EncodeTiledFn enc = encode_fn();
    if (!enc) return UBP_E_CUDA;
    CUtensorMap tm;
    const cuuint64_t dims[2] = {(cuuint64_t)Nc, (cuuint64_t)pl->dims.C};
    const cuuint64_t strides[1] = {(cuuint64_t)ldx * 4};
    const cuuint32_t box[2] = {(cuuint32_t)CS, (cuuint32_t)KT};
    const cuuint32_t estr[2] = {1, 1};
    CUresult cr = enc(&tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float *>(X), dims, strides, box, estr,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) { set_last_cuda_error(-(int)cr); return UBP_E_CUDA; }

    auto kern = ubp_spmm_kernel<NBK, P, V, WR, WC, KT, DUPW, KRUN>;
    const size_t smem = stage_bytes * stages;
    static bool attr_done[64] = {};                  // per device: opt in to large dynamic shared memory once
    int dev = 0;
    if (int rc = check(cudaGetDevice(&dev))) return rc;
    if (dev < 0 || dev >= 64 || !attr_done[dev]) {
        if (int rc = check(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget)))
            return rc;
        if (dev >= 0 && dev < 64) attr_done[dev] = true;
    }

    SpmmArgs a;
    a.plan = static_cast<const uint8_t *>(pl->dev);
    a.bias = bias; a.Y = Y; a.ldy = ldy; a.Nc = Nc; a.M = pl->dims.M;
    a.nkt = pl->img.nkt; a.NG = pl->img.NG; a.stages = stages; a.stage_bytes = (uint32_t)stage_bytes; a.relu = relu;
    // one CTA per SM is resident (shared memory); give every SM about one CTA and let it walk its strips
    const int nstrips = (int)((Nc + CS - 1) / CS);
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    int gy = (kTwoPerSm && stages == 3 ? 2 * sms : sms) / pl->img.NG;
    if (gy < 1) gy = 1;
    if (gy > nstrips) gy = nstrips;
    // even out the strips per CTA: with k strips each at most, do not launch more CTAs than needed for that k
    const int per = (nstrips + gy - 1) / gy;
    gy = (nstrips + per - 1) / per;
    a.nstrips = nstrips;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)pl->img.NG, (unsigned)gy);
    cfg.blockDim = dim3(WR * WC * 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tm, a);
    if (e == cudaSuccess) e = cudaGetLastError();
    return check(e);
}

template <int NBK, int P>
static int launch_simple(const ubp_plan *pl, const float *X, int64_t ldx, int64_t Nc, const float *bias, int relu,
                         float *Y, int64_t ldy, cudaStream_t stream)
{
    dim3 grid((unsigned)((Nc + 127) / 128), (unsigned)pl->img.NP);
    ubp_spmm_simple_kernel<NBK, P><<<grid, 128, 0, stream>>>(
        static_cast<const uint8_t *>(pl->dev), X, ldx, Nc, bias, relu, Y, ldy, pl->dims.M, pl->img.NP, pl->img.nkt,
        pl->img.NG, pl->cfg.WR, pl->cfg.KT, pl->cfg.dupw);
    return check(cudaGetLastError());
}

// Dispatch helpers: only the kernels a configuration kind can use are instantiated.
template <int KIND, int NBK, int P, int V, int WR, int WC, int KT, bool DUP>
struct CfgLaunch {
    static int main_kernel(const ubp_plan *pl, const float *X, int64_t ldx, int64_t Nc, const float *bias, int relu,
                           float *Y, int64_t ldy, cudaStream_t s)
    {
        if constexpr (KIND == 0) return launch_main<NBK, P, V, WR, WC, KT, DUP, false>(pl, X, ldx, Nc, bias, relu, Y, ldy, s);
        else if constexpr (KIND == 5) return launch_main<NBK, P, V, WR, WC, KT, DUP, true>(pl, X, ldx, Nc, bias, relu, Y, ldy, s);
        else return UBP_E_UNSUPPORTED;
    }
    static int simple_kernel(const ubp_plan *pl, const float *X, int64_t ldx, int64_t Nc, const float *bias, int relu,
                             float *Y, int64_t ldy, cudaStream_t s)
    {
        if constexpr (KIND == 0 || KIND == 2) return launch_simple<NBK, P>(pl, X, ldx, Nc, bias, relu, Y, ldy, s);
        else if constexpr (KIND == 5) {
            dim3 grid((unsigned)((Nc + 127) / 128), (unsigned)pl->img.NP);
            ubp_spmm_krun_simple_kernel<NBK, P><<<grid, 128, 0, s>>>(
                static_cast<const uint8_t *>(pl->dev), X, ldx, Nc, bias, relu, Y, ldy, pl->dims.M, pl->dims.C, pl->img.NP,
                pl->img.nkt, pl->img.NG, pl->cfg.WR, pl->cfg.KT);
            return check(cudaGetLastError());
        } else return UBP_E_UNSUPPORTED;
    }
    static int conv_kernel(const ubp_plan *pl, const float *in, int B, int H, int Wd, int64_t isb, int64_t isc,
                           const float *bias, int relu, float *out, int64_t osb, int64_t osc, cudaStream_t s, int stride)
    {
        if constexpr (KIND == 1 || KIND == 3) {
            const int64_t total = (int64_t)B * ((H - 1) / stride + 1) * ((Wd - 1) / stride + 1);
            dim3 grid((unsigned)((total + 127) / 128), (unsigned)pl->img.NP);
            ubp_conv3x3_simple_kernel<NBK, P><<<grid, 128, 0, s>>>(
                static_cast<const uint8_t *>(pl->dev), in, B, H, Wd, isb, isc, bias, relu, out, osb, osc, pl->dims.M,
                pl->img.NP, pl->img.nkt, pl->img.NG, pl->cfg.WR, pl->cfg.KT, stride);
            return check(cudaGetLastError());
        } else {
            return UBP_E_UNSUPPORTED;
        }
    }
};

int launch_spmm(const ubp_plan *pl, const float *X, int64_t ldx, int64_t Nc, const float *bias, int relu,
                float *Y, int64_t ldy, void *stream_)
{
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const KernelCfg &c = pl->cfg;
    const bool fast = ((reinterpret_cast<uintptr_t>(X) | reinterpret_cast<uintptr_t>(Y)) & 15) == 0 &&
                      (ldx % 4 == 0) && (ldy % 4 == 0) && (int64_t)ldx * 4 < (1ll << 40) &&
                      pl->dims.C < (1 << 30) && Nc < (1ll << 31);
    int rc = UBP_E_UNSUPPORTED;
    if (c.kind == 4) return launch_wros(pl, X, ldx, Nc, bias, relu, Y, ldy, stream_);
    if (fast && c.kind == 2) return launch_spmm_tc(pl, X, ldx, Nc, bias, relu, Y, ldy, stream);
#define UBP_CFG(ID, KIND, NBK, P_, V_, WR_, WC_, KT_, DUP)                                                \
    if (fast && c.id == ID)                                                                               \
        rc = CfgLaunch<KIND, NBK, P_, V_, WR_, WC_, KT_, (DUP != 0)>::main_kernel(pl, X, ldx, Nc, bias, relu, Y, ldy, stream);
#include "ubp_cfgs.inc"
#undef UBP_CFG
    if (rc != UBP_E_UNSUPPORTED) return rc;
    // slower kernel: unaligned operands, or a plan group too large to stage
#define UBP_CFG(ID, KIND, NBK, P_, V_, WR_, WC_, KT_, DUP) \
    if (c.id == ID)                                        \
        return CfgLaunch<KIND, NBK, P_, V_, WR_, WC_, KT_, (DUP != 0)>::simple_kernel(pl, X, ldx, Nc, bias, relu, Y, ldy, stream);
#include "ubp_cfgs.inc"
#undef UBP_CFG
    return UBP_E_UNSUPPORTED;
}

size_t conv3x3_strided_scratch_bytes(int C, int B, int H, int Wd, int stride)
{
    if (stride != 2 || C <= 0 || B <= 0 || H <= 0 || Wd <= 0) return 0;
    const int64_t cols = (int64_t)B * ((H - 1) / 2 + 1) * ((Wd - 1) / 2 + 1);
    return (size_t)4 * C * ((cols + 3) & ~(int64_t)3) * sizeof(float);
}

int launch_conv3x3(const ubp_plan *pl, const float *in, int B, int H, int Wd, int64_t isb, int64_t isc,
                   const float *bias, int relu, float *out, int64_t osb, int64_t osc, void *stream_, int stride,
                   void *scratch, size_t scratch_bytes)
{
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const KernelCfg &c = pl->cfg;
    const int64_t ohw = (int64_t)((H - 1) / stride + 1) * ((Wd - 1) / stride + 1);
    const int64_t total = (int64_t)B * ohw;
    // stride 2 with scratch: gather the four phase planes, then the padded-grid kernel with every tap a shift of one plane
    if (stride == 2 && scratch && cfg_conv3_shift(c) && osb == ohw && (reinterpret_cast<uintptr_t>(out) & 15) == 0 && osc % 4 == 0 &&
        osc >= total && total < (1ll << 30) && (reinterpret_cast<uintptr_t>(scratch) & 15) == 0 &&
        scratch_bytes >= conv3x3_strided_scratch_bytes(pl->dims.C, B, H, Wd, 2)) {
        const int Ho = (H - 1) / 2 + 1, Wo = (Wd - 1) / 2 + 1, C = pl->dims.C;
        const int64_t ld = (total + 3) & ~(int64_t)3;
        int sms = 148, devid = 0;
        if (cudaGetDevice(&devid) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, devid);
        int ncols = 0;
        if (conv3_pair_tile(pl->dims.M, C, B, Ho, Wo, sms, &ncols)) {
            float *planes = static_cast<float *>(scratch);
            if (int rc = launch_phase_planes(in, C, B, H, Wd, isb, isc, planes, ld, stream_)) return rc;
            tc::TcArgs a{};
            a.X = planes; a.conv = 1; a.H = Ho; a.W = Wo; a.isb = ohw; a.isc = ld; a.stride = 1;
            a.bias = bias; a.Y = out; a.ldy = osc; a.Nc = total; a.M = pl->dims.M; a.K = C * 9; a.relu = relu;
            a.status = reinterpret_cast<int *>(pl->dev); a.rpc = 128;
            const uint8_t *dev = static_cast<const uint8_t *>(pl->dev);
            const int rc = launch_conv3_pair(dev + pl->img.tc16_off, planes, ld, &a, pl->dims.M, C, B, Ho, Wo, sms, stream_, 1);
            if (rc != UBP_E_UNSUPPORTED) return rc;
        }
    }
    // tensor-core path: needs the output as one [M][B*Ho*Wo] matrix (batch stride = plane size) with 16-byte rows
    if (c.kind == 3 && osb == ohw && (reinterpret_cast<uintptr_t>(out) & 15) == 0 && osc % 4 == 0 &&
        osc >= total && total < (1ll << 31) && (int64_t)B * H * Wd < (1ll << 31))
        return launch_conv3x3_tc(pl, in, B, H, Wd, isb, isc, bias, relu, out, osc, stream_, stride);
#define UBP_CFG(ID, KIND, NBK, P_, V_, WR_, WC_, KT_, DUP) \
    if (c.id == ID)                                        \
        return CfgLaunch<KIND, NBK, P_, V_, WR_, WC_, KT_, (DUP != 0)>::conv_kernel(pl, in, B, H, Wd, isb, isc, bias, relu, out, osb, osc, stream, stride);
#include "ubp_cfgs.inc"
#undef UBP_CFG
    return UBP_E_UNSUPPORTED;
}

// Every stride-th pixel of every stride-th row of each input plane, into a dense channel-major tensor
// [C][B][Ho][Wo]: the activations a strided 1x1 convolution reads. One CTA per (four channels, image); a thread takes
// output pixels (yo, xo) of the four planes: four independent loads in flight, one 32-bit division per pixel.
constexpr int SUBS_CH = 4;
__global__ void __launch_bounds__(256) ubp_subsample_kernel(const float *__restrict__ in, int C, int B, int H, int Wd,
                                                             int64_t isb, int64_t isc, int stride, int Ho, int Wo,
                                                             float *__restrict__ out)
{
    const int c0 = (int)blockIdx.x * SUBS_CH, b = blockIdx.y;
    const int ohw = Ho * Wo;
    const float *src = in + (size_t)b * isb + (size_t)c0 * isc;
    for (int i = threadIdx.x; i < ohw; i += 256) {
        const int yo = i / Wo, xo = i - yo * Wo;
        const size_t off = (size_t)(yo * stride) * Wd + (size_t)xo * stride;
        float v[SUBS_CH];
#pragma unroll
        for (int k = 0; k < SUBS_CH; ++k) v[k] = c0 + k < C ? __ldg(src + (size_t)k * isc + off) : 0.f;
#pragma unroll
        for (int k = 0; k < SUBS_CH; ++k)
            if (c0 + k < C) out[((size_t)(c0 + k) * B + b) * ohw + i] = v[k];
    }
}

int launch_subsample(const float *in, int C, int B, int H, int Wd, int64_t isb, int64_t isc, int stride, float *out,
                     void *stream_)
{
    const int Ho = (H - 1) / stride + 1, Wo = (Wd - 1) / stride + 1;
    const int64_t total = (int64_t)C * B * Ho * Wo;
    if (total == 0) return UBP_OK;
    if (B > 65535 || (int64_t)Ho * Wo >= (1ll << 30)) return UBP_E_UNSUPPORTED;
    ubp_subsample_kernel<<<dim3((unsigned)((C + SUBS_CH - 1) / SUBS_CH), (unsigned)B), 256, 0, static_cast<cudaStream_t>(stream_)>>>(
        in, C, B, H, Wd, isb, isc, stride, Ho, Wo, out);
    return check(cudaGetLastError());
}

}  // namespace ubp
