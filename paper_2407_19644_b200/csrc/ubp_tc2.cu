// Two-CTA form of the tensor-core kernel, for the 1x1 product and the 3x3 implicit GEMM (see ubp_tc.cu for the
// arithmetic: densified panels, three TF32 products per fp32 product, fp32 accumulation in tensor memory).
//
// A cluster of two CTAs (two SMs) computes tiles of 256 output rows x N columns with tcgen05.mma.cta_group::2:
// every MMA has M = 256, CTA r supplies rows 128r..128r+127 of W from its own shared memory and columns
// r*N/2 .. r*N/2 + N/2 - 1 of X from its own shared memory, and keeps its 128 rows x N columns of the accumulator in
// its own tensor memory. Per SM that halves the X operand reads of the one-CTA kernel, which is what bounds that
// kernel on shared-memory bandwidth.
//
// X is not transposed at all here. The activations lie in memory as [channel][column] with columns contiguous, which
// is the "MN-major" form of the B operand; for 32-bit elements the tensor core reads that form from shared memory in
// the 128-byte swizzle with 32-byte atoms, which is also a TMA swizzle mode. So TMA copies [16 channels] x [32
// columns] boxes of X straight into the operand layout, and the MMA consumes the raw fp32 words: the tensor core
// drops the low 13 mantissa bits itself, i.e. it multiplies by Xh. The only work left for the SM's threads is the
// low part Xl = X - Xh, an elementwise pass from the raw tile to a second tile in the same layout.
//
// The kernel is persistent: at most one CTA pair per SM pair, each walking the tiles pair, pair + #pairs, ...
// The copy / Xl / MMA pipeline runs straight through tile boundaries, and there are two accumulators in tensor
// memory, so the epilogue of tile t (tensor memory -> bias, ReLU -> global memory) runs under the main loop of
// tile t + 1.
//
// 3x3 (stride 1, padding 1; template parameter CONV): the reduction index is k = tap * C + channel with C a multiple
// of 16, so a chunk belongs to one tap, i.e. to one shift dy * W + dx of the flattened (b, y, x) column axis. TMA
// cannot start a row at an odd element, so it copies the chunk's 16 channel rows for the tile's columns plus a halo
// either side, and the Xl warps cut the shifted tile out of that copy, zero the taps that fall outside the image,
// and write both Xh and Xl in the operand layout.
//
// Per CTA: warp 0 = TMA producer (its Wh / Wl rows and its X columns, one 3-D box each per chunk); warp 1 = in the
// leader CTA (cluster rank 0) issues all MMAs for the pair (the whole warp walks the loop, one elected lane issues)
// and commits stages and accumulators back to BOTH CTAs (tcgen05.commit with a cluster multicast mask);
// warps 2..9 = Xl pass (two groups taking turns on the chunks); warps 10..17 = epilogue (on a CTA's last tile,
// when nothing is left to overlap with, the Xl warps take half of the epilogue). The Xl warps of
// BOTH CTAs arrive on one barrier per stage in the leader's shared memory (the peer's through a mapa-translated
// address) once their CTA's copies have landed and its Xl tile is written, so the issuing thread waits once per
// chunk; the epilogue warps of both CTAs likewise hand an accumulator back to the leader. Every waiter sees every
// phase of the barriers it waits on (a parity wait cannot tell phase k from phase k + 2).
// No TMA load is multicast. All waits are bounded; a wait that runs out sets the plan's status word, and every path
// ends in the same cluster barrier and tensor-memory release.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "ubp_internal.h"
#include "ubp_tc_common.cuh"

namespace ubp {

namespace {

using namespace tc;

constexpr int T2_XL_WARPS = 8;                            // warps 2..9
constexpr int T2_XL_GROUPS = 2;                           // two groups of four warps take turns on the chunks
constexpr int T2_EPI_WARPS = 8;                           // warps 10..17
constexpr int T2_THREADS = (2 + T2_XL_WARPS + T2_EPI_WARPS) * 32;
constexpr int T2_MAX_STAGES = 8;                          // pipeline stages: as many as fit, at most this
constexpr uint32_t T2_A_HALF = 128 * TC_KC * 4;           // Wh or Wl chunk of this CTA's 128 rows: 8 KB
constexpr uint32_t T2_XG = 32 * TC_KC * 4;                // one box of X: 16 channels x 32 columns, 2 KB
constexpr uint32_t T2_PIPE_BUDGET = 222 * 1024;           // pipeline stages together
// a stage = Wh + Wl chunk (16 KB) + raw X + Xl of `ngrp` 32-column boxes (2 KB each): 20 .. 32 KB, 8 or 6 stages.
// The count is a multiple of T2_XL_GROUPS so that a stage always belongs to the same group of Xl warps: a waiter
// must see every phase of a barrier it waits on (a parity wait cannot tell phase k from phase k + 2).
// For 3x3 a stage also holds the raw copy the shifted tiles are cut from: 16 channels x (columns + 2 x halo) floats,
// halo = image width + 1 rounded up to a multiple of 4 (0 for 1x1), padded to a multiple of 1 KB.
__host__ __device__ constexpr uint32_t t2_raw_bytes(int ngrp, int halo)
{
    return halo ? (((uint32_t)(ngrp * 32 + 2 * halo) * TC_KC * 4 + 1023u) & ~1023u) : 0u;
}
__host__ __device__ constexpr uint32_t t2_stage_bytes(int ngrp, int halo)
{
    return 2 * T2_A_HALF + 2 * (uint32_t)ngrp * T2_XG + t2_raw_bytes(ngrp, halo);
}
__host__ __device__ constexpr int t2_stages(int ngrp, int halo)
{
    const int s = (int)(T2_PIPE_BUDGET / t2_stage_bytes(ngrp, halo));
    return (s > T2_MAX_STAGES ? T2_MAX_STAGES : s) / T2_XL_GROUPS * T2_XL_GROUPS;
}
constexpr uint32_t SWZ_128B_ATOM32 = 1;                   // descriptor layout type: 128-byte swizzle, 32-byte atoms
constexpr uint32_t T2_LBO = T2_XG;                        // next 32 columns
constexpr uint32_t T2_SBO = 4 * 128;                      // next 4 channels
constexpr uint32_t T2_ACC_COLS = 256;                     // tensor-memory columns per accumulator

// instruction descriptor: D = f32, A = B = tf32, A K-major, B MN-major, M = 256 (two CTAs), N = n
__device__ __forceinline__ uint32_t make_idesc2(int n)
{
    return (1u << 4) | (2u << 7) | (2u << 10) | (1u << 16) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}
// One chunk's six MMAs (two 8-channel steps x {Wh Xh, Wl Xh, Wh Xl}) and the commit that hands the stage back to
// both CTAs, in a single statement, with a non-blocking test of the NEXT chunk's barrier issued first and its result
// read last, so that the test's latency is hidden behind the MMA issue. Descriptor offsets are in 16-byte units: the
// next 8 channels of W are 32 bytes on (+2), of X eight 128-byte rows on (+64). Returns whether the next chunk's
// barrier phase has completed. Executed by a whole converged warp: one elected lane issues the MMAs and the
// commit, the operands stay warp-uniform.
__device__ __forceinline__ bool mma2_chunk(uint32_t d_tmem, uint64_t dWh, uint64_t dX, uint32_t w_lo_off,
                                           uint32_t x_lo_off, uint32_t idesc, uint32_t acc_first, uint32_t next_bar,
                                           uint32_t next_parity, uint32_t empty_bar)
{
    uint32_t ready;
    asm volatile(
        "{\n\t.reg .pred pn, pa, pt, pe;\n\t.reg .b64 wh, wl, xh, xl;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 pn, [%8], %9;\n\t"
        "elect.sync _|pe, 0xffffffff;\n\t"
        "setp.ne.b32 pa, %7, 0;\n\t"
        "setp.eq.b32 pt, %10, 0;\n\t"
        "cvt.u64.u32 wl, %4;\n\tadd.s64 wl, wl, %2;\n\t"
        "cvt.u64.u32 xl, %5;\n\tadd.s64 xl, xl, %3;\n\t"
        // (Wh is used twice per 8 channels: the second product takes it from the tensor core's operand collector)
        "@pe tcgen05.mma.cta_group::2.kind::tf32.collector::a::fill [%1], %2, %3, %6, pa;\n\t"
        "@pe tcgen05.mma.cta_group::2.kind::tf32.collector::a::lastuse [%1], %2, xl, %6, pt;\n\t"
        "@pe tcgen05.mma.cta_group::2.kind::tf32 [%1], wl, %3, %6, pt;\n\t"
        "add.s64 wh, %2, 2;\n\tadd.s64 wl, wl, 2;\n\tadd.s64 xh, %3, 64;\n\tadd.s64 xl, xl, 64;\n\t"
        "@pe tcgen05.mma.cta_group::2.kind::tf32.collector::a::fill [%1], wh, xh, %6, pt;\n\t"
        "@pe tcgen05.mma.cta_group::2.kind::tf32.collector::a::lastuse [%1], wh, xl, %6, pt;\n\t"
        "@pe tcgen05.mma.cta_group::2.kind::tf32 [%1], wl, xh, %6, pt;\n\t"
        "@pe tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%11], %12;\n\t"
        "selp.u32 %0, 1, 0, pn;\n\t}"
        : "=r"(ready)
        : "r"(d_tmem), "l"(dWh), "l"(dX), "r"(w_lo_off), "r"(x_lo_off), "r"(idesc), "r"(acc_first), "r"(next_bar),
          "r"(next_parity), "r"(0u), "r"(empty_bar), "h"((uint16_t)3)
        : "memory");
    return ready != 0;
}

template <bool CONV>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(T2_THREADS, 1)
ubp_tc2_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX, const TcArgs a,
               const int xmode, const int nrp, const int ntiles)
{
    constexpr int MAXS = T2_MAX_STAGES;
    constexpr uint32_t TMEM_COLS = 2 * T2_ACC_COLS;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    // identical layout in both CTAs: the multicast commits and the remote arrives address barriers by offset
    __shared__ __align__(8) uint64_t bar_full[MAXS], bar_go[MAXS], bar_empty[MAXS], bar_acc_full[2], bar_acc_empty[2],
        bar_last;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();
    const int N = a.ntile, NH = N / 2;                     // tile columns; columns whose X this CTA holds
    const int ngrp = NH / 32;                              // 32-column boxes per chunk in this CTA
    const uint32_t x_bytes = (uint32_t)ngrp * T2_XG;       // Xh (1x1: the raw X tile) and Xl bytes per stage
    const int x3d = CONV ? 0 : xmode;                      // 1x1: X copied by one 3-D box per chunk
    const int halo = CONV ? xmode : 0;                     // 3x3: columns copied beyond either end of the tile
    const uint32_t stage_bytes = t2_stage_bytes(ngrp, halo);
    const uint32_t raw_row = (uint32_t)(NH + 2 * halo) * 4;                   // 3x3: the copy the shifted tiles are cut from
    const int S = t2_stages(ngrp, halo);
    const int nchunk = (a.K + TC_KC - 1) / TC_KC;
    const uint32_t tx = 2 * T2_A_HALF + (CONV ? raw_row * TC_KC : x_bytes);
    const int Cin = CONV ? a.K / 9 : a.K;                  // 3x3: reduction index k = tap * Cin + channel, Cin % 16 == 0
    // this pair's tiles: pair, pair + npairs, ...; tile t = (row pair t % nrp, column tile t / nrp)
    const int npairs = (int)(gridDim.x >> 1), pair = (int)(blockIdx.x >> 1);
    const int nmy = pair < ntiles ? (ntiles - pair + npairs - 1) / npairs : 0;
    auto tile_row0 = [&](int i) { return ((pair + i * npairs) % nrp) * 256 + (int)rank * 128; };
    auto tile_col0 = [&](int i) { return (int64_t)((pair + i * npairs) / nrp) * N; };

    // one chunk's copies: Wh and Wl rows of this CTA in one 3-D box, the raw X columns in one 3-D box (or one 2-D
    // box per 32 columns when the column count is not a multiple of 32)
    auto issue_chunk = [&](int c, int st, int row0, int xcol) {
        uint8_t *stage = smem + (size_t)st * stage_bytes;
        const uint32_t bar = smem_u32(&bar_full[st]);
        mbar_expect_tx(bar, tx);
        tma_load_3d(smem_u32(stage), &tmW, c * TC_KC, row0, 0, bar);
        if (CONV) {
            // 16 channels of the chunk's tap, columns xcol - halo .. xcol + NH + halo - 1 of the flattened (b, y, x)
            // axis: every tap's shift dy * W + dx (at most W + 1 <= halo either way) lies inside
            const int ch0 = (c * TC_KC) % Cin;
            tma_load_2d(smem_u32(stage + 2 * T2_A_HALF + 2 * x_bytes), &tmX, xcol - halo, ch0, bar);
        } else if (x3d) {
            tma_load_3d(smem_u32(stage + 2 * T2_A_HALF), &tmX, 0, c * TC_KC, xcol >> 5, bar);
        } else {
            for (int g = 0; g < ngrp; ++g)
                tma_load_2d(smem_u32(stage + 2 * T2_A_HALF + g * T2_XG), &tmX, xcol + 32 * g, c * TC_KC, bar);
        }
    };

    // Launched with programmatic stream serialisation (as ubp_tc3.cu): let the next kernel become resident early, set
    // up everything that reads no global data, then wait for the earlier kernel before the first copy.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (threadIdx.x == 0) {
        prefetch_tensormap(&tmW);
        prefetch_tensormap(&tmX);
        abort_flag = 0;
        for (int s = 0; s < S; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_go[s]), 2 * (T2_XL_WARPS / T2_XL_GROUPS));   // used in the leader CTA only
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&bar_acc_full[b]), 1);
            mbar_init(smem_u32(&bar_acc_empty[b]), 2 * T2_EPI_WARPS);   // used in the leader CTA only
        }
        mbar_init(smem_u32(&bar_last), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    // cluster barrier, first half: arrive once this CTA's barriers exist; the wait follows the wait for the earlier
    // kernel, when the other CTA has normally arrived long ago
    asm volatile("barrier.cluster.arrive.release;" ::: "memory");
    if (warp == 1) {   // tensor memory of the pair: the same warp of both CTAs allocates
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");     // every thread: nothing below may overtake the earlier kernel
    // the first copy lands in this CTA's own memory and signals its own barrier: start it before the rest of the
    // set-up completes, so that the first data is on its way meanwhile
    if (threadIdx.x == 0 && nmy > 0) issue_chunk(0, 0, tile_row0(0), (int)(tile_col0(0) + (int64_t)rank * NH));
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("barrier.cluster.wait.acquire;" ::: "memory");   // both CTAs' barriers exist before anyone signals them
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_slot;

    bool ok = true;
    if (warp == 0) {
        // ---------------- TMA producer: one ring of S stages straight through all of this pair's tiles
        if (lane == 0) {
            int st = 1 % S, round = 1 / S;                 // chunk (0, 0) was started above
            for (int i = 0; i < nmy && ok; ++i) {
                const int row0 = tile_row0(i), xcol = (int)(tile_col0(i) + (int64_t)rank * NH);
                for (int c = (i == 0 ? 1 : 0); c < nchunk; ++c) {
                    if (round > 0) {                       // the stage's previous contents must have been consumed
                        ok = mbar_wait_relaxed(smem_u32(&bar_empty[st]), (uint32_t)(round - 1) & 1u, &abort_flag);
                        if (!ok) break;
                    }
                    issue_chunk(c, st, row0, xcol);
                    if (++st == S) { st = 0; ++round; }
                }
            }
        }
    } else if (warp == 1) {
        if (rank == 0) {
            // ---------------- leader: MMA issuer for the pair. The whole warp walks the loop so that descriptors and
            // barrier addresses stay warp-uniform; one elected lane issues the tcgen05 instructions.
            const uint32_t idesc = make_idesc2(N);
            const uint64_t dWh0 = make_desc(smem_u32(smem), 16, 512, SWZ_64B);
            const uint64_t dX0 = make_desc(smem_u32(smem) + 2 * T2_A_HALF, T2_LBO, T2_SBO, SWZ_128B_ATOM32);
            const uint32_t stage_u = stage_bytes >> 4;
            int st = 0;
            uint32_t ph = 0;
            // one wait per chunk: the Xl warps of the pair arrive on bar_go after their own copies (W and X) have
            // landed and their Xl tile is written
            bool ready = nmy > 0 && mbar_try_wait(smem_u32(&bar_go[0]), 0);
            for (int i = 0; i < nmy && ok; ++i) {
                const int b = i & 1;
                const uint32_t acc = tmem_base + (uint32_t)b * T2_ACC_COLS;
                if (i >= 2) {                              // the epilogue of tile i - 2 must have read this accumulator
                    ok = mbar_wait(smem_u32(&bar_acc_empty[b]), (uint32_t)((i >> 1) - 1) & 1u, &abort_flag);
                    if (!ok) break;
                }
                for (int c = 0; c < nchunk; ++c) {
                    if (!ready) ok = mbar_wait(smem_u32(&bar_go[st]), ph, &abort_flag);
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint64_t soff = (uint64_t)((uint32_t)st * stage_u);
                    int nst = st + 1;
                    uint32_t nph = ph;
                    if (nst == S) { nst = 0; nph ^= 1u; }
                    // (the commit inside hands stage st back to both CTAs once these MMAs have read it)
                    ready = mma2_chunk(acc, dWh0 + soff, dX0 + soff, T2_A_HALF >> 4, x_bytes >> 4, idesc, c > 0 ? 1u : 0u,
                                       smem_u32(&bar_go[nst]), nph, smem_u32(&bar_empty[st]));
                    st = nst; ph = nph;
                }
                if (!ok) break;
                mma2_commit_both(smem_u32(&bar_acc_full[b]));     // accumulator complete: epilogue warps of both CTAs
                if (i == nmy - 1) mma2_commit_both(smem_u32(&bar_last));
            }
        }
    } else if (warp < 2 + T2_XL_WARPS) {
        // ---------------- Xl = X - Xh, elementwise on the tile as TMA laid it out (same offsets in both tiles).
        // Two groups of four warps take turns (chunk f belongs to group f mod 2): the pass is a short dependent
        // chain (load, split, store, proxy fence, arrive), so two chunks in flight double its rate. Thread i of a
        // group takes the 16-byte pieces i, i + 128, ... of the tile.
        constexpr int GT = (T2_XL_WARPS / T2_XL_GROUPS) * 32;
        const int grp = (warp - 2) / (T2_XL_WARPS / T2_XL_GROUPS);
        const int gt = (int)threadIdx.x - 64 - grp * GT;
        const int npiece = ngrp * (int)(T2_XG / 16);
        const int total = nmy * nchunk;
        int st = grp;                                      // the stage count is even: stages grp, grp + 2, ...
        uint32_t ph = 0;
        const int cg = lane, cw = (gt >> 5);               // 3x3: column group and first channel of this thread
        unsigned long long tap_ok = 0;                     // 3x3: bit tap * 4 + e: tap inside the image for column 4 cg + e
        int mask_tile = -1;
        for (int f = grp; f < total && ok; f += T2_XL_GROUPS) {
            ok = mbar_wait_relaxed(smem_u32(&bar_full[st]), ph, &abort_flag);
            if (!ok) break;
            uint8_t *xr = smem + (size_t)st * stage_bytes + 2 * T2_A_HALF;
            if (CONV) {
                // 3x3: cut the tap's shifted, border-masked tile out of the raw copy and write Xh and Xl in the
                // operand layout. Lane cg of a warp owns columns 4 cg .. 4 cg + 3 of the CTA's part of the tile,
                // warp w of the group the channels w, w + 4, w + 8, w + 12 of the chunk.
                const int ti = f / nchunk, c = f - ti * nchunk;
                if (ti != mask_tile) {                     // new tile: which taps of my four columns are inside the image
                    mask_tile = ti;
                    const int64_t n0 = tile_col0(ti) + (int64_t)rank * NH + 4 * cg;
                    const int hw = a.H * a.W;
                    tap_ok = 0;
                    for (int e = 0; e < 4; ++e) {
                        const int64_t n = n0 + e;
                        if (cg * 4 >= NH || n >= a.Nc) continue;
                        const int pix = (int)(n % hw), y = pix / a.W, x = pix - y * a.W;
                        for (int tp = 0; tp < 9; ++tp) {
                            const int yy = y + tp / 3 - 1, xx = x + tp % 3 - 1;
                            if (yy >= 0 && yy < a.H && xx >= 0 && xx < a.W) tap_ok |= 1ull << (tp * 4 + e);
                        }
                    }
                }
                if (cg * 4 < NH) {
                    const int tp = (c * TC_KC) / Cin;
                    const int sh = (tp / 3 - 1) * a.W + (tp % 3 - 1) + halo;      // >= 0: offset into the raw rows
                    const uint32_t ok4 = (uint32_t)(tap_ok >> (tp * 4)) & 15u;
                    const uint8_t *raw = xr + 2 * x_bytes;
                    const uint32_t rpitch = raw_row;
                    const int o = 4 * cg + sh, ob = o & ~3, r = o & 3;          // r is the same for every lane
                    const uint32_t dst = (uint32_t)(cg >> 3) * T2_XG + (uint32_t)(cg & 1) * 16u;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int k = cw + 4 * i;
                        const float4 lo4 = *reinterpret_cast<const float4 *>(raw + k * rpitch + ob * 4);
                        const float4 hi4 = *reinterpret_cast<const float4 *>(raw + k * rpitch + ob * 4 + 16);
                        float4 v;
                        if (r == 0) v = lo4;
                        else if (r == 1) v = make_float4(lo4.y, lo4.z, lo4.w, hi4.x);
                        else if (r == 2) v = make_float4(lo4.z, lo4.w, hi4.x, hi4.y);
                        else v = make_float4(lo4.w, hi4.x, hi4.y, hi4.z);
                        if (!(ok4 & 1u)) v.x = 0.f;
                        if (!(ok4 & 2u)) v.y = 0.f;
                        if (!(ok4 & 4u)) v.z = 0.f;
                        if (!(ok4 & 8u)) v.w = 0.f;
                        float4 h, l;
                        h.x = __uint_as_float(__float_as_uint(v.x) & 0xffffe000u); l.x = v.x - h.x;
                        h.y = __uint_as_float(__float_as_uint(v.y) & 0xffffe000u); l.y = v.y - h.y;
                        h.z = __uint_as_float(__float_as_uint(v.z) & 0xffffe000u); l.z = v.z - h.z;
                        h.w = __uint_as_float(__float_as_uint(v.w) & 0xffffe000u); l.w = v.w - h.w;
                        // row k of the 32-column box: 128 bytes whose 32-byte atoms are XOR-swizzled with k mod 4
                        const uint32_t off = dst + (uint32_t)k * 128u + ((((uint32_t)(cg & 7) >> 1) ^ ((uint32_t)k & 3u)) << 5);
                        *reinterpret_cast<float4 *>(xr + off) = h;
                        *reinterpret_cast<float4 *>(xr + x_bytes + off) = l;
                    }
                }
            } else
            for (int i = gt; i < npiece; i += GT) {
                const float4 v = *reinterpret_cast<const float4 *>(xr + i * 16);
                float4 lo;
                lo.x = v.x - __uint_as_float(__float_as_uint(v.x) & 0xffffe000u);
                lo.y = v.y - __uint_as_float(__float_as_uint(v.y) & 0xffffe000u);
                lo.z = v.z - __uint_as_float(__float_as_uint(v.z) & 0xffffe000u);
                lo.w = v.w - __uint_as_float(__float_as_uint(v.w) & 0xffffe000u);
                *reinterpret_cast<float4 *>(xr + x_bytes + i * 16) = lo;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // make the writes visible to the MMA unit
            __syncwarp();
            if (lane == 0) {
                if (rank == 0) mbar_arrive(smem_u32(&bar_go[st]));
                else mbar_arrive_remote(smem_u32(&bar_go[st]), 0);
            }
            st += T2_XL_GROUPS;
            if (st >= S) { st -= S; ph ^= 1u; }
        }
        // ---------------- the last tile has nothing to overlap with: take the 16-column units 2, 3, 6, 7, ... of its epilogue.
        // Its own barrier (one phase) rather than the accumulator's, whose earlier phases these warps did not see.
        if (ok && nmy > 0) ok = mbar_wait_relaxed(smem_u32(&bar_last), 0, &abort_flag);
        if (ok && nmy > 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int i = nmy - 1;
            epilogue_blocks(a, tmem_base + (uint32_t)(i & 1) * T2_ACC_COLS, warp & 3, 2 + ((warp - 2) >> 2), 4, N,
                            tile_row0(i), tile_col0(i), lane, 0u, rank);
        }
    } else {
        // ---------------- epilogue warps: tile i's accumulator while the main loop works on tile i + 1
        const int part = (warp - 2 - T2_XL_WARPS) >> 2;       // two warps share a lane quarter and split the columns
        for (int i = 0; i < nmy && ok; ++i) {
            const int b = i & 1;
            ok = mbar_wait_relaxed(smem_u32(&bar_acc_full[b]), (uint32_t)(i >> 1) & 1u, &abort_flag);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const bool last = i == nmy - 1;
            epilogue_blocks(a, tmem_base + (uint32_t)b * T2_ACC_COLS, warp & 3, part, last ? 4 : 2, N, tile_row0(i),
                            tile_col0(i), lane, last ? 0u : smem_u32(&bar_acc_empty[b]), rank);
        }
    }
    if (!ok && lane == 0) atomicExch(a.status, 1);
    // every thread of both CTAs comes here: neither CTA may free tensor memory or leave while the other could
    // still be the target of the pair's MMAs or commits
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    cluster_sync();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

}  // namespace

// Launch the pair kernel on tiles of 256 rows x `ntile` columns (a multiple of 64): one persistent CTA pair per SM
// pair, or fewer if there are fewer tiles.
// tmW: 3-D map over the plan's dense part (channel, row, {Wh, Wl}), box 16 x 128 x 2, 64-byte swizzle.
// 1x1 (halo == 0): tmX in the 128-byte swizzle with 32-byte atoms; x3d != 0: 3-D map (column in group, channel,
// 32-column group) with box 32 x 16 x ntile/64; x3d == 0: 2-D map (column, channel) with box 32 x 16.
// 3x3 (halo = image width + 1 rounded up to a multiple of 4): tmX is a plain 2-D map (flattened (b, y, x) column,
// channel) with box (ntile/2 + 2 halo) x 16.
int launch_tc_pair(const CUtensorMap_st *tmW, const CUtensorMap_st *tmX, int x3d, int halo, const void *args_, int M,
                   int64_t Nc, int ntile, int sms, void *stream)
{
    TcArgs a = *static_cast<const TcArgs *>(args_);
    a.ntile = ntile;
    const int ngrp = ntile / 64;
    size_t smem = (size_t)t2_stages(ngrp, halo) * t2_stage_bytes(ngrp, halo) + 1024;
    if (smem < TC_PAIR_MIN_SMEM) smem = TC_PAIR_MIN_SMEM;   // one CTA per SM, whatever the tile width (see the constant)
    static bool done[2][64] = {};
    int devid = 0;
    if (cudaGetDevice(&devid) != cudaSuccess) devid = -1;
    const int which = halo ? 1 : 0;
    if (devid < 0 || devid >= 64 || !done[which][devid]) {
        cudaError_t e = halo ? cudaFuncSetAttribute(ubp_tc2_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                    (int)(T2_PIPE_BUDGET + 1024))
                             : cudaFuncSetAttribute(ubp_tc2_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                    (int)(T2_PIPE_BUDGET + 1024));
        if (e != cudaSuccess) { set_last_cuda_error((int)e); return UBP_E_CUDA; }
        // the smallest launch this function ever makes must already fill an SM (a query, nothing is launched)
        int per_sm = 0;
        e = halo ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, ubp_tc2_kernel<true>, T2_THREADS, TC_PAIR_MIN_SMEM)
                 : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, ubp_tc2_kernel<false>, T2_THREADS, TC_PAIR_MIN_SMEM);
        if (e != cudaSuccess) { set_last_cuda_error((int)e); return UBP_E_CUDA; }
        if (per_sm != 1) return UBP_E_UNSUPPORTED;
        if (devid >= 0 && devid < 64) done[which][devid] = true;
    }
    const int nrp = (M + 255) / 256;
    const long long ntiles = (long long)nrp * ((Nc + ntile - 1) / ntile);
    if (ntiles <= 0) return UBP_OK;
    if (ntiles > 0x7fffffffll) return UBP_E_UNSUPPORTED;
    const long long pairs = ntiles < sms / 2 ? ntiles : sms / 2;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * pairs));
    cfg.blockDim = dim3(T2_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = halo ? cudaLaunchKernelEx(&cfg, ubp_tc2_kernel<true>, *tmW, *tmX, a, halo, nrp, (int)ntiles)
                         : cudaLaunchKernelEx(&cfg, ubp_tc2_kernel<false>, *tmW, *tmX, a, x3d, nrp, (int)ntiles);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) { set_last_cuda_error((int)e); return UBP_E_CUDA; }
    return UBP_OK;
}

// how many pipeline stages the pair kernel gets for a tile width and halo (0 = too few to run)
int tc_pair_stages(int ntile, int halo) { return t2_stages(ntile / 64, halo); }

}  // namespace ubp
