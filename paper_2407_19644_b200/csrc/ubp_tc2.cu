// Two-CTA form of the tensor-core kernel for the 1x1 product (see ubp_tc.cu for the arithmetic: densified panels,
// three TF32 products per fp32 product, fp32 accumulation in tensor memory).
//
// A cluster of two CTAs (two SMs) computes one tile of 256 output rows x N columns with
// tcgen05.mma.cta_group::2: every MMA has M = 256, CTA r supplies rows 128r..128r+127 of W from its own shared
// memory and columns r*N/2 .. r*N/2 + N/2 - 1 of X from its own shared memory, and keeps its 128 rows x N columns of
// the accumulator in its own tensor memory. Per SM that halves the X operand reads of the one-CTA kernel, which is
// what bounds that kernel on shared-memory bandwidth.
//
// X is not transposed at all here. The activations lie in memory as [channel][column] with columns contiguous, which
// is the "MN-major" form of the B operand; for 32-bit elements the tensor core reads that form from shared memory in
// the 128-byte swizzle with 32-byte atoms, which is also a TMA swizzle mode. So TMA copies [16 channels] x [32
// columns] boxes of X straight into the operand layout, and the MMA consumes the raw fp32 words: the tensor core
// drops the low 13 mantissa bits itself, i.e. it multiplies by Xh. The only work left for the SM's threads is the
// low part Xl = X - Xh, an elementwise pass from the raw tile to a second tile in the same layout.
//
// Per CTA: warp 0 = TMA producer (its Wh / Wl rows and its X columns, one 3-D box each per chunk); warps 2..17 = two
// groups of eight warps that take turns (chunk c belongs to group c mod 2) computing Xl, and later the epilogue of the CTA's 128 rows; warp 1 =
// in the leader CTA (cluster rank 0) one thread issues all MMAs for the pair and commits stages back to BOTH CTAs
// (tcgen05.commit with a cluster multicast mask); in the peer CTA one thread relays "my copies have landed" and "my
// Xl is written" to barriers in the leader's shared memory (mbarrier.arrive on a mapa-translated address).
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

constexpr int T2_SPLIT_WARPS = 16;                        // warps 2..17
constexpr int T2_GROUPS = 2;                              // groups of eight warps taking turns on the chunks
constexpr int T2_THREADS = (2 + T2_SPLIT_WARPS) * 32;
constexpr int T2_MAX_STAGES = 8;                          // pipeline stages: as many as fit, at most this
constexpr uint32_t T2_A_HALF = 128 * TC_KC * 4;           // Wh or Wl chunk of this CTA's 128 rows: 8 KB
constexpr uint32_t T2_XG = 32 * TC_KC * 4;                // one box of X: 16 channels x 32 columns, 2 KB
constexpr uint32_t T2_SMEM_BUDGET = 196 * 1024;           // pipeline stages together
// a stage = Wh + Wl chunk (16 KB) + raw X + Xl of `ngrp` 32-column boxes (2 KB each): 20 .. 32 KB, 8 or 6 stages.
// The count is a multiple of T2_GROUPS so that a stage always belongs to the same group of Xl warps: a waiter must
// see every phase of a barrier it waits on (a parity wait cannot tell phase k from phase k + 2).
__host__ __device__ constexpr int t2_stages(int ngrp)
{
    const int s = (int)(T2_SMEM_BUDGET / (2 * T2_A_HALF + 2 * (uint32_t)ngrp * T2_XG));
    return (s > T2_MAX_STAGES ? T2_MAX_STAGES : s) / T2_GROUPS * T2_GROUPS;
}
constexpr uint32_t SWZ_128B_ATOM32 = 1;                   // descriptor layout type: 128-byte swizzle, 32-byte atoms
constexpr uint32_t T2_LBO = T2_XG;                        // next 32 columns
constexpr uint32_t T2_SBO = 4 * 128;                      // next 4 channels
constexpr int T2_PITCH = 36;                              // floats per row of an epilogue staging tile

__device__ __forceinline__ uint32_t cluster_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// arrive on the barrier at the same shared-memory offset in CTA `rank` of the cluster. What the arrival stands for
// (TMA writes, or generic writes already followed by a proxy fence) sits in the sender's own shared memory and is
// read there by its own tensor core, so no cluster-scope release is needed; with one the arrive cost ~700 cycles.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t local_bar, uint32_t rank)
{
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_bar), "r"(rank));
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(remote) : "memory");
}
// instruction descriptor: D = f32, A = B = tf32, A K-major, B MN-major, M = 256 (two CTAs), N = n
__device__ __forceinline__ uint32_t make_idesc2(int n)
{
    return (1u << 4) | (2u << 7) | (2u << 10) | (1u << 16) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}
// completion of all MMAs issued so far arrives on the barrier at this offset in both CTAs of the pair
__device__ __forceinline__ void mma2_commit_both(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((uint16_t)3) : "memory");
}


// One chunk's six MMAs (two 8-channel steps x {Wh Xh, Wl Xh, Wh Xl}) in a single statement, with the barrier
// test for the NEXT chunk issued first and its result read last, so that the test's latency is hidden behind the
// MMA issue. Descriptor offsets are in 16-byte units: the next 8 channels of W are 32 bytes on (+2), of X eight
// 128-byte rows on (+64). Returns whether the next chunk's barrier phase has completed.
__device__ __forceinline__ bool mma2_chunk(uint32_t d_tmem, uint64_t dWh, uint64_t dX, uint32_t w_lo_off,
                                           uint32_t x_lo_off, uint32_t idesc, uint32_t acc_first, uint32_t next_bar,
                                           uint32_t next_parity)
{
    uint32_t ready;
    asm volatile(
        "{\n\t.reg .pred pn, pa, pt;\n\t.reg .b64 wh, wl, xh, xl;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 pn, [%8], %9;\n\t"
        "setp.ne.b32 pa, %7, 0;\n\t"
        "setp.eq.b32 pt, %10, 0;\n\t"
        "cvt.u64.u32 wl, %4;\n\tadd.s64 wl, wl, %2;\n\t"
        "cvt.u64.u32 xl, %5;\n\tadd.s64 xl, xl, %3;\n\t"
        "tcgen05.mma.cta_group::2.kind::tf32 [%1], %2, %3, %6, pa;\n\t"
        "tcgen05.mma.cta_group::2.kind::tf32 [%1], wl, %3, %6, pt;\n\t"
        "tcgen05.mma.cta_group::2.kind::tf32 [%1], %2, xl, %6, pt;\n\t"
        "add.s64 wh, %2, 2;\n\tadd.s64 wl, wl, 2;\n\tadd.s64 xh, %3, 64;\n\tadd.s64 xl, xl, 64;\n\t"
        "tcgen05.mma.cta_group::2.kind::tf32 [%1], wh, xh, %6, pt;\n\t"
        "tcgen05.mma.cta_group::2.kind::tf32 [%1], wl, xh, %6, pt;\n\t"
        "tcgen05.mma.cta_group::2.kind::tf32 [%1], wh, xl, %6, pt;\n\t"
        "selp.u32 %0, 1, 0, pn;\n\t}"
        : "=r"(ready)
        : "r"(d_tmem), "l"(dWh), "l"(dX), "r"(w_lo_off), "r"(x_lo_off), "r"(idesc), "r"(acc_first), "r"(next_bar),
          "r"(next_parity), "r"(0u)
        : "memory");
    return ready != 0;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(T2_THREADS, 1)
ubp_tc2_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX, const TcArgs a,
               const int x3d)
{
    constexpr int MAXS = T2_MAX_STAGES;
    constexpr uint32_t TMEM_COLS = 256;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    // identical layout in both CTAs: the multicast commit and the remote arrives address barriers by offset
    __shared__ __align__(8) uint64_t bar_full[MAXS], bar_go[MAXS], bar_empty[MAXS], bar_acc;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();
    const int N = a.ntile, NH = N / 2;                     // tile columns; columns whose X this CTA holds
    const int ngrp = NH / 32;                              // 32-column boxes per chunk in this CTA
    const uint32_t x_bytes = (uint32_t)ngrp * T2_XG;       // raw X (and Xl) bytes per stage
    const uint32_t stage_bytes = 2 * T2_A_HALF + 2 * x_bytes;
    const int S = t2_stages(ngrp);
    const int row0 = (int)(blockIdx.x >> 1) * 256 + (int)rank * 128;      // this CTA's 128 output rows
    const int64_t col0 = (int64_t)blockIdx.y * N;
    const int xcol = (int)(col0 + (int64_t)rank * NH);     // first X column this CTA holds
    const int nchunk = (a.K + TC_KC - 1) / TC_KC;
    const uint32_t tx = 2 * T2_A_HALF + x_bytes;

    // one chunk's copies: Wh and Wl rows of this CTA in one 3-D box, the raw X columns in one 3-D box (or one 2-D
    // box per 32 columns when the column count is not a multiple of 32)
    auto issue_chunk = [&](int c, int st) {
        uint8_t *stage = smem + (size_t)st * stage_bytes;
        const uint32_t bar = smem_u32(&bar_full[st]);
        mbar_expect_tx(bar, tx);
        tma_load_3d(smem_u32(stage), &tmW, c * TC_KC, row0, 0, bar);
        if (x3d) {
            tma_load_3d(smem_u32(stage + 2 * T2_A_HALF), &tmX, 0, c * TC_KC, xcol >> 5, bar);
        } else {
            for (int g = 0; g < ngrp; ++g)
                tma_load_2d(smem_u32(stage + 2 * T2_A_HALF + g * T2_XG), &tmX, xcol + 32 * g, c * TC_KC, bar);
        }
    };

    constexpr int EARLY = 1;      // chunks whose copies start before the CTA-wide and cluster-wide barriers
    if (threadIdx.x == 0) {
        prefetch_tensormap(&tmW);
        prefetch_tensormap(&tmX);
        abort_flag = 0;
        for (int s = 0; s < S; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_go[s]), 2 * (T2_SPLIT_WARPS / T2_GROUPS));   // used in the leader CTA only
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        mbar_init(smem_u32(&bar_acc), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        // the first copies land in this CTA's own memory and signal its own barriers: start them before the
        // tensor-memory allocation and the cluster barrier, so that the first data is on its way meanwhile
        for (int c = 0; c < EARLY && c < nchunk; ++c) issue_chunk(c, c);
    }
    if (warp == 1) {   // tensor memory of the pair: the same warp of both CTAs allocates
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    cluster_sync();                                        // both CTAs' barriers exist before anyone signals them
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_slot;

    bool ok = true;
    if (warp == 0) {
        // ---------------- TMA producer (the first EARLY chunks were started above)
        if (lane == 0) {
            for (int c = EARLY; c < S && c < nchunk; ++c) issue_chunk(c, c);
            int st = 0;
            uint32_t ph = 0;
            for (int c = S; c < nchunk && ok; ++c) {
                ok = mbar_wait_relaxed(smem_u32(&bar_empty[st]), ph, &abort_flag);
                if (!ok) break;
                issue_chunk(c, st);
                if (++st == S) { st = 0; ph ^= 1u; }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            // ---------------- leader: MMA issuer for the pair
            const uint32_t idesc = make_idesc2(N);
            const uint64_t dWh0 = make_desc(smem_u32(smem), 16, 512, SWZ_64B);
            const uint64_t dX0 = make_desc(smem_u32(smem) + 2 * T2_A_HALF, T2_LBO, T2_SBO, SWZ_128B_ATOM32);
            const uint32_t stage_u = stage_bytes >> 4;
            int st = 0;
            uint32_t ph = 0;
            // one wait per chunk: the eight Xl warps of the pair arrive on bar_go after their own copies (W and X)
            // have landed and their Xl tile is written
            bool ready = mbar_try_wait(smem_u32(&bar_go[0]), 0);
            for (int c = 0; c < nchunk && ok; ++c) {
                if (!ready) ok = mbar_wait(smem_u32(&bar_go[st]), ph, &abort_flag);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint64_t soff = (uint64_t)((uint32_t)st * stage_u);
                int nst = st + 1;
                uint32_t nph = ph;
                if (nst == S) { nst = 0; nph ^= 1u; }
                ready = mma2_chunk(tmem_base, dWh0 + soff, dX0 + soff, T2_A_HALF >> 4, x_bytes >> 4, idesc, c > 0 ? 1u : 0u,
                                   smem_u32(&bar_go[nst]), nph);
                mma2_commit_both(smem_u32(&bar_empty[st]));   // both CTAs may refill this stage afterwards
                if (c + 1 >= nchunk) ready = true;
                st = nst; ph = nph;
            }
            if (ok) mma2_commit_both(smem_u32(&bar_acc));
        }
    } else {
        // ---------------- Xl = X - Xh, elementwise on the tile as TMA laid it out (same offsets in both tiles);
        // group `grp` of eight warps owns chunks grp, grp + 2, ... (and with them stages grp, grp + 2, ...: the stage
        // count is even); thread i of the group takes the 16-byte pieces i, i + 256, ... of the tile
        constexpr int GT = (T2_SPLIT_WARPS / T2_GROUPS) * 32;      // threads per group
        const int grp = (warp - 2) / (T2_SPLIT_WARPS / T2_GROUPS);
        const int gt = (int)(threadIdx.x - 64) - grp * GT;
        const int npiece = ngrp * (int)(T2_XG / 16);
        int st = grp;
        uint32_t ph = 0;
        for (int c = grp; c < nchunk && ok; c += T2_GROUPS) {
            ok = mbar_wait_relaxed(smem_u32(&bar_full[st]), ph, &abort_flag);
            if (!ok) break;
            uint8_t *xr = smem + (size_t)st * stage_bytes + 2 * T2_A_HALF;
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
            st += T2_GROUPS;
            if (st >= S) { st -= S; ph ^= 1u; }
        }
        // ---------------- epilogue of this CTA's 128 rows x N columns
        if (ok) ok = mbar_wait_relaxed(smem_u32(&bar_acc), 0, &abort_flag);
        if (ok) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int q = warp & 3;                           // tensor-memory lanes 32q .. 32q+31
            const int part = (warp - 2) >> 2;                 // four warps share a lane quarter and split the columns
            // registers -> shared memory (row per lane, 144-byte pitch) -> registers with 8 lanes per row, so that
            // every store instruction writes four complete 128-byte row segments; all MMAs of the pair are done
            // (bar_acc), so the pipeline stages are free to be reused
            float *tile_s = reinterpret_cast<float *>(smem) + (warp - 2) * 32 * T2_PITCH;
            const int sub_row = lane >> 3, sub_col = (lane & 7) * 4;
            const int rbase = row0 + q * 32;
#pragma unroll 1
            for (int cc = part; cc < N / 32; cc += T2_SPLIT_WARPS / 4) {
                uint32_t r[32];
                tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(cc * 32), r);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                for (int v = 0; v < 8; ++v)
                    *reinterpret_cast<float4 *>(tile_s + lane * T2_PITCH + 4 * v) =
                        make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]),
                                    __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3]));
                __syncwarp();
                const int64_t col = col0 + cc * 32 + sub_col;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int rr = i * 4 + sub_row;
                    const int row = rbase + rr;
                    float4 o = *reinterpret_cast<const float4 *>(tile_s + rr * T2_PITCH + sub_col);
                    if (row < a.M) {
                        const float b = a.bias ? __ldg(a.bias + row) : 0.f;
                        o.x += b; o.y += b; o.z += b; o.w += b;
                        if (a.relu) { o.x = fmaxf(o.x, 0.f); o.y = fmaxf(o.y, 0.f); o.z = fmaxf(o.z, 0.f); o.w = fmaxf(o.w, 0.f); }
                        float *yrow = a.Y + (size_t)row * a.ldy;
                        if (col + 3 < a.Nc && (a.ldy & 3) == 0) {
                            *reinterpret_cast<float4 *>(yrow + col) = o;
                        } else {
                            if (col < a.Nc) yrow[col] = o.x;
                            if (col + 1 < a.Nc) yrow[col + 1] = o.y;
                            if (col + 2 < a.Nc) yrow[col + 2] = o.z;
                            if (col + 3 < a.Nc) yrow[col + 3] = o.w;
                        }
                    }
                }
                __syncwarp();
            }
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


// Launch the pair kernel: grid.x = 2 x (256-row tiles), grid.y = column tiles of `ntile` columns (a multiple of 64).
// tmW: 3-D map over the plan's dense part (channel, row, {Wh, Wl}), box 16 x 128 x 2, 64-byte swizzle.
// tmX: 128-byte swizzle with 32-byte atoms; x3d != 0: 3-D map (column in group, channel, 32-column group) with box
// 32 x 16 x ntile/64; x3d == 0: 2-D map (column, channel) with box 32 x 16.
int launch_tc_pair(const CUtensorMap_st *tmW, const CUtensorMap_st *tmX, int x3d, const void *args_, int M, int64_t Nc,
                   int ntile, void *stream)
{
    TcArgs a = *static_cast<const TcArgs *>(args_);
    a.ntile = ntile;
    const int ngrp = ntile / 64;
    const size_t smem = (size_t)t2_stages(ngrp) * (2 * T2_A_HALF + 2 * (size_t)ngrp * T2_XG) + 1024;
    static bool done[64] = {};
    int devid = 0;
    if (cudaGetDevice(&devid) != cudaSuccess) devid = -1;
    if (devid < 0 || devid >= 64 || !done[devid]) {
        cudaError_t e = cudaFuncSetAttribute(ubp_tc2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)(T2_SMEM_BUDGET + 1024));
        if (e != cudaSuccess) { set_last_cuda_error((int)e); return UBP_E_CUDA; }
        if (devid >= 0 && devid < 64) done[devid] = true;
    }
    dim3 grid((unsigned)(2 * ((M + 255) / 256)), (unsigned)((Nc + ntile - 1) / ntile));
    ubp_tc2_kernel<<<grid, T2_THREADS, smem, static_cast<cudaStream_t>(stream)>>>(*tmW, *tmX, a, x3d);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_last_cuda_error((int)e); return UBP_E_CUDA; }
    return UBP_OK;
}

}  // namespace ubp
