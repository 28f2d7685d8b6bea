// Device helpers shared by the tensor-core kernels (one-CTA and two-CTA variants): mbarrier / TMA / tcgen05
// wrappers, descriptor encoders and the kernel argument block.
#ifndef UBP_TC_COMMON_CUH_
#define UBP_TC_COMMON_CUH_

#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>

namespace ubp {
namespace tc {

constexpr int TC_KC = 16;          // channels per pipeline stage
constexpr uint32_t SWZ_NONE = 0, SWZ_64B = 4;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
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
__device__ __forceinline__ uint64_t global_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// bounded wait (one second unless the caller gives another limit); false if it ran out or another thread of the
// CTA already gave up
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                          uint64_t limit_ns = 1000000000ull)
{
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_ns();
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 0u) {
            if (*abort_flag) return false;
            if (global_ns() - t0 > limit_ns) break;
        }
    }
    *abort_flag = 1;
    return false;
}
// same, for waiters that are not on the critical path: sleep between polls so they do not take issue slots
// from the thread that feeds the tensor core
__device__ __forceinline__ bool mbar_wait_relaxed(uint32_t bar, uint32_t parity, volatile int *abort_flag)
{
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_ns();
    for (uint32_t it = 1;; ++it) {
        __nanosleep(40);
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 0u) {
            if (*abort_flag) return false;
            if (global_ns() - t0 > 1000000000ull) break;
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

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *tm, int c0, int c1, int c2, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(c2), "r"(bar) : "memory");
}
// one contiguous copy global -> shared memory (both 16-byte aligned, size a multiple of 16), completing on a barrier
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap *tm)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(tm) : "memory");
}

// shared-memory matrix descriptor (tcgen05): start address, leading / stride byte offsets (all >> 4),
// descriptor version 1, swizzle mode in the top three bits
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t swizzle)
{
    return (uint64_t)((saddr >> 4) & 0x3fffu) | ((uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32) | (1ull << 46) | ((uint64_t)swizzle << 61);
}

// instruction descriptor: D = f32, A = B = tf32, both K-major, M = 128, N given at run time (multiple of 16)
__device__ __forceinline__ uint32_t make_idesc(int n)
{
    return (1u << 4) | (2u << 7) | (2u << 10) | (0u << 15) | (0u << 16) | ((uint32_t)(n >> 3) << 17) |
           ((uint32_t)(128 >> 4) << 24);
}

__device__ __forceinline__ void mma_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t kIdesc,
                                         uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(kIdesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}

// The CTA-pair kernels allocate all 512 tensor-memory columns of their SM and then meet the other CTA of the pair at
// a cluster barrier. Two such CTAs resident on one SM could therefore block each other for good (each pair holding
// one SM's tensor memory and waiting for the other's). The launchers rule that out by never asking for less dynamic
// shared memory than this: more than half of what an SM has (228 KB), so a second CTA of any of these kernels never
// fits beside the first.
constexpr size_t TC_PAIR_MIN_SMEM = 118 * 1024;

// ---------------------------------------------------------------- the checked build (-DUBP_DEBUG)
// Every index that a kernel takes from the plan or computes for shared or global memory is compared with the extent it
// has to stay in before it is used. A failing check sets the plan's status word (2: shared memory or plan contents,
// 3: global memory; the first failure wins) and the access is skipped: nothing traps, the kernel runs to its end and
// ubp_plan_check reports UBP_E_DEVICE. The ordinary build compiles the checks away.
#ifdef UBP_DEBUG
__device__ __forceinline__ bool dbg_check(bool ok, int *status, int code)
{
    if (!ok && status) atomicCAS(status, 0, code);
    return ok;
}
__device__ __forceinline__ uint32_t dbg_dynamic_smem()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%dynamic_smem_size;" : "=r"(r));
    return r;
}
#define UBP_CHK_SMEM(ok, status) (::ubp::tc::dbg_check((ok), (status), 2))
#define UBP_CHK_GMEM(ok, status) (::ubp::tc::dbg_check((ok), (status), 3))
#else
#define UBP_CHK_SMEM(ok, status) (true)
#define UBP_CHK_GMEM(ok, status) (true)
#endif

struct TcArgs {
    const float *X;          // 1x1: [K][ldx]; 3x3: input tensor, element (b, c, y, x) at b*isb + c*isc + y*W + x
    int64_t ldx;
    int conv;                // 0 = 1x1 product, 1 = 3x3 / stride 1 / pad 1 implicit GEMM (k = tap * C + channel)
    int H, W;                // 3x3 only: input plane size; output column n = b*Ho*Wo + yo*Wo + xo
    int stride;              // 3x3 only: 1, or > 1 (one-CTA kernel only): output pixel (yo, xo) is centred on input
                             // pixel (yo*stride, xo*stride), Ho = (H-1)/stride + 1, Wo = (W-1)/stride + 1
    int64_t isb, isc;        // 3x3 only: input batch / channel strides (elements)
    const float *bias;
    float *Y;
    int64_t ldy;
    int64_t Nc;
    int M, K;
    int ntile;               // columns per CTA: multiple of 32, <= 256
    int relu;
    int *status;             // plan status word
    int rpc;                 // CTA-pair kernels: output rows per CTA: 128 (0 means 128)
    int dup;                 // bf16 CTA-pair kernel, layers of at most 128 rows: both CTAs of a pair multiply the SAME
                             // 128-row weight tile (the pair's MMA needs 256 rows; the second half repeats the first) and
                             // each stores the whole rows of its own half of the tile's columns
    int mt;                  // bf16 CTA-pair kernel: 256-row MMA tiles a pair stacks on ONE staged activation tile
                             // (1, or 2 = tiles of 512 rows, one per pair); 0 means 1
    int s2;                  // bf16 CTA-pair kernel, 1x1 with stride 2: output row length Wo (0 = ordinary product). The
                             // tensor map then shows the input as (2 W floats of a row pair, row pair, channel) and a
                             // box brings the EVEN rows of whole output rows: per channel, output column j of the tile
                             // is float 2 j of the copy (W = 2 Wo); a CTA's columns are whole output rows
};


// ---------------------------------------------------------------- helpers of the CTA-pair kernels
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
// (TMA writes, generic writes already followed by a proxy fence, completed tensor-memory reads) sits in the
// sender's own SM and is consumed there by its own tensor core, so no cluster-scope release is needed; with one
// the arrive cost ~700 cycles.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t local_bar, uint32_t rank)
{
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_bar), "r"(rank));
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(remote) : "memory");
}
// completion of all MMAs issued so far arrives on the barrier at this offset in both CTAs of the pair (called by
// a whole converged warp; one elected lane issues it)
__device__ __forceinline__ void mma2_commit_both(uint32_t bar)
{
    asm volatile(
        "{\n\t.reg .pred pe;\n\telect.sync _|pe, 0xffffffff;\n\t"
        "@pe tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;\n\t}"
        ::"r"(bar), "h"((uint16_t)3) : "memory");
}

__device__ __forceinline__ void tmem_ld_16x256b_x2(uint32_t taddr, uint32_t (&r)[8])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.16x256b.x2.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
        : "r"(taddr) : "memory");
}

// Epilogue of 32 rows (tensor-memory lane quarter q of accumulator `acc`) x the 16-column units first, first + step,
// ... of one CTA's 128 x N part of a tile, without shared memory (the MMA operands and the copies already use all
// of its bandwidth). The accumulator is read in the 16 x 256-bit shape: lane t gets, per group j of 8 columns,
// the column pair 8j + 2(t mod 4) of rows t/4 and t/4 + 8 of a 16-row half. Neighbouring lanes exchange one pair
// each, after which a lane holds 16 consecutive bytes of a row and the four lanes of a row its 64 bytes of the unit:
// every 16-byte store instruction of the warp writes two whole sectors in each of eight rows; bias and ReLU are
// applied in registers. (Units of 16 columns rather than 32 so that the warps sharing a
// lane quarter get equal shares of tile widths such as 192 or 224.)
// `done_bar` != 0: once this warp's last tensor-memory read has completed, lane 0 arrives on that barrier of the
// leader CTA (the accumulator may be overwritten from then on).
// (checked build) last column a tile that starts at col0 may touch
__device__ __forceinline__ int64_t tile_cols_end(int64_t col0, int N) { return col0 + N - 1; }

__device__ __forceinline__ void epilogue_blocks(const TcArgs &a, uint32_t acc, int q, int first, int step, int N,
                                                int row0, int64_t col0, int lane, uint32_t done_bar, uint32_t rank)
{
    // this CTA's units of the tile: all of them, or -- layers of at most 128 rows, where both CTAs of the pair hold
    // the whole product (TcArgs::dup) -- the half of the columns that belongs to its rank
    const int nall = N / 16;
    const int u0 = a.dup ? (int)rank * (nall / 2) : 0, u1 = a.dup ? u0 + nall / 2 : nall;
    // matrix row of this lane's four accumulator rows (tensor-memory lanes 32 q + t/4 + {0, 8, 16, 24}), -1 beyond the matrix
    int rows[4];
    float bias[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = row0 + q * 32 + (lane >> 2) + 8 * i;
        rows[i] = r < a.M ? r : -1;
        bias[i] = (a.bias && rows[i] >= 0) ? __ldg(a.bias + rows[i]) : 0.f;
    }
#pragma unroll 1
    for (int cc = u0 + first; cc < u1; cc += step) {
        uint32_t r[2][8];
        tmem_ld_16x256b_x2(acc + ((uint32_t)(q * 32) << 16) + (uint32_t)(cc * 16), r[0]);
        tmem_ld_16x256b_x2(acc + ((uint32_t)(q * 32 + 16) << 16) + (uint32_t)(cc * 16), r[1]);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        if (done_bar && cc + step >= u1) {
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            if (lane == 0) {
                if (rank == 0) mbar_arrive(done_bar);
                else mbar_arrive_remote(done_bar, 0);
            }
        }
        // Lanes 2i and 2i + 1 swap a column pair, so that every lane holds four consecutive columns of each of its rows
        // (even lanes: columns 4i .. 4i + 3 of the unit, odd lanes: 8 + 4i ..) and the warp's 16-byte stores write the
        // unit's 64 bytes of a row as two whole sectors.
        const bool odd = (lane & 1) != 0;
        const int64_t cb = col0 + cc * 16 + (odd ? 8 + 2 * ((lane & 3) - 1) : 2 * (lane & 3));
#pragma unroll
        for (int half = 0; half < 2; ++half)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const uint32_t p0x = r[half][2 * h], p0y = r[half][2 * h + 1];           // columns 2 (t mod 4) + {0, 1}
                const uint32_t p1x = r[half][4 + 2 * h], p1y = r[half][4 + 2 * h + 1];   // columns 8 + 2 (t mod 4) + {0, 1}
                const uint32_t gx = __shfl_xor_sync(0xffffffffu, odd ? p0x : p1x, 1);
                const uint32_t gy = __shfl_xor_sync(0xffffffffu, odd ? p0y : p1y, 1);
                const int row = rows[2 * half + h];
                if (row < 0) continue;
                float *yrow = a.Y + (size_t)row * a.ldy;
                const float b = bias[2 * half + h];
                float4 o = odd ? make_float4(__uint_as_float(gx), __uint_as_float(gy), __uint_as_float(p1x), __uint_as_float(p1y))
                               : make_float4(__uint_as_float(p0x), __uint_as_float(p0y), __uint_as_float(gx), __uint_as_float(gy));
                o.x += b; o.y += b; o.z += b; o.w += b;
                if (a.relu) { o.x = fmaxf(o.x, 0.f); o.y = fmaxf(o.y, 0.f); o.z = fmaxf(o.z, 0.f); o.w = fmaxf(o.w, 0.f); }
                if (!UBP_CHK_GMEM(cb >= 0 && row < a.M && (tile_cols_end(col0, N) >= cb + 3), a.status)) continue;
                if (cb + 3 < a.Nc) *reinterpret_cast<float4 *>(yrow + cb) = o;
                else {
                    if (cb < a.Nc) yrow[cb] = o.x;
                    if (cb + 1 < a.Nc) yrow[cb + 1] = o.y;
                    if (cb + 2 < a.Nc) yrow[cb + 2] = o.z;
                }
            }
    }
    // a warp with no unit of its own still owes its arrival
    if (done_bar && u0 + first >= u1) {
        if (lane == 0) {
            if (rank == 0) mbar_arrive(done_bar);
            else mbar_arrive_remote(done_bar, 0);
        }
    }
}

}  // namespace tc
}  // namespace ubp
#endif
