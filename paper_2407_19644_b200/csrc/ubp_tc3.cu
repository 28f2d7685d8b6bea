// CTA-pair tensor-core kernel with bf16 products (1x1 and 3x3): the persistent pipeline of ubp_tc2.cu with every
// fp32 product w * x replaced by three bf16 products instead of three TF32 products,
//     w = w1 + w2 + (..),  x = x1 + x2 + (..)    (w1 = bf16(w), w2 = bf16(w - w1), likewise x)
//     w x ~= w1 x1 + w2 x1 + w1 x2,
// accumulated in fp32 in tensor memory. bf16 keeps 8 significant bits, so |w - w1 - w2| <= 2^-16 |w| and the three
// dropped terms are each <= 2^-16 |w||x|: error <= 3 * 2^-16 |w||x| per product (measured on the test layers:
// ~1-4 * 10^-6 of sum |w||x|), inside the 1e-4 gate, against ~2^-20 for the TF32 split. In exchange a 16-channel
// chunk takes three MMAs of K = 16 instead of six of K = 8 and its operands are half as many bytes: half the
// tensor-core time and little more than half the shared-memory traffic, the two bounds of ubp_tc2.cu.
//
// Differences from ubp_tc2.cu: the plan supplies W1 / W2 (bf16, K-major, 32-byte swizzle) already tiled into the
// 8 KB blocks a chunk needs, so a chunk's weights are one contiguous bulk copy; the tensor core cannot take the raw
// fp32 activations any more, so TMA copies the chunk's 16 channel rows as they are (plus a halo for 3x3) and the
// pass warps write BOTH x1 and x2, in the MN-major bf16 operand layout (64 columns x 8 channels atoms in the
// 128-byte swizzle; LBO = next 64 columns, SBO = next 8 channels); a pipeline stage holds one or two chunks
// (template parameter SUB), laid out by kind so that the weight blocks of its chunks arrive in one bulk copy and
// (1x1) their channel rows in one box; three threads issue the copies (lane 0 of warp 0 and of two extra warps after
// the epilogue warps); a pair may stack two 256-row MMA tiles on one staged activation tile (TcArgs::mt); layers of
// at most 128 rows run both CTAs on the one row tile (TcArgs::dup); a 1x1 with stride 2 reads the full-resolution
// input itself (template parameter S2, TcArgs::s2). Barriers, persistence, the two accumulators and the epilogue
// are those of ubp_tc2.cu.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "ubp_internal.h"
#include "ubp_tc_common.cuh"

namespace ubp {

namespace {

using namespace tc;

constexpr int T3_XL_WARPS = 8;                            // warps 2..9: the split pass
constexpr int T3_XL_GROUPS = 2;                           // two groups of four warps take turns on the chunks
constexpr int T3_EPI_WARPS = 8;                           // warps 10..17
// Copies are issued by three threads (lane 0 of warp 0 and of the last two warps): one for the weight copies of the first
// MMA tile, one for the activation copies, one for the weight copies of a stacked second MMA tile. With a single
// producer thread the ISSUE of a stage's copies was what a chunk waited for (each copy instruction holds its thread for
// the order of 100 cycles).
constexpr int T3_PROD2_WARP = 2 + T3_XL_WARPS + T3_EPI_WARPS;   // first of the two extra producer warps
constexpr int T3_THREADS = (T3_PROD2_WARP + 2) * 32;
constexpr int T3_MAX_STAGES = 8;
#ifndef T3_PRE
#define T3_PRE 1
#endif
#ifndef T3_SUB2_FROM
#define T3_SUB2_FROM 32                                   // chunks in the reduction from which a stage holds two
#endif
constexpr uint32_t T3_A_PART = 128 * TC_KC * 2;           // W1 or W2 chunk of this CTA's 128 rows: 4 KB
constexpr uint32_t T3_ATOM = 64 * TC_KC * 2;              // x1 or x2 of 64 columns x 16 channels: 2 KB
constexpr uint32_t T3_PIPE_BUDGET = 222 * 1024;
constexpr uint32_t SWZ_32B = 6, SWZ_128B = 2;             // descriptor layout types
constexpr uint32_t T3_ACC_COLS = 256;                     // tensor-memory columns per accumulator

// a chunk = W1 + W2 block (8 KB) + x1 + x2 tiles (2 KB per started 64 columns each) + the raw fp32 rows
// (16 channels x (columns + 2 x halo) floats, padded to 1 KB). The stage count is a multiple of the group count so
// that a stage always belongs to the same group of pass warps (a waiter must see every phase of its barrier).
__host__ __device__ constexpr uint32_t t3_x_bytes(int nh) { return (uint32_t)((nh + 63) / 64) * T3_ATOM; }
__host__ __device__ constexpr uint32_t t3_raw_bytes(int nh, int halo)
{
    return ((uint32_t)(nh + 2 * halo) * TC_KC * 4 + 1023u) & ~1023u;
}
// one chunk's part of a stage
// (np = pieces per operand: 2, or 3 for the variant whose products are exact to fp32's last bits)
// (mt = 256-row MMA tiles stacked on the same activation tile: each brings its own weight block)
__host__ __device__ constexpr uint32_t t3_chunk_bytes(int nh, int halo, int np, int mt = 1)
{
    return (uint32_t)(mt * np) * T3_A_PART + (uint32_t)np * t3_x_bytes(nh) + t3_raw_bytes(nh, halo);
}
// A stage holds `sub` chunks, part by part: the weight blocks of all its chunks (per MMA tile of a stack the chunks one
// after the other, as they lie in the plan: ONE bulk copy per MMA tile and stage), then each chunk's x1 / x2 tiles,
// then the raw rows of all chunks (1x1: consecutive channels, ONE tensor copy per stage). With two, every barrier round trip (copies landed -> split pass -> MMA issue -> stage
// free) serves 32 channels: fewer waits per channel, which pays on long reductions (3x3: 144 chunks; 1024 channels)
// where the pass or the issue thread is the bound; with one, the pipeline fills and drains in finer steps, which
// pays on short reductions (512 channels: 32 chunks).
__host__ __device__ constexpr uint32_t t3_stage_bytes(int nh, int halo, int sub, int np, int mt = 1)
{
    return (uint32_t)sub * t3_chunk_bytes(nh, halo, np, mt);
}
__host__ __device__ constexpr int t3_stages(int nh, int halo, int sub, int np, int mt = 1)
{
    const int s = (int)(T3_PIPE_BUDGET / t3_stage_bytes(nh, halo, sub, np, mt));
    return (s > T3_MAX_STAGES ? T3_MAX_STAGES : s) / T3_XL_GROUPS * T3_XL_GROUPS;
}

// instruction descriptor: D = f32, A = B = bf16, A K-major, B MN-major, M = 256 (two CTAs), N = n
__device__ __forceinline__ uint32_t make_idesc3(int n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}

// One chunk's three MMAs (K = 16 each: w1 x1, w1 x2, w2 x1; the second takes w1 from the tensor core's operand collector,
// where the first left it, instead of reading it from shared memory again -- shared memory is this kernel's wall) and, after a stage's last chunk (`last`), the commit that
// hands the stage back to both CTAs, in a single statement, with a non-blocking test of the NEXT stage's barrier
// issued first and its result read last. Executed by a whole converged warp: one elected lane issues. Returns
// whether the next stage is ready.
__device__ __forceinline__ bool mma3_chunk(uint32_t d_tmem, uint64_t dW1, uint64_t dX1, uint32_t w2_off, uint32_t x2_off,
                                           uint32_t idesc, uint32_t acc_first, uint32_t next_bar, uint32_t next_parity,
                                           uint32_t empty_bar, uint32_t last)
{
    uint32_t ready;
    asm volatile(
        "{\n\t.reg .pred pn, pa, pt, pe, pc;\n\t.reg .b64 w2, x2;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 pn, [%8], %9;\n\t"
        "elect.sync _|pe, 0xffffffff;\n\t"
        "setp.ne.b32 pc, %13, 0;\n\t"
        "and.pred pc, pc, pe;\n\t"
        "setp.ne.b32 pa, %7, 0;\n\t"
        "setp.eq.b32 pt, %10, 0;\n\t"
        "cvt.u64.u32 w2, %4;\n\tadd.s64 w2, w2, %2;\n\t"
        "cvt.u64.u32 x2, %5;\n\tadd.s64 x2, x2, %3;\n\t"
        "@pe tcgen05.mma.cta_group::2.kind::f16.collector::a::fill [%1], %2, %3, %6, pa;\n\t"
        "@pe tcgen05.mma.cta_group::2.kind::f16.collector::a::lastuse [%1], %2, x2, %6, pt;\n\t"
        "@pe tcgen05.mma.cta_group::2.kind::f16 [%1], w2, %3, %6, pt;\n\t"
        "@pc tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%11], %12;\n\t"
        "selp.u32 %0, 1, 0, pn;\n\t}"
        : "=r"(ready)
        : "r"(d_tmem), "l"(dW1), "l"(dX1), "r"(w2_off), "r"(x2_off), "r"(idesc), "r"(acc_first), "r"(next_bar),
          "r"(next_parity), "r"(0u), "r"(empty_bar), "h"((uint16_t)3), "r"(last)
        : "memory");
    return ready != 0;
}

// The same for operands in THREE bf16 pieces (w = w1 + w2 + w3 exactly, likewise x): the six products whose pieces'
// orders add up to at most four, w1 x1, w2 x1, w1 x2, w3 x1, w2 x2, w1 x3; what is dropped is below 2^-23 |w x|.
__device__ __forceinline__ bool mma6_chunk(uint32_t d_tmem, uint64_t dW1, uint64_t dX1, uint32_t w_step, uint32_t x_step,
                                           uint32_t idesc, uint32_t acc_first, uint32_t next_bar, uint32_t next_parity,
                                           uint32_t empty_bar, uint32_t last)
{
    uint32_t ready;
    asm volatile(
        "{\n\t.reg .pred pn, pa, pt, pe, pc;\n\t.reg .b64 w2, w3, x2, x3, ws, xs;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 pn, [%8], %9;\n\t"
        "elect.sync _|pe, 0xffffffff;\n\t"
        "setp.ne.b32 pc, %13, 0;\n\t"
        "and.pred pc, pc, pe;\n\t"
        "setp.ne.b32 pa, %7, 0;\n\t"
        "setp.eq.b32 pt, %10, 0;\n\t"
        "cvt.u64.u32 ws, %4;\n\tadd.s64 w2, ws, %2;\n\tadd.s64 w3, w2, ws;\n\t"
        "cvt.u64.u32 xs, %5;\n\tadd.s64 x2, xs, %3;\n\tadd.s64 x3, x2, xs;\n\t"
        "@pe tcgen05.mma.cta_group::2.kind::f16.collector::a::fill [%1], %2, %3, %6, pa;\n\t"
        "@pe tcgen05.mma.cta_group::2.kind::f16.collector::a::use [%1], %2, x2, %6, pt;\n\t"
        "@pe tcgen05.mma.cta_group::2.kind::f16.collector::a::lastuse [%1], %2, x3, %6, pt;\n\t"
        "@pe tcgen05.mma.cta_group::2.kind::f16.collector::a::fill [%1], w2, %3, %6, pt;\n\t"
        "@pe tcgen05.mma.cta_group::2.kind::f16.collector::a::lastuse [%1], w2, x2, %6, pt;\n\t"
        "@pe tcgen05.mma.cta_group::2.kind::f16 [%1], w3, %3, %6, pt;\n\t"
        "@pc tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%11], %12;\n\t"
        "selp.u32 %0, 1, 0, pn;\n\t}"
        : "=r"(ready)
        : "r"(d_tmem), "l"(dW1), "l"(dX1), "r"(w_step), "r"(x_step), "r"(idesc), "r"(acc_first), "r"(next_bar),
          "r"(next_parity), "r"(0u), "r"(empty_bar), "h"((uint16_t)3), "r"(last)
        : "memory");
    return ready != 0;
}

// eight fp32 -> three bf16 pieces each (x = x1 + x2 + x3 exactly: 8 + 8 + 8 significant bits), packed two per word
__device__ __forceinline__ void split8x3(const float (&v)[8], uint4 &p1, uint4 &p2, uint4 &p3)
{
    uint32_t a1[4], a2[4], a3[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __nv_bfloat162 a = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
        const float2 af = __bfloat1622float2(a);
        const float r0 = v[2 * i] - af.x, r1 = v[2 * i + 1] - af.y;
        const __nv_bfloat162 b = __floats2bfloat162_rn(r0, r1);
        const float2 bf = __bfloat1622float2(b);
        const __nv_bfloat162 c = __floats2bfloat162_rn(r0 - bf.x, r1 - bf.y);
        a1[i] = *reinterpret_cast<const uint32_t *>(&a);
        a2[i] = *reinterpret_cast<const uint32_t *>(&b);
        a3[i] = *reinterpret_cast<const uint32_t *>(&c);
    }
    p1 = make_uint4(a1[0], a1[1], a1[2], a1[3]);
    p2 = make_uint4(a2[0], a2[1], a2[2], a2[3]);
    p3 = make_uint4(a3[0], a3[1], a3[2], a3[3]);
}

// eight fp32 -> their bf16 heads (x1) and the bf16 of the remainders (x2), packed two per word
__device__ __forceinline__ void split8(const float (&v)[8], uint4 &h, uint4 &l)
{
    uint32_t hh[4], ll[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __nv_bfloat162 a = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
        const float2 af = __bfloat1622float2(a);
        const __nv_bfloat162 b = __floats2bfloat162_rn(v[2 * i] - af.x, v[2 * i + 1] - af.y);
        hh[i] = *reinterpret_cast<const uint32_t *>(&a);
        ll[i] = *reinterpret_cast<const uint32_t *>(&b);
    }
    h = make_uint4(hh[0], hh[1], hh[2], hh[3]);
    l = make_uint4(ll[0], ll[1], ll[2], ll[3]);
}

// four fp32 -> bf16 heads and bf16 remainders, packed two per word
__device__ __forceinline__ void split4(const float4 &v, uint2 &h, uint2 &l)
{
    const __nv_bfloat162 a0 = __floats2bfloat162_rn(v.x, v.y), a1 = __floats2bfloat162_rn(v.z, v.w);
    const float2 f0 = __bfloat1622float2(a0), f1 = __bfloat1622float2(a1);
    const __nv_bfloat162 b0 = __floats2bfloat162_rn(v.x - f0.x, v.y - f0.y), b1 = __floats2bfloat162_rn(v.z - f1.x, v.w - f1.y);
    h = make_uint2(*reinterpret_cast<const uint32_t *>(&a0), *reinterpret_cast<const uint32_t *>(&a1));
    l = make_uint2(*reinterpret_cast<const uint32_t *>(&b0), *reinterpret_cast<const uint32_t *>(&b1));
}

// (S2: the 1x1 product with stride 2 read straight from the full-resolution input, see TcArgs::s2 -- an instance of its
// own: as a run-time branch it cost the ordinary kernel's split pass 1.5 - 4 %)
template <bool CONV, int SUB, int NP, bool S2 = false>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(T3_THREADS, 1)
ubp_tc3_kernel(const uint8_t *__restrict__ W16, const __grid_constant__ CUtensorMap tmX, const TcArgs a,
               const int halo, const int nrp, const int ntiles)
{
    constexpr int MAXS = T3_MAX_STAGES;
    constexpr uint32_t TMEM_COLS = 2 * T3_ACC_COLS;

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
    const uint32_t xb = t3_x_bytes(NH);                    // x1 (and x2) bytes per chunk
    // MT 256-row MMA tiles share the staged activations (MT = 2: the pair owns tiles of 512 rows, their two
    // accumulators side by side in tensor memory, so a tile's epilogue is not hidden under the next tile's main loop;
    // the split pass then runs once for both)
    const int MT = a.mt > 1 ? 2 : 1;
    const uint32_t wbytes = (uint32_t)(MT * NP) * T3_A_PART;   // weight blocks at the head of a chunk
    const uint32_t stage_bytes = (uint32_t)SUB * t3_chunk_bytes(NH, halo, NP, MT);
    // inside a stage: weight blocks [MMA tile][chunk], x tiles [chunk][piece], raw rows [chunk]
    const uint32_t xoff = (uint32_t)SUB * wbytes, xchunk = (uint32_t)NP * xb, roff = xoff + (uint32_t)SUB * xchunk;
    const uint32_t raw_row = (uint32_t)(NH + 2 * halo) * 4;   // bytes per channel row of the raw copy
    const int S = t3_stages(NH, halo, SUB, NP, MT);
    const int nchunk = (a.K + TC_KC - 1) / TC_KC;
    const int nstage = (nchunk + SUB - 1) / SUB;     // stages per tile; the last one may hold a single chunk
    const uint32_t raw_chunk = raw_row * TC_KC;            // raw bytes per chunk
    constexpr bool XMERGED = !CONV && SUB > 1;             // one tensor copy brings the rows of all the stage's chunks
    const int Cin = CONV ? a.K / 9 : a.K;                  // 3x3: reduction index k = tap * Cin + channel, Cin % 16 == 0
    // this pair's tiles: pair, pair + npairs, ...; tile t = (row pair t % nrp, column tile t / nrp)
    const int npairs = (int)(gridDim.x >> 1), pair = (int)(blockIdx.x >> 1);
    const int nmy = pair < ntiles ? (ntiles - pair + npairs - 1) / npairs : 0;
    const int rpc = 128;                                   // output rows per CTA
    // first row of this CTA in the tile's first MMA tile; MMA tile m of the tile starts 2 m rpc rows further on
    // (layers of at most 128 rows: both CTAs take the layer's only row tile, see TcArgs::dup)
    auto tile_row0 = [&](int i) { return (((pair + i * npairs) % nrp) * 2 * MT + (a.dup ? 0 : (int)rank)) * rpc; };
    auto tile_col0 = [&](int i) { return (int64_t)((pair + i * npairs) / nrp) * N; };

    // one stage's copies (stage sg of a tile = chunks sg * SUB ...): per chunk the W1 / W2 block of this CTA's 128
    // rows (8 KB, stored in the plan exactly as it must lie in shared memory: one contiguous bulk copy) and 16
    // channel rows of the input for this CTA's columns (3x3: the channels of the chunk's tap, and a halo of columns
    // either side). The weight copies come first and announce the bytes of both; the activation copies may follow
    // later (the kernel's first stages start their weight copies before the previous kernel in the stream is done).
    // (the thread that issues MMA tile 0's weights also announces the stage's bytes; the other copies may complete
    // before that: the phase cannot end until the announcing arrival has come)
    auto issue_w = [&](int sg, int st, int row0, int m) {
        const uint32_t bar = smem_u32(&bar_full[st]);
        const int c0 = sg * SUB, nsub = nchunk - c0 < SUB ? nchunk - c0 : SUB;
        // (a merged activation copy always brings the whole box: rows past the last channel arrive as zeros)
        if (m == 0) mbar_expect_tx(bar, (uint32_t)nsub * wbytes + (uint32_t)(XMERGED ? SUB : nsub) * raw_chunk);
        uint8_t *stage = smem + (size_t)st * stage_bytes;
        bulk_load(smem_u32(stage + (uint32_t)(m * SUB) * (NP * T3_A_PART)),
                  W16 + ((size_t)(row0 / rpc + 2 * m) * nchunk + c0) * (NP * T3_A_PART), (uint32_t)nsub * (NP * T3_A_PART), bar);
    };
    auto issue_x = [&](int sg, int st, int xcol) {
        const uint32_t bar = smem_u32(&bar_full[st]);
        const int c0 = sg * SUB, nsub = nchunk - c0 < SUB ? nchunk - c0 : SUB;
        uint8_t *raw = smem + (size_t)st * stage_bytes + roff;
        if constexpr (S2) {
            // stride 2: the even input rows of this CTA's NH / Wo output rows, all the stage's channels in one box
            // (`halo` = NH / 2 here: it only sizes the raw rows, 2 NH floats per channel)
            tma_load_3d(smem_u32(raw), &tmX, 0, xcol / a.s2, c0 * TC_KC, bar);
        } else if constexpr (XMERGED) {
            tma_load_2d(smem_u32(raw), &tmX, xcol - halo, c0 * TC_KC, bar);
        } else {
#pragma unroll
            for (int u = 0; u < SUB; ++u) {
                if (u >= nsub) break;
                const int c = c0 + u;
                tma_load_2d(smem_u32(raw + (uint32_t)u * raw_chunk), &tmX, xcol - halo, CONV ? (c * TC_KC) % Cin : c * TC_KC, bar);
            }
        }
    };
    // stages whose weight copies start before the wait for the previous kernel
    const int npre = nmy * nstage < (T3_PRE < S ? T3_PRE : S) ? nmy * nstage : (T3_PRE < S ? T3_PRE : S);   // never beyond the ring

    // Launched with programmatic stream serialisation, the grid may become resident while the kernel before it in
    // the stream is still running: let the kernel after this one do the same, set up everything that reads no global
    // data, and only then wait for the earlier kernel's results (a plain launch passes both instructions at once).
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (threadIdx.x == 0) {
        prefetch_tensormap(&tmX);
        abort_flag = 0;
        for (int s = 0; s < S; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_go[s]), 2 * (T3_XL_WARPS / T3_XL_GROUPS));   // used in the leader CTA only
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&bar_acc_full[b]), 1);
            mbar_init(smem_u32(&bar_acc_empty[b]), 2 * T3_EPI_WARPS);            // used in the leader CTA only
        }
        mbar_init(smem_u32(&bar_last), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        // The first copies land in this CTA's own memory and signal its own barriers: start them before the
        // tensor-memory allocation and the cluster barrier. The weights are constants of the layer, so the copies of
        // the ring's first stages do not wait for the kernel before this one; the activations may be its output.
        for (int f = 0; f < npre; ++f)
            for (int m = 0; m < MT; ++m) issue_w(f % nstage, f, tile_row0(f / nstage), m);
    }
    // Cluster barrier, first half: every thread arrives once its CTA's barriers exist (thread 0: after it has
    // initialised them). The wait comes after the wait for the earlier kernel, by when the other CTA has normally
    // arrived long ago: the barrier's round trip is off the path.
    asm volatile("barrier.cluster.arrive.release;" ::: "memory");
    if (warp == 1) {   // tensor memory of the pair: the same warp of both CTAs allocates
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");     // every thread: nothing below may overtake the earlier kernel
    if (threadIdx.x == 0)
        for (int f = 0; f < npre; ++f) issue_x(f % nstage, f, (int)(tile_col0(f / nstage) + (int64_t)rank * NH));
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("barrier.cluster.wait.acquire;" ::: "memory");   // both CTAs' barriers exist before anyone signals them
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_slot;

    bool ok = true;
    if (warp == 0 || warp >= T3_PROD2_WARP) {
        // ---------------- TMA producers: one ring of S stages straight through all of this pair's tiles; each of the
        // three threads issues its own kind of copy for every stage (what: 0 = weights of MMA tile 0, 1 = activations,
        // 2 = weights of a stacked second MMA tile) and waits for the stage itself
        const int what = warp == 0 ? 0 : warp - T3_PROD2_WARP + 1;
        if (lane == 0 && (what < 2 || MT == 2)) {
            int st = npre % S, round = npre / S;           // the first npre stages were started above
            int f = 0;                                     // stages counted through all tiles
            for (int i = 0; i < nmy && ok; ++i) {
                const int row0 = tile_row0(i), xcol = (int)(tile_col0(i) + (int64_t)rank * NH);
                for (int sg = 0; sg < nstage; ++sg, ++f) {
                    if (f < npre) continue;
                    if (round > 0) {                       // the stage's previous contents must have been consumed
                        ok = mbar_wait(smem_u32(&bar_empty[st]), (uint32_t)(round - 1) & 1u, &abort_flag);   // polling: one lane per warp
                        if (!ok) break;
                    }
                    if (what == 1) issue_x(sg, st, xcol);
                    else issue_w(sg, st, row0, what >> 1);
                    if (++st == S) { st = 0; ++round; }
                }
            }
        }
    } else if (warp == 1) {
        if (rank == 0) {
            // ---------------- leader: MMA issuer for the pair (whole warp converged, one elected lane issues)
            const uint32_t idesc = make_idesc3(N);
            const uint64_t dW0 = make_desc(smem_u32(smem), 16, 256, SWZ_32B);
            const uint64_t dX0 = make_desc(smem_u32(smem) + xoff, 2048, 1024, SWZ_128B);
            const uint32_t stage_u = stage_bytes >> 4, wchunk_u = (NP * T3_A_PART) >> 4, xchunk_u = xchunk >> 4;
            int st = 0;
            uint32_t ph = 0;
            bool ready = nmy > 0 && mbar_try_wait(smem_u32(&bar_go[0]), 0);
            for (int i = 0; i < nmy && ok; ++i) {
                // two accumulators take turns -- or, with stacked tiles, one tile owns both and the next tile waits
                // for this one's epilogue
                const int b = MT == 2 ? 0 : (i & 1);
                const uint32_t acc = tmem_base + (uint32_t)b * T3_ACC_COLS;
                if (MT == 2 ? i >= 1 : i >= 2) {           // the epilogue of the tile that used it must have read this accumulator
                    ok = mbar_wait(smem_u32(&bar_acc_empty[b]), (uint32_t)(MT == 2 ? i - 1 : (i >> 1) - 1) & 1u, &abort_flag);
                    if (!ok) break;
                }
                for (int sg = 0; sg < nstage; ++sg) {
                    if (!ready) ok = mbar_wait(smem_u32(&bar_go[st]), ph, &abort_flag);
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint64_t soff = (uint64_t)((uint32_t)st * stage_u);
                    int nst = st + 1;
                    uint32_t nph = ph;
                    if (nst == S) { nst = 0; nph ^= 1u; }
                    const int nsub = nchunk - sg * SUB < SUB ? nchunk - sg * SUB : SUB;
#pragma unroll
                    for (int u = 0; u < SUB; ++u)
                        if (u < nsub) {
                            if constexpr (NP == 3) {
                                ready = mma6_chunk(acc, dW0 + soff + (uint64_t)(u * wchunk_u), dX0 + soff + (uint64_t)(u * xchunk_u),
                                                   T3_A_PART >> 4, xb >> 4, idesc, (sg > 0 || u > 0) ? 1u : 0u, smem_u32(&bar_go[nst]), nph,
                                                   smem_u32(&bar_empty[st]), u == nsub - 1 ? 1u : 0u);
                            } else {
                                // every MMA tile of the stack on the same x1 / x2; the stage goes back after the last one
                                for (int m = 0; m < MT; ++m)
                                    ready = mma3_chunk(acc + (uint32_t)m * T3_ACC_COLS,
                                                       dW0 + soff + (uint64_t)((uint32_t)(m * SUB + u) * wchunk_u),
                                                       dX0 + soff + (uint64_t)(u * xchunk_u), T3_A_PART >> 4, xb >> 4, idesc,
                                                       (sg > 0 || u > 0) ? 1u : 0u, smem_u32(&bar_go[nst]), nph,
                                                       smem_u32(&bar_empty[st]), (u == nsub - 1 && m == MT - 1) ? 1u : 0u);
                            }
                        }
                    st = nst; ph = nph;
                }
                if (!ok) break;
                mma2_commit_both(smem_u32(&bar_acc_full[b]));     // accumulator complete: epilogue warps of both CTAs
                if (i == nmy - 1) mma2_commit_both(smem_u32(&bar_last));
            }
        }
    } else if (warp < 2 + T3_XL_WARPS) {
        // ---------------- split pass: raw fp32 rows -> x1, x2 (bf16) in the operand layout. Two groups of four
        // warps take turns on the chunks. Thread (cg, kq) of a group: columns 8 cg .. 8 cg + 7 of the CTA's part
        // of the tile, channels kq and kq + 8 of the chunk.
        constexpr int GT = (T3_XL_WARPS / T3_XL_GROUPS) * 32;
        const int grp = (warp - 2) / (T3_XL_WARPS / T3_XL_GROUPS);
        const int gt = (int)threadIdx.x - 64 - grp * GT;
        // Up to 64 columns per CTA: 8 column groups x 16 channels, one channel per thread; wider: 16 column groups x 8
        // channel pairs, two channels per thread.
        const bool narrow = NH <= 64;
        const int cg = narrow ? (gt & 7) : (gt & 15), kq = narrow ? (gt >> 3) : (gt >> 4);
        const int nk = narrow ? 1 : 2;
        const bool mine = cg * 8 < NH;
        const int total = nmy * nstage;
        const uint32_t dst = (uint32_t)(cg >> 3) * T3_ATOM;   // 64-column atom; inside it row k is 128 bytes whose
        const uint32_t c16 = (uint32_t)(cg & 7);              // 16-byte pieces are XOR-swizzled with k mod 8
        unsigned long long tap_lo = 0;                         // 3x3: bit tap * 8 + e (taps 0..7): tap inside the image
        uint32_t tap_hi = 0;                                   //      for column 8 cg + e; tap 8 in tap_hi
        int mask_tile = -1;
        // tile and stage in the tile of this group's current stage; 3x3: tap and first channel of its first chunk,
        // kept by increments (a division per chunk is what the pass cannot afford)
        int ti = grp / nstage, sg = grp % nstage;
        int tp = CONV ? (sg * SUB * TC_KC) / Cin : 0, ch = CONV ? (sg * SUB * TC_KC) % Cin : 0;
        int st = grp;                                      // the stage count is even: stages grp, grp + 2, ...
        uint32_t ph = 0;
        for (int f = grp; f < total && ok; f += T3_XL_GROUPS) {
            ok = mbar_wait_relaxed(smem_u32(&bar_full[st]), ph, &abort_flag);
            if (!ok) break;
            if (CONV && ti != mask_tile) {                 // new tile: which taps of my eight columns are inside the image
                mask_tile = ti;
                const int64_t n0 = tile_col0(ti) + (int64_t)rank * NH + 8 * cg;
                const uint32_t hw = (uint32_t)(a.H * a.W);
                tap_lo = 0; tap_hi = 0;
                if (mine && n0 < a.Nc) {
                    // pixel of the first column by two 32-bit divisions (column numbers are below 2^31), the other
                    // seven by stepping; a tap is inside the image when its row and its column are
                    uint32_t pix = (uint32_t)n0 % hw;
                    int y = (int)(pix / (uint32_t)a.W), x = (int)(pix - (uint32_t)y * (uint32_t)a.W);
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        if (n0 + e < a.Nc) {
                            const uint32_t rows = (y > 0 ? 1u : 0u) | 2u | (y < a.H - 1 ? 4u : 0u);
                            const uint32_t cols = (x > 0 ? 1u : 0u) | 2u | (x < a.W - 1 ? 4u : 0u);
#pragma unroll
                            for (int t9 = 0; t9 < 9; ++t9)
                                if (((rows >> (t9 / 3)) & (cols >> (t9 % 3)) & 1u) != 0u) {
                                    if (t9 < 8) tap_lo |= 1ull << (t9 * 8 + e); else tap_hi |= 1u << e;
                                }
                        }
                        if (++x == a.W) { x = 0; if (++y == a.H) y = 0; }
                    }
                }
            }
            const int nsub = nchunk - sg * SUB < SUB ? nchunk - sg * SUB : SUB;
            int tpu = tp, chu = ch;                        // 3x3: tap / channel of chunk u of the stage
#pragma unroll
            for (int u = 0; u < SUB; ++u) {
                if (u >= nsub) break;
                uint8_t *x1 = smem + (size_t)st * stage_bytes + xoff + (uint32_t)u * xchunk;
                const uint8_t *raw = smem + (size_t)st * stage_bytes + roff + (uint32_t)u * raw_chunk;
                int sh = 0;
                uint32_t ok8 = 0xffu;
                if (CONV) {
                    sh = (tpu / 3 - 1) * a.W + (tpu % 3 - 1) + halo;        // >= 0: offset into the raw rows
                    ok8 = tpu < 8 ? (uint32_t)(tap_lo >> (tpu * 8)) & 0xffu : tap_hi;
                    chu += TC_KC;
                    if (chu >= Cin) { chu = 0; ++tpu; }
                }
                if (!CONV && !S2 && NP == 2 && !narrow) {
                    // 1x1, more than 64 columns per CTA: thread (j, kq) takes the 16-byte pieces j and 16 + j of its
                    // rows -- columns 4 j .. 4 j + 3 of both 64-column atoms -- so that eight neighbouring threads read
                    // 128 contiguous bytes (eight columns per thread = 32-byte steps cost every 128-bit load two
                    // wavefronts: 37 % of the kernel's shared-memory wavefronts were such conflicts) and a half warp's
                    // 8-byte stores fill one 128-byte row of an atom
                    const uint32_t j = (uint32_t)cg;
                    const bool has2 = 64 + 4 * (int)j < NH;
                    // (checked build: the last byte this thread reads lies inside its raw rows and the CTA's shared memory,
                    // its writes inside the two atoms of the x1 / x2 tiles)
                    [[maybe_unused]] const uint32_t rd_end = (has2 ? 256u : 0u) + j * 16u + 16u;
                    if (UBP_CHK_SMEM(rd_end <= raw_row && (size_t)(raw - smem_raw) + 15u * raw_row + rd_end <= tc::dbg_dynamic_smem() &&
                                     2u * T3_ATOM <= xb, a.status)) {
#pragma unroll
                        for (int i = 0; i < 2; ++i) {
                            const int k = kq + 8 * i;
                            const uint8_t *rowp = raw + k * raw_row;
                            const float4 qa = *reinterpret_cast<const float4 *>(rowp + j * 16u);
                            uint2 h, l;
                            split4(qa, h, l);
                            const uint32_t off = (uint32_t)k * 128u + (((j >> 1) ^ ((uint32_t)k & 7u)) << 4) + (j & 1u) * 8u;
                            *reinterpret_cast<uint2 *>(x1 + off) = h;
                            *reinterpret_cast<uint2 *>(x1 + xb + off) = l;
                            if (has2) {
                                const float4 qb = *reinterpret_cast<const float4 *>(rowp + 256u + j * 16u);
                                split4(qb, h, l);
                                *reinterpret_cast<uint2 *>(x1 + T3_ATOM + off) = h;
                                *reinterpret_cast<uint2 *>(x1 + xb + T3_ATOM + off) = l;
                            }
                        }
                    }
                } else
                // (checked build: the columns this thread needs lie inside the raw rows, everything it reads inside the
                // CTA's shared memory, its writes inside the x1 / x2 tiles)
                if (mine && UBP_CHK_SMEM(sh >= 0 && (uint32_t)((S2 ? 16 * cg + 8 : 8 * cg + sh) + 8) * 4u <= raw_row &&
                                         (size_t)(raw - smem_raw) + 15u * raw_row + (uint32_t)((8 * cg + sh) & ~3) * 4u + 48u <= tc::dbg_dynamic_smem() &&
                                         dst + 16u * 128u <= xb, a.status)) {
                    constexpr bool s2 = S2;
                    const int o = s2 ? 16 * cg : 8 * cg + sh, ob = o & ~3, r = o & 3;      // r is the same for every lane
#pragma unroll
                    for (int i = 0; i < 2; ++i) {
                        if (i >= nk) break;
                        const int k = kq + 8 * i;
                        const float4 q0 = *reinterpret_cast<const float4 *>(raw + k * raw_row + ob * 4);
                        const float4 q1 = *reinterpret_cast<const float4 *>(raw + k * raw_row + ob * 4 + 16);
                        float v[8];
                        if constexpr (s2) {    // every other pixel of the even rows: floats 2 j of the copy
                            const float4 q2 = *reinterpret_cast<const float4 *>(raw + k * raw_row + ob * 4 + 32);
                            const float4 q3 = *reinterpret_cast<const float4 *>(raw + k * raw_row + ob * 4 + 48);
                            v[0] = q0.x; v[1] = q0.z; v[2] = q1.x; v[3] = q1.z; v[4] = q2.x; v[5] = q2.z; v[6] = q3.x; v[7] = q3.z;
                        } else if (!CONV || r == 0) {
                            v[0] = q0.x; v[1] = q0.y; v[2] = q0.z; v[3] = q0.w; v[4] = q1.x; v[5] = q1.y; v[6] = q1.z; v[7] = q1.w;
                        } else {
                            const float4 q2 = *reinterpret_cast<const float4 *>(raw + k * raw_row + ob * 4 + 32);
                            const float t[12] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w, q2.x, q2.y, q2.z, q2.w};
                            if (r == 1) { for (int e = 0; e < 8; ++e) v[e] = t[e + 1]; }
                            else if (r == 2) { for (int e = 0; e < 8; ++e) v[e] = t[e + 2]; }
                            else { for (int e = 0; e < 8; ++e) v[e] = t[e + 3]; }
                        }
                        if (CONV) {
#pragma unroll
                            for (int e = 0; e < 8; ++e) if (!((ok8 >> e) & 1u)) v[e] = 0.f;
                        }
                        const uint32_t off = dst + (uint32_t)k * 128u + ((c16 ^ ((uint32_t)k & 7u)) << 4);
                        if constexpr (NP == 3) {
                            uint4 p1, p2, p3;
                            split8x3(v, p1, p2, p3);
                            *reinterpret_cast<uint4 *>(x1 + off) = p1;
                            *reinterpret_cast<uint4 *>(x1 + xb + off) = p2;
                            *reinterpret_cast<uint4 *>(x1 + 2 * xb + off) = p3;
                        } else {
                            uint4 h, l;
                            split8(v, h, l);
                            *reinterpret_cast<uint4 *>(x1 + off) = h;
                            *reinterpret_cast<uint4 *>(x1 + xb + off) = l;
                        }
                    }
                }
            }
            // this group's next stage is T3_XL_GROUPS stages on
            for (int g = 0; g < T3_XL_GROUPS; ++g) {
                if (++sg == nstage) { sg = 0; ++ti; tp = 0; ch = 0; }
                else if (CONV) {
                    for (int u = 0; u < SUB; ++u) { ch += TC_KC; if (ch >= Cin) { ch = 0; ++tp; } }
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // make the writes visible to the MMA unit
            __syncwarp();
            if (lane == 0) {
                if (rank == 0) mbar_arrive(smem_u32(&bar_go[st]));
                else mbar_arrive_remote(smem_u32(&bar_go[st]), 0);
            }
            st += T3_XL_GROUPS;
            if (st >= S) { st -= S; ph ^= 1u; }
        }
        // ---------------- the last tile has nothing to overlap with: take the 16-column units 2, 3, 6, 7, ... of its epilogue.
        // Its own barrier (one phase) rather than the accumulator's, whose earlier phases these warps did not see.
        if (ok && nmy > 0) ok = mbar_wait_relaxed(smem_u32(&bar_last), 0, &abort_flag);
        if (ok && nmy > 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int i = nmy - 1;
            for (int m = 0; m < MT; ++m)
                epilogue_blocks(a, tmem_base + (uint32_t)(MT == 2 ? m : (i & 1)) * T3_ACC_COLS, warp & 3, 2 + ((warp - 2) >> 2), 4, N,
                                tile_row0(i) + 2 * m * rpc, tile_col0(i), lane, 0u, rank);
        }
    } else {
        // ---------------- epilogue warps: tile i's accumulator while the main loop works on tile i + 1
        const int part = (warp - 2 - T3_XL_WARPS) >> 2;       // two warps share a lane quarter and split the columns
        for (int i = 0; i < nmy && ok; ++i) {
            const int b = MT == 2 ? 0 : (i & 1);
            ok = mbar_wait_relaxed(smem_u32(&bar_acc_full[b]), (uint32_t)(MT == 2 ? i : (i >> 1)) & 1u, &abort_flag);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const bool last = i == nmy - 1;
            for (int m = 0; m < MT; ++m)     // (stacked: the accumulators go back once the second one has been read)
                epilogue_blocks(a, tmem_base + (uint32_t)(b + m) * T3_ACC_COLS, warp & 3, part, last ? 4 : 2, N,
                                tile_row0(i) + 2 * m * rpc, tile_col0(i), lane,
                                (last || m != MT - 1) ? 0u : smem_u32(&bar_acc_empty[b]), rank);
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

// Launch the bf16 pair kernel on tiles of 256 rows x `ntile` columns (a multiple of 16; of 32 where both CTAs take the one row tile).
// W16: the plan's bf16 part: 8 KB blocks [row tile of 128][chunk] = [W1, W2][128 rows][16 channels], pre-swizzled.
// chunks per pipeline stage: two on reductions of 32 chunks and more (where the ring still gets four stages), else one
int tc_pair_bf16_sub(int K, int ntile, int halo, int pieces, int mt)
{
    return pieces == 2 && (K + TC_KC - 1) / TC_KC >= T3_SUB2_FROM && t3_stages(ntile / 2, halo, 2, pieces, mt) >= 4 ? 2 : 1;
}

// tmX: plain 2-D fp32 map (column, channel), box (ntile/2 + 2 halo) x 16 -- 1x1: x 16 tc_pair_bf16_sub(...), one copy
// per stage; halo = 0 for 1x1, image width + 1 rounded up to a multiple of 4 for 3x3 (columns = the flattened
// (b, y, x) axis).
int launch_tc_pair_bf16(const void *W16, const CUtensorMap_st *tmX, int conv, int halo, const void *args_,
                        int M, int64_t Nc, int ntile, int sms, void *stream, int pieces, int mt)
{
    TcArgs a = *static_cast<const TcArgs *>(args_);
    a.ntile = ntile;
    a.mt = mt;
    const int nh = ntile / 2;
    if (ntile % 16 != 0 || (a.dup && ntile % 32 != 0) || ntile < 32 || ntile > 256) return UBP_E_UNSUPPORTED;
    if (pieces != 2 && !(pieces == 3 && !conv)) return UBP_E_UNSUPPORTED;
    // tiles of 512 rows: two-piece 1x1 products of layers whose rows fill whole 512-row tiles
    if (mt != 1 && !(mt == 2 && pieces == 2 && !conv && ((M + 255) / 256) % 2 == 0)) return UBP_E_UNSUPPORTED;
    const int sub = tc_pair_bf16_sub(a.K, ntile, halo, pieces, mt);
    if (t3_stages(nh, halo, sub, pieces, mt) < 4) return UBP_E_UNSUPPORTED;
    size_t smem = (size_t)t3_stages(nh, halo, sub, pieces, mt) * t3_stage_bytes(nh, halo, sub, pieces, mt) + 1024;
    if (smem < TC_PAIR_MIN_SMEM) smem = TC_PAIR_MIN_SMEM;   // one CTA per SM, whatever the tile width (see the constant)
    static bool done[7][64] = {};
    int devid = 0;
    if (cudaGetDevice(&devid) != cudaSuccess) devid = -1;
    if (a.s2 && (conv || pieces != 2)) return UBP_E_UNSUPPORTED;
    const int which = a.s2 ? 5 + (sub == 2 ? 1 : 0) : pieces == 3 ? 4 : (conv ? 2 : 0) + (sub == 2 ? 1 : 0);
    using KernelFn = void (*)(const uint8_t *, const CUtensorMap, const TcArgs, const int, const int, const int);
    const KernelFn kernels[7] = {ubp_tc3_kernel<false, 1, 2>, ubp_tc3_kernel<false, 2, 2>, ubp_tc3_kernel<true, 1, 2>,
                                 ubp_tc3_kernel<true, 2, 2>, ubp_tc3_kernel<false, 1, 3>,
                                 ubp_tc3_kernel<false, 1, 2, true>, ubp_tc3_kernel<false, 2, 2, true>};
    const KernelFn kern = kernels[which];
    if (devid < 0 || devid >= 64 || !done[which][devid]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(T3_PIPE_BUDGET + 1024));
        if (e != cudaSuccess) { set_last_cuda_error((int)e); return UBP_E_CUDA; }
        // the smallest launch this function ever makes must already fill an SM (a query, nothing is launched)
        int per_sm = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, T3_THREADS, TC_PAIR_MIN_SMEM);
        if (e != cudaSuccess) { set_last_cuda_error((int)e); return UBP_E_CUDA; }
        if (per_sm != 1) return UBP_E_UNSUPPORTED;
        if (devid >= 0 && devid < 64) done[which][devid] = true;
    }
    const int nrp = (M + 256 * mt - 1) / (256 * mt);
    const long long ntiles = (long long)nrp * ((Nc + ntile - 1) / ntile);
    if (ntiles <= 0) return UBP_OK;
    if (ntiles > 0x7fffffffll) return UBP_E_UNSUPPORTED;
    const long long pairs = ntiles < sms / 2 ? ntiles : sms / 2;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * pairs));
    cfg.blockDim = dim3(T3_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, static_cast<const uint8_t *>(W16), *tmX, a, halo, nrp, (int)ntiles);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) { set_last_cuda_error((int)e); return UBP_E_CUDA; }
    return UBP_OK;
}

int tc_pair_bf16_stages_sub(int ntile, int halo, int sub, int mt) { return t3_stages(ntile / 2, halo, sub, 2, mt); }
// how many pipeline stages the bf16 pair kernel gets for a tile width and halo
int tc_pair_bf16_stages(int ntile, int halo, int mt) { return t3_stages(ntile / 2, halo, 1, 2, mt); }

}  // namespace ubp
