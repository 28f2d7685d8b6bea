// 3x3 / stride 1 / pad 1 convolution of a block-pruned layer as an implicit GEMM on CTA pairs, with the nine taps taken
// as SHIFTS OF ONE STAGED OPERAND (block = Nb output channels x one input channel x all nine taps, Section 3.1; bf16
// products as in ubp_tc3.cu: w x ~= w1 x1 + w2 x1 + w1 x2, fp32 accumulation in tensor memory).
//
// ubp_tc3.cu copies and splits the activations of a 16-channel chunk once per TAP, cutting a shifted, border-masked
// tile for each of the nine; that pass bounds it (about 790 cycles per tap and chunk against 290 of MMA). Here:
//   * the outputs are computed on the zero-PADDED pixel grid: column p = (b, yp, xp) with yp in [0, H+2), xp in
//     [0, W+2); on that grid tap (dy, dx) is the pure shift (dy-1) (W+2) + (dx-1), no tap ever wraps into a
//     neighbouring row or image and no mask is needed. Padded positions are computed and thrown away
//     (H W / ((H+2)(W+2)) of the MMA work is useful: 77 % at 14 x 14, 87 % at 28 x 28);
//   * per 16-channel group the raw fp32 rows of the real pixels a tile touches come in by ONE TMA copy, and the pass
//     warps build the operand ONCE: for every padded position of the tile and a halo of W+3 positions either side,
//     the eight channels of a k-group as 16 contiguous bytes (x1), likewise x2; padded positions are zeros. This is
//     the K-major operand layout WITHOUT swizzle whose core matrices (8 positions x 16 bytes) lie back to back, so a
//     descriptor may start at ANY position: the MMAs of tap (dy, dx) use start + 16 bytes x (halo + shift);
//   * the weights of a channel group (nine taps x 8 KB per CTA, the plan's bf16 tiling indexed as chunk = tap * C/16 +
//     group) come as one barrier phase of a two-stage ring; the leader issues the group's 27 MMAs back to back.
// Roles per CTA (608 threads): warp 0 weight producer (bulk copies), warp 1 MMA issuer (leader CTA only), warp 2 raw-row
// producer (TMA),
// warps 3-10 operand pass (they also tell the leader that this CTA's weights of the group have landed), warps 11-18
// epilogue (tile i while the main loop works on tile i + 1; two accumulators). All waits are bounded; no load is
// multicast.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "ubp_internal.h"
#include "ubp_tc_common.cuh"

namespace ubp {

namespace {

using namespace tc;

constexpr int C3_PASS_WARPS = 8, C3_EPI_WARPS = 8;
constexpr int C3_FIRST_PASS = 3, C3_FIRST_EPI = C3_FIRST_PASS + C3_PASS_WARPS;
constexpr int C3_THREADS = (C3_FIRST_EPI + C3_EPI_WARPS) * 32;          // 608
constexpr int C3_MAX_XS = 6;                   // stages of raw rows and of built operands (one group step each): 2 .. 6
constexpr int C3_MAX_WG = 4;                   // stages of the weight ring; a stage holds the taps of one group step
                                               // (nine, 72 KB; stride 2: at most six, 48 KB)
constexpr uint32_t C3_W_BYTES = 2 * 128 * TC_KC * 2;                      // W1 + W2 of one (tap, group): 8 KB
constexpr uint32_t C3_ACC_COLS = 256;
constexpr uint32_t C3_SWZ_32B = 6;

struct C3Geom {
    int N;            // padded positions per tile (multiple of 16, <= 256); each CTA holds N / 2
    int halo;         // W + 3: the largest shift
    int E;            // staged positions per CTA: N / 2 + 2 halo, rounded up to a multiple of 8 (<= 256)
    int rawn;         // real pixels copied per channel row: E + 4 rounded up to a multiple of 4
    int xs;           // stages of raw rows / built operands
    int nrp;          // row pairs (256 output rows each)
    int ntiles;       // nrp x column tiles
    int Pn;           // padded positions in all: B (H+2) (W+2)
    int cg;           // channel groups: C / 16
    int wg;           // weight stages: 2 (nine taps each; stride 2: at most six taps each)
    int s2;           // 1: stride 2 -- X holds the four phase planes (rows phase * C + channel), a tile's group steps are
                      // (channel group, phase pair {0, 1} or {2, 3}): a stage holds the raw rows and the operands of both
                      // phases of the pair, and each phase has its own taps, all of them shifts of 0 or -1
};
// The taps of a group step and their shifts on the padded grid (row pitch Wp). Stride 1: all nine, shift (dy-1) Wp +
// (dx-1). Stride 2: output (yo, xo) reads input (2 yo + dy - 1, 2 xo + dx - 1) = plane (dy != 1, dx != 1) at
// (yo - [dy == 0], xo - [dx == 0]).
// (stride 2: `hf` = which phase pair; taps of phase 2 hf first, then those of phase 2 hf + 1; `sub` = which of the
// stage's two operands the tap reads)
__device__ __forceinline__ int c3_ntaps(int s2, int hf) { return !s2 ? 9 : (hf == 0 ? 3 : 6); }
__device__ __forceinline__ void c3_tap(int s2, int hf, int t, int Wp, int &tap, int &shift, int &sub)
{
    if (!s2) { tap = t; shift = (t / 3 - 1) * Wp + (t % 3 - 1); sub = 0; return; }
    // phase = 2 * (dy != 1) + (dx != 1); taps of a phase in ascending order
    int dy, dx;
    if (hf == 0) {
        if (t == 0) { dy = 1; dx = 1; sub = 0; }                               // phase 0
        else { dy = 1; dx = t == 1 ? 0 : 2; sub = 1; }                         // phase 1
    } else {
        if (t < 2) { dy = t == 0 ? 0 : 2; dx = 1; sub = 0; }                   // phase 2
        else { dy = t < 4 ? 0 : 2; dx = (t & 1) ? 2 : 0; sub = 1; }            // phase 3
    }
    tap = 3 * dy + dx;
    shift = (dy == 0 ? -Wp : 0) + (dx == 0 ? -1 : 0);
}
__host__ __device__ inline uint32_t c3_raw1_bytes(const C3Geom &g) { return (uint32_t)g.rawn * TC_KC * 4; }      // one phase's raw rows
__host__ __device__ inline uint32_t c3_raw_bytes(const C3Geom &g) { return (g.s2 ? 2u : 1u) * c3_raw1_bytes(g); }
__host__ __device__ inline uint32_t c3_kg_bytes(const C3Geom &g) { return (uint32_t)g.E * 16; }                 // one k-group of x1 or x2
__host__ __device__ inline uint32_t c3_op1_bytes(const C3Geom &g) { return 4 * c3_kg_bytes(g); }                 // x1, x2 x two k-groups
__host__ __device__ inline uint32_t c3_op_bytes(const C3Geom &g) { return (g.s2 ? 2u : 1u) * c3_op1_bytes(g); }
__host__ __device__ inline uint32_t c3_wg_bytes(const C3Geom &g) { return (g.s2 ? 6u : 9u) * C3_W_BYTES; }        // 72 or 48 KB
__host__ __device__ inline uint32_t c3_off_op(const C3Geom &g) { return (uint32_t)g.wg * c3_wg_bytes(g); }
__host__ __device__ inline uint32_t c3_off_raw(const C3Geom &g) { return c3_off_op(g) + (uint32_t)g.xs * ((c3_op_bytes(g) + 127u) & ~127u); }
__host__ __device__ inline uint32_t c3_off_epi(const C3Geom &g) { return c3_off_raw(g) + (uint32_t)g.xs * ((c3_raw_bytes(g) + 127u) & ~127u); }
__host__ __device__ inline uint32_t c3_smem_bytes(const C3Geom &g) { return c3_off_epi(g) + 8u * 2560u; }          // 8 epilogue warps x 2.5 KB

// Padded position p -> how many real pixels lie before it in the padded order (= the column of the activation matrix
// it maps to when it is a real pixel) and whether it is one. Positions outside [0, Pn) are padding.
__device__ __forceinline__ void c3_pad_map(int p, int H, int W, int Pn, int total_real, int &before, bool &real)
{
    if (p < 0) { before = 0; real = false; return; }
    if (p >= Pn) { before = total_real; real = false; return; }
    const uint32_t Wp = (uint32_t)W + 2u, HWp = ((uint32_t)H + 2u) * Wp;
    const uint32_t b = (uint32_t)p / HWp, rem = (uint32_t)p - b * HWp;
    const uint32_t yp = rem / Wp, xp = rem - yp * Wp;
    const bool inrow = yp >= 1u && yp <= (uint32_t)H;
    const uint32_t yc = yp == 0u ? 0u : (yp - 1u < (uint32_t)H ? yp - 1u : (uint32_t)H);
    const uint32_t xc = !inrow ? 0u : (xp == 0u ? 0u : (xp - 1u < (uint32_t)W ? xp - 1u : (uint32_t)W));
    before = (int)(b * (uint32_t)(H * W) + yc * (uint32_t)W + xc);
    real = inrow && xp >= 1u && xp <= (uint32_t)W;
}

// instruction descriptor: D = f32, A = B = bf16, both K-major, M = 256 (two CTAs), N = n
__device__ __forceinline__ uint32_t c3_idesc(int n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}

// the three MMAs of one (tap, channel group) step; after a group's last tap (`last_tap`) two commits hand the operand
// stage and the weight stage back to both CTAs. One elected lane of a converged warp.
__device__ __forceinline__ void c3_mma_step(uint32_t d_tmem, uint64_t dW1, uint64_t dX1, uint32_t w2_off, uint32_t x2_off,
                                            uint32_t idesc, uint32_t acc_first, uint32_t w_empty_bar, uint32_t g_empty_bar,
                                            uint32_t last_tap)
{
    asm volatile(
        "{\n\t.reg .pred pa, pt, pe, pg;\n\t.reg .b64 w2, x2;\n\t"
        "elect.sync _|pe, 0xffffffff;\n\t"
        "setp.ne.b32 pg, %9, 0;\n\t"
        "and.pred pg, pg, pe;\n\t"
        "setp.ne.b32 pa, %6, 0;\n\t"
        "setp.eq.b32 pt, %10, 0;\n\t"
        "cvt.u64.u32 w2, %3;\n\tadd.s64 w2, w2, %1;\n\t"
        "cvt.u64.u32 x2, %4;\n\tadd.s64 x2, x2, %2;\n\t"
        "@pe tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %5, pa;\n\t"
        "@pe tcgen05.mma.cta_group::2.kind::f16 [%0], w2, %2, %5, pt;\n\t"
        "@pe tcgen05.mma.cta_group::2.kind::f16 [%0], %1, x2, %5, pt;\n\t"
        "@pg tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%7], %11;\n\t"
        "@pg tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%8], %11;\n\t}"
        ::"r"(d_tmem), "l"(dW1), "l"(dX1), "r"(w2_off), "r"(x2_off), "r"(idesc), "r"(acc_first), "r"(w_empty_bar),
          "r"(g_empty_bar), "r"(last_tap), "r"(0u), "h"((uint16_t)3)
        : "memory");
}

// eight fp32 -> their bf16 heads (x1) and the bf16 of the remainders (x2), packed two per word
__device__ __forceinline__ void c3_split8(const float (&v)[8], uint4 &h, uint4 &l)
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

__device__ __forceinline__ void c3_tmem_ld16(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}

constexpr uint32_t C3_EPI_PITCH = 80;                        // bytes per staged row of 16 floats (conflict-free 16-byte writes)
constexpr uint32_t C3_EPI_STAGE = 32 * C3_EPI_PITCH;         // per warp

// Epilogue of 32 rows (lane quarter q of accumulator `acc`) x the 16-position units first, first + step, ... of one
// CTA's 128 x N part of a tile on the PADDED grid: real positions are stored at their column of the output matrix,
// padded ones dropped. A unit is read with one row per lane, turned round through `stage` (this warp's 2.5 KB of shared
// memory) and written two rows per instruction, a lane per position: the real positions of a row are neighbouring
// columns of the output, so an instruction writes up to 64 contiguous bytes in each of its two rows.
__device__ __forceinline__ void c3_epilogue(const TcArgs &a, const C3Geom &g, uint32_t acc, int q, int first, int step,
                                            int row0, int p0, int lane, uint32_t done_bar, uint32_t rank, uint8_t *stage)
{
    const int nunit = g.N / 16;
    const int total_real = (int)a.Nc;
    const int jpos = lane & 15, rsub = lane >> 4;
    // the bias of the quarter's 32 rows, one per lane, fetched once (a load per row inside the store loop made every
    // iteration wait for it)
    const int brow = row0 + q * 32 + lane;
    const float bias_l = (a.bias && brow < a.M) ? __ldg(a.bias + brow) : 0.f;
#pragma unroll 1
    for (int cc = first; cc < nunit; cc += step) {
        uint32_t r[16];
        c3_tmem_ld16(acc + ((uint32_t)(q * 32) << 16) + (uint32_t)(cc * 16), r);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        if (done_bar && cc + step >= nunit) {
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            if (lane == 0) {
                if (rank == 0) mbar_arrive(done_bar);
                else mbar_arrive_remote(done_bar, 0);
            }
        }
        // where this lane's position of the unit goes (the same for all 32 rows)
        int before; bool real;
        c3_pad_map(p0 + cc * 16 + jpos, a.H, a.W, g.Pn, total_real, before, real);
        const int col = real ? before : -1;
#pragma unroll
        for (int v = 0; v < 4; ++v)
            *reinterpret_cast<uint4 *>(stage + lane * C3_EPI_PITCH + v * 16) = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
        __syncwarp();
#pragma unroll 4
        for (int k = 0; k < 16; ++k) {                     // (every lane takes part in the shuffle)
            const int rr = 2 * k + rsub;
            const int row = row0 + q * 32 + rr;
            const float bv = __shfl_sync(0xffffffffu, bias_l, rr);
            if (col >= 0 && row < a.M) {
                float o = *reinterpret_cast<const float *>(stage + rr * C3_EPI_PITCH + jpos * 4) + bv;
                if (a.relu) o = fmaxf(o, 0.f);
                if (UBP_CHK_GMEM(col < total_real, a.status)) a.Y[(size_t)row * a.ldy + col] = o;
            }
        }
        __syncwarp();
    }
    if (done_bar && first >= nunit) {          // a warp with no unit of its own still owes its arrival
        if (lane == 0) {
            if (rank == 0) mbar_arrive(done_bar);
            else mbar_arrive_remote(done_bar, 0);
        }
    }
}

// The same for the LAST tile of a pair, where nothing runs beside the epilogue and the weight ring is free to stage
// in: units of 32 positions, a row of the unit per store instruction (up to 128 contiguous bytes).
constexpr uint32_t C3_EPI32_PITCH = 144;                     // bytes per staged row of 32 floats (conflict-free 16-byte writes)
constexpr uint32_t C3_EPI32_STAGE = 32 * C3_EPI32_PITCH;     // per warp
__device__ __forceinline__ void c3_epilogue32(const TcArgs &a, const C3Geom &g, uint32_t acc, int q, int first, int step,
                                              int row0, int p0, int lane, uint8_t *stage)
{
    const int nunit = (g.N + 31) / 32;
    const int total_real = (int)a.Nc;
    const int brow = row0 + q * 32 + lane;                  // (bias once per lane, as above)
    const float bias_l = (a.bias && brow < a.M) ? __ldg(a.bias + brow) : 0.f;
#pragma unroll 1
    for (int cc = first; cc < nunit; cc += step) {
        uint32_t r[32];
        tmem_ld32(acc + ((uint32_t)(q * 32) << 16) + (uint32_t)(cc * 32), r);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        int before; bool real;
        c3_pad_map(p0 + cc * 32 + lane, a.H, a.W, g.Pn, total_real, before, real);
        const int col = (real && cc * 32 + lane < g.N) ? before : -1;
#pragma unroll
        for (int v = 0; v < 8; ++v)
            *reinterpret_cast<uint4 *>(stage + lane * C3_EPI32_PITCH + v * 16) = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
        __syncwarp();
        // The unit's real positions are consecutive output columns. Where that run starts at an even column (always so
        // for even image widths whose padded rows divide the unit: 14 x 14), a lane takes a PAIR of columns of one of
        // two rows and writes 8 bytes: half as many store instructions, each of which the memory system makes wait.
        const uint32_t mask = __ballot_sync(0xffffffffu, col >= 0);
        const int nreal = __popc(mask);
        const int c0 = __shfl_sync(0xffffffffu, col, mask ? __ffs(mask) - 1 : 0);
        if (mask != 0u && (c0 & 1) == 0 && (a.ldy & 1) == 0) {
            const int rs = lane >> 4, m = lane & 15;
            const int s0 = 2 * m < nreal ? (int)__fns(mask, 0, 2 * m + 1) : -1;          // lanes (positions) of my two columns
            const int s1 = 2 * m + 1 < nreal ? (int)__fns(mask, 0, 2 * m + 2) : -1;
#pragma unroll 4
            for (int k = 0; k < 16; ++k) {
                const int rr = 2 * k + rs;
                const int row = row0 + q * 32 + rr;
                const float bv = __shfl_sync(0xffffffffu, bias_l, rr);
                if (s0 >= 0 && row < a.M) {
                    float o0 = *reinterpret_cast<const float *>(stage + rr * C3_EPI32_PITCH + s0 * 4) + bv;
                    float o1 = s1 >= 0 ? *reinterpret_cast<const float *>(stage + rr * C3_EPI32_PITCH + s1 * 4) + bv : 0.f;
                    if (a.relu) { o0 = fmaxf(o0, 0.f); o1 = fmaxf(o1, 0.f); }
                    float *dst = a.Y + (size_t)row * a.ldy + c0 + 2 * m;
                    if (UBP_CHK_GMEM(c0 + 2 * m < total_real, a.status)) {
                        if (s1 >= 0) *reinterpret_cast<float2 *>(dst) = make_float2(o0, o1);
                        else *dst = o0;
                    }
                }
            }
        } else {
#pragma unroll 4
            for (int rr = 0; rr < 32; ++rr) {              // (every lane takes part in the shuffle)
                const int row = row0 + q * 32 + rr;
                const float bv = __shfl_sync(0xffffffffu, bias_l, rr);
                if (col >= 0 && row < a.M) {
                    float o = *reinterpret_cast<const float *>(stage + rr * C3_EPI32_PITCH + lane * 4) + bv;
                    if (a.relu) o = fmaxf(o, 0.f);
                    if (UBP_CHK_GMEM(col < total_real, a.status)) a.Y[(size_t)row * a.ldy + col] = o;
                }
            }
        }
        __syncwarp();
    }
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(C3_THREADS, 1)
ubp_conv3_kernel(const uint8_t *__restrict__ W16, const __grid_constant__ CUtensorMap tmX, const TcArgs a, const C3Geom g)
{
    constexpr uint32_t TMEM_COLS = 2 * C3_ACC_COLS;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    // identical layout in both CTAs: the multicast commits and the remote arrives address barriers by offset
    __shared__ __align__(8) uint64_t raw_full[C3_MAX_XS], raw_empty[C3_MAX_XS], g_full[C3_MAX_XS], g_empty[C3_MAX_XS],
        wg_full[C3_MAX_WG], wg_empty[C3_MAX_WG], acc_full[2], acc_empty[2], bar_last;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();
    const int N = g.N, NH = N / 2, Wp = a.W + 2, XS = g.xs, WG = g.wg;
    const uint32_t wg_bytes = c3_wg_bytes(g);
    const int total_real = (int)a.Nc;
    const uint32_t kgb = c3_kg_bytes(g), op_stride = (c3_op_bytes(g) + 127u) & ~127u, raw_stride = (c3_raw_bytes(g) + 127u) & ~127u;
    const uint32_t off_op = c3_off_op(g), off_raw = c3_off_raw(g);
    const int npairs = (int)(gridDim.x >> 1), pair = (int)(blockIdx.x >> 1);
    const int nmy = pair < g.ntiles ? (g.ntiles - pair + npairs - 1) / npairs : 0;
    const int nchunk = 9 * g.cg;
    const int GT = g.s2 ? 2 * g.cg : g.cg;                 // group steps per tile: channel groups (x two phase pairs)
    const int NSUB = g.s2 ? 2 : 1;                         // phases (raw blocks, operands) per stage
    const uint32_t raw1 = c3_raw1_bytes(g), op1 = c3_op1_bytes(g);
    const int G = nmy * GT;                                // group steps of this pair
    const int Cin = g.cg * TC_KC;
    auto tile_row0 = [&](int i) { return (((pair + i * npairs) % g.nrp) * 2 + (int)rank) * 128; };
    auto tile_p0 = [&](int i) { return ((pair + i * npairs) / g.nrp) * N; };
    // first staged padded position of this CTA for tile i, and the (4-aligned) first real pixel its raw copy holds
    auto tile_qa = [&](int i) { return tile_p0(i) + (int)rank * NH - g.halo; };
    auto tile_ra = [&](int i) {
        int before; bool real;
        c3_pad_map(tile_qa(i) < 0 ? 0 : tile_qa(i), a.H, a.W, g.Pn, total_real, before, real);
        return before & ~3;
    };

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (threadIdx.x == 0) {
        prefetch_tensormap(&tmX);
        abort_flag = 0;
        for (int s = 0; s < XS; ++s) {
            mbar_init(smem_u32(&raw_full[s]), 1);
            mbar_init(smem_u32(&raw_empty[s]), C3_PASS_WARPS);
            mbar_init(smem_u32(&g_full[s]), 2 * C3_PASS_WARPS);          // used in the leader CTA only
            mbar_init(smem_u32(&g_empty[s]), 1);
        }
        for (int s = 0; s < g.wg; ++s) {
            mbar_init(smem_u32(&wg_full[s]), 1);
            mbar_init(smem_u32(&wg_empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&acc_full[b]), 1);
            mbar_init(smem_u32(&acc_empty[b]), 2 * C3_EPI_WARPS);        // used in the leader CTA only
        }
        mbar_init(smem_u32(&bar_last), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    // Cluster barrier, first half: every thread arrives once its CTA's barriers exist (thread 0: after it has
    // initialised them); the wait comes after the wait for the earlier kernel, when the other CTA has normally arrived
    // long ago, so the barrier's round trip is off the path.
    asm volatile("barrier.cluster.arrive.release;" ::: "memory");
    if (warp == 1) {   // tensor memory of the pair: the same warp of both CTAs allocates
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");     // every thread: nothing below may overtake the earlier kernel
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("barrier.cluster.wait.acquire;" ::: "memory");   // both CTAs' barriers exist before anyone signals them
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_slot;

    bool ok = true;
    if (warp == 0) {
        // ---------------- weight producer: the taps of a group step as ONE barrier phase (up to nine bulk copies), as far
        // ahead as the ring has stages. (The raw rows have a producer of their own, warp 2: a single thread that
        // served both rings issued a step's weights only after the previous step's had landed.)
        if (lane == 0) {
            for (int gs = 0; gs < G && ok; ++gs) {
                const int i = gs / GT, gl = gs % GT;
                const int chg = g.s2 ? gl >> 1 : gl, ph = g.s2 ? gl & 1 : 0, nt = c3_ntaps(g.s2, ph);
                const uint8_t *wrow = W16 + (size_t)(tile_row0(i) / 128) * nchunk * C3_W_BYTES;
                const int s = gs % WG, use = gs / WG;
                if (use > 0) ok = mbar_wait_relaxed(smem_u32(&wg_empty[s]), (uint32_t)(use - 1) & 1u, &abort_flag);
                if (!ok) break;
                const uint32_t bar = smem_u32(&wg_full[s]);
                mbar_expect_tx(bar, (uint32_t)nt * C3_W_BYTES);
                for (int t = 0; t < nt; ++t) {
                    int tap, shift, sub;
                    c3_tap(g.s2, ph, t, Wp, tap, shift, sub);
                    bulk_load(smem_u32(smem + (size_t)s * wg_bytes + (size_t)t * C3_W_BYTES),
                              wrow + (size_t)(tap * g.cg + chg) * C3_W_BYTES, C3_W_BYTES, bar);
                }
            }
        }
    } else if (warp == 1) {
        if (rank == 0) {
            // ---------------- leader: MMA issuer for the pair (whole warp converged, one elected lane issues)
            const uint32_t idesc = c3_idesc(N);
            int gs = 0;
            for (int i = 0; i < nmy && ok; ++i) {
                const int b = i & 1;
                const uint32_t acc = tmem_base + (uint32_t)b * C3_ACC_COLS;
                if (i >= 2) {                              // the epilogue of tile i - 2 must have read this accumulator
                    ok = mbar_wait(smem_u32(&acc_empty[b]), (uint32_t)((i >> 1) - 1) & 1u, &abort_flag);
                    if (!ok) break;
                }
                for (int gl = 0; gl < GT && ok; ++gl, ++gs) {
                    // the operand of the group is built in both CTAs and both have the group's weights
                    const int xs = gs % XS, wgs = gs % WG;
                    ok = mbar_wait(smem_u32(&g_full[xs]), (uint32_t)(gs / XS) & 1u, &abort_flag);
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t op = smem_u32(smem + off_op + (size_t)xs * op_stride);
                    const uint32_t wb = smem_u32(smem + (size_t)wgs * wg_bytes);
                    const int ph = g.s2 ? gl & 1 : 0, nt = c3_ntaps(g.s2, ph);
#pragma unroll 3
                    for (int t = 0; t < nt; ++t) {
                        int tap, shift, sub;
                        c3_tap(g.s2, ph, t, Wp, tap, shift, sub);
                        const uint64_t dW = make_desc(wb + (uint32_t)t * C3_W_BYTES, 16, 256, C3_SWZ_32B);
                        const uint64_t dX = make_desc(op + (uint32_t)sub * op1 + (uint32_t)(g.halo + shift) * 16u, kgb, 128, SWZ_NONE);
                        c3_mma_step(acc, dW, dX, (C3_W_BYTES / 2) >> 4, (2 * kgb) >> 4, idesc, (gl | t) ? 1u : 0u,
                                    smem_u32(&wg_empty[wgs]), smem_u32(&g_empty[xs]), t == nt - 1 ? 1u : 0u);
                    }
                }
                if (!ok) break;
                mma2_commit_both(smem_u32(&acc_full[b]));         // accumulator complete: epilogue warps of both CTAs
                if (i == nmy - 1) mma2_commit_both(smem_u32(&bar_last));
            }
        }
    } else if (warp == 2) {
        // ---------------- raw-row producer: one TMA copy per group step (16 channel rows of the real pixels the CTA's
        // staged positions cover), XS steps ahead
        if (lane == 0) {
            for (int r = 0; r < G && ok; ++r) {
                const int xs = r % XS, use = r / XS;
                if (use > 0) ok = mbar_wait_relaxed(smem_u32(&raw_empty[xs]), (uint32_t)(use - 1) & 1u, &abort_flag);
                if (!ok) break;
                const uint32_t bar = smem_u32(&raw_full[xs]);
                mbar_expect_tx(bar, c3_raw_bytes(g));
                const int rl = r % GT;                     // group step inside its tile
                for (int sub = 0; sub < NSUB; ++sub)       // stride 2: rows of phase 2 (rl & 1) + sub, channel group rl >> 1
                    tma_load_2d(smem_u32(smem + off_raw + (size_t)xs * raw_stride + (size_t)sub * raw1), &tmX, tile_ra(r / GT),
                                g.s2 ? (2 * (rl & 1) + sub) * Cin + (rl >> 1) * TC_KC : rl * TC_KC, bar);
            }
        }
    } else if (warp < C3_FIRST_EPI) {
        // ---------------- operand pass: once per channel group, raw fp32 rows of the real pixels -> x1, x2 (bf16) for
        // every staged padded position, K-major without swizzle: [x1 k-group 0][x1 k-group 1][x2 0][x2 1], position e of
        // a k-group at e * 16 bytes. Thread = (k-group, positions l and l + 128).
        const int pt = (int)threadIdx.x - C3_FIRST_PASS * 32;
        const int kg = pt >> 7, l = pt & 127;
        int src[2] = {-1, -1};
        int cur_tile = -1;
        for (int gs = 0; gs < G && ok; ++gs) {
            const int i = gs / GT;
            if (i != cur_tile) {                           // new tile: where in the raw copy each of my positions comes from
                cur_tile = i;
                const int qa = tile_qa(i), ra = tile_ra(i);
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int e = l + 128 * u;
                    int before; bool real;
                    c3_pad_map(qa + e, a.H, a.W, g.Pn, total_real, before, real);
                    src[u] = (e < g.E && real) ? before - ra : -1;
                }
            }
            const int xs = gs % XS, use = gs / XS;
            ok = mbar_wait_relaxed(smem_u32(&raw_full[xs]), (uint32_t)use & 1u, &abort_flag);
            if (ok && use > 0) ok = mbar_wait_relaxed(smem_u32(&g_empty[xs]), (uint32_t)(use - 1) & 1u, &abort_flag);
            if (!ok) break;
            for (int sub = 0; sub < NSUB; ++sub) {
            const float *raw = reinterpret_cast<const float *>(smem + off_raw + (size_t)xs * raw_stride + (size_t)sub * raw1) + (size_t)(kg * 8) * g.rawn;
            uint8_t *x1 = smem + off_op + (size_t)xs * op_stride + (size_t)sub * op1 + (size_t)kg * kgb;
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int e = l + 128 * u;
                if (e >= g.E) break;
                // (checked build: the source column lies in the raw copy, the stage inside the CTA's shared memory)
                if (!UBP_CHK_SMEM(src[u] < g.rawn && (size_t)(smem - smem_raw) + off_op + (size_t)(xs + 1) * op_stride <= tc::dbg_dynamic_smem() &&
                                  (size_t)(smem - smem_raw) + off_raw + (size_t)xs * raw_stride + c3_raw_bytes(g) <= tc::dbg_dynamic_smem(), a.status)) break;
                float v[8];
#pragma unroll
                for (int c = 0; c < 8; ++c) v[c] = src[u] >= 0 ? raw[(size_t)c * g.rawn + src[u]] : 0.f;
                uint4 h, lo;
                c3_split8(v, h, lo);
                *reinterpret_cast<uint4 *>(x1 + (size_t)e * 16) = h;
                *reinterpret_cast<uint4 *>(x1 + 2 * kgb + (size_t)e * 16) = lo;
            }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // make the writes visible to the MMA unit
            // this CTA's weights of the group must have landed too before the leader may issue the group's MMAs
            ok = mbar_wait_relaxed(smem_u32(&wg_full[gs % WG]), (uint32_t)(gs / WG) & 1u, &abort_flag);
            if (!ok) break;
            __syncwarp();
            if (lane == 0) {
                if (rank == 0) mbar_arrive(smem_u32(&g_full[xs]));
                else mbar_arrive_remote(smem_u32(&g_full[xs]), 0);
                mbar_arrive(smem_u32(&raw_empty[xs]));
            }
        }
        // ---------------- the last tile has nothing to overlap with: take the units 2, 3, 6, 7, ... of its epilogue.
        // Its own barrier (one phase) rather than the accumulator's, whose earlier phases these warps did not see; the
        // weight stages are free by then (every MMA has completed) and serve as these warps' staging memory.
        if (ok && nmy > 0) ok = mbar_wait_relaxed(smem_u32(&bar_last), 0, &abort_flag);
        if (ok && nmy > 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int i = nmy - 1;
            c3_epilogue32(a, g, tmem_base + (uint32_t)(i & 1) * C3_ACC_COLS, warp & 3, 2 + ((warp - C3_FIRST_PASS) >> 2), 4,
                          tile_row0(i), tile_p0(i), lane, smem + (size_t)(8 + warp - C3_FIRST_PASS) * C3_EPI32_STAGE);
        }
    } else {
        // ---------------- epilogue warps: tile i's accumulator while the main loop works on tile i + 1
        const int part = (warp - C3_FIRST_EPI) >> 2;          // two warps share a lane quarter and split the units
        for (int i = 0; i < nmy && ok; ++i) {
            const int b = i & 1;
            ok = mbar_wait_relaxed(smem_u32(&acc_full[b]), (uint32_t)(i >> 1) & 1u, &abort_flag);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (i == nmy - 1)       // the weight ring is free by now (every MMA has completed): stage the last tile there
                c3_epilogue32(a, g, tmem_base + (uint32_t)b * C3_ACC_COLS, warp & 3, part, 4, tile_row0(i), tile_p0(i), lane,
                              smem + (size_t)(warp - C3_FIRST_EPI) * C3_EPI32_STAGE);
            else
                c3_epilogue(a, g, tmem_base + (uint32_t)b * C3_ACC_COLS, warp & 3, part, 2, tile_row0(i), tile_p0(i), lane,
                            smem_u32(&acc_empty[b]), rank, smem + c3_off_epi(g) + (size_t)(warp - C3_FIRST_EPI) * C3_EPI_STAGE);
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

// Tile width for a launch: the padded positions per tile (a multiple of 16) that gives the pairs the fewest, cheapest
// rounds. A step (tap, channel group) costs its three MMAs (about 1.6 cycles per position) or, for narrow tiles, what
// the copy of its 8 KB of weights needs at the L2 -> SM rate (about 260 cycles); a tile adds its epilogue.
static bool c3_geometry(int M, int C, int B, int H, int W, int sms, int s2, C3Geom *out)
{
    if (C % TC_KC != 0 || M <= 128) return false;
    const long long Pn = (long long)B * (H + 2) * (W + 2);
    if (Pn >= (1ll << 30) || (long long)B * H * W >= (1ll << 30)) return false;
    C3Geom best{};
    double best_cost = 1e300;
    const int pairs_max = sms / 2;
    for (int n = 256; n >= 64; n -= 16) {
        C3Geom g{};
        g.N = n; g.halo = W + 3; g.cg = C / TC_KC; g.Pn = (int)Pn; g.nrp = (M + 255) / 256; g.s2 = s2;
        g.E = (n / 2 + 2 * g.halo + 7) & ~7;
        if (g.E > 256) continue;
        g.rawn = (g.E + 4 + 3) & ~3;
        if (g.rawn > 256) continue;                         // TMA box limit
        const long long tiles = (long long)g.nrp * ((Pn + n - 1) / n);
        if (tiles > 0x7fffffffll) continue;
        g.ntiles = (int)tiles;
        // stride 2 has twice the group steps with half the MMAs each: deeper rings hide the hand-offs
        g.wg = 2;
        g.xs = s2 ? 4 : 3;
        while (g.xs > 2 && c3_smem_bytes(g) > 224u * 1024u) --g.xs;
        if (c3_smem_bytes(g) > 224u * 1024u) continue;
        const long long pairs = tiles < pairs_max ? tiles : pairs_max;
        const long long rounds = (tiles + pairs - 1) / pairs;
        const double step = 1.6 * n > 260.0 ? 1.6 * n : 260.0;      // three MMAs, or the 8 KB of weights at the L2 -> SM rate
        const double cost = (double)rounds * (9.0 * g.cg * step + 25.0 * n + 2500.0);
        if (cost < best_cost) { best_cost = cost; best = g; }
    }
    if (best_cost == 1e300) return false;
    *out = best;
    return true;
}

// Which tile the padded-grid kernel would use for this layer (false: it cannot take it).
bool conv3_pair_tile(int M, int C, int B, int H, int W, int sms, int *tile_cols)
{
    C3Geom g;
    if (!c3_geometry(M, C, B, H, W, sms, 0, &g)) return false;
    if (tile_cols) *tile_cols = g.N;
    return true;
}

// Launch on tiles of 256 rows x N padded positions. X: the input as one [C][B*H*W] matrix (rows 16-byte aligned, row
// stride isc floats); s2: X is instead the four phase planes of a stride-2 layer, [4*C][B*H*W] with H x W the OUTPUT
// plane (launch_phase_planes below writes them), and a.H, a.W, a.Nc describe that plane; W16: the plan's bf16 part (8 KB blocks [128-row tile][chunk = tap * C/16 + group]).
// Returns UBP_E_UNSUPPORTED when the layer does not fit this kernel (the caller then uses the per-tap kernel).
int launch_conv3_pair(const void *W16, const float *X, int64_t isc, const void *args_, int M, int C, int B, int H, int W,
                      int sms, void *stream, int s2)
{
    C3Geom g;
    if (!c3_geometry(M, C, B, H, W, sms, s2, &g)) return UBP_E_UNSUPPORTED;
    TcArgs a = *static_cast<const TcArgs *>(args_);
    a.ntile = g.N;
    typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                      const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                      CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeTiledFn enc = nullptr;
    if (!enc) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess) return UBP_E_CUDA;
        enc = reinterpret_cast<EncodeTiledFn>(p);
    }
    CUtensorMap tmX;
    const cuuint64_t dims[2] = {(cuuint64_t)a.Nc, (cuuint64_t)(s2 ? 4 * C : C)};
    const cuuint64_t strides[1] = {(cuuint64_t)isc * 4};
    const cuuint32_t box[2] = {(cuuint32_t)g.rawn, TC_KC};
    const cuuint32_t estr[2] = {1, 1};
    CUresult cr = enc(&tmX, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float *>(X), dims, strides, box, estr,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) { set_last_cuda_error(-(int)cr); return UBP_E_CUDA; }
    size_t smem = (size_t)c3_smem_bytes(g) + 1024;
    if (smem < TC_PAIR_MIN_SMEM) smem = TC_PAIR_MIN_SMEM;   // one CTA per SM, whatever the tile width (see the constant)
    static bool done[64] = {};
    int devid = 0;
    if (cudaGetDevice(&devid) != cudaSuccess) devid = -1;
    if (devid < 0 || devid >= 64 || !done[devid]) {
        cudaError_t e = cudaFuncSetAttribute(ubp_conv3_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 226 * 1024);
        if (e != cudaSuccess) { set_last_cuda_error((int)e); return UBP_E_CUDA; }
        int per_sm = 0;                                     // a query, nothing is launched
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, ubp_conv3_kernel, C3_THREADS, TC_PAIR_MIN_SMEM);
        if (e != cudaSuccess) { set_last_cuda_error((int)e); return UBP_E_CUDA; }
        if (per_sm != 1) return UBP_E_UNSUPPORTED;
        if (devid >= 0 && devid < 64) done[devid] = true;
    }
    const long long pairs = g.ntiles < sms / 2 ? g.ntiles : sms / 2;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * pairs));
    cfg.blockDim = dim3(C3_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, ubp_conv3_kernel, static_cast<const uint8_t *>(W16), tmX, a, g);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) { set_last_cuda_error((int)e); return UBP_E_CUDA; }
    return UBP_OK;
}

// Stride 2: the four phase planes of the input, P[2 py + px][c][b][yo][xo] = in[b][c][2 yo + py][2 xo + px] (zero
// outside the image), as a matrix of 4*C rows of `ld` floats: on them every tap of the strided 3x3 is a shift of 0 or
// -1 of one plane.
// One CTA per (four channels, image), no shared memory: a thread takes the pixel pair (y, 2 xo), (y, 2 xo + 1) of
// each of the four planes (eight independent loads in flight) and writes them to phases 2 (y & 1) and 2 (y & 1) + 1 at
// (y / 2, xo): reads and writes run along the image rows. (A CTA per plane that went through shared memory spent its
// time on the load -> barrier -> store latency of 8192 tiny CTAs: 28 us for 51 MB.)
constexpr int PP_CH = 4;
__global__ void __launch_bounds__(256) ubp_phase_planes_kernel(const float *__restrict__ in, int C, int B, int H, int Wd,
                                                                int64_t isb, int64_t isc, int Ho, int Wo, int64_t ld,
                                                                float *__restrict__ out)
{
    const int c0 = (int)blockIdx.x * PP_CH, b = blockIdx.y;
    const int items = 2 * Ho * Wo, ohw = Ho * Wo;
    const float *src = in + (size_t)b * isb + (size_t)c0 * isc;
    for (int i = threadIdx.x; i < items; i += 256) {
        const int y = i / Wo, xo = i - y * Wo;
        const int x = 2 * xo;
        const bool in0 = y < H, in1 = in0 && x + 1 < Wd;
        float v0[PP_CH], v1[PP_CH];
#pragma unroll
        for (int k = 0; k < PP_CH; ++k) {
            const bool ch = c0 + k < C;
            const float *p = src + (size_t)k * isc + (size_t)y * Wd + x;
            v0[k] = (ch && in0) ? __ldg(p) : 0.f;
            v1[k] = (ch && in1) ? __ldg(p + 1) : 0.f;
        }
        const int ph = (y & 1) * 2;
        const size_t o = (size_t)b * ohw + (size_t)(y >> 1) * Wo + xo;
#pragma unroll
        for (int k = 0; k < PP_CH; ++k) {
            if (c0 + k >= C) break;
            out[((size_t)ph * C + c0 + k) * ld + o] = v0[k];
            out[((size_t)(ph + 1) * C + c0 + k) * ld + o] = v1[k];
        }
    }
}

int launch_phase_planes(const float *in, int C, int B, int H, int Wd, int64_t isb, int64_t isc, float *out, int64_t ld,
                        void *stream)
{
    const int Ho = (H - 1) / 2 + 1, Wo = (Wd - 1) / 2 + 1;
    if (B == 0 || C == 0) return UBP_OK;
    if (B > 65535 || (int64_t)2 * Ho * Wo >= (1ll << 30)) return UBP_E_UNSUPPORTED;
    ubp_phase_planes_kernel<<<dim3((unsigned)((C + PP_CH - 1) / PP_CH), (unsigned)B), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        in, C, B, H, Wd, isb, isc, Ho, Wo, ld, out);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_last_cuda_error((int)e); return UBP_E_CUDA; }
    return UBP_OK;
}

}  // namespace ubp

