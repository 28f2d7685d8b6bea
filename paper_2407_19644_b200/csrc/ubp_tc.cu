// Tensor-core variant of the 1x1 product: the block-row panels are densified
// (the masked weight as a plain M x K matrix) and the product runs on the
// tcgen05 tensor cores in TF32 with a three-term split that keeps fp32 accuracy:
//     W = Wh + Wl,  X = Xh + Xl   (h = top 19 bits, l = remainder)
//     W X ~= Wh Xh + Wl Xh + Wh Xl          (the dropped Wl Xl term is ~2^-20 |w||x|)
// all three accumulated in fp32 in tensor memory. It does 3 / density times the
// multiply-adds of the sparse kernel but on a unit ~15x faster than the FP32
// pipes, so it wins at low and moderate sparsity; the sparse SIMT kernel wins
// when few blocks survive. Which one runs is the plan's choice (variant).
//
// CTA tile: (128 * MT) output rows x 256 columns; K is walked in chunks of 16.
// Warp roles: warp 0 issues TMA copies of the Wh / Wl chunks from the plan;
// warps 2-17 read the X chunk from global memory (one column and 8 channels per
// thread, coalesced across the warp), split it into Xh and Xl and write both transposed
// into shared memory (the tensor core wants both operands with the reduction
// index contiguous); warp 1 issues the MMAs (one thread) and owns tensor memory;
// then warps 2-17 read the accumulators back (tcgen05.ld), add bias, apply ReLU
// and store. Operand layouts: W is K-major with the 64-byte swizzle (rows of 16
// floats, exactly what TMA writes for a 16 x 128 box); X is K-major without
// swizzle (8-column x 4-channel core matrices of 128 contiguous bytes).
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "ubp_internal.h"
#include "ubp_tc_common.cuh"

namespace ubp {

namespace {

using namespace tc;

constexpr int TC_N = 256;          // columns per CTA
constexpr int TC_SPLIT_WARPS = 16; // warps 2..17 transpose/split X and run the epilogue
constexpr int TC_THREADS = (2 + TC_SPLIT_WARPS) * 32;
constexpr uint32_t A_HALF_BYTES = 128 * TC_KC * 4;          // one 128-row chunk of Wh or Wl: 8 KB
constexpr uint32_t B_BYTES = TC_KC * TC_N * 4;              // Xh or Xl chunk: 16 KB
constexpr uint32_t B_LBO = 128;                             // next 4 channels of the same 8 columns
constexpr uint32_t B_SBO = (TC_KC / 4) * 128;               // next 8 columns: 512 B


template <int MT>
__global__ void __launch_bounds__(TC_THREADS, 1)
ubp_tc_kernel(const __grid_constant__ CUtensorMap tmWh, const __grid_constant__ CUtensorMap tmWl, const TcArgs a)
{
    constexpr uint32_t A_BYTES = MT * 2 * A_HALF_BYTES;                 // [half][hi, lo]
    constexpr uint32_t STAGE_BYTES = A_BYTES + 2 * B_BYTES;             // + Xh + Xl
    constexpr int S = (MT == 2) ? 3 : 4;
    constexpr uint32_t TMEM_COLS = MT * TC_N;                           // 256 or 512

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    // the swizzled operand tiles need 1024-byte aligned bases: round the dynamic window up ourselves
    uint8_t *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    __shared__ __align__(8) uint64_t bar_full[S], bar_ready[S], bar_empty[S], bar_acc;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row0 = blockIdx.x * (128 * MT);
    const int64_t col0 = (int64_t)blockIdx.y * a.ntile;
    const int nchunk = (a.K + TC_KC - 1) / TC_KC;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < S; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_ready[s]), TC_SPLIT_WARPS);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        mbar_init(smem_u32(&bar_acc), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {   // tensor memory: the whole warp allocates, the address lands in shared memory
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_slot;

    bool ok = true;
    if (warp == 0) {
        // ---------------- TMA producer: Wh / Wl chunks of this row tile
        if (lane == 0) {
            for (int c = 0; c < nchunk && ok; ++c) {
                const int st = c % S;
                if (c >= S) ok = mbar_wait_relaxed(smem_u32(&bar_empty[st]), ((c / S) - 1) & 1, &abort_flag);
                if (!ok) break;
                uint8_t *stage = smem + (size_t)st * STAGE_BYTES;
                const uint32_t bar = smem_u32(&bar_full[st]);
                mbar_expect_tx(bar, A_BYTES);
#pragma unroll
                for (int h = 0; h < MT; ++h) {
                    tma_load_2d(smem_u32(stage + (2 * h) * A_HALF_BYTES), &tmWh, c * TC_KC, row0 + h * 128, bar);
                    tma_load_2d(smem_u32(stage + (2 * h + 1) * A_HALF_BYTES), &tmWl, c * TC_KC, row0 + h * 128, bar);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (one thread)
        if (lane == 0) {
            const uint32_t kIdesc = make_idesc(a.ntile);
            // W: K-major, 64-byte rows, 8-row groups 512 B apart (64-byte swizzle);
            // X: K-major core matrices of 8 columns x 4 channels (128 B), next 4 channels +128 B, next 8 columns +512 B
            const uint64_t dWh0 = make_desc(smem_u32(smem), 16, 512, SWZ_64B);
            const uint64_t dXh0 = make_desc(smem_u32(smem) + A_BYTES, B_LBO, B_SBO, SWZ_NONE);
            for (int c = 0; c < nchunk && ok; ++c) {
                const int st = c % S;
                ok = mbar_wait(smem_u32(&bar_full[st]), (c / S) & 1, &abort_flag) &&
                     mbar_wait(smem_u32(&bar_ready[st]), (c / S) & 1, &abort_flag);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                // descriptors of this stage = descriptors of stage 0 + the stage offset in the address field
                // (16-byte units; shared-memory addresses stay below 2^18, so the 14-bit field never carries)
                const uint64_t soff = (uint64_t)((uint32_t)st * (STAGE_BYTES >> 4));
#pragma unroll
                for (int h = 0; h < MT; ++h) {
                    const uint32_t d = tmem_base + h * TC_N;
#pragma unroll
                    for (int ks = 0; ks < TC_KC / 8; ++ks) {
                        // W: 8 channels further = +32 B (2 units); X: 8 channels further = +256 B (16 units)
                        const uint64_t dWh = dWh0 + soff + (uint64_t)(h * (2 * A_HALF_BYTES >> 4) + ks * 2);
                        const uint64_t dWl = dWh + (A_HALF_BYTES >> 4);
                        const uint64_t dXh = dXh0 + soff + (uint64_t)(ks * 16);
                        const uint64_t dXl = dXh + (B_BYTES >> 4);
                        mma_tf32(d, dWh, dXh, kIdesc, (c > 0 || ks > 0) ? 1u : 0u);
                        mma_tf32(d, dWl, dXh, kIdesc, 1u);
                        mma_tf32(d, dWh, dXl, kIdesc, 1u);
                    }
                }
                mma_commit(smem_u32(&bar_empty[st]));       // stage may be refilled once these MMAs have read it
            }
            if (ok) mma_commit(smem_u32(&bar_acc));          // accumulators complete
        }
    } else {
        // ---------------- warps 2-17: X chunk from global memory -> Xh, Xl transposed into the stage
        const int t = (threadIdx.x - 64) & 255;              // column col0 + t of the tile
        const int kh = (threadIdx.x - 64) >> 8;              // which 8 of the chunk's 16 channels
        constexpr int KH = TC_KC / 2;
        constexpr int PD = 3;                                // chunks of X in flight in registers (covers L2 latency)
        float xr[PD][KH];
        const bool col_live = t < a.ntile && col0 + t < a.Nc;
        const float *xcol = a.X + (col_live ? col0 + t : 0) + (size_t)kh * KH * a.ldx;
        // 3x3: this thread's output pixel and which of its nine taps fall inside the image
        const float *pix_base = a.X;
        uint32_t tap_ok = 0;
        if (a.conv && col_live) {
            const int64_t n = col0 + t;
            const int sd = a.stride > 1 ? a.stride : 1;
            const int Ho = (a.H - 1) / sd + 1, Wo = (a.W - 1) / sd + 1;
            const int hw = Ho * Wo;
            const int b = (int)(n / hw), pix = (int)(n - (int64_t)b * hw);
            const int y = (pix / Wo) * sd, x = (pix % Wo) * sd;       // the input pixel under the centre tap
            pix_base = a.X + (size_t)b * a.isb + (size_t)y * a.W + x;
#pragma unroll
            for (int tp = 0; tp < 9; ++tp) {
                const int yy = y + tp / 3 - 1, xx = x + tp % 3 - 1;
                if (yy >= 0 && yy < a.H && xx >= 0 && xx < a.W) tap_ok |= 1u << tp;
            }
        }
        auto load_chunk = [&](int c, float (&dst)[KH]) {
            if (a.conv) {
                // implicit lowering: reduction index k = tap * C + channel reads the input plane in place; the
                // 8 channels of this thread normally share one tap, so tap test and offset are per chunk
                const int C = a.K / 9;
                const int k0 = c * TC_KC + kh * KH;
                int tp = k0 / C, ch = k0 - tp * C;
                if (ch + KH <= C) {
                    const bool live = tp < 9 && ((tap_ok >> tp) & 1u);
                    const float *p = pix_base + (size_t)ch * a.isc + ((tp / 3 - 1) * a.W + (tp % 3 - 1));
#pragma unroll
                    for (int i = 0; i < KH; ++i) dst[i] = live ? __ldg(p + (size_t)i * a.isc) : 0.f;
                } else {
#pragma unroll
                    for (int i = 0; i < KH; ++i) {
                        const bool live = tp < 9 && ((tap_ok >> tp) & 1u);
                        const int doff = (tp / 3 - 1) * a.W + (tp % 3 - 1);
                        dst[i] = live ? __ldg(pix_base + (size_t)ch * a.isc + doff) : 0.f;
                        if (++ch == C) { ch = 0; ++tp; }
                    }
                }
                return;
            }
            const float *p = xcol + (size_t)c * TC_KC * a.ldx;
            if (col_live && (c + 1) * TC_KC <= a.K) {
#pragma unroll
                for (int k = 0; k < KH; ++k) dst[k] = __ldg(p + (size_t)k * a.ldx);
            } else {
#pragma unroll
                for (int k = 0; k < KH; ++k)
                    dst[k] = (col_live && c * TC_KC + kh * KH + k < a.K) ? __ldg(p + (size_t)k * a.ldx) : 0.f;
            }
        };
        const uint32_t off = (uint32_t)(t & 7) * 16u + (uint32_t)(t >> 3) * B_SBO + (uint32_t)kh * (KH / 4) * B_LBO;
        auto split_chunk = [&](int c, const float (&src)[KH]) -> bool {
            const int st = c % S;
            if (c >= S && !mbar_wait_relaxed(smem_u32(&bar_empty[st]), ((c / S) - 1) & 1, &abort_flag)) return false;
            uint8_t *xh = smem + (size_t)st * STAGE_BYTES + A_BYTES + off;
            uint8_t *xl = xh + B_BYTES;
#pragma unroll
            for (int kc = 0; kc < KH / 4; ++kc) {
                float4 hi, lo;
                const float v0 = src[4 * kc], v1 = src[4 * kc + 1], v2 = src[4 * kc + 2], v3 = src[4 * kc + 3];
                hi.x = __uint_as_float(__float_as_uint(v0) & 0xffffe000u); lo.x = v0 - hi.x;
                hi.y = __uint_as_float(__float_as_uint(v1) & 0xffffe000u); lo.y = v1 - hi.y;
                hi.z = __uint_as_float(__float_as_uint(v2) & 0xffffe000u); lo.z = v2 - hi.z;
                hi.w = __uint_as_float(__float_as_uint(v3) & 0xffffe000u); lo.w = v3 - hi.w;
                *reinterpret_cast<float4 *>(xh + kc * B_LBO) = hi;
                *reinterpret_cast<float4 *>(xl + kc * B_LBO) = lo;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // make the writes visible to the MMA unit
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bar_ready[st]));
            return true;
        };
#pragma unroll
        for (int d = 0; d < PD; ++d)
            if (d < nchunk) load_chunk(d, xr[d]);
        for (int c0 = 0; c0 < nchunk && ok; c0 += PD) {
#pragma unroll
            for (int d = 0; d < PD; ++d) {
                const int c = c0 + d;
                if (c < nchunk && ok) {
                    ok = split_chunk(c, xr[d]);
                    if (c + PD < nchunk) load_chunk(c + PD, xr[d]);
                }
            }
        }
        // ---------------- epilogue: accumulators -> registers -> bias, ReLU -> global
        if (ok) ok = mbar_wait_relaxed(smem_u32(&bar_acc), 0, &abort_flag);
        if (ok) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int q = warp & 3;                           // this warp may touch tensor-memory lanes 32q .. 32q+31
            const int cpart = (warp - 2) >> 2;                // four warps share a lane group and split the columns
            // Each 32 x 32 block goes registers -> shared memory (row per lane, 144-byte pitch) -> registers with
            // 8 lanes per row, so that every store instruction writes four complete 128-byte row segments.
            // The pipeline stages are idle by now (all MMAs have completed), so their memory is reused.
            constexpr int PITCH = 36;                         // floats
            float *tile = reinterpret_cast<float *>(smem) + (warp - 2) * 32 * PITCH;
            const int sub_row = lane >> 3, sub_col = (lane & 7) * 4;
#pragma unroll 1
            for (int h = 0; h < MT; ++h) {
                const int rbase = row0 + h * 128 + q * 32;
#pragma unroll 1
                for (int cc = cpart; cc < a.ntile / 32; cc += TC_SPLIT_WARPS / 4) {
                    uint32_t r[32];
                    tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(h * TC_N + cc * 32), r);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int v = 0; v < 8; ++v)
                        *reinterpret_cast<float4 *>(tile + lane * PITCH + 4 * v) =
                            make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]),
                                        __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3]));
                    __syncwarp();
                    const int64_t col = col0 + cc * 32 + sub_col;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int rr = i * 4 + sub_row;
                        const int row = rbase + rr;
                        float4 o = *reinterpret_cast<const float4 *>(tile + rr * PITCH + sub_col);
                        if (row < a.M) {
                            const float b = a.bias ? __ldg(a.bias + row) : 0.f;
                            o.x += b; o.y += b; o.z += b; o.w += b;
                            if (a.relu) { o.x = fmaxf(o.x, 0.f); o.y = fmaxf(o.y, 0.f); o.z = fmaxf(o.z, 0.f); o.w = fmaxf(o.w, 0.f); }
                            float *yrow = a.Y + (size_t)row * a.ldy;
                            if (col + 3 < a.Nc) {
                                *reinterpret_cast<float4 *>(yrow + col) = o;
                            } else {
                                if (col < a.Nc) yrow[col] = o.x;
                                if (col + 1 < a.Nc) yrow[col + 1] = o.y;
                                if (col + 2 < a.Nc) yrow[col + 2] = o.z;
                            }
                        }
                    }
                    __syncwarp();
                }
            }
        }
    }
    if (!ok && lane == 0) atomicExch(a.status, 1);
    // every thread comes here; tensor memory is released by the warp that allocated it
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn tc_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

int encode_2d(CUtensorMap *tm, const void *base, uint64_t inner, uint64_t outer, uint64_t row_bytes, uint32_t box_in,
              uint32_t box_out, CUtensorMapSwizzle swz)
{
    EncodeTiledFn enc = tc_encode_fn();
    if (!enc) return UBP_E_CUDA;
    const cuuint64_t dims[2] = {inner, outer};
    const cuuint64_t strides[1] = {row_bytes};
    const cuuint32_t box[2] = {box_in, box_out};
    const cuuint32_t estr[2] = {1, 1};
    CUresult cr = enc(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void *>(base), dims, strides, box, estr,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) { set_last_cuda_error(-(int)cr); return UBP_E_CUDA; }
    return UBP_OK;
}

int encode_3d(CUtensorMap *tm, const void *base, const uint64_t (&dims)[3], uint64_t stride1_bytes, uint64_t stride2_bytes,
              const uint32_t (&box)[3], CUtensorMapSwizzle swz, CUtensorMapDataType dtype = CU_TENSOR_MAP_DATA_TYPE_FLOAT32)
{
    EncodeTiledFn enc = tc_encode_fn();
    if (!enc) return UBP_E_CUDA;
    const cuuint64_t d[3] = {dims[0], dims[1], dims[2]};
    const cuuint64_t strides[2] = {stride1_bytes, stride2_bytes};
    const cuuint32_t b[3] = {box[0], box[1], box[2]};
    const cuuint32_t estr[3] = {1, 1, 1};
    CUresult cr = enc(tm, dtype, 3, const_cast<void *>(base), d, strides, b, estr,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) { set_last_cuda_error(-(int)cr); return UBP_E_CUDA; }
    return UBP_OK;
}

}  // namespace


// two-CTA kernel (ubp_tc2.cu)
int launch_tc_pair(const CUtensorMap_st *tmW, const CUtensorMap_st *tmX, int x3d, int halo, const void *args, int M,
                   int64_t Nc, int ntile, int sms, void *stream);
int tc_pair_stages(int ntile, int halo);
// same pipeline with three bf16 products per fp32 product (ubp_tc3.cu)
int launch_tc_pair_bf16(const void *W16, const CUtensorMap_st *tmX, int conv, int halo, const void *args,
                        int M, int64_t Nc, int ntile, int sms, void *stream, int pieces, int mt);
int tc_pair_bf16_stages(int ntile, int halo, int mt = 1);
int tc_pair_bf16_sub(int K, int ntile, int halo, int pieces, int mt);
int tc_pair_bf16_stages_sub(int ntile, int halo, int sub, int mt);

// Tile choice for one launch: which kernel (1 = one CTA per tile, 2 = CTA pair per tile), tile rows and columns.
// Each candidate's time is estimated as (waves over the SMs) x (chunks x cycles per chunk + a fixed per-tile cost)
// and the cheapest kept.
// conv_w: 0 = 1x1 product; > 0 = 3x3 on images `conv_w` pixels wide whose operands the pair kernel can take;
// < 0 = 3x3, one-CTA kernel only.
// bf16 != 0: the CTA-pair kernel multiplies with three bf16 products (ubp_tc3.cu) instead of three TF32 products.
void tc_choose(int M, int K, int64_t Nc, int conv_w, int bf16, int sms, int *kernel, int *rows, int *cols)
{
    const int conv = conv_w != 0;
    const int nchunk = (K + TC_KC - 1) / TC_KC;
    double best = 1e300;
    int best_mt = 1, best_n = TC_N;
    for (int mt = 1; mt <= 2; ++mt)
        for (int n = 64; n <= TC_N; n += 32) {
            const long long tiles = (long long)((M + 128 * mt - 1) / (128 * mt)) * ((Nc + n - 1) / n);
            const long long waves = (tiles + sms - 1) / sms;
            // Per 16-channel chunk: 6 MMAs per 128-row half, n/2 cycles each; shared memory carries the MMAs'
            // operand reads (4 KB of W + 32 B per column each) plus the W (TMA) and X (transposing warps) writes at
            // ~120 B/cycle; the transposing warps themselves need ~1150 cycles per chunk (1500 with two halves:
            // measured with in-kernel timers). Per tile ~6000 cycles of prologue plus an epilogue ~ its outputs.
            const double mma = mt * 3.0 * (TC_KC / 8) * (n / 2.0);
            const double smem_bytes = mt * 3.0 * (TC_KC / 8) * (4096.0 + 32.0 * n) + mt * 16384.0 + 128.0 * n;
            double per_chunk = mma > smem_bytes / 120.0 ? mma : smem_bytes / 120.0;
            const double floor_chunk = mt == 1 ? 1150.0 : 1500.0;
            if (per_chunk < floor_chunk) per_chunk = floor_chunk;
            const double t = (double)waves * (nchunk * per_chunk + 6000.0 + 40.0 * mt * n);
            if (t < best) { best = t; best_mt = mt; best_n = n; }
        }
    *kernel = 1; *rows = 128 * best_mt; *cols = best_n;
    // Two-CTA kernel for the 1x1 product (256 rows per CTA pair; X goes from global memory into the operand layout
    // by TMA, each SM holds and reads only half of the X tile; persistent, the epilogue of a tile runs under the
    // main loop of the next). Calibrated on forced tile widths: a chunk takes its MMA time (6 MMAs of n/2 cycles,
    // ~10 % more in practice) or, for narrow tiles, the time shared memory needs for it (MMA operand reads 24 KB of
    // W + 96 B per column, copies 16 KB + 32 B per column, Xl pass 64 B per column, at ~120 B/cycle: ~500 + n/2
    // cycles); a tile takes its chunks or, if longer, its epilogue on eight warps (~45 cycles per column); per
    // launch ~4400 cycles of pipeline fill and ~4500 + 30 per column of drain and last epilogue.
    // 3x3: the shifted tiles are cut from a raw copy with a halo of image width + 1 columns either side, which
    // adds shared-memory traffic (raw copy in, two reads of it, Xh and Xl out: ~560 + n cycles per chunk, measured
    // ~740 at n = 192) and leaves fewer stages.
    const int halo = conv_w > 0 ? (conv_w + 1 + 3) & ~3 : 0;
    // (layers of at most 128 rows: only the bf16 kernel, whose two CTAs then both take the one row tile and split the columns)
    if ((M > 128 || bf16) && conv_w >= 0 && (!conv || ((K / 9) % TC_KC == 0 && halo <= 64))) {
        double best2 = 1e300;
        int best2_n = 0;
        // tile widths: multiples of 64 for the TF32 kernel (X arrives in 32-column boxes per CTA), of 32 for the bf16
        // kernel here (the estimate was calibrated on those; see the refinement below)
        for (int n = 64; n <= 256; n += bf16 ? 32 : 64) {
            if (conv && (n / 2 + 2 * halo > 256 || (bf16 ? tc_pair_bf16_stages(n, halo) : tc_pair_stages(n, halo)) < 4)) continue;
            const long long ntiles = (long long)((M + 255) / 256) * ((Nc + n - 1) / n);
            const long long pairs = ntiles < sms / 2 ? ntiles : sms / 2;
            const long long per_pair = (ntiles + pairs - 1) / pairs;
            // bf16 products (calibrated the same way): three MMAs of K = 16 per chunk, n/2 cycles each; below that
            // a floor of ~470 + n/3 cycles that is nearly flat in n - the copies (W in 32-byte row pieces, the raw
            // fp32 rows) arrive at ~32 B/cycle/SM, the rate of the L2-to-SM path; 3x3: the shifted-tile pass
            // (~700 + 0.6 n). A tile costs its chunks or its epilogue (~50 cycles per column) plus ~2500 cycles of
            // hand-over between tiles.
            double per_chunk = bf16 == 2 ? 3.3 * n : (bf16 ? 1.65 * n : 3.3 * n);     // bf16 == 2: three pieces, six MMAs
            const double smem_chunk = bf16 ? (conv ? 700.0 + 0.6 * n : 470.0 + 0.33 * n) : (conv ? 560.0 + 1.0 * n : 500.0 + 0.5 * n);
            if (per_chunk < smem_chunk) per_chunk = smem_chunk;
            double per_tile = nchunk * per_chunk;
            const double epi = (bf16 ? 50.0 * n : 45.0 * n) * (M > 128 ? 1.0 : 0.5);   // <= 128 rows: half the columns per CTA
            if (per_tile < epi) per_tile = epi;
            if (bf16) per_tile += 2500.0;
            const double t = 4400.0 + (double)per_pair * per_tile + 4500.0 + 30.0 * n;
            if (t < best2) { best2 = t; best2_n = n; }
        }
        int best2_rows = 256;
        // bf16 1x1, rows in whole 512-row tiles: a pair may stack two 256-row MMA
        // tiles on one staged activation tile (one copy and one split pass serve both; a chunk then brings two weight
        // blocks and its six MMAs: measured ~585-605 cycles per chunk at 96 and 192 columns) instead of making two
        // rounds; narrow stacked tiles lose against one round of wide plain ones, which the estimate reproduces
        if (bf16 == 1 && !conv && ((M + 255) / 256) % 2 == 0) {
            for (int n = 64; n <= 256; n += 32) {
                const long long ntiles = (long long)((M + 511) / 512) * ((Nc + n - 1) / n);
                if (tc_pair_bf16_stages(n, 0, 2) < 4) continue;
                const long long pairs = ntiles < sms / 2 ? ntiles : sms / 2;
                const long long per_pair = (ntiles + pairs - 1) / pairs;
                double per_chunk = 3.3 * n;
                if (per_chunk < 600.0 + 0.33 * n) per_chunk = 600.0 + 0.33 * n;
                // (both accumulators belong to one tile: every tile's epilogue, ~100 cycles per column, is exposed)
                const double t = 4400.0 + (double)per_pair * (nchunk * per_chunk + 2500.0) + (double)(per_pair - 1) * 100.0 * n +
                                 4500.0 + 60.0 * n;
                if (t < best2) { best2 = t; best2_n = n; best2_rows = 512; }
            }
        }
        // The bf16 kernel takes widths in steps of 16 columns (the MMA's step; its epilogue works in 16-column units;
        // layers of at most 128 rows, whose CTAs halve the units between them, stay on multiples of 32): 16 columns
        // less where every pair still gets its one tile. (Offered every multiple of 16 directly, the estimate traded a
        // round for narrower tiles where that loses: chain L4 / L5 +6 ... +13 %; 16 columns less at the same three
        // rounds: L4 -1.4 %, L5 +1 %.)
        if (bf16 && !conv && M > 128 && best2_n >= 96) {
            auto rounds = [&](int n) {
                const long long ntiles = (long long)((M + best2_rows - 1) / best2_rows) * ((Nc + n - 1) / n);
                const long long pairs = ntiles < sms / 2 ? ntiles : sms / 2;
                return (ntiles + pairs - 1) / pairs;
            };
            if (rounds(best2_n) == 1 && rounds(best2_n - 16) == 1) best2_n -= 16;
        }
        // (three pieces exist on the pair kernel only: never weigh it against the one-CTA TF32 kernel)
        if (best2_n && (best2 < best || bf16 == 2)) { *kernel = 2; *rows = best2_rows; *cols = best2_n; }
    }
}

static int launch_tc_common(const ubp_plan *pl, TcArgs a, cudaStream_t stream)
{
    const int M = pl->dims.M, K = a.K;
    const int64_t Nc = a.Nc;
    const uint8_t *dev = static_cast<const uint8_t *>(pl->dev);
    const float *Wh = reinterpret_cast<const float *>(dev + pl->img.tc_off);
    const float *Wl = Wh + (size_t)M * pl->img.tc_kp;
    int rc;
    a.M = M;
    a.status = reinterpret_cast<int *>(pl->dev);
    int sms = 148, devid = 0;
    if (cudaGetDevice(&devid) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, devid);
    int kernel, rows, best_n;
    // 3x3 on CTA pairs needs the input as one [channel][b, y, x] matrix with 16-byte aligned rows
    const bool conv_pair_ok = a.conv && a.isb == (int64_t)a.H * a.W && a.isc % 4 == 0 &&
                              (reinterpret_cast<uintptr_t>(a.X) & 15) == 0 && a.isc >= Nc;
    const int bf16 = cfg_bf16(pl->cfg) ? (cfg_pieces(pl->cfg) == 3 ? 2 : 1) : 0;   // 1: two bf16 pieces, 2: three
    tc_choose(M, K, Nc, a.conv ? (conv_pair_ok && a.stride <= 1 ? a.W : -1) : 0, bf16, sms, &kernel, &rows, &best_n);
    if (a.conv && conv_pair_ok && a.stride <= 1 && cfg_conv3_shift(pl->cfg)) {
        // the padded-grid kernel where it takes the layer; otherwise on through the per-tap kernels below
        a.rpc = 128;
        rc = launch_conv3_pair(dev + pl->img.tc16_off, a.X, a.isc, &a, M, K / 9, (int)(Nc / ((int64_t)a.H * a.W)), a.H, a.W, sms, stream);
        if (rc != UBP_E_UNSUPPORTED) return rc;
    }
    if (kernel == 2 && bf16) {
        CUtensorMap tmX;
        // the input as (column, channel): 16 channel rows of the CTA's columns per chunk, plus the halo for 3x3; 1x1: the
        // rows of all the chunks of a pipeline stage in one box
        const int halo = a.conv ? (a.W + 1 + 3) & ~3 : 0;
        const int box_rows = a.conv ? TC_KC : TC_KC * tc_pair_bf16_sub(K, best_n, halo, cfg_pieces(pl->cfg), rows / 256);
        if ((rc = encode_2d(&tmX, a.X, (uint64_t)Nc, (uint64_t)(a.conv ? K / 9 : K), (uint64_t)(a.conv ? a.isc : a.ldx) * 4,
                            (uint32_t)(best_n / 2 + 2 * halo), (uint32_t)box_rows, CU_TENSOR_MAP_SWIZZLE_NONE))) return rc;
        a.rpc = 128;
        a.dup = M <= 128 ? 1 : 0;          // one row tile: both CTAs of a pair take it and split the columns between them
        return launch_tc_pair_bf16(dev + pl->img.tc16_off, &tmX, a.conv, halo, &a, M, Nc, best_n, sms, stream, cfg_pieces(pl->cfg),
                                   rows / 256);
    }
    if (kernel == 2) {
        // Wh and Wl as one 3-D tensor (channel, row, part): one copy per chunk brings both
        CUtensorMap tmW, tmX;
        const uint64_t wdims[3] = {(uint64_t)pl->img.tc_kp, (uint64_t)M, 2};
        const uint32_t wbox[3] = {TC_KC, 128, 2};
        if ((rc = encode_3d(&tmW, Wh, wdims, (uint64_t)pl->img.tc_kp * 4, (uint64_t)M * pl->img.tc_kp * 4, wbox,
                            CU_TENSOR_MAP_SWIZZLE_64B))) return rc;
        // X as (column in a group of 32, channel, group): one copy per chunk brings all of a CTA's columns in the
        // operand layout. Needs whole groups; otherwise one 2-D copy per group.
        const int x3d = (!a.conv && Nc % 32 == 0) ? 1 : 0;
        const int halo = a.conv ? (a.W + 1 + 3) & ~3 : 0;
        if (a.conv) {
            rc = encode_2d(&tmX, a.X, (uint64_t)Nc, (uint64_t)(K / 9), (uint64_t)a.isc * 4, (uint32_t)(best_n / 2 + 2 * halo),
                           TC_KC, CU_TENSOR_MAP_SWIZZLE_NONE);
        } else if (x3d) {
            const uint64_t xdims[3] = {32, (uint64_t)K, (uint64_t)(Nc / 32)};
            const uint32_t xbox[3] = {32, TC_KC, (uint32_t)(best_n / 64)};
            rc = encode_3d(&tmX, a.X, xdims, (uint64_t)a.ldx * 4, 128, xbox, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B);
        } else {
            rc = encode_2d(&tmX, a.X, (uint64_t)Nc, (uint64_t)K, (uint64_t)a.ldx * 4, 32, TC_KC,
                           CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B);
        }
        if (rc) return rc;
        return launch_tc_pair(&tmW, &tmX, x3d, halo, &a, M, Nc, best_n, sms, stream);
    }
    CUtensorMap tmWh, tmWl;
    if ((rc = encode_2d(&tmWh, Wh, (uint64_t)pl->img.tc_kp, (uint64_t)M, (uint64_t)pl->img.tc_kp * 4, TC_KC, 128,
                        CU_TENSOR_MAP_SWIZZLE_64B))) return rc;
    if ((rc = encode_2d(&tmWl, Wl, (uint64_t)pl->img.tc_kp, (uint64_t)M, (uint64_t)pl->img.tc_kp * 4, TC_KC, 128,
                        CU_TENSOR_MAP_SWIZZLE_64B))) return rc;
    a.ntile = best_n;
    const bool use2 = rows == 256;
    const unsigned ncols = (unsigned)((Nc + best_n - 1) / best_n);
    auto launch = [&](auto kern, int MT, size_t smem) -> int {
        static bool done[2][64] = {};
        if (devid < 0 || devid >= 64 || !done[MT - 1][devid]) {
            cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) { set_last_cuda_error((int)e); return UBP_E_CUDA; }
            if (devid >= 0 && devid < 64) done[MT - 1][devid] = true;
        }
        dim3 grid((unsigned)((M + 128 * MT - 1) / (128 * MT)), ncols);
        kern<<<grid, TC_THREADS, smem, stream>>>(tmWh, tmWl, a);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) { set_last_cuda_error((int)e); return UBP_E_CUDA; }
        return UBP_OK;
    };
    if (use2) return launch(ubp_tc_kernel<2>, 2, (size_t)3 * (2 * 2 * A_HALF_BYTES + 2 * B_BYTES) + 1024);
    return launch(ubp_tc_kernel<1>, 1, (size_t)4 * (1 * 2 * A_HALF_BYTES + 2 * B_BYTES) + 1024);
}

int launch_spmm_tc(const ubp_plan *pl, const float *X, int64_t ldx, int64_t Nc, const float *bias, int relu,
                   float *Y, int64_t ldy, void *stream_)
{
    TcArgs a{};
    a.X = X; a.ldx = ldx; a.conv = 0; a.bias = bias; a.Y = Y; a.ldy = ldy; a.Nc = Nc; a.K = pl->dims.C; a.relu = relu;
    return launch_tc_common(pl, a, static_cast<cudaStream_t>(stream_));
}

// 1x1 with stride 2 on the bf16 CTA-pair kernel WITHOUT a gathered copy of the input: the tensor map shows the input
// [C][B][H][W] (rows contiguous over the images, H and W even) as (2 W floats of a row pair, B H / 2 row pairs, C); a box
// of W floats x (tile columns / Wo) row pairs x the stage's channels brings the even rows, and the split pass takes
// every other float. A CTA's half tile is whole output rows: NH a multiple of Wo (and of 8), N = 2 NH a multiple of 16.
// UBP_E_UNSUPPORTED where the plan, the shapes or the alignment do not allow it (the caller then gathers first).
int launch_spmm_tc_s2(const ubp_plan *pl, const float *in, int B, int H, int Wd, int64_t isc, const float *bias, int relu,
                      float *out, int64_t ldy, void *stream_)
{
    const int M = pl->dims.M, K = pl->dims.C;
    if (pl->cfg.kind != 2 || !cfg_bf16(pl->cfg) || cfg_pieces(pl->cfg) != 2 || pl->img.tc16_off == 0) return UBP_E_UNSUPPORTED;
    if ((H & 1) || (Wd & 3) || Wd > 256 || isc % 4 != 0 || isc < (int64_t)B * H * Wd || ldy % 4 != 0) return UBP_E_UNSUPPORTED;
    if (((reinterpret_cast<uintptr_t>(in) | reinterpret_cast<uintptr_t>(out)) & 15) != 0) return UBP_E_UNSUPPORTED;
    const int Ho = H / 2, Wo = Wd / 2;
    const int64_t Nc = (int64_t)B * Ho * Wo;
    if (Nc >= (1ll << 31) || (int64_t)B * H / 2 >= (1ll << 31)) return UBP_E_UNSUPPORTED;
    int sms = 148, devid = 0;
    if (cudaGetDevice(&devid) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, devid);
    // half-tile widths: the multiples of lcm(Wo, 8) from 32 up to 128 columns
    int unit = Wo;
    while (unit % 8 != 0) unit += Wo;
    if (unit > 128) return UBP_E_UNSUPPORTED;
    const int nchunk = (K + TC_KC - 1) / TC_KC;
    double best = 1e300;
    int best_nh = 0, best_mt = 1;
    for (int mt = 1; mt <= 2; ++mt) {
        if (mt == 2 && (M <= 128 || ((M + 255) / 256) % 2 != 0)) continue;
        for (int nh = unit; nh <= 128; nh += unit) {
            if (nh < 32 || (M <= 128 && (2 * nh) % 32 != 0)) continue;      // tiles of 64 columns and more, as tc_choose
            // (the raw rows are twice as long as the tile: `halo` = nh / 2 sizes them)
            const int sub = tc_pair_bf16_sub(K, 2 * nh, nh / 2, 2, mt);
            const int stages = tc_pair_bf16_stages_sub(2 * nh, nh / 2, sub, mt);
            if (stages < 4) continue;
            const int n = 2 * nh;
            const long long ntiles = (long long)((M + 256 * mt - 1) / (256 * mt)) * ((Nc + n - 1) / n);
            const long long pairs = ntiles < sms / 2 ? ntiles : sms / 2;
            const long long per_pair = (ntiles + pairs - 1) / pairs;
            // the estimate of tc_choose for plain and stacked tiles
            double per_chunk = mt == 2 ? 3.3 * n : 1.65 * n;
            const double floor_chunk = mt == 2 ? 600.0 + 0.33 * n : 470.0 + 0.33 * n;
            if (per_chunk < floor_chunk) per_chunk = floor_chunk;
            const double t = mt == 2 ? 4400.0 + (double)per_pair * (nchunk * per_chunk + 2500.0) + (double)(per_pair - 1) * 100.0 * n + 4500.0 + 60.0 * n
                                     : 4400.0 + (double)per_pair * ((nchunk * per_chunk > 50.0 * n ? nchunk * per_chunk : 50.0 * n) + 2500.0) + 4500.0 + 30.0 * n;
            if (t < best) { best = t; best_nh = nh; best_mt = mt; }
        }
    }
    if (!best_nh) return UBP_E_UNSUPPORTED;
    const int sub = tc_pair_bf16_sub(K, 2 * best_nh, best_nh / 2, 2, best_mt);
    CUtensorMap tmX;
    const uint64_t dims[3] = {(uint64_t)(2 * Wd), (uint64_t)((int64_t)B * H / 2), (uint64_t)K};
    const uint32_t box[3] = {(uint32_t)Wd, (uint32_t)(best_nh / Wo), (uint32_t)(TC_KC * sub)};
    int rc;
    if ((rc = encode_3d(&tmX, in, dims, (uint64_t)(2 * Wd) * 4, (uint64_t)isc * 4, box, CU_TENSOR_MAP_SWIZZLE_NONE))) return rc;
    TcArgs a{};
    a.X = in; a.ldx = isc; a.conv = 0; a.bias = bias; a.Y = out; a.ldy = ldy; a.Nc = Nc; a.K = K; a.relu = relu;
    a.M = M;
    a.status = reinterpret_cast<int *>(pl->dev);
    a.rpc = 128;
    a.dup = M <= 128 ? 1 : 0;
    a.s2 = Wo;
    const uint8_t *dev = static_cast<const uint8_t *>(pl->dev);
    return launch_tc_pair_bf16(dev + pl->img.tc16_off, &tmX, 0, best_nh / 2, &a, M, Nc, 2 * best_nh, sms, stream_, 2, best_mt);
}

int launch_conv3x3_tc(const ubp_plan *pl, const float *in, int B, int H, int Wd, int64_t isb, int64_t isc,
                      const float *bias, int relu, float *out, int64_t out_ld, void *stream_, int stride)
{
    TcArgs a{};
    a.X = in; a.ldx = 0; a.conv = 1; a.H = H; a.W = Wd; a.isb = isb; a.isc = isc; a.stride = stride;
    a.bias = bias; a.Y = out; a.ldy = out_ld; a.K = pl->dims.C * 9; a.relu = relu;
    a.Nc = (int64_t)B * ((H - 1) / stride + 1) * ((Wd - 1) / stride + 1);
    return launch_tc_common(pl, a, static_cast<cudaStream_t>(stream_));
}

}  // namespace ubp
