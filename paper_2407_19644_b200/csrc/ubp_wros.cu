// The paper's own dataflow on the GPU, straight from the canonical arrays (no re-bucketed plan): comparison kernels
// for the claims of Section 3.3 / Section 5.4 (unaligned with weight rotation ~ aligned; "naive" unaligned slower).
//
// A thread owns four adjacent activation columns and walks the start rows ("tiles") i = 0, 1, 2, ... with row step 1,
// exactly like the paper's microkernel: for every block that starts at row i it loads the activation vector of the
// block's input channel and does Nb multiply-adds into Nb stationary accumulators.
//   * weight-rotating output-stationary form (variant 60; Section 4.2): the stored weights are already rotated, the
//     weight in slot p belongs to the output row rho with rho mod Nb = p, so the inner loop is R[p] += v[p] * x for
//     every block of every tile; after tile i the finished row i sits in slot i mod Nb, is stored and cleared. The
//     row loop is unrolled Nb times so that i mod Nb is a compile-time constant (registers cannot be indexed).
//   * naive form (variant 61; Section 3.3 "Naive implementation"): accumulator t holds row i + t of the current
//     tile; the weights are fetched in row order, v[(i + t) mod Nb]; after the tile R[0] is stored and every
//     accumulator moves down one place. The row loop is deliberately not unrolled, so the moves are real.
// Output rows are split over CTAs in ranges; a range's walk begins Nb - 1 tiles early (blocks that start above the
// range but reach into it), accumulating without storing: one writer per output, fixed summation order.
// The aligned pattern (every start a multiple of Nb) and element-wise pruning (Nb = 1) run through the same code.
#include <cuda_runtime.h>

#include <cstdint>

#include "ubp_internal.h"
#include "ubp_tc_common.cuh"

namespace ubp {

namespace {

struct WrosArgs {
    const int32_t *indptr, *indices;
    const float *values;
    const float *X;
    int64_t ldx, Nc;
    const float *bias;
    float *Y;
    int64_t ldy;
    int M, relu, rows_per_cta;
    int C, m;                // input channels and blocks of the layer (what the checked build compares indices with)
    int *status;             // plan status word
};

constexpr int WROS_THREADS = 128;

template <bool VEC>
__device__ __forceinline__ float4 load_x(const float *p, int64_t col, int64_t Nc)
{
    if (VEC && col + 3 < Nc) return *reinterpret_cast<const float4 *>(p + col);
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (col < Nc) v.x = p[col];
    if (col + 1 < Nc) v.y = p[col + 1];
    if (col + 2 < Nc) v.z = p[col + 2];
    if (col + 3 < Nc) v.w = p[col + 3];
    return v;
}

template <bool VEC>
__device__ __forceinline__ void store_row(const WrosArgs &a, int row, int64_t col, float4 r)
{
    const float b = a.bias ? __ldg(a.bias + row) : 0.f;
    r.x += b; r.y += b; r.z += b; r.w += b;
    if (a.relu) { r.x = fmaxf(r.x, 0.f); r.y = fmaxf(r.y, 0.f); r.z = fmaxf(r.z, 0.f); r.w = fmaxf(r.w, 0.f); }
    float *y = a.Y + (size_t)row * a.ldy;
    if (VEC && col + 3 < a.Nc) { *reinterpret_cast<float4 *>(y + col) = r; return; }
    if (col < a.Nc) y[col] = r.x;
    if (col + 1 < a.Nc) y[col + 1] = r.y;
    if (col + 2 < a.Nc) y[col + 2] = r.z;
    if (col + 3 < a.Nc) y[col + 3] = r.w;
}

__device__ __forceinline__ void fma4(float4 &acc, float w, const float4 &x)
{
    acc.x = fmaf(w, x.x, acc.x); acc.y = fmaf(w, x.y, acc.y); acc.z = fmaf(w, x.z, acc.z); acc.w = fmaf(w, x.w, acc.w);
}

template <int NB, bool NAIVE, bool VEC>
__global__ void __launch_bounds__(WROS_THREADS)
ubp_wros_kernel(const WrosArgs a)
{
    const int64_t col = ((int64_t)blockIdx.x * WROS_THREADS + threadIdx.x) * 4;
    if (col >= a.Nc) return;
    const int r0 = (int)blockIdx.y * a.rows_per_cta;
    const int r1 = r0 + a.rows_per_cta < a.M ? r0 + a.rows_per_cta : a.M;
    const int t_first = r0 - (NB - 1) > 0 ? r0 - (NB - 1) : 0;      // first tile that can reach row r0
    float4 R[NB];
#pragma unroll
    for (int p = 0; p < NB; ++p) R[p] = make_float4(0.f, 0.f, 0.f, 0.f);

    if (!NAIVE) {
        // tiles in groups of NB so that the slot of the finished row, tile mod NB, is static
        for (int i = t_first / NB * NB; i < r1; i += NB) {
#pragma unroll
            for (int r = 0; r < NB; ++r) {
                const int tile = i + r;
                if (tile < t_first || tile >= r1) continue;
                const int b1 = __ldg(a.indptr + tile + 1);
                for (int b = __ldg(a.indptr + tile); b < b1; ++b) {
                    if (!UBP_CHK_GMEM(b >= 0 && b < a.m && (unsigned)__ldg(a.indices + b) < (unsigned)a.C, a.status)) break;
                    const float4 x = load_x<VEC>(a.X + (size_t)__ldg(a.indices + b) * a.ldx, col, a.Nc);
                    const float *v = a.values + (size_t)b * NB;
#pragma unroll
                    for (int p = 0; p < NB; ++p) fma4(R[p], __ldg(v + p), x);
                }
                if (tile >= r0) store_row<VEC>(a, tile, col, R[r]);      // row `tile` is complete: slot tile mod NB
                R[r] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
    } else {
#pragma unroll 1
        for (int tile = t_first; tile < r1; ++tile) {
            const int b1 = __ldg(a.indptr + tile + 1);
            for (int b = __ldg(a.indptr + tile); b < b1; ++b) {
                if (!UBP_CHK_GMEM(b >= 0 && b < a.m && (unsigned)__ldg(a.indices + b) < (unsigned)a.C, a.status)) break;
                const float4 x = load_x<VEC>(a.X + (size_t)__ldg(a.indices + b) * a.ldx, col, a.Nc);
                const float *v = a.values + (size_t)b * NB;
#pragma unroll
                for (int t = 0; t < NB; ++t) fma4(R[t], __ldg(v + (tile + t) % NB), x);   // row tile + t of the block
            }
            if (tile >= r0) store_row<VEC>(a, tile, col, R[0]);
#pragma unroll
            for (int t = 0; t + 1 < NB; ++t) R[t] = R[t + 1];        // the outputs move down one place
            R[NB - 1] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
    }
}

template <int NB>
int launch_nb(const WrosArgs &a, bool naive, bool vec, dim3 grid, cudaStream_t s)
{
    if (naive) {
        if (vec) ubp_wros_kernel<NB, true, true><<<grid, WROS_THREADS, 0, s>>>(a);
        else ubp_wros_kernel<NB, true, false><<<grid, WROS_THREADS, 0, s>>>(a);
    } else {
        if (vec) ubp_wros_kernel<NB, false, true><<<grid, WROS_THREADS, 0, s>>>(a);
        else ubp_wros_kernel<NB, false, false><<<grid, WROS_THREADS, 0, s>>>(a);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_last_cuda_error((int)e); return UBP_E_CUDA; }
    return UBP_OK;
}

}  // namespace

// Plan image of the format-direct variants: the canonical arrays themselves at img.wros_off[0..2] (indptr, indices,
// values). Row ranges: enough CTAs to fill the device a few times over, but at least 4 Nb rows each so that the Nb - 1
// tiles a range walks without storing stay a small part of its work.
int launch_wros(const ubp_plan *pl, const float *X, int64_t ldx, int64_t Nc, const float *bias, int relu, float *Y,
                int64_t ldy, void *stream)
{
    const uint8_t *dev = static_cast<const uint8_t *>(pl->dev);
    WrosArgs a;
    a.indptr = reinterpret_cast<const int32_t *>(dev + pl->img.wros_off[0]);
    a.indices = reinterpret_cast<const int32_t *>(dev + pl->img.wros_off[1]);
    a.values = reinterpret_cast<const float *>(dev + pl->img.wros_off[2]);
    a.X = X; a.ldx = ldx; a.Nc = Nc; a.bias = bias; a.Y = Y; a.ldy = ldy; a.M = pl->dims.M; a.relu = relu;
    a.C = pl->dims.C; a.m = (int)pl->img.entries; a.status = static_cast<int *>(pl->dev);
    const int Nb = pl->dims.Nb;
    const int64_t strips = (Nc + 4 * WROS_THREADS - 1) / (4 * WROS_THREADS);
    if (strips > 0x7fffffffll) return UBP_E_UNSUPPORTED;
    int sms = 148, devid = 0;
    if (cudaGetDevice(&devid) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, devid);
    int64_t groups = (8ll * sms + strips - 1) / strips;               // aim at ~8 CTAs per SM
    int rows = (int)((a.M + groups - 1) / groups);
    if (rows < 4 * Nb) rows = 4 * Nb;
    if (rows > a.M) rows = a.M;
    a.rows_per_cta = rows;
    const dim3 grid((unsigned)strips, (unsigned)((a.M + rows - 1) / rows));
    const bool vec = ((reinterpret_cast<uintptr_t>(X) | reinterpret_cast<uintptr_t>(Y)) & 15) == 0 && ldx % 4 == 0 && ldy % 4 == 0;
    const bool naive = pl->cfg.id == 61;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    switch (Nb) {
        case 1: return launch_nb<1>(a, naive, vec, grid, s);
        case 2: return launch_nb<2>(a, naive, vec, grid, s);
        case 4: return launch_nb<4>(a, naive, vec, grid, s);
        case 8: return launch_nb<8>(a, naive, vec, grid, s);
        case 16: return launch_nb<16>(a, naive, vec, grid, s);
        default: return UBP_E_UNSUPPORTED;
    }
}

}  // namespace ubp
