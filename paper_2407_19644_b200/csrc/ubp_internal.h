// Internal declarations shared by the library's translation units.
#ifndef UBP_INTERNAL_H_
#define UBP_INTERNAL_H_

#include <cstddef>
#include <cstdint>
#include <vector>

#include "ubp.h"

namespace ubp {

// ---- format (ubp_format.cpp)
int pack(const float *W, const uint8_t *mask, int M, int C, int R, int Nb,
         void *blob, size_t blob_cap, size_t *blob_len);
int unpack(const void *blob, size_t len, float *W_out, uint8_t *mask_out);
int blob_view(const void *blob, size_t len, ubp_view_t *v);

// ---- kernel configurations (ubp_plan.cpp)
// A configuration fixes how blocks are bucketed (plan geometry) and which
// kernel instantiation consumes them.
struct KernelCfg {
    int id;        // 1-based variant id
    int kind;      // 4 = 1x1 product walked from the canonical arrays in the paper's own dataflow (ubp_wros.cu);
                   // 0 = 1x1 product (R == 1), 1 = implicit 3x3 (R == 9), 2 = 1x1 on tensor cores (densified
                   //     panels, 3 x TF32) with the kind-0 plan of the same geometry embedded as its fallback,
                   // 3 = 3x3 as an implicit GEMM on tensor cores with the kind-1 plan embedded
    int nbk;       // rows per plan entry; divides the layer's Nb
    int P;         // rows per panel (one warp's output rows)
    int V;         // float4 column groups per lane (a warp covers 128*V columns)
    int WR, WC;    // warps per CTA along rows / columns
    int KT;        // input channels per staged tile
    int dupw;      // weights stored twice (w, w) for packed f32x2 multiply-add
};
const std::vector<KernelCfg> &kernel_cfgs();
// tensor-core variants whose CTA-pair kernel uses three bf16 products per fp32 product instead of three TF32 products
// 64..67: 3x3 with the taps as shifts of one staged operand on the padded pixel grid (ubp_conv3.cu; bf16 products too)
inline bool cfg_conv3_shift(const KernelCfg &c) { return c.id >= 64 && c.id <= 67; }
// 84..87: the bf16 CTA-pair kernel with every operand in THREE bf16 pieces (exact) and six products per fp32 product
inline int cfg_pieces(const KernelCfg &c) { return (c.id >= 84 && c.id <= 87) ? 3 : 2; }
inline bool cfg_bf16(const KernelCfg &c)
{
    return (c.id >= 34 && c.id <= 37) || (c.id >= 44 && c.id <= 47) || cfg_conv3_shift(c) || cfg_pieces(c) == 3;
}
const KernelCfg *find_cfg(int id);
// Whether the dense tensor-core form beats the sparse kernel for a layer with `dens` of its weights kept. Measured on
// B200, launches back to back, blocks of 4: the tensor-core kernel takes the same time at every sparsity; the sparse
// kernel re-stages the activations once per 128 output rows and pays a fixed cost per (panel, channel tile, start offset),
// so it shrinks slowly: 512x512x6272 at 92 / 95 / 97 % sparsity 19.4 / 16.8 / 15.4 us against 16.7; 1024x1024x3136
// 36.3 / 31.3 / 28.4 against 22.4; 2048x2048x8192 286 / 234 / 210 against 152; 256x256x50176 31.9 / 28.1 / 26.7 against
// 25.7. Hence: from 3 % kept on, and for layers of a million weights or more from 0.5 % on.
inline bool tensor_core_pays(int M, int C, double dens)
{
    return dens >= 0.03 || ((int64_t)M * C >= (1ll << 20) && dens >= 0.005);
}
// pick a configuration for a layer (variant == 0)
const KernelCfg *auto_cfg(int M, int C, int R, int Nb, int64_t m);

// ---- plan (ubp_plan.cpp)
// Device image layout (all offsets from the image base, which is 256-byte aligned):
//   [0, 256)            header; int32 status word at byte 0 (0 = fine)
//   [256, ...)          uint32 group_off[nkt * NG + 1], in 16-byte units from the base
//   groups in (kt, g) order, each 16-byte aligned:
//       uint32 poff[WR + 1]            byte offsets of the panel sub-segments from the group start
//       per panel: uint16 fo[F + 1]    entry offsets per fragment (F = P + nbk - 1), padded to 16
//                  uint16 jl[n + 4]    input channel inside the tile (4 zero entries of read-ahead slack), padded to 16
//                  float  w[n + 2][nbk][R][dup]   un-rotated weights of the entry (2 zero entries of slack), padded to 16
struct PlanImage {
    std::vector<uint8_t> bytes;
    int nkt = 0, NP = 0, NG = 0, F = 0;
    int64_t entries = 0;
    uint32_t max_group_bytes = 0;
    // kind 2 only: byte offset of the dense part (Wh [M][tc_kp] then Wl [M][tc_kp], floats) and its row length
    size_t tc_off = 0;
    int tc_kp = 0;
    // and of the same weight as two bf16 pieces (W1 = the weight rounded to bf16, W2 = the remainder rounded to bf16),
    // tiled: 8 KB blocks [row tile][chunk of 16 channels] = [piece][128 rows][16 channels] in the 32-byte swizzle;
    // row tile t holds rows 128 t .. 128 t + 127 of the matrix in order (rows beyond M are zero; whole pairs of tiles);
    // tc16_kp = reduction length padded to whole chunks
    size_t tc16_off = 0;
    int tc16_kp = 0;
    int tc16_pieces = 2;     // bf16 pieces per weight in that part (3: W3 = the remainder after W1 + W2, blocks of 12 KB)
    // kind 4 only: byte offsets of the canonical arrays indptr [M+1], indices [m], values [m][Nb] in the image
    size_t wros_off[3] = {0, 0, 0};
};
int build_plan_image(const ubp_view_t &v, const KernelCfg &cfg, bool count_only, PlanImage &img, size_t *bytes);

}  // namespace ubp

constexpr uint32_t kPlanMagic = 0x50504255u;   // "UBPP": first word of a live plan handle

struct ubp_plan {
    uint32_t magic;                 // 'UBPP'
    ubp_view_t dims;                // M, C, R, Nb, m (pointers unused)
    ubp::KernelCfg cfg;
    ubp::PlanImage img;             // host copy (kept until free)
    void *dev;                      // caller's device buffer
    size_t dev_bytes;
};

// ---- launches (ubp_kernels.cu)
namespace ubp {
int launch_spmm(const ubp_plan *plan, const float *X, int64_t ldx, int64_t Nc, const float *bias, int relu,
                float *Y, int64_t ldy, void *stream);
// tensor-core tile choice for a launch over Nc columns: kernel 1 = one CTA per tile, 2 = CTA pair per tile;
// conv_w = 0: 1x1; > 0: 3x3 on images conv_w pixels wide (operands fit the pair kernel); < 0: 3x3, one CTA only
void tc_choose(int M, int K, int64_t Nc, int conv_w, int bf16, int sms, int *kernel, int *rows, int *cols);
int launch_spmm_tc(const ubp_plan *plan, const float *X, int64_t ldx, int64_t Nc, const float *bias, int relu,
                   float *Y, int64_t ldy, void *stream);
// 1x1, stride 2, straight from the full-resolution input (bf16 CTA-pair kernel); UBP_E_UNSUPPORTED if not applicable
int launch_spmm_tc_s2(const ubp_plan *plan, const float *in, int B, int H, int Wd, int64_t isc, const float *bias, int relu,
                      float *out, int64_t ldy, void *stream);
int launch_conv3x3_tc(const ubp_plan *plan, const float *in, int B, int H, int Wd, int64_t isb, int64_t isc,
                      const float *bias, int relu, float *out, int64_t out_ld, void *stream, int stride = 1);
// tensor-core implicit GEMM when the plan and the layouts allow it (stride 1: CTA pairs where the operands qualify;
// stride > 1: the one-CTA kernel, whose loaders gather the taps pixel by pixel); else one lane per output pixel
int launch_conv3x3(const ubp_plan *plan, const float *in, int B, int H, int Wd, int64_t isb, int64_t isc,
                   const float *bias, int relu, float *out, int64_t osb, int64_t osc, void *stream, int stride = 1,
                   void *scratch = nullptr, size_t scratch_bytes = 0);
// bytes of scratch the stride-2 3x3 fast path needs (phase planes), 0 for other strides
size_t conv3x3_strided_scratch_bytes(int C, int B, int H, int Wd, int stride);
int launch_subsample(const float *in, int C, int B, int H, int Wd, int64_t isb, int64_t isc, int stride, float *out,
                     void *stream);
// the paper's dataflow on the canonical arrays (ubp_wros.cu): variants 60 (weight rotation) and 61 (naive shift)
int launch_wros(const ubp_plan *plan, const float *X, int64_t ldx, int64_t Nc, const float *bias, int relu, float *Y,
                int64_t ldy, void *stream);
// 3x3 on the padded pixel grid, taps as descriptor shifts (ubp_conv3.cu); UBP_E_UNSUPPORTED when the layer does not fit
int launch_conv3_pair(const void *W16, const float *X, int64_t isc, const void *args, int M, int C, int B, int H, int W,
                      int sms, void *stream, int s2 = 0);
// stride 2: the four phase planes of the input as a [4*C][ld] matrix (ubp_conv3.cu)
int launch_phase_planes(const float *in, int C, int B, int H, int Wd, int64_t isb, int64_t isc, float *out, int64_t ld,
                        void *stream);
bool conv3_pair_tile(int M, int C, int B, int H, int W, int sms, int *tile_cols);
void set_last_cuda_error(int e);
}

#endif
