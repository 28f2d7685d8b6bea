// extern "C" surface of the library (declared in include/ubp.h): argument
// checks, plan life cycle, and dispatch to the launchers. No device
// synchronisation except in ubp_plan_check.
#include <cuda_runtime.h>

#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "ubp_internal.h"

namespace ubp {
static thread_local int g_last_cuda = 0;
void set_last_cuda_error(int e) { g_last_cuda = e; }
}  // namespace ubp

extern "C" {

const char *ubp_strerror(int status)
{
    switch (status) {
        case UBP_OK: return "ok";
        case UBP_E_ARG: return "invalid argument";
        case UBP_E_RAGGED: return "mask has a run of ones that is not a whole number of blocks";
        case UBP_E_SPACE: return "buffer too small or out of host memory";
        case UBP_E_FORMAT: return "malformed blob or plan";
        case UBP_E_CUDA: return "CUDA call failed";
        case UBP_E_UNSUPPORTED: return "unsupported configuration";
        case UBP_E_DEVICE: return "a kernel gave up on a bounded wait";
        case UBP_E_STATIC_LIMIT: return "layer's plan exceeds the fixed device scratch of ubp_spmm_static";
        default: return "unknown status";
    }
}

int ubp_last_cuda_error(void) { return ubp::g_last_cuda; }

int ubp_pack(const float *W, const uint8_t *mask, int M, int C, int R, int Nb,
             void *blob, size_t blob_cap, size_t *blob_len)
{
    try { return ubp::pack(W, mask, M, C, R, Nb, blob, blob_cap, blob_len); }
    catch (const std::bad_alloc &) { return UBP_E_SPACE; }
}

int ubp_unpack(const void *blob, size_t len, float *W_out, uint8_t *mask_out)
{
    try { return ubp::unpack(blob, len, W_out, mask_out); }
    catch (const std::bad_alloc &) { return UBP_E_SPACE; }
}

int ubp_blob_view(const void *blob, size_t len, ubp_view_t *view) { return ubp::blob_view(blob, len, view); }

int ubp_pack_kmajor(const float *W, const uint8_t *mask, int M, int C, int B,
                    void *blob, size_t blob_cap, size_t *blob_len)
{
    if (!W || !mask || !blob_len || M < 1 || C < 1 || B < 1 || B > C) return UBP_E_ARG;
    try {
        // the same layer seen from the other side: rows <-> columns, so runs along the input channels of one output
        // row become runs along the rows of one column, which is what the packer cuts into blocks
        std::vector<float> Wt((size_t)M * C);
        std::vector<uint8_t> mt((size_t)M * C);
        for (int i = 0; i < M; ++i)
            for (int j = 0; j < C; ++j) {
                Wt[(size_t)j * M + i] = W[(size_t)i * C + j];
                mt[(size_t)j * M + i] = mask[(size_t)i * C + j];
            }
        return ubp::pack(Wt.data(), mt.data(), C, M, 1, B, blob, blob_cap, blob_len);
    } catch (const std::bad_alloc &) { return UBP_E_SPACE; }
}

int ubp_kmajor_to_plan_blob(const void *kblob, size_t klen, void *blob, size_t blob_cap, size_t *blob_len)
{
    if (!kblob || !blob_len) return UBP_E_ARG;
    ubp_view_t v;
    if (int rc = ubp::blob_view(kblob, klen, &v)) return rc;
    if (v.R != 1) return UBP_E_UNSUPPORTED;
    try {
        const int M = v.C, C = v.M;            // the layer's own output / input channel counts
        std::vector<float> Wt((size_t)M * C), W((size_t)M * C);
        std::vector<uint8_t> mt((size_t)M * C), mask((size_t)M * C);
        if (int rc = ubp::unpack(kblob, klen, Wt.data(), mt.data())) return rc;
        for (int j = 0; j < C; ++j)
            for (int i = 0; i < M; ++i) {
                W[(size_t)i * C + j] = Wt[(size_t)j * M + i];
                mask[(size_t)i * C + j] = mt[(size_t)j * M + i];
            }
        return ubp::pack(W.data(), mask.data(), M, C, 1, 1, blob, blob_cap, blob_len);
    } catch (const std::bad_alloc &) { return UBP_E_SPACE; }
}

int ubp_variant_count(void) { return (int)ubp::kernel_cfgs().size(); }

int ubp_variant_at(int index)
{
    const auto &c = ubp::kernel_cfgs();
    if (index < 0 || index >= (int)c.size()) return UBP_E_ARG;
    return c[(size_t)index].id;
}

int ubp_variant_describe(int variant, char *buf, size_t cap)
{
    const ubp::KernelCfg *c = ubp::find_cfg(variant);
    if (!c || !buf || cap == 0) return UBP_E_ARG;
    const char *prod = ubp::cfg_pieces(*c) == 3 ? "6xBF16, three pieces" : (ubp::cfg_bf16(*c) ? "3xBF16" : "3xTF32");
    char kind[64];
    if (c->kind == 4) {
        std::snprintf(buf, cap, "spmm-from-canonical-arrays %s", c->id == 61 ? "naive(outputs shifted per start row)"
                                                                            : "weight-rotating output-stationary");
        return UBP_OK;
    }
    if (c->kind == 0) std::snprintf(kind, sizeof kind, "spmm");
    else if (c->kind == 5) std::snprintf(kind, sizeof kind, "spmm-k-runs(blocks along the input channels)");
    else if (c->kind == 1) std::snprintf(kind, sizeof kind, "conv3x3");
    else std::snprintf(kind, sizeof kind, "%s-tensorcore(%s) fallback", c->kind == 2 ? "spmm" : "conv3x3", prod);
    std::snprintf(buf, cap, "%s nbk=%d panel=%d cols/warp=%d warps=%dx%d ktile=%d%s", kind, c->nbk, c->P, 128 * c->V,
                  c->WR, c->WC, c->KT, c->dupw ? " dupw" : "");
    return UBP_OK;
}

static int resolve_cfg(const ubp_view_t &v, int variant, const ubp::KernelCfg **cfg)
{
    const ubp::KernelCfg *c = variant == 0 ? ubp::auto_cfg(v.M, v.C, v.R, v.Nb, v.m) : ubp::find_cfg(variant);
    if (!c) return variant == 0 ? UBP_E_UNSUPPORTED : UBP_E_ARG;
    if (c->kind == 5) return UBP_E_ARG;          // K-run configurations take a K-major blob: ubp_plan_build_kmajor
    *cfg = c;
    return UBP_OK;
}

int ubp_plan_size(const void *blob, size_t len, int variant, size_t *dev_bytes)
{
    if (!dev_bytes) return UBP_E_ARG;
    ubp_view_t v;
    int rc = ubp::blob_view(blob, len, &v);
    if (rc) return rc;
    const ubp::KernelCfg *cfg;
    if ((rc = resolve_cfg(v, variant, &cfg))) return rc;
    try {
        ubp::PlanImage img;
        return ubp::build_plan_image(v, *cfg, true, img, dev_bytes);
    } catch (const std::bad_alloc &) { return UBP_E_SPACE; }
}

int ubp_plan_image(const void *blob, size_t len, int variant, void *host_buf, size_t cap, int32_t geom[8])
{
    if (!host_buf || !geom) return UBP_E_ARG;
    ubp_view_t v;
    int rc = ubp::blob_view(blob, len, &v);
    if (rc) return rc;
    const ubp::KernelCfg *cfg;
    if ((rc = resolve_cfg(v, variant, &cfg))) return rc;
    try {
        ubp::PlanImage img;
        size_t need = 0;
        if ((rc = ubp::build_plan_image(v, *cfg, false, img, &need))) return rc;
        if (cap < need) return UBP_E_SPACE;
        std::memcpy(host_buf, img.bytes.data(), need);
        geom[0] = cfg->nbk; geom[1] = cfg->P; geom[2] = cfg->KT; geom[3] = cfg->WR; geom[4] = cfg->dupw;
        geom[5] = img.nkt; geom[6] = img.NP; geom[7] = img.NG;
    } catch (const std::bad_alloc &) { return UBP_E_SPACE; }
    return UBP_OK;
}

// Build the image of `v` for `cfg`, copy it to the device and hand back the handle. The handle's dims are the LAYER's:
// for a K-run configuration (kind 5) the blob is that of the transposed layer, so rows and channels swap places.
static int plan_build_view(const ubp_view_t &v, const ubp::KernelCfg *cfg, void *dev_buf, size_t dev_bytes, void *stream,
                           ubp_plan_t **plan)
{
    ubp_plan *p = nullptr;
    try {
        p = new ubp_plan();
        p->magic = kPlanMagic;
        p->dims = v; p->dims.indptr = nullptr; p->dims.indices = nullptr; p->dims.values = nullptr;
        if (cfg->kind == 5) { p->dims.M = v.C; p->dims.C = v.M; }
        p->cfg = *cfg;
        size_t need = 0;
        int rc = ubp::build_plan_image(v, *cfg, false, p->img, &need);
        if (!rc && dev_bytes < need) rc = UBP_E_SPACE;
        if (rc) { delete p; return rc; }
        p->dev = dev_buf; p->dev_bytes = need;
    } catch (const std::bad_alloc &) { delete p; return UBP_E_SPACE; }
    cudaError_t e = cudaMemcpyAsync(dev_buf, p->img.bytes.data(), p->img.bytes.size(), cudaMemcpyHostToDevice,
                                    static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) { ubp::set_last_cuda_error((int)e); delete p; return UBP_E_CUDA; }
    *plan = p;
    return UBP_OK;
}

int ubp_plan_build(const void *blob, size_t len, int variant, void *dev_buf, size_t dev_bytes,
                   void *stream, ubp_plan_t **plan)
{
    if (!plan || !dev_buf || (reinterpret_cast<uintptr_t>(dev_buf) & 255)) return UBP_E_ARG;
    *plan = nullptr;
    ubp_view_t v;
    int rc = ubp::blob_view(blob, len, &v);
    if (rc) return rc;
    const ubp::KernelCfg *cfg;
    if ((rc = resolve_cfg(v, variant, &cfg))) return rc;
    return plan_build_view(v, cfg, dev_buf, dev_bytes, stream, plan);
}

// The other orientation: which configuration a K-major blob (of the transposed layer) runs on, and whether it first has
// to be re-expressed in the layer's own orientation as single-channel blocks (the tensor-core kernels densify the
// weight and do not care; the element-wise sparse configuration serves run lengths the K-run kernel has no
// instantiation for).
static int resolve_kmajor(const ubp_view_t &kv, int variant, const ubp::KernelCfg **cfg, bool *convert)
{
    const int M = kv.C, C = kv.M, B = kv.Nb;
    if (kv.R != 1) return UBP_E_UNSUPPORTED;
    const ubp::KernelCfg *c = nullptr;
    if (variant == 0) {
        const double dens = (double)kv.m * B / ((double)M * C);
        const int krun = B == 2 ? 70 : B == 4 ? 71 : B == 8 ? 72 : B == 16 ? 73 : 0;
        if ((ubp::tensor_core_pays(M, C, dens) && M >= 128 && C >= 64) || !krun) c = ubp::auto_cfg(M, C, 1, 1, (int64_t)kv.m * B);
        else c = ubp::find_cfg(krun);
    } else {
        c = ubp::find_cfg(variant);
    }
    if (!c) return variant == 0 ? UBP_E_UNSUPPORTED : UBP_E_ARG;
    *cfg = c;
    *convert = c->kind != 5;
    return UBP_OK;
}

static int kmajor_prepare(const void *kblob, size_t klen, int variant, const ubp::KernelCfg **cfg, std::vector<uint8_t> &conv,
                          ubp_view_t *v)
{
    ubp_view_t kv;
    int rc = ubp::blob_view(kblob, klen, &kv);
    if (rc) return rc;
    bool convert = false;
    if ((rc = resolve_kmajor(kv, variant, cfg, &convert))) return rc;
    if (!convert) { *v = kv; return UBP_OK; }
    size_t n = 0;
    if ((rc = ubp_kmajor_to_plan_blob(kblob, klen, nullptr, 0, &n))) return rc;
    conv.resize(n);
    if ((rc = ubp_kmajor_to_plan_blob(kblob, klen, conv.data(), n, &n))) return rc;
    return ubp::blob_view(conv.data(), n, v);
}

int ubp_plan_size_kmajor(const void *kblob, size_t klen, int variant, size_t *dev_bytes)
{
    if (!dev_bytes) return UBP_E_ARG;
    try {
        const ubp::KernelCfg *cfg;
        std::vector<uint8_t> conv;
        ubp_view_t v;
        if (int rc = kmajor_prepare(kblob, klen, variant, &cfg, conv, &v)) return rc;
        ubp::PlanImage img;
        return ubp::build_plan_image(v, *cfg, true, img, dev_bytes);
    } catch (const std::bad_alloc &) { return UBP_E_SPACE; }
}

int ubp_plan_build_kmajor(const void *kblob, size_t klen, int variant, void *dev_buf, size_t dev_bytes, void *stream,
                          ubp_plan_t **plan)
{
    if (!plan || !dev_buf || (reinterpret_cast<uintptr_t>(dev_buf) & 255)) return UBP_E_ARG;
    *plan = nullptr;
    try {
        const ubp::KernelCfg *cfg;
        std::vector<uint8_t> conv;
        ubp_view_t v;
        if (int rc = kmajor_prepare(kblob, klen, variant, &cfg, conv, &v)) return rc;
        return plan_build_view(v, cfg, dev_buf, dev_bytes, stream, plan);
    } catch (const std::bad_alloc &) { return UBP_E_SPACE; }
}

int ubp_plan_image_kmajor(const void *kblob, size_t klen, int variant, void *host_buf, size_t cap, int32_t geom[8])
{
    if (!host_buf || !geom) return UBP_E_ARG;
    try {
        const ubp::KernelCfg *cfg;
        std::vector<uint8_t> conv;
        ubp_view_t v;
        if (int rc = kmajor_prepare(kblob, klen, variant, &cfg, conv, &v)) return rc;
        ubp::PlanImage img;
        size_t need = 0;
        if (int rc = ubp::build_plan_image(v, *cfg, false, img, &need)) return rc;
        if (cap < need) return UBP_E_SPACE;
        std::memcpy(host_buf, img.bytes.data(), need);
        geom[0] = cfg->nbk; geom[1] = cfg->P; geom[2] = cfg->KT; geom[3] = cfg->WR; geom[4] = cfg->dupw;
        geom[5] = img.nkt; geom[6] = img.NP; geom[7] = img.NG;
    } catch (const std::bad_alloc &) { return UBP_E_SPACE; }
    return UBP_OK;
}

void ubp_plan_free(ubp_plan_t *plan)
{
    if (plan && plan->magic == kPlanMagic) { plan->magic = 0; delete plan; }
}

int ubp_plan_info(const ubp_plan_t *plan, ubp_plan_info_t *info)
{
    if (!plan || plan->magic != kPlanMagic || !info) return UBP_E_ARG;
    info->M = plan->dims.M; info->C = plan->dims.C; info->R = plan->dims.R; info->Nb = plan->dims.Nb; info->m = plan->dims.m;
    info->variant = plan->cfg.id; info->panel_rows = plan->cfg.P; info->k_tile = plan->cfg.KT;
    info->entries = plan->img.entries; info->dev_bytes = (int64_t)plan->dev_bytes;
    return UBP_OK;
}

int ubp_plan_tile_choice(const ubp_plan_t *plan, int64_t Nc, int image_width, int *kernel, int *tile_rows, int *tile_cols)
{
    if (!plan || plan->magic != kPlanMagic || Nc < 0 || !kernel || !tile_rows || !tile_cols) return UBP_E_ARG;
    if (plan->dims.R == 9 && image_width == 0) return UBP_E_ARG;
    const ubp::KernelCfg &c = plan->cfg;
    if (c.kind == 2 || c.kind == 3) {
        int sms = 148, devid = 0;
        if (cudaGetDevice(&devid) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, devid);
        ubp::tc_choose(plan->dims.M, plan->dims.C * plan->dims.R, Nc, c.kind == 3 ? (image_width > 0 ? image_width : -1) : 0, ubp::cfg_bf16(c) ? (ubp::cfg_pieces(c) == 3 ? 2 : 1) : 0, sms, kernel, tile_rows,
                       tile_cols);
    } else if (c.kind == 4) {
        *kernel = 3; *tile_rows = 0; *tile_cols = 512;       // row ranges are chosen per launch; 128 threads x 4 columns
    } else {
        *kernel = 0; *tile_rows = c.P * c.WR; *tile_cols = 128 * c.V * c.WC;
    }
    return UBP_OK;
}

int ubp_plan_tile_choice_conv(const ubp_plan_t *plan, int B, int H, int Wd, int stride, int *kernel, int *tile_rows,
                              int *tile_cols)
{
    if (!plan || plan->magic != kPlanMagic || !kernel || !tile_rows || !tile_cols) return UBP_E_ARG;
    if (plan->dims.R != 9 || B < 1 || H < 1 || Wd < 1 || stride < 1) return UBP_E_ARG;
    const ubp::KernelCfg &c = plan->cfg;
    int sms = 148, devid = 0;
    if (cudaGetDevice(&devid) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, devid);
    int n = 0;
    const int Hq = stride == 2 ? (H - 1) / 2 + 1 : H, Wq = stride == 2 ? (Wd - 1) / 2 + 1 : Wd;      // stride 2: phase planes
    if ((stride == 1 || stride == 2) && ubp::cfg_conv3_shift(c) && ubp::conv3_pair_tile(plan->dims.M, plan->dims.C, B, Hq, Wq, sms, &n)) {
        *kernel = 4; *tile_rows = 256; *tile_cols = n;
        return UBP_OK;
    }
    const int64_t Nc = (int64_t)B * ((H - 1) / stride + 1) * ((Wd - 1) / stride + 1);
    return ubp_plan_tile_choice(plan, Nc, stride == 1 ? Wd : -Wd, kernel, tile_rows, tile_cols);
}

int ubp_plan_check(const ubp_plan_t *plan, void *stream)
{
    if (!plan || plan->magic != kPlanMagic) return UBP_E_ARG;
    int word = 0;
    cudaError_t e = cudaMemcpyAsync(&word, plan->dev, sizeof word, cudaMemcpyDeviceToHost, static_cast<cudaStream_t>(stream));
    if (e == cudaSuccess) e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) { ubp::set_last_cuda_error((int)e); return UBP_E_CUDA; }
    return word == 0 ? UBP_OK : UBP_E_DEVICE;
}

int ubp_spmm(const ubp_plan_t *plan, const float *X, int64_t ldx, int64_t Nc,
             const float *bias, int relu, float *Y, int64_t ldy, void *stream)
{
    if (!plan || plan->magic != kPlanMagic) return UBP_E_ARG;
    if (plan->dims.R != 1 || plan->cfg.kind == 1 || plan->cfg.kind == 3) return UBP_E_ARG;
    if (Nc < 0) return UBP_E_ARG;
    if (Nc == 0) return UBP_OK;
    if (!X || !Y || ldx < Nc || ldy < Nc) return UBP_E_ARG;
    return ubp::launch_spmm(plan, X, ldx, Nc, bias, relu, Y, ldy, stream);
}

int ubp_conv1x1(const ubp_plan_t *plan, const float *in, int B, int H, int Wd,
                int64_t in_stride_b, int64_t in_stride_c, const float *bias, int relu,
                float *out, int64_t out_stride_b, int64_t out_stride_c, void *stream)
{
    if (!plan || plan->magic != kPlanMagic) return UBP_E_ARG;
    if (plan->dims.R != 1 || plan->cfg.kind == 1 || plan->cfg.kind == 3) return UBP_E_ARG;
    if (B < 0 || H <= 0 || Wd <= 0) return UBP_E_ARG;
    if (B == 0) return UBP_OK;
    if (!in || !out) return UBP_E_ARG;
    const int64_t hw = (int64_t)H * Wd;
    if (in_stride_b == hw && out_stride_b == hw) {          // channel-major: one product over all images
        if (in_stride_c < hw * B || out_stride_c < hw * B) return UBP_E_ARG;
        return ubp::launch_spmm(plan, in, in_stride_c, hw * B, bias, relu, out, out_stride_c, stream);
    }
    if (in_stride_c < hw || out_stride_c < hw || in_stride_b < 0 || out_stride_b < 0) return UBP_E_ARG;
    for (int b = 0; b < B; ++b) {                            // one product per image
        int rc = ubp::launch_spmm(plan, in + (size_t)b * in_stride_b, in_stride_c, hw, bias, relu,
                                  out + (size_t)b * out_stride_b, out_stride_c, stream);
        if (rc) return rc;
    }
    return UBP_OK;
}

int ubp_conv3x3_implicit(const ubp_plan_t *plan, const float *in, int B, int H, int Wd,
                         int64_t in_stride_b, int64_t in_stride_c, const float *bias, int relu,
                         float *out, int64_t out_stride_b, int64_t out_stride_c, void *stream)
{
    if (!plan || plan->magic != kPlanMagic) return UBP_E_ARG;
    if (plan->dims.R != 9 || (plan->cfg.kind != 1 && plan->cfg.kind != 3)) return UBP_E_ARG;
    if (B < 0 || H <= 0 || Wd <= 0) return UBP_E_ARG;
    if (B == 0) return UBP_OK;
    if (!in || !out) return UBP_E_ARG;
    const int64_t hw = (int64_t)H * Wd;
    if (in_stride_c < hw || out_stride_c < hw || in_stride_b < 0 || out_stride_b < 0) return UBP_E_ARG;
    return ubp::launch_conv3x3(plan, in, B, H, Wd, in_stride_b, in_stride_c, bias, relu, out, out_stride_b,
                               out_stride_c, stream);
}

int ubp_conv3x3_strided(const ubp_plan_t *plan, const float *in, int B, int H, int Wd, int stride,
                        int64_t in_stride_b, int64_t in_stride_c, const float *bias, int relu,
                        float *out, int64_t out_stride_b, int64_t out_stride_c, void *stream)
{
    if (stride == 1)
        return ubp_conv3x3_implicit(plan, in, B, H, Wd, in_stride_b, in_stride_c, bias, relu, out, out_stride_b,
                                    out_stride_c, stream);
    if (!plan || plan->magic != kPlanMagic) return UBP_E_ARG;
    if (plan->dims.R != 9 || (plan->cfg.kind != 1 && plan->cfg.kind != 3)) return UBP_E_ARG;
    if (stride < 1 || B < 0 || H <= 0 || Wd <= 0) return UBP_E_ARG;
    if (B == 0) return UBP_OK;
    if (!in || !out) return UBP_E_ARG;
    const int64_t hw = (int64_t)H * Wd;
    const int64_t ohw = (int64_t)((H - 1) / stride + 1) * ((Wd - 1) / stride + 1);
    if (in_stride_c < hw || out_stride_c < ohw || in_stride_b < 0 || out_stride_b < 0) return UBP_E_ARG;
    return ubp::launch_conv3x3(plan, in, B, H, Wd, in_stride_b, in_stride_c, bias, relu, out, out_stride_b,
                               out_stride_c, stream, stride);
}

size_t ubp_conv3x3_strided_scratch(int C, int B, int H, int Wd, int stride)
{
    return ubp::conv3x3_strided_scratch_bytes(C, B, H, Wd, stride);
}

int ubp_conv3x3_strided_ws(const ubp_plan_t *plan, const float *in, int B, int H, int Wd, int stride,
                           int64_t in_stride_b, int64_t in_stride_c, void *scratch, size_t scratch_bytes,
                           const float *bias, int relu, float *out, int64_t out_stride_b, int64_t out_stride_c, void *stream)
{
    if (stride == 1 || !scratch)
        return ubp_conv3x3_strided(plan, in, B, H, Wd, stride, in_stride_b, in_stride_c, bias, relu, out, out_stride_b,
                                   out_stride_c, stream);
    if (!plan || plan->magic != kPlanMagic) return UBP_E_ARG;
    if (plan->dims.R != 9 || (plan->cfg.kind != 1 && plan->cfg.kind != 3)) return UBP_E_ARG;
    if (stride < 1 || B < 0 || H <= 0 || Wd <= 0) return UBP_E_ARG;
    if (B == 0) return UBP_OK;
    if (!in || !out || ((uintptr_t)scratch & 15u) != 0) return UBP_E_ARG;
    const int64_t hw = (int64_t)H * Wd;
    const int64_t ohw = (int64_t)((H - 1) / stride + 1) * ((Wd - 1) / stride + 1);
    if (in_stride_c < hw || out_stride_c < ohw || in_stride_b < 0 || out_stride_b < 0) return UBP_E_ARG;
    if (scratch_bytes < ubp_conv3x3_strided_scratch(plan->dims.C, B, H, Wd, stride)) return UBP_E_SPACE;
    return ubp::launch_conv3x3(plan, in, B, H, Wd, in_stride_b, in_stride_c, bias, relu, out, out_stride_b, out_stride_c,
                               stream, stride, scratch, scratch_bytes);
}

size_t ubp_conv1x1_strided_scratch(int C, int B, int H, int Wd, int stride)
{
    if (C <= 0 || B <= 0 || H <= 0 || Wd <= 0 || stride <= 1) return 0;
    return (size_t)C * B * ((H - 1) / stride + 1) * ((Wd - 1) / stride + 1) * sizeof(float);
}

int ubp_conv1x1_strided(const ubp_plan_t *plan, const float *in, int B, int H, int Wd, int stride,
                        int64_t in_stride_b, int64_t in_stride_c, void *scratch, size_t scratch_bytes,
                        const float *bias, int relu, float *out, int64_t out_stride_b, int64_t out_stride_c, void *stream)
{
    if (stride == 1)
        return ubp_conv1x1(plan, in, B, H, Wd, in_stride_b, in_stride_c, bias, relu, out, out_stride_b, out_stride_c, stream);
    if (!plan || plan->magic != kPlanMagic) return UBP_E_ARG;
    if (plan->dims.R != 1 || plan->cfg.kind == 1 || plan->cfg.kind == 3) return UBP_E_ARG;
    if (stride < 1 || B < 0 || H <= 0 || Wd <= 0) return UBP_E_ARG;
    if (B == 0) return UBP_OK;
    if (!in || !out || !scratch || ((uintptr_t)scratch & 15u) != 0) return UBP_E_ARG;
    const int64_t hw = (int64_t)H * Wd;
    if (in_stride_c < hw || in_stride_b < 0) return UBP_E_ARG;
    const int C = plan->dims.C;
    if (scratch_bytes < ubp_conv1x1_strided_scratch(C, B, H, Wd, stride)) return UBP_E_SPACE;
    const int Ho = (H - 1) / stride + 1, Wo = (Wd - 1) / stride + 1;
    // stride 2, one channel-major product over all images, on the bf16 CTA-pair kernel: straight from the
    // full-resolution input (its copies bring the even rows, its split pass takes every other pixel); no gather
    if (stride == 2 && in_stride_b == hw && out_stride_b == (int64_t)Ho * Wo && out_stride_c >= (int64_t)B * Ho * Wo) {
        const int rc = ubp::launch_spmm_tc_s2(plan, in, B, H, Wd, in_stride_c, bias, relu, out, out_stride_c, stream);
        if (rc != UBP_E_UNSUPPORTED) return rc;
    }
    float *xs = static_cast<float *>(scratch);
    if (int rc = ubp::launch_subsample(in, C, B, H, Wd, in_stride_b, in_stride_c, stride, xs, stream)) return rc;
    return ubp_conv1x1(plan, xs, B, Ho, Wo, (int64_t)Ho * Wo, (int64_t)B * Ho * Wo, bias, relu, out, out_stride_b,
                       out_stride_c, stream);
}

}  // extern "C"
