// ubp_spmm_static: the 1x1 product for callers that cannot allocate device
// memory. The plan (the only scratch the product needs besides its inputs and
// outputs) lives in a fixed device array that is part of this library's image.
#include <cuda_runtime.h>

#include <mutex>
#include <new>

#include "ubp_internal.h"
#include "ubp_tc_common.cuh"

#define UBP_STATIC_PLAN_BYTES (2u * 1024u * 1024u)

// Every device that loads the library carries this array until the process
// exits. In host code the name below is only a handle for the runtime, not a
// device address: the address is looked up once per device (static_plan_ptr).
static __device__ __align__(256) unsigned char g_static_plan[UBP_STATIC_PLAN_BYTES];

namespace {

std::mutex g_mu;
void *g_ptr[64] = {};

// Device address of g_static_plan on the current device; resolved on first use.
int static_plan_ptr(void **out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { ubp::set_last_cuda_error((int)e); return UBP_E_CUDA; }
    if (dev < 0 || dev >= 64) return UBP_E_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_ptr[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_plan);
        if (e != cudaSuccess || !p) { ubp::set_last_cuda_error((int)e); return UBP_E_CUDA; }
        g_ptr[dev] = p;
    }
    *out = g_ptr[dev];
    return UBP_OK;
}

}  // namespace

// ---- bounded-wait self test -------------------------------------------------------------------------------
namespace {
// One thread waits on a barrier nobody ever completes, through the wait routine of the tensor-core kernels
// (tc::mbar_wait) with the caller's limit; when it gives up the plan's status word is set.
__global__ void ubp_wait_selftest_kernel(int *status, unsigned long long limit_ns)
{
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        ubp::tc::mbar_init(ubp::tc::smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (!ubp::tc::mbar_wait(ubp::tc::smem_u32(&bar), 0, &abort_flag, limit_ns)) atomicExch(status, 1);
    }
}
}  // namespace

extern "C" {

int ubp_plan_clear_status(const ubp_plan_t *plan, void *stream)
{
    if (!plan || plan->magic != kPlanMagic || !plan->dev) return UBP_E_ARG;
    cudaError_t e = cudaMemsetAsync(plan->dev, 0, sizeof(int), static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) { ubp::set_last_cuda_error((int)e); return UBP_E_CUDA; }
    return UBP_OK;
}

int ubp_selftest_bounded_wait(const ubp_plan_t *plan, unsigned limit_us, void *stream)
{
    if (!plan || plan->magic != kPlanMagic || !plan->dev || limit_us == 0 || limit_us > 1000000u) return UBP_E_ARG;
    ubp_wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<int *>(plan->dev),
                                                                             (unsigned long long)limit_us * 1000ull);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { ubp::set_last_cuda_error((int)e); return UBP_E_CUDA; }
    return UBP_OK;
}

size_t ubp_static_plan_capacity(void) { return UBP_STATIC_PLAN_BYTES; }

int ubp_spmm_static(const void *blob, size_t len, const float *X, int64_t ldx, int64_t Nc,
                    const float *bias, int relu, float *Y, int64_t ldy, void *stream)
{
    ubp_view_t v;
    int rc = ubp::blob_view(blob, len, &v);
    if (rc) return rc;
    if (v.R != 1 || Nc < 0) return UBP_E_ARG;
    if (Nc == 0) return UBP_OK;
    if (!X || !Y || ldx < Nc || ldy < Nc) return UBP_E_ARG;
    {
        // The plan is uploaded from a host buffer that dies with this call. Outside capture the runtime stages the
        // bytes before cudaMemcpyAsync returns; a captured copy would keep the host pointer and every replay would
        // read freed memory. So a capturing stream is refused before anything is touched.
        cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
        cudaError_t ce = cudaStreamIsCapturing(static_cast<cudaStream_t>(stream), &cs);
        if (ce != cudaSuccess) { ubp::set_last_cuda_error((int)ce); return UBP_E_CUDA; }
        if (cs != cudaStreamCaptureStatusNone) return UBP_E_UNSUPPORTED;
    }
    const ubp::KernelCfg *cfg = ubp::auto_cfg(v.M, v.C, v.R, v.Nb, v.m);
    if (!cfg) return UBP_E_UNSUPPORTED;
    try {
        ubp_plan tmp;                       // host-only handle, lives for this call
        tmp.magic = 0;
        tmp.dims = v;
        tmp.cfg = *cfg;
        size_t need = 0;
        if ((rc = ubp::build_plan_image(v, *cfg, true, tmp.img, &need))) return rc;
        if (need > UBP_STATIC_PLAN_BYTES && cfg->kind == 2) {
            // the tensor-core plan carries a dense copy of the weight; the sparse plan of the same geometry is
            // much smaller, so try that before giving up
            for (const auto &c : ubp::kernel_cfgs())
                if (c.kind == 0 && c.nbk == cfg->nbk && c.P == cfg->P && c.KT == cfg->KT && c.WR == cfg->WR &&
                    c.V == cfg->V && c.WC == cfg->WC && c.dupw == cfg->dupw) { cfg = &c; break; }
            tmp.cfg = *cfg;
            if ((rc = ubp::build_plan_image(v, *cfg, true, tmp.img, &need))) return rc;
        }
        if (need > UBP_STATIC_PLAN_BYTES) return UBP_E_STATIC_LIMIT;
        if ((rc = ubp::build_plan_image(v, *cfg, false, tmp.img, &need))) return rc;
        void *dev = nullptr;
        if ((rc = static_plan_ptr(&dev))) return rc;
        tmp.dev = dev;
        tmp.dev_bytes = need;
        // The image starts with a zeroed header (status word included), so the copy also clears
        // whatever the previous call left in the array. The source is pageable host memory: the
        // runtime stages it before returning, so the image may be freed when this function returns.
        cudaError_t e = cudaMemcpyAsync(dev, tmp.img.bytes.data(), need, cudaMemcpyHostToDevice,
                                        static_cast<cudaStream_t>(stream));
        if (e != cudaSuccess) { ubp::set_last_cuda_error((int)e); return UBP_E_CUDA; }
        return ubp::launch_spmm(&tmp, X, ldx, Nc, bias, relu, Y, ldy, stream);
    } catch (const std::bad_alloc &) { return UBP_E_SPACE; }
}

}  // extern "C"
