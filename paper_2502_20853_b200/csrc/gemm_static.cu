// mxfp4_gemm_static: the block-scaled product for callers that cannot allocate device memory.
//
// Some callers sit where no allocation may happen: a plugin that is handed its tensors by a
// host runtime with a sealed memory pool, code running while a stream is being captured, or a
// latency-critical step whose rules forbid touching the allocator.  mxfp4_gemm asks such a caller
// for split-K scratch it has no way to provide.  This entry point keeps that scratch inside the
// library instead, in a fixed array in device global memory that is part of the loaded module.
#include <mutex>

#include "common.cuh"

namespace mx {
mxfp4_status_t gemm(mxfp4_mat_t a, mxfp4_mat_t b, void *d, int64_t ldd, int out_dtype, const void *bias, void *workspace,
                    size_t workspace_bytes, uint32_t *dev_status, cudaStream_t st, bool allow_split);
size_t gemm_workspace_bytes(int64_t m, int64_t n, int64_t kc);
}  // namespace mx

// The scratch itself.  It exists once per GPU that loads this library and stays until the process
// exits.  In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[MXFP4_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_lock;
void *g_scratch_ptr[kMaxDevices];   // device address of g_static_scratch on each device, once looked up

// Device address of the scratch array on the current device (looked up on first use).
mxfp4_status_t scratch_on_current_device(void **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MXFP4_CUDA_ERROR;
    std::lock_guard<std::mutex> hold(g_lock);
    if (!g_scratch_ptr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return MXFP4_CUDA_ERROR;
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return MXFP4_OK;
}

}  // namespace

extern "C" mxfp4_status_t mxfp4_gemm_static(mxfp4_mat_t a, mxfp4_mat_t b, void *d, int64_t ldd, int32_t out_dtype,
                                            const void *bias_bf16, uint32_t *dev_status, void *stream)
{
    const size_t need = mx::gemm_workspace_bytes(a.rows, b.rows, a.cols);
    if (need > (size_t)MXFP4_STATIC_SCRATCH_BYTES) return MXFP4_WORKSPACE_TOO_SMALL;
    void *scratch = nullptr;
    if (need > 0) {
        const mxfp4_status_t s = scratch_on_current_device(&scratch);
        if (s) return s;
    }
    return mx::gemm(a, b, d, ldd, out_dtype, bias_bf16, scratch, need ? (size_t)MXFP4_STATIC_SCRATCH_BYTES : 0, dev_status,
                    static_cast<cudaStream_t>(stream), true);
}
