// Shared by the GEMM and the tile quantizer: mbarrier / TMA / elect wrappers (device) and the host-side helpers
// around tensor maps and per-device state.
#pragma once
#include <cuda.h>

#include <cstring>
#include <mutex>

#include "common.cuh"

namespace mx {

constexpr uint32_t kWaitSpinLimit = 1u << 22;   // x ~64 ns backoff  =>  ~0.3 s before a bounded wait gives up

// ---- PTX wrappers --------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false if it gave up (or another role already did).  The non-blocking test comes first: in a
// pipeline that runs ahead most waits find their barrier complete.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag, uint32_t *dev_status,
                                          uint32_t limit = kWaitSpinLimit)
{
    if (mbar_test_wait(bar, parity)) return true;
    for (uint32_t spin = 0; spin < limit; spin++) {
        if (mbar_try_wait(bar, parity)) return true;
        if (spin > 64) {
            if (*abort_flag) return false;
            __nanosleep(64);
        }
    }
    *abort_flag = 1u;
    if (dev_status) atomicOr(dev_status, MXFP4_DEV_TIMEOUT);
    return false;
}

// The same for a converged warp; the result is made uniform so that the warp leaves its loop together.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag, uint32_t *dev_status,
                                               uint32_t limit = kWaitSpinLimit)
{
    return __all_sync(0xFFFFFFFFu, mbar_wait(bar, parity, abort_flag, dev_status, limit));
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap *map, int x, int y, int z, uint32_t src)
{
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%1, %2, %3}], [%4];"
                 ::"l"(map), "r"(x), "r"(y), "r"(z), "r"(src) : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, int x, int y, uint32_t src)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"(map), "r"(x), "r"(y), "r"(src) : "memory");
}
// untiled store of `bytes` (a multiple of 16) from shared to global memory, both 16-byte aligned
__device__ __forceinline__ void bulk_store(void *dst, uint32_t src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// One lane of a converged warp.  The single-thread roles run their loops with the whole warp and let only this lane
// issue: addresses and descriptors then stay warp-uniform, which cuts the instruction overhead per MMA by a third.
__device__ __forceinline__ bool elect_one()
{
    uint32_t leader;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(leader));
    return leader != 0;
}


// ---- host side -------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// cuTensorMapEncodeTiled through a small per-thread cache: an encoded map is a pure function of the arguments, and a
// training loop asks for the same few dozen maps (same buffers, same shapes) step after step; outside a CUDA graph the
// encodes would otherwise be paid on every call.
struct TensorMapKey {
    uint64_t ptr, gdim[3], gstride[2];
    uint32_t box[3], estr[3], rank, dtype, interleave, swizzle, promo, oob;
};
static CUresult encode_tiled_cached(CUtensorMap *map, CUtensorMapDataType dtype, cuuint32_t rank, void *ptr, const cuuint64_t *gdim,
                                    const cuuint64_t *gstride, const cuuint32_t *box, const cuuint32_t *estr, CUtensorMapInterleave il,
                                    CUtensorMapSwizzle sw, CUtensorMapL2promotion promo, CUtensorMapFloatOOBfill oob)
{
    constexpr int kSlots = 64;
    struct Slot { TensorMapKey key; CUtensorMap map; bool used; };
    thread_local Slot slots[kSlots];
    thread_local int next = 0;
    EncodeTiledFn fn = get_encode_fn();
    if (!fn || rank < 1 || rank > 3) return CUDA_ERROR_NOT_SUPPORTED;
    TensorMapKey k;
    memset(&k, 0, sizeof(k));
    k.ptr = reinterpret_cast<uint64_t>(ptr);
    for (cuuint32_t i = 0; i < rank; i++) { k.gdim[i] = gdim[i]; k.box[i] = box[i]; k.estr[i] = estr[i]; }
    for (cuuint32_t i = 0; i + 1 < rank; i++) k.gstride[i] = gstride[i];
    k.rank = rank; k.dtype = (uint32_t)dtype; k.interleave = (uint32_t)il; k.swizzle = (uint32_t)sw; k.promo = (uint32_t)promo; k.oob = (uint32_t)oob;
    for (int i = 0; i < kSlots; i++)
        if (slots[i].used && memcmp(&slots[i].key, &k, sizeof(k)) == 0) {
            *map = slots[i].map;
            return CUDA_SUCCESS;
        }
    const CUresult r = fn(map, dtype, rank, ptr, gdim, gstride, box, estr, il, sw, promo, oob);
    if (r == CUDA_SUCCESS) {
        Slot &s = slots[next];
        next = (next + 1) % kSlots;
        s.key = k;
        s.map = *map;
        s.used = true;
    }
    return r;
}

// Host-side state is kept per device ordinal: a process may drive several GPUs, and function attributes, SM counts and
// the capability check belong to the device that is current at the call.
constexpr int kMaxDevices = 64;
static std::mutex g_dev_lock;

static int current_device()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
    return dev;
}

static int sm_count()
{
    static int n[kMaxDevices];
    const int dev = current_device();
    if (dev < 0) return 148;
    std::lock_guard<std::mutex> hold(g_dev_lock);
    if (!n[dev] && cudaDeviceGetAttribute(&n[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) n[dev] = 148;
    return n[dev];
}

// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) once per kernel and device; `done` is the kernel's own table.
template <typename Kernel>
static cudaError_t set_smem_once(bool (&done)[kMaxDevices], Kernel kernel, int bytes)
{
    const int dev = current_device();
    if (dev < 0) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> hold(g_dev_lock);
    if (done[dev]) return cudaSuccess;
    const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) done[dev] = true;
    return e;
}

}  // namespace mx
