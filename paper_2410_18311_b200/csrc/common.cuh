// Shared host/device helpers of the CoreInfer sm_100a library (not part of the ABI).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include <stdio.h>
#include <stdarg.h>

#include "coreinfer.h"

namespace coreinfer {

// ---------------------------------------------------------------- host ------
void set_error(const char* fmt, ...);

#define CI_FAIL(code, ...)                     \
    do {                                       \
        ::coreinfer::set_error(__VA_ARGS__);   \
        return (code);                         \
    } while (0)

#define CI_CUDA(expr)                                                                \
    do {                                                                             \
        cudaError_t e__ = (expr);                                                    \
        if (e__ != cudaSuccess) {                                                    \
            ::coreinfer::set_error("%s failed: %s", #expr, cudaGetErrorString(e__)); \
            return COREINFER_ERR_CUDA;                                               \
        }                                                                            \
    } while (0)

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline size_t dtype_size(coreinfer_dtype dt) { return dt == COREINFER_F32 ? 4 : 2; }
static inline bool dtype_known(coreinfer_dtype dt) { return dt == COREINFER_F32 || dt == COREINFER_BF16 || dt == COREINFER_F16; }
static inline bool kind_known(coreinfer_ffn_kind k)
{
    return k == COREINFER_FFN_RELU || k == COREINFER_FFN_RELU_GATED || k == COREINFER_FFN_SILU_GATED;
}
static inline bool kind_gated(coreinfer_ffn_kind k) { return k != COREINFER_FFN_RELU; }

// Cached per-device properties (SM count, opt-in shared memory).
struct DeviceInfo {
    int device;
    int sm_count;
    int smem_optin;
    int cc_major;
};
coreinfer_status device_info(DeviceInfo* out);

// Optional phase timing.  Built with -DCOREINFER_STAMPS, the persistent decode kernels store the
// SM cycle counter at fixed points of every layer into the buffer registered with
// coreinfer_debug_stamps(): [CTA][layer][kStampSlots] 64-bit words.  In the normal build
// the macro is empty and the registration call reports UNSUPPORTED.
constexpr int kStampSlots = 16;
unsigned long long* stamps_buffer(size_t need_bytes);   // NULL unless a large enough buffer is registered
#ifdef COREINFER_STAMPS
#define CI_STAMP(buf, base, id)                                  \
    do {                                                         \
        if (buf) (buf)[(base) + (id)] = (unsigned long long)clock64(); \
    } while (0)
#else
#define CI_STAMP(buf, base, id) do { } while (0)
#endif

// --------------------------------------------------------------- device -----
// Status word values written by kernels (first word of a decode workspace).
enum : unsigned { kStatusOk = 0u, kStatusTimeout = 5u };

#ifdef __CUDACC__

// Gate nonlinearity of the gated FFN kinds: ReLU, or SiLU g / (1 + exp(-g)) in fp32.
__device__ __forceinline__ float gate_activation(float g, int silu)
{
    return silu ? g / (1.0f + __expf(-g)) : fmaxf(g, 0.f);
}

__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---- mbarrier (shared::cta) ----
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Same test, but the thread may be parked by the hardware for up to `hint_ns` while the phase is
// incomplete (it resumes at once when the phase completes): a waiting warp then costs no issue slots.
__device__ __forceinline__ bool mbar_try_wait_parked(uint32_t bar, uint32_t parity, uint32_t hint_ns)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(hint_ns)
        : "memory");
    return ok != 0;
}

// 1-D bulk copy global -> shared of this CTA, completion counted on an mbarrier.
// dst, src 16-byte aligned; bytes a multiple of 16.  The copy targets this CTA alone.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
        : "memory");
}

// Shared-memory increment by 32-bit shared-window address (no generic address conversion).
__device__ __forceinline__ void red_shared_inc(uint32_t addr)
{
    asm volatile("red.shared.add.u32 [%0], 1;" ::"r"(addr) : "memory");
}

__device__ __forceinline__ void named_bar_sync(int id, int nthreads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// Arrival without waiting; `nthreads` counts the arriving and the waiting threads of the barrier.
__device__ __forceinline__ void named_bar_arrive(int id, int nthreads)
{
    asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned* p)
{
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Arrival on a counter with release semantics at GPU scope (no value returned).
__device__ __forceinline__ void red_release_add(unsigned* p, unsigned v)
{
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

__device__ __forceinline__ void red_add_v4(float* p, float a, float b, float c, float d)
{
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(a), "f"(b), "f"(c),
                 "f"(d)
                 : "memory");
}

// Bulk reduction shared -> global by the copy engine: adds `bytes` / 4 fp32 values at `src` (shared
// memory of this CTA, written through the generic proxy and fenced with fence_proxy_async before)
// into `dst`, element by element, each addition atomic.  Joined to the thread's bulk group.
__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void bulk_reduce_add_f32(float* dst, uint32_t src, uint32_t bytes)
{
    asm volatile("cp.reduce.async.bulk.global.shared::cta.bulk_group.add.f32 [%0], [%1], %2;"
                 ::"l"(dst), "r"(src), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// Returns when every bulk group of this thread has completed (reads and writes).
__device__ __forceinline__ void bulk_wait_all()
{
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

#endif  // __CUDACC__

}  // namespace coreinfer
