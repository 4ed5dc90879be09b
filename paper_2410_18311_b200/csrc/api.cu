// Host-only pieces of the ABI: the fraction rule, error text, device properties,
// and the status word read-back.
#include "common.cuh"

#include <math.h>
#include <string.h>

namespace coreinfer {

static thread_local char g_error[512] = "";

void set_error(const char* fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_error, sizeof g_error, fmt, ap);
    va_end(ap);
}

static thread_local unsigned long long* g_stamps = nullptr;
static thread_local size_t g_stamps_bytes = 0;

unsigned long long* stamps_buffer(size_t need_bytes)
{
    return (g_stamps && g_stamps_bytes >= need_bytes) ? g_stamps : nullptr;
}

coreinfer_status device_info(DeviceInfo* out)
{
    static thread_local DeviceInfo cache[64];
    static thread_local bool have[64] = {false};
    int dev = 0;
    CI_CUDA(cudaGetDevice(&dev));
    if (dev >= 0 && dev < 64 && have[dev]) {
        *out = cache[dev];
        return COREINFER_OK;
    }
    DeviceInfo di;
    di.device = dev;
    CI_CUDA(cudaDeviceGetAttribute(&di.sm_count, cudaDevAttrMultiProcessorCount, dev));
    CI_CUDA(cudaDeviceGetAttribute(&di.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    CI_CUDA(cudaDeviceGetAttribute(&di.cc_major, cudaDevAttrComputeCapabilityMajor, dev));
    if (di.cc_major != 10)
        CI_FAIL(COREINFER_ERR_CUDA,
                "device %d has compute capability %d.x; this library is built for sm_100a only", dev,
                di.cc_major);
    if (dev >= 0 && dev < 64) {
        cache[dev] = di;
        have[dev] = true;
    }
    *out = di;
    return COREINFER_OK;
}

}  // namespace coreinfer

extern "C" {

int32_t coreinfer_count(double frac, int32_t n)
{
    if (n <= 0) return 0;
    double c = ceil(frac * (double)n - 1e-6);
    if (c < 0.0) c = 0.0;
    if (c > (double)n) c = (double)n;
    return (int32_t)c;
}

const char* coreinfer_last_error(void) { return coreinfer::g_error; }

coreinfer_status coreinfer_debug_stamps(void* stamps, size_t bytes)
{
#ifdef COREINFER_STAMPS
    if (stamps && (reinterpret_cast<uintptr_t>(stamps) & 7u))
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "stamps must be 8-byte aligned");
    coreinfer::g_stamps = (unsigned long long*)stamps;
    coreinfer::g_stamps_bytes = stamps ? bytes : 0;
    return COREINFER_OK;
#else
    (void)stamps;
    (void)bytes;
    CI_FAIL(COREINFER_ERR_UNSUPPORTED, "this library was built without COREINFER_STAMPS");
#endif
}

coreinfer_status coreinfer_workspace_status(const void* workspace, void* cuda_stream)
{
    if (!workspace) CI_FAIL(COREINFER_ERR_INVALID_ARG, "workspace is NULL");
    cudaStream_t st = (cudaStream_t)cuda_stream;
    CI_CUDA(cudaStreamSynchronize(st));
    unsigned word = 0;
    CI_CUDA(cudaMemcpy(&word, workspace, sizeof word, cudaMemcpyDeviceToHost));
    if (word == coreinfer::kStatusOk) return COREINFER_OK;
    CI_FAIL(COREINFER_ERR_TIMEOUT, "a bounded device-side wait gave up (status word %u)", word);
}

}  // extern "C"
