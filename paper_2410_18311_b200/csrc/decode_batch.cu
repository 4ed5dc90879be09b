// Decode FFN over compacted weights for 2..8 sequences that share one core set
// (Section 4.2 applied to a small batch): the plain kernels, used for fp32 and for bf16 rows the
// tensor-core kernel (decode_batch_mma.cu) is not built for.  Two streaming kernels:
//   up:   one warp per core neuron forms h[b, k] for every sequence b (fp32, kept in
//         the caller's workspace, [batch, K]);
//   down: CTAs tile (column block, neuron range), accumulate partial y[b, :] in
//         registers and add them into y with vector reductions.
// Each weight row is read from HBM once and used by all sequences.
#include "common.cuh"

namespace coreinfer {

constexpr int kCtrlBytesB = 256;
constexpr int kUpWarps = 8;
constexpr int kDownThreads = 256;
constexpr int kDownRows = 64;    // neurons per down-phase CTA

template <typename T> struct VecB;
template <> struct VecB<__nv_bfloat16> {
    static constexpr int kElems = 8;
    static __device__ __forceinline__ void unpack(const uint4& q, float (&f)[8])
    {
        f[0] = __uint_as_float(q.x << 16); f[1] = __uint_as_float(q.x & 0xffff0000u);
        f[2] = __uint_as_float(q.y << 16); f[3] = __uint_as_float(q.y & 0xffff0000u);
        f[4] = __uint_as_float(q.z << 16); f[5] = __uint_as_float(q.z & 0xffff0000u);
        f[6] = __uint_as_float(q.w << 16); f[7] = __uint_as_float(q.w & 0xffff0000u);
    }
    static __device__ __forceinline__ float load1(const void* p, int i)
    {
        return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p)[i]);
    }
};
template <> struct VecB<float> {
    static constexpr int kElems = 4;
    static __device__ __forceinline__ void unpack(const uint4& q, float (&f)[4])
    {
        f[0] = __uint_as_float(q.x); f[1] = __uint_as_float(q.y);
        f[2] = __uint_as_float(q.z); f[3] = __uint_as_float(q.w);
    }
    static __device__ __forceinline__ float load1(const void* p, int i)
    {
        return reinterpret_cast<const float*>(p)[i];
    }
};

template <typename T, int B, bool GATED>
__global__ void __launch_bounds__(kUpWarps * 32)
batch_up_kernel(const uint4* __restrict__ x, const uint4* __restrict__ w_up,
                const uint4* __restrict__ w_gate, const void* __restrict__ b_up, float* __restrict__ h,
                int nv, int K)
{
    using V = VecB<T>;
    constexpr int E = V::kElems;
    const int lane = threadIdx.x & 31;
    const int k = blockIdx.x * kUpWarps + (threadIdx.x >> 5);
    if (k >= K) return;
    float u[B], g[B];
#pragma unroll
    for (int b = 0; b < B; ++b) { u[b] = 0.f; g[b] = 0.f; }
    for (int v = lane; v < nv; v += 32) {
        float wu[E], wg[E];
        V::unpack(__ldcs(&w_up[(size_t)k * nv + v]), wu);
        if (GATED) V::unpack(__ldcs(&w_gate[(size_t)k * nv + v]), wg);
#pragma unroll
        for (int b = 0; b < B; ++b) {
            float xv[E];
            V::unpack(x[(size_t)b * nv + v], xv);
#pragma unroll
            for (int e = 0; e < E; ++e) {
                u[b] = fmaf(wu[e], xv[e], u[b]);
                if (GATED) g[b] = fmaf(wg[e], xv[e], g[b]);
            }
        }
    }
#pragma unroll
    for (int b = 0; b < B; ++b) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            u[b] += __shfl_xor_sync(0xffffffffu, u[b], o);
            if (GATED) g[b] += __shfl_xor_sync(0xffffffffu, g[b], o);
        }
    }
    if (lane == 0) {
#pragma unroll
        for (int b = 0; b < B; ++b) {
            float hv;
            if (GATED) {
                hv = fmaxf(g[b], 0.f) * u[b];
            } else {
                float t = u[b] + (b_up ? V::load1(b_up, k) : 0.f);
                hv = fmaxf(t, 0.f);
            }
            h[(size_t)b * K + k] = hv;
        }
    }
}

// grid = (column blocks, neuron blocks).  y must be zero on entry.
template <typename T, int B>
__global__ void __launch_bounds__(kDownThreads)
batch_down_kernel(const float* __restrict__ h, const uint4* __restrict__ w_down,
                  const void* __restrict__ b_down, float* __restrict__ y, int nv, int K, int d)
{
    using V = VecB<T>;
    constexpr int E = V::kElems;
    __shared__ float h_s[B][kDownRows];
    const int v = blockIdx.x * kDownThreads + threadIdx.x;
    const int k0 = blockIdx.y * kDownRows;
    const int k1 = min(k0 + kDownRows, K);
    for (int i = threadIdx.x; i < B * kDownRows; i += kDownThreads) {
        const int b = i / kDownRows, r = i % kDownRows;
        h_s[b][r] = (k0 + r < k1) ? h[(size_t)b * K + k0 + r] : 0.f;
    }
    __syncthreads();
    if (v >= nv) return;
    float acc[B][E];
#pragma unroll
    for (int b = 0; b < B; ++b)
#pragma unroll
        for (int e = 0; e < E; ++e)
            acc[b][e] = (blockIdx.y == 0 && b_down) ? V::load1(b_down, v * E + e) : 0.f;
    for (int k = k0; k < k1; ++k) {
        float w[E];
        V::unpack(__ldcs(&w_down[(size_t)k * nv + v]), w);
#pragma unroll
        for (int b = 0; b < B; ++b) {
            const float hk = h_s[b][k - k0];
#pragma unroll
            for (int e = 0; e < E; ++e) acc[b][e] = fmaf(hk, w[e], acc[b][e]);
        }
    }
#pragma unroll
    for (int b = 0; b < B; ++b)
#pragma unroll
        for (int e = 0; e < E; e += 4)
            red_add_v4(y + (size_t)b * d + (size_t)v * E + e, acc[b][e], acc[b][e + 1], acc[b][e + 2],
                       acc[b][e + 3]);
}

template <typename T, int B>
static coreinfer_status run_b(const void* x, bool gated, int d_model, const coreinfer_layer& ly, float* y,
                              float* h, cudaStream_t st)
{
    const int K = ly.K;
    const int nv = (int)((size_t)d_model * sizeof(T) / 16);
    CI_CUDA(cudaMemsetAsync(y, 0, (size_t)B * d_model * sizeof(float), st));
    const int gu = (K + kUpWarps - 1) / kUpWarps;
    if (gated)
        batch_up_kernel<T, B, true><<<gu, kUpWarps * 32, 0, st>>>(
            (const uint4*)x, (const uint4*)ly.w_up_c, (const uint4*)ly.w_gate_c, nullptr, h, nv, K);
    else
        batch_up_kernel<T, B, false><<<gu, kUpWarps * 32, 0, st>>>(
            (const uint4*)x, (const uint4*)ly.w_up_c, nullptr, ly.b_up_c, h, nv, K);
    CI_CUDA(cudaGetLastError());
    dim3 gd((nv + kDownThreads - 1) / kDownThreads, (K + kDownRows - 1) / kDownRows);
    batch_down_kernel<T, B><<<gd, kDownThreads, 0, st>>>(h, (const uint4*)ly.w_downT_c, ly.b_down, y, nv, K,
                                                          d_model);
    CI_CUDA(cudaGetLastError());
    return COREINFER_OK;
}

template <typename T>
static coreinfer_status run_t(int batch, const void* x, bool gated, int d_model, const coreinfer_layer& ly,
                              float* y, float* h, cudaStream_t st)
{
    switch (batch) {
        case 2: return run_b<T, 2>(x, gated, d_model, ly, y, h, st);
        case 3: return run_b<T, 3>(x, gated, d_model, ly, y, h, st);
        case 4: return run_b<T, 4>(x, gated, d_model, ly, y, h, st);
        case 5: return run_b<T, 5>(x, gated, d_model, ly, y, h, st);
        case 6: return run_b<T, 6>(x, gated, d_model, ly, y, h, st);
        case 7: return run_b<T, 7>(x, gated, d_model, ly, y, h, st);
        case 8: return run_b<T, 8>(x, gated, d_model, ly, y, h, st);
        default: CI_FAIL(COREINFER_ERR_UNSUPPORTED, "batch %d not built", batch);
    }
}

// decode_batch_mma.cu: tensor-core kernel for bf16 rows of up to 4096 columns
coreinfer_status decode_batched_mma(const void* x, int batch, bool gated, int d_model, const coreinfer_layer& ly,
                                    float* y, unsigned* status, const DeviceInfo& di, cudaStream_t st);

coreinfer_status decode_batched(const void* x, int batch, coreinfer_dtype dtype, coreinfer_ffn_kind kind,
                                int d_model, const coreinfer_layer& ly, float* y, void* workspace,
                                cudaStream_t st)
{
    DeviceInfo di;
    coreinfer_status s = device_info(&di);
    if (s != COREINFER_OK) return s;
    const bool gated = kind == COREINFER_FFN_RELU_GATED;
    CI_CUDA(cudaMemsetAsync(workspace, 0, kCtrlBytesB, st));   // status word
    if (dtype == COREINFER_BF16) {
        s = decode_batched_mma(x, batch, gated, d_model, ly, y, (unsigned*)workspace, di, st);
        if (s != COREINFER_ERR_UNSUPPORTED) return s;          // otherwise: shape not built there, use the plain kernels
    }
    float* h = (float*)((uint8_t*)workspace + kCtrlBytesB);
    if (dtype == COREINFER_BF16) return run_t<__nv_bfloat16>(batch, x, gated, d_model, ly, y, h, st);
    return run_t<float>(batch, x, gated, d_model, ly, y, h, st);
}

}  // namespace coreinfer
