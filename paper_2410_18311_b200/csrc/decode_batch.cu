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
template <> struct VecB<__half> {
    static constexpr int kElems = 8;
    static __device__ __forceinline__ void unpack(const uint4& q, float (&f)[8])
    {
        const __half2* h = reinterpret_cast<const __half2*>(&q);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 t = __half22float2(h[i]);
            f[2 * i] = t.x;
            f[2 * i + 1] = t.y;
        }
    }
    static __device__ __forceinline__ float load1(const void* p, int i)
    {
        return __half2float(reinterpret_cast<const __half*>(p)[i]);
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
                int nv, int K, int silu)
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
                hv = gate_activation(g[b], silu) * u[b];
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
static coreinfer_status run_b(const void* x, bool gated, int silu, int d_model, const coreinfer_layer& ly, float* y,
                              float* h, cudaStream_t st)
{
    const int K = ly.K;
    const int nv = (int)((size_t)d_model * sizeof(T) / 16);
    CI_CUDA(cudaMemsetAsync(y, 0, (size_t)B * d_model * sizeof(float), st));
    const int gu = (K + kUpWarps - 1) / kUpWarps;
    if (gated)
        batch_up_kernel<T, B, true><<<gu, kUpWarps * 32, 0, st>>>(
            (const uint4*)x, (const uint4*)ly.w_up_c, (const uint4*)ly.w_gate_c, nullptr, h, nv, K, silu);
    else
        batch_up_kernel<T, B, false><<<gu, kUpWarps * 32, 0, st>>>(
            (const uint4*)x, (const uint4*)ly.w_up_c, nullptr, ly.b_up_c, h, nv, K, 0);
    CI_CUDA(cudaGetLastError());
    dim3 gd((nv + kDownThreads - 1) / kDownThreads, (K + kDownRows - 1) / kDownRows);
    batch_down_kernel<T, B><<<gd, kDownThreads, 0, st>>>(h, (const uint4*)ly.w_downT_c, ly.b_down, y, nv, K,
                                                          d_model);
    CI_CUDA(cudaGetLastError());
    return COREINFER_OK;
}

template <typename T>
static coreinfer_status run_t(int batch, const void* x, bool gated, int silu, int d_model, const coreinfer_layer& ly,
                              float* y, float* h, cudaStream_t st)
{
    switch (batch) {
        case 2: return run_b<T, 2>(x, gated, silu, d_model, ly, y, h, st);
        case 3: return run_b<T, 3>(x, gated, silu, d_model, ly, y, h, st);
        case 4: return run_b<T, 4>(x, gated, silu, d_model, ly, y, h, st);
        case 5: return run_b<T, 5>(x, gated, silu, d_model, ly, y, h, st);
        case 6: return run_b<T, 6>(x, gated, silu, d_model, ly, y, h, st);
        case 7: return run_b<T, 7>(x, gated, silu, d_model, ly, y, h, st);
        case 8: return run_b<T, 8>(x, gated, silu, d_model, ly, y, h, st);
        default: CI_FAIL(COREINFER_ERR_UNSUPPORTED, "batch %d not built", batch);
    }
}

// decode_batch_mma.cu: tensor-core kernel for bf16 rows of up to 4096 columns
coreinfer_status decode_batched_mma(const void* x, int batch, bool gated, int silu, int d_model, const coreinfer_layer& ly,
                                    float* y, unsigned* status, const DeviceInfo& di, cudaStream_t st);
bool decode_batched_mma_serves(int d_model, int K, const DeviceInfo& di);
coreinfer_status decode_stack_batched_mma(const coreinfer_layer* layers, int L, const void* x0, int batch, bool gated,
                                          int silu, int d_model, float* y_last, float* y_layers, void* x_layers, float* ybuf,
                                          unsigned* ctrl, const DeviceInfo& di, cudaStream_t st);

coreinfer_status decode_batched(const void* x, int batch, coreinfer_dtype dtype, coreinfer_ffn_kind kind,
                                int d_model, const coreinfer_layer& ly, float* y, void* workspace,
                                cudaStream_t st, bool clear_status)
{
    DeviceInfo di;
    coreinfer_status s = device_info(&di);
    if (s != COREINFER_OK) return s;
    const bool gated = kind_gated(kind);
    const int silu = kind == COREINFER_FFN_SILU_GATED;
    if (clear_status) CI_CUDA(cudaMemsetAsync(workspace, 0, kCtrlBytesB, st));   // status word
    if (dtype == COREINFER_BF16) {
        s = decode_batched_mma(x, batch, gated, silu, d_model, ly, y, (unsigned*)workspace, di, st);
        if (s != COREINFER_ERR_UNSUPPORTED) return s;          // otherwise: shape not built there, use the plain kernels
    }
    float* h = (float*)((uint8_t*)workspace + kCtrlBytesB);
    if (dtype == COREINFER_BF16) return run_t<__nv_bfloat16>(batch, x, gated, silu, d_model, ly, y, h, st);
    if (dtype == COREINFER_F16) return run_t<__half>(batch, x, gated, silu, d_model, ly, y, h, st);
    return run_t<float>(batch, x, gated, silu, d_model, ly, y, h, st);
}

// ------------------------------------------------------------- stack, batch 2..8 --
static __device__ __forceinline__ float to_f(float v) { return v; }
static __device__ __forceinline__ float to_f(__nv_bfloat16 v) { return __bfloat162float(v); }
static __device__ __forceinline__ float to_f(__half v) { return __half2float(v); }
template <typename T> static __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }
template <> __device__ __forceinline__ __half from_f<__half>(float v) { return __float2half_rn(v); }

// Glue between two layers for the per-layer path, one CTA per sequence: x_next = round((x + y) /
// rms(x + y)), the same formula (rsqrtf of the mean square) as in the batch-1 stack kernel.
template <typename T>
__global__ void __launch_bounds__(256)
batch_glue_kernel(const T* __restrict__ x, const float* __restrict__ y, T* __restrict__ x_next,
                  T* __restrict__ x_dump, int d, float inv_d)
{
    __shared__ float part[8];
    const size_t base = (size_t)blockIdx.x * d;
    float ss = 0.f;
    for (int j = threadIdx.x; j < d; j += 256) {
        const float v = to_f(x[base + j]) + y[base + j];
        ss = fmaf(v, v, ss);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += part[w];
    const float inv = rsqrtf(tot * inv_d);
    for (int j = threadIdx.x; j < d; j += 256) {
        const float v = (to_f(x[base + j]) + y[base + j]) * inv;
        const T r = from_f<T>(v);
        x_next[base + j] = r;
        if (x_dump) x_dump[base + j] = r;
    }
}

static size_t align256(size_t b) { return (b + 255) & ~(size_t)255; }

// layer scratch (status word + h) | three y buffers | two x buffers (ping-pong)
size_t decode_stack_batched_workspace_bytes(int batch, int d_model, int K_max)
{
    return align256(kCtrlBytesB + (size_t)batch * K_max * sizeof(float)) + 5 * align256((size_t)batch * d_model * sizeof(float));
}

// The stack for 2..8 sequences.  Outputs as in the batch-1 stack: y_layers / x_layers
// [L][batch][d_model] when given.  Where the tensor-core kernel serves every layer the whole
// stack is one persistent launch (decode_batch_mma.cu); otherwise per layer one batched FFN call
// and one glue launch.
coreinfer_status decode_stack_batched(const coreinfer_layer* layers, int L, const void* x0, int batch,
                                      coreinfer_dtype dtype, coreinfer_ffn_kind kind, int d_model, float* y_last,
                                      float* y_layers, void* x_layers, void* workspace, size_t workspace_bytes,
                                      cudaStream_t st)
{
    int Kmax = 0;
    for (int l = 0; l < L; ++l) Kmax = layers[l].K > Kmax ? layers[l].K : Kmax;
    const size_t need = decode_stack_batched_workspace_bytes(batch, d_model, Kmax);
    if (!workspace || !aligned16(workspace)) CI_FAIL(COREINFER_ERR_WORKSPACE, "workspace is NULL or misaligned");
    if (workspace_bytes < need)
        CI_FAIL(COREINFER_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, need);
    const size_t esize = dtype_size(dtype);
    const size_t row = (size_t)batch * d_model;
    const size_t ybytes = align256(row * sizeof(float));
    uint8_t* w = (uint8_t*)workspace;
    uint8_t* y0 = w + align256(kCtrlBytesB + (size_t)batch * Kmax * sizeof(float));
    float* ybuf = (float*)y0;                                    // three buffers, ybytes apart
    uint8_t* xbuf[2] = {y0 + 3 * ybytes, y0 + 4 * ybytes};
    const bool gated = kind_gated(kind);
    const int silu = kind == COREINFER_FFN_SILU_GATED;

    DeviceInfo di;
    coreinfer_status s = device_info(&di);
    if (s != COREINFER_OK) return s;
    bool one_launch = dtype == COREINFER_BF16 && ybytes == row * sizeof(float);
    for (int l = 0; l < L && one_launch; ++l) one_launch = decode_batched_mma_serves(d_model, layers[l].K, di);

    CI_CUDA(cudaMemsetAsync(workspace, 0, kCtrlBytesB, st));      // status word (sticky over the layers), barrier counter
    if (x_layers) CI_CUDA(cudaMemcpyAsync(x_layers, x0, row * esize, cudaMemcpyDeviceToDevice, st));

    if (one_launch) {
        // what the kernel adds into before it can have cleared it itself
        if (y_layers) CI_CUDA(cudaMemsetAsync(y_layers, 0, (size_t)L * row * sizeof(float), st));
        CI_CUDA(cudaMemsetAsync(y_last, 0, row * sizeof(float), st));
        CI_CUDA(cudaMemsetAsync(ybuf, 0, 2 * ybytes, st));
        s = decode_stack_batched_mma(layers, L, x0, batch, gated, silu, d_model, y_last, y_layers, x_layers, ybuf,
                                     (unsigned*)workspace, di, st);
        if (s != COREINFER_ERR_UNSUPPORTED) {
            if (s != COREINFER_OK) return s;
            if (y_layers)
                CI_CUDA(cudaMemcpyAsync(y_last, y_layers + (size_t)(L - 1) * row, row * sizeof(float),
                                        cudaMemcpyDeviceToDevice, st));
            return COREINFER_OK;
        }
    }

    const void* x_in = x0;
    for (int l = 0; l < L; ++l) {
        const bool last = (l == L - 1);
        float* y_out = y_layers ? y_layers + (size_t)l * row : (last ? y_last : ybuf);
        s = decode_batched(x_in, batch, dtype, kind, d_model, layers[l], y_out, workspace, st, false);
        if (s != COREINFER_OK) return s;
        if (last) {
            if (y_out != y_last) CI_CUDA(cudaMemcpyAsync(y_last, y_out, row * sizeof(float), cudaMemcpyDeviceToDevice, st));
            break;
        }
        void* x_next = xbuf[l & 1];
        void* dump = x_layers ? (void*)((uint8_t*)x_layers + (size_t)(l + 1) * row * esize) : nullptr;
        if (dtype == COREINFER_BF16)
            batch_glue_kernel<__nv_bfloat16><<<batch, 256, 0, st>>>((const __nv_bfloat16*)x_in, y_out, (__nv_bfloat16*)x_next,
                                                                   (__nv_bfloat16*)dump, d_model, 1.0f / (float)d_model);
        else if (dtype == COREINFER_F16)
            batch_glue_kernel<__half><<<batch, 256, 0, st>>>((const __half*)x_in, y_out, (__half*)x_next, (__half*)dump,
                                                            d_model, 1.0f / (float)d_model);
        else
            batch_glue_kernel<float><<<batch, 256, 0, st>>>((const float*)x_in, y_out, (float*)x_next, (float*)dump,
                                                           d_model, 1.0f / (float)d_model);
        CI_CUDA(cudaGetLastError());
        x_in = x_next;
    }
    return COREINFER_OK;
}

}  // namespace coreinfer
