// Dense FFN on the uncompacted weights: the pre-fill pass whose intermediate activations
// are ranked by Definition 1.  Reference-quality register-tiled kernels on the fp32 pipes
// (exact products of fp32 or bf16 inputs, fp32 sums):
//   up:   H[T, N] = act(X[T, d] . W_up[N, d]^T (+ b_up))   or   relu(X . W_gate^T) * (X . W_up^T)
//   down: Y[T, d] = H[T, N] . W_down[d, N]^T + b_down       (H read back as stored fp32)
// Both are "A row-major times B row-major transposed" contractions over the inner index.
#include "common.cuh"

namespace coreinfer {

constexpr int kBM = 128, kBN = 64, kBK = 16;
constexpr int kGemmThreads = 256;

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <> __device__ __forceinline__ float to_f32<__half>(__half v) { return __half2float(v); }

// C[M, Nn] = epilogue(A[M, Kk] . B[Nn, Kk]^T).  GATED: a second B matrix (the gate) and
// C = max(A.Bg^T, 0) * (A.B^T); otherwise C = A.B^T + bias[n], with ReLU if RELU.
template <typename TA, typename TB, bool GATED, bool RELU>
__global__ void __launch_bounds__(kGemmThreads)
gemm_nt_kernel(const TA* __restrict__ A, const TB* __restrict__ B, const TB* __restrict__ Bg,
               const TB* __restrict__ bias, float* __restrict__ C, int M, int Nn, int Kk, int silu)
{
    __shared__ float As[kBK][kBM + 4];
    __shared__ float Bs[kBK][kBN + 4];
    __shared__ float Gs[GATED ? kBK : 1][kBN + 4];
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const int m0 = blockIdx.y * kBM, n0 = blockIdx.x * kBN;
    float acc[8][4], accg[GATED ? 8 : 1][4];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) { acc[i][j] = 0.f; if (GATED) accg[i][j] = 0.f; }

    const int lk = tid & 15;        // inner index within the tile
    const int lr = tid >> 4;        // 0..15: row within a 16-row slice
    for (int k0 = 0; k0 < Kk; k0 += kBK) {
        const int k = k0 + lk;
#pragma unroll
        for (int r = 0; r < kBM / 16; ++r) {
            const int m = m0 + lr + r * 16;
            As[lk][lr + r * 16] = (m < M && k < Kk) ? to_f32<TA>(A[(size_t)m * Kk + k]) : 0.f;
        }
#pragma unroll
        for (int r = 0; r < kBN / 16; ++r) {
            const int n = n0 + lr + r * 16;
            const bool ok = n < Nn && k < Kk;
            Bs[lk][lr + r * 16] = ok ? to_f32<TB>(B[(size_t)n * Kk + k]) : 0.f;
            if (GATED) Gs[lk][lr + r * 16] = ok ? to_f32<TB>(Bg[(size_t)n * Kk + k]) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < kBK; ++kk) {
            float a[8], b[4], g[4];
            const float4 a0 = *reinterpret_cast<const float4*>(&As[kk][ty * 8]);
            const float4 a1 = *reinterpret_cast<const float4*>(&As[kk][ty * 8 + 4]);
            a[0] = a0.x; a[1] = a0.y; a[2] = a0.z; a[3] = a0.w;
            a[4] = a1.x; a[5] = a1.y; a[6] = a1.z; a[7] = a1.w;
            const float4 b0 = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
            b[0] = b0.x; b[1] = b0.y; b[2] = b0.z; b[3] = b0.w;
            if (GATED) {
                const float4 g0 = *reinterpret_cast<const float4*>(&Gs[kk][tx * 4]);
                g[0] = g0.x; g[1] = g0.y; g[2] = g0.z; g[3] = g0.w;
            }
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
                    if (GATED) accg[i][j] = fmaf(a[i], g[j], accg[i][j]);
                }
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int m = m0 + ty * 8 + i;
        if (m >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx * 4 + j;
            if (n >= Nn) continue;
            float v;
            if (GATED) {
                v = gate_activation(accg[i][j], silu) * acc[i][j];
            } else {
                v = acc[i][j] + (bias ? to_f32<TB>(bias[n]) : 0.f);
                if (RELU) v = fmaxf(v, 0.f);
            }
            C[(size_t)m * Nn + n] = v;
        }
    }
}

template <typename T>
static coreinfer_status dense_t(const void* x, int T_, bool gated, int silu, int d, int N, const void* w_up,
                                const void* w_gate, const void* w_down, const void* b_up, const void* b_down,
                                float* h_out, float* y_out, cudaStream_t st)
{
    if (h_out) {
        dim3 grid((N + kBN - 1) / kBN, (T_ + kBM - 1) / kBM);
        if (gated)
            gemm_nt_kernel<T, T, true, false><<<grid, kGemmThreads, 0, st>>>(
                (const T*)x, (const T*)w_up, (const T*)w_gate, nullptr, h_out, T_, N, d, silu);
        else
            gemm_nt_kernel<T, T, false, true><<<grid, kGemmThreads, 0, st>>>(
                (const T*)x, (const T*)w_up, nullptr, (const T*)b_up, h_out, T_, N, d, 0);
        CI_CUDA(cudaGetLastError());
    }
    if (y_out) {
        dim3 grid((d + kBN - 1) / kBN, (T_ + kBM - 1) / kBM);
        gemm_nt_kernel<float, T, false, false><<<grid, kGemmThreads, 0, st>>>(
            h_out, (const T*)w_down, nullptr, (const T*)b_down, y_out, T_, d, N, 0);
        CI_CUDA(cudaGetLastError());
    }
    return COREINFER_OK;
}

}  // namespace coreinfer

using namespace coreinfer;

extern "C" coreinfer_status coreinfer_ffn_dense_ref(const void* x, int32_t T, coreinfer_dtype dtype,
                                                    coreinfer_ffn_kind kind, int32_t d_model, int32_t d_ff,
                                                    const void* w_up, const void* w_gate, const void* w_down,
                                                    const void* b_up, const void* b_down, float* h_out,
                                                    float* y_out, void* cuda_stream)
{
    if (!dtype_known(dtype)) CI_FAIL(COREINFER_ERR_UNSUPPORTED, "dtype %d is not supported", (int)dtype);
    if (!kind_known(kind)) CI_FAIL(COREINFER_ERR_UNSUPPORTED, "ffn kind %d is not supported", (int)kind);
    const bool gated = kind_gated(kind);
    const int silu = kind == COREINFER_FFN_SILU_GATED;
    if (T < 1 || d_model < 1 || d_ff < 1)
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "T = %d, d_model = %d, d_ff = %d must be >= 1", T, d_model, d_ff);
    if (!x || !w_up || !w_down) CI_FAIL(COREINFER_ERR_INVALID_ARG, "x / w_up / w_down is NULL");
    if (gated != (w_gate != nullptr))
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "w_gate must be given for the gated FFN and only for it");
    if (gated && b_up) CI_FAIL(COREINFER_ERR_INVALID_ARG, "the gated FFN has no up bias");
    if (y_out && !h_out) CI_FAIL(COREINFER_ERR_INVALID_ARG, "y_out needs h_out (y is computed from the stored h)");
    if (!h_out) return COREINFER_OK;   // nothing asked for
    DeviceInfo di;
    coreinfer_status s = device_info(&di);
    if (s != COREINFER_OK) return s;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (dtype == COREINFER_BF16)
        return dense_t<__nv_bfloat16>(x, T, gated, silu, d_model, d_ff, w_up, w_gate, w_down, b_up, b_down, h_out,
                                      y_out, st);
    if (dtype == COREINFER_F16)
        return dense_t<__half>(x, T, gated, silu, d_model, d_ff, w_up, w_gate, w_down, b_up, b_down, h_out, y_out, st);
    return dense_t<float>(x, T, gated, silu, d_model, d_ff, w_up, w_gate, w_down, b_up, b_down, h_out, y_out, st);
}
