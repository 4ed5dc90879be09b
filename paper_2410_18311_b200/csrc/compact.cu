// One-shot weight compaction after pre-fill (Section 5.3: only the selected neurons are
// deployed for decoding).  Pure byte movement.
//   rows:    w_up_c[k, :]   = w_up[S[k], :]   (and the same for w_gate)   -- 16-byte vector copies
//   columns: w_downT_c[k, j] = w_down[j, S[k]]                             -- tiled transpose:
//            a CTA reads a [64 rows j] x [64 selected columns] patch with the selected
//            columns varying fastest across lanes (ascending indices, so neighbouring lanes
//            hit neighbouring sectors), turns it in shared memory and writes 64-element
//            contiguous runs of the output rows.
#include "common.cuh"

namespace coreinfer {

constexpr int kTile = 64;

__global__ void __launch_bounds__(256)
gather_rows_kernel(const uint4* __restrict__ w_up, const uint4* __restrict__ w_gate,
                   const int32_t* __restrict__ S, uint4* __restrict__ up_c, uint4* __restrict__ gate_c,
                   int nv)
{
    const int k = blockIdx.x;
    const size_t n = (size_t)S[k];
    const uint4* src = (blockIdx.y == 0 ? w_up : w_gate) + n * nv;
    uint4* dst = (blockIdx.y == 0 ? up_c : gate_c) + (size_t)k * nv;
    for (int v = threadIdx.x; v < nv; v += blockDim.x) dst[v] = __ldcs(&src[v]);
}

template <typename U>
__global__ void __launch_bounds__(256)
gather_elems_kernel(const U* __restrict__ b, const int32_t* __restrict__ S, U* __restrict__ b_c, int K)
{
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k < K) b_c[k] = b[S[k]];
}

template <typename U>
__global__ void __launch_bounds__(256)
gather_cols_T_kernel(const U* __restrict__ w_down, const int32_t* __restrict__ S, U* __restrict__ downT_c,
                     int d, int N, int K)
{
    constexpr int PAD = sizeof(U) == 2 ? 2 : 1;     // odd word stride between tile rows
    __shared__ U tile[kTile][kTile + PAD];
    __shared__ int32_t cols[kTile];
    const int k0 = blockIdx.x * kTile;
    const int j0 = blockIdx.y * kTile;
    const int tx = threadIdx.x & (kTile - 1);
    const int ty = threadIdx.x / kTile;              // 0..3
    if (threadIdx.x < kTile) cols[threadIdx.x] = (k0 + threadIdx.x < K) ? S[k0 + threadIdx.x] : -1;
    __syncthreads();
    const int col = cols[tx];
#pragma unroll 4
    for (int jj = ty; jj < kTile; jj += 4) {
        const int j = j0 + jj;
        if (col >= 0 && j < d) tile[tx][jj] = w_down[(size_t)j * N + col];
    }
    __syncthreads();
#pragma unroll 4
    for (int kk = ty; kk < kTile; kk += 4) {
        const int k = k0 + kk, j = j0 + tx;
        if (k < K && j < d) downT_c[(size_t)k * d + j] = tile[kk][tx];
    }
}

__global__ void verify_init_kernel(int32_t* report)
{
    report[0] = 0;
    report[1] = 0x7fffffff;
}

// report[0]: number of positions k whose index is out of [0, d_ff) or not above its predecessor;
// report[1]: the first such position (INT_MAX while there is none).
__global__ void verify_core_idx_kernel(const int32_t* __restrict__ idx, int K, int d_ff, int32_t* report)
{
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= K) return;
    const int32_t v = idx[k];
    const bool bad = v < 0 || v >= d_ff || (k > 0 && idx[k - 1] >= v);
    if (bad) {
        atomicAdd(&report[0], 1);
        atomicMin(&report[1], k);
    }
}

}  // namespace coreinfer

using namespace coreinfer;

extern "C" coreinfer_status coreinfer_verify_core_idx(const int32_t* core_idx, int32_t K, int32_t d_ff,
                                                      int32_t* report, void* cuda_stream)
{
    if (!core_idx || !report) CI_FAIL(COREINFER_ERR_INVALID_ARG, "core_idx / report is NULL");
    if (d_ff < 1 || K < 1 || K > d_ff) CI_FAIL(COREINFER_ERR_INVALID_ARG, "K = %d outside 1..d_ff (%d)", K, d_ff);
    DeviceInfo di;
    coreinfer_status s = device_info(&di);
    if (s != COREINFER_OK) return s;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    verify_init_kernel<<<1, 1, 0, st>>>(report);
    CI_CUDA(cudaGetLastError());
    verify_core_idx_kernel<<<(K + 255) / 256, 256, 0, st>>>(core_idx, K, d_ff, report);
    CI_CUDA(cudaGetLastError());
    return COREINFER_OK;
}

extern "C" coreinfer_status coreinfer_compact(const void* w_up, const void* w_gate, const void* w_down,
                                              const void* b_up, coreinfer_dtype dtype, int32_t d_model,
                                              int32_t d_ff, const int32_t* core_idx, int32_t K,
                                              void* w_up_c, void* w_gate_c, void* w_downT_c, void* b_up_c,
                                              void* cuda_stream)
{
    if (!dtype_known(dtype)) CI_FAIL(COREINFER_ERR_UNSUPPORTED, "dtype %d is not supported", (int)dtype);
    const size_t es = dtype_size(dtype);
    if (d_model < 1 || d_ff < 1 || ((size_t)d_model * es) % 16 != 0)
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "d_model %d / d_ff %d: a weight row must be a positive multiple of 16 bytes",
                d_model, d_ff);
    if (K < 1 || K > d_ff) CI_FAIL(COREINFER_ERR_INVALID_ARG, "K = %d outside 1..d_ff (%d)", K, d_ff);
    if (!w_up || !w_down || !core_idx || !w_up_c || !w_downT_c)
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "a required pointer is NULL");
    if ((w_gate == nullptr) != (w_gate_c == nullptr))
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "w_gate and w_gate_c must both be given or both be NULL");
    if ((b_up == nullptr) != (b_up_c == nullptr))
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "b_up and b_up_c must both be given or both be NULL");
    if (!aligned16(w_up) || !aligned16(w_up_c) || !aligned16(w_downT_c) || !aligned16(w_down) ||
        (w_gate && (!aligned16(w_gate) || !aligned16(w_gate_c))))
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "weight pointers must be 16-byte aligned");
    DeviceInfo di;
    coreinfer_status s = device_info(&di);
    if (s != COREINFER_OK) return s;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int nv = (int)((size_t)d_model * es / 16);

    gather_rows_kernel<<<dim3((unsigned)K, w_gate ? 2u : 1u), 256, 0, st>>>(
        (const uint4*)w_up, (const uint4*)w_gate, core_idx, (uint4*)w_up_c, (uint4*)w_gate_c, nv);
    CI_CUDA(cudaGetLastError());
    dim3 grid((unsigned)((K + kTile - 1) / kTile), (unsigned)((d_model + kTile - 1) / kTile));
    if (es == 2) {
        gather_cols_T_kernel<uint16_t><<<grid, 256, 0, st>>>((const uint16_t*)w_down, core_idx,
                                                             (uint16_t*)w_downT_c, d_model, d_ff, K);
        CI_CUDA(cudaGetLastError());
        if (b_up) {
            gather_elems_kernel<uint16_t><<<(K + 255) / 256, 256, 0, st>>>((const uint16_t*)b_up, core_idx,
                                                                          (uint16_t*)b_up_c, K);
            CI_CUDA(cudaGetLastError());
        }
    } else {
        gather_cols_T_kernel<uint32_t><<<grid, 256, 0, st>>>((const uint32_t*)w_down, core_idx,
                                                             (uint32_t*)w_downT_c, d_model, d_ff, K);
        CI_CUDA(cudaGetLastError());
        if (b_up) {
            gather_elems_kernel<uint32_t><<<(K + 255) / 256, 256, 0, st>>>((const uint32_t*)b_up, core_idx,
                                                                          (uint32_t*)b_up_c, K);
            CI_CUDA(cudaGetLastError());
        }
    }
    return COREINFER_OK;
}
