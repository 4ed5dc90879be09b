// Core sets over several sentences: what Section 3.2 (Insight-1: stability, Insight-2:
// similarity) and Section 4.1 (similarity-guided prediction) build on top of Definition 2.
//   - count vectors add up (Eq. 3 is a sum over tokens; a semantic group counts in how many of
//     its sentences' core sets a neuron appears), and the set is the top fraction by count;
//   - the similarity of two sets is |shared| / |involved|;
//   - an input joins the semantic group whose centroid is nearest;
//   - a deployed set can be changed in place: only the rows whose neuron leaves are rewritten.
// All integer work except the centroid distances (double sums in a fixed order).
#include "common.cuh"

namespace coreinfer {

coreinfer_status launch_select_top(const int32_t* f, int N, int K, int max_count, int32_t* S, const DeviceInfo& di,
                                   cudaStream_t st);     // select.cu

__global__ void counts_add_kernel(int32_t* __restrict__ acc, const int32_t* __restrict__ f, int n)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) acc[i] += f[i];
}

// the members of one set are distinct, so no two threads touch the same counter
__global__ void counts_add_set_kernel(int32_t* __restrict__ acc, const int32_t* __restrict__ S, int K, int N)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= K) return;
    const int32_t n = S[i];
    if (n >= 0 && n < N) acc[n] += 1;
}

// is v a member of the ascending list A[0 .. K)?
__device__ __forceinline__ bool in_sorted(const int32_t* A, int K, int32_t v)
{
    int lo = 0, hi = K;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (A[mid] < v) lo = mid + 1; else hi = mid;
    }
    return lo < K && A[lo] == v;
}

__global__ void set_pair_kernel(int32_t* out, int32_t a, int32_t b)
{
    out[0] = a;
    out[1] = b;
}

// out[0] += number of members of B found in A (A ascending), out[1] -= the same; on entry
// out = (0, KA + KB).
__global__ void similarity_kernel(const int32_t* __restrict__ A, int KA, const int32_t* __restrict__ B, int KB,
                                  int32_t* out)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    const bool hit = i < KB && in_sorted(A, KA, B[i]);
    const unsigned m = __ballot_sync(0xffffffffu, hit);
    if ((threadIdx.x & 31) == 0 && m) {
        const int c = __popc(m);
        atomicAdd(&out[0], c);
        atomicSub(&out[1], c);
    }
}

// One warp per centroid: squared Euclidean distance in double, lanes take elements lane, lane + 32,
// ...; the 32 partial sums are added in a fixed tree.  One more kernel picks the smallest
// (equal distances: lower group).
__global__ void centroid_dist_kernel(const float* __restrict__ C, int G, int D, const float* __restrict__ v,
                                     double* __restrict__ dist2)
{
    const int g = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (g >= G) return;
    double s = 0.0;
    for (int i = lane; i < D; i += 32) {
        const double t = (double)v[i] - (double)C[(size_t)g * D + i];
        s = fma(t, t, s);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) dist2[g] = s;
}

__global__ void centroid_argmin_kernel(const double* __restrict__ dist2, int G, int32_t* __restrict__ group)
{
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    int best = 0;
    double bd = dist2[0];
    for (int g = 1; g < G; ++g)
        if (dist2[g] < bd) { bd = dist2[g]; best = g; }
    *group = best;
}

// One CTA.  flags: [d_ff] bytes of scratch.  slot_neuron[K] (any order) -> which slots hold a
// neuron outside S_new (ascending), which members of S_new are not held; pair them in ascending
// slot / ascending neuron order, record the pairs and update slot_neuron.
constexpr int kDeltaThreads = 1024;

__device__ __forceinline__ int delta_block_scan(int v, int* warp_tot, int* total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = warp_tot[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, w, o);
            if (lane >= o) w += t;
        }
        warp_tot[lane] = w;
    }
    __syncthreads();
    const int base = warp > 0 ? warp_tot[warp - 1] : 0;
    *total = warp_tot[31];
    __syncthreads();
    return base + incl - v;
}

__global__ void __launch_bounds__(kDeltaThreads, 1)
set_delta_kernel(int32_t* __restrict__ slot_neuron, int K, const int32_t* __restrict__ S_new, int N,
                 uint8_t* __restrict__ flags, int32_t* __restrict__ slots, int32_t* __restrict__ neurons,
                 int32_t* __restrict__ n_changed)
{
    __shared__ int warp_tot[32];
    const int tid = threadIdx.x;
    for (int i = tid; i < N; i += kDeltaThreads) flags[i] = 0;
    __syncthreads();
    for (int p = tid; p < K; p += kDeltaThreads) {
        const int32_t n = slot_neuron[p];
        if (n >= 0 && n < N) flags[n] = 1;                      // held now
    }
    __syncthreads();
    // contiguous runs per thread keep the pairing in ascending order
    const int per = (K + kDeltaThreads - 1) / kDeltaThreads;
    const int p0 = min(tid * per, K), p1 = min(p0 + per, K);
    int leave = 0, enter = 0;
    for (int p = p0; p < p1; ++p) {
        leave += in_sorted(S_new, K, slot_neuron[p]) ? 0 : 1;
        const int32_t n = S_new[p];
        enter += (n >= 0 && n < N && flags[n]) ? 0 : 1;
    }
    int tot_leave, tot_enter;
    int li = delta_block_scan(leave, warp_tot, &tot_leave);
    int ei = delta_block_scan(enter, warp_tot, &tot_enter);
    for (int p = p0; p < p1; ++p) {
        if (!in_sorted(S_new, K, slot_neuron[p])) slots[li++] = p;
        const int32_t n = S_new[p];
        if (!(n >= 0 && n < N && flags[n])) neurons[ei++] = n;
    }
    __syncthreads();
    __threadfence_block();
    const int nch = min(tot_leave, tot_enter);                  // equal for two sets of K distinct members
    for (int i = tid; i < nch; i += kDeltaThreads) slot_neuron[slots[i]] = neurons[i];
    if (tid == 0) *n_changed = nch;
}

// Rows of the compacted buffers listed in `slots` are refilled with the weights of `neurons`;
// the number of pairs is read from device memory, blocks beyond it return at once.
template <typename E>
__global__ void __launch_bounds__(256)
compact_rows_kernel(const uint4* __restrict__ w_up, const uint4* __restrict__ w_gate, const E* __restrict__ w_down,
                    const E* __restrict__ b_up, const int32_t* __restrict__ slots, const int32_t* __restrict__ neurons,
                    const int32_t* __restrict__ n_changed, uint4* __restrict__ up_c, uint4* __restrict__ gate_c,
                    E* __restrict__ down_c, E* __restrict__ bup_c, int nv, int d_model, int d_ff, int K)
{
    const int i = blockIdx.x;
    if (i >= *n_changed) return;
    const int p = slots[i];
    const int n = neurons[i];
    if (p < 0 || p >= K || n < 0 || n >= d_ff) return;
    for (int v = threadIdx.x; v < nv; v += 256) {
        up_c[(size_t)p * nv + v] = w_up[(size_t)n * nv + v];
        if (w_gate) gate_c[(size_t)p * nv + v] = w_gate[(size_t)n * nv + v];
    }
    for (int j = threadIdx.x; j < d_model; j += 256) down_c[(size_t)p * d_model + j] = w_down[(size_t)j * d_ff + n];
    if (b_up && threadIdx.x == 0) bup_c[p] = b_up[n];
}

}  // namespace coreinfer

using namespace coreinfer;

extern "C" {

coreinfer_status coreinfer_counts_add(int32_t* counts, const int32_t* f, int32_t d_ff, void* cuda_stream)
{
    if (!counts || !f || d_ff < 1) CI_FAIL(COREINFER_ERR_INVALID_ARG, "counts / f NULL or d_ff < 1");
    DeviceInfo di;
    coreinfer_status s = device_info(&di);
    if (s != COREINFER_OK) return s;
    counts_add_kernel<<<(d_ff + 255) / 256, 256, 0, (cudaStream_t)cuda_stream>>>(counts, f, d_ff);
    CI_CUDA(cudaGetLastError());
    return COREINFER_OK;
}

coreinfer_status coreinfer_counts_add_set(int32_t* counts, const int32_t* core_idx, int32_t K, int32_t d_ff,
                                          void* cuda_stream)
{
    if (!counts || !core_idx) CI_FAIL(COREINFER_ERR_INVALID_ARG, "counts / core_idx is NULL");
    if (d_ff < 1 || K < 1 || K > d_ff) CI_FAIL(COREINFER_ERR_INVALID_ARG, "K = %d outside 1..d_ff (%d)", K, d_ff);
    DeviceInfo di;
    coreinfer_status s = device_info(&di);
    if (s != COREINFER_OK) return s;
    counts_add_set_kernel<<<(K + 255) / 256, 256, 0, (cudaStream_t)cuda_stream>>>(counts, core_idx, K, d_ff);
    CI_CUDA(cudaGetLastError());
    return COREINFER_OK;
}

coreinfer_status coreinfer_top_by_count(const int32_t* counts, int32_t d_ff, int32_t max_count, double frac,
                                        int32_t* core_idx, void* cuda_stream)
{
    if (!counts || !core_idx) CI_FAIL(COREINFER_ERR_INVALID_ARG, "counts / core_idx is NULL");
    if (d_ff < 1 || max_count < 0) CI_FAIL(COREINFER_ERR_INVALID_ARG, "d_ff = %d, max_count = %d", d_ff, max_count);
    if (!(frac > 0.0 && frac <= 1.0)) CI_FAIL(COREINFER_ERR_INVALID_ARG, "frac = %g must lie in (0, 1]", frac);
    const int K = coreinfer_count(frac, d_ff);
    if (K < 1) CI_FAIL(COREINFER_ERR_INVALID_ARG, "frac = %g selects no neuron of d_ff = %d", frac, d_ff);
    DeviceInfo di;
    coreinfer_status s = device_info(&di);
    if (s != COREINFER_OK) return s;
    return launch_select_top(counts, d_ff, K, max_count, core_idx, di, (cudaStream_t)cuda_stream);
}

coreinfer_status coreinfer_core_similarity(const int32_t* set_a, int32_t K_a, const int32_t* set_b, int32_t K_b,
                                           int32_t* shared_involved, void* cuda_stream)
{
    if (!set_a || !set_b || !shared_involved) CI_FAIL(COREINFER_ERR_INVALID_ARG, "a pointer is NULL");
    if (K_a < 1 || K_b < 1) CI_FAIL(COREINFER_ERR_INVALID_ARG, "K_a = %d, K_b = %d must be >= 1", K_a, K_b);
    DeviceInfo di;
    coreinfer_status s = device_info(&di);
    if (s != COREINFER_OK) return s;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    set_pair_kernel<<<1, 1, 0, st>>>(shared_involved, 0, K_a + K_b);
    CI_CUDA(cudaGetLastError());
    similarity_kernel<<<(K_b + 255) / 256, 256, 0, st>>>(set_a, K_a, set_b, K_b, shared_involved);
    CI_CUDA(cudaGetLastError());
    return COREINFER_OK;
}

size_t coreinfer_nearest_centroid_workspace_bytes(int32_t G) { return G < 1 ? 0 : (size_t)G * sizeof(double); }

coreinfer_status coreinfer_nearest_centroid(const float* centroids, int32_t G, int32_t D, const float* v,
                                            int32_t* group_out, void* workspace, size_t workspace_bytes,
                                            void* cuda_stream)
{
    if (!centroids || !v || !group_out) CI_FAIL(COREINFER_ERR_INVALID_ARG, "a pointer is NULL");
    if (G < 1 || D < 1) CI_FAIL(COREINFER_ERR_INVALID_ARG, "G = %d, D = %d must be >= 1", G, D);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 7u))
        CI_FAIL(COREINFER_ERR_WORKSPACE, "workspace is NULL or not 8-byte aligned");
    if (workspace_bytes < coreinfer_nearest_centroid_workspace_bytes(G))
        CI_FAIL(COREINFER_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes,
                coreinfer_nearest_centroid_workspace_bytes(G));
    DeviceInfo di;
    coreinfer_status s = device_info(&di);
    if (s != COREINFER_OK) return s;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    centroid_dist_kernel<<<(G + 7) / 8, 256, 0, st>>>(centroids, G, D, v, (double*)workspace);
    CI_CUDA(cudaGetLastError());
    centroid_argmin_kernel<<<1, 32, 0, st>>>((const double*)workspace, G, group_out);
    CI_CUDA(cudaGetLastError());
    return COREINFER_OK;
}

size_t coreinfer_update_core_set_workspace_bytes(int32_t d_ff, int32_t K)
{
    if (d_ff < 1 || K < 1) return 0;
    return (((size_t)d_ff + 255) & ~(size_t)255) + 2 * (((size_t)K * sizeof(int32_t) + 255) & ~(size_t)255) + 256;
}

coreinfer_status coreinfer_update_core_set(const void* w_up, const void* w_gate, const void* w_down, const void* b_up,
                                           coreinfer_dtype dtype, int32_t d_model, int32_t d_ff,
                                           int32_t* slot_neuron, const int32_t* core_idx_new, int32_t K,
                                           void* w_up_c, void* w_gate_c, void* w_downT_c, void* b_up_c,
                                           int32_t* n_changed_out, void* workspace, size_t workspace_bytes,
                                           void* cuda_stream)
{
    if (!dtype_known(dtype)) CI_FAIL(COREINFER_ERR_UNSUPPORTED, "dtype %d is not supported", (int)dtype);
    const size_t es = dtype_size(dtype);
    if (d_model < 1 || d_ff < 1 || ((size_t)d_model * es) % 16 != 0)
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "d_model %d / d_ff %d: a weight row must be a positive multiple of 16 bytes",
                d_model, d_ff);
    if (K < 1 || K > d_ff) CI_FAIL(COREINFER_ERR_INVALID_ARG, "K = %d outside 1..d_ff (%d)", K, d_ff);
    if (!w_up || !w_down || !slot_neuron || !core_idx_new || !w_up_c || !w_downT_c || !n_changed_out)
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "a required pointer is NULL");
    if ((w_gate == nullptr) != (w_gate_c == nullptr) || (b_up == nullptr) != (b_up_c == nullptr))
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "w_gate / w_gate_c and b_up / b_up_c must be given together");
    if (!aligned16(w_up) || !aligned16(w_up_c) || (w_gate && (!aligned16(w_gate) || !aligned16(w_gate_c))))
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "weight pointers must be 16-byte aligned");
    if (!workspace || !aligned16(workspace)) CI_FAIL(COREINFER_ERR_WORKSPACE, "workspace is NULL or misaligned");
    if (workspace_bytes < coreinfer_update_core_set_workspace_bytes(d_ff, K))
        CI_FAIL(COREINFER_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes,
                coreinfer_update_core_set_workspace_bytes(d_ff, K));
    DeviceInfo di;
    coreinfer_status s = device_info(&di);
    if (s != COREINFER_OK) return s;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    uint8_t* flags = (uint8_t*)workspace;
    const size_t kb = ((size_t)K * sizeof(int32_t) + 255) & ~(size_t)255;
    int32_t* slots = (int32_t*)(flags + (((size_t)d_ff + 255) & ~(size_t)255));
    int32_t* neurons = (int32_t*)((uint8_t*)slots + kb);
    set_delta_kernel<<<1, kDeltaThreads, 0, st>>>(slot_neuron, K, core_idx_new, d_ff, flags, slots, neurons, n_changed_out);
    CI_CUDA(cudaGetLastError());
    const int nv = (int)((size_t)d_model * es / 16);
    if (es == 2)
        compact_rows_kernel<uint16_t><<<K, 256, 0, st>>>((const uint4*)w_up, (const uint4*)w_gate, (const uint16_t*)w_down,
                                                         (const uint16_t*)b_up, slots, neurons, n_changed_out, (uint4*)w_up_c,
                                                         (uint4*)w_gate_c, (uint16_t*)w_downT_c, (uint16_t*)b_up_c, nv,
                                                         d_model, d_ff, K);
    else
        compact_rows_kernel<uint32_t><<<K, 256, 0, st>>>((const uint4*)w_up, (const uint4*)w_gate, (const uint32_t*)w_down,
                                                         (const uint32_t*)b_up, slots, neurons, n_changed_out, (uint4*)w_up_c,
                                                         (uint4*)w_gate_c, (uint32_t*)w_downT_c, (uint32_t*)b_up_c, nv,
                                                         d_model, d_ff, K);
    CI_CUDA(cudaGetLastError());
    return COREINFER_OK;
}

}  // extern "C"
