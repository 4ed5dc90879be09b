// Pre-fill activations on the tensor cores: A = act(X W_up^T (+ b_up)), or gated
// A = gate(X W_gate^T) * (X W_up^T), gate = ReLU or SiLU: the [T, d_ff] tensor that Definition 1 ranks (the paper
// obtains it as a by-product of the dense pre-fill pass, Section 4.2 / Fig. 1).  bf16 or fp16 inputs,
// exact products, fp32 accumulation in tensor memory, fp32 output.
//
// One persistent CTA per SM walks output tiles of 128 prompt rows x 256 neurons (128 when gated).  Warp 0 (one lane) feeds a ring of
// shared-memory stages with 2-D tensor copies (128-byte swizzle, each stage a 128 x 64 slice of X
// and a 256 (128) x 64 slice of each weight matrix); warp 1 (one lane) issues tcgen05.mma (M 128, N 256 or 128, K 16, four per
// stage and matrix) into one of two accumulator sets in tensor memory and hands stages back
// through tcgen05.commit; warps 2..5 read a finished accumulator set (tcgen05.ld, 32 columns at a
// time, each thread one output row), apply bias / ReLU / gate product and store, while the MMA
// warp already works on the next tile.  Rows and neurons beyond the matrix edges are zero-filled
// by the tensor copies and masked in the epilogue.  Every wait is bounded; a wait that gives up
// sets the status word, and all roles leave their loops, drain, free tensor memory and return.
#include "common.cuh"

#include <cuda.h>

namespace coreinfer {

constexpr int kTcBM = 128;                 // prompt rows per tile
// Neurons per tile: up to 256 (the widest MMA) where one weight matrix is multiplied, up to 128
// where the gate matrix doubles the accumulators; the two accumulator sets sit 256 columns apart
// in tensor memory and the gate's accumulator 128 columns after the up projection's.  The host
// picks the width per call (a multiple of 32) so that the tiles fill whole waves of SMs.
constexpr int kTcMaxBN = 256;
constexpr int kTcMaxBNGated = 128;
constexpr uint32_t kTcAccStride = 256;     // tensor-memory columns between the two accumulator sets
constexpr uint32_t kTcGateOfs = 128;       // columns between the two accumulators of a gated set
constexpr int kTcBK = 64;                  // reduction slice per stage: 128 bytes of bf16 = one swizzle row
constexpr int kTcUmmaK = 16;
constexpr int kTcThreads = 192;            // warp 0 copies, warp 1 MMA + tensor memory, warps 2..5 epilogue
constexpr int kTcMaxStages = 8;
constexpr uint32_t kTcTileBytes = kTcBM * kTcBK * 2;     // 16 KiB: one 128 x 64 bf16 slice
constexpr long long kTcWaitCycles = 3000000000LL;

struct TcParams {
    int T, N, d;
    int gated;
    int silu;                   // gated: 0 ReLU gate, 1 SiLU gate
    uint32_t idesc;             // tcgen05 instruction descriptor (operand formats, tile shape)
    int stages;
    int tiles_m, tiles_n;
    int bn;                     // neurons per tile
    long long ld_out;           // row stride of `out`, elements
    void* out;                  // [T][ld_out] in the output type
    int out_kind;               // 0 fp32, 1 bf16, 2 fp16 (rounded to nearest even once, after the activation)
    const void* bias;           // [N] in the input type, or NULL (not gated)
    int f16;                    // inputs are fp16 (else bf16)
    unsigned* status;
};

// ---- tcgen05 / tensor-copy wrappers (one PTX instruction each) ----
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]^T, bf16 x bf16 -> fp32, both operands K-major.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}
// The barrier receives one arrival when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 lanes x 32 consecutive fp32 columns: thread i of the warp receives row (lane base + i).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// 2-D tensor copy global -> shared of this CTA (coordinates: c0 along the row, c1 the row), no
// other CTA involved; completion counted in bytes on the barrier.  c0 * 2 bytes is a multiple of 16.
__device__ __forceinline__ void tensor_g2s_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}

// Shared-memory matrix descriptor of a 128 x 64 bf16 slice stored by a 128-byte-swizzled tensor
// copy: rows of 128 bytes, groups of eight rows 1024 bytes apart (stride byte offset), K-major.
__device__ __forceinline__ uint64_t smem_desc_k_sw128(uint32_t addr)
{
    return (uint64_t)((addr >> 4) & 0x3fffu) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}

// Returns false when the wait gave up (status word set, abort flag raised).
__device__ __forceinline__ bool tc_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned* status)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        if (mbar_try_wait_parked(bar, parity, 2000u)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > kTcWaitCycles) {
            *abort_flag = 1;
            atomicMax(status, (unsigned)kStatusTimeout);
            return false;
        }
    }
}

template <bool GATED>
__global__ void __launch_bounds__(kTcThreads, 1)
prefill_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_up,
                  const __grid_constant__ CUtensorMap map_gate, const TcParams p)
{
    constexpr int NB = GATED ? 2 : 1;                          // weight matrices per stage
    const int BN = p.bn;
    const uint32_t W_TILE_BYTES = (uint32_t)BN * kTcBK * 2;    // one weight slice: BN rows of 128 bytes
    const uint32_t STAGE_BYTES = kTcTileBytes + NB * W_TILE_BYTES;
    constexpr uint32_t TMEM_COLS = 2 * kTcAccStride;           // two accumulator sets: all 512 columns
    const uint32_t IDESC = p.idesc;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* tiles = smem;                                                          // [stages][1 + NB][16 KiB]
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(tiles + (size_t)p.stages * STAGE_BYTES);
    uint64_t* empty_bar = full_bar + kTcMaxStages;
    uint64_t* acc_full = empty_bar + kTcMaxStages;                                  // [2] accumulator set ready for the epilogue
    uint64_t* acc_empty = acc_full + 2;                                             // [2] accumulator set free for the MMA warp
    uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(acc_empty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_base_s + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(smem_u32(&full_bar[s]), 1);
            mbar_init(smem_u32(&empty_bar[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&acc_full[a]), 1);
            mbar_init(smem_u32(&acc_empty[a]), 4);             // one arrival per epilogue warp
        }
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_base_s), TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_base_s;

    const int n_tiles = p.tiles_m * p.tiles_n;
    const int kblocks = (p.d + kTcBK - 1) / kTcBK;

    if (warp == 0) {
        // ------------------------------------------------------------ copies --
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0;
            for (int tile = blockIdx.x; tile < n_tiles && !*abort_flag; tile += gridDim.x) {
                // neighbouring CTAs share the weight slice (same tile_n), so it is read from HBM once
                const int m0 = (tile % p.tiles_m) * kTcBM, n0 = (tile / p.tiles_m) * BN;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!tc_wait(smem_u32(&empty_bar[s]), ph ^ 1u, abort_flag, p.status)) break;
                    const uint32_t fb = smem_u32(&full_bar[s]);
                    const uint32_t dst = smem_u32(tiles + (size_t)s * STAGE_BYTES);
                    mbar_arrive_expect_tx(fb, STAGE_BYTES);
                    tensor_g2s_2d(dst, &map_x, kb * kTcBK, m0, fb);
                    tensor_g2s_2d(dst + kTcTileBytes, &map_up, kb * kTcBK, n0, fb);
                    if (GATED) tensor_g2s_2d(dst + kTcTileBytes + W_TILE_BYTES, &map_gate, kb * kTcBK, n0, fb);
                    if (++s == p.stages) { s = 0; ph ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // --------------------------------------------------------------- MMA --
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0;
            int it = 0;
            for (int tile = blockIdx.x; tile < n_tiles && !*abort_flag; tile += gridDim.x, ++it) {
                const int a = it & 1;
                const uint32_t aph = (uint32_t)((it >> 1) & 1);
                if (!tc_wait(smem_u32(&acc_empty[a]), aph ^ 1u, abort_flag, p.status)) break;
                tc_fence_after();
                const uint32_t d_up = tmem_base + (uint32_t)a * kTcAccStride;
                bool ok = true;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!(ok = tc_wait(smem_u32(&full_bar[s]), ph, abort_flag, p.status))) break;
                    tc_fence_after();
                    const uint32_t base = smem_u32(tiles + (size_t)s * STAGE_BYTES);
                    const uint64_t da = smem_desc_k_sw128(base);
                    const uint64_t db = smem_desc_k_sw128(base + kTcTileBytes);
                    const uint64_t dg = smem_desc_k_sw128(base + kTcTileBytes + W_TILE_BYTES);
#pragma unroll
                    for (int k4 = 0; k4 < kTcBK / kTcUmmaK; ++k4) {
                        const uint32_t acc = (kb > 0 || k4 > 0) ? 1u : 0u;
                        const uint64_t koff = (uint64_t)(k4 * kTcUmmaK * 2 >> 4);       // 32 bytes per step, in 16-byte units
                        umma_bf16(d_up, da + koff, db + koff, IDESC, acc);
                        if (GATED) umma_bf16(d_up + kTcGateOfs, da + koff, dg + koff, IDESC, acc);
                    }
                    umma_commit(smem_u32(&empty_bar[s]));       // the stage is free once these MMAs have read it
                    if (++s == p.stages) { s = 0; ph ^= 1u; }
                }
                if (!ok) break;
                umma_commit(smem_u32(&acc_full[a]));            // the accumulators are complete
            }
        }
    } else {
        // ---------------------------------------------------------- epilogue --
        const int q = warp & 3;                                  // tensor-memory lane quarter this warp may read
        int it = 0;
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++it) {
            if (*abort_flag) break;
            const int a = it & 1;
            const uint32_t aph = (uint32_t)((it >> 1) & 1);
            const int m0 = (tile % p.tiles_m) * kTcBM, n0 = (tile / p.tiles_m) * BN;
            if (!tc_wait(smem_u32(&acc_full[a]), aph, abort_flag, p.status)) break;
            tc_fence_after();
            const int row = m0 + q * 32 + lane;
            const uint32_t t_up = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)a * kTcAccStride;
            const size_t orow_ofs = (size_t)(row < p.T ? row : 0) * p.ld_out;
            float* orow = reinterpret_cast<float*>(p.out) + orow_ofs;
            uint16_t* orow16 = reinterpret_cast<uint16_t*>(p.out) + orow_ofs;
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t u[32], g[32];
                tmem_ld32(t_up + (uint32_t)(c * 32), u);
                if (GATED) tmem_ld32(t_up + kTcGateOfs + (uint32_t)(c * 32), g);
                tmem_ld_wait();
                const int nbase = n0 + c * 32;
                if (row < p.T) {
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        float v[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            float uu = __uint_as_float(u[j + e]);
                            if (GATED) {
                                v[e] = gate_activation(__uint_as_float(g[j + e]), p.silu) * uu;
                            } else {
                                if (p.bias && nbase + j + e < p.N)
                                    uu += p.f16 ? __half2float(reinterpret_cast<const __half*>(p.bias)[nbase + j + e])
                                                : __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p.bias)[nbase + j + e]);
                                v[e] = fmaxf(uu, 0.f);
                            }
                        }
                        if (p.out_kind == 0) {
                            if (nbase + j + 3 < p.N) {
                                *reinterpret_cast<float4*>(orow + nbase + j) = make_float4(v[0], v[1], v[2], v[3]);
                            } else {
#pragma unroll
                                for (int e = 0; e < 4; ++e)
                                    if (nbase + j + e < p.N) orow[nbase + j + e] = v[e];
                            }
                        } else {
                            uint16_t h[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                h[e] = p.out_kind == 1 ? __bfloat16_as_ushort(__float2bfloat16_rn(v[e]))
                                                       : __half_as_ushort(__float2half_rn(v[e]));
                            if (nbase + j + 3 < p.N) {
                                *reinterpret_cast<uint2*>(orow16 + nbase + j) =
                                    make_uint2((uint32_t)h[0] | ((uint32_t)h[1] << 16), (uint32_t)h[2] | ((uint32_t)h[3] << 16));
                            } else {
#pragma unroll
                                for (int e = 0; e < 4; ++e)
                                    if (nbase + j + e < p.N) orow16[nbase + j + e] = h[e];
                            }
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&acc_empty[a]));
        }
    }

    // Leaving: nothing may still be landing in this CTA's shared memory, and tensor memory goes back.
    tc_fence_before();
    __syncthreads();
    if (warp == 0 && lane == 0 && *abort_flag) {
        // after a wait that gave up, copies may be in flight: give them a bounded time to land
        const long long t0 = clock64();
        while (clock64() - t0 < 20000000LL) __nanosleep(1000);
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// Tile width for a call: the tiles run in waves of one per SM, a wave lasts about as long as its
// width, so the width (a multiple of 32 up to the kind's maximum, at least half of it) with the
// smallest waves x width wins; the wider one on a tie.
static int tc_pick_bn(bool gated, int T, int N, int sms)
{
    const int max_bn = gated ? kTcMaxBNGated : kTcMaxBN;
    const long long tiles_m = (T + kTcBM - 1) / kTcBM;
    int best = max_bn;
    long long best_cost = -1;
    for (int bn = max_bn; bn >= max_bn / 2; bn -= 32) {
        const long long tiles = tiles_m * ((N + bn - 1) / bn);
        const long long cost = ((tiles + sms - 1) / sms) * bn;
        if (best_cost < 0 || cost < best_cost) {
            best_cost = cost;
            best = bn;
        }
    }
    return best;
}

// cuTensorMapEncodeTiled, looked up through the runtime (the library links no libcuda symbol).
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static coreinfer_status encode_fn(EncodeTiledFn* out)
{
    static EncodeTiledFn cached = nullptr;
    if (!cached) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        CI_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
        if (qres != cudaDriverEntryPointSuccess || !fn)
            CI_FAIL(COREINFER_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
        cached = (EncodeTiledFn)fn;
    }
    *out = cached;
    return COREINFER_OK;
}

// [rows][cols] bf16 or fp16 row-major, read in boxes of `box_rows` rows x 64 columns with the 128-byte swizzle.
static coreinfer_status make_map(CUtensorMap* map, const void* base, int rows, int cols, bool f16, int box_rows)
{
    EncodeTiledFn enc;
    coreinfer_status s = encode_fn(&enc);
    if (s != COREINFER_OK) return s;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kTcBK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = enc(map, f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) CI_FAIL(COREINFER_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
    return COREINFER_OK;
}

}  // namespace coreinfer

using namespace coreinfer;

extern "C" {

size_t coreinfer_prefill_activations_workspace_bytes(void) { return 256; }

coreinfer_status coreinfer_prefill_activations(const void* x, int32_t T, coreinfer_dtype dtype, coreinfer_ffn_kind kind,
                                               int32_t d_model, int32_t d_ff, const void* w_up, const void* w_gate,
                                               const void* b_up, void* act_out, coreinfer_dtype act_dtype, int64_t ld_act,
                                               void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    if (dtype != COREINFER_BF16 && dtype != COREINFER_F16)
        CI_FAIL(COREINFER_ERR_UNSUPPORTED, "the tensor-core pre-fill takes bf16 or fp16 inputs (dtype %d given); "
                                           "use coreinfer_ffn_dense_ref for fp32", (int)dtype);
    if (!kind_known(kind)) CI_FAIL(COREINFER_ERR_UNSUPPORTED, "ffn kind %d is not supported", (int)kind);
    const bool gated = kind_gated(kind);
    const bool f16 = dtype == COREINFER_F16;
    if (T < 1 || d_model < 1 || d_ff < 1) CI_FAIL(COREINFER_ERR_INVALID_ARG, "T, d_model, d_ff must be >= 1");
    if (d_model % 8 != 0) CI_FAIL(COREINFER_ERR_INVALID_ARG, "d_model %d: a row must be a multiple of 16 bytes", d_model);
    if (!x || !w_up || !act_out || !aligned16(x) || !aligned16(w_up) || !aligned16(act_out))
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "x / w_up / act_out NULL or not 16-byte aligned");
    if (gated != (w_gate != nullptr) || (w_gate && !aligned16(w_gate)))
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "w_gate must be given (16-byte aligned) exactly for the gated FFN");
    if (gated && b_up) CI_FAIL(COREINFER_ERR_INVALID_ARG, "the gated FFN has no up bias");
    if (!dtype_known(act_dtype)) CI_FAIL(COREINFER_ERR_UNSUPPORTED, "act_dtype %d is not supported", (int)act_dtype);
    const int act_per16 = 16 / (int)dtype_size(act_dtype);
    if (ld_act < d_ff || (ld_act % act_per16) != 0)
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "ld_act must be >= d_ff and a multiple of %d (rows of whole 16-byte pieces)", act_per16);
    if (!workspace || !aligned16(workspace)) CI_FAIL(COREINFER_ERR_WORKSPACE, "workspace is NULL or misaligned");
    if (workspace_bytes < coreinfer_prefill_activations_workspace_bytes())
        CI_FAIL(COREINFER_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes,
                coreinfer_prefill_activations_workspace_bytes());
    DeviceInfo di;
    coreinfer_status s = device_info(&di);
    if (s != COREINFER_OK) return s;
    cudaStream_t st = (cudaStream_t)cuda_stream;

    CUtensorMap map_x, map_up, map_gate;
    const int bn = tc_pick_bn(gated, T, d_ff, di.sm_count);
    if ((s = make_map(&map_x, x, T, d_model, f16, kTcBM)) != COREINFER_OK) return s;
    if ((s = make_map(&map_up, w_up, d_ff, d_model, f16, bn)) != COREINFER_OK) return s;
    if ((s = make_map(&map_gate, gated ? w_gate : w_up, d_ff, d_model, f16, bn)) != COREINFER_OK) return s;

    TcParams p;
    p.T = T;
    p.N = d_ff;
    p.d = d_model;
    p.gated = gated ? 1 : 0;
    p.silu = kind == COREINFER_FFN_SILU_GATED;
    p.f16 = f16 ? 1 : 0;
    // instruction descriptor: fp32 accumulate (bit 4), A and B format (bits 7.. and 10..: 0 fp16, 1 bf16; one
    // instruction takes both operands in the same format), both K-major, N >> 3 at bit 17, M >> 4 at bit 24
    const uint32_t fmt = f16 ? 0u : 1u;
    p.idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(kTcBM >> 4) << 24);
    p.tiles_m = (T + kTcBM - 1) / kTcBM;
    p.tiles_n = (d_ff + bn - 1) / bn;
    p.bn = bn;
    p.ld_out = ld_act;
    p.out = act_out;
    p.out_kind = act_dtype == COREINFER_F32 ? 0 : (act_dtype == COREINFER_BF16 ? 1 : 2);
    p.bias = b_up;
    p.status = (unsigned*)workspace;
    const size_t stage = (size_t)kTcTileBytes + (size_t)(gated ? 2 : 1) * bn * kTcBK * 2;
    const size_t fixed = 1024 /* alignment slack */ + (2 * kTcMaxStages + 4) * sizeof(uint64_t) + 64;
    long long stages = ((long long)di.smem_optin - (long long)fixed) / (long long)stage;
    if (stages > kTcMaxStages) stages = kTcMaxStages;
    if (stages < 2) CI_FAIL(COREINFER_ERR_UNSUPPORTED, "not enough shared memory for two pipeline stages");
    p.stages = (int)stages;
    const size_t smem = fixed + (size_t)p.stages * stage;
    const int n_tiles = p.tiles_m * p.tiles_n;
    const int grid = n_tiles < di.sm_count ? n_tiles : di.sm_count;

    CI_CUDA(cudaMemsetAsync(workspace, 0, 256, st));
    if (gated) {
        CI_CUDA(cudaFuncSetAttribute(prefill_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        prefill_tc_kernel<true><<<grid, kTcThreads, smem, st>>>(map_x, map_up, map_gate, p);
    } else {
        CI_CUDA(cudaFuncSetAttribute(prefill_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        prefill_tc_kernel<false><<<grid, kTcThreads, smem, st>>>(map_x, map_up, map_gate, p);
    }
    CI_CUDA(cudaGetLastError());
    return COREINFER_OK;
}

}  // extern "C"
