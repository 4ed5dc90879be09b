// Decode FFN over compacted weights for 2..8 sequences that share one core set (Section 4.2
// applied to a small batch), bf16, one layer per launch.
//
// With eight sequences the work per weight byte is eight times that of batch 1 and the fp32
// pipes would become the limit, so here the sequences sit on the N = 8 side of
// mma.sync.m16n8k16 (bf16 inputs, fp32 accumulate): this is the one place where the path is a
// real dense contraction.  The streaming structure is that of the batch-1 kernel: one CTA per
// SM owns a slab of neurons, a producer warp fills a ring of shared-memory slots with 1-D bulk
// copies (slot stride = row + 16 bytes, so that the 8 rows of an ldmatrix tile fall into
// different banks), and sixteen consumer warps each own d_model / 16 columns.
//   up:   A = 16 weight rows (8 up + 8 gate rows when gated) x 16 columns from the ring,
//         B = x^T fragments kept in registers; the sixteen warps' 16 x 8 partial tiles are
//         added in shared memory, then bias + ReLU (or gate product) gives h in fp32.
//   down: A = the transposed view (ldmatrix.trans) of 16 down rows, B = h split exactly into
//         three bf16 parts (hi + mid + lo = the fp32 value), three MMAs per tile; the
//         [d_model / 16 columns] x [8 sequences] accumulators stay in registers for the slab.
//   out:  tiles are turned in shared memory and added to y with vector reductions.
// Every wait is bounded as in the batch-1 kernel.
#include "common.cuh"

namespace coreinfer {

constexpr int kMmaWarps = 16;
constexpr int kMmaThreads = kMmaWarps * 32;
constexpr int kMmaBlock = kMmaThreads + 32;
constexpr int kMmaMaxSlots = 64;
constexpr int kMmaMaxTiles = 16;                    // d_model / 16 warps / 16 columns <= 16  ->  d_model <= 4096
constexpr long long kMmaWaitCycles = 3000000000LL;

struct MmaParams {
    const uint8_t* up;
    const uint8_t* gate;
    const uint8_t* down;
    const __nv_bfloat16* bup;
    const __nv_bfloat16* bdown;
    const __nv_bfloat16* x;     // [B][d]
    float* y;                   // [B][d], zero on entry
    unsigned* status;
    int K, d, B, row_bytes, slot_stride, n_slots, rpad;
    int silu;                   // gated: 0 ReLU gate, 1 SiLU gate
};

// shared memory besides the ring: zero row, barriers, scratch, h parts, flags, sums of squares
static size_t mma_fixed_smem(int slot_stride, int rpad)
{
    return (size_t)slot_stride + 2 * kMmaMaxSlots * sizeof(uint64_t) + kMmaWarps * 128 * sizeof(float)
           + (size_t)3 * 8 * rpad * sizeof(__nv_bfloat16) + 16 + kMmaWarps * 8 * sizeof(float) + 128;
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&a)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&a)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ bool mma_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned* status)
{
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    const long long t0 = clock64();
    for (;;) {
        if (mbar_try_wait_parked(bar, parity, 4000u)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > kMmaWaitCycles) {
            *abort_flag = 1;
            atomicMax(status, (unsigned)kStatusTimeout);
            return false;
        }
    }
}

template <bool GATED>
__global__ void __launch_bounds__(kMmaBlock, 1)
decode_batch_mma_kernel(const MmaParams p)
{
    constexpr int NMAT = GATED ? 2 : 1;
    constexpr int RU = 16 / NMAT;                    // neurons per up unit (16 tile rows)

    extern __shared__ __align__(128) uint8_t smem[];
    const int NS = p.n_slots;
    uint8_t* ring = smem;
    uint8_t* zero_row = ring + (size_t)NS * p.slot_stride;                       // a row of zeros for padded tile rows
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(zero_row + p.slot_stride);
    uint64_t* empty_bar = full_bar + kMmaMaxSlots;
    float* scratch = reinterpret_cast<float*>(empty_bar + kMmaMaxSlots);         // [16 warps][128]: partial tiles / output staging
    __nv_bfloat16* hpart = reinterpret_cast<__nv_bfloat16*>(scratch + kMmaWarps * 128);   // [3][8][rpad]
    volatile int* abort_flag = reinterpret_cast<volatile int*>(hpart + 3 * 8 * p.rpad);

    const int tid = threadIdx.x;
    const int G = gridDim.x, cta = blockIdx.x;
    const int k0 = (int)(((long long)cta * p.K) / G), k1 = (int)(((long long)(cta + 1) * p.K) / G);
    const int n = k1 - k0;
    const int n_up_units = (n + RU - 1) / RU;
    const int n_dn_units = (n + 15) / 16;

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(smem_u32(&full_bar[s]), 1);
            mbar_init(smem_u32(&empty_bar[s]), kMmaWarps);
        }
        *abort_flag = 0;
        mbar_fence_init();
    }
    for (int i = tid; i < p.slot_stride / 16; i += kMmaBlock) reinterpret_cast<uint4*>(zero_row)[i] = make_uint4(0, 0, 0, 0);
    for (int i = tid; i < 3 * 8 * p.rpad; i += kMmaBlock) hpart[i] = __float2bfloat16(0.f);
    __syncthreads();

    // ======================================================== producer warp ==
    if (tid >= kMmaThreads) {
        const int lane = tid - kMmaThreads;
        const int round_max = NS < 8 ? NS : 8;
        const int n_up_items = n * NMAT;
        const int total = n_up_items + n;
        int slot0 = 0;
        uint32_t phase0 = 0;
        long long issued = 0;
        for (int q0 = 0; q0 < total; q0 += round_max) {
            if (*abort_flag) break;
            const int cnt = min(round_max, total - q0);
            if (lane < cnt) {
                const int q = q0 + lane;
                const uint8_t* src;
                if (q < n_up_items) {
                    // unit u holds cnt_u up rows followed (gated) by the same neurons' gate rows
                    const int u = q / (RU * NMAT);
                    const int w = q - u * RU * NMAT;
                    const int cnt_u = min(RU, n - u * RU);
                    const int r = w % cnt_u, m = w / cnt_u;
                    src = (m ? p.gate : p.up) + (size_t)(k0 + u * RU + r) * p.row_bytes;
                } else {
                    src = p.down + (size_t)(k0 + q - n_up_items) * p.row_bytes;
                }
                int sl = slot0 + lane;
                uint32_t ph = phase0;
                if (sl >= NS) { sl -= NS; ph ^= 1u; }
                if (mma_wait(smem_u32(&empty_bar[sl]), ph ^ 1u, abort_flag, p.status)) {
                    const uint32_t fb = smem_u32(&full_bar[sl]);
                    mbar_arrive_expect_tx(fb, (uint32_t)p.row_bytes);
                    bulk_g2s(smem_u32(ring + (size_t)sl * p.slot_stride), src, (uint32_t)p.row_bytes, fb);
                }
            }
            __syncwarp();
            slot0 += cnt;
            if (slot0 >= NS) { slot0 -= NS; phase0 ^= 1u; }
            issued += cnt;
        }
        for (int sl = lane; sl < NS; sl += 32) {      // leave only when nothing is in flight into this CTA
            const long long uses = issued / NS + (sl < (int)(issued % NS) ? 1 : 0);
            if (uses == 0) continue;
            const uint32_t fb = smem_u32(&full_bar[sl]);
            const uint32_t ph = (uint32_t)((uses - 1) & 1);
            const long long t0 = clock64();
            while (!mbar_try_wait(fb, ph))
                if (clock64() - t0 > kMmaWaitCycles) { atomicMax(p.status, (unsigned)kStatusTimeout); break; }
        }
        return;
    }

    // ============================================================ consumers ==
    const int lane = tid & 31, warp = tid >> 5;
    const int JW = p.d / kMmaWarps;                   // columns of this warp (a multiple of 16)
    const int jw = warp * JW;
    const int ntile = JW / 16;                        // <= kMmaMaxTiles

    // x^T fragments: B[k][n] = x[n][jw + 16 t + k]; lane holds k = 2 (lane % 4) + {0, 1} (+ 8), n = lane / 4
    uint32_t xb[kMmaMaxTiles][2];
    {
        const int nb = lane >> 2;
        const uint32_t* xrow = reinterpret_cast<const uint32_t*>(p.x + (size_t)(nb < p.B ? nb : 0) * p.d);
#pragma unroll
        for (int t = 0; t < kMmaMaxTiles; ++t) {
            xb[t][0] = xb[t][1] = 0u;
            if (t < ntile && nb < p.B) {
                const int j = jw + t * 16 + (lane & 3) * 2;
                xb[t][0] = xrow[j >> 1];
                xb[t][1] = xrow[(j + 8) >> 1];
            }
        }
    }

    int slot = 0;
    uint32_t phase = 0;
    auto wait_items = [&](int cnt) {
        int sl = slot;
        uint32_t ph = phase;
        for (int j = 0; j < cnt; ++j) {
            mma_wait(smem_u32(&full_bar[sl]), ph, abort_flag, p.status);
            if (++sl == NS) { sl = 0; ph ^= 1u; }
        }
    };
    auto item_addr = [&](int j) -> uint32_t {
        int sl = slot + j;
        if (sl >= NS) sl -= NS;
        return smem_u32(ring + (size_t)sl * p.slot_stride);
    };
    auto release_items = [&](int cnt) {       // cnt <= 16
        __syncwarp();
        if (lane < cnt && !*abort_flag) {
            int sl = slot + lane;
            if (sl >= NS) sl -= NS;
            mbar_arrive(smem_u32(&empty_bar[sl]));
        }
        slot += cnt;
        if (slot >= NS) { slot -= NS; phase ^= 1u; }
    };
    const uint32_t zero_addr = smem_u32(zero_row);

    // ------------------------------------------------------ up (+ gate) units --
    for (int u = 0; u < n_up_units; ++u) {
        const int cnt = min(RU, n - u * RU);
        wait_items(cnt * NMAT);
        // tile row of this lane (for ldmatrix lane l addresses row l % 16, column half l / 16)
        const int tr = lane & 15;
        uint32_t rowaddr;
        if (GATED) {
            const int r = tr & 7, m = tr >> 3;
            rowaddr = r < cnt ? item_addr(m * cnt + r) : zero_addr;
        } else {
            rowaddr = tr < cnt ? item_addr(tr) : zero_addr;
        }
        rowaddr += (uint32_t)(jw + 8 * (lane >> 4)) * 2u;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int t = 0; t < kMmaMaxTiles; ++t) {
            if (t < ntile) {
                uint32_t a[4];
                ldmatrix_x4(a, rowaddr + (uint32_t)t * 32u);
                mma_bf16_16816(acc, a, xb[t][0], xb[t][1]);
            }
        }
        release_items(cnt * NMAT);
        // partial tile of this warp: rows m = lane / 4 (+ 8), sequences 2 (lane % 4) + {0, 1}
        float* mine = scratch + warp * 128;
        mine[(lane >> 2) * 8 + (lane & 3) * 2] = acc[0];
        mine[(lane >> 2) * 8 + (lane & 3) * 2 + 1] = acc[1];
        mine[((lane >> 2) + 8) * 8 + (lane & 3) * 2] = acc[2];
        mine[((lane >> 2) + 8) * 8 + (lane & 3) * 2 + 1] = acc[3];
        named_bar_sync(1, kMmaThreads);
        if (tid < RU * 8) {
            const int r = tid >> 3, nb = tid & 7;
            float uu = 0.f, gg = 0.f;
#pragma unroll
            for (int w = 0; w < kMmaWarps; ++w) {
                uu += scratch[w * 128 + r * 8 + nb];
                if (GATED) gg += scratch[w * 128 + (r + 8) * 8 + nb];
            }
            float h = 0.f;
            if (r < cnt) {
                if (GATED) {
                    h = gate_activation(gg, p.silu) * uu;
                } else {
                    if (p.bup) uu += __bfloat162float(p.bup[k0 + u * RU + r]);
                    h = fmaxf(uu, 0.f);
                }
            }
            // h = h1 + h2 + h3 exactly (three bf16 parts cover the 24-bit significand)
            const __nv_bfloat16 h1 = __float2bfloat16_rn(h);
            const float r1 = h - __bfloat162float(h1);
            const __nv_bfloat16 h2 = __float2bfloat16_rn(r1);
            const __nv_bfloat16 h3 = __float2bfloat16_rn(r1 - __bfloat162float(h2));
            const int kk = u * RU + r;
            hpart[(0 * 8 + nb) * p.rpad + kk] = h1;
            hpart[(1 * 8 + nb) * p.rpad + kk] = h2;
            hpart[(2 * 8 + nb) * p.rpad + kk] = h3;
        }
        named_bar_sync(1, kMmaThreads);
    }

    // --------------------------------------------------------------- down units --
    float dacc[kMmaMaxTiles][4];
#pragma unroll
    for (int t = 0; t < kMmaMaxTiles; ++t) { dacc[t][0] = dacc[t][1] = dacc[t][2] = dacc[t][3] = 0.f; }
    for (int ku = 0; ku < n_dn_units; ++ku) {
        const int kk0 = ku * 16;
        const int cnt = min(16, n - kk0);
        wait_items(cnt);
        // transposed tile: lane l addresses stored row k = 8 (l / 16) + l % 8, column block (l / 8) % 2
        const int kr = ((lane >> 4) << 3) + (lane & 7);
        uint32_t rowaddr = (kr < cnt ? item_addr(kr) : zero_addr) + (uint32_t)(jw + 8 * ((lane >> 3) & 1)) * 2u;
        uint32_t hb[3][2];
#pragma unroll
        for (int s3 = 0; s3 < 3; ++s3) {
            const uint32_t* hrow = reinterpret_cast<const uint32_t*>(hpart + (size_t)(s3 * 8 + (lane >> 2)) * p.rpad + kk0);
            hb[s3][0] = hrow[lane & 3];
            hb[s3][1] = hrow[(lane & 3) + 4];
        }
#pragma unroll
        for (int t = 0; t < kMmaMaxTiles; ++t) {
            if (t < ntile) {
                uint32_t a[4];
                ldmatrix_x4_trans(a, rowaddr + (uint32_t)t * 32u);
                mma_bf16_16816(dacc[t], a, hb[0][0], hb[0][1]);
                mma_bf16_16816(dacc[t], a, hb[1][0], hb[1][1]);
                mma_bf16_16816(dacc[t], a, hb[2][0], hb[2][1]);
            }
        }
        release_items(cnt);
    }

    // ---------------------------------------------------------------- output --
    // dacc[t]: columns j = jw + 16 t + lane / 4 (+ 8), sequences 2 (lane % 4) + {0, 1}.  Turn each tile
    // in this warp's scratch so that a lane owns 4 consecutive columns of one sequence.
    float* st = scratch + warp * 128;            // [8 sequences][16 columns]
    named_bar_sync(1, kMmaThreads);              // the up phase's last use of the scratch is over
#pragma unroll
    for (int t = 0; t < kMmaMaxTiles; ++t) {
        if (t < ntile) {
            const int jl = lane >> 2, nb = (lane & 3) * 2;
            st[nb * 16 + jl] = dacc[t][0];
            st[(nb + 1) * 16 + jl] = dacc[t][1];
            st[nb * 16 + jl + 8] = dacc[t][2];
            st[(nb + 1) * 16 + jl + 8] = dacc[t][3];
            __syncwarp();
            const int nn = lane >> 2, jq = (lane & 3) * 4;
            float4 v = *reinterpret_cast<const float4*>(st + nn * 16 + jq);
            const int j = jw + t * 16 + jq;
            if (nn < p.B) {
                if (cta == 0 && p.bdown) {
                    v.x += __bfloat162float(p.bdown[j]);     v.y += __bfloat162float(p.bdown[j + 1]);
                    v.z += __bfloat162float(p.bdown[j + 2]); v.w += __bfloat162float(p.bdown[j + 3]);
                }
                red_add_v4(p.y + (size_t)nn * p.d + j, v.x, v.y, v.z, v.w);
            }
            __syncwarp();
        }
    }
}

// Returns COREINFER_ERR_UNSUPPORTED (without setting an error text) when the shape is not built here.
// y is cleared here, on the stream, before the launch.
coreinfer_status decode_batched_mma(const void* x, int batch, bool gated, int silu, int d_model, const coreinfer_layer& ly,
                                    float* y, unsigned* status, const DeviceInfo& di, cudaStream_t st)
{
    if (d_model % (kMmaWarps * 16) != 0 || d_model / (kMmaWarps * 16) > kMmaMaxTiles) return COREINFER_ERR_UNSUPPORTED;
    MmaParams p;
    p.up = (const uint8_t*)ly.w_up_c;
    p.gate = (const uint8_t*)ly.w_gate_c;
    p.down = (const uint8_t*)ly.w_downT_c;
    p.bup = (const __nv_bfloat16*)ly.b_up_c;
    p.bdown = (const __nv_bfloat16*)ly.b_down;
    p.x = (const __nv_bfloat16*)x;
    p.y = y;
    p.status = status;
    p.silu = silu;
    p.K = ly.K;
    p.d = d_model;
    p.B = batch;
    p.row_bytes = d_model * 2;
    p.slot_stride = p.row_bytes + 16;
    const int G = di.sm_count;
    const int rmax = (ly.K + G - 1) / G + 1;
    p.rpad = (rmax + 15) & ~15;
    const size_t fixed = (size_t)p.slot_stride                      /* zero row */
                         + 2 * kMmaMaxSlots * sizeof(uint64_t) + kMmaWarps * 128 * sizeof(float)
                         + (size_t)3 * 8 * p.rpad * sizeof(__nv_bfloat16) + 16 + 128;
    long long slots = ((long long)di.smem_optin - (long long)fixed) / p.slot_stride;
    if (slots > kMmaMaxSlots) slots = kMmaMaxSlots;
    if (slots < 17) return COREINFER_ERR_UNSUPPORTED;
    p.n_slots = (int)slots;
    const size_t smem = fixed + (size_t)p.n_slots * p.slot_stride;
    CI_CUDA(cudaMemsetAsync(y, 0, (size_t)batch * d_model * sizeof(float), st));
    auto kern = gated ? decode_batch_mma_kernel<true> : decode_batch_mma_kernel<false>;
    CI_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    kern<<<G, kMmaBlock, smem, st>>>(p);
    CI_CUDA(cudaGetLastError());
    return COREINFER_OK;
}

// Whether decode_batched_mma serves this shape (same conditions as above).
bool decode_batched_mma_serves(int d_model, int K, const DeviceInfo& di)
{
    if (d_model % (kMmaWarps * 16) != 0 || d_model / (kMmaWarps * 16) > kMmaMaxTiles) return false;
    const size_t stride = (size_t)d_model * 2 + 16;
    const int rmax = (K + di.sm_count - 1) / di.sm_count + 1;
    const size_t fixed = stride + 2 * kMmaMaxSlots * sizeof(uint64_t) + kMmaWarps * 128 * sizeof(float)
                         + (size_t)3 * 8 * ((rmax + 15) & ~15) * sizeof(__nv_bfloat16) + 16 + 128;
    return ((long long)di.smem_optin - (long long)fixed) / (long long)stride >= 17;
}


// =============================================================================
// The whole stack for 2..8 sequences in one persistent, cooperatively launched kernel.
//
// Launching the kernel above once per layer costs, per layer, the hand-over between two
// launches (a 227 KB CTA cannot share its SM with its successor, so nothing of the next layer
// overlaps the flush of the partial outputs) and a separate glue kernel: 17 of 30 us at the
// gated Llama shape.  Here the CTAs stay resident: the producer warp walks all layers and is
// already filling the ring with the next layer's weights while the consumers flush their partial
// y (vector reductions into the layer's target), meet at a grid barrier (one thread per CTA:
// release arrival, bounded acquire polling), read the sum back and form the next input -- the
// residual and RMS normalisation of the batch-1 kernel, per sequence -- directly as the x^T
// fragments of the next layer.  Targets rotate over three buffers as in the batch-1 kernel.
struct StackLayerB {
    const uint8_t* up;
    const uint8_t* gate;
    const uint8_t* down;
    const __nv_bfloat16* bup;
    const __nv_bfloat16* bdown;
    int K;
    int pad;
};

struct MmaStackParams {
    int L, d, B, row_bytes, slot_stride, n_slots, rpad;
    int silu;                     // gated: 0 ReLU gate, 1 SiLU gate
    int runahead;                 // ring items of the next layer the producer may request before this layer's exchange is over
    float inv_d;
    const __nv_bfloat16* x0;      // [B][d]
    float* y_last;                // [B][d], zero on entry
    float* y_layers;              // [L][B][d] zero on entry, or NULL
    __nv_bfloat16* x_layers;      // [L][B][d] or NULL (row 0 is written by the host)
    float* ybuf;                  // [3][B][d]; buffers 0 and 1 zero on entry
    unsigned* ctrl;               // [0] status word, [1] grid-barrier arrivals; zero on entry
    unsigned long long* stamps;   // [CTA][layer][kStampSlots] cycle counts, or NULL (COREINFER_STAMPS builds)
    StackLayerB layers[COREINFER_MAX_LAYERS];
};

__device__ __forceinline__ void stack_slab(int cta, int G, int K, int* k0, int* k1)
{
    *k0 = (int)(((long long)cta * K) / G);
    *k1 = (int)(((long long)(cta + 1) * K) / G);
}

// One thread per CTA, after a CTA barrier that follows every consumer's reductions: the release
// publishes them (they are ordered before it through that barrier).  Barrier b completes at
// (b + 1) * G arrivals.  Bounded: gives up after kMmaWaitCycles or when another CTA has.
__device__ __forceinline__ void stack_grid_barrier(unsigned* ctrl, unsigned target, volatile int* abort_flag)
{
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(&ctrl[1]), "r"(1u) : "memory");
    const long long t0 = clock64();
    unsigned it = 0;
    for (;;) {
        if (ld_acquire_gpu(&ctrl[1]) >= target) break;
        __nanosleep(32);
        if ((++it & 255u) == 0u) {
            if (ld_acquire_gpu(&ctrl[0]) != kStatusOk) { *abort_flag = 1; break; }
            if (clock64() - t0 > kMmaWaitCycles) {
                *abort_flag = 1;
                atomicMax(&ctrl[0], (unsigned)kStatusTimeout);
                break;
            }
        }
    }
}

template <bool GATED>
__global__ void __launch_bounds__(kMmaBlock, 1)
decode_batch_stack_kernel(const __grid_constant__ MmaStackParams p)
{
    constexpr int NMAT = GATED ? 2 : 1;
    constexpr int UR = 16;                           // ring rows per unit (8-row units were slower: twice the barrier phases)
    constexpr int RU = UR / NMAT;                    // neurons per up unit

    extern __shared__ __align__(128) uint8_t smem[];
    const int NS = p.n_slots;
    uint8_t* ring = smem;
    uint8_t* zero_row = ring + (size_t)NS * p.slot_stride;
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(zero_row + p.slot_stride);
    uint64_t* empty_bar = full_bar + kMmaMaxSlots;
    float* scratch = reinterpret_cast<float*>(empty_bar + kMmaMaxSlots);
    __nv_bfloat16* hpart = reinterpret_cast<__nv_bfloat16*>(scratch + kMmaWarps * 128);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(hpart + 3 * 8 * p.rpad);
    volatile int* layers_done = abort_flag + 1;                                   // layers whose exchange this CTA has behind it
    float* ssq = reinterpret_cast<float*>(const_cast<int*>(abort_flag) + 4);     // [16 warps][8 sequences]

    const int tid = threadIdx.x;
    const int G = gridDim.x, cta = blockIdx.x;
    const size_t row = (size_t)p.B * p.d;

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(smem_u32(&full_bar[s]), 1);
            mbar_init(smem_u32(&empty_bar[s]), kMmaWarps);
        }
        *abort_flag = 0;
        *layers_done = 0;
        mbar_fence_init();
    }
    for (int i = tid; i < p.slot_stride / 16; i += kMmaBlock) reinterpret_cast<uint4*>(zero_row)[i] = make_uint4(0, 0, 0, 0);
    for (int i = tid; i < 3 * 8 * p.rpad; i += kMmaBlock) hpart[i] = __float2bfloat16(0.f);
    __syncthreads();

    // ======================================================== producer warp ==
    if (tid >= kMmaThreads) {
        const int lane = tid - kMmaThreads;
        const int round_max = NS < 8 ? NS : 8;
        int slot0 = 0;
        uint32_t phase0 = 0;
        long long issued = 0;
        for (int l = 0; l < p.L; ++l) {
            const StackLayerB& ly = p.layers[l];
            int k0, k1;
            stack_slab(cta, G, ly.K, &k0, &k1);
            const int n = k1 - k0;
            const int n_up_items = n * NMAT;
            const int total = n_up_items + n;
            for (int q0 = 0, cnt = 0; q0 < total; q0 += cnt) {
                if (*abort_flag) break;
                cnt = min(round_max, total - q0);
                // The exchange of the layer before (reductions, barrier, read-back) queues behind
                // every weight request in flight, so only a limited number of this layer's rows
                // is requested before that exchange is over.
                if (l > 0 && q0 + cnt > p.runahead && *layers_done < l) {
                    if (q0 < p.runahead) {
                        cnt = p.runahead - q0;
                    } else {
                        const long long t0 = clock64();
                        while (*layers_done < l && !*abort_flag) {
                            __nanosleep(64);
                            if (clock64() - t0 > kMmaWaitCycles) { *abort_flag = 1; atomicMax(p.ctrl, (unsigned)kStatusTimeout); }
                        }
                    }
                }
                if (lane < cnt) {
                    const int q = q0 + lane;
                    const uint8_t* src;
                    if (q < n_up_items) {
                        const int u = q / (RU * NMAT);
                        const int w = q - u * RU * NMAT;
                        const int cnt_u = min(RU, n - u * RU);
                        const int r = w % cnt_u, m = w / cnt_u;
                        src = (m ? ly.gate : ly.up) + (size_t)(k0 + u * RU + r) * p.row_bytes;
                    } else {
                        src = ly.down + (size_t)(k0 + q - n_up_items) * p.row_bytes;
                    }
                    int sl = slot0 + lane;
                    uint32_t ph = phase0;
                    if (sl >= NS) { sl -= NS; ph ^= 1u; }
                    if (mma_wait(smem_u32(&empty_bar[sl]), ph ^ 1u, abort_flag, p.ctrl)) {
                        const uint32_t fb = smem_u32(&full_bar[sl]);
                        mbar_arrive_expect_tx(fb, (uint32_t)p.row_bytes);
                        bulk_g2s(smem_u32(ring + (size_t)sl * p.slot_stride), src, (uint32_t)p.row_bytes, fb);
                    }
                }
                __syncwarp();
                slot0 += cnt;
                if (slot0 >= NS) { slot0 -= NS; phase0 ^= 1u; }
                issued += cnt;
            }
        }
        for (int sl = lane; sl < NS; sl += 32) {      // leave only when nothing is in flight into this CTA
            const long long uses = issued / NS + (sl < (int)(issued % NS) ? 1 : 0);
            if (uses == 0) continue;
            const uint32_t fb = smem_u32(&full_bar[sl]);
            const uint32_t ph = (uint32_t)((uses - 1) & 1);
            const long long t0 = clock64();
            while (!mbar_try_wait(fb, ph))
                if (clock64() - t0 > kMmaWaitCycles) { atomicMax(p.ctrl, (unsigned)kStatusTimeout); break; }
        }
        return;
    }

    // ============================================================ consumers ==
    const int lane = tid & 31, warp = tid >> 5;
    const int JW = p.d / kMmaWarps;
    const int jw = warp * JW;
    const int ntile = JW / 16;
    const int nb = lane >> 2;                          // sequence of this lane's B-fragment entries
    const bool live = nb < p.B;
    const size_t rowofs = (size_t)(live ? nb : 0) * p.d;
    const int c0 = jw + (lane & 3) * 2;                // first of this lane's columns in tile 0

    uint32_t xb[kMmaMaxTiles][2];
    {
        const uint32_t* xrow = reinterpret_cast<const uint32_t*>(p.x0 + rowofs);
#pragma unroll
        for (int t = 0; t < kMmaMaxTiles; ++t) {
            xb[t][0] = xb[t][1] = 0u;
            if (t < ntile && live) {
                const int j = c0 + t * 16;
                xb[t][0] = xrow[j >> 1];
                xb[t][1] = xrow[(j + 8) >> 1];
            }
        }
    }

    int slot = 0;
    uint32_t phase = 0;
    auto wait_items = [&](int cnt) {
        int sl = slot;
        uint32_t ph = phase;
        for (int j = 0; j < cnt; ++j) {
            mma_wait(smem_u32(&full_bar[sl]), ph, abort_flag, p.ctrl);
            if (++sl == NS) { sl = 0; ph ^= 1u; }
        }
    };
    auto item_addr = [&](int j) -> uint32_t {
        int sl = slot + j;
        if (sl >= NS) sl -= NS;
        return smem_u32(ring + (size_t)sl * p.slot_stride);
    };
    auto release_items = [&](int cnt) {
        __syncwarp();
        if (lane < cnt && !*abort_flag) {
            int sl = slot + lane;
            if (sl >= NS) sl -= NS;
            mbar_arrive(smem_u32(&empty_bar[sl]));
        }
        slot += cnt;
        if (slot >= NS) { slot -= NS; phase ^= 1u; }
    };
    const uint32_t zero_addr = smem_u32(zero_row);
    unsigned long long* const stamps = tid == 0 ? p.stamps : nullptr;

    for (int l = 0; l < p.L; ++l) {
        const StackLayerB& ly = p.layers[l];
        int k0, k1;
        stack_slab(cta, G, ly.K, &k0, &k1);
        const int n = k1 - k0;
        const int n_up_units = (n + RU - 1) / RU;
        const int n_dn_units = (n + UR - 1) / UR;
        const bool last = (l == p.L - 1);
        float* ytarget = p.y_layers ? p.y_layers + (size_t)l * row : (last ? p.y_last : p.ybuf + (size_t)(l % 3) * row);
        const size_t sb = ((size_t)cta * p.L + l) * kStampSlots;
        (void)sb;
        CI_STAMP(stamps, sb, 0);

        // ---------------------------------------------------- up (+ gate) units --
        for (int u = 0; u < n_up_units; ++u) {
            const int cnt = min(RU, n - u * RU);
            wait_items(cnt * NMAT);
            const int tr = lane & 15;
            uint32_t rowaddr;
            if (GATED) {
                const int r = tr & 7, m = tr >> 3;
                rowaddr = r < cnt ? item_addr(m * cnt + r) : zero_addr;
            } else {
                rowaddr = tr < cnt ? item_addr(tr) : zero_addr;
            }
            rowaddr += (uint32_t)(jw + 8 * (lane >> 4)) * 2u;
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int t = 0; t < kMmaMaxTiles; ++t) {
                if (t < ntile) {
                    uint32_t a[4];
                    ldmatrix_x4(a, rowaddr + (uint32_t)t * 32u);
                    mma_bf16_16816(acc, a, xb[t][0], xb[t][1]);
                }
            }
            release_items(cnt * NMAT);
            float* mine = scratch + warp * 128;
            mine[(lane >> 2) * 8 + (lane & 3) * 2] = acc[0];
            mine[(lane >> 2) * 8 + (lane & 3) * 2 + 1] = acc[1];
            mine[((lane >> 2) + 8) * 8 + (lane & 3) * 2] = acc[2];
            mine[((lane >> 2) + 8) * 8 + (lane & 3) * 2 + 1] = acc[3];
            named_bar_sync(1, kMmaThreads);
            if (tid < RU * 8) {
                const int r = tid >> 3, sq = tid & 7;
                float uu = 0.f, gg = 0.f;
#pragma unroll
                for (int w = 0; w < kMmaWarps; ++w) {
                    uu += scratch[w * 128 + r * 8 + sq];
                    if (GATED) gg += scratch[w * 128 + (r + 8) * 8 + sq];
                }
                float h = 0.f;
                if (r < cnt) {
                    if (GATED) {
                        h = gate_activation(gg, p.silu) * uu;
                    } else {
                        if (ly.bup) uu += __bfloat162float(ly.bup[k0 + u * RU + r]);
                        h = fmaxf(uu, 0.f);
                    }
                }
                const __nv_bfloat16 h1 = __float2bfloat16_rn(h);
                const float r1 = h - __bfloat162float(h1);
                const __nv_bfloat16 h2 = __float2bfloat16_rn(r1);
                const __nv_bfloat16 h3 = __float2bfloat16_rn(r1 - __bfloat162float(h2));
                const int kk = u * RU + r;
                hpart[(0 * 8 + sq) * p.rpad + kk] = h1;
                hpart[(1 * 8 + sq) * p.rpad + kk] = h2;
                hpart[(2 * 8 + sq) * p.rpad + kk] = h3;
            }
            // h beyond the last up unit, as far as the down units read it, is zero (an earlier,
            // larger slab may have left values there)
            if (u == n_up_units - 1)
                for (int i = tid; i < 3 * 8 * 16; i += kMmaThreads) {
                    const int kk = n_up_units * RU + (i & 15);
                    if (kk < (n_dn_units - 1) * UR + 16) hpart[(size_t)(i >> 4) * p.rpad + kk] = __float2bfloat16(0.f);
                }
            named_bar_sync(1, kMmaThreads);
        }

        CI_STAMP(stamps, sb, 1);
        // ------------------------------------------------------------ down units --
        float dacc[kMmaMaxTiles][4];
#pragma unroll
        for (int t = 0; t < kMmaMaxTiles; ++t) { dacc[t][0] = dacc[t][1] = dacc[t][2] = dacc[t][3] = 0.f; }
        for (int ku = 0; ku < n_dn_units; ++ku) {
            const int kk0 = ku * UR;
            const int cnt = min(UR, n - kk0);
            wait_items(cnt);
            const int kr = ((lane >> 4) << 3) + (lane & 7);
            uint32_t rowaddr = (kr < cnt ? item_addr(kr) : zero_addr) + (uint32_t)(jw + 8 * ((lane >> 3) & 1)) * 2u;
            uint32_t hb[3][2];
#pragma unroll
            for (int s3 = 0; s3 < 3; ++s3) {
                const uint32_t* hrow = reinterpret_cast<const uint32_t*>(hpart + (size_t)(s3 * 8 + (lane >> 2)) * p.rpad + kk0);
                hb[s3][0] = hrow[lane & 3];
                hb[s3][1] = hrow[(lane & 3) + 4];
            }
#pragma unroll
            for (int t = 0; t < kMmaMaxTiles; ++t) {
                if (t < ntile) {
                    uint32_t a[4];
                    ldmatrix_x4_trans(a, rowaddr + (uint32_t)t * 32u);
                    mma_bf16_16816(dacc[t], a, hb[0][0], hb[0][1]);
                    mma_bf16_16816(dacc[t], a, hb[1][0], hb[1][1]);
                    mma_bf16_16816(dacc[t], a, hb[2][0], hb[2][1]);
                }
            }
            release_items(cnt);
        }

        CI_STAMP(stamps, sb, 3);
        // ---------------------------------------------------------------- flush --
        float* st = scratch + warp * 128;            // [8 sequences][16 columns]
        named_bar_sync(1, kMmaThreads);              // the up phase's last use of the scratch is over
#pragma unroll
        for (int t = 0; t < kMmaMaxTiles; ++t) {
            if (t < ntile) {
                const int jl = lane >> 2, sq = (lane & 3) * 2;
                st[sq * 16 + jl] = dacc[t][0];
                st[(sq + 1) * 16 + jl] = dacc[t][1];
                st[sq * 16 + jl + 8] = dacc[t][2];
                st[(sq + 1) * 16 + jl + 8] = dacc[t][3];
                __syncwarp();
                const int nn = lane >> 2, jq = (lane & 3) * 4;
                float4 v = *reinterpret_cast<const float4*>(st + nn * 16 + jq);
                const int j = jw + t * 16 + jq;
                if (nn < p.B) {
                    if (cta == 0 && ly.bdown) {
                        v.x += __bfloat162float(ly.bdown[j]);     v.y += __bfloat162float(ly.bdown[j + 1]);
                        v.z += __bfloat162float(ly.bdown[j + 2]); v.w += __bfloat162float(ly.bdown[j + 3]);
                    }
                    red_add_v4(ytarget + (size_t)nn * p.d + j, v.x, v.y, v.z, v.w);
                }
                __syncwarp();
            }
        }
        if (last) { CI_STAMP(stamps, sb, 4); break; }

        // ------------------------------------------------- cross-CTA sum, glue --
        named_bar_sync(1, kMmaThreads);              // every consumer's reductions precede the arrival
        CI_STAMP(stamps, sb, 4);
        if (tid == 0 && !*abort_flag) stack_grid_barrier(p.ctrl, (unsigned)(l + 1) * (unsigned)G, abort_flag);
        named_bar_sync(1, kMmaThreads);
        CI_STAMP(stamps, sb, 7);
        // the target layer l + 2 will add into, if it is one of the rotating buffers: every CTA
        // has read it for the last time before it arrived at the barrier above
        if (!p.y_layers && l + 2 < p.L - 1) {
            float4* z = reinterpret_cast<float4*>(p.ybuf + (size_t)((l + 2) % 3) * row);
            for (int i = cta * kMmaThreads + tid; i < (int)(row / 4); i += G * kMmaThreads) z[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        // next input, per sequence: (x + y) / rms(x + y), rounded; the four lanes of a sequence
        // cover this warp's columns, the sixteen warps' sums of squares meet in shared memory
        {
            const float* yrow = ytarget + rowofs;
            float2 v[kMmaMaxTiles][2];
            float ss = 0.f;
#pragma unroll
            for (int t = 0; t < kMmaMaxTiles; ++t) {
                v[t][0] = v[t][1] = make_float2(0.f, 0.f);
                if (t < ntile && live) {
                    const int j = c0 + t * 16;
                    const float2 y0 = __ldcg(reinterpret_cast<const float2*>(yrow + j));
                    const float2 y1 = __ldcg(reinterpret_cast<const float2*>(yrow + j + 8));
                    v[t][0] = make_float2(__uint_as_float(xb[t][0] << 16) + y0.x, __uint_as_float(xb[t][0] & 0xffff0000u) + y0.y);
                    v[t][1] = make_float2(__uint_as_float(xb[t][1] << 16) + y1.x, __uint_as_float(xb[t][1] & 0xffff0000u) + y1.y);
                    ss = fmaf(v[t][0].x, v[t][0].x, ss);
                    ss = fmaf(v[t][0].y, v[t][0].y, ss);
                    ss = fmaf(v[t][1].x, v[t][1].x, ss);
                    ss = fmaf(v[t][1].y, v[t][1].y, ss);
                }
            }
            ss += __shfl_xor_sync(0xffffffffu, ss, 1);
            ss += __shfl_xor_sync(0xffffffffu, ss, 2);
            if ((lane & 3) == 0) ssq[warp * 8 + nb] = ss;
            named_bar_sync(1, kMmaThreads);
            CI_STAMP(stamps, sb, 8);
            if (tid == 0) *layers_done = l + 1;      // the sums have been read: the producer may go on
            float tot = 0.f;
#pragma unroll
            for (int w = 0; w < kMmaWarps; ++w) tot += ssq[w * 8 + nb];
            const float inv = rsqrtf(tot * p.inv_d);
            uint32_t* xd = (cta == (l + 1) % G && p.x_layers)
                               ? reinterpret_cast<uint32_t*>(p.x_layers + (size_t)(l + 1) * row + rowofs) : nullptr;
#pragma unroll
            for (int t = 0; t < kMmaMaxTiles; ++t) {
                xb[t][0] = xb[t][1] = 0u;
                if (t < ntile && live) {
                    const __nv_bfloat162 a = __floats2bfloat162_rn(v[t][0].x * inv, v[t][0].y * inv);
                    const __nv_bfloat162 b = __floats2bfloat162_rn(v[t][1].x * inv, v[t][1].y * inv);
                    xb[t][0] = *reinterpret_cast<const uint32_t*>(&a);
                    xb[t][1] = *reinterpret_cast<const uint32_t*>(&b);
                    if (xd) {
                        const int j = c0 + t * 16;
                        xd[j >> 1] = xb[t][0];
                        xd[(j + 8) >> 1] = xb[t][1];
                    }
                }
            }
        }
        CI_STAMP(stamps, sb, 9);
    }
}

// The stack in one launch; conditions as for decode_batched_mma, for every layer.  The caller has
// checked them (decode_batched_mma_serves), cleared ctrl (256 bytes), y_last, y_layers (when
// given) and the first two of the three rotating buffers at ybuf.
coreinfer_status decode_stack_batched_mma(const coreinfer_layer* layers, int L, const void* x0, int batch, bool gated,
                                          int silu, int d_model, float* y_last, float* y_layers, void* x_layers, float* ybuf,
                                          unsigned* ctrl, const DeviceInfo& di, cudaStream_t st)
{
    static thread_local MmaStackParams p;
    int Kmax = 0;
    for (int l = 0; l < L; ++l) {
        p.layers[l].up = (const uint8_t*)layers[l].w_up_c;
        p.layers[l].gate = (const uint8_t*)layers[l].w_gate_c;
        p.layers[l].down = (const uint8_t*)layers[l].w_downT_c;
        p.layers[l].bup = (const __nv_bfloat16*)layers[l].b_up_c;
        p.layers[l].bdown = (const __nv_bfloat16*)layers[l].b_down;
        p.layers[l].K = layers[l].K;
        p.layers[l].pad = 0;
        Kmax = layers[l].K > Kmax ? layers[l].K : Kmax;
    }
    p.L = L;
    p.silu = silu;
    p.d = d_model;
    p.B = batch;
    p.row_bytes = d_model * 2;
    p.slot_stride = p.row_bytes + 16;
    p.inv_d = 1.0f / (float)d_model;
    p.runahead = 16;        // one unit; 0 .. whole ring measured within 5 % of one another
    p.x0 = (const __nv_bfloat16*)x0;
    p.y_last = y_last;
    p.y_layers = y_layers;
    p.x_layers = (__nv_bfloat16*)x_layers;
    p.ybuf = ybuf;
    p.ctrl = ctrl;
    const int G = di.sm_count;
    p.stamps = stamps_buffer((size_t)G * L * kStampSlots * sizeof(unsigned long long));
    const int rmax = (Kmax + G - 1) / G + 1;
    p.rpad = ((rmax + 15) & ~15) + 16;      // the zeroed tail of h may reach one tile past the slab
    const size_t fixed = mma_fixed_smem(p.slot_stride, p.rpad);
    long long slots = ((long long)di.smem_optin - (long long)fixed) / p.slot_stride;
    if (slots > kMmaMaxSlots) slots = kMmaMaxSlots;
    if (slots < 17) return COREINFER_ERR_UNSUPPORTED;
    p.n_slots = (int)slots;
    const size_t smem = fixed + (size_t)p.n_slots * p.slot_stride;
    auto kern = gated ? decode_batch_stack_kernel<true> : decode_batch_stack_kernel<false>;
    CI_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)G);
    cfg.blockDim = dim3((unsigned)kMmaBlock);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;    // the CTAs wait on one another at layer ends
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    CI_CUDA(cudaLaunchKernelEx(&cfg, kern, p));
    return COREINFER_OK;
}

}  // namespace coreinfer
