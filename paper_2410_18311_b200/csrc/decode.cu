// Decode-stage FFN over compacted core-neuron weights (Section 4.2), batch 1.
//
// One persistent kernel, one CTA per SM.  Per layer a CTA owns a contiguous slab
// of the K core neurons and streams that slab's rows exactly once: first the up
// (and gate) rows to form h for its neurons, then the matching rows of the
// transposed down matrix to form its partial y.  Rows arrive through a ring of
// shared-memory slots filled by 1-D bulk copies (one elected producer thread,
// one mbarrier pair per slot).  The weights of a layer do not depend on its
// input, so the producer runs ahead across layer boundaries and HBM stays busy
// while the CTAs exchange partial outputs.
//
// Exchange per layer: every CTA adds its partial y (d_model fp32) into one
// global vector with vector reductions, then all CTAs meet at a grid barrier,
// read the full y, and each forms the next layer's input redundantly in
// registers.  Every wait (slot barriers, grid barrier) is bounded: when one
// gives up, the CTA marks the workspace status word, stops waiting everywhere,
// runs the rest of its schedule without synchronising on data, drains its own
// copies in flight and returns.
#include "common.cuh"

namespace coreinfer {

constexpr int kMaxSlots = 64;
constexpr int kConsumerThreads = 256;
constexpr int kConsumerWarps = kConsumerThreads / 32;
constexpr int kBlockThreads = kConsumerThreads + 32;   // + one producer warp
constexpr int kCtrlBytes = 256;                        // status word, barrier counter, padding
constexpr int kSplitRotate = 41;                       // per-layer rotation of the slab split
constexpr long long kWaitCycles = 3000000000LL;        // bound of every device-side wait (~1.5 s)

struct LayerDev {
    const uint8_t* up;
    const uint8_t* gate;
    const uint8_t* down;
    const void* bup;
    const void* bdown;
    int K;
    int pad;
};

struct DecodeParams {
    int L, d, nv, row_bytes, slot_bytes, n_slots, rmax;
    const void* x0;
    float* y_last;
    float* y_layers;
    void* x_layers;
    float* ybuf;        // [L-1][d]: reduction targets of layers 0 .. L-2
    unsigned* ctrl;     // [0] status word, [1] grid-barrier arrival counter
    LayerDev layers[COREINFER_MAX_LAYERS];
};

__host__ __device__ __forceinline__ void slab_of(int cta, int G, int layer, int K, int* k0, int* k1)
{
    int vc = (int)(((long long)cta + (long long)layer * kSplitRotate) % G);
    *k0 = (int)(((long long)vc * K) / G);
    *k1 = (int)(((long long)(vc + 1) * K) / G);
}

// ------------------------------------------------------------ element types --
template <typename T> struct Elem;
template <> struct Elem<__nv_bfloat16> {
    static constexpr int kPairs = 4;   // float2 per 16-byte vector
    static __device__ __forceinline__ void unpack(const uint4& q, float2 (&f)[4])
    {
        f[0] = make_float2(__uint_as_float(q.x << 16), __uint_as_float(q.x & 0xffff0000u));
        f[1] = make_float2(__uint_as_float(q.y << 16), __uint_as_float(q.y & 0xffff0000u));
        f[2] = make_float2(__uint_as_float(q.z << 16), __uint_as_float(q.z & 0xffff0000u));
        f[3] = make_float2(__uint_as_float(q.w << 16), __uint_as_float(q.w & 0xffff0000u));
    }
    static __device__ __forceinline__ float round(float v)
    {
        return __bfloat162float(__float2bfloat16_rn(v));
    }
    static __device__ __forceinline__ uint32_t pack2(float a, float b)
    {
        __nv_bfloat162 t = __floats2bfloat162_rn(a, b);
        return *reinterpret_cast<uint32_t*>(&t);
    }
    static __device__ __forceinline__ uint4 pack(const float2 (&f)[4])
    {
        return make_uint4(pack2(f[0].x, f[0].y), pack2(f[1].x, f[1].y), pack2(f[2].x, f[2].y),
                          pack2(f[3].x, f[3].y));
    }
    static __device__ __forceinline__ float load1(const void* p, int i)
    {
        return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p)[i]);
    }
};
template <> struct Elem<float> {
    static constexpr int kPairs = 2;
    static __device__ __forceinline__ void unpack(const uint4& q, float2 (&f)[2])
    {
        f[0] = make_float2(__uint_as_float(q.x), __uint_as_float(q.y));
        f[1] = make_float2(__uint_as_float(q.z), __uint_as_float(q.w));
    }
    static __device__ __forceinline__ float round(float v) { return v; }
    static __device__ __forceinline__ uint4 pack(const float2 (&f)[2])
    {
        return make_uint4(__float_as_uint(f[0].x), __float_as_uint(f[0].y), __float_as_uint(f[1].x),
                          __float_as_uint(f[1].y));
    }
    static __device__ __forceinline__ float load1(const void* p, int i)
    {
        return reinterpret_cast<const float*>(p)[i];
    }
};

// ------------------------------------------------------------- bounded waits --
// Returns false (and poisons the CTA) when the wait gives up.
__device__ __forceinline__ bool wait_slot(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          unsigned* status)
{
    if (*abort_flag) return false;
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > kWaitCycles) {
            *abort_flag = 1;
            atomicMax(status, (unsigned)kStatusTimeout);
            return false;
        }
    }
}

// All consumer threads call this.  The arrival counter is zeroed by the host before
// the launch; barrier number b (0-based) completes when it reaches (b + 1) * G.
__device__ __forceinline__ void grid_barrier(unsigned* ctrl, unsigned target,
                                             volatile int* abort_flag)
{
    named_bar_sync(1, kConsumerThreads);
    if (threadIdx.x == 0 && !*abort_flag) {
        __threadfence();
        atomicAdd(&ctrl[1], 1u);
        const long long t0 = clock64();
        for (;;) {
            if (ld_acquire_gpu(&ctrl[1]) >= target) break;
            if (ld_acquire_gpu(&ctrl[0]) != kStatusOk) { *abort_flag = 1; break; }
            if (clock64() - t0 > kWaitCycles) {
                *abort_flag = 1;
                atomicMax(&ctrl[0], (unsigned)kStatusTimeout);
                break;
            }
        }
        __threadfence();
    }
    named_bar_sync(1, kConsumerThreads);
}

// 8 values per lane -> 8 warp totals, one per group of 4 lanes (9 shuffles).
// On return lane l holds the total of value ((l>>4)&1)*4 + ((l>>3)&1)*2 + ((l>>2)&1).
__device__ __forceinline__ float warp_reduce8(const float (&v)[8], int lane)
{
    float a[4];
    const bool hi16 = lane & 16;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float send = hi16 ? v[i] : v[i + 4];
        float keep = hi16 ? v[i + 4] : v[i];
        a[i] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
    }
    float b[2];
    const bool hi8 = lane & 8;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        float send = hi8 ? a[i] : a[i + 2];
        float keep = hi8 ? a[i + 2] : a[i];
        b[i] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
    }
    const bool hi4 = lane & 4;
    float send = hi4 ? b[0] : b[1];
    float keep = hi4 ? b[1] : b[0];
    float c = keep + __shfl_xor_sync(0xffffffffu, send, 4);
    c += __shfl_xor_sync(0xffffffffu, c, 2);
    c += __shfl_xor_sync(0xffffffffu, c, 1);
    return c;
}

// ------------------------------------------------------------------- kernel --
// Ring stream order of one CTA and one layer (producer and consumers walk it in
// lock step): for each group of rows {g0 .. g0+R-1}: the up rows, then (gated)
// the gate rows; after all groups, the down rows k0 .. k1-1.
template <typename T, int VPT, bool GATED>
__global__ void __launch_bounds__(kBlockThreads, 1)
decode_stack_kernel(const __grid_constant__ DecodeParams p)
{
    using E = Elem<T>;
    constexpr int PAIRS = E::kPairs;
    constexpr int EPV = PAIRS * 2;               // elements per 16-byte vector
    constexpr int R = GATED ? 4 : 8;             // rows per up-phase group
    constexpr int NMAT = GATED ? 2 : 1;

    extern __shared__ __align__(128) uint8_t smem[];
    uint8_t* ring = smem;
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(ring + (size_t)p.n_slots * p.slot_bytes);
    uint64_t* empty_bar = full_bar + kMaxSlots;
    float* red = reinterpret_cast<float*>(empty_bar + kMaxSlots);   // [NMAT][warps][rmax]
    float* h_s = red + NMAT * kConsumerWarps * p.rmax;              // [rmax]
    float* ss_red = h_s + p.rmax;                                   // [warps]
    volatile int* abort_flag = reinterpret_cast<volatile int*>(ss_red + kConsumerWarps);

    const int tid = threadIdx.x;
    const int G = gridDim.x;
    const int cta = blockIdx.x;
    const int NS = p.n_slots;

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(smem_u32(&full_bar[s]), 1);
            mbar_init(smem_u32(&empty_bar[s]), kConsumerWarps);
        }
        *abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();

    // ======================================================== producer warp ==
    if (tid >= kConsumerThreads) {
        if (tid == kConsumerThreads) {
            long long it = 0;
            bool live = true;
            auto issue = [&](const uint8_t* src) {
                const int slot = (int)(it % NS);
                const uint32_t ph = (uint32_t)((it / NS) & 1);
                if (live && !wait_slot(smem_u32(&empty_bar[slot]), ph ^ 1u, abort_flag, p.ctrl))
                    live = false;
                if (live) {
                    const uint32_t fb = smem_u32(&full_bar[slot]);
                    mbar_arrive_expect_tx(fb, (uint32_t)p.row_bytes);
                    bulk_g2s(smem_u32(ring + (size_t)slot * p.slot_bytes), src, (uint32_t)p.row_bytes, fb);
                    ++it;
                }
            };
            for (int l = 0; l < p.L && live; ++l) {
                const LayerDev& ly = p.layers[l];
                int k0, k1;
                slab_of(cta, G, l, ly.K, &k0, &k1);
                for (int g0 = k0; g0 < k1 && live; g0 += R) {
                    const int ge = min(g0 + R, k1);
                    for (int k = g0; k < ge; ++k) issue(ly.up + (size_t)k * p.row_bytes);
                    if (GATED)
                        for (int k = g0; k < ge; ++k) issue(ly.gate + (size_t)k * p.row_bytes);
                }
                for (int k = k0; k < k1 && live; ++k) issue(ly.down + (size_t)k * p.row_bytes);
            }
            // Do not leave while a copy into this CTA's shared memory is in flight.
            const long long first = it > NS ? it - NS : 0;
            for (long long i = first; i < it; ++i) {
                const uint32_t fb = smem_u32(&full_bar[(int)(i % NS)]);
                const uint32_t ph = (uint32_t)((i / NS) & 1);
                const long long t0 = clock64();
                while (!mbar_try_wait(fb, ph))
                    if (clock64() - t0 > kWaitCycles) { atomicMax(p.ctrl, (unsigned)kStatusTimeout); break; }
            }
        }
        return;
    }

    // ============================================================ consumers ==
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const int nv = p.nv;
    const int d = p.d;

    // this thread's columns: 16-byte vectors tid, tid + 256, ...
    float2 xr[VPT][PAIRS];
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = tid + i * kConsumerThreads;
        uint4 q = make_uint4(0, 0, 0, 0);
        if (v < nv) q = reinterpret_cast<const uint4*>(p.x0)[v];
        E::unpack(q, xr[i]);
        if (p.x_layers && cta == 0 && v < nv) reinterpret_cast<uint4*>(p.x_layers)[v] = q;
    }
    if (p.L > 1) {   // reductions of the last layer land here after at least one grid barrier
        const uint4 z = make_uint4(0, 0, 0, 0);
        if (cta == 0)
            for (int i = tid; i < d / 4; i += kConsumerThreads) reinterpret_cast<uint4*>(p.y_last)[i] = z;
        if (p.y_layers && cta == 1 % G)
            for (int i = tid; i < d / 4; i += kConsumerThreads)
                reinterpret_cast<uint4*>(p.y_layers + (size_t)(p.L - 1) * d)[i] = z;
    }

    long long it = 0;
    auto acquire = [&]() -> const uint8_t* {
        const int slot = (int)(it % NS);
        wait_slot(smem_u32(&full_bar[slot]), (uint32_t)((it / NS) & 1), abort_flag, p.ctrl);
        return ring + (size_t)slot * p.slot_bytes;
    };
    auto release = [&]() {
        const int slot = (int)(it % NS);
        __syncwarp();
        if (lane == 0 && !*abort_flag) mbar_arrive(smem_u32(&empty_bar[slot]));
        ++it;
    };

    for (int l = 0; l < p.L; ++l) {
        const LayerDev& ly = p.layers[l];
        int k0, k1;
        slab_of(cta, G, l, ly.K, &k0, &k1);
        const int nrows = k1 - k0;

        // ------------------------------------------------ up (+ gate) phase --
        for (int g0 = k0; g0 < k1; g0 += R) {
            const int ge = min(g0 + R, k1);
            float part[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) part[j] = 0.f;
#pragma unroll
            for (int m = 0; m < NMAT; ++m) {
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    if (g0 + r < ge) {
                        const uint8_t* row = acquire();
                        float2 acc = make_float2(0.f, 0.f);
#pragma unroll
                        for (int i = 0; i < VPT; ++i) {
                            const int v = tid + i * kConsumerThreads;
                            if (v < nv) {
                                const uint4 q = *reinterpret_cast<const uint4*>(row + (size_t)v * 16);
                                float2 w[PAIRS];
                                E::unpack(q, w);
#pragma unroll
                                for (int c = 0; c < PAIRS; ++c) acc = __ffma2_rn(w[c], xr[i][c], acc);
                            }
                        }
                        release();
                        part[m * R + r] = acc.x + acc.y;
                    }
                }
            }
            const float tot = warp_reduce8(part, lane);
            if ((lane & 3) == 0) {
                const int j = ((lane >> 4) & 1) * 4 + ((lane >> 3) & 1) * 2 + ((lane >> 2) & 1);
                const int m = j / R, r = j % R;
                if (g0 + r < ge) red[(m * kConsumerWarps + warp) * p.rmax + (g0 - k0) + r] = tot;
            }
        }
        named_bar_sync(1, kConsumerThreads);
        for (int r = tid; r < nrows; r += kConsumerThreads) {
            float u = 0.f;
#pragma unroll
            for (int w = 0; w < kConsumerWarps; ++w) u += red[w * p.rmax + r];
            float h;
            if (GATED) {
                float g = 0.f;
#pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w) g += red[(kConsumerWarps + w) * p.rmax + r];
                h = fmaxf(g, 0.f) * u;
            } else {
                if (ly.bup) u += E::load1(ly.bup, k0 + r);
                h = fmaxf(u, 0.f);
            }
            h_s[r] = h;
        }
        named_bar_sync(1, kConsumerThreads);

        // ------------------------------------------------------- down phase --
        float2 yacc[VPT][PAIRS];
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int v = tid + i * kConsumerThreads;
#pragma unroll
            for (int c = 0; c < PAIRS; ++c) yacc[i][c] = make_float2(0.f, 0.f);
            if (cta == 0 && ly.bdown && v < nv) {   // the bias enters the sum exactly once
#pragma unroll
                for (int c = 0; c < PAIRS; ++c)
                    yacc[i][c] = make_float2(E::load1(ly.bdown, v * EPV + 2 * c),
                                             E::load1(ly.bdown, v * EPV + 2 * c + 1));
            }
        }
        for (int r = 0; r < nrows; ++r) {
            const uint8_t* row = acquire();
            const float hk = h_s[r];
            if (hk != 0.f) {
                const float2 hh = make_float2(hk, hk);
#pragma unroll
                for (int i = 0; i < VPT; ++i) {
                    const int v = tid + i * kConsumerThreads;
                    if (v < nv) {
                        const uint4 q = *reinterpret_cast<const uint4*>(row + (size_t)v * 16);
                        float2 w[PAIRS];
                        E::unpack(q, w);
#pragma unroll
                        for (int c = 0; c < PAIRS; ++c) yacc[i][c] = __ffma2_rn(w[c], hh, yacc[i][c]);
                    }
                }
            }
            release();
        }

        // ----------------------------------------- cross-CTA sum of partial y --
        const bool last = (l == p.L - 1);
        float* ytarget = last ? p.y_last : p.ybuf + (size_t)l * d;
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int v = tid + i * kConsumerThreads;
            if (v < nv) {
#pragma unroll
                for (int c = 0; c < PAIRS; c += 2) {
                    float* dst = ytarget + (size_t)v * EPV + 2 * c;
                    red_add_v4(dst, yacc[i][c].x, yacc[i][c].y, yacc[i][c + 1].x, yacc[i][c + 1].y);
                    if (last && p.y_layers)
                        red_add_v4(p.y_layers + (size_t)l * d + (size_t)v * EPV + 2 * c, yacc[i][c].x,
                                   yacc[i][c].y, yacc[i][c + 1].x, yacc[i][c + 1].y);
                }
            }
        }
        if (last) break;

        grid_barrier(p.ctrl, (unsigned)(l + 1) * (unsigned)G, abort_flag);

        // ------------------------- next input: (x + y) / rms(x + y), rounded --
        float ss = 0.f;
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int v = tid + i * kConsumerThreads;
            if (v < nv) {
#pragma unroll
                for (int c = 0; c < PAIRS; c += 2) {
                    const float4 t = __ldcg(reinterpret_cast<const float4*>(ytarget + (size_t)v * EPV + 2 * c));
                    if (p.y_layers && cta == l % G)
                        *reinterpret_cast<float4*>(p.y_layers + (size_t)l * d + (size_t)v * EPV + 2 * c) = t;
                    xr[i][c].x += t.x;
                    xr[i][c].y += t.y;
                    xr[i][c + 1].x += t.z;
                    xr[i][c + 1].y += t.w;
                }
#pragma unroll
                for (int c = 0; c < PAIRS; ++c) {
                    ss = fmaf(xr[i][c].x, xr[i][c].x, ss);
                    ss = fmaf(xr[i][c].y, xr[i][c].y, ss);
                }
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        if (lane == 0) ss_red[warp] = ss;
        named_bar_sync(1, kConsumerThreads);
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) tot += ss_red[w];
        const float inv = 1.0f / sqrtf(tot / (float)d);
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int v = tid + i * kConsumerThreads;
#pragma unroll
            for (int c = 0; c < PAIRS; ++c) {
                xr[i][c].x = E::round(xr[i][c].x * inv);
                xr[i][c].y = E::round(xr[i][c].y * inv);
            }
            if (p.x_layers && cta == (l + 1) % G && v < nv)
                reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(p.x_layers) +
                                         (size_t)(l + 1) * p.row_bytes)[v] = E::pack(xr[i]);
        }
    }
}

// ------------------------------------------------------------------- host ---
static size_t fixed_smem_bytes(int rmax, bool gated)
{
    size_t b = 2 * kMaxSlots * sizeof(uint64_t);
    b += (size_t)(gated ? 2 : 1) * kConsumerWarps * rmax * sizeof(float);
    b += (size_t)rmax * sizeof(float);
    b += kConsumerWarps * sizeof(float) + 16;
    return (b + 127) & ~(size_t)127;
}

template <typename T, int VPT, bool GATED>
static coreinfer_status launch_one(const DecodeParams& p, int grid, size_t smem, bool cooperative,
                                   cudaStream_t st)
{
    auto kern = decode_stack_kernel<T, VPT, GATED>;
    static thread_local size_t configured[64] = {0};
    int dev = 0;
    CI_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64 || configured[dev] < smem) {
        CI_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        if (dev >= 0 && dev < 64) configured[dev] = smem;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kBlockThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = cooperative ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    CI_CUDA(cudaLaunchKernelEx(&cfg, kern, p));
    return COREINFER_OK;
}

template <typename T, bool GATED>
static coreinfer_status launch_vpt(int vpt, const DecodeParams& p, int grid, size_t smem, bool coop,
                                   cudaStream_t st)
{
    if (vpt <= 1) return launch_one<T, 1, GATED>(p, grid, smem, coop, st);
    if (vpt <= 2) return launch_one<T, 2, GATED>(p, grid, smem, coop, st);
    if (vpt <= 3) return launch_one<T, 3, GATED>(p, grid, smem, coop, st);
    if (vpt <= 5) return launch_one<T, 5, GATED>(p, grid, smem, coop, st);
    return launch_one<T, 8, GATED>(p, grid, smem, coop, st);
}

static coreinfer_status check_common(const void* x, int batch, coreinfer_dtype dtype,
                                     coreinfer_ffn_kind kind, int d_model)
{
    if (dtype != COREINFER_F32 && dtype != COREINFER_BF16)
        CI_FAIL(COREINFER_ERR_UNSUPPORTED, "dtype %d is not supported", (int)dtype);
    if (kind != COREINFER_FFN_RELU && kind != COREINFER_FFN_RELU_GATED)
        CI_FAIL(COREINFER_ERR_UNSUPPORTED, "ffn kind %d is not supported", (int)kind);
    if (batch < 1 || batch > COREINFER_MAX_BATCH)
        CI_FAIL(COREINFER_ERR_UNSUPPORTED, "batch %d outside 1..%d", batch, COREINFER_MAX_BATCH);
    if (d_model < 1 || ((size_t)d_model * dtype_size(dtype)) % 16 != 0)
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "d_model %d: a row must be a positive multiple of 16 bytes", d_model);
    if (!x || !aligned16(x)) CI_FAIL(COREINFER_ERR_INVALID_ARG, "x is NULL or not 16-byte aligned");
    return COREINFER_OK;
}

static coreinfer_status check_layer(const coreinfer_layer& ly, int l, coreinfer_ffn_kind kind)
{
    const bool gated = kind == COREINFER_FFN_RELU_GATED;
    if (ly.K < 1) CI_FAIL(COREINFER_ERR_INVALID_ARG, "layer %d: K = %d < 1", l, ly.K);
    if (!ly.w_up_c || !ly.w_downT_c || !aligned16(ly.w_up_c) || !aligned16(ly.w_downT_c))
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "layer %d: w_up_c / w_downT_c NULL or not 16-byte aligned", l);
    if (gated && (!ly.w_gate_c || !aligned16(ly.w_gate_c)))
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "layer %d: gated FFN needs a 16-byte aligned w_gate_c", l);
    if (!gated && ly.w_gate_c) CI_FAIL(COREINFER_ERR_INVALID_ARG, "layer %d: w_gate_c given for a non-gated FFN", l);
    if (gated && ly.b_up_c) CI_FAIL(COREINFER_ERR_INVALID_ARG, "layer %d: the gated FFN has no up bias", l);
    return COREINFER_OK;
}

// Shared by the one-layer and the stack entry points (batch 1).
static coreinfer_status decode_stack_b1(const coreinfer_layer* layers, int L, const void* x0,
                                        coreinfer_dtype dtype, coreinfer_ffn_kind kind, int d_model,
                                        float* y_last, float* y_layers, void* x_layers,
                                        void* workspace, size_t workspace_bytes, size_t need_ws,
                                        cudaStream_t st)
{
    DeviceInfo di;
    coreinfer_status s = device_info(&di);
    if (s != COREINFER_OK) return s;
    if (!workspace || !aligned16(workspace)) CI_FAIL(COREINFER_ERR_WORKSPACE, "workspace is NULL or misaligned");
    if (workspace_bytes < need_ws)
        CI_FAIL(COREINFER_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, need_ws);
    const bool gated = kind == COREINFER_FFN_RELU_GATED;
    const size_t esize = dtype_size(dtype);

    static thread_local DecodeParams p;   // large; filled per call, passed by value to the launch
    p.L = L;
    p.d = d_model;
    p.row_bytes = (int)(d_model * esize);
    p.nv = p.row_bytes / 16;
    p.slot_bytes = (p.row_bytes + 127) & ~127;
    const int G = di.sm_count;
    int Kmax = 0;
    for (int l = 0; l < L; ++l) {
        s = check_layer(layers[l], l, kind);
        if (s != COREINFER_OK) return s;
        p.layers[l].up = (const uint8_t*)layers[l].w_up_c;
        p.layers[l].gate = (const uint8_t*)layers[l].w_gate_c;
        p.layers[l].down = (const uint8_t*)layers[l].w_downT_c;
        p.layers[l].bup = layers[l].b_up_c;
        p.layers[l].bdown = layers[l].b_down;
        p.layers[l].K = layers[l].K;
        p.layers[l].pad = 0;
        if (layers[l].K > Kmax) Kmax = layers[l].K;
    }
    p.rmax = (Kmax + G - 1) / G + 1;
    const int vpt = (p.nv + kConsumerThreads - 1) / kConsumerThreads;
    if (vpt > 8)
        CI_FAIL(COREINFER_ERR_UNSUPPORTED, "d_model %d is too wide for this kernel (max %d bytes per row)",
                d_model, 8 * kConsumerThreads * 16);
    const size_t fixed = fixed_smem_bytes(p.rmax, gated);
    if (fixed + (size_t)p.slot_bytes > (size_t)di.smem_optin)
        CI_FAIL(COREINFER_ERR_UNSUPPORTED, "K = %d, d_model = %d do not fit in shared memory", Kmax, d_model);
    long long slots = ((long long)di.smem_optin - (long long)fixed) / p.slot_bytes;
    if (slots > kMaxSlots) slots = kMaxSlots;
    p.n_slots = (int)slots;
    const size_t smem = fixed + (size_t)p.n_slots * p.slot_bytes;
    p.x0 = x0;
    p.y_last = y_last;
    p.y_layers = y_layers;
    p.x_layers = x_layers;
    p.ctrl = (unsigned*)workspace;
    p.ybuf = (float*)((uint8_t*)workspace + kCtrlBytes);

    // Control words and the reduction targets start at zero.
    if (L > 1) {
        CI_CUDA(cudaMemsetAsync(workspace, 0, kCtrlBytes + (size_t)(L - 1) * d_model * sizeof(float), st));
    } else {
        CI_CUDA(cudaMemsetAsync(workspace, 0, kCtrlBytes, st));
        CI_CUDA(cudaMemsetAsync(y_last, 0, (size_t)d_model * sizeof(float), st));
        if (y_layers) CI_CUDA(cudaMemsetAsync(y_layers, 0, (size_t)d_model * sizeof(float), st));
    }
    const bool coop = L > 1;
    if (dtype == COREINFER_BF16)
        return gated ? launch_vpt<__nv_bfloat16, true>(vpt, p, G, smem, coop, st)
                     : launch_vpt<__nv_bfloat16, false>(vpt, p, G, smem, coop, st);
    return gated ? launch_vpt<float, true>(vpt, p, G, smem, coop, st)
                 : launch_vpt<float, false>(vpt, p, G, smem, coop, st);
}

// decode_batch.cu
coreinfer_status decode_batched(const void* x, int batch, coreinfer_dtype dtype, coreinfer_ffn_kind kind,
                                int d_model, const coreinfer_layer& ly, float* y, void* workspace,
                                cudaStream_t st);

}  // namespace coreinfer

using namespace coreinfer;

extern "C" {

size_t coreinfer_ffn_decode_workspace_bytes(int32_t batch, int32_t d_model, int32_t K)
{
    if (batch < 1 || d_model < 1 || K < 1) return 0;
    if (batch == 1) return kCtrlBytes;
    return kCtrlBytes + (size_t)batch * (size_t)K * sizeof(float);   // h [batch, K]
}

size_t coreinfer_ffn_decode_stack_workspace_bytes(int32_t L, int32_t batch, int32_t d_model, int32_t K_max)
{
    (void)K_max;
    if (L < 1 || batch < 1 || d_model < 1) return 0;
    return kCtrlBytes + (size_t)L * (size_t)batch * (size_t)d_model * sizeof(float);
}

coreinfer_status coreinfer_ffn_decode(const void* x, int32_t batch, coreinfer_dtype dtype,
                                      coreinfer_ffn_kind kind, int32_t d_model, int32_t K,
                                      const void* w_up_c, const void* w_gate_c, const void* w_downT_c,
                                      const void* b_up_c, const void* b_down, float* y,
                                      void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    coreinfer_status s = check_common(x, batch, dtype, kind, d_model);
    if (s != COREINFER_OK) return s;
    if (!y || !aligned16(y)) CI_FAIL(COREINFER_ERR_INVALID_ARG, "y is NULL or not 16-byte aligned");
    coreinfer_layer ly = {w_up_c, w_gate_c, w_downT_c, b_up_c, b_down, K, 0};
    s = check_layer(ly, 0, kind);
    if (s != COREINFER_OK) return s;
    const size_t need = coreinfer_ffn_decode_workspace_bytes(batch, d_model, K);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (batch == 1)
        return decode_stack_b1(&ly, 1, x, dtype, kind, d_model, y, nullptr, nullptr, workspace,
                               workspace_bytes, need, st);
    if (!workspace || !aligned16(workspace)) CI_FAIL(COREINFER_ERR_WORKSPACE, "workspace is NULL or misaligned");
    if (workspace_bytes < need)
        CI_FAIL(COREINFER_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, need);
    return decode_batched(x, batch, dtype, kind, d_model, ly, y, workspace, st);
}

coreinfer_status coreinfer_ffn_decode_stack(const coreinfer_layer* layers, int32_t L, const void* x0,
                                            int32_t batch, coreinfer_dtype dtype,
                                            coreinfer_ffn_kind kind, int32_t d_model, float* y_last,
                                            float* y_layers, void* x_layers, void* workspace,
                                            size_t workspace_bytes, void* cuda_stream)
{
    coreinfer_status s = check_common(x0, batch, dtype, kind, d_model);
    if (s != COREINFER_OK) return s;
    if (batch != 1) CI_FAIL(COREINFER_ERR_UNSUPPORTED, "the stack entry point is built for batch 1 (got %d)", batch);
    if (!layers) CI_FAIL(COREINFER_ERR_INVALID_ARG, "layers is NULL");
    if (L < 1 || L > COREINFER_MAX_LAYERS)
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "L = %d outside 1..%d", L, COREINFER_MAX_LAYERS);
    if (!y_last || !aligned16(y_last)) CI_FAIL(COREINFER_ERR_INVALID_ARG, "y_last is NULL or not 16-byte aligned");
    if ((y_layers && !aligned16(y_layers)) || (x_layers && !aligned16(x_layers)))
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "y_layers / x_layers not 16-byte aligned");
    const size_t need = coreinfer_ffn_decode_stack_workspace_bytes(L, batch, d_model, 0);
    return decode_stack_b1(layers, L, x0, dtype, kind, d_model, y_last, y_layers, x_layers, workspace,
                           workspace_bytes, need, (cudaStream_t)cuda_stream);
}


// ---------------------------------------------------------------------------
// Variant of the stack entry point that needs no workspace from the caller.
//
// Some callers cannot obtain device memory at the time they decode: an inference server that
// handed every free byte of HBM to its own pools at start-up, a plug-in that runs inside a host
// framework which forbids cudaMalloc on its threads because the call synchronises the whole
// device, a latency-critical loop in which an allocator call is not acceptable.  For them the
// scratch of the stack kernel (control words + the per-layer reduction targets) lives in a
// fixed array inside the library image.  The array costs kNoAllocScratchBytes of HBM on every
// GPU that loads the library, for the life of the process.
constexpr size_t kNoAllocScratchBytes = 4u << 20;   // 4 MiB: L * d_model * 4 + 256 must fit
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

// The array's name is only a handle on the host; its device address comes from
// cudaGetSymbolAddress, once per device, with that device current.
static coreinfer_status noalloc_scratch_ptr(void** out)
{
    static thread_local void* cached[64] = {nullptr};
    int dev = 0;
    CI_CUDA(cudaGetDevice(&dev));
    if (dev >= 0 && dev < 64 && cached[dev]) {
        *out = cached[dev];
        return COREINFER_OK;
    }
    void* p = nullptr;
    CI_CUDA(cudaGetSymbolAddress(&p, g_noalloc_scratch));
    if (!p) CI_FAIL(COREINFER_ERR_CUDA, "cudaGetSymbolAddress returned a NULL address");
    if (dev >= 0 && dev < 64) cached[dev] = p;
    *out = p;
    return COREINFER_OK;
}

coreinfer_status coreinfer_ffn_decode_stack_noalloc(const coreinfer_layer* layers, int32_t L,
                                                    const void* x0, int32_t batch,
                                                    coreinfer_dtype dtype, coreinfer_ffn_kind kind,
                                                    int32_t d_model, float* y_last, float* y_layers,
                                                    void* x_layers, void* cuda_stream)
{
    coreinfer_status s = check_common(x0, batch, dtype, kind, d_model);
    if (s != COREINFER_OK) return s;
    if (batch != 1) CI_FAIL(COREINFER_ERR_UNSUPPORTED, "the stack entry point is built for batch 1 (got %d)", batch);
    if (!layers) CI_FAIL(COREINFER_ERR_INVALID_ARG, "layers is NULL");
    if (L < 1 || L > COREINFER_MAX_LAYERS)
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "L = %d outside 1..%d", L, COREINFER_MAX_LAYERS);
    if (!y_last || !aligned16(y_last)) CI_FAIL(COREINFER_ERR_INVALID_ARG, "y_last is NULL or not 16-byte aligned");
    if ((y_layers && !aligned16(y_layers)) || (x_layers && !aligned16(x_layers)))
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "y_layers / x_layers not 16-byte aligned");
    const size_t need = coreinfer_ffn_decode_stack_workspace_bytes(L, batch, d_model, 0);
    if (need > kNoAllocScratchBytes)
        CI_FAIL(COREINFER_ERR_UNSUPPORTED,
                "L = %d, d_model = %d need %zu bytes of scratch; the built-in scratch holds %zu "
                "(use coreinfer_ffn_decode_stack with a workspace)", L, d_model, need, kNoAllocScratchBytes);
    void* scratch = nullptr;
    s = noalloc_scratch_ptr(&scratch);
    if (s != COREINFER_OK) return s;
    // decode_stack_b1 zeroes the control words and the reduction targets it uses on the stream
    // before the launch, so whatever the previous call left in the array does not matter.
    return decode_stack_b1(layers, L, x0, dtype, kind, d_model, y_last, y_layers, x_layers, scratch,
                           kNoAllocScratchBytes, need, (cudaStream_t)cuda_stream);
}

}  // extern "C"
