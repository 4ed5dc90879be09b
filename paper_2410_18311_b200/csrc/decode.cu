// Decode-stage FFN over compacted core-neuron weights (Section 4.2), batch 1.
//
// One persistent kernel, one CTA per SM.  Per layer a CTA owns a contiguous slab of the K core
// neurons and streams that slab's rows exactly once: first the up (and gate) rows to form h for
// its neurons, then the matching rows of the transposed down matrix to form its partial y.
// Rows arrive in batches of BATCH rows through a ring of shared-memory batch slots filled by 1-D
// bulk copies (a producer warp; one full/empty mbarrier pair per batch slot, all rows of a batch
// complete on the same barrier).  The weights of a layer do not depend on its input, so the
// producer runs ahead across layer boundaries.
//
// Consumers own columns: thread t holds the x values of its 16-byte vectors t, t + NC, ... in
// registers for the whole layer and its partial y likewise.  They walk the stream of batches with
// two register buffers: the rows of the next batch are requested from shared memory (one barrier
// test, BATCH * VPT 16-byte loads, the slot freed at once) before the arithmetic of the current
// batch starts, so that barrier and shared-memory latencies are hidden behind the arithmetic; the
// per-row costs of a warp are one sixteen-byte load per vector and its multiply-adds.
//
// Exchange per layer: the CTA's partial y (d_model fp32) is assembled in shared memory and added
// into a global vector with one bulk reduction; one lane of a third kind of warp, the exchange
// warp, waits for it, arrives at a grid barrier (release), polls for everybody else's arrival
// (acquire) and brings the sum back with one bulk copy, on whose barrier the consumers sleep --
// after they have pulled the first two batches of the next layer into their register buffers,
// which frees two more batch slots for the producer; every thread then forms its columns of the
// next layer's input.  While the exchange is on, the producer requests only a limited
// number of rows: a first part before the exchange (landed by then), a second part once this
// CTA's arrival is out (a fence waits for the SM's bulk copies in flight, so none is issued
// before), paced.  Every wait (slot barriers, grid barrier, read-back) is bounded: when one gives
// up, the CTA marks the workspace status word, stops waiting everywhere, runs the rest of its
// schedule without synchronising on data, drains its own copies in flight and returns.
#include "common.cuh"

#include <stdlib.h>

namespace coreinfer {

constexpr int kMaxBatchSlots = 64;
constexpr int kMaxConsumers = 512;                     // consumer threads per CTA (16 warps) + one producer warp
constexpr int kMaxWarps = kMaxConsumers / 32;
constexpr int kMaxVpt = 3;                             // 16-byte vectors of a row per consumer thread
constexpr int kCtrlBytes = 256;                        // status word, barrier counter, padding
constexpr int kYBuffers = 3;                           // rotating reduction targets: in use, being read, being cleared
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
    int L, d, nv, row_bytes, slot_bytes, n_bslots, rmax;
    int nc;             // consumer threads (a multiple of 32); the producer warp follows them
    int runahead;       // batches of the next layer requested before this layer's exchange is over
    int trickle;        // further batches, requested one by one once this CTA's arrival at the grid barrier is out
    int trickle_gap;    // cycles between two such requests
    int silu;           // gated FFN: 0 ReLU gate, 1 SiLU gate
    float inv_d;        // 1 / d_model
    int ysum_ofs;       // shared-memory offset of the buffer holding the CTA's partial y
    const void* x0;
    float* y_last;
    float* y_layers;
    void* x_layers;
    float* ybuf;        // [kYBuffers][d]: reduction targets, buffer l % 3 serves layer l
    unsigned* ctrl;     // [0] status word, [1] grid-barrier arrival counter
    unsigned long long* stamps;   // [CTA][layer][kStampSlots] cycle counts, or NULL (COREINFER_STAMPS builds)
    LayerDev layers[COREINFER_MAX_LAYERS];
};

// 32-bit arithmetic (a 64-bit division costs several hundred cycles per layer on the device);
// the host refuses K * G >= 2^32.
__host__ __device__ __forceinline__ void slab_of(int cta, int G, int layer, int K, int* k0, int* k1)
{
    const unsigned g = (unsigned)G;
    const unsigned vc = ((unsigned)cta + (unsigned)layer * (unsigned)kSplitRotate) % g;
    *k0 = (int)(vc * (unsigned)K / g);
    *k1 = (int)((vc + 1u) * (unsigned)K / g);
}

// rows per batch (register budget: two buffers of 4 * rows * vectors per thread)
__host__ __device__ constexpr int batch_for(int vpt) { return vpt <= 1 ? 4 : 2; }
// consumer threads at most: with three vectors per thread 14 warps, which leaves 128 registers a thread
__host__ __device__ constexpr int max_consumers(int vpt) { return vpt <= 2 ? kMaxConsumers : 448; }

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
    // a0 += sum of even-position products, a1 += sum of odd-position products of the 8 bf16
    // pairs (w, x): mixed-precision FMA, the bf16 product is exact in fp32, one rounding per add
    static __device__ __forceinline__ void dot(const uint4& w, const uint4& x, float& a0, float& a1)
    {
        const uint32_t ws[4] = {w.x, w.y, w.z, w.w}, xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int c = 0; c < 4; ++c)
            asm("{\n\t.reg .b16 wl, wh, xl, xh;\n\t"
                "mov.b32 {wl, wh}, %2;\n\tmov.b32 {xl, xh}, %3;\n\t"
                "fma.rn.f32.bf16 %0, wl, xl, %0;\n\tfma.rn.f32.bf16 %1, wh, xh, %1;\n\t}"
                : "+f"(a0), "+f"(a1) : "r"(ws[c]), "r"(xs[c]));
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
template <> struct Elem<__half> {
    static constexpr int kPairs = 4;
    static __device__ __forceinline__ void unpack(const uint4& q, float2 (&f)[4])
    {
        const __half2* h = reinterpret_cast<const __half2*>(&q);
#pragma unroll
        for (int c = 0; c < 4; ++c) f[c] = __half22float2(h[c]);
    }
    // as for bf16: mixed-precision FMA, the fp16 product is exact in fp32, one rounding per add
    static __device__ __forceinline__ void dot(const uint4& w, const uint4& x, float& a0, float& a1)
    {
        const uint32_t ws[4] = {w.x, w.y, w.z, w.w}, xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int c = 0; c < 4; ++c)
            asm("{\n\t.reg .b16 wl, wh, xl, xh;\n\t"
                "mov.b32 {wl, wh}, %2;\n\tmov.b32 {xl, xh}, %3;\n\t"
                "fma.rn.f32.f16 %0, wl, xl, %0;\n\tfma.rn.f32.f16 %1, wh, xh, %1;\n\t}"
                : "+f"(a0), "+f"(a1) : "r"(ws[c]), "r"(xs[c]));
    }
    static __device__ __forceinline__ uint32_t pack2(float a, float b)
    {
        __half2 t = __floats2half2_rn(a, b);
        return *reinterpret_cast<uint32_t*>(&t);
    }
    static __device__ __forceinline__ uint4 pack(const float2 (&f)[4])
    {
        return make_uint4(pack2(f[0].x, f[0].y), pack2(f[1].x, f[1].y), pack2(f[2].x, f[2].y),
                          pack2(f[3].x, f[3].y));
    }
    static __device__ __forceinline__ float load1(const void* p, int i)
    {
        return __half2float(reinterpret_cast<const __half*>(p)[i]);
    }
};
template <> struct Elem<float> {
    static constexpr int kPairs = 2;
    static __device__ __forceinline__ void unpack(const uint4& q, float2 (&f)[2])
    {
        f[0] = make_float2(__uint_as_float(q.x), __uint_as_float(q.y));
        f[1] = make_float2(__uint_as_float(q.z), __uint_as_float(q.w));
    }
    static __device__ __forceinline__ void dot(const uint4& w, const uint4& x, float& a0, float& a1)
    {
        a0 = fmaf(__uint_as_float(w.x), __uint_as_float(x.x), a0);
        a1 = fmaf(__uint_as_float(w.y), __uint_as_float(x.y), a1);
        a0 = fmaf(__uint_as_float(w.z), __uint_as_float(x.z), a0);
        a1 = fmaf(__uint_as_float(w.w), __uint_as_float(x.w), a1);
    }
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
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    const long long t0 = clock64();
    for (;;) {
        if (mbar_try_wait_parked(bar, parity, 4000u)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > kWaitCycles) {
            *abort_flag = 1;
            atomicMax(status, (unsigned)kStatusTimeout);
            return false;
        }
    }
}

// Grid barrier: one thread per CTA, after it has seen the CTA's work complete, arrives with
// red_release_add(&ctrl[1], 1) and then calls this.  The arrival counter is zeroed by the host
// before the launch; barrier number b (0-based) completes when it reaches (b + 1) * G.  The
// arrival is a release at GPU scope (what this thread has observed, the completed bulk reduction
// and the CTA's earlier plain writes included, becomes visible before it), the poll an acquire.
__device__ __forceinline__ void grid_wait(unsigned* ctrl, unsigned target, volatile int* abort_flag)
{
    const long long t0 = clock64();
    unsigned it = 0;
    for (;;) {
        if (ld_acquire_gpu(&ctrl[1]) >= target) break;
        __nanosleep(32);
        if ((++it & 255u) == 0u) {             // now and then: has another CTA given up? out of time?
            if (ld_acquire_gpu(&ctrl[0]) != kStatusOk) { *abort_flag = 1; break; }
            if (clock64() - t0 > kWaitCycles) {
                *abort_flag = 1;
                atomicMax(&ctrl[0], (unsigned)kStatusTimeout);
                break;
            }
        }
    }
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

// 4 values per lane -> 4 warp totals, one per group of 8 lanes (5 shuffles).
// On return lane l holds the total of value ((l>>4)&1)*2 + ((l>>3)&1).
__device__ __forceinline__ float warp_reduce4(const float (&v)[4], int lane)
{
    float a[2];
    const bool hi16 = lane & 16;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        float send = hi16 ? v[i] : v[i + 2];
        float keep = hi16 ? v[i + 2] : v[i];
        a[i] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
    }
    const bool hi8 = lane & 8;
    float send = hi8 ? a[0] : a[1];
    float keep = hi8 ? a[1] : a[0];
    float c = keep + __shfl_xor_sync(0xffffffffu, send, 8);
    c += __shfl_xor_sync(0xffffffffu, c, 4);
    c += __shfl_xor_sync(0xffffffffu, c, 2);
    c += __shfl_xor_sync(0xffffffffu, c, 1);
    return c;
}

__device__ __forceinline__ float warp_reduce_n(const float (&v)[8], int lane) { return warp_reduce8(v, lane); }
__device__ __forceinline__ float warp_reduce_n(const float (&v)[4], int lane) { return warp_reduce4(v, lane); }

// ------------------------------------------------------------------- kernel --
// Ring stream order of one CTA and one layer (producer and consumers walk it in lock step): for
// each slab row k0 .. k1-1 its up row, then (gated) its gate row; after those, the down rows
// k0 .. k1-1.  Each of the two phases is cut into batches of BATCH rows (the last one of a phase
// may hold fewer); every batch takes one batch slot of the ring, whatever it holds.
template <typename T, int VPT, bool GATED>
__global__ void __launch_bounds__(max_consumers(VPT) + 64, 1)
decode_stack_kernel(const __grid_constant__ DecodeParams p)
{
    using E = Elem<T>;
    constexpr int PAIRS = E::kPairs;
    constexpr int EPV = PAIRS * 2;                   // elements per 16-byte vector
    constexpr int NMAT = GATED ? 2 : 1;
    constexpr int BATCH = batch_for(VPT);            // rows per batch
    constexpr int WIN = 2 * BATCH;                   // row sums per cross-lane reduction: one turn of the two register buffers

    extern __shared__ __align__(128) uint8_t smem[];
    const int NB = p.n_bslots;
    const int NC = p.nc;
    const int nwarps = NC >> 5;
    const uint32_t bslot_bytes = (uint32_t)BATCH * (uint32_t)p.slot_bytes;
    uint8_t* ring = smem;
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(ring + (size_t)NB * bslot_bytes);
    uint64_t* empty_bar = full_bar + kMaxBatchSlots;
    uint64_t* y_bar = empty_bar + kMaxBatchSlots;                   // completion of the read-back copy (+ 8 bytes padding)
    float* red = reinterpret_cast<float*>(y_bar + 2);               // [NMAT][nwarps][rmax]
    float* h_s = red + NMAT * nwarps * p.rmax;                      // [rmax]
    float* ss_red = h_s + p.rmax;                                   // [kMaxWarps]
    volatile int* abort_flag = reinterpret_cast<volatile int*>(ss_red + kMaxWarps);
    volatile int* layers_done = abort_flag + 1;                     // layers whose exchange this CTA has completed
    volatile int* arrived = abort_flag + 2;                         // layers for which this CTA's grid-barrier arrival is out
    float* ysum = reinterpret_cast<float*>(smem + p.ysum_ofs);      // [d]: the CTA's partial y, then the sum

    const int tid = threadIdx.x;
    const int G = gridDim.x;
    const int cta = blockIdx.x;

    if (tid == 0) {
        for (int s = 0; s < NB; ++s) {
            mbar_init(smem_u32(&full_bar[s]), 1);
            mbar_init(smem_u32(&empty_bar[s]), (uint32_t)nwarps);   // one arrival per consumer warp
        }
        mbar_init(smem_u32(y_bar), 1);
        *abort_flag = 0;
        *layers_done = 0;
        *arrived = 0;
        mbar_fence_init();
    }
    if (tid < kMaxWarps) ss_red[tid] = 0.f;
    __syncthreads();

    // ======================================================== producer warp ==
    // Eight lanes issue copies: one round fills up to 8 / BATCH consecutive batch slots, lane j
    // taking row j % BATCH of batch j / BATCH of the round.  Every lane waits for its batch slot to
    // be free; the lane of the batch's first row announces the bytes of the whole batch.
    if (tid >= NC && tid < NC + 32) {
        const int lane = tid - NC;
        constexpr int RB = 8 / BATCH;
        const int round_max = NB < RB ? NB : RB;
        int bs0 = 0;                  // batch slot of the round's first batch
        uint32_t phase0 = 0;          // parity of the ring pass that slot belongs to
        long long issued = 0;         // batches
        for (int l = 0; l < p.L; ++l) {
            const LayerDev& ly = p.layers[l];
            int k0, k1;
            slab_of(cta, G, l, ly.K, &k0, &k1);
            const int n = k1 - k0;
            const int n_up = n * NMAT;                               // rows of the up (+ gate) phase
            const int nbu = (n_up + BATCH - 1) / BATCH;              // its batches
            const int nbt = nbu + (n + BATCH - 1) / BATCH;           // + those of the down rows
            long long t_next = 0;                                    // earliest time of the next paced request
            for (int b0 = 0, cnt = 0; b0 < nbt; b0 += cnt) {
                if (*abort_flag) break;
                cnt = min(round_max, nbt - b0);
                // Requests in flight delay the few small messages of the previous layer's exchange,
                // and its fence waits for this SM's copies in flight.  So while that exchange is on,
                // only `runahead` batches of this layer are requested at once (they have landed
                // when the exchange starts); `trickle` more follow one at a time, `trickle_gap`
                // cycles apart, after this CTA's arrival at the grid barrier is out; the rest wait
                // for the end of the exchange.  Lane 0 decides for the warp.
                int limited = 0;
                if (l > 0 && b0 + cnt > p.runahead) {
                    limited = *layers_done < l;
                    limited = __shfl_sync(0xffffffffu, limited, 0);
                }
                if (limited) {
                    if (b0 < p.runahead) {
                        cnt = p.runahead - b0;
                    } else {
                        int go = 0;                                  // 1: one paced batch, 2: the exchange is over
                        if (lane == 0) {
                            const long long t0 = clock64();
                            for (;;) {
                                if (*layers_done >= l || *abort_flag) { go = 2; break; }
                                const long long now = clock64();
                                if (b0 < p.runahead + p.trickle && *arrived >= l && now >= t_next) {
                                    t_next = now + p.trickle_gap;
                                    go = 1;
                                    break;
                                }
                                __nanosleep(32);
                                if (now - t0 > kWaitCycles) { *abort_flag = 1; atomicMax(p.ctrl, (unsigned)kStatusTimeout); }
                            }
                        }
                        go = __shfl_sync(0xffffffffu, go, 0);
                        if (go == 1) cnt = 1;
                    }
                }
                if (lane < cnt * BATCH) {
                    const int bi = lane / BATCH, r = lane % BATCH;
                    const int b = b0 + bi;
                    const uint8_t* src = nullptr;                    // stays NULL for a row the batch does not hold
                    int nreal;
                    if (b < nbu) {
                        const int q = b * BATCH + r;
                        nreal = min(BATCH, n_up - b * BATCH);
                        if (q < n_up)
                            src = ((GATED && (q % NMAT)) ? ly.gate : ly.up) + (size_t)(k0 + q / NMAT) * p.row_bytes;
                    } else {
                        const int q = (b - nbu) * BATCH + r;
                        nreal = min(BATCH, n - (b - nbu) * BATCH);
                        if (q < n) src = ly.down + (size_t)(k0 + q) * p.row_bytes;
                    }
                    int bs = bs0 + bi;
                    uint32_t ph = phase0;
                    if (bs >= NB) { bs -= NB; ph ^= 1u; }
                    if (wait_slot(smem_u32(&empty_bar[bs]), ph ^ 1u, abort_flag, p.ctrl)) {
                        const uint32_t fb = smem_u32(&full_bar[bs]);
                        // (a copy of another lane may complete before this announcement: the barrier's
                        // pending arrival keeps the phase open until the announcement is made)
                        if (r == 0) mbar_arrive_expect_tx(fb, (uint32_t)nreal * (uint32_t)p.row_bytes);
                        if (src)
                            bulk_g2s(smem_u32(ring + (size_t)bs * bslot_bytes + (size_t)r * p.slot_bytes), src,
                                     (uint32_t)p.row_bytes, fb);
                    }
                }
                __syncwarp();
                bs0 += cnt;
                if (bs0 >= NB) { bs0 -= NB; phase0 ^= 1u; }
                issued += cnt;
            }
        }
        // Do not leave while a copy into this CTA's shared memory is in flight: wait (bounded)
        // for the last fill of every batch slot.  (After an abort a counted batch may not have
        // been issued; its wait then runs into the bound, which only delays the return.)
        for (int bs = lane; bs < NB; bs += 32) {
            const long long uses = issued / NB + (bs < (int)(issued % NB) ? 1 : 0);
            if (uses == 0) continue;
            const uint32_t fb = smem_u32(&full_bar[bs]);
            const uint32_t ph = (uint32_t)((uses - 1) & 1);
            const long long t0 = clock64();
            while (!mbar_try_wait(fb, ph))
                if (clock64() - t0 > kWaitCycles) { atomicMax(p.ctrl, (unsigned)kStatusTimeout); break; }
        }
        return;
    }

    // ======================================================== exchange warp ==
    // One lane runs every layer's exchange, so that all consumer warps are free to pull the
    // first batches of the next layer into their registers meanwhile: it waits (CTA barrier 2)
    // until the consumers have assembled the CTA's partial y in shared memory, sends it as one
    // bulk reduction and waits for that, arrives at the grid barrier (a release: the consumers'
    // earlier plain writes to global memory, such as the cleared target of a later layer, are
    // known to this thread through the CTA barrier), waits for everybody else's arrival, and
    // issues the copy that brings the sum back into the same buffer; the consumers sleep on that
    // copy's barrier.
    if (tid >= NC + 32) {
        const int lane = tid - NC - 32;
        unsigned long long* const stamps = lane == 0 ? p.stamps : nullptr;
        for (int l = 0; l < p.L; ++l) {
            named_bar_sync(2, NC + 32);
            if (lane == 0) {
                const size_t sb = ((size_t)cta * p.L + l) * kStampSlots;
                (void)sb;
                float* ytarget = p.ybuf + (size_t)(l % kYBuffers) * p.d;
                CI_STAMP(stamps, sb, 4);
                if (!*abort_flag) {
                    bulk_reduce_add_f32(ytarget, smem_u32(ysum), (uint32_t)p.d * (uint32_t)sizeof(float));
                    bulk_wait_all();
                    CI_STAMP(stamps, sb, 5);
                    red_release_add(&p.ctrl[1], 1u);
                    *arrived = l + 1;         // the fence is behind us: the producer may go on, paced
                    CI_STAMP(stamps, sb, 6);
                    grid_wait(p.ctrl, (unsigned)(l + 1) * (unsigned)G, abort_flag);
                    CI_STAMP(stamps, sb, 7);
                }
                if (!*abort_flag) {
                    const uint32_t yb = smem_u32(y_bar);
                    mbar_arrive_expect_tx(yb, (uint32_t)p.d * (uint32_t)sizeof(float));
                    bulk_g2s(smem_u32(ysum), ytarget, (uint32_t)p.d * (uint32_t)sizeof(float), yb);
                    *layers_done = l + 1;     // the exchange's last request is on its way: the producer may go on freely
                }
            }
            __syncwarp();
        }
        return;
    }

    // ============================================================ consumers ==
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const int nv = p.nv;
    const int d = p.d;

    // this thread's columns: 16-byte vectors tid, tid + NC, ...  vofs[] is clamped so that loads
    // never need a branch (threads beyond the row read vector 0 against a zero x).
    uint4 xq[VPT];                // x in the weight type, as loaded
    int vofs[VPT];
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = tid + i * NC;
        vofs[i] = (v < nv ? v : 0) * 16;
        uint4 q = make_uint4(0, 0, 0, 0);
        if (v < nv) q = reinterpret_cast<const uint4*>(p.x0)[v];
        xq[i] = q;
        if (p.x_layers && cta == 0 && v < nv) reinterpret_cast<uint4*>(p.x_layers)[v] = q;
    }

    int bslot = 0;                // batch slot of the next batch of the stream
    uint32_t phase = 0;
    const uint32_t ring_u32 = smem_u32(ring);
    // wait for the next batch, request its rows from shared memory (q[j][i] = vector i of row j),
    // free the slot.  The loads of one warp are performed in order with its arrival that follows.
    auto fetch = [&](uint4 (&q)[BATCH][VPT]) {
        const uint32_t fb = smem_u32(&full_bar[bslot]);
        if (!mbar_try_wait(fb, phase)) wait_slot(fb, phase, abort_flag, p.ctrl);
        const uint32_t base = ring_u32 + (uint32_t)bslot * bslot_bytes;
#pragma unroll
        for (int j = 0; j < BATCH; ++j)
#pragma unroll
            for (int i = 0; i < VPT; ++i)
                asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                             : "=r"(q[j][i].x), "=r"(q[j][i].y), "=r"(q[j][i].z), "=r"(q[j][i].w)
                             : "r"(base + (uint32_t)j * (uint32_t)p.slot_bytes + (uint32_t)vofs[i]));
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&empty_bar[bslot]));
        if (++bslot == NB) { bslot = 0; phase ^= 1u; }
    };

    unsigned long long* const stamps = tid == 0 ? p.stamps : nullptr;
    // The two register buffers live across layers: while the exchange of layer l is on, the
    // first two batches of layer l + 1 are pulled into them (their slots are free for the
    // producer at once), so a layer starts with up to two batches in registers besides the ring.
    uint4 qa[BATCH][VPT], qb[BATCH][VPT];
    auto batches_of = [&](int l) {
        int k0, k1;
        slab_of(cta, G, l, p.layers[l].K, &k0, &k1);
        const int n = k1 - k0;
        return (n * NMAT + BATCH - 1) / BATCH + (n + BATCH - 1) / BATCH;
    };
    {
        const int nb0 = batches_of(0);
        if (nb0 > 0) fetch(qa);
        if (nb0 > 1) fetch(qb);
    }
    for (int l = 0; l < p.L; ++l) {
        const LayerDev& ly = p.layers[l];
        int k0, k1;
        slab_of(cta, G, l, ly.K, &k0, &k1);
        const int nrows = k1 - k0;
        const int n_up = nrows * NMAT;
        const int nbu = (n_up + BATCH - 1) / BATCH;
        const int nbt = nbu + (nrows + BATCH - 1) / BATCH;
        const size_t sb = ((size_t)cta * p.L + l) * kStampSlots;
        (void)sb;
        CI_STAMP(stamps, sb, 0);

        float2 yacc[VPT][PAIRS];
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int v = tid + i * NC;
#pragma unroll
            for (int c = 0; c < PAIRS; ++c) yacc[i][c] = make_float2(0.f, 0.f);
            if (cta == 0 && ly.bdown && v < nv) {   // the bias enters the sum exactly once
#pragma unroll
                for (int c = 0; c < PAIRS; ++c)
                    yacc[i][c] = make_float2(E::load1(ly.bdown, v * EPV + 2 * c),
                                             E::load1(ly.bdown, v * EPV + 2 * c + 1));
            }
        }
        float part[WIN];          // row sums of the current pair of batches (this thread's columns)
#pragma unroll
        for (int j = 0; j < WIN; ++j) part[j] = 0.f;

        // One batch: its arithmetic, from the register buffer `q`.  `half` says which of the two
        // buffers it is, i.e. which half of part[] an up batch fills.
        auto process = [&](uint4 (&q)[BATCH][VPT], int b, const int H) {
            if (b < nbu) {
                // ------------------------------------------------ up (+ gate) rows --
#pragma unroll
                for (int j = 0; j < BATCH; ++j) {
                    float a0 = 0.f, a1 = 0.f;
#pragma unroll
                    for (int i = 0; i < VPT; ++i) E::dot(q[j][i], xq[i], a0, a1);
                    part[H * BATCH + j] = a0 + a1;
                }
                if (H == 1 || b == nbu - 1) {
                    // the pair of batches is complete (or the phase ends on its first half, whose
                    // second half then holds stale sums of rows that do not exist: not stored)
                    const float tot = warp_reduce_n(part, lane);
                    const int vi = WIN == 8 ? ((lane >> 4) & 1) * 4 + ((lane >> 3) & 1) * 2 + ((lane >> 2) & 1)
                                            : ((lane >> 4) & 1) * 2 + ((lane >> 3) & 1);
                    const int item = (b - H) * BATCH + vi;           // position in the up phase
                    if ((lane & (32 / WIN - 1)) == 0 && item < n_up)
                        red[((item % NMAT) * nwarps + warp) * p.rmax + item / NMAT] = tot;
                }
                if (b == nbu - 1) {
                    CI_STAMP(stamps, sb, 1);
                    named_bar_sync(1, NC);
                    for (int r = tid; r < nrows; r += NC) {
                        float u = 0.f;
                        for (int w = 0; w < nwarps; ++w) u += red[w * p.rmax + r];
                        float h;
                        if (GATED) {
                            float g = 0.f;
                            for (int w = 0; w < nwarps; ++w) g += red[(nwarps + w) * p.rmax + r];
                            h = gate_activation(g, p.silu) * u;
                        } else {
                            if (ly.bup) u += E::load1(ly.bup, k0 + r);
                            h = fmaxf(u, 0.f);
                        }
                        h_s[r] = h;
                    }
                    named_bar_sync(1, NC);
                    CI_STAMP(stamps, sb, 2);
                }
            } else {
                // ------------------------------------------------------- down rows --
                const int r0 = (b - nbu) * BATCH;
#pragma unroll
                for (int j = 0; j < BATCH; ++j) {
                    const float hk = (r0 + j < nrows) ? h_s[r0 + j] : 0.f;
                    if (hk != 0.f) {                              // uniform: ReLU zeros cost no arithmetic
                        const float2 hh = make_float2(hk, hk);
#pragma unroll
                        for (int i = 0; i < VPT; ++i) {
                            float2 w[PAIRS];
                            E::unpack(q[j][i], w);
#pragma unroll
                            for (int c = 0; c < PAIRS; ++c) yacc[i][c] = __ffma2_rn(w[c], hh, yacc[i][c]);
                        }
                    }
                }
            }
        };

        {
            // on entry qa holds batch 0 and qb batch 1 of this layer (where they exist)
            for (int b = 0; b < nbt; b += 2) {
                process(qa, b, 0);
                if (b + 2 < nbt) fetch(qa);
                if (b + 1 < nbt) process(qb, b + 1, 1);
                if (b + 3 < nbt) fetch(qb);
            }
            if (nbt == 0) {                          // a CTA without neurons still meets the others at the barriers
                named_bar_sync(1, NC);
                named_bar_sync(1, NC);
            }
        }
        CI_STAMP(stamps, sb, 3);

        // ----------------------------------------- cross-CTA sum of partial y --
        // Every CTA adds its partial into the layer's target; after the grid barrier every CTA
        // reads the sum back.  Targets rotate over three buffers: while layer l's is read, the
        // one layer l+2 will use is cleared (last read before the barrier of l).
        const bool last = (l == p.L - 1);
        // One sum per CTA leaves the chip, as one bulk reduction from shared memory (L2 then
        // sees 128-byte line reductions instead of a thousand 16-byte atomics per CTA).
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int v = tid + i * NC;
            if (v < nv) {
#pragma unroll
                for (int c = 0; c < PAIRS; c += 2)
                    *reinterpret_cast<float4*>(ysum + (size_t)v * EPV + 2 * c) =
                        make_float4(yacc[i][c].x, yacc[i][c].y, yacc[i][c + 1].x, yacc[i][c + 1].y);
            }
        }
        fence_proxy_async();          // these generic-proxy writes are read by the copy engine next
        named_bar_arrive(2, NC + 32);  // hands the partial to the exchange warp; nobody waits here
        // while the exchange runs: the first two batches of the next layer into the registers
        if (!last) {
            const int nbn = batches_of(l + 1);
            if (nbn > 0) fetch(qa);
            if (nbn > 1) fetch(qb);
        }
        wait_slot(smem_u32(y_bar), (uint32_t)(l & 1), abort_flag, p.ctrl);
        CI_STAMP(stamps, sb, 8);

        // ------------------------- next input: (x + y) / rms(x + y), rounded --
        float ssp[4] = {0.f, 0.f, 0.f, 0.f};   // four chains of the sum of squares
        float2 xn[VPT][PAIRS];        // x + y in fp32, until the norm is known
        const bool writer = (cta == l % G);   // the CTA that stores this layer's y
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int v = tid + i * NC;
            E::unpack(xq[i], xn[i]);
            if (v < nv) {
#pragma unroll
                for (int c = 0; c < PAIRS; c += 2) {
                    const float4 t = *reinterpret_cast<const float4*>(ysum + (size_t)v * EPV + 2 * c);
                    if (writer) {
                        if (p.y_layers) *reinterpret_cast<float4*>(p.y_layers + (size_t)l * d + (size_t)v * EPV + 2 * c) = t;
                        if (last) *reinterpret_cast<float4*>(p.y_last + (size_t)v * EPV + 2 * c) = t;
                    }
                    xn[i][c].x += t.x;
                    xn[i][c].y += t.y;
                    xn[i][c + 1].x += t.z;
                    xn[i][c + 1].y += t.w;
                }
#pragma unroll
                for (int c = 0; c < PAIRS; ++c) {
                    ssp[(2 * c) & 3] = fmaf(xn[i][c].x, xn[i][c].x, ssp[(2 * c) & 3]);
                    ssp[(2 * c + 1) & 3] = fmaf(xn[i][c].y, xn[i][c].y, ssp[(2 * c + 1) & 3]);
                }
            }
        }
        float ss = (ssp[0] + ssp[1]) + (ssp[2] + ssp[3]);
        {   // clear the target that layer l + 2 will use
            float4* z = reinterpret_cast<float4*>(p.ybuf + (size_t)((l + 2) % kYBuffers) * d);
            const int n4 = d / 4;
            for (int i = cta * NC + tid; i < n4; i += G * NC) z[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        if (last) { CI_STAMP(stamps, sb, 9); break; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        if (lane == 0) ss_red[warp] = ss;
        named_bar_sync(1, NC);
        float tot = 0.f;
        {   // the warps' sums (entries beyond the last warp are zero): four 16-byte loads, same order in every thread
            const float4* s4 = reinterpret_cast<const float4*>(ss_red);
#pragma unroll
            for (int w = 0; w < kMaxWarps / 4; ++w) {
                const float4 t = s4[w];
                tot += (t.x + t.y) + (t.z + t.w);
            }
        }
        const float inv = rsqrtf(tot * p.inv_d);     // within 2 ulp of 1 / sqrt(mean square)
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int v = tid + i * NC;
#pragma unroll
            for (int c = 0; c < PAIRS; ++c) {
                xn[i][c].x *= inv;
                xn[i][c].y *= inv;
            }
            xq[i] = v < nv ? E::pack(xn[i]) : make_uint4(0, 0, 0, 0);       // rounds to the layer-input type
            if (p.x_layers && cta == (l + 1) % G && v < nv)
                reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(p.x_layers) +
                                         (size_t)(l + 1) * p.row_bytes)[v] = xq[i];
        }
        CI_STAMP(stamps, sb, 9);
    }
}

// ------------------------------------------------------------------- host ---
static size_t fixed_smem_bytes(int rmax, bool gated, int nwarps)
{
    size_t b = (2 * kMaxBatchSlots + 2) * sizeof(uint64_t);
    b += (size_t)(gated ? 2 : 1) * nwarps * rmax * sizeof(float);      // red
    b += (size_t)rmax * sizeof(float);                                 // h_s
    b += (size_t)kMaxWarps * sizeof(float) + 16;                       // ss_red, flags
    return (b + 127) & ~(size_t)127;
}

template <typename T, int VPT, bool GATED>
static coreinfer_status launch_one(const DecodeParams& p, int grid, size_t smem, cudaStream_t st)
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
    cfg.blockDim = dim3((unsigned)(p.nc + 64));    // consumers, producer warp, exchange warp
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

// Debugging aid: COREINFER_RING_SLOTS=n in the environment (read once) caps the ring of the
// batch-1 stack kernel at n rows, so that tests can make the ring wrap every few rows.
static int ring_slots_cap()
{
    static const int cap = [] {
        const char* e = getenv("COREINFER_RING_SLOTS");
        return e ? atoi(e) : 0;
    }();
    return cap;
}

template <typename T, bool GATED>
static coreinfer_status launch_shape(int vpt, const DecodeParams& p, int grid, size_t smem, cudaStream_t st)
{
    if (vpt <= 1) return launch_one<T, 1, GATED>(p, grid, smem, st);
    if (vpt == 2) return launch_one<T, 2, GATED>(p, grid, smem, st);
    return launch_one<T, 3, GATED>(p, grid, smem, st);
}

static coreinfer_status check_common(const void* x, int batch, coreinfer_dtype dtype,
                                     coreinfer_ffn_kind kind, int d_model)
{
    if (!dtype_known(dtype)) CI_FAIL(COREINFER_ERR_UNSUPPORTED, "dtype %d is not supported", (int)dtype);
    if (!kind_known(kind)) CI_FAIL(COREINFER_ERR_UNSUPPORTED, "ffn kind %d is not supported", (int)kind);
    if (batch < 1 || batch > COREINFER_MAX_BATCH)
        CI_FAIL(COREINFER_ERR_UNSUPPORTED, "batch %d outside 1..%d", batch, COREINFER_MAX_BATCH);
    if (d_model < 1 || ((size_t)d_model * dtype_size(dtype)) % 16 != 0)
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "d_model %d: a row must be a positive multiple of 16 bytes", d_model);
    if (!x || !aligned16(x)) CI_FAIL(COREINFER_ERR_INVALID_ARG, "x is NULL or not 16-byte aligned");
    return COREINFER_OK;
}

static coreinfer_status check_layer(const coreinfer_layer& ly, int l, coreinfer_ffn_kind kind)
{
    const bool gated = kind_gated(kind);
    if (ly.K < 1) CI_FAIL(COREINFER_ERR_INVALID_ARG, "layer %d: K = %d < 1", l, ly.K);
    if (!ly.w_up_c || !ly.w_downT_c || !aligned16(ly.w_up_c) || !aligned16(ly.w_downT_c))
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "layer %d: w_up_c / w_downT_c NULL or not 16-byte aligned", l);
    if (gated && (!ly.w_gate_c || !aligned16(ly.w_gate_c)))
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "layer %d: gated FFN needs a 16-byte aligned w_gate_c", l);
    if (!gated && ly.w_gate_c) CI_FAIL(COREINFER_ERR_INVALID_ARG, "layer %d: w_gate_c given for a non-gated FFN", l);
    if (gated && ly.b_up_c) CI_FAIL(COREINFER_ERR_INVALID_ARG, "layer %d: the gated FFN has no up bias", l);
    return COREINFER_OK;
}


static size_t b1_workspace_bytes(int d_model)
{
    return kCtrlBytes + (size_t)kYBuffers * (size_t)d_model * sizeof(float);
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
    const bool gated = kind_gated(kind);
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
    p.rmax = ((Kmax + G - 1) / G + 1 + 3) & ~3;     // a multiple of 4 keeps the arrays behind it 16-byte aligned
    if ((unsigned long long)Kmax * (unsigned long long)G >= (1ull << 32))
        CI_FAIL(COREINFER_ERR_UNSUPPORTED, "K = %d is too large for the slab split (K * SM count must stay below 2^32)", Kmax);
    p.inv_d = 1.0f / (float)d_model;
    p.silu = kind == COREINFER_FFN_SILU_GATED;
    // Consumer threads: every thread owns `vpt` 16-byte vectors of a row; as many warps as the
    // row needs, 16 at most.
    const int vpt = (p.nv + kMaxConsumers - 1) / kMaxConsumers;
    if (vpt > kMaxVpt)
        CI_FAIL(COREINFER_ERR_UNSUPPORTED, "d_model %d is too wide for this kernel (max %d bytes per row)",
                d_model, kMaxVpt * max_consumers(kMaxVpt) * 16);
    p.nc = (((p.nv + vpt - 1) / vpt) + 31) & ~31;
    if (p.nc > max_consumers(vpt))
        CI_FAIL(COREINFER_ERR_UNSUPPORTED, "d_model %d is too wide for this kernel (max %d bytes per row)",
                d_model, kMaxVpt * max_consumers(kMaxVpt) * 16);
    const int batch = batch_for(vpt);
    const size_t bslot_bytes = (size_t)batch * p.slot_bytes;
    const size_t fixed0 = fixed_smem_bytes(p.rmax, gated, p.nc / 32);
    const size_t fixed = fixed0 + (((size_t)d_model * sizeof(float) + 127) & ~(size_t)127);    // + the partial y / the sum
    long long bslots = ((long long)di.smem_optin - (long long)fixed) / (long long)bslot_bytes;
    if (bslots > kMaxBatchSlots) bslots = kMaxBatchSlots;
    if (ring_slots_cap() > 0 && bslots > ring_slots_cap() / batch) bslots = ring_slots_cap() / batch;
    if (bslots < 2)
        CI_FAIL(COREINFER_ERR_UNSUPPORTED, "K = %d, d_model = %d do not fit in shared memory", Kmax, d_model);
    p.n_bslots = (int)bslots;
    const size_t smem = fixed + (size_t)p.n_bslots * bslot_bytes;
    // While an exchange is on, the next layer's rows are requested in two parts (measured on the
    // four model shapes): about 100 KB ahead of the exchange (40 KB for rows wider than 12 KB) --
    // more would still be in flight when the CTA's fence runs, and a fence waits for the SM's own
    // copies in flight -- and the rest of the ring after the CTA's arrival, one batch per 1000
    // cycles and 32 KB, which is a little above the pace at which HBM serves one SM.
    const int rows_ahead = (p.slot_bytes <= 12 * 1024 ? 100 : 40) * 1024 / p.slot_bytes;
    p.runahead = rows_ahead / batch < 1 ? 1 : rows_ahead / batch;
    if (p.runahead > p.n_bslots) p.runahead = p.n_bslots;
    p.trickle = p.n_bslots - p.runahead + 2;     // + the two slots the consumers empty into their registers meanwhile
    p.trickle_gap = (int)(1000ll * (long long)bslot_bytes / 32768);
    p.ysum_ofs = (int)((size_t)p.n_bslots * bslot_bytes + fixed0);
    p.x0 = x0;
    p.y_last = y_last;
    p.y_layers = y_layers;
    p.x_layers = x_layers;
    p.ctrl = (unsigned*)workspace;
    p.ybuf = (float*)((uint8_t*)workspace + kCtrlBytes);
    p.stamps = stamps_buffer((size_t)G * L * kStampSlots * sizeof(unsigned long long));

    // Control words and the reduction targets start at zero.
    CI_CUDA(cudaMemsetAsync(workspace, 0, b1_workspace_bytes(d_model), st));
    if (dtype == COREINFER_BF16)
        return gated ? launch_shape<__nv_bfloat16, true>(vpt, p, G, smem, st)
                     : launch_shape<__nv_bfloat16, false>(vpt, p, G, smem, st);
    if (dtype == COREINFER_F16)
        return gated ? launch_shape<__half, true>(vpt, p, G, smem, st)
                     : launch_shape<__half, false>(vpt, p, G, smem, st);
    return gated ? launch_shape<float, true>(vpt, p, G, smem, st)
                 : launch_shape<float, false>(vpt, p, G, smem, st);
}

// decode_batch.cu
coreinfer_status decode_batched(const void* x, int batch, coreinfer_dtype dtype, coreinfer_ffn_kind kind,
                                int d_model, const coreinfer_layer& ly, float* y, void* workspace,
                                cudaStream_t st, bool clear_status);
size_t decode_stack_batched_workspace_bytes(int batch, int d_model, int K_max);
coreinfer_status decode_stack_batched(const coreinfer_layer* layers, int L, const void* x0, int batch,
                                      coreinfer_dtype dtype, coreinfer_ffn_kind kind, int d_model, float* y_last,
                                      float* y_layers, void* x_layers, void* workspace, size_t workspace_bytes,
                                      cudaStream_t st);

}  // namespace coreinfer

using namespace coreinfer;

extern "C" {

size_t coreinfer_ffn_decode_workspace_bytes(int32_t batch, int32_t d_model, int32_t K)
{
    if (batch < 1 || d_model < 1 || K < 1) return 0;
    if (batch == 1) return b1_workspace_bytes(d_model);
    return kCtrlBytes + (size_t)batch * (size_t)K * sizeof(float);   // h [batch, K]
}

size_t coreinfer_ffn_decode_stack_workspace_bytes(int32_t L, int32_t batch, int32_t d_model, int32_t K_max)
{
    if (L < 1 || batch < 1 || d_model < 1) return 0;
    if (batch == 1) return b1_workspace_bytes(d_model);
    if (K_max < 1) return 0;
    return decode_stack_batched_workspace_bytes(batch, d_model, K_max);
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
    return decode_batched(x, batch, dtype, kind, d_model, ly, y, workspace, st, true);
}

coreinfer_status coreinfer_ffn_decode_stack(const coreinfer_layer* layers, int32_t L, const void* x0,
                                            int32_t batch, coreinfer_dtype dtype,
                                            coreinfer_ffn_kind kind, int32_t d_model, float* y_last,
                                            float* y_layers, void* x_layers, void* workspace,
                                            size_t workspace_bytes, void* cuda_stream)
{
    coreinfer_status s = check_common(x0, batch, dtype, kind, d_model);
    if (s != COREINFER_OK) return s;
    if (!layers) CI_FAIL(COREINFER_ERR_INVALID_ARG, "layers is NULL");
    if (L < 1 || L > COREINFER_MAX_LAYERS)
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "L = %d outside 1..%d", L, COREINFER_MAX_LAYERS);
    if (!y_last || !aligned16(y_last)) CI_FAIL(COREINFER_ERR_INVALID_ARG, "y_last is NULL or not 16-byte aligned");
    if ((y_layers && !aligned16(y_layers)) || (x_layers && !aligned16(x_layers)))
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "y_layers / x_layers not 16-byte aligned");
    if (batch > 1) {
        // 2..8 sequences sharing the core sets: one batched FFN launch and one glue launch per layer
        for (int l = 0; l < L; ++l) {
            s = check_layer(layers[l], l, kind);
            if (s != COREINFER_OK) return s;
        }
        return decode_stack_batched(layers, L, x0, batch, dtype, kind, d_model, y_last, y_layers, x_layers, workspace,
                                    workspace_bytes, (cudaStream_t)cuda_stream);
    }
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
// scratch of the stack kernel (control words + the rotating reduction targets) lives in a
// fixed array inside the library image.  The array costs kNoAllocScratchBytes of HBM on every
// GPU that loads the library, for the life of the process.
constexpr size_t kNoAllocScratchBytes = 128u << 10;   // 128 KiB: 256 + 12 * d_model bytes must fit
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
    if (!layers) CI_FAIL(COREINFER_ERR_INVALID_ARG, "layers is NULL");
    if (L < 1 || L > COREINFER_MAX_LAYERS)
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "L = %d outside 1..%d", L, COREINFER_MAX_LAYERS);
    if (!y_last || !aligned16(y_last)) CI_FAIL(COREINFER_ERR_INVALID_ARG, "y_last is NULL or not 16-byte aligned");
    if ((y_layers && !aligned16(y_layers)) || (x_layers && !aligned16(x_layers)))
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "y_layers / x_layers not 16-byte aligned");
    if (batch != 1) CI_FAIL(COREINFER_ERR_UNSUPPORTED, "this entry point is built for batch 1 (got %d)", batch);
    const size_t need = coreinfer_ffn_decode_stack_workspace_bytes(L, batch, d_model, 0);
    if (need > kNoAllocScratchBytes)
        CI_FAIL(COREINFER_ERR_UNSUPPORTED,
                "d_model = %d needs %zu bytes of scratch; the built-in scratch holds %zu "
                "(use coreinfer_ffn_decode_stack with a workspace)", d_model, need, kNoAllocScratchBytes);
    void* scratch = nullptr;
    s = noalloc_scratch_ptr(&scratch);
    if (s != COREINFER_OK) return s;
    // decode_stack_b1 zeroes the control words and the reduction targets it uses on the stream
    // before the launch, so whatever the previous call left in the array does not matter.
    return decode_stack_b1(layers, L, x0, dtype, kind, d_model, y_last, y_layers, x_layers, scratch,
                           kNoAllocScratchBytes, need, (cudaStream_t)cuda_stream);
}

}  // extern "C"
