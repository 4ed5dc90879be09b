// Decode-stage FFN over compacted core-neuron weights (Section 4.2), batch 1.
//
// One persistent kernel, one CTA per SM.  Per layer a CTA owns a contiguous slab of the K core
// neurons and streams that slab's rows exactly once: first the up (and gate) rows to form h for
// its neurons, then the matching rows of the transposed down matrix to form its partial y.
// Rows arrive through a ring of shared-memory slots filled by 1-D bulk copies (a producer warp,
// one full/empty mbarrier pair per slot).  The weights of a layer do not depend on its input,
// so the producer runs ahead across layer boundaries and HBM stays busy while the CTAs exchange
// partial outputs.
//
// Consumers own columns: thread t of a group holds the x values of its 16-byte vectors
// t, t + 256, ... in registers for the whole layer and its partial y likewise.  They take ring
// items in batches: wait for the batch, pull every vector of all its rows into registers with
// no branch in between (so the loads overlap), free the slots at once, and only then do the
// arithmetic; slots are held for a few hundred cycles whatever the arithmetic costs.  For rows
// of at most 8 KB two such groups take alternate batches, so that one group's shared-memory
// reads overlap the other's arithmetic; wider rows use one group.
//
// Exchange per layer: the CTA's partial y (d_model fp32) is assembled in shared memory and added
// into a global vector with one bulk reduction; one thread waits for it, arrives at a grid
// barrier (release), polls for everybody else's arrival (acquire) and brings the sum back with
// one bulk copy, on whose barrier the other consumers sleep; every group then forms the next
// layer's input redundantly in registers.  Every wait (slot barriers, grid barrier, read-back)
// is bounded: when one gives up, the CTA marks the workspace status word, stops waiting
// everywhere, runs the rest of its schedule without synchronising on data, drains its own
// copies in flight and returns.
#include "common.cuh"

#include <stdlib.h>

namespace coreinfer {

constexpr int kMaxSlots = 64;
constexpr int kGroupThreads = 256;                     // consumer threads per group
constexpr int kGroupWarps = kGroupThreads / 32;
constexpr int kCtrlBytes = 256;                        // status word, barrier counter, padding
constexpr int kYCopies = 1;                            // copies of a reduction target (more spread same-address adds, but cost more to read back)
constexpr int kYBuffers = 3;                           // rotating targets: in use, being read, being cleared
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
    int runahead;       // ring items of the next layer the producer may request before this layer's exchange is over
    float inv_d;        // 1 / d_model
    int ysum_ofs;       // shared-memory offset of the buffer holding the CTA's partial y
    const void* x0;
    float* y_last;
    float* y_layers;
    void* x_layers;
    float* ybuf;        // [kYBuffers][kYCopies][d]: reduction targets, buffer l % 3 serves layer l
    unsigned* ctrl;     // [0] status word, [1] grid-barrier arrival counter
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

// items per consumer batch for one group (register budget: 4 * items * vectors per thread)
__host__ __device__ constexpr int batch_for(int groups, int vpt)
{
    return groups == 2 ? 4 : (vpt <= 2 ? 8 : (vpt <= 4 ? 4 : 2));
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

// One thread per CTA calls this, after it has seen the CTA's work complete.  The arrival
// counter is zeroed by the host before the launch; barrier number b (0-based) completes when it
// reaches (b + 1) * G.  The arrival is a release at GPU scope (what this thread has observed,
// the completed bulk reduction and the CTA's earlier plain writes included, becomes visible
// before it), the poll an acquire.
__device__ __forceinline__ void grid_arrive_and_wait(unsigned* ctrl, unsigned target, volatile int* abort_flag)
{
    red_release_add(&ctrl[1], 1u);
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

// ------------------------------------------------------------------- kernel --
// Ring stream order of one CTA and one layer (producer and consumers walk it in lock step): for
// each slab row k0 .. k1-1 its up row, then (gated) its gate row; after those, the down rows
// k0 .. k1-1.  Within each of the two phases the items are cut into batches of BATCH.  With two
// consumer groups every batch takes BATCH ring slots, the last batch of a phase being filled up
// with empty items (no copy: the producer completes their barrier by a plain arrival), and the
// batches of the whole launch are dealt out in turn: batch number g of the launch belongs to
// group g % NG and starts at ring position (g * BATCH) % slots.  The ring holds a multiple of
// NG * BATCH slots, so a slot is read by the same group in every pass of the ring: a group that
// tests a slot's barrier has itself consumed the slot's previous fill, and can therefore never
// mistake the parity of a fill that is still in flight for that of the one it wants.
template <typename T, int NG, int VPT, bool GATED>
__global__ void __launch_bounds__(NG * kGroupThreads + 32, 1)
decode_stack_kernel(const __grid_constant__ DecodeParams p)
{
    using E = Elem<T>;
    constexpr int PAIRS = E::kPairs;
    constexpr int EPV = PAIRS * 2;                   // elements per 16-byte vector
    constexpr int NMAT = GATED ? 2 : 1;
    constexpr int NC = NG * kGroupThreads;           // consumer threads
    constexpr int BATCH = batch_for(NG, VPT);        // ring items per batch
    constexpr int PADB = NG > 1 ? BATCH : 1;         // a phase takes a multiple of PADB ring slots
    constexpr int FLUSH = 16 / BATCH;                // own up batches per cross-lane reduction (16 row sums)

    extern __shared__ __align__(128) uint8_t smem[];
    uint8_t* ring = smem;
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(ring + (size_t)p.n_slots * p.slot_bytes);
    uint64_t* empty_bar = full_bar + kMaxSlots;
    uint64_t* y_bar = empty_bar + kMaxSlots;                        // completion of the read-back copy (+ 8 bytes padding)
    float* red = reinterpret_cast<float*>(y_bar + 2);               // [NMAT][kGroupWarps][rmax]
    float* h_s = red + NMAT * kGroupWarps * p.rmax;                 // [rmax]
    float* ss_red = h_s + p.rmax;                                   // [NG][kGroupWarps]
    volatile int* abort_flag = reinterpret_cast<volatile int*>(ss_red + NG * kGroupWarps);
    volatile int* layers_done = abort_flag + 1;                     // layers whose exchange this CTA has completed
    float* ysum = reinterpret_cast<float*>(smem + p.ysum_ofs);      // [VPT * 256 * EPV]: the CTA's partial y

    const int tid = threadIdx.x;
    const int G = gridDim.x;
    const int cta = blockIdx.x;
    const int NS = p.n_slots;

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(smem_u32(&full_bar[s]), 1);
            mbar_init(smem_u32(&empty_bar[s]), kGroupWarps);     // the warps of the group that reads the slot
        }
        mbar_init(smem_u32(y_bar), 1);
        *abort_flag = 0;
        *layers_done = 0;
        mbar_fence_init();
    }
    __syncthreads();

    // ======================================================== producer warp ==
    // Up to eight lanes issue copies: one round fills up to min(8, ring slots) consecutive ring
    // items, lane j taking item j of the round (its own slot, its own wait on that slot's
    // "empty" barrier), so the latency of one issue is not the issue rate.
    if (tid >= NC) {
        const int lane = tid - NC;
        const int round_max = NS < 8 ? NS : 8;
        int slot0 = 0;                // ring position of the round's first item
        uint32_t phase0 = 0;          // parity of the ring pass that position belongs to
        long long issued = 0;
        for (int l = 0; l < p.L; ++l) {
            const LayerDev& ly = p.layers[l];
            int k0, k1;
            slab_of(cta, G, l, ly.K, &k0, &k1);
            const int n = k1 - k0;
            const int n_up = n * NMAT;            // items of the up (+ gate) phase
            const int p_up = (n_up + PADB - 1) / PADB * PADB;          // ring slots of that phase
            const int total = p_up + (n + PADB - 1) / PADB * PADB;     // + those of the down rows
            for (int q0 = 0, cnt = 0; q0 < total; q0 += cnt) {
                if (*abort_flag) break;
                cnt = min(round_max, total - q0);
                // Every weight request in flight delays the few small messages of the previous
                // layer's exchange (adds, arrival, poll, read-back), which queue behind it.  So
                // only a limited number of this layer's rows is requested before that exchange is
                // over: a round is cut at the limit, and beyond it the producer waits.
                if (l > 0 && q0 + cnt > p.runahead && *layers_done < l) {
                    if (q0 < p.runahead) {
                        cnt = p.runahead - q0;
                    } else {
                        const long long t0 = clock64();
                        while (*layers_done < l && !*abort_flag) {
                            __nanosleep(64);
                            if (clock64() - t0 > kWaitCycles) { *abort_flag = 1; atomicMax(p.ctrl, (unsigned)kStatusTimeout); }
                        }
                    }
                }
                if (lane < cnt) {
                    const int q = q0 + lane;
                    const uint8_t* src = nullptr;         // stays NULL for an empty item
                    if (q < n_up) {
                        const int row = k0 + q / NMAT;
                        src = ((GATED && (q % NMAT)) ? ly.gate : ly.up) + (size_t)row * p.row_bytes;
                    } else if (q >= p_up && q - p_up < n) {
                        src = ly.down + (size_t)(k0 + q - p_up) * p.row_bytes;
                    }
                    int sl = slot0 + lane;
                    uint32_t ph = phase0;
                    if (sl >= NS) { sl -= NS; ph ^= 1u; }
                    if (wait_slot(smem_u32(&empty_bar[sl]), ph ^ 1u, abort_flag, p.ctrl)) {
                        const uint32_t fb = smem_u32(&full_bar[sl]);
                        if (src) {
                            mbar_arrive_expect_tx(fb, (uint32_t)p.row_bytes);
                            bulk_g2s(smem_u32(ring + (size_t)sl * p.slot_bytes), src, (uint32_t)p.row_bytes, fb);
                        } else {
                            mbar_arrive(fb);
                        }
                    }
                }
                __syncwarp();
                slot0 += cnt;
                if (slot0 >= NS) { slot0 -= NS; phase0 ^= 1u; }
                issued += cnt;
            }
        }
        // Do not leave while a copy into this CTA's shared memory is in flight: wait (bounded)
        // for the last copy issued into every slot.  (After an abort a counted item may not have
        // been issued; its wait then runs into the bound, which only delays the return.)
        for (int sl = lane; sl < NS; sl += 32) {
            const long long uses = issued / NS + (sl < (int)(issued % NS) ? 1 : 0);
            if (uses == 0) continue;
            const uint32_t fb = smem_u32(&full_bar[sl]);
            const uint32_t ph = (uint32_t)((uses - 1) & 1);
            const long long t0 = clock64();
            while (!mbar_try_wait(fb, ph))
                if (clock64() - t0 > kWaitCycles) { atomicMax(p.ctrl, (unsigned)kStatusTimeout); break; }
        }
        return;
    }

    // ============================================================ consumers ==
    const int grp = tid / kGroupThreads;          // consumer group of this thread
    const int gt = tid % kGroupThreads;           // thread within the group
    const int lane = tid & 31;
    const int gw = gt >> 5;                       // warp within the group
    const int nv = p.nv;
    const int d = p.d;

    // this thread's columns: 16-byte vectors gt, gt + 256, ...  vofs[] is clamped so that loads
    // never need a branch (threads beyond the row read vector 0 against a zero x).
    uint4 xq[VPT];                // x in the weight type, as loaded
    int vofs[VPT];
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = gt + i * kGroupThreads;
        vofs[i] = (v < nv ? v : 0) * 16;
        uint4 q = make_uint4(0, 0, 0, 0);
        if (v < nv) q = reinterpret_cast<const uint4*>(p.x0)[v];
        xq[i] = q;
        if (p.x_layers && cta == 0 && grp == 0 && v < nv) reinterpret_cast<uint4*>(p.x_layers)[v] = q;
    }

    int slot = 0;                 // ring position of the next item of the stream
    uint32_t phase = 0;
    int gbatch = 0;               // two groups: number, within the launch, of the current phase's first batch
    auto skip_n = [&](int n) {    // ring slots that belong to the other group
        slot += n;
        if (slot >= NS) { slot -= NS; phase ^= 1u; }
    };
    // wait for the next n items, pull them into registers (q[j][i] = vector i of item j), free them
    auto fetch = [&](uint4 (&q)[BATCH][VPT], int n) {
        const int held = NG > 1 ? BATCH : n;      // ring slots of this batch (two groups: empty items included)
        {
            // test all barriers of the batch back to back (the tests overlap); only if one is
            // not complete yet fall back to the bounded waits, one by one
            bool ready = true;
#pragma unroll
            for (int j = 0; j < BATCH; ++j) {
                int sl = slot + (j < held ? j : 0);
                uint32_t ph = phase;
                if (sl >= NS) { sl -= NS; ph ^= 1u; }
                ready &= mbar_try_wait(smem_u32(&full_bar[sl]), ph);
            }
            if (!ready) {
                int sl = slot;
                uint32_t ph = phase;
                for (int j = 0; j < held; ++j) {
                    wait_slot(smem_u32(&full_bar[sl]), ph, abort_flag, p.ctrl);
                    if (++sl == NS) { sl = 0; ph ^= 1u; }
                }
            }
        }
        if (n == BATCH) {
#pragma unroll
            for (int j = 0; j < BATCH; ++j) {
                int sl = slot + j;
                if (sl >= NS) sl -= NS;
                const uint8_t* row = ring + (size_t)sl * p.slot_bytes;
#pragma unroll
                for (int i = 0; i < VPT; ++i) q[j][i] = *reinterpret_cast<const uint4*>(row + vofs[i]);
            }
        } else {
#pragma unroll
            for (int j = 0; j < BATCH; ++j) {
                int sl = slot + (j < n ? j : 0);
                if (sl >= NS) sl -= NS;
                const uint8_t* row = ring + (size_t)sl * p.slot_bytes;
#pragma unroll
                for (int i = 0; i < VPT; ++i) {
                    q[j][i] = *reinterpret_cast<const uint4*>(row + vofs[i]);
                    if (j >= n) q[j][i] = make_uint4(0, 0, 0, 0);
                }
            }
        }
        __syncwarp();
        if (lane < held && !*abort_flag) {
            int sl = slot + lane;
            if (sl >= NS) sl -= NS;
            mbar_arrive(smem_u32(&empty_bar[sl]));
        }
        skip_n(held);
    };

    for (int l = 0; l < p.L; ++l) {
        const LayerDev& ly = p.layers[l];
        int k0, k1;
        slab_of(cta, G, l, ly.K, &k0, &k1);
        const int nrows = k1 - k0;
        const int n_up = nrows * NMAT;

        // ------------------------------------------------ up (+ gate) phase --
        {
            const int nb = (n_up + BATCH - 1) / BATCH;
            float part[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) part[j] = 0.f;
            int own = 0;                          // own batches accumulated in part[]
            int first_b = 0;                      // first of them
            for (int b = 0; b < nb; ++b) {
                const int cnt = min(BATCH, n_up - b * BATCH);
                if (NG > 1 && ((gbatch + b) % NG) != grp) { skip_n(BATCH); continue; }
                uint4 q[BATCH][VPT];
                fetch(q, cnt);
                if (own == 0) first_b = b;
#pragma unroll
                for (int f = 0; f < FLUSH; ++f) {
                    if (f == own) {               // uniform; keeps part[] statically indexed
#pragma unroll
                        for (int j = 0; j < BATCH; ++j) {
                            float a0 = 0.f, a1 = 0.f;
#pragma unroll
                            for (int i = 0; i < VPT; ++i) E::dot(q[j][i], xq[i], a0, a1);
                            part[f * BATCH + j] = a0 + a1;
                        }
                    }
                }
                ++own;
                if (own == FLUSH || b + NG >= nb) {
                    // two independent 8-value reductions (their shuffles interleave)
                    float lo[8], hi[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) { lo[j] = part[j]; hi[j] = part[8 + j]; }
                    const float tot_lo = warp_reduce8(lo, lane);
                    const float tot_hi = warp_reduce8(hi, lane);
                    if ((lane & 3) == 0) {
                        const int vi = ((lane >> 4) & 1) * 4 + ((lane >> 3) & 1) * 2 + ((lane >> 2) & 1);
#pragma unroll
                        for (int half = 0; half < 2; ++half) {
                            const int pi = half * 8 + vi;                      // index in part[]
                            const int f = pi / BATCH, j = pi % BATCH;          // own batch f of the window, item j
                            const int item = (first_b + f * NG) * BATCH + j;   // position in the up phase
                            if (f < own && item < n_up)
                                red[((item % NMAT) * kGroupWarps + gw) * p.rmax + item / NMAT] = half ? tot_hi : tot_lo;
                        }
                    }
#pragma unroll
                    for (int j = 0; j < 16; ++j) part[j] = 0.f;
                    own = 0;
                }
            }
            gbatch += nb;
        }
        named_bar_sync(1, NC);
        for (int r = tid; r < nrows; r += NC) {
            float u = 0.f;
#pragma unroll
            for (int w = 0; w < kGroupWarps; ++w) u += red[w * p.rmax + r];
            float h;
            if (GATED) {
                float g = 0.f;
#pragma unroll
                for (int w = 0; w < kGroupWarps; ++w) g += red[(kGroupWarps + w) * p.rmax + r];
                h = fmaxf(g, 0.f) * u;
            } else {
                if (ly.bup) u += E::load1(ly.bup, k0 + r);
                h = fmaxf(u, 0.f);
            }
            h_s[r] = h;
        }
        named_bar_sync(1, NC);

        // ------------------------------------------------------- down phase --
        float2 yacc[VPT][PAIRS];
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int v = gt + i * kGroupThreads;
#pragma unroll
            for (int c = 0; c < PAIRS; ++c) yacc[i][c] = make_float2(0.f, 0.f);
            if (cta == 0 && grp == 0 && ly.bdown && v < nv) {   // the bias enters the sum exactly once
#pragma unroll
                for (int c = 0; c < PAIRS; ++c)
                    yacc[i][c] = make_float2(E::load1(ly.bdown, v * EPV + 2 * c),
                                             E::load1(ly.bdown, v * EPV + 2 * c + 1));
            }
        }
        {
            const int nb = (nrows + BATCH - 1) / BATCH;
            for (int b = 0; b < nb; ++b) {
                const int cnt = min(BATCH, nrows - b * BATCH);
                if (NG > 1 && ((gbatch + b) % NG) != grp) { skip_n(BATCH); continue; }
                uint4 q[BATCH][VPT];
                fetch(q, cnt);
#pragma unroll
                for (int j = 0; j < BATCH; ++j) {
                    const float hk = (j < cnt) ? h_s[b * BATCH + j] : 0.f;
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
            gbatch += nb;
        }

        // ----------------------------------------- cross-CTA sum of partial y --
        // Every CTA adds its partial into the layer's target; after the grid barrier every CTA
        // reads the sum back.  Targets rotate over three buffers: while layer l's is read, the
        // one layer l+2 will use is cleared (last read before the barrier of l).
        const bool last = (l == p.L - 1);
        float* ybase = p.ybuf + (size_t)(l % kYBuffers) * kYCopies * d;
        float* ytarget = ybase + (size_t)(cta & (kYCopies - 1)) * d;
        // One sum per CTA leaves the chip, as one bulk reduction: group 1 hands its partial to
        // group 0 through shared memory, group 0 leaves the CTA's partial there, and the copy
        // engine adds the whole vector into the target (L2 then sees 128-byte line reductions
        // instead of a thousand 16-byte atomics per CTA, whose acknowledgements a fence had to
        // wait for).
        if (NG == 2) {
            if (grp == 1) {
#pragma unroll
                for (int i = 0; i < VPT; ++i)
#pragma unroll
                    for (int c = 0; c < PAIRS; c += 2)
                        *reinterpret_cast<float4*>(ysum + (size_t)(gt + i * kGroupThreads) * EPV + 2 * c) =
                            make_float4(yacc[i][c].x, yacc[i][c].y, yacc[i][c + 1].x, yacc[i][c + 1].y);
            }
            named_bar_sync(1, NC);
        }
        if (grp == 0) {
#pragma unroll
            for (int i = 0; i < VPT; ++i) {
#pragma unroll
                for (int c = 0; c < PAIRS; c += 2) {
                    float4* cell = reinterpret_cast<float4*>(ysum + (size_t)(gt + i * kGroupThreads) * EPV + 2 * c);
                    float4 t = make_float4(yacc[i][c].x, yacc[i][c].y, yacc[i][c + 1].x, yacc[i][c + 1].y);
                    if (NG == 2) {
                        const float4 o = *cell;
                        t.x += o.x; t.y += o.y; t.z += o.z; t.w += o.w;
                    }
                    *cell = t;
                }
            }
            fence_proxy_async();          // these generic-proxy writes are read by the copy engine next
        }
        named_bar_sync(1, NC);
        // One thread runs the exchange: the CTA's reduction and the wait for its completion, the
        // arrival at the grid barrier (a release: the CTA's earlier plain writes to global memory,
        // such as the cleared target of a later layer, are known to this thread through the CTA
        // barriers since), the wait for everybody else's arrival, and the copy that brings the
        // sum back; the other consumers sleep on that copy's barrier.  The sum comes back as one
        // bulk copy into the buffer the partial left from (256 requests of 128 bytes per CTA
        // instead of some thousand 16-byte loads).
        if (tid == 0) {
            if (!*abort_flag) {
                bulk_reduce_add_f32(ytarget, smem_u32(ysum), (uint32_t)d * (uint32_t)sizeof(float));
                bulk_wait_all();
                grid_arrive_and_wait(p.ctrl, (unsigned)(l + 1) * (unsigned)G, abort_flag);
            }
            if (!*abort_flag) {
                const uint32_t yb = smem_u32(y_bar);
                mbar_arrive_expect_tx(yb, (uint32_t)(kYCopies * d) * (uint32_t)sizeof(float));
                bulk_g2s(smem_u32(ysum), ybase, (uint32_t)(kYCopies * d) * (uint32_t)sizeof(float), yb);
                *layers_done = l + 1;     // the exchange's last request is on its way: the producer may go on
            }
        }
        wait_slot(smem_u32(y_bar), (uint32_t)(l & 1), abort_flag, p.ctrl);

        // ------------------------- next input: (x + y) / rms(x + y), rounded --
        float ssp[4] = {0.f, 0.f, 0.f, 0.f};   // four chains of the sum of squares
        float2 xn[VPT][PAIRS];        // x + y in fp32, until the norm is known
        const bool writer = (cta == l % G) && grp == 0;   // the CTA that stores this layer's y
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int v = gt + i * kGroupThreads;
            E::unpack(xq[i], xn[i]);
            if (v < nv) {
#pragma unroll
                for (int c = 0; c < PAIRS; c += 2) {
                    float4 t = *reinterpret_cast<const float4*>(ysum + (size_t)v * EPV + 2 * c);
#pragma unroll
                    for (int cp = 1; cp < kYCopies; ++cp) {
                        const float4 o = *reinterpret_cast<const float4*>(ysum + (size_t)cp * d + (size_t)v * EPV + 2 * c);
                        t.x += o.x; t.y += o.y; t.z += o.z; t.w += o.w;
                    }
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
            float4* z = reinterpret_cast<float4*>(p.ybuf + (size_t)((l + 2) % kYBuffers) * kYCopies * d);
            const int n4 = kYCopies * d / 4;
            for (int i = cta * NC + tid; i < n4; i += G * NC) z[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        if (last) break;
        // every group holds all columns, so each forms the norm on its own (same sums, same order)
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        if (lane == 0) ss_red[grp * kGroupWarps + gw] = ss;
        named_bar_sync(2 + grp, kGroupThreads);
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < kGroupWarps; ++w) tot += ss_red[grp * kGroupWarps + w];
        const float inv = rsqrtf(tot * p.inv_d);     // within 2 ulp of 1 / sqrt(mean square)
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int v = gt + i * kGroupThreads;
#pragma unroll
            for (int c = 0; c < PAIRS; ++c) {
                xn[i][c].x *= inv;
                xn[i][c].y *= inv;
            }
            xq[i] = E::pack(xn[i]);       // rounds to the layer-input type
            if (p.x_layers && cta == (l + 1) % G && grp == 0 && v < nv)
                reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(p.x_layers) +
                                         (size_t)(l + 1) * p.row_bytes)[v] = xq[i];
        }
    }
}

// ------------------------------------------------------------------- host ---
// fp32 buffer in which the CTA's partial y is assembled: every thread of a group stores all its columns
static size_t ysum_smem_bytes(int groups, int vpt, size_t esize)
{
    (void)groups;
    return (size_t)kYCopies * vpt * kGroupThreads * (16 / esize) * sizeof(float);   // room for the copies read back
}

static size_t fixed_smem_bytes(int rmax, bool gated, int groups)
{
    size_t b = (2 * kMaxSlots + 2) * sizeof(uint64_t);
    b += (size_t)(gated ? 2 : 1) * kGroupWarps * rmax * sizeof(float);
    b += (size_t)rmax * sizeof(float);
    b += (size_t)groups * kGroupWarps * sizeof(float) + 16;
    return (b + 127) & ~(size_t)127;
}

template <typename T, int NG, int VPT, bool GATED>
static coreinfer_status launch_one(const DecodeParams& p, int grid, size_t smem, cudaStream_t st)
{
    auto kern = decode_stack_kernel<T, NG, VPT, GATED>;
    static thread_local size_t configured[64] = {0};
    int dev = 0;
    CI_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64 || configured[dev] < smem) {
        CI_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        if (dev >= 0 && dev < 64) configured[dev] = smem;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)(NG * kGroupThreads + 32));
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
// batch-1 stack kernel at n slots, so that tests can make the ring wrap every few rows.
static int ring_slots_cap()
{
    static const int cap = [] {
        const char* e = getenv("COREINFER_RING_SLOTS");
        return e ? atoi(e) : 0;
    }();
    return cap;
}

static int groups_for(int nv) { return nv <= 2 * kGroupThreads ? 2 : 1; }
static int vpt_for(int nv)
{
    const int v = (nv + kGroupThreads - 1) / kGroupThreads;
    return v <= 1 ? 1 : v <= 2 ? 2 : v <= 3 ? 3 : v <= 5 ? 5 : 8;
}

template <typename T, bool GATED>
static coreinfer_status launch_shape(int groups, int vpt, const DecodeParams& p, int grid, size_t smem,
                                     cudaStream_t st)
{
    if (groups == 2) {
        if (vpt <= 1) return launch_one<T, 2, 1, GATED>(p, grid, smem, st);
        return launch_one<T, 2, 2, GATED>(p, grid, smem, st);
    }
    if (vpt <= 3) return launch_one<T, 1, 3, GATED>(p, grid, smem, st);
    if (vpt <= 5) return launch_one<T, 1, 5, GATED>(p, grid, smem, st);
    return launch_one<T, 1, 8, GATED>(p, grid, smem, st);
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

static size_t b1_workspace_bytes(int d_model)
{
    return kCtrlBytes + (size_t)kYBuffers * kYCopies * (size_t)d_model * sizeof(float);
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
    if ((unsigned long long)Kmax * (unsigned long long)G >= (1ull << 32))
        CI_FAIL(COREINFER_ERR_UNSUPPORTED, "K = %d is too large for the slab split (K * SM count must stay below 2^32)", Kmax);
    p.inv_d = 1.0f / (float)d_model;
    const int groups = groups_for(p.nv);
    if ((p.nv + kGroupThreads - 1) / kGroupThreads > 8)
        CI_FAIL(COREINFER_ERR_UNSUPPORTED, "d_model %d is too wide for this kernel (max %d bytes per row)",
                d_model, 8 * kGroupThreads * 16);
    const int vpt = groups == 2 ? ((p.nv + kGroupThreads - 1) / kGroupThreads <= 1 ? 1 : 2) : vpt_for(p.nv);
    const int batch = batch_for(groups, groups == 2 ? vpt : (vpt <= 3 ? 3 : vpt));
    const size_t fixed0 = fixed_smem_bytes(p.rmax, gated, groups);
    const size_t fixed = fixed0 + ysum_smem_bytes(groups, vpt, esize);
    if (fixed + (size_t)batch * p.slot_bytes > (size_t)di.smem_optin)
        CI_FAIL(COREINFER_ERR_UNSUPPORTED, "K = %d, d_model = %d do not fit in shared memory", Kmax, d_model);
    long long slots = ((long long)di.smem_optin - (long long)fixed) / p.slot_bytes;
    if (slots > kMaxSlots) slots = kMaxSlots;
    if (ring_slots_cap() > 0 && slots > ring_slots_cap()) slots = ring_slots_cap();
    // With two groups a slot must always come back to the same group (a group never waits on the
    // other's items, so only then can it never be a full ring pass ahead of a barrier it tests):
    // every batch takes `batch` slots and the ring holds a whole number of batch pairs.
    if (groups == 2) slots -= slots % (2 * batch);
    if (slots < (long long)groups * batch)
        CI_FAIL(COREINFER_ERR_UNSUPPORTED, "the ring of %lld slots is smaller than %d batches of %d rows", slots,
                groups, batch);
    p.n_slots = (int)slots;
    const size_t smem = fixed + (size_t)p.n_slots * p.slot_bytes;
    // Measured on the four model shapes: about 100 KB of the next layer requested ahead of the
    // exchange is best (12 rows of 8 or 10 KB; 4-5 rows of 18 KB); more delays the exchange's own
    // messages, less leaves the ring empty when the consumers come back.
    p.runahead = p.slot_bytes <= 12 * 1024 ? 12 : (96 * 1024 / p.slot_bytes < 4 ? 4 : 96 * 1024 / p.slot_bytes);
    p.ysum_ofs = (int)((size_t)p.n_slots * p.slot_bytes + fixed0);
    p.x0 = x0;
    p.y_last = y_last;
    p.y_layers = y_layers;
    p.x_layers = x_layers;
    p.ctrl = (unsigned*)workspace;
    p.ybuf = (float*)((uint8_t*)workspace + kCtrlBytes);

    // Control words and the reduction targets start at zero.
    CI_CUDA(cudaMemsetAsync(workspace, 0, b1_workspace_bytes(d_model), st));
    if (dtype == COREINFER_BF16)
        return gated ? launch_shape<__nv_bfloat16, true>(groups, vpt, p, G, smem, st)
                     : launch_shape<__nv_bfloat16, false>(groups, vpt, p, G, smem, st);
    return gated ? launch_shape<float, true>(groups, vpt, p, G, smem, st)
                 : launch_shape<float, false>(groups, vpt, p, G, smem, st);
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
