// Sentence-wise core-neuron selection at pre-fill (Definition 1 / Eq. 1, Eq. 3,
// Definition 2 / Eq. 2).  Three kernels, all integer work on float bit patterns, so the
// result is exact and independent of scheduling:
//
//   select_rows_*_kernel CTAs walk rows t = cta, cta + G, ...  A row is brought into shared
//                        memory by bulk copies.  Per row: count the positives P, k = ceil(alpha P),
//                        then an MSB-first radix select finds the exact bit pattern of the k-th
//                        largest positive value and how many entries equal to it are admitted
//                        (lowest index first).  Each thread owns fixed columns of every row, so
//                        the per-neuron membership counters of Eq. 3 live in its registers: no
//                        atomics.  At the end each CTA writes its counters as one u16 row.
//                        Two builds: the fast one (up to 255 rows per CTA: byte counters, the
//                        row kept in registers, digits of 8 + 12 + 11 bits) and the general one
//                        (16-bit counters, digits of 12 + 12 + 7 bits).
//   select_count_kernel  f[n] = sum over CTAs of those rows (int32).
//   select_top_kernel    one CTA: the K-th largest count c* by a histogram search on the count
//                        value, then an index-ordered scan admits f > c*, and the lowest-index
//                        f == c* until K are taken, and writes them in ascending index.
#include "common.cuh"

namespace coreinfer {

constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kSelMaxCtas = 256;
constexpr int kSelMaxVpt = 9;                        // d_ff <= 9 * 1024 * 4 = 36864
constexpr int kSelBins = 4096;
constexpr int kSelCtrlBytes = 256;
constexpr uint32_t kCopyChunk = 32768;
constexpr long long kSelWaitCycles = 3000000000LL;

// ceil(alpha * P - 1e-6) clamped to [0, P]; same expression as coreinfer_count, with the
// product and the difference rounded separately (no contraction).
__device__ __forceinline__ int count_dev(double frac, int n)
{
    if (n <= 0) return 0;
    double c = ceil(__dsub_rn(__dmul_rn(frac, (double)n), 1e-6));
    if (c < 0.0) c = 0.0;
    if (c > (double)n) c = (double)n;
    return (int)c;
}

__device__ __forceinline__ bool is_pos_bits(uint32_t b) { return (b - 1u) < 0x7F800000u; }

// The fp32 bit patterns of the four entries of group v of a row in shared memory.  16-bit
// inputs widen exactly (bf16: its bits are the upper half of the fp32 pattern; fp16: every
// value, subnormals included, is an fp32 value), so order, sign, zero and NaN are those of the
// stored values.  in_kind: 0 fp32, 1 bf16, 2 fp16.
__device__ __forceinline__ uint32_t half_to_f32_bits(uint32_t h)
{
    return __float_as_uint(__half2float(__ushort_as_half((unsigned short)h)));
}
__device__ __forceinline__ uint4 load_group(const uint8_t* row, int v, int in_kind)
{
    if (in_kind == 0) return reinterpret_cast<const uint4*>(row)[v];
    const uint2 w = reinterpret_cast<const uint2*>(row)[v];
    if (in_kind == 1) return make_uint4(w.x << 16, w.x & 0xffff0000u, w.y << 16, w.y & 0xffff0000u);
    return make_uint4(half_to_f32_bits(w.x & 0xffffu), half_to_f32_bits(w.x >> 16),
                      half_to_f32_bits(w.y & 0xffffu), half_to_f32_bits(w.y >> 16));
}

struct SelShared {
    int warp_tot[kSelWarps];
    int bin, above, bin_count, total;
    int abort_flag;
};

// Exclusive prefix sum over the block's threads; *total gets the block sum.
__device__ __forceinline__ int block_excl_scan(int v, SelShared* sh, int* total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) sh->warp_tot[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = sh->warp_tot[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int t = __shfl_up_sync(0xffffffffu, w, o);
            if (lane >= o) w += t;
        }
        sh->warp_tot[lane] = w;
    }
    __syncthreads();
    const int base = warp > 0 ? sh->warp_tot[warp - 1] : 0;
    *total = sh->warp_tot[kSelWarps - 1];
    __syncthreads();
    return base + incl - v;
}

// hist[kSelBins] holds digit counts.  Finds the bin holding the k-th largest element
// (1 <= k <= total): sh->bin, sh->above = elements in higher bins, sh->bin_count.
// With k_from_total, k = ceil(alpha * total) is formed here (total = number of positives).
// Returns k (block-uniform); with k == 0 nothing else is written.
__device__ __forceinline__ int find_bin(const int* hist, int k, bool k_from_total, double alpha,
                                        SelShared* sh)
{
    constexpr int PER = kSelBins / kSelThreads;   // 4 bins per thread, walked from the top
    const int top = kSelBins - 1 - PER * (int)threadIdx.x;
    int c[PER], s = 0;
#pragma unroll
    for (int i = 0; i < PER; ++i) { c[i] = hist[top - i]; s += c[i]; }
    int total;
    const int before = block_excl_scan(s, sh, &total);
    if (k_from_total) k = count_dev(alpha, total);
    if (k > 0 && before < k && k <= before + s) {
        int above = before;
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            if (above < k && k <= above + c[i]) { sh->bin = top - i; sh->above = above; sh->bin_count = c[i]; }
            above += c[i];
        }
    }
    __syncthreads();
    return k;
}

// HOLD: the thread keeps its columns of the row in registers (the shared-memory buffer is
// free for the next row at once); otherwise every pass re-reads them from shared memory.
template <int VPT, bool HOLD>
__global__ void __launch_bounds__(kSelThreads, 1)
select_rows_kernel(const uint8_t* __restrict__ act, int T, int N, long long ld_bytes, int in_kind, double alpha,
                   uint16_t* __restrict__ partial, unsigned* __restrict__ status, int nbuf, int row_bytes)
{
    extern __shared__ __align__(128) uint8_t smem[];
    const int buf_bytes = (row_bytes + 127) & ~127;
    int* hist = reinterpret_cast<int*>(smem + (size_t)nbuf * buf_bytes);
    uint64_t* bars = reinterpret_cast<uint64_t*>(hist + kSelBins);   // [2]
    SelShared* sh = reinterpret_cast<SelShared*>(bars + 2);

    const int tid = threadIdx.x;
    const int G = gridDim.x;
    const int nvec = (N + 3) >> 2;         // groups of four entries

    if (tid == 0) {
        mbar_init(smem_u32(&bars[0]), 1);
        mbar_init(smem_u32(&bars[1]), 1);
        sh->abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();

    int issued[2] = {0, 0};                // thread 0: copies issued per buffer
    auto issue_row = [&](int t, int b) {   // thread 0 only
        const uint32_t bar = smem_u32(&bars[b]);
        mbar_arrive_expect_tx(bar, (uint32_t)row_bytes);
        const uint8_t* src = act + (long long)t * ld_bytes;
        const uint32_t dst = smem_u32(smem + (size_t)b * buf_bytes);
        for (uint32_t off = 0; off < (uint32_t)row_bytes; off += kCopyChunk) {
            const uint32_t n = min(kCopyChunk, (uint32_t)row_bytes - off);
            bulk_g2s(dst + off, src + off, n, bar);
        }
        ++issued[b];
    };

    int cnt[VPT][4];
#pragma unroll
    for (int i = 0; i < VPT; ++i)
#pragma unroll
        for (int e = 0; e < 4; ++e) cnt[i][e] = 0;

    if (tid == 0 && (int)blockIdx.x < T) issue_row(blockIdx.x, 0);

    int iter = 0;
    for (int t = blockIdx.x; t < T; t += G, ++iter) {
        const int b = (nbuf == 2) ? (iter & 1) : 0;
        const uint32_t parity = (nbuf == 2) ? ((iter >> 1) & 1) : (iter & 1);
        // every thread finished with the previous row (barrier at the end of the loop body)
        if (tid == 0) {
            if (nbuf == 2) { if (t + G < T) issue_row(t + G, b ^ 1); }
            else if (!HOLD && iter > 0) issue_row(t, 0);
        }

        {   // bounded wait for this row's bytes
            const uint32_t bar = smem_u32(&bars[b]);
            if (!mbar_try_wait(bar, parity)) {
                const long long t0 = clock64();
                while (!mbar_try_wait(bar, parity)) {
                    if (clock64() - t0 > kSelWaitCycles) {
                        sh->abort_flag = 1;
                        atomicMax(status, (unsigned)kStatusTimeout);
                        break;
                    }
                }
            }
        }
        __syncthreads();
        if (sh->abort_flag) break;   // block-uniform

        const uint8_t* row = smem + (size_t)b * buf_bytes;
        // masked bit patterns of vector i: 0 stands for "not positive" (or beyond d_ff)
        auto load_vec = [&](int i) -> uint4 {
            const int v = tid + i * kSelThreads;
            uint4 q = make_uint4(0, 0, 0, 0);
            if (v < nvec) q = load_group(row, v, in_kind);
            if (v * 4 + 0 >= N || !is_pos_bits(q.x)) q.x = 0u;
            if (v * 4 + 1 >= N || !is_pos_bits(q.y)) q.y = 0u;
            if (v * 4 + 2 >= N || !is_pos_bits(q.z)) q.z = 0u;
            if (v * 4 + 3 >= N || !is_pos_bits(q.w)) q.w = 0u;
            return q;
        };
        uint4 held[HOLD ? VPT : 1];
        if (HOLD) {
#pragma unroll
            for (int i = 0; i < VPT; ++i) held[i] = load_vec(i);
            __syncthreads();   // every thread holds its columns: the buffer may be refilled
            if (nbuf == 1 && tid == 0 && t + G < T) issue_row(t + G, 0);
        }
        auto vec = [&](int i) -> uint4 { return HOLD ? held[HOLD ? i : 0] : load_vec(i); };

        // ---- radix select of the k-th largest positive pattern: 12 + 12 + 7 bits ----
        uint32_t vstar = 0u;
        int need = 0, eq_total = 0;
#pragma unroll 1
        for (int pass = 0; pass < 3; ++pass) {
            const int shift = pass == 0 ? 19 : (pass == 1 ? 7 : 0);
            const uint32_t dmask = pass == 2 ? 0x7Fu : 0xFFFu;
            const int pshift = pass == 0 ? 31 : (pass == 1 ? 19 : 7);   // prefix = bits >> pshift
            for (int i = tid; i < kSelBins; i += kSelThreads) hist[i] = 0;
            __syncthreads();
#pragma unroll
            for (int i = 0; i < VPT; ++i) {
                const uint4 q = vec(i);
                const uint32_t bb[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (bb[e] != 0u && (bb[e] >> pshift) == (vstar >> pshift))
                        atomicAdd(&hist[(bb[e] >> shift) & dmask], 1);
            }
            __syncthreads();
            need = find_bin(hist, need, pass == 0, alpha, sh);
            if (need == 0) break;                      // no positive entry in this row
            vstar |= (uint32_t)sh->bin << shift;
            need -= sh->above;
            eq_total = sh->bin_count;
            __syncthreads();
        }

        // ---- membership (Eq. 1) and its count (Eq. 3) ----
        if (need == 0) {
            // nothing to count
        } else if (need == eq_total) {
#pragma unroll
            for (int i = 0; i < VPT; ++i) {
                const uint4 q = vec(i);
                cnt[i][0] += (q.x >= vstar) ? 1 : 0;   // vstar > 0, masked entries are 0
                cnt[i][1] += (q.y >= vstar) ? 1 : 0;
                cnt[i][2] += (q.z >= vstar) ? 1 : 0;
                cnt[i][3] += (q.w >= vstar) ? 1 : 0;
            }
        } else {
            // more entries equal the threshold than places left: lower index first.
            // Index order = vector round i, then thread, then element.
            int taken = 0;
#pragma unroll
            for (int i = 0; i < VPT; ++i) {
                const uint4 q = vec(i);
                const uint32_t bb[4] = {q.x, q.y, q.z, q.w};
                int c = 0;
#pragma unroll
                for (int e = 0; e < 4; ++e) c += (bb[e] == vstar) ? 1 : 0;
                int tot;
                int rank = taken + block_excl_scan(c, sh, &tot);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (bb[e] > vstar) cnt[i][e] += 1;
                    else if (bb[e] == vstar) { cnt[i][e] += (rank < need) ? 1 : 0; ++rank; }
                }
                taken += tot;
            }
        }
        __syncthreads();   // the row buffer and the shared scratch are free again
    }

    // Never leave with a copy into this CTA's shared memory in flight.  On the normal path
    // every issued copy has been waited for; after an abort this is a last bounded wait.
    __syncthreads();
    if (tid == 0) {
        for (int b = 0; b < 2; ++b) {
            if (issued[b] == 0) continue;
            const uint32_t ph = (uint32_t)((issued[b] - 1) & 1);
            const long long t0 = clock64();
            while (!mbar_try_wait(smem_u32(&bars[b]), ph))
                if (clock64() - t0 > kSelWaitCycles) { atomicMax(status, (unsigned)kStatusTimeout); break; }
        }
    }

    uint16_t* out = partial + (size_t)blockIdx.x * ((size_t)nvec * 4);
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = tid + i * kSelThreads;
        if (v < nvec) {
            uint2 w;
            w.x = (uint32_t)cnt[i][0] | ((uint32_t)cnt[i][1] << 16);
            w.y = (uint32_t)cnt[i][2] | ((uint32_t)cnt[i][3] << 16);
            reinterpret_cast<uint2*>(out)[v] = w;
        }
    }
}

// The same selection for CTAs that walk at most 255 rows (every T up to 65280).  Differences
// that matter for speed:
//  * the membership counters are bytes, four to a register, so a thread can also keep all its
//    columns of the row in registers (36 of them at d_ff = 36864).  The row buffer is free as
//    soon as every thread has its columns, the next row's copy runs during the whole selection
//    of this one, and no pass re-reads shared memory;
//  * the first radix digit is the 8 exponent bits, counted in a histogram per warp (activations
//    crowd into a handful of exponents: in one shared histogram those additions queue on the
//    same few words), then 12 and 11 mantissa bits in the shared histogram, where the entries
//    that are left spread evenly.
constexpr int kWarpHistStride = 288;     // 256 exponent bins + 32 words (one per lane) that take the increments of masked entries

template <int VPT>
__global__ void __launch_bounds__(kSelThreads, 1)
select_rows_fast_kernel(const uint8_t* __restrict__ act, int T, int N, long long ld_bytes, int in_kind, double alpha,
                        uint16_t* __restrict__ partial, unsigned* __restrict__ status, int row_bytes)
{
    extern __shared__ __align__(128) uint8_t smem[];
    const int buf_bytes = (row_bytes + 127) & ~127;
    int* hist = reinterpret_cast<int*>(smem + buf_bytes);                        // [kSelBins + 32]: bins, then one word per lane for entries that do not count
    int* whist = hist + kSelBins + 32;                                           // [kSelWarps][kWarpHistStride]
    uint64_t* bar = reinterpret_cast<uint64_t*>(whist + ((kSelWarps * kWarpHistStride + 1) & ~1));
    SelShared* sh = reinterpret_cast<SelShared*>(bar + 1);

    const int tid = threadIdx.x;
    const int G = gridDim.x;
    const int nvec = (N + 3) >> 2;         // groups of four entries

    if (tid == 0) {
        mbar_init(smem_u32(bar), 1);
        sh->abort_flag = 0;
        mbar_fence_init();
    }
    // the per-warp exponent histograms start at zero; every row's merge leaves them at zero again
    for (int i = tid; i < kSelWarps * kWarpHistStride; i += kSelThreads) whist[i] = 0;
    __syncthreads();

    int issued = 0;                        // thread 0: copies issued
    auto issue_row = [&](int t) {          // thread 0 only
        const uint32_t b = smem_u32(bar);
        mbar_arrive_expect_tx(b, (uint32_t)row_bytes);
        const uint8_t* src = act + (long long)t * ld_bytes;
        const uint32_t dst = smem_u32(smem);
        for (uint32_t off = 0; off < (uint32_t)row_bytes; off += kCopyChunk) {
            const uint32_t n = min(kCopyChunk, (uint32_t)row_bytes - off);
            bulk_g2s(dst + off, src + off, n, b);
        }
        ++issued;
    };

    uint32_t cnt8[VPT];                    // four byte counters per vector (at most 255 rows per CTA)
#pragma unroll
    for (int i = 0; i < VPT; ++i) cnt8[i] = 0u;

    if (tid == 0 && (int)blockIdx.x < T) issue_row(blockIdx.x);

    int iter = 0;
    for (int t = blockIdx.x; t < T; t += G, ++iter) {
        {   // bounded wait for this row's bytes
            const uint32_t b = smem_u32(bar);
            const uint32_t parity = (uint32_t)(iter & 1);
            if (!mbar_try_wait(b, parity)) {
                const long long t0 = clock64();
                while (!mbar_try_wait(b, parity)) {
                    if (clock64() - t0 > kSelWaitCycles) {
                        sh->abort_flag = 1;
                        atomicMax(status, (unsigned)kStatusTimeout);
                        break;
                    }
                }
            }
        }
        __syncthreads();
        if (sh->abort_flag) break;   // block-uniform

        // This thread's columns.  kMasked (sign bit alone) stands for "not positive" (or beyond
        // d_ff): its "exponent" is 256, one past the real bins, it is below every positive pattern
        // as a signed integer and far from all of them as an unsigned difference, so no loop below
        // needs a test for it.
        constexpr uint32_t kMasked = 0x80000000u;
        const uint8_t* row = smem;
        uint4 held[VPT];
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int v = tid + i * kSelThreads;
            uint4 q = make_uint4(0, 0, 0, 0);
            if (v < nvec) q = load_group(row, v, in_kind);
            q.x = is_pos_bits(q.x) ? q.x : kMasked;
            q.y = is_pos_bits(q.y) ? q.y : kMasked;
            q.z = is_pos_bits(q.z) ? q.z : kMasked;
            q.w = is_pos_bits(q.w) ? q.w : kMasked;
            held[i] = q;
        }
        if (N & 3) {                                   // ragged width: the row's last vector reaches beyond d_ff
#pragma unroll
            for (int i = 0; i < VPT; ++i) {
                const int v = tid + i * kSelThreads;
                if (v * 4 + 1 >= N) held[i].y = kMasked;
                if (v * 4 + 2 >= N) held[i].z = kMasked;
                if (v * 4 + 3 >= N) held[i].w = kMasked;
            }
        }
        __syncthreads();             // every thread holds its columns: the buffer may be refilled
        if (tid == 0 && t + G < T) issue_row(t + G);
        // the shared histogram of the second digit starts at zero (the exponent digit does not use it)
        for (int i = tid; i < kSelBins; i += kSelThreads) hist[i] = 0;

        // ---- radix select of the k-th largest positive pattern: 8 + 12 + 11 bits ----
        uint32_t vstar = 0u;
        int need = 0, eq_total = 0;
        {   // exponent digit: per-warp histograms, merged and searched by the first 256 threads
            // Every entry increments a word, its exponent's bin (masked entries: word 256, never
            // read), so the loop has neither test nor branch (a predicated atomic compiles to one).
            const uint32_t mine = smem_u32(whist + (tid >> 5) * kWarpHistStride);
#pragma unroll
            for (int i = 0; i < VPT; ++i) {
                red_shared_inc(mine + ((held[i].x >> 23) << 2));
                red_shared_inc(mine + ((held[i].y >> 23) << 2));
                red_shared_inc(mine + ((held[i].z >> 23) << 2));
                red_shared_inc(mine + ((held[i].w >> 23) << 2));
            }
            __syncthreads();
            // thread t < 256 merges bin 255 - t (so thread order is bin order from the top) and
            // leaves the per-warp words at zero for the next row
            int c = 0;
            if (tid < 256) {
#pragma unroll 8
                for (int w = 0; w < kSelWarps; ++w) {
                    c += whist[w * kWarpHistStride + 255 - tid];
                    whist[w * kWarpHistStride + 255 - tid] = 0;
                }
            }
            int total;                                 // positives of the row
            const int before = block_excl_scan(c, sh, &total);
            const int k = count_dev(alpha, total);
            if (k > 0 && before < k && k <= before + c) { sh->bin = 255 - tid; sh->above = before; sh->bin_count = c; }
            __syncthreads();
            if (k > 0) {
                vstar = (uint32_t)sh->bin << 23;
                need = k - sh->above;
                eq_total = sh->bin_count;
            }
        }
        // When the whole bin is admitted (need == eq_total) its remaining bits do not matter: every
        // entry at or above the bin's lowest pattern is a member, and the search stops early.
        // After the second digit most bins hold a single entry, so the third pass is rare.
#pragma unroll 1
        for (int pass = 1; pass < 3 && need > 0 && need != eq_total; ++pass) {
            const int shift = pass == 1 ? 11 : 0;
            const uint32_t dmask = pass == 1 ? 0xFFFu : 0x7FFu;
            const int pshift = pass == 1 ? 23 : 11;                   // prefix = bits >> pshift
            if (pass == 2) {                                          // rare: the histogram is used a second time
                for (int i = tid; i < kSelBins; i += kSelThreads) hist[i] = 0;
                __syncthreads();
            }
            {   // entries whose higher digits equal the threshold's have bits - base < 2^pshift; their
                // digit is that difference's; everything else lands in the word after the bins
                const uint32_t base = (vstar >> pshift) << pshift;
                const uint32_t hist_s = smem_u32(hist);
                const uint32_t nbins = dmask + 1u;
                auto word_of = [&](uint32_t b) {
                    const uint32_t dgt = (b - base) >> shift;
                    return hist_s + ((dgt < nbins ? dgt : (uint32_t)kSelBins) << 2);
                };
#pragma unroll
                for (int i = 0; i < VPT; ++i) {
                    red_shared_inc(word_of(held[i].x));
                    red_shared_inc(word_of(held[i].y));
                    red_shared_inc(word_of(held[i].z));
                    red_shared_inc(word_of(held[i].w));
                }
            }
            __syncthreads();
            need = find_bin(hist, need, false, alpha, sh);            // ends with a barrier: the result is published
            vstar |= (uint32_t)sh->bin << shift;
            need -= sh->above;
            eq_total = sh->bin_count;
        }

        // ---- membership (Eq. 1) and its count (Eq. 3) ----
        if (need == 0) {
            // no positive entry in this row: nothing to count
        } else if (need == eq_total) {
            // signed comparison: masked entries are the most negative integer, positives are positive
            const int lo = (int)vstar;
#pragma unroll
            for (int i = 0; i < VPT; ++i)
                cnt8[i] += ((int)held[i].x >= lo ? 1u : 0u) | ((int)held[i].y >= lo ? 0x100u : 0u) |
                           ((int)held[i].z >= lo ? 0x10000u : 0u) | ((int)held[i].w >= lo ? 0x1000000u : 0u);
        } else {
            // more entries equal the threshold than places left: lower index first.
            // Index order = vector round i, then thread, then element.
            int taken = 0;
#pragma unroll
            for (int i = 0; i < VPT; ++i) {
                const uint32_t bb[4] = {held[i].x, held[i].y, held[i].z, held[i].w};
                int c = 0;
#pragma unroll
                for (int e = 0; e < 4; ++e) c += (bb[e] == vstar) ? 1 : 0;
                int tot;
                int rank = taken + block_excl_scan(c, sh, &tot);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if ((int)bb[e] > (int)vstar) cnt8[i] += 1u << (8 * e);
                    else if (bb[e] == vstar) { cnt8[i] += (rank < need ? 1u : 0u) << (8 * e); ++rank; }
                }
                taken += tot;
            }
        }
        // no barrier here: the next row writes shared memory only after its own barriers
    }

    // Never leave with a copy into this CTA's shared memory in flight.  On the normal path
    // every issued copy has been waited for; after an abort this is a last bounded wait.
    __syncthreads();
    if (tid == 0 && issued > 0) {
        const uint32_t ph = (uint32_t)((issued - 1) & 1);
        const long long t0 = clock64();
        while (!mbar_try_wait(smem_u32(bar), ph))
            if (clock64() - t0 > kSelWaitCycles) { atomicMax(status, (unsigned)kStatusTimeout); break; }
    }

    uint16_t* out = partial + (size_t)blockIdx.x * ((size_t)nvec * 4);
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = tid + i * kSelThreads;
        if (v < nvec) {
            uint2 w;
            w.x = (cnt8[i] & 0xffu) | ((cnt8[i] & 0xff00u) << 8);
            w.y = ((cnt8[i] >> 16) & 0xffu) | ((cnt8[i] >> 24) << 16);
            reinterpret_cast<uint2*>(out)[v] = w;
        }
    }
}

// f[n] = sum over the CTAs' u16 rows.  A block covers 32 groups of 4 neurons; its 8 warps take
// every 8th row each (so the loads of a column group are spread over 8 threads) and meet in
// shared memory.
constexpr int kCountCols = 32;
constexpr int kCountSlices = 8;

__global__ void __launch_bounds__(kCountCols * kCountSlices)
select_count_kernel(const uint16_t* __restrict__ partial, int G, int n4, int N, int32_t* __restrict__ f)
{
    __shared__ int4 acc[kCountSlices][kCountCols];
    const int col = threadIdx.x & (kCountCols - 1);
    const int slice = threadIdx.x / kCountCols;
    const int v = blockIdx.x * kCountCols + col;           // group of 4 neurons
    int4 c = make_int4(0, 0, 0, 0);
    if (v * 4 < n4) {
        for (int g = slice; g < G; g += kCountSlices) {
            const uint2 w = reinterpret_cast<const uint2*>(partial + (size_t)g * n4)[v];
            c.x += w.x & 0xffff; c.y += w.x >> 16; c.z += w.y & 0xffff; c.w += w.y >> 16;
        }
    }
    acc[slice][col] = c;
    __syncthreads();
    if (slice == 0 && v * 4 < N) {
#pragma unroll
        for (int sl = 1; sl < kCountSlices; ++sl) {
            const int4 o = acc[sl][col];
            c.x += o.x; c.y += o.y; c.z += o.z; c.w += o.w;
        }
        const int n = v * 4;
        f[n] = c.x;
        if (n + 1 < N) f[n + 1] = c.y;
        if (n + 2 < N) f[n + 2] = c.z;
        if (n + 3 < N) f[n + 3] = c.w;
    }
}

// One CTA.  Thread t owns the contiguous neurons [t*C, (t+1)*C).  The K-th largest count c* is
// found with the same histogram search as a row threshold (12 high bits of the count, then, for
// counts of 4096 and more, the low bits); the members are then f > c* plus the lowest-index
// f == c* until K are taken, written in ascending index with two block scans.
// Counts crowd into a few dozen values (near alpha * beta-ish * T), so a block-wide histogram would
// serialise thousands of shared-memory atomics on the same few words.  When the first-pass bins
// fit, every warp counts into a histogram of its own (`wstride` > 0: words per warp) and the 32
// of them are added up afterwards.
__global__ void __launch_bounds__(kSelThreads, 1)
select_top_kernel(const int32_t* __restrict__ f, int N, int K, int T, int32_t* __restrict__ S, int wstride)
{
    extern __shared__ __align__(128) uint8_t smem[];
    // counts in shared memory, one pad word per 32 so that thread t's contiguous run
    // [t*C, (t+1)*C) and its neighbours' fall into different banks
    int* fs = reinterpret_cast<int*>(smem);                               // [N + N/32 + 1]
    auto at = [](int n) { return n + (n >> 5); };
    int* hist = fs + ((N + (N >> 5) + 4) & ~3);                           // [kSelBins]
    SelShared* sh = reinterpret_cast<SelShared*>(hist + kSelBins);
    int* whist = reinterpret_cast<int*>(sh + 1);                          // [kSelWarps][wstride]
    const int tid = threadIdx.x;
    for (int i = tid; i < N; i += kSelThreads) fs[at(i)] = min(max(f[i], 0), T);   // counts lie in [0, T]; anything else is clamped
    const int C = (N + kSelThreads - 1) / kSelThreads;
    const int n0 = min(tid * C, N), n1 = min(n0 + C, N);

    int shift = 0;                      // counts lie in [0, T]; the first pass looks at f >> shift
    while ((T >> shift) >= kSelBins) ++shift;
    int cstar = 0, above = 0, need = K;
    for (int pass = 0; pass < (shift > 0 ? 2 : 1); ++pass) {
        if (pass == 0 && wstride > 0) {
            for (int i = tid; i < kSelWarps * wstride; i += kSelThreads) whist[i] = 0;
            __syncthreads();
            int* mine = whist + (tid >> 5) * wstride;
            for (int n = n0; n < n1; ++n) atomicAdd(&mine[fs[at(n)] >> shift], 1);
            __syncthreads();
            const int nb = (T >> shift) + 1;
            for (int b = tid; b < kSelBins; b += kSelThreads) {
                int c = 0;
                if (b < nb)
                    for (int w = 0; w < kSelWarps; ++w) c += whist[w * wstride + b];
                hist[b] = c;
            }
            __syncthreads();
        } else {
            for (int i = tid; i < kSelBins; i += kSelThreads) hist[i] = 0;
            __syncthreads();
            for (int n = n0; n < n1; ++n) {
                const int v = fs[at(n)];
                if (pass == 0) atomicAdd(&hist[v >> shift], 1);
                else if ((v >> shift) == (cstar >> shift)) atomicAdd(&hist[v & ((1 << shift) - 1)], 1);
            }
            __syncthreads();
        }
        find_bin(hist, need, false, 0.0, sh);
        cstar |= pass == 0 ? (sh->bin << shift) : sh->bin;
        above += sh->above;
        need -= sh->above;
        __syncthreads();
    }
    // need = how many f == c* are admitted, lowest index first

    int ce = 0;
    for (int n = n0; n < n1; ++n) ce += fs[at(n)] == cstar ? 1 : 0;
    int tot;
    int rank = block_excl_scan(ce, sh, &tot);
    int cm = 0;
    {
        int r = rank;
        for (int n = n0; n < n1; ++n) {
            const int v = fs[at(n)];
            if (v > cstar) ++cm;
            else if (v == cstar) { cm += (r < need) ? 1 : 0; ++r; }
        }
    }
    int pos = block_excl_scan(cm, sh, &tot);
    for (int n = n0; n < n1; ++n) {
        const int v = fs[at(n)];
        bool m = v > cstar;
        if (v == cstar) { m = rank < need; ++rank; }
        if (m) S[pos++] = n;
    }
}

static size_t sel_fixed_smem() { return kSelBins * sizeof(int) + 2 * sizeof(uint64_t) + sizeof(SelShared) + 128; }

template <int VPT>
static coreinfer_status launch_rows(int grid, size_t smem, cudaStream_t st, const uint8_t* act, int T, int N,
                                    long long ld_bytes, int in_kind, double alpha, uint16_t* partial,
                                    unsigned* status, int nbuf, int row_bytes)
{
    auto kern = select_rows_kernel<VPT, (VPT <= 5)>;
    CI_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    kern<<<grid, kSelThreads, smem, st>>>(act, T, N, ld_bytes, in_kind, alpha, partial, status, nbuf, row_bytes);
    CI_CUDA(cudaGetLastError());
    return COREINFER_OK;
}

static size_t sel_fast_fixed_smem()
{
    return (kSelBins + 32) * sizeof(int) + ((kSelWarps * kWarpHistStride + 1) & ~1) * sizeof(int) + sizeof(uint64_t) +
           sizeof(SelShared) + 128;
}

template <int VPT>
static coreinfer_status launch_rows_fast(int grid, size_t smem, cudaStream_t st, const uint8_t* act, int T, int N,
                                         long long ld_bytes, int in_kind, double alpha, uint16_t* partial,
                                         unsigned* status, int row_bytes)
{
    auto kern = select_rows_fast_kernel<VPT>;
    CI_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    kern<<<grid, kSelThreads, smem, st>>>(act, T, N, ld_bytes, in_kind, alpha, partial, status, row_bytes);
    CI_CUDA(cudaGetLastError());
    return COREINFER_OK;
}

// The K entries of f[0 .. N) with the largest count (all counts in [0, max_count]), ascending.
coreinfer_status launch_select_top(const int32_t* f, int N, int K, int max_count, int32_t* S, const DeviceInfo& di,
                                   cudaStream_t st)
{
    const int n4 = (N + 3) & ~3;
    size_t smem_top = ((size_t)n4 + n4 / 32 + 8) * sizeof(int) + kSelBins * sizeof(int) + sizeof(SelShared) + 16;
    int top_shift = 0;
    while ((max_count >> top_shift) >= kSelBins) ++top_shift;
    int wstride = (((max_count >> top_shift) + 1 + 31) & ~31) + 1;   // odd: the warps' copies of a bin fall into different banks
    if (smem_top + (size_t)kSelWarps * wstride * sizeof(int) <= (size_t)di.smem_optin)
        smem_top += (size_t)kSelWarps * wstride * sizeof(int);
    else
        wstride = 0;
    if (smem_top > (size_t)di.smem_optin)
        CI_FAIL(COREINFER_ERR_UNSUPPORTED, "d_ff = %d: the counts do not fit in shared memory", N);
    CI_CUDA(cudaFuncSetAttribute(select_top_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_top));
    select_top_kernel<<<1, kSelThreads, smem_top, st>>>(f, N, K, max_count, S, wstride);
    CI_CUDA(cudaGetLastError());
    return COREINFER_OK;
}

}  // namespace coreinfer

using namespace coreinfer;

extern "C" {

size_t coreinfer_select_workspace_bytes(int32_t T, int32_t d_ff)
{
    if (T < 1 || d_ff < 1) return 0;
    const size_t n4 = ((size_t)d_ff + 3) & ~(size_t)3;
    const size_t ctas = (size_t)(T < kSelMaxCtas ? T : kSelMaxCtas);
    return kSelCtrlBytes + ctas * n4 * sizeof(uint16_t) + n4 * sizeof(int32_t);
}

coreinfer_status coreinfer_select_core(const void* act, coreinfer_dtype act_dtype, int32_t T, int32_t d_ff,
                                       int64_t ld_act, double alpha, double beta, int32_t* core_idx,
                                       int32_t* counts_out, void* workspace, size_t workspace_bytes,
                                       void* cuda_stream)
{
    if (!dtype_known(act_dtype))
        CI_FAIL(COREINFER_ERR_UNSUPPORTED, "activations must be fp32, bf16 or fp16 (dtype %d given)", (int)act_dtype);
    const int esize = (int)dtype_size(act_dtype);
    const int in_kind = act_dtype == COREINFER_F32 ? 0 : (act_dtype == COREINFER_BF16 ? 1 : 2);
    const int per16 = 16 / esize;          // entries per 16 bytes: rows start and end on 16-byte boundaries
    if (!act || !core_idx) CI_FAIL(COREINFER_ERR_INVALID_ARG, "act / core_idx is NULL");
    if (T < 1 || d_ff < 1) CI_FAIL(COREINFER_ERR_INVALID_ARG, "T = %d, d_ff = %d must be >= 1", T, d_ff);
    if (!(alpha > 0.0 && alpha <= 1.0) || !(beta > 0.0 && beta <= 1.0))
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "alpha = %g, beta = %g must lie in (0, 1]", alpha, beta);
    if (coreinfer_count(beta, d_ff) < 1)
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "beta = %g selects no neuron of d_ff = %d", beta, d_ff);
    if (ld_act < d_ff || (ld_act % per16) != 0 || !aligned16(act))
        CI_FAIL(COREINFER_ERR_INVALID_ARG, "act must be 16-byte aligned with ld_act >= d_ff and ld_act %% %d == 0", per16);
    if (d_ff > kSelMaxVpt * kSelThreads * 4)
        CI_FAIL(COREINFER_ERR_UNSUPPORTED, "d_ff = %d exceeds %d", d_ff, kSelMaxVpt * kSelThreads * 4);
    if (!workspace || !aligned16(workspace)) CI_FAIL(COREINFER_ERR_WORKSPACE, "workspace is NULL or misaligned");
    const size_t need = coreinfer_select_workspace_bytes(T, d_ff);
    if (workspace_bytes < need)
        CI_FAIL(COREINFER_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, need);
    DeviceInfo di;
    coreinfer_status s = device_info(&di);
    if (s != COREINFER_OK) return s;
    cudaStream_t st = (cudaStream_t)cuda_stream;

    const int n4 = (d_ff + 3) & ~3;
    const int row_bytes = (d_ff + per16 - 1) / per16 * 16;       // whole 16-byte pieces, within ld_act entries
    int G = T < di.sm_count ? T : di.sm_count;
    if (G > kSelMaxCtas) G = kSelMaxCtas;
    const size_t buf = ((size_t)row_bytes + 127) & ~(size_t)127;
    // byte counters (the fast kernel) hold 255 rows per CTA: more CTAs than SMs where that needs it
    int G_fast = G;
    if ((T + G_fast - 1) / G_fast > 255) G_fast = (T + 254) / 255;
    const bool fast = G_fast <= kSelMaxCtas && sel_fast_fixed_smem() + buf <= (size_t)di.smem_optin;
    if (fast) G = G_fast;
    if ((T + G - 1) / G > 65535)
        CI_FAIL(COREINFER_ERR_UNSUPPORTED, "T = %d: more than 65535 rows per CTA", T);
    const int K = coreinfer_count(beta, d_ff);

    unsigned* status = (unsigned*)workspace;
    uint16_t* partial = (uint16_t*)((uint8_t*)workspace + kSelCtrlBytes);
    int32_t* f = counts_out ? counts_out : (int32_t*)(partial + (size_t)(T < kSelMaxCtas ? T : kSelMaxCtas) * n4);
    CI_CUDA(cudaMemsetAsync(workspace, 0, kSelCtrlBytes, st));

    const size_t fixed = sel_fixed_smem();
    if (fixed + buf > (size_t)di.smem_optin)
        CI_FAIL(COREINFER_ERR_UNSUPPORTED, "a row of d_ff = %d does not fit in shared memory", d_ff);
    const int nbuf = (fixed + 2 * buf <= (size_t)di.smem_optin) ? 2 : 1;
    const size_t smem = fixed + nbuf * buf;
    const size_t smem_fast = sel_fast_fixed_smem() + buf;
    const int vpt = (n4 / 4 + kSelThreads - 1) / kSelThreads;
#define CI_ROWS(V)                                                                                        \
    case V:                                                                                               \
        s = fast ? launch_rows_fast<V>(G, smem_fast, st, (const uint8_t*)act, T, d_ff,                   \
                                       (long long)ld_act * esize, in_kind, alpha, partial, status,        \
                                       row_bytes)                                                         \
                 : launch_rows<V>(G, smem, st, (const uint8_t*)act, T, d_ff, (long long)ld_act * esize,   \
                                  in_kind, alpha, partial, status, nbuf, row_bytes);                      \
        break;
    switch (vpt) {
        CI_ROWS(1) CI_ROWS(2) CI_ROWS(3) CI_ROWS(4) CI_ROWS(5) CI_ROWS(6) CI_ROWS(7) CI_ROWS(8) CI_ROWS(9)
        default: CI_FAIL(COREINFER_ERR_UNSUPPORTED, "d_ff = %d not built", d_ff);
    }
#undef CI_ROWS
    if (s != COREINFER_OK) return s;

    select_count_kernel<<<(n4 / 4 + kCountCols - 1) / kCountCols, kCountCols * kCountSlices, 0, st>>>(partial, G, n4, d_ff, f);
    CI_CUDA(cudaGetLastError());

    return launch_select_top(f, d_ff, K, T, core_idx, di, st);
}

}  // extern "C"
