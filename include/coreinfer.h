/*
 * coreinfer.h -- C ABI of the CoreInfer core-sparse FFN path for NVIDIA B200 (sm_100a).
 *
 * The library implements, on one GPU, the three stages of the method:
 *   (1) sentence-wise core-neuron selection at pre-fill   (Definition 1 / Eq. 1,
 *       Eq. 3, Definition 2 / Eq. 2),
 *   (2) one-shot compaction of the selected weights       (Section 5.3: only the
 *       needed neurons are deployed, fixed for the whole decode),
 *   (3) the decode-stage FFN over those fixed neurons     (Section 4.2),
 * plus a dense FFN on the uncompacted weights that produces the pre-fill
 * activations the selection consumes.
 *
 * Conventions for every entry point
 *   - "device" pointers are CUDA device memory of the current device; "host"
 *     pointers are ordinary host memory.  Every buffer is owned by the caller.
 *     The library allocates no device memory.  Between calls it keeps a
 *     thread-local error string, per-device properties it looked up once, and
 *     the fixed scratch array of coreinfer_ffn_decode_stack_noalloc (whose
 *     contents carry no meaning from one call to the next).
 *   - Matrices are row-major and dense.  Device pointers must be 16-byte
 *     aligned; d_model * sizeof(element) must be a multiple of 16.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = default stream).
 *     Calls only enqueue work on that stream and return; they never
 *     synchronise.  Outputs are valid once the stream reaches that point.
 *   - Errors: arguments are checked on the host before anything is enqueued.
 *     A call that returns a status other than COREINFER_OK has enqueued
 *     nothing, except COREINFER_ERR_CUDA, which reports a failed launch.
 *     coreinfer_last_error() gives the reason as text.  Nothing aborts, traps
 *     or throws.
 *   - There is no CPU fallback: without a CUDA device every compute entry point
 *     fails with COREINFER_ERR_CUDA.
 *   - Sizes of "top fractions" follow one rule everywhere: coreinfer_count().
 */
#ifndef COREINFER_H_
#define COREINFER_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    COREINFER_OK = 0,
    COREINFER_ERR_INVALID_ARG = 1,   /* NULL / misaligned pointer, size or fraction out of range */
    COREINFER_ERR_UNSUPPORTED = 2,   /* dtype / kind / batch / size outside what is built */
    COREINFER_ERR_WORKSPACE = 3,     /* workspace missing or smaller than *_workspace_bytes() */
    COREINFER_ERR_CUDA = 4,          /* CUDA runtime reported an error (no device, failed launch) */
    COREINFER_ERR_TIMEOUT = 5        /* a bounded device-side wait gave up (see coreinfer_workspace_status) */
} coreinfer_status;

/* Storage types of weights and layer inputs.  F16 is the type of the paper's runs (Section 5
 * "Models": FP16 weights, FP32 intermediate activations); the workload configurations use BF16. */
typedef enum { COREINFER_F32 = 0, COREINFER_BF16 = 1, COREINFER_F16 = 2 } coreinfer_dtype;

/* FFN kinds.  RELU:        h = max(W_up x + b_up, 0)
 *             RELU_GATED:  h = max(W_gate x, 0) * (W_up x)        (no up bias)
 *             SILU_GATED:  h = silu(W_gate x) * (W_up x), silu(g) = g / (1 + exp(-g))   (no up bias)
 * and in all of them y = W_down h + b_down.  h is the "activation layer" output A(x) that
 * Definition 1 ranks.  The paper reports core neurons for SiLU models (Section 5.1, appendix
 * on LLaMA3.1-8b) without giving them another score, so Definition 1 applies to h as it
 * stands: entries of h that are not positive are never core neurons. */
typedef enum { COREINFER_FFN_RELU = 0, COREINFER_FFN_RELU_GATED = 1, COREINFER_FFN_SILU_GATED = 2 } coreinfer_ffn_kind;

#define COREINFER_MAX_BATCH 8
#define COREINFER_MAX_LAYERS 128

/* Size of a "top fraction" (Definition 1: top alpha of the positive activations of
 * a token; Definition 2: top beta of all neurons): ceil(frac * n) clamped to
 * [0, n], evaluated as ceil(frac * n - 1e-6) in double so that decimal fractions
 * whose product is an integer (0.2 * 20480) do not round up.  Pure host function. */
int32_t coreinfer_count(double frac, int32_t n);

/* Text of the last error on the calling thread (static storage, never NULL). */
const char* coreinfer_last_error(void);

/* ------------------------------------------------------------------ (1) --
 * Sentence-wise core-neuron selection (Definition 1 / Eq. 1, Eq. 3,
 * Definition 2 / Eq. 2).
 *
 * For each of the T rows of `act`, the token-wise core set is the
 * k_t = coreinfer_count(alpha, P_t) largest of its P_t positive entries
 * (positive on the bit pattern: sign clear, not zero, not NaN; equal values go
 * to the lower index).  f[n] counts the rows whose set contains n.  The result
 * is the K = coreinfer_count(beta, d_ff) neurons with the largest f (equal
 * counts go to the lower index), written in ascending index order.
 *
 *   act         device, [T, d_ff] with row stride ld_act elements; fp32 (the precision the
 *               method keeps activations in), bf16 or fp16 (widened exactly: order, sign, zero
 *               and NaN are those of the stored values).  ld_act >= d_ff and a multiple of 4
 *               (fp32) or 8 (16-bit): every row starts on a 16-byte boundary.
 *   core_idx    device, out, K int32 (capacity >= K).
 *   counts_out  device, out, [d_ff] int32 = f, or NULL.
 *   workspace   device scratch of at least coreinfer_select_workspace_bytes();
 *               contents need not be initialised and are clobbered.
 * Errors: INVALID_ARG (NULL, alignment, T < 1, d_ff < 1, alpha or beta outside
 * (0, 1]), UNSUPPORTED (dtype; d_ff or T beyond what the kernels are built
 * for, see coreinfer_last_error), WORKSPACE, CUDA. */
size_t coreinfer_select_workspace_bytes(int32_t T, int32_t d_ff);

coreinfer_status coreinfer_select_core(const void* act, coreinfer_dtype act_dtype,
                                       int32_t T, int32_t d_ff, int64_t ld_act,
                                       double alpha, double beta,
                                       int32_t* core_idx, int32_t* counts_out,
                                       void* workspace, size_t workspace_bytes,
                                       void* cuda_stream);

/* ------------------------------------------------------------------ (2) --
 * Compaction (Section 5.3: the neurons found at pre-fill are the only ones
 * deployed for decoding).  Pure data movement; outputs are byte-identical
 * copies of the selected elements.
 *
 *   w_up    device [d_ff, d_model]          w_up_c    device out [K, d_model]  = w_up[core_idx[k], :]
 *   w_gate  device [d_ff, d_model] or NULL  w_gate_c  device out [K, d_model]  (NULL iff w_gate NULL)
 *   w_down  device [d_model, d_ff]          w_downT_c device out [K, d_model]  = w_down[:, core_idx[k]]
 *   b_up    device [d_ff] or NULL           b_up_c    device out [K]           (NULL iff b_up NULL)
 *   core_idx device [K] int32, ascending, unique, each in [0, d_ff) (trusted).
 * All tensors share `dtype`.  1 <= K <= d_ff.
 * Errors: INVALID_ARG, UNSUPPORTED, CUDA. */
coreinfer_status coreinfer_compact(const void* w_up, const void* w_gate, const void* w_down,
                                   const void* b_up, coreinfer_dtype dtype,
                                   int32_t d_model, int32_t d_ff,
                                   const int32_t* core_idx, int32_t K,
                                   void* w_up_c, void* w_gate_c, void* w_downT_c, void* b_up_c,
                                   void* cuda_stream);

/* Checks a core index list before it is used: coreinfer_compact trusts `core_idx` (its gather
 * kernels read the weights at those indices without a bounds test), so a list that does not
 * come from coreinfer_select_core should pass through here first.  (A helper of the boundary;
 * the paper has no counterpart.)  Enqueues one small kernel that writes
 *   report[0] = number of positions k with core_idx[k] outside [0, d_ff) or not greater than
 *               core_idx[k-1] (the list must be strictly ascending),
 *   report[1] = the first such position, INT32_MAX if there is none,
 * to `report` (device, two int32); the caller reads them back once the stream has reached that
 * point.  Only core_idx[0 .. K) is read.
 * Errors: INVALID_ARG, CUDA. */
coreinfer_status coreinfer_verify_core_idx(const int32_t* core_idx, int32_t K, int32_t d_ff,
                                           int32_t* report, void* cuda_stream);

/* ------------------------------------------------------------------ (3) --
 * Decode FFN over compacted weights (Section 4.2), one layer:
 *   h_k = act(w_up_c[k,:] . x (+ b_up_c[k]))   [gated: max(w_gate_c[k,:] . x, 0) * (w_up_c[k,:] . x)]
 *   y_j = sum_k h_k * w_downT_c[k, j] + b_down[j]
 * h is held in fp32 and never leaves the chip (Section 5 "Models": fp32
 * intermediate activations).  Sums are fp32; their order is not fixed between
 * runs (partial results are combined with floating-point atomics).
 *
 *   x          device [batch, d_model] in `dtype`
 *   w_*_c      device [K, d_model] in `dtype` (w_gate_c NULL iff kind is RELU)
 *   b_up_c     device [K] in `dtype` or NULL (RELU only); b_down device [d_model] in `dtype` or NULL
 *   y          device out [batch, d_model] fp32
 *   workspace  device scratch of at least coreinfer_ffn_decode_workspace_bytes().
 * 1 <= batch <= COREINFER_MAX_BATCH.  At batch 1 a row (d_model elements) may take up to 21504 bytes
 * (d_model <= 10752 in bf16 / fp16, 5376 in fp32); wider rows return UNSUPPORTED.
 * Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE, CUDA. */
size_t coreinfer_ffn_decode_workspace_bytes(int32_t batch, int32_t d_model, int32_t K);

coreinfer_status coreinfer_ffn_decode(const void* x, int32_t batch, coreinfer_dtype dtype,
                                      coreinfer_ffn_kind kind, int32_t d_model, int32_t K,
                                      const void* w_up_c, const void* w_gate_c,
                                      const void* w_downT_c,
                                      const void* b_up_c, const void* b_down,
                                      float* y, void* workspace, size_t workspace_bytes,
                                      void* cuda_stream);

/* One decode step through a stack of L compacted FFN layers in a single
 * persistent launch (the decode loop of Section 4.2 over all layers: the sets are
 * fixed, so every layer's weights can be streamed without waiting for its input).
 * The paper does not describe what sits between two FFN layers; this entry point
 * chains them with a parameter-free residual + RMS normalisation,
 *   x_{l+1} = round_to_dtype( (x_l + y_l) / sqrt(mean_j (x_l + y_l)_j^2) ),
 * so that each layer truly depends on the previous one.
 *
 *   layers     host array of L descriptors (device pointers inside, same meaning
 *              as in coreinfer_ffn_decode); read during the call only.
 *   x0         device [batch, d_model] in `dtype`: input of layer 0.
 *   y_last     device out [batch, d_model] fp32: FFN output of layer L-1.
 *   y_layers   device out [L, batch, d_model] fp32: every layer's FFN output, or NULL.
 *   x_layers   device out [L, batch, d_model] in `dtype`: every layer's input as
 *              consumed, or NULL.
 *   workspace  at least coreinfer_ffn_decode_stack_workspace_bytes().
 * 1 <= batch <= COREINFER_MAX_BATCH, 1 <= L <= COREINFER_MAX_LAYERS.  batch 1 is the single
 * persistent launch described here; 2..8 sequences (sharing the core sets) read every weight
 * byte once for all sequences: in bf16 with d_model a multiple of 256 up to 4096 again as one
 * persistent launch (tensor cores, the sequences on the N side), otherwise as one batched FFN
 * launch plus one glue launch per layer.
 * Thread blocks of this launch wait on one another at layer boundaries; every
 * such wait is bounded, and a wait that gives up makes all blocks return early
 * and records COREINFER_ERR_TIMEOUT in the workspace (read it with
 * coreinfer_workspace_status after the stream has drained).  The launch is
 * cooperative: it needs the whole GPU to itself to be co-resident.
 * Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE, CUDA. */
typedef struct {
    const void* w_up_c;
    const void* w_gate_c;
    const void* w_downT_c;
    const void* b_up_c;
    const void* b_down;
    int32_t K;
    int32_t reserved;
} coreinfer_layer;

size_t coreinfer_ffn_decode_stack_workspace_bytes(int32_t L, int32_t batch, int32_t d_model,
                                                  int32_t K_max);

coreinfer_status coreinfer_ffn_decode_stack(const coreinfer_layer* layers, int32_t L,
                                            const void* x0, int32_t batch,
                                            coreinfer_dtype dtype, coreinfer_ffn_kind kind,
                                            int32_t d_model,
                                            float* y_last, float* y_layers, void* x_layers,
                                            void* workspace, size_t workspace_bytes,
                                            void* cuda_stream);

/* The same decode step as coreinfer_ffn_decode_stack for callers that cannot allocate device
 * memory when they decode.  (The paper has no counterpart: this is a deployment convenience.)
 * Typical cases: a server that gave all free HBM to its own pools at start-up and has nothing
 * left to carve a workspace from; code running under a host framework that forbids cudaMalloc
 * on its threads, since that call synchronises the device; a latency-critical loop that may
 * not call an allocator.  The kernel's scratch (control words and per-layer reduction targets)
 * sits in a fixed 128 KiB array inside the library image, so every GPU that loads the library
 * gives up 128 KiB for the life of the process, and the call itself allocates nothing (no
 * cudaMalloc / cudaFree, no allocating library routine).
 *
 * Arguments and results are those of coreinfer_ffn_decode_stack without the workspace pair,
 * for batch 1 only (any other batch returns COREINFER_ERR_UNSUPPORTED).
 * Limit: the scratch the kernel needs, 256 + 12 * d_model bytes (any number of layers), must fit
 * in 128 KiB, i.e. d_model <= 10901 (which covers every row width the batch-1 kernel takes); wider
 * models return COREINFER_ERR_UNSUPPORTED and enqueue nothing.
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress),
 * which is set-up work rather than stream work: make that first call before starting any
 * stream capture.
 * All calls share the one array.  Each call clears the part it uses on `cuda_stream` before
 * its kernel runs, so back-to-back calls on one stream are independent of what the previous
 * one left behind; two calls that can overlap on the GPU (different streams, no ordering
 * between them) race on it and give undefined results.  Because the array is private, the
 * status word of a bounded wait that gave up cannot be read back after this entry point;
 * callers that need that report use coreinfer_ffn_decode_stack.
 * Errors: INVALID_ARG, UNSUPPORTED, CUDA. */
coreinfer_status coreinfer_ffn_decode_stack_noalloc(const coreinfer_layer* layers, int32_t L,
                                                    const void* x0, int32_t batch,
                                                    coreinfer_dtype dtype, coreinfer_ffn_kind kind,
                                                    int32_t d_model,
                                                    float* y_last, float* y_layers, void* x_layers,
                                                    void* cuda_stream);

/* Synchronises `cuda_stream`, then reads the status word that the most recent
 * decode call using `workspace` left there: COREINFER_OK, or COREINFER_ERR_TIMEOUT
 * if a bounded device-side wait gave up (outputs of that call are then
 * undefined).  Returns COREINFER_ERR_CUDA if the synchronisation or copy fails. */
coreinfer_status coreinfer_workspace_status(const void* workspace, void* cuda_stream);

/* Phase timing of the persistent decode kernels (a profiling aid; the paper has no counterpart).
 * Only a library built with -DCOREINFER_STAMPS records anything; the normal build returns
 * COREINFER_ERR_UNSUPPORTED.  After this call, every coreinfer_ffn_decode_stack launch made
 * from the calling thread stores the SM cycle counter (clock64) at fixed points of each layer
 * into `stamps`: device, [CTAs = SM count][L][COREINFER_STAMP_SLOTS] 64-bit words, as long as
 * `bytes` covers that; launches with more layers than fit record nothing.  Batch-1 slots:
 * 0 layer start, 1 up rows consumed, 2 h formed, 3 down rows consumed, 4 the CTA's partial y
 * assembled, 5 its bulk reduction complete, 6 arrival at the grid barrier issued, 7 all CTAs
 * arrived, 8 sum read back, 9 next input formed.  For 2..8 sequences: 0 layer start, 1 up units
 * done, 3 down units done, 4 partial flushed, 7 all CTAs arrived, 8 sums read back, 9 next input
 * formed.  Slots not listed stay untouched.  NULL switches recording off.  The buffer is the
 * caller's and must outlive the launches. */
#define COREINFER_STAMP_SLOTS 16
coreinfer_status coreinfer_debug_stamps(void* stamps, size_t bytes);

/* ------------------------------------------------------------------ (4) --
 * Dense FFN on the uncompacted weights: the pre-fill pass whose intermediate
 * activations A = h [T, d_ff] are what Definition 1 is applied to.
 *
 *   x       device [T, d_model] in `dtype`
 *   w_up    device [d_ff, d_model]; w_gate same or NULL (NULL iff RELU); w_down device [d_model, d_ff]
 *   b_up    device [d_ff] or NULL (RELU only); b_down device [d_model] or NULL; all in `dtype`
 *   h_out   device out [T, d_ff] fp32 or NULL
 *   y_out   device out [T, d_model] fp32 or NULL (needs h_out: y is computed from the stored fp32 h)
 * Products are exact (fp32 or bf16 inputs), sums are fp32.
 * Errors: INVALID_ARG, UNSUPPORTED, CUDA. */
coreinfer_status coreinfer_ffn_dense_ref(const void* x, int32_t T, coreinfer_dtype dtype,
                                         coreinfer_ffn_kind kind, int32_t d_model, int32_t d_ff,
                                         const void* w_up, const void* w_gate, const void* w_down,
                                         const void* b_up, const void* b_down,
                                         float* h_out, float* y_out, void* cuda_stream);

/* ------------------------------------------------------------------ (6) --
 * Core sets over several sentences.
 *
 * Eq. 3 is a sum over tokens, so the counts of a prompt that arrives in pieces add up, and
 * similarity-guided prediction (Section 4.1) takes, for a semantic group of training sentences,
 * "the top gamma neurons that appear most frequently within that semantic group": the count of a
 * neuron is the number of the group's sentences whose sentence-wise core set holds it.  Both end
 * in the same rule as Definition 2: the top fraction by count, equal counts to the lower index.
 *
 *   coreinfer_counts_add      counts[n] += f[n]                 (f: the counts_out of a piece)
 *   coreinfer_counts_add_set  counts[core_idx[k]] += 1          (one sentence of a group)
 *   coreinfer_top_by_count    core_idx <- the coreinfer_count(frac, d_ff) neurons with the largest
 *                             counts, ascending.  Counts must lie in [0, max_count] (the number
 *                             of tokens or sentences counted); values outside are clamped.
 * All pointers device; int32 counts [d_ff]; members of a set must be distinct.
 * Errors: INVALID_ARG, UNSUPPORTED (d_ff too large for the kernel's shared memory), CUDA. */
coreinfer_status coreinfer_counts_add(int32_t* counts, const int32_t* f, int32_t d_ff, void* cuda_stream);
coreinfer_status coreinfer_counts_add_set(int32_t* counts, const int32_t* core_idx, int32_t K, int32_t d_ff,
                                          void* cuda_stream);
coreinfer_status coreinfer_top_by_count(const int32_t* counts, int32_t d_ff, int32_t max_count, double frac,
                                        int32_t* core_idx, void* cuda_stream);

/* Core-neuron similarity of two sets (Section 3.2, Insight-2: "the ratio of identical neurons to
 * the total number of neurons involved"; the quantity Insight-1 tracks while a sentence grows).
 * set_a must be ascending, set_b may be in any order; both device.  Writes
 * shared_involved[0] = |A and B|, shared_involved[1] = |A or B| (device, two int32); the
 * similarity is their quotient.  Errors: INVALID_ARG, CUDA. */
coreinfer_status coreinfer_core_similarity(const int32_t* set_a, int32_t K_a, const int32_t* set_b, int32_t K_b,
                                           int32_t* shared_involved, void* cuda_stream);

/* The semantic group of an input (similarity-guided prediction; appendix on its clustering: K-Means
 * on a layer's activation): the centroid at the smallest Euclidean distance from the feature
 * vector v; equal distances go to the lower group.  Which vector represents an input, and the
 * clustering that produced the centroids, are the caller's.
 *   centroids device [G, D] fp32; v device [D] fp32; group_out device int32;
 *   workspace device, 8-byte aligned, at least coreinfer_nearest_centroid_workspace_bytes(G): on
 *   return it holds the G squared distances as doubles.
 * Errors: INVALID_ARG, WORKSPACE, CUDA. */
size_t coreinfer_nearest_centroid_workspace_bytes(int32_t G);
coreinfer_status coreinfer_nearest_centroid(const float* centroids, int32_t G, int32_t D, const float* v,
                                            int32_t* group_out, void* workspace, size_t workspace_bytes,
                                            void* cuda_stream);

/* Changing a deployed core set in place.  Fig. 1 lets the sentence-wise set be updated after a
 * stability estimate; the paper gives no rule for it.  This call is the mechanism (the estimate
 * is coreinfer_core_similarity between the deployed and the newly selected set; when to act on
 * it is the caller's): only the rows whose neuron leaves the set are rewritten.
 *   slot_neuron   device in/out [K]: the neuron each row of the compacted buffers holds now (any
 *                 order; after coreinfer_compact it is the core_idx given there).
 *   core_idx_new  device [K] ascending: the set to deploy.
 * Rows whose neuron is not in core_idx_new are refilled, in ascending row order, with the
 * members of core_idx_new not held yet, in ascending neuron order (weights gathered from the
 * dense matrices as in coreinfer_compact); slot_neuron is updated; n_changed_out (device int32)
 * receives the number of rows rewritten.  Afterwards the buffers hold exactly the rows of
 * core_idx_new, in slot_neuron's order, which the decode entry points accept as they are (the
 * FFN sums over the rows in any order).
 *   workspace  device, at least coreinfer_update_core_set_workspace_bytes(d_ff, K).
 * Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE, CUDA. */
size_t coreinfer_update_core_set_workspace_bytes(int32_t d_ff, int32_t K);
coreinfer_status coreinfer_update_core_set(const void* w_up, const void* w_gate, const void* w_down,
                                           const void* b_up, coreinfer_dtype dtype,
                                           int32_t d_model, int32_t d_ff,
                                           int32_t* slot_neuron, const int32_t* core_idx_new, int32_t K,
                                           void* w_up_c, void* w_gate_c, void* w_downT_c, void* b_up_c,
                                           int32_t* n_changed_out,
                                           void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ------------------------------------------------------------------ (5) --
 * Pre-fill activations on the tensor cores: the [T, d_ff] tensor A that Definition 1 is
 * applied to, produced the way the method obtains it -- as the intermediate result of the dense
 * pre-fill pass (Section 4.2, Fig. 1) -- without the down projection:
 *   RELU:        A = max(X W_up^T + b_up, 0)        RELU_GATED:  A = max(X W_gate^T, 0) * (X W_up^T)
 * bf16 or fp16 inputs, exact products, fp32 accumulation (tcgen05.mma into tensor memory); the
 * output is fp32 (the precision the method keeps activations in, Section 5 "Models") or, rounded
 * to nearest even once after the activation, bf16 / fp16 for half the bytes.
 * The summation order differs from coreinfer_ffn_dense_ref's, so the two agree to fp32 rounding
 * (1e-4 relative), not bit for bit; selection is exact on whichever tensor it is given.
 *
 *   x        device [T, d_model] bf16            w_up   device [d_ff, d_model] bf16
 *   w_gate   device [d_ff, d_model] bf16 or NULL (NULL iff RELU)
 *   b_up     device [d_ff] bf16 or NULL (RELU only)
 *   act_out  device out [T, d_ff] of act_dtype with row stride ld_act elements (ld_act >= d_ff and a
 *            multiple of 4 for fp32, of 8 for bf16 / fp16: the layout coreinfer_select_core takes)
 *   workspace  device, at least coreinfer_prefill_activations_workspace_bytes(); its first word is
 *              a status word readable with coreinfer_workspace_status.
 * d_model must be a multiple of 8.  Any T and d_ff (edges are zero-filled and masked).
 * Errors: INVALID_ARG, UNSUPPORTED (fp32 inputs: use coreinfer_ffn_dense_ref), WORKSPACE, CUDA. */
size_t coreinfer_prefill_activations_workspace_bytes(void);

coreinfer_status coreinfer_prefill_activations(const void* x, int32_t T, coreinfer_dtype dtype,
                                               coreinfer_ffn_kind kind, int32_t d_model, int32_t d_ff,
                                               const void* w_up, const void* w_gate, const void* b_up,
                                               void* act_out, coreinfer_dtype act_dtype, int64_t ld_act,
                                               void* workspace, size_t workspace_bytes,
                                               void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* COREINFER_H_ */
