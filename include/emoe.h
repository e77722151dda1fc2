/*
 * emoe — sparse MoE layer forward on per-expert mixed-bitwidth (INT2/INT4/INT8) packed
 * weights, for NVIDIA B200 (sm_100a).  C ABI.
 *
 * Method: EdgeMoE (arXiv 2308.14352).  Section 3.2 stores every expert at its own
 * bitwidth with channel-wise linear quantisation and a float16 scale channel, and
 * decompresses (w~ = q * s) before use; Sections 1 and 2.1 define the layer: a router
 * sends each token to its Top-K experts, each expert an independent FFN.  This library
 * computes the same layer but forms q * s in registers: dequantised weights are never
 * written to memory.
 *
 * Conventions
 *   - Every function returns an int status: EMOE_OK (0) or a negative EMOE_ERR_* code.
 *     No exceptions, no abort, nothing printed.
 *   - Pointers are DEVICE pointers unless the parameter name starts with `host_`.
 *     The library never takes ownership of caller memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     Work is enqueued asynchronously; argument errors are reported synchronously,
 *     before anything is enqueued.
 *   - A context belongs to one device and must be used by one host thread at a time.
 *     Calls that share a context share its workspace: they must be ordered on the GPU
 *     (same stream, or explicit dependencies).
 *   - Matrices: an expert matrix has N output channels (rows) and K inputs (columns).
 *     ReLU experts:   m = 0  W_in [d_ff][d_model],  m = 1  W_out [d_model][d_ff].
 *     SwiGLU experts: m = 0  w1 [d_ff][d_model], m = 1  w3 [d_ff][d_model],
 *                     m = 2  w2 [d_model][d_ff].
 *
 * Storage format of a packed matrix (part of the ABI; Section 3.2 leaves it open)
 *   qmax(b) = 2^(b-1) - 1.  Per output channel n and per group g of `group` consecutive
 *   inputs (group = 0: the whole row):
 *       amax  = max |w|,   s32 = amax / qmax (IEEE fp32 division),
 *       s     = s32, or s32 rounded to fp16 (nearest even) when scale_dtype = F16,
 *       q     = clamp(round_half_even(w / s), -qmax, qmax)   (fp32 division by the
 *               STORED scale; q = 0 when s = 0).
 *   Codes: b-bit two's-complement fields; element k of row n sits at bit offset
 *   (k*b) mod 8 of byte n*(K*b/8) + (k*b)/8 (low bits first).  Scales: [N][K/group]
 *   row-major in scale_dtype.
 */
#ifndef EMOE_H_
#define EMOE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* status codes */
#define EMOE_OK 0
#define EMOE_ERR_INVALID_ARG (-1)  /* null pointer, non-positive size, top_k > E, group does not divide K ... */
#define EMOE_ERR_UNSUPPORTED (-2)  /* bits not in {2,4,8}, unknown enum value, shape outside the kernels' limits */
#define EMOE_ERR_ALIGNMENT (-3)    /* a pointer or row size is not 16-byte aligned */
#define EMOE_ERR_WORKSPACE (-4)    /* the context's workspace is too small for this call */
#define EMOE_ERR_CUDA (-5)         /* a CUDA call failed; emoe_last_cuda_error() gives its code */
#define EMOE_ERR_DEVICE_CHECK (-6) /* a kernel found inconsistent data (e.g. an expert id out of range) */
#define EMOE_ERR_CACHE_FULL (-7)   /* every slot of the expert cache is in use by an unfinished call */
#define EMOE_ERR_TIMEOUT (-8)      /* a bounded wait inside a kernel ran out; the kernel gave up and returned */
#define EMOE_ERR_RANGE (-9)        /* a value left the fp16 range of the selected kernel's operands (see emoe_moe_forward) */

/* enums (plain ints in the ABI) */
#define EMOE_DTYPE_F32 0
#define EMOE_DTYPE_F16 1
#define EMOE_DTYPE_BF16 2
#define EMOE_ACT_RELU 0
#define EMOE_ACT_SWIGLU 1
#define EMOE_GATE_SOFTMAX 0        /* gate = softmax probability of the pick over all experts */
#define EMOE_GATE_SOFTMAX_RENORM 1 /* gate = that probability / sum over the token's K picks */

#define EMOE_RANGE_SYMMETRIC 0 /* codes -qmax .. qmax, qmax = 2^(b-1) - 1 (the storage format above) */
#define EMOE_RANGE_FULL 1      /* every code of the field: -2^(b-1) .. 2^(b-1) - 1, scale = amax / 2^(b-1) */

#define EMOE_MAX_EXPERTS 256
#define EMOE_MAX_TOP_K 8

typedef struct emoe_ctx emoe_ctx;

/* One expert of a layer: its bitwidth and DEVICE pointers to its packed matrices and
 * scale channels (Section 3.2: experts of one layer may differ in bitwidth).
 * ReLU uses entries 0..1, SwiGLU 0..2 (order as listed above).  Packed matrices must be
 * 16-byte aligned, scale channels 4-byte aligned (whatever their type). */
typedef struct emoe_expert {
  int32_t bits; /* 2, 4 or 8 */
  int32_t reserved;
  const void* packed[3];
  const void* scales[3];
} emoe_expert;

/* Static description of a layer. */
typedef struct emoe_layer_desc {
  int32_t d_model;
  int32_t d_ff;
  int32_t n_experts;   /* 1 .. EMOE_MAX_EXPERTS */
  int32_t top_k;       /* 1 .. min(n_experts, EMOE_MAX_TOP_K) */
  int32_t act;         /* EMOE_ACT_* */
  int32_t gate_mode;   /* EMOE_GATE_* */
  int32_t group;       /* 0 = one scale per output channel, else inputs per scale */
  int32_t scale_dtype; /* EMOE_DTYPE_F32 | EMOE_DTYPE_F16 */
  int32_t act_dtype;   /* EMOE_DTYPE_F32 | EMOE_DTYPE_BF16: type of x and of the hidden vector */
} emoe_layer_desc;

/* ---- context ------------------------------------------------------------------------ */

/* Creates a context on `device` owning `workspace_bytes` of device scratch (intermediate
 * results of a forward call: the paper's "working buffer", Section 3.1).  Returns NULL and
 * sets *status on failure.  This is the only call (with emoe_destroy) that allocates or
 * frees device memory. */
emoe_ctx* emoe_create(int device, size_t workspace_bytes, int* status);
int emoe_destroy(emoe_ctx* ctx);

/* Scratch that forward calls over at most T tokens need; pass the maximum over the layer
 * descriptions you use to emoe_create.  Returns 0 for an invalid description. */
size_t emoe_workspace_bytes(const emoe_layer_desc* desc, int T);

/* CUDA error code of the last failed CUDA call on this context (0 if none). */
int emoe_last_cuda_error(const emoe_ctx* ctx);

/* Reads (and clears) the device-side check word: EMOE_OK; EMOE_ERR_TIMEOUT if a bounded wait
 * inside a kernel of an earlier call ran out (the kernel gave up and returned; results of that
 * call are undefined, the context stays usable); else EMOE_ERR_DEVICE_CHECK if a kernel met
 * inconsistent data (an expert id out of range); else EMOE_ERR_RANGE (see emoe_moe_forward:
 * "Range").  Synchronises `stream`. */
int emoe_device_status(emoe_ctx* ctx, void* stream);

const char* emoe_status_string(int status);

/* ---- sizes -------------------------------------------------------------------------- */

size_t emoe_packed_bytes(int N, int K, int bits);                   /* N*K*bits/8, 0 if invalid */
size_t emoe_scales_bytes(int N, int K, int group, int scale_dtype); /* N*(K/group)*sizeof, 0 if invalid */

/* ---- Section 3.2: expert-wise quantisation ------------------------------------------- */

/* Quantises and packs one matrix W[N][K] (fp32, row-major, rows = output channels) to
 * `bits` in the storage format described at the top of this file.
 *   group: 0 or a divisor of K; the scale run (group, or K when group = 0) must be a multiple
 *   of 4 inputs.
 *   out_packed: emoe_packed_bytes(N,K,bits) bytes; out_scales: emoe_scales_bytes(...).
 *   W and out_packed must be 16-byte aligned, out_scales 4-byte aligned.
 * Bit-exact with the definition: IEEE division and round-half-even, no fast-math. */
int emoe_pack_expert(emoe_ctx* ctx, const float* W, int N, int K, int bits, int group, int scale_dtype,
                     void* out_packed, void* out_scales, void* stream);

/* Moves one stored matrix [N][K] from `bits_in` to `bits_out` without the fp32 original
 * (Section 3.2, "Choosing the bitwidth": the selection puts the least important experts at
 * the lower width and widens or narrows the set until the loss target is met; an expert that
 * changes its width is re-quantised).  Each weight is decompressed in registers
 * (w~ = q * s, rounded once to fp32; exact with fp16 scales) and quantised again with the
 * arithmetic of emoe_pack_expert: the result equals emoe_pack_expert on the decompressed matrix,
 * bit for bit.  Input and output use the same `group` and `scale_dtype`; any pair of widths is
 * allowed (the same width reproduces the input when the scales are fp16).
 *   in_packed / in_scales: device buffers in the storage format, emoe_packed_bytes(N,K,bits_in)
 *   and emoe_scales_bytes(...) bytes; out_packed / out_scales: emoe_packed_bytes(N,K,bits_out)
 *   and emoe_scales_bytes(...) bytes, owned by the caller, distinct from the inputs (not in
 *   place).  Packed buffers 16-byte aligned, scale buffers 4-byte aligned.
 * Errors as for emoe_pack_expert; asynchronous on `stream`. */
int emoe_requantize_expert(emoe_ctx* ctx, const void* in_packed, const void* in_scales, int N, int K, int bits_in,
                           int bits_out, int group, int scale_dtype, void* out_packed, void* out_scales,
                           void* stream);

/* The same two calls with the reading of "the range expressible by the bitwidth" (Section 3.2)
 * as an argument.  EMOE_RANGE_SYMMETRIC is the storage format at the top of this file (what the
 * calls above use).  EMOE_RANGE_FULL uses every code of the two's-complement field:
 *       s32 = amax / 2^(b-1),  q = clamp(round_half_even(w / s), -2^(b-1), 2^(b-1) - 1),
 * so that INT2 has four levels (-2, -1, 0, 1) instead of three; a weight equal to +amax is
 * clamped to the largest positive code.  Storage layout, scale channel and every forward call are
 * unchanged: the expert kernels decode whole two's-complement fields.  Everything else as above;
 * an unknown range_mode returns EMOE_ERR_UNSUPPORTED. */
int emoe_pack_expert_mode(emoe_ctx* ctx, const float* W, int N, int K, int bits, int group, int scale_dtype,
                          int range_mode, void* out_packed, void* out_scales, void* stream);
int emoe_requantize_expert_mode(emoe_ctx* ctx, const void* in_packed, const void* in_scales, int N, int K, int bits_in,
                                int bits_out, int group, int scale_dtype, int range_mode, void* out_packed,
                                void* out_scales, void* stream);

/* ---- Sections 1, 2.1: router and Top-K gating ----------------------------------------- */

/* z[t][e] = sum_i x[t][i] * router_W[i][e] (+ bias), p = softmax(z) over all experts; the
 * top_k largest logits are selected (ties: lower expert index) and listed in descending
 * order of logit.
 *   x: [T][d] in act_dtype (F32 or BF16); router_W: [d][E] fp32;
 *   router_bias: NULL, or fp32 with bias[t*bias_token_stride + e]
 *                (bias_token_stride = 0: one vector for all tokens; = E: one per token);
 *   out_ids [T][top_k] int32, out_gates [T][top_k] fp32, out_logits NULL or [T][E] fp32.
 * Accumulation is fp32. */
int emoe_router_topk(emoe_ctx* ctx, const void* x, int act_dtype, int T, int d, const float* router_W,
                     const float* router_bias, int bias_token_stride, int E, int top_k, int gate_mode,
                     int32_t* out_ids, float* out_gates, float* out_logits, void* stream);

/* Token -> expert permutation: stable counting sort of the pair indices p = t*top_k + j by
 * expert id.  out_counts [E], out_off [E+1] (exclusive prefix sum), out_perm [n_pairs]
 * (pair indices in expert order, increasing inside an expert), out_slot_of_pair [n_pairs]
 * (the inverse: position of pair p in out_perm; may be NULL).  Ids outside [0,E) set the
 * device check word and are dropped. */
int emoe_permute(emoe_ctx* ctx, const int32_t* ids, int n_pairs, int E, int32_t* out_counts, int32_t* out_off,
                 int32_t* out_perm, int32_t* out_slot_of_pair, void* stream);

/* ---- the layer ------------------------------------------------------------------------ */

/* Full layer forward (Sections 1, 2.1 on the Section 3.2 storage):
 * router -> Top-K -> permutation -> expert FFNs on packed weights -> weighted combine.
 *   ReLU:   h = max(0, x W~in^T),            o = h W~out^T
 *   SwiGLU: h = silu(x W~1^T) * (x W~3^T),   o = h W~2^T
 *   y[t] = sum_j gate[t][j] * o[pair (t,j)],  W~[n][k] = q[n][k] * s[n][k/group].
 * With BF16 activations the hidden vector h is rounded once to bf16; with F32 it stays
 * fp32.  Only the distinct activated experts' weights are read.
 *   x [T][d_model] in desc->act_dtype; y [T][d_model] fp32.
 *   host_experts: HOST array of desc->n_experts entries holding DEVICE pointers; the
 *     library keeps a device copy per distinct table (by content), uploaded on `stream`
 *     the first time a table is seen.
 *   out_ids / out_gates ([T][top_k]) and out_perm ([T*top_k]) are optional (NULL) copies
 *   of the routing decisions.
 * Range: with BF16 activations the default tensor-core kernels carry x and the hidden vector as
 * fp16 operands (exact for bf16 values up to 65504 in magnitude) and the many-token grouped GEMM also
 * rounds q * s to fp16.  A value beyond 65504 is saturated, and a scale below 2^-14 in the grouped
 * GEMM loses bits: both set a flag that emoe_device_status reports as EMOE_ERR_RANGE, and y is then
 * not within the usual bound of the definition.  Kernel family 6 (emoe_set_ffn_path) and the
 * CUDA-core family 1 have no such limit: they follow the full bf16 exponent range.
 * Shape limits: d_model and d_ff multiples of 32 with K*bits/8 a multiple of 16 for every
 * matrix; group 0 or a multiple of 32 (INT8), 32 (INT4), 64 (INT2) dividing K.
 * Uses the context workspace (emoe_workspace_bytes). */
int emoe_moe_forward(emoe_ctx* ctx, const emoe_layer_desc* desc, const void* x, int T, const float* router_W,
                     const float* router_bias, int bias_token_stride, const emoe_expert* host_experts, float* y,
                     int32_t* out_ids, float* out_gates, int32_t* out_perm, void* stream);

/* Same layer with the routing decisions given (ids [T][top_k] in [0,E), gates [T][top_k]):
 * runs the permutation, the expert FFNs and the combine only. */
int emoe_moe_forward_routed(emoe_ctx* ctx, const emoe_layer_desc* desc, const void* x, int T, const int32_t* ids,
                            const float* gates, const emoe_expert* host_experts, float* y, int32_t* out_perm,
                            void* stream);

/* Selects the expert-FFN kernel family: 0 = automatic (default), 1 = the CUDA-core grouped
 * GEMV, 2 = the tensor-core kernel with register-staged weight loads, 3 = the fp16 mma.sync
 * kernel with the TMA-staged weight pipeline (what 0 picks for decode batches), 4 = the tcgen05
 * grouped GEMM (fp16 operands; meant for many tokens per expert), 5 = 3 and 4 in one call: experts
 * with at most 32 tokens take the streaming kernel, the others the grouped GEMM (what 0 picks for
 * large batches), 6 = the weight-streaming kernel on 8-bit integer tcgen05 operands with block-scaled
 * integer activations (no fp16 range limit; at present slower than 3).
 * 2 to 6 fail with EMOE_ERR_UNSUPPORTED in forward calls whose shape they do not take.  For tests
 * and measurements. */
int emoe_set_ffn_path(emoe_ctx* ctx, int path);

/* Every wait inside the weight-streaming kernel (on a pipeline stage, on tensor memory, on the
 * completion of an expert's hidden vectors) is bounded: after `polls` unsuccessful polls the
 * kernel records the failure, lets its copies in flight land, releases what it holds and
 * returns; emoe_device_status then reports EMOE_ERR_TIMEOUT and the context stays usable.  This
 * is the library's form of failure detection (the paper's only failure path is a mispredicted
 * preload, Section 3.3, which is corrected by loading the right expert).  polls = 0 restores the
 * default (about 0.2 s).  Applies to the forward calls that follow. */
int emoe_set_wait_limit(emoe_ctx* ctx, unsigned polls);

/* Test hook for the above: the second projection of every expert waits for `extra` more
 * completions of its first projection than will ever be counted, so that its bounded wait runs
 * out; the grid-wide wait of the one-launch routing kernel (emoe_set_fused_routing) likewise
 * waits for `extra` more arrivals than the grid has CTAs.  0 (the default) in any real use.  No
 * counterpart in the paper. */
int emoe_debug_expect_extra_completions(emoe_ctx* ctx, int extra);

/* Programmatic dependent launch along the kernels of a forward call (on by default): each
 * kernel may start its prologue while the one in front drains.  Results are identical either
 * way; switch it off to compare timings or when a tool in use does not support the attribute. */
int emoe_set_dependent_launch(emoe_ctx* ctx, int enabled);

/* Both projections of the activated experts' FFNs (paper Section 2.1: an expert is one FFN) in a
 * single launch of the weight-streaming kernel (on by default): an expert's second projection
 * starts as soon as all of its hidden vectors are written, instead of after the first
 * projection of every expert.  Results are identical either way; switch it off to run the two
 * projections as two launches (to compare timings, or to time them separately). */
int emoe_set_fused_projections(emoe_ctx* ctx, int enabled);

/* Router, Top-K, permutation, scatter and work plan (Section 2.1: every token goes to its Top-K
 * experts) in ONE launch for batches of at most 1024 token-expert pairs on the weight-streaming
 * kernels: one CTA per token; the CTAs meet at a bounded grid-wide wait on an arrival counter
 * (all of them are resident: the library checks the grid against the device's capacity), after
 * which each places its own pairs.  A forward call is then three launches.  Off by default: as
 * measured, the chain of dependent launches is a little faster than the grid-wide wait.  ids,
 * gates, permutation and outputs are identical either way.  A wait that runs out reports
 * EMOE_ERR_TIMEOUT through emoe_device_status (limit: emoe_set_wait_limit). */
int emoe_set_fused_routing(emoe_ctx* ctx, int enabled);

/* The whole layer (Sections 2.1 and 3.2: router, Top-K, the activated experts' FFNs on their
 * packed codes, gate-weighted sum) in ONE launch, for calls of at most 16 token-expert pairs on
 * layers whose matrices hold at most 8 Mi weights each (single-request decoding, the paper's
 * target, on a Switch-base-sized layer): such a call is a few microseconds of work and the chain
 * of dependent launches is most of its time.  One resident grid; a few CTAs per token form the
 * router product, every CTA makes the picks from it, all CTAs then share the rows of the first projection (one warp per row, packed codes decoded in
 * registers, fp32 accumulation), meet at a bounded grid-wide wait, and share the rows of the
 * second projection, whose sums over the token's experts are formed in a fixed order.  Applies
 * to emoe_moe_forward and emoe_moe_forward_routed when no kernel family was forced
 * (emoe_set_ffn_path 0); calls outside the limits run as before.  The router product is summed
 * in slices of the d_model axis here, so logits and gates agree with the other paths' to fp32
 * rounding (picks can differ only between experts whose logits agree that closely), and y
 * within the accumulation-order difference (fp32 sums of the same products).  A wait that runs out reports EMOE_ERR_TIMEOUT through
 * emoe_device_status (limit: emoe_set_wait_limit).
 * mode 0: never; 1: every call inside the limits; 2 (the default): calls of up to eight pairs,
 * where it was measured faster than the chain of launches (1.8 x for one pair, 1.5 x for two to
 * four on a Switch-base-sized layer, 1.25 x for eight; for sixteen the chain wins).  Other values:
 * EMOE_ERR_INVALID_ARG. */
int emoe_set_fused_layer(emoe_ctx* ctx, int mode);

/* Number of kernels the last emoe_moe_forward / emoe_moe_forward_routed call on this context
 * enqueued (router + Top-K, permutation, scatter, expert FFNs, combine: Sections 2.1 and 3.2 name
 * the steps, the count depends on the kernel family the shape takes).  0 before the first call. */
int emoe_kernels_last_forward(const emoe_ctx* ctx);

/* The routed layer forward for callers that cannot allocate device memory (the paper has no
 * counterpart: it is an addition for hosts such as a framework that owns the whole device
 * heap, a plug-in whose memory pool is fixed at start-up, or a latency-critical loop in which
 * an allocation, which may synchronise the device, is not acceptable).  Such callers cannot
 * have a context, because emoe_create allocates; this call needs none.  It computes exactly
 * what emoe_moe_forward_routed computes, with its intermediate buffers in a fixed 8 MiB array
 * that is part of the library image on every GPU that loads it (held until the process
 * exits).  It calls no cudaMalloc / cudaFree and no allocating library routine.
 *   Limits: T * top_k <= 64, and the intermediates of the call must fit the 8 MiB array
 *   (roughly: 64 * (2*d_model + 2*d_ff + 4*d_model*splits) bytes); otherwise the call
 *   returns EMOE_ERR_WORKSPACE and does nothing.  Other argument rules as for
 *   emoe_moe_forward_routed.
 *   First call on a device: looks up the array's device address (with that device made
 *   current).  Make this first call outside any stream capture.  Every call only enqueues
 *   kernels (the expert table travels as launch parameters, no host buffer is referenced after
 *   the call returns).
 *   Expert ids outside [0, n_experts) are dropped from the result and set a check word inside
 *   the array; emoe_static_device_status reads it.
 *   Sharing: every call on a device uses the same array, which keeps the previous call's
 *   contents (the call clears what has to start at zero itself).  Two calls whose GPU work
 *   overlaps (different streams without a dependency, or different host threads) race on it:
 *   order them.
 * `device` is the CUDA device ordinal; the other parameters are those of
 * emoe_moe_forward_routed. */
int emoe_moe_forward_routed_static(int device, const emoe_layer_desc* desc, const void* x, int T, const int32_t* ids,
                                   const float* gates, const emoe_expert* host_experts, float* y, void* stream);

/* Status of the calls of emoe_moe_forward_routed_static enqueued so far on `device` (the paper
 * has no counterpart): synchronises `stream`, then returns EMOE_OK, EMOE_ERR_DEVICE_CHECK (an
 * expert id was out of range) or EMOE_ERR_TIMEOUT.  The word is cleared by the next forward call,
 * not by this one.  Allocates nothing. */
int emoe_static_device_status(int device, void* stream);

/* Measurement aid (Section 4 of the paper times compute and loading separately; here the
 * expert-FFN kernels are the part bound by weight streaming).  While enabled, every forward
 * call records CUDA events on its stream around the first-projection and second-projection
 * expert kernels.  emoe_read_timing waits for the recorded events, returns the summed device
 * time of each projection (milliseconds) and the number of forward calls covered, and clears
 * the record.  Where both projections run as one launch (see emoe_set_fused_projections) the
 * whole time is returned as the first value and the second is 0.  Off by default; not for use
 * during stream capture. */
int emoe_set_timing(emoe_ctx* ctx, int enabled);
int emoe_read_timing(emoe_ctx* ctx, float* out_first_ms, float* out_second_ms, int* out_calls);

/* ---- expert cache and prefetch ------------------------------------------------------------
 * Section 3.3 of the paper keeps the experts in slow storage, holds a buffer of fixed size in
 * fast memory, preloads the experts it predicts from the previous layers' activations while the
 * current layer computes, and evicts by activation frequency and layer distance.  Here slow
 * storage is PINNED HOST memory (owned by the caller, registered once), fast memory is
 * `n_slots` equal HBM slots owned by the context, loads are asynchronous copies on a copy
 * stream, and the compute stream is made to wait (on the device, never on the host) for a
 * slot's contents.  Typical layer:  ids = router (emoe_router_topk, read back);
 * emoe_prefetch_experts(predicted experts of the next layer);  emoe_cache_acquire(ids) -> device
 * pointers for the expert table;  emoe_moe_forward_routed;  emoe_cache_release(ids). */

#define EMOE_EVICT_FORWARD 0 /* score -f/D, D = layers until the expert's layer runs again: (i - I) mod S */
#define EMOE_EVICT_PRINTED 1 /* score -f/D with D = (S - i + I) mod S as the formula is printed */
#define EMOE_EVICT_LRU 2     /* least recently used */
#define EMOE_EVICT_LFU 3     /* fewest activations so far; ties: loaded earliest */
#define EMOE_EVICT_FIFO 4    /* loaded earliest */

typedef struct emoe_cache_stats {
  int64_t hits;               /* acquire found the expert in a slot (loaded or loading) */
  int64_t misses;             /* acquire had to start the load itself */
  int64_t prefetch_hits;      /* hits on an expert whose load a prefetch started and nobody used since */
  int64_t prefetched;         /* loads started by prefetch calls */
  int64_t prefetch_redundant; /* prefetch requests for experts already in a slot */
  int64_t prefetch_refused;   /* prefetch requests dropped because every slot was in use */
  int64_t evictions;
  int64_t bytes_copied;       /* host -> device bytes of all loads started */
  int64_t exposed_copy_ns;    /* device time the compute stream stood still inside emoe_cache_acquire, waiting for
                                 slot contents (loading not hidden under compute: Section 3.3, the pipeline's
                                 failed-prediction case); counted only while emoe_cache_set_timing is on */
  int64_t timed_acquires;     /* acquire calls that contributed to exposed_copy_ns */
} emoe_cache_stats;

/* Allocates the cache of a context: n_slots x slot_bytes of device memory and two events per
 * slot (the only allocating call besides emoe_create; freed by emoe_destroy).  n_layers = S of
 * the eviction score; policy = EMOE_EVICT_*. */
int emoe_cache_create(emoe_ctx* ctx, int n_slots, size_t slot_bytes, int n_layers, int policy);

/* Registers an expert of layer `layer` under a caller-chosen id.  host_pinned_packed[3] /
 * host_pinned_scales[3]: its matrices in pinned host memory (null with 0 bytes for an absent
 * third matrix), bytes[6] their sizes (packed 0..2, then scales 0..2).  The memory stays the
 * caller's and must outlive the cache.  Packed matrices must be 16-byte aligned; inside a slot
 * every matrix starts on a 256-byte boundary. */
int emoe_register_expert(emoe_ctx* ctx, int64_t id, int layer, int bits, const void* const* host_pinned_packed,
                         const void* const* host_pinned_scales, const size_t* bytes);

/* Starts loading the listed experts (most likely first) on copy_stream unless they are in a slot
 * already; evicts by the policy; drops requests when every slot is in use.  current_layer = I of
 * the score.  Never blocks the host and never makes the compute stream wait. */
int emoe_prefetch_experts(emoe_ctx* ctx, const int64_t* ids, int n, int current_layer, void* copy_stream);

/* The listed experts are about to be used on compute_stream: experts not in a slot are loaded
 * now (on copy_stream), compute_stream waits on the device for each slot's contents, the slots
 * are protected from eviction until emoe_cache_release, activation counts go up by one, and
 * out_experts[i] receives the device pointers of ids[i] (valid until the release).
 * EMOE_ERR_CACHE_FULL if a load finds every slot protected. */
int emoe_cache_acquire(emoe_ctx* ctx, const int64_t* ids, int n, int current_layer, void* compute_stream,
                       void* copy_stream, emoe_expert* out_experts);

/* Call after the last kernel that reads the experts has been enqueued on compute_stream: a later
 * load into one of these slots waits (on the device) until that point of the stream. */
int emoe_cache_release(emoe_ctx* ctx, const int64_t* ids, int n, void* compute_stream);

/* Slot that holds the expert, -1 if none. */
int emoe_cache_slot_of(emoe_ctx* ctx, int64_t id);
int emoe_cache_get_stats(emoe_ctx* ctx, emoe_cache_stats* out);

/* Exposed-copy accounting (the paper reports compute and loading time separately, Section 4):
 * while enabled, every emoe_cache_acquire records one CUDA event on compute_stream in front of
 * its waits and one behind them; emoe_cache_get_stats waits for the recorded pairs, adds their
 * distances to exposed_copy_ns and clears the record.  With every expert resident the waits return
 * at once and the sum stays near zero; it can never exceed the time of loading on demand.  Off by
 * default; not for use during stream capture. */
int emoe_cache_set_timing(emoe_ctx* ctx, int enabled);

/* Tokens per expert of the most recent forward call on this context (the "tokens per expert"
 * counter): copies the call's per-expert pair counts (n_experts int32, host memory) after
 * synchronising `stream`.  EMOE_ERR_INVALID_ARG before the first forward call or when n_experts
 * differs from that call's. */
int emoe_last_expert_counts(emoe_ctx* ctx, int32_t* out_counts, int n_experts, void* stream);

/* The cache's bookkeeping alone, without a device (same code as behind the calls above): for
 * checking slot assignment, eviction order and counters on a host without a GPU.
 * emoe_policy_prefetch returns the slot a load would go to (-1: none), emoe_policy_acquire the
 * slot (-1: every slot protected) with *loaded = 1 on a miss; *evicted_id = id that left, or -1. */
typedef struct emoe_policy emoe_policy;
emoe_policy* emoe_policy_create(int n_slots, int n_layers, int policy);
void emoe_policy_destroy(emoe_policy* p);
int emoe_policy_register(emoe_policy* p, int64_t id, int layer, int64_t bytes);
int emoe_policy_prefetch(emoe_policy* p, int64_t id, int current_layer, int64_t* evicted_id);
int emoe_policy_acquire(emoe_policy* p, int64_t id, int current_layer, int* loaded, int64_t* evicted_id);
int emoe_policy_release(emoe_policy* p, int64_t id);
int emoe_policy_get_stats(emoe_policy* p, emoe_cache_stats* out);

/* Ranks the experts of the next layer from a first-order layer-transition prior (Section 3.3,
 * "Estimating expert activation a priori", with one previous layer as key): prior is a host
 * array [n_experts][n_experts], row p = distribution of the next layer's expert given pick p;
 * score[e] = sum over prev_ids of prior[p][e]; out_order (host, n_experts entries) lists the
 * experts by descending score, ties by lower index. */
int emoe_rank_experts(const float* prior, int n_experts, const int32_t* prev_ids, int n_prev, int32_t* out_order);

/* The statistical profile of Section 3.3 ("Opportunistic preloading") with the key the paper
 * names: the activation status of the TWO previous MoE layers.
 * emoe_build_profile2 (the offline phase): trace is a host array [n_tokens][n_layers][top_k] of
 * the experts each token activated; out_prior2 (host, [n_layers][E][E][E] floats, E = n_experts)
 * receives for every layer n >= 2 and key (a, b) the share of the tokens with a active in layer
 * n-2 and b active in layer n-1 that activated e in layer n (with top_k > 1 every (a, b) pair of
 * the two layers' picks is a key; a row sums to top_k); keys never seen get 1/E; layers 0 and 1
 * get zeros.  An id outside [0, E) returns EMOE_ERR_INVALID_ARG.
 * emoe_rank_experts2 (the online query): prior2_layer = the [E][E][E] block of the layer to be
 * predicted; score[e] = sum over a in prev2_ids, b in prev1_ids of prior2_layer[a][b][e];
 * out_order lists the experts by descending score, ties by lower index. */
int emoe_build_profile2(const int32_t* trace, int n_tokens, int n_layers, int top_k, int n_experts, float* out_prior2);
int emoe_rank_experts2(const float* prior2_layer, int n_experts, const int32_t* prev2_ids, int n_prev2,
                       const int32_t* prev1_ids, int n_prev1, int32_t* out_order);

#ifdef __cplusplus
}
#endif
#endif /* EMOE_H_ */
