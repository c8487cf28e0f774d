/*
 * aflex.h -- C ABI of the B200-native A/F decode-layer hot path.
 *
 * One decoder-layer decode step is split into an Attention side (A) and an FFN
 * side (F) that exchange hidden states once per layer (paper Section 4.3,
 * "Placement-aware A/F Data Path": the Attention group sends its outputs to the
 * FFN group, which returns the hidden states) and run as M interleaved
 * microbatches (Section 4.3, "Interleaved A/F Pipeline", Eq. 2).  The paper
 * delegates the operators' arithmetic to its serving engine; the definitions
 * implemented here are the standard ones and are restated at each entry point.
 *
 * Conventions (all entry points)
 *  - Return value: aflex_status; 0 = OK.  Nothing throws, aborts or traps.
 *  - Tensor pointers are DEVICE pointers unless the comment says "host".  They
 *    are borrowed: the caller keeps them alive and unmodified until the work
 *    enqueued by the call has finished on the stream; the library never frees
 *    or reallocates them.  All base pointers must be 16-byte aligned.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *    stream).  Work is enqueued asynchronously; no call synchronises the
 *    device unless its comment says so.
 *  - bf16 tensors are raw 16-bit patterns, row-major, innermost dimension last.
 *    Every fp32 -> bf16 store rounds to nearest even.
 *  - Arguments are validated on the host before anything is enqueued: on a
 *    non-OK return nothing was launched.  Shapes outside the supported
 *    envelope return AFLEX_ERR_UNSUPPORTED (there is no slow path and no CPU
 *    fallback).
 *  - An aflex_ctx owns a device workspace, two internal streams and events
 *    for aflex_layer_step, and a device status word.  A ctx is bound to one
 *    device and must be used by one host thread at a time.  Calls that use the
 *    same ctx must be stream-ordered with respect to each other (they share the
 *    workspace); aflex_layer_step orders its own internal streams.
 *  - Kernels are launched with programmatic stream serialization and read some
 *    INPUT tensors (KV cache, page table, lengths, weights - not activations such
 *    as q or x) before the grid dependency resolves.  This is invisible to ordinary callers (a preceding
 *    kernel, copy or event wait in the stream completes first, as usual); only a
 *    caller's own kernel that releases its dependents early
 *    (cudaTriggerProgrammaticLaunchCompletion) must not be the producer of those
 *    inputs.  Outputs and scratch are touched only after the dependency resolves.
 *  - The enqueueing calls (aflex_attn_decode, aflex_ffn_*, aflex_layer_step, aflex_decoder_layers, ...) can be
 *    captured into a CUDA graph on `stream` after one un-captured warm-up call with the same shapes (the first
 *    call sets kernel attributes and fills the host-side tensor-map cache); with a microbatch depth >= 2 the
 *    ctx's internal streams are forked from and joined to `stream`, so they become part of the capture.
 *  - Device-side waits are bounded: if one expires the kernel records
 *    AFLEX_ERR_TIMEOUT in the ctx status word and exits cleanly; read it with
 *    aflex_get_device_status.
 *
 * Supported envelope: head_dim in {64,128}; page_size 16; Hq/Hkv in {1,2,4,8};
 * batch >= 1; every seq_len >= 1; hidden, inter and Hq*head_dim multiples of 8;
 * num_experts <= 64 with top_k in {1,2} and top_k <= num_experts.
 */
#ifndef AFLEX_H_
#define AFLEX_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define AFLEX_API __attribute__((visibility("default")))
#else
#define AFLEX_API
#endif

typedef enum {
    AFLEX_OK = 0,
    AFLEX_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, M > batch, ... */
    AFLEX_ERR_UNSUPPORTED = 2, /* valid but outside the supported envelope */
    AFLEX_ERR_WORKSPACE = 3,   /* ctx workspace too small for this call */
    AFLEX_ERR_CUDA = 4,        /* a CUDA runtime/driver call failed (see aflex_last_error) */
    AFLEX_ERR_TIMEOUT = 5,     /* a bounded device-side wait expired */
    AFLEX_ERR_BOUNDS = 6       /* a device-side index check failed (page id / expert id out of range) */
} aflex_status;

typedef struct aflex_ctx aflex_ctx;

/* Static string for a status code. */
AFLEX_API const char* aflex_status_string(aflex_status s);

/* Library version, major*10000 + minor*100 + patch. */
AFLEX_API int aflex_version(void);

/*
 * Create a context on CUDA device `device`.  `workspace_bytes` is the size of
 * the device workspace the ctx allocates (0 = library default, 256 MiB); use
 * aflex_workspace_bytes to size it for a given layer.  Allocates device memory
 * and creates streams/events: call it outside any timed or captured region.
 * *out is owned by the caller and released with aflex_destroy.
 */
AFLEX_API aflex_status aflex_create(aflex_ctx** out, int device, size_t workspace_bytes);

/* Synchronises the ctx's streams, frees everything the ctx owns. NULL is OK. */
AFLEX_API aflex_status aflex_destroy(aflex_ctx* ctx);

/* Host string describing the last non-OK return on this ctx (never NULL). */
AFLEX_API const char* aflex_last_error(const aflex_ctx* ctx);

/*
 * Synchronises `stream`, then returns and clears the device status word:
 * AFLEX_OK, AFLEX_ERR_TIMEOUT or AFLEX_ERR_BOUNDS as raised by kernels
 * enqueued through this ctx.
 */
AFLEX_API aflex_status aflex_get_device_status(aflex_ctx* ctx, void* stream);

/* ---- Attention side -------------------------------------------------------
 *
 * Decode attention (the operator the paper's Sections 1-2 describe as
 * memory-bound on reads of the growing KV cache; one query token per
 * sequence).  For sequence b with n = seq_lens[b] cached tokens and query head
 * h reading KV head g = h / (Hq/Hkv):
 *     s_j  = sm_scale * <q[b,h,:], K_j>            j = 0..n-1
 *     p    = softmax(s)                            (fp32 scores and sums)
 *     out[b,h,:] = sum_j p_j V_j                   -> bf16
 *     lse[b,h]   = max_j s_j + ln sum_j exp(s_j - max)
 * Token j of sequence b is stored in physical page page_table[b][j/16], slot
 * j%16.  No mask (the n cached tokens include the one being decoded), no
 * positional term.  Slots beyond a sequence's length and pages no sequence
 * references may hold anything (including NaN) and do not affect the output.
 * The KV cache is split evenly over persistent CTAs and split sequences are merged in a fixed
 * order; the result is deterministic run to run.
 */
typedef struct {
    int num_q_heads;   /* Hq */
    int num_kv_heads;  /* Hkv, divides Hq */
    int head_dim;      /* D: 64 or 128 */
    int page_size;     /* must be 16 */
    float sm_scale;    /* 0 => 1/sqrt(D) */
} aflex_attn_desc;

typedef struct {
    const void* k_cache;          /* bf16 [num_pages][Hkv][page_size][D] */
    const void* v_cache;          /* bf16 [num_pages][Hkv][page_size][D] */
    int64_t num_pages;            /* pages in each pool; page ids must be in [0, num_pages) */
    const int32_t* page_table;    /* i32 [batch][max_pages_per_seq]; entries past ceil(len/16) are ignored */
    int max_pages_per_seq;        /* row stride of page_table; also bounds every seq_len <= 16*max_pages_per_seq */
    const int32_t* seq_lens;      /* i32 [batch], each in [1, 16*max_pages_per_seq]; a value outside that range is clamped on
                                     the device and reported as AFLEX_ERR_BOUNDS (a sequence clamped to 0 gets no output) */
    const int32_t* seq_lens_host; /* optional HOST copy of seq_lens (validated: each in [1, 16*max_pages_per_seq]); may be NULL */
} aflex_kv;

/*
 * q   bf16 [batch][Hq][D]            (device, read)
 * out bf16 [batch][Hq][D]            (device, written)
 * lse fp32 [batch][Hq] or NULL       (device, written when non-NULL)
 * Uses the ctx workspace for per-CTA partial results (a few MB, independent of batch and context).
 * Errors: INVALID_ARG (null pointers, batch < 1, a host seq_len outside its
 * range), UNSUPPORTED (envelope), WORKSPACE.
 */
AFLEX_API aflex_status aflex_attn_decode(aflex_ctx* ctx, const aflex_attn_desc* desc, const void* q,
                                         const aflex_kv* kv, int batch, void* out, float* lse, void* stream);

/*
 * Decode attention for callers that cannot allocate device memory (no counterpart in the
 * paper: it serves the integration, not the method).
 *
 * Who needs it: a process whose memory pool has already claimed the whole GPU so that any
 * later cudaMalloc fails, a plugin that must stay inside a host application's allocator, or a
 * latency-critical path where an allocation -- an implicit device-wide synchronisation -- is
 * not acceptable.  aflex_create allocates, so such callers cannot hold an aflex_ctx.  This
 * entry point takes no ctx and calls no allocating routine: the kernel's scratch (per-CTA
 * partial results, arrival counters, a status word) is a fixed ~2.7 MB array inside the
 * library's device image, present on every GPU that loads the library until the process
 * exits.  The caller still passes every input and output.
 *
 * Same arguments, layouts and arithmetic as aflex_attn_decode (the split of the work over CTAs
 * differs, so results agree to rounding, not bit for bit).  What the kernel finds wrong while
 * it runs (a length or page id out of range, an expired wait) is read with
 * aflex_attn_decode_static_status below.  Limits of the fixed
 * scratch: batch * num_kv_heads <= 16384 (otherwise AFLEX_ERR_WORKSPACE is returned and
 * nothing is launched) and at most 320 persistent CTAs are used.  Other errors:
 * AFLEX_ERR_INVALID_ARG / AFLEX_ERR_UNSUPPORTED as for aflex_attn_decode, AFLEX_ERR_CUDA.
 * There is no error string (no ctx to keep it in).
 *
 * The first call on a device looks up the scratch array's device address and raises the
 * kernel's shared-memory limit for that device; make that first call with the device
 * current and before any stream capture.  Later calls only enqueue work.
 * All calls share the one array, which keeps the previous call's contents: each call
 * re-zeroes the counters and the status word on `stream` before the kernel.  Two calls
 * that overlap on the GPU (different streams, or different host threads without ordering)
 * race on the scratch and give wrong results: order them on one stream or with events.
 * Not thread-safe on the host for first calls on the same device.
 */
AFLEX_API aflex_status aflex_attn_decode_static(const aflex_attn_desc* desc, const void* q, const aflex_kv* kv,
                                                int batch, void* out, float* lse, void* stream);

/*
 * Device-side status of the calls of aflex_attn_decode_static on the current device (no
 * counterpart in the paper either).  The kernel records what it meets while it runs in a status
 * word of the fixed scratch -- AFLEX_ERR_BOUNDS: a sequence length outside
 * [1, max_pages_per_seq * 16] (clamped; a sequence clamped to 0 gets no output) or a page id
 * outside [0, num_pages) (page 0 is read instead); AFLEX_ERR_TIMEOUT: a bounded wait expired
 * and rows are missing -- and aflex_attn_decode_static's own return value cannot carry it, since
 * the call only enqueues work.  This call copies the word to *host_status on `stream`
 * (one cudaMemcpyAsync, no allocation) and synchronises that stream; pass the stream the
 * attention calls ran on.  Every aflex_attn_decode_static call re-zeroes the word before its
 * kernel, so the value read is that of the last call enqueued before this one.  Returns
 * AFLEX_ERR_INVALID_ARG for a null pointer or when no static call has been made on the current
 * device yet, AFLEX_ERR_CUDA on a runtime error, else AFLEX_OK with *host_status set.
 */
AFLEX_API aflex_status aflex_attn_decode_static_status(int* host_status, void* stream);

/*
 * Prefill (causal) attention: the attention operator of the prefill phase (the paper's "PA" pool; Section 1: in
 * prefill both operators are dominated by matrix multiplications).  Sequence b has n = seq_lens[b] cached tokens,
 * of which the last m = q_offsets[b+1] - q_offsets[b] are being prefilled (m = n: a whole prompt; m < n: a chunk
 * behind an existing context).  Query i (0 <= i < m) sits at position n - m + i and attends to the cached tokens
 * 0 .. n - m + i, itself included:
 *     s_j = sm_scale * <q_i, K_j>,  p = softmax over j <= n - m + i,  out_i = sum_j p_j V_j  -> bf16
 * q, out: bf16 [T][Hq][D] with T = q_offsets[batch], the queries of sequence b at rows q_offsets[b] ..;
 * q_offsets: DEVICE i32 [batch + 1]; q_offsets_host: HOST copy of the same (sizes the launch); kv as for
 * aflex_attn_decode, the K/V of the prefilled tokens already in the cache.  Runs on the tcgen05 tensor cores
 * (fp32 scores and accumulation, P rounded to bf16 before the P V product).  Errors as aflex_attn_decode, plus
 * INVALID_ARG for inconsistent offsets.
 */
AFLEX_API aflex_status aflex_attn_prefill(aflex_ctx* ctx, const aflex_attn_desc* desc, const void* q, const aflex_kv* kv,
                                          int batch, const int32_t* q_offsets, const int32_t* q_offsets_host, void* out,
                                          void* stream);

/* ---- FFN side -------------------------------------------------------------
 *
 * Dense SwiGLU FFN (the decode FFN operator of the paper's Section 1: weight
 * streaming at small batch, tensor-core bound at large batch):
 *     h = silu(x W_gate^T) .* (x W_up^T)     silu(z) = z / (1 + exp(-z))
 *     y = h W_down^T
 * x bf16 [T][H]; w_gate, w_up bf16 [I][H]; w_down bf16 [H][I]; y bf16 [T][H].
 * fp32 accumulation; h is rounded to bf16 once between the two GEMMs.
 * T >= 1; H and I multiples of 8 (otherwise UNSUPPORTED).
 */
AFLEX_API aflex_status aflex_ffn_dense(aflex_ctx* ctx, const void* x, const void* w_gate, const void* w_up,
                                       const void* w_down, int T, int H, int I, void* y, void* stream);

/*
 * Top-k mixture-of-experts SwiGLU FFN (the sparse-expert FFN of the paper's
 * Section 6.4 model family):
 *   routing : idx[t][k], k < K = the K largest router logits of token t in
 *             descending order; equal logits -> lower expert id first; a NaN
 *             logit never wins.  gate[t][k] = softmax over the K selected
 *             logits (fp32).
 *   permute : assignments (t,k) sorted by (expert, t, k); counts per expert.
 *   experts : per expert e, its rows go through that expert's SwiGLU FFN
 *             (grouped GEMMs over the permuted rows).
 *   combine : y[t] = sum_{k ascending} gate[t][k] * FFN_{idx[t][k]}(x[t]) in
 *             fp32, then -> bf16.  No atomics: deterministic.
 * Exactly one of router_logits (fp32 [T][E]) and w_router (bf16 [E][H]) is
 * non-NULL; with w_router the logits are x W_router^T accumulated in fp32.
 * w_gate, w_up bf16 [E][I][H]; w_down bf16 [E][H][I].
 * Optional outputs (device, NULL to skip): topk_idx i32 [T][K], topk_gate fp32
 * [T][K], expert_counts i32 [E].
 * E <= 64, K in {1,2}, K <= E.
 */
AFLEX_API aflex_status aflex_ffn_moe(aflex_ctx* ctx, const void* x, const float* router_logits,
                                     const void* w_router, const void* w_gate, const void* w_up,
                                     const void* w_down, int T, int H, int I, int E, int top_k, void* y,
                                     int32_t* topk_idx, float* topk_gate, int32_t* expert_counts, void* stream);

/*
 * The routing and permutation steps of aflex_ffn_moe on their own (same kernel), with every integer
 * result exported: topk_idx i32 [T][K] and topk_gate fp32 [T][K] as above; expert_counts i32 [E];
 * expert_offsets i32 [E+1] = exclusive prefix of the counts (expert e owns permuted rows
 * [offsets[e], offsets[e+1])); pos i32 [T][K] = permuted row of assignment (t,k) =
 * offsets[e] + number of assignments (t',k') to the same expert e that precede (t,k) in (t,k) order.
 * All pointers device, all required.  router_logits fp32 [T][E].  Integer results are exact.
 */
AFLEX_API aflex_status aflex_moe_route(aflex_ctx* ctx, const float* router_logits, int T, int E, int top_k,
                                       int32_t* topk_idx, float* topk_gate, int32_t* expert_counts,
                                       int32_t* expert_offsets, int32_t* pos, void* stream);

/* ---- Layer step: A side, boundary, F side, as M interleaved microbatches ---
 *
 * Computes, for the whole batch,
 *     a = attention(q, kv)                       bf16 [B][Hq*D]
 *     x = a W_o^T   (x = a if w_o == NULL, which requires Hq*D == hidden)
 *     y = dense FFN(x)  or  MoE FFN(x, router)   bf16 [B][hidden]
 * scheduled as in the paper's interleaved A/F pipeline (Section 4.3, Eq. 2):
 * the batch is cut into M contiguous microbatches, enqueued in the pipeline's
 * order A_0, F_0, A_1, F_1, ...  Both "sides" live on one GPU here, so the
 * transfer term of Eq. 2 is zero, and every kernel of either side fills the
 * whole GPU: by default everything goes on the caller's stream, where each
 * kernel starts (programmatic dependent launch) while its predecessor drains.
 * With aflex_set_interleave_streams(ctx, 1) A_i (attention + W_o) is enqueued
 * on the ctx's attention stream and F_i on its FFN stream as soon as A_i has
 * finished, so that A_{i+1} may overlap F_i as on two pools; on one B200 that
 * form measured 1 - 4 % slower.  M = 1 always runs A then F on the caller's
 * stream.  The result does not depend on M, on the split or on the form.
 */
typedef struct {
    aflex_attn_desc attn;
    int hidden;            /* H */
    int inter;             /* I */
    int num_experts;       /* 0 => dense FFN */
    int top_k;             /* MoE only */
    const void* w_o;       /* bf16 [H][Hq*D], or NULL iff Hq*D == H */
    const void* w_gate;    /* dense [I][H]  | MoE [E][I][H] */
    const void* w_up;      /* dense [I][H]  | MoE [E][I][H] */
    const void* w_down;    /* dense [H][I]  | MoE [E][H][I] */
    const void* w_router;  /* MoE: bf16 [E][H] or NULL when router logits are passed */
} aflex_layer_desc;

/*
 * q bf16 [B][Hq][D]; kv as for aflex_attn_decode (rows of page_table/seq_lens
 * are per sequence, sliced per microbatch); router_logits fp32 [B][E] or NULL.
 * microbatch_depth = M >= 1, M <= min(batch, 64).  mb_offsets: HOST i32 [M+1],
 * strictly increasing from 0 to batch, or NULL for the near-equal split (the
 * first batch % M microbatches get one extra row).
 * attn_out bf16 [B][Hq][D]: optional copy of the A-side output (NULL => kept
 * in the workspace).  y bf16 [B][hidden].
 * `stream` is joined on entry (the internal streams wait for it) and on exit
 * (it waits for the last A and F work).
 */
AFLEX_API aflex_status aflex_layer_step(aflex_ctx* ctx, const aflex_layer_desc* layer, const void* q,
                                        const aflex_kv* kv, int batch, const float* router_logits,
                                        int microbatch_depth, const int32_t* mb_offsets, void* attn_out,
                                        void* y, void* stream);

/*
 * Workspace bytes that suffice for aflex_attn_decode / aflex_ffn_* /
 * aflex_layer_step on this layer with up to max_batch rows, on the CURRENT device
 * (the scratch of the persistent kernels is per SM; with no device the figure is
 * for a 148-SM part) and for any setting of aflex_set_attn_ctas.  The attention
 * scratch is per CTA, not per context token: max_pages_per_seq must be >= 1 and
 * is otherwise unused.  Host computation, nothing is enqueued.
 */
AFLEX_API size_t aflex_workspace_bytes(const aflex_layer_desc* layer, int max_batch, int max_pages_per_seq);

/*
 * Plain bf16 linear map y = x W^T with fp32 accumulation (the W_o boundary
 * projection of aflex_layer_step, exposed for testing and benchmarking).
 * x bf16 [T][K]; w bf16 [N][K]; y bf16 [T][N].  K, N multiples of 8.
 */
AFLEX_API aflex_status aflex_linear(aflex_ctx* ctx, const void* x, const void* w, int T, int K, int N,
                                    void* y, void* stream);

/* Tuning knob: number of persistent attention CTAs per launch, 1..4096 (0 = automatic: two per
 * SM).  It changes how the KV cache is split across CTAs, never the result beyond rounding. */
AFLEX_API aflex_status aflex_set_attn_ctas(aflex_ctx* ctx, int ctas);

/* A promise about q in aflex_attn_decode / aflex_layer_step on this ctx (default off).  on != 0: q is never the
 * output of the library kernel enqueued directly before the call (aflex_linear, aflex_ffn_*, aflex_layer_step);
 * the attention kernel may then read q before its grid dependency resolves, like its other inputs, and starts
 * computing while the preceding kernel drains.  q written by aflex_rope_append, by a caller's kernel, by a copy,
 * or resident from earlier work satisfies the promise. */
AFLEX_API aflex_status aflex_set_attn_q_final(aflex_ctx* ctx, int on);

/* How aflex_layer_step enqueues M >= 2 microbatches (default off; AFLEX_MB_STREAMS=2 in the
 * environment when the ctx is created turns it on).  on != 0: A_i on the ctx's attention stream, F_i on its FFN stream behind an
 * event, both joined to the caller's stream at entry and exit.  on == 0: all kernels on the caller's stream in the
 * order A_0, F_0, A_1, F_1, ...  Host-side choice only; the results are the same. */
AFLEX_API aflex_status aflex_set_interleave_streams(aflex_ctx* ctx, int on);

/* ---- Whole decoder layers, chained (Section 4.3, "Interleaved A/F Pipeline") -------------
 *
 * The interleaved pipeline launches A of layer l+1 for microbatch i as soon as F of layer l has
 * returned that microbatch's hidden states, without waiting for the layer's other microbatches.
 * To chain layers the Attention group needs its remaining operators (the paper leaves them to
 * the two model families it serves, Section 6.1; these are their public definitions):
 *
 *   A_{l,i}:  r   = hidden state entering the layer (the residual stream), bf16 [rows][H]
 *             xn  = rmsnorm(r, w_ln_attn)            rmsnorm(v, g)_j = v_j / sqrt(mean(v^2) + eps) * g_j
 *             qkv = xn W_qkv^T                       rows of W_qkv: Hq query heads, Hkv key heads,
 *                                                    Hkv value heads, D rows per head
 *             q_h = rope(norm_q(qkv_h), pos), k_g = rope(norm_k(qkv_{Hq+g}), pos), pos = seq_len - 1
 *                   norm_* = rmsnorm over the head's D entries with gains w_q_norm / w_k_norm
 *                   (skipped when NULL); rope: for i < D/2, angle = pos * theta^(-2i/D),
 *                   (v_i, v_{i+D/2}) <- (v_i cos - v_{i+D/2} sin, v_{i+D/2} cos + v_i sin)
 *             K/V cache slot (page_table[b][pos/16], g, pos%16) <- bf16(k_g), bf16(v_g)
 *             a   = attention(q, cache)              as aflex_attn_decode; the new token takes part
 *             h1  = r + a W_o^T                      what A sends to F
 *   F_{l,i}:  out = h1 + FFN(rmsnorm(h1, w_ln_ffn))  what F returns; dense SwiGLU or top-k MoE
 *                                                    (router logits = rmsnorm(h1) W_router^T)
 *
 * Intermediate tensors are bf16 (each store rounds to nearest even); sums, norms and the rotary
 * angles are formed in fp32 / fp64.  seq_lens[b] counts the token being decoded: its K/V slot is
 * WRITTEN by this call (the k_cache / v_cache pointers of aflex_kv are written through), every
 * earlier slot is read.  Two sequences must not share the page of their last token.
 */
typedef struct {
    aflex_layer_desc layer;   /* attention shape, hidden, inter, experts, W_o, FFN weights, router;
                                 w_o is required; MoE layers require w_router */
    const void* w_qkv;        /* bf16 [(Hq + 2 Hkv) * D][H] */
    const void* w_ln_attn;    /* bf16 [H] */
    const void* w_ln_ffn;     /* bf16 [H] */
    const void* w_q_norm;     /* bf16 [D], or NULL: queries are not normalised */
    const void* w_k_norm;     /* bf16 [D], or NULL */
    float rms_eps;
    float rope_theta;
} aflex_decoder_desc;

/*
 * Runs num_layers >= 1 decoder layers on hidden states x_in bf16 [B][H] -> x_out bf16 [B][H]
 * (x_out may alias x_in).  layers: HOST array [num_layers]; kvs: HOST array [num_layers], one
 * cache per layer (page_table and seq_lens may be shared between them).  Microbatching as in
 * aflex_layer_step (depth M, host offsets or NULL); with M >= 2, A_{l+1,i} waits only for
 * F_{l,i}.  The result does not depend on M or on the split.  All layers must have the same
 * hidden size.  Device-side length or page-id violations raise AFLEX_ERR_BOUNDS in the status
 * word and skip the offending write.
 */
AFLEX_API aflex_status aflex_decoder_layers(aflex_ctx* ctx, const aflex_decoder_desc* layers, const aflex_kv* kvs,
                                            int num_layers, const void* x_in, int batch, int microbatch_depth,
                                            const int32_t* mb_offsets, void* x_out, void* stream);

/* Workspace bytes that suffice for aflex_decoder_layers on this layer shape.  Pure host computation. */
AFLEX_API size_t aflex_decoder_workspace_bytes(const aflex_decoder_desc* layer, int max_batch);

/*
 * The same layers over the tokens being PREFILLED (the paper's PA and PF pools: Section 1, prefill runs the two
 * operators on whole prompts, both dominated by matrix multiplications).  Row q_offsets[b] + i of x_in is token i of
 * the last m = q_offsets[b+1] - q_offsets[b] tokens of sequence b; kvs[l].seq_lens[b] = n counts them already
 * (m = n: a whole prompt; m < n: a chunk behind a cached prefix), the token sits at position n - m + i.  Per layer:
 *   PA:  r = hidden states; qkv = rmsnorm(r) W_qkv^T; per row q / k head norms and rotary embedding at the row's
 *        position; the row's K / V cache slot is WRITTEN; a = causal attention over the cache (aflex_attn_prefill);
 *        h1 = r + a W_o^T
 *   PF:  out = h1 + FFN(rmsnorm(h1))      dense SwiGLU or top-k MoE (router logits from w_router)
 * x_in, x_out: bf16 [T][H], T = q_offsets_host[batch] (x_out may alias x_in); q_offsets: DEVICE i32 [batch + 1];
 * q_offsets_host: HOST copy.  One stream, no microbatching (both groups are compute-bound here).  Workspace from
 * aflex_prefill_workspace_bytes(layer, T).  Errors as aflex_decoder_layers and aflex_attn_prefill.
 */
AFLEX_API aflex_status aflex_prefill_layers(aflex_ctx* ctx, const aflex_decoder_desc* layers, const aflex_kv* kvs,
                                            int num_layers, const void* x_in, int batch, const int32_t* q_offsets,
                                            const int32_t* q_offsets_host, void* x_out, void* stream);
AFLEX_API size_t aflex_prefill_workspace_bytes(const aflex_decoder_desc* layer, int max_tokens);

/* ---- A/F pair: the Attention side on one GPU, the FFN side on another -----------------------
 *
 * The paper's data plane (Section 4.3, "Placement-aware A/F Data Path"; Section 5: within a node
 * the hidden states move by peer copies over NVLink): at every A/F boundary the Attention group
 * sends one [rows][H] hidden-state tensor to the FFN group, which returns one [rows][H] tensor for
 * the next layer.  Here one process drives both GPUs:
 *
 *   A_{l,i} on ctx_a's device:  h1 = r + attention-side(r)      (as aflex_decoder_layers)
 *                               peer copy h1 rows -> ctx_f's device, event
 *   F_{l,i} on ctx_f's device:  out = h1 + FFN(rmsnorm(h1, w_ln_ffn))
 *                               peer copy out rows -> ctx_a's device, event
 *   A_{l+1,i} starts when the rows of microbatch i are back (interleaved schedule, Eq. 2 with a
 *   real t_comm).  The copies are plain cudaMemcpyPeerAsync calls on the producing side's stream:
 *   the payload is in the consumer's own memory before any of its kernels reads it.
 *
 * Placement: w_qkv, w_ln_attn, w_q_norm, w_k_norm, layer.w_o, the KV caches, x_in and x_out live on
 * ctx_a's device; w_ln_ffn, layer.w_gate / w_up / w_down / w_router on ctx_f's device ("each
 * worker loads only its role-specific weights", Section 5).  The two contexts may be on the same
 * device (then the copies are device-local); both must outlive the call's work.  `stream` belongs
 * to ctx_a's device and is joined on entry and exit.  Results equal aflex_decoder_layers up to
 * one extra bf16 rounding of the returned hidden states per layer.
 */
AFLEX_API aflex_status aflex_af_decoder_layers(aflex_ctx* ctx_a, aflex_ctx* ctx_f, const aflex_decoder_desc* layers,
                                               const aflex_kv* kvs, int num_layers, const void* x_in, int batch,
                                               int microbatch_depth, const int32_t* mb_offsets, void* x_out,
                                               void* stream);
/* Workspace bytes each side needs for aflex_af_decoder_layers (pure host computation). */
AFLEX_API size_t aflex_af_workspace_bytes(const aflex_decoder_desc* layer, int max_batch, int ffn_side);

/*
 * The two small operators of the chain on their own (testing, benchmarking).
 * aflex_add_rmsnorm: s = res (+ add when add != NULL), bf16 [T][H] each, summed in fp32;
 *   res_out (optional, may alias res or add) = bf16(s); y (optional) = bf16(rmsnorm(s, w)).
 *   H multiple of 8; w bf16 [H], required when y != NULL.
 * aflex_rope_append: the q / k / v step of A_{l,i} above on qkv bf16 [B][(Hq+2Hkv)*D]:
 *   writes q_out bf16 [B][Hq][D] and the decoded token's K/V cache slots.
 */
AFLEX_API aflex_status aflex_add_rmsnorm(aflex_ctx* ctx, const void* res, const void* add, const void* w, int T, int H,
                                         float eps, void* res_out, void* y, void* stream);
AFLEX_API aflex_status aflex_rope_append(aflex_ctx* ctx, const aflex_attn_desc* desc, const void* qkv,
                                         const aflex_kv* kv, int batch, const void* w_q_norm, const void* w_k_norm,
                                         float rms_eps, float rope_theta, void* q_out, void* stream);

/* ---- Host-side decisions of the data plane and the DVFS controller ------------------------
 *
 * Pure host computation on HOST pointers: nothing is launched and no GPU setting is read or
 * changed (applying a chosen frequency is the caller's business).  Times are in one unit of the
 * caller's choice (microseconds in the tests).
 */

/* Eq. 2 (Section 4.3): depth 1 -> t_a + t_f + t_comm; depth >= 2 -> max(t_a, t_f) + t_comm / depth. */
AFLEX_API double aflex_eq2_layer_time(double t_a, double t_f, double t_comm, int depth);

/* A profiled latency curve: n >= 1 points, x strictly ascending; piecewise linear, the end
 * segments extended beyond the profiled range, a single point is a constant. */
typedef struct { int n; const double* x; const double* y; } aflex_curve;
AFLEX_API double aflex_curve_eval(const aflex_curve* curve, double x);   /* NaN on a malformed curve */

/* Predicted stage times of one microbatch ("profiled Attention/FFN latency curves", Section 4.3):
 *   t_A = attn_vs_tokens(sum of its context lengths) + attn_vs_rows(rows),  t_F = ffn_vs_rows(rows),
 *   one hidden-state transfer, either direction = comm_fixed + comm_per_row * rows;
 *   t_A and t_F are clamped at zero where an extended curve goes negative.
 * shared_memory_system != 0: both sides run on one GPU; stages then queue on one engine (they do
 * not overlap) and transfers cost nothing. */
typedef struct {
    aflex_curve attn_vs_tokens, attn_vs_rows, ffn_vs_rows;
    double comm_fixed, comm_per_row;
    int shared_memory_system;
} aflex_pipeline_model;

/*
 * Completion time of `layers` chained layers cut into `depth` microbatches at host offsets
 * [depth+1] under the interleaved schedule of Section 4.3: stages A, transfer, F, transfer back of
 * every (layer, microbatch); each of the four engines serves its stages in (layer, microbatch)
 * order; A of layer l+1 starts for a microbatch once its hidden states are back.  With depth 1 this
 * is layers * Eq. 2 (t_comm = both transfers).  Returns NaN on invalid arguments.
 */
AFLEX_API double aflex_pipeline_makespan(const aflex_pipeline_model* model, const int32_t* seq_lens_host, int batch,
                                         int depth, const int32_t* offsets, int layers);

/*
 * "Dynamic microbatch depth" and "adaptive request batching" (Section 4.3): among the candidate
 * depths[n_depths] and all contiguous splits whose boundaries are multiples of `granularity` rows,
 * the pair with the lowest aflex_pipeline_makespan.  Ties keep the smaller depth, then the
 * lexicographically smaller offsets.  best_offsets: HOST i32 [max depth + 1].  The search is
 * exhaustive; more than 4e6 candidate splits return AFLEX_ERR_UNSUPPORTED (raise the granularity).
 */
AFLEX_API aflex_status aflex_plan_microbatches(const aflex_pipeline_model* model, const int32_t* seq_lens_host,
                                               int batch, int layers, const int* depths, int n_depths,
                                               int granularity, int* best_depth, int32_t* best_offsets,
                                               double* predicted);

/* Window size of the decode DVFS controller (Section 4.4): max(w_min, round(kappa * t_switch / t_iter)),
 * halves rounded away from zero. */
AFLEX_API int aflex_dvfs_window(int w_min, double kappa, double t_switch, double t_iter);

/* Algorithm 1 (window-based decode DVFS).  Frequencies are indices into the caller's ascending
 * DA / DF lists (the last index is f_max).  t_hat / e_hat: HOST [n_da][n_df] predicted iteration
 * time and energy of every pair for the current decode state and microbatch depth. */
typedef struct { int n_da, n_df; double tau; double delta_b; int window; double t_switch; } aflex_dvfs_params;
typedef struct { int i_da, i_df; int w; int b_last; } aflex_dvfs_state;
/* One decode iteration with batch size batch_now and measured time t_iter.  Returns 0: window still
 * open, state.w advanced; 1: searched, pair kept; 2: searched, pair changed (the caller applies
 * it); -1: invalid arguments.  Among equal-energy feasible pairs the first in (DA, DF) order wins. */
AFLEX_API int aflex_dvfs_decode_step(const aflex_dvfs_params* params, const double* t_hat, const double* e_hat,
                                     int batch_now, double t_iter, aflex_dvfs_state* state);

/* Prefill pair (Section 4.4): lowest-energy pair whose predicted time, plus t_switch when it
 * differs from the current pair, fits `budget` (the tightest remaining TTFT slack).  Returns flags:
 * AFLEX_DVFS_ESCALATED when the pair exceeds the global plan's baseline in either domain,
 * AFLEX_DVFS_INFEASIBLE when nothing fits (then the pair is (f_max, f_max)); -1 on invalid arguments. */
#define AFLEX_DVFS_ESCALATED 1
#define AFLEX_DVFS_INFEASIBLE 2
AFLEX_API int aflex_dvfs_prefill_pair(int n_pa, int n_pf, const double* t_hat, const double* e_hat, double budget,
                                      double t_switch, int cur_pa, int cur_pf, int base_pa, int base_pf,
                                      int* out_pa, int* out_pf);

/* ---- Measurement support (no counterpart in the paper's method; the per-operator latency
 * profiling of its Section 4.1 is the motivation) --------------------------------------------
 *
 * The library launches a fixed set of kernel kinds (attention partial / combine, the GEMMs,
 * the MoE glue).  Launches are always counted per kind.  With profiling enabled every launch
 * is additionally bracketed by a CUDA event pair on the stream it runs on (at most 8192
 * launches are kept per enable); aflex_profile_read waits for those events and sums the
 * device time per kind.  Enabling allocates events: do it outside timed regions.
 */
AFLEX_API int aflex_num_kernel_kinds(void);
AFLEX_API const char* aflex_kernel_name(int kind);
/* Launches of `kind` since the ctx was created; kind < 0 => all kinds together. */
AFLEX_API long long aflex_launch_count(const aflex_ctx* ctx, int kind);
/* on != 0: clear collected samples and start collecting; on == 0: stop collecting. */
AFLEX_API aflex_status aflex_profile_enable(aflex_ctx* ctx, int on);
/* Blocks until the collected launches of `kind` have finished; returns their summed device
 * time (ms) and their number. */
AFLEX_API aflex_status aflex_profile_read(aflex_ctx* ctx, int kind, double* total_ms, long long* launches);

/*
 * Timeline debugging.  When the ctx was created with the environment variable AFLEX_TRACE=1,
 * the attention and GEMM kernels record a few %globaltimer stamps per CTA (CTA start, grid
 * dependency satisfied, loads issued, last MMA issued, epilogue end) into a ring of 64 launch
 * records of [4096 CTAs][8] uint64 each.  aflex_trace_read synchronises the device, copies the
 * first `launches` records to host_out (launches * 4096 * 8 uint64), reports how many launches
 * were recorded since the last read in *next_slot, and rewinds the ring.
 */
AFLEX_API aflex_status aflex_trace_read(aflex_ctx* ctx, unsigned long long* host_out, int launches, int* next_slot);

#ifdef __cplusplus
}
#endif
#endif /* AFLEX_H_ */
