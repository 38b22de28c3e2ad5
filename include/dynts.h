/*
 * dynts.h -- C ABI of the B200 (sm_100a) decode hot path of Dynamic Thinking-Token Selection:
 * GQA decode attention over a budget-limited KV cache, fused with accumulation of each retained
 * token's attention mass (its importance score), and the periodic eviction that keeps the
 * question window, the local window and the top-scoring tokens of the selection window.
 *
 * Conventions
 * -----------
 *  - "device" pointers are CUDA device memory on the current device; "host" pointers are ordinary
 *    host memory.  The library never frees caller memory.
 *  - Every call that launches work is asynchronous on the cache's stream (see
 *    dynts_cache_set_stream) unless stated otherwise.  Caller buffers must stay valid until the
 *    stream reaches the work.
 *  - Errors detectable on the host are returned before anything is launched and leave the cache
 *    unchanged; dynts_last_error() then holds a message.  Errors detected on the device (a bound
 *    that the host mirror should have made impossible) are reported by dynts_poll_error().
 *  - A handle is not thread-safe; use one thread per handle.
 *  - Shapes: L layers, Nb sequences, Hq query heads, Hkv KV heads, G = Hq / Hkv, d head_dim,
 *    cap rows per slab.  A slab is one (layer, sequence, KV head): K[cap][d], V[cap][d] in the
 *    cache dtype, pos[cap] int32, score[cap] fp32.  All tensors are contiguous, row-major, in the
 *    index order written, and 16-byte aligned.
 */
#ifndef DYNTS_H
#define DYNTS_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dynts_cache dynts_cache_t; /* opaque, owned by the library */

typedef enum dynts_status {
  DYNTS_OK = 0,
  DYNTS_ERR_INVALID_ARG = 1, /* NULL/misaligned pointer, bad index, unsupported shape */
  DYNTS_ERR_OOM = 2,         /* device or host allocation failed / storage too small */
  DYNTS_ERR_CAPACITY = 3,    /* append past the slab capacity: an eviction was skipped */
  DYNTS_ERR_BUDGET = 4,      /* question window + local window exceed the eviction target */
  DYNTS_ERR_STATE = 5,       /* call not allowed in the cache's current state */
  DYNTS_ERR_CUDA = 6,        /* a CUDA runtime call failed */
  DYNTS_ERR_DEVICE = 7       /* a kernel found an inconsistent length or bound and skipped work */
} dynts_status_t;

/* DYNTS_BF16_KV8: q, k, v, out are bf16; the slabs hold each K/V element as an 8-bit float (E4M3:
 * 1 sign, 4 exponent bits with bias 7, 3 mantissa bits, no infinities, largest finite value 448)
 * with one scale per tensor: a row element x is stored as the code nearest to x / scale (ties to
 * the even code, magnitudes beyond 448 saturate) and read as value(code) * scale.  The paper does
 * not describe this storage; it halves the bytes a decode step reads.  Needs head_dim % 16 == 0. */
typedef enum dynts_dtype { DYNTS_BF16 = 0, DYNTS_FP32 = 1, DYNTS_BF16_KV8 = 2 } dynts_dtype_t;

typedef enum dynts_score_source { DYNTS_SCORE_ATTENTION = 0, DYNTS_SCORE_EXTERNAL = 1 } dynts_score_source_t;

typedef struct dynts_config {
  int layers, batch, q_heads, kv_heads, head_dim;
  int budget;         /* B: default eviction target (rows kept per slab) */
  int window;         /* W_l: most recent rows, always kept */
  int evict_interval; /* E: decode steps between evictions; slab capacity = max budget + E */
  int capacity;       /* rows per slab; 0 => max budget + evict_interval.  A multiple of 32 lets the
                         kernels use 16-byte score accesses and whole lines of their scratch: an odd
                         row count costs the score update about 4x its loads */
  int dtype;          /* dynts_dtype_t of q, k, v, out and of the slab rows */
  const int* seq_budgets; /* host [batch] per-sequence targets, or NULL => budget for all */
  void* storage;          /* device memory for the whole cache, 256-byte aligned, or NULL:
                             the library then allocates with cudaMalloc and frees in destroy */
  size_t storage_bytes;   /* size of storage; must be >= dynts_cache_bytes(cfg) */
  void* stream;           /* cudaStream_t, NULL => the default stream */
} dynts_config_t;

/* ---- lifetime ------------------------------------------------------------------------------ */

/* Create a cache for the paper's problem statement (Section 4.2: a KV budget B with a local
 * window W_l, per layer and KV head).  Defaults: batch 1, q_heads = kv_heads, bf16,
 * evict_interval = max(window, 64); storage is allocated at the first prefill/decode so that
 * dynts_cache_set_shape can still change them.  Returns NULL on failure. */
dynts_cache_t* dynts_cache_create(int layers, int kv_heads, int head_dim, int budget, int window);

/* Change batch / q_heads / dtype / evict_interval of a cache made by dynts_cache_create; only
 * before its first prefill or decode (else DYNTS_ERR_STATE). */
dynts_status_t dynts_cache_set_shape(dynts_cache_t* c, int batch, int q_heads, int dtype, int evict_interval);

/* Bytes of device storage a cache with this configuration needs (0 if the config is invalid). */
size_t dynts_cache_bytes(const dynts_config_t* cfg);

/* Create from a full configuration; storage may come from the caller (e.g. a PyTorch tensor).
 * The storage is zeroed on the stream.  *out receives the handle. */
dynts_status_t dynts_cache_create_ex(const dynts_config_t* cfg, dynts_cache_t** out);

/* Release the handle and whatever the library allocated itself.  Synchronises the stream. */
void dynts_cache_destroy(dynts_cache_t* c);

/* All later work of this cache is issued on `stream` (a cudaStream_t). */
dynts_status_t dynts_cache_set_stream(dynts_cache_t* c, void* stream);

/* ---- the hot path -------------------------------------------------------------------------- */

/* Load prompt rows into every slab (Section 4.2: the question window W_q holds the prefill
 * tokens).  k, v: device [L, Nb, Hkv, n_tokens, d].  The first n_pinned rows get score +inf and
 * are never evicted (the paper pins all of them: n_pinned = n_tokens); the rest start at 0.
 * Positions are 0..n_tokens-1.  Replaces the sequences' previous content. */
dynts_status_t dynts_prefill(dynts_cache_t* c, const void* k, const void* v, int n_tokens, int n_pinned);

/* dynts_prefill plus the attention of the prompt itself (Eq. 4-5 for t = 1..n_tokens: position t
 * attends to positions 1..t), for a model that runs its prefill through this library.
 *   q, out: device [L, Nb, Hq, n_tokens, d];  k, v: device [L, Nb, Hkv, n_tokens, d]; bf16, d = 128.
 * The rows are stored exactly as dynts_prefill stores them (the first n_pinned pinned with score
 * +inf); prompt attention adds nothing to the scores (the paper pins the question instead of
 * scoring it).  A dense contraction: it runs on the tensor cores (tcgen05, accumulators in tensor
 * memory, operands by TMA).  Other dtypes and head sizes: DYNTS_ERR_INVALID_ARG.  A bounded wait
 * inside the kernel that runs out is reported by dynts_poll_error (DYNTS_ERR_DEVICE). */
dynts_status_t dynts_prefill_attn(dynts_cache_t* c, const void* q, const void* k, const void* v, void* out, int n_tokens,
                                  int n_pinned);

/* The attention part of dynts_prefill_attn alone (Eq. 4-5 for t = 1..n_tokens): reads q, k, v,
 * writes out, leaves the cache untouched.  Same shapes and restrictions. */
dynts_status_t dynts_prompt_attn(dynts_cache_t* c, const void* q, const void* k, const void* v, void* out, int n_tokens);

/* dynts_prefill_attn one layer at a time, for a model whose layer l + 1 prompt activations depend on
 * layer l's attention output: q, out: device [Nb, Hq, n_tokens, d]; k, v: device [Nb, Hkv, n_tokens, d].
 * Stores the layer's rows and computes its prompt attention.  Call for layers 0 .. L-1 in order with
 * the same n_tokens and n_pinned; the sequences' lengths are set with the last layer. */
dynts_status_t dynts_prefill_attn_layer(dynts_cache_t* c, int layer, const void* q, const void* k, const void* v, void* out,
                                        int n_tokens, int n_pinned);

/* The same for one sequence of a ragged batch; k, v: device [L, Hkv, n_tokens, d].  Marks the
 * sequence active. */
dynts_status_t dynts_prefill_seq(dynts_cache_t* c, int seq, const void* k, const void* v, int n_tokens, int n_pinned);

/* One decode step for all layers (Eq. 4-6).  For every slab of every active sequence:
 * append k_new/v_new as row n (position = tokens seen so far, score 0), attend with the group's
 * G query heads over rows [0, n] (the new row included) with weights softmax(q.k / sqrt(d)),
 * write out = sum_j alpha_j v_j, and add to each row's score its attention mass summed over
 * the G heads.
 *   q, out:        device [L, Nb, Hq, d]  (cache dtype; out is rounded to nearest even)
 *   k_new, v_new:  device [L, Nb, Hkv, d]
 *   scores:        NULL, or device [L, Nb, Hkv, cap] fp32 that additionally receives this step's
 *                  mass per row (rows [0, n] of each slab are overwritten, the rest untouched).
 * The cache length of each active sequence grows by one.  DYNTS_ERR_CAPACITY if any active
 * sequence is already at capacity.  Rows of inactive sequences in `out` are left untouched.
 * Stream capture: the library keeps a host copy of every sequence's length and hands it to the
 * kernel with the launch; while the stream is being captured the kernel reads the lengths from
 * device memory instead, so a captured step can be replayed.  Replays do not update the host
 * copy: capture whole cycles that return to the lengths they started from (decode steps + the
 * eviction), or do not mix replays that change the lengths with direct calls on the same cache. */
dynts_status_t dynts_decode_attn(dynts_cache_t* c, const void* q, const void* k_new, const void* v_new,
                                 void* out, float* scores);

/* The same for one layer (a model whose layer l+1 query depends on layer l's output).
 *   q, out: device [Nb, Hq, d];  k_new, v_new: device [Nb, Hkv, d];  scores: as above (full
 *   [L, Nb, Hkv, cap] buffer; only this layer's part is written).
 * Layers must be called in order 0..L-1 within a step; lengths grow after layer L-1. */
dynts_status_t dynts_decode_attn_layer(dynts_cache_t* c, int layer, const void* q, const void* k_new,
                                       const void* v_new, void* out, float* scores);

/* dynts_decode_attn with HOST buffers: brings q, k_new, v_new to the device, runs the step,
 * copies out back and synchronises the stream.  Inputs in pinned, mapped host memory
 * (cudaHostAlloc, cudaHostRegister) that is 16-byte aligned are read by the kernel in place over
 * the bus -- every input element is read once -- and, if out is such memory too, the output rows are
 * written there by the kernel; any other host memory goes through device staging buffers and
 * copies.  (Staging buffers are allocated at the first call.) */
dynts_status_t dynts_decode_attn_host(dynts_cache_t* c, const void* q, const void* k_new, const void* v_new,
                                      void* out);

/* Eviction (Section 4.2).  Every slab longer than the target keeps: rows [0, M) (question
 * window), its last `window` rows (local window), and of the rows between them the
 * k = target - M - window with the highest score, equal scores going to the lower index.
 * Survivors are compacted in place, in their original order, into rows [0, target): K, V, pos and
 * score move together.  budget <= 0 => each sequence's configured budget.  Sequences no longer
 * than the target are untouched.  DYNTS_ERR_BUDGET if M + window > target for a sequence that
 * must shrink. */
dynts_status_t dynts_evict(dynts_cache_t* c, int budget);

/* Eviction with one selection per sequence (Appendix B.1 aggregates a token's importance across
 * all layers and heads): the scores of all slabs of a sequence are summed row by row (see
 * dynts_aggregate_scores) and every slab ranks its selection window by that sum, so all layers
 * and heads keep the same tokens.  Requires that all slabs of a sequence hold the same tokens,
 * i.e. that every eviction of this cache is of this kind (or driven by shared external scores).
 * Otherwise as dynts_evict. */
dynts_status_t dynts_evict_global(dynts_cache_t* c, int budget);

/* Appendix B.1's aggregate on its own: agg[b][j] = sum over all layers and KV heads of the score
 * of row j of sequence b, the fp32 slab scores added in double precision and rounded to fp32 once.
 *   agg: device [Nb, cap] fp32, caller-owned; rows [0, len(b)) of each active sequence are
 *   written, the rest left untouched.  These are the keys dynts_evict_global ranks by. */
dynts_status_t dynts_aggregate_scores(dynts_cache_t* c, float* agg);

/* Eviction with one target per sequence; seq_targets: host [Nb]. */
dynts_status_t dynts_evict_ex(dynts_cache_t* c, const int* seq_targets);

/* No counterpart in the paper: the eviction of Section 4.2 for callers that must not allocate.
 *
 * Some callers cannot call cudaMalloc where they need an eviction: code that runs inside a
 * framework's memory-pool critical section, a real-time serving loop that forbids allocator
 * calls after start-up, or a process whose whole device memory was handed to another allocator.
 * This entry point evicts caller-owned slabs in place and allocates nothing, on the host or the
 * device, and calls no routine that allocates (none of cudaMalloc, cudaFree, torch).  The
 * gather list that connects the selection kernel to the compaction kernel, which a cache
 * object keeps in its own storage, lives here in a fixed 4 MiB array built into the library's
 * device image (every GPU that loads the library holds it until the process exits).
 *
 *   K, V:   device [n_slabs][capacity][head_dim] in `dtype`, compacted in place
 *   pos:    device [n_slabs][capacity] int32;  score: device [n_slabs][capacity] fp32
 *   n_rows: rows currently valid in every slab; n_pinned: leading rows never evicted
 * Same selection rule, tie-break and stable compaction as dynts_evict; afterwards every slab
 * holds min(n_rows, target) rows (the caller tracks the length).  Asynchronous on `stream`.
 *
 * Limits and caveats:
 *  - n_slabs * capacity (+ a small header) must fit the built-in scratch: about one million
 *    rows in total.  Larger requests return DYNTS_ERR_CAPACITY and launch nothing.
 *  - All calls on one GPU share the array, which keeps the previous call's contents; the entry
 *    point rewrites every word it later reads, so nothing needs clearing.  Two calls whose
 *    kernels may overlap on the GPU (different streams) race on it: serialise them.
 *  - The first call on each device looks up the array's device address (with that device
 *    current); make that first call before any stream capture begins. */
dynts_status_t dynts_evict_noalloc(void* K, void* V, int* pos, float* score, int n_slabs, int head_dim, int dtype,
                                   int capacity, int n_rows, int n_pinned, int window, int target, void* stream);

/* No counterpart in the paper.  The kernels of dynts_evict_noalloc re-check the lengths they were
 * given and, if they disagree (memory the caller changed while the call was in flight), record it
 * in a status word inside the built-in scratch and move nothing for that slab.  This waits for
 * `stream` and returns DYNTS_ERR_DEVICE if the most recent call on the current device recorded
 * anything, else DYNTS_OK.  Allocates nothing. */
dynts_status_t dynts_evict_noalloc_status(void* stream);

/* Scales of a DYNTS_BF16_KV8 cache (default 1, 1).  Host floats; k_scale, v_scale > 0 and finite.
 * Allowed only while no sequence holds rows (DYNTS_ERR_STATE otherwise): stored codes are not
 * re-encoded.  Choose scale ~ max|x| / 448 of the tensor to use the format's range. */
dynts_status_t dynts_cache_set_kv_scale(dynts_cache_t* c, float k_scale, float v_scale);

/* ---- predictor scores and the paper's own trigger ------------------------------------------ */

/* Where the importance scores come from.  DYNTS_SCORE_ATTENTION (default): every decode step
 * adds each retained row's attention mass to its score (Eq. 6 computed online).
 * DYNTS_SCORE_EXTERNAL: the paper's inference mode (Section 4.1, Eq. 7) -- the decode step leaves
 * the scores alone and gives the appended row score 0; the caller supplies the token's score with
 * dynts_append_scores (or writes the accumulator directly, see dynts_cache_scores).  In this mode
 * the `scores` argument of the decode calls still receives the step's attention mass if given. */
dynts_status_t dynts_cache_set_score_source(dynts_cache_t* c, int source);

/* Section 4.2: a newly generated token's importance score is stored beside its KV.  s_new: device
 * [Nb] fp32, one predictor score per sequence (Eq. 7); it becomes the score of the row appended by
 * the latest decode step in every layer and KV head of each active sequence, so all slabs of a
 * sequence rank their rows alike and retain the same tokens.  Call after dynts_decode_attn (or
 * after the last layer of a layer-by-layer step) and before the eviction. */
dynts_status_t dynts_append_scores(dynts_cache_t* c, const float* s_new);

/* Section 4.2's trigger: every active sequence whose row count has reached budget_B is reduced to
 * M + floor(ratio * W_s) + W_l rows, W_s = budget_B - M - W_l (question window, top share of the
 * selection window, local window); the others are left alone.  The paper does not say how
 * ratio * W_s is rounded: down, here.  budget_B must not exceed the capacity; call it after every
 * decode step.  DYNTS_ERR_BUDGET if M + W_l > budget_B. */
dynts_status_t dynts_evict_at_budget(dynts_cache_t* c, int budget_B, double ratio);

/* Importance Predictor head (Section 4.1, Eq. 7; Appendix A): scores[n] = MLP(h[n]) with layers
 * d -> 2d -> d/2 -> 1.  The paper calls the layers linear and names no activation: activation 0
 * applies none, 1 applies ReLU after the first two layers.
 *   h: device [batch][d] bf16 (final hidden states);  W1 [2d][d], W2 [d/2][2d], W3 [1][d/2]: device
 *   bf16, row-major [out][in];  b1 [2d], b2 [d/2], b3 [1]: device fp32 or NULL;  scores: device
 *   [batch] fp32 (ready for dynts_append_scores).  Accumulation and the hidden activations are fp32.
 *   scratch: device memory of dynts_predictor_mlp_scratch_bytes(d, batch) bytes, 16-byte aligned,
 *   caller-owned (holds partial sums between the layers; contents need not be preserved).
 * d must be a multiple of 512.  Three launches on `stream`; allocates nothing. */
size_t dynts_predictor_mlp_scratch_bytes(int d, int batch);
dynts_status_t dynts_predictor_mlp(const void* h, const void* W1, const float* b1, const void* W2, const float* b2,
                                   const void* W3, const float* b3, int d, int batch, int activation, void* scratch,
                                   size_t scratch_bytes, float* scores, void* stream);

/* ---- sequence management and inspection ---------------------------------------------------- */

/* Ragged batches: mark a sequence finished (length 0, inactive) until its next prefill_seq. */
dynts_status_t dynts_seq_reset(dynts_cache_t* c, int seq);

/* Re-reads the per-sequence lengths from the device into the host copy (synchronises the stream).
 * Needed after replays of a captured graph that changed the lengths (decode steps advance them on
 * the device only), before the next direct call that depends on them (an eviction, a decode step
 * outside a graph). */
dynts_status_t dynts_cache_refresh_lengths(dynts_cache_t* c);

/* Host mirror of a sequence's cache length (no synchronisation); -1 on a bad argument. */
int dynts_cache_len(const dynts_cache_t* c, int seq);

/* Rows per slab. */
int dynts_cache_capacity(const dynts_cache_t* c);

/* Device [L, Nb, Hkv, cap] fp32 score accumulator.  The caller may overwrite it on the cache's
 * stream to drive the eviction with external scores (e.g. a predictor's).  NULL before storage
 * exists.  (The decode step adds each step's mass with compensated summation; the compensation
 * terms live beside the scores inside the cache, move with them at an eviction, and are at most
 * one ulp of the score, so overwriting the scores needs no further call.)
 * A decode launch may leave the score update of some slabs to the next decode launch (the update
 * has nothing to overlap with at the end of a launch).  Every call of this function first enqueues
 * what is still outstanding on the cache's stream, as do eviction, export, import, prefill,
 * dynts_append_scores and dynts_synchronize: read the accumulator through a pointer obtained
 * after the decode calls whose effect you want to see, not through one kept from before. */
float* dynts_cache_scores(dynts_cache_t* c);

/* Copy one slab to host buffers (any may be NULL): K, V [n][d] in the cache dtype, pos [n] int32,
 * score [n] fp32, *n rows.  Synchronises the stream. */
dynts_status_t dynts_cache_export(dynts_cache_t* c, int layer, int seq, int head, void* K, void* V,
                                  int* pos, float* score, int* n);

/* Overwrite one slab from host buffers holding n rows (all four required).  The sequence's length
 * becomes n once every slab of it has been imported with the same n (the caller's duty).
 * Synchronises the stream. */
dynts_status_t dynts_cache_import(dynts_cache_t* c, int layer, int seq, int head, const void* K,
                                  const void* V, const int* pos, const float* score, int n, int n_pinned);

/* Reads the device status word (pinned host memory written by kernels): DYNTS_OK or
 * DYNTS_ERR_DEVICE.  Does not synchronise; call after dynts_synchronize for a definite answer. */
dynts_status_t dynts_poll_error(dynts_cache_t* c);

/* Wait for the cache's stream. */
dynts_status_t dynts_synchronize(dynts_cache_t* c);

/* Launch configuration of the decode kernel, for tuning.  variant: 0 => automatic, 1 => generic
 * FMA kernel (any supported shape), 2 => tensor-core kernel with one thread-block cluster per
 * slab, 3 => persistent streaming tensor-core kernel (TMA ring, the default where it applies);
 * 2 and 3 need bf16, d = 128, G <= 8.  cluster: for variants 1 and 2 the cluster size (1, 2, 4,
 * 8 or 16; 0 => automatic); for variant 3 the CTAs per SM (1 or 2; anything else => 2). */
dynts_status_t dynts_cache_set_launch(dynts_cache_t* c, int cluster, int variant);

/* Device-side waits are bounded: a thread that waits for a tile or a hand-over inside the streaming
 * decode kernel polls at most `polls` times (default 2^22, seconds at worst); when a wait runs
 * out the CTA raises the timeout bit of the status word, every later wait of that CTA returns at
 * once, the kernel ends, and dynts_poll_error reports DYNTS_ERR_DEVICE (that step's results are
 * void; the context stays usable).  polls >= 64. */
dynts_status_t dynts_cache_set_wait_limit(dynts_cache_t* c, unsigned int polls);

/* For tests of that path only: the next streaming decode launch of this cache omits one tile load
 * (the item-th 32-row chunk of the first CTA's piece), so that the wait for it runs out.  The
 * step's results, and the scores of the slabs that CTA covers, are void afterwards. */
dynts_status_t dynts_debug_drop_tile_load(dynts_cache_t* c, int item);

/* Launch configuration of the eviction kernel, for tuning.  split: 1, 2, 4 or 8 => the kernel that
 * keeps every thread's rows in registers, with that many CTAs sharing one slab (each takes the
 * selection decision for itself and moves its own share of the row bytes; slabs of up to 4352
 * rows, the count is halved until the row size allows it); -1 => the one-CTA-per-slab kernel that
 * keeps its keys in shared memory; 0 => automatic (the register kernel for slabs of up to 2304
 * rows, with as many CTAs per slab as still fit the GPU at once).  Results do not depend on it. */
dynts_status_t dynts_cache_set_evict_launch(dynts_cache_t* c, int split);

/* Bookkeeping of the most recent eviction, read back from the device (synchronises the stream):
 * over the slabs that shrank, the rows whose scores were scanned and the rows that changed place
 * during compaction (rows behind the first evicted one).  For traffic accounting. */
dynts_status_t dynts_evict_stats(dynts_cache_t* c, long long* rows_scanned, long long* rows_moved);

/* Number of kernels this library has launched on behalf of the cache so far. */
long long dynts_cache_launch_count(const dynts_cache_t* c);

/* Message of the calling thread's last failed call. */
const char* dynts_last_error(void);

const char* dynts_version(void);

#ifdef __cplusplus
}
#endif
#endif /* DYNTS_H */
