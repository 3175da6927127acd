/*
 * spkv.h -- C ABI of the SP-KV (Self-Pruned Key-Value attention) inference library
 * for NVIDIA B200 (sm_100a).
 *
 * The library implements the inference-time hot path of SP-KV: every new key/value
 * pair gets a utility logit from a small predictor (Eq. 1), lives in a ring of the w
 * most recent pairs (the always-visible local window), and when it leaves the ring it
 * is appended to a per-(layer, sequence, KV head) compact cache only if its utility
 * reaches the threshold tau (Eq. 2).  Attention for the query heads of a KV head then
 * runs over window U compact cache (Eq. 3-5) under grouped-query attention.
 *
 * General rules of this interface
 *   - Every function returns an int status: SPKV_OK (0) or a negative SPKV_E_* code.
 *     Nothing throws, aborts or traps the device.
 *   - "d_" arguments are DEVICE pointers, "h_" arguments are HOST pointers.  All device
 *     memory (arena, inputs, outputs, workspaces) is allocated, owned and freed by the
 *     caller; the library never allocates or frees device memory.
 *   - `stream` is a cudaStream_t passed as a plain pointer (NULL = default stream).
 *     Calls only enqueue work on it; the only calls that synchronise are spkv_status,
 *     spkv_cache_stats, spkv_safe_steps, spkv_cache_attach and the spkv_read_* helpers.
 *   - bf16 tensors are dense, row-major, 16-byte aligned.  head_dim is 128.
 *   - Argument errors are reported synchronously.  Errors found on the device (pool
 *     exhausted, context overflow, a bounded wait that ran out) are recorded in a sticky
 *     status word inside the arena and reported by spkv_status.
 *   - One host thread at a time per cache.  A sequence id may appear at most once in
 *     the seq-id list of a call.
 *
 * A "unit" is one (layer, sequence, KV head).  Units are independent of each other.
 * Positions: a unit that has received t pairs holds positions 0..t-1; the ring holds
 * positions max(0,t-w)..t-1; the compact cache holds the positions s <= t-1-w whose
 * logit passed the threshold, in ascending order.
 */
#ifndef SPKV_H_
#define SPKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct spkv_cache spkv_cache_t; /* opaque host-side handle */
typedef void *spkv_stream_t;            /* cudaStream_t */

enum {
  SPKV_OK = 0,
  SPKV_E_INVALID = -1,          /* bad argument                                        */
  SPKV_E_ARENA_TOO_SMALL = -2,  /* arena_bytes < spkv_arena_bytes(cfg)                 */
  SPKV_E_UNSUPPORTED = -3,      /* head_dim != 128, page_tokens != 64, group size > 16 */
  SPKV_E_CUDA = -4,             /* a CUDA runtime call failed                          */
  SPKV_E_POOL_EXHAUSTED = -5,   /* device: no free page; the pair was NOT stored       */
  SPKV_E_CONTEXT_OVERFLOW = -6, /* device: a unit's page table is full                 */
  SPKV_E_WORKSPACE = -7,        /* workspace missing or too small                      */
  SPKV_E_TIMEOUT = -8,          /* device: a bounded wait on a copy ran out            */
  SPKV_E_BOUNDS = -9,           /* device: a sequence id outside [0, max_seqs)         */
  SPKV_E_SCRATCH_LIMIT = -10,   /* request larger than the library's built-in scratch  */
  SPKV_E_ORDER_DECODE = -11,    /* device, overlap mode: a decode launch gave up waiting for the
                                   appends of its layer / the previous user of its workspace */
  SPKV_E_ORDER_APPEND = -12,    /* device, overlap mode: an append gave up waiting for the decode
                                   launches of its layer                                  */
  SPKV_E_BOUNDS_PAGE = -13,     /* device, SPKV_FLAG_DEBUG_BOUNDS: a page index read from a page
                                   table or the free stack names no pool page; the access was
                                   skipped or redirected to a page of the unit's own          */
  SPKV_E_CANARY = -14,          /* SPKV_FLAG_DEBUG_BOUNDS: a canary block between two regions of
                                   the arena no longer holds its pattern                      */
  SPKV_E_ATTACH = -15           /* spkv_cache_attach: no cache of this configuration in the arena */
};

typedef struct {
  int32_t n_layers;
  int32_t max_seqs;     /* sequence slots; seq ids are 0..max_seqs-1                    */
  int32_t n_q_heads;    /* multiple of n_kv_heads; group size G = n_q_heads/n_kv_heads  */
  int32_t n_kv_heads;
  int32_t head_dim;     /* must be 128                                                  */
  int32_t window;       /* w >= 1: pairs always visible (paper default 128)             */
  int32_t page_tokens;  /* must be 64                                                   */
  int32_t max_context;  /* upper bound on kept pairs per unit (sizes the page tables)   */
  int64_t pool_pages;   /* pages shared by all compact caches                           */
  float tau;            /* utility threshold in [0,1]; <= 0 keeps all, >= 1 keeps none  */
  int32_t flags;        /* 0 or an OR of SPKV_FLAG_* (below)                            */
  int32_t sink_tokens;  /* >= 0: the first sink_tokens positions of every sequence are
                           kept in the compact cache whatever their utility (the paper's
                           "Fixed Attention Sinks" ablation; its evaluation protocol uses
                           4).  0 = the method as defined by Eq. 2-4.                      */
  const uint8_t *h_local_only; /* HOST array [n_layers * n_kv_heads] or NULL, read only while
                           spkv_arena_bytes / spkv_cache_create / spkv_cache_attach run: a
                           non-zero entry declares that (layer, KV head) local-only for the
                           life of the cache (the paper's static hybrid layouts: sliding-window
                           heads beside global ones).  Such a head keeps nothing, sink positions
                           included, so its units get no page table (the arena is smaller by
                           max_context / 64 * 4 bytes per unit), the fused score + append does
                           not compute its utility (the logit is written as 0), and
                           spkv_set_head_tau refuses to change it.  n_kv_heads <= 64.        */
} spkv_config_t;

/* SPKV_FLAG_OVERLAP (off by default): consecutive hot-path launches on one stream overlap where
 * they share no data.  The fused score+append of layer l+1 runs beside the decode attention of
 * layer l, and the decode attention of layer l+1 starts on each SM as soon as that of layer l
 * has left it -- its start-up and the other's tail run under each other's page stream.  The
 * kernels then skip the wait for "everything earlier on the stream" (which would also wait
 * for the kernel they are meant to overlap) and order themselves on the device by the data
 * they really share: an append waits for the decode launches of its own layer, a decode for
 * the appends of its own layer and for the previous user of its workspace half.
 * What the caller has to guarantee in this mode, because the library cannot see foreign work
 * on the stream: the inputs of an append or decode call (x, k, v, q, seq ids) were complete
 * when the library's previous call on that stream was enqueued, and two decode calls in a row
 * do not write the same d_out.  That holds for an attention-only stack (the benchmark) and for
 * a model that stages a whole step's inputs beforehand; a model that computes q, k, v of a
 * layer between the library's calls must leave the flag off (every launch then waits for all
 * earlier work, as any stream-ordered kernel does; the library still issues its hot-path kernels
 * as programmatic dependent launches, so their block-local set-up runs under the tail of the
 * previous kernel, but they execute griddepcontrol.wait before touching an input or the cache).  Any other call of the library (prefill,
 * score, reset, ...) is a full synchronisation point either way. */
#define SPKV_FLAG_OVERLAP 1

/* SPKV_FLAG_PREFILL_PV_BF16 (off by default): the chunk attention of spkv_prefill multiplies the
 * softmax weights into the values as two bf16 terms (16 significant bits, bf16's exponent range)
 * for every unit.  By default it uses one fp16 term (11 bits) on values rescaled by a power of
 * two -- a third less tensor-core work -- and switches a unit to the two-term form by itself when
 * the largest |value| its queries can see is 2^20 or more (see spkv_prefill).  Set the flag when
 * the extra five bits matter more than the speed. */
#define SPKV_FLAG_PREFILL_PV_BF16 2

/* SPKV_FLAG_DEBUG_BOUNDS (off by default; a debugging aid for integrations, since memory checkers
 * are not always available): every page index a kernel reads from a page table or from the free
 * stack is checked against the pool's range before it is used; a violation sets the sticky status
 * SPKV_E_BOUNDS_PAGE and the access is skipped (writes) or redirected to a page of the unit's own
 * (reads), so that nothing outside the arena is touched.  spkv_status additionally verifies the
 * 256-byte canary blocks that separate the metadata regions of the arena (SPKV_E_CANARY). */
#define SPKV_FLAG_DEBUG_BOUNDS 4

/* Utility predictor f of Eq. 1 (the sigmoid is never evaluated: the decision is taken
 * in logit space, u >= tau  <=>  logit >= log(tau/(1-tau))).
 *   kind 0, linear:  logit[h] = <W1[h,:], x> + b1[h]            W1 [n_kv_heads, d_in]
 *   kind 1, MLP   :  logit[h] = <W2[h,:], SiLU(W1 x + b1)> + b2[h]
 *                    W1 [hidden, d_in], b1 [hidden], W2 [n_kv_heads, hidden], b2 [n_kv_heads]
 *                    (two-layer perceptron of the paper's reference listing)
 * Weights are bf16, biases float32, all device pointers.  d_in and hidden are multiples
 * of 8. */
typedef struct {
  int32_t kind;
  int32_t d_in;
  int32_t hidden; /* kind 1 only */
  int32_t reserved;
  const void *d_W1;
  const float *d_b1;
  const void *d_W2;
  const float *d_b2;
} spkv_predictor_t;

typedef struct {
  int64_t units;           /* n_layers * max_seqs * n_kv_heads                          */
  int64_t pairs_seen;      /* sum over units of t                                       */
  int64_t pairs_kept;      /* sum over units of compact-cache lengths                   */
  int64_t pairs_in_window; /* sum over units of min(t, w)                               */
  int64_t pairs_evicted;   /* sum over units of max(t - w, 0)                           */
  int64_t gates_open;      /* number of pairs, window included, with logit >= tau_logit */
  int64_t pages_in_use;    /* pool pages held by compact caches                         */
  int64_t pages_free;
  int64_t bytes_resident;  /* K/V bytes a decode step reads: kept + window pairs        */
  double density_all;      /* Eq. 8: gates_open / pairs_seen                            */
  double density_cache;    /* pairs_kept / pairs_evicted (fraction kept in the
                              long-term cache, the figure the paper reports)           */
} spkv_stats_t;

/* ---- cache lifetime ---------------------------------------------------------------- */

/* Bytes of device memory a cache with this configuration needs (host only). */
int spkv_arena_bytes(const spkv_config_t *cfg, size_t *out_bytes);

/* Lays the cache out inside the caller's arena (256-byte aligned device memory of at
 * least spkv_arena_bytes bytes) and enqueues its initialisation on `stream`.  The arena
 * must stay alive and untouched by the caller until spkv_cache_destroy.
 * Paper: Appendix "Inference Kernels" (paged pool, per-head page-index arrays, ring
 * window kept by metadata); here the capacity is fixed at creation instead of grown. */
int spkv_cache_create(const spkv_config_t *cfg, void *d_arena, size_t arena_bytes,
                      spkv_stream_t stream, spkv_cache_t **out);

/* Snapshot / resume.  The arena is position-independent (it holds offsets and page indices, no
 * pointers), so a snapshot of a cache is a plain copy of its arena made by the caller (device to
 * device, to the host, to a file), and a copy placed in device memory again -- at any 256-byte
 * aligned address, in this or a later process -- becomes a cache by attaching to it.
 * spkv_cache_attach checks the header cache_create wrote (magic, layout version, a hash of every
 * configuration field that fixes the layout; tau and flags may differ and take effect as given)
 * and returns a handle without initialising anything; SPKV_E_ATTACH if the header does not
 * match.  Synchronises `stream`.  Two handles on one arena must not be used at the same time. */
int spkv_cache_attach(const spkv_config_t *cfg, void *d_arena, size_t arena_bytes,
                      spkv_stream_t stream, spkv_cache_t **out);

/* Checkpoint / rollback of a live cache without copying its pool: saves (restores) the metadata
 * and the ring pages -- everything appends and prefill chunks change IN PLACE; the pairs they add
 * to the pool land behind the saved lengths and are simply forgotten by a rollback.  Valid as long
 * as no spkv_cache_reset_seq came between the two (it hands pages to other units).  Use: replaying
 * the same decode steps (benchmark repeats, speculative tokens that were rejected).
 *   d_buf: device, >= spkv_cache_checkpoint_bytes(cache) bytes.  Asynchronous on `stream`; a full
 *   synchronisation point for SPKV_FLAG_OVERLAP. */
size_t spkv_cache_checkpoint_bytes(const spkv_cache_t *cache);
int spkv_cache_checkpoint(spkv_cache_t *cache, void *d_buf, size_t bytes, spkv_stream_t stream);
int spkv_cache_rollback(spkv_cache_t *cache, const void *d_buf, size_t bytes, spkv_stream_t stream);

/* SPKV_FLAG_OVERLAP only: tells the cache that work it did not launch (a copy, another library's
 * kernel) was enqueued on the stream after its previous call and produces inputs of its next one.
 * The next hot-path launch then waits for everything earlier on the stream, as it does after any
 * other call of the library.  Call it before a step whose inputs were staged on the same stream,
 * and before capturing a CUDA graph of a step. */
int spkv_note_foreign_work(spkv_cache_t *cache);

/* Safe-step budget (paper, Appendix "Inference Kernels": capacity checks are amortised by a budget
 * of steps that cannot exhaust the headroom).  The number of further decode steps the listed
 * sequences can take, all layers and KV heads, before a page-table or pool limit COULD be hit,
 * assuming the worst case that every pair leaving a window is kept.  While the answer is n > 0
 * the next n steps cannot raise SPKV_E_POOL_EXHAUSTED / SPKV_E_CONTEXT_OVERFLOW (other sequences
 * sharing the pool must be counted in by listing them).  h_seq_ids: HOST array of B ids, B = 0 =
 * every sequence.  Synchronises `stream`.  spkv_safe_steps_from_lengths is the arithmetic alone
 * (host only): h_len / h_t [n_units] kept pairs / pairs received of the units to count. */
int spkv_safe_steps(spkv_cache_t *cache, const int32_t *h_seq_ids, int32_t B, spkv_stream_t stream,
                    int64_t *out_steps);
int spkv_safe_steps_from_lengths(const spkv_config_t *cfg, const int32_t *h_len, const int32_t *h_t,
                                 int64_t n_units, int64_t pages_free, int64_t *out_steps);

/* Byte offsets of the arena's canary blocks (256 bytes of 0xC5 each, one after every metadata
 * region), for tools that want to verify them themselves.  Host only; *n_out = their number. */
int spkv_arena_canaries(const spkv_config_t *cfg, size_t *h_offsets, int32_t cap, int32_t *n_out);

/* Frees the host handle only (the arena belongs to the caller). */
int spkv_cache_destroy(spkv_cache_t *cache);

/* Empties every unit of sequence `seq` (all layers) and returns its pages to the pool. */
int spkv_cache_reset_seq(spkv_cache_t *cache, int32_t seq, spkv_stream_t stream);

/* Changes tau for all FUTURE evictions (the paper adjusts sparsity a posteriori by
 * changing the threshold; pairs already dropped stay dropped). */
int spkv_set_tau(spkv_cache_t *cache, float tau);

/* Static hybrid layouts (the paper's hand-designed local/global mixes, e.g. a 3:1 ratio of
 * sliding-window to global heads): a (layer, KV head) may carry a threshold of its own, in
 * force for its future evictions, on the stream given.  tau >= 1 makes the head local-only
 * (window attention, nothing is ever kept: its compact cache and page table stay empty),
 * tau <= 0 makes it a full-attention head, NaN returns it to the cache-wide threshold.
 * kv_head = -1 addresses every KV head of the layer.  spkv_score's optional flags follow the
 * cache-wide threshold only.  A head that only ever needs the window is better declared in
 * spkv_config_t.h_local_only: it then costs no page table and no scoring. */
int spkv_set_head_tau(spkv_cache_t *cache, int32_t layer, int32_t kv_head, float tau,
                      spkv_stream_t stream);

/* ---- the hot path ------------------------------------------------------------------ */

/* Step 1, score + threshold (Eq. 1-2).  d_x [n_tok, d_in] bf16 -> d_logits_out
 * [n_tok, n_kv_heads] float32 (fp32 accumulation).  d_flags_out (optional, may be NULL)
 * [n_tok, n_kv_heads] uint8 = 1 where logit >= tau_logit under the current tau.
 * The two-layer form runs on the tensor cores for n_tok >= 64 when hidden is a multiple of 16
 * up to 256 (and hidden * n_kv_heads rounded up to 8 is at most 4096), on the CUDA cores
 * otherwise; the two differ in the last bits of a logit, and the flag always follows the
 * logit written. */
int spkv_score(spkv_cache_t *cache, const spkv_predictor_t *pred, const void *d_x,
               int32_t n_tok, float *d_logits_out, uint8_t *d_flags_out,
               spkv_stream_t stream);

/* Step 2, append + evict, one new pair per listed sequence and KV head (Appendix
 * "Inference Kernels": fused token append).  For each unit: the new pair (position t)
 * goes to ring slot t mod w; if t >= w the pair of position t-w leaves the ring first
 * and is appended to the unit's compact cache iff its stored logit >= tau_logit.
 *   d_seq_ids [B] int32, d_k/d_v [B, n_kv_heads, 128] bf16, d_logits [B, n_kv_heads] f32.
 * On SPKV_E_POOL_EXHAUSTED / SPKV_E_CONTEXT_OVERFLOW the evicted pair is dropped, the
 * unit's length is unchanged and the sticky status is set. */
int spkv_append_evict(spkv_cache_t *cache, int32_t layer, const int32_t *d_seq_ids, int32_t B,
                      const void *d_k, const void *d_v, const float *d_logits,
                      spkv_stream_t stream);

/* Steps 1 + 2 in one launch: scores the B new tokens with `pred` (Eq. 1; same float32
 * logits as spkv_score, bit for bit) and appends them as spkv_append_evict does.
 *   d_x [B, d_in] bf16; d_logits_out [B, n_kv_heads] float32, optional for the linear
 *   predictor (may be NULL), required for the two-layer one (scored by its own kernel). */
int spkv_score_append_evict(spkv_cache_t *cache, int32_t layer, const spkv_predictor_t *pred,
                            const int32_t *d_seq_ids, int32_t B, const void *d_x, const void *d_k,
                            const void *d_v, float *d_logits_out, spkv_stream_t stream);

/* Workspace bytes spkv_decode_attention needs for a batch of B sequences. */
size_t spkv_decode_workspace_bytes(const spkv_config_t *cfg, int32_t B);

/* Step 3, decode attention (Eq. 3-5) for the query whose pair was appended last:
 * out[b, j, :] = softmax(<q[b,j], K_vis> * sm_scale) V_vis with K_vis = ring U compact
 * cache of KV head floor(j / G).  Split over the keys across thread blocks, partial
 * results merged by their log-sum-exp weights.
 *   d_q [B, n_q_heads, 128] bf16 -> d_out [B, n_q_heads, 128] bf16;
 *   d_lse_opt [B, n_q_heads] float32 natural-log sum-exp of the scaled scores, or NULL;
 *   d_workspace: >= spkv_decode_workspace_bytes(cfg, B) bytes, 256-byte aligned, used by
 *   this cache only; it must have been zero-filled once before its first use and is then
 *   left alone by the caller (consecutive calls alternate between its two halves).
 *   Under SPKV_FLAG_OVERLAP a launch starts beneath the tail of the previous decode launch only
 *   if both calls were given the SAME workspace and batch size (the two then use different
 *   halves); with another workspace or batch the launch is an ordinary stream-ordered one --
 *   the result is the same, only the overlap is lost. */
int spkv_decode_attention(spkv_cache_t *cache, int32_t layer, const int32_t *d_seq_ids,
                          int32_t B, const void *d_q, void *d_out, float *d_lse_opt,
                          float sm_scale, void *d_workspace, size_t workspace_bytes,
                          spkv_stream_t stream);

/* spkv_decode_attention that also returns the output rows in float32, as they are before the
 * rounding to bf16 (bf16 rounding alone is up to 2^-9 |o|, which hides smaller errors of the
 * kernel from a comparison): d_out_f32 [B, n_q_heads, 128] float32, device, 16-byte aligned,
 * required.  d_out is written as usual.  Everything else as spkv_decode_attention. */
int spkv_decode_attention_f32(spkv_cache_t *cache, int32_t layer, const int32_t *d_seq_ids,
                              int32_t B, const void *d_q, void *d_out, float *d_out_f32,
                              float *d_lse_opt, float sm_scale, void *d_workspace,
                              size_t workspace_bytes, spkv_stream_t stream);

/* (No counterpart in the paper: an addition for integration.)
 * spkv_decode_attention for callers that must not allocate device memory -- code running
 * inside someone else's memory plan, where every cudaMalloc is forbidden or already spoken
 * for (a serving engine that has handed all free HBM to its own KV pool, a plugin loaded
 * into a host application, a latency-critical loop that may not touch the allocator).
 * It computes exactly what spkv_decode_attention computes, but its split-K scratch is a
 * fixed SPKV_STATIC_SCRATCH_BYTES array that is part of the library image on every GPU,
 * so no workspace is passed and nothing is allocated or freed, here or in any library
 * routine it calls.  Inputs and outputs are still the caller's.
 *   - Sizes: B and the head configuration must satisfy
 *     spkv_decode_workspace_bytes(cfg, B) <= SPKV_STATIC_SCRATCH_BYTES, otherwise the call
 *     returns SPKV_E_SCRATCH_LIMIT and does nothing (with 8 KV heads: every supported batch
 *     at 4 query heads per KV head, batches up to 32 at 8 per KV head; beyond that use
 *     spkv_decode_attention with a workspace of your own).
 *   - The first call on each device looks up the array's device address (with that device
 *     current).  Make that first call outside of any stream capture.
 *   - All calls on a device share the one array and it keeps the previous call's contents;
 *     the entry point clears the part that must start at zero on `stream` before the
 *     kernel.  Two calls whose GPU work overlaps (different streams, no dependency) race on
 *     it: keep such calls ordered.  A call that is refused (any error code) has not touched
 *     the array.
 *   - That clearing is an ordinary stream operation, so in SPKV_FLAG_OVERLAP mode a launch made
 *     through this entry point starts only after everything earlier on `stream` has finished
 *     (it never runs under the tail of the previous decode launch). */
#define SPKV_STATIC_SCRATCH_BYTES (6u << 20)
int spkv_decode_attention_static(spkv_cache_t *cache, int32_t layer, const int32_t *d_seq_ids,
                                 int32_t B, const void *d_q, void *d_out, float *d_lse_opt,
                                 float sm_scale, spkv_stream_t stream);

/* Workspace bytes spkv_prefill needs for a chunk of C pairs. */
size_t spkv_prefill_workspace_bytes(const spkv_config_t *cfg, int32_t C);

/* Companion path, chunked prefill of C pairs for one sequence and layer: equivalent to
 * C x (spkv_append_evict, spkv_decode_attention) -- the paper's chunked-prefill protocol
 * with the cache compressed after each chunk -- done as: stream compaction of the pairs
 * that leave the window (ballot + prefix sum, ascending position), tensor-core attention
 * of every query of the chunk over compact cache U window (Eq. 3-5), ring update.
 *   d_q [C, n_q_heads, 128], d_k/d_v [C, n_kv_heads, 128] bf16, d_logits [C, n_kv_heads],
 *   d_out [C, n_q_heads, 128] bf16.  d_q = d_out = NULL builds the cache state only.
 *   With queries, sm_scale must be positive and finite (SPKV_E_INVALID otherwise).
 * Precision of the weights-times-values product: one fp16 term on values rescaled by a power
 * of two taken from the largest finite |value| the chunk's queries can see (compact cache,
 * window, chunk); exact for every value within 2^28 of that maximum, off by at most 2^-39 of
 * it below; a weight below 2^-32 of its row's running maximum is dropped.  A unit where that
 * largest |value| reaches 2^20 -- and every unit under SPKV_FLAG_PREFILL_PV_BF16 -- takes two
 * bf16 terms on the unscaled values instead (no scaling, no dropped weights). */
int spkv_prefill(spkv_cache_t *cache, int32_t layer, int32_t seq, int32_t C, const void *d_q,
                 const void *d_k, const void *d_v, const float *d_logits, void *d_out,
                 float sm_scale, void *d_workspace, size_t workspace_bytes,
                 spkv_stream_t stream);

/* Soft-gated whole-sequence forward: the attention the paper trains with (Section "Training",
 * "Phase 1. Soft Gated Training", Eq. 6; the annealed gate of "Phase 2", Eq. 7; kernel notes in
 * "Training Efficiency"), forward only.  Causal attention of all T queries over all T keys of one
 * sequence in which key s gets, for query t,
 *     bias 0                 if 0 <= t - s < window      (the local window is never gated)
 *     bias log u~_s          if t - s >= window          (Eq. 6)
 *     -inf                   if s > t,
 * u~_s = (1 - alpha) sigma(logit_s) + alpha 1[logit_s >= tau_logit] (Eq. 7; alpha = 0: soft gating,
 * alpha = 1: the binary gate, i.e. the hard-gated forward of Eq. 3-5), one gate per KV head shared
 * by its query-head group.  log sigma is evaluated without forming the sigmoid; the epsilon the
 * paper's listing adds inside the logarithm guards gradients and is not applied.
 * No cache is involved and nothing is kept between calls.
 *   d_q [T, n_q_heads, 128], d_k/d_v [T, n_kv_heads, 128] bf16, d_logits [T, n_kv_heads] float32
 *   -> d_out [T, n_q_heads, 128] bf16, d_lse_opt [T, n_q_heads] float32 (natural-log sum-exp of
 *   the biased scaled scores; may be NULL).  head_dim is 128, n_q_heads / n_kv_heads <= 16.
 *   alpha in [0, 1]; tau as in spkv_config_t; sm_scale positive and finite;
 *   flags: 0 or SPKV_FLAG_PREFILL_PV_BF16 (precision of weights x values as in spkv_prefill);
 *   d_workspace: >= spkv_softgate_workspace_bytes(T, n_q_heads, n_kv_heads) bytes, 256-byte
 *   aligned (K and V are rewritten there as 64-key pages: about the size of K + V);
 *   d_status: device, one int32 that the caller has set to 0: SPKV_E_TIMEOUT is stored there if a
 *   bounded wait inside the kernel ran out.  Asynchronous on `stream`. */
size_t spkv_softgate_workspace_bytes(int32_t T, int32_t n_q_heads, int32_t n_kv_heads);
int spkv_softgate_forward(int32_t T, int32_t n_q_heads, int32_t n_kv_heads, int32_t window,
                          const void *d_q, const void *d_k, const void *d_v, const float *d_logits,
                          float alpha, float tau, float sm_scale, int32_t flags, void *d_out,
                          float *d_lse_opt, void *d_workspace, size_t workspace_bytes,
                          int32_t *d_status, spkv_stream_t stream);

/* One decode step of one layer from HOST buffers (pinned memory, or the copies are not
 * asynchronous): score -> append/evict -> decode attention with the inputs copied in and the
 * output copied out.  The copies run on two streams of the cache's own, double-buffered, so
 * that the transfers of one call overlap the kernels of its neighbours; the kernels run on
 * `stream`.  Nothing synchronises with the host.  Completion: after call i, `stream` has
 * waited for the output of call i-1; spkv_decode_step_host_flush makes `stream` wait for the
 * output of the last call -- synchronise (or order later work) after that.  The host input
 * buffers of a call must stay untouched until its copies have run (flush + synchronise).
 *   h_x [B, d_in], h_q [B, n_q_heads, 128], h_k/h_v [B, n_kv_heads, 128] bf16,
 *   h_out [B, n_q_heads, 128] bf16;
 *   d_staging: >= spkv_decode_step_staging_bytes(cfg, B, d_in) bytes (two slots of inputs,
 *   logits and output, and the decode workspace; zero-filled once before first use).  Pass
 *   the same buffer to consecutive calls; flush and synchronise before freeing or reusing it. */
size_t spkv_decode_step_staging_bytes(const spkv_config_t *cfg, int32_t B, int32_t d_in);
int spkv_decode_step_host(spkv_cache_t *cache, int32_t layer, const spkv_predictor_t *pred,
                          const int32_t *d_seq_ids, int32_t B, const void *h_x, const void *h_q,
                          const void *h_k, const void *h_v, void *h_out, float sm_scale,
                          void *d_staging, size_t staging_bytes, spkv_stream_t stream);
int spkv_decode_step_host_flush(spkv_cache_t *cache, spkv_stream_t stream);

/* One decode step of the WHOLE layer stack from device buffers, for an attention-only stack whose
 * inputs all exist before the step (Eq. 1-5 per layer; Appendix "Inference Kernels": fused token
 * append, sparse decode): the same results as, layer by layer, spkv_score_append_evict followed
 * by spkv_decode_attention on the same cache, bit for bit, in two launches -- the appends of every layer, then one
 * persistent decode-attention kernel whose blocks take page ranges of all layers from one list,
 * so that their page streams never stop between layers.  Ordinary stream-ordered launches (no
 * SPKV_FLAG_OVERLAP contract); no synchronisation.
 *   preds [n_layers]: HOST array of predictors with the same d_in (linear predictors, up to 128
 *   layers and a batch whose per-layer plans fit in shared memory take the two launches; otherwise
 *   the call makes the per-layer calls itself);
 *   d_x [L, B, d_in], d_q [L, B, n_q_heads, 128], d_k/d_v [L, B, n_kv_heads, 128] bf16, 16-byte
 *   aligned -> d_out [L, B, n_q_heads, 128] bf16; d_logits_out [L, B, n_kv_heads] float32 or NULL
 *   (required by two-layer predictors); d_lse_opt [L, B, n_q_heads] float32 or NULL;
 *   d_workspace: >= spkv_decode_stack_workspace_bytes(cfg, B) bytes, 256-byte aligned, used by this
 *   cache only, zero-filled once before its first use and then left alone.  After a sticky
 *   SPKV_E_TIMEOUT it must be zero-filled again. */
size_t spkv_decode_stack_workspace_bytes(const spkv_config_t *cfg, int32_t B);
int spkv_decode_stack(spkv_cache_t *cache, const spkv_predictor_t *preds, const int32_t *d_seq_ids,
                      int32_t B, const void *d_x, const void *d_q, const void *d_k, const void *d_v,
                      void *d_out, float *d_logits_out, float *d_lse_opt, float sm_scale,
                      void *d_workspace, size_t workspace_bytes, spkv_stream_t stream);

/* One decode step of the WHOLE layer stack from host buffers, for an attention-only stack whose
 * inputs all exist before the step.  The layers go in three chunks (a short head, the bulk, a
 * short tail; one chunk per layer below four layers): a chunk's inputs are copied
 * on a stream of the cache's own, its kernels (spkv_decode_stack's two launches over the chunk's
 * layers) run on `stream` once they have landed, and its outputs are copied
 * back on another stream of the cache's own while the next chunk computes.  `stream` ends up
 * waiting for the last output copy, so synchronising `stream` means h_out is complete; the host
 * buffers must stay untouched until then (pinned memory, or the copies serialise).  No
 * synchronisation inside the call.
 *   preds [n_layers] (host array, same d_in); h_x [L, B, d_in], h_q [L, B, n_q_heads, 128],
 *   h_k/h_v [L, B, n_kv_heads, 128] bf16 -> h_out [L, B, n_q_heads, 128] bf16;
 *   d_staging: >= spkv_decode_stack_staging_bytes(cfg, B, d_in) bytes, 256-byte aligned,
 *   zero-filled once before first use. */
size_t spkv_decode_stack_staging_bytes(const spkv_config_t *cfg, int32_t B, int32_t d_in);
int spkv_decode_stack_host(spkv_cache_t *cache, const spkv_predictor_t *preds, const int32_t *d_seq_ids,
                           int32_t B, const void *h_x, const void *h_q, const void *h_k, const void *h_v,
                           void *h_out, float sm_scale, void *d_staging, size_t staging_bytes,
                           spkv_stream_t stream);

/* ---- introspection ----------------------------------------------------------------- */

/* Synchronises `stream` and returns the sticky device status (SPKV_OK or the first
 * device-side error).  spkv_clear_status resets it. */
int spkv_status(spkv_cache_t *cache, spkv_stream_t stream);
int spkv_clear_status(spkv_cache_t *cache, spkv_stream_t stream);

/* Gate density (Eq. 8) and memory accounting; synchronises `stream`. */
int spkv_cache_stats(spkv_cache_t *cache, spkv_stream_t stream, spkv_stats_t *out);

/* Lengths of one layer: h_len / h_t [max_seqs, n_kv_heads] int32 (kept pairs / pairs
 * received); either may be NULL.  Synchronises `stream`. */
int spkv_read_lengths(spkv_cache_t *cache, int32_t layer, int32_t *h_len, int32_t *h_t,
                      spkv_stream_t stream);

/* Compact cache of one unit in logical (ascending position) order: up to `cap` pairs.
 * h_pos [cap] int32, h_k/h_v [cap,128] bf16 (each may be NULL); *n_out = stored length.
 * Synchronises `stream`. */
int spkv_read_kept(spkv_cache_t *cache, int32_t layer, int32_t seq, int32_t kvh, int32_t *h_pos,
                   void *h_k, void *h_v, int32_t cap, int32_t *n_out, spkv_stream_t stream);

/* Ring of one unit in ascending position order: min(t, w) pairs.  h_pos [w] int32,
 * h_k/h_v [w,128] bf16, h_logits [w] float32 (each may be NULL).  Synchronises. */
int spkv_read_window(spkv_cache_t *cache, int32_t layer, int32_t seq, int32_t kvh,
                     int32_t *h_pos, void *h_k, void *h_v, float *h_logits, int32_t *n_out,
                     spkv_stream_t stream);

/* The float32 logit-space threshold currently in force. */
float spkv_tau_logit(const spkv_cache_t *cache);

const char *spkv_error_string(int code);

/* Measurement aid (no counterpart in the paper): streams `bytes` bytes (rounded down to whole
 * 32 KB pages) from device memory through shared memory with the bulk copies the decode kernel
 * uses, one block per SM, and does nothing else with them.  The pages are handed out one by one
 * through an atomic counter, so that SMs that draw faster take more of them (an even split ends
 * with its slowest SM: about 3 % less on a B200).  Timed by the caller with events it gives the
 * read-only HBM rate of this GPU, the ceiling of a kernel that only reads (the usual copy figure
 * is half writes).
 *   d_buf: device, 16-byte aligned; d_sink: device, TWO 64-bit words: [0] a checksum is added to
 *   it, [1] the page counter, zero before the first call and left at zero by every call (calls
 *   that share it must not overlap on the GPU);
 *   d_status: device, one int32, set to SPKV_E_TIMEOUT if a bounded wait ran out.  Asynchronous. */
int spkv_stream_read(const void *d_buf, size_t bytes, unsigned long long *d_sink, int32_t *d_status,
                     spkv_stream_t stream);

/* Self-test of the library's bounded device waits (no counterpart in the paper).  Every copy
 * pipeline of the library waits on its copies with a clock limit; when a wait runs out the kernel
 * records SPKV_E_TIMEOUT, stops issuing, waits (bounded) for the copies it still has in flight and
 * returns -- the context stays usable.  This call runs that error path on purpose and harmlessly:
 * one thread arms a barrier for 64 bytes more than the single 32 KB copy it issues delivers, waits
 * `limit_clocks` cycles, and then drains as described.
 *   d_buf: device, 16-byte aligned, >= 32 KB readable; d_status: device, four int32:
 *   [0] SPKV_E_TIMEOUT (the wait ran out, as it must), [1] 1 = the copy in flight was waited for,
 *   [2] clocks the first wait lasted, [3] 1 = the copied data is in place.  Asynchronous. */
int spkv_wait_selftest(const void *d_buf, long long limit_clocks, int32_t *d_status, spkv_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* SPKV_H_ */
