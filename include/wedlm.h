/*
 * wedlm.h - C ABI of the WeDLM decoding-step library for NVIDIA B200 (sm_100a).
 *
 * One step of Streaming Parallel Decoding (Algorithm 1 of the WeDLM paper) works on a fixed
 * window of W slots per sequence on top of a committed prefix whose keys/values live in a
 * paged KV cache:
 *
 *   wedlm_reorder            Topological Reordering (Eq. 5-6): filled slots first, masks last,
 *                            logical position ids kept; commit length of Algorithm 1.
 *   wedlm_window_attn        RoPE at the logical ids (Section 2.2), staging of the window's
 *                            K/V behind the prefix, causal attention of the reordered window
 *                            over prefix + window (Section 5.2, "a small prefill"), GQA.
 *   wedlm_kv_append          the staging step alone ("Extend (K, V)" of Algorithm 1).
 *   wedlm_confidence_commit  per-mask-row entropy / max-prob / arg-max over the vocabulary,
 *                            selection by distance-adjusted entropy (Eq. 11), then Commit,
 *                            Predict and Refill of Algorithm 1.
 *   wedlm_window_refill      Commit + shift + Refill alone.
 *   wedlm_step_host          the three calls above for step inputs that live in host memory
 *   wedlm_step_host_lmhead   (logits from the host, or hidden states from the host with the LM head on the device).
 *   wedlm_dual_stream_*      training side (Section 4.2): two-stream input construction and its attention.
 *
 * Conventions common to every call
 *   - Every pointer named below is a DEVICE pointer unless it is the config or says "host".
 *     The caller owns all memory and the library allocates and frees nothing: scratch memory is a
 *     caller-supplied workspace sized by a query function.  The one exception is
 *     wedlm_confidence_commit_static, whose scratch is an array inside the library image.
 *   - No result of one call is remembered for the next.  What the library does keep per process is
 *     bookkeeping only: a count of the kernels it launched (wedlm_launch_count), the one-shot timing
 *     hook armed by wedlm_profile_next_attn (per host thread), per-device attributes it asked the
 *     driver for once (SM count, shared-memory opt-ins), the device address of the built-in
 *     scratch array, and the copy stream with its two events that the wedlm_step_host calls use
 *     (per host thread and device, created on first use).
 *   - Calls are asynchronous on the CUDA stream passed as `stream` (a cudaStream_t cast to
 *     void*; NULL is the legacy default stream).  No call synchronises with the host.  The
 *     wedlm_step_host calls fork their large upload onto a copy stream of the library and join it
 *     back into `stream` before they return: to the caller everything is ordered on `stream`.
 *   - All tensors are dense, row-major ("last index fastest") and need 16-byte aligned base
 *     addresses.  Index tensors are int32, flags are uint8.
 *   - "logical order" = ascending position id within the window; "physical order" = the order
 *     after wedlm_reorder.  Slot j (logical) of sequence b has position id prefix_len[b] + j.
 *   - Every call that launches work opens an NVTX range with its own name for its duration on the host
 *     (a no-op unless a timeline tool is attached).
 *   - Return value: WEDLM_OK or a negative WEDLM_ERR_* code.  Argument errors are detected on
 *     the host before anything is launched.  Data-dependent errors (a block-table entry outside
 *     the page pool) are detected on the device: the offending access is skipped and a bit is
 *     OR-ed into *status (if status != NULL); nothing traps.
 */
#ifndef WEDLM_H_
#define WEDLM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define WEDLM_OK                        0
#define WEDLM_ERR_INVALID_ARG         (-1)
#define WEDLM_ERR_UNSUPPORTED         (-2)
#define WEDLM_ERR_WORKSPACE_TOO_SMALL (-3)
#define WEDLM_ERR_CUDA                (-4)
#define WEDLM_ERR_TIMEOUT             (-5)
#define WEDLM_ERR_STATIC_SCRATCH      (-6)  /* problem too large for the built-in scratch array */

/* bits OR-ed into the device status word */
#define WEDLM_STATUS_BAD_PAGE     1   /* block_table entry outside [0, num_pages)            */
#define WEDLM_STATUS_BAD_LENGTH   2   /* prefix_len[b] < 0, > cfg.max_prefix_len, or +W beyond the table */
#define WEDLM_STATUS_WAIT_EXPIRED 4   /* a bounded on-chip wait gave up (tensor-core path)     */

#define WEDLM_DTYPE_BF16 0
#define WEDLM_DTYPE_F32  1

#define WEDLM_CONF_ENTROPY 0   /* select mask i iff  H_i + lambda * d_i <= tau   (Eq. 11) */
#define WEDLM_CONF_MAXPROB 1   /* select mask i iff  max_v p_i(v) >= maxprob_thr          */

#define WEDLM_COMMIT_STREAMING 0   /* commit the leading run of filled slots (Algorithm 1)              */
#define WEDLM_COMMIT_BLOCK     1   /* block-wise baseline of Section 5.2 / Fig. 3c: commit nothing until  */
                                   /* every active slot of the window is filled, then commit all of them */

#define WEDLM_ATTN_AUTO    0
#define WEDLM_ATTN_GENERIC 1   /* CUDA-core kernel, any supported shape, bf16 or fp32     */
#define WEDLM_ATTN_TENSOR  2   /* tcgen05 + TMA kernel, bf16, head_dim 128, page 16       */

typedef struct wedlm_config {
  int32_t batch;              /* B  sequences (any count a 1-D grid can index)             */
  int32_t window;             /* W  slots per sequence (1..1024)                           */
  int32_t n_q_heads;          /* Hq                                                        */
  int32_t n_kv_heads;         /* Hkv, divides Hq; query head h reads KV head h / (Hq/Hkv)  */
  int32_t head_dim;           /* D  (32, 64, 128 or 256)                                   */
  int32_t page_size;          /* tokens per cache page (8, 16 or 32)                       */
  int32_t max_pages_per_seq;  /* row stride of block_table                                 */
  int32_t num_pages;          /* pages in the cache pool                                   */
  int32_t vocab;              /* V                                                         */
  int32_t dtype;              /* WEDLM_DTYPE_*: storage type of q/k/v/out, cache, logits   */
  int32_t rope_style;         /* 0: pairs (d, d+D/2) "rotate-half"; 1: pairs (2d, 2d+1)    */
  float   rope_theta;         /* angle of pair d at position p is p * theta^(-2d/D)        */
  float   softmax_scale;      /* 0 selects 1/sqrt(D)                                       */
  int32_t conf_mode;          /* WEDLM_CONF_*                                              */
  float   tau;                /* entropy threshold (nats)                                  */
  float   lambda;             /* distance penalty of Eq. 11                                */
  float   maxprob_thr;
  int32_t mask_token_id;      /* token id written into fresh mask slots                    */
  int32_t max_prefix_len;     /* host-known upper bound of prefix_len[b]: sizes the key split and the  */
                              /* workspace.  A prefix_len[b] above it (the device value moved on while */
                              /* the host bound did not) is treated as max_prefix_len by the attention */
                              /* kernels and flagged WEDLM_STATUS_BAD_LENGTH; nothing is written out   */
                              /* of bounds, the rows of that sequence are then wrong.                  */
  int32_t attn_impl;          /* WEDLM_ATTN_*                                              */
  int32_t commit_mode;        /* WEDLM_COMMIT_*                                            */
  float   sample_temperature; /* 0: Sample() is the arg-max; > 0: one draw from softmax(l/T) */
  uint32_t sample_seed_lo;    /* 64-bit seed of the draws, low and high word               */
  uint32_t sample_seed_hi;
} wedlm_config_t;

/* Human-readable text of a return code.  Host pointer to a static string. */
const char* wedlm_strerror(int code);

/* Library version, major*10000 + minor*100 + patch. */
int wedlm_version(void);

/* Measurement aids and self-test: not part of the decoding path, no counterpart in the paper, and no
 * stability promise (they may change between versions without the call signatures above them changing).
 * wedlm_launch_count: kernels launched through this library by the calling process so far.
 * wedlm_profile_next_attn: the next wedlm_window_attn call made by the calling host thread records
 *   the two CUDA events (cudaEvent_t cast to void*, host handles, either may be NULL) on its stream
 *   immediately before and after its main attention kernel, so that the kernel can be timed inside
 *   a longer sequence of launches.  One-shot: the hook is cleared by that call. */
/* wedlm_selftest_wait_expiry: launches one small CTA that waits, with at most max_polls (1..2^24) polls,
 *   on an on-chip barrier that nothing ever signals - the situation the bounded waits of the tensor-core
 *   attention kernel exist for.  The kernel gives up, ORs WEDLM_STATUS_WAIT_EXPIRED into *status (device
 *   i32, required) and returns normally; the context stays usable. */
unsigned long long wedlm_launch_count(void);
int wedlm_selftest_wait_expiry(uint32_t max_polls, int32_t* status, void* stream);
int wedlm_profile_next_attn(void* event_before, void* event_after);

/*
 * Topological Reordering (Eq. 5-6) and commit length (Algorithm 1, Commit).
 *   filled        in  u8  [B,W] logical order; non-zero = the slot holds a predicted token
 *   window_tokens in  i32 [B,W] logical order, or NULL (then tokens_phys is not written)
 *   prefix_len    in  i32 [B]
 *   window_len    in  i32 [B] number of active slots (<= W), or NULL for W everywhere.
 *                     Slots at or beyond window_len count as trailing masks.
 *   perm          out i32 [B,W]  perm[i] = logical slot that sits at physical row i
 *   inv_perm      out i32 [B,W]  inv_perm[perm[i]] = i
 *   pos_ids       out i32 [B,W]  pos_ids[i] = prefix_len + perm[i]
 *   tokens_phys   out i32 [B,W]  window_tokens[perm[i]], or NULL
 *   n_filled      out i32 [B]    number of filled active slots (= first mask's physical row)
 *   n_commit      out i32 [B]    length of the leading run of filled slots in logical order
 *                                (WEDLM_COMMIT_BLOCK: window_len if every active slot is filled, else 0)
 */
int wedlm_reorder(const wedlm_config_t* cfg, const uint8_t* filled, const int32_t* window_tokens,
                  const int32_t* prefix_len, const int32_t* window_len,
                  int32_t* perm, int32_t* inv_perm, int32_t* pos_ids, int32_t* tokens_phys,
                  int32_t* n_filled, int32_t* n_commit, void* stream);

/* Bytes of workspace wedlm_window_attn needs for this config (uses batch, window, heads,
 * head_dim, dtype, max_prefix_len, attn_impl, and the SM count of the current device).  It holds the
 * rotated queries and, when the batch has fewer work units than the GPU has CTA slots, room for the
 * partial results of keys that are split between CTAs (up to about 2*SMs/Hkv pieces per query row,
 * so a single long sequence can use the whole GPU); only the part that a launch uses is touched.
 * Returns 0 on an invalid config. */
size_t wedlm_window_attn_workspace_bytes(const wedlm_config_t* cfg);

/*
 * One attention layer of the step's forward (Section 5.2; RoPE per Section 2.2).
 *   q            in  [B,W,Hq,D]  window queries, physical order, before RoPE
 *   k, v         in  [B,W,Hkv,D] window keys / values, physical order, k before RoPE
 *   k_cache,
 *   v_cache   in/out [num_pages,Hkv,page_size,D]  paged cache; K stored already rotated.
 *                    Rows prefix_len[b] .. prefix_len[b]+W-1 of sequence b are OVERWRITTEN
 *                    with the rotated k and v of physical rows 0..W-1 (staging).  Because the
 *                    committed slots are the first physical rows, a later commit of n tokens
 *                    is just prefix_len += n.  The pages covering prefix_len+W tokens must be
 *                    present in the block table.
 *   block_table  in  i32 [B,max_pages_per_seq]
 *   prefix_len   in  i32 [B]
 *   pos_ids      in  i32 [B,W]   from wedlm_reorder
 *   out          out [B,W,Hq,D]  out[b,i,h] = softmax over {prefix} U {window rows j <= i} of
 *                                scale * <q~, k~>, times V
 *   kv_slot_idx  out i32 [B,W]   cache slot (page*page_size + offset) of physical row i, or NULL
 *   workspace        scratch of at least wedlm_window_attn_workspace_bytes(cfg) bytes
 *   status    in/out i32 [1] or NULL; WEDLM_STATUS_* bits are OR-ed in, never cleared
 */
int wedlm_window_attn(const wedlm_config_t* cfg, const void* q, const void* k, const void* v,
                      void* k_cache, void* v_cache, const int32_t* block_table,
                      const int32_t* prefix_len, const int32_t* pos_ids, void* out,
                      int32_t* kv_slot_idx, void* workspace, size_t workspace_bytes,
                      int32_t* status, void* stream);

/*
 * "Extend (K, V)" of Algorithm 1 as a call of its own: write rows i < count[b] of k, v to the
 * cache positions prefix_len[b] + i of sequence b.
 *   pos_ids   in i32 [B,W] or NULL.  Non-NULL: k is rotated at these positions before it is
 *                stored.  NULL: k is stored as given (already rotated).
 *   count     in i32 [B] or NULL (= W rows).
 *   kv_slot_idx out i32 [B,W] or NULL; rows >= count are set to -1.
 */
int wedlm_kv_append(const wedlm_config_t* cfg, const void* k, const void* v, const int32_t* pos_ids,
                    void* k_cache, void* v_cache, const int32_t* block_table,
                    const int32_t* prefix_len, const int32_t* count, int32_t* kv_slot_idx,
                    int32_t* status, void* stream);

/* Bytes of workspace wedlm_confidence_commit needs (uses batch, window, vocab, dtype, sample_temperature). */
size_t wedlm_confidence_workspace_bytes(const wedlm_config_t* cfg);

/*
 * Confidence over the vocabulary (entropy of Section 5.2), selection by Eq. 11, and the Commit /
 * Predict / Refill lines of Algorithm 1, for every sequence.
 *   logits         in  [B,W,V]  physical order; only mask rows (n_filled[b] <= i < window_len[b])
 *                               are read
 *   perm, n_filled, n_commit  in   from wedlm_reorder of the same window state
 *   window_tokens  in/out i32 [B,W] logical order
 *   filled         in/out u8  [B,W]
 *   prefix_len     in/out i32 [B]   += committed_count
 *   window_len     in/out i32 [B] or NULL (= W, not written)
 *   remaining_budget in/out i32 [B] or NULL (unlimited): fresh mask slots still allowed;
 *                               Refill appends min(committed_count, budget)
 *   argmax         out i32 [B,W] physical rows; -1 on rows that are not active masks
 *   maxprob, entropy, lse  out f32 [B,W]; NaN on rows that are not active masks (each may be NULL)
 *   committed_tokens out i32 [B,W] first committed_count[b] entries valid, rest -1
 *   committed_count  out i32 [B]
 *   filled_count     out i32 [B]  masks filled this step
 *   status        in/out i32 [1] or NULL; WEDLM_STATUS_WAIT_EXPIRED is OR-ed in if a bounded on-chip wait of the
 *                               streaming pass gave up (the statistics of some rows are then missing)
 * Order of operations per sequence: commit the n_commit leading slots; among the remaining
 * masks compute d = logical distance to the leftmost mask; select; if nothing is selected and a
 * mask exists, select the single best-scoring mask (leftmost on ties) so that decoding always
 * progresses; write arg-max tokens into the selected slots; shift the window left by n_commit;
 * append fresh masks.
 *
 * Sample() at a temperature (Algorithm 1 writes W[i] <- Sample(l_i); Section 6.1 evaluates at 0.1).  With
 * cfg->sample_temperature = T > 0 every slot filled in this step receives one draw from softmax(l / T)
 * instead of the arg-max: token = arg-max over v of l_v / T + g_v (lowest v on ties) with Gumbel noise
 * g_v = -ln(-ln u_v).  The uniforms are stateless, so a draw depends only on (seed, b, logical position,
 * token id):  mix(x): x ^= x>>16; x *= 0x7FEB352D; x ^= x>>15; x *= 0x846CA68B; x ^= x>>16 (mod 2^32);
 * key = mix(mix(seed_lo + 0x9E3779B9*b) ^ seed_hi ^ (0x85EBCA6B*pos)), pos = prefix_len[b] + logical slot;
 * u_v = ((mix(key ^ 0x9E3779B9*v) >> 9) + 0.5) * 2^-23.  Confidences (entropy, max-prob, lse) and the
 * selection are those of the raw logits; `argmax` reports the draw on the rows filled in this step and the
 * greedy arg-max on the other mask rows.  Only the selected rows are read a second time; within a row only
 * tokens whose logit is within 19.6 T of the maximum can win and only they are hashed, so the extra cost
 * grows with T.  Rows whose logits are all -inf are not supported with T > 0.  Advance the seed (or rely on
 * the positions advancing) between steps as the application requires; a given (seed, b, pos) always draws
 * the same noise.  The workspace is larger with T > 0 (wedlm_confidence_workspace_bytes accounts for it).
 */
int wedlm_confidence_commit(const wedlm_config_t* cfg, const void* logits, const int32_t* perm,
                            const int32_t* n_filled, const int32_t* n_commit,
                            int32_t* window_tokens, uint8_t* filled, int32_t* prefix_len,
                            int32_t* window_len, int32_t* remaining_budget,
                            int32_t* argmax, float* maxprob, float* entropy, float* lse,
                            int32_t* committed_tokens, int32_t* committed_count,
                            int32_t* filled_count, void* workspace, size_t workspace_bytes,
                            int32_t* status, void* stream);

/*
 * wedlm_confidence_commit fused with the LM head (Algorithm 1 takes its logits from Forward; here the last
 * step of that forward, logits = hidden . lm_head^T, is computed tile by tile on the tensor cores and reduced
 * in place, so the [B,W,V] logits never exist in memory).  bf16 only; hidden must be a multiple of 64.
 *   hidden        H
 *   hidden_states in  bf16 [B,W,H]  physical order (after the model's final norm)
 *   lm_head       in  bf16 [V,H]    row v = output embedding of token v
 *   tilt_ids      in  i32  [B,W] or NULL: the logit of token tilt_ids[b,i] of physical row i gets +tilt
 *                 (the additive tilt toward a target sequence of the end-to-end configuration); -1 = none
 *   all other arguments as in wedlm_confidence_commit; statistics come from fp32 logits (not rounded to bf16).
 *   cfg->sample_temperature must be 0 (the logits are never stored, so there is nothing to draw from after the
 *   selection): WEDLM_ERR_UNSUPPORTED otherwise.
 * Only the mask rows get logits (Algorithm 1 predicts from l_mask): their hidden states are first gathered into a
 * dense matrix inside the workspace, so the tensor-core tiles hold nothing but rows that count.
 * Workspace: wedlm_lmhead_confidence_workspace_bytes(cfg, hidden) bytes = the chunk partials
 * (batch*window*ceil(vocab/128)*16, an upper bound: the vocabulary tile width, 128..256, is chosen per launch), the
 * row map and the gathered hidden states (batch*window*hidden*2).
 *   status        in/out i32 [1] or NULL; WEDLM_STATUS_WAIT_EXPIRED if a bounded on-chip wait gave up
 */
size_t wedlm_lmhead_confidence_workspace_bytes(const wedlm_config_t* cfg, int32_t hidden);
int wedlm_lmhead_confidence_commit(const wedlm_config_t* cfg, int32_t hidden, const void* hidden_states,
                                   const void* lm_head, const int32_t* tilt_ids, float tilt,
                                   const int32_t* perm, const int32_t* n_filled, const int32_t* n_commit,
                                   int32_t* window_tokens, uint8_t* filled, int32_t* prefix_len,
                                   int32_t* window_len, int32_t* remaining_budget,
                                   int32_t* argmax, float* maxprob, float* entropy, float* lse,
                                   int32_t* committed_tokens, int32_t* committed_count,
                                   int32_t* filled_count, void* workspace, size_t workspace_bytes,
                                   int32_t* status, void* stream);

/*
 * wedlm_confidence_commit without a workspace argument, for hosts that must not allocate device
 * memory while they run.  (The paper has no counterpart to this call; it exists for deployment.)
 *
 * Who needs it: a serving process that gave nearly all of HBM to its KV-cache pool when it started,
 * so that a later cudaMalloc may fail and in any case stalls the device; or a decode loop that bans
 * allocator calls after warm-up.  Such a caller passes inputs and outputs exactly as for
 * wedlm_confidence_commit; the per-chunk partials go to an array of WEDLM_STATIC_SCRATCH_BYTES that
 * is part of the library image.  Every GPU context that loads the library holds that array until the
 * process exits.
 *
 *   - Limit: wedlm_confidence_workspace_bytes(cfg) must not exceed WEDLM_STATIC_SCRATCH_BYTES
 *     (4 MiB = 262144 chunk partials; batch*window*ceil(vocab/8192) for bf16, /4096 for fp32).
 *     Larger problems return WEDLM_ERR_STATIC_SCRATCH and launch nothing.
 *   - The first call on each device looks up the array's device address with that device current.
 *     The array is part of the library's device image, which the CUDA runtime places in device memory
 *     when it loads the module on that device; with lazy module loading that can be this first call.
 *     Make the first call early (at start-up, before memory becomes scarce) and before starting any
 *     stream capture.  Later calls query nothing and allocate nothing.
 *   - All calls on a device share the one array.  It keeps whatever the previous call left there;
 *     this routine needs none of it zeroed.  Two calls whose kernels can overlap on the GPU (different
 *     streams, no ordering between them) race on the array: serialise them.
 *   - The call performs no cudaMalloc / cudaFree and uses no allocating library routine.
 */
#define WEDLM_STATIC_SCRATCH_BYTES (4u << 20)
int wedlm_confidence_commit_static(const wedlm_config_t* cfg, const void* logits, const int32_t* perm,
                                   const int32_t* n_filled, const int32_t* n_commit,
                                   int32_t* window_tokens, uint8_t* filled, int32_t* prefix_len,
                                   int32_t* window_len, int32_t* remaining_budget,
                                   int32_t* argmax, float* maxprob, float* entropy, float* lse,
                                   int32_t* committed_tokens, int32_t* committed_count,
                                   int32_t* filled_count, int32_t* status, void* stream);

/*
 * Commit + shift + Refill of Algorithm 1 alone, for callers that did the selection themselves
 * and already wrote their fills into window_tokens / filled.
 *   n_commit in i32 [B]  slots to commit (from wedlm_reorder, i.e. counted BEFORE the fills of
 *                        this step: only those rows' K/V are cache-valid)
 * Other arguments as in wedlm_confidence_commit.
 */
int wedlm_window_refill(const wedlm_config_t* cfg, const int32_t* n_commit,
                        int32_t* window_tokens, uint8_t* filled, int32_t* prefix_len,
                        int32_t* window_len, int32_t* remaining_budget,
                        int32_t* committed_tokens, int32_t* committed_count, void* stream);

/*
 * One whole step of Algorithm 1 (reorder -> window attention -> confidence / commit / refill) for callers whose
 * step inputs live in HOST memory.  The call enqueues, on `stream`: the host-to-device copies of the inputs into
 * `workspace`, the kernels of wedlm_reorder, wedlm_window_attn and wedlm_confidence_commit, and the device-to-host
 * copies of the results; it returns without waiting (synchronise the stream before reading the outputs).  The largest
 * upload (logits, or hidden states) travels on a copy stream of the library while reorder and attention run, and is
 * joined back into `stream` in front of the confidence pass.  Use page-locked host memory, or the copies serialise
 * with the host.
 *   h_filled, h_window_tokens, h_prefix_len   host, in/out: the window state, updated in place by the step
 *   h_window_len, h_remaining_budget          host, in/out, each may be NULL (meaning as in wedlm_confidence_commit)
 *   h_block_table, h_q, h_k, h_v, h_logits    host, in: layouts as in wedlm_window_attn / wedlm_confidence_commit.
 *       Of the logits only the rows the step reads are sent: after reordering these are, per sequence, the physical
 *       rows [n_filled, window_len).  The CPU reads h_filled (and h_window_len) DURING this call to find them, so
 *       both must be final when it is made.
 *   k_cache, v_cache                          device, resident cache pool (the window's K/V are staged into it)
 *   h_committed_tokens [B,W], h_committed_count [B], h_filled_count [B] (may be NULL)   host, out
 *   workspace       device, wedlm_step_host_workspace_bytes(cfg) bytes, 16-byte aligned; holds the device copies of
 *                   every input, every intermediate and output of the three calls, and their scratch
 *   attn_out        host pointer to a device pointer, or NULL: receives the address (inside workspace) of the
 *                   attention output [B,W,Hq,D] for the layers that follow
 *   status          device i32 [1] or NULL
 */
size_t wedlm_step_host_workspace_bytes(const wedlm_config_t* cfg);
int wedlm_step_host(const wedlm_config_t* cfg, uint8_t* h_filled, int32_t* h_window_tokens, int32_t* h_prefix_len,
                    int32_t* h_window_len, int32_t* h_remaining_budget, const int32_t* h_block_table,
                    const void* h_q, const void* h_k, const void* h_v, const void* h_logits,
                    void* k_cache, void* v_cache, int32_t* h_committed_tokens, int32_t* h_committed_count,
                    int32_t* h_filled_count, void* workspace, size_t workspace_bytes, void** attn_out,
                    int32_t* status, void* stream);

/*
 * The same step with the LM head inside it (Algorithm 1, "(l, K_W, V_W) <- Forward(W, K, V)" followed by Predict):
 * instead of [B,W,V] logits the host hands over the hidden states of the window rows, and the output embedding
 * stays resident on the device.  The confidence pass is wedlm_lmhead_confidence_commit, so no logits ever exist
 * and the per-step traffic over the host link shrinks from B*W*V to B*W*hidden elements.  bf16 only.
 *   hidden            H (multiple of 64)
 *   h_hidden_states   host, in  bf16 [B,W,H] physical order (all rows are sent)
 *   lm_head           device, in bf16 [V,H]
 *   h_tilt_ids, tilt  host i32 [B,W] or NULL, and the additive tilt (as in wedlm_lmhead_confidence_commit)
 * Everything else as in wedlm_step_host; workspace of wedlm_step_host_lmhead_workspace_bytes(cfg, hidden) bytes.
 * cfg->sample_temperature must be 0.
 */
size_t wedlm_step_host_lmhead_workspace_bytes(const wedlm_config_t* cfg, int32_t hidden);
int wedlm_step_host_lmhead(const wedlm_config_t* cfg, int32_t hidden, uint8_t* h_filled, int32_t* h_window_tokens,
                           int32_t* h_prefix_len, int32_t* h_window_len, int32_t* h_remaining_budget,
                           const int32_t* h_block_table, const void* h_q, const void* h_k, const void* h_v,
                           const void* h_hidden_states, const void* lm_head, const int32_t* h_tilt_ids, float tilt,
                           void* k_cache, void* v_cache, int32_t* h_committed_tokens, int32_t* h_committed_count,
                           int32_t* h_filled_count, void* workspace, size_t workspace_bytes, void** attn_out,
                           int32_t* status, void* stream);

/*
 * Dual-Stream Masking for training (Section 4.2): the forward-pass pieces that need no data or weights.
 *
 * cfg fields used: batch = N sequences, window = block size B, n_q_heads, n_kv_heads, head_dim, page_size
 * (B must be a multiple of it; the tensor-core path needs page_size 16), dtype, rope_style, rope_theta,
 * softmax_scale, attn_impl, mask_token_id.  Every other field is ignored.
 * n_blocks = K = ceil(L / B) blocks per stream; Lp = K*B rows per stream (rows at or beyond L are padding).
 * All pointers are device pointers.
 *
 * wedlm_dual_stream_construct - Eq. 8-9 with block-wise masking and intra-block Topological Reordering:
 *   tokens   in  i32 [N,L]     the clean sequence
 *   masked   in  u8  [N,L]     non-zero = this logical position of the prediction stream is masked
 *   x_input  out i32 [N,2,Lp]  stream 0 = memory stream (tokens as they are), stream 1 = prediction stream:
 *                              inside every block the observed tokens first, the masked ones (mask_token_id)
 *                              last, both in ascending logical order; padding rows carry mask_token_id
 *   p_input  out i32 [N,2,Lp]  logical position of every physical row; both streams use positions 0..L-1
 *   is_mask  out u8  [N,Lp] or NULL   prediction-stream rows that are masked (the rows that enter the loss)
 *   n_observed out i32 [N,K] or NULL  observed tokens per block
 *
 * wedlm_dual_stream_attn - attention under the pattern of the "Attention Pattern" paragraph: a row of block k,
 * in either stream, sees the memory-stream rows at positions below k*B and the rows of its own block that are
 * physically not later than itself (for the memory stream this is plain causal attention).  RoPE at p_input.
 *   q        in  [N,2,Lp,Hq,D]   physical order (stream 0 memory, stream 1 prediction), un-rotated
 *   k, v     in  [N,2,Lp,Hkv,D]
 *   out      out [N,2,Lp,Hq,D]   rows of padding slots are computed like any other row and carry no meaning
 *   workspace    wedlm_dual_stream_workspace_bytes(cfg, n_blocks) bytes, 16-byte aligned: rotated K and V of
 *                both streams in page layout, one page table per (sequence, stream, block), scratch
 *   status   in/out i32 [1] or NULL, WEDLM_STATUS_* bits
 * Padding rows must hold finite numbers.  Returns WEDLM_ERR_UNSUPPORTED if B is not a multiple of page_size.
 */
int wedlm_dual_stream_construct(const wedlm_config_t* cfg, int32_t n_blocks, int32_t seq_len,
                                const int32_t* tokens, const uint8_t* masked, int32_t* x_input,
                                int32_t* p_input, uint8_t* is_mask, int32_t* n_observed, void* stream);
size_t wedlm_dual_stream_workspace_bytes(const wedlm_config_t* cfg, int32_t n_blocks);
int wedlm_dual_stream_attn(const wedlm_config_t* cfg, int32_t n_blocks, const void* q, const void* k,
                           const void* v, const int32_t* p_input, void* out, void* workspace,
                           size_t workspace_bytes, int32_t* status, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* WEDLM_H_ */
