/*
 * stairs.h - C-ABI of the B200 (sm_100a) "stairs" assisted greedy generation library.
 *
 * Method (D. Grigaliunas and M. Lukosevicius, "Inference acceleration for large language
 * models using 'stairs' assisted greedy generation", Section 3.3, Fig. 4 and Fig. 5): a small
 * assistant model greedily drafts k tokens; the k+1 sub-sequences
 * context+draft[:r], r = 0..k, are given to the main model as one batch; the main
 * model's greedy token is taken for every row; rows are then walked in order and a
 * drafted token is kept only while it equals the main model's token for the
 * previous row.  The output is token for token the main model's own greedy output
 * (Sections 1 and 5), produced in fewer main-model iterations.
 *
 * Because row r is a prefix of row r+1, the k+1 rows hold only k+1 distinct new
 * positions over a shared, already cached prefix.  The library therefore runs the
 * batch as k+1 new positions with a staircase mask (row r sees the prefix and new
 * positions 0..r) over a paged KV cache.
 *
 * Conventions
 *  - Every function returns a stairs_status (0 = success) and never throws or aborts;
 *    stairs_last_error() gives a text for the last failure on that context.
 *  - "_host" pointers are host memory, "_dev" pointers are device memory on the
 *    context's device.  The caller owns every buffer it passes in.
 *  - Weights are device pointers owned by the caller, borrowed until stairs_destroy().
 *    Every matrix is row-major [out_features, in_features]; matrices are fp32
 *    (wdtype 0) or bf16 (wdtype 1); norm gains/biases are always fp32.  There are no
 *    linear biases.
 *  - The library allocates no device memory: KV pages, activations and status words
 *    live in the caller's workspace (size from stairs_workspace_bytes()).
 *  - stairs_prefill / stairs_draft / stairs_validate enqueue work on the borrowed
 *    stream and return without waiting; stairs_generate, stairs_validate_host,
 *    stairs_sequence and stairs_sync wait.  A context is not thread-safe.
 *  - Request state (the committed token sequence and its length) lives on the device.
 */
#ifndef STAIRS_H_
#define STAIRS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct stairs_ctx stairs_ctx; /* opaque, library-owned */

enum stairs_status {
  STAIRS_OK = 0,
  STAIRS_EINVAL = 1,       /* bad argument or configuration                         */
  STAIRS_ENOSPC = 2,       /* workspace too small, KV pool exhausted, sequence full */
  STAIRS_ESTATE = 3,       /* call order (e.g. validate before prefill)             */
  STAIRS_ECUDA = 4,        /* a CUDA call failed                                    */
  STAIRS_ETIMEOUT = 5,     /* a bounded device-side wait expired                    */
  STAIRS_EUNSUPPORTED = 6  /* shape outside what the kernels handle                 */
};

/* Transformer architecture (decoder-only, pre-norm).  norm: 0 LayerNorm (gain+bias),
 * 1 RMSNorm (gain).  act: 0 two-matrix MLP with exact GELU, 1 SwiGLU (gate, up, down).
 * pos: 0 learned absolute position embedding added to the token embedding, 1 rotary
 * embedding on q and k (element i pairs with i + head_dim/2, angle pos * theta^(-2i/hd)).
 * n_heads must be a multiple of n_kv_heads (grouped-query attention). */
typedef struct stairs_model {
  int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ff, vocab, max_pos;
  int32_t norm, act, pos;
  float rope_theta, norm_eps;
  int32_t wdtype; /* 0 fp32, 1 bf16 */
} stairs_model;

typedef struct stairs_layer_w {
  const void *norm1_w, *norm1_b; /* [d_model] fp32; bias NULL for RMSNorm           */
  const void *wq, *wk, *wv;      /* [Hq*hd, d], [Hkv*hd, d], [Hkv*hd, d]            */
  const void *wo;                /* [d, Hq*hd]                                      */
  const void *norm2_w, *norm2_b;
  const void *w_gate_or_fc1;     /* [d_ff, d]                                       */
  const void *w_up;              /* [d_ff, d]; NULL for the two-matrix MLP          */
  const void *w_down_or_fc2;     /* [d, d_ff]                                       */
} stairs_layer_w;

typedef struct stairs_weights {
  const void *tok_emb;                     /* [vocab, d]                            */
  const void *pos_emb;                     /* [max_pos, d]; NULL with rotary        */
  const void *final_norm_w, *final_norm_b; /* fp32                                  */
  const void *lm_head;                     /* [vocab, d]                            */
  const stairs_layer_w *layers;            /* host array of n_layers entries        */
} stairs_weights;

typedef struct stairs_config {
  uint32_t struct_size;   /* sizeof(stairs_config), for ABI checking                 */
  stairs_model target;    /* main model                                              */
  stairs_model draft;     /* assistant; must share d_model, vocab, wdtype and the
                             norm/act/pos family with the target; n_layers 0 = none  */
  int32_t max_requests;   /* request slots 0..max_requests-1                         */
  int32_t max_seq_len;    /* tokens per request, prompt + generated                  */
  int32_t k_max;          /* largest draft length per validate call (0..63)          */
  int32_t kv_page_tokens; /* tokens per KV page: 16, 32, 64 or 128                   */
  int32_t kv_pages;       /* pages in the pool; 0 = enough for every slot to reach
                             max_seq_len                                             */
  int32_t prefill_chunk;  /* rows per prefill pass; 0 = 256                          */
  int32_t device;         /* CUDA device ordinal                                     */
  int32_t gemm_impl;      /* 0 = best available (bf16: one persistent kernel per pass
                             of <= 64 rows, tensor-core GEMMs otherwise), 1 = force
                             the plain SIMT kernels (reference path for cross-checks),
                             2 = tensor-core GEMMs, one launch per GEMM               */
  void *stream;           /* cudaStream_t, borrowed; NULL = default stream           */
  void *workspace;        /* device memory, 256-byte aligned                         */
  size_t workspace_bytes;
  uint64_t wait_limit_cycles; /* bound for device-side waits; 0 = library default    */
} stairs_config;

typedef struct stairs_stats {
  int32_t iterations;  /* validate calls made                                       */
  int32_t drafted;     /* drafted tokens offered                                    */
  int32_t accepted;    /* drafted tokens kept                                       */
  int32_t emitted;     /* new tokens produced (before truncation to max_new)        */
  float prefill_ms, draft_ms, validate_ms, total_ms; /* device time per phase       */
} stairs_stats;

/* Bytes of workspace stairs_init() needs for this configuration (0 on a bad config). */
size_t stairs_workspace_bytes(const stairs_config *cfg);

/* Creates a context.  `target` and `draft` describe device weight pointers; `draft` may
 * be NULL when cfg->draft.n_layers == 0.  A draft that is the target's first layers
 * (early exit) is expressed by pointing its layer entries at the target's tensors.
 * The workspace's state area is cleared.  Errors: EINVAL, ENOSPC, EUNSUPPORTED, ECUDA. */
int stairs_init(const stairs_config *cfg, const stairs_weights *target,
                const stairs_weights *draft, stairs_ctx **out);

/* Starts request `req` from a prompt of n_prompt >= 2 tokens (host memory): stores the
 * tokens as the request's sequence and computes K/V of prompt[0..n_prompt-2] in both
 * models' caches (the last prompt token is the first row of the next validate call).
 * Any earlier state of the slot is dropped.  Errors: EINVAL, ENOSPC. */
int stairs_prefill(stairs_ctx *ctx, int req, const int32_t *prompt_host, int n_prompt);

/* Assistant step (Section 3.3, first step): greedily drafts k tokens after the request's
 * committed sequence with the draft model and writes them to draft_dev[0..k-1].  Does
 * not change the committed sequence.  Errors: EINVAL, ESTATE, ENOSPC. */
int stairs_draft(stairs_ctx *ctx, int req, int k, int32_t *draft_dev);

/* Main-model stairs pass (Section 3.3, Fig. 4 and Fig. 5) for n_req requests at once.
 * Request i (slot req_ids_host[i]) contributes k_host[i]+1 rows: its committed sequence
 * followed by the first r tokens of draft_dev[i*k_max .. i*k_max+k_host[i]-1].
 *   target_tokens_dev[i*(k_max+1) + r]  main model's greedy token for row r (lowest id
 *                                       on ties), r = 0..k_host[i]
 *   accept_len_dev[i]                   number of drafted tokens kept: the first r with
 *                                       draft[r] != target_tokens[r], or k_host[i]
 *   logits_dev_or_null                  if not NULL, fp32 [total_rows, vocab] scores of
 *                                       every row, rows ordered request by request
 * commit != 0 appends the accept_len+1 new tokens (kept drafts, then the main model's
 * token) to each request's sequence; commit == 0 leaves all request state unchanged, so
 * the call is a pure function of (cache, draft).  k = 0 is plain greedy decoding.
 * Errors: EINVAL, ESTATE, ENOSPC. */
int stairs_validate(stairs_ctx *ctx, int n_req, const int32_t *req_ids_host,
                    const int32_t *k_host, const int32_t *draft_dev,
                    int32_t *target_tokens_dev, int32_t *accept_len_dev,
                    float *logits_dev_or_null, int commit);

/* The same pass with host buffers: copies the drafts in, runs, copies target tokens and
 * accept lengths out and waits.  draft_host is [n_req, k_max], target_tokens_host
 * [n_req, k_max+1], accept_len_host [n_req]. */
int stairs_validate_host(stairs_ctx *ctx, int n_req, const int32_t *req_ids_host,
                         const int32_t *k_host, const int32_t *draft_host,
                         int32_t *target_tokens_host, int32_t *accept_len_host, int commit);

/* Whole generation (Section 3.2 cycle with the Section 3.3 step): prefill, then repeat
 * {draft min(k, remaining-1) tokens, validate with commit} until max_new tokens exist or
 * `eos` (if >= 0) was emitted.  Writes the new tokens to out_host[0..*n_out-1]
 * (capacity max_new).  k = 0 generates with the main model alone.  Waits for completion.
 * Errors: as above. */
int stairs_generate(stairs_ctx *ctx, int req, const int32_t *prompt_host, int n_prompt,
                    int k, int max_new, int32_t eos, int32_t *out_host, int32_t *n_out,
                    stairs_stats *stats_or_null);

/* The same generation with a draft length that follows the acceptance, the schedule of the
 * sequential assisted generation the paper compares stairs with (Section 3.2; Section 4.1: that
 * method sets the length dynamically): the first iteration drafts k_first (>= 1) tokens; after an
 * iteration that kept every drafted token the next one drafts two more (at most k_max), after
 * any other iteration one fewer (at least one).  Checking the drafts left to right in one causal
 * pass is what the deduplicated stairs pass does anyway, so the two methods differ only in this
 * schedule here; the output is still the main model's own greedy output.  Errors: as above. */
int stairs_generate_adaptive(stairs_ctx *ctx, int req, const int32_t *prompt_host, int n_prompt,
                             int k_first, int max_new, int32_t eos, int32_t *out_host,
                             int32_t *n_out, stairs_stats *stats_or_null);

/* Copies the request's committed sequence length (and, if seq_host != NULL, up to
 * capacity tokens of the sequence) to the host.  Waits. */
int stairs_sequence(stairs_ctx *ctx, int req, int32_t *seq_host, int capacity, int32_t *n_seq);

/* Rolls request `req` back to its first n_tokens committed tokens (2 <= n_tokens <= current
 * length; the host must know the current length, e.g. from stairs_sequence).  Cache entries
 * past the new end are simply overwritten by later calls.  Enqueued on the stream. */
int stairs_truncate(stairs_ctx *ctx, int req, int n_tokens);

/* Waits for the stream and reports a device-side failure recorded since the last call
 * (ETIMEOUT if a bounded wait expired). */
int stairs_sync(stairs_ctx *ctx);

/* Number of kernels this context has launched so far. */
int64_t stairs_launch_count(const stairs_ctx *ctx);

/* Frees the slot's KV pages and forgets its sequence. */
int stairs_reset(stairs_ctx *ctx, int req);

int stairs_destroy(stairs_ctx *ctx);

/* Text of the last error on this context ("" if none); ctx NULL gives the last error of
 * a failed stairs_init / stairs_workspace_bytes on this thread. */
const char *stairs_last_error(const stairs_ctx *ctx);

/* Greedy token per row and accept length per request, computed from logits the caller
 * already holds - for callers that must not allocate device memory at all.  (The paper has
 * no counterpart to this entry point; it exists for the callers described here.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a memory pool that
 * owns the whole device, in a latency-critical section where an allocation would
 * synchronise the device, or in a plug-in that is only handed finished buffers.  Such a
 * caller cannot create a context either, because a context needs a workspace.  This call
 * takes only inputs and outputs; its one piece of scratch (one packed 64-bit argmax key per
 * row) lives in a fixed array inside the library, 8 KB, which every GPU that loads the
 * library holds until the process exits.  It calls no cudaMalloc/cudaFree and no allocating
 * library routine.
 *
 *   logits_dev        fp32 [n_rows, ld], row r of request i at row off(i)+r, where off(i) is
 *                     the sum of k_host[j]+1 over j < i; n_rows = sum of k_host[i]+1
 *   draft_dev         int32 [n_req, k_max]
 *   target_tokens_dev int32 [n_req, k_max+1]   (out) argmax of each row, lowest id on ties
 *   accept_len_dev    int32 [n_req]            (out) first r with draft[r] != target[r], else k
 *
 * Limits: n_rows <= STAIRS_STATIC_MAX_ROWS, 1 <= n_req <= STAIRS_STATIC_MAX_REQ,
 * 0 <= k_host[i] <= k_max <= 63; anything larger returns STAIRS_ENOSPC or STAIRS_EINVAL with
 * a text in stairs_last_error(NULL).  Work is enqueued on `stream` (NULL = default stream)
 * of the current device.  The first call on a device looks up the array's device address
 * (cudaGetSymbolAddress); make that first call before starting any stream capture.  All
 * calls share the array and it keeps the previous call's keys: each call clears the part it
 * uses before use, and two calls that overlap on the GPU (different streams, no ordering
 * between them) race on it - order them. */
#define STAIRS_STATIC_MAX_ROWS 1024
#define STAIRS_STATIC_MAX_REQ 64
int stairs_accept_static(const float *logits_dev, int vocab, int ld, int n_req, const int32_t *k_host,
                         const int32_t *draft_dev, int k_max, int32_t *target_tokens_dev,
                         int32_t *accept_len_dev, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* STAIRS_H_ */
