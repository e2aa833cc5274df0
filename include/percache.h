/*
 * percache.h — C ABI of the reuse-prefill library (one model, one GPU per handle).
 *
 * The operation is the one PerCache's QKV-cache tier performs at query time
 * (paper Section 3.2.2 "QKV Cache Reuse", Appendix B.1 "Inference implementation
 * details"): a prompt is an ordered list of knowledge chunks followed by the
 * user's query tokens; tensors of chunks already in the cache are loaded and
 * concatenated in order, the rows they cover are dropped from every block's
 * attention input, projection and position encoding run on the remaining rows
 * only (each at its true position in the full sequence), the computed tensors are
 * concatenated with the loaded ones and the rest of the block proceeds normally.
 * Tensors computed for chunks that were not cached are sliced per chunk and kept
 * (Section 3.2.1, cache slicer).
 *
 * Deliberate differences from the paper's prototype, all documented in the design
 * notes: only K and V are cached (bf16, 16-token pages, K stored before rotation
 * and rotated to its slot's position when gathered); a chunk may hit at any place
 * of the list, not only as part of a prefix; only the new rows (missed chunks and
 * query tokens) continue through the blocks and are returned.
 *
 * General rules
 *  - Every function returns 0 (PERCACHE_OK) or a negative PERCACHE_E_* code; nothing
 *    throws or aborts across this boundary.  percache_strerror() names a code.
 *  - A handle is not thread-safe.  All device work of a handle runs on the stream
 *    given at creation; calls return after that work has finished.
 *  - A call that is refused before its device work starts (every argument, capacity and space check) leaves the
 *    store exactly as it was, also when eviction is on: victims are chosen first but dropped only when the kernels
 *    are about to write.  A call whose device work fails (PERCACHE_E_CUDA, PERCACHE_E_DEVICE_TIMEOUT) stores
 *    nothing and leaves the store consistent, but chunks it evicted to make room stay evicted, and the assembled
 *    context of the previous call is forgotten (percache_decode then returns PERCACHE_E_INVAL).
 *  - Number formats: the store is bf16, the residual stream fp32, every operand of a projection or of the attention
 *    is fp16 with fp32 accumulation.  fp16 carries magnitudes up to 65504; every conversion to fp16 inside the
 *    library saturates (a larger value becomes +-65504, never infinity), so out-of-range weights, cached values or
 *    activations (a SwiGLU product, a rotated key) are clipped and the call stays finite.  Results are only
 *    meaningful while normed activations, projections and SwiGLU products stay within that range; bf16 values below
 *    2^-24 in magnitude flush to zero as operands.
 *  - The library never frees or keeps caller memory: every caller buffer may be
 *    released as soon as the call returns.
 *  - There is no CPU fallback: without a CUDA device every call that needs one fails
 *    with PERCACHE_E_CUDA.
 */
#ifndef PERCACHE_H_
#define PERCACHE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define PERCACHE_API __attribute__((visibility("default")))
#else
#define PERCACHE_API
#endif

#define PERCACHE_OK                 0
#define PERCACHE_E_INVAL           -1   /* bad argument (NULL, negative size, unsupported shape)        */
#define PERCACHE_E_NOMEM           -2   /* host or device allocation failed                            */
#define PERCACHE_E_NOSPACE         -3   /* the paged store has too few free pages                      */
#define PERCACHE_E_EXISTS          -4   /* chunk id already stored                                     */
#define PERCACHE_E_LEN_MISMATCH    -5   /* chunk id stored with a different token count                */
#define PERCACHE_E_MISS_NO_INPUT   -6   /* chunk is not stored and no hidden states were given for it  */
#define PERCACHE_E_CAPACITY        -7   /* prompt / batch exceeds a limit fixed at creation            */
#define PERCACHE_E_DEVICE_TIMEOUT  -8   /* a bounded wait inside a kernel ran out; results are invalid */
#define PERCACHE_E_CUDA            -9   /* a CUDA runtime / driver call failed                         */
#define PERCACHE_E_NOTFOUND        -10  /* chunk id not stored (has / drop)                            */

#define PERCACHE_PAGE_TOKENS 16

/* percache_config_t.flags */
#define PERCACHE_FLAG_REFERENCE_KERNELS  1u  /* debugging aid: run every GEMM and the attention with the plain
                                                one-thread-per-output CUDA kernels instead of the tcgen05 ones */
#define PERCACHE_FLAG_PHASE_TIMING       2u  /* record CUDA events around every kernel class (see stats)       */
#define PERCACHE_FLAG_REFERENCE_ATTENTION 4u /* debugging aid: plain attention kernel, tcgen05 GEMMs            */
#define PERCACHE_FLAG_SINGLE_CTA_GEMM   16u  /* debugging aid: never run a GEMM on CTA pairs (256 x 256 tiles)     */
#define PERCACHE_FLAG_NO_SMALL_ROW_KERNELS 32u /* debugging aid: calls with at most 8 rows (decode) use the tcgen05
                                                GEMMs like any other instead of the weight-streaming kernels     */
#define PERCACHE_FLAG_EVICT_LFU          8u  /* when the store is full, evict least-frequently-used chunks instead
                                                of failing with PERCACHE_E_NOSPACE (see percache_set_store_limit)  */

#define PERCACHE_FLAG_GATHER_FREE       128u  /* take the gather-free form of percache_prefill whenever it is possible
                                                (see percache_prefill), not only when the cached part dominates   */
#define PERCACHE_FLAG_ALWAYS_GATHER     256u  /* never take it: always assemble the contiguous context              */
#define PERCACHE_FLAG_PAPER_MODE         64u  /* creation only: the handle works exactly as the paper states the scheme
                                                (see "Paper-faithful mode" below)                                 */

typedef struct percache percache_t;   /* opaque */

typedef struct {
  int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn;
  float   rope_theta, rms_eps;
  int32_t page_tokens;              /* must be PERCACHE_PAGE_TOKENS                                         */
  int64_t pool_pages;               /* capacity of the paged store, in pages (each page: 16 tokens, all
                                       layers, K and V)                                                    */
  int32_t max_prompt_tokens;        /* longest prompt (chunks + query); also the largest RoPE position + 1  */
  int32_t max_batch_prompts;        /* most prompts in one percache_prefill call                            */
  int64_t max_batch_ctx_tokens;     /* most context tokens (sum of prompt lengths) in one call              */
  int64_t max_batch_new_rows;       /* most new rows (missed-chunk tokens + query tokens) in one call       */
  int32_t device;                   /* CUDA device ordinal                                                  */
  void*   stream;                   /* cudaStream_t of the caller, or NULL for the default stream           */
  uint32_t flags;                   /* PERCACHE_FLAG_*                                                      */
} percache_config_t;

/* One layer's parameters: bf16, row-major [out_features][in_features] (norm gains: [d_model]).
 * Host or device pointers (see weights_on_device); copied during percache_create. */
typedef struct {
  const void *attn_norm, *wq, *wk, *wv, *wo, *ffn_norm, *w_gate, *w_up, *w_down;
} percache_layer_weights_t;

/* Create a handle: allocates the paged store, work buffers and a private copy of the weights on
 * cfg->device.  Supported shapes: head_dim 128; d_model, d_ffn multiples of 64; n_q_heads an even multiple
 * of n_kv_heads (the attention kernel pairs the query heads of a KV head).  Device allocation failure -> PERCACHE_E_NOMEM; the handle is not created. */
PERCACHE_API int percache_create(const percache_config_t* cfg, const percache_layer_weights_t* layers /*[n_layers]*/,
                    int32_t weights_on_device, percache_t** out);

/* Free everything the handle owns.  NULL is accepted. */
PERCACHE_API int percache_destroy(percache_t* h);

/* Insert a chunk's unrotated K and V for all layers (what a prefill of that chunk collected; paper
 * Section 3.2.1).  k, v: bf16 [n_layers][n_tokens][n_kv_heads][head_dim], host or device memory as
 * ptr_is_device says.  Copied into ceil(n_tokens/16) pages before return.  An id that is already stored
 * is not overwritten: PERCACHE_E_EXISTS. */
PERCACHE_API int percache_put_chunk_kv(percache_t* h, uint64_t chunk_id, int32_t n_tokens,
                          const void* k, const void* v, int32_t ptr_is_device);

/* How the chunks of a prompt are matched against the store.
 *  PERCACHE_MATCH_CHUNK_ID     a chunk hits when its id is stored, at whatever place of the list it appears (the
 *                              K/V of layers > 0 were then computed in some other context).
 *  PERCACHE_MATCH_PREFIX_PATH  the paper's rule (Section 3.2.2): entries are nodes of a tree whose paths are chunk
 *                              lists; the first chunk is looked up, then the second as its child, and so on until
 *                              the first mismatch; every later chunk is computed.  The store key of a node is
 *                              percache_path_key() of the ids from the first chunk to that node, and the chunks a
 *                              call computes are stored under their path keys.  Reuse then equals full prefill.
 * Path keys and plain chunk ids share the handle's one 64-bit key space (two keys collide with probability 2^-64);
 * percache_has_chunk / _drop_chunk / _chunk_info / _get_chunk_kv take whichever key an entry was stored under. */
#define PERCACHE_MATCH_CHUNK_ID    0
#define PERCACHE_MATCH_PREFIX_PATH 1

/* Key of the tree node reached by the path chunk_ids[0..n-1] (n = 0: the root's seed). */
PERCACHE_API uint64_t percache_path_key(const uint64_t* chunk_ids, int32_t n);

/* A prompt: ordered chunk list plus query tokens (paper Section 3, system overview). */
typedef struct {
  int32_t n_chunks;
  const uint64_t* chunk_ids;            /* host [n_chunks]                                                 */
  const int32_t*  chunk_len;            /* host [n_chunks], tokens per chunk (> 0)                          */
  const void* const* chunk_hidden;      /* host [n_chunks] of pointers to bf16 [len][d_model] layer-0 input;
                                           an entry (or the whole array) may be NULL for a chunk expected to
                                           hit; NULL for a chunk that misses -> PERCACHE_E_MISS_NO_INPUT    */
  int32_t n_query;                      /* >= 0                                                             */
  const void* query_hidden;             /* bf16 [n_query][d_model]                                          */
  int32_t hidden_on_device;             /* 1: chunk_hidden[i] and query_hidden point to device memory       */
  int32_t match_mode;                   /* PERCACHE_MATCH_*                                                 */
  int32_t reuse_tail_drop;              /* PERCACHE_MATCH_PREFIX_PATH only, else must be 0 (paper Appendix B,
                                           tokenisation paragraph): the tensors of the last reuse_tail_drop tokens
                                           of the final matched chunk are not reused; those tokens are computed
                                           from chunk_hidden (which must then be given for that chunk) and are not
                                           stored again.  0 <= drop <= that chunk's length                      */
} percache_prompt_t;

typedef struct {
  float*   out_hidden;         /* caller-allocated fp32 [out_capacity_rows][d_model]: final residual stream of
                                  the new rows, in prompt order (no final norm)                             */
  int64_t  out_capacity_rows;  /* fewer than n_new -> PERCACHE_E_CAPACITY                                   */
  int32_t  out_on_device;      /* 1: out_hidden is device memory                                            */
  uint8_t* hit_mask;           /* caller-allocated host [n_chunks] or NULL; 1 = served from the store       */
  int32_t  n_new, n_total;     /* written by the call: new rows and total context tokens of this prompt     */
} percache_result_t;

/* Reuse-prefill of a batch of independent prompts (paper Section 3.2.2, Appendix B.1).
 * Hits are decided against the store as it is when the call starts: a chunk hits when its id is stored
 * with the same length (different length -> PERCACHE_E_LEN_MISMATCH).  On success every missed chunk is
 * stored (its K/V as computed inside its prompt; if two prompts of the batch miss the same id, the
 * first prompt's is kept) and query tokens are not.  Too few free pages -> PERCACHE_E_NOSPACE.
 * Synchronous: returns after the stream has drained.
 * Two forms compute the same result.  The default one copies every cached token's K and V into a contiguous context
 * (K rotated to its position there) and lets the attention read that.  The gather-free one leaves them in their
 * pages: the attention walks the prompt's page table, rotates K as it loads it and reads V where it is, so the fetch
 * and its traffic disappear; there P and V enter the second attention product as bf16 (the store's format) instead
 * of fp16.  It is taken when the batch has at least 8 cached tokens per new row and no prompt more than 256 new rows
 * (or PERCACHE_FLAG_GATHER_FREE is set), every chunk length and reuse_tail_drop is a multiple of 16 and
 * PERCACHE_FLAG_ALWAYS_GATHER is not set; rows that are not stored (query tokens) then occupy pages of the store for
 * the duration of the call (they count against the store limit).  After a gather-free call there is no assembled
 * context and percache_debug_read_ctx returns PERCACHE_E_INVAL.  If a decode reserve is set, those pages (and page
 * slots for the tokens to be decoded) stay occupied after the call and the first percache_decode step runs the
 * skipped fetch over all slots, which builds the context and gives the pages back; with PERCACHE_FLAG_GATHER_FREE
 * set at that time the decode steps instead read the pages themselves (K rotated on load; each step's attention is
 * about 40 % slower, no context is ever built, the pages stay occupied).  Any later percache_prefill call, successful
 * or not, gives the pages back and ends that batch's decode steps.  Without a decode reserve percache_decode after a
 * gather-free call returns PERCACHE_E_INVAL. */
PERCACHE_API int percache_prefill(percache_t* h, const percache_prompt_t* prompts, int32_t n_prompts,
                     percache_result_t* results /*[n_prompts]*/);

/* Paper-faithful mode (a handle created with PERCACHE_FLAG_PAPER_MODE).  percache_prefill then computes what the
 * paper describes, without the three departures listed at the top of this file:
 *  - matching is the prefix-tree walk (every prompt must use PERCACHE_MATCH_PREFIX_PATH, Section 3.2.2);
 *  - a node holds the chunk's Q, K and V of every block (Sections 3.2.1 and 5.3: all three projections are skipped
 *    for cached rows), bf16, Q and K after position encoding at the positions the node has on its path;
 *  - all L_total rows of the prompt run through every block; the L_pre rows of the matched chain skip only the
 *    projections and the position encoding, for the others the position counter starts at L_pre (Appendix B.1);
 *    reuse_tail_drop shortens L_pre by the tail of the chain's last node (Appendix B, tokenisation paragraph);
 *  - out_hidden receives ALL n_total rows (out_capacity_rows >= n_total); n_new still counts the computed rows.
 * Q, K (both rotated) and V of every row are rounded to bf16 before the attention uses them, loaded or computed
 * alike, because that is what the store holds.  The attention reads Q, K and V of all rows straight from the pages
 * through a per-prompt page table (nothing is gathered or rotated at query time).  Restrictions of this mode: hidden
 * states must be given for every chunk (the whole prompt is embedded); chunk lengths and reuse_tail_drop must be
 * multiples of 16 (pages are copied whole; the query may have any length); max_batch_new_rows bounds the rows of a
 * batch, i.e. the sum of n_total; percache_put_chunk_kv, _put_chunk_synthetic and percache_decode return
 * PERCACHE_E_INVAL; the debugging flags that select the plain kernels are refused.  percache_get_chunk_kv returns the
 * node's K (rotated) and V, percache_get_chunk_q its Q: bf16 [n_layers][n_tokens][n_q_heads][head_dim], host. */
PERCACHE_API int percache_get_chunk_q(percache_t* h, uint64_t chunk_id, void* q_host);

/* Decode step after a prefill (paper Section 2.1: inference is a prefill over the prompt followed by a decode
 * stage that produces one token at a time, attending to the keys and values of everything before it).
 * One token per prompt of the LAST percache_prefill call: hidden is bf16 [n_prompts][d_model] (row b continues
 * prompt b; host or device memory per hidden_on_device), n_prompts must equal that call's.  Row b is at position
 * n_total_b + (tokens decoded so far); it runs through every block like a new row of the prefill and attends to
 * the prompt's assembled context plus itself; its rotated K and its V are appended to that context (they are
 * not chunk content: nothing is stored).  out_hidden: caller-allocated fp32 [n_prompts][d_model], final residual
 * stream (no final norm).  The context keeps percache_set_decode_reserve() free slots behind every prompt; a
 * prompt that has used them all, or would pass max_prompt_tokens, -> PERCACHE_E_CAPACITY and nothing changes.
 * Any later percache_prefill starts a new batch and discards the decoded tokens.  Synchronous. */
PERCACHE_API int percache_decode(percache_t* h, int32_t n_prompts, const void* hidden, int32_t hidden_on_device,
                    float* out_hidden, int32_t out_on_device);

/* Context slots kept free behind every prompt of later percache_prefill calls, so that percache_decode can
 * append tokens (default 0: no decode).  A batch needs sum(n_total) + n_prompts * tokens_per_prompt <=
 * max_batch_ctx_tokens, else percache_prefill returns PERCACHE_E_CAPACITY. */
PERCACHE_API int percache_set_decode_reserve(percache_t* h, int32_t tokens_per_prompt);

/* *n_tokens = stored length, or PERCACHE_E_NOTFOUND. n_tokens may be NULL. */
PERCACHE_API int percache_has_chunk(percache_t* h, uint64_t chunk_id, int32_t* n_tokens);

/* Remove a chunk and free its pages (used to restore the cache state between timed runs). */
PERCACHE_API int percache_drop_chunk(percache_t* h, uint64_t chunk_id);

/* Capacity management (paper Section 3.2.1: a retrieval counter per cached entry, least-frequently-used
 * eviction under a configurable storage limit).  Every stored chunk counts the prompts that used it: 1 when a
 * prompt first stores it (or percache_put_chunk_* inserts it), +1 for every later prompt occurrence that hits it.
 * With PERCACHE_FLAG_EVICT_LFU, a call that needs more pages than the limit leaves free evicts chunks in order
 * of (count ascending, insertion order ascending), never one the calling batch itself hits, until the new pages
 * fit; if they cannot fit the call fails with PERCACHE_E_NOSPACE and nothing is evicted.  Eviction is applied
 * after every host-side check of the call has passed.
 * percache_set_store_limit: limit in pages, 1..pool_pages (default pool_pages).  Lowering it below the current
 * use evicts at once (LFU order) when the flag is set, else fails with PERCACHE_E_NOSPACE. */
PERCACHE_API int percache_set_store_limit(percache_t* h, int64_t pages);

/* *n_tokens = stored length, *retrievals = the chunk's counter; either pointer may be NULL. */
PERCACHE_API int percache_chunk_info(percache_t* h, uint64_t chunk_id, int32_t* n_tokens, int64_t* retrievals);

/* Read a stored chunk back: k, v host buffers bf16 [n_layers][n_tokens][n_kv_heads][head_dim]. */
PERCACHE_API int percache_get_chunk_kv(percache_t* h, uint64_t chunk_id, void* k_host, void* v_host);

/* Fill a new chunk with the synthetic integer pool values of the batched-serving workload:
 * element e of (chunk, which in {K=0,V=1}, layer) takes the 64-bit counter
 *   ((((seed << 20) + chunk_id) * 2 + which) * 64 + layer) << 24) + e
 * through the SplitMix64 output function, and the value (b0 + b1 + b2 + b3 - 126) / 64 with b_i the four
 * lowest 6-bit fields of the result (exact in bf16).  Same errors as percache_put_chunk_kv. */
PERCACHE_API int percache_put_chunk_synthetic(percache_t* h, uint64_t chunk_id, int32_t n_tokens, uint64_t seed);

/* Kernel classes for phase timing. */
enum {
  PERCACHE_PH_GATHER = 0,   /* gather + re-RoPE of hit tokens, all layers                */
  PERCACHE_PH_NORM,         /* both RMSNorms                                              */
  PERCACHE_PH_QKV,          /* QKV projection + RoPE + scatter                           */
  PERCACHE_PH_ATTN,         /* causal GQA attention of the new rows                      */
  PERCACHE_PH_OPROJ,        /* output projection + residual                              */
  PERCACHE_PH_GATEUP,       /* gate/up projection + SwiGLU                               */
  PERCACHE_PH_DOWN,         /* down projection + residual                                */
  PERCACHE_PH_IO,           /* input staging and output copies                           */
  PERCACHE_PH_COUNT
};

typedef struct {
  /* last percache_prefill call */
  int32_t n_prompts, chunks_hit, chunks_missed;
  int64_t ctx_tokens, hit_tokens, new_rows;
  int64_t pages_used, pages_free;
  double  host_plan_us;                        /* lookup + page allocation + index assembly       */
  double  device_us;                           /* first kernel start to last kernel end (events)  */
  double  phase_us[PERCACHE_PH_COUNT];         /* filled when PERCACHE_FLAG_PHASE_TIMING is set   */
  int32_t phase_launches[PERCACHE_PH_COUNT];   /* kernels launched per class (always filled)      */
  int64_t attn_visible_pairs;                  /* sum over new rows of (position + 1)             */
  int64_t evictions;                           /* chunks evicted by the last prefill / put call   */
  int32_t gather_free;                         /* 1: the last prefill took the gather-free form   */
  int32_t reserved0;
} percache_stats_t;

PERCACHE_API int percache_get_stats(percache_t* h, percache_stats_t* out);

/* Replace the handle's flags (any PERCACHE_FLAG_* bits) after creation. */
PERCACHE_API int percache_set_flags(percache_t* h, uint32_t flags);

/* Integer plan of the last successful percache_prefill (host int32 arrays, caller-allocated).
 * which: 0 cu_ctx [n_prompts+1]; 1 cu_new [n_prompts+1]; 2 slot_chunk [ctx_tokens] (index into the prompt's
 * chunk list, n_chunks for query tokens); 3 slot_offset [ctx_tokens]; 4 slot_is_new [ctx_tokens];
 * 5 row_slot [new_rows] (slot of every new row inside its prompt = its position).
 * Returns the number of elements written, or a negative code (PERCACHE_E_CAPACITY if capacity is short). */
PERCACHE_API int64_t percache_debug_read_plan(percache_t* h, int32_t which, int32_t* out, int64_t capacity);

/* Host-only: the attention kernel's work schedule for tiles of given lengths, without a device (the part of
 * percache_prefill's index assembly that cuts every tile's units into items and deals them to the persistent
 * CTAs; the kernel itself is the causal GQA attention of the new rows over the assembled context, paper
 * Appendix B.1).  n_blocks [n_tiles]: context blocks (128 slots) each tile sees; units_per_tile: KV heads x
 * query-head pairs; n_ctas: CTAs available (one per SM); max_partial_slots: parts that may write partial results.
 * items_out: caller-allocated [items_capacity][6] int32 rows (tile, unit, blk_begin, blk_end, partial_slot or -1,
 * cta), in execution order.  counts_out [4]: items, CTAs used, split units, estimated makespan in quarter blocks.
 * Returns PERCACHE_OK, PERCACHE_E_INVAL, or PERCACHE_E_CAPACITY when items_capacity is short. */
PERCACHE_API int percache_debug_attn_plan(const int32_t* n_blocks, int32_t n_tiles, int32_t units_per_tile, int32_t n_ctas,
                             int32_t max_partial_slots, int32_t* items_out, int64_t items_capacity,
                             int64_t* counts_out);

/* Debugging aid for parity checks at full size and depth: while host_buf is set, every percache_prefill (and
 * percache_decode) call also copies the fp32 residual stream of its rows as it enters each decoder block, and once
 * more after the last block, to host_buf laid out [n_layers + 1][rows of the call][d_model] (entry l = input of
 * block l, entry n_layers = the call's output).  A checker can then feed block l's input to a reference
 * implementation and compare single blocks, which keeps the check affordable where a whole reference run is not.
 * host_buf: caller-owned host memory of capacity_floats floats that must stay valid until it is unset with NULL; a
 * prefill that needs more than the capacity fails with PERCACHE_E_CAPACITY before anything runs.  The copies
 * serialise the call's kernels: never leave this on while timing. */
PERCACHE_API int percache_debug_capture_layers(percache_t* h, float* host_buf, int64_t capacity_floats);

/* Assembled context of the last call: rotated K and V of one prompt and layer as fp16
 * [n_total + tokens decoded since][n_kv_heads][head_dim], copied to host buffers that hold capacity_tokens tokens
 * each (fewer than needed -> PERCACHE_E_CAPACITY, nothing is written).  PERCACHE_E_INVAL when the last call left no
 * assembled context (gather-free form, paper-faithful mode). */
PERCACHE_API int percache_debug_read_ctx(percache_t* h, int32_t prompt, int32_t layer, void* k_host, void* v_host,
                                         int64_t capacity_tokens);

/* Failure-path check that is safe to run: one tiny kernel waits, through the very wait function every tcgen05
 * kernel of this library uses, on a shared-memory barrier nobody arrives at.  The first waiter's limit is limit_us
 * (1..2000): its wait runs out and it records a code in the error word; a second waiter with a 1000 times longer
 * limit must leave as soon as it sees that code.  Nothing is in flight (no bulk copy, no tensor memory), the kernel
 * returns normally and the device stays usable.  Returns PERCACHE_E_DEVICE_TIMEOUT when the wait ran out as
 * designed (the mapping percache_prefill applies to a non-zero error word), PERCACHE_OK if the error word stayed
 * zero.  code_out: the recorded code (901 = the probe); waited_ns [2]: how long the two waiters waited.  Either
 * pointer may be NULL. */
PERCACHE_API int percache_debug_wait_probe(int32_t device, uint32_t limit_us, int32_t* code_out, uint64_t* waited_ns);

/* C[M][N] (fp32, host) = A[M][K] * B[N][K]^T with fp16 inputs (host), through the tcgen05 GEMM
 * (use_reference = 0), the plain kernel (1), or the tcgen05 GEMM on CTA pairs with 256 x 256 tiles (2; needs
 * N % 256 == 0).  Test hook for the GEMM core. */
PERCACHE_API int percache_debug_gemm(int32_t device, int32_t M, int32_t N, int32_t K, const void* a_f16, const void* b_f16,
                        float* c, int32_t use_reference);

/* The same GEMM as percache_debug_gemm(use_reference = 0) for callers that cannot allocate device memory.
 * The paper has no counterpart; this exists for two kinds of caller: one whose process has already given
 * all device memory to another allocator (so a raw cudaMalloc would fail), and one inside a serving loop
 * that must avoid the device-wide synchronisation of cudaMalloc / cudaFree.  The device copies of A, B, C
 * and the kernel's error word live in a fixed PERCACHE_NOALLOC_SCRATCH_BYTES array inside the library image
 * (every GPU that loads the library holds that much until the process exits).  The call itself performs no
 * cudaMalloc, cudaFree or other allocating routine.
 *  - Sizes: 256 + pad128(M)*K*2 + N*K*2 + M*N*4 bytes (each term rounded up to 256) must fit in the array,
 *    otherwise PERCACHE_E_CAPACITY and nothing runs.  K % 64 == 0, N % 128 == 0 as for percache_debug_gemm.
 *  - a_f16, b_f16, c are host buffers owned by the caller; the call returns after the result is in c.
 *  - The first call on a device looks up the array's device address; make that call before starting any
 *    stream capture on that device.
 *  - All calls share the one array and it keeps the previous call's bytes; the call clears what must start
 *    at zero.  Two calls whose GPU work overlaps (for instance from two host threads using the same device)
 *    race on it: serialise them. */
#define PERCACHE_NOALLOC_SCRATCH_BYTES (16u << 20)
PERCACHE_API int percache_debug_gemm_noalloc(int32_t device, int32_t M, int32_t N, int32_t K, const void* a_f16,
                                const void* b_f16, float* c);

/* QA-bank lookup (paper Section 3.4.1 "Similar Query Reuse"): cosine similarity of each query embedding with
 * every stored query embedding, the most similar entry, and whether its similarity exceeds tau_query (then the
 * cached answer of that entry can be returned without running the model).
 * bank: device fp32 [n_entries][dim] (dim a multiple of 4, rows 16-byte aligned); queries: device fp32
 * [n_queries][dim], n_queries <= 8 (PERCACHE_E_CAPACITY beyond).  Outputs are host arrays [n_queries]:
 * best_index (lowest index among equal maxima), best_score (cosine, fp32 arithmetic), hit (score > tau_query).
 * kernel_us: optional (may be NULL); receives the kernel's duration from CUDA events on the stream.
 * Runs on `stream` (a cudaStream_t or NULL) and returns after it has finished.  One lookup at a time per
 * device and process (the running maxima live in one device-side array of the library). */
PERCACHE_API int percache_qa_top1(int32_t device, void* stream, const float* bank, int32_t n_entries, int32_t dim,
                     const float* queries, int32_t n_queries, float tau_query, int32_t* best_index,
                     float* best_score, uint8_t* hit, float* kernel_us);

PERCACHE_API const char* percache_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* PERCACHE_H_ */
