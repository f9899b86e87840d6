/*
 * ckv -- CentroidKV hot path for NVIDIA B200 (sm_100a): Chunked Soft Matching KV-cache
 * clustering, degree-weighted centroid merge, online append, and decode attention over
 * the compressed cache.  C ABI; no C++ or framework types cross this boundary.
 *
 * Conventions
 *  - Every pointer is a DEVICE pointer owned by the caller unless its comment says "host".
 *    The library allocates and frees nothing and keeps no global state that a call could observe (the one
 *    exception is ckv_decode_attn_static, whose scratch array is shared by every call: see its comment).
 *  - All work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL = the
 *    default stream) and the calls return without synchronising.  The kernels are launched with programmatic
 *    stream serialization among themselves; towards the caller they behave like ordinary stream work (a call's results are
 *    complete when the last of its kernels is).  Only a caller kernel that is itself launched with the programmatic
 *    serialization attribute directly behind a call has to execute griddepcontrol.wait (cudaGridDependencySynchronize)
 *    before it reads the call's results, as that attribute always requires.
 *  - The return value is a ckv_status.  Argument errors are found on the host before any
 *    launch and leave every output untouched.
 *  - Tensors are row-major.  K and V of one sequence: [L, H, cap, D] (layers, KV heads,
 *    token capacity, head_dim) of which the first `len` tokens of every (layer, head)
 *    are valid; deg and logdeg: [L, H, cap].  K and V must be 16-byte aligned.
 *  - Thread safety: calls on distinct streams with distinct workspaces and outputs do
 *    not interfere (again except ckv_decode_attn_static).
 *  - This version supports D = 128 and even chunk sizes 2..256 (or 0 = no chunking); anything else
 *    returns CKV_ERR_UNSUPPORTED.
 */
#ifndef CKV_H_
#define CKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { CKV_F32 = 0, CKV_BF16 = 1 } ckv_dtype;

typedef enum {
  CKV_SELECT_GLOBAL = 0, /* rank the edges of all chunks of a (layer, head) together (Sec. 5.2 last paragraph, Sec. 5.3) */
  CKV_SELECT_CHUNK = 1   /* rank the edges inside each chunk */
} ckv_select;

typedef enum {
  CKV_OK = 0,
  CKV_ERR_INVALID_ARG = 1, /* null pointer, negative size, odd chunk, overlapping src/dst ... */
  CKV_ERR_ALIGNMENT = 2,   /* K, V, q or out not 16-byte aligned */
  CKV_ERR_CAPACITY = 3,    /* a destination cache is too small for what would be written */
  CKV_ERR_WORKSPACE = 4,   /* workspace NULL or smaller than ckv_*_workspace_bytes says */
  CKV_ERR_NO_PROGRESS = 5, /* the ratio schedule merges nothing although the budget is not met */
  CKV_ERR_UNSUPPORTED = 6, /* head_dim, chunk size or group size outside this version's range */
  CKV_ERR_CUDA = 7         /* a CUDA runtime call failed (launch configuration, invalid stream ...) */
  /* There is no "timeout" status.  The calls return before their kernels run, so a bounded wait inside a kernel that
   * gives up cannot be reported here: the compress kernels (the only ones that wait on asynchronous copies, tensor-core
   * completions or each other) record it in a status word at the start of their workspace, which ckv_workspace_status
   * reads.  The decode kernels contain no such wait and have no status word. */
} ckv_status;

/* One sequence's KV cache over all layers and KV heads, with the cluster degrees N of Sec. 3
 * (n_t = number of original tokens merged into slot t). */
typedef struct ckv_cache {
  void* k;         /* [L, H, cap, D] */
  void* v;         /* [L, H, cap, D] */
  int32_t* deg;    /* [L, H, cap] cluster degree n_t >= 1.  As a source: NULL means all ones.  As a destination: required. */
  float* logdeg;   /* [L, H, cap] natural log of deg, kept for Eq. 3's bias.  As a destination: NULL = not maintained. */
  int32_t L, H, D; /* layers, KV heads, head_dim */
  int32_t dtype;   /* ckv_dtype of k and v */
  int64_t cap;     /* capacity in tokens of every (layer, head) slab */
  int64_t len;     /* valid tokens; the same for every (layer, head), since the merge count depends on shapes only */
  int64_t pending; /* appended tokens at the tail that have not yet formed a full chunk (append path) */
} ckv_cache;

/* Algorithm 1's inputs and Eq. 4's schedule. */
typedef struct ckv_params {
  int32_t chunk;        /* c: chunk size, even; 0 = no chunking: every A token is matched against every B token of its
                           (layer, head) -- plain Bipartite Soft Matching, Sec. 5.2 / Table 8 "w/o chunk"; bf16 only,
                           ckv_compress_prefill and ckv_compress_append_recluster only */
  int32_t n_sink;       /* n1: leading tokens never merged */
  int32_t n_recent;     /* n2: trailing tokens never merged */
  int32_t n_rounds_max; /* upper bound on clustering rounds per call */
  float r_init;         /* Eq. 4: ratio of round 0 = fraction of the matched edges that are merged */
  float r_decay;        /* Eq. 4: delta_r */
  float r_min;          /* floor: r_j = max(r_init - j * r_decay, r_min) */
  int32_t select;       /* ckv_select */
  int64_t budget;       /* B: target cache length, sinks and recent tokens included.  0 = run exactly n_rounds_max rounds.
                           ckv_compress_append applies it to each completed window of `chunk` appended tokens. */
} ckv_params;

/* Host-only: what a ckv_compress_prefill call with this source length would do (Algorithm 1's
 * `while s > B` loop with Eq. 4): the final length, the number of rounds, the capacity the
 * destination needs.  Any output pointer (host) may be NULL.  No GPU is touched. */
int ckv_compress_plan(int64_t len, const ckv_params* params, int64_t* out_len, int64_t* rounds,
                      int64_t* dst_cap_needed);

/* Host-only: bytes of workspace ckv_compress_prefill / ckv_compress_append need for a cache of
 * this shape (k, v, deg pointers are not read).  Returns 0 for invalid arguments. */
size_t ckv_workspace_bytes(const ckv_cache* shape, const ckv_params* params);

/* Algorithm 1, pre-filling branch; one round is Sec. 5.2 (chunks, alternating split, cosine
 * similarity of Eq. 2, one edge per A token), Sec. 5.3 (merge the top fraction r of the ranked
 * edges, Eq. 4) and Eq. 5 (degree-weighted centroids of K and V, degrees summed).
 * Compresses src (len tokens) into dst: sinks, then the survivors of the middle in their
 * original order with each centroid at its B token's place, then the recent tokens.
 * dst must not overlap src or the workspace; dst->cap must be at least what ckv_compress_plan
 * reports.  On return dst->len (host field) is the new length, dst->pending is 0.
 * CKV_OK does not imply dst->len <= params->budget: the loop also ends after n_rounds_max rounds (with Eq. 4's
 * defaults 0.8 / 0.2 floored at 0.2, a 25 % budget takes six).  Compare dst->len, or *rounds_done with what
 * ckv_compress_plan reports for a large n_rounds_max.  CKV_ERR_NO_PROGRESS is returned only when a round would
 * merge nothing.
 * assign: optional [L, H, src->len] int32, receives for each source token the dst slot that
 * holds it (its cluster).  rounds_done: optional host pointer. */
int ckv_compress_prefill(const ckv_cache* src, ckv_cache* dst, const ckv_params* params, int32_t* assign,
                         void* workspace, size_t workspace_bytes, void* cuda_stream, int64_t* rounds_done);

/* Algorithm 1, decoding branch, `K = [K, k], V = [V, v], N = [N, 1]`: appends t_new tokens
 * (k_new, v_new: [L, H, t_new, D], cache dtype) with degree 1.  Whenever the appended tail
 * reaches `chunk` tokens that window alone is clustered as a stand-alone sequence (no sinks
 * or recent tokens inside it) with Eq. 4's schedule until it is no longer than params->budget
 * (0: exactly n_rounds_max rounds), and the result replaces the window.
 * cache->len and cache->pending (host fields) are updated; CKV_ERR_CAPACITY if the cache
 * cannot hold the tokens. */
int ckv_compress_append(ckv_cache* cache, const void* k_new, const void* v_new, int32_t t_new,
                        const ckv_params* params, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The same step for Bz sequences that decode in lock step: one new token per sequence, written by a single launch
 * (a serving batch of 64 otherwise pays 64 one-token copy launches per step).  caches: HOST array [Bz] of caches
 * with the same L, H, D and dtype; k_new, v_new: device [L, H, Bz, D], token b belongs to caches[b].  A sequence
 * whose appended tail reaches `chunk` tokens has that window clustered exactly as ckv_compress_append does; the host
 * fields len and pending of every cache are updated.  Workspace: ckv_workspace_bytes of any of the caches.  Nothing is
 * enqueued if an argument check fails (CKV_ERR_CAPACITY if some cache is full). */
int ckv_compress_append_batch(ckv_cache* caches, int32_t Bz, const void* k_new, const void* v_new, const ckv_params* params,
                              void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Algorithm 1, decoding branch, as printed: `K = [K, k], V = [V, v], N = [N, 1]`, and `if s >= B + g` one call of
 * CentroidKV over the whole cache, with B = params->budget (> 0) and g = interval (> 0).  The round keeps the sinks
 * and recent tokens, carries the degrees along, uses the ratio of round 0 (params->r_init; n_rounds_max is not
 * used) and, with CKV_SELECT_GLOBAL, merges min(floor(r * n_edges), s - B) edges, so the cache returns to B whenever
 * the ratio allows.  A round cannot run in place: it compresses `cache` into `spare` and the two structs then swap
 * their buffers (k, v, deg, logdeg, cap), so that on return `cache` again describes the live cache and `spare` the
 * other buffer; both need deg, the same L, H, D, dtype and a capacity of at least budget + interval.  t_new tokens
 * are processed as t_new decoding steps.  cache->len (host field) is updated, cache->pending set to 0;
 * *reclusterings (host, optional) receives the number of rounds run.  Workspace: ckv_workspace_bytes for a cache of
 * this shape with len = budget + interval and n_rounds_max = 1.  CKV_ERR_NO_PROGRESS if a round merges nothing. */
int ckv_compress_append_recluster(ckv_cache* cache, ckv_cache* spare, const void* k_new, const void* v_new, int32_t t_new,
                                  const ckv_params* params, int32_t interval, void* workspace, size_t workspace_bytes,
                                  void* cuda_stream, int64_t* reclusterings);

/* The kernels wait on asynchronous copies with a bounded number of polls; a wait that gives up sets a
 * status word at the start of the workspace instead of hanging.  This call copies that word to
 * *status_host (host pointer) and synchronises the stream: 0 = every wait completed, nonzero = some
 * output of the last ckv_compress_* call on this workspace is incomplete.  The paper has no counterpart. */
int ckv_workspace_status(const void* workspace, void* cuda_stream, int32_t* status_host);

/* One layer of one sequence for decode attention: k, v: [H, cap, D]; logdeg: [H, cap] or NULL
 * (all degrees one: Eq. 1). */
typedef struct ckv_layer_view {
  const void* k;
  const void* v;
  const float* logdeg;
  int64_t len;
  int64_t cap;
} ckv_layer_view;

/* Host-only: workspace bytes of ckv_decode_attn (split partials). */
size_t ckv_decode_workspace_bytes(int32_t Bz, int32_t H, int32_t G, int32_t D, int64_t max_len);

/* Eq. 3 / Algorithm 1 decoding branch: out = softmax(q K^T * scale + log N) V for one layer and
 * a batch of Bz sequences.  views_dev: device array [Bz]; q, out: [Bz, H*G, D] in `dtype`;
 * query head j reads KV head j / G; G <= 8.  max_len (host): an upper bound on every
 * views_dev[b].len, used to size the grid.  A sequence with len 0 gets zeros. */
int ckv_decode_attn(const ckv_layer_view* views_dev, int32_t Bz, int32_t H, int32_t G, int32_t D, int32_t dtype,
                    const void* q, void* out, float scale, int64_t max_len, void* workspace,
                    size_t workspace_bytes, void* cuda_stream);

/* ---- Paged cache (the block layout of serving engines; the paper's Appendix on its vLLM integration names the flow
 * read pages -> compress -> write back).  One layer's pool: k_pages, v_pages [n_pages, H, page_tokens, D],
 * deg_pages int32 and logdeg_pages fp32 [n_pages, H, page_tokens]; page_tokens a power of two >= 32.  A sequence owns
 * the pages its block table lists: logical token t sits in page block_table[t / page_tokens] at offset t % page_tokens.
 * Which pages are free is the caller's bookkeeping: after a compression to out_len tokens a sequence needs
 * ceil(out_len / page_tokens) pages and can return the rest. */
typedef struct ckv_paged_view {
  const int32_t* block_table; /* device, at least ceil(len / page_tokens) entries */
  int64_t len;
} ckv_paged_view;

/* Eq. 3 over a paged cache: as ckv_decode_attn, with views_dev a device array [Bz] of ckv_paged_view.  bf16 only in
 * this version (CKV_ERR_UNSUPPORTED otherwise); logdeg_pages NULL = all degrees one.  Workspace as ckv_decode_attn. */
int ckv_decode_attn_paged(const ckv_paged_view* views_dev, const void* k_pages, const void* v_pages, const float* logdeg_pages,
                          int32_t page_tokens, int32_t Bz, int32_t H, int32_t G, int32_t D, int32_t dtype, const void* q,
                          void* out, float scale, int64_t max_len, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* One decoding step of Algorithm 1 on a paged cache in a single launch: `K = [K, k], V = [V, v], N = [N, 1]` and Eq. 3
 * over the result.  views_dev[b].len is the length BEFORE the step; sequence b's new token k_new, v_new [Bz, H, D] is
 * written to slot len of its pages (the page block_table[len / page_tokens] must already belong to the sequence) with
 * degree 1 and log-degree 0, and the attention runs over len + 1 tokens, the new one read straight from k_new / v_new.
 * The device views are not modified: the caller raises len for the next step.  max_len (host): an upper bound on every
 * len + 1.  deg_pages is required, logdeg_pages NULL = all degrees one.  Otherwise as ckv_decode_attn_paged. */
int ckv_decode_append_attn_paged(const ckv_paged_view* views_dev, void* k_pages, void* v_pages, int32_t* deg_pages,
                                 float* logdeg_pages, int32_t page_tokens, int32_t Bz, int32_t H, int32_t G, int32_t D, int32_t dtype,
                                 const void* k_new, const void* v_new, const void* q, void* out, float scale, int64_t max_len,
                                 void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Copies one sequence's first `len` tokens of one layer between its pages and a contiguous slab k, v [H, cap, D],
 * deg [H, cap] (logdeg [H, cap] optional): gather = pages -> slab (to run ckv_compress_* on it), scatter = slab -> pages
 * (degrees and their logarithms are written to the pages as well; deg NULL on scatter = all ones).  deg_pages may be
 * NULL on gather (the slab then gets ones).  block_table: device, ceil(len / page_tokens) entries. */
int ckv_pages_gather(const int32_t* block_table, int64_t len, const void* k_pages, const void* v_pages, const int32_t* deg_pages,
                     int32_t page_tokens, int32_t H, int32_t D, int32_t dtype, void* k, void* v, int32_t* deg, float* logdeg,
                     int64_t cap, void* cuda_stream);
int ckv_pages_scatter(const int32_t* block_table, int64_t len, const void* k, const void* v, const int32_t* deg, int64_t cap,
                      int32_t page_tokens, int32_t H, int32_t D, int32_t dtype, void* k_pages, void* v_pages, int32_t* deg_pages,
                      float* logdeg_pages, void* cuda_stream);

/* ---- Clustering a paged cache directly (the paper's Appendix on its vLLM integration: read pages -> compress -> write
 * back -> free blocks).  A sequence's cache lives in pages of per-layer pools that all layers index with one block
 * table.  A round cannot run in place (thread blocks would overwrite rows that others still read), so the rounds
 * alternate between the sequence's own pages and scratch pages of the same pools: round 0 reads through block_table and
 * writes through scratch_table, round 1 the other way round (from position 0 of the sequence's own pages), and so on.
 * With an odd number of rounds the result therefore sits in the first pages of scratch_table, otherwise in the first
 * pages of block_table; ckv_pages_plan tells which, and how many pages the sequence keeps: the caller swaps the
 * tables if need be and returns every other page to its free list.  The contents of all pages of both tables are
 * overwritten.  This version: bf16, D = 128, chunk 64, page_tokens a power of two >= 64, up to 64 layers per call
 * (CKV_ERR_UNSUPPORTED otherwise: ckv_pages_gather -> ckv_compress_prefill -> ckv_pages_scatter serves the rest). */
typedef struct ckv_page_pool { /* one layer's pool */
  void* k_pages;       /* [n_pages, H, page_tokens, D] */
  void* v_pages;       /* [n_pages, H, page_tokens, D] */
  int32_t* deg_pages;  /* [n_pages, H, page_tokens], required */
  float* logdeg_pages; /* [n_pages, H, page_tokens] or NULL */
} ckv_page_pool;

/* Host-only: Algorithm 1's loop for a paged sequence of `len` tokens: final length, rounds, the scratch pages the call
 * needs, whether the result ends up in the scratch pages (1) or in the sequence's own (0), and the number of pages the
 * sequence keeps afterwards: ceil(out_len / page_tokens).  Any output pointer may be NULL. */
int ckv_pages_plan(int64_t len, const ckv_params* params, int32_t page_tokens, int64_t* out_len, int64_t* rounds,
                   int64_t* scratch_pages, int32_t* result_in_scratch, int64_t* pages_kept);

/* Host-only: workspace bytes of ckv_compress_paged (per-edge arrays of rounds ranked per head, staging of each round's
 * shorter last chunk); 0 for invalid arguments. */
size_t ckv_paged_workspace_bytes(int32_t L, int32_t H, int32_t D, int32_t dtype, int64_t len, const ckv_params* params);

/* Algorithm 1, pre-filling branch, on a paged sequence (Sec. 5.2, Sec. 5.3, Eq. 4, Eq. 5 as ckv_compress_prefill).
 * pools: HOST array [L]; block_table, scratch_table: device; has_deg: 0 = the source pages carry no degrees (all
 * ones).  *out_len, *result_in_scratch (host, optional) as ckv_pages_plan reports them.  CKV_ERR_CAPACITY if
 * scratch_pages is less than the plan needs. */
int ckv_compress_paged(const ckv_page_pool* pools, int32_t L, int32_t H, int32_t D, int32_t dtype, int32_t page_tokens,
                       const int32_t* block_table, int64_t len, int32_t has_deg, const int32_t* scratch_table,
                       int64_t scratch_pages, const ckv_params* params, void* workspace, size_t workspace_bytes,
                       void* cuda_stream, int64_t* out_len, int32_t* result_in_scratch);

/* ckv_decode_attn for callers that cannot hand over a workspace because they cannot allocate device
 * memory at the point of the call: code running inside a serving engine's steady-state loop whose memory
 * pool is frozen after start-up, a plug-in that is given only its input and output tensors, or a host
 * that must not call cudaMalloc (it synchronises the device).  The split partials go to a fixed 4 MiB
 * array that is part of the library image, so every GPU that loads the library holds those 4 MiB until
 * the process exits.  Same arguments, results and status codes as ckv_decode_attn, minus the workspace.
 * Limits: Bz * H * G * 132 floats per split must fit in the array (1 Mi floats), else CKV_ERR_CAPACITY;
 * when the usual number of sequence splits does not fit, fewer splits are used (slower, same result).
 * The call allocates and frees nothing.  The first call on each device looks up the array's device
 * address (a host-side runtime query, that device being current) and should therefore come before any
 * stream capture.  All calls on a device share the one array, which keeps whatever the last call
 * wrote (nothing in it needs clearing: each launch overwrites every partial it later reads); two
 * calls whose kernels overlap on the GPU (different streams) race on it -- serialise them.
 * The paper has no counterpart for this entry point. */
int ckv_decode_attn_static(const ckv_layer_view* views_dev, int32_t Bz, int32_t H, int32_t G, int32_t D, int32_t dtype,
                           const void* q, void* out, float scale, int64_t max_len, void* cuda_stream);

/* Host-only: a static string for a ckv_status. */
const char* ckv_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* CKV_H_ */
