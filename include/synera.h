/*
 * synera.h -- C ABI of the cloud-side batched verification step of Synera
 * (arxiv 2511.07423), implemented as hand-written CUDA for NVIDIA B200 (sm_100a).
 *
 * The step (paper Sec. 3.4 "partial prefill", Sec. 4.5 "flatten -> forward -> verify"):
 * many devices offload short token chunks; each chunk is appended to that request's cached
 * context (a paged KV cache), a decoder-only transformer is run over the ragged batch, and
 * the LLM's greedy argmax at every chunk position is compared with the drafted tokens
 * (Sec. 3.1, "draft & verify") to give, per request, the number of accepted drafts and the
 * correction token.
 *
 * Conventions
 *   - Every function returns an int status: SYN_OK (0) or a negative SYN_E_* code.  No
 *     exceptions, no abort, nothing is printed.  syn_strerror() names a code.
 *   - "HOST" / "DEVICE" beside a pointer says where the memory must live.  The caller owns
 *     every array it passes; the library keeps no caller pointer after a call returns,
 *     except where stated (syn_plan keeps nothing either: it copies).
 *   - All validation of a call happens on the host before any kernel is launched; on error
 *     nothing is written (outputs and KV cache untouched).
 *   - One call at a time per syn_model.  The library allocates device memory with
 *     cudaMalloc on the current device; it does not link or call PyTorch.
 *   - Matrices are bf16, row-major [out_features][in_features] (y = x W^T); RMSNorm gains are
 *     bf16 [d_model].  There are no biases.
 *   - Arithmetic: every matrix product takes IEEE half-precision operands and accumulates in fp32; the
 *     residual stream, the softmax statistics and the logits are fp32.  The library's packed copy of the
 *     bf16 weights is half precision: a bf16 value of magnitude >= 2^-17 converts exactly, smaller ones
 *     round to a multiple of 2^-24.  Activations and the cached K and V are half precision too (11
 *     significant bits; bf16 would keep 8), clamped to +-65504 where bf16 would have had the range.
 */
#ifndef SYNERA_H_
#define SYNERA_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    SYN_OK = 0,
    SYN_E_INVALID_ARG = -1,    /* NULL pointer, zero size, unsupported shape                    */
    SYN_E_CHUNK_LEN = -2,      /* a chunk length outside [1, SYN_MAX_CHUNK]                     */
    SYN_E_UNCACHED = -3,       /* n_uncached[i] outside [1, chunk length]                       */
    SYN_E_PAGE_OOB = -4,       /* a used page id outside [0, n_pages)                           */
    SYN_E_CAPACITY = -5,       /* ctx + chunk exceeds max_pages * page_size                     */
    SYN_E_TOKEN_OOB = -6,      /* a token id outside [0, vocab)                                 */
    SYN_E_PAGE_ALIAS = -7,     /* two chunk tokens of the batch map to the same KV slot         */
    SYN_E_OOM = -8,            /* device or host allocation failed                              */
    SYN_E_ARCH = -9,           /* current device is not compute capability 10.x                 */
    SYN_E_CUDA = -10,          /* a CUDA runtime/driver call failed                             */
    SYN_E_DEVICE_TIMEOUT = -11 /* a bounded wait inside a kernel ran out; results are invalid   */
};

/* Longest chunk of one request in one call: the fixed chunk length of the paper's chunked partial
 * prefill (Sec. 4.5).  Verification chunks are tens of tokens at most (Sec. 3.4); a longer
 * uncached run is fed in several calls. */
#define SYN_MAX_CHUNK 32

typedef struct syn_model syn_model; /* packed device copy of the weights + workspaces */
typedef struct syn_kv syn_kv;       /* paged KV pool                                   */
typedef struct syn_plan syn_plan;   /* device-resident description of one batch        */

/* Decoder shape (Llama family: RMSNorm, rotate-half RoPE, grouped-query attention, SwiGLU).
 * Supported: head_dim 64 or 128; d_model a multiple of 128; n_q_heads a multiple of
 * n_kv_heads with group size <= 8; (n_q_heads*head_dim) and (n_kv_heads*head_dim)
 * multiples of 128; d_ffn a multiple of 8. */
typedef struct {
    uint32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab;
    float rope_base; /* theta_i = rope_base^(-2i/head_dim) */
    float rms_eps;
    uint32_t flags;  /* must be 0 */
} syn_model_desc;

/* Weight pointers, all bf16.  Per-layer arrays hold n_layers pointers (the arrays themselves
 * are HOST memory).  location: 0 = the matrices are in HOST memory, 1 = in DEVICE memory. */
typedef struct {
    const void *embed;      /* [vocab][d_model]   */
    const void *lm_head;    /* [vocab][d_model]   */
    const void *final_norm; /* [d_model]          */
    const void *const *wq;  /* [n_q_heads*head_dim][d_model]  */
    const void *const *wk;  /* [n_kv_heads*head_dim][d_model] */
    const void *const *wv;  /* [n_kv_heads*head_dim][d_model] */
    const void *const *wo;  /* [d_model][n_q_heads*head_dim]  */
    const void *const *wg;  /* [d_ffn][d_model]  gate         */
    const void *const *wu;  /* [d_ffn][d_model]  up           */
    const void *const *wd;  /* [d_model][d_ffn]  down         */
    const void *const *norm1; /* [d_model] gain before attention */
    const void *const *norm2; /* [d_model] gain before the MLP   */
    int32_t location;
} syn_weights;

/* The LLM that verifies (paper Sec. 3.1).  Makes the library's own packed device copy of the
 * weights, layer by layer (tiles of 128 output features x 64 inputs in the tensor cores' shared-
 * memory order; q|k|v in one matrix with the two halves of a head's rotation side by side, gate
 * and up features of the same 64 columns in one tile, d_ffn padded to a multiple of 64 with
 * zeros), so the caller's copy may be freed afterwards.
 * Errors: SYN_E_INVALID_ARG (NULL, unsupported shape, flags != 0), SYN_E_ARCH, SYN_E_OOM,
 * SYN_E_CUDA.  *out is written only on success. */
int syn_model_load(const syn_model_desc *desc, const syn_weights *weights, syn_model **out);
void syn_model_free(syn_model *m);

/* The cache that holds every request's prefix (paper Sec. 3.4: "an existing KV-cached
 * prefix").  n_pages physical pages of page_size tokens for every layer, bf16, zero-filled.
 * Position p of a request lives in page page_table[p / page_size], row p % page_size.
 * page_size must be 16.  Errors: SYN_E_INVALID_ARG, SYN_E_OOM, SYN_E_CUDA. */
int syn_kv_alloc(syn_model *m, uint32_t n_pages, uint32_t page_size, syn_kv **out);
void syn_kv_free(syn_kv *kv);

/* Place externally produced (already rotated) K and V of one request and one layer at logical
 * positions pos0 .. pos0+n_pos-1, e.g. a prefix computed on another server.  k, v: DEVICE bf16
 * [n_pos][n_kv_heads][head_dim] (the pool itself holds half precision: import converts, exactly for
 * magnitudes in [2^-17, 65504], export rounds back to bf16); page_table: HOST int32, at least ceil((pos0+n_pos)/page_size)
 * entries.  Blocking: the call allocates a small device buffer for the slot list, synchronises
 * `cuda_stream` and returns when the copy is done.
 * syn_kv_export is the inverse (reads the same positions into k, v).
 * Errors: SYN_E_INVALID_ARG, SYN_E_PAGE_OOB, SYN_E_CUDA. */
int syn_kv_import(syn_kv *kv, uint32_t layer, const int32_t *page_table, int32_t pos0, int32_t n_pos,
                  const void *k, const void *v, void *cuda_stream);
int syn_kv_export(syn_kv *kv, uint32_t layer, const int32_t *page_table, int32_t pos0, int32_t n_pos,
                  void *k, void *v, void *cuda_stream);

/* One batched verification step: execute_partialprefill(B_verify, L_uncached) of the paper's
 * scheduler (Algorithm 1) followed by the verification of Sec. 4.5.
 *
 * Request i contributes the chunk chunk_tokens[chunk_offsets[i] .. chunk_offsets[i+1]) of
 * n_i tokens, 1 <= n_i <= SYN_MAX_CHUNK: first u_i = n_uncached[i] >= 1 tokens the device has
 * already accepted but the cloud has not cached (Sec. 3.4, "device-accepted tokens"), then
 * n_i - u_i pending-verify draft tokens.  The chunk is appended after the ctx_lens[i] cached
 * tokens: K and V of all n_i tokens are written at positions ctx_lens[i] .. ctx_lens[i]+n_i-1
 * through page_tables[i][.], and token j attends to positions 0 .. ctx_lens[i]+j.
 * The argmax at chunk index u_i-1+j judges draft j (the engine outputs q(x|prefix),
 * q(x|prefix,x~_1), ...: gamma+1 distributions for gamma drafts, Sec. 4.5).
 *   accept_len[i]       = number of leading drafts equal to the argmax, in [0, n_i-u_i]
 *   correction_token[i] = argmax at the first mismatch; the bonus token (argmax after the last
 *                         draft) when every draft is accepted.  Ties: lowest token id.
 * After the call the caller advances ctx_lens[i] by u_i + accept_len[i]; slots of rejected
 * drafts are simply overwritten by a later call.  A prefill is this call with u_i = n_i.
 *
 * HOST inputs: req_ids [n_req] (opaque labels, may be NULL), chunk_tokens [T],
 * chunk_offsets [n_req+1] (chunk_offsets[0] = 0, T = chunk_offsets[n_req]),
 * page_tables [n_req][max_pages] (entries beyond a request's used pages are ignored),
 * ctx_lens [n_req], n_uncached [n_req] or NULL (= 1 each).
 * HOST outputs: accept_len [n_req], correction_token [n_req].
 * logits_out: NULL, or DEVICE fp32 [T][vocab] receiving every chunk position's logits.
 * The call returns after the results are in the host arrays (it synchronises cuda_stream).
 * Errors: SYN_E_INVALID_ARG, SYN_E_CHUNK_LEN, SYN_E_UNCACHED, SYN_E_PAGE_OOB, SYN_E_CAPACITY,
 * SYN_E_TOKEN_OOB, SYN_E_PAGE_ALIAS, SYN_E_OOM (workspace growth), SYN_E_CUDA,
 * SYN_E_DEVICE_TIMEOUT. */
int syn_verify_batch(syn_model *m, syn_kv *kv, int32_t n_req, const int64_t *req_ids,
                     const int32_t *chunk_tokens, const int32_t *chunk_offsets,
                     const int32_t *page_tables, int32_t max_pages, const int32_t *ctx_lens,
                     const int32_t *n_uncached, int32_t *accept_len, int32_t *correction_token,
                     float *logits_out, void *cuda_stream);

/* The same step split in two, for callers that keep the batch description on the device
 * (and for timing the kernels alone).  syn_plan_create validates exactly like
 * syn_verify_batch, runs the host planner (token positions, KV slots, attention work list;
 * the "flatten" of Sec. 4.5) and uploads the result.  syn_verify_run launches the step
 * asynchronously on cuda_stream; accept_len_dev / correction_dev are DEVICE int32 [n_req];
 * top1_dev is NULL or DEVICE int32 [T] (argmax per chunk position).  It does not synchronise:
 * call syn_model_status after synchronising the stream to learn of a device-side timeout.
 * A plan may be run any number of times (each run rewrites the same KV slots).
 * A plan belongs to the cache it was created with: its page ids and KV slots were checked against
 * that cache's size, so syn_verify_run, syn_op_attention and syn_op_attention_static return
 * SYN_E_INVALID_ARG, before any launch, when they are given another cache (or that cache freed and
 * another allocated in its place). */
int syn_plan_create(syn_model *m, syn_kv *kv, int32_t n_req, const int32_t *chunk_tokens,
                    const int32_t *chunk_offsets, const int32_t *page_tables, int32_t max_pages,
                    const int32_t *ctx_lens, const int32_t *n_uncached, syn_plan **out);
void syn_plan_free(syn_plan *p);
int syn_verify_run(syn_model *m, syn_kv *kv, const syn_plan *p, int32_t *accept_len_dev,
                   int32_t *correction_dev, int32_t *top1_dev, float *logits_out, void *cuda_stream);
int syn_model_status(syn_model *m); /* SYN_OK or SYN_E_DEVICE_TIMEOUT / SYN_E_CUDA; blocking */

/* Counters of a step (algorithmic work, for roofline arithmetic) and, measured, its times. */
typedef struct {
    int32_t n_req, n_tokens;       /* B and T                                               */
    int64_t ctx_tokens;            /* sum of ctx_lens                                       */
    int64_t weight_bytes;          /* bf16 bytes of all projections streamed once per step  */
    int64_t kv_read_bytes;         /* sum over requests of (ctx+n) * 2*Hkv*hd*2 * n_layers   */
    int64_t kv_write_bytes;        /* T * 2*Hkv*hd*2 * n_layers                             */
    double dense_flops;            /* 2 * T * projection parameters                         */
    double attn_flops;             /* 4 * Hq*hd * n_layers * sum over tokens of keys seen    */
    int32_t attn_items, attn_split_items; /* attention work items per layer / those that are partial */
    int32_t kernel_launches;       /* kernels launched by one syn_verify_run                */
    int32_t attn_rows;             /* row tile of the attention kernel the batch was planned for: 64 (warp-level MMAs) or 128 (tcgen05) */
    int64_t h2d_bytes;             /* batch description uploaded per step by syn_verify_batch */
    double t_gpu_ms;               /* device time of the step, first kernel to last (CUDA events); 0 unless profiling is on */
    double t_wall_ms;              /* host wall time of the blocking call that ran it; 0 unless profiling is on  */
} syn_step_stats;
/* The last step launched on this model by syn_verify_batch, syn_verify_batch_sampled or syn_verify_run
 * (the paper's cloud runtime reports per-iteration execution time, Sec. 6.7).  With syn_set_profile on,
 * t_gpu_ms is filled (the call then waits for that step to finish) and, for the blocking calls,
 * t_wall_ms.  SYN_E_INVALID_ARG before the first step.  syn_plan_stats: the counters of a plan. */
int syn_last_step_stats(syn_model *m, syn_step_stats *out);
int syn_plan_stats(const syn_plan *p, syn_step_stats *out);

/* The host planner of syn_plan_create / syn_verify_batch on its own, without a device: the same
 * validation (same error codes, same order) and the same outputs, written to caller-provided HOST
 * arrays: pos, slot [T] (token position ctx+j and KV slot page*page_size+row; either may be NULL),
 * items [items_cap][SYN_PLAN_ITEM_FIELDS] = the attention work list in CTA order, each row being
 * (first query token, query tokens, kv head, request, first key, one past the last key, position of
 * the first query token, index of its partial or -1, merge group or -1) (NULL to skip;
 * SYN_E_CAPACITY if items_cap is too small, *n_items then holds the count needed), cta_begin
 * [n_sm + 1] (CTA k owns items cta_begin[k] .. cta_begin[k+1]; NULL to skip), *n_cta, *stats (may be
 * NULL; h2d_bytes is left 0).  n_sm = number of CTAs to plan for (the device's SM count). */
#define SYN_PLAN_ITEM_FIELDS 9
int syn_plan_host(const syn_model_desc *desc, uint32_t n_pages, uint32_t page_size, int32_t n_sm, int32_t n_req,
                  const int32_t *chunk_tokens, const int32_t *chunk_offsets, const int32_t *page_tables,
                  int32_t max_pages, const int32_t *ctx_lens, const int32_t *n_uncached, int32_t *pos, int32_t *slot,
                  int32_t *items, int32_t items_cap, int32_t *n_items, int32_t *cta_begin, int32_t *n_cta,
                  syn_step_stats *stats);


/* Per-kernel-class device timing.  With profiling on, syn_verify_run / syn_verify_batch bracket
 * every launch with CUDA events on the caller's stream.  syn_get_profile synchronises the device,
 * adds up the elapsed time and launch count of each class since the last call, and clears them.
 * Classes: 0 prep, 1 qkv GEMM, 2 attention, 3 attention merge, 4 o GEMM, 5 gate/up GEMM,
 * 6 down GEMM, 7 lm_head GEMM, 8 verify (greedy compare, and the sampling stage of
 * syn_verify_batch_sampled), 9 unused (the residual update and the norm statistic are part of the
 * o and down GEMMs).  ms, launches: HOST arrays of SYN_N_KERNEL_CLASSES. */
#define SYN_N_KERNEL_CLASSES 10
int syn_set_profile(syn_model *m, int on);
int syn_get_profile(syn_model *m, double *ms, int32_t *launches);

const char *syn_strerror(int code);
/* Name of the CUDA error (e.g. "cudaErrorLaunchOutOfResources") behind the most recent SYN_E_CUDA or
 * SYN_E_OOM returned on the calling thread; "" if there was none.  Static storage. */
const char *syn_last_cuda_error(void);

/* ---- single operations, exported for per-kernel tests and roofline measurements ------- */

/* y[T][N] (fp32, DEVICE) = x[T][K] (half precision, DEVICE) * W[N][K]^T (bf16, DEVICE): the tcgen05
 * GEMM used by every projection, with a plain store epilogue.  The first call with a given w
 * (pointer and shape) packs it into the library's tiled layout; later calls reuse the packed copy:
 * call syn_op_linear_reset after the contents of w changed or w was freed (a new matrix may land at
 * the old address).  K a multiple of 64 is not required (TMA zero-fills the tail) but K*2 bytes must
 * be a multiple of 16; N arbitrary.  Blocks until the result is there.
 * syn_op_linear_as runs the same product under the schedule the step uses for the projection with
 * epilogue `schedule_as` (0 plain, 1 qkv, 2 residual, 3 SwiGLU, 4 lm_head; see syn_gemm_plan_host), so
 * that every schedule can be checked against a plain matrix product; 5 and 6 take the CTA-pair kernel
 * with items of 512 and of 256 features whatever the shape, 7 and 8 the same as residual projections
 * (K shared between clusters where the shape allows it).
 * Errors: SYN_E_INVALID_ARG, SYN_E_CUDA, SYN_E_DEVICE_TIMEOUT. */
int syn_op_linear(const void *x, const void *w, float *y, int32_t T, int32_t N, int32_t K, void *cuda_stream);
int syn_op_linear_as(const void *x, const void *w, float *y, int32_t T, int32_t N, int32_t K, int32_t schedule_as,
                     void *cuda_stream);
int syn_op_linear_reset(void);

/* Test hooks for the bounded device-side waits (SYN_E_DEVICE_TIMEOUT).  syn_debug_set_spin_limit: the
 * number of SM cycles after which a wait inside the projection kernels gives up (0 restores the default,
 * about two seconds); applies to launches made afterwards, process-wide.  syn_debug_linear_counter:
 * overwrite one of the arrival counters of syn_op_linear's own workspace (index in [0, 2 * SMs)), so
 * that a wait for a count that can no longer be reached runs out; the counters are cleared again when
 * the timeout is reported.  A wait that runs out unwinds normally: the kernel ends, the results of
 * that call are invalid, the next call works.
 * syn_debug_set_schedule: 0 (default) lets every projection take the kernel its shape calls for (CTA
 * pairs from 256 tokens on); 1 keeps all of them on the one-CTA kernel, so that both can be measured
 * and checked on the same batch.  Process-wide.
 * syn_debug_set_attention: which attention kernel the plans made AFTERWARDS are laid out for (a plan
 * keeps its kernel): 0 (default) the cheaper of the two for the batch by the planner's cost model, 1 the
 * warp-level-MMA kernel (row tiles of 64), 2 the tcgen05 kernel (row tiles of 128: a whole chunk of up to
 * 128 / G tokens is one work item per kv head).  Process-wide. */
int syn_debug_set_spin_limit(int64_t cycles);
int syn_debug_linear_counter(int32_t index, int32_t value);
int syn_debug_set_schedule(int32_t which);
int syn_debug_set_attention(int32_t which);

/* The ragged paged attention of the step on its own (paper Sec. 3.2 attention equation over a
 * paged cache).  q: DEVICE half precision [T][n_q_heads*head_dim] (rotated); out: DEVICE half
 * precision, same shape.  The plan supplies page tables, lengths and the work list; the chunk's K/V must
 * already be in the pool of `layer`.  Asynchronous on cuda_stream. */
int syn_op_attention(syn_model *m, syn_kv *kv, const syn_plan *p, uint32_t layer, const void *q, void *out,
                     void *cuda_stream);

/* syn_op_attention for callers that must not allocate device memory while they run: code between
 * cudaStreamBeginCapture and EndCapture, a serving loop whose memory pool was sized up front and
 * handed out completely, or a host thread that may not take the allocator's lock.  (The paper has
 * no counterpart; this is a service of the library.)  Same arguments, same result and same
 * asynchronous behaviour as syn_op_attention, but the partial results of work items that cover
 * only part of a request's keys live in a fixed array inside the library instead of a workspace
 * that grows on demand.  The array holds SYN_STATIC_MAX_PARTS partials of 64 rows, or half as many of
 * the 128-row kind of a plan made for the tcgen05 kernel (about 8.5 MB of every GPU that loads the
 * library, from load to exit).  The call itself allocates and frees nothing; the
 * model, cache and plan it is given were of course allocated earlier by their own calls.
 *   - A plan with more partial work items than that (attn_split_items x attn_rows of syn_plan_stats()
 *     above SYN_STATIC_MAX_PARTS x 64) is refused with SYN_E_CAPACITY before anything is launched.
 *   - The first call on each device looks up the array's device address (with that device
 *     current); make that first call outside any stream capture.
 *   - All calls on a device share the one array.  It keeps the previous call's contents; nothing
 *     in it needs clearing, because every partial that is read is written earlier in the same
 *     call.  Two calls that overlap on the GPU (different streams) race on it: serialise them.
 * Errors: SYN_E_INVALID_ARG, SYN_E_CAPACITY, SYN_E_CUDA. */
#define SYN_STATIC_MAX_PARTS 256
int syn_op_attention_static(syn_model *m, syn_kv *kv, const syn_plan *p, uint32_t layer, const void *q, void *out,
                            void *cuda_stream);

/* The projection kernel's schedule without a device (tests): how a y[T][N] = x[T][K] w[N][K]^T
 * projection with the given epilogue (0 plain store, 1 QKV, 2 residual update, 3 SwiGLU, 4 lm_head)
 * is cut up on n_sm SMs.  syn_gemm_plan_host fills out[SYN_GEMM_PLAN_FIELDS] = {feature pairs of 256,
 * token tiles, tokens per tile, k-blocks of 64, CTAs, pair mode, CTAs that share a tile's K range
 * (reduce-scatter), k-blocks of each, K parts of a leftover pair tile, k-blocks of a helper part}.  syn_gemm_work_host returns 1 and
 * fills out[SYN_GEMM_WORK_FIELDS] = {pair, token tile, first 128-feature tile, one past the last,
 * first k-block, one past the last, split-K part, role (0 whole K, 1 helper, 2 owner), leftover
 * tile, helper part} for work item i of CTA cta, 0 when that CTA has no item i.
 * Errors: SYN_E_INVALID_ARG. */
#define SYN_GEMM_PLAN_FIELDS 10
#define SYN_GEMM_WORK_FIELDS 10
int syn_gemm_plan_host(int32_t T, int32_t N, int32_t K, int32_t n_sm, int32_t epilogue, int32_t *out);
int syn_gemm_work_host(int32_t T, int32_t N, int32_t K, int32_t n_sm, int32_t epilogue, int32_t cta, int32_t i,
                       int32_t *out);

/* The same for the CTA-pair kernel that serves projections of 256 tokens and more: clusters of two CTAs
 * share a token tile.  syn_gemm2_plan_host fills out[SYN_GEMM2_PLAN_FIELDS] = {item shape (0: the shape
 * stays on the one-CTA kernel, 1: items of 512 features, 2: items of 256 features), feature groups of that
 * size, token tiles, tokens per tile, k-blocks of 64, clusters, clusters that share a tile's K range
 * (reduce-scatter; 1: none), k-blocks of each, and, for the items left after the full waves, the number of
 * K parts each is cut into (0: not cut) and how many of them get one part more}.  `force`: 0, or 1 / 2 to
 * take that item shape whatever the size.  syn_gemm2_work_host returns 1 and fills
 * out[SYN_GEMM2_WORK_FIELDS] = {feature group, token tile, first k-block, one past the last, tile index,
 * K part, K parts of the tile, cluster of part 0, counter index} for work item i of a cluster, 0 when it
 * has no item i.  Errors: SYN_E_INVALID_ARG. */
#define SYN_GEMM2_PLAN_FIELDS 10
#define SYN_GEMM2_WORK_FIELDS 9
int syn_gemm2_plan_host(int32_t T, int32_t N, int32_t K, int32_t n_sm, int32_t epilogue, int32_t force, int32_t *out);
int syn_gemm2_work_host(int32_t T, int32_t N, int32_t K, int32_t n_sm, int32_t epilogue, int32_t force, int32_t cluster,
                        int32_t i, int32_t *out);

/* Sampling-based verification (paper Sec. 4.2, "Compression before transmission": for
 * verification the LLM needs the drafts and the SLM's distributions, of which the device sends
 * the most probable entries as its sampling method, top-1 / top-k / top-p, keeps them; Sec. 3.1:
 * draft and verify).  The step is syn_verify_batch's; the greedy compare is replaced by:
 *   q_t  = the LLM's distribution at chunk index t as its own sampling method keeps it:
 *          softmax(logits / temperature) over the top_k largest logits (ties: lower id), then the
 *          shortest prefix, in decreasing probability, whose mass reaches top_p of that; renormalised;
 *   draft at chunk index t >= u_i (token x) with transmitted SLM probability p_t(x) is kept iff
 *          rand_accept[t] * p_t(x) < q_{t-1}(x)           (probability min(1, q / p));
 *   accept_len = number of leading drafts kept; at the first draft not kept the correction token
 *          is drawn from the positive part of q_{t-1} - p_t, otherwise from q at the last chunk
 *          index: inverse CDF at rand_sample[i] over the candidates in increasing token id.
 * top_k = 1 with the SLM sending its top-1 is the greedy rule.
 * HOST inputs beside syn_verify_batch's: slm_ids / slm_probs [T][slm_k], row t = the transmitted
 * distribution chunk token t was drawn from (rows of the u_i accepted tokens are ignored; id -1 =
 * unused entry; probabilities in [0, 1], used as sent); rand_accept [T] and rand_sample [n_req],
 * uniform in [0, 1), drawn by the caller.
 * logits_out: NULL (the library keeps the step's logits in its own workspace) or DEVICE fp32
 * [T][vocab].  Errors: those of syn_verify_batch; SYN_E_INVALID_ARG for a configuration outside
 * 1 <= top_k, slm_k <= SYN_SAMPLE_MAX_K, 0 < top_p <= 1, temperature > 0, or a draw outside [0, 1);
 * SYN_E_TOKEN_OOB for an SLM id outside [-1, vocab). */
#define SYN_SAMPLE_MAX_K 64
typedef struct {
    int32_t top_k;
    float top_p;
    float temperature;
    int32_t slm_k;
} syn_sampling;
int syn_verify_batch_sampled(syn_model *m, syn_kv *kv, int32_t n_req, const int64_t *req_ids,
                             const int32_t *chunk_tokens, const int32_t *chunk_offsets, const int32_t *page_tables,
                             int32_t max_pages, const int32_t *ctx_lens, const int32_t *n_uncached,
                             const syn_sampling *cfg, const int32_t *slm_ids, const float *slm_probs,
                             const float *rand_accept, const float *rand_sample, int32_t *accept_len,
                             int32_t *correction_token, float *logits_out, void *cuda_stream);

/* The sampling stage alone, on logits the caller supplies (DEVICE fp32 [T][vocab]; everything
 * else HOST, as above): per-kernel parity and timing.  Needs no model.  Synchronises cuda_stream. */
int syn_op_sample_verify(const float *logits, int32_t T, int32_t vocab, int32_t n_req, const int32_t *chunk_tokens,
                         const int32_t *chunk_offsets, const int32_t *n_uncached, const syn_sampling *cfg,
                         const int32_t *slm_ids, const float *slm_probs, const float *rand_accept,
                         const float *rand_sample, int32_t *accept_len, int32_t *correction_token, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* SYNERA_H_ */
