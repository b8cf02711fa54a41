/* Verification-aware scheduler of the cloud runtime (paper Sec. 4.5, Algorithm 1) as a host loop
 * over syn_verify_batch.
 *
 * Every iteration is either a prefill iteration or a verification iteration, never a mix
 * (Sec. 4.5: prompts have thousands of tokens, verification requests tens; mixing them leaves
 * bubbles).  Waiting prefill requests come first: if any exist, the iteration forwards the next
 * chunk of every one of them (chunked partial prefill, fixed chunks of SYN_MAX_CHUNK tokens, all
 * of them "uncached": u = n) and ends.  Otherwise every waiting verification request is batched
 * with its number of uncached tokens and executed as one partial prefill
 * (execute_partialprefill(B_verify, L_uncached)).  Completed requests leave the active set at
 * the end of an iteration, and their pages go back to the pool.
 *
 * The scheduler owns the bookkeeping the paper leaves to its serving engine: the page table and
 * the cached length of every request, and a free list over the pool's pages.  All of it is host
 * code; the forward pass is syn_verify_batch.  A scheduler may be created without a model
 * (m == NULL, kv == NULL): syn_sched_peek and syn_sched_commit then still work, so the policy
 * can be driven and tested without a GPU; syn_sched_step needs a model.
 *
 * Threading: one thread at a time per scheduler.  Pointers returned through syn_sched_batch stay
 * valid until the next call on the same scheduler.
 */
#ifndef SYNERA_SCHED_H
#define SYNERA_SCHED_H

#include "synera.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct syn_sched syn_sched;

enum { SYN_SCHED_IDLE = 0, SYN_SCHED_PREFILL = 1, SYN_SCHED_VERIFY = 2 };

/* Further error codes (the SYN_E_* of synera.h apply as well). */
enum {
    SYN_E_SCHED_UNKNOWN_REQ = -20, /* no live request with this id                                  */
    SYN_E_SCHED_DUPLICATE = -21,   /* a live request with this id exists already                    */
    SYN_E_SCHED_STATE = -22,       /* the request cannot take this call now (still prefilling, a
                                      chunk already waiting, a batch peeked but not committed, ...) */
    SYN_E_SCHED_NO_BATCH = -23     /* commit without a peeked batch                                  */
};

/* One batch, in exactly the arrays syn_verify_batch takes (HOST memory owned by the scheduler). */
typedef struct {
    int32_t kind;                 /* SYN_SCHED_IDLE: nothing to run, the other fields are zero */
    int32_t n_req;
    int32_t n_tokens;             /* chunk_offsets[n_req] */
    int32_t max_pages;
    const int64_t *req_ids;       /* [n_req], arrival order                                   */
    const int32_t *chunk_tokens;  /* [n_tokens]                                               */
    const int32_t *chunk_offsets; /* [n_req + 1]                                              */
    const int32_t *page_tables;   /* [n_req][max_pages], unused entries -1                    */
    const int32_t *ctx_lens;      /* [n_req] cached tokens before the iteration               */
    const int32_t *n_uncached;    /* [n_req] u_i; prefill iterations: u_i = chunk length      */
} syn_sched_batch;

/* What one iteration did to one request. */
typedef struct {
    int64_t req_id;
    int32_t kind;             /* SYN_SCHED_PREFILL or SYN_SCHED_VERIFY                               */
    int32_t n_tokens;         /* chunk tokens forwarded                                             */
    int32_t accept_len;       /* verification: accepted drafts; prefill: 0                          */
    int32_t correction_token; /* verification: correction (or bonus) token; prefill: the LLM's
                                 argmax after the chunk's last token                                 */
    int32_t ctx_len;          /* cached tokens after the iteration: + n (prefill),
                                 + u + accept_len (verification)                                     */
    int32_t prompt_done;      /* prefill: 1 once the whole prompt is cached, else 0; verification: 1 */
} syn_sched_result;

typedef struct {
    int64_t iterations[3];      /* by kind (idle calls counted under SYN_SCHED_IDLE)                */
    int64_t tokens[3];          /* chunk tokens forwarded, by kind                                  */
    int64_t requests[3];        /* batch entries, by kind                                           */
    int64_t deferred;           /* batch entries put off for lack of free pages or token budget     */
    double host_seconds;        /* spent in the scheduler's own code: batching, tables, commit      */
    double execute_seconds;     /* spent inside syn_verify_batch (host wall clock of the call)      */
    int32_t live_requests, free_pages;
} syn_sched_stats;

/* m, kv: the model and its cache, or both NULL (policy only).  n_pages / page_size describe the
 * pool (they must be the values kv was allocated with; page_size must be 16).  max_batch_tokens
 * bounds the chunk tokens of one iteration (>= SYN_MAX_CHUNK); requests beyond it wait, in
 * arrival order.  Errors: SYN_E_INVALID_ARG, SYN_E_OOM. */
int syn_sched_create(syn_model *m, syn_kv *kv, uint32_t n_pages, uint32_t page_size, int32_t max_batch_tokens,
                     syn_sched **out);
void syn_sched_free(syn_sched *s);

/* A new request with its prompt (HOST, n_prompt >= 1; copied).  It joins the prefill queue
 * (get_next_prefill_request of Algorithm 1 returns the queue's entries in arrival order).
 * Errors: SYN_E_INVALID_ARG, SYN_E_SCHED_DUPLICATE, SYN_E_OOM. */
int syn_sched_add_request(syn_sched *s, int64_t req_id, const int32_t *prompt, int32_t n_prompt);

/* A verification request for a live request whose prompt is cached: n tokens (HOST, copied),
 * the first n_uncached >= 1 accepted by the device but not cached in the cloud, the rest
 * pending-verify drafts (Sec. 3.4).  1 <= n <= SYN_MAX_CHUNK.  One chunk per request may wait.
 * Errors: SYN_E_INVALID_ARG, SYN_E_CHUNK_LEN, SYN_E_UNCACHED, SYN_E_SCHED_UNKNOWN_REQ,
 * SYN_E_SCHED_STATE. */
int syn_sched_add_verify(syn_sched *s, int64_t req_id, const int32_t *tokens, int32_t n, int32_t n_uncached);

/* Marks a request complete.  It leaves, and its pages are freed, at the next iteration boundary:
 * remove_completed runs when an iteration is committed and again before the next one is formed.
 * A chunk of it that still waits is discarded.
 * Errors: SYN_E_SCHED_UNKNOWN_REQ. */
int syn_sched_finish(syn_sched *s, int64_t req_id);

/* Forms the next iteration's batch by Algorithm 1 and returns it without running it.  Pages for
 * the chunk's positions are taken from the free list here; a request that cannot get its pages,
 * or that no longer fits max_batch_tokens, stays queued (counted in `deferred`).  A second peek
 * before commit returns the same batch.  If prefill requests wait but none of them can be served,
 * the iteration falls through to the verification requests (which is what frees pages).
 * Errors: SYN_E_INVALID_ARG; SYN_E_CAPACITY when requests wait but the pool has no pages for any
 * of them (nothing is batched; finishing a request and peeking again makes progress). */
int syn_sched_peek(syn_sched *s, syn_sched_batch *out);

/* Applies the results of the peeked batch (HOST arrays [n_req] in the batch's order, as
 * syn_verify_batch returns them): advances the cached lengths, moves requests whose prompt is
 * complete to the active set, runs remove_completed.  results (may be NULL) receives up to cap
 * entries, *n_results the number written.  With an idle batch only remove_completed runs.
 * Errors: SYN_E_INVALID_ARG, SYN_E_SCHED_NO_BATCH. */
int syn_sched_commit(syn_sched *s, const int32_t *accept_len, const int32_t *correction_token,
                     syn_sched_result *results, int32_t cap, int32_t *n_results);

/* One iteration of Algorithm 1's loop: peek, syn_verify_batch on cuda_stream, commit.
 * *kind receives what ran.  On an error of syn_verify_batch the batch stays peeked and nothing
 * is committed.  Errors: those of the three calls; SYN_E_INVALID_ARG without a model. */
int syn_sched_step(syn_sched *s, syn_sched_result *results, int32_t cap, int32_t *n_results, int32_t *kind,
                   void *cuda_stream);

int syn_sched_get_stats(const syn_sched *s, syn_sched_stats *out);

#ifdef __cplusplus
}
#endif
#endif
