// Verification-aware scheduler (paper Sec. 4.5, Algorithm 1): host bookkeeping around
// syn_verify_batch.  See include/synera_sched.h for the contract.
#include <algorithm>
#include <chrono>
#include <cstdint>
#include <cstring>
#include <deque>
#include <new>
#include <unordered_map>
#include <vector>

#include "../../include/synera_sched.h"

namespace {

struct Request {
    int64_t id = 0;
    std::vector<int32_t> pages;    // logical page k -> physical page
    int32_t ctx = 0;               // cached tokens
    std::vector<int32_t> prompt;   // prefill: the whole prompt
    int32_t prompt_pos = 0;        // prompt tokens already cached
    bool prefilling = true;
    std::vector<int32_t> chunk;    // waiting verification chunk
    int32_t u = 0;
    bool chunk_waiting = false;
    bool finished = false;
};

double now_s() {
    return std::chrono::duration<double>(std::chrono::steady_clock::now().time_since_epoch()).count();
}

}  // namespace

struct syn_sched {
    syn_model* m = nullptr;
    syn_kv* kv = nullptr;
    int32_t n_pages = 0, P = 16, budget = 0;
    std::vector<int32_t> free_pages;   // stack; the lowest id is on top at the start
    std::unordered_map<int64_t, Request> reqs;
    std::deque<int64_t> prefill_q, verify_q;   // arrival order
    // the peeked batch
    bool have_batch = false;
    bool idle_peeked = false;   // the last peek found nothing to run
    int32_t kind = SYN_SCHED_IDLE, max_pages = 0;
    std::vector<int64_t> ids;
    std::vector<int32_t> toks, offs, tables, ctx, unc, acc, cor;
    syn_sched_stats st;
};

namespace {

// Pages for positions [0, upto) of a request; false (and nothing taken) if the pool cannot give them.
bool reserve_pages(syn_sched* s, Request& r, int32_t upto) {
    const int32_t need = (upto + s->P - 1) / s->P - (int32_t)r.pages.size();
    if (need <= 0) return true;
    if ((int32_t)s->free_pages.size() < need) return false;
    for (int32_t k = 0; k < need; ++k) {
        r.pages.push_back(s->free_pages.back());
        s->free_pages.pop_back();
    }
    return true;
}

// remove_completed of Algorithm 1: finished requests leave, their pages return to the pool.
void remove_completed(syn_sched* s) {
    bool any = false;
    for (auto it = s->reqs.begin(); it != s->reqs.end();) {
        if (it->second.finished) {
            for (auto p = it->second.pages.rbegin(); p != it->second.pages.rend(); ++p) s->free_pages.push_back(*p);
            it = s->reqs.erase(it);
            any = true;
        } else {
            ++it;
        }
    }
    if (!any) return;
    auto gone = [&](int64_t id) { return s->reqs.find(id) == s->reqs.end(); };
    s->prefill_q.erase(std::remove_if(s->prefill_q.begin(), s->prefill_q.end(), gone), s->prefill_q.end());
    s->verify_q.erase(std::remove_if(s->verify_q.begin(), s->verify_q.end(), gone), s->verify_q.end());
}

void clear_batch(syn_sched* s) {
    s->have_batch = false;
    s->kind = SYN_SCHED_IDLE;
    s->max_pages = 0;
    s->ids.clear(); s->toks.clear(); s->offs.clear(); s->tables.clear(); s->ctx.clear(); s->unc.clear();
}

// One pass over a queue: every live entry joins the batch with its next chunk while the token
// budget lasts (arrival order: the first one that does not fit ends the pass) and the pool has
// pages for it (one that cannot get pages is skipped, later ones may still fit).
// Returns the number of live entries left waiting.
int64_t gather(syn_sched* s, const std::deque<int64_t>& q, bool prefill) {
    int32_t total = 0;
    int64_t waiting = 0;
    bool full = false;
    for (int64_t id : q) {
        auto it = s->reqs.find(id);
        if (it == s->reqs.end() || it->second.finished) continue;
        Request& r = it->second;
        const int32_t n = prefill ? std::min<int32_t>(SYN_MAX_CHUNK, (int32_t)r.prompt.size() - r.prompt_pos)
                                  : (int32_t)r.chunk.size();
        if (full || total + n > s->budget) {
            full = true;
            ++waiting;
            continue;
        }
        if (!reserve_pages(s, r, r.ctx + n)) {
            ++waiting;
            continue;
        }
        const int32_t* src = prefill ? r.prompt.data() + r.prompt_pos : r.chunk.data();
        s->ids.push_back(id);
        s->toks.insert(s->toks.end(), src, src + n);
        s->offs.push_back(total + n);
        s->ctx.push_back(r.ctx);
        s->unc.push_back(prefill ? n : r.u);
        s->max_pages = std::max<int32_t>(s->max_pages, (r.ctx + n + s->P - 1) / s->P);
        total += n;
    }
    return waiting;
}

}  // namespace

extern "C" int syn_sched_create(syn_model* m, syn_kv* kv, uint32_t n_pages, uint32_t page_size, int32_t max_batch_tokens,
                                syn_sched** out) {
    if (!out || n_pages == 0 || page_size != 16 || max_batch_tokens < SYN_MAX_CHUNK || (m == nullptr) != (kv == nullptr))
        return SYN_E_INVALID_ARG;
    syn_sched* s = new (std::nothrow) syn_sched();
    if (!s) return SYN_E_OOM;
    s->m = m; s->kv = kv;
    s->n_pages = (int32_t)n_pages; s->P = (int32_t)page_size; s->budget = max_batch_tokens;
    s->free_pages.resize(n_pages);
    for (uint32_t k = 0; k < n_pages; ++k) s->free_pages[k] = (int32_t)(n_pages - 1 - k);
    std::memset(&s->st, 0, sizeof(s->st));
    s->offs.reserve(64);
    *out = s;
    return SYN_OK;
}

extern "C" void syn_sched_free(syn_sched* s) { delete s; }

extern "C" int syn_sched_add_request(syn_sched* s, int64_t req_id, const int32_t* prompt, int32_t n_prompt) {
    if (!s || !prompt || n_prompt < 1) return SYN_E_INVALID_ARG;
    if (s->reqs.find(req_id) != s->reqs.end()) return SYN_E_SCHED_DUPLICATE;
    Request r;
    r.id = req_id;
    r.prompt.assign(prompt, prompt + n_prompt);
    s->reqs.emplace(req_id, std::move(r));
    s->prefill_q.push_back(req_id);
    return SYN_OK;
}

extern "C" int syn_sched_add_verify(syn_sched* s, int64_t req_id, const int32_t* tokens, int32_t n, int32_t n_uncached) {
    if (!s || !tokens) return SYN_E_INVALID_ARG;
    if (n < 1 || n > SYN_MAX_CHUNK) return SYN_E_CHUNK_LEN;
    if (n_uncached < 1 || n_uncached > n) return SYN_E_UNCACHED;
    auto it = s->reqs.find(req_id);
    if (it == s->reqs.end()) return SYN_E_SCHED_UNKNOWN_REQ;
    Request& r = it->second;
    if (r.finished || r.prefilling || r.chunk_waiting) return SYN_E_SCHED_STATE;
    r.chunk.assign(tokens, tokens + n);
    r.u = n_uncached;
    r.chunk_waiting = true;
    s->verify_q.push_back(req_id);
    return SYN_OK;
}

extern "C" int syn_sched_finish(syn_sched* s, int64_t req_id) {
    if (!s) return SYN_E_INVALID_ARG;
    auto it = s->reqs.find(req_id);
    if (it == s->reqs.end()) return SYN_E_SCHED_UNKNOWN_REQ;
    it->second.finished = true;
    return SYN_OK;
}

static void fill_out(const syn_sched* s, syn_sched_batch* out) {
    std::memset(out, 0, sizeof(*out));
    out->kind = s->kind;
    if (s->kind == SYN_SCHED_IDLE) return;
    out->n_req = (int32_t)s->ids.size();
    out->n_tokens = s->offs.back();
    out->max_pages = s->max_pages;
    out->req_ids = s->ids.data();
    out->chunk_tokens = s->toks.data();
    out->chunk_offsets = s->offs.data();
    out->page_tables = s->tables.data();
    out->ctx_lens = s->ctx.data();
    out->n_uncached = s->unc.data();
}

extern "C" int syn_sched_peek(syn_sched* s, syn_sched_batch* out) {
    if (!s || !out) return SYN_E_INVALID_ARG;
    if (!s->have_batch) {
        clear_batch(s);
        s->idle_peeked = false;
        remove_completed(s);   // requests finished since the last iteration ended leave before the next is formed
        s->offs.push_back(0);
        // prefill requests first; only when none could be batched, the verification requests
        int64_t waiting = gather(s, s->prefill_q, true);
        s->kind = SYN_SCHED_PREFILL;
        if (s->ids.empty()) {
            waiting += gather(s, s->verify_q, false);
            s->kind = SYN_SCHED_VERIFY;
        }
        if (s->ids.empty()) {
            clear_batch(s);
            if (waiting > 0) return SYN_E_CAPACITY;   // work is queued but the pool has no pages for any of it
            s->idle_peeked = true;                    // not held: the next peek looks at the queues again
        } else {
            s->st.deferred += waiting;
            const size_t B = s->ids.size();
            s->tables.assign(B * (size_t)s->max_pages, -1);
            for (size_t i = 0; i < B; ++i) {
                const Request& r = s->reqs.find(s->ids[i])->second;
                const int32_t used = (s->ctx[i] + (s->offs[i + 1] - s->offs[i]) + s->P - 1) / s->P;
                std::copy(r.pages.begin(), r.pages.begin() + used, s->tables.begin() + i * (size_t)s->max_pages);
            }
            s->have_batch = true;
        }
    }
    fill_out(s, out);
    return SYN_OK;
}

extern "C" int syn_sched_commit(syn_sched* s, const int32_t* accept_len, const int32_t* correction_token,
                                syn_sched_result* results, int32_t cap, int32_t* n_results) {
    if (!s || cap < 0 || (cap > 0 && !results)) return SYN_E_INVALID_ARG;
    if (!s->have_batch) {
        if (!s->idle_peeked) return SYN_E_SCHED_NO_BATCH;
        s->idle_peeked = false;
        s->st.iterations[SYN_SCHED_IDLE] += 1;
        remove_completed(s);
        if (n_results) *n_results = 0;
        return SYN_OK;
    }
    const int32_t B = (int32_t)s->ids.size();
    if (B > 0 && (!accept_len || !correction_token)) return SYN_E_INVALID_ARG;
    if (s->kind == SYN_SCHED_VERIFY)
        for (int32_t i = 0; i < B; ++i) {
            const int32_t n = s->offs[i + 1] - s->offs[i];
            if (accept_len[i] < 0 || accept_len[i] > n - s->unc[i]) return SYN_E_INVALID_ARG;
        }
    int32_t written = 0;
    for (int32_t i = 0; i < B; ++i) {
        Request& r = s->reqs.find(s->ids[i])->second;
        const int32_t n = s->offs[i + 1] - s->offs[i];
        syn_sched_result res;
        res.req_id = r.id;
        res.kind = s->kind;
        res.n_tokens = n;
        res.correction_token = correction_token[i];
        if (s->kind == SYN_SCHED_PREFILL) {
            r.ctx += n;
            r.prompt_pos += n;
            res.accept_len = 0;
            res.prompt_done = r.prompt_pos == (int32_t)r.prompt.size();
            if (res.prompt_done) {
                r.prefilling = false;
                r.prompt.clear();
                r.prompt.shrink_to_fit();
            }
        } else {
            // the u accepted tokens and the accepted drafts stay cached; the slots of rejected
            // drafts are overwritten by the request's next chunk
            r.ctx += s->unc[i] + accept_len[i];
            r.chunk_waiting = false;
            res.accept_len = accept_len[i];
            res.prompt_done = 1;
        }
        res.ctx_len = r.ctx;
        if (written < cap) results[written++] = res;
    }
    if (s->kind == SYN_SCHED_PREFILL) {
        auto done = [&](int64_t id) { auto it = s->reqs.find(id); return it == s->reqs.end() || !it->second.prefilling; };
        s->prefill_q.erase(std::remove_if(s->prefill_q.begin(), s->prefill_q.end(), done), s->prefill_q.end());
    } else if (s->kind == SYN_SCHED_VERIFY) {
        auto done = [&](int64_t id) { auto it = s->reqs.find(id); return it == s->reqs.end() || !it->second.chunk_waiting; };
        s->verify_q.erase(std::remove_if(s->verify_q.begin(), s->verify_q.end(), done), s->verify_q.end());
    }
    s->st.iterations[s->kind] += 1;
    s->st.requests[s->kind] += B;
    s->st.tokens[s->kind] += B ? s->offs.back() : 0;
    remove_completed(s);
    clear_batch(s);
    if (n_results) *n_results = written;
    return SYN_OK;
}

extern "C" int syn_sched_step(syn_sched* s, syn_sched_result* results, int32_t cap, int32_t* n_results, int32_t* kind,
                              void* cuda_stream) {
    if (!s || !s->m) return SYN_E_INVALID_ARG;
    const double t0 = now_s();
    syn_sched_batch b;
    int rc = syn_sched_peek(s, &b);
    if (rc) return rc;
    const double t1 = now_s();
    if (b.kind != SYN_SCHED_IDLE) {
        s->acc.resize(b.n_req);
        s->cor.resize(b.n_req);
        rc = syn_verify_batch(s->m, s->kv, b.n_req, b.req_ids, b.chunk_tokens, b.chunk_offsets, b.page_tables, b.max_pages,
                              b.ctx_lens, b.n_uncached, s->acc.data(), s->cor.data(), nullptr, cuda_stream);
        if (rc) return rc;
    }
    const double t2 = now_s();
    if (kind) *kind = b.kind;
    rc = syn_sched_commit(s, s->acc.data(), s->cor.data(), results, cap, n_results);
    const double t3 = now_s();
    s->st.host_seconds += (t1 - t0) + (t3 - t2);
    s->st.execute_seconds += t2 - t1;
    return rc;
}

extern "C" int syn_sched_get_stats(const syn_sched* s, syn_sched_stats* out) {
    if (!s || !out) return SYN_E_INVALID_ARG;
    *out = s->st;
    out->live_requests = (int32_t)s->reqs.size();
    out->free_pages = (int32_t)s->free_pages.size();
    return SYN_OK;
}
