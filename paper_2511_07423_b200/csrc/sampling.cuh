// Sampling-based verification behind the lm_head (paper Sec. 4.2: the device transmits the SLM's
// top-k / top-p probabilities; Sec. 3.1: draft and verify).  Two kernels over the fp32 logits the
// lm_head projection wrote:
//   topk_rows_kernel      the SYN_SAMPLE_MAX_K largest logits of every row that judges a draft,
//                         exact (radix select on the ordered bit pattern), ties to the lower id
//   sample_verify_kernel  per request: the LLM's kept distribution q per position, the keep test
//                         r * p(x~) < q(x~) draft by draft, the replacement from the positive part
//                         of q - p at the first draft not kept, one more token from q otherwise
// All uniform draws are inputs.  Sums run in a fixed serial order (at most 64 terms), so results do
// not depend on the launch shape.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace syn {

constexpr int SAMPLE_MAX_K = 64;
constexpr int TOPK_THREADS = 512;

__device__ __forceinline__ uint32_t f32_order_key(float x) {   // larger float <=> larger key
    const uint32_t u = __float_as_uint(x);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Request of a chunk row: the i with offsets[i] <= row < offsets[i + 1].
__device__ __forceinline__ int request_of_row(const int* __restrict__ offsets, int n_req, int row) {
    int lo = 0, hi = n_req - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (offsets[mid] <= row) lo = mid; else hi = mid - 1;
    }
    return lo;
}

constexpr int TOPK_CAND_CAP = 1024;

// One block per chunk row.  Rows before a request's index u - 1 judge nothing and are skipped.
// out_id / out_logit [T][SAMPLE_MAX_K]: the k largest logits in decreasing order (equal logits:
// increasing id); entries k.. hold id -1.
//
// Fast path: the k-th largest of the threads' own maxima is a threshold that at least k elements
// reach; the elements that reach it (about k in a row of distinct values) are collected and
// ranked exactly.  The maxima come from a pass over the row, or, when the projection that wrote
// the logits also stored the maximum of every 32-feature group (warp_max), from those few
// thousand values, so that the row itself is read once.  A row with so many elements at the threshold that
// they overflow the candidate buffer (long runs of equal logits) takes the radix path instead:
// select the k-th largest bit pattern byte by byte, then gather in index order.
__global__ void __launch_bounds__(TOPK_THREADS)
topk_rows_kernel(const float* __restrict__ logits, int V, const int* __restrict__ offsets, const int* __restrict__ uncached,
                 int n_req, int k, const uint32_t* __restrict__ warp_max, int n_warp_max, int* __restrict__ out_id,
                 float* __restrict__ out_logit) {
    __shared__ uint32_t tmax[TOPK_THREADS];
    __shared__ int cand_id[TOPK_CAND_CAP];
    __shared__ float cand_logit[TOPK_CAND_CAP];
    __shared__ uint32_t hist[256];
    __shared__ uint32_t sel[2];                 // radix path: prefix, remaining count
    __shared__ int warp_gt[TOPK_THREADS / 32], warp_eq[TOPK_THREADS / 32];
    __shared__ int needed, n_cand;
    __shared__ uint32_t tau;
    const int row = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    pdl_wait();
    if (tid == 0) {
        const int i = request_of_row(offsets, n_req, row);
        needed = row - offsets[i] >= uncached[i] - 1;
        n_cand = 0;
    }
    __syncthreads();
    if (!needed) return;
    const float* x = logits + (size_t)row * V;
    const int kk = min(k, V);
    int* oid = out_id + (size_t)row * SAMPLE_MAX_K;
    float* ol = out_logit + (size_t)row * SAMPLE_MAX_K;
    if (tid < SAMPLE_MAX_K && tid >= kk) { oid[tid] = -1; ol[tid] = 0.f; }

    // ---- fast path (all comparisons on the ordered bit patterns; 0 stands for "no element")
    uint32_t mx = 0u;
    if (warp_max && n_warp_max * 32 >= V) {
        const uint32_t* gm = warp_max + (size_t)row * n_warp_max;
        for (int i = tid; i < n_warp_max; i += TOPK_THREADS) mx = max(mx, gm[i]);
    } else {
        for (int i = tid; i < V; i += TOPK_THREADS) mx = max(mx, f32_order_key(x[i]));
    }
    tmax[tid] = mx;
    __syncthreads();
    {
        int rank = 0;
        for (int j = 0; j < TOPK_THREADS; ++j) rank += tmax[j] > mx || (tmax[j] == mx && j < tid);
        if (rank == kk - 1) tau = mx;
    }
    __syncthreads();
    const uint32_t thr = tau;   // 0 when fewer than kk threads saw an element: then every element is a candidate
    auto offer = [&](int i, float v) {
        if (f32_order_key(v) >= thr) {
            const int pos = atomicAdd(&n_cand, 1);
            if (pos < TOPK_CAND_CAP) { cand_id[pos] = i; cand_logit[pos] = v; }
        }
    };
    if ((V & 3) == 0) {   // rows start 16-byte aligned: four logits a load
        const float4* x4 = reinterpret_cast<const float4*>(x);
        for (int i = tid; i < (V >> 2); i += TOPK_THREADS) {
            const float4 v = x4[i];
            offer(4 * i, v.x); offer(4 * i + 1, v.y); offer(4 * i + 2, v.z); offer(4 * i + 3, v.w);
        }
    } else {
        for (int i = tid; i < V; i += TOPK_THREADS) offer(i, x[i]);
    }
    __syncthreads();
    int nc = n_cand;
    if (nc > TOPK_CAND_CAP) {
        // ---- radix path: afterwards sel[0] is the key of the kk-th largest element and sel[1] how
        // many elements with exactly that key belong to the kk largest
        if (tid == 0) { sel[0] = 0u; sel[1] = (uint32_t)kk; }
        __syncthreads();
        uint32_t mask = 0u;
        for (int pass = 0; pass < 4; ++pass) {
            const int shift = 24 - 8 * pass;
            for (int b = tid; b < 256; b += TOPK_THREADS) hist[b] = 0u;
            __syncthreads();
            const uint32_t prefix = sel[0];
            for (int i = tid; i < V; i += TOPK_THREADS) {
                const uint32_t key = f32_order_key(x[i]);
                if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
            }
            __syncthreads();
            if (tid == 0) {
                uint32_t rem = sel[1], cum = 0u;
                int b = 255;
                for (; b > 0; --b) {
                    if (cum + hist[b] >= rem) break;
                    cum += hist[b];
                }
                sel[0] = prefix | ((uint32_t)b << shift);
                sel[1] = rem - cum;
            }
            mask |= 255u << shift;
            __syncthreads();
        }
        const uint32_t kstar = sel[0];
        const int take_eq = (int)sel[1];
        const int n_gt = kk - take_eq;
        // gather in index order: every element above the threshold, and the first take_eq equal to
        // it.  A warp owns a contiguous range, so ranks inside the row are prefix counts.
        const int per_warp = ((V + (TOPK_THREADS / 32) - 1) / (TOPK_THREADS / 32) + 31) / 32 * 32;
        const int w0 = min(V, warp * per_warp), w1 = min(V, w0 + per_warp);
        int c_gt = 0, c_eq = 0;
        for (int base = w0; base < w1; base += 32) {
            const int i = base + lane;
            const uint32_t key = i < w1 ? f32_order_key(x[i]) : 0u;
            c_gt += __popc(__ballot_sync(0xFFFFFFFFu, i < w1 && key > kstar));
            c_eq += __popc(__ballot_sync(0xFFFFFFFFu, i < w1 && key == kstar));
        }
        if (lane == 0) { warp_gt[warp] = c_gt; warp_eq[warp] = c_eq; }
        __syncthreads();
        int gt_base = 0, eq_base = 0;
        for (int w = 0; w < warp; ++w) { gt_base += warp_gt[w]; eq_base += warp_eq[w]; }
        const uint32_t lt = (1u << lane) - 1u;
        for (int base = w0; base < w1; base += 32) {
            const int i = base + lane;
            const float v = i < w1 ? x[i] : 0.f;
            const uint32_t key = i < w1 ? f32_order_key(v) : 0u;
            const uint32_t m_gt = __ballot_sync(0xFFFFFFFFu, i < w1 && key > kstar);
            const uint32_t m_eq = __ballot_sync(0xFFFFFFFFu, i < w1 && key == kstar);
            if (i < w1 && key > kstar) {
                const int r = gt_base + __popc(m_gt & lt);
                if (r < n_gt) { cand_id[r] = i; cand_logit[r] = v; }
            } else if (i < w1 && key == kstar) {
                const int r = eq_base + __popc(m_eq & lt);
                if (r < take_eq) { cand_id[n_gt + r] = i; cand_logit[n_gt + r] = v; }
            }
            gt_base += __popc(m_gt);
            eq_base += __popc(m_eq);
        }
        __syncthreads();
        nc = kk;
    }
    // ---- rank the candidates (decreasing logit, then increasing id); the first kk are the result
    for (int c = tid; c < nc; c += TOPK_THREADS) {
        const float v = cand_logit[c];
        const int id = cand_id[c];
        int rank = 0;
        for (int j = 0; j < nc; ++j) rank += (cand_logit[j] > v) || (cand_logit[j] == v && cand_id[j] < id);
        if (rank < kk) { oid[rank] = id; ol[rank] = v; }
    }
}

struct SampleParams {
    const int* tokens;        // [T] chunk tokens
    const int* offsets;       // [n_req + 1]
    const int* uncached;      // [n_req]
    const int* topk_id;       // [T][SAMPLE_MAX_K]
    const float* topk_logit;  // [T][SAMPLE_MAX_K]
    const int* slm_id;        // [T][slm_k]: row t = the distribution chunk token t was drawn from
    const float* slm_prob;    // [T][slm_k]
    const float* rand_accept; // [T]
    const float* rand_sample; // [n_req]
    int* accept_len;          // [n_req]
    int* correction;          // [n_req]
    int n_req, top_k, slm_k;
    float top_p, inv_temperature;
};

// One block of SAMPLE_MAX_K threads per request; thread t owns the t-th most probable kept token.
__global__ void __launch_bounds__(SAMPLE_MAX_K)
sample_verify_kernel(SampleParams p) {
    __shared__ float w[SAMPLE_MAX_K], q[SAMPLE_MAX_K], res[SAMPLE_MAX_K];
    __shared__ int ids[SAMPLE_MAX_K], by_id[SAMPLE_MAX_K];
    __shared__ int m_keep, decision, picked;
    __shared__ float kept_mass;
    const int i = blockIdx.x, t = threadIdx.x;
    pdl_wait();
    const int b = p.offsets[i], n = p.offsets[i + 1] - b, u = p.uncached[i];

    // q of chunk row `row` into ids[] / q[] (entries m_keep.. are zero)
    auto build_q = [&](int row) {
        const int id = p.topk_id[(size_t)row * SAMPLE_MAX_K + t];
        const float l0 = p.topk_logit[(size_t)row * SAMPLE_MAX_K];
        const float lt = p.topk_logit[(size_t)row * SAMPLE_MAX_K + t];
        const bool live = t < p.top_k && id >= 0;
        ids[t] = live ? id : -1;
        w[t] = live ? expf((lt - l0) * p.inv_temperature) : 0.f;
        __syncthreads();
        if (t == 0) {
            float total = 0.f;
            int kk = 0;
            for (int s = 0; s < SAMPLE_MAX_K; ++s) { total += w[s]; kk += ids[s] >= 0; }
            int m = kk;
            if (p.top_p < 1.f) {
                const float want = p.top_p * total;
                float c = 0.f;
                for (int s = 0; s < kk; ++s) {
                    c += w[s];
                    if (c >= want) { m = s + 1; break; }
                }
            }
            float kept = 0.f;
            for (int s = 0; s < m; ++s) kept += w[s];
            m_keep = m;
            kept_mass = kept;
        }
        __syncthreads();
        q[t] = t < m_keep ? w[t] / kept_mass : 0.f;
        __syncthreads();
    };
    // inverse CDF over the kept tokens in increasing id with weights wt[]; result in `picked`
    auto draw = [&](const float* wt, float r) {
        const int m = m_keep;
        if (t < m) {
            int rank = 0;
            for (int s = 0; s < m; ++s) rank += ids[s] < ids[t];
            by_id[rank] = t;
        }
        __syncthreads();
        if (t == 0) {
            float total = 0.f;
            for (int s = 0; s < m; ++s) total += wt[by_id[s]];
            int pick = -1;
            if (total > 0.f) {
                const float target = r * total;
                float c = 0.f;
                for (int s = 0; s < m; ++s) {
                    const float ws = wt[by_id[s]];
                    if (ws <= 0.f) continue;
                    c += ws;
                    pick = ids[by_id[s]];
                    if (target < c) break;
                }
            }
            picked = pick >= 0 ? pick : ids[0];   // an empty positive part: the most probable token
        }
        __syncthreads();
    };

    int a = 0;
    for (int j = 0; j < n - u; ++j) {
        const int td = b + u + j;              // row of the draft token
        build_q(td - 1);
        const int x = p.tokens[td];
        if (t == 0) {
            float qx = 0.f, px = 0.f;
            for (int s = 0; s < m_keep; ++s) qx += ids[s] == x ? q[s] : 0.f;
            for (int e = 0; e < p.slm_k; ++e) px += p.slm_id[(size_t)td * p.slm_k + e] == x ? p.slm_prob[(size_t)td * p.slm_k + e] : 0.f;
            decision = p.rand_accept[td] * px < qx;
        }
        __syncthreads();
        if (decision) {
            ++a;
            continue;
        }
        // positive part of q - p over the kept tokens
        float pon = 0.f;
        if (t < m_keep)
            for (int e = 0; e < p.slm_k; ++e)
                pon += p.slm_id[(size_t)td * p.slm_k + e] == ids[t] ? p.slm_prob[(size_t)td * p.slm_k + e] : 0.f;
        res[t] = t < m_keep ? fmaxf(q[t] - pon, 0.f) : 0.f;
        __syncthreads();
        draw(res, p.rand_sample[i]);
        if (t == 0) { p.accept_len[i] = a; p.correction[i] = picked; }
        return;
    }
    build_q(b + n - 1);
    draw(q, p.rand_sample[i]);
    if (t == 0) { p.accept_len[i] = a; p.correction[i] = picked; }
}

}  // namespace syn
