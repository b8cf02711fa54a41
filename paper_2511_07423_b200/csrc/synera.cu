// Host side of the library: C ABI, weight packing, KV pool, step planner and the launch
// sequence of one verification step.  See include/synera.h for the contract of every entry point.
#include "../../include/synera.h"

#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <chrono>
#include <cmath>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "attention2.cuh"
#include "gemm.cuh"
#include "gemm2.cuh"
#include "sampling.cuh"

using namespace syn;
typedef __nv_bfloat16 bf16;
// Slot of one helper part's stored accumulators: two tiles of 128 features x up to 256 tokens, fp32.
constexpr size_t GEMM_FIX_SLOT_BYTES = (size_t)2 * 128 * 256 * 4;
constexpr int GEMM_FLAG_INTS = 4;   // arrival / release counters of the exchanges: ints per SM
constexpr int GEMM_MAX_SPLITS = 8;   // most CTAs that share one pair tile's K range
// Limit of the kernels' bounded waits in SM cycles (syn_debug_set_spin_limit; tests shorten it).
static long long g_spin_limit = SYN_SPIN_LIMIT_CYCLES;
// 0: every projection takes the kernel its shape calls for; 1: the one-CTA kernel always (syn_debug_set_schedule).
static int g_schedule = 0;
// Attention kernel: 0 = whichever the planner's cost model makes cheaper for the batch, 1 = warp-level MMAs
// (64-row tiles), 2 = tcgen05 (128-row tiles).
static int g_attention = 0;

// Name of the last CUDA error a call of this library met on this thread (for syn_last_cuda_error).
static thread_local const char* g_last_cuda_error = "";
static inline cudaError_t note_cuda(cudaError_t e) {
    if (e != cudaSuccess) g_last_cuda_error = cudaGetErrorName(e);
    return e;
}
// cudaGetLastError after a launch, recorded like any other failing call
static inline bool launch_ok() { return note_cuda(cudaGetLastError()) == cudaSuccess; }

#define CU_OK(expr)                              \
    do {                                         \
        cudaError_t _e = note_cuda(expr);        \
        if (_e != cudaSuccess) {                 \
            (void)cudaGetLastError();            \
            return _e == cudaErrorMemoryAllocation ? SYN_E_OOM : SYN_E_CUDA; \
        }                                        \
    } while (0)

// Launch with programmatic stream serialization: the kernel may start while its predecessor in the
// stream still runs; every kernel of the step calls pdl_wait() before it touches anything an earlier
// kernel produces or still reads.
template <typename... KArgs, typename... Args>
static cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr;
    memset(&attr, 0, sizeof(attr));
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return note_cuda(cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...));
}

// The same for a kernel whose CTAs form clusters of two.
template <typename... KArgs, typename... Args>
static cudaError_t launch_pdl_pairs(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    memset(attr, 0, sizeof(attr));
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return note_cuda(cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...));
}

// ------------------------------------------------------------------------------------------ small kernels

// Token embedding (paper Sec. 4.5: the flattened batch enters the transformer), the first layer's
// GEMM operand bf16(x * gain) with the sums of x^2 per 32 features its RMSNorm scale is made of,
// RoPE table, argmax reset.
__global__ void __launch_bounds__(256)
prep_kernel(const bf16* __restrict__ embed, const int* __restrict__ tokens, const int* __restrict__ pos,
            const bf16* __restrict__ gain, const double* __restrict__ inv_freq, float* __restrict__ x,
            op16* __restrict__ xg, float* __restrict__ ssq, float2* __restrict__ rope, unsigned long long* __restrict__ best,
            int d, int half) {
    const int t = blockIdx.x, lane = threadIdx.x & 31;
    pdl_launch_dependents();
    pdl_wait();
    const bf16* e = embed + (size_t)tokens[t] * d;
    for (int f0 = (threadIdx.x >> 5) * 32; f0 < d; f0 += blockDim.x) {   // one warp per group of 32 features
        const int f = f0 + lane;
        const float v = __bfloat162float(e[f]);
        x[(size_t)t * d + f] = v;
        xg[(size_t)t * d + f] = to_op(v * __bfloat162float(gain[f]));
        float ss = v * v;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
        if (lane == 0) ssq[(size_t)t * (d >> 5) + (f0 >> 5)] = ss;
    }
    if (threadIdx.x == 0) best[t] = 0ull;
    for (int i = threadIdx.x; i < half; i += blockDim.x) {
        double sn, cs;
        sincos((double)pos[t] * inv_freq[i], &sn, &cs);
        rope[(size_t)t * half + i] = make_float2((float)cs, (float)sn);
    }
}

// Greedy verification (paper Sec. 3.1 "draft & verify", Sec. 4.5): one thread per request.
__global__ void verify_kernel(const unsigned long long* __restrict__ best, const int* __restrict__ tokens,
                              const int* __restrict__ offsets, const int* __restrict__ n_uncached, int n_req,
                              int* __restrict__ accept_len, int* __restrict__ correction, int* __restrict__ top1_out) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    pdl_wait();
    if (i >= n_req) return;
    const int b = offsets[i], n = offsets[i + 1] - b, u = n_uncached[i];
    if (top1_out)
        for (int j = 0; j < n; ++j) top1_out[b + j] = (int)(0xFFFFFFFFu - (uint32_t)(best[b + j] & 0xFFFFFFFFull));
    int a = 0;
    while (a < n - u && (int)(0xFFFFFFFFu - (uint32_t)(best[b + u - 1 + a] & 0xFFFFFFFFull)) == tokens[b + u + a]) ++a;
    accept_len[i] = a;
    correction[i] = (int)(0xFFFFFFFFu - (uint32_t)(best[b + u - 1 + a] & 0xFFFFFFFFull));
}

// Copy K/V of logical positions between a dense bf16 [n_pos][Hkv][hd] buffer and the paged pool (half precision).
__global__ void kv_copy_kernel(op16* pool_layer, const int* __restrict__ slots, bf16* k, bf16* v, int n_kv_heads, int hd,
                               int page_size, int to_pool) {
    const int i = blockIdx.x;
    const int s = slots[i], page = s / page_size, row = s % page_size;
    for (int e = threadIdx.x; e < n_kv_heads * hd; e += blockDim.x) {
        const int h = e / hd, dd = e % hd;
        const size_t ok = ((((size_t)page * n_kv_heads + h) * 2 + 0) * page_size + row) * hd + dd;
        const size_t ov = ok + (size_t)page_size * hd;
        const size_t oi = (size_t)i * n_kv_heads * hd + e;
        if (to_pool) {
            pool_layer[ok] = to_op(__bfloat162float(k[oi]));
            pool_layer[ov] = to_op(__bfloat162float(v[oi]));
        } else {
            k[oi] = __float2bfloat16(__half2float(pool_layer[ok]));
            v[oi] = __float2bfloat16(__half2float(pool_layer[ov]));
        }
    }
}

// ------------------------------------------------------------------------------------------ objects

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn g_encode = nullptr;

static int load_driver_entry() {
    if (g_encode) return SYN_OK;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    CU_OK(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
    if (!fn || qres != cudaDriverEntryPointSuccess) return SYN_E_CUDA;
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    return SYN_OK;
}

// 2-D 16-bit row-major [rows][cols] (pitch in elements), box = box_rows x 64 columns, 128-byte swizzle.
static int make_map_2d(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols, uint64_t pitch, uint32_t box_rows) {
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {pitch * 2};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g_encode(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SYN_OK : SYN_E_CUDA;
}

// 2-D view of a packed weight matrix for the CTA-pair kernel: rows of 128 bytes (64 bf16), no
// swizzle (the tiles already are shared-memory images); one box = the two 128-row tiles of a
// feature pair for one k-block (QUAD items) or one of them (DUO items).
struct WMaps {
    CUtensorMap quad, duo;
};
static int make_wmaps(const void* packed, int packed_rows, int K, WMaps* out) {
    const uint64_t n_pairs = (uint64_t)((packed_rows + 511) / 512 * 2), nkb = (uint64_t)((K + 63) / 64);
    cuuint64_t dims[2] = {64, n_pairs * nkb * 256};
    cuuint64_t strides[1] = {128};
    cuuint32_t estr[2] = {1, 1};
    for (int k = 0; k < 2; ++k) {
        cuuint32_t box[2] = {64, k == 0 ? 256u : 128u};
        if (g_encode(k == 0 ? &out->quad : &out->duo, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(packed), dims, strides,
                     box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return SYN_E_CUDA;
    }
    return SYN_OK;
}

struct syn_model {
    syn_model_desc desc;
    int f_pad, n_sm, gu_rows, qkv_rows, v_rows;
    bf16 *embed = nullptr, *final_norm = nullptr;
    op16* lm_head = nullptr;
    std::vector<op16*> wqkv, wo, wgu, wd;                 // projections in the packed tile layout (half precision)
    std::vector<bf16*> norm1, norm2;
    std::vector<WMaps> tm_wqkv, tm_wo, tm_wgu, tm_wd;      // their tensor maps
    WMaps tm_lm_head;
    double* inv_freq = nullptr;
    int* status_dev = nullptr;
    // workspace (grow-only)
    int t_cap = 0;
    float *x = nullptr, *ssq = nullptr;   // residual stream; sums of x^2 per token and 32 features
    op16 *xn = nullptr,   // half(x * gain of the next RMSNorm): the operand of the qkv, gate/up and lm_head projections
         *q = nullptr, *attn = nullptr, *act = nullptr;
    float2* rope = nullptr;
    unsigned long long* best = nullptr;
    int *acc_dev = nullptr, *corr_dev = nullptr;
    int b_cap = 0;
    CUtensorMap tm_xn, tm_attn, tm_act, tm_q, tm_q4;
    float* fix_part = nullptr;      // stored accumulators of K-split remainder tiles (one slot per SM)
    int* fix_flag = nullptr;        // their arrival / release counters, [GEMM_FLAG_INTS * n_sm], zero between launches
    float* part_o = nullptr;
    float2* part_ml = nullptr;
    int* group_count = nullptr;     // per merge group: partial items completed (zero between launches)
    int part_cap = 0;
    syn_plan* scratch_plan = nullptr;
    // sampling-based verification (grow-only): logits of a step, the rows' top-k lists, the
    // transmitted SLM distributions and the uniform draws
    struct SampleWs {
        float *logits = nullptr, *topk_logit = nullptr, *slm_prob = nullptr, *rand_accept = nullptr, *rand_sample = nullptr;
        int *topk_id = nullptr, *slm_id = nullptr;
        uint32_t* warp_max = nullptr;   // [t_cap][v_rows / 32]: per-group maxima stored by the lm_head epilogue
        size_t logits_cap = 0;
        int t_cap = 0, b_cap = 0, slm_cap = 0;
    } sw;
    int* pinned_out = nullptr;
    int pinned_out_cap = 0;
    // what syn_last_step_stats reports: the counters of the last step launched on this model and,
    // with profiling on, its device time (events around the whole step) and the wall time of the
    // blocking call
    syn_step_stats last_stats;
    bool have_last = false, step_timed = false;
    cudaEvent_t step_a = nullptr, step_b = nullptr;
    double last_wall_ms = 0.0;
    // per-class event timing
    bool profile = false;
    struct Ev { cudaEvent_t a, b; int cls; };
    std::vector<Ev> ev_used, ev_free;
};

// Brackets one launch with events when profiling is on.
struct ProfScope {
    syn_model* m; cudaStream_t st; syn_model::Ev ev; bool on;
    ProfScope(syn_model* m_, int cls, cudaStream_t st_) : m(m_), st(st_), on(m_ && m_->profile) {
        if (!on) return;
        if (!m->ev_free.empty()) { ev = m->ev_free.back(); m->ev_free.pop_back(); }
        else if (cudaEventCreate(&ev.a) != cudaSuccess || cudaEventCreate(&ev.b) != cudaSuccess) { on = false; return; }
        ev.cls = cls;
        cudaEventRecord(ev.a, st);
    }
    ~ProfScope() {
        if (!on) return;
        cudaEventRecord(ev.b, st);
        m->ev_used.push_back(ev);
    }
};

struct syn_kv {
    syn_model* model;
    op16* pool = nullptr;   // half precision (K and V enter and leave through syn_kv_import / syn_kv_export as bf16)
    uint32_t n_pages, page_size;
    size_t layer_elems;
    CUtensorMap tm_kv, tm_kv5;   // boxes of 32 rows (K and V of a page and head); of 16 rows (K or V) with both 64-dim halves
};

struct syn_plan {
    syn_step_stats stats;
    int n_req = 0, T = 0, max_pages = 0, n_items = 0, n_cta = 0, n_groups = 0, n_parts = 0;
    int row_cap = 64;   // rows of an attention item's tile: which attention kernel the work list was made for
    // one device buffer and its pinned host mirror
    uint8_t *dev = nullptr, *host = nullptr;
    size_t cap = 0, used = 0;
    // offsets into the buffer
    size_t o_tokens, o_pos, o_slot, o_offsets, o_uncached, o_tables, o_items, o_cta, o_groups;
    // the cache the page ids and slots were validated against
    const syn_kv* kv = nullptr;
    const void* kv_pool = nullptr;
    uint32_t kv_pages = 0;
    template <class Tp> Tp* d(size_t off) const { return reinterpret_cast<Tp*>(dev + off); }
    template <class Tp> Tp* h(size_t off) const { return reinterpret_cast<Tp*>(host + off); }
};

static void free_workspace(syn_model* m) {
    cudaFree(m->x); cudaFree(m->ssq); cudaFree(m->xn); cudaFree(m->q); cudaFree(m->attn); cudaFree(m->act);
    cudaFree(m->rope); cudaFree(m->best);
    m->x = m->ssq = nullptr; m->xn = m->q = m->attn = m->act = nullptr; m->rope = nullptr; m->best = nullptr;
    m->t_cap = 0;
}

static int ensure_workspace(syn_model* m, int T, int B, int n_parts) {
    const syn_model_desc& c = m->desc;
    const int q_dim = c.n_q_heads * c.head_dim;
    if (T > m->t_cap) {
        free_workspace(m);
        const int cap = (T + 255) / 256 * 256;
        CU_OK(cudaMalloc(&m->x, (size_t)cap * c.d_model * 4));
        CU_OK(cudaMalloc(&m->ssq, (size_t)cap * (c.d_model / 32) * 4));
        CU_OK(cudaMalloc(&m->xn, (size_t)cap * c.d_model * 2));
        CU_OK(cudaMalloc(&m->q, (size_t)cap * q_dim * 2));
        CU_OK(cudaMalloc(&m->attn, (size_t)cap * q_dim * 2));
        CU_OK(cudaMalloc(&m->act, (size_t)cap * m->f_pad * 2));
        CU_OK(cudaMalloc(&m->rope, (size_t)cap * (c.head_dim / 2) * 8));
        CU_OK(cudaMalloc(&m->best, (size_t)cap * 8));
        CU_OK(cudaMemset(m->xn, 0, (size_t)cap * c.d_model * 2));
        CU_OK(cudaMemset(m->q, 0, (size_t)cap * q_dim * 2));
        CU_OK(cudaMemset(m->attn, 0, (size_t)cap * q_dim * 2));
        CU_OK(cudaMemset(m->act, 0, (size_t)cap * m->f_pad * 2));
        m->t_cap = cap;
        int r;
        if ((r = make_map_2d(&m->tm_xn, m->xn, cap, c.d_model, c.d_model, GEMM_BOX_ROWS))) return r;
        if ((r = make_map_2d(&m->tm_attn, m->attn, cap, q_dim, q_dim, GEMM_BOX_ROWS))) return r;
        if ((r = make_map_2d(&m->tm_act, m->act, cap, m->f_pad, m->f_pad, GEMM_BOX_ROWS))) return r;
        // Q tile of the attention kernel: [token][128-byte line][64]; box = min(16, 64/G) tokens x (G * hd/64) lines
        const uint32_t G = c.n_q_heads / c.n_kv_heads, halves = c.head_dim / 64;
        const uint32_t box_tokens = std::min(16u, 64u / G);
        cuuint64_t dims[3] = {64, (cuuint64_t)q_dim / 64, (cuuint64_t)cap};
        cuuint64_t strides[2] = {128, (cuuint64_t)q_dim * 2};
        cuuint32_t box[3] = {64, G * halves, box_tokens};
        cuuint32_t estr[3] = {1, 1, 1};
        if (g_encode(&m->tm_q, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, m->q, dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return SYN_E_CUDA;
        // Q tile of the tensor-memory attention kernel: [token][head][64-dim half][64]; one box = one half of the
        // G heads of a kv head for min(32, 128 / G) tokens, i.e. rows (token, head) of 128 bytes
        cuuint64_t dims4[4] = {64, halves, c.n_q_heads, (cuuint64_t)cap};
        cuuint64_t strides4[3] = {128, (cuuint64_t)c.head_dim * 2, (cuuint64_t)q_dim * 2};
        cuuint32_t box4[4] = {64, 1, G, std::min((uint32_t)SYN_MAX_CHUNK, 128u / G)};
        cuuint32_t estr4[4] = {1, 1, 1, 1};
        if (g_encode(&m->tm_q4, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, m->q, dims4, strides4, box4, estr4,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return SYN_E_CUDA;
    }
    if (!m->fix_part) {
        CU_OK(cudaMalloc(&m->fix_part, (size_t)m->n_sm * GEMM_FIX_SLOT_BYTES));
        CU_OK(cudaMalloc(&m->fix_flag, (size_t)GEMM_FLAG_INTS * m->n_sm * 4));
        CU_OK(cudaMemset(m->fix_flag, 0, (size_t)GEMM_FLAG_INTS * m->n_sm * 4));
    }
    if (B > m->b_cap) {
        cudaFree(m->acc_dev); cudaFree(m->corr_dev);
        m->acc_dev = m->corr_dev = nullptr; m->b_cap = 0;
        const int cap = (B + 255) / 256 * 256;
        CU_OK(cudaMalloc(&m->acc_dev, (size_t)cap * 4));
        CU_OK(cudaMalloc(&m->corr_dev, (size_t)cap * 4));
        m->b_cap = cap;
    }
    if (n_parts > m->part_cap) {
        cudaFree(m->part_o); cudaFree(m->part_ml); cudaFree(m->group_count);
        m->part_o = nullptr; m->part_ml = nullptr; m->group_count = nullptr; m->part_cap = 0;
        const int cap = (n_parts + 255) / 256 * 256;
        CU_OK(cudaMalloc(&m->part_o, (size_t)cap * 128 * c.head_dim * 4));   // rows of the larger tile
        CU_OK(cudaMalloc(&m->part_ml, (size_t)cap * 128 * 8));
        CU_OK(cudaMalloc(&m->group_count, (size_t)cap * 4));   // a group has >= 2 parts: cap/2 would do
        CU_OK(cudaMemset(m->group_count, 0, (size_t)cap * 4));
        m->part_cap = cap;
    }
    return SYN_OK;
}

// ------------------------------------------------------------------------------------------ model

extern "C" void syn_model_free(syn_model* m) {
    if (!m) return;
    for (auto& v : {&m->wqkv, &m->wo, &m->wgu, &m->wd})
        for (op16* p : *v) cudaFree(p);
    for (auto& v : {&m->norm1, &m->norm2})
        for (bf16* p : *v) cudaFree(p);
    cudaFree(m->embed); cudaFree(m->lm_head); cudaFree(m->final_norm); cudaFree(m->inv_freq); cudaFree(m->status_dev);
    free_workspace(m);
    cudaFree(m->acc_dev); cudaFree(m->corr_dev); cudaFree(m->part_o); cudaFree(m->part_ml); cudaFree(m->group_count);
    cudaFree(m->fix_part); cudaFree(m->fix_flag);
    if (m->pinned_out) cudaFreeHost(m->pinned_out);
    cudaFree(m->sw.logits); cudaFree(m->sw.topk_logit); cudaFree(m->sw.topk_id); cudaFree(m->sw.slm_id);
    cudaFree(m->sw.slm_prob); cudaFree(m->sw.rand_accept); cudaFree(m->sw.rand_sample); cudaFree(m->sw.warp_max);
    if (m->scratch_plan) syn_plan_free(m->scratch_plan);
    for (auto* v : {&m->ev_used, &m->ev_free})
        for (auto& e : *v) { cudaEventDestroy(e.a); cudaEventDestroy(e.b); }
    if (m->step_a) cudaEventDestroy(m->step_a);
    if (m->step_b) cudaEventDestroy(m->step_b);
    delete m;
}

static int syn_model_load_impl(const syn_model_desc* desc, const syn_weights* w, syn_model** out) {
    if (!desc || !w || !out) return SYN_E_INVALID_ARG;
    const syn_model_desc c = *desc;
    if (c.flags != 0 || c.n_layers == 0 || c.vocab == 0 || c.d_ffn == 0) return SYN_E_INVALID_ARG;
    if (c.head_dim != 64 && c.head_dim != 128) return SYN_E_INVALID_ARG;
    if (c.d_model == 0 || c.d_model % 128 != 0 || c.d_ffn % 8 != 0) return SYN_E_INVALID_ARG;
    if (c.n_kv_heads == 0 || c.n_q_heads % c.n_kv_heads != 0 || c.n_q_heads / c.n_kv_heads > 8) return SYN_E_INVALID_ARG;
    if ((c.n_q_heads * c.head_dim) % 128 != 0 || (c.n_kv_heads * c.head_dim) % 128 != 0) return SYN_E_INVALID_ARG;
    if (!(c.rope_base > 0.f) || !(c.rms_eps >= 0.f)) return SYN_E_INVALID_ARG;
    if (!w->embed || !w->lm_head || !w->final_norm || !w->wq || !w->wk || !w->wv || !w->wo || !w->wg || !w->wu ||
        !w->wd || !w->norm1 || !w->norm2 || (w->location != 0 && w->location != 1))
        return SYN_E_INVALID_ARG;
    for (uint32_t l = 0; l < c.n_layers; ++l)
        if (!w->wq[l] || !w->wk[l] || !w->wv[l] || !w->wo[l] || !w->wg[l] || !w->wu[l] || !w->wd[l] || !w->norm1[l] ||
            !w->norm2[l])
            return SYN_E_INVALID_ARG;
    int dev = 0;
    cudaDeviceProp prop;
    CU_OK(cudaGetDevice(&dev));
    CU_OK(cudaGetDeviceProperties(&prop, dev));
    if (prop.major != 10) return SYN_E_ARCH;
    int r = load_driver_entry();
    if (r) return r;

    syn_model* m = new (std::nothrow) syn_model();
    if (!m) return SYN_E_OOM;
    m->desc = c;
    m->n_sm = prop.multiProcessorCount;
    m->f_pad = (c.d_ffn + 63) / 64 * 64;
    const int d = c.d_model, q_dim = c.n_q_heads * c.head_dim, kv_dim = c.n_kv_heads * c.head_dim, f = c.d_ffn;
    m->qkv_rows = q_dim + 2 * kv_dim;
    m->gu_rows = 2 * m->f_pad;
    m->v_rows = (c.vocab + 127) / 128 * 128;
    const int loc = w->location;
    const cudaMemcpyKind kind = loc ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice;

#define LOAD_FAIL(code)        \
    do {                       \
        syn_model_free(m);     \
        return (code);         \
    } while (0)
#define CU_M(expr)                                                                        \
    do {                                                                                  \
        cudaError_t _e = (expr);                                                          \
        if (_e != cudaSuccess) {                                                          \
            (void)cudaGetLastError();                                                     \
            LOAD_FAIL(_e == cudaErrorMemoryAllocation ? SYN_E_OOM : SYN_E_CUDA);          \
        }                                                                                 \
    } while (0)

    CU_M(cudaMalloc(&m->embed, (size_t)c.vocab * d * 2));
    CU_M(cudaMemcpy(m->embed, w->embed, (size_t)c.vocab * d * 2, kind));
    CU_M(cudaMalloc(&m->final_norm, (size_t)d * 2));
    CU_M(cudaMemcpy(m->final_norm, w->final_norm, (size_t)d * 2, kind));
    // staging buffer for host-resident sources (largest single matrix)
    bf16* stage[3] = {nullptr, nullptr, nullptr};
    if (!loc) {
        const size_t big = std::max((size_t)c.vocab * d, std::max((size_t)f * d, (size_t)q_dim * d));
        for (int k = 0; k < 3; ++k) {
            const size_t n = k == 0 ? big : (k == 1 ? std::max((size_t)f * d, (size_t)kv_dim * d) : (size_t)kv_dim * d);
            cudaError_t e = cudaMalloc(&stage[k], n * 2);
            if (e != cudaSuccess) {
                (void)cudaGetLastError();
                for (int j = 0; j < k; ++j) cudaFree(stage[j]);
                LOAD_FAIL(SYN_E_OOM);
            }
        }
    }
    // pack `n` row-major sources (rows[i] x src_k each) into a new tile-layout buffer of `packed_rows` x K
    auto pack = [&](const void* const* srcs, const int* rows, int n, int mode, int src_k, int packed_rows,
                    op16** out_ptr) -> int {
        const int n_mt = (packed_rows + 511) / 512 * 4, nkb = (src_k + 63) / 64;   // an even number of feature pairs (zero rows at the end)
        op16* outp = nullptr;
        cudaError_t e = cudaMalloc(&outp, (size_t)n_mt * nkb * 128 * 64 * 2);
        if (e != cudaSuccess) { (void)cudaGetLastError(); return SYN_E_OOM; }
        *out_ptr = outp;
        PackSrc ps;
        memset(&ps, 0, sizeof(ps));
        ps.mode = mode; ps.src_k = src_k; ps.hd = (int)c.head_dim;
        for (int i = 0; i < n; ++i) {
            ps.rows[i] = rows[i];
            if (loc) ps.p[i] = (const bf16*)srcs[i];
            else {
                if (cudaMemcpy(stage[i], srcs[i], (size_t)rows[i] * src_k * 2, cudaMemcpyHostToDevice) != cudaSuccess) {
                    cudaFree(outp);
                    *out_ptr = nullptr;
                    return SYN_E_CUDA;
                }
                ps.p[i] = stage[i];
            }
        }
        pack_weight_kernel<<<dim3(n_mt, nkb), 256>>>(ps, outp, nkb);
        if (cudaGetLastError() != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) {
            cudaFree(outp);
            *out_ptr = nullptr;
            return SYN_E_CUDA;
        }
        return SYN_OK;
    };
#define PACK_OR_FAIL(call)                                  \
    do {                                                    \
        int _r = (call);                                    \
        if (_r) {                                           \
            for (int j = 0; j < 3; ++j) cudaFree(stage[j]); \
            LOAD_FAIL(_r);                                  \
        }                                                   \
    } while (0)
    {
        const void* srcs[1] = {w->lm_head};
        const int rows[1] = {(int)c.vocab};
        PACK_OR_FAIL(pack(srcs, rows, 1, 0, d, c.vocab, &m->lm_head));
        PACK_OR_FAIL(make_wmaps(m->lm_head, m->v_rows, d, &m->tm_lm_head));
    }
    for (uint32_t l = 0; l < c.n_layers; ++l) {
        bf16 *n1 = nullptr, *n2 = nullptr;
        op16* pk = nullptr;
        {
            const void* srcs[3] = {w->wq[l], w->wk[l], w->wv[l]};
            const int rows[3] = {q_dim, kv_dim, kv_dim};
            PACK_OR_FAIL(pack(srcs, rows, 3, 2, d, m->qkv_rows, &pk));
            m->wqkv.push_back(pk);
            WMaps wm;
            PACK_OR_FAIL(make_wmaps(pk, m->qkv_rows, d, &wm));
            m->tm_wqkv.push_back(wm);
        }
        {
            const void* srcs[1] = {w->wo[l]};
            const int rows[1] = {d};
            PACK_OR_FAIL(pack(srcs, rows, 1, 0, q_dim, d, &pk));
            m->wo.push_back(pk);
            WMaps wm;
            PACK_OR_FAIL(make_wmaps(pk, d, q_dim, &wm));
            m->tm_wo.push_back(wm);
        }
        {   // a tile holds the gate and the up rows of the same 64 features; rows of the padded tail are zero
            const void* srcs[2] = {w->wg[l], w->wu[l]};
            const int rows[2] = {f, f};
            PACK_OR_FAIL(pack(srcs, rows, 2, 1, d, m->gu_rows, &pk));
            m->wgu.push_back(pk);
            WMaps wm;
            PACK_OR_FAIL(make_wmaps(pk, m->gu_rows, d, &wm));
            m->tm_wgu.push_back(wm);
        }
        {   // down projection: K = d_ffn, zero-padded to f_pad by the k-block tail
            const void* srcs[1] = {w->wd[l]};
            const int rows[1] = {d};
            PACK_OR_FAIL(pack(srcs, rows, 1, 0, f, d, &pk));
            m->wd.push_back(pk);
            WMaps wm;
            PACK_OR_FAIL(make_wmaps(pk, d, m->f_pad, &wm));
            m->tm_wd.push_back(wm);
        }
        CU_M(cudaMalloc(&n1, (size_t)d * 2)); m->norm1.push_back(n1);
        CU_M(cudaMalloc(&n2, (size_t)d * 2)); m->norm2.push_back(n2);
        CU_M(cudaMemcpy(n1, w->norm1[l], (size_t)d * 2, kind));
        CU_M(cudaMemcpy(n2, w->norm2[l], (size_t)d * 2, kind));
    }
    for (int j = 0; j < 3; ++j) cudaFree(stage[j]);
#undef PACK_OR_FAIL
    std::vector<double> inv(c.head_dim / 2);
    for (uint32_t i = 0; i < c.head_dim / 2; ++i) inv[i] = std::pow((double)c.rope_base, -2.0 * (double)i / (double)c.head_dim);
    CU_M(cudaMalloc(&m->inv_freq, inv.size() * 8));
    CU_M(cudaMemcpy(m->inv_freq, inv.data(), inv.size() * 8, cudaMemcpyHostToDevice));
    CU_M(cudaMalloc(&m->status_dev, 4));
    CU_M(cudaMemset(m->status_dev, 0, 4));
    CU_M(cudaFuncSetAttribute(gemm_kernel<GEMM_WAVES>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM_MAX));
    CU_M(cudaFuncSetAttribute(gemm_kernel<GEMM_KSPLIT>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM_MAX));
    CU_M(cudaFuncSetAttribute(gemm_kernel<GEMM_RSPLIT>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM_MAX));
    CU_M(cudaFuncSetAttribute(gemm2_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM_MAX));
    CU_M(cudaFuncSetAttribute(gemm2_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM_MAX));
    CU_M(cudaFuncSetAttribute(attn_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnSmem<128>::TOTAL));
    CU_M(cudaFuncSetAttribute(attn_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnSmem<64>::TOTAL));
    CU_M(cudaFuncSetAttribute(attn2_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, Attn2Smem<128>::TOTAL));
    CU_M(cudaFuncSetAttribute(attn2_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, Attn2Smem<64>::TOTAL));
    CU_M(cudaDeviceSynchronize());
    *out = m;
    return SYN_OK;
#undef CU_M
#undef LOAD_FAIL
}

// ------------------------------------------------------------------------------------------ KV pool

extern "C" void syn_kv_free(syn_kv* kv) {
    if (!kv) return;
    cudaFree(kv->pool);
    delete kv;
}

extern "C" int syn_kv_alloc(syn_model* m, uint32_t n_pages, uint32_t page_size, syn_kv** out) {
    if (!m || !out || n_pages == 0 || page_size != 16) return SYN_E_INVALID_ARG;
    const syn_model_desc& c = m->desc;
    const uint64_t blocks = (uint64_t)c.n_layers * n_pages * c.n_kv_heads * 2;
    if (blocks > 0x7FFFFFFFull) return SYN_E_INVALID_ARG;
    syn_kv* kv = new (std::nothrow) syn_kv();
    if (!kv) return SYN_E_OOM;
    kv->model = m;
    kv->n_pages = n_pages;
    kv->page_size = page_size;
    kv->layer_elems = (size_t)n_pages * c.n_kv_heads * 2 * page_size * c.head_dim;
    const size_t bytes = kv->layer_elems * c.n_layers * 2;
    cudaError_t e = cudaMalloc(&kv->pool, bytes);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        delete kv;
        return e == cudaErrorMemoryAllocation ? SYN_E_OOM : SYN_E_CUDA;
    }
    if (cudaMemset(kv->pool, 0, bytes) != cudaSuccess) {
        syn_kv_free(kv);
        return SYN_E_CUDA;
    }
    // pool as a 2-D tensor [blocks * 16 rows][head_dim]; a box of 32 rows x 64 columns is one
    // 64-element half of the K rows and the V rows of one (page, kv head)
    if (make_map_2d(&kv->tm_kv, kv->pool, blocks * page_size, c.head_dim, c.head_dim, 2 * page_size) != SYN_OK) {
        syn_kv_free(kv);
        return SYN_E_CUDA;
    }
    {
        // The 16 K rows (or the 16 V rows) of a page and head as one box for the tensor-memory attention
        // kernel, landing in shared memory as [rows 0-7: dims 0-63][rows 0-7: dims 64-127][rows 8-15: ...]:
        // the 8-row groups of consecutive boxes are then evenly spaced for either 64-dim half, which a tcgen05
        // operand descriptor needs.  Dimensions: dim in a half, row in a group, half, group, 16-row block.
        const cuuint64_t hd2 = (cuuint64_t)c.head_dim * 2;
        cuuint64_t dims[5] = {64, 8, c.head_dim / 64, 2, (cuuint64_t)blocks};
        cuuint64_t strides[4] = {hd2, 128, 8 * hd2, 16 * hd2};
        cuuint32_t box[5] = {64, 8, c.head_dim / 64, 2, 1};
        cuuint32_t estr[5] = {1, 1, 1, 1, 1};
        if (g_encode(&kv->tm_kv5, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 5, kv->pool, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
            syn_kv_free(kv);
            return SYN_E_CUDA;
        }
    }
    if (cudaDeviceSynchronize() != cudaSuccess) {
        syn_kv_free(kv);
        return SYN_E_CUDA;
    }
    *out = kv;
    return SYN_OK;
}

static int kv_copy(syn_kv* kv, uint32_t layer, const int32_t* page_table, int32_t pos0, int32_t n_pos, void* k, void* v,
                   void* stream, int to_pool) {
    if (!kv || !page_table || !k || !v || pos0 < 0 || n_pos <= 0 || layer >= kv->model->desc.n_layers)
        return SYN_E_INVALID_ARG;
    const int P = (int)kv->page_size;
    std::vector<int> slots(n_pos);
    for (int i = 0; i < n_pos; ++i) {
        const int p = pos0 + i, page = page_table[p / P];
        if (page < 0 || (uint32_t)page >= kv->n_pages) return SYN_E_PAGE_OOB;
        slots[i] = page * P + p % P;
    }
    int* d_slots = nullptr;
    CU_OK(cudaMalloc(&d_slots, (size_t)n_pos * 4));
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(d_slots, slots.data(), (size_t)n_pos * 4, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e == cudaSuccess) {
        const syn_model_desc& c = kv->model->desc;
        kv_copy_kernel<<<n_pos, 128, 0, st>>>(kv->pool + kv->layer_elems * layer, d_slots, (bf16*)k, (bf16*)v,
                                              c.n_kv_heads, c.head_dim, P, to_pool);
        e = cudaGetLastError();
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    }
    cudaFree(d_slots);
    return e == cudaSuccess ? SYN_OK : SYN_E_CUDA;
}

static int syn_kv_import_impl(syn_kv* kv, uint32_t layer, const int32_t* page_table, int32_t pos0, int32_t n_pos,
                             const void* k, const void* v, void* stream) {
    return kv_copy(kv, layer, page_table, pos0, n_pos, const_cast<void*>(k), const_cast<void*>(v), stream, 1);
}
static int syn_kv_export_impl(syn_kv* kv, uint32_t layer, const int32_t* page_table, int32_t pos0, int32_t n_pos, void* k,
                             void* v, void* stream) {
    return kv_copy(kv, layer, page_table, pos0, n_pos, k, v, stream, 0);
}

// ------------------------------------------------------------------------------------------ planner

extern "C" void syn_plan_free(syn_plan* p) {
    if (!p) return;
    cudaFree(p->dev);
    if (p->host) cudaFreeHost(p->host);
    delete p;
}

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Host-side result of planning one batch (no device involved).
struct HostPlan {
    int T = 0, n_cta = 0, n_parts = 0, row_cap = 64;
    std::vector<int> pos, slot, cta_begin;
    std::vector<AttnItem> items;          // sorted by CTA
    std::vector<MergeGroup> groups;
    syn_step_stats stats;
};

// Validate the batch, then build token positions, KV slots and the attention work list
// (the "flatten" of paper Sec. 4.5).  Pure host code.
static int plan_compute(const syn_model_desc& c, int P, uint32_t n_pages, int n_sm, int32_t n_req,
                        const int32_t* chunk_tokens, const int32_t* chunk_offsets, const int32_t* page_tables,
                        int32_t max_pages, const int32_t* ctx_lens, const int32_t* n_uncached, int attention, HostPlan& hp) {
    if (n_req <= 0 || !chunk_tokens || !chunk_offsets || !page_tables || !ctx_lens || max_pages <= 0 || n_sm <= 0)
        return SYN_E_INVALID_ARG;
    const int G = c.n_q_heads / c.n_kv_heads, Hkv = c.n_kv_heads;
    if (chunk_offsets[0] != 0) return SYN_E_INVALID_ARG;
    int64_t ctx_sum = 0, keys_seen = 0, kv_units = 0;
    for (int i = 0; i < n_req; ++i) {
        const int64_t n = (int64_t)chunk_offsets[i + 1] - chunk_offsets[i];
        if (n < 1 || n > SYN_MAX_CHUNK) return SYN_E_CHUNK_LEN;
        const int u = n_uncached ? n_uncached[i] : 1;
        if (u < 1 || u > n) return SYN_E_UNCACHED;
        if (ctx_lens[i] < 0) return SYN_E_INVALID_ARG;
        if ((int64_t)ctx_lens[i] + n > (int64_t)max_pages * P) return SYN_E_CAPACITY;
        const int used = (int)((ctx_lens[i] + n + P - 1) / P);
        const int32_t* row = page_tables + (size_t)i * max_pages;
        uint32_t worst = 0;   // a negative id is a large unsigned one
        for (int k = 0; k < used; ++k) worst = std::max(worst, (uint32_t)row[k]);
        if (worst >= n_pages) return SYN_E_PAGE_OOB;
        ctx_sum += ctx_lens[i];
        kv_units += ctx_lens[i] + n;
        keys_seen += n * (int64_t)ctx_lens[i] + n * (n + 1) / 2;
    }
    const int T = chunk_offsets[n_req];
    for (int t = 0; t < T; ++t)
        if (chunk_tokens[t] < 0 || (uint32_t)chunk_tokens[t] >= c.vocab) return SYN_E_TOKEN_OOB;
    std::vector<int>& pos = hp.pos;
    std::vector<int>& slot = hp.slot;
    pos.assign(T, 0);
    slot.assign(T, 0);
    for (int i = 0; i < n_req; ++i)
        for (int j = 0, b = chunk_offsets[i]; b + j < chunk_offsets[i + 1]; ++j) {
            const int pp = ctx_lens[i] + j;
            pos[b + j] = pp;
            slot[b + j] = page_tables[(size_t)i * max_pages + pp / P] * P + pp % P;
        }
    {
        // Two chunk tokens may not share a KV slot.  Inside a request the chunk's slots differ unless
        // two of its (at most three) pages are the same page; between requests they can only meet in
        // a page both chunks write.  So look at the pages first, and at the slots only if a page
        // is written twice.
        std::vector<int> pg;
        pg.reserve((size_t)n_req * 3);
        for (int i = 0; i < n_req; ++i) {
            const int first = ctx_lens[i] / P, last = (ctx_lens[i] + (chunk_offsets[i + 1] - chunk_offsets[i]) - 1) / P;
            for (int k = first; k <= last; ++k) pg.push_back(page_tables[(size_t)i * max_pages + k]);
        }
        std::sort(pg.begin(), pg.end());
        if (std::adjacent_find(pg.begin(), pg.end()) != pg.end()) {
            std::vector<int> s2(slot);
            std::sort(s2.begin(), s2.end());
            if (std::adjacent_find(s2.begin(), s2.end()) != s2.end()) return SYN_E_PAGE_ALIAS;
        }
    }
    // Attention work list: (request, kv head, token group, key range).  Cost of an item, in SM
    // cycles: its 64-key stages times a per-stage time that grows with the number of 16-row query
    // tiles (more tensor work per key byte), plus a fixed overhead per item; the figures are a
    // least-squares fit to per-CTA durations measured on full batches.  A key range is split only
    // when one unit alone would exceed a CTA's fair share: every split costs an fp32 partial and a
    // merge.
    const int n_cta_max = n_sm;
    // Two kernels: the warp-level-MMA one (row tiles of 64: a stage costs more the more 16-row tiles the
    // item has, and a chunk of more than 64 / G tokens is several items that each read the request's keys)
    // and the tensor-memory one (row tiles of 128: the same time per stage whatever the number of rows,
    // a larger fixed cost per item).  Unless one is asked for, the batch takes the cheaper by this model.
    static const int STAGE_COST[5] = {0, 1040, 1200, 1500, 1540};
    const int WIDE_STAGE_COST = 1450;
    auto total_of = [&](bool w) {
        const int tpg = w ? std::min(SYN_MAX_CHUNK, 128 / G) : std::min(16, 64 / G);
        int64_t sum = 0;
        for (int i = 0; i < n_req; ++i) {
            const int n = chunk_offsets[i + 1] - chunk_offsets[i];
            for (int j0 = 0; j0 < n; j0 += tpg) {
                const int nj = std::min(tpg, n - j0);
                sum += ((int64_t)((ctx_lens[i] + j0 + nj + 63) / 64) * (w ? WIDE_STAGE_COST : STAGE_COST[(nj * G + 15) / 16]) + (w ? 8000 : 5500)) * Hkv;
            }
        }
        return sum;
    };
    // (The tensor-memory kernel must win by 3 %: it draws more power, and under the power cap a step that uses it
    // runs its other kernels at a lower clock; at 544 tokens of the 8B shape the two kernels are level and the step
    // is not faster with it.)
    const bool wide = attention == 2 || (attention == 0 && total_of(true) * 103 < total_of(false) * 100);
    hp.row_cap = wide ? 128 : 64;
    const int tok_per_group = wide ? std::min(SYN_MAX_CHUNK, 128 / G) : std::min(16, 64 / G);
    const int ITEM_COST = wide ? 8000 : 5500, PART_COST = wide ? 4000 : 3000;
    auto unit_cost = [&](int L, int nj) {
        return (int64_t)((L + 63) / 64) * (wide ? WIDE_STAGE_COST : STAGE_COST[(nj * G + 15) / 16]) + ITEM_COST;
    };
    const int64_t total_cost = total_of(wide);
    const int64_t share = std::max<int64_t>(8 * (wide ? WIDE_STAGE_COST : STAGE_COST[4]) + ITEM_COST, (total_cost + n_cta_max - 1) / n_cta_max);
    std::vector<AttnItem> items;
    std::vector<int> item_cost;
    std::vector<MergeGroup>& groups = hp.groups;
    groups.clear();
    int n_parts = 0;
    for (int i = 0; i < n_req; ++i) {
        const int b = chunk_offsets[i], n = chunk_offsets[i + 1] - b;
        for (int j0 = 0; j0 < n; j0 += tok_per_group) {
            const int nj = std::min(tok_per_group, n - j0);
            const int L = ctx_lens[i] + j0 + nj;
            int np = (int)std::min<int64_t>(64, (unit_cost(L, nj) + share - 1) / share);
            int len = ((L + np - 1) / np + 63) / 64 * 64;
            np = (L + len - 1) / len;
            for (int h = 0; h < Hkv; ++h) {
                if (np > 1) {
                    MergeGroup g = {b + j0, nj, h, n_parts, np, 0, 0, 0};
                    groups.push_back(g);
                }
                for (int k = 0; k < np; ++k) {
                    AttnItem it = {b + j0, nj, h, i, k * len, std::min(L, (k + 1) * len), ctx_lens[i] + j0,
                                   np > 1 ? n_parts + k : -1, np > 1 ? (int)groups.size() - 1 : -1, 0, 0, 0};
                    items.push_back(it);
                    item_cost.push_back((int)unit_cost(it.kv_end - it.kv_begin, nj) + (np > 1 ? PART_COST : 0));
                }
                if (np > 1) n_parts += np;
            }
        }
    }
    const int n_items = (int)items.size();
    const int n_cta = std::min(n_cta_max, n_items);
    // longest first (equal costs: lower index first), each to the least loaded CTA (ties: lower CTA);
    // both orders are carried in one 64-bit key
    std::vector<int> order(n_items), owner(n_items);
    auto cost = [&](int i) { return item_cost[i]; };
    {
        // stable radix sort of the indices by decreasing cost, 11 bits a pass
        int top = 0;
        for (int i = 0; i < n_items; ++i) top = std::max(top, item_cost[i]);
        std::vector<int> tmp(n_items);
        for (int i = 0; i < n_items; ++i) order[i] = i;
        int hist[2048];
        for (int shift = 0; shift < 32 && (top >> shift) != 0; shift += 11) {
            memset(hist, 0, sizeof(hist));
            for (int i = 0; i < n_items; ++i) hist[2047 - ((item_cost[order[i]] >> shift) & 2047)]++;
            int run = 0;
            for (int b = 0; b < 2048; ++b) { const int h = hist[b]; hist[b] = run; run += h; }
            for (int i = 0; i < n_items; ++i) tmp[hist[2047 - ((item_cost[order[i]] >> shift) & 2047)]++] = order[i];
            order.swap(tmp);
        }
    }
    std::vector<int>& count = hp.cta_begin;
    count.assign(n_cta + 1, 0);
    {
        std::vector<uint64_t> heap(n_cta);   // (load << 16) | cta, smallest at the root
        for (int k = 0; k < n_cta; ++k) heap[k] = (uint64_t)k;   // all loads 0: already a heap
        for (int i : order) {
            const uint64_t top = heap[0];
            const int k = (int)(top & 0xFFFFu);
            owner[i] = k;
            count[k + 1]++;
            const uint64_t v = (((top >> 16) + (uint64_t)cost(i)) << 16) | (uint64_t)k;
            int at = 0;   // the root grows: sift it down
            for (;;) {
                int ch = 2 * at + 1;
                if (ch >= n_cta) break;
                if (ch + 1 < n_cta && heap[ch + 1] < heap[ch]) ++ch;
                if (heap[ch] >= v) break;
                heap[at] = heap[ch];
                at = ch;
            }
            heap[at] = v;
        }
    }
    // Local search on the greedy result: relieve the most loaded CTA by moving one of its items to
    // another CTA, or by exchanging it for a cheaper one, as long as that lowers the larger of the
    // two loads; partners are the least loaded CTAs.  Only when the greedy result is more than 1 %
    // above the mean; stops within 0.3 % of it.
    if (n_cta > 1) {
        std::vector<int64_t> load(n_cta, 0);
        int64_t sum = 0;
        for (int i = 0; i < n_items; ++i) {
            load[owner[i]] += cost(i);
            sum += cost(i);
        }
        const int64_t mean = sum / n_cta;
        if (*std::max_element(load.begin(), load.end()) > mean + mean / 100) {
            std::vector<std::vector<int>> held(n_cta);
            for (int i = 0; i < n_items; ++i) held[owner[i]].push_back(i);
            std::vector<int> by_load(n_cta);   // CTAs by increasing load, kept sorted
            for (int k = 0; k < n_cta; ++k) by_load[k] = k;
            auto lighter = [&](int x, int y) { return load[x] != load[y] ? load[x] < load[y] : x < y; };
            std::sort(by_load.begin(), by_load.end(), lighter);
            auto resort = [&](int k) {   // k's load changed: move it to its place
                int at = (int)(std::find(by_load.begin(), by_load.end(), k) - by_load.begin());
                while (at + 1 < n_cta && lighter(by_load[at + 1], k)) { by_load[at] = by_load[at + 1]; ++at; }
                while (at > 0 && lighter(k, by_load[at - 1])) { by_load[at] = by_load[at - 1]; --at; }
                by_load[at] = k;
            };
            const int64_t good = mean + mean / 333;
            const int n_cand = std::min(n_cta - 1, 16);
            for (int round = 0; round < 128; ++round) {
                const int hi = by_load[n_cta - 1];
                if (load[hi] <= good) break;
                int64_t best = load[hi];
                int bi = -1, bk = -1, bj = -1;   // position in held[hi], the other CTA, position in held[bk] (-1: move)
                for (int a = 0; a < (int)held[hi].size(); ++a) {
                    const int64_t ca = cost(held[hi][a]);
                    for (int q = 0; q < n_cand; ++q) {
                        const int k = by_load[q];
                        if (std::max(load[hi] - ca, load[k] + ca) < best) {
                            best = std::max(load[hi] - ca, load[k] + ca);
                            bi = a; bk = k; bj = -1;
                        }
                        for (int b2 = 0; b2 < (int)held[k].size(); ++b2) {
                            const int64_t dlt = ca - cost(held[k][b2]);
                            if (dlt > 0 && std::max(load[hi] - dlt, load[k] + dlt) < best) {
                                best = std::max(load[hi] - dlt, load[k] + dlt);
                                bi = a; bk = k; bj = b2;
                            }
                        }
                    }
                }
                if (bi < 0 || load[hi] - best < mean / 1000) break;   // nothing, or next to nothing, to gain
                const int ia = held[hi][bi];
                if (bj < 0) {
                    load[hi] -= cost(ia); load[bk] += cost(ia);
                    owner[ia] = bk;
                    held[bk].push_back(ia);
                    held[hi].erase(held[hi].begin() + bi);
                } else {
                    const int ib = held[bk][bj];
                    const int64_t dlt = cost(ia) - cost(ib);
                    load[hi] -= dlt; load[bk] += dlt;
                    owner[ia] = bk; owner[ib] = hi;
                    held[hi][bi] = ib; held[bk][bj] = ia;
                }
                resort(hi);
                resort(bk);
            }
            std::fill(count.begin(), count.end(), 0);
            for (int i = 0; i < n_items; ++i) count[owner[i] + 1]++;
        }
    }
    for (int k = 0; k < n_cta; ++k) count[k + 1] += count[k];
    hp.items.assign(n_items, AttnItem());
    {
        std::vector<int> cur(count.begin(), count.end() - 1);
        for (int i : order) hp.items[cur[owner[i]]++] = items[i];
    }
    hp.T = T; hp.n_cta = n_cta; hp.n_parts = n_parts;

    syn_step_stats& s = hp.stats;
    memset(&s, 0, sizeof(s));
    const double d = c.d_model, qd = (double)c.n_q_heads * c.head_dim, kd = (double)Hkv * c.head_dim;
    const double params = c.n_layers * (d * (qd + 2 * kd) + qd * d + 3.0 * d * c.d_ffn) + d * c.vocab;
    s.n_req = n_req; s.n_tokens = T; s.ctx_tokens = ctx_sum;
    s.weight_bytes = (int64_t)(params * 2);
    s.kv_read_bytes = kv_units * (int64_t)(2 * kd * 2) * c.n_layers;
    s.kv_write_bytes = (int64_t)T * (int64_t)(2 * kd * 2) * c.n_layers;
    s.dense_flops = 2.0 * T * params;
    s.attn_flops = 4.0 * qd * c.n_layers * (double)keys_seen;
    s.attn_items = n_items; s.attn_split_items = n_parts;
    s.kernel_launches = 1 + c.n_layers * 5 + 2;
    s.attn_rows = hp.row_cap;
    return SYN_OK;
}

// plan_compute, then pack everything into the plan's pinned buffer (grown on demand).
static int plan_build(syn_plan* p, syn_model* m, syn_kv* kv, int32_t n_req, const int32_t* chunk_tokens,
                      const int32_t* chunk_offsets, const int32_t* page_tables, int32_t max_pages, const int32_t* ctx_lens,
                      const int32_t* n_uncached) {
    if (!m || !kv || kv->model != m) return SYN_E_INVALID_ARG;
    HostPlan hp;
    int r = plan_compute(m->desc, (int)kv->page_size, kv->n_pages, m->n_sm, n_req, chunk_tokens, chunk_offsets, page_tables,
                         max_pages, ctx_lens, n_uncached, g_attention, hp);
    if (r) return r;
    const int T = hp.T, n_items = (int)hp.items.size(), n_cta = hp.n_cta;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    p->o_tokens = take((size_t)T * 4);
    p->o_pos = take((size_t)T * 4);
    p->o_slot = take((size_t)T * 4);
    p->o_offsets = take((size_t)(n_req + 1) * 4);
    p->o_uncached = take((size_t)n_req * 4);
    p->o_tables = take((size_t)n_req * max_pages * 4);
    p->o_items = take((size_t)n_items * sizeof(AttnItem));
    p->o_cta = take((size_t)(n_cta + 1) * 4);
    p->o_groups = take(std::max<size_t>(1, hp.groups.size()) * sizeof(MergeGroup));
    if (off > p->cap) {
        cudaFree(p->dev);
        if (p->host) cudaFreeHost(p->host);
        p->dev = p->host = nullptr;
        p->cap = 0;
        const size_t cap = align_up(off + off / 2, 4096);
        CU_OK(cudaMalloc(&p->dev, cap));
        CU_OK(cudaMallocHost(&p->host, cap));
        p->cap = cap;
    }
    p->used = off;
    memcpy(p->h<int>(p->o_tokens), chunk_tokens, (size_t)T * 4);
    memcpy(p->h<int>(p->o_pos), hp.pos.data(), (size_t)T * 4);
    memcpy(p->h<int>(p->o_slot), hp.slot.data(), (size_t)T * 4);
    memcpy(p->h<int>(p->o_offsets), chunk_offsets, (size_t)(n_req + 1) * 4);
    for (int i = 0; i < n_req; ++i) p->h<int>(p->o_uncached)[i] = n_uncached ? n_uncached[i] : 1;
    memcpy(p->h<int>(p->o_tables), page_tables, (size_t)n_req * max_pages * 4);
    memcpy(p->h<AttnItem>(p->o_items), hp.items.data(), (size_t)n_items * sizeof(AttnItem));
    memcpy(p->h<int>(p->o_cta), hp.cta_begin.data(), (size_t)(n_cta + 1) * 4);
    if (!hp.groups.empty()) memcpy(p->h<MergeGroup>(p->o_groups), hp.groups.data(), hp.groups.size() * sizeof(MergeGroup));
    p->n_req = n_req; p->T = T; p->max_pages = max_pages; p->n_items = n_items; p->n_cta = n_cta;
    p->n_groups = (int)hp.groups.size(); p->n_parts = hp.n_parts;
    p->row_cap = hp.row_cap;
    p->stats = hp.stats;
    p->stats.h2d_bytes = (int64_t)off;
    p->kv = kv; p->kv_pool = kv->pool; p->kv_pages = kv->n_pages;
    return SYN_OK;
}

// The planner without a device: same validation and the same work list as syn_plan_create, returned
// in caller-provided HOST arrays.
static int syn_plan_host_impl(const syn_model_desc* desc, uint32_t n_pages, uint32_t page_size, int32_t n_sm, int32_t n_req,
                             const int32_t* chunk_tokens, const int32_t* chunk_offsets, const int32_t* page_tables,
                             int32_t max_pages, const int32_t* ctx_lens, const int32_t* n_uncached, int32_t* pos,
                             int32_t* slot, int32_t* items, int32_t items_cap, int32_t* n_items, int32_t* cta_begin,
                             int32_t* n_cta, syn_step_stats* stats) {
    if (!desc || page_size != 16 || !n_items || !n_cta) return SYN_E_INVALID_ARG;
    if (desc->n_kv_heads == 0 || desc->n_q_heads % desc->n_kv_heads != 0 || desc->n_q_heads / desc->n_kv_heads > 8)
        return SYN_E_INVALID_ARG;
    HostPlan hp;
    int r = plan_compute(*desc, (int)page_size, n_pages, n_sm, n_req, chunk_tokens, chunk_offsets, page_tables, max_pages,
                         ctx_lens, n_uncached, g_attention, hp);
    if (r) return r;
    *n_items = (int)hp.items.size();
    *n_cta = hp.n_cta;
    if (pos) memcpy(pos, hp.pos.data(), (size_t)hp.T * 4);
    if (slot) memcpy(slot, hp.slot.data(), (size_t)hp.T * 4);
    if (items) {
        if (items_cap < *n_items) return SYN_E_CAPACITY;
        for (int i = 0; i < *n_items; ++i) {
            const AttnItem& it = hp.items[i];
            const int32_t row[SYN_PLAN_ITEM_FIELDS] = {it.q_tok, it.nj, it.kvh, it.req, it.kv_begin, it.kv_end, it.q_pos0,
                                                       it.part, it.grp};
            memcpy(items + (size_t)i * SYN_PLAN_ITEM_FIELDS, row, sizeof(row));
        }
    }
    if (cta_begin) memcpy(cta_begin, hp.cta_begin.data(), (size_t)(hp.n_cta + 1) * 4);
    if (stats) *stats = hp.stats;
    return SYN_OK;
}

static int syn_plan_create_impl(syn_model* m, syn_kv* kv, int32_t n_req, const int32_t* chunk_tokens,
                               const int32_t* chunk_offsets, const int32_t* page_tables, int32_t max_pages,
                               const int32_t* ctx_lens, const int32_t* n_uncached, syn_plan** out) {
    if (!out) return SYN_E_INVALID_ARG;
    syn_plan* p = new (std::nothrow) syn_plan();
    if (!p) return SYN_E_OOM;
    int r = plan_build(p, m, kv, n_req, chunk_tokens, chunk_offsets, page_tables, max_pages, ctx_lens, n_uncached);
    if (r == SYN_OK) {
        cudaError_t e = cudaMemcpy(p->dev, p->host, p->used, cudaMemcpyHostToDevice);
        if (e != cudaSuccess) r = SYN_E_CUDA;
    }
    if (r == SYN_OK) r = ensure_workspace(m, p->T, p->n_req, p->n_parts);
    if (r != SYN_OK) {
        syn_plan_free(p);
        return r;
    }
    *out = p;
    return SYN_OK;
}

extern "C" int syn_plan_stats(const syn_plan* p, syn_step_stats* out) {
    if (!p || !out) return SYN_E_INVALID_ARG;
    *out = p->stats;
    return SYN_OK;
}

extern "C" int syn_last_step_stats(syn_model* m, syn_step_stats* out) {
    if (!m || !out || !m->have_last) return SYN_E_INVALID_ARG;
    *out = m->last_stats;
    if (m->step_timed) {
        float ms = 0.f;
        CU_OK(cudaEventSynchronize(m->step_b));
        CU_OK(cudaEventElapsedTime(&ms, m->step_a, m->step_b));
        out->t_gpu_ms = ms;
        out->t_wall_ms = m->last_wall_ms;
    }
    return SYN_OK;
}

// A plan's page ids and KV slots were checked against one cache: only that cache may run it.
static bool plan_matches(const syn_plan* p, const syn_kv* kv) {
    return p->kv == kv && p->kv_pool == kv->pool && p->kv_pages == kv->n_pages;
}

// ------------------------------------------------------------------------------------------ launches

// The launch shape of one projection D[rows][T] = Wpacked[rows][K] * X[T][K]^T: token tiling, work
// decomposition, CTA count.  Host arithmetic only (also exported as syn_gemm_plan_host so that the
// schedule can be checked without a device).  `mode` = the epilogue the schedule is made for.
static int gemm_plan(int T, int packed_rows, int K, int n_sm, int mode, bool may_ksplit, GemmParams& g, int& n_cta) {
    g.num_kb = (K + 63) / 64;
    g.n_pairs = (packed_rows + 255) / 256;
    g.n_tt = (T + 255) / 256;
    // A projection with fewer pair tiles than SMs can share a tile's K range between CTAs (reduce-
    // scatter, GEMM_RSPLIT): always for the residual projections, whose K is long and whose output is
    // narrow; for qkv from a few hundred tokens on, where single 128-feature tiles would ask L2 for
    // the token tile twice as often; parts of at least 4 (residual) or 8 (qkv) k-blocks.
    const int tiles_nat = g.n_pairs * g.n_tt;
    const bool qkv_split = mode == EPI_QKV && T >= 256 && n_sm / tiles_nat >= 2 && g.num_kb >= 16;
    if (mode != EPI_RESID) {
        // Few feature tiles and few tokens: narrower token tiles (32 tokens at least) put more SMs to
        // work; the weights are then read by several CTAs, which costs only L2 bandwidth.
        const int want = n_sm / std::max(1, 2 * g.n_pairs), most = (T + 31) / 32;
        if (!qkv_split) g.n_tt = std::max(g.n_tt, std::min(want, most));
    } else if (g.n_pairs * g.n_tt < n_sm && n_sm / (g.n_pairs * g.n_tt) < 2) {
        // Residual projection whose pair tiles cover more than half of the SMs but not all: K cannot be
        // split, so narrower token tiles (64 tokens at least) fill the machine instead; every CTA still
        // walks the whole K, on a smaller item.
        const int fit = n_sm / g.n_pairs, most = (T + 63) / 64;
        g.n_tt = std::max(g.n_tt, std::min(fit, most));
    }
    g.TN = (((T + g.n_tt - 1) / g.n_tt) + 15) / 16 * 16;
    g.n_tt = (T + g.TN - 1) / g.TN;   // rounding the width up may leave the last tiles without tokens
    g.n_stages = gemm_stages(g.TN);
    g.ksplit = 1; g.kper = 0; g.n_sm = n_sm;
    g.splits = 1;
    g.kb_per_split = g.num_kb;
    // every token tile must hold a token: an empty one would issue an MMA of width 0
    if (g.n_stages < 2 || g.TN < 16 || g.TN > 256 || (g.n_tt - 1) * g.TN >= T) return SYN_E_INVALID_ARG;
    const int tiles = g.n_pairs * g.n_tt;
    g.pair_mode = tiles >= n_sm;
    if ((mode == EPI_RESID || qkv_split) && tiles < n_sm) {
        const int min_kb = mode == EPI_RESID ? 4 : 8;
        int sp = std::min(GEMM_MAX_SPLITS, std::min(n_sm / tiles, std::max(1, g.num_kb / min_kb)));
        g.kb_per_split = (g.num_kb + sp - 1) / sp;
        g.splits = (g.num_kb + g.kb_per_split - 1) / g.kb_per_split;
        g.pair_mode = 1;
    }
    if (g.splits > 1) n_cta = tiles * g.splits;
    else n_cta = std::min(n_sm, g.pair_mode ? tiles : 2 * tiles);
    // fewer pair tiles than SMs but more single tiles: one wave that mixes whole pair tiles and single tiles
    // (two waves of single tiles would take longer than one pair tile)
    if (g.splits == 1 && !g.pair_mode && 2 * tiles > n_sm) g.pair_mode = 2;
    if (g.splits == 1 && g.pair_mode == 1 && may_ksplit) {
        // The tiles left after the full waves: cut along K over otherwise idle CTAs (parts of at
        // least 8 k-blocks; helpers and owners are different CTAs, so R * parts <= n_cta).
        const int rem = tiles % n_cta;
        if (rem > 0) {
            const int parts = std::min(std::min(8, n_cta / rem), g.num_kb / 8);
            if (parts >= 2) {
                // the owner part also adds the others and finishes the tile: about half a helper's k range
                const int H = parts - 1;
                int kper = (2 * g.num_kb + 2 * H) / (2 * H + 1);
                while (H * kper >= g.num_kb) --kper;
                g.ksplit = parts;
                g.kper = kper;
            }
        }
    }
    return SYN_OK;
}

// One projection with the epilogue `ep`; `plan_mode` = the epilogue its schedule is made for (the
// same, except in the test hook, which runs any schedule with the plain store epilogue).
static int launch_gemm(syn_model* prof_m, int cls, int n_sm, int* status, const op16* w_packed, int packed_rows, int K,
                       const CUtensorMap& tmB, EpiParams ep, cudaStream_t st, float* fix_part, int* fix_flag,
                       int plan_mode = -1) {
    ProfScope prof(cls >= 0 ? prof_m : nullptr, cls, st);
    GemmParams g;
    memset(&g, 0, sizeof(g));
    int n_cta = 0;
    if (plan_mode < 0) plan_mode = ep.mode;
    if (!fix_part || !fix_flag) return SYN_E_INVALID_ARG;
    const int pr = gemm_plan(ep.T, packed_rows, K, n_sm, plan_mode, plan_mode != EPI_RESID, g, n_cta);
    if (pr) return pr;
    g.w = w_packed;
    g.status = status;
    g.fix_part = fix_part; g.fix_flag = fix_flag;
    g.spin_limit = g_spin_limit;
    const int smem = gemm_fixed_smem(g.TN) + g.n_stages * gemm_stage_bytes(g.TN);
    cudaError_t le;
    if (g.splits > 1) le = launch_pdl(gemm_kernel<GEMM_RSPLIT>, dim3(n_cta), dim3(GEMM_THREADS), smem, st, tmB, g, ep);
    else if (g.ksplit > 1) le = launch_pdl(gemm_kernel<GEMM_KSPLIT>, dim3(n_cta), dim3(GEMM_THREADS), smem, st, tmB, g, ep);
    else le = launch_pdl(gemm_kernel<GEMM_WAVES>, dim3(n_cta), dim3(GEMM_THREADS), smem, st, tmB, g, ep);
    return le == cudaSuccess ? SYN_OK : SYN_E_CUDA;
}

// Schedules of the CTA-pair kernel (gemm2.cuh).
enum { PAIR_NONE = 0, PAIR_QUAD = 1, PAIR_DUO = 2 };

// Launch shape of a projection on CTA pairs, or PAIR_NONE when the one-CTA kernel serves it better
// (few tokens: the pair kernel's token tiles are the natural 256-token cut, it has no narrow tiles).
// Host arithmetic only.  `force`: PAIR_QUAD / PAIR_DUO to take that item shape regardless (test hook).
static int gemm2_plan(int T, int packed_rows, int K, int n_sm, int mode, int force, Gemm2Params& g, int& n_cl) {
    memset(&g, 0, sizeof(g));
    const int n_pairs = (packed_rows + 255) / 256, n_cl_max = n_sm / 2;
    g.num_kb = (K + 63) / 64;
    g.n_tt = (T + 255) / 256;
    g.TN = (((T + g.n_tt - 1) / g.n_tt) + 15) / 16 * 16;
    g.n_tt = (T + g.TN - 1) / g.TN;
    g.splits = 1; g.kb_per_split = g.num_kb; g.n_sm = n_sm;
    if (n_cl_max < 1 || (force == PAIR_NONE && T < 256)) return PAIR_NONE;
    const int quad_items = (n_pairs + 1) / 2 * g.n_tt, duo_items = n_pairs * g.n_tt;
    int kind = force;
    const bool may_split = mode == EPI_RESID;
    if (kind == PAIR_NONE) {
        if (quad_items >= n_cl_max) kind = PAIR_QUAD;                                   // full waves of 512-feature items
        else if (4 * quad_items >= 3 * n_cl_max) kind = PAIR_QUAD;                      // one wave, at least three quarters full: measured
                                                                                        // 7-9 % ahead of 256-feature items in two rounds
        else if (!may_split && 8 * quad_items >= 5 * n_cl_max) kind = PAIR_QUAD;        // (without a residual epilogue already from five
                                                                                        // eighths: qkv at 921 tokens 94 us against 102)
        else if (may_split && g.num_kb >= 96 && n_cl_max / quad_items >= 2) kind = PAIR_QUAD;   // long K: shared between clusters
        else if (2 * duo_items >= n_cl_max) kind = PAIR_DUO;
        else return PAIR_NONE;
    }
    const int items = kind == PAIR_QUAD ? quad_items : duo_items;
    g.n_groups = kind == PAIR_QUAD ? (n_pairs + 1) / 2 : n_pairs;
    if (may_split && items < n_cl_max && n_cl_max / items >= 2) {
        const int sp = std::min(GEMM_MAX_SPLITS, std::min(n_cl_max / items, std::max(1, g.num_kb / 8)));
        g.kb_per_split = (g.num_kb + sp - 1) / sp;
        g.splits = (g.num_kb + g.kb_per_split - 1) / g.kb_per_split;
    }
    n_cl = g.splits > 1 ? items * g.splits : std::min(n_cl_max, items);
    // Fewer than three full waves and a last round that fills less than half of the clusters: the one-CTA kernel,
    // whose leftover tiles cost less (helper parts first, short owner parts last), is the faster one there
    // (gate/up at 544 tokens: 168 items on 74 clusters, 2.27 waves: 130 us here against 118 us).
    if (force == PAIR_NONE && g.splits == 1 && items > n_cl && items / n_cl < 3 && items % n_cl != 0 && 2 * (items % n_cl) < n_cl)
        return PAIR_NONE;
    if (g.splits == 1 && items > n_cl) {
        // items left after the full waves: cut along K into one part per cluster (parts of at least 8 k-blocks,
        // at most GEMM_MAX_SPLITS of them), so that the last round takes a fraction of an item's time.  (Helper
        // parts that run first and an owner part that runs last, as in the one-CTA kernel, measured slower here:
        // gate/up 138 against 130 us at 544 tokens, 241 against 201 us at 921: the owner adds up to seven stored
        // parts alone, where the reduce-scatter shares that work between all the tile's clusters.)
        const int rem = items % n_cl;
        if (rem > 0 && n_cl / rem >= 2) {
            int base = n_cl / rem, extra = n_cl % rem;
            const int most = std::min(GEMM_MAX_SPLITS, g.num_kb / 8);
            if (base + (extra > 0 ? 1 : 0) > most) { base = most; extra = 0; }
            if (base >= 2) { g.rem_base = base; g.rem_extra = extra; }
        }
    }
    g.n_stages = gemm2_stages(g.TN, kind == PAIR_DUO);
    if (g.n_stages < 2 || g.TN < 16 || g.TN > 256 || (g.n_tt - 1) * g.TN >= T) return PAIR_NONE;
    return kind;
}

// One projection with the epilogue `ep` on whichever kernel its shape calls for.  `plan_mode` = the
// epilogue the schedule is made for (the same, except in the test hook); `force_pair`: test hook.
static int launch_proj(syn_model* prof_m, int cls, int n_sm, int* status, const op16* w_packed, const WMaps* wm, int packed_rows,
                       int K, const CUtensorMap& tmB, EpiParams ep, cudaStream_t st, float* fix_part, int* fix_flag,
                       int plan_mode = -1, int force_pair = PAIR_NONE) {
    if (plan_mode < 0) plan_mode = ep.mode;
    Gemm2Params g2;
    int n_cl = 0;
    const int kind = (wm && (g_schedule != 1 || force_pair != PAIR_NONE)) ? gemm2_plan(ep.T, packed_rows, K, n_sm, plan_mode, force_pair, g2, n_cl)
                                                                            : PAIR_NONE;
    if (kind == PAIR_NONE) return launch_gemm(prof_m, cls, n_sm, status, w_packed, packed_rows, K, tmB, ep, st, fix_part, fix_flag, plan_mode);
    if (!fix_part || !fix_flag) return SYN_E_INVALID_ARG;
    ProfScope prof(cls >= 0 ? prof_m : nullptr, cls, st);
    g2.status = status; g2.spin_limit = g_spin_limit;
    g2.fix_part = fix_part; g2.fix_flag = fix_flag;
    const bool duo = kind == PAIR_DUO;
    const int smem = gemm_fixed_smem(g2.TN) + g2.n_stages * gemm2_stage_bytes(g2.TN, duo);
    const cudaError_t le = duo ? launch_pdl_pairs(gemm2_kernel<true>, dim3(2 * n_cl), dim3(GEMM_THREADS), smem, st, wm->duo, tmB, g2, ep)
                               : launch_pdl_pairs(gemm2_kernel<false>, dim3(2 * n_cl), dim3(GEMM_THREADS), smem, st, wm->quad, tmB, g2, ep);
    return le == cudaSuccess ? SYN_OK : SYN_E_CUDA;
}

static void attn_params(AttnParams& ap, const syn_model* m, const syn_kv* kv, const syn_plan* p, uint32_t layer, op16* out,
                        float* part_o, float2* part_ml, int* group_count) {
    const syn_model_desc& c = m->desc;
    ap.items = p->d<AttnItem>(p->o_items);
    ap.cta_begin = p->d<int>(p->o_cta);
    ap.page_tables = p->d<int>(p->o_tables);
    ap.max_pages = p->max_pages;
    ap.n_kv_heads = c.n_kv_heads;
    ap.group = c.n_q_heads / c.n_kv_heads;
    ap.q_dim = c.n_q_heads * c.head_dim;
    ap.row_cap = p->row_cap;
    ap.q_box_tokens = p->row_cap == 128 ? std::min(SYN_MAX_CHUNK, 128 / ap.group) : std::min(16, 64 / ap.group);
    ap.layer_block0 = (int)(2ull * layer * kv->n_pages * c.n_kv_heads);
    ap.scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)c.head_dim));
    ap.out = out;
    ap.part_o = part_o;
    ap.part_ml = part_ml;
    ap.groups = p->d<MergeGroup>(p->o_groups);
    ap.group_count = group_count;
    ap.status = m->status_dev;
    ap.n_items = p->n_items; ap.n_req = p->n_req; ap.n_tokens = p->T; ap.n_pages = (int)kv->n_pages;
    ap.n_parts = p->n_parts; ap.n_groups = p->n_groups;
}

static int launch_attention(syn_model* m, syn_kv* kv, const syn_plan* p, uint32_t layer, const CUtensorMap& tmQ,
                            op16* out, cudaStream_t st) {
    const syn_model_desc& c = m->desc;
    AttnParams ap;
    attn_params(ap, m, kv, p, layer, out, m->part_o, m->part_ml, m->group_count);
    {
        ProfScope prof(m, 2, st);
        cudaError_t e;
        if (p->row_cap == 128 && c.head_dim == 128)
            e = launch_pdl(attn2_kernel<128>, dim3(p->n_cta), dim3(ATT2_THREADS), Attn2Smem<128>::TOTAL, st, m->tm_q4, kv->tm_kv5, ap);
        else if (p->row_cap == 128)
            e = launch_pdl(attn2_kernel<64>, dim3(p->n_cta), dim3(ATT2_THREADS), Attn2Smem<64>::TOTAL, st, m->tm_q4, kv->tm_kv5, ap);
        else if (c.head_dim == 128)
            e = launch_pdl(attn_kernel<128>, dim3(p->n_cta), dim3(ATT_THREADS), AttnSmem<128>::TOTAL, st, tmQ, kv->tm_kv, ap);
        else
            e = launch_pdl(attn_kernel<64>, dim3(p->n_cta), dim3(ATT_THREADS), AttnSmem<64>::TOTAL, st, tmQ, kv->tm_kv, ap);
        if (e != cudaSuccess) return SYN_E_CUDA;
    }
    return SYN_OK;
}

static int run_step(syn_model* m, syn_kv* kv, const syn_plan* p, int* acc_dev, int* corr_dev, int* top1_dev,
                    float* logits_out, cudaStream_t st, uint32_t* warp_max = nullptr) {
    const syn_model_desc& c = m->desc;
    const int T = p->T, d = c.d_model, q_dim = c.n_q_heads * c.head_dim, kv_dim = c.n_kv_heads * c.head_dim;
    if (T > m->t_cap || p->n_req > m->b_cap || p->n_parts > m->part_cap) return SYN_E_INVALID_ARG;
    const int* tokens = p->d<int>(p->o_tokens);
    const float inv_d = 1.0f / (float)d;
    m->last_stats = p->stats;
    m->have_last = true;
    m->step_timed = false;
    m->last_wall_ms = 0.0;
    if (m->profile) {
        if (!m->step_a) CU_OK(cudaEventCreate(&m->step_a));
        if (!m->step_b) CU_OK(cudaEventCreate(&m->step_b));
        CU_OK(cudaEventRecord(m->step_a, st));
    }
    {
        ProfScope prof(m, 0, st);
        if (launch_pdl(prep_kernel, dim3(T), dim3(256), 0, st, m->embed, tokens, p->d<int>(p->o_pos), m->norm1[0], m->inv_freq,
                       m->x, m->xn, m->ssq, m->rope, m->best, d, (int)(c.head_dim / 2)) != cudaSuccess)
            return SYN_E_CUDA;
    }
    EpiParams base;
    memset(&base, 0, sizeof(base));
    base.T = T;
    // the consumers of a normalised operand: RMSNorm scale from the partial sums of x^2
    EpiParams scaled = base;
    scaled.ssq_in = m->ssq; scaled.n_ssq = d / 32; scaled.inv_d = inv_d; scaled.eps = c.rms_eps;
    // the writers of the residual stream: x += D, next operand bf16(x * gain), new partial sums
    EpiParams resid = base;
    resid.mode = EPI_RESID; resid.N = d; resid.d = d; resid.x = m->x; resid.xg = m->xn; resid.ssq_out = m->ssq;
    int r;
    for (uint32_t l = 0; l < c.n_layers; ++l) {
        EpiParams e = scaled;
        e.mode = EPI_QKV; e.N = m->qkv_rows;
        e.q = m->q; e.q_dim = q_dim; e.kv_dim = kv_dim; e.hd = c.head_dim; e.n_kv_heads = c.n_kv_heads;
        e.page_size = kv->page_size; e.rope = m->rope; e.pool = kv->pool + kv->layer_elems * l;
        e.slot = p->d<int>(p->o_slot);
        if ((r = launch_proj(m, 1, m->n_sm, m->status_dev, m->wqkv[l], &m->tm_wqkv[l], m->qkv_rows, d, m->tm_xn, e, st, m->fix_part, m->fix_flag)))
            return r;
        if ((r = launch_attention(m, kv, p, l, m->tm_q, m->attn, st))) return r;
        e = resid;
        e.gain = m->norm2[l];
        if ((r = launch_proj(m, 4, m->n_sm, m->status_dev, m->wo[l], &m->tm_wo[l], d, q_dim, m->tm_attn, e, st, m->fix_part, m->fix_flag)))
            return r;
        e = scaled;
        e.mode = EPI_SWIGLU; e.N = m->gu_rows; e.act = m->act; e.f_pad = m->f_pad;
        if ((r = launch_proj(m, 5, m->n_sm, m->status_dev, m->wgu[l], &m->tm_wgu[l], m->gu_rows, d, m->tm_xn, e, st, m->fix_part, m->fix_flag)))
            return r;
        e = resid;
        e.gain = l + 1 < c.n_layers ? m->norm1[l + 1] : m->final_norm;
        if ((r = launch_proj(m, 6, m->n_sm, m->status_dev, m->wd[l], &m->tm_wd[l], d, m->f_pad, m->tm_act, e, st, m->fix_part, m->fix_flag)))
            return r;
    }
    EpiParams e = scaled;
    e.mode = EPI_LMHEAD; e.N = m->v_rows; e.vocab = c.vocab; e.logits = logits_out; e.best = m->best;
    e.warp_max = warp_max; e.n_warp_max = m->v_rows / 32;
    if ((r = launch_proj(m, 7, m->n_sm, m->status_dev, m->lm_head, &m->tm_lm_head, m->v_rows, d, m->tm_xn, e, st, m->fix_part, m->fix_flag)))
        return r;
    {
        ProfScope prof(m, 8, st);
        if (launch_pdl(verify_kernel, dim3((p->n_req + 127) / 128), dim3(128), 0, st, m->best, tokens, p->d<int>(p->o_offsets),
                       p->d<int>(p->o_uncached), p->n_req, acc_dev, corr_dev, top1_dev) != cudaSuccess)
            return SYN_E_CUDA;
    }
    if (m->profile) {
        CU_OK(cudaEventRecord(m->step_b, st));
        m->step_timed = true;
    }
    return SYN_OK;
}

static int syn_verify_run_impl(syn_model* m, syn_kv* kv, const syn_plan* p, int32_t* accept_len_dev, int32_t* correction_dev,
                              int32_t* top1_dev, float* logits_out, void* cuda_stream) {
    if (!m || !kv || !p || kv->model != m || !plan_matches(p, kv) || !accept_len_dev || !correction_dev) return SYN_E_INVALID_ARG;
    return run_step(m, kv, p, accept_len_dev, correction_dev, top1_dev, logits_out, reinterpret_cast<cudaStream_t>(cuda_stream));
}

extern "C" int syn_set_profile(syn_model* m, int on) {
    if (!m) return SYN_E_INVALID_ARG;
    m->profile = on != 0;
    return SYN_OK;
}

static int syn_get_profile_impl(syn_model* m, double* ms, int32_t* launches) {
    if (!m || !ms || !launches) return SYN_E_INVALID_ARG;
    CU_OK(cudaDeviceSynchronize());
    for (int i = 0; i < SYN_N_KERNEL_CLASSES; ++i) { ms[i] = 0.0; launches[i] = 0; }
    for (auto& e : m->ev_used) {
        float t = 0.f;
        if (cudaEventElapsedTime(&t, e.a, e.b) == cudaSuccess && e.cls >= 0 && e.cls < SYN_N_KERNEL_CLASSES) {
            ms[e.cls] += t;
            launches[e.cls] += 1;
        }
        m->ev_free.push_back(e);
    }
    m->ev_used.clear();
    return SYN_OK;
}

extern "C" int syn_model_status(syn_model* m) {
    if (!m) return SYN_E_INVALID_ARG;
    int s = 0;
    if (cudaMemcpy(&s, m->status_dev, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return SYN_E_CUDA;
    if (s) {
        cudaMemset(m->status_dev, 0, 4);
        if (m->group_count) cudaMemset(m->group_count, 0, (size_t)m->part_cap * 4);   // an aborted step may leave counts
        if (m->fix_flag) cudaMemset(m->fix_flag, 0, (size_t)GEMM_FLAG_INTS * m->n_sm * 4);
        return SYN_E_DEVICE_TIMEOUT;
    }
    return SYN_OK;
}

static int syn_verify_batch_impl(syn_model* m, syn_kv* kv, int32_t n_req, const int64_t* req_ids, const int32_t* chunk_tokens,
                                const int32_t* chunk_offsets, const int32_t* page_tables, int32_t max_pages,
                                const int32_t* ctx_lens, const int32_t* n_uncached, int32_t* accept_len,
                                int32_t* correction_token, float* logits_out, void* cuda_stream) {
    (void)req_ids;
    if (!m || !accept_len || !correction_token) return SYN_E_INVALID_ARG;
    if (!m->scratch_plan) {
        m->scratch_plan = new (std::nothrow) syn_plan();
        if (!m->scratch_plan) return SYN_E_OOM;
    }
    syn_plan* p = m->scratch_plan;
    int r = plan_build(p, m, kv, n_req, chunk_tokens, chunk_offsets, page_tables, max_pages, ctx_lens, n_uncached);
    if (r) return r;
    if ((r = ensure_workspace(m, p->T, p->n_req, p->n_parts))) return r;
    if (n_req > m->pinned_out_cap) {
        if (m->pinned_out) cudaFreeHost(m->pinned_out);
        m->pinned_out = nullptr; m->pinned_out_cap = 0;
        const int cap = (n_req + 255) / 256 * 256;
        CU_OK(cudaMallocHost(&m->pinned_out, (size_t)cap * 12));
        m->pinned_out_cap = cap;
    }
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    CU_OK(cudaMemcpyAsync(p->dev, p->host, p->used, cudaMemcpyHostToDevice, st));
    if ((r = run_step(m, kv, p, m->acc_dev, m->corr_dev, nullptr, logits_out, st))) return r;
    int* po = m->pinned_out;
    CU_OK(cudaMemcpyAsync(po, m->acc_dev, (size_t)n_req * 4, cudaMemcpyDeviceToHost, st));
    CU_OK(cudaMemcpyAsync(po + m->pinned_out_cap, m->corr_dev, (size_t)n_req * 4, cudaMemcpyDeviceToHost, st));
    CU_OK(cudaMemcpyAsync(po + 2 * m->pinned_out_cap, m->status_dev, 4, cudaMemcpyDeviceToHost, st));
    CU_OK(cudaStreamSynchronize(st));
    if (po[2 * m->pinned_out_cap]) {
        cudaMemset(m->status_dev, 0, 4);
        if (m->group_count) cudaMemset(m->group_count, 0, (size_t)m->part_cap * 4);
        if (m->fix_flag) cudaMemset(m->fix_flag, 0, (size_t)GEMM_FLAG_INTS * m->n_sm * 4);
        return SYN_E_DEVICE_TIMEOUT;
    }
    memcpy(accept_len, po, (size_t)n_req * 4);
    memcpy(correction_token, po + m->pinned_out_cap, (size_t)n_req * 4);
    return SYN_OK;
}

// ------------------------------------------------------------------------------------------ sampling-based verification

static int check_sampling(const syn_sampling* cfg, int vocab, int T, int n_req, const int32_t* slm_ids, const float* slm_probs,
                          const float* rand_accept, const float* rand_sample) {
    if (!cfg || !slm_ids || !slm_probs || !rand_accept || !rand_sample) return SYN_E_INVALID_ARG;
    if (cfg->top_k < 1 || cfg->top_k > SYN_SAMPLE_MAX_K || cfg->slm_k < 1 || cfg->slm_k > SYN_SAMPLE_MAX_K) return SYN_E_INVALID_ARG;
    if (!(cfg->top_p > 0.f && cfg->top_p <= 1.f) || !(cfg->temperature > 0.f)) return SYN_E_INVALID_ARG;
    for (size_t i = 0; i < (size_t)T * cfg->slm_k; ++i) {
        if (slm_ids[i] < -1 || slm_ids[i] >= vocab) return SYN_E_TOKEN_OOB;
        if (!(slm_probs[i] >= 0.f && slm_probs[i] <= 1.f)) return SYN_E_INVALID_ARG;
    }
    for (int t = 0; t < T; ++t)
        if (!(rand_accept[t] >= 0.f && rand_accept[t] < 1.f)) return SYN_E_INVALID_ARG;
    for (int i = 0; i < n_req; ++i)
        if (!(rand_sample[i] >= 0.f && rand_sample[i] < 1.f)) return SYN_E_INVALID_ARG;
    return SYN_OK;
}

// The two kernels behind the lm_head; every pointer is device memory.
static int sample_stage(syn_model* prof_m, cudaStream_t st, const float* logits, int T, int V, int n_req, const int* tokens,
                        const int* offsets, const int* uncached, const syn_sampling& cfg, int* topk_id, float* topk_logit,
                        const int* slm_id, const float* slm_prob, const float* rand_accept, const float* rand_sample,
                        int* acc_dev, int* corr_dev, const uint32_t* warp_max = nullptr, int n_warp_max = 0) {
    ProfScope prof(prof_m, 8, st);
    if (launch_pdl(topk_rows_kernel, dim3(T), dim3(TOPK_THREADS), 0, st, logits, V, offsets, uncached, n_req, (int)cfg.top_k,
                   warp_max, n_warp_max, topk_id, topk_logit) != cudaSuccess)
        return SYN_E_CUDA;
    SampleParams sp;
    sp.tokens = tokens; sp.offsets = offsets; sp.uncached = uncached;
    sp.topk_id = topk_id; sp.topk_logit = topk_logit;
    sp.slm_id = slm_id; sp.slm_prob = slm_prob; sp.rand_accept = rand_accept; sp.rand_sample = rand_sample;
    sp.accept_len = acc_dev; sp.correction = corr_dev;
    sp.n_req = n_req; sp.top_k = cfg.top_k; sp.slm_k = cfg.slm_k;
    sp.top_p = cfg.top_p; sp.inv_temperature = 1.0f / cfg.temperature;
    if (launch_pdl(sample_verify_kernel, dim3(n_req), dim3(SAMPLE_MAX_K), 0, st, sp) != cudaSuccess) return SYN_E_CUDA;
    return SYN_OK;
}

static int ensure_sample_ws(syn_model* m, int T, int B, int slm_k, bool own_logits) {
    syn_model::SampleWs& w = m->sw;
    const size_t need_logits = own_logits ? (size_t)T * m->desc.vocab : 0;
    if (need_logits > w.logits_cap) {
        cudaFree(w.logits); w.logits = nullptr; w.logits_cap = 0;
        CU_OK(cudaMalloc(&w.logits, need_logits * 4));
        w.logits_cap = need_logits;
    }
    if (T > w.t_cap) {
        cudaFree(w.topk_id); cudaFree(w.topk_logit); cudaFree(w.rand_accept); cudaFree(w.warp_max);
        w.topk_id = nullptr; w.topk_logit = nullptr; w.rand_accept = nullptr; w.warp_max = nullptr; w.t_cap = 0;
        const int cap = (T + 255) / 256 * 256;
        CU_OK(cudaMalloc(&w.warp_max, (size_t)cap * (m->v_rows / 32) * 4));
        CU_OK(cudaMalloc(&w.topk_id, (size_t)cap * SAMPLE_MAX_K * 4));
        CU_OK(cudaMalloc(&w.topk_logit, (size_t)cap * SAMPLE_MAX_K * 4));
        CU_OK(cudaMalloc(&w.rand_accept, (size_t)cap * 4));
        w.t_cap = cap;
        w.slm_cap = 0;
    }
    if (T * slm_k > w.slm_cap) {
        cudaFree(w.slm_id); cudaFree(w.slm_prob);
        w.slm_id = nullptr; w.slm_prob = nullptr; w.slm_cap = 0;
        const int cap = w.t_cap * slm_k;
        CU_OK(cudaMalloc(&w.slm_id, (size_t)cap * 4));
        CU_OK(cudaMalloc(&w.slm_prob, (size_t)cap * 4));
        w.slm_cap = cap;
    }
    if (B > w.b_cap) {
        cudaFree(w.rand_sample); w.rand_sample = nullptr; w.b_cap = 0;
        const int cap = (B + 255) / 256 * 256;
        CU_OK(cudaMalloc(&w.rand_sample, (size_t)cap * 4));
        w.b_cap = cap;
    }
    return SYN_OK;
}

static int syn_verify_batch_sampled_impl(syn_model* m, syn_kv* kv, int32_t n_req, const int64_t* req_ids,
                                        const int32_t* chunk_tokens, const int32_t* chunk_offsets, const int32_t* page_tables,
                                        int32_t max_pages, const int32_t* ctx_lens, const int32_t* n_uncached,
                                        const syn_sampling* cfg, const int32_t* slm_ids, const float* slm_probs,
                                        const float* rand_accept, const float* rand_sample, int32_t* accept_len,
                                        int32_t* correction_token, float* logits_out, void* cuda_stream) {
    (void)req_ids;
    if (!m || !accept_len || !correction_token) return SYN_E_INVALID_ARG;
    if (!m->scratch_plan) {
        m->scratch_plan = new (std::nothrow) syn_plan();
        if (!m->scratch_plan) return SYN_E_OOM;
    }
    syn_plan* p = m->scratch_plan;
    int r = plan_build(p, m, kv, n_req, chunk_tokens, chunk_offsets, page_tables, max_pages, ctx_lens, n_uncached);
    if (r) return r;
    if ((r = check_sampling(cfg, (int)m->desc.vocab, p->T, n_req, slm_ids, slm_probs, rand_accept, rand_sample))) return r;
    if ((r = ensure_workspace(m, p->T, p->n_req, p->n_parts))) return r;
    if ((r = ensure_sample_ws(m, p->T, n_req, cfg->slm_k, logits_out == nullptr))) return r;
    if (n_req > m->pinned_out_cap) {
        if (m->pinned_out) cudaFreeHost(m->pinned_out);
        m->pinned_out = nullptr; m->pinned_out_cap = 0;
        const int cap = (n_req + 255) / 256 * 256;
        CU_OK(cudaMallocHost(&m->pinned_out, (size_t)cap * 12));
        m->pinned_out_cap = cap;
    }
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    syn_model::SampleWs& w = m->sw;
    float* logits = logits_out ? logits_out : w.logits;
    CU_OK(cudaMemcpyAsync(p->dev, p->host, p->used, cudaMemcpyHostToDevice, st));
    CU_OK(cudaMemcpyAsync(w.slm_id, slm_ids, (size_t)p->T * cfg->slm_k * 4, cudaMemcpyHostToDevice, st));
    CU_OK(cudaMemcpyAsync(w.slm_prob, slm_probs, (size_t)p->T * cfg->slm_k * 4, cudaMemcpyHostToDevice, st));
    CU_OK(cudaMemcpyAsync(w.rand_accept, rand_accept, (size_t)p->T * 4, cudaMemcpyHostToDevice, st));
    CU_OK(cudaMemcpyAsync(w.rand_sample, rand_sample, (size_t)n_req * 4, cudaMemcpyHostToDevice, st));
    if ((r = run_step(m, kv, p, m->acc_dev, m->corr_dev, nullptr, logits, st, w.warp_max))) return r;
    // the greedy results of the step are replaced by the sampled ones
    if ((r = sample_stage(m, st, logits, p->T, (int)m->desc.vocab, n_req, p->d<int>(p->o_tokens), p->d<int>(p->o_offsets),
                          p->d<int>(p->o_uncached), *cfg, w.topk_id, w.topk_logit, w.slm_id, w.slm_prob, w.rand_accept,
                          w.rand_sample, m->acc_dev, m->corr_dev, w.warp_max, m->v_rows / 32)))
        return r;
    int* po = m->pinned_out;
    CU_OK(cudaMemcpyAsync(po, m->acc_dev, (size_t)n_req * 4, cudaMemcpyDeviceToHost, st));
    CU_OK(cudaMemcpyAsync(po + m->pinned_out_cap, m->corr_dev, (size_t)n_req * 4, cudaMemcpyDeviceToHost, st));
    CU_OK(cudaMemcpyAsync(po + 2 * m->pinned_out_cap, m->status_dev, 4, cudaMemcpyDeviceToHost, st));
    CU_OK(cudaStreamSynchronize(st));
    if (po[2 * m->pinned_out_cap]) {
        cudaMemset(m->status_dev, 0, 4);
        if (m->group_count) cudaMemset(m->group_count, 0, (size_t)m->part_cap * 4);
        if (m->fix_flag) cudaMemset(m->fix_flag, 0, (size_t)GEMM_FLAG_INTS * m->n_sm * 4);
        return SYN_E_DEVICE_TIMEOUT;
    }
    memcpy(accept_len, po, (size_t)n_req * 4);
    memcpy(correction_token, po + m->pinned_out_cap, (size_t)n_req * 4);
    return SYN_OK;
}

// ------------------------------------------------------------------------------------------ single ops

// The sampling stage alone on logits the caller supplies (device, fp32 [T][vocab]).
static int syn_op_sample_verify_impl(const float* logits, int32_t T, int32_t vocab, int32_t n_req, const int32_t* chunk_tokens,
                                    const int32_t* chunk_offsets, const int32_t* n_uncached, const syn_sampling* cfg,
                                    const int32_t* slm_ids, const float* slm_probs, const float* rand_accept,
                                    const float* rand_sample, int32_t* accept_len, int32_t* correction_token,
                                    void* cuda_stream) {
    if (!logits || T <= 0 || vocab <= 0 || n_req <= 0 || !chunk_tokens || !chunk_offsets || !n_uncached || !accept_len ||
        !correction_token)
        return SYN_E_INVALID_ARG;
    if (chunk_offsets[0] != 0 || chunk_offsets[n_req] != T) return SYN_E_INVALID_ARG;
    for (int i = 0; i < n_req; ++i) {
        const int n = chunk_offsets[i + 1] - chunk_offsets[i];
        if (n < 1 || n > SYN_MAX_CHUNK) return SYN_E_CHUNK_LEN;
        if (n_uncached[i] < 1 || n_uncached[i] > n) return SYN_E_UNCACHED;
    }
    for (int t = 0; t < T; ++t)
        if (chunk_tokens[t] < 0 || chunk_tokens[t] >= vocab) return SYN_E_TOKEN_OOB;
    int r = check_sampling(cfg, vocab, T, n_req, slm_ids, slm_probs, rand_accept, rand_sample);
    if (r) return r;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    const size_t n_slm = (size_t)T * cfg->slm_k;
    // one device block: tokens, offsets, uncached, slm ids | slm probs, draws | top-k lists | results
    const size_t n_i = (size_t)T + (n_req + 1) + n_req + n_slm + (size_t)T * SAMPLE_MAX_K + 2 * (size_t)n_req;
    const size_t n_f = n_slm + T + n_req + (size_t)T * SAMPLE_MAX_K;
    int* di = nullptr;
    float* df = nullptr;
    CU_OK(cudaMalloc(&di, n_i * 4));
    if (note_cuda(cudaMalloc(&df, n_f * 4)) != cudaSuccess) { cudaFree(di); return SYN_E_OOM; }
    int *d_tok = di, *d_off = d_tok + T, *d_unc = d_off + n_req + 1, *d_sid = d_unc + n_req, *d_tid = d_sid + n_slm,
        *d_acc = d_tid + (size_t)T * SAMPLE_MAX_K, *d_cor = d_acc + n_req;
    float *d_sp = df, *d_ra = d_sp + n_slm, *d_rs = d_ra + T, *d_tl = d_rs + n_req;
    std::vector<int> out(2 * (size_t)n_req);
    bool ok = cudaMemcpyAsync(d_tok, chunk_tokens, (size_t)T * 4, cudaMemcpyHostToDevice, st) == cudaSuccess &&
              cudaMemcpyAsync(d_off, chunk_offsets, (size_t)(n_req + 1) * 4, cudaMemcpyHostToDevice, st) == cudaSuccess &&
              cudaMemcpyAsync(d_unc, n_uncached, (size_t)n_req * 4, cudaMemcpyHostToDevice, st) == cudaSuccess &&
              cudaMemcpyAsync(d_sid, slm_ids, n_slm * 4, cudaMemcpyHostToDevice, st) == cudaSuccess &&
              cudaMemcpyAsync(d_sp, slm_probs, n_slm * 4, cudaMemcpyHostToDevice, st) == cudaSuccess &&
              cudaMemcpyAsync(d_ra, rand_accept, (size_t)T * 4, cudaMemcpyHostToDevice, st) == cudaSuccess &&
              cudaMemcpyAsync(d_rs, rand_sample, (size_t)n_req * 4, cudaMemcpyHostToDevice, st) == cudaSuccess;
    r = ok ? sample_stage(nullptr, st, logits, T, vocab, n_req, d_tok, d_off, d_unc, *cfg, d_tid, d_tl, d_sid, d_sp, d_ra, d_rs,
                          d_acc, d_cor)
           : SYN_E_CUDA;
    if (r == SYN_OK && (note_cuda(cudaMemcpyAsync(out.data(), d_acc, 2 * (size_t)n_req * 4, cudaMemcpyDeviceToHost, st)) != cudaSuccess ||
                        note_cuda(cudaStreamSynchronize(st)) != cudaSuccess))
        r = SYN_E_CUDA;
    cudaFree(di);
    cudaFree(df);
    if (r) return r;
    memcpy(accept_len, out.data(), (size_t)n_req * 4);
    memcpy(correction_token, out.data() + n_req, (size_t)n_req * 4);
    return SYN_OK;
}

// Process-wide context of the single-projection test hook: status word, exchange workspace, and the
// packed copy of the last weight matrix seen.
struct LinearCtx {
    int n_sm = 0;
    int* status = nullptr;
    float* fix_part = nullptr;
    int* fix_flag = nullptr;
    op16* packed = nullptr;
    const void* packed_src = nullptr;
    int packed_n = 0, packed_k = 0;
    WMaps wm;
};
static LinearCtx g_lin;

static int linear_ctx_init() {
    if (g_lin.status) return SYN_OK;
    int dev = 0;
    cudaDeviceProp prop;
    CU_OK(cudaGetDevice(&dev));
    CU_OK(cudaGetDeviceProperties(&prop, dev));
    if (prop.major != 10) return SYN_E_ARCH;
    g_lin.n_sm = prop.multiProcessorCount;
    CU_OK(cudaFuncSetAttribute(gemm_kernel<GEMM_WAVES>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM_MAX));
    CU_OK(cudaFuncSetAttribute(gemm_kernel<GEMM_KSPLIT>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM_MAX));
    CU_OK(cudaFuncSetAttribute(gemm_kernel<GEMM_RSPLIT>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM_MAX));
    CU_OK(cudaFuncSetAttribute(gemm2_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM_MAX));
    CU_OK(cudaFuncSetAttribute(gemm2_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM_MAX));
    CU_OK(cudaMalloc(&g_lin.fix_part, (size_t)g_lin.n_sm * GEMM_FIX_SLOT_BYTES));
    CU_OK(cudaMalloc(&g_lin.fix_flag, (size_t)GEMM_FLAG_INTS * g_lin.n_sm * 4));
    CU_OK(cudaMemset(g_lin.fix_flag, 0, (size_t)GEMM_FLAG_INTS * g_lin.n_sm * 4));
    CU_OK(cudaMalloc(&g_lin.status, 4));
    CU_OK(cudaMemset(g_lin.status, 0, 4));
    return SYN_OK;
}

extern "C" int syn_op_linear_reset(void) {
    if (g_lin.packed) {
        CU_OK(cudaDeviceSynchronize());
        cudaFree(g_lin.packed);
    }
    g_lin.packed = nullptr; g_lin.packed_src = nullptr; g_lin.packed_n = g_lin.packed_k = 0;
    return SYN_OK;
}

extern "C" int syn_op_linear_as(const void* x, const void* w, float* y, int32_t T, int32_t N, int32_t K, int32_t schedule_as,
                                void* cuda_stream) {
    if (!x || !w || !y || T <= 0 || N <= 0 || K <= 0 || K % 8 != 0 || schedule_as < EPI_PLAIN || schedule_as > EPI_LMHEAD + 4)
        return SYN_E_INVALID_ARG;
    int r = load_driver_entry();
    if (r) return r;
    if ((r = linear_ctx_init())) return r;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    const int n_mt = (N + 511) / 512 * 4, nkb = (K + 63) / 64;
    if (g_lin.packed_src != w || g_lin.packed_n != N || g_lin.packed_k != K) {
        if ((r = syn_op_linear_reset())) return r;
        CU_OK(cudaMalloc(&g_lin.packed, (size_t)n_mt * nkb * 128 * 64 * 2));
        PackSrc ps;
        memset(&ps, 0, sizeof(ps));
        ps.p[0] = (const bf16*)w; ps.rows[0] = N; ps.src_k = K;
        pack_weight_kernel<<<dim3(n_mt, nkb), 256, 0, st>>>(ps, g_lin.packed, nkb);
        if (!launch_ok()) return SYN_E_CUDA;
        CU_OK(cudaStreamSynchronize(st));   // the GEMM requests weight tiles before it waits for its predecessor
        g_lin.packed_src = w; g_lin.packed_n = N; g_lin.packed_k = K;
        if ((r = make_wmaps(g_lin.packed, n_mt * 128, K, &g_lin.wm))) return r;
    }
    CUtensorMap tmB;
    if ((r = make_map_2d(&tmB, x, T, K, K, GEMM_BOX_ROWS))) return r;
    EpiParams e;
    memset(&e, 0, sizeof(e));
    e.mode = EPI_PLAIN; e.T = T; e.N = N; e.y = y; e.ldy = N;
    // 0..4: the schedule the step would take for that epilogue; 5, 6: CTA pairs with QUAD / DUO items; 7, 8: the
    // same as residual projections (K shared between clusters where the shape allows it)
    const int force = schedule_as <= EPI_LMHEAD ? PAIR_NONE : (schedule_as == 5 || schedule_as == 7 ? PAIR_QUAD : PAIR_DUO);
    const int plan_mode = schedule_as <= EPI_LMHEAD ? schedule_as : (schedule_as >= 7 ? EPI_RESID : EPI_PLAIN);
    r = launch_proj(nullptr, -1, g_lin.n_sm, g_lin.status, g_lin.packed, &g_lin.wm, (N + 127) / 128 * 128, K, tmB, e, st, g_lin.fix_part,
                    g_lin.fix_flag, plan_mode, force);
    if (r) return r;
    CU_OK(cudaStreamSynchronize(st));
    int sflag = 0;
    CU_OK(cudaMemcpy(&sflag, g_lin.status, 4, cudaMemcpyDeviceToHost));
    if (sflag) {
        cudaMemset(g_lin.status, 0, 4);
        cudaMemset(g_lin.fix_flag, 0, (size_t)GEMM_FLAG_INTS * g_lin.n_sm * 4);
        return SYN_E_DEVICE_TIMEOUT;
    }
    return SYN_OK;
}

extern "C" int syn_op_linear(const void* x, const void* w, float* y, int32_t T, int32_t N, int32_t K, void* cuda_stream) {
    return syn_op_linear_as(x, w, y, T, N, K, EPI_PLAIN, cuda_stream);
}

extern "C" int syn_debug_set_spin_limit(int64_t cycles) {
    if (cycles < 0) return SYN_E_INVALID_ARG;
    g_spin_limit = cycles == 0 ? SYN_SPIN_LIMIT_CYCLES : (long long)cycles;
    return SYN_OK;
}

extern "C" int syn_debug_set_schedule(int32_t which) {
    if (which < 0 || which > 1) return SYN_E_INVALID_ARG;
    g_schedule = which;
    return SYN_OK;
}

extern "C" int syn_debug_set_attention(int32_t which) {
    if (which < 0 || which > 2) return SYN_E_INVALID_ARG;
    g_attention = which;
    return SYN_OK;
}

extern "C" int syn_debug_linear_counter(int32_t index, int32_t value) {
    int r = linear_ctx_init();
    if (r) return r;
    if (index < 0 || index >= GEMM_FLAG_INTS * g_lin.n_sm) return SYN_E_INVALID_ARG;
    CU_OK(cudaDeviceSynchronize());
    CU_OK(cudaMemcpy(g_lin.fix_flag + index, &value, 4, cudaMemcpyHostToDevice));
    return SYN_OK;
}

static int syn_op_attention_impl(syn_model* m, syn_kv* kv, const syn_plan* p, uint32_t layer, const void* q, void* out,
                                void* cuda_stream) {
    if (!m || !kv || !p || kv->model != m || !plan_matches(p, kv) || !q || !out || layer >= m->desc.n_layers)
        return SYN_E_INVALID_ARG;
    const syn_model_desc& c = m->desc;
    const int q_dim = c.n_q_heads * c.head_dim;
    if (p->T > m->t_cap || p->n_parts > m->part_cap) return SYN_E_INVALID_ARG;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    // the Q tensor map is bound to the workspace buffer: stage the caller's q there
    CU_OK(cudaMemcpyAsync(m->q, q, (size_t)p->T * q_dim * 2, cudaMemcpyDeviceToDevice, st));
    return launch_attention(m, kv, p, layer, m->tm_q, (op16*)out, st);
}

// ------------------------------------------------------------------------------------------ no-allocation attention

// Scratch of syn_op_attention_static: the fp32 partial outputs and (max, sum) pairs of attention
// work items that cover only part of a request's keys, and the per-group completion counters.  File-scope device memory, so every GPU that
// loads the library holds these ~8.5 MB from load to exit.  Host code may not pass these names to a
// kernel (on the host they are stand-ins, not device addresses): static_scratch() asks the runtime
// for the device addresses once per device.
static __device__ __align__(256) float g_static_part_o[(size_t)SYN_STATIC_MAX_PARTS * 64 * 128];
static __device__ __align__(256) float2 g_static_part_ml[(size_t)SYN_STATIC_MAX_PARTS * 64];
static __device__ __align__(256) int g_static_group_count[SYN_STATIC_MAX_PARTS];

static int static_scratch(float** part_o, float2** part_ml, int** group_count) {
    constexpr int MAX_DEV = 64;
    static float* o_of[MAX_DEV];
    static float2* ml_of[MAX_DEV];
    static int* cnt_of[MAX_DEV];
    static std::mutex lock;   // two host threads may make the first call on a device together
    int dev = -1;
    CU_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= MAX_DEV) return SYN_E_INVALID_ARG;
    std::lock_guard<std::mutex> hold(lock);
    if (!o_of[dev]) {   // first call on this device (which is current): resolve the symbols
        void *a = nullptr, *b = nullptr, *cn = nullptr;
        CU_OK(cudaGetSymbolAddress(&a, g_static_part_o));
        CU_OK(cudaGetSymbolAddress(&b, g_static_part_ml));
        CU_OK(cudaGetSymbolAddress(&cn, g_static_group_count));
        if (!a || !b || !cn) return SYN_E_CUDA;
        ml_of[dev] = static_cast<float2*>(b);
        cnt_of[dev] = static_cast<int*>(cn);
        o_of[dev] = static_cast<float*>(a);
    }
    *part_o = o_of[dev];
    *part_ml = ml_of[dev];
    *group_count = cnt_of[dev];
    return SYN_OK;
}

static int syn_op_attention_static_impl(syn_model* m, syn_kv* kv, const syn_plan* p, uint32_t layer, const void* q,
                                       void* out, void* cuda_stream) {
    if (!m || !kv || !p || kv->model != m || !plan_matches(p, kv) || !q || !out || layer >= m->desc.n_layers)
        return SYN_E_INVALID_ARG;
    const syn_model_desc& c = m->desc;
    const int q_dim = c.n_q_heads * c.head_dim;
    if (p->T > m->t_cap) return SYN_E_INVALID_ARG;
    if ((int64_t)p->n_parts * p->row_cap > (int64_t)SYN_STATIC_MAX_PARTS * 64) return SYN_E_CAPACITY;
    float* part_o = nullptr;
    float2* part_ml = nullptr;
    int* group_count = nullptr;
    int r = static_scratch(&part_o, &part_ml, &group_count);
    if (r) return r;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    CU_OK(cudaMemcpyAsync(m->q, q, (size_t)p->T * q_dim * 2, cudaMemcpyDeviceToDevice, st));
    // the group counters must start at zero; every partial row that is read is written first
    CU_OK(cudaMemsetAsync(group_count, 0, (size_t)SYN_STATIC_MAX_PARTS * 4, st));
    AttnParams ap;
    attn_params(ap, m, kv, p, layer, (op16*)out, part_o, part_ml, group_count);
    if (p->row_cap == 128 && c.head_dim == 128)
        attn2_kernel<128><<<p->n_cta, ATT2_THREADS, Attn2Smem<128>::TOTAL, st>>>(m->tm_q4, kv->tm_kv5, ap);
    else if (p->row_cap == 128)
        attn2_kernel<64><<<p->n_cta, ATT2_THREADS, Attn2Smem<64>::TOTAL, st>>>(m->tm_q4, kv->tm_kv5, ap);
    else if (c.head_dim == 128)
        attn_kernel<128><<<p->n_cta, ATT_THREADS, AttnSmem<128>::TOTAL, st>>>(m->tm_q, kv->tm_kv, ap);
    else
        attn_kernel<64><<<p->n_cta, ATT_THREADS, AttnSmem<64>::TOTAL, st>>>(m->tm_q, kv->tm_kv, ap);
    return launch_ok() ? SYN_OK : SYN_E_CUDA;
}

// The projection schedule without a device (tests): the launch shape, and work item i of CTA `cta`.
extern "C" int syn_gemm_plan_host(int32_t T, int32_t N, int32_t K, int32_t n_sm, int32_t epilogue, int32_t* out) {
    if (T <= 0 || N <= 0 || K <= 0 || n_sm <= 0 || n_sm > 65535 || epilogue < EPI_PLAIN || epilogue > EPI_LMHEAD || !out)
        return SYN_E_INVALID_ARG;
    GemmParams g;
    memset(&g, 0, sizeof(g));
    int n_cta = 0;
    const int r = gemm_plan(T, (N + 255) / 256 * 256, K, n_sm, epilogue, epilogue != EPI_RESID, g, n_cta);
    if (r) return r;
    const int v[SYN_GEMM_PLAN_FIELDS] = {g.n_pairs, g.n_tt, g.TN, g.num_kb, n_cta, g.pair_mode, g.splits, g.kb_per_split, g.ksplit, g.kper};
    memcpy(out, v, sizeof(v));
    return SYN_OK;
}

extern "C" int syn_gemm_work_host(int32_t T, int32_t N, int32_t K, int32_t n_sm, int32_t epilogue, int32_t cta, int32_t i,
                                  int32_t* out) {
    if (T <= 0 || N <= 0 || K <= 0 || n_sm <= 0 || n_sm > 65535 || epilogue < EPI_PLAIN || epilogue > EPI_LMHEAD || !out || i < 0)
        return SYN_E_INVALID_ARG;
    GemmParams g;
    memset(&g, 0, sizeof(g));
    int n_cta = 0;
    const int r = gemm_plan(T, (N + 255) / 256 * 256, K, n_sm, epilogue, epilogue != EPI_RESID, g, n_cta);
    if (r) return r;
    if (cta < 0 || cta >= n_cta) return SYN_E_INVALID_ARG;
    GemmWork w;
    const bool have = g.ksplit > 1 ? gemm_work<true>(g, cta, n_cta, i, w) : gemm_work<false>(g, cta, n_cta, i, w);
    if (!have) return 0;
    const int v[SYN_GEMM_WORK_FIELDS] = {w.pair, w.tt, w.mt_lo, w.mt_hi, w.kb0, w.kb1, w.split, w.role, w.rtile, w.hpart};
    memcpy(out, v, sizeof(v));
    return 1;
}


// ------------------------------------------------------------------------------------------ exported wrappers
// No C++ exception crosses the C ABI: the host code behind these entry points uses std::vector.
#define SYN_GUARD(call)                  \
    try {                                \
        return (call);                   \
    } catch (const std::bad_alloc&) {    \
        return SYN_E_OOM;                \
    } catch (...) {                      \
        return SYN_E_INVALID_ARG;        \
    }

extern "C" int syn_model_load(const syn_model_desc* desc, const syn_weights* w, syn_model** out) {
    SYN_GUARD(syn_model_load_impl(desc, w, out));
}

extern "C" int syn_kv_import(syn_kv* kv, uint32_t layer, const int32_t* page_table, int32_t pos0, int32_t n_pos, const void* k, const void* v, void* stream) {
    SYN_GUARD(syn_kv_import_impl(kv, layer, page_table, pos0, n_pos, k, v, stream));
}

extern "C" int syn_kv_export(syn_kv* kv, uint32_t layer, const int32_t* page_table, int32_t pos0, int32_t n_pos, void* k, void* v, void* stream) {
    SYN_GUARD(syn_kv_export_impl(kv, layer, page_table, pos0, n_pos, k, v, stream));
}

extern "C" int syn_plan_host(const syn_model_desc* desc, uint32_t n_pages, uint32_t page_size, int32_t n_sm, int32_t n_req, const int32_t* chunk_tokens, const int32_t* chunk_offsets, const int32_t* page_tables, int32_t max_pages, const int32_t* ctx_lens, const int32_t* n_uncached, int32_t* pos, int32_t* slot, int32_t* items, int32_t items_cap, int32_t* n_items, int32_t* cta_begin, int32_t* n_cta, syn_step_stats* stats) {
    SYN_GUARD(syn_plan_host_impl(desc, n_pages, page_size, n_sm, n_req, chunk_tokens, chunk_offsets, page_tables, max_pages, ctx_lens, n_uncached, pos, slot, items, items_cap, n_items, cta_begin, n_cta, stats));
}

extern "C" int syn_plan_create(syn_model* m, syn_kv* kv, int32_t n_req, const int32_t* chunk_tokens, const int32_t* chunk_offsets, const int32_t* page_tables, int32_t max_pages, const int32_t* ctx_lens, const int32_t* n_uncached, syn_plan** out) {
    SYN_GUARD(syn_plan_create_impl(m, kv, n_req, chunk_tokens, chunk_offsets, page_tables, max_pages, ctx_lens, n_uncached, out));
}

extern "C" int syn_verify_run(syn_model* m, syn_kv* kv, const syn_plan* p, int32_t* accept_len_dev, int32_t* correction_dev, int32_t* top1_dev, float* logits_out, void* cuda_stream) {
    SYN_GUARD(syn_verify_run_impl(m, kv, p, accept_len_dev, correction_dev, top1_dev, logits_out, cuda_stream));
}

extern "C" int syn_get_profile(syn_model* m, double* ms, int32_t* launches) {
    SYN_GUARD(syn_get_profile_impl(m, ms, launches));
}

extern "C" int syn_verify_batch(syn_model* m, syn_kv* kv, int32_t n_req, const int64_t* req_ids, const int32_t* chunk_tokens, const int32_t* chunk_offsets, const int32_t* page_tables, int32_t max_pages, const int32_t* ctx_lens, const int32_t* n_uncached, int32_t* accept_len, int32_t* correction_token, float* logits_out, void* cuda_stream) {
    const auto t0 = std::chrono::steady_clock::now();
    int r;
    try {
        r = syn_verify_batch_impl(m, kv, n_req, req_ids, chunk_tokens, chunk_offsets, page_tables, max_pages, ctx_lens, n_uncached, accept_len, correction_token, logits_out, cuda_stream);
    } catch (const std::bad_alloc&) {
        return SYN_E_OOM;
    } catch (...) {
        return SYN_E_INVALID_ARG;
    }
    if (m && m->profile) m->last_wall_ms = std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now() - t0).count();
    return r;
}

extern "C" int syn_verify_batch_sampled(syn_model* m, syn_kv* kv, int32_t n_req, const int64_t* req_ids, const int32_t* chunk_tokens, const int32_t* chunk_offsets, const int32_t* page_tables, int32_t max_pages, const int32_t* ctx_lens, const int32_t* n_uncached, const syn_sampling* cfg, const int32_t* slm_ids, const float* slm_probs, const float* rand_accept, const float* rand_sample, int32_t* accept_len, int32_t* correction_token, float* logits_out, void* cuda_stream) {
    const auto t0 = std::chrono::steady_clock::now();
    int r;
    try {
        r = syn_verify_batch_sampled_impl(m, kv, n_req, req_ids, chunk_tokens, chunk_offsets, page_tables, max_pages, ctx_lens, n_uncached, cfg, slm_ids, slm_probs, rand_accept, rand_sample, accept_len, correction_token, logits_out, cuda_stream);
    } catch (const std::bad_alloc&) {
        return SYN_E_OOM;
    } catch (...) {
        return SYN_E_INVALID_ARG;
    }
    if (m && m->profile) m->last_wall_ms = std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now() - t0).count();
    return r;
}

extern "C" int syn_op_sample_verify(const float* logits, int32_t T, int32_t vocab, int32_t n_req, const int32_t* chunk_tokens, const int32_t* chunk_offsets, const int32_t* n_uncached, const syn_sampling* cfg, const int32_t* slm_ids, const float* slm_probs, const float* rand_accept, const float* rand_sample, int32_t* accept_len, int32_t* correction_token, void* cuda_stream) {
    SYN_GUARD(syn_op_sample_verify_impl(logits, T, vocab, n_req, chunk_tokens, chunk_offsets, n_uncached, cfg, slm_ids, slm_probs, rand_accept, rand_sample, accept_len, correction_token, cuda_stream));
}

extern "C" int syn_op_attention(syn_model* m, syn_kv* kv, const syn_plan* p, uint32_t layer, const void* q, void* out, void* cuda_stream) {
    SYN_GUARD(syn_op_attention_impl(m, kv, p, layer, q, out, cuda_stream));
}

extern "C" int syn_op_attention_static(syn_model* m, syn_kv* kv, const syn_plan* p, uint32_t layer, const void* q, void* out, void* cuda_stream) {
    SYN_GUARD(syn_op_attention_static_impl(m, kv, p, layer, q, out, cuda_stream));
}

// The CTA-pair schedule without a device (tests).
extern "C" int syn_gemm2_plan_host(int32_t T, int32_t N, int32_t K, int32_t n_sm, int32_t epilogue, int32_t force, int32_t* out) {
    if (T <= 0 || N <= 0 || K <= 0 || n_sm <= 0 || n_sm > 65535 || epilogue < EPI_PLAIN || epilogue > EPI_LMHEAD || force < PAIR_NONE ||
        force > PAIR_DUO || !out)
        return SYN_E_INVALID_ARG;
    Gemm2Params g;
    int n_cl = 0;
    const int kind = gemm2_plan(T, (N + 255) / 256 * 256, K, n_sm, epilogue, force, g, n_cl);
    const int v[SYN_GEMM2_PLAN_FIELDS] = {kind, g.n_groups, g.n_tt, g.TN, g.num_kb, n_cl, g.splits, g.kb_per_split, g.rem_base, g.rem_extra};
    memcpy(out, v, sizeof(v));
    return SYN_OK;
}

extern "C" int syn_gemm2_work_host(int32_t T, int32_t N, int32_t K, int32_t n_sm, int32_t epilogue, int32_t force, int32_t cluster,
                                   int32_t i, int32_t* out) {
    if (T <= 0 || N <= 0 || K <= 0 || n_sm <= 0 || n_sm > 65535 || epilogue < EPI_PLAIN || epilogue > EPI_LMHEAD || force < PAIR_NONE ||
        force > PAIR_DUO || !out || i < 0)
        return SYN_E_INVALID_ARG;
    Gemm2Params g;
    int n_cl = 0;
    const int kind = gemm2_plan(T, (N + 255) / 256 * 256, K, n_sm, epilogue, force, g, n_cl);
    if (kind == PAIR_NONE || cluster < 0 || cluster >= n_cl) return SYN_E_INVALID_ARG;
    Gemm2Work w;
    if (!gemm2_work(g, cluster, n_cl, i, w)) return 0;
    const int v[SYN_GEMM2_WORK_FIELDS] = {w.grp, w.tt, w.kb0, w.kb1, w.tile, w.split, w.nsplit, w.first_cl, w.counter};
    memcpy(out, v, sizeof(v));
    return 1;
}

extern "C" const char* syn_last_cuda_error(void) { return g_last_cuda_error; }

extern "C" const char* syn_strerror(int code) {
    switch (code) {
        case SYN_OK: return "ok";
        case SYN_E_INVALID_ARG: return "invalid argument";
        case SYN_E_CHUNK_LEN: return "chunk length outside [1, 32]";
        case -20: return "scheduler: no live request with this id";
        case -21: return "scheduler: a live request with this id exists already";
        case -22: return "scheduler: the request cannot take this call in its present state";
        case -23: return "scheduler: commit without a peeked batch";
        case SYN_E_UNCACHED: return "n_uncached outside [1, chunk length]";
        case SYN_E_PAGE_OOB: return "page id out of range";
        case SYN_E_CAPACITY: return "context + chunk exceeds the page table";
        case SYN_E_TOKEN_OOB: return "token id out of range";
        case SYN_E_PAGE_ALIAS: return "two chunk tokens map to the same KV slot";
        case SYN_E_OOM: return "out of memory";
        case SYN_E_ARCH: return "device is not sm_100";
        case SYN_E_CUDA: return "CUDA call failed";
        case SYN_E_DEVICE_TIMEOUT: return "bounded device-side wait ran out";
        default: return "unknown error";
    }
}
