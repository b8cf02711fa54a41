// Ragged multi-query attention over the paged KV cache (paper Sec. 3.2 attention equation,
// applied to a chunk of 1..16 query tokens per request appended to a cached prefix, Sec. 3.4).
//
// One work item = (request, kv head, token sub-range of the chunk, key range).  The G query heads
// that share the kv head and the chunk's tokens are packed into one tile of rows (row = j*G + g,
// at most 64), so every K/V byte of the item is read from HBM once.  A persistent CTA walks a
// host-planned list of items.  One producer warp streams pages (TMA, 128-byte swizzle, one box of
// 32 rows x 128 bytes per page and 64-element half: K and V of 16 tokens) and the item's Q tile
// through mbarrier rings; its lanes hold the page-table entries of eight stages and fetch the next
// eight stages' entries meanwhile (its warpgroup gives most of its registers to the consumers).
// Eight consumer warps form two groups that take alternate stages, so
// every scheduler of the SM holds two warps; inside a group the four warps split the item's row
// tiles and, when there are fewer than four row tiles, the pages of the stage.  QK^T and PV run on
// warp-level MMAs (m16n8k16, half-precision operands, fp32 accumulate) with an online softmax in fp32 (base 2).
// The (max, sum, O) triples of the warps that share a row tile are merged in shared memory in a
// fixed order.  An item that covers only part of a request's keys writes an fp32 partial; the CTA
// that completes the last partial of a row group (a counter per group, reset by that CTA) combines
// them in part order, so the result does not depend on which CTA arrives last.
#pragma once
#include "ptx.cuh"

namespace syn {

struct AttnItem {
    int q_tok;      // index of the first query token of this item in the flattened batch
    int nj;         // query tokens in this item (rows = nj * G <= AttnParams::row_cap)
    int kvh;        // kv head
    int req;        // request (page table row)
    int kv_begin;   // first key position (multiple of 64)
    int kv_end;     // one past the last key position this item reads
    int q_pos0;     // position of the item's first query token (ctx + j0): row j sees keys <= q_pos0 + j
    int part;       // -1: sole item of its rows -> writes the output; else index of its partial
    int grp;        // merge group of a partial item (index into AttnParams::groups), else -1
    int pad0, pad1, pad2;
};

// Row group whose keys were split over several items.
struct MergeGroup {
    int q_tok, nj, kvh, part0, n_parts, pad0, pad1, pad2;
};

struct AttnParams {
    const AttnItem* items;      // sorted by CTA
    const int* cta_begin;       // [n_cta + 1]
    const int* page_tables;     // [B][max_pages]
    int max_pages;
    int n_kv_heads, group;      // G = Hq / Hkv
    int q_dim;                  // Hq * hd
    int q_box_tokens;           // tokens of the Q tile's TMA box: min(16, 64 / G) (tensor-memory kernel: min(32, 128 / G))
    int row_cap;                // rows of an item's tile: 64 (128 in the tensor-memory kernel); row stride of the partials
    int layer_block0;           // 2 * layer * n_pages * Hkv: first (K|V) block of this layer in the pool map
    float scale_log2;           // log2(e) / sqrt(hd)
    op16* out;                  // [T][q_dim]
    float* part_o;              // [n_parts][row_cap][hd]
    float2* part_ml;            // [n_parts][row_cap] (max in log2 units, sum)
    const MergeGroup* groups;   // [n_groups]
    int* group_count;           // [n_groups] partials completed so far; zero between launches
    int* status;                // 0 ok, 1 a bounded wait ran out, 2 the work list failed a bounds check
    // extents for the kernel's own bounds checks of the work list
    int n_items, n_req, n_tokens, n_pages, n_parts, n_groups;
};

// The work list is host-made; the kernel still refuses an item that would index out of bounds.
__device__ __forceinline__ bool attn_item_ok(const AttnItem& it, const AttnParams& p) {
    const bool ok = it.q_tok >= 0 && it.nj >= 1 && it.q_tok + it.nj <= p.n_tokens && it.nj * p.group <= p.row_cap &&
                    it.kvh >= 0 && it.kvh < p.n_kv_heads && it.req >= 0 && it.req < p.n_req && it.kv_begin >= 0 &&
                    (it.kv_begin & 63) == 0 && it.kv_begin < it.kv_end && ((it.kv_end - 1) >> 4) < p.max_pages &&
                    (it.part < 0 || (it.part < p.n_parts && it.grp >= 0 && it.grp < p.n_groups));
    return ok;
}

constexpr int ATT_STAGE_PAGES = 4;
constexpr int ATT_CONSUMER_WARPS = 8;
constexpr int ATT_THREADS = (ATT_CONSUMER_WARPS + 4) * 32;   // two consumer warpgroups + the producer's warpgroup
constexpr int ATT_PRODUCER_REGS = 40, ATT_CONSUMER_REGS = 232;   // 2 x 232 + 40 per scheduler slot <= 512
constexpr int ATT_LAUNCH_REGS = 168;                              // what ptxas grants 384 threads per CTA
static_assert(ATT_CONSUMER_WARPS * ATT_CONSUMER_REGS + 4 * ATT_PRODUCER_REGS <= (ATT_CONSUMER_WARPS + 4) * ATT_LAUNCH_REGS,
              "the consumers' increase must fit in what the producer's warpgroup gives back");

template <int HD>
struct AttnSmem {
    static constexpr int PAGE_BYTES = 2 * 16 * HD * 2;            // K and V of one page, one head
    static constexpr int STAGE_BYTES = ATT_STAGE_PAGES * PAGE_BYTES;
    // An odd number of stages: the two consumer groups take alternate stages, so the uses of one
    // slot alternate between the groups.  A parity wait must never run two phases ahead of its
    // barrier, and loads land out of order, so each group waits on a "full" barrier of its own per
    // slot, which it observes phase by phase.
    static constexpr int STAGES = HD == 128 ? 5 : 11;
    static_assert(STAGES % 2 == 1, "slot uses must alternate between the two consumer groups");
    static constexpr int Q_BYTES = 64 * HD * 2;                    // at most 64 rows
    static constexpr int MERGE_BYTES = 4 * 16 * (HD + 4) * 4;      // four slots: O[16][HD] + (m, l)[16]
    static constexpr int TOTAL = 1024 + STAGES * STAGE_BYTES + 2 * Q_BYTES + MERGE_BYTES + 512;
};

// byte offset of the 16-byte chunk `c16` of 128-byte line `line` under the 128-byte swizzle
__device__ __forceinline__ uint32_t swz(uint32_t line, uint32_t c16) { return line * 128u + ((c16 ^ (line & 7u)) << 4); }

__device__ __forceinline__ float ex2_approx(float x) {   // 2^x; -inf -> +0
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// One warp's share of one stage: NPG pages starting at `first_page`, one 16-row tile of queries.
// m is kept in log2 units (raw score * scale_log2).  FULL: all NPG pages hold keys of the item.
template <int HD, int NPG, bool FULL>
__device__ __forceinline__ void attn_consume_stage(const uint8_t* stage, int first_page, int n_valid_pages,
                                                   int stage_kv0, const uint32_t (&qf)[HD / 16][4], float (&o)[HD / 8][4],
                                                   float (&m)[2], float (&l)[2], int lim0, int lim1, float scale_log2,
                                                   bool need_mask, int lane) {
    constexpr int PAGE_BYTES = 2 * 16 * HD * 2;
    constexpr int KSPLIT = NPG >= 4 ? 1 : 2;   // independent accumulator chains when few pages
    const int c = lane & 3;
    const int mi = lane >> 3;
    const uint32_t page0 = smem_u32(stage) + (uint32_t)first_page * PAGE_BYTES;

    // S = Q K^T (raw scores)
    float acc[KSPLIT][NPG * 2][4];
#pragma unroll
    for (int a = 0; a < KSPLIT; ++a)
#pragma unroll
        for (int i = 0; i < NPG * 2; ++i) acc[a][i][0] = acc[a][i][1] = acc[a][i][2] = acc[a][i][3] = 0.f;
    {
        const int tok = ((mi >> 1) << 3) + (lane & 7);
#pragma unroll
        for (int ks = 0; ks < HD / 16; ++ks) {
            const int ch = 2 * ks + (mi & 1);
            const uint32_t off = (uint32_t)(ch >> 3) * 4096u + swz(tok, ch & 7);
#pragma unroll
            for (int pg = 0; pg < NPG; ++pg) {
                if (FULL || first_page + pg < n_valid_pages) {
                    uint32_t b0, b1, b2, b3;
                    ldsm_x4(page0 + pg * PAGE_BYTES + off, b0, b1, b2, b3);
                    mma_f16_16816(acc[ks % KSPLIT][pg * 2], qf[ks], b0, b1);
                    mma_f16_16816(acc[ks % KSPLIT][pg * 2 + 1], qf[ks], b2, b3);
                }
            }
        }
    }
    float s[NPG * 2][4];
#pragma unroll
    for (int i = 0; i < NPG * 2; ++i)
#pragma unroll
        for (int e = 0; e < 4; ++e) s[i][e] = KSPLIT == 2 ? acc[0][i][e] + acc[KSPLIT - 1][i][e] : acc[0][i][e];
    if (!FULL) {
#pragma unroll
        for (int pg = 0; pg < NPG; ++pg)
            if (first_page + pg >= n_valid_pages) {
#pragma unroll
                for (int e = 0; e < 4; ++e) s[pg * 2][e] = s[pg * 2 + 1][e] = -INFINITY;
            }
    }
    if (need_mask) {  // causal rule: row j sees key positions <= q_pos0 + j
#pragma unroll
        for (int pg = 0; pg < NPG; ++pg) {
            const int kv0 = stage_kv0 + (first_page + pg) * 16;
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int key = kv0 + nt * 8 + 2 * c + (e & 1);
                    if (key > ((e & 2) ? lim1 : lim0)) s[pg * 2 + nt][e] = -INFINITY;
                }
        }
    }
    // online softmax (base 2), rows g and g + 8
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int i = 0; i < NPG * 2; ++i) {
        mx[0] = fmaxf(mx[0], fmaxf(s[i][0], s[i][1]));
        mx[1] = fmaxf(mx[1], fmaxf(s[i][2], s[i][3]));
    }
    float corr[2], base[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xFFFFFFFFu, mx[r], 1));
        mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xFFFFFFFFu, mx[r], 2));
        mx[r] = fmaxf(m[r], mx[r] * scale_log2);
        base[r] = mx[r] == -INFINITY ? 0.f : mx[r];
        corr[r] = ex2_approx(m[r] - base[r]);  // m = -inf -> 0
        m[r] = mx[r];
        l[r] *= corr[r];
    }
    // once the running maxima have settled the factors are exactly 1 in every lane: skip the pass
    if (!__all_sync(0xFFFFFFFFu, corr[0] == 1.f && corr[1] == 1.f)) {
#pragma unroll
        for (int nt = 0; nt < HD / 8; ++nt) {
            o[nt][0] *= corr[0];
            o[nt][1] *= corr[0];
            o[nt][2] *= corr[1];
            o[nt][3] *= corr[1];
        }
    }
    // P = exp2(S * scale - m), O += P V
    const int tokv = ((mi & 1) << 3) + (lane & 7);
#pragma unroll
    for (int pg = 0; pg < NPG; ++pg) {
        if (FULL || first_page + pg < n_valid_pages) {
            uint32_t pa[4];
            {
                const float p00 = ex2_approx(fmaf(s[pg * 2][0], scale_log2, -base[0]));
                const float p01 = ex2_approx(fmaf(s[pg * 2][1], scale_log2, -base[0]));
                const float p02 = ex2_approx(fmaf(s[pg * 2][2], scale_log2, -base[1]));
                const float p03 = ex2_approx(fmaf(s[pg * 2][3], scale_log2, -base[1]));
                const float p10 = ex2_approx(fmaf(s[pg * 2 + 1][0], scale_log2, -base[0]));
                const float p11 = ex2_approx(fmaf(s[pg * 2 + 1][1], scale_log2, -base[0]));
                const float p12 = ex2_approx(fmaf(s[pg * 2 + 1][2], scale_log2, -base[1]));
                const float p13 = ex2_approx(fmaf(s[pg * 2 + 1][3], scale_log2, -base[1]));
                l[0] += (p00 + p01) + (p10 + p11);
                l[1] += (p02 + p03) + (p12 + p13);
                pa[0] = pack_op(p00, p01);
                pa[1] = pack_op(p02, p03);
                pa[2] = pack_op(p10, p11);
                pa[3] = pack_op(p12, p13);
            }
            const uint32_t vb = page0 + pg * PAGE_BYTES + 2048;  // V rows follow the K rows
#pragma unroll
            for (int np = 0; np < HD / 16; ++np) {  // two n8 tiles (16 dims) per ldmatrix
                const int ch = 2 * np + (mi >> 1);
                uint32_t b0, b1, b2, b3;
                ldsm_x4_t(vb + (uint32_t)(ch >> 3) * 4096u + swz(tokv, ch & 7), b0, b1, b2, b3);
                mma_f16_16816(o[2 * np], pa, b0, b1);
                mma_f16_16816(o[2 * np + 1], pa, b2, b3);
            }
        }
    }
}

// Fold another warp's (m, l, O) of the same rows, stored in a merge slot, into this warp's.
template <int HD>
__device__ __forceinline__ void attn_fold_slot(const float* oth, float (&o)[HD / 8][4], float (&m)[2], float (&l)[2], int g,
                                               int c) {
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int rr = g + 8 * r;
        const float m2 = oth[rr * (HD + 4) + HD], l2 = oth[rr * (HD + 4) + HD + 1];
        const float mn = fmaxf(m[r], m2);
        const float bs = mn == -INFINITY ? 0.f : mn;
        const float c1 = ex2_approx(m[r] - bs), c2 = ex2_approx(m2 - bs);
        m[r] = mn;
        l[r] = l[r] * c1 + l2 * c2;
#pragma unroll
        for (int nt = 0; nt < HD / 8; ++nt) {
            const float2 ov = *reinterpret_cast<const float2*>(oth + rr * (HD + 4) + nt * 8 + 2 * c);
            o[nt][2 * r] = o[nt][2 * r] * c1 + ov.x * c2;
            o[nt][2 * r + 1] = o[nt][2 * r + 1] * c1 + ov.y * c2;
        }
    }
}

template <int HD>
__device__ __forceinline__ void attn_store_slot(float* mine, const float (&o)[HD / 8][4], const float (&m)[2],
                                                const float (&l)[2], int g, int c) {
#pragma unroll
    for (int nt = 0; nt < HD / 8; ++nt) {
        *reinterpret_cast<float2*>(mine + g * (HD + 4) + nt * 8 + 2 * c) = make_float2(o[nt][0], o[nt][1]);
        *reinterpret_cast<float2*>(mine + (g + 8) * (HD + 4) + nt * 8 + 2 * c) = make_float2(o[nt][2], o[nt][3]);
    }
    if (c == 0) {
        mine[g * (HD + 4) + HD] = m[0];
        mine[g * (HD + 4) + HD + 1] = l[0];
        mine[(g + 8) * (HD + 4) + HD] = m[1];
        mine[(g + 8) * (HD + 4) + HD + 1] = l[1];
    }
}

__device__ __forceinline__ void consumer_bar() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

template <int HD>
__global__ void __launch_bounds__(ATT_THREADS, 1)
attn_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmKV, AttnParams p) {
    using SM = AttnSmem<HD>;
    constexpr int HALVES = HD / 64;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* stages = smem;
    uint8_t* qbuf = smem + SM::STAGES * SM::STAGE_BYTES;
    float* merge = reinterpret_cast<float*>(qbuf + 2 * SM::Q_BYTES);
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(merge) + SM::MERGE_BYTES);
    uint64_t* empty_bar = full_bar + 2 * SM::STAGES;   // full_bar[group][slot]
    uint64_t* qfull_bar = empty_bar + SM::STAGES;
    uint64_t* qempty_bar = qfull_bar + 2;
    int* last_flag = reinterpret_cast<int*>(qempty_bar + 2);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int it_begin = p.cta_begin[blockIdx.x], it_end = p.cta_begin[blockIdx.x + 1];
    const int G = p.group;

    if (threadIdx.x == 0) {
        tma_prefetch_desc(&tmQ);
        tma_prefetch_desc(&tmKV);
        for (int s = 0; s < SM::STAGES; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&full_bar[SM::STAGES + s], 1);
            mbar_init(&empty_bar[s], 4);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(&qfull_bar[s], 1);
            mbar_init(&qempty_bar[s], ATT_CONSUMER_WARPS);
        }
        mbar_fence_init();
    }
    pdl_launch_dependents();
    __syncthreads();
    pdl_wait();   // Q and the chunk's K/V come from the preceding projection kernel

    if (warp >= ATT_CONSUMER_WARPS) {
        // ------------------------------------------------------------ producer (one warp of its warpgroup)
        reg_dealloc<ATT_PRODUCER_REGS>();   // the whole warpgroup hands registers to the consumers
        if (warp > ATT_CONSUMER_WARPS) return;
        uint32_t st = 0;  // running stage counter
        bool ok = true;
        const int my_pg = lane / HALVES, my_half = lane % HALVES;
        for (int it = it_begin; it < it_end && ok; ++it) {
            const AttnItem item = p.items[it];
            if (!attn_item_ok(item, p)) break;   // the consumers flag it and stop waiting
            const int qi = it - it_begin, qb = qi & 1;
            if (lane == 0) {
                if (qi >= 2) ok = mbar_wait(&qempty_bar[qb], ((qi >> 1) - 1) & 1, p.status);
                if (ok) {
                    mbar_expect_tx(&qfull_bar[qb], (uint32_t)p.q_box_tokens * G * HD * 2u);
                    tma_load_3d(qbuf + qb * SM::Q_BYTES, &tmQ, &qfull_bar[qb], 0, item.kvh * G * HALVES, item.q_tok);
                }
            }
            ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
            // Page-table entries: the warp holds the entries of 8 stages (32 pages, one per lane) and fetches the
            // next 32 while those are in use, so no load's latency sits between two stages' requests.
            const int* pt = p.page_tables + (size_t)item.req * p.max_pages;
            const int first_page = item.kv_begin >> 4, last_page = (item.kv_end - 1) >> 4;
            int ent_cur = first_page + lane <= last_page ? pt[first_page + lane] : 0;
            int ent_next = first_page + 32 + lane <= last_page ? pt[first_page + 32 + lane] : 0;
            int k = 0;   // stage of the item
            for (int kv0 = item.kv_begin; kv0 < item.kv_end; kv0 += 16 * ATT_STAGE_PAGES, ++st, ++k) {
                const int s = st % SM::STAGES;
                if (k > 0 && (k & 7) == 0) {
                    ent_cur = ent_next;
                    const int nidx = first_page + (k >> 3) * 32 + 32 + lane;
                    ent_next = nidx <= last_page ? pt[nidx] : 0;
                }
                int page = __shfl_sync(0xFFFFFFFFu, ent_cur, ((k & 7) * ATT_STAGE_PAGES + my_pg) & 31);
                const int npg = min(ATT_STAGE_PAGES, (item.kv_end - kv0 + 15) >> 4);
                uint64_t* fb = &full_bar[(st & 1u) * SM::STAGES + s];   // the consuming group's barrier
                if (lane == 0) {
                    if (st >= (uint32_t)SM::STAGES) ok = mbar_wait(&empty_bar[s], ((st / SM::STAGES) - 1) & 1, p.status);
                    if (ok) mbar_expect_tx(fb, npg * SM::PAGE_BYTES);
                }
                ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
                if (my_pg < npg && (unsigned)page >= (unsigned)p.n_pages) {
                    atomicExch(p.status, 2);
                    page = 0;
                }
                if (my_pg < npg) {
                    const int row0 = (p.layer_block0 + 2 * (page * p.n_kv_heads + item.kvh)) * 16;
                    tma_load_2d(stages + s * SM::STAGE_BYTES + my_pg * SM::PAGE_BYTES + my_half * 4096, &tmKV, fb,
                                my_half * 64, row0);
                }
            }
        }
        return;
    }

    // ---------------------------------------------------------------- consumers (warps 0..7)
    reg_alloc<ATT_CONSUMER_REGS>();
    // A wait that runs out sets `ok` = false; the warp then skips all further waits and arithmetic
    // but still walks the items and takes part in every named barrier, so no other warp is left
    // waiting for it.
    const int cg = warp >> 2, w4 = warp & 3;   // stage-parity group, position inside the group
    const int g = lane >> 2, c = lane & 3;
    uint32_t st = 0;
    bool ok = true;
    const bool list_ok = it_begin >= 0 && it_begin <= it_end && it_end <= p.n_items;
    if (!list_ok && threadIdx.x == 0) atomicExch(p.status, 2);
    for (int it = it_begin; list_ok && it < it_end; ++it) {
        const AttnItem item = p.items[it];
        if (!attn_item_ok(item, p)) {   // uniform over the CTA: every warp leaves here together
            if (threadIdx.x == 0) atomicExch(p.status, 2);
            break;
        }
        const int qi = it - it_begin, qb = qi & 1;
        const int rows = item.nj * G;
        const int n_mt = (rows + 15) >> 4;
        const int npw = n_mt >= 3 ? 4 : n_mt;        // row-tile slots of a group (1, 2 or 4) == pages per warp
        const int mt = w4 % npw, kg = w4 / npw;      // row tile and page group of this warp
        const bool active = mt < n_mt;

        // Q fragments of this warp's row tile
        uint32_t qf[HD / 16][4];
        if (ok) ok = mbar_wait(&qfull_bar[qb], (qi >> 1) & 1, p.status);
        {
            const uint32_t qs = smem_u32(qbuf + qb * SM::Q_BYTES);
            const int mi = lane >> 3;
            const int row = mt * 16 + ((mi & 1) << 3) + (lane & 7);
#pragma unroll
            for (int ks = 0; ks < HD / 16; ++ks) {
                const int ch = 2 * ks + (mi >> 1);
                const uint32_t line = row * HALVES + (ch >> 3);
                if (active && ok) ldsm_x4(qs + swz(line, ch & 7), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
                else qf[ks][0] = qf[ks][1] = qf[ks][2] = qf[ks][3] = 0u;
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&qempty_bar[qb]);

        float o[HD / 8][4];
#pragma unroll
        for (int nt = 0; nt < HD / 8; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
        float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};
        const int lim0 = item.q_pos0 + (mt * 16 + g) / G, lim1 = item.q_pos0 + (mt * 16 + g + 8) / G;

        for (int kv0 = item.kv_begin; kv0 < item.kv_end; kv0 += 16 * ATT_STAGE_PAGES, ++st) {
            if ((int)(st & 1u) != cg) continue;
            const int s = st % SM::STAGES;
            // this group's own "full" barrier of the slot: it completes one phase per use of the slot
            // by this group, i.e. every second use
            if (ok) ok = mbar_wait(&full_bar[cg * SM::STAGES + s], ((st / SM::STAGES) >> 1) & 1, p.status);
            if (active && ok) {
                const int npg = min(ATT_STAGE_PAGES, (item.kv_end - kv0 + 15) >> 4);
                const bool need_mask = kv0 + 16 * ATT_STAGE_PAGES - 1 > item.q_pos0;
                const bool full = npg == ATT_STAGE_PAGES;
                const uint8_t* sp = stages + s * SM::STAGE_BYTES;
                if (npw == 4) {
                    if (full) attn_consume_stage<HD, 4, true>(sp, 0, npg, kv0, qf, o, m, l, lim0, lim1, p.scale_log2, need_mask, lane);
                    else attn_consume_stage<HD, 4, false>(sp, 0, npg, kv0, qf, o, m, l, lim0, lim1, p.scale_log2, need_mask, lane);
                } else if (npw == 2) {
                    if (full) attn_consume_stage<HD, 2, true>(sp, kg * 2, npg, kv0, qf, o, m, l, lim0, lim1, p.scale_log2, need_mask, lane);
                    else attn_consume_stage<HD, 2, false>(sp, kg * 2, npg, kv0, qf, o, m, l, lim0, lim1, p.scale_log2, need_mask, lane);
                } else {
                    if (full) attn_consume_stage<HD, 1, true>(sp, kg, npg, kv0, qf, o, m, l, lim0, lim1, p.scale_log2, need_mask, lane);
                    else attn_consume_stage<HD, 1, false>(sp, kg, npg, kv0, qf, o, m, l, lim0, lim1, p.scale_log2, need_mask, lane);
                }
            }
            __syncwarp();
            if (lane == 0 && ok) mbar_arrive(&empty_bar[s]);
        }

        // row sums across the quad
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            l[r] += __shfl_xor_sync(0xFFFFFFFFu, l[r], 1);
            l[r] += __shfl_xor_sync(0xFFFFFFFFu, l[r], 2);
        }
        // merge 1: the other stage-parity group's state of the same (row tile, page group)
        float* slot = merge + w4 * 16 * (HD + 4);
        consumer_bar();                               // slots free: the previous item's readers are done
        if (cg == 1) attn_store_slot<HD>(slot, o, m, l, g, c);
        consumer_bar();
        if (cg == 0) {
            attn_fold_slot<HD>(slot, o, m, l, g, c);
            // merge 2: the page groups of a row tile, in the fixed order kg = 1, 2, 3
            if (npw < 4) {
                if (kg > 0) attn_store_slot<HD>(slot, o, m, l, g, c);
                asm volatile("bar.sync 2, 128;" ::: "memory");
                if (kg == 0)
                    for (int k2 = 1; k2 < 4 / npw; ++k2) attn_fold_slot<HD>(merge + (k2 * npw + mt) * 16 * (HD + 4), o, m, l, g, c);
            }
            // write: final output (half precision) or fp32 partial
            if (active && kg == 0 && ok) {
#pragma unroll
                for (int r = 0; r < 2; ++r) {
                    const int row = mt * 16 + g + 8 * r;
                    if (row < rows) {
                        const int j = row / G, gq = row - j * G;
                        if (item.part < 0) {
                            const float inv = l[r] > 0.f ? 1.f / l[r] : 0.f;
                            op16* dst = p.out + (size_t)(item.q_tok + j) * p.q_dim + (item.kvh * G + gq) * HD;
#pragma unroll
                            for (int nt = 0; nt < HD / 8; ++nt)
                                *reinterpret_cast<uint32_t*>(dst + nt * 8 + 2 * c) =
                                    pack_op(o[nt][2 * r] * inv, o[nt][2 * r + 1] * inv);
                        } else {
                            float* dst = p.part_o + ((size_t)item.part * p.row_cap + row) * HD;
#pragma unroll
                            for (int nt = 0; nt < HD / 8; ++nt)
                                *reinterpret_cast<float2*>(dst + nt * 8 + 2 * c) = make_float2(o[nt][2 * r], o[nt][2 * r + 1]);
                            if (c == 0) p.part_ml[(size_t)item.part * p.row_cap + row] = make_float2(m[r], l[r]);
                        }
                    }
                }
            }
        }
        // a partial item: count it; the CTA that completes the group combines the partials
        if (item.part >= 0) {
            __threadfence();
            consumer_bar();
            if (threadIdx.x == 0) {
                const MergeGroup gr = p.groups[item.grp];
                const int done = atomicAdd(p.group_count + item.grp, 1);
                const int last = done == gr.n_parts - 1;
                if (last) p.group_count[item.grp] = 0;   // ready for the next launch
                *last_flag = last;
            }
            consumer_bar();
            if (*last_flag) {
                __threadfence();
                // 4 threads per row, each 1/4 of the row's columns; all loads of a thread are independent
                const MergeGroup gr = p.groups[item.grp];
                constexpr int CW = HD / 4;   // columns per thread
                const int row = threadIdx.x >> 2, c0 = (threadIdx.x & 3) * CW;
                if (row < rows) {
                    float mx = -INFINITY;
                    for (int k = 0; k < gr.n_parts; ++k) mx = fmaxf(mx, __ldcg(&p.part_ml[(size_t)(gr.part0 + k) * p.row_cap + row]).x);
                    const float bs = mx == -INFINITY ? 0.f : mx;
                    float lsum = 0.f;
                    float4 acc[CW / 4];
#pragma unroll
                    for (int i = 0; i < CW / 4; ++i) acc[i] = make_float4(0.f, 0.f, 0.f, 0.f);
                    for (int k = 0; k < gr.n_parts; ++k) {
                        const float2 ml = __ldcg(&p.part_ml[(size_t)(gr.part0 + k) * p.row_cap + row]);
                        const float w = ex2_approx(ml.x - bs);
                        lsum += ml.y * w;
                        const float4* src = reinterpret_cast<const float4*>(p.part_o + ((size_t)(gr.part0 + k) * p.row_cap + row) * HD + c0);
#pragma unroll
                        for (int i = 0; i < CW / 4; ++i) {
                            const float4 v = __ldcg(src + i);
                            acc[i].x += v.x * w; acc[i].y += v.y * w; acc[i].z += v.z * w; acc[i].w += v.w * w;
                        }
                    }
                    const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
                    const int j = row / G, gq = row - j * G;
                    uint2* dst = reinterpret_cast<uint2*>(p.out + (size_t)(gr.q_tok + j) * p.q_dim + (gr.kvh * G + gq) * HD + c0);
#pragma unroll
                    for (int i = 0; i < CW / 4; ++i)
                        dst[i] = make_uint2(pack_op(acc[i].x * inv, acc[i].y * inv), pack_op(acc[i].z * inv, acc[i].w * inv));
                }
            }
        }
    }
}

}  // namespace syn
