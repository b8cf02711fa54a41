// Ragged multi-query attention over the paged KV cache on the tensor-memory path (paper Sec. 3.2
// attention equation, applied to a chunk of query tokens appended to a cached prefix, Sec. 3.4).
//
// Same work items as attention.cuh (request, kv head, token sub-range, key range), but the row tile
// of an item is 128 rows (row = j * G + g): a chunk of up to 128 / G tokens is ONE item per kv head,
// so every K/V byte of a request is read once per kv head however long the chunk is.  Both products
// run on tcgen05.mma with M = 128, in stages of 64 keys:
//   S = Q K^T : A = the Q tile (K-major, 128-byte swizzle), B = 64 keys of K (K-major), D = S in tensor
//               memory, as TWO partial sums over halves of the head dimension (see the MMA issuer);
//   O += P V  : A = P (half precision, written by the softmax warps into shared memory in the
//               K-major swizzled layout), B = V as it lies in the cache, [key][dim], i.e. an MN-major
//               operand, D = O in tensor memory for the whole item.
// Warp roles: warp 3 streams pages (TMA: one request brings the 16 K rows of a page, another its 16 V
// rows, each as [rows 0-7: dims 0-63][rows 0-7: dims 64-127][rows 8-15: ...], so that the 8-row groups
// of a stage's four pages are evenly spaced for either half of the head dimension; requests are the
// scarce resource of this loop, about 80 cycles each; K and V have rings of their own because a
// stage's K is free as soon as its scores are done, its V only after P V) and the Q tile through
// mbarriers; one thread of warp 2 issues every MMA; warps 4..7 and 8..11 are two softmax groups (one
// thread per row each) that take alternate stages, each with its own score buffer, P buffer, running
// (max, sum) and O accumulator in tensor memory; the first group combines the two at the end of the
// item and writes the result.  A group's softmax of a stage (fp32, base 2) therefore has two stage
// times, and the scores of its next stage are computed as soon as it has read the current ones.  The
// running maximum used for P is only raised when a stage's maximum exceeds it by more than 2^8 (P
// stays well inside half precision); O in tensor memory is rescaled at those moments only, and the
// final division by the row sum uses the same maximum, so the result is the exact softmax.
// Items that cover part of a request's keys store fp32 partials (m, l, O) that the CTA completing a
// row group combines in part order, as in attention.cuh.  Every wait is bounded.
#pragma once
#include "attention.cuh"

namespace syn {

constexpr int ATT2_THREADS = 384;
constexpr int ATT2_ROWS = 128;
constexpr int ATT2_STAGE_KEYS = 64;
constexpr float ATT2_RESCALE_GAP = 8.0f;   // log2 units
// The producer and the MMA issuer sit on the schedulers of the softmax warps that own rows 96..127 and 64..95: with
// fewer than 128 rows in a tile those are the warps with the least (or nothing) to do.
constexpr int ATT2_PRODUCER_WARP = 3, ATT2_MMA_WARP = 2;

template <int HD>
struct Attn2Smem {
    static constexpr int HALVES = HD / 64;
    static constexpr int GROUP_BYTES = HALVES * 1024;                 // 8 rows: [64-dim half][8 rows][128 bytes]
    static constexpr int BOX_BYTES = 2 * GROUP_BYTES;                 // the K rows (or the V rows) of a page
    static constexpr int K_BYTES = ATT_STAGE_PAGES * BOX_BYTES;       // K (or V) of a stage: [page][group][half][8 rows][128 bytes]
    static constexpr int Q_BYTES = HALVES * ATT2_ROWS * 128;          // [half][128 rows][128 bytes]
    static constexpr int P_BYTES = ATT2_ROWS * 128;                   // [128 rows][64 keys]
    static constexpr int K_SLOTS = HD == 128 ? 4 : 8;                 // K is released when the stage's scores are done,
    static constexpr int V_SLOTS = HD == 128 ? 6 : 12;                // V when its P V is
    static constexpr int BAR_BYTES = 512 + ATT2_ROWS * 8;             // barriers, then (max, sum) of the second group's rows
    static constexpr int TOTAL = 1024 + (K_SLOTS + V_SLOTS) * K_BYTES + Q_BYTES + 2 * P_BYTES + BAR_BYTES;
    static_assert(TOTAL <= 232448, "shared memory of one CTA");
    static constexpr int TMEM_COLS = 512;   // O of the two groups at 0 and 128; their score buffers (2 x 64 columns) at 256 and 384
};

__device__ __forceinline__ void att2_bar() { asm volatile("bar.sync 1, 128;" ::: "memory"); }         // first softmax group
__device__ __forceinline__ void att2_bar_both() { asm volatile("bar.sync 2, 256;" ::: "memory"); }    // both softmax groups

template <int HD>
__global__ void __launch_bounds__(ATT2_THREADS, 1)
attn2_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmKV, AttnParams p) {
    using SM = Attn2Smem<HD>;
    constexpr int HALVES = SM::HALVES, KS = SM::K_SLOTS, VS = SM::V_SLOTS;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* kring = smem;
    uint8_t* vring = kring + KS * SM::K_BYTES;
    uint8_t* qbuf = vring + VS * SM::K_BYTES;
    uint8_t* pbuf = qbuf + SM::Q_BYTES;
    uint64_t* k_full = reinterpret_cast<uint64_t*>(pbuf + 2 * SM::P_BYTES);
    uint64_t* k_empty = k_full + KS;     // the stage's scores are complete
    uint64_t* v_full = k_empty + KS;
    uint64_t* v_empty = v_full + VS;     // the stage's P V is complete
    uint64_t* q_full = v_empty + VS;
    uint64_t* q_empty = q_full + 1;      // the item's last QK^T has read the tile
    uint64_t* s_full = q_empty + 1;      // [group] scores of a stage are in tensor memory
    uint64_t* s_empty = s_full + 2;      // [group] its warps have read them
    uint64_t* p_full = s_empty + 2;      // [group] P of a stage is in shared memory (and O rescaled if need be)
    uint64_t* p_empty = p_full + 2;      // [group] the stage's P V is complete
    uint64_t* o_full = p_empty + 2;      // the item's last P V is complete
    uint64_t* o_empty = o_full + 1;      // the first group has read both O
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(o_empty + 1);
    int* last_flag = reinterpret_cast<int*>(tmem_slot + 1);
    static_assert((2 * KS + 2 * VS + 12) * 8 + 8 <= 512, "barrier area");
    float2* ml_x = reinterpret_cast<float2*>(reinterpret_cast<uint8_t*>(k_full) + 512);   // [128]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int it_begin = p.cta_begin[blockIdx.x], it_end = p.cta_begin[blockIdx.x + 1];
    const int G = p.group;
    const bool list_ok = it_begin >= 0 && it_begin <= it_end && it_end <= p.n_items;

    if (threadIdx.x == 0) {
        tma_prefetch_desc(&tmQ);
        tma_prefetch_desc(&tmKV);
        for (int s = 0; s < KS; ++s) {
            mbar_init(&k_full[s], 1);
            mbar_init(&k_empty[s], 1);
        }
        for (int s = 0; s < VS; ++s) {
            mbar_init(&v_full[s], 1);
            mbar_init(&v_empty[s], 1);
        }
        mbar_init(q_full, 1);
        mbar_init(q_empty, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&s_full[s], 1);
            mbar_init(&s_empty[s], 4);
            mbar_init(&p_full[s], 4);
            mbar_init(&p_empty[s], 1);
        }
        mbar_init(o_full, 1);
        mbar_init(o_empty, 4);
        mbar_fence_init();
        if (!list_ok) atomicExch(p.status, 2);
    }
    if (warp == ATT2_MMA_WARP) {
        tmem_alloc(tmem_slot, SM::TMEM_COLS);
        tmem_relinquish();
    }
    pdl_launch_dependents();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();   // Q and the chunk's K/V come from the preceding projection kernel

    if (warp == ATT2_PRODUCER_WARP) {
        // ------------------------------------------------------------ producer
        // lane -> (page of the stage, K or V): one request each
        const int my_pg = lane >> 1, my_v = lane & 1;
        uint32_t st = 0;
        bool ok = true;
        for (int it = it_begin; list_ok && it < it_end && ok; ++it) {
            const AttnItem item = p.items[it];
            if (!attn_item_ok(item, p)) break;   // the other roles flag it and stop as well
            const int qi = it - it_begin;
            if (lane == 0) {
                if (qi >= 1) ok = mbar_wait(q_empty, (uint32_t)(qi - 1) & 1u, p.status);
                if (ok) {
                    mbar_expect_tx(q_full, (uint32_t)p.q_box_tokens * G * HD * 2u);
                    for (int h = 0; h < HALVES; ++h)
                        tma_load_4d(qbuf + h * (ATT2_ROWS * 128), &tmQ, q_full, 0, h, item.kvh * G, item.q_tok);
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
            for (int kv0 = item.kv_begin; kv0 < item.kv_end; kv0 += ATT2_STAGE_KEYS, ++st, ++k) {
                const int ks = st % KS, vs = st % VS;
                if (k > 0 && (k & 7) == 0) {
                    ent_cur = ent_next;
                    const int nidx = first_page + (k >> 3) * 32 + 32 + lane;
                    ent_next = nidx <= last_page ? pt[nidx] : 0;
                }
                int page = __shfl_sync(0xFFFFFFFFu, ent_cur, ((k & 7) * ATT_STAGE_PAGES + my_pg) & 31);
                const int npg = min(ATT_STAGE_PAGES, (item.kv_end - kv0 + 15) >> 4);
                if (lane == 0) {
                    if (st >= (uint32_t)KS) ok = mbar_wait(&k_empty[ks], ((st / KS) - 1) & 1u, p.status);
                    if (ok && st >= (uint32_t)VS) ok = mbar_wait(&v_empty[vs], ((st / VS) - 1) & 1u, p.status);
                    if (ok) {
                        mbar_expect_tx(&k_full[ks], (uint32_t)npg * SM::BOX_BYTES);
                        mbar_expect_tx(&v_full[vs], (uint32_t)npg * SM::BOX_BYTES);
                    }
                }
                ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
                if (my_pg < npg && (unsigned)page >= (unsigned)p.n_pages) {
                    atomicExch(p.status, 2);
                    page = 0;
                }
                if (my_pg < npg) {
                    tma_load_5d((my_v ? vring + vs * SM::K_BYTES : kring + ks * SM::K_BYTES) + my_pg * SM::BOX_BYTES, &tmKV,
                                my_v ? &v_full[vs] : &k_full[ks], 0, 0, 0, 0,
                                p.layer_block0 + 2 * (page * p.n_kv_heads + item.kvh) + my_v);
                }
            }
        }
    } else if (warp == ATT2_MMA_WARP) {
        // ------------------------------------------------------------ MMA issuer (one thread)
        // Two streams of work share the tensor pipe: the scores of stage k (ready when its K has
        // landed and the owning softmax group has read its previous scores) and O += P V of stage k
        // (ready when that group has written P).  The thread issues whichever is ready, both
        // interleaved when both are.  An MMA into the accumulator of its predecessor waits about 144
        // cycles for it, more than these small MMAs take, so the scores are two partial sums over
        // halves of the head dimension (the softmax warps add them) and consecutive MMAs alternate
        // between accumulators.
        if (elect_one()) {
            uint32_t st = 0;   // global stage counter of the item's first stage
            bool ok = true;
            const uint32_t idesc_pv = umma_idesc_f16_bmn(ATT2_ROWS, HD);
            constexpr int QK_STEPS = HD / 32;   // k-steps of 16 dims per partial sum
            for (int it = it_begin; list_ok && it < it_end && ok; ++it) {
                const AttnItem item = p.items[it];
                if (!attn_item_ok(item, p)) break;
                const int qi = it - it_begin;
                ok = mbar_wait(q_full, (uint32_t)qi & 1u, p.status);
                if (!ok) break;
                const uint32_t q_addr = smem_u32(qbuf);
                const int n_st = (item.kv_end - item.kv_begin + ATT2_STAGE_KEYS - 1) / ATT2_STAGE_KEYS;
                auto pages_of = [&](int k) { return min(ATT_STAGE_PAGES, (item.kv_end - item.kv_begin - k * ATT2_STAGE_KEYS + 15) >> 4); };
                int nq = 0, np = 0;   // next stage of the item whose scores / whose P V is to be issued
                long long t0 = 0;
                uint32_t idle = 0;
                while (np < n_st) {
                    const uint32_t tq = st + nq, tp = st + np;
                    bool qk = nq < n_st && mbar_test(&k_full[tq % KS], (tq / KS) & 1u) &&
                              ((tq >> 1) == 0 || mbar_test(&s_empty[tq & 1u], ((tq >> 1) - 1) & 1u));
                    bool pv = np < nq && mbar_test(&p_full[tp & 1u], (tp >> 1) & 1u) && mbar_test(&v_full[tp % VS], (tp / VS) & 1u) &&
                              (np >= 2 || qi == 0 || mbar_test(o_empty, (uint32_t)(qi - 1) & 1u));
                    if (!qk && !pv) {
                        if ((++idle & 0x3FFu) == 0) {
                            const long long now = clock64();
                            if (t0 == 0) t0 = now;
                            else if (now - t0 > SYN_SPIN_LIMIT_CYCLES) {
                                atomicExch(p.status, 1);
                                ok = false;
                                break;
                            }
                        }
                        continue;
                    }
                    idle = 0;
                    t0 = 0;
                    tc_fence_after();
                    const uint32_t k_addr = smem_u32(kring + (tq % KS) * SM::K_BYTES);
                    const uint32_t idesc_qk = umma_idesc_f16(ATT2_ROWS, 16 * (qk ? pages_of(nq) : 1));
                    const uint32_t s_tmem = tmem_base + 256 + (tq & 1u) * 128;
                    const uint32_t p_addr = smem_u32(pbuf + (tp & 1u) * SM::P_BYTES);
                    const uint32_t v_addr = smem_u32(vring + (tp % VS) * SM::K_BYTES);
                    const uint32_t o_tmem = tmem_base + (tp & 1u) * 128;
                    const int npv = pv ? pages_of(np) : 0;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        if (qk && i < QK_STEPS) {
                            // partial sum A: dims [0, HD/2) -> columns 0..63 of the buffer; B: dims [HD/2, HD) -> 64..127
                            const uint32_t qa = 2 * i, ka = 2 * i;
                            const uint32_t qb = HD == 128 ? ((ATT2_ROWS * 128) >> 4) + 2 * i : 2 * (i + QK_STEPS);
                            const uint32_t kb = HD == 128 ? (1024 >> 4) + 2 * i : 2 * (i + QK_STEPS);   // the second half's 8 rows follow the first's
                            umma_bf16(s_tmem, umma_desc_k128(q_addr) + qa, umma_desc_k128s(k_addr, SM::GROUP_BYTES) + ka, idesc_qk, i != 0);
                            umma_bf16(s_tmem + 64, umma_desc_k128(q_addr) + qb, umma_desc_k128s(k_addr, SM::GROUP_BYTES) + kb, idesc_qk, i != 0);
                        }
                        if (i < npv)   // the group's first stage of the item starts its O afresh
                            umma_bf16(o_tmem, umma_desc_k128(p_addr) + 2 * i,
                                      umma_desc_mn128(v_addr + i * SM::BOX_BYTES, 1024, SM::GROUP_BYTES), idesc_pv, !(np < 2 && i == 0));
                    }
                    if (qk) {
                        umma_commit(&s_full[tq & 1u]);
                        umma_commit(&k_empty[tq % KS]);
                        if (nq == n_st - 1) umma_commit(q_empty);
                        ++nq;
                    }
                    if (pv) {
                        umma_commit(&v_empty[tp % VS]);
                        umma_commit(&p_empty[tp & 1u]);
                        if (np == n_st - 1) umma_commit(o_full);
                        ++np;
                    }
                }
                st += (uint32_t)n_st;
            }
        }
        __syncwarp();
    } else if (warp >= 4) {
        // ------------------------------------------------------------ softmax groups and epilogue (thread = row)
        // A wait that runs out sets `ok` = false; the warp then skips all further waits and tensor-memory
        // traffic but still walks the items and takes part in every named barrier.
        const int wg = (warp - 4) >> 2, wq = (warp - 4) & 3, row = wq * 32 + lane;   // group, lane quarter, row of the tile
        const uint32_t t_lane = tmem_base + ((uint32_t)(wq * 32) << 16);
        const uint32_t o_col = (uint32_t)wg * 128, s_col = 256 + (uint32_t)wg * 128;
        uint32_t st = 0;
        bool ok = true;   // uniform over the warp: the tensor-memory loads and stores are warp-wide
        auto wait_all = [&](uint64_t* bar, uint32_t parity) {
            const bool r = mbar_wait(bar, parity, p.status);
            return __all_sync(0xFFFFFFFFu, r) != 0;
        };
        for (int it = it_begin; list_ok && it < it_end; ++it) {
            const AttnItem item = p.items[it];
            if (!attn_item_ok(item, p)) {   // uniform over the CTA
                if (threadIdx.x == 128) atomicExch(p.status, 2);
                break;
            }
            const int qi = it - it_begin;
            const int rows = item.nj * G;
            const bool live = row < rows;
            const bool wlive = wq * 32 < rows;   // a warp none of whose rows exist only keeps the barriers' counts
            const int j = row / G, gq = row - j * G;
            const int lim = item.q_pos0 + j;   // last visible key position of this row
            float m_used = -INFINITY, l = 0.f;
            bool first = true;                 // this group's first stage of the item
            for (int kv0 = item.kv_begin; kv0 < item.kv_end; kv0 += ATT2_STAGE_KEYS, ++st) {
                if ((int)(st & 1u) != wg) continue;
                const uint32_t us = st >> 1;   // use number of this group's buffers
                uint32_t s0[32], s1[32];
                if (ok) ok = wait_all(&s_full[wg], us & 1u);
                if (ok && wlive) {
                    // the two partial sums of the scores (halves of the head dimension)
                    uint32_t b0[32];
                    tc_fence_after();
                    tmem_ld32(t_lane + s_col, s0);
                    tmem_ld32(t_lane + s_col + 64, b0);
                    tmem_ld_wait();
#pragma unroll
                    for (int c = 0; c < 32; ++c) s0[c] = __float_as_uint(__uint_as_float(s0[c]) + __uint_as_float(b0[c]));
                    tmem_ld32(t_lane + s_col + 32, s1);
                    tmem_ld32(t_lane + s_col + 96, b0);
                    tmem_ld_wait();
#pragma unroll
                    for (int c = 0; c < 32; ++c) s1[c] = __float_as_uint(__uint_as_float(s1[c]) + __uint_as_float(b0[c]));
                    tc_fence_before();
                } else {
#pragma unroll
                    for (int c = 0; c < 32; ++c) s0[c] = s1[c] = 0u;
                }
                __syncwarp();
                if (lane == 0 && ok) mbar_arrive(&s_empty[wg]);
                if (wlive) {
                // keys this row sees in the stage: positions < min(kv_end, lim + 1)
                const int nvalid = min(item.kv_end, lim + 1) - kv0;
                if (nvalid < ATT2_STAGE_KEYS) {
#pragma unroll
                    for (int c = 0; c < 32; ++c) {
                        if (c >= nvalid) s0[c] = 0xFF800000u;        // -inf
                        if (c + 32 >= nvalid) s1[c] = 0xFF800000u;
                    }
                }
                float mx = -INFINITY;
#pragma unroll
                for (int c = 0; c < 32; ++c) mx = fmaxf(mx, fmaxf(__uint_as_float(s0[c]), __uint_as_float(s1[c])));
                const float ms = mx * p.scale_log2;
                if (first) {
                    m_used = live ? ms : 0.f;
                } else {
                    const bool grow = live && ms > m_used + ATT2_RESCALE_GAP;
                    if (__any_sync(0xFFFFFFFFu, grow)) {
                        // O is rescaled in tensor memory: this group's previous P V must have completed
                        if (ok) ok = wait_all(&p_empty[wg], (us - 1) & 1u);
                        const float corr = grow ? ex2_approx(m_used - ms) : 1.f;
                        if (grow) {
                            m_used = ms;
                            l *= corr;
                        }
                        if (ok) {
                            tc_fence_after();
#pragma unroll 1
                            for (int ch = 0; ch < HD / 32; ++ch) {
                                uint32_t o[32];
                                tmem_ld32(t_lane + o_col + ch * 32, o);
                                tmem_ld_wait();
#pragma unroll
                                for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * corr);
                                tmem_st32(t_lane + o_col + ch * 32, o);
                            }
                            tmem_st_wait();
                        }
                    }
                }
                // P = exp2(S * scale - m), row sum, P to shared memory (K-major, 128-byte swizzle)
                if (us >= 1 && ok) ok = wait_all(&p_empty[wg], (us - 1) & 1u);
                const float base = m_used == -INFINITY ? 0.f : m_used;
                uint32_t pw[32];
                float sum = 0.f;
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    const float a = ex2_approx(fmaf(__uint_as_float(s0[2 * c]), p.scale_log2, -base));
                    const float b = ex2_approx(fmaf(__uint_as_float(s0[2 * c + 1]), p.scale_log2, -base));
                    const float c2 = ex2_approx(fmaf(__uint_as_float(s1[2 * c]), p.scale_log2, -base));
                    const float d = ex2_approx(fmaf(__uint_as_float(s1[2 * c + 1]), p.scale_log2, -base));
                    sum += (a + b) + (c2 + d);
                    pw[c] = pack_op(a, b);   // (rows beyond the tile's hold garbage: they only meet themselves in the products)
                    pw[16 + c] = pack_op(c2, d);
                }
                l += sum;
                if (ok) {
                    uint8_t* prow = pbuf + wg * SM::P_BYTES;
#pragma unroll
                    for (int c16 = 0; c16 < 8; ++c16)
                        *reinterpret_cast<uint4*>(prow + swz(row, c16)) =
                            make_uint4(pw[4 * c16], pw[4 * c16 + 1], pw[4 * c16 + 2], pw[4 * c16 + 3]);
                    fence_proxy_async_smem();
                    tc_fence_before();
                }
                } else if (us >= 1 && ok) {
                    // keeps this warp in step with the others: one arrival per warp and phase on p_full
                    ok = wait_all(&p_empty[wg], (us - 1) & 1u);
                }
                __syncwarp();
                if (lane == 0 && ok) mbar_arrive(&p_full[wg]);
                first = false;
            }
            // ---- end of the item: the second group hands its (max, sum) to the first, which combines the
            // two O accumulators: O / l in half precision, or the fp32 partial (m, l, O) of a split item
            if (wg == 1) ml_x[row] = make_float2(m_used, l);
            att2_bar_both();
            float2 other = make_float2(-INFINITY, 0.f);
            if (wg == 0) other = ml_x[row];
            att2_bar_both();   // the slot may be written again
            if (wg == 1) continue;
            const float m_all = fmaxf(m_used, other.x);
            const float bs_all = m_all == -INFINITY ? 0.f : m_all;
            const float wa = ex2_approx(m_used - bs_all), wb = ex2_approx(other.x - bs_all);   // -inf -> 0
            const float l_all = l * wa + other.y * wb;
            if (ok) ok = wait_all(o_full, (uint32_t)qi & 1u);
            if (ok) {
                tc_fence_after();
                const float inv = item.part < 0 ? (l_all > 0.f ? 1.f / l_all : 0.f) : 1.f;
                const float fa = wa * inv, fb = wb * inv;
#pragma unroll 1
                for (int ch = 0; ch < HD / 32; ++ch) {
                    uint32_t oa[32], ob[32];
                    tmem_ld32(t_lane + ch * 32, oa);
                    tmem_ld32(t_lane + 128 + ch * 32, ob);
                    tmem_ld_wait();
                    float v[32];
#pragma unroll
                    for (int c = 0; c < 32; ++c)   // a group without a stage in this item holds stale numbers: weight 0 drops them
                        v[c] = (wa > 0.f ? __uint_as_float(oa[c]) * fa : 0.f) + (wb > 0.f ? __uint_as_float(ob[c]) * fb : 0.f);
                    if (live) {
                        if (item.part < 0) {
                            uint4* dst = reinterpret_cast<uint4*>(p.out + (size_t)(item.q_tok + j) * p.q_dim + (item.kvh * G + gq) * HD + ch * 32);
#pragma unroll
                            for (int c = 0; c < 4; ++c)
                                dst[c] = make_uint4(pack_op(v[8 * c], v[8 * c + 1]), pack_op(v[8 * c + 2], v[8 * c + 3]),
                                                    pack_op(v[8 * c + 4], v[8 * c + 5]), pack_op(v[8 * c + 6], v[8 * c + 7]));
                        } else {
                            float4* dst = reinterpret_cast<float4*>(p.part_o + ((size_t)item.part * p.row_cap + row) * HD + ch * 32);
#pragma unroll
                            for (int c = 0; c < 8; ++c) dst[c] = make_float4(v[4 * c], v[4 * c + 1], v[4 * c + 2], v[4 * c + 3]);
                        }
                    }
                }
                tc_fence_before();
                if (live && item.part >= 0) p.part_ml[(size_t)item.part * p.row_cap + row] = make_float2(m_all, l_all);
            }
            __syncwarp();
            if (lane == 0 && ok) mbar_arrive(o_empty);
            // a partial item: count it; the CTA that completes the group combines the partials in part order
            if (item.part >= 0) {
                __threadfence();
                att2_bar();
                if (threadIdx.x == 128) {
                    const MergeGroup gr = p.groups[item.grp];
                    const int done = atomicAdd(p.group_count + item.grp, 1);
                    const int last = done == gr.n_parts - 1;
                    if (last) p.group_count[item.grp] = 0;   // ready for the next launch
                    *last_flag = last;
                }
                att2_bar();
                if (*last_flag) {
                    __threadfence();
                    const MergeGroup gr = p.groups[item.grp];
                    if (live) {
                        float mx = -INFINITY;
                        for (int k = 0; k < gr.n_parts; ++k)
                            mx = fmaxf(mx, __ldcg(&p.part_ml[(size_t)(gr.part0 + k) * p.row_cap + row]).x);
                        const float bs = mx == -INFINITY ? 0.f : mx;
                        float lsum = 0.f;
                        for (int k = 0; k < gr.n_parts; ++k) {
                            const float2 ml = __ldcg(&p.part_ml[(size_t)(gr.part0 + k) * p.row_cap + row]);
                            lsum += ml.y * ex2_approx(ml.x - bs);
                        }
                        const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
                        op16* orow = p.out + (size_t)(gr.q_tok + j) * p.q_dim + (gr.kvh * G + gq) * HD;
#pragma unroll 1
                        for (int ch = 0; ch < HD / 32; ++ch) {
                            float4 acc[8];
#pragma unroll
                            for (int c = 0; c < 8; ++c) acc[c] = make_float4(0.f, 0.f, 0.f, 0.f);
                            for (int k = 0; k < gr.n_parts; ++k) {
                                const float w = ex2_approx(__ldcg(&p.part_ml[(size_t)(gr.part0 + k) * p.row_cap + row]).x - bs);
                                const float4* src = reinterpret_cast<const float4*>(p.part_o + ((size_t)(gr.part0 + k) * p.row_cap + row) * HD + ch * 32);
#pragma unroll
                                for (int c = 0; c < 8; ++c) {
                                    const float4 v = __ldcg(src + c);
                                    acc[c].x += v.x * w; acc[c].y += v.y * w; acc[c].z += v.z * w; acc[c].w += v.w * w;
                                }
                            }
                            uint4* dst = reinterpret_cast<uint4*>(orow + ch * 32);
#pragma unroll
                            for (int c = 0; c < 4; ++c)
                                dst[c] = make_uint4(pack_op(acc[2 * c].x * inv, acc[2 * c].y * inv), pack_op(acc[2 * c].z * inv, acc[2 * c].w * inv),
                                                    pack_op(acc[2 * c + 1].x * inv, acc[2 * c + 1].y * inv),
                                                    pack_op(acc[2 * c + 1].z * inv, acc[2 * c + 1].w * inv));
                        }
                    }
                }
            }
        }
    }
    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == ATT2_MMA_WARP) {
        tc_fence_after();
        tmem_dealloc(tmem_base, SM::TMEM_COLS);
    }
}

}  // namespace syn
