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
// Warp roles: warp 0 streams K and V pages (TMA, boxes of 16 rows x 128 bytes, separate rings for K
// and V because a stage's K is free two steps before its V) and the Q tile through mbarriers; one
// thread of warp 1 issues every MMA; warps 4..7 (one thread per row) do the online softmax in fp32
// (base 2) and the item's epilogue.  Pipeline: while the softmax warps work on stage k - 1, the
// tensor pipe computes the scores of stage k and O += P V of stage k - 2.  The running maximum used
// for P is only raised when a stage's maximum exceeds it by more than 2^8 (P stays well inside half
// precision); O in tensor memory is rescaled at those moments only, and the final division by the
// row sum uses the same maximum, so the result is the exact softmax whatever the moments were.
// Items that cover part of a request's keys store fp32 partials (m, l, O) that the CTA completing a
// row group combines in part order, as in attention.cuh.  Every wait is bounded.
#pragma once
#include "attention.cuh"

namespace syn {

constexpr int ATT2_THREADS = 256;
constexpr int ATT2_ROWS = 128;
constexpr int ATT2_STAGE_KEYS = 64;
constexpr float ATT2_RESCALE_GAP = 8.0f;   // log2 units

template <int HD>
struct Attn2Smem {
    static constexpr int HALVES = HD / 64;
    static constexpr int KBOX_BYTES = 16 * 128;                       // 16 keys x 64 dims
    static constexpr int K_BYTES = HALVES * ATT2_STAGE_KEYS * 128;    // K (or V) of a stage: [half][64 keys][128 bytes]
    static constexpr int Q_BYTES = HALVES * ATT2_ROWS * 128;          // [half][128 rows][128 bytes]
    static constexpr int P_BYTES = ATT2_ROWS * 128;                   // [128 rows][64 keys]
    static constexpr int K_SLOTS = HD == 128 ? 4 : 6;                 // K is released when the stage's scores are done,
    static constexpr int V_SLOTS = HD == 128 ? 6 : 8;                 // V two steps later
    static constexpr int BAR_BYTES = 512;
    static constexpr int TOTAL = 1024 + (K_SLOTS + V_SLOTS) * K_BYTES + Q_BYTES + 2 * P_BYTES + BAR_BYTES;
    static constexpr int TMEM_COLS = 512;   // O: HD columns at 0; two score buffers of 2 x 64 columns at 128 and 256
};

__device__ __forceinline__ void att2_bar() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

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
    uint64_t* s_full = q_empty + 1;      // [2] scores of a stage are in tensor memory
    uint64_t* s_empty = s_full + 2;      // [2] the softmax warps have read them
    uint64_t* p_full = s_empty + 2;      // [2] P of a stage is in shared memory (and O rescaled if need be)
    uint64_t* p_empty = p_full + 2;      // [2] the stage's P V is complete
    uint64_t* o_full = p_empty + 2;      // the item's last P V is complete
    uint64_t* o_empty = o_full + 1;      // the softmax warps have read O
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(o_empty + 1);
    int* last_flag = reinterpret_cast<int*>(tmem_slot + 1);
    static_assert((2 * KS + 2 * VS + 12) * 8 + 8 <= SM::BAR_BYTES, "barrier area");

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
    if (warp == 1) {
        tmem_alloc(tmem_slot, SM::TMEM_COLS);
        tmem_relinquish();
    }
    pdl_launch_dependents();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();   // Q and the chunk's K/V come from the preceding projection kernel

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        // lane -> (page of the stage, 64-dim half, K or V) for the 16-row boxes of a stage
        const int my_pg = lane / (2 * HALVES), my_half = (lane / 2) % HALVES, my_v = lane & 1;
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
            const int* pt = p.page_tables + (size_t)item.req * p.max_pages;
            const int last_page = (item.kv_end - 1) >> 4;
            int pidx = (item.kv_begin >> 4) + my_pg;
            int page = (my_pg < ATT_STAGE_PAGES && pidx <= last_page) ? pt[pidx] : 0;
            for (int kv0 = item.kv_begin; kv0 < item.kv_end; kv0 += ATT2_STAGE_KEYS, ++st) {
                const int ks = st % KS, vs = st % VS;
                const int nidx = pidx + ATT_STAGE_PAGES;
                const int page_next = (my_pg < ATT_STAGE_PAGES && nidx <= last_page) ? pt[nidx] : 0;
                const int npg = min(ATT_STAGE_PAGES, (item.kv_end - kv0 + 15) >> 4);
                if (lane == 0) {
                    if (st >= (uint32_t)KS) ok = mbar_wait(&k_empty[ks], ((st / KS) - 1) & 1u, p.status);
                    if (ok && st >= (uint32_t)VS) ok = mbar_wait(&v_empty[vs], ((st / VS) - 1) & 1u, p.status);
                    if (ok) {
                        mbar_expect_tx(&k_full[ks], (uint32_t)npg * HALVES * SM::KBOX_BYTES);
                        mbar_expect_tx(&v_full[vs], (uint32_t)npg * HALVES * SM::KBOX_BYTES);
                    }
                }
                ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
                if (my_pg < npg && (unsigned)page >= (unsigned)p.n_pages) {
                    atomicExch(p.status, 2);
                    page = 0;
                }
                if (my_pg < npg) {
                    const int row0 = (p.layer_block0 + 2 * (page * p.n_kv_heads + item.kvh) + my_v) * 16;
                    uint8_t* dst = (my_v ? vring + vs * SM::K_BYTES : kring + ks * SM::K_BYTES) +
                                   my_half * (ATT2_STAGE_KEYS * 128) + my_pg * SM::KBOX_BYTES;
                    tma_load_2d(dst, &tmKV, my_v ? &v_full[vs] : &k_full[ks], my_half * 64, row0);
                }
                page = page_next;
                pidx = nidx;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (one thread)
        // An MMA into the accumulator of its predecessor waits about 144 cycles for it, more than
        // these small MMAs take, so three accumulators are in flight and consecutive MMAs go to
        // different ones: the scores of stage k as two partial sums over halves of the head
        // dimension (the softmax warps add them), and O += P V of stage k - 2.
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
                // step k: scores of stage k (k < n_st) interleaved with P V of stage k - 2 (k >= 2)
                for (int k = 0; k < n_st + 2 && ok; ++k) {
                    const bool qk = k < n_st, pv = k >= 2;
                    const uint32_t tq = st + k, tp = st + k - 2;
                    uint32_t k_addr = 0, idesc_qk = 0, s_tmem = 0, p_addr = 0, v_addr = 0;
                    int npv = 0;
                    if (qk) {
                        ok = mbar_wait(&k_full[tq % KS], (tq / KS) & 1u, p.status);
                        if (ok && (tq >> 1) >= 1) ok = mbar_wait(&s_empty[tq & 1u], ((tq >> 1) - 1) & 1u, p.status);
                        k_addr = smem_u32(kring + (tq % KS) * SM::K_BYTES);
                        idesc_qk = umma_idesc_f16(ATT2_ROWS, 16 * pages_of(k));
                        s_tmem = tmem_base + 128 + (tq & 1u) * 128;
                    }
                    if (pv && ok) {
                        ok = mbar_wait(&p_full[tp & 1u], (tp >> 1) & 1u, p.status);
                        if (ok) ok = mbar_wait(&v_full[tp % VS], (tp / VS) & 1u, p.status);
                        if (ok && k == 2 && qi >= 1) ok = mbar_wait(o_empty, (uint32_t)(qi - 1) & 1u, p.status);
                        p_addr = smem_u32(pbuf + (tp & 1u) * SM::P_BYTES);
                        v_addr = smem_u32(vring + (tp % VS) * SM::K_BYTES);
                        npv = pages_of(k - 2);
                    }
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        if (qk && i < QK_STEPS) {
                            // partial sum A: dims [0, HD/2) -> columns 0..63 of the buffer; B: dims [HD/2, HD) -> 64..127
                            const uint32_t qa = 2 * i, ka = 2 * i;
                            const uint32_t qb = HD == 128 ? ((ATT2_ROWS * 128) >> 4) + 2 * i : 2 * (i + QK_STEPS);
                            const uint32_t kb = HD == 128 ? ((ATT2_STAGE_KEYS * 128) >> 4) + 2 * i : 2 * (i + QK_STEPS);
                            umma_bf16(s_tmem, umma_desc_k128(q_addr) + qa, umma_desc_k128(k_addr) + ka, idesc_qk, i != 0);
                            umma_bf16(s_tmem + 64, umma_desc_k128(q_addr) + qb, umma_desc_k128(k_addr) + kb, idesc_qk, i != 0);
                        }
                        if (pv && i < npv)
                            umma_bf16(tmem_base, umma_desc_k128(p_addr) + 2 * i,
                                      umma_desc_mn128(v_addr + i * 2048, ATT2_STAGE_KEYS * 128, 1024), idesc_pv, !(k == 2 && i == 0));
                    }
                    if (qk) {
                        umma_commit(&s_full[tq & 1u]);
                        umma_commit(&k_empty[tq % KS]);
                        if (k == n_st - 1) umma_commit(q_empty);
                    }
                    if (pv) {
                        umma_commit(&v_empty[tp % VS]);
                        umma_commit(&p_empty[tp & 1u]);
                        if (k == n_st + 1) umma_commit(o_full);
                    }
                }
                st += (uint32_t)n_st;
            }
        }
        __syncwarp();
    } else if (warp >= 4) {
        // ------------------------------------------------------------ softmax and epilogue (thread = row)
        // A wait that runs out sets `ok` = false; the warp then skips all further waits and tensor-memory
        // traffic but still walks the items and takes part in every named barrier.
        const int wq = warp - 4, row = wq * 32 + lane;
        const uint32_t t_lane = tmem_base + ((uint32_t)(wq * 32) << 16);
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
            const int j = row / G, gq = row - j * G;
            const int lim = item.q_pos0 + j;   // last visible key position of this row
            float m_used = -INFINITY, l = 0.f;
            for (int kv0 = item.kv_begin; kv0 < item.kv_end; kv0 += ATT2_STAGE_KEYS, ++st) {
                const uint32_t sb = st & 1u, us = st >> 1;
                uint32_t s0[32], s1[32];
                if (ok) ok = wait_all(&s_full[sb], us & 1u);
                if (ok) {
                    // the two partial sums of the scores (halves of the head dimension)
                    uint32_t b0[32];
                    tc_fence_after();
                    tmem_ld32(t_lane + 128 + sb * 128, s0);
                    tmem_ld32(t_lane + 128 + sb * 128 + 64, b0);
                    tmem_ld_wait();
#pragma unroll
                    for (int c = 0; c < 32; ++c) s0[c] = __float_as_uint(__uint_as_float(s0[c]) + __uint_as_float(b0[c]));
                    tmem_ld32(t_lane + 128 + sb * 128 + 32, s1);
                    tmem_ld32(t_lane + 128 + sb * 128 + 96, b0);
                    tmem_ld_wait();
#pragma unroll
                    for (int c = 0; c < 32; ++c) s1[c] = __float_as_uint(__uint_as_float(s1[c]) + __uint_as_float(b0[c]));
                    tc_fence_before();
                } else {
#pragma unroll
                    for (int c = 0; c < 32; ++c) s0[c] = s1[c] = 0u;
                }
                __syncwarp();
                if (lane == 0 && ok) mbar_arrive(&s_empty[sb]);
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
                const bool first = kv0 == item.kv_begin;
                if (first) {
                    m_used = live ? ms : 0.f;
                } else {
                    const bool grow = live && ms > m_used + ATT2_RESCALE_GAP;
                    if (__any_sync(0xFFFFFFFFu, grow)) {
                        // O is rescaled in tensor memory: the previous stage's P V must have completed
                        if (ok) ok = wait_all(&p_empty[(st - 1) & 1u], ((st - 1) >> 1) & 1u);
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
                                tmem_ld32(t_lane + ch * 32, o);
                                tmem_ld_wait();
#pragma unroll
                                for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * corr);
                                tmem_st32(t_lane + ch * 32, o);
                            }
                            tmem_st_wait();
                        }
                    }
                }
                // P = exp2(S * scale - m), row sum, P to shared memory (K-major, 128-byte swizzle)
                if (us >= 1 && ok) ok = wait_all(&p_empty[sb], (us - 1) & 1u);
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
                    pw[c] = live ? pack_op(a, b) : 0u;
                    pw[16 + c] = live ? pack_op(c2, d) : 0u;
                }
                l += sum;
                if (ok) {
                    uint8_t* prow = pbuf + sb * SM::P_BYTES;
#pragma unroll
                    for (int c16 = 0; c16 < 8; ++c16)
                        *reinterpret_cast<uint4*>(prow + swz(row, c16)) =
                            make_uint4(pw[4 * c16], pw[4 * c16 + 1], pw[4 * c16 + 2], pw[4 * c16 + 3]);
                    fence_proxy_async_smem();
                    tc_fence_before();
                }
                __syncwarp();
                if (lane == 0 && ok) mbar_arrive(&p_full[sb]);
            }
            // ---- the item's output: O / l (half precision), or the fp32 partial (m, l, O)
            if (ok) ok = wait_all(o_full, (uint32_t)qi & 1u);
            if (ok) {
                tc_fence_after();
                const float inv = l > 0.f ? 1.f / l : 0.f;
#pragma unroll 1
                for (int ch = 0; ch < HD / 32; ++ch) {
                    uint32_t o[32];
                    tmem_ld32(t_lane + ch * 32, o);
                    tmem_ld_wait();
                    if (live) {
                        if (item.part < 0) {
                            uint4* dst = reinterpret_cast<uint4*>(p.out + (size_t)(item.q_tok + j) * p.q_dim + (item.kvh * G + gq) * HD + ch * 32);
#pragma unroll
                            for (int c = 0; c < 4; ++c)
                                dst[c] = make_uint4(pack_op(__uint_as_float(o[8 * c]) * inv, __uint_as_float(o[8 * c + 1]) * inv),
                                                    pack_op(__uint_as_float(o[8 * c + 2]) * inv, __uint_as_float(o[8 * c + 3]) * inv),
                                                    pack_op(__uint_as_float(o[8 * c + 4]) * inv, __uint_as_float(o[8 * c + 5]) * inv),
                                                    pack_op(__uint_as_float(o[8 * c + 6]) * inv, __uint_as_float(o[8 * c + 7]) * inv));
                        } else {
                            uint4* dst = reinterpret_cast<uint4*>(p.part_o + ((size_t)item.part * p.row_cap + row) * HD + ch * 32);
#pragma unroll
                            for (int c = 0; c < 8; ++c) dst[c] = make_uint4(o[4 * c], o[4 * c + 1], o[4 * c + 2], o[4 * c + 3]);
                        }
                    }
                }
                tc_fence_before();
                if (live && item.part >= 0) p.part_ml[(size_t)item.part * p.row_cap + row] = make_float2(m_used, l);
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
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, SM::TMEM_COLS);
    }
}

}  // namespace syn
