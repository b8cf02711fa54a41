// Ragged multi-query attention over the paged KV cache (paper Sec. 3.2 attention equation,
// applied to a chunk of 1..16 query tokens per request appended to a cached prefix, Sec. 3.4).
//
// One work item = (request, kv head, token sub-range of the chunk, key range).  The G query heads
// that share the kv head and the chunk's tokens are packed into one tile of rows (row = j*G + g),
// so every K/V byte of the item is read from HBM once.  A persistent CTA walks a host-planned
// list of items: one producer warp streams pages (TMA, 128-byte swizzle, one box of 32 rows x 128 bytes
// per page and 64-element half: K and V of 16 tokens) and the item's Q tile through mbarrier rings; four consumer
// warps run QK^T and PV on warp-level MMAs (m16n8k16, bf16 in, fp32 accumulate) with an online
// softmax in fp32.  Warps split the item's row tiles and, when there are fewer than four row
// tiles, the pages of every stage; their partial (max, sum, O) triples are merged in shared memory.
// Items that cover only part of a request's keys write an fp32 partial that attn_merge_kernel
// combines.
#pragma once
#include "ptx.cuh"

namespace syn {

struct AttnItem {
    int q_tok;      // index of the first query token of this item in the flattened batch
    int nj;         // query tokens in this item (rows = nj * G <= 64)
    int kvh;        // kv head
    int req;        // request (page table row)
    int kv_begin;   // first key position (multiple of 64)
    int kv_end;     // one past the last key position this item reads
    int q_pos0;     // position of the item's first query token (ctx + j0): row j sees keys <= q_pos0 + j
    int part;       // -1: sole item of its rows -> writes the output; else index of its partial
};

struct AttnParams {
    const AttnItem* items;      // sorted by CTA
    const int* cta_begin;       // [n_cta + 1]
    const int* page_tables;     // [B][max_pages]
    int max_pages;
    int n_kv_heads, group;      // G = Hq / Hkv
    int q_dim;                  // Hq * hd
    int layer_block0;           // 2 * layer * n_pages * Hkv: first (K|V) block of this layer in the pool map
    float scale_log2;           // log2(e) / sqrt(hd)
    __nv_bfloat16* out;         // [T][q_dim]
    float* part_o;              // [n_parts][64][hd]
    float2* part_ml;            // [n_parts][64] (max in log2 units, sum)
    int* status;
};

constexpr int ATT_STAGE_PAGES = 4;
constexpr int ATT_THREADS = 160;

template <int HD>
struct AttnSmem {
    static constexpr int PAGE_BYTES = 2 * 16 * HD * 2;            // K and V of one page, one head
    static constexpr int STAGE_BYTES = ATT_STAGE_PAGES * PAGE_BYTES;
    static constexpr int STAGES = HD == 128 ? 4 : 8;
    static constexpr int Q_BYTES = 16 * 8 * HD * 2;                // up to G = 8 heads x 16 tokens (box), rows used <= 64
    static constexpr int MERGE_BYTES = 4 * 16 * (HD + 4) * 4;      // per consumer warp: O[16][HD] + (m, l)[16]
    static constexpr int TOTAL = 1024 + STAGES * STAGE_BYTES + 2 * Q_BYTES + MERGE_BYTES + 512;
};

// byte offset of the 16-byte chunk `c16` of 128-byte line `line` under the 128-byte swizzle
__device__ __forceinline__ uint32_t swz(uint32_t line, uint32_t c16) { return line * 128u + ((c16 ^ (line & 7u)) << 4); }

template <int HD, int NPG>
__device__ __forceinline__ void attn_consume_stage(const uint8_t* stage, int first_page, int n_valid_pages,
                                                   int stage_kv0, const uint32_t (&qf)[HD / 16][4], float (&o)[HD / 8][4],
                                                   float (&m)[2], float (&l)[2], int row_j0, int row_j1, int q_pos0,
                                                   float scale_log2, bool need_mask, int lane) {
    constexpr int PAGE_BYTES = 2 * 16 * HD * 2;
    const int c = lane & 3;
    float s[NPG * 2][4];
#pragma unroll
    for (int i = 0; i < NPG * 2; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = -INFINITY;

    // S = Q K^T for this warp's pages
#pragma unroll
    for (int pg = 0; pg < NPG; ++pg) {
        if (first_page + pg < n_valid_pages) {
            const uint32_t kb = smem_u32(stage) + (first_page + pg) * PAGE_BYTES;  // page: [half][K rows | V rows][64]
            float acc[2][4] = {};
#pragma unroll
            for (int ks = 0; ks < HD / 16; ++ks) {
                const int mi = lane >> 3;
                const int tok = ((mi >> 1) << 3) + (lane & 7);
                const int ch = 2 * ks + (mi & 1);
                uint32_t b0, b1, b2, b3;
                ldsm_x4(kb + (ch >> 3) * 4096 + swz(tok, ch & 7), b0, b1, b2, b3);
                mma_bf16_16816(acc[0], qf[ks], b0, b1);
                mma_bf16_16816(acc[1], qf[ks], b2, b3);
            }
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) s[pg * 2 + nt][e] = acc[nt][e] * scale_log2;
            if (need_mask) {  // causal rule: row j sees key positions <= q_pos0 + j
                const int kv0 = stage_kv0 + (first_page + pg) * 16;
#pragma unroll
                for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int key = kv0 + nt * 8 + 2 * c + (e & 1);
                        const int lim = q_pos0 + ((e & 2) ? row_j1 : row_j0);
                        if (key > lim) s[pg * 2 + nt][e] = -INFINITY;
                    }
            }
        }
    }
    // online softmax (base 2), rows g and g + 8
    float mx[2] = {m[0], m[1]};
#pragma unroll
    for (int i = 0; i < NPG * 2; ++i) {
        mx[0] = fmaxf(mx[0], fmaxf(s[i][0], s[i][1]));
        mx[1] = fmaxf(mx[1], fmaxf(s[i][2], s[i][3]));
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xFFFFFFFFu, mx[r], 1));
        mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xFFFFFFFFu, mx[r], 2));
    }
    float corr[2], base[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        base[r] = mx[r] == -INFINITY ? 0.f : mx[r];
        corr[r] = exp2f(m[r] - base[r]);  // m = -inf -> 0
        m[r] = mx[r];
        l[r] *= corr[r];
    }
#pragma unroll
    for (int nt = 0; nt < HD / 8; ++nt) {
        o[nt][0] *= corr[0];
        o[nt][1] *= corr[0];
        o[nt][2] *= corr[1];
        o[nt][3] *= corr[1];
    }
    // P = exp2(S - m), O += P V
#pragma unroll
    for (int pg = 0; pg < NPG; ++pg) {
        if (first_page + pg < n_valid_pages) {
            uint32_t pa[4];
            {
                float p00 = exp2f(s[pg * 2][0] - base[0]), p01 = exp2f(s[pg * 2][1] - base[0]);
                float p02 = exp2f(s[pg * 2][2] - base[1]), p03 = exp2f(s[pg * 2][3] - base[1]);
                float p10 = exp2f(s[pg * 2 + 1][0] - base[0]), p11 = exp2f(s[pg * 2 + 1][1] - base[0]);
                float p12 = exp2f(s[pg * 2 + 1][2] - base[1]), p13 = exp2f(s[pg * 2 + 1][3] - base[1]);
                l[0] += p00 + p01 + p10 + p11;
                l[1] += p02 + p03 + p12 + p13;
                pa[0] = pack_bf16(p00, p01);
                pa[1] = pack_bf16(p02, p03);
                pa[2] = pack_bf16(p10, p11);
                pa[3] = pack_bf16(p12, p13);
            }
            const uint32_t vb = smem_u32(stage) + (first_page + pg) * PAGE_BYTES + 2048;  // V rows follow the K rows
#pragma unroll
            for (int np = 0; np < HD / 16; ++np) {  // two n8 tiles (16 dims) per ldmatrix
                const int mi = lane >> 3;
                const int tok = ((mi & 1) << 3) + (lane & 7);
                const int ch = 2 * np + (mi >> 1);
                uint32_t b0, b1, b2, b3;
                ldsm_x4_t(vb + (ch >> 3) * 4096 + swz(tok, ch & 7), b0, b1, b2, b3);
                mma_bf16_16816(o[2 * np], pa, b0, b1);
                mma_bf16_16816(o[2 * np + 1], pa, b2, b3);
            }
        }
    }
}

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
    uint64_t* empty_bar = full_bar + SM::STAGES;
    uint64_t* qfull_bar = empty_bar + SM::STAGES;
    uint64_t* qempty_bar = qfull_bar + 2;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int it_begin = p.cta_begin[blockIdx.x], it_end = p.cta_begin[blockIdx.x + 1];
    const int G = p.group;

    if (threadIdx.x == 0) {
        tma_prefetch_desc(&tmQ);
        tma_prefetch_desc(&tmKV);
        for (int s = 0; s < SM::STAGES; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 4);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(&qfull_bar[s], 1);
            mbar_init(&qempty_bar[s], 4);
        }
        mbar_fence_init();
    }
    __syncthreads();

    if (warp == 4) {
        // ------------------------------------------------------------ producer
        if (elect_one()) {
            uint32_t st = 0;  // running stage counter
            bool ok = true;
            for (int it = it_begin; it < it_end && ok; ++it) {
                const AttnItem item = p.items[it];
                const int qi = it - it_begin;
                const int qb = qi & 1;
                if (qi >= 2) ok = mbar_wait(&qempty_bar[qb], ((qi >> 1) - 1) & 1, p.status);
                if (!ok) break;
                const uint32_t q_bytes = 16u * G * HD * 2u;
                mbar_expect_tx(&qfull_bar[qb], q_bytes);
                tma_load_3d(qbuf + qb * SM::Q_BYTES, &tmQ, &qfull_bar[qb], 0, item.kvh * G * HALVES, item.q_tok);
                const int* pt = p.page_tables + (size_t)item.req * p.max_pages;
                for (int kv0 = item.kv_begin; kv0 < item.kv_end; kv0 += 16 * ATT_STAGE_PAGES, ++st) {
                    const int s = st % SM::STAGES;
                    if (st >= (uint32_t)SM::STAGES) ok = mbar_wait(&empty_bar[s], ((st / SM::STAGES) - 1) & 1, p.status);
                    if (!ok) break;
                    const int npg = min(ATT_STAGE_PAGES, (item.kv_end - kv0 + 15) >> 4);
                    mbar_expect_tx(&full_bar[s], npg * SM::PAGE_BYTES);
                    for (int pg = 0; pg < npg; ++pg) {
                        const int page = pt[(kv0 >> 4) + pg];
                        const int row0 = (p.layer_block0 + 2 * (page * p.n_kv_heads + item.kvh)) * 16;
                        for (int h = 0; h < HALVES; ++h)
                            tma_load_2d(stages + s * SM::STAGE_BYTES + pg * SM::PAGE_BYTES + h * 4096, &tmKV, &full_bar[s],
                                        h * 64, row0);
                    }
                }
            }
        }
        __syncwarp();
        return;
    }

    // ---------------------------------------------------------------- consumers (warps 0..3)
    const int g = lane >> 2, c = lane & 3;
    uint32_t st = 0;
    bool ok = true;
    for (int it = it_begin; it < it_end && ok; ++it) {
        const AttnItem item = p.items[it];
        const int qi = it - it_begin, qb = qi & 1;
        const int rows = item.nj * G;
        const int n_mt = (rows + 15) >> 4;
        const int npw = n_mt >= 3 ? 4 : n_mt;        // pages of a stage per warp == row-tile slots (1, 2 or 4)
        const int mt = warp % npw, kg = warp / npw;  // row tile and page group of this warp
        const bool active = mt < n_mt;

        // Q fragments of this warp's row tile
        uint32_t qf[HD / 16][4];
        ok = mbar_wait(&qfull_bar[qb], (qi >> 1) & 1, p.status);
        if (!ok) break;
        {
            const uint32_t qs = smem_u32(qbuf + qb * SM::Q_BYTES);
            const int mi = lane >> 3;
            const int row = mt * 16 + ((mi & 1) << 3) + (lane & 7);
#pragma unroll
            for (int ks = 0; ks < HD / 16; ++ks) {
                const int ch = 2 * ks + (mi >> 1);
                const uint32_t line = row * HALVES + (ch >> 3);
                if (active) ldsm_x4(qs + swz(line, ch & 7), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
                else qf[ks][0] = qf[ks][1] = qf[ks][2] = qf[ks][3] = 0u;
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&qempty_bar[qb]);

        float o[HD / 8][4];
#pragma unroll
        for (int nt = 0; nt < HD / 8; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
        float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};
        const int row_j0 = (mt * 16 + g) / G, row_j1 = (mt * 16 + g + 8) / G;

        for (int kv0 = item.kv_begin; kv0 < item.kv_end; kv0 += 16 * ATT_STAGE_PAGES, ++st) {
            const int s = st % SM::STAGES;
            ok = mbar_wait(&full_bar[s], (st / SM::STAGES) & 1, p.status);
            if (!ok) break;
            if (active) {
                const int npg = min(ATT_STAGE_PAGES, (item.kv_end - kv0 + 15) >> 4);
                const bool need_mask = kv0 + 16 * ATT_STAGE_PAGES - 1 > item.q_pos0;
                const uint8_t* sp = stages + s * SM::STAGE_BYTES;
                if (npw == 4)
                    attn_consume_stage<HD, 4>(sp, 0, npg, kv0, qf, o, m, l, row_j0, row_j1, item.q_pos0, p.scale_log2,
                                              need_mask, lane);
                else if (npw == 2)
                    attn_consume_stage<HD, 2>(sp, kg * 2, npg, kv0, qf, o, m, l, row_j0, row_j1, item.q_pos0,
                                              p.scale_log2, need_mask, lane);
                else
                    attn_consume_stage<HD, 1>(sp, kg, npg, kv0, qf, o, m, l, row_j0, row_j1, item.q_pos0, p.scale_log2,
                                              need_mask, lane);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty_bar[s]);
        }
        if (!ok) break;

        // row sums across the quad
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            l[r] += __shfl_xor_sync(0xFFFFFFFFu, l[r], 1);
            l[r] += __shfl_xor_sync(0xFFFFFFFFu, l[r], 2);
        }
        // merge the page groups of a row tile through shared memory (fixed order: kg = 1, 2, 3)
        if (npw < 4) {
            float* mine = merge + warp * 16 * (HD + 4);
            if (kg > 0) {
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
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (kg == 0) {
                for (int k2 = 1; k2 < 4 / npw; ++k2) {
                    const float* oth = merge + (k2 * npw + mt) * 16 * (HD + 4);
#pragma unroll
                    for (int r = 0; r < 2; ++r) {
                        const int rr = g + 8 * r;
                        const float m2 = oth[rr * (HD + 4) + HD], l2 = oth[rr * (HD + 4) + HD + 1];
                        const float mn = fmaxf(m[r], m2);
                        const float bs = mn == -INFINITY ? 0.f : mn;
                        const float c1 = exp2f(m[r] - bs), c2 = exp2f(m2 - bs);
                        m[r] = mn;
                        l[r] = l[r] * c1 + l2 * c2;
#pragma unroll
                        for (int nt = 0; nt < HD / 8; ++nt) {
                            float2 ov = *reinterpret_cast<const float2*>(oth + rr * (HD + 4) + nt * 8 + 2 * c);
                            o[nt][2 * r] = o[nt][2 * r] * c1 + ov.x * c2;
                            o[nt][2 * r + 1] = o[nt][2 * r + 1] * c1 + ov.y * c2;
                        }
                    }
                }
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");
        }
        // write: final output (bf16) or fp32 partial
        if (active && kg == 0) {
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                const int row = mt * 16 + g + 8 * r;
                if (row < rows) {
                    const int j = row / G, gq = row - j * G;
                    if (item.part < 0) {
                        const float inv = l[r] > 0.f ? 1.f / l[r] : 0.f;
                        __nv_bfloat16* dst = p.out + (size_t)(item.q_tok + j) * p.q_dim + (item.kvh * G + gq) * HD;
#pragma unroll
                        for (int nt = 0; nt < HD / 8; ++nt)
                            *reinterpret_cast<uint32_t*>(dst + nt * 8 + 2 * c) =
                                pack_bf16(o[nt][2 * r] * inv, o[nt][2 * r + 1] * inv);
                    } else {
                        float* dst = p.part_o + ((size_t)item.part * 64 + row) * HD;
#pragma unroll
                        for (int nt = 0; nt < HD / 8; ++nt)
                            *reinterpret_cast<float2*>(dst + nt * 8 + 2 * c) = make_float2(o[nt][2 * r], o[nt][2 * r + 1]);
                        if (c == 0) p.part_ml[(size_t)item.part * 64 + row] = make_float2(m[r], l[r]);
                    }
                }
            }
        }
    }
}

// Combine the partials of row groups whose keys were split over several items.
struct MergeGroup {
    int q_tok, nj, kvh, part0, n_parts, pad0, pad1, pad2;
};

template <int HD>
__global__ void attn_merge_kernel(const MergeGroup* groups, const float* part_o, const float2* part_ml,
                                  __nv_bfloat16* out, int G, int q_dim) {
    const MergeGroup gr = groups[blockIdx.x];
    const int rows = gr.nj * G;
    for (int row = threadIdx.y; row < rows; row += blockDim.y) {
        float mx = -INFINITY;
        for (int k = 0; k < gr.n_parts; ++k) mx = fmaxf(mx, part_ml[(size_t)(gr.part0 + k) * 64 + row].x);
        const float bs = mx == -INFINITY ? 0.f : mx;
        float lsum = 0.f;
        float acc[HD / 32] = {};
        for (int k = 0; k < gr.n_parts; ++k) {
            const float2 ml = part_ml[(size_t)(gr.part0 + k) * 64 + row];
            const float w = exp2f(ml.x - bs);
            lsum += ml.y * w;
            const float* src = part_o + ((size_t)(gr.part0 + k) * 64 + row) * HD;
#pragma unroll
            for (int i = 0; i < HD / 32; ++i) acc[i] += src[threadIdx.x + 32 * i] * w;
        }
        const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
        const int j = row / G, gq = row - j * G;
        __nv_bfloat16* dst = out + (size_t)(gr.q_tok + j) * q_dim + (gr.kvh * G + gq) * HD;
#pragma unroll
        for (int i = 0; i < HD / 32; ++i) dst[threadIdx.x + 32 * i] = __float2bfloat16(acc[i] * inv);
    }
}

}  // namespace syn
