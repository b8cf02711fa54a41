// The projection GEMM on CTA pairs (clusters of two, tcgen05 cta_group::2), for batches of a few
// hundred tokens and more, where the one-CTA kernel is held back by what its operands cost to bring
// from L2: a 256-feature x 192-token item needs 56 KB per 64-wide k-block for 768 tensor-core cycles.
// Here the two CTAs of a cluster share one token tile: each loads HALF of its rows, and the MMA
// (M = 256, issued by the CTA of rank 0) reads both halves, so the same item costs 44 KB per k-block
// and CTA.  Same orientation and weight layout as gemm.cuh (D[feature][token], pre-swizzled weight
// tiles); the weights come through a tensor map here (rows of 128 bytes, no swizzle: the image is
// already the shared-memory one) because a load of either CTA must signal the rank-0 CTA's barrier.
// Two shapes of work item:
//   QUAD: a cluster owns TWO neighbouring feature pairs (512 features) x one token tile; CTA r holds
//         pair 2 pp + r in two accumulators (its two 128-feature tiles), taken in turn by the MMAs;
//   DUO : a cluster owns ONE pair (256 features) x one token tile, CTA r its tile r; the two
//         accumulators take alternate k-steps (an MMA into the accumulator of the MMA before it
//         waits for it) and the epilogue adds them.  For projections with few pair tiles (qkv, o).
// Schedule: items in full waves over the clusters, item = wave * clusters + cluster, token tile
// fastest (neighbouring clusters then stream the same weights).  With K shared by S clusters of a tile
// (projections with few tiles and a long K: down) the CTAs of equal rank exchange accumulators as in
// gemm.cuh's reduce-scatter.  Epilogues: those of gemm.cuh (epi_unit).
#pragma once
#include "gemm.cuh"

namespace syn {

struct Gemm2Params {
    int num_kb;      // k-blocks of 64
    int n_groups;    // QUAD: pairs of feature pairs; DUO: feature pairs
    int n_tt, TN;    // token tiles of TN columns (multiple of 16, <= 256)
    int n_stages;
    int splits, kb_per_split;   // splits > 1: every cluster owns one (tile, k range); reduce-scatter between clusters
    int rem_base, rem_extra;    // splits == 1, rem_base > 1: the R items left after the full waves are cut along K, the
                                // first rem_extra of them into rem_base + 1 parts, the others into rem_base parts, one
                                // part per cluster, so that the last round keeps every cluster busy for a fraction of an item
    float* fix_part;            // splits > 1: exchange slots, one per CTA
    int* fix_flag;              // splits > 1: two counters per (tile, rank)
    int n_sm;
    int* status;
    long long spin_limit;
};

__host__ __device__ inline int gemm2_a_bytes(bool duo) { return duo ? GEMM_TILE_BYTES : GEMM_A_BYTES; }
__host__ __device__ inline int gemm2_half_boxes(int TN) { return (TN / 2 + GEMM_BOX_ROWS - 1) / GEMM_BOX_ROWS; }
__host__ __device__ inline int gemm2_stage_bytes(int TN, bool duo) { return gemm2_a_bytes(duo) + gemm2_half_boxes(TN) * GEMM_BOX_BYTES; }
__host__ inline int gemm2_stages(int TN, bool duo) {
    int s = (GEMM_SMEM_MAX - gemm_fixed_smem(TN)) / gemm2_stage_bytes(TN, duo);
    return s > GEMM_MAX_STAGES ? GEMM_MAX_STAGES : s;
}

struct Gemm2Work {
    int grp, tt, kb0, kb1, tile;
    int split, nsplit;   // nsplit > 1: part `split` of a tile whose K is shared by nsplit clusters
    int first_cl;        // nsplit > 1: the cluster that holds part 0 (the others follow)
    int counter;         // nsplit > 1: which counter pair the tile's clusters meet on
};

// Work item i of cluster `cl` of `n_cl`.
__host__ __device__ __forceinline__ bool gemm2_work(const Gemm2Params& g, int cl, int n_cl, int i, Gemm2Work& w) {
    const int n_tiles = g.n_groups * g.n_tt;
    w.split = 0; w.nsplit = 1; w.first_cl = 0; w.counter = 0; w.kb0 = 0; w.kb1 = g.num_kb;
    if (g.splits > 1) {
        if (i > 0 || cl >= n_tiles * g.splits) return false;
        w.tile = cl / g.splits;
        w.split = cl - w.tile * g.splits;
        w.nsplit = g.splits; w.first_cl = w.tile * g.splits; w.counter = w.tile;
        w.grp = w.tile / g.n_tt; w.tt = w.tile - w.grp * g.n_tt;
        w.kb0 = w.split * g.kb_per_split;
        w.kb1 = w.kb0 + g.kb_per_split < g.num_kb ? w.kb0 + g.kb_per_split : g.num_kb;
        return true;
    }
    const int fw = n_tiles / n_cl;
    if (g.rem_base > 1 && i == fw) {
        // the last round: item r of the leftovers, part `split` of its K
        const int wide = g.rem_extra * (g.rem_base + 1);
        int r;
        if (cl < wide) {
            r = cl / (g.rem_base + 1);
            w.nsplit = g.rem_base + 1; w.first_cl = r * (g.rem_base + 1);
        } else {
            r = g.rem_extra + (cl - wide) / g.rem_base;
            w.nsplit = g.rem_base; w.first_cl = wide + (r - g.rem_extra) * g.rem_base;
        }
        w.tile = fw * n_cl + r;
        if (w.tile >= n_tiles) return false;
        w.split = cl - w.first_cl; w.counter = r;
        w.grp = w.tile / g.n_tt; w.tt = w.tile - w.grp * g.n_tt;
        w.kb0 = (int)((long long)w.split * g.num_kb / w.nsplit);
        w.kb1 = (int)((long long)(w.split + 1) * g.num_kb / w.nsplit);
        return true;
    }
    w.tile = i * n_cl + cl;
    if (w.tile >= n_tiles || (g.rem_base > 1 && i > fw)) return false;
    w.grp = w.tile / g.n_tt; w.tt = w.tile - w.grp * g.n_tt;
    return true;
}

template <bool DUO>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm2_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, Gemm2Params g, EpiParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int stage_bytes = gemm2_stage_bytes(g.TN, DUO);
    constexpr int A_BYTES = DUO ? GEMM_TILE_BYTES : GEMM_A_BYTES;
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + g.n_stages * stage_bytes);   // used in the rank-0 CTA
    uint64_t* empty_bar = full_bar + GEMM_MAX_STAGES;   // own: the stage's MMAs are done (commit arrives in both CTAs)
    uint64_t* accf_bar = empty_bar + GEMM_MAX_STAGES;   // own: accumulators complete
    uint64_t* acce_bar = accf_bar + 1;                  // rank 0's: accumulators drained by the epilogue warps of both CTAs
    uint64_t* rs_bar = acce_bar + 1;                    // own: RMSNorm scales of the item's tokens are in rs_s
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(rs_bar + 1);
    float* rs_s = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(full_bar) + GEMM_BAR_BYTES);   // [2][rs stride]
    float* scr_s = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(full_bar) + gemm_scr_offset(g.TN));   // [epilogue warp][16][33]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int n_cl = gridDim.x >> 1, cl = (int)cluster_id_x();
    const long long limit = g.spin_limit;
    pdl_launch_dependents();
    constexpr uint32_t acc_stride = 256, tmem_cols = 512;

    if (threadIdx.x == 0) {
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
        for (int s = 0; s < g.n_stages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        mbar_init(accf_bar, 1);
        mbar_init(acce_bar, 2 * GEMM_EPI_WARPS);
        mbar_init(rs_bar, GEMM_EPI_WARPS);
        mbar_fence_init();
    }
    if (warp == 1) {
        tmem_alloc_pair(tmem_slot, tmem_cols);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();   // both CTAs' barriers exist before either signals the other's
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------ producer (one per CTA)
        if (elect_one()) {
            uint32_t it = 0;
            bool ok = true;
            Gemm2Work w;
            for (int i = 0; ok && gemm2_work(g, cl, n_cl, i, w); ++i) {
                const int n0 = w.tt * g.TN;
                const int nn = (min(g.TN, p.T - n0) + 15) & ~15;
                const int half = nn >> 1;                          // token rows this CTA brings
                const int nbox = (half + GEMM_BOX_ROWS - 1) / GEMM_BOX_ROWS;
                const uint32_t my_bytes = (uint32_t)(A_BYTES + nbox * GEMM_BOX_BYTES);
                // rows of the weight map: [pair][k-block][2][128]
                const int pair = DUO ? w.grp : 2 * w.grp + (int)rank;
                const int nk = w.kb1 - w.kb0, rot = gemm_k_rotation(cl, n_cl, nk);
                // the weights never depend on an earlier kernel: the first item's ring is requested
                // before waiting for the predecessor, whose output is only the token operand
                const int n_early = i == 0 ? min(nk, g.n_stages) : 0;
                for (int j = 0; j < n_early; ++j) {
                    const int kb = w.kb0 + (j + rot) % nk;
                    if (rank == 0) mbar_expect_tx(&full_bar[j], 2 * my_bytes);
                    tma_load_2d_pair(smem + j * stage_bytes, &tmA, mapa_rank(smem_u32(&full_bar[j]), 0), 0,
                                     ((pair * g.num_kb + kb) * 2 + (DUO ? (int)rank : 0)) * 128);
                }
                if (i == 0) pdl_wait();
                for (int j = 0; j < nk; ++j, ++it) {
                    const int kb = w.kb0 + (j + rot) % nk;
                    const int s = it % g.n_stages;
                    if (it >= (uint32_t)g.n_stages && !mbar_wait(&empty_bar[s], ((it / g.n_stages) - 1) & 1, g.status, limit)) {
                        ok = false;
                        break;
                    }
                    uint8_t* a_s = smem + s * stage_bytes;
                    uint8_t* b_s = a_s + A_BYTES;
                    const uint32_t fb = mapa_rank(smem_u32(&full_bar[s]), 0);
                    if (j >= n_early) {
                        if (rank == 0) mbar_expect_tx(&full_bar[s], 2 * my_bytes);
                        tma_load_2d_pair(a_s, &tmA, fb, 0, ((pair * g.num_kb + kb) * 2 + (DUO ? (int)rank : 0)) * 128);
                    }
                    for (int b = 0; b < nbox; ++b)
                        tma_load_2d_pair(b_s + b * GEMM_BOX_BYTES, &tmB, fb, kb * GEMM_BK, n0 + (int)rank * half + b * GEMM_BOX_ROWS);
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (rank 0 only)
        if (rank == 0 && elect_one()) {
            uint32_t it = 0;
            bool ok = true;
            Gemm2Work w;
            for (int i = 0; ok && gemm2_work(g, cl, n_cl, i, w); ++i) {
                const uint32_t nn = (uint32_t)((min(g.TN, p.T - w.tt * g.TN) + 15) & ~15);
                const uint32_t idesc = umma_idesc_f16(256, nn);
                if (i > 0) {   // the epilogues of both CTAs must have drained the previous item's accumulators
                    ok = mbar_wait(acce_bar, (i - 1) & 1, g.status, limit);
                    if (!ok) break;
                    tc_fence_after();
                }
                const int nk = w.kb1 - w.kb0;
                for (int j = 0; j < nk; ++j, ++it) {
                    const int s = it % g.n_stages;
                    ok = mbar_wait(&full_bar[s], (it / g.n_stages) & 1, g.status, limit);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_addr = smem_u32(smem + s * stage_bytes);
                    const uint64_t db = umma_desc_k128(a_addr + A_BYTES);
                    // consecutive MMAs go to different accumulators: an MMA into the accumulator of its
                    // predecessor waits for it
#pragma unroll
                    for (int k = 0; k < GEMM_BK / 16; ++k) {  // 16 bf16 = 32 bytes = 2 descriptor address units
                        if (DUO) {
                            umma_bf16_pair(tmem_base + (k & 1) * acc_stride, umma_desc_k128(a_addr) + 2 * k, db + 2 * k, idesc,
                                           j > 0 || k >= 2);
                        } else {
                            for (int mt = 0; mt < 2; ++mt)
                                umma_bf16_pair(tmem_base + mt * acc_stride, umma_desc_k128(a_addr + mt * GEMM_TILE_BYTES) + 2 * k,
                                               db + 2 * k, idesc, j > 0 || k > 0);
                        }
                    }
                    umma_commit_pair(&empty_bar[s]);
                }
                if (ok) umma_commit_pair(accf_bar);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ epilogue (both CTAs)
        const int e = warp - 2;
        const int grp = e >> 2;               // the groups take the 16-token chunks round robin
        constexpr int NGRP = GEMM_EPI_WARPS / 4;
        const int quarter = warp & 3;         // TMEM lane quarter this warp may read
        const bool scaled = p.ssq_in != nullptr;
        const uint32_t acce_c = mapa_rank(smem_u32(acce_bar), 0);
        float* const scr = scr_s + e * EPI_SCR_FLOATS;
        bool ok = true;
        Gemm2Work w;
        pdl_wait();   // the epilogues read and write buffers of earlier kernels
        for (int i = 0; ok && gemm2_work(g, cl, n_cl, i, w); ++i) {
            const int n0 = w.tt * g.TN;
            const int n_valid = min(g.TN, p.T - n0);
            const int nchunks = (n_valid + EPI_COLS - 1) / EPI_COLS;
            float* const rsi = rs_s + (i & 1) * gemm_rs_stride(g.TN);
            if (scaled) {   // while the main loop runs: the scales of this item's tokens
                epi_rms_scales(p, rsi, n0, n_valid, e, lane);
                __syncwarp();
                if (lane == 0) mbar_arrive(rs_bar);
            }
            ok = mbar_wait(accf_bar, i & 1, g.status, limit);
            if (ok && scaled) ok = mbar_wait(rs_bar, i & 1, g.status, limit);
            if (!ok) break;
            tc_fence_after();
            // this CTA's features: QUAD both tiles of pair 2 grp + rank, DUO tile `rank` of pair grp
            const int n_mt = DUO ? 1 : 2;
            const int row0 = DUO ? w.grp * 256 + (int)rank * 128 : (2 * w.grp + (int)rank) * 256;
            const int total_chunks = n_mt * nchunks;
            if (w.nsplit > 1) {
                // ---- reduce-scatter between the S clusters that share this tile, CTAs of equal rank
                // (see gemm.cuh): this CTA keeps the chunks [c_lo, c_hi) and hands the others over.
                const int S = w.nsplit, sp = w.split, cnt = w.counter * 2 + (int)rank;   // counter pair of (tile, rank)
                const int cpt = g.TN / EPI_COLS;
                const size_t slot_elems = (size_t)2 * cpt * 128 * EPI_COLS;
                const int c_lo = sp * nchunks / S, c_hi = (sp + 1) * nchunks / S;
                float* const mine = g.fix_part + (size_t)blockIdx.x * slot_elems;
                int nth = 0;
                for (int mt = 0; mt < n_mt; ++mt)
                    for (int c = 0; c < nchunks; ++c) {
                        if (c >= c_lo && c < c_hi) continue;
                        if ((nth++ & (NGRP - 1)) != grp) continue;
                        uint32_t r[EPI_COLS];
                        tmem_ld16(tmem_base + mt * acc_stride + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(c * EPI_COLS), r);
                        if (DUO) {
                            uint32_t r2[EPI_COLS];
                            tmem_ld16(tmem_base + acc_stride + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(c * EPI_COLS), r2);
                            tmem_ld_wait();
#pragma unroll
                            for (int v = 0; v < EPI_COLS; ++v) r[v] = __float_as_uint(__uint_as_float(r[v]) + __uint_as_float(r2[v]));
                        } else {
                            tmem_ld_wait();
                        }
                        uint4* dst = reinterpret_cast<uint4*>(mine + (((size_t)mt * cpt + c) * 4 + quarter) * 32 * EPI_COLS) + lane;
#pragma unroll
                        for (int v = 0; v < EPI_COLS / 4; ++v) dst[v * 32] = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
                    }
                __threadfence();
                __syncwarp();
                if (lane == 0) atomicAdd(g.fix_flag + cnt, 1);
                if (lane == 0) {
                    const int want = S * GEMM_EPI_WARPS;
                    const long long t_end = clock64() + limit;
                    while (ld_acquire_gpu(g.fix_flag + cnt) < want) {
                        if (clock64() > t_end) {
                            atomicExch(g.status, 1);
                            break;
                        }
                    }
                }
                __syncwarp();
                nth = 0;
                for (int mt = 0; mt < n_mt; ++mt)
                    for (int c = c_lo; c < c_hi; ++c) {
                        if ((nth++ & (NGRP - 1)) != grp) continue;
                        const int m0 = row0 + mt * 128;
                        uint32_t own[EPI_COLS], r[EPI_COLS];
                        tmem_ld16(tmem_base + mt * acc_stride + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(c * EPI_COLS), own);
                        if (DUO) {
                            tmem_ld16(tmem_base + acc_stride + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(c * EPI_COLS), r);
                            tmem_ld_wait();
#pragma unroll
                            for (int v = 0; v < EPI_COLS; ++v) own[v] = __float_as_uint(__uint_as_float(own[v]) + __uint_as_float(r[v]));
                        } else {
                            tmem_ld_wait();
                        }
                        const size_t at = (((size_t)mt * cpt + c) * 4 + quarter) * 32 * EPI_COLS;
                        for (int q = 0; q < S; ++q) {   // fixed order: the parts in split order
                            if (q == sp) {
#pragma unroll
                                for (int v = 0; v < EPI_COLS; ++v)
                                    r[v] = q == 0 ? own[v] : __float_as_uint(__uint_as_float(r[v]) + __uint_as_float(own[v]));
                            } else {
                                const size_t peer = (size_t)((w.first_cl + q) * 2 + (int)rank);   // the CTA of the same rank in the cluster of part q
                                const float4* src = reinterpret_cast<const float4*>(g.fix_part + peer * slot_elems + at) + lane;
#pragma unroll
                                for (int v = 0; v < EPI_COLS / 4; ++v) {
                                    const float4 q4 = __ldcg(src + v * 32);
                                    if (q == 0) {
                                        r[4 * v] = __float_as_uint(q4.x); r[4 * v + 1] = __float_as_uint(q4.y);
                                        r[4 * v + 2] = __float_as_uint(q4.z); r[4 * v + 3] = __float_as_uint(q4.w);
                                    } else {
                                        r[4 * v] = __float_as_uint(__uint_as_float(r[4 * v]) + q4.x);
                                        r[4 * v + 1] = __float_as_uint(__uint_as_float(r[4 * v + 1]) + q4.y);
                                        r[4 * v + 2] = __float_as_uint(__uint_as_float(r[4 * v + 2]) + q4.z);
                                        r[4 * v + 3] = __float_as_uint(__uint_as_float(r[4 * v + 3]) + q4.w);
                                    }
                                }
                            }
                        }
                        const int tc0 = n0 + c * EPI_COLS, ncols = min(EPI_COLS, n_valid - c * EPI_COLS);
                        if (m0 < p.N) epi_dispatch(p.mode, p, r, scaled ? rsi + c * EPI_COLS : nullptr, scr, m0, tc0, ncols, quarter, lane);
                    }
                __syncwarp();
                if (lane == 0 && atomicAdd(g.fix_flag + 2 * g.n_sm + cnt, 1) == S * GEMM_EPI_WARPS - 1) {
                    g.fix_flag[cnt] = 0;
                    g.fix_flag[2 * g.n_sm + cnt] = 0;
                }
                continue;
            }
            for (int ci = grp; ci < total_chunks; ci += NGRP) {
                const int mt = ci / nchunks, c = ci % nchunks;
                const int m0 = row0 + mt * 128;
                uint32_t r[EPI_COLS];
                tmem_ld16(tmem_base + mt * acc_stride + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(c * EPI_COLS), r);
                if (DUO) {
                    uint32_t r2[EPI_COLS];
                    tmem_ld16(tmem_base + acc_stride + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(c * EPI_COLS), r2);
                    tmem_ld_wait();
#pragma unroll
                    for (int v = 0; v < EPI_COLS; ++v) r[v] = __float_as_uint(__uint_as_float(r[v]) + __uint_as_float(r2[v]));
                } else {
                    tmem_ld_wait();
                }
                if (ci + NGRP >= total_chunks) {   // last TMEM read of this warp for this item
                    tc_fence_before();
                    if (lane == 0) mbar_arrive_cluster(acce_c);
                }
                const int tc0 = n0 + c * EPI_COLS, ncols = min(EPI_COLS, n_valid - c * EPI_COLS);
                if (m0 < p.N) epi_dispatch(p.mode, p, r, scaled ? rsi + c * EPI_COLS : nullptr, scr, m0, tc0, ncols, quarter, lane);
            }
            if (grp >= total_chunks) {   // a group without any chunk still releases the accumulators
                tc_fence_before();
                if (lane == 0) mbar_arrive_cluster(acce_c);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();   // the partner may still read this CTA's shared memory or tensor memory until here
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, tmem_cols);
    }
}

}  // namespace syn
