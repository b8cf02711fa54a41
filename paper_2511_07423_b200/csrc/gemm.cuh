// Projection GEMM of the verification step for sm_100a, "swap-AB" orientation:
//   D[feature][token] = sum_k W[feature][k] * X[token][k]
// The weight matrix is the UMMA A operand (M = 128 output features per tile; a CTA normally owns a
// PAIR of such tiles that share one token tile), the ragged token batch is the UMMA B operand
// (N = 16..256 tokens), so a batch of T tokens pads to a multiple of 16 instead of 128.  Weights are
// stored pre-tiled and pre-swizzled ([feature pair][k-block][2][128 x 64] images of the
// 128-byte-swizzled shared-memory tile), so a stage's weights are ONE contiguous bulk copy;
// activations come through a TMA tensor map.  One persistent CTA per SM walks a static schedule.
// Three variants of the kernel (template parameter):
//   GEMM_WAVES  : whole pair tiles in full waves, leftovers as single 128-feature tiles;
//   GEMM_KSPLIT : as above, but the pair tiles left over after the full waves are cut along K into
//                 parts on different CTAs (the "helper" parts run first and store their fp32
//                 accumulators, the "owner" part runs last on another CTA, adds them in part order
//                 and finishes the tile);
//   GEMM_RSPLIT : projections with fewer pair tiles than SMs (o, down, qkv at a few hundred tokens):
//                 every tile's K range is split over S CTAs that run at the same time; each CTA
//                 keeps a contiguous share of the tile's token columns, hands the accumulators of
//                 the other columns to their keepers through global memory, adds what it receives
//                 in split order (so the sum does not depend on timing) and runs the epilogue on
//                 its own columns: a reduce-scatter, after which all S CTAs share the epilogue.
// Every CTA starts its k loop at a different k-block, so the CTAs that share a token tile do not
// ask L2 for the same lines at the same moment.  Accumulation is tcgen05.mma into TMEM, read back
// with tcgen05.ld by sixteen epilogue warps; a thread then holds one output feature for sixteen
// tokens; a warp turns its 32 x 16 block round in shared memory, so that every lane reads and writes
// 16-byte pieces of token-major rows:
//   EPI_QKV    : RMSNorm scale, RoPE on q and k (the partner dimension sits 16 lanes away), q store,
//                paged-KV append
//   EPI_RESID  : x += D (the residual stream, fp32), the next projection's operand bf16(x * gain) and
//                the sums of x^2 over each group of 32 features that the next RMSNorm needs
//   EPI_SWIGLU : RMSNorm scale, silu(gate) * up (a gate feature and its up feature sit 16 lanes apart)
//   EPI_LMHEAD : RMSNorm scale, optional logits, vocabulary argmax (warp reduction, packed 64-bit atomicMax)
//   EPI_PLAIN  : fp32 store (test hook)
// RMSNorm is split between producer and consumer: the kernel that writes the residual stream
// (EPI_RESID, or prep_kernel for the first layer) stores bf16(x * gain) and partial sums of x^2; the
// projection that consumes it multiplies its accumulators by the token's 1/sqrt(mean(x^2) + eps),
// a per-column scalar in this orientation, which its epilogue warps work out from the partial sums
// while the main loop runs.
#pragma once
#include "ptx.cuh"

namespace syn {

enum { EPI_PLAIN = 0, EPI_QKV = 1, EPI_RESID = 2, EPI_SWIGLU = 3, EPI_LMHEAD = 4 };
enum { GEMM_WAVES = 0, GEMM_KSPLIT = 1, GEMM_RSPLIT = 2 };

struct EpiParams {
    int mode;
    int T;  // valid tokens
    int N;  // valid output features (rows of W)
    // PLAIN
    float* y;
    int ldy;
    // QKV
    op16* q;
    int q_dim, kv_dim, hd, n_kv_heads, page_size;
    const float2* rope;  // [T][hd/2] (cos, sin)
    op16* pool;          // this layer's pool: [page][kvh][K|V][row][hd]
    const int* slot;     // [T] page * page_size + row
    // RMSNorm scale of the token operand (QKV, SWIGLU, LMHEAD; NULL: the operand is used as it is)
    const float* ssq_in; // [T][n_ssq] partial sums of x^2 of the operand's source rows
    int n_ssq;           // a multiple of 4
    float inv_d, eps;
    // RESID
    float* x;            // [T][d] residual stream, updated in place
    const __nv_bfloat16* gain;   // [d] gain of the NEXT RMSNorm
    op16* xg;            // [T][d] half(x * gain): the next projection's operand
    float* ssq_out;      // [T][d / 32]
    int d;
    // SWIGLU
    op16* act;
    int f_pad;
    // LMHEAD
    float* logits;
    int vocab;
    unsigned long long* best;
    uint32_t* warp_max;   // NULL, or [T][n_warp_max]: the ordered bit pattern of the largest logit of every
    int n_warp_max;       // 32-feature group of a token (0 for a group without a valid feature)
};

__device__ __forceinline__ uint32_t orderable_f32(float v) {   // monotone map of a float to unsigned
    uint32_t u = __float_as_uint(v);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ unsigned long long pack_argmax_key(uint32_t key, int idx) {
    return ((unsigned long long)key << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)idx);
}

// Row order inside one packed 128-feature tile.  TMEM lane l of the tile belongs to warp quarter
// q = l / 32; partners that an epilogue combines (the two RoPE halves of a head dimension, a gate
// feature and its up feature) sit 16 lanes apart in the same warp, so they meet by one shuffle.
//   rope tiles (q and k rows): quarter q covers head q / (hd/32) of the tile, dims
//     [16 s, 16 s + 16) for lanes 0..15 and the same dims + hd/2 for lanes 16..31, s = q % (hd/32)
//   gate/up tiles: quarter q lanes 0..15 = gate features 64 b + 16 q + lane, lanes 16..31 = the up
//     features of the same indices (b = tile index)
//   every other tile: feature = tile base + lane
__host__ __device__ __forceinline__ int rope_tile_feature(int l, int hd) {   // offset inside the tile's 128 features
    const int half = hd >> 1, groups = half >> 4, q = l >> 5, ll = l & 31;
    return (q / groups) * hd + 16 * (q % groups) + (ll & 15) + ((ll & 16) ? half : 0);
}

constexpr int GEMM_EPI_WARPS = 16;               // four groups of four (one warp per TMEM lane quarter)

// Epilogue of one 16-token chunk of one warp: a[j] = D[feature of this lane][token t0 + j] (tokens
// j >= ncols are padding), already summed and scaled.  In this orientation a lane holds ONE output
// feature for sixteen tokens, while every output is token-major in memory, so the 32 x 16 block is
// first turned round in a shared-memory scratch of the warp (16 rows of 33 floats: no bank conflicts
// either way).  Afterwards the lanes walk the block row by row: eight neighbouring lanes cover the 32
// columns of one token with four columns each, so that a warp-wide access touches whole 32-byte
// sectors of four tokens' rows (the cost of these epilogues is the number of sectors and of memory
// instructions they issue, not their arithmetic).
// `m0` = first packed row of the tile, `quarter` = warp's TMEM lane quarter.
constexpr int EPI_COLS = 16;
constexpr int EPI_SCR_STRIDE = 33;
constexpr int EPI_SCR_FLOATS = EPI_COLS * EPI_SCR_STRIDE;   // per epilogue warp

__device__ __forceinline__ uint2 pack4_op(float a, float b, float c, float d) { return make_uint2(pack_op(a, b), pack_op(c, d)); }

template <int MODE>
__device__ __forceinline__ void epi_unit(const EpiParams& p, const float (&a)[EPI_COLS], float* scr, int m0, int t0, int ncols,
                                         int quarter, int lane) {
    __syncwarp();   // the previous chunk's rows have been read
#pragma unroll
    for (int j = 0; j < EPI_COLS; ++j) scr[j * EPI_SCR_STRIDE + lane] = a[j];
    __syncwarp();
    const int tq = lane >> 3, c0 = (lane & 7) * 4;   // token (+ 4 i) and first of four columns of this lane
    if (MODE == EPI_PLAIN) {
        const int f = m0 + quarter * 32 + c0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int t = tq + 4 * i;
            const float* row = scr + t * EPI_SCR_STRIDE + c0;
            if (t < ncols) {
                float* dst = p.y + (size_t)(t0 + t) * p.ldy + f;
                if ((p.ldy & 3) == 0 && f + 4 <= p.N) {
                    *reinterpret_cast<float4*>(dst) = make_float4(row[0], row[1], row[2], row[3]);
                } else {
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        if (f + k < p.N) dst[k] = row[k];
                }
            }
        }
    } else if (MODE == EPI_RESID) {
        // x += D; operand of the next projection bf16(x * gain); sum of x^2 over this warp's 32 features
        const int f = m0 + quarter * 32 + c0;
        const uint2 gb = __ldg(reinterpret_cast<const uint2*>(p.gain + f));
        const __nv_bfloat162 g01 = *reinterpret_cast<const __nv_bfloat162*>(&gb.x);
        const __nv_bfloat162 g23 = *reinterpret_cast<const __nv_bfloat162*>(&gb.y);
        float4 xv[4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
            xv[i] = tq + 4 * i < ncols ? *reinterpret_cast<const float4*>(p.x + (size_t)(t0 + tq + 4 * i) * p.d + f)
                                       : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int t = tq + 4 * i;
            const bool tv = t < ncols;
            const float* row = scr + t * EPI_SCR_STRIDE + c0;
            const float4 nx = make_float4(xv[i].x + row[0], xv[i].y + row[1], xv[i].z + row[2], xv[i].w + row[3]);
            float ss = tv ? (nx.x * nx.x + nx.y * nx.y) + (nx.z * nx.z + nx.w * nx.w) : 0.f;
            if (tv) {
                const size_t at = (size_t)(t0 + t) * p.d + f;
                *reinterpret_cast<float4*>(p.x + at) = nx;
                *reinterpret_cast<uint2*>(p.xg + at) = pack4_op(nx.x * __low2float(g01), nx.y * __high2float(g01),
                                                                  nx.z * __low2float(g23), nx.w * __high2float(g23));
            }
            ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 1);   // the eight lanes of the token, a fixed order
            ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 2);
            ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 4);
            if (tv && (lane & 7) == 0) p.ssq_out[(size_t)(t0 + t) * (p.d >> 5) + ((m0 >> 5) + quarter)] = ss;
        }
    } else if (MODE == EPI_QKV) {
        const int which = m0 < p.q_dim ? 0 : (m0 < p.q_dim + p.kv_dim ? 1 : 2);
        const int region0 = which == 0 ? 0 : (which == 1 ? p.q_dim : p.q_dim + p.kv_dim);
        const int half = p.hd >> 1;
        const size_t page_stride = (size_t)p.n_kv_heads * 2 * 16 * p.hd;
        // KV slot (page * 16 + row) of token lane & 15, handed round by shuffles
        const int my_slot = (which > 0 && (lane & 15) < ncols) ? __ldg(p.slot + t0 + (lane & 15)) : 0;
        if (which < 2) {
            // q and k tiles: columns 0..15 of the block are the dims [d0, d0 + 16) of one head, columns 16..31
            // the same dims + hd/2 (rope_tile_feature); a lane rotates its four columns with their partners
            const int groups = half >> 4;
            const int fhead = (m0 - region0) + (quarter / groups) * p.hd;   // first feature of the head, inside q or k
            const bool hi = c0 >= 16;
            const int dim = 16 * (quarter % groups) + (c0 & 15);            // lower dim of the pair
            float4 w[4][2];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float4* cs = reinterpret_cast<const float4*>(p.rope + (size_t)(t0 + tq + 4 * i) * half + dim);   // 4 x (cos, sin)
                const bool tv = tq + 4 * i < ncols;
                w[i][0] = tv ? __ldg(cs) : make_float4(1.f, 0.f, 1.f, 0.f);
                w[i][1] = tv ? __ldg(cs + 1) : make_float4(1.f, 0.f, 1.f, 0.f);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int t = tq + 4 * i;
                const float* mine = scr + t * EPI_SCR_STRIDE + c0;
                const float* part = scr + t * EPI_SCR_STRIDE + (c0 ^ 16);
                const float sg = hi ? 1.f : -1.f;   // dim i: x cos - y sin; dim i + hd/2: y cos + x sin
                const float o0 = mine[0] * w[i][0].x + sg * part[0] * w[i][0].y;
                const float o1 = mine[1] * w[i][0].z + sg * part[1] * w[i][0].w;
                const float o2 = mine[2] * w[i][1].x + sg * part[2] * w[i][1].y;
                const float o3 = mine[3] * w[i][1].z + sg * part[3] * w[i][1].w;
                const int sl = __shfl_sync(0xFFFFFFFFu, my_slot, t);
                if (t < ncols) {
                    op16* dst;
                    if (which == 0) dst = p.q + (size_t)(t0 + t) * p.q_dim + fhead;
                    else dst = p.pool + (size_t)(sl >> 4) * page_stride + ((size_t)(fhead / p.hd) * 2) * 16 * p.hd + (size_t)(sl & 15) * p.hd;
                    *reinterpret_cast<uint2*>(dst + dim + (hi ? half : 0)) = pack4_op(o0, o1, o2, o3);
                }
            }
        } else {
            // v tiles: features in natural order
            const int fr = (m0 - region0) + quarter * 32 + c0;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int t = tq + 4 * i;
                const float* row = scr + t * EPI_SCR_STRIDE + c0;
                const int sl = __shfl_sync(0xFFFFFFFFu, my_slot, t);
                if (t < ncols) {
                    op16* dst = p.pool + (size_t)(sl >> 4) * page_stride + ((size_t)(fr / p.hd) * 2 + 1) * 16 * p.hd +
                                         (size_t)(sl & 15) * p.hd + (fr & (p.hd - 1));
                    *reinterpret_cast<uint2*>(dst) = pack4_op(row[0], row[1], row[2], row[3]);
                }
            }
        }
    } else if (MODE == EPI_SWIGLU) {
        // columns 0..15 of the block hold gate features, columns 16..31 the matching up features: 16
        // outputs per token; four neighbouring lanes cover them, eight tokens per pass
        const int tq8 = lane >> 2, g0 = (lane & 3) * 4;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int t = tq8 + 8 * i;
            const float* row = scr + t * EPI_SCR_STRIDE + g0;
            float h[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) h[k] = __fdividef(row[k], 1.0f + __expf(-row[k])) * row[16 + k];
            if (t < ncols)
                *reinterpret_cast<uint2*>(p.act + (size_t)(t0 + t) * p.f_pad + (m0 >> 1) + 16 * quarter + g0) = pack4_op(h[0], h[1], h[2], h[3]);
        }
    } else {  // EPI_LMHEAD
        const int f = m0 + quarter * 32 + c0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int t = tq + 4 * i;
            const bool tv = t < ncols;
            const float* row = scr + t * EPI_SCR_STRIDE + c0;
            const float v[4] = {row[0], row[1], row[2], row[3]};
            if (p.logits && tv) {
                float* dst = p.logits + (size_t)(t0 + t) * p.vocab + f;
                if ((p.vocab & 3) == 0 && f + 4 <= p.vocab) {
                    *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[1], v[2], v[3]);
                } else {
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        if (f + k < p.vocab) dst[k] = v[k];
                }
            }
            // largest logit of the token among this lane's features, lowest id on ties; then over the
            // token's eight lanes (the packed key orders by logit, then by lower id)
            unsigned long long mine = 0ull;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const unsigned long long key = f + k < p.vocab ? pack_argmax_key(orderable_f32(v[k]), f + k) : 0ull;
                if (key > mine) mine = key;
            }
#pragma unroll
            for (int o = 1; o < 8; o <<= 1) {
                const unsigned long long other = __shfl_xor_sync(0xFFFFFFFFu, mine, o);
                if (other > mine) mine = other;
            }
            if (tv && (lane & 7) == 0) {
                if (mine) atomicMax(p.best + t0 + t, mine);
                // the group's maximum of the token (0: no valid feature): a threshold source for a later top-k
                if (p.warp_max) p.warp_max[(size_t)(t0 + t) * p.n_warp_max + (m0 >> 5) + quarter] = (uint32_t)(mine >> 32);
            }
        }
    }
}

__device__ __forceinline__ void epi_dispatch(int mode, const EpiParams& p, const uint32_t (&r)[EPI_COLS], const float* rs, float* scr,
                                             int m0, int t0, int ncols, int quarter, int lane) {
    float a[EPI_COLS];
#pragma unroll
    for (int j = 0; j < EPI_COLS; ++j) a[j] = __uint_as_float(r[j]);
    if (rs != nullptr) {
#pragma unroll
        for (int j = 0; j < EPI_COLS; ++j) a[j] *= rs[j];
    }
    switch (mode) {
        case EPI_PLAIN: epi_unit<EPI_PLAIN>(p, a, scr, m0, t0, ncols, quarter, lane); break;
        case EPI_QKV: epi_unit<EPI_QKV>(p, a, scr, m0, t0, ncols, quarter, lane); break;
        case EPI_RESID: epi_unit<EPI_RESID>(p, a, scr, m0, t0, ncols, quarter, lane); break;
        case EPI_SWIGLU: epi_unit<EPI_SWIGLU>(p, a, scr, m0, t0, ncols, quarter, lane); break;
        default: epi_unit<EPI_LMHEAD>(p, a, scr, m0, t0, ncols, quarter, lane); break;
    }
}

// RMSNorm scales of the tokens n0 .. n0 + n_valid - 1 from the partial sums of x^2 their source rows
// carry: one warp per token (warp `e` of GEMM_EPI_WARPS takes every sixteenth), a fixed reduction
// order, so every CTA that needs a token's scale gets the same bits.
__device__ __forceinline__ void epi_rms_scales(const EpiParams& p, float* dst, int n0, int n_valid, int e, int lane) {
    const int nq = p.n_ssq >> 2;
    for (int t = e; t < n_valid; t += GEMM_EPI_WARPS) {
        const float4* row = reinterpret_cast<const float4*>(p.ssq_in + (size_t)(n0 + t) * p.n_ssq);
        float sum = 0.f;
        for (int i = lane; i < nq; i += 32) {
            const float4 v = __ldcg(row + i);
            sum += (v.x + v.y) + (v.z + v.w);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
        if (lane == 0) dst[t] = rsqrtf(sum * p.inv_d + p.eps);
    }
}

// ------------------------------------------------------------------------------------------
// Weight packing: row-major sources -> [pair][k-block][2][128 rows x 64 cols], each 16 KB tile
// stored as the 128-byte-swizzled shared-memory image (16-byte chunk c of row r at chunk c ^ (r & 7)).
// mode 0: packed row pr = row pr of the concatenation of up to three matrices.
// mode 1: gate/up: tile b holds gate and up features [64 b, 64 b + 64) in the lane order of
//         epi_unit (quarter q: lanes 0..15 gate 64 b + 16 q + lane, lanes 16..31 the same up rows).
// mode 2: q | k | v concatenation; q and k tiles in the RoPE lane order (rope_tile_feature), v plain.
// ------------------------------------------------------------------------------------------
struct PackSrc {
    const __nv_bfloat16* p[3];
    int rows[3];
    int mode;
    int src_k;   // valid columns of the sources (row pitch)
    int hd;      // mode 2: head dimension
};

__global__ void pack_weight_kernel(PackSrc src, op16* __restrict__ out, int num_kb) {
    const int mtile = blockIdx.x, kb = blockIdx.y;
    op16* tile = out + (((size_t)(mtile >> 1) * num_kb + kb) * 2 + (mtile & 1)) * (128 * 64);
    for (int i = threadIdx.x; i < 128 * 8; i += blockDim.x) {
        const int r = i >> 3, c = i & 7;
        const __nv_bfloat16* row = nullptr;
        if (src.mode == 0) {
            int q = mtile * 128 + r;
            for (int k = 0; k < 3 && !row; ++k) {
                if (q < src.rows[k]) row = src.p[k] + (size_t)q * src.src_k;
                q -= src.rows[k];
            }
        } else if (src.mode == 1) {
            const int sr = mtile * 64 + 16 * (r >> 5) + (r & 15);
            if (sr < src.rows[0]) row = src.p[(r & 16) ? 1 : 0] + (size_t)sr * src.src_k;
        } else {
            int base = mtile * 128, k = 0;   // region of this tile (regions are multiples of 128 rows)
            while (k < 2 && base >= src.rows[k]) base -= src.rows[k++];
            const int q = base + (k < 2 ? rope_tile_feature(r, src.hd) : r);
            if (q < src.rows[k]) row = src.p[k] + (size_t)q * src.src_k;
        }
        uint4 v = make_uint4(0, 0, 0, 0);
        const int col = kb * 64 + c * 8;
        if (row) {
            __nv_bfloat16 tmp[8];
            if (col + 8 <= src.src_k && (((uintptr_t)(row + col)) & 15) == 0) {
                *reinterpret_cast<uint4*>(tmp) = *reinterpret_cast<const uint4*>(row + col);
            } else {
                for (int e = 0; e < 8; ++e) tmp[e] = col + e < src.src_k ? row[col + e] : __float2bfloat16(0.f);
            }
            // bf16 -> half: exact for every weight of magnitude >= 2^-17
            v = make_uint4(pack_op(__bfloat162float(tmp[0]), __bfloat162float(tmp[1])), pack_op(__bfloat162float(tmp[2]), __bfloat162float(tmp[3])),
                           pack_op(__bfloat162float(tmp[4]), __bfloat162float(tmp[5])), pack_op(__bfloat162float(tmp[6]), __bfloat162float(tmp[7])));
        }
        *reinterpret_cast<uint4*>(tile + r * 64 + ((c ^ (r & 7)) << 3)) = v;
    }
}

// ------------------------------------------------------------------------------------------
// The kernel.  One persistent CTA per SM, 576 threads: warp 0 = producer (bulk copy of the weight
// tiles + TMA boxes of the token tile), warp 1 = TMEM owner and MMA issuer, warps 2..17 = epilogue
// (four groups of four; a group covers the four TMEM lane quarters; draining TMEM is limited per
// warp, so many warps share it).
// ------------------------------------------------------------------------------------------
constexpr int GEMM_BK = 64;                        // bf16 elements per k-block = one 128-byte swizzle row
constexpr int GEMM_TILE_BYTES = 128 * GEMM_BK * 2; // 16 KB: one 128-feature tile of one k-block
constexpr int GEMM_A_BYTES = 2 * GEMM_TILE_BYTES;  // stage room for a pair
constexpr int GEMM_BOX_ROWS = 32;                  // token rows per B box
constexpr int GEMM_BOX_BYTES = GEMM_BOX_ROWS * GEMM_BK * 2;
constexpr int GEMM_MAX_STAGES = 8;
constexpr int GEMM_THREADS = (2 + GEMM_EPI_WARPS) * 32;
constexpr int GEMM_SMEM_MAX = 232448;
constexpr int GEMM_BAR_BYTES = 256;                // mbarriers and the TMEM address word

__host__ __device__ inline int gemm_stage_bytes(int TN) { return GEMM_A_BYTES + ((TN + 31) / 32) * GEMM_BOX_BYTES; }
// RMSNorm scales of an item's tokens, two buffers (items alternate); rounded up so that an epilogue
// that takes 32 columns at a time stays inside the buffer
__host__ __device__ inline int gemm_rs_stride(int TN) { return (TN + 31) & ~31; }
__host__ __device__ inline int gemm_scr_offset(int TN) { return GEMM_BAR_BYTES + 2 * gemm_rs_stride(TN) * 4; }   // from the barriers
__host__ inline int gemm_fixed_smem(int TN) { return 1024 /*align*/ + gemm_scr_offset(TN) + GEMM_EPI_WARPS * EPI_SCR_FLOATS * 4; }
__host__ inline int gemm_stages(int TN) {
    int s = (GEMM_SMEM_MAX - gemm_fixed_smem(TN)) / gemm_stage_bytes(TN);
    return s > GEMM_MAX_STAGES ? GEMM_MAX_STAGES : s;
}

struct GemmParams {
    const op16* w;              // packed weights
    int num_kb;                 // k-blocks of 64
    int n_pairs;                // 256-feature pairs
    int n_tt, TN;               // token tiles of TN columns (multiple of 16, <= 256)
    int n_stages;
    int splits, kb_per_split;   // splits > 1 (GEMM_RSPLIT): every CTA owns one (pair tile, k range)
    int pair_mode;              // 1: pair tiles in full waves + remainder as singles; 0: all singles;
                                // 2: one wave of n_cta items, pair tiles first, the rest as singles
    int ksplit;                 // pair mode, > 1: the remainder's pair tiles are cut along K into this many parts
    int kper;                   // ksplit: k-blocks of a helper part, (ksplit - 1) * kper < num_kb
    float* fix_part;            // ksplit: fp32 partial accumulators of the helper parts, [slot][2][TN/16][4][32][16];
                                // splits > 1: the exchange slots of the CTAs, same layout, slot = CTA index
    int* fix_flag;              // ksplit: per remainder tile, epilogue warps of helpers that have stored; then
                                // [n_sm + tile]: owner warps that are done reading (the last one clears both);
                                // splits > 1: the same two counters per pair tile
    int n_sm;
    int* status;
    long long spin_limit;       // SM cycles after which a wait gives up and sets *status
};

struct GemmWork {
    int pair, tt, mt_lo, mt_hi, kb0, kb1, split;
    int role;    // 0: the item's whole K; 1: helper part (accumulators go to fix_part); 2: owner part (adds the helpers')
    int rtile;   // role 1, 2: index of the remainder tile
    int hpart;   // role 1: which helper part
};

// Static schedule: work item i of CTA `cta`.  Returns false when the CTA is done.
// KSPLIT: the kernel variant that cuts the remainder's pair tiles along K (launched only when
// GemmParams::ksplit > 1; the plain variant carries none of that code).
template <bool KSPLIT>
__host__ __device__ __forceinline__ bool gemm_work(const GemmParams& g, int cta, int n_cta, int i, GemmWork& w) {
    const int n_tiles = g.n_pairs * g.n_tt;
    w.split = 0; w.kb0 = 0; w.kb1 = g.num_kb; w.mt_lo = 0; w.mt_hi = 2;
    w.role = 0; w.rtile = 0; w.hpart = 0;
    if (g.splits > 1) {
        if (i > 0 || cta >= n_tiles * g.splits) return false;
        const int tile = cta / g.splits;
        w.split = cta - tile * g.splits;
        w.pair = tile / g.n_tt; w.tt = tile - w.pair * g.n_tt;
        w.kb0 = w.split * g.kb_per_split;
        w.kb1 = w.kb0 + g.kb_per_split < g.num_kb ? w.kb0 + g.kb_per_split : g.num_kb;
        return true;
    }
    if (KSPLIT) {
        // Full waves of pair tiles; the R tiles of the remainder are cut along K into ksplit parts on
        // different CTAs.  The helper parts run FIRST on CTAs 0 .. R (ksplit - 1) - 1, the owner part
        // (the last k range) runs LAST on the last R CTAs and adds the helpers' stored accumulators,
        // which by then have long been written.
        const int fw = n_tiles / n_cta, R = n_tiles - fw * n_cta, H = g.ksplit - 1;
        const int kper = g.kper;   // k-blocks of a helper part; the owner takes the (shorter) rest
        const bool helper = cta < R * H, owner = cta >= n_cta - R;
        int wave = i;
        if (helper) {
            if (i == 0) {
                w.role = 1; w.rtile = cta / H; w.hpart = cta - w.rtile * H;
                const int tile = fw * n_cta + w.rtile;
                w.pair = tile / g.n_tt; w.tt = tile - w.pair * g.n_tt;
                w.kb0 = w.hpart * kper; w.kb1 = w.kb0 + kper;
                return true;
            }
            wave = i - 1;
        }
        if (wave < fw) {
            const int tile = wave * n_cta + cta;
            w.pair = tile / g.n_tt; w.tt = tile - w.pair * g.n_tt;
            return true;
        }
        if (owner && wave == fw) {
            w.role = 2; w.rtile = cta - (n_cta - R);
            const int tile = fw * n_cta + w.rtile;
            w.pair = tile / g.n_tt; w.tt = tile - w.pair * g.n_tt;
            w.kb0 = H * kper; w.kb1 = g.num_kb;
            return true;
        }
        return false;
    }
    if (g.pair_mode == 1) {
        const int fw = n_tiles / n_cta;
        if (i < fw) {
            const int tile = i * n_cta + cta;
            w.pair = tile / g.n_tt; w.tt = tile - w.pair * g.n_tt;
            return true;
        }
        const int r = (i - fw) * n_cta + cta;
        if (r >= (n_tiles - fw * n_cta) * 2) return false;
        const int tile = fw * n_cta + (r >> 1);
        w.pair = tile / g.n_tt; w.tt = tile - w.pair * g.n_tt;
        w.mt_lo = r & 1; w.mt_hi = w.mt_lo + 1;
        return true;
    }
    if (g.pair_mode == 2) {
        // One item per CTA and more single tiles than CTAs: the first 2 n_tiles - n_cta pair tiles stay
        // whole, the others run as two single tiles, so that n_cta CTAs cover everything in one wave.
        if (i > 0) return false;
        const int whole = 2 * n_tiles - n_cta;
        if (cta < whole) {
            w.pair = cta / g.n_tt; w.tt = cta - w.pair * g.n_tt;
            return true;
        }
        const int r = cta - whole, tile = whole + (r >> 1);
        w.pair = tile / g.n_tt; w.tt = tile - w.pair * g.n_tt;
        w.mt_lo = r & 1; w.mt_hi = w.mt_lo + 1;
        return true;
    }
    const int sidx = i * n_cta + cta;
    if (sidx >= n_tiles * 2) return false;
    const int mtile = sidx / g.n_tt;
    w.tt = sidx - mtile * g.n_tt;
    w.pair = mtile >> 1;
    w.mt_lo = mtile & 1; w.mt_hi = w.mt_lo + 1;
    return true;
}

// Every CTA walks its k-blocks from a different starting point (and wraps): at any moment the CTAs
// that share a token tile then ask L2 for different lines of it instead of all for the same ones.
// The schedule is static, so the summation order of a given output is the same in every run.
__device__ __forceinline__ int gemm_k_rotation(int cta, int n_cta, int nk) {
    return (int)(((long long)cta * nk) / n_cta);
}

__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

template <int VARIANT>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmB, GemmParams g, EpiParams p) {
    constexpr bool KSPLIT = VARIANT == GEMM_KSPLIT;
    constexpr bool RSPLIT = VARIANT == GEMM_RSPLIT;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int stage_bytes = gemm_stage_bytes(g.TN);
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + g.n_stages * stage_bytes);
    uint64_t* empty_bar = full_bar + GEMM_MAX_STAGES;
    uint64_t* accf_bar = empty_bar + GEMM_MAX_STAGES;   // accumulators complete (MMA -> epilogue)
    uint64_t* acce_bar = accf_bar + 1;                  // accumulators drained (epilogue -> MMA)
    uint64_t* rs_bar = acce_bar + 1;                    // RMSNorm scales of the item's tokens are in rs_s
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(rs_bar + 1);
    float* rs_s = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(full_bar) + GEMM_BAR_BYTES);   // [2][rs stride]
    float* scr_s = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(full_bar) + gemm_scr_offset(g.TN));   // [epilogue warp][16][33]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_cta = gridDim.x, cta = blockIdx.x;
    const long long limit = g.spin_limit;
    pdl_launch_dependents();
    uint32_t acc_stride = 32;
    while ((int)acc_stride < g.TN) acc_stride <<= 1;
    const uint32_t tmem_cols = 2 * acc_stride;

    if (threadIdx.x == 0) {
        tma_prefetch_desc(&tmB);
        for (int s = 0; s < g.n_stages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        mbar_init(accf_bar, 1);
        mbar_init(acce_bar, GEMM_EPI_WARPS);
        mbar_init(rs_bar, GEMM_EPI_WARPS);
        mbar_fence_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        if (elect_one()) {
            uint32_t it = 0;
            bool ok = true;
            GemmWork w;
            for (int i = 0; ok && gemm_work<KSPLIT>(g, cta, n_cta, i, w); ++i) {
                const int n0 = w.tt * g.TN;
                const int nbox = (((min(g.TN, p.T - n0) + 15) & ~15) + 31) >> 5;
                const uint32_t a_bytes = (uint32_t)(w.mt_hi - w.mt_lo) * GEMM_TILE_BYTES;
                const op16* wsrc = g.w + ((size_t)w.pair * g.num_kb) * (2 * 128 * 64) + (size_t)w.mt_lo * (128 * 64);
                const int nk = w.kb1 - w.kb0, rot = gemm_k_rotation(cta, n_cta, nk);
                // The weights never depend on an earlier kernel: the first item's weight tiles of the
                // whole ring are requested before waiting for the predecessor, whose output is only the
                // token operand.
                const int n_early = i == 0 ? min(nk, g.n_stages) : 0;
                for (int j = 0; j < n_early; ++j) {
                    const int kb = w.kb0 + (j + rot) % nk;
                    uint8_t* a_s = smem + j * stage_bytes;
                    mbar_expect_tx(&full_bar[j], a_bytes + nbox * GEMM_BOX_BYTES);
                    bulk_load(a_s + w.mt_lo * GEMM_TILE_BYTES, wsrc + (size_t)kb * (2 * 128 * 64), a_bytes, &full_bar[j]);
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
                    uint8_t* b_s = a_s + GEMM_A_BYTES;
                    if (j >= n_early) {
                        mbar_expect_tx(&full_bar[s], a_bytes + nbox * GEMM_BOX_BYTES);
                        bulk_load(a_s + w.mt_lo * GEMM_TILE_BYTES, wsrc + (size_t)kb * (2 * 128 * 64), a_bytes, &full_bar[s]);
                    }
                    for (int b = 0; b < nbox; ++b)
                        tma_load_2d(b_s + b * GEMM_BOX_BYTES, &tmB, &full_bar[s], kb * GEMM_BK, n0 + b * GEMM_BOX_ROWS);
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (elect_one()) {
            uint32_t it = 0;
            bool ok = true;
            GemmWork w;
            for (int i = 0; ok && gemm_work<KSPLIT>(g, cta, n_cta, i, w); ++i) {
                const uint32_t nn = (uint32_t)((min(g.TN, p.T - w.tt * g.TN) + 15) & ~15);
                const uint32_t idesc = umma_idesc_f16(128, nn);
                if (i > 0) {   // the epilogue must have drained the previous item's accumulators
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
                    const uint64_t db = umma_desc_k128(a_addr + GEMM_A_BYTES);
                    // consecutive MMAs alternate between the two accumulators: back-to-back MMAs into
                    // one accumulator wait for each other
#pragma unroll
                    for (int k = 0; k < GEMM_BK / 16; ++k)  // 16 bf16 = 32 bytes = 2 descriptor address units
                        for (int mt = w.mt_lo; mt < w.mt_hi; ++mt) {
                            const uint64_t da = umma_desc_k128(a_addr + mt * GEMM_TILE_BYTES);
                            umma_bf16(tmem_base + mt * acc_stride, da + 2 * k, db + 2 * k, idesc, j > 0 || k > 0);
                        }
                    umma_commit(&empty_bar[s]);
                }
                if (ok) umma_commit(accf_bar);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ epilogue
        const int e = warp - 2;
        const int grp = e >> 2;               // the groups take the 16-token chunks round robin
        constexpr int NGRP = GEMM_EPI_WARPS / 4;
        const int quarter = warp & 3;         // TMEM lane quarter this warp may read
        const bool scaled = p.ssq_in != nullptr;
        float* const scr = scr_s + e * EPI_SCR_FLOATS;
        bool ok = true;
        GemmWork w;
        pdl_wait();   // the epilogues read and write buffers of earlier kernels
        for (int i = 0; ok && gemm_work<KSPLIT>(g, cta, n_cta, i, w); ++i) {
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
            const int total_chunks = (w.mt_hi - w.mt_lo) * nchunks;
            if (RSPLIT) {
                // ---- reduce-scatter over the S CTAs that share this tile.  CTA `split` keeps the
                // chunks [c_lo, c_hi) of both 128-feature tiles.  Exchange slot of a CTA:
                // [tile of the pair][chunk][lane quarter][4][lane][4 floats], so that one 16-byte access
                // per lane covers 512 contiguous bytes per warp.
                const int S = g.splits, sp = w.split, tile = cta / S;
                const int cpt = g.TN / EPI_COLS;
                const size_t slot_elems = (size_t)2 * cpt * 128 * EPI_COLS;
                const int c_lo = sp * nchunks / S, c_hi = (sp + 1) * nchunks / S;
                float* const mine = g.fix_part + (size_t)cta * slot_elems;
                int nth = 0;
                for (int mt = 0; mt < 2; ++mt)
                    for (int c = 0; c < nchunks; ++c) {
                        if (c >= c_lo && c < c_hi) continue;
                        if ((nth++ & (NGRP - 1)) != grp) continue;
                        uint32_t r[EPI_COLS];
                        tmem_ld16(tmem_base + mt * acc_stride + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(c * EPI_COLS), r);
                        tmem_ld_wait();
                        uint4* dst = reinterpret_cast<uint4*>(mine + (((size_t)mt * cpt + c) * 4 + quarter) * 32 * EPI_COLS) + lane;
#pragma unroll
                        for (int v = 0; v < EPI_COLS / 4; ++v) dst[v * 32] = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
                    }
                __threadfence();        // this warp's share of the accumulators is in memory
                __syncwarp();
                if (lane == 0) atomicAdd(g.fix_flag + tile, 1);
                // all warps of all S CTAs must have stored before anyone reads; the CTAs of a tile are
                // neighbours in the grid and the grid is at most one CTA per SM, so they run together
                if (lane == 0) {
                    const int want = S * GEMM_EPI_WARPS;
                    const long long t_end = clock64() + limit;
                    while (ld_acquire_gpu(g.fix_flag + tile) < want) {
                        if (clock64() > t_end) {
                            atomicExch(g.status, 1);
                            break;
                        }
                    }
                }
                __syncwarp();
                nth = 0;
                for (int mt = 0; mt < 2; ++mt)
                    for (int c = c_lo; c < c_hi; ++c) {
                        if ((nth++ & (NGRP - 1)) != grp) continue;
                        const int m0 = w.pair * 256 + mt * 128;
                        uint32_t own[EPI_COLS], r[EPI_COLS];
                        tmem_ld16(tmem_base + mt * acc_stride + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(c * EPI_COLS), own);
                        tmem_ld_wait();
                        const size_t at = (((size_t)mt * cpt + c) * 4 + quarter) * 32 * EPI_COLS;
                        for (int q = 0; q < S; ++q) {   // fixed order: the parts in split order
                            if (q == sp) {
#pragma unroll
                                for (int v = 0; v < EPI_COLS; ++v)
                                    r[v] = q == 0 ? own[v] : __float_as_uint(__uint_as_float(r[v]) + __uint_as_float(own[v]));
                            } else {
                                const float4* src = reinterpret_cast<const float4*>(g.fix_part + (size_t)(tile * S + q) * slot_elems + at) + lane;
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
                // the last warp of the tile's CTAs to finish reading clears the counters for the next launch
                __syncwarp();
                if (lane == 0 && atomicAdd(g.fix_flag + g.n_sm + tile, 1) == S * GEMM_EPI_WARPS - 1) {
                    g.fix_flag[tile] = 0;
                    g.fix_flag[g.n_sm + tile] = 0;
                }
                continue;
            }
            if (!KSPLIT || w.role == 0) {
                for (int ci = grp; ci < total_chunks; ci += NGRP) {
                    const int mt = w.mt_lo + ci / nchunks, c = ci % nchunks;
                    const int m0 = w.pair * 256 + mt * 128;
                    uint32_t r[EPI_COLS];
                    tmem_ld16(tmem_base + mt * acc_stride + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(c * EPI_COLS), r);
                    tmem_ld_wait();
                    if (ci + NGRP >= total_chunks) {   // last TMEM read of this warp for this item
                        tc_fence_before();
                        if (lane == 0) mbar_arrive(acce_bar);
                    }
                    const int tc0 = n0 + c * EPI_COLS, ncols = min(EPI_COLS, n_valid - c * EPI_COLS);
                    if (m0 < p.N) epi_dispatch(p.mode, p, r, scaled ? rsi + c * EPI_COLS : nullptr, scr, m0, tc0, ncols, quarter, lane);
                }
                if (grp >= total_chunks) {   // a group without any chunk still releases the accumulators
                    tc_fence_before();
                    if (lane == 0) mbar_arrive(acce_bar);
                }
                continue;
            }
            // ---- a part of a K-split remainder tile.  Stored accumulators:
            // [part][tile of the pair][chunk][lane quarter][4][lane][4 floats], so that one 16-byte access
            // per lane covers 512 contiguous bytes per warp.
            const int H = g.ksplit - 1, cpt = g.TN / EPI_COLS;   // helper parts per tile, chunk slots per tile
            const size_t part_elems = (size_t)2 * cpt * 128 * EPI_COLS;
            if (w.role == 1) {
                float* mine = g.fix_part + (size_t)(w.rtile * H + w.hpart) * part_elems;
                for (int ci = grp; ci < total_chunks; ci += NGRP) {
                    const int mt = w.mt_lo + ci / nchunks, c = ci % nchunks;
                    uint32_t r[EPI_COLS];
                    tmem_ld16(tmem_base + mt * acc_stride + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(c * EPI_COLS), r);
                    tmem_ld_wait();
                    if (ci + NGRP >= total_chunks) {
                        tc_fence_before();
                        if (lane == 0) mbar_arrive(acce_bar);
                    }
                    uint4* dst = reinterpret_cast<uint4*>(mine + (((size_t)mt * cpt + c) * 4 + quarter) * 32 * EPI_COLS) + lane;
#pragma unroll
                    for (int v = 0; v < EPI_COLS / 4; ++v) dst[v * 32] = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
                }
                if (grp >= total_chunks) {
                    tc_fence_before();
                    if (lane == 0) mbar_arrive(acce_bar);
                }
                __threadfence();        // this warp's part of the accumulators is in memory
                __syncwarp();
                if (lane == 0) atomicAdd(g.fix_flag + w.rtile, 1);
                continue;
            }
            // owner: the helpers ran first; the wait is bounded all the same
            if (lane == 0) {
                const int want = H * GEMM_EPI_WARPS;
                const long long t_end = clock64() + limit;
                while (ld_acquire_gpu(g.fix_flag + w.rtile) < want) {
                    if (clock64() > t_end) {
                        atomicExch(g.status, 1);
                        break;
                    }
                }
            }
            __syncwarp();
            for (int ci = grp; ci < total_chunks; ci += NGRP) {
                const int mt = w.mt_lo + ci / nchunks, c = ci % nchunks;
                const int m0 = w.pair * 256 + mt * 128;
                uint32_t r[EPI_COLS];
                tmem_ld16(tmem_base + mt * acc_stride + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(c * EPI_COLS), r);
                tmem_ld_wait();
                if (ci + NGRP >= total_chunks) {
                    tc_fence_before();
                    if (lane == 0) mbar_arrive(acce_bar);
                }
                const size_t at = (((size_t)mt * cpt + c) * 4 + quarter) * 32 * EPI_COLS;
                for (int h = 0; h < H; ++h) {   // fixed order: own k range, then the helpers' in part order
                    const float4* src = reinterpret_cast<const float4*>(g.fix_part + (size_t)(w.rtile * H + h) * part_elems + at) + lane;
#pragma unroll
                    for (int v = 0; v < EPI_COLS / 4; ++v) {
                        const float4 q4 = __ldcg(src + v * 32);
                        r[4 * v] = __float_as_uint(__uint_as_float(r[4 * v]) + q4.x);
                        r[4 * v + 1] = __float_as_uint(__uint_as_float(r[4 * v + 1]) + q4.y);
                        r[4 * v + 2] = __float_as_uint(__uint_as_float(r[4 * v + 2]) + q4.z);
                        r[4 * v + 3] = __float_as_uint(__uint_as_float(r[4 * v + 3]) + q4.w);
                    }
                }
                const int tc0 = n0 + c * EPI_COLS, ncols = min(EPI_COLS, n_valid - c * EPI_COLS);
                if (m0 < p.N) epi_dispatch(p.mode, p, r, scaled ? rsi + c * EPI_COLS : nullptr, scr, m0, tc0, ncols, quarter, lane);
            }
            if (grp >= total_chunks) {
                tc_fence_before();
                if (lane == 0) mbar_arrive(acce_bar);
            }
            // the last warp to finish reading clears the tile's counters for the next launch
            __syncwarp();
            if (lane == 0 && atomicAdd(g.fix_flag + g.n_sm + w.rtile, 1) == GEMM_EPI_WARPS - 1) {
                g.fix_flag[w.rtile] = 0;
                g.fix_flag[g.n_sm + w.rtile] = 0;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, tmem_cols);
    }
}

}  // namespace syn
