// Projection GEMM of the verification step for sm_100a, "swap-AB" orientation:
//   D[feature][token] = sum_k W[feature][k] * X[token][k]
// The weight matrix is the UMMA A operand (M = 128 output features per CTA, streamed from HBM
// exactly once), the ragged token batch is the UMMA B operand (N = 16..256 tokens), so a batch of
// T tokens pads to a multiple of 16 instead of 128.  Operands are staged by TMA (128-byte swizzle)
// through an mbarrier ring, accumulated by tcgen05.mma in TMEM, read back with tcgen05.ld and
// transposed through shared memory into a token-major tile that the fused epilogues consume:
//   EPI_QKV    : RMSNorm row scale, RoPE on q and k, q store, paged-KV append of k and v
//   EPI_RESID  : residual add into the fp32 stream, next layer's bf16 operand (x * gain), sum x^2
//   EPI_SWIGLU : RMSNorm row scale, silu(gate) * up
//   EPI_LMHEAD : RMSNorm row scale, optional logits, vocabulary argmax (packed 64-bit atomicMax)
//   EPI_PLAIN  : fp32 store (test hook)
// RMSNorm is folded as rmsnorm(x) g W = rstd(x) * ((x g) W): the producer epilogue writes bf16(x g)
// and per-128-feature partial sums of x^2; the consumer reduces them (fixed order) to rstd.
#pragma once
#include "ptx.cuh"

namespace syn {

enum { EPI_PLAIN = 0, EPI_QKV = 1, EPI_RESID = 2, EPI_SWIGLU = 3, EPI_LMHEAD = 4 };

struct EpiParams {
    int mode;
    int T;  // valid tokens
    int N;  // valid output features (rows of W)
    // RMSNorm statistics of the input rows (QKV, SWIGLU, LMHEAD): sumsq_in[tile * t_stride + t]
    const float* sumsq_in;
    int n_sumsq_tiles;
    int t_stride;
    float inv_d, eps;
    // PLAIN
    float* y;
    int ldy;
    // QKV
    __nv_bfloat16* q;
    int q_dim, kv_dim, hd, n_kv_heads, page_size;
    const float2* rope;  // [T][hd/2] (cos, sin)
    __nv_bfloat16* pool; // this layer's pool: [page][kvh][K|V][row][hd]
    const int* slot;     // [T] page * page_size + row
    // RESID
    float* x;
    int d;
    __nv_bfloat16* xn;
    const __nv_bfloat16* gain_next;
    float* sumsq_out;
    // SWIGLU
    __nv_bfloat16* act;
    int f_pad;
    // LMHEAD
    float* logits;
    int vocab;
    unsigned long long* best;
};

__device__ __forceinline__ unsigned long long pack_argmax(float v, int idx) {
    uint32_t u = __float_as_uint(v);
    u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    return ((unsigned long long)u << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)idx);
}

// Consume one staged chunk: stage[c][f] = D[feature m0 + f][token t0 + c], c < 32, f < 128.
// Called by 4 warps (ew = 0..3); warp ew handles tokens c = ew, ew + 4, ...
__device__ __forceinline__ void epi_chunk(const EpiParams& p, const float* __restrict__ stage, int m0, int t0,
                                          int ncols, const float* __restrict__ rstd_s, int rs0, int ew, int lane) {
    const int f0 = m0 + 4 * lane;
    for (int c = ew; c < ncols; c += 4) {
        const int t = t0 + c;
        if (t >= p.T) break;
        float4 v = *reinterpret_cast<const float4*>(stage + c * 128 + 4 * lane);
        float a[4] = {v.x, v.y, v.z, v.w};
        if (p.mode == EPI_PLAIN) {
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (f0 + e < p.N) p.y[(size_t)t * p.ldy + f0 + e] = a[e];
        } else if (p.mode == EPI_QKV) {
            const float r = rstd_s[rs0 + c];
#pragma unroll
            for (int e = 0; e < 4; ++e) a[e] *= r;
            const int which = f0 < p.q_dim ? 0 : (f0 < p.q_dim + p.kv_dim ? 1 : 2);
            if (which < 2) {  // rotate-half RoPE: pair (i, i + hd/2) inside each head
                const int half = p.hd >> 1;
                const int xl = half >> 2;  // partner lane distance (16 for hd 128, 8 for hd 64)
                const int i = (4 * lane) & (p.hd - 1);
                const bool lo = i < half;
                const float2* cs = p.rope + (size_t)t * half + (lo ? i : i - half);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float o = __shfl_xor_sync(0xFFFFFFFFu, a[e], xl);
                    float2 w = cs[e];
                    a[e] = lo ? (a[e] * w.x - o * w.y) : (a[e] * w.x + o * w.y);
                }
            }
            uint2 pk = make_uint2(pack_bf16(a[0], a[1]), pack_bf16(a[2], a[3]));
            if (which == 0) {
                *reinterpret_cast<uint2*>(p.q + (size_t)t * p.q_dim + f0) = pk;
            } else {
                const int fk = f0 - p.q_dim - (which == 2 ? p.kv_dim : 0);
                const int kvh = fk / p.hd, dim = fk - kvh * p.hd;
                const int s = p.slot[t];
                const int page = s / p.page_size, row = s - page * p.page_size;
                size_t off = ((((size_t)page * p.n_kv_heads + kvh) * 2 + (which - 1)) * p.page_size + row) * p.hd + dim;
                *reinterpret_cast<uint2*>(p.pool + off) = pk;
            }
        } else if (p.mode == EPI_RESID) {
            float4 xo = *reinterpret_cast<const float4*>(p.x + (size_t)t * p.d + f0);
            float xv[4] = {xo.x + a[0], xo.y + a[1], xo.z + a[2], xo.w + a[3]};
            *reinterpret_cast<float4*>(p.x + (size_t)t * p.d + f0) = make_float4(xv[0], xv[1], xv[2], xv[3]);
            uint2 gb = *reinterpret_cast<const uint2*>(p.gain_next + f0);
            const __nv_bfloat162 g01 = *reinterpret_cast<__nv_bfloat162*>(&gb.x);
            const __nv_bfloat162 g23 = *reinterpret_cast<__nv_bfloat162*>(&gb.y);
            uint2 pk = make_uint2(pack_bf16(xv[0] * __low2float(g01), xv[1] * __high2float(g01)),
                                  pack_bf16(xv[2] * __low2float(g23), xv[3] * __high2float(g23)));
            *reinterpret_cast<uint2*>(p.xn + (size_t)t * p.d + f0) = pk;
            float ss = xv[0] * xv[0] + xv[1] * xv[1] + xv[2] * xv[2] + xv[3] * xv[3];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
            if (lane == 0) p.sumsq_out[(size_t)(m0 >> 7) * p.t_stride + t] = ss;
        } else if (p.mode == EPI_SWIGLU) {
            const float r = rstd_s[rs0 + c];
            float o[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                a[e] *= r;
                o[e] = __shfl_xor_sync(0xFFFFFFFFu, a[e], 16);  // lanes 0-15: gate, lanes 16-31: up
            }
            if (lane < 16) {
                float h[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) h[e] = a[e] / (1.0f + __expf(-a[e])) * o[e];
                uint2 pk = make_uint2(pack_bf16(h[0], h[1]), pack_bf16(h[2], h[3]));
                *reinterpret_cast<uint2*>(p.act + (size_t)t * p.f_pad + (m0 >> 1) + 4 * lane) = pk;
            }
        } else {  // EPI_LMHEAD
            const float r = rstd_s[rs0 + c];
            float bv = -INFINITY;
            int bi = 0x7FFFFFFF;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                a[e] *= r;
                if (f0 + e < p.vocab && a[e] > bv) { bv = a[e]; bi = f0 + e; }
            }
            if (p.logits) {
                if (f0 + 3 < p.vocab && (((size_t)t * p.vocab + f0) & 3) == 0) {
                    *reinterpret_cast<float4*>(p.logits + (size_t)t * p.vocab + f0) = make_float4(a[0], a[1], a[2], a[3]);
                } else {
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        if (f0 + e < p.vocab) p.logits[(size_t)t * p.vocab + f0 + e] = a[e];
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                float ov = __shfl_xor_sync(0xFFFFFFFFu, bv, o);
                int oi = __shfl_xor_sync(0xFFFFFFFFu, bi, o);
                if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
            }
            if (lane == 0 && bi != 0x7FFFFFFF) atomicMax(p.best + t, pack_argmax(bv, bi));
        }
    }
}

// rstd of the CTA's token tile from the per-feature-tile partial sums, in fixed order.
__device__ __forceinline__ void epi_rstd(const EpiParams& p, float* rstd_s, int n0, int ncols, int tid, int nthr) {
    if (p.mode == EPI_PLAIN || p.mode == EPI_RESID) return;
    for (int i = tid; i < ncols; i += nthr) {
        const int t = n0 + i;
        float s = 0.f;
        if (t < p.T)
            for (int k = 0; k < p.n_sumsq_tiles; ++k) s += p.sumsq_in[(size_t)k * p.t_stride + t];
        rstd_s[i] = rsqrtf(s * p.inv_d + p.eps);
    }
}

// ------------------------------------------------------------------------------------------
// tcgen05 kernel.  grid = (feature tiles of 128, token tiles of TN); 192 threads:
// warp 0 = TMA producer, warp 1 = TMEM owner + MMA issuer, warps 2..5 = epilogue.
// ------------------------------------------------------------------------------------------
constexpr int GEMM_BK = 64;                       // bf16 elements per k-block = one 128-byte swizzle row
constexpr int GEMM_A_BYTES = 128 * GEMM_BK * 2;   // 16 KB
constexpr int GEMM_BOX_ROWS = 32;                 // token rows per B box
constexpr int GEMM_BOX_BYTES = GEMM_BOX_ROWS * GEMM_BK * 2;
constexpr int GEMM_MAX_STAGES = 8;
constexpr int GEMM_THREADS = 192;

__host__ __device__ inline int gemm_stage_bytes(int TN) { return GEMM_A_BYTES + ((TN + 31) / 32) * GEMM_BOX_BYTES; }
__host__ inline int gemm_smem_bytes(int TN, int stages) {
    return 1024 /*align*/ + stages * gemm_stage_bytes(TN) + 2 * 32 * 128 * 4 /*staging*/ + 256 * 4 /*rstd*/ + 256;
}

__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, int K, int TN,
               int n_stages, EpiParams p, int* status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int stage_bytes = gemm_stage_bytes(TN);
    float* staging = reinterpret_cast<float*>(smem + n_stages * stage_bytes);
    float* rstd_s = staging + 2 * 32 * 128;
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(rstd_s + 256);
    uint64_t* empty_bar = full_bar + GEMM_MAX_STAGES;
    uint64_t* accum_bar = empty_bar + GEMM_MAX_STAGES;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(accum_bar + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * 128;
    const int n0 = blockIdx.y * TN;
    const int n_valid = min(TN, p.T - n0);
    const int nn = (n_valid + 15) & ~15;             // UMMA N
    const int nbox = (nn + 31) >> 5;
    const int num_kb = (K + GEMM_BK - 1) / GEMM_BK;
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < TN) tmem_cols <<= 1;

    if (threadIdx.x == 0) {
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        mbar_init(accum_bar, 1);
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
        if (elect_one()) {
            for (int kb = 0; kb < num_kb; ++kb) {
                const int s = kb % n_stages;
                if (kb >= n_stages && !mbar_wait(&empty_bar[s], ((kb / n_stages) - 1) & 1, status)) break;
                uint8_t* a_s = smem + s * stage_bytes;
                uint8_t* b_s = a_s + GEMM_A_BYTES;
                mbar_expect_tx(&full_bar[s], GEMM_A_BYTES + nbox * GEMM_BOX_BYTES);
                tma_load_2d(a_s, &tmA, &full_bar[s], kb * GEMM_BK, m0);
                for (int i = 0; i < nbox; ++i)
                    tma_load_2d(b_s + i * GEMM_BOX_BYTES, &tmB, &full_bar[s], kb * GEMM_BK, n0 + i * GEMM_BOX_ROWS);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (elect_one()) {
            const uint32_t idesc = umma_idesc_bf16(128, (uint32_t)nn);
            bool ok = true;
            for (int kb = 0; kb < num_kb && ok; ++kb) {
                const int s = kb % n_stages;
                ok = mbar_wait(&full_bar[s], (kb / n_stages) & 1, status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_addr = smem_u32(smem + s * stage_bytes);
                const uint64_t da = umma_desc_k128(a_addr);
                const uint64_t db = umma_desc_k128(a_addr + GEMM_A_BYTES);
#pragma unroll
                for (int k = 0; k < GEMM_BK / 16; ++k)  // 16 bf16 = 32 bytes = 2 descriptor address units
                    umma_bf16(tmem_base, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0);
                umma_commit(&empty_bar[s]);
            }
            umma_commit(accum_bar);
        }
        __syncwarp();
    } else {
        const int ew = warp - 2;           // epilogue warp 0..3 (work split)
        const int quarter = warp & 3;      // TMEM lane quarter this warp may read
        const int etid = threadIdx.x - 64;
        epi_rstd(p, rstd_s, n0, n_valid, etid, 128);
        asm volatile("bar.sync 1, 128;" ::: "memory");
        const bool ok = mbar_wait(accum_bar, 0, status);
        tc_fence_after();
        if (ok) {
            const int nchunks = (n_valid + 31) >> 5;
            for (int c = 0; c < nchunks; ++c) {
                uint32_t r[32];
                tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(c * 32), r);
                tmem_ld_wait();
                float* st = staging + (c & 1) * 32 * 128;
#pragma unroll
                for (int j = 0; j < 32; ++j) st[j * 128 + quarter * 32 + lane] = __uint_as_float(r[j]);
                asm volatile("bar.sync 1, 128;" ::: "memory");
                epi_chunk(p, st, m0, n0 + c * 32, min(32, n_valid - c * 32), rstd_s, c * 32, ew, lane);
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

// ------------------------------------------------------------------------------------------
// Cross-check kernel on the legacy warp-MMA path (mma.sync m16n8k16), one 128-feature x 32-token
// tile per CTA, same epilogues.  Kept for bring-up comparisons of the tcgen05 kernel; the step
// does not dispatch to it unless the library is built with SYN_GEMM_LEGACY.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128)
gemm_legacy_kernel(const __nv_bfloat16* __restrict__ W, const __nv_bfloat16* __restrict__ X, int K, int ldw, int ldx,
                   EpiParams p) {
    __shared__ __align__(16) __nv_bfloat16 As[128][40];
    __shared__ __align__(16) __nv_bfloat16 Bs[32][40];
    __shared__ __align__(16) float stage[32 * 128];
    __shared__ float rstd_s[32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, c = lane & 3;
    const int m0 = blockIdx.x * 128, n0 = blockIdx.y * 32;
    const int n_valid = min(32, p.T - n0);
    epi_rstd(p, rstd_s, n0, n_valid, threadIdx.x, 128);
    float acc[2][4][4] = {};
    for (int k0 = 0; k0 < K; k0 += 32) {
        for (int i = threadIdx.x; i < 128 * 32; i += 128) {
            int r = i >> 5, cc = i & 31;
            As[r][cc] = (m0 + r < p.N && k0 + cc < K) ? W[(size_t)(m0 + r) * ldw + k0 + cc] : __float2bfloat16(0.f);
        }
        for (int i = threadIdx.x; i < 32 * 32; i += 128) {
            int r = i >> 5, cc = i & 31;
            Bs[r][cc] = (n0 + r < p.T && k0 + cc < K) ? X[(size_t)(n0 + r) * ldx + k0 + cc] : __float2bfloat16(0.f);
        }
        __syncthreads();
#pragma unroll
        for (int ks = 0; ks < 32; ks += 16) {
            uint32_t a[2][4];
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
                int r = warp * 32 + mt * 16 + g;
                a[mt][0] = *reinterpret_cast<uint32_t*>(&As[r][ks + 2 * c]);
                a[mt][1] = *reinterpret_cast<uint32_t*>(&As[r + 8][ks + 2 * c]);
                a[mt][2] = *reinterpret_cast<uint32_t*>(&As[r][ks + 2 * c + 8]);
                a[mt][3] = *reinterpret_cast<uint32_t*>(&As[r + 8][ks + 2 * c + 8]);
            }
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
                uint32_t b0 = *reinterpret_cast<uint32_t*>(&Bs[nt * 8 + g][ks + 2 * c]);
                uint32_t b1 = *reinterpret_cast<uint32_t*>(&Bs[nt * 8 + g][ks + 2 * c + 8]);
#pragma unroll
                for (int mt = 0; mt < 2; ++mt) mma_bf16_16816(acc[mt][nt], a[mt], b0, b1);
            }
        }
        __syncthreads();
    }
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            int f = warp * 32 + mt * 16 + g, t = nt * 8 + 2 * c;
            stage[t * 128 + f] = acc[mt][nt][0];
            stage[(t + 1) * 128 + f] = acc[mt][nt][1];
            stage[t * 128 + f + 8] = acc[mt][nt][2];
            stage[(t + 1) * 128 + f + 8] = acc[mt][nt][3];
        }
    __syncthreads();
    epi_chunk(p, stage, m0, n0, n_valid, rstd_s, 0, warp, lane);
}

}  // namespace syn
