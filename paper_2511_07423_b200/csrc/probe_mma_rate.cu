// Measurement behind the projection kernels' design: the issue rate of tcgen05.mma (kind::f16, 16-bit
// operands resident in shared memory, no loads) for cta_group::1 and cta_group::2, N in {96, 192, 256},
// with 1 / 2 / 4 accumulators taken in turn.  A stand-alone program, not part of the library:
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 -o probe_mma_rate probe_mma_rate.cu && ./probe_mma_rate
// Every wait is bounded; the cluster barrier is reached by every thread unconditionally.
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdio>
#include <cstdint>
#include <cstring>
#include "ptx.cuh"
using namespace syn;

struct Res { long long cycles; int ok; };

// GROUP 1 or 2; n_acc accumulators of N columns each (n_acc * stride <= 512); nsteps k16 steps per accumulator
template <int GROUP>
__global__ void __launch_bounds__(128, 1) bench(int N, int n_acc, int nsteps, Res* out, int* status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    // A: 4 tiles of 128 x 64 bf16 (16 KB each), B: 256 rows x 64 (32 KB); zero filled
    uint64_t* bar = reinterpret_cast<uint64_t*>(smem + 4 * 16384 + 32768);
    uint32_t* slot = reinterpret_cast<uint32_t*>(bar + 2);
    for (int i = threadIdx.x; i < (4 * 16384 + 32768) / 16; i += blockDim.x) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
    const int warp = threadIdx.x >> 5;
    const uint32_t rank = GROUP == 2 ? cluster_ctarank() : 0;
    if (threadIdx.x == 0) { mbar_init(bar, 1); mbar_fence_init(); }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (warp == 1) {
        if (GROUP == 2) { tmem_alloc_pair(slot, 512); tmem_relinquish_pair(); }
        else { tmem_alloc(slot, 512); tmem_relinquish(); }
    }
    tc_fence_before();
    __syncthreads();
    if (GROUP == 2) cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = *slot;
    const int stride = 512 / n_acc;
    long long t0 = 0, t1 = 0;
    bool ok = true;
    if (warp == 0 && rank == 0) {
        if (elect_one()) {
            const uint32_t idesc = umma_idesc_f16(GROUP == 2 ? 256 : 128, N);
            const uint32_t a_addr = smem_u32(smem), b_addr = a_addr + 4 * 16384;
            t0 = clock64();
            for (int k = 0; k < nsteps; ++k)
                for (int a = 0; a < n_acc; ++a) {
                    const uint64_t da = umma_desc_k128(a_addr + (a & 3) * 16384) + 2 * (k & 3);
                    const uint64_t db = umma_desc_k128(b_addr) + 2 * (k & 3);
                    if (GROUP == 2) umma_bf16_pair(tmem_base + a * stride, da, db, idesc, k > 0);
                    else umma_bf16(tmem_base + a * stride, da, db, idesc, k > 0);
                }
            if (GROUP == 2) umma_commit_pair(bar);
            else umma_commit(bar);
        }
        __syncwarp();
    }
    if (warp == 0) {
        if (threadIdx.x == 0) {
            ok = mbar_wait(bar, 0, status, 2000000000LL);
            t1 = clock64();
            if (rank == 0 && blockIdx.x < 2) { out->cycles = t1 - t0; out->ok = ok; }
        }
        __syncwarp();
    }
    tc_fence_before();
    __syncthreads();
    if (GROUP == 2) cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        if (GROUP == 2) tmem_dealloc_pair(tmem_base, 512);
        else tmem_dealloc(tmem_base, 512);
    }
}

template <int GROUP>
static void run(int N, int n_acc, int nsteps, int grid) {
    Res* d; int* st;
    cudaMalloc(&d, sizeof(Res)); cudaMalloc(&st, 4); cudaMemset(d, 0, sizeof(Res)); cudaMemset(st, 0, 4);
    const int smem = 1024 + 4 * 16384 + 32768 + 256;
    cudaFuncSetAttribute(bench<GROUP>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    cudaLaunchConfig_t cfg; memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(128); cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute at[1]; memset(at, 0, sizeof(at));
    at[0].id = cudaLaunchAttributeClusterDimension; at[0].val.clusterDim.x = GROUP; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    Res h = {0, 0};
    for (int rep = 0; rep < 3; ++rep) {
        cudaError_t e = cudaLaunchKernelEx(&cfg, bench<GROUP>, N, n_acc, nsteps, d, st);
        if (e != cudaSuccess) { printf("launch failed: %s\n", cudaGetErrorString(e)); return; }
        e = cudaDeviceSynchronize();
        if (e != cudaSuccess) { printf("sync failed: %s\n", cudaGetErrorString(e)); return; }
        cudaMemcpy(&h, d, sizeof(Res), cudaMemcpyDeviceToHost);
    }
    const double per = (double)h.cycles / ((double)nsteps * n_acc);
    const double ideal = N / 2.0;   // 128 x N x 16 per SM at 8192 FLOP/clk/SM
    printf("group %d grid %3d N %3d acc %d steps %4d : %9lld cycles, %7.1f per MMA (ideal %5.1f, %.0f %%) ok %d\n", GROUP, grid, N, n_acc,
           nsteps, h.cycles, per, ideal, 100.0 * ideal / per, h.ok);
    cudaFree(d); cudaFree(st);
}

int main() {
    for (int grid : {2, 148}) {
        for (int N : {96, 192, 256}) {
            for (int n_acc : {1, 2, 4}) {
                if (N > 512 / n_acc) continue;
                run<1>(N, n_acc, 1024, grid);
                run<2>(N, n_acc, 1024, grid);
            }
        }
    }
    return 0;
}
