// Microbenchmark: SM cycles per tcgen05.mma.cta_group::2 (M = 256 over a CTA pair, K = 16, bf16, operands in shared
// memory) for N in {64, 128, 256} and one or two issuing threads of the leader CTA (separate accumulators): what
// the block-pair LM head's instruction stream costs with nothing else running.  Operands are zeros; every access
// is in bounds and the one wait is bounded.
//   python -m paper_2512_15176_b200.microbench mma_pair_rate
#include <cstdio>
#include <cuda_runtime.h>
#include "sm100.cuh"
using namespace sm100;

struct Cfg { int n_mma, N, issuers; };

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(128, 1) rate_kernel(Cfg c, long long* out, int* status) {
    extern __shared__ unsigned char raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 48 * 1024);
    uint32_t* slot = reinterpret_cast<uint32_t*>(bars + 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(slot + 1);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_ctarank();
    for (int i = tid; i < 48 * 1024 / 4; i += 128) reinterpret_cast<uint32_t*>(smem)[i] = 0;
    if (tid == 0) {
        for (int i = 0; i < 4; ++i) mbar_init(smem_u32(bars + i), 1);
        *abort_flag = 0;
        mbar_init_fence();
    }
    fence_proxy_async_smem();
    __syncthreads();
    if (warp == 0) tmem_alloc_pair(smem_u32(slot), 512);
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync();
    tcgen05_fence_after();
    const uint32_t tb = *slot;
    if (rank == 0 && warp >= 1 && warp <= c.issuers && lane == 0) {
        const uint32_t d = tb + (uint32_t)((warp - 1) * 256);
        const uint32_t idesc = make_idesc_bf16_pair(c.N);
        const uint64_t ad = smem_desc_sw128_kmajor(smem_u32(smem));
        const uint64_t bd = smem_desc_sw128_kmajor(smem_u32(smem + 16 * 1024));
        const long long t0 = clock64();
        for (int i = 0; i < c.n_mma; ++i) {
            const uint64_t off = (uint64_t)(((i & 3) * 32) >> 4);
            umma_bf16_ss_pair(d, ad + off, bd + off, idesc, i != 0);
        }
        const long long t1 = clock64();
        umma_commit_pair(smem_u32(bars + warp), 1);          // arrival in the leader only
        mbar_wait(smem_u32(bars + warp), 0, abort_flag);
        const long long t2 = clock64();
        if (blockIdx.x == 0) {
            out[2 * (warp - 1)] = t1 - t0;
            out[2 * (warp - 1) + 1] = t2 - t0;
        }
        if (*abort_flag) *status = 1;
    }
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync();
    if (warp == 0) {
        tcgen05_fence_after();
        tmem_dealloc_pair(tb, 512);
    }
}

int main() {
    long long* out;
    int* status;
    cudaMalloc(&out, 64);
    cudaMalloc(&status, 4);
    cudaMemset(status, 0, 4);
    cudaFuncSetAttribute(rate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
    const Cfg cfgs[] = {{4000, 256, 1}, {4000, 256, 2}, {4000, 128, 1}, {4000, 128, 2}, {4000, 64, 1}};
    for (int blocks : {2, 148}) {
        for (const Cfg& c : cfgs) {
            long long h[8] = {0};
            cudaMemset(out, 0, 64);
            rate_kernel<<<blocks, 128, 64 * 1024>>>(c, out, status);
            cudaError_t e = cudaDeviceSynchronize();
            if (e != cudaSuccess) { printf("error %s\n", cudaGetErrorString(e)); return 1; }
            cudaMemcpy(h, out, 64, cudaMemcpyDeviceToHost);
            printf("blocks %3d pair N %3d issuers %d:", blocks, c.N, c.issuers);
            for (int w = 0; w < c.issuers; ++w) printf("  issue %.1f total %.1f cyc/mma", (double)h[2 * w] / c.n_mma, (double)h[2 * w + 1] / c.n_mma);
            printf("\n");
        }
    }
    int hs = 0;
    cudaMemcpy(&hs, status, 4, cudaMemcpyDeviceToHost);
    printf("status %d\n", hs);
    return hs;
}
