// Microbenchmark: SM cycles per tcgen05.mma (cta_group::1, M = 128, K = 16, bf16) as a function of N, of where the
// 128-row operand lives (shared memory "SS" or tensor memory "TS") and of the number of issuing threads (one per
// warp, each with its own accumulator), plus the mix the attention kernel issues (two threads S = Q K^T at N = 64
// from shared memory, one thread O += P V at N = 128 with P in tensor memory).  Operands are zeros in shared
// memory; every access is in bounds and the one wait is bounded.  Prints, per issuing thread, the cycles per MMA
// until the last one was accepted ("issue") and until all had completed ("total").
//   python -m paper_2512_15176_b200.microbench mma_rate
#include <cstdio>
#include <cuda_runtime.h>
#include "sm100.cuh"
using namespace sm100;

struct Cfg { int n_mma, N, ts, issuers, mix; };

__global__ void __launch_bounds__(128, 1) rate_kernel(Cfg c, long long* out, int* status) {
    extern __shared__ unsigned char raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    // A: [128 rows][64] bf16 = 16 KB; B: [256 rows][64] bf16 = 32 KB (K-major, SW128)
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 48 * 1024);
    uint32_t* slot = reinterpret_cast<uint32_t*>(bars + 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(slot + 1);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    for (int i = tid; i < 48 * 1024 / 4; i += 128) reinterpret_cast<uint32_t*>(smem)[i] = 0;
    if (tid == 0) {
        for (int i = 0; i < 4; ++i) mbar_init(smem_u32(bars + i), 1);
        *abort_flag = 0;
        mbar_init_fence();
    }
    fence_proxy_async_smem();
    __syncthreads();
    if (warp == 0) tmem_alloc(smem_u32(slot), 512);
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tb = *slot;
    if (warp >= 1 && warp <= c.issuers && lane == 0) {
        int N = c.N, ts = c.ts;
        uint32_t d = tb + 32 + (uint32_t)((warp - 1) * c.N);
        if (c.mix) {                       // the attention kernel's mix: issuers 1, 2: SS N = 64; issuer 3: TS N = 128
            N = (warp == 3) ? 128 : 64;
            ts = (warp == 3);
            d = tb + 32 + (warp == 3 ? 256 : (warp - 1) * 128);
        }
        if (!c.mix && c.N == 256 && !c.ts) d = tb + (uint32_t)((warp - 1) * 256);
        const uint32_t idesc = make_idesc_bf16(N, 0);
        const uint64_t ad = smem_desc_sw128_kmajor(smem_u32(smem));
        const uint64_t bd = smem_desc_sw128_kmajor(smem_u32(smem + 16 * 1024));
        const int n = c.n_mma;
        const long long t0 = clock64();
        for (int i = 0; i < n; ++i) {
            const uint64_t off = (uint64_t)(((i & 3) * 32) >> 4);
            if (ts) umma_bf16_ts(d, tb + (uint32_t)((i & 3) * 8), bd + off, idesc, i != 0);
            else umma_bf16_ss(d, ad + off, bd + off, idesc, i != 0);
        }
        const long long t1 = clock64();
        umma_commit(smem_u32(bars + warp));
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
    if (warp == 0) {
        tcgen05_fence_after();
        tmem_dealloc(tb, 512);
    }
}

int main() {
    long long* out;
    int* status;
    cudaMalloc(&out, 64);
    cudaMalloc(&status, 4);
    cudaMemset(status, 0, 4);
    cudaFuncSetAttribute(rate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
    const Cfg cfgs[] = {
        {4000, 64, 0, 1, 0},  {4000, 64, 0, 2, 0},  {4000, 64, 0, 3, 0},  {4000, 128, 0, 1, 0}, {4000, 128, 0, 2, 0},
        {4000, 128, 0, 3, 0}, {4000, 256, 0, 1, 0}, {4000, 256, 0, 2, 0}, {4000, 64, 1, 1, 0},  {4000, 128, 1, 1, 0},
        {4000, 128, 1, 3, 0}, {4000, 256, 1, 1, 0}, {4000, 0, 0, 3, 1},   {4000, 32, 0, 1, 0},  {4000, 16, 0, 1, 0},
    };
    for (int blocks : {1, 148}) {
        for (const Cfg& c : cfgs) {
            long long h[8] = {0};
            cudaMemset(out, 0, 64);
            rate_kernel<<<blocks, 128, 64 * 1024>>>(c, out, status);
            cudaError_t e = cudaDeviceSynchronize();
            if (e != cudaSuccess) { printf("error %s\n", cudaGetErrorString(e)); return 1; }
            cudaMemcpy(h, out, 64, cudaMemcpyDeviceToHost);
            printf("blocks %3d N %3d %s issuers %d mix %d:", blocks, c.N, c.ts ? "TS" : "SS", c.issuers, c.mix);
            for (int w = 0; w < c.issuers; ++w) printf("  issue %.1f total %.1f cyc/mma", (double)h[2 * w] / c.n_mma, (double)h[2 * w + 1] / c.n_mma);
            printf("\n");
        }
    }
    int hs = 0;
    cudaMemcpy(&hs, status, 4, cudaMemcpyDeviceToHost);
    printf("status %d\n", hs);
    return hs;
}
