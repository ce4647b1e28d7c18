// Microbenchmark: SM cycles per warp-wide ex2.approx, per block of bf16x2 packs, and per pass of the attention
// kernel's softmax inner loop over 32 columns (multiply-add, exp2, sum, pack), with 1, 2 or 4 warps per scheduler.
//   python -m paper_2512_15176_b200.microbench xu_rate
#include <cstdio>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
__device__ __forceinline__ float ex2a(float x) { float y; asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
__device__ __forceinline__ unsigned pack(float a, float b) { unsigned r; asm volatile("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(b), "f"(a)); return r; }
// 2^x on the multiply-add pipe: integer part through the magic-number rounding, 2^f on [-0.5, 0.5] by a degree-4
// polynomial (relative error 2.7e-6), the integer part added to the exponent bits.
__device__ __forceinline__ float ex2_poly(float x) {
    x = fmaxf(x, -126.f);
    const float t = x + 12582912.f;
    const float f = x - (t - 12582912.f);
    float p = fmaf(f, 0.009560510516166687f, 0.05591703951358795f);
    p = fmaf(p, f, 0.24024981260299683f);
    p = fmaf(p, f, 0.6931219696998596f);
    p = fmaf(p, f, 0.9999991655349731f);
    return __int_as_float(__float_as_int(p) + (__float_as_int(t) << 23));
}
template <int MODE>
__global__ void k(float* out, long long* cyc, int iters) {
    float x[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) x[i] = (float)(threadIdx.x + i) * 1e-3f;
    unsigned acc = 0;
    float s = 0.f;
    __syncthreads();
    const long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
        if (MODE == 0) {            // 32 ex2
#pragma unroll
            for (int i = 0; i < 32; ++i) x[i] = ex2a(x[i]);
        } else if (MODE == 1) {     // 16 cvt
#pragma unroll
            for (int i = 0; i < 32; i += 2) acc ^= pack(x[i], x[i + 1]);
#pragma unroll
            for (int i = 0; i < 32; ++i) x[i] += 1.f;
        } else if (MODE == 2) {     // softmax inner loop: 32 fma + 32 ex2 + 32 add + 16 cvt
            float sum4[4] = {0, 0, 0, 0};
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
                const float p0 = ex2a(fmaf(x[i], 0.125f, -s));
                const float p1 = ex2a(fmaf(x[i + 1], 0.125f, -s));
                sum4[(i >> 1) & 3] += p0 + p1;
                acc ^= pack(p0, p1);
            }
            s += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
        } else if (MODE == 4) {     // the softmax loop with every other pair of columns on the multiply-add pipe
            float sum4[4] = {0, 0, 0, 0};
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
                const float a0 = fmaf(x[i], 0.125f, -s), a1 = fmaf(x[i + 1], 0.125f, -s);
                const float p0 = (i & 2) ? ex2_poly(a0) : ex2a(a0);
                const float p1 = (i & 2) ? ex2_poly(a1) : ex2a(a1);
                sum4[(i >> 1) & 3] += p0 + p1;
                acc ^= pack(p0, p1);
            }
            s += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
        } else if (MODE == 5) {     // all columns on the multiply-add pipe
            float sum4[4] = {0, 0, 0, 0};
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
                const float p0 = ex2_poly(fmaf(x[i], 0.125f, -s));
                const float p1 = ex2_poly(fmaf(x[i + 1], 0.125f, -s));
                sum4[(i >> 1) & 3] += p0 + p1;
                acc ^= pack(p0, p1);
            }
            s += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
        } else if (MODE == 3) {     // same, but bf16 by truncation (prmt) instead of cvt
            float sum4[4] = {0, 0, 0, 0};
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
                const float p0 = ex2a(fmaf(x[i], 0.125f, -s));
                const float p1 = ex2a(fmaf(x[i + 1], 0.125f, -s));
                sum4[(i >> 1) & 3] += p0 + p1;
                acc ^= __byte_perm(__float_as_uint(p0), __float_as_uint(p1), 0x7632);
            }
            s += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
        }
    }
    const long long t1 = clock64();
    if (threadIdx.x == 0 && blockIdx.x == 0) *cyc = t1 - t0;
    float r = s + (float)acc;
#pragma unroll
    for (int i = 0; i < 32; ++i) r += x[i];
    out[blockIdx.x * blockDim.x + threadIdx.x] = r;
}
int main() {
    float* out; long long* cyc;
    cudaMalloc(&out, 148 * 1024 * 4); cudaMalloc(&cyc, 8);
    const int iters = 2000;
    for (int warps : {4, 8, 16}) {
        long long h;
        k<0><<<148, warps * 32>>>(out, cyc, iters); cudaDeviceSynchronize(); cudaMemcpy(&h, cyc, 8, cudaMemcpyDeviceToHost);
        printf("warps %2d: ex2      %.2f cycles per warp-instr per SMSP-warp\n", warps, (double)h / iters / 32 / (warps / 4.0));
        k<1><<<148, warps * 32>>>(out, cyc, iters); cudaDeviceSynchronize(); cudaMemcpy(&h, cyc, 8, cudaMemcpyDeviceToHost);
        printf("warps %2d: cvt(+32 fadd) %.2f cycles per 16 cvt + 32 add block per SMSP-warp\n", warps, (double)h / iters / (warps / 4.0));
        k<2><<<148, warps * 32>>>(out, cyc, iters); cudaDeviceSynchronize(); cudaMemcpy(&h, cyc, 8, cudaMemcpyDeviceToHost);
        printf("warps %2d: softmax loop (32 cols, cvt)  %.1f cycles per warp per iteration; per SMSP-warp %.1f\n", warps, (double)h / iters, (double)h / iters / (warps / 4.0));
        k<3><<<148, warps * 32>>>(out, cyc, iters); cudaDeviceSynchronize(); cudaMemcpy(&h, cyc, 8, cudaMemcpyDeviceToHost);
        printf("warps %2d: softmax loop (32 cols, prmt) %.1f cycles per warp per iteration; per SMSP-warp %.1f\n", warps, (double)h / iters, (double)h / iters / (warps / 4.0));
        k<4><<<148, warps * 32>>>(out, cyc, iters); cudaDeviceSynchronize(); cudaMemcpy(&h, cyc, 8, cudaMemcpyDeviceToHost);
        printf("warps %2d: softmax loop (32 cols, half of the exp2 by polynomial) %.1f cycles per warp per iteration; per SMSP-warp %.1f\n", warps, (double)h / iters, (double)h / iters / (warps / 4.0));
        k<5><<<148, warps * 32>>>(out, cyc, iters); cudaDeviceSynchronize(); cudaMemcpy(&h, cyc, 8, cudaMemcpyDeviceToHost);
        printf("warps %2d: softmax loop (32 cols, all exp2 by polynomial) %.1f cycles per warp per iteration; per SMSP-warp %.1f\n", warps, (double)h / iters, (double)h / iters / (warps / 4.0));
    }
    cudaError_t e = cudaDeviceSynchronize();
    printf("%s\n", cudaGetErrorString(e));
    return e != cudaSuccess;
}
