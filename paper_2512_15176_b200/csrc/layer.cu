// The small row-wise operations of a verifier layer around the block attention:
// RMSNorm, the per-head RMSNorm of q and k followed by the rotary position
// embedding (half-split pairing, positions = committed length + block row), and
// SiLU(gate) * up.  All bf16 in and out with fp32 arithmetic; each is one pass
// over its rows, bound by launch latency at the sizes of a draft block.

#include "common.cuh"

namespace {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// One block per row.
__global__ void __launch_bounds__(256) rmsnorm_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ gamma,
                                                      __nv_bfloat16* __restrict__ y, int hid, float eps) {
    __shared__ float part[8];
    const size_t row = blockIdx.x;
    pdl_trigger();
    pdl_wait();
    const __nv_bfloat16* xr = x + row * hid;
    float ss = 0.f;
    for (int c = threadIdx.x; c < hid; c += 256) {
        const float v = __bfloat162float(xr[c]);
        ss += v * v;
    }
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += part[w];
    const float inv = rsqrtf(tot / (float)hid + eps);
    for (int c = threadIdx.x; c < hid; c += 256)
        y[row * hid + c] = __float2bfloat16(__bfloat162float(xr[c]) * inv * __bfloat162float(gamma[c]));
}

// One warp per (block row, head) of q or k: optional RMSNorm over the head's D values, then the rotation of the
// pairs (d, d + D/2) by pos * theta^(-2d/D).  In place.
// With `qkv` (the packed output [B k][(Hq + 2 Hkv) D] of one fused projection) the values are read from there and
// q, k_blk, v_blk are written (v copied as it is); without it q and k_blk are transformed in place.
__global__ void __launch_bounds__(128) qk_norm_rope_kernel(deer_kv_desc kv, const int32_t* __restrict__ seq_ids,
                                                           const __nv_bfloat16* __restrict__ qkv,
                                                           __nv_bfloat16* __restrict__ q, __nv_bfloat16* __restrict__ kb,
                                                           __nv_bfloat16* __restrict__ vb,
                                                           const __nv_bfloat16* __restrict__ q_gamma,
                                                           const __nv_bfloat16* __restrict__ k_gamma, int B, int k, int Hq, int Hkv,
                                                           int D, float eps, double log2_theta) {
    const int lane = threadIdx.x & 31;
    const long long item = (long long)blockIdx.x * 4 + (threadIdx.x >> 5);
    pdl_trigger();
    pdl_wait();
    const long long nq = (long long)B * k * Hq, nk = (long long)B * k * Hkv;
    if (item >= nq + nk + (qkv ? nk : 0)) return;
    if (item >= nq + nk) {                                        // a V head: copy out of the packed rows
        const long long r = item - nq - nk;
        const long long bi = r / Hkv;
        const int hh = (int)(r % Hkv);
        const __nv_bfloat16* src = qkv + (bi * (Hq + 2 * Hkv) + Hq + Hkv + hh) * D;
        for (int d = lane; d < D; d += 32) vb[r * D + d] = src[d];
        return;
    }
    const bool is_q = item < nq;
    const long long r = is_q ? item : item - nq;
    const int H = is_q ? Hq : Hkv;
    const long long bi = r / H;                                   // b * k + i
    const int b = (int)(bi / k), i = (int)(bi % k);
    __nv_bfloat16* v = (is_q ? q : kb) + r * D;
    const __nv_bfloat16* in = qkv ? qkv + (bi * (Hq + 2 * Hkv) + (is_q ? 0 : Hq) + (r % H)) * D : v;
    const __nv_bfloat16* gamma = is_q ? q_gamma : k_gamma;
    const int s = seq_ids[b];
    const int n = (s >= 0 && s < kv.max_seqs) ? kv.seq_len[s] : 0;
    const float pos = (float)(n + i);
    const int half = D / 2;
    // lane l holds the pairs d = l, l + 32, ... (D <= 128: at most two pairs)
    float a[2], c[2];
    float ss = 0.f;
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        const int d = lane + 32 * t;
        a[t] = c[t] = 0.f;
        if (d < half) {
            a[t] = __bfloat162float(in[d]);
            c[t] = __bfloat162float(in[d + half]);
            ss += a[t] * a[t] + c[t] * c[t];
        }
    }
    float inv = 1.f;
    if (gamma) inv = rsqrtf(warp_sum(ss) / (float)D + eps);
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        const int d = lane + 32 * t;
        if (d < half) {
            float x0 = a[t], x1 = c[t];
            if (gamma) {
                // the normalised values are what the device would store: round them as such before the rotation
                x0 = __bfloat162float(__float2bfloat16(x0 * inv * __bfloat162float(gamma[d])));
                x1 = __bfloat162float(__float2bfloat16(x1 * inv * __bfloat162float(gamma[d + half])));
            }
            // the angle in fp64: at position 30 000 an fp32 frequency alone would be off by hundredths of a radian
            const double ang = (double)pos * exp2(-(double)log2_theta * (2.0 * (double)d / (double)D));
            double sn_d, cs_d;
            sincos(ang, &sn_d, &cs_d);
            const float sn = (float)sn_d, cs = (float)cs_d;
            v[d] = __float2bfloat16(x0 * cs - x1 * sn);
            v[d + half] = __float2bfloat16(x1 * cs + x0 * sn);
        }
    }
}

__global__ void __launch_bounds__(256) swiglu_kernel(const __nv_bfloat16* __restrict__ gu, __nv_bfloat16* __restrict__ y, int I,
                                                     long long total) {
    const long long idx = (long long)blockIdx.x * 256 + threadIdx.x;
    pdl_trigger();
    pdl_wait();
    if (idx >= total) return;
    const long long m = idx / I;
    const int c = (int)(idx % I);
    const float g = __bfloat162float(gu[m * 2 * I + c]), u = __bfloat162float(gu[m * 2 * I + I + c]);
    y[idx] = __float2bfloat16(g / (1.f + __expf(-g)) * u);
}

}  // namespace

extern "C" int deer_rmsnorm(const void* x, const void* gamma, void* y, int M, int hid, float eps, void* stream) {
    DEER_CHECK_ARG(x && gamma && y, DEER_ERR_INVALID_ARG, "deer_rmsnorm: null argument");
    DEER_CHECK_ARG(M >= 0 && hid > 0 && eps >= 0.f, DEER_ERR_INVALID_ARG, "deer_rmsnorm: bad sizes");
    if (M == 0) return DEER_OK;
    DEER_CUDA(launch_pdl(rmsnorm_kernel, dim3(M), dim3(256), 0, static_cast<cudaStream_t>(stream), static_cast<const __nv_bfloat16*>(x),
                         static_cast<const __nv_bfloat16*>(gamma), static_cast<__nv_bfloat16*>(y), hid, eps));
    return DEER_OK;
}

static int qk_norm_rope(deer_kv* kv, const int32_t* seq_ids, const void* qkv, void* q, void* k_blk, void* v_blk, const void* q_gamma,
                        const void* k_gamma, int B, int k, int Hq, float eps, float theta, void* stream) {
    DEER_CHECK_ARG(kv && seq_ids && q && k_blk, DEER_ERR_INVALID_ARG, "deer_qk_norm_rope: null argument");
    DEER_CHECK_ARG((q_gamma == nullptr) == (k_gamma == nullptr), DEER_ERR_INVALID_ARG,
                   "deer_qk_norm_rope: q_gamma and k_gamma come together");
    DEER_CHECK_ARG(B >= 0 && k >= 1 && k <= DEER_MAX_BLOCK && Hq > 0 && theta > 1.f && eps >= 0.f, DEER_ERR_INVALID_ARG,
                   "deer_qk_norm_rope: bad sizes");
    if (B == 0) return DEER_OK;
    const int Hkv = kv->d.n_kv_heads, D = kv->d.head_dim;
    const long long items = (long long)B * k * (Hq + Hkv + (qkv ? Hkv : 0));
    DEER_CUDA(launch_pdl(qk_norm_rope_kernel, dim3((unsigned)((items + 3) / 4)), dim3(128), 0, static_cast<cudaStream_t>(stream), kv->d,
                         seq_ids, static_cast<const __nv_bfloat16*>(qkv), static_cast<__nv_bfloat16*>(q),
                         static_cast<__nv_bfloat16*>(k_blk), static_cast<__nv_bfloat16*>(v_blk),
                         static_cast<const __nv_bfloat16*>(q_gamma), static_cast<const __nv_bfloat16*>(k_gamma), B, k, Hq, Hkv, D, eps,
                         log2((double)theta)));
    return DEER_OK;
}

extern "C" int deer_qk_norm_rope(deer_kv* kv, const int32_t* seq_ids, void* q, void* k_blk, const void* q_gamma,
                                 const void* k_gamma, int B, int k, int Hq, float eps, float theta, void* stream) {
    return qk_norm_rope(kv, seq_ids, nullptr, q, k_blk, nullptr, q_gamma, k_gamma, B, k, Hq, eps, theta, stream);
}

extern "C" int deer_qkv_split_norm_rope(deer_kv* kv, const int32_t* seq_ids, const void* qkv, void* q, void* k_blk, void* v_blk,
                                        const void* q_gamma, const void* k_gamma, int B, int k, int Hq, float eps, float theta,
                                        void* stream) {
    DEER_CHECK_ARG(qkv && v_blk, DEER_ERR_INVALID_ARG, "deer_qkv_split_norm_rope: null argument");
    return qk_norm_rope(kv, seq_ids, qkv, q, k_blk, v_blk, q_gamma, k_gamma, B, k, Hq, eps, theta, stream);
}

extern "C" int deer_swiglu(const void* gate_up, void* y, int M, int I, void* stream) {
    DEER_CHECK_ARG(gate_up && y, DEER_ERR_INVALID_ARG, "deer_swiglu: null argument");
    DEER_CHECK_ARG(M >= 0 && I > 0, DEER_ERR_INVALID_ARG, "deer_swiglu: bad sizes");
    if (M == 0) return DEER_OK;
    const long long total = (long long)M * I;
    DEER_CUDA(launch_pdl(swiglu_kernel, dim3((unsigned)((total + 255) / 256)), dim3(256), 0, static_cast<cudaStream_t>(stream),
                         static_cast<const __nv_bfloat16*>(gate_up), static_cast<__nv_bfloat16*>(y), I, total));
    return DEER_OK;
}
