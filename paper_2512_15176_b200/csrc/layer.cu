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
// q, k_blk, v_blk are written (v copied as it is); without it q and k_blk are transformed in place.  With `part`
// the packed output does not exist yet: it is the sum of `ksplit` fp32 partial products [ksplit][B k][(Hq + 2 Hkv) D]
// (the projection's contraction was cut into ranges), summed here and rounded to bf16 as the projection would have.
__global__ void __launch_bounds__(128) qk_norm_rope_kernel(deer_kv_desc kv, const int32_t* __restrict__ seq_ids,
                                                           const __nv_bfloat16* __restrict__ qkv, const float* __restrict__ part,
                                                           int ksplit,
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
    const bool packed = qkv != nullptr || part != nullptr;
    if (item >= nq + nk + (packed ? nk : 0)) return;
    const long long part_stride = (long long)B * k * (Hq + 2 * Hkv) * D;
    // element `off` of the packed projection output, as a bf16-rounded float
    auto packed_at = [&](long long off) -> float {
        if (!part) return __bfloat162float(qkv[off]);
        float sum = 0.f;
        for (int s = 0; s < ksplit; ++s) sum += part[(long long)s * part_stride + off];
        return __bfloat162float(__float2bfloat16(sum));
    };
    if (item >= nq + nk) {                                        // a V head: copy out of the packed rows
        const long long r = item - nq - nk;
        const long long bi = r / Hkv;
        const int hh = (int)(r % Hkv);
        const long long src = (bi * (Hq + 2 * Hkv) + Hq + Hkv + hh) * D;
        if (part && D <= 128) {
            // this lane's (up to four) columns of every partial product together, four partial products in flight:
            // one column and one partial product at a time would put their load latencies end to end
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
            for (int s = 0; s < ksplit; ++s) {
                const float* ps = part + (long long)s * part_stride + src;
#pragma unroll
                for (int t = 0; t < 4; ++t)
                    if (lane + 32 * t < D) acc[t] += ps[lane + 32 * t];
            }
#pragma unroll
            for (int t = 0; t < 4; ++t)
                if (lane + 32 * t < D) vb[r * D + lane + 32 * t] = __float2bfloat16(acc[t]);
            return;
        }
        for (int d = lane; d < D; d += 32) vb[r * D + d] = __float2bfloat16(packed_at(src + d));
        return;
    }
    const bool is_q = item < nq;
    const long long r = is_q ? item : item - nq;
    const int H = is_q ? Hq : Hkv;
    const long long bi = r / H;                                   // b * k + i
    const int b = (int)(bi / k), i = (int)(bi % k);
    __nv_bfloat16* v = (is_q ? q : kb) + r * D;
    const long long in_off = (bi * (Hq + 2 * Hkv) + (is_q ? 0 : Hq) + (r % H)) * D;
    const __nv_bfloat16* gamma = is_q ? q_gamma : k_gamma;
    const int s = seq_ids[b];
    const int n = (s >= 0 && s < kv.max_seqs) ? kv.seq_len[s] : 0;
    const float pos = (float)(n + i);
    const int half = D / 2;
    // lane l holds the pairs d = l, l + 32, ... (D <= 128: at most two pairs)
    float a[2], c[2];
    float ss = 0.f;
    if (part) {
        // all of this lane's values at once: up to four columns per partial product, four partial products in flight
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        const bool two = lane + 32 < half;
#pragma unroll 4
        for (int s = 0; s < ksplit; ++s) {
            const float* ps = part + (long long)s * part_stride + in_off;
            if (lane < half) {
                acc[0] += ps[lane];
                acc[1] += ps[lane + half];
            }
            if (two) {
                acc[2] += ps[lane + 32];
                acc[3] += ps[lane + 32 + half];
            }
        }
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            a[t] = __bfloat162float(__float2bfloat16(acc[2 * t]));          // what the projection would have stored
            c[t] = __bfloat162float(__float2bfloat16(acc[2 * t + 1]));
            if (lane + 32 * t < half) ss += a[t] * a[t] + c[t] * c[t];
        }
    } else {
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            const int d = lane + 32 * t;
            a[t] = c[t] = 0.f;
            if (d < half) {
                a[t] = packed ? packed_at(in_off + d) : __bfloat162float(v[d]);
                c[t] = packed ? packed_at(in_off + d + half) : __bfloat162float(v[d + half]);
                ss += a[t] * a[t] + c[t] * c[t];
            }
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

static int qk_norm_rope(deer_kv* kv, const int32_t* seq_ids, const void* qkv, const float* part, int ksplit, void* q, void* k_blk,
                        void* v_blk, const void* q_gamma, const void* k_gamma, int B, int k, int Hq, float eps, float theta,
                        void* stream) {
    DEER_CHECK_ARG(kv && seq_ids && q && k_blk, DEER_ERR_INVALID_ARG, "deer_qk_norm_rope: null argument");
    DEER_CHECK_ARG((q_gamma == nullptr) == (k_gamma == nullptr), DEER_ERR_INVALID_ARG,
                   "deer_qk_norm_rope: q_gamma and k_gamma come together");
    DEER_CHECK_ARG(B >= 0 && k >= 1 && k <= DEER_MAX_BLOCK && Hq > 0 && theta > 1.f && eps >= 0.f, DEER_ERR_INVALID_ARG,
                   "deer_qk_norm_rope: bad sizes");
    if (B == 0) return DEER_OK;
    const int Hkv = kv->d.n_kv_heads, D = kv->d.head_dim;
    const long long items = (long long)B * k * (Hq + Hkv + ((qkv || part) ? Hkv : 0));
    DEER_CUDA(launch_pdl(qk_norm_rope_kernel, dim3((unsigned)((items + 3) / 4)), dim3(128), 0, static_cast<cudaStream_t>(stream), kv->d,
                         seq_ids, static_cast<const __nv_bfloat16*>(qkv), part, ksplit, static_cast<__nv_bfloat16*>(q),
                         static_cast<__nv_bfloat16*>(k_blk), static_cast<__nv_bfloat16*>(v_blk),
                         static_cast<const __nv_bfloat16*>(q_gamma), static_cast<const __nv_bfloat16*>(k_gamma), B, k, Hq, Hkv, D, eps,
                         log2((double)theta)));
    return DEER_OK;
}

extern "C" int deer_qk_norm_rope(deer_kv* kv, const int32_t* seq_ids, void* q, void* k_blk, const void* q_gamma,
                                 const void* k_gamma, int B, int k, int Hq, float eps, float theta, void* stream) {
    return qk_norm_rope(kv, seq_ids, nullptr, nullptr, 1, q, k_blk, nullptr, q_gamma, k_gamma, B, k, Hq, eps, theta, stream);
}

extern "C" int deer_qkv_split_norm_rope(deer_kv* kv, const int32_t* seq_ids, const void* qkv, void* q, void* k_blk, void* v_blk,
                                        const void* q_gamma, const void* k_gamma, int B, int k, int Hq, float eps, float theta,
                                        void* stream) {
    DEER_CHECK_ARG(qkv && v_blk, DEER_ERR_INVALID_ARG, "deer_qkv_split_norm_rope: null argument");
    return qk_norm_rope(kv, seq_ids, qkv, nullptr, 1, q, k_blk, v_blk, q_gamma, k_gamma, B, k, Hq, eps, theta, stream);
}

// ---- a projection and the row-wise step behind it as one call ------------------------------------------------
int deer_linear_for_tail(const void* x, const void* w, const void* residual, void* y_bf16, int M, int K, int N, void* workspace,
                         size_t workspace_bytes, int* ksplit_out, cudaStream_t st);

namespace {

// One block per row: y = sum of the partial products (or the projection's bf16 output) + residual, rounded to bf16;
// then, if gamma is given, y_norm = RMSNorm(y) * gamma over the rounded values (what a separate pass would read).
// A thread takes four neighbouring columns at a time and has the loads of four partial products in flight.
__global__ void __launch_bounds__(1024) residual_norm_tail_kernel(const float* __restrict__ part, int ksplit, const __nv_bfloat16* __restrict__ y_in,
                                                                  const __nv_bfloat16* __restrict__ residual,
                                                                  const __nv_bfloat16* __restrict__ gamma, __nv_bfloat16* __restrict__ y,
                                                                  __nv_bfloat16* __restrict__ y_norm, int M, int N, float eps) {
    __shared__ float red[32];
    pdl_trigger();
    pdl_wait();
    const int T = blockDim.x;
    const size_t row = blockIdx.x;
    const size_t stride = (size_t)M * N;
    const bool vec = (N & 3) == 0;
    float ss = 0.f;
    if (vec) {
        for (int c = threadIdx.x * 4; c < N; c += T * 4) {
            const size_t o = row * N + c;
            float v[4];
            if (part) {
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
                for (int s = 0; s < ksplit; ++s) {
                    const float4 t = __ldg(reinterpret_cast<const float4*>(part + (size_t)s * stride + o));
                    acc.x += t.x;
                    acc.y += t.y;
                    acc.z += t.z;
                    acc.w += t.w;
                }
                v[0] = acc.x; v[1] = acc.y; v[2] = acc.z; v[3] = acc.w;
                if (residual) {
                    const uint2 r = *reinterpret_cast<const uint2*>(residual + o);
                    v[0] += __uint_as_float(r.x << 16);
                    v[1] += __uint_as_float(r.x & 0xffff0000u);
                    v[2] += __uint_as_float(r.y << 16);
                    v[3] += __uint_as_float(r.y & 0xffff0000u);
                }
                uint2 ov;
                ov.x = pack_bf16(v[0], v[1]);
                ov.y = pack_bf16(v[2], v[3]);
                *reinterpret_cast<uint2*>(y + o) = ov;
                v[0] = __uint_as_float(ov.x << 16); v[1] = __uint_as_float(ov.x & 0xffff0000u);
                v[2] = __uint_as_float(ov.y << 16); v[3] = __uint_as_float(ov.y & 0xffff0000u);
            } else {
                const uint2 r = *reinterpret_cast<const uint2*>(y_in + o);      // the projection added the residual itself
                v[0] = __uint_as_float(r.x << 16); v[1] = __uint_as_float(r.x & 0xffff0000u);
                v[2] = __uint_as_float(r.y << 16); v[3] = __uint_as_float(r.y & 0xffff0000u);
            }
            ss += (v[0] * v[0] + v[1] * v[1]) + (v[2] * v[2] + v[3] * v[3]);
        }
    } else {
        for (int c = threadIdx.x; c < N; c += T) {
            const size_t o = row * N + c;
            float v;
            if (part) {
                v = 0.f;
                for (int s = 0; s < ksplit; ++s) v += part[(size_t)s * stride + o];
                if (residual) v += __bfloat162float(residual[o]);
                y[o] = __float2bfloat16(v);
                v = __bfloat162float(y[o]);
            } else {
                v = __bfloat162float(y_in[o]);
            }
            ss += v * v;
        }
    }
    if (!gamma) return;
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
    for (int w = 0; w < (T >> 5); ++w) tot += red[w];
    const float inv = rsqrtf(tot / (float)N + eps);
    const __nv_bfloat16* src = part ? y : y_in;            // this thread wrote its part of y itself a moment ago
    if (vec) {
        for (int c = threadIdx.x * 4; c < N; c += T * 4) {
            const size_t o = row * N + c;
            const uint2 r = *reinterpret_cast<const uint2*>(src + o);
            const uint2 g = *reinterpret_cast<const uint2*>(gamma + c);
            uint2 ov;
            ov.x = pack_bf16(__uint_as_float(r.x << 16) * inv * __uint_as_float(g.x << 16),
                             __uint_as_float(r.x & 0xffff0000u) * inv * __uint_as_float(g.x & 0xffff0000u));
            ov.y = pack_bf16(__uint_as_float(r.y << 16) * inv * __uint_as_float(g.y << 16),
                             __uint_as_float(r.y & 0xffff0000u) * inv * __uint_as_float(g.y & 0xffff0000u));
            *reinterpret_cast<uint2*>(y_norm + o) = ov;
        }
    } else {
        for (int c = threadIdx.x; c < N; c += T)
            y_norm[row * N + c] = __float2bfloat16(__bfloat162float(src[row * N + c]) * inv * __bfloat162float(gamma[c]));
    }
}

}  // namespace

// Threads of a tail block: one per four columns, a whole number of warps, 1024 at most.
static int tail_threads(int N) {
    int t = ((N + 3) / 4 + 31) / 32 * 32;
    return t < 32 ? 32 : (t > 1024 ? 1024 : t);
}

extern "C" size_t deer_layer_workspace_bytes(int M, int K, int N) {
    const size_t a = deer_linear_workspace_bytes(M, K, N), b = (size_t)(M > 0 ? M : 0) * (N > 0 ? N : 0) * 2;
    return a > b ? a : b;
}

extern "C" int deer_linear_qkv_rope(deer_kv* kv, const int32_t* seq_ids, const void* x, const void* w_qkv, void* q, void* k_blk,
                                    void* v_blk, const void* q_gamma, const void* k_gamma, int B, int k, int Hq, int hid, float eps,
                                    float theta, void* workspace, size_t workspace_bytes, void* stream) {
    DEER_CHECK_ARG(kv && seq_ids && x && w_qkv && q && k_blk && v_blk && workspace, DEER_ERR_INVALID_ARG,
                   "deer_linear_qkv_rope: null argument");
    DEER_CHECK_ARG(deer_aligned16(x) && deer_aligned16(w_qkv) && deer_aligned16(workspace), DEER_ERR_INVALID_ARG,
                   "deer_linear_qkv_rope: pointers must be 16-byte aligned");
    DEER_CHECK_ARG(B >= 0 && k >= 1 && k <= DEER_MAX_BLOCK && Hq > 0 && hid > 0 && hid % 64 == 0, DEER_ERR_INVALID_ARG,
                   "deer_linear_qkv_rope: bad sizes");
    if (B == 0) return DEER_OK;
    const int M = B * k, N = (Hq + 2 * kv->d.n_kv_heads) * kv->d.head_dim;
    DEER_CHECK_ARG(workspace_bytes >= deer_layer_workspace_bytes(M, hid, N), DEER_ERR_WORKSPACE,
                   "deer_linear_qkv_rope: workspace of %zu bytes needed, %zu given", deer_layer_workspace_bytes(M, hid, N), workspace_bytes);
    int ksplit = 1;
    // if the contraction is not cut, the packed bf16 output takes the room the partial products would have had
    const size_t lin_bytes = deer_linear_workspace_bytes(M, hid, N);
    int rc = deer_linear_for_tail(x, w_qkv, nullptr, workspace, M, hid, N, lin_bytes ? workspace : nullptr, lin_bytes ? workspace_bytes : 0,
                                  &ksplit, static_cast<cudaStream_t>(stream));
    if (rc != DEER_OK) return rc;
    // either the packed bf16 output or the partial products sit in the workspace now
    return qk_norm_rope(kv, seq_ids, ksplit > 1 ? nullptr : workspace, ksplit > 1 ? static_cast<const float*>(workspace) : nullptr,
                        ksplit, q, k_blk, v_blk, q_gamma, k_gamma, B, k, Hq, eps, theta, stream);
}

extern "C" int deer_linear_residual_norm(const void* x, const void* w, const void* residual, const void* gamma, void* y, void* y_norm,
                                         int M, int K, int N, float eps, void* workspace, size_t workspace_bytes, void* stream) {
    DEER_CHECK_ARG(x && w && y && (!gamma || y_norm), DEER_ERR_INVALID_ARG, "deer_linear_residual_norm: null argument");
    DEER_CHECK_ARG(deer_aligned16(x) && deer_aligned16(w) && deer_aligned16(y) && deer_aligned16(residual) && deer_aligned16(workspace),
                   DEER_ERR_INVALID_ARG, "deer_linear_residual_norm: pointers must be 16-byte aligned");
    DEER_CHECK_ARG(M >= 0 && N >= 16 && K > 0 && K % 64 == 0 && eps >= 0.f, DEER_ERR_INVALID_ARG, "deer_linear_residual_norm: bad sizes");
    if (M == 0) return DEER_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int ksplit = 1;
    int rc = deer_linear_for_tail(x, w, residual, y, M, K, N, workspace, workspace_bytes, &ksplit, st);
    if (rc != DEER_OK) return rc;
    if (ksplit > 1) {
        DEER_CUDA(launch_pdl(residual_norm_tail_kernel, dim3(M), dim3(tail_threads(N)), 0, st, (const float*)workspace, ksplit,
                             (const __nv_bfloat16*)nullptr, static_cast<const __nv_bfloat16*>(residual),
                             static_cast<const __nv_bfloat16*>(gamma), static_cast<__nv_bfloat16*>(y), static_cast<__nv_bfloat16*>(y_norm),
                             M, N, eps));
        return DEER_OK;
    }
    // the contraction was not cut: the projection has written y + residual itself, the tail only normalises
    if (!gamma) return DEER_OK;
    DEER_CUDA(launch_pdl(residual_norm_tail_kernel, dim3(M), dim3(tail_threads(N)), 0, st, (const float*)nullptr, 1, (const __nv_bfloat16*)y,
                         (const __nv_bfloat16*)nullptr, static_cast<const __nv_bfloat16*>(gamma), static_cast<__nv_bfloat16*>(y),
                         static_cast<__nv_bfloat16*>(y_norm), M, N, eps));
    return DEER_OK;
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
