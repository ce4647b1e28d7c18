// LM-head contraction with fused selection, warp-level mma.sync variant.
// z = h w^T with the vocabulary streamed once per row tile; per-row
// (max, argmax, sum exp) are reduced on the fly so the [M][V] logits never
// need to exist (they are stored only on request).  Used for shapes the
// tcgen05 kernel does not take and as its on-device cross-check.
#pragma once

#include "common.cuh"

namespace lmhead {

constexpr int VT = 128;          // vocabulary rows per tile: 8 warps x 16
constexpr int KT = 64;           // hidden elements per pipeline stage
constexpr int STAGES = 4;
constexpr int THREADS = 256;
constexpr float LOG2E = 1.4426950408889634f;

struct Partial {                 // per (vocabulary part, row): running selection state
    float m;                     // max logit
    int32_t idx;                 // its lowest index
    float s;                     // sum exp((z - m) / T)
    int32_t pad;
};

constexpr int32_t PARTIAL_ABORTED = -2;   // idx written by a block that gave up on a wait

struct Params {
    const __nv_bfloat16* h;      // [M][hid]
    const __nv_bfloat16* w;      // [V][hid]
    int M, hid, V;
    float inv_t_log2;            // log2(e) / T
    const int32_t* draft_ids;    // [M] or null
    float* out_draft_logit;      // [M] or null
    float* out_logits;           // [M][V] or null
    __nv_bfloat16* out_bf16;     // [M][V] or null: plain linear layer, y = h w^T (+ residual), nothing selected
    const __nv_bfloat16* residual;   // [M][V] or null, added before the bf16 rounding
    float* lin_part;             // linear layer: room for max_ksplit partial products [M][V] fp32, or null
    int max_ksplit;
    Partial* part;               // [nparts][M]
    int nparts;
};

__device__ __forceinline__ uint32_t sw_off(int row, int piece) {   // [rows][64] bf16 tile, 128-byte rows
    return static_cast<uint32_t>(row * 128 + ((piece ^ (row & 7)) << 4));
}

__device__ __forceinline__ void merge_sel(float& m, int32_t& idx, float& s, float m2, int32_t idx2, float s2, float inv_t_log2) {
    if (m2 > m || (m2 == m && idx2 < idx)) {
        const float t = m; m = m2; m2 = t;
        const int32_t ti = idx; idx = idx2; idx2 = ti;
        const float ts = s; s = s2; s2 = ts;
    }
    // now (m, idx) is the winner; fold the loser's sum in
    if (s2 > 0.f) s += s2 * exp2f((m2 - m) * inv_t_log2);
}

template <int BM>
__global__ void __launch_bounds__(THREADS, (BM <= 64 ? 2 : 1)) lmhead_mma_kernel(Params p) {
    constexpr int MT = BM / 16;
    constexpr int W_BYTES = VT * KT * 2;
    constexpr int H_BYTES = BM * KT * 2;
    constexpr int STAGE_BYTES = W_BYTES + H_BYTES;
    extern __shared__ __align__(128) unsigned char smem[];
    Partial* red = reinterpret_cast<Partial*>(smem + STAGES * STAGE_BYTES);   // [8 warps][BM]

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g8 = lane >> 2, t4 = lane & 3;
    const int m0 = blockIdx.x * BM;
    const int part = blockIdx.y;
    const int NG = (p.V + 15) / 16;
    const int v0 = (int)((long)part * NG / p.nparts) * 16;
    const int v1 = min(p.V, (int)((long)(part + 1) * NG / p.nparts) * 16);
    const int n_vt = (v1 > v0) ? (v1 - v0 + VT - 1) / VT : 0;
    const int KSTEPS = p.hid / KT;
    const int n_it = n_vt * KSTEPS;

    auto issue = [&](int it) {
        if (it < n_it) {
            const int vt = it / KSTEPS, ks = it % KSTEPS;
            const uint32_t wdst = smem_u32(smem + (it % STAGES) * STAGE_BYTES);
            const uint32_t hdst = wdst + W_BYTES;
            const int vbase = v0 + vt * VT;
#pragma unroll
            for (int r = 0; r < VT * 8 / THREADS; ++r) {
                const int idx = tid + r * THREADS;
                const int row = idx >> 3, pc = idx & 7;
                const int v = vbase + row;
                const bool ok = v < v1;
                cp_async16(wdst + sw_off(row, pc), p.w + (size_t)(ok ? v : 0) * p.hid + ks * KT + pc * 8, ok ? 16 : 0);
            }
#pragma unroll
            for (int r = 0; r < (BM * 8 + THREADS - 1) / THREADS; ++r) {
                const int idx = tid + r * THREADS;
                if (idx < BM * 8) {
                    const int row = idx >> 3, pc = idx & 7;
                    const int m = m0 + row;
                    const bool ok = m < p.M;
                    cp_async16(hdst + sw_off(row, pc), p.h + (size_t)(ok ? m : 0) * p.hid + ks * KT + pc * 8, ok ? 16 : 0);
                }
            }
        }
        cp_async_commit();
    };

    float acc[MT][2][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) acc[mt][nt][0] = acc[mt][nt][1] = acc[mt][nt][2] = acc[mt][nt][3] = 0.f;

    // running selection state of row (m0 + tid), held by threads tid < BM
    float run_m = -INFINITY, run_s = 0.f;
    int32_t run_idx = 0x7fffffff;

#pragma unroll
    for (int st = 0; st < STAGES - 1; ++st) issue(st);

    for (int it = 0; it < n_it; ++it) {
        cp_async_wait<STAGES - 2>();
        __syncthreads();
        issue(it + STAGES - 1);
        const unsigned char* sW = smem + (it % STAGES) * STAGE_BYTES;
        const unsigned char* sH = sW + W_BYTES;
#pragma unroll
        for (int kk = 0; kk < KT / 16; ++kk) {
            uint32_t b0, b1, b2, b3;
            {
                const int row = warp * 16 + (lane & 7) + (lane >> 4) * 8;
                ldmatrix_x4(b0, b1, b2, b3, smem_u32(sW + sw_off(row, kk * 2 + ((lane >> 3) & 1))));
            }
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                uint32_t a[4];
                const int row = mt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
                ldmatrix_x4(a[0], a[1], a[2], a[3], smem_u32(sH + sw_off(row, kk * 2 + (lane >> 4))));
                mma_bf16_16816(acc[mt][0], a, b0, b1);
                mma_bf16_16816(acc[mt][1], a, b2, b3);
            }
        }

        if ((it % KSTEPS) == KSTEPS - 1) {
            // ---- fused selection over this 128-row vocabulary tile ----
            const int vbase = v0 + (it / KSTEPS) * VT + warp * 16;
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int row = mt * 16 + half * 8 + g8;
                    const int m = m0 + row;
                    float bm = -INFINITY;
                    int32_t bi = 0x7fffffff;
                    float vals[4];
#pragma unroll
                    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int v = vbase + nt * 8 + t4 * 2 + e;
                            const float z = acc[mt][nt][half * 2 + e];
                            const bool ok = v < v1;
                            vals[nt * 2 + e] = ok ? z : -INFINITY;
                            if (ok && z > bm) { bm = z; bi = v; }
                        }
                    if (m < p.M) {
                        if (p.out_logits) {
#pragma unroll
                            for (int nt = 0; nt < 2; ++nt) {
                                const int v = vbase + nt * 8 + t4 * 2;
                                float* dst = p.out_logits + (size_t)m * p.V + v;
                                if (v + 1 < v1 && ((p.V & 1) == 0)) {
                                    *reinterpret_cast<float2*>(dst) = make_float2(vals[nt * 2], vals[nt * 2 + 1]);
                                } else {
                                    if (v < v1) dst[0] = vals[nt * 2];
                                    if (v + 1 < v1) dst[1] = vals[nt * 2 + 1];
                                }
                            }
                        }
                        if (p.draft_ids && p.out_draft_logit) {
                            const int dv = p.draft_ids[m];
#pragma unroll
                            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                                for (int e = 0; e < 2; ++e)
                                    if (dv == vbase + nt * 8 + t4 * 2 + e && dv < v1) p.out_draft_logit[m] = vals[nt * 2 + e];
                        }
                    }
                    // max / argmax over the quad (lowest index wins ties)
#pragma unroll
                    for (int o = 1; o <= 2; o <<= 1) {
                        const float om = __shfl_xor_sync(0xffffffffu, bm, o);
                        const int32_t oi = __shfl_xor_sync(0xffffffffu, bi, o);
                        if (om > bm || (om == bm && oi < bi)) { bm = om; bi = oi; }
                    }
                    float sm = 0.f;
                    if (bm > -INFINITY) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) sm += exp2f((vals[j] - bm) * p.inv_t_log2);
                    }
                    sm += __shfl_xor_sync(0xffffffffu, sm, 1);
                    sm += __shfl_xor_sync(0xffffffffu, sm, 2);
                    if (t4 == 0) {
                        Partial pr;
                        pr.m = bm; pr.idx = bi; pr.s = sm; pr.pad = 0;
                        red[warp * BM + row] = pr;
                    }
#pragma unroll
                    for (int nt = 0; nt < 2; ++nt) acc[mt][nt][half * 2] = acc[mt][nt][half * 2 + 1] = 0.f;
                }
            }
            __syncthreads();
            if (tid < BM) {
#pragma unroll
                for (int w8 = 0; w8 < 8; ++w8) {
                    const Partial pr = red[w8 * BM + tid];
                    merge_sel(run_m, run_idx, run_s, pr.m, pr.idx, pr.s, p.inv_t_log2);
                }
            }
            // the next tile's epilogue is at least one __syncthreads away
        }
    }
    cp_async_wait<0>();
    if (tid < BM && m0 + tid < p.M) {
        Partial pr;
        pr.m = run_m; pr.idx = run_idx; pr.s = run_s; pr.pad = 0;
        p.part[(size_t)part * p.M + m0 + tid] = pr;
    }
}

}  // namespace lmhead
