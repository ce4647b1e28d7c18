// Routed mixture-of-experts MLP of a Qwen3-MoE-style verifier layer at the M = B k rows of a draft block: router,
// top-k experts per row, each expert a SiLU-gated MLP, weighted sum (+ residual).
//
// At these row counts the layer is a weight stream: 32 rows x 8 experts already touch most of 128 experts, so
// nearly every expert's matrices cross HBM once per step and each meets only a handful of rows.  The rows are
// therefore regrouped by expert (counting sort of the (row, expert) pairs, rows gathered into that order) and the
// two projections run as grouped GEMMs on the tensor cores: thread block (tile, expert) streams one 256-row tile
// of that expert's weights through a TMA ring against the expert's rows (up to 128 on the TMEM lanes).  The
// gate/up projection pairs 128 gate rows with the 128 up rows of the same channels in one accumulator, so
// SiLU(gate) * up is taken in the epilogue and only the activations are written.
//
// Kernels: router logits (fp32) -> choice (softmax, top-k, renormalise) -> sort (counts, offsets, slots) -> gather ->
// grouped gate/up + SwiGLU -> grouped down -> combine.  All waits are bounded as in the other tensor-core kernels.

#include "sm100.cuh"

namespace {

using namespace sm100;

constexpr int MAX_E = 256;
constexpr int MAX_TOPK = 32;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// ---------------------------------------------------------------- router
// Logits: block (row group of 8, expert group of 8); the rows' hidden states sit in shared memory, warp w takes
// expert 8 * group + w and forms its 8 dot products at once, all of its loads of the expert's row in flight
// together.  Choice: one warp per row -- softmax over the experts, the top_k largest (lowest index among equals),
// weights renormalised to sum 1.
constexpr int RT_ROWS = 8;
constexpr int RT_EXPERTS = 8;

__global__ void __launch_bounds__(256) moe_logits_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ wr,
                                                         int M, int hid, int E, float* __restrict__ logits) {
    extern __shared__ unsigned char smem_raw[];
    __nv_bfloat16* xs = reinterpret_cast<__nv_bfloat16*>(smem_raw);                 // [8][hid]
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int m0 = blockIdx.x * RT_ROWS;
    const int e = blockIdx.y * RT_EXPERTS + warp;
    pdl_trigger();
    pdl_wait();
    const int pieces = hid / 8;
    for (int idx = tid; idx < RT_ROWS * pieces; idx += 256) {
        const int r = idx / pieces, pc = idx % pieces;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (m0 + r < M) v = *reinterpret_cast<const uint4*>(x + (size_t)(m0 + r) * hid + pc * 8);
        *reinterpret_cast<uint4*>(xs + (size_t)r * hid + pc * 8) = v;
    }
    __syncthreads();
    if (e >= E) return;
    float acc[RT_ROWS];
#pragma unroll
    for (int r = 0; r < RT_ROWS; ++r) acc[r] = 0.f;
    for (int pc0 = lane; pc0 < pieces; pc0 += 32 * 4) {
        uint4 wv[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int pc = pc0 + 32 * u;
            wv[u] = pc < pieces ? __ldg(reinterpret_cast<const uint4*>(wr + (size_t)e * hid + pc * 8)) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int pc = pc0 + 32 * u;
            if (pc >= pieces) break;
            const uint32_t ww[4] = {wv[u].x, wv[u].y, wv[u].z, wv[u].w};
#pragma unroll
            for (int r = 0; r < RT_ROWS; ++r) {
                const uint4 xv = *reinterpret_cast<const uint4*>(xs + (size_t)r * hid + pc * 8);
                const uint32_t xw[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    acc[r] = fmaf(__uint_as_float(ww[j] << 16), __uint_as_float(xw[j] << 16), acc[r]);
                    acc[r] = fmaf(__uint_as_float(ww[j] & 0xffff0000u), __uint_as_float(xw[j] & 0xffff0000u), acc[r]);
                }
            }
        }
    }
#pragma unroll
    for (int r = 0; r < RT_ROWS; ++r) {
        const float sum = warp_sum(acc[r]);
        if (lane == 0 && m0 + r < M) logits[(size_t)(m0 + r) * E + e] = sum;
    }
}

__global__ void __launch_bounds__(256) moe_choose_kernel(const float* __restrict__ logits, int M, int E, int top_k, int renorm,
                                                         int32_t* __restrict__ experts, float* __restrict__ weights) {
    const int lane = threadIdx.x & 31;
    const int m = blockIdx.x * 8 + (threadIdx.x >> 5);
    pdl_trigger();
    pdl_wait();
    if (m >= M) return;
    // lane l holds the experts l, l + 32, ...
    constexpr int PER = MAX_E / 32;
    float v[PER];
    float mx = -INFINITY;
#pragma unroll
    for (int j = 0; j < PER; ++j) {
        const int e = lane + 32 * j;
        v[j] = e < E ? logits[(size_t)m * E + e] : -INFINITY;
        mx = fmaxf(mx, v[j]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float sum = 0.f;
#pragma unroll
    for (int j = 0; j < PER; ++j) {
        v[j] = (lane + 32 * j < E) ? expf(v[j] - mx) : -1.f;      // probabilities up to the common factor 1 / sum; -1 = taken / none
        if (v[j] > 0.f) sum += v[j];
    }
    sum = warp_sum(sum);
    float chosen_w = 0.f, tot = 0.f;
    int chosen_e = -1;
    for (int t = 0; t < top_k; ++t) {
        float bv = -1.f;
        int be = 0x7fffffff;
#pragma unroll
        for (int j = 0; j < PER; ++j)
            if (v[j] > bv) {                                     // ascending j = ascending expert index: the first wins
                bv = v[j];
                be = lane + 32 * j;
            }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int oe = __shfl_xor_sync(0xffffffffu, be, o);
            if (ov > bv || (ov == bv && oe < be)) {
                bv = ov;
                be = oe;
            }
        }
        const bool none = be >= E;                               // nothing left to choose from (fewer live experts than top_k, or
                                                                 // probabilities that are not numbers): the choice stays empty
        if (!none) {
#pragma unroll
            for (int j = 0; j < PER; ++j)
                if (lane + 32 * j == be) v[j] = -1.f;            // taken
        }
        if (lane == t) {
            chosen_w = none ? 0.f : bv / sum;
            chosen_e = none ? -1 : be;
        }
        if (!none) tot += bv / sum;
    }
    if (lane < top_k) {
        experts[(size_t)m * top_k + lane] = chosen_e;
        weights[(size_t)m * top_k + lane] = (renorm && tot > 0.f) ? chosen_w / tot : chosen_w;
    }
}

// ---------------------------------------------------------------- regrouping by expert
// One block: counts per expert, exclusive offsets, a slot for every (row, choice) pair.  Which pair of an expert
// gets which of its slots is left to the atomics: no result depends on it.
// A pair whose expert is not one (an empty choice of the router) gets no slot: slot_of = -1, and the slots at the
// end that nobody took are marked with source -1.
__global__ void __launch_bounds__(1024) moe_sort_kernel(const int32_t* __restrict__ experts, int pairs, int top_k, int E,
                                                        int32_t* __restrict__ expert_off, int32_t* __restrict__ slot_src,
                                                        int32_t* __restrict__ slot_of) {
    __shared__ int cnt[MAX_E], off[MAX_E + 1], cur[MAX_E];
    const int tid = threadIdx.x;
    pdl_trigger();
    pdl_wait();
    for (int e = tid; e < E; e += 1024) cnt[e] = cur[e] = 0;
    __syncthreads();
    for (int i = tid; i < pairs; i += 1024) {
        const int e = experts[i];
        if (e >= 0 && e < E) atomicAdd(&cnt[e], 1);
    }
    __syncthreads();
    if (tid == 0) {
        int run = 0;
        for (int e = 0; e < E; ++e) {
            off[e] = run;
            run += cnt[e];
        }
        off[E] = run;
    }
    __syncthreads();
    for (int e = tid; e <= E; e += 1024) expert_off[e] = off[e];
    for (int i = off[E] + tid; i < pairs; i += 1024) slot_src[i] = -1;
    for (int i = tid; i < pairs; i += 1024) {
        const int e = experts[i];
        int slot = -1;
        if (e >= 0 && e < E) {
            slot = off[e] + atomicAdd(&cur[e], 1);
            slot_src[slot] = i / top_k;
        }
        slot_of[i] = slot;
    }
}

// Rows into expert order: xs[slot][:] = x[slot_src[slot]][:].  One block per slot.
__global__ void __launch_bounds__(256) moe_gather_kernel(const __nv_bfloat16* __restrict__ x, const int32_t* __restrict__ slot_src,
                                                         int M, int hid, __nv_bfloat16* __restrict__ xs) {
    pdl_trigger();
    pdl_wait();
    const int slot = blockIdx.x;
    const int src = slot_src[slot];
    const bool ok = src >= 0 && src < M;                          // a slot nobody took reads as zeros
    for (int pc = threadIdx.x; pc < hid / 8; pc += 256)
        *reinterpret_cast<uint4*>(xs + (size_t)slot * hid + pc * 8) =
            ok ? *reinterpret_cast<const uint4*>(x + (size_t)src * hid + pc * 8) : make_uint4(0, 0, 0, 0);
}

// y[m][:] = residual[m][:] + sum_j weights[m][j] * ys[slot_of[m][j]][:].  One block per row.
__global__ void __launch_bounds__(256) moe_combine_kernel(const __nv_bfloat16* __restrict__ ys, const int32_t* __restrict__ slot_of,
                                                          const float* __restrict__ weights, const __nv_bfloat16* __restrict__ residual,
                                                          int hid, int top_k, int pairs, __nv_bfloat16* __restrict__ y) {
    __shared__ int s_slot[MAX_TOPK];
    __shared__ float s_w[MAX_TOPK];
    pdl_trigger();
    pdl_wait();
    const int m = blockIdx.x;
    if (threadIdx.x < top_k) {
        s_slot[threadIdx.x] = slot_of[(size_t)m * top_k + threadIdx.x];
        s_w[threadIdx.x] = weights[(size_t)m * top_k + threadIdx.x];
    }
    __syncthreads();
    for (int pc = threadIdx.x; pc < hid / 8; pc += 256) {
        float acc[8];
        if (residual) {
            const uint4 rv = *reinterpret_cast<const uint4*>(residual + (size_t)m * hid + pc * 8);
            const uint32_t rw[4] = {rv.x, rv.y, rv.z, rv.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                acc[2 * j] = __uint_as_float(rw[j] << 16);
                acc[2 * j + 1] = __uint_as_float(rw[j] & 0xffff0000u);
            }
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[j] = 0.f;
        }
        for (int t = 0; t < top_k; ++t) {
            if (s_slot[t] < 0 || s_slot[t] >= pairs) continue;
            const uint4 v = *reinterpret_cast<const uint4*>(ys + (size_t)s_slot[t] * hid + pc * 8);
            const uint32_t vw[4] = {v.x, v.y, v.z, v.w};
            const float w = s_w[t];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                acc[2 * j] = fmaf(w, __uint_as_float(vw[j] << 16), acc[2 * j]);
                acc[2 * j + 1] = fmaf(w, __uint_as_float(vw[j] & 0xffff0000u), acc[2 * j + 1]);
            }
        }
        uint4 o;
        o.x = pack_bf16(acc[0], acc[1]);
        o.y = pack_bf16(acc[2], acc[3]);
        o.z = pack_bf16(acc[4], acc[5]);
        o.w = pack_bf16(acc[6], acc[7]);
        *reinterpret_cast<uint4*>(y + (size_t)m * hid + pc * 8) = o;
    }
}

// ---------------------------------------------------------------- grouped GEMM on tcgen05
// Thread block (row tile, column tile, expert): out[slot][n] = sum_c xs[slot][c] * w[expert][n][c] for the expert's
// slots [off[e] + 128 * row tile, ...) and one tile of its output columns.
//   SWIGLU: the tile is 128 channels; the accumulator's columns 0..127 are the gate rows of those channels, columns
//           128..255 their up rows (two TMA boxes of 128 weight rows each), and the epilogue writes
//           silu(gate) * up, 128 columns of out.
//   plain:  the tile is 256 output columns (again two boxes of 128 rows).
// Warp roles as in the LM-head kernel: warp 0 = TMA producer, warp 1 = MMA issuer (owns the tensor memory),
// warps 2..5 = epilogue.
constexpr int G_BK = 64;
constexpr int G_A_SPAN = 128 * G_BK * 2;          // bytes an MMA reads for its 128-row operand
constexpr int G_W_BYTES = 256 * G_BK * 2;         // 32 KB: two boxes of 128 weight rows
constexpr int G_THREADS = 192;
constexpr int G_MAX_STAGES = 6;

struct GroupArgs {
    const int32_t* expert_off;     // [E + 1]
    int K;                         // contraction length (multiple of 64)
    int w_rows_per_expert;         // rows of w per expert (2 I for gate/up, hid for down)
    int up_offset;                 // SWIGLU: distance from a gate row to its up row (I)
    int n_out;                     // output columns (I for SWIGLU, hid for plain)
    int n_slots;                   // rows of xs / out
    int x_box_rows;                // rows of xs one TMA box brings
    int a_bytes, stage_bytes, stages;
    __nv_bfloat16* out;            // [slots][n_out]
    int32_t* status;               // optional device word for DEER_ERR_TIMEOUT
};

template <bool SWIGLU>
__global__ void __launch_bounds__(G_THREADS, 1)
moe_grouped_gemm_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w, const GroupArgs a) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + a.stages * a.stage_bytes);
    // bars[0..S) full, [S..2S) empty, [2S] accumulator full        (S = G_MAX_STAGES)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * G_MAX_STAGES + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t smem_base = smem_u32(smem), bar_base = smem_u32(bars);
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (G_MAX_STAGES + s); };
    const uint32_t acc_bar = bar_base + 8u * (2 * G_MAX_STAGES);

    if (tid == 0) {
        for (int s = 0; s < a.stages; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        mbar_init(acc_bar, 1);
        *abort_flag = 0;
        mbar_init_fence();
        prefetch_tensormap(&tm_x);
        prefetch_tensormap(&tm_w);
    }
    pdl_trigger();
    pdl_wait();                                    // the offsets and the gathered rows come from the kernels before
    const int e = blockIdx.z;
    const int m_lo = a.expert_off[e] + (int)blockIdx.x * 128;
    const int rows = min(128, min(a.expert_off[e + 1], a.n_slots) - m_lo);
    if (rows <= 0 || m_lo < 0) return;             // block-uniform: this expert has no (more) rows
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), 256);
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int KB = a.K / G_BK;
    const int n0 = (int)blockIdx.y * (SWIGLU ? 128 : 256);          // first channel / output column of this tile
    const int w_row0 = e * a.w_rows_per_expert + n0;
    const int w_row1 = SWIGLU ? w_row0 + a.up_offset : w_row0 + 128;

    if (warp == 0) {
        if (lane == 0) {
            for (int kb = 0; kb < KB; ++kb) {
                const int s = kb % a.stages;
                const uint32_t ph = (uint32_t)(kb / a.stages) & 1u;
                if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) break;
                mbar_expect_tx(full_bar(s), (uint32_t)(a.a_bytes + G_W_BYTES));
                const uint32_t sa = smem_base + s * a.stage_bytes;
                tma_load_2d(sa + a.a_bytes, &tm_w, kb * G_BK, w_row0, full_bar(s));
                tma_load_2d(sa + a.a_bytes + G_W_BYTES / 2, &tm_w, kb * G_BK, w_row1, full_bar(s));
                tma_load_2d(sa, &tm_x, kb * G_BK, m_lo, full_bar(s));
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = make_idesc_bf16(256, 0);
            bool ok = true;
            for (int kb = 0; kb < KB; ++kb) {
                const int s = kb % a.stages;
                const uint32_t ph = (uint32_t)(kb / a.stages) & 1u;
                if (!mbar_wait(full_bar(s), ph, abort_flag)) { ok = false; break; }
                tcgen05_fence_after();
                const uint32_t sa = smem_base + s * a.stage_bytes;
                const uint64_t ad = smem_desc_sw128_kmajor(sa), bd = smem_desc_sw128_kmajor(sa + a.a_bytes);
#pragma unroll
                for (int k = 0; k < G_BK / 16; ++k) umma_bf16_ss(tmem_base, ad + 2 * k, bd + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
                umma_commit(empty_bar(s));
            }
            if (ok) umma_commit(acc_bar);
        }
    } else {
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const bool row_ok = row < rows;
        const bool got = mbar_wait(acc_bar, 0u, abort_flag);
        if (__all_sync(0xffffffffu, got)) {
            tcgen05_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16);
            __nv_bfloat16* dst_row = a.out + (size_t)(m_lo + (row_ok ? row : 0)) * a.n_out + n0;
            if (SWIGLU) {
                for (int c = 0; c < 128; c += 16) {
                    uint32_t g[16], u[16];
                    TMEM_LD_X16(taddr + c, g);
                    TMEM_LD_X16(taddr + 128 + c, u);
                    tmem_wait_ld();
                    if (row_ok && n0 + c < a.n_out) {
                        float v[16];
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            // the gate and up values as the device would store them: bf16, then the gated product
                            const float gj = __bfloat162float(__float2bfloat16(__uint_as_float(g[j])));
                            const float uj = __bfloat162float(__float2bfloat16(__uint_as_float(u[j])));
                            v[j] = gj / (1.f + __expf(-gj)) * uj;
                        }
                        if (n0 + c + 16 <= a.n_out) {
                            uint4 o0, o1;
                            o0.x = pack_bf16(v[0], v[1]);  o0.y = pack_bf16(v[2], v[3]);   o0.z = pack_bf16(v[4], v[5]);   o0.w = pack_bf16(v[6], v[7]);
                            o1.x = pack_bf16(v[8], v[9]);  o1.y = pack_bf16(v[10], v[11]); o1.z = pack_bf16(v[12], v[13]); o1.w = pack_bf16(v[14], v[15]);
                            *reinterpret_cast<uint4*>(dst_row + c) = o0;
                            *reinterpret_cast<uint4*>(dst_row + c + 8) = o1;
                        } else {
                            for (int j = 0; j < 16 && n0 + c + j < a.n_out; ++j) dst_row[c + j] = __float2bfloat16(v[j]);
                        }
                    }
                }
            } else {
                for (int c = 0; c < 256; c += 16) {
                    uint32_t r[16];
                    TMEM_LD_X16(taddr + c, r);
                    tmem_wait_ld();
                    if (row_ok && n0 + c < a.n_out) {
                        if (n0 + c + 16 <= a.n_out) {
                            uint4 o0, o1;
                            o0.x = pack_bf16(__uint_as_float(r[0]), __uint_as_float(r[1]));   o0.y = pack_bf16(__uint_as_float(r[2]), __uint_as_float(r[3]));
                            o0.z = pack_bf16(__uint_as_float(r[4]), __uint_as_float(r[5]));   o0.w = pack_bf16(__uint_as_float(r[6]), __uint_as_float(r[7]));
                            o1.x = pack_bf16(__uint_as_float(r[8]), __uint_as_float(r[9]));   o1.y = pack_bf16(__uint_as_float(r[10]), __uint_as_float(r[11]));
                            o1.z = pack_bf16(__uint_as_float(r[12]), __uint_as_float(r[13])); o1.w = pack_bf16(__uint_as_float(r[14]), __uint_as_float(r[15]));
                            *reinterpret_cast<uint4*>(dst_row + c) = o0;
                            *reinterpret_cast<uint4*>(dst_row + c + 8) = o1;
                        } else {
                            for (int j = 0; j < 16 && n0 + c + j < a.n_out; ++j) dst_row[c + j] = __float2bfloat16(__uint_as_float(r[j]));
                        }
                    }
                }
            }
        }
    }
    tcgen05_fence_before();
    __syncthreads();
    if (*abort_flag) {
        if (tid == 0) deer_report(a.status, DEER_ERR_TIMEOUT);
        for (int i = 0; i < 64; ++i) __nanosleep(10000);      // copies in flight land before the shared memory goes away
        __syncthreads();
    }
    if (warp == 1) {
        __syncwarp();
        tcgen05_fence_after();
        tmem_dealloc(tmem_base, 256);
    }
}

struct MoeWs {
    int32_t* experts;      // [M][top_k]
    float* weights;        // [M][top_k]
    int32_t* expert_off;   // [E + 1]
    int32_t* slot_src;     // [M top_k]
    int32_t* slot_of;      // [M][top_k]
    int32_t* status;       // [1]
    float* logits;         // [M][E]           router logits
    __nv_bfloat16* xs;     // [M top_k][hid]   rows in expert order
    __nv_bfloat16* act;    // [M top_k][I]
    __nv_bfloat16* ys;     // [M top_k][hid]
    size_t bytes;
};

MoeWs carve(void* base, int M, int hid, int E, int I, int top_k) {
    MoeWs w;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        void* p = base ? static_cast<char*>(base) + off : nullptr;
        off = (off + bytes + 255) / 256 * 256;
        return p;
    };
    const size_t pairs = (size_t)M * top_k;
    w.experts = static_cast<int32_t*>(take(pairs * 4));
    w.weights = static_cast<float*>(take(pairs * 4));
    w.expert_off = static_cast<int32_t*>(take((size_t)(E + 1) * 4));
    w.slot_src = static_cast<int32_t*>(take(pairs * 4));
    w.slot_of = static_cast<int32_t*>(take(pairs * 4));
    w.status = static_cast<int32_t*>(take(4));
    w.logits = static_cast<float*>(take((size_t)M * E * 4));
    w.xs = static_cast<__nv_bfloat16*>(take(pairs * hid * 2));
    w.act = static_cast<__nv_bfloat16*>(take(pairs * I * 2));
    w.ys = static_cast<__nv_bfloat16*>(take(pairs * hid * 2));
    w.bytes = off;
    return w;
}

int make_2d(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    const uint64_t dims[2] = {cols, rows};
    const uint64_t strides[1] = {cols * 2};
    const uint32_t box[2] = {G_BK, box_rows};
    return make_map_bf16(tm, base, 2, dims, strides, box);
}

template <bool SWIGLU>
int launch_grouped(const void* xs, size_t slots, const void* w, int E, int K, int w_rows_per_expert, int up_offset, int n_out,
                   int M, const int32_t* expert_off, __nv_bfloat16* out, int32_t* status, cudaStream_t st) {
    GroupArgs a;
    a.expert_off = expert_off;
    a.K = K;
    a.w_rows_per_expert = w_rows_per_expert;
    a.up_offset = up_offset;
    a.n_out = n_out;
    a.n_slots = (int)slots;
    a.x_box_rows = M >= 128 ? 128 : (M + 7) / 8 * 8;        // an expert never meets more rows than there are
    a.a_bytes = a.x_box_rows * 128;
    a.stage_bytes = a.a_bytes + G_W_BYTES;
    if (a.stage_bytes < G_A_SPAN) a.stage_bytes = G_A_SPAN;
    a.stages = (108 * 1024) / a.stage_bytes;            // two blocks per SM: one streams while the other starts or drains
    if (a.stages > G_MAX_STAGES) a.stages = G_MAX_STAGES;
    a.out = out;
    a.status = status;
    CUtensorMap tm_x, tm_w;
    int rc = make_2d(&tm_x, xs, slots, (uint64_t)K, (uint32_t)a.x_box_rows);
    if (rc != DEER_OK) return rc;
    rc = make_2d(&tm_w, w, (uint64_t)E * w_rows_per_expert, (uint64_t)K, 128);
    if (rc != DEER_OK) return rc;
    const int smem_bytes = a.stages * a.stage_bytes + 1024 + 256;
    const int tile = SWIGLU ? 128 : 256;
    dim3 grid((M + 127) / 128, (n_out + tile - 1) / tile, E);
    DEER_CUDA(cudaFuncSetAttribute(moe_grouped_gemm_kernel<SWIGLU>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes));
    DEER_CUDA(launch_pdl(moe_grouped_gemm_kernel<SWIGLU>, grid, dim3(G_THREADS), (size_t)smem_bytes, st, tm_x, tm_w, a));
    return DEER_OK;
}

int check_shape(int M, int hid, int E, int I, int top_k, const char* who) {
    DEER_CHECK_ARG(M >= 0 && hid > 0 && E > 0 && I > 0 && top_k > 0, DEER_ERR_INVALID_ARG, "%s: bad sizes", who);
    DEER_CHECK_ARG(E <= MAX_E && top_k <= MAX_TOPK && top_k <= E, DEER_ERR_UNSUPPORTED, "%s: at most %d experts, top_k <= min(%d, E)",
                   who, MAX_E, MAX_TOPK);
    DEER_CHECK_ARG(hid % 64 == 0 && I % 64 == 0, DEER_ERR_UNSUPPORTED, "%s: hid and I must be multiples of 64", who);
    DEER_CHECK_ARG((size_t)RT_ROWS * hid * 2 <= 200 * 1024, DEER_ERR_UNSUPPORTED, "%s: hid too large", who);
    return DEER_OK;
}

int route(const void* x, const void* w_router, int M, int hid, int E, int top_k, int renorm, float* logits, int32_t* experts,
          float* weights, cudaStream_t st) {
    const size_t smem = (size_t)RT_ROWS * hid * 2;
    DEER_CUDA(cudaFuncSetAttribute(moe_logits_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    DEER_CUDA(launch_pdl(moe_logits_kernel, dim3((M + RT_ROWS - 1) / RT_ROWS, (E + RT_EXPERTS - 1) / RT_EXPERTS), dim3(256), smem, st,
                         static_cast<const __nv_bfloat16*>(x), static_cast<const __nv_bfloat16*>(w_router), M, hid, E, logits));
    DEER_CUDA(launch_pdl(moe_choose_kernel, dim3((M + 7) / 8), dim3(256), 0, st, (const float*)logits, M, E, top_k, renorm, experts,
                         weights));
    return DEER_OK;
}

}  // namespace

extern "C" size_t deer_moe_workspace_bytes(int M, int hid, int E, int I, int top_k) {
    if (M <= 0 || hid <= 0 || E <= 0 || I <= 0 || top_k <= 0) return 0;
    return carve(nullptr, M, hid, E, I, top_k).bytes;
}

extern "C" int deer_moe_route(const void* x, const void* w_router, int M, int hid, int E, int top_k, int renormalise,
                              int32_t* experts, float* weights, void* workspace, size_t workspace_bytes, void* stream) {
    DEER_CHECK_ARG(x && w_router && experts && weights, DEER_ERR_INVALID_ARG, "deer_moe_route: null argument");
    DEER_CHECK_ARG(workspace && workspace_bytes >= (size_t)(M > 0 ? M : 0) * (E > 0 ? E : 0) * sizeof(float), DEER_ERR_WORKSPACE,
                   "deer_moe_route: the workspace holds the M x E router logits (fp32)");
    DEER_CHECK_ARG(deer_aligned16(x) && deer_aligned16(w_router), DEER_ERR_INVALID_ARG, "deer_moe_route: pointers must be 16-byte aligned");
    const int rc = check_shape(M, hid, E, 64, top_k, "deer_moe_route");
    if (rc != DEER_OK) return rc;
    if (M == 0) return DEER_OK;
    return route(x, w_router, M, hid, E, top_k, renormalise ? 1 : 0, static_cast<float*>(workspace), experts, weights,
                 static_cast<cudaStream_t>(stream));
}

extern "C" int deer_moe_mlp(const void* x, const void* w_router, const void* w_gate_up, const void* w_down, const void* residual,
                            void* y, int M, int hid, int E, int I, int top_k, void* workspace, size_t workspace_bytes, void* stream) {
    DEER_CHECK_ARG(x && w_router && w_gate_up && w_down && y, DEER_ERR_INVALID_ARG, "deer_moe_mlp: null argument");
    DEER_CHECK_ARG(deer_aligned16(x) && deer_aligned16(w_router) && deer_aligned16(w_gate_up) && deer_aligned16(w_down) &&
                       deer_aligned16(residual) && deer_aligned16(y) && deer_aligned16(workspace),
                   DEER_ERR_INVALID_ARG, "deer_moe_mlp: pointers must be 16-byte aligned");
    int rc = check_shape(M, hid, E, I, top_k, "deer_moe_mlp");
    if (rc != DEER_OK) return rc;
    if (M == 0) return DEER_OK;
    const size_t need = deer_moe_workspace_bytes(M, hid, E, I, top_k);
    DEER_CHECK_ARG(workspace && workspace_bytes >= need, DEER_ERR_WORKSPACE, "deer_moe_mlp: workspace of %zu bytes needed, %zu given",
                   need, workspace_bytes);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const MoeWs w = carve(workspace, M, hid, E, I, top_k);
    const int pairs = M * top_k;
    rc = route(x, w_router, M, hid, E, top_k, 1, w.logits, w.experts, w.weights, st);
    if (rc != DEER_OK) return rc;
    DEER_CUDA(launch_pdl(moe_sort_kernel, dim3(1), dim3(1024), 0, st, (const int32_t*)w.experts, pairs, top_k, E, w.expert_off, w.slot_src,
                         w.slot_of));
    DEER_CUDA(launch_pdl(moe_gather_kernel, dim3(pairs), dim3(256), 0, st, static_cast<const __nv_bfloat16*>(x), (const int32_t*)w.slot_src,
                         M, hid, w.xs));
    rc = launch_grouped<true>(w.xs, (size_t)pairs, w_gate_up, E, hid, 2 * I, I, I, M, w.expert_off, w.act, nullptr, st);
    if (rc != DEER_OK) return rc;
    rc = launch_grouped<false>(w.act, (size_t)pairs, w_down, E, I, hid, 0, hid, M, w.expert_off, w.ys, nullptr, st);
    if (rc != DEER_OK) return rc;
    DEER_CUDA(launch_pdl(moe_combine_kernel, dim3(M), dim3(256), 0, st, (const __nv_bfloat16*)w.ys, (const int32_t*)w.slot_of,
                         (const float*)w.weights, static_cast<const __nv_bfloat16*>(residual), hid, top_k, pairs,
                         static_cast<__nv_bfloat16*>(y)));
    return DEER_OK;
}
