// LM-head contraction with fused selection on the 5th-generation tensor cores:
// z = h w^T (Eq. 5's verifier logits) with TMA-staged operands, tcgen05.mma
// accumulating in tensor memory, and an epilogue that reduces every
// accumulator row to (max, argmax, sum exp) without the logits touching HBM
// unless they are asked for.
//
// Tile shape: the block rows of h sit on the 128 TMEM lanes (lanes beyond the
// rows that exist are never read back), the vocabulary on up to 256 accumulator
// columns.  The vocabulary is counted in granules of 16 rows; each thread block
// owns a contiguous range of them (the ranges differ by at most one granule) and
// cuts it into T tiles of g or g - 1 granules (N = 16*g <= 256), so no weight row
// is fetched twice and one TMA box brings a whole N x 64 weight tile.  The operand
// ring is as deep as shared memory allows (7 stages of 30 KB at 32 block rows),
// because the bytes in flight per SM are what cover the HBM latency.  Two
// accumulators (2 x 256 columns) let the epilogue of tile t overlap the MMAs of
// tile t+1.  With more than 128 block rows, pairs of blocks share the weight
// tiles through cta_group::2 MMAs (second kernel below).
//
// Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer (+ TMEM owner),
// warps 2..5 = epilogue (one TMEM lane quarter each).  The blocks that share a
// row tile leave their (max, argmax, sum exp) per row in the workspace; a small
// second kernel, launched so that it is resident before this one ends, merges
// them.  All waits are bounded: a wait that runs out raises the block's abort
// flag, every role leaves its loop, TMEM is freed and the kernel returns; the
// rows of such a block get the id -2 (linear-layer mode: its tiles stay
// unwritten).

#include "lmhead.cuh"
#include "sm100.cuh"

#ifdef DEER_TIMING_PROBES
// Per leader block of the block-pair kernel (row = block index, the first DEER_PROBE_ROWS of them): SM clocks the
// MMA-issuing thread spent in all (0), waiting for operands (1), waiting for an accumulator (2); MMAs issued (3).
__device__ long long g_lmhead_probe[DEER_PROBE_ROWS][DEER_PROBE_COLS];
extern "C" int deer_lmhead_probe_read(long long* host) {
    return (int)cudaMemcpyFromSymbol(host, g_lmhead_probe, sizeof(g_lmhead_probe));
}
#define LM_PROBE_T0(v) const long long v = clock64()
#define LM_PROBE_ADD(acc, v) acc += clock64() - v
#else
#define LM_PROBE_T0(v) \
    do {               \
    } while (0)
#define LM_PROBE_ADD(acc, v) \
    do {                     \
    } while (0)
#endif
namespace lmhead {
namespace umma {

using namespace sm100;

constexpr int BM = 128;
constexpr int BK = 64;                      // 64 bf16 = 128 bytes = one swizzle row
constexpr int MAXN = 256;
constexpr int MAX_STAGES = 8;
constexpr int A_SPAN = BM * BK * 2;         // bytes one MMA reads for its 128-row operand (16 KB)
constexpr int SMEM_BUDGET = 220 * 1024;     // operand ring; barriers and alignment slack come on top
constexpr int SMEM_LIMIT = 227 * 1024;      // dynamic shared memory one block may have
constexpr int THREADS = 192;

struct Args {
    int M, hid, V;
    int h_box_rows;          // rows of h one TMA box brings (<= 128, multiple of 8)
    int a_bytes;             // bytes of the h tile in a stage (h_box_rows * 128, a multiple of 1024)
    int stage_bytes;         // bytes of one stage: h tile + w tile, never less than the 16 KB an MMA reads for h
    int stages;              // pipeline depth
    int gmax;                // granules of the larger tile size (box of tm_w_hi); tm_w_lo has gmax - 1
    int T;                   // tiles per block (fewer only where a block has fewer granules than that)
    int gran;                // 16-row granules of the vocabulary
    int nparts;
    int need_sum;            // 0: argmax only
    int z_tma;               // 1: the logits leave through TMA stores from a staging area behind the operand ring
    float c2;                // log2(e) / T
    const int32_t* draft_ids;
    float* out_draft_logit;
    float* out_logits;
    __nv_bfloat16* out_bf16; // linear-layer mode: the product (+ residual) in bf16 is all that is written
    const __nv_bfloat16* residual;
    int swiglu;              // linear-layer mode: columns come in (gate, up) pairs; out_bf16 [M][V / 2] gets silu(gate) * up
    int ksplit;              // linear-layer mode, few output columns: the contraction is cut into ksplit ranges, one per
    float* lin_part;         // blockIdx.y / nparts; the partial sums go to lin_part[ksplit][M][V] (fp32) and are added up after
    Partial* part;           // [nparts][M]
};

// One 16-column slice of an accumulator row: optional store, draft-token pick, running selection.
__device__ __forceinline__ void consume16(const uint32_t (&r)[16], int vbase, int V, bool row_ok, const Args& a, size_t zrow,
                                          int draft, int grow, bool store, float& run_m, int32_t& run_i, float& run_s) {
    if (!row_ok || vbase >= V) return;
    const int nv = min(16, V - vbase);
    float v[16];
    if (a.out_bf16 && a.ksplit > 1) {
        // partial sum over this block's range of the contraction: plain fp32 stores of the rows that exist
        float* dst = a.lin_part + ((size_t)(blockIdx.y / a.nparts) * a.M * a.V) + zrow + vbase;
        if (nv == 16 && ((zrow + vbase) & 3) == 0) {
#pragma unroll
            for (int j = 0; j < 16; j += 4)
                *reinterpret_cast<float4*>(dst + j) = make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]),
                                                                  __uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
        } else {
#pragma unroll
            for (int j = 0; j < 16; ++j)
                if (j < nv) dst[j] = __uint_as_float(r[j]);
        }
        return;
    }
    if (a.out_bf16 && a.swiglu) {
        // gate / up interleaved: 16 columns = 8 (gate, up) pairs -> 8 activations = 16 contiguous bytes of the row;
        // gate and up are rounded to bf16 first, as a layer that stores them would
        __nv_bfloat16* dst = a.out_bf16 + (zrow + vbase) / 2;
        float o[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float g = __bfloat162float(__float2bfloat16(__uint_as_float(r[2 * j])));
            const float u = __bfloat162float(__float2bfloat16(__uint_as_float(r[2 * j + 1])));
            o[j] = g / (1.f + __expf(-g)) * u;
        }
        if (nv == 16 && (((zrow + vbase) / 2) & 7) == 0) {
            uint4 ov;
            ov.x = pack_bf16(o[0], o[1]);
            ov.y = pack_bf16(o[2], o[3]);
            ov.z = pack_bf16(o[4], o[5]);
            ov.w = pack_bf16(o[6], o[7]);
            *reinterpret_cast<uint4*>(dst) = ov;
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j)
                if (2 * j + 1 < nv) dst[j] = __float2bfloat16(o[j]);
        }
        return;
    }
    if (a.out_bf16) {
        // linear layer: y = acc (+ residual), rounded to bf16; 16 columns = 32 contiguous bytes of the row
        __nv_bfloat16* dst = a.out_bf16 + zrow + vbase;
        const __nv_bfloat16* res = a.residual ? a.residual + zrow + vbase : nullptr;
#pragma unroll
        for (int j = 0; j < 16; ++j) v[j] = __uint_as_float(r[j]);
        if (nv == 16 && ((zrow + vbase) & 7) == 0) {
            if (res) {
                const uint4 r0 = *reinterpret_cast<const uint4*>(res), r1 = *reinterpret_cast<const uint4*>(res + 8);
                const uint32_t rw[8] = {r0.x, r0.y, r0.z, r0.w, r1.x, r1.y, r1.z, r1.w};
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    v[2 * j] += __uint_as_float(rw[j] << 16);
                    v[2 * j + 1] += __uint_as_float(rw[j] & 0xffff0000u);
                }
            }
            uint4 o0, o1;
            o0.x = pack_bf16(v[0], v[1]);  o0.y = pack_bf16(v[2], v[3]);   o0.z = pack_bf16(v[4], v[5]);   o0.w = pack_bf16(v[6], v[7]);
            o1.x = pack_bf16(v[8], v[9]);  o1.y = pack_bf16(v[10], v[11]); o1.z = pack_bf16(v[12], v[13]); o1.w = pack_bf16(v[14], v[15]);
            *reinterpret_cast<uint4*>(dst) = o0;
            *reinterpret_cast<uint4*>(dst + 8) = o1;
        } else {
#pragma unroll
            for (int j = 0; j < 16; ++j)
                if (j < nv) dst[j] = __float2bfloat16(v[j] + (res ? __bfloat162float(res[j]) : 0.f));
        }
        return;
    }
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = (j < nv) ? __uint_as_float(r[j]) : -INFINITY;
    if (store) {
        float* dst = a.out_logits + zrow + vbase;
        if (nv == 16 && ((zrow + vbase) & 3) == 0) {
#pragma unroll
            for (int j = 0; j < 16; j += 4) *reinterpret_cast<float4*>(dst + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
        } else {
#pragma unroll
            for (int j = 0; j < 16; ++j)
                if (j < nv) dst[j] = v[j];
        }
    }
    if (draft >= vbase && draft < vbase + nv) {
        float dv = 0.f;
#pragma unroll
        for (int j = 0; j < 16; ++j)
            if (draft - vbase == j) dv = v[j];
        a.out_draft_logit[grow] = dv;
    }
    float cm = v[0];
    int ci = 0;
#pragma unroll
    for (int j = 1; j < 16; ++j)
        if (v[j] > cm) {
            cm = v[j];
            ci = j;
        }
    if (cm > run_m) {
        if (a.need_sum) run_s *= exp2f((run_m - cm) * a.c2);
        run_m = cm;
        run_i = vbase + ci;
    }
    if (a.need_sum) {
        const float nm = -run_m * a.c2;
        float s = 0.f;
#pragma unroll
        for (int j = 0; j < 16; ++j) s += exp2f(fmaf(v[j], a.c2, nm));
        run_s += s;
    }
}

// Block `part` owns the granules [part * gran / nparts, (part + 1) * gran / nparts): the counts differ by at most
// one between blocks.  Its range is cut into T tiles of `base` or `base + 1` granules (the first `extra` tiles are
// the larger ones); over all blocks only the two sizes gmax - 1 and gmax occur.
struct Tiles {
    int g0, base, extra, n;
};
__device__ __forceinline__ Tiles block_tiles(const Args& a, int part) {
    const int lo = (int)((long)part * a.gran / a.nparts), hi = (int)((long)(part + 1) * a.gran / a.nparts);
    Tiles tl;
    tl.g0 = lo;
    tl.base = (hi - lo) / a.T;
    tl.extra = (hi - lo) % a.T;
    tl.n = tl.base > 0 ? a.T : tl.extra;
    return tl;
}
// First vocabulary row and granule count of tile t.
__device__ __forceinline__ void tile_span(const Tiles& tl, int t, int& row0, int& g) {
    g = tl.base + (t < tl.extra ? 1 : 0);
    row0 = (tl.g0 + t * tl.base + min(t, tl.extra)) * 16;
}

constexpr int STAGING_BYTES = 4 * 2 * 4096;   // per epilogue warp two 32-row x 32-column fp32 boxes

// The epilogue of both kernels: warp `quarter` owns TMEM lanes 32*quarter.. (block rows m0 + 32*quarter..).
// Every accumulator row is reduced to (max, lowest argmax, sum exp); the logits, when asked for, go to a
// staging box in the TMA 128-byte swizzle (16-byte chunk index XOR row mod 8: the 32 rows of a warp then hit
// distinct banks) and leave as one 32 x 32 TMA store per column group -- full 128-byte lines per row where
// per-thread stores would write 16 bytes of each of 32 rows.  A column group of 16 (odd g) and a vocabulary
// whose row pitch is not a multiple of 16 bytes use plain stores.
template <bool PAIR>
__device__ __forceinline__ void epilogue(const Args& a, const CUtensorMap* tm_z, int quarter, int lane, int m0, int part,
                                         const Tiles& tl, uint32_t tmem_base, uint32_t tfull0,
                                         uint32_t tempty0, uint32_t staging, volatile int* abort_flag) {
    const int row = quarter * 32 + lane;
    const int grow = m0 + row;
    const bool row_ok = grow < a.M;
    const size_t zrow = (size_t)(row_ok ? grow : 0) * a.V;
    const int draft = (row_ok && a.draft_ids && a.out_draft_logit) ? a.draft_ids[grow] : -1;
    const bool z_any = a.out_logits != nullptr;
    const bool z_box = a.z_tma && (m0 + quarter * 32 < a.M);      // warp-uniform
    const uint32_t stg = staging + (uint32_t)quarter * 8192u;
    const uint32_t stg_row = (uint32_t)lane * 128u, sw = (uint32_t)(lane & 7);
    int stg_i = 0;
    float run_m = -INFINITY, run_s = 0.f;
    int32_t run_i = 0x7fffffff;
    for (int t = 0; t < tl.n; ++t) {
        const int buf = t & 1;
        const uint32_t aph = (uint32_t)(t >> 1) & 1u;
        const bool got = mbar_wait(tfull0 + 8u * buf, aph, abort_flag);
        if (!__all_sync(0xffffffffu, got)) break;          // warp-uniform, so the aligned TMEM loads stay converged
        tcgen05_fence_after();
        int row0, g;
        tile_span(tl, t, row0, g);
        const int N = g * 16;
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * MAXN);
        for (int c = 0; c < N; c += 32) {
            uint32_t r0[16], r1[16];
            TMEM_LD_X16(taddr + c, r0);
            const bool second = (c + 16 < N);
            if (second) TMEM_LD_X16(taddr + c + 16, r1);
            tmem_wait_ld();
            const bool box = z_box && second && (row0 + c < a.V);
            const bool direct = z_any && !box;
            consume16(r0, row0 + c, a.V, row_ok, a, zrow, draft, grow, direct, run_m, run_i, run_s);
            if (second) consume16(r1, row0 + c + 16, a.V, row_ok, a, zrow, draft, grow, direct, run_m, run_i, run_s);
            if (box) {
                // the store issued from this buffer two groups ago has read it
                if (lane == 0) bulk_wait_read<1>();
                __syncwarp();
                const uint32_t b = stg + (uint32_t)stg_i * 4096u + stg_row;
                stg_i ^= 1;
#pragma unroll
                for (uint32_t j = 0; j < 4; ++j) {
                    st_shared_v4(b + ((j ^ sw) << 4), r0[4 * j], r0[4 * j + 1], r0[4 * j + 2], r0[4 * j + 3]);
                    st_shared_v4(b + (((j + 4) ^ sw) << 4), r1[4 * j], r1[4 * j + 1], r1[4 * j + 2], r1[4 * j + 3]);
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    tma_store_2d(tm_z, b - stg_row, row0 + c, m0 + quarter * 32);   // rows >= M, columns >= V are clipped
                    bulk_commit();
                }
            }
        }
        tcgen05_fence_before();
        __syncwarp();
        if (lane == 0) {
            if (PAIR) mbar_arrive_cluster(map_to_cta(tempty0 + 8u * buf, 0));
            else mbar_arrive(tempty0 + 8u * buf);
        }
    }
    if (lane == 0) bulk_wait<0>();               // the staging area outlives every store that reads it
    if (row_ok && !a.out_bf16) {
        Partial pr;
        pr.m = run_m;
        pr.idx = run_i;
        pr.s = a.need_sum ? run_s : 1.f;
        pr.pad = 0;
        if (*abort_flag) pr.idx = PARTIAL_ABORTED;     // the finalisation turns this into ids of -2
        a.part[(size_t)part * a.M + grow] = pr;
    }
}

__global__ void __launch_bounds__(THREADS, 1)
lmhead_umma_kernel(const __grid_constant__ CUtensorMap tm_h, const __grid_constant__ CUtensorMap tm_w_hi,
                   const __grid_constant__ CUtensorMap tm_w_lo, const __grid_constant__ CUtensorMap tm_z, const Args a) {
    extern __shared__ unsigned char smem_raw[];
    // operand stages need 1024-byte alignment for the 128-byte swizzle
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int stage_bytes = a.stage_bytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + a.stages * stage_bytes + (a.z_tma ? STAGING_BYTES : 0));
    // bars[0..S) full, [S..2S) empty, [2S..2S+2) accumulator full, [2S+2..2S+4) accumulator empty   (S = MAX_STAGES)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * MAX_STAGES + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int m0 = blockIdx.x * BM;
    const int part = blockIdx.y % a.nparts;        // vocabulary (output-column) part
    const int ks = blockIdx.y / a.nparts;          // range of the contraction (linear layers with few columns only)
    const Tiles tl = block_tiles(a, part);
    const int n_tiles = tl.n;
    const int KBall = a.hid / BK;
    const int kb0 = (int)((long)ks * KBall / a.ksplit), KB = (int)((long)(ks + 1) * KBall / a.ksplit) - kb0;

    const uint32_t smem_base = smem_u32(smem);
    const uint32_t bar_base = smem_u32(bars);
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (MAX_STAGES + s); };
    auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * MAX_STAGES + b); };
    auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * MAX_STAGES + 2 + b); };

    // ---- set-up ---------------------------------------------------------------
    if (tid == 0) {
        for (int s = 0; s < a.stages; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(tfull_bar(b), 1);
            mbar_init(tempty_bar(b), 4);
        }
        *abort_flag = 0;
        mbar_init_fence();
    }
    // The weights are the model's: nothing that runs before this kernel writes them, so the first ring of weight
    // tiles is requested right away -- before the tensor memory is there, and before the kernel ahead of this one
    // in the stream has finished.  The h tiles of those stages follow once it has.
    int pre = 0;                                  // stages whose weight tile was requested ahead (producer thread only)
    if (tid == 0 && n_tiles > 0) {
        prefetch_tensormap(&tm_h);
        int it = 0;
        for (int t = 0; t < n_tiles && it < a.stages; ++t) {
            int row0, g;
            tile_span(tl, t, row0, g);
            const CUtensorMap* tm_w = (g == a.gmax) ? &tm_w_hi : &tm_w_lo;
            const uint32_t stage_tx = (uint32_t)(a.h_box_rows * 128 + g * 16 * 128);
            for (int kb = 0; kb < KB && it < a.stages; ++kb, ++it) {
                mbar_expect_tx(full_bar(it), stage_tx);
                tma_load_2d(smem_base + it * stage_bytes + a.a_bytes, tm_w, (kb0 + kb) * BK, row0, full_bar(it));
            }
        }
        pre = it;
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), 512);
    }
    pdl_trigger();
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();                                   // h, the draft ids and every output depend on what ran before

    // Accumulator rows at or beyond h_box_rows are never read back, and row i of an MMA depends on row i
    // of its 128-row operand only, so the h atom holds just h_box_rows rows: the rest of the 16 KB the
    // MMA reads for that operand is whatever follows in the stage (the w atom), and lands in unused lanes.
    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0 && n_tiles > 0) {
            int it = 0;
            bool ok = true;
            for (int t = 0; t < n_tiles && ok; ++t) {
                int row0, g;
                tile_span(tl, t, row0, g);
                const CUtensorMap* tm_w = (g == a.gmax) ? &tm_w_hi : &tm_w_lo;
                const uint32_t stage_tx = (uint32_t)(a.h_box_rows * 128 + g * 16 * 128);
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    const int s = it % a.stages;
                    const uint32_t sa = smem_base + s * stage_bytes;
                    if (it >= pre) {                       // the first `pre` weight tiles are on their way already
                        const uint32_t ph = (uint32_t)(it / a.stages) & 1u;
                        if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) { ok = false; break; }
                        mbar_expect_tx(full_bar(s), stage_tx);
                        tma_load_2d(sa + a.a_bytes, tm_w, (kb0 + kb) * BK, row0, full_bar(s));     // the whole N-row tile in one box
                    }
                    tma_load_2d(sa, &tm_h, (kb0 + kb) * BK, m0, full_bar(s));
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0 && n_tiles > 0) {
            int it = 0;
            bool ok = true;
            for (int t = 0; t < n_tiles && ok; ++t) {
                int row0, g;
                tile_span(tl, t, row0, g);
                const uint32_t idesc = make_idesc_bf16(g * 16, 0);
                const int buf = t & 1;
                const uint32_t aph = (uint32_t)(t >> 1) & 1u;
                if (!mbar_wait(tempty_bar(buf), aph ^ 1u, abort_flag)) break;
                tcgen05_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * MAXN);
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    const int s = it % a.stages;
                    const uint32_t ph = (uint32_t)(it / a.stages) & 1u;
                    if (!mbar_wait(full_bar(s), ph, abort_flag)) { ok = false; break; }
                    tcgen05_fence_after();
                    const uint32_t sa = smem_base + s * stage_bytes;
                    const uint64_t ad = smem_desc_sw128_kmajor(sa), bd = smem_desc_sw128_kmajor(sa + a.a_bytes);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)     // 16 bf16 = 32 bytes = 2 descriptor units along K
                        umma_bf16_ss(d_tmem, ad + 2 * k, bd + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
                    umma_commit(empty_bar(s));            // stage reusable once these MMAs have read it
                }
                if (ok) umma_commit(tfull_bar(buf));      // accumulator complete
            }
        }
    } else {
        // ---------------- epilogue: 4 warps, one TMEM lane quarter each ----------------
        epilogue<false>(a, &tm_z, warp & 3, lane, m0, part, tl, tmem_base, tfull_bar(0), tempty_bar(0),
                        smem_base + (uint32_t)(a.stages * stage_bytes), abort_flag);
    }

    // ---- tear-down ------------------------------------------------------------
    tcgen05_fence_before();
    __syncthreads();
    if (*abort_flag) {
        // give copies that are still in flight time to land before the block's shared memory goes away
        for (int i = 0; i < 64; ++i) __nanosleep(10000);
        __syncthreads();
    }
    if (warp == 1) {
        __syncwarp();
        tcgen05_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// ---- CTA-pair variant (more than 128 block rows) ------------------------------------
// Two thread blocks of a cluster share every weight tile: one tcgen05.mma with cta_group::2 covers 256 block
// rows (128 per block, in that block's tensor memory) and reads half of the N-row weight tile from each
// block's shared memory, so each block stages 16 KB of h and N/2 rows of w per 64-wide step instead of all N:
// a third less L2 -> shared-memory traffic per flop, which is what bounds the single-block kernel at these
// sizes.  Block 0 of the pair issues the MMAs.  Its `full` barriers count the bytes of both blocks' loads (the
// peer's TMA completes on the leader's barrier); `empty` and `accumulator full` arrive in both blocks through
// one multicast commit; both blocks' epilogue warps arrive on the leader's `accumulator empty`.
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(THREADS, 1)
lmhead_umma_pair_kernel(const __grid_constant__ CUtensorMap tm_h, const __grid_constant__ CUtensorMap tm_w_hi,
                        const __grid_constant__ CUtensorMap tm_w_lo, const __grid_constant__ CUtensorMap tm_z, const Args a) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int stage_bytes = a.stage_bytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + a.stages * stage_bytes + (a.z_tma ? STAGING_BYTES : 0));
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * MAX_STAGES + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_ctarank();
    const bool leader = (rank == 0);
    const int m0 = (int)(blockIdx.x >> 1) * (2 * BM) + (int)rank * BM;
    const int part = blockIdx.y % a.nparts;        // vocabulary (output-column) part
    const int ks = blockIdx.y / a.nparts;          // range of the contraction (linear layers with few columns only)
    const Tiles tl = block_tiles(a, part);
    const int n_tiles = tl.n;
    const int KBall = a.hid / BK;
    const int kb0 = (int)((long)ks * KBall / a.ksplit), KB = (int)((long)(ks + 1) * KBall / a.ksplit) - kb0;

    const uint32_t smem_base = smem_u32(smem);
    const uint32_t bar_base = smem_u32(bars);
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (MAX_STAGES + s); };
    auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * MAX_STAGES + b); };
    auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * MAX_STAGES + 2 + b); };

    if (tid == 0) {
        for (int s = 0; s < a.stages; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(tfull_bar(b), 1);
            mbar_init(tempty_bar(b), 8);         // four epilogue warps in each of the two blocks
        }
        *abort_flag = 0;
        mbar_init_fence();
    }
    if (warp == 0 && lane == 0) {
        prefetch_tensormap(&tm_h);
        prefetch_tensormap(&tm_w_hi);
        prefetch_tensormap(&tm_w_lo);
    }
    if (warp == 1) tmem_alloc_pair(smem_u32(tmem_slot), 512);
    pdl_trigger();
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync();                              // the peer's barriers exist before anything signals them
    tcgen05_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();                                   // everything above needed no input; h (and what follows) does

    if (warp == 0) {
        // ---------------- TMA producer (each block: its 128 rows of h, its half of the weight tile) ----------------
        if (lane == 0 && n_tiles > 0) {
            int it = 0;
            bool ok = true;
            for (int t = 0; t < n_tiles && ok; ++t) {
                int row0, g;
                tile_span(tl, t, row0, g);
                const int half = g * 8;                  // rows of the weight tile this block stages
                row0 += (int)rank * half;
                const CUtensorMap* tm_w = (g == a.gmax) ? &tm_w_hi : &tm_w_lo;
                const uint32_t stage_tx = 2u * (uint32_t)(A_SPAN + half * 128);
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    const int s = it % a.stages;
                    const uint32_t ph = (uint32_t)(it / a.stages) & 1u;
                    if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) { ok = false; break; }
                    if (leader) mbar_expect_tx(full_bar(s), stage_tx);
                    const uint32_t lead_full = map_to_cta(full_bar(s), 0);
                    const uint32_t sa = smem_base + s * stage_bytes;
                    tma_load_2d_pair(sa + A_SPAN, tm_w, (kb0 + kb) * BK, row0, lead_full);
                    tma_load_2d_pair(sa, &tm_h, (kb0 + kb) * BK, m0, lead_full);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader block only) ----------------
        if (leader && lane == 0 && n_tiles > 0) {
            int it = 0;
            bool ok = true;
#ifdef DEER_TIMING_PROBES
            long long w_full = 0, w_acc = 0, n_mma = 0;
#endif
            LM_PROBE_T0(t_begin);
            for (int t = 0; t < n_tiles && ok; ++t) {
                int row0, g;
                tile_span(tl, t, row0, g);
                const uint32_t idesc = make_idesc_bf16_pair(g * 16);
                const int buf = t & 1;
                const uint32_t aph = (uint32_t)(t >> 1) & 1u;
                LM_PROBE_T0(t_acc);
                if (!mbar_wait(tempty_bar(buf), aph ^ 1u, abort_flag)) break;
                LM_PROBE_ADD(w_acc, t_acc);
                tcgen05_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * MAXN);
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    const int s = it % a.stages;
                    const uint32_t ph = (uint32_t)(it / a.stages) & 1u;
                    LM_PROBE_T0(t_full);
                    if (!mbar_wait(full_bar(s), ph, abort_flag)) { ok = false; break; }
                    LM_PROBE_ADD(w_full, t_full);
                    tcgen05_fence_after();
                    const uint32_t sa = smem_base + s * stage_bytes;
                    const uint64_t ad = smem_desc_sw128_kmajor(sa), bd = smem_desc_sw128_kmajor(sa + A_SPAN);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)
                        umma_bf16_ss_pair(d_tmem, ad + 2 * k, bd + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
#ifdef DEER_TIMING_PROBES
                    n_mma += BK / 16;
#endif
                    umma_commit_pair(empty_bar(s), 3);
                }
                if (ok) umma_commit_pair(tfull_bar(buf), 3);
            }
#ifdef DEER_TIMING_PROBES
            {
                const int bi = (int)(blockIdx.y * gridDim.x + blockIdx.x) >> 1;       // leader blocks, in launch order
                if (bi < DEER_PROBE_ROWS) {
                    g_lmhead_probe[bi][0] = clock64() - t_begin;
                    g_lmhead_probe[bi][1] = w_full;
                    g_lmhead_probe[bi][2] = w_acc;
                    g_lmhead_probe[bi][3] = n_mma;
                }
            }
#endif
        }
    } else {
        // ---------------- epilogue: 4 warps in each block, one TMEM lane quarter each ----------------
        epilogue<true>(a, &tm_z, warp & 3, lane, m0, part, tl, tmem_base, tfull_bar(0), tempty_bar(0),
                       smem_base + (uint32_t)(a.stages * stage_bytes), abort_flag);
    }

    // ---- tear-down: neither block leaves while the other may still signal it or read its shared memory ----
    tcgen05_fence_before();
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(10000);
        __syncthreads();
    }
    cluster_sync();
    if (warp == 1) {
        __syncwarp();
        tcgen05_fence_after();
        tmem_dealloc_pair(tmem_base, 512);
    }
}

// ---- host side ------------------------------------------------------------------
// 2-D bf16 tensor [rows][cols] (cols contiguous), box = box_rows x 64 columns.
static int make_operand_map(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    const uint64_t dims[2] = {cols, rows};
    const uint64_t strides[1] = {cols * 2};
    const uint32_t box[2] = {BK, box_rows};
    return make_map_bf16(tm, base, 2, dims, strides, box);
}

}  // namespace umma

bool umma_supported(int M, int hid, int V) { return M > 0 && hid % umma::BK == 0 && hid >= umma::BK && V >= 16; }

// Launches the tcgen05 kernel.  Selection: *nparts_out vocabulary parts per row are left for the finalisation;
// linear layer: *ksplit_out tells whether partial products are left to be summed.
int launch_umma(const Params& p, int need_sum, int* nparts_out, cudaStream_t st, int* ksplit_out) {
    using namespace umma;
    const int sms = deer_sm_count();
    // more than 128 block rows: pairs of blocks share the weight tiles (256 rows per pair)
    const bool pair = p.M > BM;
    const int m_tiles = pair ? 2 * ((p.M + 2 * BM - 1) / (2 * BM)) : (p.M + BM - 1) / BM;
    int nparts = sms / m_tiles;
    if (nparts < 1) nparts = 1;
    const int gran = (p.V + 15) / 16;                    // 16-row granules of the vocabulary
    if (nparts > gran) nparts = gran;
    // A linear layer with few output columns would leave each block a sliver of a tile (or leave SMs idle): give the
    // blocks full 16-granule column tiles instead and cut the contraction into ranges, summed up afterwards.
    int ksplit = 1;
    if (p.out_bf16 && p.lin_part && m_tiles == 1 && gran < sms * 8) {
        const int col_parts = (gran + 15) / 16;
        const int kb_all = p.hid / BK;
        ksplit = sms / col_parts;
        if (ksplit > kb_all / 4) ksplit = kb_all / 4;    // at least four 64-wide steps per range
        if (ksplit > p.max_ksplit) ksplit = p.max_ksplit;
        if (ksplit < 1) ksplit = 1;
        if (ksplit > 1) nparts = col_parts;
    }
    const int cmax = (gran + nparts - 1) / nparts;       // granules of the largest block
    const int T = (cmax + 15) / 16;                      // tiles per block so that a tile has <= 16 granules
    Args a;
    a.M = p.M;
    a.hid = p.hid;
    a.V = p.V;
    a.h_box_rows = (p.M >= BM) ? BM : ((p.M + 7) / 8) * 8;
    a.gmax = (cmax + T - 1) / T;
    a.a_bytes = a.h_box_rows * 128;
    const int w_rows = pair ? 8 : 16;                    // weight rows per granule that one block stages
    // a stage is never shorter than the span an MMA reads for its 128-row operand
    a.stage_bytes = a.a_bytes + a.gmax * w_rows * 128;
    if (a.stage_bytes < A_SPAN) a.stage_bytes = A_SPAN;
    // logits through TMA stores need a row pitch that is a multiple of 16 bytes
    a.z_tma = (p.out_logits != nullptr && p.V % 4 == 0) ? 1 : 0;
    // as deep a ring as shared memory holds: the bytes in flight per SM are what hide the HBM latency
    a.stages = (a.z_tma ? SMEM_LIMIT - 1280 - STAGING_BYTES : SMEM_BUDGET) / a.stage_bytes;
    if (a.stages > MAX_STAGES) a.stages = MAX_STAGES;
    a.T = T;
    a.gran = gran;
    a.nparts = nparts;
    a.need_sum = need_sum;
    a.c2 = p.inv_t_log2;
    a.draft_ids = p.draft_ids;
    a.out_draft_logit = p.out_draft_logit;
    a.out_logits = p.out_logits;
    a.out_bf16 = p.out_bf16;
    a.residual = p.residual;
    a.ksplit = ksplit;
    a.swiglu = p.swiglu;
    a.lin_part = p.lin_part;
    a.part = p.part;
    CUtensorMap tm_h, tm_w_hi, tm_w_lo;
    int rc = make_operand_map(&tm_h, p.h, (uint64_t)p.M, (uint64_t)p.hid, (uint32_t)a.h_box_rows);
    if (rc != DEER_OK) return rc;
    rc = make_operand_map(&tm_w_hi, p.w, (uint64_t)p.V, (uint64_t)p.hid, (uint32_t)(a.gmax * w_rows));
    if (rc != DEER_OK) return rc;
    rc = make_operand_map(&tm_w_lo, p.w, (uint64_t)p.V, (uint64_t)p.hid, (uint32_t)((a.gmax > 1 ? a.gmax - 1 : 1) * w_rows));
    if (rc != DEER_OK) return rc;
    CUtensorMap tm_z = tm_h;                             // a valid map even when it is not used
    if (a.z_tma) {
        const uint64_t dims[2] = {(uint64_t)p.V, (uint64_t)p.M};
        const uint64_t strides[1] = {(uint64_t)p.V * 4};
        const uint32_t box[2] = {32, 32};
        rc = make_map_f32(&tm_z, p.out_logits, 2, dims, strides, box);
        if (rc != DEER_OK) return rc;
    }
    const int smem_bytes = a.stages * a.stage_bytes + (a.z_tma ? STAGING_BYTES : 0) + 1024 /*alignment slack*/ + 256 /*barriers*/;
    dim3 grid(m_tiles, nparts * ksplit);
    if (ksplit_out) *ksplit_out = ksplit;
    if (pair) {
        DEER_CUDA(cudaFuncSetAttribute(lmhead_umma_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes));
        DEER_CUDA(launch_pdl(lmhead_umma_pair_kernel, grid, dim3(umma::THREADS), (size_t)smem_bytes, st, tm_h, tm_w_hi, tm_w_lo, tm_z, a));
    } else {
        DEER_CUDA(cudaFuncSetAttribute(lmhead_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes));
        DEER_CUDA(launch_pdl(lmhead_umma_kernel, grid, dim3(umma::THREADS), (size_t)smem_bytes, st, tm_h, tm_w_hi, tm_w_lo, tm_z, a));
    }
    DEER_CUDA(cudaGetLastError());
    *nparts_out = nparts;
    return DEER_OK;
}

}  // namespace lmhead
