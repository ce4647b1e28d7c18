// Block attention on the 5th-generation tensor cores (head_dim 128).
//
// One thread block = one context chunk of one (sequence, KV head, row tile).
// The query rows that share the KV head -- block row i with its G query heads,
// row = (i - i0) * G + g -- sit on the 128 TMEM lanes.  KV pages stream through
// a ring of 64-token slots filled by TMA, one 4 KB box per page (see the slot
// layout below); S = Q K^T and O += P V are tcgen05 MMAs:
//     S (128 x 64, fp32)  = Q [smem, K-major] x K tile [smem, K-major]
//     O (128 x 128, fp32) += P [TMEM, bf16] x V tile [smem, MN-major]
// S and P are double-buffered so that the MMAs of tile t+1 overlap the softmax
// of tile t.  A thread gets a tcgen05.mma accepted only every ~100 cycles
// whatever its size, so three warps issue -- even S tiles, odd S tiles, O --
// and their streams interleave on the tensor pipe.  The softmax warps hold one row per
// thread (no shuffles), keep a running maximum that is only raised when a tile
// exceeds it by 2^8 (the accumulator in TMEM is rescaled then, which is rare),
// and emit a normalised partial output plus log2-sum-exp per chunk; the merge
// kernel combines the chunks.
//
// Warp roles: warp 0 = TMA producer, warps 1-2 = issuers of S = Q K^T (warp 1
// owns the TMEM allocation), warp 3 = issuer of O += P V, warps 4..7 = softmax
// (one TMEM lane quarter each).  Every wait is bounded: a wait that runs out raises the
// block's abort flag and the cache's status word, every role leaves its loop,
// TMEM is freed and the kernel returns.

#include "attn.cuh"
#include "sm100.cuh"

namespace attn {
namespace umma {

using namespace sm100;

constexpr int HD = 128;                        // head dim
constexpr int NSLOT = 6;                       // ring slots of 64 tokens
constexpr int Q_HALF = 128 * 128;              // [128 rows][64 d] bf16
constexpr int Q_BYTES = 2 * Q_HALF;            // 32 KB
constexpr int KV_HALF = ATT_TILE * 128;        // [64 tokens][64 d] bf16 = 8 KB
constexpr int K_BYTES = 2 * KV_HALF;           // 16 KB
constexpr int SLOT_BYTES = 2 * K_BYTES;        // K tile then V tile
constexpr int THREADS = 256;
constexpr int TMEM_COLS = 512;                 // S0 [0,64)  S1 [64,128)  P0 [128,160)  P1 [160,192)  O [256,384)
constexpr int P_COL = 128;
constexpr int O_COL = 256;
constexpr int N_BARS = 3 * NSLOT + 6;
constexpr float RESCALE_STEP = 8.f;            // raise the running maximum only when a tile exceeds it by 2^8
// Slot layout.  A K (or V) tile of 64 tokens x 128 dims is 16 KB of 1 KB swizzle atoms (8 tokens x 64 dims).
//   prefix tile: [page 0..3][token group 0..1][dim half 0..1][8 tokens][128 B] -- what one 5-D TMA box per page
//                writes; atoms of one dim half are 2 KB apart along the tokens, the two halves 1 KB apart.
//   block tile:  [dim half 0..1][64 tokens][128 B] -- the block's own rows, from k_blk / v_blk; atoms 1 KB apart
//                along the tokens, the halves 8 KB apart.
constexpr int SMEM_BYTES = Q_BYTES + NSLOT * SLOT_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;

__device__ __forceinline__ float ex2_approx(float x) {   // 2^x, one MUFU op; -inf gives 0
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__global__ void __launch_bounds__(THREADS, 1)
block_attn_umma_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kb,
                       const __grid_constant__ CUtensorMap tm_vb, const __grid_constant__ CUtensorMap tm_kpool,
                       const __grid_constant__ CUtensorMap tm_vpool, const AttnParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char* sQ = smem;                                  // [2 halves][128 rows][128 B]
    unsigned char* ring = smem + Q_BYTES;                      // [NSLOT][K: 2 halves x 64 x 128 B][V: same]
    uint64_t* bars = reinterpret_cast<uint64_t*>(ring + NSLOT * SLOT_BYTES);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + N_BARS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int c = blockIdx.x;
    const int kvh = blockIdx.y / p.row_tiles;
    const int rt = blockIdx.y % p.row_tiles;
    const int b = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int Hkv = p.kv.n_kv_heads;

    const int s = p.seq_ids[b];
    if (s < 0 || s >= p.kv.max_seqs) {
        if (tid == 0) deer_report(p.kv.status, DEER_ERR_INVALID_ARG);
        return;
    }
    const int n = p.kv.seq_len[s];
    if (n > p.max_seq_len || n < 0) {
        if (tid == 0) deer_report(p.kv.status, DEER_ERR_INVALID_ARG);
        return;
    }
    const int n_chunks = max(1, (n + p.chunk - 1) / p.chunk);
    if (c >= n_chunks) return;
    const bool last = (c == n_chunks - 1);
    const int t_begin = c * p.chunk;
    const int t_end = min(n, t_begin + p.chunk);
    const int n_prefix_tiles = (t_end > t_begin) ? (t_end - t_begin + ATT_TILE - 1) / ATT_TILE : 0;
    const int n_tiles = n_prefix_tiles + (last ? 1 : 0);          // the block rows' own K/V are one more tile
    const int32_t* pt_row = p.kv.page_table + (size_t)s * p.kv.max_pages;
    const int i0 = rt * p.ipt;                                     // first block row of this row tile
    const int ni = min(p.ipt, p.k - i0);                           // block rows in it
    const int q_box_rows = p.G * min(p.ipt, p.k);                  // rows one Q box brings

    const uint32_t bar_base = smem_u32(bars);
    const uint32_t q_full = bar_base;
    auto k_full = [&](int sl) { return bar_base + 8u * (1 + sl); };
    auto v_full = [&](int sl) { return bar_base + 8u * (1 + NSLOT + sl); };
    auto slot_empty = [&](int sl) { return bar_base + 8u * (1 + 2 * NSLOT + sl); };
    auto s_full = [&](int bf) { return bar_base + 8u * (1 + 3 * NSLOT + bf); };
    auto p_ready = [&](int bf) { return bar_base + 8u * (3 + 3 * NSLOT + bf); };
    const uint32_t o_done = bar_base + 8u * (5 + 3 * NSLOT);

    // ---- set-up ---------------------------------------------------------------
    if (tid == 0) {
        mbar_init(q_full, 1);
        for (int sl = 0; sl < NSLOT; ++sl) {
            mbar_init(k_full(sl), 1);
            mbar_init(v_full(sl), 1);
            mbar_init(slot_empty(sl), 1);
        }
        for (int bf = 0; bf < 2; ++bf) {
            mbar_init(s_full(bf), 1);
            mbar_init(p_ready(bf), 4);
        }
        mbar_init(o_done, 1);
        *abort_flag = 0;
        mbar_init_fence();
    }
    if (warp == 0 && lane == 0) {
        prefetch_tensormap(&tm_q);
        prefetch_tensormap(&tm_kpool);
        prefetch_tensormap(&tm_vpool);
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t q_addr = smem_u32(sQ);
    const uint32_t ring_addr = smem_u32(ring);

    if (warp == 0) {
        // ---------------- TMA producer (whole warp: lanes hold the page ids of a tile) ----------------
        if (lane == 0) {
            mbar_expect_tx(q_full, (uint32_t)(2 * q_box_rows * 128));
            tma_load_3d(q_addr, &tm_q, 0, kvh * p.G, b * p.k + i0, q_full);
            tma_load_3d(q_addr + Q_HALF, &tm_q, 64, kvh * p.G, b * p.k + i0, q_full);
        }
        // Lanes 0..7 each issue one copy of a tile: lane = is_v * 4 + page-in-tile (block tile: is_v * 4 + half).
        // Page ids are fetched two tiles ahead (lane L holds the id of page L & 3) and validated only when used.
        const int pj = lane & 3, is_v = (lane >> 2) & 1;
        auto page_of = [&](int tile) -> int {
            if (tile >= n_prefix_tiles || lane >= 8) return 0;
            const int lp = ((t_begin + tile * ATT_TILE) >> 4) + pj;
            if (lp * DEER_PAGE_SIZE >= t_end || lp >= p.kv.max_pages) return -1;
            return pt_row[lp];
        };
        int pg_cur = page_of(0), pg_next = page_of(1);
        for (int i = 0; i < n_tiles; ++i) {
            const int sl = i % NSLOT;
            const uint32_t par = (uint32_t)(i / NSLOT) & 1u;
            int pg = pg_cur;
            pg_cur = pg_next;
            pg_next = page_of(i + 2);
            int ok = 1;
            if (lane == 0) ok = mbar_wait(slot_empty(sl), par ^ 1u, abort_flag) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            const uint32_t kdst = ring_addr + sl * SLOT_BYTES, vdst = kdst + K_BYTES;
            const uint32_t dst = is_v ? vdst : kdst;
            const uint32_t bar = is_v ? v_full(sl) : k_full(sl);
            if (i < n_prefix_tiles) {
                const int t0 = t_begin + i * ATT_TILE;
                const int np = (min(ATT_TILE, t_end - t0) + DEER_PAGE_SIZE - 1) / DEER_PAGE_SIZE;
                if (lane == 0) {
                    mbar_expect_tx(k_full(sl), (uint32_t)np * 4096u);
                    mbar_expect_tx(v_full(sl), (uint32_t)np * 4096u);
                }
                __syncwarp();
                if (lane < 8 && pj < np) {
                    if (pg < 0 || pg >= p.kv.num_pages) {
                        deer_report(p.kv.status, DEER_ERR_BAD_PAGE);
                        pg = 0;                 // keep the copy inside the pool; the status word flags the result
                    }
                    tma_load_5d(dst + pj * 4096, is_v ? &tm_vpool : &tm_kpool, 0, 0, 0, 0, pg * Hkv + kvh, bar);
                }
            } else {
                // the block rows' own keys and values: k rows straight from k_blk / v_blk
                if (lane == 0) {
                    mbar_expect_tx(k_full(sl), (uint32_t)(2 * p.k * 128));
                    mbar_expect_tx(v_full(sl), (uint32_t)(2 * p.k * 128));
                }
                __syncwarp();
                if (lane < 8 && pj < 2) tma_load_3d(dst + pj * KV_HALF, is_v ? &tm_vb : &tm_kb, pj * 64, kvh, b * p.k, bar);
            }
        }
    } else if (warp <= 2) {
        // ---------------- issuers of S = Q K^T: warp 1 takes the even tiles, warp 2 the odd ones ----------------
        if (lane == 0) {
            const uint32_t idesc_qk = make_idesc_bf16(ATT_TILE, 0);   // S: N = 64 tokens, both operands K-major
            // Operand descriptors are built once; inside the loops only their 16-byte-unit address field moves
            // (one issuing thread: every instruction between two MMAs is latency on the critical path).
            const uint64_t q_desc = smem_desc_sw128_kmajor(q_addr);
            const uint64_t k_desc_pre = smem_desc_sw128(ring_addr, 16, 2048), k_desc_blk = smem_desc_sw128(ring_addr, 16, 1024);
            bool ok = mbar_wait(q_full, 0u, abort_flag);
            // S[i & 1] = Q K_i^T: 8 k-steps of 16 dims, 4 per 64-wide half
            auto issue_qk = [&](int i) -> bool {
                const int sl = i % NSLOT;
                if (!mbar_wait(k_full(sl), (uint32_t)(i / NSLOT) & 1u, abort_flag)) return false;
                tcgen05_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)((i & 1) * ATT_TILE);
                const bool blk = (i >= n_prefix_tiles);
                const uint64_t kd = (blk ? k_desc_blk : k_desc_pre) + (uint64_t)((sl * SLOT_BYTES) >> 4);
                const uint64_t half16 = blk ? (KV_HALF >> 4) : (1024 >> 4);     // distance between the dim halves
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk) {
                    const uint64_t ad = q_desc + (uint64_t)(((kk >> 2) * Q_HALF + (kk & 3) * 32) >> 4);
                    const uint64_t bd = kd + ((kk >> 2) ? half16 : 0) + (uint64_t)(((kk & 3) * 32) >> 4);
                    umma_bf16_ss(d_tmem, ad, bd, idesc_qk, kk != 0 ? 1u : 0u);
                }
                umma_commit(s_full(i & 1));
                return true;
            };
            // S buffer i & 1 is free again once the softmax warps have read tile i-2 out of it: p_ready of that tile
            for (int i = warp - 1; i < n_tiles && ok; i += 2) {
                if (i >= 2 && !mbar_wait(p_ready(i & 1), (uint32_t)((i - 2) >> 1) & 1u, abort_flag)) break;
                ok = issue_qk(i);
            }
        }
    } else if (warp == 3) {
        // ---------------- issuer of O += P V ----------------
        if (lane == 0) {
            const uint32_t idesc_pv = make_idesc_bf16(HD, 1);         // O: N = 128 dims, V is MN-major
            const uint64_t v_desc_pre = smem_desc_sw128(ring_addr + K_BYTES, 1024, 2048);
            const uint64_t v_desc_blk = smem_desc_sw128(ring_addr + K_BYTES, KV_HALF, 1024);
            for (int i = 0; i < n_tiles; ++i) {
                const int sl = i % NSLOT;
                if (!mbar_wait(p_ready(i & 1), (uint32_t)(i >> 1) & 1u, abort_flag)) break;
                if (!mbar_wait(v_full(sl), (uint32_t)(i / NSLOT) & 1u, abort_flag)) break;
                tcgen05_fence_after();
                const uint32_t p_tmem = tmem_base + (uint32_t)(P_COL + (i & 1) * (ATT_TILE / 2));
                const bool blk = (i >= n_prefix_tiles);
                // 16 tokens per MMA = two 8-token atoms; lbo = distance between the dim halves, sbo = between token atoms
                const uint64_t vd = (blk ? v_desc_blk : v_desc_pre) + (uint64_t)((sl * SLOT_BYTES) >> 4);
                const uint64_t step16 = blk ? (2048 >> 4) : (4096 >> 4);
#pragma unroll
                for (int kk = 0; kk < ATT_TILE / 16; ++kk)
                    umma_bf16_ts(tmem_base + O_COL, p_tmem + kk * 8, vd + kk * step16, idesc_pv, (i | kk) != 0 ? 1u : 0u);
                // S_i was complete before the softmax of tile i, hence before this point: both K and V are consumed
                umma_commit(slot_empty(sl));
                umma_commit(o_done);                      // phase i of o_done: O includes tile i
            }
        }
    } else {
        // ---------------- softmax: 4 warps, one TMEM lane quarter each, one query row per thread ----------------
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const int i_blk = i0 + row / p.G;                 // block row of this query row
        const int g = row % p.G;
        const bool row_valid = row < ni * p.G;
        const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
        const int wtid = tid - 128;                       // 0..127 within the softmax warps

        // append the block's K/V rows to the cache (one thread block per (sequence, KV head))
        if (p.append && last && rt == 0) {
            constexpr int PIECES = HD / 8;
            for (int idx = wtid; idx < p.k * PIECES; idx += 128) {
                const int j = idx / PIECES, pc = idx % PIECES;
                const int t = n + j;
                const int lp = t >> 4;
                const int pg = (lp < p.kv.max_pages) ? pt_row[lp] : -1;
                if (pg < 0 || pg >= p.kv.num_pages) {
                    deer_report(p.kv.status, DEER_ERR_BAD_PAGE);
                    continue;
                }
                const size_t src = ((size_t)(b * p.k + j) * Hkv + kvh) * HD + pc * 8;
                const size_t dst = (((size_t)pg * Hkv + kvh) * DEER_PAGE_SIZE + (t & 15)) * HD + pc * 8;
                *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.kv.k_pool) + dst) =
                    *reinterpret_cast<const uint4*>(p.k_blk + src);
                *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.kv.v_pool) + dst) =
                    *reinterpret_cast<const uint4*>(p.v_blk + src);
            }
        }

        float m_run = 0.f, l_run = 0.f;                   // running maximum (log2 domain, scaled) and row sum
        bool alive = true;
        for (int i = 0; i < n_tiles; ++i) {
            const int buf = i & 1;
            const int sl = i % NSLOT;
            const bool got = mbar_wait(s_full(buf), (uint32_t)(i >> 1) & 1u, abort_flag);
            if (!__all_sync(0xffffffffu, got)) { alive = false; break; }     // warp-uniform: the aligned TMEM ops stay converged
            tcgen05_fence_after();
            uint32_t sr[ATT_TILE];
            TMEM_LD_X32(t_lane + buf * ATT_TILE, (sr));
            TMEM_LD_X32(t_lane + buf * ATT_TILE + 32, (sr + 32));
            tmem_wait_ld();

            // columns this row may see: the valid tokens of a prefix tile, or the block rows the mask allows
            const bool is_block = (i >= n_prefix_tiles);
            const int tile_valid = is_block ? p.k : min(ATT_TILE, t_end - (t_begin + i * ATT_TILE));
            int limit = tile_valid;
            if (is_block && p.mask == DEER_MASK_CAUSAL) limit = min(p.k, i_blk + 1);
            if (limit < ATT_TILE) {                      // ragged or masked tile: hide the columns this row may not see
#pragma unroll
                for (int j = 0; j < ATT_TILE; ++j)
                    if (j >= limit) sr[j] = 0xff800000u;  // -inf
            }
            float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // four chains: one warp per scheduler needs the ILP
#pragma unroll
            for (int j = 0; j < ATT_TILE; j += 4) {
                mx4[0] = fmaxf(mx4[0], __uint_as_float(sr[j]));
                mx4[1] = fmaxf(mx4[1], __uint_as_float(sr[j + 1]));
                mx4[2] = fmaxf(mx4[2], __uint_as_float(sr[j + 2]));
                mx4[3] = fmaxf(mx4[3], __uint_as_float(sr[j + 3]));
            }
            float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
            mx *= p.scale_log2;                           // scale > 0, so the maximum commutes with it
            if (!(mx > -INFINITY)) mx = 0.f;              // lanes without a query row
            // o_done completes one phase per tile, and a parity wait can only tell the current phase from the one
            // before it: every phase is waited for, in order -- phase i-1 (O holds tiles 0..i-1) during tile i.
            bool o_synced = (i == 0);
            if (i == 0) {
                m_run = mx;
            } else if (__any_sync(0xffffffffu, mx > m_run + RESCALE_STEP)) {
                // raise the maximum: O and the row sum shrink by 2^(old - new); O is final up to tile i-1 first
                const float m_new = fmaxf(m_run, mx);
                const float alpha = ex2_approx(m_run - m_new);
                const bool od = mbar_wait(o_done, (uint32_t)(i - 1) & 1u, abort_flag);
                if (!__all_sync(0xffffffffu, od)) { alive = false; break; }
                o_synced = true;
                tcgen05_fence_after();
#pragma unroll
                for (int cc = 0; cc < HD / 32; ++cc) {
                    uint32_t orow[32];
                    TMEM_LD_X32(t_lane + O_COL + cc * 32, orow);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j) orow[j] = __float_as_uint(__uint_as_float(orow[j]) * alpha);
                    TMEM_ST_X32(t_lane + O_COL + cc * 32, orow);
                }
                tmem_wait_st();
                l_run *= alpha;
                m_run = m_new;
            }
            // P = 2^(s * scale - m), two bf16 per TMEM column, in this tile's P buffer
            uint32_t pr[ATT_TILE / 2];
            float sum4[4] = {0.f, 0.f, 0.f, 0.f};
            const float neg_m = -m_run;
#pragma unroll
            for (int j = 0; j < ATT_TILE; j += 2) {
                const float p0 = ex2_approx(fmaf(__uint_as_float(sr[j]), p.scale_log2, neg_m));
                const float p1 = ex2_approx(fmaf(__uint_as_float(sr[j + 1]), p.scale_log2, neg_m));
                sum4[(j >> 1) & 3] += p0 + p1;
                pr[j >> 1] = pack_bf16(p0, p1);
            }
            const float sum = (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
            l_run += sum;
            if (!o_synced) {                              // normally long complete: PV(i-1) was issued a softmax ago
                const bool od = mbar_wait(o_done, (uint32_t)(i - 1) & 1u, abort_flag);
                if (!__all_sync(0xffffffffu, od)) { alive = false; break; }
            }
            TMEM_ST_X32(t_lane + P_COL + buf * (ATT_TILE / 2), pr);
            tmem_wait_st();
            if (tile_valid < ATT_TILE) {
                // V rows beyond the valid tokens hold whatever was in memory; they meet P = 0, which must not
                // meet a NaN.  Zero them once the TMA copies of this slot have landed.
                const bool vf = mbar_wait(v_full(sl), (uint32_t)(i / NSLOT) & 1u, abort_flag);
                if (!__all_sync(0xffffffffu, vf)) { alive = false; break; }
                unsigned char* vt = ring + sl * SLOT_BYTES + K_BYTES;
                const int nz = (ATT_TILE - tile_valid) * 16;           // 16-byte pieces: 2 halves x 8 per token row
                for (int idx = wtid; idx < nz; idx += 128) {
                    const int t = tile_valid + (idx >> 4), half = (idx >> 3) & 1, pc = idx & 7;
                    const int off = is_block ? half * KV_HALF + t * 128
                                             : (t >> 4) * 4096 + ((t >> 3) & 1) * 2048 + half * 1024 + (t & 7) * 128;
                    *reinterpret_cast<uint4*>(vt + off + pc * 16) = make_uint4(0, 0, 0, 0);
                }
                fence_proxy_async_smem();
            }
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(p_ready(buf));
        }

        // ---- partial result of this chunk: O / l and the log2-sum-exp ----
        if (alive) {
            const bool od = mbar_wait(o_done, (uint32_t)(n_tiles - 1) & 1u, abort_flag);
            alive = __all_sync(0xffffffffu, od);
        }
        if (alive) {
            tcgen05_fence_after();
            const float inv = (l_run > 0.f) ? 1.f / l_run : 0.f;
            const size_t n_rows = (size_t)p.B * p.k * p.Hq;
            const size_t orow_idx = (size_t)(b * p.k + (row_valid ? i_blk : 0)) * p.Hq + kvh * p.G + g;
            float* dst = p.part_o + ((size_t)c * n_rows + orow_idx) * HD;
#pragma unroll
            for (int cc = 0; cc < HD / 32; ++cc) {
                uint32_t orow[32];
                TMEM_LD_X32(t_lane + O_COL + cc * 32, orow);
                tmem_wait_ld();
                if (row_valid) {
#pragma unroll
                    for (int j = 0; j < 32; j += 4)
                        *reinterpret_cast<float4*>(dst + cc * 32 + j) =
                            make_float4(__uint_as_float(orow[j]) * inv, __uint_as_float(orow[j + 1]) * inv,
                                        __uint_as_float(orow[j + 2]) * inv, __uint_as_float(orow[j + 3]) * inv);
                }
            }
            if (row_valid) p.part_lse[(size_t)c * n_rows + orow_idx] = (l_run > 0.f) ? m_run + log2f(l_run) : -INFINITY;
        }
    }

    // ---- tear-down ------------------------------------------------------------
    tcgen05_fence_before();
    __syncthreads();
    if (*abort_flag) {
        if (tid == 0) deer_report(p.kv.status, DEER_ERR_TIMEOUT);
        // give copies that are still in flight time to land before the block's shared memory goes away
        for (int i = 0; i < 64; ++i) __nanosleep(10000);
        __syncthreads();
    }
    if (warp == 1) {
        __syncwarp();
        tcgen05_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace umma

bool umma_supported(int D, int G, float scale) { return D == umma::HD && G >= 1 && G <= 128 && scale > 0.f; }

int umma_row_tiles(int k, int G) {
    const int ipt = 128 / G;                 // block rows per row tile
    return (k + ipt - 1) / ipt;
}

int launch_umma(AttnParams p, cudaStream_t st) {
    using namespace umma;
    using sm100::make_map_bf16;
    const int Hkv = p.kv.n_kv_heads;
    p.ipt = 128 / p.G;
    p.row_tiles = umma_row_tiles(p.k, p.G);
    const int box_i = p.ipt < p.k ? p.ipt : p.k;
    const uint64_t rows = (uint64_t)p.B * p.k;

    CUtensorMap tm_q, tm_kb, tm_vb, tm_kp, tm_vp;
    {   // q [B*k][Hq][128]: a box brings G heads of box_i block rows, 64 dims wide -> smem row = i * G + g
        const uint64_t dims[3] = {HD, (uint64_t)p.Hq, rows};
        const uint64_t str[2] = {HD * 2, (uint64_t)p.Hq * HD * 2};
        const uint32_t box[3] = {64, (uint32_t)p.G, (uint32_t)box_i};
        const int rc = make_map_bf16(&tm_q, p.q, 3, dims, str, box);
        if (rc != DEER_OK) return rc;
    }
    {   // k_blk / v_blk [B*k][Hkv][128]: a box brings the k rows of one sequence and KV head
        const uint64_t dims[3] = {HD, (uint64_t)Hkv, rows};
        const uint64_t str[2] = {HD * 2, (uint64_t)Hkv * HD * 2};
        const uint32_t box[3] = {64, 1, (uint32_t)p.k};
        int rc = make_map_bf16(&tm_kb, p.k_blk, 3, dims, str, box);
        if (rc != DEER_OK) return rc;
        rc = make_map_bf16(&tm_vb, p.v_blk, 3, dims, str, box);
        if (rc != DEER_OK) return rc;
    }
    {   // pools [num_pages * Hkv][16 tokens][128 dims] seen as (64 dims, 8 tokens, 2 dim halves, 2 token groups,
        // page x head): one box brings a whole 4 KB page of one KV head as four 1 KB swizzle atoms
        const uint64_t dims[5] = {64, 8, 2, 2, (uint64_t)p.kv.num_pages * Hkv};
        const uint64_t str[4] = {HD * 2, 128, 8 * HD * 2, DEER_PAGE_SIZE * HD * 2};
        const uint32_t box[5] = {64, 8, 2, 2, 1};
        int rc = make_map_bf16(&tm_kp, p.kv.k_pool, 5, dims, str, box);
        if (rc != DEER_OK) return rc;
        rc = make_map_bf16(&tm_vp, p.kv.v_pool, 5, dims, str, box);
        if (rc != DEER_OK) return rc;
    }
    DEER_CUDA(cudaFuncSetAttribute(block_attn_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
    dim3 grid(p.max_chunks, Hkv * p.row_tiles, p.B);
    block_attn_umma_kernel<<<grid, THREADS, SMEM_BYTES, st>>>(tm_q, tm_kb, tm_vb, tm_kp, tm_vp, p);
    DEER_CUDA(cudaGetLastError());
    return DEER_OK;
}

}  // namespace attn
