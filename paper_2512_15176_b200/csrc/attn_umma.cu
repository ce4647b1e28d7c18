// Block attention on the 5th-generation tensor cores (head_dim 128).
//
// Work decomposition.  A unit is one (sequence, KV head, row tile): the query
// rows that share the KV head -- block row i with its G query heads, row =
// (i - i0) * G + g -- sit on the 128 TMEM lanes.  A unit's keys are its cached
// prefix in 64-token tiles plus one more tile, the block rows' own K/V.  The
// tiles of all units, laid end to end, are cut into one equal share per thread
// block (about one block per SM), whatever the sequence lengths are; a share
// crosses unit boundaries, and each (unit, block) piece is a segment.  A unit
// that lies inside one share is written straight to the output; otherwise each
// segment emits a normalised partial output plus its log2-sum-exp, and a small
// merge kernel combines the segments of the units that were split.  With more
// than one row tile per KV head (G * k > 128) the list holds one entry per
// (sequence, KV head) and the thread blocks come in groups of row_tiles: the
// blocks of a group walk the same share, each for its own row tile, so they
// stream the same KV tiles at the same time and the second read is an L2 hit
// rather than a second pass over HBM a hundred megabytes later.
//
// Pipeline.  KV pages stream through a ring of 64-token slots filled by TMA,
// one 4 KB box per page (slot layout below).  S = Q K^T and O += P V are
// tcgen05 MMAs:
//     S (128 x 64, fp32)  = Q [smem, K-major] x K tile [smem, K-major]
//     O (128 x 128, fp32) += P [TMEM, bf16] x V tile [smem, MN-major]
// S has four buffers and P two, so the MMAs run ahead of the softmax.  A thread
// gets a tcgen05.mma accepted only every ~100 cycles whatever its size, so
// three warps issue -- even S tiles, odd S tiles, O -- and their streams
// interleave on the tensor pipe.  The softmax warps hold one row per thread (no
// shuffles); the exponentials of a segment are taken against its first tile's
// row maximum, which is raised only when a later tile's exponentials outgrow
// 2^32 (the accumulator in TMEM is rescaled then, which is rare).
//
// Warp roles: warp 0 = TMA producer, warps 1-2 = issuers of S (warp 1 owns the
// TMEM allocation), warp 3 = issuer of O, warps 4..7 = softmax (one TMEM lane
// quarter each).  Every wait is bounded: a wait that runs out raises the
// block's abort flag and the cache's status word, every role leaves its loops,
// TMEM is freed and the kernel returns.

#include "attn.cuh"
#include "sm100.cuh"

#ifdef DEER_TIMING_PROBES
// Probe table of the attention kernel: row = tile index of block PROBE_BLOCK minus PROBE_TILE0, columns:
// 0 slot free seen by the producer, 1 K landed seen by the S issuer, 2 S committed, 3 S complete seen by the softmax,
// 4 P handed over, 5 P and V seen by the O issuer, 6 O committed.
__device__ long long g_attn_probe[DEER_PROBE_ROWS][DEER_PROBE_COLS];
extern "C" int deer_attn_probe_read(long long* host) {
    return (int)cudaMemcpyFromSymbol(host, g_attn_probe, sizeof(g_attn_probe));
}
#endif
namespace attn {
namespace umma {
constexpr int PROBE_BLOCK = 20, PROBE_TILE0 = 40;      // which block and which of its tiles the probes record

using namespace sm100;

constexpr int HD = 128;                        // head dim
constexpr int NSLOT = 4;                       // ring slots of 64 tokens (a fifth made no measurable difference)
constexpr int NS = 4;                          // S buffers
constexpr int Q_HALF = 128 * 128;              // [128 rows][64 d] bf16
constexpr int Q_BYTES = 2 * Q_HALF;            // 32 KB, two of them: the next segment's Q loads early
constexpr int KV_HALF = ATT_TILE * 128;        // [64 tokens][64 d] bf16 = 8 KB
constexpr int K_BYTES = 2 * KV_HALF;           // 16 KB
constexpr int SLOT_BYTES = 2 * K_BYTES;        // K tile then V tile
constexpr int THREADS = 256;
constexpr int TMEM_COLS = 512;                 // S0..S3 [0,256)  P0 [256,288)  P1 [288,320)  O [384,512)
constexpr int P_COL = 256;
constexpr int O_COL = 384;
constexpr int MAX_SEGS = 48;                   // segments listed at a time; longer shares go in several rounds
constexpr float RESCALE_SUM = 4294967296.f;    // 2^32: a row sum over one tile beyond this raises the running maximum
// Slot layout.  A K (or V) tile of 64 tokens x 128 dims is 16 KB of 1 KB swizzle atoms (8 tokens x 64 dims).
//   prefix tile: [page 0..3][token group 0..1][dim half 0..1][8 tokens][128 B] -- what one 5-D TMA box per page
//                writes; atoms of one dim half are 2 KB apart along the tokens, the two halves 1 KB apart.
//   block tile:  [dim half 0..1][64 tokens][128 B] -- the block's own rows, from k_blk / v_blk; atoms 1 KB apart
//                along the tokens, the halves 8 KB apart.

// mbarrier indices
constexpr int BAR_Q_FULL = 0;                  // [2]
constexpr int BAR_Q_EMPTY = 2;                 // [2]  count 2: both S issuers
constexpr int BAR_K_FULL = 4;                  // [NSLOT]
constexpr int BAR_V_FULL = BAR_K_FULL + NSLOT;
constexpr int BAR_SLOT_EMPTY = BAR_V_FULL + NSLOT;
constexpr int BAR_S_FULL = BAR_SLOT_EMPTY + NSLOT;   // [NS]
constexpr int BAR_S_FREE = BAR_S_FULL + NS;          // [NS]  count 4: the softmax warps
constexpr int BAR_P_READY = BAR_S_FREE + NS;         // [2]   count 4
constexpr int BAR_O_DONE = BAR_P_READY + 2;
constexpr int N_BARS = BAR_O_DONE + 1;

struct Seg {             // one (unit, block) piece
    int b, hr;           // sequence index in the call; KV head * row_tiles + row tile
    int t_a, t_b;        // tile range within the unit; tile ceil(n / 64) is the block rows' own K/V
    int n, s;            // committed length and cache slot of the sequence
    long long u0;        // flattened position of the unit's first tile
};

constexpr int SMEM_BYTES = 2 * Q_BYTES + NSLOT * SLOT_BYTES + 1024 /*alignment slack*/ + N_BARS * 8 + 32 + MAX_SEGS * (int)sizeof(Seg);

__device__ __forceinline__ float ex2_approx(float x) {   // 2^x, one MUFU op; -inf gives 0
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Tiles of sequence b: its prefix tiles plus the block tile; 0 if the sequence cannot be used.
__device__ __forceinline__ int seq_tiles(const AttnParams& p, int b, int* n_out, int* s_out) {
    const int s = p.seq_ids[b];
    int n = -1;
    if (s >= 0 && s < p.kv.max_seqs) n = p.kv.seq_len[s];
    if (n_out) *n_out = n;
    if (s_out) *s_out = s;
    if (n < 0 || n > p.max_seq_len) return 0;
    return (n + ATT_TILE - 1) / ATT_TILE + 1;
}

// Share of thread block j out of nc over T tiles: [share_begin(j), share_begin(j + 1)).
__device__ __forceinline__ long long share_begin(long long T, int j, int nc) { return T * j / nc; }

// Warp-collective: lists up to MAX_SEGS segments of the flattened tile range [cursor, end) into segs[], in order.
// Returns their number; *cursor_out is where the next round starts (== end when the share is exhausted).
__device__ int build_segments(const AttnParams& p, int HL, int rt, long long cursor, long long end, Seg* segs,
                              long long* cursor_out, int lane) {
    int n_seg = 0;
    long long base = 0;                                   // flattened position of sequence b0's first tile
    long long next_cursor = end;
    bool cut = false;
    for (int b0 = 0; b0 < p.B && base < end && n_seg < MAX_SEGS; b0 += 32) {
        const int b = b0 + lane;
        int n = 0, s = 0;
        const int tiles = (b < p.B) ? seq_tiles(p, b, &n, &s) : 0;
        if (b < p.B && tiles == 0) deer_report(p.kv.status, DEER_ERR_INVALID_ARG);
        const long long span = (long long)tiles * HL;     // tiles this sequence contributes to the list
        long long incl = span;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const long long t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        const long long my0 = base + incl - span, my1 = base + incl;
        // units of my sequence that meet [cursor, end)
        int hr_lo = 0, hr_hi = -1;
        if (tiles > 0 && my1 > cursor && my0 < end) {
            hr_lo = cursor > my0 ? (int)((cursor - my0) / tiles) : 0;
            hr_hi = (int)(((end < my1 ? end : my1) - 1 - my0) / tiles);
        }
        const int cnt = hr_hi - hr_lo + 1 > 0 ? hr_hi - hr_lo + 1 : 0;
        int cincl = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, cincl, o);
            if (lane >= o) cincl += t;
        }
        const int off = n_seg + cincl - cnt;
        for (int e = 0; e < cnt; ++e) {
            const int idx = off + e;
            const int hr = hr_lo + e;
            const long long u0 = my0 + (long long)hr * tiles;
            if (idx < MAX_SEGS) {
                Seg sg;
                sg.b = b;
                sg.hr = hr * p.row_tiles + rt;
                sg.t_a = cursor > u0 ? (int)(cursor - u0) : 0;
                sg.t_b = end < u0 + tiles ? (int)(end - u0) : tiles;
                sg.n = n;
                sg.s = s;
                sg.u0 = u0;
                segs[idx] = sg;
            } else if (idx == MAX_SEGS) {
                next_cursor = u0;                          // the first segment that did not fit starts the next round
            }
        }
        const int total = __shfl_sync(0xffffffffu, cincl, 31);
        // at most one lane owns index MAX_SEGS; share its cursor
        const unsigned who = __ballot_sync(0xffffffffu, off <= MAX_SEGS && MAX_SEGS < off + cnt);
        if (who) next_cursor = __shfl_sync(0xffffffffu, next_cursor, __ffs(who) - 1);
        n_seg = n_seg + total < MAX_SEGS ? n_seg + total : MAX_SEGS;
        base += __shfl_sync(0xffffffffu, incl, 31);
        if (who) {
            cut = true;
            break;
        }
    }
    if (!cut && n_seg == MAX_SEGS) next_cursor = base < end ? base : end;   // the list filled up exactly at a sequence boundary
    *cursor_out = next_cursor;
    return n_seg;
}

__global__ void __launch_bounds__(THREADS, 1)
block_attn_umma_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kb,
                       const __grid_constant__ CUtensorMap tm_vb, const __grid_constant__ CUtensorMap tm_kpool,
                       const __grid_constant__ CUtensorMap tm_vpool, const AttnParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char* sQ = smem;                                  // [2 buffers][2 halves][128 rows][128 B]
    unsigned char* ring = smem + 2 * Q_BYTES;                  // [NSLOT][K tile 16 KB][V tile 16 KB]
    uint64_t* bars = reinterpret_cast<uint64_t*>(ring + NSLOT * SLOT_BYTES);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + N_BARS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile int* sh_nseg = reinterpret_cast<volatile int*>(tmem_slot + 2);
    volatile long long* sh_cursor = reinterpret_cast<volatile long long*>(tmem_slot + 4);
    Seg* segs = reinterpret_cast<Seg*>(tmem_slot + 8);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int Hkv = p.kv.n_kv_heads;
    const int HR = Hkv * p.row_tiles;                          // units per sequence
    const int j = blockIdx.x;
    const int jg = j / p.row_tiles, rt_blk = j % p.row_tiles;  // group of blocks that walk the same share; my row tile
    const int ncg = p.nc / p.row_tiles;                        // groups (nc is a multiple of row_tiles)

    // ---- what needs no input: barriers, tensor-map prefetch ----
    const uint32_t bar_base = smem_u32(bars);
    auto bar = [&](int idx) { return bar_base + 8u * idx; };
    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(BAR_Q_FULL + i), 1);
            mbar_init(bar(BAR_Q_EMPTY + i), 2);
            mbar_init(bar(BAR_P_READY + i), 4);
        }
        for (int sl = 0; sl < NSLOT; ++sl) {
            mbar_init(bar(BAR_K_FULL + sl), 1);
            mbar_init(bar(BAR_V_FULL + sl), 1);
            mbar_init(bar(BAR_SLOT_EMPTY + sl), 1);
        }
        for (int i = 0; i < NS; ++i) {
            mbar_init(bar(BAR_S_FULL + i), 1);
            mbar_init(bar(BAR_S_FREE + i), 4);
        }
        mbar_init(bar(BAR_O_DONE), 1);
        *abort_flag = 0;
        mbar_init_fence();
    }
    if (warp == 0 && lane == 0) {
        prefetch_tensormap(&tm_q);
        prefetch_tensormap(&tm_kpool);
        prefetch_tensormap(&tm_vpool);
    }
    pdl_trigger();
    pdl_wait();                                                // lengths, page table, the block's rows: written by what ran before

    // ---- this block's share of the flattened tile list ----
    long long T = 0;
    for (int b = lane; b < p.B; b += 32) {
        const int tiles = seq_tiles(p, b, nullptr, nullptr);
        T += tiles;
        // a sequence that cannot be used has no tiles, so no block will write its units' merge entries: do it here
        if (tiles == 0 && j == 0 && warp == 0)
            for (int hr = 0; hr < HR; ++hr) p.unit_parts[(size_t)b * HR + hr] = make_int2(-1, -1);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) T += __shfl_xor_sync(0xffffffffu, T, o);
    T *= Hkv;                                                  // list entries: (sequence, KV head) x tiles
    const long long share_lo = share_begin(T, jg, ncg), share_hi = share_begin(T, jg + 1, ncg);
    if (j == 0 && tid == 0) *p.total_tiles = T;                // for the merge kernel
    if (share_hi <= share_lo) return;                          // nothing to do (fewer tiles than blocks)

    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t q_addr = smem_u32(sQ);
    const uint32_t ring_addr = smem_u32(ring);
    const int q_box_rows = p.G * min(p.ipt, p.k);              // rows one Q box brings

    // Counters that run across segments and rounds; every role advances its own copy identically.
    int it = 0;          // tiles so far: ring slot it % NSLOT, S buffer it % NS, P buffer it & 1, o_done phase it
    int sg = 0;          // segments so far: Q buffer sg & 1
    long long cursor = share_lo;
    while (cursor < share_hi) {
        // ---- list the next segments of the share (warp 0), then every role walks the list ----
        if (warp == 0) {
            long long next;
            const int ns = build_segments(p, Hkv, rt_blk, cursor, share_hi, segs, &next, lane);
            if (lane == 0) {
                *sh_nseg = ns;
                *sh_cursor = next;
            }
        }
        __syncthreads();
        const int n_seg = *sh_nseg;
        cursor = *sh_cursor;

        if (warp == 0) {
            // ---------------- TMA producer ----------------
            // Lanes 0..7 each issue one copy of a tile: lane = is_v * 4 + page-in-tile (block tile: is_v * 4 + half).
            // Page ids are fetched two tiles ahead (lane L holds the id of page L & 3) and validated only when used.
            const int pj = lane & 3, is_v = (lane >> 2) & 1;
            bool ok = true;
            for (int si = 0; si < n_seg && ok; ++si, ++sg) {
                const Seg g = segs[si];
                const int kvh = g.hr / p.row_tiles, i0 = (g.hr % p.row_tiles) * p.ipt;
                const int last_tile = (g.n + ATT_TILE - 1) / ATT_TILE;       // index of the block tile
                const int32_t* pt_row = p.kv.page_table + (size_t)g.s * p.kv.max_pages;
                auto page_of = [&](int t) -> int {
                    if (t >= last_tile || t >= g.t_b || lane >= 8) return 0;
                    const int lp = t * (ATT_TILE / DEER_PAGE_SIZE) + pj;
                    if (lp * DEER_PAGE_SIZE >= g.n || lp >= p.kv.max_pages) return -1;
                    return pt_row[lp];
                };
                int pg_cur = page_of(g.t_a), pg_next = page_of(g.t_a + 1);
                // this segment's query rows
                const int qb = sg & 1;
                int okq = 1;
                if (lane == 0) okq = mbar_wait(bar(BAR_Q_EMPTY + qb), ((uint32_t)(sg >> 1) & 1u) ^ 1u, abort_flag) ? 1 : 0;
                if (!__shfl_sync(0xffffffffu, okq, 0)) { ok = false; break; }
                if (lane == 0) {
                    mbar_expect_tx(bar(BAR_Q_FULL + qb), (uint32_t)(2 * q_box_rows * 128));
                    tma_load_3d(q_addr + qb * Q_BYTES, &tm_q, 0, kvh * p.G, g.b * p.k + i0, bar(BAR_Q_FULL + qb));
                    tma_load_3d(q_addr + qb * Q_BYTES + Q_HALF, &tm_q, 64, kvh * p.G, g.b * p.k + i0, bar(BAR_Q_FULL + qb));
                }
                for (int t = g.t_a; t < g.t_b; ++t, ++it) {
                    const int sl = it % NSLOT;
                    int pg = pg_cur;
                    pg_cur = pg_next;
                    pg_next = page_of(t + 2);
                    int oks = 1;
                    if (lane == 0) oks = mbar_wait(bar(BAR_SLOT_EMPTY + sl), ((uint32_t)(it / NSLOT) & 1u) ^ 1u, abort_flag) ? 1 : 0;
                    if (!__shfl_sync(0xffffffffu, oks, 0)) { ok = false; break; }
                    DEER_PROBE(g_attn_probe, lane == 0 && blockIdx.x == PROBE_BLOCK, it - PROBE_TILE0, 0);
                    const uint32_t kdst = ring_addr + sl * SLOT_BYTES;
                    const uint32_t dst = is_v ? kdst + K_BYTES : kdst;
                    const uint32_t fb = bar((is_v ? BAR_V_FULL : BAR_K_FULL) + sl);
                    if (t < last_tile) {
                        const int np = (min(ATT_TILE, g.n - t * ATT_TILE) + DEER_PAGE_SIZE - 1) / DEER_PAGE_SIZE;
                        if (lane == 0) {
                            mbar_expect_tx(bar(BAR_K_FULL + sl), (uint32_t)np * 4096u);
                            mbar_expect_tx(bar(BAR_V_FULL + sl), (uint32_t)np * 4096u);
                        }
                        __syncwarp();
                        if (lane < 8 && pj < np) {
                            if (pg < 0 || pg >= p.kv.num_pages) {
                                deer_report(p.kv.status, DEER_ERR_BAD_PAGE);
                                pg = 0;         // keep the copy inside the pool; the status word flags the result
                            }
                            tma_load_5d(dst + pj * 4096, is_v ? &tm_vpool : &tm_kpool, 0, 0, 0, 0, pg * Hkv + kvh, fb);
                        }
                    } else {
                        // the block rows' own keys and values: k rows straight from k_blk / v_blk
                        if (lane == 0) {
                            mbar_expect_tx(bar(BAR_K_FULL + sl), (uint32_t)(2 * p.k * 128));
                            mbar_expect_tx(bar(BAR_V_FULL + sl), (uint32_t)(2 * p.k * 128));
                        }
                        __syncwarp();
                        if (lane < 8 && pj < 2) tma_load_3d(dst + pj * KV_HALF, is_v ? &tm_vb : &tm_kb, pj * 64, kvh, g.b * p.k, fb);
                    }
                }
            }
        } else if (warp <= 2) {
            // ---------------- issuers of S = Q K^T: warp 1 takes the even tiles, warp 2 the odd ones ----------------
            if (lane == 0) {
                const uint32_t idesc_qk = make_idesc_bf16(ATT_TILE, 0);   // S: N = 64 tokens, both operands K-major
                // Operand descriptors are built once; inside the loops only their 16-byte-unit address field moves.
                const uint64_t q_desc = smem_desc_sw128_kmajor(q_addr);
                const uint64_t k_desc_pre = smem_desc_sw128(ring_addr, 16, 2048), k_desc_blk = smem_desc_sw128(ring_addr, 16, 1024);
                bool ok = true;
                for (int si = 0; si < n_seg && ok; ++si, ++sg) {
                    const Seg g = segs[si];
                    const int last_tile = (g.n + ATT_TILE - 1) / ATT_TILE;
                    const int qb = sg & 1;
                    if (!mbar_wait(bar(BAR_Q_FULL + qb), (uint32_t)(sg >> 1) & 1u, abort_flag)) { ok = false; break; }
                    const uint64_t qd = q_desc + (uint64_t)((qb * Q_BYTES) >> 4);
                    for (int t = g.t_a; t < g.t_b; ++t, ++it) {
                        if ((it & 1) != warp - 1) continue;
                        const int sl = it % NSLOT, sb = it % NS;
                        // S buffer free (the softmax warps have read its previous tile), K tile landed
                        if (!mbar_wait(bar(BAR_S_FREE + sb), ((uint32_t)(it / NS) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                        if (!mbar_wait(bar(BAR_K_FULL + sl), (uint32_t)(it / NSLOT) & 1u, abort_flag)) { ok = false; break; }
                        DEER_PROBE(g_attn_probe, blockIdx.x == PROBE_BLOCK, it - PROBE_TILE0, 1);
                        tcgen05_fence_after();
                        const uint32_t d_tmem = tmem_base + (uint32_t)(sb * ATT_TILE);
                        const bool blk = (t == last_tile);
                        const uint64_t kd = (blk ? k_desc_blk : k_desc_pre) + (uint64_t)((sl * SLOT_BYTES) >> 4);
                        const uint64_t half16 = blk ? (KV_HALF >> 4) : (1024 >> 4);     // distance between the dim halves
#pragma unroll
                        for (int kk = 0; kk < HD / 16; ++kk) {      // 8 k-steps of 16 dims, 4 per 64-wide half
                            const uint64_t ad = qd + (uint64_t)(((kk >> 2) * Q_HALF + (kk & 3) * 32) >> 4);
                            const uint64_t bd = kd + ((kk >> 2) ? half16 : 0) + (uint64_t)(((kk & 3) * 32) >> 4);
                            umma_bf16_ss(d_tmem, ad, bd, idesc_qk, kk != 0 ? 1u : 0u);
                        }
                        umma_commit(bar(BAR_S_FULL + sb));
                        DEER_PROBE(g_attn_probe, blockIdx.x == PROBE_BLOCK, it - PROBE_TILE0, 2);
                    }
                    // Q buffer reusable once this warp's MMAs of the segment are done (the other S issuer says the same)
                    if (ok) umma_commit(bar(BAR_Q_EMPTY + qb));
                }
            }
        } else if (warp == 3) {
            // ---------------- issuer of O += P V ----------------
            if (lane == 0) {
                const uint32_t idesc_pv = make_idesc_bf16(HD, 1);         // O: N = 128 dims, V is MN-major
                const uint64_t v_desc_pre = smem_desc_sw128(ring_addr + K_BYTES, 1024, 2048);
                const uint64_t v_desc_blk = smem_desc_sw128(ring_addr + K_BYTES, KV_HALF, 1024);
                bool ok = true;
                for (int si = 0; si < n_seg && ok; ++si, ++sg) {
                    const Seg g = segs[si];
                    const int last_tile = (g.n + ATT_TILE - 1) / ATT_TILE;
                    for (int t = g.t_a; t < g.t_b; ++t, ++it) {
                        const int sl = it % NSLOT;
                        if (!mbar_wait(bar(BAR_P_READY + (it & 1)), (uint32_t)(it >> 1) & 1u, abort_flag)) { ok = false; break; }
                        if (!mbar_wait(bar(BAR_V_FULL + sl), (uint32_t)(it / NSLOT) & 1u, abort_flag)) { ok = false; break; }
                        DEER_PROBE(g_attn_probe, blockIdx.x == PROBE_BLOCK, it - PROBE_TILE0, 5);
                        tcgen05_fence_after();
                        const uint32_t p_tmem = tmem_base + (uint32_t)(P_COL + (it & 1) * (ATT_TILE / 2));
                        const bool blk = (t == last_tile);
                        // 16 tokens per MMA = two 8-token atoms; lbo = distance between the dim halves, sbo = between token atoms
                        const uint64_t vd = (blk ? v_desc_blk : v_desc_pre) + (uint64_t)((sl * SLOT_BYTES) >> 4);
                        const uint64_t step16 = blk ? (2048 >> 4) : (4096 >> 4);
                        const uint32_t keep = (t == g.t_a) ? 0u : 1u;      // a segment starts a new accumulation
#pragma unroll
                        for (int kk = 0; kk < ATT_TILE / 16; ++kk)
                            umma_bf16_ts(tmem_base + O_COL, p_tmem + kk * 8, vd + kk * step16, idesc_pv, kk != 0 ? 1u : keep);
                        // S of this tile was complete before its softmax, hence before this point: K and V are both consumed
                        umma_commit(bar(BAR_SLOT_EMPTY + sl));
                        umma_commit(bar(BAR_O_DONE));             // phase `it` of o_done: O includes this tile
                        DEER_PROBE(g_attn_probe, blockIdx.x == PROBE_BLOCK, it - PROBE_TILE0, 6);
                    }
                }
            }
        } else {
            // ---------------- softmax: 4 warps, one TMEM lane quarter each, one query row per thread ----------------
            const int quarter = warp & 3;
            const int row = quarter * 32 + lane;
            const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
            const int wtid = tid - 128;                       // 0..127 within the softmax warps
            bool alive = true;
            for (int si = 0; si < n_seg && alive; ++si, ++sg) {
                const Seg g = segs[si];
                const int kvh = g.hr / p.row_tiles, rt = g.hr % p.row_tiles;
                const int i0 = rt * p.ipt;                    // first block row of this row tile
                const int ni = min(p.ipt, p.k - i0);          // block rows in it
                const int i_blk = i0 + row / p.G;             // block row of this query row
                const bool row_valid = row < ni * p.G;
                const int last_tile = (g.n + ATT_TILE - 1) / ATT_TILE;
                uint32_t present, decoded;
                row_state_sets(p.row_state, g.b, p.k, lane, &present, &decoded);
                const uint32_t my_cols = visible_rows(p.mask, i_blk, (p.row_state && row_valid) ? p.row_state[(size_t)g.b * p.k + i_blk] : 1,
                                                      present, decoded);

                // append the block's K/V rows to the cache (once per (sequence, KV head): with the block tile of row tile 0);
                // with row states the decoded rows only
                if (p.append && rt == 0 && g.t_b == last_tile + 1) {
                    constexpr int PIECES = HD / 8;
                    const int32_t* pt_row = p.kv.page_table + (size_t)g.s * p.kv.max_pages;
                    for (int idx = wtid; idx < p.k * PIECES; idx += 128) {
                        const int jr = idx / PIECES, pc = idx % PIECES;
                        if (p.row_state && !((decoded >> jr) & 1u)) continue;
                        const int t = g.n + jr;
                        const int lp = t >> 4;
                        const int pg = (lp < p.kv.max_pages) ? pt_row[lp] : -1;
                        if (pg < 0 || pg >= p.kv.num_pages) {
                            deer_report(p.kv.status, DEER_ERR_BAD_PAGE);
                            continue;
                        }
                        const size_t src = ((size_t)(g.b * p.k + jr) * Hkv + kvh) * HD + pc * 8;
                        const size_t dst = (((size_t)pg * Hkv + kvh) * DEER_PAGE_SIZE + (t & 15)) * HD + pc * 8;
                        *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.kv.k_pool) + dst) =
                            *reinterpret_cast<const uint4*>(p.k_blk + src);
                        *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.kv.v_pool) + dst) =
                            *reinterpret_cast<const uint4*>(p.v_blk + src);
                    }
                }

                float m_run = 0.f, l_run = 0.f;               // running maximum (log2 domain, scaled) and row sum
                for (int t = g.t_a; t < g.t_b; ++t, ++it) {
                    const int sb = it % NS, pb = it & 1, sl = it % NSLOT;
                    const bool got = mbar_wait(bar(BAR_S_FULL + sb), (uint32_t)(it / NS) & 1u, abort_flag);
                    if (!__all_sync(0xffffffffu, got)) { alive = false; break; }   // warp-uniform: the aligned TMEM ops stay converged
                    DEER_PROBE(g_attn_probe, wtid == 0 && blockIdx.x == PROBE_BLOCK, it - PROBE_TILE0, 3);
                    tcgen05_fence_after();
                    uint32_t sr[ATT_TILE];
                    TMEM_LD_X32(t_lane + sb * ATT_TILE, (sr));
                    TMEM_LD_X32(t_lane + sb * ATT_TILE + 32, (sr + 32));
                    tmem_wait_ld();
                    tcgen05_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(BAR_S_FREE + sb));            // the S buffer may take tile it + NS

                    // columns this row may see: the valid tokens of a prefix tile, or the block rows the mask allows
                    const bool is_block = (t == last_tile);
                    const int tile_valid = is_block ? p.k : min(ATT_TILE, g.n - t * ATT_TILE);
                    if (is_block) {                           // the block rows' own tile: k <= 32 columns, a bit per column
#pragma unroll
                        for (int c = 0; c < ATT_TILE; ++c)
                            if (c >= 32 || c >= p.k || !((my_cols >> (c & 31)) & 1u)) sr[c] = 0xff800000u;   // -inf
                    } else if (tile_valid < ATT_TILE) {       // ragged prefix tile: hide the columns beyond the sequence
#pragma unroll
                        for (int c = 0; c < ATT_TILE; ++c)
                            if (c >= tile_valid) sr[c] = 0xff800000u;
                    }
                    // Row maximum of this tile (log2 domain, scaled); four chains: one warp per scheduler needs the ILP.
                    auto tile_max = [&]() -> float {
                        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                        for (int c = 0; c < ATT_TILE; c += 4) {
                            mx4[0] = fmaxf(mx4[0], __uint_as_float(sr[c]));
                            mx4[1] = fmaxf(mx4[1], __uint_as_float(sr[c + 1]));
                            mx4[2] = fmaxf(mx4[2], __uint_as_float(sr[c + 2]));
                            mx4[3] = fmaxf(mx4[3], __uint_as_float(sr[c + 3]));
                        }
                        float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
                        mx *= p.scale_log2;                   // scale > 0, so the maximum commutes with it
                        return (mx > -INFINITY) ? mx : 0.f;   // lanes without a query row, rows that see nothing here
                    };
                    // P = 2^(s * scale - m), two bf16 per TMEM column, and the row's sum over this tile
                    uint32_t pr[ATT_TILE / 2];
                    float tile_sum;
                    auto exponentials = [&]() {
                        float sum4[4] = {0.f, 0.f, 0.f, 0.f};
                        const float neg_m = -m_run;
#pragma unroll
                        for (int c = 0; c < ATT_TILE; c += 2) {
                            const float p0 = ex2_approx(fmaf(__uint_as_float(sr[c]), p.scale_log2, neg_m));
                            const float p1 = ex2_approx(fmaf(__uint_as_float(sr[c + 1]), p.scale_log2, neg_m));
                            sum4[(c >> 1) & 3] += p0 + p1;
                            pr[c >> 1] = pack_bf16(p0, p1);
                        }
                        tile_sum = (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
                    };

                    // The reference point m of a segment is its first tile's row maximum.  Subtracting a maximum only
                    // keeps the exponentials in range -- the quotient O / l does not depend on m -- so later tiles
                    // are taken against the same m without looking for their maximum, and m is raised (O and l
                    // rescaled, as any online softmax does) only when a row's sum over a tile shows that its
                    // exponentials have grown past 2^32 (or are not finite): rare, and then the tile is redone.
                    // o_done completes one phase per tile, and a parity wait can only tell the current phase from the
                    // one before it: every phase is waited for, in order -- phase it-1 during tile it.
                    bool o_synced = (it == 0);
                    if (t == g.t_a) m_run = tile_max();       // a segment starts a new accumulation
                    exponentials();
                    if (__any_sync(0xffffffffu, !(tile_sum < RESCALE_SUM))) {
                        const float m_new = fmaxf(m_run, tile_max());
                        const float alpha = ex2_approx(m_run - m_new);
                        const bool od = o_synced || mbar_wait(bar(BAR_O_DONE), (uint32_t)(it - 1) & 1u, abort_flag);
                        if (!__all_sync(0xffffffffu, od)) { alive = false; break; }
                        o_synced = true;
                        tcgen05_fence_after();
                        if (t != g.t_a) {                     // O holds the segment's tiles so far: shrink it by 2^(old - new)
#pragma unroll
                            for (int cc = 0; cc < HD / 32; ++cc) {
                                uint32_t orow[32];
                                TMEM_LD_X32(t_lane + O_COL + cc * 32, orow);
                                tmem_wait_ld();
#pragma unroll
                                for (int c = 0; c < 32; ++c) orow[c] = __float_as_uint(__uint_as_float(orow[c]) * alpha);
                                TMEM_ST_X32(t_lane + O_COL + cc * 32, orow);
                            }
                            tmem_wait_st();
                        }
                        l_run *= alpha;
                        m_run = m_new;
                        exponentials();
                    }
                    l_run += tile_sum;
                    if (!o_synced) {                          // normally long complete; also frees this P buffer (tile it-2)
                        const bool od = mbar_wait(bar(BAR_O_DONE), (uint32_t)(it - 1) & 1u, abort_flag);
                        if (!__all_sync(0xffffffffu, od)) { alive = false; break; }
                    }
                    TMEM_ST_X32(t_lane + P_COL + pb * (ATT_TILE / 2), pr);
                    tmem_wait_st();
                    if (tile_valid < ATT_TILE) {
                        // V rows beyond the valid tokens hold whatever was in memory; they meet P = 0, which must not
                        // meet a NaN.  Zero them once the TMA copies of this slot have landed.
                        const bool vf = mbar_wait(bar(BAR_V_FULL + sl), (uint32_t)(it / NSLOT) & 1u, abort_flag);
                        if (!__all_sync(0xffffffffu, vf)) { alive = false; break; }
                        unsigned char* vt = ring + sl * SLOT_BYTES + K_BYTES;
                        const int nz = (ATT_TILE - tile_valid) * 16;      // 16-byte pieces: 2 halves x 8 per token row
                        for (int idx = wtid; idx < nz; idx += 128) {
                            const int tk = tile_valid + (idx >> 4), half = (idx >> 3) & 1, pc = idx & 7;
                            const int off = is_block ? half * KV_HALF + tk * 128
                                                     : (tk >> 4) * 4096 + ((tk >> 3) & 1) * 2048 + half * 1024 + (tk & 7) * 128;
                            *reinterpret_cast<uint4*>(vt + off + pc * 16) = make_uint4(0, 0, 0, 0);
                        }
                        if (is_block && p.row_state) {        // so do the rows of positions that hold nothing
                            for (int idx = wtid; idx < p.k * 16; idx += 128) {
                                const int tk = idx >> 4, half = (idx >> 3) & 1, pc = idx & 7;
                                if (!((present >> tk) & 1u))
                                    *reinterpret_cast<uint4*>(vt + half * KV_HALF + tk * 128 + pc * 16) = make_uint4(0, 0, 0, 0);
                            }
                        }
                        fence_proxy_async_smem();
                    }
                    tcgen05_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(BAR_P_READY + pb));
                    DEER_PROBE(g_attn_probe, wtid == 0 && blockIdx.x == PROBE_BLOCK, it - PROBE_TILE0, 4);
                }
                if (!alive) break;

                // ---- this segment's result ----
                const bool od = mbar_wait(bar(BAR_O_DONE), (uint32_t)(it - 1) & 1u, abort_flag);
                if (!__all_sync(0xffffffffu, od)) { alive = false; break; }
                tcgen05_fence_after();
                const float inv = (l_run > 0.f) ? 1.f / l_run : 0.f;
                const int hq = kvh * p.G + row % p.G;
                const size_t unit = (size_t)g.b * HR + g.hr;
                const bool whole = (g.t_a == 0 && g.t_b == last_tile + 1);     // the unit has no other segment
                if (whole) {
                    // straight to the output: out[b][i][hq][:] in bf16
                    __nv_bfloat16* dst = p.out + ((size_t)(g.b * p.k + (row_valid ? i_blk : 0)) * p.Hq + hq) * HD;
#pragma unroll
                    for (int cc = 0; cc < HD / 32; ++cc) {
                        uint32_t orow[32];
                        TMEM_LD_X32(t_lane + O_COL + cc * 32, orow);
                        tmem_wait_ld();
                        if (row_valid) {
#pragma unroll
                            for (int c = 0; c < 32; c += 8) {
                                uint4 v;
                                v.x = pack_bf16(__uint_as_float(orow[c]) * inv, __uint_as_float(orow[c + 1]) * inv);
                                v.y = pack_bf16(__uint_as_float(orow[c + 2]) * inv, __uint_as_float(orow[c + 3]) * inv);
                                v.z = pack_bf16(__uint_as_float(orow[c + 4]) * inv, __uint_as_float(orow[c + 5]) * inv);
                                v.w = pack_bf16(__uint_as_float(orow[c + 6]) * inv, __uint_as_float(orow[c + 7]) * inv);
                                *reinterpret_cast<uint4*>(dst + cc * 32 + c) = v;
                            }
                        }
                    }
                    tcgen05_fence_before();
                    if (wtid == 0) p.unit_parts[unit] = make_int2(-1, -1);      // nothing for the merge kernel to do
                    continue;
                }
                // partial result: O / l and the log2-sum-exp, in slot ((sequence, KV head) index + group index, row tile)
                {
                    const size_t slot = ((size_t)g.b * Hkv + kvh + jg) * p.row_tiles + rt;
                    float* dst = p.part_o + (slot * 128 + row) * HD;
#pragma unroll
                    for (int cc = 0; cc < HD / 32; ++cc) {
                        uint32_t orow[32];
                        TMEM_LD_X32(t_lane + O_COL + cc * 32, orow);
                        tmem_wait_ld();
                        if (row_valid) {
#pragma unroll
                            for (int c = 0; c < 32; c += 4)
                                *reinterpret_cast<float4*>(dst + cc * 32 + c) =
                                    make_float4(__uint_as_float(orow[c]) * inv, __uint_as_float(orow[c + 1]) * inv,
                                                __uint_as_float(orow[c + 2]) * inv, __uint_as_float(orow[c + 3]) * inv);
                        }
                    }
                    if (row_valid) p.part_lse[slot * 128 + row] = (l_run > 0.f) ? m_run + log2f(l_run) : -INFINITY;
                    tcgen05_fence_before();                   // the next segment's first PV overwrites O after p_ready
                }
                // the segment that holds the unit's first tile tells the merge kernel which blocks share the unit
                if (g.t_a == 0 && wtid == 0) {
                    const int tiles_u = last_tile + 1;
                    const int j_lo = (int)(((g.u0 + 1) * ncg + T - 1) / T) - 1;           // last group starting at or before u0
                    const int j_hi = (int)(((g.u0 + tiles_u) * ncg + T - 1) / T) - 1;     // last group starting inside the unit
                    p.unit_parts[unit] = make_int2(j_lo, j_hi);
                }
            }
        }
        // every role is done with this list before warp 0 rewrites it
        __syncthreads();
        if (*abort_flag) break;
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

// Combines the segments of the units that were cut.  One thread block per (unit, 8 * R of its rows); a warp takes R
// rows at a time so that their loads are in flight together (R = 4, or 1 when that is what it takes to fill the GPU).
// unit_parts[u] = (first, last) block group that holds a piece of unit u, or first < 0 when the unit was written
// directly.
template <int R>
__global__ void __launch_bounds__(256) attn_umma_merge_kernel(const AttnParams p) {
    constexpr int BPU = 128 / (8 * R);                            // thread blocks per unit
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int unit = blockIdx.x / BPU;
    const int Hkv = p.kv.n_kv_heads, HR = Hkv * p.row_tiles;
    const int b = unit / HR, hr = unit % HR;
    pdl_trigger();
    pdl_wait();                                                   // the attention kernel's partial results
    // written by the block that holds the unit's first tile (by block 0 for a sequence that was skipped)
    const int2 parts = p.unit_parts[unit];
    if (parts.x < 0) return;
    const int kvh = hr / p.row_tiles, rt = hr % p.row_tiles;
    const int i0 = rt * p.ipt;
    const int n_rows_u = min(p.ipt, p.k - i0) * p.G;
    const int r0 = ((blockIdx.x % BPU) * 8 + warp) * R;           // this warp's rows r0 .. r0 + R - 1
    if (r0 >= n_rows_u) return;
    const int j_lo = parts.x, nj = parts.y - parts.x + 1;
    const int RT = p.row_tiles, ncg = p.nc / RT;
    // the pieces of a unit sit RT slots apart
    const size_t slot0 = ((size_t)b * Hkv + kvh + j_lo) * RT + rt;
    const float* __restrict__ lse_base = p.part_lse + slot0 * 128;
    const float* __restrict__ o_base = p.part_o + slot0 * 128 * HD;
    const size_t lse_step = (size_t)RT * 128, o_step = (size_t)RT * 128 * HD;
    // with fewer tiles than groups some shares are empty: their slots were never written
    const long long T = *p.total_tiles;
    const bool dense = T >= ncg;
    auto live = [&](int jj) { return dense || share_begin(T, j_lo + jj + 1, ncg) > share_begin(T, j_lo + jj, ncg); };

    float acc[R][4], wsum[R], mx[R];
#pragma unroll
    for (int q = 0; q < R; ++q) {
        acc[q][0] = acc[q][1] = acc[q][2] = acc[q][3] = 0.f;
        wsum[q] = 0.f;
        mx[q] = -INFINITY;
    }
    for (int c0 = 0; c0 < nj; c0 += 32) {
        const int jj = c0 + lane;
        const bool on = jj < nj && live(jj);
        float l[R];
#pragma unroll
        for (int q = 0; q < R; ++q) l[q] = (on && r0 + q < n_rows_u) ? lse_base[(size_t)jj * lse_step + r0 + q] : -INFINITY;
#pragma unroll
        for (int q = 0; q < R; ++q) mx[q] = fmaxf(mx[q], l[q]);
    }
#pragma unroll
    for (int q = 0; q < R; ++q)
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx[q] = fmaxf(mx[q], __shfl_xor_sync(0xffffffffu, mx[q], o));
    for (int c0 = 0; c0 < nj; c0 += 32) {
        const int jj = c0 + lane;
        const bool on = jj < nj && live(jj);
        float w_mine[R];
#pragma unroll
        for (int q = 0; q < R; ++q) {
            const float l = (on && r0 + q < n_rows_u) ? lse_base[(size_t)jj * lse_step + r0 + q] : -INFINITY;
            w_mine[q] = (l == -INFINITY) ? 0.f : exp2f(l - mx[q]);
        }
        const int cn = min(32, nj - c0);
#pragma unroll 2
        for (int e = 0; e < cn; ++e) {
            float4 v[R];
#pragma unroll
            for (int q = 0; q < R; ++q)
                v[q] = *reinterpret_cast<const float4*>(o_base + (size_t)(c0 + e) * o_step + (size_t)min(r0 + q, 127) * HD + lane * 4);
#pragma unroll
            for (int q = 0; q < R; ++q) {
                const float w = __shfl_sync(0xffffffffu, w_mine[q], e);
                if (w > 0.f) {                                // an empty share's slot was never written
                    wsum[q] += w;
                    acc[q][0] += w * v[q].x;
                    acc[q][1] += w * v[q].y;
                    acc[q][2] += w * v[q].z;
                    acc[q][3] += w * v[q].w;
                }
            }
        }
    }
#pragma unroll
    for (int q = 0; q < R; ++q) {
        const int r = r0 + q;
        if (r >= n_rows_u) break;
        const float winv = wsum[q] > 0.f ? 1.f / wsum[q] : 0.f;
        const int ir = i0 + r / p.G, hq = kvh * p.G + r % p.G;
        uint2 v;
        v.x = pack_bf16(acc[q][0] * winv, acc[q][1] * winv);
        v.y = pack_bf16(acc[q][2] * winv, acc[q][3] * winv);
        *reinterpret_cast<uint2*>(p.out + ((size_t)(b * p.k + ir) * p.Hq + hq) * HD + lane * 4) = v;
    }
}

// Thread blocks for a call: one per SM, fewer when the tiles would not give each of them a few.
static int pick_blocks(int B, int HR, int HKV, int max_seq_len) {
    const long long t_max = (long long)B * HR * ((max_seq_len + ATT_TILE - 1) / ATT_TILE + 1);
    long long nc = t_max / 8;
    if (nc > deer_sm_count()) nc = deer_sm_count();
    const int rt = HR / HKV > 0 ? HR / HKV : 1;
    nc = nc / rt * rt;                                    // whole groups of row_tiles blocks
    if (nc < rt) nc = rt;
    return (int)nc;
}

}  // namespace umma

bool umma_supported(int D, int G, float scale) { return D == umma::HD && G >= 1 && G <= 128 && scale > 0.f; }

int umma_row_tiles(int k, int G) {
    const int ipt = 128 / G;                 // block rows per row tile
    return (k + ipt - 1) / ipt;
}

size_t umma_workspace_bytes(int B, int k, int Hq, int Hkv, int max_seq_len) {
    const int G = Hq / Hkv > 0 ? Hq / Hkv : 1;
    const int HR = Hkv * umma_row_tiles(k, G);
    const size_t slots = (size_t)B * HR + umma::pick_blocks(B, HR, Hkv, max_seq_len);   // slot = unit index + block index
    return slots * 128 * (umma::HD + 1) * sizeof(float) + (size_t)B * HR * sizeof(int2) + sizeof(long long);
}

int launch_umma(AttnParams p, cudaStream_t st) {
    using namespace umma;
    using sm100::make_map_bf16;
    const int Hkv = p.kv.n_kv_heads;
    p.ipt = 128 / p.G;
    p.row_tiles = umma_row_tiles(p.k, p.G);
    const int HR = Hkv * p.row_tiles;
    p.nc = pick_blocks(p.B, HR, Hkv, p.max_seq_len);
    const size_t slots = (size_t)p.B * HR + p.nc;
    p.part_lse = p.part_o + slots * 128 * HD;
    p.total_tiles = reinterpret_cast<long long*>(p.part_lse + slots * 128);      // 8-byte aligned: slots * 128 * 129 floats
    p.unit_parts = reinterpret_cast<int2*>(p.total_tiles + 1);
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
    DEER_CUDA(launch_pdl(block_attn_umma_kernel, dim3(p.nc), dim3(THREADS), (size_t)SMEM_BYTES, st, tm_q, tm_kb, tm_vb, tm_kp, tm_vp, p));
    if ((long long)p.B * HR * 4 >= 2 * deer_sm_count())
        DEER_CUDA(launch_pdl(attn_umma_merge_kernel<4>, dim3((unsigned)(p.B * HR * 4)), dim3(256), 0, st, p));
    else
        DEER_CUDA(launch_pdl(attn_umma_merge_kernel<1>, dim3((unsigned)(p.B * HR * 16)), dim3(256), 0, st, p));
    return DEER_OK;
}

}  // namespace attn

// ---- self-test of the bounded waits ------------------------------------------------------------
namespace {
__global__ void bounded_wait_selftest_kernel(int32_t* status) {
    __shared__ uint64_t bar_word;
    __shared__ int abort_flag;
    const uint32_t bar = smem_u32(&bar_word);
    if (threadIdx.x == 0) {
        sm100::mbar_init(bar, 1);                 // one arrival expected; none will come
        abort_flag = 0;
        sm100::mbar_init_fence();
    }
    __syncthreads();
    const bool got = sm100::mbar_wait(bar, 0u, &abort_flag);    // every thread waits, as a kernel's warps do
    __syncthreads();
    if (threadIdx.x == 0 && !got && abort_flag) deer_report(status, DEER_ERR_TIMEOUT);
}
}  // namespace

extern "C" int deer_selftest_bounded_wait(deer_kv* kv, void* stream) {
    DEER_CHECK_ARG(kv, DEER_ERR_INVALID_ARG, "deer_selftest_bounded_wait: null argument");
    bounded_wait_selftest_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(kv->d.status);
    DEER_CUDA(cudaGetLastError());
    return DEER_OK;
}
