// (1) Block attention of a k <= 32 token draft block against the paged KV
// cache (Section 3.2: the verifier's parallel pass over the block is causal
// inside the block; the drafter's single-step fill is bidirectional).
//
// Work decomposition: one thread block per (context chunk, KV head x row tile,
// sequence).  The G*k query rows that share a KV head (G = Hq/Hkv) form the M
// dimension of the QK^T / PV tiles, so every KV byte streamed from HBM feeds
// G*k rows.  The context of a sequence is cut into chunks of `chunk` tokens
// ("split-KV"); each chunk's block emits a normalised partial output plus its
// log-sum-exp, and a merge kernel combines them.  The block rows' own K/V come
// straight from k_blk/v_blk as one more tile handled by the last chunk's block,
// which also appends them to the cache when asked to.

#include "attn.cuh"

namespace attn {

constexpr int ATT_ROWS = 128;     // query rows per thread block: 8 warps x 16
constexpr int ATT_STAGES = 3;
constexpr int ATT_THREADS = 256;

template <int D>
__device__ __forceinline__ uint32_t tile_off(int row, int chunk16) {
    // byte offset of 16-byte piece `chunk16` of `row` in a [rows][D] bf16 tile, XOR-swizzled
    return static_cast<uint32_t>(row * (D * 2) + ((chunk16 ^ (row & 7)) << 4));
}

template <int D>
__global__ void __launch_bounds__(ATT_THREADS, 1) block_attn_kernel(AttnParams p) {
    constexpr int PIECES = D / 8;                       // 16-byte pieces per token row
    constexpr int KS = D / 16;                          // k-steps of QK^T
    constexpr int ND = D / 8;                           // n-tiles of the output
    constexpr int TILE_BYTES = ATT_TILE * D * 2;
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* sQ = smem;                                        // [128][D]
    unsigned char* sK = smem + ATT_ROWS * D * 2;                     // [STAGES][64][D]
    unsigned char* sV = sK + ATT_STAGES * TILE_BYTES;                // [STAGES][64][D]

    const int c = blockIdx.x;
    const int kvh = blockIdx.y / p.row_tiles;
    const int rt = blockIdx.y % p.row_tiles;
    const int b = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int Hkv = p.kv.n_kv_heads;
    pdl_trigger();
    pdl_wait();

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
    const int n_tiles = n_prefix_tiles + (last ? 1 : 0);
    const int32_t* pt_row = p.kv.page_table + (size_t)s * p.kv.max_pages;
    const __nv_bfloat16* kpool = static_cast<const __nv_bfloat16*>(p.kv.k_pool);
    const __nv_bfloat16* vpool = static_cast<const __nv_bfloat16*>(p.kv.v_pool);

    uint32_t present, decoded;
    row_state_sets(p.row_state, b, p.k, lane, &present, &decoded);

    // ---- append the block's K/V rows to the cache (one block per (b, kvh)); with row states the decoded rows only ----
    if (p.append && last && rt == 0) {
        for (int idx = tid; idx < p.k * PIECES; idx += ATT_THREADS) {
            const int j = idx / PIECES, pc = idx % PIECES;
            if (p.row_state && !((decoded >> j) & 1u)) continue;
            const int t = n + j;
            const int lp = t >> 4;
            const int pg = (lp < p.kv.max_pages) ? pt_row[lp] : -1;
            if (pg < 0 || pg >= p.kv.num_pages) {
                deer_report(p.kv.status, DEER_ERR_BAD_PAGE);
                continue;
            }
            const size_t src = ((size_t)(b * p.k + j) * Hkv + kvh) * D + pc * 8;
            const size_t dst = (((size_t)pg * Hkv + kvh) * DEER_PAGE_SIZE + (t & 15)) * D + pc * 8;
            *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.kv.k_pool) + dst) =
                *reinterpret_cast<const uint4*>(p.k_blk + src);
            *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.kv.v_pool) + dst) =
                *reinterpret_cast<const uint4*>(p.v_blk + src);
        }
    }

    // ---- tile loader ----------------------------------------------------------
    auto issue_tile = [&](int ti) {
        if (ti < n_tiles) {
            const int slot = ti % ATT_STAGES;
            const uint32_t kdst = smem_u32(sK + slot * TILE_BYTES);
            const uint32_t vdst = smem_u32(sV + slot * TILE_BYTES);
            if (ti < n_prefix_tiles) {
                const int t0 = t_begin + ti * ATT_TILE;
#pragma unroll
                for (int it = 0; it < ATT_TILE * PIECES / ATT_THREADS; ++it) {
                    const int idx = tid + it * ATT_THREADS;
                    const int row = idx / PIECES, pc = idx % PIECES;
                    const int t = t0 + row;
                    const __nv_bfloat16* ksrc = kpool;
                    const __nv_bfloat16* vsrc = vpool;
                    int bytes = 0;
                    if (t < t_end) {
                        const int pg = ((t >> 4) < p.kv.max_pages) ? pt_row[t >> 4] : -1;
                        if (pg >= 0 && pg < p.kv.num_pages) {
                            const size_t off = (((size_t)pg * Hkv + kvh) * DEER_PAGE_SIZE + (t & 15)) * D + pc * 8;
                            ksrc = kpool + off;
                            vsrc = vpool + off;
                            bytes = 16;
                        } else {
                            deer_report(p.kv.status, DEER_ERR_BAD_PAGE);
                        }
                    }
                    cp_async16(kdst + tile_off<D>(row, pc), ksrc, bytes);
                    cp_async16(vdst + tile_off<D>(row, pc), vsrc, bytes);
                }
            } else {
#pragma unroll
                for (int it = 0; it < ATT_TILE * PIECES / ATT_THREADS; ++it) {
                    const int idx = tid + it * ATT_THREADS;
                    const int row = idx / PIECES, pc = idx % PIECES;
                    const int bytes = (row < p.k && ((present >> row) & 1u)) ? 16 : 0;     // rows that hold nothing read as zero
                    const size_t off = ((size_t)(b * p.k + (row < p.k ? row : 0)) * Hkv + kvh) * D + pc * 8;
                    cp_async16(kdst + tile_off<D>(row, pc), p.k_blk + off, bytes);
                    cp_async16(vdst + tile_off<D>(row, pc), p.v_blk + off, bytes);
                }
            }
        }
        cp_async_commit();
    };

    // ---- Q rows of this tile -> shared -> A fragments ---------------------------
    for (int idx = tid; idx < ATT_ROWS * PIECES; idx += ATT_THREADS) {
        const int row = idx / PIECES, pc = idx % PIECES;
        const int rr = rt * ATT_ROWS + row;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (rr < p.R) {
            const int g = rr / p.k, i = rr % p.k;
            v = *reinterpret_cast<const uint4*>(p.q + ((size_t)(b * p.k + i) * p.Hq + kvh * p.G + g) * D + pc * 8);
        }
        *reinterpret_cast<uint4*>(sQ + tile_off<D>(row, pc)) = v;
    }
#pragma unroll
    for (int st = 0; st < ATT_STAGES - 1; ++st) issue_tile(st);
    __syncthreads();

    uint32_t qf[KS][4];
    {
        const int row = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks)
            ldmatrix_x4(qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], smem_u32(sQ + tile_off<D>(row, ks * 2 + (lane >> 4))));
    }

    const int g8 = lane >> 2, t4 = lane & 3;
    const int row_lo = rt * ATT_ROWS + warp * 16 + g8;   // global row (within the KV head) of accumulator rows g and g+8
    const int row_hi = row_lo + 8;
    const int i_lo = row_lo % p.k, i_hi = row_hi % p.k;
    const uint32_t cols_lo = visible_rows(p.mask, i_lo, p.row_state ? p.row_state[(size_t)b * p.k + i_lo] : 1, present, decoded);
    const uint32_t cols_hi = visible_rows(p.mask, i_hi, p.row_state ? p.row_state[(size_t)b * p.k + i_hi] : 1, present, decoded);

    float o[ND][4];
#pragma unroll
    for (int nt = 0; nt < ND; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
    float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;

    for (int ti = 0; ti < n_tiles; ++ti) {
        cp_async_wait<ATT_STAGES - 2>();
        __syncthreads();
        issue_tile(ti + ATT_STAGES - 1);
        const int slot = ti % ATT_STAGES;
        const unsigned char* tK = sK + slot * TILE_BYTES;
        const unsigned char* tV = sV + slot * TILE_BYTES;

        // S = Q K^T  (16 rows x 64 tokens per warp)
        float sc[ATT_TILE / 8][4];
#pragma unroll
        for (int nt = 0; nt < ATT_TILE / 8; ++nt) sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
            for (int np = 0; np < ATT_TILE / 16; ++np) {
                uint32_t b0, b1, b2, b3;
                const int tok = np * 16 + (lane & 7) + (lane >> 4) * 8;
                ldmatrix_x4(b0, b1, b2, b3, smem_u32(tK + tile_off<D>(tok, ks * 2 + ((lane >> 3) & 1))));
                mma_bf16_16816(sc[np * 2], qf[ks], b0, b1);
                mma_bf16_16816(sc[np * 2 + 1], qf[ks], b2, b3);
            }
        }

        // scale to the log2 domain and mask
        const bool is_block = (ti >= n_prefix_tiles);
        const int valid = is_block ? p.k : (t_end - (t_begin + ti * ATT_TILE));
        float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < ATT_TILE / 8; ++nt) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int col = nt * 8 + t4 * 2 + e;
                bool ok_lo = col < valid, ok_hi = col < valid;
                if (is_block) {                       // valid = k <= 32 here, so col < 32 wherever ok is still true
                    ok_lo = ok_lo && ((cols_lo >> (col & 31)) & 1u);
                    ok_hi = ok_hi && ((cols_hi >> (col & 31)) & 1u);
                }
                sc[nt][e] = ok_lo ? sc[nt][e] * p.scale_log2 : -INFINITY;
                sc[nt][2 + e] = ok_hi ? sc[nt][2 + e] * p.scale_log2 : -INFINITY;
                mx_lo = fmaxf(mx_lo, sc[nt][e]);
                mx_hi = fmaxf(mx_hi, sc[nt][2 + e]);
            }
        }
        mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
        mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
        mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
        mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
        const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
        const float base_lo = (mn_lo == -INFINITY) ? 0.f : mn_lo;
        const float base_hi = (mn_hi == -INFINITY) ? 0.f : mn_hi;
        const float corr_lo = exp2f(m_lo - base_lo), corr_hi = exp2f(m_hi - base_hi);
        m_lo = mn_lo;
        m_hi = mn_hi;
        float sum_lo = 0.f, sum_hi = 0.f;
#pragma unroll
        for (int nt = 0; nt < ATT_TILE / 8; ++nt) {
            sc[nt][0] = exp2f(sc[nt][0] - base_lo);
            sc[nt][1] = exp2f(sc[nt][1] - base_lo);
            sc[nt][2] = exp2f(sc[nt][2] - base_hi);
            sc[nt][3] = exp2f(sc[nt][3] - base_hi);
            sum_lo += sc[nt][0] + sc[nt][1];
            sum_hi += sc[nt][2] + sc[nt][3];
        }
        l_lo = l_lo * corr_lo + sum_lo;
        l_hi = l_hi * corr_hi + sum_hi;
#pragma unroll
        for (int nt = 0; nt < ND; ++nt) {
            o[nt][0] *= corr_lo;
            o[nt][1] *= corr_lo;
            o[nt][2] *= corr_hi;
            o[nt][3] *= corr_hi;
        }

        // O += P V
#pragma unroll
        for (int kk = 0; kk < ATT_TILE / 16; ++kk) {
            uint32_t a[4];
            a[0] = pack_bf16(sc[kk * 2][0], sc[kk * 2][1]);
            a[1] = pack_bf16(sc[kk * 2][2], sc[kk * 2][3]);
            a[2] = pack_bf16(sc[kk * 2 + 1][0], sc[kk * 2 + 1][1]);
            a[3] = pack_bf16(sc[kk * 2 + 1][2], sc[kk * 2 + 1][3]);
            const int tok = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
            for (int dp = 0; dp < ND / 2; ++dp) {
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4_trans(b0, b1, b2, b3, smem_u32(tV + tile_off<D>(tok, dp * 2 + (lane >> 4))));
                mma_bf16_16816(o[dp * 2], a, b0, b1);
                mma_bf16_16816(o[dp * 2 + 1], a, b2, b3);
            }
        }
    }
    cp_async_wait<0>();

    // ---- partial result: o / l and log2-sum-exp -------------------------------
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
    const size_t n_rows = (size_t)p.B * p.k * p.Hq;
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        const int rr = half ? row_hi : row_lo;
        if (rr >= p.R) continue;
        const float l = half ? l_hi : l_lo;
        const float m = half ? m_hi : m_lo;
        const float inv = (l > 0.f) ? 1.f / l : 0.f;
        const int g = rr / p.k, i = rr % p.k;
        const size_t orow = (size_t)(b * p.k + i) * p.Hq + kvh * p.G + g;
        float* dst = p.part_o + ((size_t)c * n_rows + orow) * D;
#pragma unroll
        for (int nt = 0; nt < ND; ++nt) {
            float2 v = make_float2(o[nt][half * 2] * inv, o[nt][half * 2 + 1] * inv);
            *reinterpret_cast<float2*>(dst + nt * 8 + t4 * 2) = v;
        }
        if (t4 == 0) p.part_lse[(size_t)c * n_rows + orow] = (l > 0.f) ? m + log2f(l) : -INFINITY;
    }
}

// One warp per output row: combine the chunks' partial results.
template <int D>
__global__ void __launch_bounds__(256) attn_merge_kernel(AttnParams p, __nv_bfloat16* __restrict__ out) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const size_t n_rows = (size_t)p.B * p.k * p.Hq;
    const size_t orow = (size_t)blockIdx.x * 8 + warp;
    pdl_trigger();
    pdl_wait();
    if (orow >= n_rows) return;
    const int b = (int)(orow / ((size_t)p.k * p.Hq));
    const int s = p.seq_ids[b];
    if (s < 0 || s >= p.kv.max_seqs) return;
    const int n = p.kv.seq_len[s];
    if (n > p.max_seq_len || n < 0) return;
    const int n_chunks = max(1, (n + p.chunk - 1) / p.chunk);
    float mx = -INFINITY;
    for (int c = 0; c < n_chunks; ++c) mx = fmaxf(mx, p.part_lse[(size_t)c * n_rows + orow]);
    constexpr int PER = D / 32;
    float acc[PER];
#pragma unroll
    for (int e = 0; e < PER; ++e) acc[e] = 0.f;
    float wsum = 0.f;
    for (int c = 0; c < n_chunks; ++c) {
        const float lse = p.part_lse[(size_t)c * n_rows + orow];
        const float w = (lse == -INFINITY) ? 0.f : exp2f(lse - mx);
        wsum += w;
        const float* src = p.part_o + ((size_t)c * n_rows + orow) * D + lane * PER;
#pragma unroll
        for (int e = 0; e < PER; ++e) acc[e] += w * src[e];
    }
    const float inv = wsum > 0.f ? 1.f / wsum : 0.f;
    __nv_bfloat16* dst = out + orow * D + lane * PER;
#pragma unroll
    for (int e = 0; e < PER; e += 2) {
        *reinterpret_cast<__nv_bfloat162*>(dst + e) = __floats2bfloat162_rn(acc[e] * inv, acc[e + 1] * inv);
    }
}

template <int D>
constexpr int attn_smem_bytes() {
    return ATT_ROWS * D * 2 + 2 * ATT_STAGES * ATT_TILE * D * 2;
}

static int mma_row_tiles(int k, int G) { return (G * k + ATT_ROWS - 1) / ATT_ROWS; }

// The tcgen05 kernel takes head_dim 128; the warp-level kernel serves head_dim 64.
static bool use_umma(int D, int G, float scale) { return umma_supported(D, G, scale); }

}  // namespace attn

using namespace attn;

extern "C" size_t deer_block_attn_workspace_bytes(int B, int k, int Hq, int Hkv, int D, int max_seq_len) {
    if (B <= 0 || k <= 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || max_seq_len < 0) return 0;
    // room for whichever kernel variant the call ends up using
    const int G = Hq / Hkv > 0 ? Hq / Hkv : 1;
    const int mc = plan_attn(B, Hkv, mma_row_tiles(k, G), max_seq_len).max_chunks;
    size_t bytes = (size_t)mc * B * k * Hq * (D + 1) * sizeof(float);
    if (D == 128 && G <= 128) {
        const size_t b2 = umma_workspace_bytes(B, k, Hq, Hkv, max_seq_len);
        if (b2 > bytes) bytes = b2;
    }
    return bytes;
}

extern "C" int deer_block_attn(deer_kv* kv, const int32_t* seq_ids, const void* q, const void* k_blk, const void* v_blk,
                               void* out, int B, int k, int Hq, int mask, int append, float scale, int max_seq_len,
                               void* workspace, size_t workspace_bytes, void* stream) {
    return deer_block_attn_rows(kv, seq_ids, q, k_blk, v_blk, out, nullptr, B, k, Hq, mask, append, scale, max_seq_len, workspace,
                                workspace_bytes, stream);
}

extern "C" int deer_block_attn_rows(deer_kv* kv, const int32_t* seq_ids, const void* q, const void* k_blk, const void* v_blk,
                                    void* out, const int32_t* row_state, int B, int k, int Hq, int mask, int append, float scale,
                                    int max_seq_len, void* workspace, size_t workspace_bytes, void* stream) {
    DEER_CHECK_ARG(kv && seq_ids && q && k_blk && v_blk && out, DEER_ERR_INVALID_ARG, "deer_block_attn: null argument");
    DEER_CHECK_ARG(!row_state || mask == DEER_MASK_BIDIR, DEER_ERR_INVALID_ARG,
                   "deer_block_attn_rows: row states belong to the bidirectional mask");
    DEER_CHECK_ARG(deer_aligned16(q) && deer_aligned16(k_blk) && deer_aligned16(v_blk) && deer_aligned16(out) &&
                       deer_aligned16(workspace),
                   DEER_ERR_INVALID_ARG, "deer_block_attn: pointers must be 16-byte aligned");
    DEER_CHECK_ARG(k >= 1 && k <= DEER_MAX_BLOCK, DEER_ERR_UNSUPPORTED, "deer_block_attn: k must be in [1, 32]");
    DEER_CHECK_ARG(B >= 0 && B <= 65535, DEER_ERR_UNSUPPORTED, "deer_block_attn: B must be in [0, 65535]");
    const int Hkv = kv->d.n_kv_heads, D = kv->d.head_dim;
    DEER_CHECK_ARG(Hq > 0 && Hq % Hkv == 0, DEER_ERR_INVALID_ARG, "deer_block_attn: Hq must be a positive multiple of Hkv");
    DEER_CHECK_ARG(mask == DEER_MASK_CAUSAL || mask == DEER_MASK_BIDIR, DEER_ERR_INVALID_ARG, "deer_block_attn: bad mask");
    DEER_CHECK_ARG(max_seq_len >= 0, DEER_ERR_INVALID_ARG, "deer_block_attn: max_seq_len must be >= 0");
    if (B == 0) return DEER_OK;
    const size_t need = deer_block_attn_workspace_bytes(B, k, Hq, Hkv, D, max_seq_len);
    DEER_CHECK_ARG(workspace && workspace_bytes >= need, DEER_ERR_WORKSPACE,
                   "deer_block_attn: workspace of %zu bytes needed, %zu given", need, workspace_bytes);
    const int G = Hq / Hkv;
    const bool umma = use_umma(D, G, scale);
    const AttnPlan pl = plan_attn(B, Hkv, umma ? umma_row_tiles(k, G) : mma_row_tiles(k, G), max_seq_len);
    DEER_CHECK_ARG((long)Hkv * pl.row_tiles <= 65535, DEER_ERR_UNSUPPORTED, "deer_block_attn: too many KV heads");

    AttnParams p;
    p.kv = kv->d;
    p.seq_ids = seq_ids;
    p.row_state = row_state;
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.k_blk = static_cast<const __nv_bfloat16*>(k_blk);
    p.v_blk = static_cast<const __nv_bfloat16*>(v_blk);
    const size_t n_rows = (size_t)B * k * Hq;
    p.part_o = static_cast<float*>(workspace);
    p.part_lse = p.part_o + (size_t)pl.max_chunks * n_rows * D;
    p.B = B;
    p.k = k;
    p.Hq = Hq;
    p.G = Hq / Hkv;
    p.R = p.G * k;
    p.row_tiles = pl.row_tiles;
    p.ipt = 0;
    p.nc = 0;
    p.unit_parts = nullptr;
    p.total_tiles = nullptr;
    p.out = nullptr;
    p.mask = mask;
    p.append = append ? 1 : 0;
    p.scale_log2 = scale * LOG2E;
    p.chunk = pl.chunk;
    p.max_chunks = pl.max_chunks;
    p.max_seq_len = max_seq_len;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    dim3 grid(pl.max_chunks, Hkv * pl.row_tiles, B);
    const unsigned merge_blocks = (unsigned)((n_rows + 7) / 8);
    if (umma) {
        p.out = static_cast<__nv_bfloat16*>(out);
        const int rc = launch_umma(p, st);
        if (rc != DEER_OK) return rc;
    } else if (D == 128) {
        constexpr int SM = attn_smem_bytes<128>();
        DEER_CUDA(cudaFuncSetAttribute(block_attn_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM));
        DEER_CUDA(launch_pdl(block_attn_kernel<128>, grid, dim3(ATT_THREADS), (size_t)SM, st, p));
        DEER_CUDA(launch_pdl(attn_merge_kernel<128>, dim3(merge_blocks), dim3(256), 0, st, p, static_cast<__nv_bfloat16*>(out)));
    } else {
        constexpr int SM = attn_smem_bytes<64>();
        DEER_CUDA(cudaFuncSetAttribute(block_attn_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM));
        DEER_CUDA(launch_pdl(block_attn_kernel<64>, grid, dim3(ATT_THREADS), (size_t)SM, st, p));
        DEER_CUDA(launch_pdl(attn_merge_kernel<64>, dim3(merge_blocks), dim3(256), 0, st, p, static_cast<__nv_bfloat16*>(out)));
    }
    DEER_CUDA(cudaGetLastError());
    return DEER_OK;
}
