// Shared declarations of the block-attention kernels: launch parameters, the
// split of a sequence's context into chunks, and the two kernel variants.
#pragma once

#include "common.cuh"

namespace attn {

constexpr int ATT_TILE = 64;      // tokens per pipeline stage (4 pages)
constexpr float LOG2E = 1.4426950408889634f;

#ifdef __CUDACC__
// Block rows that block row i may see, as a bit per row.  Causal: rows 0..i.  Bidirectional: all k; with row
// states a masked row sees the rows that hold something, a decoded row the decoded rows, and an absent row (whose
// output nobody reads) is treated like a masked one.  `present` / `decoded` are the bit sets of the sequence's rows
// with state >= 0 / == 0 (all ones without row states).
__device__ __forceinline__ uint32_t visible_rows(int mask, int i, int state_i, uint32_t present, uint32_t decoded) {
    if (mask == DEER_MASK_CAUSAL) return i >= 31 ? 0xffffffffu : (2u << i) - 1u;
    return state_i == 0 ? decoded : present;
}
// Warp-collective: the two bit sets for sequence b (lane j looks at row j).
__device__ __forceinline__ void row_state_sets(const int32_t* row_state, int b, int k, int lane, uint32_t* present, uint32_t* decoded) {
    int st = 1;
    if (row_state) st = lane < k ? row_state[(size_t)b * k + lane] : -1;
    else if (lane >= k) st = -1;
    *present = __ballot_sync(0xffffffffu, st >= 0);
    *decoded = row_state ? __ballot_sync(0xffffffffu, st == 0) : *present;
}
#endif

struct AttnParams {
    deer_kv_desc kv;
    const int32_t* seq_ids;
    const int32_t* row_state;  // [B][k] or null: 1 masked, 0 decoded, -1 absent (bidirectional mask only)
    const __nv_bfloat16* q;
    const __nv_bfloat16* k_blk;
    const __nv_bfloat16* v_blk;
    float* part_o;     // [max_chunks][B*k*Hq][D]   normalised partial outputs of the context chunks
    float* part_lse;   // [max_chunks][B*k*Hq]      their log2-sum-exp
    int B, k, Hq, G, R, row_tiles;
    int ipt;           // tcgen05 variant: block rows per row tile (each brings its G query heads)
    int mask, append;
    float scale_log2;
    int chunk, max_chunks, max_seq_len;
    int nc;            // tcgen05 variant: thread blocks, each with an equal share of all KV tiles
    long long* total_tiles;   // tcgen05 variant: tiles of all units together, written by the attention kernel
    int2* unit_parts;  // tcgen05 variant: per unit, (first, last) block holding a piece of it; first < 0: nothing to merge
    __nv_bfloat16* out;
};

struct AttnPlan {
    int chunk, max_chunks, row_tiles;
};

// Cut a context of up to max_seq_len tokens into equal chunks so that about two waves of thread
// blocks cover the (sequence, KV head, row tile) units.
inline AttnPlan plan_attn(int B, int Hkv, int row_tiles, int max_seq_len) {
    AttnPlan pl;
    pl.row_tiles = row_tiles;
    const long units = (long)B * Hkv * row_tiles;
    const long target_blocks = 2L * deer_sm_count();
    long per_unit = (target_blocks + units - 1) / units;
    if (per_unit < 1) per_unit = 1;
    long chunk = (max_seq_len + per_unit - 1) / per_unit;
    chunk = ((chunk + ATT_TILE - 1) / ATT_TILE) * ATT_TILE;
    if (chunk < 256) chunk = 256;
    pl.chunk = (int)chunk;
    pl.max_chunks = max_seq_len > 0 ? (int)((max_seq_len + chunk - 1) / chunk) : 1;
    if (pl.max_chunks < 1) pl.max_chunks = 1;
    return pl;
}

// tcgen05 variant (head_dim 128): row tiles of floor(128 / G) block rows; the KV tiles of all
// (sequence, KV head, row tile) units form one list that is cut into equal shares, one per thread block.
// launch_umma runs the attention kernel and the merge kernel for the units that were cut.
bool umma_supported(int D, int G, float scale);
int umma_row_tiles(int k, int G);
size_t umma_workspace_bytes(int B, int k, int Hq, int Hkv, int max_seq_len);
int launch_umma(AttnParams p, cudaStream_t st);

}  // namespace attn
