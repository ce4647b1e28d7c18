// Shared declarations of the LM-head kernels: launch parameters, the per-(vocabulary part, row)
// selection state, and the rule that merges two such states.
#pragma once

#include "common.cuh"

namespace lmhead {

constexpr int KT = 64;           // hidden elements per pipeline stage (64 bf16 = one 128-byte swizzle row)
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
    int swiglu;                  // linear layer: (gate, up) column pairs -> silu(gate) * up, out_bf16 [M][V / 2]
    float* lin_part;             // linear layer: room for max_ksplit partial products [M][V] fp32, or null
    int max_ksplit;
    Partial* part;               // [nparts][M]
};

__device__ __forceinline__ void merge_sel(float& m, int32_t& idx, float& s, float m2, int32_t idx2, float s2, float inv_t_log2) {
    if (m2 > m || (m2 == m && idx2 < idx)) {
        const float t = m; m = m2; m2 = t;
        const int32_t ti = idx; idx = idx2; idx2 = ti;
        const float ts = s; s = s2; s2 = ts;
    }
    // now (m, idx) is the winner; fold the loser's sum in
    if (s2 > 0.f) s += s2 * exp2f((m2 - m) * inv_t_log2);
}

}  // namespace lmhead
