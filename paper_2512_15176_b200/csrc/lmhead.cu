// (2) LM head + selection: z = h w^T, p_AR = softmax(z / T) of Eq. 5 reduced
// on the fly to argmax / log-sum-exp / the draft token's logit.
//
// Host entry points, the cross-part finalisation and the linear layer's reduction; the tensor-core kernels are
// in lmhead_umma.cu.

#include "lmhead.cuh"

namespace lmhead {

bool umma_supported(int M, int hid, int V);
int launch_umma(const Params& p, int need_sum, int* nparts_out, cudaStream_t st, int* ksplit_out = nullptr);

struct FinalizeArgs {
    const Partial* part;
    int nparts, M;
    float inv_t_log2, inv_t;
    int32_t* out_ids;
    float* out_max_logprob;
    float* out_lse;
};

// One warp per row: the lanes stride over the vocabulary parts, then merge by shuffles.
__global__ void __launch_bounds__(256) lmhead_finalize_kernel(FinalizeArgs a) {
    pdl_trigger();
    const int m = blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    pdl_wait();                                   // the partials of the LM-head kernel
    if (m >= a.M) return;
    float rm = -INFINITY, rs = 0.f;
    int32_t ri = 0x7fffffff;
    bool aborted = false;
    // a lane's partials are requested together (one after the other their latencies would add up), then merged
    for (int pt0 = lane; pt0 < a.nparts; pt0 += 32 * 8) {
        Partial pr[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int pt = pt0 + 32 * j;
            if (pt < a.nparts) pr[j] = a.part[(size_t)pt * a.M + m];
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (pt0 + 32 * j >= a.nparts) break;
            aborted |= (pr[j].idx == PARTIAL_ABORTED);
            merge_sel(rm, ri, rs, pr[j].m, pr[j].idx, pr[j].s, a.inv_t_log2);
        }
    }
    aborted = __any_sync(0xffffffffu, aborted);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float om = __shfl_xor_sync(0xffffffffu, rm, o);
        const int32_t oi = __shfl_xor_sync(0xffffffffu, ri, o);
        const float os = __shfl_xor_sync(0xffffffffu, rs, o);
        merge_sel(rm, ri, rs, om, oi, os, a.inv_t_log2);
    }
    if (lane != 0) return;
    if (a.out_ids) a.out_ids[m] = aborted ? PARTIAL_ABORTED : ri;
    const float ls = logf(rs);
    if (a.out_max_logprob) a.out_max_logprob[m] = -ls;          // max z - logsumexp(z), T = 1
    if (a.out_lse) a.out_lse[m] = rm * a.inv_t + ls;            // logsumexp(z / T)
}

}  // namespace lmhead

extern "C" size_t deer_lmhead_workspace_bytes(int M, int hid, int V) {
    (void)hid;
    if (M <= 0 || V <= 0) return 0;
    return (size_t)deer_sm_count() * M * sizeof(lmhead::Partial);     // one Partial per (vocabulary part, row), a part per SM at most
}

extern "C" int deer_lmhead_select(const void* h, const void* w, int M, int hid, int V, int mode, float temperature,
                                  const int32_t* draft_ids, int32_t* out_ids, float* out_max_logprob, float* out_lse,
                                  float* out_draft_logit, float* out_logits, void* workspace, size_t workspace_bytes,
                                  void* stream) {
    using namespace lmhead;
    DEER_CHECK_ARG(h && w && out_ids, DEER_ERR_INVALID_ARG, "deer_lmhead_select: null argument");
    DEER_CHECK_ARG(deer_aligned16(h) && deer_aligned16(w) && deer_aligned16(workspace) && deer_aligned16(out_logits),
                   DEER_ERR_INVALID_ARG, "deer_lmhead_select: pointers must be 16-byte aligned");
    DEER_CHECK_ARG(M >= 0 && V > 0 && hid > 0, DEER_ERR_INVALID_ARG, "deer_lmhead_select: bad sizes");
    DEER_CHECK_ARG(hid % KT == 0 && V >= 16, DEER_ERR_UNSUPPORTED,
                   "deer_lmhead_select: hid must be a multiple of 64 and V at least 16");
    DEER_CHECK_ARG(mode == DEER_SEL_ARGMAX || mode == DEER_SEL_ARGMAX_LOGPROB || mode == DEER_SEL_SOFTMAX,
                   DEER_ERR_INVALID_ARG, "deer_lmhead_select: bad mode");
    float t = 1.f;
    if (mode == DEER_SEL_SOFTMAX) {
        DEER_CHECK_ARG(temperature > 0.f, DEER_ERR_INVALID_ARG, "deer_lmhead_select: temperature must be > 0");
        DEER_CHECK_ARG(out_lse, DEER_ERR_INVALID_ARG, "deer_lmhead_select: out_lse is required in SOFTMAX mode");
        t = temperature;
    }
    if (mode == DEER_SEL_ARGMAX_LOGPROB)
        DEER_CHECK_ARG(out_max_logprob, DEER_ERR_INVALID_ARG, "deer_lmhead_select: out_max_logprob is required");
    if (M == 0) return DEER_OK;
    const size_t need = deer_lmhead_workspace_bytes(M, hid, V);
    DEER_CHECK_ARG(workspace && workspace_bytes >= need, DEER_ERR_WORKSPACE,
                   "deer_lmhead_select: workspace of %zu bytes needed, %zu given", need, workspace_bytes);
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    Params p;
    p.h = static_cast<const __nv_bfloat16*>(h);
    p.w = static_cast<const __nv_bfloat16*>(w);
    p.M = M;
    p.hid = hid;
    p.V = V;
    p.inv_t_log2 = LOG2E / t;
    p.draft_ids = (mode == DEER_SEL_SOFTMAX) ? draft_ids : nullptr;
    p.out_draft_logit = (mode == DEER_SEL_SOFTMAX) ? out_draft_logit : nullptr;
    p.out_logits = out_logits;
    p.out_bf16 = nullptr;
    p.residual = nullptr;
    p.swiglu = 0;
    p.lin_part = nullptr;
    p.max_ksplit = 1;
    p.part = static_cast<Partial*>(workspace);
    int nparts = 0;
    const int rc = launch_umma(p, mode != DEER_SEL_ARGMAX, &nparts, st);
    if (rc != DEER_OK) return rc;

    FinalizeArgs fa;
    fa.part = p.part;
    fa.nparts = nparts;
    fa.M = M;
    fa.inv_t_log2 = p.inv_t_log2;
    fa.inv_t = 1.f / t;
    fa.out_ids = out_ids;
    fa.out_max_logprob = (mode == DEER_SEL_ARGMAX_LOGPROB) ? out_max_logprob : nullptr;
    fa.out_lse = (mode == DEER_SEL_SOFTMAX) ? out_lse : nullptr;
    DEER_CUDA(launch_pdl(lmhead_finalize_kernel, dim3((M + 7) / 8), dim3(256), 0, st, fa));
    return DEER_OK;
}

// ------------------------------------------------------------------------------
// A plain linear layer on the same kernels: y = x w^T (+ residual) in bf16.  The
// projections around the block attention in a verifier layer (Q/K/V, output,
// gate/up, down) are this at M = B k rows: weight-streaming at small M,
// tensor-bound above ~200 rows, exactly like the LM head without its selection.
// With few output columns (N up to ~19 000 at M <= 128) the blocks take full
// 256-column tiles and a range of the contraction each; their fp32 partial
// products land in the workspace and a second kernel adds them up.
namespace {

constexpr int LIN_MAX_KSPLIT = 16;

__global__ void __launch_bounds__(256) linear_reduce_kernel(const float* __restrict__ part, int ksplit, long long total,
                                                            const __nv_bfloat16* __restrict__ residual,
                                                            __nv_bfloat16* __restrict__ y) {
    const long long i = ((long long)blockIdx.x * 256 + threadIdx.x) * 2;
    pdl_trigger();
    pdl_wait();                                   // the partial products of the kernel before
    if (i >= total) return;
    float s0 = 0.f, s1 = 0.f;
    if (i + 1 < total && (total & 1) == 0) {
        for (int s = 0; s < ksplit; ++s) {
            const float2 v = *reinterpret_cast<const float2*>(part + (size_t)s * total + i);
            s0 += v.x;
            s1 += v.y;
        }
        if (residual) {
            s0 += __bfloat162float(residual[i]);
            s1 += __bfloat162float(residual[i + 1]);
        }
        *reinterpret_cast<uint32_t*>(y + i) = pack_bf16(s0, s1);
    } else {
        for (long long j = i; j < total && j < i + 2; ++j) {
            float t = 0.f;
            for (int s = 0; s < ksplit; ++s) t += part[(size_t)s * total + j];
            if (residual) t += __bfloat162float(residual[j]);
            y[j] = __float2bfloat16(t);
        }
    }
}

}  // namespace

// y = x w^T on the tensor-core kernels, in one of three forms:
//   ksplit_out == nullptr / *ksplit_out == 1   y (+ residual) written in bf16 by the kernel itself;
//   *ksplit_out > 1                             fp32 partial products [ksplit][M][N] left in `workspace` for the caller's
//                                               tail kernel to sum (residual is then the tail's business);
//   swiglu                                      columns are (gate, up) pairs: y [M][N / 2] = silu(gate) * up.
static int linear_launch(const void* x, const void* w, const void* residual, void* y, int M, int K, int N, int swiglu,
                         void* workspace, size_t workspace_bytes, bool leave_partials, int* ksplit_out, cudaStream_t st) {
    using namespace lmhead;
    Params p;
    p.h = static_cast<const __nv_bfloat16*>(x);
    p.w = static_cast<const __nv_bfloat16*>(w);
    p.M = M;
    p.hid = K;
    p.V = N;
    p.inv_t_log2 = LOG2E;
    p.draft_ids = nullptr;
    p.out_draft_logit = nullptr;
    p.out_logits = nullptr;
    p.out_bf16 = static_cast<__nv_bfloat16*>(y);
    p.residual = static_cast<const __nv_bfloat16*>(residual);
    p.swiglu = swiglu;
    // the contraction is cut only as far as the caller's workspace holds the partial products (none: never)
    p.lin_part = swiglu ? nullptr : static_cast<float*>(workspace);
    p.max_ksplit = (workspace && !swiglu) ? (int)(workspace_bytes / ((size_t)M * N * sizeof(float))) : 1;
    if (p.max_ksplit > LIN_MAX_KSPLIT) p.max_ksplit = LIN_MAX_KSPLIT;
    if (p.max_ksplit < 2) {
        p.lin_part = nullptr;
        p.max_ksplit = 1;
    }
    p.part = nullptr;
    int nparts = 0, ksplit = 1;
    const int rc = launch_umma(p, 0, &nparts, st, &ksplit);
    if (rc != DEER_OK) return rc;
    if (ksplit_out) *ksplit_out = ksplit;
    if (ksplit > 1 && !leave_partials) {
        const long long total = (long long)M * N;
        DEER_CUDA(launch_pdl(linear_reduce_kernel, dim3((unsigned)((total / 2 + 256) / 256)), dim3(256), 0, st,
                             (const float*)p.lin_part, ksplit, total, p.residual, p.out_bf16));
    }
    return DEER_OK;
}

extern "C" size_t deer_linear_workspace_bytes(int M, int K, int N) {
    (void)K;
    if (M <= 0 || N <= 0 || M > 128) return 0;            // larger M never cuts the contraction
    return (size_t)LIN_MAX_KSPLIT * M * N * sizeof(float);
}

extern "C" int deer_linear(const void* x, const void* w, const void* residual, void* y, int M, int K, int N, void* workspace,
                           size_t workspace_bytes, void* stream) {
    using namespace lmhead;
    DEER_CHECK_ARG(x && w && y, DEER_ERR_INVALID_ARG, "deer_linear: null argument");
    DEER_CHECK_ARG(deer_aligned16(x) && deer_aligned16(w) && deer_aligned16(y) && deer_aligned16(residual) &&
                       deer_aligned16(workspace),
                   DEER_ERR_INVALID_ARG, "deer_linear: pointers must be 16-byte aligned");
    DEER_CHECK_ARG(M >= 0 && N > 0 && K > 0, DEER_ERR_INVALID_ARG, "deer_linear: bad sizes");
    DEER_CHECK_ARG(umma_supported(M > 0 ? M : 1, K, N), DEER_ERR_UNSUPPORTED,
                   "deer_linear: K must be a multiple of 64 and N at least 16");
    if (M == 0) return DEER_OK;
    return linear_launch(x, w, residual, y, M, K, N, 0, workspace, workspace_bytes, false, nullptr, static_cast<cudaStream_t>(stream));
}

extern "C" int deer_linear_swiglu(const void* x, const void* w_pairs, void* y, int M, int K, int I, void* stream) {
    using namespace lmhead;
    DEER_CHECK_ARG(x && w_pairs && y, DEER_ERR_INVALID_ARG, "deer_linear_swiglu: null argument");
    DEER_CHECK_ARG(deer_aligned16(x) && deer_aligned16(w_pairs) && deer_aligned16(y), DEER_ERR_INVALID_ARG,
                   "deer_linear_swiglu: pointers must be 16-byte aligned");
    DEER_CHECK_ARG(M >= 0 && I > 0 && K > 0, DEER_ERR_INVALID_ARG, "deer_linear_swiglu: bad sizes");
    DEER_CHECK_ARG(K % 64 == 0 && I % 8 == 0, DEER_ERR_UNSUPPORTED, "deer_linear_swiglu: K must be a multiple of 64, I of 8");
    if (M == 0) return DEER_OK;
    return linear_launch(x, w_pairs, nullptr, y, M, K, 2 * I, 1, nullptr, 0, false, nullptr, static_cast<cudaStream_t>(stream));
}

// The projection whose tail another kernel takes over: leaves either bf16 y (+ residual) or fp32 partial products
// without the residual (see linear_launch); *ksplit_out tells which.  Used by the fused layer calls in layer.cu.
int deer_linear_for_tail(const void* x, const void* w, const void* residual, void* y_bf16, int M, int K, int N, void* workspace,
                         size_t workspace_bytes, int* ksplit_out, cudaStream_t st) {
    return linear_launch(x, w, residual, y_bf16, M, K, N, 0, workspace, workspace_bytes, true, ksplit_out, st);
}
