// (3) Acceptance rule of the draft-verify cycle (Eq. 5, Eq. 6, Algorithm 1's
// inner loop, stopped at the first rejection).
//
// GREEDY: integer prefix match.
// SAMPLE: (a) one streaming pass over the drafter logits for log-sum-exp and
// the draft token's logit of every block row; (b) a per-sequence scan for the
// first rejection, log alpha_i = min(0, log p(y_i) - log q(y_i)) against log u;
// (c) for each rejected sequence the residual max(0, p - q) of that one row in
// fp64, split over NS thread blocks, then an inverse-CDF search in vocabulary
// order.  Only (a) touches more than a few rows.

#include "common.cuh"

namespace {

constexpr int NS = 32;             // vocabulary slices per rejected row
constexpr int RES_THREADS = 256;

// ---------------------------------------------------------------- greedy
__global__ void accept_greedy_kernel(int B, int k, int kd, const int32_t* __restrict__ draft, const int32_t* __restrict__ target,
                                     int32_t eos_id, int32_t* __restrict__ accept_len, int32_t* __restrict__ out_ids,
                                     int32_t* __restrict__ n_out) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const int32_t* d = draft + (size_t)b * k;
    const int32_t* t = target + (size_t)b * k;
    int32_t* o = out_ids + (size_t)b * k;
    int a = 0;
    while (a < kd && d[a] == t[a]) ++a;          // kd = k - 1 with the extra row: then a < k and t[a] is always emitted
    int n = a < k ? a + 1 : a;
    for (int i = 0; i < k; ++i) o[i] = i < a ? d[i] : (i == a ? t[i] : -1);
    if (eos_id >= 0) {
        for (int i = 0; i < n; ++i)
            if (o[i] == eos_id) {
                for (int j = i + 1; j < n; ++j) o[j] = -1;
                n = i + 1;
                a = min(a, n);
                break;
            }
    }
    accept_len[b] = a;
    n_out[b] = n;
}

// ---------------------------------------------------------------- sample (a)
// A block per block row (the blocks stride over the rows when there are fewer
// of them): log-sum-exp of the drafter logits and the draft token's logit.
template <int THREADS, int DEPTH>
__global__ void __launch_bounds__(THREADS) draft_row_stats_kernel(int rows, int V, const float* __restrict__ q_logits,
                                                                  const int32_t* __restrict__ draft, float* __restrict__ lse_q,
                                                                  float* __restrict__ zq_draft) {
    constexpr int NW = THREADS / 32;
    __shared__ float sm[NW], ss[NW];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int row = blockIdx.x; row < rows; row += gridDim.x) {
        const float* z = q_logits + (size_t)row * V;
        float m = -INFINITY, s = 0.f;
        auto push4 = [&](const float4 x) {
            const float mx = fmaxf(fmaxf(x.x, x.y), fmaxf(x.z, x.w));
            if (mx > m) {
                s *= __expf(m - mx);
                m = mx;
            }
            s += __expf(x.x - m) + __expf(x.y - m) + __expf(x.z - m) + __expf(x.w - m);
        };
        if ((V & 3) == 0) {
            const float4* z4 = reinterpret_cast<const float4*>(z);
            const int n4 = V / 4;
            int i = threadIdx.x;
            for (; i + (DEPTH - 1) * THREADS < n4; i += DEPTH * THREADS) {       // DEPTH loads in flight per thread
                float4 x[DEPTH];
#pragma unroll
                for (int d = 0; d < DEPTH; ++d) x[d] = __ldcs(z4 + i + d * THREADS);   // read once: evict first
#pragma unroll
                for (int d = 0; d < DEPTH; ++d) push4(x[d]);
            }
            for (; i < n4; i += THREADS) push4(__ldcs(z4 + i));
        } else {
            for (int i = threadIdx.x; i < V; i += THREADS) {
                const float x = z[i];
                if (x > m) {
                    s = s * __expf(m - x) + 1.f;
                    m = x;
                } else {
                    s += __expf(x - m);
                }
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float om = __shfl_xor_sync(0xffffffffu, m, o);
            const float os = __shfl_xor_sync(0xffffffffu, s, o);
            const float nm = fmaxf(m, om);
            s = (m > -INFINITY ? s * __expf(m - nm) : 0.f) + (om > -INFINITY ? os * __expf(om - nm) : 0.f);
            m = nm;
        }
        if (lane == 0) {
            sm[warp] = m;
            ss[warp] = s;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            float M = -INFINITY;
            for (int w = 0; w < NW; ++w) M = fmaxf(M, sm[w]);
            float S = 0.f;
            for (int w = 0; w < NW; ++w) S += (sm[w] > -INFINITY) ? ss[w] * __expf(sm[w] - M) : 0.f;
            lse_q[row] = M + logf(S);
            const int y = draft[row];
            zq_draft[row] = (y >= 0 && y < V) ? z[y] : -INFINITY;
        }
        __syncthreads();                                        // sm / ss are reused by the next row
    }
}

// ---------------------------------------------------------------- sample (b)
// One warp per sequence, lane i = block row i.
__global__ void __launch_bounds__(128) accept_scan_kernel(int B, int k, int kd, const int32_t* __restrict__ draft,
                                                          const float* __restrict__ lse_p, const float* __restrict__ zp_draft,
                                                          float inv_t, const float* __restrict__ lse_q,
                                                          const float* __restrict__ zq_draft, const float* __restrict__ u,
                                                          int32_t* __restrict__ accept_len, int32_t* __restrict__ out_ids,
                                                          int32_t* __restrict__ n_out, int32_t* __restrict__ rej_pos,
                                                          int32_t* __restrict__ from_p, int32_t* __restrict__ done) {
    const int b = blockIdx.x * 4 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (b >= B) return;
    bool acc = true;
    int y = -1;
    if (lane < kd) {
        const size_t r = (size_t)b * k + lane;
        y = draft[r];
        const float log_alpha = fminf(0.f, (zp_draft[r] * inv_t - lse_p[r]) - (zq_draft[r] - lse_q[r]));
        acc = logf(u[r]) <= log_alpha;
    }
    const unsigned rejected = ~__ballot_sync(0xffffffffu, acc);
    const int a = rejected ? __ffs(rejected) - 1 : kd;    // lanes >= kd always vote "accepted"
    if (lane < k) out_ids[(size_t)b * k + lane] = lane < a ? y : -1;
    if (lane == 0) {
        accept_len[b] = a;
        n_out[b] = a < k ? a + 1 : k;
        rej_pos[b] = a < k ? a : -1;    // the row a token is drawn from: the first rejection, or the extra row
        from_p[b] = (a == kd) ? 1 : 0;  // nothing was proposed for that row: the token comes from p itself
        done[b] = 0;                    // slices of the residual pass finished so far
    }
}

// ---------------------------------------------------------------- sample (c)
// The residual of the one rejected row of a sequence, in fp64: p(v) = exp(z_p/T - lse_p) / Sp with Sp the fp64 sum of
// the numerators (lse_p is only fp32-accurate), likewise q.  The numerators are computed once (the fp64 exponential is
// what this path costs) and kept in the workspace for the second pass.
struct ResidualArgs {
    int B, k, V, slice;
    const int32_t* rej_pos;
    const int32_t* from_p;        // [B] 1: draw from p (the extra row after k-1 accepted drafts), q counts as 0
    const float* target_logits;   // [B][k][V]
    const float* draft_logits;    // [B][k][V]
    const float* lse_p;
    const float* lse_q;
    double temperature;
    const float* r;
    double* e_p;                  // [B][V]  exp(z_p/T - lse_p) of the rejected row
    double* e_q;                  // [B][V]  exp(z_q - lse_q)
    double* sums;                 // [B][NS][4]: sum e_p, sum e_q, residual mass of the slice, unused
    int32_t* done;                // [B] slices finished (zeroed by the scan kernel)
    int32_t* out_ids;
    int32_t eos_id;
    int32_t* accept_len;
    int32_t* n_out;
};

__device__ __forceinline__ double block_sum(double v, double* sh) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if (lane == 0) sh[warp] = v;
    __syncthreads();
    double t = 0.0;
    for (int w = 0; w < nw; ++w) t += sh[w];
    return t;
}

// Algorithm 1's EOS break: nothing is emitted after the first EOS (one thread per sequence).
__device__ void cut_at_eos(const ResidualArgs& a, int b) {
    int32_t* o = a.out_ids + (size_t)b * a.k;
    const int n = a.n_out[b];
    for (int j = 0; j < n; ++j)
        if (o[j] == a.eos_id) {
            for (int t = j + 1; t < n; ++t) o[t] = -1;
            a.n_out[b] = j + 1;
            a.accept_len[b] = min(a.accept_len[b], j + 1);
            break;
        }
}

// Pass 1: the fp64 normalisers, one (slice, sequence) per block.  Four tokens per thread and step where the
// rows are 16-byte aligned, so that eight exponentials are in flight per thread.
__global__ void __launch_bounds__(RES_THREADS) residual_norm_kernel(ResidualArgs a) {
    __shared__ double sh[32];
    const int b = blockIdx.y, sl = blockIdx.x;
    const int i = a.rej_pos[b];
    if (i < 0) return;
    const size_t row = (size_t)b * a.k + i;
    const float* zp = a.target_logits + row * a.V;
    const float* zq = a.draft_logits + row * a.V;
    const double lp = (double)a.lse_p[row], lq = (double)a.lse_q[row], it = 1.0 / a.temperature;
    const int v0 = sl * a.slice, v1 = min(a.V, v0 + a.slice);
    double sp = 0.0, sq = 0.0;
    double* ep = a.e_p + (size_t)b * a.V;
    double* eq = a.e_q + (size_t)b * a.V;
    int v = v0 + threadIdx.x;
    if (a.from_p[b]) {
        // the extra row: only p is needed
        for (; v < v1; v += RES_THREADS) {
            const double x = exp((double)zp[v] * it - lp);
            ep[v] = x;
            eq[v] = 0.0;
            sp += x;
        }
    } else if ((a.V & 3) == 0) {
        // v0 and V are multiples of 4, so v1 - v0 is as well
        for (int q = v0 + 4 * threadIdx.x; q < v1; q += 4 * RES_THREADS) {
            const float4 p4 = __ldg(reinterpret_cast<const float4*>(zp + q));
            const float4 q4 = __ldg(reinterpret_cast<const float4*>(zq + q));
            const double x0 = exp((double)p4.x * it - lp), x1 = exp((double)p4.y * it - lp);
            const double x2 = exp((double)p4.z * it - lp), x3 = exp((double)p4.w * it - lp);
            const double y0 = exp((double)q4.x - lq), y1 = exp((double)q4.y - lq);
            const double y2 = exp((double)q4.z - lq), y3 = exp((double)q4.w - lq);
            *reinterpret_cast<double2*>(ep + q) = make_double2(x0, x1);
            *reinterpret_cast<double2*>(ep + q + 2) = make_double2(x2, x3);
            *reinterpret_cast<double2*>(eq + q) = make_double2(y0, y1);
            *reinterpret_cast<double2*>(eq + q + 2) = make_double2(y2, y3);
            sp += (x0 + x1) + (x2 + x3);
            sq += (y0 + y1) + (y2 + y3);
        }
        v = v1;
    }
    for (; v < v1; v += RES_THREADS) {
        const double x = exp((double)zp[v] * it - lp), y = exp((double)zq[v] - lq);
        ep[v] = x;
        eq[v] = y;
        sp += x;
        sq += y;
    }
    sp = block_sum(sp, sh);
    sq = block_sum(sq, sh);
    if (threadIdx.x == 0) {
        a.sums[((size_t)b * NS + sl) * 4 + 0] = sp;
        a.sums[((size_t)b * NS + sl) * 4 + 1] = sq;
    }
}

// Pass 2: residual mass of each slice; the block that finishes a sequence's last slice then draws the token:
// inverse CDF in vocabulary order, the smallest v whose cumulative residual reaches r * (total residual mass),
// from p itself if that mass is 0.
__global__ void __launch_bounds__(RES_THREADS) residual_pick_kernel(ResidualArgs a) {
    constexpr int NW = RES_THREADS / 32;
    __shared__ double sh[32];
    __shared__ double s_mass[NS], s_psum[NS];
    __shared__ double warp_tot[NW];
    __shared__ int s_last, s_hit;
    const int b = blockIdx.y, sl = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int i = a.rej_pos[b];
    if (i < 0) {
        if (sl == 0 && tid == 0 && a.eos_id >= 0) cut_at_eos(a, b);
        return;
    }
    const double* ep = a.e_p + (size_t)b * a.V;
    const double* eq = a.e_q + (size_t)b * a.V;
    double Sp = 0.0, Sq = 0.0;
#pragma unroll
    for (int j = 0; j < NS; ++j) {
        Sp += a.sums[((size_t)b * NS + j) * 4 + 0];
        Sq += a.sums[((size_t)b * NS + j) * 4 + 1];
    }
    const double ip = 1.0 / Sp, iq = a.from_p[b] ? 0.0 : 1.0 / Sq;
    auto resid2 = [&](double x, double y) {
        const double res = x * ip - y * iq;
        return res > 0.0 ? res : 0.0;
    };
    {
        const int v0 = sl * a.slice, v1 = min(a.V, v0 + a.slice);
        double acc = 0.0;
        int v = v0 + tid;
        if ((a.V & 1) == 0) {
            // slices start at multiples of 4 and V is even: pairs stay inside the slice and 16-byte aligned
            for (int q = v0 + 2 * tid; q < v1; q += 2 * RES_THREADS) {
                const double2 x = *reinterpret_cast<const double2*>(ep + q);
                const double2 y = *reinterpret_cast<const double2*>(eq + q);
                acc += resid2(x.x, y.x) + resid2(x.y, y.y);
            }
            v = v1;
        }
        for (; v < v1; v += RES_THREADS) acc += resid2(ep[v], eq[v]);
        acc = block_sum(acc, sh);
        if (tid == 0) {
            a.sums[((size_t)b * NS + sl) * 4 + 2] = acc;
            __threadfence();
            s_last = (atomicAdd(a.done + b, 1) == NS - 1) ? 1 : 0;
        }
        __syncthreads();
        if (!s_last) return;
        __threadfence();
    }
    // ---- the last block of the sequence: locate the slice, then the token inside it ----
    const volatile double* vs = a.sums;
    if (tid < NS) {
        s_mass[tid] = vs[((size_t)b * NS + tid) * 4 + 2];
        s_psum[tid] = vs[((size_t)b * NS + tid) * 4 + 0];
    }
    __syncthreads();
    double S = 0.0;
#pragma unroll
    for (int j = 0; j < NS; ++j) S += s_mass[j];
    const bool use_p = !(S > 0.0);
    const double target = (double)a.r[b] * (use_p ? 1.0 : S);
    double base = 0.0;
    int hs = 0;
    for (; hs < NS - 1; ++hs) {
        const double m = use_p ? s_psum[hs] * ip : s_mass[hs];
        if (base + m >= target) break;
        base += m;
    }
    auto weight = [&](int v) { return use_p ? ep[v] * ip : resid2(ep[v], eq[v]); };
    // Warp w owns a contiguous span of the slice, walked 32 consecutive tokens at a time (coalesced).
    const int v0 = hs * a.slice, v1 = min(a.V, v0 + a.slice);
    const int span = ((v1 - v0 + NW - 1) / NW + 31) / 32 * 32;
    const int w0 = min(v1, v0 + warp * span), w1 = min(v1, w0 + span);
    double mine = 0.0;
    for (int v = w0 + lane; v < w1; v += 32) mine += weight(v);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mine += __shfl_xor_sync(0xffffffffu, mine, o);
    if (tid == 0) s_hit = -1;
    if (lane == 0) warp_tot[warp] = mine;
    __syncthreads();
    double before = base;
    for (int w = 0; w < warp; ++w) before += warp_tot[w];
    if (before < target && before + mine >= target) {
        // the one warp whose span straddles the target: running inclusive scans of 32 tokens
        double cum = before;
        int hit = -1;
        for (int c = w0; c < w1 && hit < 0; c += 32) {
            const int v = c + lane;
            const double wv = v < w1 ? weight(v) : 0.0;
            double incl = wv;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const double t = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += t;
            }
            const unsigned reach = __ballot_sync(0xffffffffu, v < w1 && cum + incl >= target);
            if (reach) hit = c + __ffs(reach) - 1;
            cum += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (hit < 0) {
            // rounding left the walk just short of the warp's total: last token of the span with weight
            for (int c = ((w1 - w0 - 1) / 32) * 32 + w0; c >= w0 && hit < 0; c -= 32) {
                const int v = c + lane;
                const unsigned pos = __ballot_sync(0xffffffffu, v < w1 && weight(v) > 0.0);
                if (pos) hit = c + 31 - __clz(pos);
            }
        }
        if (lane == 0) s_hit = hit;
    }
    __syncthreads();
    if (tid == 0) {
        int hit = s_hit;
        if (!(target > 0.0)) hit = 0;         // r = 0: the smallest v whose cumulative sum is >= 0 is the first token
        if (hit < 0) {
            // the target lies beyond the slice's last cumulative sum by rounding: the last token with weight up to there
            for (int v = v1 - 1; v >= 0; --v)
                if (weight(v) > 0.0) {
                    hit = v;
                    break;
                }
        }
        a.out_ids[(size_t)b * a.k + i] = hit;
        if (a.eos_id >= 0) cut_at_eos(a, b);
    }
}

// ---------------------------------------------------------------- loop book-keeping
// One thread per sequence: append this block's chosen tokens to the sequence's output, decide whether the
// sequence has finished (EOS or length limit), and how many cache rows survive (Algorithm 1's outer loop).
__global__ void emit_kernel(int B, int k, const int32_t* __restrict__ accept_len, const int32_t* __restrict__ out_ids,
                            const int32_t* __restrict__ n_out, int32_t eos_id, int32_t max_new, int32_t* __restrict__ tokens,
                            int32_t* __restrict__ n_tokens, int32_t* __restrict__ finished, int32_t* __restrict__ keep,
                            int pending) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    if (finished[b]) {
        keep[b] = 0;
        return;
    }
    const int have = n_tokens[b];
    int m = n_out[b];
    m = m < 0 ? 0 : (m > k ? k : m);
    if (m > max_new - have) m = max_new - have;
    if (m < 0) m = 0;
    bool eos = false;
    for (int i = 0; i < m; ++i) {
        const int32_t t = out_ids[(size_t)b * k + i];
        tokens[(size_t)b * max_new + have + i] = t;
        eos |= (eos_id >= 0 && t == eos_id);
    }
    n_tokens[b] = have + m;
    const int a = accept_len[b];
    keep[b] = (a < m ? (a < 0 ? 0 : a) : m) + pending;    // pending: row 0 was the token emitted last; it stays too
    if (eos || have + m >= max_new) finished[b] = 1;
}

struct SampleWs {
    float* lse_q;
    float* zq_draft;
    int32_t* rej_pos;
    int32_t* from_p;
    double* e_p;
    double* e_q;
    double* sums;
    int32_t* done;
    size_t bytes;
};

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

SampleWs carve(void* base, int B, int k, int V) {
    SampleWs w;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        void* p = base ? static_cast<char*>(base) + off : nullptr;
        off = align_up(off + bytes, 256);
        return p;
    };
    w.lse_q = static_cast<float*>(take((size_t)B * k * sizeof(float)));
    w.zq_draft = static_cast<float*>(take((size_t)B * k * sizeof(float)));
    w.rej_pos = static_cast<int32_t*>(take((size_t)B * sizeof(int32_t)));
    w.from_p = static_cast<int32_t*>(take((size_t)B * sizeof(int32_t)));
    w.e_p = static_cast<double*>(take((size_t)B * V * sizeof(double)));
    w.e_q = static_cast<double*>(take((size_t)B * V * sizeof(double)));
    w.sums = static_cast<double*>(take((size_t)B * NS * 4 * sizeof(double)));
    w.done = static_cast<int32_t*>(take((size_t)B * sizeof(int32_t)));
    w.bytes = off;
    return w;
}

}  // namespace

extern "C" int deer_emit(int B, int k, const int32_t* accept_len, const int32_t* out_ids, const int32_t* n_out, int32_t eos_id,
                         int32_t max_new, int32_t* tokens, int32_t* n_tokens, int32_t* finished, int32_t* keep, int flags,
                         void* stream) {
    DEER_CHECK_ARG((flags & ~DEER_EMIT_PENDING) == 0, DEER_ERR_INVALID_ARG, "deer_emit: unknown flags");
    DEER_CHECK_ARG(accept_len && out_ids && n_out && (tokens || max_new == 0) && n_tokens && finished && keep, DEER_ERR_INVALID_ARG,
                   "deer_emit: null argument");
    DEER_CHECK_ARG(k >= 1 && k <= DEER_MAX_BLOCK, DEER_ERR_UNSUPPORTED, "deer_emit: k must be in [1, 32]");
    DEER_CHECK_ARG(B >= 0 && max_new >= 0, DEER_ERR_INVALID_ARG, "deer_emit: B and max_new must not be negative");
    if (B == 0) return DEER_OK;
    emit_kernel<<<(B + 127) / 128, 128, 0, static_cast<cudaStream_t>(stream)>>>(B, k, accept_len, out_ids, n_out, eos_id, max_new,
                                                                               tokens, n_tokens, finished, keep,
                                                                               (flags & DEER_EMIT_PENDING) ? 1 : 0);
    DEER_CUDA(cudaGetLastError());
    return DEER_OK;
}

extern "C" size_t deer_accept_workspace_bytes(int mode, int B, int k, int V) {
    mode &= ~DEER_ACC_BONUS;
    if ((mode != DEER_ACC_SAMPLE && mode != DEER_ACC_SAMPLE_PRESTATS) || B <= 0 || k <= 0 || V <= 0) return 0;
    return carve(nullptr, B, k, V).bytes;
}

extern "C" int deer_draft_stats(int B, int k, int V, const int32_t* draft_ids, const float* draft_logits, void* workspace,
                                size_t workspace_bytes, void* stream) {
    DEER_CHECK_ARG(draft_ids && draft_logits, DEER_ERR_INVALID_ARG, "deer_draft_stats: null argument");
    DEER_CHECK_ARG(k >= 1 && k <= DEER_MAX_BLOCK, DEER_ERR_UNSUPPORTED, "deer_draft_stats: k must be in [1, 32]");
    DEER_CHECK_ARG(B >= 0 && B <= 65535 && V > 0, DEER_ERR_INVALID_ARG, "deer_draft_stats: bad sizes");
    if (B == 0) return DEER_OK;
    DEER_CHECK_ARG(deer_aligned16(draft_logits) && deer_aligned16(workspace), DEER_ERR_INVALID_ARG,
                   "deer_draft_stats: logits and workspace must be 16-byte aligned");
    const size_t need = deer_accept_workspace_bytes(DEER_ACC_SAMPLE, B, k, V);
    DEER_CHECK_ARG(workspace && workspace_bytes >= need, DEER_ERR_WORKSPACE,
                   "deer_draft_stats: workspace of %zu bytes needed, %zu given", need, workspace_bytes);
    const SampleWs w = carve(workspace, B, k, V);
    // Meant to run beside the attention kernel, whose blocks take 56 K of an SM's 64 K registers and most of its
    // shared memory.  Two things let a block of this kernel share an SM with one of those: at most one block per SM
    // (one block of 256 threads and 32 registers per SM, striding over the rows; a block per row filled the SMs first and
    // the two kernels took turns), and the same shared-memory carve-out as that kernel asks for -- blocks of kernels
    // with different carve-outs do not share an SM at all (measured: without it the LM head beside this kernel took
    // 496 us instead of 283).
    const int rows = B * k, sms = deer_sm_count();
    DEER_CUDA(cudaFuncSetAttribute(draft_row_stats_kernel<256, 4>, cudaFuncAttributePreferredSharedMemoryCarveout, 100));
    draft_row_stats_kernel<256, 4><<<rows < sms ? rows : sms, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        rows, V, draft_logits, draft_ids, w.lse_q, w.zq_draft);
    DEER_CUDA(cudaGetLastError());
    return DEER_OK;
}

extern "C" int deer_accept(int mode, int B, int k, int V, const int32_t* draft_ids, const int32_t* target_ids,
                           const float* target_logits, const float* target_lse, const float* target_draft_logit,
                           float temperature, const float* draft_logits, const float* u, const float* r, int32_t eos_id,
                           int32_t* accept_len, int32_t* out_ids, int32_t* n_out, void* workspace, size_t workspace_bytes,
                           void* stream) {
    const int kd = (mode & DEER_ACC_BONUS) ? k - 1 : k;     // drafts under test
    mode &= ~DEER_ACC_BONUS;
    DEER_CHECK_ARG(mode == DEER_ACC_GREEDY || mode == DEER_ACC_SAMPLE || mode == DEER_ACC_SAMPLE_PRESTATS, DEER_ERR_INVALID_ARG,
                   "deer_accept: bad mode");
    DEER_CHECK_ARG(draft_ids && accept_len && out_ids && n_out, DEER_ERR_INVALID_ARG, "deer_accept: null argument");
    DEER_CHECK_ARG(k >= 1 && k <= DEER_MAX_BLOCK, DEER_ERR_UNSUPPORTED, "deer_accept: k must be in [1, 32]");
    DEER_CHECK_ARG(B >= 0 && B <= 65535, DEER_ERR_UNSUPPORTED, "deer_accept: B must be in [0, 65535]");
    if (B == 0) return DEER_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (mode == DEER_ACC_GREEDY) {
        DEER_CHECK_ARG(target_ids, DEER_ERR_INVALID_ARG, "deer_accept: target_ids is required in GREEDY mode");
        accept_greedy_kernel<<<(B + 127) / 128, 128, 0, st>>>(B, k, kd, draft_ids, target_ids, eos_id, accept_len, out_ids, n_out);
        DEER_CUDA(cudaGetLastError());
        return DEER_OK;
    }
    DEER_CHECK_ARG(target_logits && target_lse && target_draft_logit && draft_logits && u && r, DEER_ERR_INVALID_ARG,
                   "deer_accept: SAMPLE mode needs target_logits, target_lse, target_draft_logit, draft_logits, u and r");
    DEER_CHECK_ARG(V > 0 && temperature > 0.f, DEER_ERR_INVALID_ARG, "deer_accept: V and temperature must be positive");
    DEER_CHECK_ARG(deer_aligned16(draft_logits) && deer_aligned16(target_logits) && deer_aligned16(workspace),
                   DEER_ERR_INVALID_ARG, "deer_accept: logits and workspace must be 16-byte aligned");
    const size_t need = deer_accept_workspace_bytes(mode, B, k, V);
    DEER_CHECK_ARG(workspace && workspace_bytes >= need, DEER_ERR_WORKSPACE,
                   "deer_accept: workspace of %zu bytes needed, %zu given", need, workspace_bytes);
    const SampleWs w = carve(workspace, B, k, V);

    if (mode == DEER_ACC_SAMPLE) {       // otherwise deer_draft_stats has left them in the workspace
        draft_row_stats_kernel<256, 2><<<B * k, 256, 0, st>>>(B * k, V, draft_logits, draft_ids, w.lse_q, w.zq_draft);
        DEER_CUDA(cudaGetLastError());
    }
    accept_scan_kernel<<<(B + 3) / 4, 128, 0, st>>>(B, k, kd, draft_ids, target_lse, target_draft_logit, 1.f / temperature,
                                                     w.lse_q, w.zq_draft, u, accept_len, out_ids, n_out, w.rej_pos,
                                                     w.from_p, w.done);
    DEER_CUDA(cudaGetLastError());

    ResidualArgs a;
    a.B = B;
    a.k = k;
    a.V = V;
    a.slice = ((V + NS - 1) / NS + 3) / 4 * 4;
    a.rej_pos = w.rej_pos;
    a.from_p = w.from_p;
    a.target_logits = target_logits;
    a.draft_logits = draft_logits;
    a.lse_p = target_lse;
    a.lse_q = w.lse_q;
    a.temperature = (double)temperature;
    a.r = r;
    a.e_p = w.e_p;
    a.e_q = w.e_q;
    a.sums = w.sums;
    a.done = w.done;
    a.out_ids = out_ids;
    a.eos_id = eos_id;
    a.accept_len = accept_len;
    a.n_out = n_out;
    residual_norm_kernel<<<dim3(NS, B), RES_THREADS, 0, st>>>(a);
    DEER_CUDA(cudaGetLastError());
    residual_pick_kernel<<<dim3(NS, B), RES_THREADS, 0, st>>>(a);
    DEER_CUDA(cudaGetLastError());
    return DEER_OK;
}
