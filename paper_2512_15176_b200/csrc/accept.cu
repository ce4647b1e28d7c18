// (3) Acceptance rule of the draft-verify cycle (Eq. 5, Eq. 6, Algorithm 1's
// inner loop, stopped at the first rejection).
//
// GREEDY: integer prefix match.
// SAMPLE: (a) one streaming pass over the drafter logits for log-sum-exp and
// the draft token's logit of every block row; (b) a per-sequence scan for the
// first rejection, log alpha_i = min(0, log p(y_i) - log q(y_i)) against log u;
// (c) for each rejected sequence the residual max(0, p - q) of that one row,
// split over NS thread blocks, then an inverse-CDF search in vocabulary order.
// (b) and (c) are one kernel.  Only (a) touches more than a few rows.

#include "common.cuh"
#include "greedy.cuh"

namespace {

constexpr int NS = 128;            // vocabulary slices per rejected row (NS <= RES_THREADS)
constexpr int RES_THREADS = 256;

// ---------------------------------------------------------------- greedy
__global__ void accept_greedy_kernel(int B, int k, int kd, const int32_t* __restrict__ draft, const int32_t* __restrict__ target,
                                     int32_t eos_id, int32_t* __restrict__ accept_len, int32_t* __restrict__ out_ids,
                                     int32_t* __restrict__ n_out) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    pdl_trigger();
    pdl_wait();
    if (b >= B) return;
    int n;
    const int a = greedy_accept_row(draft + (size_t)b * k, target + (size_t)b * k, out_ids + (size_t)b * k, k, kd, eos_id, &n);
    accept_len[b] = a;
    n_out[b] = n;
}

// ---------------------------------------------------------------- sample (a)
// A block per block row (the blocks stride over the rows when there are fewer
// of them): log-sum-exp of the drafter logits and the draft token's logit.
template <int THREADS, int DEPTH>
__global__ void __launch_bounds__(THREADS) draft_row_stats_kernel(int rows, int V, const float* __restrict__ q_logits,
                                                                  const int32_t* __restrict__ draft, float* __restrict__ lse_q,
                                                                  float* __restrict__ zq_draft, int* __restrict__ done, int n_done) {
    constexpr int NW = THREADS / 32;
    __shared__ float sm[NW], ss[NW];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    pdl_trigger();
    pdl_wait();
    // the arrival counters of the acceptance kernel that follows on this workspace start at zero
    if (blockIdx.x == 0)
        for (int j = threadIdx.x; j < n_done; j += THREADS) done[j] = 0;
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

// ---------------------------------------------------------------- sample (b) + (c)
// One kernel, NS thread blocks per sequence.  Every block first repeats the sequence's scan (warp 0, lane i =
// block row i: log alpha_i against log u_i, Eq. 5) and so knows the first rejected row by itself; block 0 writes
// the accepted prefix.  Then each block sums the residual max(0, p - q) of that row (Eq. 6) over its slice of the
// vocabulary, and the block that arrives last draws the token by inverse CDF in vocabulary order.
//   p(v) = exp(z_p[v]/T - lse_p) (0 below the truncation threshold, if there is one), q(v) = exp(z_q[v] - lse_q):
// the exponentials in fp32 (expf, 2 ulp), their differences summed in fp64.  lse_p and lse_q are fp32 values,
// so p and q carry a common relative error of ~1e-6 each; the cumulative residual is off by a few 1e-6 of its
// total at most, and the draw agrees with an exact evaluation whenever r * S keeps 1e-4 * S away from the edges
// of the drawn token's cell.
struct SampleArgs {
    int B, k, kd, V, slice;
    const int32_t* draft;
    const float* target_logits;   // [B][k][V]
    const float* draft_logits;    // [B][k][V]
    const float* lse_p;           // [B][k]  logsumexp(z_p / T) (over the kept tokens, if truncated)
    const float* zp_draft;        // [B][k]  z_p[draft]
    const float* tau;             // [B][k] or null: tokens with z_p < tau have p = 0
    const float* lse_q;
    const float* zq_draft;
    float inv_t;
    const float* u;
    const float* r;
    double* sums;                 // [B][NS][2]: residual mass, p mass of the slice
    int* done;                    // [B] slices finished (zeroed by draft_row_stats_kernel)
    int32_t eos_id;
    int32_t* accept_len;
    int32_t* out_ids;
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
__device__ void cut_at_eos(const SampleArgs& a, int b) {
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

__global__ void __launch_bounds__(RES_THREADS) accept_sample_kernel(SampleArgs a) {
    constexpr int NW = RES_THREADS / 32;
    __shared__ double sh[32];
    __shared__ double s_mass[NS], s_psum[NS];
    __shared__ double warp_tot[NW];
    __shared__ int s_acc, s_last, s_hit;
    const int b = blockIdx.y, sl = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    pdl_trigger();
    pdl_wait();

    // ---- the scan: first rejected row of this sequence ----
    if (warp == 0) {
        bool acc = true;
        int y = -1;
        if (lane < a.kd) {
            const size_t row = (size_t)b * a.k + lane;
            y = a.draft[row];
            const float zp = a.zp_draft[row];
            float log_p = zp * a.inv_t - a.lse_p[row];
            if (a.tau && zp < a.tau[row]) log_p = -INFINITY;        // outside the kept set: never accepted
            const float log_alpha = fminf(0.f, log_p - (a.zq_draft[row] - a.lse_q[row]));
            acc = logf(a.u[row]) <= log_alpha;
        }
        const unsigned rejected = ~__ballot_sync(0xffffffffu, acc);
        const int n_acc = rejected ? __ffs(rejected) - 1 : a.kd;    // lanes >= kd always vote "accepted"
        if (lane == 0) s_acc = n_acc;
        if (sl == 0) {
            if (lane < a.k) a.out_ids[(size_t)b * a.k + lane] = lane < n_acc ? y : -1;
            if (lane == 0) {
                a.accept_len[b] = n_acc;
                a.n_out[b] = n_acc < a.k ? n_acc + 1 : a.k;
            }
        }
    }
    __syncthreads();
    const int n_acc = s_acc;
    const int i = n_acc < a.k ? n_acc : -1;       // the row a token is drawn from: the first rejection, or the extra row
    const bool from_p = (n_acc == a.kd);          // nothing was proposed for that row: the token comes from p itself
    if (i < 0) {
        if (sl == 0 && tid == 0 && a.eos_id >= 0) cut_at_eos(a, b);
        return;
    }
    const size_t row = (size_t)b * a.k + i;
    const float* __restrict__ zp = a.target_logits + row * a.V;
    const float* __restrict__ zq = a.draft_logits + row * a.V;
    const float lp = a.lse_p[row], lq = a.lse_q[row], it = a.inv_t;
    const float tau = a.tau ? a.tau[row] : -INFINITY;
    auto p_of = [&](float z) { return z >= tau ? expf(fmaf(z, it, -lp)) : 0.f; };
    auto q_of = [&](float z) { return from_p ? 0.f : expf(z - lq); };
    auto resid = [&](float x, float y) { return fmaxf(x - y, 0.f); };

    // ---- residual mass and p mass of this block's slice ----
    {
        const int v0 = sl * a.slice, v1 = min(a.V, v0 + a.slice);
        double acc = 0.0, accp = 0.0;
        int v = v0 + tid;
        if ((a.V & 3) == 0) {
            // v0 and V are multiples of 4, so v1 - v0 is as well
            for (int q = v0 + 4 * tid; q < v1; q += 4 * RES_THREADS) {
                const float4 p4 = __ldg(reinterpret_cast<const float4*>(zp + q));
                const float4 q4 = __ldg(reinterpret_cast<const float4*>(zq + q));
                const float x0 = p_of(p4.x), x1 = p_of(p4.y), x2 = p_of(p4.z), x3 = p_of(p4.w);
                const float y0 = q_of(q4.x), y1 = q_of(q4.y), y2 = q_of(q4.z), y3 = q_of(q4.w);
                acc += ((double)resid(x0, y0) + (double)resid(x1, y1)) + ((double)resid(x2, y2) + (double)resid(x3, y3));
                accp += ((double)x0 + (double)x1) + ((double)x2 + (double)x3);
            }
            v = v1;
        }
        for (; v < v1; v += RES_THREADS) {
            const float x = p_of(zp[v]);
            acc += (double)resid(x, q_of(zq[v]));
            accp += (double)x;
        }
        acc = block_sum(acc, sh);
        accp = block_sum(accp, sh);
        if (tid == 0) {
            a.sums[((size_t)b * NS + sl) * 2 + 0] = acc;
            a.sums[((size_t)b * NS + sl) * 2 + 1] = accp;
            __threadfence();
            s_last = (atomicAdd(a.done + b, 1) == NS - 1) ? 1 : 0;     // zeroed by the pass over the drafter's logits
        }
        __syncthreads();
        if (!s_last) return;
        __threadfence();
    }
    // ---- the last block of the sequence: locate the slice, then the token inside it ----
    const volatile double* vs = a.sums;
    if (tid < NS) {
        s_mass[tid] = vs[((size_t)b * NS + tid) * 2 + 0];
        s_psum[tid] = vs[((size_t)b * NS + tid) * 2 + 1];
    }
    __syncthreads();
    double S = 0.0, Sp = 0.0;
#pragma unroll
    for (int j = 0; j < NS; ++j) {
        S += s_mass[j];
        Sp += s_psum[j];
    }
    const bool use_p = !(S > 0.0);              // no residual mass at all: draw from p itself
    const double target = (double)a.r[b] * (use_p ? Sp : S);
    double base = 0.0;
    int hs = 0;
    for (; hs < NS - 1; ++hs) {
        const double m = use_p ? s_psum[hs] : s_mass[hs];
        if (base + m >= target) break;
        base += m;
    }
    auto weight = [&](int v) { return (double)(use_p ? p_of(zp[v]) : resid(p_of(zp[v]), q_of(zq[v]))); };
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
                            int32_t* __restrict__ appended, int pending) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    pdl_trigger();
    pdl_wait();
    if (b >= B) return;
    if (finished[b]) {
        keep[b] = 0;
        if (appended) appended[b] = 0;
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
    if (appended) appended[b] = m;
    const int a = accept_len[b];
    keep[b] = (a < m ? (a < 0 ? 0 : a) : m) + pending;    // pending: row 0 was the token emitted last; it stays too
    if (eos || have + m >= max_new) finished[b] = 1;
}

// ---------------------------------------------------------------- the drafter's block between iterations
// One thread per sequence: the re-fill rule (masked rows whose best token is confident enough become decoded; if
// none is, the most confident one does).
__global__ void refill_kernel(int B, int k, const int32_t* __restrict__ ids, const float* __restrict__ logprob, float log_threshold,
                              int32_t* __restrict__ row_state, int32_t* __restrict__ tokens, int32_t* __restrict__ left) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    pdl_trigger();
    pdl_wait();
    if (b >= B) return;
    int32_t* st = row_state + (size_t)b * k;
    int n_masked = 0, n_chosen = 0, best = -1;
    float best_lp = -INFINITY;
    for (int i = 0; i < k; ++i) {
        if (st[i] != 1) continue;
        ++n_masked;
        const float lp = logprob[(size_t)b * k + i];
        if (best < 0 || lp > best_lp) {           // the first row wins among equals
            best = i;
            best_lp = lp;
        }
        if (lp >= log_threshold) {
            st[i] = 0;
            tokens[(size_t)b * k + i] = ids[(size_t)b * k + i];
            ++n_chosen;
        }
    }
    if (n_masked > 0 && n_chosen == 0) {
        st[best] = 0;
        tokens[(size_t)b * k + best] = ids[(size_t)b * k + best];
        n_chosen = 1;
    }
    if (left) left[b] = n_masked - n_chosen;
}

__global__ void refresh_rows_kernel(int B, int k, const int32_t* __restrict__ appended, int32_t* __restrict__ row_state) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    pdl_trigger();
    pdl_wait();
    if (idx >= B * k) return;
    const int b = idx / k, i = idx % k;
    row_state[idx] = i < appended[b] ? 0 : -1;
}

struct SampleWs {
    float* lse_q;
    float* zq_draft;
    double* sums;
    int* done;
    size_t bytes;
};

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

SampleWs carve(void* base, int B, int k) {
    SampleWs w;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        void* p = base ? static_cast<char*>(base) + off : nullptr;
        off = align_up(off + bytes, 256);
        return p;
    };
    w.lse_q = static_cast<float*>(take((size_t)B * k * sizeof(float)));
    w.zq_draft = static_cast<float*>(take((size_t)B * k * sizeof(float)));
    w.sums = static_cast<double*>(take((size_t)B * NS * 2 * sizeof(double)));
    w.done = static_cast<int*>(take((size_t)B * sizeof(int)));
    w.bytes = off;
    return w;
}

}  // namespace

extern "C" int deer_refill(int B, int k, const int32_t* ids, const float* logprob, float log_threshold, int32_t* row_state,
                           int32_t* tokens, int32_t* left, void* stream) {
    DEER_CHECK_ARG(ids && logprob && row_state && tokens, DEER_ERR_INVALID_ARG, "deer_refill: null argument");
    DEER_CHECK_ARG(k >= 1 && k <= DEER_MAX_BLOCK, DEER_ERR_UNSUPPORTED, "deer_refill: k must be in [1, 32]");
    DEER_CHECK_ARG(B >= 0, DEER_ERR_INVALID_ARG, "deer_refill: B must not be negative");
    if (B == 0) return DEER_OK;
    DEER_CUDA(launch_pdl(refill_kernel, dim3((B + 127) / 128), dim3(128), 0, static_cast<cudaStream_t>(stream), B, k, ids, logprob,
                         log_threshold, row_state, tokens, left));
    return DEER_OK;
}

extern "C" int deer_refresh_rows(int B, int k, const int32_t* appended, int32_t* row_state, void* stream) {
    DEER_CHECK_ARG(appended && row_state, DEER_ERR_INVALID_ARG, "deer_refresh_rows: null argument");
    DEER_CHECK_ARG(k >= 1 && k <= DEER_MAX_BLOCK, DEER_ERR_UNSUPPORTED, "deer_refresh_rows: k must be in [1, 32]");
    DEER_CHECK_ARG(B >= 0, DEER_ERR_INVALID_ARG, "deer_refresh_rows: B must not be negative");
    if (B == 0) return DEER_OK;
    DEER_CUDA(launch_pdl(refresh_rows_kernel, dim3((B * k + 127) / 128), dim3(128), 0, static_cast<cudaStream_t>(stream), B, k, appended,
                         row_state));
    return DEER_OK;
}

extern "C" int deer_emit(int B, int k, const int32_t* accept_len, const int32_t* out_ids, const int32_t* n_out, int32_t eos_id,
                         int32_t max_new, int32_t* tokens, int32_t* n_tokens, int32_t* finished, int32_t* keep,
                         int32_t* appended, int flags, void* stream) {
    DEER_CHECK_ARG((flags & ~DEER_EMIT_PENDING) == 0, DEER_ERR_INVALID_ARG, "deer_emit: unknown flags");
    DEER_CHECK_ARG(accept_len && out_ids && n_out && (tokens || max_new == 0) && n_tokens && finished && keep, DEER_ERR_INVALID_ARG,
                   "deer_emit: null argument");
    DEER_CHECK_ARG(k >= 1 && k <= DEER_MAX_BLOCK, DEER_ERR_UNSUPPORTED, "deer_emit: k must be in [1, 32]");
    DEER_CHECK_ARG(B >= 0 && max_new >= 0, DEER_ERR_INVALID_ARG, "deer_emit: B and max_new must not be negative");
    if (B == 0) return DEER_OK;
    DEER_CUDA(launch_pdl(emit_kernel, dim3((B + 127) / 128), dim3(128), 0, static_cast<cudaStream_t>(stream), B, k, accept_len, out_ids,
                         n_out, eos_id, max_new, tokens, n_tokens, finished, keep, appended, (flags & DEER_EMIT_PENDING) ? 1 : 0));
    return DEER_OK;
}

extern "C" size_t deer_accept_workspace_bytes(int mode, int B, int k, int V) {
    mode &= ~DEER_ACC_BONUS;
    if ((mode != DEER_ACC_SAMPLE && mode != DEER_ACC_SAMPLE_PRESTATS) || B <= 0 || k <= 0 || V <= 0) return 0;
    return carve(nullptr, B, k).bytes;
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
    const SampleWs w = carve(workspace, B, k);
    // Meant to run beside the attention kernel, whose blocks take 56 K of an SM's 64 K registers and most of its
    // shared memory.  Two things let a block of this kernel share an SM with one of those: at most one block per SM
    // (one block of 256 threads and 32 registers per SM, striding over the rows; a block per row filled the SMs first and
    // the two kernels took turns), and the same shared-memory carve-out as that kernel asks for -- blocks of kernels
    // with different carve-outs do not share an SM at all (measured: without it the LM head beside this kernel took
    // 496 us instead of 283).
    const int rows = B * k, sms = deer_sm_count();
    DEER_CUDA(cudaFuncSetAttribute(draft_row_stats_kernel<256, 4>, cudaFuncAttributePreferredSharedMemoryCarveout, 100));
    DEER_CUDA(launch_pdl(draft_row_stats_kernel<256, 4>, dim3(rows < sms ? rows : sms), dim3(256), 0, static_cast<cudaStream_t>(stream),
                         rows, V, draft_logits, draft_ids, w.lse_q, w.zq_draft, w.done, B));
    return DEER_OK;
}

extern "C" int deer_accept(int mode, int B, int k, int V, const int32_t* draft_ids, const int32_t* target_ids,
                           const float* target_logits, const float* target_lse, const float* target_draft_logit,
                           float temperature, const float* draft_logits, const float* u, const float* r, int32_t eos_id,
                           int32_t* accept_len, int32_t* out_ids, int32_t* n_out, void* workspace, size_t workspace_bytes,
                           void* stream) {
    return deer_accept_truncated(mode, B, k, V, draft_ids, target_ids, target_logits, target_lse, target_draft_logit, nullptr,
                                 temperature, draft_logits, u, r, eos_id, accept_len, out_ids, n_out, workspace, workspace_bytes,
                                 stream);
}

extern "C" int deer_accept_truncated(int mode, int B, int k, int V, const int32_t* draft_ids, const int32_t* target_ids,
                                     const float* target_logits, const float* target_lse, const float* target_draft_logit,
                                     const float* target_tau, float temperature, const float* draft_logits, const float* u,
                                     const float* r, int32_t eos_id, int32_t* accept_len, int32_t* out_ids, int32_t* n_out,
                                     void* workspace, size_t workspace_bytes, void* stream) {
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
        DEER_CUDA(launch_pdl(accept_greedy_kernel, dim3((B + 127) / 128), dim3(128), 0, st, B, k, kd, draft_ids, target_ids, eos_id,
                             accept_len, out_ids, n_out));
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
    const SampleWs w = carve(workspace, B, k);

    if (mode == DEER_ACC_SAMPLE) {       // otherwise deer_draft_stats has left them in the workspace
        DEER_CUDA(launch_pdl(draft_row_stats_kernel<256, 2>, dim3(B * k), dim3(256), 0, st, B * k, V, draft_logits, draft_ids, w.lse_q,
                             w.zq_draft, w.done, B));
    }
    SampleArgs a;
    a.B = B;
    a.k = k;
    a.kd = kd;
    a.V = V;
    a.slice = ((V + NS - 1) / NS + 3) / 4 * 4;
    a.draft = draft_ids;
    a.target_logits = target_logits;
    a.draft_logits = draft_logits;
    a.lse_p = target_lse;
    a.zp_draft = target_draft_logit;
    a.tau = target_tau;
    a.lse_q = w.lse_q;
    a.zq_draft = w.zq_draft;
    a.inv_t = 1.f / temperature;
    a.u = u;
    a.r = r;
    a.sums = w.sums;
    a.done = w.done;
    a.eos_id = eos_id;
    a.accept_len = accept_len;
    a.out_ids = out_ids;
    a.n_out = n_out;
    DEER_CUDA(launch_pdl(accept_sample_kernel, dim3(NS, B), dim3(RES_THREADS), 0, st, a));
    return DEER_OK;
}
