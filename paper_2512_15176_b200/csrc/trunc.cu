// Top-k / nucleus truncation of the verifier's distribution: one threshold per row of logits.
//
// Both truncations keep an upper level set {v : z[v] >= tau} of the row, so the work is a selection problem:
// find the logit value at which the number of tokens at or above it reaches top_k, or at which their probability
// mass reaches top_p of the mass under consideration.  One thread block per row (two blocks per SM walking rows,
// so that the rows in flight stay in L2 between passes):
//   1. a histogram pass over the row: tokens are binned by logit value, 2048 bins below the row's largest
//      possible logit T * lse, a count and a probability mass per bin;
//   2. a scan over the bins, from the top down, finds the bin in which the target is crossed;
//   3. a second pass gathers that bin's tokens (a few hundred for any smooth distribution) into shared memory,
//      where the threshold is found exactly: tie groups whole, counts exact, masses in fp64.
// If the bin holds more tokens than shared memory takes (heavy ties), it is binned again by bit pattern until it
// does.  Top-k runs first; the nucleus then looks only at the tokens top-k kept, as samplers do.
// A small top_k on a long row (the usual sampler setting) takes one pass instead: a strided sample of the row
// places a cut that leaves a few hundred tokens, the pass gathers everything above the cut, and top-k and the
// nucleus inside it are both resolved in that list; a list that came out short or long falls back to the above.
// Probabilities are 2^(z c - lse c), c = log2(e) / T, by the hardware's exp2 (2 ulp): the masses only decide in
// which bin and at which tie group a target is crossed, and enter the result as log(kept mass).

#include "common.cuh"

namespace {

constexpr int NB = 2048;           // bins per level (+ 1 for what lies below the binned range)
constexpr int CAP = 1024;          // candidates resolved exactly in shared memory
constexpr int THREADS = 512;        // two blocks per SM: one streams its row while the other scans, sorts or waits
constexpr int LIST = THREADS;      // candidates of the one-pass path: one per thread in the sort
constexpr int NW = THREADS / 32;
constexpr float LOG2E = 1.4426950408889634f;

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// Monotone map of a float to an unsigned integer (larger float -> larger key).
__device__ __forceinline__ uint32_t okey(float z) {
    const uint32_t b = __float_as_uint(z);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

struct Row {
    const float* z;
    int V;
    float c, lc;              // p(v) = 2^(z c - lc)
    float floor_z;            // tokens below it are not there (dropped by an earlier truncation)
};

struct Level {                // how the tokens under consideration are binned; bin 0 holds the largest
    int by_key;               // 0: by value below ztop; 1: by bit pattern within [klo, khi]
    float ztop, scale;
    uint32_t klo, khi;
};

__device__ __forceinline__ int bin_of(const Level& lv, float z) {
    if (!lv.by_key) {
        const float d = fmaxf(lv.ztop - z, 0.f) * lv.scale;
        return d >= (float)NB ? NB : (int)d;
    }
    const uint32_t k = okey(z);
    if (k > lv.khi || k < lv.klo) return -1;
    return (int)(((unsigned long long)(lv.khi - k) * NB) / ((unsigned long long)(lv.khi - lv.klo) + 1ull));
}

struct Shared {
    int cnt[NB + 1];
    float mass[NB + 1];
    float cz[CAP];
    float cp[CAP];
    double wsum_d[NW];
    int wsum_i[NW];
    int n_cand, cross_bin, found;
    uint32_t kmin, kmax;
    float tau;
    double res_mass;
    int res_cnt;
    double tot_mass;
};

// Applies f(z) to every token of the row that is under consideration (z >= floor_z), -0 folded into +0.  Four
// 16-byte loads per thread are in flight at a time: a pass is a stream over 600 KB, bound by load latency otherwise.
template <typename F>
__device__ __forceinline__ void for_each_token(const Row& r, F f) {
    const int tid = threadIdx.x;
    if ((r.V & 3) == 0) {
        const float4* z4 = reinterpret_cast<const float4*>(r.z);
        const int n4 = r.V >> 2;
        for (int i0 = tid; i0 < n4; i0 += 4 * THREADS) {
            float4 x[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = i0 + u * THREADS;
                x[u] = i < n4 ? __ldg(z4 + i) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (i0 + u * THREADS >= n4) break;
                const float e[4] = {x[u].x + 0.f, x[u].y + 0.f, x[u].z + 0.f, x[u].w + 0.f};
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (e[j] >= r.floor_z) f(e[j]);
            }
        }
    } else {
        for (int i = tid; i < r.V; i += THREADS) {
            const float x = r.z[i] + 0.f;
            if (x >= r.floor_z) f(x);
        }
    }
}

// Exclusive prefix over the threads of (count, mass); totals in *tc, *tm.  All threads call it.
__device__ __forceinline__ void block_scan(int c, double m, int& ec, double& em, int* tc, double* tm, Shared& sh) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int ic = c;
    double im = m;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, ic, o);
        const double u = __shfl_up_sync(0xffffffffu, im, o);
        if (lane >= o) {
            ic += t;
            im += u;
        }
    }
    __syncthreads();
    if (lane == 31) {
        sh.wsum_i[warp] = ic;
        sh.wsum_d[warp] = im;
    }
    __syncthreads();
    int bc = 0;
    double bm = 0.0;
    int allc = 0;
    double allm = 0.0;
    for (int w = 0; w < NW; ++w) {
        if (w < warp) {
            bc += sh.wsum_i[w];
            bm += sh.wsum_d[w];
        }
        allc += sh.wsum_i[w];
        allm += sh.wsum_d[w];
    }
    ec = bc + ic - c;
    em = bm + im - m;
    *tc = allc;
    *tm = allm;
}

enum { BY_COUNT = 0, BY_MASS = 1 };

// Finds, among the tokens of the row under consideration, the value tau of the first tie group (from the top)
// with which the running count reaches k_target (BY_COUNT) or the running mass reaches frac * (their total mass)
// (BY_MASS).  Leaves tau and the count and mass of the tokens >= tau in sh.tau / sh.res_cnt / sh.res_mass.
__device__ void select_level_set(const Row& r, int kind, int k_target, float frac, Shared& sh) {
    const int tid = threadIdx.x;
    Level lv;
    lv.by_key = 0;
    lv.ztop = r.lc / r.c;                                       // T * lse >= the largest logit
    lv.scale = (float)NB / ((logf((float)r.V) + 20.f) / (r.c / LOG2E));   // NB bins over T * (log V + 20) below it
    lv.klo = 0;
    lv.khi = 0xffffffffu;
    int above_cnt = 0;
    double above_mass = 0.0, target_mass = 0.0;
    constexpr int PER = (NB + 1 + THREADS - 1) / THREADS;
    for (int level = 0; level < 8; ++level) {
        for (int i = tid; i <= NB; i += THREADS) {
            sh.cnt[i] = 0;
            sh.mass[i] = 0.f;
        }
        if (tid == 0) sh.cross_bin = NB + 1;
        __syncthreads();
        for_each_token(r, [&](float z) {
            const int b = bin_of(lv, z);
            if (b >= 0) {
                atomicAdd(&sh.cnt[b], 1);
                atomicAdd(&sh.mass[b], ex2_approx(fmaf(z, r.c, -r.lc)));
            }
        });
        __syncthreads();
        // thread t owns the bins [t * PER, t * PER + PER)
        int c = 0;
        double m = 0.0;
        for (int j = 0; j < PER; ++j) {
            const int b = tid * PER + j;
            if (b <= NB) {
                c += sh.cnt[b];
                m += (double)sh.mass[b];
            }
        }
        int ec, tc;
        double em, tm;
        block_scan(c, m, ec, em, &tc, &tm, sh);
        if (level == 0) target_mass = (double)frac * tm;       // the mass under consideration is what this level saw
        {
            int rc = above_cnt + ec;
            double rm = above_mass + em;
            for (int j = 0; j < PER; ++j) {
                const int b = tid * PER + j;
                if (b > NB) break;
                const int nc = rc + sh.cnt[b];
                const double nm = rm + (double)sh.mass[b];
                const bool crossed = sh.cnt[b] > 0 && (kind == BY_COUNT ? nc >= k_target : nm >= target_mass);
                if (crossed) {
                    atomicMin(&sh.cross_bin, b);
                    break;
                }
                rc = nc;
                rm = nm;
            }
        }
        __syncthreads();
        int bx = sh.cross_bin;
        __syncthreads();
        if (bx > NB) {
            // the target lies beyond everything (rounding, or k_target above the number of tokens): the last bin
            // that holds something is where the walk ends
            if (tid == 0) sh.cross_bin = -1;
            __syncthreads();
            for (int j = 0; j < PER; ++j) {
                const int b = tid * PER + j;
                if (b <= NB && sh.cnt[b] > 0) atomicMax(&sh.cross_bin, b);
            }
            __syncthreads();
            bx = sh.cross_bin;
            __syncthreads();
            if (bx < 0) {                                       // nothing under consideration at all
                if (tid == 0) {
                    sh.tau = r.floor_z;
                    sh.res_cnt = above_cnt;
                    sh.res_mass = above_mass;
                }
                __syncthreads();
                return;
            }
        }
        // totals of the bins above the crossing one join `above`
        {
            int c2 = 0;
            double m2 = 0.0;
            for (int j = 0; j < PER; ++j) {
                const int b = tid * PER + j;
                if (b < bx) {
                    c2 += sh.cnt[b];
                    m2 += (double)sh.mass[b];
                }
            }
            int e1, t1;
            double e2, t2;
            block_scan(c2, m2, e1, e2, &t1, &t2, sh);
            above_cnt += t1;
            above_mass += t2;
        }
        const int n_in_bin = sh.cnt[bx];
        __syncthreads();
        if (n_in_bin <= CAP) {
            // ---- gather the bin's tokens and resolve exactly ----
            if (tid == 0) sh.n_cand = 0;
            __syncthreads();
            for_each_token(r, [&](float z) {
                if (bin_of(lv, z) == bx) {
                    const int slot = atomicAdd(&sh.n_cand, 1);
                    if (slot < CAP) {
                        sh.cz[slot] = z;
                        sh.cp[slot] = ex2_approx(fmaf(z, r.c, -r.lc));
                    }
                }
            });
            __syncthreads();
            const int n = min(sh.n_cand, CAP);
            if (tid == 0) sh.found = 0;
            __syncthreads();
            // The gather order varies from run to run; sums over a candidate's ">" and ">=" sets are taken in
            // fp64, where the order does not show at the precision that matters.
            for (int j = tid; j < n; j += THREADS) {
                const float zj = sh.cz[j];
                int gc = 0, gec = 0;
                double gm = 0.0, gem = 0.0;
                for (int i = 0; i < n; ++i) {
                    const float zi = sh.cz[i];
                    const double pi = (double)sh.cp[i];
                    if (zi > zj) {
                        ++gc;
                        gm += pi;
                    }
                    if (zi >= zj) {
                        ++gec;
                        gem += pi;
                    }
                }
                const bool hit = (kind == BY_COUNT) ? (above_cnt + gc < k_target && above_cnt + gec >= k_target)
                                                    : (above_mass + gm < target_mass && above_mass + gem >= target_mass);
                if (hit) {                                      // every member of the tie group writes the same values
                    sh.tau = zj;
                    sh.res_cnt = above_cnt + gec;
                    sh.res_mass = above_mass + gem;
                    sh.found = 1;
                }
            }
            __syncthreads();
            if (!sh.found) {
                // rounding put the target just outside this bin's exact sums: end the walk at the bin's nearest end
                const bool before = (kind == BY_COUNT) ? (above_cnt >= k_target) : (above_mass >= target_mass);
                float zsel = before ? -INFINITY : INFINITY;
                for (int i = tid; i < n; i += THREADS) zsel = before ? fmaxf(zsel, sh.cz[i]) : fminf(zsel, sh.cz[i]);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    const float t = __shfl_xor_sync(0xffffffffu, zsel, o);
                    zsel = before ? fmaxf(zsel, t) : fminf(zsel, t);
                }
                float* wf = reinterpret_cast<float*>(sh.wsum_i);
                if ((tid & 31) == 0) wf[tid >> 5] = zsel;
                __syncthreads();
                for (int w = 0; w < NW; ++w) zsel = before ? fmaxf(zsel, wf[w]) : fminf(zsel, wf[w]);
                __syncthreads();
                int gec = 0;
                double gem = 0.0;
                for (int i = tid; i < n; i += THREADS)
                    if (sh.cz[i] >= zsel) {
                        ++gec;
                        gem += (double)sh.cp[i];
                    }
                int e1, t1;
                double e2, t2;
                block_scan(gec, gem, e1, e2, &t1, &t2, sh);
                if (tid == 0) {
                    sh.tau = zsel;
                    sh.res_cnt = above_cnt + t1;
                    sh.res_mass = above_mass + t2;
                }
            }
            __syncthreads();
            return;
        }
        // ---- too many tokens in one bin: bin it again by bit pattern between its smallest and largest member ----
        if (tid == 0) {
            sh.kmin = 0xffffffffu;
            sh.kmax = 0u;
        }
        __syncthreads();
        {
            uint32_t lo = 0xffffffffu, hi = 0u;
            for_each_token(r, [&](float z) {
                if (bin_of(lv, z) == bx) {
                    const uint32_t k = okey(z);
                    lo = min(lo, k);
                    hi = max(hi, k);
                }
            });
            atomicMin(&sh.kmin, lo);
            atomicMax(&sh.kmax, hi);
        }
        __syncthreads();
        const uint32_t klo = sh.kmin, khi = sh.kmax;
        __syncthreads();
        if (klo == khi) {
            // one value fills the bin: it is the tie group at which the target is crossed
            if (tid == 0) {
                const uint32_t b = (khi & 0x80000000u) ? (khi & 0x7fffffffu) : ~khi;
                sh.tau = __uint_as_float(b);
                sh.res_cnt = above_cnt + n_in_bin;
                sh.res_mass = above_mass + (double)sh.mass[bx];
            }
            __syncthreads();
            return;
        }
        lv.by_key = 1;
        lv.klo = klo;
        lv.khi = khi;
    }
    // not reached for 32-bit keys (every level by bit pattern narrows the range 2048-fold); keep everything under
    // consideration rather than return an undefined threshold
    if (tid == 0) {
        sh.tau = r.floor_z;
        sh.res_cnt = above_cnt;
        sh.res_mass = above_mass;
    }
    __syncthreads();
}

// Top-k and the nucleus inside it (top_k = 0: the nucleus of the whole row, whose mass is 1 by the definition of
// lse), resolved in a candidate list that is complete above some cut and holds at least top_k tokens: the list is sorted (descending, one element per thread: a bitonic network, in registers by
// shuffles within a warp and through shared memory across warps), the probabilities are summed along it in fp64, and
// both thresholds are read off at the ends of tie groups.  Result in sh.tau / res_cnt / res_mass; false, and no
// result, when the nucleus reaches below the list.
static_assert(LIST <= CAP, "the list lives in the exact stage's arrays");
__device__ bool resolve_sorted(const Row& r, Shared& sh, int n, int top_k, float top_p) {
    const int tid = threadIdx.x;
    int P = 32;
    while (P < n) P <<= 1;
    float x = tid < n ? sh.cz[tid] : -INFINITY;
    __syncthreads();
    for (int size = 2; size <= P; size <<= 1) {
        const bool desc = (tid & size) == 0;
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            float y;
            if (stride >= 32) {
                sh.cz[tid] = x;
                __syncthreads();
                y = sh.cz[tid ^ stride];
                __syncthreads();
            } else {
                y = __shfl_xor_sync(0xffffffffu, x, stride);
            }
            const bool lower = (tid & stride) == 0;
            x = (lower == desc) ? fmaxf(x, y) : fminf(x, y);
        }
    }
    sh.cz[tid] = x;
    __syncthreads();
    const double p = tid < n ? (double)ex2_approx(fmaf(x, r.c, -r.lc)) : 0.0;
    int ec, tc;
    double em, tm;
    block_scan(tid < n ? 1 : 0, p, ec, em, &tc, &tm, sh);
    const double upto = em + p;                                   // mass of the list down to and including this element
    const bool group_end = tid < n && (tid == n - 1 || sh.cz[tid + 1] != x);
    if (top_k > 0) {
        const float tau_k = sh.cz[top_k - 1];
        if (group_end && x == tau_k) {
            sh.tau = x;
            sh.res_cnt = tid + 1;
            sh.res_mass = upto;
        }
    } else if (tid == n - 1) {
        sh.res_cnt = n;                                           // nothing cut by count: the set under consideration
        sh.res_mass = 1.0;                                        // is the row, and the list must reach its nucleus
        sh.tot_mass = upto;
    }
    __syncthreads();
    if (top_p >= 1.f) return true;
    const int cnt_k = sh.res_cnt;
    const double target = (double)top_p * sh.res_mass;
    const bool reaches = top_k > 0 || sh.tot_mass >= target;
    __syncthreads();
    if (!reaches) return false;
    if (tid == 0) sh.cross_bin = cnt_k - 1;                       // rounding may leave the whole set just short of the target
    __syncthreads();
    if (group_end && tid < cnt_k && upto >= target) atomicMin(&sh.cross_bin, tid);
    __syncthreads();
    if (tid == sh.cross_bin) {
        sh.tau = x;
        sh.res_cnt = tid + 1;
        sh.res_mass = upto;
    }
    __syncthreads();
    return true;
}

// The usual case of a long row and a small top_k, or a nucleus of a few hundred tokens at most (any peaked
// distribution), in one pass over the row.  A sample of 32 tokens per thread, in evenly spaced 128-byte runs, is
// binned first; the bin at which the sample's running count reaches a chosen number gives a cut theta
// that, for the whole row, is expected to leave a few hundred tokens: at least top_k and no more than the exact
// stage holds.  The pass over the row then appends every token >= theta to the candidate list in shared memory
// (no histogram: a compare per token), and both the top-k threshold and the nucleus inside the top-k set are
// resolved in the sorted list.  The sample only places the cut: the list is complete above theta whatever it was.
// A list that came out too short or too long is taken again with the cut moved; if that does not settle it, or the
// nucleus is longer than a list can be, nothing is decided (returns false: the general selection takes over).
__device__ bool one_pass(const Row& r, int top_k, float top_p, Shared& sh) {
    const int tid = threadIdx.x;
    constexpr int SAMPLE4 = 8;                                    // float4 loads per thread in the sample
    const int n4 = r.V >> 2;
    if ((r.V & 3) != 0 || n4 < 8 * SAMPLE4 * THREADS) return false;
    Level lv;
    lv.by_key = 0;
    lv.ztop = r.lc / r.c;
    lv.scale = (float)NB / ((logf((float)r.V) + 20.f) / (r.c / LOG2E));
    lv.klo = 0;
    lv.khi = 0xffffffffu;
    constexpr int PER = (NB + 1 + THREADS - 1) / THREADS;
    for (int i = tid; i <= NB; i += THREADS) sh.cnt[i] = 0;
    if (tid == 0) {
        sh.cross_bin = NB + 1;
        sh.n_cand = 0;
    }
    __syncthreads();
    {
        const float4* z4 = reinterpret_cast<const float4*>(r.z);
        // runs of 128 bytes (a DRAM burst is used whole), evenly spaced over the row
        const int run_stride = n4 / (SAMPLE4 * THREADS / 8);
        float4 x[SAMPLE4];
#pragma unroll
        for (int u = 0; u < SAMPLE4; ++u) {
            const int j = u * THREADS + tid;
            x[u] = __ldg(z4 + (size_t)(j >> 3) * run_stride + (j & 7));
        }
#pragma unroll
        for (int u = 0; u < SAMPLE4; ++u) {
            atomicAdd(&sh.cnt[bin_of(lv, x[u].x + 0.f)], 1);
            atomicAdd(&sh.cnt[bin_of(lv, x[u].y + 0.f)], 1);
            atomicAdd(&sh.cnt[bin_of(lv, x[u].z + 0.f)], 1);
            atomicAdd(&sh.cnt[bin_of(lv, x[u].w + 0.f)], 1);
        }
    }
    __syncthreads();
    // the list should hold about max(2 top_k, top_k + 256) tokens, and at most 3/4 of its capacity (which is what a
    // nucleus alone gets, its size being unknown)
    const int want = top_k > 0 ? min(max(2 * top_k, top_k + 256), 3 * LIST / 4) : 3 * LIST / 4;
    const float ratio = (float)r.V / (float)(4 * SAMPLE4 * THREADS);
    int s_target = max((int)ceilf((float)want / ratio), 4);
    int c = 0;
    for (int j = 0; j < PER; ++j) {
        const int b = tid * PER + j;
        if (b <= NB) c += sh.cnt[b];
    }
    int ec, tc;
    double em, tm;
    block_scan(c, 0.0, ec, em, &tc, &tm, sh);
    // A list that came out too long or too short moves the cut by what it counted and takes the pass again (the row
    // is in L2 by then): three attempts at most.
    for (int attempt = 0; attempt < 3; ++attempt) {
        if (tid == 0) {
            sh.cross_bin = NB + 1;
            sh.n_cand = 0;
        }
        __syncthreads();
        {
            int rc = ec;
            for (int j = 0; j < PER; ++j) {
                const int b = tid * PER + j;
                if (b > NB) break;
                rc += sh.cnt[b];
                if (rc >= s_target) {
                    atomicMin(&sh.cross_bin, b);
                    break;
                }
            }
        }
        __syncthreads();
        const int bs = sh.cross_bin;
        __syncthreads();
        if (bs >= NB) return false;                               // the cut would fall below the binned range
        const float theta = lv.ztop - (float)(bs + 1) / lv.scale;
        {
            const float4* z4 = reinterpret_cast<const float4*>(r.z);
            auto keep = [&](float z) {
                if (z >= theta) {
                    const int slot = atomicAdd(&sh.n_cand, 1);
                    if (slot < LIST) sh.cz[slot] = z + 0.f;
                }
            };
            for (int i0 = tid; i0 < n4; i0 += 4 * THREADS) {
                float4 x[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int i = i0 + u * THREADS;
                    x[u] = i < n4 ? __ldg(z4 + i) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (fmaxf(fmaxf(x[u].x, x[u].y), fmaxf(x[u].z, x[u].w)) >= theta) {   // one test per 16 bytes; few pass
                        keep(x[u].x);
                        keep(x[u].y);
                        keep(x[u].z);
                        keep(x[u].w);
                    }
            }
        }
        __syncthreads();
        const int n = sh.n_cand;
        __syncthreads();
        int s_next;
        if (n > LIST) {
            s_next = (int)((float)s_target * (0.6f * (float)LIST / (float)n));
        } else if (n < max(top_k, 1)) {
            s_next = (int)ceilf((float)s_target * 1.5f * (float)want / (float)max(n, 1));
        } else {
            if (resolve_sorted(r, sh, n, top_k, top_p)) return true;
            if (2 * n > LIST) return false;                       // the nucleus is longer than a list can be
            s_next = 2 * s_target;
        }
        if (s_next < 1 || s_next == s_target) return false;
        s_target = s_next;
    }
    return false;
}

__global__ void __launch_bounds__(THREADS, 2) truncate_kernel(int M, int V, const float* __restrict__ logits,
                                                              const float* __restrict__ lse, float inv_t, int top_k, float top_p,
                                                              float* __restrict__ tau_out, float* __restrict__ lse_out) {
    extern __shared__ unsigned char smem_raw[];
    Shared& sh = *reinterpret_cast<Shared*>(smem_raw);
    pdl_trigger();
    pdl_wait();
    for (int m = blockIdx.x; m < M; m += gridDim.x) {
        Row r;
        r.z = logits + (size_t)m * V;
        r.V = V;
        r.c = inv_t * LOG2E;
        r.lc = lse[m] * LOG2E;
        r.floor_z = -INFINITY;
        float tau = -INFINITY;
        double mass = 1.0;
        bool any = false;
        bool done = false;
        const bool cut_by_count = top_k > 0 && top_k < V;
        if (cut_by_count ? top_k <= LIST / 4 : top_p < 1.f) {
            done = one_pass(r, cut_by_count ? top_k : 0, top_p, sh);
            __syncthreads();
            if (done) {
                tau = sh.tau;
                mass = sh.res_mass;
                any = true;
            }
            __syncthreads();
        }
        if (!done && top_k > 0 && top_k < V) {
            select_level_set(r, BY_COUNT, top_k, 0.f, sh);
            tau = sh.tau;
            mass = sh.res_mass;
            any = true;
            __syncthreads();
        }
        if (!done && top_p < 1.f) {
            r.floor_z = tau;
            select_level_set(r, BY_MASS, 0, top_p, sh);
            tau = sh.tau;
            mass = sh.res_mass;
            any = true;
            __syncthreads();
        }
        if (threadIdx.x == 0) {
            tau_out[m] = tau;
            lse_out[m] = any ? lse[m] + (float)log(mass) : lse[m];
        }
        __syncthreads();
    }
}

}  // namespace

extern "C" int deer_truncate(int M, int V, const float* target_logits, const float* target_lse, float temperature, int top_k,
                             float top_p, float* tau, float* lse_trunc, void* stream) {
    DEER_CHECK_ARG(target_logits && target_lse && tau && lse_trunc, DEER_ERR_INVALID_ARG, "deer_truncate: null argument");
    DEER_CHECK_ARG(deer_aligned16(target_logits), DEER_ERR_INVALID_ARG, "deer_truncate: logits must be 16-byte aligned");
    DEER_CHECK_ARG(M >= 0 && V > 0, DEER_ERR_INVALID_ARG, "deer_truncate: bad sizes");
    DEER_CHECK_ARG(temperature > 0.f && top_p > 0.f, DEER_ERR_INVALID_ARG, "deer_truncate: temperature and top_p must be positive");
    if (M == 0) return DEER_OK;
    const int sms = deer_sm_count();
    DEER_CUDA(cudaFuncSetAttribute(truncate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(Shared)));
    DEER_CUDA(launch_pdl(truncate_kernel, dim3(M < 2 * sms ? M : 2 * sms), dim3(THREADS), sizeof(Shared), static_cast<cudaStream_t>(stream), M, V,
                         target_logits, target_lse, 1.f / temperature, top_k, top_p, tau, lse_trunc));
    return DEER_OK;
}
