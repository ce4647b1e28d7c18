// Paged-KV manager: the committed prefix x_{1:j} as pages, with reserve (room
// for the next block) and commit/rollback to the accepted length
// (Section 3.2 and Algorithm 1's update of j).
//
// Both kernels run as ONE thread block: thread b owns sequence seq_ids[b],
// a block-wide exclusive scan gives each sequence its offset on the free
// stack, so the result is the same as visiting the sequences one after the
// other while every sequence still moves its pages in parallel.

#include <stdarg.h>
#include <string.h>

#include <new>

#include "common.cuh"
#include "greedy.cuh"

// ---- error text ------------------------------------------------------------
static thread_local char g_err[512] = "";

void deer_set_error(const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}

extern "C" const char* deer_last_error(void) { return g_err; }

// ---- handle ----------------------------------------------------------------
extern "C" int deer_kv_create(deer_kv** kv, const deer_kv_desc* desc) {
    DEER_CHECK_ARG(kv && desc, DEER_ERR_INVALID_ARG, "deer_kv_create: null argument");
    const deer_kv_desc& d = *desc;
    DEER_CHECK_ARG(d.k_pool && d.v_pool && d.page_table && d.seq_len && d.n_pages && d.free_stack && d.free_top && d.status,
                   DEER_ERR_INVALID_ARG, "deer_kv_create: null device pointer in desc");
    DEER_CHECK_ARG(deer_aligned16(d.k_pool) && deer_aligned16(d.v_pool), DEER_ERR_INVALID_ARG,
                   "deer_kv_create: pools must be 16-byte aligned");
    DEER_CHECK_ARG(d.page_size == DEER_PAGE_SIZE, DEER_ERR_UNSUPPORTED, "deer_kv_create: page_size must be 16");
    DEER_CHECK_ARG(d.head_dim == 64 || d.head_dim == 128, DEER_ERR_UNSUPPORTED, "deer_kv_create: head_dim must be 64 or 128");
    DEER_CHECK_ARG(d.num_pages > 0 && d.n_kv_heads > 0 && d.max_seqs > 0 && d.max_pages > 0, DEER_ERR_INVALID_ARG,
                   "deer_kv_create: sizes must be positive");
    deer_kv* h = new (std::nothrow) deer_kv;
    DEER_CHECK_ARG(h, DEER_ERR_INVALID_ARG, "deer_kv_create: out of host memory");
    h->d = d;
    *kv = h;
    return DEER_OK;
}

extern "C" int deer_kv_destroy(deer_kv* kv) {
    delete kv;
    return DEER_OK;
}

extern "C" int deer_kv_status(deer_kv* kv, int32_t* code, void* stream) {
    DEER_CHECK_ARG(kv && code, DEER_ERR_INVALID_ARG, "deer_kv_status: null argument");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    DEER_CUDA(cudaMemcpyAsync(code, kv->d.status, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    DEER_CUDA(cudaMemsetAsync(kv->d.status, 0, sizeof(int32_t), st));
    DEER_CUDA(cudaStreamSynchronize(st));
    return DEER_OK;
}

// ---- kernels ---------------------------------------------------------------
constexpr int KV_THREADS = 1024;

// Exclusive scan of one int per thread over the block; returns the exclusive
// prefix, *total gets the block sum.
__device__ __forceinline__ int block_exclusive_scan(int v, int* total, int* warp_sums) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = warp_sums[lane];
        int wi = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int t = __shfl_up_sync(0xffffffffu, wi, o);
            if (lane >= o) wi += t;
        }
        warp_sums[lane] = wi - w;  // exclusive
        if (lane == 31) *total = wi;
    }
    __syncthreads();
    return warp_sums[warp] + incl - v;
}

__global__ void __launch_bounds__(KV_THREADS)
kv_reserve_kernel(deer_kv_desc d, const int32_t* __restrict__ seq_ids, int B, int k) {
    __shared__ int warp_sums[32];
    __shared__ int total;
    __shared__ int bad;
    const int b = threadIdx.x;
    pdl_trigger();
    pdl_wait();
    if (b == 0) bad = 0;
    __syncthreads();
    int s = -1, have = 0, need_pages = 0;
    if (b < B) {
        s = seq_ids[b];
        if (s < 0 || s >= d.max_seqs) {
            atomicExch(&bad, DEER_ERR_INVALID_ARG);
            s = -1;
        } else {
            have = d.n_pages[s];
            need_pages = (d.seq_len[s] + k + d.page_size - 1) / d.page_size;
            if (need_pages > d.max_pages) atomicExch(&bad, DEER_ERR_NO_PAGES);
        }
    }
    const int extra = (s >= 0 && need_pages > have) ? need_pages - have : 0;
    const int offset = block_exclusive_scan(extra, &total, warp_sums);
    const int top = *d.free_top;
    if (b == 0 && total > top) bad = DEER_ERR_NO_PAGES;
    __syncthreads();
    if (bad) {
        if (b == 0) deer_report(d.status, bad);
        return;
    }
    if (extra > 0) {
        int32_t* row = d.page_table + (size_t)s * d.max_pages;
        for (int j = 0; j < extra; ++j) row[have + j] = d.free_stack[top - 1 - (offset + j)];
        d.n_pages[s] = need_pages;
    }
    __syncthreads();
    if (b == 0) *d.free_top = top - total;
}

// The body of the commit for thread b of the block: seq_len[s] += keep (clamped), pages wholly beyond the new length
// go back to the free stack.  `keep` is this thread's sequence's value; every thread of the block calls it.
__device__ __forceinline__ void commit_rows(const deer_kv_desc& d, const int32_t* __restrict__ seq_ids, int keep, int B, int k,
                                            int* warp_sums, int* total) {
    const int b = threadIdx.x;
    int s = -1, have = 0, need_pages = 0;
    if (b < B) {
        s = seq_ids[b];
        if (s < 0 || s >= d.max_seqs) {
            deer_report(d.status, DEER_ERR_INVALID_ARG);
            s = -1;
        } else {
            int kp = keep;
            kp = kp < 0 ? 0 : (kp > k ? k : kp);
            have = d.n_pages[s];
            int n = d.seq_len[s] + kp;
            const int cap = have * d.page_size;     // rows can only be kept where pages were reserved
            if (n > cap) {
                deer_report(d.status, DEER_ERR_BAD_PAGE);
                n = cap;
            }
            d.seq_len[s] = n;
            need_pages = (n + d.page_size - 1) / d.page_size;
        }
    }
    const int surplus = (s >= 0 && have > need_pages) ? have - need_pages : 0;
    const int offset = block_exclusive_scan(surplus, total, warp_sums);
    const int top = *d.free_top;
    if (top + *total > d.num_pages) {         // inconsistent state: more pages returned than exist
        if (b == 0) deer_report(d.status, DEER_ERR_BAD_PAGE);
        return;
    }
    if (surplus > 0) {
        int32_t* row = d.page_table + (size_t)s * d.max_pages;
        for (int j = 0; j < surplus; ++j) {
            d.free_stack[top + offset + j] = row[have - 1 - j];
            row[have - 1 - j] = -1;
        }
        d.n_pages[s] = need_pages;
    }
    __syncthreads();
    if (b == 0) *d.free_top = top + *total;
}

__global__ void __launch_bounds__(KV_THREADS)
kv_commit_kernel(deer_kv_desc d, const int32_t* __restrict__ seq_ids, const int32_t* __restrict__ keep, int B, int k) {
    __shared__ int warp_sums[32];
    __shared__ int total;
    pdl_trigger();
    pdl_wait();
    commit_rows(d, seq_ids, threadIdx.x < B ? keep[threadIdx.x] : 0, B, k, warp_sums, &total);
}

// Greedy acceptance and the commit of what it accepted, one thread per sequence: the end of a greedy verify step in
// one launch.  The mirror_* pointers, when given, receive a second copy of the three results (page-locked host
// memory the device can write: the host-buffer step then needs no copy back).
__global__ void __launch_bounds__(KV_THREADS)
kv_accept_commit_kernel(deer_kv_desc d, const int32_t* __restrict__ seq_ids, int B, int k, int kd, const int32_t* __restrict__ draft,
                        const int32_t* __restrict__ target, int32_t eos_id, int32_t* __restrict__ accept_len,
                        int32_t* __restrict__ out_ids, int32_t* __restrict__ n_out, int32_t* __restrict__ mirror_accept_len,
                        int32_t* __restrict__ mirror_out_ids, int32_t* __restrict__ mirror_n_out) {
    __shared__ int warp_sums[32];
    __shared__ int total;
    const int b = threadIdx.x;
    pdl_trigger();
    pdl_wait();
    int a = 0;
    if (b < B) {
        int n;
        a = greedy_accept_row(draft + (size_t)b * k, target + (size_t)b * k, out_ids + (size_t)b * k, k, kd, eos_id, &n);
        accept_len[b] = a;
        n_out[b] = n;
        if (mirror_accept_len) {
            mirror_accept_len[b] = a;
            mirror_n_out[b] = n;
            for (int i = 0; i < k; ++i) mirror_out_ids[(size_t)b * k + i] = out_ids[(size_t)b * k + i];
            __threadfence_system();
        }
    }
    commit_rows(d, seq_ids, a, B, k, warp_sums, &total);
}

// ---- entry points ----------------------------------------------------------
extern "C" int deer_kv_reserve(deer_kv* kv, const int32_t* seq_ids, int B, int k, void* stream) {
    DEER_CHECK_ARG(kv && seq_ids, DEER_ERR_INVALID_ARG, "deer_kv_reserve: null argument");
    DEER_CHECK_ARG(B >= 0 && B <= KV_THREADS, DEER_ERR_UNSUPPORTED, "deer_kv_reserve: B must be in [0, %d]", KV_THREADS);
    DEER_CHECK_ARG(k >= 0 && k <= DEER_MAX_BLOCK, DEER_ERR_UNSUPPORTED, "deer_kv_reserve: k must be in [0, 32]");
    if (B == 0) return DEER_OK;
    DEER_CUDA(launch_pdl(kv_reserve_kernel, dim3(1), dim3(KV_THREADS), 0, static_cast<cudaStream_t>(stream), kv->d, seq_ids, B, k));
    return DEER_OK;
}

extern "C" int deer_kv_commit(deer_kv* kv, const int32_t* seq_ids, const int32_t* keep, int B, int k, void* stream) {
    DEER_CHECK_ARG(kv && seq_ids && keep, DEER_ERR_INVALID_ARG, "deer_kv_commit: null argument");
    DEER_CHECK_ARG(B >= 0 && B <= KV_THREADS, DEER_ERR_UNSUPPORTED, "deer_kv_commit: B must be in [0, %d]", KV_THREADS);
    DEER_CHECK_ARG(k >= 0 && k <= DEER_MAX_BLOCK, DEER_ERR_UNSUPPORTED, "deer_kv_commit: k must be in [0, 32]");
    if (B == 0) return DEER_OK;
    DEER_CUDA(launch_pdl(kv_commit_kernel, dim3(1), dim3(KV_THREADS), 0, static_cast<cudaStream_t>(stream), kv->d, seq_ids, keep, B, k));
    return DEER_OK;
}

// deer_accept_commit with a second copy of the results written to mirror_* (all three or none; memory the device
// can write, e.g. page-locked host memory).  Not part of the C ABI: the host-buffer step uses it.
int deer_accept_commit_mirrored(deer_kv* kv, const int32_t* seq_ids, int mode, int B, int k, const int32_t* draft_ids,
                                const int32_t* target_ids, int32_t eos_id, int32_t* accept_len, int32_t* out_ids, int32_t* n_out,
                                int32_t* mirror_accept_len, int32_t* mirror_out_ids, int32_t* mirror_n_out, void* stream) {
    DEER_CHECK_ARG(kv && seq_ids && draft_ids && target_ids && accept_len && out_ids && n_out, DEER_ERR_INVALID_ARG,
                   "deer_accept_commit: null argument");
    DEER_CHECK_ARG((mode & ~DEER_ACC_BONUS) == DEER_ACC_GREEDY, DEER_ERR_UNSUPPORTED,
                   "deer_accept_commit: greedy acceptance only (sampling takes deer_accept, then deer_kv_commit)");
    DEER_CHECK_ARG(B >= 0 && B <= KV_THREADS, DEER_ERR_UNSUPPORTED, "deer_accept_commit: B must be in [0, %d]", KV_THREADS);
    DEER_CHECK_ARG(k >= 1 && k <= DEER_MAX_BLOCK, DEER_ERR_UNSUPPORTED, "deer_accept_commit: k must be in [1, 32]");
    if (B == 0) return DEER_OK;
    const int kd = (mode & DEER_ACC_BONUS) ? k - 1 : k;
    DEER_CUDA(launch_pdl(kv_accept_commit_kernel, dim3(1), dim3(KV_THREADS), 0, static_cast<cudaStream_t>(stream), kv->d, seq_ids, B, k,
                         kd, draft_ids, target_ids, eos_id, accept_len, out_ids, n_out, mirror_accept_len, mirror_out_ids,
                         mirror_n_out));
    return DEER_OK;
}

extern "C" int deer_accept_commit(deer_kv* kv, const int32_t* seq_ids, int mode, int B, int k, const int32_t* draft_ids,
                                  const int32_t* target_ids, int32_t eos_id, int32_t* accept_len, int32_t* out_ids, int32_t* n_out,
                                  void* stream) {
    return deer_accept_commit_mirrored(kv, seq_ids, mode, B, k, draft_ids, target_ids, eos_id, accept_len, out_ids, n_out, nullptr,
                                       nullptr, nullptr, stream);
}
