// One greedy verify step driven from host buffers: the end-to-end form of
// Algorithm 1's loop body on the verifier side (copy the block in, score it,
// accept, commit, copy the results out).
//
// The five copies in, eight kernels and three copies out are sixteen
// enqueue calls; issued one by one they cost more host time than the copies
// take on the bus.  So the sequence is captured once into a CUDA graph, keyed
// by every argument (the whole cache descriptor and the whole staging-buffer
// struct included: a graph holds them by value), and replayed with one launch
// while the arguments stay the same (a decoding loop calls with the same
// buffers every step).  A few graphs are kept, so that callers that alternate
// do not evict each other.  Pageable host buffers, the legacy default stream
// and a stream that is already being captured take the plain path.

#include <string.h>

#include <mutex>

#include <cuda.h>

#include "common.cuh"

namespace {

// Everything the recorded copies and kernels hold by value.  Compared with memcmp, so it is filled field by field
// into zeroed memory (no padding bytes left undefined).
struct StepKey {
    deer_kv_desc kv;
    deer_step_dev dev;
    const void* kv_handle;
    const void* w;
    const void* host[8];
    int i[6];
    float scale;
    int device;
};

struct StepCache {
    StepKey key;
    cudaGraphExec_t exec = nullptr;
    unsigned long long used = 0;      // value of g_clock at the last launch: the least recently used entry is replaced
};

constexpr int N_CACHED = 4;
std::mutex g_mu;
StepCache g_cache[N_CACHED];
unsigned long long g_clock = 0;

// A second stream for the copies that the attention does not need (hidden states, draft ids): they cross the bus
// while the attention kernel runs.  Created on first use; they belong to the device that was current then and are
// made anew when the call comes on another device (the cached graph is keyed by the device as well).
cudaStream_t g_side = nullptr;
cudaEvent_t g_fork = nullptr, g_join = nullptr;
int g_side_device = -1;

int side_stream() {
    int device = 0;
    DEER_CUDA(cudaGetDevice(&device));
    if (g_side && g_side_device == device) return DEER_OK;
    g_side = nullptr;                 // the old ones stay with their device for the life of the process
    DEER_CUDA(cudaStreamCreateWithFlags(&g_side, cudaStreamNonBlocking));
    DEER_CUDA(cudaEventCreateWithFlags(&g_fork, cudaEventDisableTiming));
    DEER_CUDA(cudaEventCreateWithFlags(&g_join, cudaEventDisableTiming));
    g_side_device = device;
    return DEER_OK;
}

// True when [p, p + bytes) lies inside one allocation (host or device): a single copy must not cross from one
// allocation into a neighbour that merely happens to follow it in the address space.
bool one_allocation(const void* p, size_t bytes) {
    typedef CUresult (*range_fn)(CUdeviceptr*, size_t*, CUdeviceptr);
    static range_fn fn = [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuMemGetAddressRange", &f, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess)
            f = nullptr;
        cudaGetLastError();
        return reinterpret_cast<range_fn>(f);
    }();
    if (!fn) return false;
    CUdeviceptr base = 0;
    size_t size = 0;
    if (fn(&base, &size, reinterpret_cast<CUdeviceptr>(p)) != CUDA_SUCCESS) return false;
    const CUdeviceptr a = reinterpret_cast<CUdeviceptr>(p);
    return a >= base && a + bytes <= base + size;
}

int enqueue(deer_kv* kv, const deer_step_dev* dev, const void* w, const void* q_host, const void* k_blk_host,
            const void* v_blk_host, const void* h_host, const int32_t* draft_ids_host, int B, int k, int Hq, int hid, int V,
            float scale, int max_seq_len, int32_t* accept_len_host, int32_t* out_ids_host, int32_t* n_out_host, void* stream,
            bool fork) {
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int Hkv = kv->d.n_kv_heads, D = kv->d.head_dim;
    const size_t M = (size_t)B * k;
    // fork (worth its extra calls only where they are recorded once): hidden states and draft ids on the second stream
    int rc = DEER_OK;
    cudaStream_t sh = st;
    if (fork) {
        rc = side_stream();
        if (rc != DEER_OK) return rc;
        sh = g_side;
        DEER_CUDA(cudaEventRecord(g_fork, st));
        DEER_CUDA(cudaStreamWaitEvent(g_side, g_fork, 0));
    }
    DEER_CUDA(cudaMemcpyAsync(dev->h, h_host, M * hid * 2, cudaMemcpyHostToDevice, sh));
    DEER_CUDA(cudaMemcpyAsync(dev->draft_ids, draft_ids_host, M * sizeof(int32_t), cudaMemcpyHostToDevice, sh));
    if (fork) DEER_CUDA(cudaEventRecord(g_join, g_side));
    // q, k_blk and v_blk go in one copy where they follow one another in memory on both sides
    const size_t q_bytes = M * Hq * D * 2, kv_bytes = M * Hkv * D * 2;
    auto at = [](const void* p, size_t off) { return static_cast<const char*>(p) + off; };
    if (at(q_host, q_bytes) == k_blk_host && at(k_blk_host, kv_bytes) == v_blk_host && at(dev->q, q_bytes) == dev->k_blk &&
        at(dev->k_blk, kv_bytes) == dev->v_blk && one_allocation(q_host, q_bytes + 2 * kv_bytes) &&
        one_allocation(dev->q, q_bytes + 2 * kv_bytes)) {
        DEER_CUDA(cudaMemcpyAsync(dev->q, q_host, q_bytes + 2 * kv_bytes, cudaMemcpyHostToDevice, st));
    } else {
        DEER_CUDA(cudaMemcpyAsync(dev->q, q_host, q_bytes, cudaMemcpyHostToDevice, st));
        DEER_CUDA(cudaMemcpyAsync(dev->k_blk, k_blk_host, kv_bytes, cudaMemcpyHostToDevice, st));
        DEER_CUDA(cudaMemcpyAsync(dev->v_blk, v_blk_host, kv_bytes, cudaMemcpyHostToDevice, st));
    }
    rc = deer_kv_reserve(kv, dev->seq_ids, B, k, stream);
    if (rc != DEER_OK) return rc;
    rc = deer_block_attn(kv, dev->seq_ids, dev->q, dev->k_blk, dev->v_blk, dev->attn_out, B, k, Hq, DEER_MASK_CAUSAL, 1, scale,
                         max_seq_len, dev->attn_ws, dev->attn_ws_bytes, stream);
    if (rc != DEER_OK) return rc;
    if (fork) DEER_CUDA(cudaStreamWaitEvent(st, g_join, 0));
    rc = deer_lmhead_select(dev->h, w, (int)M, hid, V, DEER_SEL_ARGMAX, 1.f, nullptr, dev->target_ids, nullptr, nullptr, nullptr,
                            nullptr, dev->lm_ws, dev->lm_ws_bytes, stream);
    if (rc != DEER_OK) return rc;
    // In the recorded form (page-locked result buffers, which the device can write) the last kernel leaves a second
    // copy of the results in the host buffers itself; otherwise they are copied back, in one piece where they follow
    // one another inside one allocation on both sides.
    if (fork) {
        void *ma = nullptr, *mo = nullptr, *mn = nullptr;        // the host buffers as the device addresses them
        if (cudaHostGetDevicePointer(&ma, accept_len_host, 0) == cudaSuccess && cudaHostGetDevicePointer(&mo, out_ids_host, 0) == cudaSuccess &&
            cudaHostGetDevicePointer(&mn, n_out_host, 0) == cudaSuccess) {
            return deer_accept_commit_mirrored(kv, dev->seq_ids, DEER_ACC_GREEDY, B, k, dev->draft_ids, dev->target_ids, -1,
                                               dev->accept_len, dev->out_ids, dev->n_out, static_cast<int32_t*>(ma),
                                               static_cast<int32_t*>(mo), static_cast<int32_t*>(mn), stream);
        }
        cudaGetLastError();
    }
    rc = deer_accept_commit(kv, dev->seq_ids, DEER_ACC_GREEDY, B, k, dev->draft_ids, dev->target_ids, -1, dev->accept_len,
                            dev->out_ids, dev->n_out, stream);
    if (rc != DEER_OK) return rc;
    if (accept_len_host + B == out_ids_host && out_ids_host + M == n_out_host && dev->accept_len + B == dev->out_ids &&
        dev->out_ids + M == dev->n_out && one_allocation(accept_len_host, (2 * (size_t)B + M) * sizeof(int32_t)) &&
        one_allocation(dev->accept_len, (2 * (size_t)B + M) * sizeof(int32_t))) {
        DEER_CUDA(cudaMemcpyAsync(accept_len_host, dev->accept_len, (2 * (size_t)B + M) * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    } else {
        DEER_CUDA(cudaMemcpyAsync(accept_len_host, dev->accept_len, (size_t)B * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
        DEER_CUDA(cudaMemcpyAsync(out_ids_host, dev->out_ids, M * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
        DEER_CUDA(cudaMemcpyAsync(n_out_host, dev->n_out, (size_t)B * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    }
    return DEER_OK;
}

bool pinned(const void* p) {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, p) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return at.type == cudaMemoryTypeHost;
}

}  // namespace

extern "C" int deer_verify_step_host(deer_kv* kv, const deer_step_dev* dev, const void* w, const void* q_host,
                                     const void* k_blk_host, const void* v_blk_host, const void* h_host,
                                     const int32_t* draft_ids_host, int B, int k, int Hq, int hid, int V, float scale,
                                     int max_seq_len, int32_t* accept_len_host, int32_t* out_ids_host, int32_t* n_out_host,
                                     void* stream) {
    DEER_CHECK_ARG(kv && dev && w && q_host && k_blk_host && v_blk_host && h_host && draft_ids_host && accept_len_host &&
                       out_ids_host && n_out_host,
                   DEER_ERR_INVALID_ARG, "deer_verify_step_host: null argument");
    DEER_CHECK_ARG(B > 0 && k >= 1 && k <= DEER_MAX_BLOCK, DEER_ERR_UNSUPPORTED, "deer_verify_step_host: bad B or k");
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    DEER_CUDA(cudaStreamIsCapturing(st, &cap));
    // the legacy default stream cannot be captured
    const bool use_graph = st != nullptr && cap == cudaStreamCaptureStatusNone && pinned(q_host) && pinned(k_blk_host) &&
                           pinned(v_blk_host) && pinned(h_host) && pinned(draft_ids_host) && pinned(accept_len_host) &&
                           pinned(out_ids_host) && pinned(n_out_host);
    if (!use_graph) {
        const int rc = enqueue(kv, dev, w, q_host, k_blk_host, v_blk_host, h_host, draft_ids_host, B, k, Hq, hid, V, scale,
                               max_seq_len, accept_len_host, out_ids_host, n_out_host, stream, false);
        if (rc != DEER_OK) return rc;
        DEER_CUDA(cudaStreamSynchronize(st));
        return DEER_OK;
    }

    StepKey key;
    memset(&key, 0, sizeof(key));
    {
        const deer_kv_desc& d = kv->d;
        key.kv.k_pool = d.k_pool; key.kv.v_pool = d.v_pool; key.kv.page_table = d.page_table; key.kv.seq_len = d.seq_len;
        key.kv.n_pages = d.n_pages; key.kv.free_stack = d.free_stack; key.kv.free_top = d.free_top; key.kv.status = d.status;
        key.kv.num_pages = d.num_pages; key.kv.n_kv_heads = d.n_kv_heads; key.kv.head_dim = d.head_dim;
        key.kv.page_size = d.page_size; key.kv.max_seqs = d.max_seqs; key.kv.max_pages = d.max_pages;
        key.dev.q = dev->q; key.dev.k_blk = dev->k_blk; key.dev.v_blk = dev->v_blk; key.dev.attn_out = dev->attn_out;
        key.dev.h = dev->h; key.dev.seq_ids = dev->seq_ids; key.dev.draft_ids = dev->draft_ids;
        key.dev.target_ids = dev->target_ids; key.dev.accept_len = dev->accept_len; key.dev.out_ids = dev->out_ids;
        key.dev.n_out = dev->n_out; key.dev.attn_ws = dev->attn_ws; key.dev.attn_ws_bytes = dev->attn_ws_bytes;
        key.dev.lm_ws = dev->lm_ws; key.dev.lm_ws_bytes = dev->lm_ws_bytes;
    }
    key.kv_handle = kv;
    key.w = w;
    const void* hosts[8] = {q_host, k_blk_host, v_blk_host, h_host, draft_ids_host, accept_len_host, out_ids_host, n_out_host};
    for (int j = 0; j < 8; ++j) key.host[j] = hosts[j];
    const int ints[6] = {B, k, Hq, hid, V, max_seq_len};
    for (int j = 0; j < 6; ++j) key.i[j] = ints[j];
    key.scale = scale;
    DEER_CUDA(cudaGetDevice(&key.device));

    std::lock_guard<std::mutex> lock(g_mu);
    StepCache* slot = nullptr;
    for (StepCache& c : g_cache)
        if (c.exec && memcmp(&c.key, &key, sizeof(key)) == 0) slot = &c;
    if (!slot) {
        slot = &g_cache[0];
        for (StepCache& c : g_cache)
            if (!c.exec || (slot->exec && c.used < slot->used)) slot = &c;     // a free entry, else the least recently used
        if (slot->exec) {
            cudaGraphExecDestroy(slot->exec);
            slot->exec = nullptr;
        }
        DEER_CUDA(cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal));
        const int rc = enqueue(kv, dev, w, q_host, k_blk_host, v_blk_host, h_host, draft_ids_host, B, k, Hq, hid, V, scale,
                               max_seq_len, accept_len_host, out_ids_host, n_out_host, stream, true);
        cudaGraph_t graph = nullptr;
        const cudaError_t ce = cudaStreamEndCapture(st, &graph);      // always, so that the stream leaves capture mode
        if (rc != DEER_OK) {
            if (graph) cudaGraphDestroy(graph);
            cudaGetLastError();
            return rc;
        }
        DEER_CUDA(ce);
        const cudaError_t ci = cudaGraphInstantiate(&slot->exec, graph, 0);
        cudaGraphDestroy(graph);
        if (ci != cudaSuccess) slot->exec = nullptr;
        DEER_CUDA(ci);
        slot->key = key;
    }
    slot->used = ++g_clock;
    DEER_CUDA(cudaGraphLaunch(slot->exec, st));
    DEER_CUDA(cudaStreamSynchronize(st));
    return DEER_OK;
}
