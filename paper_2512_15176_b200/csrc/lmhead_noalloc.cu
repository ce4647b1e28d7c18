// deer_lmhead_select_static: the LM head + selection call for callers that
// cannot hand the library any scratch memory.
//
// Some hosts of this library may not allocate device memory at the point where
// they call it: a serving loop whose memory pool is sealed after start-up, a
// plug-in that is only given its input and output tensors, or code running
// inside a region where the CUDA allocator must not be entered.  For them the
// cross-block partial results of the LM head live in a fixed array that is part
// of the library image itself, so the call needs nothing beyond inputs and
// outputs.  The price: the array is sized for at most DEER_STATIC_MAX_ROWS rows,
// every GPU that loads the library carries it until the process exits, and all
// calls on one GPU share it.

#include <mutex>

#include "common.cuh"

namespace {

// Room for 2 * 148 vocabulary parts x DEER_STATIC_MAX_ROWS rows x 16 bytes of selection state (the call uses one
// part per SM) and the arrival words behind them.  The runtime zero-fills it when the library is loaded.
constexpr size_t STATIC_SCRATCH_BYTES = (size_t)2 * 148 * DEER_STATIC_MAX_ROWS * 16;

static __device__ __align__(256) unsigned char g_lmhead_scratch[STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
std::mutex g_mu;
void* g_scratch_addr[MAX_DEVICES] = {};   // device address of g_lmhead_scratch on each device, once resolved

// In host code `g_lmhead_scratch` is only a handle for the runtime, not a
// device address; the address valid on the current device has to be asked for.
int scratch_for_current_device(void** out, cudaStream_t st) {
    int dev = -1;
    DEER_CUDA(cudaGetDevice(&dev));
    DEER_CHECK_ARG(dev >= 0 && dev < MAX_DEVICES, DEER_ERR_UNSUPPORTED, "deer_lmhead_select_static: device index %d not supported", dev);
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[dev]) {
        // the look-up is a runtime call that a stream capture must not see: say so instead of spoiling the capture
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        DEER_CUDA(cudaStreamIsCapturing(st, &cap));
        DEER_CHECK_ARG(cap == cudaStreamCaptureStatusNone, DEER_ERR_UNSUPPORTED,
                       "deer_lmhead_select_static: the first call on a device must come before any stream capture");
        void* p = nullptr;
        DEER_CUDA(cudaGetSymbolAddress(&p, g_lmhead_scratch));
        DEER_CHECK_ARG(p != nullptr, DEER_ERR_CUDA, "deer_lmhead_select_static: scratch symbol has no device address");
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return DEER_OK;
}

}  // namespace

extern "C" size_t deer_lmhead_static_max_rows(void) { return DEER_STATIC_MAX_ROWS; }

extern "C" int deer_lmhead_select_static(const void* h, const void* w, int M, int hid, int V, int mode, float temperature,
                                         const int32_t* draft_ids, int32_t* out_ids, float* out_max_logprob, float* out_lse,
                                         float* out_draft_logit, float* out_logits, void* stream) {
    DEER_CHECK_ARG(M >= 0 && M <= DEER_STATIC_MAX_ROWS, DEER_ERR_UNSUPPORTED,
                   "deer_lmhead_select_static: M = %d exceeds the built-in scratch (at most %d rows); "
                   "use deer_lmhead_select with a caller workspace",
                   M, DEER_STATIC_MAX_ROWS);
    DEER_CHECK_ARG(deer_lmhead_workspace_bytes(DEER_STATIC_MAX_ROWS, hid, V) <= STATIC_SCRATCH_BYTES, DEER_ERR_UNSUPPORTED,
                   "deer_lmhead_select_static: built-in scratch too small for this shape");
    void* scratch = nullptr;
    const int rc = scratch_for_current_device(&scratch, static_cast<cudaStream_t>(stream));
    if (rc != DEER_OK) return rc;
    // Every (vocabulary part, row) slot the merge reads is rewritten by this call's own blocks, and the arrival
    // words are put back to zero by the block that arrives last, so nothing has to be cleared between calls.
    return deer_lmhead_select(h, w, M, hid, V, mode, temperature, draft_ids, out_ids, out_max_logprob, out_lse, out_draft_logit,
                              out_logits, scratch, STATIC_SCRATCH_BYTES, stream);
}
