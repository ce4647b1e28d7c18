// Shared device helpers and host-side plumbing for the DEER hot-path library.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include "deer.h"

struct deer_kv {
    deer_kv_desc d;
};

// ---- host-side error text (per thread) -------------------------------------
void deer_set_error(const char* fmt, ...);

#define DEER_CHECK_ARG(cond, code, ...)        \
    do {                                       \
        if (!(cond)) {                         \
            deer_set_error(__VA_ARGS__);       \
            return (code);                     \
        }                                      \
    } while (0)

#define DEER_CUDA(call)                                                                   \
    do {                                                                                  \
        cudaError_t e_ = (call);                                                          \
        if (e_ != cudaSuccess) {                                                          \
            deer_set_error("%s failed: %s (%s:%d)", #call, cudaGetErrorString(e_), __FILE__, __LINE__); \
            return DEER_ERR_CUDA;                                                         \
        }                                                                                 \
    } while (0)

static inline bool deer_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Streaming multiprocessors of the current device (asked once per device).  Grids and workspaces are sized by it.
// Where no device can be asked (a host without a GPU sizing a workspace) it is a B200's 148.
inline int deer_sm_count() {
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        cudaGetLastError();
        return 148;
    }
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
            cudaGetLastError();
            n = 148;
        }
        cached[dev] = n;
    }
    return cached[dev];
}

// Launches `kernel` so that it may overlap the tail of the kernel before it in the stream (see pdl_wait below).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---- device helpers --------------------------------------------------------
#ifdef __CUDACC__

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// 16-byte async copy global -> shared; src_bytes = 0 zero-fills the destination.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}

// D(16x8, f32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Programmatic dependent launch.  A kernel launched with launch_pdl() may become resident while the kernel before
// it in the stream is still running: its blocks set up what needs no input (barriers, tensor memory, tensor-map
// prefetch) and then sit in pdl_wait() until that kernel has completed and its writes are visible.  pdl_trigger()
// in a running kernel lets the next one be launched from that point on.  Every kernel of the library executes
// pdl_wait() in every thread before its first read of global memory, so the completion of a kernel implies the
// completion of everything before it; both instructions do nothing in a kernel launched the plain way.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Record the first data-dependent error seen by any kernel.
__device__ __forceinline__ void deer_report(int32_t* status, int32_t code) {
    if (status) atomicCAS(status, 0, code);
}

#endif  // __CUDACC__

// ---- calls between the library's own files (not part of the C ABI) ----------------------
int deer_accept_commit_mirrored(deer_kv* kv, const int32_t* seq_ids, int mode, int B, int k, const int32_t* draft_ids,
                                const int32_t* target_ids, int32_t eos_id, int32_t* accept_len, int32_t* out_ids, int32_t* n_out,
                                int32_t* mirror_accept_len, int32_t* mirror_out_ids, int32_t* mirror_n_out, void* stream);

// ---- timing probes (measurement builds only) -----------------------------------------
// `python -m paper_2512_15176_b200.build --probes` compiles the library a second time with DEER_TIMING_PROBES
// defined (libdeer_probes.so): a few kernels then record SM clock values at the hand-overs of their pipelines, for
// `profile_case.py --probes` to read.  Nothing is skipped or reordered; without the define the macros vanish.
#ifdef DEER_TIMING_PROBES
#define DEER_PROBE_ROWS 64
#define DEER_PROBE_COLS 8
#define DEER_PROBE(table, on, row, col)                                                     \
    do {                                                                                    \
        if ((on) && (row) >= 0 && (row) < DEER_PROBE_ROWS) (table)[(row)][(col)] = clock64(); \
    } while (0)
#else
#define DEER_PROBE(table, on, row, col) \
    do {                                \
    } while (0)
#endif
