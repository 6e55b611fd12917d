// Internal declarations shared by the library's translation units (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "graft.h"

struct graft_ctx {
    int device;
    int num_sms;
    void* ws;           // caller-owned device workspace
    size_t ws_bytes;
    unsigned* status;   // device status word = first word of the workspace
};

// the first GRAFT_WS_HEADER bytes of the workspace are reserved (status word)
#define GRAFT_WS_HEADER 256

#define GRAFT_CHECK_CUDA(expr)                          \
    do {                                                \
        cudaError_t e_ = (expr);                        \
        if (e_ != cudaSuccess) return GRAFT_ERR_CUDA;   \
    } while (0)

static inline bool graft_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Every kernel of the library is launched as a programmatic dependent of the kernel before it in the stream: its CTAs
// may be set up while that kernel still runs, and they wait (graft_wait_for_stream, the first statement of every
// kernel) until it has completed and its writes are visible, so stream order holds for every input whatever kernel
// produced it.  What is saved is the launch gap between the small kernels of a step.
#ifdef __CUDACC__
template <typename... KArgs, typename... Args>
static inline cudaError_t graft_launch(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
// first statement of a kernel: wait for the kernel before it in the stream, then let the one after it be set up
__device__ __forceinline__ void graft_wait_for_stream() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
#endif

// attention launchers (one per kernel family); both return GRAFT_OK or an error code
int graft_attn_mma_init();   // per device, called by graft_create with the device current
int graft_attn_tc_init();
int graft_attn_mma_launch(graft_ctx* ctx, const graft_attn_params* p, cudaStream_t stream);
// which: 0 = two row blocks per CTA, 1 = CTA pairs with two-SM MMAs, 2 = one row block per CTA (partners share tiles
// through L2), -1 = choose
int graft_attn_tc_launch(graft_ctx* ctx, const graft_attn_params* p, cudaStream_t stream, int which = -1);
bool graft_attn_tc_pair_supported(const graft_ctx* ctx, const graft_attn_params* p);
bool graft_attn_tc_supported(const graft_ctx* ctx, const graft_attn_params* p);
size_t graft_attn_mma_ws_bytes(int num_sms, int B, int Hq, int Hkv, int d, int T_max);
size_t graft_attn_tc_ws_bytes(int num_sms, int B, int Hq, int Hkv, int d, int T_max);
