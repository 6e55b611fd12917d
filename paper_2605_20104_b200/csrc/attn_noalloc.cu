// graft_tree_verify_attn_noalloc: the tree attention call for callers that must not allocate.
//
// The regular call keeps its split-KV partials and its status word in a workspace that the caller
// allocates and hands to graft_create.  Some callers cannot do that: code that runs after a serving
// process has handed all of its device memory to a fixed pool, plug-ins that are forbidden to touch
// the allocator because cudaMalloc may synchronise the whole device in the middle of a latency
// critical section, or a host that simply has no allocation API in reach (a thin C shim, a sandbox).
// For them this file carries its own scratch: one file-scope __device__ array of kScratchBytes that
// every GPU holding this library keeps resident until the process exits.  Nothing here calls
// cudaMalloc, cudaFree or any allocating library routine.
//
// The array's name is only a host-side handle; the device address is fetched once per device with
// cudaGetSymbolAddress (with that device current) and passed to the kernels like any workspace.
#include <mutex>
#include "graft_internal.cuh"

namespace {

constexpr size_t kScratchBytes = 40ull << 20;          // 40 MiB per GPU, fixed at build time
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
struct DeviceSetup {
    bool ready = false;
    void* scratch = nullptr;       // device address of g_noalloc_scratch on this device
    int num_sms = 0;
};
DeviceSetup g_setup[kMaxDevices];
std::mutex g_setup_mutex;

// Once per device, with that device current: resolve the scratch address, check the architecture and
// opt the attention kernels in to their shared-memory sizes.
int setup_device(int device, DeviceSetup** out) {
    if (device < 0 || device >= kMaxDevices) return GRAFT_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    DeviceSetup& s = g_setup[device];
    if (!s.ready) {
        int major = 0, num_sms = 0;
        GRAFT_CHECK_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device));
        GRAFT_CHECK_CUDA(cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, device));
        if (major != 10) return GRAFT_ERR_UNSUPPORTED;
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || ptr == nullptr) return GRAFT_ERR_CUDA;
        int rc = graft_attn_mma_init();
        if (rc == GRAFT_OK) rc = graft_attn_tc_init();
        if (rc != GRAFT_OK) return rc;
        s.scratch = ptr;
        s.num_sms = num_sms;
        s.ready = true;
    }
    *out = &s;
    return GRAFT_OK;
}

}  // namespace

extern "C" size_t graft_noalloc_scratch_bytes(void) { return kScratchBytes; }

extern "C" int graft_tree_verify_attn_noalloc(const graft_attn_params* p, void* stream, unsigned* device_flags_out) {
    if (!p) return GRAFT_ERR_INVALID_ARG;
    int device = 0;
    GRAFT_CHECK_CUDA(cudaGetDevice(&device));
    DeviceSetup* s = nullptr;
    int rc = setup_device(device, &s);
    if (rc != GRAFT_OK) return rc;

    // the shape must fit the built-in array with at least one kernel the caller allows
    if (p->B <= 0 || p->Hq <= 0 || p->Hkv <= 0 || p->T_max <= 0) return GRAFT_ERR_INVALID_ARG;
    if (p->Hq % p->Hkv != 0 || (p->d != 64 && p->d != 128) || p->T_max > 64) return GRAFT_ERR_UNSUPPORTED;
    const size_t need_mma = GRAFT_WS_HEADER + graft_attn_mma_ws_bytes(s->num_sms, p->B, p->Hq, p->Hkv, p->d, p->T_max);
    const size_t tc_bytes = graft_attn_tc_ws_bytes(s->num_sms, p->B, p->Hq, p->Hkv, p->d, p->T_max);   // 0: shape not supported
    const size_t need_tc = GRAFT_WS_HEADER + tc_bytes;
    const bool mma_fits = need_mma <= kScratchBytes, tc_fits = tc_bytes != 0 && need_tc <= kScratchBytes;
    if ((p->variant == GRAFT_ATTN_MMA_SYNC && !mma_fits) || (p->variant == GRAFT_ATTN_TCGEN05 && tc_bytes != 0 && !tc_fits) ||
        (p->variant == GRAFT_ATTN_AUTO && !mma_fits && !tc_fits))
        return GRAFT_ERR_SCRATCH_LIMIT;

    // a context on the stack, bound to the static scratch: the regular dispatch runs unchanged on it
    graft_ctx ctx;
    ctx.device = device;
    ctx.num_sms = s->num_sms;
    ctx.ws = s->scratch;
    ctx.ws_bytes = kScratchBytes;
    ctx.status = static_cast<unsigned*>(s->scratch);

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the array keeps the previous call's contents (among them the number of the last call, in the header);
    // only the status word has to start at zero (partials are always written before they are read)
    GRAFT_CHECK_CUDA(cudaMemsetAsync(ctx.status, 0, 16, st));
    rc = graft_tree_verify_attn(&ctx, p, stream);
    if (rc == GRAFT_ERR_WORKSPACE_TOO_SMALL) return GRAFT_ERR_SCRATCH_LIMIT;
    if (rc != GRAFT_OK) return rc;
    if (device_flags_out)
        GRAFT_CHECK_CUDA(cudaMemcpyAsync(device_flags_out, ctx.status, sizeof(unsigned), cudaMemcpyDeviceToDevice, st));
    return GRAFT_OK;
}
