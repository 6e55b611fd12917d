// Context management, argument checks and kernel dispatch of the C ABI.
#include <stdlib.h>
#include "graft_internal.cuh"

extern "C" size_t graft_workspace_bytes(int device, int B, int Hq, int Hkv, int d, int T_max) {
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || (d != 64 && d != 128) || T_max <= 0 || T_max > 64) return 0;
    int num_sms = 0;
    if (cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || num_sms <= 0) return 0;
    size_t a = graft_attn_mma_ws_bytes(num_sms, B, Hq, Hkv, d, T_max);
    size_t b = graft_attn_tc_ws_bytes(num_sms, B, Hq, Hkv, d, T_max);
    return GRAFT_WS_HEADER + (a > b ? a : b);
}

extern "C" int graft_create(graft_ctx** out, int device, void* workspace, size_t workspace_bytes) {
    if (!out || !workspace || workspace_bytes < GRAFT_WS_HEADER) return GRAFT_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return GRAFT_ERR_INVALID_ARG;
    int prev = 0;
    GRAFT_CHECK_CUDA(cudaGetDevice(&prev));
    GRAFT_CHECK_CUDA(cudaSetDevice(device));
    int major = 0, num_sms = 0;
    GRAFT_CHECK_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device));
    GRAFT_CHECK_CUDA(cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, device));
    if (major != 10) { cudaSetDevice(prev); return GRAFT_ERR_UNSUPPORTED; }   // sm_100a code only
    int rc = graft_attn_mma_init();
    if (rc == GRAFT_OK) rc = graft_attn_tc_init();
    // the whole workspace starts at zero: status word, and the arrival counters of the attention kernels' merge
    if (rc == GRAFT_OK && cudaMemset(workspace, 0, workspace_bytes) != cudaSuccess) rc = GRAFT_ERR_CUDA;
    if (rc == GRAFT_OK && cudaDeviceSynchronize() != cudaSuccess) rc = GRAFT_ERR_CUDA;
    cudaSetDevice(prev);
    if (rc != GRAFT_OK) return rc;
    graft_ctx* c = static_cast<graft_ctx*>(malloc(sizeof(graft_ctx)));
    if (!c) return GRAFT_ERR_INVALID_ARG;
    c->device = device;
    c->num_sms = num_sms;
    c->ws = workspace;
    c->ws_bytes = workspace_bytes;
    c->status = static_cast<unsigned*>(workspace);
    *out = c;
    return GRAFT_OK;
}

extern "C" int graft_destroy(graft_ctx* ctx) {
    if (!ctx) return GRAFT_ERR_INVALID_ARG;
    free(ctx);
    return GRAFT_OK;
}

extern "C" const char* graft_status_string(int status) {
    switch (status) {
        case GRAFT_OK: return "ok";
        case GRAFT_ERR_INVALID_ARG: return "invalid argument";
        case GRAFT_ERR_UNSUPPORTED: return "unsupported shape or device";
        case GRAFT_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case GRAFT_ERR_CUDA: return "CUDA error";
        case GRAFT_ERR_SCRATCH_LIMIT: return "shape needs more scratch than the built-in array of graft_tree_verify_attn_noalloc";
        default: return "unknown status";
    }
}

extern "C" int graft_device_status(graft_ctx* ctx, void* stream, unsigned* flags_out, int clear) {
    if (!ctx || !flags_out) return GRAFT_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    GRAFT_CHECK_CUDA(cudaMemcpyAsync(flags_out, ctx->status, sizeof(unsigned), cudaMemcpyDeviceToHost, s));
    if (clear) GRAFT_CHECK_CUDA(cudaMemsetAsync(ctx->status, 0, sizeof(unsigned), s));
    GRAFT_CHECK_CUDA(cudaStreamSynchronize(s));
    return GRAFT_OK;
}

extern "C" int graft_tree_verify_attn(graft_ctx* ctx, const graft_attn_params* p, void* stream) {
    if (!ctx || !p) return GRAFT_ERR_INVALID_ARG;
    if (p->B <= 0 || p->T_max <= 0 || p->Hq <= 0 || p->Hkv <= 0 || p->S_cap <= 0) return GRAFT_ERR_INVALID_ARG;
    if (p->T_max > 64 || (p->d != 64 && p->d != 128) || p->Hq % p->Hkv != 0) return GRAFT_ERR_UNSUPPORTED;
    if (!(p->scale > 0.f) || !(p->scale < 1e30f)) return GRAFT_ERR_INVALID_ARG;
    if (!p->Q || !p->Kc || !p->Vc || !p->O || !p->seq_len || !p->tree_size || !p->tree_anc) return GRAFT_ERR_INVALID_ARG;
    if (!graft_aligned16(p->Q) || !graft_aligned16(p->Kc) || !graft_aligned16(p->Vc) || !graft_aligned16(p->O))
        return GRAFT_ERR_INVALID_ARG;
    const int64_t strides[] = {p->q_stride_b, p->q_stride_t, p->q_stride_h, p->kv_stride_b, p->kv_stride_h,
                               p->kv_stride_s, p->o_stride_b, p->o_stride_t, p->o_stride_h};
    for (int64_t s : strides)
        if (s < 0 || s % 8 != 0) return GRAFT_ERR_INVALID_ARG;
    if (p->kv_stride_s < p->d || p->q_stride_h < p->d || p->o_stride_h < p->d) return GRAFT_ERR_INVALID_ARG;
    if (p->block_table) {
        if (p->page_size <= 0 || p->page_size % 128 != 0 || p->blocks_per_seq <= 0 || p->n_blocks <= 0) return GRAFT_ERR_INVALID_ARG;
        if ((long long)p->blocks_per_seq * p->page_size < p->S_cap) return GRAFT_ERR_INVALID_ARG;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    switch (p->variant) {
        case GRAFT_ATTN_MMA_SYNC: return graft_attn_mma_launch(ctx, p, s);
        case GRAFT_ATTN_TCGEN05:
            if (!graft_attn_tc_supported(ctx, p)) return GRAFT_ERR_UNSUPPORTED;
            return graft_attn_tc_launch(ctx, p, s);
        case GRAFT_ATTN_TCGEN05_1SM:
            if (!graft_attn_tc_supported(ctx, p) || p->block_table) return GRAFT_ERR_UNSUPPORTED;     // this kernel takes contiguous caches only
            return graft_attn_tc_launch(ctx, p, s, 0);
        case GRAFT_ATTN_TCGEN05_2SM:
            if (!graft_attn_tc_pair_supported(ctx, p)) return GRAFT_ERR_UNSUPPORTED;
            return graft_attn_tc_launch(ctx, p, s, 1);
        case GRAFT_ATTN_TCGEN05_L2PAIR:
            if (!graft_attn_tc_supported(ctx, p)) return GRAFT_ERR_UNSUPPORTED;
            return graft_attn_tc_launch(ctx, p, s, 2);
        case GRAFT_ATTN_AUTO:
            if (graft_attn_tc_supported(ctx, p)) return graft_attn_tc_launch(ctx, p, s);
            return graft_attn_mma_launch(ctx, p, s);
        default: return GRAFT_ERR_INVALID_ARG;
    }
}
