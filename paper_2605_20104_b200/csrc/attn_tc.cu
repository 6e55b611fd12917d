// Tree-masked GQA attention, tcgen05/TMEM kernel (placeholder until the kernel lands).
#include "graft_internal.cuh"

int graft_attn_tc_init() { return GRAFT_OK; }
bool graft_attn_tc_supported(const graft_ctx*, const graft_attn_params*) { return false; }
size_t graft_attn_tc_ws_bytes(int, int, int, int, int, int) { return 0; }
int graft_attn_tc_launch(graft_ctx*, const graft_attn_params*, cudaStream_t) { return GRAFT_ERR_UNSUPPORTED; }
