// graft_accept: greedy lossless acceptance, one warp per sequence.
//
// Lane l owns nodes l and l + 32.  Two ballots give the 64-bit match mask; a node is accepted when
// its ancestor-or-self mask has no unmatched bit; a warp max over (depth, -index) picks the winner;
// the path is read off the winner's ancestor mask (bit rank = position on the path).
#include "graft_internal.cuh"

namespace {

__global__ void __launch_bounds__(128) accept_kernel(graft_accept_params a, unsigned* status) {
    graft_wait_for_stream();
    const int lane = threadIdx.x & 31;
    const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (b >= a.B) return;
    const size_t row = (size_t)b * a.T_max;
    const int T = a.tree_size[b];
    int32_t* path = a.path + row;
    if (T < 1 || T > a.T_max) {
        for (int j = lane; j < a.T_max; j += 32) path[j] = -1;
        if (lane == 0) { a.n_acc[b] = 0; a.best_node[b] = -1; a.bonus[b] = -1; atomicOr(status, (unsigned)GRAFT_FLAG_BAD_SIZE); }
        return;
    }
    unsigned long long anc[2];
    bool match[2];
#pragma unroll
    for (int s = 0; s < 2; ++s) {
        const int i = lane + 32 * s;
        anc[s] = 0;
        match[s] = false;
        if (i < T) {
            anc[s] = a.tree_anc[row + i];
            if (i == 0) match[s] = true;
            else {
                const int tok = a.tree_token[row + i], p = a.tree_parent[row + i];
                if (p >= 0 && p < i) match[s] = tok >= 0 && tok == a.target_next[row + p];
            }
        }
    }
    const unsigned long long matched =
        (unsigned long long)__ballot_sync(0xffffffffu, match[0]) | ((unsigned long long)__ballot_sync(0xffffffffu, match[1]) << 32);
    int key = -1;    // depth * 64 + (63 - index): larger is better
#pragma unroll
    for (int s = 0; s < 2; ++s) {
        const int i = lane + 32 * s;
        if (i < T && anc[s] != 0 && (anc[s] & ~matched) == 0) key = max(key, (__popcll(anc[s]) - 1) * 64 + (63 - i));
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) key = max(key, __shfl_xor_sync(0xffffffffu, key, o));
    // the root always qualifies when its mask is sane; otherwise fall back to the root alone
    const int best = key < 0 ? 0 : 63 - (key & 63);
    const int owner = best & 31;
    unsigned long long banc = __shfl_sync(0xffffffffu, best < 32 ? anc[0] : anc[1], owner);
    if (key < 0) banc = 1ull;
    const int n = __popcll(banc);
    for (int j = lane; j < a.T_max; j += 32)
        if (j >= n) path[j] = -1;
    __syncwarp();
#pragma unroll
    for (int s = 0; s < 2; ++s) {
        const int i = lane + 32 * s;
        if ((banc >> i) & 1ull) path[__popcll(banc & ((1ull << i) - 1ull))] = i;
    }
    if (lane == 0) {
        a.n_acc[b] = n;
        a.best_node[b] = best;
        a.bonus[b] = a.target_next[row + best];
    }
}

}  // namespace

extern "C" int graft_accept(graft_ctx* ctx, const graft_accept_params* p, void* stream) {
    if (!ctx || !p) return GRAFT_ERR_INVALID_ARG;
    if (p->B <= 0 || p->T_max <= 0) return GRAFT_ERR_INVALID_ARG;
    if (p->T_max > 64) return GRAFT_ERR_UNSUPPORTED;
    if (!p->tree_token || !p->tree_parent || !p->tree_anc || !p->tree_size || !p->target_next || !p->n_acc ||
        !p->path || !p->best_node || !p->bonus)
        return GRAFT_ERR_INVALID_ARG;
    const int warps = 4;
    GRAFT_CHECK_CUDA(graft_launch(accept_kernel, dim3((p->B + warps - 1) / warps), dim3(warps * 32), 0, (cudaStream_t)stream, *p, ctx->status));
    return GRAFT_OK;
}
