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
    // every input is requested at once (the arrays are [B, T_max] whatever the tree's size): the kernel is one round
    // trip to memory, a few ballots and shuffles, and the stores
    const int T = a.tree_size[b];
    unsigned long long anc_in[2];
    int tok_in[2], par_in[2], next_in[2];
#pragma unroll
    for (int s = 0; s < 2; ++s) {
        const int i = lane + 32 * s;
        anc_in[s] = 0; tok_in[s] = -1; par_in[s] = -1; next_in[s] = -1;
        if (i < a.T_max) {
            anc_in[s] = a.tree_anc[row + i];
            tok_in[s] = a.tree_token[row + i];
            par_in[s] = a.tree_parent[row + i];
            next_in[s] = a.target_next[row + i];
        }
    }
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
        anc[s] = i < T ? anc_in[s] : 0;
        // the target's id at the parent sits in lane parent % 32
        const int tok = tok_in[s], p = par_in[s];
        const int pc = (p >= 0 && p < 64) ? p : 0;
        const int n0 = __shfl_sync(0xffffffffu, next_in[0], pc & 31), n1 = __shfl_sync(0xffffffffu, next_in[1], pc & 31);
        const int next_p = pc < 32 ? n0 : n1;
        match[s] = i < T && (i == 0 || (p >= 0 && p < i && tok >= 0 && tok == next_p));
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
    const int bonus = __shfl_sync(0xffffffffu, best < 32 ? next_in[0] : next_in[1], owner);
    if (lane == 0) {
        a.n_acc[b] = n;
        a.best_node[b] = best;
        a.bonus[b] = bonus;
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
