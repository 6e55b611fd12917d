// graft_retrieve_envelope and graft_path_indices: the two small index kernels around tree assembly.
//
// Envelope (retrieval section, "Lightweight parallel retrieval"): one CTA per request fills a static
// template from the request's root token, level by level: nodes of one depth are independent gathers
// from the adjacency matrix, so the critical path is the template's depth (9 for the full template),
// not its size.  It reads nothing the draft model writes, so it runs on a side stream beside drafting.
//
// Path indices (verification section, "candidate-path indices"): one 64-thread CTA per request; thread i
// owns node i, finds out whether it is a leaf, ranks the leaves by node index and writes its row from
// its ancestor mask (ancestors in increasing index = root to leaf, because parent[i] < i).
#include <limits.h>
#include "graft_internal.cuh"

namespace {

constexpr int kEnvThreads = 128;
constexpr int kEnvMax = 1024;       // template nodes held in shared memory

__global__ void __launch_bounds__(kEnvThreads) envelope_kernel(graft_envelope_params a, unsigned* status) {
    __shared__ int s_tok[kEnvMax];
    __shared__ short s_par[kEnvMax];
    __shared__ short s_depth[kEnvMax];
    __shared__ unsigned char s_rank[kEnvMax];
    __shared__ int s_maxd;
    const int b = blockIdx.x;
    unsigned flags = 0;
    int x_root = a.root_token[(size_t)b * a.root_stride];
    if (x_root < -1 || x_root >= a.V) { x_root = -1; if (threadIdx.x == 0) flags |= GRAFT_FLAG_BAD_TOKEN; }
    if (threadIdx.x == 0) s_maxd = 0;
    for (int u = threadIdx.x; u < a.N_env; u += kEnvThreads) {
        int f = a.env_parent[u], r = a.env_rank[u];
        if (f < -1 || f >= u || r < 0 || r >= a.k) { f = -2; r = 0; flags |= GRAFT_FLAG_BAD_TEMPLATE; }
        s_par[u] = (short)f;
        s_rank[u] = (unsigned char)r;
        s_tok[u] = -1;
    }
    __syncthreads();
    // depth of every node: walk to the root (a node with a bad description is its own dead end)
    for (int u = threadIdx.x; u < a.N_env; u += kEnvThreads) {
        int d = 0;
        if (s_par[u] != -2) {
            d = 1;
            for (int j = s_par[u]; j >= 0 && d < kEnvMax; j = s_par[j]) {
                if (s_par[j] == -2) break;
                ++d;
            }
            atomicMax(&s_maxd, d);
        }
        s_depth[u] = (short)d;
    }
    __syncthreads();
    const int max_d = s_maxd;
    for (int lvl = 1; lvl <= max_d; ++lvl) {
        for (int u = threadIdx.x; u < a.N_env; u += kEnvThreads) {
            if (s_depth[u] != lvl) continue;
            const int f = s_par[u];
            const int x_f = f < 0 ? x_root : s_tok[f];
            int x = -1;
            if (x_f >= 0) {
                x = a.M[(size_t)x_f * a.k + s_rank[u]];
                if (x < -1 || x >= a.V) { x = -1; flags |= GRAFT_FLAG_BAD_TOKEN; }
            }
            s_tok[u] = x;
        }
        __syncthreads();
    }
    for (int u = threadIdx.x; u < a.N_env; u += kEnvThreads)
        a.env_token[(size_t)b * a.N_env + u] = s_depth[u] ? s_tok[u] : -1;
    if (flags) atomicOr(status, flags);
}

__global__ void __launch_bounds__(64) paths_kernel(graft_paths_params a, unsigned* status) {
    __shared__ int s_par[64];
    __shared__ unsigned long long s_has_child;
    __shared__ unsigned s_leaf[2];
    const int b = blockIdx.x, i = threadIdx.x;
    unsigned flags = 0;
    int T = a.tree_size[b];
    if (T < 0 || T > a.T_max) { T = 0; if (i == 0) flags |= GRAFT_FLAG_BAD_SIZE; }
    int32_t* rows = a.path_index + (size_t)b * a.T_max * a.D_max;
    for (int e = i; e < a.T_max * a.D_max; e += 64) rows[e] = -1;
    if (i == 0) s_has_child = 0ull;
    int par = -1;
    if (i < T) {
        par = a.tree_parent[(size_t)b * a.T_max + i];
        if (i == 0 || par < 0 || par >= i) par = i == 0 ? -1 : 0;     // malformed: hang it off the root (assembly never writes this)
    }
    s_par[i] = par;
    __syncthreads();
    if (i < T && par >= 0) atomicOr(&s_has_child, 1ull << par);
    __syncthreads();
    const bool leaf = i < T && !((s_has_child >> i) & 1ull);
    const unsigned w = __ballot_sync(0xffffffffu, leaf);
    if ((i & 31) == 0) s_leaf[i >> 5] = w;
    __syncthreads();                   // also: the -1 fill above is ordered before the rows written below (same CTA)
    const unsigned long long leaves = (unsigned long long)s_leaf[0] | ((unsigned long long)s_leaf[1] << 32);
    if (leaf) {
        const int row = __popcll(leaves & ((1ull << i) - 1ull));
        unsigned long long anc = 0;
        for (int j = i; j >= 0; j = s_par[j]) anc |= 1ull << j;
        if (__popcll(anc) > a.D_max) flags |= GRAFT_FLAG_BAD_SIZE;
        int c = 0;
        for (unsigned long long m = anc; m && c < a.D_max; m &= m - 1, ++c) rows[(size_t)row * a.D_max + c] = __ffsll((long long)m) - 1;
    }
    if (i == 0) a.n_paths[b] = __popcll(leaves);
    if (flags) atomicOr(status, flags);
}

}  // namespace

extern "C" int graft_retrieve_envelope(graft_ctx* ctx, const graft_envelope_params* p, void* stream) {
    if (!ctx || !p) return GRAFT_ERR_INVALID_ARG;
    if (p->B <= 0 || p->V <= 0 || p->k <= 0 || p->N_env <= 0 || p->root_stride < 0) return GRAFT_ERR_INVALID_ARG;
    if (p->N_env > kEnvMax || p->k > 16) return GRAFT_ERR_UNSUPPORTED;
    if (!p->root_token || !p->M || !p->env_parent || !p->env_rank || !p->env_token) return GRAFT_ERR_INVALID_ARG;
    envelope_kernel<<<p->B, kEnvThreads, 0, (cudaStream_t)stream>>>(*p, ctx->status);
    GRAFT_CHECK_CUDA(cudaGetLastError());
    return GRAFT_OK;
}

extern "C" int graft_path_indices(graft_ctx* ctx, const graft_paths_params* p, void* stream) {
    if (!ctx || !p) return GRAFT_ERR_INVALID_ARG;
    if (p->B <= 0 || p->T_max <= 0 || p->D_max <= 0) return GRAFT_ERR_INVALID_ARG;
    if (p->T_max > 64 || p->D_max > 64) return GRAFT_ERR_UNSUPPORTED;
    if (!p->tree_parent || !p->tree_size || !p->path_index || !p->n_paths) return GRAFT_ERR_INVALID_ARG;
    paths_kernel<<<p->B, 64, 0, (cudaStream_t)stream>>>(*p, ctx->status);
    GRAFT_CHECK_CUDA(cudaGetLastError());
    return GRAFT_OK;
}
