// graft_build_tree: prune + graft + rebuild, one 64-thread CTA per sequence.
//
// Thread i owns draft node i, then template node i, then output node i.  Everything a node needs
// from other nodes goes through shared memory; the only global traffic is one read of the draft
// arrays, the level-wise gathers from the adjacency matrix (one dependent gather per template
// depth: the critical path the paper attributes to retrieval; with a precomputed envelope a single
// gather), and one write of the outputs.
#include <limits.h>
#include <math_constants.h>
#include "graft_internal.cuh"

namespace {

constexpr int kThreads = 64;
constexpr int kTmplCache = 128;     // template nodes and checkpoints kept in shared memory (larger inputs are read in place)
constexpr int kCkptCache = 8;

__device__ __forceinline__ bool better(float sa, int a, float sb, int b) {
    // order of "keep the top K draft nodes by cumulative path score": score desc, index asc
    return sa > sb || (sa == sb && a < b);
}

// block-wide (2 warps) max of a float / of an int, result visible to all threads
__device__ __forceinline__ float block_max(float v, float* s2) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) s2[threadIdx.x >> 5] = v;
    __syncthreads();
    return fmaxf(s2[0], s2[1]);
}
__device__ __forceinline__ int block_max_int(int v, int* s2) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, o));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) s2[threadIdx.x >> 5] = v;
    __syncthreads();
    return max(s2[0], s2[1]);
}
// 64-bit mask of a predicate over the 64 threads
__device__ __forceinline__ unsigned long long block_ballot(bool pred, unsigned* s2) {
    unsigned w = __ballot_sync(0xffffffffu, pred);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) s2[threadIdx.x >> 5] = w;
    __syncthreads();
    return (unsigned long long)s2[0] | ((unsigned long long)s2[1] << 32);
}

__global__ void __launch_bounds__(kThreads) build_tree_kernel(graft_build_params a, unsigned* status) {
    graft_wait_for_stream();
    const int b = blockIdx.x, i = threadIdx.x;
    __shared__ int s_par[64], s_depth[64], s_sel[64], s_new[64];
    __shared__ int s_tok[64], s_opar[64];
    __shared__ float s_score[64];
    __shared__ float s_f2[2];
    __shared__ int s_i2[2];
    __shared__ unsigned s_u2[2];
    __shared__ int s_tp[kTmplCache], s_tr[kTmplCache], s_te[kTmplCache];      // template parents, ranks, envelope indices
    __shared__ int s_cd[kCkptCache], s_ck[kCkptCache], s_to[kCkptCache + 1];  // checkpoint depths, keep counts, template offsets
    __shared__ float s_ct[kCkptCache];                                        // checkpoint thresholds

    int32_t* o_tok = a.tree_token + (size_t)b * a.T_max;
    int32_t* o_par = a.tree_parent + (size_t)b * a.T_max;
    int32_t* o_pos = a.tree_pos + (size_t)b * a.T_max;
    int32_t* o_src = a.tree_src + (size_t)b * a.T_max;
    uint64_t* o_anc = a.tree_anc + (size_t)b * a.T_max;
    unsigned flags = 0;

    // Every input that does not depend on another one is requested here, in one round trip to memory: the kernel is
    // a chain of dependent loads (about 0.7 us each) and little else.
    const int n = a.n_draft[b];
    const int budget = a.k_max ? a.k_max[b] : a.K_max;
    const int L = a.seq_len[b];
    int tok = -1, par = -1;
    float sc = -CUDART_INF_F;
    if (i < a.N_max) {
        tok = a.draft_token[(size_t)b * a.N_max + i];
        par = a.draft_parent[(size_t)b * a.N_max + i];
        sc = a.draft_score[(size_t)b * a.N_max + i];
    }
    const int keep_count = a.mode == GRAFT_PRUNE_TOPK ? a.keep_count[b] : 0;
    const bool tmpl_cached = a.N_tmpl <= kTmplCache, ckpt_cached = a.n_ckpt <= kCkptCache;
    if (a.mode != GRAFT_PRUNE_NONE && tmpl_cached)
        for (int u = i; u < a.N_tmpl; u += kThreads) {
            s_tp[u] = a.tmpl_parent[u];
            s_tr[u] = a.tmpl_rank[u];
            s_te[u] = a.env_token ? a.tmpl_env[u] : 0;
        }
    if (a.mode == GRAFT_PRUNE_GATED && ckpt_cached) {
        if (i < a.n_ckpt) { s_cd[i] = a.ckpt_depth[i]; s_ck[i] = a.ckpt_keep[i]; s_ct[i] = a.ckpt_log_tau[i]; }
        if (i <= a.n_ckpt && a.n_ckpt > 0) s_to[i] = a.tmpl_offset[i];
    }
    if (n < 1 || n > a.N_max || budget < 1 || budget > a.T_max || L < 0 ||
        (long long)L + a.T_max > (long long)a.S_cap) {
        if (i < a.T_max) { o_tok[i] = -1; o_par[i] = -1; o_pos[i] = 0; o_src[i] = INT_MIN; o_anc[i] = 0; }
        if (i == 0) { a.tree_size[b] = 0; atomicOr(status, (unsigned)GRAFT_FLAG_BAD_SIZE); }
        return;
    }

    // ---- 1. load, depth and validity by climbing the parent chain (strictly decreasing indices)
    if (i >= n) { tok = -1; par = -1; sc = -CUDART_INF_F; }
    if (i < n) {
        if (sc != sc) { sc = -CUDART_INF_F; if (i > 0) flags |= GRAFT_FLAG_NAN_SCORE; }
        if (i > 0 && (par < 0 || par >= i)) flags |= GRAFT_FLAG_BAD_PARENT;
    }
    s_par[i] = par;
    s_score[i] = sc;
    __syncthreads();
    int depth = 0;
    bool valid = i < n;
    if (valid) {
        for (int j = i; j > 0;) {
            int p = s_par[j];
            if (p < 0 || p >= j) { valid = false; depth = 0; break; }
            j = p;
            ++depth;
        }
    }
    s_depth[i] = valid ? depth : -1;
    __syncthreads();

    // ---- 2. keep-set
    bool sel = valid;
    bool graft = true;
    int t_lo = 0, t_hi = a.N_tmpl;
    if (a.mode == GRAFT_PRUNE_NONE) {
        graft = false;
    } else if (a.mode == GRAFT_PRUNE_TOPK || a.mode == GRAFT_PRUNE_GATED) {
        int K_draft = n, max_depth = INT_MAX;
        if (a.mode == GRAFT_PRUNE_TOPK) {
            K_draft = keep_count;
        } else {
            int stage = -1;
            for (int c = 0; c < a.n_ckpt && stage < 0; ++c) {
                const int D = ckpt_cached ? s_cd[c] : a.ckpt_depth[c];
                float smax = block_max((valid && i > 0 && depth == D) ? sc : -CUDART_INF_F, s_f2);
                if (smax <= (ckpt_cached ? s_ct[c] : a.ckpt_log_tau[c])) stage = c;     // c_d <= tau_d: gate closed, prune here
            }
            if (stage < 0) graft = false;
            else {
                K_draft = ckpt_cached ? s_ck[stage] : a.ckpt_keep[stage];
                max_depth = ckpt_cached ? s_cd[stage] : a.ckpt_depth[stage];
                t_lo = ckpt_cached ? s_to[stage] : a.tmpl_offset[stage];
                t_hi = ckpt_cached ? s_to[stage + 1] : a.tmpl_offset[stage + 1];
            }
        }
        if (graft) {
            const bool elig = valid && i > 0 && depth <= max_depth;
            int rank = 0;
            for (int j = 1; j < n; ++j) {
                const int dj = s_depth[j];
                if (dj >= 0 && dj <= max_depth && j != i && better(s_score[j], j, sc, i)) ++rank;
            }
            sel = (i == 0) || (elig && rank < K_draft - 1);
        }
    } else {  // GRAFT_PRUNE_NODE
        s_sel[i] = valid && i > 0 && depth >= a.gate_depth && sc < a.node_threshold;   // "low" marks
        __syncthreads();
        if (valid)
            for (int j = i; j > 0; j = s_par[j])
                if (s_sel[j]) { sel = false; break; }
        __syncthreads();
    }
    s_sel[i] = sel;
    __syncthreads();

    // ---- 3. stable compaction: a selected node stays if all its ancestors are selected
    bool closed = sel;
    if (sel)
        for (int j = s_par[i]; i > 0 && j >= 0; j = s_par[j]) {
            if (!s_sel[j]) { closed = false; break; }
            if (j == 0) break;
        }
    const unsigned long long closed_mask = block_ballot(closed, s_u2);
    const int before = __popcll(closed_mask & ((1ull << i) - 1ull));
    const bool kept = closed && before < budget;
    if (sel && !kept) flags |= (before >= budget) ? GRAFT_FLAG_BUDGET : GRAFT_FLAG_ORPHAN;
    const int K_kept = min(budget, __popcll(closed_mask));
    s_new[i] = kept ? before : -1;
    __syncthreads();
    // s_tok / s_opar hold the output tree from here on
    if (kept) {
        if (tok < -1 || tok >= a.V) { tok = -1; flags |= GRAFT_FLAG_BAD_TOKEN; }
        s_tok[before] = tok;
        s_opar[before] = i == 0 ? -1 : s_new[par];
        o_src[before] = i;
    }
    __syncthreads();

    // ---- 4. graft the stage template's first K_ret nodes, one dependent gather per depth
    int T = K_kept;
    if (graft) {
        const int K_ret = max(0, min(t_hi - t_lo, budget - K_kept));
        const bool from_cache = tmpl_cached && t_lo >= 0 && t_hi <= a.N_tmpl;
        const int attach = a.attach_tail && K_kept > 0 ? K_kept - 1 : 0;      // where template nodes without a template parent hang
        T += K_ret;
        const int u = i;
        int tp = -1, r = 0, du = 0;
        bool ok = true;
        if (u < K_ret) {
            tp = from_cache ? s_tp[t_lo + u] : a.tmpl_parent[t_lo + u];
            r = from_cache ? s_tr[t_lo + u] : a.tmpl_rank[t_lo + u];
            if (tp < -1 || tp >= u || r < 0 || r >= a.k) { ok = false; tp = -1; flags |= GRAFT_FLAG_BAD_TEMPLATE; }
        }
        s_par[i] = tp;                       // template-local parents (draft parents no longer needed)
        __syncthreads();
        if (u < K_ret) {
            du = 1;
            for (int j = tp; j >= 0; j = s_par[j]) {
                ++du;
                if (j >= u) { break; }       // cannot happen after the check above; bounds the loop
            }
            s_opar[K_kept + u] = tp < 0 ? attach : K_kept + tp;
            o_src[K_kept + u] = -1 - u;
        }
        if (a.env_token) {
            // the envelope holds the token of every rank path already: one independent load per node
            if (u < K_ret) {
                int x = -1;
                const int e = from_cache ? s_te[t_lo + u] : a.tmpl_env[t_lo + u];
                if (e < 0 || e >= a.N_env) flags |= GRAFT_FLAG_BAD_TEMPLATE;
                else if (ok) {
                    x = a.env_token[(size_t)b * a.N_env + e];
                    if (x < -1 || x >= a.V) { x = -1; flags |= GRAFT_FLAG_BAD_TOKEN; }
                }
                s_tok[K_kept + u] = x;
            }
        }
        const int max_d = a.env_token ? 0 : block_max_int(u < K_ret ? du : 0, s_i2);
        for (int lvl = 1; lvl <= max_d; ++lvl) {
            if (u < K_ret && du == lvl) {
                int x = -1;
                const int ptok = s_tok[tp < 0 ? attach : K_kept + tp];
                if (ok && ptok >= 0) {
                    x = a.M[(size_t)ptok * a.k + r];
                    if (x < -1 || x >= a.V) { x = -1; flags |= GRAFT_FLAG_BAD_TOKEN; }
                }
                s_tok[K_kept + u] = x;
            }
            __syncthreads();
        }
    }
    __syncthreads();

    // ---- 5. ancestor-or-self mask, position ids, padding
    if (i < a.T_max) {
        if (i < T) {
            unsigned long long anc = 0;
            for (int j = i; j >= 0; j = s_opar[j]) anc |= 1ull << j;
            o_tok[i] = s_tok[i];
            o_par[i] = s_opar[i];
            o_anc[i] = anc;
            o_pos[i] = L + __popcll(anc) - 1;
        } else {
            o_tok[i] = -1; o_par[i] = -1; o_pos[i] = 0; o_src[i] = INT_MIN; o_anc[i] = 0;
        }
    }
    if (i == 0) a.tree_size[b] = T;
    if (flags) atomicOr(status, flags);
}

}  // namespace

extern "C" int graft_build_tree(graft_ctx* ctx, const graft_build_params* p, void* stream) {
    if (!ctx || !p) return GRAFT_ERR_INVALID_ARG;
    if (p->B <= 0 || p->N_max <= 0 || p->T_max <= 0 || p->K_max <= 0 || p->V <= 0 || p->k <= 0 || p->S_cap <= 0)
        return GRAFT_ERR_INVALID_ARG;
    if (p->T_max > 64 || p->N_max > 64 || p->k > 16 || p->K_max > p->T_max) return GRAFT_ERR_UNSUPPORTED;
    if (p->mode < GRAFT_PRUNE_NONE || p->mode > GRAFT_PRUNE_NODE) return GRAFT_ERR_INVALID_ARG;
    if (!p->draft_token || !p->draft_parent || !p->draft_score || !p->n_draft || !p->seq_len) return GRAFT_ERR_INVALID_ARG;
    if (!p->tree_token || !p->tree_parent || !p->tree_pos || !p->tree_src || !p->tree_anc || !p->tree_size)
        return GRAFT_ERR_INVALID_ARG;
    if (p->N_tmpl < 0 || p->n_ckpt < 0) return GRAFT_ERR_INVALID_ARG;
    if (p->mode != GRAFT_PRUNE_NONE && p->N_tmpl > 0 && (!p->M || !p->tmpl_parent || !p->tmpl_rank)) return GRAFT_ERR_INVALID_ARG;
    if (p->env_token && (!p->tmpl_env || p->N_env <= 0 || p->attach_tail)) return GRAFT_ERR_INVALID_ARG;
    if (p->mode == GRAFT_PRUNE_TOPK && !p->keep_count) return GRAFT_ERR_INVALID_ARG;
    if (p->mode == GRAFT_PRUNE_GATED &&
        (p->n_ckpt > 0 && (!p->ckpt_depth || !p->ckpt_keep || !p->ckpt_log_tau || !p->tmpl_offset)))
        return GRAFT_ERR_INVALID_ARG;
    GRAFT_CHECK_CUDA(graft_launch(build_tree_kernel, dim3(p->B), dim3(kThreads), 0, (cudaStream_t)stream, *p, ctx->status));
    return GRAFT_OK;
}
