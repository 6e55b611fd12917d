// graft_accept_stochastic: acceptance under temperature sampling, two kernels.
//
//   softmax_stats_kernel   one CTA per tree node streams that node's V logits once and leaves the row's
//                          (max of logit / temperature, sum of exponentials) pair: which rows the walk
//                          will need is only known while walking, so all valid rows are done at once, in
//                          parallel (HBM-bound: V * 2 bytes per valid node, as the adjacency refresh);
//   accept_walk_kernel     one CTA per request: every thread of the first T computes the probability of
//                          its node's token under the parent's distribution (one gather each), one thread
//                          walks the tree with those (sequential rejection over a node's children), then
//                          the whole CTA draws the bonus token from the last node's remaining distribution:
//                          contiguous chunks per thread, block scan of the chunk sums, and the warp of the
//                          chunk that holds the target splits it once more.
#include <cuda_bf16.h>
#include <math_constants.h>
#include "graft_internal.cuh"

namespace {

constexpr int ST = 512;        // threads of the statistics kernel
constexpr int WT = 256;        // threads of the walk kernel

__device__ __forceinline__ float lo_f(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float hi_f(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// (m, s) <- (m, s) (+) (m2, s2): s counts exponentials relative to m
__device__ __forceinline__ void combine(float& m, float& s, float m2, float s2) {
    const float mn = fmaxf(m, m2);
    if (mn == -CUDART_INF_F) { m = mn; s = 0.f; return; }
    s = s * __expf(m - mn) + s2 * __expf(m2 - mn);
    m = mn;
}

__global__ void __launch_bounds__(ST, 2) softmax_stats_kernel(graft_accept_stochastic_params p, unsigned* status) {
    __shared__ float s_m[ST / 32], s_s[ST / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int r = blockIdx.x, b = r / p.T_max, i = r % p.T_max;
    int T = p.tree_size[b];
    if (T < 0 || T > p.T_max) T = 0;
    if (i >= T) return;
    const float inv_t = 1.f / p.temperature;
    const __nv_bfloat16* row = reinterpret_cast<const __nv_bfloat16*>(p.logits) + (size_t)r * p.logits_stride_row;
    const int nvec = p.V >> 3;
    float m = -CUDART_INF_F, s = 0.f;
    for (int j = tid; j < nvec; j += ST) {
        const uint4 q = __ldcs(reinterpret_cast<const uint4*>(row) + j);
        float z[8] = {lo_f(q.x) * inv_t, hi_f(q.x) * inv_t, lo_f(q.y) * inv_t, hi_f(q.y) * inv_t,
                      lo_f(q.z) * inv_t, hi_f(q.z) * inv_t, lo_f(q.w) * inv_t, hi_f(q.w) * inv_t};
        float vm = z[0];
#pragma unroll
        for (int e = 1; e < 8; ++e) vm = fmaxf(vm, z[e]);
        const float mn = fmaxf(m, vm);
        if (mn > -CUDART_INF_F) {
            float add = 0.f;
#pragma unroll
            for (int e = 0; e < 8; ++e) add += __expf(z[e] - mn);
            s = s * __expf(m - mn) + add;
            m = mn;
        }
    }
    for (int v = (nvec << 3) + tid; v < p.V; v += ST) combine(m, s, __bfloat162float(row[v]) * inv_t, 1.f);
#pragma unroll
    for (int o = 16; o; o >>= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, m, o), s2 = __shfl_xor_sync(0xffffffffu, s, o);
        combine(m, s, m2, s2);
    }
    if (lane == 0) { s_m[warp] = m; s_s[warp] = s; }
    __syncthreads();
    if (warp == 0) {
        m = lane < ST / 32 ? s_m[lane] : -CUDART_INF_F;
        s = lane < ST / 32 ? s_s[lane] : 0.f;
#pragma unroll
        for (int o = 16; o; o >>= 1) {
            const float m2 = __shfl_xor_sync(0xffffffffu, m, o), s2 = __shfl_xor_sync(0xffffffffu, s, o);
            combine(m, s, m2, s2);
        }
        if (lane == 0) { p.row_stats[2 * (size_t)r] = m; p.row_stats[2 * (size_t)r + 1] = s; }
    }
    (void)status;
}

__global__ void __launch_bounds__(WT) accept_walk_kernel(graft_accept_stochastic_params p, unsigned* status) {
    __shared__ int s_par[64], s_tok[64];
    __shared__ float s_w[64];                 // weight exp(z - m) of node i's token in its parent's row
    __shared__ int s_rej[64];                 // tokens rejected at the node the walk ended at
    __shared__ float s_scan[WT];
    __shared__ int s_nrej, s_best, s_pick, s_owner;
    __shared__ float s_rem, s_base;
    const int tid = threadIdx.x, lane = tid & 31;
    const int b = blockIdx.x;
    const int T = p.tree_size[b];
    int32_t* path = p.path + (size_t)b * p.T_max;
    for (int j = tid; j < p.T_max; j += WT) path[j] = -1;
    if (T < 1 || T > p.T_max) {
        if (tid == 0) {
            p.n_acc[b] = 0; p.best_node[b] = -1; p.bonus[b] = -1;
            if (T != 0) atomicOr(status, (unsigned)GRAFT_FLAG_BAD_SIZE);
        }
        return;
    }
    const float inv_t = 1.f / p.temperature;
    const __nv_bfloat16* lg = reinterpret_cast<const __nv_bfloat16*>(p.logits) + (size_t)b * p.T_max * p.logits_stride_row;
    const float* stats = p.row_stats + 2 * (size_t)b * p.T_max;
    if (tid < 64) {
        int par = -1, x = -1;
        float w = 0.f;
        if (tid < T) {
            par = p.tree_parent[(size_t)b * p.T_max + tid];
            x = p.tree_token[(size_t)b * p.T_max + tid];
            if (tid == 0 || par < 0 || par >= tid) par = -1;               // the root, or not a tree node: nobody's child
            else if (x >= 0 && x < p.V) w = __expf(__bfloat162float(lg[(size_t)par * p.logits_stride_row + x]) * inv_t - stats[2 * par]);
        }
        s_par[tid] = par; s_tok[tid] = x; s_w[tid] = w;
    }
    __syncthreads();
    __syncthreads();                 // (path was cleared above by all threads; the walk below writes it)
    if (tid == 0) {
        int u = 0, n = 0, nrej = 0;
        float rem = 1.f;
        for (;;) {
            path[n++] = u;
            rem = 1.f;
            nrej = 0;
            const float inv_s = 1.f / stats[2 * u + 1];
            int next = -1;
            for (int c = u + 1; c < T; ++c) {
                if (s_par[c] != u) continue;
                const int x = s_tok[c];
                float px = s_w[c] * inv_s;
                for (int j = 0; j < nrej; ++j)
                    if (s_rej[j] == x) px = 0.f;                            // that mass is gone already
                if (p.u_accept[(size_t)b * p.T_max + c] * rem < px) { next = c; break; }
                if (x >= 0 && x < p.V && px > 0.f) { rem -= px; s_rej[nrej++] = x; }
            }
            if (next < 0) break;
            u = next;
        }
        s_best = u; s_nrej = nrej; s_rem = rem; s_pick = -1; s_owner = -1;
        p.n_acc[b] = n;
        p.best_node[b] = u;
    }
    __syncthreads();
    // ---- bonus: smallest id whose running sum of remaining weight exceeds the target
    const int u = s_best, nrej = s_nrej;
    const float m = stats[2 * u], target = p.u_bonus[b] * s_rem * stats[2 * u + 1];
    const __nv_bfloat16* row = lg + (size_t)u * p.logits_stride_row;
    const int chunk = (((p.V + WT - 1) / WT) + 7) & ~7;             // per thread, a multiple of one vector
    const int lo = min(p.V, tid * chunk), hi = min(p.V, lo + chunk);
    auto weight_sum = [&](int a, int e) {                            // sum of weights over [a, e), rejected ids left out
        float acc = 0.f;
        int v = a;
        for (; v < e && (v & 7); ++v) acc += __expf(__bfloat162float(row[v]) * inv_t - m);
        for (; v + 8 <= e; v += 8) {
            const uint4 q = *reinterpret_cast<const uint4*>(row + v);
            acc += __expf(lo_f(q.x) * inv_t - m) + __expf(hi_f(q.x) * inv_t - m) + __expf(lo_f(q.y) * inv_t - m) + __expf(hi_f(q.y) * inv_t - m) +
                   __expf(lo_f(q.z) * inv_t - m) + __expf(hi_f(q.z) * inv_t - m) + __expf(lo_f(q.w) * inv_t - m) + __expf(hi_f(q.w) * inv_t - m);
        }
        for (; v < e; ++v) acc += __expf(__bfloat162float(row[v]) * inv_t - m);
        for (int j = 0; j < nrej; ++j) {
            const int x = s_rej[j];
            if (x >= a && x < e) acc -= __expf(__bfloat162float(row[x]) * inv_t - m);
        }
        return fmaxf(acc, 0.f);
    };
    const float mine = weight_sum(lo, hi);
    s_scan[tid] = mine;
    __syncthreads();
    if (tid < 32) {                    // inclusive scan of the 256 chunk sums: eight per lane, then across lanes
        float loc[8], run = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) { run += s_scan[tid * 8 + e]; loc[e] = run; }
        float incl = run;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        const float excl = incl - run;
#pragma unroll
        for (int e = 0; e < 8; ++e) s_scan[tid * 8 + e] = excl + loc[e];
    }
    __syncthreads();
    const float incl = s_scan[tid], excl = tid ? s_scan[tid - 1] : 0.f;
    if (incl > target && !(excl > target)) { s_owner = tid; s_base = excl; }     // exactly one chunk: the sums do not decrease
    __syncthreads();
    const int owner = s_owner;
    if (owner < 0) {
        // rounding left the total just below the target: the last id that still has weight
        if (tid == 0) {
            int v = p.V - 1;
            for (; v >= 0; --v) {
                bool rej = false;
                for (int j = 0; j < nrej; ++j) rej |= s_rej[j] == v;
                if (!rej && __expf(__bfloat162float(row[v]) * inv_t - m) > 0.f) break;
            }
            p.bonus[b] = v;
        }
        return;
    }
    if ((tid >> 5) == (owner >> 5)) {            // the owner's warp splits the owner's chunk into 32 pieces
        const int olo = min(p.V, owner * chunk), ohi = min(p.V, olo + chunk);
        const int piece = (ohi - olo + 31) / 32;
        const int a = min(ohi, olo + lane * piece), e = min(ohi, a + piece);
        const float part = weight_sum(a, e);
        float inc = part;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float t = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += t;
        }
        const float base = s_base + inc - part;
        const bool has = base + part > target && !(base > target);
        const unsigned who = __ballot_sync(0xffffffffu, has);
        int pick = -1;
        if (who) {
            if (lane == __ffs(who) - 1) {
                float run = base;
                for (int v = a; v < e; ++v) {
                    bool rej = false;
                    for (int j = 0; j < nrej; ++j) rej |= s_rej[j] == v;
                    if (rej) continue;
                    const float w = __expf(__bfloat162float(row[v]) * inv_t - m);
                    if (w <= 0.f) continue;
                    pick = v;                      // the last weighted id so far: the answer if rounding ends the piece early
                    run += w;
                    if (run > target) break;
                }
                p.bonus[b] = pick;
            }
        } else if (lane == 0) {
            // the piece sums round differently from the chunk sum: fall back to a plain walk of the chunk
            float run = s_base;
            for (int v = olo; v < ohi; ++v) {
                bool rej = false;
                for (int j = 0; j < nrej; ++j) rej |= s_rej[j] == v;
                if (rej) continue;
                const float w = __expf(__bfloat162float(row[v]) * inv_t - m);
                if (w <= 0.f) continue;
                pick = v;
                run += w;
                if (run > target) break;
            }
            p.bonus[b] = pick;
        }
    }
}

}  // namespace

extern "C" int graft_accept_stochastic(graft_ctx* ctx, const graft_accept_stochastic_params* p, void* stream) {
    if (!ctx || !p) return GRAFT_ERR_INVALID_ARG;
    if (p->B <= 0 || p->T_max <= 0 || p->V <= 0 || !(p->temperature > 0.f)) return GRAFT_ERR_INVALID_ARG;
    if (p->T_max > 64) return GRAFT_ERR_UNSUPPORTED;
    if (!p->logits || !p->tree_token || !p->tree_parent || !p->tree_size || !p->u_accept || !p->u_bonus || !p->row_stats ||
        !p->n_acc || !p->path || !p->best_node || !p->bonus)
        return GRAFT_ERR_INVALID_ARG;
    if (!graft_aligned16(p->logits) || p->logits_stride_row < p->V || p->logits_stride_row % 8 != 0) return GRAFT_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    softmax_stats_kernel<<<p->B * p->T_max, ST, 0, s>>>(*p, ctx->status);
    GRAFT_CHECK_CUDA(cudaGetLastError());
    accept_walk_kernel<<<p->B, WT, 0, s>>>(*p, ctx->status);
    GRAFT_CHECK_CUDA(cudaGetLastError());
    return GRAFT_OK;
}
