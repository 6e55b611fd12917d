// graft_accept_stochastic: acceptance under temperature sampling, two kernels.
//
//   softmax_stats_kernel   two CTAs per tree node stream that node's V logits once (alternate rounds of steps) and
//                          leave their (max of logit / temperature, sum of exponentials) pairs and the same pair for
//                          every step of 256 ids: which rows the walk will need is only known while
//                          walking, so all valid rows are done at once, in parallel (HBM-bound: V * 2 bytes
//                          per valid node, as the adjacency refresh);
//   accept_walk_kernel     one CTA per request: every thread of the first T computes the probability of
//                          its node's token under the parent's distribution (one gather each), one thread
//                          walks the tree with those (sequential rejection over a node's children), then
//                          the CTA draws the bonus token from the last node's remaining distribution: a scan
//                          over that row's step sums (rejected tokens taken out) finds the step that crosses
//                          the target, one warp loads its 256 ids and finds the lane and the id.
#include <cuda_bf16.h>
#include <math_constants.h>
#include "graft_internal.cuh"

namespace {

constexpr int ST = 512;        // threads of the statistics kernel
constexpr int WT = 1024;       // threads of the walk kernel
constexpr int kStep = 256;     // ids per step: eight per lane of a warp
constexpr int kMaxSteps = 2 * WT;   // steps of a row the walk kernel can scan: V <= 524288
constexpr int kParts = 2;      // CTAs that share a row of the statistics kernel (alternate rounds of steps): one CTA per row left
                               // most SMs with one row and some with two (measured: -3 us on 192 rows, -8 us on 48)

__device__ __forceinline__ float lo_f(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float hi_f(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__host__ __device__ __forceinline__ int steps_of(int V) { return (V + kStep - 1) / kStep; }
// scratch of a row: (m, s) of each part of the row, then (m, s) of every step
__host__ __device__ __forceinline__ size_t row_floats(int V) { return 2 * kParts + 2 * (size_t)steps_of(V); }

// (m, s) <- (m, s) (+) (m2, s2): s counts exponentials relative to m
__device__ __forceinline__ void combine(float& m, float& s, float m2, float s2) {
    const float mn = fmaxf(m, m2);
    if (mn == -CUDART_INF_F) { m = mn; s = 0.f; return; }
    s = s * __expf(m - mn) + s2 * __expf(m2 - mn);
    m = mn;
}

// (m, s) of a whole row from its parts' pairs, and m alone
__device__ __forceinline__ void row_pair(const float* st, float& m, float& s) {
    m = st[0]; s = st[1];
#pragma unroll
    for (int q = 1; q < kParts; ++q) combine(m, s, st[2 * q], st[2 * q + 1]);
}
__device__ __forceinline__ float row_max(const float* st) {
    float m = st[0];
#pragma unroll
    for (int q = 1; q < kParts; ++q) m = fmaxf(m, st[2 * q]);
    return m;
}

// eight scaled logits of a lane: ids v0 .. v0 + 7 of the row, -inf past its end
__device__ __forceinline__ void scaled8(const __nv_bfloat16* row, int v0, int V, float inv_t, float (&z)[8]) {
    if (v0 + 8 <= V) {
        const uint4 q = __ldcs(reinterpret_cast<const uint4*>(row + v0));
        z[0] = lo_f(q.x) * inv_t; z[1] = hi_f(q.x) * inv_t; z[2] = lo_f(q.y) * inv_t; z[3] = hi_f(q.y) * inv_t;
        z[4] = lo_f(q.z) * inv_t; z[5] = hi_f(q.z) * inv_t; z[6] = lo_f(q.w) * inv_t; z[7] = hi_f(q.w) * inv_t;
    } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) z[e] = v0 + e < V ? __bfloat162float(row[v0 + e]) * inv_t : -CUDART_INF_F;
    }
}

// kParts CTAs per tree node; a warp takes a step of 256 ids at a time (four in flight), leaves the step's
// (max, sum of exponentials relative to it) and folds it into its running pair; the CTA leaves the pair of its part.
__global__ void __launch_bounds__(ST, 2) softmax_stats_kernel(graft_accept_stochastic_params p) {
    graft_wait_for_stream();
    __shared__ float s_m[ST / 32], s_s[ST / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int r = blockIdx.x / kParts, part = blockIdx.x % kParts, b = r / p.T_max, i = r % p.T_max;
    int T = p.tree_size[b];
    if (T < 0 || T > p.T_max) T = 0;
    if (i >= T) return;
    const float inv_t = 1.f / p.temperature;
    const __nv_bfloat16* row = reinterpret_cast<const __nv_bfloat16*>(p.logits) + (size_t)r * p.logits_stride_row;
    float* out = p.row_stats + (size_t)r * row_floats(p.V);
    const int nsteps = steps_of(p.V);
    float m = -CUDART_INF_F, s = 0.f;
    constexpr int NWS = ST / 32, kFlight = 4;          // steps a warp has in flight; they share one reference maximum
    for (int st = warp + part * kFlight * NWS; st < nsteps; st += kParts * kFlight * NWS) {
        float z[kFlight][8];
        float vm = -CUDART_INF_F;
        if ((st + (kFlight - 1) * NWS + 1) * kStep <= p.V) {
            // all four steps lie inside the row: four unconditional 16-byte loads in flight
            uint4 q[kFlight];
#pragma unroll
            for (int h = 0; h < kFlight; ++h) q[h] = __ldcs(reinterpret_cast<const uint4*>(row + (st + h * NWS) * kStep + lane * 8));
#pragma unroll
            for (int h = 0; h < kFlight; ++h) {
                z[h][0] = lo_f(q[h].x) * inv_t; z[h][1] = hi_f(q[h].x) * inv_t; z[h][2] = lo_f(q[h].y) * inv_t; z[h][3] = hi_f(q[h].y) * inv_t;
                z[h][4] = lo_f(q[h].z) * inv_t; z[h][5] = hi_f(q[h].z) * inv_t; z[h][6] = lo_f(q[h].w) * inv_t; z[h][7] = hi_f(q[h].w) * inv_t;
#pragma unroll
                for (int e = 0; e < 8; ++e) vm = fmaxf(vm, z[h][e]);
            }
        } else {
#pragma unroll
            for (int h = 0; h < kFlight; ++h) {
                if (st + h * NWS < nsteps) {
                    scaled8(row, (st + h * NWS) * kStep + lane * 8, p.V, inv_t, z[h]);
#pragma unroll
                    for (int e = 0; e < 8; ++e) vm = fmaxf(vm, z[h][e]);
                } else {
#pragma unroll
                    for (int e = 0; e < 8; ++e) z[h][e] = -CUDART_INF_F;
                }
            }
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) vm = fmaxf(vm, __shfl_xor_sync(0xffffffffu, vm, o));
        float add[kFlight];
#pragma unroll
        for (int h = 0; h < kFlight; ++h) {
            add[h] = 0.f;
            if (vm > -CUDART_INF_F) {
#pragma unroll
                for (int e = 0; e < 8; ++e) add[h] += __expf(z[h][e] - vm);
            }
        }
#pragma unroll
        for (int o = 16; o; o >>= 1)
#pragma unroll
            for (int h = 0; h < kFlight; ++h) add[h] += __shfl_xor_sync(0xffffffffu, add[h], o);
        float tot = 0.f;
#pragma unroll
        for (int h = 0; h < kFlight; ++h) {
            const int sx = st + h * NWS;
            if (sx < nsteps) {
                if (lane == h) { out[2 * kParts + 2 * sx] = vm; out[2 * kParts + 2 * sx + 1] = add[h]; }
                tot += add[h];
            }
        }
        combine(m, s, vm, tot);
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
        if (lane == 0) { out[2 * part] = m; out[2 * part + 1] = s; }
    }
}

__global__ void __launch_bounds__(WT) accept_walk_kernel(graft_accept_stochastic_params p, unsigned* status) {
    graft_wait_for_stream();
    constexpr int NW = WT / 32;
    __shared__ int s_par[64], s_tok[64];
    __shared__ float s_w[64];                 // weight exp(z - m) of node i's token in its parent's row
    __shared__ float s_u[64], s_m[64], s_s[64];   // the node's random number; its row's statistics
    __shared__ int s_rej[64];                 // tokens rejected at the node the walk ended at
    __shared__ float s_rejw[64];              // and their weights
    __shared__ float s_stepw[kMaxSteps];      // remaining weight of every step of the last node's row
    __shared__ float s_wtot[NW];
    __shared__ int s_nrej, s_best, s_pick, s_step;
    __shared__ float s_rem, s_base;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.x;
    const int T = p.tree_size[b];
    int32_t* path = p.path + (size_t)b * p.T_max;
    if (T < 1 || T > p.T_max) {
        for (int j = tid; j < p.T_max; j += WT) path[j] = -1;
        if (tid == 0) {
            p.n_acc[b] = 0; p.best_node[b] = -1; p.bonus[b] = -1;
            if (T != 0) atomicOr(status, (unsigned)GRAFT_FLAG_BAD_SIZE);
        }
        return;
    }
    const float inv_t = 1.f / p.temperature;
    const size_t rf = row_floats(p.V);
    const __nv_bfloat16* lg = reinterpret_cast<const __nv_bfloat16*>(p.logits) + (size_t)b * p.T_max * p.logits_stride_row;
    const float* stats = p.row_stats + (size_t)b * p.T_max * rf;
    if (tid < 64) {
        int par = -1, x = -1;
        float w = 0.f, u = 1.f, m = 0.f, sm = 1.f;
        if (tid < T) {
            par = p.tree_parent[(size_t)b * p.T_max + tid];
            x = p.tree_token[(size_t)b * p.T_max + tid];
            u = p.u_accept[(size_t)b * p.T_max + tid];
            row_pair(stats + tid * rf, m, sm);
            if (tid == 0 || par < 0 || par >= tid) par = -1;               // the root, or not a tree node: nobody's child
            else if (x >= 0 && x < p.V) w = __expf(__bfloat162float(lg[(size_t)par * p.logits_stride_row + x]) * inv_t - row_max(stats + par * rf));
        }
        s_par[tid] = par; s_tok[tid] = x; s_w[tid] = w; s_u[tid] = u; s_m[tid] = m; s_s[tid] = sm;
    }
    __syncthreads();
    if (tid == 0) {
        int u = 0, n = 0, nrej = 0;
        float rem = 1.f;
        for (;;) {
            path[n++] = u;
            rem = 1.f;
            nrej = 0;
            const float inv_s = 1.f / s_s[u];
            int next = -1;
            for (int c = u + 1; c < T; ++c) {
                if (s_par[c] != u) continue;
                const int x = s_tok[c];
                float px = s_w[c] * inv_s;
                for (int j = 0; j < nrej; ++j)
                    if (s_rej[j] == x) px = 0.f;                            // that mass is gone already
                if (s_u[c] * rem < px) { next = c; break; }
                if (x >= 0 && x < p.V && px > 0.f) { rem -= px; s_rejw[nrej] = s_w[c]; s_rej[nrej++] = x; }
            }
            if (next < 0) break;
            u = next;
        }
        for (int j = n; j < p.T_max; ++j) path[j] = -1;
        s_best = u; s_nrej = nrej; s_rem = rem; s_pick = -1; s_step = -1;
        p.n_acc[b] = n;
        p.best_node[b] = u;
    }
    __syncthreads();
    // ---- bonus: smallest id whose running sum of remaining weight exceeds the target.  The statistics
    // kernel left the sum of every step of 256 ids; find the step, then the lane, then the id.
    const int u = s_best, nrej = s_nrej;
    const float m = s_m[u], target = p.u_bonus[b] * s_rem * s_s[u];
    const __nv_bfloat16* row = lg + (size_t)u * p.logits_stride_row;
    const float* steps = stats + u * rf + 2 * kParts;
    const int nsteps = steps_of(p.V);
    for (int st = tid; st < nsteps; st += WT) {
        const float ms = steps[2 * st];
        s_stepw[st] = ms > -CUDART_INF_F ? steps[2 * st + 1] * __expf(ms - m) : 0.f;
    }
    __syncthreads();
    if (tid < nrej) atomicAdd(&s_stepw[s_rej[tid] / kStep], -s_rejw[tid]);
    __syncthreads();
    // inclusive scan over the steps: two per thread
    const float a0 = 2 * tid < nsteps ? fmaxf(s_stepw[2 * tid], 0.f) : 0.f;
    const float a1 = 2 * tid + 1 < nsteps ? fmaxf(s_stepw[2 * tid + 1], 0.f) : 0.f;
    float inc = a0 + a1;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) s_wtot[warp] = inc;
    __syncthreads();
    float before = 0.f;
    for (int w2 = 0; w2 < warp; ++w2) before += s_wtot[w2];
    const float e0 = before + inc - a0 - a1, e1 = e0 + a0, e2 = e1 + a1;      // running sums before, between and after my two steps
    if (e1 > target && !(e0 > target)) { s_step = 2 * tid; s_base = e0; }
    else if (e2 > target && !(e1 > target)) { s_step = 2 * tid + 1; s_base = e1; }
    __syncthreads();
    const int sx = s_step;
    if (sx >= 0 && warp == 0) {
        float z[8], w[8];
        const int v0 = sx * kStep + lane * 8;
        scaled8(row, v0, p.V, inv_t, z);
#pragma unroll
        for (int e = 0; e < 8; ++e) w[e] = __expf(z[e] - m);
        for (int j = 0; j < nrej; ++j) {
            const int d = s_rej[j] - v0;
            if (d >= 0 && d < 8) {
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    if (e == d) w[e] = 0.f;
            }
        }
        const float mine = ((w[0] + w[1]) + (w[2] + w[3])) + ((w[4] + w[5]) + (w[6] + w[7]));
        float li = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float t = __shfl_up_sync(0xffffffffu, li, o);
            if (lane >= o) li += t;
        }
        const float run = s_base;
        unsigned who = __ballot_sync(0xffffffffu, run + li > target);
        const unsigned any = __ballot_sync(0xffffffffu, mine > 0.f);
        if (!who && any) who = 1u << (31 - __clz(any));               // the lanes' sums round differently from the step's: the last lane with weight
        if (who && lane == __ffs(who) - 1) {
            float r2 = run + li - mine;
            int pick = -1, last = -1;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                if (w[e] > 0.f && pick < 0) {
                    last = v0 + e;
                    r2 += w[e];
                    if (r2 > target) pick = v0 + e;
                }
            }
            s_pick = pick < 0 ? last : pick;
        }
    }
    __syncthreads();
    if (tid == 0) {
        int pick = s_pick;
        if (pick < 0) {
            // rounding left the total just below the target: the last id that still has weight
            for (pick = p.V - 1; pick >= 0; --pick) {
                bool rej = false;
                for (int j = 0; j < nrej; ++j) rej |= s_rej[j] == pick;
                if (!rej && __expf(__bfloat162float(row[pick]) * inv_t - m) > 0.f) break;
            }
        }
        p.bonus[b] = pick;
    }
}

}  // namespace

extern "C" size_t graft_accept_stochastic_scratch_floats(int B, int T_max, int V) {
    if (B <= 0 || T_max <= 0 || V <= 0) return 0;
    return (size_t)B * T_max * row_floats(V);
}

extern "C" int graft_accept_stochastic(graft_ctx* ctx, const graft_accept_stochastic_params* p, void* stream) {
    if (!ctx || !p) return GRAFT_ERR_INVALID_ARG;
    if (p->B <= 0 || p->T_max <= 0 || p->V <= 0 || !(p->temperature > 0.f)) return GRAFT_ERR_INVALID_ARG;
    if (p->T_max > 64 || steps_of(p->V) > kMaxSteps) return GRAFT_ERR_UNSUPPORTED;
    if (!p->logits || !p->tree_token || !p->tree_parent || !p->tree_size || !p->u_accept || !p->u_bonus || !p->row_stats ||
        !p->n_acc || !p->path || !p->best_node || !p->bonus)
        return GRAFT_ERR_INVALID_ARG;
    if (!graft_aligned16(p->logits) || p->logits_stride_row < p->V || p->logits_stride_row % 8 != 0) return GRAFT_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // both kernels are programmatic dependents of the kernel before them: the walk's CTAs are set up while the statistics drain
    GRAFT_CHECK_CUDA(graft_launch(softmax_stats_kernel, dim3(p->B * p->T_max * kParts), dim3(ST), 0, s, *p));
    GRAFT_CHECK_CUDA(graft_launch(accept_walk_kernel, dim3(p->B), dim3(WT), 0, s, *p, ctx->status));
    return GRAFT_OK;
}
