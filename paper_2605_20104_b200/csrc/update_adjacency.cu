// graft_update_adjacency: M[token of node] <- ids of the k largest target logits at that node, one CTA per node.
//
// The row of V logits is streamed once, a small part of it twice (out of L2), never sorted:
//   pass 1  every thread keeps the maximum of the entries it sees (packed bf16 max); the k-th largest of the
//           512 thread maxima is a lower bound tau of the row's k-th largest entry, because the k largest
//           thread maxima are k different entries;
//   pass 2  entries above tau go to a candidate list in shared memory: they all sit with the at most k-1
//           threads whose maximum is above tau, so the list is bounded by (k-1) x entries per thread; entries
//           equal to tau are unbounded in number (ties are common in bf16), but only the k with the lowest
//           ids can matter.  Normally only a dozen threads reached tau: the CTA reads just their strides
//           again (one vector per thread, 2 % of the row).  With many ties every thread reads its own stride
//           again and keeps the first k ids it meets (it meets them in increasing order);
//   select  one warp takes the k best of the list (by value, equal values by id), then the CTA fills up
//           with the lowest ids among the entries equal to tau.
// NaN is never chosen (the packed max and the comparisons ignore it); -0 and +0 are equal.
// The node with the highest flattened index wins a token that several nodes of the step carry: a CTA
// writes its row of M only if no later valid node has the same token.
#include <cuda_bf16.h>
#include <math_constants.h>
#include "graft_internal.cuh"

namespace {

constexpr int UT = 512;             // threads per CTA
constexpr int UK = 16;              // largest k
constexpr int UCAP = 4608;          // candidate list entries

__device__ __forceinline__ uint32_t hmax2_bits(uint32_t a, uint32_t b) {
    __nv_bfloat162 x = *reinterpret_cast<__nv_bfloat162*>(&a), y = *reinterpret_cast<__nv_bfloat162*>(&b);
    __nv_bfloat162 m = __hmax2(x, y);
    return *reinterpret_cast<uint32_t*>(&m);
}
__device__ __forceinline__ uint32_t heq2_bits(uint32_t a, uint32_t b) {
    __nv_bfloat162 x = *reinterpret_cast<__nv_bfloat162*>(&a), y = *reinterpret_cast<__nv_bfloat162*>(&b);
    __nv_bfloat162 m = __heq2(x, y);
    return *reinterpret_cast<uint32_t*>(&m);
}
__device__ __forceinline__ float lo_f(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float hi_f(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// (value, id) order of the result: larger value first, equal values by lower id
__device__ __forceinline__ bool before(float va, int ia, float vb, int ib) { return va > vb || (va == vb && ia < ib); }

__global__ void __launch_bounds__(UT, 2) update_kernel(graft_update_params p, unsigned* status) {
    __shared__ float s_cv[UCAP];
    __shared__ int s_ci[UCAP];
    __shared__ float s_wtop[UT / 32][UK];
    __shared__ int s_rank[(UT / 32) * UK];
    __shared__ int s_hot[UT];
    __shared__ int s_cnt, s_nhot, s_min, s_dup;
    __shared__ float s_tau;
    __shared__ int s_top[UK];

    graft_wait_for_stream();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int r = blockIdx.x, b = r / p.T_max, i = r % p.T_max;
    int T = p.tree_size[b];
    if (T < 0 || T > p.T_max) {
        if (i == 0 && tid == 0) atomicOr(status, (unsigned)GRAFT_FLAG_BAD_SIZE);
        T = 0;
    }
    if (i >= T) {                       // padding node
        if (tid == 0 && p.target_next) p.target_next[r] = -1;
        return;
    }
    const int k = p.k, V = p.V;
    const uint16_t* row = reinterpret_cast<const uint16_t*>(p.logits) + (size_t)r * p.logits_stride_row;
    const uint4* row4 = reinterpret_cast<const uint4*>(row);
    const int nvec = V >> 3, ntail = V & 7;
    if (tid == 0) { s_cnt = 0; s_nhot = 0; }

    // ---- pass 1: thread maxima
    uint32_t m0 = 0xff80ff80u, m1 = m0, m2 = m0, m3 = m0;          // -inf pairs
    // four independent 16-byte loads per thread in flight: the scan is bound by memory latency otherwise
    constexpr int UNR = 4;
    for (int v = tid; v < nvec; v += UNR * UT) {
        uint4 q[UNR];
#pragma unroll
        for (int u = 0; u < UNR; ++u) q[u] = v + u * UT < nvec ? __ldg(row4 + v + u * UT) : make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
            m0 = hmax2_bits(m0, q[u].x); m1 = hmax2_bits(m1, q[u].y); m2 = hmax2_bits(m2, q[u].z); m3 = hmax2_bits(m3, q[u].w);
        }
    }
    m0 = hmax2_bits(hmax2_bits(m0, m1), hmax2_bits(m2, m3));
    float tm = fmaxf(lo_f(m0), hi_f(m0));
    if (tid < ntail) {
        const float f = lo_f(row[(size_t)nvec * 8 + tid]);
        if (f == f) tm = fmaxf(tm, f);
    }
    // ---- tau = k-th largest of the thread maxima: each warp sorts its 32 (bitonic, descending), warp 0 picks among the tops
    float x = tm;
#pragma unroll
    for (int size = 2; size <= 32; size <<= 1)
#pragma unroll
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            const float y = __shfl_xor_sync(0xffffffffu, x, stride);
            const bool up = ((lane & size) == 0) == ((lane & stride) == 0);      // keeps the larger one
            x = up ? fmaxf(x, y) : fminf(x, y);
        }
    if (lane < UK) s_wtop[warp][lane] = x;
    if (tid < (UT / 32) * UK) s_rank[tid] = 0;
    __syncthreads();
    // The k largest of a warp are the only ones of its 32 that can be among the k largest of all: (UT / 32) * k
    // candidates.  Every candidate counts how many candidates come before it (larger, or equal with a lower index), a few
    // threads per candidate sharing the count; the one with k - 1 before it is the k-th largest.
    {
        const int nc = (UT / 32) * k;                 // <= 256
        const int parts = UT / nc;                    // >= 2 threads per candidate
        const int c = tid % nc, part = tid / nc;
        if (part < parts) {
            const float v = s_wtop[c / k][c % k];
            const int per = (nc + parts - 1) / parts;
            const int lo = part * per, hi = min(nc, lo + per);
            int ahead = 0;
            int w = lo / k, jj = lo % k;                // candidate j = w * k + jj, walked without a division per step
            for (int j = lo; j < hi; ++j) {
                const float u = s_wtop[w][jj];
                ahead += (u > v || (u == v && j < c)) ? 1 : 0;
                if (++jj == k) { jj = 0; ++w; }
            }
            if (ahead) atomicAdd(&s_rank[c], ahead);
        }
        __syncthreads();
        if (tid < nc && s_rank[tid] == k - 1) s_tau = s_wtop[tid / k][tid % k];
    }
    __syncthreads();
    const float tau = s_tau;
    const __nv_bfloat16 tb = __float2bfloat16_rn(tau);       // exact: tau is a bf16 value
    const uint32_t t16 = *reinterpret_cast<const uint16_t*>(&tb);
    const uint32_t tau2 = t16 | (t16 << 16);

    // ---- pass 2: candidates above tau and the ids of the entries equal to tau.  Only threads whose maximum
    // reached tau can hold either, and they are few (k-1 above tau, plus ties): their strides are read again by
    // the whole CTA, one 16-byte vector per thread, out of L2.  Rows with so many ties at tau that this does not fit
    // (a constant row, say) take the general path: every thread reads its stride again and keeps its first k ids.
    const int iters = (nvec + UT - 1) / UT;               // vectors per stride
    if (tm >= tau) {
        const int at = atomicAdd(&s_nhot, 1);
        s_hot[at] = tid;
    }
    __syncthreads();
    const int nhot = s_nhot;
    const bool few = (long long)nhot * iters <= UT;
    uint32_t eqmask = 0;                // few: elements of this thread's vector that equal tau
    int vbase = 0;
    int eq[UK];                         // general path: the thread's first k ids equal to tau, increasing
    int n_eq = 0, ptr = 0;
    int tail_eq = 0x7fffffff;
    auto gt = [&](float f, int id) {
        const int at = atomicAdd(&s_cnt, 1);
        if (at < UCAP) { s_cv[at] = f; s_ci[at] = id; }
    };
    if (few) {
        if (tid < nhot * iters) {
            const int v = s_hot[tid / iters] + UT * (tid % iters);
            if (v < nvec) {
                const uint4 q = __ldg(row4 + v);
                const uint32_t w[4] = {q.x, q.y, q.z, q.w};
                vbase = v * 8;
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float f = (e & 1) ? hi_f(w[e >> 1]) : lo_f(w[e >> 1]);
                    if (f > tau) gt(f, vbase + e);
                    else if (f == tau) eqmask |= 1u << e;
                }
            }
        }
    } else {
        auto visit = [&](float f, int id) {
            if (f > tau) gt(f, id);
            else if (f == tau && n_eq < k) {
#pragma unroll
                for (int q = 0; q < UK; ++q)
                    if (q == n_eq) eq[q] = id;
                ++n_eq;
            }
        };
        auto visit_word = [&](uint32_t w, int id) {
            if (hmax2_bits(w, tau2) != tau2 || heq2_bits(w, tau2) != 0u) {
                visit(lo_f(w), id);
                visit(hi_f(w), id + 1);
            }
        };
        for (int v = tid; v < nvec; v += 4 * UT) {
            uint4 q[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)      // NaN pairs past the end: never candidates
                q[u] = v + u * UT < nvec ? __ldg(row4 + v + u * UT) : make_uint4(0x7fc07fc0u, 0x7fc07fc0u, 0x7fc07fc0u, 0x7fc07fc0u);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int id = (v + u * UT) * 8;
                visit_word(q[u].x, id);
                visit_word(q[u].y, id + 2);
                visit_word(q[u].z, id + 4);
                visit_word(q[u].w, id + 6);
            }
        }
    }
    if (tid < ntail) {                  // the last V % 8 entries, one per thread (their ids are the row's largest)
        const float f = lo_f(row[(size_t)nvec * 8 + tid]);
        if (f > tau) gt(f, nvec * 8 + tid);
        else if (f == tau) tail_eq = nvec * 8 + tid;
    }
    __syncthreads();
    int n_gt = s_cnt;
    if (n_gt > UCAP) {                  // cannot happen for shapes the host accepts
        if (tid == 0) atomicOr(status, (unsigned)GRAFT_FLAG_INTERNAL);
        n_gt = UCAP;
    }

    // ---- the k best of the list (warp 0)
    int n_sel = 0;
    if (n_gt <= UT) {
        // the usual, short list: every entry counts the entries that come before it and takes that place
        if (tid < n_gt) {
            const float v = s_cv[tid];
            const int id = s_ci[tid];
            int ahead = 0;
            for (int e = 0; e < n_gt; ++e) ahead += before(s_cv[e], s_ci[e], v, id) ? 1 : 0;
            if (ahead < k) s_top[ahead] = id;
        }
    } else if (warp == 0) {
        for (int j = 0; j < k && j < n_gt; ++j) {
            float bv = -CUDART_INF_F;
            int bi = 0x7fffffff, be = -1;
            for (int e = lane; e < n_gt; e += 32) {
                const int id = s_ci[e];
                if (id >= 0 && before(s_cv[e], id, bv, bi)) { bv = s_cv[e]; bi = id; be = e; }
            }
#pragma unroll
            for (int o = 16; o; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, o), oe = __shfl_xor_sync(0xffffffffu, be, o);
                if (before(ov, oi, bv, bi)) { bv = ov; bi = oi; be = oe; }
            }
            if (lane == 0) { s_top[j] = bi; s_ci[be] = -1; }
            __syncwarp();
        }
    }
    n_sel = n_gt < k ? n_gt : k;
    __syncthreads();

    // ---- fill up with the lowest ids among the entries equal to tau: every round each thread offers the lowest
    // id it still holds and the CTA takes the minimum
    for (int j = n_sel; j < k; ++j) {
        if (tid == 0) s_min = 0x7fffffff;
        __syncthreads();
        int cur = tail_eq;
        if (few) {
            if (eqmask) cur = vbase + __ffs(eqmask) - 1;
        } else {
#pragma unroll
            for (int q = 0; q < UK; ++q)
                if (q == ptr && q < n_eq) cur = eq[q];
        }
        if (cur != 0x7fffffff) atomicMin(&s_min, cur);
        __syncthreads();
        const int won = s_min;
        if (cur == won && cur != 0x7fffffff) {          // ids are unique: exactly one thread advances
            if (few && eqmask) eqmask &= eqmask - 1;
            else if (!few && ptr < n_eq) ++ptr;
            else tail_eq = 0x7fffffff;
        }
        if (tid == 0) {
            s_top[j] = won == 0x7fffffff ? -1 : won;
            if (won == 0x7fffffff) atomicOr(status, (unsigned)GRAFT_FLAG_NAN_SCORE);     // fewer than k entries that are not NaN
        }
    }
    __syncthreads();

    // ---- results: the greedy id; the row of M unless a later node of the step carries the same token
    const int tok = p.tree_token[r];
    if (tid == 0) {
        s_dup = 0;
        if (p.target_next) p.target_next[r] = s_top[0];
        if (tok != -1 && (tok < 0 || tok >= V)) atomicOr(status, (unsigned)GRAFT_FLAG_BAD_TOKEN);
    }
    __syncthreads();
    if (tok < 0 || tok >= V) return;
    const int N = p.B * p.T_max;
    bool dup = false;
    for (int r2 = r + 1 + tid; r2 < N; r2 += UT) {
        const int b2 = r2 / p.T_max, i2 = r2 % p.T_max;
        const int T2 = p.tree_size[b2];
        if (T2 >= 0 && T2 <= p.T_max && i2 < T2 && p.tree_token[r2] == tok) dup = true;
    }
    if (dup) s_dup = 1;
    __syncthreads();
    if (!s_dup && tid < k) p.M[(size_t)tok * k + tid] = s_top[tid];
}

}  // namespace

extern "C" int graft_update_adjacency(graft_ctx* ctx, const graft_update_params* p, void* stream) {
    if (!ctx || !p) return GRAFT_ERR_INVALID_ARG;
    if (p->B <= 0 || p->T_max <= 0 || p->V <= 0 || p->k <= 0) return GRAFT_ERR_INVALID_ARG;
    if (!p->logits || !p->tree_token || !p->tree_size || !p->M) return GRAFT_ERR_INVALID_ARG;
    if (!graft_aligned16(p->logits) || p->logits_stride_row < p->V || p->logits_stride_row % 8 != 0) return GRAFT_ERR_INVALID_ARG;
    if (p->k > UK || p->V < p->k) return GRAFT_ERR_UNSUPPORTED;
    // the candidate list holds what k-1 threads can contribute
    const long long per_thread = (((long long)(p->V >> 3) + UT - 1) / UT) * 8 + 1;
    if ((p->k - 1) * per_thread > UCAP) return GRAFT_ERR_UNSUPPORTED;
    GRAFT_CHECK_CUDA(graft_launch(update_kernel, dim3(p->B * p->T_max), dim3(UT), 0, static_cast<cudaStream_t>(stream), *p, ctx->status));
    return GRAFT_OK;
}
