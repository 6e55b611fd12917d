// Split-KV merge shared by the attention kernels.
//
// Partial slot layout (floats): O[BR][D] un-normalised relative to the slot's own row maxima, then
// m2[BR] (row maximum in the log2 domain, -inf if the split saw no visible key for the row), then
// l[BR] (row sum of 2^(s*scale*log2e - m2)).
// One warp per output row of the padded [T_max * G] row space of a (b, h_kv): rows of real nodes whose
// sequence was split are merged with  M = max m_i, w_i = 2^(m_i - M), O = sum w_i O_i / sum w_i l_i;
// rows of padding nodes are zeroed (LSE -inf); rows of unsplit sequences were already final.
#pragma once
#include <cuda_bf16.h>
#include <math_constants.h>
#include "attn_schedule.cuh"
#include "graft_internal.cuh"

namespace graft_merge {

constexpr float kLn2 = 0.6931471805599453f;
constexpr int kRowsPerCta = 8;      // one warp each

struct AttnArgs {
    graft_attn_params p;
    float* partial;     // workspace after the header
    int target;         // CTAs the schedule aims for
    int G;
    int dbg;            // experiment switches (0 in production)
};

__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

template <int D, int BR, int BN, bool FLOOR>
__global__ void __launch_bounds__(kRowsPerCta * 32, 2) merge_kernel(AttnArgs a, unsigned* status) {
    const graft_attn_params& p = a.p;
    const int G = a.G;
    const int rows_pad = p.T_max * G;
    const int groups = (rows_pad + kRowsPerCta - 1) / kRowsPerCta;
    int idx = blockIdx.x;
    const int grp = idx % groups; idx /= groups;
    const int h = idx % p.Hkv;
    const int b = idx / p.Hkv;
    __shared__ graft_sched::Work s_work;
    if (threadIdx.x < 32) {
        graft_sched::Work w = graft_sched::find_work<BR, BN, FLOOR>(p.seq_len, p.tree_size, p.B, p.Hkv, G, p.T_max, p.S_cap,
                                                             a.target, 0, b);
        if (threadIdx.x == 0) {
            s_work = w;
            const int T = p.tree_size[b], L = p.seq_len[b];
            if (grp == 0 && h == 0 && (T < 0 || T > p.T_max || L < 0 || (long long)L + T > p.S_cap))
                atomicOr(status, (unsigned)GRAFT_FLAG_BAD_SIZE);
        }
    }
    __syncthreads();
    const graft_sched::Work w = s_work;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r = grp * kRowsPerCta + warp;
    if (r >= rows_pad) return;
    constexpr int VPL = D / 32;      // floats per lane
    constexpr size_t SLOT = (size_t)BR * (D + 2);
    const int t = r / G, g = r % G;
    __nv_bfloat16* orow = reinterpret_cast<__nv_bfloat16*>(p.O) + (size_t)b * p.o_stride_b + (size_t)t * p.o_stride_t +
                          (size_t)(h * G + g) * p.o_stride_h + lane * VPL;
    float* lse = p.LSE ? p.LSE + ((size_t)b * p.Hq + h * G + g) * p.T_max + t : nullptr;
    if (t >= w.T) {                       // padding node: zero row
        if constexpr (VPL == 4) *reinterpret_cast<uint2*>(orow) = make_uint2(0u, 0u);
        else *reinterpret_cast<uint32_t*>(orow) = 0u;
        if (lse && lane == 0) *lse = -CUDART_INF_F;
        return;
    }
    if (w.nsplit <= 1) return;            // written by the attention kernel itself
    const int rb = r / BR, rl = r % BR;
    const float* slot0 = a.partial + (size_t)graft_sched::slot_of(w, h, 0, rb) * SLOT;
    const size_t split_stride = (size_t)w.nrb * SLOT;       // slots of consecutive splits
    float acc[VPL];
#pragma unroll
    for (int v = 0; v < VPL; ++v) acc[v] = 0.f;
    float den = 0.f;
    if (w.nsplit <= 32) {
        // common case: lane s owns split s; one round of (m, l) loads, then every O load in flight at once
        float m = -CUDART_INF_F, l = 0.f;
        if (lane < w.nsplit) {
            m = slot0[lane * split_stride + BR * D + rl];
            l = slot0[lane * split_stride + BR * D + BR + rl];
        }
        float M = m;
#pragma unroll
        for (int o = 16; o; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
        const float wgt = (m == -CUDART_INF_F) ? 0.f : exp2f(m - M);
        den = wgt * l;
        const float* orow_p = slot0 + (size_t)rl * D + lane * VPL;
        // 16 partial rows in flight per round
        for (int j0 = 0; j0 < w.nsplit; j0 += 16) {
            if constexpr (VPL == 4) {
                float4 x[16];
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    if (j0 + j < w.nsplit) x[j] = *reinterpret_cast<const float4*>(orow_p + (size_t)(j0 + j) * split_stride);
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    if (j0 + j < w.nsplit) {
                        const float wj = __shfl_sync(0xffffffffu, wgt, j0 + j);
                        acc[0] += wj * x[j].x; acc[1] += wj * x[j].y; acc[2] += wj * x[j].z; acc[3] += wj * x[j].w;
                    }
            } else {
                float2 x[16];
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    if (j0 + j < w.nsplit) x[j] = *reinterpret_cast<const float2*>(orow_p + (size_t)(j0 + j) * split_stride);
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    if (j0 + j < w.nsplit) {
                        const float wj = __shfl_sync(0xffffffffu, wgt, j0 + j);
                        acc[0] += wj * x[j].x; acc[1] += wj * x[j].y;
                    }
            }
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
        const float inv = den > 0.f ? 1.f / den : 0.f;
        if constexpr (VPL == 4) {
            *reinterpret_cast<uint2*>(orow) = make_uint2(pack2(acc[0] * inv, acc[1] * inv), pack2(acc[2] * inv, acc[3] * inv));
        } else {
            *reinterpret_cast<uint32_t*>(orow) = pack2(acc[0] * inv, acc[1] * inv);
        }
        if (lse && lane == 0) *lse = den > 0.f ? (M + log2f(den)) * kLn2 : -CUDART_INF_F;
        return;
    }
    float M = -CUDART_INF_F;
    for (int s = lane; s < w.nsplit; s += 32) M = fmaxf(M, slot0[s * split_stride + BR * D + rl]);
#pragma unroll
    for (int o = 16; o; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    for (int s0 = 0; s0 < w.nsplit; s0 += 32) {
        const int s = s0 + lane;
        float wgt = 0.f, l = 0.f;
        if (s < w.nsplit) {
            const float m = slot0[s * split_stride + BR * D + rl];
            l = slot0[s * split_stride + BR * D + BR + rl];
            wgt = (m == -CUDART_INF_F || M == -CUDART_INF_F) ? 0.f : exp2f(m - M);
        }
        den += wgt * l;
        const int cnt = min(32, w.nsplit - s0);
        const float* orow_p = slot0 + (size_t)s0 * split_stride + (size_t)rl * D + lane * VPL;
#pragma unroll 4
        for (int j = 0; j < cnt; ++j) {
            const float wj = __shfl_sync(0xffffffffu, wgt, j);
            if constexpr (VPL == 4) {
                const float4 x = *reinterpret_cast<const float4*>(orow_p + (size_t)j * split_stride);
                acc[0] += wj * x.x; acc[1] += wj * x.y; acc[2] += wj * x.z; acc[3] += wj * x.w;
            } else {
                const float2 x = *reinterpret_cast<const float2*>(orow_p + (size_t)j * split_stride);
                acc[0] += wj * x.x; acc[1] += wj * x.y;
            }
        }
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
    const float inv = den > 0.f ? 1.f / den : 0.f;
    if constexpr (VPL == 4) {
        *reinterpret_cast<uint2*>(orow) = make_uint2(pack2(acc[0] * inv, acc[1] * inv), pack2(acc[2] * inv, acc[3] * inv));
    } else {
        *reinterpret_cast<uint32_t*>(orow) = pack2(acc[0] * inv, acc[1] * inv);
    }
    if (lse && lane == 0) *lse = den > 0.f ? (M + log2f(den)) * kLn2 : -CUDART_INF_F;
}

template <int D, int BR, int BN, bool FLOOR = false>
static int launch(const AttnArgs& a, unsigned* status, cudaStream_t stream) {
    const int groups = (a.p.T_max * a.G + kRowsPerCta - 1) / kRowsPerCta;
    merge_kernel<D, BR, BN, FLOOR><<<a.p.B * a.p.Hkv * groups, kRowsPerCta * 32, 0, stream>>>(a, status);
    GRAFT_CHECK_CUDA(cudaGetLastError());
    return GRAFT_OK;
}

}  // namespace graft_merge
