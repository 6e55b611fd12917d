// Tree-masked GQA attention, register-tile kernel (mma.sync m16n8k16, bf16 in / fp32 accumulate).
//
// This is the path for small row counts and odd shapes (d = 64, unaligned cache rows), and the
// reference point the tcgen05 kernel is measured against.  One CTA = 128 rows (row r <-> tree
// node r / G, query head h*G + r % G) of one KV head against a contiguous range of 64-key tiles;
// 8 warps x 16 rows, K/V tiles double-buffered in swizzled shared memory with cp.async (16-byte
// coalesced loads), online softmax in registers, ancestor bitmask of each thread's two rows held in
// two 64-bit registers.  Partial (m, l, O) triples go to the workspace and a second kernel merges.
#include <cuda_bf16.h>
#include <math_constants.h>
#include "attn_schedule.cuh"
#include "attn_merge.cuh"
#include "graft_internal.cuh"

namespace {

constexpr int BR = 128;       // rows per CTA
constexpr int BN = 64;        // keys per tile
constexpr int NTHREADS = 256;
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool pred) {
    const int n = pred ? 16 : 0;     // src-size 0: the 16 bytes are zero-filled, nothing is read
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(n));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// byte offset of 16-byte chunk `chunk` of row `row` in a tile whose rows are D bf16 long
template <int D>
__device__ __forceinline__ uint32_t swz(int row, int chunk) {
    return (uint32_t)(row * (D * 2) + ((chunk ^ (row & 7)) << 4));
}

using MmaArgs = graft_merge::AttnArgs;

// where a sequence's cache slots live: one contiguous run, or pages of a pool looked up in the sequence's block table
struct KvPlace {
    const int32_t* table;      // the sequence's row of the block table, or nullptr
    int page_size, n_blocks;
    int64_t stride_b, stride_s;
};
// element offset of cache slot `key` (from the KV head's base); false if its table entry is out of range
__device__ __forceinline__ bool kv_offset(const KvPlace& pl, int key, size_t& off) {
    if (!pl.table) { off = (size_t)key * pl.stride_s; return true; }
    const int blk = pl.table[key / pl.page_size];
    if (blk < 0 || blk >= pl.n_blocks) return false;
    off = (size_t)blk * pl.stride_b + (size_t)(key % pl.page_size) * pl.stride_s;
    return true;
}

template <int D>
__device__ __forceinline__ bool load_kv_tile(uint32_t sK, uint32_t sV, const __nv_bfloat16* Kg, const __nv_bfloat16* Vg,
                                             const KvPlace& pl, int key0, int n_keys) {
    constexpr int CH = D / 8;
    bool all_ok = true;
    for (int c = threadIdx.x; c < BN * CH; c += NTHREADS) {
        const int row = c / CH, ch = c % CH;
        const int key = key0 + row;
        bool ok = key < n_keys;
        size_t off = 0;
        if (ok && !kv_offset(pl, key, off)) { ok = false; all_ok = false; }
        off = ok ? off + ch * 8 : 0;
        cp_async16(sK + swz<D>(row, ch), Kg + off, ok);
        cp_async16(sV + swz<D>(row, ch), Vg + off, ok);
    }
    return all_ok;
}

template <int D>
__global__ void __launch_bounds__(NTHREADS, 2) attn_mma_kernel(MmaArgs a, unsigned* status) {
    extern __shared__ __align__(128) unsigned char smem[];
    const graft_attn_params& p = a.p;
    constexpr int TILE_BYTES = BN * D * 2;
    const uint32_t sQ = smem_u32(smem);
    const uint32_t sKV = sQ + BR * D * 2;      // [stage][K, V]

    __shared__ graft_sched::Work s_work;
    if (threadIdx.x < 32) {
        graft_sched::Work w = graft_sched::find_work<BR, BN>(p.seq_len, p.tree_size, p.B, p.Hkv, a.G, p.T_max, p.S_cap,
                                                             a.target, blockIdx.x, -1);
        if (threadIdx.x == 0) s_work = w;
    }
    __syncthreads();
    const graft_sched::Work w = s_work;
    if (!w.valid) return;

    const int G = a.G;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int R = w.T * G;                       // valid rows of this (b, h)
    const int row0 = w.rb * BR;
    const int n_keys = w.L + w.T;
    const __nv_bfloat16* Qg = reinterpret_cast<const __nv_bfloat16*>(p.Q) + (size_t)w.b * p.q_stride_b +
                              (size_t)w.h * G * p.q_stride_h;
    const size_t seq_off = p.block_table ? 0 : (size_t)w.b * p.kv_stride_b;          // pages are found through the table
    const __nv_bfloat16* Kg = reinterpret_cast<const __nv_bfloat16*>(p.Kc) + seq_off + (size_t)w.h * p.kv_stride_h;
    const __nv_bfloat16* Vg = reinterpret_cast<const __nv_bfloat16*>(p.Vc) + seq_off + (size_t)w.h * p.kv_stride_h;
    const KvPlace place = {p.block_table ? p.block_table + (size_t)w.b * p.blocks_per_seq : nullptr, p.page_size, p.n_blocks,
                           p.kv_stride_b, p.kv_stride_s};
    bool table_ok = true;

    // ---- prologue: Q rows and the first two K/V tiles
    {
        constexpr int CH = D / 8;
        for (int c = threadIdx.x; c < BR * CH; c += NTHREADS) {
            const int row = c / CH, ch = c % CH;
            const int r = row0 + row;
            const bool ok = r < R;
            const int t = ok ? r / G : 0, g = ok ? r % G : 0;
            cp_async16(sQ + swz<D>(row, ch), Qg + (size_t)t * p.q_stride_t + (size_t)g * p.q_stride_h + ch * 8, ok);
        }
    }
    table_ok &= load_kv_tile<D>(sKV, sKV + TILE_BYTES, Kg, Vg, place, w.tile_lo * BN, n_keys);
    cp_async_commit();
    if (w.tile_lo + 1 < w.tile_hi)
        table_ok &= load_kv_tile<D>(sKV + 2 * TILE_BYTES, sKV + 3 * TILE_BYTES, Kg, Vg, place, (w.tile_lo + 1) * BN, n_keys);
    cp_async_commit();

    // ---- per-thread rows: lane/4 and lane/4 + 8 of the warp's 16
    const int rA = row0 + warp * 16 + (lane >> 2);
    const int rB = rA + 8;
    const bool warp_active = row0 + warp * 16 < R;
    unsigned long long ancA = 0, ancB = 0;
    if (rA < R) ancA = p.tree_anc[(size_t)w.b * p.T_max + rA / G];
    if (rB < R) ancB = p.tree_anc[(size_t)w.b * p.T_max + rB / G];

    const float sl2 = p.scale * kLog2e;
    float o[D / 8][4];
#pragma unroll
    for (int i = 0; i < D / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    float mA = -CUDART_INF_F, mB = -CUDART_INF_F, lA = 0.f, lB = 0.f;

    for (int tile = w.tile_lo; tile < w.tile_hi; ++tile) {
        const int stage = (tile - w.tile_lo) & 1;
        const uint32_t sK = sKV + stage * 2 * TILE_BYTES, sV = sK + TILE_BYTES;
        cp_async_wait<1>();
        __syncthreads();
        if (warp_active) {
            // S = Q K^T for this warp's 16 rows x 64 keys
            float s[BN / 8][4];
#pragma unroll
            for (int i = 0; i < BN / 8; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                uint32_t qa[4];
                {
                    const int id = lane >> 3;
                    ldmatrix_x4(qa, sQ + swz<D>(warp * 16 + (lane & 7) + (id & 1) * 8, ks * 2 + (id >> 1)));
                }
#pragma unroll
                for (int np = 0; np < BN / 16; ++np) {
                    uint32_t kb[4];
                    const int id = lane >> 3;
                    ldmatrix_x4(kb, sK + swz<D>(np * 16 + (lane & 7) + (id >> 1) * 8, ks * 2 + (id & 1)));
                    mma_bf16(s[2 * np], qa, kb[0], kb[1]);
                    mma_bf16(s[2 * np + 1], qa, kb[2], kb[3]);
                }
            }
            // tree mask: only tiles that reach past the cached prefix
            const int key0 = tile * BN;
            if (key0 + BN > w.L) {
#pragma unroll
                for (int nt = 0; nt < BN / 8; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int key = key0 + nt * 8 + (lane & 3) * 2 + (e & 1);
                        const unsigned long long anc = (e & 2) ? ancB : ancA;
                        const int u = key - w.L;
                        const bool vis = u < 0 || (u < w.T && ((anc >> u) & 1ull));
                        if (!vis) s[nt][e] = -CUDART_INF_F;
                    }
            }
            // online softmax
            float mxA = -CUDART_INF_F, mxB = -CUDART_INF_F;
#pragma unroll
            for (int nt = 0; nt < BN / 8; ++nt) {
                mxA = fmaxf(mxA, fmaxf(s[nt][0], s[nt][1]));
                mxB = fmaxf(mxB, fmaxf(s[nt][2], s[nt][3]));
            }
            mxA = fmaxf(mxA, __shfl_xor_sync(0xffffffffu, mxA, 1));
            mxA = fmaxf(mxA, __shfl_xor_sync(0xffffffffu, mxA, 2));
            mxB = fmaxf(mxB, __shfl_xor_sync(0xffffffffu, mxB, 1));
            mxB = fmaxf(mxB, __shfl_xor_sync(0xffffffffu, mxB, 2));
            const float mnA = fmaxf(mA, mxA), mnB = fmaxf(mB, mxB);
            // a row that has seen no visible key yet keeps m = -inf; its exponent offset is 0
            const float offA = mnA == -CUDART_INF_F ? 0.f : mnA * sl2;
            const float offB = mnB == -CUDART_INF_F ? 0.f : mnB * sl2;
            const float alA = mnA == -CUDART_INF_F ? 1.f : exp2f(mA * sl2 - offA);
            const float alB = mnB == -CUDART_INF_F ? 1.f : exp2f(mB * sl2 - offB);
            mA = mnA;
            mB = mnB;
            float sumA = 0.f, sumB = 0.f;
            uint32_t pa[BN / 16][4];
#pragma unroll
            for (int nt = 0; nt < BN / 8; ++nt) {
                const float p0 = exp2f(s[nt][0] * sl2 - offA), p1 = exp2f(s[nt][1] * sl2 - offA);
                const float p2 = exp2f(s[nt][2] * sl2 - offB), p3 = exp2f(s[nt][3] * sl2 - offB);
                sumA += p0 + p1;
                sumB += p2 + p3;
                pa[nt >> 1][(nt & 1) * 2] = pack_bf16(p0, p1);
                pa[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p2, p3);
            }
            lA = lA * alA + sumA;
            lB = lB * alB + sumB;
#pragma unroll
            for (int i = 0; i < D / 8; ++i) {
                o[i][0] *= alA; o[i][1] *= alA;
                o[i][2] *= alB; o[i][3] *= alB;
            }
            // O += P V
#pragma unroll
            for (int kk = 0; kk < BN / 16; ++kk) {
#pragma unroll
                for (int np = 0; np < D / 16; ++np) {
                    uint32_t vb[4];
                    const int id = lane >> 3;
                    ldmatrix_x4_trans(vb, sV + swz<D>(kk * 16 + (lane & 7) + (id & 1) * 8, np * 2 + (id >> 1)));
                    mma_bf16(o[2 * np], pa[kk], vb[0], vb[1]);
                    mma_bf16(o[2 * np + 1], pa[kk], vb[2], vb[3]);
                }
            }
        }
        __syncthreads();
        if (tile + 2 < w.tile_hi) table_ok &= load_kv_tile<D>(sK, sV, Kg, Vg, place, (tile + 2) * BN, n_keys);
        cp_async_commit();
    }
    cp_async_wait<0>();
    if (!table_ok) atomicOr(status, (unsigned)GRAFT_FLAG_BAD_SIZE);          // a block-table entry outside the pool: its keys read as zeros

    // ---- epilogue: quad-reduce the row sums, then either the final result or a partial
    lA += __shfl_xor_sync(0xffffffffu, lA, 1);
    lA += __shfl_xor_sync(0xffffffffu, lA, 2);
    lB += __shfl_xor_sync(0xffffffffu, lB, 1);
    lB += __shfl_xor_sync(0xffffffffu, lB, 2);
    if (!warp_active) return;
    if (w.nsplit == 1) {
        __nv_bfloat16* Og = reinterpret_cast<__nv_bfloat16*>(p.O) + (size_t)w.b * p.o_stride_b + (size_t)w.h * G * p.o_stride_h;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int r = half ? rB : rA;
            if (r >= R) continue;
            const float l = half ? lB : lA, m = half ? mB : mA;
            const float inv = l > 0.f ? 1.f / l : 0.f;
            const int t = r / G, g = r % G;
            __nv_bfloat16* orow = Og + (size_t)t * p.o_stride_t + (size_t)g * p.o_stride_h;
#pragma unroll
            for (int i = 0; i < D / 8; ++i) {
                const uint32_t v = pack_bf16(o[i][half * 2] * inv, o[i][half * 2 + 1] * inv);
                *reinterpret_cast<uint32_t*>(orow + i * 8 + (lane & 3) * 2) = v;
            }
            if (p.LSE && (lane & 3) == 0)
                p.LSE[((size_t)w.b * p.Hq + w.h * G + g) * p.T_max + t] = l > 0.f ? (m * sl2 + log2f(l)) * graft_merge::kLn2 : -CUDART_INF_F;
        }
    } else {
        const int slot = graft_sched::slot_of(w, w.h, w.split, w.rb);
        float* base = a.partial + (size_t)slot * (BR * (D + 2));
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int lr = warp * 16 + (lane >> 2) + half * 8;
            float* orow = base + (size_t)lr * D;
#pragma unroll
            for (int i = 0; i < D / 8; ++i)
                *reinterpret_cast<float2*>(orow + i * 8 + (lane & 3) * 2) = make_float2(o[i][half * 2], o[i][half * 2 + 1]);
            if ((lane & 3) == 0) {
                const float m = half ? mB : mA;
                base[BR * D + lr] = m == -CUDART_INF_F ? -CUDART_INF_F : m * sl2;
                base[BR * D + BR + lr] = half ? lB : lA;
            }
        }
    }
}

int target_ctas(int num_sms) { return num_sms * 2 * 2; }   // 2 resident CTAs per SM, 2 waves

int max_slots(int num_sms, int B, int Hq, int Hkv, int T_max) {
    const int G = Hq / Hkv;
    const int nrb_max = (T_max * G + BR - 1) / BR;
    return target_ctas(num_sms) + B * Hkv * nrb_max;
}

}  // namespace

size_t graft_attn_mma_ws_bytes(int num_sms, int B, int Hq, int Hkv, int d, int T_max) {
    return (size_t)max_slots(num_sms, B, Hq, Hkv, T_max) * BR * (d + 2) * sizeof(float);
}

template <int D>
static int launch(graft_ctx* ctx, const graft_attn_params* p, cudaStream_t stream) {
    MmaArgs a;
    a.p = *p;
    a.partial = reinterpret_cast<float*>(reinterpret_cast<char*>(ctx->ws) + GRAFT_WS_HEADER);
    a.target = target_ctas(ctx->num_sms);
    a.G = p->Hq / p->Hkv;
    a.dbg = 0;
    const int grid = max_slots(ctx->num_sms, p->B, p->Hq, p->Hkv, p->T_max);
    const size_t smem = (size_t)BR * D * 2 + 4 * (size_t)BN * D * 2;
    attn_mma_kernel<D><<<grid, NTHREADS, smem, stream>>>(a, ctx->status);
    GRAFT_CHECK_CUDA(cudaGetLastError());
    return graft_merge::launch<D, BR, BN>(a, ctx->status, stream);
}

int graft_attn_mma_init() {
    // opt in to > 48 KB of dynamic shared memory on the current device
    GRAFT_CHECK_CUDA(cudaFuncSetAttribute(attn_mma_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          BR * 128 * 2 + 4 * BN * 128 * 2));
    GRAFT_CHECK_CUDA(cudaFuncSetAttribute(attn_mma_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          BR * 64 * 2 + 4 * BN * 64 * 2));
    return GRAFT_OK;
}

int graft_attn_mma_launch(graft_ctx* ctx, const graft_attn_params* p, cudaStream_t stream) {
    if (GRAFT_WS_HEADER + graft_attn_mma_ws_bytes(ctx->num_sms, p->B, p->Hq, p->Hkv, p->d, p->T_max) > ctx->ws_bytes)
        return GRAFT_ERR_WORKSPACE_TOO_SMALL;
    return p->d == 128 ? launch<128>(ctx, p, stream) : launch<64>(ctx, p, stream);
}
