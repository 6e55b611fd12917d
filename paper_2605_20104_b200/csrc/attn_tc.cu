// Tree-masked GQA attention on the 5th-generation tensor cores: TMA -> shared memory -> tcgen05.mma
// with accumulators in tensor memory (TMEM).
//
// One CTA per SM handles up to 256 rows (two blocks of 128; row r <-> tree node r / G, query head
// h*G + r % G) of one KV head against a contiguous range of 128-key tiles, so every K/V byte crosses
// HBM once for all rows that need it.  Warp roles:
//   warp 0      TMA producer: K and V tiles (two 64-column boxes each, 128-byte swizzle) into a
//               5-slot ring of 32 KB buffers, one mbarrier pair (full / empty) per slot
//   warp 1      MMA issuer: S = Q K^T (8 x m128 n128 k16, both operands from shared memory) and
//               O += P V (8 x m128 n128 k16, P from TMEM, V as an MN-major operand); owns TMEM
//   warps 4-7   softmax of row block 0: thread i <-> TMEM lane i <-> row i
//   warps 8-11  softmax of row block 1
// The two row blocks ping-pong: while one block's softmax runs on the SIMT pipes, the tensor pipe
// works on the other block (its P V of this tile, then its Q K^T of the next).  TMEM columns:
// S0 [0,128) S1 [128,256) O0 [256,384) O1 [384,512); P (bf16) overwrites the first 64 columns of
// its S.  tcgen05.mma instructions of one thread execute in issue order, so the Q K^T that refills S
// may be issued right behind the P V that reads P from it, and "S of tile j+1 is ready" implies
// "P V of tile j is complete" (O is quiescent whenever a softmax thread rescales it).
//
// Softmax keeps a reference maximum per row and rescales O only when the maximum grows by more
// than 2^8 (P then stays below 256, harmless in bf16/fp32); the row sum absorbs the same factor.
// The ancestor bitmask of a row lives in one 64-bit register and is applied only in tiles that
// reach past the cached prefix.  Cache slots at or past L_b + T_b inside the last tile are masked in S
// and their V rows are zeroed in shared memory (0 x NaN would otherwise poison the accumulator).
//
// Every mbarrier wait is bounded: on a timeout the kernel sets GRAFT_FLAG_WAIT_TIMEOUT, stops
// waiting anywhere in the CTA, drains its outstanding copies, frees TMEM and returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <math_constants.h>
#include <stdlib.h>
#include "attn_merge.cuh"
#include "attn_schedule.cuh"
#include "graft_internal.cuh"

namespace {

constexpr int BR = 256;          // rows per CTA (two blocks of 128)
constexpr int BN = 128;          // keys per tile
constexpr int D = 128;
constexpr int NSLOT = 5;         // ring slots of 32 KB (one K or V tile each)
constexpr int TILE_BYTES = BN * D * 2;
constexpr int HALF_BYTES = TILE_BYTES / 2;    // one 64-column box
constexpr int NTHREADS = 384;
constexpr int SMEM_DYN = 2 * TILE_BYTES + NSLOT * TILE_BYTES + 1024;   // Q (2 blocks) + ring + alignment slack
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kRescaleThreshold = 8.0f;     // log2 units
constexpr long long kWaitCycles = 1ll << 31;  // about a second

using TcArgs = graft_merge::AttnArgs;

// Experiment switches (component ablations, phase timers) exist only in builds with
// -DGRAFT_TC_EXPERIMENTS; in the library build every DBG(x) is a compile-time false.
#ifdef GRAFT_TC_EXPERIMENTS
#define DBG(x) (a.dbg & (x))
#else
#define DBG(x) false
#endif

// barrier indices: ring slots; S ready / P ready per row block; O final
enum { BAR_FULL = 0, BAR_EMPTY = NSLOT, BAR_S = 2 * NSLOT, BAR_P = 2 * NSLOT + 2, BAR_O = 2 * NSLOT + 4, BAR_COUNT = 2 * NSLOT + 5 };

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: gives up after about a second, or at once if another thread of the CTA already did.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned* status) {
    if (mbar_try_wait(bar, parity)) return;
    if (*abort_flag) return;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (*abort_flag) return;
        if (clock64() - t0 > kWaitCycles) {
            *abort_flag = 1;
            atomicOr(status, (unsigned)GRAFT_FLAG_WAIT_TIMEOUT);
            return;
        }
    }
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, int w, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(w), "r"(bar) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

// 32 consecutive TMEM columns of this thread's lane
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
          "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
          "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]) : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// two fp32 lanes in one 64-bit register, for the packed fma / add of sm_100
__device__ __forceinline__ unsigned long long pack2f(float lo, float hi) {
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2f(unsigned long long v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ unsigned long long ffma2(unsigned long long a, unsigned long long b, unsigned long long c) {
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ unsigned long long fadd2(unsigned long long a, unsigned long long b) {
    unsigned long long d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Shared-memory matrix descriptor, 128-byte swizzle, 8-row groups 1024 bytes apart (SBO).
// lbo_bytes: K-major operands ignore it (16 is the canonical value); MN-major operands use it as the
// distance between 64-element column blocks.
constexpr uint64_t desc_fixed(uint32_t lbo_bytes) {
    return ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) | ((uint64_t)((1024u >> 4) & 0x3FFFu) << 32) | (1ull << 46) |
           (2ull << 61);
}
constexpr uint64_t kDescKMajor = desc_fixed(16);            // Q and K tiles
constexpr uint64_t kDescVMajor = desc_fixed(HALF_BYTES);    // V tile as an MN-major operand
// the start-address field holds (shared address >> 4); shared addresses stay below 2^18, so adding a
// 16-byte-unit offset to a descriptor's low word never carries out of the field
__device__ __forceinline__ uint64_t smem_desc(uint64_t fixed, uint32_t addr16) { return fixed | (uint64_t)addr16; }

// instruction descriptors of kind::f16: fp32 accumulate, bf16 A and B, M = 128
constexpr uint32_t kIdescBase = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t kIdescQK = kIdescBase;                // N = 128 keys; A, B both K-major
constexpr uint32_t kIdescPV = kIdescBase | (1u << 16);   // N = d = 128; B (= V) MN-major

__global__ void __launch_bounds__(NTHREADS, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap vmap, TcArgs a, unsigned* status) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t s_bar[BAR_COUNT];
    __shared__ uint32_t s_tmem;
    __shared__ int s_abort;
    __shared__ graft_sched::Work s_work;

    const graft_attn_params& p = a.p;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    const uint32_t sQ = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sRing = sQ + 2 * TILE_BYTES;
    const uint32_t bar0 = smem_u32(s_bar);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    volatile int* abort_flag = &s_abort;
    // ring load n: K (n even) or V (n odd) of this CTA's tile n / 2
    auto issue_load = [&](const graft_sched::Work& ww, int n) {
        const int slot = n % NSLOT;
        const uint32_t dst = sRing + slot * TILE_BYTES;
        const int key0 = (ww.tile_lo + (n >> 1)) * BN;
        const CUtensorMap* map = (n & 1) ? &vmap : &kmap;
        mbar_expect_tx(bar(BAR_FULL + slot), TILE_BYTES);
        tma_load_4d(dst, map, 0, key0, ww.h, ww.b, bar(BAR_FULL + slot));
        tma_load_4d(dst + HALF_BYTES, map, 64, key0, ww.h, ww.b, bar(BAR_FULL + slot));
    };

    if (warp == 0) {
        graft_sched::Work w0 = graft_sched::find_work<BR, BN, true>(p.seq_len, p.tree_size, p.B, p.Hkv, a.G, p.T_max, p.S_cap,
                                                                   a.target, blockIdx.x, -1);
        if (lane == 0) {
            s_work = w0;
            s_abort = 0;
            if (w0.valid) {
                // barriers, then the first ring loads at once: their latency overlaps the Q load below
                for (int i = 0; i < NSLOT; ++i) { mbar_init(bar(BAR_FULL + i), 1); mbar_init(bar(BAR_EMPTY + i), 1); }
                for (int i = 0; i < 2; ++i) { mbar_init(bar(BAR_S + i), 1); mbar_init(bar(BAR_P + i), 4); }
                mbar_init(bar(BAR_O), 1);
                asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
                const int n_first = DBG(128) ? 0 : min(NSLOT, 2 * (w0.tile_hi - w0.tile_lo));
                for (int n = 0; n < n_first; ++n) issue_load(w0, n);
            }
        }
    }
    __syncthreads();
    const graft_sched::Work w = s_work;
    if (!w.valid) return;
    if (DBG(128)) return;

    const int G = a.G;
    const int R = w.T * G;
    const int row0 = w.rb * BR;
    const int nblk = (R - row0 > 128) ? 2 : 1;
    const int n_keys = w.L + w.T;
    const int nt = w.tile_hi - w.tile_lo;

    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }

    // ---- Q rows into shared memory, K-major with the 128-byte swizzle (16-byte chunk c of row r at c ^ (r & 7))
    {
        const __nv_bfloat16* Qg = reinterpret_cast<const __nv_bfloat16*>(p.Q) + (size_t)w.b * p.q_stride_b +
                                  (size_t)w.h * G * p.q_stride_h;
        constexpr int PER = (BR * 16 + NTHREADS - 1) / NTHREADS;
        uint4 v[PER];
#pragma unroll
        for (int q = 0; q < PER; ++q) {
            const int c = threadIdx.x + q * NTHREADS;
            const int rl = c >> 4, ch = c & 15;
            const int r = row0 + rl;
            v[q] = make_uint4(0u, 0u, 0u, 0u);
            if (c < BR * 16 && r < R) {
                const int t = r / G, g = r % G;
                v[q] = *reinterpret_cast<const uint4*>(Qg + (size_t)t * p.q_stride_t + (size_t)g * p.q_stride_h + ch * 8);
            }
        }
#pragma unroll
        for (int q = 0; q < PER; ++q) {
            const int c = threadIdx.x + q * NTHREADS;
            if (c < BR * 16) {
                const int rl = c >> 4, ch = c & 15;
                const int blk = rl >> 7, rr = rl & 127;
                const uint32_t dst = sQ + blk * TILE_BYTES + (ch >> 3) * HALF_BYTES + rr * 128 + (((ch & 7) ^ (rr & 7)) << 4);
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(v[q].x), "r"(v[q].y), "r"(v[q].z), "r"(v[q].w) : "memory");
            }
        }
        fence_async_smem();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;

    if (warp == 0) {
        // =============================== TMA producer ===============================
        if (lane == 0) {
            const int n_total = 2 * nt;
            int n = min(NSLOT, n_total);                      // the first loads were issued before the Q load
            if (DBG(64)) {                                 // experiment: loads only, reuse a slot as soon as it landed
                for (; n < n_total; ++n) {
                    mbar_wait(bar(BAR_FULL + n % NSLOT), (n / NSLOT - 1) & 1, abort_flag, status);
                    issue_load(w, n);
                }
            } else
            for (; n < n_total; ++n) {
                mbar_wait(bar(BAR_EMPTY + n % NSLOT), (n / NSLOT - 1) & 1, abort_flag, status);
                issue_load(w, n);
            }
            // drain: every copy issued must have landed before the CTA may exit
            for (int m = max(0, n - NSLOT); m < n; ++m) mbar_wait(bar(BAR_FULL + m % NSLOT), (m / NSLOT) & 1, abort_flag, status);
        }
    } else if (DBG(64)) {
    } else if (warp == 1) {
        // =============================== MMA issuer ===============================
        if (lane == 0) {
            auto wait_full = [&](int n) { mbar_wait(bar(BAR_FULL + n % NSLOT), (n / NSLOT) & 1, abort_flag, status); };
            // S[blk] = Q[blk] K(j)^T
            auto issue_qk = [&](int blk, int j) {
                const uint32_t sK16 = (sRing + ((2 * j) % NSLOT) * TILE_BYTES) >> 4;
                const uint32_t sQ16 = (sQ + blk * TILE_BYTES) >> 4;
                if (!DBG(2))
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint32_t off16 = ((k >> 2) * HALF_BYTES + (k & 3) * 32) >> 4;
                    mma_ss(tmem + blk * 128, smem_desc(kDescKMajor, sQ16 + off16), smem_desc(kDescKMajor, sK16 + off16), kIdescQK, k > 0);
                }
                tc_commit(bar(BAR_S + blk));
                if (blk == nblk - 1) tc_commit(bar(BAR_EMPTY + (2 * j) % NSLOT));          // K tile fully read
            };
            // O[blk] (+)= P[blk] V(j)
            auto issue_pv = [&](int blk, int j) {
                const uint32_t sV16 = (sRing + ((2 * j + 1) % NSLOT) * TILE_BYTES) >> 4;
                if (!DBG(4))
#pragma unroll
                for (int k = 0; k < BN / 16; ++k)
                    mma_ts(tmem + 256 + blk * 128, tmem + blk * 128 + k * 8, smem_desc(kDescVMajor, sV16 + k * (2048 >> 4)), kIdescPV,
                           (j > 0 || k > 0) ? 1u : 0u);
                if (blk == nblk - 1) tc_commit(bar(BAR_EMPTY + (2 * j + 1) % NSLOT));      // V tile fully read
            };
            wait_full(0);
            tc_fence_after();
            for (int blk = 0; blk < nblk; ++blk) issue_qk(blk, 0);
            long long m_waitp = 0, m_waitf = 0, m_issue = 0, mc0 = clock64(), mc1;
            const bool mprof = DBG(4096) && blockIdx.x == 0;
            for (int j = 0; j < nt; ++j) {
                for (int blk = 0; blk < nblk; ++blk) {
                    mbar_wait(bar(BAR_P + blk), j & 1, abort_flag, status);
                    if (mprof) { mc1 = clock64(); m_waitp += mc1 - mc0; mc0 = mc1; }
                    if (blk == 0) wait_full(2 * j + 1);
                    if (mprof) { mc1 = clock64(); m_waitf += mc1 - mc0; mc0 = mc1; }
                    tc_fence_after();
                    issue_pv(blk, j);
                    if (mprof) { mc1 = clock64(); m_issue += mc1 - mc0; mc0 = mc1; }
                    if (j + 1 < nt) {
                        if (blk == 0) { wait_full(2 * j + 2); tc_fence_after(); }
                        if (mprof) { mc1 = clock64(); m_waitf += mc1 - mc0; mc0 = mc1; }
                        issue_qk(blk, j + 1);
                        if (mprof) { mc1 = clock64(); m_issue += mc1 - mc0; mc0 = mc1; }
                    }
                }
            }
            if (mprof) {
                unsigned* dbgw = status + 24;
                dbgw[0] = (unsigned)(m_waitp / nt); dbgw[1] = (unsigned)(m_waitf / nt); dbgw[2] = (unsigned)(m_issue / nt);
            }
            tc_commit(bar(BAR_O));
        }
    } else if (warp >= 4) {
        // =============================== softmax + epilogue ===============================
        const int blk = (warp - 4) >> 2;
        if (blk < nblk) {
            const int rl = ((warp & 3) << 5) + lane;            // row inside the block = TMEM lane
            const int r = row0 + blk * 128 + rl;
            const bool row_valid = r < R;
            const int t = row_valid ? r / G : 0, g = row_valid ? r % G : 0;
            const unsigned long long anc = row_valid ? p.tree_anc[(size_t)w.b * p.T_max + t] : 0ull;
            const uint32_t lane_bits = (uint32_t)((warp & 3) << 5) << 16;
            const uint32_t tS = tmem + lane_bits + blk * 128;
            const uint32_t tO = tmem + lane_bits + 256 + blk * 128;
            const float sl2 = p.scale * kLog2e;
            float m_ref = -CUDART_INF_F, l = 0.f;

            if (DBG(8192) && blk == 1) { const long long t0 = clock64(); while (clock64() - t0 < 1700) {} }
            long long t_wait = 0, t_p1 = 0, t_p2 = 0, t_tail = 0, tc0 = clock64(), tc1;
            const bool prof = DBG(4096) && blockIdx.x == 0 && rl == 0;
            for (int j = 0; j < nt; ++j) {
                const int key0 = (w.tile_lo + j) * BN;
                const bool boundary = key0 + BN > w.L;
                mbar_wait(bar(BAR_S + blk), j & 1, abort_flag, status);
                tc_fence_after();
                if (prof) { tc1 = clock64(); t_wait += tc1 - tc0; tc0 = tc1; }
                // pass 1: row maximum of the (masked) scores, 64 columns in flight at a time
                auto mask32 = [&](uint32_t (&x)[32], int col0) {
#pragma unroll
                    for (int q = 0; q < 32; ++q) {
                        const int u = key0 + col0 + q - w.L;
                        if (!(u < 0 || (u < w.T && ((anc >> (u & 63)) & 1ull)))) x[q] = 0xff800000u;   // -inf
                    }
                };
                auto max32 = [&](const uint32_t (&x)[32], float& m0, float& m1) {
#pragma unroll
                    for (int q = 0; q < 32; q += 4) {
                        m0 = fmax3(m0, __uint_as_float(x[q]), __uint_as_float(x[q + 1]));
                        m1 = fmax3(m1, __uint_as_float(x[q + 2]), __uint_as_float(x[q + 3]));
                    }
                };
                float mx0 = -CUDART_INF_F, mx1 = -CUDART_INF_F;
                if (!DBG(8)) {
                    uint32_t x0[32], x1[32];
                    tmem_ld32(tS, x0);
                    tmem_ld32(tS + 32, x1);
                    tmem_wait_ld();
                    if (boundary) { mask32(x0, 0); mask32(x1, 32); }
                    max32(x0, mx0, mx1);
                    max32(x1, mx0, mx1);
                    tmem_ld32(tS + 64, x0);
                    tmem_ld32(tS + 96, x1);
                    tmem_wait_ld();
                    if (boundary) { mask32(x0, 64); mask32(x1, 96); }
                    max32(x0, mx0, mx1);
                    max32(x1, mx0, mx1);
                } else {
                    mx0 = 0.f;
                }
                const float mx = fmaxf(mx0, mx1);
                if (prof) { tc1 = clock64(); t_p1 += tc1 - tc0; tc0 = tc1; }
                // reference maximum: move it only when the scores outgrow it by more than the threshold
                if (mx != -CUDART_INF_F && (m_ref == -CUDART_INF_F || (mx - m_ref) * sl2 > kRescaleThreshold)) {
                    if (m_ref != -CUDART_INF_F) {
                        const float alpha = exp2f((m_ref - mx) * sl2);
                        l *= alpha;
#pragma unroll 1
                        for (int c = 0; c < 4; ++c) {       // O of the previous tiles is complete here
                            uint32_t o[32];
                            tmem_ld32(tO + c * 32, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int q = 0; q < 32; ++q) o[q] = __float_as_uint(__uint_as_float(o[q]) * alpha);
                            tmem_st32(tO + c * 32, o);
                        }
                        tmem_wait_st();
                    }
                    m_ref = mx;
                }
                const float off = m_ref == -CUDART_INF_F ? 0.f : m_ref * sl2;
                // pass 2: P = 2^(s*scale*log2e - off) as bf16 into the first 64 columns of S.  P chunk c
                // (columns 16c..16c+15) only overwrites score columns that are already in registers.
                float sum0 = 0.f, sum1 = 0.f;
                auto exp32 = [&](const uint32_t (&x)[32], uint32_t col) {
                    uint32_t pk[16];
#pragma unroll
                    for (int q = 0; q < 32; q += 2) {
                        const float p0 = ex2(fmaf(__uint_as_float(x[q]), sl2, -off));
                        const float p1 = ex2(fmaf(__uint_as_float(x[q + 1]), sl2, -off));
                        sum0 += p0;
                        sum1 += p1;
                        pk[q >> 1] = pack_bf16(p0, p1);
                    }
                    tmem_st16(tS + col, pk);
                };
                if (DBG(1)) {
                    uint32_t pk[16];
#pragma unroll
                    for (int q = 0; q < 16; ++q) pk[q] = 0x3f803f80u;
                    if (!DBG(16)) { tmem_st16(tS, pk); tmem_st16(tS + 16, pk); tmem_st16(tS + 32, pk); tmem_st16(tS + 48, pk); }
                    sum0 = 128.f;
                } else {
                    uint32_t x0[32], x1[32];
                    tmem_ld32(tS, x0);
                    tmem_ld32(tS + 32, x1);
                    tmem_wait_ld();
                    if (boundary) { mask32(x0, 0); mask32(x1, 32); }
                    exp32(x0, 0);
                    tmem_ld32(tS + 64, x0);
                    exp32(x1, 16);
                    tmem_ld32(tS + 96, x1);
                    tmem_wait_ld();
                    if (boundary) { mask32(x0, 64); mask32(x1, 96); }
                    exp32(x0, 32);
                    exp32(x1, 48);
                }
                l += sum0 + sum1;
                if (prof) { tc1 = clock64(); t_p2 += tc1 - tc0; tc0 = tc1; }
                tmem_wait_st();
                // last tile of the sequence: zero the V rows of slots that hold no key of this tree
                if (blk == 0 && key0 + BN > n_keys) {
                    const int nV = 2 * j + 1;
                    mbar_wait(bar(BAR_FULL + nV % NSLOT), (nV / NSLOT) & 1, abort_flag, status);
                    if (key0 + rl >= n_keys) {
                        const uint32_t sV = sRing + (nV % NSLOT) * TILE_BYTES + rl * 128;
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(sV + q * 16), "r"(0u) : "memory");
                            asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(sV + HALF_BYTES + q * 16), "r"(0u) : "memory");
                        }
                    }
                    fence_async_smem();
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(BAR_P + blk));      // one arrival per warp
                if (prof) { tc1 = clock64(); t_tail += tc1 - tc0; tc0 = tc1; }
            }
            if (prof) {
                unsigned* dbgw = status + 8 + blk * 8;
                dbgw[0] = (unsigned)nt; dbgw[1] = (unsigned)(t_wait / nt); dbgw[2] = (unsigned)(t_p1 / nt);
                dbgw[3] = (unsigned)(t_p2 / nt); dbgw[4] = (unsigned)(t_tail / nt);
            }

            // ---- epilogue: O row from TMEM, final result or partial
            mbar_wait(bar(BAR_O), 0, abort_flag, status);
            tc_fence_after();
            if (w.nsplit == 1) {
                const float inv = l > 0.f ? 1.f / l : 0.f;
                __nv_bfloat16* orow = reinterpret_cast<__nv_bfloat16*>(p.O) + (size_t)w.b * p.o_stride_b + (size_t)t * p.o_stride_t +
                                      (size_t)(w.h * G + g) * p.o_stride_h;
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    uint32_t v[32];
                    tmem_ld32(tO + c * 32, v);
                    tmem_wait_ld();
                    if (row_valid) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            uint4 o4;
                            o4.x = pack_bf16(__uint_as_float(v[q * 8 + 0]) * inv, __uint_as_float(v[q * 8 + 1]) * inv);
                            o4.y = pack_bf16(__uint_as_float(v[q * 8 + 2]) * inv, __uint_as_float(v[q * 8 + 3]) * inv);
                            o4.z = pack_bf16(__uint_as_float(v[q * 8 + 4]) * inv, __uint_as_float(v[q * 8 + 5]) * inv);
                            o4.w = pack_bf16(__uint_as_float(v[q * 8 + 6]) * inv, __uint_as_float(v[q * 8 + 7]) * inv);
                            *reinterpret_cast<uint4*>(orow + c * 32 + q * 8) = o4;
                        }
                    }
                }
                if (row_valid && p.LSE)
                    p.LSE[((size_t)w.b * p.Hq + w.h * G + g) * p.T_max + t] =
                        l > 0.f ? (m_ref * sl2 + log2f(l)) * graft_merge::kLn2 : -CUDART_INF_F;
            } else {
                float* base = a.partial + (size_t)graft_sched::slot_of(w, w.h, w.split, w.rb) * ((size_t)BR * (D + 2));
                const int lr = blk * 128 + rl;
                float* prow = base + (size_t)lr * D;
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    uint32_t v[32];
                    tmem_ld32(tO + c * 32, v);
                    tmem_wait_ld();
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        *reinterpret_cast<uint4*>(prow + c * 32 + q * 4) = make_uint4(v[q * 4], v[q * 4 + 1], v[q * 4 + 2], v[q * 4 + 3]);
                }
                base[BR * D + lr] = m_ref == -CUDART_INF_F ? -CUDART_INF_F : m_ref * sl2;
                base[BR * D + BR + lr] = l;
            }
        }
    }

    // ---- teardown: everyone is past its last TMEM access; the allocating warp frees the columns
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
}

int target_ctas(int num_sms) { return num_sms; }

int max_ctas(int num_sms, int B, int Hq, int Hkv, int T_max) {
    const int G = Hq / Hkv;
    return target_ctas(num_sms) + B * Hkv * ((T_max * G + BR - 1) / BR);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

int make_kv_map(CUtensorMap* map, const void* base, const graft_attn_params* p) {
    const cuuint64_t dims[4] = {(cuuint64_t)p->d, (cuuint64_t)p->S_cap, (cuuint64_t)p->Hkv, (cuuint64_t)p->B};
    const cuuint64_t strides[3] = {(cuuint64_t)p->kv_stride_s * 2, (cuuint64_t)p->kv_stride_h * 2, (cuuint64_t)p->kv_stride_b * 2};
    const cuuint32_t box[4] = {64, (cuuint32_t)BN, 1, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUresult rc = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return rc == CUDA_SUCCESS ? GRAFT_OK : GRAFT_ERR_CUDA;
}

}  // namespace

int graft_attn_tc_init() {
    if (!g_encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn ||
            q != cudaDriverEntryPointSuccess)
            return GRAFT_ERR_CUDA;
        g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    GRAFT_CHECK_CUDA(cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_DYN));
    return GRAFT_OK;
}

bool graft_attn_tc_supported(const graft_ctx* ctx, const graft_attn_params* p) {
    if (p->d != D) return false;
    // TMA: 16-byte aligned base and strides (checked by the caller), strides below 2^40 bytes, box rows within S_cap
    if (p->kv_stride_s * 2 >= (1ll << 40) || p->kv_stride_h * 2 >= (1ll << 40) || p->kv_stride_b * 2 >= (1ll << 40)) return false;
    if (p->kv_stride_s == 0 || p->kv_stride_h == 0 || p->kv_stride_b == 0) return false;
    return GRAFT_WS_HEADER + graft_attn_tc_ws_bytes(ctx->num_sms, p->B, p->Hq, p->Hkv, p->d, p->T_max) <= ctx->ws_bytes;
}

size_t graft_attn_tc_ws_bytes(int num_sms, int B, int Hq, int Hkv, int d, int T_max) {
    if (d != D) return 0;
    return (size_t)max_ctas(num_sms, B, Hq, Hkv, T_max) * BR * (D + 2) * sizeof(float);
}

int graft_attn_tc_launch(graft_ctx* ctx, const graft_attn_params* p, cudaStream_t stream) {
    CUtensorMap kmap, vmap;
    int rc = make_kv_map(&kmap, p->Kc, p);
    if (rc == GRAFT_OK) rc = make_kv_map(&vmap, p->Vc, p);
    if (rc != GRAFT_OK) return rc;
    TcArgs a;
    a.p = *p;
    a.partial = reinterpret_cast<float*>(reinterpret_cast<char*>(ctx->ws) + GRAFT_WS_HEADER);
    a.target = target_ctas(ctx->num_sms);
    a.G = p->Hq / p->Hkv;
#ifdef GRAFT_TC_EXPERIMENTS
    a.dbg = getenv("GRAFT_TC_DEBUG") ? atoi(getenv("GRAFT_TC_DEBUG")) : 0;
#else
    a.dbg = 0;
#endif
    attn_tc_kernel<<<max_ctas(ctx->num_sms, p->B, p->Hq, p->Hkv, p->T_max), NTHREADS, SMEM_DYN, stream>>>(kmap, vmap, a, ctx->status);
    GRAFT_CHECK_CUDA(cudaGetLastError());
    if (DBG(256)) return GRAFT_OK;
    return graft_merge::launch<D, BR, BN, true>(a, ctx->status, stream);
}
