// Tree-masked GQA attention on the 5th-generation tensor cores: TMA -> shared memory -> tcgen05.mma
// with accumulators in tensor memory (TMEM).  Persistent, stream-K over key tiles.
//
// Work.  An item is (sequence b, KV head h, row block rb): up to 256 rows (two blocks of 128; row r
// <-> tree node r / G, query head h*G + r % G) against the ceil((L_b+T_b)/128) key tiles of b, so every
// K/V byte crosses HBM once for all rows that need it.  A tile of an item costs kW2 units if it carries
// two 128-row blocks and kW1 if one.  Items are laid end to end, ordered (b, h, rb); the resulting unit axis is
// cut into gridDim.x equal ranges, one per CTA (one CTA per SM), and a tile belongs to the CTA whose
// range holds its first unit.  A CTA therefore works through a few segments (item, tile range); a
// segment that covers its whole item writes the final rows, any other writes a partial (row max, row
// sum, un-normalised O) into one of the CTA's two workspace slots and records the item in the slot's
// descriptor, and merge_streamk_kernel combines the partials of an item.  When a CTA's range would be
// short (fewer than kStreamMinTiles tiles) a segment switch (results out, pipeline refill) is not
// amortised; the cut then falls back to whole pieces: every item is divided into equal pieces of
// about that length and each CTA takes exactly one piece, provided there are no more pieces than
// CTAs.  Either cut is a pure function of (seq_len, tree_size, gridDim.x), recomputed on the device
// by every CTA and by the merge kernel: no communication, no atomics on floats, no waiting between
// CTAs, bit-reproducible results for a given GPU model.
//
// Three kernels share this schedule, the TMA / tcgen05 / TMEM mechanics and the merge kernel:
//   attn_tc_kernel       one CTA per SM holds both 128-row halves of an item (below);
//   attn_tc_pair_kernel  a cluster of two CTAs, tcgen05.mma.cta_group::2 over the 256 rows, the K/V tile split
//                        between the two shared memories (the default when a KV head carries more than 256 rows);
//   attn_tc_rb_kernel    one 128-row block per CTA, partner CTAs fetch the same tiles and share them through L2
//                        (the default otherwise).
// A worker of the cut is a CTA in the first kernel and the CTA pair (2w, 2w+1) in the other two.
//
// Warp roles inside a CTA of attn_tc_kernel:
//   warp 0      TMA producer: K and V tiles (two 64-column boxes each, 128-byte swizzle) into a
//               5-slot ring of 32 KB buffers, one mbarrier pair (full / empty) per slot; the ring runs
//               ahead across segment boundaries
//   warp 1      MMA issuer: S = Q K^T (8 x m128 n128 k16, both operands from shared memory) and
//               O += P V (8 x m128 n128 k16, P from TMEM, V as an MN-major operand); owns TMEM
//   warps 2-3   Q stagers: fetch the item's Q rows into shared memory (by TMA when H_q / H_kv divides 128, else
//               16-byte asynchronous copies, swizzled, K-major); for the next segment they do so as soon as the
//               current segment's last Q K^T has completed (the MMA issuer commits a barrier right behind it)
//   warps 4-7   softmax of row block 0: thread i <-> TMEM lane i <-> row i; write results
//   warps 8-11  softmax of row block 1
// Every mbarrier wait is bounded: on a timeout the kernel sets GRAFT_FLAG_WAIT_TIMEOUT, stops
// waiting anywhere in the CTA, drains its outstanding copies, frees TMEM and returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <math_constants.h>
#include <stdlib.h>
#include <climits>
#include <type_traits>
#include "graft_internal.cuh"

namespace {

constexpr int BR = 256;          // rows per item (two blocks of 128)
constexpr int BN = 128;          // keys per tile
constexpr int D = 128;
constexpr int NSLOT = 5;         // ring slots of 32 KB (one K or V tile each)
constexpr int TILE_BYTES = BN * D * 2;
constexpr int HALF_BYTES = TILE_BYTES / 2;    // one 64-column box
constexpr int NTHREADS = 384;
constexpr int SMEM_DYN = 2 * TILE_BYTES + NSLOT * TILE_BYTES + 1024;   // Q (2 blocks) + ring + alignment slack
constexpr int MAXSEG = 16;       // segments planned per round
constexpr int kW2 = 5, kW1 = 4;        // cost units of a tile that carries two / one 128-row blocks (measured ratio ~1.25)
constexpr int kOvh = 6 * kW2;          // units charged to the start of every item: new Q, pipeline refill, results of the last one
                                       // cost a worker about as much as six tiles (measured: workers with an item boundary finished 5-8 us late)
constexpr int kStreamMinTiles = 64;   // shorter per-CTA ranges use one piece per CTA instead of stream-K
constexpr size_t SLOT_FLOATS = (size_t)BR * (D + 2);   // O[BR][D], then m2[BR], then l[BR]
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.0f;     // log2 units
constexpr long long kWaitCycles = 1ll << 31;  // about a second

// Workspace after the header: slot descriptors (2 ints per CTA), then the cut of this call (written by
// CTA 0 for the merge kernel: one CutHeader, one SeqEntry per sequence), then the partial slots.
constexpr size_t kDescBytes = 2048;
struct CutHeader { long long per; int pieces; int pad; };
struct SeqEntry { long long base; int L, T, nrb, ntiles, wlast, pad; };
// arrival counters of the in-kernel merge: one per (sequence, KV head, row block < 8, 128-row half)
__host__ __device__ constexpr size_t counter_bytes(int B, int Hkv) { return ((size_t)B * Hkv * 16 * sizeof(int) + 255) / 256 * 256; }
__host__ __device__ constexpr size_t cut_bytes(int B) { return (sizeof(CutHeader) + (size_t)B * sizeof(SeqEntry) + 255) / 256 * 256; }

struct TcArgs {
    graft_attn_params p;
    int* desc;          // [2 * grid] item id held by each partial slot of this call, -1 if none
    CutHeader* cut;     // this call's cut, followed by B SeqEntry records
    float* partial;     // 2 slots per CTA
    int* counters;      // [B * Hkv * 8 * 2] arrivals per (item, 128-row half) for the in-kernel merge: (epoch << 8) | count
    unsigned epoch;     // number of this call (24 bits): stale counts of earlier calls are ignored; every kernel reads it from call_no
    unsigned* call_no;  // [0] number of the last finished call on this workspace, [1] CTAs of the running call that are done
    int inkernel;       // the kernel merges the parts of an item itself (last arrival); else merge_streamk_kernel follows
    int single;         // row-block kernel: every item has one 128-row block (T_max * G <= 128), so every CTA is a worker of its own
    int G;
    int q_tma;          // Q tiles are fetched by TMA (group size divides 128); otherwise threads copy them
    int prof_cta;       // experiments: CTA whose timeline is recorded
};

// barrier indices: ring slots; S ready / P ready per row block; Q staged; O final; Q no longer needed
enum { BAR_FULL = 0, BAR_EMPTY = NSLOT, BAR_S = 2 * NSLOT, BAR_P = 2 * NSLOT + 2, BAR_Q = 2 * NSLOT + 4, BAR_O = 2 * NSLOT + 5,
       BAR_QFREE = 2 * NSLOT + 6, BAR_COUNT = 2 * NSLOT + 7 };

// ---------------------------------------------------------------------------------------------------
// schedule: items laid end to end, cut into equal tile ranges
// ---------------------------------------------------------------------------------------------------
struct SeqInfo {
    int b, L, T, nrb, ntiles;
    int wlast;           // cost units per tile of the last row block (kW1 or kW2); the others cost kW2
    long long base;      // position of the sequence's first item on the cut axis
    bool found;
};

// Quotient of two non-negative 64-bit numbers; nearly always both fit 32 bits, and the 64-bit division is a routine of
// a hundred-odd instructions on the one thread that plans.
__device__ __forceinline__ long long udiv(long long a, long long b) {
    if ((((unsigned long long)a | (unsigned long long)b) >> 32) == 0) return (long long)((unsigned)a / (unsigned)b);
    return a / b;
}
__device__ __forceinline__ void seq_shape(const graft_attn_params& p, int G, int b, int& L, int& T, int& nrb, int& ntiles, int& wlast) {
    L = p.seq_len[b];
    T = p.tree_size[b];
    if (T < 0 || T > p.T_max || L < 0 || (long long)L + T > (long long)p.S_cap) { L = 0; T = 0; }   // invalid: no work
    ntiles = T > 0 ? (L + T + BN - 1) / BN : 0;
    nrb = (T * G + BR - 1) / BR;
    wlast = (T * G - (nrb - 1) * BR > 128) ? kW2 : kW1;
}
// units of one KV head of a sequence
__device__ __forceinline__ long long head_units(int ntiles, int nrb, int wlast) {
    return nrb > 0 ? (long long)ntiles * (kW2 * (nrb - 1) + wlast) + (long long)nrb * kOvh : 0;
}

// An item of ntiles tiles in pieces of about `per` tiles: nsplit equal, non-empty pieces of plen tiles.
__device__ __forceinline__ void piece_shape(int ntiles, long long per, int& nsplit, int& plen) {
    nsplit = plen = 0;
    if (ntiles <= 0) return;
    long long want = udiv(ntiles, per);
    if (want < 1) want = 1;
    plen = (int)udiv(ntiles + want - 1, want);
    nsplit = (ntiles + plen - 1) / plen;
}

// Warp-cooperative scan over the sequences.  The cut axis counts units (per_piece == 0, stream-K cut) or
// pieces (per_piece > 0, one-piece-per-CTA cut with pieces of about per_piece tiles).  Returns the
// sequence whose interval holds `g` (want_b < 0) or sequence want_b; `total` receives the axis length,
// `total_tiles` the number of tiles of the batch.
__device__ __forceinline__ SeqInfo scan_sequences(const graft_attn_params& p, int G, long long g, int want_b, long long& total,
                                                  long long& total_tiles, long long per_piece, SeqEntry* table = nullptr) {
    const int lane = threadIdx.x & 31;
    SeqInfo out;
    out.found = false;
    out.b = out.L = out.T = out.nrb = out.ntiles = out.wlast = 0;
    out.base = 0;
    long long run = 0, tiles = 0;
    for (int b0 = 0; b0 < p.B; b0 += 32) {
        const int b = b0 + lane;
        int L = 0, T = 0, nrb = 0, ntiles = 0, wlast = 1;
        if (b < p.B) seq_shape(p, G, b, L, T, nrb, ntiles, wlast);
        long long cnt = (long long)p.Hkv * head_units(ntiles, nrb, wlast);
        if (per_piece > 0) {
            int nsplit, plen;
            piece_shape(ntiles, per_piece, nsplit, plen);
            cnt = (long long)p.Hkv * nrb * nsplit;
        }
        tiles += (long long)p.Hkv * nrb * ntiles;
        long long incl = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const long long v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        const long long start = run + incl - cnt;
        if (table && b < p.B) {
            SeqEntry e;
            e.base = start; e.L = L; e.T = T; e.nrb = nrb; e.ntiles = ntiles; e.wlast = wlast; e.pad = 0;
            table[b] = e;
        }
        const bool hit = b < p.B && !out.found && (want_b >= 0 ? b == want_b : (cnt > 0 && g >= start && g < start + cnt));
        const unsigned m = __ballot_sync(0xffffffffu, hit);
        if (m) {
            const int src = __ffs(m) - 1;
            out.found = true;
            out.b = b0 + src;
            out.L = __shfl_sync(0xffffffffu, L, src);
            out.T = __shfl_sync(0xffffffffu, T, src);
            out.nrb = __shfl_sync(0xffffffffu, nrb, src);
            out.ntiles = __shfl_sync(0xffffffffu, ntiles, src);
            out.wlast = __shfl_sync(0xffffffffu, wlast, src);
            out.base = __shfl_sync(0xffffffffu, start, src);
        }
        run += __shfl_sync(0xffffffffu, incl, 31);
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) tiles += __shfl_xor_sync(0xffffffffu, tiles, o);
    total = run;
    total_tiles = tiles;
    return out;
}

// The cut of a batch over `grid` CTAs (warp-cooperative).  pieces = false: stream-K, `per` units per CTA
// out of `total`; pieces = true: one piece of about `per` tiles per CTA.
__device__ __forceinline__ void choose_cut(const graft_attn_params& p, int G, int grid, long long& total, long long& per, bool& pieces,
                                           CutHeader* record = nullptr) {
    SeqEntry* table = record ? reinterpret_cast<SeqEntry*>(record + 1) : nullptr;
    long long tiles;
    (void)scan_sequences(p, G, 0, -1, total, tiles, 0, table);
    const long long per_tiles = udiv(tiles + grid - 1, grid) > 0 ? udiv(tiles + grid - 1, grid) : 1;
    pieces = false;
    per = udiv(total + grid - 1, grid);
    if (per < kW2) per = kW2;   // a range never shorter than the heaviest tile, so every CTA inside an item's span owns a tile
    if (per_tiles < kStreamMinTiles) {
        long long units, dummy;
        (void)scan_sequences(p, G, 0, -1, units, dummy, per_tiles, nullptr);
        if (units <= grid) {
            pieces = true;
            per = per_tiles;
            if (table) (void)scan_sequences(p, G, 0, -1, units, dummy, per_tiles, table);   // bases on the piece axis
        }
    }
    if (record && (threadIdx.x & 31) == 0) { record->per = per; record->pieces = pieces ? 1 : 0; record->pad = 0; }
}

// position and weight of item (h, rb) of a sequence on the unit axis
__device__ __forceinline__ void item_span(const SeqInfo& si, int h, int rb, long long& U, int& w) {
    U = si.base + (long long)h * head_units(si.ntiles, si.nrb, si.wlast) + (long long)rb * ((long long)si.ntiles * kW2 + kOvh);
    w = rb < si.nrb - 1 ? kW2 : si.wlast;
}
// An item that starts at unit U: tile 0 owns the kOvh start-up units and its own w, tile t >= 1 starts at U + kOvh + t * w.
// Number of tiles whose first unit lies below g.
__device__ __forceinline__ long long tiles_below(long long g, long long U, int w) {
    if (g <= U) return 0;
    const long long a = g - U - kOvh;
    const long long c = a > 0 ? udiv(a + w - 1, w) : 0;
    return c < 1 ? 1 : c;
}
__device__ __forceinline__ int item_id(const graft_attn_params& p, int b, int h, int rb) { return ((b * p.Hkv + h) << 3) | rb; }
// what a slot descriptor holds: the item, stamped with the call's number, so that a descriptor left by an earlier call
// (a worker that has not yet reset its own in this call) never matches
__device__ __forceinline__ int item_tag(const TcArgs& a, int id) { return id | (int)((a.epoch & 0x7fu) << 24); }
// The number of a call lives in the workspace, not in a kernel argument, so that a captured launch can be
// replayed: every CTA of the attention kernel takes "last finished call + 1" on entry, and the last CTA to
// leave publishes it (the merge kernel, which runs after the whole grid, reads it back).
__device__ __forceinline__ unsigned next_call_no(const TcArgs& a) {
    const unsigned e = (__ldcg(a.call_no) + 1u) & 0xffffffu;
    return e ? e : 1u;
}
__device__ __forceinline__ void cta_leaves(const TcArgs& a) {          // one thread per CTA, after the CTA's last use of the number
    __threadfence();
    if (atomicAdd(a.call_no + 1, 1u) == gridDim.x - 1) {
        a.call_no[1] = 0u;
        __threadfence();
        atomicExch(a.call_no, a.epoch);
    }
}

struct Seg {
    int b, h, rb;            // item
    int tile_lo, tile_hi;    // tiles [lo, hi) of the item
    int L, T;
    int slot;                // partial slot, or -1: the segment covers the whole item and writes final rows
    int c_first, c_span;     // the workers c_first .. c_first + c_span - 1 may hold parts of the item (slot descriptors tell)
    int nparts;              // how many of them do
};

// ---------------------------------------------------------------------------------------------------
// per-worker plan: a worker (a CTA, or a pair of CTAs) owns a range of the cut axis and walks it in rounds
// ---------------------------------------------------------------------------------------------------
struct Plan {
    Seg seg[MAXSEG];
    long long gnext, ghi;    // stream-K: next unit to plan, end of the worker's range
    long long per;           // units per worker (stream-K) or tiles per piece
    int nseg, npartial;
};

// Fills pl.seg with the next <= MAXSEG segments of the unit range [g, g_hi) (warp-cooperative).  A tile
// belongs to the range that holds its first unit.  Partial results go to slots 2*worker and 2*worker + 1.
__device__ __forceinline__ void plan_round(const TcArgs& a, int G, int worker, bool write_desc, Plan& pl, long long g, long long g_hi) {
    const graft_attn_params& p = a.p;
    const int lane = threadIdx.x & 31;
    int n = 0;
    int n_partial = pl.npartial;
    while (g < g_hi && n < MAXSEG) {
        long long total, tiles;
        const SeqInfo si = scan_sequences(p, G, g, -1, total, tiles, 0);
        if (!si.found) { g = g_hi; break; }
        const long long hu = head_units(si.ntiles, si.nrb, si.wlast);
        const long long seq_end = si.base + (long long)p.Hkv * hu;
        // walk the items of this sequence from the one that holds unit g
        int h = (int)udiv(g - si.base, hu);
        const long long rem = (g - si.base) - (long long)h * hu;
        int rb = (int)udiv(rem, (long long)si.ntiles * kW2 + kOvh);
        if (rb > si.nrb - 1) rb = si.nrb - 1;
        while (g < g_hi && g < seq_end && n < MAXSEG) {
            long long U;
            int w;
            item_span(si, h, rb, U, w);
            const long long item_end = U + kOvh + (long long)si.ntiles * w;
            long long t_lo = tiles_below(g, U, w), t_hi = tiles_below(g_hi, U, w);
            if (t_hi > si.ntiles) t_hi = si.ntiles;
            if (t_lo < t_hi) {
                const bool whole = t_lo == 0 && t_hi == si.ntiles;
                if (lane == 0) {
                    Seg sg;
                    sg.b = si.b;
                    sg.h = h;
                    sg.rb = rb;
                    sg.tile_lo = (int)t_lo;
                    sg.tile_hi = (int)t_hi;
                    sg.L = si.L;
                    sg.T = si.T;
                    sg.slot = whole ? -1 : 2 * worker + (n_partial < 1 ? n_partial : 1);
                    // the workers whose ranges hold a tile of this item
                    const long long per = pl.per;
                    const long long last = si.ntiles > 1 ? U + kOvh + (long long)(si.ntiles - 1) * w : U;
                    sg.c_first = (int)udiv(U, per);
                    sg.c_span = (int)udiv(last, per) - sg.c_first + 1;
                    sg.nparts = 0;
                    for (int c = sg.c_first; a.inkernel && c < sg.c_first + sg.c_span; ++c) {
                        long long lo = tiles_below(c * per, U, w), hi = tiles_below((c + 1) * per, U, w);
                        if (hi > si.ntiles) hi = si.ntiles;
                        if (lo < hi) ++sg.nparts;
                    }
                    pl.seg[n] = sg;
                    if (!whole && write_desc) a.desc[sg.slot] = item_tag(a, item_id(p, si.b, h, rb));
                }
                if (!whole) ++n_partial;
                ++n;
            }
            g = item_end < g_hi ? item_end : g_hi;
            if (++rb == si.nrb) { rb = 0; ++h; }
        }
    }
    if (lane == 0) { pl.nseg = n; pl.gnext = g; pl.npartial = n_partial; }
}

// The worker's share of the batch and its first round (warp-cooperative).  `record`: this worker writes
// the cut for the merge kernel.
__device__ __forceinline__ void plan_first(const TcArgs& a, int G, int worker, int nworkers, bool record, bool write_desc, Plan& pl) {
    const graft_attn_params& p = a.p;
    const int lane = threadIdx.x & 31;
    long long total, per;
    bool pieces;
    choose_cut(p, G, nworkers, total, per, pieces, record ? a.cut : nullptr);
    if (lane == 0) {
        pl.npartial = 0;
        pl.per = per;
        if (write_desc) {
            a.desc[2 * worker] = -1;           // this call's slot descriptors
            a.desc[2 * worker + 1] = -1;
        }
    }
    __syncwarp();
    if (pieces) {
        // exactly one piece of one item for this worker
        long long units, tiles;
        const SeqInfo si = scan_sequences(p, G, worker, -1, units, tiles, per);
        if (lane == 0) {
            pl.nseg = 0;
            pl.gnext = pl.ghi = 0;
            if (si.found) {
                int nsplit, plen;
                piece_shape(si.ntiles, per, nsplit, plen);
                const int local = (int)(worker - si.base);
                const int k = local / nsplit, sp = local % nsplit;
                Seg sg;
                sg.b = si.b;
                sg.h = k / si.nrb;
                sg.rb = k % si.nrb;
                sg.tile_lo = sp * plen;
                sg.tile_hi = min(si.ntiles, sg.tile_lo + plen);
                sg.L = si.L;
                sg.T = si.T;
                sg.slot = nsplit == 1 ? -1 : 2 * worker;
                sg.c_first = worker - sp;
                sg.c_span = sg.nparts = nsplit;
                if (nsplit > 1 && write_desc) a.desc[sg.slot] = item_tag(a, item_id(p, sg.b, sg.h, sg.rb));
                pl.seg[0] = sg;
                pl.nseg = 1;
            }
        }
    } else {
        long long g_lo = per * worker;
        long long g_hi = g_lo + per;
        if (g_hi > total) g_hi = total;
        if (g_lo > total) g_lo = total;
        if (lane == 0) pl.ghi = g_hi;
        plan_round(a, G, worker, write_desc, pl, g_lo, g_hi);
    }
}

// ---------------------------------------------------------------------------------------------------
// PTX helpers
// ---------------------------------------------------------------------------------------------------
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

__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, int w, int v, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(w), "r"(v), "r"(bar) : "memory");
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
// 32-byte global store (needs a 32-byte aligned address)
__device__ __forceinline__ void st_global_v8(void* ptr, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t a4,
                                             uint32_t a5, uint32_t a6, uint32_t a7) {
    asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(ptr), "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(a4),
                 "r"(a5), "r"(a6), "r"(a7) : "memory");
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

// instruction descriptors of kind::f16: fp32 accumulate, bf16 A and B, M = 128, N = 128
constexpr uint32_t kIdescBase = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t kIdescQK = kIdescBase;                // A, B both K-major
constexpr uint32_t kIdescPV = kIdescBase | (1u << 16);   // B (= V) MN-major

// ---------------------------------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(NTHREADS, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap vmap, const __grid_constant__ CUtensorMap qmap,
               TcArgs a, unsigned* status) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t s_bar[BAR_COUNT];
    __shared__ uint32_t s_tmem;
    __shared__ int s_abort;
    __shared__ Plan s_plan;
    Seg* const s_seg = s_plan.seg;
    int& s_nseg = s_plan.nseg;

    const graft_attn_params& p = a.p;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = a.G;
#ifdef GRAFT_TC_EXPERIMENTS
    const long long t_entry = clock64();
    const bool prof = blockIdx.x == a.prof_cta && threadIdx.x == 128;
#define STAMP(i) do { if (prof) status[16 + (i)] = (unsigned)(clock64() - t_entry); } while (0)
#else
#define STAMP(i) do { } while (0)
#endif

    const uint32_t sQ = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sRing = sQ + 2 * TILE_BYTES;
    const uint32_t bar0 = smem_u32(s_bar);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    volatile int* abort_flag = &s_abort;

    // Q rows of an item into shared memory, K-major with the 128-byte swizzle (16-byte chunk c of row r at
    // c ^ (r & 7)), by `nthr` threads numbered tid = 0 .. nthr-1; 16 independent global loads per thread and round
    auto stage_q = [&](const Seg& sg, int tid, int nthr) {
        const int R = sg.T * G;
        const int row0 = sg.rb * BR;
        const __nv_bfloat16* Qg = reinterpret_cast<const __nv_bfloat16*>(p.Q) + (size_t)sg.b * p.q_stride_b +
                                  (size_t)sg.h * G * p.q_stride_h;
        // asynchronous 16-byte copies, all in flight at once: the loads queue behind the K/V stream in a
        // saturated memory system, so their latency must overlap rather than add up
        const int step = nthr >> 4;              // rows per pass: 16 threads copy one 256-byte row
        const int ch = tid & 15;
        int r = row0 + (tid >> 4);
        int g = r % G;
        const int dt = step / G, dg = step - dt * G;
        const __nv_bfloat16* src_t = Qg + (size_t)(r / G) * p.q_stride_t + ch * 8;       // row of tree node t, head g = 0
        const size_t inc_t = (size_t)dt * p.q_stride_t;
        for (int qr = tid >> 4; qr < BR; qr += step) {
            const bool valid = r < R;
            const __nv_bfloat16* src = valid ? src_t + (size_t)g * p.q_stride_h : Qg;
            const int rr = qr & 127;
            const uint32_t dst = sQ + (qr >> 7) * TILE_BYTES + (ch >> 3) * HALF_BYTES + rr * 128 + (((ch & 7) ^ (rr & 7)) << 4);
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(valid ? 16 : 0) : "memory");   // rows past the tree read as zero
            r += step;
            g += dg;
            src_t += inc_t;
            if (g >= G) { g -= G; src_t += p.q_stride_t; }
        }
        asm volatile("cp.async.wait_all;" ::: "memory");
        fence_async_smem();
    };

    // The same Q rows by TMA (one thread): the map's box is 64 columns x G heads x 128/G tree nodes, which lands
    // as 128 rows r = t*G + g in the swizzled K-major layout.  Rows of tree nodes past the sequence's tree hold
    // whatever the caller's buffer holds there (zero past T_max); their scores stay in their own accumulator
    // rows and are never written out.  The expect_tx is one of the two arrivals of the barrier.
    auto issue_q = [&](const Seg& sg) {
        const int row0 = sg.rb * BR;
        const int nblk = (sg.T * G - row0 > 128) ? 2 : 1;
        mbar_expect_tx(bar(BAR_Q), nblk * TILE_BYTES);
        for (int blk = 0; blk < nblk; ++blk)
            for (int half = 0; half < 2; ++half)
                tma_load_5d(sQ + blk * TILE_BYTES + half * HALF_BYTES, &qmap, half * 64, 0, (row0 + blk * 128) / G, sg.h, sg.b, bar(BAR_Q));
    };

    asm volatile("griddepcontrol.wait;" ::: "memory");       // launched as a programmatic dependent: the kernel before this one is complete from here on
    a.epoch = next_call_no(a);
    if (warp == 0) plan_first(a, G, (int)blockIdx.x, (int)gridDim.x, blockIdx.x == 0, true, s_plan);
    if (threadIdx.x == 0) s_abort = 0;
    __syncthreads();
    if (s_nseg == 0) {                            // nothing for this CTA (short batch)
        if (threadIdx.x == 0) cta_leaves(a);
        return;
    }
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");      // the merge kernel may be set up from now on (it waits for this grid to end)

    // ring load n of a segment's tile t: K (which = 0) or V (which = 1)
    auto issue_load = [&](const Seg& sg, int t, int which, int n) {
        const int slot = n % NSLOT;
        const uint32_t dst = sRing + slot * TILE_BYTES;
        const CUtensorMap* map = which ? &vmap : &kmap;
        mbar_expect_tx(bar(BAR_FULL + slot), TILE_BYTES);
        tma_load_4d(dst, map, 0, t * BN, sg.h, sg.b, bar(BAR_FULL + slot));
        tma_load_4d(dst + HALF_BYTES, map, 64, t * BN, sg.h, sg.b, bar(BAR_FULL + slot));
    };
    int n_prefetched = 0;      // producer thread: ring loads already issued here, before Q is staged
    if (threadIdx.x == 0) {
        for (int i = 0; i < NSLOT; ++i) { mbar_init(bar(BAR_FULL + i), 1); mbar_init(bar(BAR_EMPTY + i), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(bar(BAR_S + i), 1); mbar_init(bar(BAR_P + i), 4); }
        mbar_init(bar(BAR_Q), 2);                  // the two stager warps
        mbar_init(bar(BAR_O), 1);
        mbar_init(bar(BAR_QFREE), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (a.q_tma) issue_q(s_seg[0]);
        // fill the ring at once: these copies overlap the staging of Q below
        for (int si = 0; si < s_nseg && n_prefetched < NSLOT; ++si) {
            const Seg sg = s_seg[si];
            for (int t = sg.tile_lo; t < sg.tile_hi && n_prefetched < NSLOT; ++t)
                for (int which = 0; which < 2 && n_prefetched < NSLOT; ++which, ++n_prefetched) issue_load(sg, t, which, n_prefetched);
        }
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (!a.q_tma) stage_q(s_seg[0], threadIdx.x, NTHREADS);      // the first segment's Q, by everyone
    STAMP(0);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    STAMP(1);

    // running counters that persist across segments and rounds (each role keeps its own copy)
    int n_load = 0;            // ring loads issued / consumed so far (2 per tile)
    int jt[2] = {0, 0};        // tiles processed so far by row block 0 / 1 (S and P barrier phases)
    int n_seg_done = 0;        // segments finished (Q and O barrier phases)

    for (;;) {                 // rounds of <= MAXSEG segments
        const int nseg = s_nseg;

        if (warp == 0) {
            // =============================== TMA producer ===============================
            if (lane == 0) {
                for (int si = 0; si < nseg; ++si) {
                    const Seg sg = s_seg[si];
                    for (int t = sg.tile_lo; t < sg.tile_hi; ++t)
                        for (int which = 0; which < 2; ++which, ++n_load) {
                            if (n_load < n_prefetched) continue;          // issued before Q was staged
                            const int slot = n_load % NSLOT, use = n_load / NSLOT;
                            if (use > 0) mbar_wait(bar(BAR_EMPTY + slot), (use - 1) & 1, abort_flag, status);
                            issue_load(sg, t, which, n_load);
                        }
                }
            }
        } else if (warp == 1) {
            // =============================== MMA issuer ===============================
            if (lane == 0) {
                auto wait_full = [&](int n) { mbar_wait(bar(BAR_FULL + n % NSLOT), (n / NSLOT) & 1, abort_flag, status); };
                for (int si = 0; si < nseg; ++si) {
                    const Seg sg = s_seg[si];
                    const int nt = sg.tile_hi - sg.tile_lo;
                    const int nblk = (sg.T * G - sg.rb * BR > 128) ? 2 : 1;
                    // S[blk] = Q[blk] K^T with the K tile of ring load n
                    auto issue_qk = [&](int blk, int n) {
                        const uint32_t sK16 = (sRing + (n % NSLOT) * TILE_BYTES) >> 4;
                        const uint32_t sQ16 = (sQ + blk * TILE_BYTES) >> 4;
#pragma unroll
                        for (int k = 0; k < D / 16; ++k) {
                            const uint32_t off16 = ((k >> 2) * HALF_BYTES + (k & 3) * 32) >> 4;
                            mma_ss(tmem + blk * 128, smem_desc(kDescKMajor, sQ16 + off16), smem_desc(kDescKMajor, sK16 + off16), kIdescQK, k > 0);
                        }
                        tc_commit(bar(BAR_S + blk));
                        if (blk == nblk - 1) tc_commit(bar(BAR_EMPTY + n % NSLOT));          // K tile fully read
                    };
                    // O[blk] (+)= P[blk] V with the V tile of ring load n
                    auto issue_pv = [&](int blk, int n, bool first) {
                        const uint32_t sV16 = (sRing + (n % NSLOT) * TILE_BYTES) >> 4;
#pragma unroll
                        for (int k = 0; k < BN / 16; ++k)
                            mma_ts(tmem + 256 + blk * 128, tmem + blk * 128 + k * 8, smem_desc(kDescVMajor, sV16 + k * (2048 >> 4)), kIdescPV,
                                   (!first || k > 0) ? 1u : 0u);
                        if (blk == nblk - 1) tc_commit(bar(BAR_EMPTY + n % NSLOT));          // V tile fully read
                    };
                    mbar_wait(bar(BAR_Q), n_seg_done & 1, abort_flag, status);                // Q of this segment staged
                    wait_full(n_load);
                    tc_fence_after();
                    for (int blk = 0; blk < nblk; ++blk) issue_qk(blk, n_load);
                    if (nt == 1) tc_commit(bar(BAR_QFREE));          // the segment's last Q K^T is in the pipe
                    for (int j = 0; j < nt; ++j) {
                        const int nV = n_load + 2 * j + 1, nK1 = n_load + 2 * j + 2;
                        for (int blk = 0; blk < nblk; ++blk) {
                            mbar_wait(bar(BAR_P + blk), (jt[blk] + j) & 1, abort_flag, status);
#ifdef GRAFT_TC_EXPERIMENTS
                            if (blockIdx.x == a.prof_cta && n_seg_done == 0 && j < 2) status[40 + j * 8 + blk * 4 + 0] = (unsigned)(clock64() - t_entry);
#endif
                            if (blk == 0) wait_full(nV);
#ifdef GRAFT_TC_EXPERIMENTS
                            if (blockIdx.x == a.prof_cta && n_seg_done == 0 && j < 2) status[40 + j * 8 + blk * 4 + 1] = (unsigned)(clock64() - t_entry);
#endif
                            tc_fence_after();
                            issue_pv(blk, nV, j == 0);
                            if (j + 1 < nt) {
                                if (blk == 0) { wait_full(nK1); tc_fence_after(); }
#ifdef GRAFT_TC_EXPERIMENTS
                                if (blockIdx.x == a.prof_cta && n_seg_done == 0 && j < 2) status[40 + j * 8 + blk * 4 + 2] = (unsigned)(clock64() - t_entry);
#endif
                                issue_qk(blk, nK1);
#ifdef GRAFT_TC_EXPERIMENTS
                                if (blockIdx.x == a.prof_cta && n_seg_done == 0 && j < 2) status[40 + j * 8 + blk * 4 + 3] = (unsigned)(clock64() - t_entry);
#endif
                                if (blk == nblk - 1 && j + 2 == nt) tc_commit(bar(BAR_QFREE));
                            }
                        }
                    }
                    tc_commit(bar(BAR_O));
                    n_load += 2 * nt;
                    for (int blk = 0; blk < nblk; ++blk) jt[blk] += nt;
                    ++n_seg_done;
                }
            }
        } else if (warp == 2 || warp == 3) {
            // =============================== Q stagers ===============================
            for (int si = 0; si < nseg; ++si) {
                const Seg sg = s_seg[si];
                // Q may be overwritten once the previous segment's last Q K^T is complete (one phase per segment)
                if (n_seg_done > 0) mbar_wait(bar(BAR_QFREE), (n_seg_done - 1) & 1, abort_flag, status);
                if (a.q_tma) {
                    // the very first segment's copy was issued (and one arrival made) by thread 0 at start-up
                    if (lane == 0) {
                        if (warp == 3) mbar_arrive(bar(BAR_Q));
                        else if (n_seg_done > 0) issue_q(sg);
                    }
                } else {
                    if (n_seg_done > 0) stage_q(sg, threadIdx.x - 64, 64);      // the first segment's Q was staged by all warps
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(BAR_Q));
                }
                ++n_seg_done;
            }
        } else if (warp >= 4) {
            // =============================== softmax, results ===============================
            const int blk = (warp - 4) >> 2;
            const int rl = ((warp & 3) << 5) + lane;            // row inside the block = TMEM lane
            const uint32_t lane_bits = (uint32_t)((warp & 3) << 5) << 16;
            const uint32_t tS = tmem + lane_bits + blk * 128;
            const uint32_t tO = tmem + lane_bits + 256 + blk * 128;
            const float sl2 = p.scale * kLog2e;
            for (int si = 0; si < nseg; ++si) {
                const Seg sg = s_seg[si];
                const int nt = sg.tile_hi - sg.tile_lo;
                const int R = sg.T * G;
                const int row0 = sg.rb * BR;
                const int nblk = (R - row0 > 128) ? 2 : 1;
                const int n_keys = sg.L + sg.T;

                if (blk < nblk) {
                    const int r = row0 + blk * 128 + rl;
                    const bool row_valid = r < R;
                    const int t = row_valid ? r / G : 0, g = row_valid ? r % G : 0;
                    const unsigned long long anc = row_valid ? p.tree_anc[(size_t)sg.b * p.T_max + t] : 0ull;
                    const unsigned long long allowed = sg.T >= 64 ? anc : (anc & ((1ull << sg.T) - 1ull));
                    float m_ref = -CUDART_INF_F, l = 0.f;

                    for (int j = 0; j < nt; ++j) {
                        const int key0 = (sg.tile_lo + j) * BN;
                        const bool boundary = key0 + BN > sg.L;
                        mbar_wait(bar(BAR_S + blk), (jt[blk] + j) & 1, abort_flag, status);
                        tc_fence_after();
                        if (j == 0) STAMP(3 + 8 * min(si, 1));
                        if (j == 1) STAMP(4 + 8 * min(si, 1));
                        // ancestor mask and the end of the tree's keys: one 32-bit word of allowed columns per chunk
                        auto mask32 = [&](uint32_t (&x)[32], int col0) {
                            const int u0 = key0 + col0 - sg.L;         // tree index of the chunk's first column
                            uint32_t w;
                            if (u0 >= 64) w = 0u;
                            else if (u0 >= 0) w = (uint32_t)(allowed >> u0);
                            else if (u0 <= -32) w = 0xffffffffu;
                            else w = (uint32_t)((allowed << (-u0)) | ((1ull << (-u0)) - 1ull));
#pragma unroll
                            for (int q = 0; q < 32; ++q)
                                if (!((w >> q) & 1u)) x[q] = 0xff800000u;   // -inf
                        };
                        auto max32 = [&](const uint32_t (&x)[32], float& m0, float& m1) {
#pragma unroll
                            for (int q = 0; q < 32; q += 4) {
                                m0 = fmax3(m0, __uint_as_float(x[q]), __uint_as_float(x[q + 1]));
                                m1 = fmax3(m1, __uint_as_float(x[q + 2]), __uint_as_float(x[q + 3]));
                            }
                        };
                        // pass 1: row maximum of the (masked) scores, 64 columns in flight at a time
                        float mx0 = -CUDART_INF_F, mx1 = -CUDART_INF_F;
                        {
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
                        }
                        const float mx = fmaxf(mx0, mx1);
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
                        {
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
                        tmem_wait_st();
                        // last tile of the sequence: zero the V rows of slots that hold no key of this tree
                        if (blk == 0 && key0 + BN > n_keys) {
                            const int nV = n_load + 2 * j + 1;
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
                    }

                    STAMP(5 + 8 * min(si, 1));
                    // ---- results of the segment: O row from TMEM, final rows or a partial
                    mbar_wait(bar(BAR_O), n_seg_done & 1, abort_flag, status);     // every MMA of the segment is complete
                    tc_fence_after();
                    STAMP(6 + 8 * min(si, 1));
                    if (sg.slot < 0) {
                        const float inv = l > 0.f ? 1.f / l : 0.f;
                        __nv_bfloat16* orow = reinterpret_cast<__nv_bfloat16*>(p.O) + (size_t)sg.b * p.o_stride_b + (size_t)t * p.o_stride_t +
                                              (size_t)(sg.h * G + g) * p.o_stride_h;
#pragma unroll 1
                        for (int c = 0; c < 4; ++c) {
                            uint32_t v[32];
                            tmem_ld32(tO + c * 32, v);
                            tmem_wait_ld();
                            if (row_valid) {
#pragma unroll
                                for (int q = 0; q < 4; ++q) {      // 16-byte stores: O strides are only guaranteed 16-byte aligned
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
                            p.LSE[((size_t)sg.b * p.Hq + sg.h * G + g) * p.T_max + t] =
                                l > 0.f ? (m_ref * sl2 + log2f(l)) * kLn2 : -CUDART_INF_F;
                    } else {
                        float* base = a.partial + (size_t)sg.slot * SLOT_FLOATS;
                        const int lr = blk * 128 + rl;
                        float* prow = base + (size_t)lr * D;
#pragma unroll 1
                        for (int c = 0; c < 4; ++c) {
                            uint32_t v[32];
                            tmem_ld32(tO + c * 32, v);
                            tmem_wait_ld();
#pragma unroll
                            for (int q = 0; q < 4; ++q)      // 32-byte stores: every store fills a whole sector
                                st_global_v8(prow + c * 32 + q * 8, v[q * 8], v[q * 8 + 1], v[q * 8 + 2], v[q * 8 + 3], v[q * 8 + 4],
                                             v[q * 8 + 5], v[q * 8 + 6], v[q * 8 + 7]);
                        }
                        base[BR * D + lr] = m_ref == -CUDART_INF_F ? -CUDART_INF_F : m_ref * sl2;
                        base[BR * D + BR + lr] = l;
                    }
                    tc_fence_before();                 // TMEM reads done before the next segment's MMAs are released
                    STAMP(7 + 8 * min(si, 1));
#ifdef GRAFT_TC_EXPERIMENTS
                    if (prof) status[15] = (unsigned)nt;
#endif
                    jt[blk] += nt;
                }
                n_load += 2 * nt;
                ++n_seg_done;
            }
        }

        // ---- next round (only batches with very many short sequences need more than one)
        __syncthreads();
        const long long g_next = s_plan.gnext, g_hi = s_plan.ghi;
        if (g_next >= g_hi) break;
        __syncthreads();
        if (warp == 0) plan_round(a, G, (int)blockIdx.x, true, s_plan, g_next, g_hi);
        __syncthreads();
        if (s_nseg == 0) break;
    }

    // ---- teardown: every copy has landed (each was waited for by the MMA issuer); the allocating warp
    // frees the TMEM columns once everyone is past its last access
    if (warp == 0 && lane == 0 && *abort_flag)      // after a timeout some copies may still be in flight
        for (int m = max(0, n_load - NSLOT); m < n_load; ++m) {
            const long long t0 = clock64();
            while (!mbar_try_wait(bar(BAR_FULL + m % NSLOT), (m / NSLOT) & 1) && clock64() - t0 < kWaitCycles) {}
        }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
    if (threadIdx.x == 0) cta_leaves(a);
}

// Rows of padding nodes (t >= T_b; all rows of a sequence whose sizes are out of range) are zero with LSE -inf.
// The kernels that merge in place have no separate pass over the output, so all their CTAs share this job.
__device__ __forceinline__ void zero_padding_rows(const TcArgs& a, unsigned* status) {
    const graft_attn_params& p = a.p;
    const int nthr = gridDim.x * blockDim.x, me = blockIdx.x * blockDim.x + threadIdx.x;
    for (int b = 0; b < p.B; ++b) {
        int T = p.tree_size[b];
        const int L = p.seq_len[b];
        if (T < 0 || T > p.T_max || L < 0 || (long long)L + T > (long long)p.S_cap) {
            T = 0;
            if (me == 0) atomicOr(status, (unsigned)GRAFT_FLAG_BAD_SIZE);
        }
        const int chunks = D / 8;                  // 16-byte chunks per output row
        const int n = (p.T_max - T) * p.Hq * chunks;
        for (int i = me; i < n; i += nthr) {
            const int ch = i % chunks, hq = (i / chunks) % p.Hq, t = T + i / (chunks * p.Hq);
            __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(p.O) + (size_t)b * p.o_stride_b + (size_t)t * p.o_stride_t + (size_t)hq * p.o_stride_h;
            *reinterpret_cast<uint4*>(o + ch * 8) = make_uint4(0u, 0u, 0u, 0u);
            if (ch == 0 && p.LSE) p.LSE[((size_t)b * p.Hq + hq) * p.T_max + t] = -CUDART_INF_F;
        }
    }
}

// ---------------------------------------------------------------------------------------------------
// the pair kernel: two CTAs (a cluster of two SMs) share every tile
// ---------------------------------------------------------------------------------------------------
// One tcgen05.mma.cta_group::2 multiplies 256 rows at once: CTA 0 of the pair owns rows 0..127 of the item,
// CTA 1 rows 128..255, each in its own tensor memory.  The B operand is split between the two shared
// memories: of a K tile each CTA fetches 64 of the 128 keys (all of d), of a V tile all 128 keys and 64 of
// the d columns, so every byte of the cache still crosses into the pair once.  With one row block per SM
// there is room for three score buffers in tensor memory (columns 0..383, O at 384..511): Q K^T runs two
// tiles ahead of P V, so the tensor pipe never waits for the buffer that holds P of the tile in the softmax.
//
// Barriers live at the same offset in both shared memories.  Copies of both CTAs complete on the leader's
// (CTA 0's) FULL and Q barriers; the softmax warps of both arrive on the leader's P barriers; everything
// the MMA thread commits is multicast to both CTAs (slot free, S ready, O final, Q free).
//
// Measured on the 64K-context configuration (per 128-key tile and pair): the sixteen 256-row MMAs take about
// 1500 cycles with the softmax arithmetic switched off and about 1850 with it, the softmax of one tile about
// 1600; the kernel is bound by the tensor pipe in this mode.
//
// The last tile of an item is fetched at keys [L+T-128, L+T) instead of a tile-aligned position: it never
// reaches past the sequence's keys (rows before key 0 are zero-filled by the copy), and the columns that
// the previous tile already covered are masked like non-ancestors.
constexpr int P_NTHREADS = 384;          // producer, Q K^T issuer, Q loader, P V issuer, eight softmax warps
constexpr int P_HALF_TILE = TILE_BYTES / 2;       // this CTA's half of a K tile or of a V tile
constexpr int P_SLOT_BYTES = 2 * P_HALF_TILE;     // one ring slot: the K half, then the V half of a tile
constexpr int P_NSLOT = 6;
constexpr int kCtrlBytes = 1024;
constexpr int P_SMEM_DYN = kCtrlBytes + TILE_BYTES + P_NSLOT * P_SLOT_BYTES + 2048;      // control, Q (128 rows), ring, softmax exchange: 227 KB
constexpr int P_NSBUF = 3;                        // score buffers in tensor memory (128 columns each), O behind them
enum { PB_FULL = 0, PB_EMPTY = P_NSLOT, PB_S = 2 * P_NSLOT, PB_P = PB_S + P_NSBUF, PB_Q = PB_P + P_NSBUF, PB_O = PB_Q + 1,
       PB_QFREE = PB_O + 1, PB_COUNT = PB_QFREE + 1 };
struct PairCtrl {
    uint64_t bar[PB_COUNT];
    Plan plan;
    uint32_t tmem;
    int abort;
    int merge_flag;
};
static_assert(sizeof(PairCtrl) <= kCtrlBytes, "control block too large");

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of this CTA's shared-memory location `addr` as seen in CTA `cta` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t cta) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(cta));
    return r;
}
// arrival on a barrier of the pair's leader.  The plain form orders tensor-memory traffic (together with the
// tcgen05 fences on both sides); the cluster-scope release also publishes ordinary shared-memory writes, at
// the price of a full memory fence (over a thousand cycles when measured), so only the Q stagers use it.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// bounded wait on a barrier that threads of the partner CTA arrive on
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// non-blocking test; issued ahead of a run of MMAs so that its latency hides behind them
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ void mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned* status) {
    if (mbar_try_wait_cluster(bar, parity)) return;
    if (*abort_flag) return;
    const long long t0 = clock64();
    while (!mbar_try_wait_cluster(bar, parity)) {
        if (*abort_flag) return;
        if (clock64() - t0 > kWaitCycles) {
            *abort_flag = 1;
            atomicOr(status, (unsigned)GRAFT_FLAG_WAIT_TIMEOUT);
            return;
        }
    }
}
// copies whose completion is counted on a barrier of the pair's leader; K/V tiles carry an L2 eviction policy: they are
// read once, so they should leave L2 before the partials do
__device__ __forceinline__ void tma_pair_4d_hint(uint32_t dst, const CUtensorMap* map, int x, int y, int z, int w, uint32_t cluster_bar, uint64_t policy) {
    asm volatile("cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4, %5}], [%6], %7;"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(w), "r"(cluster_bar), "l"(policy) : "memory");
}
__device__ __forceinline__ void tma_pair_5d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, int w, int v, uint32_t cluster_bar) {
    asm volatile("cp.async.bulk.tensor.5d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(w), "r"(v), "r"(cluster_bar) : "memory");
}
// The eight MMAs of one tile as one run of instructions (the issuing warp shares its scheduler with two busy
// softmax warps, so every instruction it does not need is time the tensor pipe waits): descriptors advance by
// constants, 2 per 16 elements of K inside a 64-element box, `a_box` / `b_box` between the boxes (16-byte units).
__device__ __forceinline__ void mma_pair_ss8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t a_box, uint32_t b_box) {
    asm volatile(
        "{\n\t"
        ".reg .pred pT, pF;\n\t"
        ".reg .b64 da, db, ia, ib;\n\t"
        "setp.eq.b32 pT, %3, %3;\n\t"
        "setp.ne.b32 pF, %3, %3;\n\t"
        "cvt.u64.u32 ia, %4;\n\t"
        "cvt.u64.u32 ib, %5;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, pF;\n\t"
        "add.s64 da, %1, 2;\n\t add.s64 db, %2, 2;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, pT;\n\t"
        "add.s64 da, %1, 4;\n\t add.s64 db, %2, 4;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, pT;\n\t"
        "add.s64 da, %1, 6;\n\t add.s64 db, %2, 6;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, pT;\n\t"
        "add.s64 da, %1, ia;\n\t add.s64 db, %2, ib;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, pT;\n\t"
        "add.s64 da, da, 2;\n\t add.s64 db, db, 2;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, pT;\n\t"
        "add.s64 da, da, 2;\n\t add.s64 db, db, 2;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, pT;\n\t"
        "add.s64 da, da, 2;\n\t add.s64 db, db, 2;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, pT;\n\t"
        "}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(a_box), "r"(b_box) : "memory");
}
// P V: A advances by 8 tensor-memory columns, B by `b_step` (16-byte units) per 16 keys; `accumulate`: O already holds tiles
__device__ __forceinline__ void mma_pair_ts8(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t b_step, uint32_t accumulate) {
    asm volatile(
        "{\n\t"
        ".reg .pred pT, p0;\n\t"
        ".reg .b64 db, ib;\n\t"
        ".reg .b32 ta;\n\t"
        "setp.eq.b32 pT, %3, %3;\n\t"
        "setp.ne.b32 p0, %5, 0;\n\t"
        "cvt.u64.u32 ib, %4;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p0;\n\t"
        "add.u32 ta, %1, 8;\n\t add.s64 db, %2, ib;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], [ta], db, %3, pT;\n\t"
        "add.u32 ta, ta, 8;\n\t add.s64 db, db, ib;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], [ta], db, %3, pT;\n\t"
        "add.u32 ta, ta, 8;\n\t add.s64 db, db, ib;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], [ta], db, %3, pT;\n\t"
        "add.u32 ta, ta, 8;\n\t add.s64 db, db, ib;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], [ta], db, %3, pT;\n\t"
        "add.u32 ta, ta, 8;\n\t add.s64 db, db, ib;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], [ta], db, %3, pT;\n\t"
        "add.u32 ta, ta, 8;\n\t add.s64 db, db, ib;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], [ta], db, %3, pT;\n\t"
        "add.u32 ta, ta, 8;\n\t add.s64 db, db, ib;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], [ta], db, %3, pT;\n\t"
        "}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(b_step), "r"(accumulate) : "memory");
}
// arrive on the barrier at this offset in both CTAs once every MMA issued so far is complete
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((unsigned short)3) : "memory");
}
// M = 256 over the pair, N = 128
constexpr uint32_t kIdescPairBase = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((256u >> 4) << 24);
constexpr uint32_t kIdescPairQK = kIdescPairBase;
constexpr uint32_t kIdescPairPV = kIdescPairBase | (1u << 16);

// ---------------------------------------------------------------------------------------------------
// pieces shared by the kernels that keep three score buffers in tensor memory (columns 0..383) and O behind
// them (384..511)
// ---------------------------------------------------------------------------------------------------
struct SoftmaxBars {
    int S, P, O;             // barrier indices: score buffer ready (x3), P written (x3), all MMAs of the segment complete
    int pv_done, pv_mod;     // barrier whose phase tile/pv_mod of index pv_done + tile % pv_mod completes with P V of `tile`
    bool remote;             // P barriers live in CTA 0 of the cluster
    // where this CTA's part of a V tile sits in shared memory (paged caches: rows past a sequence's keys are zeroed there)
    uint32_t v_base;         // slot 0
    int v_slot_bytes, v_nslot, v_boxes, v_box_stride;
    int v_full;              // barrier that tells a V slot has landed, or -1 when the score barrier implies it
};
// first key and number of already-covered columns of tile t of an item: the last tile is fetched at keys
// [L+T-128, L+T), so it never reaches past the sequence's keys (rows before key 0 are zero-filled by the copy)
// pool block of the page that holds cache slot `key` of sequence b (paged caches); an entry outside the pool gives
// n_blocks, a coordinate past the tensor map's end that the copy fills with zeros, and raises the flag
__device__ __forceinline__ int page_block(const graft_attn_params& p, int b, int key, unsigned* status) {
    const int blk = __ldg(p.block_table + (size_t)b * p.blocks_per_seq + key / p.page_size);
    if (blk < 0 || blk >= p.n_blocks) { atomicOr(status, (unsigned)GRAFT_FLAG_BAD_SIZE); return p.n_blocks; }
    return blk;
}
// With paged caches a tile must not straddle two pages, so the last tile stays aligned; what it holds past the
// sequence's keys is masked in the scores and zeroed in the V tile before P V reads it.
__device__ __forceinline__ int tile_key0(const Seg& sg, int t, int& overlap, bool paged) {
    const int n_keys = sg.L + sg.T;
    const int ntiles = (n_keys + BN - 1) / BN;
    overlap = 0;
    if (paged || t < ntiles - 1) return t * BN;
    overlap = ntiles * BN - n_keys;
    return n_keys - BN;
}

// ---------------------------------------------------------------------------------------------------
// softmax and results of a 128-row block by two warpgroups that split the columns of every tile
// ---------------------------------------------------------------------------------------------------
// Warps w and w + 4 own the same 32 rows (tensor-memory lanes) and take columns 0..63 and 64..127 of the
// score tile, so two warps per scheduler keep the exponential unit busy and a row's 64 scores stay in
// registers between the maximum pass and the exponentials.  The half-row maxima are exchanged through
// shared memory at a 64-thread named barrier (double-buffered by tile parity), so both halves move the
// reference maximum at the same tiles; each half keeps its own part of the row sum and writes 64 output columns.
struct SplitShared {
    float mx[2][2][128];     // [tile parity][half][row]; the idle parity carries the row sums at the end of a segment
};

template <bool PAGED>
__device__ __forceinline__ void softmax_rows_split(const TcArgs& a, const Plan& plan, const SoftmaxBars lay, uint32_t bar0, uint32_t tmem, int rank,
                                             SplitShared& sh, volatile int* merge_flag, int& jt, int& n_seg_done, volatile int* abort_flag, unsigned* status) {
    const graft_attn_params& p = a.p;
    const int G = a.G;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nseg = plan.nseg;
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    const int half = (warp - 4) >> 2;                   // columns 0..63 or 64..127 of the score tile, and of O
    const int rl = ((warp & 3) << 5) + lane;            // row inside this CTA's block = TMEM lane
    const int pair_bar = 1 + (warp & 3);                // the two warps that own the same 32 rows
    auto pair_sync = [&]() { asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory"); };
    const uint32_t lane_bits = (uint32_t)((warp & 3) << 5) << 16;
    const uint32_t tO = tmem + lane_bits + P_NSBUF * 128 + half * 64;      // this thread's 64 output columns
    const float sl2 = p.scale * kLog2e;
    for (int si = 0; si < nseg; ++si) {
        const Seg sg = plan.seg[si];
        const int nt = sg.tile_hi - sg.tile_lo;
        const int R = sg.T * G;
        const int r = sg.rb * BR + (int)rank * 128 + rl;
        const bool row_valid = r < R;
        const int t = row_valid ? r / G : 0, g = row_valid ? r % G : 0;
        const unsigned long long anc = row_valid ? p.tree_anc[(size_t)sg.b * p.T_max + t] : 0ull;
        const unsigned long long allowed = sg.T >= 64 ? anc : (anc & ((1ull << sg.T) - 1ull));
        float m_ref = -CUDART_INF_F, l = 0.f;

        // Tiles that lie entirely among the cached keys need no mask at all; they come first and take the loop body
        // without the masking code (the loop is sensitive to every instruction in it), the boundary tiles the full one.
        // score buffer and barrier phase of the tile at hand: kept as running values (gt % 3 and gt / 3 cost a dozen
        // instructions each time)
        int sb = jt % P_NSBUF;
        uint32_t sph = (uint32_t)(jt / P_NSBUF) & 1u;
        const uint32_t p_bar0 = lay.remote ? map_to_cta(bar(lay.P), 0u) : bar(lay.P);
        auto one_tile = [&](int j, auto masked_tag) {
            const int gt = jt + j;
            const uint32_t tS = tmem + lane_bits + sb * 128 + half * 64;      // this thread's 64 score columns
            const uint32_t tP = tmem + lane_bits + sb * 128 + half * 32;      // its 64 P values (bf16 pairs)
            constexpr bool masked = decltype(masked_tag)::value;
            int overlap = 0;
            const int key0 = masked ? tile_key0(sg, sg.tile_lo + j, overlap, PAGED) : 0;
            mbar_wait(bar(lay.S + sb), sph, abort_flag, status);
            tc_fence_after();
            uint32_t x[2][32];
#pragma unroll
            for (int c = 0; c < 2; ++c) tmem_ld32(tS + c * 32, x[c]);
            tmem_wait_ld();
            if (masked) {
                if (PAGED) {
                    // paged caches: an item's last tile may reach past the sequence's keys
                    const int n_valid = sg.L + sg.T - key0;
                    if (n_valid < BN) {
                        // the rows of the V tile past the sequence's keys may hold anything (0 x NaN would poison O): zero them
                        if (lay.v_full >= 0) mbar_wait(bar(lay.v_full + gt % lay.v_nslot), (gt / lay.v_nslot) & 1, abort_flag, status);
                        const uint32_t vs = lay.v_base + (gt % lay.v_nslot) * lay.v_slot_bytes + (uint32_t)n_valid * 128u;
                        const int nchunk = (BN - n_valid) * 8;       // 16-byte pieces per 64-column box
                        for (int bx = 0; bx < lay.v_boxes; ++bx)
                            for (int c = (int)threadIdx.x - 128; c < nchunk; c += 256)
                                asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(vs + bx * lay.v_box_stride + c * 16), "r"(0u) : "memory");
                        fence_async_smem();
                        // the MMA that reads these rows is issued from the pair's leader after the P barrier: order the
                        // stores before this thread's (relaxed) arrival there at cluster scope
                        if (lay.remote) asm volatile("fence.acq_rel.cluster;" ::: "memory");
                    }
                }
                // per 32-column chunk one word of allowed columns: cached keys not yet covered, ancestors in the tree
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const int u0 = key0 + (half * 2 + c) * 32 - sg.L;         // tree index of the chunk's first column
                    uint32_t w;
                    if (u0 >= 64) w = 0u;
                    else if (u0 >= 0) w = (uint32_t)(allowed >> u0);
                    else if (u0 <= -32) w = 0xffffffffu;
                    else w = (uint32_t)((allowed << (-u0)) | ((1ull << (-u0)) - 1ull));
                    const int cov = overlap - (half * 2 + c) * 32;            // columns of this chunk that the previous tile covered
                    if (cov >= 32) w = 0u;
                    else if (cov > 0) w &= ~((1u << cov) - 1u);
#pragma unroll
                    for (int q = 0; q < 32; ++q)
                        if (!((w >> q) & 1u)) x[c][q] = 0xff800000u;   // -inf
                }
            }
            float mx0 = -CUDART_INF_F, mx1 = -CUDART_INF_F;
#pragma unroll
            for (int c = 0; c < 2; ++c)
#pragma unroll
                for (int q = 0; q < 32; q += 4) {
                    mx0 = fmax3(mx0, __uint_as_float(x[c][q]), __uint_as_float(x[c][q + 1]));
                    mx1 = fmax3(mx1, __uint_as_float(x[c][q + 2]), __uint_as_float(x[c][q + 3]));
                }
            float mx = fmaxf(mx0, mx1);
            sh.mx[gt & 1][half][rl] = mx;
            pair_sync();                 // also: the partner's scores are in its registers, P may overwrite them
            mx = fmaxf(mx, sh.mx[gt & 1][half ^ 1][rl]);
            // reference maximum: move it only when the scores outgrow it by more than the threshold
            if (mx != -CUDART_INF_F && (m_ref == -CUDART_INF_F || (mx - m_ref) * sl2 > kRescaleThreshold)) {
                if (m_ref != -CUDART_INF_F) {
                    // O must hold every earlier tile of the segment before it is rescaled (j > 0 here)
                    mbar_wait(bar(lay.pv_done + (gt - 1) % lay.pv_mod), ((gt - 1) / lay.pv_mod) & 1, abort_flag, status);
                    tc_fence_after();
                    const float alpha = exp2f((m_ref - mx) * sl2);
                    l *= alpha;
#pragma unroll 1
                    for (int c = 0; c < 2; ++c) {
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
            // P = 2^(s*scale*log2e - off) as bf16 into the first 64 columns of this S buffer
            float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t pk[16];
#pragma unroll
                for (int q = 0; q < 32; q += 2) {
                    const float p0 = ex2(fmaf(__uint_as_float(x[c][q]), sl2, -off));
                    const float p1 = ex2(fmaf(__uint_as_float(x[c][q + 1]), sl2, -off));
                    sum0 += p0;
                    sum1 += p1;
                    pk[q >> 1] = pack_bf16(p0, p1);
                }
                tmem_st16(tP + c * 16, pk);
            }
            l += sum0 + sum1;
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {                               // one arrival per warp
                if (lay.remote) mbar_arrive_remote(p_bar0 + 8u * (uint32_t)sb);
                else mbar_arrive(p_bar0 + 8u * (uint32_t)sb);
            }
            if (++sb == P_NSBUF) { sb = 0; sph ^= 1u; }
        };
        const int n_keys_seg = sg.L + sg.T;
        const int first_masked = min(sg.L / BN, PAGED ? INT_MAX : (n_keys_seg + BN - 1) / BN - 1);      // first tile of the item that needs the mask
        const int j_plain = max(0, min(nt, first_masked - sg.tile_lo));
        for (int j = 0; j < j_plain; ++j) one_tile(j, std::false_type{});
        for (int j = j_plain; j < nt; ++j) one_tile(j, std::true_type{});

        // ---- results of the segment: the two halves of the row sum, then 64 O columns each: final rows or a partial
        const int last = (jt + nt - 1) & 1;          // the exchange buffer of the other parity is idle
        sh.mx[last ^ 1][half][rl] = l;
        mbar_wait(bar(lay.O), n_seg_done & 1, abort_flag, status);     // every MMA of the segment is complete
        tc_fence_after();
        pair_sync();
        l += sh.mx[last ^ 1][half ^ 1][rl];
        if (sg.slot < 0) {
            const float inv = l > 0.f ? 1.f / l : 0.f;
            __nv_bfloat16* orow = reinterpret_cast<__nv_bfloat16*>(p.O) + (size_t)sg.b * p.o_stride_b + (size_t)t * p.o_stride_t +
                                  (size_t)(sg.h * G + g) * p.o_stride_h + half * 64;
#pragma unroll 1
            for (int c = 0; c < 2; ++c) {
                uint32_t v[32];
                tmem_ld32(tO + c * 32, v);
                tmem_wait_ld();
                if (row_valid) {
#pragma unroll
                    for (int q = 0; q < 4; ++q) {      // 16-byte stores: O strides are only guaranteed 16-byte aligned
                        uint4 o4;
                        o4.x = pack_bf16(__uint_as_float(v[q * 8 + 0]) * inv, __uint_as_float(v[q * 8 + 1]) * inv);
                        o4.y = pack_bf16(__uint_as_float(v[q * 8 + 2]) * inv, __uint_as_float(v[q * 8 + 3]) * inv);
                        o4.z = pack_bf16(__uint_as_float(v[q * 8 + 4]) * inv, __uint_as_float(v[q * 8 + 5]) * inv);
                        o4.w = pack_bf16(__uint_as_float(v[q * 8 + 6]) * inv, __uint_as_float(v[q * 8 + 7]) * inv);
                        *reinterpret_cast<uint4*>(orow + c * 32 + q * 8) = o4;
                    }
                }
            }
            if (half == 0 && row_valid && p.LSE)
                p.LSE[((size_t)sg.b * p.Hq + sg.h * G + g) * p.T_max + t] =
                    l > 0.f ? (m_ref * sl2 + log2f(l)) * kLn2 : -CUDART_INF_F;
        } else {
            float* base = a.partial + (size_t)sg.slot * SLOT_FLOATS;
            const int lr = (int)rank * 128 + rl;
            float* prow = base + (size_t)lr * D + half * 64;
#pragma unroll 1
            for (int c = 0; c < 2; ++c) {
                uint32_t v[32];
                tmem_ld32(tO + c * 32, v);
                tmem_wait_ld();
#pragma unroll
                for (int q = 0; q < 4; ++q)      // 32-byte stores: every store fills a whole sector
                    st_global_v8(prow + c * 32 + q * 8, v[q * 8], v[q * 8 + 1], v[q * 8 + 2], v[q * 8 + 3], v[q * 8 + 4],
                                 v[q * 8 + 5], v[q * 8 + 6], v[q * 8 + 7]);
            }
            if (half == 0) {
                base[BR * D + lr] = m_ref == -CUDART_INF_F ? -CUDART_INF_F : m_ref * sl2;
                base[BR * D + BR + lr] = l;
            }
            // ---- the last part of an item to arrive merges all of them (this CTA's 128 rows): M = max m_i,
            // w_i = 2^(m_i - M), O = sum w_i O_i / sum w_i l_i.  Arrivals are counted per (item, row half of the
            // pair); the count carries the call's number, so whatever an earlier call left behind is ignored.
            if (a.inkernel) {
            __threadfence();                              // this thread's partial is visible before the arrival
            asm volatile("bar.sync 9, 256;" ::: "memory");      // the eight softmax warps
            if (warp == 4 && lane == 0) {
                unsigned* cnt = reinterpret_cast<unsigned*>(a.counters) + 2 * item_id(p, sg.b, sg.h, sg.rb) + rank;
                unsigned cur = *reinterpret_cast<volatile unsigned*>(cnt), have;
                for (;;) {
                    have = (cur >> 8) == a.epoch ? (cur & 255u) : 0u;
                    const unsigned old = atomicCAS(cnt, cur, (a.epoch << 8) | (have + 1u));
                    if (old == cur) break;
                    cur = old;
                }
                *merge_flag = (int)(have + 1u) == sg.nparts;
            }
            asm volatile("bar.sync 9, 256;" ::: "memory");
            if (*merge_flag) {
                __threadfence();                          // the other parts' stores are visible now
                // every thread merges its own 64 columns of its own row, part after part (few parts: see the launch code)
                const int id = item_tag(a, item_id(p, sg.b, sg.h, sg.rb));
                float M = -CUDART_INF_F;
                for (int c = sg.c_first; c < sg.c_first + sg.c_span; ++c) {
                    const int sl = __ldcg(a.desc + 2 * c) == id ? 2 * c : (__ldcg(a.desc + 2 * c + 1) == id ? 2 * c + 1 : -1);      // from L2: an earlier merge of this CTA may have cached the line
                    if (sl >= 0) M = fmaxf(M, __ldcg(a.partial + (size_t)sl * SLOT_FLOATS + BR * D + lr));
                }
                float acc[64];
#pragma unroll
                for (int q = 0; q < 64; ++q) acc[q] = 0.f;
                float den = 0.f;
                for (int c = sg.c_first; c < sg.c_first + sg.c_span; ++c) {
                    const int sl = __ldcg(a.desc + 2 * c) == id ? 2 * c : (__ldcg(a.desc + 2 * c + 1) == id ? 2 * c + 1 : -1);      // from L2: an earlier merge of this CTA may have cached the line
                    if (sl < 0) continue;
                    const float* pb = a.partial + (size_t)sl * SLOT_FLOATS;
                    const float m = __ldcg(pb + BR * D + lr);
                    const float w = (m == -CUDART_INF_F || M == -CUDART_INF_F) ? 0.f : exp2f(m - M);
                    den += w * __ldcg(pb + BR * D + BR + lr);
                    const float4* src = reinterpret_cast<const float4*>(pb + (size_t)lr * D + half * 64);
#pragma unroll
                    for (int q = 0; q < 16; ++q) {
                        const float4 x = __ldcg(src + q);
                        acc[4 * q] += w * x.x; acc[4 * q + 1] += w * x.y; acc[4 * q + 2] += w * x.z; acc[4 * q + 3] += w * x.w;
                    }
                }
                if (row_valid) {
                    const float inv = den > 0.f ? 1.f / den : 0.f;
                    __nv_bfloat16* orow = reinterpret_cast<__nv_bfloat16*>(p.O) + (size_t)sg.b * p.o_stride_b + (size_t)t * p.o_stride_t +
                                          (size_t)(sg.h * G + g) * p.o_stride_h + half * 64;
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        uint4 o4;
                        o4.x = pack_bf16(acc[q * 8 + 0] * inv, acc[q * 8 + 1] * inv);
                        o4.y = pack_bf16(acc[q * 8 + 2] * inv, acc[q * 8 + 3] * inv);
                        o4.z = pack_bf16(acc[q * 8 + 4] * inv, acc[q * 8 + 5] * inv);
                        o4.w = pack_bf16(acc[q * 8 + 6] * inv, acc[q * 8 + 7] * inv);
                        *reinterpret_cast<uint4*>(orow + q * 8) = o4;
                    }
                    if (half == 0 && p.LSE)
                        p.LSE[((size_t)sg.b * p.Hq + sg.h * G + g) * p.T_max + t] = den > 0.f ? (M + log2f(den)) * kLn2 : -CUDART_INF_F;
                }
            }
            }
        }
        tc_fence_before();                 // TMEM reads done before the next segment's MMAs are released
        pair_sync();                       // the partner has read this segment's sum before the next segment's tiles reuse the buffer
        jt += nt;
        ++n_seg_done;
    }
}


template <bool PAGED>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(P_NTHREADS, 1)
attn_tc_pair_kernel(const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap vmap, const __grid_constant__ CUtensorMap qmap,
                    TcArgs a, unsigned* status) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    PairCtrl& ctrl = *reinterpret_cast<PairCtrl*>(smem_raw);
    Plan& plan = ctrl.plan;
    const graft_attn_params& p = a.p;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = a.G;
    const uint32_t rank = cluster_ctarank();          // 0: leader (issues the MMAs), 1: peer
    const int worker = (int)(blockIdx.x >> 1), nworkers = (int)(gridDim.x >> 1);

    asm volatile("griddepcontrol.wait;" ::: "memory");       // launched as a programmatic dependent: the kernel before this one is complete from here on
    a.epoch = next_call_no(a);
    if ((smem_u32(smem_raw) & 1023u) != 0) {          // the tiles would miss their alignment: refuse to run (both CTAs alike)
        if (threadIdx.x == 0) { atomicOr(status, (unsigned)GRAFT_FLAG_INTERNAL); cta_leaves(a); }
        return;
    }
    const uint32_t sQ = smem_u32(smem_raw) + kCtrlBytes;
    const uint32_t sRing = sQ + TILE_BYTES;
    const uint32_t bar0 = smem_u32(ctrl.bar);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    auto leader_bar = [&](int i) { return map_to_cta(bar(i), 0u); };
    volatile int* abort_flag = &ctrl.abort;

    if (a.inkernel) zero_padding_rows(a, status);
    // both CTAs of a pair derive the same plan
    if (warp == 0) plan_first(a, G, worker, nworkers, blockIdx.x == 0, rank == 0, plan);
    if (threadIdx.x == 0) ctrl.abort = 0;
    __syncthreads();
    if (plan.nseg == 0) {                             // nothing for this pair (short batch); no cluster operation was started
        if (threadIdx.x == 0) cta_leaves(a);
        return;
    }
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");      // the merge kernel may be set up from now on (it waits for this grid to end)

    if (threadIdx.x == 0) {
        for (int i = 0; i < P_NSLOT; ++i) { mbar_init(bar(PB_FULL + i), 1); mbar_init(bar(PB_EMPTY + i), 1); }
        for (int i = 0; i < P_NSBUF; ++i) { mbar_init(bar(PB_S + i), 1); mbar_init(bar(PB_P + i), 16); }      // 8 softmax warps in each CTA
        mbar_init(bar(PB_Q), 2);                    // one arrival per CTA (with the byte count when Q goes by TMA)
        mbar_init(bar(PB_O), 1);
        mbar_init(bar(PB_QFREE), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctrl.tmem)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                               // the partner's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem = ctrl.tmem;
    SplitShared& split = *reinterpret_cast<SplitShared*>(smem_raw + kCtrlBytes + TILE_BYTES + P_NSLOT * P_SLOT_BYTES);


    // running counters that persist across segments and rounds (each role keeps its own copy)
    int jt = 0;                // tiles issued / processed so far: ring slot and use, S and P barrier phases
    int n_seg_done = 0;        // segments finished (Q, Q-free and O barrier phases)

    for (;;) {                 // rounds of <= MAXSEG segments
        const int nseg = plan.nseg;

        if (warp == 0) {
            // =============================== K/V producer (both CTAs) ===============================
            if (lane == 0) {
                uint64_t stream_once;
                asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(stream_once));
                for (int si = 0; si < nseg; ++si) {
                    const Seg sg = plan.seg[si];
                    // paged caches: the block of the next tile is looked up one tile ahead, so that the table's latency
                    // hides behind the wait for a free slot
                    int blk_next = PAGED && sg.tile_lo < sg.tile_hi ? page_block(p, sg.b, sg.tile_lo * BN, status) : 0;
                    for (int t = sg.tile_lo; t < sg.tile_hi; ++t, ++jt) {
                        int overlap;
                        const int key0 = tile_key0(sg, t, overlap, PAGED);
                        // paged caches: the copy addresses (row of the page, block of the pool) instead of (slot, sequence)
                        const int krow = PAGED ? key0 % p.page_size : key0, kblk = PAGED ? blk_next : sg.b;
                        if (PAGED && t + 1 < sg.tile_hi) blk_next = page_block(p, sg.b, (t + 1) * BN, status);
                        const int slot = jt % P_NSLOT, use = jt / P_NSLOT;
                        if (use > 0) mbar_wait(bar(PB_EMPTY + slot), (use - 1) & 1, abort_flag, status);
                        if (rank == 0) mbar_expect_tx(bar(PB_FULL + slot), 2 * P_SLOT_BYTES);      // K and V halves of both CTAs
                        const uint32_t dst = sRing + slot * P_SLOT_BYTES;
                        const uint32_t fb = leader_bar(PB_FULL + slot);
                        // 64 keys of the K tile, all of d (two 64-column boxes); all keys of the V tile, 64 columns of d
                        tma_pair_4d_hint(dst, &kmap, 0, krow + 64 * (int)rank, sg.h, kblk, fb, stream_once);
                        tma_pair_4d_hint(dst + P_HALF_TILE / 2, &kmap, 64, krow + 64 * (int)rank, sg.h, kblk, fb, stream_once);
                        tma_pair_4d_hint(dst + P_HALF_TILE, &vmap, 64 * (int)rank, krow, sg.h, kblk, fb, stream_once);
                    }
                }
            }
        } else if (warp == 1) {
            // =============================== Q K^T issuer (leader only) ===============================
            // Two threads issue the MMAs: one thread cannot issue them as fast as the tensor pipe executes them
            // (measured: the pipe was active 35 % of the time with a single issuer).  This one runs ahead and
            // fills the three score buffers; the other one (warp 3) consumes P.  They meet at the slot-free
            // barrier: buffer g % 3 may be overwritten once P V of tile g - 3 is complete.
            if (lane == 0 && rank == 0) {
                for (int si = 0; si < nseg; ++si) {
                    const Seg sg = plan.seg[si];
                    const int nt = sg.tile_hi - sg.tile_lo;
                    mbar_wait_cluster(bar(PB_Q), n_seg_done & 1, abort_flag, status);   // Q of this segment is in place in both CTAs
                    for (int j = 0; j < nt; ++j) {
                        const int gt = jt + j;
                        mbar_wait(bar(PB_FULL + gt % P_NSLOT), (gt / P_NSLOT) & 1, abort_flag, status);
                        if (gt >= P_NSBUF) mbar_wait(bar(PB_EMPTY + (gt - P_NSBUF) % P_NSLOT), ((gt - P_NSBUF) / P_NSLOT) & 1, abort_flag, status);
                        tc_fence_after();
                        // S[buffer gt % 3] = Q K^T with the K half-tiles of ring slot gt % P_NSLOT (V of the same tile lands with it)
                        const uint32_t sK16 = (sRing + (gt % P_NSLOT) * P_SLOT_BYTES) >> 4;
                        const uint32_t sQ16 = sQ >> 4;
                        mma_pair_ss8(tmem + (gt % P_NSBUF) * 128, smem_desc(kDescKMajor, sQ16), smem_desc(kDescKMajor, sK16), kIdescPairQK,
                                     HALF_BYTES >> 4, (P_HALF_TILE / 2) >> 4);
                        tc_commit_pair(bar(PB_S + gt % P_NSBUF));
                    }
                    tc_commit_pair(bar(PB_QFREE));                // the segment's last Q K^T is in the pipe
                    jt += nt;
                    ++n_seg_done;
                }
            }
        } else if (warp == 3) {
            // =============================== P V issuer (leader only) ===============================
            if (lane == 0 && rank == 0) {
                for (int si = 0; si < nseg; ++si) {
                    const Seg sg = plan.seg[si];
                    const int nt = sg.tile_hi - sg.tile_lo;
                    for (int j = 0; j < nt; ++j) {
                        const int gt = jt + j;
                        mbar_wait_cluster(bar(PB_P + gt % P_NSBUF), (gt / P_NSBUF) & 1, abort_flag, status);
                        tc_fence_after();
                        const uint32_t sV16 = (sRing + (gt % P_NSLOT) * P_SLOT_BYTES + P_HALF_TILE) >> 4;
                        mma_pair_ts8(tmem + P_NSBUF * 128, tmem + (gt % P_NSBUF) * 128, smem_desc(kDescVMajor, sV16), kIdescPairPV, 2048 >> 4, j > 0 ? 1u : 0u);
                        tc_commit_pair(bar(PB_EMPTY + gt % P_NSLOT));         // the tile's K and V are read, O holds tiles 0..j
                    }
                    tc_commit_pair(bar(PB_O));
                    jt += nt;
                }
            }
        } else if (warp == 2) {
            // =============================== Q loader (both CTAs) ===============================
            for (int si = 0; si < nseg; ++si) {
                const Seg sg = plan.seg[si];
                // Q may be overwritten once the previous segment's last Q K^T is complete
                if (n_seg_done > 0) mbar_wait(bar(PB_QFREE), (n_seg_done - 1) & 1, abort_flag, status);
                const uint32_t qb = leader_bar(PB_Q);
                const int row0 = sg.rb * BR + (int)rank * 128;
                if (a.q_tma) {
                    if (lane == 0) {
                        if (rank == 0) mbar_expect_tx(bar(PB_Q), 2 * TILE_BYTES);           // 128 rows in each CTA
                        else mbar_arrive_remote(qb);
                        tma_pair_5d(sQ, &qmap, 0, 0, row0 / G, sg.h, sg.b, qb);
                        tma_pair_5d(sQ + HALF_BYTES, &qmap, 64, 0, row0 / G, sg.h, sg.b, qb);
                    }
                } else {
                    // 16-byte asynchronous copies by the warp, K-major with the 128-byte swizzle; rows past the tree read as zero
                    const int tid = lane;
                    const int R = sg.T * G;
                    const __nv_bfloat16* Qg = reinterpret_cast<const __nv_bfloat16*>(p.Q) + (size_t)sg.b * p.q_stride_b +
                                              (size_t)sg.h * G * p.q_stride_h;
                    const int ch = tid & 15;
                    int r = row0 + (tid >> 4);
                    int g = r % G;
                    const int dt = 2 / G, dg = 2 - dt * G;                 // two rows per pass
                    const __nv_bfloat16* src_t = Qg + (size_t)(r / G) * p.q_stride_t + ch * 8;
                    const size_t inc_t = (size_t)dt * p.q_stride_t;
                    for (int qr = tid >> 4; qr < 128; qr += 2) {
                        const bool valid = r < R;
                        const __nv_bfloat16* src = valid ? src_t + (size_t)g * p.q_stride_h : Qg;
                        const uint32_t dst = sQ + (ch >> 3) * HALF_BYTES + qr * 128 + (((ch & 7) ^ (qr & 7)) << 4);
                        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(valid ? 16 : 0) : "memory");
                        r += 2;
                        g += dg;
                        src_t += inc_t;
                        if (g >= G) { g -= G; src_t += p.q_stride_t; }
                    }
                    asm volatile("cp.async.wait_all;" ::: "memory");
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(qb);
                }
                ++n_seg_done;
            }
        } else if (warp >= 4) {
            // =============================== softmax, results (both CTAs) ===============================
            // this CTA's half of a V tile: all 128 keys, 64 of the d columns, behind the K half of the slot
            const SoftmaxBars lay = {PB_S, PB_P, PB_O, PB_EMPTY, P_NSLOT, true, sRing + P_HALF_TILE, P_SLOT_BYTES, P_NSLOT, 1, 0, -1};
            softmax_rows_split<PAGED>(a, plan, lay, bar0, tmem, (int)rank, split, &ctrl.merge_flag, jt, n_seg_done, abort_flag, status);
        }

        // ---- next round (only batches with very many short sequences need more than one)
        const long long g_next = plan.gnext, g_hi = plan.ghi;
        if (g_next >= g_hi) break;
        __syncthreads();
        if (warp == 0) plan_round(a, G, worker, rank == 0, plan, g_next, g_hi);
        __syncthreads();
        if (plan.nseg == 0) break;
    }

    // ---- teardown: nobody leaves while its partner may still read its shared memory or signal its barriers;
    // both CTAs free the tensor memory of the pair
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
    if (threadIdx.x == 0) cta_leaves(a);
}

// ---------------------------------------------------------------------------------------------------
// the row-block kernel: one 128-row block per CTA, partner CTAs share every tile through L2
// ---------------------------------------------------------------------------------------------------
// CTAs 2w and 2w+1 form worker w and walk the same tiles of the same items at the same time; CTA 2w owns rows
// 0..127 of an item, CTA 2w+1 rows 128..255.  Each fetches the whole K and V tile for itself: the second
// fetch of a line is an L2 hit (two CTAs streaming the same 2 GiB measured 14.2 TB/s into the SMs at
// 7.1 TB/s from HBM), so HBM still sees every byte once.  Nothing else couples the partners: no cluster, no
// shared barrier.  With one row block per SM the MMAs are the one-SM ones (Q K^T from shared memory, P V with
// P in tensor memory at full rate), three score buffers let Q K^T run ahead of P V, and the two kinds are
// issued by different threads that meet at the V slot's free barrier (P V of tile g-3 complete).
constexpr int R_NTHREADS = 384;          // producer, MMA issuer, Q loader, one idle warp, eight softmax warps
constexpr int R_NK = 3, R_NV = 3;        // ring slots of one K tile / one V tile
constexpr int R_SMEM_DYN = kCtrlBytes + TILE_BYTES + (R_NK + R_NV) * TILE_BYTES + 2048;   // control, Q (128 rows), rings, softmax exchange: 227 KB
enum { RB_FULLK = 0, RB_EMPTYK = RB_FULLK + R_NK, RB_FULLV = RB_EMPTYK + R_NK, RB_EMPTYV = RB_FULLV + R_NV, RB_S = RB_EMPTYV + R_NV,
       RB_P = RB_S + P_NSBUF, RB_Q = RB_P + P_NSBUF, RB_O = RB_Q + 1, RB_QFREE = RB_O + 1, RB_COUNT = RB_QFREE + 1 };
struct RbCtrl {
    uint64_t bar[RB_COUNT];
    Plan plan;
    uint32_t tmem;
    int abort;
    int merge_flag;
    int blk[8];              // paged caches: pool block of the last few tiles (K looks it up, V reuses it)
};
static_assert(sizeof(RbCtrl) <= kCtrlBytes, "control block too large");

template <bool PAGED>
__global__ void __launch_bounds__(R_NTHREADS, 1)
attn_tc_rb_kernel(const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap vmap, const __grid_constant__ CUtensorMap qmap,
                  TcArgs a, unsigned* status) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    RbCtrl& ctrl = *reinterpret_cast<RbCtrl*>(smem_raw);
    Plan& plan = ctrl.plan;
    const graft_attn_params& p = a.p;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = a.G;
    // two CTAs per worker, one 128-row block each; with a single block per item (chains and other small trees) a
    // partner would only repeat the copies, so every CTA walks its own tiles
    const int rank = a.single ? 0 : (int)(blockIdx.x & 1);           // which 128-row block of an item
    const int worker = a.single ? (int)blockIdx.x : (int)(blockIdx.x >> 1), nworkers = a.single ? (int)gridDim.x : (int)(gridDim.x >> 1);

    asm volatile("griddepcontrol.wait;" ::: "memory");       // launched as a programmatic dependent: the kernel before this one is complete from here on
    a.epoch = next_call_no(a);
    if ((smem_u32(smem_raw) & 1023u) != 0) {          // the tiles would miss their alignment: refuse to run
        if (threadIdx.x == 0) { atomicOr(status, (unsigned)GRAFT_FLAG_INTERNAL); cta_leaves(a); }
        return;
    }
    const uint32_t sQ = smem_u32(smem_raw) + kCtrlBytes;
    const uint32_t sK = sQ + TILE_BYTES;
    const uint32_t sV = sK + R_NK * TILE_BYTES;
    const uint32_t bar0 = smem_u32(ctrl.bar);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    volatile int* abort_flag = &ctrl.abort;

    if (a.inkernel) zero_padding_rows(a, status);
    // both CTAs of a worker derive the same plan
    if (warp == 0) plan_first(a, G, worker, nworkers, blockIdx.x == 0, rank == 0, plan);
    if (threadIdx.x == 0) ctrl.abort = 0;
    __syncthreads();
    if (plan.nseg == 0) {                             // nothing for this worker (short batch)
        if (threadIdx.x == 0) cta_leaves(a);
        return;
    }
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");      // the merge kernel may be set up from now on (it waits for this grid to end)

    if (threadIdx.x == 0) {
        for (int i = 0; i < R_NK; ++i) { mbar_init(bar(RB_FULLK + i), 1); mbar_init(bar(RB_EMPTYK + i), 1); }
        for (int i = 0; i < R_NV; ++i) { mbar_init(bar(RB_FULLV + i), 1); mbar_init(bar(RB_EMPTYV + i), 1); }
        for (int i = 0; i < P_NSBUF; ++i) { mbar_init(bar(RB_S + i), 1); mbar_init(bar(RB_P + i), 8); }      // 8 softmax warps
        mbar_init(bar(RB_Q), 1);
        mbar_init(bar(RB_O), 1);
        mbar_init(bar(RB_QFREE), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctrl.tmem)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = ctrl.tmem;
    SplitShared& split = *reinterpret_cast<SplitShared*>(smem_raw + kCtrlBytes + TILE_BYTES + (R_NK + R_NV) * TILE_BYTES);

    // running counters that persist across segments and rounds (each role keeps its own copy)
    int jt = 0;                // tiles issued / processed so far: ring slot and use, S and P barrier phases
    int n_seg_done = 0;        // segments finished (Q, Q-free and O barrier phases)

    for (;;) {                 // rounds of <= MAXSEG segments
        const int nseg = plan.nseg;

        if (warp == 0) {
            // =============================== K/V producer ===============================
            // order of issue: K(0) K(1) V(0) K(2) V(1) ...: a K tile is wanted two tiles before its V tile
            if (lane == 0) {
                int total = 0;
                for (int si = 0; si < nseg; ++si) total += plan.seg[si].tile_hi - plan.seg[si].tile_lo;
                // tile number `idx` of this round -> its segment and tile
                auto locate = [&](int idx, Seg& sg, int& t) {
                    for (int si = 0; si < nseg; ++si) {
                        const int n = plan.seg[si].tile_hi - plan.seg[si].tile_lo;
                        if (idx < n) { sg = plan.seg[si]; t = sg.tile_lo + idx; return; }
                        idx -= n;
                    }
                };
                int pre_idx = -1, pre_blk = 0;
                auto load = [&](int idx, bool is_v) {
                    Seg sg;
                    int t = 0, overlap;
                    locate(idx, sg, t);
                    const int key0 = tile_key0(sg, t, overlap, PAGED);
                    // paged caches: K of tile idx looks the block up (one tile ahead of its use) and leaves it for V of the same tile
                    int kblk = sg.b;
                    if (PAGED) {
                        if (is_v) kblk = ctrl.blk[idx & 7];
                        else {
                            kblk = idx == pre_idx ? pre_blk : page_block(p, sg.b, key0, status);
                            ctrl.blk[idx & 7] = kblk;
                            if (idx + 1 < total) {
                                Seg s2;
                                int t2 = 0;
                                locate(idx + 1, s2, t2);
                                pre_idx = idx + 1;
                                pre_blk = page_block(p, s2.b, t2 * BN, status);
                            }
                        }
                    }
                    const int krow = PAGED ? key0 % p.page_size : key0;
                    const int g = jt + idx;              // global tile number
                    const int nslot = is_v ? R_NV : R_NK;
                    const int slot = g % nslot, use = g / nslot;
                    const int full = (is_v ? RB_FULLV : RB_FULLK) + slot, empty = (is_v ? RB_EMPTYV : RB_EMPTYK) + slot;
                    if (use > 0) mbar_wait(bar(empty), (use - 1) & 1, abort_flag, status);
                    mbar_expect_tx(bar(full), TILE_BYTES);
                    const uint32_t dst = (is_v ? sV : sK) + slot * TILE_BYTES;
                    const CUtensorMap* map = is_v ? &vmap : &kmap;
                    tma_load_4d(dst, map, 0, krow, sg.h, kblk, bar(full));
                    tma_load_4d(dst + HALF_BYTES, map, 64, krow, sg.h, kblk, bar(full));
                };
                for (int i = 0; i <= total; ++i) {
                    if (i < total) load(i, false);
                    if (i > 0) load(i - 1, true);
                }
                jt += total;
            }
        } else if (warp == 1) {
            // =============================== MMA issuer ===============================
            // One thread issues everything, so the tensor pipe keeps its order: Q K^T of tile j+3 goes in right
            // behind P V of tile j, whose P it overwrites, without a barrier round trip in between.  Up to three
            // score tiles are ahead of the softmax.
            if (lane == 0) {
                for (int si = 0; si < nseg; ++si) {
                    const Seg sg = plan.seg[si];
                    const int nt = sg.tile_hi - sg.tile_lo;
                    // `landed`: the K slot's barrier was already seen complete by an earlier test
                    auto issue_qk = [&](int gt, bool landed) {
                        if (!landed) mbar_wait(bar(RB_FULLK + gt % R_NK), (gt / R_NK) & 1, abort_flag, status);
                        tc_fence_after();
                        const uint32_t sK16 = (sK + (gt % R_NK) * TILE_BYTES) >> 4;
                        const uint32_t sQ16 = sQ >> 4;
#pragma unroll
                        for (int k = 0; k < D / 16; ++k) {
                            const uint32_t off16 = ((k >> 2) * HALF_BYTES + (k & 3) * 32) >> 4;
                            mma_ss(tmem + (gt % P_NSBUF) * 128, smem_desc(kDescKMajor, sQ16 + off16), smem_desc(kDescKMajor, sK16 + off16), kIdescQK, k > 0);
                        }
                        tc_commit(bar(RB_S + gt % P_NSBUF));
                        tc_commit(bar(RB_EMPTYK + gt % R_NK));           // K tile fully read
                    };
                    mbar_wait(bar(RB_Q), n_seg_done & 1, abort_flag, status);           // Q of this segment is in place
                    for (int j = 0; j < P_NSBUF && j < nt; ++j) issue_qk(jt + j, false);
                    if (nt <= P_NSBUF) tc_commit(bar(RB_QFREE));       // the segment's last Q K^T is in the pipe
                    // Issuing an MMA blocks until the pipe takes it and a barrier test costs a round trip of about a
                    // hundred cycles, so every barrier is tested ahead of the run of MMAs before the one that needs it.
                    bool v_ok = false, p_ok = false;
                    for (int j = 0; j < nt; ++j) {
                        const int gt = jt + j;
                        if (!v_ok) mbar_wait(bar(RB_FULLV + gt % R_NV), (gt / R_NV) & 1, abort_flag, status);
                        if (!p_ok) mbar_wait(bar(RB_P + gt % P_NSBUF), (gt / P_NSBUF) & 1, abort_flag, status);
                        const bool k_ok = j + P_NSBUF < nt && mbar_test(bar(RB_FULLK + (gt + P_NSBUF) % R_NK), ((gt + P_NSBUF) / R_NK) & 1);
                        tc_fence_after();
                        const uint32_t sV16 = (sV + (gt % R_NV) * TILE_BYTES) >> 4;
#pragma unroll
                        for (int k = 0; k < BN / 16; ++k)
                            mma_ts(tmem + P_NSBUF * 128, tmem + (gt % P_NSBUF) * 128 + k * 8, smem_desc(kDescVMajor, sV16 + k * (2048 >> 4)), kIdescPV,
                                   (j > 0 || k > 0) ? 1u : 0u);
                        tc_commit(bar(RB_EMPTYV + gt % R_NV));           // V tile fully read, O holds tiles 0..j
                        v_ok = j + 1 < nt && mbar_test(bar(RB_FULLV + (gt + 1) % R_NV), ((gt + 1) / R_NV) & 1);
                        p_ok = j + 1 < nt && mbar_test(bar(RB_P + (gt + 1) % P_NSBUF), ((gt + 1) / P_NSBUF) & 1);
                        if (j + P_NSBUF < nt) {
                            issue_qk(gt + P_NSBUF, k_ok);
                            if (j + P_NSBUF + 1 == nt) tc_commit(bar(RB_QFREE));
                        }
                    }
                    tc_commit(bar(RB_O));
                    jt += nt;
                    ++n_seg_done;
                }
            }
        } else if (warp == 2) {
            // =============================== Q loader ===============================
            for (int si = 0; si < nseg; ++si) {
                const Seg sg = plan.seg[si];
                // Q may be overwritten once the previous segment's last Q K^T is complete
                if (n_seg_done > 0) mbar_wait(bar(RB_QFREE), (n_seg_done - 1) & 1, abort_flag, status);
                const int row0 = sg.rb * BR + rank * 128;
                if (a.q_tma) {
                    if (lane == 0) {
                        mbar_expect_tx(bar(RB_Q), TILE_BYTES);
                        tma_load_5d(sQ, &qmap, 0, 0, row0 / G, sg.h, sg.b, bar(RB_Q));
                        tma_load_5d(sQ + HALF_BYTES, &qmap, 64, 0, row0 / G, sg.h, sg.b, bar(RB_Q));
                    }
                } else {
                    // 16-byte asynchronous copies by the warp, K-major with the 128-byte swizzle; rows past the tree read as zero
                    const int R = sg.T * G;
                    const __nv_bfloat16* Qg = reinterpret_cast<const __nv_bfloat16*>(p.Q) + (size_t)sg.b * p.q_stride_b +
                                              (size_t)sg.h * G * p.q_stride_h;
                    const int ch = lane & 15;
                    int r = row0 + (lane >> 4);
                    int g = r % G;
                    const int dt = 2 / G, dg = 2 - dt * G;                 // two rows per pass
                    const __nv_bfloat16* src_t = Qg + (size_t)(r / G) * p.q_stride_t + ch * 8;
                    const size_t inc_t = (size_t)dt * p.q_stride_t;
                    for (int qr = lane >> 4; qr < 128; qr += 2) {
                        const bool valid = r < R;
                        const __nv_bfloat16* src = valid ? src_t + (size_t)g * p.q_stride_h : Qg;
                        const uint32_t dst = sQ + (ch >> 3) * HALF_BYTES + qr * 128 + (((ch & 7) ^ (qr & 7)) << 4);
                        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(valid ? 16 : 0) : "memory");
                        r += 2;
                        g += dg;
                        src_t += inc_t;
                        if (g >= G) { g -= G; src_t += p.q_stride_t; }
                    }
                    asm volatile("cp.async.wait_all;" ::: "memory");
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(RB_Q));
                }
                ++n_seg_done;
            }
        } else if (warp >= 4) {
            // =============================== softmax, results ===============================
            const SoftmaxBars lay = {RB_S, RB_P, RB_O, RB_EMPTYV, R_NV, false, sV, TILE_BYTES, R_NV, 2, HALF_BYTES, RB_FULLV};
            softmax_rows_split<PAGED>(a, plan, lay, bar0, tmem, rank, split, &ctrl.merge_flag, jt, n_seg_done, abort_flag, status);
        }

        // ---- next round (only batches with very many short sequences need more than one)
        const long long g_next = plan.gnext, g_hi = plan.ghi;
        if (g_next >= g_hi) break;
        __syncthreads();
        if (warp == 0) plan_round(a, G, worker, rank == 0, plan, g_next, g_hi);
        __syncthreads();
        if (plan.nseg == 0) break;
    }

    // ---- teardown: after a timeout some copies may still be in flight: give them time to land before the
    // shared memory is handed back; the allocating warp frees the tensor memory once everyone is past its last access
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < (1ll << 22)) {}
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
    if (threadIdx.x == 0) cta_leaves(a);
}

// ---------------------------------------------------------------------------------------------------
// merge: half a warp per output row of the padded [T_max * G] row space of a (b, h_kv)
// ---------------------------------------------------------------------------------------------------
// Rows of an item that was cut across CTAs are merged with  M = max m_i, w_i = 2^(m_i - M),
// O = sum w_i O_i / sum w_i l_i;  rows of padding nodes are zeroed (LSE -inf); rows of items that one CTA
// finished alone were already final.  The set of CTAs that hold a piece of an item follows from the
// same cut as in the attention kernel.
// The kernel is a chain of dependent round trips to L2 (the recorded cut, the partial slots' descriptors with
// the parts' maxima and sums, the partial rows) and every row walks it once; what it costs is the number of
// links times the number of rows a warp takes one after the other.  So a row belongs to sixteen lanes (eight
// columns each) with lane i of them looking after part i, all rows of a launch are in flight at once as long as
// the batch allows it, and the maximum and sum of both slots of a candidate CTA are requested together with
// its descriptors instead of after them.  Items cut into many parts (few sequences on many SMs) take a whole
// warp per row instead (LPR = 32): four columns per lane and eight parts' rows in flight rather than four.
constexpr int kMergeWarps = 8;       // warps per CTA; rows per CTA is a launch parameter (one or four passes)

template <int LPR>                   // lanes per row: 16 or 32
__global__ void __launch_bounds__(kMergeWarps * 32, 4) merge_streamk_kernel(TcArgs a, int rows_per_cta, unsigned* status) {
    constexpr int kRows = kMergeWarps * (32 / LPR);        // rows of a CTA in flight
    constexpr int NL = 128 / LPR / 4;                      // 16-byte loads per lane and partial row
    constexpr int PF = 8 / NL;                             // partial rows in flight per round
    asm volatile("griddepcontrol.wait;" ::: "memory");      // launched early: nothing is read before the attention kernel is complete
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    a.epoch = __ldcg(a.call_no);                            // the call the attention kernel just finished
    const graft_attn_params& p = a.p;
    const int G = a.G;
    const int rows_pad = p.T_max * G;
    const int groups = (rows_pad + rows_per_cta - 1) / rows_per_cta;
    int idx = blockIdx.x;
    const int grp = idx % groups; idx /= groups;
    const int h = idx % p.Hkv;
    const int b = idx / p.Hkv;
    __shared__ SeqInfo s_info;
    __shared__ long long s_per;
    __shared__ int s_pieces;
    if (threadIdx.x == 0) {
        // the cut was recorded by the attention kernel: no need to scan the batch again
        const SeqEntry e = reinterpret_cast<const SeqEntry*>(a.cut + 1)[b];
        SeqInfo si;
        si.b = b; si.L = e.L; si.T = e.T; si.nrb = e.nrb; si.ntiles = e.ntiles; si.wlast = e.wlast; si.base = e.base; si.found = true;
        s_info = si;
        s_per = a.cut->per;
        s_pieces = a.cut->pieces;
        const int T = p.tree_size[b], L = p.seq_len[b];
        if (grp == 0 && h == 0 && (T < 0 || T > p.T_max || L < 0 || (long long)L + T > p.S_cap))
            atomicOr(status, (unsigned)GRAFT_FLAG_BAD_SIZE);
    }
    __syncthreads();
    const SeqInfo si = s_info;
    const long long per = s_per;
    const bool pieces = s_pieces != 0;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int hw = lane / LPR, hl = lane % LPR;             // which of the warp's rows, lane among the row's lanes
    const unsigned hmask = LPR == 32 ? 0xffffffffu : 0xffffu << (16 * hw);      // the two halves of a warp go their own ways
    for (int r = grp * rows_per_cta + (32 / LPR) * warp + hw; r < min(rows_pad, (grp + 1) * rows_per_cta); r += kRows) {
    const int t = r / G, g = r % G;
    __nv_bfloat16* orow = reinterpret_cast<__nv_bfloat16*>(p.O) + (size_t)b * p.o_stride_b + (size_t)t * p.o_stride_t +
                          (size_t)(h * G + g) * p.o_stride_h + hl * (4 * NL);
    float* lse = p.LSE ? p.LSE + ((size_t)b * p.Hq + h * G + g) * p.T_max + t : nullptr;
    if (t >= si.T) {                       // padding node: zero row
        if (NL == 2) *reinterpret_cast<uint4*>(orow) = make_uint4(0u, 0u, 0u, 0u);
        else *reinterpret_cast<uint2*>(orow) = make_uint2(0u, 0u);
        if (lse && hl == 0) *lse = -CUDART_INF_F;
        continue;
    }
    const int rb = r / BR, rl = r % BR;
    // the partial slots that hold pieces of this item, from the same cut as in the attention kernel
    int nparts, c_first = 0, piece_cta0 = 0;
    const int id = item_tag(a, item_id(p, b, h, rb));
    if (pieces) {
        int nsplit, plen;
        piece_shape(si.ntiles, per, nsplit, plen);
        nparts = nsplit;
        piece_cta0 = (int)si.base + (h * si.nrb + rb) * nsplit;      // CTA of the item's first piece
    } else {
        long long U;
        int w;
        item_span(si, h, rb, U, w);
        c_first = (int)udiv(U, per);
        const long long last = si.ntiles > 1 ? U + kOvh + (long long)(si.ntiles - 1) * w : U;      // first unit of the last tile
        nparts = (int)udiv(last, per) - c_first + 1;
    }
    if (nparts <= 1) continue;             // one CTA had the whole item and wrote the final rows
    // Part i: its slot (-1: that CTA's range held no tile of the item), maximum and sum of this row.  Stream-K: part i
    // lives in CTA c_first + i, in the slot whose descriptor names this item; both slots' values are requested at once.
    auto part = [&](int i, int& slot, float& m, float& l) {
        if (pieces) {
            slot = 2 * (piece_cta0 + i);
            const float* ml = a.partial + (size_t)slot * SLOT_FLOATS + BR * D + rl;
            m = __ldcg(ml);
            l = __ldcg(ml + BR);
        } else {
            const int c = c_first + i;
            const float* ml0 = a.partial + (size_t)(2 * c) * SLOT_FLOATS + BR * D + rl;
            const int d0 = __ldcg(a.desc + 2 * c), d1 = __ldcg(a.desc + 2 * c + 1);
            const float m0 = __ldcg(ml0), l0 = __ldcg(ml0 + BR), m1 = __ldcg(ml0 + SLOT_FLOATS), l1 = __ldcg(ml0 + SLOT_FLOATS + BR);
            slot = d0 == id ? 2 * c : (d1 == id ? 2 * c + 1 : -1);
            m = d0 == id ? m0 : m1;
            l = d0 == id ? l0 : l1;
        }
        if (slot < 0) { m = -CUDART_INF_F; l = 0.f; }
    };
    // lane hl keeps part hl (the first LPR); items cut into more parts than that walk the rest in rounds of LPR
    int slot0 = -1;
    float m0 = -CUDART_INF_F, l0 = 0.f;
    if (hl < nparts) part(hl, slot0, m0, l0);
    float M = m0;
    for (int i = LPR + hl; i < nparts; i += LPR) {
        int sl;
        float m, l;
        part(i, sl, m, l);
        M = fmaxf(M, m);
    }
#pragma unroll
    for (int o = LPR / 2; o; o >>= 1) M = fmaxf(M, __shfl_xor_sync(hmask, M, o));
    float acc[4 * NL];
#pragma unroll
    for (int q = 0; q < 4 * NL; ++q) acc[q] = 0.f;
    float den = 0.f;
    for (int i0 = 0; i0 < nparts; i0 += LPR) {
        int slot = slot0;
        float m = m0, l = l0;
        if (i0 > 0) {
            slot = -1; m = -CUDART_INF_F; l = 0.f;
            if (i0 + hl < nparts) part(i0 + hl, slot, m, l);
        }
        const float wgt = (m == -CUDART_INF_F || M == -CUDART_INF_F) ? 0.f : exp2f(m - M);
        den += wgt * l;
        const int cnt = min(LPR, nparts - i0);
        for (int j0 = 0; j0 < cnt; j0 += PF) {       // eight 16-byte loads in flight per round
            float4 x[PF][NL];
#pragma unroll
            for (int j = 0; j < PF; ++j)
                if (j0 + j < cnt) {
                    // the owner lane of part j0 + j knows whether it exists; a missing part has weight 0
                    const int sj = __shfl_sync(hmask, slot, j0 + j, LPR);
                    const float4* src = reinterpret_cast<const float4*>(a.partial + (size_t)(sj < 0 ? 0 : sj) * SLOT_FLOATS + (size_t)rl * D) + hl * NL;
#pragma unroll
                    for (int q = 0; q < NL; ++q) x[j][q] = sj >= 0 ? __ldcg(src + q) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
            for (int j = 0; j < PF; ++j)
                if (j0 + j < cnt) {
                    const float wj = __shfl_sync(hmask, wgt, j0 + j, LPR);
#pragma unroll
                    for (int q = 0; q < NL; ++q) {
                        acc[4 * q] += wj * x[j][q].x; acc[4 * q + 1] += wj * x[j][q].y; acc[4 * q + 2] += wj * x[j][q].z; acc[4 * q + 3] += wj * x[j][q].w;
                    }
                }
        }
    }
#pragma unroll
    for (int o = LPR / 2; o; o >>= 1) den += __shfl_xor_sync(hmask, den, o);
    const float inv = den > 0.f ? 1.f / den : 0.f;
    if (NL == 2)
        *reinterpret_cast<uint4*>(orow) = make_uint4(pack_bf16(acc[0] * inv, acc[1] * inv), pack_bf16(acc[2] * inv, acc[3] * inv),
                                                     pack_bf16(acc[4 * NL - 4] * inv, acc[4 * NL - 3] * inv), pack_bf16(acc[4 * NL - 2] * inv, acc[4 * NL - 1] * inv));
    else
        *reinterpret_cast<uint2*>(orow) = make_uint2(pack_bf16(acc[0] * inv, acc[1] * inv), pack_bf16(acc[2] * inv, acc[3] * inv));
    if (lse && hl == 0) *lse = den > 0.f ? (M + log2f(den)) * kLn2 : -CUDART_INF_F;
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;
constexpr int kMaxDevices = 64;
int g_pair_clusters[kMaxDevices] = {0};      // resident 2-CTA clusters of the pair kernel per device (0: not asked yet)

int make_kv_map(CUtensorMap* map, const void* base, const graft_attn_params* p, int box_rows = BN) {
    // contiguous caches: (d, slot, KV head, sequence); paged: (d, row of the page, KV head, block of the pool)
    const cuuint64_t dims[4] = {(cuuint64_t)p->d, (cuuint64_t)(p->block_table ? p->page_size : p->S_cap), (cuuint64_t)p->Hkv,
                                (cuuint64_t)(p->block_table ? p->n_blocks : p->B)};
    const cuuint64_t strides[3] = {(cuuint64_t)p->kv_stride_s * 2, (cuuint64_t)p->kv_stride_h * 2, (cuuint64_t)p->kv_stride_b * 2};
    const cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 1, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUresult rc = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return rc == CUDA_SUCCESS ? GRAFT_OK : GRAFT_ERR_CUDA;
}

// Q [B, T_max, Hq, d] seen as (d, g, t, KV head, b): one box is 128 consecutive rows r = t*G + g of one KV head.
int make_q_map(CUtensorMap* map, const graft_attn_params* p, int G) {
    const cuuint64_t dims[5] = {(cuuint64_t)p->d, (cuuint64_t)G, (cuuint64_t)p->T_max, (cuuint64_t)p->Hkv, (cuuint64_t)p->B};
    const cuuint64_t strides[4] = {(cuuint64_t)p->q_stride_h * 2, (cuuint64_t)p->q_stride_t * 2, (cuuint64_t)p->q_stride_h * 2 * G,
                                   (cuuint64_t)p->q_stride_b * 2};
    const cuuint32_t box[5] = {64, (cuuint32_t)G, (cuuint32_t)(128 / G), 1, 1};
    const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    const CUresult rc = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(p->Q), dims, strides, box, estr,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return rc == CUDA_SUCCESS ? GRAFT_OK : GRAFT_ERR_CUDA;
}

// TMA wants 16-byte aligned base and strides, strides below 2^40 bytes; the box wants G to divide 128
bool q_map_possible(const graft_attn_params* p, int G) {
    if (G < 1 || 128 % G != 0) return false;
    const long long st[3] = {p->q_stride_h, p->q_stride_t, p->q_stride_b};
    for (long long v : st)
        if (v <= 0 || (v * 2) % 16 != 0 || v * 2 * G >= (1ll << 40)) return false;
    return (reinterpret_cast<uintptr_t>(p->Q) & 15) == 0;
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
    // pair kernel: how many 2-CTA clusters fit on the device at once (SMs that cannot be paired stay idle)
    GRAFT_CHECK_CUDA(cudaFuncSetAttribute(attn_tc_pair_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, P_SMEM_DYN));
    GRAFT_CHECK_CUDA(cudaFuncSetAttribute(attn_tc_pair_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, P_SMEM_DYN));
    GRAFT_CHECK_CUDA(cudaFuncSetAttribute(attn_tc_rb_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, R_SMEM_DYN));
    GRAFT_CHECK_CUDA(cudaFuncSetAttribute(attn_tc_rb_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, R_SMEM_DYN));
    int dev = 0;
    GRAFT_CHECK_CUDA(cudaGetDevice(&dev));
    if (dev >= 0 && dev < kMaxDevices && g_pair_clusters[dev] == 0) {
        int sms = 0;
        GRAFT_CHECK_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(sms & ~1));
        cfg.blockDim = dim3(P_NTHREADS);
        cfg.dynamicSmemBytes = P_SMEM_DYN;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = 2;
        attr.val.clusterDim.y = 1;
        attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, attn_tc_pair_kernel<false>, &cfg) != cudaSuccess) { (void)cudaGetLastError(); n = 0; }
        g_pair_clusters[dev] = n > 0 ? (n < sms / 2 ? n : sms / 2) : -1;      // -1: the pair kernel cannot run here
    }
    return GRAFT_OK;
}

// number of resident CTA pairs of the pair kernel on the current device (0 if it cannot run)
static int pair_clusters() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 0;
    return g_pair_clusters[dev] > 0 ? g_pair_clusters[dev] : 0;
}

// The pair kernel pays off when items carry more than 128 rows (the second SM of a pair would otherwise idle).
bool graft_attn_tc_pair_supported(const graft_ctx* ctx, const graft_attn_params* p) {
    if (!graft_attn_tc_supported(ctx, p)) return false;
    return pair_clusters() > 0;
}

bool graft_attn_tc_supported(const graft_ctx* ctx, const graft_attn_params* p) {
    if (p->d != D) return false;
    if ((long long)p->B * p->Hkv * 8 >= (1ll << 24)) return false;      // item ids share a word with the call stamp
    // TMA: 16-byte aligned base and strides (checked by the caller), strides below 2^40 bytes
    if (p->kv_stride_s * 2 >= (1ll << 40) || p->kv_stride_h * 2 >= (1ll << 40) || p->kv_stride_b * 2 >= (1ll << 40)) return false;
    if (p->kv_stride_s == 0 || p->kv_stride_h == 0 || p->kv_stride_b == 0) return false;
    return GRAFT_WS_HEADER + graft_attn_tc_ws_bytes(ctx->num_sms, p->B, p->Hq, p->Hkv, p->d, p->T_max) <= ctx->ws_bytes;
}

// two partial slots per CTA, one CTA per SM (independent of the batch), plus the recorded cut
size_t graft_attn_tc_ws_bytes(int num_sms, int B, int, int Hkv, int d, int) {
    if (d != D) return 0;
    return kDescBytes + cut_bytes(B) + counter_bytes(B, Hkv) + (size_t)num_sms * 2 * SLOT_FLOATS * sizeof(float);
}

int graft_attn_tc_launch(graft_ctx* ctx, const graft_attn_params* p, cudaStream_t stream, int which) {
    const int G = p->Hq / p->Hkv;
    // which: 0 two row blocks per CTA, 1 CTA pairs with two-SM MMAs, 2 one row block per CTA with partners sharing
    // tiles through L2, < 0 choose.  Measured: kernels 1 and 2 are within a few per cent of each other and both
    // beat kernel 0 everywhere; the pair kernel wins when a KV head carries more than 256 rows, the row-block
    // kernel otherwise.
    if (which < 0) which = (p->T_max * G > 256 && graft_attn_tc_pair_supported(ctx, p)) ? 1 : 2;
    const bool use_pair = which == 1, use_rb = which == 2;
    if (use_pair && !graft_attn_tc_pair_supported(ctx, p)) return GRAFT_ERR_UNSUPPORTED;
    CUtensorMap kmap, vmap;
    int rc = make_kv_map(&kmap, p->Kc, p, use_pair ? 64 : BN);
    if (rc == GRAFT_OK) rc = make_kv_map(&vmap, p->Vc, p);
    CUtensorMap qmap = kmap;                 // unused placeholder unless Q goes by TMA
    const bool q_tma = q_map_possible(p, G);
    if (rc == GRAFT_OK && q_tma) rc = make_q_map(&qmap, p, G);
    if (rc != GRAFT_OK) return rc;
    TcArgs a;
    a.p = *p;
    a.desc = reinterpret_cast<int*>(reinterpret_cast<char*>(ctx->ws) + GRAFT_WS_HEADER);
    a.cut = reinterpret_cast<CutHeader*>(reinterpret_cast<char*>(ctx->ws) + GRAFT_WS_HEADER + kDescBytes);
    a.counters = reinterpret_cast<int*>(reinterpret_cast<char*>(ctx->ws) + GRAFT_WS_HEADER + kDescBytes + cut_bytes(p->B));
    a.partial = reinterpret_cast<float*>(reinterpret_cast<char*>(ctx->ws) + GRAFT_WS_HEADER + kDescBytes + cut_bytes(p->B) + counter_bytes(p->B, p->Hkv));
    a.epoch = 0u;
    a.call_no = ctx->status + 4;            // two words of the workspace header
    // Merge in the kernel (by the last part of an item to arrive) only for short calls whose items are cut into two or
    // three parts: there the second launch costs more than one CTA reading all parts of its 128 rows alone.  The host
    // only knows the shapes: an item is about one KV head of one sequence, so there are about workers / (B * H_kv) + 1
    // parts per item.  Measured (Qwen3-14B heads, 74 workers, in-kernel against the merge kernel): 8 x 4K -5 us of 60,
    // 8 x 8K -5 of 91, 5 x 8K -3 of 87, the ragged batch of sixteen -3 of 173; but 16 x 4K +3, 12 x 8K +1, and from 16K
    // context on, where an early part has left L2 by the time the last one arrives, +15 to +17 us (5, 6, 8 x 16K;
    // 5, 6 x 32K), +11 on 5 x 64K; a single sequence cut into nine +70 %.
    a.G = G;
    a.q_tma = q_tma ? 1 : 0;
    a.single = use_rb && p->T_max * G <= 128 ? 1 : 0;
    const int workers = a.single ? ctx->num_sms : ctx->num_sms / 2;
    const long long heads = (long long)p->B * p->Hkv;
    a.inkernel = (use_pair || use_rb) && workers <= 2 * heads && heads <= workers && p->S_cap <= 12288 ? 1 : 0;
    a.prof_cta = 0;
#ifdef GRAFT_TC_EXPERIMENTS
    if (getenv("GRAFT_TC_PROF_CTA")) a.prof_cta = atoi(getenv("GRAFT_TC_PROF_CTA"));
#endif
    int grid = ctx->num_sms;
#ifdef GRAFT_TC_EXPERIMENTS
    if (getenv("GRAFT_TC_GRID")) grid = atoi(getenv("GRAFT_TC_GRID"));
#endif
    if (use_pair) {
        int pairs = pair_clusters();
        if (pairs > ctx->num_sms / 2) pairs = ctx->num_sms / 2;       // the workspace has two slots per SM
        GRAFT_CHECK_CUDA(graft_launch(p->block_table ? attn_tc_pair_kernel<true> : attn_tc_pair_kernel<false>, dim3(2 * pairs),
                                      dim3(P_NTHREADS), P_SMEM_DYN, stream, kmap, vmap, qmap, a, ctx->status));
    } else if (use_rb) {
        const int rb_grid = a.single ? ctx->num_sms : ctx->num_sms & ~1;
        GRAFT_CHECK_CUDA(graft_launch(p->block_table ? attn_tc_rb_kernel<true> : attn_tc_rb_kernel<false>, dim3(rb_grid),
                                      dim3(R_NTHREADS), R_SMEM_DYN, stream, kmap, vmap, qmap, a, ctx->status));
    } else
    GRAFT_CHECK_CUDA(graft_launch(attn_tc_kernel, dim3(grid), dim3(NTHREADS), SMEM_DYN, stream, kmap, vmap, qmap, a, ctx->status));
    GRAFT_CHECK_CUDA(cudaGetLastError());
    if (a.inkernel) return GRAFT_OK;               // merged in place: the last part of an item to finish combined them
    // Items in about four parts or fewer: half a warp per row; more: a warp per row.  Few rows: all of them in flight at
    // once (the merge is latency-bound); many rows: four passes, to keep the CTA count down
    const int rows_pad = p->T_max * a.G;
    const bool half_warp = 2 * (long long)workers <= 7 * (long long)p->B * p->Hkv;        // workers / items + 1 <= 4.5 parts
    const int rows_flight = kMergeWarps * (half_warp ? 2 : 1);
    const int rows_per_cta = (long long)p->B * p->Hkv * rows_pad >= 65536 ? 4 * rows_flight : rows_flight;
    const int groups = (rows_pad + rows_per_cta - 1) / rows_per_cta;
    // programmatic dependent launch: the merge CTAs are set up while the attention kernel still runs and wait
    // (griddepcontrol.wait) until it has completed and its writes are visible
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p->B * p->Hkv * groups));
    cfg.blockDim = dim3(kMergeWarps * 32);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    GRAFT_CHECK_CUDA(cudaLaunchKernelEx(&cfg, half_warp ? merge_streamk_kernel<16> : merge_streamk_kernel<32>, a, rows_per_cta, ctx->status));
    return GRAFT_OK;
}
