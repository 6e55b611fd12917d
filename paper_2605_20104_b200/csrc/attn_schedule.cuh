// Split-KV schedule shared by the attention kernels and their merge kernel.
//
// A work item is (sequence b, KV head h, row block rb): BR rows (row r <-> tree node r / G, query
// head h*G + r % G) against all ceil((L_b+T_b)/BN) key tiles of the sequence.  Each item is cut along
// the key axis into nsplit_b nearly equal contiguous pieces so that the whole batch yields about
// `target` CTAs; a CTA is one (item, split).  The cut is a pure function of (seq_len, tree_size,
// target), computed redundantly by every CTA from the device-resident lengths (the host never
// sees them), so the attention grid and the merge grid agree without any communication.
//
// CTA order inside a sequence: ((h * nsplit + split) * nrb + rb): the row blocks that read the same
// keys are neighbours in launch order and run concurrently, so the second reader hits L2.
#pragma once
#include <stdint.h>

namespace graft_sched {

struct Work {
    int b, h, rb, split;     // what this CTA computes
    int nsplit, nrb;         // of its sequence
    int tile_lo, tile_hi;    // key tiles [lo, hi)
    int L, T;                // cached length and tree size (0, 0 for an invalid sequence)
    int first_slot;          // partial slot of (h = 0, split = 0, rb = 0) of this sequence
    bool valid;
};

__device__ __forceinline__ void seq_dims(const int32_t* seq_len, const int32_t* tree_size, int b, int T_max,
                                         int S_cap, int& L, int& T) {
    L = seq_len[b];
    T = tree_size[b];
    if (T < 0 || T > T_max || L < 0 || (long long)L + T > (long long)S_cap) { L = 0; T = 0; }
}

// FLOOR = false: ceil(ntiles / chunk) pieces (a little over `target` CTAs, for kernels that run several
// CTAs per SM in waves); FLOOR = true: floor(ntiles / chunk) pieces, so the grid stays within `target`
// whenever no sequence is shorter than one chunk (for one-CTA-per-SM kernels that must fit one wave).
template <int BR, int BN, bool FLOOR>
__device__ __forceinline__ void seq_shape(int L, int T, int G, int chunk, int& ntiles, int& nrb, int& nsplit,
                                          int& per) {
    ntiles = T > 0 ? (L + T + BN - 1) / BN : 0;
    nrb = (T * G + BR - 1) / BR;
    nsplit = 0;
    per = 0;
    if (ntiles > 0) {
        const int want = FLOOR ? max(1, ntiles / chunk) : (ntiles + chunk - 1) / chunk;
        per = (ntiles + want - 1) / want;
        nsplit = (ntiles + per - 1) / per;       // every split non-empty
    }
}

// Tiles per CTA so that the batch gives about `target` CTAs.  Called by a full warp.
template <int BR, int BN>
__device__ __forceinline__ int chunk_size(const int32_t* seq_len, const int32_t* tree_size, int B, int Hkv, int G,
                                          int T_max, int S_cap, int target) {
    const int lane = threadIdx.x & 31;
    long long total = 0;
    for (int b = lane; b < B; b += 32) {
        int L, T;
        seq_dims(seq_len, tree_size, b, T_max, S_cap, L, T);
        const int ntiles = T > 0 ? (L + T + BN - 1) / BN : 0;
        total += (long long)Hkv * ((T * G + BR - 1) / BR) * ntiles;
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
    long long c = (total + target - 1) / target;
    return c < 1 ? 1 : (c > 0x3fffffff ? 0x3fffffff : (int)c);
}

// Maps CTA `cta` to its work.  Called by a full warp; every lane returns the same Work.
// With want_b >= 0 the lookup is by sequence instead (used by the merge kernel): first_slot,
// nsplit, nrb, L, T of sequence want_b.
template <int BR, int BN, bool FLOOR = false>
__device__ __forceinline__ Work find_work(const int32_t* seq_len, const int32_t* tree_size, int B, int Hkv, int G,
                                          int T_max, int S_cap, int target, int cta, int want_b) {
    const int lane = threadIdx.x & 31;
    const int chunk = chunk_size<BR, BN>(seq_len, tree_size, B, Hkv, G, T_max, S_cap, target);
    Work w;
    w.valid = false;
    w.b = w.h = w.rb = w.split = w.nsplit = w.nrb = w.tile_lo = w.tile_hi = w.L = w.T = w.first_slot = 0;
    int run = 0;
    for (int base = 0; base < B; base += 32) {
        const int b = base + lane;
        int L = 0, T = 0, ntiles = 0, nrb = 0, nsplit = 0, per = 0, cnt = 0;
        if (b < B) {
            seq_dims(seq_len, tree_size, b, T_max, S_cap, L, T);
            seq_shape<BR, BN, FLOOR>(L, T, G, chunk, ntiles, nrb, nsplit, per);
            cnt = Hkv * nrb * nsplit;
        }
        int incl = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        const int start = run + incl - cnt;
        const bool hit = b < B && (want_b >= 0 ? b == want_b : (cta >= start && cta < start + cnt));
        const unsigned m = __ballot_sync(0xffffffffu, hit);
        if (m) {
            const int src = __ffs(m) - 1;
            w.valid = true;
            w.b = base + src;
            w.L = __shfl_sync(0xffffffffu, L, src);
            w.T = __shfl_sync(0xffffffffu, T, src);
            w.nrb = __shfl_sync(0xffffffffu, nrb, src);
            w.nsplit = __shfl_sync(0xffffffffu, nsplit, src);
            w.first_slot = __shfl_sync(0xffffffffu, start, src);
            const int per_s = __shfl_sync(0xffffffffu, per, src);
            const int nt = __shfl_sync(0xffffffffu, ntiles, src);
            if (want_b < 0) {
                const int local = cta - w.first_slot;
                w.rb = local % w.nrb;
                w.split = (local / w.nrb) % w.nsplit;
                w.h = local / (w.nrb * w.nsplit);
                w.tile_lo = w.split * per_s;
                w.tile_hi = min(nt, w.tile_lo + per_s);
            }
            return w;
        }
        run += __shfl_sync(0xffffffffu, incl, 31);
    }
    return w;
}

__device__ __forceinline__ int slot_of(const Work& w, int h, int split, int rb) {
    return w.first_slot + (h * w.nsplit + split) * w.nrb + rb;
}

}  // namespace graft_sched
