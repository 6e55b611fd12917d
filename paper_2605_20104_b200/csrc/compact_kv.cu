// graft_compact_kv: move the accepted path's K/V rows to contiguous cache slots, in place.
//
// One CTA per (sequence, KV head, layer, K-or-V).  Destination slot L+j can be the source slot of
// an earlier path entry, so the CTA first stages every source row it needs in shared memory
// (at most 64 rows x 256 B), synchronises, and only then stores.  Rows already in place are skipped.
#include "graft_internal.cuh"

namespace {

constexpr int kThreads = 256;

__global__ void __launch_bounds__(kThreads) compact_kernel(graft_compact_params a, unsigned* status) {
    graft_wait_for_stream();
    extern __shared__ uint4 stage[];            // [n_acc][d/8] 16-byte chunks
    __shared__ int s_path[64];
    __shared__ int s_ok;
    int idx = blockIdx.x;
    const int which = idx & 1; idx >>= 1;       // 0: K, 1: V
    const int h = idx % a.Hkv; idx /= a.Hkv;
    const int b = idx % a.B;
    const int layer = idx / a.B;
    const int L = a.seq_len[b];
    const int n = a.n_acc[b];
    // asked for together with the two above (the array is [B, T_max] whatever n_acc says): one round trip less
    const int path_in = (int)threadIdx.x < a.T_max ? a.path[(size_t)b * a.T_max + threadIdx.x] : -1;
    const int chunks = a.d / 8;

    if (threadIdx.x == 0) s_ok = 1;
    __syncthreads();
    bool bad = n < 0 || n > a.T_max || L < 0;
    if (!bad && threadIdx.x < n) {
        const int pj = path_in;
        s_path[threadIdx.x] = pj;
        if (pj < (int)threadIdx.x || pj >= a.T_max || (long long)L + pj >= a.S_cap) bad = true;
    }
    if (bad) s_ok = 0;
    __syncthreads();
    const bool first = h == 0 && layer == 0 && which == 0 && threadIdx.x == 0;
    if (!s_ok) {
        if (first) { a.new_seq_len[b] = L; atomicOr(status, (unsigned)GRAFT_FLAG_BAD_PATH); }
        return;
    }
    if (first) a.new_seq_len[b] = L + n;

    uint16_t* base = reinterpret_cast<uint16_t*>(which ? a.Vc : a.Kc) + (size_t)layer * a.layer_stride +
                     (a.block_table ? 0 : (size_t)b * a.kv_stride_b) + (size_t)h * a.kv_stride_h;
    // element offset of cache slot s of this sequence: contiguous, or through the block table (-1: entry out of range)
    const int32_t* table = a.block_table ? a.block_table + (size_t)b * a.blocks_per_seq : nullptr;
    auto slot = [&](int s) -> long long {
        if (!table) return (long long)s * a.kv_stride_s;
        const int blk = table[s / a.page_size];
        if (blk < 0 || blk >= a.n_blocks) return -1;
        return (long long)blk * a.kv_stride_b + (long long)(s % a.page_size) * a.kv_stride_s;
    };
    bool table_ok = true;
    for (int c = threadIdx.x; c < n * chunks; c += kThreads) {
        const int j = c / chunks, part = c % chunks;
        if (s_path[j] != j) {
            const long long src = slot(L + s_path[j]);
            if (src < 0) { table_ok = false; stage[c] = make_uint4(0u, 0u, 0u, 0u); }
            else stage[c] = *reinterpret_cast<const uint4*>(base + src + part * 8);
        }
    }
    __syncthreads();
    for (int c = threadIdx.x; c < n * chunks; c += kThreads) {
        const int j = c / chunks, part = c % chunks;
        if (s_path[j] != j) {
            const long long dst = slot(L + j);
            if (dst < 0) table_ok = false;
            else *reinterpret_cast<uint4*>(base + dst + part * 8) = stage[c];
        }
    }
    if (!table_ok) atomicOr(status, (unsigned)GRAFT_FLAG_BAD_SIZE);
}

}  // namespace

extern "C" int graft_compact_kv(graft_ctx* ctx, const graft_compact_params* p, void* stream) {
    if (!ctx || !p) return GRAFT_ERR_INVALID_ARG;
    if (p->B <= 0 || p->Hkv <= 0 || p->d <= 0 || p->S_cap <= 0 || p->T_max <= 0 || p->n_layers <= 0)
        return GRAFT_ERR_INVALID_ARG;
    if (p->T_max > 64 || p->d % 8 != 0 || p->d > 256) return GRAFT_ERR_UNSUPPORTED;
    if (!p->Kc || !p->Vc || !p->seq_len || !p->n_acc || !p->path || !p->new_seq_len) return GRAFT_ERR_INVALID_ARG;
    if (!graft_aligned16(p->Kc) || !graft_aligned16(p->Vc) || p->layer_stride % 8 || p->kv_stride_b % 8 ||
        p->kv_stride_h % 8 || p->kv_stride_s % 8 || p->kv_stride_s < p->d)
        return GRAFT_ERR_INVALID_ARG;
    if (p->block_table) {
        if (p->page_size <= 0 || p->page_size % 128 != 0 || p->blocks_per_seq <= 0 || p->n_blocks <= 0) return GRAFT_ERR_INVALID_ARG;
        if ((long long)p->blocks_per_seq * p->page_size < p->S_cap) return GRAFT_ERR_INVALID_ARG;
    }
    const long long ctas = 2ll * p->B * p->Hkv * p->n_layers;
    if (ctas > 0x7fffffffll) return GRAFT_ERR_UNSUPPORTED;
    const size_t smem = (size_t)p->T_max * (p->d / 8) * sizeof(uint4);     // <= 32 KB
    GRAFT_CHECK_CUDA(graft_launch(compact_kernel, dim3((unsigned)ctas), dim3(kThreads), smem, (cudaStream_t)stream, *p, ctx->status));
    return GRAFT_OK;
}
