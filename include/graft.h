/*
 * graft.h - C ABI of the B200 (sm_100a) tree-verify path of a prune-then-graft speculative
 * decoding step.
 *
 * One decoding round (the paper's Algorithm 1, loop body) verifies a hybrid draft tree against the
 * target model's KV cache.  Per layer-step the caller runs, on one CUDA stream and without any host
 * synchronisation in between:
 *
 *     graft_retrieve_envelope retrieval section: the root-centred template filled from M, on a side stream
 *                             while the draft model runs (optional: graft_build_tree can do its own lookups)
 *     graft_build_tree        Algorithm 2 from "Resolve (K_draft, K_ret)" on: prune, graft, rebuild
 *     graft_path_indices      Sec. 3.3: the candidate-path table of the flattened tree (optional output)
 *     [caller: QKV projection writes the tree tokens' K/V to cache slots L_b .. L_b + T_b - 1]
 *     graft_tree_verify_attn  Sec. 3.3: tree attention of the T tree tokens over cache + ancestors
 *     [caller: lm_head gives the target logits of the tree nodes]
 *     graft_update_adjacency  retrieval section / appendix: M[x_i] <- argtopk(p_{i+1}); also target_next
 *     graft_accept            Algorithm 1 "select the accepted path" (greedy, lossless); under temperature
 *                             sampling graft_accept_stochastic takes its place
 *     graft_compact_kv        Algorithm 1 "append accepted tokens and update target KV cache"
 *
 * Conventions
 *   - Every array pointer in a params struct is a DEVICE pointer owned by the caller; the library
 *     never frees or keeps it beyond the call.  Scalars are host values.  The params struct itself
 *     is host memory and is read before the call returns.
 *   - All calls are asynchronous on `stream` (a cudaStream_t passed as void*), allocate nothing and
 *     never synchronise, except graft_create / graft_destroy / graft_device_status.
 *   - Return value: GRAFT_OK or a negative GRAFT_ERR_*.  Argument checks look only at scalars and
 *     null pointers and happen before any launch.  Data-dependent faults (a parent pointing forward,
 *     a tree larger than T_max, a cached length that would overflow S_cap, a token id outside
 *     [-1, V)) set GRAFT_FLAG_* bits in a device status word and the kernel writes a defined result
 *     for that sequence instead of faulting; read them with graft_device_status.
 *   - Notation: B sequences, H_q query heads, H_kv KV heads, G = H_q / H_kv, head dim d, L_b cached
 *     prefix length, T_b tree size (<= T_max <= 64), S_cap cache slots per sequence.  Node 0 of a tree
 *     is the root (the current token, already sampled by the target; parent -1); parent[i] < i.
 *   - Padding (so that whole buffers compare bit for bit): nodes i >= T_b have token -1, parent -1,
 *     pos 0, anc 0, src INT32_MIN; path[j >= n_acc] = -1; O rows t >= T_b are zero, LSE there -inf.
 *   - One graft_ctx per stream; calls on one ctx must not overlap on the GPU.
 *   - Launch configurations depend only on the scalars of a params struct (shapes, variant), never on device
 *     data, and no call keeps per-call state on the host: a sequence of calls can be captured in a CUDA graph
 *     once and replayed after the contents of its buffers changed (lengths, trees, K/V, random numbers).
 */
#ifndef GRAFT_H_
#define GRAFT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct graft_ctx graft_ctx;

enum {
    GRAFT_OK = 0,
    GRAFT_ERR_INVALID_ARG = -1,        /* null pointer, non-positive size, misaligned base or stride   */
    GRAFT_ERR_UNSUPPORTED = -2,        /* T_max > 64, d not in {64,128}, H_q % H_kv != 0, k > 16 ...    */
    GRAFT_ERR_WORKSPACE_TOO_SMALL = -3,
    GRAFT_ERR_CUDA = -4,               /* a CUDA runtime call or launch failed                          */
    GRAFT_ERR_SCRATCH_LIMIT = -5       /* graft_tree_verify_attn_noalloc: shape exceeds the built-in scratch */
};

/* bits of the device status word */
enum {
    GRAFT_FLAG_BAD_SIZE = 1,      /* n_draft, budget, tree_size or cached length out of range: empty result */
    GRAFT_FLAG_BAD_PARENT = 2,    /* parent[i] not in [0, i): node dropped with its subtree                 */
    GRAFT_FLAG_BAD_TOKEN = 4,     /* token id outside [-1, V): replaced by -1                               */
    GRAFT_FLAG_ORPHAN = 8,        /* selected node whose parent was not selected: dropped                   */
    GRAFT_FLAG_BUDGET = 16,       /* more kept nodes than the budget: the excess (in node order) dropped    */
    GRAFT_FLAG_BAD_TEMPLATE = 32, /* template parent or rank out of range: node hangs off the root, token -1 */
    GRAFT_FLAG_NAN_SCORE = 64,    /* NaN score: treated as -inf                                             */
    GRAFT_FLAG_BAD_PATH = 128,    /* compaction: n_acc or a path entry out of range: sequence left untouched */
    GRAFT_FLAG_WAIT_TIMEOUT = 256,/* a bounded wait inside a kernel gave up (output of that launch invalid) */
    GRAFT_FLAG_INTERNAL = 512     /* a kernel found its own set-up inconsistent and did not run (output invalid) */
};

/* prune modes of graft_build_tree */
enum {
    GRAFT_PRUNE_NONE = 0,   /* no pruning triggered: the base tree, nothing grafted (Alg. 2, "no pruning")   */
    GRAFT_PRUNE_TOPK = 1,   /* keep the top keep_count[b] nodes by cumulative path score (Alg. 2)          */
    GRAFT_PRUNE_GATED = 2,  /* checkpoint gating g_d = 1[exp(max_j S_dj) > tau_d] picks the stage (Sec. 3.1) */
    GRAFT_PRUNE_NODE = 3    /* batched rule: drop low-confidence nodes of depth >= gate_depth with their
                               subtrees and refill the freed slots (high-concurrency appendix)             */
};

/* attention kernel choice */
enum {
    GRAFT_ATTN_AUTO = 0,
    GRAFT_ATTN_MMA_SYNC = 1,   /* register-tile kernel (any supported shape; the low-row path)    */
    GRAFT_ATTN_TCGEN05 = 2,    /* TMA + tcgen05/TMEM kernels (d = 128): one of the two below        */
    GRAFT_ATTN_TCGEN05_1SM = 3,/* ... one CTA per SM holds both 128-row blocks of an item           */
    GRAFT_ATTN_TCGEN05_2SM = 4,/* ... a pair of SMs shares every tile (two-SM MMAs)                 */
    GRAFT_ATTN_TCGEN05_L2PAIR = 5 /* ... one 128-row block per SM, partner SMs share tiles through L2 */
};

/* ---- context --------------------------------------------------------------------------------- */

/* Upper bound, in bytes, of the workspace the four calls need for these shapes on `device`
 * (host-only: queries the SM count).  Returns 0 for unsupported shapes. */
size_t graft_workspace_bytes(int device, int B, int Hq, int Hkv, int d, int T_max);

/* Creates a context bound to `device` and to a caller-owned device workspace (256-byte aligned) that
 * must outlive the context.  The first 256 bytes hold the status word and are cleared here
 * (synchronous).  Nothing else is allocated on the device. */
int graft_create(graft_ctx** out, int device, void* workspace, size_t workspace_bytes);
int graft_destroy(graft_ctx* ctx);                       /* never frees caller memory */
const char* graft_status_string(int status);
/* Synchronises `stream`, returns the accumulated GRAFT_FLAG_* bits and, if `clear`, zeroes them. */
int graft_device_status(graft_ctx* ctx, void* stream, unsigned* flags_out, int clear);

/* ---- graft_build_tree ------------------------------------------------------------------------ */
/*
 * Prune the draft tree, graft retrieved tokens into the freed slots, and rebuild the arrays the
 * verifier consumes (Algorithm 2 from "Resolve (K_draft, K_ret)"; Sec. 3.2, T_s = T_s^draft U G_s^ret
 * with |T_s| = K_max; Sec. 3.3 "flattened ... rebuilds position IDs, ancestor mask").  Per sequence:
 *   1. depth of every draft node (input order is topological).
 *   2. keep-set by `mode`.  TOPK: root plus the keep_count[b]-1 best other nodes by (score desc,
 *      index asc).  GATED: checkpoints in order; checkpoint c reads smax = max score over nodes of
 *      depth ckpt_depth[c]; the first with smax <= ckpt_log_tau[c] (c_d <= tau_d) fixes the stage:
 *      K_draft = ckpt_keep[c], only nodes of depth <= ckpt_depth[c] are eligible, the template is
 *      tmpl[tmpl_offset[c] .. tmpl_offset[c+1]); no checkpoint fails -> keep all, graft nothing.
 *      NODE: a node goes if it or an ancestor has depth >= gate_depth and score < node_threshold.
 *   3. kept nodes keep their order; parents are re-indexed; at most budget = k_max[b] (else K_max).
 *   4. graft: the first K_ret = min(template length, budget - K_kept) template nodes follow, node u
 *      at index K_kept + u under the root (tmpl_parent[u] == -1) or under K_kept + tmpl_parent[u],
 *      token x_u = M[x_parent(u), tmpl_rank[u]] (Sec. 3.2 lookup equation); an empty row (-1)
 *      propagates -1.
 *   5. anc[i] = anc[parent[i]] | 1 << i (ancestor-or-self), pos[i] = L_b + popcount(anc[i]) - 1.
 * Integer outputs are exact.  tree_src[i] = draft index of a kept node, -1-u for template node u.
 */
typedef struct {
    int B, N_max, T_max, K_max, V, k, S_cap;
    int mode;
    int gate_depth;              /* NODE */
    float node_threshold;        /* NODE */
    int n_ckpt;                  /* GATED: number of checkpoints */
    int N_tmpl;                  /* length of tmpl_parent / tmpl_rank (all stages together) */
    const int32_t* draft_token;  /* [B, N_max] */
    const int32_t* draft_parent; /* [B, N_max], parent[0] = -1 */
    const float* draft_score;    /* [B, N_max] cumulative path score (TOPK, GATED) or confidence (NODE) */
    const int32_t* n_draft;      /* [B] */
    const int32_t* seq_len;      /* [B] L_b */
    const int32_t* M;            /* [V, k] adjacency matrix, -1 = empty */
    const int32_t* keep_count;   /* [B], TOPK only */
    const int32_t* k_max;        /* [B] per-sequence budget, or NULL for K_max */
    const int32_t* ckpt_depth;   /* [n_ckpt] GATED */
    const int32_t* ckpt_keep;    /* [n_ckpt] */
    const float* ckpt_log_tau;   /* [n_ckpt] natural log of tau_d */
    const int32_t* tmpl_offset;  /* [n_ckpt + 1] GATED */
    const int32_t* tmpl_parent;  /* [N_tmpl] index inside the stage's template, -1 = child of the root */
    const int32_t* tmpl_rank;    /* [N_tmpl] successor rank in [0, k) */
    int32_t* tree_token;         /* out [B, T_max] */
    int32_t* tree_parent;        /* out [B, T_max] */
    int32_t* tree_pos;           /* out [B, T_max] */
    int32_t* tree_src;           /* out [B, T_max] */
    uint64_t* tree_anc;          /* out [B, T_max], bit u of anc[t]: node u visible to node t */
    int32_t* tree_size;          /* out [B] */
    /* optional: tokens of a precomputed retrieval envelope (graft_retrieve_envelope).  With env_token
       set, template node u of the chosen stage takes env_token[b, tmpl_env[tmpl_offset[c] + u]]
       instead of its own chain of lookups in M; tmpl_parent still gives the tree structure.  The
       caller guarantees that the envelope node has the template node's rank path and that the
       envelope was filled from this call's root tokens and M; an index outside [0, N_env) sets
       GRAFT_FLAG_BAD_TEMPLATE and gives token -1. */
    int N_env;
    const int32_t* env_token;    /* [B, N_env] or NULL */
    const int32_t* tmpl_env;     /* [N_tmpl] */
    /* tail grafting for block drafters (the block-drafter appendix: keep the reliable prefix of the drafted chain
       "and attach retrieved tokens to the tail of the remaining chain"): with attach_tail != 0 a template node
       whose parent is -1 hangs off the last kept node (index K_kept - 1) instead of the root, and its token is
       looked up from that node's token.  Not together with env_token (the envelope is root-centred). */
    int attach_tail;
} graft_build_params;

int graft_build_tree(graft_ctx* ctx, const graft_build_params* p, void* stream);

/* ---- graft_retrieve_envelope ----------------------------------------------------------------- */
/*
 * Root-centred retrieval envelope (retrieval section, "Lightweight parallel retrieval": the envelope is
 * materialised in parallel with drafting and a stage-matched part of it is selected afterwards; template
 * appendix: x_u = M[x_F(u), r_u], filled level by level from the root token).  The template is a list of
 * N_env nodes, node u with env_parent[u] in [-1, u) (-1: child of the root) and env_rank[u] in [0, k).
 * env_token[b, u] is the token of node u for request b; an empty row of M (-1) or a root of -1 makes
 * the whole subtree -1.  Root ids and matrix entries outside [-1, V) count as -1 (GRAFT_FLAG_BAD_TOKEN);
 * a node with a parent index or rank out of range gets -1 (GRAFT_FLAG_BAD_TEMPLATE).
 * Request b's root is root_token[b * root_stride] (pass draft_token and N_max to read node 0 of the
 * draft trees in place).  N_env <= 1024, k <= 16.  The call reads only the root tokens, M and the
 * template, so it may run on another stream than the rest of the step; the caller orders it before
 * graft_build_tree (an event) and after the previous step's graft_update_adjacency.
 */
typedef struct {
    int B, V, k, N_env;
    const int32_t* root_token;   /* request b's root at [b * root_stride] */
    int64_t root_stride;
    const int32_t* M;            /* [V, k] */
    const int32_t* env_parent;   /* [N_env] */
    const int32_t* env_rank;     /* [N_env] */
    int32_t* env_token;          /* out [B, N_env] */
} graft_envelope_params;

int graft_retrieve_envelope(graft_ctx* ctx, const graft_envelope_params* p, void* stream);

/* ---- graft_path_indices ---------------------------------------------------------------------- */
/*
 * Candidate-path indices of the flattened tree (Sec. 3.3: "rebuilds the standard tree position IDs,
 * ancestor mask, and candidate-path indices"): one row per leaf, leaves in increasing node index; a row
 * lists the node indices from the root (0) to the leaf and then -1 up to D_max columns; rows past the
 * last leaf hold -1.  n_paths[b] = number of leaves (0 for an empty tree).  A leaf deeper than
 * D_max - 1 keeps the first D_max nodes of its path and sets GRAFT_FLAG_BAD_SIZE, as does a
 * tree_size outside [0, T_max] (no paths).  tree_parent must satisfy parent[i] < i (as
 * graft_build_tree writes it).  T_max <= 64, 1 <= D_max <= 64.
 */
typedef struct {
    int B, T_max, D_max;
    const int32_t* tree_parent;  /* [B, T_max] */
    const int32_t* tree_size;    /* [B] */
    int32_t* path_index;         /* out [B, T_max, D_max] */
    int32_t* n_paths;            /* out [B] */
} graft_paths_params;

int graft_path_indices(graft_ctx* ctx, const graft_paths_params* p, void* stream);

/* ---- graft_tree_verify_attn ------------------------------------------------------------------ */
/*
 * Tree-masked grouped-query attention (Sec. 3.3, "sends the whole hybrid tree to the target model in
 * one parallel verification pass" with the standard ancestor mask):
 *   O[b,t,h,:] = sum_j softmax_j(scale * q[b,t,h] . k_j) v_j,   j over cache slots 0 .. L_b-1 and
 *   L_b + u for every set bit u of tree_anc[b,t];  K/V of KV head h / G.
 * bf16 inputs, fp32 scores / softmax / accumulation, bf16 output (round to nearest even), optional
 * fp32 natural-log LSE.  The KV axis is split over CTAs; partial (max, sum, O) triples go to the
 * workspace and are merged with the online-softmax rule.  The split schedule is a pure function of
 * (seq_len, tree_size, SM count), so results are reproducible on one GPU model.
 * Strides are in elements; the last (d) axis is contiguous.  Q, K, V, O bases and all strides must be
 * multiples of 8 elements (16 bytes).  Cache slots at or beyond L_b + T_b are never read into a
 * result (they may hold NaN bit patterns).
 */
typedef struct {
    int B, T_max, Hq, Hkv, d, S_cap;
    float scale;
    int variant;                                     /* GRAFT_ATTN_* */
    const void* Q;  int64_t q_stride_b, q_stride_t, q_stride_h;   /* bf16 [B, T_max, Hq, d] */
    const void* Kc; const void* Vc;                                /* bf16 [B, Hkv, S_cap, d] */
    int64_t kv_stride_b, kv_stride_h, kv_stride_s;
    void* O;        int64_t o_stride_b, o_stride_t, o_stride_h;   /* bf16 [B, T_max, Hq, d] */
    float* LSE;                                      /* optional [B, Hq, T_max] */
    const int32_t* seq_len;                          /* [B] */
    const int32_t* tree_size;                        /* [B] */
    const uint64_t* tree_anc;                        /* [B, T_max] */
    /* paged caches (optional; serving-shaped variant).  With block_table set, Kc / Vc are pools
       [n_blocks, Hkv, page_size, d] (kv_stride_b = elements between blocks) and cache slot s of sequence b
       lives in block block_table[b * blocks_per_seq + s / page_size] at row s % page_size.  page_size is a
       multiple of 128; S_cap <= blocks_per_seq * page_size.  A table entry outside [0, n_blocks) reads as
       zeros and sets GRAFT_FLAG_BAD_SIZE.  Slots past L_b + T_b may hold anything, as in the contiguous layout. */
    const int32_t* block_table;                      /* [B, blocks_per_seq] or NULL */
    int page_size, blocks_per_seq, n_blocks;
} graft_attn_params;

int graft_tree_verify_attn(graft_ctx* ctx, const graft_attn_params* p, void* stream);

/*
 * The same attention for callers that cannot allocate device memory (the paper has no counterpart:
 * this is a packaging variant, not a step of the method).  A caller may be unable to allocate
 * because its process gave all device memory to a fixed pool at start-up, because it runs inside a
 * latency-critical section where cudaMalloc's device-wide synchronisation is not acceptable, or
 * because it is a thin shim with no allocator in reach.  No graft_ctx and no workspace are needed:
 * the split-KV partials and the status word live in one static device array of
 * graft_noalloc_scratch_bytes() (40 MiB) that every GPU loading this library holds until the process
 * exits.  The call allocates nothing (no cudaMalloc, cudaFree or allocating library routine).
 *   - p: exactly as for graft_tree_verify_attn; inputs and outputs still belong to the caller.
 *   - device_flags_out: optional DEVICE pointer; receives the GRAFT_FLAG_* word of this call (copied on
 *     `stream`), or NULL.
 *   - The first call on a device (made with that device current) resolves the array's device address
 *     and configures the kernels; make it before any stream capture.
 *   - Shapes whose partials do not fit the array are rejected with GRAFT_ERR_SCRATCH_LIMIT before any
 *     launch (with GRAFT_ATTN_AUTO the call falls back from the tcgen05 kernel to the register-tile
 *     kernel when only the latter's partials fit).
 *   - All calls on a GPU share the one array, which keeps the previous call's contents; the call clears
 *     the status word itself.  Two calls that overlap on the GPU (different streams) race: serialise
 *     them.
 */
size_t graft_noalloc_scratch_bytes(void);
int graft_tree_verify_attn_noalloc(const graft_attn_params* p, void* stream, unsigned* device_flags_out);

/* ---- graft_update_adjacency ------------------------------------------------------------------- */
/*
 * Online refresh of the retrieval matrix (retrieval section and appendix, "M[x_i] <- argtopk(p_{i+1})",
 * over the whole verified tree, accepted and rejected nodes, all requests in one flattened batch), and
 * the target's greedy ids for graft_accept.  Row r = b * T_max + i of `logits` holds the target's
 * next-token logits at tree node i of sequence b (softmax is monotone: the ids of the k largest logits
 * are those of the k largest probabilities).  For every node i < tree_size[b] with a token x in [0, V):
 * M[x, 0..k) <- the ids of the k largest logits of row r, by decreasing logit, equal logits by increasing
 * id; NaN is never chosen (GRAFT_FLAG_NAN_SCORE and -1 entries if fewer than k logits are not NaN).
 * When several nodes of the step carry the same token, the node with the highest r wins.  Rows of M of
 * other tokens do not change.  target_next[r] (optional) <- the first id of the list, -1 for padding
 * nodes.  Token -1 updates nothing; any other id outside [0, V) sets GRAFT_FLAG_BAD_TOKEN.
 * k <= 16; logits: 16-byte aligned base, row stride a multiple of 8 elements.
 */
typedef struct {
    int B, T_max, V, k;
    const void* logits; int64_t logits_stride_row;   /* bf16 [B * T_max, V] */
    const int32_t* tree_token;   /* [B, T_max] */
    const int32_t* tree_size;    /* [B] */
    int32_t* M;                  /* [V, k], updated in place */
    int32_t* target_next;        /* out [B, T_max], may be NULL */
} graft_update_params;

int graft_update_adjacency(graft_ctx* ctx, const graft_update_params* p, void* stream);

/* ---- graft_accept ---------------------------------------------------------------------------- */
/*
 * Greedy lossless acceptance (Algorithm 1, "select the accepted path with the standard speculative
 * decoding acceptance rule"; greedy decoding as in the paper's main experiments): node i matches when
 * tree_token[i] >= 0 and equals target_next[parent[i]]; it is accepted when it and all its ancestors
 * match (the root always is).  The deepest accepted node wins, ties by lowest index.  path lists the
 * nodes from the root to it, n_acc = its depth + 1, bonus = target_next[best].  tree_anc must be the
 * ancestor-or-self mask of tree_parent (as graft_build_tree writes it).
 */
typedef struct {
    int B, T_max;
    const int32_t* tree_token;   /* [B, T_max] */
    const int32_t* tree_parent;  /* [B, T_max] */
    const uint64_t* tree_anc;    /* [B, T_max] */
    const int32_t* tree_size;    /* [B] */
    const int32_t* target_next;  /* [B, T_max] the target's greedy id after node i */
    int32_t* n_acc;              /* out [B] */
    int32_t* path;               /* out [B, T_max] */
    int32_t* best_node;          /* out [B] */
    int32_t* bonus;              /* out [B] */
} graft_accept_params;

int graft_accept(graft_ctx* ctx, const graft_accept_params* p, void* stream);

/* ---- graft_accept_stochastic ------------------------------------------------------------------ */
/*
 * Acceptance under temperature sampling (temperature-sampling discussion; lossless-equivalence
 * proposition: the tree is verified "with the standard speculative sampling rule", a rejected position is
 * "resampled from the target correction distribution").  The tree's candidates are fixed tokens, so at a
 * node u with p = softmax(logits[u] / temperature) the children of u are tried in node order: child c with
 * token x is accepted iff u_accept[b, c] * rem < p(x), where rem (1 at first) is the mass p still holds; a
 * rejected child's token loses its mass (rem -= p(x), p(x) = 0: the correction distribution for a point-mass
 * proposal).  An accepted child becomes u.  When no child is accepted, or u is a leaf, the bonus token is
 * the smallest id whose running sum of the remaining mass (ids in increasing order) exceeds
 * u_bonus[b] * rem.  Children with token -1 or with a token that a rejected sibling carried are never
 * accepted.  Outputs as graft_accept: path (root first, -1 padded), n_acc = nodes on it, best_node = its
 * last node, bonus.  Random numbers are inputs in [0, 1).
 * Arithmetic is fp32 (row maxima and exponential sums over V entries, running sums of the bonus draw), so
 * an outcome is only defined up to that rounding when a random number falls within ~1e-5 (relative to
 * rem) of a decision boundary.
 * row_stats: caller-provided scratch of graft_accept_stochastic_scratch_floats(B, T_max, V) floats (per row the
 * max of logits / temperature and the sum of exponentials, of the parts of the row that one CTA each scans and of
 * every 256 ids).
 * logits: 16-byte aligned base, row stride a multiple of 8 elements; temperature > 0; T_max <= 64; V <= 524288.
 */
typedef struct {
    int B, T_max, V;
    float temperature;
    const void* logits; int64_t logits_stride_row;   /* bf16 [B * T_max, V] */
    const int32_t* tree_token;   /* [B, T_max] */
    const int32_t* tree_parent;  /* [B, T_max] */
    const int32_t* tree_size;    /* [B] */
    const float* u_accept;       /* [B, T_max] */
    const float* u_bonus;        /* [B] */
    float* row_stats;            /* scratch, see above */
    int32_t* n_acc;              /* out [B] */
    int32_t* path;               /* out [B, T_max] */
    int32_t* best_node;          /* out [B] */
    int32_t* bonus;              /* out [B] */
} graft_accept_stochastic_params;

size_t graft_accept_stochastic_scratch_floats(int B, int T_max, int V);     /* host only; 0 for invalid sizes */
int graft_accept_stochastic(graft_ctx* ctx, const graft_accept_stochastic_params* p, void* stream);

/* ---- graft_compact_kv ------------------------------------------------------------------------ */
/*
 * KV update after acceptance (Algorithm 1, "append accepted tokens and update target KV cache"): for
 * every layer, KV head and j < n_acc[b], cache[b, h, L_b + j, :] <- cache[b, h, L_b + path[b, j], :],
 * K and V, in place; new_seq_len[b] = L_b + n_acc[b].  No other slot changes.  Source and
 * destination ranges overlap (path[j] >= j): each CTA stages all source rows on chip before it stores.
 * Layers are layer_stride elements apart inside Kc and Vc.
 */
typedef struct {
    int B, Hkv, d, S_cap, T_max, n_layers;
    int64_t layer_stride, kv_stride_b, kv_stride_h, kv_stride_s;
    void* Kc; void* Vc;          /* bf16, in place */
    const int32_t* seq_len;      /* [B] */
    const int32_t* n_acc;        /* [B] */
    const int32_t* path;         /* [B, T_max] */
    int32_t* new_seq_len;        /* out [B] */
    /* paged caches, as in graft_attn_params (one table for all layers; layer_stride between the layers' pools) */
    const int32_t* block_table;  /* [B, blocks_per_seq] or NULL */
    int page_size, blocks_per_seq, n_blocks;
} graft_compact_params;

int graft_compact_kv(graft_ctx* ctx, const graft_compact_params* p, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* GRAFT_H_ */
