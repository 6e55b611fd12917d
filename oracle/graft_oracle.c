/*
 * CPU oracle for the tree-verify path of a prune-then-graft speculative decoding step.
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, slow, written to be checked against the paper by eye.
 * It shares nothing with the CUDA library (no header, helper, table or constant), and only
 * tests, the smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * Floating point is fp64 throughout; bf16 inputs are widened exactly.  The only
 * parallelism is an OpenMP loop over independent output rows of the attention.
 *
 * Pins (see tests/test_oracle_*.py): brute force over dense masks and explicit path
 * enumeration on tiny trees; chain tree == causal attention (library SDPA); T = 1 == plain
 * decode attention; row sums == 1; locality of the ancestor mask; split invariance;
 * the paper's stage budgets 8+52 / 24+36 / 40+20 and template depth histograms; the
 * closed form x_u = M[x_parent(u), r_u]; Propositions 1 and 2 (monotone accepted length);
 * the adjacency update against a library stable sort, against softmax probabilities, a hand-worked
 * row with ties / NaN / -inf, and the sequential definition of the duplicate-token winner;
 * the retrieval envelope against the lookup equation folded along explicit rank paths, a shift matrix
 * with a closed form, the tree assembly's own lookups and the printed shape of the full template
 * (80 nodes, 8+16+14+11+8+7+6+5+5 over depths 1..9); the candidate-path table against a top-down
 * enumeration, chain and star trees, and acceptance written over paths; stochastic acceptance against
 * a hand-worked three-token example, the empirical distribution of the first emitted token and of the
 * second given the first over 200000 draws (lossless equivalence), and greedy acceptance in the
 * low-temperature limit.
 * Parity unpinned: nothing beyond the printed per-depth counts fixes the retrieval
 * templates' exact rank paths; they are inputs here, not computed.
 */
#include <limits.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* prune modes (Algorithm 2 and the batched variant of the high-concurrency appendix) */
enum { ORC_MODE_NONE = 0, ORC_MODE_TOPK = 1, ORC_MODE_GATED = 2, ORC_MODE_NODE = 3 };

/* status bits reported per call (malformed inputs have a defined result, never a crash) */
enum {
    ORC_FLAG_BAD_SIZE = 1,    /* n_draft, budget or cached length out of range: empty tree */
    ORC_FLAG_BAD_PARENT = 2,  /* parent[i] not in [0, i): node dropped                     */
    ORC_FLAG_BAD_TOKEN = 4,   /* token id outside [-1, V): replaced by -1                  */
    ORC_FLAG_ORPHAN = 8,      /* selected node whose parent was not selected: dropped      */
    ORC_FLAG_BUDGET = 16,     /* more kept nodes than the budget: truncated                */
    ORC_FLAG_BAD_TEMPLATE = 32, /* template parent/rank out of range: token -1             */
    ORC_FLAG_NAN_SCORE = 64   /* NaN score: treated as -inf                                */
};

typedef struct {
    int B, N_max, T_max, K_max, V, k, S_cap;
    int mode;
    int gate_depth;          /* MODE_NODE */
    float node_threshold;    /* MODE_NODE: a node of depth >= gate_depth with score < this goes */
    int n_ckpt;              /* MODE_GATED */
    int N_tmpl;              /* length of tmpl_parent / tmpl_rank (all stages together) */
    const int32_t *draft_token, *draft_parent; /* [B, N_max] */
    const float *draft_score;                  /* [B, N_max] */
    const int32_t *n_draft;                    /* [B] */
    const int32_t *seq_len;                    /* [B] */
    const int32_t *M;                          /* [V, k] */
    const int32_t *keep_count;                 /* [B] (MODE_TOPK) */
    const int32_t *k_max;                      /* [B] or NULL -> K_max */
    const int32_t *ckpt_depth, *ckpt_keep;     /* [n_ckpt] */
    const float *ckpt_log_tau;                 /* [n_ckpt] */
    const int32_t *tmpl_offset;                /* [n_ckpt + 1] (MODE_GATED) */
    const int32_t *tmpl_parent, *tmpl_rank;    /* [N_tmpl] */
    int32_t *tree_token, *tree_parent, *tree_pos, *tree_src; /* [B, T_max] */
    uint64_t *tree_anc;                                      /* [B, T_max] */
    int32_t *tree_size;                                      /* [B] */
    int attach_tail;         /* 0: template nodes with parent -1 hang off the root; 1: off the last kept node (tail grafting) */
} orc_build_args;

static int popcount64(uint64_t x) {
    int c = 0;
    while (x) { c += (int)(x & 1u); x >>= 1; }
    return c;
}

/* order used by "keep the top K draft nodes by cumulative path score" (Alg. 2):
   higher score first, equal scores by lower index */
static int better(const float *s, int a, int b) {
    if (s[a] > s[b]) return 1;
    if (s[a] < s[b]) return 0;
    return a < b;
}

/*
 * Tree assembly for one step (Algorithm 2, "Resolve (K_draft, K_ret)" onwards; Sec. 3.2 last
 * equation T_s = T_s^draft U G_s^ret; Sec. 3.3 first paragraph: flatten, rebuild position ids
 * and the ancestor mask).  Returns the OR of the status bits over the batch.
 */
unsigned orc_build_tree(const orc_build_args *a) {
    unsigned flags = 0;
    for (int b = 0; b < a->B; ++b) {
        int32_t *o_tok = a->tree_token + (size_t)b * a->T_max;
        int32_t *o_par = a->tree_parent + (size_t)b * a->T_max;
        int32_t *o_pos = a->tree_pos + (size_t)b * a->T_max;
        int32_t *o_src = a->tree_src + (size_t)b * a->T_max;
        uint64_t *o_anc = a->tree_anc + (size_t)b * a->T_max;
        for (int i = 0; i < a->T_max; ++i) {      /* padding first */
            o_tok[i] = -1; o_par[i] = -1; o_pos[i] = 0; o_src[i] = INT_MIN; o_anc[i] = 0;
        }
        a->tree_size[b] = 0;

        const int n = a->n_draft[b];
        const int budget = a->k_max ? a->k_max[b] : a->K_max;
        const int L = a->seq_len[b];
        if (n < 1 || n > a->N_max || budget < 1 || budget > a->T_max || budget > 64 ||
            L < 0 || (long long)L + a->T_max > a->S_cap) {
            flags |= ORC_FLAG_BAD_SIZE;
            continue;
        }
        const int32_t *tok = a->draft_token + (size_t)b * a->N_max;
        const int32_t *par = a->draft_parent + (size_t)b * a->N_max;
        const float *raw = a->draft_score + (size_t)b * a->N_max;

        int depth[64], valid[64], sel[64], kept[64], newidx[64];
        float s[64];
        /* 1. depths (input order is topological); a node with a bad parent is dropped */
        for (int i = 0; i < n; ++i) {
            s[i] = raw[i];
            if (s[i] != s[i]) { s[i] = -INFINITY; if (i > 0) flags |= ORC_FLAG_NAN_SCORE; }
            if (i == 0) { depth[0] = 0; valid[0] = 1; continue; }
            if (par[i] < 0 || par[i] >= i) { valid[i] = 0; depth[i] = 0; flags |= ORC_FLAG_BAD_PARENT; }
            else { valid[i] = valid[par[i]]; depth[i] = depth[par[i]] + 1; }
        }

        /* 2. the keep-set */
        int graft = 1;                  /* whether retrieved nodes are appended       */
        int t_lo = 0, t_hi = a->N_tmpl; /* the stage's template inside tmpl_* arrays  */
        for (int i = 0; i < n; ++i) sel[i] = valid[i];
        if (a->mode == ORC_MODE_NONE) {
            graft = 0;                  /* no pruning -> the base tree, no grafting   */
        } else if (a->mode == ORC_MODE_TOPK || a->mode == ORC_MODE_GATED) {
            int K_draft = n, max_depth = INT_MAX;
            if (a->mode == ORC_MODE_TOPK) {
                K_draft = a->keep_count[b];
            } else {
                /* checkpoint gating: c_d = exp(max_j S_{d,j}); g_d = 1[c_d > tau_d];
                   the first checkpoint with g_d = 0 fixes the stage.  Compared as
                   max_j S_{d,j} <= log(tau_d). */
                int stage = -1;
                for (int c = 0; c < a->n_ckpt && stage < 0; ++c) {
                    float smax = -INFINITY;
                    for (int i = 1; i < n; ++i)
                        if (valid[i] && depth[i] == a->ckpt_depth[c] && s[i] > smax) smax = s[i];
                    if (smax <= a->ckpt_log_tau[c]) stage = c;
                }
                if (stage < 0) { graft = 0; }       /* survived every checkpoint */
                else {
                    K_draft = a->ckpt_keep[stage];
                    max_depth = a->ckpt_depth[stage]; /* deeper expansion was skipped */
                    t_lo = a->tmpl_offset[stage];
                    t_hi = a->tmpl_offset[stage + 1];
                }
            }
            if (graft || a->mode == ORC_MODE_TOPK) {
                /* root always kept and counted; then the best K_draft-1 eligible nodes */
                int order[64], m = 0;
                for (int i = 1; i < n; ++i) {
                    sel[i] = 0;
                    if (valid[i] && depth[i] <= max_depth) order[m++] = i;
                }
                for (int x = 1; x < m; ++x) {        /* insertion sort by `better` */
                    int v = order[x], y = x - 1;
                    while (y >= 0 && better(s, v, order[y])) { order[y + 1] = order[y]; --y; }
                    order[y + 1] = v;
                }
                for (int x = 0; x < m && x < K_draft - 1; ++x) sel[order[x]] = 1;
            }
        } else { /* ORC_MODE_NODE: a low-confidence node at or below the gate depth goes,
                    and so does everything under it */
            for (int i = 1; i < n; ++i) {
                if (!valid[i]) { sel[i] = 0; continue; }
                int removed = !sel[par[i]] || (depth[i] >= a->gate_depth && s[i] < a->node_threshold);
                sel[i] = !removed;
            }
        }

        /* 3. stable compaction; a selected node needs its parent in the tree */
        int K_kept = 0;
        for (int i = 0; i < n; ++i) {
            kept[i] = 0;
            if (!sel[i]) continue;
            if (K_kept == budget) { flags |= ORC_FLAG_BUDGET; continue; }
            if (i > 0 && !kept[par[i]]) { flags |= ORC_FLAG_ORPHAN; continue; }
            kept[i] = 1;
            newidx[i] = K_kept++;
        }
        for (int i = 0; i < n; ++i) {
            if (!kept[i]) continue;
            int j = newidx[i];
            int t = tok[i];
            if (t < -1 || t >= a->V) { t = -1; flags |= ORC_FLAG_BAD_TOKEN; }
            o_tok[j] = t;
            o_par[j] = i == 0 ? -1 : newidx[par[i]];
            o_src[j] = i;
        }

        /* 4. graft: the first K_ret nodes of the stage template, x_u = M[x_parent(u), r_u] */
        int T = K_kept;
        if (graft) {
            int K_ret = t_hi - t_lo;
            if (K_ret > budget - K_kept) K_ret = budget - K_kept;
            if (K_ret < 0) K_ret = 0;
            for (int u = 0; u < K_ret; ++u) {
                int tp = a->tmpl_parent[t_lo + u], r = a->tmpl_rank[t_lo + u];
                int j = K_kept + u, ok = 1;
                if (tp < -1 || tp >= u || r < 0 || r >= a->k) { ok = 0; flags |= ORC_FLAG_BAD_TEMPLATE; }
                /* root-centred template, or (block drafters' "keep the reliable prefix and attach retrieved tokens to the
                   tail of the remaining chain") the template continues the last kept node */
                const int attach = a->attach_tail && K_kept > 0 ? K_kept - 1 : 0;
                int p = (!ok || tp == -1) ? attach : K_kept + tp;
                int ptok = o_tok[p], x = -1;
                if (ok && ptok >= 0) {
                    x = a->M[(size_t)ptok * a->k + r];
                    if (x < -1 || x >= a->V) { x = -1; flags |= ORC_FLAG_BAD_TOKEN; }
                }
                o_tok[j] = x;
                o_par[j] = p;
                o_src[j] = -1 - u;
            }
            T += K_ret;
        }

        /* 5. ancestor-or-self bitmask and position ids */
        for (int i = 0; i < T; ++i) {
            o_anc[i] = (i == 0 ? 0 : o_anc[o_par[i]]) | ((uint64_t)1 << i);
            o_pos[i] = L + popcount64(o_anc[i]) - 1;
        }
        a->tree_size[b] = T;
    }
    return flags;
}

/* ---------------------------------------------------------------------------------- */

static double bf16_to_double(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

typedef struct {
    int B, T_max, Hq, Hkv, d, S_cap;
    double scale;
    const uint16_t *Q;          /* bf16 bits [B, T_max, Hq, d] */
    const uint16_t *Kc, *Vc;    /* bf16 bits [B, Hkv, S_cap, d] */
    const int32_t *seq_len, *tree_size; /* [B] */
    const uint64_t *tree_anc;   /* [B, T_max] */
    double *O;                  /* [B, T_max, Hq, d]; rows t >= tree_size[b] are zero */
    double *LSE;                /* [B, Hq, T_max] natural log; -inf for padding rows  */
    double *rowsum;             /* [B, Hq, T_max] sum of the normalised weights        */
} orc_attn_args;

/*
 * One output row of tree-masked attention (Sec. 3.3: the tree is verified in one pass with the
 * standard ancestor mask): query (b, t, h) attends to the L_b cached keys and to the tree
 * nodes u with bit u of anc[b, t] set, whose K/V sit at cache slot L_b + u.
 * Plain three-pass softmax: scores, max, exp / sum.
 */
static void attn_row(const orc_attn_args *a, int b, int t, int h, double *score /* [S_cap] */) {
    const int d = a->d, G = a->Hq / a->Hkv, g = h / G;
    const int L = a->seq_len[b], T = a->tree_size[b];
    const uint64_t anc = a->tree_anc[(size_t)b * a->T_max + t];
    const uint16_t *q = a->Q + (((size_t)b * a->T_max + t) * a->Hq + h) * d;
    const uint16_t *K = a->Kc + ((size_t)b * a->Hkv + g) * a->S_cap * d;
    const uint16_t *V = a->Vc + ((size_t)b * a->Hkv + g) * a->S_cap * d;
    double *o = a->O + (((size_t)b * a->T_max + t) * a->Hq + h) * d;
    const size_t li = ((size_t)b * a->Hq + h) * a->T_max + t;

    double m = -INFINITY;
    for (int j = 0; j < L + T; ++j) {
        int visible = j < L || ((anc >> (j - L)) & 1u);
        if (!visible) { score[j] = -INFINITY; continue; }
        double acc = 0.0;
        for (int c = 0; c < d; ++c) acc += bf16_to_double(q[c]) * bf16_to_double(K[(size_t)j * d + c]);
        score[j] = a->scale * acc;
        if (score[j] > m) m = score[j];
    }
    for (int c = 0; c < d; ++c) o[c] = 0.0;
    double denom = 0.0;
    for (int j = 0; j < L + T; ++j) {
        if (score[j] == -INFINITY) continue;
        double p = exp(score[j] - m);
        denom += p;
        for (int c = 0; c < d; ++c) o[c] += p * bf16_to_double(V[(size_t)j * d + c]);
    }
    double wsum = 0.0;
    for (int j = 0; j < L + T; ++j)
        if (score[j] != -INFINITY) wsum += exp(score[j] - m) / denom;
    for (int c = 0; c < d; ++c) o[c] /= denom;
    if (a->LSE) a->LSE[li] = m + log(denom);
    if (a->rowsum) a->rowsum[li] = wsum;
}

/* all rows; returns the number of threads used */
int orc_tree_attn(const orc_attn_args *a) {
    int nthreads = 1;
    const long rows = (long)a->B * a->T_max * a->Hq;
#pragma omp parallel
    {
#ifdef _OPENMP
#pragma omp single
        nthreads = omp_get_num_threads();
#endif
        double *score = (double *)malloc(sizeof(double) * (size_t)a->S_cap);
#pragma omp for schedule(dynamic, 1)
        for (long r = 0; r < rows; ++r) {
            int h = (int)(r % a->Hq);
            int t = (int)((r / a->Hq) % a->T_max);
            int b = (int)(r / ((long)a->Hq * a->T_max));
            if (t < a->tree_size[b]) {
                attn_row(a, b, t, h, score);
            } else {
                double *o = a->O + (((size_t)b * a->T_max + t) * a->Hq + h) * a->d;
                for (int c = 0; c < a->d; ++c) o[c] = 0.0;
                size_t li = ((size_t)b * a->Hq + h) * a->T_max + t;
                if (a->LSE) a->LSE[li] = -INFINITY;
                if (a->rowsum) a->rowsum[li] = 0.0;
            }
        }
        free(score);
    }
    return nthreads;
}

/* selected rows only: rows[3*i + {0,1,2}] = (b, t, h); other entries of O/LSE are untouched */
int orc_tree_attn_rows(const orc_attn_args *a, int n_rows, const int32_t *rows) {
    int nthreads = 1;
#pragma omp parallel
    {
#ifdef _OPENMP
#pragma omp single
        nthreads = omp_get_num_threads();
#endif
        double *score = (double *)malloc(sizeof(double) * (size_t)a->S_cap);
#pragma omp for schedule(dynamic, 1)
        for (int i = 0; i < n_rows; ++i) {
            int b = rows[3 * i], t = rows[3 * i + 1], h = rows[3 * i + 2];
            if (t < a->tree_size[b]) attn_row(a, b, t, h, score);
        }
        free(score);
    }
    return nthreads;
}

/* ---------------------------------------------------------------------------------- */

typedef struct {
    int B, T_max;
    const int32_t *tree_token, *tree_parent; /* [B, T_max] */
    const int32_t *tree_size;                /* [B] */
    const int32_t *target_next;              /* [B, T_max]: the target's greedy id after node i */
    int32_t *n_acc, *best_node, *bonus;      /* [B] */
    int32_t *path;                           /* [B, T_max], padded with -1 */
} orc_accept_args;

/*
 * Greedy lossless acceptance (Alg. 1, "select the accepted path with the standard acceptance
 * rule"): a direct walk over the tree.  Node i is accepted when its parent is accepted and
 * its token equals the id the target produced at the parent; the deepest accepted node wins,
 * ties by lowest index.
 */
void orc_accept(const orc_accept_args *a) {
    for (int b = 0; b < a->B; ++b) {
        const int32_t *tok = a->tree_token + (size_t)b * a->T_max;
        const int32_t *par = a->tree_parent + (size_t)b * a->T_max;
        const int32_t *nxt = a->target_next + (size_t)b * a->T_max;
        int32_t *path = a->path + (size_t)b * a->T_max;
        const int T = a->tree_size[b];
        for (int j = 0; j < a->T_max; ++j) path[j] = -1;
        if (T < 1 || T > a->T_max) { a->n_acc[b] = 0; a->best_node[b] = -1; a->bonus[b] = -1; continue; }
        int ok[64], depth[64], best = 0;
        ok[0] = 1; depth[0] = 0;
        for (int i = 1; i < T; ++i) {
            int p = par[i];
            if (p < 0 || p >= i) { ok[i] = 0; depth[i] = 0; continue; }   /* not a tree node */
            depth[i] = depth[p] + 1;
            ok[i] = ok[p] && tok[i] >= 0 && tok[i] == nxt[p];
            if (ok[i] && depth[i] > depth[best]) best = i;
        }
        int n = depth[best] + 1;
        for (int i = best, j = n - 1; j >= 0; --j, i = par[i]) path[j] = i;
        a->n_acc[b] = n;
        a->best_node[b] = best;
        a->bonus[b] = nxt[best];
    }
}

/* ---------------------------------------------------------------------------------- */

typedef struct {
    int B, Hkv, d, S_cap, T_max, n_layers;
    size_t layer_stride;                 /* elements between layers of a cache */
    const uint16_t *K_old, *V_old;       /* [n_layers][B, Hkv, S_cap, d] */
    uint16_t *K_new, *V_new;             /* same shape, written out of place */
    const int32_t *seq_len, *n_acc;      /* [B] */
    const int32_t *path;                 /* [B, T_max] */
    int32_t *new_seq_len;                /* [B] */
} orc_compact_args;

/*
 * KV update after acceptance (Alg. 1, "append accepted tokens and update target KV cache"):
 * the j-th node of the accepted path moves to slot L_b + j.  Out of place on a copy, so the
 * result is the definition itself; every other slot keeps its old bits.
 */
void orc_compact_kv(const orc_compact_args *a) {
    const size_t per_layer = (size_t)a->B * a->Hkv * a->S_cap * a->d;
    for (int l = 0; l < a->n_layers; ++l) {
        memcpy(a->K_new + l * a->layer_stride, a->K_old + l * a->layer_stride, per_layer * 2);
        memcpy(a->V_new + l * a->layer_stride, a->V_old + l * a->layer_stride, per_layer * 2);
    }
    for (int b = 0; b < a->B; ++b) {
        const int L = a->seq_len[b], n = a->n_acc[b];
        a->new_seq_len[b] = L + n;
        for (int l = 0; l < a->n_layers; ++l)
            for (int h = 0; h < a->Hkv; ++h)
                for (int j = 0; j < n; ++j) {
                    size_t base = l * a->layer_stride + ((size_t)b * a->Hkv + h) * a->S_cap * a->d;
                    size_t dst = base + (size_t)(L + j) * a->d;
                    size_t src = base + (size_t)(L + a->path[(size_t)b * a->T_max + j]) * a->d;
                    memcpy(a->K_new + dst, a->K_old + src, (size_t)a->d * 2);
                    memcpy(a->V_new + dst, a->V_old + src, (size_t)a->d * 2);
                }
    }
}

/* ------------------------------------------------------------------------------------------------
 * Online update of the adjacency matrix (the appendix equation "M[x_i] <- argtopk(p_{i+1})" and the
 * same rule in the retrieval section): for every verified tree node i of every request, in the
 * order of the flattened node index r = b * T_max + i, the row of M that belongs to the node's token
 * is replaced by the ids of the k largest entries of the target's next-token scores at that node.
 * The scores are given as logits; softmax is monotone, so the ids are the same as for probabilities.
 * Ids are listed by decreasing score, equal scores by increasing id; NaN scores are never chosen (if
 * fewer than k scores are not NaN the list is filled with -1 and the NaN flag is set).  Walking r
 * upwards makes the node with the highest r win when several nodes of the step carry one token.
 * target_next[r] is the first id of the list (the greedy target id after node i), -1 for padding.
 * Tokens outside [0, V) update nothing (ids other than -1 also set the bad-token flag).
 * ------------------------------------------------------------------------------------------------ */
unsigned orc_update_adjacency(int B, int T_max, int V, int k, const uint16_t *logits /* bf16 bits [B*T_max, V] */,
                              const int32_t *tree_token, const int32_t *tree_size, int32_t *M /* [V, k] in place */,
                              int32_t *target_next /* [B*T_max] */) {
    unsigned flags = 0;
    double *s = (double *)malloc((size_t)V * sizeof(double));
    char *taken = (char *)malloc((size_t)V);
    int32_t *top = (int32_t *)malloc((size_t)k * sizeof(int32_t));
    for (int b = 0; b < B; ++b) {
        int T = tree_size[b];
        if (T < 0 || T > T_max) { T = 0; flags |= ORC_FLAG_BAD_SIZE; }
        for (int i = 0; i < T_max; ++i) {
            const size_t r = (size_t)b * T_max + i;
            if (i >= T) { target_next[r] = -1; continue; }
            for (int v = 0; v < V; ++v) { s[v] = bf16_to_double(logits[r * V + v]); taken[v] = 0; }
            for (int j = 0; j < k; ++j) {
                int best = -1;
                for (int v = 0; v < V; ++v) {
                    if (taken[v] || s[v] != s[v]) continue;
                    if (best < 0 || s[v] > s[best]) best = v;       /* strict: the lowest id wins a tie */
                }
                top[j] = best;
                if (best >= 0) taken[best] = 1; else flags |= ORC_FLAG_NAN_SCORE;
            }
            target_next[r] = top[0];
            const int x = tree_token[r];
            if (x >= 0 && x < V) memcpy(M + (size_t)x * k, top, (size_t)k * sizeof(int32_t));
            else if (x != -1) flags |= ORC_FLAG_BAD_TOKEN;
        }
    }
    free(s); free(taken); free(top);
    return flags;
}

/* ------------------------------------------------------------------------------------------------
 * Root-centred retrieval envelope (retrieval section, "Lightweight parallel retrieval"; template
 * appendix, lookup equation x_u = M[x_F(u), r_u]): the tokens of every node of a static template,
 * filled from the request's root token in template order.  The template is a list of nodes with a
 * parent index inside the list (-1: child of the root) and a successor rank; a parent precedes its
 * children, so one pass in list order has every parent token ready.  An empty row of M (-1) and a
 * missing root make the whole subtree -1.  Root ids outside [-1, V) count as -1 (bad-token flag), and
 * so do matrix entries outside [-1, V); a node whose parent index or rank is out of range gets -1
 * (bad-template flag).  root_token[b * root_stride] is request b's root.
 * ------------------------------------------------------------------------------------------------ */
unsigned orc_retrieve_envelope(int B, int V, int k, int N_env, const int32_t *root_token, long root_stride, const int32_t *M,
                               const int32_t *env_parent, const int32_t *env_rank, int32_t *env_token /* [B, N_env] */) {
    unsigned flags = 0;
    for (int b = 0; b < B; ++b) {
        int32_t x_root = root_token[(size_t)b * root_stride];
        if (x_root < -1 || x_root >= V) { x_root = -1; flags |= ORC_FLAG_BAD_TOKEN; }
        int32_t *x = env_token + (size_t)b * N_env;
        for (int u = 0; u < N_env; ++u) {
            const int f = env_parent[u], r = env_rank[u];
            if (f < -1 || f >= u || r < 0 || r >= k) { x[u] = -1; flags |= ORC_FLAG_BAD_TEMPLATE; continue; }
            const int32_t x_f = f < 0 ? x_root : x[f];
            int32_t v = x_f >= 0 ? M[(size_t)x_f * k + r] : -1;
            if (v < -1 || v >= V) { v = -1; flags |= ORC_FLAG_BAD_TOKEN; }
            x[u] = v;
        }
    }
    return flags;
}

/* ------------------------------------------------------------------------------------------------
 * Candidate-path indices (verification section: after flattening, "position IDs, ancestor mask, and
 * candidate-path indices" are rebuilt): one row per leaf of the flattened tree, leaves in increasing
 * node index, holding the node indices from the root (index 0) down to the leaf and then -1 up to
 * D_max columns; rows past the last leaf hold -1.  n_paths[b] is the number of leaves.  A tree of size
 * 0 has no paths.  A leaf deeper than D_max - 1 keeps the first D_max nodes of its path (bad-size flag).
 * ------------------------------------------------------------------------------------------------ */
unsigned orc_path_indices(int B, int T_max, int D_max, const int32_t *tree_parent, const int32_t *tree_size,
                          int32_t *path_index /* [B, T_max, D_max] */, int32_t *n_paths /* [B] */) {
    unsigned flags = 0;
    int32_t *up = (int32_t *)malloc((size_t)(T_max + 1) * sizeof(int32_t));
    for (int b = 0; b < B; ++b) {
        const int32_t *par = tree_parent + (size_t)b * T_max;
        int32_t *rows = path_index + (size_t)b * T_max * D_max;
        for (int i = 0; i < T_max * D_max; ++i) rows[i] = -1;
        int T = tree_size[b];
        if (T < 0 || T > T_max) { T = 0; flags |= ORC_FLAG_BAD_SIZE; }
        int n = 0;
        for (int i = 0; i < T; ++i) {
            int is_leaf = 1;
            for (int j = i + 1; j < T; ++j)
                if (par[j] == i) { is_leaf = 0; break; }
            if (!is_leaf) continue;
            int len = 0;
            for (int j = i; j >= 0 && len <= T_max; j = par[j]) up[len++] = j;    /* leaf, ..., root */
            if (len > D_max) flags |= ORC_FLAG_BAD_SIZE;
            for (int c = 0; c < len && c < D_max; ++c) rows[(size_t)n * D_max + c] = up[len - 1 - c];
            ++n;
        }
        n_paths[b] = n;
    }
    free(up);
    return flags;
}

/* ------------------------------------------------------------------------------------------------
 * Stochastic acceptance (temperature sampling discussion and the lossless-equivalence proposition:
 * the hybrid tree is verified "with the standard speculative sampling rule", "a rejected position is
 * resampled from the target correction distribution").  The tree's candidates are fixed tokens (kept
 * draft nodes and retrieved nodes alike), i.e. point-mass proposals, so the rule at a node u with
 * target distribution p = softmax(logits[u] / temperature) is the sequential one over u's children in
 * node order: child c with token x is accepted with probability p(x) / rem, where rem is the mass p
 * still holds; on rejection p(x) is set to zero and rem shrinks by it (the correction distribution
 * max(0, p - proposal) renormalised, for a point-mass proposal).  An accepted child becomes the new
 * u.  When no child is accepted (or u is a leaf) the step ends and the bonus token is drawn from what
 * is left of p by inverse CDF over increasing ids.  Every emitted token is then distributed as under
 * plain sampling from the target.
 *   Random numbers are inputs: u_accept[b, c] in [0, 1) decides child c (accept iff u * rem < p(x)),
 * u_bonus[b] draws the bonus (smallest id whose running sum of remaining mass exceeds u * rem).
 * Children with token -1, or with a token a rejected sibling already carried, have probability zero.
 * margin[2b] (optional) is the smallest distance, relative to rem, between an accept decision's random
 * number and its boundary, margin[2b + 1] that of the bonus draw from the ends of the picked id's interval:
 * a float32 implementation agrees with this one whenever the margins are well above float32 rounding of
 * the sums involved.
 * ------------------------------------------------------------------------------------------------ */
unsigned orc_accept_stochastic(int B, int T_max, int V, const uint16_t *logits /* bf16 bits [B*T_max, V] */, double temperature,
                               const int32_t *tree_token, const int32_t *tree_parent, const int32_t *tree_size,
                               const float *u_accept /* [B, T_max] */, const float *u_bonus /* [B] */,
                               int32_t *n_acc, int32_t *path /* [B, T_max] */, int32_t *best_node, int32_t *bonus,
                               double *margin /* [B, 2] or NULL */) {
    unsigned flags = 0;
    double *p = (double *)malloc((size_t)V * sizeof(double));
    for (int b = 0; b < B; ++b) {
        const int32_t *tok = tree_token + (size_t)b * T_max;
        const int32_t *par = tree_parent + (size_t)b * T_max;
        int32_t *pth = path + (size_t)b * T_max;
        for (int j = 0; j < T_max; ++j) pth[j] = -1;
        const int T = tree_size[b];
        if (margin) { margin[2 * b] = 1.0; margin[2 * b + 1] = 1.0; }
        if (T < 1 || T > T_max) { n_acc[b] = 0; best_node[b] = -1; bonus[b] = -1; if (T != 0) flags |= ORC_FLAG_BAD_SIZE; continue; }
        int u = 0, n = 0;
        double rem = 1.0;
        for (;;) {
            pth[n++] = u;
            /* p = softmax(logits[u] / temperature) */
            const uint16_t *row = logits + ((size_t)b * T_max + u) * V;
            double zmax = -INFINITY, sum = 0.0;
            for (int v = 0; v < V; ++v) { double z = bf16_to_double(row[v]) / temperature; if (z > zmax) zmax = z; }
            for (int v = 0; v < V; ++v) { p[v] = exp(bf16_to_double(row[v]) / temperature - zmax); sum += p[v]; }
            for (int v = 0; v < V; ++v) p[v] /= sum;
            rem = 1.0;
            int next = -1;
            for (int c = u + 1; c < T && next < 0; ++c) {
                if (par[c] != u) continue;
                const int x = tok[c];
                const double px = (x >= 0 && x < V) ? p[x] : 0.0;
                const double r = (double)u_accept[(size_t)b * T_max + c] * rem;
                if (margin && px > 0.0) { double m = fabs(r - px) / rem; if (m < margin[2 * b]) margin[2 * b] = m; }
                if (r < px) { next = c; break; }
                if (x >= 0 && x < V) { rem -= px; p[x] = 0.0; }
            }
            if (next < 0) break;
            u = next;
        }
        /* bonus from what is left of p at u */
        const double target = (double)u_bonus[b] * rem;
        double run = 0.0;
        int pick = -1, last = -1;
        for (int v = 0; v < V; ++v) {
            if (p[v] <= 0.0) continue;
            last = v;
            const double before = run;
            run += p[v];
            if (pick < 0 && run > target) {
                pick = v;
                if (margin) {
                    margin[2 * b + 1] = fmin(target - before, run - target) / rem;
                }
            }
        }
        if (pick < 0) pick = last;             /* rounding left the running sum just below the target */
        n_acc[b] = n;
        best_node[b] = u;
        bonus[b] = pick;
    }
    free(p);
    return flags;
}
