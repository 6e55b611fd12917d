"""Seeded synthetic inputs for the tree-verify path.

This module only draws inputs: draft trees (token ids, parent pointers, cumulative
path scores), retrieval templates given as rank paths, the adjacency matrix, Q/K/V
tensors, cached lengths and the target's greedy ids.  It holds none of the method's
arithmetic (no pruning, no grafting, no masks, no attention, no acceptance), so the
CPU oracle and the CUDA path can both consume its arrays without sharing logic.

The recipes stand in for the paper's workloads (60-node EAGLE-3 style trees at ~2K
context, LongBench-style 4K-64K contexts, batch sizes 1-16 of the serving study and
the model shapes of the architecture table in the paper's evaluation appendix).
No item of any benchmark is reproduced here; everything is random with a fixed seed.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
import torch

# prune modes of graft_build_tree (values mirror include/graft.h)
MODE_NONE = 0    # keep the draft tree as is, graft nothing
MODE_TOPK = 1    # keep the top keep_count[b] nodes by cumulative path score
MODE_GATED = 2   # checkpoint gating on the depth confidence picks the stage
MODE_NODE = 3    # batched rule: drop low-confidence nodes (and their subtrees)

# thresholds of the paper's calibration table (Qwen3-8B columns, rounded means):
# stage d0 ~0.14, d1 ~0.14, d5 ~0.49
PAPER_TAU = (0.14, 0.14, 0.49)
# stage budgets of the 60-node verifier: retained draft nodes / retrieved nodes
PAPER_KEEP = (8, 24, 40)
PAPER_RET = (52, 36, 20)
# per-depth node counts of the paper's retrieval templates (template table)
PAPER_TEMPLATE_WIDTHS = {
    "full": (8, 16, 14, 11, 8, 7, 6, 5, 5),
    "d0": (8, 10, 8, 6, 5, 4, 4, 4, 3),
    "d1": (6, 7, 5, 4, 4, 3, 3, 2, 2),
    "d5": (4, 3, 3, 2, 2, 2, 2, 1, 1),
}


# --------------------------------------------------------------------------------------
# static tree shapes
# --------------------------------------------------------------------------------------
def rank_path_tree(widths: Sequence[int], caps: Sequence[int]) -> List[Tuple[int, ...]]:
    """Unbalanced static tree over successor ranks, given per-depth node counts.

    Depth-(j+1) nodes are the widths[j] cheapest one-rank extensions path+(r,), r < caps[j],
    of the depth-j nodes, where cheaper means smaller (sum of ranks, then lexicographic
    path).  Low ranks therefore get more children and the all-zero chain reaches the
    last depth.  Nodes are returned depth-major, lexicographic inside a depth, so the
    order is topological.
    """
    levels: List[List[Tuple[int, ...]]] = [[()]]
    out: List[Tuple[int, ...]] = []
    for w, cap in zip(widths, caps):
        cand = [p + (r,) for p in levels[-1] for r in range(cap)]
        cand.sort(key=lambda p: (sum(p), p))
        if len(cand) < w:
            raise ValueError("width %d not reachable (only %d candidates)" % (w, len(cand)))
        lvl = sorted(cand[:w])
        levels.append(lvl)
        out.extend(lvl)
    return out


def paths_to_parent_rank(paths: Sequence[Tuple[int, ...]]) -> Tuple[np.ndarray, np.ndarray]:
    """Rank paths -> (parent index inside the list, -1 for children of the root; rank)."""
    index = {p: i for i, p in enumerate(paths)}
    parent = np.empty(len(paths), np.int32)
    rank = np.empty(len(paths), np.int32)
    for i, p in enumerate(paths):
        parent[i] = -1 if len(p) == 1 else index[p[:-1]]
        rank[i] = p[-1]
    return parent, rank


def paper_template(name: str, k: int = 8) -> Tuple[np.ndarray, np.ndarray]:
    """One of the paper's retrieval templates (only its depth histogram is printed there;
    the rank paths come from rank_path_tree)."""
    w = PAPER_TEMPLATE_WIDTHS[name]
    return paths_to_parent_rank(rank_path_tree(w, [k] * len(w)))


def chains_template(lengths: Sequence[int]) -> Tuple[np.ndarray, np.ndarray]:
    """Chains hanging off the root: chain c follows ranks (c, 0, 0, ...)."""
    parent: List[int] = []
    rank: List[int] = []
    for c, n in enumerate(lengths):
        for j in range(n):
            parent.append(-1 if j == 0 else len(parent) - 1)
            rank.append(c if j == 0 else 0)
    return np.asarray(parent, np.int32), np.asarray(rank, np.int32)


def template_rank_paths(parent: np.ndarray, rank: np.ndarray) -> List[Tuple[int, ...]]:
    """(parent, rank) lists of a template -> the rank path of every node."""
    paths: List[Tuple[int, ...]] = []
    for f, r in zip(parent.tolist(), rank.tolist()):
        paths.append((() if f < 0 else paths[f]) + (r,))
    return paths


def retrieval_envelope(templates: Sequence[Tuple[np.ndarray, np.ndarray]]) -> Tuple[np.ndarray, np.ndarray, List[np.ndarray]]:
    """The smallest template that contains every node (rank path) of the given templates, and for each
    of them the index of its nodes inside that envelope.  Envelope nodes are ordered by depth, then
    lexicographically, so a parent always precedes its children."""
    all_paths = [template_rank_paths(tp, tr) for tp, tr in templates]
    union = sorted({q[:n] for ps in all_paths for q in ps for n in range(1, len(q) + 1)}, key=lambda q: (len(q), q))
    index = {q: i for i, q in enumerate(union)}
    env_parent, env_rank = paths_to_parent_rank(union) if union else (np.zeros(0, np.int32), np.zeros(0, np.int32))
    return env_parent, env_rank, [np.asarray([index[q] for q in ps], np.int32) for ps in all_paths]


def workload_envelope(w: "Workload") -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Envelope of a workload's stage templates and the envelope index of every template node
    (tmpl_env, laid out like tmpl_parent / tmpl_rank)."""
    if w.tmpl_offset is None:
        stages = [(w.tmpl_parent, w.tmpl_rank)]
    else:
        off = w.tmpl_offset.tolist()
        stages = [(w.tmpl_parent[a:b], w.tmpl_rank[a:b]) for a, b in zip(off[:-1], off[1:])]
    ep, er, maps = retrieval_envelope(stages)
    return ep, er, (np.concatenate(maps).astype(np.int32) if maps else np.zeros(0, np.int32))


DENSE60_WIDTHS = (8, 16, 14, 10, 7, 4)
DENSE60_CAPS = (8, 4, 2, 1, 1, 1)


def dense_tree_parents(max_depth: int = 6) -> np.ndarray:
    """EAGLE-3 style static tree: root + widths 8,16,14,10,7,4 (60 nodes at depth 6),
    per-parent child caps 8,4,2,1,1,1.  Returns parent[] with parent[0] = -1."""
    paths = rank_path_tree(DENSE60_WIDTHS[:max_depth], DENSE60_CAPS[:max_depth])
    p, _ = paths_to_parent_rank(paths)
    return np.concatenate([[-1], np.where(p < 0, 0, p + 1)]).astype(np.int32)


def random_tree_parents(rng: np.random.Generator, n: int) -> np.ndarray:
    """parent[i] uniform in [0, i); node 0 is the root."""
    par = np.full(n, -1, np.int32)
    for i in range(1, n):
        par[i] = rng.integers(0, i)
    return par


def chain_parents(n: int) -> np.ndarray:
    return np.arange(-1, n - 1, dtype=np.int32)


def star_parents(n: int) -> np.ndarray:
    p = np.zeros(n, np.int32)
    p[0] = -1
    return p


# --------------------------------------------------------------------------------------
# workload container
# --------------------------------------------------------------------------------------
@dataclass
class Workload:
    name: str
    B: int
    Hq: int
    Hkv: int
    d: int
    S_cap: int
    T_max: int
    N_max: int
    K_max: int
    V: int
    k: int
    scale: float
    # build inputs
    seq_len: np.ndarray            # int32 [B]
    draft_token: np.ndarray        # int32 [B, N_max]
    draft_parent: np.ndarray       # int32 [B, N_max]
    draft_score: np.ndarray        # float32 [B, N_max]
    n_draft: np.ndarray            # int32 [B]
    M: np.ndarray                  # int32 [V, k]
    mode: int = MODE_NONE
    keep_count: Optional[np.ndarray] = None      # int32 [B]   (MODE_TOPK)
    k_max: Optional[np.ndarray] = None           # int32 [B]   per-sequence budget
    gate_depth: int = 0                          # MODE_NODE
    node_threshold: float = 0.0                  # MODE_NODE
    ckpt_depth: Optional[np.ndarray] = None      # int32 [n_ckpt]   (MODE_GATED)
    ckpt_log_tau: Optional[np.ndarray] = None    # float32 [n_ckpt]
    ckpt_keep: Optional[np.ndarray] = None       # int32 [n_ckpt]
    tmpl_offset: Optional[np.ndarray] = None     # int32 [n_ckpt + 1]
    tmpl_parent: np.ndarray = field(default_factory=lambda: np.zeros(0, np.int32))
    tmpl_rank: np.ndarray = field(default_factory=lambda: np.zeros(0, np.int32))
    attach_tail: bool = False                    # template nodes with parent -1 continue the last kept node instead of the root
    # acceptance recipe
    p_draft: float = 0.75
    p_graft: float = 0.9
    seed: int = 0
    # attention inputs (torch bf16 on CPU; None until make_qkv is called)
    Q: Optional[torch.Tensor] = None     # [B, T_max, Hq, d]
    Kc: Optional[torch.Tensor] = None    # [B, Hkv, S_cap, d]
    Vc: Optional[torch.Tensor] = None
    std: float = 1.0

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """torch bf16 tensor -> numpy uint16 view of the same bits (no copy)."""
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def make_qkv(w: Workload, tree_size: Optional[np.ndarray] = None, poison: bool = False,
             seed: Optional[int] = None) -> None:
    """Draw Q and the K/V cache (fp32 normal -> bf16, round to nearest even, once).

    Slots [0, L_b + T_max) of every sequence hold random K/V (the tree tokens' K/V sit at
    L_b + i, as the caller's QKV projection would have left them).  With poison=True,
    every slot at or beyond L_b + tree_size[b] is overwritten with NaN bit patterns, and
    so are Q rows of padding nodes: nothing that lies outside the tree may reach an output.
    """
    g = torch.Generator(device="cpu")
    g.manual_seed(1000003 * (w.seed if seed is None else seed) + 17)
    w.Q = (torch.randn(w.B, w.T_max, w.Hq, w.d, generator=g) * w.std).to(torch.bfloat16)
    w.Kc = (torch.randn(w.B, w.Hkv, w.S_cap, w.d, generator=g) * w.std).to(torch.bfloat16)
    w.Vc = (torch.randn(w.B, w.Hkv, w.S_cap, w.d, generator=g) * w.std).to(torch.bfloat16)
    if poison:
        assert tree_size is not None
        nan = torch.tensor(float("nan"), dtype=torch.bfloat16)
        for b in range(w.B):
            end = int(w.seq_len[b]) + int(tree_size[b])
            w.Kc[b, :, end:, :] = nan
            w.Vc[b, :, end:, :] = nan
            w.Q[b, int(tree_size[b]):, :, :] = nan


def draw_target_next(tree_token: np.ndarray, tree_parent: np.ndarray, tree_size: np.ndarray,
                     tree_src: np.ndarray, V: int, p_draft: float, p_graft: float,
                     seed: int) -> np.ndarray:
    """Greedy target ids per tree node, int32 [B, T_max].

    For a node u with children c1 < c2 < ... each child draws a Bernoulli(p) (p_graft for
    grafted nodes, tree_src < 0; p_draft otherwise); target_next[u] is the token of the
    first child that drew 1 and has a real token, else a uniform id in [0, V) (which may
    match a child by accident; both sides see the same array).  Leaves get the uniform id.
    """
    B, T_max = tree_token.shape
    rng = np.random.default_rng(np.random.PCG64(7919 * seed + 1))
    u = rng.random((B, T_max))
    fallback = rng.integers(0, V, size=(B, T_max), dtype=np.int64).astype(np.int32)
    out = fallback.copy()
    for b in range(B):
        chosen = np.zeros(T_max, bool)
        for c in range(1, int(tree_size[b])):
            par = int(tree_parent[b, c])
            if par < 0 or chosen[par] or tree_token[b, c] < 0:
                continue
            p = p_graft if tree_src[b, c] < 0 else p_draft
            if u[b, c] < p:
                out[b, par] = tree_token[b, c]
                chosen[par] = True
    return out


# --------------------------------------------------------------------------------------
# draft-tree draws
# --------------------------------------------------------------------------------------
def _scores_along(parent: np.ndarray, rng: np.random.Generator) -> np.ndarray:
    """Cumulative path scores: running sums of log U(0.05, 1), so a child never scores
    above its parent (log-probabilities are <= 0).  Root score 0."""
    n = len(parent)
    s = np.zeros(n, np.float32)
    step = np.log(rng.uniform(0.05, 1.0, size=n)).astype(np.float32)
    for i in range(1, n):
        s[i] = np.float32(s[parent[i]] + step[i])
    return s


def _pack_trees(parents: List[np.ndarray], N_max: int, V: int, rng: np.random.Generator,
                scores: Optional[List[np.ndarray]] = None):
    B = len(parents)
    tok = np.full((B, N_max), -1, np.int32)
    par = np.full((B, N_max), -1, np.int32)
    sc = np.zeros((B, N_max), np.float32)
    nd = np.zeros(B, np.int32)
    for b, p in enumerate(parents):
        n = len(p)
        nd[b] = n
        par[b, :n] = p
        tok[b, :n] = rng.integers(0, V, size=n)
        sc[b, :n] = _scores_along(p, rng) if scores is None else scores[b]
    return tok, par, sc, nd


def _random_M(rng: np.random.Generator, V: int, k: int, empty_frac: float = 0.0) -> np.ndarray:
    M = rng.integers(0, V, size=(V, k), dtype=np.int64).astype(np.int32)
    if empty_frac > 0:
        M[rng.random(V) < empty_frac, :] = -1   # rows never written yet (cold start)
    return M


def _fill_chain_lengths(rng: np.random.Generator, total: int, lo: int = 4, hi: int = 8) -> List[int]:
    """Chain lengths U{lo..hi} until `total` template nodes are available (the last chain is
    cut by the builder's prefix rule, so the template may be longer than what is used)."""
    out: List[int] = []
    while sum(out) < total:
        out.append(int(rng.integers(lo, hi + 1)))
    return out


# --------------------------------------------------------------------------------------
# the five benchmark configurations (plus the paper-stage case 3')
# --------------------------------------------------------------------------------------
def config(cfg: str, *, B: Optional[int] = None, L: Optional[int] = None,
           seed: Optional[int] = None) -> Workload:
    """Build the named workload's integer inputs (call make_qkv for the tensors).

    cfg in {"1", "2", "3", "3p", "4", "5", "tail"}.  B and L override batch and context length
    (used by the tests to shrink a shape without changing its structure).
    """
    if cfg == "tail":
        return tail_block(B=B or 4, L=L or 65536, seed=16 if seed is None else seed)
    if cfg == "1":
        seed = 0 if seed is None else seed
        rng = np.random.default_rng(np.random.PCG64(seed))
        B = B or 1
        L = L or 256
        V, k, T = 1000, 8, 8
        parents = [random_tree_parents(rng, T) for _ in range(B)]
        tok, par, sc, nd = _pack_trees(parents, T, V, rng)
        return Workload(name="cfg1-tiny", B=B, Hq=4, Hkv=1, d=64, S_cap=L + T, T_max=T, N_max=T,
                        K_max=T, V=V, k=k, scale=float(np.float32(1.0 / math.sqrt(64))),
                        seq_len=np.full(B, L, np.int32), draft_token=tok, draft_parent=par,
                        draft_score=sc, n_draft=nd, M=_random_M(rng, V, k), mode=MODE_NONE,
                        p_draft=0.7, p_graft=0.7, seed=seed)
    if cfg == "2":
        seed = 2 if seed is None else seed
        rng = np.random.default_rng(np.random.PCG64(seed))
        B = B or 4
        L = L or 2048
        V, k, T = 128256, 8, 60
        parents = [dense_tree_parents() for _ in range(B)]
        tok, par, sc, nd = _pack_trees(parents, 64, V, rng)
        return Workload(name="cfg2-llama31-8b", B=B, Hq=32, Hkv=8, d=128, S_cap=L + 64, T_max=64,
                        N_max=64, K_max=T, V=V, k=k, scale=float(np.float32(1.0 / math.sqrt(128))),
                        seq_len=np.full(B, L, np.int32), draft_token=tok, draft_parent=par,
                        draft_score=sc, n_draft=nd, M=_random_M(rng, V, k), mode=MODE_NONE,
                        p_draft=0.75, p_graft=0.75, seed=seed)
    if cfg == "3":
        seed = 3 if seed is None else seed
        rng = np.random.default_rng(np.random.PCG64(seed))
        B = B or 8
        L = L or 4096
        V, k = 128256, 8
        parents = [dense_tree_parents() for _ in range(B)]
        # per-node confidence ~ U(0,1) is what the batched rule thresholds
        conf = [rng.random(60).astype(np.float32) for _ in range(B)]
        tok, par, sc, nd = _pack_trees(parents, 64, V, rng, scores=conf)
        tp, tr = chains_template(_fill_chain_lengths(rng, 64))
        return Workload(name="cfg3-prune-graft", B=B, Hq=32, Hkv=8, d=128, S_cap=L + 64, T_max=64,
                        N_max=64, K_max=64, V=V, k=k, scale=float(np.float32(1.0 / math.sqrt(128))),
                        seq_len=np.full(B, L, np.int32), draft_token=tok, draft_parent=par,
                        draft_score=sc, n_draft=nd, M=_random_M(rng, V, k), mode=MODE_NODE,
                        gate_depth=3, node_threshold=float(np.float32(0.3)),
                        tmpl_parent=tp, tmpl_rank=tr, p_draft=0.75, p_graft=0.9, seed=seed)
    if cfg == "3p":
        # one sequence per pruning stage of the paper (d0, d1, d5) plus one that survives
        seed = 33 if seed is None else seed
        rng = np.random.default_rng(np.random.PCG64(seed))
        V, k = 151936, 8
        L = L or 512
        ckpt_depth = np.asarray([1, 2, 6], np.int32)
        log_tau = np.log(np.asarray(PAPER_TAU, np.float32)).astype(np.float32)
        parents, scores = [], []
        for stage in (0, 1, 2, 3):
            p = dense_tree_parents()
            s = _scores_along(p, rng)
            depth = np.zeros(len(p), np.int32)
            for i in range(1, len(p)):
                depth[i] = depth[p[i]] + 1
            # lift every checkpoint above its threshold, then sink the stage's own one
            s = s * np.float32(0.05)
            if stage < 3:
                D = int(ckpt_depth[stage])
                s[depth >= D] += np.float32(-4.0)
            parents.append(p)
            scores.append(s.astype(np.float32))
        B = 4
        tok, par, sc, nd = _pack_trees(parents, 64, V, rng, scores=scores)
        tps, trs, off = [], [], [0]
        for name in ("d0", "d1", "d5"):
            tp, tr = paper_template(name, k)
            tps.append(tp)
            trs.append(tr)
            off.append(off[-1] + len(tp))
        return Workload(name="cfg3p-paper-stages", B=B, Hq=32, Hkv=8, d=128, S_cap=L + 64, T_max=64,
                        N_max=64, K_max=60, V=V, k=k, scale=float(np.float32(1.0 / math.sqrt(128))),
                        seq_len=np.full(B, L, np.int32), draft_token=tok, draft_parent=par,
                        draft_score=sc, n_draft=nd, M=_random_M(rng, V, k, empty_frac=0.02),
                        mode=MODE_GATED, ckpt_depth=ckpt_depth, ckpt_log_tau=log_tau,
                        ckpt_keep=np.asarray(PAPER_KEEP, np.int32),
                        tmpl_offset=np.asarray(off, np.int32),
                        tmpl_parent=np.concatenate(tps), tmpl_rank=np.concatenate(trs),
                        p_draft=0.75, p_graft=0.9, seed=seed)
    if cfg == "4":
        seed = 4 if seed is None else seed
        rng = np.random.default_rng(np.random.PCG64(seed))
        B = B or 1
        L = L or 65536
        V, k = 151936, 8
        parents = [dense_tree_parents(max_depth=4) for _ in range(B)]   # 49 nodes, depth <= 4
        tok, par, sc, nd = _pack_trees(parents, 64, V, rng)
        tp, tr = chains_template([6, 6, 6])
        return Workload(name="cfg4-qwen3-14b-long", B=B, Hq=40, Hkv=8, d=128, S_cap=L + 64,
                        T_max=64, N_max=64, K_max=48, V=V, k=k,
                        scale=float(np.float32(1.0 / math.sqrt(128))),
                        seq_len=np.full(B, L, np.int32), draft_token=tok, draft_parent=par,
                        draft_score=sc, n_draft=nd, M=_random_M(rng, V, k), mode=MODE_TOPK,
                        keep_count=np.full(B, 30, np.int32), tmpl_parent=tp, tmpl_rank=tr,
                        p_draft=0.7, p_graft=0.7, seed=seed, std=0.5)
    if cfg == "5":
        seed = 5 if seed is None else seed
        rng = np.random.default_rng(np.random.PCG64(seed))
        B = B or 16
        Lmax = L or 8192
        Lmin = max(1, Lmax // 8)
        V, k = 151936, 8
        parents = [dense_tree_parents() for _ in range(B)]
        tok, par, sc, nd = _pack_trees(parents, 64, V, rng)
        T_b = rng.integers(16, 65, size=B).astype(np.int32)
        tp, tr = chains_template(_fill_chain_lengths(rng, 64))
        return Workload(name="cfg5-qwen3-235b-ragged", B=B, Hq=64, Hkv=4, d=128, S_cap=Lmax + 64,
                        T_max=64, N_max=64, K_max=64, V=V, k=k,
                        scale=float(np.float32(1.0 / math.sqrt(128))),
                        seq_len=rng.integers(Lmin, Lmax + 1, size=B).astype(np.int32),
                        draft_token=tok, draft_parent=par, draft_score=sc, n_draft=nd,
                        M=_random_M(rng, V, k), mode=MODE_TOPK,
                        keep_count=((T_b + 1) // 2).astype(np.int32), k_max=T_b,
                        tmpl_parent=tp, tmpl_rank=tr, p_draft=0.65, p_graft=0.65, seed=seed)
    raise KeyError(cfg)


def tail_block(B: int = 4, L: int = 65536, block: int = 16, *, Hq: int = 40, Hkv: int = 8, d: int = 128, V: int = 151936,
               k: int = 8, seed: int = 16) -> Workload:
    """Block drafter with tail grafting: a drafted chain of `block` tokens whose cumulative scores fall along the
    chain, the first keep_count[b] ~ U{4..block} of them are kept (top-k by score on a chain = a prefix) and the
    rank-0 chain of retrieved tokens fills the block from the last kept token on."""
    rng = np.random.default_rng(np.random.PCG64(seed))
    tok, par, sc, nd = _pack_trees([chain_parents(block)] * B, block, V, rng)
    sc[:] = -np.cumsum(rng.random((B, block)).astype(np.float32), axis=1)       # strictly decreasing along the chain
    tp, tr = chains_template([block])
    return Workload(name="tail-block", B=B, Hq=Hq, Hkv=Hkv, d=d, S_cap=L + block, T_max=block, N_max=block, K_max=block,
                    V=V, k=k, scale=float(np.float32(1.0 / math.sqrt(d))), seq_len=np.full(B, L, np.int32),
                    draft_token=tok, draft_parent=par, draft_score=sc, n_draft=nd, M=_random_M(rng, V, k, 0.02),
                    mode=MODE_TOPK, keep_count=rng.integers(4, block + 1, size=B).astype(np.int32), tmpl_parent=tp,
                    tmpl_rank=tr, attach_tail=True, p_draft=0.8, p_graft=0.7, seed=seed, std=0.5)


def custom(parents: List[np.ndarray], *, Hq: int, Hkv: int, d: int, L: Sequence[int], V: int = 1000,
           k: int = 8, T_max: Optional[int] = None, seed: int = 0, std: float = 1.0,
           S_cap: Optional[int] = None, p: float = 0.7) -> Workload:
    """A no-prune workload around explicit parent arrays (edge-case tests)."""
    rng = np.random.default_rng(np.random.PCG64(seed))
    B = len(parents)
    T_max = T_max or max(len(p_) for p_ in parents)
    tok, par, sc, nd = _pack_trees(parents, T_max, V, rng)
    seq_len = np.asarray(L, np.int32)
    assert len(seq_len) == B
    S_cap = S_cap or int(seq_len.max()) + T_max
    return Workload(name="custom", B=B, Hq=Hq, Hkv=Hkv, d=d, S_cap=S_cap, T_max=T_max, N_max=T_max,
                    K_max=T_max, V=V, k=k, scale=float(np.float32(1.0 / math.sqrt(d))),
                    seq_len=seq_len, draft_token=tok, draft_parent=par, draft_score=sc, n_draft=nd,
                    M=_random_M(rng, V, k), mode=MODE_NONE, p_draft=p, p_graft=p, seed=seed, std=std)


def make_logits(B: int, T_max: int, V: int, seed: int, peaks: int = 12) -> np.ndarray:
    """Target logits of all tree nodes, bf16 bit patterns [B*T_max, V]: a broad body (normal, sigma 2.5) with a
    few high entries per row, as the output of an LM head looks after the final norm; rounding to bf16 makes
    equal values common, also among the largest entries.  Rows of padding nodes are filled like the others."""
    rng = np.random.default_rng(np.random.PCG64(seed))
    N = B * T_max
    x = rng.standard_normal((N, V), dtype=np.float32) * np.float32(2.5)
    cols = rng.integers(0, V, size=(N, peaks))
    vals = (rng.integers(32, 60, size=(N, peaks)) * np.float32(0.25)).astype(np.float32)     # 8.0 .. 14.75 in steps of 1/4
    np.put_along_axis(x, cols, vals, axis=1)
    return bf16_bits(torch.from_numpy(x).to(torch.bfloat16))
