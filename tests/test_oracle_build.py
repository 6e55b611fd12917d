"""Pins for the oracle's tree assembly (prune + graft + rebuild), CPU only.

What fixes the expected values: the stage budgets and template depth histograms the paper
prints (tests/golden/paper_stage_budgets.txt), the closed form x_u = M[x_parent(u), r_u], the
"no pruning -> base tree" degenerate case, structural invariants checked by climbing parent
pointers, and an independent set-based restatement of the keep rules on random trees.
"""
import os

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

from paper_2605_20104_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_stage_budgets.txt")


def read_golden():
    rows = {}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        name, keep, ret, dist = line.split()
        rows[name] = (None if keep == "-" else int(keep), int(ret), [int(x) for x in dist.split("+")])
    return rows


def climb(parent, i):
    out = []
    while i >= 0:
        out.append(i)
        i = int(parent[i])
    return out


def check_structure(o, w):
    """Invariants every built tree must satisfy, from the definitions alone."""
    for b in range(w.B):
        T = int(o["tree_size"][b])
        par, anc, pos = o["tree_parent"][b], o["tree_anc"][b], o["tree_pos"][b]
        assert par[0] == -1
        for i in range(T):
            if i:
                assert 0 <= par[i] < i
            chain = climb(par, i)
            assert int(anc[i]) == sum(1 << a for a in chain)          # ancestor-or-self bits
            assert pos[i] == w.seq_len[b] + len(chain) - 1             # position = L + depth
        # padding
        assert (o["tree_token"][b, T:] == -1).all() and (par[T:] == -1).all()
        assert (pos[T:] == 0).all() and (anc[T:] == 0).all()
        assert (o["tree_src"][b, T:] == np.iinfo(np.int32).min).all()
        # provenance is one-to-one
        src = o["tree_src"][b, :T]
        assert len(set(src.tolist())) == T


def test_golden_file_is_self_consistent():
    g = read_golden()
    for name, (keep, ret, dist) in g.items():
        assert sum(dist) == ret
        if keep is not None:
            assert keep + ret == 60                                     # K_max = K_draft + K_ret
    assert tuple(g["d0"][2]) == W.PAPER_TEMPLATE_WIDTHS["d0"]
    assert tuple(g["full"][2]) == W.PAPER_TEMPLATE_WIDTHS["full"]


@pytest.mark.parametrize("name", ["full", "d0", "d1", "d5"])
def test_template_fixture_matches_printed_histogram(name):
    g = read_golden()
    tp, tr = W.paper_template(name, 8)
    depth = np.zeros(len(tp), int)
    for u in range(len(tp)):
        assert tp[u] < u
        depth[u] = 1 if tp[u] < 0 else depth[tp[u]] + 1
    assert np.bincount(depth)[1:].tolist() == g[name][2]
    assert len(tp) == g[name][1]
    # the greedy (all rank 0) chain reaches the last depth
    zero_chain_depth = max(depth[u] for u in range(len(tp))
                           if all(tr[a] == 0 for a in climb(tp, u)))
    assert zero_chain_depth == 9


def test_paper_stages(orc):
    """One sequence per stage d0 / d1 / d5 plus one that survives every checkpoint."""
    g = read_golden()
    w = W.config("3p")
    o = orc.build_tree(w)
    assert o["flags"] == 0
    check_structure(o, w)
    for b, name in enumerate(["d0", "d1", "d5"]):
        keep, ret, dist = g[name]
        src = o["tree_src"][b]
        assert o["tree_size"][b] == 60                                  # |T_s| = K_max
        assert (src[:60] >= 0).sum() == keep and (src[:60] < 0).sum() == ret
        depth = np.array([bin(int(a)).count("1") - 1 for a in o["tree_anc"][b, :60]])
        assert np.bincount(depth[src[:60] < 0])[1:].tolist() == dist
        # kept draft nodes precede grafted ones and keep their order and tokens
        kept = src[:keep]
        assert (np.diff(kept) > 0).all() and kept[0] == 0
        assert (o["tree_token"][b, :keep] == w.draft_token[b, kept]).all()
        # retained nodes are the best-scoring eligible ones
        d_in = np.array([len(climb(w.draft_parent[b], i)) - 1 for i in range(60)])
        elig = [i for i in range(1, 60) if d_in[i] <= w.ckpt_depth[b]]
        best = sorted(elig, key=lambda i: (-w.draft_score[b, i], i))[:keep - 1]
        assert sorted([0] + best) == kept.tolist()
        # closed form of every retrieved token, through the parent's token
        off = int(w.tmpl_offset[b])
        for j in range(keep, 60):
            u = j - keep
            assert src[j] == -1 - u
            tp, r = int(w.tmpl_parent[off + u]), int(w.tmpl_rank[off + u])
            p = 0 if tp < 0 else keep + tp
            assert o["tree_parent"][b, j] == p
            ptok = int(o["tree_token"][b, p])
            want = -1 if ptok < 0 else int(w.M[ptok, r])
            assert o["tree_token"][b, j] == want
    # no checkpoint fails: the base tree comes back untouched, nothing grafted
    b = 3
    assert o["tree_size"][b] == 60
    assert (o["tree_token"][b, :60] == w.draft_token[b, :60]).all()
    assert (o["tree_parent"][b, :60] == w.draft_parent[b, :60]).all()
    assert (o["tree_src"][b, :60] == np.arange(60)).all()


def test_empty_rows_of_M_propagate(orc):
    w = W.config("3p")
    w.M[:] = -1                                                         # cold start: nothing retrievable
    o = orc.build_tree(w)
    for b in range(3):
        assert (o["tree_token"][b][o["tree_src"][b] < 0][:1] == -1).all()
        assert (o["tree_token"][b, :60][o["tree_src"][b, :60] < 0] == -1).all()
        assert o["tree_size"][b] == 60                                  # the shape stays fixed


def test_mode_none_is_identity(orc):
    for c in ("1", "2"):
        w = W.config(c)
        o = orc.build_tree(w)
        assert o["flags"] == 0
        check_structure(o, w)
        for b in range(w.B):
            n = int(w.n_draft[b])
            assert o["tree_size"][b] == n
            assert (o["tree_token"][b, :n] == w.draft_token[b, :n]).all()
            assert (o["tree_parent"][b, :n] == w.draft_parent[b, :n]).all()


def independent_build(w, b):
    """Set-based restatement of the keep rules and of the graft, written separately from the C."""
    n = int(w.n_draft[b])
    par = w.draft_parent[b]
    sc = w.draft_score[b]
    depth = [len(climb(par, i)) - 1 for i in range(n)]
    budget = int(w.k_max[b]) if w.k_max is not None else w.K_max
    tmpl = list(zip(w.tmpl_parent.tolist(), w.tmpl_rank.tolist()))
    graft = True
    if w.mode == W.MODE_NONE:
        keep, graft = set(range(n)), False
    elif w.mode == W.MODE_TOPK:
        rest = sorted(range(1, n), key=lambda i: (-sc[i], i))[:max(int(w.keep_count[b]) - 1, 0)]
        keep = {0, *rest}
    elif w.mode == W.MODE_NODE:
        bad = {i for i in range(1, n) if depth[i] >= w.gate_depth and sc[i] < np.float32(w.node_threshold)}
        keep = {i for i in range(n) if not (set(climb(par, i)) & bad)}
    else:
        stage = None
        for c in range(len(w.ckpt_depth)):
            vals = [sc[i] for i in range(1, n) if depth[i] == w.ckpt_depth[c]]
            if not vals or max(vals) <= w.ckpt_log_tau[c]:
                stage = c
                break
        if stage is None:
            keep, graft = set(range(n)), False
        else:
            elig = [i for i in range(1, n) if depth[i] <= w.ckpt_depth[stage]]
            keep = {0, *sorted(elig, key=lambda i: (-sc[i], i))[:int(w.ckpt_keep[stage]) - 1]}
            tmpl = tmpl[int(w.tmpl_offset[stage]):int(w.tmpl_offset[stage + 1])]
    keep = {i for i in keep if set(climb(par, i)) <= keep}              # parents must be present
    order = sorted(keep)[:budget]
    new = {old: j for j, old in enumerate(order)}
    tok = [int(w.draft_token[b, i]) for i in order]
    parent = [-1 if i == 0 else new[int(par[i])] for i in order]
    src = list(order)
    K = len(order)
    if graft:
        for u, (tp, r) in enumerate(tmpl[:max(budget - K, 0)]):
            p = 0 if tp < 0 else K + tp
            tok.append(-1 if tok[p] < 0 else int(w.M[tok[p], r]))
            parent.append(p)
            src.append(-1 - u)
    return tok, parent, src


@pytest.mark.parametrize("cfg", ["1", "2", "3", "3p", "4", "5"])
def test_configs_against_independent_build(orc, cfg):
    w = W.config(cfg)
    o = orc.build_tree(w)
    assert o["flags"] == 0
    check_structure(o, w)
    for b in range(w.B):
        tok, parent, src = independent_build(w, b)
        T = len(tok)
        assert o["tree_size"][b] == T
        assert o["tree_token"][b, :T].tolist() == tok
        assert o["tree_parent"][b, :T].tolist() == parent
        assert o["tree_src"][b, :T].tolist() == src


def test_cfg3_prunes_and_refills(orc):
    w = W.config("3")
    o = orc.build_tree(w)
    for b in range(w.B):
        src = o["tree_src"][b]
        kept = src[src >= 0]
        assert o["tree_size"][b] == 64
        assert 0 < (src < 0).sum() and len(kept) < 60                   # something was pruned, refilled
        d_in = np.array([len(climb(w.draft_parent[b], i)) - 1 for i in range(60)])
        low = (d_in >= 3) & (w.draft_score[b, :60] < np.float32(0.3))
        assert not low[kept].any()
        # grafted chains start at the root
        first = np.nonzero(src < 0)[0][0]
        assert o["tree_parent"][b, first] == 0


def test_cfg4_and_cfg5_sizes(orc):
    w = W.config("4")
    o = orc.build_tree(w)
    assert o["tree_size"].tolist() == [48]
    assert (o["tree_src"][0, :48] >= 0).sum() == 30
    w = W.config("5")
    o = orc.build_tree(w)
    assert (o["tree_size"] == w.k_max).all()
    assert ((o["tree_src"] >= 0).sum(1) == w.keep_count).all()


@settings(max_examples=60, deadline=None)
@given(st.integers(0, 10_000), st.integers(2, 40), st.sampled_from([W.MODE_TOPK, W.MODE_NODE, W.MODE_NONE]),
       st.integers(1, 48))
def test_random_trees_against_independent_build(seed, n, mode, budget):
    import oracle as orc
    rng = np.random.default_rng(seed)
    w = W.custom([W.random_tree_parents(rng, n), W.random_tree_parents(rng, max(2, n // 2))],
                 Hq=2, Hkv=1, d=64, L=[5, 9], V=50, T_max=48, seed=seed)
    w.mode, w.K_max = mode, budget
    w.keep_count = rng.integers(1, n + 3, size=2).astype(np.int32)
    w.gate_depth, w.node_threshold = int(rng.integers(0, 4)), float(np.float32(-1.5))
    w.tmpl_parent, w.tmpl_rank = W.paper_template("d5", 8)
    if seed % 3 == 0:                                                   # ties in the scores
        w.draft_score = np.round(w.draft_score)
    if seed % 5 == 1:                                                   # children may outscore parents
        w.draft_score = rng.normal(size=w.draft_score.shape).astype(np.float32)
    o = orc.build_tree(w)
    check_structure(o, w)
    for b in range(2):
        tok, parent, src = independent_build(w, b)
        T = len(tok)
        assert o["tree_size"][b] == T and T <= budget
        assert o["tree_token"][b, :T].tolist() == tok
        assert o["tree_parent"][b, :T].tolist() == parent
        assert o["tree_src"][b, :T].tolist() == src


def test_malformed_inputs_have_defined_results(orc):
    rng = np.random.default_rng(1)
    w = W.custom([W.random_tree_parents(rng, 10)] * 3, Hq=2, Hkv=1, d=64, L=[4, 4, 4], V=50, seed=1)
    w.draft_parent = w.draft_parent.copy()
    w.draft_token = w.draft_token.copy()
    w.n_draft = w.n_draft.copy()
    w.draft_parent[0, 4] = 7                  # points forward
    w.draft_token[1, 3] = 50                  # id == V
    w.n_draft[2] = 11                         # more nodes than N_max
    o = orc.build_tree(w)
    assert o["flags"] == orc.FLAG_BAD_PARENT | orc.FLAG_BAD_TOKEN | orc.FLAG_BAD_SIZE
    check_structure(o, w)
    dropped = {i for i in range(10) if 4 in climb(np.where(np.arange(10) == 4, -1, w.draft_parent[0]), i)}
    assert o["tree_size"][0] == 10 - len(dropped)
    assert o["tree_token"][1, 3] == -1 and o["tree_size"][1] == 10
    assert o["tree_size"][2] == 0 and (o["tree_anc"][2] == 0).all()
