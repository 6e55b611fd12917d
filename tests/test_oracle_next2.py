"""Pins of the oracle's retrieval envelope and candidate-path indices (CPU only).

Envelope: folding the rank path of every node over M from the root (the lookup equation applied
along a path written out in Python), the oracle's own tree assembly (a different routine that does
its own lookups) on every stage template of the paper-shaped workload, a permutation matrix whose
paths have a closed form, the propagation of empty rows, and the paper's printed shape of the full
template (80 nodes, depths 1..9 with 8+16+14+11+8+7+6+5+5 nodes).
Path indices: top-down enumeration over child lists (the oracle walks bottom-up), chain and star
trees, and the acceptance rule written over paths (longest matching prefix over all candidate paths)
against the oracle's parent-pointer acceptance.
"""
import numpy as np
import pytest

import oracle
from paper_2605_20104_b200 import workloads as W


def _fold(M, root, path):
    x = int(root)
    for r in path:
        if x < 0:
            return -1
        x = int(M[x, r])
    return x


def test_envelope_equals_fold_of_rank_paths():
    rng = np.random.default_rng(5)
    V, k = 257, 8
    M = rng.integers(0, V, size=(V, k)).astype(np.int32)
    tp, tr = W.paper_template("full", k)
    paths = W.rank_path_tree(W.PAPER_TEMPLATE_WIDTHS["full"], [k] * 9)     # the paths themselves, not the parent lists
    roots = rng.integers(0, V, size=7).astype(np.int32)
    out = oracle.retrieve_envelope(roots, M, tp, tr)
    assert out["flags"] == 0
    for b, root in enumerate(roots):
        want = [_fold(M, root, q) for q in paths]
        assert out["env_token"][b].tolist() == want


def test_full_template_shape_as_printed():
    tp, tr = W.paper_template("full", 8)
    assert len(tp) == 80
    depth = np.zeros(len(tp), int)
    for u, f in enumerate(tp):
        depth[u] = 1 if f < 0 else depth[f] + 1
    assert np.bincount(depth)[1:].tolist() == [8, 16, 14, 11, 8, 7, 6, 5, 5]
    # the greedy chain (rank 0 all the way) reaches depth 9
    assert (0,) * 9 in W.template_rank_paths(tp, tr)


def test_envelope_closed_form_on_a_shift_matrix():
    # M[v, r] = v + r + 1 (mod V): a node's token is root + sum of (rank + 1) along its path
    V, k = 1009, 8
    M = ((np.arange(V)[:, None] + np.arange(k)[None, :] + 1) % V).astype(np.int32)
    tp, tr = W.paper_template("d0", k)
    paths = W.template_rank_paths(tp, tr)
    roots = np.asarray([0, 17, 1008], np.int32)
    out = oracle.retrieve_envelope(roots, M, tp, tr)
    for b, root in enumerate(roots):
        assert out["env_token"][b].tolist() == [(int(root) + sum(q) + len(q)) % V for q in paths]


def test_envelope_empty_rows_and_missing_root():
    V, k = 64, 4
    rng = np.random.default_rng(2)
    M = rng.integers(0, V, size=(V, k)).astype(np.int32)
    tp, tr = W.chains_template([3, 2])
    M[5, 0] = -1                                    # the first chain breaks at its first node
    out = oracle.retrieve_envelope(np.asarray([5, -1, 70], np.int32), M, tp, tr)
    assert out["env_token"][0, :3].tolist() == [-1, -1, -1]
    assert out["env_token"][0, 3] == M[5, 1] and out["env_token"][0, 4] == M[M[5, 1], 0]
    assert (out["env_token"][1] == -1).all() and (out["env_token"][2] == -1).all()
    assert out["flags"] == oracle.FLAG_BAD_TOKEN     # root 70 is outside [-1, V)
    bad = oracle.retrieve_envelope(np.asarray([1], np.int32), M, np.asarray([-1, 1], np.int32), np.asarray([0, 9], np.int32))
    assert bad["flags"] == oracle.FLAG_BAD_TEMPLATE and bad["env_token"][0, 1] == -1


def test_root_stride_reads_the_first_draft_token():
    w = W.config("2")
    ep, er, _ = W.workload_envelope(w)
    a = oracle.retrieve_envelope(w.draft_token, w.M, ep, er, root_stride=w.N_max)
    b = oracle.retrieve_envelope(np.ascontiguousarray(w.draft_token[:, 0]), w.M, ep, er)
    assert (a["env_token"] == b["env_token"]).all() and a["env_token"].shape == (w.B, len(ep))


@pytest.mark.parametrize("cfg", ["3", "4", "5"])
def test_stage_templates_select_from_the_envelope(cfg):
    """The grafted tokens of an assembled tree are the envelope's tokens of the same rank paths: for every
    request one stage's index map reproduces all of them."""
    w = W.config(cfg)
    tree = oracle.build_tree(w)
    ep, er, tmpl_env = W.workload_envelope(w)
    env = oracle.retrieve_envelope(w.draft_token, w.M, ep, er, root_stride=w.N_max)["env_token"]
    off = [0, len(w.tmpl_parent)] if w.tmpl_offset is None else w.tmpl_offset.tolist()
    n_graft = 0
    for b in range(w.B):
        grafted = [(i, -1 - int(tree["tree_src"][b, i])) for i in range(int(tree["tree_size"][b])) if tree["tree_src"][b, i] < 0]
        if not grafted:
            continue
        n_graft += len(grafted)
        stages = [s for s in range(len(off) - 1) if max(u for _, u in grafted) < off[s + 1] - off[s]
                  and all(env[b, tmpl_env[off[s] + u]] == tree["tree_token"][b, i] for i, u in grafted)]
        assert stages, b
    assert n_graft > 0


def _top_down_paths(parent, T):
    kids = [[] for _ in range(T)]
    for i in range(1, T):
        kids[parent[i]].append(i)
    out = []

    def walk(i, prefix):
        prefix = prefix + [i]
        if not kids[i]:
            out.append(prefix)
        for c in kids[i]:
            walk(c, prefix)
    if T > 0:
        walk(0, [])
    return sorted(out, key=lambda q: q[-1])         # leaves in increasing node index


@pytest.mark.parametrize("seed", range(6))
def test_paths_against_top_down_enumeration(seed):
    rng = np.random.default_rng(seed)
    B, T_max, D_max = 5, 24, 24
    parent = np.full((B, T_max), -1, np.int32)
    size = rng.integers(0, T_max + 1, size=B).astype(np.int32)
    size[0] = T_max
    for b in range(B):
        parent[b, :size[b]] = W.random_tree_parents(rng, int(size[b]))[:size[b]] if size[b] else []
    out = oracle.path_indices(parent, size, D_max)
    assert out["flags"] == 0
    for b in range(B):
        want = _top_down_paths(parent[b].tolist(), int(size[b]))
        assert out["n_paths"][b] == len(want)
        for j, q in enumerate(want):
            assert out["path_index"][b, j, :len(q)].tolist() == q
            assert (out["path_index"][b, j, len(q):] == -1).all()
        assert (out["path_index"][b, len(want):] == -1).all()


def test_paths_chain_star_and_truncation():
    T = 9
    chain = W.chain_parents(T)[None, :]
    star = W.star_parents(T)[None, :]
    c = oracle.path_indices(chain, [T], T)
    assert c["n_paths"][0] == 1 and c["path_index"][0, 0].tolist() == list(range(T))
    s = oracle.path_indices(star, [T], 3)
    assert s["n_paths"][0] == T - 1
    assert s["path_index"][0, :T - 1].tolist() == [[0, i, -1] for i in range(1, T)]
    t = oracle.path_indices(chain, [T], 4)          # the chain is deeper than the table is wide
    assert t["flags"] == oracle.FLAG_BAD_SIZE and t["path_index"][0, 0].tolist() == [0, 1, 2, 3]
    e = oracle.path_indices(chain, [0], 4)
    assert e["n_paths"][0] == 0 and (e["path_index"] == -1).all()


@pytest.mark.parametrize("cfg", ["1", "2", "5"])
def test_acceptance_over_paths_equals_acceptance_over_parents(cfg):
    """Greedy acceptance written over candidate paths (a node is accepted while it carries the target's
    id at its parent; the longest accepted prefix over all paths wins) gives the accepted length of
    the parent-pointer rule."""
    w = W.config(cfg)
    tree = oracle.build_tree(w)
    nxt = W.draw_target_next(tree["tree_token"], tree["tree_parent"], tree["tree_size"], tree["tree_src"], w.V,
                             w.p_draft, w.p_graft, w.seed)
    acc = oracle.accept(tree["tree_token"], tree["tree_parent"], tree["tree_size"], nxt)
    paths = oracle.path_indices(tree["tree_parent"], tree["tree_size"], w.T_max)
    for b in range(w.B):
        best = 0
        for j in range(int(paths["n_paths"][b])):
            q = [i for i in paths["path_index"][b, j].tolist() if i >= 0]
            n = 0
            for parent_node, node in zip(q[:-1], q[1:]):
                if tree["tree_token"][b, node] < 0 or tree["tree_token"][b, node] != nxt[b, parent_node]:
                    break
                n += 1
            best = max(best, n)
        # the accepted path counts the root
        assert int(acc["n_acc"][b]) == (best + 1 if tree["tree_size"][b] > 0 else 0)


def test_tail_grafting_continues_the_kept_prefix():
    """Block drafter with tail grafting: the kept prefix of the drafted chain, then the rank-0 chain of the
    adjacency matrix from the last kept token on; the result is again one chain of the block's length."""
    w = W.tail_block(B=6, L=300, block=16, V=997)
    tree = oracle.build_tree(w)
    assert tree["flags"] == 0
    for b in range(w.B):
        keep = int(w.keep_count[b])
        assert tree["tree_size"][b] == 16
        assert tree["tree_parent"][b].tolist() == [-1] + list(range(15))            # one chain
        assert tree["tree_token"][b, :keep].tolist() == w.draft_token[b, :keep].tolist()
        x = int(w.draft_token[b, keep - 1])
        for i in range(keep, 16):                                                     # x_{i} = M[x_{i-1}, 0], -1 propagates
            x = int(w.M[x, 0]) if x >= 0 else -1
            assert tree["tree_token"][b, i] == x
        assert tree["tree_pos"][b].tolist() == list(range(300, 316))
        assert tree["tree_src"][b].tolist() == list(range(keep)) + [-1 - u for u in range(16 - keep)]
    # the same template hung off the root instead gives a star of two chains
    w.attach_tail = False
    root = oracle.build_tree(w)
    b = int(np.argmin(w.keep_count))
    keep = int(w.keep_count[b])
    assert root["tree_parent"][b, keep] == 0 and root["tree_token"][b, keep] == w.M[w.draft_token[b, 0], 0]
