"""Pins for the oracle's greedy acceptance and KV compaction, CPU only.

Acceptance: explicit enumeration of every root-to-node path, the textbook chain case (longest
matching prefix), the all-match and no-match extremes, and the paper's Propositions 1 and 2
(removing candidates never lengthens, grafting never shortens the accepted path).
Compaction: the closed form new[L + j] = old[L + path[j]] in numpy, identity and overlap cases.
"""
import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

from paper_2605_20104_b200 import workloads as W


def enumerate_paths(tok, par, T, nxt):
    """Every root-to-node path, scanned token by token: returns (length, node) of the winner."""
    best = (1, 0)
    for i in range(T):
        path = []
        j = i
        while j >= 0:
            path.append(j)
            j = int(par[j])
        path.reverse()
        good = all(tok[c] >= 0 and tok[c] == nxt[p] for p, c in zip(path[:-1], path[1:]))
        if good and (len(path) > best[0]):
            best = (len(path), i)
    return best


def random_case(rng, T, V=6, T_max=None):
    T_max = T_max or T
    par = np.full(T_max, -1, np.int32)
    par[:T] = W.random_tree_parents(rng, T)
    tok = np.full(T_max, -1, np.int32)
    tok[:T] = rng.integers(-1, V, size=T)          # includes the empty-retrieval sentinel -1
    nxt = rng.integers(0, V, size=T_max).astype(np.int32)
    return tok, par, nxt


@settings(max_examples=150, deadline=None)
@given(st.integers(0, 100_000), st.integers(1, 24))
def test_accept_equals_path_enumeration(seed, T):
    import oracle as orc
    rng = np.random.default_rng(seed)
    tok, par, nxt = random_case(rng, T, T_max=24)
    o = orc.accept(tok[None], par[None], np.array([T], np.int32), nxt[None])
    n, best = enumerate_paths(tok, par, T, nxt)
    assert o["n_acc"][0] == n and o["best_node"][0] == best
    assert o["bonus"][0] == nxt[best]
    path = o["path"][0]
    assert (path[n:] == -1).all() and path[0] == 0 and path[n - 1] == best
    assert all(par[path[j]] == path[j - 1] for j in range(1, n))
    assert all(path[j] >= j for j in range(n)) and (np.diff(path[:n]) > 0).all()


def test_chain_is_longest_matching_prefix(orc):
    T = 10
    par = W.chain_parents(T)
    tok = np.arange(100, 100 + T, dtype=np.int32)
    for first_miss in range(1, T + 1):
        nxt = np.concatenate([tok[1:], [7]]).astype(np.int32)            # target agrees everywhere ...
        if first_miss < T:
            nxt[first_miss - 1] = 5                                        # ... until this edge
        o = orc.accept(tok[None], par[None], np.array([T], np.int32), nxt[None])
        assert o["n_acc"][0] == first_miss
        assert o["path"][0, :first_miss].tolist() == list(range(first_miss))
        assert o["bonus"][0] == nxt[first_miss - 1]


def test_extremes(orc):
    w = W.config("2")
    tree = orc.build_tree(w)
    tok, par, size = tree["tree_token"], tree["tree_parent"], tree["tree_size"]
    # p = 0: nothing matches -> only the root, bonus is the target's id after the root
    nxt = np.full_like(tok, -5)
    o = orc.accept(tok, par, size, nxt)
    assert (o["n_acc"] == 1).all() and (o["best_node"] == 0).all() and (o["bonus"] == -5).all()
    # every node matches (all tokens equal the target's id everywhere): deepest node, lowest index
    tok1 = np.where(tok >= 0, 3, tok)
    nxt = np.full_like(tok, 3)
    o = orc.accept(tok1, par, size, nxt)
    depth = np.array([bin(int(a)).count("1") - 1 for a in tree["tree_anc"][0]])
    assert (o["n_acc"] == depth.max() + 1).all()
    assert (o["best_node"] == int(np.argmax(depth))).all()


def test_sentinel_never_matches(orc):
    par = W.chain_parents(3)
    tok = np.array([4, -1, 9], np.int32)
    nxt = np.array([-1, 9, 0], np.int32)                                   # even a -1 "target" must not match
    o = orc.accept(tok[None], par[None], np.array([3], np.int32), nxt[None])
    assert o["n_acc"][0] == 1


@settings(max_examples=100, deadline=None)
@given(st.integers(0, 100_000), st.integers(2, 20))
def test_prop1_removing_a_subtree_never_lengthens(seed, T):
    """Proposition 1: T1 subset of T2 -> accepted length on T1 <= on T2."""
    import oracle as orc
    rng = np.random.default_rng(seed)
    tok, par, nxt = random_case(rng, T, V=3)
    full = orc.accept(tok[None], par[None], np.array([T], np.int32), nxt[None])["n_acc"][0]
    cut = int(rng.integers(1, T))                                          # drop node `cut` and its subtree
    gone = np.zeros(T, bool)
    for i in range(T):
        gone[i] = (i == cut) or (par[i] >= 0 and gone[par[i]])
    keep = np.nonzero(~gone)[0]
    new = -np.ones(T, int)
    new[keep] = np.arange(len(keep))
    tok2 = tok[keep]
    par2 = np.array([-1 if par[i] < 0 else new[par[i]] for i in keep], np.int32)
    nxt2 = nxt[keep]
    sub = orc.accept(tok2[None], par2[None], np.array([len(keep)], np.int32), nxt2[None])["n_acc"][0]
    assert sub <= full


@settings(max_examples=100, deadline=None)
@given(st.integers(0, 100_000), st.integers(1, 12), st.integers(1, 10))
def test_prop2_grafting_never_shortens(seed, T, extra):
    """Proposition 2: appending grafted nodes to a fixed pruned tree cannot reduce acceptance."""
    import oracle as orc
    rng = np.random.default_rng(seed)
    tok, par, nxt = random_case(rng, T, V=3)
    base = orc.accept(tok[None], par[None], np.array([T], np.int32), nxt[None])["n_acc"][0]
    tok2 = np.concatenate([tok, rng.integers(0, 3, size=extra)]).astype(np.int32)
    par2 = np.concatenate([par, [rng.integers(0, T + j) for j in range(extra)]]).astype(np.int32)
    nxt2 = np.concatenate([nxt, rng.integers(0, 3, size=extra)]).astype(np.int32)
    more = orc.accept(tok2[None], par2[None], np.array([T + extra], np.int32), nxt2[None])["n_acc"][0]
    assert more >= base


# ----------------------------------------------------------------------------- compaction

def cache(rng, nl, B, Hkv, S, d):
    return rng.integers(0, 2 ** 16, size=(nl, B, Hkv, S, d), dtype=np.uint16)


@pytest.mark.parametrize("paths", [[[0, 2, 3]], [[0, 63]], [[0, 1, 3, 4, 5, 9]], [[0]], [[0, 1, 2, 3]],
                                   [[0, 5, 6], [0, 1, 7, 8, 20]]])
def test_compaction_closed_form(orc, paths):
    rng = np.random.default_rng(0)
    B, T_max, nl, Hkv, d = len(paths), 64, 2, 2, 8
    L = np.array([3, 11][:B], np.int32)
    S = int(L.max()) + T_max
    K, V = cache(rng, nl, B, Hkv, S, d), cache(rng, nl, B, Hkv, S, d)
    path = np.full((B, T_max), -1, np.int32)
    n_acc = np.zeros(B, np.int32)
    for b, p in enumerate(paths):
        path[b, :len(p)] = p
        n_acc[b] = len(p)
    o = orc.compact_kv(K, V, L, n_acc, path)
    Kw, Vw = K.copy(), V.copy()
    for b, p in enumerate(paths):
        for j, node in enumerate(p):
            Kw[:, b, :, L[b] + j] = K[:, b, :, L[b] + node]
            Vw[:, b, :, L[b] + j] = V[:, b, :, L[b] + node]
    assert (o["K"] == Kw).all() and (o["V"] == Vw).all()
    assert (o["new_seq_len"] == L + n_acc).all()
    if all(p == list(range(len(p))) for p in paths):
        assert (o["K"] == K).all() and (o["V"] == V).all()                 # a path already in place
