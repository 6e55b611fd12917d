"""Pins for the oracle's tree-masked attention, CPU only.

Fixed by: a dense-mask brute force (mask built by climbing parent pointers), library SDPA for the
chain == causal case, plain decode attention for T = 1, row sums, mask locality, a constant-V
closed form, permutation invariance over prefix slots and split invariance through (LSE, O).
"""
import numpy as np
import pytest
import torch

from paper_2605_20104_b200 import workloads as W


def widen(t):
    return t.to(torch.float64).numpy()


def setup(orc, parents, Hq=4, Hkv=2, d=64, L=(37,), seed=0, T_max=None, std=1.0):
    w = W.custom(parents, Hq=Hq, Hkv=Hkv, d=d, L=list(L), seed=seed, T_max=T_max, std=std)
    tree = orc.build_tree(w)
    W.make_qkv(w, tree["tree_size"], poison=True)
    return w, tree


def run(orc, w, tree, **kw):
    return orc.tree_attn(W.bf16_bits(w.Q), W.bf16_bits(w.Kc), W.bf16_bits(w.Vc), w.seq_len,
                         tree["tree_size"], tree["tree_anc"], w.scale, **kw)


def dense_mask_attention(w, parents_b, b):
    """Brute force: boolean [T, L+T] mask from parent pointers, masked softmax in numpy fp64."""
    L, T = int(w.seq_len[b]), len(parents_b)
    mask = np.zeros((T, L + T), bool)
    mask[:, :L] = True
    for t in range(T):
        i = t
        while i >= 0:
            mask[t, L + i] = True
            i = int(parents_b[i])
    Q, K, V = widen(w.Q[b, :T]), widen(w.Kc[b, :, :L + T]), widen(w.Vc[b, :, :L + T])
    G = w.Hq // w.Hkv
    O = np.zeros((T, w.Hq, w.d))
    for h in range(w.Hq):
        s = (Q[:, h] @ K[h // G].T) * w.scale
        s = np.where(mask, s, -np.inf)
        p = np.exp(s - s.max(1, keepdims=True))
        p /= p.sum(1, keepdims=True)
        O[:, h] = p @ V[h // G]
    return O


def test_bruteforce_random_trees(orc):
    rng = np.random.default_rng(3)
    parents = [W.random_tree_parents(rng, 9), W.random_tree_parents(rng, 5), W.star_parents(7)]
    w, tree = setup(orc, parents, L=(37, 1, 12), seed=3, T_max=9)
    out = run(orc, w, tree)
    for b, p in enumerate(parents):
        T = len(p)
        np.testing.assert_allclose(out["O"][b, :T], dense_mask_attention(w, p, b), rtol=0, atol=1e-12)
        assert (out["O"][b, T:] == 0).all()                              # padding rows
        assert np.isneginf(out["LSE"][b, :, T:]).all()


def test_rows_sum_to_one(orc):
    rng = np.random.default_rng(4)
    w, tree = setup(orc, [W.random_tree_parents(rng, 12)], L=(200,), seed=4)
    out = run(orc, w, tree)
    np.testing.assert_allclose(out["rowsum"][0], 1.0, rtol=0, atol=1e-13)


def test_chain_equals_causal_sdpa(orc):
    T, L = 11, 29
    w, tree = setup(orc, [W.chain_parents(T)], Hq=4, Hkv=4, L=(L,), seed=5)
    out = run(orc, w, tree)
    q = w.Q[0, :T].to(torch.float64).permute(1, 0, 2)                    # [H, T, d]
    k = w.Kc[0, :, :L + T].to(torch.float64)
    v = w.Vc[0, :, :L + T].to(torch.float64)
    mask = torch.ones(T, L + T, dtype=torch.bool).tril(diagonal=L)       # query t sees keys <= L + t
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, attn_mask=mask, scale=w.scale)
    np.testing.assert_allclose(out["O"][0, :T], ref.permute(1, 0, 2).numpy(), rtol=0, atol=1e-12)


def test_single_node_equals_decode_attention(orc):
    L = 64
    w, tree = setup(orc, [np.array([-1], np.int32)], Hq=8, Hkv=2, L=(L,), seed=6, T_max=4)
    out = run(orc, w, tree)
    K, V, q = widen(w.Kc[0, :, :L + 1]), widen(w.Vc[0, :, :L + 1]), widen(w.Q[0, 0])
    for h in range(8):
        s = (K[h // 4] @ q[h]) * w.scale
        p = np.exp(s - s.max())
        np.testing.assert_allclose(out["O"][0, 0, h], (p / p.sum()) @ V[h // 4], rtol=0, atol=1e-12)
        np.testing.assert_allclose(out["LSE"][0, h, 0], s.max() + np.log(p.sum()), rtol=0, atol=1e-12)


def test_star_sees_prefix_root_and_self_only(orc):
    T, L = 6, 10
    w, tree = setup(orc, [W.star_parents(T)], Hq=2, Hkv=1, L=(L,), seed=7)
    base = run(orc, w, tree)["O"].copy()
    # changing sibling 3's K/V must not move any other row, bit for bit
    w.Kc[0, :, L + 3] += 1.0
    w.Vc[0, :, L + 3] -= 2.0
    out = run(orc, w, tree)["O"]
    for t in range(T):
        same = (out[0, t] == base[0, t]).all()
        assert same == (t != 3)


def test_mask_locality(orc):
    rng = np.random.default_rng(8)
    par = W.random_tree_parents(rng, 14)
    L = 50
    w, tree = setup(orc, [par], Hq=2, Hkv=1, L=(L,), seed=8)
    base = run(orc, w, tree)["O"].copy()
    anc = [set() for _ in par]
    for t in range(len(par)):
        i = t
        while i >= 0:
            anc[t].add(i)
            i = int(par[i])
    for u in (2, 7, 13):
        w2 = W.custom([par], Hq=2, Hkv=1, d=64, L=[L], seed=8)
        W.make_qkv(w2, tree["tree_size"], poison=True)
        w2.Vc[0, :, L + u] += 3.0
        out = run(orc, w2, tree)["O"]
        for t in range(len(par)):
            changed = not (out[0, t] == base[0, t]).all()
            assert changed == (u in anc[t]), (u, t)


def test_constant_v_gives_that_row(orc):
    rng = np.random.default_rng(9)
    w, tree = setup(orc, [W.random_tree_parents(rng, 8)], Hq=2, Hkv=1, L=(33,), seed=9)
    row = w.Vc[0, 0, 0].clone()
    w.Vc[0, 0, :33 + 8] = row
    out = run(orc, w, tree)
    np.testing.assert_allclose(out["O"][0, :8, :], np.broadcast_to(widen(row), (8, 2, 64)), rtol=0, atol=1e-13)


def test_prefix_permutation_invariance(orc):
    rng = np.random.default_rng(10)
    L = 40
    w, tree = setup(orc, [W.random_tree_parents(rng, 8)], Hq=2, Hkv=1, L=(L,), seed=10)
    base = run(orc, w, tree)["O"].copy()
    perm = torch.from_numpy(rng.permutation(L))
    w.Kc[0, :, :L] = w.Kc[0, :, :L][:, perm]
    w.Vc[0, :, :L] = w.Vc[0, :, :L][:, perm]
    np.testing.assert_allclose(run(orc, w, tree)["O"], base, rtol=0, atol=1e-12)


def test_split_invariance_via_lse(orc):
    """Attention over a key set equals the LSE-weighted merge of attention over its parts:
    this is the specification of a split-KV merge."""
    L = 90
    w, tree = setup(orc, [np.array([-1], np.int32)], Hq=4, Hkv=2, L=(L,), seed=11, T_max=1)
    full = run(orc, w, tree)
    parts = []
    for lo, hi in ((0, 17), (17, 64), (64, L + 1)):                       # the last part holds the root
        w2 = W.custom([np.array([-1], np.int32)], Hq=4, Hkv=2, d=64, L=[hi - lo - (hi == L + 1)], seed=11,
                      T_max=1, S_cap=L + 1)
        w2.Q = w.Q
        w2.Kc, w2.Vc = w.Kc.clone(), w.Vc.clone()
        w2.Kc[:, :, :hi - lo] = w.Kc[:, :, lo:hi]
        w2.Vc[:, :, :hi - lo] = w.Vc[:, :, lo:hi]
        if hi != L + 1:                                                    # no self key in this part
            anc = np.zeros_like(tree["tree_anc"])
        else:
            anc = tree["tree_anc"]
        o = orc.tree_attn(W.bf16_bits(w2.Q), W.bf16_bits(w2.Kc), W.bf16_bits(w2.Vc), w2.seq_len,
                          tree["tree_size"], anc, w.scale)
        parts.append((o["LSE"][0, :, 0], o["O"][0, 0]))
    lse = np.logaddexp.reduce([p[0] for p in parts], axis=0)
    merged = sum(np.exp(l - lse)[:, None] * o for l, o in parts)
    np.testing.assert_allclose(merged, full["O"][0, 0], rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, full["LSE"][0, :, 0], rtol=0, atol=1e-12)


def test_rows_subset_matches_full(orc):
    rng = np.random.default_rng(12)
    w, tree = setup(orc, [W.random_tree_parents(rng, 8), W.random_tree_parents(rng, 6)], L=(20, 31), seed=12, T_max=8)
    full = run(orc, w, tree)
    rows = np.array([[0, 3, 1], [1, 5, 2], [1, 0, 0]], np.int32)
    sub = run(orc, w, tree, rows=rows)
    for b, t, h in rows:
        assert (sub["O"][b, t, h] == full["O"][b, t, h]).all()
    assert np.isnan(sub["O"][0, 0, 0]).all()


def test_gqa_head_mapping(orc):
    """Query head h reads KV head h // G: zeroing one KV head's V zeroes exactly its group."""
    rng = np.random.default_rng(13)
    w, tree = setup(orc, [W.random_tree_parents(rng, 5)], Hq=6, Hkv=3, L=(16,), seed=13)
    w.Vc[0, 1] = 0
    out = run(orc, w, tree)["O"][0, :5]
    assert (out[:, 2:4] == 0).all() and (np.abs(out[:, :2]).sum() > 0) and (np.abs(out[:, 4:]).sum() > 0)
