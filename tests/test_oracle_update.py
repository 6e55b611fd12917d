"""Pins of the oracle's adjacency update (the appendix equation M[x_i] <- argtopk(p_{i+1})): checked against
things that are not the oracle itself: a library stable sort, softmax probabilities in fp64, a row worked by
hand, and the sequential meaning of "the node with the highest index wins"."""
import numpy as np
import torch

from paper_2605_20104_b200 import workloads as W


def bits(x):
    return W.bf16_bits(torch.tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16))


def widen(b):
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def test_hand_worked_row(orc):
    # ids:        0    1    2    3     4      5     6    7
    row = [1.0, 5.0, 5.0, 3.0, np.nan, -np.inf, -0.0, 0.0]
    lg = bits([row])
    M = np.full((8, 4), -7, np.int32)
    out = orc.update_adjacency(lg, np.array([[2]], np.int32), np.array([1], np.int32), M, 4)
    assert out["M"][2].tolist() == [1, 2, 3, 0]            # 5, 5 (lower id first), 3, 1
    assert out["target_next"].tolist() == [[1]]
    assert (np.delete(out["M"], 2, axis=0) == -7).all()      # no other row changes
    assert out["flags"] == 0
    out = orc.update_adjacency(lg, np.array([[2]], np.int32), np.array([1], np.int32), np.full((8, 8), -7, np.int32), 8)
    # then -0.0 and 0.0 are equal (lower id first), then -inf; NaN is never chosen: the list ends with -1
    assert out["M"][2].tolist() == [1, 2, 3, 0, 6, 7, 5, -1]
    assert out["flags"] == 64


def test_against_stable_sort_with_many_ties(orc):
    rng = np.random.default_rng(0)
    B, T, V, k = 3, 5, 97, 8
    x = rng.integers(-4, 5, size=(B * T, V)).astype(np.float32) * 0.5       # few distinct values: ties everywhere
    lg = bits(x)
    tok = rng.permutation(V)[:B * T].reshape(B, T).astype(np.int32)      # all tokens distinct
    size = np.array([5, 3, 0], np.int32)
    M0 = rng.integers(0, V, size=(V, k)).astype(np.int32)
    out = orc.update_adjacency(lg, tok, size, M0, k)
    exp = M0.copy()
    for b in range(B):
        for i in range(T):
            r = b * T + i
            if i < size[b]:
                order = np.argsort(-widen(lg[r]), kind="stable")[:k]      # equal values keep increasing id
                exp[tok[b, i]] = order
                assert out["target_next"][b, i] == int(np.argmax(widen(lg[r])))
            else:
                assert out["target_next"][b, i] == -1
    assert (out["M"] == exp).all()


def test_same_ids_as_softmax_probabilities(orc):
    """argtopk of the distribution equals argtopk of the logits wherever the probabilities differ."""
    rng = np.random.default_rng(1)
    V, k = 300, 8
    x = rng.standard_normal((1, V)).astype(np.float32) * 3
    lg = bits(x)
    z = widen(lg[0])
    p = np.exp(z - z.max())
    p /= p.sum()
    out = orc.update_adjacency(lg, np.array([[7]], np.int32), np.array([1], np.int32), np.zeros((V, k), np.int32), k)
    got = out["M"][7]
    assert (np.diff(p[got]) <= 0).all()
    assert p[got].min() >= np.sort(p)[-k]


def test_highest_node_index_wins_and_order_of_requests(orc):
    rng = np.random.default_rng(2)
    B, T, V, k = 2, 4, 50, 3
    lg = bits(rng.standard_normal((B * T, V)).astype(np.float32))
    tok = np.array([[9, 4, 9, 1], [4, 9, -1, 2]], np.int32)     # token 9 at rows 0, 2, 5; token 4 at rows 1, 4
    size = np.array([4, 3], np.int32)
    out = orc.update_adjacency(lg, tok, size, np.zeros((V, k), np.int32), k)
    top = lambda r: np.argsort(-widen(lg[r]), kind="stable")[:k]
    assert (out["M"][9] == top(5)).all() and (out["M"][4] == top(4)).all() and (out["M"][1] == top(3)).all()
    assert (out["M"][2] == 0).all()                              # row 7 is padding (size 3): token 2 untouched
    assert out["flags"] == 0                                     # token -1 is legal and updates nothing


def test_bad_inputs_are_flagged(orc):
    lg = bits(np.zeros((2, 10), np.float32))
    out = orc.update_adjacency(lg, np.array([[10, 3]], np.int32), np.array([2], np.int32), np.zeros((10, 2), np.int32), 2)
    assert out["flags"] == 4 and out["M"][3].tolist() == [0, 1]
    out = orc.update_adjacency(lg, np.array([[1, 3]], np.int32), np.array([3], np.int32), np.ones((10, 2), np.int32), 2)
    assert out["flags"] == 1 and (out["M"] == 1).all() and (out["target_next"] == -1).all()
