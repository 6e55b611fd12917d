"""Pins of the oracle's stochastic acceptance (CPU only).

A hand-worked three-token example covering every branch, the empirical distribution of the first
emitted token over many draws against the target distribution (the lossless-equivalence
proposition), the distribution of the second token given the first, the limit of a very low
temperature against greedy acceptance, leaves and duplicate siblings.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_20104_b200 import workloads as W


def _bits(x):
    return torch.from_numpy(np.asarray(x, np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def _run(logits, temp, tok, par, size, ua, ub):
    B, T = np.asarray(tok).shape
    return oracle.accept_stochastic(_bits(logits).reshape(B * T, -1), temp, tok, par, size, ua, ub)


def test_hand_worked_example():
    # p = (0.5, 0.25, 0.25) at the root; children: node 1 carries token 0, node 2 token 1
    lg = np.log(np.asarray([0.5, 0.25, 0.25]))
    logits = np.tile(lg, (1, 3, 1))
    tok = np.asarray([[7, 0, 1]], np.int32)
    par = np.asarray([[-1, 0, 0]], np.int32)
    size = np.asarray([3], np.int32)

    def go(u1, u2, ub):
        return _run(logits, 1.0, tok, par, size, np.asarray([[0, u1, u2]], np.float32), np.asarray([ub], np.float32))
    r = go(0.4, 0.9, 0.1)                 # 0.4 < 0.5: node 1 accepted; it is a leaf; bonus from p: 0.1 -> token 0
    assert r["path"][0].tolist() == [0, 1, -1] and r["n_acc"][0] == 2 and r["best_node"][0] == 1 and r["bonus"][0] == 0
    r = go(0.4, 0.9, 0.6)                 # bonus 0.6 -> cumulative 0.5, 0.75: token 1
    assert r["bonus"][0] == 1
    r = go(0.6, 0.4, 0.0)                 # node 1 rejected, rem 0.5; node 2: 0.4 * 0.5 < 0.25 accepted
    assert r["path"][0].tolist() == [0, 2, -1] and r["best_node"][0] == 2
    r = go(0.6, 0.6, 0.3)                 # both rejected (0.6 * 0.5 >= 0.25): bonus from {2: 0.25}
    assert r["n_acc"][0] == 1 and r["best_node"][0] == 0 and r["bonus"][0] == 2
    assert abs(r["margin"][0, 0] - 0.1) < 1e-6   # |0.6 - 0.5| / 1 is the closest accept decision
    assert abs(r["margin"][0, 1] - 0.3) < 1e-6   # the bonus draw: 0.3 * 0.25 sits 0.3 (of rem) inside token 2's interval


def test_duplicate_sibling_and_empty_token():
    lg = np.log(np.asarray([0.5, 0.25, 0.25]))
    logits = np.tile(lg, (1, 4, 1))
    tok = np.asarray([[9, 0, 0, -1]], np.int32)          # node 2 repeats node 1's token, node 3 has none
    par = np.asarray([[-1, 0, 0, 0]], np.int32)
    r = _run(logits, 1.0, tok, par, np.asarray([4], np.int32), np.asarray([[0, 0.9, 0.0, 0.0]], np.float32),
             np.asarray([0.9], np.float32))
    assert r["n_acc"][0] == 1 and r["bonus"][0] == 2      # 0.9 * 0.5 = 0.45 -> past token 1's 0.25


def _first_token_counts(V, tok, par, size, logits_row, n, seed, temp=1.0):
    rng = np.random.default_rng(seed)
    T = len(tok)
    logits = np.tile(np.asarray(logits_row, np.float32), (n, T, 1))
    ua = rng.random((n, T), dtype=np.float32)
    ub = rng.random(n, dtype=np.float32)
    r = _run(logits, temp, np.tile(tok, (n, 1)).astype(np.int32), np.tile(par, (n, 1)).astype(np.int32),
             np.full(n, size, np.int32), ua, ub)
    first = np.where(r["n_acc"] > 1, np.asarray(tok)[r["path"][:, 1].clip(0)], r["bonus"])
    return np.bincount(first, minlength=V), r


@pytest.mark.parametrize("seed", [0, 1])
def test_first_emitted_token_follows_the_target_distribution(seed):
    """Lossless equivalence: whatever the candidates are, the first token is a draw from p."""
    rng = np.random.default_rng(100 + seed)
    V, n = 7, 200000
    row = rng.normal(size=V).astype(np.float32) * 1.5
    row = torch.from_numpy(row).to(torch.bfloat16).float().numpy()     # the values the oracle will see
    p = np.exp(row - row.max()); p /= p.sum()
    tok = [3, 2, 5, 2, 0, 6]                 # root; children of the root: tokens 2, 5, 2 (repeat), 0; node 5 under node 1
    par = [-1, 0, 0, 0, 0, 1]
    counts, _ = _first_token_counts(V, tok, par, 6, row, n, seed)
    sigma = np.sqrt(n * p * (1 - p))
    assert (np.abs(counts - n * p) < 4.5 * sigma + 1).all(), (counts / n, p)


def test_second_token_given_the_first():
    rng = np.random.default_rng(7)
    V, n = 5, 200000
    row = torch.from_numpy((rng.normal(size=V) * 1.2).astype(np.float32)).to(torch.bfloat16).float().numpy()
    p = np.exp(row - row.max()); p /= p.sum()
    tok = [0, 1, 2, 3]                        # node 1 (token 1) under the root; nodes 2, 3 under node 1
    par = [-1, 0, 1, 1]
    _, r = _first_token_counts(V, tok, par, 4, row, n, 3)
    took = r["n_acc"] >= 2                    # node 1 accepted: happens with probability p[1]
    assert abs(took.mean() - p[1]) < 4.5 * np.sqrt(p[1] * (1 - p[1]) / n)
    second = np.where(r["n_acc"][took] > 2, np.asarray(tok)[r["path"][took, 2].clip(0)], r["bonus"][took])
    m = took.sum()
    c = np.bincount(second, minlength=V)
    assert (np.abs(c - m * p) < 4.5 * np.sqrt(m * p * (1 - p)) + 1).all()


@pytest.mark.parametrize("cfg", ["1", "5"])
def test_low_temperature_is_greedy_acceptance(cfg):
    w = W.config(cfg)
    tree = oracle.build_tree(w)
    lg = W.make_logits(w.B, w.T_max, w.V, seed=w.seed + 3)
    upd = oracle.update_adjacency(lg, tree["tree_token"], tree["tree_size"], w.M, w.k)
    greedy = oracle.accept(tree["tree_token"], tree["tree_parent"], tree["tree_size"], upd["target_next"])
    rng = np.random.default_rng(1)
    ua = (0.05 + 0.9 * rng.random((w.B, w.T_max))).astype(np.float32)
    ub = (0.05 + 0.9 * rng.random(w.B)).astype(np.float32)
    r = oracle.accept_stochastic(lg, 1e-3, tree["tree_token"], tree["tree_parent"], tree["tree_size"], ua, ub)
    # bf16 logits tie now and then; where the largest logit is unique the two rules coincide
    f = torch.from_numpy(lg.view(np.int16)).view(torch.bfloat16).float().numpy().reshape(w.B, w.T_max, w.V)
    for b in range(w.B):
        rows = [i for i in greedy["path"][b].tolist() if i >= 0]
        top2 = np.sort(f[b, rows], axis=1)[:, -2:]
        if (top2[:, 1] > top2[:, 0]).all():
            assert r["path"][b].tolist() == greedy["path"][b].tolist()
            assert r["bonus"][b] == greedy["bonus"][b]


def test_empty_and_oversized_trees():
    logits = np.zeros((2, 2, 4), np.float32)
    r = _run(logits, 1.0, np.zeros((2, 2), np.int32), np.full((2, 2), -1, np.int32), np.asarray([0, 3], np.int32),
             np.zeros((2, 2), np.float32), np.zeros(2, np.float32))
    assert r["n_acc"].tolist() == [0, 0] and r["bonus"].tolist() == [-1, -1] and r["flags"] == oracle.FLAG_BAD_SIZE
