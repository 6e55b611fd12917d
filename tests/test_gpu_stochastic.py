"""Stochastic acceptance on the GPU against the oracle, through the C ABI.

The kernel computes in float32, the oracle in float64; the outcome of a draw is only defined up to that
rounding when a random number sits on a decision boundary, so requests are compared where the oracle's
margin (smallest distance of a random number from a boundary, relative to the remaining mass) is above
1e-3 (float32 sums over V exponentials are good to ~1e-5), and most requests must qualify.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_20104_b200 import binding as G
from paper_2605_20104_b200 import workloads as W
from paper_2605_20104_b200.step import VerifyStep

pytestmark = pytest.mark.gpu
MARGIN = 1e-3


def _compare(ref, got, min_share=0.8, check_bonus=None):
    ok = ref["margin"][:, 0] >= MARGIN
    assert ok.mean() >= min_share, ok.mean()
    for key in ("n_acc", "best_node"):
        assert (got[key][ok] == ref[key][ok]).all(), key
    assert (got["path"][ok] == ref["path"][ok]).all()
    # whatever the rounding, a result is a path from the root
    assert ((got["path"][:, 0] == 0) | (got["n_acc"] == 0)).all()
    sure = ok & (ref["margin"][:, 1] >= MARGIN)
    assert (got["bonus"][sure] == ref["bonus"][sure]).all()
    if check_bonus is not None:          # a draw that lands in a sliver of the distribution: any id whose interval is within rounding of the target
        for b in np.nonzero(ok & ~sure)[0]:
            check_bonus(int(b), int(got["bonus"][b]))
    return int(ok.sum())


def _bonus_checker(lg_bits, temp, tok, par, size, ref, ub, T_max, tol=1e-4):
    f = torch.from_numpy(lg_bits.view(np.int16)).view(torch.bfloat16).double().numpy()

    def check(b, pick):
        u = int(ref["best_node"][b])
        z = f[b * T_max + u] / temp
        p = np.exp(z - z.max())
        p /= p.sum()
        for c in range(u + 1, int(size[b])):            # the walk ended at u: every child of u was rejected
            if par[b, c] == u and tok[b, c] >= 0:
                p[tok[b, c]] = 0.0
        rem = p.sum()
        cdf = np.cumsum(p)
        target = float(ub[b]) * rem
        before = cdf[pick - 1] if pick > 0 else 0.0
        assert p[pick] > 0 and before - tol * rem <= target <= cdf[pick] + tol * rem, (b, pick, int(ref["bonus"][b]))
    return check


def _gpu(vs, lg_bits, temp, ua, ub):
    lg = torch.from_numpy(lg_bits.view(np.int16)).view(torch.bfloat16).cuda()
    vs.accept_stochastic(lg, temp, torch.from_numpy(ua).cuda(), torch.from_numpy(ub).cuda())
    torch.cuda.synchronize()
    return vs.accept_host()


@pytest.mark.parametrize("cfg,temp", [("1", 1.0), ("3", 1.0), ("5", 1.0), ("5", 0.6), ("4", 1.3)])
def test_workload_trees(cfg, temp):
    w = W.config(cfg) if cfg != "4" else W.config("4", L=512)
    tree = oracle.build_tree(w)
    lg = W.make_logits(w.B, w.T_max, w.V, seed=w.seed + 5)
    # make candidates likely: give each node's first children some of the parent's mass
    f = torch.from_numpy(lg.view(np.int16)).view(torch.bfloat16).float().numpy().reshape(w.B, w.T_max, w.V)
    rng = np.random.default_rng(w.seed + 9)
    for b in range(w.B):
        for i in range(1, int(tree["tree_size"][b])):
            x, par = int(tree["tree_token"][b, i]), int(tree["tree_parent"][b, i])
            if x >= 0 and rng.random() < 0.7:
                f[b, par, x] = f[b, par].max() + rng.normal()
    lg = torch.from_numpy(f.reshape(-1, w.V)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    ua = rng.random((w.B, w.T_max), dtype=np.float32)
    ub = rng.random(w.B, dtype=np.float32)
    ref = oracle.accept_stochastic(lg, temp, tree["tree_token"], tree["tree_parent"], tree["tree_size"], ua, ub)
    vs = VerifyStep(w, upload_qkv=False)
    vs.build()
    got = _gpu(vs, lg, temp, ua, ub)
    _compare(ref, got, 0.7 if w.B >= 4 else 0.0,
             _bonus_checker(lg, temp, tree["tree_token"], tree["tree_parent"], tree["tree_size"], ref, ub, w.T_max))
    assert vs.ctx.device_status() == 0
    assert w.B < 4 or ref["n_acc"].max() >= 2          # some candidate was accepted somewhere


@pytest.mark.parametrize("V", [1000, 1003, 40])
def test_many_small_requests(V):
    """Random trees, small vocabularies (many accepted nodes, ragged row tails)."""
    rng = np.random.default_rng(V)
    B, T = 300, 24
    parents = [W.random_tree_parents(rng, T) for _ in range(B)]
    w = W.custom(parents, Hq=8, Hkv=8, d=128, L=[64] * B, V=V, seed=V)
    tree = oracle.build_tree(w)
    size = tree["tree_size"].copy()
    tok = tree["tree_token"].copy()
    tok[:, 1:] = rng.integers(0, min(V, 12), size=(B, tree["tree_token"].shape[1] - 1))      # a dozen hot tokens: repeats among siblings
    f = (rng.normal(size=(B, w.T_max, V)) * 2.0).astype(np.float32)
    f[:, :, :12] += 6.0                       # most of the mass sits on the hot tokens, so children are often accepted
    lg = torch.from_numpy(f.reshape(-1, V)).to(torch.bfloat16)
    stride = (V + 7) // 8 * 8
    buf = torch.zeros(B * w.T_max, stride, dtype=torch.bfloat16)
    buf[:, :V] = lg
    ua = rng.random((B, w.T_max), dtype=np.float32)
    ub = rng.random(B, dtype=np.float32)
    ref = oracle.accept_stochastic(lg.view(torch.int16).numpy().view(np.uint16), 1.0, tok, tree["tree_parent"], size, ua, ub)
    vs = VerifyStep(w, upload_qkv=False)
    vs.build()
    vs.tree_token.copy_(torch.from_numpy(tok))
    dev = buf.cuda()
    vs.accept_stochastic(dev[:, :V], 1.0, torch.from_numpy(ua).cuda(), torch.from_numpy(ub).cuda())
    torch.cuda.synchronize()
    n = _compare(ref, vs.accept_host(), 0.9, _bonus_checker(lg.view(torch.int16).numpy().view(np.uint16), 1.0, tok,
                                                                tree["tree_parent"], size, ref, ub, w.T_max))
    assert n > 250 and ref["n_acc"].max() >= 3


def test_sizes_out_of_range_and_arguments():
    w = W.config("1", B=3)
    vs = VerifyStep(w, upload_qkv=False)
    vs.build()
    vs.tree_size.copy_(torch.tensor([0, w.T_max + 1, 1], dtype=torch.int32))
    lg = torch.zeros(w.B * w.T_max, w.V, dtype=torch.bfloat16, device="cuda")
    ua = torch.full((w.B, w.T_max), 0.5, device="cuda")
    ub = torch.full((w.B,), 0.5, device="cuda")
    vs.accept_stochastic(lg, 1.0, ua, ub)
    torch.cuda.synchronize()
    got = vs.accept_host()
    assert got["n_acc"].tolist() == [0, 0, 1] and got["bonus"][:2].tolist() == [-1, -1]
    assert got["bonus"][2] == w.V // 2       # uniform distribution, u = 0.5: the first id whose running sum passes one half
    assert vs.ctx.device_status() == G.FLAG_BAD_SIZE
    with pytest.raises(G.GraftError):
        vs.accept_stochastic(lg, 0.0, ua, ub)
