"""The verify step captured once in a CUDA graph and replayed on new inputs of the same shapes (the
serving-shaped use: fixed launch configuration, everything data-dependent read on the device)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_20104_b200 import binding as G
from paper_2605_20104_b200 import workloads as W
from paper_2605_20104_b200.step import VerifyStep

pytestmark = pytest.mark.gpu


def _load(vs, w, nxt):
    """New inputs into the buffers the captured launches point at."""
    for name in ("draft_token", "draft_parent", "draft_score", "n_draft", "seq_len", "M"):
        getattr(vs, name).copy_(torch.from_numpy(np.ascontiguousarray(getattr(w, name))))
    if vs.keep_count is not None:
        vs.keep_count.copy_(torch.from_numpy(w.keep_count))
    if vs.k_max is not None:
        vs.k_max.copy_(torch.from_numpy(w.k_max))
    vs.Q.copy_(w.Q)
    vs.Kc.copy_(w.Kc)
    vs.Vc.copy_(w.Vc)
    vs.target_next.copy_(torch.from_numpy(nxt))


def _reference(w):
    tree = oracle.build_tree(w)
    W.make_qkv(w, tree["tree_size"], poison=True)
    nxt = W.draw_target_next(tree["tree_token"], tree["tree_parent"], tree["tree_size"], tree["tree_src"], w.V,
                             w.p_draft, w.p_graft, w.seed)
    attn = oracle.tree_attn(W.bf16_bits(w.Q), W.bf16_bits(w.Kc), W.bf16_bits(w.Vc), w.seq_len, tree["tree_size"],
                            tree["tree_anc"], w.scale)
    acc = oracle.accept(tree["tree_token"], tree["tree_parent"], tree["tree_size"], nxt)
    return tree, nxt, attn, acc


def _check(vs, w, tree, attn, acc):
    got = vs.tree_host()
    for key in ("tree_size", "tree_token", "tree_parent", "tree_pos", "tree_src", "tree_anc"):
        assert (got[key] == tree[key]).all(), key
    O = vs.O.cpu().double().numpy()
    for b in range(w.B):
        n = int(tree["tree_size"][b])
        err = np.abs(O[b, :n] - attn["O"][b, :n])
        assert err.max() <= 2e-2 and err.mean() <= 2e-3, (b, err.max(), err.mean())
    a = vs.accept_host()
    for key in ("n_acc", "path", "best_node", "bonus"):
        assert (a[key] == acc[key]).all(), key
    assert vs.ctx.device_status() == tree["flags"]


@pytest.mark.parametrize("cfg,kw,variant", [("3", dict(B=8, L=3000), G.ATTN_AUTO),                 # row-block kernel, merge inside the kernel
                                            ("4", dict(B=1, L=20000), G.ATTN_AUTO),                # two-SM kernel + merge kernel (dependent launch)
                                            ("5", dict(), G.ATTN_TCGEN05_1SM),
                                            ("2", dict(), G.ATTN_MMA_SYNC)])
def test_captured_step_replays_on_new_inputs(cfg, kw, variant):
    w0 = W.config(cfg, **kw)
    tree0, nxt0, attn0, acc0 = _reference(w0)
    vs = VerifyStep(w0)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):                      # warm-up outside the capture
        vs.target_next.copy_(torch.from_numpy(nxt0))
        vs.build(); vs.attn(variant); vs.accept()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        vs.build(); vs.attn(variant); vs.accept()
    rng = np.random.default_rng(3)
    for rep in range(4):
        if rep == 0:
            w, tree, nxt, attn, acc = w0, tree0, nxt0, attn0, acc0
        else:
            w = W.config(cfg, seed=100 + rep, **kw)
            assert w.S_cap <= w0.S_cap or cfg == "5"
            w.seq_len = np.minimum(w.seq_len - rng.integers(0, 900, size=w.B).astype(np.int32), w0.S_cap - w0.T_max).astype(np.int32)
            w.seq_len = np.maximum(w.seq_len, 1)
            w.S_cap = w0.S_cap
            # templates and gates are configuration: they stay as captured
            w.tmpl_parent, w.tmpl_rank, w.tmpl_offset = w0.tmpl_parent, w0.tmpl_rank, w0.tmpl_offset
            w.ckpt_depth, w.ckpt_keep, w.ckpt_log_tau = w0.ckpt_depth, w0.ckpt_keep, w0.ckpt_log_tau
            tree, nxt, attn, acc = _reference(w)
        _load(vs, w, nxt)
        vs.O.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        _check(vs, w, tree, attn, acc)
