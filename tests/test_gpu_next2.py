"""Retrieval envelope, tree assembly from the envelope and candidate-path indices on the GPU against
the oracle (bit exact), through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_20104_b200 import binding as G
from paper_2605_20104_b200 import workloads as W
from paper_2605_20104_b200.step import VerifyStep

pytestmark = pytest.mark.gpu

TREE_KEYS = ("tree_size", "tree_token", "tree_parent", "tree_pos", "tree_src", "tree_anc")


def _ctx(B=4):
    return G.Context(B, 8, 8, 128, 64)


def _envelope(ctx, roots, M, ep, er, stride=1):
    B = (len(roots) + stride - 1) // stride
    out = torch.full((B, len(ep)), -7, dtype=torch.int32, device="cuda")
    G.graft_retrieve_envelope(ctx, root_token=torch.from_numpy(roots).cuda(), root_stride=stride, M=torch.from_numpy(M).cuda(),
                              env_parent=torch.from_numpy(ep).cuda(), env_rank=torch.from_numpy(er).cuda(), env_token=out)
    torch.cuda.synchronize()
    return out.cpu().numpy()


@pytest.mark.parametrize("name", ["full", "d0", "d1", "d5"])
def test_envelope_paper_templates(name):
    rng = np.random.default_rng(11)
    V, k, B = 151936, 8, 64
    M = rng.integers(-1, V, size=(V, k)).astype(np.int32)
    M[rng.random(V) < 0.05] = -1                     # some tokens have no successors yet
    roots = rng.integers(0, V, size=B).astype(np.int32)
    roots[3] = -1
    ep, er = W.paper_template(name, k)
    ctx = _ctx()
    got = _envelope(ctx, roots, M, ep, er)
    ref = oracle.retrieve_envelope(roots, M, ep, er)
    assert (got == ref["env_token"]).all()
    assert ctx.device_status() == ref["flags"] == 0


def test_envelope_large_ragged_template_and_flags():
    rng = np.random.default_rng(3)
    V, k = 5000, 16
    M = rng.integers(0, V, size=(V, k)).astype(np.int32)
    M[7, 3] = V + 5                                  # an entry outside the vocabulary
    n = 1000                                         # several passes of the CTA, deep and wide parts
    ep = np.asarray([-1] + [int(rng.integers(-1, u)) for u in range(1, n)], np.int32)
    ep[500:560] = np.arange(499, 559)                # a chain of 60 levels
    er = rng.integers(0, k, size=n).astype(np.int32)
    er[10] = k                                       # bad rank
    ep[20] = 25                                      # parent after the node
    roots = np.asarray([7, 0, V, 4999, -1], np.int32)
    ctx = _ctx()
    got = _envelope(ctx, roots, M, ep, er)
    ref = oracle.retrieve_envelope(roots, M, ep, er)
    assert (got == ref["env_token"]).all()
    assert ctx.device_status() == ref["flags"]
    assert ref["flags"] & oracle.FLAG_BAD_TEMPLATE and ref["flags"] & oracle.FLAG_BAD_TOKEN


def test_envelope_arguments():
    ctx = _ctx()
    z = torch.zeros(8, dtype=torch.int32, device="cuda")
    M = torch.zeros(16, 4, dtype=torch.int32, device="cuda")
    big = torch.zeros(1, 1025, dtype=torch.int32, device="cuda")
    with pytest.raises(G.GraftError):
        G.graft_retrieve_envelope(ctx, root_token=z, M=M, env_parent=torch.zeros(1025, dtype=torch.int32, device="cuda"),
                                  env_rank=torch.zeros(1025, dtype=torch.int32, device="cuda"), env_token=big)


@pytest.mark.parametrize("cfg", ["1", "2", "3", "4", "5"])
@pytest.mark.parametrize("side_stream", [False, True])
def test_build_from_envelope_equals_oracle_assembly(cfg, side_stream):
    w = W.config(cfg) if cfg != "4" else W.config("4", L=512)
    ref = oracle.build_tree(w)
    vs = VerifyStep(w, upload_qkv=False)
    vs.retrieve_envelope(torch.cuda.Stream() if side_stream else None)
    vs.build(from_envelope=True)
    torch.cuda.synchronize()
    got = vs.tree_host()
    for key in TREE_KEYS:
        assert (got[key] == ref[key]).all(), key
    ep, er, _ = W.workload_envelope(w)
    env_flags = 0
    if len(ep):
        env = oracle.retrieve_envelope(w.draft_token, w.M, ep, er, root_stride=w.N_max)
        assert (vs.env_token.cpu().numpy() == env["env_token"]).all()
        env_flags = env["flags"]      # the envelope looks at every template node, the assembly only at the ones it grafts
    assert vs.ctx.device_status() == ref["flags"] | env_flags
    # and the plain call still gives the same tree
    vs.build()
    torch.cuda.synchronize()
    got = vs.tree_host()
    for key in TREE_KEYS:
        assert (got[key] == ref[key]).all(), key


def test_build_from_envelope_bad_index():
    w = W.config("5")
    vs = VerifyStep(w, upload_qkv=False)
    vs.retrieve_envelope()
    vs.tmpl_env[2] = vs.env_token.shape[1]            # outside the envelope
    vs.build(from_envelope=True)
    torch.cuda.synchronize()
    assert vs.ctx.device_status() & G.FLAG_BAD_TEMPLATE


@pytest.mark.parametrize("cfg", ["1", "2", "3", "5"])
def test_path_indices_of_assembled_trees(cfg):
    w = W.config(cfg)
    ref_tree = oracle.build_tree(w)
    vs = VerifyStep(w, upload_qkv=False)
    vs.build()
    for D in (w.T_max, 12, 4):
        vs.path_indices(D)
        torch.cuda.synchronize()
        ref = oracle.path_indices(ref_tree["tree_parent"], ref_tree["tree_size"], D)
        assert (vs.path_index.cpu().numpy() == ref["path_index"]).all(), D
        assert (vs.n_paths.cpu().numpy() == ref["n_paths"]).all()
        assert vs.ctx.device_status() == ref["flags"]


@pytest.mark.parametrize("seed", range(4))
def test_path_indices_random_trees(seed):
    rng = np.random.default_rng(seed)
    B, T_max, D = 37, 64, 64
    parent = np.full((B, T_max), -1, np.int32)
    size = rng.integers(0, T_max + 1, size=B).astype(np.int32)
    size[:3] = [0, 1, T_max]
    for b in range(B):
        if size[b]:
            parent[b, :size[b]] = W.random_tree_parents(rng, int(size[b]))[:size[b]]
    parent[5, :size[5]] = W.chain_parents(int(size[5]))[:size[5]] if size[5] else []
    parent[6, :size[6]] = W.star_parents(int(size[6]))[:size[6]] if size[6] else []
    ctx = _ctx()
    out = torch.full((B, T_max, D), -9, dtype=torch.int32, device="cuda")
    n = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    G.graft_path_indices(ctx, tree_parent=torch.from_numpy(parent).cuda(), tree_size=torch.from_numpy(size).cuda(),
                         path_index=out, n_paths=n)
    torch.cuda.synchronize()
    ref = oracle.path_indices(parent, size, D)
    assert (out.cpu().numpy() == ref["path_index"]).all()
    assert (n.cpu().numpy() == ref["n_paths"]).all()
    assert ctx.device_status() == 0


def test_path_indices_bad_size_flag():
    ctx = _ctx()
    parent = torch.from_numpy(W.chain_parents(8)[None, :].copy()).cuda()
    out = torch.empty(1, 8, 8, dtype=torch.int32, device="cuda")
    n = torch.empty(1, dtype=torch.int32, device="cuda")
    G.graft_path_indices(ctx, tree_parent=parent, tree_size=torch.tensor([9], dtype=torch.int32, device="cuda"), path_index=out, n_paths=n)
    torch.cuda.synchronize()
    assert ctx.device_status() == G.FLAG_BAD_SIZE and int(n[0]) == 0 and (out == -1).all()


@pytest.mark.parametrize("block,V", [(16, 151936), (8, 500)])
def test_tail_grafting_block_drafter(block, V):
    """Keep the reliable prefix of a drafted chain, continue it with the matrix's rank-0 chain (tail grafting)."""
    w = W.tail_block(B=9, L=700, block=block, V=V)
    ref = oracle.build_tree(w)
    vs = VerifyStep(w, upload_qkv=False)
    vs.build()
    torch.cuda.synchronize()
    got = vs.tree_host()
    for key in TREE_KEYS:
        assert (got[key] == ref[key]).all(), key
    assert vs.ctx.device_status() == ref["flags"]
    assert (ref["tree_src"] < 0).any() and (got["tree_parent"][:, 1:block] == np.arange(block - 1)).all()
    with pytest.raises(G.GraftError):            # the envelope is root-centred: not together with tail grafting
        vs.retrieve_envelope()
        vs.build(from_envelope=True)
