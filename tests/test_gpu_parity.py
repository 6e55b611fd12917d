"""Parity of the CUDA path (through the C ABI) against the CPU oracle, on a B200.

Integer outputs (tree arrays, accepted paths, compacted caches) must match bit for bit.
Attention outputs: max |err| <= 2e-2 and mean |err| <= 2e-3 against the fp64 oracle on bf16 inputs
(the stated target of the benchmark); LSE within 2e-3.
"""
import numpy as np
import pytest
import torch

from paper_2605_20104_b200 import workloads as W

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 2e-2, 2e-3


@pytest.fixture(scope="module")
def G():
    from paper_2605_20104_b200 import binding
    return binding


@pytest.fixture(scope="module")
def Step():
    from paper_2605_20104_b200.step import VerifyStep
    return VerifyStep


VARIANTS = ["mma", "auto", "one", "pair", "l2pair"]      # the last three: one of the tcgen05 kernels, forced


def variant_id(G, name, w=None):
    if name in ("one", "pair", "l2pair") and w is not None and w.d != 128:
        pytest.skip("the tcgen05 kernels take d = 128 only")
    return {"mma": G.ATTN_MMA_SYNC, "auto": G.ATTN_AUTO, "tc": G.ATTN_TCGEN05, "one": G.ATTN_TCGEN05_1SM,
            "pair": G.ATTN_TCGEN05_2SM, "l2pair": G.ATTN_TCGEN05_L2PAIR}[name]


def check_tree(vs, tree):
    got = vs.tree_host()
    for k in ("tree_size", "tree_token", "tree_parent", "tree_pos", "tree_src", "tree_anc"):
        assert (got[k] == tree[k]).all(), k
    assert vs.ctx.device_status() == tree["flags"]


def check_attn(orc, w, vs, tree, rows=None):
    out = orc.tree_attn(W.bf16_bits(w.Q), W.bf16_bits(w.Kc), W.bf16_bits(w.Vc), w.seq_len, tree["tree_size"],
                        tree["tree_anc"], w.scale, rows=rows)
    O = vs.O.cpu().to(torch.float64).numpy()
    LSE = vs.LSE.cpu().to(torch.float64).numpy()
    assert np.isfinite(O).all()
    if rows is None:
        valid = np.arange(w.T_max)[None, :] < tree["tree_size"][:, None]           # [B, T_max]
        err = np.abs(O - out["O"])[valid]
        assert (O[~valid] == 0).all()                                                # padding rows are zero
        lse_valid = np.broadcast_to(valid[:, None, :], LSE.shape)
        assert np.isneginf(LSE[~lse_valid]).all()
        with np.errstate(invalid="ignore"):
            lse_err = np.abs(LSE - out["LSE"])[lse_valid]
    else:
        err = np.stack([np.abs(O[b, t, h] - out["O"][b, t, h]) for b, t, h in rows])
        lse_err = np.array([abs(LSE[b, h, t] - out["LSE"][b, h, t]) for b, t, h in rows])
    assert err.max() <= MAX_ABS, err.max()
    assert err.mean() <= MEAN_ABS, err.mean()
    assert lse_err.max() <= 2e-3, lse_err.max()
    return err.max(), err.mean()


def check_accept_and_compact(orc, w, vs, tree):
    nxt = W.draw_target_next(tree["tree_token"], tree["tree_parent"], tree["tree_size"], tree["tree_src"], w.V,
                             w.p_draft, w.p_graft, w.seed)
    vs.target_next.copy_(torch.from_numpy(nxt))
    vs.accept()
    want = orc.accept(tree["tree_token"], tree["tree_parent"], tree["tree_size"], nxt)
    got = vs.accept_host()
    for k in ("n_acc", "path", "best_node", "bonus"):
        assert (got[k] == want[k]).all(), k
    K_old, V_old = W.bf16_bits(w.Kc), W.bf16_bits(w.Vc)
    ref = orc.compact_kv(K_old, V_old, w.seq_len, want["n_acc"], want["path"])
    vs.compact()
    Kd = vs.Kc.cpu().view(torch.int16).numpy().view(np.uint16)
    Vd = vs.Vc.cpu().view(torch.int16).numpy().view(np.uint16)
    assert (Kd == ref["K"]).all() and (Vd == ref["V"]).all()
    assert (vs.new_seq_len.cpu().numpy() == ref["new_seq_len"]).all()
    assert vs.ctx.device_status() == 0
    return want


def full_case(orc, G, Step, w, variant, rows=None, poison=True):
    tree = orc.build_tree(w)
    W.make_qkv(w, tree["tree_size"], poison=poison)
    vs = Step(w)
    vs.build()
    check_tree(vs, tree)
    vs.attn(variant_id(G, variant, w))
    torch.cuda.synchronize()
    e = check_attn(orc, w, vs, tree, rows)
    assert vs.ctx.device_status() == 0
    acc = check_accept_and_compact(orc, w, vs, tree)
    return e, acc


# ---------------------------------------------------------------------------------------------
# small shapes, compared element by element
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("variant", VARIANTS)
def test_cfg1_tiny(orc, G, Step, variant):
    full_case(orc, G, Step, W.config("1"), variant)


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("cfg,B,L", [("2", 2, 300), ("3", 3, 517), ("3p", None, 200), ("4", 2, 1000), ("5", 5, 1500)])
def test_configs_reduced_context(orc, G, Step, cfg, B, L, variant):
    """The five shapes with a shorter cache: several key tiles and a ragged tail, every element."""
    full_case(orc, G, Step, W.config(cfg, B=B, L=L), variant)


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("Hq,Hkv,d", [(4, 1, 64), (8, 8, 128), (10, 2, 128), (16, 1, 128), (2, 2, 64)])
@pytest.mark.parametrize("shape", ["chain", "star", "single", "random"])
def test_tree_shapes(orc, G, Step, Hq, Hkv, d, shape, variant):
    rng = np.random.default_rng(Hq * 1000 + Hkv * 100 + d + len(shape))
    T = 23
    parents = {"chain": W.chain_parents(T), "star": W.star_parents(T), "single": np.array([-1], np.int32),
               "random": W.random_tree_parents(rng, T)}[shape]
    w = W.custom([parents, W.random_tree_parents(rng, 7)], Hq=Hq, Hkv=Hkv, d=d, L=[129, 64], T_max=32, seed=11)
    full_case(orc, G, Step, w, variant)


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("L", [0, 1, 63, 64, 65, 127, 128, 191])
def test_tile_boundaries(orc, G, Step, L, variant):
    """Cached lengths around the key-tile size, including an empty cache (tree keys only)."""
    rng = np.random.default_rng(L)
    w = W.custom([W.random_tree_parents(rng, 64), W.random_tree_parents(rng, 3)], Hq=8, Hkv=2, d=128, L=[L, L + 5],
                 T_max=64, seed=L)
    full_case(orc, G, Step, w, variant)


@pytest.mark.parametrize("variant", VARIANTS)
def test_max_tree_and_many_row_blocks(orc, G, Step, variant):
    """T = 64 with G = 16: 1024 rows per KV head, i.e. the largest row count the ABI admits."""
    rng = np.random.default_rng(5)
    w = W.custom([W.random_tree_parents(rng, 64), W.random_tree_parents(rng, 17)], Hq=32, Hkv=2, d=128, L=[700, 300],
                 T_max=64, seed=5)
    full_case(orc, G, Step, w, variant)


@pytest.mark.parametrize("variant", VARIANTS)
def test_strided_cache_and_no_lse(orc, G, Step, variant):
    """Token-major cache [B, S, H_kv, d] viewed as [B, H_kv, S, d]; LSE pointer omitted."""
    rng = np.random.default_rng(6)
    w = W.custom([W.random_tree_parents(rng, 20)], Hq=8, Hkv=4, d=128, L=[333], T_max=32, seed=6)
    tree = orc.build_tree(w)
    W.make_qkv(w, tree["tree_size"], poison=True)
    vs = Step(w)
    vs.build()
    Kt = vs.Kc.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)      # same values, token-major storage
    Vt = vs.Vc.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    vs.LSE.fill_(7.0)
    G.graft_tree_verify_attn(vs.ctx, Q=vs.Q, Kc=Kt, Vc=Vt, O=vs.O, seq_len=vs.seq_len, tree_size=vs.tree_size,
                             tree_anc=vs.tree_anc, scale=w.scale, LSE=None, variant=variant_id(G, variant, w))
    torch.cuda.synchronize()
    assert (vs.LSE == 7.0).all()
    out = orc.tree_attn(W.bf16_bits(w.Q), W.bf16_bits(w.Kc), W.bf16_bits(w.Vc), w.seq_len, tree["tree_size"],
                        tree["tree_anc"], w.scale)
    err = np.abs(vs.O.cpu().to(torch.float64).numpy() - out["O"])[0, :20]
    assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS


@pytest.mark.parametrize("variant", VARIANTS)
def test_mask_locality_on_device(orc, G, Step, variant):
    """Changing K/V of a tree node moves exactly the rows that have it as an ancestor-or-self
    (same split schedule, so untouched rows must be bit-identical)."""
    rng = np.random.default_rng(9)
    par = W.random_tree_parents(rng, 30)
    w = W.custom([par], Hq=4, Hkv=2, d=128, L=[200], T_max=32, seed=9)
    tree = orc.build_tree(w)
    W.make_qkv(w, tree["tree_size"], poison=True)
    vs = Step(w)
    vs.build()
    vs.attn(variant_id(G, variant, w))
    base = vs.O.clone()
    u = 11
    vs.Vc[0, :, 200 + u] += 2.0
    vs.Kc[0, :, 200 + u] *= -1.0
    vs.attn(variant_id(G, variant, w))
    changed = (vs.O != base).flatten(2).any(-1)[0].cpu().numpy()          # [T_max]
    anc = tree["tree_anc"][0]
    for t in range(30):
        assert changed[t] == bool((int(anc[t]) >> u) & 1), t


def test_malformed_inputs_match_oracle_flags(orc, G, Step):
    rng = np.random.default_rng(1)
    w = W.custom([W.random_tree_parents(rng, 10)] * 4, Hq=2, Hkv=1, d=64, L=[4, 4, 4, 4], V=50, seed=1)
    w.draft_parent = w.draft_parent.copy()
    w.draft_token = w.draft_token.copy()
    w.n_draft = w.n_draft.copy()
    w.draft_score = w.draft_score.copy()
    w.draft_parent[0, 4] = 7
    w.draft_token[1, 3] = 50
    w.n_draft[2] = 11
    w.draft_score[3, 5] = np.nan
    w.mode, w.keep_count = W.MODE_TOPK, np.array([10, 10, 10, 6], np.int32)
    w.tmpl_parent, w.tmpl_rank = W.chains_template([3])
    tree = orc.build_tree(w)
    assert tree["flags"] != 0
    vs = Step(w)
    vs.build()
    check_tree(vs, tree)


@pytest.mark.parametrize("seed", range(6))
def test_random_builds(orc, G, Step, seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(2, 48))
    w = W.custom([W.random_tree_parents(rng, int(rng.integers(2, n + 1))) for _ in range(9)], Hq=2, Hkv=1, d=64,
                 L=[5] * 9, V=50, T_max=48, seed=seed)
    w.mode = [W.MODE_TOPK, W.MODE_NODE, W.MODE_NONE][seed % 3]
    w.K_max = int(rng.integers(1, 49))
    w.keep_count = rng.integers(1, n + 3, size=9).astype(np.int32)
    w.gate_depth, w.node_threshold = int(rng.integers(0, 4)), float(np.float32(-1.5))
    w.tmpl_parent, w.tmpl_rank = W.paper_template("d5", 8)
    if seed % 2:
        w.draft_score = rng.normal(size=w.draft_score.shape).astype(np.float32)   # orphans possible
    tree = orc.build_tree(w)
    vs = Step(w)
    vs.build()
    check_tree(vs, tree)


@pytest.mark.parametrize("paths", [[[0, 2, 3]], [[0, 63]], [[0, 1, 3, 4, 5, 9]], [[0]], [[0, 5, 6], [0, 1, 7, 8, 20]]])
def test_compaction_overlap_cases(orc, G, Step, paths):
    """In-place moves whose destination is another entry's source."""
    B = len(paths)
    rng = np.random.default_rng(0)
    w = W.custom([W.chain_parents(64)] * B, Hq=4, Hkv=2, d=128, L=[3, 11][:B], T_max=64, seed=0)
    W.make_qkv(w)
    vs = Step(w, n_layers=3)
    path = np.full((B, 64), -1, np.int32)
    n_acc = np.zeros(B, np.int32)
    for b, p in enumerate(paths):
        path[b, :len(p)] = p
        n_acc[b] = len(p)
    vs.path.copy_(torch.from_numpy(path))
    vs.n_acc.copy_(torch.from_numpy(n_acc))
    K_old = vs.Kc.cpu().view(torch.int16).numpy().view(np.uint16)
    V_old = vs.Vc.cpu().view(torch.int16).numpy().view(np.uint16)
    ref = orc.compact_kv(K_old, V_old, w.seq_len, n_acc, path)
    vs.compact()
    assert (vs.Kc.cpu().view(torch.int16).numpy().view(np.uint16) == ref["K"]).all()
    assert (vs.Vc.cpu().view(torch.int16).numpy().view(np.uint16) == ref["V"]).all()
    assert (vs.new_seq_len.cpu().numpy() == ref["new_seq_len"]).all()


def test_compaction_rejects_bad_path(orc, G, Step):
    w = W.custom([W.chain_parents(8)], Hq=2, Hkv=1, d=64, L=[5], T_max=8, seed=0)
    W.make_qkv(w)
    vs = Step(w)
    before = vs.Kc.clone()
    vs.path.copy_(torch.tensor([[0, 9, -1, -1, -1, -1, -1, -1]], dtype=torch.int32))
    vs.n_acc.fill_(2)
    vs.compact()
    assert vs.ctx.device_status() == G.FLAG_BAD_PATH
    assert (vs.Kc == before).all() and vs.new_seq_len.item() == 5


def test_host_side_argument_errors(G, Step):
    w = W.config("1")
    W.make_qkv(w)
    vs = Step(w)
    vs.build()
    kw = dict(Q=vs.Q, Kc=vs.Kc, Vc=vs.Vc, O=vs.O, seq_len=vs.seq_len, tree_size=vs.tree_size, tree_anc=vs.tree_anc)
    with pytest.raises(G.GraftError) as e:
        G.graft_tree_verify_attn(vs.ctx, scale=-1.0, **kw)
    assert e.value.code == G.ERR_INVALID_ARG
    with pytest.raises(G.GraftError) as e:
        G.graft_tree_verify_attn(vs.ctx, scale=w.scale, variant=17, **kw)
    assert e.value.code == G.ERR_INVALID_ARG
    small = G.Context(1, 4, 1, 64, 8, workspace=torch.empty(1024, dtype=torch.uint8, device="cuda"))
    with pytest.raises(G.GraftError) as e:
        G.graft_tree_verify_attn(small, scale=w.scale, **kw)
    assert e.value.code == G.ERR_WORKSPACE_TOO_SMALL
    assert G.graft_workspace_bytes(0, 1, 5, 2, 128, 8) == 0          # H_q not a multiple of H_kv
    assert G.graft_workspace_bytes(0, 1, 4, 2, 96, 8) == 0           # head dim
    assert G.graft_workspace_bytes(0, 1, 4, 2, 128, 65) == 0         # tree larger than the 64-bit mask


# ---------------------------------------------------------------------------------------------
# the five configurations at full size, in the launch configuration the benchmark times;
# integer outputs compared in full, attention on sampled rows the oracle computes one by one
# ---------------------------------------------------------------------------------------------
def sample_rows(rng, tree_size, Hq, n):
    rows = []
    B = len(tree_size)
    for _ in range(n):
        b = int(rng.integers(0, B))
        rows.append((b, int(rng.integers(0, tree_size[b])), int(rng.integers(0, Hq))))
    # always include the root and the last node of every sequence
    for b in range(B):
        rows += [(b, 0, 0), (b, int(tree_size[b]) - 1, Hq - 1)]
    return np.array(rows, np.int32)


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("cfg,B,n_rows", [("2", None, 400), ("3", None, 300), ("4", 1, 96), ("4", 4, 64), ("5", None, 300)])
def test_full_size_configs(orc, G, Step, cfg, B, n_rows, variant):
    w = W.config(cfg, B=B)
    tree = orc.build_tree(w)
    rows = sample_rows(np.random.default_rng(int(cfg) + 100), tree["tree_size"], w.Hq, n_rows)
    full_case(orc, G, Step, w, variant, rows=rows)


# ---------------------------------------------------------------------------------------------
# schedule edge cases of the persistent attention kernel
# ---------------------------------------------------------------------------------------------
def test_many_short_sequences(orc, G, Step):
    """Far more (sequence, KV head) items than SMs, one or two key tiles each: every CTA walks through
    many whole items, in more than one planning round."""
    rng = np.random.default_rng(21)
    B = 300
    parents = [W.random_tree_parents(rng, int(rng.integers(1, 9))) for _ in range(B)]
    L = rng.integers(0, 200, size=B).tolist()
    w = W.custom(parents, Hq=8, Hkv=8, d=128, L=L, T_max=8, seed=21)
    full_case(orc, G, Step, w, "auto")


@pytest.mark.parametrize("L0", [9000, 20000])
@pytest.mark.parametrize("variant", ["mma", "one", "auto", "pair", "l2pair"])
def test_one_long_sequence_among_short_ones(orc, G, Step, variant, L0):
    """Enough (sequence, KV head) items that the kernels merge the parts of an item themselves, and one item that is
    cut across most of the workers: its last part merges dozens of partials.  With the longer context the merge
    kernel runs instead, half a warp per row, and walks an item of more than sixteen parts in rounds."""
    rng = np.random.default_rng(27)
    B = 12
    parents = [W.random_tree_parents(rng, int(rng.integers(8, 33))) for _ in range(B)]
    L = [L0] + [int(x) for x in rng.integers(50, 400, size=B - 1)]
    w = W.custom(parents, Hq=16, Hkv=4, d=128, L=L, T_max=32, seed=27)
    rows = sample_rows(np.random.default_rng(127), orc.build_tree(w)["tree_size"], w.Hq, 400)
    full_case(orc, G, Step, w, variant, rows=rows)


@pytest.mark.parametrize("variant", ["auto", "pair", "l2pair"])
def test_repeated_calls_on_one_context(orc, G, Step, variant):
    """The kernels that merge in place keep arrival counters and slot descriptors in the workspace across calls: the
    same call three times, then a different batch on the same context, all exact and the repeats bit-identical."""
    rng = np.random.default_rng(29)
    parents = [W.random_tree_parents(rng, 24) for _ in range(8)]
    w = W.custom(parents, Hq=32, Hkv=8, d=128, L=[700, 650, 900, 300, 1200, 800, 750, 1000], T_max=32, seed=29)
    tree = orc.build_tree(w)
    W.make_qkv(w, tree["tree_size"], poison=True)
    vs = Step(w)
    vs.build()
    outs = []
    for _ in range(3):
        vs.O.fill_(float("nan"))
        vs.attn(variant_id(G, variant, w))
        torch.cuda.synchronize()
        check_attn(orc, w, vs, tree)
        outs.append(vs.O.cpu().view(torch.int16).numpy().copy())
    assert (outs[0] == outs[1]).all() and (outs[0] == outs[2]).all()
    # other (shorter: the cache is poisoned past the old ends) lengths, same buffers
    vs.seq_len[:] = torch.tensor([5, 600, 64, 300, 127, 128, 129, 1], dtype=torch.int32)
    w.seq_len = vs.seq_len.cpu().numpy().copy()
    vs.attn(variant_id(G, variant, w))
    torch.cuda.synchronize()
    check_attn(orc, w, vs, tree)
    assert vs.ctx.device_status() == 0


def test_one_and_two_block_items_mixed(orc, G, Step):
    """G = 16 with tree sizes whose last row block has at most / more than 128 rows, ragged lengths:
    items of different cost per tile on the cut axis, several row blocks per KV head."""
    rng = np.random.default_rng(22)
    sizes = [5, 8, 9, 16, 17, 24, 25, 40, 41, 64, 33, 3]
    parents = [W.random_tree_parents(rng, n) for n in sizes]
    L = rng.integers(100, 3000, size=len(sizes)).tolist()
    w = W.custom(parents, Hq=32, Hkv=2, d=128, L=L, T_max=64, seed=22)
    full_case(orc, G, Step, w, "auto")


def test_invalid_sequence_inside_a_batch(orc, G, Step):
    """A sequence whose tree_size is out of range is skipped (zero rows, BAD_SIZE flag); the others are exact."""
    rng = np.random.default_rng(23)
    w = W.custom([W.random_tree_parents(rng, 20) for _ in range(3)], Hq=8, Hkv=2, d=128, L=[500, 300, 900], T_max=32,
                 seed=23)
    tree = orc.build_tree(w)
    W.make_qkv(w, tree["tree_size"], poison=True)
    vs = Step(w)
    vs.build()
    vs.tree_size[1] = 33                                   # larger than T_max: invalid
    for variant in VARIANTS:
        vs.O.fill_(float("nan"))
        vs.attn(variant_id(G, variant, w))
        torch.cuda.synchronize()
        assert vs.ctx.device_status() == G.FLAG_BAD_SIZE
        O = vs.O.cpu().to(torch.float64).numpy()
        assert (O[1] == 0).all()
        out = orc.tree_attn(W.bf16_bits(w.Q), W.bf16_bits(w.Kc), W.bf16_bits(w.Vc), w.seq_len, tree["tree_size"],
                            tree["tree_anc"], w.scale)
        for b in (0, 2):
            err = np.abs(O[b, :20] - out["O"][b, :20])
            assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS
            assert (O[b, 20:] == 0).all()


@pytest.mark.parametrize("variant", ["auto", "l2pair", "one", "pair", "mma"])
@pytest.mark.parametrize("B,L0", [(1, 20000), (6, 3000)])
def test_chain_only_trees(orc, G, Step, variant, B, L0):
    """Chains of 16 nodes (the tail-block proposals): one 128-row block per KV head, the case in which every CTA of the
    row-block kernel walks tiles of its own; a single long sequence is cut across all of them, a batch merges in place."""
    rng = np.random.default_rng(B)
    parents = [W.chain_parents(int(n)) for n in ([16] if B == 1 else rng.integers(1, 17, size=B))]
    L = [L0] if B == 1 else [int(x) for x in rng.integers(100, L0, size=B)]
    w = W.custom(parents, Hq=40, Hkv=8, d=128, L=L, T_max=16, seed=40 + B)
    rows = sample_rows(np.random.default_rng(B), orc.build_tree(w)["tree_size"], w.Hq, 300)
    full_case(orc, G, Step, w, variant, rows=rows)


@pytest.mark.parametrize("Hq,Hkv,T", [(32, 8, 32), (40, 8, 48)])
def test_kernels_take_turns_on_one_workspace(orc, G, Step, Hq, Hkv, T):
    """All attention kernels share one workspace (slot descriptors, arrival counters, the call number): a dozen calls
    in a row, the kernel and the lengths changing from call to call, every one exact.  The first shape gives one
    128-row block per item (every CTA its own tiles in the row-block kernel), the second two."""
    rng = np.random.default_rng(Hq)
    B = 6
    parents = [W.random_tree_parents(rng, int(rng.integers(T // 2, T + 1))) for _ in range(B)]
    L0 = [2500, 1800, 900, 2200, 600, 1500]
    w = W.custom(parents, Hq=Hq, Hkv=Hkv, d=128, L=L0, T_max=T, seed=Hq)
    tree = orc.build_tree(w)
    W.make_qkv(w, tree["tree_size"], poison=True)
    vs = Step(w)
    vs.build()
    order = ["l2pair", "pair", "one", "auto", "mma", "pair", "l2pair", "l2pair", "one", "pair", "auto", "l2pair"]
    for n, variant in enumerate(order):
        # lengths only ever shrink: the cache is poisoned past the first call's ends
        w.seq_len = np.maximum(1, np.asarray(L0) - rng.integers(0, 500, size=B) * (n > 0)).astype(np.int32)
        vs.seq_len.copy_(torch.from_numpy(w.seq_len))
        vs.O.fill_(float("nan"))
        vs.attn(variant_id(G, variant, w))
        torch.cuda.synchronize()
        rows = sample_rows(np.random.default_rng(n), tree["tree_size"], w.Hq, 200)
        check_attn(orc, w, vs, tree, rows)
    assert vs.ctx.device_status() == 0
