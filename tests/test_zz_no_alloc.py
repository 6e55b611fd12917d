"""graft_tree_verify_attn_noalloc: the attention entry point for callers that cannot allocate.

Some users of this library have no way to obtain a workspace: all of their device memory was
handed to a fixed pool when the process started, or they sit in a latency-critical section where
an allocation (which may stall the whole device) is off limits.  For them the library carries a
static 40 MiB scratch array on every GPU.  This test drives that entry point through the C ABI and
checks it against the regular, workspace-based call on the same inputs: two calls in a row on
different shapes, so that whatever the first call left in the shared array cannot leak into the
second.  It is collected last on purpose; it depends on no other test.
"""
import numpy as np
import pytest
import torch

from paper_2605_20104_b200 import workloads as W

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 2e-2, 2e-3      # the attention tolerance of the parity tests


def make_case(seed, parents, Hq, Hkv, d, L, T_max):
    import oracle
    from paper_2605_20104_b200.step import VerifyStep
    w = W.custom(parents, Hq=Hq, Hkv=Hkv, d=d, L=L, T_max=T_max, seed=seed)
    tree = oracle.build_tree(w)
    W.make_qkv(w, tree["tree_size"], poison=True)
    vs = VerifyStep(w)
    vs.build()
    return w, vs


def run_both(G, w, vs):
    """Reference: the existing entry point with its caller-allocated workspace.  Under test: the
    no-allocation entry point on the same device buffers, writing to separate outputs."""
    vs.attn()
    torch.cuda.synchronize()
    O_ref, LSE_ref = vs.O.clone(), vs.LSE.clone()
    O = torch.full_like(vs.O, float("nan"))
    LSE = torch.full_like(vs.LSE, float("nan"))
    flags = torch.full((1,), -1, dtype=torch.int32, device=O.device)
    G.graft_tree_verify_attn_noalloc(Q=vs.Q, Kc=vs.Kc, Vc=vs.Vc, O=O, seq_len=vs.seq_len, tree_size=vs.tree_size,
                                     tree_anc=vs.tree_anc, scale=w.scale, LSE=LSE, device_flags_out=flags)
    torch.cuda.synchronize()
    assert flags.item() == 0
    err = (O.double() - O_ref.double()).abs()
    assert torch.isfinite(O).all()
    assert err.max().item() <= MAX_ABS and err.mean().item() <= MEAN_ABS
    fin = torch.isfinite(LSE_ref)
    assert (torch.isfinite(LSE) == fin).all()
    assert (LSE[fin] - LSE_ref[fin]).abs().max().item() <= 2e-3


def test_noalloc_matches_workspace_call_twice_in_a_row():
    from paper_2605_20104_b200 import binding as G
    assert G.graft_noalloc_scratch_bytes() == 40 << 20
    rng = np.random.default_rng(7)
    # first call: long context, split over many CTAs, so the scratch array fills with partials
    w1, vs1 = make_case(1, [W.random_tree_parents(rng, 48), W.random_tree_parents(rng, 20)], 10, 2, 128, [9000, 700], 64)
    run_both(G, w1, vs1)
    # second call: another shape and another kernel family (d = 64) over the same, now dirty, array
    w2, vs2 = make_case(2, [W.random_tree_parents(rng, 8)], 4, 1, 64, [1500], 8)
    run_both(G, w2, vs2)
    # and the first shape again
    run_both(G, w1, vs1)


def test_noalloc_rejects_shapes_beyond_its_scratch():
    from paper_2605_20104_b200 import binding as G
    rng = np.random.default_rng(8)
    # d = 64 runs on the register-tile kernel only; 64 sequences x 8 KV heads x 256 rows need more
    # partial slots than the 40 MiB array holds
    w, vs = make_case(3, [W.random_tree_parents(rng, 64)] * 64, 32, 8, 64, [64] * 64, 64)
    O = torch.zeros_like(vs.O)
    with pytest.raises(G.GraftError) as e:
        G.graft_tree_verify_attn_noalloc(Q=vs.Q, Kc=vs.Kc, Vc=vs.Vc, O=O, seq_len=vs.seq_len, tree_size=vs.tree_size,
                                         tree_anc=vs.tree_anc, scale=w.scale)
    assert e.value.code == G.ERR_SCRATCH_LIMIT
    assert "scratch" in str(e.value)
    assert (O == 0).all()                      # nothing ran
