"""Paged K/V caches: the same attention and compaction results as with contiguous caches (the oracle's layout),
with the cache scattered over a pool through a random block table and every unused slot of the pool poisoned."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_20104_b200 import binding as G
from paper_2605_20104_b200 import workloads as W
from paper_2605_20104_b200.step import VerifyStep

pytestmark = pytest.mark.gpu


def make_pool(w, tree_size, page_size, rng, extra_blocks=5):
    """Scatter w.Kc / w.Vc [B, Hkv, S_cap, d] into pools [n_blocks, Hkv, page_size, d]; slots no sequence owns, and
    slots past a sequence's keys, hold NaN bit patterns."""
    B, Hkv, S_cap, d = w.Kc.shape
    per_seq = (S_cap + page_size - 1) // page_size
    n_blocks = B * per_seq + extra_blocks
    table = rng.permutation(n_blocks)[:B * per_seq].reshape(B, per_seq).astype(np.int32)
    nan = torch.tensor(float("nan"), dtype=torch.bfloat16)
    Kp = torch.full((n_blocks, Hkv, page_size, d), float("nan"), dtype=torch.bfloat16)
    Vp = torch.full((n_blocks, Hkv, page_size, d), float("nan"), dtype=torch.bfloat16)
    for b in range(B):
        end = int(w.seq_len[b]) + int(tree_size[b])
        for j in range(per_seq):
            lo, hi = j * page_size, min((j + 1) * page_size, end)
            if hi > lo:
                Kp[table[b, j], :, :hi - lo] = w.Kc[b, :, lo:hi]
                Vp[table[b, j], :, :hi - lo] = w.Vc[b, :, lo:hi]
    return Kp, Vp, table


def gather_pool(Kp, table, S_cap):
    B, per_seq = table.shape
    page = Kp.shape[2]
    out = torch.stack([torch.cat([Kp[table[b, j]] for j in range(per_seq)], dim=1)[:, :S_cap] for b in range(B)])
    return out


@pytest.mark.parametrize("cfg,kw,page", [("1", dict(), 128), ("5", dict(), 256), ("4", dict(B=2, L=3000), 128), ("2", dict(), 512),
                                         ("4", dict(B=1, L=20000), 1024), ("3", dict(B=8, L=1111), 128), ("tail", dict(B=3, L=5000), 256)])
def test_paged_attention_and_compaction(cfg, kw, page):
    w = W.config(cfg, **kw)
    tree = oracle.build_tree(w)
    W.make_qkv(w, tree["tree_size"], poison=True)
    rng = np.random.default_rng(page)
    Kp, Vp, table = make_pool(w, tree["tree_size"], page, rng)
    nxt = W.draw_target_next(tree["tree_token"], tree["tree_parent"], tree["tree_size"], tree["tree_src"], w.V,
                             w.p_draft, w.p_graft, w.seed)
    ref = oracle.tree_attn(W.bf16_bits(w.Q), W.bf16_bits(w.Kc), W.bf16_bits(w.Vc), w.seq_len, tree["tree_size"],
                           tree["tree_anc"], w.scale)
    acc = oracle.accept(tree["tree_token"], tree["tree_parent"], tree["tree_size"], nxt)
    kv = oracle.compact_kv(W.bf16_bits(w.Kc), W.bf16_bits(w.Vc), w.seq_len, acc["n_acc"], acc["path"])

    vs = VerifyStep(w, upload_qkv=False)
    vs.Q = w.Q.cuda()
    vs.build()
    Kd, Vd, td = Kp.cuda(), Vp.cuda(), torch.from_numpy(table).cuda()
    tc = (G.ATTN_TCGEN05_2SM, G.ATTN_TCGEN05_L2PAIR) if w.d == 128 else ()
    for variant in (G.ATTN_AUTO, G.ATTN_MMA_SYNC) + tc:
        vs.O.fill_(float("nan"))
        G.graft_tree_verify_attn(vs.ctx, Q=vs.Q, Kc=Kd, Vc=Vd, O=vs.O, seq_len=vs.seq_len, tree_size=vs.tree_size,
                                 tree_anc=vs.tree_anc, scale=w.scale, LSE=vs.LSE, variant=variant, block_table=td, S_cap=w.S_cap)
        torch.cuda.synchronize()
        O = vs.O.cpu().double().numpy()
        for b in range(w.B):
            n = int(tree["tree_size"][b])
            err = np.abs(O[b, :n] - ref["O"][b, :n])
            assert err.max() <= 2e-2 and err.mean() <= 2e-3, (b, err.max(), err.mean())
            assert (O[b, n:] == 0).all()
    vs.target_next.copy_(torch.from_numpy(nxt))
    vs.accept()
    G.graft_compact_kv(vs.ctx, Kc=Kd, Vc=Vd, seq_len=vs.seq_len, n_acc=vs.n_acc, path=vs.path, new_seq_len=vs.new_seq_len,
                       block_table=td, S_cap=w.S_cap)
    torch.cuda.synchronize()
    assert (vs.new_seq_len.cpu().numpy() == kv["new_seq_len"]).all()
    Kg = gather_pool(Kd.cpu(), table, w.S_cap).view(torch.int16).numpy().view(np.uint16)
    Vg = gather_pool(Vd.cpu(), table, w.S_cap).view(torch.int16).numpy().view(np.uint16)
    for b in range(w.B):
        end = int(w.seq_len[b]) + int(tree["tree_size"][b])       # everything the sequence owns, moved rows included
        assert (Kg[b, :, :end] == kv["K"][b, :, :end]).all() and (Vg[b, :, :end] == kv["V"][b, :, :end]).all()
    assert vs.ctx.device_status() == 0


def test_paged_table_entry_out_of_range_is_flagged():
    w = W.config("1")
    tree = oracle.build_tree(w)
    W.make_qkv(w, tree["tree_size"])
    Kp, Vp, table = make_pool(w, tree["tree_size"], 128, np.random.default_rng(0))
    table[0, 0] = Kp.shape[0]                       # one past the pool
    vs = VerifyStep(w, upload_qkv=False)
    vs.Q = w.Q.cuda()
    vs.build()
    G.graft_tree_verify_attn(vs.ctx, Q=vs.Q, Kc=Kp.cuda(), Vc=Vp.cuda(), O=vs.O, seq_len=vs.seq_len, tree_size=vs.tree_size,
                             tree_anc=vs.tree_anc, scale=w.scale, block_table=torch.from_numpy(table).cuda(), S_cap=w.S_cap)
    torch.cuda.synchronize()
    assert vs.ctx.device_status() == G.FLAG_BAD_SIZE
    with pytest.raises(G.GraftError):               # pages must be multiples of 128 keys
        G.graft_tree_verify_attn(vs.ctx, Q=vs.Q, Kc=Kp.cuda()[:, :, :100], Vc=Vp.cuda()[:, :, :100], O=vs.O, seq_len=vs.seq_len,
                                 tree_size=vs.tree_size, tree_anc=vs.tree_anc, scale=w.scale,
                                 block_table=torch.from_numpy(table).cuda(), S_cap=w.S_cap)
