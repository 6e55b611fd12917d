"""graft_update_adjacency on the GPU against the oracle: M and target_next bit for bit."""
import numpy as np
import pytest
import torch

from paper_2605_20104_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def G():
    from paper_2605_20104_b200 import binding
    return binding


def run_gpu(G, lg_bits, tok, size, M0, want_next=True, pad_to=None):
    """lg_bits: uint16 [N, V].  The device copy has a row stride that is a multiple of 8 elements."""
    N, V = lg_bits.shape
    B, T = tok.shape
    stride = pad_to or (V + 7) // 8 * 8
    buf = torch.full((N, stride), float("nan"), dtype=torch.bfloat16, device="cuda")     # NaN in the padding columns
    buf[:, :V] = torch.from_numpy(lg_bits.view(np.int16).copy()).view(torch.bfloat16).cuda()
    lg = buf[:, :V]
    ctx = G.Context(B, 8, 8, 128, T, device=0)
    M = torch.from_numpy(M0.copy()).cuda()
    nxt = torch.full((B, T), -9, dtype=torch.int32, device="cuda") if want_next else None
    G.graft_update_adjacency(ctx, logits=lg, tree_token=torch.from_numpy(tok).cuda(), tree_size=torch.from_numpy(size).cuda(),
                             M=M, target_next=nxt)
    torch.cuda.synchronize()
    return M.cpu().numpy(), None if nxt is None else nxt.cpu().numpy(), ctx.device_status()


def check(orc, G, lg, tok, size, M0, k, **kw):
    ref = orc.update_adjacency(lg, tok, size, M0, k)
    M, nxt, flags = run_gpu(G, lg, tok, size, M0, **kw)
    assert (M == ref["M"]).all()
    if nxt is not None:
        assert (nxt == ref["target_next"]).all()
    assert flags == ref["flags"]
    return ref


def bits(x):
    return W.bf16_bits(torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16))


@pytest.mark.parametrize("V", [16, 97, 1000, 4099, 40000])
@pytest.mark.parametrize("k", [1, 4, 8, 16])
def test_random_rows_with_ties(orc, G, V, k):
    rng = np.random.default_rng(V * 31 + k)
    B, T = 3, 6
    x = np.round(rng.standard_normal((B * T, V)) * 4) * 0.5          # half-integer values: ties everywhere, also at the top
    lg = bits(x)
    tok = rng.integers(0, V, size=(B, T)).astype(np.int32)           # duplicates occur for small V
    tok[1, 2] = -1
    size = np.array([6, 4, 0], np.int32)
    M0 = rng.integers(0, V, size=(V, k)).astype(np.int32)
    check(orc, G, lg, tok, size, M0, k)


def test_constant_and_degenerate_rows(orc, G):
    """All entries equal (every entry ties with the threshold), -inf rows, rows with NaN, fewer than k numbers."""
    V, k = 5000, 8
    x = np.zeros((6, V), np.float32)
    x[1] = -np.inf
    x[2] = np.nan
    x[2, [7, 4000, 12]] = [1.0, 1.0, -np.inf]                          # three numbers only: -1 entries and the NaN flag
    x[3, ::2] = -0.0
    x[4] = np.linspace(-1, 1, V)
    x[4, 100:140] = np.nan
    x[5, :] = 3.0
    x[5, 4321] = np.inf
    tok = np.arange(6, dtype=np.int32).reshape(1, 6) * 11
    ref = check(orc, G, bits(x), tok, np.array([6], np.int32), np.full((V, k), -5, np.int32), k)
    assert ref["M"][0].tolist() == list(range(8)) and ref["M"][22].tolist() == [7, 4000, 12, -1, -1, -1, -1, -1]
    assert ref["flags"] == G.FLAG_NAN_SCORE


def test_one_thread_holds_all_large_entries(orc, G):
    """The largest entries all sit in the stride of one thread: the candidate list, not the thread maxima, finds them."""
    V, k = 40960, 8
    x = np.random.default_rng(5).standard_normal((2, V)).astype(np.float32)
    x[0, 8 * 17::4096] = 50.0 + np.arange(10)                           # ids 136, 4232, ...: all read by thread 17
    x[1, 8 * 300 + 3::4096] = 60.0
    tok = np.array([[3, 9]], np.int32)
    check(orc, G, bits(x), tok, np.array([2], np.int32), np.zeros((V, k), np.int32), k)


def test_duplicate_tokens_across_requests_and_flags(orc, G):
    rng = np.random.default_rng(9)
    B, T, V, k = 4, 8, 2048, 8
    lg = bits(rng.standard_normal((B * T, V)).astype(np.float32) * 3)
    tok = rng.integers(0, 12, size=(B, T)).astype(np.int32)            # 12 tokens over 32 nodes
    tok[3, 7] = V + 5                                                   # out of range: flagged, no update
    size = np.array([8, 5, 9, 8], np.int32)                             # 9 > T_max: that sequence is skipped and flagged
    ref = check(orc, G, lg, tok, size, np.full((V, k), -1, np.int32), k)
    assert ref["flags"] == (G.FLAG_BAD_TOKEN | G.FLAG_BAD_SIZE)


def test_no_target_next_and_strided_rows(orc, G):
    rng = np.random.default_rng(11)
    V, k = 3001, 8
    lg = bits(rng.standard_normal((8, V)).astype(np.float32))
    tok = rng.integers(0, V, size=(2, 4)).astype(np.int32)
    check(orc, G, lg, tok, np.array([4, 4], np.int32), np.zeros((V, k), np.int32), k, want_next=False, pad_to=3200)


def test_full_vocabulary(orc, G):
    """Qwen3 vocabulary, the long-context configuration's node count, generator-shaped logits."""
    B, T, V, k = 4, 64, 151936, 8
    lg = W.make_logits(B, T, V, seed=4)
    rng = np.random.default_rng(4)
    tok = rng.integers(0, V, size=(B, T)).astype(np.int32)
    tok[:, 0] = 1234                                                    # every root carries the same token
    size = np.array([48, 48, 60, 64], np.int32)
    M0 = rng.integers(0, V, size=(V, k)).astype(np.int32)
    check(orc, G, lg, tok, size, M0, k)


def test_argument_checks(G):
    ctx = G.Context(1, 8, 8, 128, 4, device=0)
    i32 = torch.int32
    lg = torch.zeros(4, 64, dtype=torch.bfloat16, device="cuda")
    tok = torch.zeros(1, 4, dtype=i32, device="cuda")
    size = torch.ones(1, dtype=i32, device="cuda")
    with pytest.raises(G.GraftError) as e:
        G.graft_update_adjacency(ctx, logits=lg, tree_token=tok, tree_size=size, M=torch.zeros(64, 17, dtype=i32, device="cuda"))
    assert e.value.code == G.ERR_UNSUPPORTED
    with pytest.raises(G.GraftError) as e:
        G.graft_update_adjacency(ctx, logits=lg[:, 1:], tree_token=tok, tree_size=size, M=torch.zeros(63, 8, dtype=i32, device="cuda"))
    assert e.value.code == G.ERR_INVALID_ARG
