"""ctypes binding of libgraft.so: the same entry points as include/graft.h, taking torch CUDA
tensors.  Argument marshalling only; every step of the path runs in the library's kernels.
PyTorch supplies device memory and the stream, nothing else.

Importing this module loads the library and raises if it has not been built
(`python -m paper_2605_20104_b200.build`): there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgraft.so")

if not os.path.exists(LIB_PATH):
    raise ImportError("libgraft.so is not built; run `python -m paper_2605_20104_b200.build` "
                      "(the CUDA library is the only implementation, there is no fallback)")
_lib = C.CDLL(LIB_PATH)

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE_TOO_SMALL, ERR_CUDA, ERR_SCRATCH_LIMIT = 0, -1, -2, -3, -4, -5
FLAG_BAD_SIZE, FLAG_BAD_PARENT, FLAG_BAD_TOKEN, FLAG_ORPHAN = 1, 2, 4, 8
FLAG_BUDGET, FLAG_BAD_TEMPLATE, FLAG_NAN_SCORE, FLAG_BAD_PATH, FLAG_WAIT_TIMEOUT, FLAG_INTERNAL = 16, 32, 64, 128, 256, 512
PRUNE_NONE, PRUNE_TOPK, PRUNE_GATED, PRUNE_NODE = 0, 1, 2, 3
ATTN_AUTO, ATTN_MMA_SYNC, ATTN_TCGEN05, ATTN_TCGEN05_1SM, ATTN_TCGEN05_2SM, ATTN_TCGEN05_L2PAIR = 0, 1, 2, 3, 4, 5

EXPORTS = ("graft_workspace_bytes", "graft_create", "graft_destroy", "graft_status_string", "graft_device_status",
           "graft_build_tree", "graft_tree_verify_attn", "graft_accept", "graft_compact_kv",
           "graft_noalloc_scratch_bytes", "graft_tree_verify_attn_noalloc", "graft_update_adjacency",
           "graft_retrieve_envelope", "graft_path_indices", "graft_accept_stochastic",
           "graft_accept_stochastic_scratch_floats")

_vp = C.c_void_p


class BuildParams(C.Structure):
    _fields_ = ([(n, C.c_int) for n in ("B", "N_max", "T_max", "K_max", "V", "k", "S_cap", "mode", "gate_depth")] +
                [("node_threshold", C.c_float), ("n_ckpt", C.c_int), ("N_tmpl", C.c_int)] +
                [(n, _vp) for n in ("draft_token", "draft_parent", "draft_score", "n_draft", "seq_len", "M", "keep_count",
                                    "k_max", "ckpt_depth", "ckpt_keep", "ckpt_log_tau", "tmpl_offset", "tmpl_parent",
                                    "tmpl_rank", "tree_token", "tree_parent", "tree_pos", "tree_src", "tree_anc",
                                    "tree_size")] +
                [("N_env", C.c_int), ("env_token", _vp), ("tmpl_env", _vp), ("attach_tail", C.c_int)])


class EnvelopeParams(C.Structure):
    _fields_ = ([(n, C.c_int) for n in ("B", "V", "k", "N_env")] + [("root_token", _vp), ("root_stride", C.c_int64)] +
                [(n, _vp) for n in ("M", "env_parent", "env_rank", "env_token")])


class AcceptStochasticParams(C.Structure):
    _fields_ = ([(n, C.c_int) for n in ("B", "T_max", "V")] + [("temperature", C.c_float), ("logits", _vp),
                 ("logits_stride_row", C.c_int64)] +
                [(n, _vp) for n in ("tree_token", "tree_parent", "tree_size", "u_accept", "u_bonus", "row_stats", "n_acc", "path",
                                    "best_node", "bonus")])


class PathsParams(C.Structure):
    _fields_ = ([(n, C.c_int) for n in ("B", "T_max", "D_max")] +
                [(n, _vp) for n in ("tree_parent", "tree_size", "path_index", "n_paths")])


class AttnParams(C.Structure):
    _fields_ = ([(n, C.c_int) for n in ("B", "T_max", "Hq", "Hkv", "d", "S_cap")] +
                [("scale", C.c_float), ("variant", C.c_int),
                 ("Q", _vp), ("q_stride_b", C.c_int64), ("q_stride_t", C.c_int64), ("q_stride_h", C.c_int64),
                 ("Kc", _vp), ("Vc", _vp),
                 ("kv_stride_b", C.c_int64), ("kv_stride_h", C.c_int64), ("kv_stride_s", C.c_int64),
                 ("O", _vp), ("o_stride_b", C.c_int64), ("o_stride_t", C.c_int64), ("o_stride_h", C.c_int64),
                 ("LSE", _vp), ("seq_len", _vp), ("tree_size", _vp), ("tree_anc", _vp),
                 ("block_table", _vp), ("page_size", C.c_int), ("blocks_per_seq", C.c_int), ("n_blocks", C.c_int)])


class AcceptParams(C.Structure):
    _fields_ = ([("B", C.c_int), ("T_max", C.c_int)] +
                [(n, _vp) for n in ("tree_token", "tree_parent", "tree_anc", "tree_size", "target_next", "n_acc", "path",
                                    "best_node", "bonus")])


class UpdateParams(C.Structure):
    _fields_ = ([(n, C.c_int) for n in ("B", "T_max", "V", "k")] + [("logits", _vp), ("logits_stride_row", C.c_int64)] +
                [(n, _vp) for n in ("tree_token", "tree_size", "M", "target_next")])


class CompactParams(C.Structure):
    _fields_ = ([(n, C.c_int) for n in ("B", "Hkv", "d", "S_cap", "T_max", "n_layers")] +
                [(n, C.c_int64) for n in ("layer_stride", "kv_stride_b", "kv_stride_h", "kv_stride_s")] +
                [(n, _vp) for n in ("Kc", "Vc", "seq_len", "n_acc", "path", "new_seq_len", "block_table")] +
                [(n, C.c_int) for n in ("page_size", "blocks_per_seq", "n_blocks")])


_lib.graft_workspace_bytes.restype = C.c_size_t
_lib.graft_workspace_bytes.argtypes = [C.c_int] * 6
_lib.graft_create.restype = C.c_int
_lib.graft_create.argtypes = [C.POINTER(_vp), C.c_int, _vp, C.c_size_t]
_lib.graft_destroy.restype = C.c_int
_lib.graft_destroy.argtypes = [_vp]
_lib.graft_status_string.restype = C.c_char_p
_lib.graft_status_string.argtypes = [C.c_int]
_lib.graft_device_status.restype = C.c_int
_lib.graft_device_status.argtypes = [_vp, _vp, C.POINTER(C.c_uint), C.c_int]
for _name, _typ in (("graft_build_tree", BuildParams), ("graft_tree_verify_attn", AttnParams),
                    ("graft_accept", AcceptParams), ("graft_compact_kv", CompactParams),
                    ("graft_update_adjacency", UpdateParams), ("graft_retrieve_envelope", EnvelopeParams),
                    ("graft_path_indices", PathsParams), ("graft_accept_stochastic", AcceptStochasticParams)):
    getattr(_lib, _name).restype = C.c_int
    getattr(_lib, _name).argtypes = [_vp, C.POINTER(_typ), _vp]


_lib.graft_noalloc_scratch_bytes.restype = C.c_size_t
_lib.graft_noalloc_scratch_bytes.argtypes = []
_lib.graft_accept_stochastic_scratch_floats.restype = C.c_size_t
_lib.graft_accept_stochastic_scratch_floats.argtypes = [C.c_int] * 3
_lib.graft_tree_verify_attn_noalloc.restype = C.c_int
_lib.graft_tree_verify_attn_noalloc.argtypes = [C.POINTER(AttnParams), _vp, _vp]


class GraftError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s: %s (%d)" % (where, _lib.graft_status_string(code).decode(), code))


def _check(code: int, where: str) -> None:
    if code != OK:
        raise GraftError(code, where)


def _ptr(t: Optional[torch.Tensor], dtype=None) -> Optional[int]:
    if t is None:
        return None
    assert t.is_cuda, "device tensor expected"
    if dtype is not None:
        assert t.dtype == dtype, (t.dtype, dtype)
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def graft_workspace_bytes(device: int, B: int, Hq: int, Hkv: int, d: int, T_max: int) -> int:
    return int(_lib.graft_workspace_bytes(device, B, Hq, Hkv, d, T_max))


class Context:
    """graft_ctx plus the torch-allocated workspace it is bound to."""

    def __init__(self, B: int, Hq: int, Hkv: int, d: int, T_max: int, device: Optional[int] = None,
                 workspace: Optional[torch.Tensor] = None):
        self.device = torch.cuda.current_device() if device is None else device
        if workspace is None:
            n = graft_workspace_bytes(self.device, B, Hq, Hkv, d, T_max)
            if n == 0:
                raise GraftError(ERR_UNSUPPORTED, "graft_workspace_bytes")
            workspace = torch.empty(n, dtype=torch.uint8, device="cuda:%d" % self.device)
        self.workspace = workspace
        h = _vp()
        _check(_lib.graft_create(C.byref(h), self.device, workspace.data_ptr(), workspace.numel()), "graft_create")
        self.handle = h

    def close(self) -> None:
        if self.handle:
            _lib.graft_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def device_status(self, clear: bool = True) -> int:
        """Synchronises the current stream and returns the accumulated GRAFT_FLAG_* bits."""
        f = C.c_uint(0)
        _check(_lib.graft_device_status(self.handle, _stream(), C.byref(f), int(clear)), "graft_device_status")
        return int(f.value)


def launch(name: str, ctx: Context, params) -> None:
    """Issues entry point `name` with an already marshalled params struct (see *_params below);
    lets a caller that repeats a call with the same buffers skip the marshalling."""
    _check(getattr(_lib, name)(ctx.handle, C.byref(params), _stream()), name)


def build_tree_params(*, mode: int, K_max: int, V: int, k: int, S_cap: int,
                     draft_token, draft_parent, draft_score, n_draft, seq_len, M=None, keep_count=None, k_max=None,
                     gate_depth: int = 0, node_threshold: float = 0.0, ckpt_depth=None, ckpt_keep=None,
                     ckpt_log_tau=None, tmpl_offset=None, tmpl_parent=None, tmpl_rank=None,
                     tree_token, tree_parent, tree_pos, tree_src, tree_anc, tree_size,
                     env_token=None, tmpl_env=None, attach_tail: bool = False) -> BuildParams:
    """env_token [B, N_env] / tmpl_env [N_tmpl]: take the grafted tokens from a precomputed retrieval envelope."""
    B, N_max = draft_token.shape
    T_max = tree_token.shape[1]
    i32, f32 = torch.int32, torch.float32
    p = BuildParams(B=B, N_max=N_max, T_max=T_max, K_max=K_max, V=V, k=k, S_cap=S_cap, mode=mode, gate_depth=gate_depth,
                    node_threshold=node_threshold, n_ckpt=0 if ckpt_depth is None else ckpt_depth.numel(),
                    N_tmpl=0 if tmpl_parent is None else tmpl_parent.numel(),
                    draft_token=_ptr(draft_token, i32), draft_parent=_ptr(draft_parent, i32),
                    draft_score=_ptr(draft_score, f32), n_draft=_ptr(n_draft, i32), seq_len=_ptr(seq_len, i32),
                    M=_ptr(M, i32), keep_count=_ptr(keep_count, i32), k_max=_ptr(k_max, i32),
                    ckpt_depth=_ptr(ckpt_depth, i32), ckpt_keep=_ptr(ckpt_keep, i32),
                    ckpt_log_tau=_ptr(ckpt_log_tau, f32), tmpl_offset=_ptr(tmpl_offset, i32),
                    tmpl_parent=_ptr(tmpl_parent, i32), tmpl_rank=_ptr(tmpl_rank, i32),
                    tree_token=_ptr(tree_token, i32), tree_parent=_ptr(tree_parent, i32), tree_pos=_ptr(tree_pos, i32),
                    tree_src=_ptr(tree_src, i32), tree_anc=_ptr(tree_anc, torch.int64), tree_size=_ptr(tree_size, i32),
                    N_env=0 if env_token is None else env_token.shape[1],
                    env_token=_ptr(env_token, i32), tmpl_env=_ptr(tmpl_env, i32), attach_tail=int(attach_tail))
    return p


def graft_build_tree(ctx: Context, **kw) -> None:
    launch("graft_build_tree", ctx, build_tree_params(**kw))


def tree_verify_attn_params(*, Q, Kc, Vc, O, seq_len, tree_size, tree_anc, scale: float,
                            LSE=None, variant: int = ATTN_AUTO, block_table=None, S_cap: Optional[int] = None) -> AttnParams:
    """Q, O: bf16 [B, T_max, Hq, d]; Kc, Vc: bf16 [B, Hkv, S_cap, d] (any strides with a contiguous
    last axis); tree_anc: int64 [B, T_max] holding the 64-bit masks.
    Paged caches: block_table int32 [B, blocks_per_seq] and Kc, Vc pools [n_blocks, Hkv, page_size, d];
    S_cap (logical slots per sequence) then defaults to blocks_per_seq * page_size."""
    bf = torch.bfloat16
    B, T_max, Hq, d = Q.shape
    paged = {}
    if block_table is None:
        _, Hkv, S_cap, _ = Kc.shape
    else:
        n_blocks, Hkv, page_size, _ = Kc.shape
        assert block_table.shape[0] == B and block_table.is_contiguous()
        S_cap = block_table.shape[1] * page_size if S_cap is None else S_cap
        paged = dict(block_table=_ptr(block_table, torch.int32), page_size=page_size, blocks_per_seq=block_table.shape[1],
                     n_blocks=n_blocks)
    assert Q.stride(3) == 1 and Kc.stride(3) == 1 and Vc.stride(3) == 1 and O.stride(3) == 1
    assert Kc.stride() == Vc.stride() and Kc.shape == Vc.shape and O.shape == Q.shape
    p = AttnParams(B=B, T_max=T_max, Hq=Hq, Hkv=Hkv, d=d, S_cap=S_cap, scale=scale, variant=variant,
                   Q=_ptr(Q, bf), q_stride_b=Q.stride(0), q_stride_t=Q.stride(1), q_stride_h=Q.stride(2),
                   Kc=_ptr(Kc, bf), Vc=_ptr(Vc, bf), kv_stride_b=Kc.stride(0), kv_stride_h=Kc.stride(1),
                   kv_stride_s=Kc.stride(2),
                   O=_ptr(O, bf), o_stride_b=O.stride(0), o_stride_t=O.stride(1), o_stride_h=O.stride(2),
                   LSE=_ptr(LSE, torch.float32), seq_len=_ptr(seq_len, torch.int32),
                   tree_size=_ptr(tree_size, torch.int32), tree_anc=_ptr(tree_anc, torch.int64), **paged)
    return p


def graft_tree_verify_attn(ctx: Context, **kw) -> None:
    launch("graft_tree_verify_attn", ctx, tree_verify_attn_params(**kw))


def graft_noalloc_scratch_bytes() -> int:
    return int(_lib.graft_noalloc_scratch_bytes())


def graft_tree_verify_attn_noalloc(*, device_flags_out=None, **kw) -> None:
    """The attention call for callers that cannot allocate: no Context, no workspace; scratch is the
    library's static 40 MiB device array.  Same tensor arguments as graft_tree_verify_attn.
    device_flags_out: optional int32 CUDA tensor (1 element) that receives the call's status flags."""
    p = tree_verify_attn_params(**kw)
    _check(_lib.graft_tree_verify_attn_noalloc(C.byref(p), _stream(), _ptr(device_flags_out, torch.int32)),
           "graft_tree_verify_attn_noalloc")


def accept_params(*, tree_token, tree_parent, tree_anc, tree_size, target_next, n_acc, path, best_node,
                  bonus) -> AcceptParams:
    i32 = torch.int32
    B, T_max = tree_token.shape
    p = AcceptParams(B=B, T_max=T_max, tree_token=_ptr(tree_token, i32), tree_parent=_ptr(tree_parent, i32),
                     tree_anc=_ptr(tree_anc, torch.int64), tree_size=_ptr(tree_size, i32),
                     target_next=_ptr(target_next, i32), n_acc=_ptr(n_acc, i32), path=_ptr(path, i32),
                     best_node=_ptr(best_node, i32), bonus=_ptr(bonus, i32))
    return p


def update_adjacency_params(*, logits, tree_token, tree_size, M, target_next=None) -> UpdateParams:
    """logits: bf16 [B*T_max, V] (rows may be strided); M: int32 [V, k], updated in place."""
    i32 = torch.int32
    B, T_max = tree_token.shape
    assert logits.dim() == 2 and logits.shape[0] == B * T_max and logits.stride(1) == 1
    V, k = M.shape
    assert logits.shape[1] == V and M.is_contiguous()
    return UpdateParams(B=B, T_max=T_max, V=V, k=k, logits=_ptr(logits, torch.bfloat16),
                        logits_stride_row=logits.stride(0), tree_token=_ptr(tree_token, i32), tree_size=_ptr(tree_size, i32),
                        M=_ptr(M, i32), target_next=_ptr(target_next, i32) if target_next is not None else None)


def graft_update_adjacency(ctx: Context, **kw) -> None:
    launch("graft_update_adjacency", ctx, update_adjacency_params(**kw))


def retrieve_envelope_params(*, root_token, M, env_parent, env_rank, env_token, root_stride: int = 1) -> EnvelopeParams:
    """root_token: int32, request b's root at element b * root_stride (draft_token with root_stride = N_max reads the
    draft trees' node 0 in place); env_token: int32 [B, N_env] out."""
    i32 = torch.int32
    B, N_env = env_token.shape
    V, k = M.shape
    assert M.is_contiguous() and env_token.is_contiguous() and env_parent.numel() == N_env and env_rank.numel() == N_env
    assert root_token.numel() > (B - 1) * root_stride
    return EnvelopeParams(B=B, V=V, k=k, N_env=N_env, root_token=_ptr(root_token, i32), root_stride=root_stride,
                          M=_ptr(M, i32), env_parent=_ptr(env_parent, i32), env_rank=_ptr(env_rank, i32),
                          env_token=_ptr(env_token, i32))


def graft_retrieve_envelope(ctx: Context, **kw) -> None:
    launch("graft_retrieve_envelope", ctx, retrieve_envelope_params(**kw))


def path_indices_params(*, tree_parent, tree_size, path_index, n_paths) -> PathsParams:
    """path_index: int32 [B, T_max, D_max] out; n_paths: int32 [B] out."""
    i32 = torch.int32
    B, T_max, D_max = path_index.shape
    assert tree_parent.shape == (B, T_max) and path_index.is_contiguous()
    return PathsParams(B=B, T_max=T_max, D_max=D_max, tree_parent=_ptr(tree_parent, i32), tree_size=_ptr(tree_size, i32),
                       path_index=_ptr(path_index, i32), n_paths=_ptr(n_paths, i32))


def graft_path_indices(ctx: Context, **kw) -> None:
    launch("graft_path_indices", ctx, path_indices_params(**kw))


def accept_stochastic_params(*, logits, temperature: float, tree_token, tree_parent, tree_size, u_accept, u_bonus, row_stats,
                             n_acc, path, best_node, bonus) -> AcceptStochasticParams:
    """logits: bf16 [B*T_max, V] (rows may be strided); u_accept float32 [B, T_max], u_bonus float32 [B] in [0, 1);
    row_stats: float32 scratch of graft_accept_stochastic_scratch_floats(B, T_max, V) elements."""
    i32, f32 = torch.int32, torch.float32
    B, T_max = tree_token.shape
    assert logits.dim() == 2 and logits.shape[0] == B * T_max and logits.stride(1) == 1
    assert u_accept.shape == (B, T_max) and u_bonus.shape == (B,)
    assert row_stats.numel() >= graft_accept_stochastic_scratch_floats(B, T_max, logits.shape[1])
    return AcceptStochasticParams(B=B, T_max=T_max, V=logits.shape[1], temperature=temperature, logits=_ptr(logits, torch.bfloat16),
                                  logits_stride_row=logits.stride(0), tree_token=_ptr(tree_token, i32),
                                  tree_parent=_ptr(tree_parent, i32), tree_size=_ptr(tree_size, i32),
                                  u_accept=_ptr(u_accept, f32), u_bonus=_ptr(u_bonus, f32), row_stats=_ptr(row_stats, f32),
                                  n_acc=_ptr(n_acc, i32), path=_ptr(path, i32), best_node=_ptr(best_node, i32),
                                  bonus=_ptr(bonus, i32))


def graft_accept_stochastic_scratch_floats(B: int, T_max: int, V: int) -> int:
    return int(_lib.graft_accept_stochastic_scratch_floats(B, T_max, V))


def graft_accept_stochastic(ctx: Context, **kw) -> None:
    launch("graft_accept_stochastic", ctx, accept_stochastic_params(**kw))


def graft_accept(ctx: Context, **kw) -> None:
    launch("graft_accept", ctx, accept_params(**kw))


def compact_kv_params(*, Kc, Vc, seq_len, n_acc, path, new_seq_len, block_table=None, S_cap: Optional[int] = None) -> CompactParams:
    """Kc, Vc: bf16 [B, Hkv, S_cap, d] or [n_layers, B, Hkv, S_cap, d], compacted in place.
    Paged caches: block_table int32 [B, blocks_per_seq] and pools [n_blocks, Hkv, page_size, d] (or with a leading
    layer axis)."""
    bf, i32 = torch.bfloat16, torch.int32
    if Kc.dim() == 4:
        n_layers, layer_stride, off = 1, 0, 0
    else:
        n_layers, layer_stride, off = Kc.shape[0], Kc.stride(0), 1
    B, Hkv, S_cap_, d = Kc.shape[off:]
    paged = {}
    if block_table is not None:
        n_blocks, page_size, B = B, S_cap_, block_table.shape[0]
        S_cap_ = block_table.shape[1] * page_size if S_cap is None else S_cap
        paged = dict(block_table=_ptr(block_table, i32), page_size=page_size, blocks_per_seq=block_table.shape[1], n_blocks=n_blocks)
    S_cap = S_cap_
    assert Kc.stride() == Vc.stride() and Kc.stride(-1) == 1
    p = CompactParams(B=B, Hkv=Hkv, d=d, S_cap=S_cap, T_max=path.shape[1], n_layers=n_layers, layer_stride=layer_stride,
                      kv_stride_b=Kc.stride(off), kv_stride_h=Kc.stride(off + 1), kv_stride_s=Kc.stride(off + 2),
                      Kc=_ptr(Kc, bf), Vc=_ptr(Vc, bf), seq_len=_ptr(seq_len, i32), n_acc=_ptr(n_acc, i32),
                      path=_ptr(path, i32), new_seq_len=_ptr(new_seq_len, i32), **paged)
    return p


def graft_compact_kv(ctx: Context, **kw) -> None:
    launch("graft_compact_kv", ctx, compact_kv_params(**kw))
