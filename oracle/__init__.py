"""ctypes front end of the CPU oracle (oracle/graft_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the benchmark's
CPU-baseline leg; the CUDA package never imports it.  Argument marshalling only: all of the
oracle's arithmetic is in the C file.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "graft_oracle.c")
_LIB = os.path.join(_HERE, "libgraft_oracle.so")

MODE_NONE, MODE_TOPK, MODE_GATED, MODE_NODE = 0, 1, 2, 3
FLAG_BAD_SIZE, FLAG_BAD_PARENT, FLAG_BAD_TOKEN, FLAG_ORPHAN = 1, 2, 4, 8
FLAG_BUDGET, FLAG_BAD_TEMPLATE, FLAG_NAN_SCORE = 16, 32, 64


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O3 -march=native -fopenmp).  Idempotent."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O3", "-march=native", "-fopenmp", "-std=c11", "-shared", "-fPIC",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_i32p = C.POINTER(C.c_int32)
_f32p = C.POINTER(C.c_float)
_u16p = C.POINTER(C.c_uint16)
_u64p = C.POINTER(C.c_uint64)
_f64p = C.POINTER(C.c_double)


class _BuildArgs(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("B", "N_max", "T_max", "K_max", "V", "k", "S_cap", "mode", "gate_depth")] + [
        ("node_threshold", C.c_float), ("n_ckpt", C.c_int), ("N_tmpl", C.c_int),
        ("draft_token", _i32p), ("draft_parent", _i32p), ("draft_score", _f32p), ("n_draft", _i32p),
        ("seq_len", _i32p), ("M", _i32p), ("keep_count", _i32p), ("k_max", _i32p),
        ("ckpt_depth", _i32p), ("ckpt_keep", _i32p), ("ckpt_log_tau", _f32p), ("tmpl_offset", _i32p),
        ("tmpl_parent", _i32p), ("tmpl_rank", _i32p),
        ("tree_token", _i32p), ("tree_parent", _i32p), ("tree_pos", _i32p), ("tree_src", _i32p),
        ("tree_anc", _u64p), ("tree_size", _i32p), ("attach_tail", C.c_int)]


class _AttnArgs(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("B", "T_max", "Hq", "Hkv", "d", "S_cap")] + [
        ("scale", C.c_double), ("Q", _u16p), ("Kc", _u16p), ("Vc", _u16p),
        ("seq_len", _i32p), ("tree_size", _i32p), ("tree_anc", _u64p),
        ("O", _f64p), ("LSE", _f64p), ("rowsum", _f64p)]


class _AcceptArgs(C.Structure):
    _fields_ = [("B", C.c_int), ("T_max", C.c_int), ("tree_token", _i32p), ("tree_parent", _i32p),
                ("tree_size", _i32p), ("target_next", _i32p), ("n_acc", _i32p), ("best_node", _i32p),
                ("bonus", _i32p), ("path", _i32p)]


class _CompactArgs(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("B", "Hkv", "d", "S_cap", "T_max", "n_layers")] + [
        ("layer_stride", C.c_size_t), ("K_old", _u16p), ("V_old", _u16p), ("K_new", _u16p), ("V_new", _u16p),
        ("seq_len", _i32p), ("n_acc", _i32p), ("path", _i32p), ("new_seq_len", _i32p)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_build_tree.restype = C.c_uint
        _lib.orc_tree_attn.restype = C.c_int
        _lib.orc_tree_attn_rows.restype = C.c_int
        _lib.orc_accept.restype = None
        _lib.orc_compact_kv.restype = None
        _lib.orc_update_adjacency.restype = C.c_uint
    return _lib


def _p(a: Optional[np.ndarray], typ, dtype):
    if a is None:
        return C.cast(None, typ)
    assert a.dtype == dtype and a.flags["C_CONTIGUOUS"], (a.dtype, dtype)
    return a.ctypes.data_as(typ)


def _arr(a, dtype) -> Optional[np.ndarray]:
    return None if a is None else np.ascontiguousarray(a, dtype=dtype)


def build_tree(w) -> dict:
    """Tree assembly on a workload (any object with the Workload fields).  Returns a dict of
    tree_token, tree_parent, tree_pos, tree_src (int32 [B, T_max]), tree_anc (uint64 [B, T_max]),
    tree_size (int32 [B]) and flags (int)."""
    B, T = w.B, w.T_max
    out = dict(tree_token=np.empty((B, T), np.int32), tree_parent=np.empty((B, T), np.int32),
               tree_pos=np.empty((B, T), np.int32), tree_src=np.empty((B, T), np.int32),
               tree_anc=np.empty((B, T), np.uint64), tree_size=np.empty(B, np.int32))
    keep = dict(dt=_arr(w.draft_token, np.int32), dp=_arr(w.draft_parent, np.int32),
                ds=_arr(w.draft_score, np.float32), nd=_arr(w.n_draft, np.int32), sl=_arr(w.seq_len, np.int32),
                M=_arr(w.M, np.int32), kc=_arr(w.keep_count, np.int32), km=_arr(w.k_max, np.int32),
                cd=_arr(w.ckpt_depth, np.int32), ck=_arr(w.ckpt_keep, np.int32),
                ct=_arr(w.ckpt_log_tau, np.float32), to=_arr(w.tmpl_offset, np.int32),
                tp=_arr(w.tmpl_parent, np.int32), tr=_arr(w.tmpl_rank, np.int32))
    a = _BuildArgs(B=B, N_max=w.N_max, T_max=T, K_max=w.K_max, V=w.V, k=w.k, S_cap=w.S_cap, mode=w.mode,
                   gate_depth=w.gate_depth, node_threshold=w.node_threshold,
                   n_ckpt=0 if keep["cd"] is None else len(keep["cd"]), N_tmpl=len(keep["tp"]),
                   draft_token=_p(keep["dt"], _i32p, np.int32), draft_parent=_p(keep["dp"], _i32p, np.int32),
                   draft_score=_p(keep["ds"], _f32p, np.float32), n_draft=_p(keep["nd"], _i32p, np.int32),
                   seq_len=_p(keep["sl"], _i32p, np.int32), M=_p(keep["M"], _i32p, np.int32),
                   keep_count=_p(keep["kc"], _i32p, np.int32), k_max=_p(keep["km"], _i32p, np.int32),
                   ckpt_depth=_p(keep["cd"], _i32p, np.int32), ckpt_keep=_p(keep["ck"], _i32p, np.int32),
                   ckpt_log_tau=_p(keep["ct"], _f32p, np.float32), tmpl_offset=_p(keep["to"], _i32p, np.int32),
                   tmpl_parent=_p(keep["tp"], _i32p, np.int32), tmpl_rank=_p(keep["tr"], _i32p, np.int32),
                   tree_token=_p(out["tree_token"], _i32p, np.int32), tree_parent=_p(out["tree_parent"], _i32p, np.int32),
                   tree_pos=_p(out["tree_pos"], _i32p, np.int32), tree_src=_p(out["tree_src"], _i32p, np.int32),
                   tree_anc=_p(out["tree_anc"], _u64p, np.uint64), tree_size=_p(out["tree_size"], _i32p, np.int32),
                   attach_tail=int(bool(getattr(w, "attach_tail", False))))
    out["flags"] = int(lib().orc_build_tree(C.byref(a)))
    return out


def _attn_args(Q, Kc, Vc, seq_len, tree_size, tree_anc, scale, O, LSE, rowsum):
    B, T_max, Hq, d = Q.shape
    _, Hkv, S_cap, _ = Kc.shape
    return _AttnArgs(B=B, T_max=T_max, Hq=Hq, Hkv=Hkv, d=d, S_cap=S_cap, scale=float(scale),
                     Q=_p(Q, _u16p, np.uint16), Kc=_p(Kc, _u16p, np.uint16), Vc=_p(Vc, _u16p, np.uint16),
                     seq_len=_p(seq_len, _i32p, np.int32), tree_size=_p(tree_size, _i32p, np.int32),
                     tree_anc=_p(tree_anc, _u64p, np.uint64), O=_p(O, _f64p, np.float64),
                     LSE=_p(LSE, _f64p, np.float64), rowsum=_p(rowsum, _f64p, np.float64))


def tree_attn(Q, Kc, Vc, seq_len, tree_size, tree_anc, scale, rows: Optional[np.ndarray] = None) -> dict:
    """Tree-masked attention in fp64.  Q [B,T_max,Hq,d], Kc/Vc [B,Hkv,S_cap,d] are uint16 arrays
    holding bf16 bits.  With rows (int32 [n,3] of (b,t,h)) only those rows are computed; the
    rest of O stays NaN.  Returns O, LSE, rowsum and the thread count used."""
    Q, Kc, Vc = (np.ascontiguousarray(x, np.uint16) for x in (Q, Kc, Vc))
    seq_len, tree_size = _arr(seq_len, np.int32), _arr(tree_size, np.int32)
    tree_anc = _arr(tree_anc, np.uint64)
    B, T_max, Hq, d = Q.shape
    fill = 0.0 if rows is None else np.nan
    O = np.full((B, T_max, Hq, d), fill, np.float64)
    LSE = np.full((B, Hq, T_max), fill, np.float64)
    rowsum = np.full((B, Hq, T_max), fill, np.float64)
    a = _attn_args(Q, Kc, Vc, seq_len, tree_size, tree_anc, scale, O, LSE, rowsum)
    if rows is None:
        nt = lib().orc_tree_attn(C.byref(a))
    else:
        # every row once: the C loop hands rows to threads, and a row listed twice would be written by two of them at once
        rows = np.unique(np.ascontiguousarray(rows, np.int32).reshape(-1, 3), axis=0)
        nt = lib().orc_tree_attn_rows(C.byref(a), C.c_int(len(rows)), _p(rows, _i32p, np.int32))
    return dict(O=O, LSE=LSE, rowsum=rowsum, threads=int(nt))


def accept(tree_token, tree_parent, tree_size, target_next) -> dict:
    tt, tp = _arr(tree_token, np.int32), _arr(tree_parent, np.int32)
    ts, tn = _arr(tree_size, np.int32), _arr(target_next, np.int32)
    B, T = tt.shape
    out = dict(n_acc=np.empty(B, np.int32), best_node=np.empty(B, np.int32), bonus=np.empty(B, np.int32),
               path=np.empty((B, T), np.int32))
    a = _AcceptArgs(B=B, T_max=T, tree_token=_p(tt, _i32p, np.int32), tree_parent=_p(tp, _i32p, np.int32),
                    tree_size=_p(ts, _i32p, np.int32), target_next=_p(tn, _i32p, np.int32),
                    n_acc=_p(out["n_acc"], _i32p, np.int32), best_node=_p(out["best_node"], _i32p, np.int32),
                    bonus=_p(out["bonus"], _i32p, np.int32), path=_p(out["path"], _i32p, np.int32))
    lib().orc_accept(C.byref(a))
    return out


def compact_kv(Kc, Vc, seq_len, n_acc, path) -> dict:
    """Kc/Vc: uint16 [B,Hkv,S_cap,d] or [n_layers,B,Hkv,S_cap,d].  Returns new K, V (copies) and
    new_seq_len."""
    Kc, Vc = np.ascontiguousarray(Kc, np.uint16), np.ascontiguousarray(Vc, np.uint16)
    shp = Kc.shape
    if Kc.ndim == 4:
        Kc, Vc = Kc[None], Vc[None]
    nl, B, Hkv, S_cap, d = Kc.shape
    sl, na, pa = _arr(seq_len, np.int32), _arr(n_acc, np.int32), _arr(path, np.int32)
    Kn, Vn = np.empty_like(Kc), np.empty_like(Vc)
    nsl = np.empty(B, np.int32)
    a = _CompactArgs(B=B, Hkv=Hkv, d=d, S_cap=S_cap, T_max=pa.shape[1], n_layers=nl,
                     layer_stride=B * Hkv * S_cap * d, K_old=_p(Kc, _u16p, np.uint16), V_old=_p(Vc, _u16p, np.uint16),
                     K_new=_p(Kn, _u16p, np.uint16), V_new=_p(Vn, _u16p, np.uint16),
                     seq_len=_p(sl, _i32p, np.int32), n_acc=_p(na, _i32p, np.int32), path=_p(pa, _i32p, np.int32),
                     new_seq_len=_p(nsl, _i32p, np.int32))
    lib().orc_compact_kv(C.byref(a))
    return dict(K=Kn.reshape(shp), V=Vn.reshape(shp), new_seq_len=nsl)


def update_adjacency(logits_bits, tree_token, tree_size, M, k: int) -> dict:
    """logits_bits: uint16 (bf16 bit patterns) [B*T_max, V]; M: int32 [V, k].  Returns the updated copy of M,
    target_next [B, T_max] and the flag word."""
    lg = np.ascontiguousarray(logits_bits, np.uint16)
    tt, ts = _arr(tree_token, np.int32), _arr(tree_size, np.int32)
    B, T = tt.shape
    V = lg.shape[1]
    assert lg.shape[0] == B * T and M.shape == (V, k)
    Mn = np.array(M, dtype=np.int32, order="C", copy=True)
    tn = np.empty((B, T), np.int32)
    flags = lib().orc_update_adjacency(C.c_int(B), C.c_int(T), C.c_int(V), C.c_int(k), _p(lg, _u16p, np.uint16),
                                       _p(tt, _i32p, np.int32), _p(ts, _i32p, np.int32), _p(Mn, _i32p, np.int32),
                                       _p(tn, _i32p, np.int32))
    return dict(M=Mn, target_next=tn, flags=int(flags))


def retrieve_envelope(root_token, M, env_parent, env_rank, root_stride: int = 1) -> dict:
    """root_token: int32, request b's root at [b * root_stride]; M: int32 [V, k]; the template as parent / rank
    lists.  Returns env_token [B, N_env] and the flag word."""
    rt = np.ascontiguousarray(root_token, np.int32).reshape(-1)
    Mc = np.ascontiguousarray(M, np.int32)
    ep, er = _arr(env_parent, np.int32), _arr(env_rank, np.int32)
    V, k = Mc.shape
    B = (len(rt) + root_stride - 1) // root_stride
    out = np.empty((B, len(ep)), np.int32)
    fn = lib().orc_retrieve_envelope
    fn.restype = C.c_uint
    flags = fn(C.c_int(B), C.c_int(V), C.c_int(k), C.c_int(len(ep)), _p(rt, _i32p, np.int32), C.c_long(root_stride),
               _p(Mc, _i32p, np.int32), _p(ep, _i32p, np.int32), _p(er, _i32p, np.int32), _p(out, _i32p, np.int32))
    return dict(env_token=out, flags=int(flags))


def path_indices(tree_parent, tree_size, D_max: int) -> dict:
    """tree_parent: int32 [B, T_max]; returns path_index [B, T_max, D_max], n_paths [B] and the flag word."""
    tp, ts = _arr(tree_parent, np.int32), _arr(tree_size, np.int32)
    B, T = tp.shape
    out = np.empty((B, T, D_max), np.int32)
    n = np.empty(B, np.int32)
    fn = lib().orc_path_indices
    fn.restype = C.c_uint
    flags = fn(C.c_int(B), C.c_int(T), C.c_int(D_max), _p(tp, _i32p, np.int32), _p(ts, _i32p, np.int32),
               _p(out, _i32p, np.int32), _p(n, _i32p, np.int32))
    return dict(path_index=out, n_paths=n, flags=int(flags))


def accept_stochastic(logits_bits, temperature: float, tree_token, tree_parent, tree_size, u_accept, u_bonus) -> dict:
    """logits_bits: uint16 (bf16 bit patterns) [B*T_max, V]; u_accept float32 [B, T_max], u_bonus float32 [B].
    Returns n_acc, path, best_node, bonus, margin (float64 [B, 2]: accept decisions, bonus draw) and the flag word."""
    lg = np.ascontiguousarray(logits_bits, np.uint16)
    tt, tp, ts = _arr(tree_token, np.int32), _arr(tree_parent, np.int32), _arr(tree_size, np.int32)
    ua, ub = _arr(u_accept, np.float32), _arr(u_bonus, np.float32)
    B, T = tt.shape
    V = lg.shape[1]
    assert lg.shape[0] == B * T and ua.shape == (B, T) and ub.shape == (B,)
    out = dict(n_acc=np.empty(B, np.int32), best_node=np.empty(B, np.int32), bonus=np.empty(B, np.int32),
               path=np.empty((B, T), np.int32), margin=np.empty((B, 2), np.float64))
    fn = lib().orc_accept_stochastic
    fn.restype = C.c_uint
    flags = fn(C.c_int(B), C.c_int(T), C.c_int(V), _p(lg, _u16p, np.uint16), C.c_double(temperature),
               _p(tt, _i32p, np.int32), _p(tp, _i32p, np.int32), _p(ts, _i32p, np.int32), _p(ua, _f32p, np.float32),
               _p(ub, _f32p, np.float32), _p(out["n_acc"], _i32p, np.int32), _p(out["path"], _i32p, np.int32),
               _p(out["best_node"], _i32p, np.int32), _p(out["bonus"], _i32p, np.int32), _p(out["margin"], _f64p, np.float64))
    out["flags"] = int(flags)
    return out
