"""One verify step on device buffers: build -> attention -> accept -> compact.

`VerifyStep` owns the device tensors of one workload (allocated through torch) and issues the four
C-ABI calls on the current stream with no host synchronisation in between.  It is plumbing for
tests, the benchmark and the smoke check: no arithmetic of the method happens here.
"""
from __future__ import annotations

from typing import Dict, Optional

import numpy as np
import torch

from . import binding as G
from .workloads import Workload, workload_envelope


def _dev(a, dtype=None, device="cuda"):
    if a is None:
        return None
    if isinstance(a, np.ndarray):
        a = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        a = a.to(dtype)
    return a.to(device, non_blocking=False).contiguous()


class VerifyStep:
    def __init__(self, w: Workload, n_layers: int = 1, device: Optional[int] = None, upload_qkv: bool = True):
        self.w = w
        self.dev = "cuda:%d" % (torch.cuda.current_device() if device is None else device)
        d = self.dev
        i32 = torch.int32
        B, T = w.B, w.T_max
        self.ctx = G.Context(B, w.Hq, w.Hkv, w.d, T, device=torch.device(d).index)
        # build inputs
        self.draft_token = _dev(w.draft_token, device=d)
        self.draft_parent = _dev(w.draft_parent, device=d)
        self.draft_score = _dev(w.draft_score, device=d)
        self.n_draft = _dev(w.n_draft, device=d)
        self.seq_len = _dev(w.seq_len, device=d)
        self.M = _dev(w.M, device=d)
        self.keep_count = _dev(w.keep_count, device=d)
        self.k_max = _dev(w.k_max, device=d)
        self.ckpt_depth = _dev(w.ckpt_depth, device=d)
        self.ckpt_keep = _dev(w.ckpt_keep, device=d)
        self.ckpt_log_tau = _dev(w.ckpt_log_tau, device=d)
        self.tmpl_offset = _dev(w.tmpl_offset, device=d)
        self.tmpl_parent = _dev(w.tmpl_parent, device=d) if len(w.tmpl_parent) else None
        self.tmpl_rank = _dev(w.tmpl_rank, device=d) if len(w.tmpl_rank) else None
        # build outputs
        self.tree_token = torch.empty(B, T, dtype=i32, device=d)
        self.tree_parent = torch.empty(B, T, dtype=i32, device=d)
        self.tree_pos = torch.empty(B, T, dtype=i32, device=d)
        self.tree_src = torch.empty(B, T, dtype=i32, device=d)
        self.tree_anc = torch.empty(B, T, dtype=torch.int64, device=d)
        self.tree_size = torch.empty(B, dtype=i32, device=d)
        # attention
        self.n_layers = n_layers
        self.Q = self.Kc = self.Vc = None
        if upload_qkv and w.Q is not None:
            self.set_qkv(w.Q, w.Kc, w.Vc)
        self.O = torch.empty(B, T, w.Hq, w.d, dtype=torch.bfloat16, device=d)
        self.LSE = torch.empty(B, w.Hq, T, dtype=torch.float32, device=d)
        # accept / compact
        self.target_next = torch.zeros(B, T, dtype=i32, device=d)
        self.n_acc = torch.empty(B, dtype=i32, device=d)
        self.path = torch.empty(B, T, dtype=i32, device=d)
        self.best_node = torch.empty(B, dtype=i32, device=d)
        self.bonus = torch.empty(B, dtype=i32, device=d)
        self.new_seq_len = torch.empty(B, dtype=i32, device=d)

    def set_qkv(self, Q: torch.Tensor, Kc: torch.Tensor, Vc: torch.Tensor) -> None:
        """Kc/Vc may be [B,Hkv,S_cap,d] (replicated over layers for compaction) or carry a leading
        layer axis; attention reads layer 0."""
        self.Q = Q.to(self.dev)
        if Kc.dim() == 4 and self.n_layers > 1:
            Kc = Kc.unsqueeze(0).expand(self.n_layers, *Kc.shape)
            Vc = Vc.unsqueeze(0).expand(self.n_layers, *Vc.shape)
        self.Kc = Kc.to(self.dev).contiguous()
        self.Vc = Vc.to(self.dev).contiguous()

    # ---- the four calls -------------------------------------------------------------------------
    # Each call marshals its params struct once per distinct set of buffers and re-issues the
    # cached struct afterwards, so a benchmark loop is not bound by Python-side marshalling.
    def _cached(self, key, make):
        cache = self.__dict__.setdefault("_params", {})
        if key not in cache:
            cache[key] = make()
        return cache[key]

    def retrieve_envelope(self, stream: Optional[torch.cuda.Stream] = None) -> None:
        """Fills the retrieval envelope of the workload's templates from the draft trees' root tokens; on `stream`
        (a side stream beside drafting) the next build() waits for it through an event."""
        if not hasattr(self, "env_token"):
            ep, er, te = workload_envelope(self.w)
            self.env_parent, self.env_rank, self.tmpl_env = (_dev(a, device=self.dev) for a in (ep, er, te))
            self.env_token = torch.empty(self.w.B, len(ep), dtype=torch.int32, device=self.dev) if len(ep) else None
            self._env_event = torch.cuda.Event()
        if self.env_token is None:          # the workload grafts nothing
            return
        params = self._cached("envelope", lambda: G.retrieve_envelope_params(
            root_token=self.draft_token, root_stride=self.w.N_max, M=self.M, env_parent=self.env_parent,
            env_rank=self.env_rank, env_token=self.env_token))
        if stream is None:
            G.launch("graft_retrieve_envelope", self.ctx, params)
        else:
            stream.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(stream):
                G.launch("graft_retrieve_envelope", self.ctx, params)
                self._env_event.record(stream)
            torch.cuda.current_stream().wait_event(self._env_event)

    def path_indices(self, D_max: Optional[int] = None) -> None:
        """Candidate-path table of the tree build() left: path_index [B, T_max, D_max], n_paths [B]."""
        D = self.w.T_max if D_max is None else D_max
        if getattr(self, "path_index", None) is None or self.path_index.shape[2] != D:
            self.path_index = torch.empty(self.w.B, self.w.T_max, D, dtype=torch.int32, device=self.dev)
            self.n_paths = torch.empty(self.w.B, dtype=torch.int32, device=self.dev)
        G.launch("graft_path_indices", self.ctx, self._cached(("paths", self.path_index.data_ptr()), lambda: G.path_indices_params(
            tree_parent=self.tree_parent, tree_size=self.tree_size, path_index=self.path_index, n_paths=self.n_paths)))

    def build(self, from_envelope: bool = False) -> None:
        """from_envelope: take the grafted tokens from the envelope retrieve_envelope() filled."""
        if from_envelope and self.env_token is not None:
            G.launch("graft_build_tree", self.ctx, self._cached("build_env", lambda: self._build_params(True)))
        else:
            G.launch("graft_build_tree", self.ctx, self._cached("build", self._build_params))

    def _build_params(self, from_envelope: bool = False):
        w = self.w
        env = dict(env_token=self.env_token, tmpl_env=self.tmpl_env) if from_envelope else {}
        return G.build_tree_params(**env, attach_tail=getattr(w, "attach_tail", False), mode=w.mode, K_max=w.K_max, V=w.V, k=w.k, S_cap=w.S_cap,
                           draft_token=self.draft_token, draft_parent=self.draft_parent, draft_score=self.draft_score,
                           n_draft=self.n_draft, seq_len=self.seq_len, M=self.M, keep_count=self.keep_count,
                           k_max=self.k_max, gate_depth=w.gate_depth, node_threshold=w.node_threshold,
                           ckpt_depth=self.ckpt_depth, ckpt_keep=self.ckpt_keep, ckpt_log_tau=self.ckpt_log_tau,
                           tmpl_offset=self.tmpl_offset, tmpl_parent=self.tmpl_parent, tmpl_rank=self.tmpl_rank,
                           tree_token=self.tree_token, tree_parent=self.tree_parent, tree_pos=self.tree_pos,
                                   tree_src=self.tree_src, tree_anc=self.tree_anc, tree_size=self.tree_size)

    def attn(self, variant: int = G.ATTN_AUTO, lse: bool = True) -> None:
        def make():
            K0 = self.Kc if self.Kc.dim() == 4 else self.Kc[0]
            V0 = self.Vc if self.Vc.dim() == 4 else self.Vc[0]
            return G.tree_verify_attn_params(Q=self.Q, Kc=K0, Vc=V0, O=self.O, seq_len=self.seq_len,
                                             tree_size=self.tree_size, tree_anc=self.tree_anc, scale=self.w.scale,
                                             LSE=self.LSE if lse else None, variant=variant)
        key = ("attn", self.Q.data_ptr(), self.Kc.data_ptr(), self.Vc.data_ptr(), variant, lse)
        G.launch("graft_tree_verify_attn", self.ctx, self._cached(key, make))

    def update_adjacency(self, logits: torch.Tensor) -> None:
        """logits: bf16 [B*T_max, V] on the device; refreshes M in place and writes target_next for accept()."""
        key = ("update", logits.data_ptr())
        G.launch("graft_update_adjacency", self.ctx, self._cached(key, lambda: G.update_adjacency_params(
            logits=logits, tree_token=self.tree_token, tree_size=self.tree_size, M=self.M, target_next=self.target_next)))

    def accept(self) -> None:
        G.launch("graft_accept", self.ctx, self._cached("accept", lambda: G.accept_params(
            tree_token=self.tree_token, tree_parent=self.tree_parent, tree_anc=self.tree_anc, tree_size=self.tree_size,
            target_next=self.target_next, n_acc=self.n_acc, path=self.path, best_node=self.best_node, bonus=self.bonus)))

    def accept_stochastic(self, logits: torch.Tensor, temperature: float, u_accept: torch.Tensor, u_bonus: torch.Tensor) -> None:
        """Acceptance under temperature sampling: logits bf16 [B*T_max, V], random numbers float32 [B, T_max] and [B]."""
        need = G.graft_accept_stochastic_scratch_floats(self.w.B, self.w.T_max, logits.shape[1])
        if getattr(self, "row_stats", None) is None or self.row_stats.numel() < need:
            self.row_stats = torch.empty(need, dtype=torch.float32, device=self.dev)
        key = ("accept_s", logits.data_ptr(), u_accept.data_ptr(), u_bonus.data_ptr(), temperature)
        G.launch("graft_accept_stochastic", self.ctx, self._cached(key, lambda: G.accept_stochastic_params(
            logits=logits, temperature=temperature, tree_token=self.tree_token, tree_parent=self.tree_parent,
            tree_size=self.tree_size, u_accept=u_accept, u_bonus=u_bonus, row_stats=self.row_stats, n_acc=self.n_acc,
            path=self.path, best_node=self.best_node, bonus=self.bonus)))

    def compact(self) -> None:
        key = ("compact", self.Kc.data_ptr(), self.Vc.data_ptr())
        G.launch("graft_compact_kv", self.ctx, self._cached(key, lambda: G.compact_kv_params(
            Kc=self.Kc, Vc=self.Vc, seq_len=self.seq_len, n_acc=self.n_acc, path=self.path,
            new_seq_len=self.new_seq_len)))

    def run(self, variant: int = G.ATTN_AUTO) -> None:
        self.build()
        self.attn(variant)
        self.accept()
        self.compact()

    # ---- host views -----------------------------------------------------------------------------
    def tree_host(self) -> Dict[str, np.ndarray]:
        return dict(tree_token=self.tree_token.cpu().numpy(), tree_parent=self.tree_parent.cpu().numpy(),
                    tree_pos=self.tree_pos.cpu().numpy(), tree_src=self.tree_src.cpu().numpy(),
                    tree_anc=self.tree_anc.cpu().numpy().view(np.uint64), tree_size=self.tree_size.cpu().numpy())

    def accept_host(self) -> Dict[str, np.ndarray]:
        return dict(n_acc=self.n_acc.cpu().numpy(), path=self.path.cpu().numpy(),
                    best_node=self.best_node.cpu().numpy(), bonus=self.bonus.cpu().numpy())
