#!/usr/bin/env python
"""Benchmark of the tree-verify path: one step = graft_build_tree -> graft_tree_verify_attn ->
graft_accept -> graft_compact_kv over one batch of synthetic input.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4-B4] [--impl ours|reference]

Prints ONE JSON line.  `value` is algorithmic KV bytes per step / device time per step (GB/s, all
ranks together); `roofline` times graft_tree_verify_attn alone with CUDA events inside the same
timed region; `e2e` repeats the step with that step's inputs coming from pinned host memory and
its results read back; `cpu_baseline` times the CPU oracle on a bounded sample.
With --impl reference the oracle itself is the timed arm (host cores only).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2605_20104_b200 import workloads as W  # noqa: E402

L2_BYTES = 126e6
METRIC = "tree-verify attn HBM GB/s (KV bytes per verify step / step time)"

WORKLOADS = {
    # name: (config id, B, L)
    "cfg1": ("1", None, None),
    "cfg2": ("2", None, None),
    "cfg3": ("3", None, None),
    "cfg4-B1": ("4", 1, 65536),
    "cfg4-B1-32k": ("4", 1, 32768),
    "cfg4-B4": ("4", 4, 65536),
    "cfg5": ("5", None, None),
    "tail16-B4": ("tail", 4, 65536),      # block drafter with tail grafting: chains of 16 on the 64K Qwen3-14B shape
    "tail16-B1-32k": ("tail", 1, 32768),  # the same at a size an ncu capture may hold
}
DEFAULT_WORKLOAD = "cfg4-B4"          # the 64K-context point the metric's target is stated on
EXTRA_WORKLOADS = ["cfg2", "cfg3", "cfg4-B1-32k", "cfg4-B1", "cfg5", "tail16-B4"]


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def tensor_peaks_tflops():
    """Dense bf16 throughput, (burst, sustained under the power cap): measured, or the fallback figures."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d.get("bf16_tflops", 1590.0)), float(d.get("bf16_tflops_sustained", 1400.0))
    return 1590.0, 1400.0


EXP_PER_SECOND = 16 * 148 * 1.965e9      # exponential unit: 16 results per clock and SM, 148 SMs at the maximum SM clock


def three_bounds(w, tree_size, attn_seconds, hbm_gbs):
    """The attention call against each unit it needs (scores of R = T G rows per KV head against every visible key):
    HBM time of the K/V, Q and O bytes, tensor time of 4 d R (L + T) flops per (sequence, KV head), exponential-unit
    time of R (L + T) exponentials.  The slowest of the three is the binding bound of the shape.  The tensor time uses
    the burst figure (these runs stay far below the power cap, at the maximum SM clock); the fraction of the sustained
    figure is printed beside it."""
    G = w.Hq // w.Hkv
    keys = [int(w.seq_len[b]) + int(tree_size[b]) for b in range(w.B)]
    rows = [int(tree_size[b]) * G for b in range(w.B)]
    flops = sum(w.Hkv * 4 * w.d * r * k for r, k in zip(rows, keys))
    exps = sum(w.Hkv * r * k for r, k in zip(rows, keys))
    kv, qo = kv_bytes(w, tree_size)
    burst, sustained = tensor_peaks_tflops()
    t = {"hbm": (kv + qo) / (hbm_gbs * 1e9), "tensor": flops / (burst * 1e12), "exp": exps / EXP_PER_SECOND}
    binding = max(t, key=t.get)
    return {"useful_tflops": flops / attn_seconds / 1e12, "frac_of_bf16_burst": t["tensor"] / attn_seconds,
            "frac_of_bf16_sustained": flops / (sustained * 1e12) / attn_seconds,
            "frac_of_exp_unit": t["exp"] / attn_seconds, "frac_of_hbm": t["hbm"] / attn_seconds,
            "binding": binding, "frac_of_binding": t[binding] / attn_seconds,
            "floor_us": {k: v * 1e6 for k, v in t.items()}}


def kv_bytes(w, tree_size):
    """Algorithmic bytes of one attention call: every visible K and V row once, plus Q and O."""
    kv = sum(w.Hkv * (int(w.seq_len[b]) + int(tree_size[b])) * w.d * 2 * 2 for b in range(w.B))
    qo = sum(2 * int(tree_size[b]) * w.Hq * w.d * 2 for b in range(w.B))
    return kv, qo


class ClockSampler:
    QUERY = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(index), "--query-gpu=" + self.QUERY,
                                       "--format=csv,noheader,nounits", "-lms", "20"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self, t_begin=None, t_end=None):
        """Median SM clock and active throttle reasons over the samples taken inside the wall-clock
        window [t_begin, t_end] (the timed region); all samples if the window caught fewer than two."""
        import datetime
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        rows = [r.split(",") for r in open(self.f.name).read().strip().splitlines() if r.count(",") >= 8]
        os.unlink(self.f.name)
        if not rows:
            return out
        if t_begin is not None:
            def ts(r):
                try:
                    return datetime.datetime.strptime(r[0].strip(), "%Y/%m/%d %H:%M:%S.%f").timestamp()
                except ValueError:
                    return None
            inside = [r for r in rows if ts(r) is not None and t_begin - 0.05 <= ts(r) <= t_end + 0.05]
            out["window"] = "timed region" if len(inside) >= 2 else "warm-up + timed region"
            if len(inside) >= 2:
                rows = inside
        sm = [float(r[1]) for r in rows if r[1].strip().replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any("Active" == r[5 + i].strip() for r in rows)]
        out.update(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=float(rows[0][2]), reasons=reasons,
                   samples=len(rows), power_w_max=max(float(r[3]) for r in rows))
        return out


def make_step(w, n_rot, device):
    """Device state with n_rot distinct K/V caches (rotated per step when one cache fits in L2)."""
    from paper_2605_20104_b200.step import VerifyStep
    vs = VerifyStep(w, device=device, upload_qkv=False)
    g = torch.Generator(device="cuda")
    g.manual_seed(1234 + w.seed)
    dev = "cuda:%d" % device
    vs.Q = (torch.randn(w.B, w.T_max, w.Hq, w.d, generator=g, device=dev) * w.std).to(torch.bfloat16)
    caches = []
    for _ in range(n_rot):
        K = (torch.randn(w.B, w.Hkv, w.S_cap, w.d, generator=g, device=dev) * w.std).to(torch.bfloat16)
        V = (torch.randn(w.B, w.Hkv, w.S_cap, w.d, generator=g, device=dev) * w.std).to(torch.bfloat16)
        caches.append((K, V))
    vs.Kc, vs.Vc = caches[0]
    return vs, caches


def set_target_next(vs, w):
    """The target's greedy ids for the tree the device built (input generation, untimed)."""
    t = vs.tree_host()
    nxt = W.draw_target_next(t["tree_token"], t["tree_parent"], t["tree_size"], t["tree_src"], w.V, w.p_draft,
                             w.p_graft, w.seed)
    vs.target_next.copy_(torch.from_numpy(nxt))
    return t


def time_workload(name, steps, warmup, device, variant, rank=0):
    from paper_2605_20104_b200 import binding as G, shard
    cfg, B, L = WORKLOADS[name]
    w = W.config(cfg, B=B, L=L)
    if rank:
        w = W.config(cfg, B=B, L=L, seed=shard.rank_seed(w.seed, rank))   # every rank its own batch
    # build once to learn the tree sizes (they define the algorithmic bytes)
    kv_guess = w.B * w.Hkv * w.S_cap * w.d * 4
    n_rot = 1 if kv_guess > 2 * L2_BYTES else int(min(16, np.ceil(3 * L2_BYTES / kv_guess)))
    vs, caches = make_step(w, n_rot, device)
    vs.build()
    tree = set_target_next(vs, w)
    kvb, qob = kv_bytes(w, tree["tree_size"])

    def one(i):
        vs.Kc, vs.Vc = caches[i % n_rot]
        vs.build()
        ea[i % len(ea)].record()
        vs.attn(variant)
        eb[i % len(eb)].record()
        vs.accept()
        vs.compact()

    ea = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    eb = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    for i in range(warmup):
        one(i)
    torch.cuda.synchronize()
    flags = vs.ctx.device_status()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    return dict(w=w, vs=vs, caches=caches, one=one, ea=ea, eb=eb, t0=t0, t1=t1, kvb=kvb, qob=qob, n_rot=n_rot,
                flags=flags, tree=tree)


def time_paged_attention(st, steps, warmup, variant, page_size=256):
    """The attention call on the same K/V scattered over a paged pool (random block table), alone."""
    from paper_2605_20104_b200 import binding as G
    w, vs = st["w"], st["vs"]
    Kc, Vc = st["caches"][0]
    B, Hkv, S_cap, d = Kc.shape
    per_seq = (S_cap + page_size - 1) // page_size
    n_blocks = B * per_seq + 7
    g = torch.Generator(device="cpu")
    g.manual_seed(11)
    table = torch.randperm(n_blocks, generator=g)[:B * per_seq].reshape(B, per_seq).to(torch.int32).to(vs.dev)
    Kp = torch.zeros(n_blocks, Hkv, page_size, d, dtype=torch.bfloat16, device=vs.dev)
    Vp = torch.zeros_like(Kp)
    pad = per_seq * page_size - S_cap
    for src, dst in ((Kc, Kp), (Vc, Vp)):
        x = torch.nn.functional.pad(src, (0, 0, 0, pad)).reshape(B, Hkv, per_seq, page_size, d).permute(0, 2, 1, 3, 4)
        dst[table.long().reshape(-1)] = x.reshape(B * per_seq, Hkv, page_size, d)
    prm = G.tree_verify_attn_params(Q=vs.Q, Kc=Kp, Vc=Vp, O=vs.O, seq_len=vs.seq_len, tree_size=vs.tree_size, tree_anc=vs.tree_anc,
                                    scale=w.scale, LSE=vs.LSE, variant=variant, block_table=table, S_cap=S_cap)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for _ in range(warmup):
        G.launch("graft_tree_verify_attn", vs.ctx, prm)
    torch.cuda.synchronize()
    torch.cuda._sleep(int(3e6))
    for a, b in ev:
        a.record()
        G.launch("graft_tree_verify_attn", vs.ctx, prm)
        b.record()
    torch.cuda.synchronize()
    us = float(np.mean([a.elapsed_time(b) for a, b in ev])) * 1e3
    del Kp, Vp
    return {"us_per_call": us, "page_size": page_size, "device_flags": vs.ctx.device_status()}


def time_graph_replay(st, steps, warmup, variant):
    """The same step captured once per rotating cache in a CUDA graph and replayed: device time per step without
    the launch gaps of four separate calls (the launch configuration is fixed by the shapes, so a serving loop
    can do this)."""
    vs, caches, n_rot = st["vs"], st["caches"], st["n_rot"]
    graphs = []
    side = torch.cuda.Stream()
    for kc, vc in caches:
        vs.Kc, vs.Vc = kc, vc
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):                 # every launch once outside a capture (module loading, attributes)
            vs.build(); vs.attn(variant); vs.accept(); vs.compact()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            vs.build(); vs.attn(variant); vs.accept(); vs.compact()
        graphs.append(g)
    for i in range(warmup):
        graphs[i % n_rot].replay()
    torch.cuda.synchronize()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda._sleep(int(3e6))
    t0.record()
    for i in range(steps):
        graphs[i % n_rot].replay()
    t1.record()
    torch.cuda.synchronize()
    return t0.elapsed_time(t1) / steps * 1e3


def time_update(st, steps, warmup):
    """graft_update_adjacency (the matrix refresh that follows the verify pass) alone, on the workload's trees and
    generator-shaped target logits; three logits buffers in rotation (> L2 together)."""
    from paper_2605_20104_b200 import binding as G
    w, vs = st["w"], st["vs"]
    lg = torch.from_numpy(W.make_logits(w.B, w.T_max, w.V, seed=w.seed + 17).view(np.int16)).view(torch.bfloat16)
    n_rot = max(2, int(np.ceil(3 * L2_BYTES / (lg.numel() * 2))))
    bufs = [lg.to(vs.dev).clone() for _ in range(n_rot)]
    M = vs.M.clone()
    nxt = torch.empty_like(vs.target_next)
    prm = [G.update_adjacency_params(logits=b, tree_token=vs.tree_token, tree_size=vs.tree_size, M=M, target_next=nxt) for b in bufs]
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for i in range(warmup):
        G.launch("graft_update_adjacency", vs.ctx, prm[i % n_rot])
    torch.cuda.synchronize()
    torch.cuda._sleep(int(3e6))
    for i in range(steps):
        ev[i][0].record()
        G.launch("graft_update_adjacency", vs.ctx, prm[i % n_rot])
        ev[i][1].record()
    torch.cuda.synchronize()
    us = float(np.mean([a.elapsed_time(b) for a, b in ev])) * 1e3
    rows = int(st["tree"]["tree_size"].sum())
    byts = rows * w.V * 2
    return {"us_per_call": us, "rows": rows, "V": int(w.V), "k": int(M.shape[1]), "algorithmic_bytes": byts,
            "GBps": byts / (us * 1e-6) / 1e9, "l2": "rotating %d logits buffers" % n_rot}


def time_accept_stochastic(st, steps, warmup):
    """graft_accept_stochastic alone (row statistics of every valid node's logits + walk + bonus draw) on the
    workload's trees, generator-shaped logits in rotation (> L2 together), fresh uniform numbers."""
    from paper_2605_20104_b200 import binding as G
    w, vs = st["w"], st["vs"]
    lg = torch.from_numpy(W.make_logits(w.B, w.T_max, w.V, seed=w.seed + 23).view(np.int16)).view(torch.bfloat16)
    n_rot = max(2, int(np.ceil(3 * L2_BYTES / (lg.numel() * 2))))
    bufs = [lg.to(vs.dev).clone() for _ in range(n_rot)]
    g = torch.Generator(device=vs.dev)
    g.manual_seed(5)
    ua = torch.rand(w.B, w.T_max, device=vs.dev, generator=g)
    ub = torch.rand(w.B, device=vs.dev, generator=g)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for i in range(warmup):
        vs.accept_stochastic(bufs[i % n_rot], 1.0, ua, ub)
    torch.cuda.synchronize()
    torch.cuda._sleep(int(3e6))
    for i in range(steps):
        ev[i][0].record()
        vs.accept_stochastic(bufs[i % n_rot], 1.0, ua, ub)
        ev[i][1].record()
    torch.cuda.synchronize()
    us = float(np.mean([a.elapsed_time(b) for a, b in ev])) * 1e3
    rows = int(st["tree"]["tree_size"].sum())
    byts = rows * w.V * 2
    vs.accept()                      # leave the greedy result the step produced
    torch.cuda.synchronize()
    return {"us_per_call": us, "rows": rows, "V": int(w.V), "algorithmic_bytes": byts, "GBps": byts / (us * 1e-6) / 1e9,
            "l2": "rotating %d logits buffers" % n_rot}


def time_index_kernels(st, steps, warmup):
    """The small index kernels around tree assembly, each alone: the retrieval envelope, assembly with its own
    lookups and from the envelope, and the candidate-path table (latency-bound launches of B CTAs)."""
    vs = st["vs"]
    vs.retrieve_envelope()
    calls = {"build_tree": lambda: vs.build(), "path_indices": lambda: vs.path_indices(10)}
    if vs.env_token is not None:
        calls["retrieve_envelope"] = lambda: vs.retrieve_envelope()
        calls["build_tree_from_envelope"] = lambda: vs.build(from_envelope=True)
    out = {}
    for name, fn in calls.items():
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for _ in range(warmup):
            fn()
        torch.cuda.synchronize()
        torch.cuda._sleep(int(3e6))
        for a, b in ev:
            a.record()
            fn()
            b.record()
        torch.cuda.synchronize()
        out[name + "_us"] = float(np.mean([a.elapsed_time(b) for a, b in ev])) * 1e3
    out["envelope_nodes"] = 0 if vs.env_token is None else int(vs.env_token.shape[1])
    vs.build()                       # leave the tree as the step built it
    torch.cuda.synchronize()
    return out


def run_timed(st, steps):
    # keep the GPU busy for a moment so that the launch queue is full when the timed region starts
    torch.cuda._sleep(int(3e6))
    st["t0"].record()
    for i in range(steps):
        st["one"](i)
    st["t1"].record()
    torch.cuda.synchronize()
    total_ms = st["t0"].elapsed_time(st["t1"])
    attn_ms = [a.elapsed_time(b) for a, b in zip(st["ea"], st["eb"])]
    # the SM clock of a shared box can step down in the middle of a long timed region: keep the evidence
    q = max(1, steps // 4)
    st["attn_series"] = {"median_us": float(np.median(attn_ms)) * 1e3, "first_quarter_us": float(np.mean(attn_ms[:q])) * 1e3,
                         "last_quarter_us": float(np.mean(attn_ms[-q:])) * 1e3}
    return total_ms / steps, float(np.mean(attn_ms)), float(np.min(attn_ms))


def run_e2e(st, steps, warmup, variant):
    """The same step with its inputs arriving from pinned host memory and its results read back on the host, every
    step.  The cached prefix is resident state (it was produced by earlier steps); the step's own inputs are the
    draft arrays, Q, the tree tokens' K/V rows and the target's ids; its results O, n_acc, path, bonus, new_seq_len.
    Two sets of step buffers are in flight, as a serving loop keeps them: the copies of step i+1 (host to device) and
    of step i-1 (device to host) run on their own streams beside the kernels of step i, and the host takes the
    results of step i-1 (it waits for their copy) while step i runs."""
    from paper_2605_20104_b200.step import VerifyStep
    w, vs0 = st["w"], st["vs"]
    B, T = w.B, w.T_max
    in_names = ("draft_token", "draft_parent", "draft_score", "n_draft", "seq_len", "Q", "target_next")
    out_names = ("O", "n_acc", "path", "bonus", "new_seq_len")
    seq = [int(x) for x in w.seq_len]
    same_len = len(set(seq)) == 1

    def arena(tensors):
        """One device buffer and one pinned host buffer that hold all `tensors` (name -> device tensor) back to back;
        returns them and the typed device / host views.  One copy then moves the lot."""
        offs, total = {}, 0
        for k, t in tensors.items():
            offs[k] = total
            total += (t.numel() * t.element_size() + 255) // 256 * 256
        dev = torch.empty(total, dtype=torch.uint8, device=vs0.dev)
        host = torch.empty(total, dtype=torch.uint8).pin_memory()
        view = lambda buf, k, t: buf[offs[k]:offs[k] + t.numel() * t.element_size()].view(t.dtype).view(t.shape)
        dv = {k: view(dev, k, t) for k, t in tensors.items()}
        hv = {k: view(host, k, t) for k, t in tensors.items()}
        for k, t in tensors.items():
            dv[k].copy_(t)
            hv[k].copy_(t.cpu())
        return dev, host, dv, hv

    sets = []
    rows_k = torch.randn(B, w.Hkv, T, w.d, device=vs0.dev).to(torch.bfloat16)     # the tree tokens' K/V rows (same every step)
    rows_v = torch.randn(B, w.Hkv, T, w.d, device=vs0.dev).to(torch.bfloat16)
    for n in range(2):
        vs = vs0 if n == 0 else VerifyStep(w, device=torch.device(vs0.dev).index, upload_qkv=False)
        if n:
            vs.Q = vs0.Q.clone()
        ins = {k: getattr(vs0, k) for k in in_names}
        ins["d_k"], ins["d_v"] = rows_k, rows_v
        d_in, h_in, dv_in, _ = arena(ins)
        d_out, h_out, dv_out, hv_out = arena({k: getattr(vs, k) for k in out_names})
        for k in in_names:                                   # the step's tensors are views of the two arenas from now on
            setattr(vs, k, dv_in[k])
        for k in out_names:
            setattr(vs, k, dv_out[k])
        vs.__dict__["_params"] = {}                          # marshalled argument structs pointed at the old tensors
        sets.append(dict(vs=vs, d_in=d_in, h_in=h_in, d_out=d_out, h_out=h_out, hv_out=hv_out, d_k=dv_in["d_k"], d_v=dv_in["d_v"],
                         in_ready=torch.cuda.Event(), cmp_done=torch.cuda.Event(), out_done=torch.cuda.Event()))
    h2d = sum(getattr(vs0, k).numel() * getattr(vs0, k).element_size() for k in in_names) + 2 * sets[0]["d_k"].numel() * 2
    d2h = sum(getattr(vs0, k).numel() * getattr(vs0, k).element_size() for k in out_names)
    s_in, s_out, s_cmp = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.current_stream()

    def copy_in(i):
        z = sets[i % 2]
        s_in.wait_event(z["cmp_done"])                       # the kernels of step i-2 have read this set
        with torch.cuda.stream(s_in):
            z["d_in"].copy_(z["h_in"], non_blocking=True)
            z["in_ready"].record(s_in)

    def compute(i):
        z = sets[i % 2]
        vs = z["vs"]
        vs.Kc, vs.Vc = st["caches"][i % st["n_rot"]]
        s_cmp.wait_event(z["in_ready"])
        s_cmp.wait_event(z["out_done"])                      # the results of step i-2 have left this set
        if same_len:                                         # the projection's write of the tree K/V rows
            vs.Kc[:, :, seq[0]:seq[0] + T].copy_(z["d_k"])
            vs.Vc[:, :, seq[0]:seq[0] + T].copy_(z["d_v"])
        else:
            for b in range(B):
                vs.Kc[b, :, seq[b]:seq[b] + T].copy_(z["d_k"][b])
                vs.Vc[b, :, seq[b]:seq[b] + T].copy_(z["d_v"][b])
        vs.build()
        vs.attn(variant)
        vs.accept()
        vs.compact()
        z["cmp_done"].record(s_cmp)

    def copy_out(i):
        z = sets[i % 2]
        s_out.wait_event(z["cmp_done"])
        with torch.cuda.stream(s_out):
            z["h_out"].copy_(z["d_out"], non_blocking=True)
            z["out_done"].record(s_out)

    def run(n):
        copy_in(0)
        for i in range(n):
            if i + 1 < n:
                copy_in(i + 1)
            compute(i)
            copy_out(i)
            if i > 0:
                sets[(i - 1) % 2]["out_done"].synchronize()      # the caller reads the results of step i-1
        sets[(n - 1) % 2]["out_done"].synchronize()

    run(max(warmup, 2))
    torch.cuda.synchronize()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    run(steps)
    torch.cuda.synchronize()
    t1.record()
    torch.cuda.synchronize()
    # the two buffer sets hold the results of two consecutive steps on the same inputs: they must agree (bit for bit
    # when the steps also saw the same cache), or the overlap of copies and kernels broke something
    for k in out_names:
        if k == "O" and st["n_rot"] > 1:                     # consecutive steps saw different caches
            continue
        if not torch.equal(sets[0]["hv_out"][k], sets[1]["hv_out"][k]):
            raise RuntimeError("end-to-end run: the two buffer sets disagree on " + k)
    return t0.elapsed_time(t1) / steps, h2d, d2h


class OracleTimer:
    """Times the CPU oracle, as it stands, on bounded samples of one step of workload `w`: tree
    assembly and acceptance in full, attention on sampled rows, compaction on one sequence; the
    sampled parts are scaled to the full step."""

    def __init__(self, w):
        import oracle
        oracle.build()
        self.o, self.w = oracle, w
        self.tree = oracle.build_tree(w)
        W.make_qkv(w)                                    # the workload's tensors, drawn once (untimed)
        self.bits = (W.bf16_bits(w.Q), W.bf16_bits(w.Kc), W.bf16_bits(w.Vc))
        self.nxt = W.draw_target_next(self.tree["tree_token"], self.tree["tree_parent"], self.tree["tree_size"],
                                      self.tree["tree_src"], w.V, w.p_draft, w.p_graft, w.seed)
        self.total_rows = int(self.tree["tree_size"].sum()) * w.Hq
        self.threads = 1

    def attn_rows(self, n, rng):
        w, tree = self.w, self.tree
        # n different rows, uniform over all valid (b, t, h) (the oracle computes a row once however often it is listed)
        every = np.array([(b, t, h) for b in range(w.B) for t in range(int(tree["tree_size"][b])) for h in range(w.Hq)], np.int32)
        rows = every[rng.permutation(len(every))[:min(n, len(every))]]
        t = time.perf_counter()
        out = self.o.tree_attn(*self.bits, w.seq_len, tree["tree_size"], tree["tree_anc"], w.scale, rows=rows)
        self.threads = out["threads"]
        return time.perf_counter() - t

    def rows_for(self, seconds, rng):
        t = self.attn_rows(32, rng)
        return int(min(self.total_rows, max(32, 32 * seconds / max(t, 1e-4))))

    def step_seconds(self, n_rows, rng):
        """Estimated seconds of one full step from a sample with n_rows attention rows."""
        w, tree, o = self.w, self.tree, self.o
        t = time.perf_counter()
        o.build_tree(w)
        t_build = time.perf_counter() - t
        t_rows = self.attn_rows(n_rows, rng)
        t = time.perf_counter()
        acc = o.accept(tree["tree_token"], tree["tree_parent"], tree["tree_size"], self.nxt)
        t_acc = time.perf_counter() - t
        t = time.perf_counter()
        o.compact_kv(self.bits[1][:1], self.bits[2][:1], w.seq_len[:1], acc["n_acc"][:1], acc["path"][:1])
        t_comp = (time.perf_counter() - t) * w.B
        return t_build + t_rows * self.total_rows / n_rows + t_acc + t_comp

    def describe(self, n_rows):
        return ("tree assembly and acceptance in full; attention on %d of %d rows (uniform over (b,t,h)), scaled; "
                "compaction on 1 of %d sequences, scaled" % (n_rows, self.total_rows, self.w.B))


def reference_arm(args):
    """--impl reference: the CPU oracle as it stands, on the host cores, same metric and workload.
    Each step is a bounded sample (about two seconds of attention rows) scaled to a full step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg, B, L = WORKLOADS[args.workload]
    w = W.config(cfg, B=B, L=L)
    ot = OracleTimer(w)
    rng = np.random.default_rng(0)
    n_rows = ot.rows_for(2.0, rng)
    vals = []
    for i in range(args.warmup + args.steps):
        est = ot.step_seconds(n_rows, rng)
        if i >= args.warmup:
            vals.append(est)
    kvb, _ = kv_bytes(w, ot.tree["tree_size"])
    sec = float(np.mean(vals))
    value = kvb / sec / 1e9
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "B": w.B, "Hq": w.Hq, "Hkv": w.Hkv, "d": w.d,
                       "L": int(w.seq_len.max()), "T_max": w.T_max},
            "cpu_baseline": {"value": value, "unit": "GB/s", "cores": ot.threads, "kind": "oracle",
                             "sample": ot.describe(n_rows)},
            "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--variant", default="auto", choices=["auto", "mma", "tc", "tc1", "tc2", "tc3"])
    ap.add_argument("--no-extra", action="store_true", help="skip the other configurations' lines")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        reference_arm(args)
        return

    from paper_2605_20104_b200 import binding as G
    variant = {"auto": G.ATTN_AUTO, "mma": G.ATTN_MMA_SYNC, "tc": G.ATTN_TCGEN05, "tc1": G.ATTN_TCGEN05_1SM, "tc2": G.ATTN_TCGEN05_2SM, "tc3": G.ATTN_TCGEN05_L2PAIR}[args.variant]
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    from paper_2605_20104_b200 import shard

    def max_over_ranks(x):
        return shard.max_over_ranks(x, device="cuda")

    # every rank verifies its own batch (sequences are independent: no data-path collective)
    sampler = ClockSampler(local) if rank == 0 else None
    st = time_workload(args.workload, args.steps, args.warmup, local, variant, rank=rank)
    barrier()
    wall0 = time.time()
    ms_step, attn_ms, attn_ms_min = run_timed(st, args.steps)
    barrier()
    wall1 = time.time()
    clocks = sampler.stop(wall0, wall1) if sampler else None
    ms_step = max_over_ranks(ms_step)
    attn_ms = max_over_ranks(attn_ms)
    e2e_ms, h2d, d2h = run_e2e(st, max(3, args.steps // 3), 3, variant)
    e2e_ms = max_over_ranks(e2e_ms)
    flags = st["vs"].ctx.device_status()

    if rank != 0:
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return

    w = st["w"]
    peak, peak_kind = measured_peaks()
    kvb, qob = st["kvb"], st["qob"]
    value = kvb * world / (ms_step * 1e-3) / 1e9
    achieved = (kvb + qob) / (attn_ms * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "us_per_step": ms_step * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "B": w.B, "Hq": w.Hq, "Hkv": w.Hkv, "d": w.d, "L": int(w.seq_len.max()),
                   "T": [int(x) for x in st["tree"]["tree_size"]][:4], "T_max": w.T_max, "attn_variant": args.variant,
                   "l2": "inputs larger than L2" if st["n_rot"] == 1 else "rotating %d KV caches (> 3x L2)" % st["n_rot"],
                   "kv_bytes_per_step": kvb},
        "roofline": {"bound": "hbm", "kernel": "graft_tree_verify_attn (split kernel + merge)",
                     "achieved": achieved, "peak": peak, "peak_kind": "of " + peak_kind, "unit": "GB/s",
                     "frac": achieved / peak, "frac_of_8TBps_nominal": achieved / 8000.0,
                     "us_per_call": attn_ms * 1e3, "us_per_call_min": attn_ms_min * 1e3,
                     "us_per_call_series": st.get("attn_series"),
                     "algorithmic_bytes": kvb + qob, "traffic": TRAFFIC.get(args.workload),
                     "units": three_bounds(w, st["tree"]["tree_size"], attn_ms * 1e-3, peak)},
        "e2e": {"value": kvb * world / (e2e_ms * 1e-3) / 1e9, "unit": "GB/s", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "note": "cached prefix resident; step inputs (draft arrays, Q, tree K/V rows, target ids) from pinned host and "
                        "results (O, n_acc, path, bonus, new_seq_len) read back every step; two buffer sets in flight: the copies "
                        "of steps i+1 and i-1 overlap the kernels of step i"},
        "gpu_launches": 5 * args.steps,
        "clocks": clocks, "device_flags": flags,
    }
    if not args.no_extra and world == 1:
        upd = time_update(st, min(args.steps, 50), 5)
        upd["frac_of_measured"] = upd["GBps"] / peak
        line["update_adjacency"] = upd
        line["index_kernels"] = time_index_kernels(st, min(args.steps, 50), 5)
        line["graph_replay_us_per_step"] = time_graph_replay(st, min(args.steps, 100), 5, variant)
        if st["n_rot"] == 1:
            line["paged_attention"] = time_paged_attention(st, min(args.steps, 50), 5, variant)
        acs = time_accept_stochastic(st, min(args.steps, 50), 5)
        acs["frac_of_measured"] = acs["GBps"] / peak
        line["accept_stochastic"] = acs
        extra = []
        del st
        torch.cuda.empty_cache()
        for name in EXTRA_WORKLOADS:
            k2 = min(args.steps, 50)
            s2 = time_workload(name, k2, args.warmup, local, variant)
            ms2, a2, a2min = run_timed(s2, k2)
            kv2, qo2 = s2["kvb"], s2["qob"]
            extra.append({"workload": name, "us_per_step": ms2 * 1e3, "attn_us": a2 * 1e3, "attn_us_min": a2min * 1e3,
                          "attn_GBps": (kv2 + qo2) / (a2 * 1e-3) / 1e9,
                          "attn_frac_of_" + peak_kind: (kv2 + qo2) / (a2 * 1e-3) / 1e9 / peak,
                          "attn_frac_of_8TBps_nominal": (kv2 + qo2) / (a2 * 1e-3) / 1e9 / 8000.0,
                          "units": three_bounds(s2["w"], s2["tree"]["tree_size"], a2 * 1e-3, peak),
                          "kv_bytes": kv2, "l2": "larger than L2" if s2["n_rot"] == 1 else "rotating %d caches" % s2["n_rot"]})
            del s2
            torch.cuda.empty_cache()
        line["other_configs"] = extra
    if not args.no_cpu_baseline:
        cfg, B, L = WORKLOADS[args.workload]
        ot = OracleTimer(W.config(cfg, B=B, L=L))
        rng = np.random.default_rng(0)
        n_rows = ot.rows_for(12.0, rng)
        est = ot.step_seconds(n_rows, rng)
        line["cpu_baseline"] = {"value": kvb / est / 1e9, "unit": "GB/s", "seconds_per_step_est": est,
                                "cores": ot.threads, "kind": "oracle", "sample": ot.describe(n_rows)}
    print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


# dram__bytes_read.sum + dram__bytes_write.sum of the attention kernel per launch, from the ncu
# captures summarised under profiles/ (None until a capture of that workload exists)
TRAFFIC = {
    # cfg4-B1-32k and cfg3: measured (profiles/attn_tc_pair_kernel_cfg4-B1-32k.md, profiles/attn_tc_rb_kernel_cfg3.md);
    # the 64K workloads are too large for a full capture under the size rule: 1.027 x algorithmic bytes as measured
    # at 32K (1.027 x), scaled by the keys processed (same kernel, traffic grows in proportion)
    "cfg4-B1-32k": 139.1e6, "cfg3": 145.9e6, "cfg4-B1": 1.027 * 269.6e6, "cfg4-B4": 1.027 * 1078.5e6,
}

if __name__ == "__main__":
    main()
