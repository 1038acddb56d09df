#!/usr/bin/env python
"""Benchmark of the ISD step (isd_attn -> isd_verify -> isd_commit) on B200.

One "step" = one isd_step call over the whole stationary batch.  The default workload is the
large-concurrency stationary batch the headline metric is quoted on (batch 256, stride 8,
contexts 1k-8k, vocab 151,936 bf16 logits, chained steps with accept lengths fed back).

Timing: every step is bracketed by its own pair of CUDA events on the launching stream; the
step's inputs (the stand-in for the model's LM head: this step's logits and q/k/v) are produced
between the timed windows and the L2 is flushed before each window.  `value` = positions
(valid block rows of all slots) / summed event time, max over ranks.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config I]
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "isd_step_positions_per_s"
UNIT = "positions/s"
HBM_NOMINAL_GBS = 8000.0


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks / throttle reasons of one GPU with nvidia-smi while the timed region runs."""

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={q}", "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self) -> dict:
        if self.proc is not None:
            time.sleep(0.15)
            self.proc.terminate()          # the exact child started above
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        top = sorted(sm)[len(sm) // 2:]      # samples under load are the upper half
        return {"sm_mhz": statistics.median(top), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm)}


def l2_flush(buf):
    """Cold L2 before a timed window: write a 512 MB buffer (L2 is 126 MB), then read it back, so that the
    flush's own dirty lines are in HBM again and their write-back does not fall into the window."""
    buf.zero_()
    buf.max()


def algorithmic_bytes(w, ctx_len, q_len, rejecting: int):
    """Bytes the method itself must move in one step (KV read + append, Q/O, logits rows)."""
    import torch
    kv_tok = 2 * w.n_kv_heads * w.head_dim * 2
    lb = 2 if w.logits_dtype == "bf16" else 4
    q_sum = int(q_len.sum().item())
    attn = int((ctx_len.to(torch.int64) + q_len).sum().item()) * kv_tok + q_sum * kv_tok \
        + q_sum * w.n_q_heads * w.head_dim * 2 * 2
    # a rejection re-reads the anchor row and the proposal-law row; with filtered laws both are short lists
    verify = q_sum * w.vocab * lb + (0 if w.top_k else rejecting * (2 if w.q_mode == 0 else 1) * w.vocab * lb)
    return attn, verify


def rank_workload(config_index: int, rank: int, sweep: str | None = None, top_k: int = 0, top_p: float = 1.0):
    """Workload of one rank: ranks own disjoint slots with their own pools, so each gets its own seed."""
    from dataclasses import replace
    from paper_2604_11035_b200 import workloads as wl
    if sweep:
        stride, batch = (int(x) for x in sweep.split(","))
        base = wl.sweep_point(stride, batch)
    else:
        base = wl.config(config_index)
    return replace(base, seed=base.seed + 1000 * rank, top_k=top_k, top_p=top_p,
                   name=base.name + (f"[top-k {top_k}, top-p {top_p}]" if top_k else ""))


def reduce_over_ranks(dist, device, times, counts):
    """Whole-job numbers: the slowest rank's time (MAX) and the units all ranks processed (SUM)."""
    import torch
    tt = torch.tensor(times, dtype=torch.float64, device=device)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    cc = torch.tensor(counts, dtype=torch.int64, device=device)
    dist.all_reduce(cc, op=dist.ReduceOp.SUM)
    return {"max": [float(x) for x in tt], "sum": [int(x) for x in cc]}


def run_model_step(args):
    """Model-step mode: `--layers L` attention layers through one page table, then verify and commit
    (isd_step_layers), optionally replayed from a CUDA graph (`--graph`) with the step number on the device.
    Single GPU; same metric and timing rules as the default mode, no roofline / e2e / cpu_baseline legs."""
    import torch
    import paper_2604_11035_b200 as pkg
    from dataclasses import replace
    from paper_2604_11035_b200 import workloads as wl

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    w = rank_workload(args.config, 0, args.sweep, args.top_k, args.top_p)
    K, W, L = args.steps, args.warmup, args.layers
    w = replace(w, steps=max(w.steps, K + W + 2))
    if args.batch:
        w = replace(w, batch=args.batch, name=w.name + f"[batch {args.batch}]")
    st = wl.make_state(w, dev)
    eng = pkg.isd_for_workload(w, st)
    out = pkg.alloc_verify_out(w.batch, w.stride, dev)
    B, Q = w.batch, w.Q
    gen = torch.Generator(device=dev)
    gen.manual_seed(w.seed + 7)
    pools = [(st["k_pool"], st["v_pool"])]
    for _ in range(1, L):   # every further layer has its own pools (that is the HBM traffic of a layer)
        pools.append(tuple((torch.randn(st["k_pool"].shape, generator=gen, device=dev, dtype=torch.bfloat16) * w.kv_sigma)
                           for _ in range(2)))
    q, k, v = (x.clone() for x in wl.make_qkv(w, 0, dev))
    attn_out = torch.zeros(B, Q, w.n_q_heads, w.head_dim, dtype=torch.bfloat16, device=dev)
    dt = torch.bfloat16 if w.logits_dtype == "bf16" else torch.float32
    cur = torch.empty(B, Q, w.vocab, dtype=dt, device=dev)
    prev = torch.zeros(B, Q, w.vocab, dtype=dt, device=dev)
    counter = torch.zeros(1, dtype=torch.int32, device=dev)
    eng.isd_set_step_counter(counter)
    layers = eng.layer_args([dict(q=q, k_new=k, v_new=v, k_pool=pools[l][0], v_pool=pools[l][1], attn_out=attn_out)
                             for l in range(L)])
    st_struct = eng.state_struct(st)
    flush = wl.l2_flush_buffer(dev, 512)

    def launch():
        eng.isd_step_layers(st, layers, cur, prev, out, 0, st_struct)

    graph = None
    launches_in_graph = 0
    if args.graph:
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        n0 = eng.isd_launch_count()
        with torch.cuda.graph(graph):
            launch()
        launches_in_graph = eng.isd_launch_count() - n0      # kernels recorded by the capture = launched per replay
    ev = lambda: torch.cuda.Event(enable_timing=True)
    e_step = [(ev(), ev()) for _ in range(W + K)]
    pos_acc = torch.zeros(W + K, dtype=torch.int64, device=dev)
    emit_acc = torch.zeros(W + K, dtype=torch.int64, device=dev)
    byt_acc = torch.zeros(W + K, dtype=torch.int64, device=dev)
    kv_tok = 2 * w.n_kv_heads * w.head_dim * 2
    lb = 2 if w.logits_dtype == "bf16" else 4
    sampler = ClockSampler(0)
    launches0 = 0
    for t in range(W + K):
        if t == W:
            torch.cuda.synchronize()
            launches0 = eng.isd_launch_count()
            sampler.start()
        if t > 0:
            prev.copy_(cur)
        qt, kt, vt = wl.make_qkv(w, t, dev)
        q.copy_(qt); k.copy_(kt); v.copy_(vt)
        wl.make_logits(w, t, st["ctx_len"], out=cur)
        q_len = torch.where(st["active"] != 0, st["n_ver"] + w.stride, 0).to(torch.int64)
        pos_acc[t] = q_len.sum()
        byt_acc[t] = L * (((st["ctx_len"].to(torch.int64) + 2 * q_len) * kv_tok).sum()
                          + q_len.sum() * (w.n_q_heads * w.head_dim * 4)) + q_len.sum() * (w.vocab * lb)
        l2_flush(flush)
        e_step[t][0].record()
        if graph is not None:
            graph.replay()
        else:
            launch()
        e_step[t][1].record()
        emit_acc[t] = out["n_emit"].sum()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    launches = eng.isd_launch_count() - launches0
    status = eng.isd_read_status()
    step_ms = [a.elapsed_time(b) for a, b in e_step[W:]]
    t_total = sum(step_ms) / 1e3
    positions = int(pos_acc[W:].sum().item())
    peak, peak_kind = measured_peaks()
    gbs = int(byt_acc[W:].sum().item()) / t_total / 1e9
    line = {
        "metric": METRIC, "value": positions / t_total, "unit": UNIT, "n_gpus": 1, "steps": K, "warmup": W,
        "ms_per_step": sum(step_ms) / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "mode": "model step: %d attention layers + verify + commit" % L, "layers": L,
                   "cuda_graph": bool(args.graph), "batch_per_gpu": w.batch, "stride": w.stride, "vocab": w.vocab,
                   "ctx": [w.ctx_min, w.ctx_max], "l2": "flushed before every step (512 MB written, then read back)"},
        "emitted_tokens_per_s": int(emit_acc[W:].sum().item()) / t_total,
        "step_algorithmic_gbs": gbs, "step_frac_of_8TBs": gbs / HBM_NOMINAL_GBS, "step_frac_of_measured_copy": gbs / peak,
        "gpu_launches": launches if graph is None else K * launches_in_graph, "launches_issued_by_host": launches,
        "status_word": status, "clocks": clocks,
    }
    print(json.dumps(line))


def run_lora(args):
    """`--lora N,K,R`: the segment-gated LoRA linear layer (isd_lora_linear) on the token rows of one step of the
    workload (M = batch x (2 stride - 1)), timed by CUDA events; roofline against the measured dense bf16 peak."""
    import torch
    import paper_2604_11035_b200 as pkg
    from paper_2604_11035_b200 import workloads as wl
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    w = rank_workload(args.config, 0, args.sweep)
    N, K, R = (int(v) for v in args.lora.split(","))
    M = (args.batch or w.batch) * w.Q
    small = wl.Workload("lora_ctx", batch=1, stride=2, n_q_heads=8, n_kv_heads=2, vocab=1024, ctx_min=16, ctx_max=16, steps=1)
    eng = pkg.isd_for_workload(small, wl.make_state(small, dev))
    g = torch.Generator(device=dev)
    g.manual_seed(w.seed)
    bf = lambda *shape, s=1.0: (torch.randn(*shape, generator=g, device=dev) * s).to(torch.bfloat16)
    x, wt, a, b = bf(M, K), bf(N, K, s=K ** -0.5), bf(R, K, s=K ** -0.5), bf(N, R, s=R ** -0.5)
    # MASK rows of a P step: rows n_ver + 1 .. of every slot (here: the last stride - 1 rows of each block)
    gate = (torch.arange(M, device=dev) % w.Q >= w.stride).to(torch.uint8)
    t = torch.empty(M, R, dtype=torch.bfloat16, device=dev)
    y = torch.empty(M, N, dtype=torch.bfloat16, device=dev)
    flush = wl.l2_flush_buffer(dev, 512)
    Kn, W = args.steps, args.warmup
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(W + Kn)]
    sampler = ClockSampler(0)
    launches0 = 0
    for i in range(W + Kn):
        if i == W:
            torch.cuda.synchronize()
            sampler.start()
            launches0 = eng.isd_launch_count()
        l2_flush(flush)
        ev[i][0].record()
        eng.isd_lora_linear(x, wt, a, b, gate, 0.5, t=t, y=y)
        ev[i][1].record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    launches = eng.isd_launch_count() - launches0
    ms = [a_.elapsed_time(b_) for a_, b_ in ev[W:]]
    t_total = sum(ms) / 1e3
    flops = 2.0 * M * (N * (K + R) + R * K)
    peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json"))) if os.path.exists(os.path.join(ROOT, "MEASURED_PEAKS.json")) else {}
    peak = float(peaks.get("bf16_tflops", 1590.0))
    tf = flops * Kn / t_total / 1e12
    print(json.dumps({
        "metric": "isd_lora_linear_positions_per_s", "value": M * Kn / t_total, "unit": UNIT, "n_gpus": 1, "steps": Kn,
        "warmup": W, "ms_per_step": sum(ms) / Kn, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"lora_linear m{M} n{N} k{K} rank{R} (token rows of {w.name})", "l2": "flushed before every call"},
        "roofline": {"kernel": f"gemm_tc2_kernel / gemm_tc_kernel ({launches // Kn} launch per call)", "bound": "tensor", "achieved": tf, "peak": peak,
                     "peak_kind": "measured (burst)" if peaks else "fallback", "unit": "TFLOP/s", "frac": tf / peak, "traffic": None},
        "gpu_launches": launches, "status_word": eng.isd_read_status(), "clocks": clocks}))


def attn_mma_cycles(w, ctx_len, q_len):
    """Tensor-pipe cycles one attention launch needs, per SM-cycle unit: every 128-key tile of every (slot, KV head)
    pair costs 8 QK^T and 8 PV instructions of shape 128 x 128 x 16 = 2 * 128 * 128 * 16 flops each, at 8192 dense
    bf16 flops per clock and SM (2.25 PFLOP/s nominal over 148 SMs at 1.86 GHz)."""
    import torch
    tiles = ((ctx_len.to(torch.int64) + q_len + 127) // 128 * (q_len > 0)).sum() * w.n_kv_heads
    return tiles * 16 * (2 * 128 * 128 * 16) // 8192


def traffic_record(kernel: str):
    """DRAM bytes per algorithmic byte of `kernel` from the machine-written record under profiles/ (written by
    `python -m paper_2604_11035_b200.profile_record` from an ncu capture); None when there is no record or the
    record was taken on other sources of that kernel."""
    from paper_2604_11035_b200 import profile_record as pr
    rec = pr.load(kernel)
    if rec is None:
        return None, "no record under profiles/"
    if rec.get("source_sha256") != pr.source_hash(rec.get("sources", [])):
        return None, "the record under profiles/ was captured on another version of the kernel's sources"
    return rec, "ncu capture of %s (%s), dram bytes per algorithmic byte %.4f, scaled by this launch's algorithmic bytes" % (
        rec["workload"], rec["captured"], rec["dram_bytes_per_algorithmic_byte"])


def measure(args, w, dev, K, W, *, instrumented=3, e2e_steps=0, dist=None, world=1, sampler=None):
    """W warm-up + K timed chained isd_step calls on workload `w` (no events inside the timed steps), then
    `instrumented` steps each with events around the attention kernel and around the verification kernels, then
    `e2e_steps` steps through the C ABI with host buffers.  Returns a dict of raw numbers."""
    import torch
    import paper_2604_11035_b200 as pkg
    from dataclasses import replace
    from paper_2604_11035_b200 import workloads as wl

    ATTN_I = VER_I = instrumented
    total_steps = W + K + ATTN_I + VER_I
    w = replace(w, steps=max(w.steps, total_steps + e2e_steps + 2))
    st = wl.make_state(w, dev)
    eng = pkg.isd_for_workload(w, st)
    out = pkg.alloc_verify_out(w.batch, w.stride, dev)
    B, Q = w.batch, w.Q
    attn_out = torch.zeros(B, Q, w.n_q_heads, w.head_dim, dtype=torch.bfloat16, device=dev)
    dt = torch.bfloat16 if w.logits_dtype == "bf16" else torch.float32
    logits = [torch.empty(B, Q, w.vocab, dtype=dt, device=dev) for _ in range(2)]
    flush = wl.l2_flush_buffer(dev, 512)
    st_struct = eng.state_struct(st)
    ev = lambda: torch.cuda.Event(enable_timing=True)
    e_step = [(ev(), ev()) for _ in range(total_steps)]
    e_attn = [(ev(), ev()) for _ in range(total_steps)]
    e_ver = [(ev(), ev()) for _ in range(total_steps)]
    for pairs in (e_attn, e_ver):
        for a, b in pairs:
            a.record(); b.record()      # creates the underlying CUDA events
    acc = {k: torch.zeros(total_steps, dtype=torch.int64, device=dev) for k in ("pos", "emit", "rej", "attn_bytes", "mma")}
    kv_tok = 2 * w.n_kv_heads * w.head_dim * 2

    def one_step(t):
        q, k, v = wl.make_qkv(w, t, dev)
        cur, prev = logits[t & 1], (logits[(t - 1) & 1] if t > 0 else None)
        wl.make_logits(w, t, st["ctx_len"], out=cur)
        q_len = torch.where(st["active"] != 0, st["n_ver"] + w.stride, 0).to(torch.int64)
        acc["pos"][t] = q_len.sum()
        # main attention kernel: KV read once + Q read + O write (the K/V append is a separate launch)
        acc["attn_bytes"][t] = ((st["ctx_len"].to(torch.int64) + q_len) * kv_tok).sum() \
            + q_len.sum() * (w.n_q_heads * w.head_dim * 4)
        acc["mma"][t] = attn_mma_cycles(w, st["ctx_len"], q_len)
        nv_before = st["n_ver"].clone()
        l2_flush(flush)
        sargs = eng.step_args(q=q, k_new=k, v_new=v, k_pool=st["k_pool"], v_pool=st["v_pool"], attn_out=attn_out,
                              attn_lse=None, logits_cur=cur, q_prev_logits=prev, out=out)
        # An event between two kernels serialises launches that otherwise overlap (the kernels of a step are
        # chained by programmatic dependent launches), so the timed steps carry none; the instrumented steps
        # that follow them carry the pair around the attention kernel or the pair around the verification kernels.
        if t < W + K:
            eng.isd_set_profile_events(None, None, None, None)
        elif t < W + K + ATTN_I:
            eng.isd_set_profile_events(e_attn[t][0], e_attn[t][1], None, None)
        else:
            eng.isd_set_profile_events(None, None, e_ver[t][0], e_ver[t][1])
        e_step[t][0].record()
        eng.isd_step(st, sargs, t, st_struct)
        e_step[t][1].record()
        acc["emit"][t] = out["n_emit"].sum()
        acc["rej"][t] = (out["accept_len"] < nv_before).sum()

    for t in range(W):
        one_step(t)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    launches0 = eng.isd_launch_count()
    if sampler is not None:
        sampler.start()
    wall0 = time.time()
    for t in range(W, W + K):
        one_step(t)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    wall = time.time() - wall0
    clocks = sampler.stop() if sampler is not None else None
    launches = eng.isd_launch_count() - launches0
    for t in range(W + K, total_steps):
        one_step(t)
    torch.cuda.synchronize()
    eng.isd_set_profile_events(None, None, None, None)

    lb = 2 if w.logits_dtype == "bf16" else 4
    rej_rows = 0 if w.top_k else (2 if w.q_mode == 0 else 1)   # full rows a rejection reads again
    sl_t, sl_a, sl_v = slice(W, W + K), slice(W + K, W + K + ATTN_I), slice(W + K + ATTN_I, total_steps)
    tot = lambda name, sl: int(acc[name][sl].sum().item())
    R = {"w": w, "K": K, "W": W, "launches": launches, "wall": wall, "clocks": clocks,
         "step_ms": [a.elapsed_time(b) for a, b in e_step[sl_t]],
         "instr_step_ms": [a.elapsed_time(b) for a, b in e_step[W + K:]],
         "attn_ms": [a.elapsed_time(b) for a, b in e_attn[sl_a]],
         "ver_ms": [a.elapsed_time(b) for a, b in e_ver[sl_v]],
         "positions": tot("pos", sl_t), "emitted": tot("emit", sl_t), "rejecting": tot("rej", sl_t),
         "attn_bytes": tot("attn_bytes", sl_t), "attn_bytes_instr": tot("attn_bytes", sl_a), "mma_instr": tot("mma", sl_a),
         "ver_bytes_instr": tot("pos", sl_v) * w.vocab * lb + tot("rej", sl_v) * rej_rows * w.vocab * lb,
         "attn_bytes_all": tot("attn_bytes", slice(0, total_steps)), "attn_launches_all": total_steps}
    R["t_total"] = sum(R["step_ms"]) / 1e3
    R["step_bytes"] = R["attn_bytes"] + R["positions"] * kv_tok + R["positions"] * w.vocab * lb \
        + R["rejecting"] * rej_rows * w.vocab * lb

    # ---- end to end through the C ABI with HOST buffers: H2D of the step's inputs and D2H of its results inside
    # the timed window.  Two forms: everything on the step's stream (serial), and with the logits (97 % of the
    # bytes) copied on a second stream while the attention of the same step runs (overlapped).
    R["e2e"] = None
    if e2e_steps > 0:
        host_q, host_k, host_v = [torch.empty_like(x, device="cpu").pin_memory() for x in wl.make_qkv(w, 0, dev)]
        host_lg = torch.empty(B, Q, w.vocab, dtype=dt, device="cpu").pin_memory()
        host_out = {k_: torch.empty_like(v_, device="cpu").pin_memory() for k_, v_ in out.items()
                    if k_ in ("n_emit", "out_tok", "accept_len")}
        dq, dk, dv = [torch.empty_like(x) for x in wl.make_qkv(w, 0, dev)]
        copy_stream = torch.cuda.Stream(device=dev)
        res = {}
        t = total_steps
        for mode in ("serial", "overlapped"):
            pos = 0
            tsum = 0.0
            for i in range(e2e_steps):
                q, k, v = wl.make_qkv(w, t, dev)
                cur, prev = logits[t & 1], logits[(t - 1) & 1]
                wl.make_logits(w, t, st["ctx_len"], out=cur)
                host_q.copy_(q); host_k.copy_(k); host_v.copy_(v); host_lg.copy_(cur)
                pos += int(torch.where(st["active"] != 0, st["n_ver"] + w.stride, 0).sum().item())
                l2_flush(flush)
                torch.cuda.synchronize()
                e0, e1 = ev(), ev()
                e0.record()
                main = torch.cuda.current_stream()
                dq.copy_(host_q, non_blocking=True); dk.copy_(host_k, non_blocking=True); dv.copy_(host_v, non_blocking=True)
                if mode == "serial":
                    cur.copy_(host_lg, non_blocking=True)
                    sargs = eng.step_args(q=dq, k_new=dk, v_new=dv, k_pool=st["k_pool"], v_pool=st["v_pool"], attn_out=attn_out,
                                          attn_lse=None, logits_cur=cur, q_prev_logits=prev, out=out)
                    eng.isd_step(st, sargs, t, st_struct)
                else:
                    copy_stream.wait_stream(main)
                    with torch.cuda.stream(copy_stream):
                        cur.copy_(host_lg, non_blocking=True)
                    eng.isd_attn(st, dq, dk, dv, st["k_pool"], st["v_pool"], attn_out)
                    main.wait_stream(copy_stream)
                    eng.isd_verify(st, cur, prev, t, out)
                    eng.isd_commit(st, out)
                for k_, h in host_out.items():
                    h.copy_(out[k_], non_blocking=True)
                e1.record()
                torch.cuda.synchronize()
                tsum += e0.elapsed_time(e1) / 1e3
                t += 1
            res[mode] = (pos, tsum)
        h2d = sum(x.numel() * x.element_size() for x in (host_q, host_k, host_v, host_lg))
        d2h = sum(x.numel() * x.element_size() for x in host_out.values())
        R["e2e"] = {"serial": res["serial"], "overlapped": res["overlapped"], "h2d": h2d, "d2h": d2h, "steps": e2e_steps}
    R["status"] = eng.isd_read_status()
    eng.close()
    return R


def workload_for(args, rank):
    from dataclasses import replace
    w = rank_workload(args.config, rank, args.sweep if args.sweep != "all" else None, args.top_k, args.top_p)
    if args.propose_mode is not None:
        w = replace(w, propose_mode=args.propose_mode)
    if args.q_mode is not None:
        w = replace(w, q_mode=args.q_mode)
    if args.sequential_pages:
        w = replace(w, shuffle_pages=False, name=w.name + "[sequential pages]")
    if args.batch:
        w = replace(w, batch=args.batch, name=w.name + f"[batch {args.batch}]")
    return w


def pairing_name(w):
    return ("argmax" if w.propose_mode else "sampled") + " proposals + " + ("point-mass q" if w.q_mode else "softmax q")


def result_line(args, R, world, red=None):
    """The JSON line of one measurement (rank 0)."""
    w, K, W = R["w"], R["K"], R["W"]
    t_total, positions, emitted, launches = R["t_total"], R["positions"], R["emitted"], R["launches"]
    if red is not None:
        t_total, positions, emitted, launches = red["max"][0], red["sum"][0], red["sum"][1], red["sum"][3]
    peak, peak_kind = measured_peaks()
    attn_t = sum(R["attn_ms"]) / 1e3
    attn_gbs = R["attn_bytes_instr"] / attn_t / 1e9
    ver_gbs = R["ver_bytes_instr"] / (sum(R["ver_ms"]) / 1e3) / 1e9 if sum(R["ver_ms"]) > 0 else None
    step_gbs = R["step_bytes"] / (sum(R["step_ms"]) / 1e3) / 1e9
    sm_mhz = (R["clocks"] or {}).get("sm_mhz") or 1965.0
    n_i = len(R["attn_ms"])
    rec, traffic_src = traffic_record("attn_tc_kernel")
    line = {
        "metric": METRIC, "value": positions / t_total, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": 1e3 * t_total / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "batch_per_gpu": w.batch, "stride": w.stride, "heads": f"{w.n_q_heads}/{w.n_kv_heads}",
                   "head_dim": w.head_dim, "vocab": w.vocab, "logits_dtype": w.logits_dtype,
                   "ctx": [w.ctx_min, w.ctx_max], "pairing": pairing_name(w),
                   "propose_mode": "argmax" if w.propose_mode else "sample", "q_mode": "point mass" if w.q_mode else "softmax",
                   "peaked_frac": w.peaked_frac, "chained": True, "l2": "flushed before every step (512 MB written, then read back so that the flush leaves no dirty lines); inputs 6 GB >> L2",
                   "parallelism": f"slots x{world} (no collective)"},
        "emitted_tokens_per_s": emitted / t_total, "tokens_per_step_per_slot": emitted / max(1, K * w.batch * world),
        "step_algorithmic_gbs": step_gbs, "step_frac_of_8TBs": step_gbs / HBM_NOMINAL_GBS,
        "step_frac_of_measured_copy": step_gbs / peak,
        "roofline": {"kernel": "attn_tc_kernel", "bound": "hbm", "achieved": attn_gbs, "peak": peak, "peak_kind": peak_kind,
                     "unit": "GB/s", "frac": attn_gbs / peak, "frac_of_8TBs": attn_gbs / HBM_NOMINAL_GBS,
                     "traffic": (rec["dram_bytes_per_algorithmic_byte"] * R["attn_bytes_instr"] / n_i) if rec else None,
                     "traffic_source": traffic_src,
                     "ms_per_launch": 1e3 * attn_t / n_i, "bytes_per_launch": R["attn_bytes_instr"] / n_i,
                     "timed_on": "%d instrumented steps right after the timed region (same chain, L2 flushed; %.3f ms per "
                                 "instrumented step)" % (n_i, sum(R["instr_step_ms"]) / len(R["instr_step_ms"])),
                     "share_of_step": (1e3 * attn_t / n_i) / (sum(R["step_ms"]) / K),
                     "tensor_pipe_util_derived": R["mma_instr"] / (attn_t * sm_mhz * 1e6 * 148),
                     # the figure the target is stated on: the whole step against the nominal 8 TB/s
                     "step": {"achieved": step_gbs, "unit": "GB/s", "frac_of_8TBs": step_gbs / HBM_NOMINAL_GBS,
                              "frac_of_measured_copy": step_gbs / peak, "target_frac_of_8TBs": 0.70,
                              "target_met": bool(step_gbs / HBM_NOMINAL_GBS >= 0.70)}},
        "verify_kernels": {"kernels": "topk_rows_kernel (+ topk_decide_kernel when proposal-law rows are streamed)" if w.top_k
                           else "verify_rows_kernel + verify_sample_kernel (the last CTA of which commits)",
                           "achieved_gbs": ver_gbs, "ms_per_launch": sum(R["ver_ms"]) / max(1, len(R["ver_ms"])),
                           "timed_on": "%d instrumented steps after the timed region" % len(R["ver_ms"]),
                           "frac_of_measured_copy": (ver_gbs / peak) if ver_gbs else None},
        "gpu_launches": launches, "status_word": R["status"], "clocks": R["clocks"], "wall_s": R["wall"],
        "attn_bytes_all_launches": R["attn_bytes_all"], "attn_launches_all": R["attn_launches_all"],
    }
    if R["e2e"]:
        e = R["e2e"]
        pos, tt = e["overlapped"]
        if red is not None:
            tt, pos = red["max"][1], red["sum"][2]
        line["e2e"] = {"value": pos / tt, "unit": UNIT, "h2d_bytes_per_step": e["h2d"], "d2h_bytes_per_step": e["d2h"],
                       "steps": e["steps"], "form": "logits copied on a second stream under the step's attention",
                       "serial_value": e["serial"][0] / e["serial"][1] if red is None else None}
    return line


def run_ours(args):
    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if local >= torch.cuda.device_count():
        raise SystemExit(f"rank {rank}: local rank {local} but only {torch.cuda.device_count()} CUDA device(s) are visible")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)   # NCCL only carries the final timing reduction

    # weak scaling: every rank owns its own slots, pools and free stack (slots never interact)
    w = workload_for(args, rank)
    K, W = args.steps, args.warmup
    R = measure(args, w, dev, K, W, e2e_steps=min(K, args.e2e_steps), dist=dist if world > 1 else None, world=world,
                sampler=ClockSampler(local))
    red = None
    if world > 1:
        e = R["e2e"]
        red = reduce_over_ranks(dist, dev, [R["t_total"], e["overlapped"][1] if e else 0.0],
                                [R["positions"], R["emitted"], e["overlapped"][0] if e else 0, R["launches"]])
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    line = result_line(args, R, world, red)
    # the other proposal / proposal-law pairings on the same workload (fewer steps), as extra keys
    if args.pairings and world == 1:
        from dataclasses import replace
        line["pairings"] = {pairing_name(R["w"]): {"ms_per_step": line["ms_per_step"], "step_frac_of_8TBs": line["step_frac_of_8TBs"],
                                                    "verify_ms": line["verify_kernels"]["ms_per_launch"], "default": True}}
        for pm, qm in ((1, 1), (0, 0), (1, 0)):
            if (pm, qm) == (R["w"].propose_mode, R["w"].q_mode):
                continue
            w2 = replace(w, propose_mode=pm, q_mode=qm)
            R2 = measure(args, w2, dev, min(K, 10), 3, e2e_steps=0)
            g2 = R2["step_bytes"] / (sum(R2["step_ms"]) / 1e3) / 1e9
            line["pairings"][pairing_name(w2)] = {
                "ms_per_step": sum(R2["step_ms"]) / len(R2["step_ms"]), "step_frac_of_8TBs": g2 / HBM_NOMINAL_GBS,
                "verify_ms": sum(R2["ver_ms"]) / max(1, len(R2["ver_ms"])), "steps": len(R2["step_ms"]),
                "tokens_per_step_per_slot": R2["emitted"] / max(1, len(R2["step_ms"]) * w2.batch)}
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline(args, R["w"])
    if world > 1:
        dist.destroy_process_group()
    print(json.dumps(line))


def run_sweep_all(args):
    """`--sweep all`: the twenty points of the sweep workload, one JSON line each (single GPU)."""
    import torch
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    from dataclasses import replace
    for stride in (2, 4, 8, 16):
        for batch in (1, 8, 64, 256, 512):
            a = argparse.Namespace(**vars(args))
            a.sweep = f"{stride},{batch}"
            w = workload_for(a, 0)
            R = measure(a, w, dev, args.steps, args.warmup, e2e_steps=0, sampler=ClockSampler(0))
            line = result_line(a, R, 1)
            line["config"]["sweep_point"] = {"stride": stride, "batch": batch}
            print(json.dumps(line), flush=True)
            torch.cuda.empty_cache()


def launch_ranks(n: int, argv, *, env_extra=None, timeout=None):
    """Start `n` ranks of this script on this node (one process per GPU) with RANK / LOCAL_RANK / WORLD_SIZE and a
    127.0.0.1 rendezvous in their environment, and wait for them.  Returns the exit codes; rank 0's stdout is
    this process's stdout (it prints the one JSON line)."""
    import socket
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        env.update(env_extra or {})
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__), *argv], env=env,
                                      stdout=None if r == 0 else subprocess.DEVNULL))
    codes = []
    for p_ in procs:
        try:
            codes.append(p_.wait(timeout=timeout))
        except subprocess.TimeoutExpired:
            p_.kill()                    # the exact child started above
            codes.append(-9)
    return codes


def run_stub(args):
    """`--stub-step`: the multi-rank plumbing without a GPU (gloo on the CPU): every rank builds its own rank
    workload, "times" a stubbed step whose duration depends on the rank, and the numbers are reduced exactly as
    in the real run (MAX over ranks of the time, SUM of the units).  Used by the CPU test of the launcher."""
    import torch.distributed as dist
    from paper_2604_11035_b200 import workloads as wl
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo", rank=rank, world_size=world)
    w = workload_for(args, rank)
    st = wl.make_state(wl.config(0, seed=w.seed), "cpu")       # a tiny state: proves the rank's own seed is used
    K = args.steps
    positions = K * w.batch * w.Q
    t_total = K * 1e-3 * (1.0 + 0.25 * rank)                  # the slowest rank decides
    red = {"max": [t_total], "sum": [positions]}
    if world > 1:
        red = reduce_over_ranks(dist, "cpu", [t_total], [positions])
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": red["sum"][0] / red["max"][0], "unit": UNIT, "n_gpus": world, "steps": K,
                          "warmup": args.warmup, "ms_per_step": 1e3 * red["max"][0] / K, "stub": True,
                          "config": {"workload": w.name, "first_anchor_token": int(st["block_tok"][0, 0])}}))


def oracle_sample_step(w, n_slots, step_seed=0):
    """One oracle step (attention + verify + commit) on the first `n_slots` slots of workload `w`.

    Returns (positions, seconds, threads).  Inputs are generated on the CPU by the shared generators.
    """
    import numpy as np
    import torch
    from dataclasses import replace
    import oracle
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from helpers import bits16, logits_np, oracle_step, state_to_np
    from paper_2604_11035_b200 import workloads as wl
    ws = replace(w, batch=n_slots, steps=2, name=w.name + f"[first {n_slots} slots]")
    st = wl.make_state(ws, "cpu")
    s = state_to_np(st)
    threads = oracle.max_threads()
    oracle.set_threads(threads)
    # step 0 (bootstrap, untimed) so that the timed step verifies N-1 proposals per slot like a P step
    q, k, v = [bits16(x) for x in wl.make_qkv(ws, 0, "cpu")]
    lg0 = logits_np(wl.make_logits(ws, 0, torch.from_numpy(s["ctx_len"])))
    oracle_step(ws, s, q, k, v, lg0, None, 0)
    q, k, v = [bits16(x) for x in wl.make_qkv(ws, 1, "cpu")]
    lg1 = logits_np(wl.make_logits(ws, 1, torch.from_numpy(s["ctx_len"])))
    positions = int((s["n_ver"] + ws.stride).sum())
    t0 = time.time()
    oracle_step(ws, s, q, k, v, lg1, lg0, 1)
    return positions, time.time() - t0, threads


def cpu_baseline(args, w):
    import oracle
    oracle.build()
    n = args.cpu_slots or max(2, min(w.batch, 8 * oracle.max_threads()))   # about 10 s of host work
    pos, sec, threads = oracle_sample_step(w, n)
    return {"value": pos / sec, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"one P step (attention + verify + commit) of the first {n} slots of {w.name}, "
                      f"{pos} positions in {sec:.2f} s, fp64 C oracle with OpenMP over slots"}


def run_reference(args):
    """The reference arm of this tier is the fp64 CPU oracle, timed as it stands on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2604_11035_b200 import workloads as wl
    oracle.build()
    w = wl.config(args.config)
    n = args.cpu_slots or max(2, min(w.batch, 8 * oracle.max_threads()))
    K, W = args.steps, args.warmup
    K = min(K, 5)
    W = min(W, 1)
    for _ in range(W):
        oracle_sample_step(w, n)
    pos = sec = 0
    threads = 1
    for _ in range(K):
        p, s, threads = oracle_sample_step(w, n)
        pos += p
        sec += s
    value = pos / sec
    sample = (f"each step = one P step of the first {n} slots of {w.name} ({pos // K} positions), "
              f"fp64 C oracle, OpenMP over slots")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": K, "warmup": W, "ms_per_step": 1e3 * sec / K, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, help="workload index 0..4 (2 = batch 256, stride 8, ctx 1k-8k)")
    ap.add_argument("--propose-mode", type=int, default=None, choices=[0, 1])
    ap.add_argument("--q-mode", type=int, default=None, choices=[0, 1],
                    help="1: point-mass q (verification variant for argmax proposals)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-slots", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (smaller captures under ncu)")
    ap.add_argument("--sweep", default=None, metavar="STRIDE,BATCH|all",
                    help="one point of the sweep workload (stride in 2,4,8,16; batch in 1,8,64,256,512) instead of --config; "
                         "`all`: the twenty points, one JSON line each")
    ap.add_argument("--top-k", type=int, default=0, help="verify on top-k / top-p filtered laws (0 = plain softmax laws)")
    ap.add_argument("--top-p", type=float, default=1.0)
    ap.add_argument("--lora", default=None, metavar="N,K,RANK", help="time the segment-gated LoRA linear layer on the step's token rows")
    ap.add_argument("--layers", type=int, default=0, help="model-step mode: this many attention layers per step (isd_step_layers)")
    ap.add_argument("--graph", action="store_true", help="model-step mode: replay the step from a CUDA graph")
    ap.add_argument("--sequential-pages", action="store_true", help="identity page order instead of a shuffled pool")
    ap.add_argument("--no-pairings", dest="pairings", action="store_false",
                    help="skip the extra keys that time the other proposal / proposal-law pairings")
    ap.add_argument("--stub-step", action="store_true", help="CPU self-test of the multi-rank plumbing (gloo, no GPU)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    # one process per GPU: when this is not already a rank of a multi-process launch, --gpus N > 1 starts the N
    # ranks itself (the driver's torchrun launch sets WORLD_SIZE and is left alone)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not args.lora and args.layers == 0 and args.sweep != "all":
        if not args.stub_step and args.impl == "ours":
            import torch
            if args.gpus > torch.cuda.device_count():
                raise SystemExit(f"--gpus {args.gpus}: only {torch.cuda.device_count()} CUDA device(s) are visible on this node")
        codes = launch_ranks(args.gpus, sys.argv[1:])
        sys.exit(max(abs(c) for c in codes))
    if args.stub_step:
        run_stub(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.sweep == "all":
        run_sweep_all(args)
    elif args.lora:
        run_lora(args)
    elif args.layers > 0 or args.graph:
        args.layers = max(1, args.layers)
        run_model_step(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
