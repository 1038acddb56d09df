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
    if args.graph:
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            launch()
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
        flush.zero_()
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
                   "ctx": [w.ctx_min, w.ctx_max], "l2": "flushed (512 MB write) before every step"},
        "emitted_tokens_per_s": int(emit_acc[W:].sum().item()) / t_total,
        "step_algorithmic_gbs": gbs, "step_frac_of_8TBs": gbs / HBM_NOMINAL_GBS, "step_frac_of_measured_copy": gbs / peak,
        "gpu_launches": launches if graph is None else K * (3 * L + (3 if w.top_k else 2)), "launches_issued_by_host": launches,
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
        flush.zero_()
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


def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2604_11035_b200 as pkg
    from paper_2604_11035_b200 import workloads as wl

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    # weak scaling: every rank owns its own slots, pools and free stack (slots never interact)
    w = rank_workload(args.config, rank, args.sweep, args.top_k, args.top_p)
    if args.propose_mode is not None:
        from dataclasses import replace
        w = replace(w, propose_mode=args.propose_mode)
    if args.q_mode is not None:
        from dataclasses import replace
        w = replace(w, q_mode=args.q_mode, name=w.name + f"[q_mode {args.q_mode}]")
    K, W = args.steps, args.warmup
    from dataclasses import replace
    VER_STEPS = 6   # instrumented steps after the timed region: 3 carry the events around the attention kernel,
                    # 3 those around the verification kernels (an event between two kernels serialises launches
                    # that the timed steps overlap, so the timed steps carry none)
    ATTN_INSTR = 3
    w = replace(w, steps=max(w.steps, K + W + args.e2e_steps + VER_STEPS + 2))
    if args.sequential_pages:
        w = replace(w, shuffle_pages=False, name=w.name + "[sequential pages]")
    if args.batch:
        w = replace(w, batch=args.batch, name=w.name + f"[batch {args.batch}]")
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
    total_steps = W + K + VER_STEPS
    e_step = [(ev(), ev()) for _ in range(total_steps)]
    e_attn = [(ev(), ev()) for _ in range(total_steps)]
    e_ver = [(ev(), ev()) for _ in range(total_steps)]
    for pairs in (e_step, e_attn, e_ver):
        for a, b in pairs:
            a.record(); b.record()      # creates the underlying CUDA events
    pos_acc = torch.zeros(total_steps, dtype=torch.int64, device=dev)
    emit_acc = torch.zeros(total_steps, dtype=torch.int64, device=dev)
    rej_acc = torch.zeros(total_steps, dtype=torch.int64, device=dev)
    attn_bytes_acc = torch.zeros(total_steps, dtype=torch.int64, device=dev)
    kv_tok = 2 * w.n_kv_heads * w.head_dim * 2

    def one_step(t, timed_events=True):
        q, k, v = wl.make_qkv(w, t, dev)
        cur, prev = logits[t & 1], (logits[(t - 1) & 1] if t > 0 else None)
        wl.make_logits(w, t, st["ctx_len"], out=cur)
        q_len = torch.where(st["active"] != 0, st["n_ver"] + w.stride, 0).to(torch.int64)
        pos_acc[t] = q_len.sum()
        # main attention kernel: KV read once + Q read + O write (the K/V append is a separate launch)
        attn_bytes_acc[t] = ((st["ctx_len"].to(torch.int64) + q_len) * kv_tok).sum() \
            + q_len.sum() * (w.n_q_heads * w.head_dim * 4)
        nv_before = st["n_ver"].clone()
        flush.zero_()                                   # L2 flush: 512 MB > 126 MB L2
        sargs = eng.step_args(q=q, k_new=k, v_new=v, k_pool=st["k_pool"], v_pool=st["v_pool"], attn_out=attn_out,
                              attn_lse=None, logits_cur=cur, q_prev_logits=prev, out=out)
        if t < W + K:
            eng.isd_set_profile_events(None, None, None, None)
        elif t < W + K + ATTN_INSTR:
            eng.isd_set_profile_events(e_attn[t][0], e_attn[t][1], None, None)
        else:
            eng.isd_set_profile_events(None, None, e_ver[t][0], e_ver[t][1])
        e_step[t][0].record()
        eng.isd_step(st, sargs, t, st_struct)
        e_step[t][1].record()
        emit_acc[t] = out["n_emit"].sum()
        rej_acc[t] = (out["accept_len"] < nv_before).sum()

    sampler = ClockSampler(local)
    for t in range(W):
        one_step(t)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    launches0 = eng.isd_launch_count()
    sampler.start()
    wall0 = time.time()
    for t in range(W, W + K):
        one_step(t)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    wall = time.time() - wall0
    clocks = sampler.stop()
    launches = eng.isd_launch_count() - launches0
    for t in range(W + K, W + K + VER_STEPS):
        one_step(t)
    torch.cuda.synchronize()
    eng.isd_set_profile_events(None, None, None, None)
    status = eng.isd_read_status()

    step_ms = [a.elapsed_time(b) for a, b in e_step[W:W + K]]
    attn_ms = [a.elapsed_time(b) for a, b in e_attn[W + K:W + K + ATTN_INSTR]]
    ver_ms = [a.elapsed_time(b) for a, b in e_ver[W + K + ATTN_INSTR:]]
    instr_step_ms = [a.elapsed_time(b) for a, b in e_step[W + K:]]
    ver_positions = int(pos_acc[W + K + ATTN_INSTR:].sum().item())
    ver_rejecting = int(rej_acc[W + K + ATTN_INSTR:].sum().item())
    t_total = sum(step_ms) / 1e3
    positions = int(pos_acc[W:W + K].sum().item())
    emitted = int(emit_acc[W:W + K].sum().item())
    rejecting = int(rej_acc[W:W + K].sum().item())
    lb = 2 if w.logits_dtype == "bf16" else 4
    attn_bytes = int(attn_bytes_acc[W:W + K].sum().item())
    attn_bytes_instr = int(attn_bytes_acc[W + K:W + K + ATTN_INSTR].sum().item())
    # full rows a rejection reads again (filtered laws: short lists instead; point-mass q: no proposal-law row)
    rej_rows = 0 if w.top_k else (2 if w.q_mode == 0 else 1)
    verify_bytes = positions * w.vocab * lb + rejecting * rej_rows * w.vocab * lb

    # ---- end to end through the C ABI with HOST buffers: H2D of the step's inputs and D2H of its
    # results inside the timed window (fewer steps: the logits alone are > 1 GB per step)
    e2e_steps = min(K, args.e2e_steps)
    e2e = None
    if e2e_steps > 0:
        host_q, host_k, host_v = [torch.empty_like(x, device="cpu").pin_memory() for x in wl.make_qkv(w, 0, dev)]
        host_lg = torch.empty(B, Q, w.vocab, dtype=dt, device="cpu").pin_memory()
        host_out = {k_: torch.empty_like(v_, device="cpu").pin_memory() for k_, v_ in out.items()
                    if k_ in ("n_emit", "out_tok", "accept_len")}
        dq, dk, dv = [torch.empty_like(x) for x in wl.make_qkv(w, 0, dev)]
        e2e_pos, e2e_t = 0, 0.0
        t_base = W + K + VER_STEPS          # the chain goes on where the instrumented steps left it
        ee = [(ev(), ev()) for _ in range(e2e_steps)]
        for i in range(e2e_steps):
            t = t_base + i
            q, k, v = wl.make_qkv(w, t, dev)
            cur, prev = logits[t & 1], logits[(t - 1) & 1]
            wl.make_logits(w, t, st["ctx_len"], out=cur)
            host_q.copy_(q); host_k.copy_(k); host_v.copy_(v); host_lg.copy_(cur)
            e2e_pos += int(torch.where(st["active"] != 0, st["n_ver"] + w.stride, 0).sum().item())
            flush.zero_()
            torch.cuda.synchronize()
            ee[i][0].record()
            dq.copy_(host_q, non_blocking=True); dk.copy_(host_k, non_blocking=True); dv.copy_(host_v, non_blocking=True)
            cur.copy_(host_lg, non_blocking=True)
            sargs = eng.step_args(q=dq, k_new=dk, v_new=dv, k_pool=st["k_pool"], v_pool=st["v_pool"], attn_out=attn_out,
                                  attn_lse=None, logits_cur=cur, q_prev_logits=prev, out=out)
            eng.isd_step(st, sargs, t, st_struct)
            for k_, h in host_out.items():
                h.copy_(out[k_], non_blocking=True)
            ee[i][1].record()
            torch.cuda.synchronize()
            e2e_t += ee[i][0].elapsed_time(ee[i][1]) / 1e3
        h2d = sum(x.numel() * x.element_size() for x in (host_q, host_k, host_v, host_lg))
        d2h = sum(x.numel() * x.element_size() for x in host_out.values())
        e2e = {"pos": e2e_pos, "t": e2e_t, "h2d": h2d, "d2h": d2h, "steps": e2e_steps}

    # ---- reduce over ranks: max time, summed positions
    if world > 1:
        red = reduce_over_ranks(dist, dev, [t_total, e2e["t"] if e2e else 0.0],
                                [positions, emitted, e2e["pos"] if e2e else 0, launches])
        t_total, positions, emitted, launches = red["max"][0], red["sum"][0], red["sum"][1], red["sum"][3]
        if e2e:
            e2e["t"], e2e["pos"] = red["max"][1], red["sum"][2]
    if rank != 0:
        eng.close()
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peaks()
    attn_gbs = attn_bytes_instr / (sum(attn_ms) / 1e3) / 1e9
    ver_bytes_timed = ver_positions * w.vocab * lb + ver_rejecting * rej_rows * w.vocab * lb   # of the steps that carry the events
    ver_gbs = ver_bytes_timed / (sum(ver_ms) / 1e3) / 1e9 if sum(ver_ms) > 0 else None
    step_bytes = attn_bytes + positions * kv_tok + verify_bytes      # + K/V append writes
    line = {
        "metric": METRIC, "value": positions / t_total, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": 1e3 * t_total / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "batch_per_gpu": w.batch, "stride": w.stride, "heads": f"{w.n_q_heads}/{w.n_kv_heads}",
                   "head_dim": w.head_dim, "vocab": w.vocab, "logits_dtype": w.logits_dtype,
                   "ctx": [w.ctx_min, w.ctx_max], "propose_mode": "argmax" if w.propose_mode else "sample",
                   "peaked_frac": w.peaked_frac, "chained": True, "l2": "flushed (512 MB write) before every step; inputs 6 GB >> L2",
                   "parallelism": f"slots x{world} (no collective)"},
        "emitted_tokens_per_s": emitted / t_total, "tokens_per_step_per_slot": emitted / max(1, K * w.batch * world),
        "step_algorithmic_gbs": step_bytes / (sum(step_ms) / 1e3) / 1e9,
        "step_frac_of_8TBs": step_bytes / (sum(step_ms) / 1e3) / 1e9 / HBM_NOMINAL_GBS,
        "step_frac_of_measured_copy": step_bytes / (sum(step_ms) / 1e3) / 1e9 / peak,
        "roofline": {"kernel": "attn_tc_kernel", "bound": "hbm", "achieved": attn_gbs, "peak": peak, "peak_kind": peak_kind,
                     "unit": "GB/s", "frac": attn_gbs / peak, "frac_of_8TBs": attn_gbs / HBM_NOMINAL_GBS,
                     "traffic": None, "ms_per_launch": sum(attn_ms) / len(attn_ms),
                     "bytes_per_launch": attn_bytes_instr / len(attn_ms),
                     "timed_on": "%d instrumented steps right after the timed region (same chain, L2 flushed; %.3f ms per "
                                 "instrumented step)" % (len(attn_ms), sum(instr_step_ms) / len(instr_step_ms)),
                     "share_of_step": (sum(attn_ms) / len(attn_ms)) / (sum(step_ms) / K)},
        "verify_kernels": {"kernels": "topk_rows_kernel (+ topk_decide_kernel when proposal-law rows are streamed)" if w.top_k else "verify_rows_kernel + verify_sample_kernel", "achieved_gbs": ver_gbs, "ms_per_launch": sum(ver_ms) / max(1, len(ver_ms)),
                           "timed_on": "%d instrumented steps after the timed region" % len(ver_ms),
                               "frac_of_measured_copy": (ver_gbs / peak) if ver_gbs else None},
        "gpu_launches": launches, "status_word": status, "clocks": clocks, "wall_s": wall,
    }
    if e2e:
        line["e2e"] = {"value": e2e["pos"] / e2e["t"], "unit": UNIT, "h2d_bytes_per_step": e2e["h2d"],
                       "d2h_bytes_per_step": e2e["d2h"], "steps": e2e["steps"]}
    # DRAM traffic per launch: ncu capture of a smaller case of the same kernel (see profiles/), scaled by
    # the algorithmic bytes of this launch (the kernel's traffic is proportional to the KV bytes it streams)
    prof = os.path.join(ROOT, "profiles", "attn_tc_kernel_sweep_n8_b64.md")
    if os.path.exists(prof):
        import re
        m = re.search(r"dram_bytes_per_algorithmic_byte = ([0-9.]+)", open(prof).read())
        if m:
            line["roofline"]["traffic"] = float(m.group(1)) * attn_bytes_instr / len(attn_ms)
            line["roofline"]["traffic_source"] = "ncu capture of B=64 case scaled by algorithmic bytes"
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline(args, w)
    eng.close()
    if world > 1:
        dist.destroy_process_group()
    print(json.dumps(line))


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
    ap.add_argument("--sweep", default=None, metavar="STRIDE,BATCH",
                    help="one point of the sweep workload (stride in 2,4,8,16; batch in 1,8,64,256,512) instead of --config")
    ap.add_argument("--top-k", type=int, default=0, help="verify on top-k / top-p filtered laws (0 = plain softmax laws)")
    ap.add_argument("--top-p", type=float, default=1.0)
    ap.add_argument("--lora", default=None, metavar="N,K,RANK", help="time the segment-gated LoRA linear layer on the step's token rows")
    ap.add_argument("--layers", type=int, default=0, help="model-step mode: this many attention layers per step (isd_step_layers)")
    ap.add_argument("--graph", action="store_true", help="model-step mode: replay the step from a CUDA graph")
    ap.add_argument("--sequential-pages", action="store_true", help="identity page order instead of a shuffled pool")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    elif args.lora:
        run_lora(args)
    elif args.layers > 0 or args.graph:
        args.layers = max(1, args.layers)
        run_model_step(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
