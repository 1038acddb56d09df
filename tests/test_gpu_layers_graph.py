"""Multi-layer step and CUDA-graph replay of a step vs the fp64 oracle (needs a B200).

isd_step_layers: every layer attends through the same page table and lengths with its own pools; the
oracle runs its attention once per layer on that layer's inputs, then verify and commit once.
Graph replay: a step captured once and replayed must advance its step number on the device
(isd_set_step_counter), otherwise every replay would draw the same random numbers.
"""
from dataclasses import replace

import numpy as np
import pytest
import torch

import oracle
import paper_2604_11035_b200 as isd_pkg
from helpers import bits16, compare_verify_and_state, logits_np, oracle_step, state_to_np
from paper_2604_11035_b200 import workloads as wl
from paper_2604_11035_b200.workloads import Workload

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_multi_layer_step_matches_oracle_layer_by_layer():
    L, steps = 3, 4
    w = Workload("layers", batch=5, stride=4, n_q_heads=32, n_kv_heads=8, vocab=4096 + 8 * 11, ctx_min=3,
                 ctx_max=600, logits_dtype="bf16", logit_sigma=2.0, peaked_frac=0.6, steps=steps,
                 propose_mode=0, seed=91)
    oracle.set_threads(oracle.max_threads())
    st = wl.make_state(w, DEV)
    s = state_to_np(st)
    # layer 0 uses the pools of the generated state, the others their own random pools of the same shape
    gen = torch.Generator(device=DEV)
    gen.manual_seed(1234)
    pools = [(st["k_pool"], st["v_pool"])]
    for _ in range(1, L):
        pools.append(tuple((torch.randn(st["k_pool"].shape, generator=gen, device=DEV) * w.kv_sigma).to(torch.bfloat16)
                           for _ in range(2)))
    pools_np = [(bits16(k).copy(), bits16(v).copy()) for k, v in pools]
    eng = isd_pkg.isd_for_workload(w, st)
    out = isd_pkg.alloc_verify_out(w.batch, w.stride, DEV)
    ao = [torch.zeros(w.batch, w.Q, w.n_q_heads, w.head_dim, dtype=torch.bfloat16, device=DEV) for _ in range(L)]
    al = [torch.zeros(w.batch, w.Q, w.n_q_heads, dtype=torch.float32, device=DEV) for _ in range(L)]
    prev = prev_np = None
    rejections = 0
    for t in range(steps):
        qkv = [wl.make_qkv(replace(w, seed=w.seed + 100 * l), t, DEV) for l in range(L)]
        lg = wl.make_logits(w, t, torch.from_numpy(s["ctx_len"]).to(DEV))
        layers = eng.layer_args([dict(q=qkv[l][0], k_new=qkv[l][1], v_new=qkv[l][2], k_pool=pools[l][0],
                                      v_pool=pools[l][1], attn_out=ao[l], attn_lse=al[l]) for l in range(L)])
        eng.isd_step_layers(st, layers, lg, prev, out, t)
        torch.cuda.synchronize()

        # ---- oracle: attention of every layer on the pre-commit state, then verify + commit once
        n_ver_before, ctx_before = s["n_ver"].copy(), s["ctx_len"].copy()
        q_len = np.where(s["active"] != 0, s["n_ver"] + w.stride, 0).astype(np.int32)
        for l in range(L):
            o_attn, o_lse = oracle.attn(
                Hq=w.n_q_heads, Hkv=w.n_kv_heads, D=w.head_dim, page_size=wl.PAGE, num_pages=s["num_pages"],
                sm_scale=1.0 / np.sqrt(w.head_dim), ctx_len=s["ctx_len"], q_len=q_len, active=s["active"],
                page_table=s["page_table"], q=bits16(qkv[l][0]), k_new=bits16(qkv[l][1]), v_new=bits16(qkv[l][2]),
                k_pool=pools_np[l][0], v_pool=pools_np[l][1], slot_status=s["slot_status"])
            g_out = ao[l].to(torch.float64).cpu().numpy()
            g_lse = al[l].to(torch.float64).cpu().numpy()
            gk, gv = bits16(pools[l][0]), bits16(pools[l][1])
            for b in range(w.batch):
                ql = int(q_len[b])
                e = np.abs(g_out[b, :ql] - o_attn[b, :ql]).max()
                assert e < 2.0 ** -7 * np.abs(o_attn[b, :ql]).max() + 1e-3, (t, l, b, e)
                assert np.abs(g_lse[b, :ql] - o_lse[b, :ql]).max() < 2e-2
                n = int(ctx_before[b]) + ql                     # appended rows of this layer's pools
                for pos in range(int(ctx_before[b]), n):
                    pg = s["page_table"][b, pos // 16]
                    assert np.array_equal(gk[pg, :, pos % 16], pools_np[l][0][pg, :, pos % 16]), (t, l, b, pos)
                    assert np.array_equal(gv[pg, :, pos % 16], pools_np[l][1][pg, :, pos % 16]), (t, l, b, pos)
        lg_np = logits_np(lg)
        _, _, vr, _ = oracle_step(w, s, None, None, None, lg_np, prev_np, t, do_attn=False)
        compare_verify_and_state(w, t, out, st, vr, s, n_ver_before)
        rejections += int((vr.accept_len < n_ver_before).sum())
        prev, prev_np = lg, lg_np
    assert rejections > 0
    assert eng.isd_read_status() == 0
    assert eng.isd_launch_count() == steps * (3 * L + 2)   # per layer: append, attention, combine; then rows, sampling (+ commit)
    eng.close()


def test_captured_step_replays_with_a_device_step_counter():
    steps = 5
    w = Workload("graph", batch=6, stride=4, n_q_heads=32, n_kv_heads=8, vocab=4096, ctx_min=20, ctx_max=400,
                 logits_dtype="f32", logit_sigma=2.0, peaked_frac=0.5, steps=steps, propose_mode=0, seed=17)
    oracle.set_threads(oracle.max_threads())
    st = wl.make_state(w, DEV)
    s = state_to_np(st)
    eng = isd_pkg.isd_for_workload(w, st)
    out = isd_pkg.alloc_verify_out(w.batch, w.stride, DEV)
    ctx0 = st["ctx_len"].clone()
    # fixed buffers the captured step reads; the host refreshes them between replays
    q, k, v = (x.clone() for x in wl.make_qkv(w, 0, DEV))
    cur = wl.make_logits(w, 0, ctx0).clone()
    prev = torch.zeros_like(cur)
    ao = torch.zeros(w.batch, w.Q, w.n_q_heads, w.head_dim, dtype=torch.bfloat16, device=DEV)
    counter = torch.zeros(1, dtype=torch.int32, device=DEV)
    eng.isd_set_step_counter(counter)
    args = eng.step_args(q=q, k_new=k, v_new=v, k_pool=st["k_pool"], v_pool=st["v_pool"], attn_out=ao,
                         attn_lse=None, logits_cur=cur, q_prev_logits=prev, out=out)
    st_struct = eng.state_struct(st)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        eng.isd_step(st, args, 12345, st_struct=st_struct)   # the host step argument is ignored: the counter rules
        prev.copy_(cur)                                      # this step's logits are the next step's proposal laws
    prev_np = None
    rejections = 0
    for t in range(steps):
        qt, kt, vt = wl.make_qkv(w, t, DEV)
        lg = wl.make_logits(w, t, ctx0)      # inputs fixed in advance (independent of the state), as a replay needs
        q.copy_(qt); k.copy_(kt); v.copy_(vt); cur.copy_(lg)
        graph.replay()
        torch.cuda.synchronize()
        n_ver_before = s["n_ver"].copy()
        lg_np = logits_np(lg)
        _, _, vr, _ = oracle_step(w, s, bits16(qt), bits16(kt), bits16(vt), lg_np, prev_np, t)
        assert int(counter.item()) == t + 1
        compare_verify_and_state(w, t, out, st, vr, s, n_ver_before)
        rejections += int((vr.accept_len < n_ver_before).sum())
        prev_np = lg_np
    # two different steps drew different noise: with a frozen step number the chain above could not match
    assert rejections > 0
    assert eng.isd_read_status() == 0
    eng.isd_set_step_counter(None)
    eng.close()
