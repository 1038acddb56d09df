"""CUDA path vs fp64 oracle, element by element, through the C ABI (needs a B200)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2604_11035_b200 as isd_pkg
from helpers import STATE_KEYS, bits16, compare_verify_and_state, logits_np, oracle_step, state_to_np
from paper_2604_11035_b200 import workloads as wl
from paper_2604_11035_b200.workloads import Workload
from parity import run_chain_parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def assert_clean(rep, allow_exempt=0):
    assert rep["mismatches"] == 0, rep["details"]
    assert rep["exempt_flips"] <= allow_exempt, rep
    assert rep["attn_max_abs_err"] < 2e-2 and rep["lse_max_abs_err"] < 2e-2, rep
    assert rep["alpha_max_abs_err"] < 2e-2 and rep["qstats_max_abs_err"] < 2e-2, rep
    assert rep["gpu_launches"] > 0


def test_config0_tiny():
    rep = run_chain_parity(wl.config(0), steps=4, device=DEV)
    assert_clean(rep)
    assert rep["positions"] > 0 and rep["emitted"] >= 4


@pytest.mark.parametrize("dtype,propose_mode,q_mode,N", [
    ("f32", 0, 0, 4), ("bf16", 0, 0, 4), ("bf16", 1, 0, 8), ("bf16", 1, 1, 3), ("f32", 0, 0, 2), ("bf16", 0, 0, 16)])
def test_ragged_multi_tile_chain(dtype, propose_mode, q_mode, N):
    # several 128-key tiles per slot, ragged tails, mixed P / NP steps, pages shuffled
    w = Workload("ragged", batch=5, stride=N, n_q_heads=32, n_kv_heads=8, vocab=4096 + 8 * 37, ctx_min=3,
                 ctx_max=700, logits_dtype=dtype, logit_sigma=2.0, peaked_frac=0.6, steps=8,
                 propose_mode=propose_mode, q_mode=q_mode, seed=40 + N)
    rep = run_chain_parity(w, steps=8, device=DEV)
    assert_clean(rep)
    assert rep["rejections"] > 0 and rep["tpf"] > 1.0


@pytest.mark.parametrize("dtype,propose_mode,q_mode,N,top_k,top_p", [
    ("bf16", 0, 0, 4, 50, 0.95), ("f32", 0, 0, 4, 8, 0.7), ("bf16", 1, 0, 8, 50, 0.95), ("bf16", 1, 1, 3, 20, 1.0),
    ("bf16", 0, 0, 2, 1, 1.0), ("f32", 0, 0, 3, 64, 0.5)])
def test_filtered_laws_chain(dtype, propose_mode, q_mode, N, top_k, top_p):
    # top-k / top-p filtered verification: ragged rows, ties (bf16 logits repeat values), mixed P / NP steps
    w = Workload("filtered", batch=6, stride=N, n_q_heads=8, n_kv_heads=2, vocab=8192 + 8 * 29, ctx_min=3,
                 ctx_max=300, logits_dtype=dtype, logit_sigma=2.0, peaked_frac=0.5, steps=8,
                 propose_mode=propose_mode, q_mode=q_mode, seed=60 + N + top_k, top_k=top_k, top_p=top_p)
    rep = run_chain_parity(w, steps=8, device=DEV)
    assert_clean(rep)
    assert rep["tpf"] >= 1.0
    if top_k > 1:
        assert rep["rejections"] > 0


def test_filtered_laws_full_vocab_and_batch():
    # the serving configuration at the benchmark's vocabulary and a batch that fills the machine several times
    w = Workload("filtered_big", batch=96, stride=8, vocab=151936, ctx_min=64, ctx_max=512, logits_dtype="bf16",
                 peaked_frac=0.9, steps=4, propose_mode=0, seed=71, top_k=50, top_p=0.95)
    rep = run_chain_parity(w, steps=3, device=DEV, attn_slots=[0, 95])
    assert_clean(rep)
    assert rep["rejections"] > 0


def _structured_logits(w, t, dtype):
    """Rows that stress the top-k selection: monotone in the index, constant, long runs of equal values, the
    best entries at the very end, almost everything masked out; slots 6 and 7 are ordinary random rows."""
    V, Q = w.vocab, w.Q
    g = torch.Generator(device="cpu")
    g.manual_seed(1000 + t)
    lg = torch.randn(w.batch, Q, V, generator=g) * 2.0
    i = torch.arange(V, dtype=torch.float32)
    shift = torch.arange(Q, dtype=torch.float32)[:, None]
    lg[0] = i[None, :] * 2e-4 + 0.01 * shift                        # upwards: every element beats the ones before it
    lg[1] = -i[None, :] * 2e-4 - 0.01 * shift                       # downwards
    lg[2] = 0.25 + 0.0 * shift                                      # one value everywhere
    lg[3] = torch.floor((i[None, :] + 37 * shift + 11 * t) / 3000.0) * 0.5   # runs of 3000 equal values, rising
    lg[4, :, V - 200:] += 6.0                                       # the top of the row sits in its last stage
    mask = torch.rand(Q, V, generator=g) < 0.9995
    lg[5][mask] = float("-inf")                                     # fewer finite entries than top_k
    return lg.to(dtype).to(DEV)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_filtered_selection_on_structured_rows(dtype):
    # rows on which the single-stream selection has to give up and start over (upward rows, runs of equal values),
    # next to rows it handles directly; every output and the committed state must equal the oracle's
    steps = 3
    w = Workload("structured", batch=8, stride=4, n_q_heads=8, n_kv_heads=2, vocab=40000 + 8 * 3, ctx_min=5,
                 ctx_max=200, logits_dtype=dtype, steps=steps, propose_mode=0, seed=33, top_k=50, top_p=0.95)
    oracle.set_threads(oracle.max_threads())
    st, eng, out = _fresh(w)
    s = state_to_np(st)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    prev = prev_np = None
    for t in range(steps):
        lg = _structured_logits(w, t, tdt)
        q, k, v = wl.make_qkv(w, t, DEV)
        n_ver_before = s["n_ver"].copy()
        _step(w, st, eng, out, t, prev, logits=lg)
        lg_np = logits_np(lg)
        _, _, vr, _ = oracle_step(w, s, bits16(q), bits16(k), bits16(v), lg_np, prev_np, t)
        compare_verify_and_state(w, t, out, st, vr, s, n_ver_before)
        prev, prev_np = lg, lg_np
    assert eng.isd_read_status() == 0
    eng.close()


def test_filtered_proposal_law_rows_cached_or_streamed():
    # On a rejection the filtered proposal law of the rejected position is needed.  When q_prev_logits is the very
    # buffer the previous call selected from, the lists of that call are reused; any other buffer (here: a copy)
    # is streamed and selected again.  Both routes must give the same step, bit for bit.
    w = Workload("qcache", batch=6, stride=4, n_q_heads=8, n_kv_heads=2, vocab=8192 + 8 * 5, ctx_min=3, ctx_max=200,
                 logits_dtype="bf16", logit_sigma=2.0, peaked_frac=0.5, steps=6, propose_mode=0, seed=44,
                 top_k=50, top_p=0.95)
    runs = []
    for copy_prev in (False, True):
        st, eng, out = _fresh(w)
        prev, acc, rejections = None, [], 0
        for t in range(6):
            n_ver_before = st["n_ver"].clone()
            fed = prev.clone() if (copy_prev and prev is not None) else prev
            prev, _ = _step(w, st, eng, out, t, fed)
            rejections += int((out["accept_len"] < n_ver_before).sum())
            acc.append([x.clone() for x in out.values()] + [st[k].clone() for k in STATE_KEYS])
        assert eng.isd_read_status() & ~isd_pkg.binding.ST_EMPTY_RESIDUAL == 0
        eng.close()
        runs.append(acc)
        assert rejections > 0
    for a, b in zip(*runs):
        for x, y in zip(a, b):
            assert torch.equal(x.view(torch.uint8) if x.dtype.is_floating_point else x,
                               y.view(torch.uint8) if y.dtype.is_floating_point else y)


def test_temperature_and_relaxed_acceptance():
    w = Workload("temp", batch=6, stride=4, n_q_heads=8, n_kv_heads=2, vocab=2048, ctx_min=20, ctx_max=200,
                 logits_dtype="f32", logit_sigma=2.0, peaked_frac=0.5, steps=6, propose_mode=0, seed=77)
    st_kw = dict(inv_temperature=0.7, tau=0.5)
    # the oracle helper takes the same scalars
    import parity
    orig = parity.oracle_step
    parity.oracle_step = lambda *a, **k: orig(*a, inv_temperature=0.7, tau=0.5, **k)
    try:
        rep = run_chain_parity(w, steps=6, device=DEV, **st_kw)
    finally:
        parity.oracle_step = orig
    assert_clean(rep)


def test_config1_moderate_full():
    rep = run_chain_parity(wl.config(1), steps=2, device=DEV, attn_slots=lambda t: [t, 7 + 3 * t, 31 - t])
    assert_clean(rep)
    assert rep["rejections"] > 0


def test_config2_stationary_batch_full_size_sampled_attention():
    # full launch configuration of the benchmark; verify/commit compared on all 256 slots,
    # attention on sampled slots (the oracle needs ~1 s per slot)
    # (here with sampled proposals judged against their softmax law, Algorithm 1 to the letter; the 100-step chain
    # below runs the workload's own pairing, argmax proposals against a point mass)
    w = wl.config(2, steps=4, propose_mode=0, q_mode=0)
    rep = run_chain_parity(w, steps=3, device=DEV, attn_slots=lambda t: [(37 * t) % 256, (100 + 41 * t) % 256, 255 - t],
                           check_pools=True)
    assert_clean(rep)
    assert rep["positions"] >= 256 * 8


def test_config3_long_context_sampled():
    rep = run_chain_parity(wl.config(3), steps=2, device=DEV, attn_slots=lambda t: [(5 * t + 3) % 16])
    assert_clean(rep)


def test_config2_hundred_chained_steps_at_full_batch():
    # the stationary batch as the benchmark definition states it: 100 chained isd_step calls at batch 256 with the
    # accept lengths fed back; verification, commit, page tables and the free stack are compared on every slot at
    # every step (about fifty fresh pages per slot come off the stack over the run), attention and the appended
    # K/V rows on a rotating pair of slots every tenth step
    w = wl.config(2)
    assert w.steps == 100 and w.batch == 256
    pick = lambda t: [(7 * t) % w.batch, (7 * t + 131) % w.batch] if t % 10 == 0 else []
    rep = run_chain_parity(w, steps=100, device=DEV, attn_slots=pick)
    # about 130,000 accept tests: a couple of dozen fall within 1e-4 of their uniform draw, and one of those is
    # decided the other way in fp32 (the exemption the benchmark definition grants; counted, the slot-step skipped,
    # the chain re-synchronised from the oracle).  Everything else is exact.
    assert rep["near_threshold"] >= rep["exempt_flips"]
    assert_clean(rep, allow_exempt=2)
    assert rep["positions"] > 100 * 256 * 8 and rep["rejections"] > 1000
    assert 3.5 < rep["tpf"] < 4.6            # the workload is tuned to the paper's stride-8 operating point (TPF 4.01)


@pytest.mark.parametrize("stride,batch,pairing", [(2, 1, (1, 1)), (2, 512, (1, 1)), (16, 1, (0, 0)), (16, 512, (1, 1)),
                                                  (8, 64, (1, 0)), (4, 256, (0, 0))])
def test_config4_sweep_points(stride, batch, pairing):
    # corners and centre of the sweep (stride in 2..16 x batch in 1..512 at context 4,096, seeds fixed per point):
    # two chained steps (an NP step, then a P step) with verification and commit compared on every slot and
    # attention on a sample of at most three slots that moves with the step
    from dataclasses import replace
    w = replace(wl.sweep_point(stride, batch), propose_mode=pairing[0], q_mode=pairing[1])
    pick = lambda t: sorted({(11 * t + 1) % batch, (batch // 2 + 5 * t) % batch, (batch - 1 - t) % batch})
    rep = run_chain_parity(w, steps=2, device=DEV, attn_slots=pick)
    assert_clean(rep)
    assert rep["positions"] == batch * stride + batch * (2 * stride - 1)


def _fresh(w, **kw):
    st = wl.make_state(w, DEV)
    eng = isd_pkg.isd_for_workload(w, st, **kw)
    out = isd_pkg.alloc_verify_out(w.batch, w.stride, DEV)
    return st, eng, out


def _step(w, st, eng, out, t, prev, logits=None):
    q, k, v = wl.make_qkv(w, t, DEV)
    lg = wl.make_logits(w, t, st["ctx_len"]) if logits is None else logits
    ao = torch.zeros(w.batch, w.Q, w.n_q_heads, w.head_dim, dtype=torch.bfloat16, device=DEV)
    args = eng.step_args(q=q, k_new=k, v_new=v, k_pool=st["k_pool"], v_pool=st["v_pool"], attn_out=ao,
                         attn_lse=None, logits_cur=lg, q_prev_logits=prev, out=out)
    eng.isd_step(st, args, t)
    torch.cuda.synchronize()
    return lg, ao


def test_run_to_run_determinism():
    w = Workload("det", batch=7, stride=4, n_q_heads=32, n_kv_heads=8, vocab=8192, ctx_min=50, ctx_max=900,
                 logits_dtype="bf16", peaked_frac=0.5, steps=4, propose_mode=0, seed=5)
    snaps = []
    for _ in range(2):
        st, eng, out = _fresh(w)
        prev = None
        acc = []
        for t in range(4):
            prev, ao = _step(w, st, eng, out, t, prev)
            acc.append([x.clone() for x in out.values()] + [ao.clone()] + [st[k].clone() for k in STATE_KEYS])
        snaps.append(acc)
        eng.close()
    for a, b in zip(snaps[0], snaps[1]):
        for x, y in zip(a, b):
            assert torch.equal(x.view(torch.uint8) if x.dtype.is_floating_point else x,
                               y.view(torch.uint8) if y.dtype.is_floating_point else y)


@pytest.mark.parametrize("top_k,top_p", [(0, 1.0), (20, 0.9)], ids=["plain", "filtered"])
def test_inactive_slots_and_empty_batch(top_k, top_p):
    w = Workload("inact", batch=4, stride=3, n_q_heads=8, n_kv_heads=2, vocab=1024, ctx_min=10, ctx_max=90,
                 logits_dtype="f32", steps=3, propose_mode=0, seed=8, top_k=top_k, top_p=top_p)
    st, eng, out = _fresh(w)
    st["active"][1] = 0
    before = {k: st[k].clone() for k in STATE_KEYS}
    kp = st["k_pool"].clone()
    _step(w, st, eng, out, 0, None)
    assert st["ctx_len"][1] == before["ctx_len"][1] and torch.equal(st["block_tok"][1], before["block_tok"][1])
    assert (st["ctx_len"][[0, 2, 3]] == before["ctx_len"][[0, 2, 3]] + 1).all()
    st["active"][:] = 0
    snap = {k: st[k].clone() for k in STATE_KEYS}
    kp = st["k_pool"].clone()
    _step(w, st, eng, out, 1, None)
    for k in STATE_KEYS:
        assert torch.equal(st[k], snap[k])
    assert torch.equal(st["k_pool"], kp)
    assert eng.isd_read_status() == 0
    eng.close()


@pytest.mark.parametrize("top_k,top_p", [(0, 1.0), (20, 0.9)], ids=["plain", "filtered"])
def test_faults_set_status_bits_and_freeze_the_slot(top_k, top_p):
    # (filtered: the decide kernel runs as clusters of two CTAs; frozen and inactive slots leave before its barriers)
    w = Workload("fault", batch=5, stride=3, n_q_heads=8, n_kv_heads=2, vocab=1024, ctx_min=30, ctx_max=60,
                 logits_dtype="f32", steps=4, propose_mode=0, seed=9, top_k=top_k, top_p=top_p)
    st, eng, out = _fresh(w)
    s_np = state_to_np(st)                              # oracle starts from the same generated state
    lg0 = wl.make_logits(w, 0, torch.from_numpy(s_np["ctx_len"]).to(DEV))
    prev, _ = _step(w, st, eng, out, 0, None, logits=lg0)   # bootstrap: everyone proposes
    q0, k0, v0 = wl.make_qkv(w, 0, DEV)
    oracle_step(w, s_np, bits16(q0), bits16(k0), bits16(v0), logits_np(lg0), None, 0)
    assert (st["n_ver"] == 2).all() and np.all(s_np["n_ver"] == 2)
    lg = wl.make_logits(w, 1, torch.from_numpy(s_np["ctx_len"]).to(DEV))
    lg[1, 0, 5] = float("nan")                          # non-finite anchor row
    st["block_tok"][2, 1] = w.vocab + 3                 # proposal id out of range
    st["page_table"][3, 0] = st["num_pages"] + 9        # page id out of range
    s_np["block_tok"][2, 1] = w.vocab + 3
    s_np["page_table"][3, 0] = st["num_pages"] + 9
    before = {k: st[k].clone() for k in STATE_KEYS}
    q, k, v = wl.make_qkv(w, 1, DEV)
    _step(w, st, eng, out, 1, prev, logits=lg)
    oracle_step(w, s_np, bits16(q), bits16(k), bits16(v), logits_np(lg), logits_np(prev), 1)
    status = st["slot_status"].cpu().numpy().view(np.uint32)
    assert status[1] & isd_pkg.binding.ST_NONFINITE_LOGIT
    assert status[2] & isd_pkg.binding.ST_BAD_TOKEN_ID
    assert status[3] & isd_pkg.binding.ST_BAD_PAGE_ID
    assert status[0] == 0 and status[4] == 0
    assert np.array_equal(status != 0, s_np["slot_status"] != 0)
    for b in (1, 2, 3):                                 # frozen
        assert st["ctx_len"][b] == before["ctx_len"][b] and st["n_ver"][b] == before["n_ver"][b]
    for b in (0, 4):                                    # healthy slots advanced exactly like the oracle's
        assert st["ctx_len"][b].item() == s_np["ctx_len"][b]
        assert np.array_equal(st["block_tok"][b].cpu().numpy(), s_np["block_tok"][b])
    g = eng.isd_read_status()
    assert g & 4 and g & 8 and g & 16
    assert eng.isd_read_status() == 0                   # cleared by the read
    eng.close()


def test_pool_exhaustion_and_capacity_match_the_oracle():
    w = Workload("pool", batch=6, stride=4, n_q_heads=8, n_kv_heads=2, vocab=512, ctx_min=40, ctx_max=56,
                 logits_dtype="f32", peaked_frac=1.0, steps=1, propose_mode=1, seed=10)
    st, eng, out = _fresh(w)
    st["free_top"][0] = 3                               # nearly empty pool
    s_np = state_to_np(st)
    prev = prev_np = None
    for t in range(12):
        q, k, v = wl.make_qkv(w, t, DEV)
        lg = wl.make_logits(w, t, torch.from_numpy(s_np["ctx_len"]).to(DEV))
        ao = torch.zeros(w.batch, w.Q, w.n_q_heads, w.head_dim, dtype=torch.bfloat16, device=DEV)
        args = eng.step_args(q=q, k_new=k, v_new=v, k_pool=st["k_pool"], v_pool=st["v_pool"], attn_out=ao,
                             attn_lse=None, logits_cur=lg, q_prev_logits=prev, out=out)
        eng.isd_step(st, args, t)
        torch.cuda.synchronize()
        oracle_step(w, s_np, bits16(q), bits16(k), bits16(v), logits_np(lg), prev_np, t)
        prev, prev_np = lg, logits_np(lg)
        for name in ("ctx_len", "n_ver", "free_top"):
            assert np.array_equal(st[name].cpu().numpy(), s_np[name]), (t, name)
        assert np.array_equal(st["slot_status"].cpu().numpy().view(np.uint32), s_np["slot_status"]), t
    status = s_np["slot_status"]
    assert np.any(status & oracle.ST_POOL_EXHAUSTED) or np.any(status & oracle.ST_SLOT_CAPACITY)
    eng.close()


def test_release_returns_pages():
    w = Workload("rel", batch=3, stride=2, n_q_heads=8, n_kv_heads=2, vocab=256, ctx_min=20, ctx_max=40,
                 logits_dtype="f32", steps=2, seed=12)
    st, eng, out = _fresh(w)
    s_np = state_to_np(st)
    slots = torch.tensor([2, 0], dtype=torch.int32, device=DEV)
    eng.isd_release(st, slots)
    torch.cuda.synchronize()
    oracle.release(N=w.stride, page_size=16, ctx_len=s_np["ctx_len"], n_ver=s_np["n_ver"],
                   page_table=s_np["page_table"], free_stack=s_np["free_stack"], free_top=s_np["free_top"],
                   active=s_np["active"], slots=[2, 0])
    top = int(s_np["free_top"][0])
    assert st["free_top"].item() == top
    assert np.array_equal(st["free_stack"].cpu().numpy()[:top], s_np["free_stack"][:top])
    assert np.array_equal(st["active"].cpu().numpy(), s_np["active"])
    eng.close()


def test_invalid_arguments_return_error_codes():
    with pytest.raises(isd_pkg.IsdError, match="unsupported"):
        isd_pkg.Isd(batch=1, stride=2, n_q_heads=8, n_kv_heads=2, vocab=64, max_pages_per_slot=4, num_pages=8,
                    logits_dtype="f32", head_dim=64)
    with pytest.raises(isd_pkg.IsdError, match="unsupported"):
        isd_pkg.Isd(batch=1, stride=16, n_q_heads=64, n_kv_heads=8, vocab=64, max_pages_per_slot=4, num_pages=8,
                    logits_dtype="f32")
    with pytest.raises(isd_pkg.IsdError, match="invalid"):
        isd_pkg.Isd(batch=0, stride=2, n_q_heads=8, n_kv_heads=2, vocab=64, max_pages_per_slot=4, num_pages=8,
                    logits_dtype="f32")


@pytest.mark.parametrize("seed", [300, 301, 302])
@pytest.mark.parametrize("propose_mode,q_mode,N,B", [(1, 1, 8, 1), (0, 0, 4, 2), (1, 0, 16, 1), (0, 0, 2, 3), (1, 1, 4, 20)])
def test_small_batches_at_the_full_vocabulary(seed, propose_mode, q_mode, N, B):
    # Small batches take other launch shapes than the benchmark's batch: a row of the row pass is cut into up to
    # sixteen CTAs (one partial per CTA, merged in chunks at the head of the sampling kernel) and a sampled row into
    # up to sixteen pieces; steps that reject make no proposals.  Several seeds, five chained steps each.
    w = Workload("small_full_vocab", batch=B, stride=N, n_q_heads=8, n_kv_heads=2, vocab=151936, ctx_min=3, ctx_max=300,
                 logits_dtype="bf16", logit_sigma=3.0, peaked_frac=0.7, steps=5, propose_mode=propose_mode,
                 q_mode=q_mode, seed=seed)
    rep = run_chain_parity(w, steps=5, device=DEV)
    assert_clean(rep)
