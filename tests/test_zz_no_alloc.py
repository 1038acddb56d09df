"""isd_verify_static: the verification entry point for callers that cannot allocate device memory.

Some hosts of the library (an engine whose own allocator owns all free device memory, a thread on
which allocation is forbidden) cannot go through isd_create, which owns isd_verify's scratch.  The
static variant keeps that scratch in a fixed array inside the library.  These tests drive it through
the C ABI on calls in a row and check every output against isd_verify's on the same inputs and
against the fp64 oracle, at the layout's upper bounds as well, and that the call leaves the amount
of free device memory alone.  The file is collected last so that a failure here cannot hide the
other GPU tests.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2604_11035_b200 as isd_pkg
from helpers import abs_diff_nan_aware, logits_np, state_to_np
from paper_2604_11035_b200 import workloads as wl
from paper_2604_11035_b200.workloads import Workload

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _compare(ref, new, tag):
    for name in ("accept", "accept_len", "n_emit", "repl_tok", "out_tok", "new_prop_tok"):
        assert torch.equal(ref[name], new[name]), (tag, name)
    ev = ref["accept"] >= 0
    assert torch.allclose(ref["alpha"][ev], new["alpha"][ev], atol=2e-2, rtol=0), tag
    assert torch.allclose(ref["new_q_stats"], new["new_q_stats"], atol=2e-2, rtol=0, equal_nan=True), tag  # NaN: no proposals made


def _oracle_verify(w, st, lg, prev, t):
    """The oracle's verification of the same step, from the state and logits the GPU call sees."""
    s = state_to_np(st)
    return oracle.verify(
        N=w.stride, V=w.vocab, logits_dtype=0 if w.logits_dtype == "f32" else 1, q_mode=w.q_mode,
        propose_mode=w.propose_mode, inv_temperature=1.0, tau=0.0, seed=w.seed, step=t, n_ver=s["n_ver"],
        active=s["active"], block_tok=s["block_tok"], q_row0=s["q_row0"], logits_cur=logits_np(lg),
        q_prev=None if prev is None else logits_np(prev), slot_status=s["slot_status"])


def _compare_with_oracle(w, new, vr, tag):
    g = {k: v.cpu().numpy() for k, v in new.items()}
    near = (vr.accept >= 0) & (np.abs(vr.alpha - vr.u) < 1e-4)
    assert not near.any(), "pick another seed: an acceptance test sits within 1e-4 of its uniform draw"
    for name in ("accept", "accept_len", "n_emit", "repl_tok", "out_tok", "new_prop_tok"):
        assert np.array_equal(g[name], getattr(vr, name)), (tag, name)
    ev = vr.accept >= 0
    assert np.abs(g["alpha"][ev] - vr.alpha[ev]).max(initial=0.0) < 2e-2, tag
    assert abs_diff_nan_aware(g["new_q_stats"], vr.new_q_stats).max() < 2e-2, tag


def _chain(w, steps, check_free_memory=False):
    st = wl.make_state(w, DEV)
    eng = isd_pkg.isd_for_workload(w, st)
    ref = isd_pkg.alloc_verify_out(w.batch, w.stride, DEV)
    new = isd_pkg.alloc_verify_out(w.batch, w.stride, DEV)
    prev = None
    rejections = 0
    for t in range(steps):                               # NP step, then P steps back to back
        lg = wl.make_logits(w, t, st["ctx_len"])
        for o in new.values():
            o.fill_(-7)                                  # stale contents must not leak through
        vr = _oracle_verify(w, st, lg, prev, t)
        eng.isd_verify(st, lg, prev, t, ref)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        isd_pkg.isd_verify_static(eng.cfg, st, lg, prev, t, new)
        torch.cuda.synchronize()
        if check_free_memory and t > 0:                  # (the first call on a device resolves the array's address)
            assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the free device memory"
        _compare(ref, new, f"step {t}")
        _compare_with_oracle(w, new, vr, f"step {t}")
        rejections += int((ref["accept"] == 0).sum())
        assert int(st["slot_status"].abs().sum()) == 0
        eng.isd_commit(st, ref)                          # advance the state for the next call
        prev = lg
    eng.close()
    return rejections


@pytest.mark.parametrize("dtype,propose_mode", [("bf16", 0), ("f32", 1)])
def test_static_verify_matches_isd_verify_and_the_oracle_on_consecutive_calls(dtype, propose_mode):
    w = Workload("noalloc", batch=24, stride=4, n_q_heads=8, n_kv_heads=2, vocab=8192 + 64, ctx_min=20, ctx_max=300,
                 logits_dtype=dtype, logit_sigma=2.0, peaked_frac=0.5, steps=4, propose_mode=propose_mode, seed=91)
    assert _chain(w, 3, check_free_memory=True) > 0, "the workload should exercise the residual pass as well"


def test_static_verify_at_the_bounds_of_its_layout_then_a_small_call():
    # the array is laid out for 64 slots, 31 block rows and 16 pieces per row: a call at those bounds (a short
    # vocabulary keeps the oracle quick; 16 pieces need >= 16 x 8192 elements, so the piece bound is reached by the
    # next case), then a small call that finds the big one's contents in the array
    big = Workload("noalloc_bounds", batch=64, stride=16, n_q_heads=8, n_kv_heads=2, vocab=4096, ctx_min=20, ctx_max=200,
                   logits_dtype="f32", logit_sigma=2.0, peaked_frac=0.7, steps=4, propose_mode=0, seed=93)
    assert _chain(big, 3) > 0
    wide = Workload("noalloc_pieces", batch=2, stride=2, n_q_heads=8, n_kv_heads=2, vocab=16 * 8192, ctx_min=20, ctx_max=60,
                    logits_dtype="bf16", logit_sigma=2.0, peaked_frac=0.5, steps=4, propose_mode=0, seed=94)
    _chain(wide, 3)                                      # 6 rows on 148 SMs: every row is cut into 16 pieces
    small = Workload("noalloc_small", batch=3, stride=3, n_q_heads=8, n_kv_heads=2, vocab=1024, ctx_min=20, ctx_max=60,
                     logits_dtype="f32", logit_sigma=2.0, peaked_frac=0.5, steps=4, propose_mode=1, seed=95)
    _chain(small, 3)


def test_static_verify_rejects_batches_beyond_its_capacity():
    w = Workload("noalloc_big", batch=65, stride=2, n_q_heads=8, n_kv_heads=2, vocab=256, ctx_min=8, ctx_max=16,
                 logits_dtype="f32", steps=2, seed=92)
    st = wl.make_state(w, DEV)
    eng = isd_pkg.isd_for_workload(w, st)
    out = isd_pkg.alloc_verify_out(w.batch, w.stride, DEV)
    lg = wl.make_logits(w, 0, st["ctx_len"])
    with pytest.raises(isd_pkg.IsdError, match="ISD_STATIC_MAX_BATCH"):
        isd_pkg.isd_verify_static(eng.cfg, st, lg, None, 0, out)
    eng.close()
