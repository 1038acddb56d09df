"""isd_verify_static: the verification entry point for callers that cannot allocate device memory.

Some hosts of the library (an engine whose own allocator owns all free device memory, a thread on
which allocation is forbidden) cannot go through isd_create, which owns isd_verify's scratch.  The
static variant keeps that scratch in a fixed array inside the library.  This test drives it through
the C ABI on two calls in a row and checks every output against isd_verify's on the same inputs.
It is collected last so that a failure here cannot hide the other GPU tests.
"""
import numpy as np
import pytest
import torch

import paper_2604_11035_b200 as isd_pkg
from paper_2604_11035_b200 import workloads as wl
from paper_2604_11035_b200.workloads import Workload

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _compare(ref, new, tag):
    for name in ("accept", "accept_len", "n_emit", "repl_tok", "out_tok", "new_prop_tok"):
        assert torch.equal(ref[name], new[name]), (tag, name)
    ev = ref["accept"] >= 0
    assert torch.allclose(ref["alpha"][ev], new["alpha"][ev], atol=2e-2, rtol=0), tag
    assert torch.allclose(ref["new_q_stats"], new["new_q_stats"], atol=2e-2, rtol=0), tag


@pytest.mark.parametrize("dtype,propose_mode", [("bf16", 0), ("f32", 1)])
def test_static_verify_matches_isd_verify_on_consecutive_calls(dtype, propose_mode):
    w = Workload("noalloc", batch=24, stride=4, n_q_heads=8, n_kv_heads=2, vocab=8192 + 64, ctx_min=20, ctx_max=300,
                 logits_dtype=dtype, logit_sigma=2.0, peaked_frac=0.5, steps=4, propose_mode=propose_mode, seed=91)
    st = wl.make_state(w, DEV)
    eng = isd_pkg.isd_for_workload(w, st)
    ref = isd_pkg.alloc_verify_out(w.batch, w.stride, DEV)
    new = isd_pkg.alloc_verify_out(w.batch, w.stride, DEV)
    prev = None
    saw_reject = False
    for t in range(3):                                   # NP step, then two P steps back to back
        lg = wl.make_logits(w, t, st["ctx_len"])
        for o in new.values():
            o.fill_(-7)                                  # stale contents must not leak through
        eng.isd_verify(st, lg, prev, t, ref)
        isd_pkg.isd_verify_static(eng.cfg, st, lg, prev, t, new)
        torch.cuda.synchronize()
        _compare(ref, new, f"step {t}")
        saw_reject |= bool((ref["accept"] == 0).any())
        assert int(st["slot_status"].abs().sum()) == 0
        eng.isd_commit(st, ref)                          # advance the state for the next call
        prev = lg
    assert saw_reject, "the workload should exercise the residual pass as well"
    eng.close()


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
