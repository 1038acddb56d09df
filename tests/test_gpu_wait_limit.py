"""A device-side wait that runs out returns a status instead of hanging (needs a B200).

Every wait inside the kernels is bounded in time.  Here one is made to run out on purpose, from the
host and without any fault: a readiness counter of the fused LoRA layer is preset to a value its
readers can never see complete, the wait limit is set to 20 ms, and the call must come back with
ISD_ST_KERNEL_TIMEOUT in the status word, leave the context usable, and the next call must be an
ordinary, correct one again.
"""
import time

import numpy as np
import pytest
import torch

import oracle
import paper_2604_11035_b200 as isd_pkg
from paper_2604_11035_b200.binding import ST_KERNEL_TIMEOUT
from test_gpu_lora import _engine, _f64, _inputs, _tolerance

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_reports_a_status_and_the_context_stays_usable():
    # rank 768 at 6200 rows: the one-CTA kernel with the fused down-projection (49 row blocks of t, 3 blocks each)
    M, N, K, R = 6200, 288, 128, 768
    eng = _engine()
    x, w, a, b, gate = _inputs(M, N, K, R, seed=5)
    ref = oracle.lora_linear(_f64(x), _f64(w), _f64(a), _f64(b), gate.cpu().numpy(), 0.6)
    tol = _tolerance(ref, _f64(x), _f64(a), _f64(b), gate.cpu().numpy(), 0.6)
    y0 = eng.isd_lora_linear(x, w, a, b, gate, 0.6)
    torch.cuda.synchronize()
    assert (np.abs(_f64(y0) - ref) <= tol).all() and eng.isd_read_status() == 0

    eng.isd_set_wait_limit(20)
    blk = 3
    eng.isd_test_preset_lora_counter(blk, 0x40000000)     # 0x40000000 + 3 arrivals never equals 3
    t0 = time.time()
    y1 = eng.isd_lora_linear(x, w, a, b, gate, 0.6)
    torch.cuda.synchronize()
    took = time.time() - t0
    status = eng.isd_read_status()
    assert status & ST_KERNEL_TIMEOUT, hex(status)
    assert 0.015 < took < 2.0, took                       # the readers gave up after about the limit, not after seconds
    # rows outside the poisoned block are complete and correct
    rows = np.ones(M, bool)
    rows[blk * 128:(blk + 1) * 128] = False
    assert (np.abs(_f64(y1) - ref)[rows] <= tol[rows]).all()

    # the kernel left its counters cleared: the next call is an ordinary one, identical to the first
    y2 = eng.isd_lora_linear(x, w, a, b, gate, 0.6)
    torch.cuda.synchronize()
    assert eng.isd_read_status() == 0
    assert torch.equal(y2.view(torch.int16), y0.view(torch.int16))
    eng.close()


def test_wait_limit_argument_is_checked():
    eng = _engine()
    with pytest.raises(isd_pkg.IsdError, match="invalid"):
        eng.isd_set_wait_limit(0)
    eng.close()
