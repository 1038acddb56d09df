"""Segment-gated LoRA linear layer on the tensor cores vs the fp64 oracle (needs a B200)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2604_11035_b200 as isd_pkg
from paper_2604_11035_b200 import workloads as wl
from paper_2604_11035_b200.workloads import Workload

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _engine():
    w = Workload("lora", batch=1, stride=2, n_q_heads=8, n_kv_heads=2, vocab=1024, ctx_min=16, ctx_max=16, steps=1)
    st = wl.make_state(w, DEV)
    return isd_pkg.isd_for_workload(w, st)


def _inputs(M, N, K, R, seed):
    g = torch.Generator(device=DEV)
    g.manual_seed(seed)
    bf = lambda *shape, s=1.0: (torch.randn(*shape, generator=g, device=DEV) * s).to(torch.bfloat16)
    x, w, a, b = bf(M, K), bf(N, K, s=K ** -0.5), bf(R, K, s=K ** -0.5), bf(N, R, s=R ** -0.5)
    gate = (torch.rand(M, generator=g, device=DEV) < 0.5).to(torch.uint8)
    return x, w, a, b, gate


def _f64(t):
    return t.to(torch.float64).cpu().numpy()


def _tolerance(ref, x, a, b, gate, scale):
    """Error bound derived from the arithmetic: fp32 accumulation of exact bf16 products (negligible), the gated
    down-projection t rounded to bf16 once (relative 2^-8 per element, propagated through |b|), and the result
    rounded to bf16 (relative 2^-8 of the value)."""
    t_abs = np.abs((np.asarray(gate)[:, None] != 0) * scale * (x @ a.T))
    through_t = 2.0 ** -8 * (t_abs @ np.abs(b).T)
    return 2.0 ** -8 * (np.abs(ref) + through_t) + through_t + 1e-3


@pytest.mark.parametrize("M,N,K,R", [(200, 96, 128, 64), (128, 256, 64, 64), (517, 544, 448, 192), (1, 32, 64, 64)])
def test_small_and_ragged_shapes(M, N, K, R):
    eng = _engine()
    x, w, a, b, gate = _inputs(M, N, K, R, seed=M + N)
    scale = 0.75
    y = eng.isd_lora_linear(x, w, a, b, gate, scale)
    torch.cuda.synchronize()
    ref = oracle.lora_linear(_f64(x), _f64(w), _f64(a), _f64(b), gate.cpu().numpy(), scale)
    tol = _tolerance(ref, _f64(x), _f64(a), _f64(b), gate.cpu().numpy(), scale)
    err = np.abs(_f64(y) - ref)
    assert (err <= tol).all(), (float(err.max()), np.unravel_index(err.argmax(), err.shape))
    # clean rows see the base weights only: bit-identical to the same call with the adapter gated off everywhere
    y0 = eng.isd_lora_linear(x, w, a, b, torch.zeros_like(gate), scale)
    torch.cuda.synchronize()
    clean = (gate == 0)
    assert torch.equal(y[clean].view(torch.int16), y0[clean].view(torch.int16))
    assert eng.isd_read_status() == 0
    eng.close()


@pytest.mark.parametrize("R", [128, 1024])
def test_model_sized_layer_sampled_rows(R):
    # token rows of the benchmark batch (256 slots x 15 rows), hidden size 4096, the two adapter ranks of the paper
    M, N, K = 3840, 4096, 4096
    eng = _engine()
    x, w, a, b, gate = _inputs(M, N, K, R, seed=9)
    y = eng.isd_lora_linear(x, w, a, b, gate, 0.5)
    torch.cuda.synchronize()
    rows = np.array([0, 1, 127, 128, 1000, 2047, 3000, 3839])
    ref = oracle.lora_linear(_f64(x[rows]), _f64(w), _f64(a), _f64(b), gate.cpu().numpy()[rows], 0.5)
    tol = _tolerance(ref, _f64(x[rows]), _f64(a), _f64(b), gate.cpu().numpy()[rows], 0.5)
    err = np.abs(_f64(y[rows]) - ref)
    assert (err <= tol).all(), float(err.max())
    assert eng.isd_read_status() == 0
    eng.close()


def test_repeated_calls_reuse_the_scratch_and_big_ranks_take_two_launches():
    # The one-launch form hands t from CTA to CTA through readiness flags that every launch must leave cleared:
    # with a stale flag the second K segment would read the previous call's t.  Same buffers, the gate flipped
    # between calls; every call is checked in full.  Rank 512 = two blocks of t per row block, still one launch;
    # rank 320 is neither below one MMA's width nor a multiple of it: two launches.
    eng = _engine()
    for (M, N, K, R), launches in (((300, 288, 256, 128), 1), ((300, 544, 192, 512), 1), ((260, 160, 128, 320), 2)):
        x, w, a, b, gate = _inputs(M, N, K, R, seed=3 * M + R)
        t = torch.empty(M, R, dtype=torch.bfloat16, device=DEV)
        y = torch.empty(M, N, dtype=torch.bfloat16, device=DEV)
        for call in range(3):
            g = gate if call % 2 == 0 else 1 - gate
            n0 = eng.isd_launch_count()
            eng.isd_lora_linear(x, w, a, b, g, 1.25, t=t, y=y)
            torch.cuda.synchronize()
            assert eng.isd_launch_count() - n0 == launches
            ref = oracle.lora_linear(_f64(x), _f64(w), _f64(a), _f64(b), g.cpu().numpy(), 1.25)
            tol = _tolerance(ref, _f64(x), _f64(a), _f64(b), g.cpu().numpy(), 1.25)
            err = np.abs(_f64(y) - ref)
            assert (err <= tol).all(), (M, R, call, float(err.max()))
    assert eng.isd_read_status() == 0
    eng.close()


@pytest.mark.parametrize("M,N,K,R,launches", [(6200, 288, 128, 768, 1), (6200, 544, 192, 320, 2)])
def test_one_cta_form_of_the_kernel(M, N, K, R, launches):
    # The library picks the kernel by shape alone.  Rank 768 at 6200 rows has 25 x 3 blocks of t (256 rows each):
    # more than the 74 CTA pairs, but its 49 x 3 blocks of 128 rows fit the 148 CTAs, so the one-CTA kernel runs
    # with the fused down-projection and the column strips of its last round.  Rank 320 is neither below 256 nor a
    # multiple of it: two launches of the one-CTA kernel, t first.
    eng = _engine()
    x, w, a, b, gate = _inputs(M, N, K, R, seed=7 * M + R)
    n0 = eng.isd_launch_count()
    y = eng.isd_lora_linear(x, w, a, b, gate, 0.6)
    torch.cuda.synchronize()
    assert eng.isd_launch_count() - n0 == launches
    ref = oracle.lora_linear(_f64(x), _f64(w), _f64(a), _f64(b), gate.cpu().numpy(), 0.6)
    tol = _tolerance(ref, _f64(x), _f64(a), _f64(b), gate.cpu().numpy(), 0.6)
    err = np.abs(_f64(y) - ref)
    assert (err <= tol).all(), float(err.max())
    assert eng.isd_read_status() == 0
    eng.close()


def test_captured_layer_replays():
    # the layer is one launch with device-side hand-over counters that each launch leaves cleared, so a captured
    # call can be replayed with new inputs in the same buffers
    M, N, K, R = 300, 288, 256, 128
    eng = _engine()
    x, w, a, b, gate = _inputs(M, N, K, R, seed=11)
    t = torch.empty(M, R, dtype=torch.bfloat16, device=DEV)
    y = torch.empty(M, N, dtype=torch.bfloat16, device=DEV)
    eng.isd_lora_linear(x, w, a, b, gate, 0.5, t=t, y=y)   # warm-up outside the capture (function attributes)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        eng.isd_lora_linear(x, w, a, b, gate, 0.5, t=t, y=y)
    for replay in range(3):
        x2, _, _, _, gate2 = _inputs(M, N, K, R, seed=100 + replay)
        x.copy_(x2)
        gate.copy_(gate2)
        y.zero_()
        graph.replay()
        torch.cuda.synchronize()
        ref = oracle.lora_linear(_f64(x), _f64(w), _f64(a), _f64(b), gate.cpu().numpy(), 0.5)
        tol = _tolerance(ref, _f64(x), _f64(a), _f64(b), gate.cpu().numpy(), 0.5)
        err = np.abs(_f64(y) - ref)
        assert (err <= tol).all(), (replay, float(err.max()))
    assert eng.isd_read_status() == 0
    eng.close()
