"""Pins for the oracle's segment-gated LoRA linear layer (CPU only).

R-ISD (Sec. 3.2, "h_j <- W x_j + 1[j in M] BA x_j"): the LoRA residual is applied on [MASK] rows only, so that
clean rows are computed with the base weights alone.  Expectations: the two limiting gates reduce to a plain
linear layer with the base weights and with the merged weights W + s BA (the identity LoRA merging rests on),
every row depends on its own gate only, and a loop written element by element agrees on a small case.
"""
import numpy as np

import oracle


def _case(M=12, N=10, K=16, R=4, seed=0):
    rng = np.random.default_rng(seed)
    return (rng.normal(size=(M, K)), rng.normal(size=(N, K)), rng.normal(size=(R, K)), rng.normal(size=(N, R)),
            rng.integers(0, 2, M).astype(np.uint8))


def test_gate_off_is_the_base_layer_and_gate_on_is_the_merged_layer():
    x, w, a, b, _ = _case()
    s = 0.37
    off = oracle.lora_linear(x, w, a, b, np.zeros(len(x), np.uint8), s)
    on = oracle.lora_linear(x, w, a, b, np.ones(len(x), np.uint8), s)
    assert np.allclose(off, np.einsum("mk,nk->mn", x, w), rtol=0, atol=1e-12)
    merged = w + s * np.einsum("nr,rk->nk", b, a)
    assert np.allclose(on, np.einsum("mk,nk->mn", x, merged), rtol=0, atol=1e-11)


def test_rows_are_gated_independently():
    x, w, a, b, gate = _case(seed=3)
    s = 1.5
    y = oracle.lora_linear(x, w, a, b, gate, s)
    off = oracle.lora_linear(x, w, a, b, np.zeros_like(gate), s)
    on = oracle.lora_linear(x, w, a, b, np.ones_like(gate), s)
    assert gate.any() and not gate.all()
    assert np.array_equal(y[gate == 0], off[gate == 0])
    assert np.allclose(y[gate == 1], on[gate == 1], rtol=0, atol=1e-12)


def test_element_by_element_loop_on_a_small_case():
    x, w, a, b, gate = _case(M=5, N=4, K=6, R=3, seed=5)
    s = -0.8
    y = oracle.lora_linear(x, w, a, b, gate, s)
    for m in range(5):
        for n in range(4):
            base = sum(w[n, k] * x[m, k] for k in range(6))
            lora = sum(b[n, r] * sum(a[r, k] * x[m, k] for k in range(6)) for r in range(3))
            assert abs(y[m, n] - (base + (s * lora if gate[m] else 0.0))) < 1e-12
