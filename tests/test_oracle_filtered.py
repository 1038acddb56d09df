"""Pins for the top-k / top-p filtered verification of the oracle (CPU only).

The paper's serving configuration samples with temperature, top-k = 50 and top-p = 0.95
(appendix, sampling configuration tables); Algorithm 1 itself is stated on plain softmax laws.
The filtered variant applies Algorithm 1 to the filtered, renormalised laws.  Expectations come
from the definition of the filter written a second, independent way (a full sort in numpy), from
its limiting cases (k = V with p = 1 is no filter; k = 1 is greedy decoding) and from the laws the
acceptance rule preserves.
"""
import numpy as np

import oracle
from helpers import oracle_step, tiny_state
from test_oracle_verify import chi2_p, rows_from_probs, softmax32, wl_tiny


def filtered_law_by_sorting(row, top_k, top_p):
    """Support and probabilities of the filtered law: stable full sort, cumulative sum, renormalise."""
    row = np.asarray(row, np.float64)
    order = np.lexsort((np.arange(len(row)), -row))          # value descending, then index ascending
    kept = order[:top_k]
    w = np.exp(row[kept] - row[kept[0]])
    cum = np.cumsum(w)
    reached = np.nonzero(cum >= top_p * w.sum())[0]
    n = int(reached[0]) + 1 if len(reached) else len(kept)
    p = np.zeros(len(row))
    p[kept[:n]] = w[:n] / w[:n].sum()
    return p


def test_support_matches_an_independent_sort_based_filter_including_ties():
    rng = np.random.default_rng(3)
    for trial in range(200):
        V = int(rng.integers(2, 300))
        row = np.round(rng.normal(0, 2.5, V) * 4) / 4       # quantised: many exact ties
        k = int(rng.integers(1, min(V, 64) + 1))
        p = float(rng.choice([0.3, 0.5, 0.8, 0.95, 1.0]))
        got = oracle.filter_row(row, k, p)
        want = filtered_law_by_sorting(row, k, p)
        assert np.array_equal(np.isfinite(got), want > 0), (trial, V, k, p)
        assert np.array_equal(got[np.isfinite(got)], row[np.isfinite(got)])   # kept entries are untouched


def test_nucleus_is_the_shortest_prefix_that_reaches_top_p():
    rng = np.random.default_rng(4)
    for _ in range(100):
        V, k, p = 200, 50, float(rng.uniform(0.2, 0.99))
        row = rng.normal(0, 3, V)
        kept = np.isfinite(oracle.filter_row(row, k, p))
        topk = np.sort(row)[::-1][:k]
        w = np.exp(topk - topk[0])
        n = int(kept.sum())
        assert 1 <= n <= k
        assert w[:n].sum() >= p * w.sum() * (1 - 1e-12)              # reaches top_p of the top-k mass ...
        assert n == 1 or w[:n - 1].sum() < p * w.sum() * (1 + 1e-12)  # ... and no shorter prefix does
        assert np.array_equal(np.sort(row[kept])[::-1], topk[:n])    # and it is a prefix of the top-k order


def _random_two_steps(top_k, top_p, seed, B=300, N=4, V=24, propose_mode=0):
    rng = np.random.default_rng(seed)
    w = wl_tiny(B, N, V, seed, propose_mode)
    Q = 2 * N - 1
    out = []
    s = tiny_state(B, N, V)
    prev = None
    for t in range(3):
        lg = rng.normal(0, 2, (B, Q, V)).astype(np.float32)
        _, _, vr, _ = oracle_step(w, s, None, None, None, lg, prev, t, do_attn=False, top_k=top_k, top_p=top_p)
        out.append(vr)
        prev = lg
    return out, s


def test_no_filter_limit_equals_the_unfiltered_rule():
    a, sa = _random_two_steps(0, 1.0, seed=11)
    b, sb = _random_two_steps(24, 1.0, seed=11)         # k = V keeps everything, p = 1 keeps all of it
    for va, vb in zip(a, b):
        for name in ("accept", "accept_len", "n_emit", "repl_tok", "out_tok", "new_prop_tok"):
            assert np.array_equal(getattr(va, name), getattr(vb, name)), name
        assert np.allclose(va.new_q_stats, vb.new_q_stats, rtol=0, atol=1e-12, equal_nan=True)  # NaN: no proposals made
    for k in ("ctx_len", "n_ver", "block_tok"):
        assert np.array_equal(sa[k], sb[k])


def test_top_k_one_is_greedy_decoding():
    # every law is a point mass on its argmax: proposals are argmaxes, a proposal is accepted iff the
    # anchor's argmax agrees (alpha is 1 or 0), and the replacement / bonus token is the anchor's argmax
    B, N, V = 200, 4, 16
    rng = np.random.default_rng(7)
    w = wl_tiny(B, N, V, 21)
    s = tiny_state(B, N, V)
    l0 = rng.normal(0, 2, (B, 2 * N - 1, V)).astype(np.float32)
    _, _, v0, _ = oracle_step(w, s, None, None, None, l0, None, 0, do_attn=False, top_k=1, top_p=0.9)
    assert np.array_equal(v0.new_prop_tok, l0[:, 1:N].argmax(-1))
    assert np.array_equal(v0.repl_tok, l0[:, 0].argmax(-1))
    l1 = rng.normal(0, 2, (B, 2 * N - 1, V)).astype(np.float32)
    l1[: B // 2, 0] = l0[: B // 2, 1]                   # first anchor agrees with the first proposal law
    _, _, v1, _ = oracle_step(w, s, None, None, None, l1, l0, 1, do_attn=False, top_k=1, top_p=0.9)
    agree0 = l1[:, 0].argmax(-1) == v0.new_prop_tok[:, 0]
    assert np.array_equal(v1.accept[:, 0] == 1, agree0)
    assert np.all(agree0[: B // 2])
    ev = v1.accept >= 0
    assert np.all(np.isin(v1.alpha[ev], (0.0, 1.0)))
    rej = v1.accept_len < N - 1
    rows = np.arange(B)
    assert np.array_equal(v1.repl_tok[rej], l1[rows[rej], v1.accept_len[rej]].argmax(-1))   # residual = anchor's point mass


def test_filtered_laws_of_proposal_bonus_and_finalised_token():
    B, N, V, k, p = 6000, 2, 12, 5, 0.8
    rng = np.random.default_rng(5)
    q_law, p_law, b_law = rng.dirichlet(np.ones(V) * 0.7, size=3)
    wl_ = wl_tiny(B, N, V, 31)
    st = tiny_state(B, N, V)
    pad = np.full(V, 1.0 / V)
    l0 = rows_from_probs(B, N, [pad, q_law, pad])
    _, _, v0, _ = oracle_step(wl_, st, None, None, None, l0, None, 0, do_attn=False, top_k=k, top_p=p)
    qf = filtered_law_by_sorting(np.log(softmax32(l0[0, 1])), k, p)
    assert chi2_p(np.bincount(v0.new_prop_tok[:, 0], minlength=V), qf) > 1e-3        # proposals follow filtered q
    l1 = rows_from_probs(B, N, [p_law, b_law, pad])
    _, _, v1, _ = oracle_step(wl_, st, None, None, None, l1, l0, 1, do_attn=False, top_k=k, top_p=p)
    pf = filtered_law_by_sorting(np.log(softmax32(l1[0, 0])), k, p)
    bf = filtered_law_by_sorting(np.log(softmax32(l1[0, 1])), k, p)
    # the token finalised at the verified position follows the filtered anchor law (losslessness of the rule)
    assert chi2_p(np.bincount(v1.out_tok[:, 0], minlength=V), pf) > 1e-3
    acc = v1.accept[:, 0] == 1
    assert abs(acc.mean() - np.minimum(pf, qf).sum()) < 4 * np.sqrt(0.25 / B)        # P(accept) = sum min(p~, q~)
    assert chi2_p(np.bincount(v1.repl_tok[acc], minlength=V), bf) > 1e-3             # bonus follows its filtered law
    resid = np.maximum(0.0, pf - qf)
    assert chi2_p(np.bincount(v1.repl_tok[~acc], minlength=V), resid) > 1e-3         # replacement follows the residual
