"""Pins for the oracle's verify / propose / commit chain (CPU only).

Every expectation here comes from the paper's statements or from mathematics,
never from the oracle itself: the p/q rule's closed forms, the laws the rule is
proved to preserve, brute-force products on tiny vocabularies, the TPF closed
form (Eq. 3) and the worked example of the step-by-step figure.
"""
import os

import numpy as np
import pytest
import scipy.special
import scipy.stats

import oracle
from helpers import oracle_step, tiny_state
from paper_2604_11035_b200.workloads import Workload

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def wl_tiny(B, N, V, seed, propose_mode=0, q_mode=0):
    return Workload("t", batch=B, stride=N, vocab=V, logits_dtype="f32", propose_mode=propose_mode,
                    q_mode=q_mode, seed=seed)


def rows_from_probs(B, N, probs_by_row):
    """[B, Q, V] fp32 logits whose row r is log(probs_by_row[r]) for every slot."""
    Q = 2 * N - 1
    lg = np.log(np.asarray(probs_by_row, dtype=np.float64))
    assert lg.shape[0] == Q
    return np.ascontiguousarray(np.broadcast_to(lg[None], (B,) + lg.shape)).astype(np.float32)


def softmax32(row):
    """Law actually encoded by fp32 logits."""
    r = np.asarray(row, np.float32).astype(np.float64)
    e = np.exp(r - r.max())
    return e / e.sum()


def chi2_p(counts, probs):
    counts, probs = np.asarray(counts, float), np.asarray(probs, float)
    keep = probs > 0
    assert counts[~keep].sum() == 0
    return scipy.stats.chisquare(counts[keep], probs[keep] / probs[keep].sum() * counts[keep].sum()).pvalue


def two_step(B, N, V, q_rows, p_rows, seed, propose_mode=0, tau=0.0, q_mode=0):
    """Step 0 = NP step proposing from q_rows (rows 1..N-1), step 1 = P step judging with p_rows."""
    Q = 2 * N - 1
    w = wl_tiny(B, N, V, seed, propose_mode, q_mode)
    s = tiny_state(B, N, V)
    pad = [np.full(V, 1.0 / V)] * Q
    l0 = rows_from_probs(B, N, ([pad[0]] + list(q_rows) + pad)[:Q])
    _, _, v0, _ = oracle_step(w, s, None, None, None, l0, None, 0, do_attn=False)
    assert np.all(s["n_ver"] == N - 1) and np.all(s["q_row0"] == 1)
    l1 = rows_from_probs(B, N, (list(p_rows) + pad)[:Q])
    s_before = {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in s.items()}
    _, _, v1, _ = oracle_step(w, s, None, None, None, l1, l0, 1, do_attn=False, tau=tau)
    return w, s_before, s, v0, v1, l0, l1


# --------------------------------------------------------------------------- accept rule
def test_identical_laws_always_accept():
    # "For AR models p = q by construction, yielding alpha = 1" (Sec. 2): ratio 1 accepts for every u.
    B, N, V = 4000, 4, 8
    rng = np.random.default_rng(1)
    laws = rng.dirichlet(np.ones(V), size=N - 1)
    _, _, s, v0, v1, _, _ = two_step(B, N, V, laws, list(laws) + [np.full(V, 1 / V)], seed=5)
    assert np.all(v1.accept == 1) and np.all(v1.accept_len == N - 1) and np.all(v1.n_emit == N)
    assert np.allclose(v1.alpha, 1.0)
    assert np.all(s["n_ver"] == N - 1)
    assert np.array_equal(v1.out_tok[:, :N - 1], v0.new_prop_tok)


def test_zero_anchor_probability_never_accepts():
    B, N, V = 3000, 2, 4
    q = np.array([0.7, 0.1, 0.1, 0.1])
    w = wl_tiny(B, N, V, 9, propose_mode=1)     # argmax proposals: always token 0
    s = tiny_state(B, N, V)
    l0 = rows_from_probs(B, N, [np.full(V, .25), q, np.full(V, .25)])
    oracle_step(w, s, None, None, None, l0, None, 0, do_attn=False)
    assert np.all(s["block_tok"][:, 1] == 0)
    l1 = rows_from_probs(B, N, [np.full(V, .25)] * 3)
    l1[:, 0, 0] = -np.inf                        # p(x^) = 0
    _, _, v1, _ = oracle_step(w, s, None, None, None, l1, l0, 1, do_attn=False)
    assert np.all(v1.accept[:, 0] == 0) and np.all(v1.accept_len == 0) and np.all(v1.n_emit == 1)
    assert np.all(v1.alpha[:, 0] == 0.0)
    assert np.all(v1.repl_tok != 0)              # residual excludes the rejected token
    assert np.all(s["n_ver"] == 0)               # next step is a pure stride


def test_accept_decision_is_u_below_ratio_and_counts_match():
    # accept iff u < min(1, p(x)/q(x)), u on the 2^-24 lattice (Algorithm 1, strict <)
    B, N, V = 20000, 2, 4
    q = np.array([0.4, 0.3, 0.2, 0.1])
    p = np.array([0.1, 0.2, 0.3, 0.4])
    w, sb, s, v0, v1, l0, l1 = two_step(B, N, V, [q], [p, np.full(V, .25)], seed=21)
    p32, q32 = softmax32(l1[0, 0]), softmax32(l0[0, 1])
    x = v0.new_prop_tok[:, 0]
    ratio = np.minimum(1.0, p32[x] / q32[x])
    assert np.allclose(v1.alpha[:, 0], ratio, rtol=1e-12)
    u = np.array([oracle.uniform(w.seed, 1, b, 1) for b in range(B)])
    assert np.array_equal(v1.u[:, 0], u)
    assert np.array_equal(v1.accept[:, 0] == 1, u < ratio)
    # closed form: for fixed alpha exactly ceil(alpha * 2^24) lattice points accept
    for tok in range(V):
        a = ratio[x == tok][0]
        thresh = int(np.ceil(a * 2 ** 24))
        k = (u[x == tok] * 2 ** 24).astype(np.int64)
        assert np.array_equal(v1.accept[x == tok, 0] == 1, k < thresh)
    # mean acceptance over x^ ~ q equals sum_i min(p_i, q_i)
    want = np.minimum(p32, q32).sum()
    got = (v1.accept[:, 0] == 1).mean()
    assert abs(got - want) < 4 * np.sqrt(want * (1 - want) / B)


def test_relaxed_acceptance_is_monotone_in_tau():
    B, N, V = 5000, 3, 8
    rng = np.random.default_rng(3)
    q = rng.dirichlet(np.ones(V), size=N - 1)
    p = rng.dirichlet(np.ones(V), size=N)
    lens = []
    for tau in (0.0, 0.5, 1.0):
        _, _, _, v0, v1, l0, l1 = two_step(B, N, V, q, p, seed=33, tau=tau)
        lens.append(v1.accept_len.copy())
        x = v0.new_prop_tok[:, 0]
        ratio = np.minimum(1.0, (1 + tau) * softmax32(l1[0, 0])[x] / softmax32(l0[0, 1])[x])
        assert np.allclose(v1.alpha[:, 0], ratio, rtol=1e-6)
    assert np.all(lens[0] <= lens[1]) and np.all(lens[1] <= lens[2])
    assert lens[2].sum() > lens[0].sum()


# --------------------------------------------------------------------------- laws
def test_proposal_residual_final_and_bonus_laws():
    B, N, V = 120000, 2, 4
    q = np.array([0.50, 0.25, 0.15, 0.10])
    p = np.array([0.20, 0.20, 0.35, 0.25])
    bonus = np.array([0.1, 0.6, 0.1, 0.2])
    free = np.array([0.3, 0.3, 0.2, 0.2])
    Q = 3
    w = wl_tiny(B, N, V, 77)
    s = tiny_state(B, N, V)
    l0 = rows_from_probs(B, N, [free, q, np.full(V, .25)])
    _, _, v0, _ = oracle_step(w, s, None, None, None, l0, None, 0, do_attn=False)
    l1 = rows_from_probs(B, N, [p, bonus, np.full(V, .25)])
    _, _, v1, _ = oracle_step(w, s, None, None, None, l1, l0, 1, do_attn=False)
    p32, q32 = softmax32(l1[0, 0]), softmax32(l0[0, 1])
    cnt = lambda t: np.bincount(t, minlength=V)
    # NP step: the free token is an exact AR sample of row 0 (Algorithm 1, "quality-guaranteed")
    assert chi2_p(cnt(v0.repl_tok), softmax32(l0[0, 0])) > 1e-3
    assert np.all(v0.n_emit == 1) and np.all(v0.accept_len == 0)
    # proposals follow q
    assert chi2_p(cnt(v0.new_prop_tok[:, 0]), q32) > 1e-3
    rej = v1.accept[:, 0] == 0
    acc = ~rej
    # on rejection the replacement follows normalize(max(0, p - q)) and avoids tokens with p <= q
    resid = np.maximum(0.0, p32 - q32)
    assert chi2_p(cnt(v1.repl_tok[rej]), resid) > 1e-3
    # the finalised token at the judged position follows p exactly (losslessness)
    assert chi2_p(cnt(v1.out_tok[:, 0]), p32) > 1e-3
    # all accepted -> bonus token from the final anchor row
    assert chi2_p(cnt(v1.repl_tok[acc]), softmax32(l1[0, 1])) > 1e-3
    assert np.all(v1.n_emit[acc] == 2) and np.all(v1.n_emit[rej] == 1)
    assert np.all(v1.out_tok[acc, 0] == v0.new_prop_tok[acc, 0])
    assert np.all(v1.out_tok[rej, 1] == -1)


def test_two_token_vocab_residual_is_a_point_mass():
    B, N, V = 4000, 2, 2
    _, _, _, v0, v1, _, _ = two_step(B, N, V, [np.array([0.8, 0.2])], [np.array([0.3, 0.7]), np.array([.5, .5])], seed=4)
    rej = v1.accept[:, 0] == 0
    assert rej.sum() > 100
    assert np.all(v0.new_prop_tok[rej, 0] == 0)   # only the over-proposed token can be rejected
    assert np.all(v1.repl_tok[rej] == 1)


def test_one_hot_q_mode():
    # argmax proposals judged against a point mass: accept w.p. p(x^); residual = p without x^
    B, N, V = 60000, 2, 4
    p = np.array([0.55, 0.25, 0.15, 0.05])
    w = wl_tiny(B, N, V, 13, propose_mode=1, q_mode=1)
    s = tiny_state(B, N, V)
    l0 = rows_from_probs(B, N, [np.full(V, .25), np.array([0.4, 0.3, 0.2, 0.1]), np.full(V, .25)])
    oracle_step(w, s, None, None, None, l0, None, 0, do_attn=False)
    l1 = rows_from_probs(B, N, [p, np.full(V, .25), np.full(V, .25)])
    _, _, v1, _ = oracle_step(w, s, None, None, None, l1, None, 1, do_attn=False)
    p32 = softmax32(l1[0, 0])
    acc = v1.accept[:, 0] == 1
    assert abs(acc.mean() - p32[0]) < 4 * np.sqrt(p32[0] * (1 - p32[0]) / B)
    resid = p32.copy(); resid[0] = 0
    assert chi2_p(np.bincount(v1.repl_tok[~acc], minlength=V), resid) > 1e-3
    assert chi2_p(np.bincount(v1.out_tok[:, 0], minlength=V), p32) > 1e-3


# --------------------------------------------------------------------------- prefix structure / brute force
def test_prefix_structure_bounds_and_brute_force_products():
    B, N, V = 100000, 3, 3
    rng = np.random.default_rng(8)
    q = rng.dirichlet(np.ones(V) * 2, size=N - 1)
    p = rng.dirichlet(np.ones(V) * 2, size=N)
    _, sb, s, v0, v1, l0, l1 = two_step(B, N, V, q, p, seed=99)
    acc = v1.accept
    for b in range(0, B, 997):
        row = list(acc[b])
        k = v1.accept_len[b]
        assert row[:k] == [1] * k
        if k < N - 1:
            assert row[k] == 0 and row[k + 1:] == [-1] * (N - 2 - k)
    assert v1.accept_len.min() >= 0 and v1.accept_len.max() <= N - 1
    assert np.array_equal(v1.n_emit, v1.accept_len + 1)
    assert v1.n_emit.min() >= 1 and v1.n_emit.max() <= N
    # brute force: P(a >= j) = prod_{k <= j} sum_i min(p_k,i , q_k,i)
    prod = 1.0
    for j in range(1, N):
        prod *= np.minimum(softmax32(l1[0, j - 1]), softmax32(l0[0, j])).sum()
        got = (v1.accept_len >= j).mean()
        assert abs(got - prod) < 4.5 * np.sqrt(prod * (1 - prod) / B), (j, got, prod)
    # joint law of (a, y) by enumeration for a = 0: P(a=0, y) = residual_1(y) * (1 - sum min)
    p1, q1 = softmax32(l1[0, 0]), softmax32(l0[0, 1])
    joint = np.maximum(0, p1 - q1)
    sel = v1.accept_len == 0
    emp = np.bincount(v1.repl_tok[sel], minlength=V) / B
    assert np.all(np.abs(emp - joint) < 4.5 * np.sqrt(np.maximum(joint, 1e-4) / B))
    # state machine after the step
    allacc = v1.accept_len == sb["n_ver"]
    assert np.array_equal(s["n_ver"], np.where(allacc, N - 1, 0))
    assert np.array_equal(s["ctx_len"], sb["ctx_len"] + v1.n_emit)
    assert np.array_equal(s["block_tok"][:, 0], v1.repl_tok)


# --------------------------------------------------------------------------- worked example + TPF
def _golden_rows():
    rows = []
    for line in open(os.path.join(GOLDEN, "isd_steps_figure.txt")):
        if line.strip() and not line.startswith("#"):
            f = line.split()
            rows.append((f[0],) + tuple(int(x) for x in f[1:]))
    return rows


@pytest.mark.parametrize("case", _golden_rows(), ids=lambda c: c[0])
def test_step_by_step_figure(case):
    name, N, n_ver, rejected, want_a, want_emit, want_next, want_growth = case
    B, V, Q = 3, 8, 2 * N - 1
    w = wl_tiny(B, N, V, 1, propose_mode=1)
    s = tiny_state(B, N, V)
    law = np.array([0.3, 0.2, 0.1, 0.1, 0.1, 0.1, 0.05, 0.05])
    l0 = rows_from_probs(B, N, [law] * Q)
    oracle_step(w, s, None, None, None, l0, None, 0, do_attn=False)
    if n_ver == 0:
        s = tiny_state(B, N, V)      # judge the bootstrap step itself
        ctx0 = s["ctx_len"].copy()
        _, _, v, _ = oracle_step(w, s, None, None, None, l0, None, 0, do_attn=False)
    else:
        ctx0 = s["ctx_len"].copy()
        l1 = rows_from_probs(B, N, [law] * Q)     # identical laws: accepted ...
        if rejected:
            l1[:, rejected - 1, 0] = -np.inf       # ... except one proposal with p(x^) = 0
        _, _, v, _ = oracle_step(w, s, None, None, None, l1, l0, 1, do_attn=False)
    assert np.all(v.accept_len == want_a) and np.all(v.n_emit == want_emit)
    assert np.all(s["n_ver"] == want_next)
    assert np.all(s["ctx_len"] - ctx0 == want_growth)
    mask = V - 1
    if want_next == 0:   # "propose only": anchor followed by MASK rows
        assert np.all(s["block_tok"][:, 1:] == mask)
    else:                # next block = [bonus, fresh proposals, MASK...]
        assert np.array_equal(s["block_tok"][:, 1:N], v.new_prop_tok)
        assert np.all(s["block_tok"][:, N:] == mask)


def tpf_closed_form(N, c):
    # Eq. 3 with uniform per-position acceptance c
    return sum([2.0] + [c ** k for k in range(1, N - 1)]) / (2.0 - c ** (N - 1))


@pytest.mark.parametrize("N,c", [(2, 0.9), (4, 0.9), (8, 0.9), (4, 1.0), (4, 0.0), (3, 0.5)])
def test_free_running_chain_matches_tpf_closed_form(N, c):
    B, V, steps, Q = 300, 2, 240, 2 * N - 1
    if c == 0.0:
        p_law, q_law = np.array([1.0, 1e-30]), np.array([1e-30, 1.0])
    else:
        d = (1.0 - c) / 2
        p_law, q_law = np.array([0.5 + d, 0.5 - d]), np.array([0.5 - d, 0.5 + d])
    w = wl_tiny(B, N, V, 1234 + N)
    s = tiny_state(B, N, V, ctx=16, pages_per_slot=(16 + steps * N + Q) // 16 + 3)
    lp, lq = np.log(p_law).astype(np.float32), np.log(q_law).astype(np.float32)
    prev = None
    emitted = 0
    for t in range(steps):
        rows = np.arange(Q)[None, :]
        clean = rows <= s["n_ver"][:, None]            # anchor + proposals give p, MASK rows give q
        cur = np.where(clean[:, :, None], lp[None, None, :], lq[None, None, :]).astype(np.float32)
        cur = np.ascontiguousarray(cur)
        _, _, v, _ = oracle_step(w, s, None, None, None, cur, prev, t, do_attn=False)
        assert np.all(s["slot_status"] == 0)
        emitted += int(v.n_emit.sum())
        prev = cur
    tpf = emitted / (B * steps)
    want = tpf_closed_form(N, c)
    if c in (0.0, 1.0):
        # limits stated with Eq. 3: TPF = N at p = 1 and 1 at p = 0 (first NP step costs a little)
        assert abs(tpf - want) < N / steps + 1e-9
    else:
        assert abs(tpf - want) < 0.035, (tpf, want)


# --------------------------------------------------------------------------- temperature
def _softmax64(x):
    x = np.asarray(x, np.float64)
    e = np.exp(x - x.max())
    return e / e.sum()


@pytest.mark.parametrize("inv_t", [0.5, 2.0])
def test_temperature_scales_both_laws_before_the_ratio_and_the_draws(inv_t):
    # Sampling configuration of the appendix (temperature T): every law is softmax(logits / T).  The ratio
    # and the Gumbel-max draws are written out here in numpy from the raw fp32 logits; scaling only one of
    # the two laws, or dividing where the oracle multiplies by 1/T, changes alpha and the token laws.
    B, N, V = 60000, 3, 6
    Q = 2 * N - 1
    rng = np.random.default_rng(int(inv_t * 10))
    raw0 = rng.normal(0, 1.5, (Q, V)).astype(np.float32)
    raw1 = rng.normal(0, 1.5, (Q, V)).astype(np.float32)
    l0 = np.ascontiguousarray(np.broadcast_to(raw0[None], (B, Q, V)))
    l1 = np.ascontiguousarray(np.broadcast_to(raw1[None], (B, Q, V)))
    w = wl_tiny(B, N, V, 55)
    s = tiny_state(B, N, V)
    _, _, v0, _ = oracle_step(w, s, None, None, None, l0, None, 0, do_attn=False, inv_temperature=inv_t)
    cnt = lambda t: np.bincount(t, minlength=V)
    # NP step: free token from row 0, proposals from MASK rows 1..N-1, all at temperature T
    assert chi2_p(cnt(v0.repl_tok), _softmax64(raw0[0].astype(np.float64) * inv_t)) > 1e-3
    for m in range(1, N):
        assert chi2_p(cnt(v0.new_prop_tok[:, m - 1]), _softmax64(raw0[m].astype(np.float64) * inv_t)) > 1e-3
    # a wrong exponent would be visible: the same counts do not fit the untempered law
    assert chi2_p(cnt(v0.repl_tok), _softmax64(raw0[0])) < 1e-6
    _, _, v1, _ = oracle_step(w, s, None, None, None, l1, l0, 1, do_attn=False, inv_temperature=inv_t)
    x = v0.new_prop_tok[:, 0]
    p = _softmax64(raw1[0].astype(np.float64) * inv_t)
    q = _softmax64(raw0[1].astype(np.float64) * inv_t)
    assert np.allclose(v1.alpha[:, 0], np.minimum(1.0, p[x] / q[x]), rtol=1e-12)
    # second position, where it was evaluated
    ev = v1.accept[:, 1] >= 0
    x2 = v0.new_prop_tok[:, 1]
    p2 = _softmax64(raw1[1].astype(np.float64) * inv_t)
    q2 = _softmax64(raw0[2].astype(np.float64) * inv_t)
    assert ev.sum() > 1000
    assert np.allclose(v1.alpha[ev, 1], np.minimum(1.0, p2[x2[ev]] / q2[x2[ev]]), rtol=1e-12)
    # losslessness at temperature T: the finalised first token follows the tempered anchor law
    assert chi2_p(cnt(v1.out_tok[:, 0]), p) > 1e-3
    rej = v1.accept[:, 0] == 0
    assert chi2_p(cnt(v1.repl_tok[rej]), np.maximum(0.0, p - q)) > 1e-3
    assert not np.any(s["slot_status"] & oracle.ST_EMPTY_RESIDUAL)


# --------------------------------------------------------------------------- cached proposal-law statistics
@pytest.mark.parametrize("propose_mode", [0, 1])
@pytest.mark.parametrize("inv_t,top_k,top_p", [(1.0, 0, 1.0), (0.7, 0, 1.0), (1.3, 5, 0.8)])
def test_proposal_law_statistics_are_lse_and_logit_of_the_mask_rows(propose_mode, inv_t, top_k, top_p):
    # new_q_stats[b, m-1] = {LSE(row * invT), row[x^] * invT} of MASK row n_ver + m (the two scalars the next
    # step's accept test uses instead of re-reading the row); with a filter on, of the filtered law's support.
    B, N, V = 7, 4, 40
    Q = 2 * N - 1
    rng = np.random.default_rng(17 + propose_mode)
    lg = rng.normal(0, 2.0, (B, Q, V)).astype(np.float32)
    w = wl_tiny(B, N, V, 3, propose_mode=propose_mode)
    for n_ver in (0, N - 1):
        s = tiny_state(B, N, V, n_ver=n_ver)
        s["block_tok"][:, 1:n_ver + 1] = rng.integers(0, V, (B, n_ver))
        prev = rng.normal(0, 2.0, (B, Q, V)).astype(np.float32)
        # even slots: the proposal law of every proposal is the law that judges it (p / q = 1: all accepted);
        # odd slots: unrelated laws and random proposals (rejected, except by luck)
        for j in range(1, n_ver + 1):
            prev[0::2, int(s["q_row0"][0]) + j - 1] = lg[0::2, j - 1]
            s["block_tok"][0::2, j] = lg[0::2, j - 1].argmax(-1)   # inside the support of any filter
        q_stats_before = s["q_stats"].copy()
        _, _, v, _ = oracle_step(w, s, None, None, None, lg, prev, 4, do_attn=False, inv_temperature=inv_t,
                                 top_k=top_k, top_p=top_p)
        proposes = v.accept_len == n_ver
        assert np.all(proposes[0::2]) and (n_ver == 0 or not np.all(proposes[1::2]))
        for b in range(B):
            if not proposes[b]:
                # Sec. 3.2 (adaptive stride): after a rejection the later tokens are discarded and the next step is
                # a pure stride step, so no proposals are made from MASK rows conditioned on them
                assert np.all(v.new_prop_tok[b] == -1) and np.all(np.isnan(v.new_q_stats[b]))
                assert s["n_ver"][b] == 0 and np.array_equal(s["q_stats"][b], q_stats_before[b])
                continue
            for m in range(1, N):
                row = lg[b, n_ver + m].astype(np.float64) * float(np.float32(inv_t))
                if top_k:
                    order = np.lexsort((np.arange(V), -row))[:top_k]
                    wgt = np.exp(row[order] - row[order[0]])
                    reached = np.nonzero(np.cumsum(wgt) >= float(np.float32(top_p)) * wgt.sum())[0]
                    keep = order[:int(reached[0]) + 1 if len(reached) else len(order)]
                    support = np.zeros(V, bool)
                    support[keep] = True
                    row = np.where(support, row, -np.inf)
                xh = int(v.new_prop_tok[b, m - 1])
                assert np.isfinite(row[xh])
                if propose_mode == 1:
                    assert xh == int(np.argmax(row))
                assert abs(v.new_q_stats[b, m - 1, 0] - scipy.special.logsumexp(row)) < 1e-12
                assert v.new_q_stats[b, m - 1, 1] == row[xh]
            # and the next step's accept test consumes exactly these two numbers through commit
            assert np.array_equal(s["q_stats"][b], v.new_q_stats[b])
            assert np.array_equal(s["block_tok"][b, 1:N], v.new_prop_tok[b])


# --------------------------------------------------------------------------- data faults
def test_verify_status_branches_and_frozen_slots():
    # Data faults never abort: an out-of-range proposal id or a NaN / +inf logit sets its bit on the slot,
    # the commit leaves that slot where it was, and its neighbours advance.
    B, N, V = 5, 3, 16
    Q = 2 * N - 1
    rng = np.random.default_rng(2)
    w = wl_tiny(B, N, V, 8)
    s = tiny_state(B, N, V)
    l0 = rng.normal(0, 1, (B, Q, V)).astype(np.float32)
    oracle_step(w, s, None, None, None, l0, None, 0, do_attn=False)
    assert np.all(s["n_ver"] == N - 1)
    l1 = rng.normal(0, 1, (B, Q, V)).astype(np.float32)
    s["block_tok"][1, 1] = V + 2          # proposal id outside the vocabulary
    s["block_tok"][2, 2] = -1             # negative id (reached only if the first proposal is accepted)
    l1[3, 0, 5] = np.nan                  # NaN in an anchor row
    l1[4, N, 0] = np.inf                  # +inf in a MASK row (-inf would be legal)
    before = {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in s.items()}
    _, _, v, _ = oracle_step(w, s, None, None, None, l1, l0, 1, do_attn=False)
    st = s["slot_status"]
    assert st[0] == 0
    assert st[1] == oracle.ST_BAD_TOKEN_ID
    # the faulty slot's outputs stay at their defaults
    assert v.n_emit[1] == 0 and v.accept_len[1] == 0 and v.repl_tok[1] == -1
    assert np.all(v.out_tok[1] == -1) and np.all(v.new_prop_tok[1] == -1) and np.all(v.accept[1] == -1)
    if v.accept[2, 0] == 1:
        assert st[2] == oracle.ST_BAD_TOKEN_ID and v.n_emit[2] == 0
    else:
        assert st[2] == 0 and v.n_emit[2] == 1   # the loop stopped at the rejection before the bad id
    assert st[3] & oracle.ST_NONFINITE_LOGIT and st[4] & oracle.ST_NONFINITE_LOGIT
    for b in (1, 3, 4):                   # frozen by the commit: lengths, roles, block and pages unchanged
        for k in ("ctx_len", "n_ver", "q_row0"):
            assert s[k][b] == before[k][b], (b, k)
        assert np.array_equal(s["block_tok"][b], before["block_tok"][b])
        assert np.array_equal(s["page_table"][b], before["page_table"][b])
    assert s["ctx_len"][0] == before["ctx_len"][0] + v.n_emit[0] and v.n_emit[0] >= 1
    # -inf is a legal logit (probability zero), not a fault
    s2 = tiny_state(B, N, V)
    l2 = rng.normal(0, 1, (B, Q, V)).astype(np.float32)
    l2[:, :, 3] = -np.inf
    _, _, v2, _ = oracle_step(w, s2, None, None, None, l2, None, 0, do_attn=False)
    assert np.all(s2["slot_status"] == 0) and np.all(v2.repl_tok != 3) and np.all(v2.new_prop_tok != 3)
