"""Pins for the oracle's attention and commit/allocator (CPU only)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import bits16, oracle_step, state_to_np, tiny_state
from paper_2604_11035_b200 import workloads as wl
from paper_2604_11035_b200.workloads import Workload


def small_wl(B=3, N=3, Hq=4, Hkv=2, ctx=(5, 70), seed=0, **kw):
    return Workload("a", batch=B, stride=N, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=128, vocab=64,
                    ctx_min=ctx[0], ctx_max=ctx[1], logits_dtype="f32", seed=seed, **kw)


def f32(bits):
    return torch.from_numpy(bits.astype(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()


def run_attn(w, s, q, k, v, n_ver=None, scale=None):
    if n_ver is not None:
        s["n_ver"][:] = n_ver
    q_len = (s["n_ver"] + w.stride).astype(np.int32)
    out, lse = oracle.attn(Hq=w.n_q_heads, Hkv=w.n_kv_heads, D=w.head_dim, page_size=16,
                           num_pages=s["num_pages"], sm_scale=scale or 1 / np.sqrt(w.head_dim),
                           ctx_len=s["ctx_len"], q_len=q_len, active=s["active"], page_table=s["page_table"],
                           q=q, k_new=k, v_new=v, k_pool=s["k_pool"], v_pool=s["v_pool"],
                           slot_status=s["slot_status"])
    return out, lse, q_len


def gather_kv(w, s, b, pool, new, upto):
    """Logical KV rows 0..upto-1 of slot b as [Hkv, upto, D] fp64, through the page table."""
    ctx = int(s["ctx_len"][b])
    rows = []
    for j in range(upto):
        if j < ctx:
            page = s["page_table"][b, j // 16]
            rows.append(f32(pool[page, :, j % 16, :]))
        else:
            rows.append(f32(new[b, j - ctx]))
    return np.stack(rows, axis=1)


@pytest.mark.parametrize("n_ver", [0, 2])
def test_attention_matches_torch_sdpa_fp64(n_ver):
    w = small_wl()
    st = wl.make_state(w, "cpu")
    s = state_to_np(st)
    q, k, v = [bits16(t) for t in wl.make_qkv(w, 0, "cpu")]
    kp0, vp0 = s["k_pool"].copy(), s["v_pool"].copy()
    out, lse, q_len = run_attn(w, s, q, k, v, n_ver=n_ver)
    G = w.n_q_heads // w.n_kv_heads
    for b in range(w.batch):
        ctx, ql = int(s["ctx_len"][b]), int(q_len[b])
        K = torch.from_numpy(gather_kv(w, s, b, kp0, k, ctx + ql)).repeat_interleave(G, dim=0)
        Vv = torch.from_numpy(gather_kv(w, s, b, vp0, v, ctx + ql)).repeat_interleave(G, dim=0)
        Qq = torch.from_numpy(f32(q[b, :ql])).permute(1, 0, 2)           # [Hq, ql, D]
        mask = torch.arange(ctx + ql)[None, :] <= (ctx + torch.arange(ql))[:, None]
        ref = torch.nn.functional.scaled_dot_product_attention(Qq, K, Vv, attn_mask=mask)
        assert np.allclose(out[b, :ql], ref.permute(1, 0, 2).numpy(), rtol=1e-10, atol=1e-12)
        sc = torch.einsum("hqd,hkd->hqk", Qq, K) / np.sqrt(w.head_dim)
        ref_lse = torch.logsumexp(sc.masked_fill(~mask, -np.inf), dim=-1)
        assert np.allclose(lse[b, :ql], ref_lse.T.numpy(), rtol=1e-12)
        assert np.all(np.isnan(out[b, ql:]))                              # padding rows untouched
    # K/V append: block rows land bit-exactly at positions ctx .. ctx+q_len-1, nothing else moves
    kp, vp = kp0.copy(), vp0.copy()
    for b in range(w.batch):
        for r in range(int(q_len[b])):
            pos = int(s["ctx_len"][b]) + r
            page = s["page_table"][b, pos // 16]
            kp[page, :, pos % 16, :] = k[b, r]
            vp[page, :, pos % 16, :] = v[b, r]
    assert np.array_equal(kp, s["k_pool"]) and np.array_equal(vp, s["v_pool"])
    # reading the appended rows back from the pages gives the same attention (paged-only view)
    s2 = dict(s); s2["ctx_len"] = (s["ctx_len"] + q_len).astype(np.int32); s2["n_ver"] = s["n_ver"].copy()
    w1 = Workload("d", batch=w.batch, stride=1, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads, vocab=64)
    for r in range(w.stride + n_ver):
        s3 = dict(s2); s3["ctx_len"] = (s["ctx_len"] + r).astype(np.int32)
        s3["k_pool"], s3["v_pool"] = s["k_pool"].copy(), s["v_pool"].copy()
        s3["n_ver"] = np.zeros(w.batch, np.int32); s3["slot_status"] = np.zeros(w.batch, np.uint32)
        o1, _, _ = run_attn(w1, s3, np.ascontiguousarray(q[:, r:r + 1]), np.ascontiguousarray(k[:, r:r + 1]),
                            np.ascontiguousarray(v[:, r:r + 1]))
        assert np.allclose(o1[:, 0], out[:, r], rtol=1e-10, atol=1e-12)


def test_identical_keys_give_running_mean_of_values():
    # all scores equal -> row r averages exactly the first ctx + r + 1 value rows (causal limit)
    w = small_wl(B=2, N=4, ctx=(20, 40), seed=3)
    s = state_to_np(wl.make_state(w, "cpu"))
    q, k, v = [bits16(t) for t in wl.make_qkv(w, 0, "cpu")]
    one = bits16(torch.ones(1, dtype=torch.bfloat16))[0]
    s["k_pool"][:] = one
    k[:] = one
    vp0 = s["v_pool"].copy()
    out, _, q_len = run_attn(w, s, q, k, v, n_ver=3)
    G = w.n_q_heads // w.n_kv_heads
    for b in range(w.batch):
        ctx = int(s["ctx_len"][b])
        Vv = gather_kv(w, s, b, vp0, v, ctx + int(q_len[b]))
        for r in range(int(q_len[b])):
            for h in range(w.n_q_heads):
                assert np.allclose(out[b, r, h], Vv[h // G, :ctx + r + 1].mean(axis=0), rtol=1e-12, atol=1e-14)


def test_dominant_key_reveals_paging_gqa_and_causal_reach():
    # one key per (slot, kv head) gets a huge score; values encode (logical index, kv head)
    w = small_wl(B=2, N=3, Hq=4, Hkv=2, ctx=(40, 60), seed=5)
    s = state_to_np(wl.make_state(w, "cpu"))
    bf = lambda x: bits16(torch.tensor(x, dtype=torch.bfloat16))
    q = np.zeros((w.batch, w.Q, w.n_q_heads, 128), np.uint16); q[..., 0] = bf([32.0])[0]
    k = np.zeros((w.batch, w.Q, w.n_kv_heads, 128), np.uint16)
    v = np.zeros_like(k)
    s["k_pool"][:] = 0
    G = w.n_q_heads // w.n_kv_heads
    for b in range(w.batch):
        ctx = int(s["ctx_len"][b])
        for j in range(ctx):
            page = s["page_table"][b, j // 16]
            for g in range(w.n_kv_heads):
                s["v_pool"][page, g, j % 16, :] = 0
                s["v_pool"][page, g, j % 16, 0] = bf([float(j)])[0]
                s["v_pool"][page, g, j % 16, 1] = bf([float(g + 1)])[0]
        for r in range(w.Q):
            for g in range(w.n_kv_heads):
                v[b, r, g, 0] = bf([float(ctx + r)])[0]
                v[b, r, g, 1] = bf([float(g + 1)])[0]
    # hot key: committed position 17 for kv head 0; block row 1 for kv head 1
    for b in range(w.batch):
        page = s["page_table"][b, 17 // 16]
        s["k_pool"][page, 0, 17 % 16, 0] = bf([32.0])[0]
        k[b, 1, 1, 0] = bf([32.0])[0]
    out, _, q_len = run_attn(w, s, q, k, v, n_ver=2, scale=1.0)
    for b in range(w.batch):
        ctx = int(s["ctx_len"][b])
        for r in range(int(q_len[b])):
            for h in range(w.n_q_heads):
                g = h // G
                assert abs(out[b, r, h, 1] - (g + 1)) < 1e-9            # GQA head mapping
                if g == 0:
                    assert abs(out[b, r, h, 0] - 17.0) < 1e-6           # page-table lookup
                elif r >= 1:
                    assert abs(out[b, r, h, 0] - (ctx + 1)) < 1e-6      # own block row is visible
                else:                                                   # row 0 cannot see row 1
                    assert abs(out[b, r, h, 0] - (ctx + 0) / 2.0) < 1e-6   # mean of indices 0..ctx


def test_page_permutation_leaves_result_bit_identical():
    w = small_wl(seed=7)
    s = state_to_np(wl.make_state(w, "cpu"))
    q, k, v = [bits16(t) for t in wl.make_qkv(w, 0, "cpu")]
    s2 = {a: (b.copy() if isinstance(b, np.ndarray) else b) for a, b in s.items()}
    perm = np.random.default_rng(0).permutation(s["num_pages"]).astype(np.int32)   # old id -> new id
    s2["k_pool"][perm] = s["k_pool"]
    s2["v_pool"][perm] = s["v_pool"]
    s2["page_table"] = np.where(s["page_table"] >= 0, perm[np.maximum(s["page_table"], 0)], -1).astype(np.int32)
    o1, l1, _ = run_attn(w, s, q, k, v, n_ver=1)
    o2, l2, _ = run_attn(w, s2, q, k, v, n_ver=1)
    assert np.array_equal(o1, o2, equal_nan=True) and np.array_equal(l1, l2, equal_nan=True)


def test_bad_page_id_sets_status_not_crash():
    w = small_wl(seed=9)
    s = state_to_np(wl.make_state(w, "cpu"))
    q, k, v = [bits16(t) for t in wl.make_qkv(w, 0, "cpu")]
    s["page_table"][1, 0] = s["num_pages"] + 5
    out, _, _ = run_attn(w, s, q, k, v)
    assert s["slot_status"][1] & oracle.ST_BAD_PAGE_ID
    assert np.all(np.isnan(out[1])) and not np.any(np.isnan(out[0, :w.stride]))


# --------------------------------------------------------------------------- commit / allocator
def check_conservation(s, Q):
    owned = []
    for b in range(len(s["ctx_len"])):
        if s["active"][b]:
            n = (int(s["ctx_len"][b]) + Q + 15) // 16
            owned += list(s["page_table"][b, :n])
    free = list(s["free_stack"][:int(s["free_top"][0])])
    allp = owned + free
    assert len(set(allp)) == len(allp), "a page is owned twice"
    assert set(allp) == set(range(s["num_pages"])), "a page leaked"


def test_commit_allocator_against_dictionary_model():
    B, N, V = 6, 4, 16
    Q = 2 * N - 1
    rng = np.random.default_rng(2)
    s = tiny_state(B, N, V, ctx=9, pages_per_slot=6)     # 32-page pool
    assert s["num_pages"] <= 40
    check_conservation(s, Q)
    model_free = list(s["free_stack"][:int(s["free_top"][0])])
    model_tab = {b: list(s["page_table"][b, :(9 + Q + 15) // 16]) for b in range(B)}
    model_ctx = {b: 9 for b in range(B)}
    for t in range(60):
        a = rng.integers(0, N, B).astype(np.int32)
        a = np.minimum(a, s["n_ver"]).astype(np.int32)
        repl = rng.integers(0, V, B).astype(np.int32)
        newp = rng.integers(0, V, (B, N - 1)).astype(np.int32)
        nq = rng.normal(size=(B, N - 1, 2))
        before = {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in s.items()}
        oracle.commit(N=N, page_size=16, mask_token=V - 1, ctx_len=s["ctx_len"], n_ver=s["n_ver"],
                      block_tok=s["block_tok"], q_row0=s["q_row0"], q_stats=s["q_stats"],
                      page_table=s["page_table"], free_stack=s["free_stack"], free_top=s["free_top"],
                      active=s["active"], slot_status=s["slot_status"], accept_len=a, repl_tok=repl,
                      new_prop_tok=newp, new_q_stats=nq)
        for b in range(B):   # plain-dict allocator: pop from the top of the stack, slots ascending
            if before["slot_status"][b]:
                assert s["ctx_len"][b] == before["ctx_len"][b]           # frozen
                continue
            want_ctx = model_ctx[b] + int(a[b]) + 1
            want_pages = (want_ctx + Q + 15) // 16
            if want_pages > s["page_table"].shape[1]:
                assert s["slot_status"][b] & oracle.ST_SLOT_CAPACITY
                assert s["ctx_len"][b] == before["ctx_len"][b]
                continue
            need = want_pages - len(model_tab[b])
            if need > len(model_free):
                assert s["slot_status"][b] & oracle.ST_POOL_EXHAUSTED
                model_free = []      # later requests fail as well (served requests are a prefix)
                continue
            for _ in range(need):
                model_tab[b].append(model_free.pop())
            model_ctx[b] = want_ctx
            assert s["ctx_len"][b] == want_ctx
            assert list(s["page_table"][b, :want_pages]) == model_tab[b]
            assert s["n_ver"][b] == (N - 1 if a[b] == before["n_ver"][b] else 0)
            assert s["q_row0"][b] == before["n_ver"][b] + 1
            assert s["block_tok"][b, 0] == repl[b]
            # the proposal-law statistics follow the proposals: kept when the proposals are (nothing rejected),
            # otherwise no proposals were made and the old ones stay
            if a[b] == before["n_ver"][b]:
                assert np.array_equal(s["q_stats"][b], nq[b])
                assert np.array_equal(s["block_tok"][b, 1:N], newp[b])
            else:
                assert np.array_equal(s["q_stats"][b], before["q_stats"][b])
                assert np.all(s["block_tok"][b, 1:N] == V - 1)
        if not np.any(s["slot_status"] & oracle.ST_POOL_EXHAUSTED):
            assert list(s["free_stack"][:int(s["free_top"][0])]) == model_free
            check_conservation(s, Q)
    assert np.any(s["slot_status"] != 0), "the test should drive the pool or a slot to its limit"


def test_commit_keeps_committed_kv_and_release_returns_pages():
    w = small_wl(B=4, N=3, ctx=(10, 50), seed=11, steps=6)
    s = state_to_np(wl.make_state(w, "cpu"))
    w = Workload(**{**w.__dict__, "propose_mode": 0})
    prev = None
    hist = {b: [] for b in range(w.batch)}       # logical KV rows every slot should hold
    for b in range(w.batch):
        for j in range(int(s["ctx_len"][b])):
            hist[b].append(s["k_pool"][s["page_table"][b, j // 16], :, j % 16, :].copy())
    for t in range(6):
        q, k, v = [bits16(x) for x in wl.make_qkv(w, t, "cpu")]
        lg = wl.make_logits(w, t, torch.from_numpy(s["ctx_len"])).numpy()
        _, _, vr, q_len = oracle_step(w, s, q, k, v, lg, prev, t)
        prev = lg
        for b in range(w.batch):
            hist[b] += [k[b, r].copy() for r in range(int(vr.n_emit[b]))]   # anchor + accepted rows
            assert len(hist[b]) == s["ctx_len"][b]
            for j, row in enumerate(hist[b]):
                assert np.array_equal(s["k_pool"][s["page_table"][b, j // 16], :, j % 16, :], row)
        check_conservation(s, w.Q)
    top = int(s["free_top"][0])
    owned = (int(s["ctx_len"][1]) + w.Q + 15) // 16
    oracle.release(N=w.stride, page_size=16, ctx_len=s["ctx_len"], n_ver=s["n_ver"], page_table=s["page_table"],
                   free_stack=s["free_stack"], free_top=s["free_top"], active=s["active"], slots=[1])
    assert s["free_top"][0] == top + owned and s["active"][1] == 0
    check_conservation(s, w.Q)
