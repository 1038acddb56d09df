"""Test helpers: run the CPU oracle on a workload state held as numpy arrays."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2604_11035_b200 import workloads as wl

STATE_KEYS = ("ctx_len", "n_ver", "block_tok", "q_row0", "q_stats", "page_table", "free_stack",
              "free_top", "active", "slot_status")


def bits16(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> uint16 bit patterns on the host."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def logits_np(t: torch.Tensor) -> np.ndarray:
    return bits16(t) if t.dtype == torch.bfloat16 else t.detach().cpu().numpy()


def state_to_np(st: dict) -> dict:
    out = {}
    for k in STATE_KEYS:
        a = st[k].detach().cpu().numpy().copy()
        if k == "slot_status":
            a = a.view(np.uint32)
        if k == "q_stats":
            a = a.astype(np.float64)
        out[k] = a
    out["k_pool"] = bits16(st["k_pool"]).copy()
    out["v_pool"] = bits16(st["v_pool"]).copy()
    out["num_pages"] = st["num_pages"]
    return out


def oracle_step(w: wl.Workload, s: dict, q, k_new, v_new, logits_cur, q_prev, step, *,
                inv_temperature=1.0, tau=0.0, mask_token=None, do_attn=True, sm_scale=None, top_k=None, top_p=None):
    """One full oracle step (attention, verify, commit) on numpy state `s`, in place.

    Returns (attn_out, attn_lse, VerifyResult, q_len_before).
    """
    N = w.stride
    ldt = 0 if w.logits_dtype == "f32" else 1
    top_k = w.top_k if top_k is None else top_k       # the workload's sampling configuration unless overridden
    top_p = w.top_p if top_p is None else top_p
    q_len = np.where(s["active"] != 0, s["n_ver"] + N, 0).astype(np.int32)
    out = lse = None
    if do_attn:
        out, lse = oracle.attn(
            Hq=w.n_q_heads, Hkv=w.n_kv_heads, D=w.head_dim, page_size=wl.PAGE, num_pages=s["num_pages"],
            sm_scale=(sm_scale if sm_scale else 1.0 / np.sqrt(w.head_dim)), ctx_len=s["ctx_len"], q_len=q_len,
            active=s["active"], page_table=s["page_table"], q=q, k_new=k_new, v_new=v_new,
            k_pool=s["k_pool"], v_pool=s["v_pool"], slot_status=s["slot_status"])
    vr = oracle.verify(
        N=N, V=w.vocab, logits_dtype=ldt, q_mode=w.q_mode, propose_mode=w.propose_mode,
        inv_temperature=inv_temperature, tau=tau, seed=w.seed, step=step, n_ver=s["n_ver"],
        active=s["active"], block_tok=s["block_tok"], q_row0=s["q_row0"], logits_cur=logits_cur,
        q_prev=q_prev, slot_status=s["slot_status"], top_k=top_k, top_p=top_p)
    oracle.commit(
        N=N, page_size=wl.PAGE, mask_token=(w.vocab - 1 if mask_token is None else mask_token),
        ctx_len=s["ctx_len"], n_ver=s["n_ver"], block_tok=s["block_tok"], q_row0=s["q_row0"],
        q_stats=s["q_stats"], page_table=s["page_table"], free_stack=s["free_stack"],
        free_top=s["free_top"], active=s["active"], slot_status=s["slot_status"],
        accept_len=vr.accept_len, repl_tok=vr.repl_tok, new_prop_tok=vr.new_prop_tok,
        new_q_stats=vr.new_q_stats)
    return out, lse, vr, q_len


def abs_diff_nan_aware(a, b):
    """|a - b| where NaN means \"not produced\": 0 where both are NaN, inf where only one is."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    na, nb = np.isnan(a), np.isnan(b)
    d = np.abs(np.where(na, 0.0, a) - np.where(nb, 0.0, b))
    return np.where(na & nb, 0.0, np.where(na | nb, np.inf, d))


def tiny_state(B, N, V, *, n_ver=0, ctx=32, pages_per_slot=8, seed=0):
    """Minimal numpy state for verify/commit-only oracle tests (no KV pools)."""
    Q = 2 * N - 1
    NP = N - 1
    rng = np.random.default_rng(seed)
    num_pages = B * pages_per_slot + 4
    have = (ctx + Q + 15) // 16
    pt = np.full((B, pages_per_slot), -1, np.int32)
    ids = rng.permutation(num_pages).astype(np.int32)
    pt[:, :have] = ids[:B * have].reshape(B, have)
    fs = np.full(num_pages, -1, np.int32)
    nfree = num_pages - B * have
    fs[:nfree] = ids[B * have:]
    return dict(
        ctx_len=np.full(B, ctx, np.int32), n_ver=np.full(B, n_ver, np.int32),
        block_tok=np.zeros((B, Q), np.int32), q_row0=np.ones(B, np.int32),
        q_stats=np.zeros((B, NP, 2)), page_table=pt, free_stack=fs,
        free_top=np.array([nfree], np.int32), active=np.ones(B, np.uint8),
        slot_status=np.zeros(B, np.uint32), num_pages=num_pages)


def compare_verify_and_state(w, t, out, st, vr, s, n_ver_before):
    """Bit-exact comparison of the verification outputs and the committed state of every slot."""
    N, Q = w.stride, w.Q
    g = {k: v.cpu().numpy() for k, v in out.items()}
    gst = {k: st[k].cpu().numpy() for k in STATE_KEYS}
    for b in range(w.batch):
        evaluated = vr.accept[b] >= 0
        near = evaluated & (np.abs(vr.alpha[b] - vr.u[b]) < 1e-4)
        assert not near.any(), "pick another seed: an acceptance test sits within 1e-4 of its uniform draw"
        assert np.array_equal(g["accept"][b], vr.accept[b]), (t, b, g["accept"][b], vr.accept[b])
        for name in ("accept_len", "n_emit", "repl_tok", "out_tok", "new_prop_tok"):
            assert np.array_equal(g[name][b], getattr(vr, name)[b]), (t, b, name, g[name][b], getattr(vr, name)[b])
        ev = np.where(evaluated)[0]
        if len(ev):
            assert np.abs(g["alpha"][b][ev] - vr.alpha[b][ev]).max() < 2e-2
        if N > 1:
            assert abs_diff_nan_aware(g["new_q_stats"][b], vr.new_q_stats[b]).max() < 2e-2  # NaN: no proposals made
        for name in ("ctx_len", "n_ver", "q_row0"):
            assert gst[name][b] == s[name][b], (t, b, name)
        assert np.array_equal(gst["block_tok"][b], s["block_tok"][b]), (t, b)
        own = (int(s["ctx_len"][b]) + Q + 15) // 16
        assert np.array_equal(gst["page_table"][b, :own], s["page_table"][b, :own]), (t, b)
    top = int(s["free_top"][0])
    assert gst["free_top"][0] == top and np.array_equal(gst["free_stack"][:top], s["free_stack"][:top])
    assert np.array_equal(gst["slot_status"].view(np.uint32), s["slot_status"])
