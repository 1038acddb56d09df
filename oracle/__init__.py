"""ctypes loader for the fp64 CPU oracle of the ISD step (``isd_oracle.c``).

TEST INFRASTRUCTURE ONLY: importable from ``tests/``, from the smoke check and
from the benchmark's CPU-baseline leg.  The CUDA library and its Python binding
never import this package, and this package never imports them.

All arrays are numpy, host memory.  bf16 data travels as ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "isd_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

ST_POOL_EXHAUSTED = 1
ST_SLOT_CAPACITY = 2
ST_BAD_TOKEN_ID = 4
ST_BAD_PAGE_ID = 8
ST_NONFINITE_LOGIT = 16
ST_EMPTY_RESIDUAL = 32

TAG_ACCEPT, TAG_FINAL, TAG_PROPOSE = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (fp64, OpenMP) if the shared object is stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra",
             "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_uniform.restype = C.c_double
        _lib.orc_uniform.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32]
        _lib.orc_gumbel.restype = C.c_double
        _lib.orc_gumbel.argtypes = [C.c_uint64] + [C.c_uint32] * 5
        _lib.orc_logsumexp.restype = C.c_double
        _lib.orc_logsumexp.argtypes = [C.c_void_p, C.c_int]
        _lib.orc_set_threads.argtypes = [C.c_int]
        _lib.orc_max_threads.restype = C.c_int
        _lib.orc_get_threads.restype = C.c_int
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _chk(a, dtype, shape=None):
    assert isinstance(a, np.ndarray) and a.dtype == dtype and a.flags.c_contiguous, (a.dtype, dtype)
    if shape is not None:
        assert tuple(a.shape) == tuple(shape), (a.shape, shape)
    return a


def set_threads(n: int) -> None:
    lib().orc_set_threads(int(n))


def max_threads() -> int:
    return int(lib().orc_max_threads())


def philox4x32_10(ctr, key):
    c = (C.c_uint32 * 4)(*[int(x) & 0xFFFFFFFF for x in ctr])
    k = (C.c_uint32 * 2)(*[int(x) & 0xFFFFFFFF for x in key])
    o = (C.c_uint32 * 4)()
    lib().orc_philox4x32_10(c, k, o)
    return [int(x) for x in o]


def uniform(seed, step, slot, position) -> float:
    return float(lib().orc_uniform(seed, step, slot, position))


def gumbel(seed, step, slot, tag, position, vocab_index) -> float:
    return float(lib().orc_gumbel(seed, step, slot, tag, position, vocab_index))


def logsumexp(row) -> float:
    row = np.ascontiguousarray(row, dtype=np.float64)
    return float(lib().orc_logsumexp(_p(row), row.shape[0]))


@dataclass
class VerifyResult:
    accept: np.ndarray        # [B, N-1] int8
    alpha: np.ndarray         # [B, N-1] f64
    u: np.ndarray             # [B, N-1] f64
    accept_len: np.ndarray    # [B] i32
    n_emit: np.ndarray        # [B] i32
    repl_tok: np.ndarray      # [B] i32
    out_tok: np.ndarray       # [B, N] i32
    new_prop_tok: np.ndarray  # [B, N-1] i32
    new_q_stats: np.ndarray   # [B, N-1, 2] f64
    final_margin: np.ndarray  # [B] f64
    prop_margin: np.ndarray   # [B, N-1] f64


def filter_row(row, top_k, top_p):
    """Top-k then top-p filtered law of a scaled fp64 row: a copy with -inf outside the support."""
    r = np.ascontiguousarray(np.array(row, dtype=np.float64))
    f = lib().orc_filter_row
    f.restype = None
    f.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_double]
    f(_p(r), r.shape[0], int(top_k), float(top_p))
    return r


def verify(*, N, V, logits_dtype, q_mode, propose_mode, inv_temperature, tau, seed, step,
           n_ver, active, block_tok, q_row0, logits_cur, q_prev, slot_status, top_k=0, top_p=1.0) -> VerifyResult:
    """Algorithm 1's introspection loop, bonus branch and stride loop for every slot (top_k > 0: on the
    top-k / top-p filtered laws)."""
    B = n_ver.shape[0]
    Q, NP = 2 * N - 1, N - 1
    ldt = np.float32 if logits_dtype == 0 else np.uint16
    _chk(n_ver, np.int32, (B,)); _chk(active, np.uint8, (B,)); _chk(block_tok, np.int32, (B, Q))
    _chk(q_row0, np.int32, (B,)); _chk(logits_cur, ldt, (B, Q, V)); _chk(slot_status, np.uint32, (B,))
    if q_prev is not None:
        _chk(q_prev, ldt, (B, Q, V))
    r = VerifyResult(
        accept=np.zeros((B, NP), np.int8), alpha=np.zeros((B, NP)), u=np.zeros((B, NP)),
        accept_len=np.zeros(B, np.int32), n_emit=np.zeros(B, np.int32), repl_tok=np.zeros(B, np.int32),
        out_tok=np.zeros((B, N), np.int32), new_prop_tok=np.zeros((B, NP), np.int32),
        new_q_stats=np.zeros((B, NP, 2)), final_margin=np.zeros(B), prop_margin=np.zeros((B, NP)))
    f = lib().orc_verify_filtered
    f.restype = C.c_int
    f.argtypes = [C.c_int, C.c_double] + [C.c_int] * 6 + [C.c_double, C.c_double, C.c_uint64, C.c_uint32] + [C.c_void_p] * 18
    rc = f(int(top_k), float(np.float32(top_p)), B, N, V, logits_dtype, q_mode, propose_mode, float(np.float32(inv_temperature)),
           float(np.float32(tau)), seed, step,
           _p(n_ver), _p(active), _p(block_tok), _p(q_row0), _p(logits_cur), _p(q_prev),
           _p(r.accept), _p(r.alpha), _p(r.u), _p(r.accept_len), _p(r.n_emit), _p(r.repl_tok),
           _p(r.out_tok), _p(r.new_prop_tok), _p(r.new_q_stats), _p(r.final_margin),
           _p(r.prop_margin), _p(slot_status))
    assert rc == 0, rc
    return r


def attn(*, Hq, Hkv, D, page_size, num_pages, sm_scale, ctx_len, q_len, active, page_table,
         q, k_new, v_new, k_pool, v_pool, slot_status, want_lse=True):
    """Strict-causal attention of every block row (plain definition) + K/V append in place.

    Returns (out [B,Q,Hq,D] f64, lse [B,Q,Hq] f64); rows >= q_len stay NaN.
    """
    B, Q = q.shape[0], q.shape[1]
    max_pages = page_table.shape[1]
    _chk(ctx_len, np.int32, (B,)); _chk(q_len, np.int32, (B,)); _chk(active, np.uint8, (B,))
    _chk(page_table, np.int32, (B, max_pages)); _chk(q, np.uint16, (B, Q, Hq, D))
    _chk(k_new, np.uint16, (B, Q, Hkv, D)); _chk(v_new, np.uint16, (B, Q, Hkv, D))
    _chk(k_pool, np.uint16, (num_pages, Hkv, page_size, D)); _chk(v_pool, np.uint16, (num_pages, Hkv, page_size, D))
    _chk(slot_status, np.uint32, (B,))
    out = np.full((B, Q, Hq, D), np.nan)
    lse = np.full((B, Q, Hq), np.nan) if want_lse else None
    f = lib().orc_attn
    f.restype = C.c_int
    f.argtypes = [C.c_int] * 8 + [C.c_double] + [C.c_void_p] * 12
    rc = f(B, Q, Hq, Hkv, D, page_size, max_pages, num_pages, float(sm_scale),
           _p(ctx_len), _p(q_len), _p(active), _p(page_table), _p(q), _p(k_new), _p(v_new),
           _p(k_pool), _p(v_pool), _p(out), _p(lse), _p(slot_status))
    assert rc == 0, rc
    return out, lse


def commit(*, N, page_size, mask_token, ctx_len, n_ver, block_tok, q_row0, q_stats, page_table,
           free_stack, free_top, active, slot_status, accept_len, repl_tok, new_prop_tok, new_q_stats):
    """KV commit / rollback, next-step block and page acquisition, in place."""
    B = ctx_len.shape[0]
    Q, NP = 2 * N - 1, N - 1
    max_pages = page_table.shape[1]
    _chk(ctx_len, np.int32, (B,)); _chk(n_ver, np.int32, (B,)); _chk(block_tok, np.int32, (B, Q))
    _chk(q_row0, np.int32, (B,)); _chk(q_stats, np.float64, (B, NP, 2)); _chk(page_table, np.int32)
    _chk(free_stack, np.int32); _chk(free_top, np.int32, (1,)); _chk(active, np.uint8, (B,))
    _chk(slot_status, np.uint32, (B,)); _chk(accept_len, np.int32, (B,)); _chk(repl_tok, np.int32, (B,))
    _chk(new_prop_tok, np.int32, (B, NP)); _chk(new_q_stats, np.float64, (B, NP, 2))
    f = lib().orc_commit
    f.restype = C.c_int
    f.argtypes = [C.c_int] * 5 + [C.c_void_p] * 14
    rc = f(B, N, page_size, max_pages, mask_token, _p(ctx_len), _p(n_ver), _p(block_tok), _p(q_row0),
           _p(q_stats), _p(page_table), _p(free_stack), _p(free_top), _p(active), _p(slot_status),
           _p(accept_len), _p(repl_tok), _p(new_prop_tok), _p(new_q_stats))
    assert rc == 0, rc


def release(*, N, page_size, ctx_len, n_ver, page_table, free_stack, free_top, active, slots):
    B = ctx_len.shape[0]
    slots = np.ascontiguousarray(slots, dtype=np.int32)
    f = lib().orc_release
    f.restype = C.c_int
    f.argtypes = [C.c_int] * 4 + [C.c_void_p] * 7 + [C.c_int]
    rc = f(B, N, page_size, page_table.shape[1], _p(ctx_len), _p(n_ver), _p(page_table),
           _p(free_stack), _p(free_top), _p(active), _p(slots), slots.shape[0])
    assert rc == 0, rc


def lora_linear(x, w, a, b, gate, scale):
    """Segment-gated LoRA linear layer of the lossless R-ISD variant (Eq. 5 and the R-ISD paragraph of Sec. 3.2):
    row j of the output is W x_j, plus scale * B A x_j only where gate[j] is set (the [MASK] rows); clean rows see
    the base weights alone, which is what makes their verification lossless.  Plain fp64 definition:
    x [M, K], w [N, K], a [R, K], b [N, R], gate [M] -> y [M, N]."""
    x, w, a, b = (np.asarray(t, np.float64) for t in (x, w, a, b))
    g = (np.asarray(gate) != 0).astype(np.float64)[:, None]
    return x @ w.T + g * float(scale) * ((x @ a.T) @ b.T)
