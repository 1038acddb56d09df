"""Thin ctypes binding of libisd.so: argument marshalling only.

Every step of the ISD path runs inside the CUDA library; this module turns torch
tensors into device pointers and forwards them.  There is no CPU fallback: if the
library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libisd.so")

ST_POOL_EXHAUSTED, ST_SLOT_CAPACITY, ST_BAD_TOKEN_ID = 1, 2, 4
ST_BAD_PAGE_ID, ST_NONFINITE_LOGIT, ST_EMPTY_RESIDUAL = 8, 16, 32
ST_KERNEL_TIMEOUT = 0x80000000

EXPORTS = ["isd_create", "isd_destroy", "isd_attn", "isd_verify", "isd_commit", "isd_step",
           "isd_release", "isd_read_status", "isd_set_profile_events", "isd_launch_count", "isd_strerror",
           "isd_verify_static", "isd_step_layers", "isd_set_step_counter", "isd_lora_linear", "isd_set_wait_limit",
           "isd_test_preset_lora_counter", "isd_test_lora_work_item", "isd_test_verify_grid"]


class IsdConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "batch", "stride", "n_q_heads", "n_kv_heads", "head_dim", "page_size", "vocab",
        "max_pages_per_slot", "num_pages", "logits_dtype", "q_mode", "propose_mode", "mask_token_id")] + [("sm_scale", C.c_float), ("inv_temperature", C.c_float), ("tau", C.c_float),
                         ("seed", C.c_uint64), ("top_k", C.c_int32), ("top_p", C.c_float)]


class IsdBatchState(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in (
        "ctx_len", "n_ver", "block_tok", "q_row0", "q_stats", "page_table", "free_stack", "free_top",
        "active", "slot_status")]


class IsdVerifyOut(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in (
        "accept", "alpha", "accept_len", "n_emit", "repl_tok", "out_tok", "new_prop_tok", "new_q_stats")]


class IsdStepArgs(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in (
        "q", "k_new", "v_new", "k_pool", "v_pool", "attn_out", "attn_lse", "logits_cur", "q_prev_logits")] + \
        [("out", IsdVerifyOut)]


class IsdLayerArgs(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("q", "k_new", "v_new", "k_pool", "v_pool", "attn_out", "attn_lse")]


class IsdLoraArgs(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("x", "w", "a", "b", "gate", "t", "y")] + \
        [(n, C.c_int32) for n in ("m", "n", "k", "rank")] + [("scale", C.c_float)]


_lib = None


def load():
    """Load libisd.so (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2604_11035_b200.build` "
                               "(there is no fallback path)")
        lib = C.CDLL(LIB_PATH)
        vp = C.c_void_p
        lib.isd_create.argtypes = [C.POINTER(IsdConfig), C.POINTER(vp)]
        lib.isd_destroy.argtypes = [vp]
        lib.isd_attn.argtypes = [vp, C.POINTER(IsdBatchState)] + [vp] * 8
        lib.isd_verify.argtypes = [vp, C.POINTER(IsdBatchState), vp, vp, C.c_uint64, C.POINTER(IsdVerifyOut), vp]
        lib.isd_commit.argtypes = [vp, C.POINTER(IsdBatchState), C.POINTER(IsdVerifyOut), vp]
        lib.isd_step.argtypes = [vp, C.POINTER(IsdBatchState), C.POINTER(IsdStepArgs), C.c_uint64, vp]
        lib.isd_release.argtypes = [vp, C.POINTER(IsdBatchState), vp, C.c_int32, vp]
        lib.isd_read_status.argtypes = [vp, C.POINTER(C.c_uint32), vp]
        lib.isd_set_profile_events.argtypes = [vp] * 5
        lib.isd_set_profile_events.restype = C.c_int
        lib.isd_verify_static.argtypes = [C.POINTER(IsdConfig), C.POINTER(IsdBatchState), vp, vp, C.c_uint64,
                                          C.POINTER(IsdVerifyOut), vp]
        lib.isd_verify_static.restype = C.c_int
        lib.isd_step_layers.argtypes = [vp, C.POINTER(IsdBatchState), C.POINTER(IsdLayerArgs), C.c_int32, vp, vp,
                                        C.POINTER(IsdVerifyOut), C.c_uint64, vp]
        lib.isd_step_layers.restype = C.c_int
        lib.isd_set_step_counter.argtypes = [vp, vp]
        lib.isd_set_step_counter.restype = C.c_int
        lib.isd_lora_linear.argtypes = [vp, C.POINTER(IsdLoraArgs), vp]
        lib.isd_lora_linear.restype = C.c_int
        lib.isd_set_wait_limit.argtypes = [vp, C.c_uint32]
        lib.isd_set_wait_limit.restype = C.c_int
        lib.isd_test_preset_lora_counter.argtypes = [vp, C.c_int32, C.c_uint32, vp]
        lib.isd_test_preset_lora_counter.restype = C.c_int
        lib.isd_test_lora_work_item.argtypes = [C.c_int32] * 6 + [C.POINTER(C.c_int32)]
        lib.isd_test_lora_work_item.restype = C.c_int
        lib.isd_test_verify_grid.argtypes = [C.POINTER(IsdConfig), C.c_int32, C.POINTER(C.c_int32)]
        lib.isd_test_verify_grid.restype = C.c_int
        lib.isd_launch_count.argtypes = [vp]
        lib.isd_launch_count.restype = C.c_int64
        lib.isd_strerror.argtypes = [C.c_int]
        lib.isd_strerror.restype = C.c_char_p
        for n in EXPORTS[:8]:
            getattr(lib, n).restype = C.c_int
        _lib = lib
    return _lib


class IsdError(RuntimeError):
    pass


def lora_work_item(m: int, n: int, rank: int, num_sms: int, unit_index: int, item: int) -> dict:
    """Host-only view of isd_lora_linear's work assignment (see isd_test_lora_work_item in include/isd.h)."""
    out = (C.c_int32 * 9)()
    rc = load().isd_test_lora_work_item(m, n, rank, num_sms, unit_index, item, out)
    if rc != 0:
        raise IsdError(f"isd_test_lora_work_item failed: {load().isd_strerror(rc).decode()} ({rc})")
    keys = ("form", "units", "n_items", "pre", "m0", "n0", "cols", "tile_rows", "tile_cols")
    return dict(zip(keys, [int(x) for x in out]))


def verify_grid(batch: int, stride: int, vocab: int, propose_mode: int, num_sms: int) -> dict:
    """Host-only view of the launch shape isd_verify picks (see isd_test_verify_grid in include/isd.h)."""
    cfg = IsdConfig()
    cfg.batch, cfg.stride, cfg.vocab, cfg.propose_mode = batch, stride, vocab, propose_mode
    out = (C.c_int32 * 4)()
    rc = load().isd_test_verify_grid(C.byref(cfg), num_sms, out)
    if rc != 0:
        raise IsdError(f"isd_test_verify_grid failed: {load().isd_strerror(rc).decode()} ({rc})")
    return dict(zip(("row_splits", "sample_splits", "row_ctas", "sample_ctas"), [int(x) for x in out]))


def _check(rc: int, what: str):
    if rc != 0:
        raise IsdError(f"{what} failed: {load().isd_strerror(rc).decode()} ({rc})")


def _ptr(t):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device, contiguous tensors only"
    return t.data_ptr() if t.numel() > 0 else None


def _stream():
    return torch.cuda.current_stream().cuda_stream


def alloc_verify_out(B: int, N: int, device) -> dict:
    NP = N - 1
    i32 = dict(dtype=torch.int32, device=device)
    return dict(
        accept=torch.zeros(B, NP, dtype=torch.int8, device=device),
        alpha=torch.zeros(B, NP, dtype=torch.float32, device=device),
        accept_len=torch.zeros(B, **i32), n_emit=torch.zeros(B, **i32), repl_tok=torch.zeros(B, **i32),
        out_tok=torch.zeros(B, N, **i32), new_prop_tok=torch.zeros(B, NP, **i32),
        new_q_stats=torch.zeros(B, NP, 2, dtype=torch.float32, device=device))


def isd_verify_static(cfg: IsdConfig, st: dict, logits_cur, q_prev_logits, step: int, out: dict):
    """isd_verify for callers that must not allocate device memory: no context, the scratch is a fixed
    array inside the library (batch <= 64).  Calls must not overlap on the GPU; see include/isd.h."""
    s, o = Isd.state_struct(st), Isd.out_struct(out)
    _check(load().isd_verify_static(C.byref(cfg), C.byref(s), _ptr(logits_cur), _ptr(q_prev_logits), step,
                                    C.byref(o), _stream()), "isd_verify_static")


class Isd:
    """One ISD context (scratch owner).  Methods mirror the C entry points by name."""

    def __init__(self, *, batch, stride, n_q_heads, n_kv_heads, vocab, max_pages_per_slot, num_pages,
                 logits_dtype, head_dim=128, page_size=16, q_mode=0, propose_mode=0, mask_token_id=None,
                 sm_scale=0.0, inv_temperature=1.0, tau=0.0, seed=0, top_k=0, top_p=1.0):
        if not torch.cuda.is_available():
            raise IsdError("a CUDA device is required (there is no CPU path)")
        self.lib = load()
        ld = {"f32": 0, "bf16": 1, torch.float32: 0, torch.bfloat16: 1, 0: 0, 1: 1}[logits_dtype]
        self.cfg = IsdConfig(batch, stride, n_q_heads, n_kv_heads, head_dim, page_size, vocab,
                             max_pages_per_slot, num_pages, ld, q_mode, propose_mode,
                             vocab - 1 if mask_token_id is None else mask_token_id,
                             sm_scale, inv_temperature, tau, seed, top_k, top_p)
        self.ctx = C.c_void_p()
        _check(self.lib.isd_create(C.byref(self.cfg), C.byref(self.ctx)), "isd_create")
        self.N, self.B = stride, batch

    def close(self):
        if getattr(self, "ctx", None) and self.ctx.value:
            self.lib.isd_destroy(self.ctx)
            self.ctx = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- struct marshalling
    @staticmethod
    def state_struct(st: dict) -> IsdBatchState:
        return IsdBatchState(*[_ptr(st[n]) for n, _ in IsdBatchState._fields_])

    @staticmethod
    def out_struct(out: dict) -> IsdVerifyOut:
        return IsdVerifyOut(*[_ptr(out[n]) for n, _ in IsdVerifyOut._fields_])

    # -- entry points
    def isd_attn(self, st, q, k_new, v_new, k_pool, v_pool, attn_out, attn_lse=None):
        s = self.state_struct(st)
        _check(self.lib.isd_attn(self.ctx, C.byref(s), _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_pool),
                                 _ptr(v_pool), _ptr(attn_out), _ptr(attn_lse), _stream()), "isd_attn")

    def isd_verify(self, st, logits_cur, q_prev_logits, step, out):
        s, o = self.state_struct(st), self.out_struct(out)
        _check(self.lib.isd_verify(self.ctx, C.byref(s), _ptr(logits_cur), _ptr(q_prev_logits), step,
                                   C.byref(o), _stream()), "isd_verify")

    def isd_commit(self, st, out):
        s, o = self.state_struct(st), self.out_struct(out)
        _check(self.lib.isd_commit(self.ctx, C.byref(s), C.byref(o), _stream()), "isd_commit")

    def step_args(self, *, q, k_new, v_new, k_pool, v_pool, attn_out, attn_lse, logits_cur, q_prev_logits, out):
        return IsdStepArgs(_ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_pool), _ptr(v_pool), _ptr(attn_out),
                           _ptr(attn_lse), _ptr(logits_cur), _ptr(q_prev_logits), self.out_struct(out))

    def isd_step(self, st, args: IsdStepArgs, step: int, st_struct: IsdBatchState | None = None):
        s = st_struct if st_struct is not None else self.state_struct(st)
        _check(self.lib.isd_step(self.ctx, C.byref(s), C.byref(args), step, _stream()), "isd_step")

    def layer_args(self, layers):
        """Host array of isd_layer_args from dicts with q, k_new, v_new, k_pool, v_pool, attn_out[, attn_lse]."""
        arr = (IsdLayerArgs * len(layers))()
        for i, a in enumerate(layers):
            arr[i] = IsdLayerArgs(_ptr(a["q"]), _ptr(a["k_new"]), _ptr(a["v_new"]), _ptr(a["k_pool"]), _ptr(a["v_pool"]),
                                  _ptr(a["attn_out"]), _ptr(a.get("attn_lse")))
        return arr

    def isd_step_layers(self, st, layers, logits_cur, q_prev_logits, out, step: int,
                        st_struct: IsdBatchState | None = None):
        """`layers`: what layer_args returned (keep it alive across calls that reuse it)."""
        s = st_struct if st_struct is not None else self.state_struct(st)
        o = self.out_struct(out)
        _check(self.lib.isd_step_layers(self.ctx, C.byref(s), layers, len(layers), _ptr(logits_cur),
                                        _ptr(q_prev_logits), C.byref(o), step, _stream()), "isd_step_layers")

    def isd_lora_linear(self, x, w, a, b, gate, scale: float, t=None, y=None):
        """y = x w^T + gate * scale * (x a^T) b^T on bf16 CUDA tensors; allocates t / y when not given."""
        m, k = x.shape
        n, rank = b.shape
        t = torch.empty(m, rank, dtype=torch.bfloat16, device=x.device) if t is None else t
        y = torch.empty(m, n, dtype=torch.bfloat16, device=x.device) if y is None else y
        args = IsdLoraArgs(_ptr(x), _ptr(w), _ptr(a), _ptr(b), _ptr(gate), _ptr(t), _ptr(y), m, n, k, rank, scale)
        _check(self.lib.isd_lora_linear(self.ctx, C.byref(args), _stream()), "isd_lora_linear")
        return y

    def isd_set_step_counter(self, counter):
        """`counter`: a CUDA uint32 / int32 tensor of one element, or None."""
        _check(self.lib.isd_set_step_counter(self.ctx, _ptr(counter)), "isd_set_step_counter")

    def isd_set_wait_limit(self, milliseconds: int):
        """Time limit of every wait inside the kernels (default 250 ms); see include/isd.h."""
        _check(self.lib.isd_set_wait_limit(self.ctx, int(milliseconds)), "isd_set_wait_limit")

    def isd_test_preset_lora_counter(self, row_block: int, value: int):
        """Test hook: see include/isd.h (makes the readers of one row block of t run into their wait limit)."""
        _check(self.lib.isd_test_preset_lora_counter(self.ctx, row_block, value, _stream()), "isd_test_preset_lora_counter")

    def isd_release(self, st, slots):
        s = self.state_struct(st)
        _check(self.lib.isd_release(self.ctx, C.byref(s), _ptr(slots), slots.numel(), _stream()), "isd_release")

    def isd_read_status(self) -> int:
        v = C.c_uint32(0)
        _check(self.lib.isd_read_status(self.ctx, C.byref(v), _stream()), "isd_read_status")
        return int(v.value)

    def isd_set_profile_events(self, attn_start=None, attn_stop=None, verify_start=None, verify_stop=None):
        """Events are torch.cuda.Event objects (created with enable_timing=True and already recorded once)."""
        h = [None if e is None else e.cuda_event for e in (attn_start, attn_stop, verify_start, verify_stop)]
        _check(self.lib.isd_set_profile_events(self.ctx, *h), "isd_set_profile_events")

    def isd_launch_count(self) -> int:
        return int(self.lib.isd_launch_count(self.ctx))
