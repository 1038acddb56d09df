"""Seeded synthetic inputs shaped like the paper's serving workloads.

This module only draws inputs (random tensors, page-table shuffles, a synthetic
"model" that says which token a logits row is peaked on).  It holds none of the
ISD step's arithmetic and is shared by the CUDA path's tests/benchmark and by
the CPU oracle's tests.

Synthetic model: the token the (imaginary) model favours at absolute position
``pos`` of slot ``b`` is ``favoured_token(b, pos)``; a position is *peaked* with
probability ``peaked_frac``.  A logits row sitting at position ``P`` predicts the
token at ``P + 1`` (logit shift), whether the row is a clean row (anchor law p)
or a [MASK] row (proposal law q): if ``P + 1`` is peaked, the favoured token's
logit is raised to ``row_max + peak_bump`` in that row.  Proposals made from a
[MASK] row and the anchor row that judges them one step later therefore agree on
peaked positions and are independent noise elsewhere, which sets the accept rate.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch

PAGE = 16


@dataclass(frozen=True)
class Workload:
    name: str
    batch: int
    stride: int
    n_q_heads: int = 32
    n_kv_heads: int = 8
    head_dim: int = 128
    vocab: int = 151936
    ctx_min: int = 1024
    ctx_max: int = 8192
    logits_dtype: str = "bf16"      # "bf16" | "f32"
    logit_sigma: float = 3.0
    peaked_frac: float = 0.0
    peak_bump: float = 8.0
    kv_sigma: float = 0.5
    steps: int = 2                  # chained steps the pool must be able to hold
    shuffle_pages: bool = True
    propose_mode: int = 1           # 1 = argmax proposals (paper's serving setting), 0 = sampled
    q_mode: int = 0
    seed: int = 0
    top_k: int = 0                  # > 0: top-k / top-p filtered laws (the paper's serving sampling configuration)
    top_p: float = 1.0

    @property
    def Q(self) -> int:
        return 2 * self.stride - 1

    @property
    def max_pages_per_slot(self) -> int:
        return (self.ctx_max + self.steps * self.stride + self.Q + PAGE - 1) // PAGE + 1


def config(i: int, **kw) -> Workload:
    """The five workloads the benchmark definition lists (index 0..4)."""
    if i == 0:
        w = Workload("tiny_b1_n4_ctx256", batch=1, stride=4, n_q_heads=8, n_kv_heads=2, vocab=4096,
                     ctx_min=256, ctx_max=256, logits_dtype="f32", logit_sigma=2.0, shuffle_pages=False,
                     propose_mode=0, seed=0)
    elif i == 1:
        w = Workload("moderate_b32_n4_ctx512-4096", batch=32, stride=4, ctx_min=512, ctx_max=4096,
                     logit_sigma=3.0, peaked_frac=0.2, propose_mode=0, seed=1)
    elif i == 2:
        # argmax proposals judged against a point mass: the paper's serving setting in its distribution-preserving form
        w = Workload("stationary_b256_n8_ctx1k-8k", batch=256, stride=8, ctx_min=1024, ctx_max=8192,
                     logit_sigma=3.0, peaked_frac=0.9, steps=100, q_mode=1, seed=2)
    elif i == 3:
        w = Workload("longctx_b16_n4_ctx32k", batch=16, stride=4, ctx_min=32768, ctx_max=32768,
                     logit_sigma=2.0, propose_mode=0, seed=3)
    elif i == 4:
        w = sweep_point(8, 256)
    else:
        raise ValueError(i)
    return replace(w, **kw) if kw else w


def sweep_point(stride: int, batch: int) -> Workload:
    strides, batches = [2, 4, 8, 16], [1, 8, 64, 256, 512]
    seed = 5000 + 100 * strides.index(stride) + batches.index(batch)
    return Workload(f"sweep_n{stride}_b{batch}_ctx4096", batch=batch, stride=stride, ctx_min=4096,
                    ctx_max=4096, peaked_frac=0.9, q_mode=1, seed=seed)


def _gen(device, *keys) -> torch.Generator:
    g = torch.Generator(device=device)
    s = 0x9E3779B97F4A7C15
    for k in keys:
        s = (s * 6364136223846793005 + int(k) + 1442695040888963407) % (1 << 63)
    g.manual_seed(s)
    return g


def _mix(b: torch.Tensor, pos: torch.Tensor, salt: int) -> torch.Tensor:
    """Cheap integer hash of (slot, position) -> 31-bit value (int64 tensor)."""
    x = (b * 0x9E3779B1 + pos * 0x85EBCA77 + salt * 0xC2B2AE3D + 0x27D4EB2F) & 0x7FFFFFFF
    x = ((x ^ (x >> 15)) * 0x2C1B3C6D) & 0x7FFFFFFF
    x = ((x ^ (x >> 12)) * 0x297A2D39) & 0x7FFFFFFF
    return x ^ (x >> 15)


def favoured_token(w: Workload, b: torch.Tensor, pos: torch.Tensor) -> torch.Tensor:
    return _mix(b, pos, 2 * w.seed + 1) % w.vocab


def is_peaked(w: Workload, b: torch.Tensor, pos: torch.Tensor) -> torch.Tensor:
    return _mix(b, pos, 2 * w.seed + 2) < int(w.peaked_frac * float(1 << 31))


def make_state(w: Workload, device) -> dict:
    """Initial stationary-batch state + KV pools (every slot starts with an NP step)."""
    dev = torch.device(device)
    B, Q, NP = w.batch, w.Q, w.stride - 1
    g = _gen("cpu", w.seed, 101)
    ctx = torch.randint(w.ctx_min, w.ctx_max + 1, (B,), generator=g, dtype=torch.int64)
    mp = w.max_pages_per_slot
    have = (ctx + Q + PAGE - 1) // PAGE
    grow = (w.steps * w.stride + PAGE - 1) // PAGE + 1
    num_pages = int((have + grow).sum().item()) + 8
    order = torch.randperm(num_pages, generator=g) if w.shuffle_pages else torch.arange(num_pages)
    page_table = torch.full((B, mp), -1, dtype=torch.int32)
    off = 0
    for b in range(B):
        n = int(have[b])
        page_table[b, :n] = order[off:off + n].to(torch.int32)
        off += n
    n_free = num_pages - off
    free_stack = torch.full((num_pages,), -1, dtype=torch.int32)
    free_stack[:n_free] = order[off:].to(torch.int32)
    block_tok = torch.full((B, Q), w.vocab - 1, dtype=torch.int32)
    block_tok[:, 0] = torch.randint(0, w.vocab, (B,), generator=g, dtype=torch.int64).to(torch.int32)
    gd = _gen(dev, w.seed, 102)
    pool_shape = (num_pages, w.n_kv_heads, PAGE, w.head_dim)
    k_pool = (torch.randn(pool_shape, generator=gd, device=dev, dtype=torch.float32) * w.kv_sigma).to(torch.bfloat16)
    v_pool = (torch.randn(pool_shape, generator=gd, device=dev, dtype=torch.float32) * w.kv_sigma).to(torch.bfloat16)
    st = dict(
        ctx_len=ctx.to(torch.int32), n_ver=torch.zeros(B, dtype=torch.int32), block_tok=block_tok,
        q_row0=torch.zeros(B, dtype=torch.int32), q_stats=torch.zeros(B, NP, 2, dtype=torch.float32),
        page_table=page_table, free_stack=free_stack, free_top=torch.tensor([n_free], dtype=torch.int32),
        active=torch.ones(B, dtype=torch.uint8), slot_status=torch.zeros(B, dtype=torch.int32))
    st = {k: v.to(dev) for k, v in st.items()}
    st.update(k_pool=k_pool, v_pool=v_pool, num_pages=num_pages)
    return st


def make_qkv(w: Workload, step: int, device):
    """Queries / keys / values of the block rows for one step (post-RoPE stand-ins)."""
    dev = torch.device(device)
    g = _gen(dev, w.seed, 200, step)
    B, Q = w.batch, w.Q
    q = torch.randn((B, Q, w.n_q_heads, w.head_dim), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    k = (torch.randn((B, Q, w.n_kv_heads, w.head_dim), generator=g, device=dev, dtype=torch.float32) * w.kv_sigma).to(torch.bfloat16)
    v = (torch.randn((B, Q, w.n_kv_heads, w.head_dim), generator=g, device=dev, dtype=torch.float32) * w.kv_sigma).to(torch.bfloat16)
    return q, k, v


def make_logits(w: Workload, step: int, ctx_len: torch.Tensor, out: torch.Tensor | None = None) -> torch.Tensor:
    """This step's logits [B, Q, V] given the committed lengths (device tensor, no host sync)."""
    dev = ctx_len.device
    B, Q, V = w.batch, w.Q, w.vocab
    dt = torch.bfloat16 if w.logits_dtype == "bf16" else torch.float32
    g = _gen(dev, w.seed, 300, step)
    if out is None:
        out = torch.empty((B, Q, V), device=dev, dtype=dt)
    if dt == torch.float32:
        out.normal_(0.0, w.logit_sigma, generator=g)
    else:
        chunk = max(1, (1 << 26) // (Q * V))
        for b0 in range(0, B, chunk):
            t = torch.randn((min(chunk, B - b0), Q, V), generator=g, device=dev, dtype=torch.float32)
            out[b0:b0 + chunk] = (t * w.logit_sigma).to(dt)
    if w.peaked_frac > 0.0:
        b = torch.arange(B, device=dev, dtype=torch.int64)[:, None].expand(B, Q)
        pos = ctx_len.to(torch.int64)[:, None] + torch.arange(Q, device=dev, dtype=torch.int64)[None, :] + 1
        tok = favoured_token(w, b, pos)
        peaked = is_peaked(w, b, pos)
        row_max = out.amax(dim=2).to(torch.float32)
        cur = torch.gather(out, 2, tok[:, :, None]).squeeze(2).to(torch.float32)
        val = torch.where(peaked, row_max + w.peak_bump, cur).to(dt)
        out.scatter_(2, tok[:, :, None], val[:, :, None])
    return out


def l2_flush_buffer(device, mbytes: int = 512) -> torch.Tensor:
    return torch.empty(mbytes << 20, dtype=torch.uint8, device=device)
