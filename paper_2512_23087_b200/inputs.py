"""Seeded synthetic workloads shaped like LLM-RL logit batches.

This module only draws random numbers and arranges them; it contains none of
the method's arithmetic (no max, log-sum-exp, mask or gradient) and is the one
module that both the CUDA path's callers and the CPU oracle's callers use, so
that both sides receive the same bits.

Structure of a batch (the logit-perturbation model of Sec. 4.2: infer = train +
epsilon): each row is a heavy-tailed or Gaussian base over the whole vocabulary
with a handful of strongly boosted "head" tokens, the inference logits are the
training logits plus small noise (rounded to the storage type), the sampled
token is drawn from softmax(infer) by the Gumbel-max construction, and the
upstream gradient is standard normal.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import torch


@dataclass(frozen=True)
class RowWorkload:
    """One row-kernel configuration."""
    name: str
    T: int
    V: int
    dtype: str            # "f32" | "bf16" | "f16": storage type of the logits
    base: str             # "normal" | "student_t3"
    scale: float          # multiplies the base draw
    head_boost: float     # added to the head tokens
    head_max: int         # k ~ U{1..head_max} head tokens per row
    infer_sigma: float    # standard deviation of infer - train
    rhos: tuple           # thresholds the configuration is run with
    backward: bool
    grad_dtype: str = ""  # defaults to dtype


@dataclass(frozen=True)
class FusedWorkload:
    """The LM-head configuration: hidden x W_vocab^T, logits never stored."""
    name: str
    T: int
    H: int
    V: int
    w_sigma: float
    infer_sigma: float
    rhos: tuple


WORKLOADS = {
    "c0_small_f32": RowWorkload("c0_small_f32", 64, 4096, "f32", "normal", 3.0, 12.0, 8, 0.01,
                                (1e-3,), True),
    "c1_bf16_fwd": RowWorkload("c1_bf16_fwd", 8192, 151936, "bf16", "normal", 3.0, 15.0, 8, 0.02,
                               (1e-4, 1e-3), False),
    "c2_bf16_fwdbwd": RowWorkload("c2_bf16_fwdbwd", 32768, 151936, "bf16", "normal", 3.0, 15.0, 8,
                                  0.02, (1e-4, 1e-3), True),
    "c3_f32_heavy": RowWorkload("c3_f32_heavy", 16384, 262144, "f32", "student_t3", 4.0, 15.0, 16,
                                0.05, (1e-4,), True),
    "c4_fused_lmhead": FusedWorkload("c4_fused_lmhead", 16384, 4096, 151936, 0.02, 0.02,
                                     (1e-4, 1e-3)),
}

_TORCH_DTYPE = {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}


def torch_dtype(name: str) -> torch.dtype:
    return _TORCH_DTYPE[name]


@dataclass
class RowBatch:
    train: torch.Tensor      # [T, V] storage dtype
    infer: torch.Tensor      # [T, V] storage dtype
    ids: torch.Tensor        # [T] int64
    upstream: torch.Tensor   # [T] float32
    meta: dict = field(default_factory=dict)


def _gen(device, seed: int, stream: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((int(seed) * 1000003 + int(stream) * 7919 + 12345) % (2 ** 63 - 1))
    return g


def _base_draw(kind: str, rows: int, V: int, g: torch.Generator, device) -> torch.Tensor:
    x = torch.randn(rows, V, generator=g, device=device, dtype=torch.float32)
    if kind == "normal":
        return x
    if kind == "student_t3":
        # Student-t with 3 degrees of freedom: N / sqrt(chi2_3 / 3)
        c = torch.zeros_like(x)
        for _ in range(3):
            n = torch.randn(rows, V, generator=g, device=device, dtype=torch.float32)
            c.addcmul_(n, n)
        return x / torch.sqrt(c / 3.0)
    raise ValueError(kind)


def make_rows(w: RowWorkload, seed: int = 0, device="cpu", T: int | None = None,
              V: int | None = None, chunk_rows: int = 512, ld: int | None = None) -> RowBatch:
    """Generate a batch for ``w``; ``T``/``V`` override the sizes (parity cases).

    Rows are drawn in chunks, each from its own generator stream, so peak
    temporary memory stays near ``chunk_rows * V`` floats.  ``ld`` (>= V) gives
    the logit matrices a padded row stride; the padding holds a large positive
    value so that any read past column V shows up as a wrong result.
    """
    T = w.T if T is None else T
    V = w.V if V is None else V
    ld = V if ld is None else ld
    dt = _TORCH_DTYPE[w.dtype]
    device = torch.device(device)
    train = torch.empty(T, ld, dtype=dt, device=device)
    infer = torch.empty(T, ld, dtype=dt, device=device)
    if ld > V:
        train[:, V:] = 3.0e4
        infer[:, V:] = 3.0e4
    ids = torch.empty(T, dtype=torch.int64, device=device)
    for c, r0 in enumerate(range(0, T, chunk_rows)):
        rows = min(chunk_rows, T - r0)
        g = _gen(device, seed, c)
        z = _base_draw(w.base, rows, V, g, device).mul_(w.scale)
        k = torch.randint(1, w.head_max + 1, (rows, 1), generator=g, device=device)
        pos = torch.randint(0, V, (rows, w.head_max), generator=g, device=device)
        use = torch.arange(w.head_max, device=device).unsqueeze(0) < k
        # unused slots point at the first head position, which is always used
        pos = torch.where(use, pos, pos[:, :1])
        head = torch.zeros(rows, V, dtype=torch.bool, device=device)
        head.scatter_(1, pos, True)
        z += head.to(torch.float32) * w.head_boost
        zt = z.to(dt)
        train[r0:r0 + rows, :V] = zt
        zi = (zt.to(torch.float32)
              + torch.randn(rows, V, generator=g, device=device, dtype=torch.float32) * w.infer_sigma).to(dt)
        infer[r0:r0 + rows, :V] = zi
        ids[r0:r0 + rows] = _gumbel_argmax(zi, g)
        del z, head, zt, zi
    upstream = torch.randn(T, generator=_gen(device, seed, 1 << 20), device=device, dtype=torch.float32)
    return RowBatch(train[:, :V] if ld > V else train, infer[:, :V] if ld > V else infer, ids, upstream,
                    meta={"workload": w.name, "T": T, "V": V, "ld": ld, "seed": seed, "dtype": w.dtype})


def _gumbel_argmax(z_stored: torch.Tensor, g: torch.Generator) -> torch.Tensor:
    """A draw from softmax(z) at temperature 1: argmax_k (z_k + Gumbel_k)."""
    u = torch.rand(z_stored.shape, generator=g, device=z_stored.device, dtype=torch.float32)
    u.clamp_(min=1e-30, max=1.0 - 1e-7)
    gumbel = -torch.log(-torch.log(u))
    return torch.argmax(z_stored.to(torch.float32) + gumbel, dim=1)


@dataclass
class FusedBatch:
    hidden: torch.Tensor     # [T, H] bf16
    w_vocab: torch.Tensor    # [V, H] bf16
    infer: torch.Tensor      # [T, V] bf16
    ids: torch.Tensor        # [T] int64
    upstream: torch.Tensor   # [T] float32
    meta: dict = field(default_factory=dict)


def make_fused(w: FusedWorkload, seed: int = 0, device="cpu", T: int | None = None,
               H: int | None = None, V: int | None = None, chunk_rows: int = 1024) -> FusedBatch:
    """hidden ~ N(0,1), W ~ N(0, w_sigma^2), both bf16.  The inference logits
    are what an inference engine would return for the same parameters: the
    product of the stored operands plus N(0, infer_sigma^2), rounded to bf16.
    The product is formed here in float32 by ``torch.matmul`` chunk by chunk
    only to build that input; it is discarded afterwards."""
    T = w.T if T is None else T
    H = w.H if H is None else H
    V = w.V if V is None else V
    device = torch.device(device)
    g = _gen(device, seed, 1 << 21)
    hidden = torch.randn(T, H, generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)
    w_vocab = torch.empty(V, H, dtype=torch.bfloat16, device=device)
    for r0 in range(0, V, 16384):
        rows = min(16384, V - r0)
        w_vocab[r0:r0 + rows] = (torch.randn(rows, H, generator=g, device=device, dtype=torch.float32)
                                 * w.w_sigma).to(torch.bfloat16)
    infer = torch.empty(T, V, dtype=torch.bfloat16, device=device)
    ids = torch.empty(T, dtype=torch.int64, device=device)
    wf = w_vocab.to(torch.float32)
    for c, r0 in enumerate(range(0, T, chunk_rows)):
        rows = min(chunk_rows, T - r0)
        gc = _gen(device, seed, (1 << 22) + c)
        z = hidden[r0:r0 + rows].to(torch.float32) @ wf.t()
        zi = (z + torch.randn(rows, V, generator=gc, device=device, dtype=torch.float32)
              * w.infer_sigma).to(torch.bfloat16)
        infer[r0:r0 + rows] = zi
        ids[r0:r0 + rows] = _gumbel_argmax(zi, gc)
        del z, zi
    del wf
    upstream = torch.randn(T, generator=_gen(device, seed, 1 << 23), device=device, dtype=torch.float32)
    return FusedBatch(hidden, w_vocab, infer, ids, upstream,
                      meta={"workload": w.name, "T": T, "H": H, "V": V, "seed": seed})


def shard_rows(T: int, rank: int, world: int) -> tuple[int, int]:
    """Contiguous block of rows [r0, r1) that ``rank`` of ``world`` owns.
    Rows are independent, so sharding needs no exchange of data."""
    per = (T + world - 1) // world
    r0 = min(T, per * rank)
    return r0, min(T, r0 + per)
