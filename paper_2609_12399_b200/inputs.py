"""Seeded synthetic inputs for the beam-shared GDN decode path.

This module only draws numbers.  It holds none of the method's arithmetic (no
recurrence, no fold, no ancestry bookkeeping): both the CPU oracle and the CUDA
library consume the tensors it returns, so nothing here may depend on either.

Every element is a pure function of ``(seed, kind, request, layer, step, beam,
head, element)`` through a counter-based 32-bit hash, so any subset of beams,
heads or prompt tokens can be regenerated on its own (the CPU baseline only
draws the records its sampled chains touch), on CPU or on a CUDA device (torch
integer ops only; the floating-point tail - log, cos, sqrt - may differ in the
last ulp between devices, so a test always draws once and hands the same
tensor to both sides).

Distributions (the GR-shaped workloads of the benchmark configs): q and k are
N(0,1) vectors L2-normalised in fp64 and then rounded to the storage dtype,
v ~ N(0,1), alpha ~ U(0.9, 1.0), beta = sigmoid(N(0,1)); prompt tokens use the
same distributions; parents are uniform or bounded-Zipf over the previous beam.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Optional

import torch

_M32 = 0xFFFFFFFF

# tensor kinds (part of the hash key)
PROMPT_K, PROMPT_V, PROMPT_ALPHA, PROMPT_BETA = 1, 2, 3, 4
DEC_K, DEC_V, DEC_ALPHA, DEC_BETA, DEC_Q = 5, 6, 7, 8, 9
PARENT_U, PARENT_PERM = 10, 11


@dataclass(frozen=True)
class Workload:
    """One synthetic workload: shapes, dtypes and the parent-selection law."""

    name: str
    R: int            # requests
    L: int            # GDN layers
    H: int            # heads (key heads == value heads)
    dk: int
    dv: int
    dtype: str        # storage dtype of q, k, v: "fp32" or "bf16"
    prompt_len: int
    W: int            # beam width
    D: int            # decode calls (= records on a chain at the last call)
    parents: str      # "uniform" or "zipf"
    zipf_s: float
    seed: int

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "fp32" else torch.bfloat16

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "fp32" else 2

    @property
    def record_bytes(self) -> int:
        """k + v in the storage dtype plus fp32 alpha and beta."""
        return (self.dk + self.dv) * self.elem_bytes + 8

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


WORKLOADS = (
    Workload("cfg0_tiny", 1, 1, 2, 32, 32, "fp32", 64, 8, 3, "uniform", 0.0, 12399),
    Workload("cfg1_beam128", 1, 1, 16, 128, 128, "bf16", 4096, 128, 4, "uniform", 0.0, 12400),
    Workload("cfg2_beam512_zipf", 1, 1, 32, 128, 128, "bf16", 16384, 512, 4, "zipf", 1.2, 12401),
    Workload("cfg3_batch8_beam1024", 8, 1, 32, 128, 128, "bf16", 8192, 1024, 6, "uniform", 0.0, 12402),
    Workload("cfg4_stack16_beam512", 4, 16, 32, 128, 128, "bf16", 16384, 512, 8, "zipf", 1.5, 12403),
)


# ----------------------------------------------------------------------------
# counter-based hash (uint32 values carried in int64 tensors; no overflow)
# ----------------------------------------------------------------------------
def _mul32(x: torch.Tensor, c: int) -> torch.Tensor:
    lo = x * (c & 0xFFFF)
    hi = ((x * (c >> 16)) & 0xFFFF) << 16
    return (lo + hi) & _M32


def _mix(x: torch.Tensor) -> torch.Tensor:
    x = _mul32(x ^ (x >> 16), 0x7FEB352D)
    x = _mul32(x ^ (x >> 15), 0x846CA68B)
    return x ^ (x >> 16)


def _mix_int(x: int) -> int:
    x &= _M32
    x = ((x ^ (x >> 16)) * 0x7FEB352D) & _M32
    x = ((x ^ (x >> 15)) * 0x846CA68B) & _M32
    return x ^ (x >> 16)


def _key(seed: int, kind: int, stream: int, *ids: int) -> tuple[int, int]:
    h = _mix_int(seed ^ 0x9E3779B9)
    for v in (kind, stream, *ids):
        h = _mix_int(h ^ _mix_int((v + 0x632BE5AB) & _M32))
    return h, _mix_int(h ^ 0x85EBCA6B)


def _uniform(key: tuple[int, int], counter: torch.Tensor) -> torch.Tensor:
    """fp64 uniforms in the open interval (0, 1), one per counter value."""
    h = _mix(_mix(counter ^ key[0]) ^ key[1])
    return (h.to(torch.float64) + 0.5) * (1.0 / 4294967296.0)


def _normal(seed, kind, ids, counter) -> torch.Tensor:
    u1 = _uniform(_key(seed, kind, 0, *ids), counter)
    u2 = _uniform(_key(seed, kind, 1, *ids), counter)
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)


def _counter(rows: torch.Tensor, heads: torch.Tensor, H: int, dim: int) -> torch.Tensor:
    """Counter of element (row, head, e) in a dense [rows, H, dim] tensor."""
    e = torch.arange(dim, device=rows.device, dtype=torch.int64)
    return ((rows[:, None, None] * H + heads[None, :, None]) * dim + e[None, None, :])


def _index(n: int, sel, device) -> torch.Tensor:
    if sel is None:
        return torch.arange(n, device=device, dtype=torch.int64)
    return torch.as_tensor(sel, dtype=torch.int64, device=device).reshape(-1)


def _vectors(wl, kind, ids, rows, heads, dim, unit: bool) -> torch.Tensor:
    z = _normal(wl.seed, kind, ids, _counter(rows, heads, wl.H, dim))
    if unit:
        z = z / torch.linalg.vector_norm(z, dim=-1, keepdim=True)
    return z.to(wl.torch_dtype)


def _gates(wl, kind_a, kind_b, ids, rows, heads):
    c = _counter(rows, heads, wl.H, 1)[..., 0]
    alpha = 0.9 + 0.1 * _uniform(_key(wl.seed, kind_a, 0, *ids), c)
    beta = torch.sigmoid(_normal(wl.seed, kind_b, ids, c))
    return alpha.to(torch.float32), beta.to(torch.float32)


# ----------------------------------------------------------------------------
# public generators
# ----------------------------------------------------------------------------
def decode_token(wl: Workload, req: int, layer: int, step: int, beams=None, heads=None,
                 device="cpu") -> dict:
    """The token every beam appends at decode call ``step``.

    Returns k [n, h, dk], v [n, h, dv] in the storage dtype and alpha, beta
    [n, h] in fp32, for the selected beams / heads (all when None).
    """
    rows, hs = _index(wl.W, beams, device), _index(wl.H, heads, device)
    ids = (req, layer, step)
    alpha, beta = _gates(wl, DEC_ALPHA, DEC_BETA, ids, rows, hs)
    return {
        "k": _vectors(wl, DEC_K, ids, rows, hs, wl.dk, unit=True),
        "v": _vectors(wl, DEC_V, ids, rows, hs, wl.dv, unit=False),
        "alpha": alpha,
        "beta": beta,
    }


def decode_query(wl: Workload, req: int, layer: int, step: int, beams=None, heads=None,
                 device="cpu") -> torch.Tensor:
    """q [n, h, dk] in the storage dtype for decode call ``step``."""
    rows, hs = _index(wl.W, beams, device), _index(wl.H, heads, device)
    return _vectors(wl, DEC_Q, (req, layer, step), rows, hs, wl.dk, unit=True)


def prompt_tokens(wl: Workload, req: int, layer: int, tok_begin: int = 0,
                  tok_end: Optional[int] = None, heads=None, device="cpu") -> dict:
    """Prompt tokens [tok_begin, tok_end): k [n, h, dk], v [n, h, dv], alpha, beta [n, h]."""
    tok_end = wl.prompt_len if tok_end is None else tok_end
    rows = torch.arange(tok_begin, tok_end, device=device, dtype=torch.int64)
    hs = _index(wl.H, heads, device)
    ids = (req, layer, 0)
    alpha, beta = _gates(wl, PROMPT_ALPHA, PROMPT_BETA, ids, rows, hs)
    return {
        "k": _vectors(wl, PROMPT_K, ids, rows, hs, wl.dk, unit=True),
        "v": _vectors(wl, PROMPT_V, ids, rows, hs, wl.dv, unit=False),
        "alpha": alpha,
        "beta": beta,
    }


def parents(wl: Workload, req: int, step: int, W_prev: Optional[int] = None,
            W_new: Optional[int] = None) -> torch.Tensor:
    """Parent of every beam of decode call ``step`` (>= 1) in the previous beam, int32 [W_new] on CPU.

    uniform: each child picks a parent uniformly.  zipf: P(rank i) ~ i^-s over
    i = 1..W_prev by inverse CDF on a seeded uniform, with ranks mapped to beams
    through a fresh seeded permutation per step, so popular parents are not
    always the low indices; several children naming one parent is the
    duplication the beam search produces.
    """
    if step < 1:
        raise ValueError("decode call 0 has no parents: every beam starts at the shared state")
    W_prev = wl.W if W_prev is None else W_prev
    W_new = wl.W if W_new is None else W_new
    c = torch.arange(W_new, dtype=torch.int64)
    u = _uniform(_key(wl.seed, PARENT_U, 0, req, step), c)
    if wl.parents == "uniform":
        idx = torch.clamp((u * W_prev).to(torch.int64), max=W_prev - 1)
    elif wl.parents == "zipf":
        ranks = torch.arange(1, W_prev + 1, dtype=torch.float64)
        cdf = torch.cumsum(ranks.pow(-wl.zipf_s), 0)
        cdf = cdf / cdf[-1]
        rank = torch.clamp(torch.searchsorted(cdf, u), max=W_prev - 1)
        pkey = _uniform(_key(wl.seed, PARENT_PERM, 0, req, step),
                        torch.arange(W_prev, dtype=torch.int64))
        perm = torch.argsort(pkey, stable=True)
        idx = perm[rank]
    else:
        raise ValueError(f"unknown parent law {wl.parents!r}")
    return idx.to(torch.int32)
