"""Drive one synthetic workload through the C ABI: argument plumbing only.

``WorkloadRun`` owns a context sized for a :class:`inputs.Workload`, fills the shared states, and runs
decode calls (reorder -> per layer: append, decode) on tensors the caller or the seeded generators
provide.  Nothing here computes any part of the method; every step is a library call.
"""
from __future__ import annotations

from typing import Optional

import torch

from . import inputs
from .binding import MAX_BATCH, Onela, make_config


class WorkloadRun:
    def __init__(self, wl: inputs.Workload, device="cuda", out_dtype: Optional[str] = None, flags: int = 0,
                 extra_slots: int = 0):
        self.wl = wl
        self.device = torch.device(device)
        self.out_dtype = out_dtype or wl.dtype
        slots = wl.R * wl.W * wl.D + extra_slots
        self.cfg = make_config(wl.R, wl.L, wl.H, wl.dk, wl.dv, wl.W, wl.D, wl.dtype, self.out_dtype, slots, flags)
        self.ctx = Onela(self.cfg, device=self.device)
        self.torch_out_dtype = self.ctx.out_dtype

    # ---- shared states -------------------------------------------------------------------------
    def prefill_states(self, overrides: Optional[dict] = None, chunk_tokens: int = 4096, stream=None):
        """Fill every (request, layer) store slot: from ``overrides[(r, l)]`` (fp32 [H, dv, dk]) where
        given, else by generating the seeded prompt on the device and running the prefill kernel."""
        wl, overrides = self.wl, overrides or {}
        for r in range(wl.R):
            for l in range(wl.L):
                if (r, l) in overrides:
                    s0 = overrides[(r, l)].to(self.device, torch.float32).contiguous()
                    self.ctx.onela_init_shared_state(r, l, s0, stream)
                    continue
                parts = [inputs.prompt_tokens(wl, r, l, a, min(a + chunk_tokens, wl.prompt_len), device=self.device)
                         for a in range(0, wl.prompt_len, chunk_tokens)]
                tok = {n: torch.cat([p[n] for p in parts]).contiguous() for n in ("k", "v", "alpha", "beta")}
                self.ctx.onela_prefill_shared_state(r, l, tok["k"], tok["v"], tok["alpha"], tok["beta"], stream)
                del parts, tok
        torch.cuda.synchronize(self.device)

    # ---- inputs of one decode call ----------------------------------------------------------------
    def generate_call(self, t: int, device=None) -> dict:
        """Seeded inputs of decode call t for all requests and layers, batched over requests:
        parents int32 [R, W] (None at t = 0); per layer k, v [R, W, H, d], alpha, beta [R, W, H], q [R, W, H, dk]."""
        wl = self.wl
        device = self.device if device is None else device
        call = {"parents": None, "layers": []}
        if t > 0:
            call["parents"] = torch.stack([inputs.parents(wl, r, t) for r in range(wl.R)]).to(device)
        for l in range(wl.L):
            toks = [inputs.decode_token(wl, r, l, t, device=device) for r in range(wl.R)]
            lay = {n: torch.stack([tk[n] for tk in toks]).contiguous() for n in ("k", "v", "alpha", "beta")}
            lay["q"] = torch.stack([inputs.decode_query(wl, r, l, t, device=device) for r in range(wl.R)]).contiguous()
            call["layers"].append(lay)
        return call

    def alloc_outputs(self) -> list:
        wl = self.wl
        return [torch.empty((wl.R, wl.W, wl.H, wl.dv), dtype=self.torch_out_dtype, device=self.device)
                for _ in range(wl.L)]

    # ---- one decode call through the library ------------------------------------------------------
    def run_call(self, call: dict, outs: list, stream=None, decode_events=None, fused: bool = False,
                 group_events: bool = False):
        """reorder_beams once, then append_records + decode_step per layer, batched over all requests
        (in chunks of at most ONELA_MAX_BATCH); with ``fused`` the two per-layer calls are the one-launch
        append_decode_step.  ``decode_events``: optional list that receives (start, end, launches) CUDA event
        pairs: around every decode launch, or - with ``group_events`` and fused launches, where nothing else
        runs between the layers - one pair around all the layers' launches of the call."""
        wl, ctx = self.wl, self.ctx
        for r0 in range(0, wl.R, MAX_BATCH):
            n = min(MAX_BATCH, wl.R - r0)
            par = None if call["parents"] is None else call["parents"][r0:r0 + n]
            ctx.onela_reorder_beams(r0, n, par, wl.W, stream)
            per_group = decode_events is not None and group_events and fused
            if per_group:
                g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                g0.record(stream)
            for l, lay in enumerate(call["layers"]):
                sl = slice(r0, r0 + n)
                if not fused:
                    ctx.onela_append_records(r0, n, l, lay["k"][sl], lay["v"][sl], lay["alpha"][sl], lay["beta"][sl], stream)
                if decode_events is not None and not per_group:
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(stream)
                if fused:
                    ctx.onela_append_decode_step(r0, n, l, lay["k"][sl], lay["v"][sl], lay["alpha"][sl], lay["beta"][sl],
                                                 lay["q"][sl], outs[l][sl], stream)
                else:
                    ctx.onela_decode_step(r0, n, l, lay["q"][sl], outs[l][sl], stream)
                if decode_events is not None and not per_group:
                    e1.record(stream)
                    decode_events.append((e0, e1, 1))
            if per_group:
                g1.record(stream)
                decode_events.append((g0, g1, len(call["layers"])))
