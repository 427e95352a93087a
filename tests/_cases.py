"""Shared helpers of the GPU parity tests: build a seeded case, run it through the C ABI and through
the CPU oracle, and compare.  The case tensors come from the seeded generators (and S_0 from the
oracle's prefill of the seeded prompt); the same tensors feed both sides."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_2609_12399_b200 as P
from paper_2609_12399_b200 import inputs

REL_L2_BAR = 5e-3   # the stated parity bar: relative L2 per (beam, head) output vector against fp64


def rel_l2(got: np.ndarray, ref: np.ndarray) -> np.ndarray:
    """Per-vector relative L2 over the last axis, guarded for near-zero references."""
    dv = ref.shape[-1]
    den = np.maximum(np.linalg.norm(ref, axis=-1), 1e-6 * np.sqrt(dv))
    return np.linalg.norm(got.astype(np.float64) - ref, axis=-1) / den


def make_case(wl: inputs.Workload, widths=None, device="cpu") -> dict:
    """All inputs of a workload: S0[(r,l)] fp32 [H,dv,dk] (oracle prefill of the seeded prompt),
    tok[(r,l,t)], q[(r,l,t)], parents[(r,t)] (None at t = 0), widths[t]."""
    widths = list(widths) if widths is not None else [wl.W] * wl.D
    case = {"wl": wl, "widths": widths, "S0": {}, "tok": {}, "q": {}, "parents": {}}
    for r in range(wl.R):
        for t in range(len(widths)):
            case["parents"][(r, t)] = None if t == 0 else inputs.parents(wl, r, t, W_prev=widths[t - 1], W_new=widths[t])
        for l in range(wl.L):
            p = inputs.prompt_tokens(wl, r, l, device=device)
            S = oracle.prefill(p["k"], p["v"], p["alpha"], p["beta"])
            case["S0"][(r, l)] = torch.from_numpy(S.astype(np.float32))
            for t, W in enumerate(widths):
                beams = torch.arange(W)
                case["tok"][(r, l, t)] = {n: x.cpu() for n, x in inputs.decode_token(wl, r, l, t, beams=beams, device=device).items()}
                case["q"][(r, l, t)] = inputs.decode_query(wl, r, l, t, beams=beams, device=device).cpu()
    return case


def run_oracle(case, upto=None, sel=None) -> tuple[dict, dict]:
    """Oracle outputs outs[(r,l,t)] fp64 [W_t,H,dv] (or [n_sel,dv]) and chains[(r,t)] int [W_t, t+1]
    (beam index at every call, oldest first) for every decode call."""
    wl, widths = case["wl"], case["widths"]
    outs, chains = {}, {}
    for r in range(wl.R):
        for l in range(wl.L):
            for t in range(len(widths) if upto is None else upto):
                steps = [case["tok"][(r, l, j)] for j in range(t + 1)]
                par = [case["parents"][(r, j)] for j in range(t + 1)]
                o, ch = oracle.decode(case["S0"][(r, l)], steps, par, case["q"][(r, l, t)], sel=sel, return_chains=True)
                outs[(r, l, t)] = o
                if sel is None:
                    chains[(r, t)] = ch.reshape(widths[t], wl.H, t + 1)[:, 0, :]
    return outs, chains


def run_library(case, out_dtype="fp32", flags=0, batched=True, device="cuda", fused=False) -> tuple[dict, dict, P.Onela]:
    """The same case through the C ABI.  Returns outs[(r,l,t)] (torch, CPU), slots[(r,t)] int32 [W_t, t+1]
    (global slot ids from onela_export_chains) and the context (kept alive for further queries)."""
    wl, widths = case["wl"], case["widths"]
    T = len(widths)
    cfg = P.make_config(wl.R, wl.L, wl.H, wl.dk, wl.dv, max(widths), T, wl.dtype, out_dtype,
                        wl.R * sum(widths), flags)
    ctx = P.Onela(cfg, device=device)
    dev = torch.device(device)
    for (r, l), S in case["S0"].items():
        ctx.onela_init_shared_state(r, l, S.to(dev))
    outs, slots = {}, {}
    groups = [list(range(wl.R))] if batched else [[r] for r in range(wl.R)]
    for t, W in enumerate(widths):
        for g in groups:
            r0, n = g[0], len(g)
            par = None if t == 0 else torch.stack([case["parents"][(r, t)] for r in g]).to(dev)
            ctx.onela_reorder_beams(r0, n, par, W)
            for l in range(wl.L):
                tk = {nm: torch.stack([case["tok"][(r, l, t)][nm] for r in g]).to(dev) for nm in ("k", "v", "alpha", "beta")}
                q = torch.stack([case["q"][(r, l, t)] for r in g]).to(dev)
                out = torch.empty((n, W, wl.H, wl.dv), dtype=ctx.out_dtype, device=dev)
                if fused:     # one launch: append + decode
                    ctx.onela_append_decode_step(r0, n, l, tk["k"], tk["v"], tk["alpha"], tk["beta"], q, out)
                else:
                    ctx.onela_append_records(r0, n, l, tk["k"], tk["v"], tk["alpha"], tk["beta"])
                    ctx.onela_decode_step(r0, n, l, q, out)
                for i, r in enumerate(g):
                    outs[(r, l, t)] = out[i].float().cpu()
            for r in g:
                slots[(r, t)] = ctx.onela_export_chains(r).cpu().numpy()
    torch.cuda.synchronize()
    return outs, slots, ctx


def expected_slots(case, chains, batched=True) -> dict:
    """Global slot ids from the documented rule: one bump cursor; a reorder over a batch of requests
    assigns base(req, t) = cursor, cursor += W_t in request order; record of beam i at call t = base + i."""
    wl, widths = case["wl"], case["widths"]
    base, cursor = {}, 0
    for t, W in enumerate(widths):
        for r in range(wl.R):     # batched or one request at a time: the same order of allocation
            base[(r, t)] = cursor
            cursor += W
    out = {}
    for (r, t), ch in chains.items():
        out[(r, t)] = ch + np.array([base[(r, j)] for j in range(t + 1)])[None, :]
    return out


def check_parity(case, outs, ref, bar=REL_L2_BAR, tight=None, label=""):
    worst = 0.0
    for key, o in outs.items():
        e = rel_l2(o.numpy(), ref[key])
        worst = max(worst, float(e.max()))
        assert e.max() <= bar, f"{label} {key}: rel-L2 {e.max():.3e} > {bar}"
        if tight is not None:
            assert e.max() <= tight, f"{label} {key}: rel-L2 {e.max():.3e} above the expected {tight} for this arithmetic"
    return worst
