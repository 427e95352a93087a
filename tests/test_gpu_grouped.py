"""Grouped value heads (num_v_heads = g * num_heads: value head j reads the queries and keys of key head j // g)
through the C ABI against the oracle's grouped evaluation: outputs within the path's bar (tight for fp32 records),
ancestry rows bit-exact, and the split record planes (k per key head, v and gates per value head) byte for byte."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_12399_b200 as P
from paper_2609_12399_b200 import binding, inputs

from _cases import REL_L2_BAR, rel_l2

pytestmark = pytest.mark.gpu

CFG1 = inputs.WORKLOADS[1]


def _grouped_case(wl, g):
    """Inputs of a workload with wl.H VALUE heads; the key side keeps every g-th head of the seeded draws."""
    Hk = wl.H // g
    case = {"S0": {}, "tok": {}, "q": {}, "parents": {}}
    for r in range(wl.R):
        for t in range(wl.D):
            case["parents"][(r, t)] = None if t == 0 else inputs.parents(wl, r, t)
        for l in range(wl.L):
            p = inputs.prompt_tokens(wl, r, l)
            S = oracle.prefill_grouped(p["k"][:, ::g], p["v"], p["alpha"], p["beta"])
            case["S0"][(r, l)] = torch.from_numpy(S.astype(np.float32))
            for t in range(wl.D):
                tk = inputs.decode_token(wl, r, l, t)
                case["tok"][(r, l, t)] = {"k": tk["k"][:, ::g].contiguous(), "v": tk["v"], "alpha": tk["alpha"], "beta": tk["beta"]}
                case["q"][(r, l, t)] = inputs.decode_query(wl, r, l, t)[:, ::g].contiguous()
    assert case["q"][(0, 0, 0)].shape[1] == Hk
    return case


def _run(wl, g, out_dtype, fused, tight=None, flags=0):
    Hk = wl.H // g
    case = _grouped_case(wl, g)
    cfg = P.make_config(wl.R, wl.L, Hk, wl.dk, wl.dv, wl.W, wl.D, wl.dtype, out_dtype, wl.R * wl.W * wl.D, flags, num_v_heads=wl.H)
    ctx = P.Onela(cfg, device="cuda")
    # the warp-specialised tensor-core kernel takes dk = 128 with bf16 records, grouped or not; the tiled one the
    # other shapes; the CUDA-core kernel runs only when forced
    assert ctx.onela_uses_tensor_core_path() == (0 if flags else 1 if (wl.dk == 128 and wl.dtype == "bf16") else 2)
    dev = torch.device("cuda")
    for (r, l), S in case["S0"].items():
        ctx.onela_init_shared_state(r, l, S.to(dev))
    worst = 0.0
    for t in range(wl.D):
        par = None if t == 0 else torch.stack([case["parents"][(r, t)] for r in range(wl.R)]).to(dev)
        ctx.onela_reorder_beams(0, wl.R, par, wl.W)
        for l in range(wl.L):
            tk = {n: torch.stack([case["tok"][(r, l, t)][n] for r in range(wl.R)]).to(dev) for n in ("k", "v", "alpha", "beta")}
            q = torch.stack([case["q"][(r, l, t)] for r in range(wl.R)]).to(dev)
            out = torch.empty((wl.R, wl.W, wl.H, wl.dv), dtype=ctx.out_dtype, device=dev)
            if fused:
                ctx.onela_append_decode_step(0, wl.R, l, tk["k"], tk["v"], tk["alpha"], tk["beta"], q, out)
            else:
                ctx.onela_append_records(0, wl.R, l, tk["k"], tk["v"], tk["alpha"], tk["beta"])
                ctx.onela_decode_step(0, wl.R, l, q, out)
            for r in range(wl.R):
                steps = [case["tok"][(r, l, j)] for j in range(t + 1)]
                pars = [case["parents"][(r, j)] for j in range(t + 1)]
                ref = oracle.decode_grouped(case["S0"][(r, l)], steps, pars, case["q"][(r, l, t)])
                e = rel_l2(out[r].float().cpu().numpy(), ref)
                worst = max(worst, float(e.max()))
                assert e.max() <= (tight or REL_L2_BAR), f"request {r} layer {l} call {t}: rel-L2 {e.max():.3e}"
    assert ctx.onela_poll_device_status() == (0, 0)
    return case, ctx, worst


@pytest.mark.parametrize("g,fused,flags", [(2, False, 0), (4, True, 0), (2, True, P.FLAG_FORCE_GENERIC), (1, True, 0)])
def test_grouped_heads_bf16(g, fused, flags):
    """Tensor-core kernel (separate and fused append) and, forced, the CUDA-core kernels; g = 1 with num_v_heads set
    is the ungrouped path."""
    wl = CFG1.scaled(R=2, L=2, H=8, W=70, D=3, prompt_len=64, parents="zipf", zipf_s=1.3, seed=1300 + g)
    _run(wl, g, "bf16", fused, flags=flags)


def test_grouped_heads_on_the_tensor_core_kernel_many_segments_and_depth():
    """More (request, value head) pairs than SMs, staged and gathered ancestors, ragged groups: the grouped
    instantiation of the tensor-core kernel walks several segments per CTA."""
    wl = CFG1.scaled(R=6, L=1, H=32, W=100, D=6, prompt_len=32, parents="zipf", zipf_s=1.4, seed=1330)
    _, ctx, worst = _run(wl, 4, "fp32", True)
    assert ctx.onela_uses_tensor_core_path() and worst <= REL_L2_BAR


def test_grouped_heads_fp32_is_tight_and_other_shapes():
    """fp32 records and the 64 x 64 shape: the tiled tensor-core kernel within the bar, the CUDA-core kernel (fp32
    throughout) within rounding."""
    for flags, tight in ((0, None), (P.FLAG_FORCE_GENERIC, 5e-6)):
        _run(CFG1.scaled(H=4, dtype="fp32", W=33, D=4, prompt_len=48, seed=1310), 2, "fp32", True, tight=tight, flags=flags)
        _run(CFG1.scaled(H=6, dk=64, dv=64, dtype="fp32", W=20, D=3, prompt_len=32, seed=1311), 3, "fp32", False, tight=tight, flags=flags)
    _run(CFG1.scaled(H=4, dk=128, dv=256, W=40, D=3, prompt_len=32, seed=1312), 2, "fp32", True)


@pytest.mark.parametrize("dk,dv,dtype,g", [(64, 64, "bf16", 2), (64, 64, "fp32", 4), (128, 128, "fp32", 2), (128, 256, "fp32", 3)])
def test_grouped_heads_on_the_tiled_tensor_core_kernel(dk, dv, dtype, g):
    """The shapes the warp-specialised kernel does not take, grouped: deeper chains with shared ancestors, several
    requests and layers, a ragged last tile of beams, bf16 outputs."""
    wl = CFG1.scaled(R=2, L=2, H=2 * g, dk=dk, dv=dv, dtype=dtype, W=45, D=5, prompt_len=32, parents="zipf", zipf_s=1.4, seed=1340 + dk + dv)
    _, ctx, worst = _run(wl, g, "bf16" if dtype == "bf16" else "fp32", dtype == "bf16")
    assert ctx.onela_uses_tensor_core_path() == 2 and worst <= REL_L2_BAR


@pytest.mark.parametrize("fused", [False, True])
def test_split_record_planes_hold_the_appended_bytes(fused):
    wl = CFG1.scaled(R=1, L=1, H=4, W=10, D=2, prompt_len=16, seed=1320)
    g, Hk = 2, 2
    case, ctx, _ = _run(wl, g, "fp32", fused)
    c = ctx.cfg
    al = lambda n: (n + 1023) // 1024 * 1024
    n_idx = c.num_requests * c.max_steps * c.max_beam * 4
    off_s0 = al(16) + al(2 * n_idx) + al(n_idx) + al(n_idx) + al(c.num_requests * (c.max_steps + 1) * 4)
    off_gates = off_s0 + al(c.num_requests * c.num_layers * wl.H * c.dv * c.dk * 4)
    off_k = off_gates + al(c.num_layers * wl.H * c.arena_slots * 8)
    off_v = off_k + al(c.num_layers * Hk * c.arena_slots * c.dk * 2)
    ws = ctx.workspace[ctx.workspace_ptr - ctx.workspace.data_ptr():]
    gates = ws[off_gates:off_gates + wl.H * c.arena_slots * 8].view(torch.float32).view(wl.H, c.arena_slots, 2).cpu()
    kp = ws[off_k:off_k + Hk * c.arena_slots * c.dk * 2].view(torch.bfloat16).view(Hk, c.arena_slots, c.dk).cpu()
    vp = ws[off_v:off_v + wl.H * c.arena_slots * c.dv * 2].view(torch.bfloat16).view(wl.H, c.arena_slots, c.dv).cpu()
    for t in range(wl.D):
        base = ctx.onela_get_step_base(0, t)
        tk = case["tok"][(0, 0, t)]
        for h in range(Hk):
            assert torch.equal(kp[h, base:base + wl.W], tk["k"][:, h])
        for h in range(wl.H):
            assert torch.equal(vp[h, base:base + wl.W], tk["v"][:, h])
            assert torch.equal(gates[h, base:base + wl.W, 0], tk["alpha"][:, h])
            assert torch.equal(gates[h, base:base + wl.W, 1], tk["beta"][:, h])
    # resident bytes: k once per key head, v and the gates per value head
    slots = wl.W * wl.D
    assert ctx.onela_get_stats()["arena_bytes_used"] == slots * (Hk * c.dk * 2 + wl.H * (c.dv * 2 + 8))
