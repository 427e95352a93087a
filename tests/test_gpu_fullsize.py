"""Parity at the benchmark configs' FULL sizes, in the launch configuration bench.py times (all requests
of a layer in one batched call, the one-launch append_decode_step, bf16 outputs, the tensor-core kernel).

For the checked (request, layer) pairs the oracle replays EVERY (beam, head) unit of EVERY decode call:
all of config 2, one pair per request of config 3, first and last layer of every request of config 4.
S_0 is an input of the decode path: for a few pairs it comes from the oracle's fp64 prefill of the seeded
prompt, for the others it is read back from the library's store (the prefill kernel's result, itself checked
against the oracle's prefill elsewhere) and handed to the oracle, so both sides consume identical inputs.
Integer work is checked everywhere: the ancestry rows of every request at every call against Eq. 5.  One more
property holds at any size and is checked on every unit of every pair: the tensor-core kernel and the
CUDA-core kernel, which share no device code, agree.
"""
import numpy as np
import pytest
import torch

import oracle
from oracle import evaluators as ev
import paper_2609_12399_b200 as P
from paper_2609_12399_b200 import inputs
from paper_2609_12399_b200.runner import WorkloadRun

from _cases import REL_L2_BAR, rel_l2

pytestmark = pytest.mark.gpu


def _oracle_state(wl, r, l):
    parts = [inputs.prompt_tokens(wl, r, l, a, min(a + 2048, wl.prompt_len), device="cuda")
             for a in range(0, wl.prompt_len, 2048)]
    p = {n: torch.cat([x[n] for x in parts]).cpu() for n in ("k", "v", "alpha", "beta")}
    return torch.from_numpy(oracle.prefill(p["k"], p["v"], p["alpha"], p["beta"]).astype(np.float32))


def _run_and_check(wl, oracle_pairs, store_pairs, check_calls, flags=0, keep_calls=(), fused=True):
    """Run the whole generation; compare every unit of the calls in `check_calls` for the given pairs with the
    oracle.  `oracle_pairs` take S_0 from the oracle's prefill, `store_pairs` from the library's store."""
    run = WorkloadRun(wl, "cuda", "bf16", flags=flags)
    S0 = {pr: _oracle_state(wl, *pr) for pr in oracle_pairs}
    run.prefill_states(overrides=S0)
    for pr in store_pairs:
        S0[pr] = run.ctx.onela_export_shared_state(*pr).cpu()
    pairs = list(oracle_pairs) + list(store_pairs)
    outs = run.alloc_outputs()
    hist = {pr: {"tok": [], "par": [None]} for pr in pairs}
    parents_all = {r: [None] for r in range(wl.R)}
    worst, kept, units = 0.0, {}, 0
    for t in range(wl.D):
        call = run.generate_call(t)
        run.run_call(call, outs, fused=fused)     # fused: the launch configuration bench.py times
        torch.cuda.synchronize()
        if t > 0:
            par = call["parents"].cpu().numpy()
            for r in range(wl.R):
                parents_all[r].append(par[r])
        # ancestry rows of EVERY request: Eq. 5 table + the slot rule (base(req, t) = t*R*W + r*W here)
        for r in range(wl.R):
            rows = ev.ancestry_table(parents_all[r], [wl.W] * (t + 1))
            want = rows + np.array([j * wl.R * wl.W + r * wl.W for j in range(t + 1)])[None, :]
            got = run.ctx.onela_export_chains(r).cpu().numpy()
            assert np.array_equal(got, want), f"ancestry rows of request {r} at call {t}"
        for (r, l) in pairs:
            lay = call["layers"][l]
            hist[(r, l)]["tok"].append({n: lay[n][r].cpu() for n in ("k", "v", "alpha", "beta")})
            if t > 0:
                hist[(r, l)]["par"].append(parents_all[r][t])
            if t in check_calls:
                ref = oracle.decode(S0[(r, l)], hist[(r, l)]["tok"], hist[(r, l)]["par"], lay["q"][r].cpu())
                e = rel_l2(outs[l][r].float().cpu().numpy(), ref)
                units += e.size
                worst = max(worst, float(e.max()))
                assert e.max() <= REL_L2_BAR, f"pair {(r, l)} call {t}: rel-L2 {e.max():.3e}"
        if t in keep_calls:
            kept[t] = [o.clone() for o in outs]
        assert torch.isfinite(outs[0].float()).all()
    assert run.ctx.onela_poll_device_status() == (0, 0)
    return worst, kept, run, units


def _two_kernels_agree(wl, calls):
    """Every unit of every (request, layer) pair at the given calls: tensor-core kernel against CUDA-core kernel."""
    _, tc, run, _ = _run_and_check(wl, [], [], [], keep_calls=calls)
    assert run.ctx.onela_uses_tensor_core_path()
    del run
    _, cc, run2, _ = _run_and_check(wl, [], [], [], flags=P.FLAG_FORCE_GENERIC, keep_calls=calls, fused=False)
    assert not run2.ctx.onela_uses_tensor_core_path()
    for t in calls:
        for l in range(wl.L):
            assert rel_l2(tc[t][l].float().cpu().numpy(), cc[t][l].float().cpu().numpy()).max() <= REL_L2_BAR, (t, l)


def test_config2_beam512_zipf_every_call():
    """32 heads, beam 512, depth 4, Zipf(1.2) parents, 16384-token prompt: every unit of every call against the
    oracle (65 536 decodes), and the two kernels against each other on every unit of every call."""
    wl = inputs.WORKLOADS[2]
    worst, _, run, units = _run_and_check(wl, [(0, 0)], [], range(wl.D))
    assert run.ctx.onela_uses_tensor_core_path() and units == wl.D * wl.W * wl.H
    del run
    _two_kernels_agree(wl, list(range(wl.D)))


def test_config3_batch8_beam1024():
    """8 requests in one shared arena, beam 1024, depth 6, uniform parents: every unit of every call of every
    request (fused launches), every unit of two requests with separate append and decode launches, and the two
    kernels against each other at the deepest call."""
    wl = inputs.WORKLOADS[3]
    _, _, _, units = _run_and_check(wl, [(0, 0), (7, 0)], [(r, 0) for r in range(1, 7)], range(wl.D))
    assert units == wl.R * wl.D * wl.W * wl.H
    _run_and_check(wl, [], [(3, 0), (4, 0)], range(wl.D), fused=False)
    _two_kernels_agree(wl, [wl.D - 1])


def test_config4_stack16_beam512():
    """16 layers x 4 requests, beam 512, depth 8, Zipf(1.5) parents with heavy duplication: every unit of every
    call for the first and the last layer of every request (plus one middle layer), and the two kernels against
    each other on every unit of the deepest call of all 64 (request, layer) pairs."""
    wl = inputs.WORKLOADS[4]
    store = [(r, l) for r in range(wl.R) for l in (0, wl.L - 1) if (r, l) not in ((0, 0), (3, 15))]
    _, _, _, units = _run_and_check(wl, [(0, 0), (3, 15), (1, 7)], store, range(wl.D))
    assert units == 9 * wl.D * wl.W * wl.H
    _two_kernels_agree(wl, [wl.D - 1])
