"""GPU parity of the tensor-core kernel for chains with heavily shared ancestors (ONELA_FLAG_SHARED_CHAINS)
against the fp64 full-state oracle, through the C ABI: every (beam, head) output of every decode call."""
import numpy as np
import pytest
import torch

import paper_2609_12399_b200 as P
from paper_2609_12399_b200 import inputs

from _cases import check_parity, expected_slots, make_case, run_library, run_oracle

pytestmark = pytest.mark.gpu

CFG4 = inputs.WORKLOADS[4]


def distinct_counts(case):
    """Per request and decode call: (distinct older records, those older than the parents), from the parents."""
    wl, widths = case["wl"], case["widths"]
    out = {}
    for r in range(wl.R):
        table = None
        for t, W in enumerate(widths):
            own = torch.arange(W)[None, :]
            table = own if t == 0 else torch.cat([table[:, case["parents"][(r, t)].long()], own], 0)
            counts = [len(torch.unique(table[l])) for l in range(t)]
            out[(r, t)] = (sum(counts), sum(counts[:-1]))
    return out


def _check(wl, out_dtype, fused, widths=None):
    case = make_case(wl, widths=widths)
    counts = distinct_counts(case)
    assert max(c[0] for c in counts.values()) <= 160 and max(c[1] for c in counts.values()) <= 64, counts
    ref, chains = run_oracle(case)
    outs, slots, ctx = run_library(case, out_dtype=out_dtype, flags=P.FLAG_SHARED_CHAINS, fused=fused)
    assert ctx.onela_poll_device_status() == (0, 0)
    want = expected_slots(case, chains)
    assert all(np.array_equal(slots[k], want[k]) for k in want)
    worst = check_parity(case, outs, ref, label="shared-chains kernel")
    return worst, counts


@pytest.mark.parametrize("out_dtype,fused", [("fp32", True), ("bf16", True), ("fp32", False)])
def test_small_stack_matches_oracle(out_dtype, fused):
    wl = CFG4.scaled(R=2, L=2, H=3, W=112, D=5, prompt_len=96)
    worst, _ = _check(wl, out_dtype, fused)
    assert worst < (3e-3 if out_dtype == "bf16" else 1.5e-3)


def test_deep_chains_ragged_beam():
    wl = CFG4.scaled(R=1, L=1, H=5, W=200, D=8, prompt_len=64)
    worst, counts = _check(wl, "fp32", True)
    assert worst < 1.5e-3, (worst, counts)


def test_more_than_128_distinct_records():
    # enough beams and a flatter parent law that some call has more than 128 distinct older records
    wl = CFG4.scaled(R=1, L=1, H=2, W=512, D=8, prompt_len=64)
    worst, counts = _check(wl, "fp32", True)
    assert max(c[0] for c in counts.values()) > 128, counts
    assert worst < 1.5e-3, (worst, counts)


def test_full_size_stack_every_unit():
    """The beam-512 decode stack at full width and depth (4 requests x 32 heads x 512 beams, depth 8, Zipf(1.5)), two
    layers: every unit of every call from the second on, first and last layer of every request."""
    from test_gpu_fullsize import _run_and_check
    wl = CFG4.scaled(L=2)
    pairs = [(r, l) for r in range(wl.R) for l in range(wl.L)]
    _, _, run, units = _run_and_check(wl, [], pairs, range(1, wl.D), flags=P.FLAG_SHARED_CHAINS)
    assert units == len(pairs) * (wl.D - 1) * wl.W * wl.H


def test_more_pairs_than_sms_several_segments_per_cta():
    """More (request, head) pairs than SMs, so a CTA works through several segments (S_0, the node tables and U are
    rebuilt between them, the beams' index bytes when the request changes), with a ragged last group."""
    wl = CFG4.scaled(R=5, L=1, H=34, W=60, D=4, prompt_len=32, seed=77)
    worst, _ = _check(wl, "fp32", True)
    assert worst < 1.5e-3
