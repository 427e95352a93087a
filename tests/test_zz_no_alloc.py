"""onela_select_beams_static: beam selection for hosts that cannot give the library device memory - a server that
handed the whole GPU to its own pool, a plug-in on a borrowed stream where cudaMalloc's device-wide stall is not
allowed.  It keeps its partial lists in an array built into the library instead of a workspace.

Checked here through the C ABI: its parents, codes and scores equal those of onela_select_beams (the workspace
version) and those of the selection oracle, on two calls in a row with different inputs - the second call finds the
first call's leftovers in the shared array and must not be disturbed by them - and that no call allocates device
memory: neither PyTorch's allocator nor the driver's count of free bytes moves (the very first call of a process
loads the library's device code, so one call is made before the counts are taken).  Requests beyond the built-in
array's room are refused.

This file sorts last on purpose: a run that stops at the first failure has then run every other test."""
import pytest
import torch

import oracle.select
import paper_2609_12399_b200 as P
from paper_2609_12399_b200 import binding

pytestmark = pytest.mark.gpu


def _inputs(seed, R, W_prev, C, quant=None):
    gen = torch.Generator().manual_seed(seed)
    bs = torch.log_softmax(torch.randn((R, W_prev), generator=gen), -1)
    lp = torch.log_softmax(torch.randn((R, W_prev, C), generator=gen), -1)
    if quant:
        bs, lp = torch.round(bs * quant) / quant, torch.round(lp * quant) / quant      # exact ties
    return bs.float().cuda(), lp.float().cuda()


def _outputs(R, W_new):
    return (torch.empty((R, W_new), dtype=torch.int32, device="cuda"), torch.empty((R, W_new), dtype=torch.int32, device="cuda"),
            torch.empty((R, W_new), dtype=torch.float32, device="cuda"))


def test_static_selection_matches_the_workspace_version_twice_and_allocates_nothing():
    R, W, C = 2, 512, 256
    cfg = P.make_config(R, 1, 2, 128, 128, W, 2, "bf16", "bf16", R * W * 2, 0)
    ctx = P.Onela(cfg, device="cuda")
    for r in range(R):
        ctx.onela_init_shared_state(r, 0, torch.zeros(2, 128, 128, device="cuda"))
    ctx.onela_reorder_beams(0, R, None, W)                     # the workspace version reads W_prev from the context
    # first call: many candidates (parts + merge through the built-in array); second: ties, a different width,
    # fewer survivors - it runs over whatever the first call left in the array
    cases = [(_inputs(71, R, W, C), W), (_inputs(72, R, W, C, quant=4), 300)]
    P.onela_select_beams_static(*cases[0][0], W, *_outputs(R, W))     # module load and the array's address: once per process
    torch.cuda.synchronize()
    for (bs, lp), W_new in cases:
        want = _outputs(R, W_new)
        ctx.onela_select_beams(0, R, bs, lp, C, W_new, *want)
        got = _outputs(R, W_new)
        torch.cuda.synchronize()
        before = torch.cuda.memory_allocated(), torch.cuda.memory_reserved(), torch.cuda.mem_get_info()[0]
        P.onela_select_beams_static(bs, lp, W_new, *got)
        torch.cuda.synchronize()
        assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved(), torch.cuda.mem_get_info()[0]) == before
        assert torch.equal(got[0], want[0]), "parents"
        assert torch.equal(got[1], want[1]), "codes"
        assert torch.equal(got[2].view(torch.int32), want[2].view(torch.int32)), "scores, bit for bit"
        for r in range(R):      # and the oracle's selection, request by request
            op, oc, osc = oracle.select.select_beams(bs[r].cpu().numpy(), lp[r].cpu().numpy(), W_new)
            assert (got[0][r].cpu().numpy() == op).all() and (got[1][r].cpu().numpy() == oc).all()
            assert (got[2][r].cpu().numpy().view("int32") == osc.view("int32")).all()
    assert ctx.onela_poll_device_status() == (0, 0)


def test_sizes_beyond_the_built_in_array_are_refused():
    bs, lp = _inputs(73, 3, 8, 16)                             # three requests: one more than the array has room for
    with pytest.raises(binding.OnelaError) as e:
        P.onela_select_beams_static(bs, lp, 8, *_outputs(3, 8))
    assert e.value.status == binding.E_CAPACITY
    bs, lp = _inputs(74, 1, 8, 16)
    with pytest.raises(binding.OnelaError) as e:
        P.onela_select_beams_static(bs, lp, 1025, *_outputs(1, 1025))    # more survivors than a list holds
    assert e.value.status == binding.E_CAPACITY
    with pytest.raises(binding.OnelaError) as e:
        P.onela_select_beams_static(bs, lp, 129, *_outputs(1, 129))      # more survivors than candidates
    assert e.value.status == binding.E_CAPACITY
    P.onela_select_beams_static(bs, lp, 128, *_outputs(1, 128))          # everything: a full sort
    torch.cuda.synchronize()
