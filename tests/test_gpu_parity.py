"""Parity of the CUDA path against the CPU oracle, element by element, through the C ABI.

Bar: ancestry chains and slot ids bit-exact; outputs within 5e-3 relative L2 per (beam, head) vector
of the fp64 oracle.  Where the arithmetic allows a much tighter bound (fp32 fold and contraction with
fp32 output: rounding only), that bound is asserted as well so a regression cannot hide under the bar.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_12399_b200 as P
from paper_2609_12399_b200 import binding, inputs

from _cases import (REL_L2_BAR, check_parity, expected_slots, make_case, rel_l2, run_library, run_oracle)

pytestmark = pytest.mark.gpu

CFG0, CFG1 = inputs.WORKLOADS[0], inputs.WORKLOADS[1]


def _small(base, **kw):
    return base.scaled(**kw)


def _full_check(case, out_dtype, flags=0, batched=True, tight=None, fused=False):
    ref, chains = run_oracle(case)
    outs, slots, ctx = run_library(case, out_dtype=out_dtype, flags=flags, batched=batched, fused=fused)
    want = expected_slots(case, chains)
    for key in want:
        assert np.array_equal(slots[key], want[key]), f"ancestry rows of {key} differ"
    worst = check_parity(case, outs, ref, tight=tight)
    assert ctx.onela_poll_device_status() == (0, 0)
    return worst, ctx


def test_config0_tiny_reference():
    """1 request, 1 layer, 2 heads, dk = dv = 32, fp32, beam 8, 3 calls, uniform parents."""
    worst, ctx = _full_check(make_case(CFG0), "fp32", tight=2e-6)
    assert not ctx.onela_uses_tensor_core_path()


@pytest.mark.parametrize("out_dtype,tight", [("fp32", None), ("bf16", None)])
def test_config1_beam128(out_dtype, tight):
    """16 heads, dk = dv = 128, bf16 records, beam 128, depth 4, uniform parents; every call, every unit."""
    _full_check(make_case(CFG1), out_dtype, tight=tight)


@pytest.mark.parametrize("out_dtype", ["fp32", "bf16"])
def test_config1_fused_append_decode(out_dtype):
    """The one-launch append + decode entry point on config 1: same outputs, same chains."""
    _full_check(make_case(CFG1), out_dtype, fused=True)


def test_fused_append_decode_other_paths():
    _full_check(make_case(CFG0), "fp32", fused=True, tight=2e-6)                       # CUDA-core shapes: two launches inside
    wl = CFG1.scaled(R=3, L=2, H=4, W=77, D=4, prompt_len=96, parents="zipf", zipf_s=1.3, seed=78)
    _full_check(make_case(wl), "bf16", fused=True)                                      # ragged width, shared ancestors
    _full_check(make_case(wl, widths=[77, 5, 130, 48]), "fp32", fused=True, batched=False)


def test_config1_cuda_core_kernel_is_fp32_accurate():
    _full_check(make_case(CFG1.scaled(prompt_len=256)), "fp32", flags=P.FLAG_FORCE_GENERIC, tight=5e-6)


@pytest.mark.parametrize("W", [1, 31, 33, 77, 200])
def test_ragged_beam_widths(W):
    """Beam widths that are not a multiple of any tile: a partial tail tile, and tiles of one beam."""
    wl = CFG1.scaled(H=3, W=W, D=3, prompt_len=64, seed=500 + W)
    _full_check(make_case(wl), "fp32")
    _full_check(make_case(wl), "fp32", flags=P.FLAG_FORCE_GENERIC, tight=5e-6)


def test_multi_request_multi_layer_batched_and_unbatched():
    wl = CFG1.scaled(R=3, L=2, H=4, W=40, D=3, prompt_len=96, parents="zipf", zipf_s=1.3, seed=77)
    case = make_case(wl)
    _full_check(case, "bf16", batched=True)
    _full_check(case, "fp32", batched=False)


@pytest.mark.parametrize("fused", [False, True])
def test_many_short_segments_per_cta(fused):
    """More (request, head) pairs than three per SM, each a single group or two: every CTA of the tensor-core
    kernel walks through several segments, alternating its two S_0 / staging buffers, with staged ancestors
    (Zipf parents, depth 4) and a ragged last group."""
    wl = CFG1.scaled(R=20, L=1, H=32, W=40, D=4, prompt_len=16, parents="zipf", zipf_s=1.4, seed=4242)
    _full_check(make_case(wl), "bf16", fused=fused)
    wl = CFG1.scaled(R=12, L=1, H=32, W=70, D=3, prompt_len=16, parents="uniform", seed=4243)
    _full_check(make_case(wl), "fp32", fused=fused)


def test_degenerate_shapes():
    """A single beam; the largest batch one call takes (64 requests) with one head and one beam each; one group
    that is exactly full (48 beams) and one that has a single beam in its second group (49)."""
    _full_check(make_case(CFG1.scaled(H=2, W=1, D=3, prompt_len=32, seed=701)), "fp32")
    _full_check(make_case(CFG1.scaled(R=64, H=1, W=1, D=2, prompt_len=8, seed=702)), "bf16", fused=True)
    _full_check(make_case(CFG1.scaled(H=2, W=48, D=2, prompt_len=32, seed=703)), "fp32", fused=True)
    _full_check(make_case(CFG1.scaled(H=2, W=49, D=2, prompt_len=32, parents="zipf", zipf_s=2.0, seed=704)), "fp32", fused=True)


def test_released_slots_are_reused_while_another_request_goes_on():
    """Continuous batching: request 0 finishes after two calls and is released; a new generation starts in its slot
    and lands on the freed record slots while request 1 keeps decoding.  Both must match the oracle: the newcomer is
    not disturbed by stale records, the survivor's records are not touched."""
    wl = CFG1.scaled(R=2, L=1, H=4, W=40, D=4, prompt_len=64, parents="zipf", zipf_s=1.3, seed=911)
    case = make_case(wl)
    ref, _ = run_oracle(case)
    W = wl.W
    cfg = P.make_config(wl.R, wl.L, wl.H, wl.dk, wl.dv, W, wl.D, wl.dtype, "fp32", 6 * W, 0)
    ctx = P.Onela(cfg, device="cuda")
    dev = torch.device("cuda")

    def step(r, t):
        par = None if t == 0 else case["parents"][(r, t)][None].to(dev)
        ctx.onela_reorder_beams(r, 1, par, W)
        tk = {n: x[None].to(dev) for n, x in case["tok"][(r, 0, t)].items()}
        out = torch.empty((1, W, wl.H, wl.dv), dtype=torch.float32, device=dev)
        ctx.onela_append_decode_step(r, 1, 0, tk["k"], tk["v"], tk["alpha"], tk["beta"], case["q"][(r, 0, t)][None].to(dev), out)
        e = rel_l2(out[0].cpu().numpy(), ref[(r, 0, t)])
        assert e.max() <= REL_L2_BAR, f"request {r} call {t}: rel-L2 {e.max():.3e}"

    for r in range(2):
        ctx.onela_init_shared_state(r, 0, case["S0"][(r, 0)].to(dev))
    for t in range(2):
        for r in range(2):
            step(r, t)
    assert [ctx.onela_get_step_base(r, t) for r in range(2) for t in range(2)] == [0, 2 * W, W, 3 * W]
    ctx.onela_release_request(0)
    ctx.onela_init_shared_state(0, 0, case["S0"][(0, 0)].to(dev))      # the next prompt in slot 0
    step(0, 0)                                                          # -> freed [0, W)
    step(1, 2)                                                          # -> freed [2W, 3W)
    step(0, 1)                                                          # -> the cursor
    step(1, 3)
    assert [ctx.onela_get_step_base(0, t) for t in range(2)] == [0, 4 * W]
    assert [ctx.onela_get_step_base(1, t) for t in range(4)] == [W, 3 * W, 2 * W, 5 * W]
    assert ctx.onela_poll_device_status() == (0, 0)


def test_varying_beam_width_between_calls():
    wl = CFG1.scaled(H=2, W=96, D=4, prompt_len=64, seed=91)
    _full_check(make_case(wl, widths=[96, 17, 64, 5]), "fp32")


def test_depth_one_and_max_depth():
    _full_check(make_case(CFG1.scaled(H=2, W=64, D=1, prompt_len=64)), "fp32")
    _full_check(make_case(CFG1.scaled(H=2, W=48, D=12, prompt_len=64, parents="zipf", zipf_s=1.5)), "fp32")


@pytest.mark.parametrize("dk,dv,dtype", [(64, 64, "bf16"), (64, 64, "fp32"), (128, 128, "fp32"), (128, 256, "bf16"),
                                         (256, 256, "bf16"), (32, 32, "bf16"), (128, 512, "bf16"), (256, 512, "bf16")])
def test_other_geometries(dk, dv, dtype):
    wl = CFG1.scaled(H=2, dk=dk, dv=dv, dtype=dtype, W=37, D=3, prompt_len=48, seed=dk + dv)
    _, ctx = _full_check(make_case(wl), "fp32")
    # key width 128 with bf16 records runs on the warp-specialised tensor-core kernel at every value width (256 and 512
    # as two and four value tiles of 128 outputs); the other shapes from 64 x 64 up on the tiled tensor-core kernel;
    # 32 x 32 on CUDA cores
    assert ctx.onela_uses_tensor_core_path() == (1 if (dk == 128 and dtype == "bf16") else 2 if dk >= 64 else 0)


@pytest.mark.parametrize("dk,dv,dtype", [(64, 64, "bf16"), (64, 64, "fp32"), (128, 128, "fp32"), (128, 256, "fp32"), (128, 512, "fp32"),
                                         (256, 256, "bf16"), (256, 256, "fp32"), (256, 512, "bf16"), (256, 512, "fp32")])
@pytest.mark.parametrize("fused,out_dtype", [(True, "bf16"), (False, "fp32")])
def test_tiled_tensor_core_kernel(dk, dv, dtype, fused, out_dtype):
    """Key widths 64 and 256, value widths to 512 and fp32 records (Section 4.1's operator suite) on the tiled tcgen05
    kernel: deeper chains with shared ancestors, several requests and layers, beam widths with a ragged last tile and
    more than one tile; every unit against the oracle, and against the CUDA-core kernel, whose contraction shares no
    code with it."""
    wl = CFG1.scaled(R=2, L=2, H=3, dk=dk, dv=dv, dtype=dtype, W=77, D=5, prompt_len=48, parents="zipf", zipf_s=1.4, seed=950 + dk + dv)
    case = make_case(wl)
    ref, chains = run_oracle(case)
    outs, slots, ctx = run_library(case, out_dtype=out_dtype, fused=fused)
    assert ctx.onela_uses_tensor_core_path() == 2 and ctx.onela_poll_device_status() == (0, 0)
    want = expected_slots(case, chains)
    for key in want:
        assert np.array_equal(slots[key], want[key])
    check_parity(case, outs, ref)
    outs_cc, _, ctx_cc = run_library(case, out_dtype=out_dtype, flags=P.FLAG_FORCE_GENERIC, fused=fused)
    assert ctx_cc.onela_uses_tensor_core_path() == 0
    for key in outs:
        assert rel_l2(outs[key].numpy(), outs_cc[key].double().numpy()).max() <= REL_L2_BAR
    # the arena rows [k | v] and the gates of every layer hold the appended bytes (with `fused` the decode launch wrote them)
    c = ctx.cfg
    al = lambda n: (n + 1023) // 1024 * 1024
    n_idx = c.num_requests * c.max_steps * c.max_beam * 4
    off_s0 = al(16) + al(2 * n_idx) + al(n_idx) + al(n_idx) + al(c.num_requests * (c.max_steps + 1) * 4)
    off_gates = off_s0 + al(c.num_requests * c.num_layers * c.num_heads * c.dv * c.dk * 4)
    off_kv = off_gates + al(c.num_layers * c.num_heads * c.arena_slots * 8)
    ws = ctx.workspace[ctx.workspace_ptr - ctx.workspace.data_ptr():]
    row, eb, td = dk + dv, (2 if dtype == "bf16" else 4), (torch.bfloat16 if dtype == "bf16" else torch.float32)
    for lay in range(wl.L):
        g0 = off_gates + lay * c.num_heads * c.arena_slots * 8
        k0 = off_kv + lay * c.num_heads * c.arena_slots * row * eb
        gates = ws[g0:g0 + c.num_heads * c.arena_slots * 8].view(torch.float32).view(c.num_heads, c.arena_slots, 2).cpu()
        kv = ws[k0:k0 + c.num_heads * c.arena_slots * row * eb].view(td).view(c.num_heads, c.arena_slots, row).cpu()
        for r in range(wl.R):
            for t in range(wl.D):
                base = ctx.onela_get_step_base(r, t)
                tk = case["tok"][(r, lay, t)]
                for h in range(wl.H):
                    assert torch.equal(kv[h, base:base + wl.W, :dk], tk["k"][:, h])
                    assert torch.equal(kv[h, base:base + wl.W, dk:], tk["v"][:, h])
                    assert torch.equal(gates[h, base:base + wl.W, 0], tk["alpha"][:, h])
                    assert torch.equal(gates[h, base:base + wl.W, 1], tk["beta"][:, h])


def test_tiled_tensor_core_kernel_edge_cases():
    """A single beam, exactly one full tile of 32 beams, one beam more, depth 1 and a long chain; keys and states far
    from unit scale (the operand rows' power-of-two scales must absorb them)."""
    for W, D, seed in ((1, 3, 1), (32, 2, 2), (33, 1, 3), (40, 12, 4)):
        wl = CFG1.scaled(H=2, dk=256, dv=256, W=W, D=D, prompt_len=32, parents="zipf", zipf_s=1.5, seed=970 + seed)
        _, ctx = _full_check(make_case(wl), "fp32")
        assert ctx.onela_uses_tensor_core_path() == 2
    wl = CFG1.scaled(H=2, dk=64, dv=64, dtype="fp32", W=50, D=4, prompt_len=16, seed=979)
    case = make_case(wl)
    for key in case["S0"]:
        case["S0"][key] = case["S0"][key] * 3.0e4
    for key in case["q"]:
        case["q"][key] = case["q"][key] * 1.0e-3
    _, ctx = _full_check(case, "fp32")
    assert ctx.onela_uses_tensor_core_path() == 2


@pytest.mark.parametrize("dv", [256, 512])
@pytest.mark.parametrize("fused,out_dtype", [(True, "bf16"), (False, "fp32")])
def test_wide_values_on_the_tensor_cores(dv, fused, out_dtype):
    """Value widths 256 and 512 (Section 4.1's operator suite) on the tcgen05 kernel: deeper chains with shared ancestors,
    several requests and layers, ragged beams; the arena rows hold the appended bytes; and the CUDA-core kernel, which
    shares no device code, agrees on every unit."""
    wl = CFG1.scaled(R=2, L=2, H=3, dk=128, dv=dv, W=77, D=5, prompt_len=48, parents="zipf", zipf_s=1.4, seed=900 + dv)
    case = make_case(wl)
    ref, chains = run_oracle(case)
    outs, slots, ctx = run_library(case, out_dtype=out_dtype, fused=fused)
    assert ctx.onela_uses_tensor_core_path() and ctx.onela_poll_device_status() == (0, 0)
    check_parity(case, outs, ref)
    outs_cc, _, ctx_cc = run_library(case, out_dtype=out_dtype, flags=P.FLAG_FORCE_GENERIC, fused=fused)
    assert not ctx_cc.onela_uses_tensor_core_path()
    for key in outs:
        assert rel_l2(outs[key].numpy(), outs_cc[key].double().numpy()).max() <= REL_L2_BAR
    # the arena rows [k | v] of the last layer, byte for byte
    c = ctx.cfg
    al = lambda n: (n + 1023) // 1024 * 1024
    n_idx = c.num_requests * c.max_steps * c.max_beam * 4
    off_s0 = al(16) + al(2 * n_idx) + al(n_idx) + al(n_idx) + al(c.num_requests * (c.max_steps + 1) * 4)
    off_gates = off_s0 + al(c.num_requests * c.num_layers * c.num_heads * c.dv * c.dk * 4)
    off_kv = off_gates + al(c.num_layers * c.num_heads * c.arena_slots * 8)
    ws = ctx.workspace[ctx.workspace_ptr - ctx.workspace.data_ptr():]
    row = 128 + dv
    lay = wl.L - 1
    g0 = off_gates + lay * c.num_heads * c.arena_slots * 8
    k0 = off_kv + lay * c.num_heads * c.arena_slots * row * 2
    gates = ws[g0:g0 + c.num_heads * c.arena_slots * 8].view(torch.float32).view(c.num_heads, c.arena_slots, 2).cpu()
    kv = ws[k0:k0 + c.num_heads * c.arena_slots * row * 2].view(torch.bfloat16).view(c.num_heads, c.arena_slots, row).cpu()
    for r in range(wl.R):
        for t in range(wl.D):
            base = ctx.onela_get_step_base(r, t)
            tk = case["tok"][(r, lay, t)]
            for h in range(wl.H):
                assert torch.equal(kv[h, base:base + wl.W, :128], tk["k"][:, h])
                assert torch.equal(kv[h, base:base + wl.W, 128:], tk["v"][:, h])
                assert torch.equal(gates[h, base:base + wl.W, 0], tk["alpha"][:, h])
                assert torch.equal(gates[h, base:base + wl.W, 1], tk["beta"][:, h])


@pytest.mark.parametrize("dk,dv,dtype", [(128, 128, "bf16"), (64, 64, "bf16"), (256, 512, "fp32")])
def test_alpha1_beta0_reduces_to_matvec_on_gpu(dk, dv, dtype):
    """On both tensor-core kernels (the second and third shapes run the tiled one)."""
    wl = CFG1.scaled(H=2, dk=dk, dv=dv, dtype=dtype, W=64, D=3, prompt_len=64)
    case = make_case(wl)
    for tk in case["tok"].values():
        tk["alpha"].fill_(1.0)
        tk["beta"].zero_()
    outs, _, _ = run_library(case, out_dtype="fp32")
    for (r, l, t), o in outs.items():
        want = np.einsum("hij,bhj->bhi", case["S0"][(r, l)].double().numpy(), case["q"][(r, l, t)].double().numpy())
        assert rel_l2(o.numpy(), want).max() <= REL_L2_BAR


@pytest.mark.parametrize("dk,dv,dtype", [(128, 128, "bf16"), (64, 64, "fp32"), (256, 256, "bf16")])
def test_shared_chains_give_identical_outputs_on_gpu(dk, dv, dtype):
    wl = CFG1.scaled(H=2, dk=dk, dv=dv, dtype=dtype, W=64, D=3, prompt_len=64)
    case = make_case(wl)
    case["parents"][(0, 2)] = torch.full((64,), 5, dtype=torch.int32)
    for n in ("k", "v", "alpha", "beta"):
        x = case["tok"][(0, 0, 2)][n]
        x[:] = x[0]
    case["q"][(0, 0, 2)][:] = case["q"][(0, 0, 2)][0]
    outs, _, _ = run_library(case, out_dtype="fp32")
    o = outs[(0, 0, 2)]
    assert torch.equal(o, o[0:1].expand_as(o))


@pytest.mark.parametrize("fused", [False, True])
def test_records_are_stored_bit_exactly_and_never_rewritten(fused):
    """The arena planes hold exactly the appended bytes at slot base(req, t) + beam, head-major, and a
    later reorder/append leaves earlier records untouched (read straight out of the workspace); the same
    through the fused append + decode launch."""
    wl = CFG1.scaled(R=2, H=3, W=20, D=3, prompt_len=32, seed=5)
    case = make_case(wl)
    outs, slots, ctx = run_library(case, out_dtype="fp32", fused=fused)
    c = ctx.cfg
    al = lambda n: (n + 1023) // 1024 * 1024
    off_tables = al(16)
    n_idx = c.num_requests * c.max_steps * c.max_beam * 4
    off_s0 = (off_tables + al(2 * n_idx)                    # ancestry tables (double-buffered)
              + al(n_idx) + al(n_idx)                       # distinct-record index: per-beam positions, slot list
              + al(c.num_requests * (c.max_steps + 1) * 4)) # ... and per-level offsets
    off_gates = off_s0 + al(c.num_requests * c.num_layers * c.num_heads * c.dv * c.dk * 4)
    off_kv = off_gates + al(c.num_layers * c.num_heads * c.arena_slots * 8)
    ws = ctx.workspace[ctx.workspace_ptr - ctx.workspace.data_ptr():]
    gates = ws[off_gates:off_gates + c.num_heads * c.arena_slots * 8].view(torch.float32).view(c.num_heads, c.arena_slots, 2).cpu()
    kv = ws[off_kv:off_kv + c.num_heads * c.arena_slots * 512].view(torch.bfloat16).view(c.num_heads, c.arena_slots, 256).cpu()
    for r in range(wl.R):
        for t in range(wl.D):
            base = ctx.onela_get_step_base(r, t)
            tk = case["tok"][(r, 0, t)]
            for h in range(wl.H):
                assert torch.equal(kv[h, base:base + wl.W, :128], tk["k"][:, h])
                assert torch.equal(kv[h, base:base + wl.W, 128:], tk["v"][:, h])
                assert torch.equal(gates[h, base:base + wl.W, 0], tk["alpha"][:, h])
                assert torch.equal(gates[h, base:base + wl.W, 1], tk["beta"][:, h])


def test_out_of_range_parent_is_reported_not_trapped():
    wl = CFG1.scaled(H=2, W=16, D=2, prompt_len=32)
    case = make_case(wl)
    bad = case["parents"][(0, 1)].clone()
    bad[3] = 16          # one past the previous beam
    case["parents"][(0, 1)] = bad
    outs, slots, ctx = run_library(case, out_dtype="fp32")
    code, detail = ctx.onela_poll_device_status()
    assert code == binding.E_DEVICE_CHECK and detail == 16
    assert ctx.onela_poll_device_status() == (0, 0)          # reading clears the sticky word
    assert slots[(0, 1)][3, 0] == 0                          # the offending index was clamped to parent 0
    assert torch.isfinite(outs[(0, 0, 1)]).all()


def test_prefill_kernel_matches_oracle_prefill():
    for wl in (CFG0, CFG1.scaled(H=4, prompt_len=300)):
        cfg = P.make_config(1, 1, wl.H, wl.dk, wl.dv, 8, 2, wl.dtype, "fp32", 16)
        ctx = P.Onela(cfg)
        p = inputs.prompt_tokens(wl, 0, 0)
        ctx.onela_prefill_shared_state(0, 0, *(p[n].cuda() for n in ("k", "v", "alpha", "beta")))
        got = ctx.onela_export_shared_state(0, 0).cpu().double().numpy()
        want = oracle.prefill(p["k"], p["v"], p["alpha"], p["beta"])
        err = np.linalg.norm(got - want, axis=(1, 2)) / np.linalg.norm(want, axis=(1, 2))
        assert err.max() < 1e-5, err      # fp32 recurrence against the fp64 one


def test_two_contexts_interleaved_on_one_stream():
    """Two contexts of different shapes take turns on the same stream: per-launch set-up that depends on the shape
    (group partition, head counts) must follow the call, not the previous context's."""
    wa = CFG1.scaled(R=2, H=4, W=130, D=3, prompt_len=32, parents="zipf", zipf_s=1.3, seed=931)
    wb = CFG1.scaled(R=1, H=7, W=49, D=3, prompt_len=32, seed=932)
    cases = [make_case(wa), make_case(wb)]
    refs = [run_oracle(c)[0] for c in cases]
    dev = torch.device("cuda")
    ctxs = []
    for wl, case in zip((wa, wb), cases):
        cfg = P.make_config(wl.R, 1, wl.H, wl.dk, wl.dv, wl.W, wl.D, wl.dtype, "fp32", wl.R * wl.W * wl.D, 0)
        ctx = P.Onela(cfg, device="cuda")
        for r in range(wl.R):
            ctx.onela_init_shared_state(r, 0, case["S0"][(r, 0)].to(dev))
        ctxs.append(ctx)
    for t in range(3):
        outs = []
        for wl, case, ctx in zip((wa, wb), cases, ctxs):       # a, b, a, b, ... with no synchronisation in between
            par = None if t == 0 else torch.stack([case["parents"][(r, t)] for r in range(wl.R)]).to(dev)
            ctx.onela_reorder_beams(0, wl.R, par, wl.W)
            tk = {n: torch.stack([case["tok"][(r, 0, t)][n] for r in range(wl.R)]).to(dev) for n in ("k", "v", "alpha", "beta")}
            q = torch.stack([case["q"][(r, 0, t)] for r in range(wl.R)]).to(dev)
            out = torch.empty((wl.R, wl.W, wl.H, wl.dv), dtype=torch.float32, device=dev)
            ctx.onela_append_decode_step(0, wl.R, 0, tk["k"], tk["v"], tk["alpha"], tk["beta"], q, out)
            outs.append(out)
        for wl, ref, out in zip((wa, wb), refs, outs):
            for r in range(wl.R):
                assert rel_l2(out[r].cpu().numpy(), ref[(r, 0, t)]).max() <= REL_L2_BAR
    assert all(c.onela_poll_device_status() == (0, 0) for c in ctxs)


def test_empty_prompt_gives_the_zero_state():
    """A prompt of no tokens: the prefill call stores S_0 = 0 and the decode outputs come from the records alone."""
    wl = CFG1.scaled(H=2, W=24, D=2, prompt_len=0, seed=88)
    cfg = P.make_config(1, 1, wl.H, wl.dk, wl.dv, wl.W, wl.D, wl.dtype, "fp32", wl.W * wl.D, 0)
    ctx = P.Onela(cfg, device="cuda")
    empty = lambda *shape: torch.empty(shape, device="cuda")
    ctx.onela_prefill_shared_state(0, 0, empty(0, wl.H, wl.dk).to(wl.torch_dtype), empty(0, wl.H, wl.dv).to(wl.torch_dtype),
                                   empty(0, wl.H), empty(0, wl.H))
    assert torch.count_nonzero(ctx.onela_export_shared_state(0, 0)) == 0
    S0 = np.zeros((wl.H, wl.dv, wl.dk), np.float32)
    steps, pars = [], []
    for t in range(wl.D):
        par = None if t == 0 else inputs.parents(wl, 0, t)
        tk = inputs.decode_token(wl, 0, 0, t)
        q = inputs.decode_query(wl, 0, 0, t)
        steps.append(tk); pars.append(par)
        ctx.onela_reorder_beams(0, 1, None if par is None else par[None].cuda(), wl.W)
        out = torch.empty((1, wl.W, wl.H, wl.dv), dtype=torch.float32, device="cuda")
        ctx.onela_append_decode_step(0, 1, 0, *(tk[n][None].cuda() for n in ("k", "v", "alpha", "beta")), q[None].cuda(), out)
        ref = oracle.decode(S0, steps, pars, q)
        assert rel_l2(out[0].cpu().numpy(), ref).max() <= REL_L2_BAR


def test_init_then_export_round_trip():
    wl = CFG1.scaled(H=2)
    ctx = P.Onela(P.make_config(1, 1, 2, 128, 128, 8, 2, "bf16", "fp32", 16))
    S = torch.randn(2, 128, 128, generator=torch.Generator().manual_seed(1))
    ctx.onela_init_shared_state(0, 0, S.cuda())
    back = ctx.onela_export_shared_state(0, 0).cpu()
    assert torch.equal(back, S)      # the store keeps S_0 bit for bit, on every path


def test_batched_state_store_equals_the_single_calls():
    """All layers of a range of requests in one call: the same bytes in the store as the per-(request, layer) calls,
    other requests untouched."""
    R, L, H = 3, 2, 2
    cfg = P.make_config(R, L, H, 128, 128, 8, 2, "bf16", "fp32", 64)
    ctx = P.Onela(cfg)
    S = torch.randn(R, L, H, 128, 128, generator=torch.Generator().manual_seed(7))
    ctx.onela_init_shared_state(0, 0, (S[0, 0] + 1).cuda())
    ctx.onela_init_shared_state(0, 1, (S[0, 1] + 1).cuda())
    ctx.onela_init_shared_states(1, 2, S[1:3].cuda())
    for r in (1, 2):
        for l in range(L):
            assert torch.equal(ctx.onela_export_shared_state(r, l).cpu(), S[r, l])
    assert torch.equal(ctx.onela_export_shared_state(0, 1).cpu(), S[0, 1] + 1)
    assert ctx.onela_poll_device_status() == (0, 0)


@pytest.mark.parametrize("dk,dv,dtype", [(128, 128, "bf16"), (256, 256, "fp32")])
@pytest.mark.parametrize("s0_unit,q_unit", [(1e-6, 1.0), (3e4, 1.0), (1.0, 1e-5), (1.0, 2e3), (1e-5, 1e-4), (1e4, 50.0)])
def test_tensor_core_operands_keep_their_precision_at_any_scale(s0_unit, q_unit, dk, dv, dtype):
    """The tensor-core kernel feeds fp16 operands; per-head and per-beam powers of two keep them inside the format's
    range, so states and queries far from unit scale decode as accurately as unit-scale ones (states of 1e-6 or
    queries of 1e-5 would otherwise sink into fp16's subnormals, states of 3e4 x 128 terms overflow it)."""
    wl = CFG1.scaled(H=2, dk=dk, dv=dv, dtype=dtype, W=70, D=3, prompt_len=48, parents="zipf", zipf_s=1.5, seed=4242)
    case = make_case(wl)
    for key in case["S0"]:
        case["S0"][key] = (case["S0"][key].double() * s0_unit).float()
    for key in case["q"]:
        case["q"][key] = (case["q"][key].double() * q_unit).to(case["q"][key].dtype)
    for fused in (True, False):
        outs, _, ctx = run_library(case, out_dtype="fp32", fused=fused)
        assert ctx.onela_uses_tensor_core_path()
        assert ctx.onela_poll_device_status() == (0, 0)
        ref, _ = run_oracle(case)
        for key, o in outs.items():
            assert rel_l2(o.numpy(), ref[key]).max() <= REL_L2_BAR


@pytest.mark.parametrize("key_norm,beta_lo,beta_hi", [(2.5, 0.5, 1.0), (1.0, 1.0, 2.0), (3.0, 0.6, 0.9)])
def test_keys_and_gates_outside_the_stable_range_on_the_tiled_kernel(key_norm, beta_lo, beta_hi):
    """The same inputs through the tiled tensor-core kernel (its operand rows are scaled by their exact largest element)."""
    wl = CFG1.scaled(H=2, dk=64, dv=64, dtype="fp32", W=100, D=8, prompt_len=32, parents="zipf", zipf_s=1.5, seed=607)
    case = make_case(wl)
    g = torch.Generator().manual_seed(8)
    for key, tok in case["tok"].items():
        tok["k"] = (tok["k"].double() * key_norm).to(tok["k"].dtype)
        tok["beta"] = (beta_lo + (beta_hi - beta_lo) * torch.rand(tok["beta"].shape, generator=g)).float()
    ref, _ = run_oracle(case)
    outs, _, ctx = run_library(case, out_dtype="fp32", fused=True)
    assert ctx.onela_uses_tensor_core_path() == 2 and ctx.onela_poll_device_status() == (0, 0)
    for key, o in outs.items():
        assert np.isfinite(o.numpy()).all()
        assert rel_l2(o.numpy(), ref[key]).max() <= REL_L2_BAR, key


@pytest.mark.parametrize("key_norm,beta_lo,beta_hi", [(2.5, 0.5, 1.0), (1.0, 1.0, 2.0), (3.0, 0.6, 0.9)])
@pytest.mark.parametrize("flags", [0, P.FLAG_SHARED_CHAINS, P.FLAG_FORCE_GENERIC])
def test_keys_and_gates_outside_the_stable_range(key_norm, beta_lo, beta_hi, flags):
    """Eq. 1 puts no bound on k or beta.  With |k| = 2-3 or beta in (1, 2) a fold step lengthens the folded query
    (by up to |1 - beta |k|^2| per level), so after eight levels it is orders of magnitude longer than q.  The fp16
    operand rows of the tensor-core kernels take their power-of-two scale from the folded row itself, so these
    inputs decode at the same bar as normalised ones - on every kernel."""
    wl = CFG1.scaled(H=2, W=100, D=8, prompt_len=32, parents="zipf", zipf_s=1.5, seed=606)
    case = make_case(wl)
    g = torch.Generator().manual_seed(7)
    for key, tok in case["tok"].items():
        tok["k"] = (tok["k"].double() * key_norm).to(tok["k"].dtype)
        tok["beta"] = (beta_lo + (beta_hi - beta_lo) * torch.rand(tok["beta"].shape, generator=g)).float()
    ref, _ = run_oracle(case)
    for fused in (True, False):
        outs, _, ctx = run_library(case, out_dtype="fp32", flags=flags, fused=fused)
        assert ctx.onela_poll_device_status() == (0, 0)
        for key, o in outs.items():
            assert np.isfinite(o.numpy()).all()
            assert rel_l2(o.numpy(), ref[key]).max() <= REL_L2_BAR, key
