"""Device-side global beam selection (onela_select_beams) against the selection oracle: bit-exact parents, codes
and scores (the order is unique: best first, ties to the smaller flat index), and a whole generation whose parent
maps never leave the device - select -> reorder -> fused append + decode per layer, captured in one CUDA graph per
step - against the full-state oracle driven by the oracle's own selections."""
import numpy as np
import pytest
import torch

import oracle
from oracle import select as osel
import paper_2609_12399_b200 as P
from paper_2609_12399_b200 import inputs

from _cases import REL_L2_BAR, rel_l2

pytestmark = pytest.mark.gpu

CFG1 = inputs.WORKLOADS[1]


def _ctx(R, W, steps=2, H=2):
    cfg = P.make_config(R, 1, H, 128, 128, W, steps, "bf16", "bf16", R * W * steps, 0)
    ctx = P.Onela(cfg, device="cuda")
    for r in range(R):
        ctx.onela_init_shared_state(r, 0, torch.zeros(H, 128, 128, device="cuda"))
    return ctx


def _logp(gen, shape, quant=None):
    x = torch.randn(shape, generator=gen)
    x = torch.log_softmax(x, dim=-1)
    if quant:                                   # coarse values: many exact ties
        x = torch.round(x * quant) / quant
    return x.float()


def _compare(ctx, R, W_prev, C, W_new, bs, lp):
    par = torch.empty((R, W_new), dtype=torch.int32, device="cuda")
    code = torch.empty_like(par)
    sc = torch.empty((R, W_new), dtype=torch.float32, device="cuda")
    ctx.onela_select_beams(0, R, bs.cuda(), lp.cuda(), C, W_new, par, code, sc)
    torch.cuda.synchronize()
    for r in range(R):
        p, c, s = osel.select_beams(bs[r].numpy(), lp[r].numpy(), W_new)
        assert np.array_equal(par[r].cpu().numpy(), p), f"parents of request {r}"
        assert np.array_equal(code[r].cpu().numpy(), c), f"codes of request {r}"
        assert np.array_equal(sc[r].cpu().numpy().view(np.uint32), s.view(np.uint32)), f"scores of request {r}"


@pytest.mark.parametrize("W_prev,C,W_new,quant", [(512, 256, 512, None), (512, 256, 512, 4), (37, 50, 64, 2),
                                                  (1024, 256, 1024, None), (8, 8, 64, None), (5, 3, 1, None)])
def test_select_matches_oracle_bit_for_bit(W_prev, C, W_new, quant):
    R = 3
    gen = torch.Generator().manual_seed(1000 + W_prev + C)
    ctx = _ctx(R, max(W_prev, W_new))
    ctx.onela_reorder_beams(0, R, None, W_prev)     # opens call 1 with W_prev beams, so selection sees W_prev parents
    bs = _logp(gen, (R, W_prev), quant)
    lp = _logp(gen, (R, W_prev, C), quant)
    _compare(ctx, R, W_prev, C, W_new, bs, lp)


def test_select_from_the_root_and_special_values():
    R, C = 2, 300
    ctx = _ctx(R, 64)
    gen = torch.Generator().manual_seed(5)
    lp = _logp(gen, (R, 1, C))
    lp[0, 0, 7] = float("nan"); lp[0, 0, 9] = float("inf"); lp[0, 0, 11] = float("-inf")
    lp[1, 0, :40] = -0.0; lp[1, 0, 40:80] = 0.0
    _compare(ctx, R, 1, C, 64, torch.zeros(R, 1), lp)


def test_generation_driven_by_device_side_selection_in_cuda_graphs():
    wl = CFG1.scaled(R=2, L=2, H=4, W=48, D=3, prompt_len=64, seed=321)
    R, L, H, W, C = wl.R, wl.L, wl.H, wl.W, 64
    cfg = P.make_config(R, L, H, wl.dk, wl.dv, W, wl.D, "bf16", "fp32", R * W * wl.D, 0)
    ctx = P.Onela(cfg, device="cuda")
    S0 = {}
    for r in range(R):
        for l in range(L):
            p = inputs.prompt_tokens(wl, r, l)
            S0[(r, l)] = torch.from_numpy(oracle.prefill(p["k"], p["v"], p["alpha"], p["beta"]).astype(np.float32))
            ctx.onela_init_shared_state(r, l, S0[(r, l)].cuda())
    gen = torch.Generator().manual_seed(99)
    # device buffers reused by every step's graph
    d_bs = torch.zeros((R, W), dtype=torch.float32, device="cuda")
    d_par = torch.empty((R, W), dtype=torch.int32, device="cuda")
    d_code = torch.empty_like(d_par)
    d_sc = torch.empty((R, W), dtype=torch.float32, device="cuda")
    outs = [torch.empty((R, W, H, wl.dv), dtype=torch.float32, device="cuda") for _ in range(L)]
    h_bs = np.zeros((R, 1), np.float32)                      # oracle side: cumulative scores of the current beams
    tok_hist = {(r, l): [] for r in range(R) for l in range(L)}
    par_hist = {r: [None] for r in range(R)}
    side = torch.cuda.Stream()
    for t in range(wl.D):
        W_prev = 1 if t == 0 else W
        lp = _logp(gen, (R, W_prev, C), quant=8)
        d_lp = lp.cuda()
        toks = [{n: torch.stack([inputs.decode_token(wl, r, l, t)[n] for r in range(R)]).cuda() for n in ("k", "v", "alpha", "beta")}
                for l in range(L)]
        qs = [torch.stack([inputs.decode_query(wl, r, l, t) for r in range(R)]).cuda() for l in range(L)]
        bs_in = d_bs[:, :W_prev].contiguous()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                ctx.onela_select_beams(0, R, bs_in, d_lp, C, W, d_par, d_code, d_sc)
                ctx.onela_reorder_beams(0, R, None if t == 0 else d_par, W)
                for l in range(L):
                    ctx.onela_append_decode_step(0, R, l, toks[l]["k"], toks[l]["v"], toks[l]["alpha"], toks[l]["beta"], qs[l], outs[l])
        g.replay()
        torch.cuda.synchronize()
        assert ctx.onela_poll_device_status() == (0, 0)
        # oracle: its own selection, then the full-state replay along its own parent maps
        next_bs = np.zeros((R, W), np.float32)
        for r in range(R):
            p, c, sc = osel.select_beams(h_bs[r], lp[r].numpy(), W)
            assert np.array_equal(d_par[r].cpu().numpy(), p) and np.array_equal(d_code[r].cpu().numpy(), c)
            next_bs[r] = sc
            if t > 0:
                par_hist[r].append(p)
            for l in range(L):
                tok_hist[(r, l)].append({n: toks[l][n][r].cpu() for n in toks[l]})
                ref = oracle.decode(S0[(r, l)], tok_hist[(r, l)], par_hist[r], qs[l][r].cpu())
                assert rel_l2(outs[l][r].cpu().numpy(), ref).max() <= REL_L2_BAR, (t, r, l)
        h_bs = next_bs
        d_bs.copy_(d_sc)                                         # the survivors' scores are the next step's beam scores
