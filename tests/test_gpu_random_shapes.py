"""Randomised shapes: the tensor-core kernel (ungrouped and grouped instantiations, fused and separate append) against
the CUDA-core kernels, which share no device code with it, on every unit of seeded random workloads - request
counts, head counts, value-head groups, beam widths that change from call to call (single beams, exactly full and
barely spilling 48-beam groups), depths to 9, uniform and Zipf parents.  A property that holds at any shape; the
oracle comparisons elsewhere anchor both kernels."""
import random

import numpy as np
import pytest
import torch

import paper_2609_12399_b200 as P
from paper_2609_12399_b200 import inputs

from _cases import REL_L2_BAR, rel_l2

pytestmark = pytest.mark.gpu

CFG1 = inputs.WORKLOADS[1]


def _generation(it, R, Hk, g, widths, fused, wl, flags, dk=128, dv=128, dtype="bf16"):
    Hv, D = Hk * g, len(widths)
    cfg = P.make_config(R, 1, Hk, dk, dv, max(widths), D, dtype, "fp32", R * sum(widths), flags, num_v_heads=Hv)
    ctx = P.Onela(cfg, device="cuda")
    gen = torch.Generator().manual_seed(it)
    td = torch.bfloat16 if dtype == "bf16" else torch.float32
    for r in range(R):
        ctx.onela_init_shared_state(r, 0, torch.randn((Hv, dv, dk), generator=gen).cuda())
    unit = lambda *shape: torch.nn.functional.normalize(torch.randn(shape, generator=gen), dim=-1).to(td).cuda()
    outs = []
    for t, W in enumerate(widths):
        par = None if t == 0 else torch.stack([inputs.parents(wl, r, t, W_prev=widths[t - 1], W_new=W) for r in range(R)]).cuda()
        ctx.onela_reorder_beams(0, R, par, W)
        k, q = unit(R, W, Hk, dk), unit(R, W, Hk, dk)
        v = torch.randn((R, W, Hv, dv), generator=gen).to(td).cuda()
        a = (torch.rand((R, W, Hv), generator=gen) * 0.1 + 0.9).cuda()
        b = torch.sigmoid(torch.randn((R, W, Hv), generator=gen)).cuda()
        out = torch.empty((R, W, Hv, dv), dtype=torch.float32, device="cuda")
        if fused:
            ctx.onela_append_decode_step(0, R, 0, k, v, a, b, q, out)
        else:
            ctx.onela_append_records(0, R, 0, k, v, a, b)
            ctx.onela_decode_step(0, R, 0, q, out)
        outs.append(out.cpu().numpy())
    assert ctx.onela_poll_device_status() == (0, 0)
    return outs, ctx.onela_uses_tensor_core_path()


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_tensor_core_and_cuda_core_kernels_agree_on_random_shapes(seed):
    rnd = random.Random(seed)
    for it in range(12):
        g = rnd.choice([1, 1, 2, 4])
        Hk = rnd.choice([1, 2, 3, 5, 8, 16])
        R = rnd.choice([1, 2, 3, 5, 8, 13])
        widths = [rnd.choice([1, 7, 16, 33, 47, 48, 49, 95, 96, 97, 130, 200, 301]) for _ in range(rnd.randint(1, 9))]
        fused = rnd.random() < 0.6
        wl = CFG1.scaled(R=R, L=1, H=Hk * g, W=max(widths), D=len(widths), prompt_len=0, parents=rnd.choice(["uniform", "zipf"]),
                         zipf_s=rnd.choice([1.1, 1.5, 2.5]), seed=1000 * seed + it)
        tc, used_tc = _generation(it, R, Hk, g, widths, fused, wl, 0)
        cc, used_cc = _generation(it, R, Hk, g, widths, fused, wl, P.FLAG_FORCE_GENERIC)
        assert used_tc and not used_cc
        for t, (x, y) in enumerate(zip(tc, cc)):
            e = rel_l2(x, y.astype(np.float64))
            assert e.max() <= REL_L2_BAR, f"case {it} (R={R}, Hk={Hk}, g={g}, widths={widths}, fused={fused}) call {t}: {e.max():.3e}"


@pytest.mark.parametrize("seed", [21, 22])
def test_tiled_tensor_core_and_cuda_core_kernels_agree_on_random_shapes(seed):
    """The same property for the tiled tcgen05 kernel: the other head shapes and record dtypes, grouped where the
    library takes groups, beam widths around its 32- and 64-beam tiles."""
    rnd = random.Random(seed)
    shapes = [(64, 64, "bf16"), (64, 64, "fp32"), (128, 128, "fp32"), (128, 256, "fp32"), (128, 512, "fp32"),
              (256, 256, "bf16"), (256, 256, "fp32"), (256, 512, "bf16")]
    for it in range(10):
        dk, dv, dtype = rnd.choice(shapes)
        g = rnd.choice([1, 2, 4]) if (dk, dv) in ((64, 64), (128, 128), (128, 256)) else 1
        Hk = rnd.choice([1, 2, 3, 5])
        R = rnd.choice([1, 2, 3, 5])
        widths = [rnd.choice([1, 7, 31, 32, 33, 63, 64, 65, 130, 200]) for _ in range(rnd.randint(1, 9))]
        fused = rnd.random() < 0.6
        wl = CFG1.scaled(R=R, L=1, H=Hk * g, W=max(widths), D=len(widths), prompt_len=0, parents=rnd.choice(["uniform", "zipf"]),
                         zipf_s=rnd.choice([1.1, 1.5, 2.5]), seed=1000 * seed + it)
        tc, used_tc = _generation(it, R, Hk, g, widths, fused, wl, 0, dk, dv, dtype)
        cc, used_cc = _generation(it, R, Hk, g, widths, fused, wl, P.FLAG_FORCE_GENERIC, dk, dv, dtype)
        assert used_tc == 2 and used_cc == 0
        for t, (x, y) in enumerate(zip(tc, cc)):
            e = rel_l2(x, y.astype(np.float64))
            assert e.max() <= REL_L2_BAR, f"case {it} ({dk}x{dv} {dtype}, R={R}, Hk={Hk}, g={g}, widths={widths}, fused={fused}) call {t}: {e.max():.3e}"
