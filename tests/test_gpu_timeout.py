"""The bounded waits of the tensor-core decode kernels, exercised without a fault: a second build of the library
(same sources, a short wait limit, one test hook) makes ONE fold-warp arrival of CTA 0 go missing, so the wait for
that group's operand rows runs out.  The kernel must return, the sticky status word must say ONELA_E_TIMEOUT with
the CTA's index, and the same context must decode correctly afterwards.  Runs in a child process so that the
product library and the test-hooks library never share a process."""
import subprocess
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


def _child():
    import ctypes

    import numpy as np
    import torch

    sys.path.insert(0, str(ROOT))
    sys.path.insert(0, str(ROOT / "tests"))
    import paper_2609_12399_b200 as P
    from paper_2609_12399_b200 import binding, build, inputs

    binding.LIB_PATH = build.build_testhooks()
    lib = binding.load_library()
    lib.onela_testhook_drop_full_arrival.restype = ctypes.c_int
    lib.onela_testhook_drop_full_arrival.argtypes = [ctypes.c_int]
    from _cases import REL_L2_BAR, make_case, rel_l2, run_oracle

    wl = inputs.WORKLOADS[1].scaled(H=2, W=200, D=2, prompt_len=32, seed=31)     # 5 groups per (request, head)
    case = make_case(wl)
    ref, _ = run_oracle(case)
    dev = torch.device("cuda")
    cfg = P.make_config(wl.R, wl.L, wl.H, wl.dk, wl.dv, wl.W, wl.D, wl.dtype, "fp32", wl.R * wl.W * wl.D, 0)
    ctx = P.Onela(cfg, device="cuda")
    assert ctx.onela_uses_tensor_core_path()
    ctx.onela_init_shared_state(0, 0, case["S0"][(0, 0)].to(dev))
    out = torch.empty((1, wl.W, wl.H, wl.dv), dtype=torch.float32, device=dev)
    for t in range(wl.D):
        par = None if t == 0 else case["parents"][(0, t)][None].to(dev)
        ctx.onela_reorder_beams(0, 1, par, wl.W)
        tk = {n: case["tok"][(0, 0, t)][n][None].to(dev) for n in ("k", "v", "alpha", "beta")}
        q = case["q"][(0, 0, t)][None].to(dev)
        ctx.onela_append_records(0, 1, 0, tk["k"], tk["v"], tk["alpha"], tk["beta"])
        if t == wl.D - 1:
            # the arrival goes missing: the call returns, the status word reports the expired wait of CTA 0
            assert lib.onela_testhook_drop_full_arrival(1) == 0
            ctx.onela_decode_step(0, 1, 0, q, out)
            torch.cuda.synchronize()
            code, detail = ctx.onela_poll_device_status()
            assert (code, detail) == (binding.E_TIMEOUT, 0), (code, detail)
            assert lib.onela_testhook_drop_full_arrival(0) == 0
            assert ctx.onela_poll_device_status() == (0, 0)          # polling cleared the word
        # the same context decodes the call correctly (a decode may be repeated any number of times)
        ctx.onela_decode_step(0, 1, 0, q, out)
        torch.cuda.synchronize()
        assert ctx.onela_poll_device_status() == (0, 0)
        e = rel_l2(out[0].cpu().numpy(), ref[(0, 0, t)])
        assert e.max() <= REL_L2_BAR, (t, float(e.max()))
    print("timeout reported and recovered")


def _child_tiled():
    """The tiled kernel's one wait (for a tile's MMAs): CTA (0, 0, 0) leaves its first tile's MMAs and their commit
    out, so the wait runs out; every thread of the CTA agrees on that before going on, the CTA frees its tensor
    memory and returns."""
    import ctypes

    import torch

    sys.path.insert(0, str(ROOT))
    sys.path.insert(0, str(ROOT / "tests"))
    import paper_2609_12399_b200 as P
    from paper_2609_12399_b200 import binding, build, inputs

    binding.LIB_PATH = build.build_testhooks()
    lib = binding.load_library()
    lib.onela_testhook_tiled_skip_issue.restype = ctypes.c_int
    lib.onela_testhook_tiled_skip_issue.argtypes = [ctypes.c_int]
    from _cases import REL_L2_BAR, make_case, rel_l2, run_oracle

    wl = inputs.WORKLOADS[1].scaled(H=2, dk=256, dv=256, W=100, D=2, prompt_len=32, seed=32)     # two tiles of value rows
    case = make_case(wl)
    ref, _ = run_oracle(case)
    dev = torch.device("cuda")
    cfg = P.make_config(wl.R, wl.L, wl.H, wl.dk, wl.dv, wl.W, wl.D, wl.dtype, "fp32", wl.R * wl.W * wl.D, 0)
    ctx = P.Onela(cfg, device="cuda")
    assert ctx.onela_uses_tensor_core_path() == 2
    ctx.onela_init_shared_state(0, 0, case["S0"][(0, 0)].to(dev))
    out = torch.empty((1, wl.W, wl.H, wl.dv), dtype=torch.float32, device=dev)
    for t in range(wl.D):
        par = None if t == 0 else case["parents"][(0, t)][None].to(dev)
        ctx.onela_reorder_beams(0, 1, par, wl.W)
        tk = {n: case["tok"][(0, 0, t)][n][None].to(dev) for n in ("k", "v", "alpha", "beta")}
        q = case["q"][(0, 0, t)][None].to(dev)
        ctx.onela_append_records(0, 1, 0, tk["k"], tk["v"], tk["alpha"], tk["beta"])
        if t == wl.D - 1:
            assert lib.onela_testhook_tiled_skip_issue(1) == 0
            ctx.onela_decode_step(0, 1, 0, q, out)
            torch.cuda.synchronize()
            code, detail = ctx.onela_poll_device_status()
            assert (code, detail) == (binding.E_TIMEOUT, 0), (code, detail)
            assert lib.onela_testhook_tiled_skip_issue(0) == 0
            assert ctx.onela_poll_device_status() == (0, 0)
        ctx.onela_decode_step(0, 1, 0, q, out)
        torch.cuda.synchronize()
        assert ctx.onela_poll_device_status() == (0, 0)
        e = rel_l2(out[0].cpu().numpy(), ref[(0, 0, t)])
        assert e.max() <= REL_L2_BAR, (t, float(e.max()))
    print("timeout reported and recovered")


@pytest.mark.gpu
@pytest.mark.parametrize("which", ["child", "child_tiled"])
def test_expired_wait_is_reported_and_the_context_stays_usable(which):
    r = subprocess.run([sys.executable, __file__, which], capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stdout + r.stderr
    assert "timeout reported and recovered" in r.stdout


if __name__ == "__main__" and sys.argv[1:] == ["child"]:
    _child()
if __name__ == "__main__" and sys.argv[1:] == ["child_tiled"]:
    _child_tiled()
