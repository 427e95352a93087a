"""Clock-stamped timeline of one CTA of the shared-chains decode kernel (ONELA_FLAG_SHARED_CHAINS).

    python -m paper_2609_12399_b200.wy_timeline [depth]

Builds a debug copy of the library (`-DONELA_WY_TL`: the kernel keeps clock64 stamps of CTA 0's role milestones in
shared memory and writes them out when it ends; the product library has no such code), runs the beam-512 decode stack
cut to ONE layer (4 requests x 32 heads x 512 beams, Zipf(1.5) parents, seeded inputs, a random S_0) through the C ABI
and prints the stamps of the launch at the given chain depth (default 8), in microseconds at 1.9 GHz.  One warp per
role is stamped: fold warp 0, epilogue warp 0, solver warp 0, and the solver warp that issues the first MMA set.
"""
from __future__ import annotations

import ctypes
import sys

import torch

from . import binding, build, inputs

NAMES = {1: "fold.start", 2: "fold.math", 3: "fold.buffers", 4: "fold.full", 10: "setup.start", 11: "setup.staged", 12: "setup.mma",
         13: "setup.U", 14: "setup.done", 15: "setup.copies_out", 16: "setup.nodes", 17: "setup.index", 18: "setup.s0", 19: "setup.landed",
         50: "setup.vmax", 51: "setup.pmax", 52: "setup.usync", 20: "epi.wait", 21: "epi.acc", 22: "epi.T", 23: "epi.done",
         30: "sol.wait", 31: "sol.g", 32: "sol.extracted", 33: "sol.solved", 34: "sol.issued", 35: "sol.loaded", 36: "sol.fma",
         37: "sol.stored", 38: "sol.bar", 40: "iss.wait", 41: "iss.full", 42: "iss.out"}


def main(depth_show: int = 8) -> None:
    binding.LIB_PATH = build.build_timeline()
    lib = binding.load_library()
    lib.onela_debug_wy_timeline.restype = ctypes.c_int
    lib.onela_debug_wy_timeline.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
    from .binding import FLAG_SHARED_CHAINS, Onela, make_config

    wl = inputs.WORKLOADS[4].scaled(L=1, prompt_len=64)
    dev = torch.device("cuda")
    cfg = make_config(wl.R, wl.L, wl.H, wl.dk, wl.dv, wl.W, wl.D, wl.dtype, "bf16", wl.R * wl.W * wl.D, FLAG_SHARED_CHAINS)
    ctx = Onela(cfg, device="cuda")
    S0 = torch.randn(wl.R * wl.H, wl.dv, wl.dk, device=dev, generator=torch.Generator(device=dev).manual_seed(1)) * 0.1
    for r in range(wl.R):
        ctx.onela_init_shared_state(r, 0, S0[r * wl.H:(r + 1) * wl.H].contiguous())
    buf = (ctypes.c_ulonglong * 800)()
    cnt = (ctypes.c_int * 4)()
    for t in range(wl.D):
        par = None if t == 0 else torch.stack([inputs.parents(wl, r, t, W_prev=wl.W, W_new=wl.W) for r in range(wl.R)]).to(dev)
        ctx.onela_reorder_beams(0, wl.R, par, wl.W)
        beams = torch.arange(wl.W)
        tk = {nm: torch.stack([inputs.decode_token(wl, r, 0, t, beams=beams, device=dev)[nm] for r in range(wl.R)])
              for nm in ("k", "v", "alpha", "beta")}
        q = torch.stack([inputs.decode_query(wl, r, 0, t, beams=beams, device=dev) for r in range(wl.R)])
        out = torch.empty((wl.R, wl.W, wl.H, wl.dv), dtype=torch.bfloat16, device=dev)
        torch.cuda.synchronize()
        lib.onela_debug_wy_timeline(buf, cnt)          # clears the stamps of earlier launches
        ctx.onela_append_decode_step(0, wl.R, 0, tk["k"], tk["v"], tk["alpha"], tk["beta"], q, out)
        torch.cuda.synchronize()
        cap = lib.onela_debug_wy_timeline(buf, cnt)
        if t + 1 != depth_show:
            continue
        ev = []
        for role in range(4):
            for i in range(cnt[role]):
                x = buf[role * cap + i]
                ev.append((x >> 56, ("fold", "epi", "sol", "iss")[role], (x >> 48) & 0xff, x & 0xffffffffffff))
        if not ev:
            print("no stamps (depth 1 runs the other kernel)")
            continue
        t0 = min(e[3] for e in ev)
        ev.sort(key=lambda e: e[3])
        print("depth", t + 1, "events", len(ev), "(cycles / 1.9 GHz)")
        for e in ev:
            print("%8.2f us  %-4s  %-16s g=%d" % ((e[3] - t0) / 1900.0, e[1], NAMES.get(e[0], str(e[0])), e[2]))
    assert ctx.onela_poll_device_status() == (0, 0)


if __name__ == "__main__":
    main(int(sys.argv[1]) if len(sys.argv) > 1 else 8)
