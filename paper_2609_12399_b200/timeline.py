"""Clock-stamped timeline of one CTA of the tensor-core decode kernels.

    python -m paper_2609_12399_b200.timeline [--kernel ws|wy] [--workload cfg2|cfg4] [--depth D] [--cta C]

Builds a debug copy of the library (`-DONELA_WS_TL -DONELA_WY_TL`: the kernels keep clock64 stamps of CTA 0's role
milestones in shared memory and write them out when the CTA ends; the product library has no such code), runs the
workload cut to ONE layer (seeded inputs, a random S_0) through the C ABI with the fused append + decode call, and prints
the stamps of the launch at the given chain depth in microseconds at 1.9 GHz, one warp per role:
  ws (decode_ws_kernel):  fold warp 0, the epilogue warp that issues the MMAs, one storing epilogue warp;
  wy (decode_wy_kernel, ONELA_FLAG_SHARED_CHAINS): fold warp 0, epilogue warp 0, solver warp 0, the issuing solver warp.
"""
from __future__ import annotations

import argparse
import ctypes

import torch

from . import binding, build, inputs

WY_NAMES = {1: "fold.start", 2: "fold.math", 3: "fold.buffers", 4: "fold.full", 10: "setup.start", 11: "setup.staged", 12: "setup.mma",
            13: "setup.U", 14: "setup.done", 15: "setup.copies_out", 16: "setup.nodes", 17: "setup.index", 18: "setup.s0", 19: "setup.landed",
            50: "setup.vmax", 51: "setup.pmax", 52: "setup.usync", 20: "epi.wait", 21: "epi.acc", 22: "epi.T", 23: "epi.done",
            30: "sol.wait", 31: "sol.g", 32: "sol.extracted", 33: "sol.solved", 34: "sol.issued", 35: "sol.loaded", 36: "sol.fma",
            37: "sol.stored", 38: "sol.bar", 40: "iss.wait", 41: "iss.full", 42: "iss.out"}
WS_NAMES = {1: "cta.ready", 2: "deps.waited", 3: "s0.in_tmem", 10: "quad.start", 11: "heads.landed", 12: "folded", 13: "slot.free",
            14: "rows.written", 20: "issue.wait", 21: "issue.rows_seen", 22: "issue.out", 30: "epi.wait", 31: "epi.acc", 32: "epi.transposed",
            33: "epi.stored", 40: "role.done"}


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--kernel", default="ws", choices=["ws", "wy"])
    ap.add_argument("--workload", default="cfg4", choices=["cfg2", "cfg4"])
    ap.add_argument("--depth", type=int, default=0, help="chain depth of the launch to show (default: the deepest)")
    ap.add_argument("--cta", type=int, default=0, help="ws: the CTA whose roles are stamped (default 0)")
    ap.add_argument("--layers", type=int, default=1,
                    help="launch the call over this many layers back to back and show the LAST launch (its start then "
                         "overlaps its predecessor's tail, as in a decoder's layer loop)")
    args = ap.parse_args()
    binding.LIB_PATH = build.build_timeline()
    lib = binding.load_library()
    fn = lib.onela_debug_wy_timeline if args.kernel == "wy" else lib.onela_debug_ws_timeline
    fn.restype = ctypes.c_int
    fn.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
    if args.kernel == "ws" and args.cta:
        lib.onela_debug_ws_timeline_cta(ctypes.c_int(args.cta))
    roles = ("fold", "epi", "sol", "iss") if args.kernel == "wy" else ("fold", "issue", "store")
    names = WY_NAMES if args.kernel == "wy" else WS_NAMES
    from .binding import FLAG_SHARED_CHAINS, Onela, make_config

    wl = inputs.WORKLOADS[int(args.workload[3])].scaled(L=max(1, args.layers), prompt_len=64)
    depth_show = args.depth or wl.D
    dev = torch.device("cuda")
    cfg = make_config(wl.R, wl.L, wl.H, wl.dk, wl.dv, wl.W, wl.D, wl.dtype, "bf16", wl.R * wl.W * wl.D,
                      FLAG_SHARED_CHAINS if args.kernel == "wy" else 0)
    ctx = Onela(cfg, device="cuda")
    S0 = torch.randn(wl.R * wl.H, wl.dv, wl.dk, device=dev, generator=torch.Generator(device=dev).manual_seed(1)) * 0.1
    for r in range(wl.R):
        for l in range(wl.L):
            ctx.onela_init_shared_state(r, l, S0[r * wl.H:(r + 1) * wl.H].contiguous())
    buf = (ctypes.c_ulonglong * 800)()
    cnt = (ctypes.c_int * 4)()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    for t in range(wl.D):
        par = None if t == 0 else torch.stack([inputs.parents(wl, r, t, W_prev=wl.W, W_new=wl.W) for r in range(wl.R)]).to(dev)
        ctx.onela_reorder_beams(0, wl.R, par, wl.W)
        beams = torch.arange(wl.W)
        tk = {nm: torch.stack([inputs.decode_token(wl, r, 0, t, beams=beams, device=dev)[nm] for r in range(wl.R)])
              for nm in ("k", "v", "alpha", "beta")}
        q = torch.stack([inputs.decode_query(wl, r, 0, t, beams=beams, device=dev) for r in range(wl.R)])
        outs = [torch.empty((wl.R, wl.W, wl.H, wl.dv), dtype=torch.bfloat16, device=dev) for _ in range(wl.L)]
        flush.zero_()                                   # cold L2, as in the benchmark's timing of these workloads
        torch.cuda.synchronize()
        fn(buf, cnt)                                    # clears the stamps of earlier launches
        if wl.L > 1:
            torch.cuda._sleep(int(2.0e6))               # the layers' launches queue up behind a short spin
        for l in range(wl.L):                           # (every layer gets the same seeded token: timing only)
            ctx.onela_append_decode_step(0, wl.R, l, tk["k"], tk["v"], tk["alpha"], tk["beta"], q, outs[l])
        torch.cuda.synchronize()
        cap = fn(buf, cnt)
        if t + 1 != depth_show:
            continue
        ev = []
        for role in range(len(roles)):
            for i in range(cnt[role]):
                x = buf[role * cap + i]
                ev.append((x >> 56, roles[role], (x >> 48) & 0xff, x & 0xffffffffffff))
        if not ev:
            print("no stamps (this launch ran the other kernel)")
            continue
        t0 = min(e[3] for e in ev)
        ev.sort(key=lambda e: e[3])
        print(args.kernel, args.workload, "depth", t + 1, "events", len(ev), "(cycles / 1.9 GHz)")
        for e in ev:
            print("%8.2f us  %-5s  %-16s g=%d" % ((e[3] - t0) / 1900.0, e[1], names.get(e[0], str(e[0])), e[2]))
    assert ctx.onela_poll_device_status() == (0, 0)


if __name__ == "__main__":
    main()
