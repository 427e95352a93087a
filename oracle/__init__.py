"""ORACLE - test infrastructure only.

Slow, plain fp64 CPU statements of what the beam-shared Gated DeltaNet decode
computes, written from the paper's equations.  Only ``tests/``, the smoke check
and the benchmark's CPU-baseline leg may import this package; the CUDA library
never does, and nothing here imports the CUDA library or its binding.

* :func:`decode`   - oracle A (C, ``gdn_fullstate.c``): materialise every unit's full state by
  replaying Eq. 1 from S_0 along its parent-pointer chain, then o = S q.
* :func:`prefill`  - Eq. 1 from the zero state over a prompt (how S_0 is defined).
* :mod:`oracle.evaluators` - independent numpy evaluators used as cross-checks: the paper's
  forward projection replay (Eq. 3-4) and the ancestry table recurrence (Eq. 5).

Pins (tests/test_oracle_pins.py): hand-worked examples, the alpha=1/beta=0 and
beta=1/unit-k invariants, one-hot closed forms, dense brute force over every
lineage of tiny beams, linearity, and agreement of the three evaluators.
"""
from __future__ import annotations

import ctypes
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "gdn_fullstate.c"
_LIB = _HERE / "liboracle_gdn.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile the C oracle with gcc (portable flags: the .so may run on another host)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        cmd = ["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC", "-o", str(_LIB), str(_SRC)]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(str(build()))
        pp_f = ctypes.POINTER(ctypes.c_void_p)
        lib.oracle_gdn_decode.restype = ctypes.c_int
        lib.oracle_gdn_decode.argtypes = [
            ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
            pp_f, pp_f, pp_f, pp_f, pp_f, ctypes.c_void_p,
            ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int]
        lib.oracle_gdn_prefill.restype = ctypes.c_int
        lib.oracle_gdn_prefill.argtypes = [ctypes.c_int] * 4 + [ctypes.c_void_p] * 5 + [ctypes.c_int]
        lib.oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def num_threads() -> int:
    """Threads the C oracle will use (OpenMP's default: the cores visible to the process)."""
    return int(_load().oracle_num_threads())


def _f32(x) -> np.ndarray:
    """fp32 C-contiguous numpy view of a numpy array or torch tensor (bf16/fp32 widen exactly)."""
    if hasattr(x, "detach"):
        x = x.detach().cpu().float().numpy()
    return np.ascontiguousarray(x, dtype=np.float32)


def _i32(x) -> np.ndarray:
    if hasattr(x, "detach"):
        x = x.detach().cpu().numpy()
    return np.ascontiguousarray(x, dtype=np.int32)


def _ptr_array(arrs):
    out = (ctypes.c_void_p * max(len(arrs), 1))()
    for i, a in enumerate(arrs):
        out[i] = None if a is None else a.ctypes.data
    return out


def decode(S0, steps, parents, q, sel=None, nthreads: int = 0, return_chains: bool = False):
    """Oracle A: full-state replay for one request and one layer.

    S0       [H, dv, dk]
    steps    list over decode calls t of dicts k [W_t, H, dk], v [W_t, H, dv], alpha, beta [W_t, H]
    parents  list over t; parents[0] is None (call 0 starts at S0), parents[t] int [W_t]
    q        [W_{T-1}, H, dk]  (with no steps: [n, H, dk], output S0 q)
    sel      None for every (beam, head), else (beams, heads) index arrays of equal length
    Returns  out fp64 [W, H, dv] (sel None) or [n_sel, dv]; with return_chains also the
             beam index of each unit at every call, oldest first, int32 [n_sel, T].
    """
    lib = _load()
    S0 = _f32(S0)
    H, dv, dk = S0.shape
    T = len(steps)
    ks = [_f32(s["k"]) for s in steps]
    vs = [_f32(s["v"]) for s in steps]
    als = [_f32(s["alpha"]) for s in steps]
    bes = [_f32(s["beta"]) for s in steps]
    q = _f32(q)
    W = np.array([k.shape[0] for k in ks] or [q.shape[0]], dtype=np.int32)
    for t in range(T):
        assert ks[t].shape == (W[t], H, dk) and vs[t].shape == (W[t], H, dv)
        assert als[t].shape == (W[t], H) and bes[t].shape == (W[t], H)
    assert q.shape == (W[-1], H, dk)
    ps = [None if (t == 0 or parents[t] is None) else _i32(parents[t]) for t in range(T)]
    for t in range(1, T):
        assert ps[t] is not None and ps[t].shape == (W[t],)
    if sel is None:
        bb, hh = np.meshgrid(np.arange(W[-1]), np.arange(H), indexing="ij")
        beams, heads = _i32(bb.reshape(-1)), _i32(hh.reshape(-1))
    else:
        beams, heads = _i32(sel[0]).reshape(-1), _i32(sel[1]).reshape(-1)
        assert beams.shape == heads.shape
    n = beams.shape[0]
    out = np.empty((n, dv), dtype=np.float64)
    chains = np.empty((n, max(T, 1)), dtype=np.int32)
    rc = lib.oracle_gdn_decode(H, dk, dv, T, W.ctypes.data, S0.ctypes.data,
                               _ptr_array(ks), _ptr_array(vs), _ptr_array(als), _ptr_array(bes),
                               _ptr_array(ps), q.ctypes.data, n, beams.ctypes.data, heads.ctypes.data,
                               out.ctypes.data, chains.ctypes.data, nthreads)
    if rc != 0:
        raise ValueError("parent index outside the previous beam")
    if sel is None:
        out = out.reshape(int(W[-1]), H, dv)
    if return_chains:
        return out, chains[:, :T]
    return out


def prefill(k, v, alpha, beta, nthreads: int = 0) -> np.ndarray:
    """Eq. 1 from the zero state over N prompt tokens: k [N, H, dk], v [N, H, dv], gates [N, H] -> fp64 [H, dv, dk]."""
    lib = _load()
    k, v, alpha, beta = _f32(k), _f32(v), _f32(alpha), _f32(beta)
    N, H, dk = k.shape
    dv = v.shape[2]
    assert v.shape == (N, H, dv) and alpha.shape == (N, H) and beta.shape == (N, H)
    S = np.empty((H, dv, dk), dtype=np.float64)
    lib.oracle_gdn_prefill(H, dk, dv, N, k.ctypes.data, v.ctypes.data, alpha.ctypes.data,
                           beta.ctypes.data, S.ctypes.data, nthreads)
    return S


def decode_grouped(S0, steps, parents, q, sel=None, nthreads: int = 0, return_chains: bool = False):
    """Grouped value heads: Hv value heads share Hk = Hv / g key heads (value head j reads the query and keys of
    key head j // g; states, values and gates are per value head).  By definition this is the ungrouped recurrence
    with every key head's q and k repeated g times, which is how it is evaluated.

    S0 [Hv, dv, dk]; steps: k [W_t, Hk, dk], v [W_t, Hv, dv], alpha, beta [W_t, Hv]; q [W, Hk, dk]."""
    S0 = _f32(S0)
    Hv = S0.shape[0]
    q = _f32(q)
    Hk = q.shape[1]
    assert Hv % Hk == 0
    g = Hv // Hk
    wide = [dict(s, k=np.repeat(_f32(s["k"]), g, axis=1)) for s in steps]
    return decode(S0, wide, parents, np.repeat(q, g, axis=1), sel=sel, nthreads=nthreads, return_chains=return_chains)


def prefill_grouped(k, v, alpha, beta, nthreads: int = 0) -> np.ndarray:
    """Eq. 1 from the zero state with grouped value heads: k [N, Hk, dk], v [N, Hv, dv], gates [N, Hv]."""
    k, v = _f32(k), _f32(v)
    g = v.shape[1] // k.shape[1]
    assert g * k.shape[1] == v.shape[1]
    return prefill(np.repeat(k, g, axis=1), v, alpha, beta, nthreads)
