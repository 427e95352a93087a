"""ctypes binding of the C ABI in include/onela.h: same names, argument marshalling only.

Every step of the decode path runs inside libonela.so; this module converts torch tensors to device
pointers, checks shapes and dtypes, and raises on a negative status.  It fails loudly when the library
is missing or cannot be loaded: there is no fallback of any kind.
"""
from __future__ import annotations

import ctypes
from ctypes import POINTER, c_char_p, c_int32, c_int64, c_size_t, c_uint32, c_void_p
from pathlib import Path

import torch

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libonela.so"

OK, E_INVAL, E_CAPACITY, E_ORDER, E_CUDA, E_UNSUPPORTED, E_DEVICE_CHECK, E_TIMEOUT = 0, -1, -2, -3, -4, -5, -6, -7
DTYPE_F32, DTYPE_BF16 = 0, 1
MAX_BATCH = 64
FLAG_DRY_RUN, FLAG_FORCE_GENERIC, FLAG_GTR_DELTA, FLAG_SHARED_CHAINS = 1, 2, 4, 8

_TORCH_DTYPE = {DTYPE_F32: torch.float32, DTYPE_BF16: torch.bfloat16}
_DTYPE_CODE = {torch.float32: DTYPE_F32, torch.bfloat16: DTYPE_BF16, "fp32": DTYPE_F32, "bf16": DTYPE_BF16}


class OnelaConfig(ctypes.Structure):
    _fields_ = [("num_requests", c_int32), ("num_layers", c_int32), ("num_heads", c_int32), ("dk", c_int32),
                ("dv", c_int32), ("max_beam", c_int32), ("max_steps", c_int32), ("rec_dtype", c_int32),
                ("out_dtype", c_int32), ("arena_slots", c_int64), ("flags", c_uint32), ("num_v_heads", c_int32)]

    @property
    def value_heads(self) -> int:
        """Value heads: num_v_heads, or num_heads when that is 0 (one value head per key head)."""
        return self.num_v_heads or self.num_heads


class OnelaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


_lib = None

# name -> (restype, argtypes); the ABI test checks this table against the header
PROTOTYPES = {
    "onela_workspace_bytes": (c_size_t, [POINTER(OnelaConfig)]),
    "onela_create": (c_int32, [POINTER(OnelaConfig), c_void_p, c_size_t, POINTER(c_void_p)]),
    "onela_destroy": (c_int32, [c_void_p]),
    "onela_reset": (c_int32, [c_void_p, c_void_p]),
    "onela_init_shared_state": (c_int32, [c_void_p, c_int32, c_int32, c_void_p, c_void_p]),
    "onela_init_shared_states": (c_int32, [c_void_p, c_int32, c_int32, c_void_p, c_void_p]),
    "onela_prefill_shared_state": (c_int32, [c_void_p, c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_void_p,
                                             c_int32, c_void_p]),
    "onela_export_shared_state": (c_int32, [c_void_p, c_int32, c_int32, c_void_p, c_void_p]),
    "onela_reorder_beams": (c_int32, [c_void_p, c_int32, c_int32, c_void_p, c_int32, c_void_p]),
    "onela_release_request": (c_int32, [c_void_p, c_int32]),
    "onela_select_beams_static": (c_int32, [c_void_p, c_void_p, c_int32, c_int32, c_int32, c_int32, c_void_p, c_void_p,
                                            c_void_p, c_void_p]),
    "onela_select_beams": (c_int32, [c_void_p, c_int32, c_int32, c_void_p, c_void_p, c_int32, c_int32, c_void_p, c_void_p,
                                     c_void_p, c_void_p]),
    "onela_append_records": (c_int32, [c_void_p, c_int32, c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_void_p,
                                       c_void_p]),
    "onela_append_decode_step": (c_int32, [c_void_p, c_int32, c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_void_p,
                                           c_void_p, c_void_p, c_void_p]),
    "onela_decode_step": (c_int32, [c_void_p, c_int32, c_int32, c_int32, c_void_p, c_void_p, c_void_p]),
    "onela_export_chains": (c_int32, [c_void_p, c_int32, c_void_p, POINTER(c_int32), POINTER(c_int32), c_void_p]),
    "onela_poll_device_status": (c_int32, [c_void_p, POINTER(c_int32), POINTER(c_int32)]),
    "onela_get_stats": (c_int32, [c_void_p, POINTER(c_int64), POINTER(c_int64), POINTER(c_int64)]),
    "onela_get_step_base": (c_int32, [c_void_p, c_int32, c_int32, POINTER(c_int32)]),
    "onela_launch_count": (c_int64, [c_void_p]),
    "onela_uses_tensor_core_path": (c_int32, [c_void_p]),
    "onela_status_string": (c_char_p, [c_int32]),
}


def load_library() -> ctypes.CDLL:
    """Load libonela.so (built in-tree by build.py).  Raises if it is missing: no fallback exists."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2609_12399_b200.build` "
                               "(or __graft_entry__.build()) first; there is no CPU or PyTorch fallback")
        lib = ctypes.CDLL(str(LIB_PATH))
        for name, (res, args) in PROTOTYPES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return load_library().onela_status_string(status).decode()


def _check(status: int, where: str) -> None:
    if status != OK:
        raise OnelaError(status, where)


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def make_config(num_requests, num_layers, num_heads, dk, dv, max_beam, max_steps, rec_dtype, out_dtype,
                arena_slots, flags=0, num_v_heads=0) -> OnelaConfig:
    return OnelaConfig(num_requests, num_layers, num_heads, dk, dv, max_beam, max_steps,
                       _DTYPE_CODE[rec_dtype], _DTYPE_CODE[out_dtype], arena_slots, flags, num_v_heads)


def onela_select_beams_static(beam_scores, cand_logp, W_new, parents_out, codes_out, scores_out, stream=None) -> None:
    """Beam selection for callers without a workspace or a context (see onela.h): shapes are read off the tensors
    (beam_scores [R, W_prev] fp32, cand_logp [R, W_prev, C] fp32, outputs [R, W_new]); allocates nothing."""
    R, W_prev, C = cand_logp.shape
    for t, dt, shape, name in ((beam_scores, torch.float32, (R, W_prev), "beam_scores"), (cand_logp, torch.float32, (R, W_prev, C), "cand_logp"),
                               (parents_out, torch.int32, (R, W_new), "parents_out"), (codes_out, torch.int32, (R, W_new), "codes_out"),
                               (scores_out, torch.float32, (R, W_new), "scores_out")):
        if t.device.type != "cuda" or t.dtype != dt or tuple(t.shape) != shape or not t.is_contiguous():
            raise ValueError(f"{name}: expected a contiguous CUDA {dt} tensor of shape {shape}")
    _check(load_library().onela_select_beams_static(
        c_void_p(beam_scores.data_ptr()), c_void_p(cand_logp.data_ptr()), R, W_prev, C, W_new, c_void_p(parents_out.data_ptr()),
        c_void_p(codes_out.data_ptr()), c_void_p(scores_out.data_ptr()), c_void_p(_stream_ptr(stream))), "onela_select_beams_static")


def onela_workspace_bytes(cfg: OnelaConfig) -> int:
    return int(load_library().onela_workspace_bytes(ctypes.byref(cfg)))


class Onela:
    """A context over a torch-owned workspace.  Methods mirror the C entry points one to one."""

    def __init__(self, cfg: OnelaConfig, device="cuda", workspace_ptr: int | None = None):
        self.lib = load_library()
        self.cfg = cfg
        self.device = torch.device(device)
        nbytes = onela_workspace_bytes(cfg)
        if nbytes == 0:
            raise OnelaError(E_INVAL, "onela_workspace_bytes")
        self.workspace_bytes = nbytes
        dry = bool(cfg.flags & FLAG_DRY_RUN)
        if workspace_ptr is not None:
            self.workspace, ptr = None, workspace_ptr
        elif dry and self.device.type != "cuda":
            self.workspace, ptr = None, 1024  # never dereferenced: a dry run launches nothing
        else:
            # over-allocate to guarantee the 1024-byte alignment whatever the caching allocator returns
            self.workspace = torch.empty(nbytes + 1024, dtype=torch.uint8, device=self.device)
            ptr = (self.workspace.data_ptr() + 1023) // 1024 * 1024
        self.workspace_ptr = ptr
        h = c_void_p()
        _check(self.lib.onela_create(ctypes.byref(cfg), c_void_p(ptr), nbytes, ctypes.byref(h)), "onela_create")
        self.handle = h
        self.rec_dtype = _TORCH_DTYPE[cfg.rec_dtype]
        self.out_dtype = _TORCH_DTYPE[cfg.out_dtype]

    def close(self):
        if getattr(self, "handle", None):
            self.lib.onela_destroy(self.handle)
            self.handle = None

    def __del__(self):
        self.close()

    # --- marshalling helpers ---
    def _dry(self) -> bool:
        return bool(self.cfg.flags & FLAG_DRY_RUN)

    def _ptr(self, t, dtype, shape, name):
        if t is None:
            return None
        if self._dry() and not isinstance(t, torch.Tensor):
            return c_void_p(int(t))     # dry runs accept a fake, non-null address
        if not isinstance(t, torch.Tensor):
            raise TypeError(f"{name}: expected a torch tensor")
        if not self._dry() and t.device.type != "cuda":
            raise ValueError(f"{name}: must live on the CUDA device")
        if t.dtype != dtype or tuple(t.shape) != tuple(shape) or not t.is_contiguous():
            raise ValueError(f"{name}: expected contiguous {dtype} of shape {tuple(shape)}, got {t.dtype} {tuple(t.shape)}")
        return c_void_p(t.data_ptr())

    def _width(self, req_begin):
        d, w = c_int32(), c_int32()
        self.lib.onela_export_chains(self.handle, req_begin, None, ctypes.byref(d), ctypes.byref(w), None)
        return d.value, w.value

    # --- the C entry points ---
    def onela_reset(self, stream=None):
        _check(self.lib.onela_reset(self.handle, c_void_p(0 if self._dry() else _stream_ptr(stream))), "onela_reset")

    def onela_init_shared_state(self, request, layer, S0, stream=None):
        c = self.cfg
        p = self._ptr(S0, torch.float32, (c.value_heads, c.dv, c.dk), "S0")
        _check(self.lib.onela_init_shared_state(self.handle, request, layer, p, self._s(stream)), "onela_init_shared_state")

    def onela_init_shared_states(self, req_begin, req_count, S0, stream=None):
        c = self.cfg
        p = self._ptr(S0, torch.float32, (req_count, c.num_layers, c.value_heads, c.dv, c.dk), "S0")
        _check(self.lib.onela_init_shared_states(self.handle, req_begin, req_count, p, self._s(stream)), "onela_init_shared_states")

    def onela_prefill_shared_state(self, request, layer, k, v, alpha, beta, stream=None):
        c = self.cfg
        n = int(k.shape[0])
        _check(self.lib.onela_prefill_shared_state(
            self.handle, request, layer, self._ptr(k, self.rec_dtype, (n, c.num_heads, c.dk), "k"),
            self._ptr(v, self.rec_dtype, (n, c.num_heads, c.dv), "v"),
            self._ptr(alpha, torch.float32, (n, c.num_heads), "alpha"),
            self._ptr(beta, torch.float32, (n, c.num_heads), "beta"), n, self._s(stream)), "onela_prefill_shared_state")

    def onela_export_shared_state(self, request, layer, stream=None) -> torch.Tensor:
        """Returns the stored S_0 of (request, layer) as fp32 [H, dv, dk] on the device."""
        c = self.cfg
        out = torch.empty((c.value_heads, c.dv, c.dk), dtype=torch.float32, device=self.device)
        _check(self.lib.onela_export_shared_state(self.handle, request, layer, c_void_p(out.data_ptr()),
                                                  self._s(stream)), "onela_export_shared_state")
        return out

    def onela_reorder_beams(self, req_begin, req_count, parents, W_new, stream=None):
        p = None if parents is None else self._ptr(parents, torch.int32, (req_count, W_new), "parents")
        _check(self.lib.onela_reorder_beams(self.handle, req_begin, req_count, p, W_new, self._s(stream)),
               "onela_reorder_beams")

    def onela_release_request(self, request):
        _check(self.lib.onela_release_request(self.handle, request), "onela_release_request")

    def onela_select_beams(self, req_begin, req_count, beam_scores, cand_logp, C, W_new, parents_out, codes_out, scores_out,
                           stream=None):
        depth, W = self._width(req_begin)
        W_prev = W if depth >= 1 else 1
        _check(self.lib.onela_select_beams(
            self.handle, req_begin, req_count,
            self._ptr(beam_scores, torch.float32, (req_count, W_prev), "beam_scores"),
            self._ptr(cand_logp, torch.float32, (req_count, W_prev, C), "cand_logp"), C, W_new,
            self._ptr(parents_out, torch.int32, (req_count, W_new), "parents_out"),
            self._ptr(codes_out, torch.int32, (req_count, W_new), "codes_out"),
            self._ptr(scores_out, torch.float32, (req_count, W_new), "scores_out"), self._s(stream)), "onela_select_beams")

    def onela_append_records(self, req_begin, req_count, layer, k, v, alpha, beta, stream=None):
        c = self.cfg
        _, W = self._width(req_begin)
        _check(self.lib.onela_append_records(
            self.handle, req_begin, req_count, layer,
            self._ptr(k, self.rec_dtype, (req_count, W, c.num_heads, c.dk), "k"),
            self._ptr(v, self.rec_dtype, (req_count, W, c.value_heads, c.dv), "v"),
            self._ptr(alpha, torch.float32, (req_count, W, c.value_heads), "alpha"),
            self._ptr(beta, torch.float32, (req_count, W, c.value_heads), "beta"), self._s(stream)), "onela_append_records")

    def onela_decode_step(self, req_begin, req_count, layer, q, out, stream=None):
        c = self.cfg
        _, W = self._width(req_begin)
        _check(self.lib.onela_decode_step(
            self.handle, req_begin, req_count, layer,
            self._ptr(q, self.rec_dtype, (req_count, W, c.num_heads, c.dk), "q"),
            self._ptr(out, self.out_dtype, (req_count, W, c.value_heads, c.dv), "out"), self._s(stream)), "onela_decode_step")

    def onela_append_decode_step(self, req_begin, req_count, layer, k, v, alpha, beta, q, out, stream=None):
        c = self.cfg
        _, W = self._width(req_begin)
        _check(self.lib.onela_append_decode_step(
            self.handle, req_begin, req_count, layer,
            self._ptr(k, self.rec_dtype, (req_count, W, c.num_heads, c.dk), "k"),
            self._ptr(v, self.rec_dtype, (req_count, W, c.value_heads, c.dv), "v"),
            self._ptr(alpha, torch.float32, (req_count, W, c.value_heads), "alpha"),
            self._ptr(beta, torch.float32, (req_count, W, c.value_heads), "beta"),
            self._ptr(q, self.rec_dtype, (req_count, W, c.num_heads, c.dk), "q"),
            self._ptr(out, self.out_dtype, (req_count, W, c.value_heads, c.dv), "out"), self._s(stream)),
            "onela_append_decode_step")

    def onela_export_chains(self, request, stream=None) -> torch.Tensor:
        """Returns int32 [W, depth] global slot ids (oldest first) on the device."""
        d, w = self._width(request)
        if d < 1:
            raise OnelaError(E_ORDER, "onela_export_chains")
        out = torch.empty((w, d), dtype=torch.int32, device=self.device)
        _check(self.lib.onela_export_chains(self.handle, request, c_void_p(out.data_ptr()), None, None,
                                            self._s(stream)), "onela_export_chains")
        return out

    def onela_poll_device_status(self):
        code, detail = c_int32(), c_int32()
        _check(self.lib.onela_poll_device_status(self.handle, ctypes.byref(code), ctypes.byref(detail)),
               "onela_poll_device_status")
        return code.value, detail.value

    def onela_get_stats(self):
        a, b, c = c_int64(), c_int64(), c_int64()
        _check(self.lib.onela_get_stats(self.handle, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)), "onela_get_stats")
        return {"s0_bytes": a.value, "arena_bytes_used": b.value, "index_bytes": c.value}

    def onela_get_step_base(self, request, step) -> int:
        b = c_int32()
        _check(self.lib.onela_get_step_base(self.handle, request, step, ctypes.byref(b)), "onela_get_step_base")
        return b.value

    def onela_launch_count(self) -> int:
        return int(self.lib.onela_launch_count(self.handle))

    def onela_uses_tensor_core_path(self) -> int:
        """0: CUDA-core kernels; 1: the warp-specialised tcgen05 kernel; 2: the tiled tcgen05 kernel."""
        return int(self.lib.onela_uses_tensor_core_path(self.handle))

    def depth_and_width(self, request):
        return self._width(request)

    def _s(self, stream):
        return c_void_p(0) if self._dry() and self.device.type != "cuda" else c_void_p(_stream_ptr(stream))
