"""ctypes binding of libtopk.so — argument marshalling only.

Every function has the name and the meaning of its C counterpart in
``include/topk.h``; tensors are passed as raw device pointers.  PyTorch is used
for device memory and streams, nothing else: all computation happens in the
library's CUDA kernels.  There is no fallback: if the library is missing or a
call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

from . import build as _build

TK_MODE_UNI = 0
TK_MODE_BIDIR = 1
TK_MODE_EF = 2

EXPORTS = ["tk_workspace_bytes", "tk_init", "tk_step", "tk_step_uplink", "tk_messages", "tk_step_server", "tk_step_host", "tk_topk", "tk_topk_noalloc", "tk_topk_noalloc_status", "tk_ef_bytes",
           "tk_ef_attach", "tk_ef_state", "tk_set_diagnostics", "tk_diagnostics", "tk_set_kdown",
           "tk_last_uplink", "tk_last_aggregate", "tk_last_downlink", "tk_status", "tk_set_profile",
           "tk_set_force_general", "tk_set_cand_cap", "tk_set_bound_reuse", "tk_comm_model", "tk_set_graph", "tk_launch_count", "tk_debug_phase_clock", "tk_destroy", "tk_release_scratch", "tk_strerror"]


class TkError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__("%s failed: %s (%d)" % (what, strerror(code), code))
        self.code = code


class tk_stats(ctypes.Structure):
    _fields_ = [("device_status", ctypes.c_int32), ("rows_general", ctypes.c_int32),
                ("union_size", ctypes.c_int64), ("downlink_count", ctypes.c_int64),
                ("cand_min", ctypes.c_int64), ("cand_max", ctypes.c_int64),
                ("select_ms_sum", ctypes.c_float), ("select_samples", ctypes.c_int32)]


class tk_diag(ctypes.Structure):
    _fields_ = [("nonzero_fraction", ctypes.c_double), ("union_fraction", ctypes.c_double),
                ("compression_factor", ctypes.c_double), ("one_minus_gamma_up_max", ctypes.c_double),
                ("one_minus_gamma_down", ctypes.c_double), ("rho", ctypes.c_double)]


class tk_comm(ctypes.Structure):
    _fields_ = [("uplink_words", ctypes.c_int64), ("downlink_words_uni_max", ctypes.c_int64),
                ("downlink_words_uni", ctypes.c_int64), ("downlink_words_bi", ctypes.c_int64),
                ("time_uni", ctypes.c_double), ("time_uni_union", ctypes.c_double), ("time_bi", ctypes.c_double),
                ("compression_factor", ctypes.c_double)]


_lib = None


def library_path() -> str:
    return _build.LIB


def load(build_if_missing: bool = True):
    """Open libtopk.so (building it first when the sources are newer and nvcc exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if build_if_missing:
        try:
            _build.build()
        except Exception:
            if not os.path.exists(_build.LIB):
                raise
    if not os.path.exists(_build.LIB):
        raise RuntimeError("libtopk.so is missing; run `python -m paper_2209_15203_b200.build`")
    lib = ctypes.CDLL(_build.LIB)
    vp, i64, i32, f32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_float
    lib.tk_workspace_bytes.argtypes = [i64, i32, i64, i64]
    lib.tk_workspace_bytes.restype = ctypes.c_size_t
    lib.tk_init.argtypes = [ctypes.POINTER(vp), i64, i32, i64, i64, vp, vp, ctypes.c_size_t, vp]
    lib.tk_step.argtypes = [vp, vp, vp, f32, ctypes.c_int]
    lib.tk_step_host.argtypes = [vp, vp, vp, f32, ctypes.c_int]
    lib.tk_step_uplink.argtypes = [vp, vp, i32, i32, f32, ctypes.c_int]
    lib.tk_step_uplink.restype = ctypes.c_int
    lib.tk_messages.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(ctypes.c_size_t)]
    lib.tk_messages.restype = ctypes.c_int
    lib.tk_step_server.argtypes = [vp, vp, f32, ctypes.c_int]
    lib.tk_step_server.restype = ctypes.c_int
    lib.tk_topk.argtypes = [vp, vp, i32, i64, i64, vp, vp]
    lib.tk_topk_noalloc.argtypes = [vp, i32, i64, i64, vp, vp, vp]
    lib.tk_topk_noalloc.restype = ctypes.c_int
    lib.tk_topk_noalloc_status.argtypes = []
    lib.tk_topk_noalloc_status.restype = ctypes.c_int
    lib.tk_set_bound_reuse.argtypes = [vp, ctypes.c_int]
    lib.tk_set_bound_reuse.restype = ctypes.c_int
    lib.tk_set_cand_cap.argtypes = [vp, i64]
    lib.tk_set_cand_cap.restype = ctypes.c_int
    lib.tk_comm_model.argtypes = [i32, i64, i64, i64, ctypes.c_double, ctypes.c_double, ctypes.c_double,
                                  ctypes.c_double, ctypes.POINTER(tk_comm)]
    lib.tk_comm_model.restype = ctypes.c_int
    lib.tk_ef_bytes.argtypes = [i64, i32, i64]
    lib.tk_ef_bytes.restype = ctypes.c_size_t
    lib.tk_ef_attach.argtypes = [vp, vp, ctypes.c_size_t]
    lib.tk_ef_attach.restype = ctypes.c_int
    lib.tk_ef_state.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(vp)]
    lib.tk_ef_state.restype = ctypes.c_int
    lib.tk_set_diagnostics.argtypes = [vp, ctypes.c_int]
    lib.tk_set_diagnostics.restype = ctypes.c_int
    lib.tk_diagnostics.argtypes = [vp, ctypes.POINTER(tk_diag), ctypes.POINTER(ctypes.c_double)]
    lib.tk_diagnostics.restype = ctypes.c_int
    lib.tk_set_kdown.argtypes = [vp, i64]
    lib.tk_last_uplink.argtypes = [vp, vp, vp]
    lib.tk_last_aggregate.argtypes = [vp, vp, vp, ctypes.POINTER(i64)]
    lib.tk_last_downlink.argtypes = [vp, vp, vp, ctypes.POINTER(i64)]
    lib.tk_status.argtypes = [vp, ctypes.POINTER(tk_stats)]
    lib.tk_set_profile.argtypes = [vp, ctypes.c_int]
    lib.tk_set_force_general.argtypes = [vp, ctypes.c_int]
    lib.tk_set_graph.argtypes = [vp, ctypes.c_int]
    lib.tk_set_graph.restype = ctypes.c_int
    lib.tk_launch_count.argtypes = [vp]
    lib.tk_launch_count.restype = i64
    lib.tk_debug_phase_clock.argtypes = [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double), ctypes.c_int32]
    lib.tk_debug_phase_clock.restype = ctypes.c_int
    lib.tk_destroy.argtypes = [vp]
    lib.tk_destroy.restype = None
    lib.tk_release_scratch.argtypes = []
    lib.tk_release_scratch.restype = None
    lib.tk_strerror.argtypes = [ctypes.c_int]
    lib.tk_strerror.restype = ctypes.c_char_p
    for name in ("tk_init", "tk_step", "tk_step_host", "tk_topk", "tk_set_kdown", "tk_last_uplink",
                 "tk_last_aggregate", "tk_last_downlink", "tk_status", "tk_set_profile", "tk_set_force_general"):
        getattr(lib, name).restype = ctypes.c_int
    _lib = lib
    return lib


def strerror(code: int) -> str:
    return load().tk_strerror(code).decode()


def _check(code: int, what: str) -> None:
    if code != 0:
        raise TkError(code, what)


def _dev(t: torch.Tensor, dtype: torch.dtype) -> int:
    if not (t.is_cuda and t.is_contiguous() and t.dtype == dtype):
        raise ValueError("expected a contiguous CUDA tensor of dtype %s" % dtype)
    return t.data_ptr()


def tk_workspace_bytes(d: int, N: int, K_up: int, K_down: int) -> int:
    return int(load().tk_workspace_bytes(d, N, K_up, K_down))


class Context:
    """Owns a tk_ctx and the workspace tensor it lives in."""

    def __init__(self, d: int, N: int, K_up: int, K_down: int, p: torch.Tensor,
                 device: Optional[torch.device] = None, stream: Optional[torch.cuda.Stream] = None):
        lib = load()
        self.d, self.N, self.K_up, self.K_down = d, N, K_up, K_down
        self.device = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
        nbytes = tk_workspace_bytes(d, N, K_up, K_down)
        if nbytes == 0:
            raise TkError(-1, "tk_workspace_bytes")
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
            self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
            p_host = p.detach().to("cpu", torch.float32).contiguous()
            handle = ctypes.c_void_p()
            _check(lib.tk_init(ctypes.byref(handle), d, N, K_up, K_down, p_host.data_ptr(),
                               self.workspace.data_ptr(), nbytes, self.stream.cuda_stream), "tk_init")
        self._h = handle
        self.ucap = min(N * K_up, d)
        self.last_mode = None

    def close(self) -> None:
        if getattr(self, "_h", None):
            load().tk_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the calls of include/topk.h --
    def tk_step(self, w: torch.Tensor, grads: torch.Tensor, alpha: float, mode: int) -> None:
        assert w.numel() == self.d and grads.numel() == self.N * self.d
        _check(load().tk_step(self._h, _dev(w, torch.float32), _dev(grads, torch.float32), alpha, mode), "tk_step")
        self.last_mode = mode

    def tk_step_uplink(self, grads_local: torch.Tensor, row0: int, alpha: float, mode: int) -> None:
        rows = grads_local.numel() // self.d
        assert grads_local.numel() == rows * self.d
        _check(load().tk_step_uplink(self._h, _dev(grads_local, torch.float32), row0, rows, alpha, mode),
               "tk_step_uplink")

    def tk_messages(self) -> torch.Tensor:
        """The message buffer as an int64 view [N][K_up] of the workspace (one 8-byte entry =
        int32 index in the low half, fp32 bits in the high half), for the all-gather."""
        ptr, per_row = ctypes.c_void_p(), ctypes.c_size_t()
        _check(load().tk_messages(self._h, ctypes.byref(ptr), ctypes.byref(per_row)), "tk_messages")
        off = (ptr.value - self.workspace.data_ptr()) // 8
        return self.workspace.view(torch.int64)[off:off + self.N * self.K_up].view(self.N, self.K_up)

    def tk_step_server(self, w: torch.Tensor, alpha: float, mode: int) -> None:
        assert w.numel() == self.d
        _check(load().tk_step_server(self._h, _dev(w, torch.float32), alpha, mode), "tk_step_server")
        self.last_mode = mode

    def tk_step_host(self, w_host: torch.Tensor, grads_host: torch.Tensor, alpha: float, mode: int) -> None:
        for t in (w_host, grads_host):
            if t.is_cuda or not t.is_contiguous() or t.dtype != torch.float32:
                raise ValueError("expected contiguous float32 host tensors")
        assert w_host.numel() == self.d and grads_host.numel() == self.N * self.d
        with torch.cuda.device(self.device):
            _check(load().tk_step_host(self._h, w_host.data_ptr(), grads_host.data_ptr(), alpha, mode),
                   "tk_step_host")
        self.last_mode = mode

    def tk_topk(self, x: torch.Tensor, K: int) -> Tuple[torch.Tensor, torch.Tensor]:
        return tk_topk(x, K, ctx=self)

    def tk_ef_attach(self) -> None:
        """Allocate (with torch) and attach the error memories; epsilon = delta = 0."""
        lib = load()
        nbytes = int(lib.tk_ef_bytes(self.d, self.N, self.K_down))
        if nbytes == 0:
            raise TkError(-1, "tk_ef_bytes")
        with torch.cuda.device(self.device):
            self.ef_memory = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
            _check(lib.tk_ef_attach(self._h, self.ef_memory.data_ptr(), nbytes), "tk_ef_attach")

    def tk_ef_state(self) -> Tuple[torch.Tensor, torch.Tensor]:
        """Views of epsilon [N][d] and delta [d] inside the attached memory."""
        e, dl = ctypes.c_void_p(), ctypes.c_void_p()
        _check(load().tk_ef_state(self._h, ctypes.byref(e), ctypes.byref(dl)), "tk_ef_state")
        base = self.ef_memory.data_ptr()
        flat = self.ef_memory.view(torch.float32)
        eo, do = (e.value - base) // 4, (dl.value - base) // 4
        return flat[eo:eo + self.N * self.d].view(self.N, self.d), flat[do:do + self.d]

    def tk_set_diagnostics(self, level) -> None:
        """0 = off, 1 = cheap diagnostics, 2 = also the gap constant (re-reads the gradients)."""
        _check(load().tk_set_diagnostics(self._h, int(level)), "tk_set_diagnostics")

    def tk_diagnostics(self):
        """(tk_diag, per-worker 1 - gamma list) of the last step."""
        out = tk_diag()
        per = (ctypes.c_double * self.N)()
        _check(load().tk_diagnostics(self._h, ctypes.byref(out), per), "tk_diagnostics")
        return out, list(per)

    def tk_set_kdown(self, K_down: int) -> None:
        _check(load().tk_set_kdown(self._h, K_down), "tk_set_kdown")
        self.K_down = K_down

    def tk_last_uplink(self) -> Tuple[torch.Tensor, torch.Tensor]:
        idx = torch.empty((self.N, self.K_up), dtype=torch.int32, device=self.device)
        val = torch.empty((self.N, self.K_up), dtype=torch.float32, device=self.device)
        _check(load().tk_last_uplink(self._h, idx.data_ptr(), val.data_ptr()), "tk_last_uplink")
        return idx, val

    def _msg(self, fn, name: str, n: int) -> Tuple[torch.Tensor, torch.Tensor]:
        idx = torch.empty(n, dtype=torch.int32, device=self.device)
        val = torch.empty(n, dtype=torch.float32, device=self.device)
        count = ctypes.c_int64(0)
        _check(fn(self._h, idx.data_ptr(), val.data_ptr(), ctypes.byref(count)), name)
        return idx[:count.value], val[:count.value]

    def tk_last_aggregate(self) -> Tuple[torch.Tensor, torch.Tensor]:
        return self._msg(load().tk_last_aggregate, "tk_last_aggregate", self.ucap)

    def tk_last_downlink(self) -> Tuple[torch.Tensor, torch.Tensor]:
        n = self.K_down if (self.last_mode is not None and self.last_mode & TK_MODE_BIDIR) else self.ucap
        return self._msg(load().tk_last_downlink, "tk_last_downlink", max(n, 1))

    def tk_status(self, check: bool = True) -> tk_stats:
        st = tk_stats()
        rc = load().tk_status(self._h, ctypes.byref(st))
        if check:
            _check(rc, "tk_status")
        return st

    def tk_set_profile(self, every: int) -> None:
        """0 = off; n = timestamp the streaming pass of every n-th step."""
        _check(load().tk_set_profile(self._h, int(every)), "tk_set_profile")

    def tk_set_graph(self, on: bool) -> None:
        _check(load().tk_set_graph(self._h, 1 if on else 0), "tk_set_graph")

    def tk_set_force_general(self, on: bool) -> None:
        _check(load().tk_set_force_general(self._h, 1 if on else 0), "tk_set_force_general")

    def tk_set_bound_reuse(self, on: bool) -> None:
        _check(load().tk_set_bound_reuse(self._h, 1 if on else 0), "tk_set_bound_reuse")

    def tk_set_cand_cap(self, cap: int) -> None:
        """Testing aid: cap every row's candidate list (0 restores the laid-out capacity)."""
        _check(load().tk_set_cand_cap(self._h, int(cap)), "tk_set_cand_cap")

    def tk_launch_count(self) -> int:
        return int(load().tk_launch_count(self._h))

    PHASE_STAMPS = ("sampling starts", "sampling ends", "streaming pass starts", "streaming pass ends",
                    "verification starts", "verification ends",
                    "uplink select starts", "uplink: candidates loaded", "uplink: first level done",
                    "uplink: threshold known", "uplink select ends",
                    "server sum starts", "server sum ends",
                    "downlink select starts", "downlink: entries loaded", "downlink: first level done",
                    "downlink: threshold known", "downlink select ends")

    def tk_debug_phase_clock(self):
        """(first_us, last_us) per stamp of PHASE_STAMPS for the last step, and re-arms the stamps.
        Needs a library built with -DTK_PHASE_CLOCK=1 (raises otherwise)."""
        n = len(self.PHASE_STAMPS)
        first = (ctypes.c_double * n)()
        last = (ctypes.c_double * n)()
        _check(load().tk_debug_phase_clock(self._h, first, last, n), "tk_debug_phase_clock")
        return list(first), list(last)


def tk_topk(x: torch.Tensor, K: int, ctx: Optional[Context] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Top_K of every row of x ([rows][d] or [d]): (idx int32, val float32), ascending index."""
    x2 = x if x.dim() == 2 else x.reshape(1, -1)
    rows, d = x2.shape
    idx = torch.empty((rows, K), dtype=torch.int32, device=x.device)
    val = torch.empty((rows, K), dtype=torch.float32, device=x.device)
    with torch.cuda.device(x.device):
        # The library runs on the context's stream, or on the legacy default stream without a
        # context; x and the fresh outputs belong to torch's current stream.  Order the two.
        cur = torch.cuda.current_stream(x.device)
        run = ctx.stream if ctx is not None else torch.cuda.default_stream(x.device)
        if run != cur:
            run.wait_stream(cur)
        _check(load().tk_topk(ctx._h if ctx is not None else None, _dev(x2, torch.float32), rows, d, K,
                              idx.data_ptr(), val.data_ptr()), "tk_topk")
        if run != cur:
            cur.wait_stream(run)
    if x.dim() == 1:
        return idx[0], val[0]
    return idx, val


def tk_topk_noalloc(x: torch.Tensor, K: int, idx: torch.Tensor, val: torch.Tensor,
                    stream: Optional[torch.cuda.Stream] = None) -> None:
    """Top_K of every row of x into the caller's idx / val tensors without any device
    allocation: the library's scratch is a fixed array inside the library image (see
    include/topk.h for its size, the set-up done by the first call and the rule that
    overlapping calls race).  Raises TkError(-6) when the problem does not fit."""
    x2 = x if x.dim() == 2 else x.reshape(1, -1)
    rows, d = x2.shape
    assert idx.numel() == rows * K and val.numel() == rows * K
    with torch.cuda.device(x.device):
        s = stream if stream is not None else torch.cuda.current_stream(x.device)
        _check(load().tk_topk_noalloc(_dev(x2, torch.float32), rows, d, K, _dev(idx, torch.int32),
                                      _dev(val, torch.float32), s.cuda_stream), "tk_topk_noalloc")


def tk_comm_model(N: int, K_up: int, K_down: int, union_size: int, alpha1: float, beta1: float,
                  alpha2: float, beta2: float) -> tk_comm:
    """Section 4.2's words per step and transfer times (host arithmetic only; needs no GPU)."""
    out = tk_comm()
    _check(load().tk_comm_model(N, K_up, K_down, union_size, alpha1, beta1, alpha2, beta2, ctypes.byref(out)),
           "tk_comm_model")
    return out


def tk_topk_noalloc_status() -> int:
    """Waits for the device, then returns and clears the sticky status word of tk_topk_noalloc
    (0, or the negative TK_ERR_* code a kernel's consistency check raised)."""
    return int(load().tk_topk_noalloc_status())


def tk_release_scratch() -> None:
    load().tk_release_scratch()
