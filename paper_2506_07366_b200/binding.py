"""ctypes binding of libmoegps.so: argument marshalling only.

Every function here has the name of the C entry point it forwards to (include/moegps.h); tensors are
torch CUDA tensors of which only `data_ptr()` crosses the boundary.  There is no CPU path: if the
shared library is missing or cannot be loaded the import of this module raises.
"""
from __future__ import annotations

import ctypes
import dataclasses
import os

import torch

from . import build as _build

_c_int32_p = ctypes.POINTER(ctypes.c_int32)


class moegps_shape_t(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("T", "D", "F", "E", "K", "S", "gate_mode", "row_align", "c_max")]


@dataclasses.dataclass(frozen=True)
class Shape:
    T: int
    D: int
    F: int
    E: int
    K: int
    S: int
    gate_mode: int = 0
    row_align: int = 128
    c_max: int = 0

    @property
    def R(self) -> int:
        return self.T * self.K

    @property
    def Rcap(self) -> int:
        return self.T * self.K + self.S * (self.row_align - 1)

    def c_struct(self) -> moegps_shape_t:
        return moegps_shape_t(*(getattr(self, f[0]) for f in moegps_shape_t._fields_))


OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED_SHAPE, ERR_WORKSPACE_TOO_SMALL, ERR_CUDA = -1, -2, -3, -4
ERR_UNIMPLEMENTED, ERR_BAD_INDEX, ERR_TIMEOUT, ERR_HIST_MISMATCH = -5, -6, -7, -8
ERR_STATIC_SCRATCH_EXCEEDED = -9

EXPORTS = (
    "moegps_create", "moegps_destroy", "moegps_rcap", "moegps_workspace_bytes", "moegps_route",
    "moegps_route_histogram", "moegps_route_prepare", "moegps_dispatch_prepared", "moegps_route_logits", "moegps_histogram", "moegps_plan", "moegps_pack", "moegps_pack_slots", "moegps_dispatch", "moegps_dispatch_shares", "moegps_dispatch_static",
    "moegps_expert_ffn", "moegps_expert_ffn_gate_up", "moegps_expert_ffn_down", "moegps_combine",
    "moegps_status", "moegps_launch_count", "moegps_last_cuda_error", "moegps_error_string",
    "moegps_selftest_bounded_wait", "moegps_predictor_update", "moegps_predictor_update_ema", "moegps_error_rate",
)


class MoegpsError(RuntimeError):
    def __init__(self, code: int, where: str, cuda_error: int = 0):
        self.code = code
        msg = _lib().moegps_error_string(code).decode()
        if cuda_error:
            msg += f" (cudaError {cuda_error})"
        super().__init__(f"{where}: {msg} [{code}]")


_LIB = None


def library_path() -> str:
    """The in-tree build, unless MOEGPS_LIBRARY names another build of the same library."""
    return os.environ.get("MOEGPS_LIBRARY") or _build.LIB_PATH


def _lib():
    """Loads libmoegps.so (never builds it implicitly on a machine without nvcc; never falls back)."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = library_path()
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: build it with `python -m paper_2506_07366_b200.build` "
                          "(there is no fallback path)")
    lib = ctypes.CDLL(path)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    sig = {
        "moegps_create": (ctypes.c_int, [ctypes.POINTER(vp), ctypes.POINTER(moegps_shape_t), ctypes.c_int]),
        "moegps_destroy": (ctypes.c_int, [vp]),
        "moegps_rcap": (i64, [ctypes.POINTER(moegps_shape_t)]),
        "moegps_workspace_bytes": (ctypes.c_size_t, [ctypes.POINTER(moegps_shape_t)]),
        "moegps_route": (ctypes.c_int, [vp] * 7),
        "moegps_route_histogram": (ctypes.c_int, [vp] * 8),
        "moegps_route_prepare": (ctypes.c_int, [vp] * 9),
        "moegps_dispatch_prepared": (ctypes.c_int, [vp] * 12),
        "moegps_route_logits": (ctypes.c_int, [vp] * 6),
        "moegps_histogram": (ctypes.c_int, [vp] * 4),
        "moegps_plan": (ctypes.c_int, [vp, vp, i32, vp, vp, vp, vp, vp]),
        "moegps_pack": (ctypes.c_int, [vp, vp, vp, vp, i32, vp, vp, vp, vp, vp]),
        "moegps_pack_slots": (ctypes.c_int, [vp, vp, vp, i32, vp, vp, vp, vp, vp, vp]),
        "moegps_dispatch": (ctypes.c_int, [vp] * 12),
        "moegps_dispatch_shares": (ctypes.c_int, [vp] * 13),
        "moegps_dispatch_static": (ctypes.c_int, [vp] * 11),
        "moegps_expert_ffn": (ctypes.c_int, [vp] * 10),
        "moegps_expert_ffn_gate_up": (ctypes.c_int, [vp] * 8),
        "moegps_expert_ffn_down": (ctypes.c_int, [vp] * 7),
        "moegps_combine": (ctypes.c_int, [vp] * 6),
        "moegps_selftest_bounded_wait": (ctypes.c_int, [vp, i64, vp]),
        "moegps_predictor_update": (ctypes.c_int, [vp] * 5),
        "moegps_predictor_update_ema": (ctypes.c_int, [vp, vp, vp, i32, vp, vp]),
        "moegps_error_rate": (ctypes.c_int, [vp] * 5),
        "moegps_status": (ctypes.c_int, [vp, vp, _c_int32_p]),
        "moegps_launch_count": (i64, [vp]),
        "moegps_last_cuda_error": (ctypes.c_int, [vp]),
        "moegps_error_string": (ctypes.c_char_p, [ctypes.c_int]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)          # AttributeError if the library does not export it
        fn.restype = res
        fn.argtypes = args
    _LIB = lib
    return lib


def _ptr(t, dtype, shape, name, allow_none=False):
    if t is None:
        if allow_none:
            return None
        raise ValueError(f"{name} is required")
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} must have shape {tuple(shape)}, got {tuple(t.shape)}")
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    if isinstance(stream, torch.cuda.Stream):
        return ctypes.c_void_p(stream.cuda_stream)
    return ctypes.c_void_p(int(stream))


class Context:
    """Owns one moegps_ctx_t.  Methods carry the C names without the prefix."""

    def __init__(self, shape: Shape, device: int | None = None):
        lib = _lib()
        if not torch.cuda.is_available():
            raise RuntimeError("moegps needs a CUDA device (sm_100a); there is no CPU path")
        self.shape = shape
        self.device = torch.cuda.current_device() if device is None else int(device)
        self._h = ctypes.c_void_p()
        cs = shape.c_struct()
        rc = lib.moegps_create(ctypes.byref(self._h), ctypes.byref(cs), self.device)
        if rc != OK:
            self._h = ctypes.c_void_p()
            raise MoegpsError(rc, "moegps_create")

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            _lib().moegps_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc, where):
        if rc != OK:
            raise MoegpsError(rc, where, _lib().moegps_last_cuda_error(self._h))

    # -- the six steps ------------------------------------------------------------------------
    def route(self, x, w_router, bias, topk_idx, topk_w, stream=None):
        s = self.shape
        self._check(_lib().moegps_route(
            self._h, _ptr(x, torch.bfloat16, (s.T, s.D), "x"),
            _ptr(w_router, torch.bfloat16, (s.E, s.D), "w_router"),
            _ptr(bias, torch.float32, (s.E,), "bias", allow_none=True),
            _ptr(topk_idx, torch.int32, (s.T, s.K), "topk_idx"),
            _ptr(topk_w, torch.float32, (s.T, s.K), "topk_w"), _stream(stream)), "moegps_route")

    def route_histogram(self, x, w_router, bias, topk_idx, topk_w, hist, stream=None):
        s = self.shape
        self._check(_lib().moegps_route_histogram(
            self._h, _ptr(x, torch.bfloat16, (s.T, s.D), "x"),
            _ptr(w_router, torch.bfloat16, (s.E, s.D), "w_router"),
            _ptr(bias, torch.float32, (s.E,), "bias", allow_none=True),
            _ptr(topk_idx, torch.int32, (s.T, s.K), "topk_idx"),
            _ptr(topk_w, torch.float32, (s.T, s.K), "topk_w"),
            _ptr(hist, torch.int32, (s.E,), "hist"), _stream(stream)), "moegps_route_histogram")

    def route_prepare(self, x, w_router, bias, topk_idx, topk_w, hist, workspace, stream=None):
        s = self.shape
        if workspace is None or workspace.numel() * workspace.element_size() < workspace_bytes(s):
            raise MoegpsError(ERR_WORKSPACE_TOO_SMALL, "moegps_route_prepare")
        self._check(_lib().moegps_route_prepare(
            self._h, _ptr(x, torch.bfloat16, (s.T, s.D), "x"),
            _ptr(w_router, torch.bfloat16, (s.E, s.D), "w_router"),
            _ptr(bias, torch.float32, (s.E,), "bias", allow_none=True),
            _ptr(topk_idx, torch.int32, (s.T, s.K), "topk_idx"),
            _ptr(topk_w, torch.float32, (s.T, s.K), "topk_w"),
            _ptr(hist, torch.int32, (s.E,), "hist"),
            _ptr(workspace, workspace.dtype, None, "workspace"), _stream(stream)), "moegps_route_prepare")

    def dispatch_prepared(self, x, topk_idx, hist, replicas, slot_off, slot_row_off, row_pair, pair_row, xp,
                          workspace, stream=None):
        s = self.shape
        if workspace is None or workspace.numel() * workspace.element_size() < workspace_bytes(s):
            raise MoegpsError(ERR_WORKSPACE_TOO_SMALL, "moegps_dispatch_prepared")
        self._check(_lib().moegps_dispatch_prepared(
            self._h, _ptr(x, torch.bfloat16, (s.T, s.D), "x"),
            _ptr(topk_idx, torch.int32, (s.T, s.K), "topk_idx"),
            _ptr(hist, torch.int32, (s.E,), "hist"),
            _ptr(replicas, torch.int32, (s.E,), "replicas"),
            _ptr(slot_off, torch.int32, (s.E + 1,), "slot_off"),
            _ptr(slot_row_off, torch.int32, (s.S + 1,), "slot_row_off"),
            _ptr(row_pair, torch.int32, (s.Rcap,), "row_pair"),
            _ptr(pair_row, torch.int32, (s.T, s.K), "pair_row"),
            _ptr(xp, torch.bfloat16, (s.Rcap, s.D), "xp"),
            _ptr(workspace, workspace.dtype, None, "workspace"), _stream(stream)), "moegps_dispatch_prepared")

    def route_logits(self, x, w_router, bias, logits, stream=None):
        s = self.shape
        self._check(_lib().moegps_route_logits(
            self._h, _ptr(x, torch.bfloat16, (s.T, s.D), "x"),
            _ptr(w_router, torch.bfloat16, (s.E, s.D), "w_router"),
            _ptr(bias, torch.float32, (s.E,), "bias", allow_none=True),
            _ptr(logits, torch.float32, (s.T, s.E), "logits"), _stream(stream)), "moegps_route_logits")

    def histogram(self, topk_idx, hist, stream=None):
        s = self.shape
        self._check(_lib().moegps_histogram(
            self._h, _ptr(topk_idx, torch.int32, (s.T, s.K), "topk_idx"),
            _ptr(hist, torch.int32, (s.E,), "hist"), _stream(stream)), "moegps_histogram")

    def plan(self, predicted_hist, n_slots, replicas, slot_off, slot_expert, bound, stream=None):
        s = self.shape
        self._check(_lib().moegps_plan(
            self._h, _ptr(predicted_hist, torch.int32, (s.E,), "predicted_hist"), int(n_slots),
            _ptr(replicas, torch.int32, (s.E,), "replicas"),
            _ptr(slot_off, torch.int32, (s.E + 1,), "slot_off"),
            _ptr(slot_expert, torch.int32, (s.S,), "slot_expert"),
            _ptr(bound, torch.int32, (1,), "bound"), _stream(stream)), "moegps_plan")

    def pack(self, predicted_hist, home, capacity, n_devices, placement, share, load, iterations, stream=None):
        s, g = self.shape, int(n_devices)
        self._check(_lib().moegps_pack(
            self._h, _ptr(predicted_hist, torch.int32, (s.E,), "predicted_hist"),
            _ptr(home, torch.int32, (s.E,), "home"), _ptr(capacity, torch.int32, (g,), "capacity"), g,
            _ptr(placement, torch.int32, (s.E, g), "placement"), _ptr(share, torch.int32, (s.E, g), "share"),
            _ptr(load, torch.int32, (g,), "load"), _ptr(iterations, torch.int32, (1,), "iterations"),
            _stream(stream)), "moegps_pack")

    def pack_slots(self, placement, share, n_devices, replicas, slot_off, slot_expert, slot_share, slot_device,
                   stream=None):
        s, g = self.shape, int(n_devices)
        self._check(_lib().moegps_pack_slots(
            self._h, _ptr(placement, torch.int32, (s.E, g), "placement"), _ptr(share, torch.int32, (s.E, g), "share"), g,
            _ptr(replicas, torch.int32, (s.E,), "replicas"), _ptr(slot_off, torch.int32, (s.E + 1,), "slot_off"),
            _ptr(slot_expert, torch.int32, (s.S,), "slot_expert"), _ptr(slot_share, torch.int32, (s.S,), "slot_share"),
            _ptr(slot_device, torch.int32, (s.S,), "slot_device"), _stream(stream)), "moegps_pack_slots")

    def dispatch_shares(self, x, topk_idx, hist, replicas, slot_off, slot_share, slot_row_off, row_pair, pair_row,
                        xp, workspace, stream=None):
        s = self.shape
        if workspace is None or workspace.numel() * workspace.element_size() < workspace_bytes(s):
            raise MoegpsError(ERR_WORKSPACE_TOO_SMALL, "moegps_dispatch_shares")
        self._check(_lib().moegps_dispatch_shares(
            self._h, _ptr(x, torch.bfloat16, (s.T, s.D), "x"),
            _ptr(topk_idx, torch.int32, (s.T, s.K), "topk_idx"),
            _ptr(hist, torch.int32, (s.E,), "hist"),
            _ptr(replicas, torch.int32, (s.E,), "replicas"),
            _ptr(slot_off, torch.int32, (s.E + 1,), "slot_off"),
            _ptr(slot_share, torch.int32, (s.S,), "slot_share"),
            _ptr(slot_row_off, torch.int32, (s.S + 1,), "slot_row_off"),
            _ptr(row_pair, torch.int32, (s.Rcap,), "row_pair"),
            _ptr(pair_row, torch.int32, (s.T, s.K), "pair_row"),
            _ptr(xp, torch.bfloat16, (s.Rcap, s.D), "xp"),
            _ptr(workspace, workspace.dtype, None, "workspace"), _stream(stream)), "moegps_dispatch_shares")

    def dispatch(self, x, topk_idx, hist, replicas, slot_off, slot_row_off, row_pair, pair_row, xp,
                 workspace, stream=None):
        s = self.shape
        if workspace is None or workspace.numel() * workspace.element_size() < workspace_bytes(s):
            raise MoegpsError(ERR_WORKSPACE_TOO_SMALL, "moegps_dispatch")
        self._check(_lib().moegps_dispatch(
            self._h, _ptr(x, torch.bfloat16, (s.T, s.D), "x"),
            _ptr(topk_idx, torch.int32, (s.T, s.K), "topk_idx"),
            _ptr(hist, torch.int32, (s.E,), "hist"),
            _ptr(replicas, torch.int32, (s.E,), "replicas"),
            _ptr(slot_off, torch.int32, (s.E + 1,), "slot_off"),
            _ptr(slot_row_off, torch.int32, (s.S + 1,), "slot_row_off"),
            _ptr(row_pair, torch.int32, (s.Rcap,), "row_pair"),
            _ptr(pair_row, torch.int32, (s.T, s.K), "pair_row"),
            _ptr(xp, torch.bfloat16, (s.Rcap, s.D), "xp"),
            _ptr(workspace, workspace.dtype, None, "workspace"), _stream(stream)), "moegps_dispatch")

    def dispatch_static(self, x, topk_idx, hist, replicas, slot_off, slot_row_off, row_pair, pair_row, xp,
                        stream=None):
        """dispatch() for callers that cannot hand over a workspace (no allocator available where
        they run): the scratch is a fixed 1 MiB array inside the library, shared by every call on
        the device, so overlapping calls must be serialised; ceil(T*K/256)*E must be <= 262144.
        This method allocates nothing either."""
        s = self.shape
        self._check(_lib().moegps_dispatch_static(
            self._h, _ptr(x, torch.bfloat16, (s.T, s.D), "x"),
            _ptr(topk_idx, torch.int32, (s.T, s.K), "topk_idx"),
            _ptr(hist, torch.int32, (s.E,), "hist"),
            _ptr(replicas, torch.int32, (s.E,), "replicas"),
            _ptr(slot_off, torch.int32, (s.E + 1,), "slot_off"),
            _ptr(slot_row_off, torch.int32, (s.S + 1,), "slot_row_off"),
            _ptr(row_pair, torch.int32, (s.Rcap,), "row_pair"),
            _ptr(pair_row, torch.int32, (s.T, s.K), "pair_row"),
            _ptr(xp, torch.bfloat16, (s.Rcap, s.D), "xp"), _stream(stream)), "moegps_dispatch_static")

    def expert_ffn(self, xp, slot_row_off, slot_expert, w_gate, w_up, w_down, h_ws, yp, stream=None):
        s = self.shape
        self._check(_lib().moegps_expert_ffn(
            self._h, _ptr(xp, torch.bfloat16, (s.Rcap, s.D), "xp"),
            _ptr(slot_row_off, torch.int32, (s.S + 1,), "slot_row_off"),
            _ptr(slot_expert, torch.int32, (s.S,), "slot_expert"),
            _ptr(w_gate, torch.bfloat16, (s.E, s.F, s.D), "w_gate"),
            _ptr(w_up, torch.bfloat16, (s.E, s.F, s.D), "w_up"),
            _ptr(w_down, torch.bfloat16, (s.E, s.D, s.F), "w_down"),
            _ptr(h_ws, torch.bfloat16, (s.Rcap, s.F), "h_ws"),
            _ptr(yp, torch.bfloat16, (s.Rcap, s.D), "yp"), _stream(stream)), "moegps_expert_ffn")

    def expert_ffn_gate_up(self, xp, slot_row_off, slot_expert, w_gate, w_up, h_ws, stream=None):
        s = self.shape
        self._check(_lib().moegps_expert_ffn_gate_up(
            self._h, _ptr(xp, torch.bfloat16, (s.Rcap, s.D), "xp"),
            _ptr(slot_row_off, torch.int32, (s.S + 1,), "slot_row_off"),
            _ptr(slot_expert, torch.int32, (s.S,), "slot_expert"),
            _ptr(w_gate, torch.bfloat16, (s.E, s.F, s.D), "w_gate"),
            _ptr(w_up, torch.bfloat16, (s.E, s.F, s.D), "w_up"),
            _ptr(h_ws, torch.bfloat16, (s.Rcap, s.F), "h_ws"), _stream(stream)), "moegps_expert_ffn_gate_up")

    def expert_ffn_down(self, h_ws, slot_row_off, slot_expert, w_down, yp, stream=None):
        s = self.shape
        self._check(_lib().moegps_expert_ffn_down(
            self._h, _ptr(h_ws, torch.bfloat16, (s.Rcap, s.F), "h_ws"),
            _ptr(slot_row_off, torch.int32, (s.S + 1,), "slot_row_off"),
            _ptr(slot_expert, torch.int32, (s.S,), "slot_expert"),
            _ptr(w_down, torch.bfloat16, (s.E, s.D, s.F), "w_down"),
            _ptr(yp, torch.bfloat16, (s.Rcap, s.D), "yp"), _stream(stream)), "moegps_expert_ffn_down")

    def combine(self, yp, pair_row, topk_w, out, stream=None):
        s = self.shape
        self._check(_lib().moegps_combine(
            self._h, _ptr(yp, torch.bfloat16, (s.Rcap, s.D), "yp"),
            _ptr(pair_row, torch.int32, (s.T, s.K), "pair_row"),
            _ptr(topk_w, torch.float32, (s.T, s.K), "topk_w"),
            _ptr(out, torch.bfloat16, (s.T, s.D), "out"), _stream(stream)), "moegps_combine")

    def predictor_update(self, hist, state, predicted_hist, stream=None):
        s = self.shape
        self._check(_lib().moegps_predictor_update(
            self._h, _ptr(hist, torch.int32, (s.E,), "hist"), _ptr(state, torch.int64, (s.E,), "state"),
            _ptr(predicted_hist, torch.int32, (s.E,), "predicted_hist"), _stream(stream)),
            "moegps_predictor_update")

    def predictor_update_ema(self, hist, state, shift, predicted_hist, stream=None):
        s = self.shape
        self._check(_lib().moegps_predictor_update_ema(
            self._h, _ptr(hist, torch.int32, (s.E,), "hist"), _ptr(state, torch.int64, (s.E,), "state"), int(shift),
            _ptr(predicted_hist, torch.int32, (s.E,), "predicted_hist"), _stream(stream)),
            "moegps_predictor_update_ema")

    def error_rate(self, predicted_hist, hist, error_rate, stream=None):
        s = self.shape
        self._check(_lib().moegps_error_rate(
            self._h, _ptr(predicted_hist, torch.int32, (s.E,), "predicted_hist"),
            _ptr(hist, torch.int32, (s.E,), "hist"), _ptr(error_rate, torch.float64, (1,), "error_rate"),
            _stream(stream)), "moegps_error_rate")

    def selftest_bounded_wait(self, limit_cycles: int = 2_000_000, stream=None):
        """Launches a kernel whose wait can never be satisfied; status() then reports ERR_TIMEOUT."""
        self._check(_lib().moegps_selftest_bounded_wait(self._h, int(limit_cycles), _stream(stream)),
                    "moegps_selftest_bounded_wait")

    # -- bookkeeping --------------------------------------------------------------------------
    def status(self, stream=None) -> int:
        """Synchronises the stream and returns (and clears) the device status word."""
        h = ctypes.c_int32(0)
        self._check(_lib().moegps_status(self._h, _stream(stream), ctypes.byref(h)), "moegps_status")
        return int(h.value)

    def check_status(self, stream=None):
        st = self.status(stream)
        if st != OK:
            raise MoegpsError(st, "device status")

    def launch_count(self) -> int:
        return int(_lib().moegps_launch_count(self._h))


def rcap(shape: Shape) -> int:
    cs = shape.c_struct()
    return int(_lib().moegps_rcap(ctypes.byref(cs)))


def workspace_bytes(shape: Shape) -> int:
    cs = shape.c_struct()
    return int(_lib().moegps_workspace_bytes(ctypes.byref(cs)))


def error_string(code: int) -> str:
    return _lib().moegps_error_string(int(code)).decode()
