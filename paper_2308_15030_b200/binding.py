"""ctypes binding of libswapmoe.so: argument marshalling only.

Every step of the layer runs inside the library's CUDA kernels; this module turns
torch tensors / numpy arrays into the plain pointers and sizes of the C ABI
(include/swapmoe.h) and raises on a non-zero status.  There is no fallback: if
the library cannot be loaded the import of :func:`lib` raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np

from . import build as _build

F32, BF16 = 0, 1
N_STAGES = 6
# stage 1 has had no kernel of its own since the scan moved into the permute kernel: its slot measures an empty interval
STAGE_NAMES = ("router_gate", "(scan: no kernel of its own)", "scan_permute_gather", "gemm1_act", "gemm2", "combine")
ACT_RELU, ACT_SWIGLU = 0, 1

TAPS = {
    "logits": (0, np.float32), "uidx": (1, np.int32), "ugate": (2, np.float32),
    "midx": (3, np.int32), "mgate": (4, np.float32), "slot": (5, np.int32),
    "count": (6, np.int32), "offset": (7, np.int32), "perm": (8, np.int32),
    "inv": (9, np.int32), "xnorm": (10, np.float32),
    "h": (11, None), "y": (12, np.float32),       # h comes in the layer's dtype (bf16 as uint16 bit patterns)
}

EXPORTS = [
    "swapmoe_create", "swapmoe_destroy", "swapmoe_set_router", "swapmoe_set_resident",
    "swapmoe_forward", "swapmoe_forward_timed", "swapmoe_debug_rerun_gemm", "swapmoe_forward_from_logits", "swapmoe_forward_host",
    "swapmoe_forward_host_async", "swapmoe_host_wait",
    "swapmoe_read_importance", "swapmoe_read_importance_kind", "swapmoe_topk_importance", "swapmoe_load_slot_async",
    "swapmoe_debug_copy", "swapmoe_device_status", "swapmoe_launch_count",
    "swapmoe_workspace_bytes", "swapmoe_set_gemm_path", "swapmoe_status_string",
    "swapmoe_route_static", "swapmoe_selftest_bounded_wait", "swapmoe_read_touched_slots",
    "swapmoe_read_scores_async", "swapmoe_read_decode_prefetch",
]


class SwapMoEError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__("%s: %s (%d)" % (where, status_string(status), status))


class Config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("E", "d_model", "d_ff", "top_k", "K", "dtype", "act", "renorm_topk",
                 "max_tokens", "spare_slots")]


_lib = None


def lib() -> ctypes.CDLL:
    """Loads (building if needed) the CUDA library; raises if that fails."""
    global _lib
    if _lib is None:
        path = os.environ.get("SWAPMOE_LIB")      # explicit library file, e.g. an instrumented build
        if not path:
            path = _build.LIB if os.path.exists(_build.LIB) and os.environ.get("SWAPMOE_NO_REBUILD") \
                else _build.build()
        L = ctypes.CDLL(path)
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
        L.swapmoe_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(Config)]
        L.swapmoe_destroy.argtypes = [vp]
        L.swapmoe_set_router.argtypes = [vp, vp, vp, vp]
        L.swapmoe_set_resident.argtypes = [vp, vp, vp, vp, vp, vp]
        L.swapmoe_forward.argtypes = [vp, vp, vp, i32, vp]
        L.swapmoe_forward_timed.argtypes = [vp, vp, vp, i32, vp, ctypes.POINTER(vp)]
        L.swapmoe_debug_rerun_gemm.argtypes = [vp, vp, i32, vp]
        L.swapmoe_forward_from_logits.argtypes = [vp, vp, vp, vp, i32, vp]
        L.swapmoe_forward_host.argtypes = [vp, vp, vp, i32, vp]
        L.swapmoe_forward_host_async.argtypes = [vp, vp, vp, i32, vp]
        L.swapmoe_host_wait.argtypes = [vp]
        L.swapmoe_read_importance.argtypes = [vp, vp, i32, vp]
        L.swapmoe_read_importance_kind.argtypes = [vp, i32, vp, i32, vp]
        L.swapmoe_topk_importance.argtypes = [vp, i32, i32, vp]
        L.swapmoe_load_slot_async.argtypes = [vp, i32, vp, vp, vp, vp, vp]
        L.swapmoe_debug_copy.argtypes = [vp, i32, vp, ctypes.c_size_t, vp]
        L.swapmoe_device_status.argtypes = [vp, vp, vp]
        L.swapmoe_launch_count.argtypes = [vp]
        L.swapmoe_launch_count.restype = i64
        L.swapmoe_workspace_bytes.argtypes = [vp]
        L.swapmoe_workspace_bytes.restype = i64
        L.swapmoe_set_gemm_path.argtypes = [vp, i32]
        L.swapmoe_route_static.argtypes = [vp] * 4 + [i32] * 7 + [vp] * 11
        L.swapmoe_selftest_bounded_wait.argtypes = [vp, i32, vp]
        L.swapmoe_read_touched_slots.argtypes = [vp, vp, i32, vp]
        L.swapmoe_read_scores_async.argtypes = [vp, i32, vp, i32, vp]
        L.swapmoe_read_decode_prefetch.argtypes = [vp, vp, vp, i32, vp]
        L.swapmoe_status_string.argtypes = [i32]
        L.swapmoe_status_string.restype = ctypes.c_char_p
        for n in EXPORTS:
            if n not in ("swapmoe_launch_count", "swapmoe_workspace_bytes", "swapmoe_status_string"):
                getattr(L, n).restype = i32
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().swapmoe_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != 0:
        raise SwapMoEError(status, where)


def _np_ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def topk_importance(imp: np.ndarray, K: int) -> np.ndarray:
    imp = np.ascontiguousarray(imp, dtype=np.float32)
    out = np.empty(int(K), dtype=np.int32)
    _check(lib().swapmoe_topk_importance(_np_ptr(imp), imp.size, int(K), _np_ptr(out)),
           "swapmoe_topk_importance")
    return out


ROUTE_STATIC_MAX_TOKENS = 8192


def route_static(x, Wr, expert_to_slot, enorm, top_k: int, K: int, dtype: int, renorm_topk: int,
                 logits, uidx, ugate, midx, mgate, slot, xnorm, count, offset, imp, stream=None) -> None:
    """Router stage through the entry point that allocates nothing.

    For callers that may not allocate device memory (all tensors, outputs included,
    are the caller's; the library's scratch is a fixed array inside the library).
    Every argument is a CUDA torch tensor; ``imp`` is accumulated in place.
    """
    T, d = int(x.shape[0]), int(x.shape[1])
    E = int(Wr.shape[0])
    _check(lib().swapmoe_route_static(
        x.data_ptr(), Wr.data_ptr(), expert_to_slot.data_ptr(), enorm.data_ptr(), T, d, E, int(top_k),
        int(K), int(dtype), int(renorm_topk), logits.data_ptr(), uidx.data_ptr(), ugate.data_ptr(),
        midx.data_ptr(), mgate.data_ptr(), slot.data_ptr(), xnorm.data_ptr(), count.data_ptr(),
        offset.data_ptr(), imp.data_ptr(), _stream_ptr(stream)), "swapmoe_route_static")


class Layer:
    """One MoE layer served from K resident Virtual-Expert slots (thin handle)."""

    def __init__(self, E: int, d_model: int, d_ff: int, top_k: int, K: int, dtype: int,
                 act: int = ACT_RELU, renorm_topk: int = 0, max_tokens: int = 1,
                 spare_slots: int = 0):
        self.cfg = Config(E, d_model, d_ff, top_k, K, dtype, act, renorm_topk, max_tokens,
                          spare_slots)
        self._h = ctypes.c_void_p()
        _check(lib().swapmoe_create(ctypes.byref(self._h), ctypes.byref(self.cfg)), "swapmoe_create")
        self._keep = {}
        self.last_T = 0

    # -- lifetime
    def close(self) -> None:
        if self._h:
            lib().swapmoe_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- set-up
    def set_router(self, Wr, enorm: np.ndarray, stream=None) -> None:
        enorm = np.ascontiguousarray(enorm, dtype=np.float32)
        assert enorm.size == self.cfg.E
        self._keep["Wr"] = Wr
        _check(lib().swapmoe_set_router(self._h, Wr.data_ptr(), _np_ptr(enorm), _stream_ptr(stream)),
               "swapmoe_set_router")

    def set_resident(self, slot_to_expert: Sequence[int], arena_in, arena_out,
                     phys_slot: Optional[Sequence[int]] = None, stream=None) -> None:
        s2e = np.ascontiguousarray(slot_to_expert, dtype=np.int32)
        assert s2e.size == self.cfg.K
        ph = None if phys_slot is None else np.ascontiguousarray(phys_slot, dtype=np.int32)
        self._keep["arena_in"], self._keep["arena_out"] = arena_in, arena_out
        _check(lib().swapmoe_set_resident(self._h, _np_ptr(s2e), None if ph is None else _np_ptr(ph),
                                          arena_in.data_ptr(), arena_out.data_ptr(),
                                          _stream_ptr(stream)), "swapmoe_set_resident")

    def set_gemm_path(self, path: int) -> None:
        _check(lib().swapmoe_set_gemm_path(self._h, int(path)), "swapmoe_set_gemm_path")

    # -- hot path
    def forward(self, x, out, n_tokens: Optional[int] = None, stream=None) -> None:
        T = int(x.shape[0]) if n_tokens is None else int(n_tokens)
        self.last_T = T
        _check(lib().swapmoe_forward(self._h, x.data_ptr(), out.data_ptr(), T, _stream_ptr(stream)),
               "swapmoe_forward")

    def forward_timed(self, x, out, events, n_tokens: Optional[int] = None, stream=None) -> None:
        """Like forward, recording the N_STAGES + 1 torch.cuda.Event objects at stage boundaries."""
        T = int(x.shape[0]) if n_tokens is None else int(n_tokens)
        self.last_T = T
        assert len(events) == N_STAGES + 1
        for e in events:              # torch creates the CUDA event lazily, on its first record
            if not e.cuda_event:
                e.record()
        arr = (ctypes.c_void_p * (N_STAGES + 1))(*[e.cuda_event for e in events])
        _check(lib().swapmoe_forward_timed(self._h, x.data_ptr(), out.data_ptr(), T,
                                           _stream_ptr(stream), arr), "swapmoe_forward_timed")

    def rerun_gemm(self, out, which: int, stream=None) -> None:
        """Launches grouped GEMM-1 (which = 1) or GEMM-2 (2) again on the state the last forward left (timing aid)."""
        _check(lib().swapmoe_debug_rerun_gemm(self._h, out.data_ptr(), int(which), _stream_ptr(stream)),
               "swapmoe_debug_rerun_gemm")

    def forward_from_logits(self, x, logits, out, stream=None) -> None:
        T = int(x.shape[0])
        self.last_T = T
        _check(lib().swapmoe_forward_from_logits(self._h, x.data_ptr(), logits.data_ptr(),
                                                 out.data_ptr(), T, _stream_ptr(stream)),
               "swapmoe_forward_from_logits")

    def forward_host(self, x_host, out_host, n_tokens: Optional[int] = None, stream=None) -> None:
        """x_host/out_host: CPU torch tensors (pinned for speed) or numpy arrays."""
        T = int(x_host.shape[0]) if n_tokens is None else int(n_tokens)
        self.last_T = T
        xp = x_host.data_ptr() if hasattr(x_host, "data_ptr") else x_host.ctypes.data
        op = out_host.data_ptr() if hasattr(out_host, "data_ptr") else out_host.ctypes.data
        _check(lib().swapmoe_forward_host(self._h, xp, op, T, _stream_ptr(stream)),
               "swapmoe_forward_host")

    def forward_host_async(self, x_host, out_host, n_tokens: Optional[int] = None, stream=None) -> None:
        """Pipelined host path (pinned CPU tensors); out_host is valid after host_wait()."""
        T = int(x_host.shape[0]) if n_tokens is None else int(n_tokens)
        self.last_T = T
        _check(lib().swapmoe_forward_host_async(self._h, x_host.data_ptr(), out_host.data_ptr(), T,
                                                _stream_ptr(stream)), "swapmoe_forward_host_async")

    def host_wait(self) -> None:
        _check(lib().swapmoe_host_wait(self._h), "swapmoe_host_wait")

    # -- importance and swapping
    def read_importance(self, reset: bool = False, stream=None) -> np.ndarray:
        imp = np.empty(self.cfg.E, dtype=np.float32)
        _check(lib().swapmoe_read_importance(self._h, _np_ptr(imp), int(bool(reset)),
                                             _stream_ptr(stream)), "swapmoe_read_importance")
        return imp

    def read_scores_async(self, kinds: Sequence[str], out_pinned, reset: bool = False, stream=None) -> None:
        """Enqueues one small kernel that writes the scores named in `kinds` ("eq1", "count", "eq1_masked") into a
        pinned float32 tensor [3, E] (row 0 / 1 / 2 for the three scores); no wait - synchronise with the stream
        before reading it."""
        mask = sum(1 << {"eq1": 0, "count": 1, "eq1_masked": 2}[k] for k in kinds)
        assert out_pinned.is_pinned() and out_pinned.numel() >= 3 * self.cfg.E
        _check(lib().swapmoe_read_scores_async(self._h, mask, out_pinned.data_ptr(), int(bool(reset)),
                                               _stream_ptr(stream)), "swapmoe_read_scores_async")

    def read_decode_prefetch(self, reset: bool = False, stream=None):
        """(hits, touched): slots served by one-launch decode steps whose expert had been prefetched to L2, and all."""
        h, t = ctypes.c_int64(0), ctypes.c_int64(0)
        _check(lib().swapmoe_read_decode_prefetch(self._h, ctypes.byref(h), ctypes.byref(t), int(bool(reset)),
                                                  _stream_ptr(stream)), "swapmoe_read_decode_prefetch")
        return int(h.value), int(t.value)

    def read_touched_slots(self, reset: bool = False, stream=None) -> int:
        """Slots that received at least one pair, summed over the forwards since the last reset."""
        v = ctypes.c_int64(0)
        _check(lib().swapmoe_read_touched_slots(self._h, ctypes.byref(v), int(bool(reset)), _stream_ptr(stream)),
               "swapmoe_read_touched_slots")
        return int(v.value)

    def read_score(self, kind: str, reset: bool = False, stream=None) -> np.ndarray:
        """kind: "eq1" (Eq. 1, unmasked routing), "count" (token counts), "eq1_masked"."""
        k = {"eq1": 0, "count": 1, "eq1_masked": 2}[kind]
        out = np.empty(self.cfg.E, dtype=np.float32)
        _check(lib().swapmoe_read_importance_kind(self._h, k, _np_ptr(out), int(bool(reset)),
                                                  _stream_ptr(stream)), "swapmoe_read_importance_kind")
        return out

    def load_slot_async(self, phys: int, in_host_pinned, out_host_pinned, compute_stream, side_stream,
                        done_event=None) -> None:
        """The copy runs on side_stream behind everything enqueued so far on compute_stream."""
        if done_event is not None and not done_event.cuda_event:
            done_event.record(side_stream)      # torch creates the CUDA event on its first record
        ev = None if done_event is None else done_event.cuda_event
        _check(lib().swapmoe_load_slot_async(self._h, int(phys), in_host_pinned.data_ptr(),
                                             out_host_pinned.data_ptr(), _stream_ptr(compute_stream),
                                             _stream_ptr(side_stream), ev), "swapmoe_load_slot_async")

    # -- inspection
    def tap(self, name: str, stream=None) -> np.ndarray:
        which, dt = TAPS[name]
        c, T = self.cfg, self.last_T
        if dt is None:
            dt = np.uint16 if c.dtype == BF16 else np.float32
        shape = {"logits": (T, c.E), "count": (c.K,), "offset": (c.K + 1,), "perm": (T * c.top_k,),
                 "inv": (T * c.top_k,), "xnorm": (T,), "h": (T * c.top_k, c.d_ff),
                 "y": (T * c.top_k, c.d_model)}.get(name, (T, c.top_k))
        a = np.empty(shape, dtype=dt)
        _check(lib().swapmoe_debug_copy(self._h, which, _np_ptr(a), a.nbytes, _stream_ptr(stream)),
               "swapmoe_debug_copy")
        return a

    def device_status(self, stream=None):
        detail = ctypes.c_int32(0)
        st = lib().swapmoe_device_status(self._h, ctypes.byref(detail), _stream_ptr(stream))
        return int(st), int(detail.value)

    def selftest_bounded_wait(self, limit_ms: int = 20, stream=None) -> None:
        _check(lib().swapmoe_selftest_bounded_wait(self._h, int(limit_ms), _stream_ptr(stream)),
               "swapmoe_selftest_bounded_wait")

    @property
    def launch_count(self) -> int:
        return int(lib().swapmoe_launch_count(self._h))

    @property
    def workspace_bytes(self) -> int:
        return int(lib().swapmoe_workspace_bytes(self._h))
