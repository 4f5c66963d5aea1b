"""CPU oracle of the Virtual-Expert MoE-layer forward (test infrastructure only).

Thin ctypes wrapper around ``swapmoe_oracle.c`` (plain C, double precision).
Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA product never does.  Nothing here imports the CUDA package's
kernels or binding either.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "swapmoe_oracle.c")
_LIB = os.path.join(_HERE, "libswapmoe_oracle.so")
_lib = None

ACT_RELU = 0
ACT_SWIGLU = 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP) into a shared object beside its source."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_num_threads.restype = ctypes.c_int
        _lib.oracle_gate.restype = ctypes.c_int
        _lib.oracle_invert_slot_table.restype = ctypes.c_int
        _lib.oracle_remap.restype = ctypes.c_int
        _lib.oracle_forward.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


def _i32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.int32)


def _f64(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float64)


def logits(x, Wr):
    x, Wr = _f32(x), _f32(Wr)
    T, d = x.shape
    E = Wr.shape[0]
    out = np.empty((T, E), dtype=np.float64)
    lib().oracle_logits(_p(x), _p(Wr), T, d, E, _p(out))
    return out


def gate(logits_, k, renorm, allowed=None):
    l = _f64(logits_)
    T, E = l.shape
    idx = np.empty((T, k), dtype=np.int32)
    g = np.empty((T, k), dtype=np.float64)
    al = _i32(allowed)
    rc = lib().oracle_gate(_p(l), T, E, int(k), int(renorm), _p(al), _p(idx), _p(g))
    if rc != 0:
        raise ValueError("fewer than k experts allowed")
    return idx, g


def invert_slot_table(slot_to_expert, E):
    s2e = _i32(slot_to_expert)
    e2s = np.empty(E, dtype=np.int32)
    rc = lib().oracle_invert_slot_table(_p(s2e), len(s2e), int(E), _p(e2s))
    if rc != 0:
        raise ValueError("bad slot table")
    return e2s


def permute(slot, K):
    s = _i32(slot).reshape(-1)
    n = s.size
    count = np.empty(K, dtype=np.int32)
    offset = np.empty(K + 1, dtype=np.int32)
    perm = np.empty(n, dtype=np.int32)
    inv = np.empty(n, dtype=np.int32)
    lib().oracle_permute(_p(s), n, int(K), _p(count), _p(offset), _p(perm), _p(inv))
    return count, offset, perm, inv


def importance(x, uidx, ugate, enorm, imp=None):
    x = _f32(x)
    T, d = x.shape
    uidx = _i32(uidx)
    k = uidx.shape[1]
    enorm = _f32(enorm)
    imp = np.zeros(enorm.size, dtype=np.float64) if imp is None else _f64(imp).copy()
    lib().oracle_importance(_p(x), T, d, k, _p(uidx), _p(_f64(ugate)), _p(enorm), _p(imp))
    return imp


def importance_count(uidx, E, imp=None):
    uidx = _i32(uidx)
    T, k = uidx.shape
    imp = np.zeros(E, dtype=np.float64) if imp is None else _f64(imp).copy()
    lib().oracle_importance_count(T, k, _p(uidx), _p(imp))
    return imp


def topk_importance(imp, K):
    imp = _f64(imp)
    out = np.empty(K, dtype=np.int32)
    lib().oracle_topk_importance(_p(imp), imp.size, int(K), _p(out))
    return out


def expert_hidden(x, slot, phys_slot, arena_in, *, k, act, token_subset=None):
    """h[p, :] = act(W_in[slot[p]] x[p // k]) for every pair p in flat (token, j) order; rows of
    tokens outside ``token_subset`` stay zero."""
    x, arena_in = _f32(x), _f32(arena_in)
    T, d = x.shape
    f = arena_in.shape[2]
    slot, phys = _i32(slot).reshape(-1), _i32(phys_slot)
    sub = _i32(token_subset)
    h = np.zeros((T * k, f), np.float64)
    lib().oracle_expert_hidden(_p(x), T, d, f, int(k), int(act), _p(slot), _p(phys), _p(arena_in),
                               _p(sub), 0 if sub is None else sub.size, _p(h))
    return h


def forward(x, Wr, enorm, slot_to_expert, arena_in, arena_out, *, k, act, renorm,
            phys_slot=None, ext_logits=None, token_subset=None, imp=None, want_y=False):
    """Run the whole layer; returns a dict of every intermediate and the output.

    ``arena_in`` [P, nin, f, d] and ``arena_out`` [P, d, f] hold the resident experts;
    ``ext_logits`` (float32 [T, E]) replaces the router product when given;
    ``token_subset`` limits the FFN/combine to the listed tokens (other rows of
    ``out`` are left as zeros) - routing and importance always cover all tokens.
    """
    x, Wr, enorm = _f32(x), _f32(Wr), _f32(enorm)
    arena_in, arena_out = _f32(arena_in), _f32(arena_out)
    T, d = x.shape
    E = Wr.shape[0]
    s2e = _i32(slot_to_expert)
    K = s2e.size
    f = arena_out.shape[2]
    phys = _i32(np.arange(K) if phys_slot is None else phys_slot)
    ext = _f32(ext_logits)
    sub = _i32(token_subset)
    n = T * k
    r = {
        "logits": np.zeros((T, E), np.float64),
        "uidx": np.zeros((T, k), np.int32), "ugate": np.zeros((T, k), np.float64),
        "midx": np.zeros((T, k), np.int32), "mgate": np.zeros((T, k), np.float64),
        "slot": np.zeros((T, k), np.int32),
        "count": np.zeros(K, np.int32), "offset": np.zeros(K + 1, np.int32),
        "perm": np.zeros(n, np.int32), "inv": np.zeros(n, np.int32),
        "out": np.zeros((T, d), np.float64),
        "imp": np.zeros(E, np.float64) if imp is None else _f64(imp).copy(),
    }
    y = np.zeros((n, d), np.float64) if want_y else None
    rc = lib().oracle_forward(
        _p(x), _p(Wr), _p(ext), _p(enorm), _p(s2e), _p(phys), _p(arena_in), _p(arena_out),
        T, d, f, E, int(k), K, int(act), int(renorm), _p(sub), 0 if sub is None else sub.size,
        _p(r["logits"]), _p(r["uidx"]), _p(r["ugate"]), _p(r["midx"]), _p(r["mgate"]),
        _p(r["slot"]), _p(r["count"]), _p(r["offset"]), _p(r["perm"]), _p(r["inv"]),
        _p(y), _p(r["out"]), _p(r["imp"]))
    if rc != 0:
        raise ValueError("oracle_forward: invalid slot table or K < top_k")
    if want_y:
        r["y"] = y
    return r
