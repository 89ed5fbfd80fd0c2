"""LASER routing oracle -- TEST INFRASTRUCTURE, not a product path.

Thin ctypes access to ``laser_oracle.c`` (plain C, compiled with gcc) plus two
pure-Python restatements used as cross-checks on tiny inputs
(``oracle.alg1_literal``).  Nothing here imports, links or calls the CUDA
library; only tests, the smoke check and the benchmark's CPU-baseline leg may
import this package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "laser_oracle.c")
_LIB = os.path.join(_HERE, "liblaser_oracle.so")

_GCC_FLAGS = ["-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
              "-shared", "-fPIC"]


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc if the shared object is missing or stale."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", *_GCC_FLAGS, "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        i32, i64, f32 = ctypes.c_int32, ctypes.c_int64, ctypes.c_float
        vp = ctypes.c_void_p
        L.lo_logits.argtypes = [vp, i64, vp, i64, vp, i32, i32, i32, vp]
        L.lo_logits.restype = None
        L.lo_exp32.argtypes = [f32]
        L.lo_exp32.restype = f32
        L.lo_softmax.argtypes = [vp, i32, vp]
        L.lo_softmax.restype = None
        L.lo_route.argtypes = [vp, i32, i32, i32, i32, f32, f32, i32, vp, vp, vp, vp]
        L.lo_route.restype = i32
        L.lo_route_relaxed.argtypes = [vp, i32, i32, i32, i32, f32, f32, i32, i32, vp, vp, vp, vp]
        L.lo_route_relaxed.restype = i32
        L.lo_philox4x32_10.argtypes = [vp, vp, vp]
        L.lo_philox4x32_10.restype = None
        L.lo_route_random.argtypes = [vp, i32, i32, i32, i32, f32, f32, i32, ctypes.c_uint64, i32,
                                      vp, vp, vp, vp, vp]
        L.lo_route_random.restype = i32
        L.lo_topk.argtypes = [vp, i32, i32, i32, vp]
        L.lo_topk.restype = None
        L.lo_dispatch.argtypes = [vp, i32, i32, i32, vp, vp]
        L.lo_dispatch.restype = None
        L.lo_bins.argtypes = [vp, vp, i32, vp]
        L.lo_bins.restype = None
        _lib = L
    return _lib


def _p(a: np.ndarray) -> ctypes.c_void_p:
    return ctypes.c_void_p(a.ctypes.data)


def _c(a, dtype) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dtype)


def logits(hidden_bits: np.ndarray, wg_bits: np.ndarray, bias=None) -> np.ndarray:
    """x = h W^T + b from bf16 bit patterns (uint16 arrays [T,d], [E,d])."""
    h = _c(hidden_bits, np.uint16)
    w = _c(wg_bits, np.uint16)
    T, d = h.shape
    E, d2 = w.shape
    assert d == d2
    b = None if bias is None else _c(bias, np.float32)
    x = np.empty((T, E), np.float32)
    lib().lo_logits(_p(h), d, _p(w), d, _p(b) if b is not None else None, T, d, E, _p(x))
    return x


def exp32(y: float) -> np.float32:
    return np.float32(lib().lo_exp32(ctypes.c_float(float(y))))


def softmax(x: np.ndarray) -> np.ndarray:
    """Row-wise fp32 softmax with the oracle's fixed arithmetic; x: [T,E] or [E]."""
    x2 = _c(np.atleast_2d(x), np.float32)
    s = np.empty_like(x2)
    for t in range(x2.shape[0]):
        lib().lo_softmax(_p(x2[t]), x2.shape[1], _p(s[t]))
    return s.reshape(np.shape(x))


def route(x: np.ndarray, loads: np.ndarray, k: int, c: int, eps_high: float, t_fix: float,
          renormalize: bool = True):
    """Sequential LASER routing from fp32 logits.

    Returns (expert_ids [T,k] int32, weights [T,k] float32, loads_out [E] int32,
    cstar [T] int32 with 0 = top-k branch).  ``loads`` is not modified.
    """
    x = _c(x, np.float32)
    T, E = x.shape
    L = _c(loads, np.int32).copy()
    ids = np.empty((T, k), np.int32)
    w = np.empty((T, k), np.float32)
    cs = np.empty((T,), np.int32)
    rc = lib().lo_route(_p(x), T, E, k, c, eps_high, t_fix, int(bool(renormalize)),
                        _p(L), _p(ids), _p(w), _p(cs))
    if rc != 0:
        raise ValueError("lo_route rejected its arguments")
    return ids, w, L, cs


def route_relaxed(x: np.ndarray, loads: np.ndarray, k: int, c: int, eps_high: float,
                  t_fix: float, granularity: int, renormalize: bool = True):
    """The RELAXED load update (not the method's rule): a token sees the loads as they stood
    at the start of its chunk of ``granularity`` tokens (0 = one snapshot per call).  Same
    return values as ``route``; ``granularity = 1`` is ``route``."""
    x = _c(x, np.float32)
    T, E = x.shape
    L = _c(loads, np.int32).copy()
    ids = np.empty((T, k), np.int32)
    w = np.empty((T, k), np.float32)
    cs = np.empty((T,), np.int32)
    rc = lib().lo_route_relaxed(_p(x), T, E, k, c, eps_high, t_fix, int(bool(renormalize)),
                                int(granularity), _p(L), _p(ids), _p(w), _p(cs))
    if rc != 0:
        raise ValueError("lo_route_relaxed rejected its arguments")
    return ids, w, L, cs


def philox4x32_10(counter, key) -> np.ndarray:
    """Four 32-bit words of Philox4x32-10 for a 4-word counter and a 2-word key."""
    ctr = _c(counter, np.uint32)
    ky = _c(key, np.uint32)
    out = np.empty(4, np.uint32)
    lib().lo_philox4x32_10(_p(ctr), _p(ky), _p(out))
    return out


def route_random(x: np.ndarray, loads: np.ndarray, k: int, c: int, eps_high: float, t_fix: float,
                 seed: int, layer: int = 0, renormalize: bool = True):
    """Routing with RANDOM trimming (the pool is sampled down to c* candidates with Philox).
    Returns (expert_ids, weights, loads_out, cstar, cand [T,c] with -1 for unused)."""
    x = _c(x, np.float32)
    T, E = x.shape
    L = _c(loads, np.int32).copy()
    ids = np.empty((T, k), np.int32)
    w = np.empty((T, k), np.float32)
    cs = np.empty((T,), np.int32)
    cand = np.empty((T, c), np.int32)
    rc = lib().lo_route_random(_p(x), T, E, k, c, eps_high, t_fix, int(bool(renormalize)),
                               ctypes.c_uint64(int(seed)), int(layer), _p(L), _p(ids), _p(w), _p(cs),
                               _p(cand))
    if rc != 0:
        raise ValueError("lo_route_random rejected its arguments")
    return ids, w, L, cs, cand


def topk(x: np.ndarray, k: int) -> np.ndarray:
    x = _c(x, np.float32)
    T, E = x.shape
    ids = np.empty((T, k), np.int32)
    lib().lo_topk(_p(x), T, E, k, _p(ids))
    return ids


def dispatch(ids: np.ndarray, E: int):
    """(offsets [E+1], perm [T*k]) of the stable grouping of pair ids by expert."""
    ids = _c(ids, np.int32)
    T, k = ids.shape
    offsets = np.empty((E + 1,), np.int32)
    perm = np.empty((T * k,), np.int32)
    lib().lo_dispatch(_p(ids), T, k, E, _p(offsets), _p(perm))
    return offsets, perm


def bins(counts: np.ndarray, expert_to_bin: np.ndarray, bin_loads: np.ndarray) -> np.ndarray:
    counts = _c(counts, np.int32)
    e2b = _c(expert_to_bin, np.int32)
    out = _c(bin_loads, np.int32).copy()
    lib().lo_bins(_p(counts), _p(e2b), counts.shape[0], _p(out))
    return out


def route_full(hidden_bits, wg_bits, bias, loads, expert_to_bin, bin_loads,
               k, c, eps_high, t_fix, renormalize=True, x=None, granularity=1,
               random_seed=None, layer=0):
    """Whole path: logits (unless given) -> routing -> dispatch -> bins.  Dict of arrays.
    ``granularity != 1`` selects the relaxed load update of ``route_relaxed``; ``random_seed``
    selects RANDOM trimming (``route_random``) for layer index ``layer``."""
    if x is None:
        x = logits(hidden_bits, wg_bits, bias)
    E = x.shape[1]
    if random_seed is not None:
        assert granularity == 1
        ids, w, L, cs, _ = route_random(x, loads, k, c, eps_high, t_fix, random_seed, layer,
                                        renormalize)
    elif granularity == 1:
        ids, w, L, cs = route(x, loads, k, c, eps_high, t_fix, renormalize)
    else:
        ids, w, L, cs = route_relaxed(x, loads, k, c, eps_high, t_fix, granularity, renormalize)
    offsets, perm = dispatch(ids, E)
    counts = (L - np.asarray(loads, np.int32)).astype(np.int32)
    out = dict(logits=x, expert_ids=ids, weights=w, loads=L, cstar=cs,
               offsets=offsets, perm=perm, counts=counts)
    if expert_to_bin is not None and bin_loads is not None:
        out["bin_loads"] = bins(counts, expert_to_bin, bin_loads)
    return out
