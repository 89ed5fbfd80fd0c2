"""Python binding of the LASER routing C ABI (``include/laser.h``).

Argument marshalling only: every step of the routing path runs in the CUDA kernels of
``liblaser.so``.  torch is used for device memory and streams.  There is no fallback: if the
shared library has not been built, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblaser.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build the CUDA library first "
        "(python -c 'import __graft_entry__ as g; g.build()'); there is no CPU fallback")

_lib = ctypes.CDLL(LIB_PATH)

OK = 0
ERR_INVALID_ARG = -1
ERR_UNSUPPORTED = -2
ERR_WORKSPACE_TOO_SMALL = -3
ERR_MISALIGNED = -4
ERR_CUDA = -5
ERR_STATIC_SCRATCH = -6
STATIC_SCRATCH_BYTES = 4 * 1024 * 1024
DEV_LOAD_OVERFLOW = 1
DEV_TIMEOUT = 2
MAX_EXPERTS = 256
ROUTER_AUTO, ROUTER_TILE, ROUTER_SPLITK, ROUTER_TILE_ONESHOT = 0, 1, 2, 3

EXPORTS = ("laser_version", "laser_strerror", "laser_workspace_bytes", "laser_route",
           "laser_route_layers", "laser_route_layers_profiled", "laser_host_arena_bytes",
           "laser_route_host", "laser_route_static", "laser_imbalance",
           "laser_score_stats")
# include/laser_test_hooks.h: controls for the tests, not part of the routing interface
TEST_EXPORTS = ("laser_test_set_router", "laser_test_withhold_tile", "laser_test_launch_empty")


class LaserParams(ctypes.Structure):
    _fields_ = [("T", ctypes.c_int32), ("d", ctypes.c_int32), ("E", ctypes.c_int32),
                ("k", ctypes.c_int32), ("c", ctypes.c_int32),
                ("eps_high", ctypes.c_float), ("t_fix", ctypes.c_float),
                ("trim_mode", ctypes.c_int32), ("update_granularity", ctypes.c_int32),
                ("renormalize", ctypes.c_int32), ("n_bins", ctypes.c_int32),
                ("fresh_loads", ctypes.c_int32),
                ("ld_hidden", ctypes.c_int64), ("ld_w", ctypes.c_int64),
                ("seed", ctypes.c_uint64)]


_vp, _i32, _sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
_pp = ctypes.POINTER(LaserParams)
_lib.laser_version.restype = ctypes.c_int
_lib.laser_strerror.argtypes = [ctypes.c_int]
_lib.laser_strerror.restype = ctypes.c_char_p
_lib.laser_workspace_bytes.argtypes = [_pp, ctypes.POINTER(_sz)]
_lib.laser_workspace_bytes.restype = ctypes.c_int
_lib.laser_route.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _pp, _vp, _vp, _vp, _vp, _vp, _vp,
                             _vp, _sz, _vp]
_lib.laser_route.restype = ctypes.c_int
_lib.laser_route_layers.argtypes = [_i32, _vp, _vp, _vp, _vp, _vp, _vp, _pp, _vp, _vp,
                                    _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
_lib.laser_route_layers.restype = ctypes.c_int
_lib.laser_route_layers_profiled.argtypes = _lib.laser_route_layers.argtypes + [_vp]
_lib.laser_route_layers_profiled.restype = ctypes.c_int
_lib.laser_host_arena_bytes.argtypes = [_i32, _pp, ctypes.POINTER(_sz)]
_lib.laser_host_arena_bytes.restype = ctypes.c_int
_lib.laser_route_host.argtypes = [_i32, _vp, _vp, _vp, _vp, _vp, _vp, _pp, _vp, _vp,
                                  _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
_lib.laser_route_host.restype = ctypes.c_int
_lib.laser_route_static.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _pp, _vp, _vp, _vp, _vp, _vp,
                                    _vp, _vp]
_lib.laser_route_static.restype = ctypes.c_int


_lib.laser_imbalance.argtypes = [_i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.laser_imbalance.restype = ctypes.c_int


_lib.laser_score_stats.argtypes = [_i32, _i32, _i32, _i32, _vp, ctypes.c_float, _i32, _i32, _vp,
                                   _vp, _vp]
_lib.laser_score_stats.restype = ctypes.c_int
STATS_WORDS = 72
_lib.laser_test_set_router.argtypes = [ctypes.c_int]
_lib.laser_test_set_router.restype = ctypes.c_int
_lib.laser_test_withhold_tile.argtypes = [ctypes.c_int, ctypes.c_longlong]
_lib.laser_test_withhold_tile.restype = ctypes.c_int
_lib.laser_test_launch_empty.argtypes = [_vp]
_lib.laser_test_launch_empty.restype = ctypes.c_int


class LaserError(RuntimeError):
    def __init__(self, status: int):
        self.status = status
        super().__init__(f"laser: {strerror(status)} ({status})")


def test_set_router(mode: int) -> int:
    """laser_test_set_router: ROUTER_AUTO / ROUTER_TILE / ROUTER_SPLITK; returns the previous
    mode.  For tests."""
    prev = int(_lib.laser_test_set_router(int(mode)))
    if prev < 0:
        raise ValueError("unknown router mode %r" % (mode,))
    return prev


def test_withhold_tile(tile: int, wait_cycles: int = 0) -> None:
    """laser_test_withhold_tile: router tile `tile` publishes no ready flag and the selection's
    waits give up after `wait_cycles` clock cycles; tile < 0 restores.  For tests."""
    if int(_lib.laser_test_withhold_tile(int(tile), int(wait_cycles))) != 0:
        raise ValueError("wait_cycles must be positive")


def test_launch_empty(stream=None) -> None:
    """laser_test_launch_empty: one empty kernel on the stream (launch-floor measurements)."""
    import torch

    s = torch.cuda.current_stream() if stream is None else stream
    if int(_lib.laser_test_launch_empty(s.cuda_stream)) != 0:
        raise LaserError(ERR_CUDA)


test_launch_empty.__test__ = False
test_set_router.__test__ = False          # not pytest cases, whatever the names suggest
test_withhold_tile.__test__ = False


def version() -> int:
    return int(_lib.laser_version())


def strerror(status: int) -> str:
    return _lib.laser_strerror(int(status)).decode()


def make_params(T, d, E, k, c, eps_high, t_fix, renormalize=1, n_bins=1, ld_hidden=None,
                ld_w=None, trim_mode=0, update_granularity=1, seed=0,
                fresh_loads=0) -> LaserParams:
    return LaserParams(T, d, E, k, c, eps_high, t_fix, trim_mode, update_granularity,
                       int(renormalize), n_bins, int(fresh_loads),
                       d if ld_hidden is None else ld_hidden,
                       d if ld_w is None else ld_w, seed)


def workspace_bytes(p: LaserParams) -> int:
    out = _sz(0)
    rc = _lib.laser_workspace_bytes(ctypes.byref(p), ctypes.byref(out))
    if rc != OK:
        raise LaserError(rc)
    return int(out.value)


def host_arena_bytes(n_layers: int, p: LaserParams) -> int:
    out = _sz(0)
    rc = _lib.laser_host_arena_bytes(n_layers, ctypes.byref(p), ctypes.byref(out))
    if rc != OK:
        raise LaserError(rc)
    return int(out.value)


def _ptr(t) -> Optional[int]:
    return None if t is None else int(t.data_ptr())


def _floats(v: Optional[Sequence[float]]):
    if v is None:
        return None, None
    arr = (ctypes.c_float * len(v))(*[float(x) for x in v])
    return arr, ctypes.cast(arr, _vp)


def route_raw(hidden, w_g, bias, loads, expert_to_bin, bin_loads, p, expert_ids, weights,
              offsets, perm, logits_out, status_word, workspace, workspace_nbytes,
              stream=0) -> int:
    """laser_route with raw integer device addresses (or None); returns the status code."""
    return int(_lib.laser_route(hidden, w_g, bias, loads, expert_to_bin, bin_loads,
                                ctypes.byref(p), expert_ids, weights, offsets, perm, logits_out,
                                status_word, workspace, workspace_nbytes, stream))


@dataclass
class RouteResult:
    expert_ids: "object"
    weights: "object"
    offsets: "object"
    perm: "object"
    loads: "object"
    bin_loads: "object"
    logits: "object"
    status: "object"


def route_layers(hidden, w_g, bias, loads, p: LaserParams, *, expert_to_bin=None,
                 bin_loads=None, eps_high=None, t_fix=None, want_logits=False, out=None,
                 workspace=None, stream=None, stage_events=None) -> RouteResult:
    """laser_route_layers on torch CUDA tensors.

    hidden [L,T,d] bf16, w_g [L,E,d] bf16, bias [L,E] f32 or None, loads [L,E] int32
    (updated in place), bin_loads [L,B] int32 or None (updated in place).  ``out`` may carry
    preallocated outputs from an earlier RouteResult; otherwise they are allocated here.
    ``stage_events``: four torch.cuda.Event objects (already recorded once, so that their
    handles exist) to be recorded between the stages.
    """
    import torch

    L = hidden.shape[0]
    dev = hidden.device
    T, E, k = p.T, p.E, p.k
    if out is None:
        out = RouteResult(
            torch.empty((L, T, k), dtype=torch.int32, device=dev),
            torch.empty((L, T, k), dtype=torch.float32, device=dev),
            torch.empty((L, E + 1), dtype=torch.int32, device=dev),
            torch.empty((L, T * k), dtype=torch.int32, device=dev),
            loads, bin_loads,
            torch.empty((L, T, E), dtype=torch.float32, device=dev) if want_logits else None,
            torch.zeros((1,), dtype=torch.int32, device=dev))
    need = workspace_bytes(p) * L
    if workspace is None:
        workspace = torch.empty((need,), dtype=torch.uint8, device=dev)
    eps_arr, eps_p = _floats(eps_high)
    tf_arr, tf_p = _floats(t_fix)
    s = torch.cuda.current_stream(dev) if stream is None else stream
    ev_p = None
    if stage_events is not None:
        ev_arr = (_vp * 4)(*[None if e is None else int(e.cuda_event) for e in stage_events])
        ev_p = ctypes.cast(ev_arr, _vp)
    rc = _lib.laser_route_layers_profiled(
        L, _ptr(hidden), _ptr(w_g), _ptr(bias), _ptr(loads), _ptr(expert_to_bin),
        _ptr(bin_loads), ctypes.byref(p), eps_p, tf_p, _ptr(out.expert_ids), _ptr(out.weights),
        _ptr(out.offsets), _ptr(out.perm), _ptr(out.logits), _ptr(out.status),
        _ptr(workspace), workspace.numel(), s.cuda_stream, ev_p)
    if rc != OK:
        raise LaserError(rc)
    return out


def route(hidden, w_g, bias, loads, p: LaserParams, *, bin_loads=None, **kw) -> RouteResult:
    """laser_route for one layer: hidden [T,d], w_g [E,d], bias [E], loads [E] (in place)."""
    r = route_layers(hidden[None], w_g[None], None if bias is None else bias[None], loads[None],
                     p, bin_loads=None if bin_loads is None else bin_loads[None], **kw)
    return RouteResult(r.expert_ids[0], r.weights[0], r.offsets[0], r.perm[0], loads, bin_loads,
                       None if r.logits is None else r.logits[0], r.status)


def route_static(hidden, w_g, bias, loads, p: LaserParams, out: RouteResult, *,
                 expert_to_bin=None, bin_loads=None, stream=None) -> RouteResult:
    """laser_route_static for one layer, for callers that must not allocate: every tensor,
    the outputs in ``out`` included, is preallocated by the caller (hidden [T,d], w_g [E,d],
    bias [E] or None, loads [E] in place, out.expert_ids / weights [T,k], out.offsets [E+1],
    out.perm [T*k], out.logits [T,E] or None, out.status [1]); the scratch is the library's
    built-in array, so no workspace is passed.  Raises LaserError(ERR_STATIC_SCRATCH) when
    the shape needs more than STATIC_SCRATCH_BYTES."""
    import torch

    s = torch.cuda.current_stream(hidden.device) if stream is None else stream
    rc = _lib.laser_route_static(
        _ptr(hidden), _ptr(w_g), _ptr(bias), _ptr(loads), _ptr(expert_to_bin), _ptr(bin_loads),
        ctypes.byref(p), _ptr(out.expert_ids), _ptr(out.weights), _ptr(out.offsets),
        _ptr(out.perm), _ptr(out.logits), _ptr(out.status), s.cuda_stream)
    if rc != OK:
        raise LaserError(rc)
    return out


def imbalance(offsets, n_bins: int, expert_to_bin=None, placement=None, stream=None):
    """laser_imbalance on the offsets [L, E+1] of a finished call (torch CUDA int32 tensor).
    placement: optional [n_bins, E] fp32 matrix A (columns sum to 1), used instead of the map.
    Returns (I [L], I_bins [L], aggregate [2] = (I_agg, bin-level I_agg)) as device tensors;
    MV of a layer is I - 1."""
    import torch

    L, E1 = offsets.shape
    dev = offsets.device
    I = torch.empty((L,), dtype=torch.float32, device=dev)
    Ib = torch.empty((L,), dtype=torch.float32, device=dev)
    agg = torch.empty((2,), dtype=torch.float32, device=dev)
    s = torch.cuda.current_stream(dev) if stream is None else stream
    rc = _lib.laser_imbalance(L, E1 - 1, n_bins, _ptr(offsets), _ptr(expert_to_bin),
                              _ptr(placement), _ptr(I), _ptr(Ib), _ptr(agg), s.cuda_stream)
    if rc != OK:
        raise LaserError(rc)
    return I, Ib, agg


def score_stats(logits, k: int, near_ratio: float = 0.5, plateau_max: int = 4, stats=None,
                stream=None):
    """laser_score_stats on logits [L, T, E] (torch CUDA fp32).  Pass the returned `stats`
    [L, 72] int64 back in to accumulate further batches.  Returns (stats, means [L, 4])."""
    import torch

    L, T, E = logits.shape
    dev = logits.device
    accumulate = stats is not None
    if stats is None:
        stats = torch.empty((L, STATS_WORDS), dtype=torch.int64, device=dev)
    means = torch.empty((L, 4), dtype=torch.float32, device=dev)
    s = torch.cuda.current_stream(dev) if stream is None else stream
    rc = _lib.laser_score_stats(L, T, E, k, _ptr(logits), near_ratio, plateau_max,
                                int(accumulate), _ptr(stats), _ptr(means), s.cuda_stream)
    if rc != OK:
        raise LaserError(rc)
    return stats, means


def route_host(hidden, w_g, bias, loads, p: LaserParams, arena, *, expert_to_bin=None,
               bin_loads=None, eps_high=None, t_fix=None, out=None, stream=None):
    """laser_route_host: every array is a HOST (ideally pinned) torch tensor except ``arena``
    (device uint8 tensor of at least host_arena_bytes).  Returns (expert_ids, weights,
    offsets, perm, status) host tensors; loads / bin_loads are updated in place."""
    import torch

    L = hidden.shape[0]
    T, E, k = p.T, p.E, p.k
    if out is None:
        pin = dict(pin_memory=True)
        out = (torch.empty((L, T, k), dtype=torch.int32, **pin),
               torch.empty((L, T, k), dtype=torch.float32, **pin),
               torch.empty((L, E + 1), dtype=torch.int32, **pin),
               torch.empty((L, T * k), dtype=torch.int32, **pin),
               torch.zeros((1,), dtype=torch.int32, **pin))
    eps_arr, eps_p = _floats(eps_high)
    tf_arr, tf_p = _floats(t_fix)
    s = torch.cuda.current_stream(arena.device) if stream is None else stream
    rc = _lib.laser_route_host(
        L, _ptr(hidden), _ptr(w_g), _ptr(bias), _ptr(loads), _ptr(expert_to_bin),
        _ptr(bin_loads), ctypes.byref(p), eps_p, tf_p, _ptr(out[0]), _ptr(out[1]), _ptr(out[2]),
        _ptr(out[3]), _ptr(out[4]), _ptr(arena), arena.numel(), s.cuda_stream)
    if rc != OK:
        raise LaserError(rc)
    return out
