"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol
the header declares, and rejects bad arguments before touching the device."""
import ctypes
import os
import re

import pytest

from paper_2510_03293_b200 import laser

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions(header="laser.h"):
    text = open(os.path.join(ROOT, "include", header)).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(laser_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    assert sorted(os.listdir(os.path.join(ROOT, "include"))) == ["laser.h", "laser_test_hooks.h"]
    names = declared_functions()
    assert set(names) == set(laser.EXPORTS)
    hooks = declared_functions("laser_test_hooks.h")
    assert set(hooks) == set(laser.TEST_EXPORTS)
    lib = ctypes.CDLL(laser.LIB_PATH)
    for n in names + hooks:
        assert hasattr(lib, n), n
    assert laser.version() >= 100
    assert laser.strerror(0) == "ok" and "unknown" in laser.strerror(-99)


def test_hooks_reject_bad_settings_and_restore():
    assert laser.test_set_router(laser.ROUTER_TILE) == laser.ROUTER_AUTO
    assert laser.test_set_router(laser.ROUTER_AUTO) == laser.ROUTER_TILE
    with pytest.raises(ValueError):
        laser.test_set_router(7)
    assert laser.test_set_router(laser.ROUTER_AUTO) == laser.ROUTER_AUTO   # unchanged by the bad call
    with pytest.raises(ValueError):
        laser.test_withhold_tile(0, 0)
    laser.test_withhold_tile(-1)


def test_no_environment_lookups_in_the_library_sources():
    csrc = os.path.join(ROOT, "paper_2510_03293_b200", "csrc")
    for name in os.listdir(csrc):
        assert "getenv" not in open(os.path.join(csrc, name)).read(), name


def good(**over):
    kw = dict(T=128, d=256, E=8, k=2, c=4, eps_high=0.5, t_fix=0.5, renormalize=1, n_bins=4)
    kw.update(over)
    return laser.make_params(**kw)


@pytest.mark.parametrize("over,status", [
    (dict(T=-1), laser.ERR_INVALID_ARG),
    (dict(d=0), laser.ERR_INVALID_ARG),
    (dict(d=250), laser.ERR_INVALID_ARG),
    (dict(E=0), laser.ERR_INVALID_ARG),
    (dict(E=257, c=4), laser.ERR_INVALID_ARG),
    (dict(k=0), laser.ERR_INVALID_ARG),
    (dict(k=5, c=4), laser.ERR_INVALID_ARG),
    (dict(c=9), laser.ERR_INVALID_ARG),
    (dict(eps_high=-0.1), laser.ERR_INVALID_ARG),
    (dict(eps_high=float("nan")), laser.ERR_INVALID_ARG),
    (dict(t_fix=1.5), laser.ERR_INVALID_ARG),
    (dict(n_bins=0), laser.ERR_INVALID_ARG),
    (dict(ld_hidden=128), laser.ERR_INVALID_ARG),
    (dict(ld_hidden=260), laser.ERR_MISALIGNED),
    (dict(trim_mode=7), laser.ERR_INVALID_ARG),
    (dict(update_granularity=7), laser.ERR_UNSUPPORTED),
    (dict(update_granularity=-32), laser.ERR_INVALID_ARG),
    (dict(T=2**30, k=4, c=4), laser.ERR_INVALID_ARG),
])
def test_bad_parameters_are_rejected(over, status):
    p = good(**over)
    with pytest.raises(laser.LaserError) as e:
        laser.workspace_bytes(p)
    assert e.value.status == status
    # the routing entry point refuses the same parameters without launching anything
    assert laser.route_raw(256, 256, None, 256, None, None, p, 256, 256, 256, 256, None, None,
                           256, 1 << 30) == status


def test_pointer_checks_come_before_any_launch():
    p = good()
    need = laser.workspace_bytes(p)
    assert need > 0 and need % 256 == 0
    args = dict(hidden=4096, w_g=4096, loads=4096, ids=4096, w=4096, off=4096, perm=4096, ws=4096)

    def call(**o):
        a = dict(args); a.update(o)
        return laser.route_raw(a["hidden"], a["w_g"], None, a["loads"], None, None, p, a["ids"],
                               a["w"], a["off"], a["perm"], None, None, a["ws"],
                               o.get("ws_bytes", need))

    assert call(w_g=None) == laser.ERR_INVALID_ARG
    assert call(loads=None) == laser.ERR_INVALID_ARG
    assert call(ids=None) == laser.ERR_INVALID_ARG
    assert call(ws=None) == laser.ERR_INVALID_ARG
    assert call(hidden=4096 + 2) == laser.ERR_MISALIGNED
    assert call(ws=4096 + 16) == laser.ERR_MISALIGNED
    assert call(ws_bytes=need - 1) == laser.ERR_WORKSPACE_TOO_SMALL


def test_workspace_grows_with_the_trimming_size():
    small = laser.workspace_bytes(good(T=4096, c=4))
    large = laser.workspace_bytes(good(T=4096, c=8))
    assert large > small
    assert laser.host_arena_bytes(2, good()) > 2 * laser.workspace_bytes(good())


def test_metric_entry_points_check_their_arguments_before_any_launch():
    """laser_imbalance and laser_score_stats return INVALID_ARG for bad sizes and missing
    pointers without touching the device (fake non-null pointers are never dereferenced)."""
    import ctypes

    lib = laser._lib
    P = ctypes.c_void_p

    def imb(L=2, E=8, B=4, off=4096, out=4096, placement=None):
        return lib.laser_imbalance(L, E, B, P(off), None, P(placement) if placement else None,
                                   P(out), None, None, None)

    assert imb(L=0) == laser.ERR_INVALID_ARG
    assert imb(L=70000) == laser.ERR_INVALID_ARG
    assert imb(E=0) == laser.ERR_INVALID_ARG and imb(E=257) == laser.ERR_INVALID_ARG
    assert imb(B=0) == laser.ERR_INVALID_ARG
    assert imb(B=9) == laser.ERR_INVALID_ARG              # more bins than experts without a matrix
    assert imb(B=2000, placement=4096) == laser.ERR_INVALID_ARG
    assert imb(off=None) == laser.ERR_INVALID_ARG and imb(out=None) == laser.ERR_INVALID_ARG

    def stats(L=2, T=64, E=8, k=2, x=4096, ratio=0.5, pmax=3, out=4096):
        return lib.laser_score_stats(L, T, E, k, P(x), ctypes.c_float(ratio), pmax, 0, P(out),
                                     None, None)

    assert stats(L=0) == laser.ERR_INVALID_ARG
    assert stats(T=-1) == laser.ERR_INVALID_ARG
    assert stats(E=300) == laser.ERR_INVALID_ARG
    assert stats(k=0) == laser.ERR_INVALID_ARG and stats(k=9) == laser.ERR_INVALID_ARG
    assert stats(ratio=1.5) == laser.ERR_INVALID_ARG and stats(ratio=-0.1) == laser.ERR_INVALID_ARG
    assert stats(ratio=float("nan")) == laser.ERR_INVALID_ARG
    assert stats(pmax=0) == laser.ERR_INVALID_ARG
    assert stats(x=None) == laser.ERR_INVALID_ARG and stats(out=None) == laser.ERR_INVALID_ARG
    assert stats(L=65535, T=1 << 15) == laser.ERR_INVALID_ARG   # 2^30 tokens or more
