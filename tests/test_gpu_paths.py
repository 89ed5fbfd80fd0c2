"""GPU parity on the library paths that the common shapes never enter: many experts per token
(k above 8 and above 32), candidate lists wider than a warp on the 128-column router, rows
whose scores all tie, load counters too large for the packed 32-bit keys, and the status a
call returns when one of its bounded device-side waits runs out."""
import numpy as np
import pytest

from paper_2510_03293_b200 import synth
from gpu_util import check_against_oracle, run_gpu

pytestmark = pytest.mark.gpu

ROUTERS = ["tile", "splitk"]


@pytest.fixture
def force_router():
    from paper_2510_03293_b200 import laser

    def choose(name):
        laser.test_set_router({"tile": laser.ROUTER_TILE, "splitk": laser.ROUTER_SPLITK,
                               "oneshot": laser.ROUTER_TILE_ONESHOT}[name])

    yield choose
    laser.test_set_router(laser.ROUTER_AUTO)


def layer(T, d, E, seed, sigma=0.03, with_bias=True):
    return synth.make_layer(T, d, E, sigma, 1.2, seed=seed, stream=E * 11 + d, with_bias=with_bias)


@pytest.mark.parametrize("router", ROUTERS)
@pytest.mark.parametrize("T,d,E,k,c,eps,tfix,renorm,B", [
    (600, 256, 64, 12, 20, 0.50, 0.30, 1, 8),     # k in 9..32: generic dispatch body, E > 32
    (500, 256, 32, 16, 32, 0.70, 0.20, 0, 4),     # k = 16, c = 32 on the E <= 32 fixed point
    (300, 128, 256, 40, 48, 0.40, 0.10, 1, 32),   # k > 32: one-warp scan through k, not c
    (400, 256, 100, 5, 40, 0.30, 0.05, 1, 10),    # c > 32 with 128 accumulator columns
    (300, 128, 48, 33, 48, 0.90, 0.00, 0, 6),     # k > 32 with every expert a candidate
])
def test_many_slots_and_wide_candidate_lists(cuda_device, force_router, router, T, d, E, k, c,
                                             eps, tfix, renorm, B):
    force_router(router)
    hb, wb, bias = layer(T, d, E, seed=T + 3 * E + k)
    rng = np.random.default_rng(E * 1000 + k)
    loads0 = rng.integers(0, 6, E).astype(np.int32)
    bins0 = rng.integers(0, 50, B).astype(np.int32)
    g = run_gpu(cuda_device, hb, wb, bias, loads0, k, c, eps, tfix, renorm, B, bins0=bins0)
    ref = check_against_oracle(g, hb, wb, bias, loads0, k, c, eps, tfix, renorm, B, bins0=bins0)
    assert int((ref["cstar"] > k).sum()) > 0, "no token took a load-dependent decision"


@pytest.mark.parametrize("router", ROUTERS)
@pytest.mark.parametrize("E,k,c", [(64, 6, 8), (64, 6, 24), (256, 8, 16), (128, 4, 40)])
@pytest.mark.parametrize("skewed", [False, True])
def test_rows_whose_scores_all_tie(cuda_device, force_router, router, E, k, c, skewed):
    """W_g = 0 and no bias: every logit is 0, so every ranking is decided by the index alone
    (Algorithm 1 breaks load ties by score, and equal scores go to the lower index) and every
    choice by the loads alone.  With t_fix = 1 all c best experts are candidates."""
    force_router(router)
    T = 400
    hb, _, _ = layer(T, 128, E, seed=E + k)
    wb = np.zeros((E, 128), np.uint16)
    rng = np.random.default_rng(E + c)
    loads0 = (rng.integers(0, 40, E) * rng.integers(0, 2, E)).astype(np.int32) if skewed \
        else np.zeros(E, np.int32)
    g = run_gpu(cuda_device, hb, wb, None, loads0, k, c, 0.9, 1.0)
    ref = check_against_oracle(g, hb, wb, None, loads0, k, c, 0.9, 1.0)
    assert np.all(ref["cstar"] == c)
    assert np.all(g["logits"] == 0.0)
    # every candidate list is experts 0..c-1: only those receive tokens
    assert int(g["loads"][c:].sum()) == int(loads0[c:].sum())
    if not skewed:
        assert g["loads"][:c].max() - g["loads"][:c].min() <= 1


@pytest.mark.parametrize("router", ROUTERS)
@pytest.mark.parametrize("T,E,k,c", [(64, 64, 6, 8), (700, 64, 6, 8), (333, 8, 2, 4),
                                     (200, 256, 8, 16)])
def test_loads_beyond_the_packed_key_range(cuda_device, force_router, router, T, E, k, c):
    """Load counters of 2^25 and more do not fit the 32-bit (load, rank) keys; the call then
    takes the one-warp scan with 64-bit keys, also when the router's tiles are shorter than the
    scan's groups of 32 tokens (split-K router: 16 tokens per tile)."""
    force_router(router)
    hb, wb, bias = layer(T, 256, E, seed=T + E)
    rng = np.random.default_rng(T)
    loads0 = ((1 << 25) + rng.integers(0, 5, E)).astype(np.int32)
    g = run_gpu(cuda_device, hb, wb, bias, loads0, k, c, 0.6, 0.5, 0, 4,
                bins0=np.zeros(4, np.int32))
    ref = check_against_oracle(g, hb, wb, bias, loads0, k, c, 0.6, 0.5, 0, 4,
                               bins0=np.zeros(4, np.int32))
    assert int((ref["cstar"] > k).sum()) > 0


@pytest.mark.parametrize("router,T,d,E,k,c,tile", [
    ("tile", 1000, 256, 8, 2, 4, 1),       # warp-level router, 128-token tiles
    ("tile", 1000, 256, 64, 6, 8, 2),      # tensor-memory router, persistent blocks
    ("tile", 1000, 256, 256, 8, 16, 3),    # ... with 256 accumulator columns
    ("oneshot", 1000, 256, 64, 6, 8, 2),   # ... one tile per block
    ("splitk", 300, 256, 64, 6, 8, 5),     # split-K router, 16-token tiles, fused dispatch off
    ("splitk", 200, 256, 64, 6, 8, 3),     # ... dispatch inside the selection block
    ("tile", 700, 128, 256, 8, 40, 0),     # one-warp scan (candidate lists wider than a warp)
])
def test_a_wait_that_runs_out_sets_the_timeout_bit(cuda_device, force_router, router, T, d, E, k,
                                                   c, tile):
    """One router tile publishes no ready flag and the selection's wait limit is about a
    millisecond: the call must come back with LASER_DEV_TIMEOUT set and every output buffer's
    surroundings untouched, and the next ordinary call must be exact again."""
    from paper_2510_03293_b200 import laser

    force_router(router)
    hb, wb, bias = layer(T, d, E, seed=T + E + tile)
    z = np.zeros(E, np.int32)
    laser.test_withhold_tile(tile, 2_000_000)
    try:
        g = run_gpu(cuda_device, hb, wb, bias, z, k, c, 0.5, 0.5)   # checks the canaries
    finally:
        laser.test_withhold_tile(-1)
    assert g["status"] & laser.DEV_TIMEOUT
    # tokens before the withheld tile's batch may have been counted; never more than all
    assert 0 <= int(g["loads"].sum()) <= T * k and int(g["loads"].min()) >= 0
    g = run_gpu(cuda_device, hb, wb, bias, z, k, c, 0.5, 0.5)
    check_against_oracle(g, hb, wb, bias, z, k, c, 0.5, 0.5)


@pytest.mark.parametrize("T,d,E,k,c", [(100, 256, 64, 6, 8), (112, 128, 256, 8, 16),
                                       (17, 64, 100, 5, 20), (64, 2048, 64, 6, 8),
                                       (1, 256, 64, 6, 8), (97, 512, 8, 2, 4)])
def test_calls_of_a_few_tiles_run_as_one_cluster_per_layer(cuda_device, T, d, E, k, c):
    """At most 112 tokens: the layer's router tiles and its selection block are launched as one
    thread-block cluster and meet at the cluster barrier instead of ready flags.  Several
    layers at once must equal the layers routed one by one, and each the oracle."""
    import torch

    from paper_2510_03293_b200 import laser
    from gpu_util import to_dev_bf16

    dev = cuda_device
    L = 5
    layers = [layer(T, d, E, seed=700 + l + T) for l in range(L)]
    hb = np.stack([x[0] for x in layers]); wb = np.stack([x[1] for x in layers])
    bias = np.stack([x[2] for x in layers])
    rng = np.random.default_rng(T + E)
    loads0 = rng.integers(0, 4, (L, E)).astype(np.int32)
    p = laser.make_params(T, d, E, k, c, 0.5, 0.5, 1, 4)
    loads = torch.from_numpy(loads0.copy()).to(dev)
    bins = torch.zeros((L, 4), dtype=torch.int32, device=dev)
    # a workspace full of ones: nothing clears it for this kind of call, and nothing has to
    ws = torch.full((laser.workspace_bytes(p) * L,), 0x5A, dtype=torch.uint8, device=dev)
    r = laser.route_layers(to_dev_bf16(hb, dev), to_dev_bf16(wb, dev),
                           torch.from_numpy(bias).to(dev), loads, p, bin_loads=bins,
                           want_logits=True, workspace=ws)
    torch.cuda.synchronize()
    assert int(r.status.item()) == 0
    for l in range(L):
        g = dict(expert_ids=r.expert_ids[l].cpu().numpy(), weights=r.weights[l].cpu().numpy(),
                 offsets=r.offsets[l].cpu().numpy(), perm=r.perm[l].cpu().numpy(),
                 loads=loads[l].cpu().numpy(), bin_loads=bins[l].cpu().numpy(),
                 logits=r.logits[l].cpu().numpy(), status=0)
        check_against_oracle(g, hb[l], wb[l], bias[l], loads0[l], k, c, 0.5, 0.5, 1, 4,
                             bins0=np.zeros(4, np.int32))


@pytest.mark.parametrize("router", ROUTERS)
@pytest.mark.parametrize("T,d,E,k,c", [(0, 64, 8, 2, 4), (90, 128, 64, 6, 8), (700, 256, 8, 2, 4),
                                       (900, 128, 64, 6, 8), (600, 128, 256, 8, 16),
                                       (300, 128, 256, 8, 40)])
def test_a_call_that_starts_from_empty_counters(cuda_device, force_router, router, T, d, E, k, c):
    """fresh_loads = 1: whatever the load and bin counters hold on entry is ignored; the call
    equals the oracle started from zero loads, and the counters return the call's own counts."""
    force_router(router)
    hb, wb, bias = layer(T, d, E, seed=T + E + 5)
    rng = np.random.default_rng(T + c)
    junk_loads = rng.integers(-5, 1 << 28, E).astype(np.int32)
    junk_bins = rng.integers(-5, 1 << 28, 4).astype(np.int32)
    g = run_gpu(cuda_device, hb, wb, bias, junk_loads, k, c, 0.5, 0.5, 1, 4, bins0=junk_bins,
                fresh=1)
    zero_l, zero_b = np.zeros(E, np.int32), np.zeros(4, np.int32)
    check_against_oracle(g, hb, wb, bias, zero_l, k, c, 0.5, 0.5, 1, 4, bins0=zero_b)
    assert int(g["loads"].sum()) == T * k and int(g["bin_loads"].sum()) == T * k


def bf16_bits(x):
    """bf16 bit patterns of values that are exactly representable (small integers, halves)."""
    return (np.asarray(x, np.float32).view(np.uint32) >> 16).astype(np.uint16)


@pytest.mark.parametrize("router", ROUTERS + ["oneshot"])
@pytest.mark.parametrize("T,d,E,k,c", [(500, 64, 64, 6, 8), (700, 32, 256, 8, 16),
                                       (300, 64, 128, 4, 12), (400, 48, 8, 2, 4)])
def test_rows_with_many_equal_logits(cuda_device, force_router, router, T, d, E, k, c):
    """Hidden states and gate weights from {-1, 0, 1}: logits are small integers, most of them
    shared by several experts of a row, so rankings are decided by the index inside groups of
    equal logits next to groups that differ (the sorting-network epilogues have to notice)."""
    force_router(router)
    rng = np.random.default_rng(T + E)
    hb = bf16_bits(rng.integers(-1, 2, (T, d)))
    wb = bf16_bits(rng.integers(-1, 2, (E, d)))
    bias = (rng.integers(0, 3, E) * 0.5).astype(np.float32)
    loads0 = rng.integers(0, 3, E).astype(np.int32)
    g = run_gpu(cuda_device, hb, wb, bias, loads0, k, c, 0.9, 0.2, 1, 4,
                bins0=np.zeros(4, np.int32))
    check_against_oracle(g, hb, wb, bias, loads0, k, c, 0.9, 0.2, 1, 4,
                         bins0=np.zeros(4, np.int32))
