"""GPU parity: the CUDA path through the C ABI against the CPU oracle, element by element,
on small and odd shapes that still span several tiles and a ragged tail."""
import numpy as np
import pytest

from paper_2510_03293_b200 import synth
import oracle
from gpu_util import check_against_oracle, run_gpu, to_dev_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture
def force_router():
    """Selects the router by hand for one test (small shapes otherwise always take the
    split-K router) and restores the automatic choice afterwards."""
    from paper_2510_03293_b200 import laser

    def choose(name):
        laser.test_set_router({"tile": laser.ROUTER_TILE, "splitk": laser.ROUTER_SPLITK,
                               "oneshot": laser.ROUTER_TILE_ONESHOT}[name])

    yield choose
    laser.test_set_router(laser.ROUTER_AUTO)


def layer(T, d, E, seed, sigma=0.02, alpha=1.2, with_bias=True):
    return synth.make_layer(T, d, E, sigma, alpha, seed=seed, stream=E * 7 + d, with_bias=with_bias)


CASES = [
    # T, d, E, k, c, eps, tfix, renorm, n_bins
    (1, 4096, 8, 2, 4, 0.64, 0.6, 1, 4),
    (2, 4096, 8, 2, 4, 0.64, 0.6, 1, 4),
    (31, 264, 8, 2, 4, 0.64, 0.6, 1, 8),
    (33, 8, 8, 2, 8, 0.64, 0.6, 0, 2),
    (257, 1032, 8, 1, 3, 0.5, 0.5, 1, 1),
    (2048, 4096, 8, 2, 4, 0.6419, 0.6, 1, 4),
    (1000, 2048, 64, 6, 8, 0.40, 0.80, 0, 8),
    (515, 512, 64, 6, 10, 0.30, 0.50, 1, 8),
    (300, 1024, 2, 1, 2, 0.8, 0.3, 1, 2),
    (300, 1024, 2, 2, 2, 0.8, 0.3, 1, 1),
    (400, 520, 5, 2, 5, 0.7, 0.4, 1, 5),
    (300, 256, 13, 3, 7, 0.6, 0.5, 1, 4),
    (200, 256, 24, 4, 9, 0.5, 0.5, 0, 3),
    (150, 256, 100, 5, 20, 0.3, 0.3, 1, 10),
    (130, 512, 128, 8, 16, 0.3, 0.25, 1, 16),
    (777, 1024, 256, 8, 16, 0.30, 0.25, 1, 32),
    (100, 256, 256, 8, 40, 0.30, 0.10, 1, 32),      # candidate sets wider than a warp
    # enough tokens for the 128-token-tile routers (fewer tokens take the split-K router)
    (5000, 256, 8, 2, 4, 0.6, 0.5, 1, 4),
    (5000, 256, 13, 3, 7, 0.6, 0.5, 1, 4),
    (5000, 264, 24, 4, 9, 0.5, 0.5, 0, 3),
    (4900, 512, 64, 6, 8, 0.40, 0.80, 0, 8),
    (5000, 256, 100, 5, 20, 0.3, 0.3, 1, 10),
    (5000, 256, 200, 8, 16, 0.3, 0.25, 1, 8),
    (4800, 128, 256, 8, 40, 0.30, 0.10, 1, 32),
]


@pytest.mark.parametrize("T,d,E,k,c,eps,tfix,renorm,B", CASES)
def test_route_matches_oracle(cuda_device, T, d, E, k, c, eps, tfix, renorm, B):
    sigma = 0.02 if E < 256 else 0.04
    hb, wb, bias = layer(T, d, E, seed=T + E, sigma=sigma)
    rng = np.random.default_rng(T * 31 + E)
    loads0 = rng.integers(0, 5, E).astype(np.int32)
    bins0 = rng.integers(0, 100, B).astype(np.int32)
    g = run_gpu(cuda_device, hb, wb, bias, loads0, k, c, eps, tfix, renorm, B, bins0=bins0)
    ref = check_against_oracle(g, hb, wb, bias, loads0, k, c, eps, tfix, renorm, B, bins0=bins0)
    if T >= 100 and d >= 1024 and 0 < eps < 1 and c > k:
        frac = float((ref["cstar"] > 0).mean())
        assert 0.005 < frac < 0.995, f"only one branch exercised (expanded fraction {frac})"


@pytest.mark.parametrize("T,d,E,k,c,eps,tfix,renorm,B", [
    (1000, 2048, 64, 6, 8, 0.40, 0.80, 0, 8), (515, 512, 64, 6, 10, 0.30, 0.50, 1, 8),
    (4900, 512, 64, 6, 8, 0.40, 0.80, 0, 8), (700, 264, 48, 4, 12, 0.5, 0.4, 1, 6),
    (130, 256, 33, 3, 5, 0.5, 0.5, 1, 3), (40000, 128, 64, 6, 8, 0.5, 0.6, 1, 8),
    (777, 1024, 256, 8, 16, 0.30, 0.25, 1, 32), (1500, 264, 200, 8, 12, 0.3, 0.25, 0, 8),
    (300, 128, 129, 4, 4, 0.5, 0.5, 1, 3), (40000, 64, 256, 8, 16, 0.4, 0.3, 1, 16)])
@pytest.mark.parametrize("router", ["tile", "oneshot"])
def test_both_forms_of_the_tensor_memory_router(cuda_device, force_router, router, T, d, E, k, c, eps,
                                            tfix, renorm, B):
    """32 < E <= 64, and 128 < E <= 256 with lists of at most 16, have a persistent router
    (several tiles per block, more tiles than blocks in the cases of 40000 tokens) and a
    one-tile-per-block form; both must equal the oracle."""
    force_router(router)
    test_route_matches_oracle(cuda_device, T, d, E, k, c, eps, tfix, renorm, B)


@pytest.mark.parametrize("T,d,E,k,c,eps,tfix,renorm,B", [c_ for c_ in CASES if c_[0] < 4000])
def test_small_cases_through_the_tile_routers(cuda_device, force_router, T, d, E, k, c, eps, tfix,
                                              renorm, B):
    force_router("tile")
    test_route_matches_oracle(cuda_device, T, d, E, k, c, eps, tfix, renorm, B)


def test_vanilla_and_load_only_settings(cuda_device):
    hb, wb, bias = layer(600, 512, 64, seed=5)
    z = np.zeros(64, np.int32)
    g = run_gpu(cuda_device, hb, wb, bias, z, 6, 8, 0.0, 0.8)           # eps_high = 0: top-k
    ref = check_against_oracle(g, hb, wb, bias, z, 6, 8, 0.0, 0.8)
    assert np.all(ref["cstar"] == 0)
    g = run_gpu(cuda_device, hb, wb, bias, z, 6, 64, 2.0, 0.0)          # load-only, c = E
    ref = check_against_oracle(g, hb, wb, bias, z, 6, 64, 2.0, 0.0)
    assert np.all(ref["cstar"] == 64)
    L = g["loads"]
    assert L.max() - L.min() <= 1 and int(L.sum()) == 600 * 6
    hb, wb, bias = layer(64, 256, 256, seed=6)
    z = np.zeros(256, np.int32)
    g = run_gpu(cuda_device, hb, wb, bias, z, 8, 256, 2.0, 0.0)         # load-only at E = 256
    check_against_oracle(g, hb, wb, bias, z, 8, 256, 2.0, 0.0)
    assert g["loads"].max() - g["loads"].min() <= 1


def test_k_equals_E_and_c_equals_k(cuda_device):
    hb, wb, bias = layer(200, 256, 8, seed=8)
    L0 = np.arange(8, dtype=np.int32) * 3
    for k, c in [(8, 8), (3, 3), (1, 1)]:
        g = run_gpu(cuda_device, hb, wb, bias, L0, k, c, 2.0, 0.5)
        check_against_oracle(g, hb, wb, bias, L0, k, c, 2.0, 0.5)


def test_degenerate_scores_and_loads(cuda_device):
    # all-equal logits (W_g = 0, no bias): ties resolve to the lower index, then loads decide
    hb, _, _ = layer(300, 256, 8, seed=9)
    wb = np.zeros((8, 256), np.uint16)
    z = np.zeros(8, np.int32)
    g = run_gpu(cuda_device, hb, wb, None, z, 2, 8, 0.9, 1.0)
    check_against_oracle(g, hb, wb, None, z, 2, 8, 0.9, 1.0)
    assert g["loads"].max() - g["loads"].min() <= 1
    # heavily pre-skewed loads
    hb, wb, bias = layer(300, 256, 8, seed=10)
    L0 = np.array([10**6, 0, 5, 10**6, 7, 7, 0, 123456], np.int32)
    g = run_gpu(cuda_device, hb, wb, bias, L0, 2, 5, 0.9, 0.3)
    check_against_oracle(g, hb, wb, bias, L0, 2, 5, 0.9, 0.3)


def test_empty_call_writes_zero_offsets(cuda_device):
    hb = np.zeros((0, 64), np.uint16)
    _, wb, bias = layer(4, 64, 8, seed=1)
    L0 = np.arange(8, dtype=np.int32)
    g = run_gpu(cuda_device, hb, wb, bias, L0, 2, 4, 0.5, 0.5, bins0=np.ones(1, np.int32),
                want_logits=False)
    assert np.array_equal(g["offsets"], np.zeros(9, np.int32))
    assert np.array_equal(g["loads"], L0) and g["bin_loads"].tolist() == [1]


def test_custom_expert_to_bin(cuda_device):
    hb, wb, bias = layer(500, 256, 8, seed=12)
    e2b = np.array([2, 0, 1, 2, 2, 0, 1, 0], np.int32)
    z = np.zeros(8, np.int32)
    g = run_gpu(cuda_device, hb, wb, bias, z, 2, 4, 0.64, 0.6, n_bins=3, e2b=e2b,
                bins0=np.zeros(3, np.int32))
    check_against_oracle(g, hb, wb, bias, z, 2, 4, 0.64, 0.6, n_bins=3, e2b=e2b,
                         bins0=np.zeros(3, np.int32))
    assert int(g["bin_loads"].sum()) == 500 * 2


def test_run_twice_is_bit_identical(cuda_device):
    hb, wb, bias = layer(3000, 512, 64, seed=14)
    z = np.zeros(64, np.int32)
    a = run_gpu(cuda_device, hb, wb, bias, z, 6, 8, 0.4, 0.8)
    b = run_gpu(cuda_device, hb, wb, bias, z, 6, 8, 0.4, 0.8)
    for name in ("expert_ids", "weights", "offsets", "perm", "loads", "logits"):
        assert np.array_equal(a[name], b[name])


def test_split_call_carries_the_load_state(cuda_device):
    hb, wb, bias = layer(1001, 512, 8, seed=15)
    z = np.zeros(8, np.int32)
    whole = run_gpu(cuda_device, hb, wb, bias, z, 2, 4, 0.64, 0.6)
    first = run_gpu(cuda_device, hb[:500], wb, bias, z, 2, 4, 0.64, 0.6)
    second = run_gpu(cuda_device, hb[500:], wb, bias, first["loads"], 2, 4, 0.64, 0.6)
    assert np.array_equal(whole["expert_ids"], np.vstack([first["expert_ids"], second["expert_ids"]]))
    assert np.array_equal(whole["loads"], second["loads"])


def test_layers_batch_equals_single_calls_and_host_entry(cuda_device):
    import torch

    from paper_2510_03293_b200 import laser

    dev = cuda_device
    Lr, T, d, E, k, c, B = 3, 700, 512, 8, 2, 4, 4
    eps = [0.7159, 0.6419, 0.6285]
    tf = [0.6, 0.5, 0.6]
    layers = [layer(T, d, E, seed=100 + l) for l in range(Lr)]
    hb = np.stack([x[0] for x in layers]); wb = np.stack([x[1] for x in layers])
    bias = np.stack([x[2] for x in layers])
    p = laser.make_params(T, d, E, k, c, 0.0, 0.0, 1, B)
    loads = torch.zeros((Lr, E), dtype=torch.int32, device=dev)
    bins = torch.zeros((Lr, B), dtype=torch.int32, device=dev)
    r = laser.route_layers(to_dev_bf16(hb, dev), to_dev_bf16(wb, dev),
                           torch.from_numpy(bias).to(dev), loads, p, bin_loads=bins,
                           eps_high=eps, t_fix=tf, want_logits=True)
    torch.cuda.synchronize()
    singles = []
    for l in range(Lr):
        g = run_gpu(dev, hb[l], wb[l], bias[l], np.zeros(E, np.int32), k, c, eps[l], tf[l], 1, B,
                    bins0=np.zeros(B, np.int32))
        check_against_oracle(g, hb[l], wb[l], bias[l], np.zeros(E, np.int32), k, c, eps[l], tf[l],
                             1, B, bins0=np.zeros(B, np.int32))
        singles.append(g)
        assert np.array_equal(r.expert_ids[l].cpu().numpy(), g["expert_ids"])
        assert np.array_equal(r.weights[l].cpu().numpy(), g["weights"])
        assert np.array_equal(r.offsets[l].cpu().numpy(), g["offsets"])
        assert np.array_equal(r.perm[l].cpu().numpy(), g["perm"])
        assert np.array_equal(loads[l].cpu().numpy(), g["loads"])
        assert np.array_equal(bins[l].cpu().numpy(), g["bin_loads"])
    # the host-buffer entry point gives the same answer
    arena = torch.empty((laser.host_arena_bytes(Lr, p),), dtype=torch.uint8, device=dev)
    h_loads = torch.zeros((Lr, E), dtype=torch.int32).pin_memory()
    h_bins = torch.zeros((Lr, B), dtype=torch.int32).pin_memory()
    ids, w, off, perm, status = laser.route_host(
        torch.from_numpy(hb.view(np.int16)).pin_memory(), torch.from_numpy(wb.view(np.int16)).pin_memory(),
        torch.from_numpy(bias).pin_memory(), h_loads, p, arena, bin_loads=h_bins, eps_high=eps,
        t_fix=tf)
    for l in range(Lr):
        assert np.array_equal(ids[l].numpy(), singles[l]["expert_ids"])
        assert np.array_equal(w[l].numpy(), singles[l]["weights"])
        assert np.array_equal(off[l].numpy(), singles[l]["offsets"])
        assert np.array_equal(perm[l].numpy(), singles[l]["perm"])
        assert np.array_equal(h_loads[l].numpy(), singles[l]["loads"])
        assert np.array_equal(h_bins[l].numpy(), singles[l]["bin_loads"])
    assert int(status.item()) == 0


def test_load_overflow_sets_the_status_bit(cuda_device):
    hb, wb, bias = layer(50, 256, 8, seed=16)
    L0 = np.full(8, 2**31 - 1, np.int32)
    g = run_gpu(cuda_device, hb, wb, bias, L0, 2, 4, 0.64, 0.6)
    assert g["status"] & 1
    L1 = np.zeros(8, np.int32)
    assert run_gpu(cuda_device, hb, wb, bias, L1, 2, 4, 0.64, 0.6)["status"] == 0


def _route_layers_strided(dev, hb, wb, bias, ld_h, ld_w, k, c, eps, tfix, B):
    """Routes [L,T,d] inputs stored with row pitches ld_h / ld_w (> d, padded with NaN bits so
    that any read of the padding shows up in the logits)."""
    import torch

    from paper_2510_03293_b200 import laser

    L, T, d = hb.shape
    E = wb.shape[1]
    hp = np.full((L, T, ld_h), 0x7FC0, np.uint16); hp[:, :, :d] = hb
    wp = np.full((L, E, ld_w), 0x7FC0, np.uint16); wp[:, :, :d] = wb
    p = laser.make_params(T, d, E, k, c, eps, tfix, 1, B, ld_hidden=ld_h, ld_w=ld_w)
    loads = torch.zeros((L, E), dtype=torch.int32, device=dev)
    bins = torch.zeros((L, B), dtype=torch.int32, device=dev)
    r = laser.route_layers(to_dev_bf16(hp, dev), to_dev_bf16(wp, dev),
                           torch.from_numpy(bias).to(dev), loads, p, bin_loads=bins,
                           want_logits=True)
    torch.cuda.synchronize()
    return r, loads, bins


@pytest.mark.parametrize("router", ["tile", "splitk"])
@pytest.mark.parametrize("L,T,d,E,k,c,ld_h,ld_w", [
    (3, 200, 264, 64, 6, 8, 264, 264),      # tensor-memory router: tiles straddle layers, d % 64 != 0
    (2, 333, 520, 100, 5, 12, 528, 536),    # ... with padded rows and 128 accumulator columns
    (2, 150, 256, 256, 8, 16, 320, 256),    # ... 256 accumulator columns, two-pass epilogue
    (3, 300, 264, 8, 2, 4, 272, 280),       # warp-level router with padded rows
    (8, 4100, 128, 256, 8, 16, 128, 128),   # persistent routers: more tiles than blocks, tiles of
    (11, 5000, 64, 64, 6, 8, 64, 64),       # different layers one after the other in a block
])
def test_batched_layers_ragged_tiles_and_row_pitch(cuda_device, force_router, router, L, T, d, E,
                                                   k, c, ld_h, ld_w):
    force_router(router)   # both routers on the same small inputs
    layers = [layer(T, d, E, seed=200 + l + E, sigma=0.05) for l in range(L)]
    hb = np.stack([x[0] for x in layers]); wb = np.stack([x[1] for x in layers])
    bias = np.stack([x[2] for x in layers])
    B = 4
    r, loads, bins = _route_layers_strided(cuda_device, hb, wb, bias, ld_h, ld_w, k, c, 0.5, 0.5, B)
    assert int(r.status.item()) == 0
    for l in range(L):
        g = dict(expert_ids=r.expert_ids[l].cpu().numpy(), weights=r.weights[l].cpu().numpy(),
                 offsets=r.offsets[l].cpu().numpy(), perm=r.perm[l].cpu().numpy(),
                 loads=loads[l].cpu().numpy(), bin_loads=bins[l].cpu().numpy(),
                 logits=r.logits[l].cpu().numpy(), status=0)
        assert np.isfinite(g["logits"]).all()
        check_against_oracle(g, hb[l], wb[l], bias[l], np.zeros(E, np.int32), k, c, 0.5, 0.5, 1, B,
                             bins0=np.zeros(B, np.int32))


def test_more_layers_than_one_launch_holds(cuda_device):
    """70 layers: the library routes them in groups of 64 layers per launch."""
    import torch

    from paper_2510_03293_b200 import laser

    dev = cuda_device
    Lr, T, d, E, k, c, B = 70, 40, 64, 8, 2, 4, 2
    layers = [layer(T, d, E, seed=300 + l, sigma=0.2) for l in range(Lr)]
    hb = np.stack([x[0] for x in layers]); wb = np.stack([x[1] for x in layers])
    bias = np.stack([x[2] for x in layers])
    eps = [0.55 + 0.002 * l for l in range(Lr)]
    p = laser.make_params(T, d, E, k, c, 0.0, 0.5, 1, B)
    loads = torch.zeros((Lr, E), dtype=torch.int32, device=dev)
    bins = torch.zeros((Lr, B), dtype=torch.int32, device=dev)
    r = laser.route_layers(to_dev_bf16(hb, dev), to_dev_bf16(wb, dev),
                           torch.from_numpy(bias).to(dev), loads, p, bin_loads=bins, eps_high=eps,
                           want_logits=True)
    torch.cuda.synchronize()
    assert int(r.status.item()) == 0
    for l in (0, 1, 63, 64, 69):
        g = dict(expert_ids=r.expert_ids[l].cpu().numpy(), weights=r.weights[l].cpu().numpy(),
                 offsets=r.offsets[l].cpu().numpy(), perm=r.perm[l].cpu().numpy(),
                 loads=loads[l].cpu().numpy(), bin_loads=bins[l].cpu().numpy(),
                 logits=r.logits[l].cpu().numpy(), status=0)
        check_against_oracle(g, hb[l], wb[l], bias[l], np.zeros(E, np.int32), k, c, eps[l], 0.5, 1,
                             B, bins0=np.zeros(B, np.int32))


# ---- relaxed load update (a separate variant; the default everywhere else is the rule) -------
def _run_relaxed(dev, hb, wb, bias, loads0, k, c, eps, tfix, G, B):
    import torch

    from paper_2510_03293_b200 import laser

    T, d = hb.shape
    E = wb.shape[0]
    p = laser.make_params(T, d, E, k, c, eps, tfix, 1, B, update_granularity=G)
    loads = torch.from_numpy(loads0.copy()).to(dev)
    bins = torch.zeros(B, dtype=torch.int32, device=dev)
    r = laser.route(to_dev_bf16(hb, dev), to_dev_bf16(wb, dev), torch.from_numpy(bias).to(dev),
                    loads, p, bin_loads=bins, want_logits=True)
    torch.cuda.synchronize()
    assert int(r.status.item()) == 0
    return r, loads, bins


@pytest.mark.parametrize("router", ["tile", "splitk"])
@pytest.mark.parametrize("T,d,E,k,c,eps,tfix", [
    (1500, 256, 8, 2, 4, 0.7, 0.4),      # E <= 32 path
    (1500, 256, 64, 6, 10, 0.5, 0.4),    # shared-memory masks
    (700, 128, 256, 8, 40, 0.30, 0.10),  # one-warp scan (candidate sets wider than a warp)
])
@pytest.mark.parametrize("G", [0, 32, 96, 256, 1024])
def test_relaxed_granularity_matches_its_oracle(cuda_device, force_router, router, T, d, E, k, c,
                                                eps, tfix, G):
    force_router(router)
    hb, wb, bias = layer(T, d, E, seed=400 + E + G, sigma=0.05)
    loads0 = np.random.default_rng(G + E).integers(0, 4, E).astype(np.int32)
    B = 4
    r, loads, bins = _run_relaxed(cuda_device, hb, wb, bias, loads0, k, c, eps, tfix, G, B)
    x = r.logits.cpu().numpy()
    ref = oracle.route_full(hb, wb, bias, loads0, synth.default_expert_to_bin(E, B),
                            np.zeros(B, np.int32), k, c, eps, tfix, True, x=x, granularity=G)
    assert np.array_equal(r.expert_ids.cpu().numpy(), ref["expert_ids"])
    assert np.array_equal(r.offsets.cpu().numpy(), ref["offsets"])
    assert np.array_equal(r.perm.cpu().numpy(), ref["perm"])
    assert np.array_equal(loads.cpu().numpy(), ref["loads"])
    assert np.array_equal(bins.cpu().numpy(), ref["bin_loads"])
    assert np.array_equal(r.weights.cpu().numpy().view(np.uint32), ref["weights"].view(np.uint32))
    if G in (32, 96):   # the variant really differs from the rule on these inputs
        exact = oracle.route(x, loads0, k, c, eps, tfix, True)
        assert not np.array_equal(exact[0], ref["expert_ids"])


# ---- RANDOM trimming -------------------------------------------------------------------
@pytest.mark.parametrize("router", ["tile", "splitk"])
@pytest.mark.parametrize("T,d,E,k,c,eps,tfix", [
    (900, 256, 8, 2, 3, 0.8, 0.3),       # warp-level / split-K routers
    (900, 256, 64, 6, 8, 0.6, 0.3),      # tensor-memory router, 64 columns
    (600, 128, 100, 5, 12, 0.5, 0.2),    # 128 columns
    (500, 128, 256, 8, 16, 0.3, 0.3),    # 256 columns (two-pass epilogue)
])
def test_random_trimming_matches_its_oracle(cuda_device, force_router, router, T, d, E, k, c, eps,
                                            tfix):
    import torch

    from paper_2510_03293_b200 import laser

    force_router(router)
    dev = cuda_device
    Lr, B, seed = 2, 4, 0xC0FFEE1234
    layers = [layer(T, d, E, seed=500 + l + E, sigma=0.08) for l in range(Lr)]
    hb = np.stack([x[0] for x in layers]); wb = np.stack([x[1] for x in layers])
    bias = np.stack([x[2] for x in layers])
    p = laser.make_params(T, d, E, k, c, eps, tfix, 1, B, trim_mode=1, seed=seed)
    loads = torch.zeros((Lr, E), dtype=torch.int32, device=dev)
    bins = torch.zeros((Lr, B), dtype=torch.int32, device=dev)
    r = laser.route_layers(to_dev_bf16(hb, dev), to_dev_bf16(wb, dev),
                           torch.from_numpy(bias).to(dev), loads, p, bin_loads=bins,
                           want_logits=True)
    torch.cuda.synchronize()
    assert int(r.status.item()) == 0
    trimmed = 0
    for l in range(Lr):
        x = r.logits[l].cpu().numpy()
        ref = oracle.route_full(hb[l], wb[l], bias[l], np.zeros(E, np.int32),
                                synth.default_expert_to_bin(E, B), np.zeros(B, np.int32), k, c,
                                eps, tfix, True, x=x, random_seed=seed, layer=l)
        assert np.array_equal(r.expert_ids[l].cpu().numpy(), ref["expert_ids"]), l
        assert np.array_equal(r.offsets[l].cpu().numpy(), ref["offsets"])
        assert np.array_equal(r.perm[l].cpu().numpy(), ref["perm"])
        assert np.array_equal(loads[l].cpu().numpy(), ref["loads"])
        assert np.array_equal(bins[l].cpu().numpy(), ref["bin_loads"])
        assert np.array_equal(r.weights[l].cpu().numpy().view(np.uint32),
                              ref["weights"].view(np.uint32))
        top = oracle.route(x, np.zeros(E, np.int32), k, c, eps, tfix, True)
        trimmed += int((top[0] != ref["expert_ids"]).any(1).sum())
    assert trimmed > 0   # the sampling really changed assignments on these inputs


def test_imbalance_kernel_matches_the_fp64_figures(cuda_device):
    import torch

    from oracle import alg1_literal as lit
    from paper_2510_03293_b200 import laser

    rng = np.random.default_rng(5)
    for Lr, E, B in [(1, 8, 4), (32, 8, 8), (27, 64, 8), (3, 256, 32), (70, 13, 5)]:
        counts = rng.integers(0, 5000, (Lr, E)).astype(np.int64)
        counts[0, :] = 0 if Lr > 1 else counts[0, :]          # a layer without assignments
        e2b = rng.integers(0, B, E).astype(np.int32)
        e2b[:B] = np.arange(B)
        off = np.zeros((Lr, E + 1), np.int32)
        off[:, 1:] = np.cumsum(counts, 1)
        I, Ib, agg = laser.imbalance(torch.from_numpy(off).to(cuda_device), B,
                                     torch.from_numpy(e2b).to(cuda_device))
        torch.cuda.synchronize()
        ref = lit.imbalance_stats(counts, e2b, B)
        assert np.allclose(I.cpu().numpy(), ref["I"], rtol=2e-6, atol=0)
        assert np.allclose(Ib.cpu().numpy(), ref["I_bins"], rtol=2e-6, atol=0)
        assert abs(float(agg[0]) - ref["I_agg"]) <= 4e-6 * ref["I_agg"]
        assert abs(float(agg[1]) - ref["I_agg_bins"]) <= 4e-6 * ref["I_agg_bins"]
        # general placement: every expert split over two devices, columns summing to 1
        A = np.zeros((B, E), np.float32)
        f = rng.integers(1, 8, E) / 8.0
        A[e2b, np.arange(E)] += f
        A[(e2b + 1) % B, np.arange(E)] += 1.0 - f
        I2, Ib2, agg2 = laser.imbalance(torch.from_numpy(off).to(cuda_device), B,
                                        placement=torch.from_numpy(A).to(cuda_device))
        torch.cuda.synchronize()
        ref2 = lit.imbalance_stats(counts, None, B, A)
        assert np.array_equal(I2.cpu().numpy(), I.cpu().numpy())
        assert np.allclose(Ib2.cpu().numpy(), ref2["I_bins"], rtol=2e-6, atol=0)
        assert abs(float(agg2[1]) - ref2["I_agg_bins"]) <= 4e-6 * ref2["I_agg_bins"]


@pytest.mark.parametrize("T,E,k,near,pmax", [(1, 8, 2, 0.5, 3), (777, 8, 2, 0.5, 3),
                                              (1000, 32, 4, 0.25, 6), (515, 64, 6, 0.3, 8),
                                              (300, 13, 13, 1.0, 1), (260, 200, 8, 0.0, 200),
                                              (129, 256, 8, 0.5, 16)])
def test_score_statistics_match_the_oracle(cuda_device, T, E, k, near, pmax):
    """Integer words (tokens, M_k and s_max sums, regimes, n_near, histogram) bit for bit; the
    entropy sum within T units of 2^-32 for the per-token rounding plus 1e-9 relative for the
    two double-precision logarithms."""
    import torch

    import oracle
    from oracle import score_stats as st
    from paper_2510_03293_b200 import laser

    rng = np.random.default_rng(1000 * E + T)
    Lr = 2
    x = (rng.standard_normal((Lr, T, E)) * rng.choice([0.3, 2.0, 6.0], (Lr, T, 1))).astype(np.float32)
    x[0, 0, :] = 0.0                       # a flat row
    x[-1, -1, :] = 0.0; x[-1, -1, E // 2] = 50.0   # a one-hot row
    xd = torch.from_numpy(x).to(cuda_device)
    stats, means = laser.score_stats(xd, k, near, pmax)
    stats2, means2 = laser.score_stats(xd, k, near, pmax, stats=stats.clone())
    torch.cuda.synchronize()
    got, got2 = stats.cpu().numpy(), stats2.cpu().numpy()
    assert np.array_equal(got2, 2 * got)       # accumulation over two batches
    for l in range(Lr):
        ref = st.score_stats(x[l], oracle.softmax(x[l]), k, near, pmax)
        g = got[l]
        assert g[0] == T
        assert g[1] == round(ref["mass_sum"] * 2**32) and g[7] == round(ref["smax_sum"] * 2**32)
        assert abs(int(g[2]) - ref["entropy_sum"] * 2**32) <= T + 1e-9 * ref["entropy_sum"] * 2**32 + 1
        assert g[3:6].tolist() == ref["regimes"] and g[6] == ref["near_sum"]
        assert g[8:].tolist() == ref["mass_hist"]
        m = means.cpu().numpy()[l]
        want = [ref["mean_mass"], ref["mean_entropy"], ref["mean_smax"], ref["mean_near"]]
        assert np.allclose(m, want, rtol=3e-7, atol=1e-9)
    assert np.array_equal(means.cpu().numpy(), means2.cpu().numpy())


@pytest.mark.parametrize("router", ["tile", "splitk"])
def test_id_and_weight_arrays_on_4_byte_boundaries(cuda_device, force_router, router):
    """The caller's id and weight arrays only have to be 4-byte aligned: the tensor-memory
    router's 8-byte record stores must not be used then, and the results must not change."""
    force_router(router)
    hb, wb, bias = layer(700, 512, 64, seed=31)
    z = np.zeros(64, np.int32)
    a = run_gpu(cuda_device, hb, wb, bias, z, 6, 8, 0.4, 0.8)
    b = run_gpu(cuda_device, hb, wb, bias, z, 6, 8, 0.4, 0.8, skew=1)
    for name in ("expert_ids", "weights", "offsets", "perm", "loads"):
        assert np.array_equal(a[name], b[name]), name
    check_against_oracle(b, hb, wb, bias, z, 6, 8, 0.4, 0.8)
