"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times (all
layers of a workload in one laser_route_layers call, inputs generated on the device).

Every integer output and the weights are compared with the CPU oracle fed the GPU's fp32
logits, for every layer and token; the logits themselves are checked on sampled rows against
the oracle's fp64-accumulated contraction (the full contraction would take the CPU minutes)."""
import numpy as np
import pytest

import oracle
from paper_2510_03293_b200 import synth

pytestmark = pytest.mark.gpu


def run_workload(dev, name, layers=None, sample_rows=48):
    import torch

    from paper_2510_03293_b200 import laser

    w = synth.WORKLOADS[name]
    L = w.layers if layers is None else layers
    data = synth.make_workload_torch(w, dev, seed=3, layers=L)
    p = laser.make_params(w.T, w.d, w.E, w.k, w.c, w.eps_high[0], w.t_fix, w.renormalize, w.n_bins)
    loads = torch.zeros((L, w.E), dtype=torch.int32, device=dev)
    bins = torch.zeros((L, w.n_bins), dtype=torch.int32, device=dev)
    r = laser.route_layers(data["hidden"], data["w_g"], data["bias"], loads, p, bin_loads=bins,
                           eps_high=data["eps_high"], t_fix=data["t_fix"], want_logits=True)
    torch.cuda.synchronize()
    assert int(r.status.item()) == 0
    e2b = synth.default_expert_to_bin(w.E, w.n_bins)
    rng = np.random.default_rng(11)
    expanded = differs = 0
    for l in range(L):
        x = r.logits[l].cpu().numpy()
        ref = oracle.route_full(None, None, None, np.zeros(w.E, np.int32), e2b,
                                np.zeros(w.n_bins, np.int32), w.k, w.c, data["eps_high"][l],
                                data["t_fix"][l], bool(w.renormalize), x=x)
        assert np.array_equal(r.expert_ids[l].cpu().numpy(), ref["expert_ids"]), (name, l)
        assert np.array_equal(r.offsets[l].cpu().numpy(), ref["offsets"]), (name, l)
        assert np.array_equal(r.perm[l].cpu().numpy(), ref["perm"]), (name, l)
        assert np.array_equal(loads[l].cpu().numpy(), ref["loads"]), (name, l)
        assert np.array_equal(bins[l].cpu().numpy(), ref["bin_loads"]), (name, l)
        assert np.array_equal(r.weights[l].cpu().numpy().view(np.uint32),
                              ref["weights"].view(np.uint32)), (name, l)
        expanded += int((ref["cstar"] > 0).sum())
        differs += int((np.sort(ref["expert_ids"], 1) != np.sort(oracle.topk(x, w.k), 1)).any(1).sum())
        # sampled rows of the contraction, including the first and last token and tile edges
        rows = np.unique(np.concatenate([[0, 127, 128, w.T - 129, w.T - 1],
                                         rng.integers(0, w.T, sample_rows)]))
        rows_t = torch.from_numpy(rows).to(dev)
        hb = data["hidden"][l].index_select(0, rows_t).view(torch.int16).cpu().numpy().view(np.uint16)
        wb = data["w_g"][l].view(torch.int16).cpu().numpy().view(np.uint16)
        x_ref = oracle.logits(hb, wb, data["bias"][l].cpu().numpy())
        err = float(np.max(np.abs(x[rows] - x_ref)))
        assert err <= 1e-3, (name, l, err)
    # both branches of the rule were exercised at this size
    assert 0 < expanded < L * w.T and differs > 0


def test_mixtral_shaped_all_layers(cuda_device):
    run_workload(cuda_device, "mixtral")


def test_deepseek_shaped_all_layers(cuda_device):
    run_workload(cuda_device, "deepseek")


def test_tiny(cuda_device):
    run_workload(cuda_device, "tiny", sample_rows=256)


def test_stress_shape(cuda_device):
    run_workload(cuda_device, "stress", sample_rows=32)


def test_decode_stream_carries_loads(cuda_device):
    """64-token steps with the load state carried from step to step give the same assignments
    as one call over the concatenated tokens (per-token load updates make this exact)."""
    import torch

    from paper_2510_03293_b200 import laser

    dev = cuda_device
    w = synth.WORKLOADS["decode"]
    steps = 24
    data = synth.make_workload_torch(w, dev, seed=5, layers=steps)
    wg, bias = data["w_g"][:1].contiguous(), data["bias"][:1].contiguous()
    p = laser.make_params(w.T, w.d, w.E, w.k, w.c, w.eps_high[0], w.t_fix, w.renormalize, w.n_bins)
    loads = torch.zeros((1, w.E), dtype=torch.int32, device=dev)
    ids = []
    for s in range(steps):
        r = laser.route_layers(data["hidden"][s:s + 1], wg, bias, loads, p)
        ids.append(r.expert_ids[0].clone())
    torch.cuda.synchronize()
    p_all = laser.make_params(w.T * steps, w.d, w.E, w.k, w.c, w.eps_high[0], w.t_fix,
                              w.renormalize, w.n_bins)
    loads_all = torch.zeros((1, w.E), dtype=torch.int32, device=dev)
    r_all = laser.route_layers(data["hidden"].reshape(1, steps * w.T, w.d), wg, bias, loads_all,
                               p_all, want_logits=True)
    torch.cuda.synchronize()
    assert torch.equal(torch.cat(ids, 0), r_all.expert_ids[0])
    assert torch.equal(loads, loads_all)
    ref = oracle.route(r_all.logits[0].cpu().numpy(), np.zeros(w.E, np.int32), w.k, w.c,
                       w.eps_high[0], w.t_fix, bool(w.renormalize))
    assert np.array_equal(r_all.expert_ids[0].cpu().numpy(), ref[0])
    assert np.array_equal(loads_all[0].cpu().numpy(), ref[2])
