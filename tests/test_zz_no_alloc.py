"""laser_route_static, the entry point for callers that cannot allocate device memory (its
scratch is an array inside the library), must give exactly what laser_route gives.

The file name sorts last on purpose: a run that stops at the first failure has then already
run every other test.  Two calls in a row are checked, the second on a smaller, different
problem, so that what the first call left behind in the shared scratch array is still there
when the second one starts."""
import numpy as np
import pytest

from paper_2510_03293_b200 import synth
from gpu_util import run_gpu, to_dev_bf16

pytestmark = pytest.mark.gpu


def route_static_once(dev, hb, wb, bias, loads0, bins0, k, c, eps, tfix, renorm, n_bins):
    import torch

    from paper_2510_03293_b200 import laser

    T, d = hb.shape
    E = wb.shape[0]
    p = laser.make_params(T, d, E, k, c, eps, tfix, renorm, n_bins)
    loads = torch.from_numpy(loads0.copy()).to(dev)
    bins = torch.from_numpy(bins0.copy()).to(dev)
    out = laser.RouteResult(
        torch.full((T, k), -7, dtype=torch.int32, device=dev),
        torch.full((T, k), -7.0, dtype=torch.float32, device=dev),
        torch.full((E + 1,), -7, dtype=torch.int32, device=dev),
        torch.full((T * k,), -7, dtype=torch.int32, device=dev),
        loads, bins,
        torch.full((T, E), -7.0, dtype=torch.float32, device=dev),
        torch.zeros((1,), dtype=torch.int32, device=dev))
    hidden, wg, bias_d = to_dev_bf16(hb, dev), to_dev_bf16(wb, dev), torch.from_numpy(bias).to(dev)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info(dev)[0]      # the driver's own count of free bytes
    laser.route_static(hidden, wg, bias_d, loads, p, out, bin_loads=bins)
    torch.cuda.synchronize()
    free_after = torch.cuda.mem_get_info(dev)[0]
    return dict(free_before=free_before, free_after=free_after,
                expert_ids=out.expert_ids.cpu().numpy(), weights=out.weights.cpu().numpy(),
                offsets=out.offsets.cpu().numpy(), perm=out.perm.cpu().numpy(),
                loads=loads.cpu().numpy(), bin_loads=bins.cpu().numpy(),
                logits=out.logits.cpu().numpy(), status=int(out.status.item()))


def test_static_scratch_entry_matches_laser_route_twice_in_a_row(cuda_device):
    dev = cuda_device
    calls = [
        # T, d, E, k, c, eps, tfix, renorm, bins
        (3000, 512, 64, 6, 8, 0.40, 0.80, 0, 8),
        (777, 1024, 8, 2, 4, 0.6419, 0.60, 1, 4),
    ]
    for i, (T, d, E, k, c, eps, tfix, renorm, B) in enumerate(calls):
        hb, wb, bias = synth.make_layer(T, d, E, 0.02, 1.2, seed=900 + i, stream=3)
        rng = np.random.default_rng(77 + i)
        loads0 = rng.integers(0, 4, E).astype(np.int32)
        bins0 = rng.integers(0, 9, B).astype(np.int32)
        got = route_static_once(dev, hb, wb, bias, loads0, bins0, k, c, eps, tfix, renorm, B)
        want = run_gpu(dev, hb, wb, bias, loads0, k, c, eps, tfix, renorm, B, bins0=bins0)
        assert got["status"] == 0 and want["status"] == 0
        # the same kernels on the same inputs: every output agrees bit for bit
        for name in ("expert_ids", "offsets", "perm", "loads", "bin_loads"):
            assert np.array_equal(got[name], want[name]), (i, name)
        assert np.array_equal(got["weights"].view(np.uint32), want["weights"].view(np.uint32))
        assert np.array_equal(got["logits"].view(np.uint32), want["logits"].view(np.uint32))
        assert int(got["offsets"][-1]) == T * k
        if i > 0:
            # nothing was allocated or freed on the device by the call itself (the first call
            # on a device may still load the kernels' code, so only later calls are held to it)
            assert got["free_after"] == got["free_before"], (got["free_before"], got["free_after"])


def test_static_scratch_entry_refuses_shapes_beyond_its_array(cuda_device):
    import torch

    from paper_2510_03293_b200 import laser

    p = laser.make_params(131072, 256, 256, 8, 16, 0.3, 0.25, 1, 32)
    assert laser.workspace_bytes(p) > laser.STATIC_SCRATCH_BYTES
    dummy = torch.zeros((64,), dtype=torch.int32, device=cuda_device)
    out = laser.RouteResult(dummy, dummy, dummy, dummy, dummy, None, None, dummy)
    with pytest.raises(laser.LaserError) as e:
        laser.route_static(dummy, dummy, None, dummy, p, out)
    assert e.value.status == laser.ERR_STATIC_SCRATCH
    assert int(dummy.abs().sum().item()) == 0      # nothing was launched, nothing written
