"""Helpers shared by the GPU parity tests: run one routing call through the C ABI with
canary-padded outputs and compare it with the CPU oracle fed the GPU's own fp32 logits."""
import numpy as np

import oracle
from paper_2510_03293_b200 import synth

CANARY_I = -1234567
CANARY_F = 1.0e30
PAD = 64


def to_dev_bf16(bits, dev):
    import torch

    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(dev).view(torch.bfloat16)


class Padded:
    """A device tensor with PAD sentinel elements on both sides of the payload."""

    def __init__(self, shape, dtype, dev, fill, skew=0):
        import torch

        n = int(np.prod(shape)) if len(shape) else 1
        self.fill = fill
        self.buf = torch.full((n + 2 * PAD + skew,), fill, dtype=dtype, device=dev)
        # skew = 1 puts a 4-byte type on an address that is not a multiple of 8
        self.view = self.buf[PAD + skew:PAD + skew + n].view(*shape)

    def intact(self):
        b = self.buf
        lo = self.view.data_ptr() - b.data_ptr()
        lo //= b.element_size()
        return bool((b[:lo] == self.fill).all().item() and
                    (b[lo + self.view.numel():] == self.fill).all().item())


def run_gpu(dev, hb, wb, bias, loads0, k, c, eps, tfix, renorm=1, n_bins=1, e2b=None,
            bins0=None, want_logits=True, skew=0, fresh=0):
    """One laser_route call; returns dict of numpy outputs.  Checks the canaries."""
    import torch

    from paper_2510_03293_b200 import laser

    T, d = hb.shape
    E = wb.shape[0]
    p = laser.make_params(T, d, E, k, c, eps, tfix, renorm, n_bins, fresh_loads=fresh)
    hidden = to_dev_bf16(hb, dev) if T > 0 else torch.empty((0, d), dtype=torch.bfloat16, device=dev)
    wg = to_dev_bf16(wb, dev)
    loads = torch.from_numpy(np.asarray(loads0, np.int32).copy()).to(dev)
    bins = None if bins0 is None else torch.from_numpy(np.asarray(bins0, np.int32).copy()).to(dev)
    pads = dict(
        ids=Padded((1, T, k), torch.int32, dev, CANARY_I, skew),
        w=Padded((1, T, k), torch.float32, dev, CANARY_F, skew),
        off=Padded((1, E + 1), torch.int32, dev, CANARY_I),
        perm=Padded((1, T * k), torch.int32, dev, CANARY_I),
        logits=Padded((1, T, E), torch.float32, dev, CANARY_F),
    )
    out = laser.RouteResult(pads["ids"].view, pads["w"].view, pads["off"].view, pads["perm"].view,
                            loads, bins, pads["logits"].view if want_logits else None,
                            torch.zeros((1,), dtype=torch.int32, device=dev))
    laser.route_layers(hidden[None], wg[None],
                       None if bias is None else torch.from_numpy(bias).to(dev)[None],
                       loads[None], p,
                       expert_to_bin=None if e2b is None else torch.from_numpy(e2b).to(dev),
                       bin_loads=None if bins is None else bins[None], out=out)
    torch.cuda.synchronize()
    for name, pd in pads.items():
        assert pd.intact(), f"canary around {name} overwritten"
    return dict(expert_ids=out.expert_ids[0].cpu().numpy(), weights=out.weights[0].cpu().numpy(),
                offsets=out.offsets[0].cpu().numpy(), perm=out.perm[0].cpu().numpy(),
                loads=loads.cpu().numpy(), bin_loads=None if bins is None else bins.cpu().numpy(),
                logits=out.logits[0].cpu().numpy() if want_logits else None,
                status=int(out.status.item()))


def check_against_oracle(g, hb, wb, bias, loads0, k, c, eps, tfix, renorm=1, n_bins=1,
                         e2b=None, bins0=None, logit_tol=1e-3):
    """Bit-exact ids / weights / offsets / perm / loads / bins given the GPU's fp32 logits;
    logits within logit_tol (max abs) of the fp64-accumulated oracle logits."""
    T, E = hb.shape[0], wb.shape[0]
    if T > 0:
        x_ref = oracle.logits(hb, wb, bias)
        err = float(np.max(np.abs(g["logits"] - x_ref)))
        assert err <= logit_tol, f"logits max abs err {err}"
    if e2b is None:
        e2b = synth.default_expert_to_bin(E, n_bins)
    ref = oracle.route_full(hb, wb, bias, np.asarray(loads0, np.int32), e2b,
                            None if bins0 is None else np.asarray(bins0, np.int32),
                            k, c, eps, tfix, bool(renorm),
                            x=g["logits"] if T > 0 else np.zeros((0, E), np.float32))
    for name in ("expert_ids", "offsets", "perm", "loads"):
        assert np.array_equal(g[name], ref[name]), f"{name} differs from the oracle"
    assert np.array_equal(g["weights"].view(np.uint32), ref["weights"].view(np.uint32)), "weights differ"
    if bins0 is not None:
        assert np.array_equal(g["bin_loads"], ref["bin_loads"]), "bin_loads differ"
    assert g["status"] == 0
    return ref
