#!/usr/bin/env python
"""Benchmark of the LASER routing path: routed tokens/s for router + LASER + dispatch.

A step is one pass of the whole path (router contraction, score epilogue, ordered load-aware
selection, load update, dispatch, bin accounting) over every layer of the Mixtral-8x7B-shaped
workload: 32 independent MoE layers x 16384 tokens, d=4096 bf16, E=8, k=2, loads reset per
step.  Inputs are seeded synthetic tensors (4.3 GB of hidden states, larger than L2).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints one JSON line.  Without --workload the line is the Mixtral-shaped workload's, and its
"workloads" key carries the same measurements for the other four shapes (tiny, DeepSeek-shaped,
decode stream, E = 256 stress), each with its roofline fraction, routing statistics and the
agreement with the CPU oracle run on its own logits.  With --impl reference the CPU oracle is
timed on the host cores on a bounded sample of the same workload.  --workload decode runs the
decode stream (4096 successive 64-token calls with the load state carried along) as one replayed
CUDA graph and reports the latency per call.  --gpus N without a torchrun environment starts N
replica processes itself.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "routed tokens/sec per B200 (router+LASER+dispatch)"
UNIT = "tokens/s"


def measured_peak_hbm():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def algorithmic_bytes_per_token(w) -> float:
    """Bytes the method must move per token: the bf16 hidden row, k x (id, weight, perm entry)
    and the amortised W_g."""
    return 2.0 * w.d + 12.0 * w.k + 2.0 * w.E * w.d / w.T


def workload_config(w, n_layers, n_copies=1):
    gb = 2.0 * n_layers * w.T * w.d / 1e9
    cache = ("inputs (%.2f GB per step) exceed the 126 MB L2" % gb) if n_copies == 1 else \
        ("inputs (%.3f GB per step) rotate over %d copies (%.2f GB), more than twice the 126 MB L2"
         % (gb, n_copies, gb * n_copies))
    return {"workload": "%s: %d layers x T=%d, d=%d bf16, E=%d, k=%d, c=%d, %d bins" %
            (w.name, n_layers, w.T, w.d, w.E, w.k, w.c, w.n_bins),
            "tokens_per_step": n_layers * w.T, "t_fix": w.t_fix, "eps_high": list(w.eps_high),
            "cache": cache}


DECODE_NODES_PER_CALL = 1   # calls of at most 112 tokens: one kernel (a thread-block cluster per layer)


def launches_per_step(w, L) -> int:
    """Kernels the library enqueues per step, per group of at most 64 layers: the fused
    router + selection kernel and the dispatch kernel (calls of at most 512 tokens have their
    dispatch done inside the first kernel)."""
    return (1 if w.T <= 512 else 2) * ((L + 63) // 64)


def kernel_sources_digest() -> str:
    """Digest of the CUDA sources: DRAM counters taken with ncu only describe the kernels they
    were taken from."""
    import hashlib

    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2510_03293_b200", "csrc")
    for name in sorted(os.listdir(csrc)):
        with open(os.path.join(csrc, name), "rb") as f:
            h.update(name.encode()); h.update(f.read())
    return h.hexdigest()[:16]


def recorded_traffic(workload: str, tokens: int):
    """DRAM bytes (read + write) per launch of the router + selection kernel from the ncu
    capture summarised under profiles/, scaled by tokens; None if the kernels have changed
    since the capture or no capture exists for this workload."""
    try:
        with open(os.path.join(ROOT, "profiles", "dram_traffic.json")) as f:
            rec = json.load(f)
        if rec.get("sources_digest") != kernel_sources_digest():
            return None
        return rec["workloads"][workload]["dram_bytes_per_token"] * tokens
    except Exception:
        return None


def router_kernel_name(w, L) -> str:
    if L * ((w.T + 127) // 128) * 4 <= 148:
        return "k12_route_select_splitk (split-K contraction + score epilogue + ordered selection)"
    if 32 < w.E <= 64:
        return ("k12_route_select_tcp (persistent tcgen05 contraction + score epilogue + ordered "
                "selection)")
    if w.E > 64:
        return "k12_route_select_tc (tcgen05 contraction + score epilogue + ordered selection)"
    return "k12_route_select (mma.sync contraction + score epilogue + ordered selection)"


# --------------------------------------------------------------------------- CPU oracle arm
def oracle_pass(oracle, np, layers_data, w, eps, tfix):
    """The oracle's whole path on a list of (hidden_bits, wg_bits, bias) layers."""
    from paper_2510_03293_b200 import synth

    e2b = synth.default_expert_to_bin(w.E, w.n_bins)
    t0 = time.perf_counter()
    for l, (hb, wb, bias) in enumerate(layers_data):
        oracle.route_full(hb, wb, bias, np.zeros(w.E, np.int32), e2b, np.zeros(w.n_bins, np.int32),
                          w.k, w.c, eps[l], tfix[l], bool(w.renormalize))
    return time.perf_counter() - t0


def run_reference(args, w):
    import numpy as np

    import oracle
    from paper_2510_03293_b200 import synth

    if int(os.environ.get("RANK", "0")) != 0:
        return
    oracle.build()
    n_sample = min(w.layers, args.ref_layers)
    data = [synth.make_workload_layer(w, l) for l in range(n_sample)]
    eps = [w.eps_for_layer(l) for l in range(n_sample)]
    tfix = [w.t_fix] * n_sample
    for _ in range(args.warmup):
        oracle_pass(oracle, np, data[:1], w, eps, tfix)
    times = [oracle_pass(oracle, np, data, w, eps, tfix) for _ in range(args.steps)]
    sec = sum(times) / len(times)
    value = n_sample * w.T / sec
    cores = len(os.sched_getaffinity(0))
    sample = "%d of %d layers per step (%d tokens)" % (n_sample, w.layers, n_sample * w.T)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": workload_config(w, n_sample),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "100"], stdout=fd,
                stderr=subprocess.DEVNULL)
            os.close(fd)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        try:
            rows = [r.strip().split(", ") for r in open(self.path) if r.strip()]
            os.unlink(self.path)
        except Exception:
            return out
        sm, reasons, mx = [], set(), None
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1])); mx = float(r[2])
            except ValueError:
                continue
            for name, v in zip(names, r[5:9]):
                if v.strip().lower() == "active":
                    reasons.add(name)
        if sm:
            sm.sort()
            out.update(sm_mhz=sm[len(sm) // 2], sm_max_mhz=mx, reasons=sorted(reasons),
                       samples=len(sm))
        return out


# --------------------------------------------------------------------------- GPU arm
def aggregate_replicas(total_ms, steps, tokens_per_rank, dist, device):
    """Whole-job numbers of N independent replicas (the path does not shard: tokens of a layer
    form one dependency chain).  Time is the MAX over ranks, throughput the tokens of all ranks
    over that time.  Returns (ms_per_step, tokens_per_second)."""
    world = 1
    if dist is not None:
        import torch

        t = torch.tensor([float(total_ms)], device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
        world = dist.get_world_size()
    ms_per_step = total_ms / steps
    return ms_per_step, world * tokens_per_rank / (ms_per_step * 1e-3)


class Context:
    """Rank, device and (for N > 1 replicas) the process group of this process."""

    def __init__(self):
        import torch

        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        torch.cuda.set_device(self.local)
        self.dev = torch.device("cuda", self.local)
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            dist.init_process_group("nccl", device_id=self.dev)
            self.dist = dist

    def barrier(self):
        import torch

        if self.dist is not None:
            self.dist.barrier()
        torch.cuda.synchronize()

    def close(self):
        if self.dist is not None:
            self.dist.barrier()
            self.dist.destroy_process_group()


def new_events(torch, n):
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(n)]
    for e in evs:
        e.record()
    return evs


def percentile(v, q):
    s = sorted(v)
    pos = (len(s) - 1) * q
    lo = int(pos)
    hi = min(lo + 1, len(s) - 1)
    return s[lo] + (s[hi] - s[lo]) * (pos - lo)


def run_layers(args, w, ctx, full):
    """One workload of independent layers.  full: also the end-to-end leg, the CPU baseline
    leg and the sustained loop (the headline workload); otherwise the device-timed figures,
    the routing statistics and the oracle sample only."""
    import numpy as np
    import torch

    from paper_2510_03293_b200 import laser, synth

    dev, dist, rank, world = ctx.dev, ctx.dist, ctx.rank, ctx.world
    L = w.layers if args.layers is None else args.layers
    data = synth.make_workload_torch(w, dev, seed=args.seed + rank, layers=L)
    p = laser.make_params(w.T, w.d, w.E, w.k, w.c, w.eps_high[0], w.t_fix, w.renormalize, w.n_bins,
                          update_granularity=args.granularity,
                          trim_mode=0 if args.random_trim is None else 1,
                          seed=args.random_trim or 0, fresh_loads=1)
    # every step starts from empty load counters (the method resets the loads per batch): the
    # call itself does that (fresh_loads), no memset between steps
    state = torch.zeros((L * (w.E + w.n_bins),), dtype=torch.int32, device=dev)
    loads = state[:L * w.E].view(L, w.E)
    bins = state[L * w.E:].view(L, w.n_bins)
    ws = torch.empty((laser.workspace_bytes(p) * L,), dtype=torch.uint8, device=dev)
    out = None
    exact_ids = exact_imb = None
    if args.granularity != 1:
        # the rule's own result on the same inputs, to report how far the variant drifts
        p1 = laser.make_params(w.T, w.d, w.E, w.k, w.c, w.eps_high[0], w.t_fix, w.renormalize,
                               w.n_bins)
        r1 = laser.route_layers(data["hidden"], data["w_g"], data["bias"], loads, p1,
                                bin_loads=bins, eps_high=data["eps_high"], t_fix=data["t_fix"],
                                workspace=ws)
        torch.cuda.synchronize()
        exact_ids = r1.expert_ids.sort(dim=2).values.clone()
        c1 = (r1.offsets[:, 1:] - r1.offsets[:, :-1]).double()
        exact_imb = float((c1.max(1).values / c1.mean(1)).mean().item())
        del r1

    # inputs that fit the 126 MB L2 are rotated over enough copies to exceed twice its size
    in_bytes = data["hidden"].numel() * 2
    n_copies = 1 if in_bytes > (256 << 20) else -(-(256 << 20) // in_bytes)
    hiddens = [data["hidden"]] + [data["hidden"].clone() for _ in range(n_copies - 1)]
    it = 0

    def step(events=None, eps=None):
        nonlocal out, it
        out = laser.route_layers(hiddens[it % n_copies], data["w_g"], data["bias"], loads, p,
                                 bin_loads=bins, eps_high=data["eps_high"] if eps is None else eps,
                                 t_fix=data["t_fix"], out=out, workspace=ws, stage_events=events)
        it += 1

    def timed_steps(n, eps=None, all_stages=False):
        """n steps with their stage events; returns (total ms, per-step stage events).  The
        timed region brackets only the router + selection kernel (events 1 and 2): every event
        in the stream keeps the next launch from overlapping the end of the previous one."""
        stage = [new_events(torch, 4) for _ in range(n)]
        if not all_stages:
            stage = [[None, ev[1], ev[2], None] for ev in stage]
        t_begin, t_end = new_events(torch, 2)
        ctx.barrier()
        t_begin.record()
        for i in range(n):
            step(stage[i], eps)
        t_end.record()
        ctx.barrier()
        return t_begin.elapsed_time(t_end), stage

    warm = max(3, args.warmup)
    for _ in range(warm):
        step()
    sampler = ClockSampler(ctx.local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    total_ms, stage = timed_steps(args.steps)
    clocks = sampler.stop() if rank == 0 else None
    tokens = L * w.T
    ms_per_step, value = aggregate_replicas(total_ms, args.steps, tokens, dist, dev)

    k1 = sum(ev[1].elapsed_time(ev[2]) for ev in stage) / args.steps
    # the other stages from a second pass with all four events (not the timed region)
    _, stage4 = timed_steps(args.steps, all_stages=True)
    clear = sum(ev[0].elapsed_time(ev[1]) for ev in stage4) / args.steps
    k3 = sum(ev[2].elapsed_time(ev[3]) for ev in stage4) / args.steps
    peak, peak_kind = measured_peak_hbm()
    bytes_per_launch = algorithmic_bytes_per_token(w) * tokens
    achieved = bytes_per_launch / (k1 * 1e-3) / 1e9
    path_gbs = bytes_per_launch / (ms_per_step * 1e-3) / 1e9

    status = int(out.status.item())
    I_layers, I_bins, I_agg = laser.imbalance(out.offsets, w.n_bins)
    imb = float(I_layers.double().mean().item())

    result = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": warm, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "accumulate": "f32 (logits, scores and weights in f32; ids, loads, dispatch in int32)",
        "data": "synthetic", "config": workload_config(w, L, n_copies),
        "roofline": {"bound": "hbm", "kernel": router_kernel_name(w, L),
                     "achieved": achieved, "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": recorded_traffic(w.name, tokens),
                     "bytes_per_launch": bytes_per_launch},
        "path": {"flags_clear_ms": clear, "router_select_ms": k1, "dispatch_ms": k3,
                 "path_gbs": path_gbs, "path_frac_of_hbm_peak": path_gbs / peak,
                 "path_frac_of_8tbs": path_gbs / 8000.0,
                 "events": "router_select_ms from events inside the timed steps; flags_clear_ms "
                           "and dispatch_ms from a second pass of as many steps with all four "
                           "stage events; path_* from ms_per_step"},
        "routing": {"mean_imbalance_max_over_mean": imb, "I_agg": float(I_agg[0].item()),
                    "I_agg_bins": float(I_agg[1].item()),
                    "MV_max_over_layers": float(I_layers.max().item()) - 1.0,
                    "status_word": status},
        "trimming": "TOP" if args.random_trim is None else "RANDOM (Philox4x32-10, seed %d)" %
                    args.random_trim,
        "variant": ("the method's rule: loads updated after every token" if args.granularity == 1
                    else "RELAXED, not the method's rule: loads seen refreshed every %s tokens"
                    % (args.granularity or "call (snapshot)")),
        "gpu_launches": launches_per_step(w, L) * args.steps,
        "clocks": clocks,
    }

    plain = args.granularity == 1 and args.random_trim is None
    if plain and world == 1:
        # the same launch with every token on the top-k branch (eps_high = 0): what the router,
        # the score epilogue and the bookkeeping of the selection cost when nothing is decided
        n0 = max(3, min(args.steps, 8))
        zero = [0.0] * L
        for _ in range(2):
            step(eps=zero)
        _, st0 = timed_steps(n0, zero)
        k1_0 = sum(ev[1].elapsed_time(ev[2]) for ev in st0) / n0
        step()                       # leave the outputs of the rule itself behind
        torch.cuda.synchronize()
        result["selection"] = {
            "router_select_ms_without_decisions": k1_0,
            "kernel_ns_per_token_of_a_layer": k1 * 1e6 / w.T,
            "budget_ns_per_token_at_70pct_of_hbm_peak":
                bytes_per_launch / (0.7 * peak * 1e9) * 1e9 / w.T,
            "note": "the ordered selection is one dependency chain per layer, all layers "
                    "concurrent and overlapped with the router: kernel time / tokens of a layer "
                    "bounds a chain step from above"}

    # end to end through the host-buffer entry point: H2D of the inputs, D2H of the results
    if full and rank == 0:
        result["e2e"] = e2e_host(args, w, L, data, p, laser, torch, dev)
    if rank == 0 and world == 1 and not args.no_cpu_baseline and plain:
        base = cpu_baseline_and_agreement(args, w, L, data, np, torch, laser, synth, dev, full)
        if full:
            result["cpu_baseline"] = base.pop("cpu_baseline")
        else:
            result["cpu_oracle_sample"] = base.pop("cpu_baseline")
        result["routing"].update(base.pop("routing"))
        result["agreement"] = base.pop("agreement")
        if "selection" in result:
            nd = result["routing"]["decision_tokens_frac"] * w.T
            result["selection"]["decision_tokens_per_layer"] = nd
            if nd > 0:
                result["selection"]["extra_ns_per_decision_token"] = \
                    max(0.0, k1 - result["selection"]["router_select_ms_without_decisions"]) * 1e6 / nd
    if full and rank == 0 and world == 1 and args.sustained_seconds > 0:
        n = max(args.steps, int(args.sustained_seconds * 1e3 / ms_per_step) + 1)
        sampler = ClockSampler(ctx.local)
        sampler.start()
        time.sleep(0.2)
        e0, e1 = new_events(torch, 2)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(n):
            step()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / n
        result["sustained"] = {"steps": n, "seconds": ms * n * 1e-3, "ms_per_step": ms,
                               "value": tokens / (ms * 1e-3),
                               "path_frac_of_hbm_peak": bytes_per_launch / (ms * 1e-3) / 1e9 / peak,
                               "clocks": sampler.stop()}
    if args.imbalance_batches > 0 and rank == 0:
        result["imbalance_study"] = imbalance_study(args, w, L, data, laser, synth, torch, dev,
                                                    loads, bins, ws)
    if args.score_stats and rank == 0:
        result["score_stats"] = score_stats_report(args, w, L, data, p, laser, torch, loads, bins,
                                                   ws)
    if exact_ids is not None:
        same = (out.expert_ids.sort(dim=2).values == exact_ids).all(dim=2)
        result["drift_from_the_rule"] = {
            "tokens_with_a_different_expert_set": float(1.0 - same.double().mean().item()),
            "mean_imbalance_of_the_rule": exact_imb, "mean_imbalance_of_this_variant": imb}
    del data, hiddens, out, ws, state
    torch.cuda.empty_cache()
    return result


def imbalance_study(args, w, L, data, laser, synth, torch, dev, loads, bins, ws):
    """The evaluation's balance figures over several batches: I_agg (P50 and P95 over batches) and
    MV (mean over layers and batches of I_L - 1), for the method next to its two baselines --
    plain top-k (eps_high = 0: every token takes the top-k branch) and load-only (eps_high > 1,
    t_fix = 0, c = E: every expert is a candidate, chosen by load alone).  Same gate weights,
    a fresh seeded batch of hidden states each time, loads starting from zero; the figures come
    from the imbalance kernel, the percentiles from the B values it returned."""
    policies = {
        "laser": dict(c=w.c, eps=data["eps_high"], tfix=data["t_fix"]),
        "top_k": dict(c=w.c, eps=[0.0] * L, tfix=data["t_fix"]),
        "load_only": dict(c=w.E, eps=[2.0] * L, tfix=[0.0] * L),
    }
    agg = {name: [] for name in policies}
    agg_bins = {name: [] for name in policies}
    mv = {name: [] for name in policies}
    ws_lo = None
    for b in range(args.imbalance_batches):
        hidden = synth.make_workload_torch(w, dev, seed=args.seed + 7919 * (b + 1),
                                           layers=L)["hidden"]
        for name, pol in policies.items():
            p = laser.make_params(w.T, w.d, w.E, w.k, pol["c"], pol["eps"][0], pol["tfix"][0],
                                  w.renormalize, w.n_bins)
            if pol["c"] != w.c and ws_lo is None:
                ws_lo = torch.empty((laser.workspace_bytes(p) * L,), dtype=torch.uint8, device=dev)
            loads.zero_(); bins.zero_()
            r = laser.route_layers(hidden, data["w_g"], data["bias"], loads, p, bin_loads=bins,
                                   eps_high=pol["eps"], t_fix=pol["tfix"],
                                   workspace=ws if pol["c"] == w.c else ws_lo)
            I, Ib, a = laser.imbalance(r.offsets, w.n_bins)
            torch.cuda.synchronize()
            agg[name].append(float(a[0].item()))
            agg_bins[name].append(float(a[1].item()))
            mv[name].append(float((I.double() - 1.0).mean().item()))
            del r
        del hidden

    def pct(v, q):
        s = sorted(v)
        pos = (len(s) - 1) * q
        lo = int(pos)
        hi = min(lo + 1, len(s) - 1)
        return s[lo] + (s[hi] - s[lo]) * (pos - lo)

    return {"batches": args.imbalance_batches,
            "policies": {name: {"I_agg_P50": pct(agg[name], 0.5), "I_agg_P95": pct(agg[name], 0.95),
                                "I_agg_bins_P50": pct(agg_bins[name], 0.5),
                                "MV_mean": sum(mv[name]) / len(mv[name])}
                         for name in policies}}


def score_stats_report(args, w, L, data, p, laser, torch, loads, bins, ws):
    """Gate-score statistics of the batch by layer band (thirds of the layer index): mean M_k,
    mean entropy, regime shares, and the M_k median read off the histogram -- the figures the
    thresholds are calibrated from.  The logits come from the routing call itself."""
    loads.zero_(); bins.zero_()
    r = laser.route_layers(data["hidden"], data["w_g"], data["bias"], loads, p, bin_loads=bins,
                           eps_high=data["eps_high"], t_fix=data["t_fix"], workspace=ws,
                           want_logits=True)
    for _ in range(3):
        stats, means = laser.score_stats(r.logits, w.k, 0.5, max(2, w.E // 4))
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    stats, means = laser.score_stats(r.logits, w.k, 0.5, max(2, w.E // 4))
    t1.record()
    torch.cuda.synchronize()
    st, mn = stats.cpu().double(), means.cpu().double()
    bands = {}
    for name, lo, hi in (("early", 0, -(-L // 3)), ("middle", -(-L // 3), -(-2 * L // 3)),
                         ("final", -(-2 * L // 3), L)):
        if hi <= lo:
            continue
        s = st[lo:hi].sum(0)
        hist = s[8:]
        half, acc, median_bin = s[0] / 2, 0.0, 63
        for b in range(64):
            acc += float(hist[b])
            if acc >= float(half):
                median_bin = b
                break
        bands[name] = {"layers": [lo, hi - 1], "mean_M_k": float(mn[lo:hi, 0].mean()),
                       "mean_entropy_nats": float(mn[lo:hi, 1].mean()),
                       "share_single_head": float(s[3] / s[0]), "share_plateau": float(s[4] / s[0]),
                       "share_smooth": float(s[5] / s[0]),
                       "M_k_median_bin_of_64": median_bin}
    return {"near_ratio": 0.5, "plateau_max": max(2, w.E // 4), "bands": bands,
            "kernel_ms": t0.elapsed_time(t1),
            "logits_bytes": r.logits.numel() * 4,
            "note": "one call (memset and two kernels) on logits just written, so partly in L2"}


def run_decode(args, w, ctx, full):
    """Decode stream: `S` successive calls of T tokens each, same W_g, load state carried
    from call to call.  One bench step = one pass over the whole stream, replayed as a CUDA
    graph; plain stream launches are timed beside it, then every call on its own (launch to
    completion) for the latency distribution, next to the same figures for an empty kernel."""
    import numpy as np
    import torch

    from paper_2510_03293_b200 import laser, synth

    dev = ctx.dev
    S = args.decode_steps or w.layers
    data = synth.make_workload_torch(w, dev, seed=args.seed, layers=S)
    hidden = data["hidden"]                      # [S, T, d]: call s routes hidden[s]
    wg, bias = data["w_g"][:1].contiguous(), data["bias"][:1].contiguous()
    p = laser.make_params(w.T, w.d, w.E, w.k, w.c, w.eps_high[0], w.t_fix, w.renormalize, w.n_bins)
    loads = torch.zeros((1, w.E), dtype=torch.int32, device=dev)
    bins = torch.zeros((1, w.n_bins), dtype=torch.int32, device=dev)
    ws = torch.empty((laser.workspace_bytes(p),), dtype=torch.uint8, device=dev)
    outs = laser.RouteResult(
        torch.empty((S, w.T, w.k), dtype=torch.int32, device=dev),
        torch.empty((S, w.T, w.k), dtype=torch.float32, device=dev),
        torch.empty((S, w.E + 1), dtype=torch.int32, device=dev),
        torch.empty((S, w.T * w.k), dtype=torch.int32, device=dev),
        loads, bins, None, torch.zeros((1,), dtype=torch.int32, device=dev))

    def one_call(s_):
        o = laser.RouteResult(outs.expert_ids[s_:s_ + 1], outs.weights[s_:s_ + 1],
                              outs.offsets[s_:s_ + 1], outs.perm[s_:s_ + 1], loads, bins, None,
                              outs.status)
        laser.route_layers(hidden[s_:s_ + 1], wg, bias, loads, p, bin_loads=bins, out=o,
                           workspace=ws)

    def one_pass():
        loads.zero_(); bins.zero_()
        for s_ in range(S):
            one_call(s_)

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        one_pass()                                # first calls outside any capture
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            one_pass()
        empty_graph = torch.cuda.CUDAGraph()
        laser.test_launch_empty(side)
        torch.cuda.synchronize()
        with torch.cuda.graph(empty_graph, stream=side):
            for _ in range(S):
                laser.test_launch_empty(side)
    torch.cuda.synchronize()

    def timed(fn, n):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    def each_alone(fn, n):
        """us from launch to completion of n calls made one at a time (the stream is idle
        before each): what a decode loop that needs the result before its next step sees."""
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        us = []
        for i in range(n):
            torch.cuda.synchronize()
            e0.record()
            fn(i)
            e1.record()
            e1.synchronize()
            us.append(e0.elapsed_time(e1) * 1e3)
        return {"mean": sum(us) / len(us), "p50": percentile(us, 0.5), "p99": percentile(us, 0.99),
                "calls": n}

    for _ in range(max(3, args.warmup)):
        graph.replay()
    sampler = ClockSampler(ctx.local)
    sampler.start(); time.sleep(0.3)
    ms_graph = timed(graph.replay, args.steps)
    clocks = sampler.stop()
    ids_graph = outs.expert_ids.clone(); loads_graph = loads.clone()
    ms_plain = timed(one_pass, max(1, min(args.steps, 3)))
    same = bool(torch.equal(ids_graph, outs.expert_ids) and torch.equal(loads_graph, loads))
    status = int(outs.status.item())
    loads.zero_(); bins.zero_()
    latency = each_alone(one_call, S)
    floor_alone = each_alone(lambda i: laser.test_launch_empty(), min(S, 1024))
    for _ in range(3):
        empty_graph.replay()
    floor_graph_us = timed(empty_graph.replay, max(3, min(args.steps, 10))) * 1e3 / S

    # end to end: every call copies its hidden states in and its results out
    h_hidden = hidden[:min(S, 256)].cpu().pin_memory()
    h_wg, h_bias = wg.cpu().pin_memory(), bias.cpu().pin_memory()
    h_loads = torch.zeros((1, w.E), dtype=torch.int32).pin_memory()
    h_bins = torch.zeros((1, w.n_bins), dtype=torch.int32).pin_memory()
    arena = torch.empty((laser.host_arena_bytes(1, p),), dtype=torch.uint8, device=dev)
    host_out = None
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for s_ in range(h_hidden.shape[0]):
        host_out = laser.route_host(h_hidden[s_:s_ + 1], h_wg, h_bias, h_loads, p, arena,
                                    bin_loads=h_bins, out=host_out)
    e2e_sec = (time.perf_counter() - t0) / h_hidden.shape[0]
    h2d = sum(t.numel() * t.element_size() for t in (h_hidden[:1], h_wg, h_bias, h_loads, h_bins))
    d2h = sum(t.numel() * t.element_size() for t in host_out) + (w.E + w.n_bins) * 4

    peak, peak_kind = measured_peak_hbm()
    tokens = S * w.T
    bytes_per_pass = algorithmic_bytes_per_token(w) * tokens
    gbs = bytes_per_pass / (ms_graph * 1e-3) / 1e9
    result = {
        "metric": METRIC, "value": tokens / (ms_graph * 1e-3), "unit": UNIT, "n_gpus": 1,
        "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms_graph,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "accumulate": "f32 (logits, scores and weights in f32; ids, loads, dispatch in int32)", "data": "synthetic",
        "config": {"workload": "decode: %d successive calls x T=%d, d=%d bf16, E=%d, k=%d, c=%d, "
                               "loads carried across calls" % (S, w.T, w.d, w.E, w.k, w.c),
                   "tokens_per_step": tokens,
                   "cache": "every call reads its own %.2f MB of hidden states (%.2f GB per pass)"
                            % (2.0 * w.T * w.d / 1e6, 2.0 * tokens * w.d / 1e9)},
        "decode": {"us_per_call_graph": ms_graph * 1e3 / S, "us_per_call_stream_launches":
                   ms_plain * 1e3 / S, "calls_per_pass": S, "graph_equals_stream_launches": same,
                   "latency_us_one_call_at_a_time": latency,
                   "launch_floor_us": {"empty_kernel_one_at_a_time": floor_alone,
                                       "empty_kernel_per_graph_node": floor_graph_us},
                   "graph_nodes_per_call": DECODE_NODES_PER_CALL},
        "roofline": {"bound": "hbm", "kernel": router_kernel_name(w, 1), "achieved": gbs,
                     "peak": peak, "peak_kind": peak_kind, "unit": "GB/s", "frac": gbs / peak,
                     "traffic": recorded_traffic(w.name, w.T), "bytes_per_launch": bytes_per_pass / S,
                     "note": "latency-bound: 0.26 MB per call"},
        "path": {"path_gbs": gbs, "path_frac_of_hbm_peak": gbs / peak,
                 "path_frac_of_8tbs": gbs / 8000.0},
        "routing": {"status_word": status},
        "gpu_launches": launches_per_step(w, 1) * S * args.steps, "clocks": clocks,
        "e2e": {"value": w.T / e2e_sec, "unit": UNIT, "ms_per_step": e2e_sec * 1e3 * S,
                "us_per_call": e2e_sec * 1e6, "h2d_bytes_per_step": h2d * S,
                "d2h_bytes_per_step": d2h * S, "calls_timed": int(h_hidden.shape[0])},
    }
    if not args.no_cpu_baseline:
        # the oracle on the concatenated stream (per-token load updates make one call over all
        # the tokens equal to the sequence of calls), first 16384 tokens
        n_calls = min(S, 16384 // w.T)
        cat = {"hidden": hidden[:n_calls].reshape(1, n_calls * w.T, w.d), "w_g": wg, "bias": bias,
               "eps_high": [w.eps_high[0]], "t_fix": [w.t_fix]}
        wcat = dataclasses_replace(w, T=n_calls * w.T, layers=1)
        base = cpu_baseline_and_agreement(args, wcat, 1, cat, np, torch, laser, synth, dev, False)
        result["cpu_oracle_sample"] = base["cpu_baseline"]
        result["routing"].update(base["routing"])
        result["agreement"] = base["agreement"]
        result["agreement"]["sample"] = ("the first %d calls as one call of %d tokens; " %
                                         (n_calls, n_calls * w.T)) + "oracle on its own logits"
    del data, hidden, outs, graph, empty_graph
    torch.cuda.empty_cache()
    return result


def e2e_host(args, w, L, data, p, laser, torch, dev):
    h_hidden = data["hidden"].cpu().pin_memory()
    h_wg = data["w_g"].cpu().pin_memory()
    h_bias = data["bias"].cpu().pin_memory()
    h_loads = torch.zeros((L, w.E), dtype=torch.int32).pin_memory()
    h_bins = torch.zeros((L, w.n_bins), dtype=torch.int32).pin_memory()
    arena = torch.empty((laser.host_arena_bytes(L, p),), dtype=torch.uint8, device=dev)
    outs = None
    times = []
    n = max(1, min(args.steps, args.e2e_steps))
    for i in range(n + 1):
        h_loads.zero_(); h_bins.zero_()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        outs = laser.route_host(h_hidden, h_wg, h_bias, h_loads, p, arena, bin_loads=h_bins,
                                eps_high=data["eps_high"], t_fix=data["t_fix"], out=outs)
        if i > 0:
            times.append(time.perf_counter() - t0)
    sec = sum(times) / len(times)
    h2d = sum(t.numel() * t.element_size() for t in (h_hidden, h_wg, h_bias, h_loads, h_bins))
    d2h = sum(t.numel() * t.element_size() for t in outs) + \
        sum(t.numel() * t.element_size() for t in (h_loads, h_bins))
    return {"value": L * w.T / sec, "unit": UNIT, "ms_per_step": sec * 1e3,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": n}


def cpu_baseline_and_agreement(args, w, L, data, np, torch, laser, synth, dev, full):
    """The CPU-baseline leg: the oracle as it stands, on the host cores, on a bounded sample of
    the workload.  Its first sampled layer (the first 16384 tokens of it for longer layers) is
    also compared with the GPU path: the oracle computes its OWN logits in fp64 from the same
    bf16 inputs, so one token that falls on the other side of a threshold changes the loads seen
    by every later token; reported are how many tokens still choose the same expert set, the
    first token that differs, and the balance figures of both runs.  (The bit-exact comparison
    given the GPU's fp32 logits is repeated here on the same sample.)"""
    import oracle

    oracle.build()
    i16 = torch.int16
    Ts = min(w.T, 16384)
    n_sample = min(L, args.ref_layers) if full else 1
    layers_data = []
    for l in range(n_sample):
        hb = data["hidden"][l, :Ts].view(i16).cpu().numpy().view(np.uint16)
        wb = data["w_g"][l].view(i16).cpu().numpy().view(np.uint16)
        layers_data.append((hb, wb, data["bias"][l].cpu().numpy()))
    ws_ = dataclasses_replace(w, T=Ts)
    e2b = synth.default_expert_to_bin(w.E, w.n_bins)
    z, zb = np.zeros(w.E, np.int32), np.zeros(w.n_bins, np.int32)
    eps0, tf0 = data["eps_high"][0], data["t_fix"][0]
    # first pass, kept: the oracle's whole path on layer 0 with its own logits
    t0 = time.perf_counter()
    hb, wb, bias = layers_data[0]
    ref = oracle.route_full(hb, wb, bias, z, e2b, zb, w.k, w.c, eps0, tf0, bool(w.renormalize))
    first = time.perf_counter() - t0
    total, passes = 0.0, 0
    budget = args.cpu_seconds if full else 0.0
    while total < budget and passes < 64:
        total += oracle_pass(oracle, np, layers_data, ws_, data["eps_high"], data["t_fix"])
        passes += 1
    if passes == 0:
        total, passes, n_timed = first, 1, 1
    else:
        n_timed = n_sample
    sec = total / passes
    cores = len(os.sched_getaffinity(0))
    base = {"value": n_timed * Ts / sec, "unit": UNIT, "cores": cores, "kind": "oracle",
            "seconds": total,
            "sample": "%d of %d layers%s (%d tokens) x %d passes, fp64 contraction with OpenMP over "
                      "tokens, ordered scan on one core" %
                      (n_timed, L, "" if Ts == w.T else ", first %d tokens of each" % Ts,
                       n_timed * Ts, passes)}

    # the GPU path on the same sample
    p = laser.make_params(Ts, w.d, w.E, w.k, w.c, eps0, tf0, w.renormalize, w.n_bins)
    loads = torch.zeros((1, w.E), dtype=torch.int32, device=dev)
    r = laser.route_layers(data["hidden"][:1, :Ts].contiguous(), data["w_g"][:1], data["bias"][:1],
                           loads, p, want_logits=True)
    torch.cuda.synchronize()
    ids_g = r.expert_ids[0].cpu().numpy()
    x_g = r.logits[0].cpu().numpy()
    cnt_g = np.diff(r.offsets[0].cpu().numpy()).astype(np.float64)
    exact = oracle.route(x_g, z, w.k, w.c, eps0, tf0, bool(w.renormalize))
    same = (np.sort(ids_g, 1) == np.sort(ref["expert_ids"], 1)).all(1)
    differ = np.flatnonzero(~same)
    cnt_o = ref["counts"].astype(np.float64)
    imb = lambda c: float(c.max() / c.mean()) if c.sum() > 0 else 1.0
    agreement = {
        "sample": "layer 0, %d tokens; oracle on its own fp64-accumulated logits" % Ts,
        "set_agreement_frac": float(same.mean()),
        "first_divergent_token": int(differ[0]) if differ.size else None,
        "logits_max_abs_err": float(np.max(np.abs(x_g - ref["logits"]))),
        "imbalance_gpu": imb(cnt_g), "imbalance_oracle": imb(cnt_o),
        "MV_gpu": imb(cnt_g) - 1.0, "MV_oracle": imb(cnt_o) - 1.0,
        "bit_exact_given_gpu_logits": bool(np.array_equal(ids_g, exact[0]) and
                                           np.array_equal(loads[0].cpu().numpy(), exact[2])),
    }
    # routing statistics of the sample (oracle run): expansion rule and final assignment
    cs = ref["cstar"]
    x = ref["logits"]
    expanded = cs > 0
    order = np.argsort(-x, axis=1, kind="stable")[:, :w.c]
    sc = np.take_along_axis(oracle.softmax(x), order, 1)
    thr = (np.float32(tf0) * sc[:, 0]).astype(np.float32)
    m_prime = (sc >= thr[:, None]).sum(1)
    topk = np.sort(oracle.topk(x, w.k), 1)
    routing = {
        "expanded_frac": float(expanded.mean()),
        "mean_m_prime": float(m_prime[expanded].mean()) if expanded.any() else 0.0,
        "mean_cstar": float(cs[expanded].mean()) if expanded.any() else 0.0,
        "decision_tokens_frac": float((cs > w.k).mean()),
        "differs_from_topk_frac": float((np.sort(ref["expert_ids"], 1) != topk).any(1).mean()),
    }
    return {"cpu_baseline": base, "agreement": agreement, "routing": routing}


def dataclasses_replace(w, **kw):
    import dataclasses

    return dataclasses.replace(w, **kw)


def one_core_oracle(name):
    """The oracle's whole path on one workload layer with OpenMP held to one thread (a child
    process, since the thread count is fixed when the library loads)."""
    code = ("import sys, time, json, numpy as np; sys.path.insert(0, %r); import oracle; "
            "from paper_2510_03293_b200 import synth; w = synth.WORKLOADS[%r]; "
            "hb, wb, b = synth.make_workload_layer(w, 0); "
            "e2b = synth.default_expert_to_bin(w.E, w.n_bins); "
            "f = lambda: oracle.route_full(hb, wb, b, np.zeros(w.E, np.int32), e2b, "
            "np.zeros(w.n_bins, np.int32), w.k, w.c, w.eps_for_layer(0), w.t_fix, bool(w.renormalize)); "
            "f(); t = time.perf_counter(); f(); print(json.dumps(time.perf_counter() - t))" % (ROOT, name))
    try:
        out = subprocess.run([sys.executable, "-c", code], env=dict(os.environ, OMP_NUM_THREADS="1"),
                             capture_output=True, text=True, timeout=120)
        sec = float(json.loads(out.stdout.strip().splitlines()[-1]))
    except Exception as e:   # noqa: BLE001
        return {"error": repr(e)}
    from paper_2510_03293_b200 import synth

    w = synth.WORKLOADS[name]
    return {"value": w.T / sec, "unit": UNIT, "cores": 1, "kind": "oracle", "seconds": sec,
            "sample": "one layer of %d tokens, one pass" % w.T}


def free_port():
    import socket

    with socket.socket() as s_:
        s_.bind(("127.0.0.1", 0))
        return s_.getsockname()[1]


def spawn_replicas(n, argv):
    """Starts n copies of this program, one per GPU, as the ranks of one job (the launch torchrun
    would do) and returns the largest exit code.  Rank 0 prints the JSON line."""
    port = free_port()
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + argv, env=env))
    return max(p_.wait() for p_ in procs)


def selftest_replicas():
    """CPU check of the replica plumbing (gloo): every rank reports a different time; the line
    must carry the slowest one and the tokens of all ranks."""
    import torch
    import torch.distributed as dist

    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, value = aggregate_replicas(10.0 * (rank + 1), 5, 1000, dist, torch.device("cpu"))
    dist.barrier()
    dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"n_gpus": world, "ms_per_step": ms, "value": value}))


SUB_WORKLOADS = ("tiny", "deepseek", "decode", "stress")
# what a sub-workload's record keeps (the full records are printed by --workload NAME)
SUB_KEYS = ("value", "unit", "ms_per_step", "steps", "config", "roofline", "path", "routing",
            "selection", "agreement", "cpu_oracle_sample", "cpu_oracle_one_core", "decode",
            "gpu_launches", "clocks")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="laser", choices=["laser", "reference"])
    ap.add_argument("--workload", default=None,
                    help="one workload only (tiny, mixtral, deepseek, decode, stress); default: "
                         "mixtral as the line's value with the other four under 'workloads'")
    ap.add_argument("--layers", type=int, default=None, help="override the layer count")
    ap.add_argument("--tokens", type=int, default=None,
                    help="override the tokens per layer (small cases for profiling)")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--ref-layers", type=int, default=8)
    ap.add_argument("--cpu-seconds", type=float, default=12.0,
                    help="CPU work spent on the cpu_baseline leg")
    ap.add_argument("--sustained-seconds", type=float, default=2.0,
                    help="length of the sustained loop of the headline step (0 = skip)")
    ap.add_argument("--decode-steps", type=int, default=None,
                    help="decode stream: successive 64-token calls per pass (default 4096)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--eps-high", type=float, default=None,
                    help="override eps_high of every layer (0 = vanilla top-k, 2 = always expand)")
    ap.add_argument("--t-fix", type=float, default=None, help="override t_fix of every layer")
    ap.add_argument("--c", type=int, default=None, help="override the trimming size c")
    ap.add_argument("--random-trim", type=int, default=None, metavar="SEED",
                    help="RANDOM trimming (Algorithm 1's second mode) with this generator seed "
                         "instead of TOP trimming")
    ap.add_argument("--imbalance-batches", type=int, default=0, metavar="B",
                    help="after the timed run, route B more batches under the method, plain "
                         "top-k and load-only, and report I_agg P50/P95 and MV of each")
    ap.add_argument("--score-stats", action="store_true",
                    help="add the gate-score statistics of the batch by layer band")
    ap.add_argument("--granularity", type=int, default=1,
                    help="load-update granularity: 1 = the method's rule (default); 0 or a "
                         "multiple of 32 = the RELAXED variant, reported as such with its drift "
                         "from the rule")
    ap.add_argument("--selftest-replicas", action="store_true", help=argparse.SUPPRESS)
    args = ap.parse_args()

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl != "reference":
        sys.exit(spawn_replicas(args.gpus, sys.argv[1:]))
    if args.selftest_replicas:
        return selftest_replicas()

    from paper_2510_03293_b200 import synth

    def workload(name):
        w = synth.WORKLOADS[name]
        over = {}
        if args.eps_high is not None:
            over["eps_high"] = (args.eps_high,)
        if args.t_fix is not None:
            over["t_fix"] = args.t_fix
        if args.c is not None:
            over["c"] = args.c
        if args.tokens is not None:
            over["T"] = args.tokens
        return dataclasses_replace(w, **over) if over else w

    headline = args.workload or "mixtral"
    if args.impl == "reference":
        return run_reference(args, workload(headline))

    ctx = Context()
    run = lambda w, full: (run_decode if w.persistent_loads else run_layers)(args, w, ctx, full)
    result = run(workload(headline), True)
    if args.workload is None and ctx.world == 1 and args.layers is None and args.tokens is None:
        subs = {}
        for name in SUB_WORKLOADS:
            r = run(workload(name), False)
            if name == "tiny" and not args.no_cpu_baseline:
                r["cpu_oracle_one_core"] = one_core_oracle(name)
            subs[name] = {k_: r[k_] for k_ in SUB_KEYS if k_ in r}
        result["workloads"] = subs
    ctx.close()
    if ctx.rank == 0:
        print(json.dumps(result))


if __name__ == "__main__":
    main()
