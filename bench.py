#!/usr/bin/env python
"""Benchmark of the MoE layer hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload decode|prefill|search]
                    [--tokens T] [--beta calibrated|0] [--kept full|r6|r4] [--impl ours|reference]

One step = one pass of the whole hot path (router, permutation, both grouped GEMMs, combine;
or the pruning search) over one batch of seeded synthetic tokens at the Mixtral-8x7B layer
shape.  Prints ONE JSON line.  The timed region is R blocks of exactly --steps steps (median
block reported, best beside it).  The default run (decode, T = 128, all experts, beta = 0, one
GPU) also measures the other configured workloads afterwards and reports them under "matrix":
decode at other batch sizes and on pruned layers, prefill with skipping off and on, the search.  With N > 1 (launched by torch.distributed.run) every rank runs
an independent replica on its own GPU: the path has no exchange step, so no collective sits
on the data path; timing is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2402_14800_b200 import synth  # noqa: E402

H, F, E = synth.MIXTRAL["h"], synth.MIXTRAL["f"], synth.MIXTRAL["E"]
FLOP_PER_PAIR = 2 * 3 * H * F
KEPT = {"full": 0xFF, "r6": 0x3F, "r4": 0x0F}
NOMINAL_HBM_GBS = 8000.0      # vendor figure, context beside the measured copy bandwidth
NOMINAL_BF16_TFLOPS = 2250.0  # vendor dense bf16 figure, context beside the measured cuBLAS rates


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm=float(d["hbm_gbs"]), tf_burst=float(d["bf16_tflops"]),
                    tf_sust=float(d["bf16_tflops_sustained"]), source="measured")
    return dict(hbm=6650.0, tf_burst=1590.0, tf_sust=1400.0, source="fallback")


def kernel_source_sha256(kernel: str = ""):
    """Hash of the source file of the grouped GEMMs with its shared header: any edit to either
    (kernel bodies, tile decoding, epilogues, descriptors) voids the recorded counters."""
    import hashlib
    hsh = hashlib.sha256()
    for name in ("gemm_sm100.cu", "common.h"):
        hsh.update(open(os.path.join(ROOT, "paper_2402_14800_b200", "csrc", name), "rb").read())
    return hsh.hexdigest()


def single_token_gemv() -> bool:
    """Whether the library runs a single token through its matrix-vector kernels (its default)
    rather than the grouped GEMMs (forced by either switch)."""
    return (os.environ.get("MOE_SINGLE_KERNEL", "") != "gemm"
            and os.environ.get("MOE_DECODE_KERNEL", "") not in ("wm", "td"))


def recorded_traffic(workload: str, kernel: str):
    """DRAM bytes per launch of the dominant kernel from the committed ncu capture of this
    workload, or None when there is none, it is of another kernel than the one that ran, or
    the GEMM sources changed since."""
    try:
        rec = json.load(open(os.path.join(ROOT, "profiles", "traffic.json"))).get(workload)
        if (rec and rec["kernel"] == kernel
                and kernel_source_sha256(rec["kernel_function"]) == rec["kernel_source_sha256"]):
            return rec["dram_bytes"]
    except Exception:
        pass
    return None


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if not self.proc:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except Exception:
                continue
            try:
                pw.append(float(r[2]))
            except Exception:
                pass
            for n, v in zip(names, r[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    samples=len(sm), power_w=float(np.median(pw)) if pw else None, reasons=sorted(reasons))


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def max_over_ranks(v: float, dev=None) -> float:
    """Max of a per-rank scalar over all ranks (identity for a single process)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(v)
    on_gpu = dist.get_backend() == "nccl"
    t = torch.tensor([v], dtype=torch.float64, device=dev if on_gpu else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(units_per_rank_step: float, steps: int, ms_total_max: float, world: int) -> float:
    """Replicas: every rank processes its own units; the job's rate is all of them over the
    slowest rank's time."""
    return world * units_per_rank_step * steps / (ms_total_max * 1e-3)


def workload_name(a):
    if a.workload == "search":
        return "search_T%d_r%s" % (a.tokens, a.search_r)
    return "%s_T%d_%s_beta-%s" % (a.workload, a.tokens, a.kept, a.beta)


def layer_config(a, T, kept_mask, beta, pairs, touched, world):
    """The `config` object of a single-layer line; both arms build it here so that the two lines
    name the same workload with the same keys."""
    return {"workload": workload_name(a), "h": H, "f": F, "E": E, "tokens": T,
            "kept_mask": kept_mask, "beta": beta, "pairs": pairs, "experts_touched": touched,
            "parallelism": "replicas x%d, no collective" % world,
            "l2": "per step the kernels stream %.2f GB of weights, far above the 126 MB L2"
                  % (touched * 3 * H * F * 2 / 1e9) if a.workload != "search" else
                  "inputs and intermediates are GBs, far above the 126 MB L2"}


# ------------------------------------------------------------------------- reference arm

def oracle_sample(a, W_host, x_host, beta, n_sample):
    from oracle import moe_oracle as O
    xs = x_host[:n_sample]
    t0 = time.perf_counter()
    if a.workload == "search":
        for r in (6, 4):
            O.prune_search_allexperts(xs, W_host["Wg"], W_host["W1"], W_host["W3"], W_host["W2"], r)
    else:
        O.moe_forward(xs, W_host["Wg"], W_host["W1"], W_host["W3"], W_host["W2"], KEPT[a.kept], beta)
    return time.perf_counter() - t0


def units_per_step(a):
    # tokens for the forward workloads; subsets x tokens for the search (28 + 70 subsets)
    return a.tokens * (98 if a.workload == "search" else 1)


def metric_unit(a):
    if a.workload == "search":
        return "pruning-search subsets*tokens/s on 1 B200 (Mixtral-shaped layer, r=6 and r=4)", "subsets*tokens/s"
    return "MoE-layer tokens/s on 1 B200 (decode/prefill, +-skip/prune); % HBM or bf16 peak", "tokens/s"


def host_inputs(a, device):
    """Weights, tokens and the calibration batch; drawn on `device`, copies on the host."""
    W = synth.make_layer_weights(H, F, E, seed=0, device=device)
    x = synth.make_tokens(a.tokens, H, seed=1, device=device)
    xcal = synth.make_tokens(4096, H, seed=1001, device=device)
    return W, x, xcal


def run_reference_stack(a):
    """Oracle over the first layers of the stack (each layer's weights are 2.8 GB on the host, so
    only min(layers, 4) layers are walked; the sample line says so)."""
    from oracle import moe_oracle as O
    dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    b = synth.bf16_bits
    nl = min(a.layers, 4)
    n_sample = max(1, min(a.tokens, 8))
    xh = b(synth.make_tokens(a.tokens, H, seed=1, device=dev))[:n_sample]
    Ws = []
    for l in range(nl):
        W = synth.make_layer_weights(H, F, E, seed=100 + l, device=dev)
        Ws.append(dict(Wg=b(W.W_gate), W1=b(W.W1), W3=b(W.W3), W2=b(W.W2)))
        del W
    times = []
    for _ in range(a.steps):
        t0 = time.perf_counter()
        cur = xh
        for Wh in Ws:
            xn = O.rmsnorm(cur, 1e-5)
            cur = O.moe_forward(xn, Wh["Wg"], Wh["W1"], Wh["W3"], Wh["W2"], 0xFF, 0.0, residual=cur)["y"]
        times.append(time.perf_counter() - t0)
    # tokens/s through a 32-layer stack, extrapolated linearly from the layers walked
    value = n_sample * a.steps / (sum(times) * a.layers / nl)
    sample = "%d of %d tokens through %d of %d layers per step, scaled to all layers" % (
        n_sample, a.tokens, nl, a.layers)
    line = {
        "impl": "reference",
        "metric": "MoE-stack tokens/s on 1 B200 (32 layers, RMSNorm + residual, attention omitted)",
        "value": value, "unit": "tokens/s", "n_gpus": a.gpus, "steps": a.steps, "warmup": a.warmup,
        "ms_per_step": 1e3 * sum(times) / a.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "stack%d_T%d_full_beta-0" % (a.layers, a.tokens), "h": H, "f": F, "E": E},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": O.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


def run_reference(a):
    rank, world, local = dist_env()
    if rank != 0:
        return 0
    if a.workload == "stack":
        return run_reference_stack(a)
    from oracle import moe_oracle as O
    dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    W, x, xcal = host_inputs(a, dev)
    b = synth.bf16_bits
    Wh = dict(Wg=b(W.W_gate), W1=b(W.W1), W3=b(W.W3), W2=b(W.W2))
    xh = b(x)
    beta = 0.0
    if a.beta == "calibrated" and a.workload != "search":
        beta = O.beta_median(O.route(b(xcal), Wh["Wg"], KEPT[a.kept], 0.0)["ratio"])
    del W
    # size the per-step sample from a probe so that K steps take about a minute in total
    probe = 2
    dt = oracle_sample(a, Wh, xh, beta, probe)
    budget_s = 60.0
    n_sample = int(max(1, min(a.tokens, 128, budget_s / max(a.steps, 1) / (dt / probe))))
    for _ in range(min(a.warmup, 1)):
        oracle_sample(a, Wh, xh, beta, 1)
    times = [oracle_sample(a, Wh, xh, beta, n_sample) for _ in range(a.steps)]
    per_unit = (98 if a.workload == "search" else 1)
    value = n_sample * per_unit * a.steps / sum(times)
    metric, unit = metric_unit(a)
    sample = "%d of %d tokens per step, oracle as it stands" % (n_sample, a.tokens)
    # the workload's pair and expert counts, from the oracle's own routing of the whole batch
    kept_mask = KEPT[a.kept]
    if a.workload == "search":
        pairs = touched = 0
    else:
        rt = O.route(xh, Wh["Wg"], kept_mask, beta)
        alive = np.ones_like(rt["idx"], dtype=bool)
        alive[:, 1] = rt["skipped"] == 0
        pairs = int(alive.sum())
        touched = int(len(np.unique(rt["idx"][alive])))
    line = {
        "impl": "reference", "metric": metric, "value": value, "unit": unit, "n_gpus": a.gpus,
        "steps": a.steps, "warmup": a.warmup, "ms_per_step": 1e3 * sum(times) / a.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": layer_config(a, a.tokens, kept_mask, beta, pairs, touched, max(a.gpus, 1)),
        "cpu_baseline": {"value": value, "unit": unit, "cores": O.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


# -------------------------------------------------------------------------------- our arm

def max_over_ranks_vec(v, dev=None):
    """Element-wise max of a per-rank list over all ranks (identity for a single process)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(a) for a in v]
    on_gpu = dist.get_backend() == "nccl"
    t = torch.tensor(list(v), dtype=torch.float64, device=dev if on_gpu else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(a) for a in t.tolist()]


def make_barrier(world, dev):
    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize(dev)
    return barrier


MIN_REPEATS = 30  # blocks of the timed region at least (--min-repeats)


def timed_blocks(step, steps, warmup, stream, dev, rank, local, world, target_s=1.5, max_s=20.0,
                 min_repeats=None):
    """W warm-up steps, then R blocks of exactly `steps` steps each, every block bracketed by a
    barrier + device synchronisation on both sides and timed with CUDA events on the launching
    stream (max over ranks per block).  R is chosen so that the blocks cover about `target_s`
    seconds (at least `min_repeats`, fewer only when that would exceed `max_s`): a block of a few
    milliseconds alone is a burst at full clock, the repeats reach the clock the board settles at
    and give nvidia-smi time to sample it.  Returns the block times and the clock record."""
    barrier = make_barrier(world, dev)
    with torch.cuda.stream(stream):
        for _ in range(max(warmup, 3)):
            step()
    barrier()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    with torch.cuda.stream(stream):
        ev[0].record(stream)
        for _ in range(steps):
            step()
        ev[1].record(stream)
    barrier()
    est_ms = max_over_ranks(ev[0].elapsed_time(ev[1]), dev)
    if min_repeats is None:
        min_repeats = MIN_REPEATS
    R = max(min_repeats, int(np.ceil(target_s * 1e3 / max(est_ms, 1e-3))))
    R = max(min(5, min_repeats), min(R, int(max_s * 1e3 / max(est_ms, 1e-3))))
    events = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(R)]
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    barrier()
    for e0, e1 in events:
        with torch.cuda.stream(stream):
            e0.record(stream)
            for _ in range(steps):
                step()
            e1.record(stream)
        barrier()
    clocks = sampler.stop() if rank == 0 else None
    blocks = max_over_ranks_vec([e0.elapsed_time(e1) for e0, e1 in events], dev)
    return blocks, clocks


def timing_record(blocks, steps, clocks):
    med, best = float(np.median(blocks)), float(min(blocks))
    rec = {"repeats": len(blocks), "steps_per_block": steps, "ms_per_step_median": med / steps,
           "ms_per_step_best": best / steps, "ms_per_step_mean": float(np.mean(blocks)) / steps,
           "how": "CUDA events around each block of `steps` steps, barrier + synchronise on both sides "
                  "of every block, max over ranks per block; value and ms_per_step are the median block"}
    if clocks and clocks.get("sm_mhz"):
        # time x clock: comparable between a burst at full clock and a run at the power cap
        rec["sm_cycles_per_step_median"] = med / steps * 1e-3 * clocks["sm_mhz"] * 1e6
    return rec


def decode_kernel_name(T, r_kept):
    forced = os.environ.get("MOE_DECODE_KERNEL", "")
    if T == 1 and single_token_gemv():
        return "gemv_route_gate_up_kernel"
    # the library's crossover: many tokens per expert -> token-major decode kernel
    token_major = forced == "td" or (forced != "wm" and 2 * T >= 40 * r_kept and r_kept <= 6)
    return "gemm_tokens_d_kernel<gate_up>" if token_major else "gemm_weights_m_kernel<gate_up>"


def launches_per_forward(T):
    # T = 1: routing + gate/up matrix-vector kernel, down kernel with the weighted sum
    #   (with the GEMM path forced: routing, gate/up GEMM, down GEMM, combine);
    # T <= 256: router, permute+gather, gate/up GEMM, down GEMM, combine;
    # larger T: router, scan, scatter, gather, gate/up GEMM, down GEMM, combine
    if T == 1:
        return 2 if single_token_gemv() else 4
    return 5 if T <= 256 else 7


def forward_case(layer, x, y, beta, workload, wname, steps, warmup, stream, dev, rank, local, world, peaks,
                 kept, target_s, max_s=20.0):
    """One forward workload: routing facts, timed blocks, a pass with an event at every stage
    boundary (per-kernel durations for the roofline), and the roofline record."""
    from paper_2402_14800_b200 import binding
    T = x.shape[0]
    stats = binding.RoutingStats(T, E, dev)
    with torch.cuda.stream(stream):
        layer.forward(x, beta, y=y, stats=stats)
    stream.synchronize()
    pairs = 2 * T - int(stats.n_skipped.item())
    touched = int(stats.n_experts_touched.item())

    def step():
        layer.forward(x, beta, y=y)

    blocks, clocks = timed_blocks(step, steps, warmup, stream, dev, rank, local, world, target_s, max_s)
    timing = timing_record(blocks, steps, clocks)
    ms_step = timing["ms_per_step_median"]
    # the same steps once more with an event at every stage boundary.  (The events sit between the
    # kernels, so this pass does not overlap one kernel's launch with its predecessor's tail; the
    # step time comes from the blocks above.)
    n_prof = int(max(steps, min(2000, np.ceil(min(0.3, target_s) * 1e3 / max(ms_step, 1e-3)))))
    layer.profile_enable(True)
    with torch.cuda.stream(stream):
        for _ in range(n_prof):
            step()
    stage_ms, ncalls = layer.profile_read()
    layer.profile_enable(False)
    if layer.device_status() != 0:
        raise RuntimeError("a bounded wait inside a kernel expired during the timed steps")
    gu_ms, dn_ms = stage_ms[1] / ncalls, stage_ms[2] / ncalls
    stages = {"route_permute_ms": stage_ms[0] / ncalls, "gate_up_ms": gu_ms, "down_ms": dn_ms,
              "combine_ms": stage_ms[3] / ncalls, "steps": ncalls}
    r_kept = bin(kept).count("1")
    if workload == "decode":
        gu_bytes = touched * 2 * F * H * 2 + pairs * H * 2 + pairs * F * 2
        dn_bytes = touched * H * F * 2 + pairs * F * 2 + 2 * pairs * H * 4
        ach = gu_bytes / (gu_ms * 1e-3) / 1e9
        kernel = decode_kernel_name(T, r_kept)
        roofline = {"bound": "hbm", "kernel": kernel, "achieved": ach,
                    "peak": peaks["hbm"], "unit": "GB/s", "frac": ach / peaks["hbm"],
                    "traffic": recorded_traffic(wname, kernel),
                    "peak_source": peaks["source"], "algorithmic_bytes": gu_bytes,
                    "frac_of_nominal_8TBs": ach / NOMINAL_HBM_GBS,
                    "down_kernel": {"achieved": dn_bytes / (dn_ms * 1e-3) / 1e9,
                                    "frac": dn_bytes / (dn_ms * 1e-3) / 1e9 / peaks["hbm"]},
                    "whole_step_frac": (gu_bytes + dn_bytes) / (ms_step * 1e-3) / 1e9 / peaks["hbm"]}
    else:
        gu_flop = pairs * 4 * H * F
        dn_flop = pairs * 2 * H * F
        ach = gu_flop / (gu_ms * 1e-3) / 1e12
        step_tf = (gu_flop + dn_flop) / (ms_step * 1e-3) / 1e12
        roofline = {"bound": "tensor", "kernel": "gemm_tokens_m_kernel<gate_up>", "achieved": ach,
                    "peak": peaks["tf_sust"], "unit": "TFLOP/s", "frac": ach / peaks["tf_sust"],
                    "traffic": recorded_traffic(wname, "gemm_tokens_m_kernel<gate_up>"),
                    "peak_source": peaks["source"] + " (sustained bf16; these runs sit at the power cap)",
                    "frac_of_burst": ach / peaks["tf_burst"],
                    "frac_of_nominal_dense_bf16": ach / NOMINAL_BF16_TFLOPS,
                    "algorithmic_flop": gu_flop,
                    "down_kernel": {"achieved": dn_flop / (dn_ms * 1e-3) / 1e12,
                                    "frac": dn_flop / (dn_ms * 1e-3) / 1e12 / peaks["tf_sust"],
                                    "frac_of_burst": dn_flop / (dn_ms * 1e-3) / 1e12 / peaks["tf_burst"]},
                    "whole_step_tflops": step_tf,
                    "whole_step_frac": step_tf / peaks["tf_sust"],
                    "whole_step_frac_of_burst": step_tf / peaks["tf_burst"]}
    return dict(T=T, beta=beta, pairs=pairs, touched=touched, timing=timing, clocks=clocks, stages=stages,
                roofline=roofline, ms_step=ms_step, blocks=blocks)


def search_case(layer, x, steps, warmup, stream, dev, rank, local, world, peaks, target_s, max_s=20.0):
    """The pruning search for r = 6 and r = 4 over one evaluation of the experts."""
    T = x.shape[0]

    def step():
        layer.prune_search_multi(x, [6, 4])

    blocks, clocks = timed_blocks(step, steps, warmup, stream, dev, rank, local, world, target_s, max_s,
                                  min_repeats=min(5, MIN_REPEATS))
    timing = timing_record(blocks, steps, clocks)
    ms_step = timing["ms_per_step_median"]
    layer.profile_enable(True)
    with torch.cuda.stream(stream):
        for _ in range(max(2, min(steps, 5))):
            step()
    stage_ms, ncalls = layer.profile_read()
    layer.profile_enable(False)
    chunks = (T + 8191) // 8192
    n_search = ncalls // (chunks + 1)   # a search records one set of marks per chunk and one for the enumerations
    # r = 6 and r = 4 share one evaluation of each token's E - 4 + 2 = 6 top-ranked experts
    dense = os.environ.get("MOE_SEARCH_DENSE", "") == "1"
    K = E if dense else E - 4 + 2
    gu_ms, dn_ms, en_ms = (stage_ms[i] / n_search for i in (1, 2, 3))
    gu_flop, dn_flop = 4 * T * K * H * F, 2 * T * K * H * F
    # one enumeration pass for both sizes reads the K evaluated expert outputs of every token once
    en_bytes = T * H * 2 * K + T * E * 4
    ach = gu_flop / (gu_ms * 1e-3) / 1e12
    step_tf = (gu_flop + dn_flop) / (ms_step * 1e-3) / 1e12
    roofline = {"bound": "tensor", "kernel": "gemm_tokens_m_kernel<gate_up> (expert evaluations of the search)",
                "achieved": ach, "peak": peaks["tf_sust"], "unit": "TFLOP/s", "frac": ach / peaks["tf_sust"],
                "traffic": None, "frac_of_burst": ach / peaks["tf_burst"],
                "frac_of_nominal_dense_bf16": ach / NOMINAL_BF16_TFLOPS,
                "algorithmic_flop": gu_flop,
                "peak_source": peaks["source"] + " (sustained bf16; these runs sit at the power cap)",
                "down_kernel": {"achieved": dn_flop / (dn_ms * 1e-3) / 1e12,
                                "frac": dn_flop / (dn_ms * 1e-3) / 1e12 / peaks["tf_sust"],
                                "frac_of_burst": dn_flop / (dn_ms * 1e-3) / 1e12 / peaks["tf_burst"]},
                "enumerate_kernel": {"bound": "hbm", "ms": en_ms, "algorithmic_bytes": en_bytes,
                                     "achieved": en_bytes / (en_ms * 1e-3) / 1e9, "unit": "GB/s",
                                     "frac": en_bytes / (en_ms * 1e-3) / 1e9 / peaks["hbm"]},
                "whole_step_tflops": step_tf, "whole_step_frac": step_tf / peaks["tf_sust"],
                "whole_step_frac_of_burst": step_tf / peaks["tf_burst"]}
    stages = {"route_permute_ms": stage_ms[0] / n_search, "gate_up_ms": gu_ms, "down_ms": dn_ms,
              "enumerate_ms": en_ms, "searches": n_search}
    # per chunk: route, count, scan, scatter, gather, 2 GEMMs; then enumerate + reduce per size
    return dict(T=T, timing=timing, clocks=clocks, stages=stages, roofline=roofline, ms_step=ms_step,
                launches_per_step=chunks * 7 + 2 * 2)


def matrix_rows(W, xcal, layers, stream, dev, rank, local, world, peaks, head, rows):
    """The other configured workloads, measured in the same invocation after the headline: decode
    at T = 1 / 8 / 32 and on pruned layers, prefill at T = 2048 / 8192 / 32768 with skipping off
    and on, the pruning search at T = 32768.  Each row has its own timed blocks, clock record and
    roofline fractions; speed-ups are against the same kernels on the unpruned layer at beta = 0."""
    from paper_2402_14800_b200 import binding
    base_ms = {}   # `rows` is the caller's list: what has been measured survives a failure later on

    def layer_for(kname):
        if kname not in layers:
            layers[kname] = binding.MoeLayer(W.W_gate, W.W1, W.W3, W.W2, KEPT[kname])
            layers[kname].set_stream(stream)
        return layers[kname]

    betas = {}

    def beta_for(kname, mode):
        if mode == "0":
            return 0.0
        if kname not in betas:
            betas[kname] = layer_for(kname).calibrate_beta(xcal)
        return betas[kname]

    plan = [("decode", 1, "full", "0"), ("decode", 1, "full", "calibrated"), ("decode", 8, "full", "0"),
            ("decode", 32, "full", "0"), ("decode", 128, "full", "calibrated"), ("decode", 128, "r6", "0"),
            ("decode", 128, "r4", "0"), ("decode", 128, "r4", "calibrated"),
            ("prefill", 2048, "full", "0"), ("prefill", 2048, "full", "calibrated"),
            ("prefill", 8192, "full", "0"), ("prefill", 8192, "full", "calibrated"),
            ("prefill", 8192, "r4", "calibrated"),
            ("prefill", 32768, "full", "0"), ("prefill", 32768, "full", "calibrated")]
    base_ms[("decode", 128)] = head["ms_step"]
    xs = {}
    for workload, T, kname, mode in plan:
        if T not in xs:
            xs[T] = synth.make_tokens(T, H, seed=1, device=dev)
        x = xs[T]
        y = torch.empty_like(x)
        steps = {"decode": 200, "prefill": max(3, 4096 * 10 // T)}[workload]
        wname = "%s_T%d_%s_beta-%s" % (workload, T, kname, mode)
        c = forward_case(layer_for(kname), x, y, beta_for(kname, mode), workload, wname, steps, 3, stream, dev,
                         rank, local, world, peaks, KEPT[kname], target_s=1.2 if workload == "decode" else 2.0,
                         max_s=6.0)
        if kname == "full" and mode == "0":
            base_ms[(workload, T)] = c["ms_step"]
        rf = c["roofline"]
        row = {"workload": wname, "tokens": T, "kept": kname, "beta": c["beta"], "pairs": c["pairs"],
               "experts_touched": c["touched"], "tokens_per_s": T / (c["ms_step"] * 1e-3),
               "ms_per_step": c["ms_step"], "ms_per_step_best": c["timing"]["ms_per_step_best"],
               "repeats": c["timing"]["repeats"], "steps_per_block": steps,
               "sm_cycles_per_step": c["timing"].get("sm_cycles_per_step_median"),
               "bound": rf["bound"], "kernel": rf["kernel"], "unit": rf["unit"],
               "gate_up_achieved": rf["achieved"], "gate_up_frac": rf["frac"],
               "down_frac": rf["down_kernel"]["frac"], "whole_step_frac": rf["whole_step_frac"],
               "stages": c["stages"], "clocks": c["clocks"]}
        if rf["bound"] == "tensor":
            row.update(flop_per_step=c["pairs"] * FLOP_PER_PAIR, whole_step_tflops=rf["whole_step_tflops"],
                       gate_up_frac_of_burst=rf["frac_of_burst"],
                       whole_step_frac_of_burst=rf["whole_step_frac_of_burst"],
                       gate_up_frac_of_nominal_dense_bf16=rf["frac_of_nominal_dense_bf16"],
                       peak_sustained=peaks["tf_sust"], peak_burst=peaks["tf_burst"])
        else:
            row.update(algorithmic_bytes=rf["algorithmic_bytes"], peak=peaks["hbm"])
        b = base_ms.get((workload, T))
        if b is not None and not (kname == "full" and mode == "0"):
            row["speedup_vs_unpruned_beta0"] = b / c["ms_step"]
        rows.append(row)
        del y
    xs.clear()
    # the search (layer with all experts kept)
    T = 32768
    x = synth.make_tokens(T, H, seed=1, device=dev)
    c = search_case(layer_for("full"), x, 3, 3, stream, dev, rank, local, world, peaks, target_s=1.5, max_s=8.0)
    rf = c["roofline"]
    rows.append({"workload": "search_T%d_r6+4" % T, "tokens": T, "subsets": 98,
                 "subsets_tokens_per_s": 98 * T / (c["ms_step"] * 1e-3), "ms_per_step": c["ms_step"],
                 "ms_per_step_best": c["timing"]["ms_per_step_best"], "repeats": c["timing"]["repeats"],
                 "steps_per_block": 3, "sm_cycles_per_step": c["timing"].get("sm_cycles_per_step_median"),
                 "bound": "tensor", "kernel": rf["kernel"], "unit": "TFLOP/s",
                 "flop_per_step": 6 * T * 6 * H * F, "gate_up_achieved": rf["achieved"],
                 "gate_up_frac": rf["frac"], "gate_up_frac_of_burst": rf["frac_of_burst"],
                 "down_frac": rf["down_kernel"]["frac"], "whole_step_tflops": rf["whole_step_tflops"],
                 "whole_step_frac": rf["whole_step_frac"], "whole_step_frac_of_burst": rf["whole_step_frac_of_burst"],
                 "enumerate_kernel": rf["enumerate_kernel"], "peak_sustained": peaks["tf_sust"],
                 "peak_burst": peaks["tf_burst"], "stages": c["stages"], "clocks": c["clocks"]})
    return rows


def stack_matrix_rows(stream, dev, rank, local, world, peaks, n_layers=32, T=16, cal_tokens=4096):
    """Two rows of the 32-layer stack (x <- x + MoE_l(RMSNorm(x)), a seed per layer, attention left
    out) at decode size: all experts kept, and pruned to r = 4 with each layer's subset from the
    layer-wise search on calibration states of the unpruned stack (searched while the unpruned
    stack is built).  The stacks are built one after the other: 90 GB, then 45 GB of weights."""
    from paper_2402_14800_b200 import binding
    x = synth.make_tokens(T, H, seed=1, device=dev)
    y = torch.empty_like(x)
    rows = []

    def time_stack(layers, name, masks, extra):
        for l in layers:
            l.set_stream(stream)
        betas = [0.0] * len(layers)
        touched = []
        with torch.cuda.stream(stream):
            cur = x
            stats = binding.RoutingStats(T, E, dev)
            for layer in layers:
                cur = layer.forward(binding.rmsnorm(cur, stream=stream), 0.0, residual=cur, stats=stats)
                stream.synchronize()
                touched.append(int(stats.n_experts_touched.item()))
        blocks, clocks = timed_blocks(lambda: binding.stack_forward(layers, x, betas, 1e-5, y), 3, 3, stream, dev,
                                      rank, local, world, target_s=1.0, max_s=5.0, min_repeats=10)
        tr = timing_record(blocks, 3, clocks)
        ms = tr["ms_per_step_median"]
        nbytes = sum(touched) * 3 * H * F * 2
        row = {"workload": name, "tokens": T, "layers": len(layers), "tokens_per_s": T / (ms * 1e-3),
               "ms_per_step": ms, "ms_per_step_best": tr["ms_per_step_best"], "repeats": tr["repeats"],
               "steps_per_block": 3, "weight_bytes": sum(l.weight_bytes for l in layers),
               "experts_touched_sum": sum(touched), "bound": "hbm", "unit": "GB/s",
               "algorithmic_bytes": nbytes, "whole_step_frac": nbytes / (ms * 1e-3) / 1e9 / peaks["hbm"],
               "peak": peaks["hbm"], "kept_masks": masks, "clocks": clocks}
        row.update(extra)
        return row

    # pass 1: the unpruned stack; every layer is searched for r = 4 on the way
    state = synth.make_tokens(cal_tokens, H, seed=1001, device=dev)
    layers, masks4, search_s = [], [], 0.0
    for l in range(n_layers):
        W = synth.make_layer_weights(H, F, E, seed=100 + l, device=dev)
        layer = binding.MoeLayer(W.W_gate, W.W1, W.W3, W.W2, 0xFF)
        del W
        if layers:
            layer.share_scratch(layers[0])
        xn = binding.rmsnorm(state)
        torch.cuda.synchronize(dev)
        t0 = time.perf_counter()
        masks4.append(layer.prune_search(xn, 4)[1])
        search_s += time.perf_counter() - t0
        state = layer.forward(xn, 0.0, residual=state)
        layers.append(layer)
    del state, xn
    rows.append(time_stack(layers, "stack%d_T%d_full_beta-0" % (n_layers, T), [0xFF] * n_layers, {}))
    for layer in reversed(layers):
        layer.close()
    layers = []
    torch.cuda.empty_cache()
    # pass 2: the stack pruned to the searched subsets
    for l in range(n_layers):
        W = synth.make_layer_weights(H, F, E, seed=100 + l, device=dev)
        layer = binding.MoeLayer(W.W_gate, W.W1, W.W3, W.W2, masks4[l])
        del W
        if layers:
            layer.share_scratch(layers[0])
        layers.append(layer)
    rows.append(time_stack(layers, "stack%d_T%d_r4_beta-0" % (n_layers, T), masks4,
                           {"search_wall_s_all_layers": search_s, "calibration_tokens": cal_tokens,
                            "speedup_vs_unpruned_beta0": rows[0]["ms_per_step"] / 1.0}))
    rows[1]["speedup_vs_unpruned_beta0"] = rows[0]["ms_per_step"] / rows[1]["ms_per_step"]
    for layer in reversed(layers):
        layer.close()
    torch.cuda.empty_cache()
    return rows


def run_ours(a):
    from paper_2402_14800_b200 import binding, build
    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (sm_100a); there is no CPU fallback")
    build.build()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    peaks = measured_peaks()
    barrier = make_barrier(world, dev)

    W, x, xcal = host_inputs(a, dev)
    kept = KEPT[a.kept]
    layer = binding.MoeLayer(W.W_gate, W.W1, W.W3, W.W2, kept if a.workload != "search" else 0xFF)
    stream = torch.cuda.Stream(dev)
    layer.set_stream(stream)
    beta = 0.0
    if a.beta == "calibrated" and a.workload != "search":
        beta = layer.calibrate_beta(xcal)
    T = a.tokens
    y = torch.empty_like(x)

    if a.workload == "search":
        c = search_case(layer, x, a.steps, a.warmup, stream, dev, rank, local, world, peaks, a.target_seconds)
        launches_per_step = c["launches_per_step"]
        pairs = touched = 0
    else:
        c = forward_case(layer, x, y, beta, a.workload, workload_name(a), a.steps, a.warmup, stream, dev, rank,
                         local, world, peaks, kept, a.target_seconds)
        launches_per_step = launches_per_forward(T)
        pairs, touched = c["pairs"], c["touched"]
    ms_step = c["ms_step"]
    value = whole_job_value(units_per_step(a), 1, ms_step, world)
    timing, clocks, roofline, stages = c["timing"], c["clocks"], c["roofline"], c["stages"]

    # end to end through the host-buffer entry point (forward workloads only)
    e2e = None
    if a.workload != "search":
        xh = x.cpu().pin_memory()
        yh = torch.empty_like(xh).pin_memory()
        for _ in range(3):
            layer.forward_host(xh, beta, yh)
        n_e2e = max(3, min(a.steps, 50))
        reps = []
        for _ in range(5):
            barrier()
            t0 = time.perf_counter()
            for _ in range(n_e2e):
                layer.forward_host(xh, beta, yh)
            torch.cuda.synchronize(dev)
            reps.append(time.perf_counter() - t0)
        dt = float(np.median(max_over_ranks_vec(reps, dev)))
        e2e = {"value": world * T * n_e2e / dt, "unit": "tokens/s", "h2d_bytes_per_step": T * H * 2,
               "d2h_bytes_per_step": T * H * 2,
               "timing": "host wall clock around %d C-ABI calls with host buffers, median of 5 such "
                         "blocks, max over ranks" % n_e2e}
    else:
        # the search already returns its losses to host memory inside the timed call
        e2e = {"value": value, "unit": "subsets*tokens/s", "h2d_bytes_per_step": 0,
               "d2h_bytes_per_step": 98 * 4 + 8,
               "timing": "inputs resident on device; losses and argmin are copied to the host inside the call"}

    # oracle on the host cores, bounded sample (rank 0, N = 1 only)
    cpu = None
    if rank == 0 and world == 1 and not a.no_cpu_baseline:
        from oracle import moe_oracle as O
        b = synth.bf16_bits
        Wh = dict(Wg=b(W.W_gate), W1=b(W.W1), W3=b(W.W3), W2=b(W.W2))
        xhb = b(x)
        n_sample = min(T, a.ref_sample if a.workload != "search" else max(4, a.ref_sample // 16))
        dt = oracle_sample(a, Wh, xhb, beta, n_sample)
        per_unit = 98 if a.workload == "search" else 1
        cpu = {"value": n_sample * per_unit / dt, "unit": metric_unit(a)[1], "cores": O.num_threads(),
               "kind": "oracle", "sample": "%d of %d tokens, one pass, %.1f s" % (n_sample, T, dt)}
        del Wh, xhb

    # reconstruction loss of the searched subset against the pruning baselines of the paper's
    # comparison (activation frequency, random), all on the same synthetic calibration batch
    baselines = None
    if a.workload == "search" and rank == 0:
        from itertools import combinations
        counts = layer.coselection(x)
        baselines = {}
        for r_, (losses, best) in zip((6, 4), layer.prune_search_multi(x, [6, 4])):
            masks = [sum(1 << i for i in c_) for c_ in combinations(range(E), r_)]
            fmask = layer.frequency_subset(counts, r_)
            baselines["r%d" % r_] = {"searched_subset": best, "searched_loss": min(losses),
                                     "frequency_subset": fmask, "frequency_loss": losses[masks.index(fmask)],
                                     "random_mean_loss": float(np.mean(losses)),
                                     "worst_loss": max(losses)}

        # concentration of ||f_e0 - f_e1|| that the appendix' derivation of the skipping rule assumes
        d = layer.top2_distance(x[:min(T, 8192)].contiguous()).double()
        baselines["top2_distance"] = {"tokens": int(d.numel()), "mean": float(d.mean()),
                                      "std_over_mean": float(d.std() / d.mean())}

    # the rest of the configured workloads (single GPU, default workload only)
    matrix = None
    if a.matrix and world == 1 and rank == 0 and workload_name(a) == "decode_T128_full_beta-0":
        layers = {a.kept: layer}
        t0 = time.perf_counter()
        # the headline line must come out whatever happens in the extra rows
        matrix = []
        try:
            matrix_rows(W, xcal, layers, stream, dev, rank, local, world, peaks, c, matrix)
        except Exception as e:  # noqa: BLE001
            matrix.append({"workload": "matrix", "error": repr(e)})
        for k, l in layers.items():
            if l is not layer:
                l.close()
        if a.stack_rows:
            del W
            W = None
            torch.cuda.empty_cache()
            try:
                matrix += stack_matrix_rows(stream, dev, rank, local, world, peaks)
            except Exception as e:  # noqa: BLE001
                matrix.append({"workload": "stack rows", "error": repr(e)})
        matrix_s = time.perf_counter() - t0

    if rank == 0:
        metric, unit = metric_unit(a)
        line = {
            "metric": metric, "value": value, "unit": unit, "n_gpus": world, "steps": a.steps,
            "warmup": max(a.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": layer_config(a, T, kept, beta, pairs, touched, world),
            "timing": timing, "clocks": clocks, "e2e": e2e,
            "gpu_launches": launches_per_step * a.steps * timing["repeats"],
            "gpu_launches_per_step": launches_per_step, "roofline": roofline,
            "cpu_baseline": cpu, "stages": stages,
        }
        if baselines:
            line["pruning_baselines"] = baselines
        if matrix is not None:
            line["matrix"] = matrix
            line["matrix_wall_s"] = matrix_s
        print(json.dumps(line), flush=True)
    layer.close()
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    return 0


# ----------------------------------------------------------------- stack of 32 layers

def run_stack(a):
    """x_{l+1} = x_l + MoE_l(RMSNorm(x_l)) over `--layers` Mixtral-shaped layers (attention left
    out), each layer with its own seed.  Pruned variants take each layer's kept subset from the
    layer-wise search on calibration states of the unpruned stack; beta is calibrated per layer."""
    from paper_2402_14800_b200 import binding, build
    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (sm_100a); there is no CPU fallback")
    build.build()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    peaks = measured_peaks()
    T, NL = a.tokens, a.layers
    r = {"full": 8, "r6": 6, "r4": 4}[a.kept]
    x = synth.make_tokens(T, H, seed=1, device=dev)
    state = synth.make_tokens(a.cal_tokens, H, seed=1001, device=dev)
    layers, betas, masks, search_ms = [], [], [], 0.0
    # the result of an earlier search of the same stack (masks, losses, betas) is reloaded
    # instead of searching again: the pruned layers are then built straight from the masks
    from paper_2402_14800_b200 import pruning_io
    pmeta = {"E": E, "r": r, "n_layers": NL, "h": H, "f": F, "calibration_tokens": a.cal_tokens,
             "search_mode": a.search_mode if r < 8 else "none", "weight_seed0": 100, "calibration_seed": 1001}
    pfile = a.pruning_file or "pruning_stack%d_%s_%s_cal%d.json" % (NL, a.kept, a.search_mode, a.cal_tokens)
    loaded = None
    if r < 8 and os.path.exists(pfile) and not a.research:
        loaded = pruning_io.load_pruning(pfile, expect_meta=pmeta)
    all_losses, cal_betas = [], []
    state_p = state.clone() if (r < 8 and a.search_mode == "progressive" and loaded is None) else None
    if loaded is not None:
        for l in range(NL):
            W = synth.make_layer_weights(H, F, E, seed=100 + l, device=dev)
            layer = binding.MoeLayer(W.W_gate, W.W1, W.W3, W.W2, loaded[l]["kept_mask"])
            if layers:
                layer.share_scratch(layers[0])
            layers.append(layer)
            masks.append(loaded[l]["kept_mask"])
            betas.append(loaded[l]["beta"] if a.beta == "calibrated" else 0.0)
            del W
    for l in range(NL if loaded is None else 0):
        W = synth.make_layer_weights(H, F, E, seed=100 + l, device=dev)
        xn = binding.rmsnorm(state)
        xn_cal = xn
        if r == 8:
            layer = binding.MoeLayer(W.W_gate, W.W1, W.W3, W.W2, 0xFF)
            if layers:
                layer.share_scratch(layers[0])
            state = layer.forward(xn, 0.0, residual=state)
            mask = 0xFF
        else:
            full = binding.MoeLayer(W.W_gate, W.W1, W.W3, W.W2, 0xFF)
            if layers:
                full.share_scratch(layers[0])  # one set of search scratch for the whole stack
            torch.cuda.synchronize(dev)
            t0 = time.perf_counter()
            if state_p is None:
                # layer-wise: every layer is searched on the unpruned stack's states
                losses_l, mask = full.prune_search(xn, r)
            else:
                # progressive: input from the pruned stack so far, target from the unpruned stack
                F_ref = full.forward(xn, 0.0).float()
                xn_cal = binding.rmsnorm(state_p)
                losses_l, mask = full.prune_search_progressive(xn_cal, F_ref, r)
                del F_ref
            all_losses.append(losses_l)
            search_ms += 1e3 * (time.perf_counter() - t0)
            state = full.forward(xn, 0.0, residual=state)
            torch.cuda.synchronize(dev)
            full.close()
            layer = binding.MoeLayer(W.W_gate, W.W1, W.W3, W.W2, mask)
            if layers:
                layer.share_scratch(layers[0])
            if state_p is not None:
                state_p = layer.forward(xn_cal, 0.0, residual=state_p)
        cal_betas.append(layer.calibrate_beta(xn_cal))   # stored with the masks whatever --beta says
        betas.append(cal_betas[-1] if a.beta == "calibrated" else 0.0)
        masks.append(mask)
        layers.append(layer)
        del W
    if r < 8 and loaded is None and rank == 0:
        pruning_io.save_pruning(pfile, pmeta, [{"kept_mask": m, "losses": ls, "beta": b}
                                               for m, ls, b in zip(masks, all_losses, cal_betas)])
    # how far the pruned stack's calibration states ended up from the unpruned stack's
    drift = None
    if loaded is not None:
        pass
    elif state_p is not None:
        drift = float((state_p.float() - state.float()).norm() / state.float().norm())
    elif r < 8:
        sp = synth.make_tokens(a.cal_tokens, H, seed=1001, device=dev)
        for layer in layers:
            sp = layer.forward(binding.rmsnorm(sp), 0.0, residual=sp)
        drift = float((sp.float() - state.float()).norm() / state.float().norm())
        del sp
    del state
    stream = torch.cuda.Stream(dev)
    for layer in layers:
        layer.set_stream(stream)
    weight_bytes = sum(l.weight_bytes for l in layers)
    y = torch.empty_like(x)

    # routing facts per layer (untimed): experts touched and pairs, along the real trajectory
    touched, pairs = [], []
    with torch.cuda.stream(stream):
        cur = x
        stats = binding.RoutingStats(T, E, dev)
        for layer, b in zip(layers, betas):
            xn = binding.rmsnorm(cur, stream=stream)
            cur = layer.forward(xn, b, residual=cur, stats=stats)
            stream.synchronize()
            touched.append(int(stats.n_experts_touched.item()))
            pairs.append(2 * T - int(stats.n_skipped.item()))

    def step():
        binding.stack_forward(layers, x, betas, 1e-5, y)

    barrier = make_barrier(world, dev)
    blocks, clocks = timed_blocks(step, a.steps, a.warmup, stream, dev, rank, local, world, a.target_seconds,
                                  max_s=30.0, min_repeats=min(MIN_REPEATS, 10))
    timing = timing_record(blocks, a.steps, clocks)
    ms_step = timing["ms_per_step_median"]
    value = whole_job_value(T, 1, ms_step, world)

    xh = x.cpu().pin_memory()
    yh = torch.empty_like(xh).pin_memory()
    xd = torch.empty_like(x)
    n_e2e = max(3, min(a.steps, 20))
    barrier()
    t0 = time.perf_counter()
    with torch.cuda.stream(stream):
        for _ in range(n_e2e):
            xd.copy_(xh, non_blocking=True)
            binding.stack_forward(layers, xd, betas, 1e-5, y)
            yh.copy_(y, non_blocking=True)
            stream.synchronize()
    dt = time.perf_counter() - t0
    e2e = {"value": world * T * n_e2e / dt, "unit": "tokens/s", "h2d_bytes_per_step": T * H * 2,
           "d2h_bytes_per_step": T * H * 2,
           "timing": "host wall clock; pinned-host copies around moe_stack_forward on one stream"}

    if T <= 256:
        nbytes = sum(touched) * 3 * H * F * 2
        ach = nbytes / (ms_step * 1e-3) / 1e9
        roofline = {"bound": "hbm", "kernel": "whole stack step (weight-major GEMMs dominate)",
                    "achieved": ach, "peak": peaks["hbm"], "unit": "GB/s", "frac": ach / peaks["hbm"],
                    "traffic": None, "peak_source": peaks["source"], "algorithmic_bytes": nbytes}
    else:
        flop = sum(pairs) * FLOP_PER_PAIR
        ach = flop / (ms_step * 1e-3) / 1e12
        roofline = {"bound": "tensor", "kernel": "whole stack step (token-major GEMMs dominate)",
                    "achieved": ach, "peak": peaks["tf_sust"], "unit": "TFLOP/s",
                    "frac": ach / peaks["tf_sust"], "traffic": None,
                    "frac_of_burst": ach / peaks["tf_burst"],
                    "frac_of_nominal_dense_bf16": ach / NOMINAL_BF16_TFLOPS,
                    "peak_source": peaks["source"] + " (sustained bf16)"}
    if rank == 0:
        per_layer = ((2 if single_token_gemv() else 4) if T == 1 else (5 if T <= 256 else 7)) + 1   # the layer's kernels + its RMSNorm
        line = {
            "metric": "MoE-stack tokens/s on 1 B200 (32 layers, RMSNorm + residual, attention omitted)",
            "value": value, "unit": "tokens/s", "n_gpus": world, "steps": a.steps,
            "warmup": max(a.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "stack%d_T%d_%s_beta-%s" % (NL, T, a.kept, a.beta), "h": H, "f": F,
                       "E": E, "tokens": T, "layers": NL, "kept_masks": masks,
                       "betas": [round(b, 4) for b in betas], "weight_bytes": weight_bytes,
                       "experts_touched_sum": sum(touched), "pairs_sum": sum(pairs),
                       "search_ms_total": search_ms, "calibration_tokens": a.cal_tokens,
                       "pruning_file": (pfile if r < 8 else None),
                       "pruning_reloaded": loaded is not None,
                       "search_mode": a.search_mode if r < 8 else None,
                       "final_state_rel_error_vs_unpruned": drift,
                       "parallelism": "replicas x%d, no collective" % world,
                       "l2": "each layer streams its own weights (GBs), far above the 126 MB L2"},
            "timing": timing, "clocks": clocks, "e2e": e2e,
            "gpu_launches": per_layer * NL * a.steps * timing["repeats"],
            "roofline": roofline, "cpu_baseline": None, "stages": None,
        }
        print(json.dumps(line), flush=True)
    for layer in reversed(layers):
        layer.close()
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="decode", choices=["decode", "prefill", "search", "stack"])
    ap.add_argument("--layers", type=int, default=32)
    ap.add_argument("--cal-tokens", type=int, default=4096)
    ap.add_argument("--search-mode", default="layerwise", choices=["layerwise", "progressive"])
    ap.add_argument("--pruning-file", default=None,
                    help="stack workload: JSON with the per-layer kept masks, losses and betas; reloaded when it "
                         "exists and matches, written after a search (default: a name derived from the configuration)")
    ap.add_argument("--research", action="store_true", help="stack workload: search again even if the file exists")
    ap.add_argument("--tokens", type=int, default=None)
    ap.add_argument("--beta", default="0", choices=["0", "calibrated"])
    ap.add_argument("--kept", default="full", choices=list(KEPT))
    ap.add_argument("--search-r", default="6+4")
    ap.add_argument("--ref-sample", type=int, default=128)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-matrix", dest="matrix", action="store_false",
                    help="headline workload only (the default decode run also measures the other configured workloads)")
    ap.add_argument("--min-repeats", type=int, default=30,
                    help="blocks of --steps steps in the timed region at least (1 with --target-seconds 0 for a profiler)")
    ap.add_argument("--no-stack-rows", dest="stack_rows", action="store_false",
                    help="leave the two 32-layer stack rows (90 GB + 45 GB of weights) out of the matrix")
    ap.add_argument("--target-seconds", type=float, default=1.5,
                    help="device time the repeated blocks of the timed region should cover")
    a = ap.parse_args()
    global MIN_REPEATS
    MIN_REPEATS = max(1, a.min_repeats)
    if a.tokens is None:
        a.tokens = {"decode": 128, "prefill": 8192, "search": 32768, "stack": 16}[a.workload]
    if a.steps is None:
        a.steps = {"decode": 2000, "prefill": 100, "search": 5, "stack": 10}[a.workload] if a.impl == "ours" else 5
    if a.impl == "reference":
        return run_reference(a)
    if a.workload == "stack":
        return run_stack(a)
    return run_ours(a)


if __name__ == "__main__":
    sys.exit(main())
