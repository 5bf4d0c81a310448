#!/usr/bin/env python
"""Benchmark of the encoder hot path (plan -> varlen attention fwd -> bwd -> merge) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A step is one pass of the whole hot path over one synthetic microbatch shaped like the ViT-L
configuration: 32 variable-resolution images (256-4096 patches each), 16 heads of 64, bf16,
encoder trained (forward + backward), the encoder output merged into 16 x 8192 LLM tokens.
With N > 1 (torchrun, one rank per GPU) every rank runs its own microbatch (weak scaling, no
data-path collective); the reported value is the whole job's attention TFLOP/s.

Prints ONE JSON line.  `--impl reference` times the fp64 CPU oracle on a bounded sample of the same
workload on the host cores (rank 0 only).
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2607_03229_b200 import workloads as W  # noqa: E402

METRIC = "varlen encoder attn fwd+bwd TFLOP/s & % BF16 peak; merge GB/s (1 B200)"
UNIT = "TFLOP/s"
NOMINAL_BF16_TFLOPS = 2250.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


WORKLOADS = {
    "vit_l": lambda seed: W.vit_l(seed=seed),
    "qwen2vl": lambda seed: W.qwen2vl(seed=seed + 1),
    "qwen2vl_frozen": lambda seed: W.qwen2vl(seed=seed + 1, trained=False),
    "video_tail": lambda seed: W.video_tail(seed=seed + 2),
    "mix10": lambda seed: W.modality_mix(0.10, seed=seed + 3),
    "mix25": lambda seed: W.modality_mix(0.25, seed=seed + 3),
    "mix50": lambda seed: W.modality_mix(0.50, seed=seed + 3),
    "mix75": lambda seed: W.modality_mix(0.75, seed=seed + 3),
    "mix75_frozen": lambda seed: W.modality_mix(0.75, seed=seed + 3, trained=False),
    "tiny": lambda seed: W.tiny(seed=seed - 1),
}
WORKLOAD_TEXT = {
    "vit_l": "vit_l: 32 images of 16..64 x 16..64 patches packed varlen, 16 heads x 64, bf16, trained (fwd+bwd), + merge "
             "of the encoder output into 16 x 8192 LLM tokens at hidden 1024",
    "qwen2vl": "qwen2vl: patch counts log-uniform in [64,16384] packed to 65536 tokens, 16 heads x 80, bf16, trained",
    "qwen2vl_frozen": "qwen2vl: patch counts log-uniform in [64,16384] packed to 65536 tokens, 16 heads x 80, bf16, frozen",
    "video_tail": "video_tail: 200 images of 64..256 patches + 4 clips of 16384 tokens, 16 heads x 80, bf16, trained",
    "mix10": "modality mix 10%: 8 x 8192 LLM tokens at hidden 4096, images of 256..4096 patches, 16 heads x 64, trained, + merge",
    "mix25": "modality mix 25%: 8 x 8192 LLM tokens at hidden 4096, images of 256..4096 patches, 16 heads x 64, trained, + merge",
    "mix50": "modality mix 50%: 8 x 8192 LLM tokens at hidden 4096, images of 256..4096 patches, 16 heads x 64, trained, + merge",
    "mix75": "modality mix 75%: 8 x 8192 LLM tokens at hidden 4096, images of 256..4096 patches, 16 heads x 64, trained, + merge",
    "mix75_frozen": "modality mix 75%: 8 x 8192 LLM tokens at hidden 4096, images of 256..4096 patches, 16 heads x 64, frozen, + merge",
    "tiny": "tiny: 4 images of 16/49/64/100 patches, 4 heads x 64, trained, + merge into 512 tokens at hidden 256",
}
_WORKLOAD_NAME = "vit_l"


def workload_for(rank: int):
    """The benchmark's microbatch for one rank (default: the ViT-L configuration the metric is quoted on)."""
    from paper_2607_03229_b200 import dist as D
    return WORKLOADS[_WORKLOAD_NAME](D.rank_seed(W.BASE_SEED + 2, rank))


# ----------------------------------------------------------------------------- oracle sample (CPU arms)
def oracle_sample(w, target_flops: float):
    """A bounded sample of the workload for the CPU oracle: (segment, head) pairs taken in the order
    (s0,h0), (s1,h0), ..., (s_last,h0), (s0,h1), ... -- the segment list is in drawing order, not sorted by size,
    so a prefix of this order sees the workload's mix of segment lengths -- until their algorithmic fwd+bwd FLOPs
    (14 * D * n^2 each) reach `target_flops`.  Both CPU legs (cpu_baseline and --impl reference) use this rule."""
    counts = [int(n) for n in w.patch_counts]
    segs = [i for i, n in enumerate(counts) if n > 0]
    pairs, acc = [], 0.0
    for h in range(w.n_heads):
        for sgm in segs:
            if pairs and acc >= target_flops:
                return pairs, acc
            pairs.append((sgm, h))
            acc += 14.0 * w.head_dim * counts[sgm] * counts[sgm]
    return pairs, acc


def sample_text(w, pairs, flops):
    n_seg = len({p_[0] for p_ in pairs})
    n_all = sum(1 for n in w.patch_counts if n > 0) * w.n_heads
    return (f"{len(pairs)} of {n_all} (segment, head) pairs ({n_seg} distinct segments, heads 0..{max(p_[1] for p_ in pairs)}; "
            f"{flops:.3g} algorithmic fwd+bwd FLOPs), one oracle call per pair on contiguous slices")


def oracle_inputs(w, pairs):
    """Seeded bf16 inputs of the sampled pairs (one [n, 1, D] quadruple per pair) and a merge problem over the
    sampled segments' tokens."""
    cu = np.concatenate([[0], np.cumsum(w.patch_counts)]).astype(np.int64)
    per_pair = []
    for i, (sgm, h) in enumerate(pairs):
        n = int(w.patch_counts[sgm])
        per_pair.append(tuple(W.normal_bf16(w.seed + i, 10 + j, (n, 1, w.head_dim)) for j in range(4)))
    merge = None
    if w.merge_hidden is not None:
        segs = sorted({p_[0] for p_ in pairs})
        rows = np.concatenate([np.arange(cu[s_], cu[s_ + 1]) for s_ in segs])
        pos = w.positions[rows].astype(np.int32)
        pos = (pos - pos.min()).astype(np.int32)
        merge = (W.normal_bf16(w.seed, 20, (rows.size, w.merge_hidden)),
                 W.normal_bf16(w.seed, 21, (int(pos.max()) + 1, w.merge_hidden)), pos)
    return per_pair, merge


def run_oracle_sample(w, pairs, inputs):
    """One oracle pass over the sample: the plan, then forward and backward of every sampled pair, then the merge
    of the sampled segments' rows.  Returns seconds."""
    import oracle
    per_pair, merge = inputs
    t0 = time.perf_counter()
    oracle.seg_plan(w.patch_counts, 256, 128, True)
    for (sgm, h), (q, k, v, do) in zip(pairs, per_pair):
        cu = np.array([0, q.shape[0]], dtype=np.int32)
        oracle.attn_fwd(q, k, v, cu, w.softmax_scale)
        oracle.attn_bwd(do, q, k, v, cu, w.softmax_scale)
    if merge is not None:
        oracle.merge_tokens(*merge)
    return time.perf_counter() - t0


def calibrate_oracle_rate(w) -> float:
    """Algorithmic FLOP/s of the oracle on this host, from a one-segment, one-head run."""
    import oracle
    n, D = 768, w.head_dim
    x = [W.normal_bf16(1, i, (n, 1, D)) for i in range(4)]
    cu = np.array([0, n], dtype=np.int32)
    oracle.attn_fwd(x[0], x[1], x[2], cu, 0.125)  # builds / loads the library
    t0 = time.perf_counter()
    oracle.attn_fwd(x[0], x[1], x[2], cu, 0.125)
    oracle.attn_bwd(x[3], x[0], x[1], x[2], cu, 0.125)
    dt = time.perf_counter() - t0
    return 14.0 * D * n * n / dt


def reference_arm(args):
    """The oracle, as it stands, on the host cores; every step is one pass over a bounded sample (same selection rule
    as cpu_baseline) sized so that warm-up + steps end within about 150 s."""
    from paper_2607_03229_b200 import dist as D
    rank, _, world = D.env_world()
    if rank != 0:
        return 0
    import oracle
    w = workload_for(0)
    rate = calibrate_oracle_rate(w)
    budget_s = min(20.0, 150.0 / max(1, args.steps + args.warmup))
    pairs, flops = oracle_sample(w, min(rate * budget_s, w.flops()))
    inputs = oracle_inputs(w, pairs)
    for _ in range(args.warmup):
        run_oracle_sample(w, pairs, inputs)
    times = [run_oracle_sample(w, pairs, inputs) for _ in range(args.steps)]
    ms = 1e3 * float(np.mean(times))
    value = flops / (ms * 1e-3) / 1e12
    sample = sample_text(w, pairs, flops)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD_TEXT[_WORKLOAD_NAME] + "; one microbatch per GPU", "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.n_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_uuid: str):
        self.uuid = gpu_uuid
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.uuid, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.perf_counter(), line.strip()))

    def stop(self, t_begin: float, t_end: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"], "samples": 0}
        time.sleep(0.06)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        rows = [ln for (t, ln) in self.lines if t_begin <= t <= t_end + 0.05] or [ln for (_, ln) in self.lines[-1:]]
        sm, mx, reasons, power = [], [], set(), []
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for ln in rows:
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
                power.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower() == "active":
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------- our arm
SM_COUNT = 148
DENSE_BF16_FLOPS_PER_CLK_PER_SM = 8192.0     # tcgen05 kind::f16, dense: the tensor pipe's cycle peak


def gpu_uuid(torch, dev, local_rank):
    props = torch.cuda.get_device_properties(dev)
    return "GPU-" + str(props.uuid) if hasattr(props, "uuid") else str(local_rank)


def timed_region(torch, B, H, w, buf, K, sampler_uuid, barrier):
    """K whole steps between two events (barrier + synchronize on both sides), with the library's own events
    around the forward, backward-main and merge kernels of every step.  Returns ms per step, mean ms per kernel
    and the clocks sampled meanwhile."""
    kernels = ["fwd"] + (["bwd_main"] if w.trained else []) + (["merge"] if w.merge_hidden is not None else [])
    slots = {"fwd": B.PROFILE_FWD, "bwd_main": B.PROFILE_BWD_MAIN, "merge": B.PROFILE_MERGE}
    ev = {name: [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
          for name in kernels}
    for name in ev:                      # create the event handles before the region
        for a_, b_ in ev[name]:
            a_.record(), b_.record()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(sampler_uuid)
    torch.cuda.synchronize()
    barrier()
    sampler.start()
    time.sleep(0.12)
    torch.cuda.synchronize()
    t_begin = time.perf_counter()
    e0.record()
    for i in range(K):
        for name in kernels:
            B.load().mpipe_set_profile_events(slots[name], ev[name][i][0].cuda_event, ev[name][i][1].cuda_event)
        H.run_step(w, buf)
    e1.record()
    torch.cuda.synchronize()
    t_end = time.perf_counter()
    for slot in slots.values():
        B.load().mpipe_set_profile_events(slot, None, None)
    barrier()
    clocks = sampler.stop(t_begin, t_end)
    assert int(buf.status[0]) == 0, f"device status {buf.status.tolist()}"
    kern_ms = {name: float(np.mean([a_.elapsed_time(b_) for a_, b_ in ev[name]])) for name in ev}
    return e0.elapsed_time(e1) / K, kern_ms, clocks


def rates(w, ms_step, kern_ms, clocks, peaks):
    """TFLOP/s and GB/s of one measured region, with the fractions of every peak and of the tensor pipe's cycle
    peak at the sampled clock (FLOPs / (time x median SM MHz x 148 SMs x 8192 FLOPs per clock))."""
    T = w.total_tokens
    out = {"ms_per_step": ms_step, "step_tflops": w.flops(True, w.trained) / (ms_step * 1e-3) / 1e12,
           "sm_mhz": clocks.get("sm_mhz"), "reasons": clocks.get("reasons"), "clock_samples": clocks.get("samples")}
    mhz = clocks.get("sm_mhz") or 0.0
    cyc_peak = mhz * 1e6 * SM_COUNT * DENSE_BF16_FLOPS_PER_CLK_PER_SM / 1e12 if mhz else None

    def tf(flops, ms):
        return flops / (ms * 1e-3) / 1e12

    out["fwd_ms"], out["fwd_tflops"] = kern_ms["fwd"], tf(w.flops(True, False), kern_ms["fwd"])
    if w.trained:
        out["bwd_main_ms"], out["bwd_main_tflops"] = kern_ms["bwd_main"], tf(w.flops(False, True), kern_ms["bwd_main"])
    if w.merge_hidden is not None and T > 0:
        out["merge_ms"] = kern_ms["merge"]
        out["merge_gbs"] = float(T) * (4 * w.merge_hidden + 4) / (kern_ms["merge"] * 1e-3) / 1e9
        out["merge_frac_of_hbm_peak"] = out["merge_gbs"] / peaks["hbm_gbs"]
    out["step_frac"] = {"of_measured_burst": out["step_tflops"] / peaks["bf16_tflops"],
                        "of_measured_sustained": out["step_tflops"] / peaks["bf16_tflops_sustained"],
                        "of_nominal_2250": out["step_tflops"] / NOMINAL_BF16_TFLOPS,
                        "of_cycle_peak_at_sampled_clock": out["step_tflops"] / cyc_peak if cyc_peak else None}
    return out


def repeat_count(ms_per_step: float, K: int, min_seconds: float, cap: int = 40) -> int:
    """How many K-step regions to time so that they cover `min_seconds` of GPU time, between 1 and `cap`."""
    return int(min(cap, max(1, np.ceil(min_seconds * 1e3 / max(ms_per_step * K, 1e-3)))))


def pick_peak(clocks, peaks):
    """The measured peak whose clock regime matches the run.  The burst GEMM figure was taken at the maximum SM
    clock, the sustained one power-capped at about two thirds of it: a run whose median sampled clock is within
    5 % of the maximum is compared with the burst figure, any other with the sustained one.  Both fractions and the
    clock-independent fraction of the tensor pipe's cycle peak are printed next to the chosen one."""
    mhz, mx = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
    if mhz and mx and mhz >= 0.95 * mx:
        return peaks["bf16_tflops"], f"burst bf16 GEMM (median SM clock {mhz:.0f} MHz = full clock)"
    return peaks["bf16_tflops_sustained"], f"sustained bf16 GEMM (median SM clock {mhz} MHz, below full clock)"


def merge_rotating(torch, B, w, dev, n_sets=4, iters=12):
    """The merge alone over `n_sets` rotating source / destination sets, so that nothing a launch touches is
    still in L2 from the previous launch of the same set (4 sets x ~0.9 GB against 126 MB of L2)."""
    T, hid = w.total_tokens, w.merge_hidden
    pos = torch.from_numpy(np.ascontiguousarray(w.positions, dtype=np.int32)).to(dev)
    srcs = [torch.randn((T, hid), device=dev, dtype=torch.float32).to(torch.bfloat16) for _ in range(n_sets)]
    embs = [torch.zeros((w.n_llm_tokens, hid), device=dev, dtype=torch.bfloat16) for _ in range(n_sets)]
    st = torch.zeros(4, dtype=torch.int32, device=dev)
    for i in range(n_sets):
        B.merge_tokens(srcs[i], embs[i], pos, B.TRAINED, st)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
    torch.cuda.synchronize()
    for i, (a_, b_) in enumerate(evs):
        a_.record()
        B.merge_tokens(srcs[i % n_sets], embs[i % n_sets], pos, B.TRAINED, st)
        b_.record()
    torch.cuda.synchronize()
    assert int(st[0]) == 0
    ms = float(np.median([a_.elapsed_time(b_) for a_, b_ in evs]))
    nbytes = float(T) * (4 * hid + 4)
    return {"ms": ms, "gbs": nbytes / (ms * 1e-3) / 1e9, "algorithmic_bytes": nbytes, "buffer_sets": n_sets,
            "launches": iters + n_sets}


def recorded_traffic(kernel: str, workload: str):
    """DRAM bytes per launch from the tracked ncu summary table (profiles/dram_traffic.json), or None."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    try:
        with open(path) as f:
            return json.load(f).get(f"{kernel}@{workload}")
    except (OSError, ValueError):
        return None


CONFIG_BLOCK = ("qwen2vl", "qwen2vl_frozen", "video_tail", "mix10", "mix25", "mix50", "mix75")


def ours_arm(args):
    import torch
    from paper_2607_03229_b200 import binding as B
    from paper_2607_03229_b200 import dist as D
    from paper_2607_03229_b200 import hotpath as H

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    rank, local_rank, world = D.init("nccl")
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}: launch N>1 with torchrun, one rank per GPU")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    B.load()
    peaks, peak_kind = load_peaks()
    uuid = gpu_uuid(torch, dev, local_rank)

    w = workload_for(rank)
    T, Hh, Dh = w.total_tokens, w.n_heads, w.head_dim
    buf = H.allocate(w, dev)
    n_kernels = H.kernels_per_step(w)
    K, Wm = args.steps, max(args.warmup, 3)

    for _ in range(Wm):
        H.run_step(w, buf)
    torch.cuda.synchronize()
    assert int(buf.status[0]) == 0, f"device status {buf.status.tolist()}"

    # ---- timed regions: K whole steps each, inputs resident in HBM.  The K-step region is repeated R times so
    # that the measurement covers at least ~2 s of GPU time (clocks settle, the sampler sees them); ms_per_step
    # is the median over the repeats and every repeat's clocks are reported.
    ms0, _, _ = timed_region(torch, B, H, w, buf, K, uuid, D.barrier)
    # every rank must run the same number of regions (each one ends in a barrier): the count comes from the
    # slowest rank's first region, not from this rank's
    (ms0_all,), _ = D.reduce_max_sum([ms0], [0.0], device=dev)
    R = 1 if args.profile_mode else repeat_count(ms0_all, K, args.min_seconds)
    repeats = [timed_region(torch, B, H, w, buf, K, uuid, D.barrier) for _ in range(R)]
    order = np.argsort([r[0] for r in repeats])
    ms_step, kern_ms, clocks = repeats[int(order[len(order) // 2])]
    region_total_s = sum(r[0] for r in repeats) * K * 1e-3
    launches_timed = n_kernels * K * (R + 1)

    # ---- end to end: host buffers in, results out, copies inside the timed region.  Every step copies its
    # own inputs from pinned host memory and its own results back; three streams and two device buffer sets
    # let the upload of step i+1 and the download of step i-1 run beside the kernels of step i.
    Ke = 1 if args.profile_mode else min(K, 30)
    bufs = [buf, H.allocate(w, dev)]

    def ins(bf):
        return [bf.q, bf.k, bf.v] + ([bf.dout] if w.trained else [])

    def outs(bf):
        return [bf.o] + ([bf.dq, bf.dk, bf.dv] if w.trained else [])

    host_in = [torch.empty(tuple(x.shape), dtype=torch.bfloat16).pin_memory() for x in ins(buf)]
    for hbuf, dbuf in zip(host_in, ins(buf)):
        hbuf.copy_(dbuf)
    host_out = [[torch.empty(tuple(x.shape), dtype=torch.bfloat16).pin_memory() for x in outs(buf)] for _ in range(2)]
    h2d = sum(x.numel() * x.element_size() for x in host_in) + (w.positions.nbytes if w.positions is not None else 0)
    d2h = sum(x.numel() * x.element_size() for x in host_out[0])
    s_in, s_run, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    ev_in = [torch.cuda.Event() for _ in range(2)]      # inputs of buffer set j are on the device
    ev_run = [torch.cuda.Event() for _ in range(2)]     # kernels on buffer set j are done
    ev_out = [torch.cuda.Event() for _ in range(2)]     # results of buffer set j are on the host

    def e2e_steps(n):
        for i in range(n):
            j = i & 1
            with torch.cuda.stream(s_in):
                s_in.wait_event(ev_run[j])               # the kernels that last read these inputs are done
                for hbuf, dbuf in zip(host_in, ins(bufs[j])):
                    dbuf.copy_(hbuf, non_blocking=True)
                ev_in[j].record(s_in)
            with torch.cuda.stream(s_run):
                s_run.wait_event(ev_in[j])
                s_run.wait_event(ev_out[j])              # the previous results of this set have been read back
                H.run_step(w, bufs[j], stream=s_run)     # includes the host plan and its upload
                ev_run[j].record(s_run)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_run[j])
                for hbuf, dbuf in zip(host_out[j], outs(bufs[j])):
                    hbuf.copy_(dbuf, non_blocking=True)
                ev_out[j].record(s_out)

    torch.cuda.synchronize()
    e2e_steps(2)
    torch.cuda.synchronize()
    D.barrier()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record(s_in)
    e2e_steps(Ke)
    s_out.synchronize()
    f1.record(s_out)
    torch.cuda.synchronize()
    D.barrier()
    ms_e2e = max(f0.elapsed_time(f1), 0.0) / Ke
    assert all(int(b_.status[0]) == 0 for b_ in bufs)
    del bufs, host_in, host_out

    # ---- the other configurations, a few steps each (rank 0 of a 1-GPU run only): evidence for head_dim 80, the
    # largest configuration and the modality-mix sweep on the same box and build as the headline line
    configs = {}
    merge_rot = None
    if world == 1 and not args.profile_mode and _WORKLOAD_NAME == "vit_l" and not args.no_configs:
        del buf
        torch.cuda.empty_cache()
        for name in CONFIG_BLOCK:
            wc = WORKLOADS[name](W.BASE_SEED + 2)
            bc = H.allocate(wc, dev)
            for _ in range(3):
                H.run_step(wc, bc)
            torch.cuda.synchronize()
            kc = int(min(30, max(5, np.ceil(300.0 / max(1e-3, 1e3 * wc.flops(True, wc.trained) / 700e12)))))
            ms_c, kern_c, clk_c = timed_region(torch, B, H, wc, bc, kc, uuid, D.barrier)
            configs[name] = dict(rates(wc, ms_c, kern_c, clk_c, peaks), steps=kc, tokens=wc.total_tokens, sum_n2=wc.sum_n2,
                                 heads=wc.n_heads, head_dim=wc.head_dim, mode="trained" if wc.trained else "frozen")
            launches_timed += H.kernels_per_step(wc) * kc
            if name == "mix75":
                merge_rot = merge_rotating(torch, B, wc, dev)
                launches_timed += merge_rot["launches"]
            del bc
            torch.cuda.empty_cache()

    # ---- reduce over ranks: max of times, sum of work
    flops_step = w.flops(True, w.trained)
    (ms_step_mx, ms_e2e_mx), (flops_all, launches) = D.reduce_max_sum(
        [ms_step, ms_e2e], [flops_step, float(launches_timed)], device=dev)

    if rank == 0:
        value = flops_all / (ms_step_mx * 1e-3) / 1e12
        breakdown = rates(w, ms_step, kern_ms, clocks, peaks)
        breakdown["repeats"] = {"ms_per_step": [round(r[0], 4) for r in repeats],
                                "sm_mhz": [r[2].get("sm_mhz") for r in repeats],
                                "power_w_max": [r[2].get("power_w_max") for r in repeats],
                                "power_capped": [("sw_power_cap" in (r[2].get("reasons") or [])) for r in repeats]}
        breakdown["timed_seconds_total"] = region_total_s
        if configs:
            breakdown["configs"] = configs
        peak_tf, peak_text = pick_peak(clocks, peaks)
        top, top_tf, top_ms = ((f"attn_bwd_kernel<{Dh}>", breakdown["bwd_main_tflops"], kern_ms["bwd_main"]) if w.trained
                               else (f"attn_fwd_kernel<{Dh}>", breakdown["fwd_tflops"], kern_ms["fwd"]))
        mhz = clocks.get("sm_mhz") or 0.0
        cyc_peak = mhz * 1e6 * SM_COUNT * DENSE_BF16_FLOPS_PER_CLK_PER_SM / 1e12 if mhz else None
        rec = recorded_traffic(top, _WORKLOAD_NAME)
        roofline = {"kernel": top, "bound": "tensor", "achieved": top_tf, "peak": peak_tf, "unit": "TFLOP/s",
                    "frac": top_tf / peak_tf, "peak_kind": f"{peak_kind}, {peak_text}",
                    "frac_of_measured_burst": top_tf / peaks["bf16_tflops"],
                    "frac_of_measured_sustained": top_tf / peaks["bf16_tflops_sustained"],
                    "frac_of_nominal_2250": top_tf / NOMINAL_BF16_TFLOPS,
                    "frac_of_cycle_peak": top_tf / cyc_peak if cyc_peak else None,
                    "kernel_ms": top_ms, "flops_per_launch": w.flops(False, True) if w.trained else w.flops(True, False),
                    "traffic": rec["dram_bytes_per_launch"] if rec else None,
                    "traffic_source": rec.get("source") if rec else None,
                    "target_50pct_of_bf16_peak_met": bool(value / world / peak_tf >= 0.5)}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
            "ms_per_step": ms_step_mx, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD_TEXT[_WORKLOAD_NAME] + "; one microbatch per GPU",
                       "tokens_rank0": T, "sum_n2_rank0": w.sum_n2, "heads": Hh, "head_dim": Dh,
                       "mode": "trained (fwd+bwd)" if w.trained else "frozen (fwd only)",
                       "l2": "inputs_exceed_l2" if T * Hh * Dh * 2 * 4 > 126e6 else "inputs_fit_l2 (no flush)",
                       "timing": f"{R} repeats of the {K}-step region (median reported; {region_total_s:.2f} s of steps in all)",
                       "step": "host plan + upload, attn fwd" + (", attn bwd (prepass, main, convert)" if w.trained else "")
                               + (", merge" if w.merge_hidden is not None else "")},
            "breakdown": breakdown,
            "roofline": roofline,
            "e2e": {"value": flops_all / (ms_e2e_mx * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": ms_e2e_mx,
                    "steps": Ke, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h)},
            "gpu_launches": int(launches),
            "clocks": clocks,
        }
        if merge_rot is not None:
            rec_m = recorded_traffic("merge_rows_kernel<true>", "mix75")
            line["roofline_merge"] = {"kernel": "merge_rows_kernel<true>", "workload": "modality mix 75% (805 MB per launch), "
                                      f"{merge_rot['buffer_sets']} rotating buffer sets", "bound": "hbm",
                                      "achieved": merge_rot["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                      "frac": merge_rot["gbs"] / peaks["hbm_gbs"], "peak_kind": f"{peak_kind}, copy bandwidth",
                                      "kernel_ms": merge_rot["ms"], "algorithmic_bytes": merge_rot["algorithmic_bytes"],
                                      "traffic": rec_m["dram_bytes_per_launch"] if rec_m else None}
        if world == 1 and not args.profile_mode and _WORKLOAD_NAME == "vit_l":
            line["cpu_baseline"] = cpu_baseline(w, full=args.cpu_baseline_full)
        if args.profile_mode:
            line["profile_mode"] = True
        print(json.dumps(line))
    D.shutdown()
    return 0


# ----------------------------------------------------------------------------- encoder-layer line (--workload *_layer)
LAYER_WORKLOADS = {"vit_l_layer": "vit_l", "qwen2vl_layer": "qwen2vl_frozen", "vit_l_layer_trained": "vit_l",
                   "qwen2vl_layer_trained": "qwen2vl"}


def layer_flops(w, ffn):
    """Algorithmic FLOPs of one layer forward: the four projections (2 * T * in * out each) + attention 4 * H * D * sum n^2."""
    hidden = w.n_heads * w.head_dim
    gemm = 2.0 * w.total_tokens * hidden * (3 * hidden + hidden + 2 * ffn)
    return gemm, gemm + w.flops(True, False)


def layer_arm(args):
    """The whole packed encoder layer forward (frozen mode: the layer a frozen encoder executes per microbatch) through
    mpipe_encoder_layer_fwd.  Same line format; `roofline` covers linear_fwd_kernel over the layer's four projections."""
    import torch
    from paper_2607_03229_b200 import binding as B
    from paper_2607_03229_b200 import dist as D

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    rank, local_rank, world = D.init("nccl")
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}: launch N>1 with torchrun, one rank per GPU")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    B.load()
    peaks, peak_kind = load_peaks()
    base = LAYER_WORKLOADS[_WORKLOAD_NAME]
    w = WORKLOADS[base](D.rank_seed(W.BASE_SEED + 2, rank))
    T, Hh, Dh = w.total_tokens, w.n_heads, w.head_dim
    hidden, ffn = Hh * Dh, 4 * Hh * Dh
    gen = torch.Generator(device=dev)
    gen.manual_seed(w.seed)

    def rnd(shape, std, mean=0.0):
        return (torch.randn(shape, device=dev, generator=gen) * std + mean).to(torch.bfloat16)

    params = {"ln1_gamma": rnd((hidden,), 0.1, 1.0), "ln1_beta": rnd((hidden,), 0.1), "w_qkv": rnd((3 * hidden, hidden), hidden ** -0.5),
              "b_qkv": rnd((3 * hidden,), 0.1), "w_o": rnd((hidden, hidden), hidden ** -0.5), "b_o": rnd((hidden,), 0.1),
              "ln2_gamma": rnd((hidden,), 0.1, 1.0), "ln2_beta": rnd((hidden,), 0.1), "w_fc1": rnd((ffn, hidden), hidden ** -0.5),
              "b_fc1": rnd((ffn,), 0.1), "w_fc2": rnd((hidden, ffn), ffn ** -0.5), "b_fc2": rnd((hidden,), 0.1)}
    weights = B.LayerWeights.from_tensors(**params)
    x = rnd((T, hidden), 1.0)
    y = torch.empty_like(x)
    trained = _WORKLOAD_NAME.endswith("_trained")
    plan = B.seg_plan(w.patch_counts, B.TRAINED if trained else B.FROZEN).to_device(dev)
    ws = torch.empty(B.encoder_layer_workspace_bytes(T, hidden, ffn), dtype=torch.uint8, device=dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    lse = torch.empty((Hh, T), dtype=torch.float32, device=dev) if trained else None
    if trained:
        dy, dx = rnd((T, hidden), 1.0), torch.empty_like(x)
        grads_t = {k_: torch.zeros(v_.shape, dtype=torch.float32, device=dev) for k_, v_ in params.items()}
        grads = B.LayerGrads.from_tensors(**grads_t)
        ws_b = torch.empty(B.encoder_layer_bwd_workspace_bytes(T, hidden, Hh, ffn), dtype=torch.uint8, device=dev)
    rope = None
    if base.startswith("qwen2vl"):   # the Qwen2-VL-like configuration carries a 2-D rotary encoding of q and k
        rope = tuple(torch.from_numpy(t).to(dev) for t in W.rope2d_tables(w.patch_counts, Dh))
    def step(xin=x, yout=y, st=None):
        B.encoder_layer_fwd(xin, yout, weights, Hh, ffn, plan, w.softmax_scale, 1e-6, ws, lse, status, st, rope)
        if trained:
            B.encoder_layer_bwd(dy, xin, dx, weights, grads, Hh, ffn, plan, w.softmax_scale, 1e-6, lse, ws, ws_b, status, st, rope)
    K, Wm = args.steps, max(args.warmup, 3)
    for _ in range(Wm):
        step()
    torch.cuda.synchronize()
    assert int(status[0]) == 0, f"device status {status.tolist()}"
    uuid = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid) if hasattr(
        torch.cuda.get_device_properties(dev), "uuid") else str(local_rank)
    sampler = ClockSampler(uuid)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    D.barrier()
    sampler.start()
    time.sleep(0.15)
    torch.cuda.synchronize()
    t_begin = time.perf_counter()
    e0.record()
    for _ in range(K):
        step()
    e1.record()
    torch.cuda.synchronize()
    t_end = time.perf_counter()
    D.barrier()
    clocks = sampler.stop(t_begin, t_end)
    ms_step = e0.elapsed_time(e1) / K

    # ---- per-kernel durations: the same launches, one at a time, each between its own pair of events
    norm = torch.empty_like(x); qkv = torch.empty((T, 3 * hidden), dtype=torch.bfloat16, device=dev)
    attn = torch.empty_like(x); x1 = torch.empty_like(x); fc1 = torch.empty((T, ffn), dtype=torch.bfloat16, device=dev)
    q3 = qkv.view(T, 3, Hh, Dh)
    stages = [
        ("layernorm", lambda: B.layernorm_fwd(x, params["ln1_gamma"], params["ln1_beta"], norm, 1e-6)),
        ("linear_qkv", lambda: B.linear_fwd(norm, params["w_qkv"], qkv, params["b_qkv"], None, False, status)),
        ("rope", (lambda: B.rope_apply(qkv, rope[0], rope[1], Hh, Dh)) if rope is not None else None),
        ("attn_fwd", lambda: B.varlen_attn_fwd(q3[:, 0], q3[:, 1], q3[:, 2], attn.view(T, Hh, Dh), lse, plan, w.softmax_scale, status)),
        ("linear_out", lambda: B.linear_fwd(attn, params["w_o"], x1, params["b_o"], x, False, status)),
        ("linear_fc1", lambda: B.linear_fwd(norm, params["w_fc1"], fc1, params["b_fc1"], None, True, status)),
        ("linear_fc2", lambda: B.linear_fwd(fc1, params["w_fc2"], y, params["b_fc2"], x1, False, status)),
    ]
    if trained:
        stages.append(("layer_bwd (all of mpipe_encoder_layer_bwd)", lambda: B.encoder_layer_bwd(
            dy, x, dx, weights, grads, Hh, ffn, plan, w.softmax_scale, 1e-6, lse, ws, ws_b, status, None, rope)))
    Kk = min(K, 20)
    kern_ms = {}
    step()   # leaves a consistent forward workspace for the backward stage
    for name, fn in stages:
        if fn is None:
            continue
        fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(Kk):
            fn()
        b.record()
        torch.cuda.synchronize()
        kern_ms[name] = a.elapsed_time(b) / Kk
    assert int(status[0]) == 0

    # ---- end to end: x from pinned host memory, y back to the host, every step
    Ke = 1 if args.profile_mode else min(K, 20)
    hx = torch.empty(tuple(x.shape), dtype=torch.bfloat16).pin_memory()
    hx.copy_(x)
    hy = torch.empty(tuple(y.shape), dtype=torch.bfloat16).pin_memory()
    hdy = torch.empty(tuple(y.shape), dtype=torch.bfloat16).pin_memory() if trained else None
    hdx = torch.empty(tuple(y.shape), dtype=torch.bfloat16).pin_memory() if trained else None
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    f0.record()
    for _ in range(Ke):
        x.copy_(hx, non_blocking=True)
        if trained:
            dy.copy_(hdy, non_blocking=True)
        step()
        hy.copy_(y, non_blocking=True)
        if trained:
            hdx.copy_(dx, non_blocking=True)
    f1.record()
    torch.cuda.synchronize()
    ms_e2e = f0.elapsed_time(f1) / Ke

    gemm_flops, flops_step = layer_flops(w, ffn)
    n_launch = 8 if rope is not None else 7
    if trained:   # algorithmic backward work: input and weight gradient of every projection (2x the forward's) + attention
        flops_step = 3.0 * gemm_flops + w.flops(True, True)    # backward (10 H D sum n^2); the recomputed fc1 is not counted
        n_launch += 22 if rope is not None else 21   # the backward's launches (fc1 stores GELU(u) and u in one launch)
    (ms_step_mx, ms_e2e_mx), (flops_all, launches) = D.reduce_max_sum(
        [ms_step, ms_e2e], [flops_step, float(n_launch * K)], device=dev)
    if rank == 0:
        value = flops_all / (ms_step_mx * 1e-3) / 1e12
        lin_ms = sum(v for k_, v in kern_ms.items() if k_.startswith("linear"))
        lin_tf = gemm_flops / (lin_ms * 1e-3) / 1e12
        peak_tf = peaks["bf16_tflops_sustained"]
        line = {
            "metric": "packed encoder layer " + ("forward + backward" if trained else "forward") +
                      " (norms, QKV/out/MLP projections, varlen attention) TFLOP/s (1 B200)",
            "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm, "ms_per_step": ms_step_mx,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": _WORKLOAD_NAME + ": one pre-norm encoder layer over the packed microbatch of " +
                       WORKLOAD_TEXT[base].split(":")[0] + f", hidden {hidden}, ffn {ffn}, " + ("trained (forward + backward)" if trained else "frozen (forward only)") +
                       "; one microbatch per GPU",
                       "tokens_rank0": T, "sum_n2_rank0": w.sum_n2, "heads": Hh, "head_dim": Dh,
                       "l2": "inputs_exceed_l2", "step": "mpipe_encoder_layer_fwd: LN, QKV" + (", 2-D rope" if rope is not None else "") +
                               ", attention, out-proj + residual, LN, fc1 + GELU, fc2 + residual" +
                               ("; mpipe_encoder_layer_bwd: input and weight gradients of the four projections, bias and norm "
                                "gradients, attention backward, two recomputed norms" if trained else "")},
            "breakdown": {"kernel_ms": kern_ms, "linear_tflops": lin_tf,
                          "attn_fwd_tflops": w.flops(True, False) / (kern_ms["attn_fwd"] * 1e-3) / 1e12,
                          "layernorm_gbs": 4.0 * T * hidden / (kern_ms["layernorm"] * 1e-3) / 1e9,
                          "frac_of_bf16_peak": {"measured_sustained": value / world / peak_tf, "measured_burst": value / world / peaks["bf16_tflops"],
                                                "nominal_2250": value / world / NOMINAL_BF16_TFLOPS}},
            "roofline": {"kernel": "linear_fwd_kernel (4 launches per step)", "bound": "tensor", "achieved": lin_tf, "peak": peak_tf,
                         "unit": "TFLOP/s", "frac": lin_tf / peak_tf, "peak_kind": f"{peak_kind}, sustained bf16 GEMM", "traffic": None},
            "e2e": {"value": flops_all / (ms_e2e_mx * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": ms_e2e_mx, "steps": Ke,
                    "h2d_bytes_per_step": int(hx.numel() * 2) * (2 if trained else 1),
                    "d2h_bytes_per_step": int(hy.numel() * 2) * (2 if trained else 1)},
            "gpu_launches": int(launches), "clocks": clocks,
        }
        if world == 1 and not args.profile_mode:
            line["cpu_baseline"] = layer_cpu_baseline(w, hidden, ffn, trained)
        if args.profile_mode:
            line["profile_mode"] = True
        print(json.dumps(line))
    D.shutdown()
    return 0


def layer_cpu_baseline(w, hidden, ffn, trained=False):
    """The layer oracle on the first segments of the workload (a few thousand tokens), one pass on the host cores."""
    import oracle
    from oracle import layer as OL
    m, tok = 0, 0
    while m < len(w.patch_counts) and (m == 0 or tok + w.patch_counts[m] <= 20000):
        tok += w.patch_counts[m]
        m += 1
    counts = w.patch_counts[:m]
    pb = W.layer_params_bf16(w.seed, hidden, ffn)
    ow = OL.LayerWeights(g1=OL.widen(pb["ln1_gamma"]), b1=OL.widen(pb["ln1_beta"]), wqkv=OL.widen(pb["w_qkv"]), bqkv=OL.widen(pb["b_qkv"]),
                         wo=OL.widen(pb["w_o"]), bo=OL.widen(pb["b_o"]), g2=OL.widen(pb["ln2_gamma"]), b2=OL.widen(pb["ln2_beta"]),
                         w1=OL.widen(pb["w_fc1"]), bb1=OL.widen(pb["b_fc1"]), w2=OL.widen(pb["w_fc2"]), bb2=OL.widen(pb["b_fc2"]))
    x = W.normal_bf16(w.seed, 0, (tok, hidden))
    cu = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    oracle.build()
    t0 = time.perf_counter()
    if trained:   # the oracle's backward runs its own forward first
        OL.encoder_layer_bwd(x, ow, cu, w.n_heads, w.softmax_scale, 1e-6, W.normal_bf16(w.seed, 1, (tok, hidden)))
    else:
        OL.encoder_layer_fwd(x, ow, cu, w.n_heads, w.softmax_scale, 1e-6)
    dt = time.perf_counter() - t0
    sq = float(sum(n * n for n in counts))
    flops = 2.0 * tok * hidden * (4 * hidden + 2 * ffn) * (3 if trained else 1) + (14.0 if trained else 4.0) * hidden * sq
    return {"value": flops / dt / 1e12, "unit": UNIT, "cores": oracle.n_threads(), "kind": "oracle", "seconds": dt,
            "sample": f"first {m} of {len(w.patch_counts)} segments ({tok} tokens, {flops:.3g} algorithmic FLOPs), one pass"}



def cpu_baseline(w, full=False):
    """The oracle as it stands on the host cores: a bounded sample (about 15 s of CPU work), or with `full` every
    (segment, head) pair of the workload (about a minute for the ViT-L configuration)."""
    import oracle
    rate = calibrate_oracle_rate(w)
    pairs, flops = oracle_sample(w, w.flops() * 2 if full else rate * 15.0)
    dt = run_oracle_sample(w, pairs, oracle_inputs(w, pairs))
    return {"value": flops / dt / 1e12, "unit": UNIT, "cores": oracle.n_threads(), "kind": "oracle", "seconds": dt,
            "sample": ("the whole workload: " if len(pairs) == sum(1 for n in w.patch_counts if n > 0) * w.n_heads else "") +
                      sample_text(w, pairs, flops) + ", one pass"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=("ours", "reference"), default="ours")
    ap.add_argument("--workload", choices=sorted(WORKLOADS) + sorted(LAYER_WORKLOADS), default="vit_l",
                    help="which synthetic configuration to run (default: vit_l, the one the metric is quoted on; "
                         "the others are for the per-config results table)")
    ap.add_argument("--min-seconds", type=float, default=2.0,
                    help="repeat the K-step timed region until the steps timed add up to about this many seconds")
    ap.add_argument("--no-configs", action="store_true", help="skip the per-configuration block of the default run")
    ap.add_argument("--cpu-baseline-full", action="store_true",
                    help="time the oracle on the WHOLE workload (about a minute of CPU) instead of the bounded sample")
    ap.add_argument("--profile-mode", action="store_true",
                    help="skip the end-to-end and CPU-baseline legs (for short runs under a profiler; the line "
                         "such a run prints is not a benchmark value)")
    args = ap.parse_args()
    global _WORKLOAD_NAME
    _WORKLOAD_NAME = args.workload
    if args.workload in LAYER_WORKLOADS:
        if args.impl == "reference":
            print(json.dumps({"impl": "reference", "unavailable": "the reference arm covers the attention metric only (default workload)"}))
            return 0
        return layer_arm(args)
    if args.impl == "reference":
        return reference_arm(args)
    return ours_arm(args)


if __name__ == "__main__":
    sys.exit(main())
