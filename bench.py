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
# dram__bytes_read.sum + dram__bytes_write.sum of one attn_bwd_kernel<64> launch on this workload, from the
# ncu capture summarised in profiles/attn_bwd_kernel_vit_l.md.
BWD_MAIN_DRAM_BYTES_PER_LAUNCH = 1.0274e9


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
    """A bounded sample of the workload for the CPU oracle: the first m segments and first h heads whose
    algorithmic fwd+bwd FLOPs (14 * h * D * sum n^2) stay near `target_flops`."""
    counts = w.patch_counts
    per_head = [14.0 * w.head_dim * n * n for n in counts]
    h = w.n_heads
    while h > 1 and per_head[0] * h > target_flops:
        h //= 2
    m, acc = 0, 0.0
    while m < len(counts) and (m == 0 or acc + per_head[m] * h <= target_flops):
        acc += per_head[m] * h
        m += 1
    return m, h, acc


def run_oracle_sample(w, m: int, h: int, inputs=None):
    """One oracle pass (plan, fwd, bwd, merge of the sampled rows) over the sample.  Returns seconds."""
    import oracle
    counts = w.patch_counts[:m]
    T = int(sum(counts))
    if inputs is None:
        shape = (T, h, w.head_dim)
        inputs = tuple(W.normal_bf16(w.seed, 10 + i, shape) for i in range(4))
        pos = (w.positions[:T] - w.positions[0]).astype(np.int32)   # the sampled images' runs and the gaps between them
        emb = W.normal_bf16(w.seed, 21, (int(pos.max()) + 1, w.merge_hidden))
        src = W.normal_bf16(w.seed, 20, (T, w.merge_hidden))
        inputs = inputs + (emb, src, pos)
    q, k, v, do, emb, src, pos = inputs
    t0 = time.perf_counter()
    cu = oracle.seg_plan(counts, 256, 128, True)[0]
    oracle.attn_fwd(q, k, v, cu, w.softmax_scale)
    oracle.attn_bwd(do, q, k, v, cu, w.softmax_scale)
    oracle.merge_tokens(src, emb, pos)
    return time.perf_counter() - t0, inputs


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
    """The oracle, as it stands, on the host cores; bounded sample sized from --steps/--warmup."""
    from paper_2607_03229_b200 import dist as D
    rank, _, world = D.env_world()
    if rank != 0:
        return 0
    import oracle
    w = workload_for(0)
    rate = calibrate_oracle_rate(w)
    budget_s = 150.0 / max(1, args.steps + args.warmup)
    m, h, flops = oracle_sample(w, min(rate * min(budget_s, 20.0), w.flops()))
    inputs = None
    for _ in range(args.warmup):
        _, inputs = run_oracle_sample(w, m, h, inputs)
    times = []
    for _ in range(args.steps):
        dt, inputs = run_oracle_sample(w, m, h, inputs)
        times.append(dt)
    ms = 1e3 * float(np.mean(times))
    value = flops / (ms * 1e-3) / 1e12
    sample = (f"first {m} of {len(w.patch_counts)} segments x first {h} of {w.n_heads} heads "
              f"({int(sum(w.patch_counts[:m]))} tokens, {flops:.3g} algorithmic FLOPs per step)")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": "vit_l: 32 images of 16..64 x 16..64 patches, 16 heads x 64, trained, + merge",
                   "sample": sample},
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

    w = workload_for(rank)
    T, Hh, Dh = w.total_tokens, w.n_heads, w.head_dim
    buf = H.allocate(w, dev)
    n_kernels = H.kernels_per_step(w)
    K, Wm = args.steps, max(args.warmup, 3)

    for _ in range(Wm):
        H.run_step(w, buf)
    torch.cuda.synchronize()
    assert int(buf.status[0]) == 0, f"device status {buf.status.tolist()}"

    # ---- timed region: K whole steps, inputs resident in HBM, per-kernel events recorded alongside
    kernels = ["fwd"] + (["bwd_main"] if w.trained else []) + (["merge"] if w.merge_hidden is not None else [])
    ev = {name: [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
          for name in kernels}
    slots = {"fwd": B.PROFILE_FWD, "bwd_main": B.PROFILE_BWD_MAIN, "merge": B.PROFILE_MERGE}
    uuid = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid) if hasattr(
        torch.cuda.get_device_properties(dev), "uuid") else str(local_rank)
    sampler = ClockSampler(uuid)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for name in ev:                      # create the event handles before the region
        for a, b in ev[name]:
            a.record(), b.record()
    torch.cuda.synchronize()
    D.barrier()
    sampler.start()
    time.sleep(0.15)
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
    D.barrier()
    clocks = sampler.stop(t_begin, t_end)
    assert int(buf.status[0]) == 0, f"device status {buf.status.tolist()}"
    ms_step = e0.elapsed_time(e1) / K
    kern_ms = {name: float(np.mean([a.elapsed_time(b) for a, b in ev[name]])) for name in ev}

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
    t0 = time.perf_counter()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record(s_in)
    e2e_steps(Ke)
    s_out.synchronize()
    f1.record(s_out)
    torch.cuda.synchronize()
    D.barrier()
    ms_e2e = max(f0.elapsed_time(f1), 0.0) / Ke
    assert all(int(b_.status[0]) == 0 for b_ in bufs)

    # ---- reduce over ranks: max of times, sum of work
    flops_step = w.flops(True, w.trained)
    merge_bytes = float(T) * (4 * w.merge_hidden + 4) if w.merge_hidden is not None else 0.0
    (ms_step_mx, ms_e2e_mx), (flops_all, launches) = D.reduce_max_sum(
        [ms_step, ms_e2e], [flops_step, float(n_kernels * K)], device=dev)

    if rank == 0:
        value = flops_all / (ms_step_mx * 1e-3) / 1e12
        fwd_tf = w.flops(True, False) / (kern_ms["fwd"] * 1e-3) / 1e12       # this rank's kernels, per launch
        breakdown = {"fwd_ms": kern_ms["fwd"], "fwd_tflops": fwd_tf}
        if w.trained:
            bwd_tf = w.flops(False, True) / (kern_ms["bwd_main"] * 1e-3) / 1e12
            breakdown.update({"bwd_main_ms": kern_ms["bwd_main"], "bwd_main_tflops": bwd_tf})
        if w.merge_hidden is not None and T > 0:
            merge_gbs = merge_bytes / (kern_ms["merge"] * 1e-3) / 1e9
            breakdown.update({"merge_ms": kern_ms["merge"], "merge_gbs": merge_gbs,
                              "merge_frac_of_hbm_peak": merge_gbs / peaks["hbm_gbs"]})
        breakdown["attn_frac_of_bf16_peak"] = {"measured_sustained": value / world / peaks["bf16_tflops_sustained"],
                                               "measured_burst": value / world / peaks["bf16_tflops"],
                                               "nominal_2250": value / world / NOMINAL_BF16_TFLOPS}
        peak_tf = peaks["bf16_tflops_sustained"]
        top, top_tf = (f"attn_bwd_kernel<{Dh}>", bwd_tf) if w.trained else (f"attn_fwd_kernel<{Dh}>", fwd_tf)
        traffic = BWD_MAIN_DRAM_BYTES_PER_LAUNCH if (_WORKLOAD_NAME == "vit_l" and w.trained) else None
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
            "ms_per_step": ms_step_mx, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD_TEXT[_WORKLOAD_NAME] + "; one microbatch per GPU",
                       "tokens_rank0": T, "sum_n2_rank0": w.sum_n2, "heads": Hh, "head_dim": Dh,
                       "mode": "trained (fwd+bwd)" if w.trained else "frozen (fwd only)",
                       "l2": "inputs_exceed_l2" if T * Hh * Dh * 2 * 4 > 126e6 else "inputs_fit_l2 (no flush)",
                       "step": "host plan + upload, attn fwd" + (", attn bwd (prepass, main, convert)" if w.trained else "")
                               + (", merge" if w.merge_hidden is not None else "")},
            "breakdown": breakdown,
            "roofline": {"kernel": top, "bound": "tensor", "achieved": top_tf, "peak": peak_tf, "unit": "TFLOP/s",
                         "frac": top_tf / peak_tf, "peak_kind": f"{peak_kind}, sustained bf16 GEMM", "traffic": traffic},
            "e2e": {"value": flops_all / (ms_e2e_mx * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": ms_e2e_mx,
                    "steps": Ke, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h)},
            "gpu_launches": int(launches),
            "clocks": clocks,
        }
        if world == 1 and not args.profile_mode and _WORKLOAD_NAME == "vit_l":
            line["cpu_baseline"] = cpu_baseline(w)
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
        n_launch += 23 if rope is not None else 22   # + the activation kernel of a trained forward, - the projection no longer recomputed
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



def cpu_baseline(w):
    """The oracle as it stands on the host cores, on a bounded sample (about 10-20 s of CPU work)."""
    import oracle
    rate = calibrate_oracle_rate(w)
    m, h, flops = oracle_sample(w, rate * 12.0)
    dt, _ = run_oracle_sample(w, m, h)
    return {"value": flops / dt / 1e12, "unit": UNIT, "cores": oracle.n_threads(), "kind": "oracle", "seconds": dt,
            "sample": f"first {m} of {len(w.patch_counts)} segments x first {h} of {w.n_heads} heads "
                      f"({int(sum(w.patch_counts[:m]))} tokens, {flops:.3g} algorithmic fwd+bwd FLOPs), one pass"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=("ours", "reference"), default="ours")
    ap.add_argument("--workload", choices=sorted(WORKLOADS) + sorted(LAYER_WORKLOADS), default="vit_l",
                    help="which synthetic configuration to run (default: vit_l, the one the metric is quoted on; "
                         "the others are for the per-config results table)")
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
