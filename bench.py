#!/usr/bin/env python
"""Benchmark of the prepacked-prefill hot path on B200.

One "step" = one pass of the whole path over one synthetic batch already resident in HBM:
pp_pack (host) -> pp_prefill_attention (table build + upload, restart RoPE kernel, packed
attention kernel) -> pp_unpack_kv. The headline value is useful (non-padding) prompt tokens per
second. Prints ONE JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

With --gpus N > 1 (under torchrun) every rank runs its own copy of the batch (the path has no
exchange step: weak scaling, no collective on the data path).
--impl reference times the float64 CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "useful_prefill_tokens_per_s"
UNIT = "tokens/s"
DEFAULT_WORKLOAD = "llama2_7b"

# DRAM traffic of one attention-kernel launch (dram__bytes_read.sum + dram__bytes_write.sum) from
# the ncu captures summarised in profiles/attention_<workload>.md (fused-route launches; long_mix: a
# launch of the three-call route, which reads and writes the same tensors); None where no capture
# exists for the workload.
NCU_ATTENTION_TRAFFIC_BYTES = {"llama2_7b": 562.4e6, "many_short": 424.2e6, "long_mix": 3.82e9}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML (read-only) while a timed
    region runs."""

    def __init__(self, cuda_index: int, period_s: float = 0.002):
        self.period = period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            import torch
            props = torch.cuda.get_device_properties(cuda_index)
            try:        # NVML and CUDA may number the GPUs differently: match by UUID
                self.h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(props.uuid)).encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(cuda_index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _names(self, mask: int):
        nv = self.nv
        table = [("sw_power_cap", "nvmlClocksEventReasonSwPowerCap", "nvmlClocksThrottleReasonSwPowerCap"),
                 ("hw_slowdown", "nvmlClocksEventReasonHwSlowdown", "nvmlClocksThrottleReasonHwSlowdown"),
                 ("hw_thermal_slowdown", "nvmlClocksEventReasonHwThermalSlowdown", "nvmlClocksThrottleReasonHwThermalSlowdown"),
                 ("sw_thermal_slowdown", "nvmlClocksEventReasonSwThermalSlowdown", "nvmlClocksThrottleReasonSwThermalSlowdown"),
                 ("hw_power_brake", "nvmlClocksEventReasonHwPowerBrakeSlowdown", "nvmlClocksThrottleReasonHwPowerBrakeSlowdown")]
        out = []
        for name, a, b in table:
            bit = getattr(nv, a, None)
            if bit is None:
                bit = getattr(nv, b, None)
            if bit is not None and (mask & int(bit)):
                out.append(name)
        return out

    def _loop(self):
        nv = self.nv
        get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
            getattr(nv, "nvmlDeviceGetCurrentClocksThrottleReasons")
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                self.reasons.update(self._names(int(get_reasons(self.h))))
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread is not None:
            self._stop.set()
            self._thread.join()
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def workload_counts(cfg, lengths):
    l = lengths.astype(np.int64)
    total = int(l.sum())
    pairs = int((l * (l + 1) // 2).sum())
    d, hq, hkv = cfg.head_dim, cfg.n_q_heads, cfg.n_kv_heads
    return dict(
        total_tokens=total,
        useful_flops=4 * hq * d * pairs,                       # QK^T and PV, 2*D flops each per visible pair
        attn_bytes=2 * total * d * (2 * hq + 2 * hkv),         # read Q', K', V once, write O once
        rope_bytes=4 * total * d * (hq + hkv),                 # read + write Q and K
        unpack_bytes=8 * total * d * hkv)                      # read K', V; write both caches


def max_over_ranks(ms: float, dist=None, device="cpu") -> float:
    """Slowest rank's time: the timed region of a multi-rank run ends when the last rank does."""
    if dist is None:
        return float(ms)
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(world: int, tokens_per_rank: int, ms_per_step: float) -> float:
    """Replicas only: every rank prefills its own copy of the batch, no data-path collective."""
    return world * tokens_per_rank / (ms_per_step * 1e-3)


_FLUSH = None      # set by main() for workloads smaller than the L2: a buffer to overwrite before every timed call


def time_loop(fn, iters, warmup=3):
    import torch
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    if _FLUSH is not None:
        # small workload: every call is timed on its own, after the L2 has been overwritten; the flush
        # kernel also gives the host the time to queue the call, so the events bracket device time
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
        for a, b in evs:
            _FLUSH.fill_(1)
            a.record()
            fn()
            b.record()
        torch.cuda.synchronize()
        return sum(a.elapsed_time(b) for a, b in evs) / iters
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # A few milliseconds of device-side delay in front of the first event let the host queue all the
    # calls before the first one starts, so the events bracket launches that run back to back: the
    # average is the kernel's duration (with its in-stream table upload), not the host's enqueue rate.
    if hasattr(torch.cuda, "_sleep"):
        torch.cuda._sleep(10_000_000)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters          # ms per call


_QKV_CACHE = {}


def oracle_sample(cfg, lengths, budget_s, max_prompts=None):
    """Time the oracle, as it stands, on the first prompts of the workload (original order) until
    `budget_s` of CPU time is spent or all prompts are done. Returns (tokens, seconds, n_prompts)."""
    import torch

    from oracle import prepack_oracle as orc
    from workloads import make_qkv
    n = len(lengths) if max_prompts is None else min(max_prompts, len(lengths))
    tok_needed = int(lengths[:n].sum())
    if _QKV_CACHE.get("key") != (cfg.name, tok_needed):      # inputs are drawn once, outside the timing
        _QKV_CACHE.update(key=(cfg.name, tok_needed), qkv=make_qkv(cfg, tok_needed))
    q, k, v = _QKV_CACHE["qkv"]
    f64 = lambda t: t.to(torch.float32).numpy().astype(np.float64)
    tokens, done, off = 0, 0, 0
    t0 = time.perf_counter()
    for i in range(n):
        l = int(lengths[i])
        orc.prefill_prompt(f64(q[off:off + l]), f64(k[off:off + l]), f64(v[off:off + l]), cfg.rope_base)
        off += l
        tokens += l
        done += 1
        if time.perf_counter() - t0 > budget_s:
            break
    return tokens, time.perf_counter() - t0, done


def workload_config(cfg, name, lengths, n_bins, capacity, world):
    """The `config` object of the JSON line; both arms (--impl ours / reference) print the same one."""
    d, hq, hkv = cfg.head_dim, cfg.n_q_heads, cfg.n_kv_heads
    T = int(lengths.sum())
    rows = int(n_bins) * int(capacity)
    # one step touches q, k (read and written back), v, o and both cache pools
    stream_mb = (rows * d * 2 * (2 * hq + 3 * hkv) + T * d * 2 * 2 * hkv) / 1e6
    l2 = (f"no flush: each step streams {stream_mb:.0f} MB of tensors, larger than the 126 MB L2"
          if stream_mb > 2 * 126 else
          f"flushed: each step touches only {stream_mb:.1f} MB, so a 1 GB buffer is overwritten before every "
          "timed step and the steps are timed one by one")
    return {"workload": name, "description": cfg.description, "n_prompts": int(len(lengths)),
            "total_tokens": T, "n_bins": int(n_bins), "capacity": int(capacity),
            "n_q_heads": hq, "n_kv_heads": hkv, "head_dim": d, "rope_base": cfg.rope_base, "path": "fused",
            "parallelism": f"replicas x{world}" if world > 1 else "single GPU", "l2": l2}, stream_mb


def run_reference(args):
    """--impl reference: the float64 CPU oracle on the host cores. Every step is the whole workload
    where `--steps + --warmup` such passes fit in about five minutes, otherwise a bounded sample of it
    (the first prompts in original order), named in cpu_baseline.sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import prepack_oracle as orc
    from workloads import CONFIGS, prompt_lengths
    cfg = CONFIGS[args.workload]
    lengths = prompt_lengths(args.workload)
    cores = len(os.sched_getaffinity(0))
    total_steps = args.steps + args.warmup
    # calibrate on a short sample: the oracle's cost per prompt grows with l^2 (attention) and l (the rest)
    tok, sec, n_cal = oracle_sample(cfg, lengths, 2.0)
    l = lengths.astype(np.float64)
    work = l * l + 256.0 * l
    est_whole = sec * work.sum() / work[:n_cal].sum()
    if est_whole * total_steps <= 300.0:
        n_prompts = len(lengths)
    else:
        per_step_budget = max(0.5, 120.0 / max(total_steps, 1))
        cum = np.cumsum(work) * (sec / work[:n_cal].sum())
        n_prompts = max(1, int(np.searchsorted(cum, per_step_budget, side="right")))
    for _ in range(args.warmup):
        oracle_sample(cfg, lengths, 1e9, n_prompts)
    t_tot, tok_tot = 0.0, 0
    for _ in range(args.steps):
        tok, sec, _ = oracle_sample(cfg, lengths, 1e9, n_prompts)
        t_tot += sec
        tok_tot += tok
    value = tok_tot / t_tot
    whole = n_prompts == len(lengths)
    sample = (f"the whole workload per step ({tok} tokens, {len(lengths)} prompts), all heads, numpy float64" if whole else
              f"first {n_prompts} of {len(lengths)} prompts ({tok} tokens) per step, all heads, numpy float64")
    pk = orc.ffd_pack([int(x) for x in lengths])
    config, _ = workload_config(cfg, args.workload, lengths, pk["n_bins"], pk["capacity"], 1)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_tot / max(args.steps, 1),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-padded", action="store_true", help="skip the padded-batch comparison run")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--kernel-iters", type=int, default=50)
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import torch

    import paper_2404_09529_b200 as pp
    from paper_2404_09529_b200.runner import PrefillBatch
    from workloads import CONFIGS, make_qkv, prompt_lengths

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the prepack-b200 path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    peaks = load_peaks()
    cfg = CONFIGS[args.workload]
    lengths = prompt_lengths(args.workload)
    counts = workload_counts(cfg, lengths)
    T = counts["total_tokens"]
    q_tok, k_tok, v_tok = make_qkv(cfg, T, device="cuda")

    batch = PrefillBatch(lengths, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.rope_base, mode="packed")
    batch.load(q_tok, k_tok, v_tok)
    # The whole path has two public routes through the C ABI: three calls (pp_pack +
    # pp_prefill_attention + pp_unpack_kv) or two (pp_pack + pp_prefill_fused). Both are timed over the
    # same K steps; the headline is the fused route (config.path), the other is reported beside it.
    routes = {"three_call": lambda: batch.run(repack=True), "fused": lambda: batch.run_fused(repack=True)}
    config, stream_mb = workload_config(cfg, args.workload, lengths, batch.pack.n_bins, batch.pack.capacity, world)
    # A step that touches less than about twice the L2 would find its inputs there on the next step:
    # such workloads are timed step by step, with a 1 GB buffer overwritten before each.
    # (1 GB rather than just more than the L2: the overwrite must also outlast the host's enqueueing
    # of the step behind it, or the events would bracket host time)
    flush = torch.empty(1 << 30, dtype=torch.uint8, device="cuda") if stream_mb <= 2 * 126 else None
    global _FLUSH
    _FLUSH = flush

    def timed_region(step):
        batch.load(q_tok, k_tok, v_tok)          # raw Q/K again (the three-call route rotates q in place)
        for _ in range(max(args.warmup, 3)):
            step()
        barrier()
        sampler = ClockSampler(torch.cuda.current_device())
        sampler.start()
        barrier()
        if flush is None:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(args.steps):
                step()
            e1.record()
            barrier()
            ms = e0.elapsed_time(e1)
        else:
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
            for a, b in evs:
                flush.fill_(1)
                a.record()
                step()
                b.record()
            barrier()
            ms = sum(a.elapsed_time(b) for a, b in evs)
        clk = sampler.stop()
        if batch.device_status() != 0:
            raise SystemExit("device-side wait gave up during the timed region")
        return max_over_ranks(ms, dist, "cuda") / args.steps, clk

    route_ms, route_clocks = {}, {}
    for name, fn in routes.items():
        route_ms[name], route_clocks[name] = timed_region(fn)
    path = "fused"
    ms_per_step, clocks = route_ms[path], route_clocks[path]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    value = whole_job_tokens_per_s(world, T, ms_per_step)
    batch.load(q_tok, k_tok, v_tok)

    # ---------------------------------------------------------------- host share of a step (rank-local)
    import time as _time
    t0 = _time.perf_counter()
    for _ in range(50):
        pp.pp_pack(lengths, 0)
    pack_us = (_time.perf_counter() - t0) / 50 * 1e6
    enqueue_us = 0.0
    for _ in range(20):
        torch.cuda.synchronize()                 # idle device: the call returns as soon as it has enqueued
        t0 = _time.perf_counter()
        routes[path]()
        enqueue_us += (_time.perf_counter() - t0) / 20 * 1e6     # pack + table build + copies + launches
    torch.cuda.synchronize()
    host = {"pp_pack_us": pack_us, "enqueue_us_per_step": enqueue_us,
            "note": "host time to pack and enqueue one step; it overlaps the previous step's kernels"}
    batch.load(q_tok, k_tok, v_tok)

    # ---------------------------------------------------------------- per-kernel times (rank-local)
    n_it = args.kernel_iters
    ms_rope = time_loop(lambda: batch.run(flags=pp.PP_FLAG_ROPE_ONLY, unpack=False), n_it)
    ms_attn = time_loop(lambda: batch.run(flags=pp.PP_FLAG_SKIP_ROPE, unpack=False), n_it)
    ms_unpack = time_loop(batch.run_unpack_only, n_it)
    ms_rope_unpack = time_loop(lambda: batch.run_fused(flags=pp.PP_FLAG_ROPE_ONLY), n_it)
    ms_attn_fused = time_loop(lambda: batch.run_fused(flags=pp.PP_FLAG_SKIP_ROPE), n_it)
    fused_k_bytes = 2 * T * cfg.head_dim * cfg.n_kv_heads * 5     # K read, K' and K cache written, V read, V cache written
    kernels = {
        "rope_unpack_fused": {"ms": ms_rope_unpack, "gbs": fused_k_bytes / ms_rope_unpack * 1e-6,
                              "frac_hbm": fused_k_bytes / ms_rope_unpack * 1e-6 / peaks["hbm_gbs"]},
        "attention_fused": {"ms": ms_attn_fused, "tflops": counts["useful_flops"] / ms_attn_fused * 1e-9,
                            "frac_bf16_peak": counts["useful_flops"] / ms_attn_fused * 1e-9 / peaks["bf16_tflops"],
                            "frac_bf16_datasheet": counts["useful_flops"] / ms_attn_fused * 1e-9 / 2250.0,
                            "gbs": counts["attn_bytes"] / ms_attn_fused * 1e-6,
                            "frac_hbm": counts["attn_bytes"] / ms_attn_fused * 1e-6 / peaks["hbm_gbs"]},
        "rope": {"ms": ms_rope, "gbs": counts["rope_bytes"] / ms_rope * 1e-6,
                 "frac_hbm": counts["rope_bytes"] / ms_rope * 1e-6 / peaks["hbm_gbs"]},
        "attention": {"ms": ms_attn, "tflops": counts["useful_flops"] / ms_attn * 1e-9,
                      "frac_bf16_peak": counts["useful_flops"] / ms_attn * 1e-9 / peaks["bf16_tflops"],
                      "frac_bf16_datasheet": counts["useful_flops"] / ms_attn * 1e-9 / 2250.0,
                      "gbs": counts["attn_bytes"] / ms_attn * 1e-6,
                      "frac_hbm": counts["attn_bytes"] / ms_attn * 1e-6 / peaks["hbm_gbs"]},
        "unpack": {"ms": ms_unpack, "gbs": counts["unpack_bytes"] / ms_unpack * 1e-6,
                   "frac_hbm": counts["unpack_bytes"] / ms_unpack * 1e-6 / peaks["hbm_gbs"]},
    }
    # the attention kernel dominates; which roofline binds it depends on the workload's FLOP/byte
    intensity = counts["useful_flops"] / counts["attn_bytes"]
    ridge = peaks["bf16_tflops"] * 1e3 / peaks["hbm_gbs"]
    traffic = NCU_ATTENTION_TRAFFIC_BYTES.get(args.workload)
    # the attention kernel as launched in the headline route
    dom = kernels["attention_fused"] if path == "fused" else kernels["attention"]
    if intensity < ridge:
        roofline = {"kernel": "attention", "bound": "hbm", "achieved": dom["gbs"],
                    "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": dom["frac_hbm"],
                    "traffic": traffic, "peak_source": peaks["source"] + " (burst copy)",
                    "flop_per_byte": intensity, "ridge_flop_per_byte": ridge}
    else:
        # the burst peak is the stricter denominator; the loop that times the kernel runs long enough
        # to sit at the power cap like the sustained cuBLAS measurement, so that fraction is given too
        roofline = {"kernel": "attention", "bound": "tensor", "achieved": dom["tflops"],
                    "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": dom["frac_bf16_peak"],
                    "traffic": traffic, "peak_source": peaks["source"] + " (burst, kernel timed alone)",
                    "peak_sustained": peaks["bf16_tflops_sustained"],
                    "frac_of_sustained_peak": dom["tflops"] / peaks["bf16_tflops_sustained"],
                    "flop_per_byte": intensity, "ridge_flop_per_byte": ridge}

    # ---------------------------------------------------------------- padded-batch mode of the same kernels
    padded = None
    if not args.no_padded and rank == 0:
        pb = PrefillBatch(lengths, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.rope_base, mode="padded")
        pb.load(q_tok, k_tok, v_tok)
        n_pad = max(3, min(args.steps, 30))
        # the packed path timed the same way as the padded one (device time of queued steps), so
        # that the ratios compare like with like even where a step is shorter than its enqueue time
        if path == "fused":
            ms_packed_dev = time_loop(lambda: batch.run_fused(repack=True), n_pad)
            ms_packed_dev_norepack = time_loop(lambda: batch.run_fused(), n_pad)
        else:
            ms_packed_dev = time_loop(lambda: batch.run(repack=True), n_pad)
            ms_packed_dev_norepack = time_loop(lambda: batch.run(), n_pad)
        if path == "fused":
            ms_pad = time_loop(lambda: pb.run_fused(repack=True), n_pad)
            ms_pad_attn = time_loop(lambda: pb.run_fused(flags=pp.PP_FLAG_SKIP_ROPE), max(3, n_pad // 2))
        else:
            ms_pad = time_loop(lambda: pb.run(repack=True), n_pad)
            ms_pad_attn = time_loop(lambda: pb.run(flags=pp.PP_FLAG_SKIP_ROPE, unpack=False), max(3, n_pad // 2))
        padded = {"tokens_per_s": T / (ms_pad * 1e-3), "ms_per_step": ms_pad, "attention_ms": ms_pad_attn,
                  "rows_computed": int(pb.pack.n_bins) * int(pb.pack.capacity),
                  "packed_ms_per_step_same_timing": ms_packed_dev,
                  "speedup_packed_vs_padded": ms_pad / ms_packed_dev,
                  "attention_speedup_packed_vs_padded": ms_pad_attn / dom["ms"]}
        del pb
        torch.cuda.empty_cache()
        # one prompt per bin with its true length: masking and tile skipping without the packing
        vb = PrefillBatch(lengths, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.rope_base, mode="varlen")
        vb.load(q_tok, k_tok, v_tok)
        if path == "fused":
            ms_var = time_loop(lambda: vb.run_fused(), n_pad)
        else:
            ms_var = time_loop(lambda: vb.run(), n_pad)
        padded["unpacked_varlen"] = {"tokens_per_s": T / (ms_var * 1e-3), "ms_per_step": ms_var,
                                     "rows_allocated": int(vb.pack.n_bins) * int(vb.pack.capacity),
                                     "speedup_packed_vs_unpacked_varlen": ms_var / ms_packed_dev_norepack}
        del vb
        torch.cuda.empty_cache()

    # ---------------------------------------------------------------- end to end from host buffers
    params = pp.AttnParams(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.rope_base, 0.0, 0, 0, 0)
    arena_bytes = pp.pp_prefill_host_arena_bytes(params, lengths)
    arena = torch.empty(arena_bytes, dtype=torch.uint8, device="cuda")
    hq, hk, hv = (t.cpu().pin_memory() for t in (q_tok, k_tok, v_tok))
    ho = torch.empty_like(hq).pin_memory()
    hkc = torch.empty(hk.numel(), dtype=torch.bfloat16).pin_memory()
    hvc = torch.empty(hv.numel(), dtype=torch.bfloat16).pin_memory()
    stream = torch.cuda.current_stream().cuda_stream
    e2e_step = lambda: pp.pp_prefill_host(params, lengths, hq, hk, hv, ho, hkc, hvc, arena, arena_bytes, stream)
    e2e_steps = max(3, min(args.steps, 20))
    for _ in range(3):
        e2e_step()
    barrier()
    e0.record()
    for _ in range(e2e_steps):
        e2e_step()
    e1.record()
    barrier()
    ms_e2e = e0.elapsed_time(e1)
    ms_e2e = max_over_ranks(ms_e2e, dist, "cuda")
    h2d = (hq.numel() + hk.numel() + hv.numel()) * 2
    d2h = (ho.numel() + hkc.numel() + hvc.numel()) * 2
    e2e = {"value": whole_job_tokens_per_s(world, T, ms_e2e / e2e_steps), "unit": UNIT, "h2d_bytes_per_step": h2d,
           "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": ms_e2e / e2e_steps,
           "api": "pp_prefill_host (pinned host buffers, contiguous copies, groups of prompts pipelined over streams)"}

    # ---------------------------------------------------------------- CPU baseline: the oracle as it stands
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        tok, sec, n_done = oracle_sample(cfg, lengths, 15.0)
        cpu_baseline = {"value": tok / sec, "unit": UNIT, "cores": len(os.sched_getaffinity(0)), "kind": "oracle",
                        "sample": f"first {n_done} of {len(lengths)} prompts in original order ({tok} tokens), "
                                  f"all heads, numpy float64, {sec:.1f} s"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": config,
            "clocks": clocks, "e2e": e2e, "gpu_launches": 2 * args.steps, "roofline": roofline,
            "launches_note": "fused route: rope_unpack_kernel + attention_kernel per step; the cos/sin table "
                             "kernel runs once (first warm-up step) and is kept while the bin capacity stays the same",
            "cpu_baseline": cpu_baseline, "host": host, "kernels": kernels, "padded": padded,
            "routes": {"three_call": {"tokens_per_s": whole_job_tokens_per_s(world, T, route_ms["three_call"]),
                                      "ms_per_step": route_ms["three_call"],
                                      "api": "pp_pack + pp_prefill_attention + pp_unpack_kv"},
                       "fused": {"tokens_per_s": whole_job_tokens_per_s(world, T, route_ms["fused"]),
                                 "ms_per_step": route_ms["fused"], "api": "pp_pack + pp_prefill_fused"}},
            "attention": {"useful_tflops": dom["tflops"],
                          "frac_bf16_peak_measured": dom["frac_bf16_peak"],
                          "frac_bf16_peak_datasheet": dom["frac_bf16_datasheet"]},
            "peaks": peaks,
        }
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
