"""Measurement sweeps over the prefill and decode paths, on synthetic batches (Sections 5.2, 6 and 7 of the paper).

``predictor``: batches of k prompts with lengths uniform in [1, 512]; for every batch the packed
and the padded (full-batching) path are timed and the speedup is regressed on the two batch
statistics the paper uses: the bin reduction r / k and the padding per prompt m - L / k
(m = longest prompt, L = total tokens, r = bins after packing). Attention layer only.

``dataset``: a stream of prompts is prefilled (a) bin-packed as a whole, once, and processed in
launches of a fixed number of bins of that one packing, (b) in batches of consecutive prompts after sorting the stream by
length, each padded to its own maximum, (c) in batches in arrival order, padded. Reports useful
tokens per second of each schedule.

``generation``: decode steps over the per-prompt caches (Section 7: a batch of nine prompts of one
token and one of 1000 tokens, 20 generated tokens), against the same steps with every prompt
declared as long as the longest (what padded caches cost).

``shapes``: batches of 16 prompts whose lengths follow lognormal distributions fitted to the
minimum / mean / maximum prompt length the paper reports for each of its six evaluation sets
(appendix table of dataset length statistics; lengths only, no text), on the attention-layer shapes
of the 1.3 B and 7 B models of its model table: packed against padded path, per length profile.

Each prints one JSON object. They only marshal arguments: all arithmetic runs in the library.

    python -m paper_2404_09529_b200.sweep predictor [--batches 40] [--k 16]
    python -m paper_2404_09529_b200.sweep dataset [--prompts 4096] [--batch 16]
    python -m paper_2404_09529_b200.sweep generation [--tokens 20]
    python -m paper_2404_09529_b200.sweep shapes [--batches 8] [--k 16]
"""
from __future__ import annotations

import argparse
import json
import time

import numpy as np
import torch

from .runner import DecodeBatch, PrefillBatch

# Llama-2-7B attention layer shape
HQ, HKV, D, BASE = 32, 32, 128, 10000.0


def _time_ms(fn, iters: int = 5, warmup: int = 2) -> float:
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # a few milliseconds of device-side delay first, so that the host has queued every call before
    # the first one starts: the events then bracket device time, not the host's enqueue rate (these
    # batches are small enough for a step to be shorter than the time it takes to enqueue it)
    if hasattr(torch.cuda, "_sleep"):
        torch.cuda._sleep(4_000_000)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def predictor(n_batches: int, k: int, seed: int, probe=None) -> dict:
    """`probe(packed_batch, padded_batch, q, k, v, lengths)`, if given, is called with the first batch
    after both paths have run on the same tensors (tests check the outputs)."""
    rng = np.random.default_rng(seed)
    gen = torch.Generator(device="cuda").manual_seed(seed)
    rows = []
    for i in range(n_batches):
        lengths = rng.integers(1, 513, size=k).astype(np.int32)
        t = int(lengths.sum())
        tensors = tuple(torch.randn(t, h, D, generator=gen, device="cuda").to(torch.bfloat16) for h in (HQ, HKV, HKV))
        packed = PrefillBatch(lengths, HQ, HKV, D, BASE, mode="packed")
        padded = PrefillBatch(lengths, HQ, HKV, D, BASE, mode="padded")
        packed.load(*tensors); padded.load(*tensors)
        ms_packed = _time_ms(lambda: packed.run_fused(repack=True))
        ms_padded = _time_ms(lambda: padded.run_fused(repack=True))
        assert packed.device_status() == 0 and padded.device_status() == 0
        if probe is not None and i == 0:
            packed.load(*tensors); padded.load(*tensors)
            packed.run_fused(); padded.run_fused()
            torch.cuda.synchronize()
            probe(packed, padded, *tensors, lengths)
        m, total, r = int(lengths.max()), int(lengths.sum()), int(packed.pack.n_bins)
        rows.append({"r_over_k": r / k, "pad_per_prompt": m - total / k, "speedup": ms_padded / ms_packed,
                     "ms_packed": ms_packed, "ms_padded": ms_padded})
        del packed, padded
    x = np.array([[1.0, row["r_over_k"], row["pad_per_prompt"]] for row in rows])
    y = np.array([row["speedup"] for row in rows])
    coef, *_ = np.linalg.lstsq(x, y, rcond=None)
    pred = x @ coef
    ss_res, ss_tot = float(((y - pred) ** 2).sum()), float(((y - y.mean()) ** 2).sum())
    return {"sweep": "predictor", "k": k, "batches": n_batches, "lengths": "uniform int in [1, 512]",
            "layer": {"n_q_heads": HQ, "n_kv_heads": HKV, "head_dim": D},
            "speedup_mean": float(y.mean()), "speedup_min": float(y.min()), "speedup_max": float(y.max()),
            "fit": {"intercept": float(coef[0]), "r_over_k": float(coef[1]), "pad_per_prompt": float(coef[2]),
                    "r2": 1.0 - ss_res / ss_tot if ss_tot > 0 else 1.0},
            "rows": rows}


def dataset(n_prompts: int, batch: int, seed: int, bins_per_launch: int = 0, probe=None) -> dict:
    """Section 6: the whole stream of prompts is bin-packed once (pp_pack, bin size = the longest prompt
    of the stream), the bins are then processed `bins_per_launch` at a time (default: the bin count a
    launch of `batch` * 16 average prompts fills), each launch through pp_prefill_fused on its slice of
    the one packing. Compared on the same stream with length-ordered batching (sort, padded batches of
    `batch`) and with padded batches in arrival order. `probe(batch, q, k, v, lengths)`, if given, is
    called once with a finished launch of every schedule (tests check its outputs)."""
    from . import binding as B
    rng = np.random.default_rng(seed)
    gen = torch.Generator(device="cuda").manual_seed(seed)
    lengths = np.clip(np.rint(np.exp(np.log(200.0) + 0.8 * rng.standard_normal(n_prompts))), 8, 2048).astype(np.int32)
    total = int(lengths.sum())

    def qkv(ls):
        t = int(ls.sum())
        return tuple(torch.randn(t, h, D, generator=gen, device="cuda").to(torch.bfloat16) for h in (HQ, HKV, HKV))

    def run_launch(b, tensors, ls, repack, probed):
        b.load(*tensors)
        ms = _time_ms(lambda: b.run_fused(repack=repack), iters=3, warmup=1)
        assert b.device_status() == 0
        if probe is not None and not probed:
            b.load(*tensors)
            b.run_fused(repack=repack)
            torch.cuda.synchronize()
            probe(b, *tensors, ls)
        return ms

    # (a) one packing of the whole stream, launches of consecutive bins
    t0 = time.perf_counter()
    whole = B.pp_pack(lengths, 0)
    pack_ms = (time.perf_counter() - t0) * 1e3
    if bins_per_launch <= 0:
        bins_per_launch = max(1, int(round(batch * 16 * float(lengths.mean()) / whole.capacity)))
    ms_prepacked, launches = 0.0, 0
    for b0 in range(0, whole.n_bins, bins_per_launch):
        b1 = min(b0 + bins_per_launch, whole.n_bins)
        part, prompts = whole.slice_bins(b0, b1)
        ls = lengths[prompts]
        bt = PrefillBatch(ls, HQ, HKV, D, BASE, pack=part)
        ms_prepacked += run_launch(bt, qkv(ls), ls, False, launches > 0)
        launches += 1
        del bt

    def run_padded(groups):
        ms = 0.0
        for i, g in enumerate(groups):
            bt = PrefillBatch(g, HQ, HKV, D, BASE, mode="padded")
            ms += run_launch(bt, qkv(g), g, True, i > 0)
            del bt
        return ms

    # (b) length-ordered batching: sort, then padded batches of `batch`
    order = np.sort(lengths)
    ms_sorted = run_padded([order[i:i + batch] for i in range(0, n_prompts, batch)])
    # (c) arrival order, padded batches of `batch`
    ms_arrival = run_padded([lengths[i:i + batch] for i in range(0, n_prompts, batch)])
    tps = lambda ms: total / (ms * 1e-3)
    return {"sweep": "dataset", "prompts": n_prompts, "total_tokens": total,
            "lengths": "lognormal(median 200, sigma 0.8) clipped to [8, 2048]",
            "layer": {"n_q_heads": HQ, "n_kv_heads": HKV, "head_dim": D},
            "prepacked": {"bins": int(whole.n_bins), "capacity": int(whole.capacity), "bins_per_launch": bins_per_launch,
                          "launches": launches, "pack_ms_host": pack_ms, "ms": ms_prepacked,
                          "tokens_per_s": tps(ms_prepacked),
                          "fill": total / (int(whole.n_bins) * int(whole.capacity))},
            "length_ordered_padded": {"batch": batch, "ms": ms_sorted, "tokens_per_s": tps(ms_sorted)},
            "arrival_order_padded": {"batch": batch, "ms": ms_arrival, "tokens_per_s": tps(ms_arrival)},
            "speedup_vs_arrival_order": ms_arrival / ms_prepacked,
            "speedup_vs_length_ordered": ms_sorted / ms_prepacked}


def generation(n_tokens: int, seed: int) -> dict:
    gen = torch.Generator(device="cuda").manual_seed(seed)

    def per_token_ms(lengths):
        dec = DecodeBatch(lengths, HQ, HKV, D, BASE, room=n_tokens + 4)
        dec.k_cache.normal_(generator=gen)              # any finite cache contents cost the same
        dec.v_cache.normal_(generator=gen)
        k = len(lengths)
        qn = torch.randn(k, HQ, D, generator=gen, device="cuda").to(torch.bfloat16)
        kn = torch.randn(k, HKV, D, generator=gen, device="cuda").to(torch.bfloat16)
        vn = torch.randn(k, HKV, D, generator=gen, device="cuda").to(torch.bfloat16)
        dec.step(qn, kn, vn)                             # warm-up (also sizes the workspace)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n_tokens):
            dec.step(qn, kn, vn)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n_tokens

    cases = {"toy_9x1_1x1000": np.array([1] * 9 + [1000], np.int32),
             "lognormal_64": np.clip(np.rint(np.exp(np.log(200.0) + 0.8 * np.random.default_rng(seed).standard_normal(64))),
                                     8, 2048).astype(np.int32)}
    out = {"sweep": "generation", "tokens": n_tokens, "layer": {"n_q_heads": HQ, "n_kv_heads": HKV, "head_dim": D}}
    for name, lengths in cases.items():
        ms_true = per_token_ms(lengths)
        ms_padded = per_token_ms(np.full_like(lengths, lengths.max()))
        out[name] = {"prompts": int(len(lengths)), "cached_tokens": int(lengths.sum()),
                     "padded_cached_tokens": int(lengths.max()) * int(len(lengths)),
                     "ms_per_token": ms_true, "ms_per_token_padded": ms_padded, "speedup": ms_padded / ms_true}
    return out


# Length profiles: (mu, sigma) of ln(length) fitted to the reported mean, clipped to the reported
# [min, max] of each evaluation set.
LENGTH_PROFILES = {
    "wiki256": (4.195, 0.437, 1, 256),
    "wiki512": (4.656, 0.512, 6, 512),
    "mmlu": (3.525, 1.126, 4, 1102),
    "hh_rlhf": (5.275, 0.684, 22, 1620),
    "alpaca": (4.709, 0.504, 43, 527),
    "samsum": (4.939, 0.618, 21, 942),
}
# attention-layer shapes (query heads, KV heads, head_dim): hidden 2048 / 16 heads and 4096 / 32 heads
LAYER_SHAPES = {"1.3b": (16, 16, 128), "7b": (32, 32, 128)}


def shapes(n_batches: int, k: int, seed: int) -> dict:
    gen = torch.Generator(device="cuda").manual_seed(seed)
    out = {"sweep": "shapes", "k": k, "batches": n_batches,
           "lengths": "lognormal fitted to each evaluation set's reported min / mean / max", "profiles": {}}
    for pname, (mu, sigma, lo, hi) in LENGTH_PROFILES.items():
        rng = np.random.default_rng(seed)
        batches = [np.clip(np.rint(np.exp(mu + sigma * rng.standard_normal(k))), lo, hi).astype(np.int32)
                   for _ in range(n_batches)]
        row = {"mean_length": float(np.mean([b.mean() for b in batches])),
               "mean_bins": None, "models": {}}
        for mname, (hq, hkv, d) in LAYER_SHAPES.items():
            ms_packed = ms_padded = 0.0
            bins = 0
            for lengths in batches:
                t = int(lengths.sum())
                q = torch.randn(t, hq, d, generator=gen, device="cuda").to(torch.bfloat16)
                kk = torch.randn(t, hkv, d, generator=gen, device="cuda").to(torch.bfloat16)
                v = torch.randn(t, hkv, d, generator=gen, device="cuda").to(torch.bfloat16)
                for mode in ("packed", "padded"):
                    b = PrefillBatch(lengths, hq, hkv, d, BASE, mode=mode)
                    b.load(q, kk, v)
                    ms = _time_ms(lambda: b.run_fused(repack=True))
                    assert b.device_status() == 0
                    if mode == "packed":
                        ms_packed += ms
                        bins += int(b.pack.n_bins)
                    else:
                        ms_padded += ms
                    del b
            row["mean_bins"] = bins / n_batches
            row["models"][mname] = {"ms_packed": ms_packed / n_batches, "ms_padded": ms_padded / n_batches,
                                    "speedup": ms_padded / ms_packed}
        out["profiles"][pname] = row
    return out


def main() -> None:
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    sub = ap.add_subparsers(dest="cmd", required=True)
    p = sub.add_parser("predictor")
    p.add_argument("--batches", type=int, default=40)
    p.add_argument("--k", type=int, default=16)
    p.add_argument("--seed", type=int, default=0)
    d = sub.add_parser("dataset")
    d.add_argument("--prompts", type=int, default=4096)
    d.add_argument("--batch", type=int, default=16)
    d.add_argument("--seed", type=int, default=0)
    gsub = sub.add_parser("generation")
    gsub.add_argument("--tokens", type=int, default=20)
    gsub.add_argument("--seed", type=int, default=0)
    ssub = sub.add_parser("shapes")
    ssub.add_argument("--batches", type=int, default=8)
    ssub.add_argument("--k", type=int, default=16)
    ssub.add_argument("--seed", type=int, default=0)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("the sweeps need a GPU: the library has no CPU path")
    if args.cmd == "predictor":
        out = predictor(args.batches, args.k, args.seed)
    elif args.cmd == "dataset":
        out = dataset(args.prompts, args.batch, args.seed)
    elif args.cmd == "generation":
        out = generation(args.tokens, args.seed)
    else:
        out = shapes(args.batches, args.k, args.seed)
    print(json.dumps(out))


if __name__ == "__main__":
    main()
