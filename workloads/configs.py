"""The five synthetic workloads (length distributions + attention-layer shapes).

The paper measured on text datasets (MMLU, SamSum, Alpaca, Wikitext, HH-RLHF,
Section 4.1); none of them is used here. Each workload below is a seeded length
distribution plus N(0,1) bf16 Q/K/V of a Llama-like attention layer shape, and
stands in for them.

Lengths are drawn with ``numpy.random.default_rng(0)`` by the recipes in
``draw_lengths``. Because numpy does not promise identical streams across
versions, the drawn lists are also stored as JSON under ``workloads/lengths/``;
``prompt_lengths`` reads the stored list (and is what tests and the bench use).
"""
from __future__ import annotations

import json
import os
from dataclasses import dataclass

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))


@dataclass(frozen=True)
class WorkloadConfig:
    index: int          # 1-based, also used in the Q/K/V seed (1000 + index)
    name: str
    n_prompts: int      # k
    n_q_heads: int      # Hq
    n_kv_heads: int     # Hkv
    head_dim: int       # D
    rope_base: float
    description: str


CONFIGS = {
    "tiny": WorkloadConfig(1, "tiny", 8, 4, 4, 64, 10000.0,
                           "8 prompts, lengths uniform int in [16,128]"),
    "llama2_7b": WorkloadConfig(2, "llama2_7b", 64, 32, 32, 128, 10000.0,
                                "64 prompts, lognormal(median 200, sigma 0.8) clipped to [8,2048]"),
    "llama3_8b_gqa": WorkloadConfig(3, "llama3_8b_gqa", 256, 32, 8, 128, 500000.0,
                                    "256 prompts, 70% U[20,200] / 30% U[1000,4000]"),
    "long_mix": WorkloadConfig(4, "long_mix", 16, 32, 32, 128, 500000.0,
                               "16 prompts, log-uniform in [128,32768]"),
    "many_short": WorkloadConfig(5, "many_short", 2048, 32, 8, 64, 500000.0,
                                 "2048 prompts, Pareto(alpha 1.5, min 8) clipped to [8,8192]"),
}


def get_config(name: str) -> WorkloadConfig:
    return CONFIGS[name]


def draw_lengths(name: str, seed: int = 0) -> np.ndarray:
    """Draw the prompt lengths of workload ``name`` (exact draw order matters)."""
    rng = np.random.default_rng(seed)
    k = CONFIGS[name].n_prompts
    if name == "tiny":
        l = rng.integers(16, 129, size=k)
    elif name == "llama2_7b":
        z = rng.standard_normal(k)
        l = np.clip(np.rint(np.exp(np.log(200.0) + 0.8 * z)), 8, 2048)
    elif name == "llama3_8b_gqa":
        u = rng.random(k)
        a = rng.integers(20, 201, k)
        b = rng.integers(1000, 4001, k)
        l = np.where(u < 0.7, a, b)
    elif name == "long_mix":
        u = rng.random(k)
        l = np.clip(np.rint(np.exp(np.log(128.0) + u * (np.log(32768.0) - np.log(128.0)))),
                    128, 32768)
    elif name == "many_short":
        u = rng.random(k)
        l = np.clip(np.floor(8.0 * (1.0 - u) ** (-1.0 / 1.5)), 8, 8192)
    else:
        raise KeyError(name)
    return np.asarray(l, dtype=np.int64).astype(np.int32)


def _lengths_path(name: str) -> str:
    return os.path.join(_HERE, "lengths", f"{name}.json")


def prompt_lengths(name: str) -> np.ndarray:
    """The stored seed-0 length list of workload ``name`` (int32, original prompt order)."""
    with open(_lengths_path(name)) as f:
        return np.asarray(json.load(f)["lengths"], dtype=np.int32)


def make_qkv(cfg: WorkloadConfig, total_tokens: int, device: str = "cpu",
             seed: int | None = None):
    """N(0,1) Q [T,Hq,D], K [T,Hkv,D], V [T,Hkv,D] in bf16, real tokens in original
    prompt order. Drawn in fp32 in the order Q, K, V from one generator seeded
    1000 + cfg.index on ``device``, then rounded to bf16."""
    g = torch.Generator(device=device)
    g.manual_seed(1000 + cfg.index if seed is None else seed)
    out = []
    for heads in (cfg.n_q_heads, cfg.n_kv_heads, cfg.n_kv_heads):
        x = torch.randn((total_tokens, heads, cfg.head_dim), generator=g,
                        dtype=torch.float32, device=device)
        out.append(x.to(torch.bfloat16))
        del x
    return tuple(out)


def split_by_prompt(x: torch.Tensor, lengths) -> list:
    """Views of a token-major tensor [T, ...], one per prompt, original order."""
    outs, o = [], 0
    for l in lengths:
        l = int(l)
        outs.append(x[o:o + l])
        o += l
    return outs


def write_length_fixtures() -> None:
    """Regenerate workloads/lengths/*.json from the recipes (run by hand)."""
    os.makedirs(os.path.join(_HERE, "lengths"), exist_ok=True)
    for name in CONFIGS:
        l = draw_lengths(name)
        with open(_lengths_path(name), "w") as f:
            json.dump({"workload": name, "seed": 0, "numpy": np.__version__,
                       "lengths": [int(v) for v in l]}, f)
            f.write("\n")


if __name__ == "__main__":
    write_length_fixtures()
