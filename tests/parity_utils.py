"""Shared helpers of the GPU parity tests: run the CUDA path through the C-ABI binding and
compare it element by element with the float64 oracle."""
import numpy as np
import torch

from oracle import prepack_oracle as orc
from paper_2404_09529_b200.runner import PrefillBatch
from workloads import split_by_prompt

# spec tolerances for bf16 outputs and caches against the float64 oracle
MAX_ABS_TOL = 2e-2
MEAN_ABS_TOL = 2e-3


def to64(x: torch.Tensor) -> np.ndarray:
    return x.detach().to("cpu", torch.float32).numpy().astype(np.float64)


class ErrStat:
    def __init__(self):
        self.max_abs, self.sum_abs, self.n = 0.0, 0.0, 0

    def add(self, got: np.ndarray, ref: np.ndarray):
        assert got.shape == ref.shape, (got.shape, ref.shape)
        assert np.all(np.isfinite(got))
        d = np.abs(got - ref)
        self.max_abs = max(self.max_abs, float(d.max()) if d.size else 0.0)
        self.sum_abs += float(d.sum())
        self.n += d.size

    @property
    def mean_abs(self):
        return self.sum_abs / max(self.n, 1)

    def check(self, what):
        assert self.n > 0, what
        assert self.max_abs <= MAX_ABS_TOL, (what, "max", self.max_abs)
        assert self.mean_abs <= MEAN_ABS_TOL, (what, "mean", self.mean_abs)


def run_cuda(lengths, q_tok, k_tok, v_tok, hq, hkv, d, base, mode="packed", fused=False, room=0, guard=False):
    batch = PrefillBatch(lengths, hq, hkv, d, base, mode=mode, room=room, guard=guard)
    batch.load(q_tok, k_tok, v_tok)
    batch.run_fused() if fused else batch.run()
    torch.cuda.synchronize()
    assert batch.device_status() == 0
    if guard:
        batch.assert_untouched()
    return batch


def compare_full(batch, lengths, q_tok, k_tok, v_tok, base, prompts=None):
    """Every row, head and cache element of the chosen prompts (default all) against the oracle."""
    o_cuda = split_by_prompt(batch.o_tokens().cpu(), lengths)
    qs, ks, vs = (split_by_prompt(t.cpu(), lengths) for t in (q_tok, k_tok, v_tok))
    e_o, e_k, e_v = ErrStat(), ErrStat(), ErrStat()
    for i in (range(len(lengths)) if prompts is None else prompts):
        o_ref, kc_ref, vc_ref = orc.prefill_prompt(to64(qs[i]), to64(ks[i]), to64(vs[i]), base)
        kc, vc = batch.caches(i)
        l = int(lengths[i])                       # a cache block may have spare rows behind the prompt
        e_o.add(to64(o_cuda[i]), o_ref)
        e_k.add(to64(kc[:, :l]), kc_ref)
        e_v.add(to64(vc[:, :l]), vc_ref)
    e_o.check("O"); e_k.check("K cache"); e_v.check("V cache")
    assert e_v.max_abs == 0.0
    return e_o, e_k, e_v


def oracle_refs(lengths, q_tok, k_tok, v_tok, base):
    """The oracle's (O, K cache, V cache) of every prompt alone, computed once for several runs."""
    qs, ks, vs = (split_by_prompt(t.cpu(), lengths) for t in (q_tok, k_tok, v_tok))
    return [orc.prefill_prompt(to64(qs[i]), to64(ks[i]), to64(vs[i]), base) for i in range(len(lengths))]


def compare_with_refs(batch, lengths, refs):
    """Every row, head and cache element of every prompt against precomputed oracle results."""
    o_cuda = split_by_prompt(batch.o_tokens().cpu(), lengths)
    e_o, e_k, e_v = ErrStat(), ErrStat(), ErrStat()
    for i, (o_ref, kc_ref, vc_ref) in enumerate(refs):
        kc, vc = batch.caches(i)
        l = int(lengths[i])
        e_o.add(to64(o_cuda[i]), o_ref)
        e_k.add(to64(kc[:, :l]), kc_ref)
        e_v.add(to64(vc[:, :l]), vc_ref)
    e_o.check("O"); e_k.check("K cache"); e_v.check("V cache")
    assert e_v.max_abs == 0.0
    return e_o, e_k, e_v


def expected_schedule(seg_bins, hq, hkv):
    """What the attention kernel's host scheduler must choose for a packing, restated from its rule
    (independent of the library): seg_bins is a list of bins, each a list of segment lengths in
    placement order. Mean number of 128-row key tiles per 128-row query tile, counting for a query
    tile the key rows from the 128-aligned start of the first prompt it touches to its last row:
    below 8 the kernel runs its independent mode (64-row key tiles, template <D, true>), otherwise
    its shared-stream mode (template <D, false>), pairing two query heads when the GQA group is even
    and two consecutive row tiles otherwise. Returns (mode, pairing) as pp_prefill_schedule_info
    numbers them."""
    q_tiles = kv_tiles = 0
    for segs in seg_bins:
        starts = np.concatenate([[0], np.cumsum(segs)])
        used = int(starts[-1])
        for q0 in range(0, used, 128):
            s = int(np.searchsorted(starts[:-1], q0, side="right")) - 1
            kv_lo = (int(starts[s]) // 128) * 128
            kv_tiles += (min(q0 + 128, used) - kv_lo + 127) // 128
            q_tiles += 1
    independent = kv_tiles / q_tiles < 8.0
    if independent:
        return 1, 2
    return 0, (0 if (hq // hkv) % 2 == 0 else 1)


def compare_sampled(batch, lengths, q_tok, k_tok, v_tok, base, prompts, kv_heads, n_rows, seed=0):
    """Sampled query rows of the query heads that read `kv_heads`, plus the full K/V cache of
    those KV heads, for the chosen prompts."""
    rng = np.random.default_rng(seed)
    hq, hkv = batch.hq, batch.hkv
    g = hq // hkv
    q_heads = [kv * g + t for kv in kv_heads for t in range(g)]
    prefix = np.concatenate([[0], np.cumsum(np.asarray(lengths, dtype=np.int64))])
    o_all = batch.o_tokens()
    e_o, e_k, e_v = ErrStat(), ErrStat(), ErrStat()
    for i in prompts:
        l = int(lengths[i])
        sl = slice(int(prefix[i]), int(prefix[i + 1]))
        q = to64(q_tok[sl][:, q_heads]); k = to64(k_tok[sl][:, kv_heads]); v = to64(v_tok[sl][:, kv_heads])
        rows = np.unique(np.concatenate([[0, l - 1, min(l - 1, 127), min(l - 1, 128)],
                                         rng.integers(0, l, size=n_rows)]))
        o_ref, kc_ref, vc_ref = orc.prefill_prompt(q, k, v, base, rows=rows)
        e_o.add(to64(o_all[sl][rows][:, q_heads]), o_ref)
        kc, vc = batch.caches(i)
        e_k.add(to64(kc[kv_heads][:, :l]), kc_ref)
        e_v.add(to64(vc[kv_heads][:, :l]), vc_ref)
    e_o.check("O"); e_k.check("K cache"); e_v.check("V cache")
    assert e_v.max_abs == 0.0
    return e_o, e_k, e_v
