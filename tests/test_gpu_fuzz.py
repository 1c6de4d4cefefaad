"""Seeded random shapes through both public routes and both batch modes, against the float64 oracle:
lengths around the tile sizes (64 / 128 rows), many prompts per bin, GQA groups 1..8, both head sizes."""
import numpy as np
import pytest
import torch

from parity_utils import compare_full
from paper_2404_09529_b200.runner import PrefillBatch

pytestmark = pytest.mark.gpu


def _draw(rng):
    d = int(rng.choice([64, 128]))
    hkv = int(rng.choice([1, 2, 4]))
    hq = hkv * int(rng.choice([1, 2, 3, 4, 8]))
    k = int(rng.integers(1, 32))
    kind = int(rng.integers(0, 4))
    if kind == 0:
        lengths = rng.integers(1, 20, size=k)
    elif kind == 1:
        lengths = rng.integers(1, 300, size=k)
    elif kind == 2:
        lengths = np.concatenate([rng.integers(1, 10, size=k), rng.integers(500, 1200, size=max(1, k // 8))])
    else:
        lengths = rng.choice([63, 64, 65, 127, 128, 129, 191, 192, 193, 255, 256, 257], size=k)
    return lengths.astype(np.int32), hq, hkv, d, float(rng.choice([10000.0, 500000.0]))


def _draw_long(rng):
    """A few long prompts next to short ones: the shared-stream mode of the attention kernel, with head
    pairs (even GQA group) or paired row tiles (odd group), tile counts odd and even."""
    d = int(rng.choice([64, 128]))
    hkv = int(rng.choice([1, 2]))
    hq = hkv * int(rng.choice([1, 2, 3]))
    lengths = np.concatenate([rng.integers(1400, 3300, size=int(rng.integers(1, 4))),
                              rng.integers(1, 200, size=int(rng.integers(0, 6)))])
    return lengths.astype(np.int32), hq, hkv, d, float(rng.choice([10000.0, 500000.0]))


@pytest.mark.parametrize("seed", range(6))
def test_random_long_shapes_full_parity(seed):
    rng = np.random.default_rng(5000 + seed)
    lengths, hq, hkv, d, base = _draw_long(rng)
    t = int(lengths.sum())
    gen = torch.Generator().manual_seed(100 + seed)
    q = torch.randn(t, hq, d, generator=gen).to(torch.bfloat16)
    k = torch.randn(t, hkv, d, generator=gen).to(torch.bfloat16)
    v = torch.randn(t, hkv, d, generator=gen).to(torch.bfloat16)
    from parity_utils import compare_with_refs, oracle_refs
    refs = oracle_refs(lengths, q, k, v, base)
    for fused in (False, True):
        b = PrefillBatch(lengths, hq, hkv, d, base, guard=True)
        b.load(q, k, v)
        b.run_fused() if fused else b.run()
        torch.cuda.synchronize()
        assert b.device_status() == 0
        b.assert_untouched()
        compare_with_refs(b, lengths, refs)


@pytest.mark.parametrize("seed", range(12))
def test_random_shapes_full_parity(seed):
    rng = np.random.default_rng(1000 + seed)
    lengths, hq, hkv, d, base = _draw(rng)
    t = int(lengths.sum())
    gen = torch.Generator().manual_seed(seed)
    q = torch.randn(t, hq, d, generator=gen).to(torch.bfloat16)
    k = torch.randn(t, hkv, d, generator=gen).to(torch.bfloat16)
    v = torch.randn(t, hkv, d, generator=gen).to(torch.bfloat16)
    modes = ("packed", "padded") if len(lengths) * int(lengths.max()) <= 20000 else ("packed",)
    for mode in modes:
        for fused in (False, True):
            b = PrefillBatch(lengths, hq, hkv, d, base, mode=mode)
            b.load(q, k, v)
            b.run_fused() if fused else b.run()
            torch.cuda.synchronize()
            assert b.device_status() == 0
            compare_full(b, lengths, q, k, v, base)
