"""The measurement sweeps run end to end on small inputs (GPU only: the library has no CPU path), and
one batch of each is checked against the float64 oracle: every row, head and cache element of its
longest and its shortest prompt."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _check_against_oracle(batch, q, k, v, lengths):
    from parity_utils import compare_full
    order = np.argsort(lengths)
    compare_full(batch, np.asarray(lengths), q, k, v, batch.rope_base, prompts=sorted({int(order[0]), int(order[-1])}))


def test_predictor_sweep_small():
    from paper_2404_09529_b200 import sweep
    seen = []

    def probe(packed, padded, q, k, v, lengths):
        _check_against_oracle(packed, q, k, v, lengths)
        _check_against_oracle(padded, q, k, v, lengths)
        seen.append(len(lengths))

    out = sweep.predictor(n_batches=4, k=8, seed=1, probe=probe)
    assert seen == [8]
    assert out["batches"] == 4 and len(out["rows"]) == 4
    for row in out["rows"]:
        assert 0.0 < row["r_over_k"] <= 1.0 and row["pad_per_prompt"] >= 0.0
        assert row["ms_packed"] > 0.0 and row["ms_padded"] > 0.0
    assert set(out["fit"]) == {"intercept", "r_over_k", "pad_per_prompt", "r2"}


def test_dataset_sweep_small():
    from paper_2404_09529_b200 import sweep
    seen = []

    def probe(batch, q, k, v, lengths):
        _check_against_oracle(batch, q, k, v, lengths)
        seen.append(batch.mode)

    out = sweep.dataset(n_prompts=64, batch=8, seed=1, bins_per_launch=3, probe=probe)
    assert seen == ["prepacked", "padded", "padded"]
    assert out["total_tokens"] > 0
    # one packing of the whole stream: bins of the stream-wide capacity, cut into launches of 3 bins
    pre = out["prepacked"]
    assert pre["launches"] == -(-pre["bins"] // 3) and pre["launches"] > 1
    assert pre["bins"] * pre["capacity"] >= out["total_tokens"] and 0.5 < pre["fill"] <= 1.0
    for key in ("prepacked", "length_ordered_padded", "arrival_order_padded"):
        assert out[key]["tokens_per_s"] > 0.0
    # with a lognormal length mix, padding to the batch maximum in arrival order wastes the most
    assert out["speedup_vs_arrival_order"] > 1.0


def test_generation_sweep_small():
    from paper_2404_09529_b200 import sweep
    out = sweep.generation(n_tokens=3, seed=1)
    toy = out["toy_9x1_1x1000"]
    assert toy["cached_tokens"] == 1009 and toy["padded_cached_tokens"] == 10000
    assert toy["ms_per_token"] > 0.0 and toy["ms_per_token_padded"] > 0.0


def test_shapes_sweep_small():
    from paper_2404_09529_b200 import sweep
    out = sweep.shapes(n_batches=1, k=8, seed=1)
    assert set(out["profiles"]) == set(sweep.LENGTH_PROFILES)
    for name, row in out["profiles"].items():
        lo, hi = sweep.LENGTH_PROFILES[name][2:]
        assert lo <= row["mean_length"] <= hi and 1 <= row["mean_bins"] <= 8
        for model in sweep.LAYER_SHAPES:
            assert row["models"][model]["ms_packed"] > 0.0 and row["models"][model]["ms_padded"] > 0.0
