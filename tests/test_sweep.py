"""The measurement sweeps run end to end on small inputs (GPU only: the library has no CPU path)."""
import pytest

pytestmark = pytest.mark.gpu


def test_predictor_sweep_small():
    from paper_2404_09529_b200 import sweep
    out = sweep.predictor(n_batches=4, k=8, seed=1)
    assert out["batches"] == 4 and len(out["rows"]) == 4
    for row in out["rows"]:
        assert 0.0 < row["r_over_k"] <= 1.0 and row["pad_per_prompt"] >= 0.0
        assert row["ms_packed"] > 0.0 and row["ms_padded"] > 0.0
    assert set(out["fit"]) == {"intercept", "r_over_k", "pad_per_prompt", "r2"}


def test_dataset_sweep_small():
    from paper_2404_09529_b200 import sweep
    out = sweep.dataset(n_prompts=64, batch=8, seed=1)
    assert out["total_tokens"] > 0
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
