"""Pins for the float64 CPU oracle: each test ties it to something other than itself --
a hand-worked example, a closed form, a library routine, brute force, or the paper's
claim that packed, padded and one-prompt-at-a-time prefill agree exactly."""
import json
import math
import os

import numpy as np
import pytest
import torch

from oracle import prepack_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand_prompts(rng, lengths, hq, hkv, d):
    qs = [rng.standard_normal((l, hq, d)) for l in lengths]
    ks = [rng.standard_normal((l, hkv, d)) for l in lengths]
    vs = [rng.standard_normal((l, hkv, d)) for l in lengths]
    return qs, ks, vs


# ----------------------------------------------------------------------------- packing

def _bins_of(pack):
    ptr = pack["bin_seg_ptr"]
    return ([pack["seg_prompt"][ptr[b]:ptr[b + 1]] for b in range(pack["n_bins"])],
            [pack["seg_start"][ptr[b]:ptr[b + 1]] for b in range(pack["n_bins"])])


def test_pack_tiny_hand_worked():
    """Algorithm 1 (BINPACK) on the tiny workload, against the hand-worked fixture."""
    g = json.load(open(os.path.join(GOLDEN, "pack_tiny.json")))
    pack = orc.ffd_pack(g["lengths"], 0)
    bins, starts = _bins_of(pack)
    assert pack["capacity"] == g["capacity"]
    assert pack["n_bins"] == g["n_bins"]
    assert bins == g["bins"]
    assert starts == g["seg_start"]
    assert pack["bin_used"] == g["loads"]
    assert pack["bin_of"] == g["bin_of"]
    assert pack["off_of"] == g["off_of"]
    pos, seg = orc.restart_position_ids(pack)
    # bin 1 holds prompt 1 (87 tokens) then prompt 6 (24 tokens), then one pad row
    expect = list(range(87)) + list(range(24)) + [0]
    assert pos[1].tolist() == expect
    assert seg[1].tolist() == [1] * 87 + [2] * 24 + [-1]


def test_pack_small_hand_worked_cases():
    g = json.load(open(os.path.join(GOLDEN, "pack_small_cases.json")))
    for case in g["cases"]:
        pack = orc.ffd_pack(case["lengths"], case["capacity"])
        bins, starts = _bins_of(pack)
        assert bins == case["bins"], case
        assert starts == case["seg_start"], case


def _check_pack_invariants(lengths, cap_arg):
    pack = orc.ffd_pack(lengths, cap_arg)
    k, m = len(lengths), pack["capacity"]
    r = pack["n_bins"]
    total = int(sum(lengths))
    assert sorted(pack["seg_prompt"]) == list(range(k))            # every prompt exactly once
    assert all(u <= m for u in pack["bin_used"])
    assert math.ceil(total / m) <= r <= k                          # Section 3.1: r <= k
    assert pack["bin_seg_ptr"][0] == 0 and pack["bin_seg_ptr"][-1] == k
    for i in range(k):
        b, off = pack["bin_of"][i], pack["off_of"][i]
        segs = range(pack["bin_seg_ptr"][b], pack["bin_seg_ptr"][b + 1])
        s = [s for s in segs if pack["seg_prompt"][s] == i]
        assert len(s) == 1 and pack["seg_start"][s[0]] == off and pack["seg_len"][s[0]] == lengths[i]
    # segments of a bin tile it contiguously from 0
    for b in range(r):
        off = 0
        for s in range(pack["bin_seg_ptr"][b], pack["bin_seg_ptr"][b + 1]):
            assert pack["seg_start"][s] == off
            off += pack["seg_len"][s]
        assert off == pack["bin_used"][b]
    # first-fit property, replayed: when an item was placed in bin b it fit in no earlier bin
    order = sorted(range(k), key=lambda i: (-lengths[i], i))
    loads = [0] * r
    for i in order:
        b = pack["bin_of"][i]
        assert pack["off_of"][i] == loads[b]
        for e in range(b):
            assert loads[e] + lengths[i] > m
        loads[b] += lengths[i]
    return pack


def test_pack_invariants_random():
    rng = np.random.default_rng(123)
    for trial in range(200):
        k = int(rng.integers(1, 60))
        hi = int(rng.integers(1, 200))
        lengths = rng.integers(1, hi + 1, size=k).tolist()
        cap = 0 if trial % 3 else max(lengths) + int(rng.integers(0, 50))
        _check_pack_invariants(lengths, cap)


def test_pack_best_and_worst_case():
    """Section 3.3: best case r = L/m, worst case r = k."""
    assert orc.ffd_pack([7] * 9, 0)["n_bins"] == 9
    assert orc.ffd_pack([8, 4, 4, 2, 2, 2, 2], 0)["n_bins"] == 3       # L = 24, m = 8
    assert orc.ffd_pack([8, 5, 5, 5], 0)["n_bins"] == 4                # nothing pairs up


def test_pack_rejects_bad_lengths():
    with pytest.raises(ValueError):
        orc.ffd_pack([3, 0, 2], 0)
    with pytest.raises(ValueError):
        orc.ffd_pack([], 0)
    with pytest.raises(ValueError):
        orc.ffd_pack([3, 9], 8)


def test_independent_mask_is_block_lower_triangular():
    pack = orc.ffd_pack([3, 2, 5], 0)          # bins [[2],[0,1]]
    assert _bins_of(pack)[0] == [[2], [0, 1]]
    m1 = orc.independent_mask(pack, 1).astype(int)
    expect = np.array([[1, 0, 0, 0, 0],
                       [1, 1, 0, 0, 0],
                       [1, 1, 1, 0, 0],
                       [0, 0, 0, 1, 0],
                       [0, 0, 0, 1, 1]])
    assert (m1 == expect).all()
    assert (orc.independent_mask(pack, 0) == np.tril(np.ones((5, 5), dtype=bool))).all()


# ----------------------------------------------------------------------------- RoPE

def test_rope_matches_complex_rotation():
    """(x_j + i x_{j+D/2}) * exp(i p theta_j), theta_j = base^(-2j/D)."""
    rng = np.random.default_rng(1)
    l, h, d, base = 9, 3, 16, 10000.0
    x = rng.standard_normal((l, h, d))
    pos = rng.integers(0, 5000, size=l)
    out = orc.rope_rotate(x, pos, base)
    for t in range(l):
        for j in range(d // 2):
            theta = base ** (-2.0 * j / d)
            z = (x[t, :, j] + 1j * x[t, :, j + d // 2]) * np.exp(1j * pos[t] * theta)
            assert np.allclose(out[t, :, j], z.real, atol=1e-12, rtol=0)
            assert np.allclose(out[t, :, j + d // 2], z.imag, atol=1e-12, rtol=0)


def test_rope_frequencies_endpoints():
    th = orc.rope_frequencies(128, 500000.0)
    assert th[0] == 1.0
    assert abs(th[32] - 500000.0 ** -0.5) < 1e-18      # j = D/4 -> base^(-1/2)
    assert abs(th[63] * 500000.0 ** (126 / 128) - 1.0) < 1e-12
    assert np.all(np.diff(th) < 0)


def test_rope_position_zero_is_identity_and_norm_preserving():
    rng = np.random.default_rng(2)
    x = rng.standard_normal((6, 2, 8))
    out = orc.rope_rotate(x, np.zeros(6, dtype=int), 10000.0)
    assert np.array_equal(out, x)
    out = orc.rope_rotate(x, np.arange(6) * 1000, 10000.0)
    n_in = x[..., :4] ** 2 + x[..., 4:] ** 2
    n_out = out[..., :4] ** 2 + out[..., 4:] ** 2
    assert np.allclose(n_in, n_out, atol=1e-12)


def test_rope_scores_depend_on_relative_position_only():
    rng = np.random.default_rng(3)
    q, k = rng.standard_normal((1, 1, 32)), rng.standard_normal((1, 1, 32))
    def score(pq, pk):
        return float(np.sum(orc.rope_rotate(q, [pq], 5e5) * orc.rope_rotate(k, [pk], 5e5)))
    assert abs(score(40, 7) - score(40 + 777, 7 + 777)) < 1e-11
    assert abs(score(40, 7) - score(41, 7)) > 1e-6


# ----------------------------------------------------------------------------- attention

@pytest.mark.parametrize("hq,hkv", [(4, 4), (4, 2), (6, 1)])
def test_single_prompt_matches_torch_sdpa_fp64(hq, hkv):
    """One prompt alone reduces to causal scaled-dot-product attention (library routine)."""
    rng = np.random.default_rng(4)
    l, d, base = 37, 16, 10000.0
    q, k, v = rng.standard_normal((l, hq, d)), rng.standard_normal((l, hkv, d)), rng.standard_normal((l, hkv, d))
    o, kc, vc = orc.prefill_prompt(q, k, v, base)
    # the rotation for the library path comes from the complex form, not from rope_rotate
    def crot(x):
        half = d // 2
        theta = base ** (-2.0 * np.arange(half) / d)
        z = (x[..., :half] + 1j * x[..., half:]) * np.exp(1j * np.arange(l)[:, None, None] * theta)
        return np.concatenate([z.real, z.imag], axis=-1)
    tq = torch.from_numpy(crot(q)).permute(1, 0, 2)[None]
    tk = torch.from_numpy(crot(k)).permute(1, 0, 2)[None].repeat_interleave(hq // hkv, dim=1)
    tv = torch.from_numpy(v).permute(1, 0, 2)[None].repeat_interleave(hq // hkv, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)
    ref = ref[0].permute(1, 0, 2).numpy()
    assert np.allclose(o, ref, atol=1e-12, rtol=0)
    assert np.allclose(kc, np.transpose(crot(k), (1, 0, 2)), atol=1e-12, rtol=0)
    assert np.array_equal(vc, np.transpose(v, (1, 0, 2)))


def test_closed_forms():
    rng = np.random.default_rng(5)
    l, hq, hkv, d = 21, 4, 2, 8
    q = rng.standard_normal((l, hq, d))
    v = rng.standard_normal((l, hkv, d))
    # keys all zero -> every score is 0 -> uniform weights over the causal prefix
    o, _, _ = orc.prefill_prompt(q, np.zeros((l, hkv, d)), v, 10000.0)
    prefix_mean = np.cumsum(v, axis=0) / np.arange(1, l + 1)[:, None, None]
    for h in range(hq):
        assert np.allclose(o[:, h], prefix_mean[:, h // 2], atol=1e-12)
    # identical value rows -> output is that row
    k = rng.standard_normal((l, hkv, d))
    vrow = rng.standard_normal((1, hkv, d))
    o, _, _ = orc.prefill_prompt(q, k, np.repeat(vrow, l, axis=0), 10000.0)
    for h in range(hq):
        assert np.allclose(o[:, h], vrow[0, h // 2][None, :], atol=1e-12)
    # first token sees only itself; position 0 leaves K row 0 untouched
    o, kc, vc = orc.prefill_prompt(q, k, v, 10000.0)
    for h in range(hq):
        assert np.array_equal(o[0, h], v[0, h // 2])
    assert np.array_equal(kc[:, 0, :], k[0])


def test_rows_and_heads_subset_matches_full():
    rng = np.random.default_rng(6)
    q, k, v = rng.standard_normal((50, 4, 8)), rng.standard_normal((50, 2, 8)), rng.standard_normal((50, 2, 8))
    o, _, _ = orc.prefill_prompt(q, k, v, 10000.0)
    rows, heads = [0, 7, 49], [1, 3]
    o2, _, _ = orc.prefill_prompt(q, k, v, 10000.0, rows=rows, q_heads=heads, row_block=2)
    assert np.allclose(o2, o[rows][:, heads], atol=1e-13)


def test_brute_force_agrees():
    rng = np.random.default_rng(7)
    for l in (1, 5, 16):
        q, k, v = rng.standard_normal((l, 2, 8)), rng.standard_normal((l, 2, 8)), rng.standard_normal((l, 2, 8))
        o, kc, _ = orc.prefill_prompt(q, k, v, 10000.0)
        bo, bkc = orc.brute_force_prompt(q.tolist(), k.tolist(), v.tolist(), 10000.0)
        assert np.allclose(o, np.array(bo), atol=1e-12, rtol=0)
        assert np.allclose(kc, np.array(bkc), atol=1e-12, rtol=0)
    # GQA in the brute force too
    q, k, v = rng.standard_normal((6, 4, 8)), rng.standard_normal((6, 2, 8)), rng.standard_normal((6, 2, 8))
    o, _, _ = orc.prefill_prompt(q, k, v, 500000.0)
    bo, _ = orc.brute_force_prompt(q.tolist(), k.tolist(), v.tolist(), 500000.0)
    assert np.allclose(o, np.array(bo), atol=1e-12, rtol=0)


# ----------------------------------------------------------------------------- the paper's exactness claim

@pytest.mark.parametrize("hq,hkv", [(4, 4), (4, 1)])
def test_packed_equals_padded_equals_alone(hq, hkv):
    """Section 3.3: prepacking computes exactly the caches of padded full batching."""
    rng = np.random.default_rng(8)
    lengths = [112, 87, 73, 46, 50, 20, 24, 17]
    qs, ks, vs = _rand_prompts(rng, lengths, hq, hkv, 16)
    o_a, kc_a, vc_a = orc.prefill_batch(qs, ks, vs, 10000.0)
    o_p, kc_p, vc_p = orc.packed_dense_prefill(qs, ks, vs, 10000.0)
    o_f, kc_f, vc_f = orc.padded_prefill(qs, ks, vs, 10000.0)
    for i in range(len(lengths)):
        for a, b in ((o_p[i], o_a[i]), (o_f[i], o_a[i]), (kc_p[i], kc_a[i]), (kc_f[i], kc_a[i]),
                     (vc_p[i], vc_a[i]), (vc_f[i], vc_a[i])):
            assert a.shape == b.shape
            assert np.max(np.abs(a - b)) <= 1e-12


def test_no_cross_prompt_probability_mass():
    """Section 3.2: no prompt attends to another one in the same bin."""
    rng = np.random.default_rng(9)
    lengths = [9, 30, 14, 7, 16, 5]
    qs, ks, vs = _rand_prompts(rng, lengths, 2, 2, 8)
    o, _, _, pack, probs = orc.packed_dense_prefill(qs, ks, vs, 10000.0, return_probs=True)
    assert pack["n_bins"] < len(lengths)
    _, seg = orc.restart_position_ids(pack)
    for b in range(pack["n_bins"]):
        same = (seg[b][:, None] == seg[b][None, :]) & (seg[b][:, None] >= 0)
        for h in range(2):
            assert np.all(probs[b][h][~same] == 0.0)
            live = seg[b] >= 0
            assert np.allclose(probs[b][h][live].sum(axis=1), 1.0, atol=1e-14)
    # and changing one prompt leaves every other prompt's result untouched
    qs2, ks2, vs2 = [x.copy() for x in qs], [x.copy() for x in ks], [x.copy() for x in vs]
    qs2[2] *= 50.0; ks2[2] *= -50.0; vs2[2] += 1000.0
    o2, kc2, _ = orc.packed_dense_prefill(qs2, ks2, vs2, 10000.0)
    for i in range(len(lengths)):
        if i != 2:
            assert np.array_equal(o2[i], o[i])


def test_restart_positions_matter_for_k_cache():
    """Relative-position invariance hides a wrong restart from O; the K cache exposes it."""
    rng = np.random.default_rng(10)
    qs, ks, vs = _rand_prompts(rng, [6, 4], 2, 2, 8)
    _, kc, _ = orc.packed_dense_prefill(qs, ks, vs, 10000.0, capacity=10)
    # prompt 1 sits at offset 6 in the bin; its cache must still equal a rotation by 0..3
    assert np.allclose(kc[1], np.transpose(orc.rope_rotate(ks[1], np.arange(4), 10000.0), (1, 0, 2)),
                       atol=1e-13)
    wrong = np.transpose(orc.rope_rotate(ks[1], np.arange(6, 10), 10000.0), (1, 0, 2))
    assert np.max(np.abs(kc[1] - wrong)) > 1e-3


def test_decode_step_equals_last_row_of_the_extended_prompt():
    """Pin of the generation step: decoding token l from the caches of tokens 0..l-1 must give the
    last attention row and the caches of an (l + 1)-token prefill (Sections 3.2 and 7)."""
    rng = np.random.default_rng(11)
    for (l, hq, hkv, d) in [(1, 2, 2, 8), (5, 4, 2, 16), (37, 4, 1, 64)]:
        q = rng.standard_normal((l + 1, hq, d))
        k = rng.standard_normal((l + 1, hkv, d))
        v = rng.standard_normal((l + 1, hkv, d))
        o_full, kc_full, vc_full = orc.prefill_prompt(q, k, v, 10000.0)
        _, kc, vc = orc.prefill_prompt(q[:l], k[:l], v[:l], 10000.0)
        o, kc2, vc2 = orc.decode_step(q[l], k[l], v[l], kc, vc, 10000.0)
        assert np.max(np.abs(o - o_full[l])) < 1e-12
        assert np.max(np.abs(kc2 - kc_full)) < 1e-12 and np.array_equal(vc2, vc_full)


def test_decode_step_closed_forms():
    """All cached values equal to the new value: the output is that value whatever the scores; an
    empty history cannot exist (l >= 1), but l = 1 with identical keys gives the mean of two values."""
    rng = np.random.default_rng(12)
    hq, hkv, d, l = 4, 2, 16, 9
    row = rng.standard_normal((hkv, d))
    kc = rng.standard_normal((hkv, l, d))
    vc = np.repeat(row[:, None, :], l, axis=1)
    o, _, _ = orc.decode_step(rng.standard_normal((hq, d)), rng.standard_normal((hkv, d)), row, kc, vc, 5e5)
    assert np.max(np.abs(o - np.repeat(row, hq // hkv, axis=0))) < 1e-12
    # a zero query gives uniform weights over the l + 1 positions
    vc = rng.standard_normal((hkv, l, d))
    v_new = rng.standard_normal((hkv, d))
    o, _, v_all = orc.decode_step(np.zeros((hq, d)), rng.standard_normal((hkv, d)), v_new, kc, vc, 5e5)
    assert np.max(np.abs(o - np.repeat(v_all.mean(axis=1), hq // hkv, axis=0))) < 1e-12
