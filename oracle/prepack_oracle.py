"""CPU oracle for prepacked prefill attention -- TEST INFRASTRUCTURE ONLY.

This file is a plain, slow, float64 statement of what the prefill hot path of
"prepacking" computes. It is imported only by tests, by the smoke check and by
the benchmark's CPU-baseline leg; the CUDA library never touches it and shares
no code, table or helper with it.

What is computed, and where the paper fixes it:

* Section 3.3 states that prepacking yields exactly the KV caches (and hence the
  attention outputs) of a padded full batch; packing is only a cheaper route.
  The oracle therefore never packs in its main entry point: ``prefill_prompt``
  runs one prompt alone with positions 0..l-1 (Section 3.2, restart positional
  encoding = "the same as in the unpacked prompt") and the ordinary causal mask
  (Section 2.1; M[i, j] = 1 iff i >= j, Section 3.2).
* Section 2.1 gives attention as softmax(Q K^T / sqrt(d)) V. The readings taken
  where the paper is loose: the scale is 1/sqrt(head_dim); attention is per head
  and query head h reads KV head h // (Hq // Hkv); the positional encoding is
  rotary in the "rotate-half" pairing (j, j + D/2) with theta_j = base^(-2j/D);
  the cache of one layer is K after the rotation and V unrotated.
* ``ffd_pack`` is textbook first-fit-decreasing (Section 3.1, Algorithm 1 (BINPACK))
  with the tie rules spelled out in its docstring.
* ``restart_position_ids`` / ``independent_mask`` / ``packed_dense_prefill`` spell
  out Algorithm 1 (TENSORIZE to UNPACK) on dense tensors (TENSORIZE, INDEPENDENT-MASK,
  RESTART-PE, UNPACK); ``padded_prefill`` is the full-batching baseline of
  Section 4.2. They exist so that tests can check the paper's exactness claim
  against ``prefill_prompt``.
* ``brute_force_prompt`` is a pure-Python loop version for tiny inputs.
* ``decode_step`` is one generation step over a prompt's own caches (Section 7,
  prepacking for generation): the new token at position l, appended and attended.

Parity pins (tests/test_oracle_pins.py): complex-number form of the rotation,
torch SDPA in float64, closed forms (identical keys, identical values, first
row), packed == padded == alone, zero cross-prompt probability mass, brute force,
the hand-worked packing of the tiny workload, and decode step == last row of the
extended prompt's prefill. No function is unpinned.

All floating point here is float64. Inputs are expected to be bf16-representable
values already upcast to float64 by the caller.
"""
from __future__ import annotations

import math

import numpy as np

# --------------------------------------------------------------------------- #
# Rotary positional encoding (rotate-half pairing)
# --------------------------------------------------------------------------- #


def rope_frequencies(head_dim: int, base: float) -> np.ndarray:
    """theta_j = base^(-2j/D) for j in [0, D/2)."""
    j = np.arange(head_dim // 2, dtype=np.float64)
    return np.power(np.float64(base), -2.0 * j / np.float64(head_dim))


def rope_rotate(x: np.ndarray, positions: np.ndarray, base: float) -> np.ndarray:
    """Rotate x [l, H, D] (float64) by the angles positions[t] * theta_j.

    out[..., j]       = x[..., j] * cos - x[..., j + D/2] * sin
    out[..., j + D/2] = x[..., j + D/2] * cos + x[..., j] * sin
    """
    x = np.asarray(x, dtype=np.float64)
    half = x.shape[-1] // 2
    theta = rope_frequencies(x.shape[-1], base)
    ang = np.asarray(positions, dtype=np.float64)[:, None] * theta[None, :]   # [l, D/2]
    c = np.cos(ang)[:, None, :]
    s = np.sin(ang)[:, None, :]
    lo, hi = x[..., :half], x[..., half:]
    return np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)


# --------------------------------------------------------------------------- #
# One prompt alone: the definition of the result (Sections 2.1, 3.2, 3.3)
# --------------------------------------------------------------------------- #


def _softmax_rows(s: np.ndarray) -> np.ndarray:
    m = np.max(s, axis=-1, keepdims=True)
    e = np.exp(s - m)
    return e / np.sum(e, axis=-1, keepdims=True)


def prefill_prompt(q, k, v, base: float, rows=None, q_heads=None, row_block: int = 1024):
    """Causal self-attention of ONE prompt, alone, positions 0..l-1.

    q [l, Hq, D], k, v [l, Hkv, D] float64 (pre-rotation). Returns
      o       [n_rows, n_heads, D]  attention output for the requested query rows/heads
      k_cache [Hkv, l, D]           rotated keys
      v_cache [Hkv, l, D]           values, unrotated
    ``rows`` (default all) selects query rows; ``q_heads`` (default all) query heads.
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    l, n_q_heads, d = q.shape
    n_kv_heads = k.shape[1]
    group = n_q_heads // n_kv_heads
    pos = np.arange(l)
    q_rot = rope_rotate(q, pos, base)
    k_rot = rope_rotate(k, pos, base)
    rows = np.arange(l) if rows is None else np.asarray(rows, dtype=np.int64)
    heads = list(range(n_q_heads)) if q_heads is None else list(q_heads)
    scale = 1.0 / math.sqrt(d)
    o = np.empty((len(rows), len(heads), d), dtype=np.float64)
    for hi, h in enumerate(heads):
        kv = h // group
        kh = k_rot[:, kv, :]                      # [l, D]
        vh = v[:, kv, :]
        for r0 in range(0, len(rows), row_block):
            rr = rows[r0:r0 + row_block]
            s = (q_rot[rr, h, :] @ kh.T) * scale  # [nr, l]
            s = np.where(np.arange(l)[None, :] <= rr[:, None], s, -np.inf)
            o[r0:r0 + len(rr), hi, :] = _softmax_rows(s) @ vh
    k_cache = np.ascontiguousarray(np.transpose(k_rot, (1, 0, 2)))
    v_cache = np.ascontiguousarray(np.transpose(v, (1, 0, 2)))
    return o, k_cache, v_cache


def prefill_batch(qs, ks, vs, base: float):
    """Run every prompt alone; lists in original prompt order."""
    outs = [prefill_prompt(q, k, v, base) for q, k, v in zip(qs, ks, vs)]
    return [o for o, _, _ in outs], [kc for _, kc, _ in outs], [vc for _, _, vc in outs]


def brute_force_prompt(q, k, v, base: float):
    """Same result as ``prefill_prompt`` with pure-Python loops and math.fsum.
    Only for a handful of tokens."""
    l, n_q_heads, d = len(q), len(q[0]), len(q[0][0])
    n_kv_heads = len(k[0])
    group = n_q_heads // n_kv_heads
    half = d // 2

    def rot(vec, p):
        out = [0.0] * d
        for j in range(half):
            ang = p * float(base) ** (-2.0 * j / d)
            c, s = math.cos(ang), math.sin(ang)
            out[j] = vec[j] * c - vec[j + half] * s
            out[j + half] = vec[j + half] * c + vec[j] * s
        return out

    qr = [[rot([float(t) for t in q[a][h]], a) for h in range(n_q_heads)] for a in range(l)]
    kr = [[rot([float(t) for t in k[a][h]], a) for h in range(n_kv_heads)] for a in range(l)]
    o = [[[0.0] * d for _ in range(n_q_heads)] for _ in range(l)]
    for a in range(l):
        for h in range(n_q_heads):
            kv = h // group
            sc = [math.fsum(qr[a][h][t] * kr[b][kv][t] for t in range(d)) / math.sqrt(d)
                  for b in range(a + 1)]
            mx = max(sc)
            e = [math.exp(x - mx) for x in sc]
            z = math.fsum(e)
            for t in range(d):
                o[a][h][t] = math.fsum(e[b] / z * float(v[b][kv][t]) for b in range(a + 1))
    k_cache = [[kr[a][h] for a in range(l)] for h in range(n_kv_heads)]
    return o, k_cache


# --------------------------------------------------------------------------- #
# BINPACK: first-fit-decreasing (Section 3.1; Algorithm 1 (BINPACK))
# --------------------------------------------------------------------------- #


def ffd_pack(lengths, capacity: int = 0):
    """First-fit-decreasing bin packing of prompt lengths.

    Tie rules (the paper names the heuristic only): items are taken by length
    descending, equal lengths by original index ascending; each item goes into the
    lowest-numbered open bin with enough room left, else a new bin is opened; bins
    are numbered in creation order and hold their items in placement order.
    capacity == 0 means the longest prompt (Algorithm 1 (bin size)).

    Returns a dict of int lists:
      n_bins, capacity,
      bin_seg_ptr [r+1]  segments of bin b are bin_seg_ptr[b] .. bin_seg_ptr[b+1]-1
      seg_prompt  [k]    original prompt index of each segment (bin-major)
      seg_start   [k]    bin-local start offset of each segment (the paper's idx)
      seg_len     [k]
      bin_of, off_of [k] inverse map in original prompt order
      bin_used    [r]    occupied rows of each bin
    """
    lengths = [int(x) for x in lengths]
    k = len(lengths)
    if k == 0:
        raise ValueError("no prompts")
    if min(lengths) < 1:
        raise ValueError("prompt length < 1")
    cap = max(lengths) if capacity == 0 else int(capacity)
    if max(lengths) > cap:
        raise ValueError("prompt longer than bin capacity")
    order = sorted(range(k), key=lambda i: (-lengths[i], i))
    bins = []      # list of lists of prompt indices
    loads = []
    for i in order:
        placed = False
        for b in range(len(bins)):
            if loads[b] + lengths[i] <= cap:
                bins[b].append(i)
                loads[b] += lengths[i]
                placed = True
                break
        if not placed:
            bins.append([i])
            loads.append(lengths[i])
    bin_seg_ptr, seg_prompt, seg_start, seg_len = [0], [], [], []
    bin_of, off_of = [0] * k, [0] * k
    for b, items in enumerate(bins):
        off = 0
        for i in items:
            seg_prompt.append(i)
            seg_start.append(off)
            seg_len.append(lengths[i])
            bin_of[i], off_of[i] = b, off
            off += lengths[i]
        bin_seg_ptr.append(len(seg_prompt))
    return dict(n_bins=len(bins), capacity=cap, bin_seg_ptr=bin_seg_ptr, seg_prompt=seg_prompt,
                seg_start=seg_start, seg_len=seg_len, bin_of=bin_of, off_of=off_of,
                bin_used=loads)


# --------------------------------------------------------------------------- #
# Algorithm 1 (TENSORIZE to UNPACK) on dense tensors (cross-check formulations)
# --------------------------------------------------------------------------- #


def restart_position_ids(pack) -> tuple:
    """RESTART-PE: position ids [r, m] restarting at 0 at each segment start, and
    segment ids [r, m] (index into the seg_* arrays). Tail padding: position 0, id -1."""
    r, m = pack["n_bins"], pack["capacity"]
    pos = np.zeros((r, m), dtype=np.int32)
    seg = np.full((r, m), -1, dtype=np.int32)
    for b in range(r):
        for s in range(pack["bin_seg_ptr"][b], pack["bin_seg_ptr"][b + 1]):
            a, n = pack["seg_start"][s], pack["seg_len"][s]
            pos[b, a:a + n] = np.arange(n)
            seg[b, a:a + n] = s
    return pos, seg


def independent_mask(pack, b: int) -> np.ndarray:
    """INDEPENDENT-MASK of bin b: M'[a:e, a:e] = lower-triangular ones for every
    prompt span [a, e) of the bin; zero elsewhere (Section 3.2)."""
    m = pack["capacity"]
    mask = np.zeros((m, m), dtype=bool)
    for s in range(pack["bin_seg_ptr"][b], pack["bin_seg_ptr"][b + 1]):
        a, n = pack["seg_start"][s], pack["seg_len"][s]
        mask[a:a + n, a:a + n] = np.tril(np.ones((n, n), dtype=bool))
    return mask


def tensorize(xs, pack) -> np.ndarray:
    """TENSORIZE: per-prompt arrays [l_i, H, D] -> dense [r, m, H, D], tail zero-padded."""
    r, m = pack["n_bins"], pack["capacity"]
    out = np.zeros((r, m) + tuple(xs[0].shape[1:]), dtype=np.float64)
    for i, x in enumerate(xs):
        b, off = pack["bin_of"][i], pack["off_of"][i]
        out[b, off:off + x.shape[0]] = x
    return out


def _dense_masked_attention(q_rot, k_rot, v, mask, return_probs=False):
    """q_rot [m, Hq, D], k_rot, v [m, Hkv, D], mask [m, m] bool; rows with an empty
    mask (padding) give zeros."""
    m, n_q_heads, d = q_rot.shape
    group = n_q_heads // k_rot.shape[1]
    o = np.zeros((m, n_q_heads, d), dtype=np.float64)
    probs = np.zeros((n_q_heads, m, m), dtype=np.float64)
    live = mask.any(axis=1)
    for h in range(n_q_heads):
        kv = h // group
        s = (q_rot[:, h, :] @ k_rot[:, kv, :].T) / math.sqrt(d)
        s = np.where(mask, s, -np.inf)
        p = np.zeros((m, m), dtype=np.float64)
        p[live] = _softmax_rows(s[live])
        o[:, h, :] = p @ v[:, kv, :]
        probs[h] = p
    return (o, probs) if return_probs else o


def packed_dense_prefill(qs, ks, vs, base: float, capacity: int = 0, return_probs=False):
    """Algorithm 1 with dense masks: pack, tensorize, independent mask, restart
    positions, attention per bin, unpack to original prompt order."""
    lengths = [x.shape[0] for x in qs]
    pack = ffd_pack(lengths, capacity)
    pos, _ = restart_position_ids(pack)
    qb, kb, vb = tensorize(qs, pack), tensorize(ks, pack), tensorize(vs, pack)
    o_b, kc_b, probs = [], [], []
    for b in range(pack["n_bins"]):
        q_rot = rope_rotate(qb[b], pos[b], base)
        k_rot = rope_rotate(kb[b], pos[b], base)
        res = _dense_masked_attention(q_rot, k_rot, vb[b], independent_mask(pack, b),
                                      return_probs)
        if return_probs:
            o_b.append(res[0])
            probs.append(res[1])
        else:
            o_b.append(res)
        kc_b.append(k_rot)
    os_, kcs, vcs = [], [], []
    for i, l in enumerate(lengths):                     # UNPACK, original order
        b, off = pack["bin_of"][i], pack["off_of"][i]
        os_.append(o_b[b][off:off + l])
        kcs.append(np.transpose(kc_b[b][off:off + l], (1, 0, 2)))
        vcs.append(np.transpose(vb[b][off:off + l], (1, 0, 2)))
    if return_probs:
        return os_, kcs, vcs, pack, probs
    return os_, kcs, vcs


def padded_prefill(qs, ks, vs, base: float):
    """Full batching (Section 4.2): right-pad every prompt to m with zeros, positions
    0..m-1, plain causal mask over all m rows, keep the first l_i rows."""
    lengths = [x.shape[0] for x in qs]
    m = max(lengths)
    causal = np.tril(np.ones((m, m), dtype=bool))
    pos = np.arange(m)
    os_, kcs, vcs = [], [], []
    for q, k, v, l in zip(qs, ks, vs, lengths):
        def pad(x):
            out = np.zeros((m,) + x.shape[1:], dtype=np.float64)
            out[:l] = x
            return out
        q_rot = rope_rotate(pad(q), pos, base)
        k_rot = rope_rotate(pad(k), pos, base)
        o = _dense_masked_attention(q_rot, k_rot, pad(v), causal)
        os_.append(o[:l])
        kcs.append(np.transpose(k_rot[:l], (1, 0, 2)))
        vcs.append(np.transpose(pad(v)[:l], (1, 0, 2)))
    return os_, kcs, vcs


# --------------------------------------------------------------------------- #
# One generation step over per-prompt caches (Section 7: prepacking for generation)
# --------------------------------------------------------------------------- #


def decode_step(q_new, k_new, v_new, k_cache, v_cache, base: float):
    """The token that follows a prompt of l tokens, for one prompt alone.

    q_new [Hq, D], k_new, v_new [Hkv, D]: the new token's (unrotated) projections; k_cache
    [Hkv, l, D] holds the rotated keys of positions 0..l-1 and v_cache [Hkv, l, D] the values.
    The new token sits at position l: its query and key are rotated by l * theta_j, key and value
    are appended to the caches, and the query attends to all l + 1 positions (the causal mask of
    the last row of an (l + 1)-token prompt). Returns (o [Hq, D], k_cache' [Hkv, l+1, D],
    v_cache' [Hkv, l+1, D]). Everything float64.
    """
    q_new, k_new, v_new = (np.asarray(x, dtype=np.float64) for x in (q_new, k_new, v_new))
    k_cache, v_cache = np.asarray(k_cache, dtype=np.float64), np.asarray(v_cache, dtype=np.float64)
    hq, d = q_new.shape
    hkv, l, _ = k_cache.shape
    g = hq // hkv
    pos = np.array([l], dtype=np.int64)
    q_rot = rope_rotate(q_new[None], pos, base)[0]             # [Hq, D]
    k_rot = rope_rotate(k_new[None], pos, base)[0]             # [Hkv, D]
    k_all = np.concatenate([k_cache, k_rot[:, None, :]], axis=1)
    v_all = np.concatenate([v_cache, v_new[:, None, :]], axis=1)
    o = np.empty((hq, d), dtype=np.float64)
    scale = 1.0 / math.sqrt(d)
    for h in range(hq):
        s = (k_all[h // g] @ q_rot[h]) * scale                 # [l + 1]
        p = np.exp(s - s.max())
        p /= p.sum()
        o[h] = p @ v_all[h // g]
    return o, k_all, v_all
