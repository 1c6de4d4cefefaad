"""Element-by-element parity (GPU against the float64 oracle) of the attention kernel variants and
unpack paths that the five workloads do not reach, each case pinned to the variant it selects.

The attention kernel is compiled four times, attention_kernel<D, kIndep> for D in {64, 128} and
kIndep in {false, true}; the host scheduler picks kIndep from the packing (mean key tiles per query
tile) and, in the shared-stream mode (kIndep = false), pairs either two query heads of one KV head
(even GQA group) or two consecutive row tiles of one head (odd group). Each case below states the
variant and pairing it must select; the test recomputes that choice from the rule and also asks the
library (pp_prefill_schedule_info), so a case cannot silently drift to another variant.

case                         D    group  variant                    pairing       what it adds
[3000,1500,700]    2/2       64   1      <64,false>                 row tiles     D=64 shared-stream (4-stage rings, N=64 P.V)
[3000,1500,700]    4/1       64   4      <64,false>                 head pairs    the same with two heads per item
[2500,1300,129]    2/2       128  1      <128,false>                row tiles     slot 1 joins the key stream late (jb1 > 0)
[2432,640]         2/2       128  1      <128,false>                row tiles     odd tile counts: unpaired last row tile
[2500,1300,129]    3/1       64   3      <64,false>                 row tiles     odd group > 1, late join, D=64
[2432,640]         3/1       64   3      <64,false>                 row tiles     odd group > 1, unpaired tile, D=64
Padded mode declares every prompt as long as the longest, so these cases stay in the shared-stream
mode there as well (asserted)."""
import numpy as np
import pytest
import torch

import paper_2404_09529_b200 as pp
from parity_utils import compare_with_refs, expected_schedule, oracle_refs, run_cuda
from paper_2404_09529_b200.runner import DecodeBatch, PrefillBatch
from workloads import split_by_prompt

pytestmark = pytest.mark.gpu


def _case(lengths, hq, hkv, d, seed):
    g = torch.Generator().manual_seed(seed)
    t = int(np.sum(lengths))
    mk = lambda h: torch.randn((t, h, d), generator=g).to(torch.bfloat16)
    return mk(hq), mk(hkv), mk(hkv)


def _assert_schedule(batch, hq, hkv, want_mode, want_pairing, unpaired=None, late=None):
    pk = batch.pack
    seg_bins = [[int(x) for x in pk.seg_len[pk.bin_seg_ptr[b]:pk.bin_seg_ptr[b + 1]]] for b in range(pk.n_bins)]
    assert expected_schedule(seg_bins, hq, hkv) == (want_mode, want_pairing)
    info = pp.pp_prefill_schedule_info(batch.params, pk)
    assert (info["mode"], info["pairing"]) == (want_mode, want_pairing), info
    if unpaired is not None:
        assert (info["unpaired_entries"] > 0) == unpaired, info
    if late is not None:
        assert (info["late_joining_entries"] > 0) == late, info


# lengths, Hq, Hkv, D, pairing (0 = head pairs, 1 = row tiles), unpaired last tile?, late-joining slot?
SHARED_CASES = [
    ([3000, 1500, 700], 2, 2, 64, 1, False, False),
    ([3000, 1500, 700], 4, 1, 64, 0, False, False),
    ([2500, 1300, 129], 2, 2, 128, 1, False, True),
    ([2432, 640], 2, 2, 128, 1, True, False),
    ([2500, 1300, 129], 3, 1, 64, 1, False, True),
    ([2432, 640], 3, 1, 64, 1, True, False),
]


@pytest.mark.parametrize("lengths,hq,hkv,d,pairing,unpaired,late", SHARED_CASES)
def test_shared_stream_variants_full_parity(lengths, hq, hkv, d, pairing, unpaired, late):
    lengths = np.asarray(lengths, np.int32)
    base = 500000.0
    q, k, v = _case(lengths, hq, hkv, d, seed=int(lengths.sum()) + d + hq)
    refs = oracle_refs(lengths, q, k, v, base)
    for mode in ("packed", "padded"):
        for fused in (False, True):
            b = run_cuda(lengths, q, k, v, hq, hkv, d, base, mode, fused=fused, guard=True)
            if mode == "packed":
                _assert_schedule(b, hq, hkv, 0, pairing, unpaired, late)
            else:
                _assert_schedule(b, hq, hkv, 0, pairing)
            compare_with_refs(b, lengths, refs)


# lengths, Hq, Hkv, D, query heads folded into a query tile (independent mode: the largest of 8, 4, 2
# that divides the GQA group; 1 = MHA or an odd group)
FOLD_CASES = [
    ([129, 1, 1, 127, 40, 3], 2, 1, 64, 2),
    ([300, 5, 129, 64, 1, 250, 33, 8, 8, 8, 90, 2], 8, 2, 128, 4),
    ([515, 130, 129, 128, 64, 33, 17, 9, 3, 2, 1], 8, 1, 64, 8),
    ([8] * 40 + [31, 33, 65], 16, 1, 128, 8),                  # group 16: two folds of 8 per KV head
    ([200, 77, 130, 31, 12], 6, 2, 64, 1),                     # group 3: no fold
    ([200, 77, 130, 31, 12], 12, 2, 128, 2),                   # group 6: folds of 2
]


@pytest.mark.parametrize("lengths,hq,hkv,d,fold", FOLD_CASES)
def test_head_folding_variants_full_parity(lengths, hq, hkv, d, fold):
    """Independent mode with GQA: the query tile is 128 / fold bin rows x fold heads. Every fold the
    scheduler can choose, both batch modes, both routes, guard regions around every output."""
    lengths = np.asarray(lengths, np.int32)
    base = 10000.0
    q, k, v = _case(lengths, hq, hkv, d, seed=hq * 100 + d)
    refs = oracle_refs(lengths, q, k, v, base)
    for mode in ("packed", "padded"):
        for fused in (False, True):
            b = run_cuda(lengths, q, k, v, hq, hkv, d, base, mode, fused=fused, guard=True)
            info = pp.pp_prefill_schedule_info(b.params, b.pack)
            assert info["mode"] == 1 and info["heads_folded"] == fold, info
            compare_with_refs(b, lengths, refs)


@pytest.mark.parametrize("room", [1, 7, 64])
@pytest.mark.parametrize("lengths,hq,hkv,d", [
    ([112, 87, 73, 46, 50, 20, 24, 17], 4, 4, 64),          # several prompts per bin, independent mode
    ([300, 5, 129, 64, 1, 250, 33, 8, 8, 8, 90, 2], 8, 2, 128),
])
def test_caches_with_spare_rows_and_guards(lengths, hq, hkv, d, room):
    """cache_cap = length + room: UNPACK writes rows [0, length) of every cache block and nothing
    else. The pools are pre-filled with a sentinel and every output buffer sits between sentinel
    guard regions; spare rows and guards must come back bit-unchanged from pp_unpack_kv, from
    pp_prefill_fused and from pp_unpack_kv_static, and the filled rows must match the oracle."""
    lengths = np.asarray(lengths, np.int32)
    base = 10000.0
    q, k, v = _case(lengths, hq, hkv, d, seed=room)
    refs = oracle_refs(lengths, q, k, v, base)
    rooms = room if room != 7 else (np.arange(len(lengths)) % 3 * 7 + 1).astype(np.int32)   # mixed spare rows
    for mode in ("packed", "padded"):
        three = run_cuda(lengths, q, k, v, hq, hkv, d, base, mode, fused=False, room=rooms, guard=True)
        compare_with_refs(three, lengths, refs)
        fused = run_cuda(lengths, q, k, v, hq, hkv, d, base, mode, fused=True, room=rooms, guard=True)
        compare_with_refs(fused, lengths, refs)
        assert torch.equal(three.k_cache, fused.k_cache) and torch.equal(three.v_cache, fused.v_cache)
        # the entry point without a workspace, on the same packed tensors, into fresh sentinel pools
        st = PrefillBatch(lengths, hq, hkv, d, base, mode=mode, room=rooms, guard=True)
        pp.pp_unpack_kv_static(three.params, three.bin_of, three.off_of, three.lengths, three.kk, three.v,
                               st.k_cache, st.v_cache, st.cache_off, st.cache_cap,
                               torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        st.assert_untouched()
        assert torch.equal(st.k_cache, three.k_cache) and torch.equal(st.v_cache, three.v_cache)


def test_prefill_with_room_then_decode_on_the_same_caches():
    """The hand-over of Section 7: UNPACK fills cache blocks that have room to grow, and the decode
    step appends to and reads those very blocks (no copy in between)."""
    from oracle import prepack_oracle as orc
    from parity_utils import MAX_ABS_TOL, MEAN_ABS_TOL, to64
    lengths = np.array([300, 17, 255, 256, 257, 64], np.int32)
    hq, hkv, d, base, n_steps = 8, 2, 128, 500000.0, 3
    q, k, v = _case(lengths, hq, hkv, d, seed=31)
    refs = oracle_refs(lengths, q, k, v, base)
    pre = run_cuda(lengths, q, k, v, hq, hkv, d, base, fused=True, room=n_steps + 2, guard=True)
    compare_with_refs(pre, lengths, refs)
    dec = DecodeBatch.from_prefill(pre)
    kc, vc = [r[1] for r in refs], [r[2] for r in refs]
    g = torch.Generator().manual_seed(77)
    for step in range(n_steps):
        qn, kn, vn = (torch.randn(len(lengths), h, d, generator=g).to(torch.bfloat16) for h in (hq, hkv, hkv))
        got = to64(dec.step(qn.cuda(), kn.cuda(), vn.cuda()))
        torch.cuda.synchronize()
        errs = []
        for i in range(len(lengths)):
            o_ref, kc[i], vc[i] = orc.decode_step(to64(qn[i]), to64(kn[i]), to64(vn[i]), kc[i], vc[i], base)
            errs.append(np.abs(got[i] - o_ref).ravel())
            l = int(lengths[i]) + step + 1
            ck, cv = dec.caches(i)
            assert np.max(np.abs(to64(ck[:, :l]) - kc[i])) <= MAX_ABS_TOL
            assert np.array_equal(to64(cv[:, :l]), vc[i])
            assert bool((ck[:, l:] == PrefillBatch.SENTINEL).all()) and bool((cv[:, l:] == PrefillBatch.SENTINEL).all())
        e = np.concatenate(errs)
        assert e.max() <= MAX_ABS_TOL and e.mean() <= MEAN_ABS_TOL, (step, e.max(), e.mean())


def test_unknown_flag_bits_are_rejected():
    lengths = np.array([40, 9], np.int32)
    b = PrefillBatch(lengths, 2, 2, 64, 10000.0)
    for bad in (0x100, 0x200, 0x8, 1 << 20):
        with pytest.raises(pp.PrepackError) as err:
            b.run(flags=bad)
        assert err.value.status == -1
        with pytest.raises(pp.PrepackError):
            b.run_fused(flags=bad)
    torch.cuda.synchronize()


def test_keep_rope_table_flag_gives_identical_results():
    lengths = np.array([700, 300, 250, 150, 90, 5, 5], np.int32)
    q, k, v = _case(lengths, 8, 2, 128, seed=3)
    b = PrefillBatch(lengths, 8, 2, 128, 500000.0)
    b.load(q, k, v)
    b.run_fused()
    torch.cuda.synchronize()
    ref = (b.o_tokens().clone(), b.k_cache.clone(), b.v_cache.clone())
    b.load(q, k, v)
    b.k_cache.zero_(); b.v_cache.zero_(); b.o.zero_()
    b.run_fused(flags=pp.PP_FLAG_KEEP_ROPE_TABLE)
    torch.cuda.synchronize()
    assert b.device_status() == 0
    for a, c in zip(ref, (b.o_tokens(), b.k_cache, b.v_cache)):
        assert torch.equal(a, c)
