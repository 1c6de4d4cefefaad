"""pp_unpack_kv_static: the unpack scatter for callers that may not allocate device memory (a
serving loop with a frozen memory pool, a plug-in without an allocator). Its per-prompt table
sits in a fixed device array inside the library, so this file checks that the result is the packed
source rows, bit for bit and nothing else written, and the same as pp_unpack_kv gives, twice in a
row with different batches (the table keeps the previous call's contents), and that a batch beyond
the built-in limit is refused. Collected last on purpose."""
import numpy as np
import pytest
import torch

import paper_2404_09529_b200 as pp


def test_static_unpack_rejects_more_prompts_than_its_table_holds():
    kmax = pp.pp_unpack_static_max_prompts()
    assert kmax == 4096
    k = kmax + 1
    params = pp.AttnParams(4, 4, 64, 10000.0, 0.0, 8, k, 0)
    ones = np.ones(k, np.int32)
    with pytest.raises(pp.PrepackError) as err:
        pp.pp_unpack_kv_static(params, np.arange(k), np.zeros(k), ones, 0x1000, 0x1000, 0x1000, 0x1000,
                               np.arange(k) * 256, ones)
    assert err.value.status == -9
    assert "built-in scratch" in pp.pp_strerror(-9)


def _expected_pools(b, fill):
    """What UNPACK must leave in the cache pools, taken straight from the packed source rows:
    cache[i][h][p] = packed[bin_of[i], off_of[i] + p, h] for p < lengths[i]; everything else keeps
    `fill`. A row permutation done with torch indexing, no library call."""
    out = []
    for packed, pool in ((b.kk, b.k_cache), (b.v, b.v_cache)):
        want = torch.full_like(pool, fill)
        for i in range(b.k):
            l, cap = int(b.lengths[i]), int(b.cache_cap[i])
            rows = packed[int(b.bin_of[i]), int(b.off_of[i]):int(b.off_of[i]) + l]        # [l, Hkv, D]
            off = int(b.cache_off[i])
            want[off:off + b.hkv * cap * b.d].view(b.hkv, cap, b.d)[:, :l] = rows.permute(1, 0, 2)
        out.append(want)
    return out


@pytest.mark.gpu
def test_static_unpack_matches_source_rows_and_workspace_unpack_twice_in_a_row():
    from paper_2404_09529_b200.runner import PrefillBatch
    stream = torch.cuda.current_stream().cuda_stream
    # two calls in a row with different batches and shapes (the built-in table keeps the previous
    # call's contents); the second has spare rows behind every prompt's cache block
    cases = [([112, 87, 73, 46, 50, 20, 24, 17], 4, 4, 64, 0),
             ([300, 5, 129, 64, 1, 250, 33, 8, 8, 8, 90, 2], 8, 2, 128, 5)]
    for lengths, hq, hkv, d, room in cases:
        g = torch.Generator().manual_seed(len(lengths))
        t = int(np.sum(lengths))
        q, k, v = (torch.randn((t, h, d), generator=g).to(torch.bfloat16) for h in (hq, hkv, hkv))
        b = PrefillBatch(lengths, hq, hkv, d, 10000.0, room=room)
        b.load(q, k, v)
        b.k_cache.fill_(7.0); b.v_cache.fill_(7.0)
        b.run()                                   # rotary + attention + pp_unpack_kv (workspace version)
        torch.cuda.synchronize()
        want_k, want_v = _expected_pools(b, 7.0)
        assert float(want_k.float().abs().sum()) > 0
        got_k = torch.full_like(want_k, 7.0)
        got_v = torch.full_like(want_v, 7.0)
        pp.pp_unpack_kv_static(b.params, b.bin_of, b.off_of, b.lengths, b.kk, b.v, got_k, got_v,
                               b.cache_off, b.cache_cap, stream)
        torch.cuda.synchronize()
        # pure copy: bit exact against the source rows, spare rows untouched, and the same as pp_unpack_kv
        assert torch.equal(got_k, want_k) and torch.equal(got_v, want_v)
        assert torch.equal(got_k, b.k_cache) and torch.equal(got_v, b.v_cache)
