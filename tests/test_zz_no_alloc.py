"""pp_unpack_kv_static: the unpack scatter for callers that may not allocate device memory (a
serving loop with a frozen memory pool, a plug-in without an allocator). Its per-prompt table
sits in a fixed device array inside the library, so this file checks that the result is the one
pp_unpack_kv gives, twice in a row with different batches (the table keeps the previous call's
contents), and that a batch beyond the built-in limit is refused. Collected last on purpose."""
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


@pytest.mark.gpu
def test_static_unpack_matches_workspace_unpack_twice_in_a_row():
    from paper_2404_09529_b200.runner import PrefillBatch
    stream = torch.cuda.current_stream().cuda_stream
    cases = [([112, 87, 73, 46, 50, 20, 24, 17], 4, 4, 64),
             ([300, 5, 129, 64, 1, 250, 33, 8, 8, 8, 90, 2], 8, 2, 128)]   # more prompts, other shape
    for lengths, hq, hkv, d in cases:
        g = torch.Generator().manual_seed(len(lengths))
        t = int(np.sum(lengths))
        q, k, v = (torch.randn((t, h, d), generator=g).to(torch.bfloat16) for h in (hq, hkv, hkv))
        b = PrefillBatch(lengths, hq, hkv, d, 10000.0)
        b.load(q, k, v)
        b.run()                                   # rotary + attention + pp_unpack_kv (workspace version)
        torch.cuda.synchronize()
        expect_k, expect_v = b.k_cache.clone(), b.v_cache.clone()
        assert float(expect_k.float().abs().sum()) > 0
        got_k = torch.full_like(expect_k, 7.0)
        got_v = torch.full_like(expect_v, 7.0)
        pp.pp_unpack_kv_static(b.params, b.bin_of, b.off_of, b.lengths, b.kk, b.v, got_k, got_v,
                               b.cache_off, b.cache_cap, stream)
        torch.cuda.synchronize()
        assert torch.equal(got_k, expect_k) and torch.equal(got_v, expect_v)   # pure copy: bit exact
