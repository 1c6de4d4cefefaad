"""Generation step over the per-prompt caches (pp_decode_step) against the float64 oracle."""
import numpy as np
import pytest
import torch

from oracle import prepack_oracle as orc
from parity_utils import MAX_ABS_TOL, MEAN_ABS_TOL, to64
from workloads import split_by_prompt

pytestmark = pytest.mark.gpu


def _case(lengths, hq, hkv, d, seed):
    g = torch.Generator().manual_seed(seed)
    t = int(np.sum(lengths))
    mk = lambda h: torch.randn(t, h, d, generator=g).to(torch.bfloat16)
    return mk(hq), mk(hkv), mk(hkv)


@pytest.mark.parametrize("lengths,hq,hkv,d,base", [
    (np.array([1, 1, 1, 1000, 1, 1, 1, 1, 1, 1], np.int32), 8, 8, 128, 10000.0),   # the paper's toy mix
    (np.array([300, 17, 255, 256, 257, 64], np.int32), 8, 2, 128, 500000.0),
    (np.array([40, 9, 513], np.int32), 4, 4, 64, 10000.0),
    # enough (chunk, KV head) pairs for the 256-key chunks (smaller batches run 64-key chunks)
    (np.array([255, 256, 257, 511, 512, 513, 767, 768, 300, 64, 1000, 129] * 4, np.int32), 16, 16, 64, 10000.0),
])
def test_decode_steps_match_oracle(lengths, hq, hkv, d, base):
    from paper_2404_09529_b200.runner import DecodeBatch, PrefillBatch
    n_steps = 3
    q, k, v = _case(lengths, hq, hkv, d, seed=21)
    pre = PrefillBatch(lengths, hq, hkv, d, base)
    pre.load(q, k, v)
    pre.run_fused()
    torch.cuda.synchronize()
    assert pre.device_status() == 0
    dec = DecodeBatch(lengths, hq, hkv, d, base, room=n_steps + 1)
    dec.adopt(pre)
    # oracle state: caches of every prompt alone
    qs, ks, vs = (split_by_prompt(x, lengths) for x in (q, k, v))
    ref = [orc.prefill_prompt(to64(a), to64(b), to64(c), base) for a, b, c in zip(qs, ks, vs)]
    kc = [r[1] for r in ref]
    vc = [r[2] for r in ref]
    g = torch.Generator().manual_seed(99)
    for step in range(n_steps):
        qn = torch.randn(len(lengths), hq, d, generator=g).to(torch.bfloat16)
        kn = torch.randn(len(lengths), hkv, d, generator=g).to(torch.bfloat16)
        vn = torch.randn(len(lengths), hkv, d, generator=g).to(torch.bfloat16)
        o = dec.step(qn.cuda(), kn.cuda(), vn.cuda())
        torch.cuda.synchronize()
        got = to64(o)
        errs = []
        for i in range(len(lengths)):
            o_ref, kc[i], vc[i] = orc.decode_step(to64(qn[i]), to64(kn[i]), to64(vn[i]), kc[i], vc[i], base)
            errs.append(np.abs(got[i] - o_ref))
            l = int(lengths[i]) + step + 1
            ck, cv = dec.caches(i)
            assert np.max(np.abs(to64(ck[:, :l]) - kc[i])) <= MAX_ABS_TOL       # rotated keys, bf16-rounded
            assert np.array_equal(to64(cv[:, :l]), vc[i])                       # values are copied bit for bit
        e = np.concatenate([x.ravel() for x in errs])
        assert e.max() <= MAX_ABS_TOL and e.mean() <= MEAN_ABS_TOL, (step, e.max(), e.mean())


def test_decode_argument_checks():
    import paper_2404_09529_b200 as pp
    params = pp.AttnParams(4, 4, 64, 10000.0, 0.0, 1, 1, 0)
    lengths = np.array([5, 3], np.int32)
    nb = pp.pp_decode_workspace_bytes(params, lengths)
    assert nb > 0
    ws = torch.empty(nb, dtype=torch.uint8, device="cuda")
    host = torch.empty(nb, dtype=torch.uint8).pin_memory()
    x = torch.zeros(2, 4, 64, dtype=torch.bfloat16, device="cuda")
    cache = torch.zeros(2 * 4 * 8 * 64, dtype=torch.bfloat16, device="cuda")
    off = np.array([0, 4 * 8 * 64], np.int64)
    with pytest.raises(pp.PrepackError):       # no room for the new token of prompt 0
        pp.pp_decode_step(params, lengths, x, x, x, x.clone(), cache, cache.clone(), off, np.array([5, 8], np.int32),
                          ws, host, nb)
    with pytest.raises(pp.PrepackError):       # workspace too small
        pp.pp_decode_step(params, lengths, x, x, x, x.clone(), cache, cache.clone(), off, np.array([8, 8], np.int32),
                          ws, host, 16)
