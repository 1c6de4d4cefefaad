"""Host-side checks that need no GPU: pp_pack bit-exact against the oracle packer, RESTART-PE
ids, argument validation of every entry point, and that the library exports what pp.h declares."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2404_09529_b200 as pp
from oracle import prepack_oracle as orc
from workloads import CONFIGS, prompt_lengths

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _assert_same_packing(lengths, capacity=0):
    ref = orc.ffd_pack(lengths, capacity)
    got = pp.pp_pack(lengths, capacity)
    assert got.n_bins == ref["n_bins"] and got.capacity == ref["capacity"]
    for name in ("bin_seg_ptr", "seg_prompt", "seg_start", "seg_len", "bin_of", "off_of"):
        assert getattr(got, name).tolist() == ref[name], name
    return ref, got


@pytest.mark.parametrize("name", list(CONFIGS))
def test_pack_matches_oracle_on_workloads(name):
    ref, got = _assert_same_packing(prompt_lengths(name))
    pos_ref, seg_ref = orc.restart_position_ids(ref)
    pos, seg = pp.pp_fill_position_ids(got)
    assert np.array_equal(pos, pos_ref) and np.array_equal(seg, seg_ref)


def test_workload_statistics_match_recipe():
    # T, m and r of the five stored length lists
    expect = {"tiny": (429, 112, 4), "llama2_7b": (17554, 960, 19), "llama3_8b_gqa": (239975, 3991, 61),
              "long_mix": (108169, 22861, 5), "many_short": (44284, 1272, 35)}
    for name, (total, m, r) in expect.items():
        l = prompt_lengths(name)
        p = pp.pp_pack(l)
        assert (int(l.sum()), int(l.max()), p.n_bins) == (total, m, r)
        assert len(l) == CONFIGS[name].n_prompts


def test_pack_fuzz_against_oracle():
    rng = np.random.default_rng(7)
    for trial in range(300):
        k = int(rng.integers(1, 400))
        hi = int(rng.integers(1, 3000))
        lengths = rng.integers(1, hi + 1, size=k)
        if trial % 4 == 0:                      # many ties
            lengths = rng.choice([3, 5, 8, 13, 64], size=k)
        cap = 0 if trial % 3 else int(lengths.max()) + int(rng.integers(0, 100))
        _assert_same_packing(lengths, cap)


def test_pack_large_k():
    rng = np.random.default_rng(11)
    lengths = np.clip(np.floor(8 * (1 - rng.random(4096)) ** (-1 / 1.5)), 8, 8192).astype(np.int32)
    _assert_same_packing(lengths)


def test_padded_mode_packing_is_one_bin_per_prompt():
    p = pp.pp_pack(np.full(7, 50, dtype=np.int32))
    assert p.n_bins == 7 and p.seg_prompt.tolist() == list(range(7)) and p.seg_start.tolist() == [0] * 7


def test_pack_errors():
    lib = pp.load_library()
    n = ctypes.c_int32()
    l = np.array([3, 0, 2], np.int32)
    i32p = ctypes.POINTER(ctypes.c_int32)
    none = ctypes.cast(None, i32p)
    assert lib.pp_pack(l.ctypes.data_as(i32p), 3, 0, ctypes.byref(n), none, none, none, none, none, none, none) == -2
    l = np.array([3, 9], np.int32)
    assert lib.pp_pack(l.ctypes.data_as(i32p), 2, 8, ctypes.byref(n), none, none, none, none, none, none, none) == -2
    assert lib.pp_pack(l.ctypes.data_as(i32p), 0, 0, ctypes.byref(n), none, none, none, none, none, none, none) == -1
    assert lib.pp_pack(none, 2, 0, ctypes.byref(n), none, none, none, none, none, none, none) == -1
    # outputs other than n_bins are optional
    assert lib.pp_pack(l.ctypes.data_as(i32p), 2, 0, ctypes.byref(n), none, none, none, none, none, none, none) == 0
    assert n.value == 2
    assert pp.pp_strerror(-2).startswith("prompt length")
    with pytest.raises(pp.PrepackError):
        pp.pp_pack([4, -1])


def test_library_exports_every_declared_symbol():
    text = open(os.path.join(ROOT, "include", "pp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = set(re.findall(r"\b(pp_[a-z_0-9]+)\s*\(", text))
    assert {"pp_pack", "pp_prefill_attention", "pp_unpack_kv"} <= names
    lib = ctypes.CDLL(pp.lib_path())
    for name in sorted(names):
        assert hasattr(lib, name), name


def _params(**kw):
    base = dict(n_q_heads=4, n_kv_heads=4, head_dim=64, rope_base=10000.0, softmax_scale=0.0,
                capacity=112, n_bins=4, flags=0)
    base.update(kw)
    return pp.AttnParams(**base)


def test_prefill_argument_validation_happens_before_any_device_work():
    """Fake (never dereferenced) addresses: every error below is detected on the host."""
    pack = pp.pp_pack([112, 87, 73, 46, 50, 20, 24, 17])
    ws = pp.pp_prefill_workspace_bytes(_params(), pack.k)
    assert ws > 0
    host = np.zeros(ws, np.uint8)
    A = 0x10000

    def call(params, pack=pack, q=A, k=A, v=A, o=A, w=A, hw=host, wb=ws):
        try:
            pp.pp_prefill_attention(params, pack, q, k, v, o, w, hw, wb)
        except pp.PrepackError as e:
            return e.status
        return 0

    assert call(_params(head_dim=96)) == -4
    assert call(_params(n_q_heads=6, n_kv_heads=4)) == -4
    assert call(_params(), q=A + 8) == -5
    assert call(_params(), w=A + 4) == -5
    assert call(_params(), wb=ws - 4) == -3
    assert call(_params(), q=0) == -1
    assert call(_params(capacity=100)) == -2          # a segment overflows the bin
    assert call(_params(n_bins=3)) == -1              # CSR does not end at k
    bad = pp.pp_pack([112, 87, 73, 46, 50, 20, 24, 17])
    bad.seg_start[2] = 80                             # gap inside a bin
    assert call(_params(), pack=bad) == -1
    assert pp.pp_prefill_workspace_bytes(_params(head_dim=32), 8) == 0
    # flag bits the header does not define (two of them were internal options once) are refused
    for bad in (0x100, 0x200, 0x8, 1 << 30):
        assert call(_params(flags=bad)) == -1
        assert call(_params(flags=bad | pp.PP_FLAG_SKIP_ROPE)) == -1


def test_unpack_argument_validation():
    p = _params(n_bins=2, capacity=10)
    ws = pp.pp_unpack_workspace_bytes(2)
    host = np.zeros(ws, np.uint8)
    A = 0x10000

    def call(bin_of=(0, 1), off_of=(0, 0), lengths=(5, 10), cache_off=(0, 5 * 4 * 64), cache_cap=(5, 10),
             kc=A, wb=ws):
        try:
            pp.pp_unpack_kv(p, bin_of, off_of, lengths, A, A, kc, A, cache_off, cache_cap, A, host, wb)
        except pp.PrepackError as e:
            return e.status
        return 0

    assert call(lengths=(5, 11)) == -2                 # longer than its cache
    assert call(off_of=(6, 0)) == -1                   # runs past the bin
    assert call(bin_of=(0, 2)) == -1
    assert call(cache_off=(0, 4)) == -5
    assert call(kc=A + 2) == -5
    assert call(wb=ws - 1) == -3
    assert call(cache_cap=(4, 10)) == -2


def test_schedule_info_matches_the_scheduling_rule():
    """pp_prefill_schedule_info (host only) against the rule restated in the test helpers, on packings
    around the mode threshold and with odd / even GQA groups."""
    import sys, os
    sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
    from parity_utils import expected_schedule
    rng = np.random.default_rng(7)
    for trial in range(60):
        kind = trial % 3
        if kind == 0:
            lengths = rng.integers(1, 400, size=int(rng.integers(1, 40)))
        elif kind == 1:
            lengths = rng.integers(600, 4000, size=int(rng.integers(1, 6)))
        else:
            lengths = np.concatenate([rng.integers(900, 1400, size=3), rng.integers(1, 50, size=int(rng.integers(0, 30)))])
        hkv = int(rng.choice([1, 2]))
        hq = hkv * int(rng.choice([1, 2, 3, 4]))
        pk = pp.pp_pack(lengths)
        info = pp.pp_prefill_schedule_info(_params(n_q_heads=hq, n_kv_heads=hkv, capacity=pk.capacity, n_bins=pk.n_bins), pk)
        seg_bins = [[int(x) for x in pk.seg_len[pk.bin_seg_ptr[b]:pk.bin_seg_ptr[b + 1]]] for b in range(pk.n_bins)]
        assert (info["mode"], info["pairing"]) == expected_schedule(seg_bins, hq, hkv), (lengths, hq, hkv, info)
        assert info["key_tile_rows"] == (64 if info["mode"] == 1 else 128)
        assert info["entries"] >= pk.n_bins and info["steps"] >= info["entries"]


def test_per_device_once_guard(tmp_path):
    """The record that keeps per-device kernel set-up from running twice (and, above all, from being
    skipped on a second GPU): compiled on its own with the host compiler and driven from two threads."""
    import shutil, subprocess, textwrap
    gxx = shutil.which("g++")
    if gxx is None:
        pytest.skip("no host C++ compiler")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    src = tmp_path / "once.cpp"
    src.write_text(textwrap.dedent("""
        #include "pp_device_once.h"
        #include <cstdio>
        #include <thread>
        int main() {
          pp::DeviceOnce once;
          for (int d = -2; d < 200; ++d) if (once.done(d)) return 1;          // nothing done at start
          once.mark(0);
          if (!once.done(0) || once.done(1) || once.done(63) || once.done(64)) return 2;   // per device
          once.mark(64); once.mark(127);
          if (!once.done(64) || !once.done(127) || once.done(65) || once.done(126)) return 3;
          once.mark(-1); once.mark(128); once.mark(1000);                      // out of range: never recorded
          if (once.done(-1) || once.done(128) || once.done(1000)) return 4;
          pp::DeviceOnce shared;
          std::thread a([&] { for (int d = 0; d < 128; d += 2) shared.mark(d); });
          std::thread b([&] { for (int d = 1; d < 128; d += 2) shared.mark(d); });
          a.join(); b.join();
          for (int d = 0; d < 128; ++d) if (!shared.done(d)) return 5;         // no lost update
          std::puts("ok");
          return 0;
        }
    """))
    exe = tmp_path / "once"
    inc = os.path.join(root, "paper_2404_09529_b200", "csrc")
    subprocess.run([gxx, "-std=c++17", "-O1", "-pthread", "-I", inc, str(src), "-o", str(exe)], check=True)
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0 and out.stdout.strip() == "ok", (out.returncode, out.stdout, out.stderr)
