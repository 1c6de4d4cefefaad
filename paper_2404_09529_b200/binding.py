"""ctypes binding of libprepack_b200.so. Argument marshalling only: no arithmetic of the
method lives here. Function names and argument order follow ``include/pp.h``."""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import numpy as np

_PKG_DIR = os.path.dirname(os.path.abspath(__file__))
_LIB_NAME = "libprepack_b200.so"
_lib = None

PP_FLAG_SKIP_ROPE = 1
PP_FLAG_ROPE_ONLY = 2
PP_FLAG_KEEP_ROPE_TABLE = 4


class PrepackError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        detail = pp_strerror(status)
        cuda = pp_last_cuda_error() if status == -6 else ""
        super().__init__(f"{where}: {detail} (status {status})" + (f" [{cuda}]" if cuda else ""))


class AttnParams(ctypes.Structure):
    """Mirror of ``pp_attn_params``."""
    _fields_ = [("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("rope_base", ctypes.c_float),
                ("softmax_scale", ctypes.c_float), ("capacity", ctypes.c_int32),
                ("n_bins", ctypes.c_int32), ("flags", ctypes.c_int32)]


def lib_path() -> str:
    return os.path.join(_PKG_DIR, _LIB_NAME)


def load_library():
    """Load the shared library. There is no fallback: without it nothing in this package works."""
    global _lib
    if _lib is not None:
        return _lib
    path = lib_path()
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: build it with `python -m paper_2404_09529_b200.build` "
                          "(needs nvcc); prepack-b200 has no CPU or PyTorch fallback")
    lib = ctypes.CDLL(path)
    i32p, i64p, vp = ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int64), ctypes.c_void_p
    pp = ctypes.POINTER(AttnParams)
    sig = {
        "pp_version": (ctypes.c_int, []),
        "pp_strerror": (ctypes.c_char_p, [ctypes.c_int]),
        "pp_last_cuda_error": (ctypes.c_char_p, []),
        "pp_pack": (ctypes.c_int, [i32p, ctypes.c_int32, ctypes.c_int32, i32p, i32p, i32p, i32p, i32p, i32p, i32p, i32p]),
        "pp_fill_position_ids": (ctypes.c_int, [ctypes.c_int32, ctypes.c_int32, i32p, i32p, i32p, i32p, i32p]),
        "pp_prefill_schedule_info": (ctypes.c_int, [pp, i32p, i32p, i32p, ctypes.c_int32, i32p]),
        "pp_prefill_workspace_bytes": (ctypes.c_size_t, [pp, ctypes.c_int32]),
        "pp_prefill_attention": (ctypes.c_int, [pp, i32p, i32p, i32p, ctypes.c_int32, vp, vp, vp, vp, vp, vp,
                                                ctypes.c_size_t, vp, vp]),
        "pp_prefill_fused_workspace_bytes": (ctypes.c_size_t, [pp, ctypes.c_int32]),
        "pp_prefill_fused_host_bytes": (ctypes.c_size_t, [pp, ctypes.c_int32]),
        "pp_prefill_fused": (ctypes.c_int, [pp, i32p, i32p, i32p, i32p, ctypes.c_int32, i32p, vp, vp, vp, vp, vp, vp,
                                            i64p, i32p, vp, vp, ctypes.c_size_t, vp, vp]),
        "pp_selftest_bounded_wait": (ctypes.c_int, [vp, ctypes.c_uint32, vp]),
        "pp_unpack_workspace_bytes": (ctypes.c_size_t, [ctypes.c_int32]),
        "pp_unpack_kv": (ctypes.c_int, [pp, i32p, i32p, i32p, ctypes.c_int32, vp, vp, vp, vp, i64p, i32p, vp, vp,
                                        ctypes.c_size_t, vp]),
        "pp_unpack_static_max_prompts": (ctypes.c_int32, []),
        "pp_unpack_kv_static": (ctypes.c_int, [pp, i32p, i32p, i32p, ctypes.c_int32, vp, vp, vp, vp, i64p, i32p, vp]),
        "pp_decode_workspace_bytes": (ctypes.c_size_t, [pp, i32p, ctypes.c_int32]),
        "pp_decode_step": (ctypes.c_int, [pp, i32p, ctypes.c_int32, vp, vp, vp, vp, vp, vp, i64p, i32p, vp, vp,
                                          ctypes.c_size_t, vp]),
        "pp_prefill_host_arena_bytes": (ctypes.c_size_t, [pp, i32p, ctypes.c_int32]),
        "pp_prefill_host_groups": (ctypes.c_int32, [ctypes.c_int32]),
        "pp_prefill_host": (ctypes.c_int, [pp, i32p, ctypes.c_int32, vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    _lib = lib
    return lib


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _p32(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))


def _addr(x) -> int:
    """Address of a torch tensor / numpy array / raw int."""
    if x is None:
        return 0
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    raise TypeError(type(x))


def _check(status: int, where: str) -> None:
    if status != 0:
        raise PrepackError(status, where)


def pp_version() -> int:
    return load_library().pp_version()


def pp_strerror(status: int) -> str:
    return load_library().pp_strerror(status).decode()


def pp_last_cuda_error() -> str:
    return load_library().pp_last_cuda_error().decode()


@dataclass
class Packing:
    """Output arrays of ``pp_pack`` (numpy int32)."""
    n_bins: int
    capacity: int
    bin_seg_ptr: np.ndarray
    seg_prompt: np.ndarray
    seg_start: np.ndarray
    seg_len: np.ndarray
    bin_of: np.ndarray
    off_of: np.ndarray

    @property
    def k(self) -> int:
        return int(self.seg_start.shape[0])

    def slice_bins(self, b0: int, b1: int):
        """Bins [b0, b1) as a packing of their own (index bookkeeping only). Returns (packing, prompts):
        `prompts` are the original indices of the prompts in those bins, ascending, and the packing's
        seg_prompt / bin_of / off_of refer to positions in that list."""
        s0, s1 = int(self.bin_seg_ptr[b0]), int(self.bin_seg_ptr[b1])
        seg_prompt = self.seg_prompt[s0:s1]
        prompts = np.sort(seg_prompt)
        local = np.searchsorted(prompts, seg_prompt).astype(np.int32)
        return (Packing(b1 - b0, self.capacity, (self.bin_seg_ptr[b0:b1 + 1] - s0).astype(np.int32), local,
                        self.seg_start[s0:s1].copy(), self.seg_len[s0:s1].copy(),
                        (self.bin_of[prompts] - b0).astype(np.int32), self.off_of[prompts].copy()), prompts)


def pp_pack(lengths, capacity: int = 0) -> Packing:
    lib = load_library()
    l = _i32(lengths)
    k = int(l.shape[0])
    n_bins, cap = ctypes.c_int32(0), ctypes.c_int32(0)
    ptr = np.zeros(k + 1, np.int32)
    outs = [np.zeros(max(k, 1), np.int32) for _ in range(5)]
    st = lib.pp_pack(_p32(l), k, capacity, ctypes.byref(n_bins), ctypes.byref(cap), _p32(ptr),
                     *[_p32(o) for o in outs])
    _check(st, "pp_pack")
    return Packing(n_bins.value, cap.value, ptr[:n_bins.value + 1].copy(), *[o[:k] for o in outs])


def pp_fill_position_ids(pack: Packing):
    lib = load_library()
    pos = np.zeros(pack.n_bins * pack.capacity, np.int32)
    seg = np.zeros(pack.n_bins * pack.capacity, np.int32)
    st = lib.pp_fill_position_ids(pack.n_bins, pack.capacity, _p32(pack.bin_seg_ptr), _p32(pack.seg_start),
                                  _p32(pack.seg_len), _p32(pos), _p32(seg))
    _check(st, "pp_fill_position_ids")
    return pos.reshape(pack.n_bins, pack.capacity), seg.reshape(pack.n_bins, pack.capacity)


SCHEDULE_INFO_FIELDS = ("mode", "pairing", "entries", "steps", "key_tile_rows", "unpaired_entries",
                        "late_joining_entries", "heads_folded")


def pp_prefill_schedule_info(params: AttnParams, pack: Packing) -> dict:
    """The tile work list pp_prefill_attention / pp_prefill_fused would build for this packing, as a
    dict keyed by SCHEDULE_INFO_FIELDS (see include/pp.h)."""
    info = np.zeros(8, np.int32)
    st = load_library().pp_prefill_schedule_info(ctypes.byref(params), _p32(pack.bin_seg_ptr),
                                                 _p32(pack.seg_start), _p32(pack.seg_len), pack.k, _p32(info))
    _check(st, "pp_prefill_schedule_info")
    return dict(zip(SCHEDULE_INFO_FIELDS, (int(x) for x in info)))


def pp_prefill_workspace_bytes(params: AttnParams, k: int) -> int:
    return int(load_library().pp_prefill_workspace_bytes(ctypes.byref(params), k))


def pp_prefill_fused_workspace_bytes(params: AttnParams, k: int) -> int:
    return int(load_library().pp_prefill_fused_workspace_bytes(ctypes.byref(params), k))


def pp_prefill_fused_host_bytes(params: AttnParams, k: int) -> int:
    return int(load_library().pp_prefill_fused_host_bytes(ctypes.byref(params), k))


def pp_prefill_fused(params: AttnParams, pack: Packing, lengths, q, k, v, o, k_cache, v_cache, cache_off,
                     cache_cap, workspace, host_workspace, workspace_bytes: int, device_status=None,
                     stream: int = 0) -> None:
    l, cc = _i32(lengths), _i32(cache_cap)
    co = np.ascontiguousarray(np.asarray(cache_off, dtype=np.int64))
    st = load_library().pp_prefill_fused(
        ctypes.byref(params), _p32(pack.bin_seg_ptr), _p32(pack.seg_start), _p32(pack.seg_len),
        _p32(pack.seg_prompt), pack.k, _p32(l), _addr(q), _addr(k), _addr(v), _addr(o), _addr(k_cache),
        _addr(v_cache), co.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), _p32(cc), _addr(workspace),
        _addr(host_workspace), workspace_bytes, _addr(device_status), stream)
    _check(st, "pp_prefill_fused")


def pp_decode_workspace_bytes(params: AttnParams, lengths) -> int:
    l = _i32(lengths)
    return int(load_library().pp_decode_workspace_bytes(ctypes.byref(params), _p32(l), int(l.shape[0])))


def pp_decode_step(params: AttnParams, lengths, q_new, k_new, v_new, o, k_cache, v_cache, cache_off, cache_cap,
                   workspace, host_workspace, workspace_bytes: int, stream: int = 0) -> None:
    l, cc = _i32(lengths), _i32(cache_cap)
    co = np.ascontiguousarray(np.asarray(cache_off, dtype=np.int64))
    st = load_library().pp_decode_step(
        ctypes.byref(params), _p32(l), int(l.shape[0]), _addr(q_new), _addr(k_new), _addr(v_new), _addr(o),
        _addr(k_cache), _addr(v_cache), co.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), _p32(cc),
        _addr(workspace), _addr(host_workspace), workspace_bytes, stream)
    _check(st, "pp_decode_step")


def pp_selftest_bounded_wait(device_status, limit_ms: int, stream: int = 0) -> None:
    _check(load_library().pp_selftest_bounded_wait(_addr(device_status), limit_ms, stream),
           "pp_selftest_bounded_wait")


def pp_unpack_workspace_bytes(k: int) -> int:
    return int(load_library().pp_unpack_workspace_bytes(k))


def pp_prefill_attention(params: AttnParams, pack: Packing, q, k, v, o, workspace, host_workspace,
                         workspace_bytes: int, device_status=None, stream: int = 0) -> None:
    st = load_library().pp_prefill_attention(
        ctypes.byref(params), _p32(pack.bin_seg_ptr), _p32(pack.seg_start), _p32(pack.seg_len), pack.k,
        _addr(q), _addr(k), _addr(v), _addr(o), _addr(workspace), _addr(host_workspace), workspace_bytes,
        _addr(device_status), stream)
    _check(st, "pp_prefill_attention")


def pp_unpack_kv(params: AttnParams, bin_of, off_of, lengths, k_rot, v, k_cache, v_cache, cache_off, cache_cap,
                 workspace, host_workspace, workspace_bytes: int, stream: int = 0) -> None:
    b, o, l, cc = _i32(bin_of), _i32(off_of), _i32(lengths), _i32(cache_cap)
    co = np.ascontiguousarray(np.asarray(cache_off, dtype=np.int64))
    st = load_library().pp_unpack_kv(
        ctypes.byref(params), _p32(b), _p32(o), _p32(l), int(l.shape[0]), _addr(k_rot), _addr(v),
        _addr(k_cache), _addr(v_cache), co.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), _p32(cc),
        _addr(workspace), _addr(host_workspace), workspace_bytes, stream)
    _check(st, "pp_unpack_kv")


def pp_unpack_static_max_prompts() -> int:
    return int(load_library().pp_unpack_static_max_prompts())


def pp_unpack_kv_static(params: AttnParams, bin_of, off_of, lengths, k_rot, v, k_cache, v_cache, cache_off,
                        cache_cap, stream: int = 0) -> None:
    """pp_unpack_kv for callers that cannot allocate: no workspaces, at most
    pp_unpack_static_max_prompts() prompts, one shared table per GPU (see include/pp.h)."""
    b, o, l, cc = _i32(bin_of), _i32(off_of), _i32(lengths), _i32(cache_cap)
    co = np.ascontiguousarray(np.asarray(cache_off, dtype=np.int64))
    st = load_library().pp_unpack_kv_static(
        ctypes.byref(params), _p32(b), _p32(o), _p32(l), int(l.shape[0]), _addr(k_rot), _addr(v),
        _addr(k_cache), _addr(v_cache), co.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), _p32(cc), stream)
    _check(st, "pp_unpack_kv_static")


def pp_prefill_host_arena_bytes(params: AttnParams, lengths) -> int:
    l = _i32(lengths)
    return int(load_library().pp_prefill_host_arena_bytes(ctypes.byref(params), _p32(l), int(l.shape[0])))


def pp_prefill_host_groups(n_groups: int) -> int:
    """Fix the number of pipelined groups of pp_prefill_host for this thread (0 = by batch size);
    returns the previous setting."""
    return int(load_library().pp_prefill_host_groups(n_groups))


def pp_prefill_host(params: AttnParams, lengths, q_host, k_host, v_host, o_host, k_cache_host, v_cache_host,
                    arena, arena_bytes: int, stream: int = 0) -> None:
    l = _i32(lengths)
    st = load_library().pp_prefill_host(
        ctypes.byref(params), _p32(l), int(l.shape[0]), _addr(q_host), _addr(k_host), _addr(v_host),
        _addr(o_host), _addr(k_cache_host), _addr(v_cache_host), _addr(arena), arena_bytes, stream)
    _check(st, "pp_prefill_host")


class Workspaces:
    """Device workspaces plus a small ring of pinned host staging buffers for the two calls that
    upload tables. Memory plumbing only (torch allocations and events); a staging buffer is
    reused only after the copy that read it has completed."""

    def __init__(self, params: AttnParams, k: int, device="cuda", ring: int = 4):
        import torch
        self._torch = torch
        self.attn_bytes = pp_prefill_workspace_bytes(params, k)
        self.unpack_bytes = pp_unpack_workspace_bytes(k)
        if self.attn_bytes == 0 or self.unpack_bytes == 0:
            raise PrepackError(-1, "Workspaces")
        self.fused_bytes = pp_prefill_fused_workspace_bytes(params, k)
        self.fused_dev = torch.empty(self.fused_bytes, dtype=torch.uint8, device=device)
        self.attn_dev = torch.empty(self.attn_bytes, dtype=torch.uint8, device=device)
        self.unpack_dev = torch.empty(self.unpack_bytes, dtype=torch.uint8, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self._fused_host = [torch.empty(pp_prefill_fused_host_bytes(params, k), dtype=torch.uint8).pin_memory()
                            for _ in range(ring)]
        self._ring = [(torch.empty(self.attn_bytes, dtype=torch.uint8).pin_memory(),
                       torch.empty(self.unpack_bytes, dtype=torch.uint8).pin_memory(),
                       torch.cuda.Event()) for _ in range(ring)]
        self._next = 0
        self._used = [False] * ring

    def acquire(self):
        """Next (attn_host, unpack_host, slot); blocks until the slot's previous copies are done."""
        i = self._next
        self._next = (i + 1) % len(self._ring)
        a, u, ev = self._ring[i]
        if self._used[i]:
            ev.synchronize()
        return a, u, i

    def fused_host(self, slot: int):
        return self._fused_host[slot]

    def release(self, slot: int, stream=None) -> None:
        """Record, on the stream the copies were enqueued on, that slot's buffers may be reused after it."""
        self._ring[slot][2].record(stream if stream is not None else self._torch.cuda.current_stream())
        self._used[slot] = True
