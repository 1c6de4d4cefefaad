"""Memory plumbing around the C-ABI calls: lays token-major tensors out as the packed (or padded)
batch, owns the device buffers and workspaces, and calls pp_pack / pp_prefill_attention /
pp_unpack_kv in order. All arithmetic of the method happens inside the library."""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B


class PrefillBatch:
    """One batch of prompts on the device, ready to be prefilled.

    mode "packed": bins from pp_pack(lengths) (first-fit-decreasing, capacity = longest prompt).
    mode "padded": the full-batching baseline -- one bin per prompt in original order, every
    bin declared as a single segment of the full capacity, so all k*m rows are computed;
    unpack still copies only each prompt's true rows.
    mode "varlen": one bin per prompt in original order, each declared with its true length: the
    mask and tile skipping without the bin packing (isolates what packing adds).
    """

    SENTINEL = -1.0e30      # bf16 value that pre-fills guard regions and cache pools (guard=True)

    def __init__(self, lengths, n_q_heads: int, n_kv_heads: int, head_dim: int, rope_base: float,
                 mode: str = "packed", device: str = "cuda", softmax_scale: float = 0.0, room=0,
                 guard: bool = False, pack: "B.Packing | None" = None):
        """room (int or one int per prompt): spare rows in every prompt's cache block, so that
        cache_cap[i] = lengths[i] + room. guard: put sentinel-filled regions in front of and behind
        every buffer the library writes (O, K, both cache pools) and pre-fill the pools with the
        sentinel, so that `assert_untouched` can tell whether anything outside the documented
        outputs was written. pack: a packing made elsewhere (e.g. some bins of a packing of a whole
        stream of prompts, Packing.slice_bins) for exactly these prompts; mode is then "prepacked"."""
        self.device = torch.device(device)
        self.mode = "prepacked" if pack is not None else mode
        self._given_pack = pack
        self.lengths = np.ascontiguousarray(np.asarray(lengths, dtype=np.int32))
        self.k = int(self.lengths.shape[0])
        self.total_tokens = int(self.lengths.sum())
        self.hq, self.hkv, self.d = n_q_heads, n_kv_heads, head_dim
        self.rope_base, self.softmax_scale = rope_base, softmax_scale
        self._pack()
        R, M = self.pack.n_bins, self.pack.capacity
        dev, bf = self.device, torch.bfloat16
        self._guards = []
        self.q = torch.zeros((R, M, n_q_heads, head_dim), dtype=bf, device=dev)
        self.kk = self._alloc((R, M, n_kv_heads, head_dim), guard, 0.0)
        self.v = torch.zeros((R, M, n_kv_heads, head_dim), dtype=bf, device=dev)
        self.o = self._alloc((R, M, n_q_heads, head_dim), guard, 0.0)
        # per-prompt caches, one pool each, [Hkv, cap_i, D] blocks back to back in original order
        self.cache_cap = (self.lengths + np.asarray(room, dtype=np.int32)).astype(np.int32)
        cap_prefix = np.concatenate([[0], np.cumsum(self.cache_cap.astype(np.int64))])
        self.cache_off = (cap_prefix[:-1] * n_kv_heads * head_dim).astype(np.int64)
        pool = int(cap_prefix[-1]) * n_kv_heads * head_dim
        self.k_cache = self._alloc((pool,), guard, self.SENTINEL if guard else 0.0)
        self.v_cache = self._alloc((pool,), guard, self.SENTINEL if guard else 0.0)
        self.ws = B.Workspaces(self.params, self.pack.k, device=dev)
        # flat packed row of every real token, original prompt order
        rows = [np.arange(l, dtype=np.int64) + int(b) * M + int(off)
                for l, b, off in zip(self.lengths, self.bin_of, self.off_of)]
        self.token_rows = torch.from_numpy(np.concatenate(rows)).to(dev)

    def _alloc(self, shape, guard: bool, fill: float) -> torch.Tensor:
        """A device tensor of `shape`; with guard, the middle of a larger sentinel-filled buffer."""
        n = int(np.prod(shape))
        if not guard:
            return torch.full((n,), fill, dtype=torch.bfloat16, device=self.device).view(shape)
        g = 4096                                          # elements: keeps the payload 8 KB aligned
        whole = torch.full((n + 2 * g,), self.SENTINEL, dtype=torch.bfloat16, device=self.device)
        self._guards.append((whole, g, n))
        body = whole[g:g + n]
        body.fill_(fill)
        return body.view(shape)

    def assert_untouched(self) -> None:
        """Guard regions around O, K and the cache pools, and the spare rows [lengths[i], cap[i]) of
        every cache block, still hold the sentinel bit for bit (needs guard=True)."""
        assert self._guards, "PrefillBatch was built without guard=True"
        for whole, g, n in self._guards:
            for part in (whole[:g], whole[g + n:]):
                assert bool((part == self.SENTINEL).all()), "write outside an output buffer"
        for i in range(self.k):
            l = int(self.lengths[i])
            for c in self.caches(i):
                assert bool((c[:, l:] == self.SENTINEL).all()), f"spare cache rows of prompt {i} were written"

    def _pack(self) -> None:
        """BINPACK through the library (host)."""
        if self.mode == "prepacked":
            self.pack = self._given_pack
            self.bin_of, self.off_of = self.pack.bin_of, self.pack.off_of
        elif self.mode == "packed":
            self.pack = B.pp_pack(self.lengths, 0)
            self.bin_of, self.off_of = self.pack.bin_of, self.pack.off_of
        elif self.mode == "padded":
            m = int(self.lengths.max())
            self.pack = B.pp_pack(np.full(self.k, m, dtype=np.int32), 0)
            self.bin_of = np.arange(self.k, dtype=np.int32)
            self.off_of = np.zeros(self.k, dtype=np.int32)
        elif self.mode == "varlen":
            m = int(self.lengths.max())
            ar = np.arange(self.k, dtype=np.int32)
            self.pack = B.Packing(self.k, m, np.arange(self.k + 1, dtype=np.int32), ar.copy(),
                                  np.zeros(self.k, np.int32), self.lengths.copy(), ar.copy(),
                                  np.zeros(self.k, np.int32))
            self.bin_of, self.off_of = self.pack.bin_of, self.pack.off_of
        else:
            raise ValueError(self.mode)
        self.params = B.AttnParams(self.hq, self.hkv, self.d, self.rope_base, self.softmax_scale,
                                   self.pack.capacity, self.pack.n_bins, 0)

    def load(self, q_tok: torch.Tensor, k_tok: torch.Tensor, v_tok: torch.Tensor) -> None:
        """TENSORIZE: scatter token-major [T, H, D] tensors into the packed layout; padding rows zero."""
        for dst, src in ((self.q, q_tok), (self.kk, k_tok), (self.v, v_tok)):
            dst.zero_()
            dst.view(-1, dst.shape[2], dst.shape[3])[self.token_rows] = src.to(self.device)

    def run(self, flags: int = 0, repack: bool = False, unpack: bool = True) -> None:
        """One pass of the hot path on the current stream (asynchronous)."""
        if repack:
            self._pack()
        stream = torch.cuda.current_stream().cuda_stream
        host_attn, host_unpack, slot = self.ws.acquire()
        self.params.flags = flags
        B.pp_prefill_attention(self.params, self.pack, self.q, self.kk, self.v, self.o, self.ws.attn_dev,
                               host_attn, self.ws.attn_bytes, self.ws.status, stream)
        if unpack:
            B.pp_unpack_kv(self.params, self.bin_of, self.off_of, self.lengths, self.kk, self.v, self.k_cache,
                           self.v_cache, self.cache_off, self.cache_cap, self.ws.unpack_dev, host_unpack,
                           self.ws.unpack_bytes, stream)
        self.ws.release(slot)

    def run_fused(self, repack: bool = False, flags: int = 0, keep_rope_table: bool = True) -> None:
        """One pass of the hot path through the fused entry point (asynchronous). q is left untouched.
        The fused workspace is written by nothing but these calls, so from the second call with the
        same capacity on, the cos/sin table in it is declared valid (PP_FLAG_KEEP_ROPE_TABLE)."""
        if repack:
            self._pack()
        stream = torch.cuda.current_stream().cuda_stream
        _, _, slot = self.ws.acquire()
        if keep_rope_table and getattr(self, "_rope_table_capacity", None) == self.pack.capacity:
            flags |= B.PP_FLAG_KEEP_ROPE_TABLE
        self._rope_table_capacity = self.pack.capacity
        self.params.flags = flags
        B.pp_prefill_fused(self.params, self.pack, self.lengths, self.q, self.kk, self.v, self.o, self.k_cache,
                           self.v_cache, self.cache_off, self.cache_cap, self.ws.fused_dev,
                           self.ws.fused_host(slot), self.ws.fused_bytes, self.ws.status, stream)
        self.ws.release(slot)

    def run_unpack_only(self) -> None:
        stream = torch.cuda.current_stream().cuda_stream
        _, host_unpack, slot = self.ws.acquire()
        B.pp_unpack_kv(self.params, self.bin_of, self.off_of, self.lengths, self.kk, self.v, self.k_cache,
                       self.v_cache, self.cache_off, self.cache_cap, self.ws.unpack_dev, host_unpack,
                       self.ws.unpack_bytes, stream)
        self.ws.release(slot)

    def device_status(self) -> int:
        return int(self.ws.status.item())

    # ---- views of the results, original prompt order (device tensors) ----
    def o_tokens(self) -> torch.Tensor:
        """[T, Hq, D] attention outputs of the real tokens."""
        return self.o.view(-1, self.hq, self.d)[self.token_rows]

    def rotated_tokens(self):
        """([T, Hq, D], [T, Hkv, D]): q and k as they stand in the packed buffers."""
        return (self.q.view(-1, self.hq, self.d)[self.token_rows],
                self.kk.view(-1, self.hkv, self.d)[self.token_rows])

    def caches(self, i: int):
        """(k_cache_i, v_cache_i) as [Hkv, cap_i, D] views of the pools; rows [0, lengths[i]) are filled."""
        n = int(self.cache_cap[i]) * self.hkv * self.d
        off = int(self.cache_off[i])
        shape = (self.hkv, int(self.cache_cap[i]), self.d)
        return self.k_cache[off:off + n].view(shape), self.v_cache[off:off + n].view(shape)


class DecodeBatch:
    """Per-prompt KV caches with room to grow, and one generation step at a time through
    pp_decode_step. Memory plumbing only: `adopt` copies the caches a PrefillBatch has filled into
    blocks of capacity lengths[i] + room."""

    def __init__(self, lengths, n_q_heads: int, n_kv_heads: int, head_dim: int, rope_base: float,
                 room: int = 32, device: str = "cuda", softmax_scale: float = 0.0):
        self.device = torch.device(device)
        self.lengths = np.ascontiguousarray(np.asarray(lengths, dtype=np.int32)).copy()
        self.k = int(self.lengths.shape[0])
        self.hq, self.hkv, self.d = n_q_heads, n_kv_heads, head_dim
        self.cache_cap = (self.lengths + room).astype(np.int32)
        prefix = np.concatenate([[0], np.cumsum(self.cache_cap.astype(np.int64))])
        self.cache_off = (prefix[:-1] * n_kv_heads * head_dim).astype(np.int64)
        pool = int(prefix[-1]) * n_kv_heads * head_dim
        self.k_cache = torch.zeros(pool, dtype=torch.bfloat16, device=self.device)
        self.v_cache = torch.zeros(pool, dtype=torch.bfloat16, device=self.device)
        self.params = B.AttnParams(n_q_heads, n_kv_heads, head_dim, rope_base, softmax_scale, 1, 1, 0)
        self.o = torch.zeros((self.k, n_q_heads, head_dim), dtype=torch.bfloat16, device=self.device)
        self._ws_bytes = 0
        self._ws = self._host = None

    def caches(self, i: int):
        """(k_cache_i, v_cache_i) as [Hkv, cap_i, D] views; rows [0, lengths[i]) are filled."""
        cap = int(self.cache_cap[i])
        n = cap * self.hkv * self.d
        off = int(self.cache_off[i])
        shape = (self.hkv, cap, self.d)
        return self.k_cache[off:off + n].view(shape), self.v_cache[off:off + n].view(shape)

    @classmethod
    def from_prefill(cls, prefill: PrefillBatch) -> "DecodeBatch":
        """Decode straight on the cache pools a PrefillBatch (built with room > 0) has filled: the
        hand-over from UNPACK to generation, no copy in between."""
        self = cls.__new__(cls)
        self.device = prefill.device
        self.lengths = prefill.lengths.copy()
        self.k = prefill.k
        self.hq, self.hkv, self.d = prefill.hq, prefill.hkv, prefill.d
        self.cache_cap, self.cache_off = prefill.cache_cap, prefill.cache_off
        self.k_cache, self.v_cache = prefill.k_cache, prefill.v_cache
        self.params = B.AttnParams(self.hq, self.hkv, self.d, prefill.rope_base, prefill.softmax_scale, 1, 1, 0)
        self.o = torch.zeros((self.k, self.hq, self.d), dtype=torch.bfloat16, device=self.device)
        self._ws_bytes = 0
        self._ws = self._host = None
        return self

    def adopt(self, prefill: PrefillBatch) -> None:
        for i in range(self.k):
            src_k, src_v = prefill.caches(i)
            dst_k, dst_v = self.caches(i)
            l = int(self.lengths[i])
            dst_k[:, :l].copy_(src_k[:, :l])
            dst_v[:, :l].copy_(src_v[:, :l])

    def step(self, q_new: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor) -> torch.Tensor:
        """One token per prompt: q_new [k, Hq, D], k_new / v_new [k, Hkv, D] bf16 on the device."""
        need = B.pp_decode_workspace_bytes(self.params, self.lengths)
        if need > self._ws_bytes:
            self._ws_bytes = need + (need >> 2)        # lengths grow by one per step
            self._ws = torch.empty(self._ws_bytes, dtype=torch.uint8, device=self.device)
            self._host = [torch.empty(self._ws_bytes, dtype=torch.uint8).pin_memory() for _ in range(2)]
            self._copied = [None, None]                # event after the upload that last read each staging buffer
            self._turn = 0
        slot = self._turn & 1
        self._turn += 1
        if self._copied[slot] is not None:
            self._copied[slot].synchronize()
        B.pp_decode_step(self.params, self.lengths, q_new, k_new, v_new, self.o, self.k_cache, self.v_cache,
                         self.cache_off, self.cache_cap, self._ws, self._host[slot], self._ws_bytes,
                         torch.cuda.current_stream().cuda_stream)
        self._copied[slot] = torch.cuda.Event()
        self._copied[slot].record()
        self.lengths += 1
        return self.o
