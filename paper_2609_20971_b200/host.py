"""Prefill of one layer whose Q/K/V live in (pinned) host memory and whose output goes back to host memory.

The copies dominate such a call (2.4 GB over PCIe for a 128K Qwen3-30B-A3B layer against ~14 ms of kernels), so the
work is cut into query chunks and pipelined over three streams: K and V go first (statistics need all keys), then
for every chunk of query blocks the host->device copy of its Q rows, rbs_select_chunk + rbs_sparse_prefill_chunk,
and the device->host copy of its O rows overlap with the neighbouring chunks' stages.  Arithmetic is entirely in the
library's kernels; this module only moves buffers and orders streams.
"""
from __future__ import annotations

import torch

from .binding import (RBS_OP_SELECT, RBS_OP_SPARSE_PREFILL, RbsShape, alloc_stats, rbs_block_stats, rbs_select_chunk, rbs_sparse_prefill_chunk,
                      workspace_bytes)


class HostPrefill:
    """Reusable device buffers and streams for prefill_host.  All tensors [L, N, H, d] bf16; host tensors pinned."""

    def __init__(self, L: int, N: int, Hq: int, Hkv: int, d: int, block: int, device, chunk_blocks: int = 64):
        self.L, self.N, self.Hq, self.Hkv, self.d, self.B = L, N, Hq, Hkv, d, block
        self.dev = torch.device(device)
        self.M = (N + block - 1) // block
        self.chunk_blocks = max(1, min(chunk_blocks, self.M))
        bf = torch.bfloat16
        self.Qg = torch.empty(L, N, Hq, d, dtype=bf, device=self.dev)
        self.Kg = torch.empty(L, N, Hkv, d, dtype=bf, device=self.dev)
        self.Vg = torch.empty(L, N, Hkv, d, dtype=bf, device=self.dev)
        self.Og = torch.empty(L, N, Hq, d, dtype=bf, device=self.dev)
        self.stats = alloc_stats(self.Kg, block)
        W = (self.M + 31) // 32
        n_chunks = (self.M + self.chunk_blocks - 1) // self.chunk_blocks
        # one dense [L, Hq, Mq, W] mask per chunk (the library writes dense rows; a slice of a whole-sequence mask
        # along the query-block axis would not be dense for L * Hq > 1)
        self.masks = [torch.empty(L, Hq, min(self.M, q0 + self.chunk_blocks) - q0, W, dtype=torch.int32, device=self.dev)
                      for q0 in range(0, self.M, self.chunk_blocks)]
        self.density = torch.empty(n_chunks, L, Hq, dtype=torch.float32, device=self.dev)
        shape = RbsShape(L, N, Hq, Hkv, d, block)
        self.ws = torch.empty(max(256, workspace_bytes(RBS_OP_SELECT, shape)), dtype=torch.uint8, device=self.dev)
        self.ws_att = torch.empty(max(256, workspace_bytes(RBS_OP_SPARSE_PREFILL, shape)), dtype=torch.uint8, device=self.dev)
        self.s_in, self.s_out = torch.cuda.Stream(self.dev), torch.cuda.Stream(self.dev)

    def chunks(self):
        """(chunk index, first block, end block, first token, end token), last chunk first: its rows are the longest,
        so the cheapest chunk is the one whose compute and copy-out cannot overlap with anything."""
        starts = list(range(0, self.M, self.chunk_blocks))
        for c in reversed(range(len(starts))):
            q0 = starts[c]
            q1 = min(self.M, q0 + self.chunk_blocks)
            yield c, q0, q1, q0 * self.B, min(self.N, q1 * self.B)

    def run(self, Qh, Kh, Vh, Oh, alpha_base=0.22, alpha_rescue=0.18, n_sink=1, n_local=1, n_recent=1):
        """Enqueues the whole pipeline; Oh is complete once the current stream and self.s_out have been synchronised
        (call .wait()).  Returns the per-chunk densities tensor [n_chunks, L, Hq] (device)."""
        main = torch.cuda.current_stream(self.dev)
        self.s_in.wait_stream(main)          # buffers may still be in use by earlier work on the caller's stream
        self.s_out.wait_stream(main)
        with torch.cuda.stream(self.s_in):
            self.Kg.copy_(Kh, non_blocking=True)
            self.Vg.copy_(Vh, non_blocking=True)
            kv_ready = torch.cuda.Event()
            kv_ready.record(self.s_in)
        main.wait_event(kv_ready)
        rbs_block_stats(self.Kg, self.B, self.stats)
        for c, q0, q1, t0, t1 in self.chunks():
            with torch.cuda.stream(self.s_in):
                self.Qg[:, t0:t1].copy_(Qh[:, t0:t1], non_blocking=True)
                q_ready = torch.cuda.Event()
                q_ready.record(self.s_in)
            main.wait_event(q_ready)
            mc = self.masks[c]
            rbs_select_chunk(self.Qg[:, t0:t1], self.stats, self.B, self.N, q0, alpha_base, alpha_rescue, n_sink, n_local,
                             n_recent, mask=mc, density=self.density[c], workspace=self.ws)
            rbs_sparse_prefill_chunk(self.Qg[:, t0:t1], self.Kg, self.Vg, mc, self.B, q0, out=self.Og[:, t0:t1],
                                     workspace=self.ws_att)
            o_ready = torch.cuda.Event()
            o_ready.record(main)
            with torch.cuda.stream(self.s_out):
                self.s_out.wait_event(o_ready)
                Oh[:, t0:t1].copy_(self.Og[:, t0:t1], non_blocking=True)
        return self.density

    def mask(self) -> torch.Tensor:
        """The whole-sequence mask [L, Hq, M, W] assembled from the chunk masks (a copy)."""
        return torch.cat(self.masks, dim=2)

    def wait(self):
        torch.cuda.current_stream(self.dev).wait_stream(self.s_out)


def prefill_host(Qh, Kh, Vh, block: int, device="cuda:0", Oh=None, **select_args):
    """One-shot convenience wrapper: allocates a HostPrefill, runs it, waits, returns (Oh, densities)."""
    L, N, Hq, d = Qh.shape
    hp = HostPrefill(L, N, Hq, Kh.shape[2], d, block, device)
    if Oh is None:
        Oh = torch.empty_like(Qh).pin_memory()
    dens = hp.run(Qh, Kh, Vh, Oh, **select_args)
    hp.wait()
    torch.cuda.current_stream(hp.dev).synchronize()
    return Oh, dens


def prefill_varlen(Q: torch.Tensor, K: torch.Tensor, V: torch.Tensor, cu_seqlens, block: int, *, out=None,
                   alpha_base: float = 0.22, alpha_rescue: float = 0.18, n_sink: int = 1, n_local: int = 1,
                   n_recent: int = 1, streams=None):
    """A batch of prompts of different lengths packed along the token axis (no padding, nothing concatenated across
    prompts: every prompt is selected and attended on its own, as in Sec. 4.1).

    Q [T, Hq, d], K and V [T, Hkv, d] are CUDA bf16 tensors holding the prompts back to back; `cu_seqlens` (host
    ints, length n + 1, cu_seqlens[0] = 0, cu_seqlens[-1] = T) gives the boundaries.  Each prompt becomes one call of
    rbs_block_stats / rbs_select / rbs_sparse_prefill on a view of the packed buffers (the library takes strides,
    so nothing is copied); prompts are spread round-robin over `streams` (default: the current stream only).
    Returns (O [T, Hq, d], densities: list of [1, Hq] tensors, one per prompt)."""
    from .binding import rbs_select, rbs_sparse_prefill
    cu = [int(x) for x in cu_seqlens]
    if len(cu) < 2 or cu[0] != 0 or cu[-1] != Q.shape[0] or any(b <= a for a, b in zip(cu, cu[1:])):
        raise ValueError("cu_seqlens must start at 0, end at the number of packed tokens and increase strictly")
    if out is None:
        out = torch.empty_like(Q)
    cur = torch.cuda.current_stream(Q.device)
    streams = list(streams) if streams else [cur]
    for s in streams:
        if s != cur:
            s.wait_stream(cur)
    densities = []
    for k, (t0, t1) in enumerate(zip(cu, cu[1:])):
        s = streams[k % len(streams)]
        with torch.cuda.stream(s):
            q, kk, v, o = (t[t0:t1].unsqueeze(0) for t in (Q, K, V, out))
            stats = rbs_block_stats(kk, block)
            mask, dens = rbs_select(q, stats, block, alpha_base, alpha_rescue, n_sink, n_local, n_recent)
            rbs_sparse_prefill(q, kk, v, mask, block, out=o)
            densities.append(dens)
            for t in (stats.centroid, stats.radius, stats.beta, stats.rq, mask, dens):
                t.record_stream(s)       # (the calls' own workspaces are torch allocations made under stream s)
    for s in streams:
        if s != cur:
            cur.wait_stream(s)
    return out, densities
