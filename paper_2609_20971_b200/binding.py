"""Thin ctypes binding over the C ABI declared in include/rbs.h.

Argument marshalling only: tensor pointers, strides and the current CUDA stream are handed to the
library; every step of the path runs in the library's kernels.  torch provides device memory and
streams.  There is no fallback: if the shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
# RBS_DEBUG=1 in the environment selects the library built with -DRBS_DEBUG (device-side index checks that are
# reported through rbs_device_status; `python -m paper_2609_20971_b200.build --debug`)
LIB_PATH = os.path.join(_PKG, "librbs_b200_debug.so" if os.environ.get("RBS_DEBUG", "0") not in ("", "0") else "librbs_b200.so")

RBS_OP_BLOCK_STATS, RBS_OP_SELECT, RBS_OP_SPARSE_PREFILL, RBS_OP_SELECT_BOX = 0, 1, 2, 3
SELECTOR_RBS, SELECTOR_CENTROID_ONLY, SELECTOR_FULL_L2 = 0, 1, 2


class RbsShape(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int), ("seqlen", ctypes.c_int), ("n_q_heads", ctypes.c_int),
                ("n_kv_heads", ctypes.c_int), ("head_dim", ctypes.c_int), ("block", ctypes.c_int)]


class RbsTensor(ctypes.Structure):
    _fields_ = [("ptr", ctypes.c_void_p), ("stride_batch", ctypes.c_int64),
                ("stride_token", ctypes.c_int64), ("stride_head", ctypes.c_int64)]


class RbsStats(ctypes.Structure):
    _fields_ = [("centroid", ctypes.c_void_p), ("radius", ctypes.c_void_p),
                ("beta", ctypes.c_void_p), ("rq", ctypes.c_void_p)]


class RbsBox(ctypes.Structure):
    _fields_ = [("lo", ctypes.c_void_p), ("hi", ctypes.c_void_p)]


class RbsError(RuntimeError):
    pass


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads the CUDA library built by build.py; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RbsError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_20971_b200.build` "
                       "(there is no CPU fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, sz, f, i = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_float, ctypes.c_int
    lib.rbs_workspace_bytes.restype = sz
    lib.rbs_workspace_bytes.argtypes = [i, ctypes.POINTER(RbsShape)]
    lib.rbs_block_stats.restype = i
    lib.rbs_block_stats.argtypes = [ctypes.POINTER(RbsShape), RbsTensor, RbsStats, vp]
    lib.rbs_select.restype = i
    lib.rbs_select.argtypes = [ctypes.POINTER(RbsShape), RbsTensor, RbsStats, f, f, i, i, i, vp, vp, vp, vp, vp, sz, vp]
    lib.rbs_select_chunk.restype = i
    lib.rbs_select_chunk.argtypes = [ctypes.POINTER(RbsShape), i, i, RbsTensor, RbsStats, f, f, i, i, i, vp, vp, vp, vp, vp, sz, vp]
    lib.rbs_sparse_prefill_chunk.restype = i
    lib.rbs_sparse_prefill_chunk.argtypes = [ctypes.POINTER(RbsShape), i, i, RbsTensor, RbsTensor, RbsTensor, vp, RbsTensor,
                                             vp, f, vp, sz, vp]
    lib.rbs_select_variant.restype = i
    lib.rbs_select_variant.argtypes = [ctypes.POINTER(RbsShape), RbsTensor, RbsStats, i, f, f, i, i, i, vp, vp, vp, vp, vp, sz, vp]
    lib.rbs_select_static.restype = i
    lib.rbs_select_static.argtypes = [ctypes.POINTER(RbsShape), RbsTensor, RbsStats, f, f, i, i, i, vp, vp, vp, vp, vp]
    lib.rbs_mask_group_union.restype = i
    lib.rbs_mask_group_union.argtypes = [ctypes.POINTER(RbsShape), i, i, vp, vp, vp]
    lib.rbs_sparse_prefill.restype = i
    lib.rbs_sparse_prefill.argtypes = [ctypes.POINTER(RbsShape), RbsTensor, RbsTensor, RbsTensor, vp, RbsTensor,
                                       vp, f, vp, sz, vp]
    lib.rbs_sparse_prefill_grouped.restype = i
    lib.rbs_sparse_prefill_grouped.argtypes = [ctypes.POINTER(RbsShape), RbsTensor, RbsTensor, RbsTensor, vp, RbsTensor, vp, f, vp]
    lib.rbs_varlen_workspace_bytes.restype = sz
    lib.rbs_varlen_workspace_bytes.argtypes = [i, ctypes.POINTER(ctypes.c_int), i, i, i, i]
    lib.rbs_prefill_varlen.restype = i
    lib.rbs_prefill_varlen.argtypes = [i, ctypes.POINTER(ctypes.c_int), i, i, i, i, RbsTensor, RbsTensor, RbsTensor, RbsTensor,
                                       f, f, i, i, i, vp, vp, sz, vp]
    lib.rbs_device_status.restype = i
    lib.rbs_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_uint), i]
    lib.rbs_block_stats_box.restype = i
    lib.rbs_block_stats_box.argtypes = [ctypes.POINTER(RbsShape), RbsTensor, RbsStats, RbsBox, vp]
    lib.rbs_select_box.restype = i
    lib.rbs_select_box.argtypes = [ctypes.POINTER(RbsShape), RbsTensor, RbsBox, ctypes.c_double, i, i, i, vp, vp, vp, vp, sz, vp]
    lib.rbs_selftest_device_table.restype = i
    lib.rbs_selftest_device_table.argtypes = []
    lib.rbs_selftest_wait_timeout.restype = i
    lib.rbs_selftest_wait_timeout.argtypes = [ctypes.c_uint, vp, vp]
    lib.rbs_selftest_debug_check.restype = i
    lib.rbs_selftest_debug_check.argtypes = [vp, vp]
    lib.rbs_status_string.restype = ctypes.c_char_p
    lib.rbs_status_string.argtypes = [i]
    lib.rbs_version.restype = ctypes.c_char_p
    lib.rbs_version.argtypes = []
    _lib = lib
    return lib


def _check(code: int, what: str) -> None:
    if code != 0:
        raise RbsError(f"{what} failed: {load_library().rbs_status_string(code).decode()}")


def _tensor(t: torch.Tensor) -> RbsTensor:
    if t.dim() != 4 or t.dtype != torch.bfloat16 or not t.is_cuda or t.stride(3) != 1:
        raise RbsError("expected a CUDA bf16 tensor [batch, tokens, heads, head_dim] with head_dim contiguous")
    return RbsTensor(t.data_ptr(), t.stride(0), t.stride(1), t.stride(2))


def _shape(Q_or_none, K, block: int, n_q_heads: int | None = None) -> RbsShape:
    L, N, Hkv, d = K.shape
    Hq = n_q_heads if n_q_heads is not None else (Q_or_none.shape[2] if Q_or_none is not None else Hkv)
    return RbsShape(L, N, Hq, Hkv, d, block)


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr(t) -> ctypes.c_void_p:
    return ctypes.c_void_p(None if t is None else t.data_ptr())


@dataclass
class BlockStats:
    centroid: torch.Tensor  # [L, Hkv, M, d] fp32
    radius: torch.Tensor    # [L, Hkv, M]    fp32
    beta: torch.Tensor      # [L, Hkv, M]    fp32, written by rbs_select
    rq: torch.Tensor        # [L, Hkv, 2]    fp32, written by rbs_select

    def c_struct(self) -> RbsStats:
        return RbsStats(self.centroid.data_ptr(), self.radius.data_ptr(), self.beta.data_ptr(), self.rq.data_ptr())


def alloc_stats(K: torch.Tensor, block: int) -> BlockStats:
    L, N, Hkv, d = K.shape
    M = (N + block - 1) // block
    dev = K.device
    return BlockStats(torch.empty(L, Hkv, M, d, dtype=torch.float32, device=dev),
                      torch.empty(L, Hkv, M, dtype=torch.float32, device=dev),
                      torch.zeros(L, Hkv, M, dtype=torch.float32, device=dev),
                      torch.zeros(L, Hkv, 2, dtype=torch.float32, device=dev))


def workspace_bytes(op: int, shape: RbsShape) -> int:
    return int(load_library().rbs_workspace_bytes(op, ctypes.byref(shape)))


def rbs_device_status(clear: bool = True) -> int:
    """Synchronises the current stream and returns the device status word: 0 unless a bounded wait inside a
    kernel gave up (the outputs of that launch are then undefined).  `clear` resets the word."""
    code = ctypes.c_uint(0)
    rc = load_library().rbs_device_status(_stream(), ctypes.byref(code), 1 if clear else 0)
    if rc not in (0, 5, 6):     # a recorded time-out or failed debug check is the answer, not a failure of the call
        _check(rc, "rbs_device_status")
    return int(code.value)


def rbs_selftest_wait_timeout(spin_limit: int = 4096) -> torch.Tensor:
    """Launches the library's time-out self-test (one thread waits, with a short limit, on a barrier nothing arrives
    on) and returns the device flag it writes (1 = the wait gave up).  The status word then holds the code."""
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    _check(load_library().rbs_selftest_wait_timeout(spin_limit, _ptr(flag), _stream()), "rbs_selftest_wait_timeout")
    return flag


def rbs_selftest_debug_check() -> torch.Tensor | None:
    """Debug library only (RBS_DEBUG=1): runs one device-side index check that fails by construction and returns
    the device flag the guarded access leaves (1 = skipped); the status word then holds 0x1ff.  None in the
    release library, which has no such checks."""
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    rc = load_library().rbs_selftest_debug_check(_ptr(flag), _stream())
    if rc == 2:       # RBS_ERR_UNSUPPORTED: release build
        return None
    _check(rc, "rbs_selftest_debug_check")
    return flag


def rbs_version() -> str:
    return load_library().rbs_version().decode()


def rbs_block_stats(K: torch.Tensor, block: int, stats: BlockStats | None = None) -> BlockStats:
    """Key-block centroids and radii (Sec. 3.1).  K: [L, N, Hkv, d] bf16 on the GPU."""
    lib = load_library()
    if stats is None:
        stats = alloc_stats(K, block)
    shape = _shape(None, K, block)
    _check(lib.rbs_block_stats(ctypes.byref(shape), _tensor(K), stats.c_struct(), _stream()), "rbs_block_stats")
    return stats


def rbs_select(Q: torch.Tensor, stats: BlockStats, block: int, alpha_base: float = 0.22, alpha_rescue: float = 0.18,
               n_sink: int = 1, n_local: int = 1, n_recent: int = 1, *, mask: torch.Tensor | None = None,
               density: torch.Tensor | None = None, workspace: torch.Tensor | None = None, debug: bool = False,
               selector: int = 0):
    """Dual-branch block selection (Sec. 3.2).  Returns (mask uint32-as-int32 [L,Hq,M,W], density [L,Hq])
    and, with debug=True, also the base and rescue branch masks.  `selector`: SELECTOR_RBS (default),
    SELECTOR_CENTROID_ONLY or SELECTOR_FULL_L2 (the comparison selectors of the paper's ablation)."""
    lib = load_library()
    L, N, Hq, d = Q.shape
    Hkv = stats.centroid.shape[1]
    M = (N + block - 1) // block
    W = (M + 31) // 32
    shape = RbsShape(L, N, Hq, Hkv, d, block)
    dev = Q.device
    if mask is None:
        mask = torch.empty(L, Hq, M, W, dtype=torch.int32, device=dev)
    if density is None:
        density = torch.empty(L, Hq, dtype=torch.float32, device=dev)
    need = workspace_bytes(RBS_OP_SELECT, shape)
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
    dbg_b = torch.empty_like(mask) if debug else None
    dbg_r = torch.empty_like(mask) if debug else None
    if selector == SELECTOR_RBS:
        _check(lib.rbs_select(ctypes.byref(shape), _tensor(Q), stats.c_struct(), alpha_base, alpha_rescue,
                              n_sink, n_local, n_recent, _ptr(mask), _ptr(density), _ptr(dbg_b), _ptr(dbg_r),
                              _ptr(workspace), workspace.numel(), _stream()), "rbs_select")
    else:
        _check(lib.rbs_select_variant(ctypes.byref(shape), _tensor(Q), stats.c_struct(), selector, alpha_base,
                                      alpha_rescue, n_sink, n_local, n_recent, _ptr(mask), _ptr(density), _ptr(dbg_b),
                                      _ptr(dbg_r), _ptr(workspace), workspace.numel(), _stream()), "rbs_select_variant")
    if debug:
        return mask, density, dbg_b, dbg_r
    return mask, density


SELECT_STATIC_SCRATCH_BYTES = 4 << 20


def rbs_select_static(Q: torch.Tensor, stats: BlockStats, block: int, alpha_base: float = 0.22,
                      alpha_rescue: float = 0.18, n_sink: int = 1, n_local: int = 1, n_recent: int = 1, *,
                      mask: torch.Tensor, density: torch.Tensor, dbg_base: torch.Tensor | None = None,
                      dbg_rescue: torch.Tensor | None = None):
    """rbs_select for callers that may not allocate: the scratch is a fixed array inside the library, and
    this wrapper allocates nothing either, so `mask` [L,Hq,M,W] int32 and `density` [L,Hq] fp32 must be
    passed in.  Raises RbsError(RBS_ERR_WORKSPACE) when the shape needs more than
    SELECT_STATIC_SCRATCH_BYTES of scratch.  Calls on one device share the array: do not let two overlap."""
    lib = load_library()
    L, N, Hq, d = Q.shape
    shape = RbsShape(L, N, Hq, stats.centroid.shape[1], d, block)
    _check(lib.rbs_select_static(ctypes.byref(shape), _tensor(Q), stats.c_struct(), alpha_base, alpha_rescue,
                                 n_sink, n_local, n_recent, _ptr(mask), _ptr(density), _ptr(dbg_base),
                                 _ptr(dbg_rescue), _stream()), "rbs_select_static")
    return mask, density


def rbs_mask_group_union(mask: torch.Tensor, density: torch.Tensor, n_kv_heads: int, block: int, seqlen: int,
                         q_start_block: int = 0, n_q_tokens: int = -1, head_dim: int = 128):
    """In place: the mask rows [L,Hq,Mq,W] of the query heads that share a KV head become their union, and
    `density` [L,Hq] is recomputed (a variant outside the paper's per-head selector)."""
    lib = load_library()
    L, Hq = mask.shape[0], mask.shape[1]
    if not mask.is_contiguous() or mask.dtype != torch.int32 or density.dtype != torch.float32:
        raise RbsError("mask must be a contiguous int32 tensor [L,Hq,Mq,W] and density fp32 [L,Hq]")
    shape = RbsShape(L, seqlen, Hq, n_kv_heads, head_dim, block)
    _check(lib.rbs_mask_group_union(ctypes.byref(shape), q_start_block, n_q_tokens, _ptr(mask), _ptr(density),
                                    _stream()), "rbs_mask_group_union")
    return mask, density


def rbs_sparse_prefill(Q: torch.Tensor, K: torch.Tensor, V: torch.Tensor, mask: torch.Tensor | None, block: int, *,
                       out: torch.Tensor | None = None, return_lse: bool = False, softmax_scale: float = 0.0,
                       workspace: torch.Tensor | None = None):
    """Causal block-sparse attention over `mask` (Sec. 3.3); mask=None is dense causal attention (Eq. 1).
    `workspace` (uint8, at least prefill_workspace_bytes(...)): opt into the row-length-aware schedule (blocks of 128
    or 256): rows of more than 256 key tiles are cut into parts that run side by side and are merged afterwards."""
    lib = load_library()
    L, N, Hq, d = Q.shape
    shape = RbsShape(L, N, Hq, K.shape[2], d, block)
    if out is None:
        out = torch.empty_like(Q)
    lse = torch.empty(L, Hq, N, dtype=torch.float32, device=Q.device) if return_lse else None
    _check(lib.rbs_sparse_prefill(ctypes.byref(shape), _tensor(Q), _tensor(K), _tensor(V), _ptr(mask), _tensor(out),
                                  _ptr(lse), softmax_scale, _ptr(workspace),
                                  0 if workspace is None else workspace.numel(), _stream()), "rbs_sparse_prefill")
    return (out, lse) if return_lse else out


def rbs_block_stats_box(K: torch.Tensor, block: int, stats: BlockStats | None = None):
    """rbs_block_stats plus, from the same read of K, the per-coordinate minima and maxima of every block
    (App. D.2).  Returns (stats, box_lo [L, Hkv, M, d] fp32, box_hi)."""
    lib = load_library()
    if stats is None:
        stats = alloc_stats(K, block)
    lo, hi = torch.empty_like(stats.centroid), torch.empty_like(stats.centroid)
    shape = _shape(None, K, block)
    _check(lib.rbs_block_stats_box(ctypes.byref(shape), _tensor(K), stats.c_struct(), RbsBox(lo.data_ptr(), hi.data_ptr()),
                                   _stream()), "rbs_block_stats_box")
    return stats, lo, hi


def rbs_select_box(Q: torch.Tensor, box_lo: torch.Tensor, box_hi: torch.Tensor, block: int, density_param: float = 0.0405,
                   n_sink: int = 1, n_local: int = 1, n_recent: int = 1, *, debug: bool = False):
    """The Quest-style comparison selector (Sec. 4.2, Eq. quest_box): box upper bound as the block logit, the same
    aggregation over the query block, the ceil(density_param (i + 1)) best causal blocks of query block i plus the
    forced ones.  Returns (mask, density) and, with debug=True, the choice before the union with the forced blocks."""
    lib = load_library()
    L, N, Hq, d = Q.shape
    Hkv = box_lo.shape[1]
    M = (N + block - 1) // block
    shape = RbsShape(L, N, Hq, Hkv, d, block)
    mask = torch.empty(L, Hq, M, (M + 31) // 32, dtype=torch.int32, device=Q.device)
    density = torch.empty(L, Hq, dtype=torch.float32, device=Q.device)
    chosen = torch.empty_like(mask) if debug else None
    ws = torch.empty(max(256, workspace_bytes(RBS_OP_SELECT_BOX, shape)), dtype=torch.uint8, device=Q.device)
    _check(lib.rbs_select_box(ctypes.byref(shape), _tensor(Q), RbsBox(box_lo.data_ptr(), box_hi.data_ptr()), float(density_param),
                              n_sink, n_local, n_recent, _ptr(mask), _ptr(density), _ptr(chosen), _ptr(ws), ws.numel(),
                              _stream()), "rbs_select_box")
    return (mask, density, chosen) if debug else (mask, density)


def rbs_sparse_prefill_grouped(Q: torch.Tensor, K: torch.Tensor, V: torch.Tensor, mask: torch.Tensor, block: int, *,
                               out: torch.Tensor | None = None, return_lse: bool = False, softmax_scale: float = 0.0):
    """rbs_sparse_prefill for masks that are identical inside every KV group (after rbs_mask_group_union): two heads
    of a group share one stream of K/V tiles."""
    lib = load_library()
    L, N, Hq, d = Q.shape
    shape = RbsShape(L, N, Hq, K.shape[2], d, block)
    if out is None:
        out = torch.empty_like(Q)
    lse = torch.empty(L, Hq, N, dtype=torch.float32, device=Q.device) if return_lse else None
    _check(lib.rbs_sparse_prefill_grouped(ctypes.byref(shape), _tensor(Q), _tensor(K), _tensor(V), _ptr(mask), _tensor(out),
                                          _ptr(lse), softmax_scale, _stream()), "rbs_sparse_prefill_grouped")
    return (out, lse) if return_lse else out


def rbs_prefill_varlen(Q: torch.Tensor, K: torch.Tensor, V: torch.Tensor, cu_seqlens, block: int, *, out=None,
                       alpha_base: float = 0.22, alpha_rescue: float = 0.18, n_sink: int = 1, n_local: int = 1,
                       n_recent: int = 1, workspace: torch.Tensor | None = None):
    """Prompts of different lengths packed along the token axis: Q [T, Hq, d], K, V [T, Hkv, d]; `cu_seqlens` host
    ints (n + 1).  One library call for the whole batch, one reusable workspace.  Returns (O [T, Hq, d],
    density [n, Hq])."""
    lib = load_library()
    cu = [int(c) for c in cu_seqlens]
    n = len(cu) - 1
    arr = (ctypes.c_int * len(cu))(*cu)
    T, Hq, d = Q.shape
    Hkv = K.shape[1]
    if out is None:
        out = torch.empty_like(Q)
    need = int(lib.rbs_varlen_workspace_bytes(n, arr, Hq, Hkv, d, block))
    if need == 0:
        raise RbsError("rbs_prefill_varlen: cu_seqlens must start at 0 and increase strictly, and the shape must be supported")
    if cu[-1] != T:
        raise RbsError("rbs_prefill_varlen: cu_seqlens must end at the number of packed tokens")
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=Q.device)
    density = torch.empty(n, Hq, dtype=torch.float32, device=Q.device)

    def packed(t):
        if t.dim() != 3 or t.dtype != torch.bfloat16 or not t.is_cuda or t.stride(2) != 1:
            raise RbsError("expected CUDA bf16 tensors [tokens, heads, head_dim] with head_dim contiguous")
        return RbsTensor(t.data_ptr(), 0, t.stride(0), t.stride(1))
    _check(lib.rbs_prefill_varlen(n, arr, Hq, Hkv, d, block, packed(Q), packed(K), packed(V), packed(out), alpha_base,
                                  alpha_rescue, n_sink, n_local, n_recent, _ptr(density), _ptr(workspace), workspace.numel(),
                                  _stream()), "rbs_prefill_varlen")
    return out, density


def prefill_workspace_bytes(L: int, N: int, Hq: int, Hkv: int, block: int, d: int = 128) -> int:
    """Bytes of the optional rbs_sparse_prefill / rbs_sparse_prefill_chunk workspace for a sequence of N tokens."""
    return workspace_bytes(RBS_OP_SPARSE_PREFILL, RbsShape(L, N, Hq, Hkv, d, block))


def rbs_select_chunk(Q: torch.Tensor, stats: BlockStats, block: int, seqlen: int, q_start_block: int,
                     alpha_base: float = 0.22, alpha_rescue: float = 0.18, n_sink: int = 1, n_local: int = 1,
                     n_recent: int = 1, *, mask: torch.Tensor | None = None, density: torch.Tensor | None = None,
                     workspace: torch.Tensor | None = None):
    """Selection for the query chunk Q [L, Nq, Hq, d] that starts at block `q_start_block` of a sequence of `seqlen`
    tokens whose statistics are in `stats`.  Returns (mask [L,Hq,Mq,W], density [L,Hq]) of the chunk."""
    lib = load_library()
    L, Nq, Hq, d = Q.shape
    shape = RbsShape(L, seqlen, Hq, stats.centroid.shape[1], d, block)
    M, Mq = (seqlen + block - 1) // block, (Nq + block - 1) // block
    if mask is None:
        mask = torch.empty(L, Hq, Mq, (M + 31) // 32, dtype=torch.int32, device=Q.device)
    if density is None:
        density = torch.empty(L, Hq, dtype=torch.float32, device=Q.device)
    if workspace is None:
        workspace = torch.empty(max(256, workspace_bytes(RBS_OP_SELECT, shape)), dtype=torch.uint8, device=Q.device)
    _check(lib.rbs_select_chunk(ctypes.byref(shape), q_start_block, Nq, _tensor(Q), stats.c_struct(), alpha_base,
                                alpha_rescue, n_sink, n_local, n_recent, _ptr(mask), _ptr(density), None, None,
                                _ptr(workspace), workspace.numel(), _stream()), "rbs_select_chunk")
    return mask, density


def rbs_sparse_prefill_chunk(Q: torch.Tensor, K: torch.Tensor, V: torch.Tensor, mask: torch.Tensor | None, block: int,
                             q_start_block: int, *, out: torch.Tensor | None = None, return_lse: bool = False,
                             softmax_scale: float = 0.0, workspace: torch.Tensor | None = None):
    """Attention for the query chunk Q [L, Nq, Hq, d] starting at block `q_start_block`, against K, V [L, N, Hkv, d]."""
    lib = load_library()
    L, Nq, Hq, d = Q.shape
    shape = RbsShape(L, K.shape[1], Hq, K.shape[2], d, block)
    if out is None:
        out = torch.empty_like(Q)
    lse = torch.empty(L, Hq, Nq, dtype=torch.float32, device=Q.device) if return_lse else None
    _check(lib.rbs_sparse_prefill_chunk(ctypes.byref(shape), q_start_block, Nq, _tensor(Q), _tensor(K), _tensor(V),
                                        _ptr(mask), _tensor(out), _ptr(lse), softmax_scale, _ptr(workspace),
                                        0 if workspace is None else workspace.numel(), _stream()),
           "rbs_sparse_prefill_chunk")
    return (out, lse) if return_lse else out
