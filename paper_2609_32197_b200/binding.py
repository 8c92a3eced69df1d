"""ctypes binding of libsparsp.so: argument marshalling only.

Every function here has the name of the C entry point it forwards to (include/sparsp.h).  Tensors
are torch CUDA tensors used purely as device buffers; the current torch CUDA stream is passed down.
There is no fallback: if the library is missing or fails to load, importing a function works but the
first call raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsparsp.so")

SPARSP_OK = 0
SPARSP_ERR_INVALID_ARG = -1
SPARSP_ERR_UNSUPPORTED = -2
SPARSP_ERR_CAPACITY = -3
SPARSP_ERR_CUDA = -4
SPARSP_ERR_TIMEOUT = -5
SPARSP_PLAN_ONLY = 1
SPARSP_INCLUDE_LOCAL = 2

EXPORTS = [
    "sparsp_geometry", "sparsp_resolve_topk", "sparsp_placement_contiguous", "sparsp_placement_periodic",
    "sparsp_workspace_bytes", "sparsp_block_mask", "sparsp_demand_pack", "sparsp_sparse_attn_fwd",
    "sparsp_status", "sparsp_last_error", "sparsp_launch_count", "sparsp_demand_plan_noalloc",
    "sparsp_hop_mask", "sparsp_attn_merge", "sparsp_sparse_attn_fwd_packed", "sparsp_block_mask_cdf",
    "sparsp_placement_permutation", "sparsp_permute_tokens", "sparsp_sharing_histogram", "sparsp_exchange_plan",
    "sparsp_hop_chunk_mask", "sparsp_selftest_wait_timeout", "sparsp_attn_merge_rows", "sparsp_pack_segment",
    "sparsp_xchg_flag_bytes", "sparsp_xchg_export", "sparsp_xchg_connect", "sparsp_xchg_fence", "sparsp_xchg_acquire",
    "sparsp_xchg_publish", "sparsp_xchg_fetch", "sparsp_xchg_release", "sparsp_xchg_stats", "sparsp_xchg_destroy",
]
SPARSP_XCHG_HOST_MEMORY = 1


class SparspError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__(f"sparsp error {code}: {text}")
        self.code = code


class sparsp_shape(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("grid_t", ctypes.c_int32), ("grid_h", ctypes.c_int32), ("grid_w", ctypes.c_int32),
                ("n_text", ctypes.c_int32), ("block", ctypes.c_int32),
                ("stride_batch", ctypes.c_int64), ("stride_head", ctypes.c_int64),
                ("stride_token", ctypes.c_int64)]


_lib = None


def lib() -> ctypes.CDLL:
    """Loads the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            # not built yet (e.g. a fresh checkout): compile it in-tree with nvcc; if that is impossible
            # the call fails loudly -- there is no CPU fallback
            try:
                from . import build as _build
                _build.build()
            except Exception as exc:  # noqa: BLE001
                raise RuntimeError(f"{LIB_PATH} is missing and could not be built with nvcc ({exc}); "
                                   "there is no CPU fallback") from exc
        L = ctypes.CDLL(LIB_PATH)
        L.sparsp_last_error.restype = ctypes.c_char_p
        L.sparsp_launch_count.restype = ctypes.c_int64
        L.sparsp_resolve_topk.restype = ctypes.c_int32
        for name in EXPORTS:
            getattr(L, name)  # AttributeError if a declared symbol is not exported
        _lib = L
    return _lib


def _check(rc: int):
    if rc != SPARSP_OK:
        raise SparspError(rc, lib().sparsp_last_error().decode())


def _ptr(t):
    if t is None:
        return ctypes.c_void_p(0)
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


@dataclass
class Geometry:
    n_tokens: int
    n_blocks: int
    n_words: int
    n_video_blocks: int


def make_shape(heads: int, head_dim: int, grid, n_text: int, block: int, batch: int = 1,
               layout: str = "HND") -> sparsp_shape:
    """Shape for dense tensors laid out [B][H][N][d] ("HND") or [B][N][H][d] ("NHD")."""
    N = grid[0] * grid[1] * grid[2] + n_text
    if layout == "HND":
        sh, st = N * head_dim, head_dim
    elif layout == "NHD":
        sh, st = head_dim, heads * head_dim
    else:
        raise ValueError(layout)
    return sparsp_shape(batch, heads, head_dim, grid[0], grid[1], grid[2], n_text, block,
                        heads * N * head_dim, sh, st)


def sparsp_geometry(shape: sparsp_shape) -> Geometry:
    n, nb, wd, nv = ctypes.c_int64(), ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
    _check(lib().sparsp_geometry(ctypes.byref(shape), ctypes.byref(n), ctypes.byref(nb), ctypes.byref(wd),
                                 ctypes.byref(nv)))
    return Geometry(n.value, nb.value, wd.value, nv.value)


def sparsp_resolve_topk(pct: int, n_video_blocks: int) -> int:
    return int(lib().sparsp_resolve_topk(ctypes.c_int32(pct), ctypes.c_int32(n_video_blocks)))


def _placement(fn, shape, n_ranks):
    g = sparsp_geometry(shape)
    out = torch.empty(g.n_blocks, dtype=torch.int32)
    _check(fn(ctypes.byref(shape), ctypes.c_int32(n_ranks), ctypes.c_void_p(out.data_ptr())))
    return out


def sparsp_placement_contiguous(shape: sparsp_shape, n_ranks: int) -> torch.Tensor:
    return _placement(lib().sparsp_placement_contiguous, shape, n_ranks)


def sparsp_placement_periodic(shape: sparsp_shape, n_ranks: int) -> torch.Tensor:
    return _placement(lib().sparsp_placement_periodic, shape, n_ranks)


def sparsp_placement_permutation(shape: sparsp_shape, n_ranks: int, rank_of_block: torch.Tensor):
    """-> (block_of_slot int32 [NB], token_offset_of_slot int64 [NB+1], first_slot_of_rank int32 [P+1]), host."""
    g = sparsp_geometry(shape)
    rank = rank_of_block.to(torch.int32).cpu().contiguous()
    bos = torch.empty(g.n_blocks, dtype=torch.int32)
    off = torch.empty(g.n_blocks + 1, dtype=torch.int64)
    first = torch.empty(n_ranks + 1, dtype=torch.int32)
    _check(lib().sparsp_placement_permutation(ctypes.byref(shape), ctypes.c_int32(n_ranks),
                                              ctypes.c_void_p(rank.data_ptr()), ctypes.c_void_p(bos.data_ptr()),
                                              ctypes.c_void_p(off.data_ptr()), ctypes.c_void_p(first.data_ptr())))
    return bos, off, first


class sparsp_transfer(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("consumer", ctypes.c_int32), ("producer", ctypes.c_int32),
                ("round", ctypes.c_int32), ("order", ctypes.c_int32), ("head_begin", ctypes.c_int32),
                ("head_end", ctypes.c_int32), ("reserved", ctypes.c_int32), ("entry_begin", ctypes.c_int64),
                ("n_entries", ctypes.c_int64), ("byte_offset", ctypes.c_int64), ("n_bytes", ctypes.c_int64)]


def sparsp_exchange_plan(shape: sparsp_shape, n_ranks: int, cnt: torch.Tensor, seg_offset: torch.Tensor,
                         steady_chunks: int = 1, tail_chunks: int = 1):
    """-> list of sparsp_transfer (host).  cnt / seg_offset: sparsp_demand_pack's outputs (any device)."""
    c = cnt.to(torch.int32).cpu().contiguous()
    o = seg_offset.to(torch.int64).cpu().contiguous()
    n = ctypes.c_int64(0)
    args = (ctypes.byref(shape), ctypes.c_int32(n_ranks), ctypes.c_void_p(c.data_ptr()),
            ctypes.c_void_p(o.data_ptr()), ctypes.c_int32(steady_chunks), ctypes.c_int32(tail_chunks))
    rc = lib().sparsp_exchange_plan(*args, None, ctypes.c_int64(0), ctypes.byref(n))
    if rc not in (SPARSP_OK, SPARSP_ERR_CAPACITY):
        _check(rc)
    buf = (sparsp_transfer * max(n.value, 1))()
    _check(lib().sparsp_exchange_plan(*args, buf, ctypes.c_int64(n.value), ctypes.byref(n)))
    return list(buf[:n.value])


def sparsp_permute_tokens(shape, X, Y, block_of_slot, token_offset_of_slot, inverse):
    _check(lib().sparsp_permute_tokens(ctypes.byref(shape), _ptr(X), _ptr(Y), _ptr(block_of_slot),
                                       _ptr(token_offset_of_slot), ctypes.c_int32(1 if inverse else 0), _stream()))


def sparsp_sharing_histogram(shape, mask, rank_of_block, n_ranks, hist):
    _check(lib().sparsp_sharing_histogram(ctypes.byref(shape), _ptr(mask), _ptr(rank_of_block),
                                          ctypes.c_int32(n_ranks), _ptr(hist), _stream()))


def sparsp_workspace_bytes(shape: sparsp_shape, n_ranks: int) -> int:
    out = ctypes.c_int64()
    _check(lib().sparsp_workspace_bytes(ctypes.byref(shape), ctypes.c_int32(n_ranks), ctypes.byref(out)))
    return out.value


def make_workspace(shape: sparsp_shape, n_ranks: int, device="cuda") -> torch.Tensor:
    """Allocates a workspace (torch owns the memory) with its header zero-filled."""
    ws = torch.empty(sparsp_workspace_bytes(shape, n_ranks), dtype=torch.uint8, device=device)
    ws[:256].zero_()
    return ws


def sparsp_block_mask(shape, Q, K, topk_video, mask, kv_list, kv_count, pooled_q, pooled_k, workspace):
    _check(lib().sparsp_block_mask(ctypes.byref(shape), _ptr(Q), _ptr(K), ctypes.c_int32(topk_video),
                                   _ptr(mask), _ptr(kv_list), _ptr(kv_count), _ptr(pooled_q),
                                   _ptr(pooled_k), _ptr(workspace), _stream()))


def sparsp_block_mask_cdf(shape, Q, K, tau, score_scale, mask, kv_count, pooled_q, pooled_k, workspace):
    _check(lib().sparsp_block_mask_cdf(ctypes.byref(shape), _ptr(Q), _ptr(K), ctypes.c_float(tau),
                                       ctypes.c_float(score_scale), _ptr(mask), _ptr(kv_count), _ptr(pooled_q),
                                       _ptr(pooled_k), _ptr(workspace), _stream()))


def sparsp_demand_pack(shape, mask, rank_of_block, n_ranks, flags, K, V, union_mask, cnt, seg_offset,
                       seg_total, volume_bytes, packed, packed_capacity_bytes, dst_base_bytes, workspace):
    _check(lib().sparsp_demand_pack(ctypes.byref(shape), _ptr(mask), _ptr(rank_of_block),
                                    ctypes.c_int32(n_ranks), ctypes.c_int32(flags), _ptr(K), _ptr(V),
                                    _ptr(union_mask), _ptr(cnt), _ptr(seg_offset), _ptr(seg_total),
                                    _ptr(volume_bytes), _ptr(packed), ctypes.c_int64(packed_capacity_bytes),
                                    _ptr(dst_base_bytes), _ptr(workspace), _stream()))


def sparsp_demand_plan_noalloc(shape, mask, rank_of_block, n_ranks, flags, union_mask, cnt, seg_offset, seg_total,
                               volume_bytes):
    """Planning half of sparsp_demand_pack for callers that cannot allocate device memory: no workspace
    argument, the scratch is a small array inside the library.  Outputs as for SPARSP_PLAN_ONLY."""
    _check(lib().sparsp_demand_plan_noalloc(ctypes.byref(shape), _ptr(mask), _ptr(rank_of_block),
                                            ctypes.c_int32(n_ranks), ctypes.c_int32(flags), _ptr(union_mask),
                                            _ptr(cnt), _ptr(seg_offset), _ptr(seg_total), _ptr(volume_bytes),
                                            _stream()))


def sparsp_sparse_attn_fwd(shape, Q, K, V, mask, softmax_scale, O, lse, workspace):
    _check(lib().sparsp_sparse_attn_fwd(ctypes.byref(shape), _ptr(Q), _ptr(K), _ptr(V), _ptr(mask),
                                        ctypes.c_float(softmax_scale), _ptr(O), _ptr(lse), _ptr(workspace),
                                        _stream()))


def sparsp_sparse_attn_fwd_packed(shape, Q, K, V, mask, rank_of_block, n_ranks, consumer, union_mask, seg_offset,
                                  seg_total, packed, packed_capacity_bytes, dst_base_bytes, softmax_scale, O, lse,
                                  workspace):
    _check(lib().sparsp_sparse_attn_fwd_packed(ctypes.byref(shape), _ptr(Q), _ptr(K), _ptr(V), _ptr(mask),
                                               _ptr(rank_of_block), ctypes.c_int32(n_ranks), ctypes.c_int32(consumer),
                                               _ptr(union_mask), _ptr(seg_offset), _ptr(seg_total), _ptr(packed),
                                               ctypes.c_int64(packed_capacity_bytes), _ptr(dst_base_bytes),
                                               ctypes.c_float(softmax_scale), _ptr(O), _ptr(lse), _ptr(workspace),
                                               _stream()))


def sparsp_hop_mask(shape, mask, rank_of_block, n_ranks, consumer, producer, hop_mask):
    _check(lib().sparsp_hop_mask(ctypes.byref(shape), _ptr(mask), _ptr(rank_of_block), ctypes.c_int32(n_ranks),
                                 ctypes.c_int32(consumer), ctypes.c_int32(producer), _ptr(hop_mask), _stream()))


def sparsp_hop_chunk_mask(shape, mask, rank_of_block, n_ranks, consumer, producer, head_begin, head_end, hop_mask):
    _check(lib().sparsp_hop_chunk_mask(ctypes.byref(shape), _ptr(mask), _ptr(rank_of_block), ctypes.c_int32(n_ranks),
                                       ctypes.c_int32(consumer), ctypes.c_int32(producer), ctypes.c_int32(head_begin),
                                       ctypes.c_int32(head_end), _ptr(hop_mask), _stream()))


def sparsp_attn_merge(shape, O_a, lse_a, O_b, lse_b, O, lse):
    _check(lib().sparsp_attn_merge(ctypes.byref(shape), _ptr(O_a), _ptr(lse_a), _ptr(O_b), _ptr(lse_b), _ptr(O),
                                   _ptr(lse), _stream()))


def sparsp_attn_merge_rows(shape, O_a, lse_a, O_b, lse_b, O, lse, rank_of_block, n_ranks, consumer, head_begin,
                           head_end):
    _check(lib().sparsp_attn_merge_rows(ctypes.byref(shape), _ptr(O_a), _ptr(lse_a), _ptr(O_b), _ptr(lse_b), _ptr(O),
                                        _ptr(lse), _ptr(rank_of_block), ctypes.c_int32(n_ranks),
                                        ctypes.c_int32(consumer), ctypes.c_int32(head_begin), ctypes.c_int32(head_end),
                                        _stream()))


def _addr(x):
    """Raw address: an int, a torch tensor (its data pointer) or None."""
    if x is None:
        return ctypes.c_void_p(0)
    if isinstance(x, int):
        return ctypes.c_void_p(x)
    return ctypes.c_void_p(x.data_ptr())


def _stream_of(stream):
    """cudaStream_t of a torch stream (None: the current stream; 0: no stream, host-memory endpoints)."""
    if stream is None:
        return _stream()
    if isinstance(stream, int):
        return ctypes.c_void_p(stream)
    return ctypes.c_void_p(stream.cuda_stream)


def sparsp_pack_segment(shape, union_mask, rank_of_block, n_ranks, consumer, producer, cnt, seg_offset, K, V, dst,
                        dst_capacity_bytes, workspace):
    """dst: a tensor or a raw device address (a slot of the producer's window)."""
    _check(lib().sparsp_pack_segment(ctypes.byref(shape), _ptr(union_mask), _ptr(rank_of_block),
                                     ctypes.c_int32(n_ranks), ctypes.c_int32(consumer), ctypes.c_int32(producer),
                                     _ptr(cnt), _ptr(seg_offset), _ptr(K), _ptr(V), _addr(dst),
                                     ctypes.c_int64(dst_capacity_bytes), _ptr(workspace), _stream()))


def sparsp_xchg_flag_bytes(n_ranks: int, window: int) -> int:
    out = ctypes.c_int64()
    _check(lib().sparsp_xchg_flag_bytes(ctypes.c_int32(n_ranks), ctypes.c_int32(window), ctypes.byref(out)))
    return out.value


def sparsp_xchg_export(n_ranks, rank, window, slot_bytes, slots, flag_page, wait_limit_us, flags=0):
    """-> endpoint handle.  slots / flag_page: tensors or raw addresses."""
    h = ctypes.c_void_p()
    _check(lib().sparsp_xchg_export(ctypes.c_int32(n_ranks), ctypes.c_int32(rank), ctypes.c_int32(window),
                                    ctypes.c_int64(slot_bytes), _addr(slots), _addr(flag_page),
                                    ctypes.c_int64(wait_limit_us), ctypes.c_int32(flags), ctypes.byref(h)))
    return h


def sparsp_xchg_connect(x, peer, peer_slots):
    _check(lib().sparsp_xchg_connect(x, ctypes.c_int32(peer), _addr(peer_slots)))


def sparsp_xchg_fence(x):
    _check(lib().sparsp_xchg_fence(x))


def sparsp_xchg_acquire(x, use):
    """-> (slot index, slot address)"""
    slot, ptr = ctypes.c_int32(), ctypes.c_void_p()
    _check(lib().sparsp_xchg_acquire(x, ctypes.c_int64(use), ctypes.byref(slot), ctypes.byref(ptr)))
    return slot.value, ptr.value


def sparsp_xchg_publish(x, use, stream=None):
    _check(lib().sparsp_xchg_publish(x, ctypes.c_int64(use), _stream_of(stream)))


def sparsp_xchg_fetch(x, producer, use, src_offset, dst, n_bytes, copy_stream=None):
    _check(lib().sparsp_xchg_fetch(x, ctypes.c_int32(producer), ctypes.c_int64(use), ctypes.c_int64(src_offset),
                                   _addr(dst), ctypes.c_int64(n_bytes), _stream_of(copy_stream)))


def sparsp_xchg_release(x, producer, use, copy_stream=None):
    _check(lib().sparsp_xchg_release(x, ctypes.c_int32(producer), ctypes.c_int64(use), _stream_of(copy_stream)))


def sparsp_xchg_stats(x) -> dict:
    out = (ctypes.c_int64 * 8)()
    _check(lib().sparsp_xchg_stats(x, out))
    names = ("publications", "fetches", "releases", "acquires_that_waited", "bytes_fetched", "us_waiting_for_release",
             "us_waiting_for_publish", "timeouts")
    return dict(zip(names, [int(v) for v in out]))


def sparsp_xchg_destroy(x):
    _check(lib().sparsp_xchg_destroy(x))


def sparsp_status(workspace) -> int:
    code = ctypes.c_int32()
    _check(lib().sparsp_status(_ptr(workspace), _stream(), ctypes.byref(code)))
    return code.value


def sparsp_selftest_wait_timeout(workspace, limit_cycles: int):
    _check(lib().sparsp_selftest_wait_timeout(_ptr(workspace), ctypes.c_int64(limit_cycles), _stream()))


def sparsp_last_error() -> str:
    return lib().sparsp_last_error().decode()


def sparsp_launch_count() -> int:
    return int(lib().sparsp_launch_count())


# ---------------------------------------------------------------------------------------------
# allocation helpers (device buffers for the outputs; no arithmetic)
# ---------------------------------------------------------------------------------------------
def alloc_mask_outputs(shape: sparsp_shape, topk_video: int, device="cuda", with_list=True, with_pooled=False):
    g = sparsp_geometry(shape)
    B, H, d = shape.batch, shape.heads, shape.head_dim
    kept = topk_video + (g.n_blocks - g.n_video_blocks)
    out = dict(mask=torch.empty(B, H, g.n_blocks, g.n_words, dtype=torch.int32, device=device))
    out["kv_list"] = torch.full((B, H, g.n_blocks, kept), -1, dtype=torch.int32, device=device) if with_list else None
    out["kv_count"] = torch.empty(B, H, g.n_blocks, dtype=torch.int32, device=device) if with_list else None
    out["pooled_q"] = torch.empty(B, H, g.n_blocks, d, dtype=torch.float32, device=device) if with_pooled else None
    out["pooled_k"] = torch.empty(B, H, g.n_blocks, d, dtype=torch.float32, device=device) if with_pooled else None
    return out


def alloc_demand_outputs(shape: sparsp_shape, n_ranks: int, device="cuda"):
    g = sparsp_geometry(shape)
    B, H, P = shape.batch, shape.heads, n_ranks
    return dict(union_mask=torch.empty(B, P, H, g.n_words, dtype=torch.int32, device=device),
                cnt=torch.empty(B, P, P, H, dtype=torch.int32, device=device),
                seg_offset=torch.empty(B, P, P, H, dtype=torch.int64, device=device),
                seg_total=torch.empty(B, P, dtype=torch.int64, device=device),
                volume_bytes=torch.empty(B, P, dtype=torch.int64, device=device))
