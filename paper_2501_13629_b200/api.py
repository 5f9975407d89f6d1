"""ctypes binding of ``libdiffqkv.so``: same entry-point names as ``include/diffqkv.h``.

Argument marshalling only.  Every step of the attention path runs in the library's CUDA
kernels; torch is used for device memory, streams and host<->device copies.  Importing this
module loads the library and raises if it has not been built -- there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdiffqkv.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2501_13629_b200.build` "
        "(there is no CPU or PyTorch fallback)")
_lib = C.CDLL(LIB_PATH)

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_INDEX = range(8)
BF16, F32 = 0, 1

EXPORTS = (
    "diffqkv_decode_num_splits", "diffqkv_decode_workspace_bytes", "diffqkv_decode", "gqa_decode",
    "diffqkv_combine", "diffqkv_prefill", "diffqkv_augq_workspace_bytes", "diffqkv_augq",
    "diffqkv_status_string", "diffqkv_launch_count", "diffqkv_profile_split_events", "diffqkv_decode_static",
    "diffqkv_set_max_blocks", "diffqkv_topk_general_only", "diffqkv_last_decode_kernel",
    "diffqkv_last_prefill_kernel", "diffqkv_force_tensor_gemm", "diffqkv_augq_rope", "diffqkv_project", "diffqkv_cache_append",
    "diffqkv_decode_topk", "diffqkv_decode_topk_workspace_bytes", "diffqkv_decode_frontend",
    "diffqkv_decode_frontend_workspace_bytes", "diffqkv_decode_host", "diffqkv_fold_k_up",
    "diffqkv_set_tail_reserve", "diffqkv_debug_decode_timeout", "diffqkv_decode_topk_ids", "diffqkv_debug_decode_per_head_only", "diffqkv_debug_decode_cluster",
)


class CacheStruct(C.Structure):
    _fields_ = [
        ("k_cache", C.c_void_p), ("v_cache", C.c_void_p),
        ("k_stride_blk", C.c_int64), ("k_stride_head", C.c_int64), ("k_stride_tok", C.c_int64),
        ("v_stride_blk", C.c_int64), ("v_stride_head", C.c_int64), ("v_stride_tok", C.c_int64),
        ("seqlens", C.c_void_p), ("page_table", C.c_void_p),
        ("page_size", C.c_int32), ("max_pages_per_seq", C.c_int32),
        ("num_blocks", C.c_int32), ("max_seqlen", C.c_int32),
    ]


class ShapeStruct(C.Structure):
    _fields_ = [
        ("batch", C.c_int32), ("n_q", C.c_int32), ("n_k", C.c_int32), ("n_v", C.c_int32),
        ("d_qk", C.c_int32), ("d_v", C.c_int32),
        ("dtype", C.c_int), ("out_dtype", C.c_int), ("scale", C.c_float),
    ]


_lib.diffqkv_decode_num_splits.restype = C.c_int32
_lib.diffqkv_decode_num_splits.argtypes = [C.POINTER(ShapeStruct), C.c_int32]
_lib.diffqkv_decode_workspace_bytes.restype = C.c_size_t
_lib.diffqkv_decode_workspace_bytes.argtypes = [C.POINTER(ShapeStruct), C.c_int32, C.c_int32]
_DECODE_ARGS = [C.c_void_p, C.POINTER(CacheStruct), C.POINTER(ShapeStruct), C.c_int32, C.c_void_p, C.c_size_t,
                C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
for _name in ("diffqkv_decode", "gqa_decode"):
    getattr(_lib, _name).restype = C.c_int
    getattr(_lib, _name).argtypes = _DECODE_ARGS
_lib.diffqkv_decode_static.restype = C.c_int
_lib.diffqkv_decode_static.argtypes = [C.c_void_p, C.POINTER(CacheStruct), C.POINTER(ShapeStruct), C.c_int32,
                                       C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
_lib.diffqkv_combine.restype = C.c_int
_lib.diffqkv_combine.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int,
                                 C.c_void_p, C.c_void_p, C.c_void_p]
_lib.diffqkv_prefill.restype = C.c_int
_lib.diffqkv_prefill.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.POINTER(CacheStruct),
                                 C.POINTER(ShapeStruct), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
_lib.diffqkv_augq_workspace_bytes.restype = C.c_size_t
_lib.diffqkv_augq_workspace_bytes.argtypes = [C.c_int64, C.c_int32, C.c_int32]
_lib.diffqkv_augq.restype = C.c_int
_lib.diffqkv_augq.argtypes = [C.c_void_p] * 5 + [C.c_int64, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                                 C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p, C.c_void_p]
_lib.diffqkv_augq_rope.restype = C.c_int
_lib.diffqkv_augq_rope.argtypes = [C.c_void_p] * 5 + [C.c_int64, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                                      C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p,
                                                      C.c_void_p, C.c_void_p]
_lib.diffqkv_project.restype = C.c_int
_lib.diffqkv_project.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_int32, C.c_int32, C.c_void_p,
                                 C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
_lib.diffqkv_cache_append.restype = C.c_int
_lib.diffqkv_cache_append.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.POINTER(CacheStruct), C.POINTER(ShapeStruct),
                                      C.c_void_p, C.c_void_p]
_lib.diffqkv_decode_topk_workspace_bytes.restype = C.c_size_t
_lib.diffqkv_decode_topk_workspace_bytes.argtypes = [C.POINTER(ShapeStruct), C.c_int32, C.c_int32]
_lib.diffqkv_decode_topk_ids.restype = C.c_int
_lib.diffqkv_decode_topk_ids.argtypes = [C.c_void_p, C.POINTER(CacheStruct), C.POINTER(ShapeStruct), C.c_int32, C.c_void_p,
                                         C.c_size_t, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
_lib.diffqkv_decode_topk.restype = C.c_int
_lib.diffqkv_decode_topk.argtypes = [C.c_void_p, C.POINTER(CacheStruct), C.POINTER(ShapeStruct), C.c_int32, C.c_void_p,
                                     C.c_size_t, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
_lib.diffqkv_fold_k_up.restype = C.c_int
_lib.diffqkv_fold_k_up.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                   C.c_void_p, C.c_void_p]
_lib.diffqkv_status_string.restype = C.c_char_p
_lib.diffqkv_status_string.argtypes = [C.c_int]
_lib.diffqkv_launch_count.restype = C.c_int64
_lib.diffqkv_decode_frontend_workspace_bytes.restype = C.c_size_t
_lib.diffqkv_decode_frontend_workspace_bytes.argtypes = [C.POINTER(ShapeStruct), C.c_int32]
_lib.diffqkv_decode_frontend.restype = C.c_int32
_lib.diffqkv_decode_frontend.argtypes = [C.c_void_p] * 7 + [C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                         C.POINTER(CacheStruct), C.POINTER(ShapeStruct), C.c_void_p, C.c_size_t,
                                         C.c_void_p, C.c_void_p, C.c_void_p]
_lib.diffqkv_decode_host.restype = C.c_int32
_lib.diffqkv_decode_host.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(CacheStruct), C.POINTER(ShapeStruct), C.c_int32,
                                     C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
_lib.diffqkv_force_tensor_gemm.restype = None
_lib.diffqkv_force_tensor_gemm.argtypes = [C.c_int32]
_lib.diffqkv_last_prefill_kernel.restype = C.c_int32
_lib.diffqkv_last_prefill_kernel.argtypes = []
_lib.diffqkv_topk_general_only.restype = None
_lib.diffqkv_topk_general_only.argtypes = [C.c_int32]
_lib.diffqkv_debug_decode_per_head_only.restype = None
_lib.diffqkv_debug_decode_per_head_only.argtypes = [C.c_int32]
_lib.diffqkv_debug_decode_cluster.restype = None
_lib.diffqkv_debug_decode_cluster.argtypes = [C.c_int32]
_lib.diffqkv_debug_decode_timeout.restype = None
_lib.diffqkv_debug_decode_timeout.argtypes = [C.c_int64, C.c_int64]
_lib.diffqkv_set_tail_reserve.restype = None
_lib.diffqkv_set_tail_reserve.argtypes = [C.c_int32]
_lib.diffqkv_set_max_blocks.restype = None
_lib.diffqkv_set_max_blocks.argtypes = [C.c_int32]
_lib.diffqkv_profile_split_events.restype = None
_lib.diffqkv_profile_split_events.argtypes = [C.c_void_p, C.c_void_p]


class DiffQKVError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


def status_string(status: int) -> str:
    return _lib.diffqkv_status_string(int(status)).decode()


def launch_count() -> int:
    return int(_lib.diffqkv_launch_count())


def set_split_events(before: Optional[torch.cuda.Event], after: Optional[torch.cuda.Event]) -> None:
    """Benchmark hook: have decode calls record these events around their split kernel (None, None = off)."""
    _lib.diffqkv_profile_split_events(None if before is None else C.c_void_p(before.cuda_event),
                                      None if after is None else C.c_void_p(after.cuda_event))


def topk_general_only(on: bool) -> None:
    """Test hook: make diffqkv_decode_topk always select over all scores of a row; see diffqkv_topk_general_only."""
    _lib.diffqkv_topk_general_only(int(bool(on)))


def set_max_blocks(n: int) -> None:
    """Cap the persistent blocks of the TMA decode kernel (0 = one per SM); see diffqkv_set_max_blocks."""
    _lib.diffqkv_set_max_blocks(int(n))


KERNEL_NONE, KERNEL_GENERIC, KERNEL_TMA = 0, 1, 2


def set_tail_reserve(tiles: int) -> None:
    """Tail balance of the TMA decode kernel: -1 automatic, 0 off (run-to-run bitwise reproducible), n tiles per block."""
    _lib.diffqkv_set_tail_reserve(int(tiles))


def decode_cluster(mode: int) -> None:
    """Test hook: on-chip merge of the TMA decode kernel (-1 automatic, 0 never, 1 whenever the shape allows)."""
    _lib.diffqkv_debug_decode_cluster(int(mode))


def decode_per_head_only(on: bool) -> None:
    """Test hook: the generic decode path never takes its unit kernel (one block per query head instead)."""
    _lib.diffqkv_debug_decode_per_head_only(1 if on else 0)


def debug_decode_timeout(wait_limit_ns: int = 0, skip_tile: int = -1) -> None:
    """Test hook of the TMA decode kernel: bound every device wait by ``wait_limit_ns`` and never request the copies of
    flat tile ``skip_tile`` (so that the wait for it runs out); (0, -1) restores the defaults."""
    _lib.diffqkv_debug_decode_timeout(int(wait_limit_ns), int(skip_tile))


def force_tensor_gemm(on: bool) -> None:
    """Test hook: make the projections always take the tensor-core GEMM; see diffqkv_force_tensor_gemm."""
    _lib.diffqkv_force_tensor_gemm(int(bool(on)))


def last_prefill_kernel() -> int:
    """0 = no prefill yet, 1 = generic kernel, 2 = tensor-core kernel (most recent diffqkv_prefill call)."""
    return int(_lib.diffqkv_last_prefill_kernel())


def last_decode_kernel() -> int:
    """0 none yet, 1 generic split kernel, 2 TMA split kernel."""
    return int(_lib.diffqkv_last_decode_kernel())


def _dtype_code(dt: torch.dtype) -> int:
    if dt == torch.bfloat16:
        return BF16
    if dt == torch.float32:
        return F32
    raise TypeError(f"unsupported dtype {dt}")


def _p(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream_ptr(stream: Optional[torch.cuda.Stream]):
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


@dataclass
class KVCache:
    """Device-side cache description (see ``diffqkv_cache`` in the header).

    ``k`` / ``v`` are the pools: contiguous ``[batch, heads, max_seqlen, d]`` or paged
    ``[pages, heads, page_size, d]`` by default; any other layout by passing explicit
    (blk, head, tok) element strides.
    """
    k: torch.Tensor
    v: torch.Tensor
    seqlens: torch.Tensor                      # int32 [batch], device
    max_seqlen: int
    page_table: Optional[torch.Tensor] = None  # int32 [batch, max_pages_per_seq], device
    page_size: int = 0
    k_strides: Optional[Tuple[int, int, int]] = None
    v_strides: Optional[Tuple[int, int, int]] = None
    num_blocks: Optional[int] = None

    def c_struct(self) -> CacheStruct:
        ks = self.k_strides or (self.k.stride(0), self.k.stride(1), self.k.stride(2))
        vs = self.v_strides or (self.v.stride(0), self.v.stride(1), self.v.stride(2))
        assert self.seqlens.dtype == torch.int32 and self.seqlens.is_contiguous()
        pt = self.page_table
        if pt is not None:
            assert pt.dtype == torch.int32 and pt.is_contiguous() and pt.dim() == 2
        nb = self.num_blocks if self.num_blocks is not None else self.k.shape[0]
        return CacheStruct(
            self.k.data_ptr(), self.v.data_ptr(), *map(int, ks), *map(int, vs),
            self.seqlens.data_ptr(), None if pt is None else pt.data_ptr(),
            int(self.page_size), 0 if pt is None else int(pt.shape[1]), int(nb), int(self.max_seqlen))


def make_shape(batch, n_q, n_k, n_v, d_qk, d_v, dtype: torch.dtype, out_dtype: torch.dtype, scale: float):
    return ShapeStruct(batch, n_q, n_k, n_v, d_qk, d_v, _dtype_code(dtype), _dtype_code(out_dtype), float(scale))


def diffqkv_decode_num_splits(shape: ShapeStruct, max_seqlen: int) -> int:
    return int(_lib.diffqkv_decode_num_splits(C.byref(shape), max_seqlen))


def diffqkv_decode_workspace_bytes(shape: ShapeStruct, max_seqlen: int, num_splits: int = 0) -> int:
    return int(_lib.diffqkv_decode_workspace_bytes(C.byref(shape), max_seqlen, num_splits))


def _decode(fn_name, q, cache: KVCache, n_k, n_v, scale, num_splits, workspace, out, lse, dev_status,
            out_dtype, stream):
    batch, n_q, d_qk = q.shape
    d_v = cache.v.shape[-1]
    out_dtype = out_dtype or (out.dtype if out is not None else q.dtype)
    shape = make_shape(batch, n_q, n_k, n_v, d_qk, d_v, q.dtype, out_dtype, scale)
    if workspace is None:
        nbytes = diffqkv_decode_workspace_bytes(shape, cache.max_seqlen, num_splits)
        workspace = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=q.device)
    if out is None:
        out = torch.empty((batch, n_q, d_v), dtype=out_dtype, device=q.device)
    cs = cache.c_struct()
    st = getattr(_lib, fn_name)(_p(q), C.byref(cs), C.byref(shape), int(num_splits), _p(workspace),
                                workspace.numel() * workspace.element_size(), _p(out), _p(lse),
                                _p(dev_status), _stream_ptr(stream))
    if st != OK:
        raise DiffQKVError(st, fn_name)
    return out


def diffqkv_decode(q: torch.Tensor, cache: KVCache, n_k: int, n_v: int, scale: float, num_splits: int = 0,
                   workspace: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None,
                   lse: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None,
                   out_dtype: Optional[torch.dtype] = None, stream: Optional[torch.cuda.Stream] = None):
    """q [batch, n_q, d_qk] against the cache; returns out [batch, n_q, d_v] (enqueued on the stream)."""
    return _decode("diffqkv_decode", q, cache, n_k, n_v, scale, num_splits, workspace, out, lse, dev_status,
                   out_dtype, stream)


def bind_decode(q: torch.Tensor, cache: KVCache, n_k: int, n_v: int, scale: float, workspace: torch.Tensor,
                out: torch.Tensor, num_splits: int = 0, lse: Optional[torch.Tensor] = None,
                dev_status: Optional[torch.Tensor] = None, gqa: bool = False):
    """diffqkv_decode (or gqa_decode) with its argument structs built once: returns a function of no arguments that
    makes the library call on the current stream, as a C caller that keeps its diffqkv_shape / diffqkv_cache around
    does (a decode step of a few microseconds is otherwise bounded by the marshalling here, not by the GPU).  The
    tensors must stay alive and unmoved while the function is in use."""
    batch, n_q, d_qk = q.shape
    shape = make_shape(batch, n_q, n_k, n_v, d_qk, cache.v.shape[-1], q.dtype, out.dtype, scale)
    cs = cache.c_struct()
    fn = _lib.gqa_decode if gqa else _lib.diffqkv_decode
    name = "gqa_decode" if gqa else "diffqkv_decode"
    args = (_p(q), C.byref(cs), C.byref(shape), int(num_splits), _p(workspace),
            workspace.numel() * workspace.element_size(), _p(out), _p(lse), _p(dev_status))
    keep = (shape, cs, q, cache, workspace, out, lse, dev_status)

    def call():
        st = fn(*args, C.c_void_p(torch.cuda.current_stream().cuda_stream))
        if st != OK:
            raise DiffQKVError(st, name)
        return keep[5]

    return call


def diffqkv_decode_host(q_host: torch.Tensor, q_dev: torch.Tensor, cache: KVCache, n_k: int, n_v: int, scale: float,
                        workspace: torch.Tensor, out_dev: torch.Tensor, out_host: torch.Tensor, num_splits: int = 0,
                        lse: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None,
                        stream: Optional[torch.cuda.Stream] = None):
    """diffqkv_decode with the query in (pinned) host memory and the result copied back to (pinned) host memory, all on
    the stream and in one library call; q_dev / out_dev are the device staging buffers.  Returns out_host, which
    is valid once the stream has been synchronised."""
    batch, n_q, d_qk = q_host.shape
    assert not q_host.is_cuda and not out_host.is_cuda and q_dev.is_cuda and out_dev.is_cuda
    shape = make_shape(batch, n_q, n_k, n_v, d_qk, cache.v.shape[-1], q_host.dtype, out_host.dtype, scale)
    cs = cache.c_struct()
    st = _lib.diffqkv_decode_host(_p(q_host), _p(q_dev), C.byref(cs), C.byref(shape), int(num_splits), _p(workspace),
                                  workspace.numel(), _p(out_dev), _p(out_host), _p(lse), _p(dev_status),
                                  _stream_ptr(stream))
    if st != OK:
        raise DiffQKVError(st, "diffqkv_decode_host")
    return out_host


def bind_decode_host(q_host: torch.Tensor, q_dev: torch.Tensor, cache: KVCache, n_k: int, n_v: int, scale: float,
                     workspace: torch.Tensor, out_dev: torch.Tensor, out_host: torch.Tensor, num_splits: int = 0,
                     lse: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None):
    """diffqkv_decode_host with its argument structs built once: returns a function of no arguments that makes the
    library call on the current stream (what a C caller that keeps its diffqkv_shape / diffqkv_cache around does).
    The tensors must stay alive and unmoved while the function is in use."""
    batch, n_q, d_qk = q_host.shape
    assert not q_host.is_cuda and not out_host.is_cuda and q_dev.is_cuda and out_dev.is_cuda
    shape = make_shape(batch, n_q, n_k, n_v, d_qk, cache.v.shape[-1], q_host.dtype, out_host.dtype, scale)
    cs = cache.c_struct()
    args = (_p(q_host), _p(q_dev), C.byref(cs), C.byref(shape), int(num_splits), _p(workspace), workspace.numel(),
            _p(out_dev), _p(out_host), _p(lse), _p(dev_status))
    keep = (shape, cs, q_host, q_dev, cache, workspace, out_dev, out_host, lse, dev_status)

    def call():
        st = _lib.diffqkv_decode_host(*args, C.c_void_p(torch.cuda.current_stream().cuda_stream))
        if st != OK:
            raise DiffQKVError(st, "diffqkv_decode_host")
        return keep[7]

    return call


STATIC_SCRATCH_BYTES = 8 << 20


def diffqkv_decode_static(q: torch.Tensor, cache: KVCache, n_k: int, n_v: int, scale: float, out: torch.Tensor,
                          num_splits: int = 0, lse: Optional[torch.Tensor] = None,
                          dev_status: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
    """diffqkv_decode for callers that must not allocate: the split partials go to the 8 MiB array built
    into the library, and ``out`` has to be passed in (this wrapper allocates nothing either).  Raises
    DiffQKVError(ERR_WORKSPACE) when the shape needs more than STATIC_SCRATCH_BYTES.  Calls on one stream
    are ordered; calls that can overlap on the GPU share the array and race."""
    batch, n_q, d_qk = q.shape
    shape = make_shape(batch, n_q, n_k, n_v, d_qk, cache.v.shape[-1], q.dtype, out.dtype, scale)
    cs = cache.c_struct()
    st = _lib.diffqkv_decode_static(_p(q), C.byref(cs), C.byref(shape), int(num_splits), _p(out), _p(lse),
                                    _p(dev_status), _stream_ptr(stream))
    if st != OK:
        raise DiffQKVError(st, "diffqkv_decode_static")
    return out


def gqa_decode(q: torch.Tensor, cache: KVCache, n_kv: int, scale: float, num_splits: int = 0,
               workspace: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None,
               lse: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None,
               out_dtype: Optional[torch.dtype] = None, stream: Optional[torch.cuda.Stream] = None):
    """Grouped-query attention (n_k == n_v == n_kv) through the same kernels."""
    return _decode("gqa_decode", q, cache, n_kv, n_kv, scale, num_splits, workspace, out, lse, dev_status,
                   out_dtype, stream)


def diffqkv_combine(o_partial: torch.Tensor, lse_partial: torch.Tensor, out_dtype: torch.dtype = torch.float32,
                    out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None,
                    stream: Optional[torch.cuda.Stream] = None):
    """o_partial [batch, n_q, S, d_v] fp32, lse_partial [batch, n_q, S] fp32 -> out [batch, n_q, d_v]."""
    batch, n_q, S, d_v = o_partial.shape
    assert o_partial.dtype == torch.float32 and lse_partial.dtype == torch.float32
    assert o_partial.is_contiguous() and lse_partial.is_contiguous()
    if out is None:
        out = torch.empty((batch, n_q, d_v), dtype=out_dtype, device=o_partial.device)
    st = _lib.diffqkv_combine(_p(o_partial), _p(lse_partial), batch, n_q, d_v, S, _dtype_code(out.dtype),
                              _p(out), _p(lse), _stream_ptr(stream))
    if st != OK:
        raise DiffQKVError(st, "diffqkv_combine")
    return out


def diffqkv_prefill(q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor, cache: KVCache, scale: float,
                    out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None,
                    dev_status: Optional[torch.Tensor] = None, out_dtype: Optional[torch.dtype] = None,
                    stream: Optional[torch.cuda.Stream] = None):
    """q [batch, q_len, n_q, d_qk]; writes k_new / v_new into the cache, returns out [batch, q_len, n_q, d_v]."""
    batch, q_len, n_q, d_qk = q.shape
    n_k, n_v, d_v = k_new.shape[2], v_new.shape[2], v_new.shape[3]
    out_dtype = out_dtype or (out.dtype if out is not None else q.dtype)
    shape = make_shape(batch, n_q, n_k, n_v, d_qk, d_v, q.dtype, out_dtype, scale)
    if out is None:
        out = torch.empty((batch, q_len, n_q, d_v), dtype=out_dtype, device=q.device)
    cs = cache.c_struct()
    st = _lib.diffqkv_prefill(_p(q), _p(k_new), _p(v_new), q_len, C.byref(cs), C.byref(shape), _p(out), _p(lse),
                              _p(dev_status), _stream_ptr(stream))
    if st != OK:
        raise DiffQKVError(st, "diffqkv_prefill")
    return out


def diffqkv_augq_workspace_bytes(T: int, d_q0: int, d_aug: int) -> int:
    return int(_lib.diffqkv_augq_workspace_bytes(T, d_q0, d_aug))


def diffqkv_augq(h: torch.Tensor, W_Q: torch.Tensor, W_gate: torch.Tensor, W_up: torch.Tensor,
                 W_down: torch.Tensor, workspace: Optional[torch.Tensor] = None,
                 q_out: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
    """h [T, d_model] bf16, weights in nn.Linear layout [out, in]; returns q [T, d_out] bf16."""
    T, d_model = h.shape
    d_q0, d_aug, d_out = W_Q.shape[0], W_gate.shape[0], W_down.shape[0]
    if workspace is None:
        workspace = torch.empty(max(diffqkv_augq_workspace_bytes(T, d_q0, d_aug), 256), dtype=torch.uint8,
                                device=h.device)
    if q_out is None:
        q_out = torch.empty((T, d_out), dtype=torch.bfloat16, device=h.device)
    st = _lib.diffqkv_augq(_p(h), _p(W_Q), _p(W_gate), _p(W_up), _p(W_down), T, d_model, d_q0, d_aug, d_out,
                           _p(workspace), workspace.numel(), _p(q_out), _p(dev_status), _stream_ptr(stream))
    if st != OK:
        raise DiffQKVError(st, "diffqkv_augq")
    return q_out


def diffqkv_augq_rope(h: torch.Tensor, W_Q: torch.Tensor, W_gate: torch.Tensor, W_up: torch.Tensor,
                      W_down: torch.Tensor, head_dim: int, cos: torch.Tensor, sin: torch.Tensor,
                      workspace: Optional[torch.Tensor] = None, q_out: Optional[torch.Tensor] = None,
                      dev_status: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
    """diffqkv_augq with the rotary embedding fused into the last product; cos / sin [T, head_dim / 2] fp32."""
    T, d_model = h.shape
    d_q0, d_aug, d_out = W_Q.shape[0], W_gate.shape[0], W_down.shape[0]
    assert cos.dtype == torch.float32 and sin.dtype == torch.float32 and cos.is_contiguous() and sin.is_contiguous()
    assert tuple(cos.shape) == (T, head_dim // 2) and tuple(sin.shape) == (T, head_dim // 2)
    if workspace is None:
        workspace = torch.empty(max(diffqkv_augq_workspace_bytes(T, d_q0, d_aug), 256), dtype=torch.uint8,
                                device=h.device)
    if q_out is None:
        q_out = torch.empty((T, d_out), dtype=torch.bfloat16, device=h.device)
    st = _lib.diffqkv_augq_rope(_p(h), _p(W_Q), _p(W_gate), _p(W_up), _p(W_down), T, d_model, d_q0, d_aug, d_out,
                                int(head_dim), _p(cos), _p(sin), _p(workspace), workspace.numel(), _p(q_out),
                                _p(dev_status), _stream_ptr(stream))
    if st != OK:
        raise DiffQKVError(st, "diffqkv_augq_rope")
    return q_out


def diffqkv_project(x: torch.Tensor, W: torch.Tensor, head_dim: int = 0, cos: Optional[torch.Tensor] = None,
                    sin: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None,
                    dev_status: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
    """y = x W^T (W [d_out, d_in], bf16), rotated per head when cos / sin [T, head_dim / 2] fp32 are given."""
    T, d_in = x.shape
    d_out = W.shape[0]
    if cos is not None:
        assert cos.dtype == torch.float32 and sin.dtype == torch.float32 and cos.is_contiguous() and sin.is_contiguous()
        assert tuple(cos.shape) == (T, head_dim // 2) and tuple(sin.shape) == (T, head_dim // 2)
    if out is None:
        out = torch.empty((T, d_out), dtype=torch.bfloat16, device=x.device)
    st = _lib.diffqkv_project(_p(x), _p(W), T, d_in, d_out, int(head_dim), _p(cos), _p(sin), _p(out), _p(dev_status),
                              _stream_ptr(stream))
    if st != OK:
        raise DiffQKVError(st, "diffqkv_project")
    return out


def diffqkv_decode_frontend(h: torch.Tensor, W_Q: torch.Tensor, W_gate: torch.Tensor, W_up: torch.Tensor,
                            W_down: torch.Tensor, W_K: torch.Tensor, W_V: torch.Tensor, cache: KVCache, n_q: int,
                            d_qk: int, d_v: int, cos: Optional[torch.Tensor] = None,
                            sin: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                            q_out: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None,
                            stream: Optional[torch.cuda.Stream] = None):
    """One decode step's projections: returns q [batch, n_q, d_qk] = rope(aug-Q(h)) and writes the new token's
    k = rope(h W_K^T), v = h W_V^T into the cache at position seqlens[b] (seqlens is left as it is)."""
    batch, d_model = h.shape
    d_aug = W_gate.shape[0]
    n_k, n_v = W_K.shape[0] // d_qk, W_V.shape[0] // d_v
    assert W_Q.shape[0] == n_q * d_qk
    if cos is not None:
        assert cos.dtype == torch.float32 and sin.dtype == torch.float32 and cos.is_contiguous() and sin.is_contiguous()
        assert tuple(cos.shape) == (batch, d_qk // 2) and tuple(sin.shape) == (batch, d_qk // 2)
    shape = make_shape(batch, n_q, n_k, n_v, d_qk, d_v, h.dtype, h.dtype, 1.0)
    if workspace is None:
        nbytes = int(_lib.diffqkv_decode_frontend_workspace_bytes(C.byref(shape), d_aug))
        workspace = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=h.device)
    if q_out is None:
        q_out = torch.empty((batch, n_q, d_qk), dtype=torch.bfloat16, device=h.device)
    cs = cache.c_struct()
    st = _lib.diffqkv_decode_frontend(_p(h), _p(W_Q), _p(W_gate), _p(W_up), _p(W_down), _p(W_K), _p(W_V), d_model, d_aug,
                                      _p(cos), _p(sin), C.byref(cs), C.byref(shape), _p(workspace), workspace.numel(),
                                      _p(q_out), _p(dev_status), _stream_ptr(stream))
    if st != OK:
        raise DiffQKVError(st, "diffqkv_decode_frontend")
    return q_out


def diffqkv_cache_append(k_new: torch.Tensor, v_new: torch.Tensor, cache: KVCache,
                         dev_status: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
    """Write k_new [batch, q_len, n_k, d_qk] / v_new [batch, q_len, n_v, d_v] at positions seqlens[b] + i."""
    batch, q_len, n_k, d_qk = k_new.shape
    n_v, d_v = v_new.shape[2], v_new.shape[3]
    # the append does not involve query heads; any count both head counts divide satisfies the shape check
    shape = make_shape(batch, n_k * n_v, n_k, n_v, d_qk, d_v, k_new.dtype, k_new.dtype, 1.0)
    cs = cache.c_struct()
    st = _lib.diffqkv_cache_append(_p(k_new), _p(v_new), q_len, C.byref(cs), C.byref(shape), _p(dev_status),
                                   _stream_ptr(stream))
    if st != OK:
        raise DiffQKVError(st, "diffqkv_cache_append")


def diffqkv_fold_k_up(q: torch.Tensor, W_kup: torch.Tensor, out: Optional[torch.Tensor] = None,
                      stream: Optional[torch.cuda.Stream] = None):
    """q' = W_kup[hk]^T q per query head: q [..., n_q, d_q] bf16, W_kup [n_k, d_q, d_k] bf16 -> [..., n_q, d_k]."""
    n_k, d_q, d_k = W_kup.shape
    n_q = q.shape[-2]
    assert q.shape[-1] == d_q and q.is_contiguous() and W_kup.is_contiguous()
    T = q.numel() // (n_q * d_q)
    if out is None:
        out = torch.empty(q.shape[:-1] + (d_k,), dtype=torch.bfloat16, device=q.device)
    st = _lib.diffqkv_fold_k_up(_p(q), _p(W_kup), T, n_q, n_k, d_q, d_k, _p(out), _stream_ptr(stream))
    if st != OK:
        raise DiffQKVError(st, "diffqkv_fold_k_up")
    return out


def diffqkv_decode_topk(q: torch.Tensor, cache: KVCache, n_k: int, n_v: int, scale: float, topk: int,
                        workspace: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None,
                        lse: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None,
                        out_dtype: Optional[torch.dtype] = None, stream: Optional[torch.cuda.Stream] = None,
                        kept_ids: Optional[torch.Tensor] = None):
    """Decode that reads only the V rows of the `topk` highest scores of every query head; ``kept_ids`` (int32
    [batch, n_q, topk]) receives the kept tokens' positions, -1 padded."""
    batch, n_q, d_qk = q.shape
    d_v = cache.v.shape[-1]
    out_dtype = out_dtype or (out.dtype if out is not None else q.dtype)
    shape = make_shape(batch, n_q, n_k, n_v, d_qk, d_v, q.dtype, out_dtype, scale)
    if workspace is None:
        nbytes = int(_lib.diffqkv_decode_topk_workspace_bytes(C.byref(shape), cache.max_seqlen, int(topk)))
        workspace = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=q.device)
    if out is None:
        out = torch.empty((batch, n_q, d_v), dtype=out_dtype, device=q.device)
    cs = cache.c_struct()
    if kept_ids is not None:
        assert kept_ids.dtype == torch.int32 and kept_ids.is_contiguous() and tuple(kept_ids.shape) == (batch, n_q, topk)
    st = _lib.diffqkv_decode_topk_ids(_p(q), C.byref(cs), C.byref(shape), int(topk), _p(workspace), workspace.numel(),
                                      _p(out), _p(lse), _p(kept_ids), _p(dev_status), _stream_ptr(stream))
    if st != OK:
        raise DiffQKVError(st, "diffqkv_decode_topk")
    return out
