"""ctypes binding of include/fedattn.h.  Function names match the C entry points; torch tensors
supply device memory and the current CUDA stream."""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
# FEDATTN_LIBRARY overrides the path of the shared library (e.g. an instrumented build).
_LIB_PATH = os.environ.get("FEDATTN_LIBRARY") or os.path.join(_PKG, "lib", "libfedattn.so")

F32, BF16 = 0, 1
AGG_CONCAT, AGG_TOPK_KNORM, AGG_INDEXED, AGG_TOPK_TOKEN = 0, 1, 2, 3
DECODE_LOCAL, DECODE_SYNC = 0, 1

_SYMBOLS = ["fedattn_workspace_bytes", "fedattn_create", "fedattn_destroy", "fedattn_status_string",
            "fedattn_poll", "fedattn_launch_count", "fedattn_tensor_core_launch_count",
            "fedattn_selftest_wait_timeout", "fedattn_local", "fedattn_aggregate_kv",
            "fedattn_sync", "fedattn_sync_remote", "fedattn_merge", "fedattn_decode", "fedattn_decode_noalloc"]


class FedAttnError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s failed: %s (status %d)" % (where, status_string(code), code))


class Shape(C.Structure):
    """Mirror of fedattn_shape."""
    _fields_ = [("n_participants", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("dtype", C.c_int32), ("causal", C.c_int32), ("scale", C.c_float)]

    def __init__(self, n_participants, n_q_heads, n_kv_heads, head_dim, dtype, causal=1, scale=0.0):
        super().__init__(int(n_participants), int(n_q_heads), int(n_kv_heads), int(head_dim), int(dtype),
                         int(causal), float(scale))

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.dtype == BF16 else torch.float32


def library_path() -> str:
    return _LIB_PATH


def _load():
    if not os.path.exists(_LIB_PATH):
        raise ImportError("FedAttn CUDA library missing: %s (run `python paper_2511_02647_b200/build.py` "
                          "or __graft_entry__.build()); there is no fallback path" % _LIB_PATH)
    lib = C.CDLL(_LIB_PATH)
    vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
    lib.fedattn_workspace_bytes.restype = C.c_size_t
    lib.fedattn_workspace_bytes.argtypes = [C.POINTER(Shape), i64, i64]
    lib.fedattn_create.restype = C.c_int
    lib.fedattn_create.argtypes = [C.POINTER(vp), C.c_int, vp, C.c_size_t]
    lib.fedattn_destroy.restype = None
    lib.fedattn_destroy.argtypes = [vp]
    lib.fedattn_status_string.restype = C.c_char_p
    lib.fedattn_status_string.argtypes = [C.c_int]
    lib.fedattn_poll.restype = C.c_int
    lib.fedattn_poll.argtypes = [vp, vp]
    lib.fedattn_launch_count.restype = i64
    lib.fedattn_launch_count.argtypes = [vp]
    lib.fedattn_tensor_core_launch_count.restype = i64
    lib.fedattn_tensor_core_launch_count.argtypes = [vp]
    lib.fedattn_selftest_wait_timeout.restype = C.c_int
    lib.fedattn_selftest_wait_timeout.argtypes = [vp, i32, vp]
    lib.fedattn_local.restype = C.c_int
    lib.fedattn_local.argtypes = [vp, C.POINTER(Shape), vp, vp, vp, C.POINTER(i32), vp, vp, vp]
    lib.fedattn_aggregate_kv.restype = C.c_int
    lib.fedattn_aggregate_kv.argtypes = [vp, C.POINTER(Shape), i32, C.POINTER(vp), C.POINTER(vp),
                                         C.POINTER(i32), C.POINTER(i32), vp, vp, vp, vp, vp, vp, vp]
    lib.fedattn_sync.restype = C.c_int
    lib.fedattn_sync.argtypes = [vp, C.POINTER(Shape), vp, i64, vp, vp, vp, vp, i64, i32, vp, vp, vp]
    lib.fedattn_sync_remote.restype = C.c_int
    lib.fedattn_sync_remote.argtypes = [vp, C.POINTER(Shape), vp, C.POINTER(i32), vp, vp, vp, i64, i32, vp, vp, vp]
    lib.fedattn_merge.restype = C.c_int
    lib.fedattn_merge.argtypes = [vp, C.POINTER(Shape), i64, vp, vp, vp, vp, vp, vp, vp]
    lib.fedattn_decode.restype = C.c_int
    lib.fedattn_decode.argtypes = [vp, C.POINTER(Shape), i32, vp, vp, vp, i64, vp, i32, vp, vp, vp]
    lib.fedattn_decode_noalloc.restype = C.c_int
    lib.fedattn_decode_noalloc.argtypes = [C.POINTER(Shape), i32, vp, vp, vp, i64, vp, i32, vp, vp, vp]
    return lib


_lib = _load()


def exported_symbols():
    """Names declared in include/fedattn.h that the loaded library exports."""
    return [s for s in _SYMBOLS if hasattr(_lib, s)]


def status_string(code: int) -> str:
    return _lib.fedattn_status_string(int(code)).decode()


def _check(code: int, where: str):
    if code != 0:
        raise FedAttnError(code, where)


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _i32_array(xs: Sequence[int]):
    return (C.c_int32 * len(xs))(*[int(x) for x in xs])


def fedattn_workspace_bytes(shape: Shape, max_total_tokens: int, max_total_kv: int) -> int:
    return int(_lib.fedattn_workspace_bytes(C.byref(shape), int(max_total_tokens), int(max_total_kv)))


class Context:
    """Owns a device workspace tensor and the library context built around it."""

    def __init__(self, shape: Shape, max_total_tokens: int, max_total_kv: int, device: int = 0):
        nbytes = fedattn_workspace_bytes(shape, max_total_tokens, max_total_kv)
        if nbytes == 0:
            raise FedAttnError(1, "fedattn_workspace_bytes")
        self.device = int(device)
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device="cuda:%d" % self.device)
        self._h = C.c_void_p()
        _check(_lib.fedattn_create(C.byref(self._h), self.device, self.workspace.data_ptr(), nbytes),
               "fedattn_create")

    @property
    def handle(self):
        return self._h

    def poll(self, stream=None) -> int:
        """Synchronise the stream and return (and clear) the device status word."""
        return int(_lib.fedattn_poll(self._h, _stream(stream)))

    def launch_count(self) -> int:
        return int(_lib.fedattn_launch_count(self._h))

    def tensor_core_launch_count(self) -> int:
        return int(_lib.fedattn_tensor_core_launch_count(self._h))

    def selftest_wait_timeout(self, max_polls: int = 64, stream=None):
        """Launches the kernel whose bounded wait runs out (raises the TIMEOUT status word)."""
        _check(_lib.fedattn_selftest_wait_timeout(self._h, int(max_polls), _stream(stream)),
               "fedattn_selftest_wait_timeout")

    def close(self):
        if self._h:
            _lib.fedattn_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


# Every entry point comes in two forms: ``fedattn_x(...)`` marshals its arguments and calls the library;
# ``prepare_x(...)`` marshals once and returns a zero-argument callable that repeats the same call (same
# buffers, same stream), for loops in which the per-call marshalling of tensors and pointer arrays would
# cost more host time than the kernel takes on the device.  Both do argument marshalling only.
class PreparedCall:
    """A library call with its arguments already converted; calling it enqueues the work again."""

    def __init__(self, fn, args, where: str, keep):
        self._fn, self._args, self._where, self._keep = fn, args, where, keep

    def __call__(self, stream=None):
        # every entry point takes the stream last; `stream` (a raw cudaStream_t) replaces the prepared one
        code = self._fn(*self._args) if stream is None else self._fn(*self._args[:-1], stream)
        if code != 0:
            raise FedAttnError(code, self._where)


def _args_local(ctx, shape, q, k, v, cu_seqlens_host, o, lse, stream):
    cu = _i32_array(cu_seqlens_host)
    if len(cu) != shape.n_participants + 1:
        raise ValueError("cu_seqlens must have N+1 entries")
    return (ctx.handle, C.byref(shape), _ptr(q), _ptr(k), _ptr(v), cu, _ptr(o), _ptr(lse), _stream(stream))


def fedattn_local(ctx: Context, shape: Shape, q, k, v, cu_seqlens_host: Sequence[int], o, lse=None,
                  stream=None):
    _check(_lib.fedattn_local(*_args_local(ctx, shape, q, k, v, cu_seqlens_host, o, lse, stream)), "fedattn_local")


def prepare_local(ctx: Context, shape: Shape, q, k, v, cu_seqlens_host: Sequence[int], o, lse=None, stream=None):
    return PreparedCall(_lib.fedattn_local, _args_local(ctx, shape, q, k, v, cu_seqlens_host, o, lse, stream),
                        "fedattn_local", (ctx, shape, q, k, v, o, lse))


def _args_aggregate_kv(ctx, shape, mode, k_parts, v_parts, seqlens_host, k_sel_host, sel_idx_in, k_agg, v_agg, kv_pos,
                       cu_kv, sel_idx_out, stream):
    n = shape.n_participants
    if len(k_parts) != n or len(v_parts) != n or len(seqlens_host) != n:
        raise ValueError("need one K part, V part and length per participant")
    kp = (C.c_void_p * n)(*[_ptr(t) for t in k_parts])
    vp = (C.c_void_p * n)(*[_ptr(t) for t in v_parts])
    ks = None if k_sel_host is None else _i32_array(k_sel_host)
    return (ctx.handle, C.byref(shape), int(mode), kp, vp, _i32_array(seqlens_host), ks, _ptr(sel_idx_in), _ptr(k_agg),
            _ptr(v_agg), _ptr(kv_pos), _ptr(cu_kv), _ptr(sel_idx_out), _stream(stream))


def fedattn_aggregate_kv(ctx: Context, shape: Shape, mode: int, k_parts, v_parts, seqlens_host,
                         k_sel_host=None, sel_idx_in=None, k_agg=None, v_agg=None, kv_pos=None, cu_kv=None,
                         sel_idx_out=None, stream=None):
    _check(_lib.fedattn_aggregate_kv(*_args_aggregate_kv(ctx, shape, mode, k_parts, v_parts, seqlens_host, k_sel_host,
                                                         sel_idx_in, k_agg, v_agg, kv_pos, cu_kv, sel_idx_out, stream)),
           "fedattn_aggregate_kv")


def prepare_aggregate_kv(ctx: Context, shape: Shape, mode: int, k_parts, v_parts, seqlens_host, k_sel_host=None,
                         sel_idx_in=None, k_agg=None, v_agg=None, kv_pos=None, cu_kv=None, sel_idx_out=None, stream=None):
    return PreparedCall(_lib.fedattn_aggregate_kv,
                        _args_aggregate_kv(ctx, shape, mode, k_parts, v_parts, seqlens_host, k_sel_host, sel_idx_in, k_agg,
                                           v_agg, kv_pos, cu_kv, sel_idx_out, stream),
                        "fedattn_aggregate_kv", (ctx, shape, list(k_parts), list(v_parts), sel_idx_in, k_agg, v_agg, kv_pos,
                                                 cu_kv, sel_idx_out))


def _args_sync(ctx, shape, q, q_pos, k_agg, v_agg, kv_pos, total_kv, kv_head_major, o, lse, stream):
    return (ctx.handle, C.byref(shape), _ptr(q), int(q.shape[0]), _ptr(q_pos), _ptr(k_agg), _ptr(v_agg), _ptr(kv_pos),
            int(total_kv), int(bool(kv_head_major)), _ptr(o), _ptr(lse), _stream(stream))


def fedattn_sync(ctx: Context, shape: Shape, q, q_pos, k_agg, v_agg, kv_pos, total_kv: int,
                 kv_head_major: bool, o, lse=None, stream=None):
    _check(_lib.fedattn_sync(*_args_sync(ctx, shape, q, q_pos, k_agg, v_agg, kv_pos, total_kv, kv_head_major, o, lse,
                                         stream)), "fedattn_sync")


def prepare_sync(ctx: Context, shape: Shape, q, q_pos, k_agg, v_agg, kv_pos, total_kv: int, kv_head_major: bool, o,
                 lse=None, stream=None):
    return PreparedCall(_lib.fedattn_sync,
                        _args_sync(ctx, shape, q, q_pos, k_agg, v_agg, kv_pos, total_kv, kv_head_major, o, lse, stream),
                        "fedattn_sync", (ctx, shape, q, q_pos, k_agg, v_agg, kv_pos, o, lse))


def _args_sync_remote(ctx, shape, q, cu_seqlens_host, k_agg, v_agg, kv_pos, total_kv, kv_head_major, o, lse, stream):
    cu = _i32_array(cu_seqlens_host)
    if len(cu) != shape.n_participants + 1:
        raise ValueError("cu_seqlens must have N+1 entries")
    return (ctx.handle, C.byref(shape), _ptr(q), cu, _ptr(k_agg), _ptr(v_agg), _ptr(kv_pos), int(total_kv),
            int(bool(kv_head_major)), _ptr(o), _ptr(lse), _stream(stream))


def fedattn_sync_remote(ctx: Context, shape: Shape, q, cu_seqlens_host: Sequence[int], k_agg, v_agg, kv_pos,
                        total_kv: int, kv_head_major: bool, o, lse, stream=None):
    _check(_lib.fedattn_sync_remote(*_args_sync_remote(ctx, shape, q, cu_seqlens_host, k_agg, v_agg, kv_pos, total_kv,
                                                       kv_head_major, o, lse, stream)), "fedattn_sync_remote")


def prepare_sync_remote(ctx: Context, shape: Shape, q, cu_seqlens_host: Sequence[int], k_agg, v_agg, kv_pos, total_kv: int,
                        kv_head_major: bool, o, lse, stream=None):
    return PreparedCall(_lib.fedattn_sync_remote,
                        _args_sync_remote(ctx, shape, q, cu_seqlens_host, k_agg, v_agg, kv_pos, total_kv, kv_head_major, o,
                                          lse, stream),
                        "fedattn_sync_remote", (ctx, shape, q, k_agg, v_agg, kv_pos, o, lse))


def _args_merge(ctx, shape, n_rows, o_a, lse_a, o_b, lse_b, o, lse, stream):
    return (ctx.handle, C.byref(shape), int(n_rows), _ptr(o_a), _ptr(lse_a), _ptr(o_b), _ptr(lse_b), _ptr(o), _ptr(lse),
            _stream(stream))


def fedattn_merge(ctx: Context, shape: Shape, n_rows: int, o_a, lse_a, o_b, lse_b, o, lse=None, stream=None):
    _check(_lib.fedattn_merge(*_args_merge(ctx, shape, n_rows, o_a, lse_a, o_b, lse_b, o, lse, stream)), "fedattn_merge")


def prepare_merge(ctx: Context, shape: Shape, n_rows: int, o_a, lse_a, o_b, lse_b, o, lse=None, stream=None):
    return PreparedCall(_lib.fedattn_merge, _args_merge(ctx, shape, n_rows, o_a, lse_a, o_b, lse_b, o, lse, stream),
                        "fedattn_merge", (ctx, shape, o_a, lse_a, o_b, lse_b, o, lse))


def _args_decode(ctx, shape, mode, q, k_cache, v_cache, cache_stride_participant, kv_len, max_kv_len, o, lse, stream):
    return (ctx.handle, C.byref(shape), int(mode), _ptr(q), _ptr(k_cache), _ptr(v_cache), int(cache_stride_participant),
            _ptr(kv_len), int(max_kv_len), _ptr(o), _ptr(lse), _stream(stream))


def fedattn_decode(ctx: Context, shape: Shape, mode: int, q, k_cache, v_cache, cache_stride_participant: int,
                   kv_len, max_kv_len: int, o, lse=None, stream=None):
    _check(_lib.fedattn_decode(*_args_decode(ctx, shape, mode, q, k_cache, v_cache, cache_stride_participant, kv_len,
                                             max_kv_len, o, lse, stream)), "fedattn_decode")


def prepare_decode(ctx: Context, shape: Shape, mode: int, q, k_cache, v_cache, cache_stride_participant: int, kv_len,
                   max_kv_len: int, o, lse=None, stream=None):
    return PreparedCall(_lib.fedattn_decode,
                        _args_decode(ctx, shape, mode, q, k_cache, v_cache, cache_stride_participant, kv_len, max_kv_len, o,
                                     lse, stream),
                        "fedattn_decode", (ctx, shape, q, k_cache, v_cache, kv_len, o, lse))


def fedattn_decode_noalloc(shape: Shape, mode: int, q, k_cache, v_cache, cache_stride_participant: int,
                           kv_len, max_kv_len: int, o, lse=None, stream=None):
    """fedattn_decode for callers that may not allocate: no context, no workspace; the split-KV
    partials use a fixed array inside the library (bf16, head_dim 128, at most 256 output rows).
    Runs on the current CUDA device; calls that may overlap on the GPU share that array and race."""
    _check(_lib.fedattn_decode_noalloc(C.byref(shape), int(mode), _ptr(q), _ptr(k_cache), _ptr(v_cache),
                                       int(cache_stride_participant), _ptr(kv_len), int(max_kv_len), _ptr(o),
                                       _ptr(lse), _stream(stream)), "fedattn_decode_noalloc")
