"""Thin ctypes binding of librollart.so: argument marshalling only.

Every step of the path runs in the library's CUDA kernels; PyTorch supplies device memory and
streams.  There is no CPU or eager fallback: if the shared library is missing or cannot be
loaded, importing the entry points raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librollart.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_BOUNDS, ERR_TIMEOUT = range(7)
_NAMES = ["OK", "ERR_INVALID_ARG", "ERR_UNSUPPORTED", "ERR_WORKSPACE", "ERR_CUDA", "ERR_BOUNDS", "ERR_TIMEOUT"]

EXPORTS = (
    "rollart_workspace_size", "rollart_create", "rollart_destroy", "rollart_kv_append", "rollart_decode_attn",
    "rollart_obs_chunk_attn", "rollart_check", "rollart_last_error", "rollart_launch_count",
    "rollart_decode_attn_noalloc", "rollart_kv_gather", "rollart_pages_reserve", "rollart_pages_release",
    "rollart_append_decode_attn", "rollart_group_decode_attn", "rollart_group_decode_workspace_size",
    "rollart_decode_attn_fp8", "rollart_kv_append_fp8", "rollart_append_decode_attn_fp8",
    "rollart_kv_gather_fp8", "rollart_kv_append_fp8_codes", "rollart_obs_chunk_attn_fp8",
    "rollart_obs_chunk_fp8_scratch_size", "rollart_group_decode_attn_fp8",
    "rollart_obs_chunk_fp8_scratch_size_for_pages", "rollart_append_decode_attn_host", "rollart_host_staging_size",
    "rollart_pages_evict_stale", "rollart_selftest_bounded_wait",
)


class RollartError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"rollart {_NAMES[status] if 0 <= status < len(_NAMES) else status}: {message}")
        self.status = status


class _KVPool(ctypes.Structure):
    _fields_ = [("k_pool", ctypes.c_void_p), ("v_pool", ctypes.c_void_p), ("num_pages", ctypes.c_int32),
                ("page_size", ctypes.c_int32), ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32)]


class _Trajs(ctypes.Structure):
    _fields_ = [("page_table", ctypes.c_void_p), ("max_pages_per_traj", ctypes.c_int32),
                ("seq_lens", ctypes.c_void_p), ("num_traj", ctypes.c_int32)]


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads librollart.so from the package directory; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2512_22560_b200.build` "
                          "(there is no fallback path)")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float
    L.rollart_workspace_size.restype = ctypes.c_size_t
    L.rollart_workspace_size.argtypes = [i32, i32, i32, i32]
    L.rollart_create.restype = ctypes.c_int
    L.rollart_create.argtypes = [ctypes.POINTER(vp), ctypes.c_int, ctypes.c_size_t]
    L.rollart_destroy.restype = ctypes.c_int
    L.rollart_destroy.argtypes = [vp]
    L.rollart_kv_append.restype = ctypes.c_int
    L.rollart_kv_append.argtypes = [vp, ctypes.POINTER(_KVPool), ctypes.POINTER(_Trajs), vp, vp, i32, i32, vp, vp, vp, vp]
    L.rollart_kv_gather.restype = ctypes.c_int
    L.rollart_kv_gather.argtypes = [vp, ctypes.POINTER(_KVPool), ctypes.POINTER(_Trajs), vp, vp, i32, i32, vp, vp, vp]
    L.rollart_kv_gather_fp8.restype = ctypes.c_int
    L.rollart_kv_gather_fp8.argtypes = L.rollart_kv_gather.argtypes
    L.rollart_kv_append_fp8_codes.restype = ctypes.c_int
    L.rollart_kv_append_fp8_codes.argtypes = L.rollart_kv_append.argtypes
    L.rollart_pages_reserve.restype = ctypes.c_int
    L.rollart_pages_reserve.argtypes = [vp, vp, vp, i32, vp, i32, vp, i32, vp, vp, i32, vp]
    L.rollart_pages_release.restype = ctypes.c_int
    L.rollart_pages_release.argtypes = [vp, vp, vp, i32, i32, vp, i32, vp, i32, vp, i32, vp]
    L.rollart_pages_evict_stale.restype = ctypes.c_int
    L.rollart_pages_evict_stale.argtypes = [vp, vp, vp, i32, i32, vp, i32, vp, i32, vp, i32, i32, vp, vp, vp]
    L.rollart_decode_attn.restype = ctypes.c_int
    L.rollart_decode_attn.argtypes = [vp, ctypes.POINTER(_KVPool), ctypes.POINTER(_Trajs), vp, i32, i32, vp, i32, f32,
                                      vp, vp, vp]
    L.rollart_append_decode_attn_fp8.restype = ctypes.c_int
    L.rollart_append_decode_attn_fp8.argtypes = [vp, ctypes.POINTER(_KVPool), ctypes.POINTER(_Trajs), vp, i32, i32, vp, vp, vp, i32,
                                                 f32, f32, f32, vp, vp, vp, vp]
    L.rollart_kv_append_fp8.restype = ctypes.c_int
    L.rollart_kv_append_fp8.argtypes = [vp, ctypes.POINTER(_KVPool), ctypes.POINTER(_Trajs), vp, vp, i32, i32, vp, vp, f32, f32,
                                        vp, vp]
    L.rollart_decode_attn_fp8.restype = ctypes.c_int
    L.rollart_decode_attn_fp8.argtypes = [vp, ctypes.POINTER(_KVPool), ctypes.POINTER(_Trajs), vp, i32, i32, vp, i32, f32,
                                          f32, f32, vp, vp, vp]
    L.rollart_append_decode_attn.restype = ctypes.c_int
    L.rollart_append_decode_attn.argtypes = [vp, ctypes.POINTER(_KVPool), ctypes.POINTER(_Trajs), vp, i32, i32, vp, vp, vp, i32,
                                             f32, vp, vp, vp, vp]
    L.rollart_host_staging_size.restype = ctypes.c_size_t
    L.rollart_host_staging_size.argtypes = [i32, i32, i32]
    L.rollart_append_decode_attn_host.restype = ctypes.c_int
    L.rollart_append_decode_attn_host.argtypes = [vp, ctypes.POINTER(_KVPool), ctypes.POINTER(_Trajs), vp, i32, i32, vp, vp, vp, i32,
                                                  f32, vp, vp, vp, vp, ctypes.c_size_t, vp]
    L.rollart_group_decode_workspace_size.restype = ctypes.c_size_t
    L.rollart_group_decode_workspace_size.argtypes = [i32, i32, i32, i32]
    L.rollart_group_decode_attn.restype = ctypes.c_int
    L.rollart_group_decode_attn.argtypes = [vp, ctypes.POINTER(_KVPool), ctypes.POINTER(_Trajs), vp, i32, vp, vp, i32, i32,
                                            vp, i32, f32, vp, vp, vp]
    L.rollart_obs_chunk_attn.restype = ctypes.c_int
    L.rollart_obs_chunk_attn.argtypes = [vp, ctypes.POINTER(_KVPool), ctypes.POINTER(_Trajs), vp, vp, i32, i32, i32, vp,
                                         i32, f32, vp, vp, vp]
    L.rollart_group_decode_attn_fp8.restype = ctypes.c_int
    L.rollart_group_decode_attn_fp8.argtypes = [vp, ctypes.POINTER(_KVPool), ctypes.POINTER(_Trajs), vp, i32, vp, vp, i32, i32,
                                                vp, i32, f32, f32, f32, vp, vp, vp, ctypes.c_size_t, vp]
    L.rollart_obs_chunk_fp8_scratch_size.restype = ctypes.c_size_t
    L.rollart_obs_chunk_fp8_scratch_size.argtypes = [i32, i32, i32, i32]
    L.rollart_obs_chunk_fp8_scratch_size_for_pages.restype = ctypes.c_size_t
    L.rollart_obs_chunk_fp8_scratch_size_for_pages.argtypes = [i32, i32, i32, i32, i64]
    L.rollart_obs_chunk_attn_fp8.restype = ctypes.c_int
    L.rollart_obs_chunk_attn_fp8.argtypes = [vp, ctypes.POINTER(_KVPool), ctypes.POINTER(_Trajs), vp, vp, i32, i32, i32, vp,
                                             i32, f32, f32, f32, vp, vp, vp, ctypes.c_size_t, vp]
    L.rollart_decode_attn_noalloc.restype = ctypes.c_int
    L.rollart_decode_attn_noalloc.argtypes = [ctypes.c_int, ctypes.POINTER(_KVPool), ctypes.POINTER(_Trajs), vp, i32, i32,
                                              vp, i32, f32, vp, vp, vp, vp, ctypes.c_char_p, ctypes.c_size_t]
    L.rollart_check.restype = ctypes.c_int
    L.rollart_check.argtypes = [vp, vp]
    L.rollart_selftest_bounded_wait.restype = ctypes.c_int
    L.rollart_selftest_bounded_wait.argtypes = [vp, vp]
    L.rollart_last_error.restype = ctypes.c_char_p
    L.rollart_last_error.argtypes = [vp]
    L.rollart_launch_count.restype = i64
    L.rollart_launch_count.argtypes = [vp]
    _lib = L
    return L


def workspace_size(max_items: int, num_q_heads: int, num_kv_heads: int, max_seq_len: int) -> int:
    return int(load_library().rollart_workspace_size(max_items, num_q_heads, num_kv_heads, max_seq_len))


def group_decode_workspace_size(max_items: int, num_q_heads: int, num_kv_heads: int, max_seq_len: int) -> int:
    return int(load_library().rollart_group_decode_workspace_size(max_items, num_q_heads, num_kv_heads, max_seq_len))


def host_staging_size(n_items: int, num_q_heads: int, num_kv_heads: int) -> int:
    return int(load_library().rollart_host_staging_size(n_items, num_q_heads, num_kv_heads))


def _host_ptr(t: torch.Tensor, dtype) -> int:
    # pinned-ness is the caller's business here (Tensor.is_pinned costs several microseconds a call, and a pageable
    # buffer is not wrong, only slow: its copy is staged by the driver)
    if t.is_cuda or not t.is_contiguous() or t.dtype != dtype:
        raise ValueError(f"expected a contiguous host tensor of dtype {dtype}")
    return t.data_ptr()


def obs_chunk_fp8_scratch_size(n_items: int, num_kv_heads: int, page_size: int, max_seq_len: int,
                               total_pages: Optional[int] = None) -> int:
    """bytes of scratch for the fp8 chunk / group calls: the worst case (every item at max_seq_len), or, with
    total_pages, enough for contexts that hold at most that many pages in all"""
    lib = load_library()
    if total_pages is None:
        return int(lib.rollart_obs_chunk_fp8_scratch_size(n_items, num_kv_heads, page_size, max_seq_len))
    return int(lib.rollart_obs_chunk_fp8_scratch_size_for_pages(n_items, num_kv_heads, page_size, max_seq_len, int(total_pages)))


def _ptr(t: Optional[torch.Tensor], dtype=None, device=None, host_ok: bool = False) -> Optional[int]:
    """Address of a contiguous CUDA tensor (of the given dtype, on the given device).  With host_ok a host tensor is
    accepted too, provided it is pinned: a result buffer may be page-locked host memory, mapped into the device's
    address space under unified addressing, and the kernel then writes the result straight to the host (a pageable
    buffer has no device address and is refused here)."""
    if t is None:
        return None
    if not t.is_contiguous():
        raise ValueError("expected a contiguous tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"expected dtype {dtype}, got {t.dtype}")
    if t.is_cuda:
        if device is not None and t.get_device() != device:
            raise ValueError(f"tensor on cuda:{t.get_device()}, context on cuda:{device}")
    elif not host_ok:
        raise ValueError("expected a contiguous CUDA tensor")
    elif not t.is_pinned():
        raise ValueError("a host result buffer must be a pinned tensor")
    return t.data_ptr()


def decode_attn_noalloc(k_pool, v_pool, page_table, seq_lens, q, sm_scale, max_seq_len, out, lse=None, traj_ids=None,
                        device_status=None, stream=None) -> None:
    """rollart_decode_attn_noalloc: decode attention for callers that must not allocate device
    memory.  No Context is involved; the scratch is a fixed array inside the library (limits:
    n_items * num_kv_heads <= 2048, n_items <= 512).  `device_status` is an optional int32[4]
    CUDA tensor that receives the device-side status.  Calls that overlap on the GPU race on the
    shared array: keep them on one stream."""
    lib = load_library()
    dev = k_pool.device.index
    if k_pool.dim() != 4 or k_pool.shape != v_pool.shape:
        raise ValueError("pools must be [num_pages][num_kv_heads][page_size][head_dim] with equal shapes")
    n, h, p, d = k_pool.shape
    pool = _KVPool(_ptr(k_pool, torch.bfloat16, dev), _ptr(v_pool, torch.bfloat16, dev), n, p, h, d)
    if page_table.dim() != 2 or seq_lens.dim() != 1 or page_table.shape[0] != seq_lens.shape[0]:
        raise ValueError("page_table must be [num_traj][max_pages], seq_lens [num_traj]")
    trajs = _Trajs(_ptr(page_table, torch.int32, dev), page_table.shape[1], _ptr(seq_lens, torch.int32, dev),
                   page_table.shape[0])
    if q.dim() != 3 or q.shape != out.shape:
        raise ValueError("q and out must be [n_items][num_q_heads][head_dim]")
    n_items, hq, _ = q.shape
    if traj_ids is not None and traj_ids.shape[0] != n_items:
        raise ValueError("traj_ids must have one entry per item")
    if lse is not None and tuple(lse.shape) != (n_items, hq):
        raise ValueError("lse must be [n_items][num_q_heads]")
    if device_status is not None and (device_status.numel() < 4):
        raise ValueError("device_status must hold 4 int32")
    if stream is None:
        stream = torch.cuda.current_stream(dev)
    sptr = stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)
    buf = ctypes.create_string_buffer(320)
    st = lib.rollart_decode_attn_noalloc(
        dev, ctypes.byref(pool), ctypes.byref(trajs), _ptr(traj_ids, torch.int32, dev), n_items, int(max_seq_len),
        _ptr(q, torch.bfloat16, dev), hq, float(sm_scale), _ptr(out, torch.bfloat16, dev), _ptr(lse, torch.float32, dev),
        _ptr(device_status, torch.int32, dev), sptr, buf, len(buf))
    if st != OK:
        raise RollartError(st, buf.value.decode())


class BoundCall:
    """A library call with its arguments marshalled once, for a loop that repeats it on the same buffers (a decode
    loop rewrites the contents of its buffers, not their addresses): calling the object issues the call again at the
    cost of the foreign call alone.  Holds references to the tensors so that the addresses stay valid."""

    __slots__ = ("_ctx", "_fn", "_args", "_keep")

    def __init__(self, ctx, fn, args, keep):
        self._ctx, self._fn, self._args, self._keep = ctx, fn, args, keep

    def __call__(self) -> None:
        st = self._fn(*self._args)
        if st != OK:
            self._ctx._raise(st)


class Context:
    """Owns one rollart_ctx (workspace + device status word) on one CUDA device."""

    def __init__(self, device: int = 0, workspace_bytes: int = 0):
        self._lib = load_library()
        self.device = int(device)
        self._h = ctypes.c_void_p()
        st = self._lib.rollart_create(ctypes.byref(self._h), self.device, workspace_bytes)
        if st != OK:
            self._h = ctypes.c_void_p()
            raise RollartError(st, f"rollart_create(device={device}, workspace_bytes={workspace_bytes}) failed")
        self.workspace_bytes = int(workspace_bytes)

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            self._lib.rollart_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- helpers ---------------------------------------------------------------------------------
    def _raise(self, st: int):
        raise RollartError(st, self._lib.rollart_last_error(self._h).decode())

    def _stream(self, stream) -> int:
        if stream is None:
            stream = torch.cuda.current_stream(self.device)
        return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)

    def _pool(self, k_pool: torch.Tensor, v_pool: torch.Tensor) -> _KVPool:
        if k_pool.dim() != 4 or k_pool.shape != v_pool.shape:
            raise ValueError("pools must be [num_pages][num_kv_heads][page_size][head_dim] with equal shapes")
        n, h, p, d = k_pool.shape
        return _KVPool(_ptr(k_pool, torch.bfloat16, self.device), _ptr(v_pool, torch.bfloat16, self.device), n, p, h, d)

    def _pool_fp8(self, k_pool: torch.Tensor, v_pool: torch.Tensor) -> _KVPool:
        """fp8 pools travel as uint8 tensors [num_pages][num_kv_heads][page_size][head_dim] of E4M3 codes"""
        if k_pool.dim() != 4 or k_pool.shape != v_pool.shape:
            raise ValueError("pools must be [num_pages][num_kv_heads][page_size][head_dim] with equal shapes")
        n, h, p, d = k_pool.shape
        return _KVPool(_ptr(k_pool, torch.uint8, self.device), _ptr(v_pool, torch.uint8, self.device), n, p, h, d)

    def _trajs(self, page_table: torch.Tensor, seq_lens: torch.Tensor) -> _Trajs:
        if page_table.dim() != 2 or seq_lens.dim() != 1 or page_table.shape[0] != seq_lens.shape[0]:
            raise ValueError("page_table must be [num_traj][max_pages], seq_lens [num_traj]")
        return _Trajs(_ptr(page_table, torch.int32, self.device), page_table.shape[1],
                      _ptr(seq_lens, torch.int32, self.device), page_table.shape[0])

    # -- the three calls ---------------------------------------------------------------------------
    def kv_append(self, k_pool, v_pool, page_table, seq_lens, new_indptr, k_new, v_new, traj_ids=None,
                  seq_lens_out=None, stream=None) -> None:
        pool = self._pool(k_pool, v_pool)
        trajs = self._trajs(page_table, seq_lens)
        n_items = new_indptr.shape[0] - 1
        total_new = k_new.shape[0]
        if k_new.shape != v_new.shape or tuple(k_new.shape[1:]) != (pool.num_kv_heads, pool.head_dim):
            raise ValueError("k_new/v_new must be [total_new][num_kv_heads][head_dim]")
        if traj_ids is not None and traj_ids.shape[0] != n_items:
            raise ValueError("traj_ids must have one entry per item")
        if seq_lens_out is not None and seq_lens_out.shape != seq_lens.shape:
            raise ValueError("seq_lens_out must have the shape of seq_lens")
        st = self._lib.rollart_kv_append(
            self._h, ctypes.byref(pool), ctypes.byref(trajs), _ptr(traj_ids, torch.int32, self.device),
            _ptr(new_indptr, torch.int32, self.device), n_items, total_new, _ptr(k_new, torch.bfloat16, self.device),
            _ptr(v_new, torch.bfloat16, self.device), _ptr(seq_lens_out, torch.int32, self.device), self._stream(stream))
        if st != OK:
            self._raise(st)

    def kv_append_fp8(self, k_pool, v_pool, page_table, seq_lens, new_indptr, k_new, v_new, k_scale, v_scale,
                      traj_ids=None, seq_lens_out=None, stream=None) -> None:
        pool = self._pool_fp8(k_pool, v_pool)
        trajs = self._trajs(page_table, seq_lens)
        n_items = new_indptr.shape[0] - 1
        total_new = k_new.shape[0]
        if k_new.shape != v_new.shape or tuple(k_new.shape[1:]) != (pool.num_kv_heads, pool.head_dim):
            raise ValueError("k_new/v_new must be [total_new][num_kv_heads][head_dim]")
        if traj_ids is not None and traj_ids.shape[0] != n_items:
            raise ValueError("traj_ids must have one entry per item")
        if seq_lens_out is not None and seq_lens_out.shape != seq_lens.shape:
            raise ValueError("seq_lens_out must have the shape of seq_lens")
        st = self._lib.rollart_kv_append_fp8(
            self._h, ctypes.byref(pool), ctypes.byref(trajs), _ptr(traj_ids, torch.int32, self.device),
            _ptr(new_indptr, torch.int32, self.device), n_items, total_new, _ptr(k_new, torch.bfloat16, self.device),
            _ptr(v_new, torch.bfloat16, self.device), float(k_scale), float(v_scale),
            _ptr(seq_lens_out, torch.int32, self.device), self._stream(stream))
        if st != OK:
            self._raise(st)

    def pages_reserve(self, free_pages, free_count, page_size, page_table, seq_lens, new_tokens, traj_ids=None, stream=None) -> None:
        n_items = new_tokens.shape[0]
        st = self._lib.rollart_pages_reserve(
            self._h, _ptr(free_pages, torch.int32, self.device), _ptr(free_count, torch.int32, self.device), int(page_size),
            _ptr(page_table, torch.int32, self.device), page_table.shape[1], _ptr(seq_lens, torch.int32, self.device),
            page_table.shape[0], _ptr(traj_ids, torch.int32, self.device), _ptr(new_tokens, torch.int32, self.device), n_items,
            self._stream(stream))
        if st != OK:
            self._raise(st)

    def pages_release(self, free_pages, free_count, page_size, page_table, seq_lens, traj_ids, stream=None) -> None:
        st = self._lib.rollart_pages_release(
            self._h, _ptr(free_pages, torch.int32, self.device), _ptr(free_count, torch.int32, self.device),
            free_pages.shape[0], int(page_size), _ptr(page_table, torch.int32, self.device), page_table.shape[1],
            _ptr(seq_lens, torch.int32, self.device), page_table.shape[0], _ptr(traj_ids, torch.int32, self.device),
            traj_ids.shape[0], self._stream(stream))
        if st != OK:
            self._raise(st)

    def pages_evict_stale(self, free_pages, free_count, page_size, page_table, seq_lens, start_version, current_version, alpha,
                          evicted_ids, n_evicted, stream=None) -> None:
        """rollart_pages_evict_stale: releases the live trajectories started before version current_version - alpha"""
        if start_version.shape[0] != page_table.shape[0] or evicted_ids.shape[0] < page_table.shape[0]:
            raise ValueError("start_version and evicted_ids need one entry per trajectory")
        st = self._lib.rollart_pages_evict_stale(
            self._h, _ptr(free_pages, torch.int32, self.device), _ptr(free_count, torch.int32, self.device),
            free_pages.shape[0], int(page_size), _ptr(page_table, torch.int32, self.device), page_table.shape[1],
            _ptr(seq_lens, torch.int32, self.device), page_table.shape[0], _ptr(start_version, torch.int32, self.device),
            int(current_version), int(alpha), _ptr(evicted_ids, torch.int32, self.device),
            _ptr(n_evicted, torch.int32, self.device), self._stream(stream))
        if st != OK:
            self._raise(st)

    def kv_gather(self, k_pool, v_pool, page_table, seq_lens, out_indptr, k_out, v_out, traj_ids=None, stream=None) -> None:
        pool = self._pool(k_pool, v_pool)
        trajs = self._trajs(page_table, seq_lens)
        n_items = out_indptr.shape[0] - 1
        if k_out.shape != v_out.shape or tuple(k_out.shape[1:]) != (pool.num_kv_heads, pool.head_dim):
            raise ValueError("k_out/v_out must be [total_rows][num_kv_heads][head_dim]")
        if traj_ids is not None and traj_ids.shape[0] != n_items:
            raise ValueError("traj_ids must have one entry per item")
        st = self._lib.rollart_kv_gather(
            self._h, ctypes.byref(pool), ctypes.byref(trajs), _ptr(traj_ids, torch.int32, self.device),
            _ptr(out_indptr, torch.int32, self.device), n_items, k_out.shape[0], _ptr(k_out, torch.bfloat16, self.device),
            _ptr(v_out, torch.bfloat16, self.device), self._stream(stream))
        if st != OK:
            self._raise(st)

    def kv_gather_fp8(self, k_pool, v_pool, page_table, seq_lens, out_indptr, k_out, v_out, traj_ids=None, stream=None) -> None:
        """kv_gather for pools of E4M3 codes: k_out / v_out are uint8 [total_rows][num_kv_heads][head_dim]"""
        pool = self._pool_fp8(k_pool, v_pool)
        trajs = self._trajs(page_table, seq_lens)
        n_items = out_indptr.shape[0] - 1
        if k_out.shape != v_out.shape or tuple(k_out.shape[1:]) != (pool.num_kv_heads, pool.head_dim):
            raise ValueError("k_out/v_out must be [total_rows][num_kv_heads][head_dim]")
        if traj_ids is not None and traj_ids.shape[0] != n_items:
            raise ValueError("traj_ids must have one entry per item")
        st = self._lib.rollart_kv_gather_fp8(
            self._h, ctypes.byref(pool), ctypes.byref(trajs), _ptr(traj_ids, torch.int32, self.device),
            _ptr(out_indptr, torch.int32, self.device), n_items, k_out.shape[0], _ptr(k_out, torch.uint8, self.device),
            _ptr(v_out, torch.uint8, self.device), self._stream(stream))
        if st != OK:
            self._raise(st)

    def kv_append_fp8_codes(self, k_pool, v_pool, page_table, seq_lens, new_indptr, k_codes, v_codes, traj_ids=None,
                            seq_lens_out=None, stream=None) -> None:
        """kv_append of rows that already hold E4M3 codes (uint8 [total_new][num_kv_heads][head_dim]): a bit copy"""
        pool = self._pool_fp8(k_pool, v_pool)
        trajs = self._trajs(page_table, seq_lens)
        n_items = new_indptr.shape[0] - 1
        total_new = k_codes.shape[0]
        if k_codes.shape != v_codes.shape or tuple(k_codes.shape[1:]) != (pool.num_kv_heads, pool.head_dim):
            raise ValueError("k_codes/v_codes must be [total_new][num_kv_heads][head_dim]")
        if traj_ids is not None and traj_ids.shape[0] != n_items:
            raise ValueError("traj_ids must have one entry per item")
        if seq_lens_out is not None and seq_lens_out.shape != seq_lens.shape:
            raise ValueError("seq_lens_out must have the shape of seq_lens")
        st = self._lib.rollart_kv_append_fp8_codes(
            self._h, ctypes.byref(pool), ctypes.byref(trajs), _ptr(traj_ids, torch.int32, self.device),
            _ptr(new_indptr, torch.int32, self.device), n_items, total_new, _ptr(k_codes, torch.uint8, self.device),
            _ptr(v_codes, torch.uint8, self.device), _ptr(seq_lens_out, torch.int32, self.device), self._stream(stream))
        if st != OK:
            self._raise(st)

    def decode_attn(self, k_pool, v_pool, page_table, seq_lens, q, sm_scale, max_seq_len, out, lse=None,
                    traj_ids=None, stream=None) -> None:
        pool = self._pool(k_pool, v_pool)
        trajs = self._trajs(page_table, seq_lens)
        if q.dim() != 3 or q.shape != out.shape:
            raise ValueError("q and out must be [n_items][num_q_heads][head_dim]")
        n_items, hq, _ = q.shape
        if traj_ids is not None and traj_ids.shape[0] != n_items:
            raise ValueError("traj_ids must have one entry per item")
        if lse is not None and tuple(lse.shape) != (n_items, hq):
            raise ValueError("lse must be [n_items][num_q_heads]")
        st = self._lib.rollart_decode_attn(
            self._h, ctypes.byref(pool), ctypes.byref(trajs), _ptr(traj_ids, torch.int32, self.device), n_items,
            int(max_seq_len), _ptr(q, torch.bfloat16, self.device), hq, float(sm_scale),
            _ptr(out, torch.bfloat16, self.device, True), _ptr(lse, torch.float32, self.device, True), self._stream(stream))
        if st != OK:
            self._raise(st)

    def decode_attn_fp8(self, k_pool, v_pool, page_table, seq_lens, q, sm_scale, k_scale, v_scale, max_seq_len, out,
                        lse=None, traj_ids=None, stream=None) -> None:
        pool = self._pool_fp8(k_pool, v_pool)
        trajs = self._trajs(page_table, seq_lens)
        if q.dim() != 3 or q.shape != out.shape:
            raise ValueError("q and out must be [n_items][num_q_heads][head_dim]")
        n_items, hq, _ = q.shape
        if traj_ids is not None and traj_ids.shape[0] != n_items:
            raise ValueError("traj_ids must have one entry per item")
        if lse is not None and tuple(lse.shape) != (n_items, hq):
            raise ValueError("lse must be [n_items][num_q_heads]")
        st = self._lib.rollart_decode_attn_fp8(
            self._h, ctypes.byref(pool), ctypes.byref(trajs), _ptr(traj_ids, torch.int32, self.device), n_items,
            int(max_seq_len), _ptr(q, torch.bfloat16, self.device), hq, float(sm_scale), float(k_scale), float(v_scale),
            _ptr(out, torch.bfloat16, self.device, True), _ptr(lse, torch.float32, self.device, True), self._stream(stream))
        if st != OK:
            self._raise(st)

    def append_decode_attn_fp8(self, k_pool, v_pool, page_table, seq_lens, k_new, v_new, q, sm_scale, k_scale, v_scale,
                               max_seq_len, out, lse=None, traj_ids=None, seq_lens_out=None, stream=None) -> None:
        pool = self._pool_fp8(k_pool, v_pool)
        trajs = self._trajs(page_table, seq_lens)
        if q.dim() != 3 or q.shape != out.shape:
            raise ValueError("q and out must be [n_items][num_q_heads][head_dim]")
        n_items, hq, _ = q.shape
        if k_new.shape != v_new.shape or tuple(k_new.shape) != (n_items, pool.num_kv_heads, pool.head_dim):
            raise ValueError("k_new/v_new must be [n_items][num_kv_heads][head_dim]")
        if traj_ids is not None and traj_ids.shape[0] != n_items:
            raise ValueError("traj_ids must have one entry per item")
        if lse is not None and tuple(lse.shape) != (n_items, hq):
            raise ValueError("lse must be [n_items][num_q_heads]")
        st = self._lib.rollart_append_decode_attn_fp8(
            self._h, ctypes.byref(pool), ctypes.byref(trajs), _ptr(traj_ids, torch.int32, self.device), n_items,
            int(max_seq_len), _ptr(k_new, torch.bfloat16, self.device), _ptr(v_new, torch.bfloat16, self.device),
            _ptr(q, torch.bfloat16, self.device), hq, float(sm_scale), float(k_scale), float(v_scale),
            _ptr(out, torch.bfloat16, self.device, True), _ptr(lse, torch.float32, self.device, True),
            _ptr(seq_lens_out, torch.int32, self.device), self._stream(stream))
        if st != OK:
            self._raise(st)

    def append_decode_attn(self, k_pool, v_pool, page_table, seq_lens, k_new, v_new, q, sm_scale, max_seq_len, out, lse=None,
                           traj_ids=None, seq_lens_out=None, stream=None) -> None:
        pool = self._pool(k_pool, v_pool)
        trajs = self._trajs(page_table, seq_lens)
        if q.dim() != 3 or q.shape != out.shape:
            raise ValueError("q and out must be [n_items][num_q_heads][head_dim]")
        n_items, hq, _ = q.shape
        if k_new.shape != v_new.shape or tuple(k_new.shape) != (n_items, pool.num_kv_heads, pool.head_dim):
            raise ValueError("k_new/v_new must be [n_items][num_kv_heads][head_dim]")
        if traj_ids is not None and traj_ids.shape[0] != n_items:
            raise ValueError("traj_ids must have one entry per item")
        if lse is not None and tuple(lse.shape) != (n_items, hq):
            raise ValueError("lse must be [n_items][num_q_heads]")
        if seq_lens_out is not None and seq_lens_out.shape != seq_lens.shape:
            raise ValueError("seq_lens_out must have the shape of seq_lens")
        st = self._lib.rollart_append_decode_attn(
            self._h, ctypes.byref(pool), ctypes.byref(trajs), _ptr(traj_ids, torch.int32, self.device), n_items,
            int(max_seq_len), _ptr(k_new, torch.bfloat16, self.device), _ptr(v_new, torch.bfloat16, self.device),
            _ptr(q, torch.bfloat16, self.device), hq, float(sm_scale), _ptr(out, torch.bfloat16, self.device, True),
            _ptr(lse, torch.float32, self.device, True), _ptr(seq_lens_out, torch.int32, self.device), self._stream(stream))
        if st != OK:
            self._raise(st)

    def _append_decode_attn_host_args(self, k_pool, v_pool, page_table, seq_lens, k_new, v_new, q, sm_scale, max_seq_len, out,
                                      staging, lse, traj_ids, seq_lens_out, stream):
        pool = self._pool(k_pool, v_pool)
        trajs = self._trajs(page_table, seq_lens)
        if q.dim() != 3 or q.shape != out.shape:
            raise ValueError("q and out must be [n_items][num_q_heads][head_dim]")
        n_items, hq, _ = q.shape
        if k_new.shape != v_new.shape or tuple(k_new.shape) != (n_items, pool.num_kv_heads, pool.head_dim):
            raise ValueError("k_new/v_new must be [n_items][num_kv_heads][head_dim]")
        if traj_ids is not None and traj_ids.shape[0] != n_items:
            raise ValueError("traj_ids must have one entry per item")
        if lse is not None and tuple(lse.shape) != (n_items, hq):
            raise ValueError("lse must be [n_items][num_q_heads]")
        if seq_lens_out is not None and seq_lens_out.shape != seq_lens.shape:
            raise ValueError("seq_lens_out must have the shape of seq_lens")
        args = (self._h, ctypes.byref(pool), ctypes.byref(trajs), _ptr(traj_ids, torch.int32, self.device), n_items,
                int(max_seq_len), _host_ptr(k_new, torch.bfloat16), _host_ptr(v_new, torch.bfloat16), _host_ptr(q, torch.bfloat16),
                hq, float(sm_scale), _ptr(out, torch.bfloat16, self.device, True), _ptr(lse, torch.float32, self.device, True),
                _ptr(seq_lens_out, torch.int32, self.device), _ptr(staging, torch.uint8, self.device), staging.numel(),
                self._stream(stream))
        keep = (pool, trajs, k_pool, v_pool, page_table, seq_lens, k_new, v_new, q, out, staging, lse, traj_ids, seq_lens_out)
        return args, keep

    def append_decode_attn_host(self, k_pool, v_pool, page_table, seq_lens, k_new, v_new, q, sm_scale, max_seq_len, out,
                                staging, lse=None, traj_ids=None, seq_lens_out=None, stream=None) -> None:
        """append_decode_attn with q / k_new / v_new in pinned host tensors (the call enqueues their copy);
        `staging` is a uint8 CUDA tensor of at least host_staging_size(n_items, num_q_heads, num_kv_heads) bytes"""
        args, _ = self._append_decode_attn_host_args(k_pool, v_pool, page_table, seq_lens, k_new, v_new, q, sm_scale, max_seq_len,
                                                     out, staging, lse, traj_ids, seq_lens_out, stream)
        st = self._lib.rollart_append_decode_attn_host(*args)
        if st != OK:
            self._raise(st)

    def bind_append_decode_attn_host(self, k_pool, v_pool, page_table, seq_lens, k_new, v_new, q, sm_scale, max_seq_len, out,
                                     staging, lse=None, traj_ids=None, seq_lens_out=None, stream=None) -> BoundCall:
        """The same call with its arguments marshalled once: the returned object repeats it on the same buffers and the
        same stream (the one current now, unless `stream` is given)."""
        args, keep = self._append_decode_attn_host_args(k_pool, v_pool, page_table, seq_lens, k_new, v_new, q, sm_scale,
                                                        max_seq_len, out, staging, lse, traj_ids, seq_lens_out, stream)
        return BoundCall(self, self._lib.rollart_append_decode_attn_host, args, keep)

    def group_decode_attn(self, k_pool, v_pool, page_table, seq_lens, group_indptr, shared_lens, q, sm_scale, max_seq_len,
                          out, lse=None, traj_ids=None, stream=None) -> None:
        pool = self._pool(k_pool, v_pool)
        trajs = self._trajs(page_table, seq_lens)
        if q.dim() != 3 or q.shape != out.shape:
            raise ValueError("q and out must be [n_items][num_q_heads][head_dim]")
        n_items, hq, _ = q.shape
        n_groups = group_indptr.shape[0] - 1
        if shared_lens.shape[0] != n_groups:
            raise ValueError("shared_lens must have one entry per group")
        if traj_ids is not None and traj_ids.shape[0] != n_items:
            raise ValueError("traj_ids must have one entry per item")
        if lse is not None and tuple(lse.shape) != (n_items, hq):
            raise ValueError("lse must be [n_items][num_q_heads]")
        st = self._lib.rollart_group_decode_attn(
            self._h, ctypes.byref(pool), ctypes.byref(trajs), _ptr(traj_ids, torch.int32, self.device), n_items,
            _ptr(group_indptr, torch.int32, self.device), _ptr(shared_lens, torch.int32, self.device), n_groups,
            int(max_seq_len), _ptr(q, torch.bfloat16, self.device), hq, float(sm_scale),
            _ptr(out, torch.bfloat16, self.device), _ptr(lse, torch.float32, self.device), self._stream(stream))
        if st != OK:
            self._raise(st)

    def group_decode_attn_fp8(self, k_pool, v_pool, page_table, seq_lens, group_indptr, shared_lens, q, sm_scale, k_scale,
                              v_scale, max_seq_len, out, scratch, lse=None, traj_ids=None, stream=None) -> None:
        """group_decode_attn over pools of E4M3 codes; `scratch` is a uint8 CUDA tensor of at least
        obs_chunk_fp8_scratch_size(n_groups, num_kv_heads, page_size, max_seq_len) bytes"""
        pool = self._pool_fp8(k_pool, v_pool)
        trajs = self._trajs(page_table, seq_lens)
        if q.dim() != 3 or q.shape != out.shape:
            raise ValueError("q and out must be [n_items][num_q_heads][head_dim]")
        n_items, hq, _ = q.shape
        n_groups = group_indptr.shape[0] - 1
        if shared_lens.shape[0] != n_groups:
            raise ValueError("shared_lens must have one entry per group")
        if traj_ids is not None and traj_ids.shape[0] != n_items:
            raise ValueError("traj_ids must have one entry per item")
        if lse is not None and tuple(lse.shape) != (n_items, hq):
            raise ValueError("lse must be [n_items][num_q_heads]")
        st = self._lib.rollart_group_decode_attn_fp8(
            self._h, ctypes.byref(pool), ctypes.byref(trajs), _ptr(traj_ids, torch.int32, self.device), n_items,
            _ptr(group_indptr, torch.int32, self.device), _ptr(shared_lens, torch.int32, self.device), n_groups,
            int(max_seq_len), _ptr(q, torch.bfloat16, self.device), hq, float(sm_scale), float(k_scale), float(v_scale),
            _ptr(out, torch.bfloat16, self.device), _ptr(lse, torch.float32, self.device),
            _ptr(scratch, torch.uint8, self.device), scratch.numel(), self._stream(stream))
        if st != OK:
            self._raise(st)

    def obs_chunk_attn(self, k_pool, v_pool, page_table, seq_lens, q_indptr, q, sm_scale, max_seq_len, out, lse=None,
                       traj_ids=None, stream=None) -> None:
        pool = self._pool(k_pool, v_pool)
        trajs = self._trajs(page_table, seq_lens)
        if q.dim() != 3 or q.shape != out.shape:
            raise ValueError("q and out must be [total_q][num_q_heads][head_dim]")
        total_q, hq, _ = q.shape
        n_items = q_indptr.shape[0] - 1
        if traj_ids is not None and traj_ids.shape[0] != n_items:
            raise ValueError("traj_ids must have one entry per item")
        if lse is not None and tuple(lse.shape) != (total_q, hq):
            raise ValueError("lse must be [total_q][num_q_heads]")
        st = self._lib.rollart_obs_chunk_attn(
            self._h, ctypes.byref(pool), ctypes.byref(trajs), _ptr(traj_ids, torch.int32, self.device),
            _ptr(q_indptr, torch.int32, self.device), n_items, total_q, int(max_seq_len),
            _ptr(q, torch.bfloat16, self.device), hq, float(sm_scale), _ptr(out, torch.bfloat16, self.device),
            _ptr(lse, torch.float32, self.device), self._stream(stream))
        if st != OK:
            self._raise(st)

    def obs_chunk_attn_fp8(self, k_pool, v_pool, page_table, seq_lens, q_indptr, q, sm_scale, k_scale, v_scale, max_seq_len,
                           out, scratch, lse=None, traj_ids=None, stream=None) -> None:
        """obs_chunk_attn over pools of E4M3 codes; `scratch` is a uint8 CUDA tensor of at least
        obs_chunk_fp8_scratch_size(n_items, num_kv_heads, page_size, max_seq_len) bytes"""
        pool = self._pool_fp8(k_pool, v_pool)
        trajs = self._trajs(page_table, seq_lens)
        if q.dim() != 3 or q.shape != out.shape:
            raise ValueError("q and out must be [total_q][num_q_heads][head_dim]")
        total_q, hq, _ = q.shape
        n_items = q_indptr.shape[0] - 1
        if traj_ids is not None and traj_ids.shape[0] != n_items:
            raise ValueError("traj_ids must have one entry per item")
        if lse is not None and tuple(lse.shape) != (total_q, hq):
            raise ValueError("lse must be [total_q][num_q_heads]")
        st = self._lib.rollart_obs_chunk_attn_fp8(
            self._h, ctypes.byref(pool), ctypes.byref(trajs), _ptr(traj_ids, torch.int32, self.device),
            _ptr(q_indptr, torch.int32, self.device), n_items, total_q, int(max_seq_len),
            _ptr(q, torch.bfloat16, self.device), hq, float(sm_scale), float(k_scale), float(v_scale),
            _ptr(out, torch.bfloat16, self.device), _ptr(lse, torch.float32, self.device),
            _ptr(scratch, torch.uint8, self.device), scratch.numel(), self._stream(stream))
        if st != OK:
            self._raise(st)

    def selftest_bounded_wait(self, stream=None) -> None:
        """rollart_selftest_bounded_wait: enqueues a wait that must run out (about a second); the next status() / check()
        reports ERR_TIMEOUT."""
        st = self._lib.rollart_selftest_bounded_wait(self._h, self._stream(stream))
        if st != OK:
            self._raise(st)

    def check(self, stream=None) -> None:
        """Synchronises the stream and raises if a kernel recorded a device-side error."""
        st = self._lib.rollart_check(self._h, self._stream(stream))
        if st != OK:
            self._raise(st)

    def status(self, stream=None) -> int:
        return int(self._lib.rollart_check(self._h, self._stream(stream)))

    def last_error(self) -> str:
        return self._lib.rollart_last_error(self._h).decode()

    @property
    def launch_count(self) -> int:
        return int(self._lib.rollart_launch_count(self._h))
