"""CPU fp64 oracle for paged-KV rollout attention (see rollart_oracle.c for what it computes).

TEST INFRASTRUCTURE ONLY.  Nothing in the product package imports this; only the tests,
the smoke check and the bench's CPU-baseline leg do.  Arrays are numpy; bf16 data travels
as uint16 bit patterns.  Every function here is pinned by tests/test_oracle_pins.py, tests/test_oracle_pages.py
or tests/test_oracle_fp8.py.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np

from .build import build as _build

_lib = None

_STATUS = {1: "bad argument", 2: "page id out of range", 3: "length out of range"}


class OracleError(ValueError):
    pass


def lib():
    global _lib
    if _lib is None:
        # the mutation test points this at a deliberately broken build to show that the pins notice
        L = ctypes.CDLL(os.environ.get("ROLLART_ORACLE_LIB") or _build())
        L.oracle_num_threads.restype = ctypes.c_int
        for name in ("oracle_kv_append", "oracle_kv_gather", "oracle_attend", "oracle_lse_combine", "oracle_pages_reserve",
                     "oracle_pages_release", "oracle_pages_evict_stale", "oracle_e4m3_decode", "oracle_e4m3_encode"):
            getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def _check(rc: int):
    if rc != 0:
        raise OracleError(_STATUS.get(rc, f"status {rc}"))


def _pool_dims(pool: np.ndarray):
    assert pool.dtype == np.uint16 and pool.ndim == 4 and pool.flags.c_contiguous
    return pool.shape  # num_pages, Hkv, P, D


def kv_append(k_pool: np.ndarray, v_pool: np.ndarray, page_table: np.ndarray, seq_lens: np.ndarray,
              new_indptr: np.ndarray, k_new: np.ndarray, v_new: np.ndarray,
              traj_ids: Optional[np.ndarray] = None) -> np.ndarray:
    """In-place append into the uint16 pools (Sec. 6.1: each trajectory appends to its own
    context).  seq_lens = lengths before.  Returns the lengths after (a new array)."""
    num_pages, Hkv, P, D = _pool_dims(k_pool)
    assert v_pool.shape == k_pool.shape and v_pool.dtype == np.uint16 and v_pool.flags.c_contiguous
    page_table = _c(page_table, np.int32)
    seq_lens = _c(seq_lens, np.int32)
    new_indptr = _c(new_indptr, np.int32)
    n_items = len(new_indptr) - 1
    tid = None if traj_ids is None else _c(traj_ids, np.int32)
    k_new = _c(k_new, np.uint16)
    v_new = _c(v_new, np.uint16)
    total_new = int(new_indptr[-1]) if n_items >= 0 else 0
    assert k_new.size == total_new * Hkv * D and v_new.size == k_new.size
    out = seq_lens.copy()
    rc = lib().oracle_kv_append(
        _p(k_pool), _p(v_pool), ctypes.c_int32(num_pages), ctypes.c_int32(P), ctypes.c_int32(Hkv), ctypes.c_int32(D),
        _p(page_table), ctypes.c_int32(page_table.shape[1]), _p(seq_lens), ctypes.c_int32(len(seq_lens)),
        _p(tid), _p(new_indptr), ctypes.c_int32(n_items), _p(k_new), _p(v_new), _p(out))
    _check(rc)
    return out


def kv_gather(k_pool: np.ndarray, v_pool: np.ndarray, page_table: np.ndarray, seq_lens: np.ndarray,
              out_indptr: np.ndarray, traj_ids: Optional[np.ndarray] = None):
    """Contiguous copies (k_out, v_out: uint16 [total][Hkv][D]) of the first n_i tokens of each listed
    trajectory (Sec. 6.3, prefill/decode disaggregation hands a trajectory's cache to another worker)."""
    num_pages, Hkv, P, D = _pool_dims(k_pool)
    page_table = _c(page_table, np.int32)
    seq_lens = _c(seq_lens, np.int32)
    out_indptr = _c(out_indptr, np.int32)
    n_items = len(out_indptr) - 1
    tid = None if traj_ids is None else _c(traj_ids, np.int32)
    total = int(out_indptr[-1])
    k_out = np.zeros((total, Hkv, D), dtype=np.uint16)
    v_out = np.zeros((total, Hkv, D), dtype=np.uint16)
    rc = lib().oracle_kv_gather(
        _p(k_pool), _p(v_pool), ctypes.c_int32(num_pages), ctypes.c_int32(P), ctypes.c_int32(Hkv), ctypes.c_int32(D),
        _p(page_table), ctypes.c_int32(page_table.shape[1]), _p(seq_lens), ctypes.c_int32(len(seq_lens)),
        _p(tid), _p(out_indptr), ctypes.c_int32(n_items), _p(k_out), _p(v_out))
    _check(rc)
    return k_out, v_out


def pages_reserve(free_pages: np.ndarray, free_count: int, page_size: int, page_table: np.ndarray, seq_lens: np.ndarray,
                  new_tokens, traj_ids: Optional[np.ndarray] = None) -> int:
    """Pops, in item order, the pages each trajectory needs to grow by new_tokens[i] (Sec. 6.1: ADD between
    engine steps) and writes them into page_table IN PLACE.  Returns the new free count."""
    assert free_pages.dtype == np.int32 and page_table.dtype == np.int32 and page_table.flags.c_contiguous
    seq_lens = _c(seq_lens, np.int32)
    new_tokens = _c(new_tokens, np.int32)
    tid = None if traj_ids is None else _c(traj_ids, np.int32)
    cnt = ctypes.c_int32(free_count)
    rc = lib().oracle_pages_reserve(_p(free_pages), ctypes.byref(cnt), ctypes.c_int32(page_size), _p(page_table),
                                    ctypes.c_int32(page_table.shape[1]), _p(seq_lens), ctypes.c_int32(len(seq_lens)), _p(tid),
                                    _p(new_tokens), ctypes.c_int32(len(new_tokens)))
    _check(rc)
    return int(cnt.value)


def pages_release(free_pages: np.ndarray, free_count: int, page_size: int, page_table: np.ndarray, seq_lens: np.ndarray,
                  traj_ids: np.ndarray) -> int:
    """Pushes, in item order, every page of the listed trajectories (Sec. 6.1 ABORT, Sec. 6.2 stale eviction); sets
    their table entries to -1 and their lengths to 0, IN PLACE.  Returns the new free count."""
    assert free_pages.dtype == np.int32 and page_table.dtype == np.int32 and seq_lens.dtype == np.int32
    tid = _c(traj_ids, np.int32)
    cnt = ctypes.c_int32(free_count)
    rc = lib().oracle_pages_release(_p(free_pages), ctypes.byref(cnt), ctypes.c_int32(len(free_pages)), ctypes.c_int32(page_size),
                                    _p(page_table), ctypes.c_int32(page_table.shape[1]), _p(seq_lens),
                                    ctypes.c_int32(len(seq_lens)), _p(tid), ctypes.c_int32(len(tid)))
    _check(rc)
    return int(cnt.value)


def pages_evict_stale(free_pages: np.ndarray, free_count: int, page_size: int, page_table: np.ndarray, seq_lens: np.ndarray,
                      start_version, current_version: int, alpha: int):
    """Sec. 6.2 (asynchronous bound alpha): every live trajectory whose start version is older than
    current_version - alpha gives its pages back (as pages_release would for those trajectories in ascending
    order), IN PLACE.  Returns (new free count, ids of the evicted trajectories)."""
    assert free_pages.dtype == np.int32 and page_table.dtype == np.int32 and seq_lens.dtype == np.int32
    sv = _c(start_version, np.int32)
    assert len(sv) == len(seq_lens)
    cnt = ctypes.c_int32(free_count)
    ids = np.full(len(seq_lens), -1, np.int32)
    n = ctypes.c_int32(0)
    rc = lib().oracle_pages_evict_stale(_p(free_pages), ctypes.byref(cnt), ctypes.c_int32(len(free_pages)), ctypes.c_int32(page_size),
                                        _p(page_table), ctypes.c_int32(page_table.shape[1]), _p(seq_lens),
                                        ctypes.c_int32(len(seq_lens)), _p(sv), ctypes.c_int32(current_version),
                                        ctypes.c_int32(alpha), _p(ids), ctypes.byref(n))
    _check(rc)
    return int(cnt.value), ids[: n.value].copy()


def attend_rows(k_pool: np.ndarray, v_pool: np.ndarray, page_table: np.ndarray,
                row_traj, row_count, q: np.ndarray, sm_scale: float, row_begin=None):
    """out [n_rows][Hq][D] fp64 and lse [n_rows][Hq] fp64 for query rows that each see keys
    row_begin[r] <= j < row_count[r] of trajectory row_traj[r]."""
    num_pages, Hkv, P, D = _pool_dims(k_pool)
    page_table = _c(page_table, np.int32)
    row_traj = _c(row_traj, np.int32)
    row_count = _c(row_count, np.int32)
    rb = None if row_begin is None else _c(row_begin, np.int32)
    q = _c(q, np.uint16)
    n_rows = len(row_traj)
    assert q.ndim == 3 and q.shape[0] == n_rows and q.shape[2] == D
    Hq = q.shape[1]
    out = np.empty((n_rows, Hq, D), dtype=np.float64)
    lse = np.empty((n_rows, Hq), dtype=np.float64)
    rc = lib().oracle_attend(
        _p(k_pool), _p(v_pool), ctypes.c_int32(num_pages), ctypes.c_int32(P), ctypes.c_int32(Hkv), ctypes.c_int32(D),
        _p(page_table), ctypes.c_int32(page_table.shape[1]), ctypes.c_int32(page_table.shape[0]),
        ctypes.c_int64(n_rows), _p(row_traj), _p(rb), _p(row_count),
        _p(q), ctypes.c_int32(Hq), ctypes.c_float(sm_scale), _p(out), _p(lse))
    _check(rc)
    return out, lse


def decode_attn(k_pool, v_pool, page_table, seq_lens, q, sm_scale, traj_ids=None):
    """One query token per item, seeing all seq_lens[t] keys of its trajectory (lengths AFTER the
    append, so the token sees itself).  Sec. 3.1: the decode phase reads the whole context."""
    seq_lens = _c(seq_lens, np.int32)
    n = q.shape[0]
    tid = np.arange(n, dtype=np.int32) if traj_ids is None else _c(traj_ids, np.int32)
    return attend_rows(k_pool, v_pool, page_table, tid, seq_lens[tid], q, sm_scale)


def chunk_row_counts(seq_lens, q_indptr, traj_ids=None):
    """(row_traj, row_count): row j of an n-row chunk that ends trajectory t's L tokens sees
    L - n + j + 1 keys (the whole prior context and the chunk causally)."""
    seq_lens = _c(seq_lens, np.int32)
    q_indptr = _c(q_indptr, np.int32)
    n_items = len(q_indptr) - 1
    tid = np.arange(n_items, dtype=np.int32) if traj_ids is None else _c(traj_ids, np.int32)
    row_traj = np.empty(int(q_indptr[-1]), dtype=np.int32)
    row_count = np.empty(int(q_indptr[-1]), dtype=np.int32)
    for i in range(n_items):
        a, b = int(q_indptr[i]), int(q_indptr[i + 1])
        n = b - a
        L = int(seq_lens[tid[i]])
        if n > L:
            raise OracleError("chunk longer than its trajectory")
        row_traj[a:b] = tid[i]
        row_count[a:b] = L - n + np.arange(n) + 1
    return row_traj, row_count


def obs_chunk_attn(k_pool, v_pool, page_table, seq_lens, q_indptr, q, sm_scale, traj_ids=None,
                   rows: Optional[Sequence[int]] = None):
    """Attention of newly arrived observation tokens (Sec. 2.1: many-turn tasks re-process a
    growing history; with the prefix cached only the new tokens are computed).  `rows` selects a
    subset of the chunk rows (indices into q) to evaluate."""
    row_traj, row_count = chunk_row_counts(seq_lens, q_indptr, traj_ids)
    if rows is not None:
        rows = np.asarray(rows, dtype=np.int64)
        return attend_rows(k_pool, v_pool, page_table, row_traj[rows], row_count[rows], q[rows], sm_scale)
    return attend_rows(k_pool, v_pool, page_table, row_traj, row_count, q, sm_scale)


def lse_combine(parts_out: np.ndarray, parts_lse: np.ndarray):
    """Merge partial results over disjoint key ranges: parts_out [S][...][D], parts_lse [S][...]."""
    parts_out = _c(parts_out, np.float64)
    parts_lse = _c(parts_lse, np.float64)
    S = parts_out.shape[0]
    D = parts_out.shape[-1]
    inner = parts_lse.shape[1:]
    n = int(np.prod(inner)) if inner else 1
    po = parts_out.reshape(S, n, D)
    pl = parts_lse.reshape(S, n)
    out = np.empty((n, D), dtype=np.float64)
    lse = np.empty(n, dtype=np.float64)
    for i in range(n):
        a = np.ascontiguousarray(po[:, i, :])
        b = np.ascontiguousarray(pl[:, i])
        one = ctypes.c_double()
        rc = lib().oracle_lse_combine(ctypes.c_int32(S), ctypes.c_int32(D), _p(a), _p(b),
                                      out[i].ctypes.data_as(ctypes.c_void_p), ctypes.byref(one))
        _check(rc)
        lse[i] = one.value
    return out.reshape(*inner, D), lse.reshape(inner)


# ---- fp8 (E4M3) KV pools -------------------------------------------------------------------------

def e4m3_decode(codes: np.ndarray) -> np.ndarray:
    """Values (float64) of E4M3 codes (uint8)."""
    codes = _c(codes, np.uint8)
    out = np.empty(codes.shape, dtype=np.float64)
    _check(lib().oracle_e4m3_decode(_p(codes), ctypes.c_int64(codes.size), _p(out)))
    return out


def e4m3_encode(x: np.ndarray) -> np.ndarray:
    """Nearest E4M3 code (uint8) of each float32, ties to even, saturating at +-448."""
    x = _c(x, np.float32)
    out = np.empty(x.shape, dtype=np.uint8)
    _check(lib().oracle_e4m3_encode(_p(x), ctypes.c_int64(x.size), _p(out)))
    return out


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def fp8_quantize_rows(rows_bf16: np.ndarray, scale: float) -> np.ndarray:
    """E4M3 codes of bf16 rows (uint16 bit patterns) for a pool with the given scale: encode(x * (1 / scale)),
    the reciprocal and the product both rounded to fp32 (the precision the quantised append works in)."""
    inv = np.float32(1.0) / np.float32(scale)
    return e4m3_encode(bf16_bits_to_f32(rows_bf16) * inv)


def kv_append_fp8(k_pool: np.ndarray, v_pool: np.ndarray, page_table, seq_lens, new_indptr, k_new_bf16, v_new_bf16,
                  k_scale: float, v_scale: float, traj_ids=None) -> np.ndarray:
    """Quantised append into uint8 pools [pages][Hkv][P][D]: the rows are quantised, then appended by the same
    bit copy as the bf16 pools (a row of D bytes is moved as D / 2 16-bit units)."""
    assert k_pool.dtype == np.uint8 and v_pool.dtype == np.uint8 and k_pool.shape[-1] % 2 == 0
    kq = fp8_quantize_rows(k_new_bf16, k_scale)
    vq = fp8_quantize_rows(v_new_bf16, v_scale)
    return kv_append(k_pool.view(np.uint16), v_pool.view(np.uint16), page_table, seq_lens, new_indptr,
                     kq.view(np.uint16), vq.view(np.uint16), traj_ids=traj_ids)


def kv_append_fp8_codes(k_pool: np.ndarray, v_pool: np.ndarray, page_table, seq_lens, new_indptr, k_codes, v_codes,
                        traj_ids=None) -> np.ndarray:
    """Append of rows that already hold codes (uint8 [total][Hkv][D]) into uint8 pools: the bit copy of kv_append,
    a row of D bytes moved as D / 2 16-bit units (Sec. 6.3: the receiving side of a cache hand-over)."""
    assert k_pool.dtype == np.uint8 and v_pool.dtype == np.uint8 and k_pool.shape[-1] % 2 == 0
    return kv_append(k_pool.view(np.uint16), v_pool.view(np.uint16), page_table, seq_lens, new_indptr,
                     _c(k_codes, np.uint8).view(np.uint16), _c(v_codes, np.uint8).view(np.uint16), traj_ids=traj_ids)


def kv_gather_fp8(k_pool: np.ndarray, v_pool: np.ndarray, page_table, seq_lens, out_indptr, traj_ids=None):
    """kv_gather over uint8 pools of codes: (k_out, v_out) uint8 [total][Hkv][D] (Sec. 6.3: the sending side)."""
    assert k_pool.dtype == np.uint8 and v_pool.dtype == np.uint8 and k_pool.shape[-1] % 2 == 0
    k16, v16 = kv_gather(k_pool.view(np.uint16), v_pool.view(np.uint16), page_table, seq_lens, out_indptr, traj_ids=traj_ids)
    return k16.view(np.uint8), v16.view(np.uint8)


def fp8_pool_as_bf16_bits(pool: np.ndarray) -> np.ndarray:
    """The pool's values (unit scale) as bf16 bit patterns: every finite E4M3 value is a bf16 value, so this is exact.
    NaN codes become bf16 NaN."""
    v = e4m3_decode(pool).astype(np.float32)
    return (v.view(np.uint32) >> 16).astype(np.uint16)


def decode_attn_fp8(k_pool, v_pool, page_table, seq_lens, q, sm_scale, k_scale, v_scale, traj_ids=None):
    """Decode attention over fp8 pools: keys are k_scale * code value, values v_scale * code value, so the result is
    v_scale * attention(sm_scale * k_scale; code values)."""
    out, lse = decode_attn(fp8_pool_as_bf16_bits(k_pool), fp8_pool_as_bf16_bits(v_pool), page_table, seq_lens, q,
                           float(np.float32(sm_scale) * np.float32(k_scale)), traj_ids=traj_ids)
    return out * float(np.float32(v_scale)), lse


def obs_chunk_attn_fp8(k_pool, v_pool, page_table, seq_lens, q_indptr, q, sm_scale, k_scale, v_scale, traj_ids=None,
                       rows: Optional[Sequence[int]] = None):
    """Observation-chunk attention over fp8 pools: the rows and the mask of obs_chunk_attn with keys
    k_scale * code value and values v_scale * code value."""
    out, lse = obs_chunk_attn(fp8_pool_as_bf16_bits(k_pool), fp8_pool_as_bf16_bits(v_pool), page_table, seq_lens, q_indptr, q,
                              float(np.float32(sm_scale) * np.float32(k_scale)), traj_ids=traj_ids, rows=rows)
    return out * float(np.float32(v_scale)), lse
