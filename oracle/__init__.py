"""CPU oracle for the MLA decode hot path -- TEST INFRASTRUCTURE ONLY.

Thin ctypes wrapper around ``splash_oracle.c`` (plain C, fp64).  Only tests, the
smoke check and the benchmark's CPU-baseline leg may import this package; the
CUDA library never does, and this package never imports the CUDA binding.

All arrays are numpy: bf16 values travel as ``uint16`` bit patterns, e4m3 values
as ``uint8`` codes, results come back as ``float64``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "splash_oracle.c")
_LIB = os.path.join(_HERE, "libsplash_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP over (request, head) pairs)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"])
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.oracle_e4m3_to_double.restype = ctypes.c_double
        lib.oracle_e4m3_to_double.argtypes = [ctypes.c_uint8]
        lib.oracle_mla_decode.restype = ctypes.c_int
        lib.oracle_mla_decode_rows.restype = ctypes.c_int
        lib.oracle_lse_merge.restype = ctypes.c_int
        lib.oracle_kv_page_migrate.restype = ctypes.c_int
        _lib = lib
    return _lib


def num_threads() -> int:
    """Threads the OpenMP loops will use (OMP_NUM_THREADS or the core count)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env)
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:  # pragma: no cover
        return os.cpu_count() or 1


def _ptr(a, ctype):
    if a is None:
        return ctypes.POINTER(ctype)()
    return a.ctypes.data_as(ctypes.POINTER(ctype))


def e4m3_to_double(code: int) -> float:
    return float(_load().oracle_e4m3_to_double(int(code) & 0xFF))


def mla_decode(q, kv_pool, block_table, seq_lens, *, softmax_scale, kv_scales=None,
               head_begin=0, head_end=None, kv_begin=None, kv_end=None,
               page_size=64, d_v=512, pairs=None, out=None, lse=None):
    """Decode attention over a paged latent cache (see splash_oracle.c).

    q [B][H][d_qk] uint16 (bf16 bits); kv_pool [P][page_size][d_qk] uint16 (bf16)
    or uint8 (e4m3, then kv_scales [P][page_size] float32 is required).
    Returns (out [B][H][d_v] float64, lse [B][H] float64); entries outside the
    computed (request, head) set keep whatever ``out``/``lse`` held (NaN when
    they are allocated here).
    """
    lib = _load()
    assert q.dtype == np.uint16 and q.ndim == 3
    B, H, d_qk = q.shape
    assert q.strides[2] == 2
    if kv_pool.dtype == np.uint16:
        kv_dtype = 0
        assert kv_scales is None
    elif kv_pool.dtype == np.uint8:
        kv_dtype = 1
        assert kv_scales is not None and kv_scales.dtype == np.float32
        kv_scales = np.ascontiguousarray(kv_scales)
    else:
        raise TypeError("kv_pool must be uint16 (bf16 bits) or uint8 (e4m3 codes)")
    kv_pool = np.ascontiguousarray(kv_pool)
    assert kv_pool.shape[-1] == d_qk and kv_pool.shape[-2] == page_size
    block_table = np.ascontiguousarray(block_table, dtype=np.int32)
    if block_table.ndim == 1:
        block_table = block_table.reshape(B, -1) if B else block_table.reshape(0, 1)
    seq_lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    if head_end is None:
        head_end = H
    if kv_begin is not None:
        kv_begin = np.ascontiguousarray(kv_begin, dtype=np.int32)
    if kv_end is not None:
        kv_end = np.ascontiguousarray(kv_end, dtype=np.int32)
    if out is None:
        out = np.full((B, H, d_v), np.nan, dtype=np.float64)
    if lse is None:
        lse = np.full((B, H), np.nan, dtype=np.float64)
    assert out.flags.c_contiguous and lse.flags.c_contiguous
    n_pairs = 0
    if pairs is not None:
        pairs = np.ascontiguousarray(pairs, dtype=np.int32).reshape(-1, 2)
        n_pairs = pairs.shape[0]
    table_stride = block_table.shape[1] if block_table.ndim == 2 else 1
    rc = lib.oracle_mla_decode(
        ctypes.c_int(B), ctypes.c_int(H), ctypes.c_int(d_qk), ctypes.c_int(d_v),
        ctypes.c_int(page_size),
        _ptr(q, ctypes.c_uint16), ctypes.c_int64(q.strides[0] // 2), ctypes.c_int64(q.strides[1] // 2),
        kv_pool.ctypes.data_as(ctypes.c_void_p), ctypes.c_int(kv_dtype), _ptr(kv_scales, ctypes.c_float),
        _ptr(block_table, ctypes.c_int32), ctypes.c_int64(table_stride),
        _ptr(seq_lens, ctypes.c_int32),
        ctypes.c_int(head_begin), ctypes.c_int(head_end),
        _ptr(kv_begin, ctypes.c_int32), _ptr(kv_end, ctypes.c_int32),
        ctypes.c_double(float(softmax_scale)),
        _ptr(pairs, ctypes.c_int32), ctypes.c_int64(n_pairs),
        _ptr(out, ctypes.c_double), _ptr(lse, ctypes.c_double))
    if rc != 0:
        raise ValueError(f"oracle_mla_decode rejected its arguments (rc={rc})")
    return out, lse


def mla_decode_rows(q, kv_pool, block_table, seq_lens, *, softmax_scale, kv_scales=None,
                    head_begin=0, head_end=None, kv_begin=None, kv_end=None, page_size=64, d_v=512):
    """Attention for R causal query rows per request (see oracle_mla_decode_rows).

    q [B][H][R][d_qk] uint16 (bf16 bits); the R rows are the request's newest tokens.
    Returns (out [B][H][R][d_v] float64, lse [B][H][R] float64), NaN outside the head slice.
    """
    lib = _load()
    assert q.dtype == np.uint16 and q.ndim == 4 and q.flags.c_contiguous
    B, H, R, d_qk = q.shape
    if kv_pool.dtype == np.uint16:
        kv_dtype = 0
        assert kv_scales is None
    elif kv_pool.dtype == np.uint8:
        kv_dtype = 1
        assert kv_scales is not None and kv_scales.dtype == np.float32
        kv_scales = np.ascontiguousarray(kv_scales)
    else:
        raise TypeError("kv_pool must be uint16 (bf16 bits) or uint8 (e4m3 codes)")
    kv_pool = np.ascontiguousarray(kv_pool)
    block_table = np.ascontiguousarray(block_table, dtype=np.int32)
    if block_table.ndim == 1:
        block_table = block_table.reshape(B, -1) if B else block_table.reshape(0, 1)
    seq_lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    if head_end is None:
        head_end = H
    if kv_begin is not None:
        kv_begin = np.ascontiguousarray(kv_begin, dtype=np.int32)
    if kv_end is not None:
        kv_end = np.ascontiguousarray(kv_end, dtype=np.int32)
    out = np.full((B, H, R, d_v), np.nan, dtype=np.float64)
    lse = np.full((B, H, R), np.nan, dtype=np.float64)
    rc = lib.oracle_mla_decode_rows(
        ctypes.c_int(B), ctypes.c_int(H), ctypes.c_int(R), ctypes.c_int(d_qk), ctypes.c_int(d_v),
        ctypes.c_int(page_size),
        _ptr(q, ctypes.c_uint16), ctypes.c_int64(H * R * d_qk), ctypes.c_int64(R * d_qk),
        kv_pool.ctypes.data_as(ctypes.c_void_p), ctypes.c_int(kv_dtype), _ptr(kv_scales, ctypes.c_float),
        _ptr(block_table, ctypes.c_int32), ctypes.c_int64(block_table.shape[1]),
        _ptr(seq_lens, ctypes.c_int32),
        ctypes.c_int(head_begin), ctypes.c_int(head_end),
        _ptr(kv_begin, ctypes.c_int32), _ptr(kv_end, ctypes.c_int32),
        ctypes.c_double(float(softmax_scale)),
        _ptr(out, ctypes.c_double), _ptr(lse, ctypes.c_double))
    if rc != 0:
        raise ValueError(f"oracle_mla_decode_rows rejected its arguments (rc={rc})")
    return out, lse


SPARSE_ROW_BYTES = 656


def mla_decode_sparse(q, kv_pool, block_table, seq_lens, sel, sel_count, *, softmax_scale,
                      head_begin=0, head_end=None, page_size=64):
    """Decode attention over the listed tokens of a cache of 656-byte rows (see splash_oracle.c).

    q [B][H][576] uint16 (bf16 bits); kv_pool [P][page_size][656] uint8; sel [B][K] int32 token
    positions, request i uses the first sel_count[i].  Returns (out [B][H][512], lse [B][H]) float64,
    NaN outside [head_begin, head_end).
    """
    lib = _load()
    assert q.dtype == np.uint16 and q.ndim == 3 and q.strides[2] == 2 and q.shape[2] == 576
    B, H, _ = q.shape
    kv_pool = np.ascontiguousarray(kv_pool)
    assert kv_pool.dtype == np.uint8 and kv_pool.shape[-1] == SPARSE_ROW_BYTES and kv_pool.shape[-2] == page_size
    block_table = np.ascontiguousarray(block_table, dtype=np.int32)
    if block_table.ndim == 1:
        block_table = block_table.reshape(B, -1) if B else block_table.reshape(0, 1)
    seq_lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    sel = np.ascontiguousarray(sel, dtype=np.int32)
    if sel.ndim == 1:
        sel = sel.reshape(B, -1) if B else sel.reshape(0, 1)
    sel_count = np.ascontiguousarray(sel_count, dtype=np.int32)
    assert sel_count.shape == (B,) and (B == 0 or sel_count.max() <= sel.shape[1])
    if head_end is None:
        head_end = H
    out = np.full((B, H, 512), np.nan, dtype=np.float64)
    lse = np.full((B, H), np.nan, dtype=np.float64)
    rc = lib.oracle_mla_decode_sparse(
        ctypes.c_int(B), ctypes.c_int(H), ctypes.c_int(page_size),
        _ptr(q, ctypes.c_uint16), ctypes.c_int64(q.strides[0] // 2), ctypes.c_int64(q.strides[1] // 2),
        _ptr(kv_pool, ctypes.c_uint8), _ptr(block_table, ctypes.c_int32), ctypes.c_int64(block_table.shape[1]),
        _ptr(seq_lens, ctypes.c_int32), _ptr(sel, ctypes.c_int32), ctypes.c_int64(sel.shape[1]),
        _ptr(sel_count, ctypes.c_int32), ctypes.c_int(head_begin), ctypes.c_int(head_end),
        ctypes.c_double(float(softmax_scale)), _ptr(out, ctypes.c_double), _ptr(lse, ctypes.c_double))
    if rc != 0:
        raise ValueError(f"oracle_mla_decode_sparse rejected its arguments (rc={rc})")
    return out, lse


def lse_merge(part_out, part_lse):
    """Merge [parts][rows][d_v] partial outputs by their [parts][rows] LSE."""
    lib = _load()
    part_out = np.ascontiguousarray(part_out, dtype=np.float64)
    part_lse = np.ascontiguousarray(part_lse, dtype=np.float64)
    parts, rows, d_v = part_out.shape
    assert part_lse.shape == (parts, rows)
    out = np.empty((rows, d_v), dtype=np.float64)
    lse = np.empty((rows,), dtype=np.float64)
    lib.oracle_lse_merge(ctypes.c_int(parts), ctypes.c_int64(rows), ctypes.c_int(d_v),
                         _ptr(part_out, ctypes.c_double), _ptr(part_lse, ctypes.c_double),
                         _ptr(out, ctypes.c_double), _ptr(lse, ctypes.c_double))
    return out, lse


def kv_page_migrate(src_pool, dst_pool, src_page_ids, dst_page_ids, block_table, *,
                    src_scales=None, dst_scales=None, src_id_base=0, dst_id_base=0):
    """In-place page copy + table rewrite on numpy arrays (dst_pool, dst_scales,
    block_table are modified).  Pools are [P][page_size][d_qk] of any 1- or 2-byte
    dtype."""
    lib = _load()
    assert src_pool.flags.c_contiguous and dst_pool.flags.c_contiguous
    assert block_table.flags.c_contiguous and block_table.dtype == np.int32
    page_size = src_pool.shape[1]
    page_bytes = src_pool.shape[1] * src_pool.shape[2] * src_pool.itemsize
    src_page_ids = np.ascontiguousarray(src_page_ids, dtype=np.int32)
    dst_page_ids = np.ascontiguousarray(dst_page_ids, dtype=np.int32)
    assert src_page_ids.shape == dst_page_ids.shape
    lib.oracle_kv_page_migrate(
        src_pool.ctypes.data_as(ctypes.POINTER(ctypes.c_uint8)), _ptr(src_scales, ctypes.c_float),
        dst_pool.ctypes.data_as(ctypes.POINTER(ctypes.c_uint8)), _ptr(dst_scales, ctypes.c_float),
        ctypes.c_int64(page_bytes), ctypes.c_int(page_size),
        _ptr(src_page_ids, ctypes.c_int32), _ptr(dst_page_ids, ctypes.c_int32),
        ctypes.c_int64(src_page_ids.size),
        ctypes.c_int32(src_id_base), ctypes.c_int32(dst_id_base),
        _ptr(block_table, ctypes.c_int32), ctypes.c_int64(block_table.size))


# ---------------------------------------------------------------------------------------------
# DOP transfer layout changes (App. E): a tensor in global-row, local-head order is regrouped into
# owner-row, all-head order and back.  Pure permutations of whole rows of bytes, written here with
# explicit loops over (position, head) so that they can be read against the text.
def dop_pack_rows(a, b, send_row):
    """Send buffer of the forward exchange.  a [N][h][da], b [N][h][db] or None (the no-position and
    rotary parts of the query, fused into one row), send_row [n]: the source row of send position p
    (rows grouped by destination owner; row identity and head order are kept).  -> [n][h][da+db]."""
    n, h = len(send_row), a.shape[1]
    da = a.shape[2]
    db = 0 if b is None else b.shape[2]
    out = np.zeros((n, h, da + db), dtype=a.dtype)
    for p in range(n):
        for j in range(h):
            out[p, j, :da] = a[send_row[p], j]
            if b is not None:
                out[p, j, da:] = b[send_row[p], j]
    return out


def dop_unpack_rows(recv, send_row, num_rows, out=None):
    """Reverse exchange, last step: position p of recv [n][h][d] goes back to row send_row[p] of
    out [num_rows][h][d]; rows that are not listed keep what ``out`` held (zeros when allocated here)."""
    if out is None:
        out = np.zeros((num_rows,) + recv.shape[1:], dtype=recv.dtype)
    for p in range(len(send_row)):
        out[send_row[p]] = recv[p]
    return out


def dop_swap_outer(x):
    """[A][B][...] -> [B][A][...]: receive buffer in source-rank-major order [T][n][h][d] to owner-row,
    all-head order [n][T*h][d] (head s*h + j comes from rank s: global head order), and its inverse."""
    A, B = x.shape[0], x.shape[1]
    out = np.zeros((B, A) + x.shape[2:], dtype=x.dtype)
    for s in range(A):
        for r in range(B):
            out[r, s] = x[s, r]
    return out
