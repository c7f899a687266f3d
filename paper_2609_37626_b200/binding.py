"""ctypes binding of libsplash_mla.so: same names as the C ABI, argument
marshalling only.  torch supplies device memory and streams; every step of the
path runs in the library's CUDA kernels.  There is no fallback: if the shared
library has not been built the import of its symbols fails loudly.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsplash_mla.so")

SPLASH_OK = 0
SPLASH_INVALID_ARG = -1
SPLASH_UNSUPPORTED = -2
SPLASH_UNSUPPORTED_DEVICE = -3
SPLASH_CUDA_ERROR = -4
SPLASH_DEVICE_TIMEOUT = -5
SPLASH_BAD_PAGE_ID = -6
SPLASH_KV_BF16 = 0
SPLASH_KV_E4M3_TOKEN_SCALE = 1
SPLASH_KV_E4M3_BLOCK_SCALE_BF16_ROPE = 2
SPLASH_SPARSE_ROW_BYTES = 656
SPLASH_FLAG_SIMT = 1
SPLASH_FLAG_NO_PAIR = 2
SPLASH_FLAG_SPARSE_FUSED = 4
SPLASH_FLAG_VALIDATE = 8
SPLASH_FLAG_REUSE_PLAN = 16

D_QK, D_V, PAGE_SIZE = 576, 512, 64


class SplashError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"splash status {status}: {message}")
        self.status = status


class MlaShape(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32),
        ("num_requests", ctypes.c_int32),
        ("num_heads", ctypes.c_int32),
        ("d_qk", ctypes.c_int32),
        ("d_v", ctypes.c_int32),
        ("page_size", ctypes.c_int32),
        ("num_pool_pages", ctypes.c_int32),
        ("block_table_stride", ctypes.c_int32),
        ("kv_dtype", ctypes.c_int32),
        ("softmax_scale", ctypes.c_float),
        ("q_stride_request", ctypes.c_int64),
        ("q_stride_head", ctypes.c_int64),
        ("out_stride_request", ctypes.c_int64),
        ("out_stride_head", ctypes.c_int64),
        ("lse_stride_request", ctypes.c_int64),
        ("flags", ctypes.c_uint32),
        ("q_rows", ctypes.c_uint32),
    ]


class MigrateJob(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32),
        ("src_pool", ctypes.c_void_p), ("src_scales", ctypes.c_void_p),
        ("dst_pool", ctypes.c_void_p), ("dst_scales", ctypes.c_void_p),
        ("page_bytes", ctypes.c_int64),
        ("src_page_ids", ctypes.c_void_p), ("dst_page_ids", ctypes.c_void_p),
        ("n", ctypes.c_int64),
        ("src_id_base", ctypes.c_int32), ("dst_id_base", ctypes.c_int32), ("max_page_id", ctypes.c_int32),
        ("block_table", ctypes.c_void_p),
        ("num_table_entries", ctypes.c_int64),
        ("workspace", ctypes.c_void_p),
        ("workspace_bytes", ctypes.c_size_t),
    ]


_lib = None


def load() -> ctypes.CDLL:
    """Load the shared library (raises if it has not been built)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2609_37626_b200.build` "
            "(there is no CPU or eager fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    lib.splash_mla_decode.restype = ctypes.c_int
    lib.splash_mla_decode.argtypes = [ctypes.POINTER(MlaShape), vp, vp, vp, vp, vp, i32, i32, vp, vp, vp, vp, vp, sz, vp]
    lib.splash_mla_decode_migrating.restype = ctypes.c_int
    lib.splash_mla_decode_migrating.argtypes = [ctypes.POINTER(MlaShape), vp, vp, vp, vp, vp, i32, i32, vp, vp, vp, vp, vp, sz, vp,
                                                ctypes.POINTER(MigrateJob)]
    lib.splash_mla_decode_workspace_bytes.restype = sz
    lib.splash_mla_decode_workspace_bytes.argtypes = [ctypes.POINTER(MlaShape), i32, i32]
    lib.splash_mla_decode_sparse.restype = ctypes.c_int
    lib.splash_mla_decode_sparse.argtypes = [ctypes.POINTER(MlaShape), vp, vp, vp, vp, vp, i64, vp, i32, i32, i32, vp, vp, vp, sz, vp]
    lib.splash_mla_decode_sparse_workspace_bytes.restype = sz
    lib.splash_mla_decode_sparse_workspace_bytes.argtypes = [ctypes.POINTER(MlaShape), i32, i32, i32]
    lib.splash_lse_merge.restype = ctypes.c_int
    lib.splash_lse_merge.argtypes = [i32, i64, i32, vp, vp, vp, vp, vp]
    lib.splash_kv_page_migrate.restype = ctypes.c_int
    lib.splash_kv_page_migrate.argtypes = [vp, vp, vp, vp, i64, vp, vp, i64, i32, i32, i32, vp, i64, vp, sz, vp]
    lib.splash_kv_page_migrate_static.restype = ctypes.c_int
    lib.splash_kv_page_migrate_static.argtypes = [vp, vp, vp, vp, i64, vp, vp, i64, i32, i32, i32, vp, i64, vp]
    lib.splash_kv_page_migrate_workspace_bytes.restype = sz
    lib.splash_kv_page_migrate_workspace_bytes.argtypes = [i32]
    lib.splash_dop_pack_rows.restype = ctypes.c_int
    lib.splash_dop_pack_rows.argtypes = [vp, i64, i64, i64, vp, i64, i64, i64, vp, i64, i32, vp, vp]
    lib.splash_dop_swap_outer.restype = ctypes.c_int
    lib.splash_dop_swap_outer.argtypes = [vp, i64, i64, i64, vp, vp]
    lib.splash_dop_unpack_rows.restype = ctypes.c_int
    lib.splash_dop_unpack_rows.argtypes = [vp, vp, i64, i64, vp, i64, vp]
    lib.splash_status_string.restype = ctypes.c_char_p
    lib.splash_status_string.argtypes = [ctypes.c_int]
    lib.splash_last_error.restype = ctypes.c_char_p
    lib.splash_version.restype = ctypes.c_int
    lib.splash_last_launch_count.restype = ctypes.c_int
    lib.splash_set_kernel_timing.restype = ctypes.c_int
    lib.splash_set_kernel_timing.argtypes = [ctypes.c_int]
    lib.splash_get_kernel_timing.restype = ctypes.c_int
    lib.splash_get_kernel_timing.argtypes = [ctypes.POINTER(ctypes.c_float)] * 3
    lib.splash_workspace_status.restype = ctypes.c_int
    lib.splash_workspace_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int32)]
    _lib = lib
    return lib


def _check(rc: int):
    if rc != SPLASH_OK:
        lib = load()
        raise SplashError(rc, f"{lib.splash_status_string(rc).decode()}: {lib.splash_last_error().decode()}")


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream_ptr(stream: Optional[torch.cuda.Stream]):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def make_shape(q: torch.Tensor, kv_pool: torch.Tensor, block_table: torch.Tensor, out: torch.Tensor,
               lse: torch.Tensor, softmax_scale: float, flags: int = 0) -> MlaShape:
    """q [B][H][576] (one row per request) or [B][H][R][576] (R causal rows per request)."""
    q_rows = 0
    if q.dim() == 4:
        q_rows = q.shape[2]
        assert q.stride(3) == 1 and q.stride(2) == q.shape[3] and out.dim() == 4 and out.stride(3) == 1
        assert out.stride(2) == out.shape[3] and lse.dim() == 3 and lse.stride(2) == 1 and lse.stride(1) == q_rows
        B, H, _, dqk = q.shape
    else:
        B, H, dqk = q.shape
        assert q.stride(2) == 1 and out.stride(2) == 1 and lse.stride(1) == 1
    if kv_pool.dtype == torch.bfloat16:
        kv_dtype = SPLASH_KV_BF16
    else:
        kv_dtype = SPLASH_KV_E4M3_BLOCK_SCALE_BF16_ROPE if kv_pool.shape[-1] == SPLASH_SPARSE_ROW_BYTES else SPLASH_KV_E4M3_TOKEN_SCALE
    return MlaShape(
        struct_size=ctypes.sizeof(MlaShape), num_requests=B, num_heads=H, d_qk=dqk, d_v=out.shape[-1],
        page_size=kv_pool.shape[1], num_pool_pages=kv_pool.shape[0],
        block_table_stride=block_table.stride(0) if block_table.dim() == 2 and B > 0 else 0,
        kv_dtype=kv_dtype, softmax_scale=float(softmax_scale),
        q_stride_request=q.stride(0), q_stride_head=q.stride(1),
        out_stride_request=out.stride(0), out_stride_head=out.stride(1),
        lse_stride_request=lse.stride(0), flags=flags, q_rows=q_rows)


def splash_mla_decode_workspace_bytes(shape: MlaShape, head_begin: int, head_end: int) -> int:
    return int(load().splash_mla_decode_workspace_bytes(ctypes.byref(shape), head_begin, head_end))


_workspaces = {}


def _workspace(device: torch.device, nbytes: int, tag: str) -> torch.Tensor:
    key = (device.index, tag)
    ws = _workspaces.get(key)
    if ws is None or ws.numel() < nbytes:
        ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)
        _workspaces[key] = ws
    return ws


def splash_mla_decode(q: torch.Tensor, kv_pool: torch.Tensor, block_table: torch.Tensor, seq_lens: torch.Tensor, *,
                      softmax_scale: float, kv_scales: Optional[torch.Tensor] = None, head_begin: int = 0,
                      head_end: Optional[int] = None, kv_begin: Optional[torch.Tensor] = None,
                      kv_end: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None,
                      lse: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                      stream: Optional[torch.cuda.Stream] = None, flags: int = 0, migrate_job=None):
    """Decode attention of one shard; see ``splash_mla_decode`` in include/splash_mla.h.
    With ``migrate_job`` (from ``make_migrate_job``) the call is ``splash_mla_decode_migrating``: the job's pages
    move while this call decodes.

    q [B][H][576] bf16; kv_pool [P][64][576] bf16, or uint8 / float8_e4m3fn with
    kv_scales [P][64] fp32; block_table [B][stride] int32; seq_lens, kv_begin, kv_end
    [B] int32.  out [B][H][512] fp32 and lse [B][H] fp32 are allocated (uninitialised
    outside the head slice) unless given.  Returns (out, lse).
    A 4-D q [B][H][R][576] asks for R causal query rows per request (the request's R
    newest tokens); out is then [B][H][R][512] and lse [B][H][R].
    """
    lib = load()
    assert q.is_cuda and q.dtype == torch.bfloat16
    B, H = q.shape[0], q.shape[1]
    rows = (q.shape[2],) if q.dim() == 4 else ()
    if head_end is None:
        head_end = H
    if out is None:
        out = torch.empty((B, H) + rows + (D_V,), dtype=torch.float32, device=q.device)
    if lse is None:
        lse = torch.empty((B, H) + rows, dtype=torch.float32, device=q.device)
    assert block_table.dtype == torch.int32 and seq_lens.dtype == torch.int32
    shape = make_shape(q, kv_pool, block_table, out, lse, softmax_scale, flags)
    if workspace is None:
        need = splash_mla_decode_workspace_bytes(shape, head_begin, head_end)
        workspace = _workspace(q.device, need, "decode")
    if migrate_job is not None:
        rc = lib.splash_mla_decode_migrating(ctypes.byref(shape), _ptr(q), _ptr(kv_pool), _ptr(kv_scales), _ptr(block_table),
                                             _ptr(seq_lens), head_begin, head_end, _ptr(kv_begin), _ptr(kv_end),
                                             _ptr(out), _ptr(lse), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                             _stream_ptr(stream), ctypes.byref(migrate_job[0]))
        _check(rc)
        return out, lse
    rc = lib.splash_mla_decode(ctypes.byref(shape), _ptr(q), _ptr(kv_pool), _ptr(kv_scales), _ptr(block_table),
                               _ptr(seq_lens), head_begin, head_end, _ptr(kv_begin), _ptr(kv_end),
                               _ptr(out), _ptr(lse), _ptr(workspace), workspace.numel() * workspace.element_size(),
                               _stream_ptr(stream))
    _check(rc)
    return out, lse


def make_migrate_job(src_pool: torch.Tensor, dst_pool: torch.Tensor, src_page_ids: torch.Tensor,
                     dst_page_ids: torch.Tensor, block_table: torch.Tensor, *,
                     src_scales: Optional[torch.Tensor] = None, dst_scales: Optional[torch.Tensor] = None,
                     src_id_base: int = 0, dst_id_base: int = 0, max_page_id: Optional[int] = None,
                     workspace: Optional[torch.Tensor] = None):
    """The arguments of ``splash_kv_page_migrate`` as a job for ``splash_mla_decode(..., migrate_job=...)``.
    Returns (MigrateJob, tensors kept alive with it)."""
    lib = load()
    assert src_pool.is_contiguous() and dst_pool.is_contiguous() and block_table.is_contiguous()
    assert src_page_ids.dtype == torch.int32 and dst_page_ids.dtype == torch.int32
    if max_page_id is None:
        max_page_id = max(src_id_base + src_pool.shape[0], dst_id_base + dst_pool.shape[0])
    if workspace is None:
        workspace = torch.empty(int(lib.splash_kv_page_migrate_workspace_bytes(max_page_id)), dtype=torch.uint8,
                                device=src_pool.device)
    job = MigrateJob(struct_size=ctypes.sizeof(MigrateJob), src_pool=src_pool.data_ptr(),
                     src_scales=None if src_scales is None else src_scales.data_ptr(), dst_pool=dst_pool.data_ptr(),
                     dst_scales=None if dst_scales is None else dst_scales.data_ptr(),
                     page_bytes=src_pool.shape[1] * src_pool.shape[2] * src_pool.element_size(),
                     src_page_ids=src_page_ids.data_ptr(), dst_page_ids=dst_page_ids.data_ptr(), n=src_page_ids.numel(),
                     src_id_base=src_id_base, dst_id_base=dst_id_base, max_page_id=max_page_id,
                     block_table=block_table.data_ptr(), num_table_entries=block_table.numel(),
                     workspace=workspace.data_ptr(), workspace_bytes=workspace.numel())
    return job, (src_pool, dst_pool, src_page_ids, dst_page_ids, block_table, src_scales, dst_scales, workspace)


def splash_mla_decode_sparse_workspace_bytes(shape: MlaShape, max_selected: int, head_begin: int, head_end: int) -> int:
    return int(load().splash_mla_decode_sparse_workspace_bytes(ctypes.byref(shape), max_selected, head_begin, head_end))


def splash_mla_decode_sparse(q: torch.Tensor, kv_pool: torch.Tensor, block_table: torch.Tensor, seq_lens: torch.Tensor,
                             sel_tokens: torch.Tensor, sel_count: torch.Tensor, *, softmax_scale: float,
                             max_selected: Optional[int] = None, head_begin: int = 0, head_end: Optional[int] = None,
                             out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None,
                             workspace: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None,
                             flags: int = 0):
    """Decode attention over a token list per request; see ``splash_mla_decode_sparse`` in include/splash_mla.h.

    q [B][H][576] bf16; kv_pool [P][64][656] uint8 (e4m3 latent, four block scales, bf16 rope per row);
    sel_tokens [B][K] int32 token positions, request i uses the first sel_count[i] (<= max_selected, default K).
    Returns (out [B][H][512] fp32, lse [B][H] fp32).
    """
    lib = load()
    assert q.is_cuda and q.dtype == torch.bfloat16 and q.dim() == 3
    assert kv_pool.dtype == torch.uint8 and kv_pool.shape[-1] == SPLASH_SPARSE_ROW_BYTES and kv_pool.is_contiguous()
    assert sel_tokens.dtype == torch.int32 and sel_count.dtype == torch.int32 and sel_tokens.dim() == 2
    assert sel_tokens.numel() == 0 or sel_tokens.stride(1) == 1
    assert block_table.dtype == torch.int32 and seq_lens.dtype == torch.int32
    B, H = q.shape[0], q.shape[1]
    if head_end is None:
        head_end = H
    if max_selected is None:
        max_selected = sel_tokens.shape[1]
    if out is None:
        out = torch.empty((B, H, D_V), dtype=torch.float32, device=q.device)
    if lse is None:
        lse = torch.empty((B, H), dtype=torch.float32, device=q.device)
    shape = make_shape(q, kv_pool, block_table, out, lse, softmax_scale, flags)
    if workspace is None:
        need = splash_mla_decode_sparse_workspace_bytes(shape, max_selected, head_begin, head_end)
        if need == 0:
            _check(SPLASH_INVALID_ARG)
        workspace = _workspace(q.device, need, "decode")
    rc = lib.splash_mla_decode_sparse(ctypes.byref(shape), _ptr(q), _ptr(kv_pool), _ptr(block_table), _ptr(seq_lens),
                                      _ptr(sel_tokens), sel_tokens.stride(0) if B > 0 else 0, _ptr(sel_count), max_selected,
                                      head_begin, head_end, _ptr(out), _ptr(lse), _ptr(workspace),
                                      workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    _check(rc)
    return out, lse


def splash_lse_merge(part_out: torch.Tensor, part_lse: torch.Tensor, out: Optional[torch.Tensor] = None,
                     lse: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
    """Merge [parts][rows][d_v] fp32 partial outputs by their [parts][rows] LSE."""
    lib = load()
    assert part_out.is_contiguous() and part_lse.is_contiguous()
    parts, rows, d_v = part_out.shape
    if out is None:
        out = torch.empty((rows, d_v), dtype=torch.float32, device=part_out.device)
    if lse is None:
        lse = torch.empty((rows,), dtype=torch.float32, device=part_out.device)
    _check(lib.splash_lse_merge(parts, rows, d_v, _ptr(part_out), _ptr(part_lse), _ptr(out), _ptr(lse),
                                _stream_ptr(stream)))
    return out, lse


def splash_kv_page_migrate(src_pool: torch.Tensor, dst_pool: torch.Tensor, src_page_ids: torch.Tensor,
                           dst_page_ids: torch.Tensor, block_table: torch.Tensor, *,
                           src_scales: Optional[torch.Tensor] = None, dst_scales: Optional[torch.Tensor] = None,
                           src_id_base: int = 0, dst_id_base: int = 0, max_page_id: Optional[int] = None,
                           workspace: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
    """Copy listed pages pool -> pool and rewrite block_table in place."""
    lib = load()
    assert src_pool.is_contiguous() and dst_pool.is_contiguous() and block_table.is_contiguous()
    assert src_page_ids.dtype == torch.int32 and dst_page_ids.dtype == torch.int32
    page_bytes = src_pool.shape[1] * src_pool.shape[2] * src_pool.element_size()
    n = src_page_ids.numel()
    if max_page_id is None:
        max_page_id = max(src_id_base + src_pool.shape[0], dst_id_base + dst_pool.shape[0])
    if workspace is None:
        workspace = _workspace(src_pool.device, int(lib.splash_kv_page_migrate_workspace_bytes(max_page_id)), "migrate")
    _check(lib.splash_kv_page_migrate(_ptr(src_pool), _ptr(src_scales), _ptr(dst_pool), _ptr(dst_scales), page_bytes,
                                      _ptr(src_page_ids), _ptr(dst_page_ids), n, src_id_base, dst_id_base,
                                      max_page_id, _ptr(block_table), block_table.numel(), _ptr(workspace),
                                      workspace.numel(), _stream_ptr(stream)))


def splash_dop_pack_rows(a: torch.Tensor, b: Optional[torch.Tensor], send_row: torch.Tensor,
                         out: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
    """Send buffer of the DOP forward exchange: out[p][j] = a[send_row[p]][j] ++ b[send_row[p]][j].

    a [N][h][da], b [N][h][db] or None (last dimension contiguous, any row / head strides), send_row [n] int32.
    Returns out [n][h][da+db] (dense)."""
    lib = load()
    assert a.dim() == 3 and (a.numel() == 0 or a.stride(2) == 1) and send_row.dtype == torch.int32
    assert send_row.numel() == 0 or send_row.is_contiguous()
    es = a.element_size()
    n, h, da = send_row.numel(), a.shape[1], a.shape[2]
    db = 0
    if b is not None:
        assert b.dim() == 3 and (b.numel() == 0 or b.stride(2) == 1) and b.dtype == a.dtype and b.shape[:2] == a.shape[:2]
        db = b.shape[2]
    if out is None:
        out = torch.empty((n, h, da + db), dtype=a.dtype, device=a.device)
    assert out.is_contiguous() and tuple(out.shape) == (n, h, da + db)
    _check(lib.splash_dop_pack_rows(_ptr(a), da * es, a.stride(0) * es, a.stride(1) * es,
                                    _ptr(b), db * es, (b.stride(0) * es) if b is not None else 0,
                                    (b.stride(1) * es) if b is not None else 0,
                                    _ptr(send_row), n, h, _ptr(out), _stream_ptr(stream)))
    return out


def splash_dop_swap_outer(x: torch.Tensor, out: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
    """[A][B][...] -> [B][A][...] (contiguous in, contiguous out)."""
    lib = load()
    assert x.is_contiguous() and x.dim() >= 2
    A, B = x.shape[0], x.shape[1]
    inner = x.element_size()
    for d in x.shape[2:]:
        inner *= d
    if out is None:
        out = torch.empty((B, A) + tuple(x.shape[2:]), dtype=x.dtype, device=x.device)
    assert out.is_contiguous()
    _check(lib.splash_dop_swap_outer(_ptr(x), A, B, inner, _ptr(out), _stream_ptr(stream)))
    return out


def splash_dop_unpack_rows(recv: torch.Tensor, send_row: torch.Tensor, out: torch.Tensor,
                           stream: Optional[torch.cuda.Stream] = None):
    """out[send_row[p]] = recv[p]; recv [n][...] contiguous, out [N][...] with contiguous rows."""
    lib = load()
    assert recv.is_contiguous() and send_row.dtype == torch.int32 and send_row.is_contiguous()
    assert recv.shape[1:] == out.shape[1:] and out[0].is_contiguous() if out.shape[0] else True
    n = send_row.numel()
    row_bytes = recv.element_size()
    for d in recv.shape[1:]:
        row_bytes *= d
    _check(lib.splash_dop_unpack_rows(_ptr(recv), _ptr(send_row), n, row_bytes, _ptr(out),
                                      out.stride(0) * out.element_size(), _stream_ptr(stream)))
    return out


def splash_kv_page_migrate_static(src_pool: torch.Tensor, dst_pool: torch.Tensor, src_page_ids: torch.Tensor,
                                  dst_page_ids: torch.Tensor, block_table: torch.Tensor, *,
                                  src_scales: Optional[torch.Tensor] = None,
                                  dst_scales: Optional[torch.Tensor] = None, src_id_base: int = 0,
                                  dst_id_base: int = 0, max_page_id: Optional[int] = None,
                                  stream: Optional[torch.cuda.Stream] = None):
    """Page migration for callers that cannot allocate device memory: same effect as
    splash_kv_page_migrate, but the remap table is the library's built-in 1 MiB device
    array, so this wrapper passes no workspace and creates no tensor.  Page ids must stay
    below 262,144; calls that could overlap on the GPU must be ordered by the caller."""
    lib = load()
    assert src_pool.is_contiguous() and dst_pool.is_contiguous() and block_table.is_contiguous()
    assert src_page_ids.dtype == torch.int32 and dst_page_ids.dtype == torch.int32
    page_bytes = src_pool.shape[1] * src_pool.shape[2] * src_pool.element_size()
    if max_page_id is None:
        max_page_id = max(src_id_base + src_pool.shape[0], dst_id_base + dst_pool.shape[0])
    _check(lib.splash_kv_page_migrate_static(_ptr(src_pool), _ptr(src_scales), _ptr(dst_pool), _ptr(dst_scales),
                                             page_bytes, _ptr(src_page_ids), _ptr(dst_page_ids),
                                             src_page_ids.numel(), src_id_base, dst_id_base, max_page_id,
                                             _ptr(block_table), block_table.numel(), _stream_ptr(stream)))


def splash_last_launch_count() -> int:
    return int(load().splash_last_launch_count())


def splash_version() -> int:
    return int(load().splash_version())


def splash_debug_set_trace(buf: Optional[torch.Tensor]):
    lib = load()
    lib.splash_debug_set_trace.argtypes = [ctypes.c_void_p]
    lib.splash_debug_set_trace(_ptr(buf))


def splash_set_kernel_timing(enable: bool):
    _check(load().splash_set_kernel_timing(1 if enable else 0))


def splash_get_kernel_timing():
    """(plan_ms, decode_ms, combine_ms) of the last timed decode call."""
    a, b, c = ctypes.c_float(), ctypes.c_float(), ctypes.c_float()
    _check(load().splash_get_kernel_timing(ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)))
    return a.value, b.value, c.value


def splash_workspace_status(workspace: torch.Tensor):
    detail = (ctypes.c_int32 * 3)()
    rc = load().splash_workspace_status(_ptr(workspace), detail)
    return rc, list(detail)


def decode_workspace(device: torch.device) -> Optional[torch.Tensor]:
    """The cached decode workspace of the last call on this device (for status reads)."""
    return _workspaces.get((device.index, "decode"))


# ---- host-buffer convenience path (end-to-end timing, small callers) --------------
class DeviceWorkload:
    """A workload's arrays resident on the device as torch tensors."""

    def __init__(self, w, device="cuda"):
        import numpy as np
        dev = torch.device(device)
        self.q = torch.from_numpy(w.q.view(np.int16)).to(dev).view(torch.bfloat16)
        if w.kv_dtype == 0:
            self.kv_pool = torch.from_numpy(w.kv_pool.view(np.int16)).to(dev).view(torch.bfloat16)
            self.kv_scales = None
        else:
            self.kv_pool = torch.from_numpy(w.kv_pool).to(dev)
            self.kv_scales = None if w.kv_scales is None else torch.from_numpy(w.kv_scales).to(dev)
        self.block_table = torch.from_numpy(w.block_table).to(dev)
        self.seq_lens = torch.from_numpy(w.seq_lens).to(dev)
        self.kv_begin = None if w.kv_begin is None else torch.from_numpy(w.kv_begin).to(dev)
        self.kv_end = None if w.kv_end is None else torch.from_numpy(w.kv_end).to(dev)
        self.head_begin, self.head_end = w.head_begin, w.head_end
        self.softmax_scale = w.softmax_scale

    def decode(self, **kw):
        args = dict(softmax_scale=self.softmax_scale, kv_scales=self.kv_scales, head_begin=self.head_begin,
                    head_end=self.head_end, kv_begin=self.kv_begin, kv_end=self.kv_end)
        args.update(kw)
        return splash_mla_decode(self.q, self.kv_pool, self.block_table, self.seq_lens, **args)
