"""Seeded synthetic inputs for the MLA decode path.

This module only draws random numbers, rounds them to the storage formats and
lays them out in pages.  It holds none of the attention arithmetic and is the
one module that both the CPU oracle's tests and the CUDA path's tests share, so
that both sides see byte-identical inputs.

Workload shapes follow the paper's serving regimes ("many short vs a few very
long requests", Sec. 1; fixed-length batches, Sec. 5): a DP-attention request
slice, a TP/DOP head slice at 32K context, a position-sharded CP request at
256K, and an RL-rollout batch with a long-tailed length mix and fp8 KV.  The
dimensions are the DeepSeek-V3 ones of App. A: 128 heads, a 512-wide latent and
a 64-wide rotary part, softmax scale 1/sqrt(128 + 64).

Arrays are numpy: bf16 as uint16 bit patterns, e4m3 as uint8 codes.
"""
from __future__ import annotations

import concurrent.futures
import dataclasses
import math
import os
from typing import Optional

import numpy as np

D_LATENT = 512
D_ROPE = 64
D_QK = D_LATENT + D_ROPE
D_V = D_LATENT
PAGE_SIZE = 64
BASE_SEED = 20260922  # the PCG64 seed the paper uses for its own Monte-Carlo (App. B)
SOFTMAX_SCALE = 1.0 / math.sqrt(192.0)

BF16_NAN = 0x7FC0
BF16_INF = 0x7F80
E4M3_NAN = 0x7F


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns, round to nearest even (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = u >> np.uint32(16)
    r &= np.uint32(1)
    r += np.uint32(0x7FFF)
    r += u
    r >>= np.uint32(16)
    return r.astype(np.uint16)


def make_query_rows(seed: int, B: int, H: int, R: int) -> np.ndarray:
    """R query rows per request and head, [B][H][R][576] bf16 bit patterns (N(0,1), a stream of its own)."""
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, 7])))
    return f32_to_bf16_bits(rng.standard_normal((B, H, R, D_QK), dtype=np.float32))


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """bf16 bit patterns -> float32 (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def quantize_e4m3_per_token(x: np.ndarray):
    """Rows of float32 -> (e4m3 codes, one float32 scale per row).

    scale = max|x| / 448 (1 for an all-zero row); code = RNE(clamp(x / scale, +-448)).
    The cast is torch's CPU float8_e4m3fn conversion (round to nearest even); the
    clamp keeps it away from that cast's NaN-on-overflow behaviour.
    """
    import torch

    x = np.ascontiguousarray(x, dtype=np.float32)
    amax = np.abs(x).max(axis=-1)
    scale = np.where(amax > 0, amax / np.float32(448.0), np.float32(1.0)).astype(np.float32)
    y = np.clip(x / scale[..., None], -448.0, 448.0).astype(np.float32)
    codes = torch.from_numpy(y).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    return codes, scale


SPARSE_ROW_BYTES = 656        # 512 e4m3 latent codes, 4 float block scales, 64 bf16 rope values
SPARSE_BLOCK = 128            # latent dims per scale


def pack_sparse_rows(x: np.ndarray) -> np.ndarray:
    """Rows of 576 float32 -> rows of 656 bytes: the latent quantised to e4m3 in blocks of 128 dims
    (scale = max|x| / 448 over the block, 1 for an all-zero block; code = RNE(clamp(x / scale, +-448))),
    the four scales, the rope part rounded to bf16."""
    import torch

    x = np.ascontiguousarray(x, dtype=np.float32)
    n = x.shape[0]
    lat = x[:, :D_LATENT].reshape(n, D_LATENT // SPARSE_BLOCK, SPARSE_BLOCK)
    amax = np.abs(lat).max(axis=-1)
    scale = np.where(amax > 0, amax / np.float32(448.0), np.float32(1.0)).astype(np.float32)
    y = np.clip(lat / scale[..., None], -448.0, 448.0).astype(np.float32)
    codes = torch.from_numpy(y).to(torch.float8_e4m3fn).view(torch.uint8).numpy().reshape(n, D_LATENT)
    out = np.empty((n, SPARSE_ROW_BYTES), dtype=np.uint8)
    out[:, :D_LATENT] = codes
    out[:, D_LATENT:D_LATENT + 16] = scale.view(np.uint8).reshape(n, 16)
    out[:, D_LATENT + 16:] = f32_to_bf16_bits(x[:, D_LATENT:]).view(np.uint8).reshape(n, 2 * D_ROPE)
    return out


def select_tokens(seed: int, seq_lens, topk: int):
    """The token list an indexer would hand to sparse decode: for every request min(topk, s) distinct
    positions drawn uniformly from its history, in random order (the worst case for locality).
    Returns (sel [B][topk] int32, -1 beyond the count; sel_count [B] int32)."""
    seq_lens = np.asarray(seq_lens, dtype=np.int32)
    B = int(seq_lens.shape[0])
    sel = np.full((B, max(topk, 1)), -1, dtype=np.int32)
    cnt = np.minimum(seq_lens, topk).astype(np.int32)
    for i in range(B):
        rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, 11, i])))
        s, k = int(seq_lens[i]), int(cnt[i])
        if k:
            sel[i, :k] = rng.permutation(s)[:k] if s <= 4 * k else rng.choice(s, size=k, replace=False)
    return sel, cnt


def sparse_algorithmic_bytes(sel_count, h: int) -> int:
    """Sparse decode: every listed row once (656 B) and its list entry, the q slice read, out + lse written."""
    n, B = int(np.asarray(sel_count).sum()), len(sel_count)
    return n * (SPARSE_ROW_BYTES + 4) + B * h * D_QK * 2 + B * h * (D_V + 1) * 4 + 8 * B


@dataclasses.dataclass
class Workload:
    name: str
    q: np.ndarray                       # [B][H][576] uint16 (bf16 bits)
    kv_pool: np.ndarray                 # [P][64][576] uint16 (bf16) or uint8 (e4m3), or [P][64][656] uint8 (kv_dtype 2)
    kv_scales: Optional[np.ndarray]     # [P][64] float32 for e4m3, else None
    block_table: np.ndarray             # [B][stride] int32, -1 beyond the last page
    seq_lens: np.ndarray                # [B] int32
    head_begin: int
    head_end: int
    kv_begin: Optional[np.ndarray] = None   # [B] int32 or None
    kv_end: Optional[np.ndarray] = None
    softmax_scale: float = SOFTMAX_SCALE
    page_size: int = PAGE_SIZE
    used_pages: Optional[np.ndarray] = None  # pool page ids referenced by the table

    @property
    def B(self) -> int:
        return int(self.q.shape[0])

    @property
    def H(self) -> int:
        return int(self.q.shape[1])

    @property
    def kv_dtype(self) -> int:
        if self.kv_pool.dtype == np.uint16:
            return 0
        return 1 if self.kv_pool.shape[-1] == D_QK else 2

    @property
    def num_pool_pages(self) -> int:
        return int(self.kv_pool.shape[0])

    def total_tokens(self) -> int:
        lo = np.zeros_like(self.seq_lens) if self.kv_begin is None else np.maximum(self.kv_begin, 0)
        hi = self.seq_lens if self.kv_end is None else np.minimum(self.kv_end, self.seq_lens)
        return int(np.maximum(hi - lo, 0).sum())

    def algorithmic_bytes(self) -> int:
        """Each in-range cache row once per request, the q slice read, out + lse
        written, the table entries used and seq_lens."""
        h = self.head_end - self.head_begin
        row = D_QK * 2 if self.kv_dtype == 0 else D_QK + 4
        pages = int(((self.seq_lens + self.page_size - 1) // self.page_size).sum())
        return (self.total_tokens() * row + self.B * h * D_QK * 2
                + self.B * h * (D_V + 1) * 4 + 4 * pages + 4 * self.B)

    def algorithmic_flops(self) -> int:
        h = self.head_end - self.head_begin
        return 2 * h * (D_QK + D_V) * self.total_tokens()


def make_workload(name: str, seed: int, seq_lens, H: int, *, head_begin: int = 0,
                  head_end: Optional[int] = None, kv_dtype: int = 0, pool_pages: Optional[int] = None,
                  pool_factor: float = 1.25, rope_scale: float = 1.0, placement: str = "permute",
                  poison: bool = True, table_stride: Optional[int] = None,
                  extra_pool_pages: int = 0) -> Workload:
    """Draw q and a paged latent cache for the given context lengths.

    Values are i.i.d. N(0,1) (rotary columns times ``rope_scale``) rounded to bf16 (``kv_dtype`` 0),
    quantised to e4m3 with one scale per token (1), or packed into 656-byte rows (2: e4m3 latent with a
    scale per 128 dims, bf16 rope; ``pack_sparse_rows``).  Pages are dealt to requests in
    order from a seeded permutation of the pool (``placement``: "permute",
    "identity" or "reversed").  Every byte the attention must not read (unused
    pages, slots past the end of a request's last page, table padding) is poisoned
    with NaN / Inf patterns when ``poison`` is set.  ``extra_pool_pages`` appends
    untouched (poisoned) pages, e.g. the second pool of a migration.
    """
    # independent streams for the placement, the queries and (below) each KV chunk,
    # so the values do not depend on the placement or the pool size
    rng_place = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, 1])))
    rng_q = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, 2])))
    seq_lens = np.asarray(seq_lens, dtype=np.int32)
    B = int(seq_lens.shape[0])
    pages_per_req = (seq_lens.astype(np.int64) + PAGE_SIZE - 1) // PAGE_SIZE
    n_used = int(pages_per_req.sum())
    if pool_pages is None:
        pool_pages = max(1, int(math.ceil(n_used * pool_factor)))
    assert pool_pages >= n_used
    if placement == "permute":
        order = rng_place.permutation(pool_pages)
    elif placement == "identity":
        order = np.arange(pool_pages)
    elif placement == "reversed":
        order = np.arange(pool_pages)[::-1]
    else:
        raise ValueError(placement)
    used = order[:n_used].astype(np.int32)

    stride = int(pages_per_req.max()) if B else 1
    stride = max(stride, 1)
    if table_stride is not None:
        assert table_stride >= stride
        stride = table_stride
    block_table = np.full((B, stride), -1, dtype=np.int32)
    cursor = 0
    for i in range(B):
        n = int(pages_per_req[i])
        block_table[i, :n] = used[cursor:cursor + n]
        cursor += n

    q = f32_to_bf16_bits(rng_q.standard_normal((B, H, D_QK), dtype=np.float32))

    total_pages = pool_pages + extra_pool_pages
    if kv_dtype == 0:
        kv_pool = np.empty((total_pages, PAGE_SIZE, D_QK), dtype=np.uint16)
        kv_scales = None
        if poison:
            kv_pool[...] = BF16_NAN
            kv_pool[:, 1::2, :] = BF16_INF
        else:
            kv_pool[...] = 0
    elif kv_dtype == 2:
        kv_pool = np.empty((total_pages, PAGE_SIZE, SPARSE_ROW_BYTES), dtype=np.uint8)
        kv_scales = None
        kv_pool[...] = 0xFF if poison else 0          # NaN as an e4m3 code, as a float scale and as a bf16
    else:
        kv_pool = np.empty((total_pages, PAGE_SIZE, D_QK), dtype=np.uint8)
        kv_scales = np.empty((total_pages, PAGE_SIZE), dtype=np.float32)
        if poison:
            kv_pool[...] = E4M3_NAN
            kv_scales[...] = np.nan
        else:
            kv_pool[...] = 0
            kv_scales[...] = 1.0

    col_scale = None
    if rope_scale != 1.0:
        col_scale = np.ones((D_QK,), dtype=np.float32)
        col_scale[D_LATENT:] = rope_scale

    # Fill request by request in chunks of pages; every chunk draws from its own
    # child stream keyed by (seed, request, first page), so the bytes do not depend
    # on how many threads fill the pool.
    chunk_pages = 256
    jobs = []
    cursor = 0
    for i in range(B):
        n = int(pages_per_req[i])
        for p0 in range(0, n, chunk_pages):
            jobs.append((i, p0, min(n, p0 + chunk_pages), cursor))
        cursor += n

    def fill(job):
        i, p0, p1, base = job
        s = int(seq_lens[i])
        crng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, 7, i, p0])))
        t0, t1 = p0 * PAGE_SIZE, min(s, p1 * PAGE_SIZE)
        rows = crng.standard_normal((t1 - t0, D_QK), dtype=np.float32)
        if col_scale is not None:
            rows *= col_scale
        ids = used[base + p0:base + p1]
        full = (t1 - t0) // PAGE_SIZE
        rem = (t1 - t0) - full * PAGE_SIZE
        if kv_dtype == 0:
            bits = f32_to_bf16_bits(rows)
            if full:
                kv_pool[ids[:full]] = bits[:full * PAGE_SIZE].reshape(full, PAGE_SIZE, D_QK)
            if rem:
                kv_pool[ids[full], :rem] = bits[full * PAGE_SIZE:]
        elif kv_dtype == 2:
            packed = pack_sparse_rows(rows)
            if full:
                kv_pool[ids[:full]] = packed[:full * PAGE_SIZE].reshape(full, PAGE_SIZE, SPARSE_ROW_BYTES)
            if rem:
                kv_pool[ids[full], :rem] = packed[full * PAGE_SIZE:]
        else:
            codes, sc = quantize_e4m3_per_token(rows)
            if full:
                kv_pool[ids[:full]] = codes[:full * PAGE_SIZE].reshape(full, PAGE_SIZE, D_QK)
                kv_scales[ids[:full]] = sc[:full * PAGE_SIZE].reshape(full, PAGE_SIZE)
            if rem:
                kv_pool[ids[full], :rem] = codes[full * PAGE_SIZE:]
                kv_scales[ids[full], :rem] = sc[full * PAGE_SIZE:]

    workers = min(32, len(os.sched_getaffinity(0)))
    if len(jobs) > 1 and workers > 1:
        with concurrent.futures.ThreadPoolExecutor(max_workers=workers) as ex:
            list(ex.map(fill, jobs))
    else:
        for job in jobs:
            fill(job)

    return Workload(name=name, q=q, kv_pool=kv_pool, kv_scales=kv_scales, block_table=block_table,
                    seq_lens=seq_lens, head_begin=head_begin,
                    head_end=H if head_end is None else head_end, used_pages=used)


def poison_outside_ranges(w: Workload, kv_begin, kv_end) -> None:
    """Overwrite, in place, every cache row of every request that lies outside its KV range
    [kv_begin[i], kv_end[i]) with NaN / Inf patterns (for e4m3 also its scale): the cache of a
    position-sharded rank holds only the tokens it owns (App. E), the other slots of a boundary
    page hold whatever was there.  Requests must not share pages."""
    for i in range(w.B):
        s = int(w.seq_lens[i])
        lo, hi = max(0, int(kv_begin[i])), min(s, int(kv_end[i]))
        hi = max(hi, lo)
        for t in list(range(0, lo)) + list(range(hi, s)):
            page, slot = int(w.block_table[i, t // PAGE_SIZE]), t % PAGE_SIZE
            if w.kv_dtype == 0:
                w.kv_pool[page, slot, :] = BF16_NAN if (t & 1) else BF16_INF
                w.kv_pool[page, slot, 5::7] = 0xFF80                     # -Inf
            elif w.kv_dtype == 1:
                w.kv_pool[page, slot, :] = E4M3_NAN if (t & 1) else 0xFF  # both NaN codes of e4m3fn
                w.kv_scales[page, slot] = np.nan if (t % 3) else np.inf
            else:
                w.kv_pool[page, slot, :] = 0xFF


def rollout_lengths(seed: int, n: int = 512) -> np.ndarray:
    """Lognormal context lengths: median 2048, sigma 1.2, clipped to [16, 131072]."""
    rng = np.random.Generator(np.random.PCG64(seed))
    x = np.exp(math.log(2048.0) + 1.2 * rng.standard_normal(n))
    return np.clip(np.rint(x), 16, 131072).astype(np.int32)


CONFIG_NAMES = ("c1_tiny", "c2_dp_attention", "c3_tp_dop_slice", "c4_cp_long", "c5_rollout_fp8")


def config(idx: int, *, scale: float = 1.0, extra_pool_factor: float = 0.0) -> Workload:
    """The five workload configurations, 1-based.  ``scale`` < 1 shrinks request
    counts / lengths for quick tests while keeping the structure."""
    seed = BASE_SEED + idx
    if idx == 1:
        return make_workload(CONFIG_NAMES[0], seed, [1, 17, 64, 200], H=16, pool_pages=16)
    if idx == 2:
        rng = np.random.Generator(np.random.PCG64(seed))
        B = max(1, int(round(64 * scale)))
        lens = rng.integers(1024, 8192, size=B, endpoint=True).astype(np.int32)
        return make_workload(CONFIG_NAMES[1], seed + 1000, lens, H=128)
    if idx == 3:
        B = max(1, int(round(16 * scale)))
        w = make_workload(CONFIG_NAMES[2], seed, [32768] * B, H=128, head_begin=32, head_end=48)
        return w
    if idx == 4:
        s = max(64, int(round(262144 * scale)))
        return make_workload(CONFIG_NAMES[3], seed, [s], H=128, rope_scale=2.0)
    if idx == 5:
        B = max(1, int(round(512 * scale)))
        lens = rollout_lengths(seed, B)
        n_used = int(((lens.astype(np.int64) + PAGE_SIZE - 1) // PAGE_SIZE).sum())
        pool = int(math.ceil(n_used * 1.25))
        extra = int(math.ceil(n_used * extra_pool_factor))
        return make_workload(CONFIG_NAMES[4], seed + 1000, lens, H=128, kv_dtype=1,
                             pool_pages=pool, extra_pool_pages=extra)
    raise ValueError("config index must be 1..5")


def cp_ranges(seq_lens: np.ndarray, parts: int):
    """Contiguous position shards of every request: part j of T owns tokens
    [j*s/T, (j+1)*s/T) (App. E, position-sharded CP)."""
    s = seq_lens.astype(np.int64)
    out = []
    for j in range(parts):
        out.append(((s * j // parts).astype(np.int32), (s * (j + 1) // parts).astype(np.int32)))
    return out


def migration_plan(seed: int, used_pages: np.ndarray, dst_pool_pages: int, fraction: float = 0.3):
    """A seeded choice (without replacement) of ``fraction`` of the in-use pages
    and as many distinct destination page ids in a second pool."""
    rng = np.random.Generator(np.random.PCG64(seed))
    n = int(round(len(used_pages) * fraction))
    src = rng.choice(np.asarray(used_pages, dtype=np.int32), size=n, replace=False).astype(np.int32)
    assert dst_pool_pages >= n
    dst = rng.permutation(dst_pool_pages)[:n].astype(np.int32)
    return src, dst
