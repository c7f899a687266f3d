/*
 * splash_mla.h -- C ABI of the B200 (sm_100a) MLA decode library.
 *
 * One rank's attention shard under the paper's layouts, on one GPU:
 *   - TP / DOP        : a head slice [head_begin, head_end) over each request's
 *                       complete history (Sec. 3, "Computation" of DOP: every head
 *                       attends over the complete history, outputs agree with TP up
 *                       to floating-point reduction order);
 *   - DP-attention    : a request slice (the caller passes only its requests), all
 *                       heads;
 *   - CP              : a KV token range per request (App. E, position-sharded CP),
 *                       giving partial (O, LSE) that splash_lse_merge combines.
 * The cache is the head-shared latent cache of absorbed MLA: one row of
 * d_qk = d_c + d_r = 512 + 64 elements per token, the value being its first
 * d_v = d_c = 512 elements (Sec. 3 "Cost": d_q = d_c + d_r, d_z = d_c; App. A
 * dimensions).  splash_kv_page_migrate is the local part of a layout switch: the
 * "discard" primitive's repack of kept blocks into the destination view (Sec. 3,
 * Sec. 4.1 "Reuse"), after which every query must still read its complete history
 * (Sec. 4.1 "Handoff").
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer owned by the caller unless stated otherwise.
 *     The library allocates no device memory, never synchronises the host, enqueues
 *     its kernels on `stream` (a cudaStream_t passed as void*, NULL = default
 *     stream) and returns.
 *   - Return value: SPLASH_OK (0) or a negative splash_status.  On an error nothing
 *     has been launched.  splash_last_error() gives a host string for the last
 *     error of the calling thread.
 *   - Empty work (no requests, an empty head slice, n = 0 pages) is a successful
 *     no-op: idle ranks are legal (App. E: ranks that own no rows still take part).
 *   - Stream capture: every call may be recorded into a CUDA graph (Sec. 4.1: the
 *     steps after a switch replay graphs captured at startup; App. G "Graph capture").  Nothing in a call depends on values the host cannot see at
 *     capture time -- lengths, ranges, token lists and page tables are read on the
 *     device, the split-KV plan is computed there -- so a replay follows buffers that
 *     changed in place.  Make the first call of each kind on a device outside the
 *     capture (it sets kernel attributes), and leave kernel timing off while capturing.
 */
#ifndef SPLASH_MLA_H_
#define SPLASH_MLA_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define SPLASH_API __attribute__((visibility("default")))
#else
#define SPLASH_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum splash_status {
    SPLASH_OK = 0,
    SPLASH_INVALID_ARG = -1,        /* null pointer, bad range, misalignment, short workspace */
    SPLASH_UNSUPPORTED = -2,        /* dims / page size / dtype / head count not built */
    SPLASH_UNSUPPORTED_DEVICE = -3, /* the current device is not compute capability 10.x */
    SPLASH_CUDA_ERROR = -4,         /* a CUDA runtime / driver call failed */
    SPLASH_DEVICE_TIMEOUT = -5,     /* (status word only) a bounded device wait gave up */
    SPLASH_BAD_PAGE_ID = -6         /* (status word only, SPLASH_FLAG_VALIDATE) a block-table entry the call needs
                                       names no page of the pool */
} splash_status;

enum {
    SPLASH_KV_BF16 = 0,
    SPLASH_KV_E4M3_TOKEN_SCALE = 1,
    /* 656-byte rows: 512 e4m3 latent codes, 4 fp32 scales (one per 128 latent dims), 64 bf16 rope values.
     * Only splash_mla_decode_sparse reads this format. */
    SPLASH_KV_E4M3_BLOCK_SCALE_BF16_ROPE = 2
};
#define SPLASH_SPARSE_ROW_BYTES 656

/* shape.flags bits */
enum {
    /* Run the plain SIMT (fp32 CUDA-core) decode kernel instead of the tcgen05 one.
     * A diagnostic path: same plan, same partial slots, same combine; slow. */
    SPLASH_FLAG_SIMT = 1u,
    /* slices of 65..128 heads: use two independent 64-head CTAs per KV worker instead of a CTA
     * pair issuing cta_group::2 MMAs.  A diagnostic path. */
    SPLASH_FLAG_NO_PAIR = 2u,
    /* splash_mla_decode_sparse only: one kernel that gathers, dequantises and multiplies (CTA pairs) instead of
     * the gather kernel followed by the dense kernels.  Every listed row crosses HBM once; tile, query rows and
     * P are f16 in that kernel (values must lie within f16's range).  Correct, not yet the faster of the two. */
    SPLASH_FLAG_SPARSE_FUSED = 4u,
    /* splash_mla_decode only: validation mode.  One more (small) kernel between the plan and the decode kernel checks
     * every block-table entry of a page that intersects a request's range against [0, num_pool_pages) and records
     * the first bad one in the workspace status word: splash_workspace_status() then returns SPLASH_BAD_PAGE_ID with
     * detail = (request, page index within the request, the id found).  With or without the flag an id outside the
     * pool is never dereferenced (the page reads as zeros); the flag makes the mistake visible. */
    SPLASH_FLAG_VALIDATE = 8u,
    /* splash_mla_decode / splash_mla_decode_migrating only: the work partition of the previous call on this workspace is
     * taken again and the plan kernel is not launched.  The partition (App. B's linear-in-context cost: page tiles, not
     * requests, spread evenly over the CTAs) is a function of seq_lens, kv_begin / kv_end, the width head_end - head_begin,
     * the shape (num_requests, q_rows, kv_dtype, the other flag bits) and the device only -- not of q, the cache, the
     * scales or the block table -- and a decode step runs the same batch through every layer of the model: the first
     * layer's call plans, the others pass this bit.  The caller asserts that those arguments are what they were in the
     * last call WITHOUT this bit on the same workspace (nothing checks it; a different batch would be cut along the old
     * batch's boundaries and give wrong results, within bounds).  The error words of the status block are cleared as in
     * any call.  Ignored by the sparse entry point and together with SPLASH_FLAG_VALIDATE (which needs the plan's pass). */
    SPLASH_FLAG_REUSE_PLAN = 16u
};

/*
 * Shape of one decode call.  Strides are in ELEMENTS of the array they index.
 *   q    : bf16,  element (i, g, d) at q  [i*q_stride_request   + g*q_stride_head   + d], d < d_qk
 *   out  : fp32,  element (i, g, d) at out[i*out_stride_request + g*out_stride_head + d], d < d_v
 *   lse  : fp32,  element (i, g)    at lse[i*lse_stride_request + g]
 * g is the GLOBAL head id in [0, num_heads); a call touches only heads in
 * [head_begin, head_end) and leaves every other element of out / lse untouched, so
 * the slices of several calls can share one buffer.  A caller holding a compact
 * per-rank q [N][H/T][d_q] passes num_heads = H/T and the slice [0, H/T).
 */
typedef struct splash_mla_shape {
    uint32_t struct_size;        /* sizeof(splash_mla_shape), for versioning */
    int32_t num_requests;        /* B >= 0; one query row per request (decode) */
    int32_t num_heads;           /* H, 1..128 */
    int32_t d_qk;                /* 576: [0,512) latent (also V), [512,576) rotary part */
    int32_t d_v;                 /* 512 */
    int32_t page_size;           /* 64 tokens */
    int32_t num_pool_pages;      /* pages addressable from kv_pool (bounds the table's ids) */
    int32_t block_table_stride;  /* entries per request row of block_table */
    int32_t kv_dtype;            /* SPLASH_KV_BF16 or SPLASH_KV_E4M3_TOKEN_SCALE */
    float softmax_scale;         /* multiplies q.k before the softmax (configs: 1/sqrt(192)) */
    int64_t q_stride_request, q_stride_head;     /* multiples of 8 */
    int64_t out_stride_request, out_stride_head; /* multiples of 4 */
    int64_t lse_stride_request;
    uint32_t flags;              /* SPLASH_FLAG_* bits, 0 for the default path */
    uint32_t q_rows;             /* R: query rows per request, 0 or 1 = one row (decode); see splash_mla_decode */
} splash_mla_shape;

/*
 * Decode attention over a paged latent KV cache.
 *
 * For request i, head g in [head_begin, head_end) and token range
 * R_i = [max(0, kv_begin[i]), min(seq_lens[i], kv_end[i])):
 *     row_t  = kv_pool[block_table[i][t / 64]][t % 64][0..576)     (times kv_scales[..] for e4m3)
 *     l_t    = softmax_scale * sum_{d<576} q[i][g][d] * row_t[d]
 *     lse    = ln sum_{t in R_i} exp(l_t)                          (natural log, scale included)
 *     out[d] = sum_{t in R_i} exp(l_t - lse) * row_t[d],  d < 512
 * An empty R_i gives out = 0, lse = -inf.
 *
 * Several query rows per request (shape.q_rows = R > 1; a multi-token decode step or a
 * short prefill chunk: the batch entry of a request carries q_i > 1 rows, Sec. 4.1): the R
 * rows are the request's R newest tokens, whose cache rows are already written; row r sits
 * at position seq_lens[i] - R + r and attends causally, i.e. its range is
 *     [max(0, kv_begin[i]), min(kv_end[i], seq_lens[i] - (R - 1 - r))),
 * each row on its own with the formulas above.  The rows of a head are dense:
 *     q   (i, g, r, d) at q  [i*q_stride_request   + g*q_stride_head   + r*576 + d], q_stride_head   = R*576
 *     out (i, g, r, d) at out[i*out_stride_request + g*out_stride_head + r*512 + d], out_stride_head = R*512
 *     lse (i, g, r)    at lse[i*lse_stride_request + g*R + r]
 * 1 <= R <= 8.  A slice of more than 128 / R heads runs as several CTA pairs per KV worker,
 * 128 (head, row) pairs each, side by side on the same pages in one launch: the cache
 * crosses HBM once (the other pairs' reads of a page hit L2).
 *
 *   q            bf16, 16-byte aligned
 *   kv_pool      [num_pool_pages][64][576] bf16 (73,728 B / page) or e4m3 bytes
 *                (36,864 B / page); 128-byte aligned
 *   kv_scales    [num_pool_pages][64] fp32, one scale per token; required for e4m3,
 *                NULL for bf16
 *   block_table  [num_requests][block_table_stride] int32 page ids; only the entries
 *                of pages that intersect R_i are read (others may hold anything)
 *   seq_lens     [num_requests] int32
 *   kv_begin,
 *   kv_end       [num_requests] int32 each, or NULL for 0 / seq_lens[i]; need not be
 *                page aligned
 *   out, lse     fp32, 16-byte / 4-byte aligned
 *   workspace    scratch of at least splash_mla_decode_workspace_bytes() bytes,
 *                256-byte aligned; its contents on entry do not matter and two
 *                calls that may overlap on the device need different workspaces
 *
 * Only the rows of tokens in R_i enter the result.  Every other byte of the cache --
 * slots of a referenced page outside R_i (below or beyond seq_lens[i]), pages the table
 * does not reference, the scales of such slots -- may hold anything, NaN / Inf patterns
 * included: a rank of position-sharded CP owns only its own tokens of a boundary page
 * (App. E).  Results are bit-reproducible for a fixed call (same shape, lengths and
 * ranges).
 */
SPLASH_API int splash_mla_decode(const splash_mla_shape *shape,
                      const void *q, const void *kv_pool, const float *kv_scales,
                      const int32_t *block_table, const int32_t *seq_lens,
                      int32_t head_begin, int32_t head_end,
                      const int32_t *kv_begin, const int32_t *kv_end,
                      float *out, float *lse,
                      void *workspace, size_t workspace_bytes, void *stream);

/* Workspace size (host computation, no device access) for a call with this shape
 * and head slice; depends only on the shape, the slice width and the device's SM
 * count.  Returns 0 on invalid arguments. */
SPLASH_API size_t splash_mla_decode_workspace_bytes(const splash_mla_shape *shape,
                                         int32_t head_begin, int32_t head_end);

/*
 * Sparse decode: attention over a LIST of tokens per request instead of a range (the sparse
 * absorbed-MLA backend of the paper's runs, Sec. 5 "Setup": an indexer has selected the tokens
 * each decode query attends over), reading the cache row format of those runs (FP8 latent with
 * its scales, BF16 rope; Sec. 5, App. B payload).  Per token the row is 656 bytes:
 *     [0, 512)    e4m3 codes c_d of the latent
 *     [512, 528)  four fp32 scales s_b, b = d / 128
 *     [528, 656)  64 bf16 rope values r_j
 * with key columns k_d = c_d * s_{d/128} (d < 512), k_{512+j} = r_j and value v_d = k_d (d < 512).
 * For request i and head g in [head_begin, head_end), with T_i the first sel_count[i] entries
 * of sel_tokens[i * sel_stride ...] (token positions of request i, any order):
 *     l_t = softmax_scale * q[i][g] . k(t),  lse = ln sum_{t in T_i} exp(l_t),
 *     out = sum_{t in T_i} exp(l_t - lse) v(t)
 * sel_count[i] = 0 gives out = 0, lse = -inf; a position listed twice counts twice.
 *
 *   shape        kv_dtype = SPLASH_KV_E4M3_BLOCK_SCALE_BF16_ROPE, q_rows 0 or 1; the other fields
 *                as for splash_mla_decode
 *   kv_pool      [num_pool_pages][64][656] bytes (41,984 B / page), 128-byte aligned
 *   sel_tokens   int32; entry j of request i at sel_tokens[i * sel_stride + j]; entries at or
 *                beyond sel_count[i] are never read
 *   sel_count    [num_requests] int32, each in [0, max_selected]
 *   max_selected bound on sel_count (the indexer's k, e.g. 2048); sizes the workspace
 *   workspace    at least splash_mla_decode_sparse_workspace_bytes() bytes, 256-byte aligned
 *
 * All pointers are device pointers.  A list entry outside [0, seq_lens[i]), a page id outside
 * the pool or a count outside [0, max_selected] is never dereferenced; the outputs of that
 * request are then NaN.  Two stages on the device: the listed rows are gathered and dequantised
 * (code times block scale, rounded to bf16) into a dense bf16 cache inside the workspace, then
 * the dense decode kernels run over it (launch order: plan over the list counts, gather,
 * decode kernel, combine).
 */
SPLASH_API int splash_mla_decode_sparse(const splash_mla_shape *shape, const void *q, const void *kv_pool,
                             const int32_t *block_table, const int32_t *seq_lens,
                             const int32_t *sel_tokens, int64_t sel_stride, const int32_t *sel_count,
                             int32_t max_selected, int32_t head_begin, int32_t head_end,
                             float *out, float *lse, void *workspace, size_t workspace_bytes, void *stream);

/* Workspace size for splash_mla_decode_sparse (host computation).  Returns 0 on invalid arguments. */
SPLASH_API size_t splash_mla_decode_sparse_workspace_bytes(const splash_mla_shape *shape, int32_t max_selected,
                                                int32_t head_begin, int32_t head_end);

/*
 * Merge partial attention results over disjoint KV ranges (the CP combination step;
 * also the reduction of the decode kernel's internal KV splits):
 *     lse[r]    = ln sum_j exp(part_lse[j][r])
 *     out[r][d] = sum_j exp(part_lse[j][r] - lse[r]) * part_out[j][r][d]
 * Parts with lse = -inf contribute nothing (their out values are not read into the
 * result); if all are -inf, out = 0 and lse = -inf.
 *   part_out [num_parts][rows][d_v] fp32, part_lse [num_parts][rows] fp32,
 *   out [rows][d_v], lse [rows]; all contiguous, 16-byte aligned; d_v a multiple of 4;
 *   out / lse must not alias the parts.
 */
SPLASH_API int splash_lse_merge(int32_t num_parts, int64_t rows, int32_t d_v,
                     const float *part_out, const float *part_lse,
                     float *out, float *lse, void *stream);

/*
 * Copy a listed set of KV pages between two page pools in HBM and rewrite the
 * block table: page src_page_ids[j] of src_pool is copied, byte for byte, to page
 * dst_page_ids[j] of dst_pool (with its scale page when the scale pointers are
 * given), and every block-table entry equal to src_id_base + src_page_ids[j]
 * becomes dst_id_base + dst_page_ids[j].  Table ids are "arena-global": when both
 * pools are sub-ranges of the allocation that decode receives as kv_pool, the bases
 * are the pools' page offsets in it, so one table can name pages of both pools.
 * Negative entries and entries naming other pages pass through.  Source pages are
 * left intact (the caller retires them, Sec. 4.1 "Retire").
 *
 *   page_bytes       73,728 (bf16) or 36,864 (e4m3); a multiple of 16; pools 16-byte aligned
 *   src/dst_scales   [pages][64] fp32 or both NULL
 *   src/dst_page_ids [n] int32 device arrays; each duplicate-free, 0 <= id
 *   max_page_id      exclusive upper bound on src_id_base + src_page_ids[j]
 *   block_table      [num_table_entries] int32, rewritten in place
 *   workspace        at least splash_kv_page_migrate_workspace_bytes(max_page_id) bytes
 */
SPLASH_API int splash_kv_page_migrate(const void *src_pool, const float *src_scales,
                           void *dst_pool, float *dst_scales,
                           int64_t page_bytes,
                           const int32_t *src_page_ids, const int32_t *dst_page_ids, int64_t n,
                           int32_t src_id_base, int32_t dst_id_base, int32_t max_page_id,
                           int32_t *block_table, int64_t num_table_entries,
                           void *workspace, size_t workspace_bytes, void *stream);

SPLASH_API size_t splash_kv_page_migrate_workspace_bytes(int32_t max_page_id);

/*
 * A decode call that carries a page migration with it: the overlapped transfer of a layout
 * switch, in which one layer's state moves while another layer computes, so that about one
 * layer's transfer stays exposed (Sec. 4.1 "Overlapped transfer", the exposed-cost equation of
 * Sec. 4.2).  The effect is that of
 *     splash_kv_page_migrate(job...)  and  splash_mla_decode(...)
 * issued on `stream` in either order; the two must therefore be independent: the decode reads
 * none of the job's destination pages and not the job's block table (the usual case: the job
 * moves the pages of ANOTHER layer's cache; source pages may be shared, they are only read).
 *
 * How: slices of 65..128 (head, row) pairs run on CTA pairs in which the MMA-issuing warps of
 * each pair's second CTA have nothing to do; those warps copy the job's pages (16-byte
 * streaming loads and stores, byte-exact) while the rest of the kernel decodes, on SMs and
 * HBM bandwidth the decode leaves unused.  The job's table rewrite (three small kernels) runs
 * on `stream` before the decode.  Calls that do not run on the CTA-pair kernels (narrower
 * slices, SPLASH_FLAG_SIMT / NO_PAIR, more than 128 (head, row) pairs) run the plain page-copy
 * kernel after the decode instead: same results, no overlap.
 *
 * job == NULL or job->n == 0: exactly splash_mla_decode.  The job's fields are the arguments of
 * splash_kv_page_migrate, validated the same way; on an error nothing has been launched.
 */
typedef struct splash_migrate_job {
    uint32_t struct_size;                /* sizeof(splash_migrate_job) */
    const void *src_pool; const float *src_scales;
    void *dst_pool; float *dst_scales;
    int64_t page_bytes;
    const int32_t *src_page_ids, *dst_page_ids;
    int64_t n;
    int32_t src_id_base, dst_id_base, max_page_id;
    int32_t *block_table;
    int64_t num_table_entries;
    void *workspace;
    size_t workspace_bytes;
} splash_migrate_job;

SPLASH_API int splash_mla_decode_migrating(const splash_mla_shape *shape,
                      const void *q, const void *kv_pool, const float *kv_scales,
                      const int32_t *block_table, const int32_t *seq_lens,
                      int32_t head_begin, int32_t head_end,
                      const int32_t *kv_begin, const int32_t *kv_end,
                      float *out, float *lse,
                      void *workspace, size_t workspace_bytes, void *stream,
                      const splash_migrate_job *job);

/*
 * splash_kv_page_migrate without a workspace argument and without any allocation.
 * (The paper has no counterpart for this entry point; it exists for the library's
 * callers.)
 *
 * Who needs it: code that moves pages from a place where it may not allocate or
 * free device memory -- a serving loop that has already handed the whole HBM budget to
 * its KV pool and keeps no allocator of its own, a plugin or callback that runs under
 * a host framework's memory manager and must not call cudaMalloc behind its back, a
 * latency-critical path where an allocation (which can synchronise the device) is
 * not acceptable.  Such a caller has nowhere to get the remap table that
 * splash_kv_page_migrate wants as `workspace`.
 *
 * Here the table is a fixed array inside the library's own device image:
 * SPLASH_STATIC_MIGRATE_MAX_PAGE_ID (262,144) int32 entries = 1 MiB, present on every
 * GPU that loads the library for as long as the process lives.  Arguments, results and
 * error codes are those of splash_kv_page_migrate; in addition max_page_id above the
 * limit is rejected with SPLASH_INVALID_ARG and nothing is launched.  The function
 * calls no cudaMalloc / cudaFree and no allocating library routine.
 *
 *   - The first call on each device looks up the array's device address (a host-side
 *     query, no allocation); make that first call outside any stream capture.
 *   - All calls on a device share the one table, and it keeps the previous call's
 *     contents: each call first resets the entries [0, max_page_id) on `stream`.  Two
 *     calls that can overlap on the GPU (different streams, no ordering between them)
 *     race on it -- order them, or give one of them its own workspace through
 *     splash_kv_page_migrate.
 */
#define SPLASH_STATIC_MIGRATE_MAX_PAGE_ID (1 << 18)
SPLASH_API int splash_kv_page_migrate_static(const void *src_pool, const float *src_scales,
                                             void *dst_pool, float *dst_scales,
                                             int64_t page_bytes,
                                             const int32_t *src_page_ids, const int32_t *dst_page_ids, int64_t n,
                                             int32_t src_id_base, int32_t dst_id_base, int32_t max_page_id,
                                             int32_t *block_table, int64_t num_table_entries, void *stream);

/*
 * DOP transfer layout changes (App. E): the regrouping steps on either side of the two
 * all-to-alls that turn a tensor in global-row, local-head order (every rank holds its head
 * slice of all N rows) into owner-row, all-head order (every rank holds all heads of the rows
 * it owns) and back.  The collectives themselves are the caller's; these calls move whole
 * rows of bytes on one GPU, byte-exact, and keep row identity, head order and positions.
 * Sizes and pitches are in BYTES and must be even; when every pointer, size and pitch is a
 * multiple of 16 a 16-byte vector path is taken, otherwise a 2-byte scalar one.  n = 0 is a
 * successful no-op (ranks that own no rows still take part in the exchange).
 *
 * splash_dop_pack_rows: builds the send buffer of the forward exchange,
 *     send[p][j] = a[send_row[p]][j] ++ b[send_row[p]][j],    p < n, j < h,
 * where send_row lists the source rows grouped by destination owner (the caller derives the
 * all-to-all split sizes from the per-owner row counts) and a / b are the no-position and the
 * rotary part of the query (a_part_bytes / b_part_bytes per head; b may be NULL with
 * b_part_bytes = 0), fused so that one collective moves both.  Element (r, j) of a starts at
 * a + r*a_row_pitch + j*a_head_pitch.  send is dense: [n][h][a_part_bytes + b_part_bytes].
 *
 * splash_dop_swap_outer: out[r][s] = in[s][r] for blocks of inner_bytes, s < A, r < B.  With
 * A = T ranks, B = n owned rows and inner = h heads it turns the receive buffer of the forward
 * exchange (source-rank major) into all-head order [n][T*h] (head s*h + j from rank s); with
 * the roles swapped it builds the send buffer of the reverse exchange.
 *
 * splash_dop_unpack_rows: the reverse exchange's last step, out[send_row[p]] = recv[p] for rows
 * of row_bytes (recv dense, out rows out_row_pitch apart); rows not listed are left untouched.
 * send_row must not list a row twice.
 */
SPLASH_API int splash_dop_pack_rows(const void *a, int64_t a_part_bytes, int64_t a_row_pitch, int64_t a_head_pitch,
                                    const void *b, int64_t b_part_bytes, int64_t b_row_pitch, int64_t b_head_pitch,
                                    const int32_t *send_row, int64_t n, int32_t h, void *send, void *stream);
SPLASH_API int splash_dop_swap_outer(const void *in, int64_t A, int64_t B, int64_t inner_bytes, void *out, void *stream);
SPLASH_API int splash_dop_unpack_rows(const void *recv, const int32_t *send_row, int64_t n, int64_t row_bytes,
                                      void *out, int64_t out_row_pitch, void *stream);

/* Host-side helpers. */
SPLASH_API const char *splash_status_string(int status);
SPLASH_API const char *splash_last_error(void);
SPLASH_API int splash_version(void);

/* Number of kernels the last call of this thread enqueued (for launch accounting). */
SPLASH_API int splash_last_launch_count(void);

/*
 * Per-kernel timing of splash_mla_decode, for benchmarks.  While enabled (per host
 * thread), every decode call records CUDA events on its stream around its three
 * kernels (plan, decode, split combine); the events are created on first use.
 * splash_get_kernel_timing() synchronises on the last call's final event and returns
 * the three durations in milliseconds (host pointers, each may be NULL).  Off by
 * default; enabling it adds four event records per call and nothing else.  For
 * splash_mla_decode_sparse the decode figure covers the gather kernel and the decode kernel.
 */
SPLASH_API int splash_set_kernel_timing(int enable);
SPLASH_API int splash_get_kernel_timing(float *plan_ms, float *decode_ms, float *combine_ms);

/*
 * Diagnostics: give the decode kernel a device buffer of 64 x 8 + 512 int64 into which
 * CTA 0 writes SM-clock timestamps of its pipeline events for its first 64 tiles (event
 * order: stage free, TMA issued, tile landed, QK^T issued, S ready, P written, P seen,
 * P.V issued); every CTA also writes its total cycle count at [512 + CTA index].  NULL (the default) switches it off.  Per host thread.
 */
SPLASH_API int splash_debug_set_trace(void *device_buffer);

/*
 * Read the device status word at the head of a decode workspace after the caller
 * has synchronised the stream: SPLASH_OK, SPLASH_DEVICE_TIMEOUT if a bounded wait
 * inside a kernel gave up (the results of that call are then invalid), or, for a call
 * made with SPLASH_FLAG_VALIDATE, SPLASH_BAD_PAGE_ID.  The first event of a call wins
 * and stays until the next call on that workspace.  Performs a blocking 16-byte
 * device-to-host copy; not for the hot path.
 */
SPLASH_API int splash_workspace_status(const void *workspace, int32_t *detail /* host, [3], may be NULL */);

#ifdef __cplusplus
}
#endif
#endif /* SPLASH_MLA_H_ */
