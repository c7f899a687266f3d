// C ABI entry points: argument validation, workspace carving, kernel sequencing.
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <string>

#include "splash_common.cuh"

namespace splash {

namespace {
thread_local std::string g_last_error;
thread_local int g_launches = 0;
thread_local bool g_timing = false;
thread_local long long *g_trace = nullptr;
thread_local cudaEvent_t g_events[4] = {nullptr, nullptr, nullptr, nullptr};
thread_local bool g_events_recorded = false;

cudaError_t record_timing_event(int k, cudaStream_t stream) {
    if (!g_timing) return cudaSuccess;
    if (g_events[k] == nullptr) {
        cudaError_t e = cudaEventCreate(&g_events[k]);
        if (e != cudaSuccess) return e;
    }
    return cudaEventRecord(g_events[k], stream);
}

struct DeviceInfo {
    int device = -1;
    int sm_count = 0;
    int cc_major = 0;
    bool ok = false;
};

// Properties of the current device (cached per device index, under a lock: host threads may make their first calls
// at the same time).
bool current_device_info(DeviceInfo &info) {
    static DeviceInfo cache[64];
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { set_error("cudaGetDevice failed"); return false; }
    std::lock_guard<std::mutex> lock(mu);
    if (dev >= 0 && dev < 64 && cache[dev].ok) { info = cache[dev]; return true; }
    DeviceInfo d;
    d.device = dev;
    if (cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&d.cc_major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
        set_error("cudaDeviceGetAttribute failed");
        return false;
    }
    d.ok = true;
    if (dev >= 0 && dev < 64) cache[dev] = d;
    info = d;
    return true;
}

bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

int check_shape(const splash_mla_shape *s, int32_t head_begin, int32_t head_end) {
    if (s == nullptr) { set_error("shape is NULL"); return SPLASH_INVALID_ARG; }
    if (s->struct_size != sizeof(splash_mla_shape)) {
        set_error("shape.struct_size is %u, this library expects %zu", s->struct_size, sizeof(splash_mla_shape));
        return SPLASH_INVALID_ARG;
    }
    if (s->num_requests < 0) { set_error("num_requests < 0"); return SPLASH_INVALID_ARG; }
    if (s->num_heads < 1 || s->num_heads > kMaxHeads) { set_error("num_heads must be in [1, 128]"); return SPLASH_UNSUPPORTED; }
    if (s->d_qk != kDQK || s->d_v != kDV) { set_error("only d_qk = 576, d_v = 512 is built"); return SPLASH_UNSUPPORTED; }
    if (s->page_size != kPage) { set_error("only page_size = 64 is built"); return SPLASH_UNSUPPORTED; }
    if (s->kv_dtype != SPLASH_KV_BF16 && s->kv_dtype != SPLASH_KV_E4M3_TOKEN_SCALE) {
        set_error("unknown kv_dtype %d", s->kv_dtype); return SPLASH_UNSUPPORTED;
    }
    if (head_begin < 0 || head_end > s->num_heads || head_begin > head_end) {
        set_error("head slice [%d, %d) is not inside [0, %d)", head_begin, head_end, s->num_heads);
        return SPLASH_INVALID_ARG;
    }
    if (s->num_pool_pages < 0 || s->block_table_stride < 0) { set_error("negative pool / table size"); return SPLASH_INVALID_ARG; }
    if (s->q_stride_request % 8 || s->q_stride_head % 8 || s->q_stride_head < kDQK) {
        set_error("q strides must be multiples of 8 elements and q_stride_head >= 576"); return SPLASH_INVALID_ARG;
    }
    if (s->out_stride_request % 4 || s->out_stride_head % 4 || s->out_stride_head < kDV) {
        set_error("out strides must be multiples of 4 elements and out_stride_head >= 512"); return SPLASH_INVALID_ARG;
    }
    if (s->lse_stride_request < s->num_heads && s->num_requests > 1) { set_error("lse_stride_request < num_heads"); return SPLASH_INVALID_ARG; }
    if (!(s->softmax_scale == s->softmax_scale)) { set_error("softmax_scale is NaN"); return SPLASH_INVALID_ARG; }
    if (s->q_rows > (uint32_t)kMaxQRows) { set_error("q_rows must be in [1, %d] (0 = 1)", kMaxQRows); return SPLASH_UNSUPPORTED; }
    if (s->q_rows > 1) {
        const int64_t R = s->q_rows;
        if (s->q_stride_head != R * kDQK || s->out_stride_head != R * kDV) {
            set_error("with q_rows = R > 1 the rows of a head are dense: q_stride_head = R * 576, out_stride_head = R * 512");
            return SPLASH_INVALID_ARG;
        }
        if (s->lse_stride_request < s->num_heads * R && s->num_requests > 1) { set_error("lse_stride_request < num_heads * q_rows"); return SPLASH_INVALID_ARG; }
        if (s->flags & SPLASH_FLAG_NO_PAIR) { set_error("q_rows > 1 runs on the CTA-pair kernels only"); return SPLASH_UNSUPPORTED; }
    }
    return SPLASH_OK;
}

// How one decode call is cut into CTAs.
struct Tiling { int heads_per_group, num_groups, num_workers, pair_groups; };

// h = width of the slice in (virtual) heads
Tiling choose_tiling(const splash_mla_shape *s, int h, int sm_count, bool simt) {
    Tiling t;
    t.pair_groups = 1;
    if (!simt && s->q_rows > 1) {      // several query rows per request: always CTA pairs, whatever the width
        // more than 128 (head, row) pairs: several pairs per KV worker, side by side on the same pages
        t.heads_per_group = 64; t.num_groups = 2;
        t.pair_groups = (h + kMaxHeads - 1) / kMaxHeads;
        const int w = (sm_count / 2) / t.pair_groups;
        t.num_workers = w > 0 ? w : 1;
        return t;
    }
    if (simt) {
        t.heads_per_group = simt_heads_per_group();
        t.num_groups = (h + t.heads_per_group - 1) / t.heads_per_group;
        // two CTAs per SM's worth of KV workers in total, at least one
        int w = (2 * sm_count) / t.num_groups;
        t.num_workers = w > 0 ? w : 1;
        return t;
    }
    umma_tiling(s->kv_dtype, h, sm_count, &t.heads_per_group, &t.num_groups, &t.num_workers);
    return t;
}

}  // namespace

void set_error(const char *fmt, ...) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    g_last_error = buf;
}

void count_launch(int n) { g_launches += n; }

}  // namespace splash

using namespace splash;

extern "C" {

size_t splash_mla_decode_workspace_bytes(const splash_mla_shape *shape, int32_t head_begin, int32_t head_end) {
    if (check_shape(shape, head_begin, head_end) != SPLASH_OK) return 0;
    DeviceInfo dev;
    if (!current_device_info(dev)) return 0;
    // with R query rows per request the call runs over virtual heads, at most kMaxHeads of them at a time
    const int R = shape->q_rows > 1 ? (int)shape->q_rows : 1;
    const int h = (head_end - head_begin) * R;
    if (h == 0 || shape->num_requests == 0) return 256;
    // the larger of the two kernels' needs, so one workspace serves both paths
    size_t need = 0;
    for (int simt = 0; simt < 2; ++simt) {
        Tiling t = choose_tiling(shape, h, dev.sm_count, simt != 0);
        PlanView v = make_plan_view(nullptr, shape->num_requests, t.num_workers, h);
        if (v.bytes > need) need = v.bytes;
    }
    return align_up(need, 256);
}

}  // extern "C"

namespace {

// The first stage of a sparse call: gathers the listed rows into the dense cache that the decode then reads.
struct SparseStage {
    const void *pool656;
    int num_pool_pages;
    const int32_t *block_table;
    int64_t table_stride;
    const int32_t *ctx_lens, *sel, *sel_count;
    int64_t sel_stride;
    int max_selected, pages_per_request;
    int32_t *dense_table;
    bool fused;        // one kernel gathers, dequantises and multiplies (CTA pairs); else gather kernel + dense kernels
};

// Argument checks shared by the page-migration entry points (the workspace variant, the job of a decode call).
int check_migrate_args(const void *src_pool, const float *src_scales, const void *dst_pool, const float *dst_scales,
                       int64_t page_bytes, const int32_t *src_page_ids, const int32_t *dst_page_ids, int64_t n,
                       int32_t max_page_id, const int32_t *block_table, int64_t num_table_entries,
                       const void *workspace, size_t workspace_bytes) {
    if (n < 0 || num_table_entries < 0 || page_bytes <= 0 || page_bytes % 16 || max_page_id < 0) {
        set_error("bad sizes (page_bytes must be a positive multiple of 16)"); return SPLASH_INVALID_ARG;
    }
    if (n == 0) return SPLASH_OK;   // nothing moves, the table keeps every entry
    if (!src_pool || !dst_pool || !src_page_ids || !dst_page_ids) { set_error("a required pointer is NULL"); return SPLASH_INVALID_ARG; }
    if ((src_scales == nullptr) != (dst_scales == nullptr)) { set_error("give both scale pools or neither"); return SPLASH_INVALID_ARG; }
    if (num_table_entries > 0 && (!block_table || !workspace)) { set_error("block_table / workspace is NULL"); return SPLASH_INVALID_ARG; }
    if (!aligned(src_pool, 16) || !aligned(dst_pool, 16) || !aligned(src_scales, 16) || !aligned(dst_scales, 16) ||
        !aligned(workspace, 16)) {
        set_error("misaligned pointer (pools, scales, workspace: 16 B)"); return SPLASH_INVALID_ARG;
    }
    if (num_table_entries > 0 && workspace_bytes < splash_kv_page_migrate_workspace_bytes(max_page_id)) {
        set_error("workspace too small"); return SPLASH_INVALID_ARG;
    }
    if (n > 0x7fffffffLL) { set_error("too many pages"); return SPLASH_INVALID_ARG; }
    return SPLASH_OK;
}

int check_migrate_job(const splash_migrate_job *job) {
    if (job->struct_size != sizeof(splash_migrate_job)) {
        set_error("job.struct_size is %u, this library expects %zu", job->struct_size, sizeof(splash_migrate_job));
        return SPLASH_INVALID_ARG;
    }
    return check_migrate_args(job->src_pool, job->src_scales, job->dst_pool, job->dst_scales, job->page_bytes, job->src_page_ids,
                              job->dst_page_ids, job->n, job->max_page_id, job->block_table, job->num_table_entries,
                              job->workspace, job->workspace_bytes);
}

cudaError_t run_migrate_job(const splash_migrate_job *job, bool do_table, bool do_copy, cudaStream_t stream) {
    return launch_page_migrate(job->src_pool, job->src_scales, job->dst_pool, job->dst_scales, job->page_bytes, job->src_page_ids,
                               job->dst_page_ids, job->n, job->src_id_base, job->dst_id_base, job->max_page_id, job->block_table,
                               job->num_table_entries, static_cast<int32_t *>(job->workspace), do_table, do_copy, stream);
}

// One dense decode call: plan, decode kernel, combine.  With a sparse stage, seq_lens are the list counts, kv_pool
// and block_table the dense cache and its table, and the gather kernel runs between the plan and the decode kernel.
int decode_dense(const splash_mla_shape *shape, const void *q, const void *kv_pool, const float *kv_scales,
                 const int32_t *block_table, const int32_t *seq_lens, int32_t head_begin, int32_t head_end,
                 const int32_t *kv_begin, const int32_t *kv_end, float *out, float *lse,
                 void *workspace, size_t workspace_bytes, void *stream_, const SparseStage *sparse,
                 const splash_migrate_job *job = nullptr) {
    g_launches = 0;
    int rc = check_shape(shape, head_begin, head_end);
    if (rc != SPLASH_OK) return rc;
    if (job != nullptr) {
        rc = check_migrate_job(job);
        if (rc != SPLASH_OK) return rc;
        if (job->n == 0) job = nullptr;
    }
    const int B = shape->num_requests;
    if (B == 0 || head_end == head_begin) {     // idle rank: no attention to compute; its pages still move
        if (job != nullptr) {
            cudaError_t e = run_migrate_job(job, true, true, static_cast<cudaStream_t>(stream_));
            if (e != cudaSuccess) { set_error("CUDA error: %s", cudaGetErrorString(e)); return SPLASH_CUDA_ERROR; }
        }
        return SPLASH_OK;
    }
    if (!q || !kv_pool || !block_table || !seq_lens || !out || !lse || !workspace) {
        set_error("a required pointer is NULL"); return SPLASH_INVALID_ARG;
    }
    if (shape->kv_dtype == SPLASH_KV_E4M3_TOKEN_SCALE && !kv_scales) { set_error("kv_scales is NULL for e4m3 KV"); return SPLASH_INVALID_ARG; }
    if (shape->kv_dtype == SPLASH_KV_BF16 && kv_scales) { set_error("kv_scales must be NULL for bf16 KV"); return SPLASH_INVALID_ARG; }
    if (!aligned(q, 16) || !aligned(kv_pool, 128) || !aligned(out, 16) || !aligned(lse, 4) ||
        !aligned(workspace, 256) || (kv_scales && !aligned(kv_scales, 16)) || !aligned(block_table, 4) ||
        !aligned(seq_lens, 4)) {
        set_error("misaligned pointer (q/out/kv_scales 16 B, kv_pool 128 B, workspace 256 B)"); return SPLASH_INVALID_ARG;
    }
    DeviceInfo dev;
    if (!current_device_info(dev)) return SPLASH_CUDA_ERROR;
    if (dev.cc_major != 10) { set_error("device compute capability %d.x is not 10.x", dev.cc_major); return SPLASH_UNSUPPORTED_DEVICE; }

    const bool simt = (shape->flags & SPLASH_FLAG_SIMT) != 0;
    // R query rows per request: the kernels see R * num_heads virtual heads (head g, row r -> g * R + r: the rows
    // of a head are dense, so a virtual head is 576 / 512 elements from the next) and mask causally by
    // (virtual head mod R); a slice wider than 128 virtual heads runs as several CTA pairs per KV worker in ONE launch
    // chain (the loop below has a single pass).
    const int R = shape->q_rows > 1 ? (int)shape->q_rows : 1;
    const int vbegin = head_begin * R, vend = head_end * R;
    const int vstep = vend - vbegin;
    cudaError_t e = cudaSuccess;
    // a page-copy job: its table rewrite runs first; its page copy rides in the decode kernel if that is a CTA-pair
    // kernel (one pass only), else runs as a kernel of its own after the decode
    bool job_copy_pending = job != nullptr;
    if (job != nullptr) e = run_migrate_job(job, true, false, static_cast<cudaStream_t>(stream_));
    for (int vb = vbegin; vb < vend && e == cudaSuccess; vb += vstep) {
    const int ve = vb + vstep < vend ? vb + vstep : vend;
    const int h = ve - vb;
    Tiling t = choose_tiling(shape, h, dev.sm_count, simt);
    const bool fused_sparse = sparse && sparse->fused && !simt;
    if (fused_sparse) { t.heads_per_group = 64; t.num_groups = 2; t.num_workers = dev.sm_count / 2 > 0 ? dev.sm_count / 2 : 1; t.pair_groups = 1; }
    PlanView v = make_plan_view(workspace, B, t.num_workers, h);
    if (workspace_bytes < v.bytes) {
        set_error("workspace has %zu bytes, %zu needed", workspace_bytes, v.bytes); return SPLASH_INVALID_ARG;
    }
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);

    DecodeParams p;
    memset(&p, 0, sizeof p);
    p.q = q; p.kv_pool = kv_pool; p.kv_scales = kv_scales; p.block_table = block_table; p.seq_lens = seq_lens;
    p.out = out; p.lse = lse;
    p.q_stride_request = shape->q_stride_request; p.q_stride_head = R > 1 ? kDQK : shape->q_stride_head;
    p.out_stride_request = shape->out_stride_request; p.out_stride_head = R > 1 ? kDV : shape->out_stride_head;
    p.lse_stride_request = shape->lse_stride_request;
    p.B = B; p.H = shape->num_heads * R; p.head_begin = vb; p.head_end = ve; p.q_rows = R;
    p.table_stride = shape->block_table_stride; p.num_pool_pages = shape->num_pool_pages;
    p.heads_per_group = t.heads_per_group; p.num_groups = t.num_groups; p.num_workers = t.num_workers;
    p.pair_groups = t.pair_groups;
    p.softmax_scale = shape->softmax_scale;
    p.tile_start = v.tile_start; p.req_lo = v.req_lo; p.req_hi = v.req_hi; p.worker_begin = v.worker_begin;
    p.worker_req = v.worker_req;
    p.status = v.status; p.partial_lse = v.partial_lse; p.partial_out = v.partial_out; p.partial_scale = v.partial_scale;
    p.trace = g_trace;
    p.len_cap = sparse ? sparse->max_selected : -1;
    if (fused_sparse) {
        p.kv_pool = sparse->pool656; p.block_table = sparse->block_table; p.table_stride = sparse->table_stride;
        p.num_pool_pages = sparse->num_pool_pages; p.sel = sparse->sel; p.sel_stride = sparse->sel_stride;
        p.ctx_lens = sparse->ctx_lens;
    }
    p.request_overhead_tiles = kRequestOverheadTilesDefault;
    const bool pair = !simt && t.num_groups == 2 && t.heads_per_group == 64 && !(shape->flags & SPLASH_FLAG_NO_PAIR);
    if (!simt && shape->kv_dtype == SPLASH_KV_E4M3_TOKEN_SCALE)
        p.request_overhead_tiles = pair ? kRequestOverheadTilesFp8Pair : kRequestOverheadTilesFp8;
    else if (pair)
        p.request_overhead_tiles = kRequestOverheadTilesPair;
    // the bf16 CTA-pair kernel writes its partial outputs as f16
    p.partial_f16 = (pair && shape->kv_dtype == SPLASH_KV_BF16 && !fused_sparse) ? 1 : 0;
    if (job_copy_pending && pair && !fused_sparse && vend - vbegin <= vstep) {
        p.mig_src = static_cast<const uint4 *>(job->src_pool); p.mig_dst = static_cast<uint4 *>(job->dst_pool);
        p.mig_src_scales = reinterpret_cast<const uint4 *>(job->src_scales); p.mig_dst_scales = reinterpret_cast<uint4 *>(job->dst_scales);
        p.mig_src_ids = job->src_page_ids; p.mig_dst_ids = job->dst_page_ids;
        p.mig_page_vecs = job->page_bytes / 16; p.mig_n = (int32_t)job->n;
        job_copy_pending = false;
    }

    // the previous call's partition taken again (the same batch in the next layer): no plan kernel, only the error words
    // of the status block are cleared (word 8, the number of split requests, belongs to the plan)
    const bool reuse_plan = (shape->flags & SPLASH_FLAG_REUSE_PLAN) && !(shape->flags & SPLASH_FLAG_VALIDATE) && !sparse;
    e = record_timing_event(0, stream);
    if (e == cudaSuccess) {
        if (reuse_plan) {
            if (vb == vbegin) e = cudaMemsetAsync(v.status, 0, 8 * sizeof(int32_t), stream);
        } else {
            e = launch_plan(p, kv_begin, kv_end, v.tile_start, v.req_lo, v.req_hi, v.req_wfirst, v.req_wlast,
                            v.cost_start, v.worker_begin, v.split_list, v.worker_req, v.split_rec, v.status, vb == vbegin, stream);
        }
    }
    if (e == cudaSuccess) e = record_timing_event(1, stream);
    // validation mode: the table entries the call will use, checked on the device before the decode kernel runs
    if (e == cudaSuccess && (shape->flags & SPLASH_FLAG_VALIDATE) && !sparse && vb == vbegin)
        e = launch_validate_pages(p, v.req_lo, v.req_hi, stream);
    if (e == cudaSuccess && sparse && !fused_sparse)
        e = launch_sparse_gather(B, sparse->max_selected, sparse->pages_per_request, sparse->pool656, sparse->num_pool_pages,
                                 sparse->block_table, sparse->table_stride, sparse->ctx_lens, sparse->sel, sparse->sel_stride,
                                 sparse->sel_count, const_cast<void *>(kv_pool), sparse->dense_table, dev.sm_count, stream);
    if (e == cudaSuccess) {
        if (simt) e = launch_decode_simt(p, shape->kv_dtype, stream);
        else if (fused_sparse) e = launch_decode_sparse_pair(p, stream);
        else e = launch_decode_umma(p, *shape, stream);
    }
    if (e == cudaSuccess) e = record_timing_event(2, stream);
    if (e == cudaSuccess) e = launch_split_combine(p, v.split_rec, stream);
    if (e == cudaSuccess) e = record_timing_event(3, stream);
    if (e == cudaSuccess && g_timing) g_events_recorded = true;
    }
    if (e == cudaSuccess && job_copy_pending) e = run_migrate_job(job, false, true, static_cast<cudaStream_t>(stream_));
    if (e != cudaSuccess) { set_error("CUDA error: %s", cudaGetErrorString(e)); return SPLASH_CUDA_ERROR; }
    return SPLASH_OK;
}

}  // namespace

extern "C" {

int splash_mla_decode(const splash_mla_shape *shape, const void *q, const void *kv_pool, const float *kv_scales,
                      const int32_t *block_table, const int32_t *seq_lens, int32_t head_begin, int32_t head_end,
                      const int32_t *kv_begin, const int32_t *kv_end, float *out, float *lse,
                      void *workspace, size_t workspace_bytes, void *stream_) {
    return decode_dense(shape, q, kv_pool, kv_scales, block_table, seq_lens, head_begin, head_end, kv_begin, kv_end, out, lse,
                        workspace, workspace_bytes, stream_, nullptr);
}

int splash_mla_decode_migrating(const splash_mla_shape *shape, const void *q, const void *kv_pool, const float *kv_scales,
                                const int32_t *block_table, const int32_t *seq_lens, int32_t head_begin, int32_t head_end,
                                const int32_t *kv_begin, const int32_t *kv_end, float *out, float *lse,
                                void *workspace, size_t workspace_bytes, void *stream_, const splash_migrate_job *job) {
    return decode_dense(shape, q, kv_pool, kv_scales, block_table, seq_lens, head_begin, head_end, kv_begin, kv_end, out, lse,
                        workspace, workspace_bytes, stream_, nullptr, job);
}

namespace {

// Workspace of a sparse call: [dense decode workspace][dense table B * ppr][dense cache].
struct SparseView {
    splash_mla_shape dense;        // the shape of the dense call over the gathered cache
    int pages_per_request;
    size_t inner_bytes, off_table, off_pool, bytes;
};

bool make_sparse_view(const splash_mla_shape *shape, int32_t max_selected, int32_t head_begin, int32_t head_end, SparseView &v) {
    if (shape == nullptr || shape->struct_size != sizeof(splash_mla_shape)) { set_error("shape is NULL or of another version"); return false; }
    if (shape->kv_dtype != SPLASH_KV_E4M3_BLOCK_SCALE_BF16_ROPE) { set_error("sparse decode reads kv_dtype 2 (656-byte rows) only"); return false; }
    if (shape->q_rows > 1) { set_error("sparse decode takes one query row per request"); return false; }
    if (max_selected < 0 || max_selected > (1 << 20)) { set_error("max_selected must be in [0, 2^20]"); return false; }
    v.dense = *shape;
    v.dense.kv_dtype = SPLASH_KV_BF16;
    v.pages_per_request = max_selected > 0 ? (max_selected + kPage - 1) / kPage : 1;
    const int64_t pages = (int64_t)shape->num_requests * v.pages_per_request;
    if (pages > 0x7fffffffLL / kPage) { set_error("num_requests * max_selected is too large"); return false; }
    v.dense.num_pool_pages = (int32_t)pages;
    v.dense.block_table_stride = v.pages_per_request;
    if (check_shape(&v.dense, head_begin, head_end) != SPLASH_OK) return false;
    v.inner_bytes = splash_mla_decode_workspace_bytes(&v.dense, head_begin, head_end);
    if (v.inner_bytes == 0) return false;
    size_t off = align_up(v.inner_bytes, 256);
    v.off_table = off; off = align_up(off + sizeof(int32_t) * (size_t)pages, 256);
    v.off_pool = off; off += (size_t)pages * kPage * kDQK * 2;
    v.bytes = align_up(off, 256);
    return true;
}

}  // namespace

size_t splash_mla_decode_sparse_workspace_bytes(const splash_mla_shape *shape, int32_t max_selected, int32_t head_begin,
                                                int32_t head_end) {
    SparseView v;
    return make_sparse_view(shape, max_selected, head_begin, head_end, v) ? v.bytes : 0;
}

int splash_mla_decode_sparse(const splash_mla_shape *shape, const void *q, const void *kv_pool, const int32_t *block_table,
                             const int32_t *seq_lens, const int32_t *sel_tokens, int64_t sel_stride, const int32_t *sel_count,
                             int32_t max_selected, int32_t head_begin, int32_t head_end, float *out, float *lse,
                             void *workspace, size_t workspace_bytes, void *stream_) {
    g_launches = 0;
    SparseView v;
    if (!make_sparse_view(shape, max_selected, head_begin, head_end, v)) return SPLASH_INVALID_ARG;
    const int B = shape->num_requests;
    if (B == 0 || head_end == head_begin) return SPLASH_OK;
    if (!q || !kv_pool || !block_table || !seq_lens || !sel_count || !out || !lse || !workspace || (max_selected > 0 && !sel_tokens)) {
        set_error("a required pointer is NULL"); return SPLASH_INVALID_ARG;
    }
    if (!aligned(kv_pool, 128) || !aligned(workspace, 256) || !aligned(sel_tokens, 4) || !aligned(sel_count, 4) ||
        !aligned(block_table, 4) || !aligned(seq_lens, 4)) {
        set_error("misaligned pointer (kv_pool 128 B, workspace 256 B)"); return SPLASH_INVALID_ARG;
    }
    if (sel_stride < max_selected && B > 1) { set_error("sel_stride < max_selected"); return SPLASH_INVALID_ARG; }
    if (workspace_bytes < v.bytes) { set_error("workspace has %zu bytes, %zu needed", workspace_bytes, v.bytes); return SPLASH_INVALID_ARG; }
    DeviceInfo dev;
    if (!current_device_info(dev)) return SPLASH_CUDA_ERROR;
    if (dev.cc_major != 10) { set_error("device compute capability %d.x is not 10.x", dev.cc_major); return SPLASH_UNSUPPORTED_DEVICE; }
    char *ws = static_cast<char *>(workspace);
    SparseStage st;
    st.pool656 = kv_pool; st.num_pool_pages = shape->num_pool_pages; st.block_table = block_table;
    st.table_stride = shape->block_table_stride; st.ctx_lens = seq_lens; st.sel = sel_tokens; st.sel_count = sel_count;
    st.sel_stride = sel_stride; st.max_selected = max_selected; st.pages_per_request = v.pages_per_request;
    st.dense_table = reinterpret_cast<int32_t *>(ws + v.off_table);
    st.fused = (shape->flags & SPLASH_FLAG_SPARSE_FUSED) != 0 && (shape->flags & (SPLASH_FLAG_NO_PAIR | SPLASH_FLAG_SIMT)) == 0;
    // plan (over the list counts) -> gather into the dense cache -> decode kernel over the dense cache -> combine
    return decode_dense(&v.dense, q, ws + v.off_pool, nullptr, st.dense_table, sel_count, head_begin, head_end, nullptr, nullptr,
                        out, lse, workspace, v.inner_bytes, stream_, &st);
}

int splash_lse_merge(int32_t num_parts, int64_t rows, int32_t d_v, const float *part_out, const float *part_lse,
                     float *out, float *lse, void *stream_) {
    g_launches = 0;
    if (num_parts < 0 || rows < 0 || d_v <= 0 || d_v % 4) { set_error("bad sizes (d_v must be a positive multiple of 4)"); return SPLASH_INVALID_ARG; }
    if (rows == 0) return SPLASH_OK;
    if (!out || !lse || (num_parts > 0 && (!part_out || !part_lse))) { set_error("a required pointer is NULL"); return SPLASH_INVALID_ARG; }
    if (!aligned(part_out, 16) || !aligned(out, 16) || !aligned(part_lse, 4) || !aligned(lse, 4)) {
        set_error("misaligned pointer"); return SPLASH_INVALID_ARG;
    }
    if (rows > 0x7fffffffLL) { set_error("too many rows"); return SPLASH_INVALID_ARG; }
    if (num_parts > 0) {
        const char *po = reinterpret_cast<const char *>(part_out);
        const char *oo = reinterpret_cast<const char *>(out);
        size_t pbytes = (size_t)num_parts * rows * d_v * 4, obytes = (size_t)rows * d_v * 4;
        if (oo < po + pbytes && po < oo + obytes) { set_error("out aliases part_out"); return SPLASH_INVALID_ARG; }
    }
    cudaError_t e = launch_lse_merge(num_parts, rows, d_v, part_out, part_lse, out, lse, static_cast<cudaStream_t>(stream_));
    if (e != cudaSuccess) { set_error("CUDA error: %s", cudaGetErrorString(e)); return SPLASH_CUDA_ERROR; }
    return SPLASH_OK;
}

size_t splash_kv_page_migrate_workspace_bytes(int32_t max_page_id) {
    if (max_page_id < 0) return 0;
    return align_up(sizeof(int32_t) * (size_t)max_page_id, 256) + 256;
}

int splash_kv_page_migrate(const void *src_pool, const float *src_scales, void *dst_pool, float *dst_scales,
                           int64_t page_bytes, const int32_t *src_page_ids, const int32_t *dst_page_ids, int64_t n,
                           int32_t src_id_base, int32_t dst_id_base, int32_t max_page_id,
                           int32_t *block_table, int64_t num_table_entries,
                           void *workspace, size_t workspace_bytes, void *stream_) {
    g_launches = 0;
    const int rc = check_migrate_args(src_pool, src_scales, dst_pool, dst_scales, page_bytes, src_page_ids, dst_page_ids, n,
                                      max_page_id, block_table, num_table_entries, workspace, workspace_bytes);
    if (rc != SPLASH_OK || n == 0) return rc;
    cudaError_t e = launch_page_migrate(src_pool, src_scales, dst_pool, dst_scales, page_bytes, src_page_ids,
                                        dst_page_ids, n, src_id_base, dst_id_base, max_page_id, block_table,
                                        num_table_entries, static_cast<int32_t *>(workspace), true, true,
                                        static_cast<cudaStream_t>(stream_));
    if (e != cudaSuccess) { set_error("CUDA error: %s", cudaGetErrorString(e)); return SPLASH_CUDA_ERROR; }
    return SPLASH_OK;
}

int splash_kv_page_migrate_static(const void *src_pool, const float *src_scales, void *dst_pool, float *dst_scales,
                                  int64_t page_bytes, const int32_t *src_page_ids, const int32_t *dst_page_ids,
                                  int64_t n, int32_t src_id_base, int32_t dst_id_base, int32_t max_page_id,
                                  int32_t *block_table, int64_t num_table_entries, void *stream_) {
    g_launches = 0;
    if (max_page_id > kStaticMigrateMaxPageId) {
        set_error("max_page_id %d exceeds the built-in remap table of %d entries; use splash_kv_page_migrate "
                  "with a caller-provided workspace", max_page_id, kStaticMigrateMaxPageId);
        return SPLASH_INVALID_ARG;
    }
    if (n < 0 || num_table_entries < 0 || page_bytes <= 0 || page_bytes % 16 || max_page_id < 0) {
        set_error("bad sizes (page_bytes must be a positive multiple of 16)"); return SPLASH_INVALID_ARG;
    }
    if (n == 0) return SPLASH_OK;
    if (!src_pool || !dst_pool || !src_page_ids || !dst_page_ids) { set_error("a required pointer is NULL"); return SPLASH_INVALID_ARG; }
    if ((src_scales == nullptr) != (dst_scales == nullptr)) { set_error("give both scale pools or neither"); return SPLASH_INVALID_ARG; }
    if (num_table_entries > 0 && !block_table) { set_error("block_table is NULL"); return SPLASH_INVALID_ARG; }
    if (!aligned(src_pool, 16) || !aligned(dst_pool, 16) || !aligned(src_scales, 16) || !aligned(dst_scales, 16)) {
        set_error("misaligned pointer (pools, scales: 16 B)"); return SPLASH_INVALID_ARG;
    }
    if (n > 0x7fffffffLL) { set_error("too many pages"); return SPLASH_INVALID_ARG; }
    int32_t *remap = nullptr;
    cudaError_t e = static_remap_address(&remap);      // first call on a device looks the symbol up
    if (e != cudaSuccess) { set_error("cudaGetSymbolAddress failed: %s", cudaGetErrorString(e)); return SPLASH_CUDA_ERROR; }
    e = launch_page_migrate(src_pool, src_scales, dst_pool, dst_scales, page_bytes, src_page_ids, dst_page_ids, n,
                            src_id_base, dst_id_base, max_page_id, block_table, num_table_entries, remap, true, true,
                            static_cast<cudaStream_t>(stream_));
    if (e != cudaSuccess) { set_error("CUDA error: %s", cudaGetErrorString(e)); return SPLASH_CUDA_ERROR; }
    return SPLASH_OK;
}

const char *splash_status_string(int status) {
    switch (status) {
        case SPLASH_OK: return "ok";
        case SPLASH_INVALID_ARG: return "invalid argument";
        case SPLASH_UNSUPPORTED: return "unsupported shape";
        case SPLASH_UNSUPPORTED_DEVICE: return "unsupported device";
        case SPLASH_CUDA_ERROR: return "CUDA error";
        case SPLASH_DEVICE_TIMEOUT: return "device wait timed out";
        case SPLASH_BAD_PAGE_ID: return "block-table entry outside the pool";
        default: return "unknown status";
    }
}

const char *splash_last_error(void) { return g_last_error.c_str(); }

int splash_version(void) { return 100; }

int splash_last_launch_count(void) { return g_launches; }

int splash_debug_set_trace(void *device_buffer) {
    g_trace = static_cast<long long *>(device_buffer);
    return SPLASH_OK;
}

int splash_set_kernel_timing(int enable) {
    g_timing = enable != 0;
    if (!g_timing) g_events_recorded = false;
    return SPLASH_OK;
}

int splash_dop_pack_rows(const void *a, int64_t a_part_bytes, int64_t a_row_pitch, int64_t a_head_pitch,
                         const void *b, int64_t b_part_bytes, int64_t b_row_pitch, int64_t b_head_pitch,
                         const int32_t *send_row, int64_t n, int32_t h, void *send, void *stream_) {
    g_launches = 0;
    if (n < 0 || h < 0 || a_part_bytes <= 0 || b_part_bytes < 0) { set_error("negative size"); return SPLASH_INVALID_ARG; }
    if (n == 0 || h == 0) return SPLASH_OK;
    if (!a || !send || !send_row || (b_part_bytes > 0 && !b)) { set_error("a required pointer is NULL"); return SPLASH_INVALID_ARG; }
    if (b_part_bytes == 0) { b = nullptr; b_row_pitch = b_head_pitch = 0; }
    if (((a_part_bytes | b_part_bytes | a_row_pitch | a_head_pitch | b_row_pitch | b_head_pitch) & 1) || !aligned(a, 2) ||
        !aligned(send, 2) || (b && !aligned(b, 2)) || !aligned(send_row, 4)) {
        set_error("sizes, pitches and pointers must be even"); return SPLASH_INVALID_ARG;
    }
    if (a_head_pitch < a_part_bytes || (b && b_head_pitch < b_part_bytes)) { set_error("head pitch smaller than the part"); return SPLASH_INVALID_ARG; }
    if (n > 0x7fffffffLL) { set_error("too many rows"); return SPLASH_INVALID_ARG; }
    DeviceInfo dev;
    if (!current_device_info(dev)) return SPLASH_CUDA_ERROR;
    cudaError_t e = launch_dop_pack_rows(a, b, send, send_row, n, h, a_part_bytes, b_part_bytes, a_row_pitch, a_head_pitch,
                                         b_row_pitch, b_head_pitch, dev.sm_count, static_cast<cudaStream_t>(stream_));
    if (e != cudaSuccess) { set_error("CUDA error: %s", cudaGetErrorString(e)); return SPLASH_CUDA_ERROR; }
    return SPLASH_OK;
}

int splash_dop_swap_outer(const void *in, int64_t A, int64_t B, int64_t inner_bytes, void *out, void *stream_) {
    g_launches = 0;
    if (A < 0 || B < 0 || inner_bytes < 0 || (inner_bytes & 1)) { set_error("negative or odd size"); return SPLASH_INVALID_ARG; }
    if (A == 0 || B == 0 || inner_bytes == 0) return SPLASH_OK;
    if (!in || !out || !aligned(in, 2) || !aligned(out, 2)) { set_error("a required pointer is NULL or odd"); return SPLASH_INVALID_ARG; }
    {
        const char *pi = static_cast<const char *>(in), *po = static_cast<const char *>(out);
        const int64_t bytes = A * B * inner_bytes;
        if (po < pi + bytes && pi < po + bytes) { set_error("out overlaps in"); return SPLASH_INVALID_ARG; }
    }
    DeviceInfo dev;
    if (!current_device_info(dev)) return SPLASH_CUDA_ERROR;
    cudaError_t e = launch_dop_swap_outer(in, out, A, B, inner_bytes, dev.sm_count, static_cast<cudaStream_t>(stream_));
    if (e != cudaSuccess) { set_error("CUDA error: %s", cudaGetErrorString(e)); return SPLASH_CUDA_ERROR; }
    return SPLASH_OK;
}

int splash_dop_unpack_rows(const void *recv, const int32_t *send_row, int64_t n, int64_t row_bytes, void *out,
                           int64_t out_row_pitch, void *stream_) {
    g_launches = 0;
    if (n < 0 || row_bytes < 0 || ((row_bytes | out_row_pitch) & 1)) { set_error("negative or odd size"); return SPLASH_INVALID_ARG; }
    if (n == 0 || row_bytes == 0) return SPLASH_OK;
    if (!recv || !out || !send_row || !aligned(recv, 2) || !aligned(out, 2) || !aligned(send_row, 4)) {
        set_error("a required pointer is NULL or misaligned"); return SPLASH_INVALID_ARG;
    }
    if (out_row_pitch < row_bytes) { set_error("out_row_pitch smaller than a row"); return SPLASH_INVALID_ARG; }
    DeviceInfo dev;
    if (!current_device_info(dev)) return SPLASH_CUDA_ERROR;
    cudaError_t e = launch_dop_unpack_rows(recv, out, send_row, n, row_bytes, out_row_pitch, dev.sm_count,
                                           static_cast<cudaStream_t>(stream_));
    if (e != cudaSuccess) { set_error("CUDA error: %s", cudaGetErrorString(e)); return SPLASH_CUDA_ERROR; }
    return SPLASH_OK;
}

int splash_get_kernel_timing(float *plan_ms, float *decode_ms, float *combine_ms) {
    if (!g_events_recorded) { set_error("no timed decode call on this thread"); return SPLASH_INVALID_ARG; }
    cudaError_t e = cudaEventSynchronize(g_events[3]);
    float ms[3] = {0.f, 0.f, 0.f};
    for (int k = 0; k < 3 && e == cudaSuccess; ++k) e = cudaEventElapsedTime(&ms[k], g_events[k], g_events[k + 1]);
    if (e != cudaSuccess) { set_error("CUDA error: %s", cudaGetErrorString(e)); return SPLASH_CUDA_ERROR; }
    if (plan_ms) *plan_ms = ms[0];
    if (decode_ms) *decode_ms = ms[1];
    if (combine_ms) *combine_ms = ms[2];
    return SPLASH_OK;
}

int splash_workspace_status(const void *workspace, int32_t *detail) {
    if (!workspace) { set_error("workspace is NULL"); return SPLASH_INVALID_ARG; }
    int32_t host[4] = {0, 0, 0, 0};
    cudaError_t e = cudaMemcpy(host, workspace, sizeof host, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) { set_error("CUDA error: %s", cudaGetErrorString(e)); return SPLASH_CUDA_ERROR; }
    if (detail) { detail[0] = host[1]; detail[1] = host[2]; detail[2] = host[3]; }
    return host[0];
}

}  // extern "C"
