// Shared declarations of the MLA decode library: dimensions, the split-KV work
// plan that the plan kernel writes into the caller's workspace, and host helpers.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>

#include <mutex>

#include "../../include/splash_mla.h"

namespace splash {

constexpr int kDQK = 576;        // d_c + d_r (absorbed MLA row width)
constexpr int kMaxQRows = 8;      // query rows per request (multi-token decode steps, short prefill chunks)
constexpr int kDV = 512;         // d_c (value width)
constexpr int kDRope = 64;
constexpr int kDLatent = 512;
constexpr int kPage = 64;        // tokens per page
constexpr int kMaxHeads = 128;
// largest page id (exclusive) the allocation-free migrate entry point can remap: 1 MiB of table
constexpr int kStaticMigrateMaxPageId = 1 << 18;

// Cost, in page tiles, charged once per non-empty request when the plan balances work
// over CTAs (query operands, pipeline refill, epilogue): measured per kernel, passed to the
// plan kernel at launch.
constexpr int kRequestOverheadTilesDefault = 4;
constexpr int kRequestOverheadTilesFp8 = 6;        // also right for the 16- / 32-head e4m3 kernel: a TP-8 share of the rollout
                                                   // workload takes 237 / 232 / 228 / 224 / 227 / 232 / 239 us with 2 / 3 / 4 / 6 / 8 / 10 / 14
constexpr int kRequestOverheadTilesPair = 5;       // bf16 CTA-pair kernel (a segment costs 7,500 cycles, a tile 1,650)
constexpr int kRequestOverheadTilesFp8Pair = 13;   // CTA-pair kernel: tiles are cheaper, the per-request work is not

// ---- workspace layout ------------------------------------------------------
// [0, 64)                 status block (int32 x 16): [0] status, [1..3] detail
// then int32 arrays       tile_start[B+1], req_lo[B], req_hi[B], req_wfirst[B],
//                         req_wlast[B], cost_start[B+1], worker_begin[W+1], split_list[W+1]
//                         (status[8] = number of entries of split_list)
// then (256-B aligned)    partial_lse [2W][h] fp32
// then (256-B aligned)    partial_scale [2W][h] fp32 (f16 partial outputs only: the power of two a row was divided by)
// then (256-B aligned)    partial_out [2W][h][512] fp32
struct PlanView {
    int32_t *status;        // 16 ints
    int32_t *tile_start;    // [B+1] exclusive prefix of per-request tile counts
    int32_t *req_lo;        // [B] first token of the effective range
    int32_t *req_hi;        // [B] one past the last token (>= lo; == lo when empty)
    int32_t *req_wfirst;    // [B] first worker holding a piece of the request (-1 if empty)
    int32_t *req_wlast;     // [B] last such worker
    int32_t *cost_start;    // [B+1] exclusive prefix of per-request cost (tiles + overhead)
    int32_t *worker_begin;  // [W+1] global tile index where each worker starts
    int32_t *split_list;    // [W+1] requests computed in more than one piece (count in status[8])
    int32_t *worker_req;    // [W+1] the request that holds a worker's first tile (what the kernels would bisect for)
    int4 *split_rec;        // [W+1] per entry of split_list: (request, first worker, last worker, first tile of the request)
    float *partial_lse;     // [2W][h]
    float *partial_scale;   // [2W][h]
    float *partial_out;     // [2W][h][512]
    int32_t num_workers;    // W
    int32_t h;              // width of the head slice
    size_t bytes;           // total bytes needed
};

inline __host__ __device__ size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

inline __host__ PlanView make_plan_view(void *workspace, int B, int W, int h) {
    PlanView v;
    char *p = static_cast<char *>(workspace);
    size_t off = 0;
    v.status = reinterpret_cast<int32_t *>(p + off); off += 64;
    v.tile_start = reinterpret_cast<int32_t *>(p + off); off += sizeof(int32_t) * (size_t)(B + 1);
    v.req_lo = reinterpret_cast<int32_t *>(p + off); off += sizeof(int32_t) * (size_t)B;
    v.req_hi = reinterpret_cast<int32_t *>(p + off); off += sizeof(int32_t) * (size_t)B;
    v.req_wfirst = reinterpret_cast<int32_t *>(p + off); off += sizeof(int32_t) * (size_t)B;
    v.req_wlast = reinterpret_cast<int32_t *>(p + off); off += sizeof(int32_t) * (size_t)B;
    v.cost_start = reinterpret_cast<int32_t *>(p + off); off += sizeof(int32_t) * (size_t)(B + 1);
    v.worker_begin = reinterpret_cast<int32_t *>(p + off); off += sizeof(int32_t) * (size_t)(W + 1);
    v.split_list = reinterpret_cast<int32_t *>(p + off); off += sizeof(int32_t) * (size_t)(W + 1);
    v.worker_req = reinterpret_cast<int32_t *>(p + off); off += sizeof(int32_t) * (size_t)(W + 1);
    off = align_up(off, 16);
    v.split_rec = reinterpret_cast<int4 *>(p + off); off += sizeof(int4) * (size_t)(W + 1);
    off = align_up(off, 256);
    v.partial_lse = reinterpret_cast<float *>(p + off); off += sizeof(float) * (size_t)2 * W * h;
    off = align_up(off, 256);
    v.partial_scale = reinterpret_cast<float *>(p + off); off += sizeof(float) * (size_t)2 * W * h;
    off = align_up(off, 256);
    v.partial_out = reinterpret_cast<float *>(p + off); off += sizeof(float) * (size_t)2 * W * h * kDV;
    v.num_workers = W;
    v.h = h;
    v.bytes = off;
    return v;
}

// Arguments common to the decode kernels.
struct DecodeParams {
    const void *q;
    const void *kv_pool;
    const float *kv_scales;
    const int32_t *block_table;
    const int32_t *seq_lens;
    float *out;
    float *lse;
    int64_t q_stride_request, q_stride_head;
    int64_t out_stride_request, out_stride_head;
    int64_t lse_stride_request;
    int32_t B, H;
    int32_t head_begin, head_end;
    int32_t table_stride;
    int32_t num_pool_pages;
    int32_t q_rows;            // R query rows per request; the heads of a call are then virtual heads g * R + r, and
                               // row r attends causally: tokens below seq_len - (R - 1 - r)
    int32_t heads_per_group;   // heads one CTA computes
    int32_t num_groups;        // head groups per KV worker
    int32_t pair_groups;       // CTA-pair kernels: CTA pairs per KV worker (1; more when several query rows per request
                               // make more than 128 (head, row) pairs: pair g of a worker takes pairs [128 g, 128 g + 128)
                               // and the pairs of a worker stream the same pages side by side, so the second read of a
                               // page hits L2 and the cache crosses HBM once)
    float softmax_scale;
    // plan (device pointers into the workspace)
    const int32_t *tile_start, *req_lo, *req_hi, *worker_begin;
    const int32_t *worker_req;   // request holding each worker's first tile, from the plan
    int32_t *status;
    float *partial_lse, *partial_out;
    float *partial_scale;      // f16 partial outputs: row (slot, head) holds O * 2^k with 2^-k stored here
    int32_t partial_f16;       // 1: the partial outputs are f16 (same slot order, rows of 512 halves): half the bytes for the
                               // decode kernel to write and the combine kernel to read; 11 significant bits of a normalised O,
                               // each row scaled by a power of two so that its largest entry sits just below f16's maximum
                               // (exact, and no limit on the magnitude of the cache values)
    int32_t len_cap;           // >= 0: seq_lens holds list counts; one outside [0, len_cap] counts as 1 (sparse decode)
    // fused sparse decode: kv_pool holds 656-byte rows, block_table / num_pool_pages describe it, and request i
    // attends over the tokens sel[i * sel_stride + j], j < seq_lens[i], each below ctx_lens[i]
    const int32_t *sel, *ctx_lens;
    int64_t sel_stride;
    int32_t num_workers;
    // optional page-copy job carried along by the CTA-pair kernels in warps that have nothing else to do (the issuer
    // warps of each pair's second CTA): page mig_src_ids[j] of mig_src -> page mig_dst_ids[j] of mig_dst, j < mig_n,
    // mig_page_vecs 16-byte vectors per page, with the pages' scale pages when the scale pointers are set
    const uint4 *mig_src, *mig_src_scales;
    uint4 *mig_dst, *mig_dst_scales;
    const int32_t *mig_src_ids, *mig_dst_ids;
    int64_t mig_page_vecs;
    int32_t mig_n;
    int32_t request_overhead_tiles;   // per-request cost the plan adds to the tile count
    long long *trace;          // optional device buffer for pipeline timestamps (diagnostics), or NULL
};

// A worker's next piece of work: request, its relative tile range, where the
// result goes.
struct Segment {
    int32_t request;
    int32_t tile_begin, tile_end;   // page-tile indices relative to floor(lo/64)
    int32_t lo, hi;                 // effective token range of the request
    int32_t slot;                   // partial slot, or -1 when the piece is the whole request
};

// Iterates the segments of worker w in plan order.  Every thread of a CTA calls
// it with the same arguments and gets the same answer.
struct SegmentIter {
    const int32_t *ts;
    int32_t B, x, end, wb, i, w;
    __device__ void init(const DecodeParams &p, int worker) {
        ts = p.tile_start; B = p.B; w = worker;
        wb = p.worker_begin[worker]; x = wb; end = p.worker_begin[worker + 1];
        // the request containing tile x (last i with ts[i] <= x and ts[i+1] > x): the plan has it, which saves every
        // role of every CTA a bisection of a dozen dependent global loads before its first tile
        i = x < end ? p.worker_req[worker] : 0;
    }
    __device__ bool next(const DecodeParams &p, Segment &s) {
        if (x >= end) return false;
        while (ts[i + 1] <= x) ++i;                    // skip finished / empty requests
        int rs = ts[i], re = ts[i + 1];
        int seg_end = re < end ? re : end;
        s.request = i;
        s.tile_begin = x - rs;
        s.tile_end = seg_end - rs;
        s.lo = p.req_lo[i];
        s.hi = p.req_hi[i];
        bool full = (x == rs) && (seg_end == re);
        s.slot = full ? -1 : 2 * w + (rs <= wb ? 0 : 1);
        x = seg_end;
        return true;
    }
};

// Requests whose effective KV range is empty belong to no segment: O = 0, LSE = -inf is
// written by the decode CTA (worker, head group) with worker == request mod num_workers,
// for its own heads.  Called by all threads of the CTA once its segments are done.
__device__ __forceinline__ void fill_empty_requests(const DecodeParams &p, int worker, int head0, int heads_per_group,
                                                    int tid, int nthreads) {
    // The plan's arrays are a launch old and have left the caches: a loop over this worker's requests that looks at one
    // request per iteration is a chain of round trips to DRAM at the very end of the CTA (seven on the rollout workload).
    // Instead every lane looks at a request of its own -- one round trip -- and the warp then zeroes what it found.
    const int nheads = min(heads_per_group, p.head_end - head0);
    const int lane = tid & 31, wid = tid >> 5, nwarps = nthreads >> 5;
    for (int64_t j0 = (int64_t)wid * 32; worker + j0 * p.num_workers < p.B; j0 += (int64_t)nwarps * 32) {
        const int64_t mine = worker + (j0 + lane) * p.num_workers;
        const bool empty = mine < p.B && p.tile_start[mine + 1] == p.tile_start[mine];
        unsigned found = __ballot_sync(0xffffffffu, empty);
        while (found) {
            const int src = __ffs(found) - 1;
            found &= found - 1;
            const int64_t i = worker + (j0 + src) * p.num_workers;
            for (int idx = lane; idx < nheads * (kDV / 4); idx += 32) {
                const int hh = idx / (kDV / 4), c = idx % (kDV / 4);
                reinterpret_cast<float4 *>(p.out + i * p.out_stride_request + (int64_t)(head0 + hh) * p.out_stride_head)[c] =
                    make_float4(0.f, 0.f, 0.f, 0.f);
            }
            for (int hh = lane; hh < nheads; hh += 32) p.lse[i * p.lse_stride_request + head0 + hh] = -INFINITY;
        }
    }
}

// ---- programmatic dependent launch ---------------------------------------------
// The three kernels of a decode call are chained with programmatic stream serialisation:
// a dependent kernel may be scheduled while its predecessor is still running, does its
// own set-up (barriers, tensor memory), and blocks in grid_dependency_wait() before it
// touches anything the predecessor wrote.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                    Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Per-device one-time set-up of a launcher (function attributes are per device).  The set-up runs under a lock and a
// device counts as done only once it has succeeded, so a second host thread whose first call on a device comes at the
// same time waits for the attribute to be in place instead of launching without it.
struct DeviceOnce {
    std::mutex mu;
    bool done[64] = {};
    template <typename F>
    cudaError_t run(F &&setup) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return setup();
        std::lock_guard<std::mutex> lock(mu);
        if (done[dev]) return cudaSuccess;
        const cudaError_t e = setup();
        if (e == cudaSuccess) done[dev] = true;
        return e;
    }
};

// ---- host helpers (splash_api.cu) -----------------------------------------
void set_error(const char *fmt, ...);
void count_launch(int n = 1);

// kernels' host launchers
cudaError_t launch_plan(const DecodeParams &p, const int32_t *kv_begin, const int32_t *kv_end,
                        int32_t *tile_start, int32_t *req_lo, int32_t *req_hi, int32_t *req_wfirst,
                        int32_t *req_wlast, int32_t *cost_start, int32_t *worker_begin, int32_t *split_list, int32_t *worker_req, int4 *split_rec,
                        int32_t *status, bool reset_status, cudaStream_t stream);
cudaError_t launch_validate_pages(const DecodeParams &p, const int32_t *req_lo, const int32_t *req_hi, cudaStream_t stream);
cudaError_t launch_decode_sparse_pair(const DecodeParams &p, cudaStream_t stream);
cudaError_t launch_sparse_gather(int B, int max_sel, int pages_per_request, const void *kv_pool, int num_pool_pages,
                                 const int32_t *block_table, int64_t table_stride, const int32_t *seq_lens,
                                 const int32_t *sel, int64_t sel_stride, const int32_t *sel_count, void *dense_pool,
                                 int32_t *dense_table, int sm_count, cudaStream_t stream);
cudaError_t launch_dop_pack_rows(const void *a, const void *b, void *out, const int32_t *send_row, int64_t n, int h,
                                 int64_t a_bytes, int64_t b_bytes, int64_t a_row_pitch, int64_t a_head_pitch,
                                 int64_t b_row_pitch, int64_t b_head_pitch, int sm_count, cudaStream_t stream);
cudaError_t launch_dop_unpack_rows(const void *recv, void *out, const int32_t *send_row, int64_t n, int64_t row_bytes,
                                   int64_t out_row_pitch, int sm_count, cudaStream_t stream);
cudaError_t launch_dop_swap_outer(const void *in, void *out, int64_t A, int64_t Bn, int64_t inner_bytes, int sm_count,
                                  cudaStream_t stream);
cudaError_t launch_decode_simt(const DecodeParams &p, int kv_dtype, cudaStream_t stream);
int simt_heads_per_group();
// tcgen05 kernel: how it cuts a head slice of width h into CTAs, and its launcher
void umma_tiling(int kv_dtype, int h, int sm_count, int *heads_per_group, int *num_groups, int *num_workers);
cudaError_t launch_decode_umma(const DecodeParams &p, const splash_mla_shape &shape, cudaStream_t stream);
cudaError_t launch_decode_umma_fp8(const DecodeParams &p, cudaStream_t stream);
cudaError_t launch_decode_umma_fp8_narrow(const DecodeParams &p, cudaStream_t stream);   // 16 / 32 heads per CTA
cudaError_t launch_decode_umma_fp8_pair(const DecodeParams &p, cudaStream_t stream);
cudaError_t launch_decode_umma_pair(const DecodeParams &p, cudaStream_t stream);
cudaError_t launch_split_combine(const DecodeParams &p, const int4 *split_rec, cudaStream_t stream);
cudaError_t launch_lse_merge(int num_parts, int64_t rows, int d_v, const float *part_out,
                             const float *part_lse, float *out, float *lse, cudaStream_t stream);
cudaError_t launch_page_migrate(const void *src_pool, const float *src_scales, void *dst_pool,
                                float *dst_scales, int64_t page_bytes, const int32_t *src_ids,
                                const int32_t *dst_ids, int64_t n, int32_t src_base, int32_t dst_base,
                                int32_t max_page_id, int32_t *block_table, int64_t num_entries,
                                int32_t *remap, bool do_table, bool do_copy, cudaStream_t stream);

cudaError_t static_remap_address(int32_t **ptr);

}  // namespace splash
