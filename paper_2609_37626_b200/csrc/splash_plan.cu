// Split-KV work plan (device side, integer only, deterministic).
//
// The attention time of a decode step is set by the KV bytes read and the
// contraction work, both linear in the context length (the paper's per-step cost
// model, App. B: t_att = max{F_att / Phi_att, K_read / beta_KV}), so the plan
// spreads page tiles -- not requests -- evenly over the CTAs: the global sequence of
// (request, page tile) pairs is cut into `num_workers` contiguous runs of equal cost,
// where a non-empty request costs its tile count plus a fixed overhead.  A run that
// covers a whole request writes the final result; the (at most two) partial pieces
// at the ends of a run go to per-worker partial slots and are combined afterwards.
// The plan depends only on (seq_lens, kv ranges, shape), so a repeated call takes
// the same split and is bit-reproducible.
#include "splash_common.cuh"

namespace splash {

namespace {

constexpr int kPlanThreads = 1024;
constexpr int kPlanSmemRequests = 4096;
constexpr int kPlanSmemWorkers = 512;

__global__ void __launch_bounds__(kPlanThreads)
plan_kernel(int B, int W, int overhead, int len_cap, int reset_status, const int32_t *__restrict__ seq_lens, const int32_t *__restrict__ kv_begin,
            const int32_t *__restrict__ kv_end, int32_t *tile_start,
            int32_t *__restrict__ req_lo, int32_t *__restrict__ req_hi,
            int32_t *__restrict__ req_wfirst, int32_t *__restrict__ req_wlast,
            int32_t *cost_start, int32_t *worker_begin, int32_t *__restrict__ split_list, int32_t *__restrict__ worker_req,
            int4 *__restrict__ split_rec, int32_t *__restrict__ status) {
    __shared__ long long warp_tot_tiles[32], warp_tot_cost[32];
    __shared__ long long carry_tiles, carry_cost;
    __shared__ int n_split;
    // The bisections below chase a dozen dependent loads each; for the usual sizes the
    // prefix arrays live in shared memory while the plan is built and are copied out at the end.
    __shared__ int32_t s_tile[kPlanSmemRequests + 1], s_cost[kPlanSmemRequests + 1], s_wbeg[kPlanSmemWorkers + 1];
    const bool staged = B <= kPlanSmemRequests && W <= kPlanSmemWorkers;
    int32_t *const g_tile_start = tile_start, *const g_cost_start = cost_start, *const g_worker_begin = worker_begin;
    if (staged) { tile_start = s_tile; cost_start = s_cost; worker_begin = s_wbeg; }
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    grid_launch_dependents();     // the decode kernel may start its set-up now; it waits for this grid before reading the plan
    // the status block is cleared by the first pass of a call only: a later pass (more than 128 (head, row) pairs)
    // must not wipe what an earlier one recorded
    if (reset_status && tid < 16) status[tid] = 0;
    if (tid == 0) { carry_tiles = 0; carry_cost = 0; tile_start[0] = 0; cost_start[0] = 0; n_split = 0; }
    __syncthreads();

    // pass 1: effective ranges, tile counts, exclusive prefixes of tiles and of cost
    for (int base = 0; base < B; base += kPlanThreads) {
        int i = base + tid;
        long long n = 0;
        if (i < B) {
            int s = seq_lens[i];
            if (len_cap >= 0 && (s < 0 || s > len_cap)) s = 1;     // a list count out of bounds: one (poisoned) row
            int lo = kv_begin ? kv_begin[i] : 0;
            int hi = kv_end ? kv_end[i] : s;
            if (lo < 0) lo = 0;
            if (hi > s) hi = s;
            if (hi < lo) hi = lo;
            req_lo[i] = lo; req_hi[i] = hi;
            if (hi > lo) n = (hi + kPage - 1) / kPage - lo / kPage;
        }
        long long c = n > 0 ? n + overhead : 0;
        long long sn = n, sc = c;
        for (int o = 1; o < 32; o <<= 1) {
            long long a = __shfl_up_sync(0xffffffffu, sn, o);
            long long b = __shfl_up_sync(0xffffffffu, sc, o);
            if (lane >= o) { sn += a; sc += b; }
        }
        if (lane == 31) { warp_tot_tiles[wid] = sn; warp_tot_cost[wid] = sc; }
        __syncthreads();
        long long offn = carry_tiles, offc = carry_cost;
        for (int k = 0; k < wid; ++k) { offn += warp_tot_tiles[k]; offc += warp_tot_cost[k]; }
        if (i < B) { tile_start[i + 1] = (int32_t)(offn + sn); cost_start[i + 1] = (int32_t)(offc + sc); }
        __syncthreads();
        if (tid == kPlanThreads - 1) { carry_tiles = offn + sn; carry_cost = offc + sc; }
        __syncthreads();
    }
    const long long total_cost = carry_cost;
    const int total_tiles = (int)carry_tiles;

    // pass 2: worker w starts at cost floor(w * total_cost / W); the request whose
    // cost interval [cost_start[i], cost_start[i+1]) holds that value is found by
    // bisection, and a start that falls into the request's fixed overhead snaps to
    // its first tile.
    for (int w = tid; w <= W; w += kPlanThreads) {
        int g = total_tiles, first_req = 0;
        if (w < W && total_cost > 0) {
            long long target = (total_cost * w) / W;
            int lo = 0, hi = B;   // invariant cost_start[lo] <= target < cost_start[hi]
            while (hi - lo > 1) { int mid = (lo + hi) >> 1; if (cost_start[mid] <= target) lo = mid; else hi = mid; }
            while (cost_start[lo + 1] <= target) ++lo;   // (defensive; bisection already lands on a non-empty request)
            long long off = target - cost_start[lo] - overhead;
            if (off < 0) off = 0;
            g = tile_start[lo] + (int)off;
            first_req = lo;
        }
        worker_begin[w] = g;
        worker_req[w] = first_req;
    }
    __threadfence_block();
    __syncthreads();

    // pass 3: first / last worker of every request
    for (int i = tid; i < B; i += kPlanThreads) {
        int rs = tile_start[i], re = tile_start[i + 1];
        int wf = -1, wl = -1;
        if (re > rs) {
            // worker containing tile x: the w with worker_begin[w] <= x < worker_begin[w+1]
            int lo = 0, hi = W;   // invariant worker_begin[lo] <= rs < worker_begin[hi]
            while (hi - lo > 1) { int mid = (lo + hi) >> 1; if (worker_begin[mid] <= rs) lo = mid; else hi = mid; }
            wf = lo;
            int x = re - 1;
            lo = 0; hi = W;
            while (hi - lo > 1) { int mid = (lo + hi) >> 1; if (worker_begin[mid] <= x) lo = mid; else hi = mid; }
            wl = lo;
        }
        req_wfirst[i] = wf; req_wlast[i] = wl;
        // requests cut into several pieces are listed for the combine kernel (at most W - 1 of them;
        // the list order varies from run to run, the results do not depend on it)
        if (wf != wl) {
            const int e = atomicAdd(&n_split, 1);
            split_list[e] = i;
            split_rec[e] = make_int4(i, wf, wl, rs);      // all the combine kernel needs to know about the request, in one load
        }
    }
    __syncthreads();
    if (tid == 0) status[8] = n_split;
    if (staged) {
        for (int i = tid; i <= B; i += kPlanThreads) { g_tile_start[i] = s_tile[i]; g_cost_start[i] = s_cost[i]; }
        for (int w = tid; w <= W; w += kPlanThreads) g_worker_begin[w] = s_wbeg[w];
    }
}

// Validation mode: every block-table entry of a page that intersects a request's effective range must name a page of
// the pool.  One block per request (grid-stride), threads over its pages; the first offender found wins the status word.
__global__ void __launch_bounds__(256)
validate_pages_kernel(int B, int num_pool_pages, int table_stride, const int32_t *__restrict__ block_table,
                      const int32_t *__restrict__ req_lo, const int32_t *__restrict__ req_hi, int32_t *status) {
    for (int i = blockIdx.x; i < B; i += gridDim.x) {
        const int lo = req_lo[i], hi = req_hi[i];
        if (hi <= lo) continue;
        for (int pg = lo / kPage + threadIdx.x; pg < (hi + kPage - 1) / kPage; pg += blockDim.x) {
            const int id = block_table[(int64_t)i * table_stride + pg];
            if (id < 0 || id >= num_pool_pages) {
                if (atomicCAS(status, 0, (int)SPLASH_BAD_PAGE_ID) == 0) { status[1] = i; status[2] = pg; status[3] = id; }
            }
        }
    }
}

}  // namespace

cudaError_t launch_validate_pages(const DecodeParams &p, const int32_t *req_lo, const int32_t *req_hi, cudaStream_t stream) {
    const int grid = p.B < 1024 ? p.B : 1024;
    validate_pages_kernel<<<grid, 256, 0, stream>>>(p.B, p.num_pool_pages, p.table_stride, p.block_table, req_lo, req_hi, p.status);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_plan(const DecodeParams &p, const int32_t *kv_begin, const int32_t *kv_end,
                        int32_t *tile_start, int32_t *req_lo, int32_t *req_hi, int32_t *req_wfirst,
                        int32_t *req_wlast, int32_t *cost_start, int32_t *worker_begin, int32_t *split_list,
                        int32_t *worker_req, int4 *split_rec, int32_t *status, bool reset_status, cudaStream_t stream) {
    // same shared-memory carve-out as the decode kernel that follows: no reconfiguration between them
    static DeviceOnce once;
    once.run([&] {
        cudaFuncSetAttribute(plan_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        return cudaSuccess;     // a preference: a failure is not an error
    });
    plan_kernel<<<1, kPlanThreads, 0, stream>>>(p.B, p.num_workers, p.request_overhead_tiles, p.len_cap, reset_status ? 1 : 0, p.seq_lens, kv_begin, kv_end, tile_start,
                                                req_lo, req_hi, req_wfirst, req_wlast, cost_start, worker_begin, split_list, worker_req, split_rec, status);
    count_launch();
    return cudaGetLastError();
}

}  // namespace splash
