// Sparse decode, first stage: the rows an indexer selected for each request are gathered out
// of the paged cache of 656-byte rows (512 e4m3 latent codes, four float scales -- one per 128
// latent dims --, 64 bf16 rope values; Sec. 5 setup, App. B payload) into a dense, request-major
// bf16 cache in the workspace, dequantised on the way (code x block scale, rounded to bf16).  The
// dense decode kernels then run over that cache with the list lengths as context lengths.
//
// One warp per listed row: 41 16-byte loads in, 72 16-byte stores out, both coalesced.  HBM-bound:
// 656 B read + 1152 B written per listed token (and 1152 B read again by the decode kernel).  With
// rows picked uniformly at random the kernel sits at about half of the DRAM rate (4.2 TB/s of reads
// plus writes); a variant that moved the rows as 656-byte bulk copies through shared memory, with
// 2.5 times the bytes in flight per SM, ran at the same rate, so the limit is on the DRAM side
// (isolated 656-byte reads between write bursts), not the SMs' latency hiding.
#include <cuda_bf16.h>

#include "splash_common.cuh"
#include "splash_fp8.cuh"

namespace splash {

namespace {

constexpr int kSparseRowBytes = 656;
constexpr int kGatherThreads = 256;
constexpr int kRowsInFlight = 4;              // rows a warp loads before it converts any (a multiple of 4)
constexpr uint32_t kBf16NanPair = 0x7FC07FC0u;

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

// 4 codes (one 32-bit word) times a scale -> 4 bf16 (two words)
__device__ __forceinline__ uint2 dequant4(uint32_t w, float s) {
    const float2 a = umma::from_e4m3x2((uint16_t)(w & 0xffffu)), b = umma::from_e4m3x2((uint16_t)(w >> 16));
    return make_uint2(pack_bf16x2(a.x * s, a.y * s), pack_bf16x2(b.x * s, b.y * s));
}

// Grid-stride over the B * pages_per_request * 64 row slots of the dense cache, in groups of 32 slots per warp.
__global__ void __launch_bounds__(kGatherThreads, 4)
sparse_gather_kernel(int B, int max_sel, int pages_per_request, const uint8_t *__restrict__ kv_pool, int num_pool_pages,
                     const int32_t *__restrict__ block_table, int64_t table_stride, const int32_t *__restrict__ seq_lens,
                     const int32_t *__restrict__ sel, int64_t sel_stride, const int32_t *__restrict__ sel_count,
                     uint8_t *__restrict__ dense_pool, int32_t *__restrict__ dense_table) {
    // Launched as a programmatic dependent of the plan kernel, whose output it does not read: it runs beside it,
    // lets the decode kernel behind it set up early, and waits for the plan only before it exits, so that the
    // decode kernel, which waits for this grid, finds both the plan and the dense cache complete.
    grid_launch_dependents();
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * kGatherThreads + threadIdx.x) >> 5;
    const int64_t num_warps = ((int64_t)gridDim.x * kGatherThreads) >> 5;
    const int slots_per_request = pages_per_request * kPage;
    const int64_t total = (int64_t)B * slots_per_request;

    // the dense cache's page table (its context lengths are the list counts, read by the plan).  A count
    // outside [0, max_sel] is an argument error: the request then gets one poisoned row, so that its result
    // is NaN rather than plausible; the plan kernel applies the same rule.
    for (int64_t e = (int64_t)blockIdx.x * kGatherThreads + threadIdx.x; e < (int64_t)B * pages_per_request;
         e += (int64_t)gridDim.x * kGatherThreads)
        dense_table[e] = (int32_t)e;

    // A warp takes groups of 32 consecutive row slots; lane l resolves the address of slot l of the group.  That
    // address hangs on a chain of three loads (count, list entry, page id): the chain of the NEXT group advances one
    // link per batch of rows of the current group, so its latency hides behind the row loads.
    constexpr int kGroup = 32, kBatches = kGroup / kRowsInFlight;
    static_assert(kBatches >= 4, "one link of the next group's address chain per batch");
    const int64_t num_groups = (total + kGroup - 1) / kGroup;
    int n_req = 0, n_idx = 0, n_cnt = 0, n_len = 0, n_tok = 0, n_page = 0, n_state = 0;
    auto link = [&](int step, int64_t group) {
        if (group >= num_groups) { n_state = 0; return; }
        if (step == 0) {
            const int64_t slot = group * kGroup + lane;
            n_state = slot < total ? 1 : 0;
            n_req = n_state ? (int)(slot / slots_per_request) : 0;
            n_idx = n_state ? (int)(slot % slots_per_request) : 0;
            n_cnt = __ldg(sel_count + n_req);
            n_len = __ldg(seq_lens + n_req);
        } else if (step == 1) {
            const bool bad_count = n_cnt < 0 || n_cnt > max_sel;
            const int n = bad_count ? 1 : n_cnt;
            if (n_state && n_idx >= (n + kPage - 1) / kPage * kPage) n_state = 0;       // pages the decode never touches
            else if (n_state && n_idx >= n) n_state = 2;
            else if (n_state && bad_count) n_state = 3;
            n_tok = n_state == 1 ? __ldg(sel + (int64_t)n_req * sel_stride + n_idx) : 0;
        } else if (step == 2) {
            if (n_state == 1 && (n_tok < 0 || n_tok >= n_len)) n_state = 3;
            n_page = n_state == 1 ? __ldg(block_table + (int64_t)n_req * table_stride + n_tok / kPage) : 0;
        } else {
            if (n_state == 1 && (n_page < 0 || n_page >= num_pool_pages)) n_state = 3;
        }
    };
#pragma unroll
    for (int step = 0; step < 4; ++step) link(step, warp);
    for (int64_t group = warp; group < num_groups; group += num_warps) {
        const int my_state = n_state;
        const uint8_t *my_row = kv_pool + ((int64_t)n_page * kPage + n_tok % kPage) * kSparseRowBytes;
        uint8_t *const dst_group = dense_pool + group * kGroup * (int64_t)(kDQK * 2);
        const int k = lane >> 3;
#pragma unroll
        for (int b = 0; b < kBatches; ++b) {
            if (b < 4) link(b, group + num_warps);
            int state[kRowsInFlight];
            uint4 lat[kRowsInFlight], rope[kRowsInFlight / 4];
            float scale[kRowsInFlight];
#pragma unroll
            for (int u = 0; u < kRowsInFlight; ++u) {
                const int src_lane = b * kRowsInFlight + u;
                state[u] = __shfl_sync(0xffffffffu, my_state, src_lane);
                const uint8_t *row = reinterpret_cast<const uint8_t *>(__shfl_sync(0xffffffffu, reinterpret_cast<unsigned long long>(my_row), src_lane));
                if (state[u] == 1) {
                    lat[u] = __ldg(reinterpret_cast<const uint4 *>(row) + lane);
                    scale[u] = __ldg(reinterpret_cast<const float *>(row + kDLatent) + (lane >> 3));
                }
            }
            // the 128 rope bytes of a row are eight 16-byte units: lanes 8 k .. 8 k + 7 take row 4 m + k of the batch
            int rope_state[kRowsInFlight / 4];
#pragma unroll
            for (int m = 0; m < kRowsInFlight / 4; ++m) {
                const int src_lane = b * kRowsInFlight + 4 * m + k;
                rope_state[m] = __shfl_sync(0xffffffffu, my_state, src_lane);
                const uint8_t *row = reinterpret_cast<const uint8_t *>(__shfl_sync(0xffffffffu, reinterpret_cast<unsigned long long>(my_row), src_lane));
                if (rope_state[m] == 1) rope[m] = __ldg(reinterpret_cast<const uint4 *>(row + kDLatent + 16) + (lane & 7));
            }
#pragma unroll
            for (int u = 0; u < kRowsInFlight; ++u) {
                if (state[u] == 0) continue;
                uint4 *dst = reinterpret_cast<uint4 *>(dst_group + (b * kRowsInFlight + u) * (kDQK * 2));
                uint4 lo, hi;
                if (state[u] == 1) {
                    const float s = scale[u];
                    const uint2 a = dequant4(lat[u].x, s), bb = dequant4(lat[u].y, s), c = dequant4(lat[u].z, s), d = dequant4(lat[u].w, s);
                    lo = make_uint4(a.x, a.y, bb.x, bb.y); hi = make_uint4(c.x, c.y, d.x, d.y);
                } else {
                    const uint32_t fill = state[u] == 2 ? 0u : kBf16NanPair;
                    lo = hi = make_uint4(fill, fill, fill, fill);
                }
                dst[2 * lane] = lo;
                dst[2 * lane + 1] = hi;
            }
#pragma unroll
            for (int m = 0; m < kRowsInFlight / 4; ++m) {
                if (rope_state[m] == 0) continue;
                const uint32_t fill = rope_state[m] == 2 ? 0u : kBf16NanPair;
                reinterpret_cast<uint4 *>(dst_group + (b * kRowsInFlight + 4 * m + k) * (kDQK * 2))[64 + (lane & 7)] =
                    rope_state[m] == 1 ? rope[m] : make_uint4(fill, fill, fill, fill);
            }
        }
    }
    grid_dependency_wait();
}

}  // namespace

cudaError_t launch_sparse_gather(int B, int max_sel, int pages_per_request, const void *kv_pool, int num_pool_pages,
                                 const int32_t *block_table, int64_t table_stride, const int32_t *seq_lens,
                                 const int32_t *sel, int64_t sel_stride, const int32_t *sel_count, void *dense_pool,
                                 int32_t *dense_table, int sm_count, cudaStream_t stream) {
    const int64_t groups = ((int64_t)B * pages_per_request * kPage + 31) / 32;
    const int warps_per_block = kGatherThreads / 32;
    int64_t blocks = (groups + warps_per_block - 1) / warps_per_block;
    const int64_t cap = (int64_t)sm_count * 4;          // resident blocks; the loop strides over the rest
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    cudaError_t e = launch_dependent(sparse_gather_kernel, dim3((unsigned)blocks), dim3(kGatherThreads), 0, stream, B, max_sel,
                                     pages_per_request, static_cast<const uint8_t *>(kv_pool), num_pool_pages, block_table,
                                     table_stride, seq_lens, sel, sel_stride, sel_count, static_cast<uint8_t *>(dense_pool),
                                     dense_table);
    count_launch();
    return e;
}

}  // namespace splash
