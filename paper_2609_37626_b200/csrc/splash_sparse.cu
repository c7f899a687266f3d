// Sparse decode, first stage: the rows an indexer selected for each request are gathered out
// of the paged cache of 656-byte rows (512 e4m3 latent codes, four float scales -- one per 128
// latent dims --, 64 bf16 rope values; Sec. 5 setup, App. B payload) into a dense, request-major
// bf16 cache in the workspace, dequantised on the way (code x block scale, rounded to bf16).  The
// dense decode kernels then run over that cache with the list lengths as context lengths.
//
// One warp per listed row: 41 16-byte loads in, 72 16-byte stores out, both coalesced.  HBM-bound:
// 656 B read + 1152 B written per listed token (and 1152 B read again by the decode kernel).
#include <cuda_bf16.h>

#include "splash_common.cuh"
#include "splash_fp8.cuh"

namespace splash {

namespace {

constexpr int kSparseRowBytes = 656;
constexpr int kGatherThreads = 256;
constexpr int kRowsInFlight = 4;              // rows a warp loads before it converts any
constexpr uint32_t kBf16NanPair = 0x7FC07FC0u;

struct RowRegs {
    uint4 lat;        // 16 latent codes: dims [16 lane, 16 lane + 16)
    uint4 rope;       // lanes 0..7: 8 rope values
    float scale;
    int state;        // 0: nothing to do, 1: a row, 2: zero fill (tail of the last page), 3: poison (bad list entry)
};

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

// 4 codes (one 32-bit word) times a scale -> 4 bf16 (two words)
__device__ __forceinline__ uint2 dequant4(uint32_t w, float s) {
    const float2 a = umma::from_e4m3x2((uint16_t)(w & 0xffffu)), b = umma::from_e4m3x2((uint16_t)(w >> 16));
    return make_uint2(pack_bf16x2(a.x * s, a.y * s), pack_bf16x2(b.x * s, b.y * s));
}

// Grid-stride over the B * pages_per_request * 64 row slots of the dense cache.
__global__ void __launch_bounds__(kGatherThreads)
sparse_gather_kernel(int B, int max_sel, int pages_per_request, const uint8_t *__restrict__ kv_pool, int num_pool_pages,
                     const int32_t *__restrict__ block_table, int64_t table_stride, const int32_t *__restrict__ seq_lens,
                     const int32_t *__restrict__ sel, int64_t sel_stride, const int32_t *__restrict__ sel_count,
                     uint8_t *__restrict__ dense_pool, int32_t *__restrict__ dense_table, int32_t *__restrict__ dense_lens) {
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * kGatherThreads + threadIdx.x) >> 5;
    const int64_t num_warps = ((int64_t)gridDim.x * kGatherThreads) >> 5;
    const int slots_per_request = pages_per_request * kPage;
    const int64_t total = (int64_t)B * slots_per_request;

    // the dense cache's page table and context lengths.  A count outside [0, max_sel] is an argument
    // error: the request then gets one poisoned row, so that its result is NaN rather than plausible.
    for (int64_t e = (int64_t)blockIdx.x * kGatherThreads + threadIdx.x; e < (int64_t)B * pages_per_request;
         e += (int64_t)gridDim.x * kGatherThreads)
        dense_table[e] = (int32_t)e;
    for (int64_t i = (int64_t)blockIdx.x * kGatherThreads + threadIdx.x; i < B; i += (int64_t)gridDim.x * kGatherThreads) {
        const int c = sel_count[i];
        dense_lens[i] = (c < 0 || c > max_sel) ? 1 : c;
    }

    for (int64_t base = warp; base < total; base += num_warps * kRowsInFlight) {
        RowRegs r[kRowsInFlight];
#pragma unroll
        for (int u = 0; u < kRowsInFlight; ++u) {
            const int64_t slot = base + (int64_t)u * num_warps;
            r[u].state = 0;
            if (slot >= total) continue;
            const int i = (int)(slot / slots_per_request), j = (int)(slot % slots_per_request);
            const int c = sel_count[i];
            const bool bad_count = c < 0 || c > max_sel;
            const int n = bad_count ? 1 : c;
            if (j >= (n + kPage - 1) / kPage * kPage) continue;          // pages the decode never touches
            if (j >= n) { r[u].state = 2; continue; }
            const int t = bad_count ? -1 : sel[(int64_t)i * sel_stride + j];
            if (t < 0 || t >= seq_lens[i]) { r[u].state = 3; continue; }
            const int page = block_table[(int64_t)i * table_stride + t / kPage];
            if (page < 0 || page >= num_pool_pages) { r[u].state = 3; continue; }
            const uint8_t *row = kv_pool + ((int64_t)page * kPage + t % kPage) * kSparseRowBytes;
            r[u].state = 1;
            r[u].lat = __ldg(reinterpret_cast<const uint4 *>(row) + lane);
            r[u].scale = __ldg(reinterpret_cast<const float *>(row + kDLatent) + (lane >> 3));
            if (lane < 8) r[u].rope = __ldg(reinterpret_cast<const uint4 *>(row + kDLatent + 16) + lane);
        }
#pragma unroll
        for (int u = 0; u < kRowsInFlight; ++u) {
            if (r[u].state == 0) continue;
            const int64_t slot = base + (int64_t)u * num_warps;
            uint4 *dst = reinterpret_cast<uint4 *>(dense_pool + slot * (int64_t)(kDQK * 2));
            uint4 lo, hi, rope = r[u].rope;
            if (r[u].state == 1) {
                const float s = r[u].scale;
                const uint2 a = dequant4(r[u].lat.x, s), b = dequant4(r[u].lat.y, s), c = dequant4(r[u].lat.z, s),
                            d = dequant4(r[u].lat.w, s);
                lo = make_uint4(a.x, a.y, b.x, b.y); hi = make_uint4(c.x, c.y, d.x, d.y);
            } else {
                const uint32_t fill = r[u].state == 2 ? 0u : kBf16NanPair;
                lo = hi = rope = make_uint4(fill, fill, fill, fill);
            }
            dst[2 * lane] = lo;
            dst[2 * lane + 1] = hi;
            if (lane < 8) dst[64 + lane] = rope;
        }
    }
}

}  // namespace

cudaError_t launch_sparse_gather(int B, int max_sel, int pages_per_request, const void *kv_pool, int num_pool_pages,
                                 const int32_t *block_table, int64_t table_stride, const int32_t *seq_lens,
                                 const int32_t *sel, int64_t sel_stride, const int32_t *sel_count, void *dense_pool,
                                 int32_t *dense_table, int32_t *dense_lens, int sm_count, cudaStream_t stream) {
    const int64_t total = (int64_t)B * pages_per_request * kPage;
    const int warps_per_block = kGatherThreads / 32;
    int64_t blocks = (total + (int64_t)warps_per_block * kRowsInFlight - 1) / ((int64_t)warps_per_block * kRowsInFlight);
    const int64_t cap = (int64_t)sm_count * 8 * 4;      // a few waves of full SMs; the loop strides over the rest
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    sparse_gather_kernel<<<(unsigned)blocks, kGatherThreads, 0, stream>>>(
        B, max_sel, pages_per_request, static_cast<const uint8_t *>(kv_pool), num_pool_pages, block_table, table_stride,
        seq_lens, sel, sel_stride, sel_count, static_cast<uint8_t *>(dense_pool), dense_table, dense_lens);
    count_launch();
    return cudaGetLastError();
}

}  // namespace splash
