// KV page migration between two page pools in HBM, with block-table rewrite: the
// single-GPU part of a layout switch (kept blocks are repacked into the destination
// view; the table is the page metadata that must follow them).  Byte-exact.
#include "splash_common.cuh"

namespace splash {

namespace {

constexpr int kCopyThreads = 256;
constexpr int kCopyCtasPerPage = 4;

__global__ void remap_fill_kernel(int32_t *remap, int32_t n) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) remap[i] = -1;
}

__global__ void remap_scatter_kernel(int32_t *remap, const int32_t *__restrict__ src_ids,
                                     const int32_t *__restrict__ dst_ids, int64_t n, int32_t src_base,
                                     int32_t dst_base, int32_t max_page_id) {
    int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j < n) {
        int32_t s = src_base + src_ids[j];
        if (s >= 0 && s < max_page_id) remap[s] = dst_base + dst_ids[j];
    }
}

__global__ void table_rewrite_kernel(int32_t *table, int64_t num_entries, const int32_t *__restrict__ remap,
                                     int32_t max_page_id) {
    int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e < num_entries) {
        int32_t id = table[e];
        if (id >= 0 && id < max_page_id) {
            int32_t r = remap[id];
            if (r >= 0) table[e] = r;
        }
    }
}

// grid (n, kCopyCtasPerPage): 16-byte vector copy of one quarter of page j; CTA 0 of
// a page also moves its scale page.
__global__ void __launch_bounds__(kCopyThreads)
page_copy_kernel(const uint4 *__restrict__ src_pool, uint4 *__restrict__ dst_pool,
                 const uint4 *__restrict__ src_scales, uint4 *__restrict__ dst_scales,
                 int64_t page_vecs, const int32_t *__restrict__ src_ids, const int32_t *__restrict__ dst_ids) {
    const int64_t j = blockIdx.x;
    const int part = blockIdx.y;
    const int64_t s = src_ids[j], d = dst_ids[j];
    const uint4 *src = src_pool + s * page_vecs;
    uint4 *dst = dst_pool + d * page_vecs;
    const int64_t per = (page_vecs + kCopyCtasPerPage - 1) / kCopyCtasPerPage;
    const int64_t begin = per * part;
    const int64_t end = begin + per < page_vecs ? begin + per : page_vecs;
    int64_t c = begin + threadIdx.x;
    // four independent 16-byte loads in flight per thread
    for (; c + 3 * kCopyThreads < end; c += 4 * kCopyThreads) {
        uint4 v0 = __ldg(src + c), v1 = __ldg(src + c + kCopyThreads);
        uint4 v2 = __ldg(src + c + 2 * kCopyThreads), v3 = __ldg(src + c + 3 * kCopyThreads);
        dst[c] = v0; dst[c + kCopyThreads] = v1; dst[c + 2 * kCopyThreads] = v2; dst[c + 3 * kCopyThreads] = v3;
    }
    for (; c < end; c += kCopyThreads) dst[c] = __ldg(src + c);
    if (src_scales != nullptr && part == 0 && threadIdx.x < kPage * 4 / 16)
        dst_scales[d * (kPage * 4 / 16) + threadIdx.x] = __ldg(src_scales + s * (kPage * 4 / 16) + threadIdx.x);
}

// Remap table of the allocation-free entry point: lives in the library's device image,
// one copy on every GPU that loads it, until the process exits.
static __device__ __align__(256) int32_t g_static_remap[kStaticMigrateMaxPageId];

}  // namespace

// Device address of g_static_remap on the current device.  In host code the array's
// name only stands for the symbol; the address a kernel can use comes from
// cudaGetSymbolAddress, looked up once per device with that device current.
// The per-device cache is filled under a lock, so that two host threads making their first call on a device at the
// same time do not race on it (both would store the same address, but the lock costs nothing next to a launch).
cudaError_t static_remap_address(int32_t **ptr) {
    static int32_t *cache[64] = {nullptr};
    static std::mutex mu;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mu);
    if (cache[dev] == nullptr) {
        void *addr = nullptr;
        e = cudaGetSymbolAddress(&addr, g_static_remap);
        if (e != cudaSuccess) return e;
        cache[dev] = static_cast<int32_t *>(addr);
    }
    *ptr = cache[dev];
    return cudaSuccess;
}

cudaError_t launch_page_migrate(const void *src_pool, const float *src_scales, void *dst_pool,
                                float *dst_scales, int64_t page_bytes, const int32_t *src_ids,
                                const int32_t *dst_ids, int64_t n, int32_t src_base, int32_t dst_base,
                                int32_t max_page_id, int32_t *block_table, int64_t num_entries,
                                int32_t *remap, bool do_table, bool do_copy, cudaStream_t stream) {
    cudaError_t e;
    if (do_table && num_entries > 0 && max_page_id > 0) {
        remap_fill_kernel<<<(max_page_id + 255) / 256, 256, 0, stream>>>(remap, max_page_id);
        count_launch();
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        remap_scatter_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(remap, src_ids, dst_ids, n, src_base,
                                                                               dst_base, max_page_id);
        count_launch();
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        table_rewrite_kernel<<<(unsigned)((num_entries + 255) / 256), 256, 0, stream>>>(block_table, num_entries,
                                                                                        remap, max_page_id);
        count_launch();
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    if (!do_copy) return cudaSuccess;
    dim3 grid((unsigned)n, kCopyCtasPerPage);
    page_copy_kernel<<<grid, kCopyThreads, 0, stream>>>(
        static_cast<const uint4 *>(src_pool), static_cast<uint4 *>(dst_pool),
        reinterpret_cast<const uint4 *>(src_scales), reinterpret_cast<uint4 *>(dst_scales),
        page_bytes / 16, src_ids, dst_ids);
    count_launch();
    return cudaGetLastError();
}

}  // namespace splash
