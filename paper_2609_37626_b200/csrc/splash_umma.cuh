// Device-side building blocks shared by the tcgen05 decode kernels: mbarrier waits with a
// wall-clock bound, TMA loads, tcgen05 MMA / commit / tensor-memory access, descriptors.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>

#include "splash_common.cuh"

namespace splash {
namespace umma {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // 2 s

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done != 0;
}
// non-blocking probe (try_wait may suspend the thread for a while before it answers)
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done != 0;
}
__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

struct Ctx {
    volatile uint32_t *abort_flag;   // shared
    int32_t *status;                 // global, 16 ints
};

// Bounded wait.  Returns false if the CTA is aborting (this wait or another one timed out).
static __device__ __noinline__ bool mbar_wait_slow(const Ctx &ctx, uint32_t bar, uint32_t parity, int bar_id) {
    if (*ctx.abort_flag) return false;            // once the CTA is aborting no wait blocks any more
    const unsigned long long start = global_timer_ns();
    for (;;) {
        for (int k = 0; k < 256; ++k)
            if (mbar_try_wait(bar, parity)) return true;
        if (*ctx.abort_flag) return false;
        if (global_timer_ns() - start > kWaitLimitNs) {
            *ctx.abort_flag = 1;
            if (atomicCAS(ctx.status, 0, (int)SPLASH_DEVICE_TIMEOUT) == 0) {
                ctx.status[1] = (int)blockIdx.x;
                ctx.status[2] = bar_id;
                ctx.status[3] = (int)threadIdx.x;
            }
            return false;
        }
    }
}
__device__ __forceinline__ bool mbar_wait(const Ctx &ctx, uint32_t bar, uint32_t parity, int bar_id) {
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(ctx, bar, parity, bar_id);
}

// TMA store of a shared-memory tile (bulk async-group completion); coordinates outside the
// tensor are clipped
__device__ __forceinline__ void tma_store_3d(const CUtensorMap *map, uint32_t src, int c0, int c1, int c2) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
                 ::"l"(map), "r"(src), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
// Bulk copy of `bytes` (a multiple of 16; both addresses 16-byte aligned) from this CTA's shared memory to global
// memory, completion tracked by the thread's bulk async-group.
__device__ __forceinline__ void bulk_store(void *gdst, uint32_t ssrc, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(ssrc), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit_group() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// all committed groups of this thread have finished READING shared memory / have completed
__device__ __forceinline__ void bulk_wait_group_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_group() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}

__device__ __forceinline__ void tcgen05_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

// 16 consecutive fp32 columns of this warp's 32 lanes
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float (&v)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
          "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])),
          "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])),
          "r"(__float_as_uint(v[11])), "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])),
          "r"(__float_as_uint(v[15])) : "memory");
}
// 16 TMEM lanes x 64 fp32 columns in the MMA accumulator fragment layout: thread T of the
// warp gets, for k = 0..7, v[4k+0..1] = (lane T/4,     columns 8k + 2(T%4), +1) and
//                          v[4k+2..3] = (lane T/4 + 8, the same two columns).
__device__ __forceinline__ void tmem_ld_16x256b_x8(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.16x256b.x8.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// Same fragment layout, 32 columns: v[4k+0..1] = (lane T/4, columns 8k + 2(T%4), +1),
// v[4k+2..3] = (lane T/4 + 8, same columns), k = 0..3.
__device__ __forceinline__ void tmem_ld_16x256b_x4(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.16x256b.x4.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// Same fragment layout, 16 columns: k = 0..1.
__device__ __forceinline__ void tmem_ld_16x256b_x2(uint32_t taddr, float (&v)[8]) {
    uint32_t r[8];
    asm volatile(
        "tcgen05.ld.sync.aligned.16x256b.x2.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
        : "r"(taddr) : "memory");
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void softmax_bar_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// bar.sync among the 128 softmax threads that also ORs a predicate over them
__device__ __forceinline__ bool softmax_bar_or(bool pred) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.or.pred p, 1, 128, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(out) : "r"(pred ? 1u : 0u) : "memory");
    return out != 0;
}

// named barriers with a compile-time id and thread count
template <int ID, int COUNT>
__device__ __forceinline__ void named_bar_sync() {
    asm volatile("bar.sync %0, %1;" ::"n"(ID), "n"(COUNT) : "memory");
}
template <int ID, int COUNT>
__device__ __forceinline__ bool named_bar_or(bool pred) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.or.pred p, %2, %3, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(out) : "r"(pred ? 1u : 0u), "n"(ID), "n"(COUNT) : "memory");
    return out != 0;
}
// named barrier whose id is a run-time value (one of several equivalent barriers)
template <int COUNT>
__device__ __forceinline__ void named_bar_sync_dyn(int id) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "n"(COUNT) : "memory");
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Shared-memory matrix descriptor, 128-byte swizzle (layout type 2), descriptor version 1.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return (uint64_t)((saddr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | (2ull << 61);
}
// Same with the 64-byte swizzle (layout type 4).
__device__ __forceinline__ uint64_t make_desc_sw64(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return (uint64_t)((saddr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | (4ull << 61);
}

// Shared-memory matrix descriptor without swizzle (layout type 0) for an MN-major operand, used for P^T with the tokens
// on K: 16 bytes of one token (16 heads of 8 bits, 8 heads of 16) are adjacent, eight tokens make a 128-byte core matrix,
// `k_group_bytes` leads from one group of eight tokens to the next and `mn_group_bytes` from one group of heads to the next.
__device__ __forceinline__ uint64_t make_desc_mn_plain(uint32_t saddr, uint32_t k_group_bytes, uint32_t mn_group_bytes) {
    return (uint64_t)((saddr >> 4) & 0x3FFFu) | ((uint64_t)((k_group_bytes >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((mn_group_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}

// N columns of 16 TMEM lanes in the accumulator fragment layout: v[4k + e] = (lane T/4, column 8k + 2(T%4) + e),
// v[4k + 2 + e] = (lane T/4 + 8, the same column), k < N / 8, e < 2.
template <int N>
__device__ __forceinline__ void tmem_ld_frag(uint32_t taddr, float (&v)[N / 2]) {
    if constexpr (N == 16) tmem_ld_16x256b_x2(taddr, v);
    else tmem_ld_16x256b_x4(taddr, v);
}

// byte offset of (row, byte column) inside a [rows][64 B] slab in the 64-byte swizzle
__device__ __forceinline__ uint32_t sw64(uint32_t row, uint32_t col_byte) {
    return row * 64 + ((((col_byte >> 4) ^ (row >> 1)) & 3) << 4) + (col_byte & 15);
}

// Instruction descriptor: fp32 accumulate, bf16 x bf16.
__host__ __device__ constexpr uint32_t make_idesc(int M, int N, int a_mn_major, int b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// Valid rows of a tile after the token shift: page-relative tokens [a, b) land in rows
// [r_lo, r_hi) of the 64-row box when the box starts at token tok0.  The shift moves ONE cut
// end out of the page, where the TMA unit fills zeros; a range cut at both ends inside one
// page (`both`) cannot be loaded that way -- the rows of tokens [0, a) would arrive with
// whatever the cache holds there, and 0 x NaN is NaN inside P.V -- so the producers copy such a
// tile by hand (fill_rows_by_hand) and write zeros for every row outside the range.
struct TileGeom { int tok0, r_lo, r_hi, a, b; bool both; };
__device__ __forceinline__ TileGeom tile_geom(int lo, int hi, int t0) {
    int a = max(lo, t0) - t0;
    int b = min(hi, t0 + kPage) - t0;
    TileGeom g;
    g.a = a; g.b = b; g.both = a > 0 && b < kPage;
    if (b < kPage) { g.tok0 = b - kPage; g.r_lo = kPage - b + a; g.r_hi = kPage; }   // end cut: align the end to the box end
    else { g.tok0 = a; g.r_lo = 0; g.r_hi = kPage - a; }                              // front cut (or none)
    return g;
}

// What one TMA box would have delivered, written by the 32 lanes of a warp with plain loads and stores: rows
// [0, nrows) of `nchunks` chunk slabs, row r holding token tok_first + r of the page when that token lies in [a, b) and
// zeros otherwise.  kChunkBytes = 128: 16-bit elements in the 128-byte swizzle; 64: 8-bit elements in the 64-byte
// swizzle (a cache row is nine chunks either way).  `slabs` is the stage's first slab (1024-byte aligned), chunk
// src_chunk0 + c of the row goes to slab dst_slot0 + c; page == nullptr (an id outside the pool) gives zeros.  The caller
// follows up with fence.proxy.async and its barrier arrival.  Only the rare tile cut at both ends takes this path.
template <int kChunkBytes>
__device__ __forceinline__ void fill_rows_by_hand(uint8_t *slabs, uint32_t slab_bytes, int nrows, const uint8_t *page,
                                                  int tok_first, int a, int b, int src_chunk0, int dst_slot0, int nchunks, int lane) {
    constexpr int kPieces = kChunkBytes / 16;
    const int total = nrows * nchunks * kPieces;
    for (int idx = lane; idx < total; idx += 32) {
        const int j = idx % kPieces, r = (idx / kPieces) % nrows, c = idx / (kPieces * nrows);
        const int t = tok_first + r;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (page != nullptr && t >= a && t < b)
            v = __ldg(reinterpret_cast<const uint4 *>(page + (size_t)t * (9 * kChunkBytes) + (size_t)(src_chunk0 + c) * kChunkBytes + j * 16));
        const int sw = kChunkBytes == 128 ? (r & 7) : ((r >> 1) & 3);
        *reinterpret_cast<uint4 *>(slabs + (size_t)(dst_slot0 + c) * slab_bytes + (size_t)r * kChunkBytes + ((j ^ sw) << 4)) = v;
    }
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled() {
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// 4-D map (64 elements, rows, 9 chunks, outer): a 576-wide row is seen as 9 chunks of 64
// elements, so one box of (64, box_rows, 9, 1) lands in shared memory as [chunk][row][64
// elements], each chunk slab in the swizzle the MMA descriptors expect (128 B for 16-bit
// elements, 64 B for 8-bit ones).
inline bool make_map_4d(CUtensorMap *map, CUtensorMapDataType dtype, CUtensorMapSwizzle swizzle, const void *base,
                        uint64_t rows, uint64_t outer, uint64_t row_stride_bytes, uint64_t chunk_stride_bytes,
                        uint64_t outer_stride_bytes, uint32_t box_rows, uint32_t box_chunks = 9) {
    EncodeTiledFn fn = encode_tiled();
    if (!fn) { set_error("cuTensorMapEncodeTiled is not available"); return false; }
    cuuint64_t dims[4] = {64, rows, 9, outer};
    cuuint64_t strides[3] = {row_stride_bytes, chunk_stride_bytes, outer_stride_bytes};
    cuuint32_t box[4] = {64, box_rows, box_chunks, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = fn(map, dtype, 4, const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { set_error("cuTensorMapEncodeTiled failed with CUresult %d", (int)r); return false; }
    return true;
}

// 3-D map over fp32 rows for stores: (columns, rows, outer), row and outer strides in bytes
// (multiples of 16), box = (32 columns, box_rows, 1), 128-byte swizzle: the shared-memory tile
// is [box_rows][128 B] with the 16-byte chunks of row r at position (chunk ^ (r & 7)).
inline bool make_store_map_3d(CUtensorMap *map, void *base, uint64_t cols, uint64_t rows, uint64_t outer,
                              uint64_t row_stride_bytes, uint64_t outer_stride_bytes, uint32_t box_rows) {
    EncodeTiledFn fn = encode_tiled();
    if (fn == nullptr) return false;
    cuuint64_t dims[3] = {cols, rows, outer};
    cuuint64_t strides[2] = {row_stride_bytes, outer_stride_bytes};
    cuuint32_t box[3] = {32, box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace umma
}  // namespace splash
