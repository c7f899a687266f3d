// tcgen05 / TMA decode kernel for e4m3 KV (one fp32 scale per token) and NARROW head slices:
// N = 16 or 32 heads per CTA, the shard of a TP / DOP rank whose cache is kept in the paper's
// precision.  The 64-head e4m3 kernel pads such a slice to 64 rows of an MMA and to 64 heads of
// softmax work; here the problem is transposed ("tokens on M"), as in the bf16 kernel's narrow
// path, so that a 16-head slice costs 16-wide MMAs:
//
//     S^T [64 tokens x 2N]       = K_tile [64 x 576]   * [q_hi | q_lo]^T [576 x 2N]    (M = 64, K = 32)
//     O^T [512 dv    x 2N]      += V_tile^T [512 x 64] * [P_hi | 16 P_lo]^T [64 x 2N]  (4 x M = 128)
//
// The cache bytes go to the tensor cores as stored (kind::f8f6f4); V is the first 512 columns of the
// very K rows in shared memory, read as an MN-major operand.  The two bf16-precision operands are
// split into two 8-bit terms each, exactly as in the 64-head kernel: q = qs_h (hi + lo) with one
// scale per head (e4m3 + e4m3, rebuilt per request by converter warps one request ahead; the two
// terms sit side by side as 2N rows of one B operand and the softmax warps add the two halves of
// S^T), and P = hi + lo with the token scale folded into the weight in the log domain,
//     y = (q . codes) * qs_h * scale_t * softmax_scale * log2(e) + log2(scale_t),   P = 2^(y - m + 2.75),
// the row sum adding P / scale_t.  Here the two terms of P are 2N columns of ONE B operand too, so that the
// V tile -- the operand whose read from shared memory sets the pace of these narrow MMAs -- is read once
// per tile instead of twice; O^T then has a hi and a lo half that the epilogue adds, which lets the lo
// term carry its own scale: it is stored as e4m3 of 16 x the residual (three significant bits, never out
// of range since an e4m3 residual is at most 2^-4 of the value) and the epilogue adds lo / 16.  With the tokens on the TMEM lanes the token scale is one
// number per thread, and a thread's weights for its token are N adjacent bytes of an MN-major
// P^T.  A page is 36,864 bytes and the query operands are small, so five stages fit (four with 32
// heads): the loop is a ring of dependent latencies and its period is the ring divided by the stages.
//
// The softmax warps keep one reference maximum per head and move it only when a logit exceeds it by
// more than 2^6 (the headroom that e4m3's range leaves above the lift): whether any does is one
// barrier-wide OR per tile, and only then do they reduce the maxima across tokens, move the
// references and rescale O^T.  Row sums stay per thread until the request ends.
//
// Warp roles (352 threads, 480 with 32 heads): TMA producer (pages + scale pages, next page pulled into L2), 2 QK^T
// issuers (one partial accumulator of S^T each), 2 P.V issuers (two dv blocks each), N / 4 softmax /
// epilogue warps (one per TMEM lane quadrant and group of 16 heads), 2 query converter warps (a request ahead: the query operands are double buffered).  Every wait is bounded; on expiry the CTA records
// SPLASH_DEVICE_TIMEOUT and leaves in order.
#include "splash_fp8.cuh"
#include "splash_pair.cuh"

namespace splash {

namespace {

using namespace umma;

constexpr int kQkWarps = 2;                        // = partial accumulators of S^T
constexpr int kPvWarps = 2;                        // each owns two of the four dv blocks of O^T
constexpr int kWarpQk = 1;
constexpr int kWarpPv = kWarpQk + kQkWarps;
constexpr int kWarpSoftmax = kWarpPv + kPvWarps;            // 5: TMEM lane quadrant = warp & 3
constexpr int kChunks = 9;                         // 576 / 64-element (64 B) chunks
constexpr uint32_t kSlab = 64 * 64;                // one chunk of one page: 64 tokens x 64 B
constexpr uint32_t kStageBytes = kChunks * kSlab;  // 36,864
constexpr uint32_t kScaleBytes = 256;              // 64 fp32 token scales of a page
constexpr int kMaxStages = 5;
// A reference maximum moves when a logit exceeds it by more than kTau (log2 units); every move costs the tile a pass
// over O^T behind the previous tile's P.V, and with 16 or 32 heads per CTA the moves of all heads add up (kTau = 4:
// every third tile early in a request).  Weights are stored as 2^(y - m + kLift) <= 2^8.75 = 431 < 448.
constexpr float kTau = 6.0f;
constexpr float kLift = 2.75f;

enum BarrierId {
    kBarKvFull = 0,                    // [stages]
    kBarKvEmpty = kBarKvFull + kMaxStages,
    kBarQFull = kBarKvEmpty + kMaxStages,   // [2]: one per query operand buffer
    kBarQEmpty = kBarQFull + 2,        // [2]: the QK^T issuers are done with the buffer AND the softmax warps with the request
                                       // (they stage its output tile there)
    kBarSFull = kBarQEmpty + 2,        // [2]
    kBarSEmpty = kBarSFull + 2,        // [2]
    kBarPFull = kBarSEmpty + 2,        // [2]: one per P buffer.  With a single barrier the softmax warps, which may run two
                                       // tiles ahead of a P.V issuer, could complete two phases between two of its polls
    kBarOFull = kBarPFull + 2,
    kBarOEmpty,
    kNumBarriers
};

template <int N>
struct Layout {
    static constexpr int kStages = N == 16 ? 5 : 4;
    static constexpr int kSoftmaxWarps = N / 4;                // one per TMEM lane quadrant and group of 16 heads
    static constexpr int kSoftmaxThreads = 32 * kSoftmaxWarps;
    static constexpr int kWarpConvert = kWarpSoftmax + kSoftmaxWarps;
    static constexpr int kNumConvertWarps = 2;                 // four threads per head, 16 heads per pass
    static constexpr int kThreads = (kWarpConvert + kNumConvertWarps) * 32;   // 352 (N = 16) or 480 (N = 32)
    static constexpr uint32_t kQSlab = 2 * N * 64;             // one chunk of the query operand: (N hi rows, N lo rows) x 64 B
    static constexpr uint32_t kQBytes = kChunks * kQSlab;      // one buffer; there are two (request parity)
    static constexpr uint32_t kPBytes = 2 * N * 64;            // P^T: [2N / 16 groups: hi, then lo][64 tokens][16 heads], one byte each
    static constexpr uint32_t kOffKv = 0;
    static constexpr uint32_t kOffQ = kOffKv + kStages * kStageBytes;
    static constexpr uint32_t kOffP = kOffQ + 2 * kQBytes;     // double buffered (tile parity)
    static constexpr uint32_t kOffScale = kOffP + 2 * kPBytes; // float [kStages][64]
    static constexpr uint32_t kOffQs = kOffScale + kStages * kScaleBytes;   // float [4][N] query scales, by segment & 3
    static constexpr uint32_t kOffRed = kOffQs + 4 * N * 4;    // float [N][4]
    static constexpr uint32_t kOffM = kOffRed + N * 16;        // float [N] reference maxima, log2 domain
    static constexpr uint32_t kOffAlpha = kOffM + N * 4;       // float [N]
    static constexpr uint32_t kOffL = kOffAlpha + N * 4;       // float [N]
    static constexpr uint32_t kOffBar = kOffL + N * 4;
    static constexpr uint32_t kOffMisc = (kOffBar + kNumBarriers * 8 + 15) / 16 * 16;   // u32: tmem base, abort
    static constexpr uint32_t kBytes = kOffMisc + 16;
    static constexpr uint32_t kColO = 0;                       // 4 dv blocks x (N hi, N lo) columns
    static constexpr uint32_t kColS = 8 * N;                   // 2 buffers x kQkWarps partials x (N hi, N lo) columns
    static_assert(kColS + 2 * kQkWarps * 2 * N <= 512, "tensor memory overflow");
    static_assert(kBytes <= 232448, "shared memory overflow");
    static_assert(kOffQ % 1024 == 0 && kQSlab % 512 == 0 && kOffP % 128 == 0, "operands need aligned windows");
};

// ---------------------------------------------------------------- the kernel
template <int N>
__global__ void __launch_bounds__(Layout<N>::kThreads, 1)
decode_umma_fp8_narrow_kernel(const DecodeParams p, const __grid_constant__ CUtensorMap tmap_kv) {
    using L = Layout<N>;
    constexpr int kStages = L::kStages, kThreads = L::kThreads, kNumSoftmaxWarps = L::kSoftmaxWarps, kWarpConvert = L::kWarpConvert;
    constexpr int kSoftmaxThreads = L::kSoftmaxThreads;
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int worker = blockIdx.x / p.num_groups;
    const int group = blockIdx.x % p.num_groups;
    const int head0 = p.head_begin + group * N;
    const int h = p.head_end - p.head_begin;

    volatile uint32_t *misc = reinterpret_cast<volatile uint32_t *>(smem + L::kOffMisc);
    Ctx ctx{misc + 1, p.status};
    auto bar = [&](int id) -> uint32_t { return sbase + L::kOffBar + 8u * (uint32_t)id; };

    if ((sbase & 1023u) != 0) {      // swizzle atoms need an aligned window
        if (tid == 0 && atomicCAS(p.status, 0, (int)SPLASH_CUDA_ERROR) == 0) { p.status[1] = (int)blockIdx.x; p.status[2] = -100; }
        return;
    }
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(bar(kBarKvFull + s), 1); mbar_init(bar(kBarKvEmpty + s), kPvWarps); }
        for (int b = 0; b < 2; ++b) { mbar_init(bar(kBarQFull + b), L::kNumConvertWarps); mbar_init(bar(kBarQEmpty + b), kQkWarps + kNumSoftmaxWarps); }
        for (int b = 0; b < 2; ++b) { mbar_init(bar(kBarSFull + b), kQkWarps); mbar_init(bar(kBarSEmpty + b), kNumSoftmaxWarps); }
        for (int b = 0; b < 2; ++b) mbar_init(bar(kBarPFull + b), kNumSoftmaxWarps);
        mbar_init(bar(kBarOFull), kPvWarps); mbar_init(bar(kBarOEmpty), kNumSoftmaxWarps);
        misc[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sbase + L::kOffMisc), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = misc[0];
    grid_dependency_wait();       // the plan kernel's output is read from here on
    const long long t_start = clock64();

    SegmentIter it;
    it.init(p, worker);
    Segment seg;
    long long *const trace = blockIdx.x == 0 ? p.trace : nullptr;
    auto mark = [&](uint32_t tile, int ev) {
        if (trace != nullptr && tile < 64) trace[tile * 8 + ev] = clock64();
    };

    if (warp == 0) {
        // ===================================================== TMA producer (pages + their scale pages)
        uint32_t kv_it = 0;
        bool ok = true;
        while (ok && it.next(p, seg)) {
            const int first_page = seg.lo / kPage;
            const int32_t *table = p.block_table + (int64_t)seg.request * p.table_stride;
            int entry = 0;
            for (int tile = seg.tile_begin; ok && tile < seg.tile_end; ++tile) {
                const int rel = tile - seg.tile_begin;
                if ((rel & 31) == 0) {
                    int idx = tile + lane;
                    entry = idx < seg.tile_end ? table[first_page + idx] : 0;
                }
                const int page = __shfl_sync(0xffffffffu, entry, rel & 31);
                // the next page (when its table entry is among the 32 this warp holds): pulled into L2 now
                const int page_ahead = __shfl_sync(0xffffffffu, entry, (rel + 1) & 31);
                const bool ahead_ok = (rel & 31) + 1 < 32 && tile + 1 < seg.tile_end;
                const TileGeom g = tile_geom(seg.lo, seg.hi, (first_page + tile) * kPage);
                const uint32_t stage = kv_it % kStages, ph = (kv_it / kStages) & 1;
                // a page id outside the pool reads as zeros through the tensor map; its tokens get the scale 1
                const bool in_pool = page >= 0 && page < p.num_pool_pages;
                if (lane == 0) {
                    ok = mbar_wait(ctx, bar(kBarKvEmpty + stage), ph ^ 1, kBarKvEmpty + stage);
                    mark(kv_it, 0);
                    if (ok && !in_pool) {
                        float *sc1 = reinterpret_cast<float *>(smem + L::kOffScale + stage * kScaleBytes);
                        for (int t = 0; t < kPage; ++t) sc1[t] = 1.0f;
                    }
                    if (ok && !g.both) {
                        mbar_expect_tx(bar(kBarKvFull + stage), kStageBytes + (in_pool ? kScaleBytes : 0u));
                        tma_load_4d(sbase + L::kOffKv + stage * kStageBytes, &tmap_kv, bar(kBarKvFull + stage), 0, g.tok0, 0, page);
                        if (in_pool)
                            bulk_load(sbase + L::kOffScale + stage * kScaleBytes, p.kv_scales + (int64_t)page * kPage,
                                      kScaleBytes, bar(kBarKvFull + stage));
                        if (ahead_ok && page_ahead >= 0 && page_ahead < p.num_pool_pages)
                            bulk_prefetch_l2(static_cast<const uint8_t *>(p.kv_pool) + (size_t)page_ahead * (kPage * kDQK), kStageBytes);
                        mark(kv_it, 1);
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (ok && g.both) {
                    // a range cut at both ends inside this page: the warp writes the box itself, zeros outside the range
                    const uint8_t *src = in_pool ? static_cast<const uint8_t *>(p.kv_pool) + (size_t)page * (kPage * kDQK) : nullptr;
                    fill_rows_by_hand<64>(smem + L::kOffKv + stage * kStageBytes, kSlab, kPage, src, g.tok0, g.a, g.b, 0, 0, 9, lane);
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) {
                        if (in_pool) {
                            mbar_expect_tx(bar(kBarKvFull + stage), kScaleBytes);
                            bulk_load(sbase + L::kOffScale + stage * kScaleBytes, p.kv_scales + (int64_t)page * kPage,
                                      kScaleBytes, bar(kBarKvFull + stage));
                        } else {
                            mbar_arrive(bar(kBarKvFull + stage));
                        }
                    }
                }
                ++kv_it;
            }
        }
    } else if (warp < kWarpPv) {
        // ===================================================== QK^T issuers: S^T = K [q hi | q lo]^T
        if (lane == 0) {
            const int a = warp - kWarpQk;            // partial accumulator a
            constexpr uint32_t kIdescQK = make_idesc_e4m3(64, 2 * N, 0);
            uint32_t kv = 0, seg_it = 0;
            bool ok = true;
            while (ok && it.next(p, seg)) {
                const int ntiles = seg.tile_end - seg.tile_begin;
                const uint32_t qb = seg_it & 1;
                ok = mbar_wait(ctx, bar(kBarQFull + qb), (seg_it >> 1) & 1, kBarQFull + qb);
                for (int i = 0; ok && i < ntiles; ++i, ++kv) {
                    const uint32_t stage = kv % kStages, b = kv & 1;
                    ok = mbar_wait(ctx, bar(kBarKvFull + stage), (kv / kStages) & 1, kBarKvFull + stage) &&
                         mbar_wait(ctx, bar(kBarSEmpty + b), ((kv >> 1) & 1) ^ 1, kBarSEmpty + b);
                    if (!ok) break;
                    if (a == 0) mark(kv, 2);
                    tcgen05_fence_after();
                    const uint32_t k0 = sbase + L::kOffKv + stage * kStageBytes;
                    const uint32_t d = tmem_base + L::kColS + (b * kQkWarps + a) * (2 * N);
                    // 18 K = 32 steps per tile; this issuer takes every second
#pragma unroll
                    for (int t = 0; t < 18 / kQkWarps; ++t) {
                        const int ks = t * kQkWarps + a, c = ks >> 1, k = ks & 1;
                        uint64_t dk = make_desc_sw64(k0 + c * kSlab + k * 32, 16, 512);                      // A: 64 tokens x 32
                        uint64_t dq = make_desc_sw64(sbase + L::kOffQ + qb * L::kQBytes + c * L::kQSlab + k * 32, 16, 512);    // B: 2N rows x 32
                        umma_e4m3(d, dk, dq, kIdescQK, t != 0);
                    }
                    umma_commit(bar(kBarSFull + b));
                    if (a == 0) mark(kv, 3);
                }
                if (ok) umma_commit(bar(kBarQEmpty + qb));
                ++seg_it;
            }
        }
    } else if (warp < kWarpSoftmax) {
        // ===================================================== P.V issuers: [O^T hi | O^T lo] += V^T [P hi | 16 P lo]^T
        if (lane == 0) {
            const int pj = warp - kWarpPv;           // dv blocks 2 pj and 2 pj + 1
            constexpr uint32_t kIdescPV = make_idesc_e4m3(128, 2 * N, 1, 0, 1);
            uint32_t kv = 0, seg_it = 0;
            bool ok = true;
            while (ok && it.next(p, seg)) {
                const int ntiles = seg.tile_end - seg.tile_begin;
                for (int i = 0; ok && i < ntiles; ++i, ++kv) {
                    const uint32_t stage = kv % kStages;
                    ok = mbar_wait(ctx, bar(kBarPFull + (kv & 1)), (kv >> 1) & 1, kBarPFull + (kv & 1));
                    if (ok && i == 0) ok = mbar_wait(ctx, bar(kBarOEmpty), (seg_it & 1) ^ 1, kBarOEmpty);
                    if (!ok) break;
                    if (pj == 0) mark(kv, 6);
                    tcgen05_fence_after();
                    const uint32_t v0 = sbase + L::kOffKv + stage * kStageBytes;
#pragma unroll
                    for (int k = 0; k < 2; ++k) {
#pragma unroll
                        for (int jj = 0; jj < 2; ++jj) {
                            const int j = 2 * pj + jj;
                            // A: two 64-element chunks (LBO apart) x 32 tokens (SBO per 8 tokens), MN-major
                            uint64_t da = make_desc_sw64(v0 + (2 * j) * kSlab + k * 2048, kSlab, 512);
                            // B: 32 tokens (four groups of eight, 128 B apart) x 2N columns (groups of 16, 1024 B apart)
                            uint64_t db = make_desc_mn_plain(sbase + L::kOffP + (kv & 1) * L::kPBytes + k * 512, 128, 1024);
                            umma_e4m3(tmem_base + L::kColO + j * (2 * N), da, db, kIdescPV, (i != 0) || k != 0);
                        }
                    }
                    umma_commit(bar(kBarKvEmpty + stage));   // P.V done: stage free, P buffers free, O^T updated
                    if (i + 1 == ntiles) umma_commit(bar(kBarOFull));
                    if (pj == 0) mark(kv, 7);
                }
                ++seg_it;
            }
        }
    } else if (warp >= kWarpConvert) {
        // ===================================================== query converters
        // bf16 query rows -> e4m3 hi + lo operands with one scale per head, four threads per head.  The operands are
        // double buffered, so the converters work a whole request ahead: the row is read once, into registers, and
        // the latency of those loads (several microseconds while the cache streams at full rate) stays off the
        // path from one request's last tile to the next one's first.
        constexpr int kVecs = 18;                      // 8-element vectors per thread: a quarter of a row
        const int ct = (warp - kWarpConvert) * 32 + lane;   // 0..63: head ct / 4 of a pass, quarter ct % 4
        float *qs_s = reinterpret_cast<float *>(smem + L::kOffQs);
        uint32_t seg_it = 0;
        bool ok = true;
        while (ok && it.next(p, seg)) {
            const uint32_t qb = seg_it & 1;
            uint8_t *qdst = smem + L::kOffQ + qb * L::kQBytes;
            const int part = ct & 3;
            {
                // the rows of the request after this one: into L2 now, so that their loads, a request from now, are short
                SegmentIter peek = it;
                Segment nxt;
                if (peek.next(p, nxt)) {
                    const char *row0 = reinterpret_cast<const char *>(static_cast<const __nv_bfloat16 *>(p.q) +
                                       (int64_t)nxt.request * p.q_stride_request + (int64_t)head0 * p.q_stride_head);
                    const int64_t bytes = (int64_t)min(N, p.head_end - head0) * p.q_stride_head * 2;
                    for (int64_t o = (int64_t)ct * 128; o < bytes; o += 64 * 128)
                        asm volatile("prefetch.global.L2 [%0];" ::"l"(row0 + o));
                }
            }
#pragma unroll 1
            for (int pass = 0; pass < N / 16; ++pass) {
                const int hd = pass * 16 + (ct >> 2);
                const int gh = head0 + hd;
                const bool live = gh < p.head_end;
                const uint4 *src = reinterpret_cast<const uint4 *>(
                    static_cast<const __nv_bfloat16 *>(p.q) + (int64_t)seg.request * p.q_stride_request +
                    (int64_t)(live ? gh : p.head_begin) * p.q_stride_head + part * (kVecs * 8));
                // 16 heads keep the quarter row in registers between the two passes; with 32 heads (480 threads, 128
                // registers each) it is read again, nine vectors at a time, from the cache it has just come into
                constexpr int kBatch = N == 16 ? kVecs : kVecs / 2;
                uint4 x[kBatch];
                float amax = 0.f;
#pragma unroll 1
                for (int v0 = 0; v0 < kVecs; v0 += kBatch) {
#pragma unroll
                    for (int v = 0; v < kBatch; ++v) x[v] = live ? __ldg(src + v0 + v) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                    for (int v = 0; v < kBatch; ++v) {
                        const uint32_t w[4] = {x[v].x, x[v].y, x[v].z, x[v].w};
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            amax = fmaxf(amax, fabsf(__uint_as_float(w[k] << 16)));
                            amax = fmaxf(amax, fabsf(__uint_as_float(w[k] & 0xffff0000u)));
                        }
                    }
                }
                amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
                amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
                const float qs = amax > 0.f ? amax * (1.0f / 448.0f) : 1.0f;
                const float inv = amax > 0.f ? 448.0f / amax : 1.0f;
                if (pass == 0) {
                    // this buffer's previous request (two back): its QK^T retired, its output tile staged and gone
                    ok = mbar_wait(ctx, bar(kBarQEmpty + qb), ((seg_it >> 1) & 1) ^ 1, kBarQEmpty + qb);
                    if (!ok) break;
                }
                if (part == 0) qs_s[(seg_it & 3) * N + hd] = qs;
#pragma unroll 1
                for (int v0 = 0; v0 < kVecs; v0 += kBatch) {
                    if (kBatch < kVecs) {
#pragma unroll
                        for (int v = 0; v < kBatch; ++v) x[v] = live ? __ldg(src + v0 + v) : make_uint4(0u, 0u, 0u, 0u);
                    }
#pragma unroll
                    for (int v = 0; v < kBatch; ++v) {
                        const uint32_t w[4] = {x[v].x, x[v].y, x[v].z, x[v].w};
                        uint16_t hi[4], lo[4];
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const float e0 = __uint_as_float(w[k] << 16) * inv, e1 = __uint_as_float(w[k] & 0xffff0000u) * inv;
                            split_e4m3_e4m3_x2(e0, e1, hi[k], lo[k]);
                        }
                        const uint32_t d = (uint32_t)(part * (kVecs * 8) + (v0 + v) * 8);
                        // the lo rows follow the N hi rows of the chunk (N is a multiple of 8: same swizzle phase)
                        const uint32_t off = (d >> 6) * L::kQSlab + sw64((uint32_t)hd, d & 63);
                        *reinterpret_cast<uint2 *>(qdst + off) =
                            make_uint2((uint32_t)hi[0] | ((uint32_t)hi[1] << 16), (uint32_t)hi[2] | ((uint32_t)hi[3] << 16));
                        *reinterpret_cast<uint2 *>(qdst + N * 64 + off) =
                            make_uint2((uint32_t)lo[0] | ((uint32_t)lo[1] << 16), (uint32_t)lo[2] | ((uint32_t)lo[3] << 16));
                    }
                }
            }
            if (!ok) break;
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarQFull + qb));
            ++seg_it;
        }
    } else {
        // ===================================================== softmax + epilogue warps
        const int q4 = warp & 3;                       // TMEM lane quadrant of this warp
        const int sw = warp - kWarpSoftmax;            // softmax warp
        const int wq = sw & 3;                         // its slot in the per-head exchange of four
        const int h0 = 16 * (sw >> 2);                 // its group of 16 heads
        const int st = sw * 32 + lane;                 // 0 .. 8N
        // S^T comes out of tensor memory in the accumulator fragment layout, which spreads the 16 lanes that an
        // M = 64 tile has per quadrant over all 32 threads: this thread holds tokens rA and rB = rA + 8 and, of each
        // group of eight heads (its warp has two), heads 2 tq and 2 tq + 1.
        const int rA = 16 * q4 + (lane >> 2), rB = rA + 8;
        const int tq = lane & 3;
        constexpr int kR = 2;                          // groups of eight heads per warp
        const uint32_t lane_addr = (uint32_t)(32 * q4) << 16;
        float *red = reinterpret_cast<float *>(smem + L::kOffRed);
        float *m_s = reinterpret_cast<float *>(smem + L::kOffM);
        float *alpha_s = reinterpret_cast<float *>(smem + L::kOffAlpha);
        float *l_s = reinterpret_cast<float *>(smem + L::kOffL);
        const float *qs_all = reinterpret_cast<const float *>(smem + L::kOffQs);
        const float *scale_s = reinterpret_cast<const float *>(smem + L::kOffScale);
        const float scale_log2 = p.softmax_scale * kLog2e;
        uint32_t s_it = 0, seg_it = 0;
        // A failed (timed-out) wait only clears `ok`: the role keeps walking its tiles so that every thread still
        // meets the named barriers -- once the CTA aborts, waits return at once.
        bool ok = true;
        while (it.next(p, seg)) {
            // the converter warps have written this segment's query operands and scales
            ok &= mbar_wait(ctx, bar(kBarQFull + (seg_it & 1)), (seg_it >> 1) & 1, kBarQFull + (seg_it & 1));
            const float *qs_s = qs_all + (seg_it & 3) * N;
            if (st < N) m_s[st] = -INFINITY;
            float l[2 * kR];              // sums of P / scale_t over this thread's tokens: heads 8k + 2 tq + e at [2k + e]
#pragma unroll
            for (int n = 0; n < 2 * kR; ++n) l[n] = 0.f;
            named_bar_sync<1, kSoftmaxThreads>();
            const int first_page = seg.lo / kPage;
            const int ntiles = seg.tile_end - seg.tile_begin;
            for (int i = 0; i < ntiles; ++i) {
                const TileGeom g = tile_geom(seg.lo, seg.hi, (first_page + seg.tile_begin + i) * kPage);
                const bool vA = rA >= g.r_lo && rA < g.r_hi, vB = rB >= g.r_lo && rB < g.r_hi;
                const uint32_t b = s_it & 1, stage = s_it % kStages;
                ok &= mbar_wait(ctx, bar(kBarSFull + b), (s_it >> 1) & 1, kBarSFull + b);
                if (st == 0) mark(s_it, 4);
                // the scale page rode on the stage's own barrier, long complete by now
                ok &= mbar_wait(ctx, bar(kBarKvFull + stage), (s_it / kStages) & 1, kBarKvFull + stage);
                tcgen05_fence_after();
                float s[4 * kR];
                {
                    // S^T = the sum of four N-column pieces: (partial 0, partial 1) x (q hi, q lo)
                    float t0[4 * kR], t1[4 * kR], t2[4 * kR];
                    const uint32_t sb = tmem_base + lane_addr + L::kColS + b * (2 * kQkWarps * N) + h0;
                    tmem_ld_16x256b_x2(sb, s);
                    tmem_ld_16x256b_x2(sb + N, t0);
                    tmem_ld_16x256b_x2(sb + 2 * N, t1);
                    tmem_ld_16x256b_x2(sb + 3 * N, t2);
                    tmem_wait_ld();
#pragma unroll
                    for (int n = 0; n < 4 * kR; ++n) s[n] = (s[n] + t0[n]) + (t1[n] + t2[n]);
                }
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarSEmpty + b));
                // this thread's tokens: their scales, log2 of them for the weights, reciprocals for the row sums
                const float tsA = vA ? scale_s[stage * 64 + g.tok0 + rA] : 1.0f, tsB = vB ? scale_s[stage * 64 + g.tok0 + rB] : 1.0f;
                const float lgA = fast_log2(tsA), lgB = fast_log2(tsB), rtsA = fast_rcp(tsA), rtsB = fast_rcp(tsB);
                const float tslA = tsA * scale_log2, tslB = tsB * scale_log2;
                bool exceeds = false;     // some logit of these tokens lies more than kTau above its head's reference
#pragma unroll
                for (int k = 0; k < kR; ++k) {
                    const float2 q2 = *reinterpret_cast<const float2 *>(&qs_s[h0 + 8 * k + 2 * tq]);
                    const float2 m2 = *reinterpret_cast<const float2 *>(&m_s[h0 + 8 * k + 2 * tq]);
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const float qv = e ? q2.y : q2.x, lim = (e ? m2.y : m2.x) + kTau;
                        // log2-domain logit + log2(token scale)
                        const float yA = vA ? fmaf(s[4 * k + e] * qv, tslA, lgA) : -INFINITY;
                        const float yB = vB ? fmaf(s[4 * k + 2 + e] * qv, tslB, lgB) : -INFINITY;
                        s[4 * k + e] = yA; s[4 * k + 2 + e] = yB;
                        exceeds |= (yA > lim) | (yB > lim);
                    }
                }
                const bool grew = named_bar_or<1, kSoftmaxThreads>(exceeds);
                if (grew) {
                    // the rare path (the first tile of a request, then a handful of times): per-head maxima over the
                    // tile's tokens, new references for the heads that grew, their rescale factors
#pragma unroll
                    for (int k = 0; k < kR; ++k) {
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            float mx = fmaxf(s[4 * k + e], s[4 * k + 2 + e]);
                            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
                            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
                            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
                            if (lane < 4) red[(h0 + 8 * k + 2 * tq + e) * 4 + wq] = mx;
                        }
                    }
                    named_bar_sync<1, kSoftmaxThreads>();
                    if (st < N) {
                        float4 r4 = *reinterpret_cast<const float4 *>(&red[st * 4]);
                        float mt = fmaxf(fmaxf(r4.x, r4.y), fmaxf(r4.z, r4.w));
                        float m_old = m_s[st];
                        float al = 1.f;
                        if (mt > m_old + kTau) {        // also taken when m_old = -inf
                            al = (m_old == -INFINITY) ? 0.f : fast_exp2(m_old - mt);
                            m_s[st] = mt;
                        }
                        alpha_s[st] = al;
                    }
                    named_bar_sync<1, kSoftmaxThreads>();
#pragma unroll
                    for (int k = 0; k < kR; ++k) {
                        const float2 a2 = *reinterpret_cast<const float2 *>(&alpha_s[h0 + 8 * k + 2 * tq]);
                        l[2 * k] *= a2.x; l[2 * k + 1] *= a2.y;
                    }
                }
                uint16_t hiA[kR], loA[kR], hiB[kR], loB[kR];      // two adjacent heads per 16-bit word
#pragma unroll
                for (int k = 0; k < kR; ++k) {
                    const float2 m2 = *reinterpret_cast<const float2 *>(&m_s[h0 + 8 * k + 2 * tq]);
                    const float o0 = kLift - m2.x, o1 = kLift - m2.y;
                    const float a0 = fast_exp2(s[4 * k + 0] + o0), a1 = fast_exp2(s[4 * k + 1] + o1);
                    const float b0 = fast_exp2(s[4 * k + 2] + o0), b1 = fast_exp2(s[4 * k + 3] + o1);
                    l[2 * k] = fmaf(a0, rtsA, fmaf(b0, rtsB, l[2 * k]));
                    l[2 * k + 1] = fmaf(a1, rtsA, fmaf(b1, rtsB, l[2 * k + 1]));
                    // hi = the e4m3 value nearest to the weight, lo = 16 x what is left, e4m3 again
                    split_e4m3_e4m3x16_x2(a0, a1, hiA[k], loA[k]);
                    split_e4m3_e4m3x16_x2(b0, b1, hiB[k], loB[k]);
                }
                // the P.V that read this P buffer (two tiles back) must be done; a rescale of O^T also needs the
                // previous tile's P.V
                if (s_it > 1) {
                    const uint32_t prev = s_it - 2;
                    ok &= mbar_wait(ctx, bar(kBarKvEmpty + prev % kStages), (prev / kStages) & 1, kBarKvEmpty + prev % kStages);
                }
                if (grew && i > 0) {
                    const uint32_t prev = s_it - 1;
                    ok &= mbar_wait(ctx, bar(kBarKvEmpty + prev % kStages), (prev / kStages) & 1, kBarKvEmpty + prev % kStages);
                    tcgen05_fence_after();
#pragma unroll 1
                    for (int c = sw >> 2; c < 8 * N / 16; c += N / 16) {      // the warps of a quadrant share its columns
                        float o[16];
                        const uint32_t addr = tmem_base + lane_addr + L::kColO + c * 16;
                        tmem_ld16(addr, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int k = 0; k < 16; ++k) o[k] *= alpha_s[(c * 16 + k) % N];
                        tmem_st16(addr, o);
                    }
                    tmem_wait_st();
                }
                {
                    // P^T hi / lo, MN-major: the 16 heads of a group are the 16 bytes of a token's row; groups of 16
                    // heads are 1024 B apart, the lo groups follow the hi groups
                    uint8_t *pa = smem + L::kOffP + (s_it & 1) * L::kPBytes + rA * 16 + 2 * tq;
#pragma unroll
                    for (int k = 0; k < kR; ++k) {
                        uint8_t *ph = pa + (h0 >> 4) * 1024 + k * 8, *pl = ph + (N / 16) * 1024;
                        *reinterpret_cast<uint16_t *>(ph) = hiA[k]; *reinterpret_cast<uint16_t *>(ph + 8 * 16) = hiB[k];
                        *reinterpret_cast<uint16_t *>(pl) = loA[k]; *reinterpret_cast<uint16_t *>(pl + 8 * 16) = loB[k];
                    }
                }
                fence_proxy_async();
                tcgen05_fence_before();
                if (st == 0) mark(s_it, 5);
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarPFull + (s_it & 1)));
                ++s_it;
            }
            // ---- row sums: over the 16 tokens of a warp (the eight threads with this tq), then over the four warps
#pragma unroll
            for (int n = 0; n < 2 * kR; ++n) {
                float v = l[n];
                v += __shfl_xor_sync(0xffffffffu, v, 4);
                v += __shfl_xor_sync(0xffffffffu, v, 8);
                v += __shfl_xor_sync(0xffffffffu, v, 16);
                if (lane < 4) red[(h0 + 8 * (n >> 1) + 2 * tq + (n & 1)) * 4 + wq] = v;
            }
            named_bar_sync<1, kSoftmaxThreads>();
            if (st < N) {
                float4 r4 = *reinterpret_cast<const float4 *>(&red[st * 4]);
                float l = (r4.x + r4.y) + (r4.z + r4.w);
                l_s[st] = 1.f / l;
                const int gh = head0 + st;
                if (gh < p.head_end) {
                    float lse = (m_s[st] - kLift + log2f(l)) * kLn2;
                    if (seg.slot < 0) p.lse[(int64_t)seg.request * p.lse_stride_request + gh] = lse;
                    else p.partial_lse[(int64_t)seg.slot * h + (gh - p.head_begin)] = lse;
                }
            }
            named_bar_sync<1, kSoftmaxThreads>();
            // ---- epilogue: O^T block j holds dv = 128 j + TMEM lane, one column per head
            ok &= mbar_wait(ctx, bar(kBarOFull), seg_it & 1, kBarOFull);
            tcgen05_fence_after();
            float *obase;
            int64_t ostride;
            if (seg.slot < 0) {
                obase = p.out + (int64_t)seg.request * p.out_stride_request + (int64_t)head0 * p.out_stride_head;
                ostride = p.out_stride_head;
            } else {
                obase = p.partial_out + ((int64_t)seg.slot * h + (head0 - p.head_begin)) * kDV;
                ostride = kDV;
            }
            const int nvalid = min(N, p.head_end - head0);
            if (((reinterpret_cast<uintptr_t>(obase) | (uintptr_t)(ostride * 4)) & 15) == 0) {
                // Through shared memory and the bulk-copy engine: plain stores of this tile (one 128-byte line per warp
                // instruction, 64 of them per thread) take ~6,000 cycles while the cache streams, 2.5 times this.  The
                // finished request's query operands are dead by now and serve as the staging buffer, [N heads][256 dv]
                // floats, filled and drained twice.
                float *stg = reinterpret_cast<float *>(smem + L::kOffQ + (seg_it & 1) * L::kQBytes);
                static_assert(N * 256 * 4 <= (int)L::kQBytes, "the staging tile must fit a query operand buffer");
#pragma unroll 1
                for (int half = 0; half < 2; ++half) {
#pragma unroll
                    for (int jj = 0; jj < 2; ++jj) {
                        const int j = 2 * half + jj;
                        {
                            const int c = sw >> 2;        // this warp's 16 heads of the block
                            float o[16], o_lo[16];
                            tmem_ld16(tmem_base + lane_addr + L::kColO + j * (2 * N) + c * 16, o);
                            tmem_ld16(tmem_base + lane_addr + L::kColO + j * (2 * N) + N + c * 16, o_lo);
                            tmem_wait_ld();
#pragma unroll
                            for (int k = 0; k < 16; ++k) {
                                const int n = c * 16 + k;
                                stg[n * 256 + jj * 128 + 32 * q4 + lane] = fmaf(o_lo[k], 0.0625f, o[k]) * l_s[n];
                            }
                        }
                    }
                    fence_proxy_async();
                    named_bar_sync<1, kSoftmaxThreads>();
                    if (st < nvalid) {
                        bulk_store(obase + (int64_t)st * ostride + half * 256, smem_u32(stg + st * 256), 1024);
                        bulk_commit_group();
                        bulk_wait_group_read();          // the row has left shared memory
                    }
                    named_bar_sync<1, kSoftmaxThreads>();
                }
            } else {
#pragma unroll 1
                for (int j = 0; j < 4; ++j) {
                    const int dv = 128 * j + 32 * q4 + lane;
                    {
                        const int c = sw >> 2;
                        float o[16], o_lo[16];
                        tmem_ld16(tmem_base + lane_addr + L::kColO + j * (2 * N) + c * 16, o);
                        tmem_ld16(tmem_base + lane_addr + L::kColO + j * (2 * N) + N + c * 16, o_lo);
                        tmem_wait_ld();
#pragma unroll
                        for (int k = 0; k < 16; ++k) {
                            const int n = c * 16 + k;
                            if (n < nvalid) obase[(int64_t)n * ostride + dv] = fmaf(o_lo[k], 0.0625f, o[k]) * l_s[n];
                        }
                    }
                }
            }
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(bar(kBarOEmpty));
                mbar_arrive(bar(kBarQEmpty + (seg_it & 1)));      // the converters may rebuild this operand buffer
            }
            ++seg_it;
        }
    }

    fill_empty_requests(p, worker, head0, N, tid, kThreads);
    if (p.trace != nullptr && tid == 0) p.trace[512 + blockIdx.x] = clock64() - t_start;   // per-CTA cycles

    // ---- teardown
    if (*ctx.abort_flag) {
        // let bulk copies that were already issued land before the CTA's shared memory goes away
        const unsigned long long t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 200000ull) { __nanosleep(1000); }
    }
    tcgen05_fence_before();
    __syncthreads();
    if (warp == 0) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

// ---------------------------------------------------------------- host side
template <int N>
cudaError_t launch_n(const DecodeParams &p, const CUtensorMap &mkv, cudaStream_t stream) {
    const int smem = (int)Layout<N>::kBytes;
    static DeviceOnce once;
    cudaError_t e = once.run([&] { return cudaFuncSetAttribute(decode_umma_fp8_narrow_kernel<N>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem); });
    if (e != cudaSuccess) return e;
    e = launch_dependent(decode_umma_fp8_narrow_kernel<N>, dim3((unsigned)(p.num_workers * p.num_groups)), dim3(Layout<N>::kThreads),
                         (size_t)smem, stream, p, mkv);
    count_launch();
    return e;
}

}  // namespace

cudaError_t launch_decode_umma_fp8_narrow(const DecodeParams &p, cudaStream_t stream) {
    alignas(64) CUtensorMap mkv;
    if (!make_map_4d(&mkv, CU_TENSOR_MAP_DATA_TYPE_UINT8, CU_TENSOR_MAP_SWIZZLE_64B, p.kv_pool, kPage,
                     (uint64_t)(p.num_pool_pages > 0 ? p.num_pool_pages : 1), (uint64_t)kDQK, 64,
                     (uint64_t)kPage * kDQK, 64))
        return cudaErrorInvalidValue;
    switch (p.heads_per_group) {
        case 16: return launch_n<16>(p, mkv, stream);
        case 32: return launch_n<32>(p, mkv, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace splash
