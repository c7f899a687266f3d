// tcgen05 / TMA decode kernel for e4m3 KV (one fp32 scale per token) and NARROW head slices:
// N = 16 or 32 heads per CTA, the shard of a TP / DOP rank whose cache is kept in the paper's
// precision.  The 64-head e4m3 kernel pads such a slice to 64 rows of an MMA and to 64 heads of
// softmax work; here the problem is transposed ("tokens on M"), as in the bf16 kernel's narrow
// path, so that a 16-head slice costs 16-wide MMAs:
//
//     S^T [64 tokens x N heads]  = K_tile [64 x 576]   * (q_hi + q_lo)^T [576 x N]     (M = 64, K = 32)
//     O^T [512 dv    x N heads] += V_tile^T [512 x 64] * (P_hi + P_lo)^T [64 x N]      (4 x M = 128)
//
// The cache bytes go to the tensor cores as stored (kind::f8f6f4); V is the first 512 columns of the
// very K rows in shared memory, read as an MN-major operand.  The two bf16-precision operands are
// split into two 8-bit terms each, exactly as in the 64-head kernel: q = qs_h (hi + lo) with one
// scale per head (e4m3 + e4m3, rebuilt per request by converter warps one request ahead), and
// P = hi + lo (e4m3 + e5m2) with the token scale folded into the weight in the log domain,
//     y = (q . codes) * qs_h * scale_t * softmax_scale * log2(e) + log2(scale_t),   P = 2^(y - m + 4.75),
// the row sum adding P / scale_t.  With the tokens on the TMEM lanes the token scale is one
// number per thread.  A page is 36,864 bytes and the query operands are small, so five stages
// fit: the loop is a ring of dependent latencies and its period is the ring divided by the stages.
//
// Warp roles (352 threads): TMA producer (pages + scale pages, next page pulled into L2), 4 MMA
// issuers (one S^T partial accumulator and one dv block each, ready-driven), 4 softmax / epilogue
// warps (per-head maxima and sums by a warp-shuffle reduce-scatter plus a small exchange), 2 query
// converter warps.  Every wait is bounded; on expiry the CTA records SPLASH_DEVICE_TIMEOUT and leaves
// in order.
#include "splash_fp8.cuh"
#include "splash_pair.cuh"

namespace splash {

namespace {

using namespace umma;

constexpr int kMmaWarps = 4;
constexpr int kNumSoftmaxWarps = 4;
constexpr int kNumConvertWarps = 2;
constexpr int kWarpMma = 1;
constexpr int kWarpSoftmax = kWarpMma + kMmaWarps;          // 5: TMEM lane quadrant = warp & 3
constexpr int kWarpConvert = kWarpSoftmax + kNumSoftmaxWarps;
constexpr int kThreads = (kWarpConvert + kNumConvertWarps) * 32;   // 11 warps = 352 threads
constexpr int kChunks = 9;                         // 576 / 64-element (64 B) chunks
constexpr uint32_t kSlab = 64 * 64;                // one chunk of one page: 64 tokens x 64 B
constexpr uint32_t kStageBytes = kChunks * kSlab;  // 36,864
constexpr uint32_t kScaleBytes = 256;              // 64 fp32 token scales of a page
constexpr int kStages = 5;
constexpr float kTau = 4.0f;                       // lazy rescale threshold, log2 units
constexpr float kLift = 4.75f;                     // weights are stored as 2^(y - m + kLift) <= 2^8.75 = 431 < 448

enum BarrierId {
    kBarKvFull = 0,                    // [kStages]
    kBarKvEmpty = kBarKvFull + kStages,
    kBarQFull = kBarKvEmpty + kStages,
    kBarQEmpty,
    kBarQsRead,                        // the softmax warps have picked up the request's query scales
    kBarSFull,                         // [2]
    kBarSEmpty = kBarSFull + 2,        // [2]
    kBarPFull = kBarSEmpty + 2,
    kBarOFull,
    kBarOEmpty,
    kNumBarriers
};

template <int N>
struct Layout {
    static constexpr uint32_t kQSlab = N * 64;                 // one chunk of the query operand: N heads x 64 B
    static constexpr uint32_t kQBytes = kChunks * kQSlab;      // one term (hi or lo)
    static constexpr uint32_t kPBytes = N * 64;                // one term of P^T: N heads x 64 tokens, one byte each
    static constexpr uint32_t kOffKv = 0;
    static constexpr uint32_t kOffQHi = kOffKv + kStages * kStageBytes;
    static constexpr uint32_t kOffQLo = kOffQHi + kQBytes;
    static constexpr uint32_t kOffPHi = kOffQLo + kQBytes;
    static constexpr uint32_t kOffPLo = kOffPHi + kPBytes;
    static constexpr uint32_t kOffScale = kOffPLo + kPBytes;   // float [kStages][64]
    static constexpr uint32_t kOffQs = kOffScale + kStages * kScaleBytes;   // float [4][N] query scales, by segment & 3
    static constexpr uint32_t kOffRed = kOffQs + 4 * N * 4;    // float [N][4]
    static constexpr uint32_t kOffM = kOffRed + N * 16;        // float [N] running max, log2 domain
    static constexpr uint32_t kOffAlpha = kOffM + N * 4;       // float [N]
    static constexpr uint32_t kOffL = kOffAlpha + N * 4;       // float [N]
    static constexpr uint32_t kOffBar = kOffL + N * 4;
    static constexpr uint32_t kOffMisc = (kOffBar + kNumBarriers * 8 + 15) / 16 * 16;   // u32: tmem base, abort, rescale flags
    static constexpr uint32_t kBytes = kOffMisc + 16;
    static constexpr int kAcc = 4;                             // partial accumulators of S^T = issuers that take part in QK^T
    static constexpr int kSBufs = 2;
    static constexpr uint32_t kColO = 0;                       // 4 dv blocks x N columns
    static constexpr uint32_t kColS = 4 * N;                   // kSBufs x kAcc x N columns
    static_assert(kColS + kSBufs * kAcc * N <= 512, "tensor memory overflow");
    static_assert(kBytes <= 232448, "shared memory overflow");
    static_assert(kOffQHi % 1024 == 0 && kQSlab % 512 == 0 && kOffPHi % 512 == 0 && kPBytes % 512 == 0, "swizzle atoms need aligned windows");
};

// Reduce-scatter over the 32 lanes of a warp (see the bf16 kernel): on return lane L holds, in v[0 .. max(1, N/32)),
// the reduction over all lanes of the entries it owns (N = 32: head L; N = 16: head L >> 1, both lanes of a pair).
template <int CNT, int MASK, bool IS_MAX>
struct ReduceScatter {
    template <int N>
    static __device__ __forceinline__ void run(float (&v)[N], int lane) {
        if constexpr (MASK >= 1) {
            if constexpr (CNT > 1) {
                constexpr int kHalf = CNT / 2;
                const bool upper = (lane & MASK) != 0;
#pragma unroll
                for (int i = 0; i < kHalf; ++i) {
                    float keep = upper ? v[i + kHalf] : v[i];
                    float send = upper ? v[i] : v[i + kHalf];
                    float recv = __shfl_xor_sync(0xffffffffu, send, MASK);
                    v[i] = IS_MAX ? fmaxf(keep, recv) : keep + recv;
                }
                ReduceScatter<kHalf, MASK / 2, IS_MAX>::run(v, lane);
            } else {
                float recv = __shfl_xor_sync(0xffffffffu, v[0], MASK);
                v[0] = IS_MAX ? fmaxf(v[0], recv) : v[0] + recv;
                ReduceScatter<1, MASK / 2, IS_MAX>::run(v, lane);
            }
        }
    }
};

template <int N>
__device__ __forceinline__ int owned_head(int lane) { return N >= 32 ? lane : lane >> 1; }

// ---------------------------------------------------------------- the kernel
template <int N>
__global__ void __launch_bounds__(kThreads, 1)
decode_umma_fp8_narrow_kernel(const DecodeParams p, const __grid_constant__ CUtensorMap tmap_kv) {
    using L = Layout<N>;
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
        for (int s = 0; s < kStages; ++s) { mbar_init(bar(kBarKvFull + s), 1); mbar_init(bar(kBarKvEmpty + s), kMmaWarps); }
        mbar_init(bar(kBarQFull), kNumConvertWarps); mbar_init(bar(kBarQEmpty), L::kAcc);
        mbar_init(bar(kBarQsRead), kNumSoftmaxWarps);
        for (int b = 0; b < L::kSBufs; ++b) { mbar_init(bar(kBarSFull + b), L::kAcc); mbar_init(bar(kBarSEmpty + b), kNumSoftmaxWarps); }
        mbar_init(bar(kBarPFull), kNumSoftmaxWarps);
        mbar_init(bar(kBarOFull), kMmaWarps); mbar_init(bar(kBarOEmpty), kNumSoftmaxWarps);
        misc[1] = 0; misc[2] = 0; misc[3] = 0;
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
    } else if (warp >= kWarpMma && warp < kWarpMma + kMmaWarps) {
        // ===================================================== MMA issuers
        if (lane == 0) {
            const int mw = warp - kWarpMma;          // issuer index: S^T accumulator mw, dv block mw
            constexpr uint32_t kIdescQK = make_idesc_e4m3(64, N, 0);
            // the low-order term of P is e5m2 (the B operand here)
            constexpr uint32_t kIdescPV = make_idesc_e4m3(128, N, 1), kIdescPVLo = make_idesc_e4m3(128, N, 1, 1);
            uint32_t kv_it = 0, s_it = 0, p_it = 0, seg_it = 0;
            bool ok = true;
            // This issuer's share of S^T for the tile with global index kv: steps idx = mw, mw + 4, ... of the
            // 36 (18 K = 32 steps x (q hi, q lo)), into partial accumulator mw.
            auto issue_qk = [&](uint32_t kv, uint32_t sidx) {
                const uint32_t stage = kv % kStages, b = sidx % L::kSBufs;
                if (mw == 0) mark(kv, 2);
                tcgen05_fence_after();
                const uint32_t k0 = sbase + L::kOffKv + stage * kStageBytes;
                const uint32_t d = tmem_base + L::kColS + (b * L::kAcc + mw) * N;
#pragma unroll
                for (int t = 0; t < 36 / L::kAcc; ++t) {
                    const int idx = t * L::kAcc + mw, hl = idx / 18, ks = idx % 18, c = ks >> 1, k = ks & 1;
                    const uint32_t q0 = sbase + (hl ? L::kOffQLo : L::kOffQHi);
                    uint64_t dk = make_desc_sw64(k0 + c * kSlab + k * 32, 16, 512);          // A: 64 tokens x 32
                    uint64_t dq = make_desc_sw64(q0 + c * L::kQSlab + k * 32, 16, 512);      // B: N heads x 32
                    umma_e4m3(d, dk, dq, kIdescQK, t != 0);
                }
                umma_commit(bar(kBarSFull + b));
                if (mw == 0) mark(kv, 3);
            };
            // O^T block mw += V^T block mw (128 dv x 64 tokens) * (P hi + P lo)^T: 2 K = 32 steps x 2 terms
            auto issue_pv = [&](uint32_t stage, bool first_tile) {
                tcgen05_fence_after();
                const uint32_t v0 = sbase + L::kOffKv + stage * kStageBytes + (2 * mw) * kSlab;
#pragma unroll
                for (int hl = 0; hl < 2; ++hl) {
#pragma unroll
                    for (int k = 0; k < 2; ++k) {
                        // A: two 64-element chunks (LBO apart) x 32 tokens (SBO per 8 tokens), MN-major
                        uint64_t da = make_desc_sw64(v0 + k * 2048, kSlab, 512);
                        uint64_t db = make_desc_sw64(sbase + (hl ? L::kOffPLo : L::kOffPHi) + k * 32, 16, 512);
                        umma_e4m3(tmem_base + L::kColO + mw * N, da, db, hl ? kIdescPVLo : kIdescPV, (!first_tile) || (hl | k) != 0);
                    }
                }
            };
            while (ok && it.next(p, seg)) {
                const int ntiles = seg.tile_end - seg.tile_begin;
                ok = mbar_wait(ctx, bar(kBarQFull), seg_it & 1, kBarQFull);
                if (!ok) break;
                // Issue whatever is ready: P.V of tile pv_i (frees a stage) or QK^T of tile qk_i (at most two tiles
                // ahead of the softmax: two S buffers).
                int qk_i = 0, pv_i = 0;
                unsigned long long idle_since = 0;
                uint32_t idle_polls = 0;
                while (pv_i < ntiles) {
                    bool progressed = false;
                    if ((qk_i > pv_i) && mbar_test_wait(bar(kBarPFull), (p_it + pv_i) & 1)) {
                        if (pv_i == 0 && !mbar_wait(ctx, bar(kBarOEmpty), (seg_it & 1) ^ 1, kBarOEmpty)) { ok = false; break; }
                        if (mw == 0) mark(kv_it + pv_i, 6);
                        const uint32_t stage = (kv_it + pv_i) % kStages;
                        issue_pv(stage, pv_i == 0);
                        umma_commit(bar(kBarKvEmpty + stage));   // P.V done: stage free, P buffers free, O^T updated
                        if (pv_i + 1 == ntiles) umma_commit(bar(kBarOFull));
                        if (mw == 0) mark(kv_it + pv_i, 7);
                        ++pv_i;
                        progressed = true;
                    }
                    if (qk_i < ntiles && qk_i < pv_i + 2) {
                        const uint32_t kv = kv_it + qk_i, sidx = s_it + qk_i;
                        if (mbar_test_wait(bar(kBarKvFull + kv % kStages), (kv / kStages) & 1) &&
                            mbar_test_wait(bar(kBarSEmpty + sidx % L::kSBufs), ((sidx / L::kSBufs) & 1) ^ 1)) {
                            issue_qk(kv, sidx);
                            ++qk_i;
                            if (qk_i == ntiles) umma_commit(bar(kBarQEmpty));
                            progressed = true;
                        }
                    }
                    if (progressed) { idle_since = 0; idle_polls = 0; continue; }
                    if ((++idle_polls & 255u) != 0u) continue;
                    if (*ctx.abort_flag) { ok = false; break; }
                    const unsigned long long now = global_timer_ns();
                    if (idle_since == 0) idle_since = now;
                    else if (now - idle_since > kWaitLimitNs) {
                        *ctx.abort_flag = 1;
                        if (atomicCAS(ctx.status, 0, (int)SPLASH_DEVICE_TIMEOUT) == 0) {
                            ctx.status[1] = (int)blockIdx.x; ctx.status[2] = 100 + (qk_i > pv_i ? kBarPFull : kBarKvFull);
                            ctx.status[3] = pv_i;
                        }
                        ok = false; break;
                    }
                }
                kv_it += ntiles; s_it += ntiles; p_it += ntiles;
                ++seg_it;
            }
        }
    } else if (warp >= kWarpConvert) {
        // ===================================================== query converters
        // bf16 query rows -> e4m3 hi + lo operands with one scale per head, 64 / N threads per head.  They run a
        // segment ahead of the softmax warps: the operands of the next request are rebuilt as soon as the last
        // QK^T of the current one has been issued and retired.
        constexpr int kPerHead = 64 / N;               // threads per head: 4 (N = 16) or 2 (N = 32)
        constexpr int kVecs = 72 / kPerHead;           // 8-element vectors per thread
        const int ct = (warp - kWarpConvert) * 32 + lane;   // 0..63
        float *qs_s = reinterpret_cast<float *>(smem + L::kOffQs);
        uint32_t seg_it = 0;
        bool ok = true;
        while (ok && it.next(p, seg)) {
            ok = mbar_wait(ctx, bar(kBarQEmpty), (seg_it & 1) ^ 1, kBarQEmpty);
            if (!ok) break;
            const int hd = ct / kPerHead, part = ct % kPerHead;
            const int gh = head0 + hd;
            const bool live = gh < p.head_end;
            const uint4 *src = reinterpret_cast<const uint4 *>(
                static_cast<const __nv_bfloat16 *>(p.q) + (int64_t)seg.request * p.q_stride_request +
                (int64_t)(live ? gh : p.head_begin) * p.q_stride_head + part * (kVecs * 8));
            float amax = 0.f;
            if (live) {
#pragma unroll 6
                for (int v = 0; v < kVecs; ++v) {
                    uint4 x = __ldg(src + v);
                    const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        amax = fmaxf(amax, fabsf(__uint_as_float(w[k] << 16)));
                        amax = fmaxf(amax, fabsf(__uint_as_float(w[k] & 0xffff0000u)));
                    }
                }
            }
#pragma unroll
            for (int mk = 1; mk < kPerHead; mk <<= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, mk));
            const float qs = amax > 0.f ? amax * (1.0f / 448.0f) : 1.0f;
            const float inv = amax > 0.f ? 448.0f / amax : 1.0f;
            if (part == 0) qs_s[(seg_it & 3) * N + hd] = qs;
#pragma unroll 2
            for (int v = 0; v < kVecs; ++v) {
                uint4 x = live ? __ldg(src + v) : make_uint4(0u, 0u, 0u, 0u);
                const uint32_t w[4] = {x.x, x.y, x.z, x.w};
                uint16_t hi[4], lo[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const float e0 = __uint_as_float(w[k] << 16) * inv, e1 = __uint_as_float(w[k] & 0xffff0000u) * inv;
                    split_e4m3_e4m3_x2(e0, e1, hi[k], lo[k]);
                }
                const uint32_t d = (uint32_t)(part * (kVecs * 8) + v * 8);
                const uint32_t off = (d >> 6) * L::kQSlab + sw64((uint32_t)hd, d & 63);
                *reinterpret_cast<uint2 *>(smem + L::kOffQHi + off) =
                    make_uint2((uint32_t)hi[0] | ((uint32_t)hi[1] << 16), (uint32_t)hi[2] | ((uint32_t)hi[3] << 16));
                *reinterpret_cast<uint2 *>(smem + L::kOffQLo + off) =
                    make_uint2((uint32_t)lo[0] | ((uint32_t)lo[1] << 16), (uint32_t)lo[2] | ((uint32_t)lo[3] << 16));
            }
            fence_proxy_async();
            __syncwarp();
            // The softmax warps wait on QFull by phase parity, so QFull must never complete two phases ahead of
            // them: hold this request's arrival until they have entered the previous one.
            if (lane == 0) {
                if (seg_it > 0) ok = mbar_wait(ctx, bar(kBarQsRead), (seg_it - 1) & 1, kBarQsRead);
                mbar_arrive(bar(kBarQFull));
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            ++seg_it;
        }
    } else {
        // ===================================================== softmax + epilogue warps
        const int q4 = warp & 3;                       // TMEM lane quadrant of this warp
        const int sw = warp - kWarpSoftmax;            // softmax warp 0..3
        const int st = sw * 32 + lane;                 // 0..127
        const int row = 16 * q4 + lane;                // token row of the S^T tile (lanes < 16)
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
            ok &= mbar_wait(ctx, bar(kBarQFull), seg_it & 1, kBarQFull);
            const float *qs_s = qs_all + (seg_it & 3) * N;
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarQsRead));
            if (st < N) m_s[st] = -INFINITY;
            float l_own = 0.f;            // running sum of the head this lane owns (this warp's 16 tokens)
            softmax_bar_sync();
            const int first_page = seg.lo / kPage;
            const int ntiles = seg.tile_end - seg.tile_begin;
            for (int i = 0; i < ntiles; ++i) {
                const TileGeom g = tile_geom(seg.lo, seg.hi, (first_page + seg.tile_begin + i) * kPage);
                const bool valid = lane < 16 && row >= g.r_lo && row < g.r_hi;
                const uint32_t b = s_it % L::kSBufs, stage = s_it % kStages;
                ok &= mbar_wait(ctx, bar(kBarSFull + b), (s_it / L::kSBufs) & 1, kBarSFull + b);
                if (st == 0) mark(s_it, 4);
                // the scale page rode on the stage's own barrier, long complete by now
                ok &= mbar_wait(ctx, bar(kBarKvFull + stage), (s_it / kStages) & 1, kBarKvFull + stage);
                tcgen05_fence_after();
                float s[N];
                {
                    const uint32_t sb = tmem_base + lane_addr + L::kColS + b * (L::kAcc * N);
#pragma unroll
                    for (int c = 0; c < N / 16; ++c)
                        tmem_ld16(sb + c * 16, *reinterpret_cast<float(*)[16]>(&s[c * 16]));
#pragma unroll
                    for (int a = 1; a < L::kAcc; ++a) {
                        float part[N];
#pragma unroll
                        for (int c = 0; c < N / 16; ++c)
                            tmem_ld16(sb + a * N + c * 16, *reinterpret_cast<float(*)[16]>(&part[c * 16]));
                        tmem_wait_ld();
#pragma unroll
                        for (int n = 0; n < N; ++n) s[n] += part[n];
                    }
                }
                tmem_wait_ld();
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarSEmpty + b));
                // this thread's token: its scale, log2 of it for the weight, its reciprocal for the row sums
                const float ts = valid ? scale_s[stage * 64 + g.tok0 + row] : 1.0f;
                const float lg = fast_log2(ts), rts = fast_rcp(ts), tsl = ts * scale_log2;
                float mx[N];
#pragma unroll
                for (int n = 0; n < N; ++n) {
                    s[n] = valid ? fmaf(s[n] * qs_s[n], tsl, lg) : -INFINITY;      // log2-domain logit + log2(token scale)
                    mx[n] = s[n];
                }
                ReduceScatter<N, 16, true>::run(mx, lane);
                if (N >= 32 || (lane & 1) == 0) red[owned_head<N>(lane) * 4 + sw] = mx[0];
                if (st == 0) misc[2 + (i & 1)] = 0;      // this tile's "some maximum grew" flag
                softmax_bar_sync();
                if (st < N) {
                    float4 r4 = *reinterpret_cast<const float4 *>(&red[st * 4]);
                    float mt = fmaxf(fmaxf(r4.x, r4.y), fmaxf(r4.z, r4.w));
                    float m_old = m_s[st];
                    float al = 1.f;
                    if (mt > m_old + kTau) {        // also taken when m_old = -inf
                        al = (m_old == -INFINITY) ? 0.f : fast_exp2(m_old - mt);
                        m_s[st] = mt;
                        misc[2 + (i & 1)] = 1;
                    }
                    alpha_s[st] = al;
                }
                softmax_bar_sync();
                const bool rescale = misc[2 + (i & 1)] != 0;
                if (rescale) l_own *= alpha_s[owned_head<N>(lane)];
#pragma unroll
                for (int n = 0; n < N; ++n) { s[n] = fast_exp2(s[n] - m_s[n] + kLift); mx[n] = s[n] * rts; }
                ReduceScatter<N, 16, false>::run(mx, lane);      // per-head sums of P / scale_t over this warp's tokens
                l_own += mx[0];
                // P.V of the previous tile must be done with the P buffers and with O^T
                if (s_it > 0) {
                    const uint32_t prev = s_it - 1;
                    ok &= mbar_wait(ctx, bar(kBarKvEmpty + prev % kStages), (prev / kStages) & 1, kBarKvEmpty + prev % kStages);
                }
                tcgen05_fence_after();
                if (rescale && i > 0) {
#pragma unroll 1
                    for (int c = 0; c < 4 * N / 16; ++c) {
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
                if (lane < 16) {
                    // P^T hi / lo as K-major, 64-byte-swizzled B operands: row = head, byte = token.
                    // hi = the e4m3 value nearest to the weight, lo = what is left, kept as e5m2.
                    uint8_t *ph = smem + L::kOffPHi, *pl = smem + L::kOffPLo;
#pragma unroll
                    for (int n = 0; n < N; n += 2) {
                        uint16_t hi2, lo2;
                        split_e4m3_e5m2_x2(s[n], s[n + 1], hi2, lo2);
                        const uint32_t off = sw64((uint32_t)n, (uint32_t)row);     // head n + 1: same swizzle phase, 64 B on
                        ph[off] = (uint8_t)(hi2 & 0xffu); ph[off + 64] = (uint8_t)(hi2 >> 8);
                        pl[off] = (uint8_t)(lo2 & 0xffu); pl[off + 64] = (uint8_t)(lo2 >> 8);
                    }
                }
                fence_proxy_async();
                tcgen05_fence_before();
                if (st == 0) mark(s_it, 5);
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarPFull));
                ++s_it;
            }
            // ---- row sums over all four warps' partial sums
            if (N >= 32 || (lane & 1) == 0) red[owned_head<N>(lane) * 4 + sw] = l_own;
            softmax_bar_sync();
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
            softmax_bar_sync();
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
#pragma unroll 1
            for (int j = 0; j < 4; ++j) {
                const int dv = 128 * j + 32 * q4 + lane;
#pragma unroll
                for (int c = 0; c < N / 16; ++c) {
                    float o[16];
                    tmem_ld16(tmem_base + lane_addr + L::kColO + j * N + c * 16, o);
                    tmem_wait_ld();
#pragma unroll
                    for (int k = 0; k < 16; ++k) {
                        const int n = c * 16 + k;
                        if (n < nvalid) obase[(int64_t)n * ostride + dv] = o[k] * l_s[n];
                    }
                }
            }
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarOEmpty));
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
    e = launch_dependent(decode_umma_fp8_narrow_kernel<N>, dim3((unsigned)(p.num_workers * p.num_groups)), dim3(kThreads),
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
