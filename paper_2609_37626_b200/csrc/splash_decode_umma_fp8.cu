// tcgen05 / TMA decode kernel for e4m3 KV with one fp32 scale per token (sm_100a).
//
// Same structure as the bf16 kernel's 64-head path -- one CTA per (KV worker, group of 64
// heads), S = Q K^T with the heads on M, O^T += V^T P^T with dv on M, four MMA issuer
// warps, fragment-layout softmax -- but the cache bytes go to the tensor cores AS THEY ARE
// (kind::f8f6f4, K = 32 per MMA): a page is 36,864 B, four stages fit, nothing is converted
// in shared memory.  bf16 x e4m3 is not an MMA type pair, so the two bf16-precision operands
// are each split into two e4m3 terms that accumulate into the same fp32 accumulator:
//
//   q_h   = qs_h * (hi + lo),  qs_h = max|q_h| / 448, hi = e4m3(q/qs), lo = e4m3(q/qs - hi)
//   P_ht  = u_hi + u_lo,       u = 2^(y - m + 2.75) with y = log2-domain logit + log2(scale_t)
//
// i.e. the per-token scale is folded into the softmax weight in the log domain, so the
// weights of a tile are automatically normalised (u <= 2^8.75 with the lazy-rescale threshold
// of 2^6) and sit in e4m3's range; the row sum adds u / scale_t = 2^(x - m + 2.75).
// Four e4m3 products per bf16-precision product pair cost the tensor pipe the same time as
// the bf16 kernel (fp8 MMAs run at twice the rate), which is why the roofline of this
// workload is taken at the bf16 rate.
#include "splash_fp8.cuh"
#include "splash_pair.cuh"

namespace splash {

namespace {

using namespace umma;

constexpr int kThreads = 544;                      // 17 warps: producer, 2 QK issuers, 2 PV issuers, 8 softmax, 4 query converters
constexpr int kNumConvertWarps = 4;
constexpr int kQkWarps = 2;                        // = partial accumulators of S
constexpr int kPvWarps = 2;                        // each owns two of the four dv blocks of O^T
constexpr int kNumSoftmaxThreads = 256;            // two warps per TMEM lane quadrant, 32 tokens of a tile each
constexpr int kNumSoftmaxWarps = kNumSoftmaxThreads / 32;   // barriers fed by the softmax role count one arrival per warp
constexpr int kN = 64;                             // heads per CTA
constexpr int kChunks = 9;                         // 576 / 64-element (64 B) chunks
constexpr uint32_t kSlab = 64 * 64;                // one chunk of one page: 64 tokens x 64 B
constexpr uint32_t kStageBytes = kChunks * kSlab;  // 36,864
constexpr uint32_t kScaleBytes = 256;              // 64 fp32 token scales of a page
constexpr int kStages = 3;
// lazy rescale threshold, log2 units: with 64 heads per CTA every move of any head's reference costs the tile a pass over
// O^T (at 2^4 the long-context and the many-request timings were 7-9 % slower); weights are stored as
// 2^(y - m + kLift) <= 2^8.75 = 431 < 448
constexpr float kTau = 6.0f;
constexpr float kLift = 2.75f;

enum BarrierId {
    kBarKvFull = 0,
    kBarKvEmpty = kBarKvFull + kStages,
    kBarQFull = kBarKvEmpty + kStages,
    kBarQEmpty,
    kBarQsRead,                   // the softmax warps have picked up the request's query scales
    kBarSFull,                    // [2]
    kBarSEmpty = kBarSFull + 2,   // [2]
    kBarPFull = kBarSEmpty + 2,   // [2]: one per P buffer (the softmax warps may run two tiles ahead of a P.V issuer; with
                                  // a single barrier two phases could complete between two of its polls)
    kBarOFull = kBarPFull + 2,
    kBarOEmpty,
    kNumBarriers
};

// shared memory map (all swizzled regions 512-byte aligned: 8 rows x 64 B atoms)
constexpr uint32_t kOffKv = 0;
constexpr uint32_t kOffQHi = kOffKv + kStages * kStageBytes;
constexpr uint32_t kOffQLo = kOffQHi + kN * kDQK;
constexpr uint32_t kOffPHi = kOffQLo + kN * kDQK;
constexpr uint32_t kOffPLo = kOffPHi + 2 * kN * 64;         // P hi and P lo are double buffered (tile parity)
constexpr uint32_t kOffScale = kOffPLo + 2 * kN * 64;      // float [kStages][64]
constexpr uint32_t kOffQs = kOffScale + kStages * kScaleBytes;   // float [4][64] query scales, by segment & 3
constexpr uint32_t kOffAlpha = kOffQs + 4 * kN * 4;         // (four deep: the converters run ahead of the softmax warps)
constexpr uint32_t kOffL = kOffAlpha + kN * 4;
constexpr uint32_t kOffTok = kOffL + kN * 4;                // float2 [64]: (log2 scale_t, 1 / scale_t) of the tile
constexpr uint32_t kOffXch = kOffTok + 64 * 8;              // float [64][2]: per-head exchange between token halves
constexpr uint32_t kOffBar = kOffXch + kN * 8;
constexpr uint32_t kOffMisc = (kOffBar + kNumBarriers * 8 + 15) / 16 * 16;
constexpr uint32_t kSmemBytes = kOffMisc + 32;
static_assert(kSmemBytes <= 232448, "shared memory overflow");
static_assert(kOffQHi % 512 == 0 && kOffQLo % 512 == 0 && kOffPHi % 512 == 0 && kOffPLo % 512 == 0, "alignment");
// tensor memory: O^T 4 blocks x 64 columns, then 2 S buffers x 2 partial accumulators x 64 columns
constexpr uint32_t kColO = 0, kColS = 256;

__global__ void __launch_bounds__(kThreads, 1)
decode_umma_fp8_kernel(const DecodeParams p, const __grid_constant__ CUtensorMap tmap_kv) {
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int worker = blockIdx.x / p.num_groups;
    const int group = blockIdx.x % p.num_groups;
    const int head0 = p.head_begin + group * kN;
    const int h = p.head_end - p.head_begin;

    volatile uint32_t *misc = reinterpret_cast<volatile uint32_t *>(smem + kOffMisc);
    Ctx ctx{misc + 1, p.status};
    auto bar = [&](int id) -> uint32_t { return sbase + kOffBar + 8u * (uint32_t)id; };

    if ((sbase & 1023u) != 0) {
        if (tid == 0 && atomicCAS(p.status, 0, (int)SPLASH_CUDA_ERROR) == 0) { p.status[1] = (int)blockIdx.x; p.status[2] = -100; }
        return;
    }
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(bar(kBarKvFull + s), 1); mbar_init(bar(kBarKvEmpty + s), kPvWarps); }
        mbar_init(bar(kBarQFull), kNumConvertWarps); mbar_init(bar(kBarQEmpty), kQkWarps);
        mbar_init(bar(kBarQsRead), kNumSoftmaxWarps);
        for (int b = 0; b < 2; ++b) { mbar_init(bar(kBarSFull + b), kQkWarps); mbar_init(bar(kBarSEmpty + b), kNumSoftmaxWarps); }
        for (int b = 0; b < 2; ++b) mbar_init(bar(kBarPFull + b), kNumSoftmaxWarps);
        mbar_init(bar(kBarOFull), kPvWarps); mbar_init(bar(kBarOEmpty), kNumSoftmaxWarps);
        misc[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sbase + kOffMisc), "r"(512u) : "memory");
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
                // the next page (when its table entry is among the 32 this warp holds): pulled into L2 now, so that its
                // TMA load, which can only start when a stage comes free, finds it there
                const int page_ahead = __shfl_sync(0xffffffffu, entry, (rel + 1) & 31);
                const bool ahead_ok = (rel & 31) + 1 < 32 && tile + 1 < seg.tile_end;
                const TileGeom g = tile_geom(seg.lo, seg.hi, (first_page + tile) * kPage);
                const uint32_t stage = kv_it % kStages, ph = (kv_it / kStages) & 1;
                // a page id outside the pool reads as zeros through the tensor map; its
                // scale page is not fetched (plain addresses are not bounds-checked)
                const bool in_pool = page >= 0 && page < p.num_pool_pages;
                if (lane == 0) {
                    ok = mbar_wait(ctx, bar(kBarKvEmpty + stage), ph ^ 1, kBarKvEmpty + stage);
                    mark(kv_it, 0);
                    if (ok && !in_pool) {      // the page reads as zeros; give its tokens the scale 1
                        float *sc1 = reinterpret_cast<float *>(smem + kOffScale + stage * kScaleBytes);
                        for (int t = 0; t < kPage; ++t) sc1[t] = 1.0f;
                    }
                    if (ok && !g.both) {
                        mbar_expect_tx(bar(kBarKvFull + stage), kStageBytes + (in_pool ? kScaleBytes : 0u));
                        tma_load_4d(sbase + kOffKv + stage * kStageBytes, &tmap_kv, bar(kBarKvFull + stage), 0, g.tok0, 0, page);
                        if (in_pool)
                            bulk_load(sbase + kOffScale + stage * kScaleBytes, p.kv_scales + (int64_t)page * kPage,
                                      kScaleBytes, bar(kBarKvFull + stage));
                        if (ahead_ok && page_ahead >= 0 && page_ahead < p.num_pool_pages)
                            bulk_prefetch_l2(static_cast<const uint8_t *>(p.kv_pool) + (size_t)page_ahead * (kPage * kDQK), kStageBytes);
                        mark(kv_it, 1);
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (ok && g.both) {
                    // a range cut at both ends inside this page: the warp writes the box itself, zeros outside the
                    // range (the scale page still comes by bulk copy; the softmax warps mask the scales themselves)
                    const uint8_t *src = in_pool ? static_cast<const uint8_t *>(p.kv_pool) + (size_t)page * (kPage * kDQK) : nullptr;
                    fill_rows_by_hand<64>(smem + kOffKv + stage * kStageBytes, kSlab, kPage, src, g.tok0, g.a, g.b, 0, 0, 9, lane);
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) {
                        if (in_pool) {
                            mbar_expect_tx(bar(kBarKvFull + stage), kScaleBytes);
                            bulk_load(sbase + kOffScale + stage * kScaleBytes, p.kv_scales + (int64_t)page * kPage,
                                      kScaleBytes, bar(kBarKvFull + stage));
                        } else {
                            mbar_arrive(bar(kBarKvFull + stage));
                        }
                    }
                }
                ++kv_it;
            }
        }
    } else if (warp <= kQkWarps) {
        // ===================================================== QK^T issuers: S = (q hi + q lo) K^T
        if (lane == 0) {
            const int a = warp - 1;                  // partial accumulator a
            constexpr uint32_t kIdescQK = make_idesc_e4m3(64, 64, 0);
            uint32_t kv = 0, seg_it = 0;
            bool ok = true;
            while (ok && it.next(p, seg)) {
                const int ntiles = seg.tile_end - seg.tile_begin;
                ok = mbar_wait(ctx, bar(kBarQFull), seg_it & 1, kBarQFull);
                for (int i = 0; ok && i < ntiles; ++i, ++kv) {
                    const uint32_t stage = kv % kStages, b = kv & 1;
                    ok = mbar_wait(ctx, bar(kBarKvFull + stage), (kv / kStages) & 1, kBarKvFull + stage) &&
                         mbar_wait(ctx, bar(kBarSEmpty + b), ((kv >> 1) & 1) ^ 1, kBarSEmpty + b);
                    if (!ok) break;
                    if (a == 0) mark(kv, 2);
                    tcgen05_fence_after();
                    const uint32_t k0 = sbase + kOffKv + stage * kStageBytes;
                    const uint32_t d = tmem_base + kColS + (b * kQkWarps + a) * kN;
                    // 18 K = 32 steps x (q hi, q lo) = 36 MMAs per tile; this issuer takes every second
#pragma unroll
                    for (int t = 0; t < 36 / kQkWarps; ++t) {
                        const int idx = t * kQkWarps + a, hl = idx / 18, ks = idx % 18, c = ks >> 1, k = ks & 1;
                        const uint32_t q0 = sbase + (hl ? kOffQLo : kOffQHi);
                        uint64_t dq = make_desc_sw64(q0 + c * kSlab + k * 32, 16, 512);     // A: 64 heads x 32
                        uint64_t dk = make_desc_sw64(k0 + c * kSlab + k * 32, 16, 512);     // B: 64 tokens x 32
                        umma_e4m3(d, dq, dk, kIdescQK, t != 0);
                    }
                    umma_commit(bar(kBarSFull + b));
                    if (a == 0) mark(kv, 3);
                }
                if (ok) umma_commit(bar(kBarQEmpty));
                ++seg_it;
            }
        }
    } else if (warp <= kQkWarps + kPvWarps) {
        // ===================================================== P.V issuers: O^T += V^T (P hi + P lo)^T
        if (lane == 0) {
            const int pj = warp - 1 - kQkWarps;      // dv blocks 2 pj and 2 pj + 1
            // the low-order term of P is stored as e5m2: residuals of weights that fall into e4m3's
            // subnormal range (the long tail of a long context) keep three significant bits there
            constexpr uint32_t kIdescPV = make_idesc_e4m3(128, 64, 1), kIdescPVLo = make_idesc_e4m3(128, 64, 1, 1);
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
                    const uint32_t v0 = sbase + kOffKv + stage * kStageBytes;
#pragma unroll
                    for (int hl = 0; hl < 2; ++hl) {
#pragma unroll
                        for (int k = 0; k < 2; ++k) {
#pragma unroll
                            for (int jj = 0; jj < 2; ++jj) {
                                const int j = 2 * pj + jj;
                                // A: two 64-element chunks (LBO apart) x 32 tokens (SBO per 8 tokens), MN-major
                                uint64_t da = make_desc_sw64(v0 + (2 * j) * kSlab + k * 2048, kSlab, 512);
                                uint64_t db = make_desc_sw64(sbase + (hl ? kOffPLo : kOffPHi) + (kv & 1) * (kN * 64) + k * 32, 16, 512);
                                umma_e4m3(tmem_base + kColO + j * kN, da, db, hl ? kIdescPVLo : kIdescPV, (i != 0) || (hl | k) != 0);
                            }
                        }
                    }
                    umma_commit(bar(kBarKvEmpty + stage));   // P.V done: stage free, P buffers free, O^T updated
                    if (i + 1 == ntiles) umma_commit(bar(kBarOFull));
                    if (pj == 0) mark(kv, 7);
                }
                ++seg_it;
            }
        }
    } else if (warp >= 1 + kQkWarps + kPvWarps + kNumSoftmaxWarps) {
        // ===================================================== query converters
        // bf16 query rows -> e4m3 hi + lo operands with one scale per head, two threads per head.
        // They run a segment ahead of the softmax warps: the operands of the next request are
        // rebuilt as soon as the last QK^T of the current one has been issued and retired.
        const int ct = (warp - (1 + kQkWarps + kPvWarps + kNumSoftmaxWarps)) * 32 + lane;   // 0..127
        float *qs_s = reinterpret_cast<float *>(smem + kOffQs);
        uint32_t seg_it = 0;
        bool ok = true;
        while (ok && it.next(p, seg)) {
            ok = mbar_wait(ctx, bar(kBarQEmpty), (seg_it & 1) ^ 1, kBarQEmpty);
            if (!ok) break;
            {
                const int hd = ct >> 1, part = ct & 1;
                const int gh = head0 + hd;
                const bool live = gh < p.head_end;
                const uint4 *src = reinterpret_cast<const uint4 *>(
                    static_cast<const __nv_bfloat16 *>(p.q) + (int64_t)seg.request * p.q_stride_request +
                    (int64_t)(live ? gh : p.head_begin) * p.q_stride_head + part * 288);
                float amax = 0.f;
                if (live) {
#pragma unroll 6
                    for (int v = 0; v < 36; ++v) {
                        uint4 x = __ldg(src + v);
                        const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            amax = fmaxf(amax, fabsf(__uint_as_float(w[k] << 16)));
                            amax = fmaxf(amax, fabsf(__uint_as_float(w[k] & 0xffff0000u)));
                        }
                    }
                }
                amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
                const float qs = amax > 0.f ? amax * (1.0f / 448.0f) : 1.0f;
                const float inv = amax > 0.f ? 448.0f / amax : 1.0f;
                if (part == 0) qs_s[(seg_it & 3) * kN + hd] = qs;
#pragma unroll 2
                for (int v = 0; v < 36; ++v) {
                    uint4 x = live ? __ldg(src + v) : make_uint4(0u, 0u, 0u, 0u);
                    const uint32_t w[4] = {x.x, x.y, x.z, x.w};
                    uint16_t hi[4], lo[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const float e0 = __uint_as_float(w[k] << 16) * inv, e1 = __uint_as_float(w[k] & 0xffff0000u) * inv;
                        split_e4m3_e4m3_x2(e0, e1, hi[k], lo[k]);
                    }
                    const uint32_t d = (uint32_t)(part * 288 + v * 8);
                    const uint32_t off = (d >> 6) * kSlab + sw64((uint32_t)hd, d & 63);
                    *reinterpret_cast<uint2 *>(smem + kOffQHi + off) =
                        make_uint2((uint32_t)hi[0] | ((uint32_t)hi[1] << 16), (uint32_t)hi[2] | ((uint32_t)hi[3] << 16));
                    *reinterpret_cast<uint2 *>(smem + kOffQLo + off) =
                        make_uint2((uint32_t)lo[0] | ((uint32_t)lo[1] << 16), (uint32_t)lo[2] | ((uint32_t)lo[3] << 16));
                }
                fence_proxy_async();
                __syncwarp();
                // The softmax warps wait on QFull by phase parity, so QFull must never complete two
                // phases ahead of them: hold this request's arrival until they have entered the previous one.
                if (lane == 0) {
                    if (seg_it > 0) ok = mbar_wait(ctx, bar(kBarQsRead), (seg_it - 1) & 1, kBarQsRead);
                    mbar_arrive(bar(kBarQFull));
                }
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            }
            ++seg_it;
        }
    } else {
        // ===================================================== softmax + epilogue warps
        const int sw = warp - 1 - kQkWarps - kPvWarps;  // 0..7
        const int q4 = warp & 3;                       // TMEM lane quadrant of this warp
        const int hf = sw >> 2;                        // which 32 tokens of a tile this warp handles
        const int st = sw * 32 + lane;                 // 0..255
        const uint32_t lane_addr = (uint32_t)(32 * q4) << 16;
        const int hA = 16 * q4 + (lane >> 2);          // this thread's heads: hA and hA + 8
        const int tq = lane & 3;                       // its tokens: 32 hf + 8k + 2 tq + {0, 1}, k = 0..3
        float *qs_s = reinterpret_cast<float *>(smem + kOffQs);
        float *alpha_s = reinterpret_cast<float *>(smem + kOffAlpha);
        float *l_s = reinterpret_cast<float *>(smem + kOffL);
        float *xch = reinterpret_cast<float *>(smem + kOffXch);
        float2 *tok = reinterpret_cast<float2 *>(smem + kOffTok);
        const float *scale_s = reinterpret_cast<const float *>(smem + kOffScale);
        const float scale_log2 = p.softmax_scale * kLog2e;
        uint32_t s_it = 0, seg_it = 0;
        // A failed (timed-out) wait only clears `ok`; the role keeps walking its tiles so that every
        // thread still meets the named barriers -- once the CTA aborts, waits return at once.
        bool ok = true;
        while (it.next(p, seg)) {
            // the converter warps have written this segment's query operands and scales
            ok &= mbar_wait(ctx, bar(kBarQFull), seg_it & 1, kBarQFull);
            const float cqA = scale_log2 * qs_s[(seg_it & 3) * kN + hA], cqB = scale_log2 * qs_s[(seg_it & 3) * kN + hA + 8];
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarQsRead));
            float mA = -INFINITY, mB = -INFINITY, lA = 0.f, lB = 0.f;
            const int first_page = seg.lo / kPage;
            const int ntiles = seg.tile_end - seg.tile_begin;
            for (int i = 0; i < ntiles; ++i) {
                const TileGeom g = tile_geom(seg.lo, seg.hi, (first_page + seg.tile_begin + i) * kPage);
                const uint32_t stage = s_it % kStages, b = s_it & 1;
                ok &= mbar_wait(ctx, bar(kBarSFull + b), (s_it >> 1) & 1, kBarSFull + b);
                if (st == 0) mark(s_it, 4);
                // the scale page rode on the stage's own barrier, long complete by now
                ok &= mbar_wait(ctx, bar(kBarKvFull + stage), (s_it / kStages) & 1, kBarKvFull + stage);
                tcgen05_fence_after();
                float s[16];
                {
                    float part[16];
                    const uint32_t sb = tmem_base + lane_addr + kColS + (b * kQkWarps) * kN + 32 * hf;
                    tmem_ld_16x256b_x4(sb, s);
                    tmem_ld_16x256b_x4(sb + kN, part);
                    tmem_wait_ld();
#pragma unroll
                    for (int n = 0; n < 16; ++n) s[n] += part[n];
                }
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarSEmpty + b));
                // per-token table of this tile, one token per thread: (log2 scale_t, 1 / scale_t)
                const float *sc = scale_s + stage * 64 + g.tok0;
                if (st < 64) {
                    const bool v = st >= g.r_lo && st < g.r_hi;
                    const float ts = v ? sc[st] : 1.0f;
                    tok[st] = make_float2(fast_log2(ts), fast_rcp(ts));
                }
                named_bar_sync<1, kNumSoftmaxThreads>();
                // y = log2-domain logit + log2(token scale)
                float mtA = -INFINITY, mtB = -INFINITY;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int r0 = 32 * hf + 8 * k + 2 * tq;
                    const float4 t2 = *reinterpret_cast<const float4 *>(&tok[r0]);     // (lg, rts) of r0 and r0 + 1
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int r = r0 + e;
                        const bool v = r >= g.r_lo && r < g.r_hi;
                        const float ts = v ? sc[r] : 1.0f;
                        const float lg = e ? t2.z : t2.x;
                        const float yA = v ? fmaf(s[4 * k + e], cqA * ts, lg) : -INFINITY;
                        const float yB = v ? fmaf(s[4 * k + 2 + e], cqB * ts, lg) : -INFINITY;
                        s[4 * k + e] = yA; s[4 * k + 2 + e] = yB;
                        mtA = fmaxf(mtA, yA); mtB = fmaxf(mtB, yB);
                    }
                }
                mtA = fmaxf(mtA, __shfl_xor_sync(0xffffffffu, mtA, 1)); mtB = fmaxf(mtB, __shfl_xor_sync(0xffffffffu, mtB, 1));
                mtA = fmaxf(mtA, __shfl_xor_sync(0xffffffffu, mtA, 2)); mtB = fmaxf(mtB, __shfl_xor_sync(0xffffffffu, mtB, 2));
                // combine with the warp that holds the other 32 tokens of these heads
                if (tq == 0) { xch[2 * hA + hf] = mtA; xch[2 * (hA + 8) + hf] = mtB; }
                named_bar_sync_dyn<64>(2 + q4);
                {
                    const float2 xa = *reinterpret_cast<const float2 *>(&xch[2 * hA]);
                    const float2 xb = *reinterpret_cast<const float2 *>(&xch[2 * (hA + 8)]);
                    mtA = fmaxf(xa.x, xa.y); mtB = fmaxf(xb.x, xb.y);
                }
                // all eight threads of a head take the same decision from the same numbers
                bool grew = false;
                float alA = 1.f, alB = 1.f;
                if (mtA > mA + kTau) { alA = (mA == -INFINITY) ? 0.f : fast_exp2(mA - mtA); mA = mtA; lA *= alA; grew = true; }
                if (mtB > mB + kTau) { alB = (mB == -INFINITY) ? 0.f : fast_exp2(mB - mtB); mB = mtB; lB *= alB; grew = true; }
                if (tq == 0 && hf == 0) { alpha_s[hA] = alA; alpha_s[hA + 8] = alB; }
                const float offA = kLift - mA, offB = kLift - mB;
                uint16_t phiA[4], ploA[4], phiB[4], ploB[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const float4 t2 = *reinterpret_cast<const float4 *>(&tok[32 * hf + 8 * k + 2 * tq]);
                    const float a0 = fast_exp2(s[4 * k + 0] + offA), a1 = fast_exp2(s[4 * k + 1] + offA);
                    const float b0 = fast_exp2(s[4 * k + 2] + offB), b1 = fast_exp2(s[4 * k + 3] + offB);
                    lA = fmaf(a0, t2.y, lA); lA = fmaf(a1, t2.w, lA);
                    lB = fmaf(b0, t2.y, lB); lB = fmaf(b1, t2.w, lB);
                    // hi = the e4m3 value nearest to the weight, lo = what is left, kept as e5m2
                    split_e4m3_e5m2_x2(a0, a1, phiA[k], ploA[k]);
                    split_e4m3_e5m2_x2(b0, b1, phiB[k], ploB[k]);
                }
                const bool rescale = named_bar_or<1, kNumSoftmaxThreads>(grew);
                // the P.V that read this P buffer (two tiles back) must be done; a rescale of O^T also
                // needs the previous tile's P.V
                if (s_it > 1) {
                    const uint32_t prev = s_it - 2;
                    ok &= mbar_wait(ctx, bar(kBarKvEmpty + prev % kStages), (prev / kStages) & 1, kBarKvEmpty + prev % kStages);
                }
                if (rescale && i > 0) {
                    const uint32_t prev = s_it - 1;
                    ok &= mbar_wait(ctx, bar(kBarKvEmpty + prev % kStages), (prev / kStages) & 1, kBarKvEmpty + prev % kStages);
                }
                tcgen05_fence_after();
                if (rescale && i > 0) {
                    // this warp rescales columns [128 hf, 128 hf + 128) of its quadrant's O^T lanes
#pragma unroll 1
                    for (int c = 0; c < 8; ++c) {
                        float o[16];
                        const uint32_t addr = tmem_base + lane_addr + kColO + 128 * hf + c * 16;
                        tmem_ld16(addr, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int k = 0; k < 16; ++k) o[k] *= alpha_s[(c * 16 + k) % kN];
                        tmem_st16(addr, o);
                    }
                    tmem_wait_st();
                }
                {
                    // P hi / lo as K-major, 64-byte-swizzled B operands: row = head, byte = token
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint32_t offA_ = (s_it & 1) * (kN * 64) + sw64((uint32_t)hA, (uint32_t)(32 * hf + 8 * k + 2 * tq));
                        const uint32_t offB_ = offA_ + 8 * 64;           // head hA + 8: same swizzle phase
                        *reinterpret_cast<uint16_t *>(smem + kOffPHi + offA_) = phiA[k];
                        *reinterpret_cast<uint16_t *>(smem + kOffPLo + offA_) = ploA[k];
                        *reinterpret_cast<uint16_t *>(smem + kOffPHi + offB_) = phiB[k];
                        *reinterpret_cast<uint16_t *>(smem + kOffPLo + offB_) = ploB[k];
                    }
                }
                fence_proxy_async();
                tcgen05_fence_before();
                if (st == 0) mark(s_it, 5);
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarPFull + (s_it & 1)));
                ++s_it;
            }
            // ---- row sums: the 4 threads of a row, then the two token halves
            lA += __shfl_xor_sync(0xffffffffu, lA, 1); lB += __shfl_xor_sync(0xffffffffu, lB, 1);
            lA += __shfl_xor_sync(0xffffffffu, lA, 2); lB += __shfl_xor_sync(0xffffffffu, lB, 2);
            if (tq == 0) { xch[2 * hA + hf] = lA; xch[2 * (hA + 8) + hf] = lB; }
            named_bar_sync_dyn<64>(2 + q4);
            if (tq == 0 && hf == 0) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int hh = hA + 8 * e;
                    const float l = xch[2 * hh] + xch[2 * hh + 1], m = e ? mB : mA;
                    l_s[hh] = 1.f / l;
                    const int gh = head0 + hh;
                    if (gh < p.head_end) {
                        float lse = (m - kLift + log2f(l)) * kLn2;
                        if (seg.slot < 0) p.lse[(int64_t)seg.request * p.lse_stride_request + gh] = lse;
                        else p.partial_lse[(int64_t)seg.slot * h + (gh - p.head_begin)] = lse;
                    }
                }
            }
            named_bar_sync<1, kNumSoftmaxThreads>();
            // ---- epilogue: O^T block j holds dv = 128 j + TMEM lane, one column per head;
            // this warp takes blocks 2 hf and 2 hf + 1 of its quadrant's lanes
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
            const int nvalid = min(kN, p.head_end - head0);
#pragma unroll 1
            for (int jj = 0; jj < 2; ++jj) {
                const int j = 2 * hf + jj;
                const int dv = 128 * j + 32 * q4 + lane;
#pragma unroll
                for (int c = 0; c < kN / 16; ++c) {
                    float o[16];
                    tmem_ld16(tmem_base + lane_addr + kColO + j * kN + c * 16, o);
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

    fill_empty_requests(p, worker, head0, kN, tid, kThreads);

    // ---- teardown
    if (p.trace != nullptr && tid == 0) p.trace[512 + blockIdx.x] = clock64() - t_start;   // per-CTA cycles
    if (*ctx.abort_flag) {
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

}  // namespace

cudaError_t launch_decode_umma_fp8(const DecodeParams &p, cudaStream_t stream) {
    alignas(64) CUtensorMap mkv;
    if (!make_map_4d(&mkv, CU_TENSOR_MAP_DATA_TYPE_UINT8, CU_TENSOR_MAP_SWIZZLE_64B, p.kv_pool, kPage,
                     (uint64_t)(p.num_pool_pages > 0 ? p.num_pool_pages : 1), (uint64_t)kDQK, 64,
                     (uint64_t)kPage * kDQK, 64))
        return cudaErrorInvalidValue;
    static DeviceOnce once;
    cudaError_t e = once.run([&] { return cudaFuncSetAttribute(decode_umma_fp8_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes); });
    if (e != cudaSuccess) return e;
    e = launch_dependent(decode_umma_fp8_kernel, dim3((unsigned)(p.num_workers * p.num_groups)), dim3(kThreads),
                         (size_t)kSmemBytes, stream, p, mkv);
    count_launch();
    return e;
}

}  // namespace splash
