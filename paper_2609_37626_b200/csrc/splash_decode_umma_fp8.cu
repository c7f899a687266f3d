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
//   P_ht  = u_hi + u_lo,       u = 2^(y - m + 4) with y = log2-domain logit + log2(scale_t)
//
// i.e. the per-token scale is folded into the softmax weight in the log domain, so the
// weights of a tile are automatically normalised (u <= 2^8 with the lazy-rescale threshold
// of 2^4) and sit in e4m3's normal range; the row sum adds u / scale_t = 2^(x - m + 4).
// Four e4m3 products per bf16-precision product pair cost the tensor pipe the same time as
// the bf16 kernel (fp8 MMAs run at twice the rate), which is why the roofline of this
// workload is taken at the bf16 rate.
#include <cuda_fp16.h>

#include "splash_umma.cuh"

namespace splash {

namespace {

using namespace umma;

constexpr int kThreads = 288;                      // producer, 4 MMA issuers, 4 softmax warps
constexpr int kMmaWarps = 4;
constexpr int kNumSoftmaxThreads = 128;
constexpr int kN = 64;                             // heads per CTA
constexpr int kChunks = 9;                         // 576 / 64-element (64 B) chunks
constexpr uint32_t kSlab = 64 * 64;                // one chunk of one page: 64 tokens x 64 B
constexpr uint32_t kStageBytes = kChunks * kSlab;  // 36,864
constexpr uint32_t kScaleBytes = 256;              // 64 fp32 token scales of a page
constexpr int kStages = 4;
constexpr int kAcc = 4;                            // partial accumulators of S = QK issuers
constexpr float kTau = 4.0f;                       // lazy rescale threshold, log2 units
constexpr float kLift = 4.0f;                      // weights are stored as 2^(y - m + kLift) <= 2^8

enum BarrierId {
    kBarKvFull = 0,
    kBarKvEmpty = kBarKvFull + kStages,
    kBarQFull = kBarKvEmpty + kStages,
    kBarQEmpty,
    kBarSFull,
    kBarSEmpty,
    kBarPFull,
    kBarOFull,
    kBarOEmpty,
    kNumBarriers
};

// shared memory map (all swizzled regions 512-byte aligned: 8 rows x 64 B atoms)
constexpr uint32_t kOffKv = 0;
constexpr uint32_t kOffQHi = kOffKv + kStages * kStageBytes;
constexpr uint32_t kOffQLo = kOffQHi + kN * kDQK;
constexpr uint32_t kOffPHi = kOffQLo + kN * kDQK;
constexpr uint32_t kOffPLo = kOffPHi + kN * 64;
constexpr uint32_t kOffScale = kOffPLo + kN * 64;          // float [kStages][64]
constexpr uint32_t kOffQs = kOffScale + kStages * kScaleBytes;   // float [64] query scales
constexpr uint32_t kOffAlpha = kOffQs + kN * 4;
constexpr uint32_t kOffL = kOffAlpha + kN * 4;
constexpr uint32_t kOffTok = kOffL + kN * 4;                // float2 [2][64]: (log2 scale_t, 1 / scale_t) of a tile
constexpr uint32_t kOffBar = kOffTok + 2 * 64 * 8;
constexpr uint32_t kOffMisc = (kOffBar + kNumBarriers * 8 + 15) / 16 * 16;
constexpr uint32_t kSmemBytes = kOffMisc + 32;
static_assert(kSmemBytes <= 232448, "shared memory overflow");
static_assert(kOffQHi % 512 == 0 && kOffQLo % 512 == 0 && kOffPHi % 512 == 0 && kOffPLo % 512 == 0, "alignment");
// tensor memory: O^T 4 blocks x 64 columns, then 4 partial S accumulators x 64 columns
constexpr uint32_t kColO = 0, kColS = 256;

__host__ __device__ constexpr uint32_t make_idesc_e4m3(int M, int N, int a_mn_major) {
    // fp32 accumulate (bit 4), A and B formats E4M3 (= 0)
    return (1u << 4) | ((uint32_t)a_mn_major << 15) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

__device__ __forceinline__ void umma_e4m3(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// two floats -> two e4m3 bytes (first argument in the low byte), round to nearest, saturating
__device__ __forceinline__ uint16_t to_e4m3x2(float lo, float hi) {
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ float2 from_e4m3x2(uint16_t v) {
    uint32_t h2;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(v));
    __half2 h = *reinterpret_cast<__half2 *>(&h2);
    return __half22float2(h);
}
__device__ __forceinline__ float fast_log2(float x) {
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float fast_rcp(float x) {
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Split x >= 0 into hi + lo with hi carrying 4 significant bits (an e4m3 value when it is in
// e4m3's normal range): Veltkamp's splitting with 2^20 + 1, all in the fp32 pipe.
__device__ __forceinline__ void split4(float x, float &hi, float &lo) {
    const float c = x * 1048577.0f;
    hi = c - (c - x);
    lo = x - hi;
}

// byte offset of (row, byte column) inside a [rows][64 B] slab in the 64-byte swizzle
__device__ __forceinline__ uint32_t sw64(uint32_t row, uint32_t col_byte) {
    return row * 64 + ((((col_byte >> 4) ^ (row >> 1)) & 3) << 4) + (col_byte & 15);
}

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
        for (int s = 0; s < kStages; ++s) { mbar_init(bar(kBarKvFull + s), 1); mbar_init(bar(kBarKvEmpty + s), kMmaWarps); }
        mbar_init(bar(kBarQFull), kNumSoftmaxThreads); mbar_init(bar(kBarQEmpty), kAcc);
        mbar_init(bar(kBarSFull), kAcc); mbar_init(bar(kBarSEmpty), kNumSoftmaxThreads);
        mbar_init(bar(kBarPFull), kNumSoftmaxThreads);
        mbar_init(bar(kBarOFull), kMmaWarps); mbar_init(bar(kBarOEmpty), kNumSoftmaxThreads);
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
                if (lane == 0) {
                    const uint32_t stage = kv_it % kStages, ph = (kv_it / kStages) & 1;
                    ok = mbar_wait(ctx, bar(kBarKvEmpty + stage), ph ^ 1, kBarKvEmpty + stage);
                    mark(kv_it, 0);
                    if (ok) {
                        const TileGeom g = tile_geom(seg.lo, seg.hi, (first_page + tile) * kPage);
                        // a page id outside the pool reads as zeros through the tensor map; its
                        // scale page is not fetched (plain addresses are not bounds-checked)
                        const bool in_pool = page >= 0 && page < p.num_pool_pages;
                        mbar_expect_tx(bar(kBarKvFull + stage), kStageBytes + (in_pool ? kScaleBytes : 0u));
                        tma_load_4d(sbase + kOffKv + stage * kStageBytes, &tmap_kv, bar(kBarKvFull + stage), 0, g.tok0, 0, page);
                        if (in_pool)
                            bulk_load(sbase + kOffScale + stage * kScaleBytes, p.kv_scales + (int64_t)page * kPage,
                                      kScaleBytes, bar(kBarKvFull + stage));
                        mark(kv_it, 1);
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                ++kv_it;
            }
        }
    } else if (warp <= kMmaWarps) {
        // ===================================================== MMA issuers
        if (lane == 0) {
            const int mw = warp - 1;                 // partial accumulator mw of S, dv block mw of O^T
            constexpr uint32_t kIdescQK = make_idesc_e4m3(64, 64, 0);
            constexpr uint32_t kIdescPV = make_idesc_e4m3(128, 64, 1);
            uint32_t kv_it = 0, seg_it = 0;
            bool ok = true;
            // 18 K = 32 steps x (q hi, q lo) = 36 MMAs per tile; this issuer takes every fourth
            auto issue_qk = [&](uint32_t kv) {
                const uint32_t stage = kv % kStages;
                if (mw == 0) mark(kv, 2);
                tcgen05_fence_after();
                const uint32_t k0 = sbase + kOffKv + stage * kStageBytes;
                const uint32_t d = tmem_base + kColS + mw * kN;
#pragma unroll
                for (int t = 0; t < 36 / kAcc; ++t) {
                    const int idx = t * kAcc + mw, hl = idx / 18, ks = idx % 18, c = ks >> 1, k = ks & 1;
                    const uint32_t q0 = sbase + (hl ? kOffQLo : kOffQHi);
                    uint64_t dq = make_desc_sw64(q0 + c * kSlab + k * 32, 16, 512);     // A: 64 heads x 32
                    uint64_t dk = make_desc_sw64(k0 + c * kSlab + k * 32, 16, 512);     // B: 64 tokens x 32
                    umma_e4m3(d, dq, dk, kIdescQK, t != 0);
                }
                umma_commit(bar(kBarSFull));
                if (mw == 0) mark(kv, 3);
            };
            // O^T block mw += V^T (128 dv x 64 tokens) * (P hi + P lo): 2 K = 32 steps x 2 terms
            auto issue_pv = [&](uint32_t stage, bool first_tile) {
                tcgen05_fence_after();
                const uint32_t v0 = sbase + kOffKv + stage * kStageBytes + (2 * mw) * kSlab;
#pragma unroll
                for (int hl = 0; hl < 2; ++hl) {
#pragma unroll
                    for (int k = 0; k < 2; ++k) {
                        // A: two 64-element chunks (LBO apart) x 32 tokens (SBO per 8 tokens), MN-major
                        uint64_t da = make_desc_sw64(v0 + k * 2048, kSlab, 512);
                        uint64_t db = make_desc_sw64(sbase + (hl ? kOffPLo : kOffPHi) + k * 32, 16, 512);
                        umma_e4m3(tmem_base + kColO + mw * kN, da, db, kIdescPV, (!first_tile) || (hl | k) != 0);
                    }
                }
            };
            while (ok && it.next(p, seg)) {
                const int ntiles = seg.tile_end - seg.tile_begin;
                ok = mbar_wait(ctx, bar(kBarQFull), seg_it & 1, kBarQFull);
                if (!ok) break;
                int qk_i = 0, pv_i = 0;
                unsigned long long idle_since = 0;
                uint32_t spins = 0;
                while (pv_i < ntiles) {
                    bool progressed = false;
                    if (qk_i > pv_i && mbar_test_wait(bar(kBarPFull), (kv_it + pv_i) & 1)) {
                        if (pv_i == 0 && !mbar_wait(ctx, bar(kBarOEmpty), (seg_it & 1) ^ 1, kBarOEmpty)) { ok = false; break; }
                        const uint32_t stage = (kv_it + pv_i) % kStages;
                        if (mw == 0) mark(kv_it + pv_i, 6);
                        issue_pv(stage, pv_i == 0);
                        umma_commit(bar(kBarKvEmpty + stage));   // P.V done: stage free, P buffers free, O^T updated
                        if (pv_i + 1 == ntiles) umma_commit(bar(kBarOFull));
                        if (mw == 0) mark(kv_it + pv_i, 7);
                        ++pv_i;
                        progressed = true;
                    }
                    if (qk_i < ntiles && qk_i < pv_i + 2) {
                        const uint32_t kv = kv_it + qk_i;
                        if (mbar_test_wait(bar(kBarKvFull + kv % kStages), (kv / kStages) & 1) &&
                            mbar_test_wait(bar(kBarSEmpty), (kv & 1) ^ 1)) {
                            issue_qk(kv);
                            ++qk_i;
                            if (qk_i == ntiles) umma_commit(bar(kBarQEmpty));
                            progressed = true;
                        }
                    }
                    if (progressed) { idle_since = 0; spins = 0; continue; }
                    if ((++spins & 1023u) != 0) continue;
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
                kv_it += ntiles;
                ++seg_it;
            }
        }
    } else {
        // ===================================================== softmax + epilogue warps
        const int q4 = warp & 3;                       // TMEM lane quadrant of this warp
        const int st = (warp - 1 - kMmaWarps) * 32 + lane;   // 0..127
        const uint32_t lane_addr = (uint32_t)(32 * q4) << 16;
        const int hA = 16 * q4 + (lane >> 2);          // this thread's heads: hA and hA + 8
        const int tq = lane & 3;                       // its tokens: 8k + 2 tq + {0, 1}
        float *qs_s = reinterpret_cast<float *>(smem + kOffQs);
        float *alpha_s = reinterpret_cast<float *>(smem + kOffAlpha);
        float *l_s = reinterpret_cast<float *>(smem + kOffL);
        const float *scale_s = reinterpret_cast<const float *>(smem + kOffScale);
        const float scale_log2 = p.softmax_scale * kLog2e;
        uint32_t s_it = 0, seg_it = 0;
        bool ok = true;
        while (ok && it.next(p, seg)) {
            // ---- query rows -> e4m3 hi + lo, one scale per head; two threads per head
            ok = mbar_wait(ctx, bar(kBarQEmpty), (seg_it & 1) ^ 1, kBarQEmpty);
            if (!ok) break;
            {
                const int hd = st >> 1, half = st & 1;
                const int gh = head0 + hd;
                const bool live = gh < p.head_end;
                const uint4 *src = reinterpret_cast<const uint4 *>(
                    static_cast<const __nv_bfloat16 *>(p.q) + (int64_t)seg.request * p.q_stride_request +
                    (int64_t)(live ? gh : p.head_begin) * p.q_stride_head + half * 288);
                float amax = 0.f;
                if (live) {
#pragma unroll 4
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
                if (half == 0) qs_s[hd] = qs;
#pragma unroll 2
                for (int v = 0; v < 36; ++v) {
                    uint4 x = live ? __ldg(src + v) : make_uint4(0u, 0u, 0u, 0u);
                    const uint32_t w[4] = {x.x, x.y, x.z, x.w};
                    uint16_t hi[4], lo[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const float e0 = __uint_as_float(w[k] << 16) * inv, e1 = __uint_as_float(w[k] & 0xffff0000u) * inv;
                        hi[k] = to_e4m3x2(e0, e1);
                        const float2 back = from_e4m3x2(hi[k]);
                        lo[k] = to_e4m3x2(e0 - back.x, e1 - back.y);
                    }
                    const uint32_t d = (uint32_t)(half * 288 + v * 8);
                    const uint32_t off = (d >> 6) * kSlab + sw64((uint32_t)hd, d & 63);
                    *reinterpret_cast<uint2 *>(smem + kOffQHi + off) =
                        make_uint2((uint32_t)hi[0] | ((uint32_t)hi[1] << 16), (uint32_t)hi[2] | ((uint32_t)hi[3] << 16));
                    *reinterpret_cast<uint2 *>(smem + kOffQLo + off) =
                        make_uint2((uint32_t)lo[0] | ((uint32_t)lo[1] << 16), (uint32_t)lo[2] | ((uint32_t)lo[3] << 16));
                }
                fence_proxy_async();
                mbar_arrive(bar(kBarQFull));
            }
            softmax_bar_sync();                            // qs_s visible to everyone
            const float cqA = scale_log2 * qs_s[hA], cqB = scale_log2 * qs_s[hA + 8];
            float mA = -INFINITY, mB = -INFINITY, lA = 0.f, lB = 0.f;
            const int first_page = seg.lo / kPage;
            const int ntiles = seg.tile_end - seg.tile_begin;
            for (int i = 0; ok && i < ntiles; ++i) {
                const TileGeom g = tile_geom(seg.lo, seg.hi, (first_page + seg.tile_begin + i) * kPage);
                const uint32_t stage = s_it % kStages;
                ok = mbar_wait(ctx, bar(kBarSFull), s_it & 1, kBarSFull);
                if (!ok) break;
                if (st == 0) mark(s_it, 4);
                // the scale page rode on the stage's own barrier, long complete by now
                ok = mbar_wait(ctx, bar(kBarKvFull + stage), (s_it / kStages) & 1, kBarKvFull + stage);
                if (!ok) break;
                tcgen05_fence_after();
                float s[32];
                {
                    const uint32_t sb = tmem_base + lane_addr + kColS;
                    tmem_ld_16x256b_x8(sb, s);
#pragma unroll
                    for (int a = 1; a < kAcc; ++a) {
                        float part[32];
                        tmem_ld_16x256b_x8(sb + a * kN, part);
                        tmem_wait_ld();
#pragma unroll
                        for (int n = 0; n < 32; ++n) s[n] += part[n];
                    }
                }
                tmem_wait_ld();
                tcgen05_fence_before();
                mbar_arrive(bar(kBarSEmpty));
                // per-token tables of this tile, one token per thread: (log2 scale_t, 1 / scale_t)
                float2 *tok = reinterpret_cast<float2 *>(smem + kOffTok) + (s_it & 1) * 64;
                const float *sc = scale_s + stage * 64 + g.tok0;
                if (st < 64) {
                    const bool v = st >= g.r_lo && st < g.r_hi;
                    const float ts = v ? sc[st] : 1.0f;
                    tok[st] = make_float2(fast_log2(ts), fast_rcp(ts));
                }
                softmax_bar_sync();
                // y = log2-domain logit + log2(token scale)
                float mtA = -INFINITY, mtB = -INFINITY;
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const int r0 = 8 * k + 2 * tq;
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
                bool grew = false;
                float alA = 1.f, alB = 1.f;
                if (mtA > mA + kTau) { alA = (mA == -INFINITY) ? 0.f : fast_exp2(mA - mtA); mA = mtA; lA *= alA; grew = true; }
                if (mtB > mB + kTau) { alB = (mB == -INFINITY) ? 0.f : fast_exp2(mB - mtB); mB = mtB; lB *= alB; grew = true; }
                if (tq == 0) { alpha_s[hA] = alA; alpha_s[hA + 8] = alB; }
                const float offA = kLift - mA, offB = kLift - mB;
                uint16_t phiA[8], ploA[8], phiB[8], ploB[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const float4 t2 = *reinterpret_cast<const float4 *>(&tok[8 * k + 2 * tq]);
                    const float a0 = fast_exp2(s[4 * k + 0] + offA), a1 = fast_exp2(s[4 * k + 1] + offA);
                    const float b0 = fast_exp2(s[4 * k + 2] + offB), b1 = fast_exp2(s[4 * k + 3] + offB);
                    lA = fmaf(a0, t2.y, lA); lA = fmaf(a1, t2.w, lA);
                    lB = fmaf(b0, t2.y, lB); lB = fmaf(b1, t2.w, lB);
                    float h0, h1, r0, r1;
                    split4(a0, h0, r0); split4(a1, h1, r1);
                    phiA[k] = to_e4m3x2(h0, h1); ploA[k] = to_e4m3x2(r0, r1);
                    split4(b0, h0, r0); split4(b1, h1, r1);
                    phiB[k] = to_e4m3x2(h0, h1); ploB[k] = to_e4m3x2(r0, r1);
                }
                const bool rescale = softmax_bar_or(grew);
                // P.V of the previous tile must be done with the P buffers and with O^T
                if (s_it > 0) {
                    const uint32_t prev = s_it - 1;
                    ok = mbar_wait(ctx, bar(kBarKvEmpty + prev % kStages), (prev / kStages) & 1, kBarKvEmpty + prev % kStages);
                    if (!ok) break;
                }
                tcgen05_fence_after();
                if (rescale && i > 0) {
#pragma unroll 1
                    for (int c = 0; c < 4 * kN / 16; ++c) {
                        float o[16];
                        const uint32_t addr = tmem_base + lane_addr + kColO + c * 16;
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
                    for (int k = 0; k < 8; ++k) {
                        const uint32_t offA_ = sw64((uint32_t)hA, (uint32_t)(8 * k + 2 * tq));
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
                mbar_arrive(bar(kBarPFull));
                ++s_it;
            }
            if (!ok) break;
            lA += __shfl_xor_sync(0xffffffffu, lA, 1); lB += __shfl_xor_sync(0xffffffffu, lB, 1);
            lA += __shfl_xor_sync(0xffffffffu, lA, 2); lB += __shfl_xor_sync(0xffffffffu, lB, 2);
            if (tq == 0) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int hh = hA + 8 * e;
                    const float l = e ? lB : lA, m = e ? mB : mA;
                    l_s[hh] = 1.f / l;
                    const int gh = head0 + hh;
                    if (gh < p.head_end) {
                        float lse = (m - kLift + log2f(l)) * kLn2;
                        if (seg.slot < 0) p.lse[(int64_t)seg.request * p.lse_stride_request + gh] = lse;
                        else p.partial_lse[(int64_t)seg.slot * h + (gh - p.head_begin)] = lse;
                    }
                }
            }
            softmax_bar_sync();
            // ---- epilogue: O^T block j holds dv = 128 j + TMEM lane, one column per head
            ok = mbar_wait(ctx, bar(kBarOFull), seg_it & 1, kBarOFull);
            if (!ok) break;
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
            for (int j = 0; j < 4; ++j) {
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
            mbar_arrive(bar(kBarOEmpty));
            ++seg_it;
        }
    }

    // ---- teardown
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
    cudaError_t e = cudaFuncSetAttribute(decode_umma_fp8_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e != cudaSuccess) return e;
    decode_umma_fp8_kernel<<<(unsigned)(p.num_workers * p.num_groups), kThreads, kSmemBytes, stream>>>(p, mkv);
    count_launch();
    return cudaGetLastError();
}

}  // namespace splash
