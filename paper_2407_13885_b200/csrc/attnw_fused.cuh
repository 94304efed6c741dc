// Fused attention-weight kernel for sm_100a: P = Softmax(scale * Q K^T), scores never in HBM.
// (Section VII: matmul + scaling + Softmax in one kernel; Section IV for the product;
//  Eq. 1 for the max-subtracted Softmax.)
//
// One CTA owns 256 query rows of one head (two 128-row tiles) and streams the head's keys past
// them twice:
//   statistics pass  - running row maximum and row sum of exponentials, kept in registers;
//   normalise pass   - the score tiles are recomputed on the tensor cores, turned into
//                      2^(c*s - (c*max + log2 sum)) and written to HBM exactly once.
// Roles (warp-specialised, 576 threads):
//   warps 0-7 / 8-15 Softmax warps of query tile 0 / 1: two warpgroups per tile, one per half of
//                    the 128 key columns; a thread owns one row (TMEM lane) and 64 columns of
//                    every key tile, so row reductions need no shuffles; the two halves of a
//                    row are merged once, through shared memory, between the passes
//   warp 16          TMA producer: Q tiles once, K tiles through a shared-memory ring
//   warp 17          tcgen05.mma issuer; owns the TMEM allocation (4 accumulators of
//                    128 lanes x 128 fp32 columns: two per query tile, double-buffered)
// Data never moves through registers on its way to the tensor cores: TMA writes 128B-swizzled
// K-major tiles that the UMMA descriptors read directly.  P leaves through shared-memory
// staging and TMA stores (full 128-byte lines; ragged edges clipped by the tensor map).
//
// The exponentials dominate the arithmetic (2 per element against 16 MUFU results per clock
// per SM).  A share of them can be evaluated on the FMA pipes instead (Cody-Waite range
// reduction and a cubic minimax polynomial, in packed two-wide fp32 instructions); see
// ATTNW_POLY_PAIRS_* below for why that share is zero by default.
#pragma once
#include <cstdint>
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "ptx.cuh"

namespace attnw {

// Per-device status word: 0 = healthy; otherwise the code of the first bounded wait that gave up.
__device__ unsigned int g_attnw_status = 0;

// Optional per-role cycle stamps of one CTA (the analogue of the paper's per-operation runtime
// figures).  Compiled in only with -DATTNW_TIMELINE; the product build has none of it.
#ifdef ATTNW_TIMELINE
__device__ long long g_attnw_timeline[32][160];
#define ATTNW_STAMP(ev, it)                                                                       \
    do {                                                                                          \
        if (blockIdx.x == ATTNW_TIMELINE && (it) < 160) g_attnw_timeline[ev][it] = clock64();     \
    } while (0)
#else
#define ATTNW_STAMP(ev, it) \
    do {                    \
    } while (0)
#endif

constexpr int kTile = 128;           // rows per query tile = keys per key tile
constexpr int kQTilesPerCta = 2;
constexpr int kRowsPerCta = kTile * kQTilesPerCta;
constexpr int kHalf = kTile / 2;      // key columns of a tile handled by one Softmax warp
constexpr int kChunk = 32;            // columns a thread holds in registers at a time
constexpr int kSoftmaxWarps = 16;
constexpr int kProducerWarp = 16;
constexpr int kMmaWarp = 17;
constexpr int kFusedThreads = 576;
constexpr int kTmemCols = 512;
constexpr int kStageBoxBytes = 32 * 128;  // one staged store box: 32 rows x 128 bytes
constexpr long long kWaitLimitCycles = 2000000000ll;  // about one second

// Of every 8 consecutive column pairs, this many take the polynomial path (bf16 output only;
// the float32 variant keeps every exponential on the MUFU for accuracy).  Default 0: measured on
// B200, the kernel is bound by per-warp latency and, in a sustained loop, by the power the two
// tensor-core passes draw - not by MUFU throughput - so moving exponentials to the FMA pipes
// (tried at 2/8 .. 5/8) changes nothing or costs time.  Kept as a build-time knob.
#ifndef ATTNW_POLY_PAIRS_STATS
#define ATTNW_POLY_PAIRS_STATS 0
#endif
#ifndef ATTNW_POLY_PAIRS_NORM
#define ATTNW_POLY_PAIRS_NORM 0
#endif

enum : uint32_t {  // which wait gave up (low byte of the status word)
    kSiteProducerEmpty = 1,
    kSiteMmaQ = 2,
    kSiteMmaKFull = 3,
    kSiteMmaAccEmpty = 4,
    kSiteSoftmaxStats = 5,
    kSiteSoftmaxNorm = 6,
    kSiteStageFree = 7,
    kSiteStageFilled = 8,
    kSitePair = 9,
};

template <int D>
struct FusedSmem {
    static constexpr int kAtoms = D / 64;               // 128-byte swizzle atoms along d
    static constexpr int kAtomBytes = kTile * 128;      // 128 rows x 128 bytes
    static constexpr int kTileBytes = kAtoms * kAtomBytes;
    static constexpr int kStages = (D == 128) ? 3 : 6;
    static constexpr int kQOff = 0;
    static constexpr int kKOff = kQOff + kQTilesPerCta * kTileBytes;
    static constexpr int kOutOff = kKOff + kStages * kTileBytes;
    static constexpr int kBarOff = kOutOff + kSoftmaxWarps * kStageBoxBytes;
    static constexpr int kBytes = kBarOff + 256;
    static constexpr int kDynamicBytes = kBytes + 1024;  // slack to align the base to 1024
};

struct FusedBarriers {
    uint64_t q_full;
    uint64_t k_full[6];
    uint64_t k_empty[6];
    uint64_t s_full[2][2];   // [query tile][accumulator buffer]
    uint64_t s_empty[2][2];
    uint64_t out_free[4];    // [query tile * 2 + column half]: the staging buffer has been read by its store
    uint64_t out_filled[4];  // ... has been filled by the three warps that do not issue the store
    uint64_t pair_full;      // two CTAs per row block: the partner's statistics have arrived
    uint32_t tmem_base;
    uint32_t abort_flag;
    uint32_t prior_failure;
};
static_assert(sizeof(FusedBarriers) <= 256, "barrier block must fit its slot");

__device__ __noinline__ bool fused_wait_slow(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag,
                                             uint32_t site) {
    const long long t0 = clock64();
    for (uint32_t spin = 1;; ++spin) {
        if (ptx::mbar_try_wait(bar, parity)) return true;
        if ((spin & 63u) == 0) {
            if (*abort_flag) return false;
            if (clock64() - t0 > kWaitLimitCycles) {
                *abort_flag = 1;
                atomicCAS(&g_attnw_status, 0u, 0x80000000u | site);
                return false;
            }
        }
    }
}
// Bounded wait on an mbarrier phase.  false = gave up (time limit, or another role already did).
__device__ __forceinline__ bool fused_wait(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag,
                                           uint32_t site) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    return fused_wait_slow(bar, parity, abort_flag, site);
}

// One thread's 32 consecutive columns of a score tile (TMEM lane = row).
__device__ __forceinline__ void load_chunk(uint32_t taddr, float (&s)[kChunk]) {
    uint32_t r[32];
    ptx::tmem_ld_32x32b_x32(taddr, r);
    ptx::tmem_wait_ld();
#pragma unroll
    for (int j = 0; j < kChunk; ++j) s[j] = __uint_as_float(r[j]);
}

// 2^x for a packed pair, x <= ~0, on the FMA and ALU pipes (no MUFU):
//   x is clamped at -126, split as n + f with n = round(x) (adding 1.5 * 2^23 leaves n in the low
//   mantissa bits) and f in [-0.5, 0.5]; 2^f is a cubic with relative error <= 1.02e-4 and value
//   exactly 1 at f = 0; n is added into the exponent field with one integer shift-add.
// The polynomial error is far below bfloat16 resolution (2^-9) and, for the row sums, below the
// tolerance on P by more than an order of magnitude.
__device__ __forceinline__ void exp2_poly_pair(uint64_t x2, float& e0, float& e1) {
    constexpr float kMagic = 12582912.0f;  // 1.5 * 2^23
    float x0, x1;
    ptx::unpack2(x2, x0, x1);
    x0 = fmaxf(x0, -126.0f);
    x1 = fmaxf(x1, -126.0f);
    const uint64_t xc = ptx::pack2(x0, x1);
    const uint64_t t = ptx::add2(xc, ptx::pack2(kMagic, kMagic));
    const uint64_t n = ptx::add2(t, ptx::pack2(-kMagic, -kMagic));
    const uint64_t f = ptx::sub2(xc, n);
    uint64_t p = ptx::fma2(f, ptx::pack2(0.05500893294811249f, 0.05500893294811249f),
                           ptx::pack2(0.2422109693288803f, 0.2422109693288803f));
    p = ptx::fma2(p, f, ptx::pack2(0.6932829022407532f, 0.6932829022407532f));
    p = ptx::fma2(p, f, ptx::pack2(1.0f, 1.0f));
    float p0, p1, t0, t1;
    ptx::unpack2(p, p0, p1);
    ptx::unpack2(t, t0, t1);
    e0 = __int_as_float(__float_as_int(p0) + (__float_as_int(t0) << 23));
    e1 = __int_as_float(__float_as_int(p1) + (__float_as_int(t1) << 23));
}

// sum_j 2^(c2 * s_j + neg_offset) over one thread's 32-column chunk; of every 8 column pairs,
// POLY_PAIRS go through the polynomial.  RAGGED: columns >= valid do not exist and contribute nothing.
template <int POLY_PAIRS, bool RAGGED>
__device__ __forceinline__ float sum_exp2_chunk(const float (&s)[kChunk], uint64_t c2c2, float neg_offset, int valid) {
    const uint64_t off2 = ptx::pack2(neg_offset, neg_offset);
    uint64_t acc[4] = {0ull, 0ull, 0ull, 0ull};  // four packed pairs of partial sums (+0.0f bits)
#pragma unroll
    for (int j = 0; j < kChunk; j += 2) {
        const uint64_t x2 = ptx::fma2(ptx::pack2(s[j], s[j + 1]), c2c2, off2);
        float e0, e1;
        if (((j >> 1) & 7) < POLY_PAIRS) {
            exp2_poly_pair(x2, e0, e1);
        } else {
            float x0, x1;
            ptx::unpack2(x2, x0, x1);
            e0 = ptx::ex2_approx(x0);
            e1 = ptx::ex2_approx(x1);
        }
        if (RAGGED) {  // masked columns contribute nothing, also when c2 == 0
            e0 = (j + 0 < valid) ? e0 : 0.f;
            e1 = (j + 1 < valid) ? e1 : 0.f;
        }
        acc[(j >> 1) & 3] = ptx::add2(acc[(j >> 1) & 3], ptx::pack2(e0, e1));
    }
    float a0, a1, a2, a3;
    ptx::unpack2(ptx::add2(acc[0], acc[1]), a0, a1);
    ptx::unpack2(ptx::add2(acc[2], acc[3]), a2, a3);
    return (a0 + a1) + (a2 + a3);
}

template <int D, typename OutT>
__global__ void __launch_bounds__(kFusedThreads, 1)
attnw_fused_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_p, int N, int row_blocks_per_head, float scale_log2e,
                   int key_split) {
    using L = FusedSmem<D>;
    constexpr bool kBf16Out = sizeof(OutT) == 2;
    constexpr int kPolyStats = kBf16Out ? ATTNW_POLY_PAIRS_STATS : 0;
    constexpr int kPolyNorm = kBf16Out ? ATTNW_POLY_PAIRS_NORM : 0;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    FusedBarriers* bars = reinterpret_cast<FusedBarriers*>(smem + L::kBarOff);
    volatile uint32_t* abort_flag = &bars->abort_flag;

    if (threadIdx.x == 0) bars->prior_failure = *reinterpret_cast<volatile unsigned int*>(&g_attnw_status);
    __syncthreads();
    if (bars->prior_failure != 0u) {  // an earlier CTA gave up: do not queue more waits behind it
        if (key_split > 1) {          // (the partner CTA still passes the cluster barriers of set-up and teardown)
            ptx::cluster_arrive_release();
            ptx::cluster_wait_acquire();
            ptx::cluster_arrive_release();
            ptx::cluster_wait_acquire();
        }
        return;
    }

    // key_split = 1: one CTA per 256 rows walks all key tiles.  key_split = 2: a cluster of two CTAs shares the 256
    // rows; each walks half of the key tiles in both passes and the two exchange their rows' (offset, sum) between
    // the passes through distributed shared memory - the exchange of local maxima and sums of Section VII, here only
    // to fill the device when the CTAs do not divide evenly over the SMs or are fewer than the SMs.
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t pair_rank = key_split > 1 ? ptx::cluster_ctarank() : 0u;
    const int unit = static_cast<int>(blockIdx.x) / key_split;
    const int bh = unit / row_blocks_per_head;
    const int row0 = (unit % row_blocks_per_head) * kRowsPerCta;
    const int T = ((N + kTile - 1) / kTile) / key_split;  // key tiles of this CTA per pass
    const int kt0 = static_cast<int>(pair_rank) * T;      // its first key tile
    const int total_iters = 2 * T;
    const bool tile_active[2] = {row0 < N, row0 + kTile < N};

    // ---- set-up ------------------------------------------------------------------------------
    if (threadIdx.x == 0) {
        ptx::mbar_init(&bars->q_full, 1);
        for (int s = 0; s < L::kStages; ++s) {
            ptx::mbar_init(&bars->k_full[s], 1);
            ptx::mbar_init(&bars->k_empty[s], 1);
        }
        for (int q = 0; q < 2; ++q)
            for (int b = 0; b < 2; ++b) {
                ptx::mbar_init(&bars->s_full[q][b], 1);
                ptx::mbar_init(&bars->s_empty[q][b], 8);  // one arrival per Softmax warp of the tile
            }
        for (int g = 0; g < 4; ++g) {
            ptx::mbar_init(&bars->out_free[g], 1);
            ptx::mbar_init(&bars->out_filled[g], 3);
        }
        ptx::mbar_init(&bars->pair_full, 1);
        bars->abort_flag = 0;
        ptx::mbar_fence_init();
        if (key_split > 1)  // the partner's 512 (256) threads each send 8 bytes for their row
            ptx::mbar_expect_tx(&bars->pair_full, ((tile_active[0] ? 1u : 0u) + (tile_active[1] ? 1u : 0u)) * 2048u);
    }
    if (warp == kProducerWarp && lane == 0) {
        ptx::prefetch_tensormap(&tm_q);
        ptx::prefetch_tensormap(&tm_k);
        ptx::prefetch_tensormap(&tm_p);
    }
    if (warp == kMmaWarp) {
        ptx::tmem_alloc(&bars->tmem_base, kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (key_split > 1) {  // the partner writes into this CTA's shared memory: not before its barrier exists
        ptx::cluster_arrive_release();
        ptx::cluster_wait_acquire();
    }
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_base;

    if (warp == kProducerWarp) {
        // ================= TMA producer =================
        if (lane == 0) {
            const uint64_t keep = ptx::policy_evict_last();
            int n_active = (tile_active[0] ? 1 : 0) + (tile_active[1] ? 1 : 0);
            ptx::mbar_expect_tx(&bars->q_full, static_cast<uint32_t>(n_active * L::kTileBytes));
            for (int q = 0; q < 2; ++q)
                if (tile_active[q])
                    for (int a = 0; a < L::kAtoms; ++a)
                        ptx::tma_load_3d(smem + L::kQOff + q * L::kTileBytes + a * L::kAtomBytes, &tm_q, &bars->q_full,
                                         a * 64, row0 + q * kTile, bh, keep);
            int issued = 0;
            for (int it = 0; it < total_iters; ++it) {
                const int s = it % L::kStages;
                const uint32_t n = static_cast<uint32_t>(it / L::kStages);
                if (!fused_wait(&bars->k_empty[s], (n & 1u) ^ 1u, abort_flag, kSiteProducerEmpty)) break;
                ptx::mbar_expect_tx(&bars->k_full[s], static_cast<uint32_t>(L::kTileBytes));
                const int kt = kt0 + (it < T ? it : it - T);
                for (int a = 0; a < L::kAtoms; ++a)
                    ptx::tma_load_3d(smem + L::kKOff + s * L::kTileBytes + a * L::kAtomBytes, &tm_k, &bars->k_full[s],
                                     a * 64, kt * kTile, bh, keep);
                issued = it + 1;
            }
            if (*abort_flag) {
                // Unwinding: let the copies already in flight land before shared memory is released.
                const int first = issued > L::kStages ? issued - L::kStages : 0;
                for (int it = first; it < issued; ++it) {
                    const int s = it % L::kStages;
                    const uint32_t n = static_cast<uint32_t>(it / L::kStages);
                    const long long t0 = clock64();
                    while (!ptx::mbar_try_wait(&bars->k_full[s], n & 1u) && clock64() - t0 < kWaitLimitCycles / 8) {
                    }
                }
                const long long t0 = clock64();
                while (!ptx::mbar_try_wait(&bars->q_full, 0) && clock64() - t0 < kWaitLimitCycles / 8) {
                }
            }
        }
    } else if (warp == kMmaWarp) {
        // ================= MMA issuer =================
        // The whole warp walks the loop (waits, addresses, descriptors stay warp-uniform, so they live
        // in uniform registers); one elected lane issues the tensor-core instructions.
        constexpr uint32_t idesc = ptx::umma_idesc_bf16_f32(kTile, kTile);
        const uint32_t q_addr = ptx::smem_u32(smem + L::kQOff);
        const uint32_t k_addr = ptx::smem_u32(smem + L::kKOff);
        bool ok = fused_wait(&bars->q_full, 0, abort_flag, kSiteMmaQ);
        ok = __all_sync(0xffffffffu, ok);
        for (int it = 0; ok && it < total_iters; ++it) {
            const int s = it % L::kStages;
            const uint32_t n = static_cast<uint32_t>(it / L::kStages);
            ok = __all_sync(0xffffffffu, fused_wait(&bars->k_full[s], n & 1u, abort_flag, kSiteMmaKFull));
            if (!ok) break;
            const int buf = it & 1;
            const uint32_t use = static_cast<uint32_t>(it >> 1);
            const uint32_t b_addr = k_addr + static_cast<uint32_t>(s * L::kTileBytes);
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                if (!tile_active[q]) continue;
                ok = __all_sync(0xffffffffu, fused_wait(&bars->s_empty[q][buf], (use & 1u) ^ 1u, abort_flag,
                                                        kSiteMmaAccEmpty));
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>((q * 2 + buf) * kTile);
                const uint32_t a_addr = q_addr + static_cast<uint32_t>(q * L::kTileBytes);
                if (ptx::elect_one()) {
#pragma unroll
                    for (int k = 0; k < D / 16; ++k) {
                        const uint32_t off = static_cast<uint32_t>((k >> 2) * L::kAtomBytes + (k & 3) * 32);
                        ptx::umma_f16_ss(d_tmem, ptx::umma_desc_kmajor_sw128(a_addr + off),
                                         ptx::umma_desc_kmajor_sw128(b_addr + off), idesc, k > 0 ? 1u : 0u);
                    }
                    ptx::umma_commit(&bars->s_full[q][buf]);
                }
                __syncwarp();
            }
            if (!ok) break;
            if (ptx::elect_one()) ptx::umma_commit(&bars->k_empty[s]);  // the stage is free once these MMAs have read it
            __syncwarp();
        }
    } else if (warp < kSoftmaxWarps) {
        // ================= Softmax warps =================
        // warp = 8*q + 4*half + quarter: query tile q, column half of every key tile, TMEM lane quarter.
        const int q = warp >> 3;
        const int half = (warp >> 2) & 1;
        const int quarter = warp & 3;
        if (tile_active[q]) {
            const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) +
                                    static_cast<uint32_t>(q * 2 * kTile + half * kHalf);
            const float c2 = scale_log2e;
            const uint64_t c2c2 = ptx::pack2(c2, c2);
            float smax = -3.0e38f;   // running maximum of the raw scores this thread has seen
            float mb = smax;         // the offset the exponentials in l are relative to: fl(smax * c2), finite from the start
            float l = 0.0f;          // running sum of 2^(c2 * s - mb) over this thread's columns
            bool ok = true;

            // ---- statistics pass (Eq. 1: m_i and the denominator), online over key tiles ----
            for (int it = 0; it < T; ++it) {
                const int buf = it & 1;
                ok = fused_wait(&bars->s_full[q][buf], static_cast<uint32_t>(it >> 1) & 1u, abort_flag,
                                kSiteSoftmaxStats);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                ptx::tc_fence_after_sync();
#pragma unroll 1
                for (int c = 0; c < kHalf / kChunk; ++c) {
                    float s[kChunk];
                    load_chunk(t_lane + static_cast<uint32_t>(buf * kTile + c * kChunk), s);
                    if (c == kHalf / kChunk - 1) {  // last read of this accumulator: it may be overwritten now
                        ptx::tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(&bars->s_empty[q][buf]);
                    }
                    const int valid = N - (kt0 + it) * kTile - half * kHalf - c * kChunk;  // columns of this chunk that exist
                    const bool ragged = valid < kChunk;
                    if (ragged) {
#pragma unroll
                        for (int j = 0; j < kChunk; ++j)
                            if (j >= valid) s[j] = -3.0e38f;
                    }
                    float m0 = ptx::max3(s[0], s[1], s[2]), m1 = ptx::max3(s[3], s[4], s[5]);
                    float m2 = ptx::max3(s[6], s[7], s[8]), m3 = ptx::max3(s[9], s[10], s[11]);
#pragma unroll
                    for (int j = 12; j < 28; j += 8) {
                        m0 = ptx::max3(m0, s[j + 0], s[j + 1]);
                        m1 = ptx::max3(m1, s[j + 2], s[j + 3]);
                        m2 = ptx::max3(m2, s[j + 4], s[j + 5]);
                        m3 = ptx::max3(m3, s[j + 6], s[j + 7]);
                    }
                    m0 = ptx::max3(m0, s[28], s[29]);
                    m1 = ptx::max3(m1, s[30], s[31]);
                    const float new_max = fmaxf(smax, ptx::max3(fmaxf(m0, m1), m2, m3));
                    // Rescale by the difference of the two ROUNDED offsets: exactly 2^0 while the maximum
                    // stands, so no rounding residue compounds over the chunks of a long row.
                    const float mb_new = fmaxf(new_max * c2, -3.0e38f);  // finite also while every column so far is masked
                    l *= ptx::ex2_approx(mb - mb_new);
                    mb = mb_new;
                    smax = new_max;
                    l += ragged ? sum_exp2_chunk<kPolyStats, true>(s, c2c2, -mb, valid)
                                : sum_exp2_chunk<kPolyStats, false>(s, c2c2, -mb, valid);
                }
            }

            // ---- merge the two column halves of each row (both threads end with the same values) ----
            // Each warp publishes its rows' (offset, sum) in its own store-staging buffer, which is idle
            // until the normalise pass; the second barrier keeps a fast warp from reusing it too early.
            {
                float2* mine = reinterpret_cast<float2*>(smem + L::kOutOff + warp * kStageBoxBytes);
                const float2* theirs = reinterpret_cast<const float2*>(smem + L::kOutOff + (warp ^ 4) * kStageBoxBytes);
                mine[lane] = make_float2(mb, l);
                asm volatile("bar.sync %0, 256;" ::"r"(1 + q) : "memory");  // the 8 warps of tile q
                const float2 other = theirs[lane];
                asm volatile("bar.sync %0, 256;" ::"r"(1 + q) : "memory");
                const float mb_row = fmaxf(mb, other.x);
                l = l * ptx::ex2_approx(mb - mb_row) + other.y * ptx::ex2_approx(other.x - mb_row);
                mb = mb_row;
            }
            // ---- two CTAs per row block: add the partner's half of the keys ----
            if (key_split > 1) {
                // every thread sends its row's pair to the thread of the same warp and lane in the partner CTA, into
                // bytes 256.. of that warp's staging buffer (idle until the normalise pass; bytes 0..255 served the
                // merge above), and waits - bounded - for the partner's
                const uint32_t inbox = ptx::smem_u32(smem + L::kOutOff + warp * kStageBoxBytes + 256 + lane * 8);
                ptx::st_async_b64(ptx::map_to_cta(inbox, pair_rank ^ 1u), ptx::pack2(mb, l),
                                  ptx::map_to_cta(ptx::smem_u32(&bars->pair_full), pair_rank ^ 1u));
                ok = __all_sync(0xffffffffu, ok && fused_wait(&bars->pair_full, 0, abort_flag, kSitePair));
                if (ok) {
                    const float2 other = *reinterpret_cast<const float2*>(smem + L::kOutOff + warp * kStageBoxBytes + 256 + lane * 8);
                    const float mb_row = fmaxf(mb, other.x);
                    l = l * ptx::ex2_approx(mb - mb_row) + other.y * ptx::ex2_approx(other.x - mb_row);
                    mb = mb_row;
                }
            }

            // ---- normalise pass: p = 2^(c2*s - (mb + log2 l)), stored once ----
            // bf16 output: 1/l is folded into the exponent (one FFMA + one exponential per element); the
            // extra rounding of the folded offset is far below bf16 resolution.  float32 output keeps the
            // statistics pass's offset and multiplies by 1/l, so the row's common factor cancels.
            // Stores: the four warps (lane quarters) of a column half share one 128-row staging buffer and
            // leave through ONE TMA store per box - few large TMA operations instead of many small ones.
            // Warp `quarter == 0` owns the bulk group; the hand-over uses mbarriers so that these waits are
            // bounded like every other wait in the kernel.
            const float shift = kBf16Out ? mb + ptx::lg2_approx(l) : mb;
            const float inv_l = 1.0f / l;
            const int group = q * 2 + half;
            const uint32_t gbuf = ptx::smem_u32(smem + L::kOutOff + group * 4 * kStageBoxBytes);
            const uint32_t my_row = gbuf + static_cast<uint32_t>(quarter * kStageBoxBytes + lane * 128);
            uint32_t n_tiles = 0;  // boxes this group has staged so far (phase of the two hand-over barriers)
            const bool issuer = quarter == 0;
            const int out_row = row0 + q * kTile;  // first row of the group's boxes (always inside P)
            const uint32_t sw = static_cast<uint32_t>(lane & 7);
            const uint32_t row_sw = my_row + (sw << 4);  // 16-byte piece g of the row lives at row_sw ^ (g << 4)
            const uint64_t stream_out = ptx::policy_evict_first();
            const uint64_t nshift2 = ptx::pack2(-shift, -shift);
            for (int it = T; ok && it < total_iters; ++it) {
                const int kt = kt0 + it - T;
                const int buf = it & 1;
                ok = fused_wait(&bars->s_full[q][buf], static_cast<uint32_t>(it >> 1) & 1u, abort_flag,
                                kSiteSoftmaxNorm);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                // the previous store must have read the staging buffer before anyone overwrites it
                if (issuer) {
                    if (lane == 0) {
                        ptx::bulk_wait_group_read<0>();
                        ptx::mbar_arrive(&bars->out_free[group]);
                    }
                    __syncwarp();
                } else {
                    ok = __all_sync(0xffffffffu, fused_wait(&bars->out_free[group], n_tiles & 1u, abort_flag,
                                                            kSiteStageFree));
                    if (!ok) break;
                }
#pragma unroll 1
                for (int c = 0; c < kHalf / kChunk; ++c) {
                    float s[kChunk];
                    load_chunk(t_lane + static_cast<uint32_t>(buf * kTile + c * kChunk), s);
                    if (c == kHalf / kChunk - 1) {
                        ptx::tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(&bars->s_empty[q][buf]);
                    }
#pragma unroll
                    for (int j = 0; j < kChunk; j += 2) {
                        const uint64_t x2 = ptx::fma2(ptx::pack2(s[j], s[j + 1]), c2c2, nshift2);
                        if (((j >> 1) & 7) < kPolyNorm) {
                            exp2_poly_pair(x2, s[j], s[j + 1]);
                        } else {
                            float x0, x1;
                            ptx::unpack2(x2, x0, x1);
                            s[j] = ptx::ex2_approx(x0);
                            s[j + 1] = ptx::ex2_approx(x1);
                        }
                        if constexpr (!kBf16Out) {
                            s[j] *= inv_l;
                            s[j + 1] *= inv_l;
                        }
                    }
                    if constexpr (kBf16Out) {
                        // this chunk is 64 bytes of the thread's 128-byte staging row: 16-byte pieces 4c .. 4c+3
#pragma unroll
                        for (int g = 0; g < 4; ++g)
                            ptx::st_shared_v4(row_sw ^ (static_cast<uint32_t>(c * 4 + g) << 4),
                                              ptx::pack_bf16x2(s[g * 8 + 0], s[g * 8 + 1]),
                                              ptx::pack_bf16x2(s[g * 8 + 2], s[g * 8 + 3]),
                                              ptx::pack_bf16x2(s[g * 8 + 4], s[g * 8 + 5]),
                                              ptx::pack_bf16x2(s[g * 8 + 6], s[g * 8 + 7]));
                    } else {
                        // float32: one chunk fills the whole 128-byte row, so every chunk is its own box
                        if (c > 0) {
                            if (issuer) {
                                if (lane == 0) {
                                    ptx::bulk_wait_group_read<0>();
                                    ptx::mbar_arrive(&bars->out_free[group]);
                                }
                                __syncwarp();
                            } else {
                                ok = __all_sync(0xffffffffu, fused_wait(&bars->out_free[group], n_tiles & 1u,
                                                                        abort_flag, kSiteStageFree));
                                if (!ok) break;
                            }
                        }
#pragma unroll
                        for (int g = 0; g < 8; ++g)
                            ptx::st_shared_v4(my_row + ((static_cast<uint32_t>(g) ^ sw) << 4), __float_as_uint(s[g * 4 + 0]),
                                              __float_as_uint(s[g * 4 + 1]), __float_as_uint(s[g * 4 + 2]),
                                              __float_as_uint(s[g * 4 + 3]));
                    }
                    if (kBf16Out && c < kHalf / kChunk - 1) continue;  // bf16: the box is complete after both chunks
                    ptx::fence_proxy_async_smem();
                    __syncwarp();
                    if (issuer) {
                        ok = __all_sync(0xffffffffu, fused_wait(&bars->out_filled[group], n_tiles & 1u, abort_flag,
                                                                kSiteStageFilled));
                        if (!ok) break;
                        const int out_col = kt * kTile + half * kHalf + (kBf16Out ? 0 : c * kChunk);
                        if (lane == 0 && out_col < N) {
                            ptx::tma_store_3d(&tm_p, gbuf, out_col, out_row, bh, stream_out);
                            ptx::bulk_commit_group();
                        }
                    } else if (lane == 0) {
                        ptx::mbar_arrive(&bars->out_filled[group]);
                    }
                    ++n_tiles;
                }
            }
            if (lane == 0) ptx::bulk_wait_group<0>();
        }
    }

    // ---- teardown: every role falls through to here, also after a wait gave up ----
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (key_split > 1) {  // the partner may still be sending its statistics into this CTA's shared memory
        ptx::cluster_arrive_release();
        ptx::cluster_wait_acquire();
    }
    if (warp == kMmaWarp) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace attnw
