// Fused attention-weight kernel for sm_100a: P = Softmax(scale * Q K^T), scores never in HBM.
// (Section VII: matmul + scaling + Softmax in one kernel; Section IV for the product;
//  Eq. 1 for the max-subtracted Softmax.)
//
// One CTA owns 256 query rows of one head (two 128-row tiles, one per Softmax warpgroup) and
// streams the head's keys past them twice:
//   statistics pass  - running row maximum and row sum of exponentials, kept in registers;
//   normalise pass   - the score tiles are recomputed on the tensor cores, turned into
//                      2^(c*s - (c*max + log2 sum)) and written to HBM exactly once.
// Roles (warp-specialised, 320 threads):
//   warps 0-3 / 4-7  Softmax warpgroup for query tile 0 / 1; thread t owns row t of the tile
//                    (TMEM lane t), so row reductions need no shuffles
//   warp 8           TMA producer: Q tiles once, K tiles through a shared-memory ring
//   warp 9           tcgen05.mma issuer; owns the TMEM allocation (4 accumulators of
//                    128 lanes x 128 fp32 columns: two per query tile, double-buffered)
// Data never moves through registers on its way to the tensor cores: TMA writes 128B-swizzled
// K-major tiles that the UMMA descriptors read directly.  P leaves through shared-memory
// staging and TMA stores (full 128-byte lines; ragged edges clipped by the tensor map).
#pragma once
#include <cstdint>
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "ptx.cuh"

namespace attnw {

// Per-device status word: 0 = healthy; otherwise the code of the first bounded wait that gave up.
__device__ unsigned int g_attnw_status = 0;

constexpr int kTile = 128;           // rows per query tile = keys per key tile
constexpr int kQTilesPerCta = 2;
constexpr int kRowsPerCta = kTile * kQTilesPerCta;
constexpr int kSoftmaxWarps = 8;
constexpr int kProducerWarp = 8;
constexpr int kMmaWarp = 9;
constexpr int kFusedThreads = 320;
constexpr int kTmemCols = 512;
constexpr int kStageBoxBytes = 32 * 128;  // one staged store box: 32 rows x 128 bytes
constexpr long long kWaitLimitCycles = 2000000000ll;  // about one second

enum : uint32_t {  // which wait gave up (low byte of the status word)
    kSiteProducerEmpty = 1,
    kSiteMmaQ = 2,
    kSiteMmaKFull = 3,
    kSiteMmaAccEmpty = 4,
    kSiteSoftmaxStats = 5,
    kSiteSoftmaxNorm = 6,
    kSiteDrain = 7,
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
    static constexpr int kBarOff = kOutOff + kSoftmaxWarps * 2 * kStageBoxBytes;
    static constexpr int kBytes = kBarOff + 256;
    static constexpr int kDynamicBytes = kBytes + 1024;  // slack to align the base to 1024
};

struct FusedBarriers {
    uint64_t q_full;
    uint64_t k_full[6];
    uint64_t k_empty[6];
    uint64_t s_full[2][2];   // [query tile][accumulator buffer]
    uint64_t s_empty[2][2];
    uint32_t tmem_base;
    uint32_t abort_flag;
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

// Staged store of one 32-row box.  OutT = bf16: 64 columns; float: 32 columns (128 bytes/row).
template <typename OutT>
struct OutTraits;
template <>
struct OutTraits<__nv_bfloat16> {
    static constexpr int kColsPerBox = 64;
};
template <>
struct OutTraits<float> {
    static constexpr int kColsPerBox = 32;
};

template <int D, typename OutT>
__global__ void __launch_bounds__(kFusedThreads, 1)
attnw_fused_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_p, int N, int row_blocks_per_head, float scale_log2e) {
    using L = FusedSmem<D>;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t prior_failure;
    if (threadIdx.x == 0) prior_failure = *reinterpret_cast<volatile unsigned int*>(&g_attnw_status);
    __syncthreads();
    if (prior_failure != 0u) return;  // an earlier CTA gave up: do not queue more waits behind it

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    FusedBarriers* bars = reinterpret_cast<FusedBarriers*>(smem + L::kBarOff);
    volatile uint32_t* abort_flag = &bars->abort_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int bh = blockIdx.x / row_blocks_per_head;
    const int row0 = (blockIdx.x % row_blocks_per_head) * kRowsPerCta;
    const int T = (N + kTile - 1) / kTile;  // key tiles per pass
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
                ptx::mbar_init(&bars->s_empty[q][b], 4);  // one arrival per Softmax warp of the group
            }
        bars->abort_flag = 0;
        ptx::mbar_fence_init();
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
                const int kt = it < T ? it : it - T;
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
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::umma_idesc_bf16_f32(kTile, kTile);
            const uint32_t q_addr = ptx::smem_u32(smem + L::kQOff);
            const uint32_t k_addr = ptx::smem_u32(smem + L::kKOff);
            bool ok = fused_wait(&bars->q_full, 0, abort_flag, kSiteMmaQ);
            for (int it = 0; ok && it < total_iters; ++it) {
                const int s = it % L::kStages;
                const uint32_t n = static_cast<uint32_t>(it / L::kStages);
                if (!fused_wait(&bars->k_full[s], n & 1u, abort_flag, kSiteMmaKFull)) break;
                const int buf = it & 1;
                const uint32_t use = static_cast<uint32_t>(it >> 1);
                for (int q = 0; q < 2; ++q) {
                    if (!tile_active[q]) continue;
                    if (!fused_wait(&bars->s_empty[q][buf], (use & 1u) ^ 1u, abort_flag, kSiteMmaAccEmpty)) {
                        ok = false;
                        break;
                    }
                    ptx::tc_fence_after_sync();
                    const uint32_t d_tmem = tmem_base + static_cast<uint32_t>((q * 2 + buf) * kTile);
#pragma unroll
                    for (int k = 0; k < D / 16; ++k) {
                        const uint32_t off = static_cast<uint32_t>((k >> 2) * L::kAtomBytes + (k & 3) * 32);
                        const uint64_t a_desc = ptx::umma_desc_kmajor_sw128(q_addr + q * L::kTileBytes + off);
                        const uint64_t b_desc = ptx::umma_desc_kmajor_sw128(k_addr + s * L::kTileBytes + off);
                        ptx::umma_f16_ss(d_tmem, a_desc, b_desc, idesc, k > 0 ? 1u : 0u);
                    }
                    ptx::umma_commit(&bars->s_full[q][buf]);
                }
                if (!ok) break;
                ptx::umma_commit(&bars->k_empty[s]);  // the stage is free once these MMAs have read it
            }
        }
        __syncwarp();
    } else {
        // ================= Softmax warpgroups =================
        const int q = warp >> 2;                 // query tile of this warpgroup
        const int warp_in_group = warp & 3;      // TMEM lane quarter this warp may read
        if (tile_active[q]) {
            const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(warp_in_group * 32) << 16) +
                                    static_cast<uint32_t>(q * 2 * kTile);
            const float c2 = scale_log2e;
            float smax = -3.0e38f;   // running maximum of the raw scores of this thread's row
            float mb = smax * c2;    // the offset the exponentials in l are relative to: fl(smax * c2)
            float l = 0.0f;          // running sum of 2^(c2 * s - mb)
            bool ok = true;

            // ---- statistics pass (Eq. 1: m_i and the denominator), online over key tiles ----
            for (int it = 0; it < T; ++it) {
                const int buf = it & 1;
                ok = fused_wait(&bars->s_full[q][buf], static_cast<uint32_t>(it >> 1) & 1u, abort_flag,
                                kSiteSoftmaxStats);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t t_acc = t_lane + static_cast<uint32_t>(buf * kTile);
                const int valid = N - it * kTile;  // columns of this tile that exist (>= 1)
#pragma unroll 1
                for (int c = 0; c < kTile / 32; ++c) {
                    uint32_t raw[32];
                    ptx::tmem_ld_32x32b_x32(t_acc + static_cast<uint32_t>(c * 32), raw);
                    ptx::tmem_wait_ld();
                    if (c == kTile / 32 - 1) {  // the accumulator may be overwritten from here on
                        ptx::tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(&bars->s_empty[q][buf]);
                    }
                    float s[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) s[j] = __uint_as_float(raw[j]);
                    const bool ragged = valid < (c + 1) * 32;
                    if (ragged) {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (c * 32 + j >= valid) s[j] = -3.0e38f;
                    }
                    float cm0 = ptx::max3(s[0], s[1], s[2]), cm1 = ptx::max3(s[3], s[4], s[5]);
#pragma unroll
                    for (int j = 6; j < 30; j += 4) {
                        cm0 = ptx::max3(cm0, s[j], s[j + 1]);
                        cm1 = ptx::max3(cm1, s[j + 2], s[j + 3]);
                    }
                    const float new_max = fmaxf(smax, ptx::max3(cm0, cm1, fmaxf(s[30], s[31])));
                    // Rescale by the difference of the two ROUNDED offsets: exactly 2^0 while the maximum
                    // stands, so no rounding residue compounds over the chunks of a long row.
                    const float mb_new = new_max * c2;
                    l *= ptx::ex2_approx(mb - mb_new);
                    mb = mb_new;
                    smax = new_max;
                    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        float e0 = ptx::ex2_approx(fmaf(s[j + 0], c2, -mb));
                        float e1 = ptx::ex2_approx(fmaf(s[j + 1], c2, -mb));
                        float e2 = ptx::ex2_approx(fmaf(s[j + 2], c2, -mb));
                        float e3 = ptx::ex2_approx(fmaf(s[j + 3], c2, -mb));
                        if (ragged) {  // masked columns contribute nothing, also when c2 == 0
                            e0 = (c * 32 + j + 0 < valid) ? e0 : 0.f;
                            e1 = (c * 32 + j + 1 < valid) ? e1 : 0.f;
                            e2 = (c * 32 + j + 2 < valid) ? e2 : 0.f;
                            e3 = (c * 32 + j + 3 < valid) ? e3 : 0.f;
                        }
                        a0 += e0;
                        a1 += e1;
                        a2 += e2;
                        a3 += e3;
                    }
                    l += (a0 + a1) + (a2 + a3);
                }
            }

            // ---- normalise pass: p = 2^(c2*s - (c2*max + log2 l)), stored once ----
            constexpr int kCols = OutTraits<OutT>::kColsPerBox;
            // bf16 output: 1/l is folded into the exponent (one FFMA + one ex2 per element); the extra
            // rounding of the folded offset is far below bf16 resolution.  float32 output keeps the
            // statistics pass's offset and multiplies by 1/l, so the row's common factor cancels.
            const float shift = sizeof(OutT) == 2 ? mb + ptx::lg2_approx(l) : mb;
            const float inv_l = 1.0f / l;
            const uint32_t stage_base = ptx::smem_u32(smem + L::kOutOff + warp * 2 * kStageBoxBytes);
            const int out_row = row0 + q * kTile + warp_in_group * 32;  // first row of this warp's boxes
            const bool rows_exist = out_row < N;
            const uint32_t sw = static_cast<uint32_t>(lane & 7);
            const uint32_t row_off = static_cast<uint32_t>(lane) * 128u;
            const uint64_t stream_out = ptx::policy_evict_first();
            uint32_t n_boxes = 0;
            for (int it = T; ok && it < total_iters; ++it) {
                const int kt = it - T;
                const int buf = it & 1;
                ok = fused_wait(&bars->s_full[q][buf], static_cast<uint32_t>(it >> 1) & 1u, abort_flag,
                                kSiteSoftmaxNorm);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t t_acc = t_lane + static_cast<uint32_t>(buf * kTile);
#pragma unroll 1
                for (int box = 0; box < kTile / kCols; ++box) {
                    const uint32_t sbuf = stage_base + (n_boxes & 1u) * kStageBoxBytes;
                    if (lane == 0) ptx::bulk_wait_group_read<1>();  // the store that last used sbuf has read it
                    __syncwarp();
#pragma unroll
                    for (int c = 0; c < kCols / 32; ++c) {
                        uint32_t raw[32];
                        const int col = box * kCols + c * 32;
                        ptx::tmem_ld_32x32b_x32(t_acc + static_cast<uint32_t>(col), raw);
                        ptx::tmem_wait_ld();
                        if (col == kTile - 32) {
                            ptx::tc_fence_before_sync();
                            __syncwarp();
                            if (lane == 0) ptx::mbar_arrive(&bars->s_empty[q][buf]);
                        }
                        float p[32];
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            p[j] = ptx::ex2_approx(fmaf(__uint_as_float(raw[j]), c2, -shift));
                            if constexpr (sizeof(OutT) == 4) p[j] *= inv_l;
                        }
                        if constexpr (sizeof(OutT) == 2) {
#pragma unroll
                            for (int g = 0; g < 4; ++g) {  // 8 bf16 = one 16-byte chunk
                                const uint32_t chunk = static_cast<uint32_t>(c * 4 + g);
                                ptx::st_shared_v4(sbuf + row_off + ((chunk ^ sw) << 4),
                                                  ptx::pack_bf16x2(p[g * 8 + 0], p[g * 8 + 1]),
                                                  ptx::pack_bf16x2(p[g * 8 + 2], p[g * 8 + 3]),
                                                  ptx::pack_bf16x2(p[g * 8 + 4], p[g * 8 + 5]),
                                                  ptx::pack_bf16x2(p[g * 8 + 6], p[g * 8 + 7]));
                            }
                        } else {
#pragma unroll
                            for (int g = 0; g < 8; ++g) {  // 4 floats = one 16-byte chunk
                                ptx::st_shared_v4(sbuf + row_off + ((static_cast<uint32_t>(g) ^ sw) << 4),
                                                  __float_as_uint(p[g * 4 + 0]), __float_as_uint(p[g * 4 + 1]),
                                                  __float_as_uint(p[g * 4 + 2]), __float_as_uint(p[g * 4 + 3]));
                            }
                        }
                    }
                    ptx::fence_proxy_async_smem();
                    __syncwarp();
                    const int out_col = kt * kTile + box * kCols;
                    if (lane == 0) {
                        // A box that lies wholly outside P is not stored, but its (empty) group is still
                        // committed: the buffer hand-over above counts one group per box.
                        if (rows_exist && out_col < N) ptx::tma_store_3d(&tm_p, sbuf, out_col, out_row, bh, stream_out);
                        ptx::bulk_commit_group();
                    }
                    ++n_boxes;
                }
            }
            if (lane == 0) ptx::bulk_wait_group<0>();
        }
    }

    // ---- teardown: every role falls through to here, also after a wait gave up ----
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == kMmaWarp) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace attnw
