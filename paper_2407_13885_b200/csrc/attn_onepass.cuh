// Fused attention O = Softmax(scale * Q K^T) V for sm_100a in ONE pass over the keys: Attention(Q, K, V) of
// Section IV (the product with V is the paper's future work, Section VIII) with the online form of Eq. 1.
//
// A CTA owns 256 query rows (two tiles).  Per key tile j and query tile q:
//   MMA 1     S = Q_q K_j^T                       128 x 128 fp32 in tensor memory (one buffer per query tile)
//   Softmax   two threads per row, 64 columns each: a thread takes its scores to registers (the buffer is handed back
//             at once, so the next tile's MMA 1 runs meanwhile) and also reads the other thread's 64 columns for
//             their maximum, so both know the row maximum without an exchange; p = 2^(c s - mb) with the row's
//             offset mb; l += sum p; P (bf16) is written to shared memory as a K-major MMA operand
//   MMA 2     O_q += P V_j                        128 x d fp32 in tensor memory; V_j as TMA delivers it
//             ([128 keys x d], an MN-major B operand)
// The offset mb of a row follows its running maximum lazily: it moves only when the maximum has grown by more than 8
// (in the base-2 exponent), and then O's row and l are multiplied by 2^(mb_old - mb_new) - after the first tiles
// this is rare, and weights stay below 2^8.  The division by l happens once, in the epilogue.  One exponential and
// two MMA passes per element.
// Valid for any N >= 1, d in {64, 128}; Q, K, V, O bf16 [B, H, N, d].
#pragma once
#include "attn_fused.cuh"

namespace attnw {
namespace av1 {

constexpr int kSmWarps = 16;      // Softmax warps: query tile (2) x column half (2) x TMEM lane quarter (4)
constexpr int kProducer = 16;
constexpr int kMma = 17;
constexpr int kThreads = 576;
constexpr int kStages = 3;        // ring of K / V tiles (128 keys x d)
constexpr float kLazy = 8.0f;     // the offset follows the maximum only when it has grown by more than this

enum : uint32_t {  // wait sites of this kernel (low byte of the status word)
    kSiteProducerEmpty = 96,
    kSiteMmaQ = 97,
    kSiteMmaKFull = 98,
    kSiteMmaSFree = 99,
    kSiteMmaPFull = 100,
    kSiteSFull = 101,
    kSitePFree = 102,
    kSiteOFull = 103,
    kSiteOutFilled = 104,
    kSiteLFull = 105,
};

template <int D>
struct Smem {
    static constexpr int kAtoms = D / 64;
    static constexpr int kAtomBytes = kTile * 128;             // 128 rows x 128 bytes
    static constexpr int kTileBytes = kAtoms * kAtomBytes;     // a Q, K or V tile
    static constexpr int kPBytes = 2 * kAtomBytes;             // a P tile: 128 rows x 128 keys, two atoms of 64 keys
    static constexpr int kQOff = 0;
    static constexpr int kKOff = kQOff + 2 * kTileBytes;
    static constexpr int kPOff = kKOff + kStages * kTileBytes;
    static constexpr int kBarOff = kPOff + 2 * kPBytes;
    static constexpr int kBytes = kBarOff + 256;
    static constexpr int kDynamicBytes = kBytes + 1024;
};
static_assert(Smem<128>::kDynamicBytes <= 227 * 1024, "shared memory budget");

struct Barriers {
    uint64_t q_full;
    uint64_t k_full[kStages], k_empty[kStages];
    uint64_t s_full[2], s_free[2];  // per query tile: scores written / read into registers (8 warps)
    uint64_t p_full[2], p_free[2];  // per query tile: P tile written (8 warps) / read by its MMAs
    uint64_t o_full;
    uint64_t l_full[2];      // per query tile: the partial row sums of the 8 warps are in shared memory
    uint64_t out_filled[2];
    uint32_t tmem_base;
    uint32_t abort_flag;
    uint32_t prior_failure;
};
static_assert(sizeof(Barriers) <= 256, "barrier block must fit its slot");

// The bounded wait of the other kernels, but expanded in place: where a thread holds a row of scores in registers,
// a call would spill them around it.
__device__ __forceinline__ bool wait_in_place(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag, uint32_t site) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
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

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
attn_onepass_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o, int N,
                    int row_blocks_per_head, float scale_log2e) {
    using L = Smem<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    Barriers* bars = reinterpret_cast<Barriers*>(smem + L::kBarOff);
    volatile uint32_t* abort_flag = &bars->abort_flag;

    if (threadIdx.x == 0) bars->prior_failure = *reinterpret_cast<volatile unsigned int*>(&g_attnw_status);
    __syncthreads();
    if (bars->prior_failure != 0u) return;  // an earlier CTA gave up: do not queue more waits behind it

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int bh = blockIdx.x / row_blocks_per_head;
    const int row0 = (blockIdx.x % row_blocks_per_head) * kRowsPerCta;
    const int T = (N + kTile - 1) / kTile;  // key tiles
    const bool tile_active[2] = {row0 < N, row0 + kTile < N};

    // ---- set-up ------------------------------------------------------------------------------
    if (threadIdx.x == 0) {
        ptx::mbar_init(&bars->q_full, 1);
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(&bars->k_full[s], 1);
            ptx::mbar_init(&bars->k_empty[s], 1);
        }
        for (int q = 0; q < 2; ++q) {
            ptx::mbar_init(&bars->s_full[q], 1);
            ptx::mbar_init(&bars->s_free[q], 8);
            ptx::mbar_init(&bars->p_full[q], 8);
            ptx::mbar_init(&bars->p_free[q], 1);
            ptx::mbar_init(&bars->l_full[q], 8);
            ptx::mbar_init(&bars->out_filled[q], 7);
        }
        ptx::mbar_init(&bars->o_full, 1);
        bars->abort_flag = 0;
        ptx::mbar_fence_init();
    }
    if (warp == kProducer && lane == 0) {
        ptx::prefetch_tensormap(&tm_q);
        ptx::prefetch_tensormap(&tm_k);
        ptx::prefetch_tensormap(&tm_v);
        ptx::prefetch_tensormap(&tm_o);
    }
    if (warp == kMma) {
        ptx::tmem_alloc(&bars->tmem_base, kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_base;
    // tensor memory: per query tile q, scores in columns [256 q, 256 q + 128), O in [256 q + 128, 256 q + 128 + d)

    if (warp == kProducer) {
        // ================= TMA producer: Q once, then K_0, [K_{j+1}, V_j] for j = 0 .. T-1 =================
        if (lane == 0) {
            const uint64_t keep = ptx::policy_evict_last();
            int n_active = (tile_active[0] ? 1 : 0) + (tile_active[1] ? 1 : 0);
            ptx::mbar_expect_tx(&bars->q_full, static_cast<uint32_t>(n_active * L::kTileBytes));
            for (int q = 0; q < 2; ++q)
                if (tile_active[q])
                    for (int a = 0; a < L::kAtoms; ++a)
                        ptx::tma_load_3d(smem + L::kQOff + q * L::kTileBytes + a * L::kAtomBytes, &tm_q, &bars->q_full,
                                         a * 64, row0 + q * kTile, bh, keep);
            int n = 0;
            bool ok = true;
            auto load = [&](const CUtensorMap* map, int kt) {
                const int s = n % kStages;
                ok = fused_wait(&bars->k_empty[s], (static_cast<uint32_t>(n / kStages) & 1u) ^ 1u, abort_flag, kSiteProducerEmpty);
                if (!ok) return;
                ptx::mbar_expect_tx(&bars->k_full[s], static_cast<uint32_t>(L::kTileBytes));
                for (int a = 0; a < L::kAtoms; ++a)
                    ptx::tma_load_3d(smem + L::kKOff + s * L::kTileBytes + a * L::kAtomBytes, map, &bars->k_full[s], a * 64,
                                     kt * kTile, bh, keep);
                ++n;
            };
            load(&tm_k, 0);
            for (int j = 0; ok && j < T; ++j) {
                if (j + 1 < T) load(&tm_k, j + 1);
                if (ok) load(&tm_v, j);
            }
            if (*abort_flag) {
                // Unwinding: let the copies already in flight land before shared memory is released.
                const int first = n > kStages ? n - kStages : 0;
                for (int it = first; it < n; ++it) {
                    const long long t0 = clock64();
                    while (!ptx::mbar_try_wait(&bars->k_full[it % kStages], static_cast<uint32_t>(it / kStages) & 1u) &&
                           clock64() - t0 < kWaitLimitCycles / 8) {
                    }
                }
                const long long t0 = clock64();
                while (!ptx::mbar_try_wait(&bars->q_full, 0) && clock64() - t0 < kWaitLimitCycles / 8) {
                }
            }
        }
    } else if (warp == kMma) {
        // ================= MMA issuer (warp-uniform loop, one elected lane issues) =================
        constexpr uint32_t idesc_s = ptx::umma_idesc_bf16_f32(kTile, kTile);
        constexpr uint32_t idesc_o = ptx::umma_idesc_bf16_f32(kTile, D) | (1u << 16);  // B operand MN-major
        const uint32_t q_addr = ptx::smem_u32(smem + L::kQOff);
        const uint32_t k_addr = ptx::smem_u32(smem + L::kKOff);
        const uint32_t p_addr = ptx::smem_u32(smem + L::kPOff);
        bool ok = __all_sync(0xffffffffu, fused_wait(&bars->q_full, 0, abort_flag, kSiteMmaQ));
        int n = 0;  // ring counter, in step with the producer
        auto scores = [&](uint32_t j) {  // S_q = Q_q K_j^T for both query tiles
            const int s = n % kStages;
            ok = __all_sync(0xffffffffu, fused_wait(&bars->k_full[s], static_cast<uint32_t>(n / kStages) & 1u, abort_flag,
                                                    kSiteMmaKFull));
            if (!ok) return;
            const uint32_t b_addr = k_addr + static_cast<uint32_t>(s * L::kTileBytes);
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                if (!tile_active[q]) continue;
                // the row threads have the scores of tile j - 1 in registers
                ok = __all_sync(0xffffffffu, fused_wait(&bars->s_free[q], (j & 1u) ^ 1u, abort_flag, kSiteMmaSFree));
                if (!ok) return;
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(q * 2 * kTile);
                const uint32_t a_addr = q_addr + static_cast<uint32_t>(q * L::kTileBytes);
                if (ptx::elect_one()) {
#pragma unroll
                    for (int k = 0; k < D / 16; ++k) {
                        const uint32_t off = static_cast<uint32_t>((k >> 2) * L::kAtomBytes + (k & 3) * 32);
                        ptx::umma_f16_ss(d_tmem, ptx::umma_desc_kmajor_sw128(a_addr + off),
                                         ptx::umma_desc_kmajor_sw128(b_addr + off), idesc_s, k > 0 ? 1u : 0u);
                    }
                    ptx::umma_commit(&bars->s_full[q]);
                }
                __syncwarp();
            }
            if (ptx::elect_one()) ptx::umma_commit(&bars->k_empty[s]);
            __syncwarp();
            ++n;
        };
        if (ok) scores(0u);
        for (int j = 0; ok && j < T; ++j) {
            // the scores of tile j + 1 first: the tensor pipe computes them while the row threads exponentiate tile j
            if (j + 1 < T) scores(static_cast<uint32_t>(j) + 1u);
            if (!ok) break;
            const int s = n % kStages;
            ok = __all_sync(0xffffffffu, fused_wait(&bars->k_full[s], static_cast<uint32_t>(n / kStages) & 1u, abort_flag,
                                                    kSiteMmaKFull));
            if (!ok) break;
            const uint32_t v_addr = k_addr + static_cast<uint32_t>(s * L::kTileBytes);
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                if (!tile_active[q]) continue;
                ok = __all_sync(0xffffffffu, fused_wait(&bars->p_full[q], static_cast<uint32_t>(j) & 1u, abort_flag, kSiteMmaPFull));
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t o_tmem = tmem_base + static_cast<uint32_t>((q * 2 + 1) * kTile);
                const uint32_t a_base = p_addr + static_cast<uint32_t>(q * L::kPBytes);
                if (ptx::elect_one()) {
#pragma unroll
                    for (int kk = 0; kk < kTile / 16; ++kk) {  // 16 keys per instruction
                        const uint32_t a_off = static_cast<uint32_t>((kk >> 2) * L::kAtomBytes + (kk & 3) * 32);
                        ptx::umma_f16_ss(o_tmem, ptx::umma_desc_kmajor_sw128(a_base + a_off),
                                         av::umma_desc_mnmajor_sw128(v_addr + static_cast<uint32_t>(kk * 16 * 128), L::kAtomBytes),
                                         idesc_o, (j > 0 || kk > 0) ? 1u : 0u);
                    }
                    ptx::umma_commit(&bars->p_free[q]);
                }
                __syncwarp();
            }
            if (!ok) break;
            if (ptx::elect_one()) ptx::umma_commit(&bars->k_empty[s]);
            __syncwarp();
            ++n;
        }
        if (ok && ptx::elect_one()) ptx::umma_commit(&bars->o_full);
        __syncwarp();
    } else if (warp < kSmWarps) {
        // ================= Softmax warps: two threads per query row, 64 key columns of a tile each =================
        const int q = warp >> 3;
        const int half = (warp >> 2) & 1;
        const int quarter = warp & 3;
        if (tile_active[q]) {
            const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + static_cast<uint32_t>(q * 2 * kTile);
            const uint32_t t_own = t_lane + static_cast<uint32_t>(half * kHalf);
            const uint32_t t_other = t_lane + static_cast<uint32_t>((half ^ 1) * kHalf);
            const uint32_t o_own = t_lane + static_cast<uint32_t>(kTile + half * (D / 2));  // this thread's D/2 columns of O
            const float c2 = scale_log2e;
            const uint64_t c2c2 = ptx::pack2(c2, c2);
            // this row in the P tile's atom of this column half (64 keys = 128 bytes, 16-byte pieces XOR-swizzled)
            const int row = quarter * 32 + lane;
            const uint32_t p_tile = ptx::smem_u32(smem + L::kPOff + q * L::kPBytes);
            const uint32_t p_row = p_tile + static_cast<uint32_t>(half * L::kAtomBytes + row * 128);
            const uint32_t sw = static_cast<uint32_t>(lane & 7);
            float smax = -3.0e38f;  // running maximum of the raw scores of this row (all columns: both threads of a row
                                    // compute it, each from the whole tile, so they agree without an exchange)
            float mb = -3.0e38f;    // the offset the weights, l and O's row are relative to (follows smax * c2 lazily)
            float l = 0.0f;         // sum of this thread's weights
            bool ok = true;

            for (int j = 0; ok && j < T; ++j) {
                ok = __all_sync(0xffffffffu, fused_wait(&bars->s_full[q], static_cast<uint32_t>(j) & 1u, abort_flag, kSiteSFull));
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const int valid = N - j * kTile;  // key columns of this tile that exist
                // ---- maximum of the other thread's 64 columns (read and dropped) ----
                float mo = -3.0e38f;
#pragma unroll
                for (int c = 0; c < kHalf / kChunk; ++c) {
                    uint32_t r[kChunk];
                    ptx::tmem_ld_32x32b_x32(t_other + static_cast<uint32_t>(c * kChunk), r);
                    ptx::tmem_wait_ld();
                    if (valid < kTile) {
#pragma unroll
                        for (int i = 0; i < kChunk; ++i)
                            if ((half ^ 1) * kHalf + c * kChunk + i >= valid) r[i] = __float_as_uint(-3.0e38f);
                    }
                    float m0 = __uint_as_float(r[0]), m1 = __uint_as_float(r[1]), m2 = __uint_as_float(r[2]), m3 = __uint_as_float(r[3]);
#pragma unroll
                    for (int i = 4; i < kChunk; i += 8) {
                        m0 = ptx::max3(m0, __uint_as_float(r[i + 0]), __uint_as_float(r[i + 1]));
                        m1 = ptx::max3(m1, __uint_as_float(r[i + 2]), __uint_as_float(r[i + 3]));
                        if (i + 4 < kChunk) {
                            m2 = ptx::max3(m2, __uint_as_float(r[i + 4]), __uint_as_float(r[i + 5]));
                            m3 = ptx::max3(m3, __uint_as_float(r[i + 6]), __uint_as_float(r[i + 7]));
                        }
                    }
                    mo = fmaxf(mo, ptx::max3(fmaxf(m0, m1), m2, m3));
                }
                // ---- this thread's 64 scores into registers; the buffer goes back to the MMA issuer at once ----
                float s[kHalf];
                {
                    uint32_t r0[kChunk], r1[kChunk];
                    ptx::tmem_ld_32x32b_x32(t_own, r0);
                    ptx::tmem_ld_32x32b_x32(t_own + kChunk, r1);
                    ptx::tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < kChunk; ++i) {
                        s[i] = __uint_as_float(r0[i]);
                        s[kChunk + i] = __uint_as_float(r1[i]);
                    }
                }
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&bars->s_free[q]);
                if (valid < kTile) {
#pragma unroll
                    for (int i = 0; i < kHalf; ++i)
                        if (half * kHalf + i >= valid) s[i] = -3.0e38f;
                }
                // ---- row maximum, lazy offset ----
                float m0 = s[0], m1 = s[1], m2 = s[2], m3 = s[3];
#pragma unroll
                for (int i = 4; i < kHalf; i += 8) {
                    m0 = ptx::max3(m0, s[i + 0], s[i + 1]);
                    m1 = ptx::max3(m1, s[i + 2], s[i + 3]);
                    if (i + 4 < kHalf) {
                        m2 = ptx::max3(m2, s[i + 4], s[i + 5]);
                        m3 = ptx::max3(m3, s[i + 6], s[i + 7]);
                    }
                }
                smax = ptx::max3(smax, mo, ptx::max3(fmaxf(m0, m1), m2, m3));
                const float mb_cand = fmaxf(smax * c2, -3.0e38f);
                const bool move = j == 0 || mb_cand - mb > kLazy;
                // the P tile and O are free once the MMAs of the previous key tile are complete
                ok = __all_sync(0xffffffffu, wait_in_place(&bars->p_free[q], (static_cast<uint32_t>(j) & 1u) ^ 1u, abort_flag, kSitePFree));
                if (!ok) break;
                if (j == 0) {
                    mb = mb_cand;
                } else if (__any_sync(0xffffffffu, move)) {
                    // rescale this thread's part of O's row and l to the new offset (factor 1 for the rows of the warp
                    // that do not move; the other thread of the row takes the same decision)
                    const float alpha = move ? ptx::ex2_approx(mb - mb_cand) : 1.0f;
                    if (move) mb = mb_cand;
                    l *= alpha;
                    ptx::tc_fence_after_sync();
#pragma unroll 1
                    for (int c = 0; c < D / 2; c += 8) {  // 8 columns at a time: the row of scores stays in registers
                        uint32_t r[8];
                        ptx::tmem_ld_32x32b_x8(o_own + static_cast<uint32_t>(c), r);
                        ptx::tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 8; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
                        ptx::tmem_st_32x32b_x8(o_own + static_cast<uint32_t>(c), r);
                    }
                    ptx::tmem_wait_st();
                }
                // ---- weights: p = 2^(c2 s - mb) (below 2^8), row sum, bf16, into the P tile ----
                const uint64_t nmb2 = ptx::pack2(-mb, -mb);
                uint64_t acc[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
                for (int g = 0; g < kHalf / 8; ++g) {  // 8 keys = one 16-byte piece of the row
                    float p[8];
#pragma unroll
                    for (int i = 0; i < 8; i += 2) {
                        float x0, x1;
                        ptx::unpack2(ptx::fma2(ptx::pack2(s[g * 8 + i], s[g * 8 + i + 1]), c2c2, nmb2), x0, x1);
                        p[i] = ptx::ex2_approx(x0);
                        p[i + 1] = ptx::ex2_approx(x1);
                        if (valid < kTile) {  // columns beyond N: weight zero
                            p[i] = (half * kHalf + g * 8 + i < valid) ? p[i] : 0.0f;
                            p[i + 1] = (half * kHalf + g * 8 + i + 1 < valid) ? p[i + 1] : 0.0f;
                        }
                        acc[(i >> 1) & 3] = ptx::add2(acc[(i >> 1) & 3], ptx::pack2(p[i], p[i + 1]));
                    }
                    ptx::st_shared_v4(p_row + ((static_cast<uint32_t>(g) ^ sw) << 4), ptx::pack_bf16x2(p[0], p[1]),
                                      ptx::pack_bf16x2(p[2], p[3]), ptx::pack_bf16x2(p[4], p[5]), ptx::pack_bf16x2(p[6], p[7]));
                }
                float a0, a1, a2, a3;
                ptx::unpack2(ptx::add2(acc[0], acc[1]), a0, a1);
                ptx::unpack2(ptx::add2(acc[2], acc[3]), a2, a3);
                l += (a0 + a1) + (a2 + a3);
                ptx::tc_fence_before_sync();  // orders the rescale of O before the MMAs that accumulate into it
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&bars->p_full[q]);
            }

            // ---- epilogue: O / l -> bf16 -> the P tile's shared memory -> TMA stores ----
            if (ok) ok = __all_sync(0xffffffffu, fused_wait(&bars->o_full, 0, abort_flag, kSiteOFull));
            if (ok) {
                // every MMA is complete: the K / V ring is free and carries the two partial row sums to each other
                float* lx = reinterpret_cast<float*>(smem + L::kKOff);
                lx[(q * 2 + half) * kTile + row] = l;
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&bars->l_full[q]);
                ok = __all_sync(0xffffffffu, fused_wait(&bars->l_full[q], 0, abort_flag, kSiteLFull));
            }
            if (ok) {
                const float* lx = reinterpret_cast<const float*>(smem + L::kKOff);
                const float inv_l = 1.0f / (l + lx[(q * 2 + (half ^ 1)) * kTile + row]);
                ptx::tc_fence_after_sync();
#pragma unroll 1
                for (int c = 0; c < D / 2 / kChunk; ++c) {
                    float o[kChunk];
                    load_chunk(o_own + static_cast<uint32_t>(c * kChunk), o);
                    const int col = half * (D / 2) + c * kChunk;  // first of these 32 columns of O
                    const uint32_t dst = p_tile + static_cast<uint32_t>((col >> 6) * L::kAtomBytes + row * 128);
                    const uint32_t piece0 = static_cast<uint32_t>((col & 63) >> 3);
#pragma unroll
                    for (int g = 0; g < 4; ++g)
                        ptx::st_shared_v4(dst + (((piece0 + static_cast<uint32_t>(g)) ^ sw) << 4),
                                          ptx::pack_bf16x2(o[g * 8 + 0] * inv_l, o[g * 8 + 1] * inv_l),
                                          ptx::pack_bf16x2(o[g * 8 + 2] * inv_l, o[g * 8 + 3] * inv_l),
                                          ptx::pack_bf16x2(o[g * 8 + 4] * inv_l, o[g * 8 + 5] * inv_l),
                                          ptx::pack_bf16x2(o[g * 8 + 6] * inv_l, o[g * 8 + 7] * inv_l));
                }
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (quarter == 0 && half == 0) {
                    ok = __all_sync(0xffffffffu, fused_wait(&bars->out_filled[q], 0, abort_flag, kSiteOutFilled));
                    if (ok && lane == 0) {
                        for (int a = 0; a < L::kAtoms; ++a)
                            ptx::tma_store_3d(&tm_o, p_tile + static_cast<uint32_t>(a * L::kAtomBytes), a * 64, row0 + q * kTile, bh,
                                              ptx::policy_evict_first());
                        ptx::bulk_commit_group();
                        ptx::bulk_wait_group<0>();
                    }
                } else if (lane == 0) {
                    ptx::mbar_arrive(&bars->out_filled[q]);
                }
            }
        }
    }

    // ---- teardown: every role falls through to here, also after a wait gave up ----
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == kMma) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace av1
}  // namespace attnw
