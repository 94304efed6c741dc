// Fused attention O = Softmax(scale * Q K^T) V for sm_100a: Attention(Q, K, V) of Section IV, the product with V
// that the paper leaves as future work (Section VIII), without ever writing the attention weights to HBM.
//
// The structure is the two-pass kernel of attnw_fused.cuh: a CTA owns 256 query rows (two tiles that share every
// key tile); pass 1 streams the key tiles and keeps, per row, the running maximum and the sum of exponentials
// (Eq. 1); pass 2 streams them again, recomputes each score tile on the tensor cores and forms the normalised
// weights p = 2^(c s - (mb + log2 l)) - but instead of staging them for a TMA store it leaves each 128 x 128 tile
// of weights in shared memory, rounded to bf16, in exactly the 128-byte-swizzled K-major layout an MMA A operand
// has, and the MMA issuer multiplies it with the value tile: O(128 x d, fp32 in tensor memory) += P V_j.  Because
// the weights are already normalised, O needs no rescaling at any point.  The value tile is used as it arrives
// from TMA ([128 keys x d], d contiguous): an MN-major B operand.
//   tensor memory, pass 2: per query tile 128 columns for the scores and d columns for O (2 x (128 + 128) = 512)
//   shared memory: the staging buffers of the two-pass kernel hold the P tiles; the key ring also carries V tiles
// Valid for any N >= 1, d in {64, 128}; Q, K, V, O bf16 [B, H, N, d].
#pragma once
#include "attnw_fused.cuh"

namespace attnw {
namespace av {

enum : uint32_t {  // wait sites of this kernel (low byte of the status word)
    kSiteProducerEmpty = 80,
    kSiteMmaQ = 81,
    kSiteMmaKFull = 82,
    kSiteMmaAccEmpty = 83,
    kSiteMmaPFull = 84,
    kSiteSoftmaxStats = 85,
    kSiteSoftmaxNorm = 86,
    kSitePFree = 87,
    kSiteOFull = 88,
    kSiteOutFilled = 89,
};

struct Barriers {
    uint64_t q_full;
    uint64_t k_full[6];
    uint64_t k_empty[6];
    uint64_t s_full[2][2];   // [query tile][accumulator buffer]; pass 2 uses buffer 0 only
    uint64_t s_empty[2][2];
    uint64_t p_full[2];      // the 8 Softmax warps of a query tile have written its P tile
    uint64_t p_free[2];      // the MMAs that read the P tile are complete
    uint64_t o_full;         // every MMA into O is complete
    uint64_t out_filled[4];  // epilogue: a staging box is ready for its store
    uint32_t tmem_base;
    uint32_t abort_flag;
    uint32_t prior_failure;
};
static_assert(sizeof(Barriers) <= 256, "barrier block must fit its slot");

// Shared-memory descriptor of an MN-major operand in 128-byte-swizzled atoms of [8 K-rows x 64 MN-elements]:
// consecutive 8-row groups along K are 1024 bytes apart, consecutive 64-element blocks along MN `mn_block_bytes`.
__device__ __forceinline__ uint64_t umma_desc_mnmajor_sw128(uint32_t smem_addr, uint32_t mn_block_bytes) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>((mn_block_bytes >> 4) & 0x3FFFu) << 16;  // leading byte offset
    d |= static_cast<uint64_t>(1024 >> 4) << 32;                        // stride byte offset
    d |= static_cast<uint64_t>(1) << 46;                                // descriptor version (sm_100)
    d |= static_cast<uint64_t>(2) << 61;                                // layout: 128-byte swizzle
    return d;
}

template <int D>
__global__ void __launch_bounds__(kFusedThreads, 1)
attn_fused_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                  const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o, int N,
                  int row_blocks_per_head, float scale_log2e) {
    using L = FusedSmem<D>;
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
    const int T = (N + kTile - 1) / kTile;  // key tiles per pass
    const bool tile_active[2] = {row0 < N, row0 + kTile < N};
    const uint32_t u0 = static_cast<uint32_t>((T + 1) / 2);  // uses of accumulator buffer 0 in pass 1
    const uint32_t u1 = static_cast<uint32_t>(T / 2);        // ... of buffer 1, whose columns hold O in pass 2

    // ---- set-up ------------------------------------------------------------------------------
    if (threadIdx.x == 0) {
        ptx::mbar_init(&bars->q_full, 1);
        for (int s = 0; s < L::kStages; ++s) {
            ptx::mbar_init(&bars->k_full[s], 1);
            ptx::mbar_init(&bars->k_empty[s], 1);
        }
        for (int q = 0; q < 2; ++q) {
            for (int b = 0; b < 2; ++b) {
                ptx::mbar_init(&bars->s_full[q][b], 1);
                ptx::mbar_init(&bars->s_empty[q][b], 8);  // one arrival per Softmax warp of the tile
            }
            ptx::mbar_init(&bars->p_full[q], 8);
            ptx::mbar_init(&bars->p_free[q], 1);
        }
        ptx::mbar_init(&bars->o_full, 1);
        for (int g = 0; g < 4; ++g) ptx::mbar_init(&bars->out_filled[g], D == 128 ? 3 : 7);
        bars->abort_flag = 0;
        ptx::mbar_fence_init();
    }
    if (warp == kProducerWarp && lane == 0) {
        ptx::prefetch_tensormap(&tm_q);
        ptx::prefetch_tensormap(&tm_k);
        ptx::prefetch_tensormap(&tm_v);
        ptx::prefetch_tensormap(&tm_o);
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
        // Ring order: K_0 .. K_{T-1} (pass 1), then K_0, [K_{j+1}, V_j] for j = 0 .. T-1 (pass 2: the scores of tile
        // j + 1 are issued before the product of tile j, see the MMA issuer).
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
                const int s = n % L::kStages;
                const uint32_t use = static_cast<uint32_t>(n / L::kStages);
                ok = fused_wait(&bars->k_empty[s], (use & 1u) ^ 1u, abort_flag, kSiteProducerEmpty);
                if (!ok) return;
                ptx::mbar_expect_tx(&bars->k_full[s], static_cast<uint32_t>(L::kTileBytes));
                for (int a = 0; a < L::kAtoms; ++a)
                    ptx::tma_load_3d(smem + L::kKOff + s * L::kTileBytes + a * L::kAtomBytes, map, &bars->k_full[s], a * 64,
                                     kt * kTile, bh, keep);
                ++n;
            };
            for (int kt = 0; ok && kt < T; ++kt) load(&tm_k, kt);
            if (ok) load(&tm_k, 0);
            for (int j = 0; ok && j < T; ++j) {
                if (j + 1 < T) load(&tm_k, j + 1);
                if (ok) load(&tm_v, j);
            }
            if (*abort_flag) {
                // Unwinding: let the copies already in flight land before shared memory is released.
                const int first = n > L::kStages ? n - L::kStages : 0;
                for (int it = first; it < n; ++it) {
                    const long long t0 = clock64();
                    while (!ptx::mbar_try_wait(&bars->k_full[it % L::kStages], static_cast<uint32_t>(it / L::kStages) & 1u) &&
                           clock64() - t0 < kWaitLimitCycles / 8) {
                    }
                }
                const long long t0 = clock64();
                while (!ptx::mbar_try_wait(&bars->q_full, 0) && clock64() - t0 < kWaitLimitCycles / 8) {
                }
            }
        }
    } else if (warp == kMmaWarp) {
        // ================= MMA issuer (warp-uniform loop, one elected lane issues) =================
        constexpr uint32_t idesc_s = ptx::umma_idesc_bf16_f32(kTile, kTile);
        constexpr uint32_t idesc_o = ptx::umma_idesc_bf16_f32(kTile, D) | (1u << 16);  // B operand MN-major
        const uint32_t q_addr = ptx::smem_u32(smem + L::kQOff);
        const uint32_t k_addr = ptx::smem_u32(smem + L::kKOff);
        const uint32_t p_addr = ptx::smem_u32(smem + L::kOutOff);
        bool ok = __all_sync(0xffffffffu, fused_wait(&bars->q_full, 0, abort_flag, kSiteMmaQ));
        int n = 0;  // ring counter, in step with the producer
        // scores of one key tile for both query tiles into accumulator buffer `buf`, use number `use` of that buffer
        auto scores = [&](int buf, uint32_t use) {
            const int s = n % L::kStages;
            ok = __all_sync(0xffffffffu, fused_wait(&bars->k_full[s], static_cast<uint32_t>(n / L::kStages) & 1u, abort_flag,
                                                    kSiteMmaKFull));
            if (!ok) return;
            const uint32_t b_addr = k_addr + static_cast<uint32_t>(s * L::kTileBytes);
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                if (!tile_active[q]) continue;
                ok = __all_sync(0xffffffffu, fused_wait(&bars->s_empty[q][buf], (use & 1u) ^ 1u, abort_flag, kSiteMmaAccEmpty));
                if (!ok) return;
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>((q * 2 + buf) * kTile);
                const uint32_t a_addr = q_addr + static_cast<uint32_t>(q * L::kTileBytes);
                if (ptx::elect_one()) {
#pragma unroll
                    for (int k = 0; k < D / 16; ++k) {
                        const uint32_t off = static_cast<uint32_t>((k >> 2) * L::kAtomBytes + (k & 3) * 32);
                        ptx::umma_f16_ss(d_tmem, ptx::umma_desc_kmajor_sw128(a_addr + off),
                                         ptx::umma_desc_kmajor_sw128(b_addr + off), idesc_s, k > 0 ? 1u : 0u);
                    }
                    ptx::umma_commit(&bars->s_full[q][buf]);
                }
                __syncwarp();
            }
            if (ptx::elect_one()) ptx::umma_commit(&bars->k_empty[s]);
            __syncwarp();
            ++n;
        };
        // ---- pass 1 ----
        for (int it = 0; ok && it < T; ++it) scores(it & 1, static_cast<uint32_t>(it >> 1));
        // ---- pass 2: scores of tile j + 1 are issued before the product of tile j, so that the tensor pipe works
        //      on them while the Softmax warps turn the scores of tile j into weights ----
        if (ok) scores(0, u0);
        for (int j = 0; ok && j < T; ++j) {
            if (j + 1 < T) scores(0, u0 + static_cast<uint32_t>(j) + 1u);
            if (!ok) break;
            const int s = n % L::kStages;
            ok = __all_sync(0xffffffffu, fused_wait(&bars->k_full[s], static_cast<uint32_t>(n / L::kStages) & 1u, abort_flag,
                                                    kSiteMmaKFull));
            if (!ok) break;
            const uint32_t v_addr = k_addr + static_cast<uint32_t>(s * L::kTileBytes);
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                if (!tile_active[q]) continue;
                if (j == 0 && u1 > 0) {  // O takes the columns of buffer 1: its last scores of pass 1 must have been read
                    ok = __all_sync(0xffffffffu, fused_wait(&bars->s_empty[q][1], (u1 - 1u) & 1u, abort_flag, kSiteMmaAccEmpty));
                    if (!ok) break;
                }
                ok = __all_sync(0xffffffffu, fused_wait(&bars->p_full[q], static_cast<uint32_t>(j) & 1u, abort_flag, kSiteMmaPFull));
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t o_tmem = tmem_base + static_cast<uint32_t>((q * 2 + 1) * kTile);
                const uint32_t a_base = p_addr + static_cast<uint32_t>(q * 2 * 4 * kStageBoxBytes);  // two atoms of 64 keys
                if (ptx::elect_one()) {
#pragma unroll
                    for (int kk = 0; kk < kTile / 16; ++kk) {  // 16 keys per instruction
                        const uint32_t a_off = static_cast<uint32_t>((kk >> 2) * 4 * kStageBoxBytes + (kk & 3) * 32);
                        ptx::umma_f16_ss(o_tmem, ptx::umma_desc_kmajor_sw128(a_base + a_off),
                                         umma_desc_mnmajor_sw128(v_addr + static_cast<uint32_t>(kk * 16 * 128), L::kAtomBytes),
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
    } else if (warp < kSoftmaxWarps) {
        // ================= Softmax warps =================
        // warp = 8*q + 4*half + quarter: query tile q, column half of every key tile, TMEM lane quarter.
        const int q = warp >> 3;
        const int half = (warp >> 2) & 1;
        const int quarter = warp & 3;
        if (tile_active[q]) {
            const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + static_cast<uint32_t>(q * 2 * kTile);
            const float c2 = scale_log2e;
            const uint64_t c2c2 = ptx::pack2(c2, c2);
            float smax = -3.0e38f;  // running maximum of the raw scores this thread has seen
            float mb = smax;        // the offset the exponentials in l are relative to: fl(smax * c2), finite from the start
            float l = 0.0f;         // running sum of 2^(c2 * s - mb) over this thread's columns
            bool ok = true;

            // ---- pass 1: statistics (Eq. 1: m_i and the denominator), online over key tiles ----
            for (int it = 0; it < T; ++it) {
                const int buf = it & 1;
                ok = __all_sync(0xffffffffu, fused_wait(&bars->s_full[q][buf], static_cast<uint32_t>(it >> 1) & 1u, abort_flag,
                                                        kSiteSoftmaxStats));
                if (!ok) break;
                ptx::tc_fence_after_sync();
#pragma unroll 1
                for (int c = 0; c < kHalf / kChunk; ++c) {
                    float s[kChunk];
                    load_chunk(t_lane + static_cast<uint32_t>(buf * kTile + half * kHalf + c * kChunk), s);
                    if (c == kHalf / kChunk - 1) {  // last read of this accumulator: it may be overwritten now
                        ptx::tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(&bars->s_empty[q][buf]);
                    }
                    const int valid = N - it * kTile - half * kHalf - c * kChunk;  // columns of this chunk that exist
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
                    const float mb_new = fmaxf(new_max * c2, -3.0e38f);
                    l *= ptx::ex2_approx(mb - mb_new);  // rescale by the difference of the two ROUNDED offsets
                    mb = mb_new;
                    smax = new_max;
                    l += ragged ? sum_exp2_chunk<0, true>(s, c2c2, -mb, valid) : sum_exp2_chunk<0, false>(s, c2c2, -mb, valid);
                }
            }

            // ---- merge the two column halves of each row (both threads end with the same values) ----
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

            // ---- pass 2: p = 2^(c2*s - (mb + log2 l)) as bf16 into the P tile; the MMA issuer multiplies it with V ----
            const float shift = mb + ptx::lg2_approx(l);
            const uint64_t nshift2 = ptx::pack2(-shift, -shift);
            const int group = q * 2 + half;  // P atom (64 keys) this warp writes: rows quarter*32 .. +31
            const uint32_t gbuf = ptx::smem_u32(smem + L::kOutOff + group * 4 * kStageBoxBytes);
            const uint32_t my_row = gbuf + static_cast<uint32_t>(quarter * kStageBoxBytes + lane * 128);
            const uint32_t sw = static_cast<uint32_t>(lane & 7);
            const uint32_t row_sw = my_row + (sw << 4);  // 16-byte piece g of the row lives at row_sw ^ (g << 4)
            for (int j = 0; ok && j < T; ++j) {
                ok = __all_sync(0xffffffffu, fused_wait(&bars->s_full[q][0], (u0 + static_cast<uint32_t>(j)) & 1u, abort_flag,
                                                        kSiteSoftmaxNorm));
                if (!ok) break;
                ptx::tc_fence_after_sync();
#pragma unroll 1
                for (int c = 0; c < kHalf / kChunk; ++c) {
                    float s[kChunk];
                    load_chunk(t_lane + static_cast<uint32_t>(half * kHalf + c * kChunk), s);
                    if (c == kHalf / kChunk - 1) {
                        ptx::tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(&bars->s_empty[q][0]);
                    }
#pragma unroll
                    for (int jj = 0; jj < kChunk; jj += 2) {
                        float x0, x1;
                        ptx::unpack2(ptx::fma2(ptx::pack2(s[jj], s[jj + 1]), c2c2, nshift2), x0, x1);
                        s[jj] = ptx::ex2_approx(x0);
                        s[jj + 1] = ptx::ex2_approx(x1);
                    }
                    {   // columns beyond N: weight zero (their value rows are zero-filled, but 0 * inf must not arise)
                        const int valid = N - j * kTile - half * kHalf - c * kChunk;
                        if (valid < kChunk) {
#pragma unroll
                            for (int jj = 0; jj < kChunk; ++jj)
                                if (jj >= valid) s[jj] = 0.0f;
                        }
                    }
                    if (c == 0) {  // the P tile is free once the MMAs of the previous key tile have read it
                        ok = __all_sync(0xffffffffu, fused_wait(&bars->p_free[q], (static_cast<uint32_t>(j) & 1u) ^ 1u, abort_flag,
                                                                kSitePFree));
                        if (!ok) break;
                    }
#pragma unroll
                    for (int g = 0; g < 4; ++g)
                        ptx::st_shared_v4(row_sw ^ (static_cast<uint32_t>(c * 4 + g) << 4),
                                          ptx::pack_bf16x2(s[g * 8 + 0], s[g * 8 + 1]), ptx::pack_bf16x2(s[g * 8 + 2], s[g * 8 + 3]),
                                          ptx::pack_bf16x2(s[g * 8 + 4], s[g * 8 + 5]), ptx::pack_bf16x2(s[g * 8 + 6], s[g * 8 + 7]));
                }
                if (!ok) break;
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&bars->p_full[q]);
            }

            // ---- epilogue: O (fp32, tensor memory) -> bf16 -> staging -> one TMA store per box ----
            if (ok) ok = __all_sync(0xffffffffu, fused_wait(&bars->o_full, 0, abort_flag, kSiteOFull));
            if (ok) {
                ptx::tc_fence_after_sync();
                // D = 128: the warp's column half of O is the box of its group; D = 64: both halves share the box of group 2q
                const int box_group = (D == 128) ? group : q * 2;
                const uint32_t obuf = ptx::smem_u32(smem + L::kOutOff + box_group * 4 * kStageBoxBytes);
                const uint32_t o_row = obuf + static_cast<uint32_t>(quarter * kStageBoxBytes + lane * 128) + (sw << 4);
#pragma unroll 1
                for (int c = 0; c < D / 64; ++c) {
                    float o[kChunk];
                    load_chunk(t_lane + static_cast<uint32_t>(kTile + half * (D / 2) + c * kChunk), o);
                    const int piece0 = (D == 128) ? c * 4 : half * 4;
#pragma unroll
                    for (int g = 0; g < 4; ++g)
                        ptx::st_shared_v4(o_row ^ (static_cast<uint32_t>(piece0 + g) << 4),
                                          ptx::pack_bf16x2(o[g * 8 + 0], o[g * 8 + 1]), ptx::pack_bf16x2(o[g * 8 + 2], o[g * 8 + 3]),
                                          ptx::pack_bf16x2(o[g * 8 + 4], o[g * 8 + 5]), ptx::pack_bf16x2(o[g * 8 + 6], o[g * 8 + 7]));
                }
                ptx::fence_proxy_async_smem();
                __syncwarp();
                const bool issuer = quarter == 0 && (D == 128 || half == 0);
                if (issuer) {
                    ok = __all_sync(0xffffffffu, fused_wait(&bars->out_filled[box_group], 0, abort_flag, kSiteOutFilled));
                    if (ok && lane == 0) {
                        ptx::tma_store_3d(&tm_o, obuf, (D == 128) ? half * 64 : 0, row0 + q * kTile, bh, ptx::policy_evict_first());
                        ptx::bulk_commit_group();
                        ptx::bulk_wait_group<0>();
                    }
                } else if (lane == 0) {
                    ptx::mbar_arrive(&bars->out_filled[box_group]);
                }
            }
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

}  // namespace av
}  // namespace attnw
