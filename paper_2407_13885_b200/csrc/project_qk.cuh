// Queries and keys from the inputs for sm_100a: Q_h = X W^Q_h, K_h = X W^K_h for every head in one launch - the
// linear transformation in front of the attention weights (Section IV), which the paper leaves to the vendor's
// matmul and names as a step to bring into its own code (Section VIII).  The output is written head-major
// ([B, H, N, d], bf16), exactly what attnw_fused and attn_fused read, so no transposition pass is needed.
//
// A plain dense contraction, so it runs on the tensor cores: a CTA owns a 256 x 256 tile of one of the two
// outputs (256 rows of one batch entry x 256 output features = 2 or 4 heads), four 128 x 128 fp32 accumulators in
// tensor memory (all 512 columns), a 3-stage TMA ring of [256 x 64] slices of X and of the weights (64 KB a stage),
// tcgen05 MMAs of shape 128 x 256 x 16.  Weights are stored [H, d, d_model] (feature c of head h contiguous along
// d_model), which is the K-major B operand TMA can deliver as it is.
#pragma once
#include "attnw_fused.cuh"

namespace attnw {
namespace proj {

constexpr int kRows = 256;        // rows of X per CTA (two MMA row blocks)
constexpr int kCols = 256;        // output features per CTA
constexpr int kKSlice = 64;       // d_model elements per stage: one 128-byte swizzle atom
constexpr int kStages = 3;
constexpr int kGroupCols = 16;    // column tiles walked together (32 MB of weights at d_model = 4096)
constexpr int kEpiWarps = 8;      // TMEM lane quarter (4) x column half (2)
constexpr int kProducer = 8;
constexpr int kMma = 9;
constexpr int kThreads = 320;
constexpr int kAtomBytes = 128 * 128;             // 128 rows x 128 bytes
constexpr int kStageBytes = 4 * kAtomBytes;       // X rows 0-127, X rows 128-255, features 0-127, features 128-255
constexpr int kBarOff = kStages * kStageBytes;
constexpr int kDynamicBytes = kBarOff + 256 + 1024;
static_assert(kDynamicBytes <= 227 * 1024, "shared memory budget");

enum : uint32_t {  // wait sites of this kernel (low byte of the status word)
    kSiteProducerEmpty = 112,
    kSiteMmaFull = 113,
    kSiteEpiAcc = 114,
    kSiteEpiFilled = 115,
};

struct Barriers {
    uint64_t full[kStages], empty[kStages];
    uint64_t acc_full;     // every MMA of the tile is complete
    uint64_t out_filled;   // the 7 warps that do not issue the stores have staged their part of the tile
    uint32_t tmem_base;
    uint32_t abort_flag;
    uint32_t prior_failure;
};
static_assert(sizeof(Barriers) <= 256, "barrier block must fit its slot");

// grid: 2 * col_tiles * B * row_tiles CTAs.  The column tiles (Q's, then K's) are walked in groups of kGroupCols: within
// a group the tiles of one block of rows are neighbours (that block of X is fetched once per group) and the group's
// slice of the weights (kGroupCols x 256 x d_model) is small enough to stay in L2 while all row blocks pass.
__global__ void __launch_bounds__(kThreads, 1)
project_qk_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_wq,
                  const __grid_constant__ CUtensorMap tm_wk, const __grid_constant__ CUtensorMap tm_q,
                  const __grid_constant__ CUtensorMap tm_k, int N, int d_model, int H, int d, int col_tiles, int row_tiles) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    Barriers* bars = reinterpret_cast<Barriers*>(smem + kBarOff);
    volatile uint32_t* abort_flag = &bars->abort_flag;

    if (threadIdx.x == 0) bars->prior_failure = *reinterpret_cast<volatile unsigned int*>(&g_attnw_status);
    __syncthreads();
    if (bars->prior_failure != 0u) return;  // an earlier CTA gave up: do not queue more waits behind it

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int n_x = 2 * col_tiles, n_y = static_cast<int>(gridDim.x) / n_x;
    const int n_groups = (n_x + kGroupCols - 1) / kGroupCols;
    const int group = min(static_cast<int>(blockIdx.x) / (kGroupCols * n_y), n_groups - 1);
    const int in_group = static_cast<int>(blockIdx.x) - group * kGroupCols * n_y;
    const int width = group == n_groups - 1 ? n_x - group * kGroupCols : kGroupCols;
    const int tile_x = group * kGroupCols + in_group % width;
    const int tile_y = in_group / width;
    const bool keys = tile_x >= col_tiles;  // this CTA computes a tile of K, not of Q
    const int c0 = (tile_x - (keys ? col_tiles : 0)) * kCols;  // first output feature (of H * d)
    const int b = tile_y / row_tiles;
    const int r0 = (tile_y % row_tiles) * kRows;
    const int KT = (d_model + kKSlice - 1) / kKSlice;
    const CUtensorMap* tm_w = keys ? &tm_wk : &tm_wq;
    const CUtensorMap* tm_out = keys ? &tm_k : &tm_q;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(&bars->full[s], 1);
            ptx::mbar_init(&bars->empty[s], 1);
        }
        ptx::mbar_init(&bars->acc_full, 1);
        ptx::mbar_init(&bars->out_filled, kEpiWarps - 1);
        bars->abort_flag = 0;
        ptx::mbar_fence_init();
    }
    if (warp == kProducer && lane == 0) {
        ptx::prefetch_tensormap(&tm_x);
        ptx::prefetch_tensormap(tm_w);
        ptx::prefetch_tensormap(tm_out);
    }
    if (warp == kMma) {
        ptx::tmem_alloc(&bars->tmem_base, kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_base;

    if (warp == kProducer) {
        // ================= TMA producer: one [256 x 64] slice of X and one of the weights per stage =================
        if (lane == 0) {
            const uint64_t keep = ptx::policy_evict_last();
            int kt = 0;
            for (; kt < KT; ++kt) {
                const int s = kt % kStages;
                if (!fused_wait(&bars->empty[s], (static_cast<uint32_t>(kt / kStages) & 1u) ^ 1u, abort_flag, kSiteProducerEmpty)) break;
                uint8_t* st = smem + s * kStageBytes;
                ptx::mbar_expect_tx(&bars->full[s], static_cast<uint32_t>(kStageBytes));
                // rows or features beyond the tensor's extent, and d_model's ragged tail, arrive as zeros
                ptx::tma_load_3d(st + 0 * kAtomBytes, &tm_x, &bars->full[s], kt * kKSlice, r0, b, keep);
                ptx::tma_load_3d(st + 1 * kAtomBytes, &tm_x, &bars->full[s], kt * kKSlice, r0 + 128, b, keep);
                ptx::tma_load_3d(st + 2 * kAtomBytes, tm_w, &bars->full[s], kt * kKSlice, c0, 0, keep);
                ptx::tma_load_3d(st + 3 * kAtomBytes, tm_w, &bars->full[s], kt * kKSlice, c0 + 128, 0, keep);
            }
            if (*abort_flag) {
                // Unwinding: let the copies already in flight land before shared memory is released.
                const int first = kt > kStages ? kt - kStages : 0;
                for (int it = first; it < kt; ++it) {
                    const long long t0 = clock64();
                    while (!ptx::mbar_try_wait(&bars->full[it % kStages], static_cast<uint32_t>(it / kStages) & 1u) &&
                           clock64() - t0 < kWaitLimitCycles / 8) {
                    }
                }
            }
        }
    } else if (warp == kMma) {
        // ================= MMA issuer =================
        constexpr uint32_t idesc = ptx::umma_idesc_bf16_f32(128, kCols);
        const uint32_t base = ptx::smem_u32(smem);
        bool ok = true;
        for (int kt = 0; ok && kt < KT; ++kt) {
            const int s = kt % kStages;
            ok = __all_sync(0xffffffffu, fused_wait(&bars->full[s], static_cast<uint32_t>(kt / kStages) & 1u, abort_flag, kSiteMmaFull));
            if (!ok) break;
            ptx::tc_fence_after_sync();
            const uint32_t st = base + static_cast<uint32_t>(s * kStageBytes);
            if (ptx::elect_one()) {
#pragma unroll
                for (int mi = 0; mi < 2; ++mi) {
#pragma unroll
                    for (int k = 0; k < kKSlice / 16; ++k)
                        // A: 128 rows of X; B: 256 features = the two weight atoms, contiguous (8-row groups 1024 bytes apart)
                        ptx::umma_f16_ss(tmem_base + static_cast<uint32_t>(mi * kCols),
                                         ptx::umma_desc_kmajor_sw128(st + static_cast<uint32_t>(mi * kAtomBytes + k * 32)),
                                         ptx::umma_desc_kmajor_sw128(st + static_cast<uint32_t>(2 * kAtomBytes + k * 32)), idesc,
                                         (kt > 0 || k > 0) ? 1u : 0u);
                }
                ptx::umma_commit(&bars->empty[s]);
            }
            __syncwarp();
        }
        if (ok && ptx::elect_one()) ptx::umma_commit(&bars->acc_full);
        __syncwarp();
    } else {
        // ================= Epilogue warps: accumulators -> bf16 -> shared memory -> TMA stores, head-major =================
        const int quarter = warp & 3;
        const int ch = warp >> 2;  // column half of the tile (features ch*128 .. +127)
        const int row = quarter * 32 + lane;
        const uint32_t sw = static_cast<uint32_t>(lane & 7);
        bool ok = __all_sync(0xffffffffu, fused_wait(&bars->acc_full, 0, abort_flag, kSiteEpiAcc));
        if (ok) {
            ptx::tc_fence_after_sync();
            // every load was consumed and every MMA is complete: the ring is free and stages the tile as 2 x 4 boxes of
            // [128 rows x 64 features]
            const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
#pragma unroll 1
            for (int mi = 0; mi < 2; ++mi) {
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    float v[kChunk];
                    load_chunk(t_lane + static_cast<uint32_t>(mi * kCols + ch * 128 + c * kChunk), v);
                    const int atom = ch * 2 + (c >> 1);
                    const uint32_t dst = ptx::smem_u32(smem + (mi * 4 + atom) * kAtomBytes + row * 128);
#pragma unroll
                    for (int g = 0; g < 4; ++g)
                        ptx::st_shared_v4(dst + ((static_cast<uint32_t>((c & 1) * 4 + g) ^ sw) << 4),
                                          ptx::pack_bf16x2(v[g * 8 + 0], v[g * 8 + 1]), ptx::pack_bf16x2(v[g * 8 + 2], v[g * 8 + 3]),
                                          ptx::pack_bf16x2(v[g * 8 + 4], v[g * 8 + 5]), ptx::pack_bf16x2(v[g * 8 + 6], v[g * 8 + 7]));
                }
            }
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (warp == 0) {
                ok = __all_sync(0xffffffffu, fused_wait(&bars->out_filled, 0, abort_flag, kSiteEpiFilled));
                if (ok && lane == 0) {
                    const uint64_t stream_out = ptx::policy_evict_last();  // the attention kernels read Q and K next
                    for (int mi = 0; mi < 2; ++mi) {
                        if (r0 + mi * 128 >= N) continue;
                        for (int atom = 0; atom < 4; ++atom) {
                            const int col = c0 + atom * 64;  // output feature of H * d: head col / d, offset col % d
                            if (col >= H * d) continue;
                            ptx::tma_store_3d(tm_out, ptx::smem_u32(smem + (mi * 4 + atom) * kAtomBytes), col % d, r0 + mi * 128,
                                              b * H + col / d, stream_out);
                        }
                    }
                    ptx::bulk_commit_group();
                    ptx::bulk_wait_group<0>();
                }
            } else if (lane == 0) {
                ptx::mbar_arrive(&bars->out_filled);
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

}  // namespace proj
}  // namespace attnw
