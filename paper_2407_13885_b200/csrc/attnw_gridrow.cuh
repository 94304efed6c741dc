// Grid-row fused attention-weight kernel for sm_100a: the SRAM-resident design of Section VII of the paper
// with the roles of a Tensix grid row taken by a GROUP of CTAs that the kernel forms itself.
//
// The paper lays the score matrix out over a grid of cores; the cores of one grid row hold the pieces of the
// same rows of scores, compute LOCAL row maxima and sums and exchange them to obtain the GLOBAL ones before
// normalising (Section VII; Eq. 1).  Here a group of C = ceil(N / 256) <= 16 CTAs owns a 128-row block of one
// head; CTA r of the group works on the 128 x 256 slab of scores for keys [256 r, 256 r + 256).  Tensor cores
// and exponentials run once per element, and three row blocks are in flight per CTA:
//   tensor-memory columns [0, 256)    two landing slots of 128 columns: the MMA writes float32 scores here; a slot
//                                     goes back to the MMA issuer as soon as its scores are in registers
//   tensor-memory columns [256, 512)  two packed regions (one per stream = row blocks of equal parity): the
//                                     exponentials as f16 pairs, waiting for the row's statistics
// so the next row block's scores are computed, and its exponentials taken, while the statistics of the previous
// ones cross the group.  (f16 keeps 11 bits of e in [0, 1]: 5e-4 relative, next to the 2e-3 of the bf16 result.)
//
// Groups are not hardware clusters (clusters of 8 or 16 CTAs cannot occupy every SM): the grid is launched
// cooperatively with one CTA per SM, consecutive CTAs form a group, and the 16-byte (offset, sum) pair of a row
// travels through L2 as two 8-byte words that each carry a tag {value, tag, value, tag}; a reader accepts a
// pair once both tags name the row block it is waiting for.  No fence, no flag, no atomics: the tag arrives
// with the value in one 8-byte store.  Every poll is bounded.
//
// Roles of a CTA (640 threads, 20 warps; warp w may touch TMEM lanes 32 (w % 4) ...):
//   warps 0-7    exponentials, all eight on ONE row block at a time: two threads per row, thread (row, p) takes the
//                64-column boxes p and p + 2 of the slab: scores to registers, maximum, offset mb, e = 2^(c s - mb),
//                sum, e packed to f16 pairs into the stream's packed region; the thread's (mb, l) to shared memory;
//                the second of a row's two warps to finish merges the halves and posts the row's pair
//   warps 8-11   normalise, stream 0 (12-15: stream 1): a thread owns one row; waits for the C pairs of the row, forms M and 1/L - every CTA reduces redundantly, as
//                the paper's kernel does -, then per box p = e * 2^(mb_box - M) / L (one mixed-precision FMA per
//                element unpacks and scales), rounded to bf16, staged in 128-row boxes
//   warp 16      TMA producer: the CTA's key slab once per head (it stays in shared memory while the group walks
//                the head's row blocks), one 32 KB query tile per row block
//   warp 17      tcgen05.mma issuer (one elected lane), 128 x 128 x 16 per instruction
//   warps 18-19  store issuers, one per stream: one TMA store per filled box; P is written exactly once
// Valid for N <= 4096 keys and bf16 output.
//
// With -DATTNW_TIMELINE=<CTA> one lane per role of that CTA stamps clock64() per row block (events, by index):
//   13 MMA of the block issued | 0 exponentials begin, 2 slot 0 ready, 17/20 load of box k, 16/19 maximum known,
//   18/21 exponentials of box k done, 24/26 packed e stored, 4 halves posted | 10 normalise begins to wait,
//   6 halves seen + pair posted, 11 all pairs seen, 12 box 0 read, 14/15/8/9 box 2 read / staging free / staged /
//   handed to the store issuer, 7 block done.
#pragma once
#include "attnw_resident.cuh"

namespace attnw {
namespace gr {

constexpr int kSlabCols = 256;                       // key columns per CTA and row block
constexpr int kSub = 128;                            // columns per MMA landing slot
constexpr int kSubsPerBlock = kSlabCols / kSub;      // 2 landing slots = tensor-memory columns [0, 256)
constexpr int kPackedCol0 = kSlabCols;               // packed exponentials: columns [256, 512), 128 per stream
constexpr int kPackedCols = kSlabCols / 2;           // two f16 per 32-bit column
constexpr int kBoxCols = 64;                         // columns of one staged store box (128 bytes of bf16)
constexpr int kChunksPerBlock = kSlabCols / kChunk;  // 32-column chunks, each with its own offset
constexpr int kThreads = 640;                        // 8 exponential + 8 normalise warps, producer, MMA issuer, 2 store issuers
constexpr int kNormWarp0 = 8;
constexpr int kNormGroups = 2;                       // normalise warpgroups: one per stream
constexpr int kProducerWarpG = kNormWarp0 + 4 * kNormGroups;
constexpr int kMmaWarpG = kProducerWarpG + 1;
constexpr int kStoreWarpG = kProducerWarpG + 2;
constexpr int kMaxGroupCtas = 16;
constexpr int kMaxN = kSlabCols * kMaxGroupCtas;
constexpr int kXchgDepth = 4;    // row blocks i and i + 4 of a group share exchange entries (see the proof at the poll)

enum : uint32_t {  // wait sites of this kernel (low byte of the status word)
    kSiteGrKEmpty = 32,
    kSiteGrQEmpty = 33,
    kSiteGrQFull = 34,
    kSiteGrKFull = 35,
    kSiteGrSlotFree = 36,
    kSiteGrSFull = 37,
    kSiteGrPosted = 38,
    kSiteGrExchange = 39,
    kSiteGrStageFree = 40,
    kSiteGrStageFilled = 41,
};

template <int D>
struct Smem {
    static constexpr int kQStages = 2;  // query tiles in shared memory (with one, the load of the next tile shows: 1.28 against 1.13 ms)
    static constexpr int kBoxes = (D == 128) ? (kQStages == 1 ? 7 : 5) : 8;  // staged store boxes of 128 rows x 128 bytes, in one ring per stream
    static constexpr int kRing0 = (kBoxes + 1) / 2;    // (a ring has ONE filler: a parity wait is only valid one use ahead)
    static constexpr int kRing1 = kBoxes - kRing0;
    static constexpr int kAtoms = D / 64;
    static constexpr int kAtomBytes = kTile * 128;
    static constexpr int kTileBytes = kAtoms * kAtomBytes;
    static constexpr int kKAtomBytes = kSlabCols * 128;                 // key slab, atom-major: [d / 64][256 keys][128 bytes]
    static constexpr int kKOff = 0;
    static constexpr int kQOff = kKOff + 2 * kTileBytes;                // one query tile per stream
    static constexpr int kOutOff = kQOff + kQStages * kTileBytes;       // staging boxes
    static constexpr int kMbcOff = kOutOff + kBoxes * kBoxBytes;        // float mbc[2 streams][8][128 rows]: offset per box (4 of 8 in use)
    static constexpr int kPartOff = kMbcOff + 2 * kChunksPerBlock * kTile * 4;  // float2 part[2 streams][2 halves][128 rows]
    static constexpr int kBarOff = kPartOff + 2 * 2 * kTile * 8;
    static constexpr int kBytes = kBarOff + 512;
    static constexpr int kDynamicBytes = kBytes + 1024;
};
static_assert(Smem<128>::kDynamicBytes <= 227 * 1024 && Smem<64>::kDynamicBytes <= 227 * 1024, "shared memory budget");

struct Barriers {
    uint64_t k_full, k_empty;
    uint64_t q_full[2], q_empty[2];
    uint64_t s_full[kSubsPerBlock], l_free[kSubsPerBlock];  // landing slots: scores ready / scores taken to registers
    uint64_t pk_free[2][kSlabCols / kBoxCols];              // [stream][box]: the packed exponentials have been read
    uint64_t posted[2];
    uint64_t out_free[8], out_filled[8];
    uint32_t halves_done[2][4];  // [stream][TMEM lane quarter]: exponential warps that have finished a row's halves (never reset)
    uint32_t tmem_base;
    uint32_t abort_flag;
    uint32_t prior_failure;
};
static_assert(sizeof(Barriers) <= 512, "barrier block must fit its slot");

__device__ __forceinline__ void st_message(uint4* p, float a, float b, uint32_t tag) {
    asm volatile("st.relaxed.gpu.global.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(__float_as_uint(a)), "r"(tag),
                 "r"(__float_as_uint(b)), "r"(tag)
                 : "memory");
}
__device__ __forceinline__ uint4 ld_message(const uint4* p) {
    uint4 v;
    asm volatile("ld.relaxed.gpu.global.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}

// xchg: [grid CTAs][kXchgDepth][128 rows] messages of 16 bytes, owned by the library, zero before first use.
// tag_base: tags tag_base + 1 ... tag_base + (row blocks of the longest list) belong to this launch alone.
template <int D>
__global__ void __launch_bounds__(kThreads, 1)
attnw_gridrow_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                     const __grid_constant__ CUtensorMap tm_p, int N, int total_items, int group_ctas, int n_groups,
                     float scale_log2e, uint4* __restrict__ xchg, uint32_t tag_base) {
    using L = Smem<D>;
    constexpr int kBoxes = L::kBoxes;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    Barriers* bars = reinterpret_cast<Barriers*>(smem + L::kBarOff);
    volatile uint32_t* abort_flag = &bars->abort_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int group = static_cast<int>(blockIdx.x) / group_ctas;
    const int rank = static_cast<int>(blockIdx.x) % group_ctas;
    if (group >= n_groups) return;  // CTAs beyond the last whole group have no part in the launch
    const int T = (N + kTile - 1) / kTile;                          // row blocks per head
    const int col0 = rank * kSlabCols;                              // first key of this CTA's slab
    const int width = (N - col0 < kSlabCols) ? N - col0 : kSlabCols;  // keys of the slab that exist (>= 1)
    const int n_sub = (width + kSub - 1) / kSub;                    // MMA slots in use
    const int n_boxes = (width + kBoxCols - 1) / kBoxCols;          // 64-column store boxes in use, 1..4
    const int n_ktiles = (width + kTile - 1) / kTile;               // 128-key tiles of the slab that exist, 1..2
    // The group's list: a contiguous range of (head, row block) items, so that the key slab changes rarely.
    const long long begin_ll = static_cast<long long>(total_items) * group / n_groups;
    const long long end_ll = static_cast<long long>(total_items) * (group + 1) / n_groups;
    const int begin = static_cast<int>(begin_ll);
    const int n_items = static_cast<int>(end_ll - begin_ll);

    // ---- set-up ------------------------------------------------------------------------------
    if (threadIdx.x == 0) {
        ptx::mbar_init(&bars->k_full, 1);
        ptx::mbar_init(&bars->k_empty, 1);
        for (int j = 0; j < kSubsPerBlock; ++j) {
            ptx::mbar_init(&bars->s_full[j], 1);
            ptx::mbar_init(&bars->l_free[j], 8);  // one arrival per exponential warp
        }
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(&bars->q_full[s], 1);
            ptx::mbar_init(&bars->q_empty[s], 1);
            for (int b = 0; b < kSlabCols / kBoxCols; ++b) ptx::mbar_init(&bars->pk_free[s][b], 4);  // the stream's normalise warps
            ptx::mbar_init(&bars->posted[s], 8);  // one arrival per exponential warp
        }
        for (int b = 0; b < kBoxes; ++b) {
            ptx::mbar_init(&bars->out_free[b], 1);
            ptx::mbar_init(&bars->out_filled[b], 4);
        }
        for (int x = 0; x < 8; ++x) (&bars->halves_done[0][0])[x] = 0;
        bars->abort_flag = 0;
        bars->prior_failure = *reinterpret_cast<volatile unsigned int*>(&g_attnw_status);
        ptx::mbar_fence_init();
    }
    if (warp == kProducerWarpG && lane == 0) {
        ptx::prefetch_tensormap(&tm_q);
        ptx::prefetch_tensormap(&tm_k);
        ptx::prefetch_tensormap(&tm_p);
    }
    if (warp == kMmaWarpG) {
        ptx::tmem_alloc(&bars->tmem_base, kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_base;
    const bool run = bars->prior_failure == 0u && n_items > 0;  // an earlier launch step gave up: skip the work

    if (run && warp == kProducerWarpG) {
        // ================= TMA producer =================
        if (lane == 0) {
            const uint64_t keep = ptx::policy_evict_last();
            int cur_bh = -1;
            uint32_t heads = 0;
            int issued = 0;
            for (int i = 0; i < n_items; ++i) {
                const int gi = begin + i, bh = gi / T, rb = gi % T;
                const int s = i & 1;
                const uint32_t u = static_cast<uint32_t>(i) >> 1;
                if (bh != cur_bh) {  // new head: the slab may be replaced once every MMA of the old head has read it
                    if (!fused_wait(&bars->k_empty, (heads & 1u) ^ 1u, abort_flag, kSiteGrKEmpty)) break;
                    ptx::mbar_expect_tx(&bars->k_full, static_cast<uint32_t>(n_ktiles * L::kTileBytes));
                    for (int t = 0; t < n_ktiles; ++t)
                        for (int a = 0; a < L::kAtoms; ++a)
                            ptx::tma_load_3d(smem + L::kKOff + a * L::kKAtomBytes + t * L::kAtomBytes, &tm_k, &bars->k_full,
                                             a * 64, col0 + t * kTile, bh, keep);
                    ++heads;
                    cur_bh = bh;
                }
                const int qs = i % L::kQStages;
                const uint32_t uq = static_cast<uint32_t>(i / L::kQStages);
                if (!fused_wait(&bars->q_empty[qs], (uq & 1u) ^ 1u, abort_flag, kSiteGrQEmpty)) break;
                ptx::mbar_expect_tx(&bars->q_full[qs], static_cast<uint32_t>(L::kTileBytes));
                for (int a = 0; a < L::kAtoms; ++a)
                    ptx::tma_load_3d(smem + L::kQOff + qs * L::kTileBytes + a * L::kAtomBytes, &tm_q, &bars->q_full[qs], a * 64,
                                     rb * kTile, bh, keep);
                issued = i + 1;
            }
            if (*abort_flag) {
                // Unwinding: let the copies already in flight land before shared memory is released.
                const long long t0 = clock64();
                if (heads > 0)
                    while (!ptx::mbar_try_wait(&bars->k_full, (heads - 1u) & 1u) && clock64() - t0 < kWaitLimitCycles / 8) {
                    }
                for (int back = 1; back <= 2 && back <= issued; ++back) {
                    const int i = issued - back;
                    while (!ptx::mbar_try_wait(&bars->q_full[i % L::kQStages], static_cast<uint32_t>(i / L::kQStages) & 1u) &&
                           clock64() - t0 < kWaitLimitCycles / 4) {
                    }
                }
            }
        }
    } else if (run && warp == kMmaWarpG) {
        // ================= MMA issuer (warp-uniform loop, one elected lane issues) =================
        // One slot = 128 rows x kSub keys: D / 16 instructions of shape 128 x kSub x 16.  Both operands come from shared
        // memory, and the query tile is fetched again by every instruction: narrow slots hand tensor memory over sooner
        // but cost shared-memory bandwidth, which this kernel is short of.
        constexpr uint32_t idesc = ptx::umma_idesc_bf16_f32(kTile, kSub);
        const uint32_t q_addr = ptx::smem_u32(smem + L::kQOff);
        const uint32_t k_addr = ptx::smem_u32(smem + L::kKOff);
        int cur_bh = -1;
        uint32_t heads = 0;
        bool ok = true;
        for (int i = 0; ok && i < n_items; ++i) {
            const int gi = begin + i, bh = gi / T;
            const int s = i & 1;
            const uint32_t u = static_cast<uint32_t>(i) >> 1;
            const int qs = i % L::kQStages;
            ok = __all_sync(0xffffffffu, fused_wait(&bars->q_full[qs], static_cast<uint32_t>(i / L::kQStages) & 1u, abort_flag, kSiteGrQFull));
            if (!ok) break;
            if (bh != cur_bh) {
                ok = __all_sync(0xffffffffu, fused_wait(&bars->k_full, heads & 1u, abort_flag, kSiteGrKFull));
                if (!ok) break;
                ++heads;
                cur_bh = bh;
            }
            const bool last_of_head = (i + 1 == n_items) || ((gi + 1) / T != bh);
            if (n_sub == 2) {
                // Both landing slots in one 128 x 256 x 16 instruction per step: the query tile is fetched from shared
                // memory once per row block instead of once per slot (0.7 % of the launch on the headline shape).
                ok = __all_sync(0xffffffffu, fused_wait(&bars->l_free[0], (static_cast<uint32_t>(i) & 1u) ^ 1u, abort_flag, kSiteGrSlotFree)) &&
                     __all_sync(0xffffffffu, fused_wait(&bars->l_free[1], (static_cast<uint32_t>(i) & 1u) ^ 1u, abort_flag, kSiteGrSlotFree));
                if (!ok) break;
                ptx::tc_fence_after_sync();
                if (lane == 0) ATTNW_STAMP(13, i);
                constexpr uint32_t idesc2 = ptx::umma_idesc_bf16_f32(kTile, 2 * kSub);
                const uint32_t a_addr = q_addr + static_cast<uint32_t>(qs * L::kTileBytes);
                if (ptx::elect_one()) {
#pragma unroll
                    for (int k = 0; k < D / 16; ++k) {
                        const uint32_t a_off = static_cast<uint32_t>((k >> 2) * L::kAtomBytes + (k & 3) * 32);
                        const uint32_t b_off = static_cast<uint32_t>((k >> 2) * L::kKAtomBytes + (k & 3) * 32);
                        ptx::umma_f16_ss(tmem_base, ptx::umma_desc_kmajor_sw128(a_addr + a_off),
                                         ptx::umma_desc_kmajor_sw128(k_addr + b_off), idesc2, k > 0 ? 1u : 0u);
                    }
                    ptx::umma_commit(&bars->s_full[0]);
                    ptx::umma_commit(&bars->s_full[1]);
                    ptx::umma_commit(&bars->q_empty[qs]);                // the query tile may be replaced
                    if (last_of_head) ptx::umma_commit(&bars->k_empty);  // ... and the key slab
                }
                __syncwarp();
                continue;
            }
            for (int j = 0; j < n_sub; ++j) {
                // the landing slot is free once the exponential warps have taken the scores of row block i - 1 to registers
                ok = __all_sync(0xffffffffu, fused_wait(&bars->l_free[j], (static_cast<uint32_t>(i) & 1u) ^ 1u, abort_flag, kSiteGrSlotFree));
                if (!ok) break;
                ptx::tc_fence_after_sync();
                if (lane == 0 && j == 0) ATTNW_STAMP(13, i);
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(j * kSub);
                const uint32_t a_addr = q_addr + static_cast<uint32_t>(qs * L::kTileBytes);
                const uint32_t b_addr = k_addr + static_cast<uint32_t>(j * kSub * 128);  // keys kSub j ... of every atom
                if (ptx::elect_one()) {
#pragma unroll
                    for (int k = 0; k < D / 16; ++k) {
                        const uint32_t a_off = static_cast<uint32_t>((k >> 2) * L::kAtomBytes + (k & 3) * 32);
                        const uint32_t b_off = static_cast<uint32_t>((k >> 2) * L::kKAtomBytes + (k & 3) * 32);
                        ptx::umma_f16_ss(d_tmem, ptx::umma_desc_kmajor_sw128(a_addr + a_off),
                                         ptx::umma_desc_kmajor_sw128(b_addr + b_off), idesc, k > 0 ? 1u : 0u);
                    }
                    ptx::umma_commit(&bars->s_full[j]);
                    if (j == n_sub - 1) {
                        ptx::umma_commit(&bars->q_empty[qs]);                // the query tile may be replaced
                        if (last_of_head) ptx::umma_commit(&bars->k_empty);  // ... and the key slab
                    }
                }
                __syncwarp();
            }
        }
    } else if (run && (warp == kStoreWarpG || warp == kStoreWarpG + 1)) {
        // ================= store issuer: one TMA store per filled staging box, in ring order =================
        // Boxes are stored in the order (row block, 64 columns); the boxes of a stream use that stream's ring in turn.
        if (lane == 0) {
            const uint64_t stream_out = ptx::policy_evict_first();
            const uint32_t out_base = ptx::smem_u32(smem + L::kOutOff);
            bool ok = true;
            for (int i = warp - kStoreWarpG; ok && i < n_items; i += 2) {  // one store issuer per stream
                const int gi = begin + i, bh = gi / T, rb = gi % T;
                const int s = i & 1;
                const uint32_t ring = s ? L::kRing1 : L::kRing0, base = s ? L::kRing0 : 0;
                const uint32_t m0 = (static_cast<uint32_t>(i) >> 1) * static_cast<uint32_t>(n_boxes);
                for (int j = 0; j < n_boxes; ++j) {
                    const uint32_t m = m0 + static_cast<uint32_t>(j);
                    const uint32_t box = base + m % ring, use = m / ring;
                    if (!fused_wait(&bars->out_filled[box], use & 1u, abort_flag, kSiteGrStageFilled)) {
                        ok = false;
                        break;
                    }
                    ptx::tma_store_3d(&tm_p, out_base + box * kBoxBytes, col0 + j * kBoxCols, rb * kTile, bh, stream_out);
                    ptx::bulk_commit_group();
                    ptx::bulk_wait_group_read<0>();  // the store has read the box: it may be filled again
                    ptx::mbar_arrive(&bars->out_free[box]);
                }
            }
            ptx::bulk_wait_group<0>();
        }
    } else if (run && warp < kNormWarp0) {
        // ================= exponential warps: TMEM lane quarter = warp % 4, box parity = warp / 4 =================
        // All eight warps work on ONE row block at a time (both streams in turn): two threads per row, one taking the
        // even and one the odd 64-column boxes, so that every scheduler has two warps feeding its MUFU.
        const int par = warp >> 2;
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        // never exactly zero, so that a masked score (-3e38) always lands far below the offset; with scale = 0 every
        // existing score still maps to 2^0
        const float c2 = fmaxf(scale_log2e, 1.0e-30f);
        const uint64_t c2c2 = ptx::pack2(c2, c2);
        float* mbc_all = reinterpret_cast<float*>(smem + L::kMbcOff);
        float2* part_all = reinterpret_cast<float2*>(smem + L::kPartOff);
        uint4* my_msg = xchg + (static_cast<size_t>(blockIdx.x) * kXchgDepth) * kTile + row;
        const bool stamp = warp == 0 && lane == 0;
        (void)stamp;
        bool ok = true;
        for (int i = 0; ok && i < n_items; ++i) {
            const int s = i & 1;
            const uint32_t u = static_cast<uint32_t>(i) >> 1;
            float* mbc = mbc_all + s * kChunksPerBlock * kTile;
            float smax = -3.0e38f, mb = -3.0e38f, l = 0.0f;
            if (stamp) ATTNW_STAMP(0, i);
            // This thread's pieces of the row: the 64-column boxes 2k + par, k = 0, 1 (landing slot k).  A whole box is taken
            // at once: 64 scores to registers - the landing slot goes back to the MMA issuer right there -, maximum,
            // offset, exponentials, sum; the exponentials leave as f16 pairs for the stream's packed region, where they
            // wait for the row's statistics without holding up the next row block's scores.
#pragma unroll 1
            for (int k = 0; k < kSubsPerBlock; ++k) {
                const int bx = 2 * k + par;
                const int valid = width - bx * kBoxCols;  // columns of this box that exist
                uint32_t r0[kChunk], r1[kChunk];
                if (k < n_sub) {  // (every warp waits for slot 0, so that a warp without work keeps step)
                    ok = __all_sync(0xffffffffu, fused_wait(&bars->s_full[k], static_cast<uint32_t>(i) & 1u, abort_flag, kSiteGrSFull));
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    if (stamp && k == 0) ATTNW_STAMP(2, i);
                }
                if (stamp) ATTNW_STAMP(17 + 3 * k, i);
                if (valid <= 0) {  // nothing of the box is ever stored (the tensor map clips it); the slot's barrier counts every warp
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(&bars->l_free[k]);
                    continue;
                }
                {
                    const uint32_t taddr = t_lane + static_cast<uint32_t>(bx * kBoxCols);
                    ptx::tmem_ld_32x32b_x32(taddr, r0);
                    ptx::tmem_ld_32x32b_x32(taddr + kChunk, r1);
                    ptx::tmem_wait_ld();
                    ptx::tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(&bars->l_free[k]);
                }
                if (valid < kBoxCols) {
#pragma unroll
                    for (int x = 0; x < kChunk; ++x) {
                        if (x >= valid) r0[x] = 0xff61b1e6u;            // -3.0e38f
                        if (x + kChunk >= valid) r1[x] = 0xff61b1e6u;
                    }
                }
                float m0 = -3.0e38f, m1 = -3.0e38f, m2 = -3.0e38f, m3 = -3.0e38f;
#pragma unroll
                for (int x = 0; x < kChunk; x += 8) {
                    m0 = ptx::max3(m0, __uint_as_float(r0[x + 0]), __uint_as_float(r0[x + 1]));
                    m1 = ptx::max3(m1, __uint_as_float(r0[x + 2]), __uint_as_float(r0[x + 3]));
                    m2 = ptx::max3(m2, __uint_as_float(r0[x + 4]), __uint_as_float(r0[x + 5]));
                    m3 = ptx::max3(m3, __uint_as_float(r0[x + 6]), __uint_as_float(r0[x + 7]));
                    m0 = ptx::max3(m0, __uint_as_float(r1[x + 0]), __uint_as_float(r1[x + 1]));
                    m1 = ptx::max3(m1, __uint_as_float(r1[x + 2]), __uint_as_float(r1[x + 3]));
                    m2 = ptx::max3(m2, __uint_as_float(r1[x + 4]), __uint_as_float(r1[x + 5]));
                    m3 = ptx::max3(m3, __uint_as_float(r1[x + 6]), __uint_as_float(r1[x + 7]));
                }
                const float new_max = fmaxf(smax, ptx::max3(fmaxf(m0, m1), m2, m3));
                const float mb_new = fmaxf(new_max * c2, -3.0e38f);  // finite also while every column so far is masked
                l *= ptx::ex2_approx(mb - mb_new);                   // exactly 1 while the maximum stands
                mb = mb_new;
                smax = new_max;
                if (stamp) ATTNW_STAMP(16 + 3 * k, i);
                uint32_t pk[kChunk];  // the box's 64 exponentials as f16 pairs, in column order
                {
                    const uint64_t off2 = ptx::pack2(-mb, -mb);
                    uint64_t acc[4] = {0ull, 0ull, 0ull, 0ull};
                    // (masked columns hold -3e38 and c2 > 0, so their exponentials are exactly zero)
#pragma unroll
                    for (int x = 0; x < kChunk; x += 2) {
                        float a0, a1, b0, b1;
                        const uint64_t xa = ptx::fma2(ptx::pack2(__uint_as_float(r0[x]), __uint_as_float(r0[x + 1])), c2c2, off2);
                        const uint64_t xb = ptx::fma2(ptx::pack2(__uint_as_float(r1[x]), __uint_as_float(r1[x + 1])), c2c2, off2);
                        ptx::unpack2(xa, a0, a1);
                        ptx::unpack2(xb, b0, b1);
                        a0 = ptx::ex2_approx(a0);
                        a1 = ptx::ex2_approx(a1);
                        b0 = ptx::ex2_approx(b0);
                        b1 = ptx::ex2_approx(b1);
                        pk[x >> 1] = ptx::pack_f16x2(a0, a1);
                        pk[(kChunk >> 1) + (x >> 1)] = ptx::pack_f16x2(b0, b1);
                        acc[(x >> 1) & 1] = ptx::add2(acc[(x >> 1) & 1], ptx::pack2(a0, a1));
                        acc[2 + ((x >> 1) & 1)] = ptx::add2(acc[2 + ((x >> 1) & 1)], ptx::pack2(b0, b1));
                    }
                    float s0, s1, s2, s3;
                    ptx::unpack2(ptx::add2(acc[0], acc[1]), s0, s1);
                    ptx::unpack2(ptx::add2(acc[2], acc[3]), s2, s3);
                    l += (s0 + s1) + (s2 + s3);
                }
                if (stamp) ATTNW_STAMP(18 + 3 * k, i);
                // the packed region still holds this box of row block i - 2 until its normalise warps have read it
                ok = __all_sync(0xffffffffu, fused_wait(&bars->pk_free[s][bx], (u & 1u) ^ 1u, abort_flag, kSiteGrSlotFree));
                if (!ok) break;
                ptx::tc_fence_after_sync();
                ptx::tmem_st_32x32b_x32(t_lane + static_cast<uint32_t>(kPackedCol0 + s * kPackedCols + bx * (kBoxCols / 2)), pk);
                if (stamp) ATTNW_STAMP(24 + 2 * k, i);
                mbc[bx * kTile + row] = mb;  // the offset this box's e are relative to
            }
            if (!ok) break;
            part_all[(s * 2 + par) * kTile + row] = make_float2(mb, l);  // this thread's half of the row
            // The second of the two warps to get here merges the halves and posts the row's pair to every CTA of the
            // group (through L2) at once: the exchange must not wait for a normalise warp to become free.
            __threadfence_block();
            __syncwarp();
            uint32_t before = 0;
            if (lane == 0) before = atomicAdd(&bars->halves_done[s][quarter], 1u);
            before = __shfl_sync(0xffffffffu, before, 0);
            if (before & 1u) {
                __threadfence_block();
                const volatile float* pv = reinterpret_cast<const volatile float*>(part_all);
                const float pax = pv[2 * ((s * 2 + 0) * kTile + row)], pay = pv[2 * ((s * 2 + 0) * kTile + row) + 1];
                const float pbx = pv[2 * ((s * 2 + 1) * kTile + row)], pby = pv[2 * ((s * 2 + 1) * kTile + row) + 1];
                const float mc = fmaxf(pax, pbx);
                const float lc = pay * ptx::ex2_approx(pax - mc) + pby * ptx::ex2_approx(pbx - mc);
                st_message(my_msg + (i & (kXchgDepth - 1)) * kTile, mc, lc, tag_base + static_cast<uint32_t>(i) + 1u);
            }
            ptx::tmem_wait_st();
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&bars->posted[s]);
            if (stamp) ATTNW_STAMP(4, i);
        }
    } else if (run && warp < kNormWarp0 + 4 * kNormGroups) {
        // ================= normalise warps: stream s = (warp - 8) / 4, TMEM lane quarter = warp % 4 =================
        const int first = (kNormGroups == 2) ? ((warp - kNormWarp0) >> 2) : 0;
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        const uint32_t out_base = ptx::smem_u32(smem + L::kOutOff);
        const uint32_t sw = static_cast<uint32_t>(row & 7);
        const uint4* group_msg = xchg + (static_cast<size_t>(group) * group_ctas * kXchgDepth) * kTile + row;
        const float* mbc_all = reinterpret_cast<const float*>(smem + L::kMbcOff);
        const int last_cta = group_ctas - 1;
        const bool stamp = quarter == 0 && lane == 0;
        (void)stamp;
        bool ok = true;
        for (int i = first; ok && i < n_items; i += kNormGroups) {
            const int s = i & 1;
            const uint32_t u = static_cast<uint32_t>(i) >> 1;
            const float* mbc = mbc_all + s * kChunksPerBlock * kTile;
            if (stamp) ATTNW_STAMP(10, i);
            // this CTA's exponentials of the row block are in tensor memory and its chunk offsets in shared memory
            ok = __all_sync(0xffffffffu, fused_wait(&bars->posted[s], u & 1u, abort_flag, kSiteGrPosted));
            if (!ok) break;
            ptx::tc_fence_after_sync();
            if (stamp) ATTNW_STAMP(6, i);
            // ---- global statistics of the row: wait for the C pairs, reduce them (redundantly in every CTA) ----
            // Entry reuse: row blocks i and i + 4 share entries.  A CTA posts block i + 4 after it has read the
            // statistics of block i + 2, i.e. after EVERY CTA has posted block i + 2; a CTA's scores of block i + 2
            // land in the tensor memory its normalise warps have finished reading for block i, which they did after
            // reading these entries.  So nobody overwrites an entry that anyone still has to read.
            float m_row, inv_l;
            {
                const uint32_t tag = tag_base + static_cast<uint32_t>(i) + 1u;
                const uint4* src = group_msg + (i & (kXchgDepth - 1)) * kTile;
                uint4 v[kMaxGroupCtas];
                const long long t0 = clock64();
                for (uint32_t spin = 1;; ++spin) {
                    // all loads first (entries beyond the group repeat its last CTA), then the tags
#pragma unroll
                    for (int c = 0; c < kMaxGroupCtas; ++c)
                        v[c] = ld_message(src + static_cast<size_t>(c < last_cta ? c : last_cta) * kXchgDepth * kTile);
                    bool valid = true;
#pragma unroll
                    for (int c = 0; c < kMaxGroupCtas; ++c) valid = valid && v[c].y == tag && v[c].w == tag;
                    if (__all_sync(0xffffffffu, valid)) break;
                    if ((spin & 15u) == 0) {
                        bool give_up = *abort_flag != 0u;
                        if (!give_up && clock64() - t0 > kWaitLimitCycles) {
                            *abort_flag = 1;
                            atomicCAS(&g_attnw_status, 0u, 0x80000000u | kSiteGrExchange);
                            give_up = true;
                        }
                        if (__any_sync(0xffffffffu, give_up)) {
                            ok = false;
                            break;
                        }
                    }
                }
                if (!ok) break;
                if (stamp) ATTNW_STAMP(11, i);
                m_row = __uint_as_float(v[0].x);
#pragma unroll
                for (int c = 1; c < kMaxGroupCtas; ++c) m_row = fmaxf(m_row, __uint_as_float(v[c].x));
                float l_row = 0.0f;
#pragma unroll
                for (int c = 0; c < kMaxGroupCtas; ++c)
                    l_row += (c < group_ctas) ? __uint_as_float(v[c].z) * ptx::ex2_approx(__uint_as_float(v[c].x) - m_row) : 0.0f;
                inv_l = 1.0f / l_row;
            }
            // factors of the row's boxes, read before any slot is handed back (the exponential warps write the offsets
            // of row block i + 2 as soon as they own its scores)
            float f[kSlabCols / kBoxCols];
#pragma unroll
            for (int b = 0; b < kSlabCols / kBoxCols; ++b)
                f[b] = (b < n_boxes) ? ptx::ex2_approx(mbc[b * kTile + row] - m_row) * inv_l : 0.0f;
#pragma unroll
            for (int b = 0; b < kSlabCols / kBoxCols; ++b) {
                if (b < n_boxes && ok) {
                    uint32_t e[kChunk];  // the box's 64 exponentials as f16 pairs
                    ptx::tmem_ld_32x32b_x32(t_lane + static_cast<uint32_t>(kPackedCol0 + s * kPackedCols + b * (kBoxCols / 2)), e);
                    ptx::tmem_wait_ld();
                    // the box has been read: the exponentials of row block i + 2 may take its place
                    ptx::tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(&bars->pk_free[s][b]);
                    if (stamp && b == 0) ATTNW_STAMP(12, i);
                    // staging box of this (row block, 64 columns): the stream's ring entry m % ring; the store that last
                    // used the entry must have read it before anyone overwrites it
                    const uint32_t m = u * static_cast<uint32_t>(n_boxes) + static_cast<uint32_t>(b);
                    const uint32_t ring = s ? L::kRing1 : L::kRing0;
                    const uint32_t box = (s ? L::kRing0 : 0) + m % ring, use = m / ring;
                    const uint32_t my_row = out_base + box * kBoxBytes + static_cast<uint32_t>(row * 128);
                    if (stamp && b == 2) ATTNW_STAMP(14, i);
                    ok = __all_sync(0xffffffffu, fused_wait(&bars->out_free[box], (use & 1u) ^ 1u, abort_flag, kSiteGrStageFree));
                    if (stamp && b == 2) ATTNW_STAMP(15, i);
                    if (ok) {
                        // p = e * f in float32 from f16 operands (one mixed-precision FMA per element unpacks and scales);
                        // a factor below f16 range rounds to zero, where p < 6e-8 anyway
                        const uint32_t fh = ptx::pack_f16x2(f[b], f[b]);
#pragma unroll
                        for (int gg = 0; gg < 8; ++gg) {  // 8 bf16 = one 16-byte piece of the row's 128 bytes
                            uint32_t w[4];
#pragma unroll
                            for (int x = 0; x < 4; ++x) {
                                float lo, hi;
                                ptx::scale_f16x2(e[gg * 4 + x], fh, lo, hi);
                                w[x] = ptx::pack_bf16x2(lo, hi);
                            }
                            ptx::st_shared_v4(my_row + ((static_cast<uint32_t>(gg) ^ sw) << 4), w[0], w[1], w[2], w[3]);
                        }
                        if (stamp && b == 2) ATTNW_STAMP(8, i);
                        ptx::fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(&bars->out_filled[box]);
                        if (stamp && b == 2) ATTNW_STAMP(9, i);
                    }
                }
            }
            if (stamp) ATTNW_STAMP(7, i);
        }
    }

    // ---- teardown: every thread of the CTA arrives here, also after a wait gave up ----
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == kMmaWarpG) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace gr
}  // namespace attnw
