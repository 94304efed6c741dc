// SRAM-resident fused attention-weight kernel for sm_100a: the design of Section VII of the paper
// re-expressed with thread-block clusters.
//
// The paper lays the whole score matrix out over a grid of cores, keeps every core's block of scores
// in its SRAM, computes LOCAL row maxima and row sums per core and exchanges them along a grid row
// to obtain the GLOBAL ones before normalising (Section VII; Eq. 1).  Here a cluster of C <= 16 CTAs
// owns a 128-row block of one head; CTA r keeps the 128 x 512 slab of scores for keys
// [512 r, 512 r + 512) in its tensor memory (all 512 TMEM columns), so the tensor cores and the
// exponentials run ONCE per element (the two-pass kernel runs both twice):
//   sweep 1  per 128-column slot, as its MMA completes: running local maximum, e = 2^(c s - mb)
//            relative to the running offset mb, local sum; e is written back over s in TMEM
//   exchange each CTA merges its four column quarters and sends its rows' (mb, l) to every CTA of
//            the cluster through distributed shared memory (st.async + mbarrier complete_tx)
//   sweep 2  global maximum and sum per row; p = e * 2^(mb_slot - M) / L, rounded to bf16, staged,
//            written to HBM exactly once by 128-row TMA stores; the slot is handed back to the MMA
//            issuer, which already computes the next row block's scores into it.
// A cluster walks whole units of work (a head, or a range of its row blocks), so the CTA's key slab is
// loaded into shared memory once per unit and only the 32 KB query tiles stream.
// Valid for N <= 16 * 512 = 8192 keys and bf16 output; anything else takes the two-pass kernel.
#pragma once
#include "attnw_fused.cuh"

namespace attnw {

constexpr int kSlab = 512;                 // key columns per CTA: one full tensor memory
constexpr int kSlots = kSlab / kTile;      // accumulator slots of 128 columns
constexpr int kResidentThreads = 608;      // 16 Softmax warps + TMA producer + MMA issuer + store issuer
constexpr int kStoreWarp = 18;
constexpr int kMaxClusterCtas = 16;        // largest cluster; sizes above 8 are non-portable and the launch opts in
constexpr int kResidentMaxN = kSlab * kMaxClusterCtas;
constexpr int kBoxBytes = kTile * 128;     // one staged store box: 128 rows x 128 bytes

#ifndef ATTNW_POLY_PAIRS_RESIDENT
#define ATTNW_POLY_PAIRS_RESIDENT 0
#endif

enum : uint32_t {  // wait sites of this kernel (low byte of the status word)
    kSiteResKEmpty = 16,
    kSiteResQEmpty = 17,
    kSiteResKFull = 18,
    kSiteResQFull = 19,
    kSiteResSlotFree = 20,
    kSiteResSFull = 21,
    kSiteResPart = 22,
    kSiteResExchange = 23,
    kSiteResStageFree = 24,
    kSiteResStageFilled = 25,
    kSiteResStat = 26,
    kSiteResReduce = 27,
};


constexpr int kKStages = 2;        // key sub-tiles in flight in shared memory
constexpr int kS1Lag = 1;          // sweep 1 of the next row block trails sweep 2 of the current one by this many slots
constexpr int kOwnerRedSlots = 144; // owner-reduce exchange: >= C * ceil(128 / C) for every C <= 16
constexpr int kStoreLag = 3;       // stores allowed to be still reading shared memory when the next one is issued
constexpr int kStageBoxesMax = 6;  // staged store boxes: three per column half, so that about 100 KB of
                                   // stores can be in flight (the write path needs that much to stay busy)

// CMAX = 8 or 16: the largest cluster an instantiation serves.  It sizes the exchange area; with 16 one staging box
// makes room for it.  (The instantiation for CMAX = 8 is the one the headline workload runs.)
template <int D, int CMAX>
struct ResidentSmem {
    static constexpr int kStageBoxes = (CMAX <= 8) ? 6 : 5;
    static constexpr int kAtoms = D / 64;
    static constexpr int kAtomBytes = kTile * 128;
    static constexpr int kTileBytes = kAtoms * kAtomBytes;
    static constexpr int kKOff = 0;                                   // ring of key sub-tiles (128 keys each)
    static constexpr int kQOff = kKOff + kKStages * kTileBytes;       // query tile
    static constexpr int kOutOff = kQOff + kTileBytes;                // staging boxes
    static constexpr int kPartOff = kOutOff + kStageBoxes * kBoxBytes;  // float2 part[4 column quarters][128 rows]
    static constexpr int kXchgOff = kPartOff + 4 * kTile * 8;         // float2 xchg[2 parities][8 CTAs][128 rows]
    static constexpr int kStatOff = kXchgOff + 2 * CMAX * kTile * 8;  // float2 stat[128 rows]: (M, 1/L)
    static constexpr int kBarOff = kStatOff + kTile * 8;
    static constexpr int kBytes = kBarOff + 512;
    static constexpr int kDynamicBytes = kBytes + 1024;
};

static_assert(ResidentSmem<128, 8>::kDynamicBytes <= 227 * 1024 && ResidentSmem<128, 16>::kDynamicBytes <= 227 * 1024,
              "shared memory budget");

struct ResidentBarriers {
    uint64_t k_full[kKStages], k_empty[kKStages], q_full, q_empty;
    uint64_t s_full[kSlots], slot_free[kSlots];
    uint64_t part_full;
    uint64_t x_full[2];
    uint64_t red_full[2];  // owner-reduce exchange: the pairs of the rows this CTA owns have arrived
    uint64_t stat_full[4];
    uint64_t out_free[kStageBoxesMax], out_filled[kStageBoxesMax];
    uint32_t tmem_base;
    uint32_t abort_flag;
    uint32_t prior_failure;
};
static_assert(sizeof(ResidentBarriers) <= 512, "barrier block must fit its slot");

// e_j = 2^(c2 * s_j + neg_offset) for one 32-column chunk, written over s; returns sum_j e_j.
template <int POLY_PAIRS, bool RAGGED>
__device__ __forceinline__ float exp2_chunk_inplace(float (&s)[kChunk], uint64_t c2c2, float neg_offset, int valid) {
    const uint64_t off2 = ptx::pack2(neg_offset, neg_offset);
    uint64_t acc[4] = {0ull, 0ull, 0ull, 0ull};
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
        if (RAGGED) {
            e0 = (j + 0 < valid) ? e0 : 0.f;
            e1 = (j + 1 < valid) ? e1 : 0.f;
        }
        s[j] = e0;
        s[j + 1] = e1;
        acc[(j >> 1) & 3] = ptx::add2(acc[(j >> 1) & 3], ptx::pack2(e0, e1));
    }
    float a0, a1, a2, a3;
    ptx::unpack2(ptx::add2(acc[0], acc[1]), a0, a1);
    ptx::unpack2(ptx::add2(acc[2], acc[3]), a2, a3);
    return (a0 + a1) + (a2 + a3);
}

// Work list: item g = (head g / T, row block g % T); cluster c takes items c, c + G, c + 2G, ...  (neighbouring
// clusters work on neighbouring row blocks of one head, so its keys stay hot in L2).  Every role of every CTA
// of the cluster walks the same list.
// OWNER = false: every CTA receives every CTA's pairs and reduces them itself (redundantly, as the paper's kernel
// does).  OWNER = true: the alternative the paper names as future work (Section VIII): the rows are dealt out to the
// CTAs (row i belongs to CTA i mod C); the owner receives the C pairs of its rows, reduces them once and sends
// (M, 1/L) to every CTA - two hops of latency instead of one, C times fewer messages and reductions.
template <int D, int CMAX, bool OWNER>
__global__ void __launch_bounds__(kResidentThreads, 1)
attnw_resident_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                      const __grid_constant__ CUtensorMap tm_p, int N, int total_items, int cluster_ctas,
                      float scale_log2e) {
    using L = ResidentSmem<D, CMAX>;
    constexpr int kStageBoxes = L::kStageBoxes;
    constexpr int kPoly = ATTNW_POLY_PAIRS_RESIDENT;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    ResidentBarriers* bars = reinterpret_cast<ResidentBarriers*>(smem + L::kBarOff);
    volatile uint32_t* abort_flag = &bars->abort_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();
    const int cluster = static_cast<int>(ptx::cluster_id_x());
    const int n_clusters = static_cast<int>(ptx::cluster_count_x());
    const int T = (N + kTile - 1) / kTile;                    // row blocks per head
    const int col0 = static_cast<int>(rank) * kSlab;          // first key of this CTA's slab
    const int width = (N - col0 < kSlab) ? N - col0 : kSlab;  // keys of the slab that exist (>= 1)
    const int n_sub = (width + kTile - 1) / kTile;            // slots in use, 1..4

    // ---- set-up ------------------------------------------------------------------------------
    if (threadIdx.x == 0) {
        for (int st = 0; st < kKStages; ++st) {
            ptx::mbar_init(&bars->k_full[st], 1);
            ptx::mbar_init(&bars->k_empty[st], 1);
        }
        ptx::mbar_init(&bars->q_full, 1);
        ptx::mbar_init(&bars->q_empty, 1);
        for (int t = 0; t < kSlots; ++t) {
            ptx::mbar_init(&bars->s_full[t], 1);
            ptx::mbar_init(&bars->slot_free[t], kSoftmaxWarps);
        }
        ptx::mbar_init(&bars->part_full, kSoftmaxWarps);
        ptx::mbar_init(&bars->x_full[0], 1);
        ptx::mbar_init(&bars->x_full[1], 1);
        ptx::mbar_init(&bars->red_full[0], 1);
        ptx::mbar_init(&bars->red_full[1], 1);
        for (int q = 0; q < 4; ++q) ptx::mbar_init(&bars->stat_full[q], 1);
        for (int b = 0; b < kStageBoxes; ++b) {
            ptx::mbar_init(&bars->out_free[b], 1);
            ptx::mbar_init(&bars->out_filled[b], 8);  // one arrival per Softmax warp of the column half
        }
        bars->abort_flag = 0;
        bars->prior_failure = *reinterpret_cast<volatile unsigned int*>(&g_attnw_status);
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
    // Peers write into this CTA's shared memory: nobody starts before every CTA has its barriers.
    ptx::cluster_arrive_release();
    ptx::cluster_wait_acquire();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_base;
    const bool run = bars->prior_failure == 0u;  // an earlier launch step gave up: skip the work, keep the barriers

    if (run && warp == kProducerWarp) {
        // ================= TMA producer: per row block one query tile, then its key sub-tiles =================
        if (lane == 0) {
            const uint64_t keep = ptx::policy_evict_last();
            uint32_t item_n = 0, kt_n = 0;
            bool ok = true;
            for (int g = cluster; ok && g < total_items; g += n_clusters) {
                const int bh = g / T, rb = g % T;
                if (!fused_wait(&bars->q_empty, (item_n & 1u) ^ 1u, abort_flag, kSiteResQEmpty)) break;
                ptx::mbar_expect_tx(&bars->q_full, static_cast<uint32_t>(L::kTileBytes));
                for (int a = 0; a < L::kAtoms; ++a)
                    ptx::tma_load_3d(smem + L::kQOff + a * L::kAtomBytes, &tm_q, &bars->q_full, a * 64, rb * kTile, bh, keep);
                ++item_n;
                for (int t = 0; t < n_sub; ++t) {
                    const uint32_t st = kt_n % kKStages, use = kt_n / kKStages;
                    if (!fused_wait(&bars->k_empty[st], (use & 1u) ^ 1u, abort_flag, kSiteResKEmpty)) {
                        ok = false;
                        break;
                    }
                    ptx::mbar_expect_tx(&bars->k_full[st], static_cast<uint32_t>(L::kTileBytes));
                    for (int a = 0; a < L::kAtoms; ++a)
                        ptx::tma_load_3d(smem + L::kKOff + st * L::kTileBytes + a * L::kAtomBytes, &tm_k,
                                         &bars->k_full[st], a * 64, col0 + t * kTile, bh, keep);
                    ++kt_n;
                }
            }
            if (*abort_flag) {
                // Unwinding: let the copies already in flight land before shared memory is released.
                const long long t0 = clock64();
                for (uint32_t back = 1; back <= kKStages && back <= kt_n; ++back) {
                    const uint32_t n = kt_n - back;
                    while (!ptx::mbar_try_wait(&bars->k_full[n % kKStages], (n / kKStages) & 1u) &&
                           clock64() - t0 < kWaitLimitCycles / 8) {
                    }
                }
                if (item_n > 0)
                    while (!ptx::mbar_try_wait(&bars->q_full, (item_n - 1u) & 1u) && clock64() - t0 < kWaitLimitCycles / 4) {
                    }
            }
        }
    } else if (run && warp == kMmaWarp) {
        // ================= MMA issuer (warp-uniform loop, one elected lane issues) =================
        constexpr uint32_t idesc = ptx::umma_idesc_bf16_f32(kTile, kTile);
        const uint32_t q_addr = ptx::smem_u32(smem + L::kQOff);
        const uint32_t k_addr = ptx::smem_u32(smem + L::kKOff);
        uint32_t item_n = 0, kt_n = 0;
        bool ok = true;
        for (int g = cluster; ok && g < total_items; g += n_clusters) {
            ok = __all_sync(0xffffffffu, fused_wait(&bars->q_full, item_n & 1u, abort_flag, kSiteResQFull));
            if (!ok) break;
            for (int t = 0; t < n_sub; ++t) {
                const uint32_t st = kt_n % kKStages, use = kt_n / kKStages;
                ok = __all_sync(0xffffffffu, fused_wait(&bars->k_full[st], use & 1u, abort_flag, kSiteResKFull));
                if (!ok) break;
                // the slot still holds the previous row block's exponentials until its sweep 2 has read them
                ok = __all_sync(0xffffffffu, fused_wait(&bars->slot_free[t], (item_n & 1u) ^ 1u, abort_flag,
                                                        kSiteResSlotFree));
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(t * kTile);
                const uint32_t b_addr = k_addr + st * static_cast<uint32_t>(L::kTileBytes);
                if (ptx::elect_one()) {
#pragma unroll
                    for (int k = 0; k < D / 16; ++k) {
                        const uint32_t off = static_cast<uint32_t>((k >> 2) * L::kAtomBytes + (k & 3) * 32);
                        ptx::umma_f16_ss(d_tmem, ptx::umma_desc_kmajor_sw128(q_addr + off),
                                         ptx::umma_desc_kmajor_sw128(b_addr + off), idesc, k > 0 ? 1u : 0u);
                    }
                    ptx::umma_commit(&bars->s_full[t]);
                    ptx::umma_commit(&bars->k_empty[st]);                         // the key sub-tile may be replaced
                    if (t == n_sub - 1) ptx::umma_commit(&bars->q_empty);         // ... and the query tile
                }
                __syncwarp();
                ++kt_n;
            }
            ++item_n;
        }
    } else if (run && warp == kStoreWarp) {
        // ================= store issuer: one TMA store per filled staging box, in ring order =================
        // Boxes are used in the order (row block, slot, column half); box n lives in ring entry n % kStageBoxes.
        if (lane == 0) {
            const uint64_t stream_out = ptx::policy_evict_first();
            const uint32_t out_base = ptx::smem_u32(smem + L::kOutOff);
            uint32_t n = 0;
            bool ok = true;
            for (int g = cluster; ok && g < total_items; g += n_clusters) {
                const int bh = g / T, rb = g % T;
                for (int t = 0; ok && t < n_sub; ++t)
                    for (int h = 0; h < 2; ++h, ++n) {
                        const uint32_t box = n % kStageBoxes, use = n / kStageBoxes;
                        if (!fused_wait(&bars->out_filled[box], use & 1u, abort_flag, kSiteResStageFilled)) {
                            ok = false;
                            break;
                        }
                        const int out_col = col0 + t * kTile + h * (kTile / 2);
                        // a box wholly beyond the last key is not stored, but its (empty) group is still committed:
                        // the ring bookkeeping counts one bulk group per box
                        if (out_col < N)
                            ptx::tma_store_3d(&tm_p, out_base + box * kBoxBytes, out_col, rb * kTile, bh, stream_out);
                        ptx::bulk_commit_group();
                        // Once at most kStoreLag stores are still reading, store n - kStoreLag has read its ring entry:
                        // that entry is free for its next use, kStageBoxes - kStoreLag boxes ahead of the Softmax
                        // warps.  (An entry's first use needs no arrival: it starts free, and the Softmax warps
                        // wait for phase use - 1 of out_free before use >= 1.)
                        ptx::bulk_wait_group_read<kStoreLag>();
                        if (n >= kStoreLag) ptx::mbar_arrive(&bars->out_free[(n - kStoreLag) % kStageBoxes]);
                    }
            }
            ptx::bulk_wait_group<0>();
        }
    } else if (run && warp < kSoftmaxWarps) {
        // ================= Softmax warps =================
        // warp = 4 * cq + quarter: column quarter (32 of a slot's 128 columns), TMEM lane quarter.
        // Sweep 2 of a row block is interleaved, slot by slot, with sweep 1 of the next one: the stores
        // spread evenly over time (an SM cannot burst them faster than its share of the write path) and
        // the MMA of the next block into a freed slot overlaps the work on the other slots.
        const int quarter = warp & 3;
        const int cq = warp >> 2;
        const int h = cq >> 1;  // column half of a slot = staging buffer / store box
        const int row = quarter * 32 + lane;
        const uint32_t t_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + static_cast<uint32_t>(cq * kChunk);
        const float c2 = scale_log2e;
        const uint64_t c2c2 = ptx::pack2(c2, c2);
        float2* part = reinterpret_cast<float2*>(smem + L::kPartOff);
        const float2* xchg = reinterpret_cast<const float2*>(smem + L::kXchgOff);
        const uint32_t xchg_addr = ptx::smem_u32(smem + L::kXchgOff);
        float2* stat = reinterpret_cast<float2*>(smem + L::kStatOff);
        const uint32_t out_base = ptx::smem_u32(smem + L::kOutOff);
        const uint32_t sw = static_cast<uint32_t>(row & 7);
        bool ok = true;

        // sweep-1 state of the row block being accumulated
        float smax = -3.0e38f, mb = -3.0e38f, l = 0.0f;
        float mb_slot[kSlots];  // the offset each slot's exponentials are relative to

        // Sweep 1 of one slot: local maximum, exponentials written back over the scores, local sum.
        auto sweep1_slot = [&](int t, uint32_t item) {
            ok = __all_sync(0xffffffffu, fused_wait(&bars->s_full[t], item & 1u, abort_flag, kSiteResSFull));
            if (!ok) return;
            ptx::tc_fence_after_sync();
            float s[kChunk];
            load_chunk(t_base + static_cast<uint32_t>(t * kTile), s);
            const int valid = width - t * kTile - cq * kChunk;  // columns of this chunk that exist (may be <= 0)
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
            const float mb_new = fmaxf(new_max * c2, -3.0e38f);  // finite also while every column so far is masked
            l *= ptx::ex2_approx(mb - mb_new);                   // exactly 1 while the maximum stands
            mb = mb_new;
            smax = new_max;
            l += ragged ? exp2_chunk_inplace<kPoly, true>(s, c2c2, -mb, valid)
                        : exp2_chunk_inplace<kPoly, false>(s, c2c2, -mb, valid);
            uint32_t raw[kChunk];
#pragma unroll
            for (int j = 0; j < kChunk; ++j) raw[j] = __float_as_uint(s[j]);
            ptx::tmem_st_32x32b_x32(t_base + static_cast<uint32_t>(t * kTile), raw);
        };

        // End of sweep 1 of a row block: merge the CTA's four column quarters and send the rows' (mb, l)
        // to every CTA of the cluster.
        auto post_partials = [&](uint32_t item) {
            ptx::tmem_wait_st();
            if (!ok) return;
            const uint32_t par = item & 1u;
            part[cq * kTile + row] = make_float2(mb, l);
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&bars->part_full);
            if (cq == 0) {
                ok = __all_sync(0xffffffffu, fused_wait(&bars->part_full, item & 1u, abort_flag, kSiteResPart));
                if (!ok) return;
                float mc = mb, lc = 0.0f;
#pragma unroll
                for (int c = 1; c < 4; ++c) mc = fmaxf(mc, part[c * kTile + row].x);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const float2 pc = part[c * kTile + row];
                    lc += pc.y * ptx::ex2_approx(pc.x - mc);
                }
                if constexpr (!OWNER) {
                    if (warp == 0 && lane == 0)  // arm this CTA's receive barrier for the whole cluster's rows
                        ptx::mbar_expect_tx(&bars->x_full[par], static_cast<uint32_t>(cluster_ctas * kTile * 8));
                    const uint64_t payload = ptx::pack2(mc, lc);
                    const uint32_t slot_addr = xchg_addr + ((par * CMAX + rank) * kTile + row) * 8u;
                    const uint32_t bar_addr = ptx::smem_u32(&bars->x_full[par]);
                    for (int dst = 0; dst < cluster_ctas; ++dst)
                        ptx::st_async_b64(ptx::map_to_cta(slot_addr, dst), payload, ptx::map_to_cta(bar_addr, dst));
                } else {
                    // exchange area, per parity: red[C senders][rows one CTA can own], then res[128 rows]
                    const int own_stride = (kTile + cluster_ctas - 1) / cluster_ctas;
                    const int n_own = (kTile - static_cast<int>(rank) + cluster_ctas - 1) / cluster_ctas;  // rows rank, rank + C, ...
                    const uint32_t red_addr = xchg_addr + par * (kOwnerRedSlots + kTile) * 8u;
                    const uint32_t res_addr = red_addr + kOwnerRedSlots * 8u;
                    if (warp == 0 && lane == 0) {  // arm both receive barriers of this row block
                        ptx::mbar_expect_tx(&bars->red_full[par], static_cast<uint32_t>(n_own * cluster_ctas * 8));
                        ptx::mbar_expect_tx(&bars->x_full[par], static_cast<uint32_t>(kTile * 8));
                    }
                    {   // hop 1: this row's merged pair goes to the CTA that owns the row
                        const uint32_t owner = static_cast<uint32_t>(row % cluster_ctas), j = static_cast<uint32_t>(row / cluster_ctas);
                        ptx::st_async_b64(ptx::map_to_cta(red_addr + (rank * own_stride + j) * 8u, owner), ptx::pack2(mc, lc),
                                          ptx::map_to_cta(ptx::smem_u32(&bars->red_full[par]), owner));
                    }
                    // hop 2: reduce the rows this CTA owns, one thread per (owned row, destination CTA)
                    ok = __all_sync(0xffffffffu, fused_wait(&bars->red_full[par], (item >> 1) & 1u, abort_flag, kSiteResReduce));
                    if (!ok) return;
                    const float2* red = reinterpret_cast<const float2*>(smem + L::kXchgOff) + par * (kOwnerRedSlots + kTile);
                    const uint32_t res_bar = ptx::smem_u32(&bars->x_full[par]);
                    for (int idx = row; idx < n_own * cluster_ctas; idx += kTile) {
                        const int j = idx / cluster_ctas, dst = idx % cluster_ctas;
                        float2 pc[CMAX];  // all loads at once; entries beyond the cluster repeat its last CTA
#pragma unroll
                        for (int c = 0; c < CMAX; ++c) pc[c] = red[((c < cluster_ctas) ? c : cluster_ctas - 1) * own_stride + j];
                        float m_row = pc[0].x;
#pragma unroll
                        for (int c = 1; c < CMAX; ++c) m_row = fmaxf(m_row, pc[c].x);
                        float l_row = 0.0f;
#pragma unroll
                        for (int c = 0; c < CMAX; ++c)
                            l_row += (c < cluster_ctas) ? pc[c].y * ptx::ex2_approx(pc[c].x - m_row) : 0.0f;
                        const uint32_t i = static_cast<uint32_t>(j * cluster_ctas) + rank;
                        ptx::st_async_b64(ptx::map_to_cta(res_addr + i * 8u, dst), ptx::pack2(m_row, 1.0f / l_row),
                                          ptx::map_to_cta(res_bar, dst));
                    }
                }
            }
        };

        // walk the list of row blocks with one block of look-ahead
        int g = cluster;
        bool have = g < total_items;
        uint32_t item_n = 0, box_n = 0;
        if (have) {  // prologue: sweep 1 of the first row block
#pragma unroll
            for (int t = 0; t < kSlots; ++t) {
                mb_slot[t] = mb;
                if (t < n_sub && ok) {
                    sweep1_slot(t, item_n);
                    mb_slot[t] = mb;
                }
            }
            post_partials(item_n);
        }
        while (have && ok) {
            g += n_clusters;
            const bool have_next = g < total_items;
            // ---- global statistics of the current row block ----
            // One thread per row (the warps of column quarter 0) reduces the cluster's pairs; the other three warps
            // of the same TMEM lane quarter read (M, 1/L) from shared memory.  (The next write of stat[] follows
            // this CTA's next post, which needs every warp to have passed this read.)
            const uint32_t par = item_n & 1u;
            float m_row, inv_l;
            if (cq == 0) {
                ok = __all_sync(0xffffffffu, fused_wait(&bars->x_full[par], (item_n >> 1) & 1u, abort_flag, kSiteResExchange));
                if (!ok) break;
                if constexpr (!OWNER) {
                    // all exchange slots are read at once (independent loads); slots beyond the cluster are ignored
                    float2 pc[CMAX];
#pragma unroll
                    for (int c = 0; c < CMAX; ++c) pc[c] = xchg[(par * CMAX + c) * kTile + row];
                    m_row = pc[0].x;
#pragma unroll
                    for (int c = 1; c < CMAX; ++c) m_row = (c < cluster_ctas) ? fmaxf(m_row, pc[c].x) : m_row;
                    float l_row = 0.0f;
#pragma unroll
                    for (int c = 0; c < CMAX; ++c)
                        l_row += (c < cluster_ctas) ? pc[c].y * ptx::ex2_approx(pc[c].x - m_row) : 0.0f;
                    inv_l = 1.0f / l_row;
                } else {
                    const float2 ml = xchg[par * (kOwnerRedSlots + kTile) + kOwnerRedSlots + row];  // the owner's (M, 1/L)
                    m_row = ml.x;
                    inv_l = ml.y;
                }
                stat[row] = make_float2(m_row, inv_l);
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&bars->stat_full[quarter]);
            } else {
                ok = __all_sync(0xffffffffu, fused_wait(&bars->stat_full[quarter], item_n & 1u, abort_flag, kSiteResStat));
                if (!ok) break;
                const float2 ml = stat[row];
                m_row = ml.x;
                inv_l = ml.y;
            }
            float f_slot[kSlots];
#pragma unroll
            for (int t = 0; t < kSlots; ++t) f_slot[t] = ptx::ex2_approx(mb_slot[t] - m_row) * inv_l;
            // reset the sweep-1 state for the next row block
            smax = -3.0e38f;
            mb = -3.0e38f;
            l = 0.0f;

#pragma unroll
            for (int t = 0; t < kSlots; ++t) {
                if (t < n_sub && ok) {
                    // ---- sweep 2 of slot t: normalise, round, stage, store; hand the slot back ----
                    float e[kChunk];
                    load_chunk(t_base + static_cast<uint32_t>(t * kTile), e);
                    ptx::tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(&bars->slot_free[t]);
                    // staging box of this (row block, slot, column half): ring entry box_n % kStageBoxes; the store
                    // that last used the entry must have read it before anyone overwrites it
                    const uint32_t n_box = box_n * 2u + static_cast<uint32_t>(h);  // boxes alternate between the halves
                    const uint32_t box = n_box % kStageBoxes, use = n_box / kStageBoxes;
                    const uint32_t my_row = out_base + box * kBoxBytes + static_cast<uint32_t>(row * 128);
                    ok = __all_sync(0xffffffffu, fused_wait(&bars->out_free[box], (use & 1u) ^ 1u, abort_flag,
                                                            kSiteResStageFree));
                    if (ok) {
                        const uint64_t ff = ptx::pack2(f_slot[t], f_slot[t]);
#pragma unroll
                        for (int gg = 0; gg < 4; ++gg) {  // 8 bf16 = one 16-byte piece; this warp's pieces are 4*(cq&1) .. +3
                            float p[8];
#pragma unroll
                            for (int j = 0; j < 8; j += 2)
                                ptx::unpack2(ptx::mul2(ptx::pack2(e[gg * 8 + j], e[gg * 8 + j + 1]), ff), p[j], p[j + 1]);
                            ptx::st_shared_v4(my_row + ((static_cast<uint32_t>((cq & 1) * 4 + gg) ^ sw) << 4),
                                              ptx::pack_bf16x2(p[0], p[1]), ptx::pack_bf16x2(p[2], p[3]),
                                              ptx::pack_bf16x2(p[4], p[5]), ptx::pack_bf16x2(p[6], p[7]));
                        }
                        ptx::fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(&bars->out_filled[box]);
                        ++box_n;
                    }
                }
                // ---- sweep 1 of slot t - kS1Lag of the next row block: its MMA started when that slot was freed,
                //      kS1Lag slots of sweep 2 ago, and has had time to finish ----
                if (t >= kS1Lag && t - kS1Lag < n_sub && have_next && ok) {
                    sweep1_slot(t - kS1Lag, item_n + 1u);
                    mb_slot[t - kS1Lag] = mb;
                }
            }
            if (have_next && ok) {
#pragma unroll
                for (int t = kSlots - kS1Lag; t < kSlots; ++t) {  // the slots the loop above did not reach
                    if (t >= 0 && t < n_sub && ok) {
                        sweep1_slot(t, item_n + 1u);
                        mb_slot[t] = mb;
                    }
                }
                post_partials(item_n + 1u);
            }
            have = have_next;
            ++item_n;
        }
    }

    // ---- teardown: every thread of every CTA of the cluster arrives here, also after a wait gave up ----
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_arrive_release();  // no peer may still be writing into a CTA that exits
    ptx::cluster_wait_acquire();
    if (warp == kMmaWarp) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace attnw
