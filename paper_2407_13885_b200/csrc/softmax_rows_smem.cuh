// Row Softmax for rows too long for the register tier (Section VI, Eq. 1; "caching" form of Section VI-A): the row is
// read from HBM once and kept in SHARED memory - of one CTA, or, beyond a CTA's share, of a thread-block cluster whose
// CTAs hold consecutive slices of the row and exchange their local maxima and sums through distributed shared memory,
// as the cores of the paper's Softmax kernel do across the chip (Section VI-B).  One exponential per element.
//
// Per row and CTA: one bulk asynchronous copy brings the slice in (at most 96 KB, so two CTAs share an SM and one
// row's copy and barriers overlap the other's arithmetic and stores; two buffers in one CTA of 1024 threads were
// slower: the per-row barriers, not the copy, are what has to be hidden); pass 1 over shared memory: the slice's
// maximum m_c; pass 2: e = 2^((x - m_c) log2 e) written back to shared memory, the slice's sum l_c; ONE exchange of
// the pairs (m_c, l_c); M = max m_c, L = sum l_c 2^((m_c - M) log2 e); pass 3: e * 2^((m_c - M) log2 e) / L -> P
// (coalesced streaming stores).
#pragma once
#include "attnw_fused.cuh"
#include "softmax_rows.cuh"

namespace attnw {

constexpr long long kSoftmaxRowsSmemTierMinCols = 8192;  // rows longer than this may leave the register tier
constexpr long long kSoftmaxRowsRegClusterMinCols = 45056;  // rows longer than this live in the registers of a cluster

namespace srs {

constexpr int kMaxThreads = 512;  // CTAs of 512 threads (two per SM) or, for slices of up to 64 KB, 256 (three or four per SM)
constexpr int kWarps = kMaxThreads / 32;
constexpr int kSliceMaxCols = 24576;                 // 96 KB of float32 per CTA
constexpr int kMaxCluster = 16;
constexpr long long kMaxCols = static_cast<long long>(kSliceMaxCols) * kMaxCluster;  // 393216
constexpr uint32_t kPieceBytes = 16384;              // one bulk copy instruction
constexpr uint32_t kSiteRowLoad = 120;               // wait site (low byte of the status word)

struct Control {
    uint64_t full;                 // the slice of the current row has landed
    float red[kWarps];             // block reduction
    float xch[2][2][kMaxCluster];  // [row parity][0: local maxima, 1: local sums] of every CTA of the cluster
    uint32_t abort_flag;
    uint32_t prior_failure;
};
constexpr int kControlBytes = 512;
static_assert(sizeof(Control) <= kControlBytes, "control block must fit its slot");

template <bool IS_MAX, int NT>
__device__ __forceinline__ float block_reduce(float v, float* red) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const float o = __shfl_xor_sync(0xffffffffu, v, off);
        v = IS_MAX ? fmaxf(v, o) : v + o;
    }
    __syncthreads();  // red[] of the previous reduction has been read by everyone
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float acc = red[0];
#pragma unroll
    for (int w = 1; w < NT / 32; ++w) acc = IS_MAX ? fmaxf(acc, red[w]) : acc + red[w];
    return acc;
}

// grid: n_clusters * C CTAs in clusters of C; cluster i takes rows i, i + n_clusters, ...; slice_cols columns per CTA
// (a multiple of 4; the last CTA's slice may be shorter or empty).
template <typename OutT, int NT>
__global__ void __launch_bounds__(NT, NT == 256 ? 4 : 2)
softmax_rows_smem_kernel(const float* S, OutT* P, long long rows, long long cols, int slice_cols, int C) {
    extern __shared__ __align__(16) uint8_t srs_smem[];
    Control* ctl = reinterpret_cast<Control*>(srs_smem);
    float* x = reinterpret_cast<float*>(srs_smem + kControlBytes);
    volatile uint32_t* abort_flag = &ctl->abort_flag;

    const uint32_t rank = C > 1 ? ptx::cluster_ctarank() : 0u;
    const long long n_clusters = gridDim.x / C;
    const long long cluster = blockIdx.x / C;
    const long long c0 = static_cast<long long>(rank) * slice_cols;  // first column of this CTA's slice
    const int n = static_cast<int>(c0 >= cols ? 0 : (cols - c0 < slice_cols ? cols - c0 : slice_cols));  // its length
    const int nvec = n >> 2;

    if (threadIdx.x == 0) {
        ctl->prior_failure = *reinterpret_cast<volatile unsigned int*>(&g_attnw_status);
        ptx::mbar_init(&ctl->full, 1);
        ctl->abort_flag = 0;
        ptx::mbar_fence_init();
    }
    __syncthreads();
    // A CTA that sees an earlier failure still takes part in every cluster barrier below, without touching memory.
    bool ok = ctl->prior_failure == 0u;
    if (C > 1) {  // peers' control blocks are initialised before anyone writes into them
        ptx::cluster_arrive_release();
        ptx::cluster_wait_acquire();
    }

    uint32_t it = 0;
    for (long long row = cluster; row < rows; row += n_clusters, ++it) {
        const float* src = S + row * cols + c0;
        if (ok && threadIdx.x == 0 && n > 0) {
            const uint32_t bytes = static_cast<uint32_t>(n) * 4u;
            ptx::mbar_expect_tx(&ctl->full, bytes);
            for (uint32_t off = 0; off < bytes; off += kPieceBytes)
                ptx::bulk_load_1d(ptx::smem_u32(x) + off, reinterpret_cast<const uint8_t*>(src) + off,
                                  bytes - off < kPieceBytes ? bytes - off : kPieceBytes, &ctl->full);
        }
        if (ok && n > 0) ok = fused_wait(&ctl->full, it & 1u, abort_flag, kSiteRowLoad);
        ok = __syncthreads_and(ok);  // all or none of the CTA goes on

        // ---- pass 1: maximum of the slice ----
        float m = -INFINITY;
        if (ok)
            for (int i = threadIdx.x; i < nvec; i += NT) {
                const float4 v = reinterpret_cast<const float4*>(x)[i];
                m = fmaxf(m, fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w)));
            }
        m = block_reduce<true, NT>(m, ctl->red);
        const float mc = (m > -INFINITY) ? m : 0.0f;  // an empty slice (or a failure upstream): keeps inf - inf out

        // ---- pass 2: exponentials relative to the slice's maximum (kept in shared memory), their sum ----
        float l = 0.0f;
        if (ok)
            for (int i = threadIdx.x; i < nvec; i += NT) {
                float4 v = reinterpret_cast<float4*>(x)[i];
                // (x - m) first: the difference is exact near the maximum, so a constant row gives exactly 1
                v.x = sr_ex2((v.x - mc) * kLog2e);
                v.y = sr_ex2((v.y - mc) * kLog2e);
                v.z = sr_ex2((v.z - mc) * kLog2e);
                v.w = sr_ex2((v.w - mc) * kLog2e);
                reinterpret_cast<float4*>(x)[i] = v;
                l += (v.x + v.y) + (v.z + v.w);
            }
        l = block_reduce<false, NT>(l, ctl->red);

        // ---- one exchange of (maximum, sum) across the cluster; the row's maximum and sum; this slice's factor ----
        float factor;
        if (C > 1) {
            const uint32_t par = it & 1u;  // two sets of slots: a fast CTA's next row does not overwrite what a slow one reads
            if (threadIdx.x < static_cast<unsigned>(C)) {
                ptx::st_cluster_f32(ptx::map_to_cta(ptx::smem_u32(&ctl->xch[par][0][rank]), threadIdx.x), m);
                ptx::st_cluster_f32(ptx::map_to_cta(ptx::smem_u32(&ctl->xch[par][1][rank]), threadIdx.x), l);
            }
            ptx::cluster_arrive_release();
            ptx::cluster_wait_acquire();
            float M = ctl->xch[par][0][0];
            for (int c = 1; c < C; ++c) M = fmaxf(M, ctl->xch[par][0][c]);
            if (!(M > -INFINITY)) M = 0.0f;
            float L = 0.0f;
            for (int c = 0; c < C; ++c)  // the same order in every CTA; an empty slice has sum 0 and maximum -inf
                L += ctl->xch[par][1][c] * sr_ex2((ctl->xch[par][0][c] - M) * kLog2e);
            factor = sr_ex2((mc - M) * kLog2e) / L;
        } else {
            factor = 1.0f / l;
        }

        // ---- pass 3: scale and store (each thread re-reads exactly what it wrote in pass 2) ----
        if (ok) {
            OutT* dst = P + row * cols + c0;
            for (int i = threadIdx.x; i < nvec; i += NT) {
                const float4 v = reinterpret_cast<const float4*>(x)[i];
                sr_store4<OutT>(dst + 4ll * i, v.x * factor, v.y * factor, v.z * factor, v.w * factor);
            }
        }
        ptx::fence_proxy_async_smem();  // orders this row's accesses to the slice before the next bulk copy into it
        __syncthreads();                // the slice is free for the next row's copy
    }
    if (C > 1) {  // no CTA leaves while a peer may still write into its control block
        ptx::cluster_arrive_release();
        ptx::cluster_wait_acquire();
    }
}

// Clusters of how many CTAs a row of `cols` columns needs (a power of two), or 0 if it does not fit this tier.
inline int cluster_ctas_for(long long cols) {
    if (cols > kMaxCols) return 0;
    int c = 1;
    while (static_cast<long long>(c) * kSliceMaxCols < cols) c *= 2;
    return c;
}

template <typename OutT, int NT>
inline cudaError_t launch_nt(const float* S, OutT* P, long long rows, long long cols, int sm_count, int C, int slice_cols,
                             cudaStream_t stream) {
    const size_t smem = kControlBytes + static_cast<size_t>(slice_cols) * 4;
    auto kernel = softmax_rows_smem_kernel<OutT, NT>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    if (C > 8) {
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        if (e != cudaSuccess) return e;
    }
    const long long per_sm = NT == 256 ? (smem * 4 <= 224 * 1024 ? 4 : 3) : 2;
    long long n_clusters = (per_sm * sm_count) / C;  // CTAs that fit at once
    if (n_clusters < 1) n_clusters = 1;
    if (n_clusters > rows) n_clusters = rows;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(n_clusters * C));
    cfg.blockDim = dim3(NT);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(C);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, S, P, rows, cols, slice_cols, C);
}

template <typename OutT>
inline cudaError_t launch(const float* S, OutT* P, long long rows, long long cols, int sm_count, cudaStream_t stream) {
    const int C = cluster_ctas_for(cols);
    if (C == 0) return cudaErrorInvalidValue;
    const int slice_cols = static_cast<int>(((cols / 4 + C - 1) / C) * 4);
    if (slice_cols <= 16384) return launch_nt<OutT, 256>(S, P, rows, cols, sm_count, C, slice_cols, stream);
    return launch_nt<OutT, 512>(S, P, rows, cols, sm_count, C, slice_cols, stream);
}


// ---- rows kept in REGISTERS across a cluster, the next row's slice already on its way --------------------------------
// For rows beyond 32768 columns.  A CTA of NT threads holds a slice of up to 32 NT columns in registers (32 per thread,
// as the register tier does for a whole row); its shared memory only receives the NEXT row's slice.  Each WARP owns a
// contiguous piece of the slice (up to 4 KB): it waits for its piece alone, moves it to registers and at once issues
// the bulk copy of the same piece of the next row, so no barrier sits in the load pipeline and the HBM read stream
// does not pause for the reductions, the cluster exchange and the stores.  One read and one write per element, where
// the two-read kernel moves every element through L2 twice.
// CTAs of 512 threads, two per SM, whose phases overlap (CTAs of 1024 threads with slices of 32768 columns were slower
// at every length: fewer clusters of them are resident at once, 15 of 8 CTAs against 14 of 16).
constexpr int kRcThreads = 512;
constexpr int kRcVecPerThread = 8;
constexpr int kRcSliceMaxCols = kRcThreads * kRcVecPerThread * 4;                        // 16384
constexpr long long kRcMaxCols = static_cast<long long>(kRcSliceMaxCols) * kMaxCluster;  // 262144
constexpr uint32_t kSiteRcRowLoad = 121;
constexpr uint32_t kSiteRcExchange = 122;

struct RcControl {
    uint64_t full[kRcThreads / 32];  // one per warp: its piece of the current row has landed
    float red_max[kRcThreads / 32];
    float red_sum[kRcThreads / 32];
    uint64_t pairs_in[2];            // by row parity: the (maximum, sum) pairs of every CTA of the cluster have arrived
    float2 xch[2][kMaxCluster];      // [row parity][CTA]: (local maximum, local sum)
    uint32_t abort_flag;
    uint32_t prior_failure;
};
constexpr int kRcControlBytes = 1024;
static_assert(sizeof(RcControl) <= kRcControlBytes, "control block must fit its slot");

template <typename OutT>
__global__ void __launch_bounds__(kRcThreads, 2)
softmax_rows_regcluster_kernel(const float* S, OutT* P, long long rows, long long cols, int slice_cols, int C) {
    extern __shared__ __align__(16) uint8_t srs_smem[];
    RcControl* ctl = reinterpret_cast<RcControl*>(srs_smem);
    const float4* x = reinterpret_cast<const float4*>(srs_smem + kRcControlBytes);
    volatile uint32_t* abort_flag = &ctl->abort_flag;

    const uint32_t rank = C > 1 ? ptx::cluster_ctarank() : 0u;
    const long long n_clusters = gridDim.x / C;
    const long long cluster = blockIdx.x / C;
    const long long c0 = static_cast<long long>(rank) * slice_cols;
    const int n = static_cast<int>(c0 >= cols ? 0 : (cols - c0 < slice_cols ? cols - c0 : slice_cols));
    const int nvec = n >> 2;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int kWarpsRc = kRcThreads / 32;
    const int piece = (nvec + kWarpsRc - 1) / kWarpsRc;  // vectors per warp, at most 256
    const int v0 = warp * piece < nvec ? warp * piece : nvec;  // this warp's vectors: [v0, v1)
    const int v1 = v0 + piece < nvec ? v0 + piece : nvec;
    const uint32_t bytes = static_cast<uint32_t>(v1 - v0) * 16u;
    const bool full = v1 - v0 == kRcVecPerThread * 32;  // this warp's piece has all its 256 vectors

    if (threadIdx.x == 0) {
        ctl->prior_failure = *reinterpret_cast<volatile unsigned int*>(&g_attnw_status);
        for (int w = 0; w < kWarpsRc; ++w) ptx::mbar_init(&ctl->full[w], 1);
        ptx::mbar_init(&ctl->pairs_in[0], 1);
        ptx::mbar_init(&ctl->pairs_in[1], 1);
        ctl->abort_flag = 0;
        ptx::mbar_fence_init();
    }
    __syncthreads();
    bool ok = ctl->prior_failure == 0u;
    if (C > 1) {  // every CTA of the cluster runs before anyone writes into a peer
        ptx::cluster_arrive_release();
        ptx::cluster_wait_acquire();
    }
    auto issue = [&](long long row) {  // one lane: this warp's piece of `row` -> shared memory
        ptx::mbar_expect_tx(&ctl->full[warp], bytes);
        ptx::bulk_load_1d(ptx::smem_u32(x + v0), reinterpret_cast<const float4*>(S + row * cols + c0) + v0, bytes,
                          &ctl->full[warp]);
    };
    if (ok && lane == 0 && bytes > 0 && cluster < rows) issue(cluster);

    uint32_t it = 0;
    for (long long row = cluster; row < rows; row += n_clusters, ++it) {
        if (ok && bytes > 0) ok = fused_wait(&ctl->full[warp], it & 1u, abort_flag, kSiteRcRowLoad);
        float4 v[kRcVecPerThread];
        float m = -INFINITY;
        if (ok && full) {  // the common case, free of per-vector bounds checks
#pragma unroll
            for (int k = 0; k < kRcVecPerThread; ++k) {
                v[k] = x[v0 + k * 32 + lane];
                m = fmaxf(m, fmaxf(fmaxf(v[k].x, v[k].y), fmaxf(v[k].z, v[k].w)));
            }
        } else {
#pragma unroll
            for (int k = 0; k < kRcVecPerThread; ++k) {
                const int idx = v0 + k * 32 + lane;
                if (ok && idx < v1) {
                    v[k] = x[idx];
                    m = fmaxf(m, fmaxf(fmaxf(v[k].x, v[k].y), fmaxf(v[k].z, v[k].w)));
                } else {
                    v[k] = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
                }
            }
        }
        ptx::fence_proxy_async_smem();  // orders these reads before the next bulk copy into the same bytes
        __syncwarp();
        if (ok && lane == 0 && bytes > 0 && row + n_clusters < rows) issue(row + n_clusters);

        m = sr_row_reduce<kRcThreads, true>(m, ctl->red_max);
        // a warp that gave up has set the flag before the barrier inside the reduction: all or none of the CTA goes on
        ok = *abort_flag == 0u && ctl->prior_failure == 0u;
        const float mc = (m > -INFINITY) ? m : 0.0f;  // an empty slice (or a failure upstream): keeps inf - inf out
        float l = 0.0f;
#pragma unroll
        for (int k = 0; k < kRcVecPerThread; ++k) {
            // (x - m) first: the difference is exact near the maximum, so a constant row gives exactly 1
            v[k].x = sr_ex2((v[k].x - mc) * kLog2e);
            v[k].y = sr_ex2((v[k].y - mc) * kLog2e);
            v[k].z = sr_ex2((v[k].z - mc) * kLog2e);
            v[k].w = sr_ex2((v[k].w - mc) * kLog2e);
            l += (v[k].x + v[k].y) + (v[k].z + v[k].w);
        }
        l = sr_row_reduce<kRcThreads, false>(l, ctl->red_sum);

        float factor;
        if (C > 1) {
            // One exchange of (maximum, sum) across the cluster without a cluster barrier: every CTA sends its pair into
            // every CTA's slots (two sets by row parity) with a store that completes bytes on the receiver's mbarrier,
            // and waits only for its own slots to fill.  A CTA can send the pair of row r + 2 (the same parity) only
            // after receiving every pair of row r + 1, which its peers sent after reading their slots of row r.
            const uint32_t par = it & 1u;
            if (threadIdx.x < static_cast<unsigned>(C))
                ptx::st_async_b64(ptx::map_to_cta(ptx::smem_u32(&ctl->xch[par][rank]), threadIdx.x), ptx::pack2(m, l),
                                  ptx::map_to_cta(ptx::smem_u32(&ctl->pairs_in[par]), threadIdx.x));
            if (threadIdx.x == 0) ptx::mbar_expect_tx(&ctl->pairs_in[par], static_cast<uint32_t>(C) * 8u);
            if (ok) ok = fused_wait(&ctl->pairs_in[par], (it >> 1) & 1u, abort_flag, kSiteRcExchange);
            float M = ctl->xch[par][0].x;
            for (int c = 1; c < C; ++c) M = fmaxf(M, ctl->xch[par][c].x);
            if (!(M > -INFINITY)) M = 0.0f;
            float L = 0.0f;
            for (int c = 0; c < C; ++c)  // the same order in every CTA; an empty slice has sum 0 and maximum -inf
                L += ctl->xch[par][c].y * sr_ex2((ctl->xch[par][c].x - M) * kLog2e);
            factor = sr_ex2((mc - M) * kLog2e) / L;
        } else {
            factor = 1.0f / l;
        }
        if (ok) {
            OutT* dst = P + row * cols + c0 + 4ll * (v0 + lane);
            if (full) {
#pragma unroll
                for (int k = 0; k < kRcVecPerThread; ++k)
                    sr_store4<OutT>(dst + 128 * k, v[k].x * factor, v[k].y * factor, v[k].z * factor, v[k].w * factor);
            } else {
#pragma unroll
                for (int k = 0; k < kRcVecPerThread; ++k)
                    if (v0 + k * 32 + lane < v1)
                        sr_store4<OutT>(dst + 128 * k, v[k].x * factor, v[k].y * factor, v[k].z * factor, v[k].w * factor);
            }
        }
    }
    if (C > 1) {  // no CTA leaves while a peer may still write into its control block
        ptx::cluster_arrive_release();
        ptx::cluster_wait_acquire();
    }
}

inline int rc_cluster_ctas_for(long long cols) {  // any size up to 16, not only powers of two
    if (cols > kRcMaxCols) return 0;
    return static_cast<int>((cols + kRcSliceMaxCols - 1) / kRcSliceMaxCols);
}

// `resident_clusters`: the caller's per-device memo of how many clusters of this size are resident at once (0 = not
// asked yet, -1 = this cluster size cannot be launched here).
template <typename OutT>
inline cudaError_t launch_regcluster(const float* S, OutT* P, long long rows, long long cols, int* resident_clusters,
                                     cudaStream_t stream) {
    const int C = rc_cluster_ctas_for(cols);
    if (C == 0) return cudaErrorInvalidValue;
    constexpr int kSmemMax = kRcControlBytes + kRcSliceMaxCols * 4;
    const int slice_cols = static_cast<int>(((cols / 4 + C - 1) / C) * 4);
    auto kernel = softmax_rows_regcluster_kernel<OutT>;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kRcThreads);
    cfg.dynamicSmemBytes = kRcControlBytes + static_cast<size_t>(slice_cols) * 4;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(C);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (*resident_clusters == 0) {  // once per device, output type and cluster size
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMax);
        if (e == cudaSuccess && C > 8) e = cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        int n = 0;
        if (e == cudaSuccess) {
            cfg.gridDim = dim3(static_cast<unsigned>(C));
            const size_t asked = cfg.dynamicSmemBytes;
            cfg.dynamicSmemBytes = kSmemMax;  // the memo serves every row length of this cluster size
            e = cudaOccupancyMaxActiveClusters(&n, kernel, &cfg);
            cfg.dynamicSmemBytes = asked;
        }
        *resident_clusters = (e == cudaSuccess && n > 0) ? n : -1;
        if (e != cudaSuccess) (void)cudaGetLastError();
    }
    if (*resident_clusters < 0) return cudaErrorInvalidConfiguration;
    long long n_clusters = *resident_clusters;
    if (n_clusters > rows) n_clusters = rows;
    cfg.gridDim = dim3(static_cast<unsigned>(n_clusters * C));
    return cudaLaunchKernelEx(&cfg, kernel, S, P, rows, cols, slice_cols, C);
}

}  // namespace srs
}  // namespace attnw
