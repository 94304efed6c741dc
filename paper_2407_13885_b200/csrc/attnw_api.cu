// C ABI of libattnw.so: argument validation, tensor-map encoding and kernel launches.
// The contract of every entry point is stated in include/attnw.h.
#include <atomic>
#include <climits>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <mutex>

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "../../include/attnw.h"
#include "attnw_fused.cuh"
#include "attn_fused.cuh"
#include "attn_onepass.cuh"
#include "project_qk.cuh"
#include "attnw_resident.cuh"
#include "attnw_gridrow.cuh"
#include "softmax_rows.cuh"
#include "softmax_rows_smem.cuh"

namespace {

using namespace attnw;

constexpr int kMaxDevices = 64;
// Consecutive launches of the grid-row kernel use different exchange areas in turn: the last CTAs of one launch may still
// be reading the pairs of their last row block when the next launch (which starts as soon as its whole grid fits) posts.
constexpr int kGridrowAreas = 4;
constexpr uint32_t kSiteSelfTest = 127;  // wait site of attnw_selftest_wait_timeout (low byte of the status word)

// Not part of any product path: one thread waits, with the caller's limit, on an mbarrier that nobody arrives on,
// gives up, records the site in the per-device status word and returns - the unwinding every kernel's bounded wait
// follows, made reachable for a test without touching the waits of the real kernels.
__global__ void wait_timeout_selftest_kernel(long long limit_cycles) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        ptx::mbar_init(&bar, 1);
        ptx::mbar_fence_init();
        const long long t0 = clock64();
        while (!ptx::mbar_try_wait(&bar, 0u)) {
            if (clock64() - t0 > limit_cycles) {
                atomicCAS(&g_attnw_status, 0u, 0x80000000u | kSiteSelfTest);
                break;
            }
        }
    }
}

// Reads the current device's status word after the caller has synchronised; a recorded failure is cleared and
// reported once.
int read_and_clear_status(unsigned int* word_out) {
    unsigned int word = 0;
    if (cudaMemcpyFromSymbol(&word, attnw::g_attnw_status, sizeof(word)) != cudaSuccess) return ATTNW_ERR_CUDA;
    if (word_out) *word_out = word;
    if (word == 0) return ATTNW_OK;
    const unsigned int zero = 0;
    if (cudaMemcpyToSymbol(attnw::g_attnw_status, &zero, sizeof(zero)) != cudaSuccess) return ATTNW_ERR_CUDA;
    return ATTNW_ERR_TIMEOUT;
}
constexpr int kVersion = 100;  // 0.1.0

std::atomic<long long> g_launches{0};
std::atomic<int> g_rows_variant{0};   // 0 = tier by row length, 1 = caching (register tier only), 2 = recomputing with a second read, 3 = recomputing from registers
std::atomic<int> g_attn_variant{0};   // 0 = default (one pass), 1 = two-pass, 2 = one pass
std::atomic<int> g_fused_variant{0};  // 0 = choose by shape, 1 = two-pass, 2 = SRAM-resident, 3 = SRAM-resident, owner-reduce exchange
constexpr double kTwoPassPerSm = 0.9;  // measured: per-SM throughput of the two-pass kernel relative to the resident one
std::mutex g_mutex;

struct DeviceInfo {
    bool ready = false;
    int cc_major = 0;
    int sm_count = 0;
    int fused_pairs[2][2] = {};  // [d == 128][float32 P]: co-resident two-CTA clusters of the two-pass kernel, 0 = not asked yet
    int resident_clusters[2][kMaxClusterCtas + 1] = {};  // [d == 128][cluster size]: co-resident clusters, 0 = not asked yet
    // fork/join objects for launches that split a call over two kernels (created on first use)
    cudaStream_t side_stream = nullptr;
    cudaEvent_t fork_event = nullptr, join_event = nullptr;
    // grid-row kernel: co-resident CTAs per head dimension (0 = not asked yet), the exchange area in device memory
    // (created on first use, zeroed once) and the next unused message tag
    int gridrow_ctas[2] = {};
    uint4* gridrow_xchg = nullptr;
    int gridrow_xchg_ctas = 0;
    uint32_t gridrow_tag = 0;
    unsigned gridrow_launches = 0;  // selects one of kGridrowAreas exchange areas in turn
    int rc_clusters[2][17] = {};  // resident clusters of 1..16 CTAs of the register-cluster row kernel, [P is float32][CTAs]
};
std::mutex g_split_mutex;
DeviceInfo g_devices[kMaxDevices];

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode_tiled = nullptr;

// Current device's cached properties; returns an attnw_status.
int current_device(DeviceInfo** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();
        return ATTNW_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceInfo& d = g_devices[dev];
    if (!d.ready) {
        if (cudaDeviceGetAttribute(&d.cc_major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            (void)cudaGetLastError();
            return ATTNW_ERR_CUDA;
        }
        d.ready = true;
    }
    *out = &d;
    return d.cc_major == 10 ? ATTNW_OK : ATTNW_ERR_UNSUPPORTED;
}

int load_encoder() {
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_encode_tiled) return ATTNW_OK;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || fn == nullptr) {
        (void)cudaGetLastError();
        return ATTNW_ERR_CUDA;
    }
    g_encode_tiled = reinterpret_cast<EncodeTiledFn>(fn);
    return ATTNW_OK;
}

// Row-major [dim2][dim1][dim0] tensor, box {box0, box1, 1}, 128-byte swizzle (box0 * esize == 128).
int encode_3d(CUtensorMap* map, CUtensorMapDataType dtype, size_t esize, const void* base, uint64_t dim0,
              uint64_t dim1, uint64_t dim2, uint32_t box0, uint32_t box1) {
    const cuuint64_t dims[3] = {dim0, dim1, dim2};
    const cuuint64_t strides[2] = {dim0 * esize, dim0 * dim1 * esize};
    const cuuint32_t box[3] = {box0, box1, 1};
    const cuuint32_t elem_strides[3] = {1, 1, 1};
    CUresult r = g_encode_tiled(map, dtype, 3, const_cast<void*>(base), dims, strides, box, elem_strides,
                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? ATTNW_OK : ATTNW_ERR_CUDA;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool overlaps(const void* a, unsigned long long a_bytes, const void* b, unsigned long long b_bytes) {
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
    return a0 < b0 + b_bytes && b0 < a0 + a_bytes;
}

// Host-only checks of the fused call; no CUDA call is made here.
int validate_fused(const void* Q, const void* K, const void* P, int B, int H, int N, int d, float scale,
                   size_t p_esize) {
    if (!Q || !K || !P) return ATTNW_ERR_NULL_POINTER;
    if (B < 1 || H < 1 || N < 1 || d < 1) return ATTNW_ERR_BAD_SHAPE;
    if (!(scale >= 0.0f) || !std::isfinite(scale)) return ATTNW_ERR_BAD_SHAPE;
    const long long bh = static_cast<long long>(B) * H;
    if (bh > INT_MAX) return ATTNW_ERR_BAD_SHAPE;
    const long long ctas = bh * ((static_cast<long long>(N) + kRowsPerCta - 1) / kRowsPerCta);
    if (ctas > INT_MAX) return ATTNW_ERR_BAD_SHAPE;
    if (N > (1 << 24)) return ATTNW_ERR_BAD_SHAPE;  // keeps every tensor-map stride below 2^40 bytes
    if (d != 64 && d != 128) return ATTNW_ERR_UNSUPPORTED;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(P)) return ATTNW_ERR_MISALIGNED;
    if ((static_cast<unsigned long long>(N) * p_esize) % 16 != 0) return ATTNW_ERR_MISALIGNED;
    if (static_cast<unsigned long long>(N) * N * p_esize >= (1ull << 40)) return ATTNW_ERR_BAD_SHAPE;
    const unsigned long long qk_bytes = static_cast<unsigned long long>(bh) * N * d * 2ull;
    const unsigned long long p_bytes = static_cast<unsigned long long>(bh) * N * N * p_esize;
    if (overlaps(P, p_bytes, Q, qk_bytes) || overlaps(P, p_bytes, K, qk_bytes)) return ATTNW_ERR_ALIASING;
    return ATTNW_OK;
}

template <int D, typename OutT>
int launch_fused(DeviceInfo* dev, const void* Q, const void* K, void* P, int BH, int N, float scale,
                 cudaStream_t stream, bool allow_key_split = true) {
    using L = FusedSmem<D>;
    auto kernel = attnw_fused_kernel<D, OutT>;
    CUtensorMap tm_q, tm_k, tm_p;
    int rc = encode_3d(&tm_q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Q, D, N, BH, 64, kTile);
    if (rc == ATTNW_OK) rc = encode_3d(&tm_k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, K, D, N, BH, 64, kTile);
    if (rc == ATTNW_OK) {
        if (sizeof(OutT) == 2)
            rc = encode_3d(&tm_p, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, P, N, N, BH, 64, kTile);
        else
            rc = encode_3d(&tm_p, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, P, N, N, BH, 32, kTile);
    }
    if (rc != ATTNW_OK) return rc;
    // The attribute is per device and per kernel; set it on every launch path's first use.
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kDynamicBytes) != cudaSuccess) {
        (void)cudaGetLastError();
        return ATTNW_ERR_CUDA;
    }
    const int row_blocks = (N + kRowsPerCta - 1) / kRowsPerCta;
    const float scale_log2e = static_cast<float>(static_cast<double>(scale) * 1.4426950408889634074);
    const long long ctas = static_cast<long long>(BH) * row_blocks;
    // Two CTAs per 256-row block (each walks half of the key tiles; see the kernel) when that fills the device
    // better: CTAs of half the length in waves of `pairs` clusters against whole CTAs in waves of `sm_count`
    // (N = 16384, B*H = 8: 512 CTAs = 4 waves of 148 become 7 half-length waves of 74 pairs; a call with fewer
    // CTAs than SMs simply finishes in half the time).
    int key_split = 1;
    if (allow_key_split && ((N + kTile - 1) / kTile) % 2 == 0 && 2 * ctas <= INT_MAX) {
        int& pairs = dev->fused_pairs[D == 128 ? 1 : 0][sizeof(OutT) == 2 ? 0 : 1];
        if (pairs == 0) {
            cudaLaunchAttribute a[1];
            a[0].id = cudaLaunchAttributeClusterDimension;
            a[0].val.clusterDim.x = 2;
            a[0].val.clusterDim.y = 1;
            a[0].val.clusterDim.z = 1;
            cudaLaunchConfig_t c = {};
            c.blockDim = dim3(kFusedThreads, 1, 1);
            c.gridDim = dim3(static_cast<unsigned>(2 * dev->sm_count), 1, 1);
            c.dynamicSmemBytes = L::kDynamicBytes;
            c.attrs = a;
            c.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, kernel, &c) != cudaSuccess || n < 1) {
                (void)cudaGetLastError();
                n = -1;
            }
            pairs = n;
        }
        if (pairs > 0) {
            const long long whole_waves = (ctas + dev->sm_count - 1) / dev->sm_count;
            const long long half_waves = (ctas + pairs - 1) / pairs;
            if (half_waves * 51 < whole_waves * 100) key_split = 2;  // 2 % for the exchange
        }
    }
    if (key_split == 1) {
        kernel<<<static_cast<unsigned>(ctas), kFusedThreads, L::kDynamicBytes, stream>>>(tm_q, tm_k, tm_p, N, row_blocks,
                                                                                         scale_log2e, 1);
    } else {
        cudaLaunchAttribute a[1];
        a[0].id = cudaLaunchAttributeClusterDimension;
        a[0].val.clusterDim.x = 2;
        a[0].val.clusterDim.y = 1;
        a[0].val.clusterDim.z = 1;
        cudaLaunchConfig_t c = {};
        c.blockDim = dim3(kFusedThreads, 1, 1);
        c.gridDim = dim3(static_cast<unsigned>(2 * ctas), 1, 1);
        c.dynamicSmemBytes = L::kDynamicBytes;
        c.stream = stream;
        c.attrs = a;
        c.numAttrs = 1;
        if (cudaLaunchKernelEx(&c, kernel, tm_q, tm_k, tm_p, N, row_blocks, scale_log2e, 2) != cudaSuccess) {
            (void)cudaGetLastError();
            return ATTNW_ERR_CUDA;
        }
    }
    if (cudaGetLastError() != cudaSuccess) return ATTNW_ERR_CUDA;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return ATTNW_OK;
}

// How many clusters of `cluster_ctas` CTAs of the resident kernel the device can hold at once (cached).
template <int D, int CMAX>
int resident_max_clusters_impl(DeviceInfo* dev, int cluster_ctas) {  // (both exchange forms have the same footprint)
    int& cached = dev->resident_clusters[D == 128 ? 1 : 0][cluster_ctas];
    if (cached != 0) return cached;
    using L = ResidentSmem<D, CMAX>;
    auto kernel = attnw_resident_kernel<D, CMAX, false>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kDynamicBytes) != cudaSuccess ||
        (CMAX > 8 && cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess)) {
        (void)cudaGetLastError();
        return cached = -1;
    }
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(cluster_ctas);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kResidentThreads, 1, 1);
    cfg.dynamicSmemBytes = L::kDynamicBytes;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cfg.gridDim = dim3(static_cast<unsigned>(cluster_ctas * dev->sm_count), 1, 1);
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess || n < 1) {
        (void)cudaGetLastError();
        n = -1;
    }
    return cached = n;
}

template <int D>
int resident_max_clusters(DeviceInfo* dev, int cluster_ctas) {
    return cluster_ctas <= 8 ? resident_max_clusters_impl<D, 8>(dev, cluster_ctas)
                             : resident_max_clusters_impl<D, 16>(dev, cluster_ctas);
}

// SRAM-resident single-pass kernel: one cluster of ceil(N / 512) CTAs per 128-row block, persistent over
// a list of row blocks.  Returns ATTNW_ERR_UNSUPPORTED when the device cannot co-schedule such a cluster.
template <int D, int CMAX, bool OWNER>
int launch_resident_impl(DeviceInfo* dev, const void* Q, const void* K, void* P, int BH, int N, float scale,
                         cudaStream_t stream) {
    using L = ResidentSmem<D, CMAX>;
    auto kernel = attnw_resident_kernel<D, CMAX, OWNER>;
    CUtensorMap tm_q, tm_k, tm_p;
    int rc = encode_3d(&tm_q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Q, D, N, BH, 64, kTile);
    if (rc == ATTNW_OK) rc = encode_3d(&tm_k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, K, D, N, BH, 64, kTile);
    if (rc == ATTNW_OK) rc = encode_3d(&tm_p, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, P, N, N, BH, 64, kTile);
    if (rc != ATTNW_OK) return rc;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kDynamicBytes) != cudaSuccess ||
        (CMAX > 8 && cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess)) {
        (void)cudaGetLastError();
        return ATTNW_ERR_CUDA;
    }
    const int cluster_ctas = (N + kSlab - 1) / kSlab;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(cluster_ctas);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kResidentThreads, 1, 1);
    cfg.dynamicSmemBytes = L::kDynamicBytes;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const int max_clusters = resident_max_clusters<D>(dev, cluster_ctas);
    if (max_clusters < 1) return ATTNW_ERR_UNSUPPORTED;
    const int row_blocks = (N + kTile - 1) / kTile;
    const long long total_items = static_cast<long long>(BH) * row_blocks;
    if (total_items > INT_MAX) return ATTNW_ERR_BAD_SHAPE;
    const int clusters = total_items < max_clusters ? static_cast<int>(total_items) : max_clusters;
    cfg.gridDim = dim3(static_cast<unsigned>(clusters * cluster_ctas), 1, 1);
    const float scale_log2e = static_cast<float>(static_cast<double>(scale) * 1.4426950408889634074);
    if (cudaLaunchKernelEx(&cfg, kernel, tm_q, tm_k, tm_p, N, static_cast<int>(total_items), cluster_ctas, scale_log2e) !=
        cudaSuccess) {
        (void)cudaGetLastError();
        return ATTNW_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return ATTNW_OK;
}

template <int D>
int launch_resident(DeviceInfo* dev, const void* Q, const void* K, void* P, int BH, int N, float scale,
                    cudaStream_t stream, bool owner_reduce = false) {
    const bool small = (N + kSlab - 1) / kSlab <= 8;
    if (owner_reduce)
        return small ? launch_resident_impl<D, 8, true>(dev, Q, K, P, BH, N, scale, stream)
                     : launch_resident_impl<D, 16, true>(dev, Q, K, P, BH, N, scale, stream);
    return small ? launch_resident_impl<D, 8, false>(dev, Q, K, P, BH, N, scale, stream)
                 : launch_resident_impl<D, 16, false>(dev, Q, K, P, BH, N, scale, stream);
}

// Grid-row kernel: a cooperative grid of one CTA per SM; consecutive ceil(N / 256) CTAs form a group that owns a
// 128-row block and walks a contiguous part of the list of row blocks.  Returns ATTNW_ERR_UNSUPPORTED when the
// device cannot hold a whole group at once.
template <int D>
int launch_gridrow(DeviceInfo* dev, const void* Q, const void* K, void* P, int BH, int N, float scale, cudaStream_t stream) {
    using L = gr::Smem<D>;
    auto kernel = gr::attnw_gridrow_kernel<D>;
    CUtensorMap tm_q, tm_k, tm_p;
    int rc = encode_3d(&tm_q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Q, D, N, BH, 64, kTile);
    if (rc == ATTNW_OK) rc = encode_3d(&tm_k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, K, D, N, BH, 64, kTile);
    if (rc == ATTNW_OK) rc = encode_3d(&tm_p, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, P, N, N, BH, 64, kTile);
    if (rc != ATTNW_OK) return rc;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kDynamicBytes) != cudaSuccess) {
        (void)cudaGetLastError();
        return ATTNW_ERR_CUDA;
    }
    const int group_ctas = (N + gr::kSlabCols - 1) / gr::kSlabCols;
    const int row_blocks = (N + kTile - 1) / kTile;
    const long long total_items = static_cast<long long>(BH) * row_blocks;
    if (total_items > INT_MAX) return ATTNW_ERR_BAD_SHAPE;
    uint4* xchg = nullptr;
    uint32_t tag_base = 0;
    int n_groups = 0;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        int& max_ctas = dev->gridrow_ctas[D == 128 ? 1 : 0];
        if (max_ctas == 0) {
            int per_sm = 0;
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, gr::kThreads, L::kDynamicBytes) != cudaSuccess ||
                per_sm < 1) {
                (void)cudaGetLastError();
                max_ctas = -1;
            } else {
                max_ctas = dev->sm_count;  // one CTA per SM: the kernel takes all of tensor memory
            }
        }
        if (max_ctas < group_ctas) return ATTNW_ERR_UNSUPPORTED;
        n_groups = max_ctas / group_ctas;
        if (n_groups > total_items) n_groups = static_cast<int>(total_items);
        if (dev->gridrow_xchg == nullptr || dev->gridrow_xchg_ctas < max_ctas) {
            // first use on this device: the exchange area, zero so that no entry carries a valid tag
            if (dev->gridrow_xchg) cudaFree(dev->gridrow_xchg);
            dev->gridrow_xchg = nullptr;
            const size_t bytes = static_cast<size_t>(kGridrowAreas) * max_ctas * gr::kXchgDepth * kTile * sizeof(uint4);
            void* p = nullptr;
            if (cudaMalloc(&p, bytes) != cudaSuccess || cudaMemset(p, 0, bytes) != cudaSuccess ||
                cudaDeviceSynchronize() != cudaSuccess) {
                (void)cudaGetLastError();
                if (p) cudaFree(p);
                return ATTNW_ERR_CUDA;
            }
            dev->gridrow_xchg = static_cast<uint4*>(p);
            dev->gridrow_xchg_ctas = max_ctas;
            dev->gridrow_tag = 0;
        }
        xchg = dev->gridrow_xchg + static_cast<size_t>(dev->gridrow_launches++ % kGridrowAreas) * dev->gridrow_xchg_ctas *
                                       gr::kXchgDepth * kTile;
        // tags tag_base + 1 ... tag_base + (longest list) belong to this launch; 0 is never a tag
        const uint32_t longest = static_cast<uint32_t>((total_items + n_groups - 1) / n_groups);
        if (dev->gridrow_tag > 0xffffffffu - longest - 1u) dev->gridrow_tag = 0;
        tag_base = dev->gridrow_tag;
        dev->gridrow_tag += longest;
    }
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;  // every CTA of the grid is resident at once, or the launch fails
    attr[0].val.cooperative = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(gr::kThreads, 1, 1);
    cfg.gridDim = dim3(static_cast<unsigned>(n_groups * group_ctas), 1, 1);
    cfg.dynamicSmemBytes = L::kDynamicBytes;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const float scale_log2e = static_cast<float>(static_cast<double>(scale) * 1.4426950408889634074);
    const cudaError_t launched = cudaLaunchKernelEx(&cfg, kernel, tm_q, tm_k, tm_p, N, static_cast<int>(total_items), group_ctas,
                                                    n_groups, scale_log2e, xchg, tag_base);
    if (launched != cudaSuccess) {
        (void)cudaGetLastError();
        // the grid does not fit at once after all (SMs taken away from this context): let the caller choose another kernel
        return launched == cudaErrorCooperativeLaunchTooLarge ? ATTNW_ERR_UNSUPPORTED : ATTNW_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return ATTNW_OK;
}

template <int D>
int launch_attn(const void* Q, const void* K, const void* V, void* O, int BH, int N, float scale, cudaStream_t stream) {
    using L = FusedSmem<D>;
    auto kernel = av::attn_fused_kernel<D>;
    CUtensorMap tm_q, tm_k, tm_v, tm_o;
    int rc = encode_3d(&tm_q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Q, D, N, BH, 64, kTile);
    if (rc == ATTNW_OK) rc = encode_3d(&tm_k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, K, D, N, BH, 64, kTile);
    if (rc == ATTNW_OK) rc = encode_3d(&tm_v, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, V, D, N, BH, 64, kTile);
    if (rc == ATTNW_OK) rc = encode_3d(&tm_o, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, O, D, N, BH, 64, kTile);
    if (rc != ATTNW_OK) return rc;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kDynamicBytes) != cudaSuccess) {
        (void)cudaGetLastError();
        return ATTNW_ERR_CUDA;
    }
    const int row_blocks = (N + kRowsPerCta - 1) / kRowsPerCta;
    const float scale_log2e = static_cast<float>(static_cast<double>(scale) * 1.4426950408889634074);
    kernel<<<static_cast<unsigned>(BH * row_blocks), kFusedThreads, L::kDynamicBytes, stream>>>(tm_q, tm_k, tm_v, tm_o, N,
                                                                                                 row_blocks, scale_log2e);
    if (cudaGetLastError() != cudaSuccess) return ATTNW_ERR_CUDA;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return ATTNW_OK;
}

template <int D>
int launch_attn_onepass(const void* Q, const void* K, const void* V, void* O, int BH, int N, float scale, cudaStream_t stream) {
    using L = av1::Smem<D>;
    auto kernel = av1::attn_onepass_kernel<D>;
    CUtensorMap tm_q, tm_k, tm_v, tm_o;
    int rc = encode_3d(&tm_q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Q, D, N, BH, 64, kTile);
    if (rc == ATTNW_OK) rc = encode_3d(&tm_k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, K, D, N, BH, 64, kTile);
    if (rc == ATTNW_OK) rc = encode_3d(&tm_v, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, V, D, N, BH, 64, kTile);
    if (rc == ATTNW_OK) rc = encode_3d(&tm_o, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, O, D, N, BH, 64, kTile);
    if (rc != ATTNW_OK) return rc;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kDynamicBytes) != cudaSuccess) {
        (void)cudaGetLastError();
        return ATTNW_ERR_CUDA;
    }
    const int row_blocks = (N + kRowsPerCta - 1) / kRowsPerCta;
    const float scale_log2e = static_cast<float>(static_cast<double>(scale) * 1.4426950408889634074);
    kernel<<<static_cast<unsigned>(BH * row_blocks), av1::kThreads, L::kDynamicBytes, stream>>>(tm_q, tm_k, tm_v, tm_o, N,
                                                                                                 row_blocks, scale_log2e);
    if (cudaGetLastError() != cudaSuccess) return ATTNW_ERR_CUDA;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return ATTNW_OK;
}

// Host-only checks of the attention call; no CUDA call is made here.
int validate_attn(const void* Q, const void* K, const void* V, const void* O, int B, int H, int N, int d, float scale) {
    if (!Q || !K || !V || !O) return ATTNW_ERR_NULL_POINTER;
    if (B < 1 || H < 1 || N < 1 || d < 1) return ATTNW_ERR_BAD_SHAPE;
    if (!(scale >= 0.0f) || !std::isfinite(scale)) return ATTNW_ERR_BAD_SHAPE;
    const long long bh = static_cast<long long>(B) * H;
    if (bh > INT_MAX) return ATTNW_ERR_BAD_SHAPE;
    if (bh * ((static_cast<long long>(N) + kRowsPerCta - 1) / kRowsPerCta) > INT_MAX) return ATTNW_ERR_BAD_SHAPE;
    if (N > (1 << 24)) return ATTNW_ERR_BAD_SHAPE;
    if (d != 64 && d != 128) return ATTNW_ERR_UNSUPPORTED;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O)) return ATTNW_ERR_MISALIGNED;
    const unsigned long long bytes = static_cast<unsigned long long>(bh) * N * d * 2ull;
    if (overlaps(O, bytes, Q, bytes) || overlaps(O, bytes, K, bytes) || overlaps(O, bytes, V, bytes)) return ATTNW_ERR_ALIASING;
    return ATTNW_OK;
}

// Host-only checks of the projection call; no CUDA call is made here.
int validate_project(const void* X, const void* Wq, const void* Wk, const void* Q, const void* K, int B, int N, int d_model,
                     int H, int d) {
    if (!X || !Wq || !Wk || !Q || !K) return ATTNW_ERR_NULL_POINTER;
    if (B < 1 || N < 1 || d_model < 1 || H < 1 || d < 1) return ATTNW_ERR_BAD_SHAPE;
    if (N > (1 << 24) || d_model > (1 << 20)) return ATTNW_ERR_BAD_SHAPE;  // keeps every tensor-map stride below 2^40 bytes
    const long long bh = static_cast<long long>(B) * H;
    if (bh > INT_MAX || static_cast<long long>(H) * d > INT_MAX) return ATTNW_ERR_BAD_SHAPE;
    const long long col_tiles = (static_cast<long long>(H) * d + proj::kCols - 1) / proj::kCols;
    const long long row_tiles = (static_cast<long long>(N) + proj::kRows - 1) / proj::kRows;
    if (2 * col_tiles * row_tiles * B > INT_MAX) return ATTNW_ERR_BAD_SHAPE;
    if (d != 64 && d != 128) return ATTNW_ERR_UNSUPPORTED;
    if (d_model % 8 != 0) return ATTNW_ERR_MISALIGNED;  // rows of X and of the weights must start on 16-byte boundaries
    if (!aligned16(X) || !aligned16(Wq) || !aligned16(Wk) || !aligned16(Q) || !aligned16(K)) return ATTNW_ERR_MISALIGNED;
    const unsigned long long x_bytes = static_cast<unsigned long long>(B) * N * d_model * 2ull;
    const unsigned long long w_bytes = static_cast<unsigned long long>(H) * d * d_model * 2ull;
    const unsigned long long o_bytes = static_cast<unsigned long long>(bh) * N * d * 2ull;
    if (overlaps(Q, o_bytes, K, o_bytes)) return ATTNW_ERR_ALIASING;
    for (const void* out : {Q, K})
        if (overlaps(out, o_bytes, X, x_bytes) || overlaps(out, o_bytes, Wq, w_bytes) || overlaps(out, o_bytes, Wk, w_bytes))
            return ATTNW_ERR_ALIASING;
    return ATTNW_OK;
}

int launch_project(const void* X, const void* Wq, const void* Wk, void* Q, void* K, int B, int N, int d_model, int H, int d,
                   cudaStream_t stream) {
    CUtensorMap tm_x, tm_wq, tm_wk, tm_q, tm_k;
    const uint64_t hd = static_cast<uint64_t>(H) * d;
    int rc = encode_3d(&tm_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, X, d_model, N, B, proj::kKSlice, 128);
    if (rc == ATTNW_OK) rc = encode_3d(&tm_wq, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Wq, d_model, hd, 1, proj::kKSlice, 128);
    if (rc == ATTNW_OK) rc = encode_3d(&tm_wk, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Wk, d_model, hd, 1, proj::kKSlice, 128);
    if (rc == ATTNW_OK) rc = encode_3d(&tm_q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Q, d, N, static_cast<uint64_t>(B) * H, 64, 128);
    if (rc == ATTNW_OK) rc = encode_3d(&tm_k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, K, d, N, static_cast<uint64_t>(B) * H, 64, 128);
    if (rc != ATTNW_OK) return rc;
    if (cudaFuncSetAttribute(proj::project_qk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, proj::kDynamicBytes) !=
        cudaSuccess) {
        (void)cudaGetLastError();
        return ATTNW_ERR_CUDA;
    }
    const int col_tiles = static_cast<int>((hd + proj::kCols - 1) / proj::kCols);
    const int row_tiles = (N + proj::kRows - 1) / proj::kRows;
    const unsigned ctas = static_cast<unsigned>(2 * col_tiles) * static_cast<unsigned>(row_tiles) * static_cast<unsigned>(B);
    proj::project_qk_kernel<<<ctas, proj::kThreads, proj::kDynamicBytes, stream>>>(tm_x, tm_wq, tm_wk, tm_q, tm_k, N, d_model, H,
                                                                                     d, col_tiles, row_tiles);
    if (cudaGetLastError() != cudaSuccess) return ATTNW_ERR_CUDA;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return ATTNW_OK;
}

template <typename OutT>
int fused_entry(const void* Q, const void* K, void* P, int B, int H, int N, int d, float scale, void* stream) {
    int rc = validate_fused(Q, K, P, B, H, N, d, scale, sizeof(OutT));
    if (rc != ATTNW_OK) return rc;
    DeviceInfo* dev = nullptr;
    rc = current_device(&dev);
    if (rc != ATTNW_OK) return rc;
    rc = load_encoder();
    if (rc != ATTNW_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int variant = g_fused_variant.load(std::memory_order_relaxed);
    const bool resident_fits = sizeof(OutT) == 2 && N <= kResidentMaxN;
    if ((variant == 2 || variant == 3) && !resident_fits) return ATTNW_ERR_UNSUPPORTED;
    if (variant == 4) {
        if constexpr (sizeof(OutT) == 2) {
            if (N > gr::kMaxN) return ATTNW_ERR_UNSUPPORTED;
            return (d == 64) ? launch_gridrow<64>(dev, Q, K, P, B * H, N, scale, s)
                             : launch_gridrow<128>(dev, Q, K, P, B * H, N, scale, s);
        }
        return ATTNW_ERR_UNSUPPORTED;
    }
    if (variant == 3) {
        if constexpr (sizeof(OutT) == 2)
            return (d == 64) ? launch_resident<64>(dev, Q, K, P, B * H, N, scale, s, true)
                             : launch_resident<128>(dev, Q, K, P, B * H, N, scale, s, true);
        return ATTNW_ERR_UNSUPPORTED;
    }
    // Choice by shape, first candidate: the grid-row kernel (bfloat16 P, N <= 4096).  Measured against the cluster
    // kernel with its split launch and against the two-pass kernel over 19 shapes (B*H = 1 ... 128, N = 256 ... 4096,
    // d = 64 and 128) it was ahead on every one (3 to 18 %), because it runs on every SM and keeps three row blocks
    // in flight per CTA.  A device that cannot hold a whole group at once falls through to the older choice.
    if (variant == 0) {
        if constexpr (sizeof(OutT) == 2) {
            if (N <= gr::kMaxN) {
                rc = (d == 64) ? launch_gridrow<64>(dev, Q, K, P, B * H, N, scale, s)
                               : launch_gridrow<128>(dev, Q, K, P, B * H, N, scale, s);
                if (rc != ATTNW_ERR_UNSUPPORTED) return rc;
            }
        }
    }
    // Older choice by shape: the resident kernel whenever it can serve the call.  It spreads one 128-row block over the
    // C SMs of a cluster, so it also fills the device when B*H is small (B*H = 1, N = 4096, d = 128: 25 us
    // against 96 us; B*H = 12, N = 2048, d = 64: 37 against 51 us); between B*H = 8 and 16 at N = 4096 the
    // two kernels are within 2 % of each other, above that the resident kernel leads again.
    // Clusters of more than 8 CTAs (N > 4096) fit only 7 times (112 SMs): there the two-pass kernel with two CTAs per
    // row block is ahead except for a single head (B*H = 4, N = 8192: 188 against 221 us), so the choice by shape
    // stops at N = 4096; variant 2 serves N <= 8192 on request.
    const bool resident_pays = N <= 8 * kSlab;
    if (resident_fits && (variant == 2 || (variant == 0 && resident_pays))) {
        if constexpr (sizeof(OutT) == 2) {
            // Clusters of 8 cannot occupy every SM (15 x 8 = 120 of 148 on B200).  When the call is chosen by
            // shape, the heads are split: the resident kernel takes most of them on the caller's stream, and
            // the two-pass kernel, forked onto a side stream, works through the rest on the SMs the clusters
            // leave idle; the caller's stream joins before the call's work counts as done.
            const int cluster_ctas = (N + kSlab - 1) / kSlab;
            const int clusters = (d == 64) ? resident_max_clusters<64>(dev, cluster_ctas)
                                           : resident_max_clusters<128>(dev, cluster_ctas);
            const int bh = B * H;
            const int idle_sms = clusters > 0 ? dev->sm_count - clusters * cluster_ctas : 0;
            int bh_two_pass = 0;
            if (variant == 0 && idle_sms >= 8 && bh >= 8) {
                // Cost model in units of one resident row block: a cluster finishes one row block per unit, a
                // two-pass CTA (256 rows on one SM) takes 2 * C / kTwoPassPerSm units, both in whole waves.
                const long long blocks_per_head = (N + kTile - 1) / kTile;
                const long long ctas_per_head = (N + kRowsPerCta - 1) / kRowsPerCta;
                const double cta_units = 2.0 * cluster_ctas / kTwoPassPerSm;
                double best = static_cast<double>((bh * blocks_per_head + clusters - 1) / clusters);
                for (int cand = 1; cand <= bh / 2; ++cand) {
                    const double t_res = static_cast<double>(((bh - cand) * blocks_per_head + clusters - 1) / clusters);
                    const double t_two = static_cast<double>((cand * ctas_per_head + idle_sms - 1) / idle_sms) * cta_units;
                    const double t = t_res > t_two ? t_res : t_two;
                    if (t < best) {
                        best = t;
                        bh_two_pass = cand;
                    }
                }
            }
            if (bh_two_pass > 0) {
                std::lock_guard<std::mutex> lock(g_split_mutex);
                if (!dev->side_stream) {
                    if (cudaStreamCreateWithFlags(&dev->side_stream, cudaStreamNonBlocking) != cudaSuccess ||
                        cudaEventCreateWithFlags(&dev->fork_event, cudaEventDisableTiming) != cudaSuccess ||
                        cudaEventCreateWithFlags(&dev->join_event, cudaEventDisableTiming) != cudaSuccess) {
                        (void)cudaGetLastError();
                        return ATTNW_ERR_CUDA;
                    }
                }
                const int bh_res = bh - bh_two_pass;
                const size_t qk_off = static_cast<size_t>(bh_res) * N * d * 2;
                const size_t p_off = static_cast<size_t>(bh_res) * N * N * 2;
                const char* q2 = static_cast<const char*>(Q) + qk_off;
                const char* k2 = static_cast<const char*>(K) + qk_off;
                char* p2 = static_cast<char*>(P) + p_off;
                if (cudaEventRecord(dev->fork_event, s) != cudaSuccess) return ATTNW_ERR_CUDA;
                rc = (d == 64) ? launch_resident<64>(dev, Q, K, P, bh_res, N, scale, s)
                               : launch_resident<128>(dev, Q, K, P, bh_res, N, scale, s);
                if (rc != ATTNW_OK) return rc;
                if (cudaStreamWaitEvent(dev->side_stream, dev->fork_event, 0) != cudaSuccess) return ATTNW_ERR_CUDA;
                rc = (d == 64) ? launch_fused<64, OutT>(dev, q2, k2, p2, bh_two_pass, N, scale, dev->side_stream, false)
                               : launch_fused<128, OutT>(dev, q2, k2, p2, bh_two_pass, N, scale, dev->side_stream, false);
                if (cudaEventRecord(dev->join_event, dev->side_stream) != cudaSuccess ||
                    cudaStreamWaitEvent(s, dev->join_event, 0) != cudaSuccess)
                    return ATTNW_ERR_CUDA;
                return rc;
            }
        }
        rc = (d == 64) ? launch_resident<64>(dev, Q, K, P, B * H, N, scale, s)
                       : launch_resident<128>(dev, Q, K, P, B * H, N, scale, s);
        if (rc != ATTNW_ERR_UNSUPPORTED || variant == 2) return rc;  // no cluster of that size here: two-pass
    }
    if (d == 64) return launch_fused<64, OutT>(dev, Q, K, P, B * H, N, scale, s);
    return launch_fused<128, OutT>(dev, Q, K, P, B * H, N, scale, s);
}

int validate_rows(const void* S, const void* P, long long rows, long long cols, size_t p_esize, bool allow_inplace) {
    if (!S || !P) return ATTNW_ERR_NULL_POINTER;
    if (rows < 1 || cols < 1) return ATTNW_ERR_BAD_SHAPE;
    if (cols > (1ll << 40) || rows > (1ll << 40) || rows > (1ll << 62) / cols) return ATTNW_ERR_BAD_SHAPE;
    if (cols % 4 != 0) return ATTNW_ERR_MISALIGNED;
    if (!aligned16(S) || !aligned16(P)) return ATTNW_ERR_MISALIGNED;
    const unsigned long long n = static_cast<unsigned long long>(rows) * static_cast<unsigned long long>(cols);
    if (overlaps(S, n * 4ull, P, n * p_esize) && !(allow_inplace && S == P)) return ATTNW_ERR_ALIASING;
    return ATTNW_OK;
}

template <typename OutT>
int rows_entry(const void* S, void* P, long long rows, long long cols, void* stream) {
    int rc = validate_rows(S, P, rows, cols, sizeof(OutT), sizeof(OutT) == 4);
    if (rc != ATTNW_OK) return rc;
    DeviceInfo* dev = nullptr;
    rc = current_device(&dev);
    if (rc != ATTNW_OK) return rc;
    const int variant = g_rows_variant.load(std::memory_order_relaxed);
    if (variant == 3 && cols > kSoftmaxRowsRegTierMaxCols) return ATTNW_ERR_UNSUPPORTED;
    if (variant == 1 && cols > srs::kMaxCols) return ATTNW_ERR_UNSUPPORTED;
    // Longer rows can be kept in the shared memory of a CTA or of a cluster (caching form).  By default that is done
    // where it is the faster way (measured): from 8192 columns on - there the register tier needs a whole CTA of 1024
    // threads per row and stops overlapping rows - with one CTA, or a cluster of two up to 32768 columns; beyond, the
    // cluster barrier of every row costs more than the second read (from L2) of the two-read kernel.
    const int smem_ctas = cols > kSoftmaxRowsSmemTierMinCols ? srs::cluster_ctas_for(cols) : 0;
    const bool smem_default = smem_ctas == 1 || (smem_ctas == 2 && cols <= kSoftmaxRowsRegTierMaxCols);
    if ((variant == 0 && smem_default) || (variant == 1 && smem_ctas >= 1)) {
        if (srs::launch<OutT>(static_cast<const float*>(S), static_cast<OutT*>(P), rows, cols, dev->sm_count,
                              static_cast<cudaStream_t>(stream)) == cudaSuccess) {
            g_launches.fetch_add(1, std::memory_order_relaxed);
            return ATTNW_OK;
        }
        (void)cudaGetLastError();  // no cluster of that size on this device: fall through to the two-read kernel
        if (variant == 1) return ATTNW_ERR_UNSUPPORTED;
    }
    // Rows of 45057 to 262144 columns: kept in the registers of a cluster, one read and one write per element
    // (between 32769 and 45056 the slices of a cluster of three are short and the two-read kernel is ahead: measured).
    if (variant == 0 && cols > kSoftmaxRowsRegClusterMinCols && cols <= srs::kRcMaxCols) {
        const int C = srs::rc_cluster_ctas_for(cols);
        const cudaError_t ce = srs::launch_regcluster<OutT>(static_cast<const float*>(S), static_cast<OutT*>(P), rows, cols,
                                                            &dev->rc_clusters[sizeof(OutT) == 4][C],
                                                            static_cast<cudaStream_t>(stream));
        if (ce == cudaSuccess) {
            g_launches.fetch_add(1, std::memory_order_relaxed);
            return ATTNW_OK;
        }
        (void)cudaGetLastError();  // no cluster of that size on this device: the two-read kernel
    }
    cudaError_t e = softmax_rows_launch<OutT>(static_cast<const float*>(S), static_cast<OutT*>(P), rows, cols,
                                              dev->sm_count, static_cast<cudaStream_t>(stream), variant == 3 ? 1 : (variant == 2 ? 2 : 0));
    if (e != cudaSuccess) return ATTNW_ERR_CUDA;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return ATTNW_OK;
}

// ---- host-buffer entry points: staging buffers kept per device, two streams ---------------
struct HostStaging {
    void* buf[2][3] = {{nullptr, nullptr, nullptr}, {nullptr, nullptr, nullptr}};
    size_t cap[2][3] = {{0, 0, 0}, {0, 0, 0}};
    cudaStream_t stream[2] = {nullptr, nullptr};
    bool streams_ready = false;
};
HostStaging g_staging[kMaxDevices];

int staging_for_current_device(HostStaging** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ATTNW_ERR_CUDA;
    HostStaging& st = g_staging[dev];
    if (!st.streams_ready) {
        for (int i = 0; i < 2; ++i)
            if (cudaStreamCreateWithFlags(&st.stream[i], cudaStreamNonBlocking) != cudaSuccess) return ATTNW_ERR_CUDA;
        st.streams_ready = true;
    }
    *out = &st;
    return ATTNW_OK;
}

int staging_reserve(HostStaging* st, int slot, int which, size_t bytes) {
    if (st->cap[slot][which] >= bytes) return ATTNW_OK;
    if (st->buf[slot][which]) {
        // The slot's stream may still be using the old buffer.
        if (cudaStreamSynchronize(st->stream[slot]) != cudaSuccess) return ATTNW_ERR_CUDA;
        cudaFree(st->buf[slot][which]);
        st->buf[slot][which] = nullptr;
        st->cap[slot][which] = 0;
    }
    if (cudaMalloc(&st->buf[slot][which], bytes) != cudaSuccess) {
        (void)cudaGetLastError();
        return ATTNW_ERR_CUDA;
    }
    st->cap[slot][which] = bytes;
    return ATTNW_OK;
}

constexpr unsigned long long kHostChunkBytes = 256ull << 20;  // target size of one staged piece of P

// ---- attnw_fused_noalloc: the grid-row kernel with its exchange area in a static device array ----------------
// Scratch of the entry point that allocates nothing: the exchange area of the grid-row kernel for a grid of up to
// kNoAllocMaxCtas CTAs (messages of 16 bytes: [CTA][4 row blocks in flight][128 rows]) = 1.25 MiB, held by every
// GPU that loads the library until the process exits.  In host code this name is only a stand-in for the symbol:
// the device address comes from cudaGetSymbolAddress (noalloc_setup below) and is what the kernel is given.
constexpr int kNoAllocMaxCtas = 160;
static __device__ __align__(256) uint4 g_noalloc_xchg[kNoAllocMaxCtas * gr::kXchgDepth * kTile];

struct NoAllocState {
    bool ready = false;
    uint4* xchg = nullptr;   // device address of g_noalloc_xchg on this device
    int sm_count = 0;
    uint32_t tag = 0;        // next unused message tag of this device's array
};
NoAllocState g_noalloc[kMaxDevices];

// Once per device, with that device current.  Returns an attnw_status.
int noalloc_setup(NoAllocState** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();
        return ATTNW_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(g_mutex);
    NoAllocState& st = g_noalloc[dev];
    if (!st.ready) {
        int major = 0;
        void* ptr = nullptr;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&st.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            (void)cudaGetLastError();
            return ATTNW_ERR_CUDA;
        }
        if (major != 10) return ATTNW_ERR_UNSUPPORTED;
        if (cudaGetSymbolAddress(&ptr, g_noalloc_xchg) != cudaSuccess || ptr == nullptr) {
            (void)cudaGetLastError();
            return ATTNW_ERR_CUDA;
        }
        st.xchg = static_cast<uint4*>(ptr);
        st.tag = 0;  // the array is zero when the module is loaded, and zero is never a tag
        st.ready = true;
    }
    *out = &st;
    return ATTNW_OK;
}

template <int D>
int launch_gridrow_noalloc(NoAllocState* st, const void* Q, const void* K, void* P, int BH, int N, float scale,
                           cudaStream_t stream) {
    using L = gr::Smem<D>;
    auto kernel = gr::attnw_gridrow_kernel<D>;
    CUtensorMap tm_q, tm_k, tm_p;
    int rc = encode_3d(&tm_q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Q, D, N, BH, 64, kTile);
    if (rc == ATTNW_OK) rc = encode_3d(&tm_k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, K, D, N, BH, 64, kTile);
    if (rc == ATTNW_OK) rc = encode_3d(&tm_p, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, P, N, N, BH, 64, kTile);
    if (rc != ATTNW_OK) return rc;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kDynamicBytes) != cudaSuccess) {
        (void)cudaGetLastError();
        return ATTNW_ERR_CUDA;
    }
    const int group_ctas = (N + gr::kSlabCols - 1) / gr::kSlabCols;
    const long long total_items = static_cast<long long>(BH) * ((N + kTile - 1) / kTile);
    if (total_items > INT_MAX) return ATTNW_ERR_BAD_SHAPE;
    // one CTA per SM, whole groups only, and never more CTAs than the static array has entries for
    const int max_ctas = st->sm_count < kNoAllocMaxCtas ? st->sm_count : kNoAllocMaxCtas;
    if (max_ctas < group_ctas) return ATTNW_ERR_UNSUPPORTED;
    int n_groups = max_ctas / group_ctas;
    if (n_groups > total_items) n_groups = static_cast<int>(total_items);
    uint32_t tag_base = 0;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        const uint32_t longest = static_cast<uint32_t>((total_items + n_groups - 1) / n_groups);
        if (st->tag > 0xffffffffu - longest - 1u) {
            // the tags are used up (after about 4e9 row blocks): start again from a cleared array, in stream order
            if (cudaMemsetAsync(st->xchg, 0, sizeof(g_noalloc_xchg), stream) != cudaSuccess) {
                (void)cudaGetLastError();
                return ATTNW_ERR_CUDA;
            }
            st->tag = 0;
        }
        tag_base = st->tag;
        st->tag += longest;
    }
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(gr::kThreads, 1, 1);
    cfg.gridDim = dim3(static_cast<unsigned>(n_groups * group_ctas), 1, 1);
    cfg.dynamicSmemBytes = L::kDynamicBytes;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const float scale_log2e = static_cast<float>(static_cast<double>(scale) * 1.4426950408889634074);
    if (cudaLaunchKernelEx(&cfg, kernel, tm_q, tm_k, tm_p, N, static_cast<int>(total_items), group_ctas, n_groups, scale_log2e,
                           st->xchg, tag_base) != cudaSuccess) {
        (void)cudaGetLastError();
        return ATTNW_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return ATTNW_OK;
}

}  // namespace

extern "C" {

int attn_fused(const void* Q, const void* K, const void* V, void* O, int B, int H, int N, int d, float scale,
               void* stream) {
    int rc = validate_attn(Q, K, V, O, B, H, N, d, scale);
    if (rc != ATTNW_OK) return rc;
    DeviceInfo* dev = nullptr;
    rc = current_device(&dev);
    if (rc != ATTNW_OK) return rc;
    rc = load_encoder();
    if (rc != ATTNW_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (g_attn_variant.load(std::memory_order_relaxed) == 1)
        return d == 64 ? launch_attn<64>(Q, K, V, O, B * H, N, scale, s) : launch_attn<128>(Q, K, V, O, B * H, N, scale, s);
    return d == 64 ? launch_attn_onepass<64>(Q, K, V, O, B * H, N, scale, s)
                   : launch_attn_onepass<128>(Q, K, V, O, B * H, N, scale, s);
}

int attnw_project_qk(const void* X, const void* Wq, const void* Wk, void* Q, void* K, int B, int N, int d_model, int H, int d,
                     void* stream) {
    int rc = validate_project(X, Wq, Wk, Q, K, B, N, d_model, H, d);
    if (rc != ATTNW_OK) return rc;
    DeviceInfo* dev = nullptr;
    rc = current_device(&dev);
    if (rc != ATTNW_OK) return rc;
    rc = load_encoder();
    if (rc != ATTNW_OK) return rc;
    return launch_project(X, Wq, Wk, Q, K, B, N, d_model, H, d, static_cast<cudaStream_t>(stream));
}

int attnw_set_rows_variant(int variant) {
    if (variant < 0 || variant > 3) return ATTNW_ERR_BAD_SHAPE;
    g_rows_variant.store(variant, std::memory_order_relaxed);
    return ATTNW_OK;
}

int attnw_set_attn_variant(int variant) {
    if (variant < 0 || variant > 2) return ATTNW_ERR_BAD_SHAPE;
    g_attn_variant.store(variant, std::memory_order_relaxed);
    return ATTNW_OK;
}

int attnw_fused(const void* Q, const void* K, void* P, int B, int H, int N, int d, float scale, void* stream) {
    return fused_entry<__nv_bfloat16>(Q, K, P, B, H, N, d, scale, stream);
}

int attnw_fused_noalloc(const void* Q, const void* K, void* P, int B, int H, int N, int d, float scale, void* stream) {
    int rc = validate_fused(Q, K, P, B, H, N, d, scale, 2);
    if (rc != ATTNW_OK) return rc;
    if (N > gr::kMaxN) return ATTNW_ERR_UNSUPPORTED;  // beyond what the static exchange area and one group can serve
    NoAllocState* st = nullptr;
    rc = noalloc_setup(&st);
    if (rc != ATTNW_OK) return rc;
    rc = load_encoder();
    if (rc != ATTNW_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    return d == 64 ? launch_gridrow_noalloc<64>(st, Q, K, P, B * H, N, scale, s)
                   : launch_gridrow_noalloc<128>(st, Q, K, P, B * H, N, scale, s);
}

int attnw_fused_f32(const void* Q, const void* K, void* P, int B, int H, int N, int d, float scale, void* stream) {
    return fused_entry<float>(Q, K, P, B, H, N, d, scale, stream);
}

int softmax_rows(const void* S, void* P, long long rows, long long cols, void* stream) {
    return rows_entry<__nv_bfloat16>(S, P, rows, cols, stream);
}

int softmax_rows_f32(const void* S, void* P, long long rows, long long cols, void* stream) {
    return rows_entry<float>(S, P, rows, cols, stream);
}

int attnw_fused_host(const void* Q, const void* K, void* P, int B, int H, int N, int d, float scale, int p_is_f32) {
    const size_t esize = p_is_f32 ? 4 : 2;
    if (!Q || !K || !P) return ATTNW_ERR_NULL_POINTER;
    if (B < 1 || H < 1 || N < 1 || d < 1) return ATTNW_ERR_BAD_SHAPE;
    if (d != 64 && d != 128) return ATTNW_ERR_UNSUPPORTED;
    const long long bh = static_cast<long long>(B) * H;
    if (bh > INT_MAX || N > (1 << 24)) return ATTNW_ERR_BAD_SHAPE;
    if (!(scale >= 0.0f) || !std::isfinite(scale)) return ATTNW_ERR_BAD_SHAPE;
    if ((static_cast<unsigned long long>(N) * esize) % 16 != 0) return ATTNW_ERR_MISALIGNED;  // before anything is queued
    HostStaging* st = nullptr;
    int rc = staging_for_current_device(&st);
    if (rc != ATTNW_OK) return rc;
    const unsigned long long p_head = static_cast<unsigned long long>(N) * N * esize;
    const unsigned long long qk_head = static_cast<unsigned long long>(N) * d * 2ull;
    long long group = static_cast<long long>(kHostChunkBytes / p_head);
    if (group < 1) group = 1;
    if (group > bh) group = bh;
    for (int slot = 0; slot < 2; ++slot) {
        rc = staging_reserve(st, slot, 0, qk_head * group);
        if (rc == ATTNW_OK) rc = staging_reserve(st, slot, 1, qk_head * group);
        if (rc == ATTNW_OK) rc = staging_reserve(st, slot, 2, p_head * group);
        if (rc != ATTNW_OK) return rc;
    }
    const char* q = static_cast<const char*>(Q);
    const char* k = static_cast<const char*>(K);
    char* p = static_cast<char*>(P);
    int piece = 0;
    for (long long h0 = 0; h0 < bh; h0 += group, ++piece) {
        const long long g = (bh - h0 < group) ? bh - h0 : group;
        const int slot = piece & 1;
        cudaStream_t s = st->stream[slot];
        if (cudaMemcpyAsync(st->buf[slot][0], q + h0 * qk_head, g * qk_head, cudaMemcpyHostToDevice, s) != cudaSuccess ||
            cudaMemcpyAsync(st->buf[slot][1], k + h0 * qk_head, g * qk_head, cudaMemcpyHostToDevice, s) != cudaSuccess) {
            rc = ATTNW_ERR_CUDA;
            break;
        }
        rc = p_is_f32 ? attnw_fused_f32(st->buf[slot][0], st->buf[slot][1], st->buf[slot][2], 1, static_cast<int>(g), N,
                                        d, scale, s)
                      : attnw_fused(st->buf[slot][0], st->buf[slot][1], st->buf[slot][2], 1, static_cast<int>(g), N, d,
                                    scale, s);
        if (rc != ATTNW_OK) break;
        if (cudaMemcpyAsync(p + h0 * p_head, st->buf[slot][2], g * p_head, cudaMemcpyDeviceToHost, s) != cudaSuccess) {
            rc = ATTNW_ERR_CUDA;
            break;
        }
    }
    // On every path, also after an error: no copy may still be reading or writing the caller's buffers on return.
    for (int slot = 0; slot < 2; ++slot)
        if (cudaStreamSynchronize(st->stream[slot]) != cudaSuccess && rc == ATTNW_OK) rc = ATTNW_ERR_CUDA;
    if (rc != ATTNW_OK) return rc;
    return read_and_clear_status(nullptr);  // a wait that gave up inside a kernel: the result is not valid
}

int softmax_rows_host(const void* S, void* P, long long rows, long long cols, int p_is_f32) {
    const size_t esize = p_is_f32 ? 4 : 2;
    if (!S || !P) return ATTNW_ERR_NULL_POINTER;
    if (rows < 1 || cols < 1 || cols > (1ll << 40) || rows > (1ll << 40) || rows > (1ll << 62) / cols)
        return ATTNW_ERR_BAD_SHAPE;
    if (cols % 4 != 0) return ATTNW_ERR_MISALIGNED;
    HostStaging* st = nullptr;
    int rc = staging_for_current_device(&st);
    if (rc != ATTNW_OK) return rc;
    long long group = static_cast<long long>(kHostChunkBytes / (static_cast<unsigned long long>(cols) * 4ull));
    if (group < 1) group = 1;
    if (group > rows) group = rows;
    for (int slot = 0; slot < 2; ++slot) {
        rc = staging_reserve(st, slot, 0, static_cast<size_t>(group) * cols * 4);
        if (rc == ATTNW_OK) rc = staging_reserve(st, slot, 2, static_cast<size_t>(group) * cols * esize);
        if (rc != ATTNW_OK) return rc;
    }
    const char* src = static_cast<const char*>(S);
    char* dst = static_cast<char*>(P);
    int piece = 0;
    for (long long r0 = 0; r0 < rows; r0 += group, ++piece) {
        const long long g = (rows - r0 < group) ? rows - r0 : group;
        const int slot = piece & 1;
        cudaStream_t s = st->stream[slot];
        if (cudaMemcpyAsync(st->buf[slot][0], src + r0 * cols * 4, static_cast<size_t>(g) * cols * 4,
                            cudaMemcpyHostToDevice, s) != cudaSuccess) {
            rc = ATTNW_ERR_CUDA;
            break;
        }
        rc = p_is_f32 ? softmax_rows_f32(st->buf[slot][0], st->buf[slot][2], g, cols, s)
                      : softmax_rows(st->buf[slot][0], st->buf[slot][2], g, cols, s);
        if (rc != ATTNW_OK) break;
        if (cudaMemcpyAsync(dst + r0 * cols * esize, st->buf[slot][2], static_cast<size_t>(g) * cols * esize,
                            cudaMemcpyDeviceToHost, s) != cudaSuccess) {
            rc = ATTNW_ERR_CUDA;
            break;
        }
    }
    // On every path, also after an error: no copy may still be reading or writing the caller's buffers on return.
    for (int slot = 0; slot < 2; ++slot)
        if (cudaStreamSynchronize(st->stream[slot]) != cudaSuccess && rc == ATTNW_OK) rc = ATTNW_ERR_CUDA;
    if (rc != ATTNW_OK) return rc;
    return read_and_clear_status(nullptr);  // a wait that gave up inside a kernel: the result is not valid
}

int attnw_host_release(void) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ATTNW_ERR_CUDA;
    HostStaging& st = g_staging[dev];
    for (int slot = 0; slot < 2; ++slot) {
        if (st.streams_ready) cudaStreamSynchronize(st.stream[slot]);
        for (int w = 0; w < 3; ++w) {
            if (st.buf[slot][w]) cudaFree(st.buf[slot][w]);
            st.buf[slot][w] = nullptr;
            st.cap[slot][w] = 0;
        }
    }
    return ATTNW_OK;
}

int attnw_query_status(void* stream, unsigned int* device_status) {
    if (!device_status) return ATTNW_ERR_NULL_POINTER;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return ATTNW_ERR_CUDA;
    return read_and_clear_status(device_status);
}

int attnw_selftest_wait_timeout(long long limit_cycles, void* stream) {
    if (limit_cycles < 1 || limit_cycles > 2000000000ll) return ATTNW_ERR_BAD_SHAPE;  // at most about one second
    DeviceInfo* dev = nullptr;
    int rc = current_device(&dev);
    if (rc != ATTNW_OK) return rc;
    wait_timeout_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(limit_cycles);
    if (cudaGetLastError() != cudaSuccess) return ATTNW_ERR_CUDA;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return ATTNW_OK;
}

int attnw_set_fused_variant(int variant) {
    if (variant < 0 || variant > 4) return ATTNW_ERR_BAD_SHAPE;
    g_fused_variant.store(variant, std::memory_order_relaxed);
    return ATTNW_OK;
}

long long attnw_launch_count(int reset) {
    return reset ? g_launches.exchange(0, std::memory_order_relaxed) : g_launches.load(std::memory_order_relaxed);
}

const char* attnw_strerror(int code) {
    switch (code) {
        case ATTNW_OK: return "ok";
        case ATTNW_ERR_NULL_POINTER: return "a required pointer is NULL";
        case ATTNW_ERR_BAD_SHAPE: return "a size is out of range, or scale is negative or not finite";
        case ATTNW_ERR_MISALIGNED: return "a pointer or a row pitch is not a multiple of 16 bytes";
        case ATTNW_ERR_UNSUPPORTED: return "unsupported head dimension or device (needs d in {64,128}, sm_100)";
        case ATTNW_ERR_CUDA: return "a CUDA runtime or driver call failed";
        case ATTNW_ERR_TIMEOUT: return "a bounded device-side wait gave up; the output of that launch is undefined";
        case ATTNW_ERR_ALIASING: return "the output overlaps an input";
        default: return "unknown attnw status code";
    }
}

int attnw_version(void) { return kVersion; }
#ifdef ATTNW_TIMELINE
// Debug builds only (-DATTNW_TIMELINE=<cta index>): copies the cycle stamps of that CTA to the host.
int attnw_debug_timeline(long long* out) {
    if (cudaDeviceSynchronize() != cudaSuccess) return ATTNW_ERR_CUDA;
    return cudaMemcpyFromSymbol(out, attnw::g_attnw_timeline, sizeof(long long) * 32 * 160) == cudaSuccess ? ATTNW_OK
                                                                                                          : ATTNW_ERR_CUDA;
}
#endif

}  // extern "C"
