// Dedicated row-Softmax kernels over precomputed float32 scores (Section VI, Eq. 1; the
// B200 counterpart of the dedicated kernel of Section VI-B).
//
// The operation is bound by HBM traffic (4 bytes read + 2 or 4 written per element, nothing
// to contract), so there are no tensor cores here: each row is streamed in with 128-bit
// loads, kept in registers (the "caching" form of Section VI-A: every exponential is computed
// once), reduced with warp shuffles (plus one shared-memory hop when a row spans several
// warps), and written with coalesced vector stores.  Rows longer than the register tier of this file
// are kept in shared memory or in the registers of a cluster (softmax_rows_smem.cuh); the longest are
// handled by the two-read kernel below, which recomputes the exponentials (the "recomputing" form).
#pragma once
#include <cstdint>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

namespace attnw {

constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float sr_ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// A 16-byte load the compiler must issue each time it is written (the re-reading form reads a row three times).
__device__ __forceinline__ float4 sr_reload4(const float4* p) {
    float4 v;
    asm volatile("ld.global.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p) : "memory");
    return v;
}

template <typename OutT>
__device__ __forceinline__ void sr_store4(OutT* dst, float a, float b, float c, float d);

template <>
__device__ __forceinline__ void sr_store4<float>(float* dst, float a, float b, float c, float d) {
    __stcs(reinterpret_cast<float4*>(dst), make_float4(a, b, c, d));
}
template <>
__device__ __forceinline__ void sr_store4<__nv_bfloat16>(__nv_bfloat16* dst, float a, float b, float c, float d) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(a, b);
    __nv_bfloat162 hi = __floats2bfloat162_rn(c, d);
    uint2 v;
    v.x = *reinterpret_cast<uint32_t*>(&lo);
    v.y = *reinterpret_cast<uint32_t*>(&hi);
    __stcs(reinterpret_cast<uint2*>(dst), v);
}

// Reduce over the TPR threads that share a row.  TPR <= 32: shuffles inside the warp segment.
// TPR > 32: the CTA holds exactly one row; warps exchange partials through `red`.
template <int TPR, bool IS_MAX>
__device__ __forceinline__ float sr_row_reduce(float v, float* red) {
    constexpr int kShuffleSpan = TPR < 32 ? TPR : 32;
#pragma unroll
    for (int off = kShuffleSpan / 2; off > 0; off >>= 1) {
        float o = __shfl_xor_sync(0xffffffffu, v, off);
        v = IS_MAX ? fmaxf(v, o) : v + o;
    }
    if constexpr (TPR > 32) {
        constexpr int kWarps = TPR / 32;
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
        if (lane == 0) red[warp] = v;
        __syncthreads();
        float acc = red[0];
#pragma unroll
        for (int w = 1; w < kWarps; ++w) acc = IS_MAX ? fmaxf(acc, red[w]) : acc + red[w];
        v = acc;
    }
    return v;
}

// S and P carry no __restrict__ and every load is a coherent one: the float32 variant may run
// in place (P == S), where each thread overwrites exactly the elements it has loaded.
//
// Register tier: TPR threads per row, VPT float4 vectors per thread, row kept in registers.
// A CTA has max(TPR, 256) threads and handles CTA_THREADS / TPR rows per sweep.
// MODE 0: the registers keep the exponentials ("caching", Section VI-A).  MODE 1: they keep the scores and every
// exponential is computed twice, once for the sum and once for the output ("recomputing" without its extra reads).
// MODE 2: nothing is kept: the row is read for the maximum, read again for the sum and read a third time for the
// output ("recomputing" as Section VI-A states it; the second and third read come from L1 / L2).
template <int TPR, int VPT, typename OutT, int MODE = 0>
__global__ void __launch_bounds__((TPR > 256 ? TPR : 256))
softmax_rows_reg_kernel(const float* S, OutT* P, long long rows, int cols) {
    constexpr int kThreads = TPR > 256 ? TPR : 256;
    constexpr int kRowsPerCta = kThreads / TPR;
    __shared__ float red_max[TPR > 32 ? TPR / 32 : 1];
    __shared__ float red_sum[TPR > 32 ? TPR / 32 : 1];

    const int nvec = cols >> 2;
    const int sub = threadIdx.x % TPR;          // position inside the row group
    const int row_in_cta = threadIdx.x / TPR;
    const long long sweeps = (rows + kRowsPerCta - 1) / kRowsPerCta;

    for (long long sweep = blockIdx.x; sweep < sweeps; sweep += gridDim.x) {
        const long long row = sweep * kRowsPerCta + row_in_cta;
        const bool row_ok = row < rows;  // uniform per row group; whole warps when TPR >= 32
        const float4* src = reinterpret_cast<const float4*>(S + (row_ok ? row : 0) * static_cast<long long>(cols));
        float4 v[VPT];
        float m = -INFINITY;
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            const int idx = sub + k * TPR;
            if (row_ok && idx < nvec) {
                v[k] = MODE == 2 ? sr_reload4(src + idx) : __ldcs(src + idx);
                m = fmaxf(m, fmaxf(fmaxf(v[k].x, v[k].y), fmaxf(v[k].z, v[k].w)));
            } else {
                v[k] = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
            }
        }
        m = sr_row_reduce<TPR, true>(m, red_max);
        if (!row_ok) m = 0.0f;  // keeps the arithmetic below free of inf - inf
        float l = 0.0f;
        // (x - m) first: the difference is exact near the maximum, so a constant row gives exactly 1.
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            if constexpr (MODE == 2) {  // second read
                const int idx = sub + k * TPR;
                if (row_ok && idx < nvec) v[k] = sr_reload4(src + idx);
            }
            const float4 e = make_float4(sr_ex2((v[k].x - m) * kLog2e), sr_ex2((v[k].y - m) * kLog2e),
                                         sr_ex2((v[k].z - m) * kLog2e), sr_ex2((v[k].w - m) * kLog2e));
            l += (e.x + e.y) + (e.z + e.w);
            if constexpr (MODE == 0) v[k] = e;
        }
        l = sr_row_reduce<TPR, false>(l, red_sum);
        const float inv = 1.0f / l;
        OutT* dst = P + (row_ok ? row : 0) * static_cast<long long>(cols);
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            const int idx = sub + k * TPR;
            if constexpr (MODE == 2) {  // third read
                if (row_ok && idx < nvec) v[k] = sr_reload4(src + idx);
            }
            if constexpr (MODE != 0) {
                // asm volatile keeps the compiler from reusing the first pass's exponentials
                float4 e;
                asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(e.x) : "f"((v[k].x - m) * kLog2e));
                asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(e.y) : "f"((v[k].y - m) * kLog2e));
                asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(e.z) : "f"((v[k].z - m) * kLog2e));
                asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(e.w) : "f"((v[k].w - m) * kLog2e));
                v[k] = e;
            }
            if (row_ok && idx < nvec)
                sr_store4<OutT>(dst + 4ll * idx, v[k].x * inv, v[k].y * inv, v[k].z * inv, v[k].w * inv);
        }
    }
}

// Streaming tier for rows beyond the on-chip tiers: one CTA of THREADS threads per row, two CTAs per SM (two rows in
// different phases: one reads while the other reduces or writes).  First
// read: per-thread running maximum and sum (rescaled only when the maximum grows), merged
// across the CTA.  Second read (mostly from L2): exponentials recomputed, normalised, stored.
template <typename OutT, int THREADS>
__global__ void __launch_bounds__(THREADS, THREADS >= 1024 ? 1 : 2)
softmax_rows_stream_kernel(const float* S, OutT* P, long long rows, long long cols) {
    constexpr int kWarps = THREADS / 32;
    __shared__ float red_m[kWarps];
    __shared__ float red_l[kWarps];
    const long long nvec = cols >> 2;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    for (long long row = blockIdx.x; row < rows; row += gridDim.x) {
        const float4* src = reinterpret_cast<const float4*>(S + row * cols);
        float m = -INFINITY, l = 0.0f;
        // First read: four independent 16-byte loads per step (the row is meant to stay in L2 for the second read, so
        // no streaming hint here), one offset update per step.
        for (long long base = threadIdx.x; base < nvec; base += 4 * THREADS) {
            float4 x[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const long long idx = base + j * THREADS;
                x[j] = idx < nvec ? __ldg(src + idx) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
            }
            float vm = m;
#pragma unroll
            for (int j = 0; j < 4; ++j) vm = fmaxf(vm, fmaxf(fmaxf(x[j].x, x[j].y), fmaxf(x[j].z, x[j].w)));
            if (vm > m) {
                l *= sr_ex2((m - vm) * kLog2e);
                m = vm;
            }
            float acc = 0.0f;
#pragma unroll
            for (int j = 0; j < 4; ++j)  // (x - m) first: a row of equal scores gives exactly 2^0
                acc += (sr_ex2((x[j].x - m) * kLog2e) + sr_ex2((x[j].y - m) * kLog2e)) +
                       (sr_ex2((x[j].z - m) * kLog2e) + sr_ex2((x[j].w - m) * kLog2e));
            l += acc;
        }
        // merge (m, l) pairs: inside the warp, then across warps
        float wm = m;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, off));
        float wl = (m == -INFINITY) ? 0.0f : l * sr_ex2((m - wm) * kLog2e);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) wl += __shfl_xor_sync(0xffffffffu, wl, off);
        if (lane == 0) {
            red_m[warp] = wm;
            red_l[warp] = wl;
        }
        __syncthreads();
        float M = red_m[0];
#pragma unroll
        for (int w = 1; w < kWarps; ++w) M = fmaxf(M, red_m[w]);
        float L = 0.0f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) L += (red_m[w] == -INFINITY) ? 0.0f : red_l[w] * sr_ex2((red_m[w] - M) * kLog2e);
        __syncthreads();  // red_* are rewritten by the next row
        const float inv = 1.0f / L;
        OutT* dst = P + row * cols;
        for (long long base = threadIdx.x; base < nvec; base += 4 * THREADS) {  // second read: from L2, streaming out
            float4 x[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const long long idx = base + j * THREADS;
                x[j] = idx < nvec ? __ldcs(src + idx) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const long long idx = base + j * THREADS;
                if (idx < nvec)
                    sr_store4<OutT>(dst + 4 * idx, sr_ex2((x[j].x - M) * kLog2e) * inv, sr_ex2((x[j].y - M) * kLog2e) * inv,
                                    sr_ex2((x[j].z - M) * kLog2e) * inv, sr_ex2((x[j].w - M) * kLog2e) * inv);
            }
        }
    }
}

// Host-side tier selection; returns the cudaError_t of the launch.
template <int TPR, int VPT, typename OutT>
inline cudaError_t sr_launch_reg(const float* S, OutT* P, long long rows, int cols, int sm_count,
                                 cudaStream_t stream, int mode) {
    constexpr int kThreads = TPR > 256 ? TPR : 256;
    constexpr int kRowsPerCta = kThreads / TPR;
    const long long sweeps = (rows + kRowsPerCta - 1) / kRowsPerCta;
    const long long cap = static_cast<long long>(sm_count) * 64;  // enough CTAs to fill every SM several times
    const unsigned grid = static_cast<unsigned>(sweeps < cap ? sweeps : cap);
    if (mode == 1)
        softmax_rows_reg_kernel<TPR, VPT, OutT, 1><<<grid, kThreads, 0, stream>>>(S, P, rows, cols);
    else if (mode == 2)
        softmax_rows_reg_kernel<TPR, VPT, OutT, 2><<<grid, kThreads, 0, stream>>>(S, P, rows, cols);
    else
        softmax_rows_reg_kernel<TPR, VPT, OutT><<<grid, kThreads, 0, stream>>>(S, P, rows, cols);
    return cudaGetLastError();
}

constexpr long long kSoftmaxRowsRegTierMaxCols = 32768;

// mode: 0 caching, 1 recomputing from registers, 2 recomputing with re-reads (see the register-tier kernel); rows
// beyond the register tier always take the streaming kernel, which is a recomputing form with one extra read
template <typename OutT>
inline cudaError_t softmax_rows_launch(const float* S, OutT* P, long long rows, long long cols, int sm_count,
                                       cudaStream_t stream, int mode = 0) {
    const long long nvec = cols / 4;
    if (cols > kSoftmaxRowsRegTierMaxCols) {
        // Rows in flight must fit in L2 for the second read to be served from there (about 80 MB of the 126 MB are
        // usable for it): two CTAs of 512 threads per SM while they do (measured at 65536 columns: 1.15 against 1.27 ps
        // per element), one CTA of 1024 threads per SM beyond (131072 columns: 1.24 against 1.38).
        const long long row_bytes = cols * 4;
        if (row_bytes * sm_count * 2 <= (80ll << 20)) {
            const long long cap = static_cast<long long>(sm_count) * 2;
            const unsigned grid = static_cast<unsigned>(rows < cap ? rows : cap);
            softmax_rows_stream_kernel<OutT, 512><<<grid, 512, 0, stream>>>(S, P, rows, cols);
        } else {
            const long long cap = static_cast<long long>(sm_count);
            const unsigned grid = static_cast<unsigned>(rows < cap ? rows : cap);
            softmax_rows_stream_kernel<OutT, 1024><<<grid, 1024, 0, stream>>>(S, P, rows, cols);
        }
        return cudaGetLastError();
    }
    const int c = static_cast<int>(cols);
    if (nvec <= 8) return sr_launch_reg<8, 1, OutT>(S, P, rows, c, sm_count, stream, mode);
    if (nvec <= 16) return sr_launch_reg<8, 2, OutT>(S, P, rows, c, sm_count, stream, mode);
    if (nvec <= 32) return sr_launch_reg<8, 4, OutT>(S, P, rows, c, sm_count, stream, mode);
    if (nvec <= 64) return sr_launch_reg<32, 2, OutT>(S, P, rows, c, sm_count, stream, mode);
    if (nvec <= 128) return sr_launch_reg<32, 4, OutT>(S, P, rows, c, sm_count, stream, mode);
    if (nvec <= 256) return sr_launch_reg<32, 8, OutT>(S, P, rows, c, sm_count, stream, mode);
    if (nvec <= 512) return sr_launch_reg<256, 2, OutT>(S, P, rows, c, sm_count, stream, mode);
    if (nvec <= 1024) return sr_launch_reg<256, 4, OutT>(S, P, rows, c, sm_count, stream, mode);
    if (nvec <= 2048) return sr_launch_reg<256, 8, OutT>(S, P, rows, c, sm_count, stream, mode);
    if (nvec <= 4096) return sr_launch_reg<1024, 4, OutT>(S, P, rows, c, sm_count, stream, mode);
    return sr_launch_reg<1024, 8, OutT>(S, P, rows, c, sm_count, stream, mode);
}

}  // namespace attnw
