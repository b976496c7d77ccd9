// CUDA-core skinny GEMM for small batches (and the fallback when the batch is too small to be a
// real contraction for the tensor cores): y[b][r] = sum_k W[r][k] * X[b][k], bf16 weights and fp16
// activations widened exactly, fp32 accumulation.  Weights are streamed once per 8 batch rows with 16-byte loads.
#pragma once
#include "common.cuh"

namespace spiral {

__device__ __forceinline__ float dot8(const uint4& w, const uint4& x, float acc) {
    float2 a = unpack_f16(x.x), b = unpack_f16(x.y), c = unpack_f16(x.z), d = unpack_f16(x.w);
    acc = fmaf(bf16_lo(w.x), a.x, acc);
    acc = fmaf(bf16_hi(w.x), a.y, acc);
    acc = fmaf(bf16_lo(w.y), b.x, acc);
    acc = fmaf(bf16_hi(w.y), b.y, acc);
    acc = fmaf(bf16_lo(w.z), c.x, acc);
    acc = fmaf(bf16_hi(w.z), c.y, acc);
    acc = fmaf(bf16_lo(w.w), d.x, acc);
    acc = fmaf(bf16_hi(w.w), d.y, acc);
    return acc;
}

constexpr int GEMV_BC = 8;       // batch rows per pass
constexpr int GEMV_WARPS = 8;

// grid.x: groups of 2*GEMV_WARPS weight rows; grid.y: groups of GEMV_BC batch rows.
__global__ void __launch_bounds__(GEMV_WARPS * 32) gemv_kernel(const __nv_bfloat16* __restrict__ W, int rows,
                                                              int K, const __half* __restrict__ X, int n,
                                                              float* __restrict__ Y) {
    TRACE_BEGIN(6);
    grid_dependency_sync();
    TRACE_WAITED();
    int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int r0 = (blockIdx.x * GEMV_WARPS + warp) * 2;
    if (r0 >= rows) return;
    bool two = r0 + 1 < rows;
    int b0 = blockIdx.y * GEMV_BC;
    int nb = min(GEMV_BC, n - b0);
    float acc0[GEMV_BC], acc1[GEMV_BC];
#pragma unroll
    for (int b = 0; b < GEMV_BC; ++b) { acc0[b] = 0.f; acc1[b] = 0.f; }
    const __nv_bfloat16* w0 = W + (size_t)r0 * K;
    const __nv_bfloat16* w1 = W + (size_t)(two ? r0 + 1 : r0) * K;
    for (int k = lane * 8; k < K; k += 256) {
        uint4 a = ldg_stream_v4(w0 + k);
        uint4 c = ldg_stream_v4(w1 + k);
#pragma unroll
        for (int b = 0; b < GEMV_BC; ++b) {
            if (b < nb) {
                uint4 xv = ldg_v4(X + (size_t)(b0 + b) * K + k);
                acc0[b] = dot8(a, xv, acc0[b]);
                acc1[b] = dot8(c, xv, acc1[b]);
            }
        }
    }
#pragma unroll
    for (int b = 0; b < GEMV_BC; ++b) {
        float s0 = warp_sum(acc0[b]), s1 = warp_sum(acc1[b]);
        if (lane == 0 && b < nb) {
            Y[(size_t)(b0 + b) * rows + r0] = s0;
            if (two) Y[(size_t)(b0 + b) * rows + r0 + 1] = s1;
        }
    }
}

}  // namespace spiral
