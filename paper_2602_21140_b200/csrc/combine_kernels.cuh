// K_combine: weighted gather-reduce from send-buffer row order back to token
// order (E2A).  y[t,:] = bf16( sum_j coef_j * buf[dst_row[t*k+j], :] ) with
// coef_j = w[t,j] * slot_scale[slot[t,j]] (one fp32 multiply), fp32 fused
// multiply-add accumulation in ascending j, one rounding to bf16.
// Traffic: k rows read + 1 row written per token.
#pragma once

#include <cuda_bf16.h>

#include "device_utils.cuh"

namespace moe {

struct CombineParams {
    const uint4 *buf;            // [T*k, H/8]
    uint4 *y;                    // [T, H/8]
    int T, k, hv;
    const int32_t *dst_row;      // [T*k]
    const float *topk_weights;   // [T,k]
    const int32_t *topk_slot;    // [T,k]
    const float *slot_scale;     // [P]
};

constexpr int kCombineThreads = 256;
constexpr int kCombineUnroll = 2;                      // 16-byte column groups per lane
constexpr int kCombineChunk = 32 * kCombineUnroll;     // uint4 per work item (1 KB of a row)

__device__ __forceinline__ void fma_bf16x8(float (&acc)[8], const uint4 &v, float c)
{
    const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&v);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const float2 f = __bfloat1622float2(h[q]);
        acc[2 * q] = __fmaf_rn(c, f.x, acc[2 * q]);
        acc[2 * q + 1] = __fmaf_rn(c, f.y, acc[2 * q + 1]);
    }
}

__device__ __forceinline__ uint4 pack_bf16x8(const float (&acc)[8])
{
    uint4 o;
    __nv_bfloat162 *h = reinterpret_cast<__nv_bfloat162 *>(&o);
#pragma unroll
    for (int q = 0; q < 4; ++q) h[q] = __floats2bfloat162_rn(acc[2 * q], acc[2 * q + 1]);
    return o;
}

// K > 0: k known at compile time, the k row loads of a column group are all in
// flight together.  K == 0: any k <= 32, rows fetched one after the other.
template <int K>
__global__ void __launch_bounds__(kCombineThreads) k_combine_vec(CombineParams p)
{
    const unsigned full = 0xffffffffu;
    const int lane = lane_id();
    const int k = (K > 0) ? K : p.k;
    const int chunks = (p.hv + kCombineChunk - 1) / kCombineChunk;
    const long long items = (long long)p.T * chunks;
    const long long warp0 = (long long)blockIdx.x * (kCombineThreads / 32) + (threadIdx.x >> 5);
    const long long nwarps = (long long)gridDim.x * (kCombineThreads / 32);

    for (long long it = warp0; it < items; it += nwarps) {
        const int t = (int)(it / chunks);
        const int c0 = (int)(it % chunks) * kCombineChunk + lane;
        int my_row = 0; float my_coef = 0.0f;
        if (lane < k) {
            const size_t i = (size_t)t * k + lane;
            my_row = __ldg(p.dst_row + i);
            my_coef = __fmul_rn(__ldg(p.topk_weights + i), __ldg(p.slot_scale + __ldg(p.topk_slot + i)));
        }
        float acc[kCombineUnroll][8];
#pragma unroll
        for (int u = 0; u < kCombineUnroll; ++u)
#pragma unroll
            for (int q = 0; q < 8; ++q) acc[u][q] = 0.0f;

        if (K > 0) {
            uint4 v[K > 0 ? K : 1][kCombineUnroll];
#pragma unroll
            for (int j = 0; j < K; ++j) {
                const int r = __shfl_sync(full, my_row, j);
                const uint4 *src = p.buf + (size_t)r * p.hv;
#pragma unroll
                for (int u = 0; u < kCombineUnroll; ++u)
                    if (c0 + 32 * u < p.hv) v[j][u] = ld_stream_v4(src + c0 + 32 * u);
            }
#pragma unroll
            for (int j = 0; j < K; ++j) {
                const float c = __shfl_sync(full, my_coef, j);
#pragma unroll
                for (int u = 0; u < kCombineUnroll; ++u)
                    if (c0 + 32 * u < p.hv) fma_bf16x8(acc[u], v[j][u], c);
            }
        } else {
            for (int j = 0; j < k; ++j) {
                const int r = __shfl_sync(full, my_row, j);
                const float c = __shfl_sync(full, my_coef, j);
                const uint4 *src = p.buf + (size_t)r * p.hv;
#pragma unroll
                for (int u = 0; u < kCombineUnroll; ++u)
                    if (c0 + 32 * u < p.hv) fma_bf16x8(acc[u], ld_stream_v4(src + c0 + 32 * u), c);
            }
        }
        uint4 *dst = p.y + (size_t)t * p.hv;
#pragma unroll
        for (int u = 0; u < kCombineUnroll; ++u)
            if (c0 + 32 * u < p.hv) st_stream_v4(dst + c0 + 32 * u, pack_bf16x8(acc[u]));
    }
}

}  // namespace moe
