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
    // Expert parallelism over several GPUs: the rows of slot p live in the receive buffer of
    // GPU p / slots_per_gpu, reached through peer_bufs[that GPU]; dst_row then counts rows of
    // that buffer.  NULL = every row is in `buf`.
    const uint4 *const *peer_bufs;
    int slots_per_gpu;
    int P;                       // physical slots
    long long row_limit;         // rows a source buffer holds: T*k, or the receive-buffer capacity
    const uint4 *zero_row;       // [H/8] zeros: stands in for a row that was not placed
    unsigned spin_limit;         // polls before a bounded wait gives up
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
            const int slot = __ldg(p.topk_slot + i);
            const int r = __ldg(p.dst_row + i);
            if ((unsigned)slot < (unsigned)p.P && r >= 0 && r < p.row_limit) {
                my_row = r;
                my_coef = __fmul_rn(__ldg(p.topk_weights + i), __ldg(p.slot_scale + slot));
            } else {
                my_row = -1;                               // not placed: contributes nothing
            }
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
                const uint4 *src = (r >= 0) ? p.buf + (size_t)r * p.hv : p.zero_row;
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
                const uint4 *src = (r >= 0) ? p.buf + (size_t)r * p.hv : p.zero_row;
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

// ------------------------------ bulk-copy variant ---------------------------
// Each warp owns a ring of `stages` shared-memory stages; a stage holds the same
// column chunk (32*U 16-byte units) of the k rows of one token.  Lane j < k asks
// the TMA engine for row j's chunk (one bulk copy each, all counted on the
// stage's mbarrier), so many kilobytes per warp are in flight without holding
// registers, and the warp only touches a stage once it has landed.  Items
// (token, chunk) are dealt to warps in contiguous runs, so a warp re-reads the
// row indices and coefficients only when it moves to the next token, and those
// are fetched one token ahead.
constexpr int kCombineBulkMaxWarps = 8;   // warps per CTA (blockDim.x / 32), each with its own ring

__device__ __forceinline__ void combine_fetch_index(const CombineParams &p, int t, int lane,
                                                    const uint4 *&row, float &coef)
{
    // An assignment whose slot or row is out of range (a row that did not fit its receive buffer,
    // or indices left behind by a routing kernel that gave up) reads the row of zeros instead.
    row = p.zero_row; coef = 0.0f;
    if (lane < p.k && t < p.T) {
        const size_t i = (size_t)t * p.k + lane;
        const int slot = __ldg(p.topk_slot + i);
        const int r = __ldg(p.dst_row + i);
        if ((unsigned)slot < (unsigned)p.P && r >= 0 && r < p.row_limit) {
            const uint4 *base = p.peer_bufs ? p.peer_bufs[slot / p.slots_per_gpu] : p.buf;
            row = base + (size_t)r * p.hv;
            coef = __fmul_rn(__ldg(p.topk_weights + i), __ldg(p.slot_scale + slot));
        }
    }
}

// U = 16-byte units per lane and row chunk; K > 0: top_k known at compile time (the row loop
// is unrolled), K == 0: any top_k.  All item bookkeeping is incremental: the loop is close to
// being bound by instruction issue, so no division or modulo runs per item.
template <int U, int K>
__global__ void __launch_bounds__(kCombineBulkMaxWarps * 32) k_combine_bulk(CombineParams p, int stages,
                                                                         Control *ctl)
{
    extern __shared__ __align__(128) unsigned char dyn[];
    constexpr int kChunkV = 32 * U;                       // 16-byte units per row chunk
    constexpr unsigned kChunkBytes = kChunkV * 16u;
    const int lane = lane_id(), warp = threadIdx.x >> 5;
    const int kCombineBulkWarps = blockDim.x >> 5;
    const int k = (K > 0) ? K : p.k;
    const unsigned stage_bytes = (unsigned)k * kChunkBytes;
    // per-warp carve-up: [stages][k][chunk] data, then [stages][k] coefficients, then barriers
    const size_t warp_bytes = (size_t)stages * stage_bytes;
    unsigned char *ring = dyn + (size_t)warp * warp_bytes;
    float *coefs = reinterpret_cast<float *>(dyn + (size_t)kCombineBulkWarps * warp_bytes) +
                   (size_t)warp * stages * k;
    uint64_t *full = reinterpret_cast<uint64_t *>(
                         dyn + (size_t)kCombineBulkWarps * warp_bytes +
                         (((size_t)kCombineBulkWarps * stages * k * 4 + 7) & ~(size_t)7)) +
                     (size_t)warp * stages;

    if (lane == 0) {
        for (int s = 0; s < stages; ++s) mbar_init(&full[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const int chunks = (p.hv + kChunkV - 1) / kChunkV;
    const long long items = (long long)p.T * chunks;
    const long long nwarps = (long long)gridDim.x * kCombineBulkWarps;
    const long long wid = (long long)blockIdx.x * kCombineBulkWarps + warp;
    const long long per = items / nwarps, extra = items % nwarps;      // contiguous, balanced runs
    const long long first = wid * per + (wid < extra ? wid : extra);
    const int n_mine = (int)(per + (wid < extra ? 1 : 0));

    // issuing side: token / chunk / stage of the next item to request (lane j < k owns row j)
    int it_tok = (int)(first / chunks), it_chunk = (int)(first % chunks), it_stage = 0;
    const uint4 *row, *row_next; float coef, coef_next;
    // The ring is set up and the run is known; only now wait for the previous kernel (the one
    // that filled the rows and wrote dst_row).
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (n_mine == 0) return;
    combine_fetch_index(p, it_tok, lane, row, coef);
    combine_fetch_index(p, it_tok + 1, lane, row_next, coef_next);

    auto issue = [&]() {
        const int c0 = it_chunk * kChunkV;
        const unsigned bytes = (unsigned)min(kChunkV, p.hv - c0) * 16u;
        if (lane == 0) mbar_expect_tx(&full[it_stage], bytes * (unsigned)k);
        __syncwarp();
        if (lane < k) {
            coefs[it_stage * k + lane] = coef;
            bulk_load(ring + (size_t)it_stage * stage_bytes + (size_t)lane * kChunkBytes, row + c0, bytes,
                      &full[it_stage]);
        }
        if (++it_stage == stages) it_stage = 0;
        if (++it_chunk == chunks) {                        // next token: take the prefetched indices
            it_chunk = 0; ++it_tok;
            row = row_next; coef = coef_next;
            combine_fetch_index(p, it_tok + 1, lane, row_next, coef_next);
        }
    };

    const int ahead = min(stages - 1, n_mine);
    for (int n = 0; n < ahead; ++n) issue();

    // consuming side
    int tok = (int)(first / chunks), chunk = (int)(first % chunks), stage = 0;
    unsigned parity = 0;
    bool ok = true;
    int n = 0;
    for (; n < n_mine; ++n) {
        if (n + stages - 1 < n_mine) issue();              // refills the stage consumed at n-1
        unsigned spins = 0;
        while (!mbar_try_wait(&full[stage], parity)) {
            if (++spins > p.spin_limit) { ok = false; break; }
        }
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        __syncwarp();                                      // coefficients written at issue are visible
        const int c0 = chunk * kChunkV + lane;
        float acc[U][8];
#pragma unroll
        for (int u = 0; u < U; ++u)
#pragma unroll
            for (int q = 0; q < 8; ++q) acc[u][q] = 0.0f;
        const uint4 *st = reinterpret_cast<const uint4 *>(ring + (size_t)stage * stage_bytes);
        const float *cf = coefs + stage * k;
        if (K > 0) {
            uint4 v[K > 0 ? K : 1][U];
            float c[K > 0 ? K : 1];
#pragma unroll
            for (int j = 0; j < K; ++j) {
                c[j] = cf[j];
#pragma unroll
                for (int u = 0; u < U; ++u)
                    if (c0 + 32 * u < p.hv) v[j][u] = st[j * kChunkV + lane + 32 * u];
            }
#pragma unroll
            for (int j = 0; j < K; ++j)
#pragma unroll
                for (int u = 0; u < U; ++u)
                    if (c0 + 32 * u < p.hv) fma_bf16x8(acc[u], v[j][u], c[j]);
        } else {
            for (int j = 0; j < k; ++j) {
                const float c = cf[j];
#pragma unroll
                for (int u = 0; u < U; ++u)
                    if (c0 + 32 * u < p.hv) fma_bf16x8(acc[u], st[j * kChunkV + lane + 32 * u], c);
            }
        }
        uint4 *dst = p.y + (size_t)tok * p.hv;
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (c0 + 32 * u < p.hv) st_stream_v4(dst + c0 + 32 * u, pack_bf16x8(acc[u]));
        __syncwarp();                                      // every lane is done reading the stage
        if (++stage == stages) { stage = 0; parity ^= 1u; }
        if (++chunk == chunks) { chunk = 0; ++tok; }
    }
    if (!ok) {
        if (lane == 0) report_status(ctl, kDevTimeout);
        // copies issued for items n .. n+stages-1 may still be landing in this CTA's shared
        // memory: give each a bounded chance to finish before the memory is released
        for (int m = n; m < min(n_mine, n + stages); ++m) {
            unsigned spins = 0;
            while (!mbar_try_wait(&full[m % stages], (unsigned)(m / stages) & 1u) && ++spins < p.spin_limit) {}
        }
    }
}

__host__ __device__ inline size_t combine_bulk_smem(int stages, int k, int U, int kCombineBulkWarps)
{
    const size_t warp_bytes = (size_t)stages * k * 32 * U * 16;
    const size_t coef_bytes = ((size_t)kCombineBulkWarps * stages * k * 4 + 7) & ~(size_t)7;
    return kCombineBulkWarps * warp_bytes + coef_bytes + (size_t)kCombineBulkWarps * stages * 8;
}

}  // namespace moe
