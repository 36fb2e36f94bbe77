// Expert parallelism over several GPUs: the dispatch exchange (attention2expert) as
// direct stores into the receive buffers of the GPUs that host the chosen slots, with
// no staging send buffer and no separate all-to-all.
//
// GPU d of a group of G hosts the physical slots [d*spg, (d+1)*spg), spg = P/G.  Its
// receive buffer is expert-contiguous: the rows of slot p come before those of slot
// p+1, and inside a slot the rows of source GPU 0 come first, then source 1, ..., each
// source's rows in its own stable order (ascending assignment index i = t*k + j).
// With counts[g][p] = assignments of source g on slot p (every GPU holds the whole
// table after one small all-gather), source g's rows for slot p start at row
//   sum_{p' hosted by the same GPU, p' < p} sum_{g'} counts[g'][p']  +  sum_{g' < g} counts[g'][p].
#pragma once

#include "device_utils.cuh"

namespace moe {

constexpr int kEpPlanThreads = 1024;

struct EpPlanParams {
    const int32_t *counts;        // [G][P], device
    int G, g, P, spg;
    long long recv_rows;          // capacity of every receive buffer
    int32_t *src_base;            // out [P]: first row, in the owner's buffer, of this GPU's rows for slot p
    int32_t *recv_slot_offsets;   // out [spg+1]: layout of THIS GPU's receive buffer (exclusive prefix)
    Control *ctl;
};

// One small block.  First the total of every slot over all senders goes to shared memory,
// then every output element is a plain sum over (part of) its owner's run of slots.
constexpr int kEpMaxSlots = 4096;

__global__ void __launch_bounds__(kEpPlanThreads) k_ep_plan(EpPlanParams p)
{
    __shared__ int32_t s_tot[kEpMaxSlots];
    pdl_enter();
    for (int s = threadIdx.x; s < p.P; s += kEpPlanThreads) {
        int tot = 0;
        for (int g2 = 0; g2 < p.G; ++g2) tot += p.counts[(size_t)g2 * p.P + s];
        s_tot[s] = tot;
    }
    __syncthreads();
    for (int s = threadIdx.x; s < p.P; s += kEpPlanThreads) {
        const int first = (s / p.spg) * p.spg;
        long long base = 0;
        for (int q = first; q < s; ++q) base += s_tot[q];
        for (int g2 = 0; g2 < p.g; ++g2) base += p.counts[(size_t)g2 * p.P + s];
        p.src_base[s] = (int32_t)min(base, (long long)0x7fffffff);
    }
    for (int q = threadIdx.x; q <= p.spg; q += kEpPlanThreads) {
        long long off = 0;
        for (int q2 = 0; q2 < q; ++q2) off += s_tot[p.g * p.spg + q2];
        p.recv_slot_offsets[q] = (int32_t)min(off, (long long)0x7fffffff);
        if (q == p.spg && off > p.recv_rows) report_status(p.ctl, kDevCapacity);
    }
}

struct EpScatterParams {
    const uint4 *x;               // [T, H/8]
    uint4 *const *peer_bufs;      // device [G]: every GPU's receive buffer as seen from this GPU
    int T, k, hv, spg, P;
    long long recv_rows;
    const int32_t *topk_slot;     // [T,k]
    const int32_t *src_base;      // [P]
    const int32_t *pos_in_slot;   // [T*k]: stable rank of assignment i among this GPU's rows of its slot
    int32_t *dst_row;             // out [T*k]: row of assignment i in the owner's receive buffer
};

constexpr int kEpScatterThreads = 256;

// A warp takes (token, piece of 32*UNROLL 16-byte units of the row), loads the piece once
// and stores it into the k owners' buffers.  A row that would fall outside the owner's
// buffer is not written and its dst_row becomes -1 (the owner's plan kernel reports the
// overflow; the combine treats the assignment as contributing zero).
template <int UNROLL>
__global__ void __launch_bounds__(kEpScatterThreads) k_ep_scatter(EpScatterParams p)
{
    constexpr int kChunk = 32 * UNROLL;
    const unsigned full = 0xffffffffu;
    pdl_enter();
    const int lane = lane_id();
    const int chunks = (p.hv + kChunk - 1) / kChunk;
    const long long items = (long long)p.T * chunks;
    const long long warp0 = (long long)blockIdx.x * (kEpScatterThreads / 32) + (threadIdx.x >> 5);
    const long long nwarps = (long long)gridDim.x * (kEpScatterThreads / 32);

    for (long long it = warp0; it < items; it += nwarps) {
        const int t = (int)(it / chunks);
        const int c0 = (int)(it % chunks) * kChunk + lane;
        const uint4 *src = p.x + (size_t)t * p.hv;
        uint4 v[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u)
            if (c0 + 32 * u < p.hv) v[u] = ld_stream_v4(src + c0 + 32 * u);
        unsigned long long dst_bits = 0;                   // 0 = do not write
        if (lane < p.k) {
            const size_t i = (size_t)t * p.k + lane;
            const int slot = __ldg(p.topk_slot + i);
            // 64-bit: the clamped base of a hopelessly overflowed buffer plus a rank must not wrap
            long long row = -1;
            if ((unsigned)slot < (unsigned)p.P)
                row = (long long)__ldg(p.src_base + slot) + __ldg(p.pos_in_slot + i);
            const bool fits = row >= 0 && row < p.recv_rows;
            // a row that does not fit is recorded as not placed (-1): the combine skips it
            if (it % chunks == 0) p.dst_row[i] = fits ? (int)row : -1;
            if (fits)
                dst_bits = reinterpret_cast<unsigned long long>(p.peer_bufs[slot / p.spg] + (size_t)row * p.hv);
        }
        for (int j = 0; j < p.k; ++j) {
            uint4 *dst = reinterpret_cast<uint4 *>(__shfl_sync(full, dst_bits, j));
            if (dst == nullptr) continue;
#pragma unroll
            for (int u = 0; u < UNROLL; ++u)
                if (c0 + 32 * u < p.hv) st_stream_v4(dst + c0 + 32 * u, v[u]);
        }
    }
}

}  // namespace moe
