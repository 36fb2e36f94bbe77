// K_scatter: finish the permutation (dst_row, src_index) and copy every token's
// bf16 row into its k rows of the expert-contiguous send buffer.  Each x row is
// read from HBM once and written k times: (1 + k) rows of traffic per token.
//
// Two implementations of the same copy:
//   k_scatter_vec  — 128-bit loads/stores, a warp per (token, 2 KB column chunk).
//   k_scatter_bulk — the row is staged in shared memory by one bulk async copy
//                    (TMA engine, mbarrier completion) and leaves as k bulk
//                    stores; a multi-stage ring keeps loads ahead of stores.
#pragma once

#include "device_utils.cuh"

namespace moe {

struct ScatterParams {
    const uint4 *x;               // [T, H/8] 16-byte units
    uint4 *send;                  // [T*k, H/8]
    int T, k, hv;                 // hv = H/8 (uint4 per row)
    int P;                        // physical slots
    unsigned spin_limit;          // polls before a bounded wait gives up
    const int32_t *topk_slot;     // [T,k]
    const int32_t *slot_offsets;  // [P+1]
    const int32_t *pos_in_slot;   // [T*k] stable rank inside the slot (routing kernel's scratch)
    int32_t *dst_row;             // out: send-buffer row of assignment i
    int32_t *src_index;           // out: inverse permutation
    Control *ctl;
};

constexpr int kScatterThreads = 256;

// Last step of the permutation: row = slot_offsets[slot] + rank inside the slot.  Lane j < k
// owns assignment t*k + j.  Only read-only inputs are used, so any number of
// warps may resolve the same token; exactly one of them writes the result.
// A slot or row outside its range (possible only if the routing kernel gave up and left
// stale indices behind) yields -1: the assignment is recorded as not placed and no row is written.
__device__ __forceinline__ int resolve_row(const ScatterParams &p, int t, int lane, bool write_back)
{
    int row = -1;
    if (lane < p.k) {
        const size_t i = (size_t)t * p.k + lane;
        const int slot = __ldg(p.topk_slot + i);
        if ((unsigned)slot < (unsigned)p.P) {
            const long long r = (long long)__ldg(p.slot_offsets + slot) + __ldg(p.pos_in_slot + i);
            if (r >= 0 && r < (long long)p.T * p.k) row = (int)r;
        }
        if (write_back) {
            p.dst_row[i] = row;
            if (row >= 0) p.src_index[row] = (int)i;
        }
    }
    return row;
}

// UNROLL = 16-byte loads in flight per lane; a work item is 32*UNROLL 16-byte units of a row.
// POLICY = cache policy of the stores (0, the default: no L1 allocation; the others exist to
// measure what the write policy does to the combine that follows, see st_policy_v4).
template <int UNROLL, int POLICY = 0>
__global__ void __launch_bounds__(kScatterThreads) k_scatter_vec(ScatterParams p)
{
    constexpr int kChunk = 32 * UNROLL;
    const unsigned full = 0xffffffffu;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int lane = lane_id();
    const int chunks = (p.hv + kChunk - 1) / kChunk;
    const long long items = (long long)p.T * chunks;
    const long long warp0 = (long long)blockIdx.x * (kScatterThreads / 32) + (threadIdx.x >> 5);
    const long long nwarps = (long long)gridDim.x * (kScatterThreads / 32);

    const unsigned long long pol = (POLICY == 2) ? l2_policy_evict_first() : 0ull;
    bool waited = false;
    for (long long it = warp0; it < items; it += nwarps) {
        const int t = (int)(it / chunks);
        const int c0 = (int)(it % chunks) * kChunk + lane;
        const uint4 *src = p.x + (size_t)t * p.hv;
        uint4 v[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u)
            if (c0 + 32 * u < p.hv) v[u] = ld_stream_v4(src + c0 + 32 * u);
        if (!waited) {
            // x is an input of the dispatch, not a product of the routing kernel: the first rows
            // are requested while that kernel is still finishing, and only the destinations
            // (which it computes) wait for it
            asm volatile("griddepcontrol.wait;" ::: "memory");
            waited = true;
        }
        const int row = resolve_row(p, t, lane, it % chunks == 0);
        for (int j = 0; j < p.k; ++j) {
            const int r = __shfl_sync(full, row, j);
            if (r < 0) continue;
            uint4 *dst = p.send + (size_t)r * p.hv;
#pragma unroll
            for (int u = 0; u < UNROLL; ++u)
                if (c0 + 32 * u < p.hv) st_policy_v4<POLICY>(dst + c0 + 32 * u, v[u], pol);
        }
    }
}

// --------------------------- bulk-copy variant -----------------------------

constexpr int kBulkThreads = 32;   // one warp per CTA; several CTAs share an SM

// One warp per CTA walks tokens blockIdx.x, blockIdx.x + gridDim.x, ...  Stage s
// of the ring holds one row.  Lane 0 issues the loads; lane j < k issues the
// store of row j, so the k stores of a token leave from k different threads.
// Before a stage is refilled every lane waits until its own earlier stores have
// finished READING shared memory (they may still be in flight to HBM).
__global__ void __launch_bounds__(kBulkThreads) k_scatter_bulk(ScatterParams p, int stages)
{
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ __align__(8) uint64_t full_bar[8];
    const int lane = lane_id();
    const unsigned row_bytes = (unsigned)p.hv * 16u;
    const unsigned stage_bytes = (row_bytes + 127u) & ~127u;

    if (lane == 0) {
        for (int s = 0; s < stages; ++s) mbar_init(&full_bar[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();

    const int first = blockIdx.x, step = gridDim.x;
    const int n_mine = (first < p.T) ? (p.T - first + step - 1) / step : 0;

    // prologue: fill the ring except one stage
    if (lane == 0) {
        for (int n = 0; n < min(stages - 1, n_mine); ++n) {
            mbar_expect_tx(&full_bar[n], row_bytes);
            bulk_load(ring + (size_t)n * stage_bytes,
                      p.x + (size_t)(first + (size_t)n * step) * p.hv, row_bytes, &full_bar[n]);
        }
    }
    bool ok = true;
    int n_failed_at = 0;
    for (int n = 0; n < n_mine && ok; ++n) {
        const int t = first + n * step;
        const int s = n % stages;
        const int row = resolve_row(p, t, lane, true);
        // refill the stage freed in the previous iteration with token n + stages - 1
        const int n_next = n + stages - 1;
        if (n_next < n_mine) {
            if (n > 0) bulk_wait_read<0>();      // my store of iteration n-1 has left shared memory
            __syncwarp();
            if (lane == 0) {
                const int sn = n_next % stages;
                mbar_expect_tx(&full_bar[sn], row_bytes);
                bulk_load(ring + (size_t)sn * stage_bytes,
                          p.x + (size_t)(first + (size_t)n_next * step) * p.hv, row_bytes,
                          &full_bar[sn]);
            }
        }
        // wait for this token's row
        const unsigned parity = (unsigned)(n / stages) & 1u;
        unsigned spins = 0;
        while (!mbar_try_wait(&full_bar[s], parity)) {
            if (++spins > p.spin_limit) { ok = false; break; }
        }
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { n_failed_at = n; break; }
        if (lane < p.k && row >= 0) {
            bulk_store(p.send + (size_t)row * p.hv, ring + (size_t)s * stage_bytes, row_bytes);
            bulk_commit();
        }
    }
    if (!ok) {
        if (lane == 0) report_status(p.ctl, kDevTimeout);
        // loads requested for tokens n_failed_at .. n_failed_at+stages-1 may still be landing in this
        // CTA's shared memory: give each a bounded chance to finish before the memory is released
        for (int m = n_failed_at; m < min(n_mine, n_failed_at + stages); ++m) {
            unsigned spins = 0;
            while (!mbar_try_wait(&full_bar[m % stages], (unsigned)(m / stages) & 1u) && ++spins < p.spin_limit) {}
        }
    }
    bulk_wait_all();   // nothing of this CTA may still read the ring or write HBM at exit
}

}  // namespace moe
