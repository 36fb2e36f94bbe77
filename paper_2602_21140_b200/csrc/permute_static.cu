// moe_permute_static: the count / prefix-scan / stable-permutation step of a
// dispatch for callers that must not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc once they are running: a
// serving engine that has handed the whole of HBM to its own pool at start-up
// (a later cudaMalloc simply fails), or code that runs where the runtime
// forbids allocation.  For them the per-tile histograms this step needs live
// in a fixed array in the library's own device image instead of in a context
// created by moe_route_init.  Every GPU that loads the library carries that
// array (kStaticTiles * kStaticSlots * 4 bytes = 512 KiB) until the process
// exits, which is why the sizes are capped.
//
// Three launches, no waits between thread blocks:
//   1. k_static_hist : tile b (1024 consecutive assignments) counts its
//                      assignments per slot into scratch[b][0..P).
//   2. k_static_scan : one block turns the columns of scratch into exclusive
//                      prefixes over tiles, emits slot_counts / slot_offsets and
//                      adds each slot's offset to its column, so that
//                      scratch[b][p] = first row of tile b's share of slot p.
//   3. k_static_place: tile b ranks its assignments stably inside the tile and
//                      writes dst_row and src_index.
// Every scratch word that is read was written earlier in the same call, so the
// contents a previous call left behind never matter and nothing needs zeroing.
// Two calls that overlap on the GPU (different streams) share the array and
// race; keep calls on one stream or order them with events.
#include "../../include/moe_route.h"

#include <cuda_runtime.h>

#include <mutex>

namespace {

constexpr int kStaticTileItems = 1024;                 // assignments per tile
constexpr int kStaticTiles = 256;                      // => at most 262144 assignments
constexpr int kStaticSlots = 512;                      // physical slots
constexpr int kStaticThreads = 256;
constexpr int kStaticWarps = kStaticThreads / 32;
constexpr int kMaxDevices = 64;

// The scratch itself.  In host code this name is only a handle for the runtime
// (cudaGetSymbolAddress turns it into a device pointer); device code may use it
// directly.
static __device__ __align__(256) int32_t g_static_scratch[kStaticTiles * kStaticSlots];

__global__ void __launch_bounds__(kStaticThreads)
k_static_hist(const int32_t *__restrict__ slot, int n, int P, int32_t *__restrict__ scratch)
{
    __shared__ int s_hist[kStaticSlots];
    for (int p = threadIdx.x; p < P; p += kStaticThreads) s_hist[p] = 0;
    __syncthreads();
    const int base = blockIdx.x * kStaticTileItems;
    for (int i = base + threadIdx.x; i < min(n, base + kStaticTileItems); i += kStaticThreads) {
        const int sl = slot[i];
        if ((unsigned)sl < (unsigned)P) atomicAdd(&s_hist[sl], 1);   // ids outside [0,P) are ignored
    }
    __syncthreads();
    for (int p = threadIdx.x; p < P; p += kStaticThreads) scratch[blockIdx.x * P + p] = s_hist[p];
}

__global__ void __launch_bounds__(kStaticSlots)
k_static_scan(int tiles, int P, int R, int S, int32_t *__restrict__ scratch,
              int32_t *__restrict__ slot_counts, int32_t *__restrict__ slot_offsets,
              int32_t *__restrict__ rank_counts, int32_t *__restrict__ rank_offsets)
{
    __shared__ int s_tot[kStaticSlots];
    __shared__ int s_off[kStaticSlots + 1];
    const int p = threadIdx.x;
    int run = 0;
    if (p < P) {
        for (int b = 0; b < tiles; ++b) {            // column p: exclusive prefix over tiles
            const int c = scratch[b * P + p];
            scratch[b * P + p] = run;
            run += c;
        }
    }
    s_tot[p] = (p < P) ? run : 0;
    __syncthreads();
    if (p == 0) {                                     // P <= 512: a serial scan is plenty here
        int acc = 0;
        for (int q = 0; q < P; ++q) { s_off[q] = acc; acc += s_tot[q]; }
        s_off[P] = acc;
    }
    __syncthreads();
    if (p < P) {
        slot_counts[p] = s_tot[p];
        slot_offsets[p] = s_off[p];
        for (int b = 0; b < tiles; ++b) scratch[b * P + p] += s_off[p];
    }
    if (p == 0) { slot_offsets[P] = s_off[P]; rank_offsets[R] = s_off[P]; }
    for (int r = p; r < R; r += kStaticSlots) {
        int c = 0;
        for (int s = 0; s < S; ++s) c += s_tot[r * S + s];
        rank_counts[r] = c;
        rank_offsets[r] = s_off[r * S];
    }
}

__global__ void __launch_bounds__(kStaticThreads)
k_static_place(const int32_t *__restrict__ slot, int n, int P, const int32_t *__restrict__ scratch,
               int32_t *__restrict__ dst_row, int32_t *__restrict__ src_index)
{
    __shared__ int s_run[kStaticSlots];                   // rows of slot p already handed out
    __shared__ int s_wcount[kStaticWarps][kStaticSlots];  // per-warp counts of the current round
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int p = tid; p < P; p += kStaticThreads) s_run[p] = scratch[blockIdx.x * P + p];
    for (int q = tid; q < kStaticWarps * kStaticSlots; q += kStaticThreads) (&s_wcount[0][0])[q] = 0;
    __syncthreads();
    const int base = blockIdx.x * kStaticTileItems;
    for (int round = 0; round < kStaticTileItems / kStaticThreads; ++round) {
        const int i = base + round * kStaticThreads + tid;
        int sl = (i < n) ? slot[i] : -1;
        if ((unsigned)sl >= (unsigned)P) sl = -1;
        const unsigned peers = __match_any_sync(0xffffffffu, sl);
        const int before = __popc(peers & ((1u << lane) - 1u));
        if (sl >= 0 && before == 0) s_wcount[warp][sl] = __popc(peers);
        __syncthreads();
        if (sl >= 0) {
            int row = s_run[sl] + before;
            for (int w = 0; w < warp; ++w) row += s_wcount[w][sl];
            dst_row[i] = row;
            src_index[row] = i;
        }
        __syncthreads();
        for (int p = tid; p < P; p += kStaticThreads) {
            int tot = 0;
            for (int w = 0; w < kStaticWarps; ++w) { tot += s_wcount[w][p]; s_wcount[w][p] = 0; }
            s_run[p] += tot;
        }
        __syncthreads();
    }
}

// Device address of g_static_scratch, looked up once per device.
std::mutex g_lock;
int32_t *g_scratch_ptr[kMaxDevices] = {nullptr};

moe_status static_scratch(int32_t **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MOE_ERR_CUDA;
    std::lock_guard<std::mutex> guard(g_lock);
    if (!g_scratch_ptr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return MOE_ERR_CUDA;
        }
        g_scratch_ptr[dev] = static_cast<int32_t *>(p);
    }
    *out = g_scratch_ptr[dev];
    return MOE_OK;
}

}  // namespace

extern "C" moe_status moe_permute_static(const int32_t *topk_slot, int32_t n_assign,
                                         int32_t num_ranks, int32_t slots_per_rank,
                                         int32_t *slot_counts, int32_t *slot_offsets,
                                         int32_t *rank_counts, int32_t *rank_offsets,
                                         int32_t *dst_row, int32_t *src_index, void *cuda_stream)
{
    if (n_assign < 0 || num_ranks < 1 || slots_per_rank < 1) return MOE_ERR_INVALID_ARG;
    const long long P = (long long)num_ranks * slots_per_rank;
    if (P > kStaticSlots || n_assign > kStaticTiles * kStaticTileItems) return MOE_ERR_CAPACITY;
    if (!slot_counts || !slot_offsets || !rank_counts || !rank_offsets) return MOE_ERR_INVALID_ARG;
    if (n_assign > 0 && (!topk_slot || !dst_row || !src_index)) return MOE_ERR_INVALID_ARG;
    int32_t *scratch = nullptr;
    const moe_status ms = static_scratch(&scratch);
    if (ms != MOE_OK) return ms;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int tiles = (n_assign + kStaticTileItems - 1) / kStaticTileItems;
    if (tiles > 0) k_static_hist<<<tiles, kStaticThreads, 0, st>>>(topk_slot, n_assign, (int)P, scratch);
    k_static_scan<<<1, kStaticSlots, 0, st>>>(tiles, (int)P, num_ranks, slots_per_rank, scratch,
                                             slot_counts, slot_offsets, rank_counts, rank_offsets);
    if (tiles > 0)
        k_static_place<<<tiles, kStaticThreads, 0, st>>>(topk_slot, n_assign, (int)P, scratch, dst_row,
                                                        src_index);
    return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}
