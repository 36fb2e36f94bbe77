// Host side of the failure-aware MoE routing library: the C ABI declared in
// include/moe_route.h, the host half of a remap (validation, bitmap and replica
// table), context set-up and the kernel launches.  No CPU fallback exists: every
// step of the path runs in the kernels included below.
#include "../../include/moe_route.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "combine_kernels.cuh"
#include "ep_kernels.cuh"
#include "route_kernels.cuh"
#include "scatter_kernels.cuh"

namespace {

using namespace moe;

constexpr int kMaxExperts = 512;
constexpr int kMaxTopK = 16;
constexpr int kMaxReplicas = 8;
constexpr int kMaxSlots = 4096;
constexpr int kStagingSlots = 16;
constexpr size_t kMaxSmem = 227 * 1024;
constexpr int kRouteTileTarget = 148;   // tiles of a full step: one per SM of a B200
constexpr int kNumTuning = MOE_TUNE_SCATTER_STORE_POLICY + 1;

// Shape-derived launch constants.
struct Derived {
    int E, k, H, P, R, S, max_rep;
    int epl;               // experts per lane in the routing warp
    int lpt;               // lanes per token in the routing warp (8 or 16)
    int lanes_per_group;   // lanes holding one expert group (power of two), 0 if ungrouped
    int group_m;           // keys summed into a group score
    int rank_words;        // words of the rank bitmap
    int expert_words;      // words of the failed-expert bitmap
    int state_words;       // words of the whole routing-state blob
    int tokens_per_block;  // routing tile
    int p_pad;             // P rounded up to a multiple of 8 (row pitch of the per-tile counts)
    bool alias_wcount;     // routing kernel: count matrix shares the token tables' shared memory
};

bool is_pow2(int v) { return v > 0 && (v & (v - 1)) == 0; }

// `want_lpt` (8 or 16) and `want_tile` (tokens) override the automatic choices; 0 = automatic.
bool derive(const moe_config *c, Derived *d, int want_lpt = 0, int want_tile = 0)
{
    if (!c) return false;
    if (c->num_experts < 1 || c->num_experts > kMaxExperts) return false;
    if (c->top_k < 1 || c->top_k > kMaxTopK || c->top_k > c->num_experts) return false;
    if (c->hidden < 8 || c->hidden % 8 != 0) return false;
    if (c->max_tokens < 1 || c->max_tokens > 262144) return false;
    if (c->num_ranks < 1 || c->slots_per_rank < 1) return false;
    const long long P = (long long)c->num_ranks * c->slots_per_rank;
    if (P > kMaxSlots) return false;
    if (c->max_replicas < 1 || c->max_replicas > kMaxReplicas) return false;
    if (c->score_func != MOE_SCORE_SOFTMAX && c->score_func != MOE_SCORE_SIGMOID &&
        c->score_func != MOE_ROUTE_DENSE_TP)
        return false;
    if (c->score_func == MOE_ROUTE_DENSE_TP &&
        (c->n_group != 1 || c->num_experts % c->top_k != 0 || c->num_experts / c->top_k > 32 * c->top_k))
        return false;
    if (c->replica_policy != 0) return false;
    if (!(c->route_scale > 0.0f)) return false;
    if ((long long)c->max_tokens * c->top_k >= (1ll << 30)) return false;   // 30-bit scan counts
    d->E = c->num_experts; d->k = c->top_k; d->H = c->hidden; d->P = (int)P;
    d->R = c->num_ranks; d->S = c->slots_per_rank; d->max_rep = c->max_replicas;
    d->lanes_per_group = 0; d->group_m = 1;
    // lanes per token (8 or 16, at least k) and experts per lane: the smallest pair that
    // covers E and, with groups, puts every group on a power-of-two run of whole lanes
    static const int kEpl[] = {1, 2, 3, 4, 5, 6, 8, 10, 12, 16, 20, 24, 32};
    static const int kLpt[] = {8, 16};
    d->epl = 0; d->lpt = 0;
    if (c->n_group > 1) {
        if (c->topk_group < 1 || c->topk_group > c->n_group) return false;
        if (d->E % c->n_group != 0 || d->k % c->topk_group != 0) return false;
        d->group_m = d->k / c->topk_group;
        if (d->group_m != 1 && d->group_m != 2) return false;
    } else if (c->n_group != 1) {
        return false;
    }
    // 16 lanes per token above 64 experts: twice the warps in flight for the same work,
    // which measured faster than 8 lanes (the kernel is issue/latency bound)
    // ... as long as a tile is then routed in one pass of the CTA's warps (64 tokens with 16
    // lanes each).  Larger tiles take several passes, each of which waits for its logits anew;
    // eight lanes per token route 128 tokens per pass and win there (-3 us per step at 16384
    // tokens and 128 experts, -7 us at 32768), so they are tried first when the shape allows them.
    const int tile_tokens = want_tile > 0 ? want_tile
                                          : std::max(32, (c->max_tokens + kRouteTileTarget - 1) / kRouteTileTarget);
    if (want_lpt != 8 && want_lpt != 16) want_lpt = (d->E > 64 && tile_tokens <= 64) ? 16 : 0;
    for (int lpt : kLpt) {
        if (d->epl || d->k > lpt || (want_lpt && lpt < want_lpt)) continue;
        for (int epl : kEpl) {
            if (lpt * epl < d->E) continue;
            if (c->n_group > 1) {
                const int per = d->E / c->n_group;
                if (per % epl != 0) continue;
                const int lpg = per / epl;
                if (!is_pow2(lpg) || lpg * c->n_group > lpt) continue;
                d->lanes_per_group = lpg;
            }
            d->epl = epl; d->lpt = lpt;
            break;
        }
    }
    if (d->epl == 0) return false;
    d->rank_words = (d->R + 31) / 32;
    d->expert_words = (d->E + 31) / 32;
    d->state_words = kStateHeaderWords + d->rank_words + d->expert_words + d->E * d->max_rep + d->P;
    d->p_pad = (d->P + 7) & ~7;
    // Routing tile: a full step should have one tile per SM (a tile is one CTA, and all tiles of
    // a step run in one wave), but never fewer than 32 tokens; a multiple of the tokens a warp
    // routes at once.  Halved until the tile's tables fit in shared memory.
    const int per_warp = 32 / d->lpt;
    int tile = want_tile > 0 ? want_tile : std::max(32, (c->max_tokens + kRouteTileTarget - 1) / kRouteTileTarget);
    // a batch that one CTA routes in a single pass of its 32 warps needs no prefix over tiles at all
    if (want_tile <= 0 && c->max_tokens <= kRouteWarps * per_warp) tile = c->max_tokens;
    tile = (tile + per_warp - 1) / per_warp * per_warp;
    // side by side if that fits with the smallest tile, else the count matrix shares the token tables
    d->alias_wcount = route_smem_bytes(d->E, d->max_rep, per_warp, d->k, d->P, d->epl, false) > kMaxSmem - 1024;
    const bool al = d->alias_wcount;
    while (tile > per_warp &&
           (route_smem_bytes(d->E, d->max_rep, tile, d->k, d->P, d->epl, al) > kMaxSmem - 1024 || (long long)tile * d->k > 65535))
        tile = (tile / 2 + per_warp - 1) / per_warp * per_warp;
    if (route_smem_bytes(d->E, d->max_rep, tile, d->k, d->P, d->epl, al) > kMaxSmem - 1024 || (long long)tile * d->k > 65535)
        return false;
    d->tokens_per_block = tile;
    if ((c->max_tokens + tile - 1) / tile > kMaxRouteTiles) return false;
    return true;
}

// Host half of a remap (Sec. 3.4): which ranks are alive, where each expert's
// replicas are, which experts are still served, and whether routing can always
// find k experts.  `blob` receives the device layout documented in
// route_kernels.cuh.
moe_status plan_state(const moe_config *c, const Derived &d, const int32_t *slot_to_expert,
                      const std::vector<uint8_t> &failed, const std::vector<uint8_t> &expert_failed,
                      const std::vector<int32_t> &rank_order, int n_listed,
                      std::vector<int32_t> *blob, int *n_available)
{
    // the layout order must give every alive rank a place among the listed ranks
    {
        std::vector<uint8_t> listed((size_t)d.R, 0);
        for (int i = 0; i < n_listed; ++i) listed[rank_order[i]] = 1;
        for (int r = 0; r < d.R; ++r)
            if (!failed[r] && !listed[r]) return MOE_ERR_INVALID_ARG;
    }
    std::vector<int32_t> out((size_t)d.state_words, -1);
    uint32_t *alive = reinterpret_cast<uint32_t *>(out.data() + kStateHeaderWords);
    for (int w = 0; w < d.rank_words; ++w) alive[w] = 0u;
    for (int r = 0; r < d.R; ++r)
        if (!failed[r]) alive[r >> 5] |= 1u << (r & 31);
    uint32_t *lost = reinterpret_cast<uint32_t *>(out.data() + kStateHeaderWords + d.rank_words);
    for (int w = 0; w < d.expert_words; ++w) lost[w] = 0u;
    for (int e = 0; e < d.E; ++e)
        if (expert_failed[e]) lost[e >> 5] |= 1u << (e & 31);
    int32_t *table = out.data() + kStateHeaderWords + d.rank_words + d.expert_words;
    std::vector<int> n_rep((size_t)d.E, 0), n_live((size_t)d.E, 0);
    for (int p = 0; p < d.P; ++p) {               // ascending p keeps each row ascending
        const int e = slot_to_expert[p];
        if (e < 0) continue;
        if (e >= d.E) return MOE_ERR_INVALID_ARG;
        if (n_rep[e] == d.max_rep) return MOE_ERR_CAPACITY;
        table[e * d.max_rep + n_rep[e]++] = p;
        if (!failed[p / d.S] && !expert_failed[e]) ++n_live[e];
    }
    int avail = 0, fallback = -1;
    for (int e = 0; e < d.E; ++e)
        if (n_live[e] > 0) { ++avail; if (fallback < 0) fallback = e; }
    bool ok;
    if (c->score_func == MOE_ROUTE_DENSE_TP) {
        // dense-FFN groups of k shards: at least one group must have every shard live
        int healthy = 0;
        for (int g = 0; g < d.E / d.k; ++g) {
            bool all = true;
            for (int sh = 0; sh < d.k; ++sh) all = all && n_live[g * d.k + sh] > 0;
            healthy += all;
        }
        ok = healthy >= 1;
        avail = healthy;
    } else if (c->n_group <= 1) {
        ok = avail >= d.k;
    } else {
        // worst case: the kept groups are the non-empty ones with the fewest experts
        const int per = d.E / c->n_group;
        std::vector<int> cnt;
        for (int g = 0; g < c->n_group; ++g) {
            int a = 0;
            for (int e = g * per; e < (g + 1) * per; ++e) a += n_live[e] > 0;
            if (a > 0) cnt.push_back(a);
        }
        std::sort(cnt.begin(), cnt.end());
        int worst = 0;
        for (size_t i = 0; i < cnt.size() && (int)i < c->topk_group; ++i) worst += cnt[i];
        ok = worst >= d.k;
    }
    if (!ok) return MOE_ERR_INSUFFICIENT_EXPERTS;
    int32_t *order = table + d.E * d.max_rep;          // send-buffer layout: slots in logical-rank order
    for (int l = 0; l < d.R; ++l)
        for (int sl = 0; sl < d.S; ++sl) order[l * d.S + sl] = rank_order[l] * d.S + sl;
    out[0] = fallback;
    out[1] = avail;
    if (blob) blob->swap(out);
    if (n_available) *n_available = avail;
    return MOE_OK;
}

}  // namespace

struct moe_ctx {
    moe_config cfg;
    Derived d;
    int device;
    int sm_count;
    // host mirror of the routing state
    std::vector<int32_t> slot_to_expert;
    std::vector<uint8_t> failed;
    std::vector<uint8_t> expert_failed;
    std::vector<int32_t> rank_order;   // physical rank at each logical position (full permutation)
    int n_listed;                      // leading entries given by the caller; the rest own no rows
    // device state
    int32_t *d_state;
    int32_t *d_live;           // live-replica lists derived from d_state (k_derive_live)
    float *d_bias;
    float *d_slot_scale;
    ulonglong2 *d_tile_counts; // [tiles][p_pad/4] epoch-tagged per-tile, per-slot counts of the running step
    size_t scan_tiles;         // rows the array above was allocated for
    moe::Control *d_ctl;
    int32_t *d_pos;
    uint4 *d_zero_row;         // [H/8] zeros: source of an assignment that was not placed
    size_t device_bytes;
    // pinned staging ring for stream-ordered remaps
    int32_t *h_stage[kStagingSlots];
    cudaEvent_t stage_done[kStagingSlots];
    bool stage_used[kStagingSlots];
    unsigned stage_next;
    // launch choices (configure_launch); tune[] holds the overrides of moe_set_tuning, -1 = automatic
    int tune[kNumTuning];
    unsigned spin_limit;   // polls before a bounded device wait gives up
    bool pdl;              // launch with the programmatic-dependent-launch attribute
    int scatter_impl;      // 0 = vector, 1 = bulk copies
    int bulk_stages, bulk_ctas_per_sm;
    int scatter_blocks_per_sm, combine_blocks_per_sm, scatter_unroll;
    int scatter_store_policy;   // 0 = default (no L1 allocation); 1 plain, 2 L2 evict-first, 3 streaming
    int route_prefetch;    // L2 hints issued by the routing kernel before its wait (bit 0 tables, bit 1 logits)
    int combine_impl;      // 0 = vector loads, 1 = bulk-copy ring
    int combine_stages, combine_u, combine_ctas_per_sm, combine_warps;
    size_t combine_smem;
    size_t route_smem;
    // what the latest dispatch wrote, for combine
    const float *last_weights;
    const int32_t *last_slot;
    const int32_t *last_dst_row;
    int32_t last_T;
    cudaEvent_t timing_event;   // optional: recorded between routing and scatter
    // expert parallelism over several GPUs (moe_ep_attach)
    int ep_world, ep_rank, ep_spg;
    long long ep_recv_rows;
    uint4 **d_peer_bufs;        // device [ep_world]
    int32_t *d_src_base;        // device [P]
    bool ep_routed;             // the latest routing came from moe_ep_route
};

namespace {

size_t device_bytes_for(const Derived &d, int max_tokens)
{
    const size_t tiles = ((size_t)max_tokens + d.tokens_per_block - 1) / d.tokens_per_block;
    size_t b = 0;
    b += (size_t)d.state_words * 4;
    b += (size_t)d.E * (1 + d.max_rep) * 4;
    b += (size_t)d.E * 4 + (size_t)d.P * 4;
    b += tiles * (d.p_pad / 4) * sizeof(ulonglong2);
    b += sizeof(moe::Control);
    b += (size_t)max_tokens * d.k * 4;
    b += (size_t)d.H * 2;
    return b;
}

// Launch with the programmatic-dependent-launch attribute (when `pdl`), so that the kernel's
// blocks can be scheduled while the previous kernel of the stream drains.
template <typename... KArgs, typename... Args>
cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                          bool pdl, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

template <int EPL, int LPT>
cudaError_t launch_route_t(const RouteParams &p, int tiles, size_t smem, cudaStream_t st, bool pdl)
{
    // the kernel also has a few hundred bytes of static shared memory: opt in to the large
    // carve-out a little below the 48 KB default limit, not exactly at it
    if (smem + 2048 > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(k_route<EPL, LPT>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    return launch_kernel(k_route<EPL, LPT>, dim3(tiles), dim3(kRouteThreads), smem, st, pdl, p);
}

template <int LPT>
cudaError_t launch_route_lpt(int epl, const RouteParams &p, int tiles, size_t smem, cudaStream_t st, bool pdl)
{
    switch (epl) {
        case 1: return launch_route_t<1, LPT>(p, tiles, smem, st, pdl);
        case 2: return launch_route_t<2, LPT>(p, tiles, smem, st, pdl);
        case 3: return launch_route_t<3, LPT>(p, tiles, smem, st, pdl);
        case 4: return launch_route_t<4, LPT>(p, tiles, smem, st, pdl);
        case 5: return launch_route_t<5, LPT>(p, tiles, smem, st, pdl);
        case 6: return launch_route_t<6, LPT>(p, tiles, smem, st, pdl);
        case 8: return launch_route_t<8, LPT>(p, tiles, smem, st, pdl);
        case 10: return launch_route_t<10, LPT>(p, tiles, smem, st, pdl);
        case 12: return launch_route_t<12, LPT>(p, tiles, smem, st, pdl);
        case 16: return launch_route_t<16, LPT>(p, tiles, smem, st, pdl);
        case 20: return launch_route_t<20, LPT>(p, tiles, smem, st, pdl);
        case 24: return launch_route_t<24, LPT>(p, tiles, smem, st, pdl);
        case 32: return launch_route_t<32, LPT>(p, tiles, smem, st, pdl);
    }
    return cudaErrorInvalidValue;
}

cudaError_t launch_route(int epl, int lpt, const RouteParams &p, int tiles, size_t smem, cudaStream_t st,
                         bool pdl)
{
    if (lpt == 8) return launch_route_lpt<8>(epl, p, tiles, smem, st, pdl);
    if (lpt == 16) return launch_route_lpt<16>(epl, p, tiles, smem, st, pdl);
    return cudaErrorInvalidValue;
}

cudaError_t launch_combine(const CombineParams &p, int blocks, cudaStream_t st)
{
    switch (p.k) {
        case 1: k_combine_vec<1><<<blocks, kCombineThreads, 0, st>>>(p); break;
        case 2: k_combine_vec<2><<<blocks, kCombineThreads, 0, st>>>(p); break;
        case 4: k_combine_vec<4><<<blocks, kCombineThreads, 0, st>>>(p); break;
        case 6: k_combine_vec<6><<<blocks, kCombineThreads, 0, st>>>(p); break;
        case 8: k_combine_vec<8><<<blocks, kCombineThreads, 0, st>>>(p); break;
        default: k_combine_vec<0><<<blocks, kCombineThreads, 0, st>>>(p); break;
    }
    return cudaGetLastError();
}

// The routing kernel of a dispatch: everything from the gate to the per-slot offsets and the
// rank of every assignment inside its slot (the scatter adds the slot's offset).
cudaError_t enqueue_route(moe_ctx *ctx, const float *logits, int32_t T, const moe_dispatch_out *out,
                          cudaStream_t st)
{
    const Derived &d = ctx->d;
    RouteParams rp;
    rp.logits = logits; rp.T = T; rp.E = d.E; rp.k = d.k; rp.P = d.P; rp.R = d.R; rp.S = d.S;
    rp.max_rep = d.max_rep; rp.score_func = ctx->cfg.score_func; rp.n_group = ctx->cfg.n_group;
    rp.topk_group = ctx->cfg.topk_group; rp.lanes_per_group = d.lanes_per_group;
    rp.group_m = d.group_m; rp.route_scale = ctx->cfg.route_scale;
    rp.tokens_per_block = d.tokens_per_block; rp.p_pad = d.p_pad; rp.rank_words = d.rank_words;
    rp.expert_words = d.expert_words; rp.spin_limit = ctx->spin_limit;
    rp.state = ctx->d_state; rp.live = ctx->d_live; rp.bias = ctx->d_bias;
    rp.topk_ids = out->topk_ids; rp.topk_weights = out->topk_weights; rp.topk_slot = out->topk_slot;
    rp.pos_in_slot = ctx->d_pos;
    rp.slot_counts = out->slot_counts; rp.slot_offsets = out->slot_offsets;
    rp.rank_counts = out->rank_counts; rp.rank_offsets = out->rank_offsets;
    rp.tile_counts = ctx->d_tile_counts; rp.ctl = ctx->d_ctl;
    rp.prefetch = ctx->pdl ? ctx->route_prefetch : 0;
    rp.alias_wcount = d.alias_wcount ? 1 : 0;
    const int tiles = (T + d.tokens_per_block - 1) / d.tokens_per_block;
    return launch_route(d.epl, d.lpt, rp, tiles, ctx->route_smem, st, ctx->pdl);
}

// The bulk-copy ring combine over `cp` (rows in one buffer, or in the peers' receive buffers).
moe_status enqueue_combine_bulk(moe_ctx *ctx, const CombineParams &cp, cudaStream_t st)
{
    const int chunk_v = 32 * ctx->combine_u;
    const long long items = (long long)cp.T * ((cp.hv + chunk_v - 1) / chunk_v);
    const int nw = ctx->combine_warps;
    const long long want = (items + nw - 1) / nw;
    const int grid = (int)std::min<long long>(want, (long long)ctx->sm_count * ctx->combine_ctas_per_sm);
    const dim3 g(grid), b(nw * 32);
    const size_t sm = ctx->combine_smem;
    const int stg = ctx->combine_stages;
    const bool pdl = ctx->pdl;
    moe::Control *ctl = ctx->d_ctl;
    const int key = ctx->combine_u * 100 + ((cp.k == 8 || cp.k == 2) ? cp.k : 0);
    switch (key) {
        case 108: launch_kernel(k_combine_bulk<1, 8>, g, b, sm, st, pdl, cp, stg, ctl); break;
        case 208: launch_kernel(k_combine_bulk<2, 8>, g, b, sm, st, pdl, cp, stg, ctl); break;
        case 408: launch_kernel(k_combine_bulk<4, 8>, g, b, sm, st, pdl, cp, stg, ctl); break;
        case 102: launch_kernel(k_combine_bulk<1, 2>, g, b, sm, st, pdl, cp, stg, ctl); break;
        case 202: launch_kernel(k_combine_bulk<2, 2>, g, b, sm, st, pdl, cp, stg, ctl); break;
        case 402: launch_kernel(k_combine_bulk<4, 2>, g, b, sm, st, pdl, cp, stg, ctl); break;
        case 100: launch_kernel(k_combine_bulk<1, 0>, g, b, sm, st, pdl, cp, stg, ctl); break;
        case 200: launch_kernel(k_combine_bulk<2, 0>, g, b, sm, st, pdl, cp, stg, ctl); break;
        default: launch_kernel(k_combine_bulk<4, 0>, g, b, sm, st, pdl, cp, stg, ctl); break;
    }
    return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Rebuild the live-replica lists from the bitmaps and the replica table, on the stream,
// behind the state copy that precedes it.
moe_status enqueue_derive(moe_ctx *ctx, cudaStream_t st)
{
    const Derived &d = ctx->d;
    DeriveParams dp;
    dp.state = ctx->d_state; dp.E = d.E; dp.S = d.S; dp.max_rep = d.max_rep;
    dp.rank_words = d.rank_words; dp.expert_words = d.expert_words; dp.live = ctx->d_live;
    k_derive_live<<<(d.E + kDeriveThreads - 1) / kDeriveThreads, kDeriveThreads, 0, st>>>(dp);
    return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

// Copy `words` leading words of `blob` to the device state through a pinned
// staging slot, ordered on `st`.  A slot is reused only after its copy has run.
moe_status push_state(moe_ctx *ctx, const std::vector<int32_t> &blob, int words, cudaStream_t st)
{
    const unsigned s = ctx->stage_next % kStagingSlots;
    if (ctx->stage_used[s] && cudaEventSynchronize(ctx->stage_done[s]) != cudaSuccess)
        return MOE_ERR_CUDA;
    std::memcpy(ctx->h_stage[s], blob.data(), (size_t)words * 4);
    if (cudaMemcpyAsync(ctx->d_state, ctx->h_stage[s], (size_t)words * 4, cudaMemcpyHostToDevice,
                        st) != cudaSuccess)
        return MOE_ERR_CUDA;
    if (cudaEventRecord(ctx->stage_done[s], st) != cudaSuccess) return MOE_ERR_CUDA;
    ctx->stage_used[s] = true;
    ctx->stage_next++;
    return enqueue_derive(ctx, st);
}

bool stream_is_capturing(cudaStream_t st)
{
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cs) != cudaSuccess) { cudaGetLastError(); return false; }
    return cs != cudaStreamCaptureStatusNone;
}

// (Re)allocate the per-tile count rows for the context's current tile size.
bool alloc_scan_scratch(moe_ctx *ctx, cudaStream_t st)
{
    const Derived &d = ctx->d;
    const size_t tiles = ((size_t)ctx->cfg.max_tokens + d.tokens_per_block - 1) / d.tokens_per_block;
    const size_t row = (size_t)(d.p_pad / 4) * sizeof(ulonglong2);
    if (tiles > ctx->scan_tiles) {
        cudaFree(ctx->d_tile_counts);
        ctx->d_tile_counts = nullptr; ctx->scan_tiles = 0;
        if (cudaMalloc(&ctx->d_tile_counts, tiles * row) != cudaSuccess) return false;
        ctx->scan_tiles = tiles;
    }
    // tag 0 never equals an epoch (epochs start at 1 and skip 0)
    return cudaMemsetAsync(ctx->d_tile_counts, 0, ctx->scan_tiles * row, st) == cudaSuccess;
}

// The kernels with rings in dynamic shared memory may use all of it.  The attribute belongs to
// the function, not to a context, so it is set once per process to the largest size any
// context can ask for.
bool set_kernel_attributes_once()
{
    static std::once_flag once;
    static bool ok = false;
    std::call_once(once, [] {
        const cudaFuncAttribute at = cudaFuncAttributeMaxDynamicSharedMemorySize;
        const int sm = (int)(kMaxSmem - 1024);
        ok = cudaFuncSetAttribute(k_scatter_bulk, at, sm) == cudaSuccess
          && cudaFuncSetAttribute(k_combine_bulk<1, 8>, at, sm) == cudaSuccess
          && cudaFuncSetAttribute(k_combine_bulk<2, 8>, at, sm) == cudaSuccess
          && cudaFuncSetAttribute(k_combine_bulk<4, 8>, at, sm) == cudaSuccess
          && cudaFuncSetAttribute(k_combine_bulk<1, 2>, at, sm) == cudaSuccess
          && cudaFuncSetAttribute(k_combine_bulk<2, 2>, at, sm) == cudaSuccess
          && cudaFuncSetAttribute(k_combine_bulk<4, 2>, at, sm) == cudaSuccess
          && cudaFuncSetAttribute(k_combine_bulk<1, 0>, at, sm) == cudaSuccess
          && cudaFuncSetAttribute(k_combine_bulk<2, 0>, at, sm) == cudaSuccess
          && cudaFuncSetAttribute(k_combine_bulk<4, 0>, at, sm) == cudaSuccess;
    });
    return ok;
}

int tuned(const moe_ctx *ctx, int option, int dflt)
{
    return ctx->tune[option] >= 0 ? ctx->tune[option] : dflt;
}

// Launch shapes of the three kernels from the context's shape and its tuning overrides.
void configure_launch(moe_ctx *ctx)
{
    const Derived &d = ctx->d;
    ctx->route_smem = route_smem_bytes(d.E, d.max_rep, d.tokens_per_block, d.k, d.P, d.epl, d.alias_wcount);
    ctx->spin_limit = (unsigned)tuned(ctx, MOE_TUNE_SPIN_LIMIT, (int)kDefaultSpinLimit);
    ctx->pdl = tuned(ctx, MOE_TUNE_PDL, 1) != 0;
    ctx->scatter_impl = tuned(ctx, MOE_TUNE_SCATTER_IMPL, 0);
    ctx->bulk_stages = std::min(8, std::max(1, tuned(ctx, MOE_TUNE_SCATTER_BULK_STAGES, 4)));
    const size_t stage_bytes = ((size_t)d.H * 2 + 127) & ~(size_t)127;
    while (ctx->bulk_stages > 1 && ctx->bulk_stages * stage_bytes > kMaxSmem - 2048) --ctx->bulk_stages;
    if (ctx->bulk_stages * stage_bytes > kMaxSmem - 2048) ctx->scatter_impl = 0;   // row too wide to stage
    const size_t ring = ctx->bulk_stages * stage_bytes;
    const int fit = std::max(1, (int)((kMaxSmem - 1024) / (ring + 1024)));
    ctx->bulk_ctas_per_sm = std::min(fit, std::min(32, std::max(1, tuned(ctx, MOE_TUNE_SCATTER_BULK_CTAS_PER_SM, fit))));
    ctx->scatter_blocks_per_sm = std::max(1, tuned(ctx, MOE_TUNE_SCATTER_BLOCKS_PER_SM, 8));
    // one warp moves a whole row when it fits (long contiguous HBM bursts per destination
    // row measured 6.3 TB/s against 5.65 TB/s with 2 KB pieces): 16-byte units per lane
    {
        static const int kUnroll[] = {4, 8, 16, 28, 32};
        const int need = (d.H / 8 + 31) / 32;
        int un = 32;
        for (int u : kUnroll) if (u >= need) { un = u; break; }
        // ... unless the whole scatter is short (under 256 MB moved, a few tens of microseconds):
        // then the start-up of each warp's single long copy is not amortised and 2 KB pieces,
        // four times as many warps' worth of work, win (33.4 against 35.0 us per step at 4096
        // tokens of 8 KB; at 8192 tokens of 14 KB whole rows are 3 % of a step faster)
        if ((long long)ctx->cfg.max_tokens * d.H * 2 * (1 + d.k) < (256ll << 20)) un = 4;
        const int forced = tuned(ctx, MOE_TUNE_SCATTER_UNROLL, 0);
        for (int u : kUnroll) if (u == forced) un = forced;
        ctx->scatter_unroll = un;
    }
    // Row stores normally skip L1 and leave L2 early (the rows are read again only after ~1 GB of
    // other rows has passed).  A send buffer small enough to stay in the 126 MB L2 until the
    // combine reads it is written with plain stores instead: 31.8 against 33.7 us per step at 4096
    // tokens of 8 KB, k = 2 (67 MB); at 940 MB plain stores cost 4 us.
    const bool fits_l2 = (long long)ctx->cfg.max_tokens * d.k * d.H * 2 <= (80ll << 20);
    ctx->scatter_store_policy = std::min(3, tuned(ctx, MOE_TUNE_SCATTER_STORE_POLICY, fits_l2 ? 1 : 0));
    if (ctx->scatter_unroll != 28 && ctx->scatter_unroll != 16 && ctx->scatter_unroll != 4) ctx->scatter_store_policy = 0;
    ctx->route_prefetch = tuned(ctx, MOE_TUNE_ROUTE_PREFETCH, 3) & 3;
    ctx->combine_blocks_per_sm = 8;
    ctx->combine_impl = tuned(ctx, MOE_TUNE_COMBINE_IMPL, 1);
    // a ring stage holds one column chunk of all k rows: widen the chunk for small k so that a
    // stage stays near 4 KB and the ring keeps as many bytes in flight as with k = 8
    int u_auto = d.k <= 2 ? 4 : (d.k <= 4 ? 2 : 1);
    while (u_auto > 1 && 32 * u_auto > d.H / 8) u_auto /= 2;        // never wider than a row
    ctx->combine_u = tuned(ctx, MOE_TUNE_COMBINE_CHUNK, u_auto);
    if (ctx->combine_u != 1 && ctx->combine_u != 2 && ctx->combine_u != 4) ctx->combine_u = 2;
    // ring shape: with many rows per token (k >= 6) four warps per CTA with five stages each
    // (two CTAs per SM: 8 warps, ~160 KB of rings) measured 4-7 % faster than eight warps with
    // three stages; with few rows per token the wider, shallower shape is the faster one
    const bool deep = d.k >= 6;
    ctx->combine_warps = std::min(kCombineBulkMaxWarps, std::max(1, tuned(ctx, MOE_TUNE_COMBINE_WARPS, deep ? 4 : 8)));
    ctx->combine_stages = std::min(8, std::max(2, tuned(ctx, MOE_TUNE_COMBINE_STAGES, deep ? 5 : 3)));
    while (ctx->combine_stages > 2 &&
           combine_bulk_smem(ctx->combine_stages, d.k, ctx->combine_u, ctx->combine_warps) > kMaxSmem - 1024)
        --ctx->combine_stages;
    ctx->combine_smem = combine_bulk_smem(ctx->combine_stages, d.k, ctx->combine_u, ctx->combine_warps);
    if (ctx->combine_smem > kMaxSmem - 1024) ctx->combine_impl = 0;
    const int fit_c = std::max(1, (int)((kMaxSmem - 1024) / (ctx->combine_smem + 1024)));
    ctx->combine_ctas_per_sm = std::max(1, std::min(fit_c, tuned(ctx, MOE_TUNE_COMBINE_CTAS_PER_SM, fit_c)));
}

void free_ctx(moe_ctx *ctx)
{
    if (!ctx) return;
    cudaFree(ctx->d_state); cudaFree(ctx->d_live); cudaFree(ctx->d_bias); cudaFree(ctx->d_slot_scale);
    cudaFree(ctx->d_tile_counts); cudaFree(ctx->d_ctl); cudaFree(ctx->d_pos);
    cudaFree(ctx->d_zero_row);
    cudaFree(ctx->d_peer_bufs); cudaFree(ctx->d_src_base);
    for (int s = 0; s < kStagingSlots; ++s) {
        if (ctx->h_stage[s]) cudaFreeHost(ctx->h_stage[s]);
        if (ctx->stage_done[s]) cudaEventDestroy(ctx->stage_done[s]);
    }
    delete ctx;
}

}  // namespace

extern "C" {

const char *moe_status_string(moe_status s)
{
    switch (s) {
        case MOE_OK: return "MOE_OK";
        case MOE_ERR_INVALID_ARG: return "MOE_ERR_INVALID_ARG";
        case MOE_ERR_CUDA: return "MOE_ERR_CUDA";
        case MOE_ERR_INSUFFICIENT_EXPERTS: return "MOE_ERR_INSUFFICIENT_EXPERTS";
        case MOE_ERR_CAPACITY: return "MOE_ERR_CAPACITY";
        case MOE_ERR_DEVICE_TIMEOUT: return "MOE_ERR_DEVICE_TIMEOUT";
    }
    return "MOE_ERR_UNKNOWN";
}

size_t moe_workspace_bytes(const moe_config *cfg)
{
    Derived d;
    if (!derive(cfg, &d)) return 0;
    return device_bytes_for(d, cfg->max_tokens);
}

moe_status moe_plan_routing_state(const moe_config *cfg, const int32_t *slot_to_expert,
                                  const int32_t *failed_ranks, int32_t n_failed,
                                  uint32_t *rank_alive, int32_t *replica_table,
                                  int32_t *n_available)
{
    Derived d;
    if (!derive(cfg, &d) || !slot_to_expert || n_failed < 0 || (n_failed > 0 && !failed_ranks))
        return MOE_ERR_INVALID_ARG;
    std::vector<uint8_t> failed((size_t)d.R, 0);
    for (int i = 0; i < n_failed; ++i) {
        if (failed_ranks[i] < 0 || failed_ranks[i] >= d.R) return MOE_ERR_INVALID_ARG;
        failed[failed_ranks[i]] = 1;
    }
    std::vector<int32_t> blob;
    int avail = 0;
    const std::vector<uint8_t> none((size_t)d.E, 0);
    std::vector<int32_t> ident((size_t)d.R);
    for (int r = 0; r < d.R; ++r) ident[r] = r;
    const moe_status st = plan_state(cfg, d, slot_to_expert, failed, none, ident, d.R, &blob, &avail);
    if (st != MOE_OK) return st;
    if (rank_alive) std::memcpy(rank_alive, blob.data() + kStateHeaderWords, (size_t)d.rank_words * 4);
    if (replica_table)
        std::memcpy(replica_table, blob.data() + kStateHeaderWords + d.rank_words + d.expert_words,
                    (size_t)d.E * d.max_rep * 4);
    if (n_available) *n_available = avail;
    return MOE_OK;
}

moe_status moe_route_init(const moe_config *cfg, const int32_t *slot_to_expert, const float *bias,
                          const float *slot_scale, void *cuda_stream, moe_ctx **out)
{
    Derived d;
    if (!out || !slot_to_expert || !slot_scale || !derive(cfg, &d)) return MOE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    std::vector<uint8_t> failed((size_t)d.R, 0);
    std::vector<int32_t> blob;
    const std::vector<uint8_t> no_lost((size_t)d.E, 0);
    std::vector<int32_t> ident((size_t)d.R);
    for (int r = 0; r < d.R; ++r) ident[r] = r;
    moe_status ms = plan_state(cfg, d, slot_to_expert, failed, no_lost, ident, d.R, &blob, nullptr);
    if (ms != MOE_OK) return ms;

    moe_ctx *ctx = new (std::nothrow) moe_ctx();
    if (!ctx) return MOE_ERR_CUDA;
    ctx->cfg = *cfg; ctx->d = d;
    ctx->slot_to_expert.assign(slot_to_expert, slot_to_expert + d.P);
    ctx->failed = failed;
    ctx->expert_failed = no_lost;
    ctx->rank_order = ident;
    ctx->n_listed = d.R;
    ctx->last_weights = nullptr; ctx->last_slot = nullptr; ctx->last_dst_row = nullptr;
    ctx->last_T = -1;
    ctx->timing_event = nullptr;
    ctx->ep_world = 0; ctx->ep_rank = 0; ctx->ep_spg = 0; ctx->ep_recv_rows = 0;
    ctx->d_peer_bufs = nullptr; ctx->d_src_base = nullptr; ctx->ep_routed = false;
    ctx->stage_next = 0;
    for (int s = 0; s < kStagingSlots; ++s) {
        ctx->h_stage[s] = nullptr; ctx->stage_done[s] = nullptr; ctx->stage_used[s] = false;
    }
    ctx->d_state = nullptr; ctx->d_live = nullptr; ctx->d_bias = nullptr; ctx->d_slot_scale = nullptr;
    ctx->d_tile_counts = nullptr; ctx->scan_tiles = 0;
    ctx->d_ctl = nullptr; ctx->d_pos = nullptr; ctx->d_zero_row = nullptr;
    for (int i = 0; i < kNumTuning; ++i) ctx->tune[i] = -1;

    bool ok = cudaGetDevice(&ctx->device) == cudaSuccess &&
              cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, ctx->device) ==
                  cudaSuccess;
    ok = ok && cudaMalloc(&ctx->d_state, (size_t)d.state_words * 4) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->d_live, (size_t)d.E * (1 + d.max_rep) * 4) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->d_bias, (size_t)d.E * 4) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->d_slot_scale, (size_t)d.P * 4) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->d_ctl, sizeof(moe::Control)) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->d_pos, (size_t)cfg->max_tokens * d.k * 4) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->d_zero_row, (size_t)d.H * 2) == cudaSuccess;
    ok = ok && alloc_scan_scratch(ctx, st);
    for (int s = 0; s < kStagingSlots && ok; ++s) {
        ok = cudaMallocHost(&ctx->h_stage[s], (size_t)d.state_words * 4) == cudaSuccess &&
             cudaEventCreateWithFlags(&ctx->stage_done[s], cudaEventDisableTiming) == cudaSuccess;
    }
    ctx->device_bytes = device_bytes_for(d, cfg->max_tokens);
    if (ok) {
        std::vector<float> b((size_t)d.E, 0.0f);
        if (bias) std::copy(bias, bias + d.E, b.begin());
        const moe::Control c0 = {0u, 1u, kDevOk, 0};
        // synchronous pageable copies: the host arrays may be freed on return
        ok = cudaMemsetAsync(ctx->d_zero_row, 0, (size_t)d.H * 2, st) == cudaSuccess &&
             cudaMemcpyAsync(ctx->d_ctl, &c0, sizeof(c0), cudaMemcpyHostToDevice, st) == cudaSuccess &&
             cudaMemcpyAsync(ctx->d_bias, b.data(), (size_t)d.E * 4, cudaMemcpyHostToDevice, st) == cudaSuccess &&
             cudaMemcpyAsync(ctx->d_slot_scale, slot_scale, (size_t)d.P * 4, cudaMemcpyHostToDevice, st) == cudaSuccess &&
             cudaMemcpyAsync(ctx->d_state, blob.data(), (size_t)d.state_words * 4, cudaMemcpyHostToDevice, st) == cudaSuccess &&
             enqueue_derive(ctx, st) == MOE_OK &&
             cudaStreamSynchronize(st) == cudaSuccess;
    }
    ok = ok && set_kernel_attributes_once();
    if (ok) configure_launch(ctx);
    if (!ok) {
        cudaGetLastError();
        free_ctx(ctx);
        return MOE_ERR_CUDA;
    }
    *out = ctx;
    return MOE_OK;
}

moe_status moe_set_failed_ranks(moe_ctx *ctx, const int32_t *ranks, int32_t n, void *cuda_stream)
{
    if (!ctx || n < 0 || (n > 0 && !ranks)) return MOE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const Derived &d = ctx->d;
    std::vector<uint8_t> failed((size_t)d.R, 0);
    for (int i = 0; i < n; ++i) {
        if (ranks[i] < 0 || ranks[i] >= d.R) return MOE_ERR_INVALID_ARG;
        failed[ranks[i]] = 1;
    }
    std::vector<int32_t> blob;
    const moe_status ms = plan_state(&ctx->cfg, d, ctx->slot_to_expert.data(), failed, ctx->expert_failed, ctx->rank_order,
                                     ctx->n_listed, &blob, nullptr);
    if (ms != MOE_OK) return ms;
    if (stream_is_capturing(st)) return MOE_ERR_INVALID_ARG;
    // only the header and the rank bitmap change
    const moe_status ps = push_state(ctx, blob, kStateHeaderWords + d.rank_words + d.expert_words, st);
    if (ps == MOE_OK) ctx->failed.swap(failed);
    return ps;
}

moe_status moe_update_replica_map(moe_ctx *ctx, const int32_t *slot_to_expert, void *cuda_stream)
{
    if (!ctx || !slot_to_expert) return MOE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const Derived &d = ctx->d;
    std::vector<int32_t> blob;
    const moe_status ms = plan_state(&ctx->cfg, d, slot_to_expert, ctx->failed, ctx->expert_failed, ctx->rank_order,
                                     ctx->n_listed, &blob, nullptr);
    if (ms != MOE_OK) return ms;
    if (stream_is_capturing(st)) return MOE_ERR_INVALID_ARG;
    const moe_status ps = push_state(ctx, blob, d.state_words, st);
    if (ps == MOE_OK) ctx->slot_to_expert.assign(slot_to_expert, slot_to_expert + d.P);
    return ps;
}

moe_status moe_set_failed_experts(moe_ctx *ctx, const uint8_t *mask, int32_t n, void *cuda_stream)
{
    if (!ctx || (n != 0 && n != ctx->d.E) || (n > 0 && !mask)) return MOE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const Derived &d = ctx->d;
    std::vector<uint8_t> lost((size_t)d.E, 0);
    for (int e = 0; e < n; ++e) lost[e] = mask[e] ? 1 : 0;
    std::vector<int32_t> blob;
    const moe_status ms = plan_state(&ctx->cfg, d, ctx->slot_to_expert.data(), ctx->failed, lost, ctx->rank_order,
                                     ctx->n_listed, &blob, nullptr);
    if (ms != MOE_OK) return ms;
    if (stream_is_capturing(st)) return MOE_ERR_INVALID_ARG;
    const moe_status ps = push_state(ctx, blob, kStateHeaderWords + d.rank_words + d.expert_words, st);
    if (ps == MOE_OK) ctx->expert_failed.swap(lost);
    return ps;
}

moe_status moe_compact_ranks(int32_t num_ranks, const int32_t *failed_ranks, int32_t n_failed,
                             int32_t switched_rank, int32_t replaced_rank,
                             int32_t *logical_to_physical, int32_t *n_logical)
{
    if (num_ranks < 1 || n_failed < 0 || (n_failed > 0 && !failed_ranks) || !logical_to_physical || !n_logical)
        return MOE_ERR_INVALID_ARG;
    std::vector<uint8_t> failed((size_t)num_ranks, 0);
    for (int i = 0; i < n_failed; ++i) {
        if (failed_ranks[i] < 0 || failed_ranks[i] >= num_ranks) return MOE_ERR_INVALID_ARG;
        failed[failed_ranks[i]] = 1;
    }
    const bool role_switch = switched_rank >= 0 || replaced_rank >= 0;
    if (role_switch) {
        if (switched_rank < 0 || switched_rank >= num_ranks || replaced_rank < 0 || replaced_rank >= num_ranks)
            return MOE_ERR_INVALID_ARG;
        if (failed[switched_rank] || !failed[replaced_rank]) return MOE_ERR_INVALID_ARG;
    }
    // walk the old logical order: the switched rank takes the failed rank's position, other
    // failed ranks leave a gap that the following ranks close by moving down one
    int n = 0;
    for (int r = 0; r < num_ranks; ++r) {
        if (role_switch && r == replaced_rank) { logical_to_physical[n++] = switched_rank; continue; }
        if (role_switch && r == switched_rank) continue;
        if (failed[r]) continue;
        logical_to_physical[n++] = r;
    }
    *n_logical = n;
    return MOE_OK;
}

moe_status moe_set_rank_order(moe_ctx *ctx, const int32_t *logical_to_physical, int32_t n, void *cuda_stream)
{
    if (!ctx || n < 0 || n > ctx->d.R || (n > 0 && !logical_to_physical)) return MOE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const Derived &d = ctx->d;
    std::vector<int32_t> order;
    std::vector<uint8_t> seen((size_t)d.R, 0);
    if (n == 0) {                                        // back to the physical numbering
        for (int r = 0; r < d.R; ++r) order.push_back(r);
        n = d.R;
    } else {
        for (int i = 0; i < n; ++i) {
            const int r = logical_to_physical[i];
            if (r < 0 || r >= d.R || seen[r]) return MOE_ERR_INVALID_ARG;
            seen[r] = 1;
            order.push_back(r);
        }
        for (int r = 0; r < d.R; ++r)                    // unlisted ranks own no rows; keep a full permutation
            if (!seen[r]) order.push_back(r);
    }
    std::vector<int32_t> blob;
    const moe_status ms = plan_state(&ctx->cfg, d, ctx->slot_to_expert.data(), ctx->failed, ctx->expert_failed,
                                     order, n, &blob, nullptr);
    if (ms != MOE_OK) return ms;
    if (stream_is_capturing(st)) return MOE_ERR_INVALID_ARG;
    const moe_status ps = push_state(ctx, blob, d.state_words, st);
    if (ps == MOE_OK) { ctx->rank_order.swap(order); ctx->n_listed = n; }
    return ps;
}

moe_status moe_dispatch(moe_ctx *ctx, const float *logits, const void *x, int32_t T,
                        const moe_dispatch_out *out, void *cuda_stream)
{
    if (!ctx || !out || T < 0) return MOE_ERR_INVALID_ARG;
    if (T > ctx->cfg.max_tokens) return MOE_ERR_CAPACITY;
    if (T == 0) {                     // nothing to route: no launch, pointers not inspected
        ctx->last_weights = out->topk_weights; ctx->last_slot = out->topk_slot;
        ctx->last_dst_row = out->dst_row; ctx->last_T = 0;
        return MOE_OK;
    }
    if (!out->topk_ids || !out->topk_weights || !out->topk_slot || !out->slot_counts ||
        !out->slot_offsets || !out->rank_counts || !out->rank_offsets || !out->dst_row ||
        !out->src_index || !out->send_buf)
        return MOE_ERR_INVALID_ARG;
    if (!x || (!logits && ctx->cfg.score_func != MOE_ROUTE_DENSE_TP)) return MOE_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(out->send_buf) || !aligned16(logits)) return MOE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const Derived &d = ctx->d;
    ctx->last_weights = out->topk_weights; ctx->last_slot = out->topk_slot;
    ctx->last_dst_row = out->dst_row; ctx->last_T = T;

    if (enqueue_route(ctx, logits, T, out, st) != cudaSuccess) return MOE_ERR_CUDA;
    ctx->ep_routed = false;
    if (ctx->timing_event && cudaEventRecord(ctx->timing_event, st) != cudaSuccess) return MOE_ERR_CUDA;

    ScatterParams sp;
    sp.x = static_cast<const uint4 *>(x); sp.send = static_cast<uint4 *>(out->send_buf);
    sp.T = T; sp.k = d.k; sp.hv = d.H / 8; sp.P = d.P; sp.spin_limit = ctx->spin_limit;
    sp.topk_slot = out->topk_slot; sp.slot_offsets = out->slot_offsets; sp.pos_in_slot = ctx->d_pos;
    sp.dst_row = out->dst_row; sp.src_index = out->src_index; sp.ctl = ctx->d_ctl;
    if (ctx->scatter_impl == 1) {
        const unsigned stage_bytes = ((unsigned)d.H * 2u + 127u) & ~127u;
        const int grid = std::min(T, ctx->sm_count * ctx->bulk_ctas_per_sm);
        k_scatter_bulk<<<grid, kBulkThreads, (size_t)ctx->bulk_stages * stage_bytes, st>>>(sp, ctx->bulk_stages);
    } else {
        const int un = ctx->scatter_unroll;
        const int chunk = 32 * un;
        const int chunks = (sp.hv + chunk - 1) / chunk;
        const long long items = (long long)T * chunks;
        const long long want = (items + kScatterThreads / 32 - 1) / (kScatterThreads / 32);
        const int grid = (int)std::min<long long>(want, (long long)ctx->sm_count * ctx->scatter_blocks_per_sm);
        const dim3 g(grid), b(kScatterThreads);
        const bool pdl = ctx->pdl;
        switch (un * 10 + ctx->scatter_store_policy) {
            case 80: launch_kernel(k_scatter_vec<8, 0>, g, b, 0, st, pdl, sp); break;
            case 160: launch_kernel(k_scatter_vec<16, 0>, g, b, 0, st, pdl, sp); break;
            case 280: launch_kernel(k_scatter_vec<28, 0>, g, b, 0, st, pdl, sp); break;
            case 320: launch_kernel(k_scatter_vec<32, 0>, g, b, 0, st, pdl, sp); break;
            case 40: launch_kernel(k_scatter_vec<4, 0>, g, b, 0, st, pdl, sp); break;
            // the other store policies: measurement variants of the two most used shapes
            case 281: launch_kernel(k_scatter_vec<28, 1>, g, b, 0, st, pdl, sp); break;
            case 282: launch_kernel(k_scatter_vec<28, 2>, g, b, 0, st, pdl, sp); break;
            case 283: launch_kernel(k_scatter_vec<28, 3>, g, b, 0, st, pdl, sp); break;
            case 161: launch_kernel(k_scatter_vec<16, 1>, g, b, 0, st, pdl, sp); break;
            case 162: launch_kernel(k_scatter_vec<16, 2>, g, b, 0, st, pdl, sp); break;
            case 163: launch_kernel(k_scatter_vec<16, 3>, g, b, 0, st, pdl, sp); break;
            case 41: launch_kernel(k_scatter_vec<4, 1>, g, b, 0, st, pdl, sp); break;
            case 42: launch_kernel(k_scatter_vec<4, 2>, g, b, 0, st, pdl, sp); break;
            case 43: launch_kernel(k_scatter_vec<4, 3>, g, b, 0, st, pdl, sp); break;
            default: return MOE_ERR_INVALID_ARG;          // policy not built for this piece size
        }
    }
    if (cudaGetLastError() != cudaSuccess) return MOE_ERR_CUDA;
    return MOE_OK;
}

moe_status moe_combine(moe_ctx *ctx, const void *expert_buf, int32_t T, void *y, void *cuda_stream)
{
    if (!ctx || T < 0) return MOE_ERR_INVALID_ARG;
    if (ctx->last_T < 0 || T != ctx->last_T || ctx->ep_routed) return MOE_ERR_INVALID_ARG;
    if (T == 0) return MOE_OK;
    if (!expert_buf || !y || !aligned16(expert_buf) || !aligned16(y)) return MOE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const Derived &d = ctx->d;
    CombineParams cp;
    cp.buf = static_cast<const uint4 *>(expert_buf); cp.y = static_cast<uint4 *>(y);
    cp.T = T; cp.k = d.k; cp.hv = d.H / 8;
    cp.dst_row = ctx->last_dst_row; cp.topk_weights = ctx->last_weights; cp.topk_slot = ctx->last_slot;
    cp.slot_scale = ctx->d_slot_scale;
    cp.peer_bufs = nullptr; cp.slots_per_gpu = 0;
    cp.P = d.P; cp.row_limit = (long long)T * d.k; cp.zero_row = ctx->d_zero_row; cp.spin_limit = ctx->spin_limit;
    if (ctx->combine_impl == 1) return enqueue_combine_bulk(ctx, cp, st);
    const int chunks = (cp.hv + kCombineChunk - 1) / kCombineChunk;
    const long long items = (long long)T * chunks;
    const long long want = (items + kCombineThreads / 32 - 1) / (kCombineThreads / 32);
    const int grid = (int)std::min<long long>(want, (long long)ctx->sm_count * ctx->combine_blocks_per_sm);
    if (launch_combine(cp, grid, st) != cudaSuccess) return MOE_ERR_CUDA;
    return MOE_OK;
}

// ---------------------------------------------------------------------------
// Expert parallelism over several GPUs
// ---------------------------------------------------------------------------

moe_status moe_ep_plan_host(const int32_t *counts_all, int32_t world, int32_t rank, int32_t num_slots,
                            int32_t *src_base, int32_t *recv_slot_offsets)
{
    if (!counts_all || world < 1 || rank < 0 || rank >= world || num_slots < 1 || num_slots % world != 0)
        return MOE_ERR_INVALID_ARG;
    const int spg = num_slots / world;
    for (int s = 0; s < num_slots && src_base; ++s) {
        const int first = (s / spg) * spg;
        long long base = 0;
        for (int q = first; q < s; ++q)
            for (int g = 0; g < world; ++g) base += counts_all[(size_t)g * num_slots + q];
        for (int g = 0; g < rank; ++g) base += counts_all[(size_t)g * num_slots + s];
        if (base > 0x7fffffffll) return MOE_ERR_CAPACITY;
        src_base[s] = (int32_t)base;
    }
    long long off = 0;
    for (int q = 0; q <= spg && recv_slot_offsets; ++q) {
        if (off > 0x7fffffffll) return MOE_ERR_CAPACITY;
        recv_slot_offsets[q] = (int32_t)off;
        if (q < spg)
            for (int g = 0; g < world; ++g) off += counts_all[(size_t)g * num_slots + (size_t)rank * spg + q];
    }
    return MOE_OK;
}

moe_status moe_ep_attach(moe_ctx *ctx, const moe_ep_group *group, void *cuda_stream)
{
    if (!ctx || !group || !group->recv_bufs) return MOE_ERR_INVALID_ARG;
    const Derived &d = ctx->d;
    if (group->world < 1 || group->world > 1024 || group->rank < 0 || group->rank >= group->world)
        return MOE_ERR_INVALID_ARG;
    if (d.R % group->world != 0) return MOE_ERR_INVALID_ARG;          // whole simulated ranks per GPU
    if (group->recv_rows < 1 || group->recv_rows > 0x7fffffffll) return MOE_ERR_INVALID_ARG;
    if (ctx->combine_impl != 1) return MOE_ERR_INVALID_ARG;           // the ring combine is the peer-aware one
    for (int r = 0; r < d.R; ++r)                                     // physical rank numbering only
        if (ctx->n_listed != d.R || ctx->rank_order[r] != r) return MOE_ERR_INVALID_ARG;
    for (int g = 0; g < group->world; ++g)
        if (!group->recv_bufs[g] || !aligned16(group->recv_bufs[g])) return MOE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (stream_is_capturing(st)) return MOE_ERR_INVALID_ARG;
    if (ctx->ep_world != group->world) {
        cudaFree(ctx->d_peer_bufs); ctx->d_peer_bufs = nullptr; ctx->ep_world = 0;
        if (cudaMalloc(&ctx->d_peer_bufs, (size_t)group->world * sizeof(uint4 *)) != cudaSuccess) {
            cudaGetLastError();
            return MOE_ERR_CUDA;
        }
    }
    if (!ctx->d_src_base && cudaMalloc(&ctx->d_src_base, (size_t)d.P * 4) != cudaSuccess) {
        cudaGetLastError();
        return MOE_ERR_CUDA;
    }
    // synchronous copy: the host array may be freed on return
    if (cudaMemcpyAsync(ctx->d_peer_bufs, group->recv_bufs, (size_t)group->world * sizeof(void *),
                        cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return MOE_ERR_CUDA;
    ctx->ep_world = group->world; ctx->ep_rank = group->rank; ctx->ep_spg = d.P / group->world;
    ctx->ep_recv_rows = group->recv_rows;
    return MOE_OK;
}

moe_status moe_ep_route(moe_ctx *ctx, const float *logits, int32_t T, const moe_dispatch_out *out,
                        void *cuda_stream)
{
    if (!ctx || !out || T < 0) return MOE_ERR_INVALID_ARG;
    if (ctx->ep_world < 1) return MOE_ERR_INVALID_ARG;
    if (T > ctx->cfg.max_tokens) return MOE_ERR_CAPACITY;
    if (!out->slot_counts) return MOE_ERR_INVALID_ARG;
    if (T > 0 && (!out->topk_ids || !out->topk_weights || !out->topk_slot || !out->slot_offsets ||
                  !out->rank_counts || !out->rank_offsets || !out->dst_row))
        return MOE_ERR_INVALID_ARG;
    if (T > 0 && ((!logits && ctx->cfg.score_func != MOE_ROUTE_DENSE_TP) || !aligned16(logits)))
        return MOE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    ctx->last_weights = out->topk_weights; ctx->last_slot = out->topk_slot;
    ctx->last_dst_row = out->dst_row; ctx->last_T = T; ctx->ep_routed = true;
    if (T == 0) {                      // this GPU sends nothing, but its counts still take part in the exchange
        if (cudaMemsetAsync(out->slot_counts, 0, (size_t)ctx->d.P * 4, st) != cudaSuccess) return MOE_ERR_CUDA;
        return MOE_OK;
    }
    return enqueue_route(ctx, logits, T, out, st) == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

moe_status moe_ep_scatter(moe_ctx *ctx, const void *x, int32_t T, const int32_t *counts_all,
                          int32_t *recv_slot_offsets, void *cuda_stream)
{
    if (!ctx || T < 0 || !counts_all || !recv_slot_offsets) return MOE_ERR_INVALID_ARG;
    if (ctx->ep_world < 1 || !ctx->ep_routed || T != ctx->last_T) return MOE_ERR_INVALID_ARG;
    if (T > 0 && (!x || !aligned16(x))) return MOE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const Derived &d = ctx->d;
    EpPlanParams pp;
    pp.counts = counts_all; pp.G = ctx->ep_world; pp.g = ctx->ep_rank; pp.P = d.P; pp.spg = ctx->ep_spg;
    pp.recv_rows = ctx->ep_recv_rows; pp.src_base = ctx->d_src_base;
    pp.recv_slot_offsets = recv_slot_offsets; pp.ctl = ctx->d_ctl;
    if (launch_kernel(k_ep_plan, dim3(1), dim3(kEpPlanThreads), 0, st, false, pp) != cudaSuccess)
        return MOE_ERR_CUDA;
    if (T == 0) return MOE_OK;
    EpScatterParams sp;
    sp.x = static_cast<const uint4 *>(x); sp.peer_bufs = ctx->d_peer_bufs;
    sp.T = T; sp.k = d.k; sp.hv = d.H / 8; sp.spg = ctx->ep_spg; sp.P = d.P; sp.recv_rows = ctx->ep_recv_rows;
    sp.topk_slot = ctx->last_slot; sp.src_base = ctx->d_src_base; sp.pos_in_slot = ctx->d_pos;
    sp.dst_row = const_cast<int32_t *>(ctx->last_dst_row);
    const int un = ctx->scatter_unroll;
    const int chunks = (sp.hv + 32 * un - 1) / (32 * un);
    const long long items = (long long)T * chunks;
    const long long want = (items + kEpScatterThreads / 32 - 1) / (kEpScatterThreads / 32);
    const int grid = (int)std::min<long long>(want, (long long)ctx->sm_count * ctx->scatter_blocks_per_sm);
    switch (un) {
        case 8: launch_kernel(k_ep_scatter<8>, dim3(grid), dim3(kEpScatterThreads), 0, st, ctx->pdl, sp); break;
        case 16: launch_kernel(k_ep_scatter<16>, dim3(grid), dim3(kEpScatterThreads), 0, st, ctx->pdl, sp); break;
        case 28: launch_kernel(k_ep_scatter<28>, dim3(grid), dim3(kEpScatterThreads), 0, st, ctx->pdl, sp); break;
        case 32: launch_kernel(k_ep_scatter<32>, dim3(grid), dim3(kEpScatterThreads), 0, st, ctx->pdl, sp); break;
        default: launch_kernel(k_ep_scatter<4>, dim3(grid), dim3(kEpScatterThreads), 0, st, ctx->pdl, sp); break;
    }
    return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

moe_status moe_ep_combine(moe_ctx *ctx, int32_t T, void *y, void *cuda_stream)
{
    if (!ctx || T < 0) return MOE_ERR_INVALID_ARG;
    if (ctx->ep_world < 1 || !ctx->ep_routed || T != ctx->last_T) return MOE_ERR_INVALID_ARG;
    if (T == 0) return MOE_OK;
    if (!y || !aligned16(y)) return MOE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const Derived &d = ctx->d;
    CombineParams cp;
    cp.buf = nullptr; cp.y = static_cast<uint4 *>(y);
    cp.T = T; cp.k = d.k; cp.hv = d.H / 8;
    cp.dst_row = ctx->last_dst_row; cp.topk_weights = ctx->last_weights; cp.topk_slot = ctx->last_slot;
    cp.slot_scale = ctx->d_slot_scale;
    cp.peer_bufs = const_cast<const uint4 *const *>(ctx->d_peer_bufs); cp.slots_per_gpu = ctx->ep_spg;
    cp.P = d.P; cp.row_limit = ctx->ep_recv_rows; cp.zero_row = ctx->d_zero_row; cp.spin_limit = ctx->spin_limit;
    return enqueue_combine_bulk(ctx, cp, st);
}

moe_status moe_step_host_async(moe_ctx *ctx, const float *logits_host, const void *x_host, int32_t T,
                               const moe_dispatch_out *out, float *logits_dev, void *x_dev, void *y_dev,
                               void *y_host, void *cuda_stream)
{
    if (!ctx || !out || T < 0) return MOE_ERR_INVALID_ARG;
    if (T > ctx->cfg.max_tokens) return MOE_ERR_CAPACITY;
    if (T > 0 && (!logits_host || !x_host || !logits_dev || !x_dev || !y_dev || !y_host))
        return MOE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const Derived &d = ctx->d;
    if (T > 0) {
        if (cudaMemcpyAsync(logits_dev, logits_host, (size_t)T * d.E * 4, cudaMemcpyHostToDevice, st) != cudaSuccess ||
            cudaMemcpyAsync(x_dev, x_host, (size_t)T * d.H * 2, cudaMemcpyHostToDevice, st) != cudaSuccess)
            return MOE_ERR_CUDA;
    }
    moe_status ms = moe_dispatch(ctx, logits_dev, x_dev, T, out, cuda_stream);
    if (ms != MOE_OK) return ms;
    ms = moe_combine(ctx, out->send_buf, T, y_dev, cuda_stream);
    if (ms != MOE_OK) return ms;
    if (T > 0 && cudaMemcpyAsync(y_host, y_dev, (size_t)T * d.H * 2, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return MOE_ERR_CUDA;
    return MOE_OK;
}

moe_status moe_step_host(moe_ctx *ctx, const float *logits_host, const void *x_host, int32_t T,
                         const moe_dispatch_out *out, float *logits_dev, void *x_dev, void *y_dev,
                         void *y_host, void *cuda_stream)
{
    const moe_status ms = moe_step_host_async(ctx, logits_host, x_host, T, out, logits_dev, x_dev, y_dev,
                                              y_host, cuda_stream);
    if (ms != MOE_OK) return ms;
    return cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

moe_status moe_set_tuning(moe_ctx *ctx, int32_t option, int32_t value)
{
    if (!ctx || option < 0 || option >= kNumTuning || value < -1) return MOE_ERR_INVALID_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return MOE_ERR_CUDA;
    const int before = ctx->tune[option];
    ctx->tune[option] = value;
    if (option == MOE_TUNE_ROUTE_LANES_PER_TOKEN || option == MOE_TUNE_ROUTE_TOKENS_PER_TILE) {
        // the routing tile decides the size of the scan scratch: derive again and regrow it
        Derived d;
        if (!derive(&ctx->cfg, &d, std::max(0, ctx->tune[MOE_TUNE_ROUTE_LANES_PER_TOKEN]),
                    std::max(0, ctx->tune[MOE_TUNE_ROUTE_TOKENS_PER_TILE]))) {
            ctx->tune[option] = before;
            return MOE_ERR_INVALID_ARG;
        }
        const Derived old = ctx->d;
        ctx->d = d;
        if (!alloc_scan_scratch(ctx, nullptr) || cudaDeviceSynchronize() != cudaSuccess) {
            cudaGetLastError();
            ctx->d = old; ctx->tune[option] = before;
            return MOE_ERR_CUDA;
        }
        ctx->device_bytes = device_bytes_for(d, ctx->cfg.max_tokens);
    }
    configure_launch(ctx);
    if (option == MOE_TUNE_COMBINE_IMPL && ctx->ep_world > 0 && ctx->combine_impl != 1) {
        ctx->tune[option] = before;                        // the group mode needs the ring combine
        configure_launch(ctx);
        return MOE_ERR_INVALID_ARG;
    }
    return MOE_OK;
}

moe_status moe_debug_skip_ticket(moe_ctx *ctx)
{
    if (!ctx) return MOE_ERR_INVALID_ARG;
    const unsigned one = 1u;
    if (cudaDeviceSynchronize() != cudaSuccess ||
        cudaMemcpy(&ctx->d_ctl->ticket, &one, sizeof(one), cudaMemcpyHostToDevice) != cudaSuccess)
        return MOE_ERR_CUDA;
    return MOE_OK;
}

moe_status moe_set_timing_event(moe_ctx *ctx, void *cuda_event)
{
    if (!ctx) return MOE_ERR_INVALID_ARG;
    ctx->timing_event = static_cast<cudaEvent_t>(cuda_event);
    return MOE_OK;
}

moe_status moe_get_device_status(moe_ctx *ctx, int32_t *code)
{
    if (!ctx || !code) return MOE_ERR_INVALID_ARG;
    moe::Control c;
    if (cudaDeviceSynchronize() != cudaSuccess ||
        cudaMemcpy(&c, ctx->d_ctl, sizeof(c), cudaMemcpyDeviceToHost) != cudaSuccess)
        return MOE_ERR_CUDA;
    *code = c.status;
    if (c.status != kDevOk) {
        // stale look-back descriptors carry the failed step's epoch: move past it
        unsigned next = c.epoch + 1u;
        const moe::Control fresh = {0u, next ? next : 1u, kDevOk, 0};
        if (cudaMemcpy(ctx->d_ctl, &fresh, sizeof(fresh), cudaMemcpyHostToDevice) != cudaSuccess)
            return MOE_ERR_CUDA;
    }
    return MOE_OK;
}

moe_status moe_route_destroy(moe_ctx *ctx)
{
    if (!ctx) return MOE_OK;
    cudaDeviceSynchronize();
    free_ctx(ctx);
    return MOE_OK;
}

}  // extern "C"
