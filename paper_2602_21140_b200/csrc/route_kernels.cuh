// K_route: gate, availability mask, group-limited top-k, weight renormalisation,
// live-replica pick, per-slot histogram, prefix over tiles by aggregate look-back
// and the final per-slot / per-rank offsets — one kernel, one pass over the logits.
//
// Work split: a CTA of 32 warps takes one tile of `tokens_per_block` consecutive
// tokens (tiles are handed out by an atomic ticket, so every tile a CTA may wait
// for is already running).  A warp routes 32/LPT tokens at once: a token owns
// LPT consecutive lanes and lane s of them holds experts [s*EPL, (s+1)*EPL) (in
// its own column of a shared-memory table), which makes "lower lane" equal
// "lower expert id" for tie-breaks, puts a whole expert group inside a
// power-of-two run of lanes, and keeps every lane busy in the serial top-k
// rounds.  The kernel is bound by latency — instruction fetch, shared-memory
// conflicts, trips to L2 — not by arithmetic or DRAM, and is written accordingly:
// rolled loops, conflict-free tables, few dependent round trips.
//
// Prefix over tiles: the whole problem fits in one wave of CTAs (the host sizes the
// tile so that a step has about one tile per SM), so all tiles publish at about the
// same time and a chained look-back (wait for the predecessor's inclusive prefix)
// would serialise them.  Instead every tile publishes only its own per-slot counts,
// two 16-bit counts and the step's 32-bit epoch to a 64-bit word (the epoch makes a stale
// word invalid without any clearing, and data and validity arrive in one load), and sums
// the counts of ALL earlier tiles with independent 16-byte loads: one L2 round trip when
// the other tiles have already published.
#pragma once

#include "device_utils.cuh"

namespace moe {

constexpr int kRouteThreads = 1024;
constexpr int kRouteWarps = kRouteThreads / 32;

// Routing state blob in device memory (int32 words), rewritten by a remap:
//   [0] fallback expert (lowest available id)   [1] number of available experts
//   [2 .. 2+rank_words)  rank-alive bitmap, bit r of word r/32 set = rank r alive
//   [.. +expert_words)   failed-expert bitmap, bit e set = expert e masked whatever its replicas
//   [...]                replica table [E][max_rep]: ascending slot ids, -1 padded
//   [...]                slot order [P]: physical slot at each position of the send-buffer
//                        layout (logical-rank order; identity unless ranks were compacted)
constexpr int kStateHeaderWords = 2;

// A step has at most this many tiles.
constexpr int kMaxRouteTiles = 1024;

// Live-replica lists derived from the state blob: per expert 1 + max_rep words, the number of
// live replicas followed by their slots in ascending order.  k_derive_live rebuilds them on
// the stream right after every state copy, so the routing kernel loads one flat table
// instead of chasing bitmap words through the replica table in every CTA of every step.
struct DeriveParams {
    const int32_t *state;
    int E, S, max_rep, rank_words, expert_words;
    int32_t *live;            // out [E][1 + max_rep]
};

constexpr int kDeriveThreads = 256;

__global__ void __launch_bounds__(kDeriveThreads) k_derive_live(DeriveParams p)
{
    const uint32_t *alive = reinterpret_cast<const uint32_t *>(p.state + kStateHeaderWords);
    const uint32_t *lost = alive + p.rank_words;
    const int32_t *table = p.state + kStateHeaderWords + p.rank_words + p.expert_words;
    const int e = blockIdx.x * kDeriveThreads + threadIdx.x;
    if (e >= p.E) return;
    int32_t *ent = p.live + (size_t)e * (1 + p.max_rep);
    const bool expert_ok = !((lost[e >> 5] >> (e & 31)) & 1u);
    int n = 0;
    for (int r = 0; r < p.max_rep; ++r) {
        const int slot = table[e * p.max_rep + r];         // ascending, -1 padded
        ent[1 + r] = -1;
        if (slot < 0 || !expert_ok) continue;
        const int rank = slot / p.S;
        if ((alive[rank >> 5] >> (rank & 31)) & 1u) ent[1 + n++] = slot;
    }
    ent[0] = n;
}

struct RouteParams {
    const float *logits;      // [T,E]
    int T, E, k, P, R, S, max_rep;
    int score_func, n_group, topk_group, lanes_per_group, group_m;
    float route_scale;
    int tokens_per_block;
    int p_pad;                // P rounded up to a multiple of 8: row pitch of tile_counts
    int rank_words, expert_words;
    unsigned spin_limit;      // polls before a bounded wait gives up
    const int32_t *state;     // routing state blob (header and slot order are read here)
    const int32_t *live;      // derived live-replica lists [E][1 + max_rep]
    const float *bias;        // [E]
    int32_t *topk_ids;        // [T,k]
    float *topk_weights;      // [T,k]
    int32_t *topk_slot;       // [T,k]
    int32_t *pos_in_slot;     // [T*k]: stable rank of assignment i inside its slot
    int32_t *slot_counts, *slot_offsets, *rank_counts, *rank_offsets;
    int alias_wcount;         // the histogram's count matrix shares the token phase's tables (see route_smem_bytes)
    int prefetch;             // bit 0: ask the small tables into L2 before the wait; bit 1: the logits too
    ulonglong2 *tile_counts;  // [tiles][p_pad/4]: per tile, four slots to a 16-byte entry: two words
                              // of (epoch << 32 | count of the odd slot << 16 | count of the even slot)
    Control *ctl;
};

// Shared memory of the routing kernel.  The first region holds the per-warp tables of the token
// phase ([blocks][32] 16-byte entries: logits, then key codes; [blocks][32] block bests).  The
// per-warp count matrix of the histogram phase ([32][P] 16-bit) normally has a region of its own
// and is zeroed before the kernel's wait; with very many slots or experts the two do not fit
// side by side, and the matrix then shares the first region (`alias`), at the price of a
// zeroing pass and a barrier between the two phases.
__host__ __device__ inline size_t route_region0_words(int P, int epl, bool alias)
{
    const size_t code_words = (size_t)kRouteWarps * ((epl + 3) / 4) * 32 * 5;
    const size_t count_words = alias ? ((size_t)kRouteWarps * P * sizeof(uint16_t) + 3) / 4 : 0;
    return ((code_words > count_words ? code_words : count_words) + 3) & ~(size_t)3;
}

__host__ __device__ inline size_t route_smem_bytes(int E, int max_rep, int tokens_per_block, int k,
                                                   int P, int epl, bool alias)
{
    const size_t p_pad = ((size_t)P + 7) & ~(size_t)7;
    const size_t bias_words = (size_t)((epl + 3) / 4 * 4) * 16 + 16;   // bias by (expert of the lane, lane); availability bits
    size_t words = route_region0_words(P, epl, alias) + bias_words + (size_t)E * (1 + max_rep) +
                   2 * (size_t)tokens_per_block * k + 2 * p_pad + (size_t)P;
    return words * sizeof(int32_t) + (alias ? 0 : (size_t)kRouteWarps * P * sizeof(uint16_t));
}

// Route 32/LPT tokens with one warp.  Lanes [sub*LPT, (sub+1)*LPT) own token
// t_first + sub.  On return, sub-lane j < k of a token holds its j-th chosen
// expert, the weight and the physical slot.
//
// The element work is written as a short loop over blocks of four experts rather than
// unrolled over all EPL of them: every warp passes through this code about once per
// launch, and straight-line code that is run once is paced by instruction fetch (the
// unrolled form measured ~350 cycles per expert with nothing but integer work in it),
// while a loop body that stays in the instruction cache issues at full rate.  For the loop
// to be possible nothing may be indexed by the block number in registers, so a lane keeps
// its logits, then its key codes, and its per-block best codes in its own column of two
// small shared-memory tables (s_blk[b * 32 + lane], s_bmx[b * 32 + lane]: no two lanes
// ever touch the same word, so no synchronisation is needed).
template <int EPL, int LPT>
__device__ __forceinline__ void route_tokens(const RouteParams &p, int t_first, uint32_t avail_mask,
                                             const int32_t *s_live, const float *s_bias, uint4 *s_blk,
                                             uint32_t *s_bmx, int fallback_expert, int &out_id,
                                             float &out_w, int &out_slot)
{
    const unsigned full = 0xffffffffu;
    const int lane = lane_id();
    const int sub = lane / LPT, sl = lane % LPT;
    const int E = p.E;
    const int e0 = sl * EPL;
    const int t = min(t_first + sub, p.T - 1);           // lanes past the end redo the last token
    const float *row = p.logits + (size_t)t * E;
    const float neg_inf = __int_as_float(0xff800000);
    const bool sigmoid = p.score_func != 0;
    const bool grouped = p.n_group > 1;
    constexpr int kBlocks = (EPL + 3) / 4;
    uint4 *mine = s_blk + lane;
    uint32_t *mine_bmx = s_bmx + lane;

    // 1. this lane's logits, global -> shared without passing through registers (all requests
    //    are in flight together; entries past the lane's experts or past E read -inf)
    if ((EPL % 4 == 0) && (E == LPT * EPL)) {
#pragma unroll
        for (int b = 0; b < kBlocks; ++b) cp_async_16(mine + b * 32, row + e0 + 4 * b);
    } else {
#pragma unroll
        for (int q = 0; q < 4 * kBlocks; ++q) {
            float *dst = reinterpret_cast<float *>(mine + (q / 4) * 32) + (q % 4);
            if (q < EPL && e0 + q < E) cp_async_4(dst, row + e0 + q);
            else *dst = neg_inf;
        }
    }
    cp_async_wait_all();

    // 2. gate scores, availability mask, order-preserving key codes (written over the logits),
    //    the best code of every block, and the two best keys of this lane (for the group scores).
    //    Four experts per trip: four independent chains of arithmetic keep the pipeline busy,
    //    and the body still fits the instruction cache.
    float h1 = neg_inf, h2 = neg_inf;
    uint32_t lbest = 0; int lb = 0;
#pragma unroll 1
    for (int b = 0; b < kBlocks; ++b) {
        const float4 v = *reinterpret_cast<const float4 *>(mine + b * 32);
        const float lg[4] = {v.x, v.y, v.z, v.w};
        uint32_t c[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int q = 4 * b + u;
            float kf = lg[u];
            if (sigmoid) kf = __fadd_rn(sigmoid_spec(lg[u]), s_bias[q * LPT + sl]);
            const bool ok = ((avail_mask >> q) & 1u) && (lg[u] != neg_inf);
            kf = ok ? kf : neg_inf;
            if (grouped) {                                // running two best keys of the lane
                h2 = fmaxf(h2, fminf(h1, kf));
                h1 = fmaxf(h1, kf);
            }
            c[u] = key_code(kf);
        }
        *(mine + b * 32) = make_uint4(c[0], c[1], c[2], c[3]);
        const uint32_t bmax = max(max(c[0], c[1]), max(c[2], c[3]));
        mine_bmx[b * 32] = bmax;
        if (bmax > lbest) { lbest = bmax; lb = b; }      // lowest block among equals
    }

    // group-limited selection: score = sum of the (up to) group_m best finite keys
    if (grouped) {
#pragma unroll 1
        for (int off = 1; off < p.lanes_per_group; off <<= 1) {
            const float o1 = __shfl_xor_sync(full, h1, off, LPT);
            const float o2 = __shfl_xor_sync(full, h2, off, LPT);
            const float n1 = fmaxf(h1, o1);
            const float n2 = fmaxf(fminf(h1, o1), fmaxf(h2, o2));
            h1 = n1; h2 = n2;
        }
        const float gscore = (p.group_m == 1 || h2 == neg_inf) ? h1 : __fadd_rn(h1, h2);
        const int g = sl / p.lanes_per_group;
        int rank = 0;
#pragma unroll 1
        for (int gp = 0; gp < p.n_group; ++gp) {
            const float o = __shfl_sync(full, gscore, gp * p.lanes_per_group, LPT);
            rank += (o > gscore) || (o == gscore && gp < g);
        }
        if (!((g < p.n_group) && (rank < p.topk_group))) lbest = 0;   // this lane's group is not kept
    }

    // top-k: k rounds of arg-max over the codes.  A lane offers the best code it has left; the
    // winner (lowest lane among equals = lowest expert id) reads the block of four that held
    // it, blanks the first element equal to it (lowest id among equals), and finds its next best
    // from the per-block bests.
    const unsigned seg_mask = ((LPT == 32) ? 0xffffffffu : ((1u << LPT) - 1u)) << (sub * LPT);
    int my_id = fallback_expert; bool my_bad = false;
#pragma unroll 1
    for (int j = 0; j < p.k; ++j) {
        const uint32_t m = __reduce_max_sync(seg_mask, lbest);
        const unsigned ball = __ballot_sync(full, lbest == m);
        const int src = __ffs(ball & seg_mask) - 1 - sub * LPT;   // lowest lane = lowest expert id
        const bool bad = m <= kCodeNegInf;               // nothing selectable is left
        int taken_e = 0;
        if (sl == src && !bad) {                         // drop the pick, find the lane's next best
            const uint4 blk = *(mine + lb * 32);
            const int u = (blk.x == lbest) ? 0 : (blk.y == lbest) ? 1 : (blk.z == lbest) ? 2 : 3;
            reinterpret_cast<uint32_t *>(mine + lb * 32)[u] = 0u;
            taken_e = e0 + lb * 4 + u;
            const uint32_t c0 = (u == 0) ? 0u : blk.x, c1 = (u == 1) ? 0u : blk.y;
            const uint32_t c2 = (u == 2) ? 0u : blk.z, c3 = (u == 3) ? 0u : blk.w;
            mine_bmx[lb * 32] = max(max(c0, c1), max(c2, c3));
            lbest = 0; lb = 0;
#pragma unroll
            for (int b = 0; b < kBlocks; ++b) {
                const uint32_t bm = mine_bmx[b * 32];
                if (bm > lbest) { lbest = bm; lb = b; }
            }
        }
        const int sel_e = __shfl_sync(full, taken_e, src, LPT);
        if (sl == j) { my_id = bad ? fallback_expert : sel_e; my_bad = bad; }
    }

    // weights: ratio of the chosen scores, summed and divided in double.  The score of a
    // chosen expert is recomputed from its logit (same operations, same bits as above).
    float my_val = 0.0f;
    if (sl < p.k) {
        const float lgv = __ldg(row + my_id);
        my_val = sigmoid ? sigmoid_spec(lgv) : lgv;
    }
    const float v0 = __shfl_sync(full, my_val, 0, LPT);
    double u = 0.0;
    if (sl < p.k) {
        if (my_bad) u = 1.0;
        else if (!sigmoid) u = exp((double)__fsub_rn(my_val, v0));
        else u = (double)my_val;
    }
    double usum = 0.0;
#pragma unroll 1
    for (int j = 0; j < p.k; ++j) usum += __shfl_sync(full, u, j, LPT);
    out_w = (float)((double)p.route_scale * u / usum);

    // replica pick: (t mod live count)-th entry of the ascending live list
    out_id = my_id;
    out_slot = -1;
    if (sl < p.k) {
        const int32_t *ent = s_live + my_id * (1 + p.max_rep);
        out_slot = ent[1 + t % ent[0]];
    }
    if (__any_sync(full, my_bad) && lane == 0) report_status(p.ctl, kDevInsufficientExperts);
}

template <int EPL, int LPT>
__global__ void __launch_bounds__(kRouteThreads, 1) k_route(RouteParams p)
{
    extern __shared__ __align__(16) int32_t smem[];
    const int E = p.E, P = p.P, k = p.k, tb = p.tokens_per_block;
    const int NA = tb * k;
    const int live_words = 1 + p.max_rep;
    constexpr int kBlockEntries = (EPL + 3) / 4 * 32;   // one warp's [blocks][32] table
    uint4 *s_blk = reinterpret_cast<uint4 *>(smem) + (threadIdx.x >> 5) * kBlockEntries;
    uint32_t *s_bmx = reinterpret_cast<uint32_t *>(smem) + kRouteWarps * kBlockEntries * 4 +
                      (threadIdx.x >> 5) * kBlockEntries;
    // bias of expert sl * EPL + q at s_bias[q * LPT + sl] (lanes of a token read neighbouring words),
    // zero past E; then 16 words of availability bits, bit e = expert e has a live replica
    constexpr int kBiasWords = (EPL + 3) / 4 * 4 * 16;
    const int region0 = (int)route_region0_words(P, EPL, p.alias_wcount != 0);
    float *s_bias = reinterpret_cast<float *>(smem) + region0;
    uint32_t *s_avail = reinterpret_cast<uint32_t *>(s_bias + kBiasWords);               // [16]
    int32_t *s_live = smem + region0 + kBiasWords + 16;   // [E][1 + max_rep] live count, live slots
    int32_t *s_slot = s_live + E * live_words;        // [NA] slot of each assignment of the tile
    int32_t *s_lrank = s_slot + NA;                   // [NA] stable rank inside the tile
    int32_t *s_hist = s_lrank + NA;                   // [p_pad] tile histogram (running)
    int32_t *s_excl = s_hist + p.p_pad;               // [p_pad] assignments on slot p in earlier tiles
    int32_t *s_order = s_excl + p.p_pad;              // [P]  physical slot at each layout position
    uint16_t *s_wcount = p.alias_wcount ? reinterpret_cast<uint16_t *>(smem)
                                        : reinterpret_cast<uint16_t *>(s_order + P);  // [32][P] one round's counts
    __shared__ unsigned s_ticket, s_epoch;
    __shared__ int s_warp_sums[kRouteWarps];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned full = 0xffffffffu;

    // Before the wait only this CTA's own shared memory is touched.
    // (Loops that a thread passes through about once are kept rolled throughout this kernel: it
    // is paced by instruction fetch, and unrolled copies of once-run code only add to that.)
#pragma unroll 1
    for (int q = tid; q < p.p_pad; q += kRouteThreads) { s_hist[q] = 0; s_excl[q] = 0; }
    if (!p.alias_wcount) {
#pragma unroll 1
        for (int q = tid; q < kRouteWarps * P; q += kRouteThreads) s_wcount[q] = 0;
    }

    // ... apart from hints: under programmatic dependent launch this CTA may be resident well
    // before the previous kernel has finished, and the tables it is about to read were last
    // touched a whole step ago (2 GB of rows have passed through L2 since).  Asking for them now
    // turns DRAM misses on the critical path into L2 hits.  A hint cannot return stale data:
    // L2 is where every write lands.
    if (p.prefetch & 1) {
        const int words = E * live_words;
        if (tid * 32 < words) prefetch_l2(p.live + tid * 32);
        if (tid * 32 < P) prefetch_l2(p.state + kStateHeaderWords + p.rank_words + p.expert_words + E * p.max_rep + tid * 32);
        if (tid * 32 < E) prefetch_l2(p.bias + tid * 32);
        if (tid == 0) { prefetch_l2(p.ctl); prefetch_l2(p.state); }
    }
    if ((p.prefetch & 2) && p.logits != nullptr) {
        // the tile is not known before the ticket: every CTA asks for an equal share of the tensor
        const size_t total = (size_t)p.T * E * sizeof(float);
        const size_t share = ((total + gridDim.x - 1) / gridDim.x + 127) & ~(size_t)127;
        const size_t lo = (size_t)blockIdx.x * share, hi = min(total, lo + share);
#pragma unroll 1
        for (size_t off = lo + (size_t)tid * 128; off < hi; off += (size_t)kRouteThreads * 128)
            prefetch_l2(reinterpret_cast<const char *>(p.logits) + off);
    }

    // Wait for the previous kernel first and only then let the scatter be scheduled: the scatter
    // requests its first x rows before its own wait, which is safe only once whatever produced x
    // (a kernel before this one) is known to have completed.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (tid == 0) {
        // ticket (low word) and epoch (high word) share one 64-bit word: a single atomic add
        // takes the ticket and reads the epoch (the ticket never carries: it is reset every step)
        const unsigned long long te = atomicAdd(reinterpret_cast<unsigned long long *>(&p.ctl->ticket), 1ull);
        s_ticket = (unsigned)te;
        s_epoch = (unsigned)(te >> 32);
    }
    // live replica lists (availability mask and replica pick) and the layout order of the slots
#pragma unroll 1
    for (int i = tid; i < E * live_words; i += kRouteThreads) s_live[i] = p.live[i];
    if (tid < 512) {                                   // E <= 512: whole warps, one expert per thread
        const bool live = tid < E && p.live[tid * live_words] > 0;
        const unsigned bits = __ballot_sync(full, live);
        if (lane == 0) s_avail[tid >> 5] = bits;       // all 16 words are written, zero past E
    }
    if (tid < kBiasWords) {                            // every word of the table has this one writer
        const int q = tid / LPT, e = (tid % LPT) * EPL + q;
        s_bias[tid] = (p.score_func == 1 && q < EPL && e < E) ? p.bias[e] : 0.0f;
    }
    const int32_t *order = p.state + kStateHeaderWords + p.rank_words + p.expert_words + E * p.max_rep;
#pragma unroll 1
    for (int q = tid; q < P; q += kRouteThreads) s_order[q] = order[q];
    const int fallback_expert = p.state[0];
    __syncthreads();

    const unsigned ticket = s_ticket;
    const unsigned epoch = s_epoch;
    if (ticket >= gridDim.x) {
        // The control word was not armed for this step (an earlier step gave up and the host has
        // not yet read the status): route nothing rather than index past the tile arrays.
        if (tid == 0) report_status(p.ctl, kDevTimeout);
        return;
    }
    const int t0 = (int)ticket * tb;
    const int n_tok = min(tb, p.T - t0);

    // which of this lane's experts have a live replica: the same for every token it routes
    constexpr int kTokPerWarp = 32 / LPT;
    const int sub = lane / LPT, sl = lane % LPT;
    uint32_t avail_mask;
    {
        const int e0 = sl * EPL;                          // EPL <= 32 bits starting at bit e0 of the bitmap
        const uint32_t lo = s_avail[(e0 >> 5) & 15], hi = s_avail[((e0 >> 5) + 1) & 15];
        avail_mask = __funnelshift_r(lo, hi, e0 & 31);
        avail_mask &= 0xffffffffu >> (32 - EPL);
        if (e0 >= E) avail_mask = 0;
    }

    // Dense-FFN mode (score_func 2): the "experts" are the k = TP shards of E/k replicated
    // FFN groups; a group is healthy only if every shard is live.  List the healthy groups.
    const bool dense = p.score_func == 2;
    if (dense) {
        if (tid == 0) {
            int n = 0;
#pragma unroll 1
            for (int g = 0; g < E / k; ++g) {
                bool healthy = true;
#pragma unroll 1
                for (int sh = 0; sh < k; ++sh) healthy = healthy && (s_live[(g * k + sh) * live_words] > 0);
                if (healthy) s_lrank[n++] = g;             // s_lrank is free until the histogram step
            }
            s_warp_sums[0] = n;
        }
        __syncthreads();
    }
    const int n_healthy = dense ? s_warp_sums[0] : 0;

    // ---- gate, mask, selection, weights, replica: per token ----------------
#pragma unroll 1
    for (int lt0 = warp * kTokPerWarp; lt0 < tb; lt0 += kRouteWarps * kTokPerWarp) {
        const int lt = lt0 + sub;
        const int t = t0 + lt;
        int id = 0, slot = -1; float w = 0.0f;
        if (t0 + lt0 < p.T) {                            // warp-uniform: some token of the warp exists
            if (dense) {
                // tokens are dealt evenly over the healthy groups; each goes to all shards of its
                // group with weight route_scale (the shards' partial results add up in combine)
                if (sl < k && t < p.T) {
                    id = s_lrank[t % n_healthy] * k + sl;
                    w = p.route_scale;
                    slot = s_live[id * live_words + 1 + t % s_live[id * live_words]];
                }
            } else {
                route_tokens<EPL, LPT>(p, t0 + lt0, avail_mask, s_live, s_bias, s_blk, s_bmx, fallback_expert,
                                       id, w, slot);
            }
            if (t >= p.T) slot = -1;
            if (sl < k && t < p.T) {
                const size_t i = (size_t)t * k + sl;
                p.topk_ids[i] = id;
                p.topk_weights[i] = w;
                p.topk_slot[i] = slot;
            }
        }
        if (sl < k && lt < tb) s_slot[lt * k + sl] = slot;
    }
    __syncthreads();

    if (p.alias_wcount) {                              // the token phase's tables are dead: reuse them
#pragma unroll 1
        for (int q = tid; q < kRouteWarps * P; q += kRouteThreads) s_wcount[q] = 0;
        __syncthreads();
    }

    // ---- tile histogram and stable rank of every assignment inside the tile 
    // Rounds of 1024 assignments in ascending i.  Inside a round, match_any gives
    // the rank among equal slots of a warp and the per-warp counts; a scan down
    // each slot's column of counts orders the warps.
#pragma unroll 1
    for (int base = 0; base < NA; base += kRouteThreads) {
        const int i = base + tid;
        const int slot = (i < NA) ? s_slot[i] : -1;
        const unsigned peers = __match_any_sync(full, slot);
        const int rank_in_warp = __popc(peers & lanemask_lt());
        if (slot >= 0 && rank_in_warp == 0) s_wcount[warp * P + slot] = (uint16_t)__popc(peers);
        __syncthreads();
#pragma unroll 1
        for (int q = tid; q < P; q += kRouteThreads) {
            int run = s_hist[q];
#pragma unroll 4
            for (int w2 = 0; w2 < kRouteWarps; ++w2) {
                const int c = s_wcount[w2 * P + q];
                s_wcount[w2 * P + q] = (uint16_t)run;      // run < 65536: a tile has <= 32768 assignments
                run += c;
            }
            s_hist[q] = run;
        }
        __syncthreads();
        if (slot >= 0) s_lrank[i] = (int)s_wcount[warp * P + slot] + rank_in_warp;
        if (base + kRouteThreads < NA) {
            __syncthreads();
#pragma unroll 1
            for (int q = tid; q < kRouteWarps * P; q += kRouteThreads) s_wcount[q] = 0;
            __syncthreads();
        }
    }

    // ---- prefix over tiles: publish this tile's counts, sum those of all earlier tiles
    const int groups = p.p_pad / 4;                        // 16-byte entries per tile row
    {
        ulonglong2 *mine = p.tile_counts + (size_t)ticket * groups;
        const unsigned long long tag = (unsigned long long)epoch << 32;
#pragma unroll 1
        for (int q4 = tid; q4 < groups; q4 += kRouteThreads) {
            const int32_t *h = s_hist + 4 * q4;            // entries past P stay zero
            st_relaxed_v2_u64(mine + q4, tag | (unsigned)h[0] | ((unsigned)h[1] << 16),
                              tag | (unsigned)h[2] | ((unsigned)h[3] << 16));
        }
    }
    if (ticket > 0) {
        // thread = (segment g of the earlier tiles, entry q4); every load is independent of the others
        const int nseg = kRouteThreads / groups;           // >= 1: P <= 4096
        const int g = tid / groups, q4 = tid % groups;
        bool gave_up = false;
        int acc[4] = {0, 0, 0, 0};
        if (g < nseg) {
            // Up to kBatch entries are requested together and the stale ones (their tile has not
            // published yet) are requested again together, so a round of retries costs one trip
            // to L2 however many of the entries were stale.
            constexpr int kBatch = 8;
#pragma unroll 1
            for (int b0 = g; b0 < (int)ticket && !gave_up; b0 += nseg * kBatch) {
                ulonglong2 v[kBatch];
                unsigned pending = 0;
#pragma unroll
                for (int u = 0; u < kBatch; ++u)
                    if (b0 + u * nseg < (int)ticket) pending |= 1u << u;
                unsigned spins = 0;
                while (true) {
#pragma unroll
                    for (int u = 0; u < kBatch; ++u)
                        if ((pending >> u) & 1u)
                            v[u] = ld_relaxed_v2_u64(p.tile_counts + (size_t)(b0 + u * nseg) * groups + q4);
#pragma unroll
                    for (int u = 0; u < kBatch; ++u) {
                        if (((pending >> u) & 1u) && (unsigned)(v[u].x >> 32) == epoch &&
                            (unsigned)(v[u].y >> 32) == epoch) {
                            acc[0] += (int)(v[u].x & 0xffffu); acc[1] += (int)((v[u].x >> 16) & 0xffffu);
                            acc[2] += (int)(v[u].y & 0xffffu); acc[3] += (int)((v[u].y >> 16) & 0xffffu);
                            pending &= ~(1u << u);
                        }
                    }
                    if (pending == 0) break;
                    if (++spins > p.spin_limit ||
                        ((spins & 255u) == 0 && ld_relaxed_s32(&p.ctl->status) == kDevTimeout)) {
                        gave_up = true;
                        break;
                    }
                    if (spins > 4) __nanosleep(kSpinSleepNs);
                }
            }
        }
        if (groups <= 16 && (groups & (groups - 1)) == 0) {
            // few slots: lanes q4, q4 + groups, ... of a warp hold partial sums of the same
            // entry; add them up in registers before touching shared memory
#pragma unroll
            for (int u = 0; u < 4; ++u)
                for (int off = groups; off < 32; off <<= 1) acc[u] += __shfl_xor_sync(full, acc[u], off);
            if (lane >= groups) { acc[0] = acc[1] = acc[2] = acc[3] = 0; }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (acc[u]) atomicAdd(&s_excl[4 * q4 + u], acc[u]);
        if (__syncthreads_or(gave_up)) {
            // An earlier tile never published.  Nothing of this tile's placement is written, the
            // control word stays as it is, and the status word tells the host (which re-arms it).
            if (tid == 0) report_status(p.ctl, kDevTimeout);
            return;
        }
    } else {
        __syncthreads();
    }

    // stable rank of every assignment of the tile inside its slot, over all tiles
#pragma unroll 1
    for (int i = tid; i < n_tok * k; i += kRouteThreads)
        p.pos_in_slot[(size_t)t0 * k + i] = s_excl[s_slot[i]] + s_lrank[i];

    if (ticket != gridDim.x - 1) return;

    // ---- the last tile knows every total: per-slot counts and offsets -----
    // exclusive scan over the P layout positions (position q holds physical slot order[q]),
    // a contiguous chunk of positions per thread
#pragma unroll 1
    for (int q = tid; q < P; q += kRouteThreads) s_hist[q] += s_excl[q];     // totals per physical slot
    __syncthreads();
    const int chunk = (P + kRouteThreads - 1) / kRouteThreads;
    const int q0 = tid * chunk;
    int local = 0;
#pragma unroll 1
    for (int q = q0; q < min(P, q0 + chunk); ++q) local += s_hist[s_order[q]];
    int incl = local;
    for (int off = 1; off < 32; off <<= 1) {
        const int o = __shfl_up_sync(full, incl, off);
        if (lane >= off) incl += o;
    }
    if (lane == 31) s_warp_sums[warp] = incl;
    __syncthreads();                                   // also: all reads of s_excl above are done
    int warp_base = 0;
#pragma unroll 1
    for (int w2 = 0; w2 < warp; ++w2) warp_base += s_warp_sums[w2];
    int run = warp_base + incl - local;
#pragma unroll 1
    for (int q = q0; q < min(P, q0 + chunk); ++q) {
        const int slot = s_order[q];
        const int tot = s_hist[slot];
        p.slot_counts[slot] = tot;
        p.slot_offsets[slot] = run;
        s_excl[q] = run;                               // offset of layout position q
        run += tot;
    }
    if (tid == kRouteThreads - 1) {
        p.slot_offsets[P] = run;
        p.rank_offsets[p.R] = run;
    }
    __syncthreads();
#pragma unroll 1
    for (int r = tid; r < p.R; r += kRouteThreads) {   // r-th rank of the layout order
        int c = 0;
#pragma unroll 1
        for (int s = 0; s < p.S; ++s) c += s_hist[s_order[r * p.S + s]];
        p.rank_counts[r] = c;
        p.rank_offsets[r] = s_excl[r * p.S];
    }
    // every ticket of this step has been taken and every tile has read the
    // epoch (it published before this tile could finish): arm the next step
    if (tid == 0) {
        p.ctl->ticket = 0;
        unsigned next = epoch + 1u;
        p.ctl->epoch = next ? next : 1u;
    }
}

}  // namespace moe
