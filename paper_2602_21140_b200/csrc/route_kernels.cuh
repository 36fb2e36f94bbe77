// K_route: gate, availability mask, group-limited top-k, weight renormalisation,
// live-replica pick, per-slot histogram, decoupled look-back scan over tiles and
// the final per-slot / per-rank offsets — one kernel, one pass over the logits.
//
// Work split: a CTA of 8 warps takes one tile of `tokens_per_block` consecutive
// tokens (tiles are handed out by an atomic ticket, so every tile a CTA may wait
// for is already running).  A warp routes one token at a time with the experts
// laid out contiguously over lanes (lane l holds experts [l*EPL, (l+1)*EPL)),
// which makes "lower lane" equal "lower expert id" for tie-breaks and puts a
// whole expert group inside a power-of-two run of lanes.
#pragma once

#include "device_utils.cuh"

namespace moe {

constexpr int kRouteThreads = 256;
constexpr int kRouteWarps = kRouteThreads / 32;

// Routing state blob in device memory (int32 words), rewritten by a remap:
//   [0] fallback expert (lowest available id)   [1] number of available experts
//   [2 .. 2+rank_words)  rank-alive bitmap, bit r of word r/32 set = rank r alive
//   [2+rank_words ...)   replica table [E][max_rep]: ascending slot ids, -1 padded
constexpr int kStateHeaderWords = 2;

// Look-back descriptor, one 64-bit word per (tile, slot):
//   bits 63..32 epoch of the step that wrote it, 31..30 flag, 29..0 count
constexpr unsigned long long kFlagAggregate = 1ull;   // count of this tile only
constexpr unsigned long long kFlagInclusive = 2ull;   // count of tiles 0..this

struct RouteParams {
    const float *logits;      // [T,E]
    int T, E, k, P, R, S, max_rep;
    int score_func, n_group, topk_group, lanes_per_group, group_m;
    float route_scale;
    int tokens_per_block;
    int rank_words;
    const int32_t *state;     // routing state blob
    const float *bias;        // [E]
    int32_t *topk_ids;        // [T,k]
    float *topk_weights;      // [T,k]
    int32_t *topk_slot;       // [T,k]
    int32_t *pos_in_slot;     // [T*k]: stable rank of assignment i inside its slot
    int32_t *slot_counts, *slot_offsets, *rank_counts, *rank_offsets;
    unsigned long long *desc; // [tiles, P]
    Control *ctl;
};

__host__ __device__ inline size_t route_smem_bytes(int E, int max_rep, int tokens_per_block, int k,
                                                   int P)
{
    size_t words = (size_t)E + (size_t)E * max_rep + 2 * (size_t)tokens_per_block * k +
                   2 * (size_t)P + (size_t)kRouteWarps * P;
    return words * sizeof(int32_t);
}

// Route one token with the whole warp.  Lane j < k leaves with the j-th chosen
// expert, its weight and its physical slot.
template <int EPL>
__device__ __forceinline__ void route_token(const RouteParams &p, int t, const int32_t *s_nlive,
                                            const int32_t *s_live, int fallback_expert,
                                            int &out_id, float &out_w, int &out_slot)
{
    const unsigned full = 0xffffffffu;
    const int lane = lane_id();
    const int E = p.E;
    const int e0 = lane * EPL;
    const float *row = p.logits + (size_t)t * E;
    const float neg_inf = __int_as_float(0xff800000);

    float val[EPL];    // what the weight is made of: logit (softmax) or sigmoid score
    float key[EPL];    // what selection compares

    // a1 gate scores, a2 availability mask
    float lg[EPL];
    if ((EPL % 4 == 0) && (E == 32 * EPL)) {
        const float4 *row4 = reinterpret_cast<const float4 *>(row + e0);
#pragma unroll
        for (int q = 0; q < EPL / 4; ++q) {
            float4 v = __ldg(row4 + q);
            lg[4 * q] = v.x; lg[4 * q + 1] = v.y; lg[4 * q + 2] = v.z; lg[4 * q + 3] = v.w;
        }
    } else {
#pragma unroll
        for (int q = 0; q < EPL; ++q) lg[q] = (e0 + q < E) ? __ldg(row + e0 + q) : neg_inf;
    }
#pragma unroll
    for (int q = 0; q < EPL; ++q) {
        const int e = e0 + q;
        const bool in_range = e < E;
        float kf;
        if (p.score_func == 0) {
            val[q] = lg[q];
            kf = lg[q];
        } else {
            const float s = sigmoid_spec(lg[q]);
            val[q] = s;
            kf = __fadd_rn(s, in_range ? __ldg(p.bias + e) : 0.0f);
        }
        const bool ok = in_range && (s_nlive[in_range ? e : 0] > 0) && (lg[q] != neg_inf);
        key[q] = ok ? kf : neg_inf;
    }

    // a3 group-limited selection: score = sum of the (up to) group_m best finite keys
    if (p.n_group > 1) {
        float h1 = neg_inf, h2 = neg_inf;
#pragma unroll
        for (int q = 0; q < EPL; ++q) {
            const float v = key[q];
            if (v > h1) { h2 = h1; h1 = v; }
            else if (v > h2) { h2 = v; }
        }
        for (int off = 1; off < p.lanes_per_group; off <<= 1) {
            const float o1 = __shfl_xor_sync(full, h1, off);
            const float o2 = __shfl_xor_sync(full, h2, off);
            const float n1 = fmaxf(h1, o1);
            const float n2 = fmaxf(fminf(h1, o1), fmaxf(h2, o2));
            h1 = n1; h2 = n2;
        }
        const float gscore = (p.group_m == 1 || h2 == neg_inf) ? h1 : __fadd_rn(h1, h2);
        const int g = lane / p.lanes_per_group;
        int rank = 0;
        for (int gp = 0; gp < p.n_group; ++gp) {
            const float o = __shfl_sync(full, gscore, gp * p.lanes_per_group);
            rank += (o > gscore) || (o == gscore && gp < g);
        }
        const bool keep = (g < p.n_group) && (rank < p.topk_group);
        if (!keep) {
#pragma unroll
            for (int q = 0; q < EPL; ++q) key[q] = neg_inf;
        }
    }

    // a4 top-k: k rounds of warp arg-max over order-preserving integer codes
    uint32_t code[EPL];
#pragma unroll
    for (int q = 0; q < EPL; ++q) code[q] = key_code(key[q]);

    uint32_t lbest = 0; int lq = 0; float lval = 0.0f;
#pragma unroll
    for (int q = 0; q < EPL; ++q)
        if (code[q] > lbest) { lbest = code[q]; lq = q; lval = val[q]; }

    int my_id = fallback_expert; float my_val = 0.0f; bool my_bad = false;
    for (int j = 0; j < p.k; ++j) {
        const uint32_t wmax = __reduce_max_sync(full, lbest);
        const unsigned ball = __ballot_sync(full, lbest == wmax);
        const int src = __ffs(ball) - 1;                 // lowest lane = lowest expert id
        const int sel_e = __shfl_sync(full, e0 + lq, src);
        const float sel_v = __shfl_sync(full, lval, src);
        const bool bad = wmax <= kCodeNegInf;            // nothing selectable is left
        if (lane == j) {
            my_id = bad ? fallback_expert : sel_e;
            my_val = sel_v;
            my_bad = bad;
        }
        if (lane == src && !bad) {
#pragma unroll
            for (int q = 0; q < EPL; ++q) if (q == lq) code[q] = 0;
            lbest = 0; lq = 0; lval = 0.0f;
#pragma unroll
            for (int q = 0; q < EPL; ++q)
                if (code[q] > lbest) { lbest = code[q]; lq = q; lval = val[q]; }
        }
    }

    // a5 weights: ratio of the chosen scores, summed and divided in double
    double u = 0.0;
    const float v0 = __shfl_sync(full, my_val, 0);
    if (lane < p.k) {
        if (my_bad) u = 1.0;
        else if (p.score_func == 0) u = exp((double)__fsub_rn(my_val, v0));
        else u = (double)my_val;
    }
    double usum = 0.0;
    for (int j = 0; j < p.k; ++j) usum += __shfl_sync(full, u, j);
    out_w = (float)((double)p.route_scale * u / usum);

    // a6 replica pick: (t mod live count)-th entry of the ascending live list
    out_id = my_id;
    out_slot = -1;
    if (lane < p.k) {
        const int n = s_nlive[my_id];
        out_slot = s_live[my_id * p.max_rep + (t % n)];
    }
    if (__any_sync(full, my_bad) && lane == 0) report_status(p.ctl, kDevInsufficientExperts);
}

template <int EPL>
__global__ void __launch_bounds__(kRouteThreads) k_route(RouteParams p)
{
    extern __shared__ int32_t smem[];
    const int E = p.E, P = p.P, k = p.k, tb = p.tokens_per_block;
    const int NA = tb * k;
    int32_t *s_nlive = smem;                          // [E]
    int32_t *s_live = s_nlive + E;                    // [E][max_rep]
    int32_t *s_slot = s_live + E * p.max_rep;         // [NA] slot of each assignment of the tile
    int32_t *s_lrank = s_slot + NA;                   // [NA] stable rank inside the tile
    int32_t *s_hist = s_lrank + NA;                   // [P]  tile histogram (running)
    int32_t *s_excl = s_hist + P;                     // [P]  assignments on slot p in earlier tiles
    int32_t *s_wcount = s_excl + P;                   // [8][P] per-warp counts of one round
    __shared__ unsigned s_ticket, s_epoch;
    __shared__ int s_warp_sums[kRouteWarps];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned full = 0xffffffffu;

    if (tid == 0) {
        s_epoch = ld_relaxed_u32(&p.ctl->epoch);
        s_ticket = atomicAdd(&p.ctl->ticket, 1u);
    }
    // Live replica lists from the rank bitmap and the replica table (a2, a6).
    const uint32_t *alive = reinterpret_cast<const uint32_t *>(p.state + kStateHeaderWords);
    const int32_t *table = p.state + kStateHeaderWords + p.rank_words;
    for (int e = tid; e < E; e += kRouteThreads) {
        int n = 0;
        for (int r = 0; r < p.max_rep; ++r) {
            const int slot = table[e * p.max_rep + r];
            if (slot >= 0) {
                const int rank = slot / p.S;
                if ((alive[rank >> 5] >> (rank & 31)) & 1u) s_live[e * p.max_rep + n++] = slot;
            }
        }
        s_nlive[e] = n;
    }
    for (int q = tid; q < P; q += kRouteThreads) s_hist[q] = 0;
    for (int q = tid; q < kRouteWarps * P; q += kRouteThreads) s_wcount[q] = 0;
    const int fallback_expert = p.state[0];
    __syncthreads();

    const unsigned ticket = s_ticket;
    const unsigned long long epoch = s_epoch;
    const int t0 = (int)ticket * tb;
    const int n_tok = min(tb, p.T - t0);

    // ---- a1..a6 per token -------------------------------------------------
    for (int lt = warp; lt < tb; lt += kRouteWarps) {
        const int t = t0 + lt;
        int id = 0, slot = -1; float w = 0.0f;
        if (t < p.T) {
            route_token<EPL>(p, t, s_nlive, s_live, fallback_expert, id, w, slot);
            if (lane < k) {
                const size_t i = (size_t)t * k + lane;
                p.topk_ids[i] = id;
                p.topk_weights[i] = w;
                p.topk_slot[i] = slot;
            }
        }
        if (lane < k) s_slot[lt * k + lane] = slot;
    }
    __syncthreads();

    // ---- a7/a9 tile histogram and stable rank inside the tile --------------
    // Rounds of 256 assignments in ascending i; inside a round, match_any gives
    // the rank among equal slots of a warp and per-warp counts order the warps.
    for (int base = 0; base < NA; base += kRouteThreads) {
        const int i = base + tid;
        const int slot = (i < NA) ? s_slot[i] : -1;
        const unsigned peers = __match_any_sync(full, slot);
        const int rank_in_warp = __popc(peers & lanemask_lt());
        if (slot >= 0 && rank_in_warp == 0) s_wcount[warp * P + slot] = __popc(peers);
        __syncthreads();
        if (slot >= 0) {
            int r = s_hist[slot] + rank_in_warp;
            for (int w2 = 0; w2 < warp; ++w2) r += s_wcount[w2 * P + slot];
            s_lrank[i] = r;
        }
        __syncthreads();
        for (int q = tid; q < P; q += kRouteThreads) {
            int tot = 0;
#pragma unroll
            for (int w2 = 0; w2 < kRouteWarps; ++w2) {
                tot += s_wcount[w2 * P + q];
                s_wcount[w2 * P + q] = 0;
            }
            s_hist[q] += tot;
        }
        __syncthreads();
    }

    // ---- a8 decoupled look-back over tiles, one thread per slot ------------
    const bool last_tile = (ticket == gridDim.x - 1);
    for (int q = tid; q < P; q += kRouteThreads) {
        const unsigned long long mine = (unsigned long long)(unsigned)s_hist[q];
        unsigned long long *d = p.desc + (size_t)ticket * P + q;
        unsigned long long excl = 0;
        if (ticket == 0) {
            st_relaxed_u64(d, (epoch << 32) | (kFlagInclusive << 30) | mine);
        } else {
            st_relaxed_u64(d, (epoch << 32) | (kFlagAggregate << 30) | mine);
            int b = (int)ticket - 1;
            unsigned spins = 0;
            bool gave_up = false;
            while (true) {
                const unsigned long long v = ld_relaxed_u64(p.desc + (size_t)b * P + q);
                if ((v >> 32) != epoch) {                       // predecessor not there yet
                    if (++spins > kSpinLimit ||
                        ((spins & 1023u) == 0 && ld_relaxed_s32(&p.ctl->status) == kDevTimeout)) {
                        gave_up = true;
                        break;
                    }
                    __nanosleep(kSpinSleepNs);
                    continue;
                }
                excl += v & 0x3FFFFFFFull;
                if (((v >> 30) & 3ull) == kFlagInclusive || b == 0) break;
                --b;
            }
            if (gave_up) report_status(p.ctl, kDevTimeout);
            st_relaxed_u64(d, (epoch << 32) | (kFlagInclusive << 30) | ((excl + mine) & 0x3FFFFFFFull));
        }
        s_excl[q] = (int)excl;
    }
    __syncthreads();

    // stable rank of every assignment of the tile inside its slot, over all tiles
    for (int i = tid; i < n_tok * k; i += kRouteThreads)
        p.pos_in_slot[(size_t)t0 * k + i] = s_excl[s_slot[i]] + s_lrank[i];

    if (!last_tile) return;

    // ---- the last tile knows every total: a7 counts, a8 offsets -----------
    // exclusive scan over P with a contiguous chunk per thread
    const int chunk = (P + kRouteThreads - 1) / kRouteThreads;
    const int q0 = tid * chunk;
    int local = 0;
    for (int q = q0; q < min(P, q0 + chunk); ++q) {
        const int tot = s_excl[q] + s_hist[q];
        s_hist[q] = tot;
        local += tot;
    }
    int incl = local;
    for (int off = 1; off < 32; off <<= 1) {
        const int o = __shfl_up_sync(full, incl, off);
        if (lane >= off) incl += o;
    }
    if (lane == 31) s_warp_sums[warp] = incl;
    __syncthreads();
    int warp_base = 0;
    for (int w2 = 0; w2 < warp; ++w2) warp_base += s_warp_sums[w2];
    int run = warp_base + incl - local;
    __syncthreads();                                   // s_excl is about to be overwritten
    for (int q = q0; q < min(P, q0 + chunk); ++q) {
        const int tot = s_hist[q];
        p.slot_counts[q] = tot;
        p.slot_offsets[q] = run;
        s_excl[q] = run;
        run += tot;
    }
    if (tid == kRouteThreads - 1) {
        p.slot_offsets[P] = run;
        p.rank_offsets[p.R] = run;
    }
    __syncthreads();
    for (int r = tid; r < p.R; r += kRouteThreads) {
        int c = 0;
        for (int s = 0; s < p.S; ++s) c += s_hist[r * p.S + s];
        p.rank_counts[r] = c;
        p.rank_offsets[r] = s_excl[r * p.S];
    }
    // every ticket of this step has been taken and every tile has read the
    // epoch (it published before this tile could finish): arm the next step
    if (tid == 0) {
        p.ctl->ticket = 0;
        unsigned next = (unsigned)epoch + 1u;
        p.ctl->epoch = next ? next : 1u;
    }
}

}  // namespace moe
