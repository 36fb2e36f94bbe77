/*
 * CPU oracle for failure-aware MoE routing with dispatch and combine.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, single-threaded, plainly
 * written definition that the CUDA library is checked against.  It shares no
 * code, header, table or helper with the CUDA path and must never be called
 * from it.  Compile with:  gcc -O2 -ffp-contract=off -shared -fPIC
 * (contraction must stay off: every fp32 operation below is one IEEE-754
 * round-to-nearest-even operation, which is what makes expert selection
 * reproducible bit for bit on another machine).
 *
 * What the paper fixes (ReviveMoE):
 *   - Sec. 2.1: a gating function scores the experts per token and the token
 *     goes to its top-k experts.
 *   - Sec. 2.3: dispatch routes tokens to those experts; combine aggregates
 *     the experts' outputs back using the gating scores.
 *   - Sec. 3.4 "Redundant experts": on a failure, the failed replicas are
 *     taken out of the logical-to-physical map and nothing else changes.
 *   - Sec. 3.4 "Missing experts" and Sec. 4.2: an expert without a surviving
 *     copy has its routing logit set to minus infinity right before top-k,
 *     so the next-best expert takes its place.
 * Everything the paper leaves open (score function details, group-limited
 * selection, tie-breaks, replica choice, buffer order) follows the readings
 * listed in the project's design notes; each function names the reading it
 * implements.
 *
 * Pins: every function here is pinned by tests that do not call it to
 * produce their expected values (brute-force subset enumeration, numpy
 * bincount / cumsum / stable argsort, torch softmax + topk, libm exp, the
 * closed form y = c_t * x, a hand-worked example).  The replica policy
 * (token index modulo live-replica count) and the redundant-slot placement
 * recipe have no counterpart in the paper: "parity unpinned" against the
 * paper for those two, pinned only against their written definition.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int32_t num_experts;    /* E  logical experts                                  */
    int32_t top_k;          /* k                                                   */
    int32_t num_ranks;      /* R  simulated EP ranks                               */
    int32_t slots_per_rank; /* S  physical slots per rank; slot p lives on p / S   */
    int32_t score_func;     /* 0 softmax, 1 sigmoid (+ bias on the key), 2 dense TP groups */
    int32_t n_group;        /* 1 = no group-limited selection                      */
    int32_t topk_group;     /* groups kept when n_group > 1                        */
    float   route_scale;    /* multiplies the renormalised weights                 */
} oracle_cfg;

/* ------------------------------------------------------------------------ */
/* exp and sigmoid built from single IEEE fp32 operations                    */
/* ------------------------------------------------------------------------ */

/*
 * exp_spec(z): clamp z to [-87, 88]; n = round-half-even(z * log2(e));
 * r = z - n*ln2 with ln2 split in two fp32 parts and two fused
 * multiply-adds; degree-7 Taylor polynomial of e^r by Horner's rule with
 * fused multiply-adds (coefficients are 1/j! rounded to fp32); multiply by
 * 2^n, the power of two built from its exponent field.  Not in the paper:
 * it exists so that sigmoid routing keys are the same bits on CPU and GPU.
 */
float oracle_exp_spec(float z)
{
    const float log2e  = 0x1.715476p+0f;
    const float ln2_hi = 0x1.62e430p-1f;
    const float ln2_lo = -0x1.05c610p-29f;
    if (z < -87.0f) z = -87.0f;
    if (z > 88.0f) z = 88.0f;
    float n = rintf(z * log2e);
    float r = fmaf(-n, ln2_hi, z);
    r = fmaf(-n, ln2_lo, r);
    float p = 0x1.a01a02p-13f;          /* 1/5040 */
    p = fmaf(p, r, 0x1.6c16c2p-10f);    /* 1/720  */
    p = fmaf(p, r, 0x1.111112p-7f);     /* 1/120  */
    p = fmaf(p, r, 0x1.555556p-5f);     /* 1/24   */
    p = fmaf(p, r, 0x1.555556p-3f);     /* 1/6    */
    p = fmaf(p, r, 0.5f);
    p = fmaf(p, r, 1.0f);
    p = fmaf(p, r, 1.0f);
    union { uint32_t u; float f; } two_n;
    two_n.u = (uint32_t)((int32_t)n + 127) << 23;   /* n in [-126, 127] */
    return p * two_n.f;
}

/* sigmoid_spec(x) = 1 / (1 + exp_spec(-x)), one fp32 add and one fp32 divide. */
float oracle_sigmoid_spec(float x)
{
    float e = oracle_exp_spec(-x);
    float d = 1.0f + e;
    return 1.0f / d;
}

/* Array forms for dense sweeps in the tests. */
void oracle_exp_spec_array(const float *z, float *out, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) out[i] = oracle_exp_spec(z[i]);
}

void oracle_sigmoid_spec_array(const float *x, float *out, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) out[i] = oracle_sigmoid_spec(x[i]);
}

/* ------------------------------------------------------------------------ */
/* bf16 helpers (storage type uint16_t)                                       */
/* ------------------------------------------------------------------------ */

static double bf16_to_double(uint16_t b)
{
    union { uint32_t u; float f; } v;
    v.u = (uint32_t)b << 16;
    return (double)v.f;
}

/* Round a double to the nearest bf16 (8 significant bits), ties to even,
 * in one rounding (not through fp32, which could round twice). */
uint16_t oracle_double_to_bf16(double d)
{
    union { uint32_t u; float f; } v;
    if (isnan(d)) return 0x7fc0;
    if (d == 0.0) return signbit(d) ? 0x8000 : 0x0000;
    if (isinf(d)) return signbit(d) ? 0xff80 : 0x7f80;
    int e;
    double m = frexp(d, &e);            /* d = m * 2^e, 0.5 <= |m| < 1 */
    int bits = 8;                        /* significant bits of a normal bf16 */
    if (e - 1 < -126) bits -= (-126 - (e - 1));   /* subnormal range */
    double q;
    if (bits <= 0) {
        /* below half of the smallest subnormal, or exactly in between */
        q = (bits == 0) ? nearbyint(m) : 0.0;     /* |m| in [0.5,1): tie at 0.5 -> 0 */
        bits = 0;
    } else {
        q = nearbyint(ldexp(m, bits));   /* default rounding mode = ties to even */
    }
    double r = copysign(ldexp(q, e - bits), d);
    v.f = (float)r;                      /* exact: r has <= 8 significant bits */
    if (isinf(v.f)) return signbit(d) ? 0xff80 : 0x7f80;
    return (uint16_t)(v.u >> 16);
}

/* ------------------------------------------------------------------------ */
/* Step 1: routing state from the failure set (Sec. 3.4)                      */
/* ------------------------------------------------------------------------ */

/*
 * live[e*P .. e*P + n_live[e]) = slots p, ascending, with
 * slot_to_expert[p] == e whose rank p / S is not failed.  An expert is
 * available iff n_live[e] > 0: "Redundant experts" removes failed replicas
 * from the map, "Missing experts" masks an expert with none left.  An expert
 * flagged in expert_failed (may be NULL) is lost whatever its replicas: the
 * accuracy experiment of Sec. 4.2 fails experts one by one this way.
 */
static void derive_live(const oracle_cfg *c, const int32_t *slot_to_expert,
                        const uint8_t *rank_failed, const uint8_t *expert_failed,
                        int32_t *live, int32_t *n_live)
{
    const int P = c->num_ranks * c->slots_per_rank;
    for (int e = 0; e < c->num_experts; ++e) n_live[e] = 0;
    for (int p = 0; p < P; ++p) {
        int e = slot_to_expert[p];
        if (e < 0) continue;                        /* empty slot */
        if (rank_failed[p / c->slots_per_rank]) continue;
        if (expert_failed && expert_failed[e]) continue;    /* expert lost on its own (Sec. 4.2) */
        live[(size_t)e * P + n_live[e]++] = p;
    }
}

/*
 * Can top-k fail for some logits under this failure set?  Returns 1 when
 * routing is always well defined, 0 when the remap must be rejected.
 * Ungrouped: at least k available experts.  Grouped: empty groups score
 * minus infinity and are only kept when fewer than topk_group groups are
 * non-empty, so the worst case keeps the topk_group non-empty groups with
 * the fewest available experts (all non-empty groups if there are fewer).
 */
int32_t oracle_failure_set_ok(const oracle_cfg *c, const int32_t *slot_to_expert,
                              const uint8_t *rank_failed, const uint8_t *expert_failed)
{
    const int E = c->num_experts, P = c->num_ranks * c->slots_per_rank;
    int32_t *live = malloc((size_t)E * P * sizeof(int32_t));
    int32_t *n_live = malloc((size_t)E * sizeof(int32_t));
    derive_live(c, slot_to_expert, rank_failed, expert_failed, live, n_live);
    int ok;
    if (c->score_func == 2) {                            /* dense: some group keeps all its shards */
        ok = 0;
        for (int g = 0; g < E / c->top_k; ++g) {
            int all = 1;
            for (int s = 0; s < c->top_k; ++s) all = all && n_live[g * c->top_k + s] > 0;
            ok = ok || all;
        }
    } else if (c->n_group <= 1) {
        int avail = 0;
        for (int e = 0; e < E; ++e) avail += n_live[e] > 0;
        ok = avail >= c->top_k;
    } else {
        const int G = c->n_group, per = E / G;
        int *cnt = malloc((size_t)G * sizeof(int));
        int n_nonempty = 0;
        for (int g = 0; g < G; ++g) {
            int a = 0;
            for (int e = g * per; e < (g + 1) * per; ++e) a += n_live[e] > 0;
            if (a > 0) cnt[n_nonempty++] = a;
        }
        /* ascending insertion sort of the non-empty counts */
        for (int i = 1; i < n_nonempty; ++i) {
            int v = cnt[i], j = i - 1;
            while (j >= 0 && cnt[j] > v) { cnt[j + 1] = cnt[j]; --j; }
            cnt[j + 1] = v;
        }
        int take = n_nonempty < c->topk_group ? n_nonempty : c->topk_group;
        int worst = 0;
        for (int i = 0; i < take; ++i) worst += cnt[i];
        ok = worst >= c->top_k;
        free(cnt);
    }
    free(live); free(n_live);
    return ok;
}

/* ------------------------------------------------------------------------ */
/* Steps 2-6: gate, mask, groups, top-k, weights, replica  (Sec. 2.1, 3.4)    */
/* ------------------------------------------------------------------------ */

/*
 * Per token t:
 *  key[e]   = logit (softmax mode; softmax is monotone so selection needs no
 *             exp) or sigmoid_spec(logit) + bias[e] (sigmoid mode, one fp32
 *             add; the bias enters the key only, never the weight).
 *  mask     : unavailable expert -> key = -inf, right before selection; a
 *             logit that is already -inf gives key = -inf in both modes.
 *  groups   : n_group > 1: experts split in n_group equal consecutive
 *             groups; group score = fp32 sum, larger first, of the
 *             min(m, #finite) largest keys in it, m = k / topk_group; a
 *             group with no finite key scores -inf; keep the topk_group best
 *             groups (ties: lower group); keys elsewhere -> -inf.
 *  top-k    : k times argmax over unpicked experts, ties -> lower id.
 *  weights  : u_j = exp(logit_j - logit_0) (softmax; fp32 subtract, exp in
 *             double) or sigmoid_spec(logit_j) (sigmoid, no bias);
 *             w_j = route_scale * u_j / sum_j u_j in double, rounded to fp32.
 *  replica  : slot = live[e][t mod n_live[e]].
 * Returns 0, or -1 if some token finds fewer than k finite keys.
 */
int32_t oracle_route(const oracle_cfg *c, const int32_t *slot_to_expert,
                     const uint8_t *rank_failed, const uint8_t *expert_failed, const float *bias,
                     const float *logits, int32_t T,
                     int32_t *topk_ids, float *topk_weights, int32_t *topk_slot)
{
    const int E = c->num_experts, k = c->top_k;
    const int P = c->num_ranks * c->slots_per_rank;
    int32_t *live = malloc((size_t)E * P * sizeof(int32_t));
    int32_t *n_live = malloc((size_t)E * sizeof(int32_t));
    float *score = malloc((size_t)E * sizeof(float));
    float *key = malloc((size_t)E * sizeof(float));
    uint8_t *picked = malloc((size_t)E);
    int rc = 0;
    derive_live(c, slot_to_expert, rank_failed, expert_failed, live, n_live);

    if (c->score_func == 2) {
        /* Dense FFN layers (Sec. 3.4): the E "experts" are the k tensor-parallel shards of
         * E/k replicated FFN groups.  A group that lost any shard is compromised; tokens are
         * spread evenly over the healthy groups: token t goes to every shard of the
         * (t mod n_healthy)-th healthy group, each with weight route_scale (the shards'
         * partial results add up in combine). */
        const int G = E / k;
        int *healthy = malloc((size_t)G * sizeof(int));
        int n_healthy = 0;
        for (int g = 0; g < G; ++g) {
            int all = 1;
            for (int s = 0; s < k; ++s) all = all && n_live[g * k + s] > 0;
            if (all) healthy[n_healthy++] = g;
        }
        if (n_healthy == 0) rc = -1;
        for (int t = 0; t < T && rc == 0; ++t) {
            const int g = healthy[t % n_healthy];
            for (int j = 0; j < k; ++j) {
                const int e = g * k + j;
                topk_ids[(size_t)t * k + j] = e;
                topk_weights[(size_t)t * k + j] = c->route_scale;
                topk_slot[(size_t)t * k + j] = live[(size_t)e * P + (t % n_live[e])];
            }
        }
        free(healthy);
        T = 0;                                           /* nothing left for the gated path */
    }
    for (int t = 0; t < T && rc == 0; ++t) {
        const float *lg = logits + (size_t)t * E;
        for (int e = 0; e < E; ++e) {
            if (c->score_func == 0) {
                score[e] = lg[e];
                key[e] = lg[e];
            } else {
                score[e] = oracle_sigmoid_spec(lg[e]);
                key[e] = score[e] + (bias ? bias[e] : 0.0f);
            }
            if (n_live[e] == 0) key[e] = -INFINITY;
            if (lg[e] == -INFINITY) key[e] = -INFINITY;   /* a -inf logit acts as a mask in both modes */
        }

        if (c->n_group > 1) {
            const int G = c->n_group, per = E / G, m = k / c->topk_group;
            float gscore[G];
            uint8_t keep[G];
            for (int g = 0; g < G; ++g) {
                memset(picked, 0, (size_t)E);
                float sum = -INFINITY;
                for (int i = 0; i < m; ++i) {
                    int best = -1;
                    for (int e = g * per; e < (g + 1) * per; ++e) {
                        if (picked[e] || key[e] == -INFINITY) continue;
                        if (best < 0 || key[e] > key[best]) best = e;
                    }
                    if (best < 0) break;
                    picked[best] = 1;
                    sum = (i == 0) ? key[best] : sum + key[best];
                }
                gscore[g] = sum;
                keep[g] = 0;
            }
            for (int i = 0; i < c->topk_group; ++i) {
                int best = -1;
                for (int g = 0; g < G; ++g) {
                    if (keep[g]) continue;
                    if (best < 0 || gscore[g] > gscore[best]) best = g;
                }
                keep[best] = 1;
            }
            for (int e = 0; e < E; ++e)
                if (!keep[e / per]) key[e] = -INFINITY;
        }

        memset(picked, 0, (size_t)E);
        int32_t *ids = topk_ids + (size_t)t * k;
        for (int j = 0; j < k; ++j) {
            int best = -1;
            for (int e = 0; e < E; ++e) {
                if (picked[e] || key[e] == -INFINITY) continue;
                if (best < 0 || key[e] > key[best]) best = e;
            }
            if (best < 0) { rc = -1; break; }
            picked[best] = 1;
            ids[j] = best;
        }
        if (rc) break;

        double u[k], usum = 0.0;
        for (int j = 0; j < k; ++j) {
            if (c->score_func == 0) {
                float d = lg[ids[j]] - lg[ids[0]];
                u[j] = exp((double)d);
            } else {
                u[j] = (double)score[ids[j]];
            }
            usum += u[j];
        }
        for (int j = 0; j < k; ++j) {
            topk_weights[(size_t)t * k + j] = (float)((double)c->route_scale * u[j] / usum);
            int e = ids[j];
            topk_slot[(size_t)t * k + j] = live[(size_t)e * P + (t % n_live[e])];
        }
    }
    free(live); free(n_live); free(score); free(key); free(picked);
    return rc;
}

/* ------------------------------------------------------------------------ */
/* Steps 7-8: counts, offsets, stable permutation                             */
/* ------------------------------------------------------------------------ */

/*
 * slot_counts[p] = number of assignments i (i = t*k + j) with slot_i == p.
 * The send buffer lists the ranks in `rank_order` (physical rank at each logical
 * position, a permutation of 0..R-1; NULL = identity): Sec. 3.5 rebuilds the
 * communication domain with compacted logical ranks, so the layout follows the
 * logical numbering.  Walking the slots in that order (rank by rank, the S
 * slots of a rank ascending), slot_offsets[p] = rows before slot p, and
 * slot_offsets[P] = T*k.  rank_counts[l] / rank_offsets[l] belong to the l-th
 * rank of the order, rank_offsets[R] = T*k.  Walking i upward,
 * dst_row[i] = slot_offsets[p] + (assignments seen so far on p), so the rows
 * of one slot keep ascending i; src_index is the inverse permutation.
 * A failed rank receives no assignment, hence owns no rows.
 */
void oracle_permutation(const oracle_cfg *c, const int32_t *topk_slot, int32_t T,
                        const int32_t *rank_order,
                        int32_t *slot_counts, int32_t *slot_offsets,
                        int32_t *rank_counts, int32_t *rank_offsets,
                        int32_t *dst_row, int32_t *src_index)
{
    const int S = c->slots_per_rank, R = c->num_ranks, P = R * S;
    const int64_t n = (int64_t)T * c->top_k;
    for (int p = 0; p < P; ++p) slot_counts[p] = 0;
    for (int64_t i = 0; i < n; ++i) slot_counts[topk_slot[i]]++;
    int32_t run = 0;
    for (int l = 0; l < R; ++l) {
        const int r = rank_order ? rank_order[l] : l;
        rank_offsets[l] = run;
        rank_counts[l] = 0;
        for (int s = 0; s < S; ++s) {
            const int p = r * S + s;
            slot_offsets[p] = run;
            run += slot_counts[p];
            rank_counts[l] += slot_counts[p];
        }
    }
    slot_offsets[P] = run;
    rank_offsets[R] = run;
    int32_t *seen = calloc((size_t)P, sizeof(int32_t));
    for (int64_t i = 0; i < n; ++i) {
        int p = topk_slot[i];
        dst_row[i] = slot_offsets[p] + seen[p]++;
        src_index[dst_row[i]] = (int32_t)i;
    }
    free(seen);
}

/*
 * Logical-rank reassignment of Sec. 3.5.  Ranks are named by their original
 * logical rank.  A failed rank leaves a gap and every later rank moves down by
 * one; with a role switch the switched rank first takes the place of the failed
 * rank it replaces, and the place it vacates closes like any other gap.
 * Returns the number of logical ranks written to order[].
 */
int32_t oracle_compact_ranks(int32_t R, const uint8_t *rank_failed, int32_t switched_rank,
                             int32_t replaced_rank, int32_t *order)
{
    int32_t *cur = malloc((size_t)R * sizeof(int32_t));
    int n = R;
    for (int r = 0; r < R; ++r) cur[r] = r;
    if (switched_rank >= 0) {
        for (int i = 0; i < n; ++i) if (cur[i] == replaced_rank) cur[i] = switched_rank;   /* C takes l_A */
        int seen = 0;
        for (int i = 0; i < n; ++i) {                    /* the position C left is a gap: close it */
            if (cur[i] == switched_rank && i != replaced_rank) { seen = 1; continue; }
            cur[i - seen] = cur[i];
        }
        n -= seen;
    }
    int m = 0;
    for (int i = 0; i < n; ++i) {                        /* close the gaps of the (other) failed ranks */
        if (cur[i] != switched_rank && rank_failed[cur[i]]) continue;
        order[m++] = cur[i];
    }
    free(cur);
    return m;
}

/* ------------------------------------------------------------------------ */
/* Step 9: dispatch scatter into the A2E layout (Sec. 2.3)                    */
/* ------------------------------------------------------------------------ */

/* send[dst_row[i], :] = x[i / k, :], a bit copy of bf16 rows of width H. */
void oracle_scatter(const uint16_t *x, const int32_t *dst_row, int32_t T, int32_t k,
                    int32_t H, uint16_t *send)
{
    for (int64_t i = 0; i < (int64_t)T * k; ++i)
        memcpy(send + (size_t)dst_row[i] * H, x + (size_t)(i / k) * H, (size_t)H * 2);
}

/* ------------------------------------------------------------------------ */
/* Step 10: combine, the weighted gather-reduce back to token order (E2A)     */
/* ------------------------------------------------------------------------ */

/*
 * y[t,h] = bf16( sum_j (w[t,j] * slot_scale[slot[t,j]]) * buf[dst_row[t*k+j], h] ).
 * The per-slot scalar stands in for the expert FFN.  The coefficient is one
 * fp32 product (as the weights and scales are fp32 data); the sum over j is
 * taken in double in ascending j and rounded once to bf16.
 */
void oracle_combine(const uint16_t *buf, const int32_t *dst_row, const float *topk_weights,
                    const int32_t *topk_slot, const float *slot_scale,
                    int32_t T, int32_t k, int32_t H, uint16_t *y)
{
    for (int t = 0; t < T; ++t) {
        for (int h = 0; h < H; ++h) {
            double acc = 0.0;
            for (int j = 0; j < k; ++j) {
                size_t i = (size_t)t * k + j;
                float coef = topk_weights[i] * slot_scale[topk_slot[i]];
                acc += (double)coef * bf16_to_double(buf[(size_t)dst_row[i] * H + h]);
            }
            y[(size_t)t * H + h] = oracle_double_to_bf16(acc);
        }
    }
}
