/*
 * moe_route.h — C ABI of the failure-aware MoE routing library for B200 (sm_100a).
 *
 * The library implements the per-layer hot path that ReviveMoE's
 * instance-preserving recovery rewires: gate -> availability mask -> top-k ->
 * weight renormalisation -> live-replica pick -> per-slot count and prefix
 * scan -> stable permutation -> scatter of bf16 hidden states into an
 * expert-contiguous send buffer (dispatch / A2E layout), and the weighted
 * gather-reduce back to token order (combine / E2A).  Recovery is a host call
 * that rewrites only a rank-alive bitmap and a logical-to-physical replica
 * table held in device memory; kernels read both through pointers, so a CUDA
 * graph captured over moe_dispatch + moe_combine stays valid after a failure.
 *
 * Conventions
 *   - Every function returns a moe_status; no exception crosses this boundary.
 *   - "host" pointers are ordinary CPU memory and are copied before return.
 *     "device" pointers are CUDA device memory owned by the caller, on the
 *     device that was current at moe_route_init.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = default stream).
 *   - The context owns only small state: the routing tables, bias, per-slot
 *     scales, scan scratch sized from max_tokens, and pinned staging buffers.
 *   - moe_dispatch and moe_combine allocate nothing, never synchronise and
 *     never read device memory from the host: they may be captured in a graph.
 *   - Simulated EP ranks: slot p (0 <= p < P = num_ranks*slots_per_rank) lives
 *     on rank p / slots_per_rank; the send buffer is one allocation in which
 *     rank r owns rows [rank_offsets[r], rank_offsets[r+1]).
 *   - A context is not thread-safe; serialise calls on it.
 */
#ifndef MOE_ROUTE_H
#define MOE_ROUTE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct moe_ctx moe_ctx;

typedef enum {
    MOE_OK = 0,
    MOE_ERR_INVALID_ARG = 1,          /* bad size, NULL, misaligned pointer, unsupported shape     */
    MOE_ERR_CUDA = 2,                 /* a CUDA runtime call failed (no device, out of memory...) */
    MOE_ERR_INSUFFICIENT_EXPERTS = 3, /* the failure set could leave a token without k experts     */
    MOE_ERR_CAPACITY = 4,             /* T > max_tokens, or an expert has more than max_replicas   */
    MOE_ERR_DEVICE_TIMEOUT = 5        /* a bounded device-side wait gave up (see get_device_status) */
} moe_status;

/* score_func values.  MOE_ROUTE_DENSE_TP is the routing of the dense FFN layers of
 * Sec. 3.4: num_experts = groups * top_k names the top_k tensor-parallel shards
 * (expert g*top_k + s = shard s of FFN group g) of replicated FFN groups; a group
 * with any shard lost is compromised and skipped, token t goes to all shards of
 * the (t mod n_healthy)-th healthy group with weight route_scale, so tokens are
 * spread evenly over the healthy groups.  Logits are not read in this mode (the
 * pointer may be NULL); n_group must be 1 and groups <= 32 * top_k. */
enum { MOE_SCORE_SOFTMAX = 0, MOE_SCORE_SIGMOID = 1, MOE_ROUTE_DENSE_TP = 2 };

/* Limits of this library: num_experts <= 512, top_k <= 16, max_replicas <= 8,
 * num_ranks*slots_per_rank <= 4096 (and small enough for the routing kernel's
 * shared-memory tables, about 2000 slots at 512 experts), max_tokens <= 262144,
 * max_tokens*top_k < 2^30, hidden % 8 == 0.  With n_group > 1:
 * num_experts % n_group == 0, top_k % topk_group == 0, top_k/topk_group in
 * {1, 2}, and the experts of a group must map onto a power-of-two run of lanes
 * (any group size that is a power of two, or a multiple of one of
 * 1,2,3,4,5,6,8,10,12,16,20,24,32 by a power of two, qualifies).  A shape outside
 * these limits makes moe_route_init return MOE_ERR_INVALID_ARG. */
typedef struct {
    int32_t num_experts;    /* E: logical experts                                            */
    int32_t top_k;          /* k: experts per token                                          */
    int32_t hidden;         /* H: bf16 elements per token row                                */
    int32_t max_tokens;     /* largest T a dispatch may carry (sizes the scan scratch)       */
    int32_t num_ranks;      /* R: simulated EP ranks                                         */
    int32_t slots_per_rank; /* S: physical expert slots per rank                             */
    int32_t max_replicas;   /* most physical copies any logical expert may have              */
    int32_t score_func;     /* MOE_SCORE_SOFTMAX | MOE_SCORE_SIGMOID (+ bias on the key) | MOE_ROUTE_DENSE_TP */
    int32_t n_group;        /* 1 = plain top-k; > 1 = group-limited selection                */
    int32_t topk_group;     /* groups kept when n_group > 1                                  */
    int32_t replica_policy; /* 0 = replica (t mod live count) of the ascending live list     */
    float   route_scale;    /* multiplies the renormalised weights (1.0 = weights sum to 1)  */
} moe_config;

/* Device output pointers of one dispatch.  With n = T*k:
 *   topk_ids     [T,k] i32  chosen logical experts, best first
 *   topk_weights [T,k] f32  renormalised gate weights
 *   topk_slot    [T,k] i32  physical slot serving (t, j)
 *   slot_counts  [P]   i32  assignments per slot
 *   slot_offsets [P+1] i32  exclusive prefix of slot_counts, [P] = n
 *   rank_counts  [R]   i32  assignments per rank (0 for a failed rank)
 *   rank_offsets [R+1] i32  first send-buffer row of each rank, [R] = n
 *   dst_row      [n]   i32  send-buffer row of assignment i = t*k + j
 *   src_index    [n]   i32  inverse of dst_row
 *   send_buf     [n,H] bf16 row dst_row[i] holds a bit copy of x[i / k]
 * Rows of one slot keep ascending i (stable).  All pointers must be non-NULL;
 * send_buf must be 16-byte aligned. */
typedef struct {
    int32_t *topk_ids;
    float   *topk_weights;
    int32_t *topk_slot;
    int32_t *slot_counts;
    int32_t *slot_offsets;
    int32_t *rank_counts;
    int32_t *rank_offsets;
    int32_t *dst_row;
    int32_t *src_index;
    void    *send_buf;
} moe_dispatch_out;

/*
 * moe_route_init — create a context on the current device.
 * Sets up the routing state of Sec. 3.4: the logical-to-physical map
 * ("which device each replica resides on") and an all-alive rank bitmap.
 *   slot_to_expert host [P]: logical expert hosted by each physical slot, -1 = empty.
 *   bias           host [E] or NULL: added to the selection key in sigmoid mode only.
 *   slot_scale     host [P]: per-slot scalar standing in for the expert FFN in combine.
 * Returns INVALID_ARG for unsupported shapes, CAPACITY if an expert exceeds
 * max_replicas, INSUFFICIENT_EXPERTS if fewer than k experts are placed,
 * CUDA if allocation fails.  *out is written only on success.
 */
moe_status moe_route_init(const moe_config *cfg, const int32_t *slot_to_expert,
                          const float *bias, const float *slot_scale,
                          void *cuda_stream, moe_ctx **out);

/*
 * moe_set_failed_ranks — recovery after device failures (Sec. 3.4, Sec. 4.1
 * "update to the gating mechanism").  `ranks` host [n] is the ABSOLUTE set of
 * failed ranks (duplicates allowed, n = 0 revives everything).  An expert
 * whose every replica sits on a failed rank is masked before top-k ("Missing
 * experts"); an expert with a surviving replica only stops using the failed
 * copies ("Redundant experts").  Validates on the host; on any error the
 * device state is untouched.  The new state is copied with one small
 * stream-ordered transfer, so it takes effect between steps enqueued on
 * `cuda_stream`; no graph needs recapturing.  Must not be called while the
 * stream is capturing (INVALID_ARG).
 */
moe_status moe_set_failed_ranks(moe_ctx *ctx, const int32_t *ranks, int32_t n, void *cuda_stream);

/*
 * moe_update_replica_map — replace the logical-to-physical map (Sec. 3.4:
 * removing failed replicas from the map, or placing new ones).  Same
 * validation, ordering and capture rules as moe_set_failed_ranks; the
 * failed-rank set is kept.
 */
moe_status moe_update_replica_map(moe_ctx *ctx, const int32_t *slot_to_expert, void *cuda_stream);

/*
 * moe_set_failed_experts — mark logical experts as lost one by one (Sec. 4.2:
 * "selectively failing a fraction of the experts", their routing logits masked
 * to minus infinity right before top-k), on top of whatever the failed-rank set
 * already removes.  `mask` host [num_experts] u8, non-zero = lost; n must be
 * num_experts, or 0 to clear the mask.  ABSOLUTE like moe_set_failed_ranks,
 * same validation (INSUFFICIENT_EXPERTS if some token could be left with fewer
 * than k experts), ordering and capture rules.
 */
moe_status moe_set_failed_experts(moe_ctx *ctx, const uint8_t *mask, int32_t n, void *cuda_stream);

/*
 * moe_compact_ranks — host only, no CUDA call: the logical-rank reassignment of
 * Sec. 3.5.  When a device with logical rank l_A fails it leaves a gap; the
 * device at l_A + 1 takes l_A and every later one moves down by one.  With a
 * role switch, the switched device (`switched_rank`, alive) takes the logical
 * rank of the failed device it replaces (`replaced_rank`, failed) and the gap
 * it leaves behind is closed the same way; pass -1, -1 for no role switch.
 * Ranks are numbered by their original logical rank 0..num_ranks-1.
 * Writes the physical (original) rank at each new logical rank to
 * logical_to_physical[0 .. *n_logical), which must have room for num_ranks.
 */
moe_status moe_compact_ranks(int32_t num_ranks, const int32_t *failed_ranks, int32_t n_failed,
                             int32_t switched_rank, int32_t replaced_rank,
                             int32_t *logical_to_physical, int32_t *n_logical);

/*
 * moe_set_rank_order — lay the send buffer out in logical-rank order (Sec. 3.5:
 * the communication domain is rebuilt with compacted ranks).
 * logical_to_physical host [n] lists distinct physical ranks; the send buffer
 * then holds the rows of rank logical_to_physical[0] first, and so on.  Every
 * rank that is not failed must be listed (INVALID_ARG otherwise, also from a
 * later moe_set_failed_ranks that would revive an unlisted rank); unlisted
 * ranks own no rows.  n = 0 restores the physical numbering.  After this call
 * rank_counts[l] and rank_offsets[l] of moe_dispatch_out refer to the l-th
 * rank of the order, slot_counts / slot_offsets stay indexed by physical slot
 * (slot_offsets is then no longer monotone in the slot id).  Same ordering and
 * capture rules as moe_set_failed_ranks.
 */
moe_status moe_set_rank_order(moe_ctx *ctx, const int32_t *logical_to_physical, int32_t n,
                              void *cuda_stream);

/*
 * moe_dispatch — gate, mask, select, count, scan, permute and scatter
 * (Sec. 2.1 gating and top-k; Sec. 2.3 dispatch / attention2expert).
 *   logits device [T,E] f32 row-major (finite; -inf acts as a mask)
 *   x      device [T,H] bf16 row-major, 16-byte aligned
 *   out    host struct of device pointers (see moe_dispatch_out)
 * T = 0 succeeds and launches nothing.  CAPACITY if T > max_tokens.
 */
moe_status moe_dispatch(moe_ctx *ctx, const float *logits, const void *x, int32_t T,
                        const moe_dispatch_out *out, void *cuda_stream);

/*
 * moe_combine — weighted gather-reduce back to token order (Sec. 2.3
 * combine / expert2attention):
 *   y[t,:] = bf16( sum_j (w[t,j] * slot_scale[slot[t,j]]) * expert_buf[dst_row[t*k+j], :] )
 * with fp32 accumulation in ascending j and one rounding.  Uses the
 * topk_weights / topk_slot / dst_row buffers of the latest moe_dispatch on
 * this context (their pointers are remembered; the buffers stay the caller's).
 *   expert_buf device [T*k,H] bf16 in send-buffer row order, 16-byte aligned
 *   y          device [T,H]   bf16, 16-byte aligned
 * INVALID_ARG if no dispatch preceded it or T differs from that dispatch.
 */
moe_status moe_combine(moe_ctx *ctx, const void *expert_buf, int32_t T, void *y, void *cuda_stream);

/*
 * ---- Expert parallelism over several GPUs -----------------------------------
 * Sec. 2.3: "dispatch" routes tokens to their experts and "combine" brings the expert
 * outputs back; between real devices both are all-to-all exchanges (attention2expert /
 * expert2attention).  Here the exchange is part of the kernels: the scatter stores each
 * row straight into the receive buffer of the GPU that hosts the chosen slot, and the
 * combine reads its k rows from those buffers, through pointers that are valid on the
 * calling GPU (peer mappings).  No send buffer and no separate all-to-all exist.
 *
 * Group of `world` GPUs, one context per GPU, all built from the same moe_config,
 * placement and failure state.  GPU d hosts the simulated ranks
 * [d*R/world, (d+1)*R/world), i.e. the slots [d*spg, (d+1)*spg) with spg = P/world
 * (num_ranks % world == 0).  Receive buffer of GPU d, bf16 [recv_rows, H]: the rows of
 * its slots in ascending slot order; inside a slot the rows sent by GPU 0 first, then
 * GPU 1, ..., each sender's rows in its own stable order (ascending i = t*k + j).
 *
 * One step on every GPU g, all on its stream:
 *   moe_ep_route(logits_g)            -> out.topk_*, out.slot_counts = counts[g][:]
 *   all-gather of slot_counts         -> counts_all device [world][P]   (caller: NCCL or any other way)
 *   moe_ep_scatter(x_g, counts_all)   -> rows land in the owners' receive buffers; out.dst_row[i] =
 *                                        row of assignment i in its owner's buffer;
 *                                        recv_slot_offsets = layout of g's own receive buffer
 *   (all GPUs' scatters must have completed before anyone reads a receive buffer: order the
 *    streams with a collective or events; the experts then work on the receive buffers in place)
 *   moe_ep_combine(y_g)               -> y[t,:] as in moe_combine, rows fetched from the owners
 *   (all combines must have completed before the next step's scatter overwrites the buffers)
 * The rank order must be the physical one (no moe_set_rank_order) in this mode.
 */
typedef struct {
    int32_t world;            /* GPUs in the group                                              */
    int32_t rank;             /* index of the calling GPU, 0 <= rank < world                    */
    void *const *recv_bufs;   /* host [world]: device pointers, usable from the calling GPU, to
                                 every GPU's receive buffer (own buffer at [rank]); 16-byte aligned */
    int64_t recv_rows;        /* rows every receive buffer can hold (world*max_tokens*top_k always suffices) */
} moe_ep_group;

/*
 * moe_ep_attach — bind a context to its group: copies the pointer table to the device and
 * allocates the per-slot offset scratch (the only allocation of this mode, 4*P + 8*world
 * bytes on top of moe_workspace_bytes; call it at set-up, not while capturing).  May be called again with other buffers.
 * INVALID_ARG if num_ranks % world != 0, a pointer is NULL or misaligned, a rank order is
 * set, or the shape leaves no room for the bulk-copy combine.
 */
moe_status moe_ep_attach(moe_ctx *ctx, const moe_ep_group *group, void *cuda_stream);

/*
 * moe_ep_route — the routing half of a dispatch (Sec. 2.1, Sec. 3.4 masking) for this GPU's
 * T tokens: writes out->topk_ids / topk_weights / topk_slot and out->slot_counts (this
 * GPU's assignments per physical slot, the row counts[rank][:] of the exchange).
 * slot_offsets / rank_counts / rank_offsets describe this GPU's own assignments only;
 * send_buf and src_index are not used and may be NULL.  T = 0 writes zero counts.
 */
moe_status moe_ep_route(moe_ctx *ctx, const float *logits, int32_t T, const moe_dispatch_out *out,
                        void *cuda_stream);

/*
 * moe_ep_scatter — the dispatch exchange (Sec. 2.3, attention2expert).
 *   x                 device [T,H] bf16, 16-byte aligned
 *   counts_all        device [world][P] i32: slot_counts of every GPU after the all-gather
 *   recv_slot_offsets device [P/world + 1] i32 out: first row of each of this GPU's slots in
 *                     its own receive buffer, last entry = rows received
 * Writes out->dst_row of the preceding moe_ep_route.  If the rows sent to a GPU exceed
 * recv_rows the surplus rows are not written, their dst_row is -1 (moe_ep_combine then
 * lets them contribute zero and reads nothing out of range) and that GPU's device status
 * becomes MOE_ERR_CAPACITY (moe_get_device_status).  Allocates nothing, does not synchronise.
 */
moe_status moe_ep_scatter(moe_ctx *ctx, const void *x, int32_t T, const int32_t *counts_all,
                          int32_t *recv_slot_offsets, void *cuda_stream);

/*
 * moe_ep_combine — the combine exchange (Sec. 2.3, expert2attention): as moe_combine, with
 * row dst_row[t*k+j] read from the receive buffer of the GPU hosting topk_slot[t,j].
 *   y device [T,H] bf16, 16-byte aligned
 */
moe_status moe_ep_combine(moe_ctx *ctx, int32_t T, void *y, void *cuda_stream);

/*
 * moe_ep_plan_host — the layout arithmetic of the exchange on the host, no CUDA call.
 *   counts_all host [world][num_slots]
 *   src_base   host [num_slots] out (or NULL): first row, in the owner's buffer, of `rank`'s rows for each slot
 *   recv_slot_offsets host [num_slots/world + 1] out (or NULL): layout of `rank`'s own buffer
 * CAPACITY if an offset exceeds 2^31 - 1.
 */
moe_status moe_ep_plan_host(const int32_t *counts_all, int32_t world, int32_t rank, int32_t num_slots,
                            int32_t *src_base, int32_t *recv_slot_offsets);

/*
 * moe_step_host — one dispatch + combine fed from HOST memory, for callers
 * that hold activations on the CPU: copies logits and x to the given device
 * staging buffers, runs moe_dispatch and moe_combine (expert_buf = the send
 * buffer), copies y back and waits for the stream.  Host buffers should be
 * pinned for the copies to be asynchronous.
 *   logits_host [T,E] f32, x_host [T,H] bf16, y_host [T,H] bf16 (written)
 *   logits_dev, x_dev, y_dev: device staging of the same shapes.
 */
moe_status moe_step_host(moe_ctx *ctx, const float *logits_host, const void *x_host, int32_t T,
                         const moe_dispatch_out *out, float *logits_dev, void *x_dev,
                         void *y_dev, void *y_host, void *cuda_stream);

/*
 * moe_step_host_async — moe_step_host without the final wait: everything, the copy of y
 * to y_host included, is only enqueued on `cuda_stream`.  The host buffers must stay valid
 * and y_host must not be read until the caller has synchronised with the stream.  With two
 * contexts on two streams, each with its own staging and output buffers, the upload of one
 * batch overlaps the download of the other (the link carries both directions at once),
 * which is how micro-batches (Sec. 2.2) keep both directions busy.
 */
moe_status moe_step_host_async(moe_ctx *ctx, const float *logits_host, const void *x_host, int32_t T,
                               const moe_dispatch_out *out, float *logits_dev, void *x_dev,
                               void *y_dev, void *y_host, void *cuda_stream);

/*
 * moe_set_tuning — override one launch choice of a context (no counterpart in the paper).
 * A context picks kernel variants and launch shapes from its shape alone; nothing in the
 * process environment influences it.  This call replaces one choice, for measurements and
 * for tests of the non-default kernels.  `value` = -1 restores the automatic choice; a value
 * a kernel cannot honour is clamped to the nearest one it can.  The call waits for the
 * device, may reallocate the scan scratch (the two routing options) and must not be made
 * while a stream is capturing or between a dispatch and its combine.  Graphs captured
 * before the call keep the launch shapes they were captured with.
 */
typedef enum {
    MOE_TUNE_PDL = 0,                     /* 1 (default): programmatic dependent launch; 0: plain launches      */
    MOE_TUNE_SCATTER_IMPL = 1,            /* 0 (default): 128-bit vector copies; 1: bulk-copy ring               */
    MOE_TUNE_SCATTER_BULK_STAGES = 2,     /* bulk-copy scatter: ring depth, 1..8 (default 4)                     */
    MOE_TUNE_SCATTER_BULK_CTAS_PER_SM = 3,/* bulk-copy scatter: one-warp CTAs per SM (default: as many as fit)   */
    MOE_TUNE_SCATTER_BLOCKS_PER_SM = 4,   /* vector scatter: grid cap in CTAs per SM (default 8)                 */
    MOE_TUNE_SCATTER_UNROLL = 5,          /* vector scatter: 16-byte units per lane, one of 4, 8, 16, 28, 32     */
    MOE_TUNE_COMBINE_IMPL = 6,            /* 1 (default): bulk-copy ring; 0: vector loads                        */
    MOE_TUNE_COMBINE_CHUNK = 7,           /* ring combine: 16-byte units per lane and row chunk, 1, 2 or 4       */
    MOE_TUNE_COMBINE_STAGES = 8,          /* ring combine: stages per warp, 2..8                                 */
    MOE_TUNE_COMBINE_WARPS = 9,           /* ring combine: warps per CTA, 1..8                                   */
    MOE_TUNE_COMBINE_CTAS_PER_SM = 10,    /* ring combine: CTAs per SM (default: as many as fit)                 */
    MOE_TUNE_ROUTE_LANES_PER_TOKEN = 11,  /* routing: 8 or 16 lanes of a warp per token                          */
    MOE_TUNE_ROUTE_TOKENS_PER_TILE = 12,  /* routing: tokens per tile (default: max_tokens / 148, at least 32)   */
    MOE_TUNE_SPIN_LIMIT = 13,             /* polls before a bounded device wait gives up (default 1 << 20)       */
    MOE_TUNE_ROUTE_PREFETCH = 14,         /* routing: L2 hints issued while the previous kernel drains; bit 0 the
                                             routing tables, bit 1 the logits (default 3)                        */
    MOE_TUNE_SCATTER_STORE_POLICY = 15    /* vector scatter, pieces of 4, 16 or 28 units: cache policy of the row
                                             stores; 0 (default) no L1 allocation, 1 plain, 2 L2 evict-first,
                                             3 streaming                                                         */
} moe_tuning_option;

moe_status moe_set_tuning(moe_ctx *ctx, int32_t option, int32_t value);

/*
 * moe_debug_skip_ticket — test hook for the give-up path of the bounded device waits (no
 * counterpart in the paper).  Advances the tile ticket of the NEXT routing kernel by one, so
 * that no CTA ever routes the step's first tile: every other tile then waits for a
 * publication that never comes, runs out of polls (MOE_TUNE_SPIN_LIMIT), sets the status
 * word to MOE_ERR_DEVICE_TIMEOUT and returns.  Nothing faults and nothing waits without a
 * limit.  The outputs of that step are incomplete: follow it only by moe_get_device_status,
 * which re-arms the context.  Waits for the device.
 */
moe_status moe_debug_skip_ticket(moe_ctx *ctx);

/*
 * moe_set_timing_event — measurement hook (no counterpart in the paper).
 * `cuda_event` is a cudaEvent_t created by the caller with timing enabled, or
 * NULL to switch the hook off.  While set, every moe_dispatch records it on
 * its stream between the routing kernel and the scatter kernel, so a caller
 * bracketing moe_dispatch with its own events can split the two.  Not meant
 * to be left on while capturing a graph.
 */
moe_status moe_set_timing_event(moe_ctx *ctx, void *cuda_event);

/*
 * moe_get_device_status — synchronises the device and reports whether any
 * kernel of this context gave up on a bounded wait or met a token with fewer
 * than k selectable experts (possible only with -inf logits).  Writes the
 * status to *code, clears it and re-arms the scan scratch.  Never on the hot path.
 * After a wait gave up (MOE_ERR_DEVICE_TIMEOUT) the step's outputs are incomplete:
 * assignments that were not placed have dst_row = -1 and contribute zero to a combine;
 * until this call has re-armed the context, later routing kernels route nothing.
 */
moe_status moe_get_device_status(moe_ctx *ctx, int32_t *code);

/*
 * moe_plan_routing_state — the host half of a remap, with no CUDA call: from a
 * placement and a failed-rank set compute the rank-alive bitmap
 * (ceil(R/32) words, bit r set = alive), the per-expert replica table
 * [E, max_replicas] (ascending slot ids, -1 padded) and the number of
 * available experts.  Any output pointer may be NULL.  Same validation and
 * return codes as moe_set_failed_ranks.
 */
moe_status moe_plan_routing_state(const moe_config *cfg, const int32_t *slot_to_expert,
                                  const int32_t *failed_ranks, int32_t n_failed,
                                  uint32_t *rank_alive, int32_t *replica_table,
                                  int32_t *n_available);

/*
 * moe_permute_static — the count / prefix-scan / stable-permutation step of a
 * dispatch, for callers that cannot allocate device memory.  (The paper has no
 * counterpart; this exists for deployment reasons only.)
 *
 * Who needs it: a process that cannot call cudaMalloc while it is serving —
 * typically an inference engine that reserved all of HBM for its own pool at
 * start-up, so that any later allocation fails, or code running where the CUDA
 * runtime does not permit allocation.  Such a caller cannot create a context
 * with moe_route_init (which allocates scan scratch), but it can still hand
 * pre-existing buffers to this function.  The function allocates nothing, on
 * the host or the device: its scratch is a fixed 512 KiB array inside the
 * library's device image, present on every GPU that loads the library until
 * the process exits.
 *
 *   topk_slot    device [n_assign] i32  physical slot of each assignment i, in [0, P);
 *                                       entries outside that range are ignored
 *   slot_counts  device [P]   i32 out   slot_offsets device [P+1] i32 out
 *   rank_counts  device [R]   i32 out   rank_offsets device [R+1] i32 out
 *   dst_row      device [n_assign] i32 out   src_index device [n_assign] i32 out
 * with P = num_ranks * slots_per_rank; meanings as in moe_dispatch_out, ranks in their
 * physical numbering (this entry point knows no rank order).
 *
 * Limits: P <= 512 and n_assign <= 262144; anything larger returns
 * MOE_ERR_CAPACITY and launches nothing.  n_assign = 0 writes zero counts.
 * The first call on each device looks up the scratch array's device address
 * (one runtime query); make that first call before starting any stream capture.
 * With lazy module loading that first call is also the moment the driver loads
 * this function's device code, scratch array included, onto the device, which
 * takes device memory: make it at start-up, BEFORE the process claims the rest of
 * HBM (a warm-up call with n_assign = 0 is enough).  Every later call allocates
 * nothing.  All calls on a device share the one array: the function
 * rewrites every word it reads, so leftovers of earlier calls are harmless,
 * but two calls that overlap on the GPU (different streams without ordering)
 * race on it.  Work is enqueued on `cuda_stream`; the call does not wait.
 */
moe_status moe_permute_static(const int32_t *topk_slot, int32_t n_assign,
                              int32_t num_ranks, int32_t slots_per_rank,
                              int32_t *slot_counts, int32_t *slot_offsets,
                              int32_t *rank_counts, int32_t *rank_offsets,
                              int32_t *dst_row, int32_t *src_index, void *cuda_stream);

/* Device bytes a context for `cfg` allocates (0 if cfg is invalid). */
size_t moe_workspace_bytes(const moe_config *cfg);

/* Frees the context and everything it owns.  NULL is allowed. */
moe_status moe_route_destroy(moe_ctx *ctx);

/* Static, human-readable name of a status code. */
const char *moe_status_string(moe_status s);

#ifdef __cplusplus
}
#endif
#endif /* MOE_ROUTE_H */
