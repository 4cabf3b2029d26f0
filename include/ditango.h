/*
 * libditango -- selective attention-state path of DiTango on one B200 (sm_100a).
 *
 * The token sequence of one attention layer (L tokens) is split into P contiguous
 * partitions.  For a (query partition i, KV partition j) pair, the attention state is the
 * partition-normalised output OUT_ij and the log-sum-exp LSE_ij of Eq. 1 (Section 2.2.4).
 * Per denoising step a plan marks each pair COMPUTE or REUSE (Eq. 11, Eq. 13): COMPUTE pairs
 * are evaluated from the step's Q, K, V and overwrite their slot of the state cache, REUSE
 * pairs keep the state of the last step that computed them (t_c, Section 4.2.2), and all P
 * states of a query row are composed by LSE rescaling (Eq. 2) into the attention output.
 * The plan comes from the cached LSEs: partition importance weights (Eq. 8), averaged per
 * pair, thresholded with a strict '>' (Eq. 13); the local (diagonal) pair is always computed
 * (Section 4.1.2).
 *
 * Conventions
 *   - Plain C ABI.  "device" pointers are CUDA device memory of the context's device,
 *     "host" pointers are ordinary host memory.  The library never frees or keeps caller
 *     buffers, except the two cache pointers given to dt_bind_cache.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  dt_attn_states,
 *     dt_state_merge and dt_plan only enqueue work on it; they do not synchronise.
 *   - Every function returns a dt_status.  Argument errors are detected before any launch.
 *     Conditions only the device can see (REUSE of a never-computed pair, a bounded wait
 *     that ran out) are recorded in a device status word that dt_poll reads.
 *   - A context is not thread-safe: issue the calls on one context from one thread at a time.  Its device
 *     scratch (work list, tile table, partial sums, selection bits) is shared by its calls, so calls on one
 *     context must also be ordered on the device -- use one stream per context, or order streams with events.
 *     Different contexts are independent.
 *   - Natural logarithm everywhere an LSE crosses this boundary.
 *   - Limits: D in {64, 128}; 1 <= P <= 32; bf16 or fp16 inputs ("bf16" below stands for the configured
 *     input type); innermost stride 1.
 *
 * Memory layout of the state cache (caller-owned device memory, sized by dt_cache_bytes):
 *   o_state   [S (slot)][B][H][L][D]   fp32 or bf16 (dt_config.state_dtype)
 *   lse_state [S (slot)][B][H][L]      fp32
 * Pair mode (dt_config.group_size <= 1): S = P, slot j = KV partition j; row l of slot j belongs to
 * pair (i, j) with i the partition that contains l.
 * Group mode (group_size = g >= 2; Section 4.2.1): the P states of a query partition are organised as
 * m = ceil(P / g) groups of g adjacent KV partitions plus the local state, which is handled separately:
 * S = m + 1, slot 0 = the local state (i, i), slot 1 + k = the group state AS(G_k), i.e. the composition
 * (Eq. 2) of the states of group k's partitions -- without partition i in the group that contains it,
 * which therefore has g - 1 members.  A slot whose key set is empty for a query partition (a group of one
 * that is the local partition) does not exist for its rows.  Masks, t_c and W are then [P][S] arrays
 * indexed by (query partition, slot) instead of [P][P].
 */
#ifndef DITANGO_H_
#define DITANGO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dt_ctx dt_ctx; /* opaque; owns only small device scratch (work list, t_c, partial sums) */

typedef enum {
    DT_OK = 0,
    DT_ERR_INVALID_ARG = 1, /* null pointer, bad shape / stride / offsets / alignment           */
    DT_ERR_UNSUPPORTED = 2, /* D not in {64,128}, P > 32, unknown state dtype, device not sm_100 */
    DT_ERR_STATE = 3,       /* cache not bound or too small; REUSE of a pair never computed       */
    DT_ERR_CUDA = 4,        /* a CUDA runtime / driver call failed (text in dt_last_error)        */
    DT_ERR_TIMEOUT = 5,     /* a bounded device-side wait expired; the kernel returned normally   */
    DT_ERR_RANGE = 6        /* bf16 inputs: within one 128-key tile a logit (times log2 e) rose more than
                               about 100 above everything the row had seen before (exp2 overflows fp32);
                               the states of that launch are not valid.  fp16 inputs have no such limit. */
} dt_status;

enum { DT_STATE_FP32 = 0, DT_STATE_BF16 = 1 };
enum { DT_INPUT_BF16 = 0, DT_INPUT_FP16 = 1 };
enum { DT_MAX_P = 32 };

typedef struct {
    int32_t B, H, D, L, P;       /* batch, heads, head dim, tokens, partitions                      */
    const int32_t *part_offsets; /* host, P+1 ints, off[0]=0 < off[1] < ... < off[P]=L; copied      */
    float softmax_scale;         /* s in exp(s * q.k); the paper's Eq. 1 leaves it implicit          */
    int32_t state_dtype;         /* DT_STATE_FP32 or DT_STATE_BF16: storage type of cached OUT_ij    */
    int32_t device;              /* CUDA device ordinal                                              */
    int32_t group_size;          /* 0 or 1: pair mode; g >= 2: grouped cache with g partitions per group */
    int32_t input_dtype;         /* DT_INPUT_BF16 or DT_INPUT_FP16: element type of q, k, v and of the attention
                                    output (Table 1: the Wan models run in FP16); P is rounded to the same type for
                                    the PV product, accumulation stays fp32 */
} dt_config;

/* Create / destroy a context.  dt_create makes `device` current, checks it is sm_100, copies the
 * offsets and allocates the context's small device scratch.  All t_c start at -1 (empty). */
dt_status dt_create(dt_ctx **ctx_out, const dt_config *cfg);
dt_status dt_destroy(dt_ctx *ctx);

/* Closed-form size of the state cache: o_bytes = S*B*H*L*D*sizeof(state), lse_bytes = S*B*H*L*4, with
 * S = P in pair mode and ceil(P/g) + 1 in group mode (the memory saving of group-level composition).
 * Per pair this is OUT (n_i*H*D) + LSE (n_i*H) against 2*n_j*H*D for the KV it replaces
 * ("half of KV size", Section 2.2.4). */
dt_status dt_cache_bytes(const dt_config *cfg, size_t *o_bytes, size_t *lse_bytes);

/* Bind caller-owned device memory as the state cache (16-byte aligned, at least the sizes above).
 * Contents are not touched; binding does not reset t_c. */
dt_status dt_bind_cache(dt_ctx *ctx, void *o_state_dev, float *lse_state_dev, size_t o_bytes, size_t lse_bytes);

/* Eq. 1 for every COMPUTE pair, every head and every query row; REUSE pairs cost nothing and
 * their cache slots are not touched (Section 2.2.4, Fig. 6; Section 5.2 steps evict/compute/store).
 *   q, k, v        device, bf16, logical shape [B, L, H, D]; strides_blhd in elements
 *                  (stride of D must be 1, the others multiples of 8; bases 16-byte aligned)
 *   mask_dev       device, uint8 [P*P] row-major (i = query partition, j = KV partition),
 *                  non-zero = COMPUTE.  Read on the device: no host copy, no synchronisation.
 *   step           denoising step index (>= 0), recorded as t_c of every COMPUTE pair
 * A REUSE pair with t_c = -1 sets the device status to DT_ERR_STATE (see dt_poll); the COMPUTE
 * pairs are still evaluated. */
dt_status dt_attn_states(dt_ctx *ctx, const void *q_dev, const void *k_dev, const void *v_dev,
                         const int64_t strides_blhd[4], const uint8_t *mask_dev, int32_t step, void *stream);

/* The local (diagonal) pairs only -- Algorithm 1's first line of a step ("compute local attention"): the
 * states AS_t(i, i) that the planner's drift estimate needs before the plan of the step exists.  Same
 * tensors as dt_attn_states; no mask, and no REUSE check (the other pairs of the step are decided and
 * launched afterwards with dt_attn_states). */
dt_status dt_attn_local(dt_ctx *ctx, const void *q_dev, const void *k_dev, const void *v_dev,
                        const int64_t strides_blhd[4], int32_t step, void *stream);

/* Eq. 2 folded over all P cached states of each query row (fresh or reused alike):
 *   LSE[r] = log sum_j exp(LSE_ij[r]),  OUT[r] = sum_j exp(LSE_ij[r] - LSE[r]) OUT_ij[r].
 *   out_dev        device, bf16, logical [B, L, H, D] with out_strides_blhd (elements; D stride 1,
 *                  others multiples of 8, base 16-byte aligned)
 *   lse_out_dev    device, fp32 [B, H, L], or NULL */
dt_status dt_state_merge(dt_ctx *ctx, void *out_dev, const int64_t out_strides_blhd[4], float *lse_out_dev,
                         void *stream);

/* Composed reuse state (Section 2.2.4, Fig. 6: "compose states from remote partitions and cache the
 * result"; Eq. 15 is the same composition applied to groups).  While a plan holds, the REUSE states of
 * a query row do not change, so they can be composed once (Eq. 2) into a single state per row:
 *   dt_compose_reuse        comp = (+) over { j : mask[i][j] == 0 } of the cached state (i, j), for every
 *                           row of every query partition i; rows without any REUSE slot get OUT = 0,
 *                           LSE = -inf (weight zero).
 *   dt_state_merge_planned  out = (+) over { j : mask[i][j] != 0 } of the cached states, (+) comp.
 * With comp built from the same mask and an unchanged cache in the REUSE slots, the result equals
 * dt_state_merge up to rounding, while reading (computed + 1) states per row instead of P.
 *   mask_dev       device, uint8 [P*P], as in dt_attn_states
 *   comp_o_dev     device, [B][H][L][D] in the cache's state dtype, 16-byte aligned (caller-owned)
 *   comp_lse_dev   device, fp32 [B][H][L]
 * Recompose whenever the plan changes or a REUSE slot is recomputed. */
dt_status dt_compose_reuse(dt_ctx *ctx, const uint8_t *mask_dev, void *comp_o_dev, float *comp_lse_dev, void *stream);
dt_status dt_state_merge_planned(dt_ctx *ctx, const uint8_t *mask_dev, const void *comp_o_dev, const float *comp_lse_dev,
                                 void *out_dev, const int64_t out_strides_blhd[4], float *lse_out_dev, void *stream);

/* Plan from the cached LSEs (call after a step that computed every pair -- an anchor step):
 *   per row  w_j = exp(LSE_ij - logsumexp_k LSE_ik)                  (Eq. 8)
 *   W[i][j]  = mean of w_j over batch, heads and the rows of partition i
 *   target_fraction < 0 : mask[i][j] = (i == j) or (W[i][j] > eps)    (Eq. 13, strict)
 *   target_fraction >= 0: K = round(f P^2) clipped to [P, P^2]; the diagonal plus the K - P
 *                         off-diagonal pairs of largest W are COMPUTE (ties: smaller |i-j|, then
 *                         smaller i*P+j); eps_out = midpoint between the last selected and the
 *                         first unselected W (0 if all are selected; the largest off-diagonal W
 *                         if none is)
 *   mask_dev       device, uint8 [P*P], written
 *   w_dev          device, double [P*P], written; or NULL
 *   eps_out_dev    device, double [1], written (eps used or derived); or NULL */
dt_status dt_plan(dt_ctx *ctx, double eps, double target_fraction, uint8_t *mask_dev, double *w_dev,
                  double *eps_out_dev, void *stream);

/* Group-wise planning (Section 4.2.1-4.2.3): the P KV partitions form ceil(P / group_size) groups of
 * adjacent partitions; per query partition all states of a group share one decision.  The local
 * (diagonal) state is handled separately -- always COMPUTE -- so the group that contains it has one
 * member fewer.  The group's measure is the sum of its members' W (Eq. 12), compared with eps by a strict
 * '>' (Eq. 13); with target_fraction >= 0 whole groups are taken in order of decreasing measure (ties:
 * the group nearer to the local one, then the smaller index i * n_groups + k) while their members still
 * fit into K - P pairs, and eps_out is the midpoint between the last taken and the first not taken
 * measure.  group_size = 1 is dt_plan.  Other arguments as for dt_plan. */
dt_status dt_plan_grouped(dt_ctx *ctx, double eps, double target_fraction, int32_t group_size, uint8_t *mask_dev,
                          double *w_dev, double *eps_out_dev, void *stream);

/* Head-sharded planning.  The (batch, head) slices of a layer are independent in dt_attn_states and
 * dt_state_merge, so the heads of one layer may be spread over several contexts (one per GPU) with no
 * exchange there.  Only the plan needs one: W of Eq. 8 is a mean over all heads, and every shard must
 * arrive at the same mask (Section 5.1.1: the compute / reuse strategy is the same on all devices).  The
 * two halves of dt_plan, with the exchange left to the caller:
 *   dt_plan_sums       sums_dev (device, double [P*S], written) = sum over this context's batch, heads and
 *                      the rows of partition i of the per-row weights w (Eq. 8), not yet divided by a count
 *   (caller)           adds the shards' sums element by element, e.g. one all-reduce of P*S doubles
 *   dt_plan_from_sums  the plan as dt_plan / dt_plan_grouped would take it, from sums that cover total_bh
 *                      (batch, head) slices: W[i][s] = sums[i][s] / (total_bh * n_i); then the threshold or
 *                      the target fraction as there.  total_bh >= this context's B * H.
 * With one shard (total_bh = B * H) the result is bit-identical to dt_plan_grouped.  Sums of different
 * shards are added in whatever order the caller's reduction uses; W then agrees to rounding of doubles. */
dt_status dt_plan_sums(dt_ctx *ctx, double *sums_dev, void *stream);
dt_status dt_plan_from_sums(dt_ctx *ctx, const double *sums_dev, int64_t total_bh, double eps, double target_fraction,
                            int32_t group_size, uint8_t *mask_dev, double *w_dev, double *eps_out_dev, void *stream);

/* Anchor-guided selection planning, Algorithm 1 (Section 4), with its state on the device.
 *   partition importance  w(i,j)      Eq. 8, refreshed at anchors from the cached LSEs
 *   scale ratio           alpha(i,j)  Eq. 9: ||AS_ta(i,j)||_2 / ||AS_ta(i,i)||_2, the state being OUT and LSE
 *                                     stacked over all rows and heads of query partition i
 *   age penalty           delta(i,j,t) = alpha(i,j) * ||AS_t(i,i) - AS_ta(i,i)||_2            (Eq. 10)
 *   unit error            ASE(i,G,t) = sum_{j in G, j != i} w(i,j) * delta(i,j,t)            (Eq. 7, Eq. 12)
 *   decision              COMPUTE iff ASE > eps (Eq. 13); anchor iff every unit exceeds eps or the relative
 *                         drift of the local states exceeds eps_local (Eq. 14); the first step is an anchor
 *   eps update            at an anchor, eps becomes the cache_ratio-quantile of the units' predicted ASE of that
 *                         step (unchanged if they are all zero), so that about that fraction of the units is
 *                         reused under a comparable drift
 * Use per denoising step t:
 *   1. dt_attn_local(q, k, v, t)                              the local states AS_t(i,i)
 *   2. dt_planner_step(...)                                   mask of the step (diagonal included), anchor flag
 *   3. dt_attn_states(q, k, v, that mask with the diagonal cleared, t)   -- or the whole mask again
 *   4. dt_state_merge(...)
 *   5. dt_planner_commit(...)                                 on an anchor: w, alpha and the snapshot of the local
 *                                                             states are refreshed; otherwise nothing changes
 * Everything is stream-ordered; the anchor decision stays on the device (steps 3-5 read it there).
 *   snap_o_dev / snap_lse_dev   caller-owned device buffers of one cache slot ([B][H][L][D] in the cache's state
 *                               dtype, [B][H][L] fp32): the local states of the last anchor
 *   mask_dev        device, uint8 [P*P], written           is_anchor_dev  device, int32 [1] or NULL
 *   ase_dev         device, double [P * ceil(P/group_size)] (NaN for a unit without members) or NULL
 *   delta_rel_dev   device, double [1] or NULL */
typedef struct {
    int32_t group_size;   /* g of Section 4.2.1 (1 = per pair)                         */
    double eps_initial;   /* eps until the first update                                */
    double eps_local;     /* threshold on the relative drift of the local states (> 0) */
    double cache_ratio;   /* R of Algorithm 1: fraction of units to reuse, in [0, 1]   */
} dt_planner_config;
dt_status dt_planner_init(dt_ctx *ctx, const dt_planner_config *pc, void *snap_o_dev, float *snap_lse_dev,
                          size_t snap_o_bytes, size_t snap_lse_bytes, void *stream);
dt_status dt_planner_step(dt_ctx *ctx, uint8_t *mask_dev, int32_t *is_anchor_dev, double *ase_dev, double *delta_rel_dev,
                          void *stream);
dt_status dt_planner_commit(dt_ctx *ctx, void *stream);
/* Copy the planner state to the host (synchronises): w and alpha are double [P*S] (S = P in pair mode); any
 * pointer may be NULL. */
dt_status dt_planner_get(dt_ctx *ctx, double *w_host, double *alpha_host, double *eps_host, int32_t *have_anchor_host);

/* Attention output of a selective step in one pass, without the round trip through the cache: for every query
 * row the state over the keys of ALL COMPUTE slots of its partition is accumulated in one flash pass (adjacent
 * key ranges are joined), composed in the kernel's epilogue (Eq. 2) with the composed reuse state of the same
 * mask (dt_compose_reuse), and written as the attention output.  For the steps between two anchors of a plan
 * that holds: there the COMPUTE states are recomputed every step and never reused, so caching them would only
 * cost a write here and a read in the merge.
 *   mask_dev                    device, uint8 [P*S] (pair mode: [P*P]); the local slot must be COMPUTE
 *   comp_o_dev / comp_lse_dev   device, composed reuse state [B][H][L][D] (cache dtype) / [B][H][L] from
 *                               dt_compose_reuse with the same mask; both NULL: the COMPUTE slots alone
 *                               (with an all-ones mask: plain full attention)
 *   out_dev, out_strides_blhd, lse_out_dev   as for dt_state_merge
 * The state cache, t_c and the device status word are not touched: cached states of COMPUTE slots keep the
 * values of the step that last went through dt_attn_states. */
dt_status dt_attn_fused(dt_ctx *ctx, const void *q_dev, const void *k_dev, const void *v_dev,
                        const int64_t strides_blhd[4], const uint8_t *mask_dev, const void *comp_o_dev,
                        const float *comp_lse_dev, void *out_dev, const int64_t out_strides_blhd[4], float *lse_out_dev,
                        void *stream);

/* Grouped state cache (Section 4.2.1, Section 4.2.2; Dynamic Group State Compose, Eq. 15).  With
 * dt_config.group_size = g >= 2 the calls above work on slots instead of KV partitions:
 *   dt_attn_states / dt_attn_local   mask is uint8 [P*S]; a COMPUTE slot is evaluated in one pass over all keys of
 *                      its group, which yields exactly the composition (Eq. 2) of its members' states
 *   dt_state_merge     composes the S slots of every row (slots that do not exist for a row's query partition
 *                      are left out); dt_compose_reuse / dt_state_merge_planned likewise, mask [P*S]
 *   dt_plan            W is double [P*S] (importance of the slot's whole key set = sum of its members' weights,
 *                      Eq. 12); one decision per non-local slot, the local slot 0 always COMPUTE; the target
 *                      fraction still counts pairs: K = round(f*P*P), a slot costs as many as it has members
 *   dt_get_tc / dt_set_tc, dt_step_host   arrays are [P*S]
 *   dt_planner_*       Algorithm 1 with one unit per non-local slot: w, alpha, ASE and the mask are [P*S]; a group
 *                      state is one state, so ASE(i, G) = w(i, G) * alpha(i, G) * ||AS_t(i,i) - AS_ta(i,i)||_2 with
 *                      alpha from the norm of the group state (dt_planner_config.group_size must be 1)
 *   dt_plan_grouped with group_size > 1 returns DT_ERR_UNSUPPORTED (the slots already are the groups).
 * dt_num_slots       current S and g (either pointer may be NULL).
 * dt_slot_ranges     key ranges of every (query partition, slot): int32 [P*S*4] = (r1, n1, r2, n2), the keys
 *                    [r1, r1+n1) and [r2, r2+n2); n1 + n2 == 0 marks a slot that does not exist.
 * dt_group_compose   Eq. 15 with k = 2: AS(G_2k) (+) AS(G_2k+1) -> AS(G'_k) for every query partition, in place
 *                    in the cache (new slot 1 + k overwrites old slot 1 + k after both sources were read), g
 *                    doubles, S becomes ceil(m/2) + 1; t_c of a new slot is the older of its sources' (-1 if one
 *                    was never computed).  The memory behind the first S slots of the bound buffers is no
 *                    longer used.  If the planner is initialised, its w and alpha are taken again from the
 *                    composed cache (the anchor's snapshot of the local states stays).  DT_ERR_STATE if only one group is left.  Synchronises the stream.
 * dt_group_fit       the memory-driven trigger of Section 5.1.3: while the slots in use (S * B*H*L * (D*sizeof(state) + 4)
 *                    bytes) exceed max_bytes and more than one group is left, dt_group_compose; *composed (may be
 *                    NULL) = how many times.  DT_ERR_STATE if one group is left and the budget is still exceeded.
 * dt_group_reset     back to the creation-time g (an anchor step recomputes every state): all t_c = -1, the
 *                    cache contents are stale until the next all-COMPUTE step; an initialised planner treats its
 *                    next step as an anchor.  Synchronises the stream. */
dt_status dt_num_slots(dt_ctx *ctx, int32_t *slots, int32_t *group_size);
dt_status dt_slot_ranges(dt_ctx *ctx, int32_t *ranges_host);
dt_status dt_group_compose(dt_ctx *ctx, void *stream);
dt_status dt_group_fit(dt_ctx *ctx, size_t max_bytes, int32_t *composed, void *stream);
dt_status dt_group_reset(dt_ctx *ctx, void *stream);

/* The same plan computation for callers that cannot allocate device memory at the point of the
 * call: code running inside a region where the allocator must stay untouched (a fixed-memory
 * serving process that sized its pools up front, a callback on a latency-critical path, a host that
 * hands this library pre-carved buffers and forbids cudaMalloc afterwards).  The paper has no
 * counterpart; this is a packaging variant of dt_plan.
 *   - No context: the caller passes the LSE cache (device, fp32 [P][B][H][L]) and the partition
 *     offsets (HOST, P+1 ints) directly, plus the same outputs and options as dt_plan.
 *   - The per-block partial sums live in a fixed array inside the library's device image (1 MiB of
 *     floats plus a 256-byte header for the offsets; every GPU that loads the library holds it until
 *     the process exits).  Problems that need more than 262144 partial sums, i.e.
 *     B*H*P*P*ceil(max_i n_i / 1024) > 262144, are refused with DT_ERR_UNSUPPORTED and nothing runs.
 *   - Calls nothing that allocates or frees: no cudaMalloc / cudaFree, no allocating library routine.
 *     The offsets travel to the device as a kernel argument (a small kernel writes them into the
 *     array's header), so `part_offsets_host` is read before the call returns and never afterwards.
 *   - The first call on each device looks up the array's device address (the current device must
 *     be the one that owns `stream` and the buffers); make that first call outside any stream capture.
 *     The address is remembered per device for the life of the process: after a cudaDeviceReset the
 *     library has to be loaded again before this entry point is used on that device.
 *   - All calls on a device share the one array, and it keeps the previous call's contents.  Nothing
 *     in it has to start at zero (stage 1 overwrites every slot stage 2 reads), but two calls whose
 *     kernels can overlap on the GPU (different streams, no ordering between them) race on it:
 *     order them on one stream or with events.
 * Results are bit-identical to dt_plan on the same inputs. */
dt_status dt_plan_static(const float *lse_state_dev, const int32_t *part_offsets_host, int32_t B, int32_t H,
                         int32_t L, int32_t P, double eps, double target_fraction, uint8_t *mask_dev,
                         double *w_dev, double *eps_out_dev, void *stream);

/* One whole step from HOST buffers: copies q, k, v (bf16 [B,L,H,D] contiguous) and the mask to the
 * device workspace, runs dt_attn_states and dt_state_merge, copies out (bf16 [B,L,H,D]) and lse
 * (fp32 [B,H,L], may be NULL) back and synchronises `stream`.  Heads are independent, so the step runs
 * in head chunks (a few heads each): the kernels of one chunk (on `stream`) overlap the host-to-device copy of the next
 * and the device-to-host copy of the previous one, which run on two streams the context owns (ordered against
 * `stream` with events; the call returns with all three idle).  workspace_dev must hold
 * dt_step_host_workspace_bytes() bytes of device memory.  Host buffers should be pinned: pageable memory
 * makes the copies synchronous and loses the overlap. */
dt_status dt_step_host_workspace_bytes(const dt_config *cfg, size_t *bytes);
dt_status dt_step_host(dt_ctx *ctx, const void *q_host, const void *k_host, const void *v_host,
                       const uint8_t *mask_host, int32_t step, void *out_host, float *lse_out_host,
                       void *workspace_dev, size_t workspace_bytes, void *stream);

/* Cache timesteps t_c[i][j] (-1 = empty), host int32 [P*P].  Both synchronise the device.
 * Together with the cache contents they are everything needed to snapshot and resume. */
dt_status dt_get_tc(dt_ctx *ctx, int32_t *tc_host);
dt_status dt_set_tc(dt_ctx *ctx, const int32_t *tc_host);

/* Number of kernels this library has launched through `ctx` since creation. */
dt_status dt_launch_count(dt_ctx *ctx, uint64_t *count);

/* Self-test of the failure path (the paper has no counterpart): launches a one-thread kernel that waits,
 * with the library's bounded wait, on a barrier nothing will ever signal; after `limit_us` microseconds
 * (1..100000) the wait gives up and records the condition, so the next dt_poll returns DT_ERR_TIMEOUT
 * and the context stays usable.  No fault, trap or unbounded loop is involved. */
dt_status dt_selftest_wait_timeout(dt_ctx *ctx, uint32_t limit_us, void *stream);

/* Read (and clear) the device status word; synchronises the device.  Returns DT_OK,
 * DT_ERR_STATE, DT_ERR_TIMEOUT or DT_ERR_RANGE. */
dt_status dt_poll(dt_ctx *ctx);

const char *dt_status_str(dt_status s);
const char *dt_last_error(dt_ctx *ctx); /* text of the last error on this context ("" if none) */

#ifdef __cplusplus
}
#endif
#endif /* DITANGO_H_ */
