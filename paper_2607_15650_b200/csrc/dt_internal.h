// Internal declarations shared by the translation units of libditango.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "../../include/ditango.h"

namespace dt {

// Device status word bits (read by dt_poll).
enum : int { STATUS_REUSE_EMPTY = 1, STATUS_WAIT_TIMEOUT = 2, STATUS_LOGIT_RANGE = 4 };

constexpr int PLAN_CHUNK_ROWS = 1024;  // rows of one (b, h, partition) handled by one dt_plan block
constexpr int ATTN_TILE = 128;         // query rows per TMEM accumulator / keys per KV tile
constexpr int ATTN_NQ = 2;             // query tiles a CTA keeps in flight (ping-pong)

// Keys covered by the state in slot s of query partition i: [r1, r1 + n1) and [r2, r2 + n2) (token indices).
// Pair mode: slot j = KV partition j (one range).  Group mode (Section 4.2.1): slot 0 = the local partition,
// slot 1 + k = group k of g adjacent partitions, without partition i when it belongs to that group (then the
// keys left and right of it are the two ranges).  n1 + n2 == 0: the slot is empty for this query partition.
struct alignas(16) SlotRange {
    int32_t r1, n1, r2, n2;
};

struct AttnParams {
    const int32_t *off;       // device, P+1
    const SlotRange *slot_tab; // device, [P][S]
    const int32_t *worklist;  // device: [0] = number of COMPUTE states, then i | (slot << 8) per state
    // pair mode: [0].x = number of work items per (b, h), then per item (i_a | j << 8, tile_a, i_b or -1, tile_b): two
    // 128-row query tiles (partition, tile index) that attend to KV partition j.  null: items are 256-row query blocks
    const int4 *tile_pairs;
    int32_t *status;          // device status word
    void *o_state;            // [S][B][H][L][D]
    float *lse_state;         // [S][B][H][L]
    // Squared 2-norms of the states this launch writes (OUT and LSE stacked, Eq. 9), one partial sum per softmax
    // warp: [B*H][P][S][qblocks_max][ATTN_NQ * 4], or null when no planner is attached.
    float *norm_partials;
    int B, H, L, P, S;
    int in_fp16;              // q, k, v (and the fused output) are fp16 instead of bf16
    int h0, H_launch;         // heads [h0, h0 + H_launch) are processed by this launch (the whole range: 0, H)
    int qblocks_max;          // ceil(max_i n_i / (ATTN_NQ * ATTN_TILE))
    float scale_log2;         // softmax_scale * log2(e)
    // fused mode (dt_attn_fused): one pass per query block over the keys of all COMPUTE slots of its partition,
    // composed in the epilogue with the composed reuse state and written as the attention output
    const int2 *tile_tab;     // device, [P][max_tiles]: (first key, keys that count) of every K/V tile
    const int32_t *tile_cnt;  // device, [P]: tiles per query partition
    int max_tiles;
    const void *comp_o;       // composed reuse state [B][H][L][D] in the cache dtype, or null
    const float *comp_lse;    // [B][H][L]
    void *out;                // bf16 [B, L, H, D] with the strides below
    float *lse_out;           // [B][H][L], may be null
    long long sb, sl, sh;
};

enum : int { MERGE_ALL = 0, MERGE_COMPOSE = 1, MERGE_PLANNED = 2 };

struct MergeParams {
    int mode;                 // MERGE_ALL / MERGE_COMPOSE / MERGE_PLANNED
    const uint32_t *sel_bits; // device, P words: bit s = slot s takes part for rows of that query partition
                              // (from launch_merge_select; MERGE_ALL: null = every slot)
    int32_t off_val[DT_MAX_P + 1];   // partition offsets by value (used whenever sel_bits is set)
    const void *comp_o;       // composed state read by PLANNED: [B][H][L][D] in the cache's dtype
    const float *comp_lse;    // [B][H][L]
    void *comp_o_out;         // composed state written by COMPOSE
    float *comp_lse_out;
    const void *o_state;
    const float *lse_state;
    void *out;       // bf16, or fp16 if out_fp16
    int out_fp16;
    float *lse_out;  // may be null
    int32_t *status; // device status word
    int P, S, H, L;  // query partitions, cache slots
    long long R;     // B*H*L rows (the slot stride of the cache)
    long long row_begin, row_count;   // rows [row_begin, row_begin + row_count) are processed by this launch
    long long sb, sl, sh;  // output strides in elements
};

struct PlanParams {
    const float *lse_state;  // [S][R]
    const int32_t *off;      // device, P+1
    const uint32_t *nonempty; // device, P words: slots that exist for the query partition (null = all)
    const int *only_if;      // device flag, or null: the kernel returns at once while it is 0 (planner: not an anchor)
    float *partials;         // [BH][P][chunks][S]
    int P, S, BH, L, chunks;
    long long R;
};

// Decisions over the slots of a grouped cache: one unit per (query partition, non-local slot).
struct PlanSlotsParams {
    const float *partials;   // [BH][P][chunks][S]
    const int32_t *off;
    const SlotRange *slot_tab;
    const uint8_t *members;  // device, [P][S]: KV partitions a slot stands for (its size in pairs)
    int P, S, BH, chunks, group_size;
    int mode_target, K;
    double eps;
    uint8_t *mask;           // out, [P][S]
    double *w_out;           // out, [P][S], may be null
    double *eps_out;         // may be null
    const double *sums_in;   // head-sharded planning: sums over all shards, [P][S]; null = sum this context's partials
    double *sums_out;        // head-sharded planning: write this context's sums [P][S] and stop; null otherwise
    long long count_bh;      // (batch, head) slices the sums cover: BH, or the total over all shards with sums_in
};

struct PlanFinalParams {
    const float *partials;
    const int32_t *off;
    int P, BH, chunks;
    int mode_target;   // 0: threshold with eps; 1: select K pairs by rank
    int K;
    int group_size;    // g adjacent KV partitions share one decision (1 = per pair)
    double eps;
    uint8_t *mask;
    double *w_out;     // may be null
    double *eps_out;   // may be null
    const double *sums_in;   // as in PlanSlotsParams
    double *sums_out;
    long long count_bh;
};

// Planner state of Algorithm 1, resident on the device.
struct PlannerState {
    double w[DT_MAX_P * DT_MAX_P];       // partition importance weights of the last anchor (Eq. 8)
    double alpha[DT_MAX_P * DT_MAX_P];   // scale ratios of the last anchor (Eq. 9)
    double nsq[DT_MAX_P * DT_MAX_P];     // scratch: squared state norms of the anchor being committed
    double eps;                          // current threshold (Eq. 13)
    int have_anchor;                     // an anchor has been committed
    int is_anchor;                       // the step being planned is an anchor
};

struct PlannerParams {
    PlannerState *state;
    const void *o_state;          // cache
    const float *lse_state;
    const void *snap_o;           // local states of the last anchor: [B][H][L][D] in the cache dtype
    const float *snap_lse;        // [B][H][L]
    void *snap_o_out;
    float *snap_lse_out;
    const int32_t *off;           // device, P+1
    const uint32_t *nonempty;     // device, P words: slots that exist for the query partition
    float *local_partials;        // [BH][P][chunks][2]
    float *norm_partials;         // [BH][P][chunks][S]: norms taken by a pass over the cache (after a group compose)
    const float *attn_norm_partials;   // [BH][P][S][qblocks][ATTN_NQ * 4]: norms emitted by the attention epilogue
    int qblocks;
    const float *w_partials;      // [BH][P][chunks][S] from plan_partial_kernel
    uint8_t *mask;                // out, P*S
    int32_t *is_anchor_out;       // out, may be null
    double *ase_out;              // out, P * n_groups (pair mode) or P * S (grouped cache), may be null
    double *delta_rel_out;        // out, may be null
    int P, S, BH, L, D, chunks, group_size;
    int group_mode;               // grouped cache: slot 0 is the local state and every other slot is one unit
    int force;                    // refresh w and alpha although the step is no anchor (after a group compose)
    double eps_local, cache_ratio;
};

cudaError_t launch_planner_init(PlannerState *st, double eps, cudaStream_t stream);
cudaError_t launch_planner_step(const PlannerParams &p, int state_dtype, cudaStream_t stream);
cudaError_t launch_planner_commit(const PlannerParams &p, int state_dtype, cudaStream_t stream);

cudaError_t launch_worklist(const uint8_t *mask, int32_t *tc, int32_t *worklist, int32_t *status, const SlotRange *slot_tab,
                            int P, int S, int group_mode, int step, const int32_t *off, int4 *tile_pairs, cudaStream_t stream);
cudaError_t launch_attn_states(const CUtensorMap &tq, const CUtensorMap &tk, const CUtensorMap &tv,
                               const AttnParams &p, int D, int state_dtype, int num_ctas, cudaStream_t stream);
cudaError_t launch_attn_fused(const CUtensorMap &tq, const CUtensorMap &tk, const CUtensorMap &tv,
                              const AttnParams &p, int D, int state_dtype, int num_ctas, cudaStream_t stream);
cudaError_t launch_fused_tiles(const uint8_t *mask, const SlotRange *slot_tab, int P, int S, int max_tiles, int2 *tile_tab,
                               int32_t *tile_cnt, cudaStream_t stream);
cudaError_t attn_states_configure();  // sets the dynamic shared-memory attribute once per process/device
cudaError_t launch_state_merge(const MergeParams &p, int D, int state_dtype, cudaStream_t stream);
cudaError_t launch_merge_select(const uint8_t *mask, const uint32_t *nonempty, int P, int S, int want_compute,
                                uint32_t *sel_bits, cudaStream_t stream);
cudaError_t launch_plan_slots(const PlanSlotsParams &p, cudaStream_t stream);
cudaError_t launch_tc_compose(int32_t *tc, const uint32_t *nonempty_old, int P, int S_old, int S_new, cudaStream_t stream);
cudaError_t launch_plan_partial(const PlanParams &p, cudaStream_t stream);
cudaError_t launch_plan_final(const PlanFinalParams &p, cudaStream_t stream);
cudaError_t launch_wait_timeout_selftest(int32_t *status, long long limit_cycles, cudaStream_t stream);

}  // namespace dt

struct dt_ctx {
    dt_config cfg;
    std::vector<int32_t> off;
    int n_max = 0;
    int qblocks_max = 0;
    int plan_chunks = 0;
    int num_sms = 0;
    int group_size0 = 1;   // group size the context was created with (1 = pair mode)
    int group_size = 1;    // current group size (doubles with every dt_group_compose)
    int S0 = 0, S = 0;     // cache slots at creation / now
    std::vector<dt::SlotRange> slot_tab;      // [P][S]
    std::vector<uint8_t> members;             // [P][S]
    std::vector<uint32_t> nonempty;           // [P]
    dt::SlotRange *slot_tab_dev = nullptr;    // sized for S0
    uint8_t *members_dev = nullptr;
    uint32_t *nonempty_dev = nullptr;
    int32_t *off_dev = nullptr;
    int32_t *tc_dev = nullptr;
    int32_t *worklist_dev = nullptr;
    int4 *tile_pairs_dev = nullptr;   // pair mode: work items of the attention kernel
    int2 *tile_tab_dev = nullptr;     // fused mode: [P][max_tiles]
    int32_t *tile_cnt_dev = nullptr;  // [P]
    int max_tiles = 0;
    int32_t *status_dev = nullptr;
    float *plan_partials_dev = nullptr;
    uint32_t *sel_bits_dev = nullptr;
    dt::PlannerState *planner_state_dev = nullptr;
    float *planner_local_partials_dev = nullptr;
    float *planner_norm_partials_dev = nullptr;
    float *attn_norm_partials_dev = nullptr;
    void *snap_o = nullptr;
    float *snap_lse = nullptr;
    int planner_group_size = 1;
    double planner_eps_local = 0.0, planner_cache_ratio = 0.0;   // 2 * DT_MAX_P words: composition, planned merge
    void *o_state = nullptr;
    float *lse_state = nullptr;
    cudaStream_t copy_in = nullptr, copy_out = nullptr;   // dt_step_host: H2D and D2H overlap the kernels
    std::vector<cudaEvent_t> events;                       // created on first use
    uint64_t launches = 0;
    std::string err;
    void *encode_tiled = nullptr;  // cuTensorMapEncodeTiled, resolved through the runtime
};
