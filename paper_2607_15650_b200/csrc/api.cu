// C-ABI of libditango: argument checking, tensor-map encoding, launches.  No arithmetic of the
// method lives here.
#include <algorithm>
#include <cmath>
#include <cstddef>
#include <cstdio>
#include <cstring>
#include <new>

#include "dt_internal.h"

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

dt_status fail(dt_ctx *ctx, dt_status s, const char *what) {
    if (ctx) ctx->err = what ? what : "";
    return s;
}

dt_status fail_cuda(dt_ctx *ctx, cudaError_t e, const char *where) {
    if (ctx) ctx->err = std::string(where) + ": " + cudaGetErrorString(e);
    return DT_ERR_CUDA;
}

dt_status check_config(const dt_config *c, const char **why) {
    *why = "";
    if (!c || !c->part_offsets) { *why = "null config or part_offsets"; return DT_ERR_INVALID_ARG; }
    if (c->B < 1 || c->H < 1 || c->L < 1 || c->P < 1) { *why = "B, H, L, P must be positive"; return DT_ERR_INVALID_ARG; }
    if (c->D != 64 && c->D != 128) { *why = "head dim must be 64 or 128"; return DT_ERR_UNSUPPORTED; }
    if (c->P > DT_MAX_P) { *why = "more than 32 partitions"; return DT_ERR_UNSUPPORTED; }
    if (c->state_dtype != DT_STATE_FP32 && c->state_dtype != DT_STATE_BF16) { *why = "unknown state dtype"; return DT_ERR_UNSUPPORTED; }
    if (!(c->softmax_scale > 0.f) || !std::isfinite(c->softmax_scale)) { *why = "softmax_scale must be finite and > 0"; return DT_ERR_INVALID_ARG; }
    if (c->part_offsets[0] != 0 || c->part_offsets[c->P] != c->L) { *why = "offsets must start at 0 and end at L"; return DT_ERR_INVALID_ARG; }
    for (int i = 0; i < c->P; ++i)
        if (c->part_offsets[i + 1] <= c->part_offsets[i]) { *why = "offsets must be strictly increasing"; return DT_ERR_INVALID_ARG; }
    if ((long long)c->B * c->H > 65535) { *why = "B*H exceeds 65535"; return DT_ERR_UNSUPPORTED; }
    if (c->group_size < 0 || c->group_size > c->P) { *why = "group_size must be in [0, P]"; return DT_ERR_INVALID_ARG; }
    if (c->input_dtype != DT_INPUT_BF16 && c->input_dtype != DT_INPUT_FP16) { *why = "unknown input dtype"; return DT_ERR_UNSUPPORTED; }
    return DT_OK;
}

int slots_for(int P, int g) { return g <= 1 ? P : (P + g - 1) / g + 1; }

// Slot table of a context for group size g (g <= 1: pair mode).
void build_slot_table(dt_ctx *ctx, int g) {
    const int P = ctx->cfg.P;
    const std::vector<int32_t> &off = ctx->off;
    const int S = slots_for(P, g);
    ctx->group_size = g <= 1 ? 1 : g;
    ctx->S = S;
    ctx->slot_tab.assign((size_t)P * S, dt::SlotRange{0, 0, 0, 0});
    ctx->members.assign((size_t)P * S, 0);
    ctx->nonempty.assign(P, 0u);
    for (int i = 0; i < P; ++i) {
        for (int s = 0; s < S; ++s) {
            dt::SlotRange r = {0, 0, 0, 0};
            int mem = 0;
            if (g <= 1) {
                r.r1 = off[s]; r.n1 = off[s + 1] - off[s]; mem = 1;
            } else if (s == 0) {
                r.r1 = off[i]; r.n1 = off[i + 1] - off[i]; mem = 1;
            } else {
                const int lo = (s - 1) * g, hi = std::min(P, s * g);   // partitions [lo, hi) of group s - 1
                if (i >= lo && i < hi) {   // the query partition's own group: the keys left and right of it
                    r.r1 = off[lo]; r.n1 = off[i] - off[lo];
                    r.r2 = off[i + 1]; r.n2 = off[hi] - off[i + 1];
                    if (r.n1 == 0) { r.r1 = r.r2; r.n1 = r.n2; r.r2 = 0; r.n2 = 0; }
                    mem = hi - lo - 1;
                } else {
                    r.r1 = off[lo]; r.n1 = off[hi] - off[lo]; mem = hi - lo;
                }
            }
            ctx->slot_tab[(size_t)i * S + s] = r;
            ctx->members[(size_t)i * S + s] = (uint8_t)mem;
            if (r.n1 + r.n2 > 0) ctx->nonempty[i] |= 1u << s;
        }
    }
}

cudaError_t upload_slot_table(dt_ctx *ctx, cudaStream_t st) {
    const size_t n = (size_t)ctx->cfg.P * ctx->S;
    cudaError_t e = cudaMemcpyAsync(ctx->slot_tab_dev, ctx->slot_tab.data(), n * sizeof(dt::SlotRange), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->members_dev, ctx->members.data(), n, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->nonempty_dev, ctx->nonempty.data(), ctx->cfg.P * sizeof(uint32_t), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);   // the host vectors may change right after
    return e;
}

size_t state_elem_bytes(int dtype) { return dtype == DT_STATE_FP32 ? 4 : 2; }

dt_status check_strides(const int64_t s[4], const void *base, const char **why) {
    if (!s) { *why = "null strides"; return DT_ERR_INVALID_ARG; }
    if (s[3] != 1) { *why = "stride of D must be 1"; return DT_ERR_INVALID_ARG; }
    for (int d = 0; d < 3; ++d)
        if (s[d] <= 0 || (s[d] % 8) != 0) { *why = "strides of B, L, H must be positive multiples of 8 elements"; return DT_ERR_INVALID_ARG; }
    if ((reinterpret_cast<uintptr_t>(base) & 15u) != 0) { *why = "tensor base must be 16-byte aligned"; return DT_ERR_INVALID_ARG; }
    return DT_OK;
}

// bf16 [B, L, H, D] viewed as a 4-D tensor map (d, h, l, b); box = 64 elements x 1 head x 128 tokens,
// 128-byte swizzle, out-of-range rows read as zero.
dt_status encode_qkv_map(dt_ctx *ctx, CUtensorMap *tm, const void *base, const int64_t s[4]) {
    const dt_config &c = ctx->cfg;
    cuuint64_t dims[4] = {(cuuint64_t)c.D, (cuuint64_t)c.H, (cuuint64_t)c.L, (cuuint64_t)c.B};
    cuuint64_t strides[3] = {(cuuint64_t)s[2] * 2, (cuuint64_t)s[1] * 2, (cuuint64_t)s[0] * 2};
    cuuint32_t box[4] = {64, 1, (cuuint32_t)dt::ATTN_TILE, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled)(
        tm, c.input_dtype == DT_INPUT_FP16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4,
        const_cast<void *>(base), dims, strides, box, estr,
        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        char buf[96];
        snprintf(buf, sizeof buf, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
        ctx->err = buf;
        return DT_ERR_CUDA;
    }
    return DT_OK;
}

}  // namespace

extern "C" {

const char *dt_status_str(dt_status s) {
    switch (s) {
        case DT_OK: return "DT_OK";
        case DT_ERR_INVALID_ARG: return "DT_ERR_INVALID_ARG";
        case DT_ERR_UNSUPPORTED: return "DT_ERR_UNSUPPORTED";
        case DT_ERR_STATE: return "DT_ERR_STATE";
        case DT_ERR_CUDA: return "DT_ERR_CUDA";
        case DT_ERR_TIMEOUT: return "DT_ERR_TIMEOUT";
        case DT_ERR_RANGE: return "DT_ERR_RANGE";
    }
    return "DT_ERR_UNKNOWN";
}

const char *dt_last_error(dt_ctx *ctx) { return ctx ? ctx->err.c_str() : ""; }

dt_status dt_cache_bytes(const dt_config *cfg, size_t *o_bytes, size_t *lse_bytes) {
    const char *why;
    dt_status s = check_config(cfg, &why);
    if (s != DT_OK) return s;
    if (!o_bytes || !lse_bytes) return DT_ERR_INVALID_ARG;
    const size_t rows = (size_t)slots_for(cfg->P, cfg->group_size) * cfg->B * cfg->H * cfg->L;
    *o_bytes = rows * cfg->D * state_elem_bytes(cfg->state_dtype);
    *lse_bytes = rows * 4;
    return DT_OK;
}

dt_status dt_create(dt_ctx **ctx_out, const dt_config *cfg) {
    if (!ctx_out) return DT_ERR_INVALID_ARG;
    *ctx_out = nullptr;
    const char *why;
    dt_status s = check_config(cfg, &why);
    if (s != DT_OK) return s;
    cudaError_t e = cudaSetDevice(cfg->device);
    if (e != cudaSuccess) return DT_ERR_CUDA;
    cudaDeviceProp prop;
    if ((e = cudaGetDeviceProperties(&prop, cfg->device)) != cudaSuccess) return DT_ERR_CUDA;
    if (prop.major != 10) return DT_ERR_UNSUPPORTED;  // the kernels are built for sm_100a only

    dt_ctx *ctx = new (std::nothrow) dt_ctx();
    if (!ctx) return DT_ERR_CUDA;
    ctx->cfg = *cfg;
    ctx->off.assign(cfg->part_offsets, cfg->part_offsets + cfg->P + 1);
    ctx->cfg.part_offsets = ctx->off.data();
    ctx->num_sms = prop.multiProcessorCount;
    for (int i = 0; i < cfg->P; ++i) ctx->n_max = std::max(ctx->n_max, ctx->off[i + 1] - ctx->off[i]);
    const int qblock = dt::ATTN_NQ * dt::ATTN_TILE;
    ctx->qblocks_max = (ctx->n_max + qblock - 1) / qblock;
    ctx->plan_chunks = (ctx->n_max + dt::PLAN_CHUNK_ROWS - 1) / dt::PLAN_CHUNK_ROWS;

    cudaDriverEntryPointQueryResult qres;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ctx->encode_tiled, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !ctx->encode_tiled) {
        delete ctx;
        return DT_ERR_CUDA;
    }
    const int P = cfg->P, BH = cfg->B * cfg->H;
    build_slot_table(ctx, cfg->group_size);
    ctx->group_size0 = ctx->group_size;
    ctx->S0 = ctx->S;
    ctx->cfg.group_size = ctx->group_size;
    const int S = ctx->S;
    bool ok = true;
    ok = ok && cudaMalloc(&ctx->off_dev, (P + 1) * sizeof(int32_t)) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->slot_tab_dev, (size_t)P * S * sizeof(dt::SlotRange)) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->members_dev, (size_t)P * S) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->nonempty_dev, P * sizeof(uint32_t)) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->tc_dev, P * S * sizeof(int32_t)) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->worklist_dev, (1 + P * S) * sizeof(int32_t)) == cudaSuccess;
    if (ctx->group_size0 <= 1)   // pair mode: at most ceil(P * tiles / 2) items per KV partition
        ok = ok && cudaMalloc(&ctx->tile_pairs_dev, (1 + (size_t)P * (((size_t)P * ctx->qblocks_max * dt::ATTN_NQ + 1) / 2)) * sizeof(int4)) == cudaSuccess;
    ctx->max_tiles = cfg->L / dt::ATTN_TILE + 2 * DT_MAX_P + 4;   // one pass over all keys + one ragged tile per run
    ok = ok && cudaMalloc(&ctx->tile_tab_dev, (size_t)P * ctx->max_tiles * sizeof(int2)) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->tile_cnt_dev, P * sizeof(int32_t)) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->status_dev, sizeof(int32_t)) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->sel_bits_dev, 2 * DT_MAX_P * sizeof(uint32_t)) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->plan_partials_dev, (size_t)BH * P * ctx->plan_chunks * S * sizeof(float)) == cudaSuccess;
    ok = ok && cudaMemcpy(ctx->off_dev, ctx->off.data(), (P + 1) * sizeof(int32_t), cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && upload_slot_table(ctx, nullptr) == cudaSuccess;
    ok = ok && cudaMemset(ctx->tc_dev, 0xFF, P * S * sizeof(int32_t)) == cudaSuccess;  // -1 = empty
    ok = ok && cudaMemset(ctx->worklist_dev, 0, (1 + P * S) * sizeof(int32_t)) == cudaSuccess;
    ok = ok && cudaMemset(ctx->status_dev, 0, sizeof(int32_t)) == cudaSuccess;
    ok = ok && dt::attn_states_configure() == cudaSuccess;
    if (!ok) {
        dt_destroy(ctx);
        return DT_ERR_CUDA;
    }
    *ctx_out = ctx;
    return DT_OK;
}

dt_status dt_destroy(dt_ctx *ctx) {
    if (!ctx) return DT_OK;
    cudaSetDevice(ctx->cfg.device);
    cudaFree(ctx->off_dev);
    cudaFree(ctx->slot_tab_dev);
    cudaFree(ctx->members_dev);
    cudaFree(ctx->nonempty_dev);
    cudaFree(ctx->tc_dev);
    cudaFree(ctx->worklist_dev);
    cudaFree(ctx->tile_pairs_dev);
    cudaFree(ctx->tile_tab_dev);
    cudaFree(ctx->tile_cnt_dev);
    cudaFree(ctx->status_dev);
    cudaFree(ctx->plan_partials_dev);
    cudaFree(ctx->sel_bits_dev);
    cudaFree(ctx->planner_state_dev);
    cudaFree(ctx->planner_local_partials_dev);
    cudaFree(ctx->planner_norm_partials_dev);
    cudaFree(ctx->attn_norm_partials_dev);
    for (cudaEvent_t ev : ctx->events) cudaEventDestroy(ev);
    if (ctx->copy_in) cudaStreamDestroy(ctx->copy_in);
    if (ctx->copy_out) cudaStreamDestroy(ctx->copy_out);
    delete ctx;
    return DT_OK;
}

dt_status dt_bind_cache(dt_ctx *ctx, void *o_state_dev, float *lse_state_dev, size_t o_bytes, size_t lse_bytes) {
    if (!ctx) return DT_ERR_INVALID_ARG;
    if (!o_state_dev || !lse_state_dev) return fail(ctx, DT_ERR_INVALID_ARG, "null cache pointer");
    if ((reinterpret_cast<uintptr_t>(o_state_dev) & 15u) || (reinterpret_cast<uintptr_t>(lse_state_dev) & 15u))
        return fail(ctx, DT_ERR_INVALID_ARG, "cache pointers must be 16-byte aligned");
    const size_t rows0 = (size_t)ctx->S0 * ctx->cfg.B * ctx->cfg.H * ctx->cfg.L;   // slots at creation (a composed cache needs fewer)
    const size_t need_o = rows0 * ctx->cfg.D * state_elem_bytes(ctx->cfg.state_dtype), need_l = rows0 * 4;
    if (o_bytes < need_o || lse_bytes < need_l) return fail(ctx, DT_ERR_STATE, "cache buffers smaller than dt_cache_bytes");
    ctx->o_state = o_state_dev;
    ctx->lse_state = lse_state_dev;
    return DT_OK;
}

namespace {
// mask_dev == nullptr: local (diagonal) pairs only.  Heads [h0, h0 + hc) of every batch entry.
dt_status attn_launch(dt_ctx *ctx, const void *q_dev, const void *k_dev, const void *v_dev, const int64_t strides_blhd[4],
                      const uint8_t *mask_dev, int32_t step, void *stream, int h0 = 0, int hc = -1) {
    if (!q_dev || !k_dev || !v_dev) return fail(ctx, DT_ERR_INVALID_ARG, "null tensor pointer");
    if (step < 0) return fail(ctx, DT_ERR_INVALID_ARG, "step must be >= 0");
    if (!ctx->o_state) return fail(ctx, DT_ERR_STATE, "state cache not bound");
    const char *why;
    for (const void *t : {q_dev, k_dev, v_dev}) {
        dt_status s = check_strides(strides_blhd, t, &why);
        if (s != DT_OK) return fail(ctx, s, why);
    }
    CUtensorMap tq, tk, tv;
    dt_status s;
    if ((s = encode_qkv_map(ctx, &tq, q_dev, strides_blhd)) != DT_OK) return s;
    if ((s = encode_qkv_map(ctx, &tk, k_dev, strides_blhd)) != DT_OK) return s;
    if ((s = encode_qkv_map(ctx, &tv, v_dev, strides_blhd)) != DT_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const dt_config &c = ctx->cfg;
    cudaError_t e = dt::launch_worklist(mask_dev, ctx->tc_dev, ctx->worklist_dev, ctx->status_dev, ctx->slot_tab_dev, c.P,
                                        ctx->S, ctx->group_size0 > 1 ? 1 : 0, step, ctx->off_dev, ctx->tile_pairs_dev, st);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "work-list launch");
    dt::AttnParams p = {};
    p.off = ctx->off_dev;
    p.slot_tab = ctx->slot_tab_dev;
    p.worklist = ctx->worklist_dev;
    p.tile_pairs = ctx->tile_pairs_dev;
    p.status = ctx->status_dev;
    p.o_state = ctx->o_state;
    p.lse_state = ctx->lse_state;
    p.norm_partials = ctx->attn_norm_partials_dev;
    p.B = c.B; p.H = c.H; p.L = c.L; p.P = c.P; p.S = ctx->S;
    p.h0 = h0; p.H_launch = hc < 0 ? c.H : hc;
    p.in_fp16 = c.input_dtype == DT_INPUT_FP16;
    p.qblocks_max = ctx->qblocks_max;
    p.scale_log2 = c.softmax_scale * 1.44269504088896340736f;
    e = dt::launch_attn_states(tq, tk, tv, p, c.D, c.state_dtype, ctx->num_sms, st);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "attention launch");
    ctx->launches += 2;
    return DT_OK;
}
}  // namespace

dt_status dt_attn_states(dt_ctx *ctx, const void *q_dev, const void *k_dev, const void *v_dev,
                         const int64_t strides_blhd[4], const uint8_t *mask_dev, int32_t step, void *stream) {
    if (!ctx) return DT_ERR_INVALID_ARG;
    if (!mask_dev) return fail(ctx, DT_ERR_INVALID_ARG, "null mask pointer");
    return attn_launch(ctx, q_dev, k_dev, v_dev, strides_blhd, mask_dev, step, stream);
}

dt_status dt_attn_local(dt_ctx *ctx, const void *q_dev, const void *k_dev, const void *v_dev,
                        const int64_t strides_blhd[4], int32_t step, void *stream) {
    if (!ctx) return DT_ERR_INVALID_ARG;
    return attn_launch(ctx, q_dev, k_dev, v_dev, strides_blhd, nullptr, step, stream);
}

dt_status dt_attn_fused(dt_ctx *ctx, const void *q_dev, const void *k_dev, const void *v_dev,
                        const int64_t strides_blhd[4], const uint8_t *mask_dev, const void *comp_o_dev,
                        const float *comp_lse_dev, void *out_dev, const int64_t out_strides_blhd[4], float *lse_out_dev,
                        void *stream) {
    if (!ctx) return DT_ERR_INVALID_ARG;
    if (!q_dev || !k_dev || !v_dev || !mask_dev || !out_dev) return fail(ctx, DT_ERR_INVALID_ARG, "null pointer");
    if ((comp_o_dev == nullptr) != (comp_lse_dev == nullptr)) return fail(ctx, DT_ERR_INVALID_ARG, "composed state needs both OUT and LSE");
    if (comp_o_dev && (reinterpret_cast<uintptr_t>(comp_o_dev) & 15u) != 0) return fail(ctx, DT_ERR_INVALID_ARG, "composed state must be 16-byte aligned");
    const char *why;
    for (const void *t : {q_dev, k_dev, v_dev}) {
        dt_status s = check_strides(strides_blhd, t, &why);
        if (s != DT_OK) return fail(ctx, s, why);
    }
    dt_status s = check_strides(out_strides_blhd, out_dev, &why);
    if (s != DT_OK) return fail(ctx, s, why);
    CUtensorMap tq, tk, tv;
    if ((s = encode_qkv_map(ctx, &tq, q_dev, strides_blhd)) != DT_OK) return s;
    if ((s = encode_qkv_map(ctx, &tk, k_dev, strides_blhd)) != DT_OK) return s;
    if ((s = encode_qkv_map(ctx, &tv, v_dev, strides_blhd)) != DT_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const dt_config &c = ctx->cfg;
    cudaError_t e = dt::launch_fused_tiles(mask_dev, ctx->slot_tab_dev, c.P, ctx->S, ctx->max_tiles, ctx->tile_tab_dev,
                                           ctx->tile_cnt_dev, st);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "tile-table launch");
    dt::AttnParams p = {};
    p.off = ctx->off_dev;
    p.slot_tab = ctx->slot_tab_dev;
    p.worklist = ctx->worklist_dev;
    p.status = ctx->status_dev;
    p.B = c.B; p.H = c.H; p.L = c.L; p.P = c.P; p.S = ctx->S;
    p.h0 = 0; p.H_launch = c.H;
    p.in_fp16 = c.input_dtype == DT_INPUT_FP16;
    p.qblocks_max = ctx->qblocks_max;
    p.scale_log2 = c.softmax_scale * 1.44269504088896340736f;
    p.tile_tab = ctx->tile_tab_dev;
    p.tile_cnt = ctx->tile_cnt_dev;
    p.max_tiles = ctx->max_tiles;
    p.comp_o = comp_o_dev;
    p.comp_lse = comp_lse_dev;
    p.out = out_dev;
    p.lse_out = lse_out_dev;
    p.sb = out_strides_blhd[0]; p.sl = out_strides_blhd[1]; p.sh = out_strides_blhd[2];
    e = dt::launch_attn_fused(tq, tk, tv, p, c.D, c.state_dtype, ctx->num_sms, st);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "fused attention launch");
    ctx->launches += 2;
    return DT_OK;
}

namespace {
dt_status merge_rows(dt_ctx *ctx, void *out_dev, const int64_t out_strides_blhd[4], float *lse_out_dev, void *stream,
                     long long row_begin, long long row_count);
}

dt_status dt_state_merge(dt_ctx *ctx, void *out_dev, const int64_t out_strides_blhd[4], float *lse_out_dev,
                         void *stream) {
    if (!ctx) return DT_ERR_INVALID_ARG;
    return merge_rows(ctx, out_dev, out_strides_blhd, lse_out_dev, stream, 0, (long long)ctx->cfg.B * ctx->cfg.H * ctx->cfg.L);
}

namespace {
dt_status merge_rows(dt_ctx *ctx, void *out_dev, const int64_t out_strides_blhd[4], float *lse_out_dev, void *stream,
                     long long row_begin, long long row_count) {
    if (!out_dev) return fail(ctx, DT_ERR_INVALID_ARG, "null output pointer");
    if (!ctx->o_state) return fail(ctx, DT_ERR_STATE, "state cache not bound");
    const char *why;
    dt_status s = check_strides(out_strides_blhd, out_dev, &why);
    if (s != DT_OK) return fail(ctx, s, why);
    const dt_config &c = ctx->cfg;
    dt::MergeParams p = {};
    p.mode = dt::MERGE_ALL;
    if (ctx->group_size0 > 1) {   // a grouped cache has slots that do not exist for some query partitions
        p.sel_bits = ctx->nonempty_dev;
        for (int i = 0; i <= c.P; ++i) p.off_val[i] = ctx->off[i];
    }
    p.o_state = ctx->o_state;
    p.lse_state = ctx->lse_state;
    p.out = out_dev;
    p.lse_out = lse_out_dev;
    p.status = ctx->status_dev;
    p.P = c.P; p.S = ctx->S; p.H = c.H; p.L = c.L;
    p.R = (long long)c.B * c.H * c.L;
    p.row_begin = row_begin; p.row_count = row_count;
    p.out_fp16 = c.input_dtype == DT_INPUT_FP16;
    p.sb = out_strides_blhd[0]; p.sl = out_strides_blhd[1]; p.sh = out_strides_blhd[2];
    cudaError_t e = dt::launch_state_merge(p, c.D, c.state_dtype, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return fail_cuda(ctx, e, "merge launch");
    ctx->launches += 1;
    return DT_OK;
}
}  // namespace

dt_status dt_compose_reuse(dt_ctx *ctx, const uint8_t *mask_dev, void *comp_o_dev, float *comp_lse_dev, void *stream) {
    if (!ctx) return DT_ERR_INVALID_ARG;
    if (!mask_dev || !comp_o_dev || !comp_lse_dev) return fail(ctx, DT_ERR_INVALID_ARG, "null pointer");
    if ((reinterpret_cast<uintptr_t>(comp_o_dev) & 15u) != 0) return fail(ctx, DT_ERR_INVALID_ARG, "composed state must be 16-byte aligned");
    if (!ctx->o_state) return fail(ctx, DT_ERR_STATE, "state cache not bound");
    const dt_config &c = ctx->cfg;
    dt::MergeParams p = {};
    p.mode = dt::MERGE_COMPOSE;
    p.sel_bits = ctx->sel_bits_dev;
    for (int i = 0; i <= c.P; ++i) p.off_val[i] = ctx->off[i];
    cudaError_t es = dt::launch_merge_select(mask_dev, ctx->nonempty_dev, c.P, ctx->S, 0, ctx->sel_bits_dev, static_cast<cudaStream_t>(stream));
    if (es != cudaSuccess) return fail_cuda(ctx, es, "selection launch");
    p.o_state = ctx->o_state;
    p.lse_state = ctx->lse_state;
    p.comp_o_out = comp_o_dev;
    p.comp_lse_out = comp_lse_dev;
    p.status = ctx->status_dev;
    p.P = c.P; p.S = ctx->S; p.H = c.H; p.L = c.L;
    p.R = (long long)c.B * c.H * c.L;
    p.row_begin = 0; p.row_count = p.R;
    cudaError_t e = dt::launch_state_merge(p, c.D, c.state_dtype, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return fail_cuda(ctx, e, "compose launch");
    ctx->launches += 2;
    return DT_OK;
}

dt_status dt_state_merge_planned(dt_ctx *ctx, const uint8_t *mask_dev, const void *comp_o_dev, const float *comp_lse_dev,
                                 void *out_dev, const int64_t out_strides_blhd[4], float *lse_out_dev, void *stream) {
    if (!ctx) return DT_ERR_INVALID_ARG;
    if (!mask_dev || !comp_o_dev || !comp_lse_dev || !out_dev) return fail(ctx, DT_ERR_INVALID_ARG, "null pointer");
    if ((reinterpret_cast<uintptr_t>(comp_o_dev) & 15u) != 0) return fail(ctx, DT_ERR_INVALID_ARG, "composed state must be 16-byte aligned");
    if (!ctx->o_state) return fail(ctx, DT_ERR_STATE, "state cache not bound");
    const char *why;
    dt_status s = check_strides(out_strides_blhd, out_dev, &why);
    if (s != DT_OK) return fail(ctx, s, why);
    const dt_config &c = ctx->cfg;
    dt::MergeParams p = {};
    p.mode = dt::MERGE_PLANNED;
    p.sel_bits = ctx->sel_bits_dev + DT_MAX_P;
    for (int i = 0; i <= c.P; ++i) p.off_val[i] = ctx->off[i];
    cudaError_t es = dt::launch_merge_select(mask_dev, ctx->nonempty_dev, c.P, ctx->S, 1, ctx->sel_bits_dev + DT_MAX_P, static_cast<cudaStream_t>(stream));
    if (es != cudaSuccess) return fail_cuda(ctx, es, "selection launch");
    p.o_state = ctx->o_state;
    p.lse_state = ctx->lse_state;
    p.comp_o = comp_o_dev;
    p.comp_lse = comp_lse_dev;
    p.out = out_dev;
    p.lse_out = lse_out_dev;
    p.status = ctx->status_dev;
    p.P = c.P; p.S = ctx->S; p.H = c.H; p.L = c.L;
    p.R = (long long)c.B * c.H * c.L;
    p.row_begin = 0; p.row_count = p.R;
    p.out_fp16 = c.input_dtype == DT_INPUT_FP16;
    p.sb = out_strides_blhd[0]; p.sl = out_strides_blhd[1]; p.sh = out_strides_blhd[2];
    cudaError_t e = dt::launch_state_merge(p, c.D, c.state_dtype, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return fail_cuda(ctx, e, "planned merge launch");
    ctx->launches += 2;
    return DT_OK;
}

dt_status dt_plan(dt_ctx *ctx, double eps, double target_fraction, uint8_t *mask_dev, double *w_dev,
                  double *eps_out_dev, void *stream) {
    return dt_plan_grouped(ctx, eps, target_fraction, 1, mask_dev, w_dev, eps_out_dev, stream);
}

// The plan computation behind dt_plan, dt_plan_grouped and the two halves of a head-sharded plan:
//   sums_out != null : stage 1 and the fixed-order sums of this context only, written to sums_out
//   sums_in  != null : no stage 1; the plan from sums over `total_bh` (batch, head) slices
static dt_status plan_impl(dt_ctx *ctx, double eps, double target_fraction, int32_t group_size, uint8_t *mask_dev,
                           double *w_dev, double *eps_out_dev, void *stream, const double *sums_in, double *sums_out,
                           long long total_bh) {
    if (group_size < 1 || group_size > ctx->cfg.P) return fail(ctx, DT_ERR_INVALID_ARG, "group_size must be in [1, P]");
    if (ctx->group_size0 > 1 && group_size != 1)
        return fail(ctx, DT_ERR_UNSUPPORTED, "a grouped cache decides per slot: group_size must be 1 here");
    if (!mask_dev && !sums_out) return fail(ctx, DT_ERR_INVALID_ARG, "null mask pointer");
    if (!ctx->lse_state) return fail(ctx, DT_ERR_STATE, "state cache not bound");
    if (target_fraction < 0 && !std::isfinite(eps)) return fail(ctx, DT_ERR_INVALID_ARG, "eps must be finite");
    if (target_fraction > 1.0 || std::isnan(target_fraction)) return fail(ctx, DT_ERR_INVALID_ARG, "target_fraction must be <= 1");
    const dt_config &c = ctx->cfg;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    dt::PlanParams pp;
    pp.lse_state = ctx->lse_state;
    pp.off = ctx->off_dev;
    pp.partials = ctx->plan_partials_dev;
    pp.nonempty = ctx->group_size0 > 1 ? ctx->nonempty_dev : nullptr;
    pp.only_if = nullptr;
    pp.P = c.P; pp.S = ctx->S; pp.BH = c.B * c.H; pp.L = c.L; pp.chunks = ctx->plan_chunks;
    pp.R = (long long)c.B * c.H * c.L;
    cudaError_t e = cudaSuccess;
    if (!sums_in) {
        e = dt::launch_plan_partial(pp, st);
        if (e != cudaSuccess) return fail_cuda(ctx, e, "plan launch");
        ctx->launches += 1;
    }
    if (ctx->group_size0 > 1) {
        dt::PlanSlotsParams ps;
        ps.partials = ctx->plan_partials_dev;
        ps.off = ctx->off_dev;
        ps.slot_tab = ctx->slot_tab_dev;
        ps.members = ctx->members_dev;
        ps.P = c.P; ps.S = ctx->S; ps.BH = pp.BH; ps.chunks = pp.chunks; ps.group_size = ctx->group_size;
        ps.mode_target = target_fraction >= 0 ? 1 : 0;
        int Kp = (int)std::floor(target_fraction * (c.P * c.P) + 0.5);   // the budget is counted in pairs
        ps.K = std::min(std::max(Kp, c.P), c.P * c.P);
        ps.eps = eps;
        ps.mask = mask_dev;
        ps.w_out = w_dev;
        ps.eps_out = eps_out_dev;
        ps.sums_in = sums_in; ps.sums_out = sums_out; ps.count_bh = sums_in ? total_bh : pp.BH;
        e = dt::launch_plan_slots(ps, st);
        if (e != cudaSuccess) return fail_cuda(ctx, e, "plan finalise launch");
        ctx->launches += 1;
        return DT_OK;
    }
    dt::PlanFinalParams pf;
    pf.partials = ctx->plan_partials_dev;
    pf.off = ctx->off_dev;
    pf.P = c.P; pf.BH = pp.BH; pf.chunks = pp.chunks;
    pf.mode_target = target_fraction >= 0 ? 1 : 0;
    const int total = c.P * c.P;
    int K = (int)std::floor(target_fraction * total + 0.5);
    K = std::min(std::max(K, c.P), total);
    pf.K = K;
    pf.group_size = group_size;
    pf.eps = eps;
    pf.mask = mask_dev;
    pf.w_out = w_dev;
    pf.eps_out = eps_out_dev;
    pf.sums_in = sums_in; pf.sums_out = sums_out; pf.count_bh = sums_in ? total_bh : pp.BH;
    e = dt::launch_plan_final(pf, st);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "plan finalise launch");
    ctx->launches += 1;
    return DT_OK;
}

dt_status dt_plan_grouped(dt_ctx *ctx, double eps, double target_fraction, int32_t group_size, uint8_t *mask_dev,
                          double *w_dev, double *eps_out_dev, void *stream) {
    if (!ctx) return DT_ERR_INVALID_ARG;
    return plan_impl(ctx, eps, target_fraction, group_size, mask_dev, w_dev, eps_out_dev, stream, nullptr, nullptr, 0);
}

dt_status dt_plan_sums(dt_ctx *ctx, double *sums_dev, void *stream) {
    if (!ctx) return DT_ERR_INVALID_ARG;
    if (!sums_dev) return fail(ctx, DT_ERR_INVALID_ARG, "null sums pointer");
    return plan_impl(ctx, 0.0, -1.0, 1, nullptr, nullptr, nullptr, stream, nullptr, sums_dev, 0);
}

dt_status dt_plan_from_sums(dt_ctx *ctx, const double *sums_dev, int64_t total_bh, double eps, double target_fraction,
                            int32_t group_size, uint8_t *mask_dev, double *w_dev, double *eps_out_dev, void *stream) {
    if (!ctx) return DT_ERR_INVALID_ARG;
    if (!sums_dev) return fail(ctx, DT_ERR_INVALID_ARG, "null sums pointer");
    if (total_bh < (int64_t)ctx->cfg.B * ctx->cfg.H)
        return fail(ctx, DT_ERR_INVALID_ARG, "total_bh is smaller than this context's own B * H");
    return plan_impl(ctx, eps, target_fraction, group_size, mask_dev, w_dev, eps_out_dev, stream, sums_dev, nullptr, total_bh);
}

dt_status dt_step_host_workspace_bytes(const dt_config *cfg, size_t *bytes) {
    const char *why;
    dt_status s = check_config(cfg, &why);
    if (s != DT_OK) return s;
    if (!bytes) return DT_ERR_INVALID_ARG;
    const size_t elems = (size_t)cfg->B * cfg->L * cfg->H * cfg->D;
    const size_t lse = (((size_t)cfg->B * cfg->H * cfg->L * 4) + 255) & ~(size_t)255;
    *bytes = 4 * ((elems * 2 + 255) & ~(size_t)255) + lse + 1024 /* mask */;
    return DT_OK;
}

#ifndef DT_CHUNK_DIV
#define DT_CHUNK_DIV 16
#endif
#ifndef DT_CHUNK_MIN
#define DT_CHUNK_MIN 2
#endif
constexpr int DT_MAX_HEAD_CHUNKS = 64;

dt_status dt_step_host(dt_ctx *ctx, const void *q_host, const void *k_host, const void *v_host,
                       const uint8_t *mask_host, int32_t step, void *out_host, float *lse_out_host,
                       void *workspace_dev, size_t workspace_bytes, void *stream) {
    if (!ctx) return DT_ERR_INVALID_ARG;
    if (!q_host || !k_host || !v_host || !mask_host || !out_host || !workspace_dev)
        return fail(ctx, DT_ERR_INVALID_ARG, "null pointer");
    size_t need;
    dt_step_host_workspace_bytes(&ctx->cfg, &need);
    if (workspace_bytes < need) return fail(ctx, DT_ERR_INVALID_ARG, "workspace smaller than dt_step_host_workspace_bytes");
    if (reinterpret_cast<uintptr_t>(workspace_dev) & 255u) return fail(ctx, DT_ERR_INVALID_ARG, "workspace must be 256-byte aligned");
    const dt_config &c = ctx->cfg;
    const size_t elems = (size_t)c.B * c.L * c.H * c.D;
    const size_t tb = (elems * 2 + 255) & ~(size_t)255;
    const size_t lse_b = (size_t)c.B * c.H * c.L * 4;
    uint8_t *w = static_cast<uint8_t *>(workspace_dev);
    void *qd = w, *kd = w + tb, *vd = w + 2 * tb, *od = w + 3 * tb;
    float *ld = reinterpret_cast<float *>(w + 4 * tb);
    uint8_t *md = w + 4 * tb + ((lse_b + 255) & ~(size_t)255);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    // Heads are independent, so the step is cut into head chunks: chunk c + 1 is copied in (copy_in stream) and
    // chunk c - 1 copied out (copy_out stream) while chunk c is in the kernels (the caller's stream).
    // About H / DT_CHUNK_DIV heads per chunk while many remain, then smaller ones down to DT_CHUNK_MIN heads: the last
    // chunk's kernels and its copy out overlap nothing, so it should be short, but a chunk of a single head makes for
    // narrow strided copies and a thin launch.
    int bounds[DT_MAX_HEAD_CHUNKS + 1];
    int nchunks = 0;
    {
        const int base = std::max(DT_CHUNK_MIN, (c.H + DT_CHUNK_DIV - 1) / DT_CHUNK_DIV);
        int h = 0;
        bounds[0] = 0;
        while (h < c.H) {
            const int left = c.H - h;
            int sz = std::min(base, std::max(DT_CHUNK_MIN, left / 2));
            if (sz > left || nchunks + 1 == DT_MAX_HEAD_CHUNKS) sz = left;
            h += sz;
            bounds[++nchunks] = h;
        }
    }
    if (!ctx->copy_in) {
        bool ok = cudaStreamCreateWithFlags(&ctx->copy_in, cudaStreamNonBlocking) == cudaSuccess;
        ok = ok && cudaStreamCreateWithFlags(&ctx->copy_out, cudaStreamNonBlocking) == cudaSuccess;
        if (!ok) return fail(ctx, DT_ERR_CUDA, "stream creation failed");
    }
    while ((int)ctx->events.size() < 2 * nchunks + 1) {
        cudaEvent_t ev;
        if ((e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming)) != cudaSuccess) return fail_cuda(ctx, e, "event creation");
        ctx->events.push_back(ev);
    }
    // the copies may not start before earlier work of the caller's stream that uses the workspace has finished
    cudaEvent_t ev_start = ctx->events[2 * nchunks];
    if ((e = cudaEventRecord(ev_start, st)) != cudaSuccess) return fail_cuda(ctx, e, "event record");
    if ((e = cudaStreamWaitEvent(ctx->copy_in, ev_start, 0)) != cudaSuccess) return fail_cuda(ctx, e, "stream wait");
    if ((e = cudaStreamWaitEvent(ctx->copy_out, ev_start, 0)) != cudaSuccess) return fail_cuda(ctx, e, "stream wait");
    if ((e = cudaMemcpyAsync(md, mask_host, (size_t)c.P * ctx->S, cudaMemcpyHostToDevice, st)) != cudaSuccess) return fail_cuda(ctx, e, "copy mask");
    const int64_t strides[4] = {(int64_t)c.L * c.H * c.D, (int64_t)c.H * c.D, c.D, 1};
    const size_t pitch = (size_t)c.H * c.D * 2, rows2d = (size_t)c.B * c.L;
    dt_status s;
    for (int ch = 0; ch < nchunks; ++ch) {
        const int h0 = bounds[ch], h1 = bounds[ch + 1], hc = h1 - h0;
        const size_t col = (size_t)h0 * c.D * 2, width = (size_t)hc * c.D * 2;
        const void *src[3] = {q_host, k_host, v_host};
        void *dst[3] = {qd, kd, vd};
        for (int x = 0; x < 3; ++x)
            if ((e = cudaMemcpy2DAsync(static_cast<uint8_t *>(dst[x]) + col, pitch, static_cast<const uint8_t *>(src[x]) + col, pitch, width,
                                       rows2d, cudaMemcpyHostToDevice, ctx->copy_in)) != cudaSuccess)
                return fail_cuda(ctx, e, "copy q, k, v");
        cudaEvent_t ev_in = ctx->events[2 * ch], ev_done = ctx->events[2 * ch + 1];
        if ((e = cudaEventRecord(ev_in, ctx->copy_in)) != cudaSuccess) return fail_cuda(ctx, e, "event record");
        if ((e = cudaStreamWaitEvent(st, ev_in, 0)) != cudaSuccess) return fail_cuda(ctx, e, "stream wait");
        if ((s = attn_launch(ctx, qd, kd, vd, strides, md, step, stream, h0, hc)) != DT_OK) return s;
        for (int b = 0; b < c.B; ++b)
            if ((s = merge_rows(ctx, od, strides, ld, stream, ((long long)b * c.H + h0) * c.L, (long long)hc * c.L)) != DT_OK) return s;
        if ((e = cudaEventRecord(ev_done, st)) != cudaSuccess) return fail_cuda(ctx, e, "event record");
        if ((e = cudaStreamWaitEvent(ctx->copy_out, ev_done, 0)) != cudaSuccess) return fail_cuda(ctx, e, "stream wait");
        if ((e = cudaMemcpy2DAsync(static_cast<uint8_t *>(out_host) + col, pitch, static_cast<uint8_t *>(od) + col, pitch, width, rows2d,
                                   cudaMemcpyDeviceToHost, ctx->copy_out)) != cudaSuccess)
            return fail_cuda(ctx, e, "copy out");
        if (lse_out_host)
            for (int b = 0; b < c.B; ++b) {
                const size_t o = ((size_t)b * c.H + h0) * c.L;
                if ((e = cudaMemcpyAsync(lse_out_host + o, ld + o, (size_t)hc * c.L * 4, cudaMemcpyDeviceToHost, ctx->copy_out)) != cudaSuccess)
                    return fail_cuda(ctx, e, "copy lse");
            }
    }
    if ((e = cudaStreamSynchronize(ctx->copy_out)) != cudaSuccess) return fail_cuda(ctx, e, "synchronise");
    if ((e = cudaStreamSynchronize(st)) != cudaSuccess) return fail_cuda(ctx, e, "synchronise");
    return DT_OK;
}

dt_status dt_get_tc(dt_ctx *ctx, int32_t *tc_host) {
    if (!ctx || !tc_host) return DT_ERR_INVALID_ARG;
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpy(tc_host, ctx->tc_dev, ctx->cfg.P * ctx->S * sizeof(int32_t), cudaMemcpyDeviceToHost);
    return e == cudaSuccess ? DT_OK : fail_cuda(ctx, e, "dt_get_tc");
}

dt_status dt_set_tc(dt_ctx *ctx, const int32_t *tc_host) {
    if (!ctx || !tc_host) return DT_ERR_INVALID_ARG;
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpy(ctx->tc_dev, tc_host, ctx->cfg.P * ctx->S * sizeof(int32_t), cudaMemcpyHostToDevice);
    return e == cudaSuccess ? DT_OK : fail_cuda(ctx, e, "dt_set_tc");
}

dt_status dt_launch_count(dt_ctx *ctx, uint64_t *count) {
    if (!ctx || !count) return DT_ERR_INVALID_ARG;
    *count = ctx->launches;
    return DT_OK;
}

namespace {
dt::PlannerParams planner_params(dt_ctx *ctx) {
    const dt_config &c = ctx->cfg;
    dt::PlannerParams p = {};
    p.state = ctx->planner_state_dev;
    p.o_state = ctx->o_state;
    p.lse_state = ctx->lse_state;
    p.snap_o = ctx->snap_o;
    p.snap_lse = ctx->snap_lse;
    p.snap_o_out = ctx->snap_o;
    p.snap_lse_out = ctx->snap_lse;
    p.off = ctx->off_dev;
    p.nonempty = ctx->nonempty_dev;
    p.local_partials = ctx->planner_local_partials_dev;
    p.norm_partials = ctx->planner_norm_partials_dev;
    p.attn_norm_partials = ctx->attn_norm_partials_dev;
    p.qblocks = ctx->qblocks_max;
    p.w_partials = ctx->plan_partials_dev;
    p.P = c.P; p.S = ctx->S; p.BH = c.B * c.H; p.L = c.L; p.D = c.D; p.chunks = ctx->plan_chunks;
    p.group_size = ctx->planner_group_size;
    p.group_mode = ctx->group_size0 > 1 ? 1 : 0;
    p.force = 0;
    p.eps_local = ctx->planner_eps_local;
    p.cache_ratio = ctx->planner_cache_ratio;
    return p;
}
}  // namespace

dt_status dt_planner_init(dt_ctx *ctx, const dt_planner_config *pc, void *snap_o_dev, float *snap_lse_dev,
                          size_t snap_o_bytes, size_t snap_lse_bytes, void *stream) {
    if (!ctx) return DT_ERR_INVALID_ARG;
    if (!pc || !snap_o_dev || !snap_lse_dev) return fail(ctx, DT_ERR_INVALID_ARG, "null pointer");
    const dt_config &c = ctx->cfg;
    if (pc->group_size < 1 || pc->group_size > c.P) return fail(ctx, DT_ERR_INVALID_ARG, "group_size must be in [1, P]");
    if (ctx->group_size0 > 1 && pc->group_size != 1)
        return fail(ctx, DT_ERR_UNSUPPORTED, "a grouped cache decides per slot: dt_planner_config.group_size must be 1");
    if (!(pc->eps_initial >= 0.0) || !(pc->eps_local > 0.0) || !(pc->cache_ratio >= 0.0 && pc->cache_ratio <= 1.0))
        return fail(ctx, DT_ERR_INVALID_ARG, "eps_initial >= 0, eps_local > 0 and 0 <= cache_ratio <= 1 required");
    if ((long long)c.B * c.H * c.P > 65535) return fail(ctx, DT_ERR_UNSUPPORTED, "B*H*P exceeds 65535");
    const size_t rows = (size_t)c.B * c.H * c.L;
    if (snap_o_bytes < rows * c.D * state_elem_bytes(c.state_dtype) || snap_lse_bytes < rows * 4)
        return fail(ctx, DT_ERR_STATE, "snapshot buffers smaller than one cache slot");
    if ((reinterpret_cast<uintptr_t>(snap_o_dev) & 15u) != 0) return fail(ctx, DT_ERR_INVALID_ARG, "snapshot must be 16-byte aligned");
    if (!ctx->planner_state_dev) {
        const size_t BH = (size_t)c.B * c.H;
        bool ok = cudaMalloc(&ctx->planner_state_dev, sizeof(dt::PlannerState)) == cudaSuccess;
        ok = ok && cudaMalloc(&ctx->planner_local_partials_dev, BH * c.P * ctx->plan_chunks * 2 * sizeof(float)) == cudaSuccess;
        ok = ok && cudaMalloc(&ctx->planner_norm_partials_dev, BH * c.P * ctx->plan_chunks * ctx->S0 * sizeof(float)) == cudaSuccess;
        const size_t attn_norm_bytes = BH * c.P * ctx->S0 * ctx->qblocks_max * (dt::ATTN_NQ * 4) * sizeof(float);
        ok = ok && cudaMalloc(&ctx->attn_norm_partials_dev, attn_norm_bytes) == cudaSuccess;
        ok = ok && cudaMemsetAsync(ctx->attn_norm_partials_dev, 0, attn_norm_bytes, static_cast<cudaStream_t>(stream)) == cudaSuccess;
        if (!ok) return fail(ctx, DT_ERR_CUDA, "planner scratch allocation failed");
    }
    ctx->snap_o = snap_o_dev;
    ctx->snap_lse = snap_lse_dev;
    ctx->planner_group_size = pc->group_size;
    ctx->planner_eps_local = pc->eps_local;
    ctx->planner_cache_ratio = pc->cache_ratio;
    cudaError_t e = dt::launch_planner_init(ctx->planner_state_dev, pc->eps_initial, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return fail_cuda(ctx, e, "planner init launch");
    ctx->launches += 1;
    return DT_OK;
}

dt_status dt_planner_step(dt_ctx *ctx, uint8_t *mask_dev, int32_t *is_anchor_dev, double *ase_dev, double *delta_rel_dev,
                          void *stream) {
    if (!ctx) return DT_ERR_INVALID_ARG;
    if (!mask_dev) return fail(ctx, DT_ERR_INVALID_ARG, "null mask pointer");
    if (!ctx->planner_state_dev) return fail(ctx, DT_ERR_STATE, "dt_planner_init has not been called");
    if (!ctx->o_state) return fail(ctx, DT_ERR_STATE, "state cache not bound");
    dt::PlannerParams p = planner_params(ctx);
    p.mask = mask_dev;
    p.is_anchor_out = is_anchor_dev;
    p.ase_out = ase_dev;
    p.delta_rel_out = delta_rel_dev;
    cudaError_t e = dt::launch_planner_step(p, ctx->cfg.state_dtype, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return fail_cuda(ctx, e, "planner step launch");
    ctx->launches += 2;
    return DT_OK;
}

dt_status dt_planner_commit(dt_ctx *ctx, void *stream) {
    if (!ctx) return DT_ERR_INVALID_ARG;
    if (!ctx->planner_state_dev) return fail(ctx, DT_ERR_STATE, "dt_planner_init has not been called");
    const dt_config &c = ctx->cfg;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    dt::PlanParams pp;
    pp.lse_state = ctx->lse_state;
    pp.off = ctx->off_dev;
    pp.partials = ctx->plan_partials_dev;
    pp.nonempty = ctx->group_size0 > 1 ? ctx->nonempty_dev : nullptr;
    pp.only_if = nullptr;
    pp.P = c.P; pp.S = ctx->S; pp.BH = c.B * c.H; pp.L = c.L; pp.chunks = ctx->plan_chunks;
    pp.R = (long long)c.B * c.H * c.L;
    pp.only_if = &ctx->planner_state_dev->is_anchor;   // Eq. 8's weights are refreshed at anchors only
    cudaError_t e = dt::launch_plan_partial(pp, st);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "plan launch");
    dt::PlannerParams p = planner_params(ctx);
    e = dt::launch_planner_commit(p, c.state_dtype, st);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "planner commit launch");
    ctx->launches += 4;
    return DT_OK;
}

dt_status dt_planner_get(dt_ctx *ctx, double *w_host, double *alpha_host, double *eps_host, int32_t *have_anchor_host) {
    if (!ctx) return DT_ERR_INVALID_ARG;
    if (!ctx->planner_state_dev) return fail(ctx, DT_ERR_STATE, "dt_planner_init has not been called");
    dt::PlannerState hs;
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpy(&hs, ctx->planner_state_dev, sizeof hs, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "dt_planner_get");
    const int n = ctx->cfg.P * ctx->S;
    if (w_host) memcpy(w_host, hs.w, n * sizeof(double));
    if (alpha_host) memcpy(alpha_host, hs.alpha, n * sizeof(double));
    if (eps_host) *eps_host = hs.eps;
    if (have_anchor_host) *have_anchor_host = hs.have_anchor;
    return DT_OK;
}

dt_status dt_num_slots(dt_ctx *ctx, int32_t *slots, int32_t *group_size) {
    if (!ctx) return DT_ERR_INVALID_ARG;
    if (slots) *slots = ctx->S;
    if (group_size) *group_size = ctx->group_size;
    return DT_OK;
}

dt_status dt_slot_ranges(dt_ctx *ctx, int32_t *ranges_host) {
    if (!ctx || !ranges_host) return DT_ERR_INVALID_ARG;
    memcpy(ranges_host, ctx->slot_tab.data(), ctx->slot_tab.size() * sizeof(dt::SlotRange));
    return DT_OK;
}

dt_status dt_group_compose(dt_ctx *ctx, void *stream) {
    if (!ctx) return DT_ERR_INVALID_ARG;
    if (ctx->group_size0 <= 1) return fail(ctx, DT_ERR_UNSUPPORTED, "dt_group_compose needs a grouped cache (dt_config.group_size >= 2)");
    if (!ctx->o_state) return fail(ctx, DT_ERR_STATE, "state cache not bound");
    const int m_old = ctx->S - 1;
    if (m_old < 2) return fail(ctx, DT_ERR_STATE, "one group left: nothing to compose");
    const dt_config &c = ctx->cfg;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int S_old = ctx->S, m_new = (m_old + 1) / 2, S_new = m_new + 1;
    const size_t R = (size_t)c.B * c.H * c.L;
    const size_t esz = state_elem_bytes(c.state_dtype);
    // new slot 1 + k <- old slots 1 + 2k and 2 + 2k, in ascending k: a block reads its rows of both sources
    // before it writes the same rows of slot 1 + k <= 1 + 2k, and later slots only read higher ones
    for (int k = 0; k < m_new; ++k) {
        std::vector<uint32_t> sel(c.P);
        uint32_t bits = 1u << (1 + 2 * k);
        if (2 + 2 * k < S_old) bits |= 1u << (2 + 2 * k);
        for (int i = 0; i < c.P; ++i) sel[i] = bits & ctx->nonempty[i];
        cudaError_t e = cudaMemcpyAsync(ctx->sel_bits_dev, sel.data(), c.P * sizeof(uint32_t), cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);   // `sel` is a temporary
        if (e != cudaSuccess) return fail_cuda(ctx, e, "group compose selection");
        dt::MergeParams p = {};
        p.mode = dt::MERGE_COMPOSE;
        p.sel_bits = ctx->sel_bits_dev;
        for (int i = 0; i <= c.P; ++i) p.off_val[i] = ctx->off[i];
        p.o_state = ctx->o_state;
        p.lse_state = ctx->lse_state;
        p.comp_o_out = static_cast<uint8_t *>(ctx->o_state) + (size_t)(1 + k) * R * c.D * esz;
        p.comp_lse_out = ctx->lse_state + (size_t)(1 + k) * R;
        p.status = ctx->status_dev;
        p.P = c.P; p.S = S_old; p.H = c.H; p.L = c.L;
        p.R = (long long)R;
        p.row_begin = 0; p.row_count = p.R;
        e = dt::launch_state_merge(p, c.D, c.state_dtype, st);
        if (e != cudaSuccess) return fail_cuda(ctx, e, "group compose launch");
        ctx->launches += 1;
    }
    cudaError_t e = dt::launch_tc_compose(ctx->tc_dev, ctx->nonempty_dev, c.P, S_old, S_new, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);   // t_c is rewritten from the old table before it changes
    if (e != cudaSuccess) return fail_cuda(ctx, e, "group compose t_c");
    ctx->launches += 1;
    build_slot_table(ctx, ctx->group_size * 2);
    e = upload_slot_table(ctx, st);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "group compose table upload");
    if (ctx->planner_state_dev) {
        // the planner's w and alpha are indexed by slot: take them again from the composed cache (the importance
        // of a composed slot is the sum of its sources', its scale ratio needs the composed state's norm)
        dt::PlanParams pp;
        pp.lse_state = ctx->lse_state;
        pp.off = ctx->off_dev;
        pp.partials = ctx->plan_partials_dev;
        pp.nonempty = ctx->nonempty_dev;
        pp.only_if = nullptr;
        pp.P = c.P; pp.S = ctx->S; pp.BH = c.B * c.H; pp.L = c.L; pp.chunks = ctx->plan_chunks;
        pp.R = (long long)R;
        e = dt::launch_plan_partial(pp, st);
        if (e != cudaSuccess) return fail_cuda(ctx, e, "plan launch");
        dt::PlannerParams p = planner_params(ctx);
        p.force = 1;
        e = dt::launch_planner_commit(p, c.state_dtype, st);
        if (e != cudaSuccess) return fail_cuda(ctx, e, "planner refresh launch");
        ctx->launches += 3;
    }
    return DT_OK;
}

dt_status dt_group_fit(dt_ctx *ctx, size_t max_bytes, int32_t *composed, void *stream) {
    if (!ctx) return DT_ERR_INVALID_ARG;
    if (composed) *composed = 0;
    if (ctx->group_size0 <= 1) return fail(ctx, DT_ERR_UNSUPPORTED, "dt_group_fit needs a grouped cache (dt_config.group_size >= 2)");
    const dt_config &c = ctx->cfg;
    const size_t per_slot = (size_t)c.B * c.H * c.L * (c.D * state_elem_bytes(c.state_dtype) + 4);
    int n = 0;
    while ((size_t)ctx->S * per_slot > max_bytes && ctx->S - 1 >= 2) {
        dt_status s = dt_group_compose(ctx, stream);
        if (s != DT_OK) return s;
        ++n;
    }
    if (composed) *composed = n;
    return (size_t)ctx->S * per_slot > max_bytes ? fail(ctx, DT_ERR_STATE, "one group left and the cache is still above the budget") : DT_OK;
}

dt_status dt_group_reset(dt_ctx *ctx, void *stream) {
    if (!ctx) return DT_ERR_INVALID_ARG;
    if (ctx->group_size0 <= 1) return fail(ctx, DT_ERR_UNSUPPORTED, "dt_group_reset needs a grouped cache (dt_config.group_size >= 2)");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "group reset");
    build_slot_table(ctx, ctx->group_size0);
    e = upload_slot_table(ctx, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(ctx->tc_dev, 0xFF, (size_t)ctx->cfg.P * ctx->S * sizeof(int32_t), st);
    if (e == cudaSuccess && ctx->planner_state_dev)   // the planner starts over: its next step is an anchor
        e = cudaMemsetAsync(reinterpret_cast<uint8_t *>(ctx->planner_state_dev) + offsetof(dt::PlannerState, have_anchor), 0,
                            sizeof(int), st);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "group reset");
    return DT_OK;
}

dt_status dt_selftest_wait_timeout(dt_ctx *ctx, uint32_t limit_us, void *stream) {
    if (!ctx) return DT_ERR_INVALID_ARG;
    if (limit_us == 0 || limit_us > 100000) return fail(ctx, DT_ERR_INVALID_ARG, "limit_us must be in [1, 100000]");
    const long long cycles = (long long)limit_us * 2000;   // about 2 GHz
    cudaError_t e = dt::launch_wait_timeout_selftest(ctx->status_dev, cycles, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return fail_cuda(ctx, e, "self-test launch");
    ctx->launches += 1;
    return DT_OK;
}

dt_status dt_poll(dt_ctx *ctx) {
    if (!ctx) return DT_ERR_INVALID_ARG;
    int32_t word = 0;
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpy(&word, ctx->status_dev, sizeof word, cudaMemcpyDeviceToHost);
    if (e == cudaSuccess && word != 0) e = cudaMemset(ctx->status_dev, 0, sizeof word);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "dt_poll");
    if (word & dt::STATUS_WAIT_TIMEOUT) return fail(ctx, DT_ERR_TIMEOUT, "a bounded device-side wait expired");
    if (word & dt::STATUS_REUSE_EMPTY) return fail(ctx, DT_ERR_STATE, "REUSE of a pair that was never computed");
    if (word & dt::STATUS_LOGIT_RANGE)
        return fail(ctx, DT_ERR_RANGE, "a logit rose more than 100 binades above the running reference within one K/V tile");
    return DT_OK;
}

}  // extern "C"
