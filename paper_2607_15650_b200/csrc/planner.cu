// Anchor-guided selection planning on the device (Section 4, Algorithm 1).
//
// State kept in the context (device memory): partition importance weights w (Eq. 8) and scale ratios
// alpha (Eq. 9) of the last anchor, the threshold eps, and two flags (an anchor exists / this step is
// one).  The caller keeps a snapshot of the local (diagonal) states of the last anchor.
//
// Per step, after the local pairs of the step have been computed:
//   planner_local_kernel   ||AS_t(i,i) - AS_ta(i,i)||^2 and ||AS_ta(i,i)||^2 per query partition i
//                          (the state is OUT and LSE stacked), streamed with fixed-order partial sums;
//   planner_decide_kernel  delta(i) (Eq. 10's factor), ASE per unit (Eq. 7, 10, 12), anchor test (Eq. 14),
//                          COMPUTE / REUSE mask (Eq. 13), and on an anchor the new eps (R-quantile of the
//                          units' predicted errors).
// After the step's attention, if the step was an anchor (device flag; no host round trip):
//   plan_partial_kernel + planner_norm_kernel + planner_commit_kernel refresh w and alpha from the cache,
//   planner_snapshot_kernel copies the local states into the snapshot.
// No atomics: results are bit-reproducible.
#include <cuda_bf16.h>

#include "dt_internal.h"

namespace dt {
namespace {

constexpr int PL_THREADS = 256;

// 16 bytes of state elements as fp32 values: 4 (fp32 cache) or 8 (bf16 cache)
template <typename T>
struct Vec16;
template <>
struct Vec16<float> {
    static constexpr int N = 4;
    __device__ static __forceinline__ void load(const float *p, float (&v)[4]) {
        const float4 x = __ldcs(reinterpret_cast<const float4 *>(p));
        v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
    }
};
template <>
struct Vec16<__nv_bfloat16> {
    static constexpr int N = 8;
    __device__ static __forceinline__ void load(const __nv_bfloat16 *p, float (&v)[8]) {
        const uint4 x = __ldcs(reinterpret_cast<const uint4 *>(p));
        const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            v[2 * e] = __uint_as_float(w[e] << 16);
            v[2 * e + 1] = __uint_as_float(w[e] & 0xFFFF0000u);
        }
    }
};

// fixed-order block sum of two values per thread; result valid in thread 0
__device__ __forceinline__ void block_sum2(float &a, float &b) {
    __shared__ float red[2][PL_THREADS / 32];
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) {
        a += __shfl_xor_sync(0xFFFFFFFFu, a, s);
        b += __shfl_xor_sync(0xFFFFFFFFu, b, s);
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { red[0][warp] = a; red[1][warp] = b; }
    __syncthreads();
    if (threadIdx.x == 0) {
        a = 0.f; b = 0.f;
        for (int w = 0; w < PL_THREADS / 32; ++w) { a += red[0][w]; b += red[1][w]; }
    }
}

// grid (chunks, P, BH): rows [off_i + c*CH, ...) of the local state (slot i) against the snapshot
template <typename StateT>
__global__ void __launch_bounds__(PL_THREADS) planner_local_kernel(PlannerParams p) {
    const int c = blockIdx.x, i = blockIdx.y, bh = blockIdx.z;
    const int row0 = p.off[i] + c * PLAN_CHUNK_ROWS, row1 = min(row0 + PLAN_CHUNK_ROWS, p.off[i + 1]);
    const int ls = p.group_mode ? 0 : i;                          // slot of the local state
    const long long slot = ((long long)ls * p.BH + bh) * p.L;     // row index base of that slot in the cache
    const long long snap = (long long)bh * p.L;                   // row index base in the snapshot
    const StateT *o = static_cast<const StateT *>(p.o_state), *so = static_cast<const StateT *>(p.snap_o);
    float diff = 0.f, base = 0.f;
    const long long n = (long long)max(row1 - row0, 0) * p.D;      // the rows are contiguous in both buffers
    const StateT *cur = o + (slot + row0) * p.D, *old = so + (snap + row0) * p.D;
    constexpr int V = Vec16<StateT>::N;        // rows are multiples of 16 bytes and start on such a boundary
    for (long long e = (long long)threadIdx.x * V; e < n; e += (long long)PL_THREADS * V) {
        float a[V], b[V];
        Vec16<StateT>::load(cur + e, a);
        Vec16<StateT>::load(old + e, b);
#pragma unroll
        for (int u = 0; u < V; ++u) {
            diff = fmaf(a[u] - b[u], a[u] - b[u], diff);
            base = fmaf(b[u], b[u], base);
        }
    }
    for (int r = row0 + (int)threadIdx.x; r < row1; r += PL_THREADS) {
        const float a = p.lse_state[slot + r], b = p.snap_lse[snap + r];
        diff += (a - b) * (a - b);
        base += b * b;
    }
    block_sum2(diff, base);
    if (threadIdx.x == 0) {
        float *dst = p.local_partials + (((long long)bh * p.P + i) * p.chunks + c) * 2;
        dst[0] = diff;
        dst[1] = base;
    }
}

__device__ __forceinline__ bool asc_before(double ma, int fa, double mb, int fb) {
    if (ma != mb) return ma < mb;
    return fa < fb;
}

__global__ void __launch_bounds__(1024) planner_decide_kernel(PlannerParams p) {
    __shared__ double delta_s[DT_MAX_P];
    __shared__ double ase_s[DT_MAX_P * DT_MAX_P];
    __shared__ uint8_t valid_s[DT_MAX_P * DT_MAX_P];
    __shared__ double tot[2];
    __shared__ double edge[2];
    __shared__ int anchor_s;
    // pair mode: unit (i, k) = the k-th group of g adjacent slots without the local one; grouped cache: unit
    // (i, s) = slot s != 0, one state with one weight and one scale ratio
    const int P = p.P, S = p.S, g = p.group_mode ? 1 : p.group_size;
    const int ng = p.group_mode ? S : (P + g - 1) / g, nunits = P * ng;
    const int e = threadIdx.x;
    PlannerState *st = p.state;
    if (e < P) {
        double d = 0.0, b = 0.0;
        for (int bh = 0; bh < p.BH; ++bh)
            for (int c = 0; c < p.chunks; ++c) {
                const float *src = p.local_partials + (((long long)bh * P + e) * p.chunks + c) * 2;
                d += (double)src[0];
                b += (double)src[1];
            }
        delta_s[e] = sqrt(d);
        ase_s[e] = d;            // reused below as scratch for the totals
        ase_s[DT_MAX_P + e] = b;
    }
    if (e < 2) edge[e] = 0.0;
    __syncthreads();
    if (e == 0) {
        double d = 0.0, b = 0.0;
        for (int i = 0; i < P; ++i) { d += ase_s[i]; b += ase_s[DT_MAX_P + i]; }
        tot[0] = d;
        tot[1] = b;
    }
    __syncthreads();
    const int ui = e / ng, uk = e - ui * ng;
    double ase = 0.0;
    bool valid = false;
    if (e < nunits) {
        if (p.group_mode) {
            if (uk != 0 && (p.nonempty[ui] >> uk & 1u)) { ase = st->w[e] * st->alpha[e] * delta_s[ui]; valid = true; }
        } else {
            const int lo = uk * g, hi = min(P, (uk + 1) * g);
            for (int j = lo; j < hi; ++j)
                if (j != ui) { ase += st->w[ui * P + j] * st->alpha[ui * P + j] * delta_s[ui]; valid = true; }
        }
    }
    __syncthreads();
    if (e < nunits) { ase_s[e] = ase; valid_s[e] = valid ? 1 : 0; }
    const double eps = st->eps;
    const int n_valid = __syncthreads_count(valid);
    const int n_exceed = __syncthreads_count(valid && ase > eps);
    const int n_pos = __syncthreads_count(valid && ase > 0.0);
    if (e == 0) {
        const double delta_rel = tot[1] > 0.0 ? sqrt(tot[0] / tot[1]) : 0.0;
        const bool all_exceed = n_valid > 0 && n_exceed == n_valid;
        anchor_s = (!st->have_anchor || all_exceed || delta_rel > p.eps_local) ? 1 : 0;
        if (p.delta_rel_out) *p.delta_rel_out = delta_rel;
    }
    __syncthreads();
    const int is_anchor = anchor_s;
    if (is_anchor && n_pos > 0) {
        // eps <- R-quantile of the valid units' ASE: rank them ascending, midpoint of ranks r-1 and r
        int r = (int)floor(p.cache_ratio * (double)n_valid);
        r = min(max(r, 0), n_valid);
        if (valid) {
            int rank = 0;
            for (int o = 0; o < nunits; ++o)
                if (o != e && valid_s[o] && asc_before(ase_s[o], o, ase, e)) ++rank;
            if (rank == r - 1) edge[0] = ase;
            if (rank == r) edge[1] = ase;
        }
        __syncthreads();
        if (e == 0) st->eps = (r == 0) ? 0.0 : (r == n_valid ? edge[0] : 0.5 * (edge[0] + edge[1]));
    }
    if (e < P * S) {
        const int i = e / S, j = e - i * S;
        const bool local = p.group_mode ? (j == 0) : (i == j);
        const int unit = p.group_mode ? e : i * ng + j / g;
        p.mask[e] = (is_anchor || local || (valid_s[unit] && ase_s[unit] > eps)) ? 1 : 0;
    }
    if (e < nunits && p.ase_out) p.ase_out[e] = valid ? ase : nan("");
    if (e == 0) {
        st->is_anchor = is_anchor;
        if (p.is_anchor_out) *p.is_anchor_out = is_anchor;
    }
}

// grid (chunks, P * S (query partition i, slot j), BH): sum of squares of the state rows of a composed cache
template <typename StateT>
__global__ void __launch_bounds__(PL_THREADS) planner_norm_kernel(PlannerParams p) {
    const int c = blockIdx.x, i = blockIdx.y / p.S, j = blockIdx.y - i * p.S, bh = blockIdx.z;
    if (!(p.nonempty[i] >> j & 1u)) {   // no such slot for this query partition
        if (threadIdx.x == 0) p.norm_partials[(((long long)bh * p.P + i) * p.chunks + c) * p.S + j] = 0.f;
        return;
    }
    const int row0 = p.off[i] + c * PLAN_CHUNK_ROWS, row1 = min(row0 + PLAN_CHUNK_ROWS, p.off[i + 1]);
    const long long slot = ((long long)j * p.BH + bh) * p.L;
    const StateT *o = static_cast<const StateT *>(p.o_state);
    float sq = 0.f, unused = 0.f;
    const long long n = (long long)max(row1 - row0, 0) * p.D;
    const StateT *src = o + (slot + row0) * p.D;
    constexpr int V = Vec16<StateT>::N;
    for (long long e = (long long)threadIdx.x * V; e < n; e += (long long)PL_THREADS * V) {
        float a[V];
        Vec16<StateT>::load(src + e, a);
#pragma unroll
        for (int u = 0; u < V; ++u) sq = fmaf(a[u], a[u], sq);
    }
    for (int r = row0 + (int)threadIdx.x; r < row1; r += PL_THREADS) {
        const float a = p.lse_state[slot + r];
        sq += a * a;
    }
    block_sum2(sq, unused);
    if (threadIdx.x == 0) p.norm_partials[(((long long)bh * p.P + i) * p.chunks + c) * p.S + j] = sq;
}

// grid P * S, one block per (query partition i, slot j): ||AS(i, j)||^2 of an anchor, which has computed every state,
// as the sum of the attention epilogue's partials in a fixed order (thread-strided sums, then a fixed tree)
__global__ void __launch_bounds__(PL_THREADS) planner_attn_norm_kernel(PlannerParams p) {
    PlannerState *st = p.state;
    if (!st->is_anchor) return;
    __shared__ double red[PL_THREADS];
    const int e = blockIdx.x, i = e / p.S, j = e - i * p.S;
    const int per_item = p.qblocks * (ATTN_NQ * 4);
    double acc = 0.0;
    if (p.nonempty[i] >> j & 1u) {
        const long long total = (long long)p.BH * per_item;
        for (long long k = threadIdx.x; k < total; k += PL_THREADS) {
            const long long bh = k / per_item, r = k - bh * per_item;
            acc += (double)p.attn_norm_partials[((bh * p.P + i) * p.S + j) * per_item + r];
        }
    }
    red[threadIdx.x] = acc;
    __syncthreads();
    for (int s = PL_THREADS / 2; s > 0; s >>= 1) {
        if ((int)threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
        __syncthreads();
    }
    if (threadIdx.x == 0) st->nsq[e] = red[0];
}

// one block: w (Eq. 8, mean over rows and heads) and alpha (Eq. 9) from the partial sums; anchor steps only
__global__ void __launch_bounds__(1024) planner_commit_kernel(PlannerParams p) {
    PlannerState *st = p.state;
    if (!p.force && !st->is_anchor) return;
    __shared__ double nsq[DT_MAX_P * DT_MAX_P];
    const int P = p.P, S = p.S, e = threadIdx.x;
    const int i = e / S, j = e - i * S;
    if (e < P * S) {
        double w = 0.0, n = 0.0;
        for (int bh = 0; bh < p.BH; ++bh)
            for (int c = 0; c < p.chunks; ++c) {
                const long long idx = (((long long)bh * P + i) * p.chunks + c) * S + j;
                w += (double)p.w_partials[idx];
                if (p.force) n += (double)p.norm_partials[idx];
            }
        if (!p.force) n = st->nsq[e];   // from planner_attn_norm_kernel
        st->w[e] = w / ((double)p.BH * (double)(p.off[i + 1] - p.off[i]));
        nsq[e] = n;
    }
    __syncthreads();
    if (e < P * S) st->alpha[e] = sqrt(nsq[e] / nsq[i * S + (p.group_mode ? 0 : i)]);
    if (e == 0 && !p.force) st->have_anchor = 1;
}

// copies the local states (slot i, rows of partition i) into the snapshot; anchor steps only
template <typename StateT>
__global__ void __launch_bounds__(PL_THREADS) planner_snapshot_kernel(PlannerParams p) {
    if (!p.state->is_anchor) return;
    const int c = blockIdx.x, i = blockIdx.y, bh = blockIdx.z;
    const int row0 = p.off[i] + c * PLAN_CHUNK_ROWS, row1 = min(row0 + PLAN_CHUNK_ROWS, p.off[i + 1]);
    if (row1 <= row0) return;
    const long long slot = ((long long)(p.group_mode ? 0 : i) * p.BH + bh) * p.L, snap = (long long)bh * p.L;
    const uint4 *src = reinterpret_cast<const uint4 *>(static_cast<const StateT *>(p.o_state) + (slot + row0) * p.D);
    uint4 *dst = reinterpret_cast<uint4 *>(static_cast<StateT *>(p.snap_o_out) + (snap + row0) * p.D);
    const long long n16 = (long long)(row1 - row0) * p.D * (long long)sizeof(StateT) / 16;
    for (long long e = threadIdx.x; e < n16; e += PL_THREADS) dst[e] = src[e];
    for (int r = row0 + (int)threadIdx.x; r < row1; r += PL_THREADS) p.snap_lse_out[snap + r] = p.lse_state[slot + r];
}

__global__ void planner_init_kernel(PlannerState *st, double eps) {
    if (threadIdx.x == 0) {
        st->eps = eps;
        st->have_anchor = 0;
        st->is_anchor = 0;
    }
    for (int e = threadIdx.x; e < DT_MAX_P * DT_MAX_P; e += blockDim.x) {
        st->w[e] = 0.0;
        st->alpha[e] = 0.0;
    }
}

}  // namespace

cudaError_t launch_planner_init(PlannerState *st, double eps, cudaStream_t stream) {
    planner_init_kernel<<<1, 256, 0, stream>>>(st, eps);
    return cudaGetLastError();
}

cudaError_t launch_planner_step(const PlannerParams &p, int state_dtype, cudaStream_t stream) {
    dim3 grid((unsigned)p.chunks, (unsigned)p.P, (unsigned)p.BH);
    if (state_dtype == DT_STATE_FP32) planner_local_kernel<float><<<grid, PL_THREADS, 0, stream>>>(p);
    else planner_local_kernel<__nv_bfloat16><<<grid, PL_THREADS, 0, stream>>>(p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    planner_decide_kernel<<<1, 1024, 0, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_planner_commit(const PlannerParams &p, int state_dtype, cudaStream_t stream) {
    dim3 grid_n((unsigned)p.chunks, (unsigned)(p.P * p.S), (unsigned)p.BH);
    dim3 grid_s((unsigned)p.chunks, (unsigned)p.P, (unsigned)p.BH);
    cudaError_t e = cudaSuccess;
    if (p.force) {   // after a group compose the states were not written by the attention kernel: take the norms from the cache
        if (state_dtype == DT_STATE_FP32) planner_norm_kernel<float><<<grid_n, PL_THREADS, 0, stream>>>(p);
        else planner_norm_kernel<__nv_bfloat16><<<grid_n, PL_THREADS, 0, stream>>>(p);
    } else {
        planner_attn_norm_kernel<<<p.P * p.S, PL_THREADS, 0, stream>>>(p);
    }
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    planner_commit_kernel<<<1, 1024, 0, stream>>>(p);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if (p.force) return cudaSuccess;   // a refresh after a group compose keeps the anchor's snapshot
    if (state_dtype == DT_STATE_FP32) planner_snapshot_kernel<float><<<grid_s, PL_THREADS, 0, stream>>>(p);
    else planner_snapshot_kernel<__nv_bfloat16><<<grid_s, PL_THREADS, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace dt
