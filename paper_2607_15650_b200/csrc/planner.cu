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

template <typename T>
__device__ __forceinline__ float to_f32(T x);
template <>
__device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

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
    for (long long e = threadIdx.x; e < n; e += PL_THREADS) {
        const float a = to_f32(cur[e]), b = to_f32(old[e]);
        diff += (a - b) * (a - b);
        base += b * b;
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

// grid (chunks, P (query partition i), BH * S (slot j)): sum of squares of the state rows; anchor steps only
template <typename StateT>
__global__ void __launch_bounds__(PL_THREADS) planner_norm_kernel(PlannerParams p) {
    if (!p.force && !p.state->is_anchor) return;
    const int c = blockIdx.x, i = blockIdx.y, bh = blockIdx.z / p.S, j = blockIdx.z - bh * p.S;
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
    for (long long e = threadIdx.x; e < n; e += PL_THREADS) {
        const float a = to_f32(src[e]);
        sq += a * a;
    }
    for (int r = row0 + (int)threadIdx.x; r < row1; r += PL_THREADS) {
        const float a = p.lse_state[slot + r];
        sq += a * a;
    }
    block_sum2(sq, unused);
    if (threadIdx.x == 0) p.norm_partials[(((long long)bh * p.P + i) * p.chunks + c) * p.S + j] = sq;
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
                n += (double)p.norm_partials[idx];
            }
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
    dim3 grid_n((unsigned)p.chunks, (unsigned)p.P, (unsigned)(p.BH * p.S));
    dim3 grid_s((unsigned)p.chunks, (unsigned)p.P, (unsigned)p.BH);
    if (state_dtype == DT_STATE_FP32) planner_norm_kernel<float><<<grid_n, PL_THREADS, 0, stream>>>(p);
    else planner_norm_kernel<__nv_bfloat16><<<grid_n, PL_THREADS, 0, stream>>>(p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    planner_commit_kernel<<<1, 1024, 0, stream>>>(p);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if (p.force) return cudaSuccess;   // a refresh after a group compose keeps the anchor's snapshot
    if (state_dtype == DT_STATE_FP32) planner_snapshot_kernel<float><<<grid_s, PL_THREADS, 0, stream>>>(p);
    else planner_snapshot_kernel<__nv_bfloat16><<<grid_s, PL_THREADS, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace dt
