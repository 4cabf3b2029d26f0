// dt_state_merge: Eq. 2 folded over the P cached states of every query row.
//
// HBM-bound streaming kernel.  One query row (b, h, l) is handled by D / VEC consecutive
// threads, each owning VEC = 16 bytes / sizeof(state) head-dim elements; for every KV
// partition j the row's slice of OUT_ij is one 128-bit load, so a warp reads 512 contiguous
// bytes per j.  The P log-sum-exps of the row are read once per thread (same address across
// the row's threads: one broadcast transaction) and turned into weights
// exp(LSE_ij - max_j LSE_ij) / Z in fp32; the weighted sum is accumulated in fp32 and stored
// as bf16 in the [B, L, H, D] output.  Algorithmic bytes per row:
// P * (D * sizeof(state) + 4) read + 2 D + 4 written.
#include <cuda_bf16.h>

#include "dt_internal.h"

namespace dt {
namespace {

template <typename T>
struct StateVec;
template <>
struct StateVec<float> {
    static constexpr int VEC = 4;
    __device__ static __forceinline__ void load(const float *p, float (&v)[4]) {
        float4 x = __ldcs(reinterpret_cast<const float4 *>(p));
        v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
    }
};
template <>
struct StateVec<__nv_bfloat16> {
    static constexpr int VEC = 8;
    __device__ static __forceinline__ void load(const __nv_bfloat16 *p, float (&v)[8]) {
        uint4 x = __ldcs(reinterpret_cast<const uint4 *>(p));
        const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[2 * i] = __uint_as_float(w[i] << 16);
            v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
};

template <int VEC>
__device__ __forceinline__ void store_bf16(__nv_bfloat16 *p, const float (&v)[VEC]) {
    uint32_t w[VEC / 2];
#pragma unroll
    for (int i = 0; i < VEC / 2; ++i) {
        __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
        w[i] = *reinterpret_cast<uint32_t *>(&h);
    }
    if constexpr (VEC == 4) {
        __stcs(reinterpret_cast<uint2 *>(p), make_uint2(w[0], w[1]));
    } else {
        __stcs(reinterpret_cast<uint4 *>(p), make_uint4(w[0], w[1], w[2], w[3]));
    }
}

constexpr int MERGE_THREADS = 256;
constexpr int JB = 8;  // states fetched per batch of independent loads

template <typename StateT, int D>
__global__ void __launch_bounds__(MERGE_THREADS) state_merge_kernel(MergeParams p) {
    constexpr int VEC = StateVec<StateT>::VEC;
    constexpr int TPR = D / VEC;                 // threads per row
    constexpr int RPB = MERGE_THREADS / TPR;     // rows per block
    const long long row = (long long)blockIdx.x * RPB + threadIdx.x / TPR;
    const int lane = threadIdx.x % TPR;
    if (row >= p.R) return;
    const int P = p.P;
    const StateT *o_state = static_cast<const StateT *>(p.o_state);

    // weights: LSE_ij - M, then exp; P <= 32 values kept in registers
    float ls[DT_MAX_P];
    float M = -INFINITY;
#pragma unroll
    for (int j = 0; j < DT_MAX_P; ++j) {
        ls[j] = (j < P) ? __ldg(p.lse_state + (long long)j * p.R + row) : -INFINITY;
        M = fmaxf(M, ls[j]);
    }
    float Z = 0.f;
    const bool empty = (M == -INFINITY);   // no partition has any mass: output 0, LSE = -inf
#pragma unroll
    for (int j = 0; j < DT_MAX_P; ++j) {
        ls[j] = (j < P && !empty) ? __expf(ls[j] - M) : 0.f;
        Z += ls[j];
    }

    float acc[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc[e] = 0.f;
    const StateT *base = o_state + row * D + lane * VEC;
    const long long slab = p.R * D;
#pragma unroll
    for (int j0 = 0; j0 < DT_MAX_P; j0 += JB) {
        if (j0 < P) {
            float v[JB][VEC];
#pragma unroll
            for (int jj = 0; jj < JB; ++jj) {
                if (j0 + jj < P) StateVec<StateT>::load(base + (long long)(j0 + jj) * slab, v[jj]);
            }
#pragma unroll
            for (int jj = 0; jj < JB; ++jj) {
                if (j0 + jj < P) {
                    const float w = ls[j0 + jj];
#pragma unroll
                    for (int e = 0; e < VEC; ++e) acc[e] = fmaf(w, v[jj][e], acc[e]);
                }
            }
        }
    }
    const float inv = empty ? 0.f : 1.f / Z;
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc[e] *= inv;

    const long long bh = row / p.L;
    const int l = (int)(row - bh * p.L);
    const int b = (int)(bh / p.H), h = (int)(bh - (long long)b * p.H);
    __nv_bfloat16 *out = static_cast<__nv_bfloat16 *>(p.out) + b * p.sb + l * p.sl + h * p.sh + lane * VEC;
    store_bf16<VEC>(out, acc);
    if (lane == 0 && p.lse_out != nullptr) p.lse_out[row] = empty ? -INFINITY : M + __logf(Z);
}

template <typename StateT, int D>
cudaError_t launch(const MergeParams &p, cudaStream_t stream) {
    constexpr int RPB = MERGE_THREADS / (D / StateVec<StateT>::VEC);
    const long long blocks = (p.R + RPB - 1) / RPB;
    if (blocks <= 0 || blocks > 0x7FFFFFFFLL) return cudaErrorInvalidValue;
    state_merge_kernel<StateT, D><<<(unsigned)blocks, MERGE_THREADS, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_state_merge(const MergeParams &p, int D, int state_dtype, cudaStream_t stream) {
    if (state_dtype == DT_STATE_FP32) {
        return D == 64 ? launch<float, 64>(p, stream) : launch<float, 128>(p, stream);
    }
    return D == 64 ? launch<__nv_bfloat16, 64>(p, stream) : launch<__nv_bfloat16, 128>(p, stream);
}

}  // namespace dt
