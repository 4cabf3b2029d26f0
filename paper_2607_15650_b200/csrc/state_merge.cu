// dt_state_merge: Eq. 2 folded over the P cached states of every query row.
//
// HBM-bound streaming kernel.  A block owns ROWS consecutive rows (b, h, l) of the cache.  For each
// KV partition j those rows are one contiguous run of ROWS * D state elements, which one thread
// fetches with a bulk asynchronous copy (cp.async.bulk, completion counted on an mbarrier) into
// shared memory: P copies of a few KB each are in flight per block without costing a register,
// and several blocks per SM keep the memory system saturated while others compute.  Meanwhile the
// block's threads read the rows' P log-sum-exps, and each (row, 16-byte column group) thread forms
// the weights exp(LSE_ij - max_j LSE_ij) / Z in fp32.  After the copies land, the weighted sum is
// accumulated in fp32 from shared memory and stored as bf16 in the [B, L, H, D] output.
// Algorithmic bytes per row: P * (D * sizeof(state) + 4) read + 2 D + 4 written.
//
// The same kernel composes subsets: the REUSE states of a plan into one cached state per row
// (Section 2.2.4: "compose states from remote partitions and cache the result"; Eq. 15), and the
// COMPUTE states plus that composed state into the output, so a selective step reads
// (computed + 1) states per row instead of P.
//
// The wait for the copies is bounded; on expiry the block records STATUS_WAIT_TIMEOUT and returns.
#include <cuda_bf16.h>

#include "dt_internal.h"
#include "ptx_sm100.cuh"

namespace dt {
namespace {

template <typename T>
struct StateVec;
template <>
struct StateVec<float> {
    static constexpr int VEC = 4;
    __device__ static __forceinline__ void load(const float *p, float (&v)[4]) {
        const float4 x = *reinterpret_cast<const float4 *>(p);
        v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
    }
};
template <>
struct StateVec<__nv_bfloat16> {
    static constexpr int VEC = 8;
    __device__ static __forceinline__ void load(const __nv_bfloat16 *p, float (&v)[8]) {
        const uint4 x = *reinterpret_cast<const uint4 *>(p);
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
constexpr int MERGE_STAGE_BYTES = 64 * 1024;          // state bytes one block keeps in flight
constexpr long long MERGE_WAIT_LIMIT = 4000000000ll;  // SM clock cycles: about 2 s

template <typename StateT, int D>
struct MergeCfg {
    static constexpr int VEC = StateVec<StateT>::VEC;
    static constexpr int TPR = D / VEC;                       // threads per row
    static constexpr int MAX_ROWS = MERGE_THREADS / TPR;      // rows the block's threads can cover
    static constexpr int ROW_BYTES = D * (int)sizeof(StateT);
    static int rows(int nslots) {
        int r = MERGE_STAGE_BYTES / (nslots * ROW_BYTES);
        r = r < 1 ? 1 : r;
        return r > MAX_ROWS ? MAX_ROWS : r;
    }
    static size_t smem_bytes(int nslots) {
        return (size_t)nslots * rows(nslots) * ROW_BYTES + (size_t)rows(nslots) * (DT_MAX_P + 1) * sizeof(float) + 32;
    }
};

template <int VEC>
__device__ __forceinline__ void store_state(float *p, const float (&v)[VEC]) {
    *reinterpret_cast<float4 *>(p) = make_float4(v[0], v[1], v[2], v[3]);
}
template <int VEC>
__device__ __forceinline__ void store_state(__nv_bfloat16 *p, const float (&v)[VEC]) {
    store_bf16<VEC>(p, v);
}

// Which cached states of a row enter the composition:
//   MERGE_ALL      every slot j < P                                              (dt_state_merge)
//   MERGE_COMPOSE  the REUSE slots of the row's query partition (mask == 0); the result is itself a
//                  state (OUT in the cache's dtype, LSE) written to the composed-state buffers
//   MERGE_PLANNED  the COMPUTE slots (mask != 0) plus the composed state as one more source
template <typename StateT, int D>
__global__ void __launch_bounds__(MERGE_THREADS) state_merge_kernel(MergeParams p, int ROWS) {
    using Cf = MergeCfg<StateT, D>;
    constexpr int VEC = Cf::VEC, TPR = Cf::TPR;
    constexpr int NS = DT_MAX_P + 1;   // sources per row at most: P slots + the composed state
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ int32_t off_s[DT_MAX_P + 1];
    __shared__ uint32_t sel_s[DT_MAX_P];   // per query partition: bit j set = slot j takes part
    const int P = p.P;
    const int nslots = P + (p.mode == MERGE_PLANNED ? 1 : 0);
    StateT *tile = reinterpret_cast<StateT *>(smem);                                        // [nslots][ROWS][D]
    float *lse_s = reinterpret_cast<float *>(smem + (size_t)nslots * ROWS * Cf::ROW_BYTES);  // [ROWS][NS]
    uint64_t *bar_ptr = reinterpret_cast<uint64_t *>(lse_s + ROWS * NS);
    int *abort_flag = reinterpret_cast<int *>(bar_ptr + 1);
    const uint32_t bar = smem_u32(bar_ptr);

    const long long row0 = (long long)blockIdx.x * ROWS;
    const int valid = (int)min((long long)ROWS, p.R - row0);   // rows of this block that exist

    if (p.mode != MERGE_ALL) {
        if (threadIdx.x <= P) off_s[threadIdx.x] = p.off[threadIdx.x];
        if (threadIdx.x < P) {
            uint32_t bits = 0;
            for (int j = 0; j < P; ++j) {
                const bool compute = p.mask[threadIdx.x * P + j] != 0;
                if (compute == (p.mode == MERGE_PLANNED)) bits |= 1u << j;
            }
            sel_s[threadIdx.x] = bits;
        }
        __syncthreads();
    }
    // query partition of a cache row (token index l = row mod L)
    auto partition_of = [&](long long row) -> int {
        const int l = (int)(row % p.L);
        int i = 0;
        while (i + 1 < P && off_s[i + 1] <= l) ++i;
        return i;
    };
    const uint32_t all_bits = (P == 32) ? 0xFFFFFFFFu : ((1u << P) - 1u);

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        mbar_init(bar, 1);
        fence_mbar_init();
        // slots any row of the block needs: one bulk copy each (`valid` consecutive rows of slot j)
        uint32_t need = all_bits;
        if (p.mode != MERGE_ALL) {
            need = 0;
            for (int r = 0; r < valid; ++r) need |= sel_s[partition_of(row0 + r)];
        }
        const uint32_t bytes = (uint32_t)valid * Cf::ROW_BYTES;
        const uint32_t copies = (uint32_t)__popc(need) + (p.mode == MERGE_PLANNED ? 1u : 0u);
        if (copies > 0) {
            mbar_arrive_expect_tx(bar, bytes * copies);
            const StateT *src = static_cast<const StateT *>(p.o_state) + row0 * D;
            for (int j = 0; j < P; ++j)
                if (need >> j & 1u) bulk_load(smem_u32(tile + (size_t)j * ROWS * D), src + (long long)j * p.R * D, bytes, bar);
            if (p.mode == MERGE_PLANNED)
                bulk_load(smem_u32(tile + (size_t)P * ROWS * D), static_cast<const StateT *>(p.comp_o) + row0 * D, bytes, bar);
        } else {
            mbar_arrive(bar);
        }
    }
    // the rows' log-sum-exps, through shared memory so that every thread of a row sees all of them;
    // sources that do not take part get -inf, i.e. weight zero
    for (int e = threadIdx.x; e < valid * NS; e += MERGE_THREADS) {
        const int r = e / NS, j = e - r * NS;
        float x = -INFINITY;
        if (j < P) {
            const uint32_t sel = (p.mode == MERGE_ALL) ? all_bits : sel_s[partition_of(row0 + r)];
            if (sel >> j & 1u) x = __ldg(p.lse_state + (long long)j * p.R + row0 + r);
        } else if (j == P && p.mode == MERGE_PLANNED) {
            x = __ldg(p.comp_lse + row0 + r);
        }
        lse_s[r * NS + j] = x;
    }
    __syncthreads();   // also publishes the mbarrier initialisation to the waiting threads

    const int r = threadIdx.x / TPR, lane = threadIdx.x % TPR;
    const bool active = r < valid;
    float w[NS];
    float M = -INFINITY, Z = 0.f;
    if (active) {
#pragma unroll
        for (int j = 0; j < NS; ++j) {
            w[j] = (j < nslots) ? lse_s[r * NS + j] : -INFINITY;
            M = fmaxf(M, w[j]);
        }
    }
    const bool empty = (M == -INFINITY);   // no source has any mass: output 0, LSE = -inf
#pragma unroll
    for (int j = 0; j < NS; ++j) {
        w[j] = (active && j < nslots && !empty) ? __expf(w[j] - M) : 0.f;
        Z += w[j];
    }

    if (!mbar_wait_bounded(bar, 0, abort_flag, MERGE_WAIT_LIMIT)) {
        if (p.status) atomicOr(p.status, STATUS_WAIT_TIMEOUT);
        *abort_flag = 1;
        return;
    }
    if (!active) return;

    float acc[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc[e] = 0.f;
    const StateT *mine = tile + (size_t)r * D + lane * VEC;
#pragma unroll
    for (int j = 0; j < NS; ++j) {
        if (j < nslots && w[j] != 0.f) {   // a source with zero weight may not even have been copied
            float v[VEC];
            StateVec<StateT>::load(mine + (size_t)j * ROWS * D, v);
#pragma unroll
            for (int e = 0; e < VEC; ++e) acc[e] = fmaf(w[j], v[e], acc[e]);
        }
    }
    const float inv = empty ? 0.f : 1.f / Z;
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc[e] *= inv;
    const float lse_row = empty ? -INFINITY : M + __logf(Z);

    const long long row = row0 + r;
    if (p.mode == MERGE_COMPOSE) {
        store_state<VEC>(static_cast<StateT *>(p.comp_o_out) + row * D + lane * VEC, acc);
        if (lane == 0) p.comp_lse_out[row] = lse_row;
        return;
    }
    const long long bh = row / p.L;
    const int l = (int)(row - bh * p.L);
    const int b = (int)(bh / p.H), h = (int)(bh - (long long)b * p.H);
    __nv_bfloat16 *out = static_cast<__nv_bfloat16 *>(p.out) + b * p.sb + l * p.sl + h * p.sh + lane * VEC;
    store_bf16<VEC>(out, acc);
    if (lane == 0 && p.lse_out != nullptr) p.lse_out[row] = lse_row;
}

template <typename StateT, int D>
cudaError_t launch(const MergeParams &p, cudaStream_t stream) {
    using Cf = MergeCfg<StateT, D>;
    const int nslots = p.P + (p.mode == MERGE_PLANNED ? 1 : 0);
    const int rows = Cf::rows(nslots);
    const size_t smem = Cf::smem_bytes(nslots);
    const long long blocks = (p.R + rows - 1) / rows;
    if (blocks <= 0 || blocks > 0x7FFFFFFFLL) return cudaErrorInvalidValue;
    cudaError_t e = cudaFuncSetAttribute(state_merge_kernel<StateT, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         MERGE_STAGE_BYTES + MERGE_THREADS * (DT_MAX_P + 1) * (int)sizeof(float) + 32);
    if (e != cudaSuccess) return e;
    state_merge_kernel<StateT, D><<<(unsigned)blocks, MERGE_THREADS, smem, stream>>>(p, rows);
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
