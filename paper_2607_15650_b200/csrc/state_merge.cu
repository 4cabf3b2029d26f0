// dt_state_merge: Eq. 2 folded over the cached states (one per slot; P in pair mode) of every query row.
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

// VEC fp32 values -> 16-bit elements (bf16, or fp16 when `fp16`), one vector store
template <int VEC>
__device__ __forceinline__ void store_bf16(__nv_bfloat16 *p, const float (&v)[VEC], bool fp16 = false) {
    uint32_t w[VEC / 2];
#pragma unroll
    for (int i = 0; i < VEC / 2; ++i) w[i] = fp16 ? pack_f16x2(v[2 * i], v[2 * i + 1]) : pack_bf16x2(v[2 * i], v[2 * i + 1]);
    if constexpr (VEC == 4) {
        __stcs(reinterpret_cast<uint2 *>(p), make_uint2(w[0], w[1]));
    } else {
        __stcs(reinterpret_cast<uint4 *>(p), make_uint4(w[0], w[1], w[2], w[3]));
    }
}

constexpr int MERGE_THREADS = 256;
constexpr int MERGE_STAGE_BYTES = 64 * 1024;          // state bytes one block keeps in flight
constexpr long long MERGE_WAIT_LIMIT = 4000000000ll;  // SM clock cycles: about 2 s

constexpr int MERGE_CHUNK = 8;   // sources staged at a time by the subset modes

template <typename StateT, int D>
struct MergeCfg {
    static constexpr int VEC = StateVec<StateT>::VEC;
    static constexpr int TPR = D / VEC;                       // threads per row
    static constexpr int MAX_ROWS = MERGE_THREADS / TPR;      // rows the block's threads can cover
    static constexpr int ROW_BYTES = D * (int)sizeof(StateT);
    // MERGE_ALL stages all slots at once (64 KB per block, three blocks per SM) as long as the block can then
    // cover its full MAX_ROWS rows; with more slots, and in the subset modes, MERGE_CHUNK sources are staged at a
    // time for MAX_ROWS rows (32 KB per block, six blocks per SM): bulk copies stay at 4 KB instead of shrinking
    // with the slot count, and a step which needs few sources per row still keeps many bytes in flight per SM.
    static bool chunked(int mode, int P) { return mode != MERGE_ALL || MERGE_STAGE_BYTES / (P * ROW_BYTES) < MAX_ROWS; }
    static int rows(int mode, int P) {
        if (chunked(mode, P)) return MAX_ROWS;
        const int r = MERGE_STAGE_BYTES / (P * ROW_BYTES);
        return r > MAX_ROWS ? MAX_ROWS : r;
    }
    static int staged(int mode, int P) { return chunked(mode, P) ? MERGE_CHUNK : P; }
    static size_t smem_bytes(int mode, int P) {
        return (size_t)staged(mode, P) * rows(mode, P) * ROW_BYTES + (size_t)rows(mode, P) * (DT_MAX_P + 1 + 2) * sizeof(float) + 64 + 64;
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
template <typename StateT, int D, int MODE>
__global__ void __launch_bounds__(MERGE_THREADS) state_merge_kernel(const __grid_constant__ MergeParams p, int ROWS, int staged) {
    using Cf = MergeCfg<StateT, D>;
    constexpr int VEC = Cf::VEC, TPR = Cf::TPR;
    constexpr int NS = DT_MAX_P + 1;   // sources per row at most: P slots + the composed state
    extern __shared__ __align__(128) uint8_t smem[];
    const int P = p.S;   // sources in the cache: one per slot
    constexpr int EXTRA = (MODE == MERGE_PLANNED) ? 1 : 0;
    const int nslots = P + EXTRA;
    StateT *tile = reinterpret_cast<StateT *>(smem);                                         // [staged][ROWS][D]
    float *lse_s = reinterpret_cast<float *>(smem + (size_t)staged * ROWS * Cf::ROW_BYTES);   // [ROWS][NS]
    uint64_t *bar_ptr = reinterpret_cast<uint64_t *>(lse_s + ((ROWS * NS + 1) & ~1));        // 8-byte aligned
    int *abort_flag = reinterpret_cast<int *>(bar_ptr + 1);
    int *nsrc_s = abort_flag + 1;
    uint8_t *src_s = reinterpret_cast<uint8_t *>(abort_flag + 2);                             // [NS] source ids in staging order
    float *rowz_s = reinterpret_cast<float *>(src_s + ((NS + 3) & ~3));                       // [ROWS] sum of a row's weights
    float *rowm_s = rowz_s + ROWS;                                                            // [ROWS] a row's largest log-sum-exp
    const uint32_t bar = smem_u32(bar_ptr);

    const long long row0 = p.row_begin + (long long)blockIdx.x * ROWS;
    const int valid = (int)min((long long)ROWS, p.row_begin + p.row_count - row0);   // rows of this block that exist
    const uint32_t bytes = (uint32_t)valid * Cf::ROW_BYTES;

    // Token index of a cache row (row mod L) and its query partition.  The offsets travel as kernel parameters, so
    // this needs no memory access; it is instruction count that matters here (the subset modes were issue-bound on
    // a 64-bit modulo and a linear search per looked-up row): 32-bit arithmetic whenever the row count allows it, a
    // binary search once per thread, and from there a step or two along the offsets for the block's other rows.
    const bool rows32 = (p.R < (1ll << 31));
    auto mod_L = [&](long long row) -> int {
        return rows32 ? (int)((uint32_t)row % (uint32_t)p.L) : (int)(row % p.L);
    };
    auto partition_of_l = [&](int l) -> int {
        int lo = 0, hi = p.P;
#pragma unroll 1
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (p.off_val[mid] <= l) lo = mid; else hi = mid;
        }
        return lo;
    };
    // (only the threads that look rows up: thread 0 for the block's source list, and those that fetch log-sum-exps)
    const bool need_parts = ((MODE != MERGE_ALL) || (p.sel_bits != nullptr)) &&
                            (threadIdx.x == 0 || (int)threadIdx.x < valid * nslots);
    const int l_first = need_parts ? mod_L(row0) : 0;                 // token index of the block's first row
    const int i_first = need_parts ? partition_of_l(l_first) : 0;     // and its query partition
    // query partition of the block's r-th row
    auto partition_of_row = [&](int r) -> int {
        int l = l_first + r, i = i_first;
        if (l >= p.L) {               // the block runs into the next (b, h): start over from partition 0
            l %= p.L;
            i = 0;
        }
#pragma unroll 1
        while (i + 1 < p.P && p.off_val[i + 1] <= l) ++i;
        return i;
    };
    // per query partition, bit j set = slot j takes part (prepared on the device from the mask)
    auto sel_of = [&](int r) -> uint32_t { return __ldg(p.sel_bits + partition_of_row(r)); };
    const uint32_t all_bits = (P == 32) ? 0xFFFFFFFFu : ((1u << P) - 1u);
    // copies for the sources [first, first + count) of the staging order into tile slots 0..count-1
    auto stage = [&](int first, int count) {
        mbar_arrive_expect_tx(bar, bytes * (uint32_t)count);
        for (int k = 0; k < count; ++k) {
            const int src = (MODE == MERGE_ALL) ? first + k : (int)src_s[first + k];
            const StateT *g = (src < P) ? static_cast<const StateT *>(p.o_state) + ((long long)src * p.R + row0) * D
                                        : static_cast<const StateT *>(p.comp_o) + row0 * D;
            bulk_load(smem_u32(tile + (size_t)k * ROWS * D), g, bytes, bar);
        }
    };

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        mbar_init(bar, 1);
        fence_mbar_init();
        int nsrc = P;
        if (MODE != MERGE_ALL) {
            // sources any row of the block needs; its rows are consecutive, so only the partitions of its
            // two ends and those between them matter
            uint32_t need = 0;
            const int i0 = i_first, i1 = partition_of_row(valid - 1);
            if (valid >= p.L) { for (int i = 0; i < p.P; ++i) need |= __ldg(p.sel_bits + i); }   // a block longer than the sequence
            else if (i0 <= i1 && l_first + valid <= p.L) { for (int i = i0; i <= i1; ++i) need |= __ldg(p.sel_bits + i); }
            else { for (int i = 0; i < p.P; ++i) if (i >= i0 || i <= i1) need |= __ldg(p.sel_bits + i); }   // wraps into the next (b, h)
            nsrc = 0;
            for (int j = 0; j < P; ++j) if (need >> j & 1u) src_s[nsrc++] = (uint8_t)j;
            if (MODE == MERGE_PLANNED) src_s[nsrc++] = (uint8_t)P;
        }
        *nsrc_s = nsrc;
        if (nsrc > 0) stage(0, min(nsrc, staged));
    }
    // the rows' log-sum-exps, through shared memory so that every thread of a row sees all of them;
    // sources that do not take part get -inf, i.e. weight zero
    for (int e = threadIdx.x; e < valid * nslots; e += MERGE_THREADS) {
        const int r = e / nslots, j = e - r * nslots;
        float x = -INFINITY;
        if (j < P) {
            const uint32_t sel = (MODE == MERGE_ALL && p.sel_bits == nullptr) ? all_bits : sel_of(r);
            if (sel >> j & 1u) x = __ldg(p.lse_state + (long long)j * p.R + row0 + r);
        } else {
            x = __ldg(p.comp_lse + row0 + r);
        }
        lse_s[r * NS + j] = x;
    }
    __syncthreads();   // also publishes the mbarrier initialisation and the staging order

    // The weights exp(LSE_j - M) of a row are the same for every thread that works on it: eight lanes per row form them
    // once -- only the block's sources can carry mass, every other entry of the row is -inf -- and leave them in place
    // of the log-sum-exps, with the row's maximum M and the sum Z beside them.  (Every thread of the row used to repeat
    // this; the subset modes were bound by instruction issue, not by memory.)
    const int nsrc = *nsrc_s;
    {
        const int wr = threadIdx.x >> 3, wl = threadIdx.x & 7;
        if (wr < ROWS) {            // ROWS * 8 <= 256 threads, whole warps
            float *row_lse = lse_s + wr * NS;
            float m = -INFINITY;
            for (int k = wl; k < nsrc; k += 8) m = fmaxf(m, row_lse[(MODE == MERGE_ALL) ? k : (int)src_s[k]]);
#pragma unroll
            for (int sft = 1; sft < 8; sft <<= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, sft));
            float z = 0.f;
            for (int k = wl; k < nsrc; k += 8) {
                const int src = (MODE == MERGE_ALL) ? k : (int)src_s[k];
                const float w = (m == -INFINITY) ? 0.f : __expf(row_lse[src] - m);
                row_lse[src] = w;
                z += w;
            }
#pragma unroll
            for (int sft = 1; sft < 8; sft <<= 1) z += __shfl_xor_sync(0xFFFFFFFFu, z, sft);
            if (wl == 0) { rowz_s[wr] = z; rowm_s[wr] = m; }
        }
    }
    __syncthreads();
    const int r = threadIdx.x / TPR, lane = threadIdx.x % TPR;
    const bool active = r < valid;
    const float *my_w = lse_s + (active ? r : 0) * NS;
    const float Z = rowz_s[active ? r : 0], M = rowm_s[active ? r : 0];
    const bool empty = (M == -INFINITY);   // no source has any mass: output 0, LSE = -inf

    float acc[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc[e] = 0.f;
    const StateT *mine = tile + (size_t)(active ? r : 0) * D + lane * VEC;
    for (int first = 0, phase = 0; first < nsrc; first += staged, phase ^= 1) {
        const int count = min(nsrc - first, staged);
        if (first > 0) {          // the tile buffer is reused: everyone must be done with the previous chunk
            __syncthreads();
            if (threadIdx.x == 0) stage(first, count);
        }
        if (!mbar_wait_bounded(bar, (uint32_t)phase, abort_flag, MERGE_WAIT_LIMIT)) {
            if (p.status) atomicOr(p.status, STATUS_WAIT_TIMEOUT);
            *abort_flag = 1;
            // copies may still be in flight towards this block's shared memory: stay resident until they have had
            // time to land (every thread waits on the same barrier, so all of them take this way out)
            const uint64_t t0 = global_timer_ns();
            while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
            return;
        }
        if (active && !empty) {
#pragma unroll 4
            for (int k = 0; k < count; ++k) {
                const int src = (MODE == MERGE_ALL) ? first + k : (int)src_s[first + k];
                const float wt = my_w[src];
                if (wt != 0.f) {   // rows of another partition may not use this source at all
                    float v[VEC];
                    StateVec<StateT>::load(mine + (size_t)k * ROWS * D, v);
#pragma unroll
                    for (int e = 0; e < VEC; ++e) acc[e] = fmaf(wt, v[e], acc[e]);
                }
            }
        }
    }
    if (!active) return;
    const float inv = empty ? 0.f : 1.f / Z;
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc[e] *= inv;
    const float lse_row = empty ? -INFINITY : M + __logf(Z);

    const long long row = row0 + r;
    if (MODE == MERGE_COMPOSE) {
        store_state<VEC>(static_cast<StateT *>(p.comp_o_out) + row * D + lane * VEC, acc);
        if (lane == 0) p.comp_lse_out[row] = lse_row;
        return;
    }
    const long long bh = rows32 ? (long long)((uint32_t)row / (uint32_t)p.L) : row / p.L;
    const int l = (int)(row - bh * p.L);
    const int b = (int)(bh / p.H), h = (int)(bh - (long long)b * p.H);
    __nv_bfloat16 *out = static_cast<__nv_bfloat16 *>(p.out) + b * p.sb + l * p.sl + h * p.sh + lane * VEC;
    store_bf16<VEC>(out, acc, p.out_fp16 != 0);
    if (lane == 0 && p.lse_out != nullptr) p.lse_out[row] = lse_row;
}

template <typename StateT, int D, int MODE>
cudaError_t launch_mode(const MergeParams &p, cudaStream_t stream) {
    using Cf = MergeCfg<StateT, D>;
    const int rows = Cf::rows(MODE, p.S);
    const size_t smem = Cf::smem_bytes(MODE, p.S);
    const long long blocks = (p.row_count + rows - 1) / rows;
    if (blocks <= 0 || blocks > 0x7FFFFFFFLL) return cudaErrorInvalidValue;
    cudaError_t e = cudaFuncSetAttribute(state_merge_kernel<StateT, D, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         MERGE_STAGE_BYTES + MERGE_THREADS * (DT_MAX_P + 1 + 2) * (int)sizeof(float) + 256);
    if (e != cudaSuccess) return e;
    state_merge_kernel<StateT, D, MODE><<<(unsigned)blocks, MERGE_THREADS, smem, stream>>>(p, rows, Cf::staged(MODE, p.S));
    return cudaGetLastError();
}

template <typename StateT, int D>
cudaError_t launch(const MergeParams &p, cudaStream_t stream) {
    if (p.mode == MERGE_ALL) return launch_mode<StateT, D, MERGE_ALL>(p, stream);
    if (p.mode == MERGE_COMPOSE) return launch_mode<StateT, D, MERGE_COMPOSE>(p, stream);
    return launch_mode<StateT, D, MERGE_PLANNED>(p, stream);
}

// mask -> per query partition the bit set of slots that take part (REUSE slots for the composition,
// COMPUTE slots for the planned merge); slots that do not exist for the partition never do
__global__ void merge_select_kernel(const uint8_t *mask, const uint32_t *nonempty, int P, int S, int want_compute,
                                    uint32_t *sel_bits) {
    const int i = threadIdx.x;
    if (i >= P) return;
    uint32_t bits = 0;
    for (int j = 0; j < S; ++j)
        if ((mask[i * S + j] != 0) == (want_compute != 0)) bits |= 1u << j;
    sel_bits[i] = nonempty ? (bits & nonempty[i]) : bits;
}

}  // namespace

cudaError_t launch_merge_select(const uint8_t *mask, const uint32_t *nonempty, int P, int S, int want_compute,
                                uint32_t *sel_bits, cudaStream_t stream) {
    merge_select_kernel<<<1, 32, 0, stream>>>(mask, nonempty, P, S, want_compute, sel_bits);
    return cudaGetLastError();
}

cudaError_t launch_state_merge(const MergeParams &p, int D, int state_dtype, cudaStream_t stream) {
    if (state_dtype == DT_STATE_FP32) {
        return D == 64 ? launch<float, 64>(p, stream) : launch<float, 128>(p, stream);
    }
    return D == 64 ? launch<__nv_bfloat16, 64>(p, stream) : launch<__nv_bfloat16, 128>(p, stream);
}

}  // namespace dt
