// dt_plan: partition importance weights (Eq. 8) reduced to one contribution value per
// (query partition, KV partition) pair and thresholded into the COMPUTE / REUSE mask (Eq. 13),
// plus the work-list builder that turns a mask into the list of pairs dt_attn_states evaluates.
//
// Stage 1 (HBM-bound, P * 4 bytes per query row): one block handles up to PLAN_CHUNK_ROWS rows of
// one (b, h, query partition i), so all its threads share i.  Each thread reads the P cached
// LSE_ij of a row (coalesced across rows), forms w_j = exp(LSE_ij - logsumexp_k LSE_ik) in fp32
// and keeps P running sums; a fixed-order block reduction writes P partial sums to scratch.
// Stage 2 (one block): sums the partials in fp64 in a fixed order, divides by the row count,
// and either thresholds (W > eps, strict) or ranks the off-diagonal pairs to hit a target count.
// No atomics: the result is bit-reproducible from run to run.
#include <math.h>

#include "dt_internal.h"
#include "ptx_sm100.cuh"

namespace dt {
namespace {

constexpr int PLAN_THREADS = 256;
// Resident blocks per SM the stage-1 kernel is compiled for.  Left to itself the compiler keeps the PMAX row
// pointers live and takes 141 registers at PMAX = 32: one block of 8 warps per SM, far too few loads in flight.
#ifndef DT_PLAN_BLOCKS32
#define DT_PLAN_BLOCKS32 3
#endif
#ifndef DT_PLAN_BLOCKS16
#define DT_PLAN_BLOCKS16 4
#endif
#define PLAN_MIN_BLOCKS(PMAX) ((PMAX) == 32 ? DT_PLAN_BLOCKS32 : ((PMAX) == 16 ? DT_PLAN_BLOCKS16 : 6))

template <int PMAX>
__global__ void __launch_bounds__(PLAN_THREADS, PLAN_MIN_BLOCKS(PMAX)) plan_partial_kernel(PlanParams p) {
    if (p.only_if != nullptr && *p.only_if == 0) return;
    const int c = blockIdx.x, i = blockIdx.y, bh = blockIdx.z;
    const int P = p.S;   // columns: cache slots (pair mode: one per KV partition)
    const uint32_t have = p.nonempty ? p.nonempty[i] : 0xFFFFFFFFu;   // slots that exist for this query partition
    const int row0 = p.off[i] + c * PLAN_CHUNK_ROWS;
    const int row1 = min(row0 + PLAN_CHUNK_ROWS, p.off[i + 1]);
    float acc[PMAX];
#pragma unroll
    for (int j = 0; j < PMAX; ++j) acc[j] = 0.f;
    const float *base = p.lse_state + (long long)bh * p.L;
    for (int l = row0 + (int)threadIdx.x; l < row1; l += PLAN_THREADS) {
        float x[PMAX];
        float M = -INFINITY;
#pragma unroll
        for (int j = 0; j < PMAX; ++j) {
            x[j] = (j < P && (have >> j & 1u)) ? __ldcs(base + (long long)j * p.R + l) : -INFINITY;
            M = fmaxf(M, x[j]);
        }
        if (M == -INFINITY) continue;  // row without any mass: contributes nothing
        float Z = 0.f;
#pragma unroll
        for (int j = 0; j < PMAX; ++j) {
            x[j] = expf(x[j] - M);
            Z += x[j];
        }
        const float inv = 1.f / Z;
#pragma unroll
        for (int j = 0; j < PMAX; ++j) acc[j] = fmaf(x[j], inv, acc[j]);
    }
    // Block reduction in a fixed order.  Inside a warp the PMAX sums of the 32 lanes are reduced together: at each
    // step a lane keeps one half of its values and adds its partner's copies of them (lanes that differ in the
    // step's bit hold the two halves), so PMAX - 1 shuffles (plus log2(32 / PMAX) full rounds for PMAX < 32) do the
    // work of 5 * PMAX and every value is still summed by the same xor tree, 16, 8, 4, 2, 1.  Lane l ends with the
    // warp's sum of column l % PMAX.  Then the first P threads add the 8 warps.
    __shared__ float red[PLAN_THREADS / 32][PMAX];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    {
        int ofs = 16;
#pragma unroll
        for (int full = 32; full > PMAX; full >>= 1, ofs >>= 1) {   // more lanes than columns: plain rounds first
#pragma unroll
            for (int j = 0; j < PMAX; ++j) acc[j] += __shfl_xor_sync(0xFFFFFFFFu, acc[j], ofs);
        }
#pragma unroll
        for (int half = PMAX / 2; half >= 1; half >>= 1, ofs >>= 1) {
            const bool upper = (lane & ofs) != 0;
#pragma unroll
            for (int j = 0; j < half; ++j) {
                const float send = upper ? acc[j] : acc[j + half];
                const float keep = upper ? acc[j + half] : acc[j];
                acc[j] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, ofs);
            }
        }
        red[warp][lane & (PMAX - 1)] = acc[0];   // for PMAX < 32 several lanes hold (and write) the same sum
    }
    __syncthreads();
    if (threadIdx.x < P) {
        float v = 0.f;
#pragma unroll
        for (int w = 0; w < PLAN_THREADS / 32; ++w) v += red[w][threadIdx.x];
        p.partials[(((long long)bh * p.P + i) * p.chunks + c) * P + threadIdx.x] = v;
    }
}

// Sum over (b*h, chunk) of the stage-1 partial sums of every entry (i, column), all 1024 threads taking part:
// entry = e % total (consecutive threads read consecutive columns: coalesced), the `tpe` threads of an entry take
// every tpe-th partial, and the entry's first thread adds their sums in a fixed order.  Result in out_s[entry].
__device__ __forceinline__ void sum_partials(const float *partials, int P, int S, int BH, int chunks, double *scratch,
                                             double *out_s) {
    const int total = P * S, e = threadIdx.x;
    int tpe = 1;
    while (tpe * 2 * total <= 1024 && tpe < 16) tpe *= 2;
    const int ent = e % total, part = e / total;
    if (part < tpe) {
        const int i = ent / S, j = ent - i * S, K = BH * chunks;
        double s = 0.0;
        for (int k = part; k < K; k += tpe) {
            const int bh = k / chunks, c = k - bh * chunks;
            s += (double)partials[(((long long)bh * P + i) * chunks + c) * S + j];
        }
        scratch[part * total + ent] = s;
    }
    __syncthreads();
    if (e < total) {
        double s = 0.0;
        for (int q = 0; q < tpe; ++q) s += scratch[q * total + e];
        out_s[e] = s;
    }
    __syncthreads();
}

// Un-normalised sums of the per-row weights, one per (query partition, slot): this context's own (from its stage-1
// partials) or, for head-sharded planning, the sums the caller added over all shards.
__device__ __forceinline__ void load_sums(const double *sums_in, const float *partials, int P, int S, int BH, int chunks,
                                          double *scratch, double *out_s) {
    if (sums_in == nullptr) {
        sum_partials(partials, P, S, BH, chunks, scratch, out_s);
    } else {
        if ((int)threadIdx.x < P * S) out_s[threadIdx.x] = sums_in[threadIdx.x];
        __syncthreads();
    }
}

// Ranking of the decision units for a target pair count.  Strict total order: larger measure first, then smaller
// group distance, then smaller flat index.  The units are sorted by a key that encodes that order (bitonic network
// in shared memory, one element per thread), an inclusive scan over the sorted sizes gives every unit the number of
// pairs it and all units before it stand for, and a unit is taken iff that total fits the budget -- the same
// decisions as counting, per unit, the units that rank before it, in O(n log^2 n) instead of O(n^2) steps.
__device__ __forceinline__ unsigned long long descending_key(double m) {   // ascending key order = descending m
    unsigned long long u = (unsigned long long)__double_as_longlong(m);
    u = (u >> 63) ? ~u : (u | (1ull << 63));
    return ~u;
}
__device__ __forceinline__ double key_measure(unsigned long long k) {
    unsigned long long u = ~k;
    u = (u >> 63) ? (u & ~(1ull << 63)) : ~u;
    return __longlong_as_double((long long)u);
}
struct RankScratch {
    unsigned long long k1[DT_MAX_P * DT_MAX_P];   // descending_key(measure); all ones: no unit
    uint32_t k2[DT_MAX_P * DT_MAX_P];             // distance << 20 | flat index << 8 | size
    int warp_sum[32];
    uint8_t dec[DT_MAX_P * DT_MAX_P];             // decision of unit e
};
// All 1024 threads call this.  Thread e < nunits brings its unit (size 0: none).  Returns the number of units taken;
// sc.dec[e] holds the decisions, edge[0] / edge[1] the measures of the last unit taken and of the first one not
// taken (left alone where there is none), *n_units the number of units.
__device__ __forceinline__ int take_by_rank(RankScratch &sc, double m, int size, int dist, int nunits, int budget,
                                            double *edge, int *n_units) {
    const int e = threadIdx.x;
    const bool unit = e < nunits && size > 0;
    sc.k1[e] = unit ? descending_key(m) : ~0ull;
    sc.k2[e] = unit ? ((uint32_t)dist << 20 | (uint32_t)e << 8 | (uint32_t)size) : 0xFFFFFF00u;
    sc.dec[e] = 0;
    int n = 32;
    while (n < nunits) n <<= 1;          // sorted length: a power of two that covers the units
    for (int k = 2; k <= n; k <<= 1)
        for (int j = k >> 1; j > 0; j >>= 1) {
            __syncthreads();
            const int x = e ^ j;
            if (e < n && x > e) {
                const unsigned long long a1 = sc.k1[e], b1 = sc.k1[x];
                const uint32_t a2 = sc.k2[e], b2 = sc.k2[x];
                const bool gt = a1 > b1 || (a1 == b1 && (a2 >> 8) > (b2 >> 8));
                if (gt == ((e & k) == 0)) {
                    sc.k1[e] = b1; sc.k1[x] = a1;
                    sc.k2[e] = b2; sc.k2[x] = a2;
                }
            }
        }
    __syncthreads();
    // inclusive scan of the sizes in rank order
    const int lane = e & 31, warp = e >> 5;
    const uint32_t mine2 = sc.k2[e];
    const int sz = (e < n) ? (int)(mine2 & 0xFFu) : 0;
    int cum = sz;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int up = __shfl_up_sync(0xFFFFFFFFu, cum, d);
        if (lane >= d) cum += up;
    }
    if (lane == 31) sc.warp_sum[warp] = cum;
    __syncthreads();
    for (int w = 0; w < warp; ++w) cum += sc.warp_sum[w];
    const bool take = sz > 0 && cum <= budget;
    if (sz > 0) sc.dec[(mine2 >> 8) & 0xFFFu] = take ? 1 : 0;
    const int taken = __syncthreads_count(take);
    const int units = __syncthreads_count(sz > 0);
    if (sz > 0 && e == taken - 1) edge[0] = key_measure(sc.k1[e]);
    if (sz > 0 && e == taken) edge[1] = key_measure(sc.k1[e]);
    if (e == 0) *n_units = units;
    __syncthreads();
    return taken;
}

// Stage 2.  W[i][j] from the partial sums, then one decision per unit (i, k): query partition i and the
// k-th group of g adjacent KV partitions without the local one (Section 4.2.1; g = 1: single pairs).
// Unit measure = sum of its members' W (Eq. 12); COMPUTE iff measure > eps (Eq. 13), or the units of
// largest measure taken in rank order while their members fit into K - P pairs.
__global__ void __launch_bounds__(1024) plan_final_kernel(PlanFinalParams p) {
    __shared__ double W[DT_MAX_P * DT_MAX_P];
    __shared__ RankScratch sc;
    __shared__ double edge[2];
    __shared__ int n_units;
    const int P = p.P, total = P * P, g = p.group_size;
    const int ng = (P + g - 1) / g, nunits = P * ng;
    const int e = threadIdx.x;
    load_sums(p.sums_in, p.partials, P, P, p.BH, p.chunks, reinterpret_cast<double *>(sc.k1), W);   // sc.k1 is scratch here
    if (p.sums_out) {   // first half of a head-sharded plan: the caller adds the shards' sums
        if (e < total) p.sums_out[e] = W[e];
        return;
    }
    {
        const int i = e / P;
        if (e < total) {
            const double cnt = (double)p.count_bh * (double)(p.off[i + 1] - p.off[i]);
            W[e] = W[e] / cnt;
            if (p.w_out) p.w_out[e] = W[e];
        }
    }
    if (e < 2) edge[e] = 0.0;
    __syncthreads();
    // unit e = (ui, uk)
    const int ui = e / ng, uk = e - ui * ng;
    double m = 0.0;
    int size = 0, dist = 0;
    if (e < nunits) {
        const int lo = uk * g, hi = min(P, (uk + 1) * g);
        for (int j = lo; j < hi; ++j)
            if (j != ui) { m += W[ui * P + j]; ++size; }
        const int gi = ui / g;
        dist = uk > gi ? uk - gi : gi - uk;
    }
    int taken = 0;
    if (p.mode_target) {
        taken = take_by_rank(sc, m, size, dist, nunits, p.K - P, edge, &n_units);
    } else {
        sc.dec[e] = (e < nunits && size > 0 && m > p.eps) ? 1 : 0;
        __syncthreads();
    }
    if (e < total) {
        const int i = e / P, j = e - i * P;
        p.mask[e] = (i == j || sc.dec[i * ng + j / g]) ? 1 : 0;
    }
    if (e == 0 && p.eps_out) {
        double eps = p.eps;
        if (p.mode_target) {
            if (n_units == 0 || taken == n_units) eps = 0.0;
            else if (taken == 0) eps = edge[1];
            else eps = 0.5 * (edge[0] + edge[1]);
        }
        *p.eps_out = eps;
    }
}

__device__ void build_tile_pairs(bool is_compute, const int32_t *off, int P, int4 *out);

// mask -> compact list of COMPUTE states (ordered by i*S+slot), t_c update, REUSE-of-empty detection.
// mask == nullptr: the local states only, and no REUSE-of-empty check (the other states of the step are
// decided later).  Slots that do not exist for a query partition are never listed and never flagged.
__global__ void __launch_bounds__(1024) worklist_kernel(const uint8_t *mask, int32_t *tc, int32_t *worklist,
                                                        int32_t *status, const SlotRange *slot_tab, int P, int S,
                                                        int group_mode, int step, const int32_t *off, int4 *tile_pairs) {
    __shared__ int warp_cnt[32];
    const int total = P * S, e = threadIdx.x;
    bool f = false;
    if (e < total) {
        const int i = e / S, s = e - i * S;
        const bool exists = slot_tab[e].n1 + slot_tab[e].n2 > 0;
        const int local = group_mode ? 0 : i;
        f = exists && (mask ? (mask[e] != 0) : (s == local));
        if (f) tc[e] = step;
        else if (exists && mask && tc[e] < 0) atomicOr(status, STATUS_REUSE_EMPTY);
    }
    // position of a COMPUTE entry = number of COMPUTE entries with a smaller flat index
    const unsigned bal = __ballot_sync(0xFFFFFFFFu, f);
    const int lane = e & 31, warp = e >> 5;
    if (lane == 0) warp_cnt[warp] = __popc(bal);
    __syncthreads();
    int pos = __popc(bal & ((1u << lane) - 1u)), cnt = 0;
    for (int w = 0; w < 32; ++w) {
        const int c = warp_cnt[w];
        cnt += c;
        if (w < warp) pos += c;
    }
    if (f) worklist[1 + pos] = (e / S) | ((e % S) << 8);
    if (e == 0) worklist[0] = cnt;
    if (tile_pairs != nullptr) build_tile_pairs(f, off, P, tile_pairs);   // pair mode (S == P): the attention kernel's items
}

// Pair mode: the work items of the attention kernel.  For every KV partition j the 128-row query tiles of all query
// partitions i with (i, j) COMPUTE, in the order of i, taken two at a time: a partition with an odd number of tiles
// shares its last item with the first tile of the next one (both attend to the same keys), so no item runs half
// empty except the last of a KV partition.  Items are listed by j, so neighbours in the list share K/V.
// (called by all 1024 threads of worklist_kernel; is_compute = this thread's pair (i, j) = (e / P, e % P) is COMPUTE)
__device__ void build_tile_pairs(bool is_compute, const int32_t *off, int P, int4 *out) {
    __shared__ uint8_t flag[DT_MAX_P * DT_MAX_P];
    __shared__ int items_of[DT_MAX_P], base_of[DT_MAX_P + 1];
    const int e = threadIdx.x;
    if (e < P * P) flag[e] = is_compute ? 1 : 0;
    __syncthreads();
    if (e < P) {   // thread j: tiles of column j
        int tiles = 0;
        for (int i = 0; i < P; ++i)
            if (flag[i * P + e]) tiles += (off[i + 1] - off[i] + ATTN_TILE - 1) / ATTN_TILE;
        items_of[e] = (tiles + 1) / 2;
    }
    __syncthreads();
    if (e == 0) {
        int acc = 0;
        for (int j = 0; j < P; ++j) { base_of[j] = acc; acc += items_of[j]; }
        base_of[P] = acc;
        out[0] = make_int4(acc, 0, 0, 0);
    }
    __syncthreads();
    // one warp per KV partition j: lane l writes the items l, l + 32, ... of the column
    const int j = e >> 5, lane = e & 31;
    if (j < P) {
        for (int it = lane; it < items_of[j]; it += 32) {
            int4 rec = make_int4(0, 0, -1, 0);
            int seen = 0;             // tiles of the column before partition i
            for (int i = 0; i < P; ++i) {
                if (!flag[i * P + j]) continue;
                const int t_i = (off[i + 1] - off[i] + ATTN_TILE - 1) / ATTN_TILE;
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    const int g = 2 * it + q - seen;      // index of the item's q-th tile within partition i
                    if (g >= 0 && g < t_i) {
                        if (q == 0) { rec.x = i | (j << 8); rec.y = g; }
                        else { rec.z = i; rec.w = g; }
                    }
                }
                seen += t_i;
            }
            out[1 + base_of[j] + it] = rec;
        }
    }
}

// Decisions for a grouped cache (Section 4.2.1 - 4.2.3): W[i][s] from the partial sums; every non-local slot
// that exists is one decision unit whose measure is the importance of its whole key set (the sum of its
// members' weights, Eq. 12, which is what the slot's LSE yields directly).  COMPUTE iff measure > eps
// (Eq. 13), or the units of largest measure taken in rank order while their member pairs fit into K - P.
__global__ void __launch_bounds__(1024) plan_slots_kernel(PlanSlotsParams p) {
    __shared__ double sum_s[DT_MAX_P * DT_MAX_P];
    __shared__ RankScratch sc;
    __shared__ double edge[2];
    __shared__ int n_units;
    const int P = p.P, S = p.S, total = P * S, g = p.group_size;
    const int e = threadIdx.x;
    const int i = e / S, s = e - i * S;
    load_sums(p.sums_in, p.partials, P, S, p.BH, p.chunks, reinterpret_cast<double *>(sc.k1), sum_s);   // sc.k1 is scratch here
    if (p.sums_out) {
        if (e < total) p.sums_out[e] = sum_s[e];
        return;
    }
    double m = 0.0;
    int size = 0, dist = 0;
    if (e < total) {
        m = sum_s[e] / ((double)p.count_bh * (double)(p.off[i + 1] - p.off[i]));
        if (p.w_out) p.w_out[e] = m;
        size = (s == 0) ? 0 : (int)p.members[e];   // the local slot is no unit: always COMPUTE
        const int gi = i / g, k = s - 1;
        dist = k > gi ? k - gi : gi - k;
    }
    if (e < 2) edge[e] = 0.0;
    __syncthreads();
    int taken = 0;
    if (p.mode_target) {
        taken = take_by_rank(sc, m, size, dist, total, p.K - P, edge, &n_units);
    } else {
        sc.dec[e] = (e < total && size > 0 && m > p.eps) ? 1 : 0;
        __syncthreads();
    }
    if (e < total) p.mask[e] = (s == 0 || sc.dec[e]) ? 1 : 0;
    if (e == 0 && p.eps_out) {
        double eps = p.eps;
        if (p.mode_target) {
            if (n_units == 0 || taken == n_units) eps = 0.0;
            else if (taken == 0) eps = edge[1];
            else eps = 0.5 * (edge[0] + edge[1]);
        }
        *p.eps_out = eps;
    }
}

// t_c after Dynamic Group State Compose (Eq. 15, k = 2): slot 0 (local) keeps its step; new slot 1 + k takes
// the older of old slots 1 + 2k and 2 + 2k that exist (-1 if one of them was never computed).
__global__ void tc_compose_kernel(int32_t *tc, const uint32_t *nonempty_old, int P, int S_old, int S_new) {
    __shared__ int32_t old_s[DT_MAX_P * DT_MAX_P];
    const int e = threadIdx.x;
    if (e < P * S_old) old_s[e] = tc[e];
    __syncthreads();
    if (e < P * S_new) {
        const int i = e / S_new, s = e - i * S_new;
        int32_t v;
        if (s == 0) {
            v = old_s[i * S_old];
        } else {
            v = 0x7FFFFFFF;
            bool any = false;
            for (int o = 2 * s - 1; o <= 2 * s && o < S_old; ++o)
                if (nonempty_old[i] >> o & 1u) { v = min(v, old_s[i * S_old + o]); any = true; }
            if (!any) v = -1;
        }
        tc[e] = v;
    }
}

// Self-test of the bounded-wait machinery: one thread waits on an mbarrier that nobody will ever
// arrive at, with a short limit; the wait must give up, record STATUS_WAIT_TIMEOUT and return.
__global__ void wait_timeout_selftest_kernel(int32_t *status, long long limit_cycles) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        fence_mbar_init();
        if (!mbar_wait_bounded(smem_u32(&bar), 0, &abort_flag, limit_cycles)) atomicOr(status, STATUS_WAIT_TIMEOUT);
    }
}

}  // namespace

cudaError_t launch_wait_timeout_selftest(int32_t *status, long long limit_cycles, cudaStream_t stream) {
    wait_timeout_selftest_kernel<<<1, 32, 0, stream>>>(status, limit_cycles);
    return cudaGetLastError();
}

namespace {
}  // namespace

cudaError_t launch_plan_partial(const PlanParams &p, cudaStream_t stream) {
    dim3 grid((unsigned)p.chunks, (unsigned)p.P, (unsigned)p.BH);
    if (p.S <= 8) plan_partial_kernel<8><<<grid, PLAN_THREADS, 0, stream>>>(p);
    else if (p.S <= 16) plan_partial_kernel<16><<<grid, PLAN_THREADS, 0, stream>>>(p);
    else plan_partial_kernel<32><<<grid, PLAN_THREADS, 0, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_plan_final(const PlanFinalParams &p, cudaStream_t stream) {
    plan_final_kernel<<<1, 1024, 0, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_worklist(const uint8_t *mask, int32_t *tc, int32_t *worklist, int32_t *status, const SlotRange *slot_tab,
                            int P, int S, int group_mode, int step, const int32_t *off, int4 *tile_pairs, cudaStream_t stream) {
    worklist_kernel<<<1, 1024, 0, stream>>>(mask, tc, worklist, status, slot_tab, P, S, group_mode, step, off, tile_pairs);
    return cudaGetLastError();
}

cudaError_t launch_plan_slots(const PlanSlotsParams &p, cudaStream_t stream) {
    plan_slots_kernel<<<1, 1024, 0, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_tc_compose(int32_t *tc, const uint32_t *nonempty_old, int P, int S_old, int S_new, cudaStream_t stream) {
    tc_compose_kernel<<<1, 1024, 0, stream>>>(tc, nonempty_old, P, S_old, S_new);
    return cudaGetLastError();
}

}  // namespace dt

// ---------------------------------------------------------------------------------------------
// dt_plan_static: the plan computation with no allocation anywhere on its path.
//
// Stage 1's per-block partial sums need scratch memory.  dt_plan takes it from the context, which
// dt_create allocated; this entry point instead keeps it in a device array that is part of the
// library image, so a caller that must not allocate can still plan.
namespace {

constexpr int STATIC_PLAN_OFFSET_SLOTS = 64;                       // ints reserved for the P+1 offsets
constexpr size_t STATIC_PLAN_MAX_PARTIALS = 262144;                // floats (1 MiB) for stage-1 partial sums
constexpr int STATIC_PLAN_MAX_DEVICES = 64;

static __device__ __align__(256) float g_plan_static_scratch[STATIC_PLAN_OFFSET_SLOTS + STATIC_PLAN_MAX_PARTIALS];

// In host code the array's name is only a handle: the device address is looked up once per device.
float *g_plan_static_ptr[STATIC_PLAN_MAX_DEVICES] = {nullptr};

// The partition offsets reach the device as a kernel argument: they are copied when the launch is
// made, so nothing refers to the caller's host array after dt_plan_static has returned.
struct StaticOffsets {
    int32_t v[DT_MAX_P + 1];
};
__global__ void static_offsets_kernel(StaticOffsets o, int n, int32_t *dst) {
    if ((int)threadIdx.x < n) dst[threadIdx.x] = o.v[threadIdx.x];
}

}  // namespace

extern "C" dt_status dt_plan_static(const float *lse_state_dev, const int32_t *part_offsets_host, int32_t B, int32_t H,
                                    int32_t L, int32_t P, double eps, double target_fraction, uint8_t *mask_dev,
                                    double *w_dev, double *eps_out_dev, void *stream) {
    if (!lse_state_dev || !part_offsets_host || !mask_dev) return DT_ERR_INVALID_ARG;
    if (B < 1 || H < 1 || L < 1 || P < 1) return DT_ERR_INVALID_ARG;
    if (P > DT_MAX_P || (long long)B * H > 65535) return DT_ERR_UNSUPPORTED;
    if (part_offsets_host[0] != 0 || part_offsets_host[P] != L) return DT_ERR_INVALID_ARG;
    int n_max = 0;
    for (int i = 0; i < P; ++i) {
        const int n = part_offsets_host[i + 1] - part_offsets_host[i];
        if (n <= 0) return DT_ERR_INVALID_ARG;
        n_max = n > n_max ? n : n_max;
    }
    if (target_fraction < 0 && !(eps == eps && eps - eps == 0.0)) return DT_ERR_INVALID_ARG;   // eps must be finite
    if (target_fraction > 1.0 || target_fraction != target_fraction) return DT_ERR_INVALID_ARG;
    const int chunks = (n_max + dt::PLAN_CHUNK_ROWS - 1) / dt::PLAN_CHUNK_ROWS;
    const size_t need = (size_t)B * H * P * chunks * P;
    if (need > STATIC_PLAN_MAX_PARTIALS) return DT_ERR_UNSUPPORTED;   // problem larger than the built-in scratch

    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= STATIC_PLAN_MAX_DEVICES) return DT_ERR_CUDA;
    if (g_plan_static_ptr[device] == nullptr) {   // first call on this device: resolve the array's device address
        float *ptr = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void **>(&ptr), g_plan_static_scratch) != cudaSuccess || !ptr)
            return DT_ERR_CUDA;
        g_plan_static_ptr[device] = ptr;
    }
    float *scratch = g_plan_static_ptr[device];
    int32_t *off_dev = reinterpret_cast<int32_t *>(scratch);
    float *partials = scratch + STATIC_PLAN_OFFSET_SLOTS;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    StaticOffsets ov;
    for (int i = 0; i <= P; ++i) ov.v[i] = part_offsets_host[i];
    static_offsets_kernel<<<1, 64, 0, st>>>(ov, P + 1, off_dev);
    if (cudaGetLastError() != cudaSuccess) return DT_ERR_CUDA;

    dt::PlanParams pp;
    pp.lse_state = lse_state_dev;
    pp.off = off_dev;
    pp.partials = partials;
    pp.nonempty = nullptr;
    pp.only_if = nullptr;
    pp.P = P; pp.S = P; pp.BH = B * H; pp.L = L; pp.chunks = chunks;
    pp.R = (long long)B * H * L;
    if (dt::launch_plan_partial(pp, st) != cudaSuccess) return DT_ERR_CUDA;
    dt::PlanFinalParams pf;
    pf.partials = partials;
    pf.off = off_dev;
    pf.P = P; pf.BH = pp.BH; pf.chunks = chunks;
    pf.mode_target = target_fraction >= 0 ? 1 : 0;
    const int total = P * P;
    int K = (int)floor(target_fraction * total + 0.5);
    K = K < P ? P : (K > total ? total : K);
    pf.K = K;
    pf.group_size = 1;
    pf.eps = eps;
    pf.mask = mask_dev;
    pf.w_out = w_dev;
    pf.eps_out = eps_out_dev;
    pf.sums_in = nullptr; pf.sums_out = nullptr; pf.count_bh = pp.BH;
    if (dt::launch_plan_final(pf, st) != cudaSuccess) return DT_ERR_CUDA;
    return DT_OK;
}
