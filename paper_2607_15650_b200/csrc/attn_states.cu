// dt_attn_states: Eq. 1 for every COMPUTE pair -- flash attention of the query tiles of
// partition i against the keys of partition j only, emitting the partition-normalised output
// OUT_ij and LSE_ij straight into the state cache.  REUSE pairs never appear in the work list,
// so they cost no instruction and no byte.  With a grouped cache (Section 4.2.1) a work item is a
// (query partition, slot) whose keys are the slot's one or two key ranges: the group's state, the
// composition (Eq. 2) of its members' states, comes out of one pass over their keys.
//
// One persistent CTA per SM walks the work list (b*h slowest, then KV partition, then the query tiles of every query
// partition that computes it, two per item), so CTAs running at the same time share one head's K/V partition through L2.
// The two 128-row query tiles of an item need not be neighbours: a partition with an odd number of tiles leaves one over,
// which is paired with the first tile of the next query partition that attends to the same KV partition.
//
// Per CTA (12 warps; the producer warpgroup gives registers to the softmax warpgroups):
//   warps 0-3 / 4-7  softmax warpgroups for query tile 0 / 1 (128 rows each, one row per thread)
//   warp 8           TMA producer: Q tiles once per work item, K and V tiles through a ring, in the order the MMAs
//                    consume them (K_0, K_1, V_0, K_2, V_1, ...)
//   warps 9, 10      MMA issuers of query tile 0 / 1: the whole warp runs the (warp-uniform) control flow and address
//                    arithmetic, one lane issues tcgen05.mma / tcgen05.commit.  Each waits for its own barriers and
//                    for the K/V tiles itself, and hands the stages (and Q's place) back with commits of its own
//   warp 11          idle (completes the producer warpgroup for the register hand-over)
// TMEM: S | P0 | P1 | O0 | O1.  S_t = Q K_t^T (fp32) lands in S; the softmax thread reads its row, writes P =
// exp2(s*scale*log2e - m) as packed bf16 (fp16 for fp16 inputs) into P's own columns, and the PV MMA takes P from
// TMEM as its A operand and V from shared memory (MN-major) as B, accumulating in O.  P_t V_t therefore never
// stands between a softmax and its next S.  There is ONE place for S, which the two query tiles use in turn: a softmax
// thread takes its whole row into registers at once, so the place is busy only from a Q K^T to the read that follows
// it.  A softmax asks for its next S half-way through a tile (s_req); its MMA warp then issues Q K_{t+1}^T, and P_t V_t
// behind it once P_t is stored.  The turns at S keep the two tiles' softmaxes half a tile apart, so that one takes its
// exponentials while the other loads S, stores P or runs its epilogue.
// P is computed against the reference maximum m of the earlier tiles, never against the tile's own: stale
// references cancel exactly in OUT = O / l and LSE = m + log l.  bf16 inputs: when a row's running sum l reaches
// LSUM_TRIGGER, m moves up by floor(log2 l) binades and O, l are scaled by that power of two (exact).  fp16
// inputs (P overflows at 2^16): when a tile's row sum reaches ROWSUM_TRIGGER the tile's own maximum is taken and,
// if it lies more than 2^RESCALE_THRESHOLD above the reference, the reference moved and P computed again.
// Epilogue: the rows leave through warp-private shared-memory tiles so that the cache is written in whole
// 128-byte lines; the fused mode (dt_attn_fused) composes the fresh state with the composed reuse state in
// registers and stores the attention output itself.
//
// Every wait on an mbarrier is bounded; on expiry the CTA records STATUS_WAIT_TIMEOUT, leaves
// its loops, frees TMEM and returns.
#include <cuda_bf16.h>

#include "dt_internal.h"
#include "ptx_sm100.cuh"

namespace dt {
namespace {

constexpr int NUM_SOFTMAX_THREADS = ATTN_NQ * 128;
constexpr int TMA_WARP = NUM_SOFTMAX_THREADS / 32;
constexpr int MMA_WARP = TMA_WARP + 1;
constexpr int MMA_WARP_1 = TMA_WARP + 2;   // the MMA issuer of query tile 1 (MMA_WARP: query tile 0)
constexpr int ATTN_THREADS = NUM_SOFTMAX_THREADS + 128;  // producer warpgroup: TMA, MMA and two idle warps
// Per-thread register budgets after the role split.  setmaxnreg.inc can only take registers that a
// setmaxnreg.dec of the same CTA has released (registers the launch left unallocated do not count);
// a request beyond that blocks forever.  So with LAUNCH_REGS registers per thread at launch:
//   (REGS_SOFTMAX - LAUNCH_REGS) * softmax threads  <=  (LAUNCH_REGS - REGS_PRODUCER) * 128.
// LAUNCH_REGS is what ptxas assigns under __launch_bounds__(384, 1); attn_states_configure() checks it
// against the compiled kernels and refuses to run on a mismatch.
constexpr int LAUNCH_REGS = 168, REGS_SOFTMAX = 208, REGS_PRODUCER = 88;
static_assert((REGS_SOFTMAX - LAUNCH_REGS) * NUM_SOFTMAX_THREADS <= (LAUNCH_REGS - REGS_PRODUCER) * 128,
              "softmax warps would wait forever for registers nobody releases");
constexpr long long WAIT_LIMIT_CYCLES = 4000000000ll;   // SM clock cycles: about 2 s
constexpr float ROWSUM_TRIGGER = 512.0f;   // fp16 inputs: a row sum of P at or above this sends the tile through the slow path
constexpr float LSUM_TRIGGER = 16777216.0f;   // bf16 inputs: a running sum l at or above 2^24 moves the row's reference
constexpr float RESCALE_THRESHOLD = 1.0f;  // log2 units: in the slow path the reference moves if the maximum grew by more
// Key pairs (of every 8) whose exp2 runs as a cubic on the FMA pipe instead of the MUFU.  D = 64 is bound by the
// exponentials (2048 MUFU cycles per 256 x 128 tile pair against 1536 of MMA issue): two pairs in eight, every
// fourth pair, measured +2 % over one and about +10 % over none there (two adjacent pairs: +1 %; three: -8 %).  At D = 128 one pair in eight saves 4 %
// of the cycles and costs 3 % of the time at full size: the GPU runs at its power cap there, and an exponential takes
// less energy on the MUFU.
#ifndef DT_POLY_PER_8_D64
#define DT_POLY_PER_8_D64 2
#endif
#ifndef DT_POLY_PER_8_D128
#define DT_POLY_PER_8_D128 0
#endif
// After how many (1..4) of a tile's four 32-key pieces the softmax asks for the next tile's S.
#ifndef DT_S_REQ_PIECE
#define DT_S_REQ_PIECE 2
#endif

template <int D>
struct Cfg {
    static constexpr int NHALF = D / 64;                      // 64-element (128-byte) swizzle atoms per row
    static constexpr int HALF_BYTES = ATTN_TILE * 128;        // one [128 rows x 64 bf16] box
    static constexpr int TILE_BYTES = NHALF * HALF_BYTES;     // one Q, K or V tile
    static constexpr int STAGES = (D == 128) ? 4 : 8;         // K/V ring depth
    static constexpr int Q_BYTES = ATTN_NQ * TILE_BYTES;
    static constexpr int KV_BYTES = STAGES * TILE_BYTES;
    static constexpr int OUT_STAGE_BYTES = ATTN_TILE * 128;   // epilogue staging per query tile: 4 warps x [32 rows x 128 bytes]
    static constexpr int OUT_BYTES = ATTN_NQ * OUT_STAGE_BYTES;
    static constexpr int NBARS = 2 + 2 * STAGES + 7 * ATTN_NQ;
    static constexpr int SMEM_BYTES = 1024 /*alignment slack*/ + Q_BYTES + KV_BYTES + OUT_BYTES + NBARS * 8 + 64;
    // TMEM columns: S | P0 | P1 | O0 | O1.  P has columns of its own, so that P_t V_t never stands between a softmax
    // and its next S, and there is ONE place for S, which the two query tiles share: a softmax thread takes its whole row
    // of S into registers as soon as it arrives, so the place is free again a few dozen cycles after every Q K^T.  (At
    // D = 128 the 512 columns leave no room for a second place; at D = 64 there would be room, but the turns the tiles
    // take at the one place are what keeps their softmaxes half a tile apart, and measured 8 % faster than two places.)
    // After how many of a tile's four 32-key pieces the softmax asks for the next tile's S:
    static constexpr int S_REQ = DT_S_REQ_PIECE;
    static_assert(S_REQ >= 1 && S_REQ <= 4, "the request for S comes after one to four of a tile's 32-key pieces");
    static constexpr int POLY_PER_8 = (D == 64) ? DT_POLY_PER_8_D64 : DT_POLY_PER_8_D128;
    static constexpr int S_COL = 0;
    static constexpr int P_COL = 128;                                            // P tile q: P_COL + q*P_STRIDE
    static constexpr int P_STRIDE = 64;
    static constexpr int O_COL = 128 + ATTN_NQ * 64;                             // O tile q: O_COL + q*D
    static_assert(O_COL + ATTN_NQ * D <= 512, "beyond the tensor memory of an SM");
};

struct Bars {
    uint32_t q_full, q_empty;
    uint32_t kv_full, kv_empty;   // + 8*stage
    uint32_t s_full, p_full, o_full, o_free, pv_done, s_free, s_req;  // + 8*q
};

// Place of an item's K/V tiles in the order they are loaded and consumed --
// K_0, K_1, V_0, K_2, V_1, ..., K_{n-1}, V_{n-2}, V_{n-1}: Q K_{t+1}^T is issued as soon as S_t has been read,
// before P_t V_t.
__device__ __forceinline__ uint32_t k_place(int t) { return t == 0 ? 0u : (uint32_t)(2 * t - 1); }
__device__ __forceinline__ uint32_t v_place(int t, int tiles) { return t + 1 == tiles ? (uint32_t)(2 * tiles - 1) : (uint32_t)(2 * t + 2); }

// Position in the K/V ring: stage index and the parity of its current use.
template <int STAGES>
struct RingPos {
    uint32_t st = 0, ph = 0;
    __device__ __forceinline__ void advance() {
        if (++st == STAGES) { st = 0; ph ^= 1u; }
    }
};

struct WorkItem {
    int bh, b, h, i, slot;
    // The two query tiles of the item: first row (global token index), valid rows (0: the tile is absent), query
    // partition and tile index within it.  In pair mode the two tiles may come from different query partitions (they
    // share the K/V stream of slot j); otherwise they are the two halves of one 256-row block of partition i.
    int qrow[ATTN_NQ], qn[ATTN_NQ], qi[ATTN_NQ], qt[ATTN_NQ];
    int r1, n1;     // first key range of the slot
    int r2, n2;     // second key range (n2 == 0: none)
    int tiles1;     // ceil(n1 / 128)
    int tiles;      // tiles1 + ceil(n2 / 128); fused mode: tiles of the partition's tile table
    const int2 *tab; // fused mode: (first key, keys that count) per tile
    // first key of K/V tile t, and how many of its 128 keys count (may exceed 128)
    template <bool FUSED>
    __device__ __forceinline__ int2 tile(int t) const {
        if constexpr (FUSED) return __ldg(tab + t);
        return t < tiles1 ? make_int2(r1 + t * ATTN_TILE, n1 - t * ATTN_TILE)
                          : make_int2(r2 + (t - tiles1) * ATTN_TILE, n2 - (t - tiles1) * ATTN_TILE);
    }
};

// Work index -> item.  Returns false when the item has no query rows (or no keys).
// per_bh = work items per (b, h): tile pairs of the pair-mode list, COMPUTE states x query blocks with a grouped cache,
// or P x query blocks in fused mode.
template <bool FUSED>
__device__ __forceinline__ long long work_per_bh(const AttnParams &p) {
    if constexpr (FUSED) return (long long)p.P * p.qblocks_max;
    if (p.tile_pairs != nullptr) return p.tile_pairs[0].x;
    return (long long)p.worklist[0] * p.qblocks_max;
}

template <bool FUSED>
__device__ __forceinline__ bool decode_work(const AttnParams &p, long long per_bh, long long w, WorkItem &it) {
    const int bh_launch = (int)(w / per_bh);          // index among the (b, h) of this launch
    const int rem = (int)(w - (long long)bh_launch * per_bh);
    it.b = bh_launch / p.H_launch;
    it.h = p.h0 + bh_launch - it.b * p.H_launch;
    it.bh = it.b * p.H + it.h;
    if (!FUSED && p.tile_pairs != nullptr) {
        // pair mode: (i_a | j << 8, tile_a, i_b or -1, tile_b) -- two 128-row query tiles that attend to KV partition j
        const int4 e = __ldg(p.tile_pairs + 1 + rem);
        it.i = e.x & 0xFF;
        it.slot = e.x >> 8;
        const int ia[ATTN_NQ] = {it.i, e.z}, ta[ATTN_NQ] = {e.y, e.w};
#pragma unroll
        for (int q = 0; q < ATTN_NQ; ++q) {
            const bool have = ia[q] >= 0;
            const int iq = have ? ia[q] : it.i;
            it.qi[q] = iq;
            it.qt[q] = ta[q];
            it.qrow[q] = p.off[iq] + (have ? ta[q] : e.y) * ATTN_TILE;
            it.qn[q] = have ? min(p.off[iq + 1] - it.qrow[q], ATTN_TILE) : 0;
        }
    } else {
        const int pair = rem / p.qblocks_max;
        const int qb = rem - pair * p.qblocks_max;
        const int code = FUSED ? pair : p.worklist[1 + pair];
        it.i = code & 0xFF;
        it.slot = code >> 8;
        const int qs = p.off[it.i], qe = p.off[it.i + 1];
#pragma unroll
        for (int q = 0; q < ATTN_NQ; ++q) {
            it.qi[q] = it.i;
            it.qt[q] = qb * ATTN_NQ + q;
            it.qrow[q] = qs + it.qt[q] * ATTN_TILE;
            it.qn[q] = max(min(qe - it.qrow[q], ATTN_TILE), 0);
        }
    }
    if constexpr (FUSED) {
        it.tab = p.tile_tab + (long long)it.i * p.max_tiles;
        it.tiles = p.tile_cnt[it.i];
        it.r1 = it.n1 = it.r2 = it.n2 = it.tiles1 = 0;
        return it.qn[0] > 0 && it.tiles > 0;
    }
    it.tab = nullptr;
    const int4 rg = *reinterpret_cast<const int4 *>(p.slot_tab + it.i * p.S + it.slot);
    it.r1 = rg.x; it.n1 = rg.y; it.r2 = rg.z; it.n2 = rg.w;
    it.tiles1 = (it.n1 + ATTN_TILE - 1) / ATTN_TILE;
    it.tiles = it.tiles1 + (it.n2 + ATTN_TILE - 1) / ATTN_TILE;
    return it.qn[0] > 0;
}

// 32 consecutive elements of a cached state row as fp32
__device__ __forceinline__ void load_state_chunk(const float *src, float (&v)[32]) {
#pragma unroll
    for (int c = 0; c < 32; c += 4) {
        const float4 x = __ldcs(reinterpret_cast<const float4 *>(src + c));
        v[c] = x.x; v[c + 1] = x.y; v[c + 2] = x.z; v[c + 3] = x.w;
    }
}
__device__ __forceinline__ void load_state_chunk(const __nv_bfloat16 *src, float (&v)[32]) {
#pragma unroll
    for (int c = 0; c < 32; c += 8) {
        const uint4 x = __ldcs(reinterpret_cast<const uint4 *>(src + c));
        const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            v[c + 2 * e] = __uint_as_float(w[e] << 16);
            v[c + 2 * e + 1] = __uint_as_float(w[e] & 0xFFFF0000u);
        }
    }
}

// A running sum l that reached LSUM_TRIGGER moves the row's reference up by e = floor(log2(l)) binades:
// this thread's row of O (fp32, D columns) times 2^-e, in place; returns e (0 for a row below the trigger).
// Out of line: it runs once in many tiles and would only lengthen the softmax loop.
template <int D>
__device__ __noinline__ int move_reference(uint32_t o_tmem, float row_sum) {
    const bool need = !(row_sum < LSUM_TRIGGER);   // also true for inf / NaN
    const int e = need ? min(((__float_as_int(row_sum) >> 23) & 0xFF) - 127, 126) : 0;
    const float alpha = __int_as_float((127 - e) << 23);
#pragma unroll 1
    for (int c0 = 0; c0 < D; c0 += 32) {
        uint32_t o[32];
        tmem_ld_x32(o_tmem + c0, o);
        tmem_wait_ld();
#pragma unroll
        for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
        tmem_st_x32(o_tmem + c0, o);
    }
    tmem_wait_st();
    return e;
}

template <int D, typename StateT, bool FUSED, bool FP16>
__global__ void __launch_bounds__(ATTN_THREADS, 1)
attn_states_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                   const __grid_constant__ CUtensorMap tmap_v, const AttnParams p) {
    using C = Cfg<D>;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    // 1024-byte aligned carve-up (the 128-byte swizzle pattern repeats every 1024 bytes)
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t q_smem = smem_base;
    const uint32_t kv_smem = q_smem + C::Q_BYTES;
    const uint32_t out_smem = kv_smem + C::KV_BYTES;        // 1024-byte aligned: every size above is a multiple
    const uint32_t bar_base = out_smem + C::OUT_BYTES;
    Bars bars;
    bars.q_full = bar_base;
    bars.q_empty = bar_base + 8;
    bars.kv_full = bar_base + 16;
    bars.kv_empty = bars.kv_full + 8 * C::STAGES;
    bars.s_full = bars.kv_empty + 8 * C::STAGES;
    bars.p_full = bars.s_full + 8 * ATTN_NQ;
    bars.o_full = bars.p_full + 8 * ATTN_NQ;
    bars.o_free = bars.o_full + 8 * ATTN_NQ;
    bars.pv_done = bars.o_free + 8 * ATTN_NQ;   // the PV MMAs that read P[q] have completed
    bars.s_free = bars.pv_done + 8 * ATTN_NQ;   // S[q] has been read (and the next K tile has landed)
    bars.s_req = bars.s_free + 8 * ATTN_NQ;     // shared place for S: query tile q's softmax will be ready for its next S shortly

    // warp index through a shuffle: the compiler then knows that it is the same in all lanes of a warp
    const int warp = __shfl_sync(0xFFFFFFFFu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    volatile int *abort_ptr = &abort_flag;

    if (warp == TMA_WARP && lane == 0) {
        abort_flag = 0;
        mbar_init(bars.q_full, 1);
        // each of the two MMA warps hands Q's place and the K/V stages back with a commit of its own
        mbar_init(bars.q_empty, 2);
        for (int s = 0; s < C::STAGES; ++s) {
            mbar_init(bars.kv_full + 8 * s, 1);
            mbar_init(bars.kv_empty + 8 * s, 2);
        }
        for (int q = 0; q < ATTN_NQ; ++q) {
            mbar_init(bars.s_full + 8 * q, 1);
            mbar_init(bars.p_full + 8 * q, 128);   // P stored (the tile's 128 softmax threads)
            mbar_init(bars.s_free + 8 * q, 128);   // S read (only [0] is used, by both tiles in turn)
            mbar_init(bars.o_full + 8 * q, 1);
            mbar_init(bars.o_free + 8 * q, 128);
            mbar_init(bars.pv_done + 8 * q, 1);
            mbar_init(bars.s_req + 8 * q, 128);
        }
        fence_mbar_init();
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_base_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;

    const long long npairs = work_per_bh<FUSED>(p);   // work items per (b, h)
    const long long total_work = npairs * p.B * p.H_launch;

    if (warp >= TMA_WARP) {
      reg_dealloc<REGS_PRODUCER>();
      if (warp == TMA_WARP) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            prefetch_tensormap(&tmap_q);
            prefetch_tensormap(&tmap_k);
            prefetch_tensormap(&tmap_v);
            uint32_t q_phase = 0;
            RingPos<C::STAGES> ring;
            bool ok = true;
            for (long long w = blockIdx.x; w < total_work && ok; w += gridDim.x) {
                WorkItem it;
                if (!decode_work<FUSED>(p, npairs, w, it)) continue;
                ok = mbar_wait_bounded(bars.q_empty, q_phase ^ 1u, abort_ptr, WAIT_LIMIT_CYCLES);
                if (!ok) break;
                mbar_arrive_expect_tx(bars.q_full, C::Q_BYTES);
#pragma unroll
                for (int q = 0; q < ATTN_NQ; ++q)
#pragma unroll
                    for (int hf = 0; hf < C::NHALF; ++hf)
                        tma_load_4d(q_smem + q * C::TILE_BYTES + hf * C::HALF_BYTES, &tmap_q, bars.q_full, hf * 64, it.h,
                                    it.qrow[q], it.b);
                q_phase ^= 1u;
                for (int n = 0; n < 2 * it.tiles && ok; ++n) {
                    // place n of the item's load order: K_0 | K_{(n+1)/2} for odd n | V_{(n-2)/2} for even n | V_{tiles-1} last
                    const bool is_k = (n == 0) || ((n & 1) && n + 1 < 2 * it.tiles);
                    const int t = is_k ? (n + 1) / 2 : (n + 1 == 2 * it.tiles ? it.tiles - 1 : (n - 2) / 2);
                    const int key0 = it.template tile<FUSED>(t).x;
                    const uint32_t st = ring.st, ph = ring.ph;
                    ok = mbar_wait_bounded(bars.kv_empty + 8 * st, ph ^ 1u, abort_ptr, WAIT_LIMIT_CYCLES);
                    if (!ok) break;
                    mbar_arrive_expect_tx(bars.kv_full + 8 * st, C::TILE_BYTES);
#pragma unroll
                    for (int hf = 0; hf < C::NHALF; ++hf)
                        tma_load_4d(kv_smem + st * C::TILE_BYTES + hf * C::HALF_BYTES, is_k ? &tmap_k : &tmap_v,
                                    bars.kv_full + 8 * st, hf * 64, it.h, key0, it.b);
                    ring.advance();
                }
            }
            if (!ok) {
                if (!*abort_ptr) atomicOr(p.status, STATUS_WAIT_TIMEOUT);
                *abort_ptr = 1;
                // let loads that are still in flight land before the CTA's shared memory goes away
                const uint64_t t0 = global_timer_ns();
                while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
            }
        }
      } else if (warp == MMA_WARP || warp == MMA_WARP_1) {
        // ------------------------------------------------------------ MMA issuer
        {
            const bool leader = (lane == 0);
            // Every wait ends in a vote, so that no lane runs ahead of the issuing one: a lane that polled a barrier
            // two phases late would read the parity of the wrong phase and never see it complete.
            auto wait_all = [&](uint32_t bar, uint32_t parity, volatile int *abort_flag, long long limit) -> bool {
                return __all_sync(0xFFFFFFFFu, mbar_wait_bounded(bar, parity, abort_flag, limit)) != 0;
            };
            constexpr uint32_t IDESC_QK = make_idesc_bf16_f32(128, ATTN_TILE, false, FP16);
            constexpr uint32_t IDESC_PV = make_idesc_bf16_f32(128, D, true, FP16);
            uint32_t q_phase = 0, of_phase = 0;
            bool ok = true;

            // Descriptors differ only in their 14-bit start-address field (units of 16 bytes), so each
            // operand's descriptor is its base plus a small constant.
            const uint64_t qdesc0 = make_smem_desc_sw128(q_smem, 16, 1024);
            const uint64_t kdesc0 = make_smem_desc_sw128(kv_smem, 16, 1024);
            const uint64_t vdesc0 = make_smem_desc_sw128(kv_smem, C::HALF_BYTES, 1024);
            // S[q] = Q[q] K^T for the K tile in ring stage `st`
            auto issue_qk = [&](int q, uint32_t st) {
                const uint64_t a0 = qdesc0 + (uint64_t)((q * C::TILE_BYTES) >> 4);
                const uint64_t b0 = kdesc0 + (uint64_t)((st * C::TILE_BYTES) >> 4);
                const uint32_t d = tmem_base + C::S_COL;
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t koff = ((kk / 4) * C::HALF_BYTES + (kk % 4) * 32) >> 4;
                    if (leader) mma_ss(d, a0 + koff, b0 + koff, IDESC_QK, kk > 0 ? 1u : 0u);
                }
            };
            // O[q] (+)= P[q] V for the V tile in ring stage `st`
            auto issue_pv = [&](int q, uint32_t st, bool accumulate) {
                const uint64_t b0 = vdesc0 + (uint64_t)((st * C::TILE_BYTES) >> 4);
                const uint32_t d = tmem_base + C::O_COL + q * D, a = tmem_base + C::P_COL + q * C::P_STRIDE;
#pragma unroll
                for (int kk = 0; kk < ATTN_TILE / 16; ++kk)
                    if (leader) mma_ts(d, a + kk * 8, b0 + (uint64_t)((kk * 2048) >> 4), IDESC_PV, (accumulate || kk > 0) ? 1u : 0u);
            };

            {
                // One MMA warp per query tile (this one: mq), so that the two tiles' chains of wait -> issue -> commit run
                // side by side: an MMA leaves the issuing thread only as the pipe takes it, and what a single issuing warp
                // did between two groups (commit, poll, fence) was time the pipe ran dry.  This warp waits for the K/V tiles
                // itself and hands them (and Q's place) back with a commit of its own: a stage is free when both warps'
                // commits have arrived, so neither query tile can run ahead of the other by more than the ring holds.
                // Place n of the run of K/V tiles lives in ring stage (n mod STAGES).
                const int mq = warp - MMA_WARP;
                uint32_t abs0 = 0, t_phase = 0;   // tiles loaded before this item; parity of s_req / p_full (one phase per tile)
                auto wait_kv = [&](uint32_t place, uint32_t &st) -> bool {
                    const uint32_t a = abs0 + place;
                    st = a % C::STAGES;
                    return wait_all(bars.kv_full + 8 * st, (a / C::STAGES) & 1u, abort_ptr, WAIT_LIMIT_CYCLES);
                };
                // One place for S: its uses alternate strictly -- tile 0, tile 1, tile 0, ... -- because every
                // Q K^T waits until the softmax has read the S before it, and a phase of the one s_free barrier is one
                // such read.  Tile 0's warp therefore always waits for an odd phase and tile 1's for an even one (for the
                // very first use that is the phase before the first, which counts as complete).
                const uint32_t s_turn = mq ? 0u : 1u;
                for (long long w = blockIdx.x; w < total_work && ok; w += gridDim.x) {
                    WorkItem it;
                    if (!decode_work<FUSED>(p, npairs, w, it)) continue;
                    uint32_t st = 0;
                    ok = wait_all(bars.q_full, q_phase, abort_ptr, WAIT_LIMIT_CYCLES) && wait_kv(0, st);
                    if (!ok) break;
                    q_phase ^= 1u;
                    ok = wait_all(bars.s_free, s_turn, abort_ptr, WAIT_LIMIT_CYCLES);
                    if (!ok) break;
                    tc_fence_after();
                    issue_qk(mq, st);
                    if (leader) {
                        tc_commit(bars.s_full + 8 * mq);
                        tc_commit(bars.kv_empty + 8 * st);            // K_0 is free once both query tiles' MMAs have read it
                        if (it.tiles == 1) tc_commit(bars.q_empty);
                    }
                    for (int k = 0; k < it.tiles && ok; ++k) {
                        const bool more = (k + 1 < it.tiles);
                        uint32_t stv = 0;
                        bool v_waited = false;   // V_k was waited for together with K_{k+1}
                        // Q K_{k+1}^T first -- the softmax waits for it, and asks for it a little before it has
                        // stored P_k, so that S_{k+1} lands about when it is ready to read it -- then P_k V_k, which
                        // nothing waits for until the next P is to be stored
                        ok = wait_all(bars.s_req + 8 * mq, t_phase, abort_ptr, WAIT_LIMIT_CYCLES);
                        if (!ok) break;
                        if (more) {
                            {   // K_{k+1}, V_k (loaded right behind it) and the place for S behind one vote: every
                                // separate wait costs this warp a poll and a vote, and its loop is what paces the pipe
                                const uint32_t ak = abs0 + k_place(k + 1), av = abs0 + v_place(k, it.tiles);
                                st = ak % C::STAGES; stv = av % C::STAGES;
                                const bool r = mbar_wait_bounded(bars.kv_full + 8 * st, (ak / C::STAGES) & 1u, abort_ptr, WAIT_LIMIT_CYCLES) &&
                                               mbar_wait_bounded(bars.kv_full + 8 * stv, (av / C::STAGES) & 1u, abort_ptr, WAIT_LIMIT_CYCLES) &&
                                               mbar_wait_bounded(bars.s_free, s_turn, abort_ptr, WAIT_LIMIT_CYCLES);
                                ok = __all_sync(0xFFFFFFFFu, r) != 0; v_waited = true;
                            }
                            if (!ok) break;
                            tc_fence_after();
                            issue_qk(mq, st);
                            if (leader) {
                                tc_commit(bars.s_full + 8 * mq);
                                tc_commit(bars.kv_empty + 8 * st);
                                if (k + 2 == it.tiles) tc_commit(bars.q_empty);   // that was the item's last Q K^T
                            }
                        }
                        ok = wait_all(bars.p_full + 8 * mq, t_phase, abort_ptr, WAIT_LIMIT_CYCLES);   // P_k is stored
                        if (!ok) break;
                        if (v_waited) st = stv; else ok = wait_kv(v_place(k, it.tiles), st);
                        if (!ok) break;
                        if (k == 0) {  // first PV of the item: the previous item's epilogue must have drained O[mq]
                            ok = wait_all(bars.o_free + 8 * mq, of_phase ^ 1u, abort_ptr, WAIT_LIMIT_CYCLES);
                            if (!ok) break;
                        }
                        tc_fence_after();
                        issue_pv(mq, st, k > 0);
                        if (leader) {
                            tc_commit(more ? bars.pv_done + 8 * mq : bars.o_full + 8 * mq);
                            tc_commit(bars.kv_empty + 8 * st);
                        }
                        t_phase ^= 1u;
                    }
                    of_phase ^= 1u;
                    abs0 += 2u * (uint32_t)it.tiles;
                }
            }
            if (!ok) {
                if (leader && !*abort_ptr) atomicOr(p.status, STATUS_WAIT_TIMEOUT);
                *abort_ptr = 1;
            }
        }
      }
    } else {
        reg_alloc<REGS_SOFTMAX>();
        // ------------------------------------------------------------ softmax warpgroups
        const int q = warp / 4;                       // query tile handled by this warpgroup
        const int row_in_tile = (warp % 4) * 32 + lane;
        const uint32_t lane_addr = ((uint32_t)((warp % 4) * 32)) << 16;
        const uint32_t s_tmem = tmem_base + lane_addr + C::S_COL;
        const uint32_t s_free_bar = bars.s_free;   // one place for S: one barrier
        const uint32_t p_tmem = tmem_base + lane_addr + C::P_COL + q * C::P_STRIDE;
        const uint32_t o_tmem = tmem_base + lane_addr + C::O_COL + q * D;
        uint32_t s_phase = 0, o_phase = 0, pv_phase = 0;
        bool ok = true;
        StateT *o_state = static_cast<StateT *>(p.o_state);
        for (long long w = blockIdx.x; w < total_work && ok; w += gridDim.x) {
            WorkItem it;
            if (!decode_work<FUSED>(p, npairs, w, it)) continue;
            float m_used = -INFINITY, l_sum = 0.f;
            for (int t = 0; t < it.tiles; ++t) {
                const int valid = it.template tile<FUSED>(t).y;   // keys of this tile that count (issued before the wait)
                // One vote tells that S_t has arrived for every lane and (bf16 inputs) that no row's running sum l has reached
                // LSUM_TRIGGER.
                const bool s_here = mbar_wait_bounded(bars.s_full + 8 * q, s_phase, abort_ptr, WAIT_LIMIT_CYCLES);
                const bool fine = __all_sync(0xFFFFFFFFu, s_here && (FP16 || l_sum < LSUM_TRIGGER));
                s_phase ^= 1u;
                tc_fence_after();
                [[maybe_unused]] bool pv_waited = false;
                if (!fine) {
                    ok = __all_sync(0xFFFFFFFFu, s_here);
                    if (!ok) break;
                    if constexpr (!FP16) {
                        // bf16 probabilities have fp32's exponent range, so a tile's P is exact whatever the reference, and
                        // the reference can move after the fact: when the running sum l of a row has reached LSUM_TRIGGER, m
                        // moves up by e = floor(log2(l)) binades and O and l are multiplied by 2^-e, which is exact.  The test
                        // costs one compare on a value that is live anyway; made here, at the top of the next tile, the move
                        // is off the S -> P chain and the logits of a tile never have to be kept for a second pass.
                        // (O may only be touched once P_{t-1} V_{t-1} is complete: pv_done.)
                        ok = __all_sync(0xFFFFFFFFu, mbar_wait_bounded(bars.pv_done + 8 * q, pv_phase, abort_ptr, WAIT_LIMIT_CYCLES));
                        pv_phase ^= 1u;
                        pv_waited = true;
                        tc_fence_after();
                        const int e = move_reference<D>(o_tmem, l_sum);
                        m_used += (float)e;
                        l_sum *= __int_as_float((127 - e) << 23);
                    }
                }
                uint32_t s[4][32];   // this thread's row of S: 128 fp32 logits (before scaling)
                tmem_ld_x32(s_tmem + 0, s[0]);
                tmem_ld_x32(s_tmem + 32, s[1]);
                tmem_ld_x32(s_tmem + 64, s[2]);
                tmem_ld_x32(s_tmem + 96, s[3]);
                tmem_wait_ld();
                [[maybe_unused]] bool s_asked = false;   // (one request per tile, also when P is computed twice)
                bool p_place_free = t == 0 || pv_waited;   // P's columns may still be read by the previous tile's PV
                tc_fence_before();
                mbar_arrive(s_free_bar);   // S_t has been read: the next Q K^T may overwrite it
                if (valid < ATTN_TILE) {
#pragma unroll
                    for (int c = 0; c < 128; ++c)
                        if (c >= valid) s[c >> 5][c & 31] = 0xFF800000u;  // -inf
                }
                // P = exp2(s * scale_log2 - m_used) with the reference maximum of the earlier tiles; the result does not
                // depend on the reference: it cancels in OUT = O / l and LSE = m + log l.  fp16 inputs: while the row
                // sum of P stays below ROWSUM_TRIGGER no element can have exceeded it, so the tile's own maximum is not
                // needed; only when a sum reaches it (rare after the first tiles) is the maximum taken and, if it lies
                // more than 2^RESCALE_THRESHOLD above the reference, the reference moved, O and l rescaled and P
                // computed again.  bf16 inputs: see the top of the tile.
                const float2 sc2 = make_float2(p.scale_log2, p.scale_log2);
                auto row_max = [&]() -> float {   // raw maximum of the row: four chains of three-input max
                    float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                    for (int c = 0; c < 128; c += 8) {
#pragma unroll
                        for (int u = 0; u < 4; ++u)
                            mx4[u] = fmax3(mx4[u], __uint_as_float(s[(c + 2 * u) >> 5][(c + 2 * u) & 31]),
                                           __uint_as_float(s[(c + 2 * u + 1) >> 5][(c + 2 * u + 1) & 31]));
                    }
                    return fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
                };
                // one pass over the row: P to TMEM, returns the row sum
                auto exp_pass = [&](float m_ref) -> float {
                    const float2 nm2 = make_float2(-m_ref, -m_ref);
                    float2 rs4[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
                    // 64 keys as packed 16-bit pairs in the inputs' type (even key in the low half), twice.  The store has
                    // to wait until P_{t-1} V_{t-1} has read P's columns; that MMA is issued behind the next Q K^T, so both
                    // halves go out after the last exponential, when the wait has long ended (storing the first half as
                    // soon as it is complete measured 1.3 % slower at D = 128 and 5 % at D = 64).
                    uint32_t pk2[2][32];
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        uint32_t (&pk)[32] = pk2[half];
#pragma unroll
                        for (int c = half * 64; c < half * 64 + 64; c += 2) {
                            const float s0 = __uint_as_float(s[c >> 5][c & 31]), s1 = __uint_as_float(s[(c + 1) >> 5][(c + 1) & 31]);
                            const float2 x = __ffma2_rn(make_float2(s0, s1), sc2, nm2);
                            // POLY_PER_8 key pairs in eight take the polynomial, spread evenly (two in eight: every fourth)
                            const bool poly = (((c >> 1) * C::POLY_PER_8) & 7) < C::POLY_PER_8;
                            const float2 pp = poly ? exp2_poly2(x) : make_float2(ex2_approx(x.x), ex2_approx(x.y));
                            rs4[(c >> 1) & 3] = __fadd2_rn(rs4[(c >> 1) & 3], pp);
                            pk[(c >> 1) & 31] = pack_half2<FP16>(pp.x, pp.y);
                            if (c + 2 == C::S_REQ * 32 && !s_asked) {   // this many keys are done: ask for the next tile's S
                                mbar_arrive(bars.s_req + 8 * q);
                                s_asked = true;
                            }
                        }
                        if (half == 0) continue;
                        if (!p_place_free) {   // PV of tile t-1 is done with P's columns
                            ok = __all_sync(0xFFFFFFFFu, mbar_wait_bounded(bars.pv_done + 8 * q, pv_phase, abort_ptr, WAIT_LIMIT_CYCLES));
                            pv_phase ^= 1u;
                            p_place_free = true;
                            tc_fence_after();
                        }
                        tmem_st_x32(p_tmem, pk2[0]);
                        tmem_st_x32(p_tmem + 32, pk2[1]);
                    }
                    const float2 r = __fadd2_rn(__fadd2_rn(rs4[0], rs4[1]), __fadd2_rn(rs4[2], rs4[3]));
                    return r.x + r.y;
                };
                if (t == 0) m_used = row_max() * p.scale_log2;   // first tile: no earlier maximum to lean on
                float rs = exp_pass(m_used);
                if constexpr (FP16) {
                    // (the negated comparison also catches inf / NaN after an overflow)
                    if (t > 0 && __any_sync(0xFFFFFFFFu, !(rs < ROWSUM_TRIGGER))) {
                        // fp16 probabilities overflow at 2^16: take the tile's own maximum and compute P again
                        const float m_tile = row_max() * p.scale_log2;
                        const bool need = (m_tile - m_used > RESCALE_THRESHOLD);
                        if (__any_sync(0xFFFFFFFFu, need)) {
                            const float alpha = need ? ex2_approx(m_used - m_tile) : 1.0f;
                            if (need) m_used = m_tile;
                            l_sum *= alpha;
                            tmem_wait_st();
#pragma unroll
                            for (int c0 = 0; c0 < D; c0 += 32) {
                                uint32_t o[32];
                                tmem_ld_x32(o_tmem + c0, o);
                                tmem_wait_ld();
#pragma unroll
                                for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
                                tmem_st_x32(o_tmem + c0, o);
                            }
                            rs = exp_pass(m_used);
                        }
                    }
                }
                l_sum += rs;
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(bars.p_full + 8 * q);
                if (!ok) break;
            }
            if (!ok) break;
            // epilogue: OUT_ij = O / l, LSE_ij = ln2 * (m + log2 l); rows beyond the partition are dropped
            ok = __all_sync(0xFFFFFFFFu, mbar_wait_bounded(bars.o_full + 8 * q, o_phase, abort_ptr, WAIT_LIMIT_CYCLES));
            if (!ok) break;
            o_phase ^= 1u;
            tc_fence_after();
            // this warpgroup's query tile (selected, not indexed: the arrays stay in registers)
            const int my_qn = q ? it.qn[1] : it.qn[0], my_qrow = q ? it.qrow[1] : it.qrow[0];
            const int my_qi = q ? it.qi[1] : it.qi[0], my_qt = q ? it.qt[1] : it.qt[0];
            const bool row_valid = row_in_tile < my_qn;
            const int q_row = my_qrow + row_in_tile;   // this thread's query row (global token index)
            const float inv_l = 1.0f / l_sum;
            if constexpr (!FP16) {
                // a sum that is not finite: within one K/V tile a logit rose more than about 100 binades above the
                // reference (exp2 overflowed); the launch's states are not valid (dt_poll: DT_ERR_RANGE)
                if (row_valid && !(l_sum <= 3.0e38f)) atomicOr(p.status, STATUS_LOGIT_RANGE);
            }
            const float lse_fresh = 0.69314718055994530942f * (m_used + log2f(l_sum));
            if constexpr (FUSED) {
                // fresh state (+) composed reuse state (Eq. 2), straight to the attention output
                const long long crow = (long long)it.bh * p.L + q_row;
                float w_f = inv_l, w_c = 0.f, lse_row = lse_fresh;
                if (p.comp_o != nullptr && row_valid) {
                    const float lc = __ldcs(p.comp_lse + crow);
                    const float M = fmaxf(lse_fresh, lc);
                    const float ef = __expf(lse_fresh - M), ec = __expf(lc - M);   // lc = -inf: weight 0
                    const float z = ef + ec;
                    w_f = inv_l * ef / z;
                    w_c = ec / z;
                    lse_row = M + __logf(z);
                }
                __nv_bfloat16 *dst = static_cast<__nv_bfloat16 *>(p.out) + it.b * p.sb + (long long)q_row * p.sl +
                                     it.h * p.sh;
                const StateT *csrc = static_cast<const StateT *>(p.comp_o) + crow * D;
#pragma unroll
                for (int c0 = 0; c0 < D; c0 += 32) {
                    uint32_t o[32];
                    tmem_ld_x32(o_tmem + c0, o);
                    tmem_wait_ld();
                    if (c0 + 32 >= D) {  // O[q] fully read: the next item's first PV may overwrite it
                        tc_fence_before();
                        mbar_arrive(bars.o_free + 8 * q);
                    }
                    if (row_valid) {
                        float cv[32];
                        if (w_c != 0.f) {
                            load_state_chunk(csrc + c0, cv);
                        } else {
#pragma unroll
                            for (int c = 0; c < 32; ++c) cv[c] = 0.f;
                        }
#pragma unroll
                        for (int c = 0; c < 32; c += 8) {
                            uint4 v;
                            v.x = pack_half2<FP16>(fmaf(w_f, __uint_as_float(o[c]), w_c * cv[c]), fmaf(w_f, __uint_as_float(o[c + 1]), w_c * cv[c + 1]));
                            v.y = pack_half2<FP16>(fmaf(w_f, __uint_as_float(o[c + 2]), w_c * cv[c + 2]), fmaf(w_f, __uint_as_float(o[c + 3]), w_c * cv[c + 3]));
                            v.z = pack_half2<FP16>(fmaf(w_f, __uint_as_float(o[c + 4]), w_c * cv[c + 4]), fmaf(w_f, __uint_as_float(o[c + 5]), w_c * cv[c + 5]));
                            v.w = pack_half2<FP16>(fmaf(w_f, __uint_as_float(o[c + 6]), w_c * cv[c + 6]), fmaf(w_f, __uint_as_float(o[c + 7]), w_c * cv[c + 7]));
                            __stcs(reinterpret_cast<uint4 *>(dst + c0 + c), v);
                        }
                    }
                }
                if (row_valid && p.lse_out != nullptr) p.lse_out[crow] = lse_row;
            } else {
                const long long srow = ((long long)it.slot * p.B * p.H + it.bh) * p.L + q_row;
                // Rows leave through shared memory, warp by warp: each thread writes 128 bytes of its row (swizzled,
                // so the 32 lanes hit different banks), then the warp reads the 4 KB back so that 8 lanes hold the
                // 128 contiguous bytes of one row and stores them -- whole lines to the cache instead of 16 bytes per
                // lane at a 512-byte stride.  The staging area is private to the warp: only __syncwarp() is needed,
                // and no store has to be waited for.  Rows beyond the partition are skipped row by row.
                constexpr int CH = 128 / (int)sizeof(StateT);          // state elements per 128-byte chunk
                const uint32_t stage = out_smem + warp * 4096;          // [32 rows][128 bytes]
                const uint32_t my_row = stage + lane * 128;
                const int rows_left = my_qn - (row_in_tile - lane);   // valid rows of this warp's 32
                uint8_t *gbase = reinterpret_cast<uint8_t *>(o_state + (srow - lane) * D);   // row 0 of this warp
                float row_sq = lse_fresh * lse_fresh;   // ||AS||^2 of this row: OUT and LSE stacked (Eq. 9)
#pragma unroll
                for (int c0 = 0; c0 < D; c0 += CH) {
                    uint32_t o[CH / 32][32];
#pragma unroll
                    for (int u = 0; u < CH / 32; ++u) tmem_ld_x32(o_tmem + c0 + 32 * u, o[u]);
                    tmem_wait_ld();
                    if (c0 + CH >= D) {  // O[q] fully read: the next item's first PV may overwrite it
                        tc_fence_before();
                        mbar_arrive(bars.o_free + 8 * q);
                    }
#pragma unroll
                    for (int c = 0; c < 8; ++c) {   // 16-byte piece c of this row's 128 bytes
                        uint4 v;
                        if constexpr (sizeof(StateT) == 4) {
                            const float f0 = __uint_as_float(o[0][4 * c]) * inv_l, f1 = __uint_as_float(o[0][4 * c + 1]) * inv_l;
                            const float f2 = __uint_as_float(o[0][4 * c + 2]) * inv_l, f3 = __uint_as_float(o[0][4 * c + 3]) * inv_l;
                            row_sq = fmaf(f0, f0, fmaf(f1, f1, fmaf(f2, f2, fmaf(f3, f3, row_sq))));
                            v.x = __float_as_uint(f0); v.y = __float_as_uint(f1); v.z = __float_as_uint(f2); v.w = __float_as_uint(f3);
                        } else {
                            const uint32_t(&oo)[32] = o[(8 * c) / 32];
                            const int b0 = (8 * c) % 32;
                            float f[8];
#pragma unroll
                            for (int u = 0; u < 8; ++u) {
                                f[u] = __uint_as_float(oo[b0 + u]) * inv_l;
                                row_sq = fmaf(f[u], f[u], row_sq);
                            }
                            v.x = pack_bf16x2(f[0], f[1]);
                            v.y = pack_bf16x2(f[2], f[3]);
                            v.z = pack_bf16x2(f[4], f[5]);
                            v.w = pack_bf16x2(f[6], f[7]);
                        }
                        const uint32_t dst = my_row + (uint32_t)((c ^ (lane & 7)) << 4);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
                    }
                    __syncwarp();
                    const int piece = lane & 7;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {   // 4 rows per pass: lane -> (row, 16-byte piece)
                        const int r = i * 4 + (lane >> 3);
                        uint4 v;
                        const uint32_t src = stage + r * 128 + (uint32_t)((piece ^ (r & 7)) << 4);
                        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(src) : "memory");
                        if (r < rows_left)
                            __stcs(reinterpret_cast<uint4 *>(gbase + (size_t)r * D * sizeof(StateT) + (size_t)c0 * sizeof(StateT) + piece * 16), v);
                    }
                    __syncwarp();
                }
                if (row_valid) p.lse_state[srow] = lse_fresh;
                if (p.norm_partials != nullptr) {
                    // the state norms Algorithm 1 wants at an anchor come out of this epilogue instead of a pass over the
                    // cache: one partial per warp, summed by an xor butterfly (a fixed order: same bits every run)
                    if (!row_valid) row_sq = 0.f;
#pragma unroll
                    for (int sft = 16; sft > 0; sft >>= 1) row_sq += __shfl_xor_sync(0xFFFFFFFFu, row_sq, sft);
                    if (lane == 0) {
                        p.norm_partials[((((long long)it.bh * p.P + my_qi) * p.S + it.slot) * (p.qblocks_max * ATTN_NQ) + my_qt) * 4 +
                                        (warp & 3)] = row_sq;
                    }
                }
            }
        }
        if (!ok && lane == 0) {
            if (!*abort_ptr) atomicOr(p.status, STATUS_WAIT_TIMEOUT);
            *abort_ptr = 1;
        }
    }

    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 0) tmem_dealloc(tmem_base, 512);
}

template <int D, typename StateT, bool FUSED, bool FP16>
cudaError_t launch_one(const CUtensorMap &tq, const CUtensorMap &tk, const CUtensorMap &tv, const AttnParams &p,
                       int num_ctas, cudaStream_t stream) {
    attn_states_kernel<D, StateT, FUSED, FP16><<<num_ctas, ATTN_THREADS, Cfg<D>::SMEM_BYTES, stream>>>(tq, tk, tv, p);
    return cudaGetLastError();
}

template <int D, typename StateT, bool FUSED>
cudaError_t launch(const CUtensorMap &tq, const CUtensorMap &tk, const CUtensorMap &tv, const AttnParams &p,
                   int num_ctas, cudaStream_t stream) {
    return p.in_fp16 ? launch_one<D, StateT, FUSED, true>(tq, tk, tv, p, num_ctas, stream)
                     : launch_one<D, StateT, FUSED, false>(tq, tk, tv, p, num_ctas, stream);
}

template <int D, typename StateT, bool FUSED, bool FP16>
cudaError_t configure_one() {
    cudaFuncAttributes attr;
    cudaError_t e = cudaFuncGetAttributes(&attr, attn_states_kernel<D, StateT, FUSED, FP16>);
    if (e != cudaSuccess) return e;
    if (attr.numRegs != LAUNCH_REGS) return cudaErrorInvalidConfiguration;   // the register hand-over would not balance
    return cudaFuncSetAttribute(attn_states_kernel<D, StateT, FUSED, FP16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                Cfg<D>::SMEM_BYTES);
}

template <int D, typename StateT>
cudaError_t configure() {
    cudaError_t e = configure_one<D, StateT, false, false>();
    if (e == cudaSuccess) e = configure_one<D, StateT, true, false>();
    if (e == cudaSuccess) e = configure_one<D, StateT, false, true>();
    if (e == cudaSuccess) e = configure_one<D, StateT, true, true>();
    return e;
}

// Fused mode: per query partition the K/V tiles of one pass over the keys of all its COMPUTE slots.  The slots'
// key ranges are sorted and ranges that touch are joined, so only the last tile of a maximal run is ragged.
__global__ void fused_tiles_kernel(const uint8_t *mask, const SlotRange *slot_tab, int P, int S, int max_tiles, int2 *tile_tab,
                                   int32_t *tile_cnt) {
    const int i = threadIdx.x;
    if (i >= P) return;
    int start[2 * DT_MAX_P + 2], len[2 * DT_MAX_P + 2];
    int n = 0;
    for (int s = 0; s < S; ++s) {
        if (mask[i * S + s] == 0) continue;
        const SlotRange r = slot_tab[i * S + s];
        if (r.n1 > 0) { start[n] = r.r1; len[n] = r.n1; ++n; }
        if (r.n2 > 0) { start[n] = r.r2; len[n] = r.n2; ++n; }
    }
    for (int a = 1; a < n; ++a) {   // insertion sort by first key
        const int s0 = start[a], l0 = len[a];
        int b = a - 1;
        while (b >= 0 && start[b] > s0) { start[b + 1] = start[b]; len[b + 1] = len[b]; --b; }
        start[b + 1] = s0; len[b + 1] = l0;
    }
    int2 *tab = tile_tab + (long long)i * max_tiles;
    int cnt = 0;
    for (int a = 0; a < n;) {
        int s0 = start[a], l0 = len[a];
        ++a;
        while (a < n && start[a] == s0 + l0) { l0 += len[a]; ++a; }
        for (int k = 0; k < l0 && cnt < max_tiles; k += ATTN_TILE) tab[cnt++] = make_int2(s0 + k, l0 - k);
    }
    tile_cnt[i] = cnt;
}

}  // namespace

cudaError_t attn_states_configure() {
    cudaError_t e;
    if ((e = configure<64, float>()) != cudaSuccess) return e;
    if ((e = configure<128, float>()) != cudaSuccess) return e;
    if ((e = configure<64, __nv_bfloat16>()) != cudaSuccess) return e;
    return configure<128, __nv_bfloat16>();
}

cudaError_t launch_attn_states(const CUtensorMap &tq, const CUtensorMap &tk, const CUtensorMap &tv,
                               const AttnParams &p, int D, int state_dtype, int num_ctas, cudaStream_t stream) {
    if (state_dtype == DT_STATE_FP32) {
        return D == 64 ? launch<64, float, false>(tq, tk, tv, p, num_ctas, stream)
                       : launch<128, float, false>(tq, tk, tv, p, num_ctas, stream);
    }
    return D == 64 ? launch<64, __nv_bfloat16, false>(tq, tk, tv, p, num_ctas, stream)
                   : launch<128, __nv_bfloat16, false>(tq, tk, tv, p, num_ctas, stream);
}

cudaError_t launch_attn_fused(const CUtensorMap &tq, const CUtensorMap &tk, const CUtensorMap &tv,
                              const AttnParams &p, int D, int state_dtype, int num_ctas, cudaStream_t stream) {
    if (state_dtype == DT_STATE_FP32) {
        return D == 64 ? launch<64, float, true>(tq, tk, tv, p, num_ctas, stream)
                       : launch<128, float, true>(tq, tk, tv, p, num_ctas, stream);
    }
    return D == 64 ? launch<64, __nv_bfloat16, true>(tq, tk, tv, p, num_ctas, stream)
                   : launch<128, __nv_bfloat16, true>(tq, tk, tv, p, num_ctas, stream);
}

cudaError_t launch_fused_tiles(const uint8_t *mask, const SlotRange *slot_tab, int P, int S, int max_tiles, int2 *tile_tab,
                               int32_t *tile_cnt, cudaStream_t stream) {
    fused_tiles_kernel<<<1, 32, 0, stream>>>(mask, slot_tab, P, S, max_tiles, tile_tab, tile_cnt);
    return cudaGetLastError();
}

}  // namespace dt
