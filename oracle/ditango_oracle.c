/*
 * DiTango selective attention-state path -- fp64 CPU oracle.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing in the product path may call, link or
 * import this file; it exists so that the CUDA kernels can be compared with a
 * plain, slow, obviously correct restatement of what the paper defines.  It
 * shares no code, header, table or helper with the CUDA path.
 *
 * Everything is fp64, plain loops, no tiling, no online softmax, no fusion.
 * Inputs Q, K, V are bf16 (or, with in_fp16, IEEE fp16) bit patterns (uint16) in layout [B, L, H, D]; they
 * are widened exactly to double before any arithmetic.
 *
 * Notation (paper, Section 2.2.4 and Section 4):
 *   state  AS(j) = [OUT(j); LSE(j)]  of a query row against key partition j   (Eq. 1)
 *   a (+) b                          LSE-rescaled composition of two states   (Eq. 2)
 *   w(j)   = e^{LSE(j)} / sum_k e^{LSE(k)}   partition importance weight      (Eq. 8)
 *   COMPUTE iff measure > eps, else REUSE                                     (Eq. 13)
 *
 * Parity pins (tests, CPU only): full attention against a library softmax,
 * all-partition merge against full attention, K == 0 closed forms,
 * key-permutation invariance, associativity / commutativity of (+), the
 * first-order error propagation identity (Eq. 4) by finite differences,
 * row sums of w, closed-form softmax for synthetic LSE, equality case of
 * the threshold.  The target-fraction rule (orc_target_fraction) follows a
 * reading of the paper's "eps as a percentile matching a target ratio"; what
 * it computes is pinned by its invariants (count, diagonal, monotonicity) and
 * by a hand-checked two-valued measure that fixes the tie order and the
 * midpoint threshold.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

static inline double bf16_to_f64(uint16_t bits) {
    uint32_t u = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* IEEE binary16: 1 sign, 5 exponent (bias 15), 10 fraction bits; subnormals, infinities and NaN included */
static inline double f16_to_f64(uint16_t bits) {
    int sign = bits >> 15, e = (bits >> 10) & 0x1F, frac = bits & 0x3FF;
    double v;
    if (e == 0) v = ldexp((double)frac, -24);
    else if (e == 31) v = frac ? NAN : INFINITY;
    else v = ldexp((double)(1024 + frac), e - 25);
    return sign ? -v : v;
}

/* element of q, k or v as a double: the bit pattern is bf16 (in_fp16 == 0) or fp16 */
static inline double in_to_f64(uint16_t bits, int in_fp16) {
    return in_fp16 ? f16_to_f64(bits) : bf16_to_f64(bits);
}

/* exposed for the pins: widening of one bit pattern */
double orc_widen(uint16_t bits, int in_fp16) { return in_to_f64(bits, in_fp16); }

int orc_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* element (b, l, h, d) of a [B, L, H, D] tensor */
static inline size_t idx4(int b, int l, int h, int d, int L, int H, int D) {
    return (((size_t)b * L + l) * H + h) * D + d;
}

/*
 * Eq. 1: attention state of each listed query row against the keys
 * [key_begin, key_end) (one KV partition), for one (b, h).
 *   x_c   = scale * <q_r, k_c>
 *   LSE   = log sum_c exp(x_c)                (evaluated as m + log sum exp(x_c - m))
 *   OUT   = sum_c exp(x_c - LSE) v_c
 * out: [nrows, D], lse: [nrows].  Returns 0, or -1 on bad arguments.
 */
int orc_pair_state(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                   int B, int L, int H, int D, double scale, int b, int h,
                   const int32_t *rows, int nrows, int key_begin, int key_end,
                   double *out, double *lse, int in_fp16) {
    if (b < 0 || b >= B || h < 0 || h >= H || key_begin < 0 || key_end > L || key_begin >= key_end)
        return -1;
    int nk = key_end - key_begin;
    int bad = 0;
#pragma omp parallel
    {
        double *x = (double *)malloc((size_t)nk * sizeof(double));
#pragma omp for schedule(dynamic, 4)
        for (int ri = 0; ri < nrows; ++ri) {
            int r = rows[ri];
            if (r < 0 || r >= L) { bad = 1; continue; }
            const uint16_t *qr = q + idx4(b, r, h, 0, L, H, D);
            double m = -INFINITY;
            for (int c = 0; c < nk; ++c) {
                const uint16_t *kc = k + idx4(b, key_begin + c, h, 0, L, H, D);
                double dot = 0.0;
                for (int d = 0; d < D; ++d) dot += in_to_f64(qr[d], in_fp16) * in_to_f64(kc[d], in_fp16);
                x[c] = scale * dot;
                if (x[c] > m) m = x[c];
            }
            double ell = 0.0;
            for (int c = 0; c < nk; ++c) ell += exp(x[c] - m);
            double *o = out + (size_t)ri * D;
            for (int d = 0; d < D; ++d) o[d] = 0.0;
            for (int c = 0; c < nk; ++c) {
                double p = exp(x[c] - m);
                const uint16_t *vc = v + idx4(b, key_begin + c, h, 0, L, H, D);
                for (int d = 0; d < D; ++d) o[d] += p * in_to_f64(vc[d], in_fp16);
            }
            for (int d = 0; d < D; ++d) o[d] /= ell;
            lse[ri] = m + log(ell);
        }
        free(x);
    }
    return bad ? -1 : 0;
}

/*
 * Plain full attention of the listed rows over all L keys:
 *   p_c = softmax_c(scale * <q_r, k_c>),  out = sum_c p_c v_c,  lse = log sum_c exp(x_c).
 * Written separately from orc_pair_state (probabilities are normalised first,
 * then applied) so that "compose all partitions == full attention" compares
 * two different evaluations.
 */
int orc_full_attention(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                       int B, int L, int H, int D, double scale, int b, int h,
                       const int32_t *rows, int nrows, double *out, double *lse, int in_fp16) {
    if (b < 0 || b >= B || h < 0 || h >= H) return -1;
    int bad = 0;
#pragma omp parallel
    {
        double *p = (double *)malloc((size_t)L * sizeof(double));
#pragma omp for schedule(dynamic, 4)
        for (int ri = 0; ri < nrows; ++ri) {
            int r = rows[ri];
            if (r < 0 || r >= L) { bad = 1; continue; }
            const uint16_t *qr = q + idx4(b, r, h, 0, L, H, D);
            double m = -INFINITY;
            for (int c = 0; c < L; ++c) {
                const uint16_t *kc = k + idx4(b, c, h, 0, L, H, D);
                double dot = 0.0;
                for (int d = 0; d < D; ++d) dot += in_to_f64(qr[d], in_fp16) * in_to_f64(kc[d], in_fp16);
                p[c] = scale * dot;
                if (p[c] > m) m = p[c];
            }
            double z = 0.0;
            for (int c = 0; c < L; ++c) { p[c] = exp(p[c] - m); z += p[c]; }
            for (int c = 0; c < L; ++c) p[c] /= z;
            double *o = out + (size_t)ri * D;
            for (int d = 0; d < D; ++d) o[d] = 0.0;
            for (int c = 0; c < L; ++c) {
                const uint16_t *vc = v + idx4(b, c, h, 0, L, H, D);
                for (int d = 0; d < D; ++d) o[d] += p[c] * in_to_f64(vc[d], in_fp16);
            }
            lse[ri] = m + log(z);
        }
        free(p);
    }
    return bad ? -1 : 0;
}

/*
 * Eq. 2, literally, for two states of one query row:
 *   OUT = (e^{LSEa} OUTa + e^{LSEb} OUTb) / (e^{LSEa} + e^{LSEb})
 *   LSE = log(e^{LSEa} + e^{LSEb})
 * The common factor e^{max} is taken out of numerator and denominator so the
 * exponentials stay finite; a state with LSE = -inf has weight 0.
 */
void orc_compose2(const double *oa, double lsea, const double *ob, double lseb, int D,
                  double *o, double *lse) {
    double m = lsea > lseb ? lsea : lseb;
    if (m == -INFINITY) {
        for (int d = 0; d < D; ++d) o[d] = 0.0;
        *lse = -INFINITY;
        return;
    }
    double ea = exp(lsea - m), eb = exp(lseb - m);
    double z = ea + eb;
    for (int d = 0; d < D; ++d) o[d] = (ea * oa[d] + eb * ob[d]) / z;
    *lse = m + log(z);
}

/*
 * Eq. 2 folded over P states per row (one pass, global max):
 *   LSE = log sum_j e^{LSE_j},   OUT = sum_j e^{LSE_j - LSE} OUT_j.
 * o_states: [n, P, D], lse_states: [n, P]  ->  out [n, D], lse [n].
 */
void orc_merge(const double *o_states, const double *lse_states, int n, int P, int D,
               double *out, double *lse) {
#pragma omp parallel for schedule(static)
    for (int r = 0; r < n; ++r) {
        const double *ls = lse_states + (size_t)r * P;
        double M = -INFINITY;
        for (int j = 0; j < P; ++j) if (ls[j] > M) M = ls[j];
        double *o = out + (size_t)r * D;
        for (int d = 0; d < D; ++d) o[d] = 0.0;
        if (M == -INFINITY) { lse[r] = -INFINITY; continue; }
        double Z = 0.0;
        for (int j = 0; j < P; ++j) Z += exp(ls[j] - M);
        for (int j = 0; j < P; ++j) {
            double wj = exp(ls[j] - M);
            const double *oj = o_states + ((size_t)r * P + j) * D;
            for (int d = 0; d < D; ++d) o[d] += wj * oj[d];
        }
        for (int d = 0; d < D; ++d) o[d] /= Z;
        lse[r] = M + log(Z);
    }
}

/*
 * Eq. 8 per query row, reduced to one number per (query partition i, KV
 * partition j) by the arithmetic mean over batch, heads and the rows of
 * partition i:
 *   u_j(r) = exp(LSE_ij[r] - logsumexp_k LSE_ik[r]),
 *   W[i][j] = (1 / (B H n_i)) sum_{b,h,r in part i} u_j(r).
 * lse_states: [P(j), B, H, L] (fp64);  off: [P+1] partition offsets;  W: [P, P].
 */
int orc_contribution(const double *lse_states, int B, int H, int L, int P,
                     const int32_t *off, double *W) {
    if (off[0] != 0 || off[P] != L) return -1;
    for (int i = 0; i < P; ++i) if (off[i + 1] <= off[i]) return -1;
    size_t slab = (size_t)B * H * L;
    for (int i = 0; i < P; ++i) {
        for (int j = 0; j < P; ++j) W[i * P + j] = 0.0;
        for (int b = 0; b < B; ++b)
            for (int h = 0; h < H; ++h)
                for (int r = off[i]; r < off[i + 1]; ++r) {
                    size_t e = ((size_t)b * H + h) * L + r;
                    double M = -INFINITY;
                    for (int kx = 0; kx < P; ++kx) {
                        double x = lse_states[kx * slab + e];
                        if (x > M) M = x;
                    }
                    double Z = 0.0;
                    for (int kx = 0; kx < P; ++kx) Z += exp(lse_states[kx * slab + e] - M);
                    double lz = M + log(Z);
                    for (int j = 0; j < P; ++j) W[i * P + j] += exp(lse_states[j * slab + e] - lz);
                }
        double cnt = (double)B * H * (off[i + 1] - off[i]);
        for (int j = 0; j < P; ++j) W[i * P + j] /= cnt;
    }
    return 0;
}

/*
 * Eq. 13 with the always-computed local (diagonal) partition:
 *   mask[i][j] = 1 (COMPUTE) iff i == j or W[i][j] > eps; equality -> REUSE.
 */
void orc_threshold(const double *W, int P, double eps, uint8_t *mask) {
    for (int i = 0; i < P; ++i)
        for (int j = 0; j < P; ++j)
            mask[i * P + j] = (i == j || W[i * P + j] > eps) ? 1 : 0;
}

typedef struct { double w; int dist; int flat; } orc_rank_t;

static int orc_rank_cmp(const void *pa, const void *pb) {
    const orc_rank_t *a = (const orc_rank_t *)pa, *b = (const orc_rank_t *)pb;
    if (a->w != b->w) return a->w > b->w ? -1 : 1;      /* larger W first        */
    if (a->dist != b->dist) return a->dist - b->dist;   /* then smaller |i - j|  */
    return a->flat - b->flat;                           /* then smaller i*P + j  */
}

/*
 * eps chosen to hit a target computed-pair fraction f (a percentile of the
 * anchor-step measure):  K = round(f P^2) clipped to [P, P^2]; the diagonal
 * is always computed; the K - P off-diagonal pairs of largest W are selected
 * (ties: smaller |i-j|, then smaller i*P+j);  eps = midpoint between the last
 * selected and first unselected W (0 if every pair is selected; if none is
 * selected, eps = the largest off-diagonal W, so that W > eps selects none).
 * Writes the mask of that selection; returns K.
 */
int orc_target_fraction(const double *W, int P, double f, uint8_t *mask, double *eps_out) {
    int total = P * P;
    int K = (int)floor(f * total + 0.5);
    if (K < P) K = P;
    if (K > total) K = total;
    int noff = total - P;
    orc_rank_t *rk = (orc_rank_t *)malloc((size_t)(noff > 0 ? noff : 1) * sizeof(orc_rank_t));
    int n = 0;
    for (int i = 0; i < P; ++i)
        for (int j = 0; j < P; ++j)
            if (i != j) {
                rk[n].w = W[i * P + j];
                rk[n].dist = i > j ? i - j : j - i;
                rk[n].flat = i * P + j;
                ++n;
            }
    qsort(rk, (size_t)n, sizeof(orc_rank_t), orc_rank_cmp);
    for (int e = 0; e < total; ++e) mask[e] = 0;
    for (int i = 0; i < P; ++i) mask[i * P + i] = 1;
    int sel = K - P;
    for (int s = 0; s < sel; ++s) mask[rk[s].flat] = 1;
    double eps;
    if (noff == 0 || sel == noff) eps = 0.0;
    else if (sel == 0) eps = rk[0].w;
    else eps = 0.5 * (rk[sel - 1].w + rk[sel].w);
    *eps_out = eps;
    free(rk);
    return K;
}

/*
 * Group-wise organisation (Section 4.2.1-4.2.3): the P KV partitions are divided into contiguous groups
 * of g; all states of a group share one decision per query partition i, the local (diagonal) state is
 * handled separately (always computed), so the group that contains it has one member fewer.  The group
 * measure is the sum of its members' measures (Eq. 12), thresholded with a strict '>' (Eq. 13).
 *   unit (i, k): members j in [k g, min(P, (k+1) g)), j != i;   m(i,k) = sum_j W[i][j]
 * target_fraction < 0: COMPUTE iff m > eps.
 * target_fraction >= 0: K = round(f P^2) clipped to [P, P^2]; units are ranked by m (ties: smaller
 *   |k - floor(i/g)|, then smaller i * n_groups + k) and taken in that order while the pairs selected so
 *   far plus the unit's members still fit into K - P; eps = midpoint between the last taken and the first
 *   not taken measure (0 if all are taken, the largest measure if none is).
 * With g = 1 this is exactly orc_threshold / orc_target_fraction.  Returns the number of COMPUTE pairs.
 */
typedef struct { double m; int dist; int flat; int size; int i; int k; } orc_unit_t;

static int orc_unit_cmp(const void *pa, const void *pb) {
    const orc_unit_t *a = (const orc_unit_t *)pa, *b = (const orc_unit_t *)pb;
    if (a->m != b->m) return a->m > b->m ? -1 : 1;
    if (a->dist != b->dist) return a->dist - b->dist;
    return a->flat - b->flat;
}

int orc_group_plan(const double *W, int P, int g, double eps, double target_fraction, uint8_t *mask,
                   double *eps_out) {
    if (g < 1) g = 1;
    int ng = (P + g - 1) / g;
    orc_unit_t *u = (orc_unit_t *)malloc((size_t)P * ng * sizeof(orc_unit_t));
    int n = 0;
    for (int i = 0; i < P; ++i)
        for (int k = 0; k < ng; ++k) {
            int lo = k * g, hi = (k + 1) * g < P ? (k + 1) * g : P;
            double m = 0.0;
            int size = 0;
            for (int j = lo; j < hi; ++j)
                if (j != i) { m += W[i * P + j]; ++size; }
            if (size == 0) continue;
            int gi = i / g;
            u[n].m = m; u[n].dist = k > gi ? k - gi : gi - k; u[n].flat = i * ng + k; u[n].size = size;
            u[n].i = i; u[n].k = k;
            ++n;
        }
    for (int e = 0; e < P * P; ++e) mask[e] = 0;
    for (int i = 0; i < P; ++i) mask[i * P + i] = 1;
    int count = P;
    double eps_used = eps;
    if (target_fraction < 0) {
        for (int s = 0; s < n; ++s)
            if (u[s].m > eps) {
                for (int j = u[s].k * g; j < (u[s].k + 1) * g && j < P; ++j)
                    if (j != u[s].i) { mask[u[s].i * P + j] = 1; ++count; }
            }
    } else {
        int total = P * P;
        int K = (int)floor(target_fraction * total + 0.5);
        if (K < P) K = P;
        if (K > total) K = total;
        qsort(u, (size_t)n, sizeof(orc_unit_t), orc_unit_cmp);
        int budget = K - P, used = 0, taken = 0;
        while (taken < n && used + u[taken].size <= budget) {
            for (int j = u[taken].k * g; j < (u[taken].k + 1) * g && j < P; ++j)
                if (j != u[taken].i) { mask[u[taken].i * P + j] = 1; ++count; }
            used += u[taken].size;
            ++taken;
        }
        if (n == 0 || taken == n) eps_used = 0.0;
        else if (taken == 0) eps_used = u[0].m;
        else eps_used = 0.5 * (u[taken - 1].m + u[taken].m);
    }
    *eps_out = eps_used;
    free(u);
    return count;
}
