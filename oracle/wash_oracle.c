/*
 * wash_oracle.c -- plain CPU oracle for the WASH population operators.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct statement of
 * what the GPU library must compute.  It shares no code, header, table or constant
 * generator with the CUDA path, and nothing in the product may import, link or run
 * it (only the tests, the smoke check and the CPU-baseline leg of the benchmark).
 *
 * What it states, with the passage of the WASH paper each function follows:
 *
 *   wo_philox4x32_10      Philox4x32-10 counter-based generator (Salmon, Moraes,
 *                         Dror, Shaw, "Parallel random numbers: as easy as 1, 2, 3",
 *                         SC'11).  The paper names no generator; this one is fixed by
 *                         the library's determinism contract.
 *   wo_layer_probs        Layer-wise probability p_l = p (1 - l/(L-1))
 *                         (section "Layer-wise adaptation via WASH", the unnumbered
 *                         equation after Eq. 5) plus the constant / increasing
 *                         variants of Table 4.
 *   wo_shuffle            The shuffling step: Eq. 3 and the "Shuffling step" loop of
 *                         Algorithm 1; with a second stack it is the WASH+Opt variant
 *                         (section "Training methods": the optimizer state of a
 *                         shuffled parameter is permuted with it).
 *   wo_papa_ema           PAPA's pull toward the consensus, Eq. 1.
 *   wo_population_average The output of Algorithm 1: (1/N) sum_n theta_n.
 *   wo_papa_all           PAPA-all / DART step (section "Reducing distance to
 *                         consensus"): every model replaced by the average.
 *   wo_consensus_distance Average distance to the consensus (caption of Fig. 2).
 *   wo_exchange_send / wo_exchange_receive / wo_exchange_counts
 *                         The same shuffling step seen from one worker that holds one
 *                         model (the deployment the Introduction describes: parameters
 *                         travel peer to peer along the permutation).
 *
 * Readings taken where the paper is silent (each is a convention of this library,
 * not a fact of the paper; parity for them is pinned by the tests, not by the paper):
 *   - one Bernoulli draw per coordinate i, shared by all n (Algorithm 1 draws once
 *     per parameter, and Eq. 5 only holds then);
 *   - pi_i uniform over all N! permutations, fixed points allowed (Eq. 4 needs it);
 *   - gather direction, new[n] = old[pi(n)], as Eq. 3 is written;
 *   - probability p becomes the integer test  word < floor(p * 2^32);
 *   - uniform integer in [0,k] from a 32-bit word by multiply-high, no rejection;
 *   - Fisher-Yates from the top index down, one 32-bit word per swap;
 *   - Philox keying: key = seed, counter = (coordinate, tensor, step, stream tag).
 *   - Eq. 1 and the average are evaluated in binary32, terms added in the order
 *     n = 0, 1, ..., N-1, true division by N, every operation rounded once.
 *
 * Pins (tests/test_oracle_*.py): the Philox round function against cuRAND's host
 * generator and the closed forms of its Weyl constants; p = 0 identity, p = 1 all
 * selected; per-coordinate multiset preserved (Eq. 5); Eq. 4 by Monte Carlo;
 * chi-square uniformity of pi for N = 3, 4, 5; selected fraction against the
 * binomial law; last layer untouched; brute force on tiny stacks; Eq. 2 and a
 * binary64 mean with an a-priori error bound for Eq. 1 and the average; the worker
 * form against wo_shuffle on the stacked population, its slot counts against the
 * permutations drawn one by one, and the expected volume p d (N-1)/N per worker.
 */
#include <stdint.h>
#include <stddef.h>
#include <string.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { WO_LAYOUT_NP = 0, WO_LAYOUT_PN = 1 };
enum { WO_F32 = 0, WO_BF16 = 1 };
enum { WO_OK = 0, WO_ERR_ARG = -1 };

/* A population: N stacked copies of T segments.  Segment s holds numel[s]
 * coordinates that are coordinates coord_begin[s] .. of tensor tensor_id[s]
 * (a whole tensor when coord_begin is 0), stored from element offset[s] of each
 * model's row of padded_P elements. */
typedef struct {
    int32_t N;
    int32_t T;
    const int64_t *numel;
    const int64_t *offset;
    const uint32_t *tensor_id;   /* NULL: segment s is tensor s           */
    const int64_t *coord_begin;  /* NULL: every segment starts at coord 0 */
    int64_t padded_P;
    int32_t layout;
} wo_population;

static int wo_threads = 1;
void wo_set_threads(int n) { wo_threads = n < 1 ? 1 : n; }
int wo_get_threads(void) { return wo_threads; }
int wo_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_num_procs();
#else
    return 1;
#endif
}

/* ---- Philox4x32-10 (SC'11 paper, section 3.3 and its Table of multipliers) ---- */
void wo_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) {             /* bump the key by the Weyl constants */
            k0 += 0x9E3779B9u;       /* golden ratio          */
            k1 += 0xBB67AE85u;       /* sqrt(3) - 1           */
        }
        uint64_t prod0 = (uint64_t)0xD2511F53u * c0;
        uint64_t prod1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t hi0 = (uint32_t)(prod0 >> 32), lo0 = (uint32_t)prod0;
        uint32_t hi1 = (uint32_t)(prod1 >> 32), lo1 = (uint32_t)prod1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* ---- keying: which counter feeds which decision ---- */

/* 32-bit word that decides whether coordinate i of tensor t is shuffled at `step`.
 * Four neighbouring coordinates share one Philox block. */
uint32_t wo_mask_word(uint64_t seed, uint64_t step, uint32_t t, uint64_t i)
{
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t ctr[4] = { (uint32_t)(i >> 2), t, (uint32_t)step,
                        (uint32_t)((step >> 32) << 8) | 0u };
    uint32_t out[4];
    wo_philox4x32_10(ctr, key, out);
    return out[i & 3];
}

/* m-th 32-bit word (m = 0, 1, ...) of the permutation stream of coordinate (t, i). */
uint32_t wo_perm_word(uint64_t seed, uint64_t step, uint32_t t, uint64_t i, int m)
{
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t block = (uint32_t)(m >> 2);
    uint32_t ctr[4] = { (uint32_t)i, t, (uint32_t)step,
                        (uint32_t)((step >> 32) << 8) | (1u + block) };
    uint32_t out[4];
    wo_philox4x32_10(ctr, key, out);
    return out[m & 3];
}

/* probability -> integer threshold on a 32-bit word; realised probability thr/2^32 */
uint64_t wo_threshold(double p)
{
    return (uint64_t)floor(p * 4294967296.0);
}

/* pi_i for coordinate (t, i): Fisher-Yates from the top, uniform over N! up to the
 * multiply-high bias (< (k+1)/2^32 per draw). */
void wo_draw_permutation(uint64_t seed, uint64_t step, uint32_t t, uint64_t i,
                         int32_t N, int32_t *perm)
{
    for (int n = 0; n < N; ++n) perm[n] = n;
    for (int k = N - 1; k >= 1; --k) {
        int m = N - 1 - k;
        uint32_t r = wo_perm_word(seed, step, t, i, m);
        int j = (int)(((uint64_t)r * (uint64_t)(k + 1)) >> 32);   /* in [0, k] */
        int32_t tmp = perm[k]; perm[k] = perm[j]; perm[j] = tmp;
    }
}

/* ---- layer-wise probabilities ---- */
/* schedule 0: decreasing  p_l = p (1 - l/(L-1))   (the paper's default)
 *          1: constant    p_l = p                 (Table 4, middle row)
 *          2: increasing  p_l = p  l/(L-1)        (Table 4, last row)
 * L = 1 has no slope to speak of: p_0 = p. */
int wo_layer_probs(int32_t L, double p, int32_t schedule, double *out)
{
    if (L < 1 || !(p >= 0.0 && p <= 1.0) || schedule < 0 || schedule > 2) return WO_ERR_ARG;
    for (int l = 0; l < L; ++l) {
        double frac = (L == 1) ? 0.0 : (double)l / (double)(L - 1);
        if (schedule == 0) out[l] = (L == 1) ? p : p * (1.0 - frac);
        else if (schedule == 1) out[l] = p;
        else out[l] = (L == 1) ? p : p * frac;
    }
    return WO_OK;
}

/* ---- element access ---- */
static inline size_t wo_index(const wo_population *pop, int n, int64_t elem)
{
    return pop->layout == WO_LAYOUT_NP ? (size_t)n * (size_t)pop->padded_P + (size_t)elem
                                       : (size_t)elem * (size_t)pop->N + (size_t)n;
}
static inline float wo_bf16_to_f32(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16; float f; memcpy(&f, &u, 4); return f;
}
/* round to nearest, ties to even; NaN stays a (quiet) NaN */
static inline uint16_t wo_f32_to_bf16(float f)
{
    uint32_t u; memcpy(&u, &f, 4);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}
static inline float wo_load(const void *stack, int dtype, size_t idx)
{
    if (dtype == WO_F32) return ((const float *)stack)[idx];
    return wo_bf16_to_f32(((const uint16_t *)stack)[idx]);
}
static inline void wo_store(void *stack, int dtype, size_t idx, float v)
{
    if (dtype == WO_F32) ((float *)stack)[idx] = v;
    else ((uint16_t *)stack)[idx] = wo_f32_to_bf16(v);
}
static int wo_check_pop(const wo_population *pop)
{
    if (!pop || pop->N < 1 || pop->N > 1021 || pop->T < 0) return WO_ERR_ARG;
    if (pop->layout != WO_LAYOUT_NP && pop->layout != WO_LAYOUT_PN) return WO_ERR_ARG;
    return WO_OK;
}

/* ---- the shuffling step (Eq. 3, Algorithm 1 "Shuffling step") ---- */
/* permute the N values of element `elem` of one stack: new[n] = old[pi(n)], raw bits */
static void wo_permute_column(const wo_population *pop, void *stack, int dtype,
                              int64_t elem, const int32_t *perm)
{
    int N = pop->N;
    if (dtype == WO_F32) {
        uint32_t old[1024]; uint32_t *a = (uint32_t *)stack;
        for (int n = 0; n < N; ++n) old[n] = a[wo_index(pop, n, elem)];
        for (int n = 0; n < N; ++n) a[wo_index(pop, n, elem)] = old[perm[n]];
    } else {
        uint16_t old[1024]; uint16_t *a = (uint16_t *)stack;
        for (int n = 0; n < N; ++n) old[n] = a[wo_index(pop, n, elem)];
        for (int n = 0; n < N; ++n) a[wo_index(pop, n, elem)] = old[perm[n]];
    }
}

/* p_seg[s] is the shuffling probability of segment s.  stack2 (may be NULL) is a
 * second stack over the same population (the optimizer state) that follows the same
 * mask and the same permutations.  stats[0] += selected coordinates,
 * stats[1] += values whose model index changed (sum over selected i of
 * #{n : pi_i(n) != n}), counted once per coordinate whatever the number of stacks. */
int wo_shuffle(const wo_population *pop, void *stack, int32_t dtype,
               void *stack2, int32_t dtype2, const double *p_seg,
               uint64_t seed, uint64_t step, uint64_t *stats)
{
    if (wo_check_pop(pop) != WO_OK || !stack || !p_seg || pop->N < 2) return WO_ERR_ARG;
    if (step >> 56) return WO_ERR_ARG;
    for (int s = 0; s < pop->T; ++s)
        if (!(p_seg[s] >= 0.0 && p_seg[s] <= 1.0)) return WO_ERR_ARG;
    uint64_t selected = 0, moved = 0;
    for (int s = 0; s < pop->T; ++s) {                       /* for layer l            */
        const uint32_t t = pop->tensor_id ? pop->tensor_id[s] : (uint32_t)s;
        const int64_t i0 = pop->coord_begin ? pop->coord_begin[s] : 0;
        const uint64_t thr = wo_threshold(p_seg[s]);
        const int64_t d = pop->numel[s];
        int64_t c;
#pragma omp parallel for schedule(static) reduction(+ : selected, moved) num_threads(wo_threads)
        for (c = 0; c < d; ++c) {                            /* for parameter i in l   */
            const uint64_t i = (uint64_t)(i0 + c);
            uint32_t w = wo_mask_word(seed, step, t, i);
            if ((uint64_t)w >= thr) continue;                /* with probability p_l   */
            int32_t perm[1024];
            wo_draw_permutation(seed, step, t, i, pop->N, perm);   /* pi_i             */
            wo_permute_column(pop, stack, dtype, pop->offset[s] + c, perm);
            if (stack2) wo_permute_column(pop, stack2, dtype2, pop->offset[s] + c, perm);
            selected += 1;
            for (int n = 0; n < pop->N; ++n) moved += (perm[n] != n);
        }
    }
    if (stats) { stats[0] += selected; stats[1] += moved; }
    return WO_OK;
}

/* ---- consensus (population mean) of one coordinate, binary32, fixed order ---- */
static inline float wo_mean_f32(const wo_population *pop, const void *stack, int dtype, int64_t elem)
{
    float s = wo_load(stack, dtype, wo_index(pop, 0, elem));
    for (int n = 1; n < pop->N; ++n) {
        float x = wo_load(stack, dtype, wo_index(pop, n, elem));
        s = s + x;                                   /* rounded to binary32 each time */
    }
    float m = s / (float)pop->N;
    return m;
}

/* ---- PAPA EMA, Eq. 1:  theta_n <- alpha theta_n + (1 - alpha) mean ---- */
int wo_papa_ema(const wo_population *pop, void *stack, int32_t dtype, float alpha)
{
    if (wo_check_pop(pop) != WO_OK || !stack) return WO_ERR_ARG;
    if (!(alpha > 0.0f && alpha < 1.0f)) return WO_ERR_ARG;
    float one_minus_alpha = 1.0f - alpha;
    for (int s = 0; s < pop->T; ++s) {
        int64_t c;
#pragma omp parallel for schedule(static) num_threads(wo_threads)
        for (c = 0; c < pop->numel[s]; ++c) {
            int64_t elem = pop->offset[s] + c;
            float m = wo_mean_f32(pop, stack, dtype, elem);
            float pull = one_minus_alpha * m;
            for (int n = 0; n < pop->N; ++n) {
                size_t idx = wo_index(pop, n, elem);
                float keep = alpha * wo_load(stack, dtype, idx);
                float r = keep + pull;
                wo_store(stack, dtype, idx, r);
            }
        }
    }
    return WO_OK;
}

/* ---- final average (output of Algorithm 1); out is one row of padded_P elements ---- */
int wo_population_average(const wo_population *pop, const void *stack, int32_t dtype,
                          void *out, int32_t out_dtype)
{
    if (wo_check_pop(pop) != WO_OK || !stack || !out) return WO_ERR_ARG;
    for (int s = 0; s < pop->T; ++s) {
        int64_t c;
#pragma omp parallel for schedule(static) num_threads(wo_threads)
        for (c = 0; c < pop->numel[s]; ++c) {
            int64_t elem = pop->offset[s] + c;
            float m = wo_mean_f32(pop, stack, dtype, elem);
            wo_store(out, out_dtype, (size_t)elem, m);
        }
    }
    return WO_OK;
}

/* ---- PAPA-all / DART step: every model becomes the average ---- */
int wo_papa_all(const wo_population *pop, void *stack, int32_t dtype)
{
    if (wo_check_pop(pop) != WO_OK || !stack) return WO_ERR_ARG;
    for (int s = 0; s < pop->T; ++s) {
        int64_t c;
#pragma omp parallel for schedule(static) num_threads(wo_threads)
        for (c = 0; c < pop->numel[s]; ++c) {
            int64_t elem = pop->offset[s] + c;
            float m = wo_mean_f32(pop, stack, dtype, elem);
            for (int n = 0; n < pop->N; ++n) wo_store(stack, dtype, wo_index(pop, n, elem), m);
        }
    }
    return WO_OK;
}

/* ---- distance to the consensus (Fig. 2; Eq. 2 and Eq. 5 speak of its square) ----
 * For the coordinates of segments seg_lo .. seg_hi-1, in binary64 throughout:
 *   sq_out[n] = sum_i (theta_n^i - mean^i)^2 ,  mean^i = (1/N) sum_n theta_n^i .
 * The figure's quantity is (1/N) sum_n sqrt(sq_out[n]); the equations' is sum_n sq_out[n]. */
int wo_consensus_sq(const wo_population *pop, const void *stack, int32_t dtype,
                    int32_t seg_lo, int32_t seg_hi, double *sq_out)
{
    if (wo_check_pop(pop) != WO_OK || !stack || !sq_out) return WO_ERR_ARG;
    if (seg_lo < 0 || seg_hi > pop->T || seg_lo > seg_hi) return WO_ERR_ARG;
    for (int n = 0; n < pop->N; ++n) sq_out[n] = 0.0;
    for (int s = seg_lo; s < seg_hi; ++s) {
        for (int64_t c = 0; c < pop->numel[s]; ++c) {
            int64_t elem = pop->offset[s] + c;
            double mean = 0.0;
            for (int n = 0; n < pop->N; ++n) mean += (double)wo_load(stack, dtype, wo_index(pop, n, elem));
            mean /= (double)pop->N;
            for (int n = 0; n < pop->N; ++n) {
                double dlt = (double)wo_load(stack, dtype, wo_index(pop, n, elem)) - mean;
                sq_out[n] += dlt * dlt;
            }
        }
    }
    return WO_OK;
}

/* ---- the shuffling step as the workers see it (one model per worker) ----
 * The paper's deployment keeps model n on worker n; a shuffled parameter travels
 * peer to peer along the permutation (Introduction: models communicate their
 * parameters peer-to-peer following the permutation; section "WASH": each model
 * communicates p x d parameters per step in expectation).  Every worker draws the same
 * mask and the same pi_i from the shared (seed, step), so only values travel.
 *
 * Wire format (a convention of this library, the paper has none): worker n owns a
 * staging buffer.  Visit the selected coordinates in the order of the shuffling loop
 * (segment by segment, coordinate by coordinate); each one with pi_i(n) != n takes the
 * next free slot of worker n's buffer, and the slot is filled by worker pi_i(n) with
 * its own value of that coordinate.  Fixed points (pi_i(n) == n) do not travel.
 *
 * wo_exchange_send    worker `self` fills its slots in every other worker's buffer.
 *                     row = the worker's own model (padded_P elements, `offset`s as in
 *                     the population; N and layout of `pop` describe the population, the
 *                     row itself is one model).  staging[n] = worker n's buffer
 *                     (staging[self] is not touched); capacity in elements, a slot
 *                     beyond it is an error.  filled[n] (may be NULL) = slots of worker
 *                     n written by this call.
 * wo_exchange_receive worker `self` replaces its value of every selected coordinate with
 *                     pi_i(self) != self by the next slot of its own buffer.
 *                     stats[0] += selected coordinates, stats[1] += values received.
 * wo_exchange_counts  need[n] = slots worker n's buffer needs in this step.
 * A send by every worker followed by a receive by every worker is the shuffling step
 * of wo_shuffle on the stacked population: that identity is the definition, and the
 * tests pin these functions to it. */
static int wo_check_exchange(const wo_population *pop, const double *p_seg, uint64_t step)
{
    if (wo_check_pop(pop) != WO_OK || !p_seg || pop->N < 2) return WO_ERR_ARG;
    if (step >> 56) return WO_ERR_ARG;
    for (int s = 0; s < pop->T; ++s)
        if (!(p_seg[s] >= 0.0 && p_seg[s] <= 1.0)) return WO_ERR_ARG;
    return WO_OK;
}

int wo_exchange_counts(const wo_population *pop, const double *p_seg, uint64_t seed, uint64_t step,
                       int64_t *need, int64_t *selected)
{
    if (wo_check_exchange(pop, p_seg, step) != WO_OK || !need) return WO_ERR_ARG;
    for (int n = 0; n < pop->N; ++n) need[n] = 0;
    int64_t sel = 0;
    for (int s = 0; s < pop->T; ++s) {
        const uint32_t t = pop->tensor_id ? pop->tensor_id[s] : (uint32_t)s;
        const int64_t i0 = pop->coord_begin ? pop->coord_begin[s] : 0;
        const uint64_t thr = wo_threshold(p_seg[s]);
        for (int64_t c = 0; c < pop->numel[s]; ++c) {
            const uint64_t i = (uint64_t)(i0 + c);
            if ((uint64_t)wo_mask_word(seed, step, t, i) >= thr) continue;
            int32_t perm[1024];
            wo_draw_permutation(seed, step, t, i, pop->N, perm);
            sel += 1;
            for (int n = 0; n < pop->N; ++n) need[n] += (perm[n] != n);
        }
    }
    if (selected) *selected = sel;
    return WO_OK;
}

int wo_exchange_send(const wo_population *pop, int32_t self, const void *row, int32_t dtype,
                     const double *p_seg, uint64_t seed, uint64_t step,
                     void *const *staging, int64_t capacity, int64_t *filled)
{
    if (wo_check_exchange(pop, p_seg, step) != WO_OK || !row || !staging) return WO_ERR_ARG;
    if (self < 0 || self >= pop->N) return WO_ERR_ARG;
    int64_t next[1024];                                  /* next free slot of every worker's buffer */
    for (int n = 0; n < pop->N; ++n) next[n] = 0;
    if (filled) for (int n = 0; n < pop->N; ++n) filled[n] = 0;
    for (int s = 0; s < pop->T; ++s) {
        const uint32_t t = pop->tensor_id ? pop->tensor_id[s] : (uint32_t)s;
        const int64_t i0 = pop->coord_begin ? pop->coord_begin[s] : 0;
        const uint64_t thr = wo_threshold(p_seg[s]);
        for (int64_t c = 0; c < pop->numel[s]; ++c) {
            const uint64_t i = (uint64_t)(i0 + c);
            if ((uint64_t)wo_mask_word(seed, step, t, i) >= thr) continue;
            int32_t perm[1024];
            wo_draw_permutation(seed, step, t, i, pop->N, perm);
            const int64_t elem = pop->offset[s] + c;
            for (int n = 0; n < pop->N; ++n) {
                if (perm[n] == n) continue;              /* worker n keeps its own value     */
                const int64_t slot = next[n]++;
                if (perm[n] != self) continue;           /* another worker fills this slot   */
                if (slot >= capacity) return WO_ERR_ARG;
                if (dtype == WO_F32) ((uint32_t *)staging[n])[slot] = ((const uint32_t *)row)[elem];
                else ((uint16_t *)staging[n])[slot] = ((const uint16_t *)row)[elem];
                if (filled) filled[n] += 1;
            }
        }
    }
    return WO_OK;
}

int wo_exchange_receive(const wo_population *pop, int32_t self, void *row, int32_t dtype,
                        const double *p_seg, uint64_t seed, uint64_t step,
                        const void *staging_self, int64_t capacity, uint64_t *stats)
{
    if (wo_check_exchange(pop, p_seg, step) != WO_OK || !row || !staging_self) return WO_ERR_ARG;
    if (self < 0 || self >= pop->N) return WO_ERR_ARG;
    int64_t next = 0;
    uint64_t selected = 0;
    for (int s = 0; s < pop->T; ++s) {
        const uint32_t t = pop->tensor_id ? pop->tensor_id[s] : (uint32_t)s;
        const int64_t i0 = pop->coord_begin ? pop->coord_begin[s] : 0;
        const uint64_t thr = wo_threshold(p_seg[s]);
        for (int64_t c = 0; c < pop->numel[s]; ++c) {
            const uint64_t i = (uint64_t)(i0 + c);
            if ((uint64_t)wo_mask_word(seed, step, t, i) >= thr) continue;
            int32_t perm[1024];
            wo_draw_permutation(seed, step, t, i, pop->N, perm);
            selected += 1;
            if (perm[self] == self) continue;
            if (next >= capacity) return WO_ERR_ARG;
            const int64_t elem = pop->offset[s] + c;
            if (dtype == WO_F32) ((uint32_t *)row)[elem] = ((const uint32_t *)staging_self)[next];
            else ((uint16_t *)row)[elem] = ((const uint16_t *)staging_self)[next];
            next += 1;
        }
    }
    if (stats) { stats[0] += selected; stats[1] += (uint64_t)next; }
    return WO_OK;
}
