/*
 * psops_ref.c -- CPU oracle for the PSO-PS synchronisation stage.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference that the
 * CUDA library is checked against.  It shares no code, header, table or
 * constant with the CUDA sources and must never be linked into or called from
 * the product path.
 *
 * What it follows (Ye, Han, Sun, Lv: "PSO-PS: Parameter Synchronization with
 * Particle Swarm Optimization for Distributed Training of Deep Neural
 * Networks"):
 *   - Eq. 5  linear inertia decay                      -> psops_ref_inertia
 *   - Algorithm 3 (global search: argmin of the losses) -> psops_ref_argmin
 *   - Algorithm 1, the "if loss < pBest_loss" branch    -> psops_ref_pbest_select
 *   - Eq. 6 / Eq. 7 velocity and position update        -> psops_ref_update_element
 *   - Algorithm 1, the synchronisation branch as a whole -> psops_ref_sync
 *   - Section II-B, parameter averaging, step 5          -> psops_ref_average
 *   - Section II-B, synchronous SGD update               -> psops_ref_ssgd
 *   - Section II-C, step 3 (gBest from history), as an option of psops_ref_sync
 * The random numbers r1, r2 of Eq. 6 come from Philox4x32-10 (Salmon, Moraes,
 * Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3", SC'11), written
 * here from the published round definition.
 * The quadratic stand-in fitness f(x) = sum_j d_j (x_j - t_j)^2 is not in the
 * paper; it plays the role the paper gives the training loss (Section III-A:
 * the fitness of a particle is its loss, lower is better).
 *
 * Arithmetic: fp32, IEEE round-to-nearest-even, one rounding per operation
 * written below; fused multiply-add only where fmaf() is written.  Compile
 * with -ffp-contract=off so that the compiler adds no fusion of its own.
 * Subnormals are kept.
 *
 * Pins (see tests): Philox known-answer vectors and an independent
 * big-integer implementation; hand-worked K=2 and K=3 updates; exact
 * identities; brute-force selection; closed forms for the schedule and the
 * average; for the fitness, closed forms plus hand-worked cancellation cases
 * in which every level of the summation order and the rounding of a term
 * change the fp32 result.  No function in this file is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------ */
/* Philox4x32-10 (SC'11, Section 3.3 and Table 2 constants).                 */
/* One round: two 32x32->64 multiplies of counter words 0 and 2, the high    */
/* halves are xor-ed with words 1, 3 and the round key, and the words are    */
/* permuted.  The key is advanced by the Weyl constants between rounds.      */
/* ------------------------------------------------------------------------ */
void psops_ref_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2],
                             uint32_t out[4])
{
    const uint64_t mult_a = 0xD2511F53u;      /* multiplies word 0 */
    const uint64_t mult_b = 0xCD9E8D57u;      /* multiplies word 2 */
    const uint32_t weyl_a = 0x9E3779B9u;      /* golden ratio      */
    const uint32_t weyl_b = 0xBB67AE85u;      /* sqrt(3) - 1       */
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) {
            k0 += weyl_a;
            k1 += weyl_b;
        }
        uint64_t pa = mult_a * (uint64_t)c0;
        uint64_t pb = mult_b * (uint64_t)c2;
        uint32_t hi_a = (uint32_t)(pa >> 32), lo_a = (uint32_t)pa;
        uint32_t hi_b = (uint32_t)(pb >> 32), lo_b = (uint32_t)pb;
        uint32_t n0 = hi_b ^ c1 ^ k0;
        uint32_t n1 = lo_b;
        uint32_t n2 = hi_a ^ c3 ^ k1;
        uint32_t n3 = lo_a;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* A 32-bit random word -> a uniform fp32 on the 2^24-point grid of [0,1).   */
/* Both steps are exact in fp32.  (r of Eq. 6: "random number between 0 and  */
/* 1"; the half-open grid is this library's reading.)                        */
float psops_ref_uniform(uint32_t word)
{
    return (float)(word >> 8) * 0x1p-24f;
}

/* The pair (r1, r2) of Eq. 6 for particle i, element d, sync step s.        */
/* One Philox call serves the element pair (2q, 2q+1): counter               */
/* {d>>1, i, s, 0}, key = the two halves of the 64-bit seed; the even        */
/* element takes output words 0,1 and the odd element words 2,3.             */
void psops_ref_draw(uint64_t seed, uint32_t s, uint32_t i, uint64_t d,
                    float *r1, float *r2)
{
    uint32_t ctr[4] = { (uint32_t)(d >> 1), i, s, 0u };
    uint32_t key[2] = { (uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32) };
    uint32_t o[4];
    psops_ref_philox4x32_10(ctr, key, o);
    if (d & 1u) {
        *r1 = psops_ref_uniform(o[2]);
        *r2 = psops_ref_uniform(o[3]);
    } else {
        *r1 = psops_ref_uniform(o[0]);
        *r2 = psops_ref_uniform(o[1]);
    }
}

/* Eq. 5: m = m_max - t (m_max - m_min) / t_max, evaluated in double from    */
/* the fp32 hyper-parameters and rounded once to fp32.  t is clamped to      */
/* [0, t_max] (the loop of Algorithm 1 never leaves that range).             */
float psops_ref_inertia(float m_max, float m_min, int64_t t, int64_t t_max)
{
    if (t < 0) t = 0;
    if (t > t_max) t = t_max;
    double m = (double)m_max
             - (double)t * ((double)m_max - (double)m_min) / (double)t_max;
    return (float)m;
}

/* Algorithm 3: index of the smallest loss.  A strict "<" scan from index 0  */
/* keeps the lowest index among equal minima.  The paper says nothing about  */
/* NaN; here a NaN loss never beats a number (a number replaces a NaN        */
/* incumbent), and if every loss is NaN the answer is index 0.               */
int psops_ref_argmin(const float *loss, int K)
{
    int g = 0;
    for (int i = 1; i < K; ++i) {
        const int incumbent_nan = (loss[g] != loss[g]);
        const int candidate_nan = (loss[i] != loss[i]);
        if (loss[i] < loss[g] || (incumbent_nan && !candidate_nan)) g = i;
    }
    return g;
}

/* Algorithm 1, pBest branch: a particle improves only on a strictly smaller */
/* loss; its pBest_loss then becomes that loss.                              */
void psops_ref_pbest_select(const float *loss, float *pbest_loss, int K,
                            uint8_t *improved)
{
    for (int i = 0; i < K; ++i) {
        improved[i] = (uint8_t)(loss[i] < pbest_loss[i]);
        if (improved[i]) pbest_loss[i] = loss[i];
    }
}

/* Eq. 6 and Eq. 7 for one (particle, element).  pp is the particle's pBest  */
/* AFTER the pBest branch of Algorithm 1 ran (so pp == xo when it improved). */
/* k1 = c1/lambda, k2 = c2/lambda.  Rounding sequence: two subtractions,     */
/* three products, two fused multiply-adds, one addition.                    */
void psops_ref_update_element(float m, float k1, float k2, float r1, float r2,
                              float xo, float vo, float pp, float gb,
                              float *vn, float *xn)
{
    float dl = pp - xo;                 /* pBest - w  */
    float dg = gb - xo;                 /* gBest - w  */
    float t1 = k1 * r1;                 /* c1 r1 / lambda */
    float t2 = k2 * r2;                 /* c2 r2 / lambda */
    float a0 = m * vo;                  /* inertia    */
    float vnew = fmaf(t2, dg, fmaf(t1, dl, a0));
    *vn = vnew;
    *xn = xo + vnew;                    /* Eq. 7      */
}

/*
 * One synchronisation (Algorithm 1, the "t % step == 0" branch) over n
 * columns of the swarm.
 *
 *   x, v, p      K rows of stride ld, updated in place
 *   loss         K current losses (the fitness of Table I)
 *   pbest_loss   K values, updated in place
 *   t, t_max     iteration counter of Eq. 5
 *   lambda       divisor of Eq. 6
 *   seed, s      Philox key and 0-based sync counter
 *   elem_index   NULL, or n global element indices: column j then stands for
 *                element elem_index[j] of a longer vector (used to follow a
 *                sample of columns of a large swarm; elements are independent
 *                of one another once the losses are given)
 *   fixed_r      NULL, or {r1, r2} used for every draw (worked examples)
 *   g_out, improved_out   selection results (may be NULL)
 *   gbest_out    NULL or n floats: the gBest row that Eq. 6 used
 *   hist_row, hist_loss, hist_valid
 *                all NULL: gBest is the best particle of THIS iteration
 *                (Algorithm 3).  All non-NULL: the standard-PSO variant
 *                (Section II-C, step 3: gBest "from the history of all
 *                particles"): the remembered row (n floats), its loss and a
 *                0/1 flag, updated in place -- the current best replaces the
 *                remembered one only on a strictly smaller loss (or when
 *                nothing is remembered yet), and Eq. 6 uses the remembered row
 *   nthreads     >1 splits the element loop across OpenMP threads; the result
 *                is the same because every draw is a pure function of
 *                (seed, s, i, d)
 * Returns 0, or -1 if the gBest snapshot could not be allocated.
 */
int psops_ref_sync(int K, int64_t n, int64_t ld, float *x, float *v, float *p,
                   const float *loss, float *pbest_loss,
                   float m_max, float m_min, int64_t t, int64_t t_max,
                   float c1, float c2, float lambda,
                   uint64_t seed, uint32_t s,
                   const int64_t *elem_index, const float *fixed_r,
                   int *g_out, uint8_t *improved_out, float *gbest_out,
                   float *hist_row, float *hist_loss, int *hist_valid,
                   int nthreads)
{
    /* schedule scalars */
    const float m  = psops_ref_inertia(m_max, m_min, t, t_max);
    const float k1 = c1 / lambda;
    const float k2 = c2 / lambda;

    /* Algorithm 3, then the pBest branch of Algorithm 1 */
    const int g = psops_ref_argmin(loss, K);
    uint8_t *improved = (uint8_t *)malloc((size_t)(K > 0 ? K : 1));
    float *gb = (float *)malloc(sizeof(float) * (size_t)(n > 0 ? n : 1));
    if (!improved || !gb) { free(improved); free(gb); return -1; }
    psops_ref_pbest_select(loss, pbest_loss, K, improved);

    /* gBest is the best particle's weights at this iteration: copy the row   */
    /* before anything is overwritten.                                        */
    memcpy(gb, x + (size_t)g * (size_t)ld, sizeof(float) * (size_t)n);
    if (hist_row && hist_loss && hist_valid) {
        if (!*hist_valid || loss[g] < *hist_loss) {
            memcpy(hist_row, gb, sizeof(float) * (size_t)n);     /* new best in history */
            *hist_loss = loss[g];
            *hist_valid = 1;
        } else {
            memcpy(gb, hist_row, sizeof(float) * (size_t)n);     /* keep the remembered one */
        }
    }

    if (nthreads < 1) nthreads = 1;
#pragma omp parallel for num_threads(nthreads) schedule(static)
    for (int64_t j = 0; j < n; ++j) {
        const uint64_t d = elem_index ? (uint64_t)elem_index[j] : (uint64_t)j;
        for (int i = 0; i < K; ++i) {
            const size_t at = (size_t)i * (size_t)ld + (size_t)j;
            float r1, r2;
            if (fixed_r) { r1 = fixed_r[0]; r2 = fixed_r[1]; }
            else psops_ref_draw(seed, s, (uint32_t)i, d, &r1, &r2);
            const float xo = x[at];
            const float vo = v[at];
            const float pp = improved[i] ? xo : p[at];   /* pBest_i = w_i */
            float vn, xn;
            psops_ref_update_element(m, k1, k2, r1, r2, xo, vo, pp, gb[j],
                                     &vn, &xn);
            v[at] = vn;
            x[at] = xn;
            if (improved[i]) p[at] = xo;
        }
    }

    if (g_out) *g_out = g;
    if (improved_out) memcpy(improved_out, improved, (size_t)K);
    if (gbest_out) memcpy(gbest_out, gb, sizeof(float) * (size_t)n);
    free(improved);
    free(gb);
    return 0;
}

/* Parameter averaging (Section II-B, step 5): new weight = (1/n) sum_k w^k, */
/* handed back to every worker.  fp32 sum in worker order, one division.     */
void psops_ref_average(int K, int64_t n, int64_t ld, float *x, int nthreads)
{
    if (nthreads < 1) nthreads = 1;
#pragma omp parallel for num_threads(nthreads) schedule(static)
    for (int64_t j = 0; j < n; ++j) {
        float acc = x[j];
        for (int k = 1; k < K; ++k)
            acc = acc + x[(size_t)k * (size_t)ld + (size_t)j];
        const float mean = acc / (float)K;
        for (int k = 0; k < K; ++k)
            x[(size_t)k * (size_t)ld + (size_t)j] = mean;
    }
}

/* Synchronous SGD as the paper states it next to parameter averaging        */
/* (Section II-B): w_{i+1} = w_i + (1/n) alpha sum_k grad_k, handed to every  */
/* worker.  fp32: gradients summed in worker order, scale = alpha / n (one    */
/* division), one product, one addition.  w holds the n workers' (identical   */
/* or not) weights; the new weight is computed from worker 0's row.           */
void psops_ref_ssgd(int K, int64_t n, int64_t ld, float *w, const float *grad,
                    int64_t grad_ld, float alpha, int nthreads)
{
    if (nthreads < 1) nthreads = 1;
    const float scale = alpha / (float)K;
#pragma omp parallel for num_threads(nthreads) schedule(static)
    for (int64_t j = 0; j < n; ++j) {
        float acc = grad[j];
        for (int k = 1; k < K; ++k)
            acc = acc + grad[(size_t)k * (size_t)grad_ld + (size_t)j];
        const float step = scale * acc;
        const float wn = w[j] + step;
        for (int k = 0; k < K; ++k)
            w[(size_t)k * (size_t)ld + (size_t)j] = wn;
    }
}

/* ------------------------------------------------------------------------ */
/* Quadratic fitness  f(x) = sum_j dvec_j (x_j - tvec_j)^2.                  */
/* The summation order is part of the definition so that the argmin over     */
/* particles is reproducible:                                                */
/*   term_j   = dvec_j * (e*e), e = x_j - tvec_j   (three fp32 operations),  */
/*              widened to fp64; indices >= N contribute +0.0                */
/*   level 0  q_k = ((term_4k + term_4k+1) + term_4k+2) + term_4k+3          */
/*   level 1  every 32 consecutive q (128 elements) are reduced by the       */
/*            butterfly  a[l] += a[l ^ off], off = 16, 8, 4, 2, 1            */
/*   level 2  tile value m goes to slot m % 1024 (added in increasing m,     */
/*            starting from +0.0); the 1024 slots are reduced as 32 groups   */
/*            of 32 by the same butterfly; the 32 group values are added in  */
/*            group order; the result is rounded to fp32.                    */
/* ------------------------------------------------------------------------ */
static double butterfly32(double a[32])
{
    for (int off = 16; off >= 1; off >>= 1) {
        double b[32];
        for (int l = 0; l < 32; ++l) b[l] = a[l] + a[l ^ off];
        for (int l = 0; l < 32; ++l) a[l] = b[l];
    }
    return a[0];
}

static double quad_term(const float *x, const float *dvec, const float *tvec,
                        int64_t j, int64_t N)
{
    if (j >= N) return 0.0;
    float e = x[j] - tvec[j];
    float e2 = e * e;
    float term = dvec[j] * e2;
    return (double)term;
}

float psops_ref_quadratic_fitness(const float *x, const float *dvec,
                                  const float *tvec, int64_t N)
{
    double slot[1024];
    for (int tau = 0; tau < 1024; ++tau) slot[tau] = 0.0;
    const int64_t tiles = (N + 127) / 128;
    for (int64_t mt = 0; mt < tiles; ++mt) {
        double q[32];
        for (int l = 0; l < 32; ++l) {
            const int64_t j = mt * 128 + 4 * (int64_t)l;
            double a = quad_term(x, dvec, tvec, j, N);
            a = a + quad_term(x, dvec, tvec, j + 1, N);
            a = a + quad_term(x, dvec, tvec, j + 2, N);
            a = a + quad_term(x, dvec, tvec, j + 3, N);
            q[l] = a;
        }
        slot[mt % 1024] = slot[mt % 1024] + butterfly32(q);
    }
    double total = 0.0;
    for (int grp = 0; grp < 32; ++grp) {
        double a[32];
        for (int l = 0; l < 32; ++l) a[l] = slot[grp * 32 + l];
        double gsum = butterfly32(a);
        total = (grp == 0) ? gsum : total + gsum;
    }
    return (float)total;
}

/* Fitness of every particle: loss_i = f(row i of x).                        */
void psops_ref_quadratic_losses(int K, int64_t N, int64_t ld, const float *x,
                                const float *dvec, const float *tvec,
                                float *loss, int nthreads)
{
    if (nthreads < 1) nthreads = 1;
#pragma omp parallel for num_threads(nthreads) schedule(static)
    for (int i = 0; i < K; ++i)
        loss[i] = psops_ref_quadratic_fitness(x + (size_t)i * (size_t)ld,
                                              dvec, tvec, N);
}
