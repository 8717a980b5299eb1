/*
 * lgn_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, scalar CPU statement of the lognormal gradient-compression
 * path of "Neural gradients are near-lognormal: improved quantized and sparse
 * training" (arXiv 2006.08173).  It exists so that tests can decide whether
 * the CUDA library computes what the paper defines.  Only tests, the smoke
 * check and the benchmark's CPU-baseline leg may load it; the CUDA library
 * never does, and the two share no source, header, table or helper.
 *
 * Everything real-valued is fp64.  Nothing is blocked, fused, vectorised or
 * reordered: each function follows the cited passage step by step.
 *
 * Pins (each function below is checked, in the CPU test-suite, against
 * something other than itself):
 *   orc_stats_*        closed-form hand cases (powers of two), recovery of the
 *                      generator's (mu, sigma) within sampling error
 *   orc_sparsity_of    numeric quadrature of Eq. 6/7 with a library lognormal
 *                      CDF, Monte-Carlo, sigma->0 limit
 *   orc_threshold      inverse of the above; bi-modal identity l+(1-l)S'=S
 *   orc_prune_*        three-value property, unbiasedness, achieved sparsity
 *   orc_expected_rel_err / orc_fp_format
 *                      Table 2 of the paper; the constants printed in the
 *                      derivation of Eq. 4; Monte-Carlo with orc_quantize
 *   orc_quantize_*     brute force over every code of every format
 *   orc_philox4x32     known-answer vectors published with the generator (10 rounds)
 *   orc_stats_masked   hand cases (powers of two under a hand-written mask); recovery of the
 *                      right mode's generator parameters and of l on a two-mode tensor;
 *                      the identity l + (1-l) S' = S as achieved sparsity when the left mode
 *                      lies orders of magnitude below the right one (Appendix A.9)
 *   orc_scale_exp_from_max
 *                      powers of two and their neighbours by hand; the largest element's
 *                      exponent lands on E_max - 1 (checked with frexp in the test); no
 *                      element is clipped before rounding
 *   orc_cosine_similarity
 *                      Monte-Carlo: the measured cosine between a truncated lognormal sample
 *                      and its stochastically pruned copy (orc_prune_one); alpha -> 0 gives 1;
 *                      decreasing in alpha
 *   orc_threshold_for_cosine
 *                      inverse of the above (forward evaluation returns the target)
 *   orc_allocate_sparsity
 *                      hand-computed two- and three-layer budgets; the element-weighted mean of
 *                      the result equals the requested overall sparsity; the cap; layers whose
 *                      cosine is already above their floor keep the overall sparsity
 *   orc_dequantize     every code of every format against the value formula of Eq. 1-2
 *                      written out in the test; quantising the decoded value (nearest)
 *                      gives the code back
 *   orc_prefix_*       the code table of the paper's appendix written out by hand for a
 *                      worked example; decode(encode(x)) == x; length = n0 + 3 n_alpha +
 *                      (2 + width) n_fp; the paper's "4 bits at 80 %, 2 bits at 90 %"
 *   end-to-end tensors parity unpinned by the paper (it prints no worked
 *                      numeric example of a compressed tensor)
 *
 * Build: gcc -O2 -std=c99 -fPIC -shared -fno-fast-math lgn_oracle.c -lm
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------ */
/* element access: every storage type converts exactly to double       */
/* ------------------------------------------------------------------ */

enum { ORC_F32 = 0, ORC_BF16 = 1 };

static double bf16_to_double(uint16_t h)
{
    /* bfloat16 = the upper 16 bits of an IEEE binary32 */
    uint32_t w = (uint32_t)h << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

static double elem(const void *g, int dtype, uint64_t i)
{
    if (dtype == ORC_BF16)
        return bf16_to_double(((const uint16_t *)g)[i]);
    return (double)((const float *)g)[i];
}

/* round a double to the nearest bfloat16 via binary32 (ties to even both times) */
static double round_to_bf16(double v)
{
    float f = (float)v;               /* fp64 -> fp32, round to nearest even */
    uint32_t w;
    memcpy(&w, &f, sizeof w);
    uint32_t keep = w >> 16, rest = w & 0xFFFFu;
    if (rest > 0x8000u || (rest == 0x8000u && (keep & 1u)))
        keep += 1;                    /* carry may run into the exponent: that is the right value */
    w = keep << 16;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

/* ------------------------------------------------------------------ */
/* Section 3 / Appendix "bi-modal" step (3): lognormal parameters       */
/* ------------------------------------------------------------------ */

typedef struct {
    uint64_t n;         /* elements                                   */
    uint64_t nnz;       /* entries != 0 (+0 and -0 are both zero)      */
    double   mu;        /* mean of ln|g| over the nonzero entries      */
    double   sigma;     /* population std of ln|g| over the same       */
    double   zero_frac; /* l = 1 - nnz/n (0 for n == 0)                */
} orc_stats_t;

/* The analysis is done on |g| with the zero entries left out (Section 3);
 * mu and sigma are the mean and standard deviation of the natural log
 * (the two O(n) quantities the method needs, Appendix A.8).
 * Two passes, compensated (Kahan) sums. */
void orc_stats(const void *g, uint64_t n, int dtype, orc_stats_t *out)
{
    uint64_t nnz = 0;
    double sum = 0.0, comp = 0.0;
    for (uint64_t i = 0; i < n; ++i) {
        double x = elem(g, dtype, i);
        if (x == 0.0) continue;
        double y = log(fabs(x)) - comp;
        double t = sum + y;
        comp = (t - sum) - y;
        sum = t;
        ++nnz;
    }
    double mu = nnz ? sum / (double)nnz : 0.0;
    double ss = 0.0; comp = 0.0;
    for (uint64_t i = 0; i < n; ++i) {
        double x = elem(g, dtype, i);
        if (x == 0.0) continue;
        double d = log(fabs(x)) - mu;
        double y = d * d - comp;
        double t = ss + y;
        comp = (t - ss) - y;
        ss = t;
    }
    out->n = n;
    out->nnz = nnz;
    out->mu = mu;
    out->sigma = nnz ? sqrt(ss / (double)nnz) : 0.0;
    out->zero_frac = n ? 1.0 - (double)nnz / (double)n : 0.0;
}

/* Appendix "bi-modal lognormal pruning", steps (1) and (3).  The gradient before
 * batch-norm has two modes; they are told apart by the SAME entry of the gradient
 * after batch-norm (after the ReLU's backward): zero there -> left mode, non-zero
 * -> right mode.  right_mode[i] != 0 marks the right-mode entries (one byte each).
 *   l         = (entries of the left mode) / n                      step (1)
 *   mu, sigma = mean and std of ln|g| over the right-mode entries   step (3)
 * (a right-mode entry that is itself exactly zero has no logarithm and is left
 * out of the mean and the deviation, like in orc_stats; it still counts as
 * right mode in l).  out->nnz is the number of entries that entered mu and sigma;
 * out->zero_frac is l.  *n_right receives the size of the right mode. */
void orc_stats_masked(const void *g, const uint8_t *right_mode, uint64_t n, int dtype,
                      orc_stats_t *out, uint64_t *n_right)
{
    uint64_t cnt = 0, right = 0;
    double sum = 0.0, comp = 0.0;
    for (uint64_t i = 0; i < n; ++i) {
        if (!right_mode[i]) continue;
        ++right;
        double x = elem(g, dtype, i);
        if (x == 0.0) continue;
        double y = log(fabs(x)) - comp;
        double t = sum + y;
        comp = (t - sum) - y;
        sum = t;
        ++cnt;
    }
    double mu = cnt ? sum / (double)cnt : 0.0;
    double ss = 0.0; comp = 0.0;
    for (uint64_t i = 0; i < n; ++i) {
        if (!right_mode[i]) continue;
        double x = elem(g, dtype, i);
        if (x == 0.0) continue;
        double d = log(fabs(x)) - mu;
        double y = d * d - comp;
        double t = ss + y;
        comp = (t - ss) - y;
        ss = t;
    }
    out->n = n;
    out->nnz = cnt;
    out->mu = mu;
    out->sigma = cnt ? sqrt(ss / (double)cnt) : 0.0;
    out->zero_frac = n ? 1.0 - (double)right / (double)n : 0.0;
    *n_right = right;
}

/* max |g| over the whole tensor (Algorithm 1, "max(|X|)"). */
double orc_max_abs(const void *g, uint64_t n, int dtype)
{
    double m = 0.0;
    for (uint64_t i = 0; i < n; ++i) {
        double a = fabs(elem(g, dtype, i));
        if (a > m) m = a;
    }
    return m;
}

/* Algorithm 1, the scale from the maximum.  The printed line
 * "mu_l = floor(log2 max|X|) / log2(E_max)" does not give an exponent shift as it
 * stands; the text around it fixes what it is for: the scale gives up the smallest
 * elements so that the largest magnitudes stay representable.  With
 * representable exponents -E_max+1 .. E_max-1 that is the power of two that puts
 * the largest element in the top binade:
 *     e_s = floor(log2 max|X|) - (E_max - 1).
 * max_abs must be > 0. */
int orc_scale_exp_from_max(double max_abs, int n2)
{
    int ex;
    (void)frexp(max_abs, &ex);            /* max_abs = f * 2^ex, f in [0.5, 1): floor(log2) = ex - 1 */
    int Emax = 1 << (n2 - 1);
    return (ex - 1) - (Emax - 1);
}

/* ------------------------------------------------------------------ */
/* Randomness: Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11)        */
/* ------------------------------------------------------------------ */

/* One bijection round: two 32x32->64 products, cross-xored with the
 * counter and the round key. */
static void philox_round(uint32_t c[4], const uint32_t k[2])
{
    uint64_t p0 = (uint64_t)0xD2511F53u * c[0];
    uint64_t p1 = (uint64_t)0xCD9E8D57u * c[2];
    uint32_t n0 = (uint32_t)(p1 >> 32) ^ c[1] ^ k[0];
    uint32_t n1 = (uint32_t)p1;
    uint32_t n2 = (uint32_t)(p0 >> 32) ^ c[3] ^ k[1];
    uint32_t n3 = (uint32_t)p0;
    c[0] = n0; c[1] = n1; c[2] = n2; c[3] = n3;
}

void orc_philox4x32(const uint32_t ctr[4], const uint32_t key[2], int rounds, uint32_t out[4])
{
    uint32_t c[4] = { ctr[0], ctr[1], ctr[2], ctr[3] };
    uint32_t k[2] = { key[0], key[1] };
    for (int r = 0; r < rounds; ++r) {
        if (r) {                       /* Weyl key schedule between rounds */
            k[0] += 0x9E3779B9u;
            k[1] += 0xBB67AE85u;
        }
        philox_round(c, k);
    }
    memcpy(out, c, sizeof c);
}

/* The method draws 16 random bits per element from Philox4x32-7 (seven rounds:
 * the fewest for which the generator's authors report a clean BigCrush run;
 * ten is their default with a safety margin).  One 128-bit block serves the
 * eight elements 8b..8b+7: key = the seed's two halves, counter = (b low,
 * b high, 0, 0); element i takes word (i/2) mod 4, low half if i is even,
 * high half if odd.  A pure function of (seed, i). */
enum { ORC_PHILOX_ROUNDS = 7 };

uint32_t orc_rand16(uint64_t seed, uint64_t i)
{
    uint64_t blk = i >> 3;
    uint32_t ctr[4] = { (uint32_t)blk, (uint32_t)(blk >> 32), 0u, 0u };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t o[4];
    orc_philox4x32(ctr, key, ORC_PHILOX_ROUNDS, o);
    uint32_t w = o[(i >> 1) & 3u];
    return (i & 1u) ? (w >> 16) : (w & 0xFFFFu);
}

void orc_rand16_fill(uint64_t seed, uint64_t first, uint64_t n, uint16_t *out)
{
    for (uint64_t j = 0; j < n; ++j) out[j] = (uint16_t)orc_rand16(seed, first + j);
}

/* ------------------------------------------------------------------ */
/* Section 5, Eq. 6-8: sparsity as a function of the threshold          */
/* ------------------------------------------------------------------ */

/* Eq. 8 with t = alpha / e^mu and u = ln t: the expected fraction of a
 * Lognormal(mu, sigma^2) population that stochastic pruning at threshold
 * alpha sends to zero,
 *
 *   S = 1/2 + 1/(2t) * [ e^{s^2/2} erf(s/rt2 - u/(rt2 s)) + t erf(u/(rt2 s)) - e^{s^2/2} ].
 *
 * The first and last bracket terms are joined as -e^{s^2/2} erfc(.) (the
 * same number, without the cancellation of erf(.) - 1), and 1/2 + 1/2 erf(v)
 * is written 1/2 erfc(-v).  Valid for 1e-6 <= sigma <= 25 (orc_threshold
 * clamps).  Beyond z = 26 erfc is about to underflow while e^{s^2/2}/t is
 * about to overflow; there S < 1e-60 for every sigma in range and the joined
 * term is dropped (S stays monotone in u, which is all the solver needs). */
double orc_sparsity_of(double u, double sigma)
{
    const double rt2 = sqrt(2.0);
    double z = sigma / rt2 - u / (rt2 * sigma);
    double s = 0.5 * erfc(-u / (rt2 * sigma));      /* = 1/2 + 1/2 erf(u/(rt2 s)), exact in both tails */
    if (z < 26.0)
        s -= 0.5 * exp(0.5 * sigma * sigma - u) * erfc(z);
    return s;
}

/* Appendix A.9 steps (1),(2) + Eq. 8 solved for alpha.
 *   l  = fraction of the tensor that is exactly zero (the left mode)
 *   S' = (S - l) / (1 - l): sparsity still to be induced in the nonzero part
 * S' <= 0 (already sparse enough) or an all-zero tensor gives tau = 0, which
 * leaves the tensor unchanged.  sigma is clamped to [1e-6, 25] (the low end: a
 * tensor whose nonzero magnitudes are all equal; the high end is wider than
 * the whole fp32 range).  Eq. 8 is "solved numerically": here by
 * bisection on u over a bracket that holds every S' a double can express,
 * until the bracket cannot shrink.  Returns 0, or -1 for arguments outside
 * 0 <= S < 1, 0 <= l <= 1. */
int orc_threshold(double mu, double sigma, double zero_frac, double S, double *tau)
{
    *tau = 0.0;
    if (!(S >= 0.0 && S < 1.0) || !(zero_frac >= 0.0 && zero_frac <= 1.0)) return -1;
    if (zero_frac >= 1.0) return 0;
    double Sp = (S - zero_frac) / (1.0 - zero_frac);
    if (Sp <= 0.0) return 0;
    if (!(sigma >= 1e-6)) sigma = 1e-6;
    if (sigma > 25.0) sigma = 25.0;
    double lo = -(40.0 * sigma + 50.0), hi = 40.0 * sigma + 50.0;
    for (int it = 0; it < 300; ++it) {
        double mid = 0.5 * (lo + hi);
        if (mid <= lo || mid >= hi) break;
        if (orc_sparsity_of(mid, sigma) < Sp) lo = mid; else hi = mid;
    }
    *tau = exp(mu + 0.5 * (lo + hi));
    return 0;
}

/* The threshold as the kernel can hold it: rounded to the tensor's storage
 * type (fp32: one rounding; bf16: fp32 then bf16), both ties-to-even, and
 * kept finite. */
double orc_snap_tau(double tau, int dtype)
{
    double t = (dtype == ORC_BF16) ? round_to_bf16(tau) : (double)(float)tau;
    double top = (dtype == ORC_BF16) ? 0x1.FEp127 : 0x1.FFFFFEp127;
    return t > top ? top : t;
}

/* ------------------------------------------------------------------ */
/* Section 5, Eq. 5: stochastic pruning                                 */
/* ------------------------------------------------------------------ */

/* T_{alpha,eps}(x) for one element, with the element's 16 random bits h
 * given.  eps = (h + 1) / 2^16 is uniform on (0,1] in steps of 2^-16 (never
 * zero, so that alpha*eps > 0 and a zero can never reach the middle case).
 * The product alpha*eps is rounded once to fp32 (the precision the kernel
 * compares in); |x| and alpha are exact in fp32.
 *   alpha == 0               -> x, bit for bit (nothing is pruned)
 *   |x| > alpha              -> x
 *   alpha*eps <= |x| <= alpha -> sign(x)*alpha   (x == 0 stays +0)
 *   |x| < alpha*eps          -> +0 */
double orc_prune_one(double x, double tau_used, uint32_t h)
{
    if (tau_used == 0.0) return x;
    double a = fabs(x);
    if (a > tau_used) return x;
    double eps = (double)((h & 0xFFFFu) + 1u) / 65536.0;
    double thr = (double)(float)(tau_used * eps);   /* exact product, one rounding */
    if (a != 0.0 && a >= thr) return x < 0.0 ? -tau_used : tau_used;
    return 0.0;
}

static void store_elem(void *out, int dtype, uint64_t i, double v)
{
    float f = (float)v;                 /* v is representable: no rounding happens */
    if (dtype == ORC_BF16) {
        uint32_t w; memcpy(&w, &f, sizeof w);
        ((uint16_t *)out)[i] = (uint16_t)(w >> 16);
    } else {
        ((float *)out)[i] = f;
    }
}

/* Whole tensor, random bits supplied by the caller (h[i] belongs to element i). */
void orc_prune_with_bits(const void *g, void *out, uint64_t n, int dtype,
                         double tau_used, const uint16_t *h)
{
    for (uint64_t i = 0; i < n; ++i)
        store_elem(out, dtype, i, orc_prune_one(elem(g, dtype, i), tau_used, h[i]));
}

/* Whole tensor, random bits from the counter-based generator; element i of
 * this buffer is element first+i of the tensor. */
void orc_prune(const void *g, void *out, uint64_t n, int dtype,
               double tau_used, uint64_t seed, uint64_t first)
{
    for (uint64_t i = 0; i < n; ++i)
        store_elem(out, dtype, i,
                   orc_prune_one(elem(g, dtype, i), tau_used, orc_rand16(seed, first + i)));
}

/* ------------------------------------------------------------------ */
/* Section 4, Eq. 4: expected relative error and the optimal split      */
/* ------------------------------------------------------------------ */

/* Eq. 4 for n1 mantissa and n2 exponent bits, E_max = 2^(n2-1).
 *
 * Readings taken (the paper uses one symbol for two logarithms and two
 * values for the mantissa step):
 *  - The derivation treats the base-2 exponent E as N(0, s^2); for a tensor
 *    whose NATURAL log has standard deviation sigma that s is sigma/ln 2.
 *  - The mantissa step is Delta = 2^-n1, as the problem statement defines
 *    it, so that n1 = 0 (formats 1-3-0, 1-4-0, 1-5-0 of Table 2) is finite.
 *
 * With q = E_max/(rt2 s):
 *   term 1: (2 Phi(E_max/s) - 1) / (8 ln2 2^n1)           mantissa noise in range
 *   term 2: 2^(E_max-1) e^{s^2 ln^2 2 / 2} (erf(s ln2/rt2 + q) - 1)
 *   term 3: -1/2 erf(q) + 3/2 - Phi(E_max/s)
 * erf(.) - 1 is written -erfc(.), and term 3, with Phi = 1/2 + 1/2 erf(q),
 * is 1 - erf(q) = erfc(q): the same numbers without cancellation. */
double orc_expected_rel_err(double sigma, int n1, int n2)
{
    const double rt2 = sqrt(2.0), ln2 = log(2.0);
    double s = sigma / ln2;
    double Emax = ldexp(1.0, n2 - 1);
    double q = Emax / (rt2 * s);
    double Phi = 0.5 * erfc(-q);
    double t1 = (2.0 * Phi - 1.0) / (8.0 * ln2 * ldexp(1.0, n1));
    double t2 = -ldexp(1.0, (int)Emax - 1) * exp(0.5 * s * s * ln2 * ln2) * erfc(s * ln2 / rt2 + q);
    double t3 = erfc(q);
    return t1 + t2 + t3;
}

/* Section 4.3: among the splits n1 + n2 = nbits - 1 with n2 >= 1, the one
 * that minimises Eq. 4 (equal values: the smaller n2).  The per-layer scale
 * is the power of two nearest the median magnitude e^mu, e_s = floor(mu/ln2
 * + 1/2): Eq. 4 assumes the exponent distribution centred on the format's
 * range, and Algorithm 1 scales by a power of two so that X/2^e_s is an
 * exponent shift.  An all-zero tensor gets the narrowest exponent and no
 * shift.  sigma is clamped to [1e-6, 25].  Returns 0, -1 for nbits
 * outside 4..8. */
int orc_fp_format(double mu, double sigma, uint64_t nnz, int nbits,
                  int *exp_bits, int *man_bits, int *scale_exp)
{
    if (nbits < 4 || nbits > 8) return -1;
    if (nnz == 0) { *exp_bits = 1; *man_bits = nbits - 2; *scale_exp = 0; return 0; }
    if (!(sigma >= 1e-6)) sigma = 1e-6;
    if (sigma > 25.0) sigma = 25.0;
    int best = 1;
    double best_eta = orc_expected_rel_err(sigma, nbits - 2, 1);
    for (int n2 = 2; n2 <= nbits - 1; ++n2) {
        double eta = orc_expected_rel_err(sigma, nbits - 1 - n2, n2);
        if (eta < best_eta) { best_eta = eta; best = n2; }
    }
    *exp_bits = best;
    *man_bits = nbits - 1 - best;
    *scale_exp = (int)floor(mu / log(2.0) + 0.5);
    return 0;
}

/* ------------------------------------------------------------------ */
/* Section 4.1, Eq. 1-2 and Algorithm 1: the FP quantiser               */
/* ------------------------------------------------------------------ */

enum { ORC_ROUND_NEAREST = 0, ORC_ROUND_STOCHASTIC = 1 };

/* One element -> its (1 + n2 + n1)-bit code [sign | exponent field | mantissa].
 *
 * x is first divided by the layer scale 2^e_s (Algorithm 1), then written
 * M * 2^E with M in [1,2) and E integer (Eq. 1).  E_max = 2^(n2-1).
 * Eq. 2 on that E, before any rounding:
 *   E >= E_max  -> clipped.  2^E_max itself is not on the grid of a format
 *                  that also has to hold zero, so the clip value is the
 *                  largest code: exponent field 2^n2 - 1, mantissa all ones.
 *   E <= -E_max -> 0, as printed, under both roundings ("these tiny
 *                  gradients can be pruned", Section 4.4).
 *   otherwise   -> M is rounded to n1 fraction bits (step Delta = 2^-n1).
 *                  Nearest: ties to even.  Stochastic: h/2^16 of one step is
 *                  added and the sum is truncated.  M_q = 2 carries into E; if that reaches E_max
 *                  the value is clipped as above.
 * Exponent field = E + E_max in 1..2^n2-1; field 0 is zero.  Zero carries
 * sign 0.  h = the element's 16 random bits (unused for round-to-nearest). */
uint32_t orc_quantize_one(double x, int n2, int n1, int e_s, int rounding, uint32_t h)
{
    if (x == 0.0) return 0;
    int nbits = 1 + n2 + n1;
    uint32_t sign = (x < 0.0) ? (1u << (nbits - 1)) : 0u;
    uint32_t top = ((1u << n2) - 1u) << n1 | ((1u << n1) - 1u);
    int Emax = 1 << (n2 - 1);

    double a = ldexp(fabs(x), -e_s);          /* exact */
    int ex;
    double M = 2.0 * frexp(a, &ex);           /* a = M * 2^E, M in [1,2) */
    int E = ex - 1;

    if (E >= Emax) return sign | top;
    if (E <= -Emax) return 0;
    double steps = (M - 1.0) * ldexp(1.0, n1);           /* exact: M has <= 23 fraction bits */
    double m;
    if (rounding == ORC_ROUND_STOCHASTIC) {
        m = floor(steps + (double)(h & 0xFFFFu) / 65536.0);   /* exact sum */
    } else {
        m = nearbyint(steps);                            /* default mode: ties to even */
    }
    if (m == ldexp(1.0, n1)) { m = 0.0; E += 1; if (E == Emax) return sign | top; }
    return sign | ((uint32_t)(E + Emax) << n1) | (uint32_t)m;
}

/* The real value a code stands for (Algorithm 1: X_Q = 2^e_s * Q_FP(.)). */
double orc_decode(uint32_t code, int n2, int n1, int e_s)
{
    int nbits = 1 + n2 + n1;
    uint32_t field = (code >> n1) & ((1u << n2) - 1u);
    uint32_t man = code & ((1u << n1) - 1u);
    if (field == 0) return 0.0;
    int Emax = 1 << (n2 - 1);
    double v = ldexp(1.0 + ldexp((double)man, -n1), (int)field - Emax + e_s);
    return (code >> (nbits - 1)) & 1u ? -v : v;
}

/* Whole tensor -> one code per byte; random bits supplied (h may be NULL for
 * round-to-nearest). */
void orc_quantize_with_bits(const void *g, uint8_t *codes, uint64_t n, int dtype,
                            int n2, int n1, int e_s, int rounding, const uint16_t *h)
{
    for (uint64_t i = 0; i < n; ++i)
        codes[i] = (uint8_t)orc_quantize_one(elem(g, dtype, i), n2, n1, e_s, rounding, h ? h[i] : 0u);
}

/* Whole tensor, random bits from the counter-based generator. */
void orc_quantize(const void *g, uint8_t *codes, uint64_t n, int dtype,
                  int n2, int n1, int e_s, int rounding, uint64_t seed, uint64_t first)
{
    for (uint64_t i = 0; i < n; ++i) {
        uint32_t h = (rounding == ORC_ROUND_STOCHASTIC) ? orc_rand16(seed, first + i) : 0u;
        codes[i] = (uint8_t)orc_quantize_one(elem(g, dtype, i), n2, n1, e_s, rounding, h);
    }
}

/* Packed form: a little-endian bit stream, code i in bits [i*nbits, (i+1)*nbits),
 * bit b of the stream = bit (b mod 8) of byte b/8.  `packed` must hold
 * orc_packed_bytes(n, nbits) bytes; the bits past the last code are zero. */
uint64_t orc_packed_bytes(uint64_t n, int nbits)
{
    uint64_t bytes = (n * (uint64_t)nbits + 7u) / 8u;
    return (bytes + 3u) / 4u * 4u;
}

void orc_pack(const uint8_t *codes, uint64_t n, int nbits, uint8_t *packed)
{
    memset(packed, 0, orc_packed_bytes(n, nbits));
    for (uint64_t i = 0; i < n; ++i)
        for (int b = 0; b < nbits; ++b)
            if ((codes[i] >> b) & 1u) {
                uint64_t pos = i * (uint64_t)nbits + (uint64_t)b;
                packed[pos >> 3] |= (uint8_t)(1u << (pos & 7u));
            }
}

void orc_unpack(const uint8_t *packed, uint64_t n, int nbits, uint8_t *codes)
{
    for (uint64_t i = 0; i < n; ++i) {
        uint8_t c = 0;
        for (int b = 0; b < nbits; ++b) {
            uint64_t pos = i * (uint64_t)nbits + (uint64_t)b;
            if ((packed[pos >> 3] >> (pos & 7u)) & 1u) c |= (uint8_t)(1u << b);
        }
        codes[i] = c;
    }
}

/* Counts used by the sparsity checks. */
uint64_t orc_count_zeros(const void *g, uint64_t n, int dtype)
{
    uint64_t z = 0;
    for (uint64_t i = 0; i < n; ++i) z += (elem(g, dtype, i) == 0.0);
    return z;
}

/* ------------------------------------------------------------------ */
/* Appendix "Cosine similarity and heterogeneous stochastic pruning"    */
/* ------------------------------------------------------------------ */

static double Phi(double z) { return 0.5 * erfc(-z / sqrt(2.0)); }

/* Expected cosine of the angle between X and T_{alpha,eps}(X) for
 * X ~ Lognormal(mu, sigma^2) whose logarithm is cut off k standard deviations above
 * its mean (the appendix's three expectations; the lognormal is "truncated": the
 * 0.997 quantile of the data stands in for the cut).  With u = ln(alpha / e^mu):
 *
 *   E[X.T(X)]  = E||X||^2 = n e^{2 s^2} Phi(k - 2 s)                          (a)
 *   E||T(X)||^2 = n alpha e^{s^2/2} Phi((u - s^2)/s)
 *               + n e^{2 s^2} [ Phi(k - 2 s) - Phi((u - 2 s^2)/s) ]           (b)
 *   cos(theta) = (a) / sqrt((a) (b)) = sqrt((a)/(b))
 *
 * written with Phi(z) = 1/2 + 1/2 erf(z/rt2) for the printed erf terms; the scale
 * e^mu cancels, so the formulas are those of the printed mu = 0 case at alpha/e^mu.
 *
 * Reading: the main text writes the cut as erf((k s - 2 s^2)/(s rt2)), i.e. ln x <= k s,
 * while the step-by-step derivation writes ln(k s) in the same place.  The first is
 * taken: k is measured on the data, as mu and sigma are, as a high quantile
 * (0.997: the mass inside three standard deviations of a normal), which is a
 * statement about ln x in units of sigma.  Zeros of the tensor add nothing to any of
 * the three sums.  Requires u <= k s (a threshold above the cut prunes everything).
 */
double orc_cosine_similarity(double u, double sigma, double k)
{
    double s = sigma;
    double top = Phi(k - 2.0 * s);
    double a = exp(2.0 * s * s) * top;
    double b = exp(u + 0.5 * s * s) * Phi((u - s * s) / s)
             + exp(2.0 * s * s) * (top - Phi((u - 2.0 * s * s) / s));
    if (!(b > 0.0)) return 1.0;
    double c = sqrt(a / b);
    return c > 1.0 ? 1.0 : c;
}

/* The largest u (threshold in units of e^mu, log scale) whose expected cosine is
 * still >= min_cos; cos is 1 at u = -inf and falls as u grows.  Bisection on
 * [-(40 s + 50), k s].  If even u = k s keeps the cosine above min_cos, returns k s. */
double orc_threshold_for_cosine(double min_cos, double sigma, double k)
{
    double lo = -(40.0 * sigma + 50.0), hi = k * sigma;
    if (orc_cosine_similarity(hi, sigma, k) >= min_cos) return hi;
    for (int it = 0; it < 300; ++it) {
        double mid = 0.5 * (lo + hi);
        if (mid <= lo || mid >= hi) break;
        if (orc_cosine_similarity(mid, sigma, k) >= min_cos) lo = mid; else hi = mid;
    }
    return lo;
}

/* Inverse of orc_sparsity_of in u, by bisection (the same bracket as orc_threshold). */
static double u_for_sparsity(double Sp, double sigma)
{
    double lo = -(40.0 * sigma + 50.0), hi = 40.0 * sigma + 50.0;
    for (int it = 0; it < 300; ++it) {
        double mid = 0.5 * (lo + hi);
        if (mid <= lo || mid >= hi) break;
        if (orc_sparsity_of(mid, sigma) < Sp) lo = mid; else hi = mid;
    }
    return 0.5 * (lo + hi);
}

/* Heterogeneous allocation (appendix "Heterogeneous algorithm").  Layers are given in
 * backward-pass order, deepest first.  The first n_deep layers carry a floor
 * min_cos[i] on their expected cosine similarity:
 *   - at the overall sparsity S the layer's threshold is u_i (Eq. 8 with the layer's
 *     zero fraction l_i, S' = (S - l_i)/(1 - l_i));
 *   - if cos(u_i) < min_cos[i], the threshold is lowered to the one that reaches
 *     the floor, and the layer's sparsity becomes l_i + (1 - l_i) F(u_i') (Eq. 8);
 *   - otherwise it keeps S.
 * The remaining layers share one level that restores the budget,
 *   S_rest = (S * sum_all n_i - sum_deep n_i S_i) / sum_rest n_i,
 * limited to s_max (the appendix recommends a cap of 0.96-0.98 against over-pruning) and to at
 * least S.  out_S[i] receives every layer's sparsity.  Returns the element-weighted
 * mean sparsity actually allocated (below S when the cap binds). */
double orc_allocate_sparsity(int L, const uint64_t *n, const double *sigma, const double *zero_frac,
                             const double *k, int n_deep, const double *min_cos,
                             double S, double s_max, double *out_S)
{
    double total = 0.0, deep_elems = 0.0, deep_pruned = 0.0;
    for (int i = 0; i < L; ++i) total += (double)n[i];
    for (int i = 0; i < n_deep && i < L; ++i) {
        double l = zero_frac[i], s = sigma[i];
        double Si = S;
        if (s < 1e-6) s = 1e-6;
        if (l < 1.0 && S > l) {
            double Sp = (S - l) / (1.0 - l);
            double u = u_for_sparsity(Sp, s);
            double cap = k[i] * s;
            if (u > cap) u = cap;
            if (orc_cosine_similarity(u, s, k[i]) < min_cos[i]) {
                double u2 = orc_threshold_for_cosine(min_cos[i], s, k[i]);
                Si = l + (1.0 - l) * orc_sparsity_of(u2, s);
                if (Si > S) Si = S;
            }
        }
        out_S[i] = Si;
        deep_elems += (double)n[i];
        deep_pruned += (double)n[i] * Si;
    }
    double rest = total - deep_elems;
    double S_rest = S;
    if (rest > 0.0) {
        S_rest = (S * total - deep_pruned) / rest;
        if (S_rest > s_max) S_rest = s_max;
        if (S_rest < S) S_rest = S;
    }
    double pruned = deep_pruned;
    for (int i = n_deep; i < L; ++i) { out_S[i] = S_rest; pruned += (double)n[i] * S_rest; }
    return total > 0.0 ? pruned / total : 0.0;
}

/* The cut k of a tensor: the q-quantile of ln|g| over the nonzero entries, in standard
 * deviations above the mean, k = (ln|g|_(r) - mu) / sigma with r = ceil(q * nnz) (1-based
 * order statistic).  Also returns the order statistic itself through *value. */
static int cmp_double(const void *a, const void *b)
{
    double x = *(const double *)a, y = *(const double *)b;
    return (x > y) - (x < y);
}

double orc_quantile_k(const void *g, uint64_t n, int dtype, double q, double mu, double sigma, double *value)
{
    double *a = (double *)malloc((n ? n : 1) * sizeof(double));
    uint64_t m = 0;
    for (uint64_t i = 0; i < n; ++i) {
        double x = fabs(elem(g, dtype, i));
        if (x != 0.0) a[m++] = x;
    }
    double v = 0.0;
    if (m) {
        qsort(a, m, sizeof(double), cmp_double);
        uint64_t r = (uint64_t)ceil(q * (double)m);
        if (r < 1) r = 1;
        if (r > m) r = m;
        v = a[r - 1];
    }
    free(a);
    if (value) *value = v;
    return (m && sigma > 0.0) ? (log(v) - mu) / sigma : 0.0;
}

/* ------------------------------------------------------------------ */
/* Appendix "Encoding": prefix code for stochastically pruned tensors   */
/* ------------------------------------------------------------------ */

/* The paper's table gives the code words: 0 -> "0", +alpha -> "100",
 * -alpha -> "101", anything else -> "11" followed by the FP value.  It fixes
 * neither a bit order nor a container, so the stream format is this
 * repository's (the CUDA library states the same format in its header):
 *   - code words are emitted left to right as printed; the FP value follows
 *     "11" as the element's own bit pattern (32 bits fp32, 16 bits bf16),
 *     least-significant bit first;
 *   - stream bit k is bit (k mod 32) of 32-bit word (k div 32);
 *   - elements are taken in index order in blocks of 2048; block b starts at
 *     word off[b], is padded with zero bits to a whole word, and off[nblocks]
 *     is the length of the stream in words;
 *   - "0" is the pattern of +0 only (a -0 travels as an FP value, so that the
 *     code is lossless); the alpha codes exist only when alpha > 0. */
#define ORC_PREFIX_BLOCK 2048u

uint64_t orc_prefix_blocks(uint64_t n) { return (n + ORC_PREFIX_BLOCK - 1) / ORC_PREFIX_BLOCK; }

/* worst case: every element an FP value */
uint64_t orc_prefix_bound_words(uint64_t n, int dtype)
{
    uint64_t per = (dtype == ORC_BF16 ? 16u : 32u) + 2u;
    uint64_t full = n / ORC_PREFIX_BLOCK, rest = n % ORC_PREFIX_BLOCK;
    return full * ((ORC_PREFIX_BLOCK * per + 31) / 32) + (rest * per + 31) / 32;
}

static uint32_t pattern_of(const void *v, int dtype, uint64_t i)
{
    if (dtype == ORC_BF16) return ((const uint16_t *)v)[i];
    uint32_t w; memcpy(&w, (const float *)v + i, sizeof w); return w;
}

static uint32_t tau_pattern(double tau_used, int dtype)
{
    float f = (float)tau_used; uint32_t w; memcpy(&w, &f, sizeof w);
    return dtype == ORC_BF16 ? (w >> 16) : w;
}

/* 0: zero, 1: +alpha, 2: -alpha, 3: FP value */
int orc_prefix_class(uint32_t pattern, int dtype, double tau_used)
{
    uint32_t sign = dtype == ORC_BF16 ? 0x8000u : 0x80000000u;
    if (pattern == 0u) return 0;
    if (tau_used > 0.0 && (pattern & ~sign) == tau_pattern(tau_used, dtype)) return (pattern & sign) ? 2 : 1;
    return 3;
}

static void put_bit(uint32_t *stream, uint64_t *pos, int bit)
{
    if (bit) stream[*pos >> 5] |= 1u << (*pos & 31);
    ++*pos;
}

static int get_bit(const uint32_t *stream, uint64_t *pos)
{
    int b = (stream[*pos >> 5] >> (*pos & 31)) & 1u;
    ++*pos;
    return b;
}

/* stream must hold orc_prefix_bound_words(n) zero-initialised words; off holds nblocks+1 entries.
 * Returns the stream length in words. */
uint64_t orc_prefix_encode(const void *v, uint64_t n, int dtype, double tau_used,
                           uint32_t *stream, uint64_t *off)
{
    int width = dtype == ORC_BF16 ? 16 : 32;
    uint64_t pos = 0, b = 0;
    for (uint64_t i = 0; i < n; ++i) {
        if (i % ORC_PREFIX_BLOCK == 0) {
            pos = (pos + 31) / 32 * 32;            /* pad the previous block to a whole word */
            off[b++] = pos / 32;
        }
        uint32_t p = pattern_of(v, dtype, i);
        switch (orc_prefix_class(p, dtype, tau_used)) {
        case 0: put_bit(stream, &pos, 0); break;
        case 1: put_bit(stream, &pos, 1); put_bit(stream, &pos, 0); put_bit(stream, &pos, 0); break;
        case 2: put_bit(stream, &pos, 1); put_bit(stream, &pos, 0); put_bit(stream, &pos, 1); break;
        default:
            put_bit(stream, &pos, 1); put_bit(stream, &pos, 1);
            for (int k = 0; k < width; ++k) put_bit(stream, &pos, (p >> k) & 1u);
        }
    }
    pos = (pos + 31) / 32 * 32;
    off[b] = pos / 32;
    return pos / 32;
}

void orc_prefix_decode(const uint32_t *stream, const uint64_t *off, uint64_t n, int dtype,
                       double tau_used, void *out)
{
    int width = dtype == ORC_BF16 ? 16 : 32;
    uint32_t sign = dtype == ORC_BF16 ? 0x8000u : 0x80000000u;
    uint32_t tp = tau_pattern(tau_used, dtype);
    uint64_t pos = 0;
    for (uint64_t i = 0; i < n; ++i) {
        if (i % ORC_PREFIX_BLOCK == 0) pos = off[i / ORC_PREFIX_BLOCK] * 32;
        uint32_t p;
        if (!get_bit(stream, &pos)) p = 0u;
        else if (!get_bit(stream, &pos)) p = get_bit(stream, &pos) ? (tp | sign) : tp;
        else { p = 0u; for (int k = 0; k < width; ++k) p |= (uint32_t)get_bit(stream, &pos) << k; }
        if (dtype == ORC_BF16) ((uint16_t *)out)[i] = (uint16_t)p;
        else memcpy((float *)out + i, &p, sizeof p);
    }
}

/* ------------------------------------------------------------------ */
/* Algorithm 1, last step: the tensor a packed code stream stands for   */
/* ------------------------------------------------------------------ */

/* X_Q = 2^e_s * Q_FP(.) for every element of a packed stream: code i is bits
 * [i*nbits, (i+1)*nbits) of the little-endian bit stream (orc_pack), decoded by
 * orc_decode and stored in the output type.  Every decoded value has at most 7
 * significant bits, so fp32 and bf16 hold it exactly whenever its exponent is in
 * their normal range; the caller keeps formats inside that range. */
void orc_dequantize(const uint8_t *packed, uint64_t n, int nbits, int n2, int n1, int e_s,
                    int out_dtype, void *out)
{
    for (uint64_t i = 0; i < n; ++i) {
        uint32_t code = 0;
        for (int b = 0; b < nbits; ++b) {
            uint64_t bit = i * (uint64_t)nbits + (uint64_t)b;
            code |= (uint32_t)((packed[bit >> 3] >> (bit & 7)) & 1u) << b;
        }
        store_elem(out, out_dtype, i, orc_decode(code, n2, n1, e_s));
    }
}
