// Closed forms of the lognormal model, usable from host and device code.
//
//   pruned_fraction / solve_threshold : Eq. 8 (sparsity of stochastic pruning
//       as a function of the threshold) and its numerical inverse
//   expected_rel_err / choose_format  : Eq. 4 and its minimiser
//   snap_threshold_*                  : the threshold in the tensor's type
#pragma once

#include <cfloat>
#include <cmath>
#include <cstdint>
#include <cstring>

#include "lgn.h"

#if defined(__CUDACC__)
#define LGN_HD __host__ __device__ __forceinline__
#else
#define LGN_HD inline
#endif

namespace lgn {

constexpr double kLn2      = 0.693147180559945309417232121458;
constexpr double kInvSqrt2 = 0.707106781186547524400844362105;
constexpr double kSigmaMin = 1e-6;
constexpr double kSigmaMax = 25.0;

LGN_HD double clamp_sigma(double s) {
    if (!(s >= kSigmaMin)) s = kSigmaMin;
    if (s > kSigmaMax) s = kSigmaMax;
    return s;
}

LGN_HD double normal_cdf(double z) { return 0.5 * erfc(-z * kInvSqrt2); }

// Eq. 8 in the variable u = ln(alpha / e^mu).  Writing Phi for the standard
// normal CDF, the printed expression collapses to
//     F(u) = Phi(u/s) - e^{s^2/2 - u} Phi((u - s^2)/s),
// the CDF of s*N(0,1) + Exp(1) (ln of the magnitude minus ln of eps), whose
// density is the subtracted term itself.  That term is evaluated as
// exp(s^2/2 - u + ln Phi(.)) so that a huge exponential never meets a
// vanishing Phi.
LGN_HD void pruned_fraction(double u, double s, double &F, double &dF) {
    const double a = normal_cdf(u / s);
    const double pv = normal_cdf((u - s * s) / s);
    const double ex = 0.5 * s * s - u;
    double b;
    if (ex < 600.0) b = exp(ex) * pv;                      // no overflow possible: plain product
    else            b = pv > 0.0 ? exp(ex + log(pv)) : 0.0;
    F = a - b;
    dF = b;
}

// Solve F(u) = Sp for u: Newton steps kept inside a shrinking bracket
// (bisection whenever a step would leave it).  Sp in (0,1).  Once two Newton
// steps in a row shrink by more than 1000x and the last is below 1e-8, the
// iteration is in its quadratic regime and the iterate that follows is exact to
// fp64 rounding (error <= 1e-3 * 1e-3 * 1e-8), so no evaluation is spent on
// confirming it.  In the far tails (Sp within 1e-4 of 0 or 1), where F - Sp
// itself carries few significant digits, and anywhere else, it runs until the
// step vanishes.
LGN_HD double solve_threshold_u(double s, double Sp) {
    double lo = -(40.0 * s + 50.0), hi = 40.0 * s + 50.0;
    // start from the logistic approximation of the normal quantile, shifted
    // by the mean of -ln(eps)
    double q = Sp / (1.0 - Sp);
    double u = (q > 0.0 && q < 1e300) ? s * log(q) * 0.5875 + 1.0 : 0.0;
    if (!(u > lo && u < hi)) u = 0.0;
    const bool well_conditioned = Sp >= 1e-4 && Sp <= 1.0 - 1e-4;
    // A few Newton steps in fp32 first (an fp32 erfc costs a tenth of an fp64 one): they bring
    // the start to within about 1e-5 of the root, so the fp64 iteration below needs two or
    // three evaluations instead of five or six.  Only a better starting point: every decision
    // about the result is taken in fp64.
    if (Sp >= 1e-3 && Sp <= 1.0 - 1e-3 && s >= 0.05 && s <= 8.0) {
        float uf = (float)u;
        const float sf = (float)s, target = (float)Sp;
        for (int it = 0; it < 4; ++it) {
            const float ex = 0.5f * sf * sf - uf;
            if (!(ex < 60.0f)) break;
            const float a = 0.5f * erfcf(-uf / sf * 0.70710678f);
            const float b = expf(ex) * 0.5f * erfcf(-(uf - sf * sf) / sf * 0.70710678f);
            if (!(b > 1e-20f)) break;
            const float un = uf - (a - b - target) / b;
            if (!(un > (float)lo && un < (float)hi)) break;
            uf = un;
        }
        if (uf > (float)lo && uf < (float)hi) u = (double)uf;
    }
    double prev_step = 1e300;
    bool prev_newton = false;
    for (int it = 0; it < 200; ++it) {
        double F, dF;
        pruned_fraction(u, s, F, dF);
        if (F < Sp) lo = u; else hi = u;
        double un = u - (F - Sp) / dF;
        const bool newton = un > lo && un < hi;
        if (!newton) un = 0.5 * (lo + hi);
        const double step = fabs(un - u);
        const double scale = fmax(1.0, fabs(un));
        u = un;
        if (well_conditioned && newton && prev_newton && step <= 1e-8 * scale && step <= 1e-3 * prev_step) break;
        if (step <= 4e-16 * scale || !(hi > lo)) break;
        prev_step = step;
        prev_newton = newton;
    }
    return u;
}

// Appendix A.9 steps (1),(2) + Eq. 8: threshold for output sparsity S when a
// fraction l of the tensor is already zero.
LGN_HD double threshold_for(double mu, double sigma, double l, double S) {
    if (!(l < 1.0)) return 0.0;
    double Sp = (S - l) / (1.0 - l);
    if (!(Sp > 0.0)) return 0.0;
    double s = clamp_sigma(sigma);
    return exp(mu + solve_threshold_u(s, Sp));
}

// Expected cosine similarity between X and its stochastically pruned copy
// (appendix "Cosine similarity of stochastic pruning"), for ln X ~ N(mu, s^2) cut
// off k standard deviations above the mean, at threshold e^(mu+u), u <= k s:
//     cos^2 = A / B,   A = e^{2 s^2} Phi(k - 2 s)                       (= E[X.T(X)] = E|X|^2)
//                      B = e^{u + s^2/2} Phi((u - s^2)/s) + A - e^{2 s^2} Phi((u - 2 s^2)/s)
// Dividing by e^{2 s^2}: B/e^{2s^2} = P + e^{u - 3 s^2/2} Phi((u - s^2)/s) - Phi((u - 2 s^2)/s)
// with P = Phi(k - 2 s); dB/du = e^{u + s^2/2} Phi((u - s^2)/s) (the two density terms cancel).
LGN_HD void cosine_terms(double u, double s, double k, double &ratio, double &dratio) {
    const double P = normal_cdf(k - 2.0 * s);
    const double g = exp(u - 1.5 * s * s) * normal_cdf((u - s * s) / s);   // also d/du of the bracket
    const double b = P + g - normal_cdf((u - 2.0 * s * s) / s);
    ratio = b > 0.0 ? P / b : 1.0;                                          // cos^2
    dratio = b > 0.0 ? -P * g / (b * b) : 0.0;
}

LGN_HD double cosine_similarity_of(double u, double s, double k) {
    double r, dr;
    cosine_terms(u, s, k, r, dr);
    return r >= 1.0 ? 1.0 : sqrt(r);
}

// Largest u <= k s with cosine >= min_cos: Newton on cos^2(u) = min_cos^2 inside a
// shrinking bracket (cos falls monotonically in u), bisection when a step leaves it.
LGN_HD double threshold_u_for_cosine(double min_cos, double s, double k) {
    double hi = k * s, lo = -(40.0 * s + 50.0);
    if (cosine_similarity_of(hi, s, k) >= min_cos) return hi;
    const double target = min_cos * min_cos;
    double u = hi - s;
    if (!(u > lo)) u = 0.5 * (lo + hi);
    for (int it = 0; it < 200; ++it) {
        double r, dr;
        cosine_terms(u, s, k, r, dr);
        if (r >= target) lo = u; else hi = u;
        double un = dr < 0.0 ? u - (r - target) / dr : lo;
        if (!(un > lo && un < hi)) un = 0.5 * (lo + hi);
        const double step = fabs(un - u);
        u = un;
        if (step <= 4e-16 * fmax(1.0, fabs(u)) || !(hi > lo)) break;
    }
    // the answer must satisfy the floor: if rounding put the iterate just past the root,
    // walk it back by a few units in the last place (doubling), else fall back on the bracket
    double back = 2.2e-16 * fmax(1.0, fabs(u));
    for (int j = 0; j < 12 && cosine_similarity_of(u, s, k) < min_cos; ++j, back *= 2.0) u -= back;
    return cosine_similarity_of(u, s, k) >= min_cos ? u : lo;
}

LGN_HD float snap_threshold_f32(double tau) {
    float f = (float)tau;                       // round to nearest even
    if (!(f <= FLT_MAX)) f = FLT_MAX;
    return f;
}

LGN_HD float snap_threshold_bf16(double tau) {
    float f = snap_threshold_f32(tau);
    uint32_t w;
    memcpy(&w, &f, 4);
    w += 0x7FFFu + ((w >> 16) & 1u);            // round the low half away, ties to even
    w &= 0xFFFF0000u;
    if (w >= 0x7F800000u) w = 0x7F7F0000u;      // largest finite bfloat16
    memcpy(&f, &w, 4);
    return f;
}

// Eq. 4 with n1 mantissa / n2 exponent bits.  The exponent of Eq. 1 is base 2,
// so the normal law of the derivation has standard deviation sigma/ln 2; in
// terms of the natural-log sigma, E_max/(sigma/ln 2) = c and (sigma/ln 2) ln 2
// = sigma.  Mantissa step 2^-n1.
LGN_HD double expected_rel_err(double sigma, int n1, int n2) {
    double Emax = (double)(1 << (n2 - 1));
    double c = Emax * kLn2 / sigma;
    double in_range = 2.0 * normal_cdf(c) - 1.0;
    double t1 = in_range * exp2((double)-n1) / (8.0 * kLn2);
    double ez = erfc((sigma + c) * kInvSqrt2);
    double t2 = ez > 0.0 ? -exp((Emax - 1.0) * kLn2 + 0.5 * sigma * sigma + log(ez)) : 0.0;
    double t3 = erfc(c * kInvSqrt2);
    return t1 + t2 + t3;
}

LGN_HD void choose_format(double mu, double sigma, int nbits, lgn_fp_format_t &f) {
    double s = clamp_sigma(sigma);
    int best = 1;
    double best_eta = expected_rel_err(s, nbits - 2, 1);
    for (int n2 = 2; n2 <= nbits - 1; ++n2) {
        double eta = expected_rel_err(s, nbits - 1 - n2, n2);
        if (eta < best_eta) { best_eta = eta; best = n2; }
    }
    f.nbits = nbits;
    f.exp_bits = best;
    f.man_bits = nbits - 1 - best;
    f.scale_exp = (int32_t)floor(mu / kLn2 + 0.5);
}

}  // namespace lgn
