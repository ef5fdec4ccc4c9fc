// Interval arithmetic of one code given its softmax probability and the row's radius, shared by
// the general quantifier, the discrete top-k quantifier and the ensemble quantifier.
#pragma once

#include "ciar_device.cuh"

namespace ciar {

// Radius of a whole row as interval constants: a = exp(-r), b = exp(r), alpha = 1 - a,
// beta = b - 1, bma = b - a (all from double so that tiny radii keep their digits).
struct RadiusConst {
    float a, alpha, beta, bma;
};

__device__ __forceinline__ double clamp_radius(double rho, int raw, double r_max)
{
    double r = rho;
    if (raw) r = (rho > 0.0) ? rho + log1p(exp(-rho)) : log1p(exp(rho));  // Softplus, beta = 1
    return r > r_max ? r_max : r;
}

__device__ __forceinline__ RadiusConst radius_const(double r)
{
    RadiusConst k;
    const double al = -expm1(-r), be = expm1(r);
    k.a = (float)(1.0 - al);
    k.alpha = (float)al;
    k.beta = (float)be;
    k.bma = (float)(al + be);
    return k;
}

// One code's bounds from its softmax probability p (InterFuse with the max-trick, rewritten in p):
//   p^l = a p / (1 - alpha p),  p^u = b p / (1 + beta p),
//   d = p^u - p^l = p (b - a)(1 - p) / ((1 - alpha p)(1 + beta p))   -- no cancellation for small r.
__device__ __forceinline__ void bounds_from_p(float p, const RadiusConst &k, float &pl, float &d)
{
    const float den_l = fmaf(-k.alpha, p, 1.0f);
    const float den_u = fmaf(k.beta, p, 1.0f);
    const float q = __fdividef(p, den_l * den_u);
    pl = k.a * (q * den_u);
    d = k.bma * (q * (1.0f - p));
}

// The same with 1 - p given by the caller (formed from the other codes' sum when p is close to 1).
__device__ __forceinline__ void bounds_from_p_omp(float p, float omp, const RadiusConst &k, float &pl, float &d)
{
    const float den_l = fmaf(-k.alpha, p, 1.0f);
    const float den_u = fmaf(k.beta, p, 1.0f);
    const float q = __fdividef(p, den_l * den_u);
    pl = k.a * (q * den_u);
    d = k.bma * (q * omp);
}

// Normalisation step and score from the raw interval sums of n codes (interval appendix, the two scaling
// equations; uncertainty-score equation): A = sum d, B = sum p^l, AA = sum d^2, AB = sum d p^l, BB = sum (p^l)^2.
struct ScoreParts {
    double S_lo, S_up, k_lo, k_up, g, omega, mu, var;
};

__device__ __forceinline__ ScoreParts score_parts(double A, double B, double AA, double AB, double BB, double nn,
                                                  double lo_cap, double hi_cap)
{
    ScoreParts s;
    s.S_lo = B;
    s.S_up = A + B;
    s.k_lo = 1.0;
    s.k_up = 1.0;
    if (s.S_lo > 0.0 && lo_cap / s.S_lo < 1.0) s.k_lo = lo_cap / s.S_lo;
    if (s.S_up > 0.0 && hi_cap / s.S_up > 1.0) s.k_up = hi_cap / s.S_up;
    s.g = s.k_up - s.k_lo;  // delta_i = k_up d_i + g p^l_i, every term >= 0
    s.omega = s.k_up * A + s.g * B;
    s.mu = s.omega / nn;
    s.var = (s.k_up * s.k_up * AA + 2.0 * s.k_up * s.g * AB + s.g * s.g * BB) / nn - s.mu * s.mu;
    return s;
}

}  // namespace ciar
