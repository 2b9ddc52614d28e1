// The per-position verdict shared by every kernel that folds a sequence: exact power-of-two
// rescaling of partial sums, 2^x in float64, and the acceptance test itself.
#pragma once

#include <math.h>

#include "dssd_device.cuh"

namespace dssd {

constexpr unsigned kBitAccept = 1u, kBitBadToken = 2u, kBitNonFinite = 4u, kBitTimeout = 8u;

// v * 2^d for an integer d <= 0 and a normal, positive v of float32 range: exponent arithmetic,
// exact; anything below 2^-900 of v counts as nothing
__device__ __forceinline__ double scale_pow2(double v, float d)
{
    if (!(d > -900.f)) return 0.0;
    return __hiloint2double(__double2hiint(v) + ((int)d << 20), __double2loint(v));
}

// 2^x in float64 for x <= about 1 (relative error below 1e-11): x = n + f, |f| <= 1/2, and the
// degree-9 Taylor polynomial of e^(f ln 2); 0 below 2^-1000, NaN for NaN
__device__ __forceinline__ double exp2_small(double x)
{
    if (x != x) return x;
    if (!(x > -1000.0)) return 0.0;
    const int n = __double2int_rn(x);
    const double y = (x - (double)n) * 0.6931471805599453;
    double p = 2.7557319223985893e-6;
    p = fma(p, y, 2.48015873015873e-5);
    p = fma(p, y, 1.984126984126984e-4);
    p = fma(p, y, 1.388888888888889e-3);
    p = fma(p, y, 8.333333333333333e-3);
    p = fma(p, y, 4.1666666666666664e-2);
    p = fma(p, y, 1.6666666666666666e-1);
    p = fma(p, y, 0.5);
    p = fma(p, y, 1.0);
    p = fma(p, y, 1.0);
    return __hiloint2double(__double2hiint(p) + (n << 20), __double2loint(p));
}

// One position i of sequence b, given its row's sum_v 2^(l_v * c1) = S * 2^Rr (float64 S, integer
// Rr): writes lse and p_i(x_i), evaluates the acceptance test and returns the position's bits;
// Rs, invS are what the emission of this row would need.  A lane that is not live returns "accepted".
template <class Params>
__device__ __forceinline__ unsigned judge_position(const Params &P, long long b, int i, bool live, float Rr, double S,
                                                   bool bad, bool timeout, int x, float zx, float qx, float ux,
                                                   float &Rs, float &invS)
{
    const double c1 = (double)P.c1;
    // the sum has a finite logarithm iff S is positive and finite
    const bool finite = !timeout && !bad && (S > 0.0) && (S < INFINITY) && (Rr != DSSD_NEG_INF);
    unsigned bits = live ? ((finite ? 0u : kBitNonFinite) | (timeout ? kBitTimeout : 0u)) : kBitAccept;
    if (live && P.lse)
        P.lse[b * (P.gamma + 1) + i] = finite ? (Rr + __log2f((float)S)) * 0.6931471805599453f : __int_as_float(0x7fc00000);
    // 1 / S in float64: the float32 reciprocal refined by one Newton step
    double invS_d = NAN;
    if (finite) {
        const double r0 = (double)(1.0f / (float)S);
        invS_d = r0 * (2.0 - S * r0);
    }
    if (live && i < P.gamma) {
        double p = NAN;
        bool accept = false;
        if (x < 0 || x >= P.V) {
            bits |= kBitBadToken;
        } else {
            // u < min(1, p(x)/q(x)) in float64, as  u < 1  and  u * q < p  (u * q is exact)
            p = finite ? exp2_small((double)zx * c1 - (double)Rr) * invS_d : NAN;
            const double q = (double)qx;
            const double u = (double)ux;
            if (q != q || p != p) accept = false;
            else if (q <= 0.0) accept = (p > 0.0) && (u < 1.0);
            else accept = (u < 1.0) && (u * q < p);
        }
        if (P.p_tok) P.p_tok[(size_t)b * P.gamma + i] = (float)p;
        bits |= accept ? kBitAccept : 0u;
    }
    invS = finite ? (float)invS_d : __int_as_float(0x7fc00000);
    Rs = finite ? Rr : 0.f;
    return bits;
}

// (Rr, S) += a partial (pr, ps): sum_v 2^(l_v c1) = S * 2^Rr with S kept relative to the largest
// reference seen so far; partials without mass are skipped, a NaN partial marks the row
__device__ __forceinline__ void add_partial(float &Rr, double &S, bool &bad, float pr, double ps)
{
    if (ps != ps) bad = true;
    if (ps > 0.0) {
        if (pr > Rr) {
            S = (Rr == DSSD_NEG_INF || S == 0.0) ? 0.0 : scale_pow2(S, Rr - pr);
            Rr = pr;
        }
        S += scale_pow2(ps, pr - Rr);
    }
}

}  // namespace dssd
