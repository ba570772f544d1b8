// Single-pass softmax statistics and their merge (device side only).
//
// For a set S of logits the kernels carry
//     m = max z,   s = sum e^{z-m},   u = sum e^{z-m} (z-m),   (bv, bi) = greedy token
// from which the entropy of Eq. 1 (in nats) is  H = ln s - u / s.
// Two disjoint sets merge with M = max(m1, m2), a_i = e^{m_i - M}:
//     s = a1 s1 + a2 s2,   u = a1 (u1 + (m1 - M) s1) + a2 (u2 + (m2 - M) s2).
// The empty set is (m = -inf, s = 0, u = 0) and never produces inf - inf.
#pragma once
#include <cuda_runtime.h>
#include <math_constants.h>
#include <limits.h>

namespace rstitch {

// e^x and ln x on the special-function unit, asked for by name: ex2.approx / lg2.approx with the
// flush-to-zero form (a softmax term below 2^-126 adds nothing to an fp32 sum).  Relative error about
// 2^-22; the library is built without fast-math flags, so nothing else is approximate.
__device__ __forceinline__ float exp_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x * 1.4426950408889634f));
    return y;
}

__device__ __forceinline__ float log_approx(float x)
{
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y * 0.6931471805599453f;
}

struct Stats {
    float m, s, u, bv;
    int   bi;
};

__device__ __forceinline__ Stats stats_empty()
{
    Stats t;
    t.m = -CUDART_INF_F; t.s = 0.f; t.u = 0.f; t.bv = -CUDART_INF_F; t.bi = INT_MAX;
    return t;
}

// Greedy token order: larger logit first, lower vocabulary index on ties.  NaN never wins.
__device__ __forceinline__ void argmax_take(float &bv, int &bi, float v, int i)
{
    if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
}

// Add one logit; `score` is what the token choice maximises (the logit itself for the greedy
// token, the logit over the temperature plus Gumbel noise for a sampled one).
__device__ __forceinline__ void stats_push(Stats &t, float z, int idx, float score)
{
    if (z == z) argmax_take(t.bv, t.bi, score, idx);      // a NaN logit never wins
    float mn = fmaxf(t.m, z);                       // fmaxf ignores a NaN operand
    float dm = (t.m == -CUDART_INF_F) ? 0.f : (t.m - mn);
    float a  = exp_approx(dm);
    float dz = z - mn;
    float e  = exp_approx(dz);                          // NaN logit -> e = NaN -> s = NaN
    t.u = a * (t.u + dm * t.s) + e * dz;
    t.s = a * t.s + e;
    t.m = mn;
}

__device__ __forceinline__ void stats_push(Stats &t, float z, int idx) { stats_push(t, z, idx, z); }

// Merge b into a (a is the set with the lower vocabulary indices only by convention; the argmax
// comparison is order-independent).
__device__ __forceinline__ void stats_merge(Stats &a, const Stats &b)
{
    argmax_take(a.bv, a.bi, b.bv, b.bi);
    float M  = fmaxf(a.m, b.m);
    float da = (a.m == -CUDART_INF_F) ? 0.f : (a.m - M);
    float db = (b.m == -CUDART_INF_F) ? 0.f : (b.m - M);
    float ea = (a.m == -CUDART_INF_F) ? 0.f : exp_approx(da);
    float eb = (b.m == -CUDART_INF_F) ? 0.f : exp_approx(db);
    float s  = ea * a.s + eb * b.s;
    float u  = ea * (a.u + da * a.s) + eb * (b.u + db * b.s);
    a.m = M; a.s = s; a.u = u;
}

}  // namespace rstitch
