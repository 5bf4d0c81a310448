// GELU (u Phi(u), erf form) and its derivative as the projection epilogues and the stand-alone kernel evaluate them.
#pragma once
#include "sm100_ptx.cuh"

namespace mpipe {

// erf by the rational-times-Gaussian form of Abramowitz & Stegun 7.1.26 (|error| <= 1.5e-7, far below the bf16
// rounding of the result): two special-function ops and a degree-5 Horner chain instead of the library routine's branches.
__device__ __forceinline__ float erf_as(float x) {
    const float ax = fabsf(x);
    float t;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t) : "f"(fmaf(0.3275911f, ax, 1.0f)));
    float p = fmaf(1.061405429f, t, -1.453152027f);
    p = fmaf(p, t, 1.421413741f);
    p = fmaf(p, t, -0.284496736f);
    p = fmaf(p, t, 0.254829592f);
    p *= t;
    const float e = ex2_approx(-ax * ax * 1.4426950408889634f);
    return copysignf(1.0f - p * e, x);
}
__device__ __forceinline__ float gelu_erf(float u) { return 0.5f * u * (1.0f + erf_as(u * 0.7071067811865476f)); }
// d/du [u Phi(u)] = Phi(u) + u phi(u), phi the standard normal density
__device__ __forceinline__ float gelu_erf_grad(float u) {
    const float cdf = 0.5f * (1.0f + erf_as(u * 0.7071067811865476f));
    const float pdf = 0.3989422804014327f * ex2_approx(-0.5f * u * u * 1.4426950408889634f);
    return fmaf(u, pdf, cdf);
}

}  // namespace mpipe
