// Shared host/device helpers of the tdq CUDA library (not used by the CPU oracle).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <cmath>

#include "../../include/tdq.h"

namespace tdq {

// Numerical conventions of Supp. S4.8.
constexpr float kClipFloor = 1e-8f;   // every clip radius is at least this
constexpr float kStepFloor = 1e-8f;   // Delta = max(c / q_max, 1e-8)
constexpr float kStdEps = 1e-12f;     // sigma = Std + 1e-12
constexpr float kQmax = 7.0f;
// 1.5 * 2^23: adding it to |v| < 2^22 rounds v to the nearest integer, ties to even, and
// leaves that integer in the low mantissa bits as a two's complement offset.
constexpr float kRoundMagic = 12582912.0f;

extern std::atomic<uint64_t> g_launch_count;

inline tdq_status cuda_status(cudaError_t e) { return e == cudaSuccess ? TDQ_OK : TDQ_ERR_CUDA; }

// Rank ceil(frac * g), 1-indexed, inside [1, g] (Supp. S2.2).  frac is a float, so a
// product within 1e-6 of an integer counts as that integer.
inline int32_t rank_of(float frac, int32_t g) {
    const double kd = (double)frac * (double)g;
    const double kr = std::floor(kd + 0.5);
    int64_t k = (std::fabs(kd - kr) < 1e-6) ? (int64_t)kr : (int64_t)std::ceil(kd);
    if (k < 1) k = 1;
    if (k > g) k = g;
    return (int32_t)k;
}

__device__ __forceinline__ float bf16_bits_to_float(uint32_t hi16) { return __uint_as_float(hi16 << 16); }

// DCRP, Eq. 12 with the floors of Supp. S4.8, in the binary32 order the paper writes:
// c first, then Delta = c / q_max.  No multiply-add may be fused here.
__device__ __forceinline__ void dcrp_project(float c_base, float sigma, float thr, float seven_tau,
                                             uint32_t flags, float& c, float& delta) {
    float cc = c_base;
    if (flags & TDQ_ENABLE_C1) cc = fminf(cc, __fmul_rn(seven_tau, sigma));
    if (flags & TDQ_ENABLE_C2) cc = fminf(cc, __fmul_rn(14.0f, thr));
    cc = fmaxf(cc, kClipFloor);
    c = cc;
    delta = fmaxf(__fdiv_rn(cc, kQmax), kStepFloor);
}

// One element of Alg. S1 steps 5 and 7 with a true IEEE division; returns the code.
__device__ __forceinline__ int quantize_ieee(float x, float c, float delta) {
    float xt = fminf(fmaxf(x, -c), c);
    float r = __fdiv_rn(xt, delta);
    int q = __float2int_rn(r);
    return max(-8, min(7, q));
}

}  // namespace tdq
