// Shared pieces of the half-precision prefilter (score_select_f16.cu, f16_convert.cu, refine_f16.cu):
// the per-head statistics, the power-of-two scaling of the fp16 operand copies and the error bound of
// an fp16-accumulated tensor-core score.
#pragma once

#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

namespace kmip {

// Groups kept per row by the prefilter sweep for 16 < k <= 32 (k + slack, a multiple of 8); the sweep's pending
// slots take the shared memory the list leaves.
#ifndef KMIP_F16_LIST32
#define KMIP_F16_LIST32 48
#endif
constexpr int kF16List32 = KMIP_F16_LIST32;

// Per head: largest squared norm of a query row, of a key row, and of the first 16 elements of a key
// row (the partial sum after the first tensor-core step of a 32-wide head); float bits, maxima taken
// with integer atomics (the values are non-negative).
struct F16HeadStat {
    float q_n2max;
    float k_n2max;
    float k_first16_n2max;
    float pad;
};

// Power of two s such that s * sqrt(n2max) lies in [32, 64) (up to the rounding of the square root):
// products of two scaled rows stay below 4096 < 65504, and elements lose bits only below 2^-14.
__host__ __device__ inline float f16_scale_from_n2max(float n2max) {
    if (!(n2max > 0.0f) || !(n2max < 3.0e38f)) return 1.0f;
    int e = 0;
    frexpf(sqrtf(n2max), &e);  // sqrt = m * 2^e, m in [0.5, 1)
    int se = 6 - e;
    se = se < -60 ? -60 : (se > 60 ? 60 : se);
    return ldexpf(1.0f, se);
}

// |fp16 score T - exact scaled score| <= a + r * |T| for every key of the head, given the row's scaled
// norms.  The tensor cores round the fp16 accumulator to nearest once per 16-deep step: the last
// rounding is at most 2^-11 |T|, the one before (32-wide heads) at most 2^-11 times the partial sum,
// itself at most |q[0:16]| |k[0:16]|.  2^-18 |q||k| covers the internal summation, 2.5e-5 the elements
// that underflowed in the conversion (scaled norms are below 64) and subnormal results.
constexpr float kF16RelErr = 4.8923e-4f;  // 2^-11 (1 + 2^-9)
__host__ __device__ inline float f16_abs_err(int ksteps, float nq_first16, float nk_first16_max, float nq, float nk_max) {
    return (ksteps > 1 ? kF16RelErr * nq_first16 * nk_first16_max : 0.0f) + 3.8147e-6f * nq * nk_max + 2.5e-5f;
}

}  // namespace kmip
