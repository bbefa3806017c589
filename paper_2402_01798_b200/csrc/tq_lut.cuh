// The decision table of the bf16 compress kernels: what both compress files need to agree on which rows it serves.
#pragma once
#include <stdint.h>

#include "tq.h"

namespace tq {

constexpr int kLutMaxEntries = 8192;     // per sign: 64 binades
constexpr int kLutMinEntries = 2048;

// X = k * 2^16 + min(T, 2^16) for a gradient value g: the decision of the quantizer equation up to the
// random draw.  One IEEE operation per step (the build disables contraction on both sides), so host and
// device agree bit for bit.
__host__ __device__ inline uint32_t decision_x(float g, float alpha, const float* levels, const float* inv_width,
                                               uint32_t num_levels) {
    const uint32_t s = num_levels - 1;
    const float t = fminf(fmaxf(g, -alpha), alpha);          // NaN -> -alpha, +-Inf -> +-alpha
    uint32_t k = 0;
    for (uint32_t j = 1; j + 1 <= s; ++j)                     // largest j <= s - 1 with l_j <= t
        if (levels[j] <= t) k = j;
    const float p = (t - levels[k]) * inv_width[k];
    const float tf = p * 65536.0f;
    const uint32_t T = !(tf > 0.0f) ? 0u : (tf >= 65536.0f ? 65536u : static_cast<uint32_t>(rintf(tf)));
    return k * 65536u + T;
}

__host__ __device__ inline float bf16_pattern_value(uint32_t pattern16) {
#ifdef __CUDA_ARCH__
    return __uint_as_float(pattern16 << 16);
#else
    union { uint32_t u; float f; } c;
    c.u = pattern16 << 16;
    return c.f;
#endif
}

// Smallest bf16 pattern whose value is >= alpha (alpha positive and finite); at most 0x7F80 (+Inf).
__host__ __device__ inline uint32_t top_pattern(float alpha) {
#ifdef __CUDA_ARCH__
    const uint32_t u = __float_as_uint(alpha);
#else
    union { float f; uint32_t u; } c;
    c.f = alpha;
    const uint32_t u = c.u;
#endif
    uint32_t p = u >> 16;
    if ((p << 16) < u) ++p;
    return p;
}

// Whether a window of n entries per sign below `top` serves the quantizer: either it reaches down to zero, or the
// decision at +-base equals that of everything smaller (it is monotone in the value).  *base receives the window's
// first pattern.
__host__ __device__ inline bool lut_window_fits(float alpha, const float* levels, const float* inv_width, uint32_t num_levels,
                                                uint32_t top, uint32_t n, uint32_t* base) {
    if (top < n) { *base = 0; return true; }
    *base = top - (n - 1);
    return decision_x(bf16_pattern_value(*base | 0x8000u), alpha, levels, inv_width, num_levels) ==
           decision_x(bf16_pattern_value(*base), alpha, levels, inv_width, num_levels);
}

// Device-resident parameters: a row goes through the table kernel when its record is usable and the largest window
// serves it; the element-wise kernels evaluate the same rule and leave exactly those rows alone.
__host__ __device__ inline bool lut_serves_record(const tq_params_t& p, uint32_t bits, uint32_t* top, uint32_t* base) {
    if (!(p.alpha > 0.0f) || !(p.alpha <= 3.402823466e38f) || p.bits != bits || (p.flags & TQ_FLAG_INVALID)) return false;
    *top = top_pattern(p.alpha);
    return lut_window_fits(p.alpha, p.levels, p.inv_width, 1u << bits, *top, kLutMaxEntries, base);
}

}  // namespace tq
