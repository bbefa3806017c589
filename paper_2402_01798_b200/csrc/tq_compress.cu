// Client side of Algorithm 1: truncate (Section 3.1, truncation equation), stochastically round onto
// the codebook (Section 3.1, quantizer equation) and pack b-bit codes, fused in one pass.
//
// Work split: a thread owns a run of 32 consecutive elements of one worker = four groups of 8.
// A group is the unit of randomness: one Philox4x32-10 call (counter = group index, worker) yields
// 128 bits = eight 16-bit slots, one per element.  A run packs into exactly `bits` 32-bit words, so
// no thread ever shares a word with another and no shuffles or atomics are needed.
// HBM traffic per element: 4 (fp32) or 2 (bf16) bytes read, bits/8 bytes written.
#include "tq_device.cuh"
#include "tq_launch.h"

namespace tq {

// Per-worker quantizer as the kernel sees it.
struct WorkerQ {
    float alpha, inv_step, top;   // top = (float)(L-1)
    float levels[TQ_MAX_LEVELS];
    float inv_width[TQ_MAX_LEVELS];
};
struct CompressArgs {
    WorkerQ q[TQ_MAX_WORKERS];
};

// Round-up decision.  T = rint(p * 2^16) is read from the mantissa of p * 2^16 + 2^23 (one fused
// rounding, ties to even); the element rounds up iff its 16 random bits r satisfy r < T.
__device__ __forceinline__ uint32_t rounds_up(float p, uint32_t r16) {
    const float pm = __fmaf_rn(p, 65536.0f, kMagic);
    return __float_as_uint(pm) > (r16 + kMagicBits) ? 1u : 0u;
}

// Uniform codebook, l_k = -alpha + k * 2 alpha / s (Section 4.1).  Reference form of the decision:
// t = clip(g), x = (t + alpha) * inv_step, k = min(floor x, s-1), p = x - k.  Computed here as
// x = clip((g + alpha) * inv_step, 0, s), k' = floor x, p' = x - k': the affine map is monotone, so
// clipping after it gives the same x for |g| <= alpha and 0 / >= s beyond; at x = s this yields
// k' = s, p' = 0, i.e. the same code s as k = s-1, p >= 1.  NaN becomes 0 (fmaxf drops it).
__device__ __forceinline__ uint32_t code_uniform(float g, float alpha, float inv_step, float top, uint32_t r16) {
    float x = __fmul_rn(__fadd_rn(g, alpha), inv_step);
    x = fminf(fmaxf(x, 0.0f), top);
    const float xm = __fadd_rd(x, kMagic);            // mantissa now holds floor(x)
    const float p = __fsub_rn(x, __fsub_rn(xm, kMagic));
    return (__float_as_uint(xm) - kMagicBits) + rounds_up(p, r16);
}

// General codebook from shared memory: search[] holds l_1 .. l_{s-1} at indices 1 .. s-1 and +inf
// from index s on, so the branch-free binary search returns k = max{ j <= s-1 : l_j <= t }.
template <int BITS>
__device__ __forceinline__ uint32_t code_table(float g, float alpha, const float* search, const float2* cell,
                                               uint32_t r16) {
    const float t = fminf(fmaxf(g, -alpha), alpha);   // NaN -> -alpha
    uint32_t k = 0;
#pragma unroll
    for (int step = (1 << BITS) >> 1; step > 0; step >>= 1)
        if (t >= search[k + step]) k += step;
    const float2 c = cell[k];                          // (l_k, 1 / (l_{k+1} - l_k))
    const float p = __fmul_rn(__fsub_rn(t, c.x), c.y);
    return k + rounds_up(p, r16);
}

template <int BITS, bool NONUNIFORM, bool BF16>
__global__ void __launch_bounds__(kThreads)
compress_kernel(const void* __restrict__ grad, uint64_t d, uint64_t grad_stride,
                const __grid_constant__ CompressArgs args, uint32_t seed_lo, uint32_t seed_hi,
                uint32_t first_worker, uint32_t* __restrict__ packed, uint64_t words_stride, uint64_t words_out) {
    constexpr int L = 1 << BITS;
    const uint32_t wi = blockIdx.y;
    const WorkerQ& q = args.q[wi];

    __shared__ float s_search[2 * TQ_MAX_LEVELS];
    __shared__ float2 s_cell[TQ_MAX_LEVELS];
    if constexpr (NONUNIFORM) {
        if (threadIdx.x < 2 * TQ_MAX_LEVELS)
            s_search[threadIdx.x] = (threadIdx.x >= 1 && threadIdx.x <= L - 2) ? q.levels[threadIdx.x] : __int_as_float(0x7F800000);
        if (threadIdx.x < L - 1) s_cell[threadIdx.x] = make_float2(q.levels[threadIdx.x], q.inv_width[threadIdx.x]);
        __syncthreads();
    }

    const uint64_t n_runs = (d + 31) >> 5;
    const uint64_t run = static_cast<uint64_t>(blockIdx.x) * kThreads + threadIdx.x;
    if (run >= n_runs) return;

    const size_t esz = BF16 ? 2 : 4;
    const char* row = static_cast<const char*>(grad) + static_cast<uint64_t>(wi) * grad_stride * esz;
    const uint64_t j0 = run << 5;
    const bool full = j0 + 32 <= d;
    const float alpha = q.alpha, inv_step = q.inv_step, top = q.top;
    const uint32_t worker = first_worker + wi;

    float g[4][8];
    if (full) {
#pragma unroll
        for (int grp = 0; grp < 4; ++grp) load8<BF16>(row + (j0 + 8 * grp) * esz, g[grp]);
    } else {
#pragma unroll
        for (int grp = 0; grp < 4; ++grp)
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const uint64_t j = j0 + 8 * grp + e;
                g[grp][e] = j < d ? load1<BF16>(row, j) : 0.0f;
            }
    }

    uint32_t chunk[4];   // the 8*BITS packed bits of each group
#pragma unroll
    for (int grp = 0; grp < 4; ++grp) {
        const uint64_t block = (j0 >> 3) + grp;
        uint32_t rnd[4];
        philox4x32_10(static_cast<uint32_t>(block), static_cast<uint32_t>(block >> 32), worker, 0u, seed_lo, seed_hi, rnd);
        uint32_t bitsacc = 0;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const uint32_t r16 = (e & 1) ? (rnd[e >> 1] >> 16) : (rnd[e >> 1] & 0xFFFFu);
            uint32_t code;
            if constexpr (NONUNIFORM) code = code_table<BITS>(g[grp][e], alpha, s_search, s_cell, r16);
            else code = code_uniform(g[grp][e], alpha, inv_step, top, r16);
            if (!full && j0 + 8 * grp + e >= d) code = 0;     // padding bits are zero
            bitsacc |= code << (e * BITS);
        }
        chunk[grp] = bitsacc;
    }

    // four chunks of 8*BITS bits -> BITS words, LSB first
    uint32_t w[BITS];
    if constexpr (BITS == 4) { w[0] = chunk[0]; w[1] = chunk[1]; w[2] = chunk[2]; w[3] = chunk[3]; }
    if constexpr (BITS == 3) {
        w[0] = chunk[0] | (chunk[1] << 24);
        w[1] = (chunk[1] >> 8) | (chunk[2] << 16);
        w[2] = (chunk[2] >> 16) | (chunk[3] << 8);
    }
    if constexpr (BITS == 2) { w[0] = chunk[0] | (chunk[1] << 16); w[1] = chunk[2] | (chunk[3] << 16); }
    if constexpr (BITS == 1) { w[0] = chunk[0] | (chunk[1] << 8) | (chunk[2] << 16) | (chunk[3] << 24); }

    uint32_t* dst = packed + static_cast<uint64_t>(wi) * words_stride + run * BITS;
    if (run + 1 < n_runs) {   // every word of an interior run lies below words_out
        if constexpr (BITS == 4) *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
        if constexpr (BITS == 3) { dst[0] = w[0]; dst[1] = w[1]; dst[2] = w[2]; }
        if constexpr (BITS == 2) *reinterpret_cast<uint2*>(dst) = make_uint2(w[0], w[1]);
        if constexpr (BITS == 1) dst[0] = w[0];
    } else {
        // last run of the row: write its words that exist, then zero the alignment padding
        const uint64_t first = run * BITS;
#pragma unroll
        for (int i = 0; i < BITS; ++i)
            if (first + i < words_out) dst[i] = w[i];
        uint32_t* rowp = packed + static_cast<uint64_t>(wi) * words_stride;
        for (uint64_t k = first + BITS; k < words_out; ++k) rowp[k] = 0u;
    }
}

template <int BITS, bool NU, bool BF>
static cudaError_t launch(const CompressCall& c, const CompressArgs& args, dim3 grid) {
    compress_kernel<BITS, NU, BF><<<grid, kThreads, 0, c.stream>>>(
        c.grad, c.d, c.grad_stride, args, static_cast<uint32_t>(c.seed), static_cast<uint32_t>(c.seed >> 32),
        c.first_worker, c.packed, c.words_stride, c.words_out);
    return cudaGetLastError();
}

template <int BITS>
static cudaError_t dispatch(const CompressCall& c, const CompressArgs& a, dim3 grid) {
    if (c.nonuniform) return c.bf16 ? launch<BITS, true, true>(c, a, grid) : launch<BITS, true, false>(c, a, grid);
    return c.bf16 ? launch<BITS, false, true>(c, a, grid) : launch<BITS, false, false>(c, a, grid);
}

cudaError_t launch_compress(const CompressCall& c) {
    static thread_local CompressArgs args;   // 9 KB: keep it off the stack
    for (uint32_t i = 0; i < c.n_workers; ++i) {
        const tq_params_t& p = c.params[i];
        WorkerQ& q = args.q[i];
        q.alpha = p.alpha; q.inv_step = p.inv_step; q.top = static_cast<float>(p.num_levels - 1);
        for (int k = 0; k < TQ_MAX_LEVELS; ++k) { q.levels[k] = p.levels[k]; q.inv_width[k] = p.inv_width[k]; }
    }
    const uint64_t n_runs = (c.d + 31) >> 5;
    const uint64_t blocks = (n_runs + kThreads - 1) / kThreads;
    if (blocks == 0) return cudaSuccess;
    if (blocks > 0x7FFFFFFFull) return cudaErrorInvalidConfiguration;
    const dim3 grid(static_cast<unsigned>(blocks), c.n_workers);
    switch (c.bits) {
        case 1: return dispatch<1>(c, args, grid);
        case 2: return dispatch<2>(c, args, grid);
        case 3: return dispatch<3>(c, args, grid);
        default: return dispatch<4>(c, args, grid);
    }
}

}  // namespace tq
