// Server side of Algorithm 1: unpack the N workers' b-bit codes, look each up in that worker's
// codebook and average, out_j = (sum_i l^(i)[c_ij]) / N (w_i = 1/N as in Lemma 2) or sum_i w_i l^(i)[c_ij],
// fused in one streaming pass.  fp32 adds happen in worker order, so the result does not depend on
// the launch shape.
//
// Work split: a thread owns the smallest run of elements whose codes fill whole 32-bit words
// (8 elements for 4 bits, 16 for 2 bits, 32 for 1 bit: one word per worker; 32 elements = 3 words for
// 3 bits), keeps one fp32 accumulator per element in registers and walks the workers four at a time
// so that four independent loads are in flight before the dependent lookups start.
// Codebooks live in shared memory, 16 consecutive words per worker: any set of codes of one worker
// maps to distinct banks, so lookups are conflict-free.
// HBM traffic per output element: N * bits / 8 bytes read, 4 bytes written.
#include "tq_device.cuh"
#include "tq_launch.h"

namespace tq {

struct DecompressArgs {
    float table[TQ_MAX_WORKERS][TQ_MAX_LEVELS];   // levels, already multiplied by w_i when weights are given
};

__device__ __forceinline__ uint32_t ldg32_stream(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.global.nc.L1::no_allocate.b32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}

template <int BITS>
struct Unit {
    static constexpr int kElems = BITS == 4 ? 8 : (BITS == 2 ? 16 : 32);
    static constexpr int kWords = kElems * BITS / 32;
};

template <int BITS>
__global__ void __launch_bounds__(kThreads)
decompress_kernel(const uint32_t* __restrict__ packed, uint64_t words_stride, uint64_t words_valid, uint32_t n,
                  uint64_t d, const __grid_constant__ DecompressArgs args, float scale, int divide,
                  float* __restrict__ out) {
    constexpr int E = Unit<BITS>::kElems, W = Unit<BITS>::kWords;
    constexpr uint32_t kMask = (1u << BITS) - 1u;

    __shared__ float s_tab[TQ_MAX_WORKERS * TQ_MAX_LEVELS];
    for (uint32_t t = threadIdx.x; t < n * TQ_MAX_LEVELS; t += kThreads)
        s_tab[t] = args.table[t / TQ_MAX_LEVELS][t % TQ_MAX_LEVELS];
    __syncthreads();

    const uint64_t n_units = (d + E - 1) / E;
    const uint64_t u = static_cast<uint64_t>(blockIdx.x) * kThreads + threadIdx.x;
    if (u >= n_units) return;

    float acc[E];
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = 0.0f;

    const uint64_t w0 = u * W;
    for (uint32_t i0 = 0; i0 < n; i0 += 4) {
        uint32_t w[4][W + 1];
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const uint32_t* row = packed + static_cast<uint64_t>(i0 + b) * words_stride;
#pragma unroll
            for (int k = 0; k < W; ++k)
                w[b][k] = (i0 + b < n && w0 + k < words_valid) ? ldg32_stream(row + w0 + k) : 0u;
            w[b][W] = 0u;
        }
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            if (i0 + b < n) {
                const float* tab = s_tab + (i0 + b) * TQ_MAX_LEVELS;
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    const int pos = e * BITS;
                    const uint32_t code = (W == 1) ? ((w[b][0] >> pos) & kMask)
                                                   : (__funnelshift_r(w[b][pos >> 5], w[b][(pos >> 5) + 1], pos & 31) & kMask);
                    acc[e] = __fadd_rn(acc[e], tab[code]);
                }
            }
        }
    }

    // w_i = 1/N: one division by N (for N a power of two the product with 2^-k is the same value)
#pragma unroll
    for (int e = 0; e < E; ++e) {
        if (divide == 1) acc[e] = __fdiv_rn(acc[e], scale);
        else if (divide == 2) acc[e] = __fmul_rn(acc[e], scale);
    }

    const uint64_t j0 = u * E;
    if (j0 + E <= d) {
#pragma unroll
        for (int v = 0; v < E / 8; ++v) {
            const float o[8] = {acc[8 * v], acc[8 * v + 1], acc[8 * v + 2], acc[8 * v + 3],
                                acc[8 * v + 4], acc[8 * v + 5], acc[8 * v + 6], acc[8 * v + 7]};
            stg256(out + j0 + 8 * v, o);
        }
    } else {
#pragma unroll
        for (int e = 0; e < E; ++e)
            if (j0 + e < d) out[j0 + e] = acc[e];
    }
}

template <int BITS>
static cudaError_t launch(const DecompressCall& c, const DecompressArgs& args, float scale, int divide) {
    const uint64_t n_units = (c.d + Unit<BITS>::kElems - 1) / Unit<BITS>::kElems;
    const uint64_t blocks = (n_units + kThreads - 1) / kThreads;
    if (blocks == 0) return cudaSuccess;
    if (blocks > 0x7FFFFFFFull) return cudaErrorInvalidConfiguration;
    decompress_kernel<BITS><<<static_cast<unsigned>(blocks), kThreads, 0, c.stream>>>(
        c.packed, c.words_stride, c.words_valid, c.n_workers, c.d, args, scale, divide, c.out);
    return cudaGetLastError();
}

cudaError_t launch_decompress(const DecompressCall& c) {
    static thread_local DecompressArgs args;
    for (uint32_t i = 0; i < c.n_workers; ++i)
        for (int k = 0; k < TQ_MAX_LEVELS; ++k) {
            const float l = c.params[i].levels[k];
            // weighted form: each product w_i * l is rounded to fp32 once; it depends on (i, k) only,
            // so it is formed here instead of once per element
            args.table[i][k] = c.weights ? c.weights[i] * l : l;
        }
    float scale = 1.0f;
    int divide = 0;
    if (!c.weights) {
        const uint32_t n = c.n_workers;
        if ((n & (n - 1)) == 0) { divide = 2; scale = 1.0f / static_cast<float>(n); }
        else { divide = 1; scale = static_cast<float>(n); }
    }
    switch (c.bits) {
        case 1: return launch<1>(c, args, scale, divide);
        case 2: return launch<2>(c, args, scale, divide);
        case 3: return launch<3>(c, args, scale, divide);
        default: return launch<4>(c, args, scale, divide);
    }
}

}  // namespace tq
