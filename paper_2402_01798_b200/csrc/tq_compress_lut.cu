// Client side of Algorithm 1 for gradients stored as bf16: truncate (Section 3.1, truncation equation),
// stochastically round onto the codebook (Section 3.1, quantizer equation) and pack, with the part of
// the decision that does not depend on the random draw taken from a table.
//
// A bf16 element has only 2^16 possible values, and for a given quantizer the interval index k and the
// threshold T = rint(p * 2^16) of the rounding decision are functions of that value alone.  Each block
// therefore evaluates the decision once per bit pattern, with the very operations the element-wise
// kernels use (one IEEE operation per step), and stores X + 65535 with X = k * 2^16 + min(T, 2^16).  An
// element then costs one table read, and code = k + [r < T] = floor((X + 65535 - r) / 2^16) for the
// element's 16 random bits r.
//
// Table index.  Only a window of magnitudes needs entries.  Above the window's top pattern P_top (the
// smallest bf16 value >= alpha) every value is truncated to +-alpha; below its base pattern every value is
// so small that the decision equals that of zero (the host checks this by evaluating the decision at
// +-base; it is monotone in the value).  The index is clamp(|pattern| - base, 0, n - 1) + n * [negative],
// n = 2048, 4096 or 8192 entries per sign (16, 32 or 64 binades), computed for the two elements of a
// 32-bit word at once with 16-bit SIMD integer instructions.  NaN is sent to -alpha before that by a
// packed bf16 maximum with -top, which returns the operand that is a number, as fmaxf does in the
// element-wise form.
//
// Arithmetic on the floating-point pipe, without conversions: a table entry is the float with bit
// pattern 0x19000000 + (X + 65535) = 2^-77 + (X + 65535) * 2^-100, the random slot is made into
// 2^-77 + r * 2^-100 by one byte permute; their difference is exact, and a multiplication by 2^-65
// rounded down yields floor(.../2^16) * 2^-149, a denormal whose bit pattern IS the code.  Packing
// multiplies and adds such denormals (exact: fixed-point arithmetic below 2^24 * 2^-149), so the packed
// bits appear as a bit pattern too.
#include <cmath>

#include "tq_device.cuh"
#include "tq_launch.h"
#include "tq_lut.cuh"

namespace tq {

constexpr uint32_t kSlotExpBits = 0x19000000u;   // 2^-77: exponent field 50, ulp 2^-100

struct LutWorker {
    float alpha;
    uint32_t base2;       // -(base pattern) in both 16-bit halves
    uint32_t negtop2;     // the bf16 value -top in both halves
    float levels[TQ_MAX_LEVELS];
    float inv_width[TQ_MAX_LEVELS];
};
struct LutArgs {
    LutWorker q[TQ_MAX_WORKERS];
};

// ---- device ------------------------------------------------------------------------------------------

__device__ __forceinline__ uint32_t max_bf16x2(uint32_t a, uint32_t b) {
    uint32_t r; asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b)); return r;
}
// Four pairs of codes held as denormals (bit pattern = code) -> their 8 * BITS packed bits, LSB first,
// as a bit pattern.  Every intermediate is an integer below 2^24 in units of 2^-149: exact.
template <int BITS>
__device__ __forceinline__ uint32_t pack8_bits(const f32x2 (&c)[4]) {
    constexpr float B = static_cast<float>(1 << BITS), B2 = B * B;
    if constexpr (BITS <= 3) {
        f32x2 a = fma2(c[3], both(B2), c[2]);
        a = fma2(a, both(B2), c[1]);
        a = fma2(a, both(B2), c[0]);
        float ev, od;
        unpair(a, ev, od);
        return __float_as_uint(__fmaf_rn(od, B, ev));
    } else {
        float e0, o0, e1, o1;
        unpair(fma2(c[1], both(B2), c[0]), e0, o0);
        unpair(fma2(c[3], both(B2), c[2]), e1, o1);
        return __byte_perm(__float_as_uint(__fmaf_rn(o0, B, e0)), __float_as_uint(__fmaf_rn(o1, B, e1)), 0x5410u);
    }
}

struct LutCtx {
    uint32_t table;          // shared-memory address of the entries: positive values from byte 0, negative values from byte 32768
    uint32_t negtop2, nbase2, cap2;
    PhiloxRun pr;
};

__device__ __forceinline__ float lds_f32(uint32_t addr) {
    float v; asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr)); return v;
}

// Elements a thread quantizes as one piece: consecutive, loaded with 256-bit loads (lane after lane, so a
// warp's load covers one contiguous kilobyte), and packing to whole 32-bit words.
template <int BITS> struct Piece { static constexpr int kElems = (BITS == 2 || BITS == 4) ? 16 : 32; };

// One piece whose words are in registers: quantize, pack, store.  TAIL = the row's last piece, possibly partial.
template <int BITS, bool TAIL>
__device__ __forceinline__ void lut_piece(const uint32_t (&g)[Piece<BITS>::kElems / 2], uint32_t* prow, uint64_t piece, uint64_t d,
                                          uint64_t words_out, const RoundKeys& rk, const LutCtx& cx) {
    constexpr int E = Piece<BITS>::kElems, GROUPS = E / 8, WORDS = E * BITS / 32;
    const uint64_t j0 = piece * E;
    const uint32_t blk_lo = static_cast<uint32_t>(j0 >> 3);   // rows of more than 2^35 elements do not come here
    const f32x2 down = both(2.710505431213761e-20f);          // 2^-65
    uint32_t chunk[GROUPS];
#pragma unroll
    for (int grp = 0; grp < GROUPS; ++grp) {
        uint32_t rnd[4];
        philox_block(blk_lo + grp, cx.pr, rk, rnd);           // j0 >> 3 is a multiple of GROUPS: no carry
        f32x2 code[4];
#pragma unroll
        for (int h = 0; h < 4; ++h) {                          // elements 2h, 2h+1 of the group
            const uint32_t w = max_bf16x2(g[4 * grp + h], cx.negtop2);
            // byte offsets of the two entries: 4 * clamp(|pattern| - base, 0, n - 1), negative values 32 KB further on
            const uint32_t off = __viaddmin_s16x2_relu(w & 0x7FFF7FFFu, cx.nbase2, cx.cap2) * 4u + (w & 0x80008000u);
            const float y0 = lds_f32(cx.table + (off & 0xFFFFu)), y1 = lds_f32(cx.table + (off >> 16));
            const float r0 = __uint_as_float(__byte_perm(rnd[h], kSlotExpBits, 0x7610u));
            const float r1 = __uint_as_float(__byte_perm(rnd[h], kSlotExpBits, 0x7632u));
            code[h] = mul2_rd(sub2(pair(y0, y1), pair(r0, r1)), down);
            if constexpr (TAIL) {                              // padding bits are zero
                float c0, c1;
                unpair(code[h], c0, c1);
                if (j0 + 8 * grp + 2 * h >= d) c0 = 0.0f;
                if (j0 + 8 * grp + 2 * h + 1 >= d) c1 = 0.0f;
                code[h] = pair(c0, c1);
            }
        }
        chunk[grp] = pack8_bits<BITS>(code);
    }

    uint32_t w[WORDS];
    if constexpr (BITS == 4) { w[0] = chunk[0]; w[1] = chunk[1]; }
    if constexpr (BITS == 3) {
        w[0] = chunk[0] | (chunk[1] << 24);
        w[1] = (chunk[1] >> 8) | (chunk[2] << 16);
        w[2] = (chunk[2] >> 16) | (chunk[3] << 8);
    }
    if constexpr (BITS == 2) { w[0] = __byte_perm(chunk[0], chunk[1], 0x5410u); }
    if constexpr (BITS == 1) { w[0] = chunk[0] | (chunk[1] << 8) | (chunk[2] << 16) | (chunk[3] << 24); }

    uint32_t* dst = prow + piece * WORDS;
    if constexpr (!TAIL) {
        if constexpr (BITS == 4) *reinterpret_cast<uint2*>(dst) = make_uint2(w[0], w[1]);
        if constexpr (BITS == 3) { dst[0] = w[0]; dst[1] = w[1]; dst[2] = w[2]; }
        if constexpr (BITS == 2 || BITS == 1) dst[0] = w[0];
    } else {
        const uint64_t first = piece * WORDS;
#pragma unroll
        for (int i = 0; i < WORDS; ++i)
            if (first + i < words_out) dst[i] = w[i];
        for (uint64_t k = first + WORDS; k < words_out; ++k) prow[k] = 0u;
    }
}

template <int BITS>
__device__ __forceinline__ void load_piece(const char* row, uint64_t piece, uint32_t (&g)[Piece<BITS>::kElems / 2]) {
    constexpr int E = Piece<BITS>::kElems;
#pragma unroll
    for (int i = 0; i < E / 16; ++i)
        asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=r"(g[8 * i]), "=r"(g[8 * i + 1]), "=r"(g[8 * i + 2]), "=r"(g[8 * i + 3]),
                       "=r"(g[8 * i + 4]), "=r"(g[8 * i + 5]), "=r"(g[8 * i + 6]), "=r"(g[8 * i + 7])
                     : "l"(row + piece * (2 * E) + 32 * i));
}

#ifndef TQ_LUT_MIN_BLOCKS
#define TQ_LUT_MIN_BLOCKS 3
#endif
constexpr int kLutThreads = kThreads;

// A block's share of one row: build the table for quantizer q (n_entries per sign), then quantize.
template <int BITS>
__device__ __forceinline__ void lut_block(const LutWorker& q, uint32_t n_entries, float* s_table, const char* __restrict__ row,
                                          uint32_t* __restrict__ prow, uint64_t d, uint64_t words_out, uint32_t worker,
                                          const RoundKeys& rk) {
    // the table: the decision for every bit pattern of the window, both signs
    {
        const uint32_t base = (0u - q.base2) & 0xFFFFu;
        for (uint32_t i = threadIdx.x; i < 2 * n_entries; i += kLutThreads) {
            const bool neg = i >= n_entries;
            const uint32_t c = neg ? i - n_entries : i;
            const uint32_t pattern = (base + c) | (neg ? 0x8000u : 0u);
            const uint32_t x = decision_x(bf16_pattern_value(pattern), q.alpha, q.levels, q.inv_width, 1u << BITS);
            s_table[c + (neg ? kLutMaxEntries : 0)] = __uint_as_float(kSlotExpBits + x + 65535u);
        }
    }
    __syncthreads();

    constexpr int E = Piece<BITS>::kElems, PER_ITER = 32 / E;   // 32 elements per thread and iteration: four Philox blocks in flight
    const LutCtx cx{smem_addr(s_table), q.negtop2, q.base2, (n_entries - 1) * 0x00010001u, philox_run(0u, worker, rk)};
    const uint64_t interior = (d - 1) / E;                     // whole pieces before the row's last one
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * kLutThreads;

    // two sets of registers take turns: the next iteration's loads are in flight while this one is quantized
    uint64_t piece = static_cast<uint64_t>(blockIdx.x) * kLutThreads + threadIdx.x;
    uint32_t a[PER_ITER][E / 2], b[PER_ITER][E / 2];
    auto fetch = [&](uint32_t (&buf)[PER_ITER][E / 2], uint64_t first) {
#pragma unroll
        for (int k = 0; k < PER_ITER; ++k)
            if (first + k * stride < interior) load_piece<BITS>(row, first + k * stride, buf[k]);
    };
    auto quantize = [&](const uint32_t (&buf)[PER_ITER][E / 2], uint64_t first) {
#pragma unroll
        for (int k = 0; k < PER_ITER; ++k)
            if (first + k * stride < interior) lut_piece<BITS, false>(buf[k], prow, first + k * stride, d, words_out, rk, cx);
    };
    fetch(a, piece);
    while (piece < interior) {
        const uint64_t next = piece + PER_ITER * stride;
        fetch(b, next);
        quantize(a, piece);
        if (next >= interior) break;
        piece = next + PER_ITER * stride;
        fetch(a, piece);
        quantize(b, next);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {                 // the row's last piece, possibly partial
        const unsigned short* e = reinterpret_cast<const unsigned short*>(row);
        uint32_t t[E / 2];
#pragma unroll
        for (int i = 0; i < E / 2; ++i) {
            const uint64_t j = interior * E + 2 * i;
            const uint32_t lo = j < d ? __ldg(e + j) : 0u, hi = j + 1 < d ? __ldg(e + j + 1) : 0u;
            t[i] = lo | (hi << 16);
        }
        lut_piece<BITS, true>(t, prow, interior, d, words_out, rk, cx);
    }
}

// Quantizers passed by value (host-side tq_params); the host has chosen the window.
template <int BITS>
__global__ void __launch_bounds__(kLutThreads, TQ_LUT_MIN_BLOCKS)
compress_lut_kernel(const void* __restrict__ grad, uint64_t d, uint64_t grad_stride, const __grid_constant__ LutArgs args,
                    const __grid_constant__ RoundKeys rk, uint32_t n_entries, uint32_t first_worker,
                    uint32_t* __restrict__ packed, uint64_t words_stride, uint64_t words_out) {
    extern __shared__ __align__(16) float s_table[];          // kLutMaxEntries + n_entries: the negative half starts at entry kLutMaxEntries
    const uint32_t wi = blockIdx.y;
    lut_block<BITS>(args.q[wi], n_entries, s_table, static_cast<const char*>(grad) + static_cast<uint64_t>(wi) * grad_stride * 2,
                    packed + static_cast<uint64_t>(wi) * words_stride, d, words_out, first_worker + wi, rk);
}

// Quantizers read from device memory (tq_params_device).  Every block decides by lut_serves_record whether the
// table form serves its row, with the largest window; rows it does not serve are left to the element-wise
// device-parameter kernels, which are launched after this one and skip the rows served here.
template <int BITS>
__global__ void __launch_bounds__(kLutThreads, TQ_LUT_MIN_BLOCKS)
compress_lut_kernel_dev(const void* __restrict__ grad, uint64_t d, uint64_t grad_stride, const tq_params_t* __restrict__ params,
                        const __grid_constant__ RoundKeys rk, uint32_t first_worker, uint32_t* __restrict__ packed,
                        uint64_t words_stride, uint64_t words_out) {
    extern __shared__ __align__(16) float s_table[];          // 2 * kLutMaxEntries
    __shared__ LutWorker s_q;
    __shared__ bool s_serves;
    const uint32_t wi = blockIdx.y;
    if (threadIdx.x < TQ_MAX_LEVELS) {
        s_q.levels[threadIdx.x] = params[wi].levels[threadIdx.x];
        s_q.inv_width[threadIdx.x] = params[wi].inv_width[threadIdx.x];
    }
    if (threadIdx.x == 0) {
        uint32_t top = 0, base = 0;
        s_serves = lut_serves_record(params[wi], BITS, &top, &base);
        s_q.alpha = params[wi].alpha;
        s_q.base2 = ((0u - base) & 0xFFFFu) * 0x00010001u;
        s_q.negtop2 = (top | 0x8000u) * 0x00010001u;
    }
    __syncthreads();
    if (!s_serves) return;
    lut_block<BITS>(s_q, kLutMaxEntries, s_table, static_cast<const char*>(grad) + static_cast<uint64_t>(wi) * grad_stride * 2,
                    packed + static_cast<uint64_t>(wi) * words_stride, d, words_out, first_worker + wi, rk);
}

// ---- host --------------------------------------------------------------------------------------------

// Entries per sign the worker needs, 0 if no window of at most kLutMaxEntries does.
static uint32_t entries_needed(const tq_params_t& p, uint32_t top) {
    for (uint32_t n = kLutMinEntries; n <= static_cast<uint32_t>(kLutMaxEntries); n *= 2) {
        uint32_t base = 0;
        if (lut_window_fits(p.alpha, p.levels, p.inv_width, p.num_levels, top, n, &base)) return n;
    }
    return 0;
}

static uint64_t lut_blocks_per_worker(uint64_t d, uint32_t n_workers, int per_sm, int pieces_elems);

template <int BITS>
static cudaError_t launch_lut(const CompressCall& c, const LutArgs& args, uint32_t n_entries) {
    const int smem = static_cast<int>((kLutMaxEntries + n_entries) * sizeof(float));
    cudaError_t e = cudaFuncSetAttribute(compress_lut_kernel<BITS>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, compress_lut_kernel<BITS>, kLutThreads, smem);
    if (e != cudaSuccess) return e;
    const uint64_t per_worker = lut_blocks_per_worker(c.d, c.n_workers, per_sm, Piece<BITS>::kElems);
    const RoundKeys rk = round_keys(c.seed);
    compress_lut_kernel<BITS><<<dim3(static_cast<unsigned>(per_worker), c.n_workers), kLutThreads, smem, c.stream>>>(
        c.grad, c.d, c.grad_stride, args, rk, n_entries, c.first_worker, c.packed, c.words_stride, c.words_out);
    return cudaGetLastError();
}


static uint64_t lut_blocks_per_worker(uint64_t d, uint32_t n_workers, int per_sm, int pieces_elems) {
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const uint64_t tiles = (d / pieces_elems + kLutThreads - 1) / kLutThreads + 1;
    uint64_t per_worker = static_cast<uint64_t>(sms) * (per_sm < 1 ? 1 : per_sm) / n_workers;      // rounded down: one wave holds the grid
    if (per_worker > tiles) per_worker = tiles;
    return per_worker < 1 ? 1 : per_worker;
}

template <int BITS>
static cudaError_t launch_lut_dev(const CompressCall& c) {
    const int smem = static_cast<int>(2 * kLutMaxEntries * sizeof(float));
    cudaError_t e = cudaFuncSetAttribute(compress_lut_kernel_dev<BITS>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, compress_lut_kernel_dev<BITS>, kLutThreads, smem);
    if (e != cudaSuccess) return e;
    const uint64_t per_worker = lut_blocks_per_worker(c.d, c.n_workers, per_sm, Piece<BITS>::kElems);
    compress_lut_kernel_dev<BITS><<<dim3(static_cast<unsigned>(per_worker), c.n_workers), kLutThreads, smem, c.stream>>>(
        c.grad, c.d, c.grad_stride, c.params_dev, round_keys(c.seed), c.first_worker, c.packed, c.words_stride, c.words_out);
    return cudaGetLastError();
}

// Rows below this many elements keep the element-wise kernels (the table costs more than it saves).
constexpr uint64_t kLutMinElements = 1u << 18;

cudaError_t launch_compress_lut(const CompressCall& c, bool* applied) {
    *applied = false;
    if (!c.bf16 || !c.nonuniform || c.segs || c.d < kLutMinElements || c.d > (1ull << 35)) return cudaSuccess;
    if (c.params_dev) {      // the kernel decides row by row; the caller launches the element-wise kernels for the rest
        *applied = true;
        switch (c.bits) {
            case 1: return launch_lut_dev<1>(c);
            case 2: return launch_lut_dev<2>(c);
            case 3: return launch_lut_dev<3>(c);
            default: return launch_lut_dev<4>(c);
        }
    }
    static thread_local LutArgs args;
    uint32_t n_entries = 0;
    for (uint32_t i = 0; i < c.n_workers; ++i) {
        const tq_params_t& p = c.params[i];
        if (!(p.alpha > 0.0f) || !(p.alpha <= 3.402823466e38f)) return cudaSuccess;
        const uint32_t top = top_pattern(p.alpha);
        const uint32_t n = entries_needed(p, top);
        if (n == 0) return cudaSuccess;
        if (n > n_entries) n_entries = n;
    }
    for (uint32_t i = 0; i < c.n_workers; ++i) {
        const tq_params_t& p = c.params[i];
        LutWorker& q = args.q[i];
        const uint32_t top = top_pattern(p.alpha);
        const uint32_t base = top >= n_entries ? top - (n_entries - 1) : 0u;   // a larger window than needed stays valid
        q.alpha = p.alpha;
        q.base2 = ((0u - base) & 0xFFFFu) * 0x00010001u;
        q.negtop2 = (top | 0x8000u) * 0x00010001u;
        for (int k = 0; k < TQ_MAX_LEVELS; ++k) { q.levels[k] = p.levels[k]; q.inv_width[k] = p.inv_width[k]; }
    }
    *applied = true;
    switch (c.bits) {
        case 1: return launch_lut<1>(c, args, n_entries);
        case 2: return launch_lut<2>(c, args, n_entries);
        case 3: return launch_lut<3>(c, args, n_entries);
        default: return launch_lut<4>(c, args, n_entries);
    }
}

}  // namespace tq
