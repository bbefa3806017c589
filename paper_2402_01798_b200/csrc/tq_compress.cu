// Client side of Algorithm 1: truncate (Section 3.1, truncation equation), stochastically round onto
// the codebook (Section 3.1, quantizer equation) and pack b-bit codes, fused in one pass.
//
// Work split: persistent blocks walk tiles of 8192 elements of one worker; in a tile a thread owns a
// run of 32 consecutive elements = four groups of 8.  A group is the unit of randomness: one
// Philox4x32-10 call (counter = group index, worker) yields 128 bits = eight 16-bit slots, one per
// element.  A run packs into exactly `bits` 32-bit words, so no thread ever shares a word with
// another and no shuffles or atomics are needed.
// HBM traffic per element: 4 (fp32) or 2 (bf16) bytes read, bits/8 bytes written.
//
// The kernel is bound by instruction issue, and within that by the half-rate integer/compare pipe,
// so the per-element arithmetic is arranged to run on the fp32 multiply-add pipe wherever the
// result is provably the same:
//   - floor / int conversion: add 2^23 rounding down, the integer appears in the mantissa;
//   - threshold T = rint(p * 2^16): one fused multiply-add with 2^23;
//   - the random slot r as the float 2^23 + r: one byte-permute; [r < T] = sat((2^23 + T) - (2^23 + r)),
//     a saturating subtract of two exactly representable integers;
//   - uniform codebook: interval and threshold together as the one integer X = rint(x * 2^16) = k * 2^16 + T,
//     code = ceil((X - r) / 2^16), with the clamps of x done by saturating multiplies and subtracts;
//   - codes are kept as small floats and packed by exact multiply-adds (sums stay below 2^24);
//   - table offsets are formed as denormal floats whose bit pattern IS the byte offset.
#include <cuda.h>

#include <cmath>

#include "tq_device.cuh"
#include "tq_launch.h"
#include "tq_lut.cuh"

namespace tq {

constexpr int kMaxGridCells = 2048;   // finest lookup grid for the non-uniform interval search
constexpr int kMinGridCells = 32;

// Per-worker quantizer as the kernel sees it.
struct WorkerQ {
    float alpha, inv_step, top;   // top = (float)(L-1)
    float inv_step_l;             // inv_step / L when that quotient is exact and normal, else 0 (uniform mode)
    float inv_2alpha;             // maps [-alpha, alpha] to [0, 1] for the lookup grid
    float cell_scale;             // grid cells M as the denormal M * 2^-149
    uint32_t cells;               // M
    float levels[TQ_MAX_LEVELS];
    float inv_width[TQ_MAX_LEVELS];
};
struct CompressArgs {
    WorkerQ q[TQ_MAX_WORKERS];
};

// kUniformWide: the uniform codebook through the arithmetic that needs no scaled inverse step (used
// only when inv_step / L would be subnormal, i.e. alpha beyond about 2^121).
enum Search { kUniform = 0, kGrid = 1, kBinary = 2, kUniformWide = 3 };
__host__ __device__ constexpr bool is_uniform(int search) { return search == kUniform || search == kUniformWide; }

cudaError_t launch_compress_dev(const CompressCall& c);

__device__ __forceinline__ float mul_sat(float a, float b) {
    float r; asm("mul.rn.sat.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b)); return r;
}
__device__ __forceinline__ float sub_sat(float a, float b) {
    float r; asm("sub.rn.sat.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b)); return r;
}
__device__ __forceinline__ float set_ge(float a, float b) {   // 1.0f if a >= b else 0.0f (0 for NaN)
    float r; asm("set.ge.f32.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b)); return r;
}

// Grid cell of a value: floor(M * sat((g + alpha) * inv_2alpha)), returned as a float whose BIT
// PATTERN is that integer (a denormal).  Monotone in g; NaN maps to cell 0.  The same expression is
// evaluated on the host (cell_of below) when the grid resolution is chosen.
__device__ __forceinline__ float grid_cell(float g, float alpha, float inv_2alpha, float cell_scale) {
    return __fmul_rd(mul_sat(__fadd_rn(g, alpha), inv_2alpha), cell_scale);
}

// [r < T] as 1.0f / 0.0f, where T = rint(p * 2^16) and rf = 2^23 + r.  Both operands of the subtract
// are integers below 2^24, so the difference is exact; huge or infinite p saturate correctly and a
// NaN gives 0.
__device__ __forceinline__ float rounds_up(float p, float rf) {
    return sub_sat(__fmaf_rn(p, 65536.0f, kMagic), rf);
}

// Uniform codebook, l_k = -alpha + k * 2 alpha / s (Section 4.1), two elements at a time.  Reference
// form of the decision: t = clip(g), x = (t + alpha) * inv_step, k = min(floor x, s-1), p = x - k,
// T = rint(p * 2^16), code = k + [r < T].
//
// Computed here through the single integer X = rint(x * 2^16): since k * 2^16 is an integer,
// X = k * 2^16 + T (a carry when T = 2^16 is the next interval with T = 0, the same code), and
// code = k + [r < T] = ceil((X - r) / 2^16) for 0 <= r < 2^16.  With L = s + 1 a power of two:
//   sum = g + alpha                            (as the reference; for |g| <= alpha it is t + alpha)
//   y   = sat(sum * (inv_step / L))            = clip(x, 0, L) / L exactly: scaling by a power of two commutes
//                                                with the rounding of the product, and .sat sends NaN and
//                                                negatives to 0, which is where the reference sends them
//   y   = min(y, s/L)                          this is x = s, which the reference codes as s, like every g >= alpha
//   Xm  = fma(y, L * 2^16, 2^23)               = 2^23 + X, rounded to nearest-even as rint does (2^23 is even)
//   v   = Xm - (2^23 + r)                      = X - r, exact
//   cm  = fma.rp(v, 2^-16, 1.5 * 2^23)         = 1.5 * 2^23 + ceil(v / 2^16): the sum stays inside one binade
// and the caller subtracts the bias.  sum0 / sum1 are g + alpha of the pair.
struct UniformQ {
    float inv_step_l, c_top;      // inv_step / L, s / L
    f32x2 scale2;                 // L * 2^16, twice
    f32x2 scale2_dn;              // L * 2^16 * 2^-100, twice (codes as denormals, see code_uniform2_dn)
};
constexpr float kCodeBias = 12582912.0f;                 // 1.5 * 2^23
__device__ __forceinline__ f32x2 fma2_ru(f32x2 a, f32x2 b, f32x2 c) {   // round toward +infinity
    f32x2 r; asm("fma.rp.f32x2 %0, %1, %2, %3;" : "=l"(r.v) : "l"(a.v), "l"(b.v), "l"(c.v)); return r;
}
__device__ __forceinline__ f32x2 mul2_ru(f32x2 a, f32x2 b) {
    f32x2 r; asm("mul.rp.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v)); return r;
}
// min(y, s/L) runs on the integer/compare pipe, which has room here; the multiply-add pipes do not.
__device__ __forceinline__ f32x2 code_uniform2(float sum0, float sum1, const UniformQ& u, float rf0, float rf1) {
    const f32x2 y = pair(fminf(mul_sat(sum0, u.inv_step_l), u.c_top), fminf(mul_sat(sum1, u.inv_step_l), u.c_top));
    const f32x2 v = sub2(fma2(y, u.scale2, both(kMagic)), pair(rf0, rf1));
    return fma2_ru(v, both(1.52587890625e-5f), both(kCodeBias));
}
// The same with everything scaled by 2^-100: Xm = fma(y, L * 2^16 * 2^-100, 2^-77) = 2^-77 + X * 2^-100 (rounded
// at 2^-100 exactly as the unscaled form rounds at 1), the slot arrives as 2^-77 + r * 2^-100, and
// (X - r) * 2^-100 * 2^-65 rounded up is ceil((X - r) / 2^16) * 2^-149: a denormal whose bit pattern is the code
// itself, with no bias to take off (or -0 when X < r: pack8_bits' callers drop the sign bit).
constexpr uint32_t kSlotExpBits = 0x19000000u;            // 2^-77
__device__ __forceinline__ f32x2 code_uniform2_dn(float sum0, float sum1, const UniformQ& u, float rf0, float rf1) {
    const f32x2 y = pair(fminf(mul_sat(sum0, u.inv_step_l), u.c_top), fminf(mul_sat(sum1, u.inv_step_l), u.c_top));
    const f32x2 v = sub2(fma2(y, u.scale2_dn, both(6.617444900424222e-24f)), pair(rf0, rf1));
    return mul2_ru(v, both(2.710505431213761e-20f));     // 2^-65
}

// The same decision without the scaled inverse step (alpha so large that inv_step / L is subnormal):
// x = clip((g + alpha) * inv_step, 0, s), k' = floor x, p' = x - k'; at x = s this yields k' = s, p' = 0,
// i.e. the same code s as k = s-1, p >= 1.  NaN becomes 0 (fmaxf drops it).  Returns the plain code.
__device__ __forceinline__ f32x2 code_uniform2_wide(float sum0, float sum1, f32x2 inv_step2, float top, float rf0, float rf1) {
    float x0, x1;
    unpair(mul2(pair(sum0, sum1), inv_step2), x0, x1);
    const f32x2 x = pair(fminf(fmaxf(x0, 0.0f), top), fminf(fmaxf(x1, 0.0f), top));
    const f32x2 magic2 = both(kMagic);
    const f32x2 kf = sub2(add2_rd(x, magic2), magic2);                       // floor(x), exact
    float pm0, pm1;
    unpair(fma2(sub2(x, kf), both(65536.0f), magic2), pm0, pm1);            // 2^23 + rint(p * 2^16)
    return add2(kf, pair(sub_sat(pm0, rf0), sub_sat(pm1, rf1)));
}

// g + alpha for elements 2h and 2h+1 of a loaded group.  bf16 storage: the widening is part of the add
// (the stored 16 bits are an exact fp32 value, so the sum rounds as the fp32 add of the widened value).
template <bool BF16>
__device__ __forceinline__ void pair_plus_alpha(const Raw8<BF16>& g, int h, float alpha, float& sum0, float& sum1) {
    if constexpr (BF16) {
        asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %2;\n\tadd.rn.f32.bf16 %0, lo, %3;\n\tadd.rn.f32.bf16 %1, hi, %3;\n\t}"
            : "=f"(sum0), "=f"(sum1) : "r"(g.v[h]), "f"(alpha));
    } else {
        unpair(add2(pair(__uint_as_float(g.v[2 * h]), __uint_as_float(g.v[2 * h + 1])), both(alpha)), sum0, sum1);
    }
}

// General codebook through the lookup grid, two elements at a time.  s_grid[c] = (boundary, k_lo): k_lo
// counts the interior levels in cells below c and `boundary` is the one interior level inside cell c
// (NaN if none, so that not even +inf compares >= it), so
// k = k_lo + [g >= boundary] = max{ j <= s-1 : l_j <= g }.  s_cell[k] = (l_k, 1/|Delta_k|).
// g is not clipped first: beyond +-alpha the same interval is found as for the clipped value, and
// p >= 1 (or p < 0, or NaN) saturates to the same decision.
__device__ __forceinline__ f32x2 code_grid2(float g0, float g1, f32x2 alpha2, float inv_2alpha, f32x2 cell_scale2,
                                            const char* s_grid, const char* s_cell, float rf0, float rf1) {
    const f32x2 g = pair(g0, g1);
    float s0, s1;
    unpair(add2(g, alpha2), s0, s1);
    // cell = floor(M * sat((g + alpha) * inv_2alpha)) as a denormal whose bit pattern is the integer; * 8 = byte offset
    const f32x2 cell8 = mul2(mul2_rd(pair(mul_sat(s0, inv_2alpha), mul_sat(s1, inv_2alpha)), cell_scale2), both(8.0f));
    float c0, c1;
    unpair(cell8, c0, c1);
    const float2 gc0 = *reinterpret_cast<const float2*>(s_grid + __float_as_uint(c0));
    const float2 gc1 = *reinterpret_cast<const float2*>(s_grid + __float_as_uint(c1));
    const f32x2 kf = add2(pair(gc0.y, gc1.y), pair(set_ge(g0, gc0.x), set_ge(g1, gc1.x)));
    float k0, k1;
    unpair(mul2(kf, both(__uint_as_float(8u))), k0, k1);                     // bits = 8 * k
    const float2 q0 = *reinterpret_cast<const float2*>(s_cell + __float_as_uint(k0));
    const float2 q1 = *reinterpret_cast<const float2*>(s_cell + __float_as_uint(k1));
    const f32x2 p = mul2(sub2(g, pair(q0.x, q1.x)), pair(q0.y, q1.y));
    float pm0, pm1;
    unpair(fma2(p, both(65536.0f), both(kMagic)), pm0, pm1);
    return add2(kf, pair(sub_sat(pm0, rf0), sub_sat(pm1, rf1)));
}

// General codebook by branch-free binary search (used when no grid of at most kMaxGridCells cells
// separates the levels): search[] holds l_1 .. l_{s-1} at indices 1 .. s-1 and +inf from index s on.
template <int BITS>
__device__ __forceinline__ float code_binary(float g, float alpha, const float* search, const float2* cell, float rf) {
    const float t = fminf(fmaxf(g, -alpha), alpha);   // NaN -> -alpha
    uint32_t k = 0;
#pragma unroll
    for (int step = (1 << BITS) >> 1; step > 0; step >>= 1)
        if (t >= search[k + step]) k += step;
    const float2 c = cell[k];
    const float p = __fmul_rn(__fsub_rn(t, c.x), c.y);
    return __fadd_rn(static_cast<float>(k), rounds_up(p, rf));
}

// Four pairs of float codes (elements 0..7 of a group, each code < 2^BITS) -> their 8*BITS packed
// bits, LSB first.  Every partial sum is an integer below 2^24, so the fp32 arithmetic is exact.
// Returns a word whose low 8*BITS bits are the packed codes.
//
// DN (2- and 4-bit codes only): the codes are denormals whose bit pattern is the code (see
// code_uniform2_dn), sums and products of them are fixed-point arithmetic in units of 2^-149, and the
// packed bits appear as a bit pattern without any float -> integer conversion.  Bits above the low 16 of
// a partial result may be set (a sum of -0 terms is -0): the caller merges chunks by byte-permutes that
// take the low 16 bits only.
template <int BITS, bool DN>
__device__ __forceinline__ uint32_t pack8(const f32x2 (&c)[4]) {
    constexpr float B = static_cast<float>(1 << BITS), B2 = B * B;
    static_assert(!DN || BITS == 2 || BITS == 4, "the callers of the denormal form keep 16 bits of each partial result");
    if constexpr (BITS <= 3) {
        f32x2 a = fma2(c[3], both(B2), c[2]);
        a = fma2(a, both(B2), c[1]);
        a = fma2(a, both(B2), c[0]);
        float ev, od;
        unpair(a, ev, od);
        if constexpr (DN) return __float_as_uint(__fmaf_rn(od, B, ev));
        else return __float2uint_rz(__fmaf_rn(od, B, ev));
    } else {
        float e0, o0, e1, o1;
        unpair(fma2(c[1], both(B2), c[0]), e0, o0);       // elements 0..3: 16 bits
        unpair(fma2(c[3], both(B2), c[2]), e1, o1);       // elements 4..7: 16 bits
        if constexpr (DN)
            return __byte_perm(__float_as_uint(__fmaf_rn(o0, B, e0)), __float_as_uint(__fmaf_rn(o1, B, e1)), 0x5410u);
        else return __float2uint_rz(__fmaf_rn(o0, B, e0)) + (__float2uint_rz(__fmaf_rn(o1, B, e1)) << 16);
    }
}

struct RunCtx {
    float alpha, inv_step, top, inv_2alpha, cell_scale;
    UniformQ u;
    const char* s_grid; const char* s_cell; const float* s_search;
};

template <int BITS>
__device__ __forceinline__ UniformQ uniform_q(const WorkerQ& q) {
    constexpr float L = static_cast<float>(1 << BITS);
    return UniformQ{q.inv_step_l, (L - 1.0f) / L, both(L * 65536.0f), both(L * 65536.0f * 7.888609052210118e-31f)};
}

// inv_step / L for the scaled uniform path: exact when the quotient is a normal number (L is a power of
// two); 0 tells the launch to use the unscaled arithmetic instead.  Same expression on host and device.
__host__ __device__ inline float scaled_inv_step(float inv_step, uint32_t num_levels) {
    const float q = inv_step / static_cast<float>(num_levels);
    return (q >= 1.17549435e-38f && q <= 3.402823466e38f) ? q : 0.0f;
}

// the 16 random bits of slot e of a Philox block, as the float 2^23 + r (DN: 2^-77 + r * 2^-100)
template <bool DN>
__device__ __forceinline__ float slot_as_float(const uint32_t (&rnd)[4], int e) {
    return __uint_as_float(__byte_perm(rnd[e >> 1], DN ? kSlotExpBits : kMagicBits, (e & 1) ? 0x7432u : 0x7410u));
}

template <int BITS, int SEARCH, bool BF16, bool TAIL>
__device__ __forceinline__ void quantize_run(const Raw8<BF16> (&g)[4], uint32_t* prow, uint64_t run, uint64_t d, uint64_t words_out,
                                             uint32_t worker, const RoundKeys& rk, const RunCtx& cx);

// One run of 32 elements: load, quantize, pack, store.  TAIL = the last, possibly partial run of a row
// (element-wise guarded loads, zero padding bits, guarded stores and the row's alignment padding).
template <int BITS, int SEARCH, bool BF16, bool TAIL>
__device__ __forceinline__ void compress_run(const char* row, uint32_t* prow, uint64_t run, uint64_t d, uint64_t words_out,
                                             uint32_t worker, const RoundKeys& rk, const RunCtx& cx) {
    constexpr size_t esz = BF16 ? 2 : 4;
    const uint64_t j0 = run << 5;
    Raw8<BF16> g[4];
    if constexpr (!TAIL) {
#pragma unroll
        for (int grp = 0; grp < 4; ++grp) load8_raw<BF16>(row + (j0 + 8 * grp) * esz, g[grp]);
    } else {
#pragma unroll
        for (int grp = 0; grp < 4; ++grp)
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const uint64_t j = j0 + 8 * grp + e;
                set_elem<BF16>(g[grp], e, j < d ? load1<BF16>(row, j) : 0.0f);
            }
    }

    quantize_run<BITS, SEARCH, BF16, TAIL>(g, prow, run, d, words_out, worker, rk, cx);
}

// The arithmetic of one run whose 32 elements are already in registers: quantize, pack, store.
template <int BITS, int SEARCH, bool BF16, bool TAIL>
__device__ __forceinline__ void quantize_run(const Raw8<BF16> (&g)[4], uint32_t* prow, uint64_t run, uint64_t d, uint64_t words_out,
                                             uint32_t worker, const RoundKeys& rk, const RunCtx& cx) {
    const uint64_t j0 = run << 5;
    const uint32_t blk_lo = static_cast<uint32_t>(j0 >> 3);
    const PhiloxRun pr = philox_run(static_cast<uint32_t>(j0 >> 35), worker, rk);
    const f32x2 alpha2 = both(cx.alpha), inv_step2 = both(cx.inv_step), cell_scale2 = both(cx.cell_scale);
    // whole runs of the scaled uniform path hand pack8 the codes as denormals (2- and 4-bit codes)
    constexpr bool DN = SEARCH == kUniform && !TAIL && (BITS == 2 || BITS == 4);
    uint32_t chunk[4];   // the 8*BITS packed bits of each group
#pragma unroll
    for (int grp = 0; grp < 4; ++grp) {
        uint32_t rnd[4];
        philox_block(blk_lo + grp, pr, rk, rnd);                      // j0 >> 3 is a multiple of 4: no carry
        f32x2 code[4];
#pragma unroll
        for (int h = 0; h < 4; ++h) {            // elements 2h, 2h+1 of the group
            const int e = 2 * h;
            const float rf0 = slot_as_float<DN>(rnd, e), rf1 = slot_as_float<DN>(rnd, e + 1);
            if constexpr (is_uniform(SEARCH)) {
                float sum0, sum1;
                pair_plus_alpha<BF16>(g[grp], h, cx.alpha, sum0, sum1);
                if constexpr (DN) code[h] = code_uniform2_dn(sum0, sum1, cx.u, rf0, rf1);
                else if constexpr (SEARCH == kUniform) code[h] = sub2(code_uniform2(sum0, sum1, cx.u, rf0, rf1), both(kCodeBias));
                else code[h] = code_uniform2_wide(sum0, sum1, inv_step2, cx.top, rf0, rf1);
            } else {
                const float g0 = elem<BF16>(g[grp], e), g1 = elem<BF16>(g[grp], e + 1);
                if constexpr (SEARCH == kGrid)
                    code[h] = code_grid2(g0, g1, alpha2, cx.inv_2alpha, cell_scale2, cx.s_grid, cx.s_cell, rf0, rf1);
                else code[h] = pair(code_binary<BITS>(g0, cx.alpha, cx.s_search, reinterpret_cast<const float2*>(cx.s_cell), rf0),
                                    code_binary<BITS>(g1, cx.alpha, cx.s_search, reinterpret_cast<const float2*>(cx.s_cell), rf1));
            }
            if constexpr (TAIL) {                 // padding bits are zero
                float c0, c1;
                unpair(code[h], c0, c1);
                if (j0 + 8 * grp + e >= d) c0 = 0.0f;
                if (j0 + 8 * grp + e + 1 >= d) c1 = 0.0f;
                code[h] = pair(c0, c1);
            }
        }
        chunk[grp] = pack8<BITS, DN>(code);
    }

    // four chunks of 8*BITS bits -> BITS words, LSB first
    uint32_t w[BITS];
    if constexpr (BITS == 4) { w[0] = chunk[0]; w[1] = chunk[1]; w[2] = chunk[2]; w[3] = chunk[3]; }
    if constexpr (BITS == 3) {
        w[0] = chunk[0] | (chunk[1] << 24);
        w[1] = (chunk[1] >> 8) | (chunk[2] << 16);
        w[2] = (chunk[2] >> 16) | (chunk[3] << 8);
    }
    if constexpr (BITS == 2) { w[0] = __byte_perm(chunk[0], chunk[1], 0x5410u); w[1] = __byte_perm(chunk[2], chunk[3], 0x5410u); }
    if constexpr (BITS == 1) { w[0] = chunk[0] | (chunk[1] << 8) | (chunk[2] << 16) | (chunk[3] << 24); }

    uint32_t* dst = prow + run * BITS;
    if constexpr (!TAIL) {   // every word of an interior run lies below words_out
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
        for (uint64_t k = first + BITS; k < words_out; ++k) prow[k] = 0u;
    }
}

#ifndef TQ_COMPRESS_MIN_BLOCKS
#define TQ_COMPRESS_MIN_BLOCKS 4
#endif

// Per-block set-up of the shared tables for quantizer q (ends with a block barrier unless the codebook is uniform).
// s_grid must hold kMaxGridCells + 1 entries when SEARCH == kGrid.
template <int BITS, int SEARCH>
__device__ __forceinline__ void build_tables(const WorkerQ& q, float2* s_grid, float2* s_cell, float* s_search) {
    constexpr int L = 1 << BITS;
    if constexpr (!is_uniform(SEARCH)) {
        if (threadIdx.x < L - 1) s_cell[threadIdx.x] = make_float2(q.levels[threadIdx.x], q.inv_width[threadIdx.x]);
    }
    if constexpr (SEARCH == kBinary) {
        if (threadIdx.x < 2 * TQ_MAX_LEVELS)
            s_search[threadIdx.x] = (threadIdx.x >= 1 && threadIdx.x <= L - 2) ? q.levels[threadIdx.x] : __int_as_float(0x7F800000);
    }
    if constexpr (SEARCH == kGrid) {
        // cells of the interior levels l_1 .. l_{s-1} (distinct by the choice of M)
        uint32_t lc[L];
#pragma unroll
        for (int j = 1; j <= L - 2; ++j)
            lc[j] = __float_as_uint(grid_cell(q.levels[j], q.alpha, q.inv_2alpha, q.cell_scale));
        for (uint32_t c = threadIdx.x; c <= q.cells; c += kThreads) {
            float below = 0.0f, boundary = __int_as_float(0x7FC00000);   // NaN: no value compares >= it
#pragma unroll
            for (int j = 1; j <= L - 2; ++j) {
                if (lc[j] < c) below += 1.0f;
                if (lc[j] == c) boundary = q.levels[j];
            }
            s_grid[c] = make_float2(boundary, below);
        }
    }
    if constexpr (!is_uniform(SEARCH)) __syncthreads();
}

// Per-block set-up of the shared tables for quantizer q, then the block's share of the runs of one row
// (`row`: its first gradient element, `prow`: its first packed word).
// s_grid must hold kMaxGridCells + 1 entries when SEARCH == kGrid.
template <int BITS, int SEARCH, bool BF16>
__device__ __forceinline__ void compress_row(const WorkerQ& q, float2* s_grid, float2* s_cell, float* s_search,
                                             const char* __restrict__ row, uint64_t d, const RoundKeys& rk, uint32_t worker,
                                             uint32_t* __restrict__ prow, uint64_t words_out) {
    build_tables<BITS, SEARCH>(q, s_grid, s_cell, s_search);

    const uint64_t n_runs = (d + 31) >> 5;
    const RunCtx cx{q.alpha, q.inv_step, q.top, q.inv_2alpha, q.cell_scale, uniform_q<BITS>(q), reinterpret_cast<const char*>(s_grid),
                    reinterpret_cast<const char*>(s_cell), s_search};
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * kThreads;

    uint64_t run = static_cast<uint64_t>(blockIdx.x) * kThreads + threadIdx.x;
    const uint64_t interior = n_runs - 1;      // every run before the row's last one is full
    for (; run < interior; run += stride)
        compress_run<BITS, SEARCH, BF16, false>(row, prow, run, d, words_out, worker, rk, cx);
    if (run == n_runs - 1)
        compress_run<BITS, SEARCH, BF16, true>(row, prow, run, d, words_out, worker, rk, cx);
}

// The same for worker wi's row of a [N][grad_stride] block and its row of the [N][words_stride] output.
template <int BITS, int SEARCH, bool BF16>
__device__ __forceinline__ void compress_block(const WorkerQ& q, float2* s_grid, float2* s_cell, float* s_search,
                                               const void* __restrict__ grad, uint64_t d, uint64_t grad_stride,
                                               const RoundKeys& rk, uint32_t worker, uint32_t wi,
                                               uint32_t* __restrict__ packed, uint64_t words_stride, uint64_t words_out) {
    constexpr size_t esz = BF16 ? 2 : 4;
    compress_row<BITS, SEARCH, BF16>(q, s_grid, s_cell, s_search,
                                     static_cast<const char*>(grad) + static_cast<uint64_t>(wi) * grad_stride * esz, d, rk, worker,
                                     packed + static_cast<uint64_t>(wi) * words_stride, words_out);
}

// Quantizers passed by value in the kernel's parameter space (host-side tq_params).
template <int BITS, int SEARCH, bool BF16>
__global__ void __launch_bounds__(kThreads, TQ_COMPRESS_MIN_BLOCKS)
compress_kernel(const void* __restrict__ grad, uint64_t d, uint64_t grad_stride,
                const __grid_constant__ CompressArgs args, const __grid_constant__ RoundKeys rk,
                uint32_t first_worker, uint32_t* __restrict__ packed, uint64_t words_stride, uint64_t words_out) {
    __shared__ __align__(16) float2 s_grid[SEARCH == kGrid ? kMaxGridCells + 1 : 1];
    __shared__ __align__(16) float2 s_cell[TQ_MAX_LEVELS];
    __shared__ float s_search[2 * TQ_MAX_LEVELS];
    const uint32_t wi = blockIdx.y;
    compress_block<BITS, SEARCH, BF16>(args.q[wi], s_grid, s_cell, s_search, grad, d, grad_stride, rk, first_worker + wi, wi,
                                       packed, words_stride, words_out);
}

// ---------------------------------------------------------------------------------------------
// Table-mode compress with the gradient tiles brought in by the tensor-memory accelerator.
// A tile is 256 runs of 32 elements (one run per thread).  Thread 0 asks for the block's next tile as
// ONE tiled copy ({32 elements, 256 runs, 1 worker} of the [N][runs][32] view of the gradient) while
// the block is still quantizing the current one, so no warp waits on global loads and no registers are
// held by loads in flight.  The copy lands swizzled (16-byte chunk c of run r at chunk c ^ (r & 7) for
// 128-byte runs, c ^ ((r >> 1) & 3) for 64-byte runs), which makes a thread's reads of its own run
// conflict-free.  Runs past the last whole run read as zeros and are not used; the row's last run
// (possibly partial) goes through the guarded path.  Waits are bounded as in the header.
__device__ unsigned int g_compress_wait_expired = 0;

__device__ __forceinline__ void lds128(uint32_t addr, uint32_t& a, uint32_t& b, uint32_t& c, uint32_t& d) {
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(a), "=r"(b), "=r"(c), "=r"(d) : "r"(addr));
}

__device__ __forceinline__ void tma_load_tile(uint32_t dst, const CUtensorMap* map, int32_t x, int32_t y, int32_t z, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}

template <int BITS, bool BF16>
__global__ void __launch_bounds__(kThreads, TQ_COMPRESS_MIN_BLOCKS)
compress_tma_kernel(const __grid_constant__ CUtensorMap tmap, const void* __restrict__ grad, uint64_t d, uint64_t grad_stride,
                    const __grid_constant__ CompressArgs args, const __grid_constant__ RoundKeys rk,
                    uint32_t first_worker, uint32_t* __restrict__ packed, uint64_t words_stride, uint64_t words_out) {
    constexpr uint32_t kRowBytes = 32 * (BF16 ? 2 : 4), kTileBytes = kThreads * kRowBytes;
    __shared__ __align__(16) float2 s_grid[kMaxGridCells + 1];
    __shared__ __align__(16) float2 s_cell[TQ_MAX_LEVELS];
    extern __shared__ __align__(1024) unsigned char s_tile[];        // kTileBytes, then the barrier
    const uint32_t wi = blockIdx.y;
    const WorkerQ& q = args.q[wi];
    const uint32_t tile0 = smem_addr(s_tile), bar = tile0 + kTileBytes;

    const uint64_t n_runs = (d + 31) >> 5;
    const uint64_t interior = n_runs - 1;                             // every run before the row's last one is whole
    const uint32_t n_tiles = static_cast<uint32_t>((interior + kThreads - 1) / kThreads);
    uint32_t tile = blockIdx.x;
    auto issue = [&](uint32_t t) {
        mbar_expect_tx(bar, kTileBytes);
        tma_load_tile(tile0, &tmap, 0, static_cast<int32_t>(t * kThreads), static_cast<int32_t>(wi), bar);
    };
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (tile < n_tiles) issue(tile);
    }
    build_tables<BITS, kGrid>(q, s_grid, s_cell, nullptr);            // ends with a block barrier

    constexpr size_t esz = BF16 ? 2 : 4;
    const char* row = static_cast<const char*>(grad) + static_cast<uint64_t>(wi) * grad_stride * esz;
    uint32_t* prow = packed + static_cast<uint64_t>(wi) * words_stride;
    const RunCtx cx{q.alpha, q.inv_step, q.top, q.inv_2alpha, q.cell_scale, uniform_q<BITS>(q), reinterpret_cast<const char*>(s_grid),
                    reinterpret_cast<const char*>(s_cell), nullptr};
    // this thread's run starts at tile0 + tid * kRowBytes; its 16-byte chunk c sits at chunk c ^ sw: the chunk
    // bits of the run's own address are zero, so the address of chunk c is (run | sw << 4) ^ (c << 4)
    const uint32_t sw = BF16 ? ((threadIdx.x >> 1) & 3u) : (threadIdx.x & 7u);
    const uint32_t mine0 = (tile0 + threadIdx.x * kRowBytes) | (sw << 4);

    uint32_t parity = 0;
    bool expired = false;
    for (; tile < n_tiles; tile += gridDim.x) {
        const bool ok = mbar_wait(bar, parity);
        parity ^= 1u;
        const uint64_t run = static_cast<uint64_t>(tile) * kThreads + threadIdx.x;
        Raw8<BF16> g[4];         // read even if the wait ran out: the values are then never used
#pragma unroll
        for (int grp = 0; grp < 4; ++grp) {
            if constexpr (BF16) {
                lds128(mine0 ^ (static_cast<uint32_t>(grp) << 4), g[grp].v[0], g[grp].v[1], g[grp].v[2], g[grp].v[3]);
            } else {
                lds128(mine0 ^ (static_cast<uint32_t>(2 * grp) << 4), g[grp].v[0], g[grp].v[1], g[grp].v[2], g[grp].v[3]);
                lds128(mine0 ^ (static_cast<uint32_t>(2 * grp + 1) << 4), g[grp].v[4], g[grp].v[5], g[grp].v[6], g[grp].v[7]);
            }
        }
        // every thread has its run in registers: the tile buffer may be refilled.  The same barrier
        // makes the give-up decision uniform.
        if (__syncthreads_or(!ok)) { expired = true; break; }
        if (threadIdx.x == 0 && tile + gridDim.x < n_tiles) issue(tile + gridDim.x);
        if (run < interior) quantize_run<BITS, kGrid, BF16, false>(g, prow, run, d, words_out, first_worker + wi, rk, cx);
    }
    if (expired) {
        atomicAdd(&g_compress_wait_expired, 1u);
        if (threadIdx.x == 0) mbar_wait(bar, parity ^ 1u);            // the copy that did not land in time
        return;
    }
    // the row's last run, by the thread that the striding would have given it to
    if ((interior / kThreads) % gridDim.x == blockIdx.x && interior % kThreads == threadIdx.x)
        compress_run<BITS, kGrid, BF16, true>(row, prow, interior, d, words_out, first_worker + wi, rk, cx);
}

cudaError_t read_compress_wait_expired(unsigned int* count) {
    return cudaMemcpyFromSymbol(count, g_compress_wait_expired, sizeof(unsigned int));
}

// The grid cell of a value as a plain integer (device copy of the host's cell_of).
__device__ __forceinline__ uint32_t cell_index(float g, float alpha, float inv_2alpha, uint32_t cells) {
    return __float_as_uint(grid_cell(g, alpha, inv_2alpha, __uint_as_float(cells)));   // M * 2^-149 has bit pattern M
}

// Quantizers read from device memory (tq_params_device): no host round trip before the launch.
// Thread 0 turns worker wi's tq_params_t into the kernel's WorkerQ, including the choice of the lookup
// grid.  Returns false when this block has nothing to do in a kernel of kind FALLBACK:
//   FALLBACK = false (main kernel): uniform rows, rows with a lookup grid, and all-zero rows for workers
//              marked invalid (alpha = 0);
//   FALLBACK = true: only the rows whose levels no grid separates (binary search).  It is launched
//              after the main kernel and its blocks return at once for every other row, so the rarely
//              needed path costs one near-empty launch instead of registers in the main kernel.
template <int BITS, bool NONUNIFORM>
__device__ __forceinline__ void load_worker(const tq_params_t* __restrict__ params, uint32_t wi, WorkerQ& s_q) {
    if (threadIdx.x < TQ_MAX_LEVELS) {
        s_q.levels[threadIdx.x] = params[wi].levels[threadIdx.x];
        s_q.inv_width[threadIdx.x] = params[wi].inv_width[threadIdx.x];
    }
    __syncthreads();                 // the levels are in shared memory from here on
    if (threadIdx.x == 0) {
        const tq_params_t& p = params[wi];
        const float alpha = p.alpha;
        const bool ok = alpha > 0.0f && p.bits == BITS && !(p.flags & TQ_FLAG_INVALID);
        const float inv_2alpha = ok ? __fdiv_rn(1.0f, __fmul_rn(2.0f, alpha)) : 0.0f;
        s_q.alpha = ok ? alpha : 0.0f;
        s_q.inv_step = p.inv_step;
        s_q.inv_step_l = scaled_inv_step(p.inv_step, 1u << BITS);
        s_q.top = static_cast<float>((1 << BITS) - 1);
        s_q.inv_2alpha = inv_2alpha;
        uint32_t cells = 0;
        if (NONUNIFORM && ok && inv_2alpha <= 3.402823466e38f) {
            constexpr int s = (1 << BITS) - 1;
            for (uint32_t m = kMinGridCells; m <= static_cast<uint32_t>(kMaxGridCells) && cells == 0; m *= 2) {
                bool distinct = true;
                uint32_t prev = s >= 2 ? cell_index(s_q.levels[1], alpha, inv_2alpha, m) : 0u;
#pragma unroll
                for (int j = 2; j <= s - 1; ++j) {
                    const uint32_t cur = cell_index(s_q.levels[j], alpha, inv_2alpha, m);
                    distinct = distinct && cur > prev;
                    prev = cur;
                }
                if (distinct) cells = m;
            }
        }
        s_q.cells = cells;
        s_q.cell_scale = __uint_as_float(cells);
    }
    __syncthreads();
}

// Where a job's row and packed words are.  Without segments job wi is worker wi and its whole slice; with
// segments it is the pair (worker, segment) = (wi / n, wi % n) and a piece of that worker's row.
struct JobPlace {
    const char* row; uint32_t* prow; uint64_t d, words_out; uint32_t worker;
};
template <int BITS, bool BF16>
__device__ __forceinline__ JobPlace place_job(uint32_t wi, const void* grad, uint64_t d, uint64_t grad_stride, uint32_t first_worker,
                                              uint32_t* packed, uint64_t words_stride, uint64_t words_out, const SegTable& segs) {
    constexpr size_t esz = BF16 ? 2 : 4;
    if (segs.n == 0)
        return JobPlace{static_cast<const char*>(grad) + static_cast<uint64_t>(wi) * grad_stride * esz,
                        packed + static_cast<uint64_t>(wi) * words_stride, d, words_out, first_worker + wi};
    const uint32_t w = wi / segs.n, sg = wi - w * segs.n;
    const uint64_t len = segs.len[sg];
    return JobPlace{static_cast<const char*>(grad) + (static_cast<uint64_t>(w) * grad_stride + segs.off[sg]) * esz,
                    packed + static_cast<uint64_t>(w) * words_stride + segs.woff[sg], len,
                    (((len * BITS + 31) >> 5) + 3) & ~static_cast<uint64_t>(3), first_worker + w};
}

template <int BITS, bool NONUNIFORM, bool BF16>
__global__ void __launch_bounds__(kThreads, TQ_COMPRESS_MIN_BLOCKS)
compress_kernel_dev(const void* __restrict__ grad, uint64_t d, uint64_t grad_stride,
                    const tq_params_t* __restrict__ params, const __grid_constant__ RoundKeys rk,
                    uint32_t first_worker, uint32_t* __restrict__ packed, uint64_t words_stride, uint64_t words_out,
                    const __grid_constant__ SegTable segs, int table_kernel_ran) {
    if (table_kernel_ran) {          // rows the decision-table kernel served are done (same rule, evaluated by every thread)
        uint32_t top, base;
        if (lut_serves_record(params[blockIdx.y], BITS, &top, &base)) return;
    }
    __shared__ __align__(16) float2 s_grid[NONUNIFORM ? kMaxGridCells + 1 : 1];
    __shared__ __align__(16) float2 s_cell[TQ_MAX_LEVELS];
    __shared__ float s_search[2 * TQ_MAX_LEVELS];
    __shared__ WorkerQ s_q;
    const uint32_t wi = blockIdx.y;
    const JobPlace job = place_job<BITS, BF16>(wi, grad, d, grad_stride, first_worker, packed, words_stride, words_out, segs);
    load_worker<BITS, NONUNIFORM>(params, wi, s_q);
    if (!(s_q.alpha > 0.0f)) {       // invalid parameters: the row is all code 0
        for (uint64_t w = static_cast<uint64_t>(blockIdx.x) * kThreads + threadIdx.x; w < job.words_out;
             w += static_cast<uint64_t>(gridDim.x) * kThreads)
            job.prow[w] = 0u;
        return;
    }
    if constexpr (NONUNIFORM) {
        if (s_q.cells == 0) return;  // left to compress_kernel_dev_fallback
    }
    if constexpr (!NONUNIFORM) {
        if (s_q.inv_step_l == 0.0f) {    // alpha too large for the scaled inverse step
            compress_row<BITS, kUniformWide, BF16>(s_q, s_grid, s_cell, s_search, job.row, job.d, rk, job.worker, job.prow, job.words_out);
            return;
        }
    }
    compress_row<BITS, NONUNIFORM ? kGrid : kUniform, BF16>(s_q, s_grid, s_cell, s_search, job.row, job.d, rk, job.worker, job.prow,
                                                            job.words_out);
}

template <int BITS, bool BF16>
__global__ void __launch_bounds__(kThreads, TQ_COMPRESS_MIN_BLOCKS)
compress_kernel_dev_fallback(const void* __restrict__ grad, uint64_t d, uint64_t grad_stride,
                             const tq_params_t* __restrict__ params, const __grid_constant__ RoundKeys rk,
                             uint32_t first_worker, uint32_t* __restrict__ packed, uint64_t words_stride, uint64_t words_out,
                             const __grid_constant__ SegTable segs, int table_kernel_ran) {
    if (table_kernel_ran) {
        uint32_t top, base;
        if (lut_serves_record(params[blockIdx.y], BITS, &top, &base)) return;
    }
    __shared__ __align__(16) float2 s_grid[1];
    __shared__ __align__(16) float2 s_cell[TQ_MAX_LEVELS];
    __shared__ float s_search[2 * TQ_MAX_LEVELS];
    __shared__ WorkerQ s_q;
    const uint32_t wi = blockIdx.y;
    const JobPlace job = place_job<BITS, BF16>(wi, grad, d, grad_stride, first_worker, packed, words_stride, words_out, segs);
    load_worker<BITS, true>(params, wi, s_q);
    if (!(s_q.alpha > 0.0f) || s_q.cells != 0) return;
    compress_row<BITS, kBinary, BF16>(s_q, s_grid, s_cell, s_search, job.row, job.d, rk, job.worker, job.prow, job.words_out);
}

// ---- host side ---------------------------------------------------------------------------------------

// The grid cell of a value, exactly as grid_cell() computes it on the device: every step is a single
// IEEE operation (u * M is exact for M a power of two), so host and device agree bit for bit.
static uint32_t cell_of(float g, float alpha, float inv_2alpha, uint32_t cells) {
    float u = (g + alpha) * inv_2alpha;
    u = !(u > 0.0f) ? 0.0f : (u > 1.0f ? 1.0f : u);
    return static_cast<uint32_t>(std::floor(u * static_cast<float>(cells)));
}

// Smallest power-of-two grid (32 .. 2048 cells) that puts the interior levels in distinct cells; 0 if none.
static uint32_t choose_cells(const tq_params_t& p, float inv_2alpha) {
    const int s = static_cast<int>(p.num_levels) - 1;
    for (uint32_t m = kMinGridCells; m <= static_cast<uint32_t>(kMaxGridCells); m *= 2) {
        bool distinct = true;
        for (int j = 2; j <= s - 1 && distinct; ++j)
            distinct = cell_of(p.levels[j], p.alpha, inv_2alpha, m) > cell_of(p.levels[j - 1], p.alpha, inv_2alpha, m);
        if (distinct) return m;
    }
    return 0;
}

// Persistent grid: 4 resident blocks per SM spread over the workers (table modes build their lookup
// grid once per block); uniform mode has no per-block set-up, so one block per tile lets the hardware
// scheduler balance the tail.
static dim3 compress_grid(uint64_t d, uint32_t n_workers, bool persistent) {
    const uint64_t n_runs = (d + 31) >> 5;
    const uint64_t tiles = (n_runs + kThreads - 1) / kThreads;
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    uint64_t per_worker = static_cast<uint64_t>(sms) * TQ_COMPRESS_MIN_BLOCKS / n_workers;   // rounded down: one wave holds the grid
    if (!persistent || per_worker > tiles) per_worker = tiles;
    if (per_worker > 0x7FFFFFFFull) per_worker = 0x7FFFFFFFull;
    if (per_worker < 1) per_worker = 1;
    return dim3(static_cast<unsigned>(per_worker), n_workers);
}

template <int BITS, int SEARCH, bool BF>
static cudaError_t launch(const CompressCall& c, const CompressArgs& args, dim3 grid) {
    compress_kernel<BITS, SEARCH, BF><<<grid, kThreads, 0, c.stream>>>(
        c.grad, c.d, c.grad_stride, args, round_keys(c.seed), c.first_worker, c.packed, c.words_stride, c.words_out);
    return cudaGetLastError();
}

// ---- tiled copies: the tensor map of the gradient, [N][whole runs][32 elements] ------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static const EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult how;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &how) != cudaSuccess ||
            how != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// Inputs below this many elements per row keep the kernel that loads straight into registers.
constexpr uint64_t kTmaMinElements = 1u << 16;

// The map copies raw 32- or 16-bit words (no floating-point interpretation), rows past the last whole
// run read as zeros.  Returns false when the tiled path does not apply (then the direct kernel runs).
static bool make_tile_map(const CompressCall& c, CUtensorMap* map) {
    const EncodeTiledFn encode = encode_tiled_fn();
    const uint64_t whole = c.d / 32;
    if (!encode || c.d < kTmaMinElements || whole > 0x7FFFFF00ull) return false;
    const uint64_t esz = c.bf16 ? 2 : 4;
    const cuuint64_t gdim[3] = {32, whole, c.n_workers};
    const cuuint64_t row_pitch = c.n_workers > 1 ? c.grad_stride * esz : whole * 32 * esz;
    const cuuint64_t gstride[2] = {32 * esz, row_pitch};              // bytes between runs, between workers
    if (row_pitch % 16 != 0 || row_pitch >= (1ull << 40)) return false;
    const cuuint32_t box[3] = {32, static_cast<cuuint32_t>(kThreads), 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = encode(map, c.bf16 ? CU_TENSOR_MAP_DATA_TYPE_UINT16 : CU_TENSOR_MAP_DATA_TYPE_UINT32, 3,
                              const_cast<void*>(c.grad), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                              c.bf16 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

template <int BITS, bool BF>
static cudaError_t launch_tma(const CompressCall& c, const CompressArgs& args, dim3 grid, const CUtensorMap& map) {
    const int smem = kThreads * 32 * (BF ? 2 : 4) + 16;
    const cudaError_t e = cudaFuncSetAttribute(compress_tma_kernel<BITS, BF>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    compress_tma_kernel<BITS, BF><<<grid, kThreads, smem, c.stream>>>(
        map, c.grad, c.d, c.grad_stride, args, round_keys(c.seed), c.first_worker, c.packed, c.words_stride, c.words_out);
    return cudaGetLastError();
}

template <int BITS>
static cudaError_t dispatch(const CompressCall& c, const CompressArgs& a, dim3 grid, int search) {
    // Tiled copies pay for bf16 rows (3 % faster at 124 M x 8: half the bytes per element, so the wait for
    // global loads weighs more); for fp32 rows the kernel is bound by instruction issue and the extra
    // shared-memory reads and the barrier per tile cost 2-3 %, so those keep the direct kernel.
    if (search == kGrid && c.bf16) {
        alignas(64) CUtensorMap map;
        if (make_tile_map(c, &map)) return launch_tma<BITS, true>(c, a, grid, map);
    }
    if (search == kGrid) return c.bf16 ? launch<BITS, kGrid, true>(c, a, grid) : launch<BITS, kGrid, false>(c, a, grid);
    if (search == kBinary) return c.bf16 ? launch<BITS, kBinary, true>(c, a, grid) : launch<BITS, kBinary, false>(c, a, grid);
    if (search == kUniformWide) return c.bf16 ? launch<BITS, kUniformWide, true>(c, a, grid) : launch<BITS, kUniformWide, false>(c, a, grid);
    return c.bf16 ? launch<BITS, kUniform, true>(c, a, grid) : launch<BITS, kUniform, false>(c, a, grid);
}

cudaError_t launch_compress(const CompressCall& c) {
    if (c.d == 0 && !c.segs) return cudaSuccess;
    if (c.params_dev) return launch_compress_dev(c);
    {
        bool applied = false;
        const cudaError_t e = launch_compress_lut(c, &applied);
        if (applied || e != cudaSuccess) return e;
    }
    static thread_local CompressArgs args;   // 9 KB: keep it off the stack
    int search = c.nonuniform ? kGrid : kUniform;
    for (uint32_t i = 0; i < c.n_workers; ++i) {
        const tq_params_t& p = c.params[i];
        WorkerQ& q = args.q[i];
        q.alpha = p.alpha; q.inv_step = p.inv_step; q.top = static_cast<float>(p.num_levels - 1);
        q.inv_2alpha = 1.0f / (2.0f * p.alpha);
        q.inv_step_l = scaled_inv_step(p.inv_step, p.num_levels);
        if (!c.nonuniform && q.inv_step_l == 0.0f) search = kUniformWide;
        q.cells = 0; q.cell_scale = 0.0f;
        for (int k = 0; k < TQ_MAX_LEVELS; ++k) { q.levels[k] = p.levels[k]; q.inv_width[k] = p.inv_width[k]; }
        if (c.nonuniform) {
            q.cells = choose_cells(p, q.inv_2alpha);
            q.cell_scale = std::ldexp(static_cast<float>(q.cells), -149);
            if (q.cells == 0 || !std::isfinite(q.inv_2alpha)) search = kBinary;
        }
    }
    const dim3 grid = compress_grid(c.d, c.n_workers, !is_uniform(search));
    switch (c.bits) {
        case 1: return dispatch<1>(c, args, grid, search);
        case 2: return dispatch<2>(c, args, grid, search);
        case 3: return dispatch<3>(c, args, grid, search);
        default: return dispatch<4>(c, args, grid, search);
    }
}

static const SegTable kNoSegments{};

template <int BITS, bool NU, bool BF>
static cudaError_t launch_dev(const CompressCall& c, dim3 grid, int table_kernel_ran) {
    const RoundKeys rk = round_keys(c.seed);
    const SegTable& segs = c.segs ? *c.segs : kNoSegments;
    compress_kernel_dev<BITS, NU, BF><<<grid, kThreads, 0, c.stream>>>(
        c.grad, c.d, c.grad_stride, c.params_dev, rk, c.first_worker, c.packed, c.words_stride, c.words_out, segs, table_kernel_ran);
    if constexpr (NU) {
        if (cudaError_t e = cudaGetLastError()) return e;
        // a small grid: this pass is empty unless a codebook is too crowded for the lookup grid
        const dim3 small(grid.x < 16 ? grid.x : 16, grid.y);
        compress_kernel_dev_fallback<BITS, BF><<<small, kThreads, 0, c.stream>>>(
            c.grad, c.d, c.grad_stride, c.params_dev, rk, c.first_worker, c.packed, c.words_stride, c.words_out, segs, table_kernel_ran);
    }
    return cudaGetLastError();
}
template <int BITS>
static cudaError_t dispatch_dev(const CompressCall& c, dim3 grid, int lut) {
    if (c.nonuniform) return c.bf16 ? launch_dev<BITS, true, true>(c, grid, lut) : launch_dev<BITS, true, false>(c, grid, lut);
    return c.bf16 ? launch_dev<BITS, false, true>(c, grid, lut) : launch_dev<BITS, false, false>(c, grid, lut);
}

cudaError_t launch_compress_dev(const CompressCall& c) {
    // with segments: one grid row per (worker, segment) pair, sized by the longest segment
    uint64_t d = c.d;
    uint32_t jobs = c.n_workers;
    if (c.segs) {
        d = 0;
        for (uint32_t sg = 0; sg < c.segs->n; ++sg) d = c.segs->len[sg] > d ? c.segs->len[sg] : d;
        jobs = c.n_workers * c.segs->n;
    }
    // always the persistent grid here: a block first reads its quantizer from device memory and prepares it (two
    // barriers and a global round trip), which one block per tile would pay 120 000 times on a large row
    dim3 grid = compress_grid(d, jobs, true);
    // bf16 table codebooks: the decision-table kernel first; it serves the rows its window fits and the element-wise
    // kernels (a small grid then: they normally find nothing left) take the others
    bool lut = false;
    if (const cudaError_t e = launch_compress_lut(c, &lut)) return e;
    if (lut && grid.x > 16) grid.x = 16;
    if (c.launches) *c.launches = (c.nonuniform ? 2 : 1) + (lut ? 1 : 0);
    switch (c.bits) {
        case 1: return dispatch_dev<1>(c, grid, lut);
        case 2: return dispatch_dev<2>(c, grid, lut);
        case 3: return dispatch_dev<3>(c, grid, lut);
        default: return dispatch_dev<4>(c, grid, lut);
    }
}

}  // namespace tq
