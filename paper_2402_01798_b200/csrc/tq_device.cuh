// Device-side building blocks shared by the libtq kernels (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "tq.h"

namespace tq {

constexpr int kThreads = 256;
constexpr float kMagic = 8388608.0f;          // 2^23: adding it leaves an integer in the mantissa
constexpr uint32_t kMagicBits = 0x4B000000u;  // bit pattern of 2^23

// ---- 256-bit global accesses (one full 32-byte sector per lane) ---------------------------------
__device__ __forceinline__ void ldg256_stream(const void* p, uint32_t (&v)[8]) {
    asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                 : "l"(p));
}
__device__ __forceinline__ void stg256(void* p, const float (&v)[8]) {
    asm volatile("st.global.v8.f32 [%8], {%0,%1,%2,%3,%4,%5,%6,%7};"
                 :: "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]), "l"(p)
                 : "memory");
}

// Eight consecutive gradient elements as fp32.  `p` is 32-byte aligned for fp32 and 16-byte aligned
// for bf16.  bf16 -> fp32 is exact: the stored 16 bits become the high half of the fp32 pattern.
template <bool BF16>
__device__ __forceinline__ void load8(const void* p, float (&g)[8]) {
    if constexpr (!BF16) {
        uint32_t v[8];
        ldg256_stream(p, v);
#pragma unroll
        for (int i = 0; i < 8; ++i) g[i] = __uint_as_float(v[i]);
    } else {
        uint4 v;
        asm volatile("ld.global.nc.L1::no_allocate.v4.b32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            g[2 * i] = __uint_as_float(w[i] << 16);
            g[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
}

// Eight consecutive gradient elements kept as loaded (fp32: 8 words; bf16: 4 words of two), decoded
// on use.  Keeping bf16 packed halves the registers a loaded group occupies.
template <bool BF16>
struct Raw8 {
    uint32_t v[BF16 ? 4 : 8];
};
template <bool BF16>
__device__ __forceinline__ void load8_raw(const void* p, Raw8<BF16>& r) {
    if constexpr (!BF16) ldg256_stream(p, r.v);
    else asm volatile("ld.global.nc.L1::no_allocate.v4.b32 {%0,%1,%2,%3}, [%4];"
                      : "=r"(r.v[0]), "=r"(r.v[1]), "=r"(r.v[2]), "=r"(r.v[3]) : "l"(p));
}
template <bool BF16>
__device__ __forceinline__ float elem(const Raw8<BF16>& r, int e) {
    if constexpr (!BF16) return __uint_as_float(r.v[e]);
    else return __uint_as_float((e & 1) ? (r.v[e >> 1] & 0xFFFF0000u) : (r.v[e >> 1] << 16));
}
template <bool BF16>
__device__ __forceinline__ void set_elem(Raw8<BF16>& r, int e, float x) {   // fp32 bits, or an exact bf16 value
    if constexpr (!BF16) r.v[e] = __float_as_uint(x);
    else r.v[e >> 1] = (e & 1) ? ((r.v[e >> 1] & 0x0000FFFFu) | (__float_as_uint(x) & 0xFFFF0000u))
                               : ((r.v[e >> 1] & 0xFFFF0000u) | (__float_as_uint(x) >> 16));
}

// One element, any alignment (ragged tails).
template <bool BF16>
__device__ __forceinline__ float load1(const void* base, uint64_t j) {
    if constexpr (!BF16) return __ldg(reinterpret_cast<const float*>(base) + j);
    else return __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short*>(base) + j)) << 16);
}

// ---- asynchronous copies into shared memory, counted on an mbarrier ----------------------------------
// Every wait is bounded: after kWaitLimit polls the caller gets `false`, records it and winds down.
constexpr uint32_t kWaitLimit = 1u << 22;

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// global -> this block's shared memory, `bytes` a multiple of 16, both addresses 16-byte aligned
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t it = 0; it < kWaitLimit; ++it) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}


// ---- packed fp32 pairs ----------------------------------------------------------------------------
// sm_100 executes add / mul / fma on two fp32 values held in a 64-bit register pair as ONE instruction,
// each half rounded exactly like the scalar operation.  The kernels here are bound by instruction
// issue, so pairing halves the cost of every arithmetic step it applies to.
struct f32x2 { uint64_t v; };
__device__ __forceinline__ f32x2 pair(float lo, float hi) {
    f32x2 r; asm("mov.b64 %0, {%1, %2};" : "=l"(r.v) : "f"(lo), "f"(hi)); return r;
}
__device__ __forceinline__ f32x2 both(float x) { return pair(x, x); }
__device__ __forceinline__ void unpair(f32x2 p, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(p.v));
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
    f32x2 r; asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v)); return r;
}
__device__ __forceinline__ f32x2 add2_rd(f32x2 a, f32x2 b) {   // round toward -infinity
    f32x2 r; asm("add.rm.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v)); return r;
}
__device__ __forceinline__ f32x2 sub2(f32x2 a, f32x2 b) {
    f32x2 r; asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v)); return r;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
    f32x2 r; asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v)); return r;
}
__device__ __forceinline__ f32x2 mul2_rd(f32x2 a, f32x2 b) {
    f32x2 r; asm("mul.rm.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v)); return r;
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
    f32x2 r; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r.v) : "l"(a.v), "l"(b.v), "l"(c.v)); return r;
}

// ---- Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11), counter = (c0, c1, worker, 0) ------------------
// The ten round keys (key advanced by the Weyl constants) are computed once on the host: they depend on
// the seed only, and sit in the kernel's constant bank instead of registers.
struct RoundKeys {
    uint32_t k0[10], k1[10];
};
inline RoundKeys round_keys(uint64_t seed) {
    RoundKeys rk;
    uint32_t k0 = static_cast<uint32_t>(seed), k1 = static_cast<uint32_t>(seed >> 32);
    for (int r = 0; r < 10; ++r) { rk.k0[r] = k0; rk.k1[r] = k1; k0 += 0x9E3779B9u; k1 += 0xBB67AE85u; }
    return rk;
}

__device__ __forceinline__ void mul_wide(uint32_t a, uint32_t b, uint32_t& hi, uint32_t& lo) {
    uint64_t p;
    asm("mul.wide.u32 %0, %1, %2;" : "=l"(p) : "r"(a), "r"(b));
    asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(p));
}

// Within a run of elements only c0 changes, so what the first two rounds make of the other three counter
// words is computed once per run: of the 20 wide multiplies of a block, 3 drop out (the second product of
// round 1 and the first of round 2 have constant operands, and word 0 after round 1 is constant).
struct PhiloxRun {
    uint32_t a1, b1, b2, d2;
};
__device__ __forceinline__ PhiloxRun philox_run(uint32_t c1, uint32_t worker, const RoundKeys& rk) {
    uint32_t hi1, lo1;
    mul_wide(0xCD9E8D57u, worker, hi1, lo1);                  // round 1, second product
    const uint32_t c0_1 = hi1 ^ c1 ^ rk.k0[0];                // word 0 after round 1
    uint32_t hi0c, lo0c;
    mul_wide(0xD2511F53u, c0_1, hi0c, lo0c);                  // round 2, first product
    PhiloxRun r;
    r.a1 = rk.k1[0];                 // word 2 after round 1 = hi(M0 * c0) ^ 0 ^ k1[0]
    r.b1 = lo1 ^ rk.k0[1];           // word 0 after round 2 = hi(M1 * word 2) ^ lo1 ^ k0[1]
    r.b2 = hi0c ^ rk.k1[1];          // word 2 after round 2 = hi0c ^ lo(M0 * c0) ^ k1[1]
    r.d2 = lo0c;                     // word 3 after round 2
    return r;
}
__device__ __forceinline__ void philox_block(uint32_t c0, const PhiloxRun& pr, const RoundKeys& rk, uint32_t (&out)[4]) {
    uint32_t hi0, lo0, hi1, lo1;
    mul_wide(0xD2511F53u, c0, hi0, lo0);                      // round 1
    const uint32_t w2 = hi0 ^ pr.a1;
    mul_wide(0xCD9E8D57u, w2, hi1, lo1);                      // round 2
    uint32_t x0 = hi1 ^ pr.b1, x1 = lo1, x2 = lo0 ^ pr.b2, x3 = pr.d2;
#pragma unroll
    for (int r = 2; r < 10; ++r) {
        mul_wide(0xD2511F53u, x0, hi0, lo0);
        mul_wide(0xCD9E8D57u, x2, hi1, lo1);
        x0 = hi1 ^ x1 ^ rk.k0[r];
        x2 = hi0 ^ x3 ^ rk.k1[r];
        x1 = lo1;
        x3 = lo0;
    }
    out[0] = x0; out[1] = x1; out[2] = x2; out[3] = x3;
}

// ---- warp / block reductions -----------------------------------------------------------------------
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xFFFFFFFFu, v, o);
    return v;
}
__device__ __forceinline__ unsigned long long warp_sum(unsigned long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xFFFFFFFFu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_down_sync(0xFFFFFFFFu, v, o));
    return v;
}

}  // namespace tq
