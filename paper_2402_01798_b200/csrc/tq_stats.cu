// Statistics reduction feeding the parameter design of Section 4: per worker sum|g|, sum g^2, max|g|,
// the non-finite count, and for the threshold g_min the tail count n = #{|g_j| > g_min} and
// sum ln(|g_j| / g_min) (the two ingredients of the maximum-likelihood tail index of Section 5 and of
// rho, the tail mass of Section 4.1).
//
// Shape: grid = (blocks per worker, workers).  A thread walks 16-element chunks with a block-wide
// stride, keeps fp32 partial sums inside a chunk and fp64 sums across chunks, then the block reduces
// with warp shuffles and writes ONE partial record to scratch.  A ticket counter (one atomic per
// block) tells the last block of a worker to fold that worker's records in index order, so the result
// does not depend on which block finishes last.  No block ever waits for another.
//
// With an automatic threshold (g_min = kappa * mean|g|) the tail quantities need the mean first:
// pass 1 (moments) finishes the record's g_min on the device, pass 2 (tail) reads it there; the host
// is not involved in between.  With a caller-supplied g_min one fused pass does everything.
// HBM traffic per element and pass: 4 bytes (fp32) or 2 bytes (bf16) read.
#include <math_constants.h>

#include <mutex>

#include "tq_device.cuh"
#include "tq_launch.h"

namespace tq {

constexpr int kMaxBlocksPerWorker = 1024;
constexpr int kChunk = 16;

struct alignas(64) Partial {
    double sum_abs, sum_sq, sum_log2;
    unsigned long long n_tail, n_bad;
    float max_abs, pad;
};
// scratch layout: [n_workers][kMaxBlocksPerWorker] Partial, then [n_workers][2] tickets (uint32)
__host__ __device__ inline size_t tickets_offset(uint32_t n_workers) {
    return static_cast<size_t>(n_workers) * kMaxBlocksPerWorker * sizeof(Partial);
}
size_t stats_workspace_bytes(uint32_t n_workers) {
    return tickets_offset(n_workers) + static_cast<size_t>(n_workers) * 2 * sizeof(uint32_t) + 256;
}

enum Pass { kMoments = 0, kTail = 1, kBoth = 2 };

// Hardware base-2 logarithm (absolute error about 2^-22 for arguments near 1, 2 ulp elsewhere).
// Subnormal arguments are flushed; only arguments >= 1 (tail elements) are ever used.
__device__ __forceinline__ float lg2_fast(float x) {
    float r; asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x)); return r;
}

__device__ __forceinline__ float fma_sat(float a, float b, float c) {
    float r; asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c)); return r;
}

template <bool BF16, int PASS>
__global__ void __launch_bounds__(kThreads)
stats_kernel(const void* __restrict__ grad, uint64_t d_row, uint64_t grad_stride, float g_min_in, float kappa,
             tq_stats_t* __restrict__ stats, Partial* __restrict__ partials, uint32_t* __restrict__ tickets,
             const __grid_constant__ SegTable segs) {
    const uint32_t wi = blockIdx.y;          // the job: a worker, or a (worker, segment) pair
    const size_t esz = BF16 ? 2 : 4;
    uint64_t d = d_row;
    const char* row = static_cast<const char*>(grad) + static_cast<uint64_t>(wi) * grad_stride * esz;
    if (segs.n) {
        const uint32_t worker = wi / segs.n, sg = wi - worker * segs.n;
        row = static_cast<const char*>(grad) + (static_cast<uint64_t>(worker) * grad_stride + segs.off[sg]) * esz;
        d = segs.len[sg];
    }

    float g_min = g_min_in;
    if constexpr (PASS == kTail) g_min = stats[wi].g_min;     // finished by the moments pass
    const bool tail_on = (PASS != kMoments) && (g_min > 0.0f);
    // Tail elements are scaled by inv_gmin before the logarithm and the exact logarithm of inv_gmin * g_min
    // is taken out again at the end, so inv_gmin only has to keep |g| * inv_gmin inside the normal range
    // for |g| > g_min.  1 / g_min overflows for a subnormal g_min; such a threshold is scaled by 2^64 first.
    const float inv_gmin = tail_on ? __frcp_rn(g_min < 7.8886090522101181e-31f ? g_min * 18446744073709551616.0f : g_min) : 0.0f;

    double sum_abs = 0.0, sum_sq = 0.0, sum_log2 = 0.0;
    unsigned long long n_tail = 0, n_bad = 0;
    float max_abs = 0.0f;

    const uint64_t n_chunks = d / kChunk;
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * kThreads;
    for (uint64_t c = static_cast<uint64_t>(blockIdx.x) * kThreads + threadIdx.x; c < n_chunks; c += stride) {
        float g[2][8];
        load8<BF16>(row + (c * kChunk) * esz, g[0]);
        load8<BF16>(row + (c * kChunk + 8) * esz, g[1]);
        // Fast path: assume every element is finite.  A NaN or Inf (or an overflow of the fp32 partial
        // sums) shows up as a non-finite partial; the chunk is then redone element by element.
        float s_abs = 0.0f, s_sq = 0.0f, s_log = 0.0f, c_max = 0.0f;
        uint32_t c_tail = 0;
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float a = fabsf(g[h][e]);
                if constexpr (PASS != kTail) {
                    s_abs += a;
                    s_sq = fmaf(a, a, s_sq);
                    c_max = fmaxf(c_max, a);        // drops NaN, keeps Inf: only used if the chunk is clean
                }
                if constexpr (PASS != kMoments) {
                    const bool in_tail = a > g_min;  // false for NaN, true for Inf (caught below)
                    const float lg = lg2_fast(a * inv_gmin);
                    s_log += in_tail ? lg : 0.0f;
                    c_tail += in_tail ? 1u : 0u;
                }
            }
        bool clean = true;
        if constexpr (PASS != kTail) clean = (s_abs + s_sq) <= 3.402823466e38f;
        if constexpr (PASS == kTail) clean = s_log <= 3.402823466e38f;
        else if constexpr (PASS == kBoth) clean = clean && (s_log <= 3.402823466e38f);
        if (clean) {
            if constexpr (PASS != kTail) { sum_abs += s_abs; sum_sq += s_sq; max_abs = fmaxf(max_abs, c_max); }
            if constexpr (PASS != kMoments) {
                if (tail_on) { sum_log2 += s_log; n_tail += c_tail; }
            }
        } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const float a = fabsf(g[i >> 3][i & 7]);
                const bool ok = a <= 3.402823466e38f;          // false for NaN and Inf
                if constexpr (PASS != kTail) {
                    if (ok) { sum_abs += a; sum_sq += static_cast<double>(a) * a; max_abs = fmaxf(max_abs, a); }
                    else n_bad += 1;
                }
                if constexpr (PASS != kMoments) {
                    if (tail_on && ok && a > g_min) {
                        sum_log2 += log2(static_cast<double>(a) * static_cast<double>(inv_gmin));
                        n_tail += 1;
                    }
                }
            }
        }
    }
    // the d % 16 leftover elements, taken by the first threads of block 0
    if (blockIdx.x == 0) {
        const uint64_t j = n_chunks * kChunk + threadIdx.x;
        if (j < d) {
            const float a = fabsf(load1<BF16>(row, j));
            const bool ok = a <= 3.402823466e38f;
            const float av = ok ? a : 0.0f;
            if constexpr (PASS != kTail) {
                sum_abs += av; sum_sq += static_cast<double>(av) * av; max_abs = fmaxf(max_abs, av); n_bad += ok ? 0 : 1;
            }
            if constexpr (PASS != kMoments) {
                if (tail_on && ok && a > g_min) { sum_log2 += log2(static_cast<double>(a) * static_cast<double>(inv_gmin)); n_tail += 1; }
            }
        }
    }

    // block reduction: shuffles inside a warp, shared memory across the 8 warps
    __shared__ double s_d[3][kThreads / 32];
    __shared__ unsigned long long s_u[2][kThreads / 32];
    __shared__ float s_f[kThreads / 32];
    __shared__ bool s_last;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    sum_abs = warp_sum(sum_abs); sum_sq = warp_sum(sum_sq); sum_log2 = warp_sum(sum_log2);
    n_tail = warp_sum(n_tail); n_bad = warp_sum(n_bad); max_abs = warp_max(max_abs);
    if (lane == 0) {
        s_d[0][warp] = sum_abs; s_d[1][warp] = sum_sq; s_d[2][warp] = sum_log2;
        s_u[0][warp] = n_tail; s_u[1][warp] = n_bad; s_f[warp] = max_abs;
    }
    __syncthreads();
    Partial* mine = partials + static_cast<size_t>(wi) * kMaxBlocksPerWorker;
    uint32_t* ticket = tickets + wi * 2 + (PASS == kTail ? 1 : 0);
    if (threadIdx.x == 0) {
        Partial p{};
        for (int w = 0; w < kThreads / 32; ++w) {
            p.sum_abs += s_d[0][w]; p.sum_sq += s_d[1][w]; p.sum_log2 += s_d[2][w];
            p.n_tail += s_u[0][w]; p.n_bad += s_u[1][w]; p.max_abs = fmaxf(p.max_abs, s_f[w]);
        }
        mine[blockIdx.x] = p;
        __threadfence();                                       // record visible before the ticket
        s_last = atomicAdd(ticket, 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (!s_last) return;

    // last block of this worker: fold the records in index order (fixed shape, deterministic)
    __threadfence();
    Partial acc{};
    for (uint32_t b = threadIdx.x; b < gridDim.x; b += kThreads) {
        const volatile Partial* p = mine + b;
        acc.sum_abs += p->sum_abs; acc.sum_sq += p->sum_sq; acc.sum_log2 += p->sum_log2;
        acc.n_tail += p->n_tail; acc.n_bad += p->n_bad; acc.max_abs = fmaxf(acc.max_abs, p->max_abs);
    }
    acc.sum_abs = warp_sum(acc.sum_abs); acc.sum_sq = warp_sum(acc.sum_sq); acc.sum_log2 = warp_sum(acc.sum_log2);
    acc.n_tail = warp_sum(acc.n_tail); acc.n_bad = warp_sum(acc.n_bad); acc.max_abs = warp_max(acc.max_abs);
    __syncthreads();
    if (lane == 0) {
        s_d[0][warp] = acc.sum_abs; s_d[1][warp] = acc.sum_sq; s_d[2][warp] = acc.sum_log2;
        s_u[0][warp] = acc.n_tail; s_u[1][warp] = acc.n_bad; s_f[warp] = acc.max_abs;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        Partial t{};
        for (int w = 0; w < kThreads / 32; ++w) {
            t.sum_abs += s_d[0][w]; t.sum_sq += s_d[1][w]; t.sum_log2 += s_d[2][w];
            t.n_tail += s_u[0][w]; t.n_bad += s_u[1][w]; t.max_abs = fmaxf(t.max_abs, s_f[w]);
        }
        tq_stats_t* st = stats + wi;
        if constexpr (PASS != kTail) {
            st->d = d; st->n_nonfinite = t.n_bad; st->sum_abs = t.sum_abs; st->sum_sq = t.sum_sq;
            st->max_abs = t.max_abs;
            float gm = g_min_in;
            if (!(g_min_in > 0.0f))
                gm = d ? static_cast<float>(static_cast<double>(kappa) * t.sum_abs / static_cast<double>(d)) : 0.0f;
            st->g_min = gm;
            st->reserved = 0;
            if constexpr (PASS == kMoments) { st->n_tail = 0; st->sum_log_tail = 0.0; }
        }
        if constexpr (PASS != kMoments) {
            // elements were scaled by inv_gmin instead of divided by g_min: remove the exact
            // logarithm of that factor's error, n * log2(inv_gmin * g_min), then convert to ln
            double corr = 0.0;
            if (tail_on) corr = static_cast<double>(t.n_tail) * log2(static_cast<double>(inv_gmin) * static_cast<double>(g_min));
            st->n_tail = t.n_tail;
            st->sum_log_tail = (t.sum_log2 - corr) * 0.6931471805599453094;
        }
        *ticket = 0u;                                          // ready for the next call on this scratch
    }
}

static const SegTable kNoSegments{};

template <bool BF16, int PASS>
static cudaError_t launch(const StatsCall& c, dim3 grid, Partial* partials, uint32_t* tickets) {
    stats_kernel<BF16, PASS><<<grid, kThreads, 0, c.stream>>>(c.grad, c.d, c.grad_stride, c.g_min, c.kappa,
                                                              c.stats, partials, tickets, c.segs ? *c.segs : kNoSegments);
    return cudaGetLastError();
}

cudaError_t launch_stats(const StatsCall& call, int* launches) {
    *launches = 0;
    // with segments every (worker, segment) pair is a job of its own: same kernels, same scratch layout
    StatsCall c = call;
    const uint32_t n_jobs = c.segs ? c.n_workers * c.segs->n : c.n_workers;
    if (c.segs) {
        c.d = 0;
        for (uint32_t sg = 0; sg < c.segs->n; ++sg) c.d = c.segs->len[sg] > c.d ? c.segs->len[sg] : c.d;   // sizes the grid
    }
    c.n_workers = n_jobs;
    Partial* partials = static_cast<Partial*>(c.workspace);
    uint32_t* tickets = reinterpret_cast<uint32_t*>(static_cast<char*>(c.workspace) + tickets_offset(c.n_workers));
    cudaError_t e = cudaMemsetAsync(tickets, 0, static_cast<size_t>(c.n_workers) * 2 * sizeof(uint32_t), c.stream);
    if (e != cudaSuccess) return e;

    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    // 8 resident blocks of 256 threads per SM; spread them over the workers
    const uint64_t chunks = c.d / kChunk;
    uint64_t per_worker = static_cast<uint64_t>(sms) * 8 / c.n_workers;       // rounded down: a block beyond the resident set would run as a second wave
    const uint64_t useful = (chunks + kThreads - 1) / kThreads;
    if (per_worker > useful) per_worker = useful;
    if (per_worker > kMaxBlocksPerWorker) per_worker = kMaxBlocksPerWorker;
    if (per_worker < 1) per_worker = 1;
    const dim3 grid(static_cast<unsigned>(per_worker), c.n_workers);

    if (c.g_min > 0.0f) {
        e = c.bf16 ? launch<true, kBoth>(c, grid, partials, tickets) : launch<false, kBoth>(c, grid, partials, tickets);
        *launches = 1;
        return e;
    }
    e = c.bf16 ? launch<true, kMoments>(c, grid, partials, tickets) : launch<false, kMoments>(c, grid, partials, tickets);
    if (e != cudaSuccess) return e;
    *launches = 1;
    e = c.bf16 ? launch<true, kTail>(c, grid, partials, tickets) : launch<false, kTail>(c, grid, partials, tickets);
    *launches = 2;
    return e;
}

// ---------------------------------------------------------------------------------------------
// One pass with a hinted threshold.  The paper leaves the choice of g_min open (Section 4.1 only
// calls it the lower end of the power-law range); with g_min = kappa * mean|g| rounded DOWN TO A
// POWER OF TWO the tail sums can be gathered before the mean is known, for a few candidate powers of
// two at once: a caller-kept hint (the kappa * mean|g| of the previous round) names the two
// candidates nearest to it, the moments and both candidates' tail sums are accumulated in ONE pass,
// and the last block keeps the candidate that the finished mean selects.  If neither fits (first
// round, or the mean moved by more than a factor of about 1.4 to 2), a second kernel redoes the tail
// pass for the right threshold; it is launched every time and returns at once when not needed, so
// the host never has to look.  Both kernels sum log2|g| itself (not log2(|g| / g_min)) in the same
// order and remove n * log2(g_min), an integer multiple, at the end: the record is bit-identical
// whichever way it was obtained.
struct alignas(64) PartialH {
    double sum_abs, sum_sq, sum_log2[2];
    unsigned long long n_tail[2], n_bad;
    float max_abs, pad;
};
static_assert(sizeof(PartialH) == sizeof(Partial), "the hinted pass shares the scratch layout");

// Largest power of two not above x; 0 below the smallest normal number (no tail), Inf for Inf.
__device__ __forceinline__ float pow2_floor(float x) {
    return x >= 1.17549435e-38f ? __uint_as_float(__float_as_uint(x) & 0xFF800000u) : 0.0f;
}

#ifndef TQ_STATS_HINTED_BLOCKS
#define TQ_STATS_HINTED_BLOCKS 3
#endif

template <bool BF16, bool FALLBACK>
__global__ void __launch_bounds__(kThreads, TQ_STATS_HINTED_BLOCKS)
stats_hinted_kernel(const void* __restrict__ grad, uint64_t d_row, uint64_t grad_stride, float kappa,
                    tq_gmin_hint_t* __restrict__ hint, tq_stats_t* __restrict__ stats,
                    PartialH* __restrict__ partials, uint32_t* __restrict__ tickets, const __grid_constant__ SegTable segs) {
    constexpr int K = FALLBACK ? 1 : 2;
    const uint32_t wi = blockIdx.y;               // the job: a worker, or a (worker, segment) pair
    if constexpr (FALLBACK) {
        if (hint[wi].hit) return;                 // the one-pass result stands
    }
    const size_t esz = BF16 ? 2 : 4;
    uint64_t d = d_row;
    const char* row = static_cast<const char*>(grad) + static_cast<uint64_t>(wi) * grad_stride * esz;
    if (segs.n) {
        const uint32_t worker = wi / segs.n, sg = wi - worker * segs.n;
        row = static_cast<const char*>(grad) + (static_cast<uint64_t>(worker) * grad_stride + segs.off[sg]) * esz;
        d = segs.len[sg];
    }

    // candidate thresholds
    float t[2] = {CUDART_INF_F, CUDART_INF_F};
    if constexpr (FALLBACK) {
        t[0] = stats[wi].g_min;                   // finished by the hinted pass; > 0 here
    } else {
        const float level = hint[wi].level;
        if (level >= 2.3509887e-38f && level <= 3.402823466e38f) {      // from 2^-125: both candidates are normal numbers
            const uint32_t bits = __float_as_uint(level);
            const uint32_t e = bits & 0x7F800000u;
            const uint32_t lo = (bits & 0x00400000u) ? e : e - 0x00800000u;    // mantissa >= 1.5: {2^h, 2^(h+1)}, else {2^(h-1), 2^h}
            t[0] = __uint_as_float(lo);
            t[1] = __uint_as_float(lo + 0x00800000u);
        }
    }

    double sum_abs = 0.0, sum_sq = 0.0, sum_log2[2] = {0.0, 0.0};
    unsigned long long n_tail[2] = {0, 0}, n_bad = 0;
    float max_abs = 0.0f;
    const f32x2 inv_t2 = both(__frcp_rn(t[0]));     // exact: t is a power of two (0 for t = Inf: nothing is in the tail)

    // One chunk of 16 elements: fp32 partials, then into the fp64 sums (the fast path assumes finite
    // values; a non-finite partial sends the chunk through the element-wise path).
    // The integer / compare pipe runs at half rate and would bound this loop (two compares, two
    // selects and two integer adds per candidate), so the tail test is done on the multiply-add pipe:
    // with r = |g| / t exact (t a power of two), [|g| > t] = sat(r * 2^30 - 2^30): the smallest r above 1
    // gives 2^7, r <= 1 gives <= 0, NaN gives 0, Inf gives 1.  The second candidate is 2 t: same r, 2^29.
    // Counts are kept as small floats inside a chunk, and the masked sum is s + m * lg with m = 0 or 1,
    // which rounds exactly like adding lg or nothing.  log2 is taken of max(|g|, 2^-126) so that a
    // zero cannot turn 0 * (-inf) into NaN; elements that small are never in a tail (t >= 2^-126).
    auto take_chunk = [&](const Raw8<BF16> (&g)[2]) {
        float s_abs = 0.0f, c_max = 0.0f;
        f32x2 s_sq2 = both(0.0f), s_log2[2] = {both(0.0f), both(0.0f)}, cnt2[2] = {both(0.0f), both(0.0f)};
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int e = 0; e < 8; e += 2) {
                const float x0 = elem<BF16>(g[h], e), x1 = elem<BF16>(g[h], e + 1);
                const float a0 = fabsf(x0), a1 = fabsf(x1);
                s_abs += a0;
                s_abs += a1;
                const f32x2 x = pair(x0, x1);
                s_sq2 = fma2(x, x, s_sq2);
                c_max = fmaxf(fmaxf(c_max, a0), a1);
                const f32x2 lg = pair(lg2_fast(fmaxf(a0, 1.17549435e-38f)), lg2_fast(fmaxf(a1, 1.17549435e-38f)));
                float r0, r1;
                unpair(mul2(x, inv_t2), r0, r1);
#pragma unroll
                for (int k = 0; k < K; ++k) {
                    const float scale = k ? 536870912.0f : 1073741824.0f;      // 2^29 for the candidate 2 t, 2^30 for t
                    const f32x2 m = pair(fma_sat(fabsf(r0), scale, -1073741824.0f), fma_sat(fabsf(r1), scale, -1073741824.0f));
                    s_log2[k] = fma2(m, lg, s_log2[k]);
                    cnt2[k] = add2(cnt2[k], m);
                }
            }
        float q0, q1;
        unpair(s_sq2, q0, q1);
        const float s_sq = q0 + q1;
        // same test in both kernels, so that both send the same chunks through the slow path
        const bool clean = (s_abs + s_sq) <= 3.402823466e38f;
        if (clean) {
            if constexpr (!FALLBACK) { sum_abs += s_abs; sum_sq += s_sq; max_abs = fmaxf(max_abs, c_max); }
#pragma unroll
            for (int k = 0; k < K; ++k) {
                float l0, l1, n0, n1;
                unpair(s_log2[k], l0, l1);
                unpair(cnt2[k], n0, n1);
                sum_log2[k] += l0 + l1;
                n_tail[k] += static_cast<uint32_t>(n0 + n1);
            }
        } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const float a = fabsf(elem<BF16>(g[i >> 3], i & 7));
                const bool ok = a <= 3.402823466e38f;          // false for NaN and Inf
                if constexpr (!FALLBACK) {
                    if (ok) { sum_abs += a; sum_sq += static_cast<double>(a) * a; max_abs = fmaxf(max_abs, a); }
                    else n_bad += 1;
                }
#pragma unroll
                for (int k = 0; k < K; ++k)
                    if (ok && a > t[k]) { sum_log2[k] += log2(static_cast<double>(a)); n_tail[k] += 1; }
            }
        }
    };

    // A thread's chunks are c0, c0 + stride, ...; the loads of kAhead of them (128 bytes per thread) are
    // issued together, then they are summed in that same order.
    constexpr int kAhead = BF16 ? 4 : 2;
    const uint64_t n_chunks = d / kChunk;
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * kThreads;
    for (uint64_t c = static_cast<uint64_t>(blockIdx.x) * kThreads + threadIdx.x; c < n_chunks; c += kAhead * stride) {
        Raw8<BF16> g[kAhead][2];
#pragma unroll
        for (int u = 0; u < kAhead; ++u) {
            const uint64_t cu = c + u * stride;
            if (cu < n_chunks) {
                load8_raw<BF16>(row + (cu * kChunk) * esz, g[u][0]);
                load8_raw<BF16>(row + (cu * kChunk + 8) * esz, g[u][1]);
            }
        }
#pragma unroll
        for (int u = 0; u < kAhead; ++u)
            if (c + u * stride < n_chunks) take_chunk(g[u]);
    }
    // the d % 16 leftover elements, taken by the first threads of block 0
    if (blockIdx.x == 0) {
        const uint64_t j = n_chunks * kChunk + threadIdx.x;
        if (j < d) {
            const float a = fabsf(load1<BF16>(row, j));
            const bool ok = a <= 3.402823466e38f;
            if constexpr (!FALLBACK) {
                const float av = ok ? a : 0.0f;
                sum_abs += av; sum_sq += static_cast<double>(av) * av; max_abs = fmaxf(max_abs, av); n_bad += ok ? 0 : 1;
            }
#pragma unroll
            for (int k = 0; k < K; ++k)
                if (ok && a > t[k]) { sum_log2[k] += log2(static_cast<double>(a)); n_tail[k] += 1; }
        }
    }

    // block reduction: shuffles inside a warp, shared memory across the 8 warps
    __shared__ double s_d[4][kThreads / 32];
    __shared__ unsigned long long s_u[3][kThreads / 32];
    __shared__ float s_f[kThreads / 32];
    __shared__ bool s_last;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    auto block_fold = [&](PartialH& p) {       // every thread passes its values; thread 0 gets the block's
        p.sum_abs = warp_sum(p.sum_abs); p.sum_sq = warp_sum(p.sum_sq);
        p.sum_log2[0] = warp_sum(p.sum_log2[0]); p.sum_log2[1] = warp_sum(p.sum_log2[1]);
        p.n_tail[0] = warp_sum(p.n_tail[0]); p.n_tail[1] = warp_sum(p.n_tail[1]); p.n_bad = warp_sum(p.n_bad);
        p.max_abs = warp_max(p.max_abs);
        if (lane == 0) {
            s_d[0][warp] = p.sum_abs; s_d[1][warp] = p.sum_sq; s_d[2][warp] = p.sum_log2[0]; s_d[3][warp] = p.sum_log2[1];
            s_u[0][warp] = p.n_tail[0]; s_u[1][warp] = p.n_tail[1]; s_u[2][warp] = p.n_bad; s_f[warp] = p.max_abs;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            PartialH r{};
            for (int w = 0; w < kThreads / 32; ++w) {
                r.sum_abs += s_d[0][w]; r.sum_sq += s_d[1][w]; r.sum_log2[0] += s_d[2][w]; r.sum_log2[1] += s_d[3][w];
                r.n_tail[0] += s_u[0][w]; r.n_tail[1] += s_u[1][w]; r.n_bad += s_u[2][w]; r.max_abs = fmaxf(r.max_abs, s_f[w]);
            }
            p = r;
        }
    };
    PartialH p{};
    p.sum_abs = sum_abs; p.sum_sq = sum_sq; p.sum_log2[0] = sum_log2[0]; p.sum_log2[1] = sum_log2[1];
    p.n_tail[0] = n_tail[0]; p.n_tail[1] = n_tail[1]; p.n_bad = n_bad; p.max_abs = max_abs;
    block_fold(p);
    PartialH* mine = partials + static_cast<size_t>(wi) * kMaxBlocksPerWorker;
    uint32_t* ticket = tickets + wi * 2 + (FALLBACK ? 1 : 0);
    if (threadIdx.x == 0) {
        mine[blockIdx.x] = p;
        __threadfence();                                       // record visible before the ticket
        s_last = atomicAdd(ticket, 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (!s_last) return;

    // last block of this worker: fold the records in index order (fixed shape, deterministic)
    __threadfence();
    PartialH acc{};
    for (uint32_t b = threadIdx.x; b < gridDim.x; b += kThreads) {
        const volatile PartialH* q = mine + b;
        acc.sum_abs += q->sum_abs; acc.sum_sq += q->sum_sq; acc.sum_log2[0] += q->sum_log2[0]; acc.sum_log2[1] += q->sum_log2[1];
        acc.n_tail[0] += q->n_tail[0]; acc.n_tail[1] += q->n_tail[1]; acc.n_bad += q->n_bad; acc.max_abs = fmaxf(acc.max_abs, q->max_abs);
    }
    __syncthreads();
    block_fold(acc);
    if (threadIdx.x == 0) {
        tq_stats_t* st = stats + wi;
        int pick = -1;                       // candidate whose sums are the record's tail
        float g_min;
        if constexpr (FALLBACK) {
            g_min = t[0];
            pick = 0;
        } else {
            const float level = d ? static_cast<float>(static_cast<double>(kappa) * acc.sum_abs / static_cast<double>(d)) : 0.0f;
            g_min = pow2_floor(level);
            st->d = d; st->n_nonfinite = acc.n_bad; st->sum_abs = acc.sum_abs; st->sum_sq = acc.sum_sq;
            st->max_abs = acc.max_abs; st->g_min = g_min; st->reserved = 0;
            st->n_tail = 0; st->sum_log_tail = 0.0;
            uint32_t hit = 1;
            if (g_min > 0.0f) {
                if (__float_as_uint(g_min) == __float_as_uint(t[0])) pick = 0;
                else if (__float_as_uint(g_min) == __float_as_uint(t[1])) pick = 1;
                else hit = 0;
            }
            hint[wi].level = level;
            hint[wi].hit = hit;
        }
        if (pick >= 0 && g_min <= 3.402823466e38f) {
            // sum ln(a / g_min) = ln 2 * (sum log2 a - n * log2 g_min), log2 g_min an integer
            const int e2 = static_cast<int>((__float_as_uint(g_min) >> 23) & 0xFFu) - 127;
            const unsigned long long n = pick ? acc.n_tail[1] : acc.n_tail[0];
            const double s2 = pick ? acc.sum_log2[1] : acc.sum_log2[0];
            st->n_tail = n;
            st->sum_log_tail = (s2 - static_cast<double>(n) * static_cast<double>(e2)) * 0.6931471805599453094;
        }
        *ticket = 0u;                                          // ready for the next call on this scratch
    }
}

cudaError_t launch_stats_hinted(const StatsCall& call, tq_gmin_hint_t* hint, int* launches) {
    *launches = 0;
    StatsCall c = call;                          // with segments every (worker, segment) pair is a job of its own
    if (c.segs) {
        c.d = 0;
        for (uint32_t sg = 0; sg < c.segs->n; ++sg) c.d = c.segs->len[sg] > c.d ? c.segs->len[sg] : c.d;   // sizes the grid
        c.n_workers *= c.segs->n;
    }
    const SegTable& segs = c.segs ? *c.segs : kNoSegments;
    PartialH* partials = static_cast<PartialH*>(c.workspace);
    uint32_t* tickets = reinterpret_cast<uint32_t*>(static_cast<char*>(c.workspace) + tickets_offset(c.n_workers));
    cudaError_t e = cudaMemsetAsync(tickets, 0, static_cast<size_t>(c.n_workers) * 2 * sizeof(uint32_t), c.stream);
    if (e != cudaSuccess) return e;
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    // the resident blocks of 256 threads per SM, spread over the workers
    const uint64_t chunks = c.d / kChunk;
    uint64_t per_worker = static_cast<uint64_t>(sms) * TQ_STATS_HINTED_BLOCKS / c.n_workers;     // rounded down: no second wave
    const uint64_t useful = (chunks + kThreads - 1) / kThreads;
    if (per_worker > useful) per_worker = useful;
    if (per_worker > kMaxBlocksPerWorker) per_worker = kMaxBlocksPerWorker;
    if (per_worker < 1) per_worker = 1;
    const dim3 grid(static_cast<unsigned>(per_worker), c.n_workers);     // the same grid for both kernels: same summation order
    if (c.bf16) stats_hinted_kernel<true, false><<<grid, kThreads, 0, c.stream>>>(c.grad, c.d, c.grad_stride, c.kappa, hint, c.stats, partials, tickets, segs);
    else stats_hinted_kernel<false, false><<<grid, kThreads, 0, c.stream>>>(c.grad, c.d, c.grad_stride, c.kappa, hint, c.stats, partials, tickets, segs);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    *launches = 1;
    if (c.bf16) stats_hinted_kernel<true, true><<<grid, kThreads, 0, c.stream>>>(c.grad, c.d, c.grad_stride, c.kappa, hint, c.stats, partials, tickets, segs);
    else stats_hinted_kernel<false, true><<<grid, kThreads, 0, c.stream>>>(c.grad, c.d, c.grad_stride, c.kappa, hint, c.stats, partials, tickets, segs);
    e = cudaGetLastError();
    if (e == cudaSuccess) *launches = 2;
    return e;
}

// ---------------------------------------------------------------------------------------------
// Built-in scratch for callers that cannot allocate: enough for TQ_STATIC_MAX_WORKERS workers.
// It is part of the library's device image (one copy per GPU that loads the library).
constexpr size_t kStaticScratchBytes =
    static_cast<size_t>(TQ_STATIC_MAX_WORKERS) * kMaxBlocksPerWorker * sizeof(Partial) + TQ_STATIC_MAX_WORKERS * 2 * sizeof(uint32_t) + 256;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

cudaError_t launch_stats_static(const StatsCall& c, int* launches, bool* limit) {
    *launches = 0;
    *limit = c.n_workers > TQ_STATIC_MAX_WORKERS || stats_workspace_bytes(c.n_workers) > kStaticScratchBytes;
    if (*limit) return cudaSuccess;

    // In host code `g_static_scratch` is only a handle for the symbol, not a device address: the
    // address must be asked for, per device, with that device current.  Done on the first call
    // on each device and remembered.
    constexpr int kMaxDevices = 64;
    static void* s_addr[kMaxDevices] = {};
    static std::mutex s_lock;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    void* ptr = nullptr;
    {
        std::lock_guard<std::mutex> hold(s_lock);
        if (!s_addr[dev]) {
            e = cudaGetSymbolAddress(&ptr, g_static_scratch);
            if (e != cudaSuccess) return e;
            s_addr[dev] = ptr;
        }
        ptr = s_addr[dev];
    }
    StatsCall with_scratch = c;
    with_scratch.workspace = ptr;
    return launch_stats(with_scratch, launches);   // clears the tickets first, as every call does
}

}  // namespace tq
