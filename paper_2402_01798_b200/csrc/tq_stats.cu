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

template <bool BF16, int PASS>
__global__ void __launch_bounds__(kThreads)
stats_kernel(const void* __restrict__ grad, uint64_t d, uint64_t grad_stride, float g_min_in, float kappa,
             tq_stats_t* __restrict__ stats, Partial* __restrict__ partials, uint32_t* __restrict__ tickets) {
    const uint32_t wi = blockIdx.y;
    const size_t esz = BF16 ? 2 : 4;
    const char* row = static_cast<const char*>(grad) + static_cast<uint64_t>(wi) * grad_stride * esz;

    float g_min = g_min_in;
    if constexpr (PASS == kTail) g_min = stats[wi].g_min;     // finished by the moments pass
    const bool tail_on = (PASS != kMoments) && (g_min > 0.0f);
    const float inv_gmin = tail_on ? __frcp_rn(g_min) : 0.0f;

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
                if (tail_on && ok && a > g_min) { sum_log2 += __log2f(a * inv_gmin); n_tail += 1; }
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
            // elements were scaled by fl(1/g_min) instead of divided by g_min: remove the exact
            // logarithm of that factor's error, n * log2(fl(1/g_min) * g_min), then convert to ln
            double corr = 0.0;
            if (tail_on) corr = static_cast<double>(t.n_tail) * log2(static_cast<double>(inv_gmin) * static_cast<double>(g_min));
            st->n_tail = t.n_tail;
            st->sum_log_tail = (t.sum_log2 - corr) * 0.6931471805599453094;
        }
        *ticket = 0u;                                          // ready for the next call on this scratch
    }
}

template <bool BF16, int PASS>
static cudaError_t launch(const StatsCall& c, dim3 grid, Partial* partials, uint32_t* tickets) {
    stats_kernel<BF16, PASS><<<grid, kThreads, 0, c.stream>>>(c.grad, c.d, c.grad_stride, c.g_min, c.kappa,
                                                              c.stats, partials, tickets);
    return cudaGetLastError();
}

cudaError_t launch_stats(const StatsCall& c, int* launches) {
    *launches = 0;
    Partial* partials = static_cast<Partial*>(c.workspace);
    uint32_t* tickets = reinterpret_cast<uint32_t*>(static_cast<char*>(c.workspace) + tickets_offset(c.n_workers));
    cudaError_t e = cudaMemsetAsync(tickets, 0, static_cast<size_t>(c.n_workers) * 2 * sizeof(uint32_t), c.stream);
    if (e != cudaSuccess) return e;

    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    // 8 resident blocks of 256 threads per SM; spread them over the workers
    const uint64_t chunks = c.d / kChunk;
    uint64_t per_worker = (static_cast<uint64_t>(sms) * 8 + c.n_workers - 1) / c.n_workers;
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
