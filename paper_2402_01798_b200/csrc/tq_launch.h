// Internal host-side interface between the C ABI (tq_api.cu) and the kernel files.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "tq.h"

namespace tq {

// Layer groups (Section 5 quantizes groups of layers independently): every worker's row is cut into the same
// n segments, and a (worker, segment) pair is handled like a worker of its own ("job" = worker * n + segment).
// n = 0: no segments, a job is a worker and its row is the whole slice.
struct SegTable {
    uint32_t n;
    uint32_t pad;
    uint64_t off[TQ_MAX_SEGMENTS];    // first element of the segment in the row
    uint64_t len[TQ_MAX_SEGMENTS];    // elements
    uint64_t woff[TQ_MAX_SEGMENTS];   // first word of the segment's packed bits in the worker's packed row
};

struct CompressCall {
    const void* grad; bool bf16; uint64_t d, grad_stride; uint32_t n_workers;
    const tq_params_t* params;       // host array, or
    const tq_params_t* params_dev;   // device array (then bits / nonuniform come from the caller)
    uint32_t bits; bool nonuniform;
    uint64_t seed; uint32_t first_worker;
    uint32_t* packed; uint64_t words_stride, words_out;
    cudaStream_t stream;
    const SegTable* segs = nullptr;  // device parameters only: params_dev[n_workers * segs->n]; d and words_out are then unused
    int* launches = nullptr;         // device parameters only: receives the number of kernels launched
};
cudaError_t launch_compress(const CompressCall& c);
// bf16 rows through the per-bit-pattern decision table; *applied is false (and nothing is launched) when the
// table form does not fit the call, which then takes the element-wise kernels.
cudaError_t launch_compress_lut(const CompressCall& c, bool* applied);

struct DecompressCall {
    const uint32_t* packed; uint64_t words_stride, words_valid; uint32_t n_workers; uint64_t d;
    const tq_params_t* params;       // host array, or
    const tq_params_t* params_dev;   // device array (then bits comes from the caller)
    const float* weights; uint32_t bits;
    float* out; cudaStream_t stream;
    float* theta = nullptr; float* momentum_buf = nullptr; float lr = 0.0f, mu = 0.0f, wd = 0.0f;   // fused model update
    const uint32_t* const* rows = nullptr;   // host array of n_workers row pointers; when set, packed / words_stride are unused
    const SegTable* segs = nullptr;          // device parameters only: params_dev[n_workers * segs->n]; d and words_valid are then unused
};
cudaError_t launch_decompress(const DecompressCall& c);
cudaError_t read_wait_expired(unsigned int* count);
cudaError_t read_compress_wait_expired(unsigned int* count);   // the same for the tiled compress kernel   // give-ups of bounded barrier waits on the current device

struct StatsCall {
    const void* grad; bool bf16; uint64_t d, grad_stride; uint32_t n_workers;
    float g_min, kappa; tq_stats_t* stats; void* workspace; cudaStream_t stream;
    const SegTable* segs = nullptr;          // stats[n_workers * segs->n], workspace for that many jobs; d is then unused
};
// Enqueues the reduction; *launches receives the number of kernels launched.
cudaError_t launch_stats(const StatsCall& c, int* launches);
size_t stats_workspace_bytes(uint32_t n_workers);
// One-pass reduction with a power-of-two threshold and a caller-kept hint, plus the tail pass that
// runs only when the hint missed (two launches, the second usually returning at once).
cudaError_t launch_stats_hinted(const StatsCall& c, tq_gmin_hint_t* hint, int* launches);
// Same reduction with the library's built-in scratch array as workspace (c.workspace is ignored).
// *limit is set when n_workers exceeds what the array holds; nothing is launched then.
cudaError_t launch_stats_static(const StatsCall& c, int* launches, bool* limit);

// Parameter design on the device (one thread per worker); request already validated by params_request_ok.
bool params_request_ok(uint32_t num_levels, int mode, int rule, uint32_t* bits);
cudaError_t launch_params_device(const tq_stats_t* stats_dev, uint32_t n, uint32_t num_levels, uint32_t bits, uint32_t mode,
                                 double gamma, int rule, double alpha_user, tq_params_t* params_dev, cudaStream_t stream);

}  // namespace tq
