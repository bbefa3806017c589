// Internal host-side interface between the C ABI (tq_api.cu) and the kernel files.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "tq.h"

namespace tq {

struct CompressCall {
    const void* grad; bool bf16; uint64_t d, grad_stride; uint32_t n_workers;
    const tq_params_t* params; uint32_t bits; bool nonuniform;
    uint64_t seed; uint32_t first_worker;
    uint32_t* packed; uint64_t words_stride, words_out;
    cudaStream_t stream;
};
cudaError_t launch_compress(const CompressCall& c);

struct DecompressCall {
    const uint32_t* packed; uint64_t words_stride, words_valid; uint32_t n_workers; uint64_t d;
    const tq_params_t* params; const float* weights; uint32_t bits;
    float* out; cudaStream_t stream;
};
cudaError_t launch_decompress(const DecompressCall& c);

struct StatsCall {
    const void* grad; bool bf16; uint64_t d, grad_stride; uint32_t n_workers;
    float g_min, kappa; tq_stats_t* stats; void* workspace; cudaStream_t stream;
};
// Enqueues the reduction; *launches receives the number of kernels launched.
cudaError_t launch_stats(const StatsCall& c, int* launches);
size_t stats_workspace_bytes(uint32_t n_workers);
// Same reduction with the library's built-in scratch array as workspace (c.workspace is ignored).
// *limit is set when n_workers exceeds what the array holds; nothing is launched then.
cudaError_t launch_stats_static(const StatsCall& c, int* launches, bool* limit);

}  // namespace tq
