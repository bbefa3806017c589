// The C ABI of libtq (declared in include/tq.h): argument checking and kernel launches.
#include <atomic>
#include <cstdint>

#include "tq.h"
#include "tq_launch.h"

namespace {

thread_local int g_last_cuda_error = 0;
std::atomic<uint64_t> g_launches{0};

tq_status cuda_failed(cudaError_t e) {
    g_last_cuda_error = static_cast<int>(e);
    return TQ_ERR_CUDA;
}
bool aligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }
size_t elem_size(tq_dtype t) { return t == TQ_BF16 ? 2 : 4; }

// common checks on a [n_workers][grad_stride] gradient block
tq_status check_grad(const void* grad, tq_dtype dtype, uint64_t d, uint64_t stride, uint32_t n) {
    if (dtype != TQ_F32 && dtype != TQ_BF16) return TQ_ERR_INVALID_ARG;
    if (n == 0 || n > TQ_MAX_WORKERS) return TQ_ERR_INVALID_ARG;
    if (d > (1ull << 40)) return TQ_ERR_INVALID_ARG;
    if (d && !grad) return TQ_ERR_INVALID_ARG;
    if (stride < d) return TQ_ERR_INVALID_ARG;
    if (!aligned(grad, 32)) return TQ_ERR_ALIGNMENT;
    if (n > 1 && (stride * elem_size(dtype)) % 32 != 0) return TQ_ERR_ALIGNMENT;
    return TQ_OK;
}

tq_status check_params(const tq_params_t* p, uint32_t n, uint32_t* bits) {
    if (!p) return TQ_ERR_INVALID_ARG;
    const uint32_t b = p[0].bits;
    if (b < 1 || b > 4) return TQ_ERR_INVALID_ARG;
    for (uint32_t i = 0; i < n; ++i) {
        if (p[i].bits != b || p[i].num_levels != (1u << b)) return TQ_ERR_INVALID_ARG;
        if (p[i].mode != TQ_UNIFORM && p[i].mode != TQ_NONUNIFORM && p[i].mode != TQ_BISCALED) return TQ_ERR_INVALID_ARG;
        if (!(p[i].alpha > 0.0f)) return TQ_ERR_DOMAIN;
    }
    *bits = b;
    return TQ_OK;
}

}  // namespace

extern "C" {

size_t tq_packed_words(uint64_t d, uint32_t bits) {
    const uint64_t raw = (d * bits + 31) / 32;
    return static_cast<size_t>((raw + 3) / 4 * 4);
}

size_t tq_stats_workspace_bytes(uint32_t n_workers) { return tq::stats_workspace_bytes(n_workers); }

tq_status tq_stats(const void* grad_dev, tq_dtype dtype, uint64_t d, uint64_t grad_stride, uint32_t n_workers,
                   float g_min, float kappa, tq_stats_t* stats_dev, void* workspace_dev, size_t ws_bytes,
                   void* stream) {
    if (tq_status s = check_grad(grad_dev, dtype, d, grad_stride, n_workers)) return s;
    if (!stats_dev || !workspace_dev) return TQ_ERR_INVALID_ARG;
    if (!(g_min > 0.0f) && !(kappa > 0.0f)) return TQ_ERR_INVALID_ARG;
    if (!aligned(stats_dev, 8) || !aligned(workspace_dev, 256)) return TQ_ERR_ALIGNMENT;
    if (ws_bytes < tq::stats_workspace_bytes(n_workers)) return TQ_ERR_BUFFER_TOO_SMALL;
    tq::StatsCall c{grad_dev, dtype == TQ_BF16, d, grad_stride, n_workers, g_min, kappa, stats_dev, workspace_dev,
                    static_cast<cudaStream_t>(stream)};
    int launched = 0;
    const cudaError_t e = tq::launch_stats(c, &launched);
    g_launches += static_cast<uint64_t>(launched);
    return e == cudaSuccess ? TQ_OK : cuda_failed(e);
}

tq_status tq_stats_hinted(const void* grad_dev, tq_dtype dtype, uint64_t d, uint64_t grad_stride, uint32_t n_workers,
                          float kappa, tq_gmin_hint_t* hint_dev, tq_stats_t* stats_dev, void* workspace_dev,
                          size_t ws_bytes, void* stream) {
    if (tq_status s = check_grad(grad_dev, dtype, d, grad_stride, n_workers)) return s;
    if (!stats_dev || !workspace_dev || !hint_dev) return TQ_ERR_INVALID_ARG;
    if (!(kappa > 0.0f) || !(kappa <= 3.402823466e38f)) return TQ_ERR_INVALID_ARG;
    if (!aligned(stats_dev, 8) || !aligned(hint_dev, 8) || !aligned(workspace_dev, 256)) return TQ_ERR_ALIGNMENT;
    if (ws_bytes < tq::stats_workspace_bytes(n_workers)) return TQ_ERR_BUFFER_TOO_SMALL;
    tq::StatsCall c{grad_dev, dtype == TQ_BF16, d, grad_stride, n_workers, 0.0f, kappa, stats_dev, workspace_dev,
                    static_cast<cudaStream_t>(stream)};
    int launched = 0;
    const cudaError_t e = tq::launch_stats_hinted(c, hint_dev, &launched);
    g_launches += static_cast<uint64_t>(launched);
    return e == cudaSuccess ? TQ_OK : cuda_failed(e);
}

tq_status tq_stats_static(const void* grad_dev, tq_dtype dtype, uint64_t d, uint64_t grad_stride, uint32_t n_workers,
                          float g_min, float kappa, tq_stats_t* stats_dev, void* stream) {
    if (tq_status s = check_grad(grad_dev, dtype, d, grad_stride, n_workers)) return s;
    if (n_workers > TQ_STATIC_MAX_WORKERS) return TQ_ERR_STATIC_LIMIT;
    if (!stats_dev) return TQ_ERR_INVALID_ARG;
    if (!(g_min > 0.0f) && !(kappa > 0.0f)) return TQ_ERR_INVALID_ARG;
    if (!aligned(stats_dev, 8)) return TQ_ERR_ALIGNMENT;
    tq::StatsCall c{grad_dev, dtype == TQ_BF16, d, grad_stride, n_workers, g_min, kappa, stats_dev, nullptr,
                    static_cast<cudaStream_t>(stream)};
    int launched = 0;
    bool limit = false;
    const cudaError_t e = tq::launch_stats_static(c, &launched, &limit);
    if (limit) return TQ_ERR_STATIC_LIMIT;
    g_launches += static_cast<uint64_t>(launched);
    return e == cudaSuccess ? TQ_OK : cuda_failed(e);
}

tq_status tq_compress(const void* grad_dev, tq_dtype dtype, uint64_t d, uint64_t grad_stride, uint32_t n_workers,
                      const tq_params_t* params_host, uint64_t seed, uint32_t first_worker, uint32_t* packed_dev,
                      size_t words_stride, void* stream) {
    if (tq_status s = check_grad(grad_dev, dtype, d, grad_stride, n_workers)) return s;
    uint32_t bits = 0;
    if (tq_status s = check_params(params_host, n_workers, &bits)) return s;
    for (uint32_t i = 1; i < n_workers; ++i)      // one kernel per launch: all uniform, or all table codebooks
        if ((params_host[i].mode == TQ_UNIFORM) != (params_host[0].mode == TQ_UNIFORM)) return TQ_ERR_INVALID_ARG;
    const size_t need = tq_packed_words(d, bits);
    if (need && !packed_dev) return TQ_ERR_INVALID_ARG;
    if (!aligned(packed_dev, 16) || words_stride % 4 != 0) return TQ_ERR_ALIGNMENT;
    if (words_stride < need) return TQ_ERR_BUFFER_TOO_SMALL;
    if (d == 0) return TQ_OK;
    tq::CompressCall c{grad_dev, dtype == TQ_BF16, d, grad_stride, n_workers, params_host, nullptr, bits,
                       params_host[0].mode != TQ_UNIFORM, seed, first_worker, packed_dev, words_stride, need,
                       static_cast<cudaStream_t>(stream)};
    const cudaError_t e = tq::launch_compress(c);
    if (e != cudaSuccess) return cuda_failed(e);
    g_launches += 1;
    return TQ_OK;
}

tq_status tq_decompress_aggregate(const uint32_t* packed_dev, size_t words_stride, uint32_t n_workers, uint64_t d,
                                  const tq_params_t* params_host, const float* weights_host, float* out_dev,
                                  void* stream) {
    if (n_workers == 0 || n_workers > TQ_MAX_WORKERS || d > (1ull << 40)) return TQ_ERR_INVALID_ARG;
    uint32_t bits = 0;
    if (tq_status s = check_params(params_host, n_workers, &bits)) return s;
    const size_t need = tq_packed_words(d, bits);
    if (d && (!packed_dev || !out_dev)) return TQ_ERR_INVALID_ARG;
    if (!aligned(packed_dev, 16) || words_stride % 4 != 0 || !aligned(out_dev, 32)) return TQ_ERR_ALIGNMENT;
    if (words_stride < need) return TQ_ERR_BUFFER_TOO_SMALL;
    if (d == 0) return TQ_OK;
    tq::DecompressCall c{packed_dev, words_stride, need, n_workers, d, params_host, nullptr, weights_host, bits, out_dev,
                         static_cast<cudaStream_t>(stream)};
    const cudaError_t e = tq::launch_decompress(c);
    if (e != cudaSuccess) return cuda_failed(e);
    g_launches += 1;
    return TQ_OK;
}

tq_status tq_decompress_aggregate_rows(const uint32_t* const* rows_host, uint32_t n_workers, uint64_t d,
                                       const tq_params_t* params_host, const float* weights_host, float* out_dev,
                                       void* stream) {
    if (n_workers == 0 || n_workers > TQ_MAX_WORKERS || d > (1ull << 40)) return TQ_ERR_INVALID_ARG;
    uint32_t bits = 0;
    if (tq_status s = check_params(params_host, n_workers, &bits)) return s;
    if (!rows_host || (d && !out_dev)) return TQ_ERR_INVALID_ARG;
    for (uint32_t i = 0; i < n_workers; ++i) {
        if (d && !rows_host[i]) return TQ_ERR_INVALID_ARG;
        if (!aligned(rows_host[i], 16)) return TQ_ERR_ALIGNMENT;
    }
    if (!aligned(out_dev, 32)) return TQ_ERR_ALIGNMENT;
    if (d == 0) return TQ_OK;
    const size_t need = tq_packed_words(d, bits);
    tq::DecompressCall c{nullptr, 0, need, n_workers, d, params_host, nullptr, weights_host, bits, out_dev,
                         static_cast<cudaStream_t>(stream)};
    c.rows = rows_host;
    const cudaError_t e = tq::launch_decompress(c);
    if (e != cudaSuccess) return cuda_failed(e);
    g_launches += 1;
    return TQ_OK;
}

tq_status tq_params_device(const tq_stats_t* stats_dev, uint32_t n_workers, uint32_t num_levels, tq_mode mode,
                           double gamma, tq_alpha_rule alpha_rule, double alpha_user, tq_params_t* params_dev,
                           void* stream) {
    uint32_t bits = 0;
    if (!stats_dev || !params_dev || n_workers == 0 || n_workers > TQ_MAX_WORKERS * TQ_MAX_SEGMENTS) return TQ_ERR_INVALID_ARG;
    if (!tq::params_request_ok(num_levels, mode, alpha_rule, &bits)) return TQ_ERR_INVALID_ARG;
    if (alpha_rule == TQ_ALPHA_USER && !(alpha_user > 0.0)) return TQ_ERR_DOMAIN;
    if (!aligned(stats_dev, 8) || !aligned(params_dev, 8)) return TQ_ERR_ALIGNMENT;
    const cudaError_t e = tq::launch_params_device(stats_dev, n_workers, num_levels, bits, mode, gamma, alpha_rule,
                                                   alpha_user, params_dev, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_failed(e);
    g_launches += 1;
    return TQ_OK;
}

tq_status tq_compress_device_params(const void* grad_dev, tq_dtype dtype, uint64_t d, uint64_t grad_stride,
                                    uint32_t n_workers, const tq_params_t* params_dev, uint32_t num_levels, tq_mode mode,
                                    uint64_t seed, uint32_t first_worker, uint32_t* packed_dev, size_t words_stride,
                                    void* stream) {
    if (tq_status s = check_grad(grad_dev, dtype, d, grad_stride, n_workers)) return s;
    uint32_t bits = 0;
    if (!params_dev || !tq::params_request_ok(num_levels, mode, TQ_ALPHA_CLOSED, &bits)) return TQ_ERR_INVALID_ARG;
    const size_t need = tq_packed_words(d, bits);
    if (need && !packed_dev) return TQ_ERR_INVALID_ARG;
    if (!aligned(packed_dev, 16) || words_stride % 4 != 0 || !aligned(params_dev, 8)) return TQ_ERR_ALIGNMENT;
    if (words_stride < need) return TQ_ERR_BUFFER_TOO_SMALL;
    if (d == 0) return TQ_OK;
    tq::CompressCall c{grad_dev, dtype == TQ_BF16, d, grad_stride, n_workers, nullptr, params_dev, bits,
                       mode != TQ_UNIFORM, seed, first_worker, packed_dev, words_stride, need,
                       static_cast<cudaStream_t>(stream)};
    int launched = 0;
    c.launches = &launched;
    const cudaError_t e = tq::launch_compress(c);
    if (e != cudaSuccess) return cuda_failed(e);
    g_launches += static_cast<uint64_t>(launched);   // table mode: main kernel + the (usually empty) binary-search pass; bf16: + the decision-table kernel
    return TQ_OK;
}

tq_status tq_decompress_aggregate_device_params(const uint32_t* packed_dev, size_t words_stride, uint32_t n_workers,
                                                uint64_t d, const tq_params_t* params_dev, uint32_t num_levels,
                                                const float* weights_host, float* out_dev, void* stream) {
    if (n_workers == 0 || n_workers > TQ_MAX_WORKERS || d > (1ull << 40)) return TQ_ERR_INVALID_ARG;
    uint32_t bits = 0;
    if (!params_dev || !tq::params_request_ok(num_levels, TQ_UNIFORM, TQ_ALPHA_CLOSED, &bits)) return TQ_ERR_INVALID_ARG;
    const size_t need = tq_packed_words(d, bits);
    if (d && (!packed_dev || !out_dev)) return TQ_ERR_INVALID_ARG;
    if (!aligned(packed_dev, 16) || words_stride % 4 != 0 || !aligned(out_dev, 32) || !aligned(params_dev, 8)) return TQ_ERR_ALIGNMENT;
    if (words_stride < need) return TQ_ERR_BUFFER_TOO_SMALL;
    if (d == 0) return TQ_OK;
    tq::DecompressCall c{packed_dev, words_stride, need, n_workers, d, nullptr, params_dev, weights_host, bits, out_dev,
                         static_cast<cudaStream_t>(stream)};
    const cudaError_t e = tq::launch_decompress(c);
    if (e != cudaSuccess) return cuda_failed(e);
    g_launches += 1;
    return TQ_OK;
}

tq_status tq_decompress_aggregate_apply(const uint32_t* packed_dev, size_t words_stride, uint32_t n_workers, uint64_t d,
                                        const tq_params_t* params_host, const float* weights_host, float* theta_dev,
                                        float* momentum_dev, float lr, float momentum, float weight_decay, void* stream) {
    if (n_workers == 0 || n_workers > TQ_MAX_WORKERS || d > (1ull << 40)) return TQ_ERR_INVALID_ARG;
    uint32_t bits = 0;
    if (tq_status s = check_params(params_host, n_workers, &bits)) return s;
    const size_t need = tq_packed_words(d, bits);
    if (d && (!packed_dev || !theta_dev)) return TQ_ERR_INVALID_ARG;
    if (!(lr == lr) || !(momentum == momentum) || !(weight_decay == weight_decay)) return TQ_ERR_INVALID_ARG;
    if (!aligned(packed_dev, 16) || words_stride % 4 != 0 || !aligned(theta_dev, 32) || !aligned(momentum_dev, 32)) return TQ_ERR_ALIGNMENT;
    if (words_stride < need) return TQ_ERR_BUFFER_TOO_SMALL;
    if (d == 0) return TQ_OK;
    tq::DecompressCall c{packed_dev, words_stride, need, n_workers, d, params_host, nullptr, weights_host, bits, nullptr,
                         static_cast<cudaStream_t>(stream)};
    c.theta = theta_dev; c.momentum_buf = momentum_dev; c.lr = lr; c.mu = momentum; c.wd = weight_decay;
    const cudaError_t e = tq::launch_decompress(c);
    if (e != cudaSuccess) return cuda_failed(e);
    g_launches += 1;
    return TQ_OK;
}

// ---- layer groups -------------------------------------------------------------------------------------

static tq_status make_segments(const tq_segment_t* seg, uint32_t n_seg, uint32_t n_workers, uint64_t align_elems, uint32_t bits,
                               uint64_t limit, tq::SegTable* out) {
    if (!seg || n_seg == 0 || n_seg > TQ_MAX_SEGMENTS || n_workers == 0 || n_workers > TQ_MAX_WORKERS) return TQ_ERR_INVALID_ARG;
    uint64_t words = 0;
    out->n = n_seg; out->pad = 0;
    for (uint32_t s = 0; s < n_seg; ++s) {
        if (seg[s].length == 0 || seg[s].length > (1ull << 40) || seg[s].offset > (1ull << 40)) return TQ_ERR_INVALID_ARG;
        if (seg[s].offset + seg[s].length > limit) return TQ_ERR_INVALID_ARG;
        if (seg[s].offset % align_elems != 0) return TQ_ERR_ALIGNMENT;
        for (uint32_t t = 0; t < s; ++t)
            if (seg[s].offset < seg[t].offset + seg[t].length && seg[t].offset < seg[s].offset + seg[s].length) return TQ_ERR_INVALID_ARG;
        out->off[s] = seg[s].offset; out->len[s] = seg[s].length; out->woff[s] = words;
        words += bits ? tq_packed_words(seg[s].length, bits) : 0;
    }
    return TQ_OK;
}

size_t tq_segments_packed_words(const tq_segment_t* seg, uint32_t n_seg, uint32_t bits) {
    if (!seg || bits < 1 || bits > 4) return 0;
    size_t words = 0;
    for (uint32_t s = 0; s < n_seg; ++s) words += tq_packed_words(seg[s].length, bits);
    return words;
}

tq_status tq_stats_segments(const void* grad_dev, tq_dtype dtype, uint64_t grad_stride, uint32_t n_workers,
                            const tq_segment_t* segments_host, uint32_t n_segments, float g_min, float kappa,
                            tq_stats_t* stats_dev, void* workspace_dev, size_t ws_bytes, void* stream) {
    if (tq_status s = check_grad(grad_dev, dtype, 1, grad_stride, n_workers)) return s;
    static thread_local tq::SegTable segs;
    if (tq_status s = make_segments(segments_host, n_segments, n_workers, 32 / elem_size(dtype), 0, grad_stride, &segs)) return s;
    if (!stats_dev || !workspace_dev) return TQ_ERR_INVALID_ARG;
    if (!(g_min > 0.0f) && !(kappa > 0.0f)) return TQ_ERR_INVALID_ARG;
    if (!aligned(stats_dev, 8) || !aligned(workspace_dev, 256)) return TQ_ERR_ALIGNMENT;
    if (ws_bytes < tq::stats_workspace_bytes(n_workers * n_segments)) return TQ_ERR_BUFFER_TOO_SMALL;
    tq::StatsCall c{grad_dev, dtype == TQ_BF16, 0, grad_stride, n_workers, g_min, kappa, stats_dev, workspace_dev,
                    static_cast<cudaStream_t>(stream)};
    c.segs = &segs;
    int launched = 0;
    const cudaError_t e = tq::launch_stats(c, &launched);
    g_launches += static_cast<uint64_t>(launched);
    return e == cudaSuccess ? TQ_OK : cuda_failed(e);
}

tq_status tq_stats_hinted_segments(const void* grad_dev, tq_dtype dtype, uint64_t grad_stride, uint32_t n_workers,
                                   const tq_segment_t* segments_host, uint32_t n_segments, float kappa,
                                   tq_gmin_hint_t* hint_dev, tq_stats_t* stats_dev, void* workspace_dev, size_t ws_bytes,
                                   void* stream) {
    if (tq_status s = check_grad(grad_dev, dtype, 1, grad_stride, n_workers)) return s;
    static thread_local tq::SegTable segs;
    if (tq_status s = make_segments(segments_host, n_segments, n_workers, 32 / elem_size(dtype), 0, grad_stride, &segs)) return s;
    if (!stats_dev || !workspace_dev || !hint_dev) return TQ_ERR_INVALID_ARG;
    if (!(kappa > 0.0f) || !(kappa <= 3.402823466e38f)) return TQ_ERR_INVALID_ARG;
    if (!aligned(stats_dev, 8) || !aligned(hint_dev, 8) || !aligned(workspace_dev, 256)) return TQ_ERR_ALIGNMENT;
    if (ws_bytes < tq::stats_workspace_bytes(n_workers * n_segments)) return TQ_ERR_BUFFER_TOO_SMALL;
    tq::StatsCall c{grad_dev, dtype == TQ_BF16, 0, grad_stride, n_workers, 0.0f, kappa, stats_dev, workspace_dev,
                    static_cast<cudaStream_t>(stream)};
    c.segs = &segs;
    int launched = 0;
    const cudaError_t e = tq::launch_stats_hinted(c, hint_dev, &launched);
    g_launches += static_cast<uint64_t>(launched);
    return e == cudaSuccess ? TQ_OK : cuda_failed(e);
}

tq_status tq_compress_segments(const void* grad_dev, tq_dtype dtype, uint64_t grad_stride, uint32_t n_workers,
                               const tq_segment_t* segments_host, uint32_t n_segments, const tq_params_t* params_dev,
                               uint32_t num_levels, tq_mode mode, uint64_t seed, uint32_t first_worker,
                               uint32_t* packed_dev, size_t words_stride, void* stream) {
    if (tq_status s = check_grad(grad_dev, dtype, 1, grad_stride, n_workers)) return s;
    uint32_t bits = 0;
    if (!params_dev || !tq::params_request_ok(num_levels, mode, TQ_ALPHA_CLOSED, &bits)) return TQ_ERR_INVALID_ARG;
    static thread_local tq::SegTable segs;
    if (tq_status s = make_segments(segments_host, n_segments, n_workers, 32 / elem_size(dtype), bits, grad_stride, &segs)) return s;
    const size_t need = tq_segments_packed_words(segments_host, n_segments, bits);
    if (!packed_dev) return TQ_ERR_INVALID_ARG;
    if (!aligned(packed_dev, 16) || words_stride % 4 != 0 || !aligned(params_dev, 8)) return TQ_ERR_ALIGNMENT;
    if (words_stride < need) return TQ_ERR_BUFFER_TOO_SMALL;
    tq::CompressCall c{grad_dev, dtype == TQ_BF16, 0, grad_stride, n_workers, nullptr, params_dev, bits,
                       mode != TQ_UNIFORM, seed, first_worker, packed_dev, words_stride, 0,
                       static_cast<cudaStream_t>(stream)};
    c.segs = &segs;
    int launched = 0;
    c.launches = &launched;
    const cudaError_t e = tq::launch_compress(c);
    if (e != cudaSuccess) return cuda_failed(e);
    g_launches += static_cast<uint64_t>(launched);
    return TQ_OK;
}

tq_status tq_decompress_aggregate_segments(const uint32_t* packed_dev, size_t words_stride, uint32_t n_workers,
                                           const tq_segment_t* segments_host, uint32_t n_segments,
                                           const tq_params_t* params_dev, uint32_t num_levels,
                                           const float* weights_host, float* out_dev, void* stream) {
    uint32_t bits = 0;
    if (!params_dev || !tq::params_request_ok(num_levels, TQ_UNIFORM, TQ_ALPHA_CLOSED, &bits)) return TQ_ERR_INVALID_ARG;
    static thread_local tq::SegTable segs;
    if (tq_status s = make_segments(segments_host, n_segments, n_workers, 8, bits, ~0ull, &segs)) return s;
    const size_t need = tq_segments_packed_words(segments_host, n_segments, bits);
    if (!packed_dev || !out_dev) return TQ_ERR_INVALID_ARG;
    if (!aligned(packed_dev, 16) || words_stride % 4 != 0 || !aligned(out_dev, 32) || !aligned(params_dev, 8)) return TQ_ERR_ALIGNMENT;
    if (words_stride < need) return TQ_ERR_BUFFER_TOO_SMALL;
    tq::DecompressCall c{packed_dev, words_stride, 0, n_workers, 0, nullptr, params_dev, weights_host, bits, out_dev,
                         static_cast<cudaStream_t>(stream)};
    c.segs = &segs;
    const cudaError_t e = tq::launch_decompress(c);
    if (e != cudaSuccess) return cuda_failed(e);
    g_launches += 1;
    return TQ_OK;
}

const char* tq_strerror(tq_status s) {
    switch (s) {
        case TQ_OK: return "ok";
        case TQ_ERR_INVALID_ARG: return "invalid argument";
        case TQ_ERR_DOMAIN: return "parameter outside the model's domain";
        case TQ_ERR_ALIGNMENT: return "pointer or stride not aligned as required";
        case TQ_ERR_BUFFER_TOO_SMALL: return "buffer too small";
        case TQ_ERR_DEGENERATE_LEVELS: return "codebook not strictly increasing in fp32";
        case TQ_ERR_CUDA: return "CUDA runtime error";
        case TQ_ERR_STATIC_LIMIT: return "more workers than the built-in scratch of tq_stats_static holds (16)";
    }
    return "unknown status";
}

int tq_last_cuda_error(void) { return g_last_cuda_error; }
uint64_t tq_kernel_launches(void) { return g_launches.load(); }

tq_status tq_wait_expired_count(uint32_t* count_host) {
    if (!count_host) return TQ_ERR_INVALID_ARG;
    unsigned int n = 0, m = 0;
    cudaError_t e = tq::read_wait_expired(&n);
    if (e == cudaSuccess) e = tq::read_compress_wait_expired(&m);
    if (e != cudaSuccess) return cuda_failed(e);
    *count_host = n + m;
    return TQ_OK;
}

}  // extern "C"
