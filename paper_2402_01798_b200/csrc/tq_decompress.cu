// Server side of Algorithm 1: unpack the N workers' b-bit codes, look each up in that worker's
// codebook and average, out_j = (sum_i l^(i)[c_ij]) / N (w_i = 1/N as in Lemma 2) or sum_i w_i l^(i)[c_ij],
// fused in one streaming pass.  fp32 adds happen in worker order, so the result does not depend on
// the launch shape.
//
// Work split: a thread owns 32 output elements as units whose codes fill whole 32-bit words (see
// Unit below), keeps one fp32 accumulator per element in registers and walks the workers four at a
// time so that many independent loads are in flight before the dependent lookups start.
// Codebooks live in shared memory, 16 consecutive words per worker, four workers per 256 bytes: any
// set of codes of one worker maps to distinct banks, so lookups are conflict-free.
// HBM traffic per output element: N * bits / 8 bytes read, 4 bytes written.
#include "tq_device.cuh"
#include "tq_launch.h"

namespace tq {

struct DecompressArgs {
    float table[TQ_MAX_WORKERS][TQ_MAX_LEVELS];   // levels, already multiplied by w_i when weights are given
};
// Device-resident parameters: the codebooks are read from params_dev by each block; weights by value.
// Optional fused model update (Algorithm 1, last step, with the momentum SGD + weight decay of the
// paper's experiments): theta and the momentum buffer are read and written instead of `out`.
struct ApplyArgs {
    float* theta;          // nullptr: plain aggregation into `out`
    float* momentum_buf;   // may be nullptr (no momentum)
    float lr, mu, wd;
};
// Where each worker's packed row starts.  Rows need not be neighbours, nor even live on this GPU: any
// address the device can read (its own memory or a peer's mapped over NVLink) will do.
struct RowTable {
    const uint32_t* row[TQ_MAX_WORKERS];
};
struct DeviceTables {
    const tq_params_t* params_dev;    // nullptr: use DecompressArgs
    int use_weights;
    float weights[TQ_MAX_WORKERS];
};
// Layer groups: the tiles of all segments are numbered one after the other; segment sg owns tiles
// tile_begin[sg] .. tile_begin[sg + 1] - 1 and worker i's codebook for it is params_dev[i * n + sg].
struct SegTiles {
    SegTable segs;
    uint32_t tile_begin[TQ_MAX_SEGMENTS + 1];
};

__device__ __forceinline__ uint32_t ldg32_stream(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.global.nc.L1::no_allocate.b32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}

constexpr int kTabStride = 16;   // floats between consecutive workers' codebooks in shared memory: four codebooks per 256 bytes

// A unit is a run of elements decoded from one 32-bit "field": 8 / 16 / 32 elements = one packed word
// for 4 / 2 / 1 bits; for 3 bits 8 elements = 24 bits that start on a byte boundary and are cut out of
// two neighbouring words.  A thread owns 32 / kElems units, spaced one block apart, so that every
// load and every 256-bit store of a warp is contiguous, and keeps 32 accumulators in registers.
template <int BITS>
struct Unit {
    static constexpr int kElems = BITS == 2 ? 16 : (BITS == 1 ? 32 : 8);
#ifdef TQ_DECOMPRESS_ACC
    static constexpr int kUnits = TQ_DECOMPRESS_ACC / kElems > 0 ? TQ_DECOMPRESS_ACC / kElems : 1;
#else
    static constexpr int kUnits = 32 / kElems;
#endif
};

// The field of unit u of one row, all words known to be inside the row.
template <int BITS>
__device__ __forceinline__ uint32_t load_field(const uint32_t* row, uint64_t u) {
    if constexpr (BITS != 3) return ldg32_stream(row + u);
    else {
        const uint64_t wi = (3 * u) >> 2;                      // 24 u bits = 3 u bytes into the row
        const uint32_t sh = (static_cast<uint32_t>(u) * 24u) & 31u;
        const uint32_t lo = __ldg(row + wi), hi = __ldg(row + wi + 1);   // cached: neighbours share words
        return __funnelshift_r(lo, hi, sh);
    }
}
// Same with every word checked against the row's length (edge units).
template <int BITS>
__device__ __forceinline__ uint32_t load_field_guarded(const uint32_t* row, uint64_t u, uint64_t words_valid) {
    if constexpr (BITS != 3) return u < words_valid ? ldg32_stream(row + u) : 0u;
    else {
        const uint64_t wi = (3 * u) >> 2;
        const uint32_t sh = (static_cast<uint32_t>(u) * 24u) & 31u;
        const uint32_t lo = wi < words_valid ? __ldg(row + wi) : 0u;
        const uint32_t hi = wi + 1 < words_valid ? __ldg(row + wi + 1) : 0u;
        return __funnelshift_r(lo, hi, sh);
    }
}
// Words of the row a unit needs (for the interior test).
template <int BITS>
__device__ __forceinline__ uint64_t last_word_of(uint64_t u) {
    if constexpr (BITS != 3) return u;
    else return ((3 * u) >> 2) + 1;
}

// Adds one worker's dequantized values for the E codes of field f to acc[0 .. E-1].  `tab_bytes + base`
// is the worker's codebook in shared memory; base is a multiple of 256 (a group of four workers), the
// worker's place in its group is part of tab_bytes.
template <int BITS>
__device__ __forceinline__ void add_unit(f32x2* acc, uint32_t f, const char* tab_bytes, uint32_t base) {
    constexpr int E = Unit<BITS>::kElems;
    constexpr uint32_t kMask = (1u << BITS) - 1u;
    if constexpr (BITS != 3) {
        // The integer pipe is the scarce one here, so the codes are isolated once per word as bytes
        // already scaled to table offsets (code * 4), and each lookup offset then costs one
        // byte-permute: plane[j] byte m = 4 * code[m * (8 / BITS) + j]; offset = base with that byte
        // as its low byte.
        constexpr int kPerByte = 8 / BITS;
        constexpr uint32_t kPlaneMask = (kMask << 2) * 0x01010101u;
        uint32_t plane[kPerByte];
#pragma unroll
        for (int j = 0; j < kPerByte; ++j) {
            const int sh = j * BITS - 2;            // bring code j of every byte to bits 2..2+BITS
            const uint32_t v = sh < 0 ? (f << -sh) : (f >> sh);
            plane[j] = v & kPlaneMask;
        }
#pragma unroll
        for (int e = 0; e < E; e += 2) {       // two neighbouring elements per packed add
            const uint32_t off0 = __byte_perm(plane[e % kPerByte], base, 0x7650u + (e / kPerByte));
            const uint32_t off1 = __byte_perm(plane[(e + 1) % kPerByte], base, 0x7650u + ((e + 1) / kPerByte));
            acc[e / 2] = add2(acc[e / 2], pair(*reinterpret_cast<const float*>(tab_bytes + off0),
                                               *reinterpret_cast<const float*>(tab_bytes + off1)));
        }
    } else {
        // 3-bit codes do not line up with bytes: shift, then mask-and-merge with the base in one logic op
#pragma unroll
        for (int e = 0; e < E; e += 2) {
            const int sh0 = e * BITS - 2, sh1 = (e + 1) * BITS - 2;
            const uint32_t v0 = sh0 < 0 ? (f << -sh0) : (f >> sh0), v1 = f >> sh1;
            acc[e / 2] = add2(acc[e / 2], pair(*reinterpret_cast<const float*>(tab_bytes + ((v0 & (kMask << 2)) | base)),
                                               *reinterpret_cast<const float*>(tab_bytes + ((v1 & (kMask << 2)) | base))));
        }
    }
}

constexpr int kDecThreads = 128;

// Turns the accumulated sums of a thread's units into outputs: the division by N (w_i = 1/N; for N a
// power of two the product with 2^-k is the same value), then either the store of the aggregate or
// the fused model update.  Unit k of the thread is unit u0 + k * kDecThreads of the row.
template <int BITS, bool APPLY>
__device__ __forceinline__ void finish_units(f32x2 (&acc)[Unit<BITS>::kUnits][Unit<BITS>::kElems / 2], uint64_t u0, uint64_t d,
                                             float scale, int divide, const ApplyArgs& ap, float* __restrict__ out) {
    constexpr int E = Unit<BITS>::kElems, U = Unit<BITS>::kUnits;
#pragma unroll
    for (int k = 0; k < U; ++k) {
        float o[E];
#pragma unroll
        for (int e = 0; e < E / 2; ++e) unpair(acc[k][e], o[2 * e], o[2 * e + 1]);
#pragma unroll
        for (int e = 0; e < E; ++e) {
            if (divide == 1) o[e] = __fdiv_rn(o[e], scale);
            else if (divide == 2) o[e] = __fmul_rn(o[e], scale);
        }
        const uint64_t u = u0 + static_cast<uint64_t>(k) * kDecThreads;
        const uint64_t j0 = u * E;
        const bool whole = j0 + E <= d;
        if constexpr (APPLY) {
            // g += wd * theta; m = mu * m + g; theta -= lr * (m or g): fp32, one rounding per operation
#pragma unroll
            for (int v = 0; v < E / 8; ++v) {
                float th[8], mo[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const uint64_t j = j0 + 8 * v + e;
                    th[e] = (whole || j < d) ? ap.theta[j] : 0.0f;
                    mo[e] = (ap.momentum_buf && (whole || j < d)) ? ap.momentum_buf[j] : 0.0f;
                }
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    float gj = o[8 * v + e];
                    if (ap.wd != 0.0f) gj = __fadd_rn(gj, __fmul_rn(ap.wd, th[e]));
                    if (ap.momentum_buf) { mo[e] = __fadd_rn(__fmul_rn(ap.mu, mo[e]), gj); gj = mo[e]; }
                    th[e] = __fsub_rn(th[e], __fmul_rn(ap.lr, gj));
                }
                if (whole) {
                    stg256(ap.theta + j0 + 8 * v, th);
                    if (ap.momentum_buf) stg256(ap.momentum_buf + j0 + 8 * v, mo);
                } else {
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const uint64_t j = j0 + 8 * v + e;
                        if (j < d) { ap.theta[j] = th[e]; if (ap.momentum_buf) ap.momentum_buf[j] = mo[e]; }
                    }
                }
            }
        } else if (whole) {
#pragma unroll
            for (int v = 0; v < E / 8; ++v) {
                const float o8[8] = {o[8 * v], o[8 * v + 1], o[8 * v + 2], o[8 * v + 3],
                                     o[8 * v + 4], o[8 * v + 5], o[8 * v + 6], o[8 * v + 7]};
                stg256(out + j0 + 8 * v, o8);
            }
        } else {
#pragma unroll
            for (int e = 0; e < E; ++e)
                if (j0 + e < d) out[j0 + e] = o[e];
        }
    }
}

// Copies the N codebooks (already multiplied by w_i when weights are given) into shared memory.
__device__ __forceinline__ void fill_tables(float* s_tab, uint32_t n, const DecompressArgs& args, const DeviceTables& dt,
                                            uint32_t pstride = 1, uint32_t poff = 0) {
    for (uint32_t t = threadIdx.x; t < n * TQ_MAX_LEVELS; t += kDecThreads) {
        const uint32_t i = t / TQ_MAX_LEVELS, k = t % TQ_MAX_LEVELS;
        float v;
        if (dt.params_dev) {     // same rounded product w_i * l as the host forms for the by-value table
            const float l = dt.params_dev[i * pstride + poff].levels[k];
            v = dt.use_weights ? __fmul_rn(dt.weights[i], l) : l;
        } else {
            v = args.table[i][k];
        }
        s_tab[i * kTabStride + k] = v;
    }
}

// Blocks of 128 threads, eight resident per SM: the same 32 warps per SM as four blocks of 256, but
// a block that reaches its tail or its barrier leaves fewer lanes idle (measured 2-3 % faster).
// The fused update holds theta and the momentum buffer as well and gets two blocks fewer, which
// keeps it free of spills.
#ifndef TQ_DECOMPRESS_MIN_BLOCKS
#define TQ_DECOMPRESS_MIN_BLOCKS 8
#endif

template <int BITS, bool APPLY>
__global__ void __launch_bounds__(kDecThreads, APPLY ? TQ_DECOMPRESS_MIN_BLOCKS - 2 : TQ_DECOMPRESS_MIN_BLOCKS)
decompress_kernel(const __grid_constant__ RowTable rt, uint64_t words_valid, uint32_t n,
                  uint64_t d, const __grid_constant__ DecompressArgs args, const __grid_constant__ DeviceTables dt,
                  float scale, int divide, const __grid_constant__ ApplyArgs ap,
                  float* __restrict__ out) {
    constexpr int E = Unit<BITS>::kElems, U = Unit<BITS>::kUnits;

    // Every group of four codebooks starts on a 256-byte boundary of shared memory, so a table offset
    // (code * 4 < 64) can be merged into the group's base offset by the same byte-permute that
    // extracts it.  The lookups of one instruction go to one codebook, bank = code + 16 * (worker % 2):
    // they never conflict.
    __shared__ __align__(256) float s_tab[TQ_MAX_WORKERS * kTabStride];
    fill_tables(s_tab, n, args, dt);
    __syncthreads();
    const char* tab_bytes = reinterpret_cast<const char*>(s_tab);

    const uint64_t n_units = (d + E - 1) / E;
    const uint64_t u0 = static_cast<uint64_t>(blockIdx.x) * (kDecThreads * U) + threadIdx.x;   // unit k of this thread: u0 + k * kDecThreads
    if (u0 >= n_units) return;

    f32x2 acc[U][E / 2];          // fp32 accumulators, two per 64-bit register pair
#pragma unroll
    for (int k = 0; k < U; ++k)
#pragma unroll
        for (int e = 0; e < E / 2; ++e) acc[k][e] = both(0.0f);

    // interior: all U units exist and all their words lie inside the row
    const uint64_t u_last = u0 + static_cast<uint64_t>(U - 1) * kDecThreads;
    const bool interior = u_last < n_units && last_word_of<BITS>(u_last) < words_valid;

    uint32_t i = 0;
    if (interior) {
        for (; i + 4 <= n; i += 4) {          // four workers at a time: 4 * U independent fields in flight
            uint32_t f[4][U];
#pragma unroll
            for (int b = 0; b < 4; ++b)
#pragma unroll
                for (int k = 0; k < U; ++k)
                    f[b][k] = load_field<BITS>(rt.row[i + b], u0 + k * kDecThreads);
#pragma unroll
            for (int b = 0; b < 4; ++b)
#pragma unroll
                for (int k = 0; k < U; ++k)
                    add_unit<BITS>(acc[k], f[b][k], tab_bytes + b * (kTabStride * 4), i * (kTabStride * 4));
        }
    }
    for (; i < n; ++i) {                       // remaining workers, or every worker of an edge thread
        uint32_t f[U];
#pragma unroll
        for (int k = 0; k < U; ++k)
            f[k] = load_field_guarded<BITS>(rt.row[i],
                                            u0 + static_cast<uint64_t>(k) * kDecThreads, words_valid);
#pragma unroll
        for (int k = 0; k < U; ++k)
            add_unit<BITS>(acc[k], f[k], tab_bytes + (i & 3u) * (kTabStride * 4), (i & ~3u) * (kTabStride * 4));
    }

    finish_units<BITS, APPLY>(acc, u0, d, scale, divide, ap, out);
}


// ---------------------------------------------------------------------------------------------
// Bulk-copy variant for large inputs.  One block decodes one tile of kDecThreads * 32 outputs.  The
// packed bytes of the tile, kGroup workers at a time, are brought into a ring of shared-memory stages
// by asynchronous bulk copies (one per worker row, completion counted on an mbarrier), so the next
// workers' bytes are in flight while the current ones are looked up, and no registers are tied up by
// loads in flight.  A worker's bytes of one tile are contiguous in its row, start on a 16-byte
// boundary and are a multiple of 16 bytes long (rows are padded to 16 bytes), as a bulk copy needs.
// Every wait on a barrier is bounded; a wait that runs out makes the block count itself in
// g_wait_expired, wait (bounded again) for its copies still in flight and return without storing.
#ifndef TQ_DECOMPRESS_GROUP
#define TQ_DECOMPRESS_GROUP 4
#endif
constexpr int kGroup = TQ_DECOMPRESS_GROUP;   // workers per stage
#ifndef TQ_DECOMPRESS_STAGES
#define TQ_DECOMPRESS_STAGES 3
#endif

__device__ unsigned int g_wait_expired = 0;   // blocks (or threads) whose bounded wait ran out, since load

template <int BITS>
struct Tile {
    static constexpr int kUnitBytes = BITS == 3 ? 3 : 4;
    static constexpr int kUnits = kDecThreads * Unit<BITS>::kUnits;     // units per tile (a multiple of 4)
    static constexpr int kSegBytes = kUnits * kUnitBytes;               // one worker's bytes per tile (a multiple of 16)
};

// The field of local unit ul of a tile segment in shared memory (same cut as load_field; the tile's
// first unit is a multiple of 4, so the byte phase of a 3-bit unit is that of its local index).
template <int BITS>
__device__ __forceinline__ uint32_t stage_field(const uint32_t* seg, uint32_t ul) {
    if constexpr (BITS != 3) return seg[ul];
    else {
        const uint32_t wi = (3u * ul) >> 2, sh = (ul * 24u) & 31u;
        return __funnelshift_r(seg[wi], seg[wi + 1], sh);
    }
}

#ifndef TQ_DECOMPRESS_BULK_BLOCKS
#define TQ_DECOMPRESS_BULK_BLOCKS 8
#endif

template <int BITS, bool APPLY>
__global__ void __launch_bounds__(kDecThreads, APPLY ? TQ_DECOMPRESS_BULK_BLOCKS - 2 : TQ_DECOMPRESS_BULK_BLOCKS)
decompress_bulk_kernel(const __grid_constant__ RowTable rt, uint64_t words_row, uint32_t n,
                       uint64_t d_row, const __grid_constant__ DecompressArgs args, const __grid_constant__ DeviceTables dt,
                       float scale, int divide, const __grid_constant__ ApplyArgs ap_in, float* __restrict__ out_row,
                       const __grid_constant__ SegTiles st) {
    constexpr int E = Unit<BITS>::kElems, U = Unit<BITS>::kUnits, S = TQ_DECOMPRESS_STAGES;
    constexpr uint32_t kSeg = Tile<BITS>::kSegBytes;

    // [codebooks: n * 64 B][S stages of kGroup segments][16 B that a 3-bit field's second word may touch][S barriers]
    extern __shared__ __align__(1024) unsigned char smem[];
    float* s_tab = reinterpret_cast<float*>(smem);
    unsigned char* s_stage = smem + static_cast<size_t>(n) * (kTabStride * 4);
    const uint32_t stage0 = smem_addr(s_stage);
    const uint32_t bar0 = stage0 + S * kGroup * kSeg + 16;

    // which stream this block decodes: the whole rows, or one segment of them
    uint64_t tile = blockIdx.x, d = d_row, words_valid = words_row, row_shift = 0;    // row_shift: words from a row's start to the stream's
    float* out = out_row;
    ApplyArgs ap = ap_in;
    uint32_t pstride = 1, poff = 0;
    if (st.segs.n) {
        uint32_t sg = 0;
        while (sg + 1 < st.segs.n && st.tile_begin[sg + 1] <= blockIdx.x) ++sg;
        tile = blockIdx.x - st.tile_begin[sg];
        d = st.segs.len[sg];
        words_valid = (((d * BITS + 31) >> 5) + 3) & ~static_cast<uint64_t>(3);
        row_shift = st.segs.woff[sg];
        if (out) out += st.segs.off[sg];
        if (ap.theta) ap.theta += st.segs.off[sg];
        if (ap.momentum_buf) ap.momentum_buf += st.segs.off[sg];
        pstride = st.segs.n; poff = sg;
    }
    const uint64_t tile_off = tile * kSeg + row_shift * 4;                   // byte offset of the tile in every row
    const uint64_t row_bytes = (words_valid + row_shift) * 4;
    const uint32_t seg_bytes = static_cast<uint32_t>(row_bytes - tile_off < kSeg ? row_bytes - tile_off : kSeg);
    const uint32_t n_steps = (n + kGroup - 1) / kGroup;

    // step q = workers q*kGroup .. ; its bytes go to stage q % S
    auto issue = [&](uint32_t q) {
        const uint32_t st = q % S, i0 = q * kGroup;
        const uint32_t cnt = n - i0 < kGroup ? n - i0 : kGroup;
        const uint32_t bar = bar0 + 8 * st;
        mbar_expect_tx(bar, cnt * seg_bytes);
        for (uint32_t b = 0; b < cnt; ++b)
            bulk_load(stage0 + (st * kGroup + b) * kSeg, reinterpret_cast<const char*>(rt.row[i0 + b]) + tile_off, seg_bytes, bar);
    };

    if (threadIdx.x == 0) {
        for (int st = 0; st < S; ++st) mbar_init(bar0 + 8 * st, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        for (uint32_t q = 0; q < S && q < n_steps; ++q) issue(q);
    }
    fill_tables(s_tab, n, args, dt, pstride, poff);
    __syncthreads();          // barriers initialised and codebooks in place for every thread
    const char* tab_bytes = reinterpret_cast<const char*>(s_tab);

    f32x2 acc[U][E / 2];
#pragma unroll
    for (int k = 0; k < U; ++k)
#pragma unroll
        for (int e = 0; e < E / 2; ++e) acc[k][e] = both(0.0f);

    uint32_t q = 0;
    bool expired = false;
    for (; q < n_steps; ++q) {
        const uint32_t st = q % S, i0 = q * kGroup;
        const uint32_t cnt = n - i0 < kGroup ? n - i0 : kGroup;
        const bool ok = mbar_wait(bar0 + 8 * st, (q / S) & 1u);
        uint32_t f[kGroup][U];
        const uint32_t* seg = reinterpret_cast<const uint32_t*>(s_stage + static_cast<size_t>(st) * kGroup * kSeg);
#pragma unroll
        for (int b = 0; b < kGroup; ++b)
#pragma unroll
            for (int k = 0; k < U; ++k)
                f[b][k] = (ok && b < cnt) ? stage_field<BITS>(seg + b * (kSeg / 4), threadIdx.x + k * kDecThreads) : 0u;
        if (q + S < n_steps) {
            // every thread has taken its fields out of the stage: it may be refilled.  The same
            // barrier makes the give-up decision uniform.
            if (__syncthreads_or(!ok)) { expired = true; break; }
            if (threadIdx.x == 0) issue(q + S);
        } else if (!ok) {                      // one of the last S steps: no barrier left to agree on, this thread gives up alone
            expired = true;
            break;
        }
#pragma unroll
        for (int b = 0; b < kGroup; ++b) {
            if (b < cnt) {           // uniform: only the last step of a worker count not divisible by kGroup is short
#pragma unroll
                for (int k = 0; k < U; ++k)
                    add_unit<BITS>(acc[k], f[b][k], tab_bytes + b * (kTabStride * 4), i0 * (kTabStride * 4));
            }
        }
    }
    // A block barrier here would make the give-up of the last steps uniform as well; it was measured to cost 2-5 %
    // of the kernel (0.163 -> 0.167 ms and 0.161 -> 0.169 ms on 124 M x 8 with 4- and 2-bit codes), so a thread whose
    // wait runs out in one of the last S steps drops its own 32 outputs and counts itself.
    if (expired) {
        atomicAdd(&g_wait_expired, 1u);
        if (threadIdx.x == 0)      // the copies issued and not yet seen to land: steps q .. q + S - 1
            for (uint32_t r = q; r < q + S && r < n_steps; ++r) mbar_wait(bar0 + 8 * (r % S), (r / S) & 1u);
        return;
    }

    const uint64_t u0 = tile * Tile<BITS>::kUnits + threadIdx.x;
    if (u0 * E >= d) return;       // nothing of this thread's first unit (hence of any) exists
    finish_units<BITS, APPLY>(acc, u0, d, scale, divide, ap, out);
}

// Inputs of at least this many tiles go through the bulk-copy kernel; smaller ones are bound by
// launch and set-up latency and keep the simpler direct kernel.
constexpr uint64_t kBulkMinTiles = 8;

static const SegTiles kNoSegTiles{};

template <int BITS, bool APPLY>
static cudaError_t launch_bulk(const DecompressCall& c, const RowTable& rt, const DecompressArgs& args, const DeviceTables& dt,
                               float scale, int divide, const ApplyArgs& ap, uint64_t tiles, const SegTiles& st = kNoSegTiles) {
    const size_t smem = static_cast<size_t>(c.n_workers) * (kTabStride * 4) +
                        static_cast<size_t>(TQ_DECOMPRESS_STAGES) * kGroup * Tile<BITS>::kSegBytes + 16 + 8 * TQ_DECOMPRESS_STAGES;
    if (smem > 48 * 1024) {
        const cudaError_t e = cudaFuncSetAttribute(decompress_bulk_kernel<BITS, APPLY>,
                                                   cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e != cudaSuccess) return e;
    }
    decompress_bulk_kernel<BITS, APPLY><<<static_cast<unsigned>(tiles), kDecThreads, smem, c.stream>>>(
        rt, c.words_valid, c.n_workers, c.d, args, dt, scale, divide, ap, c.out, st);
    return cudaGetLastError();
}

template <int BITS>
static cudaError_t launch(const DecompressCall& c, const RowTable& rt, const DecompressArgs& args, const DeviceTables& dt, float scale,
                          int divide) {
    if (c.segs) {      // layer groups: the tiles of every segment in one grid, always through the bulk-copy kernel
        static thread_local SegTiles st;
        st.segs = *c.segs;
        const uint64_t per_tile = static_cast<uint64_t>(kDecThreads) * Unit<BITS>::kUnits * Unit<BITS>::kElems;   // elements
        uint64_t total = 0;
        for (uint32_t sg = 0; sg < c.segs->n; ++sg) {
            st.tile_begin[sg] = static_cast<uint32_t>(total);
            total += (c.segs->len[sg] + per_tile - 1) / per_tile;
            if (total > 0x7FFFFFFFull) return cudaErrorInvalidConfiguration;
        }
        st.tile_begin[c.segs->n] = static_cast<uint32_t>(total);
        const ApplyArgs ap{c.theta, c.momentum_buf, c.lr, c.mu, c.wd};
        return c.theta ? launch_bulk<BITS, true>(c, rt, args, dt, scale, divide, ap, total, st)
                       : launch_bulk<BITS, false>(c, rt, args, dt, scale, divide, ap, total, st);
    }
    const uint64_t n_units = (c.d + Unit<BITS>::kElems - 1) / Unit<BITS>::kElems;
    const uint64_t per_block = static_cast<uint64_t>(kDecThreads) * Unit<BITS>::kUnits;
    const uint64_t blocks = (n_units + per_block - 1) / per_block;
    if (blocks == 0) return cudaSuccess;
    if (blocks > 0x7FFFFFFFull) return cudaErrorInvalidConfiguration;
    const ApplyArgs ap{c.theta, c.momentum_buf, c.lr, c.mu, c.wd};
    if (blocks >= kBulkMinTiles)
        return c.theta ? launch_bulk<BITS, true>(c, rt, args, dt, scale, divide, ap, blocks)
                       : launch_bulk<BITS, false>(c, rt, args, dt, scale, divide, ap, blocks);
    if (c.theta)
        decompress_kernel<BITS, true><<<static_cast<unsigned>(blocks), kDecThreads, 0, c.stream>>>(
            rt, c.words_valid, c.n_workers, c.d, args, dt, scale, divide, ap, c.out);
    else
        decompress_kernel<BITS, false><<<static_cast<unsigned>(blocks), kDecThreads, 0, c.stream>>>(
            rt, c.words_valid, c.n_workers, c.d, args, dt, scale, divide, ap, c.out);
    return cudaGetLastError();
}

cudaError_t read_wait_expired(unsigned int* count) {
    return cudaMemcpyFromSymbol(count, g_wait_expired, sizeof(unsigned int));
}

cudaError_t launch_decompress(const DecompressCall& c) {
    static thread_local DecompressArgs args;
    static thread_local DeviceTables dt;
    static thread_local RowTable rt;
    for (uint32_t i = 0; i < c.n_workers; ++i)
        rt.row[i] = c.rows ? c.rows[i] : c.packed + static_cast<uint64_t>(i) * c.words_stride;
    dt.params_dev = c.params_dev;
    dt.use_weights = c.weights ? 1 : 0;
    for (uint32_t i = 0; i < c.n_workers; ++i) {
        dt.weights[i] = c.weights ? c.weights[i] : 0.0f;
        if (c.params_dev) continue;
        for (int k = 0; k < TQ_MAX_LEVELS; ++k) {
            const float l = c.params[i].levels[k];
            // weighted form: each product w_i * l is rounded to fp32 once; it depends on (i, k) only,
            // so it is formed here instead of once per element
            args.table[i][k] = c.weights ? c.weights[i] * l : l;
        }
    }
    float scale = 1.0f;
    int divide = 0;
    if (!c.weights) {
        const uint32_t n = c.n_workers;
        if ((n & (n - 1)) == 0) { divide = 2; scale = 1.0f / static_cast<float>(n); }
        else { divide = 1; scale = static_cast<float>(n); }
    }
    switch (c.bits) {
        case 1: return launch<1>(c, rt, args, dt, scale, divide);
        case 2: return launch<2>(c, rt, args, dt, scale, divide);
        case 3: return launch<3>(c, rt, args, dt, scale, divide);
        default: return launch<4>(c, rt, args, dt, scale, divide);
    }
}

}  // namespace tq
