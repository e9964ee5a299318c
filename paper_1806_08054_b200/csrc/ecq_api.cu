// C ABI of the ECQ-SGD codec: argument checks, launch configuration, status word.
#include <algorithm>
#include <atomic>
#include <cstdint>
#include <cstdlib>
#include <cmath>
#include <cstring>
#include <mutex>
#include <new>
#include <utility>
#include <vector>

#include <cuda.h>
#include <cuda_runtime.h>

#include "../../include/ecq.h"
#include "ecq_common.cuh"
#include "ecq_decode.cuh"
#include "ecq_decode_ring.cuh"
#include "ecq_encode.cuh"
#include "ecq_stats.cuh"
#include "ecq_entropy.cuh"

using namespace ecq;

namespace {

// Launch of one of the persistent kernels.  With `overlap` the launch carries the programmatic
// stream-serialisation attribute: the kernel may be scheduled while its predecessor in the
// stream drains (which hides the launch latency and the prologue, about 2 us a launch) and
// calls griddep_wait() before its first global access.  Only launches that fill every CTA slot
// of the GPU (`full_grid` CTAs) ask for it: their CTAs land evenly whenever they are placed,
// while a smaller grid placed into the slots an earlier kernel happens to free first would
// double up on some SMs and leave others empty (measured: 20 % slower on 128 CTAs).
template <typename... KArgs, typename... Args>
cudaError_t launch_persistent(void (*kern)(KArgs...), uint32_t grid, uint32_t full_grid,
                              uint32_t block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = grid == full_grid ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

std::atomic<uint64_t> g_launches{0};

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn tensor_map_encoder() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) ==
                cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

// Per-device set-up (kernel attributes, the built-in scratch's address) is kept in tables
// indexed by the device ordinal; contexts on devices beyond them are refused.
constexpr int kMaxDevices = 64;

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool aligned4(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 3u) == 0; }

}  // namespace

struct ecq_ctx {
    CodecParams P;
    uint64_t nb, n_words;
    int device;
    int sm_count;
    uint32_t* d_status;
    uint32_t* h_status;          // pinned
    bool tiled_ok;               // bucket is a power of two <= 4096
    int decode_kernel;           // ECQ_DECODE_AUTO / _WARP / _RING (ecq_set_decode_plan)
    uint32_t decode_max_ctas;    // 0: fill the device
    uint32_t wait_limit;         // polls an in-kernel wait makes before it gives up
    // lazily created by ecq_step_host
    std::mutex host_mu;
    cudaStream_t copy_stream;
    cudaEvent_t ev_copied[2], ev_encoded[2], ev_start;
    bool host_ready;
};

namespace {

// One row of the tiled view is 32 floats; a box is a whole tile (128 or 256 rows).  A map is a
// pure function of (base, rows), and encoding one costs microseconds on the host, which
// would dominate small vectors: each host thread keeps the maps it made in a small
// direct-mapped cache.
bool make_tile_map(CUtensorMap* tm, const float* base, uint64_t rows, uint32_t box_rows) {
    struct Entry { const float* base; uint64_t rows; uint32_t box_rows; CUtensorMap map; };
    constexpr unsigned kEntries = 256;
    thread_local Entry cache[kEntries];          // zero-initialised: base == nullptr is empty
    const uintptr_t a = reinterpret_cast<uintptr_t>(base);
    Entry& e = cache[((a >> 8) ^ (a >> 16) ^ (a >> 24) ^ box_rows) & (kEntries - 1)];
    if (e.base == base && e.rows == rows && e.box_rows == box_rows) { *tm = e.map; return true; }
    EncodeTiledFn enc = tensor_map_encoder();
    if (!enc) return false;
    // the encoder is a driver call: a host thread that has made no runtime call yet has no
    // context bound, so bind the current device's primary context once per thread
    // (cudaSetDevice does that and allocates nothing)
    thread_local bool context_bound = false;
    if (!context_bound) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaSetDevice(dev) != cudaSuccess) return false;
        context_bound = true;
    }
    const cuuint64_t dims[2] = {32, rows};
    const cuuint64_t strides[1] = {128};
    const cuuint32_t box[2] = {32, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides,
            box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    e.base = base; e.rows = rows; e.box_rows = box_rows; e.map = *tm;
    return true;
}

// Buffers of one batch entry as the launchers see them.
struct WorkerBuffers {
    const float* g;
    float* h;
    uint32_t* codes;
    float* scales;
};

template <int R, bool MODE1, int ROWS>
int launch_encode_tiled(ecq_ctx* c, uint32_t worker_base, uint32_t n_workers, uint32_t step,
                        const WorkerBuffers* wb, cudaStream_t st, uint32_t n_tiles) {
    using L = EncodeSmem<R, ROWS>;
    static std::once_flag once[kMaxDevices];
    static int occ[kMaxDevices];
    const int dev = c->device;                            // < kMaxDevices: checked at creation
    auto kern = encode_tiled_kernel<R, MODE1, ROWS>;
    std::call_once(once[dev], [&] {
        int o = 0;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal) ==
                cudaSuccess &&
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o, kern, ROWS, L::kTotal) == cudaSuccess)
            occ[dev] = o;
    });
    if (occ[dev] <= 0) return ECQ_ERR_CUDA;
    EncodeBatch bt;
    const uint64_t rows = (uint64_t)n_tiles * ROWS;
    for (uint32_t e = 0; e < (uint32_t)kMaxBatch; ++e) {
        const uint32_t src = e < n_workers ? e : 0;       // unused entries repeat entry 0
        if (e < n_workers) {
            if (!make_tile_map(&bt.tm_g[e], wb[e].g, rows, ROWS) ||
                !make_tile_map(&bt.tm_h[e], wb[e].h, rows, ROWS))
                return ECQ_ERR_CUDA;
        } else {
            bt.tm_g[e] = bt.tm_g[0];
            bt.tm_h[e] = bt.tm_h[0];
        }
        bt.g[e] = wb[src].g; bt.h[e] = wb[src].h;
        bt.codes[e] = wb[src].codes; bt.scales[e] = wb[src].scales;
    }
    const uint64_t total = (uint64_t)n_tiles * n_workers;
    const uint32_t full = (uint32_t)(c->sm_count * occ[dev]);
    uint32_t grid = full;
    if (grid > total) grid = (uint32_t)total;
    launch_persistent(kern, grid, full, (uint32_t)ROWS, (size_t)L::kTotal, st, bt, c->P, worker_base,
                      n_workers, step, c->d_status, n_tiles, c->wait_limit);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? ECQ_OK : ECQ_ERR_CUDA;
}

// Launches whose algorithmic traffic exceeds this run long enough (about 5 ms) to meet the
// board's power cap, where the 128-row shape sustains more; below it the 256-row shape wins.
constexpr uint64_t kLongLaunchBytes = 32ull << 30;

template <int R>
int launch_encode_tiled_mode(ecq_ctx* c, uint32_t worker_base, uint32_t n_workers, uint32_t step,
                             const WorkerBuffers* wb, cudaStream_t st) {
    const uint64_t bytes = (uint64_t)n_workers * c->P.d * 12;
    const bool small_tiles = bytes > kLongLaunchBytes || c->P.d < 8192;
    const uint64_t elems = small_tiles ? 4096 : 8192;
    const uint64_t n_tiles64 = c->P.d / elems;
    if (n_tiles64 == 0 || n_tiles64 * n_workers > 0xFFFFFFFFull || n_tiles64 * 256 > 0x7FFFFFFFull)
        return -1;                                        // not for the tiled path
    const uint32_t n_tiles = (uint32_t)n_tiles64;
    if (small_tiles)
        return c->P.mode ? launch_encode_tiled<R, true, 128>(c, worker_base, n_workers, step, wb, st, n_tiles)
                         : launch_encode_tiled<R, false, 128>(c, worker_base, n_workers, step, wb, st, n_tiles);
    return c->P.mode ? launch_encode_tiled<R, true, 256>(c, worker_base, n_workers, step, wb, st, n_tiles)
                     : launch_encode_tiled<R, false, 256>(c, worker_base, n_workers, step, wb, st, n_tiles);
}

int launch_encode_generic(ecq_ctx* c, uint32_t worker, uint32_t step, const float* g, float* h,
                          uint32_t* codes, float* scales, cudaStream_t st) {
    const uint64_t want = c->nb;
    const uint32_t grid = (uint32_t)(want < (uint64_t)c->sm_count * 16 ? want : (uint64_t)c->sm_count * 16);
    encode_generic_kernel<256><<<grid, 256, 0, st>>>(c->P, worker, step, g, h, codes, scales,
                                                      c->d_status, 0, c->nb);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? ECQ_OK : ECQ_ERR_CUDA;
}

// Encode n_workers vectors (workers worker_base .. worker_base + n_workers - 1).  The tiled
// path takes the whole batch in one launch; other shapes go one launch per worker.
int encode_batch_impl(ecq_ctx* c, uint32_t worker_base, uint32_t n_workers, uint32_t step,
                      const WorkerBuffers* wb, cudaStream_t st) {
    if (c->tiled_ok) {
        int rc = -1;
        switch (c->P.r) {
            case 2: rc = launch_encode_tiled_mode<2>(c, worker_base, n_workers, step, wb, st); break;
            case 3: rc = launch_encode_tiled_mode<3>(c, worker_base, n_workers, step, wb, st); break;
            case 4: rc = launch_encode_tiled_mode<4>(c, worker_base, n_workers, step, wb, st); break;
            case 5: rc = launch_encode_tiled_mode<5>(c, worker_base, n_workers, step, wb, st); break;
            case 6: rc = launch_encode_tiled_mode<6>(c, worker_base, n_workers, step, wb, st); break;
            case 7: rc = launch_encode_tiled_mode<7>(c, worker_base, n_workers, step, wb, st); break;
            case 8: rc = launch_encode_tiled_mode<8>(c, worker_base, n_workers, step, wb, st); break;
            case 9: rc = launch_encode_tiled_mode<9>(c, worker_base, n_workers, step, wb, st); break;
            default: break;
        }
        if (rc >= 0) return rc;
    }
    for (uint32_t e = 0; e < n_workers; ++e) {
        const int rc = launch_encode_generic(c, worker_base + e, step, wb[e].g, wb[e].h, wb[e].codes,
                                             wb[e].scales, st);
        if (rc != ECQ_OK) return rc;
    }
    return ECQ_OK;
}

int encode_impl(ecq_ctx* c, uint32_t worker, uint32_t step, const float* g, float* h,
                uint32_t* codes, float* scales, cudaStream_t st) {
    const WorkerBuffers wb = {g, h, codes, scales};
    return encode_batch_impl(c, worker, 1, step, &wb, st);
}

template <int R>
void launch_decode(ecq_ctx* c, uint32_t W, const MessageTable& tab, DecodeOut out, cudaStream_t st,
                   float w_recip, int w_pow2, DecodeSlice sl) {
    constexpr int G = DecodeGroup<R>::kElems;
    const uint64_t n_groups = (c->P.d + G - 1) / G;
    uint64_t blocks = (n_groups + 255) / 256;
    const uint64_t cap = (uint64_t)c->sm_count * 64;
    if (blocks > cap) blocks = cap;
    decode_mean_kernel<R><<<(uint32_t)blocks, 256, 0, st>>>(c->P, W, tab, out, n_groups,
                                                            c->n_words, w_recip, w_pow2, sl);
}

// Tiled decode: returns false when the shape is not covered (caller falls back).
template <int R, bool CARRY>
bool launch_decode_tiled(ecq_ctx* c, uint32_t W, const MessageTable& tab, DecodeOut out,
                         cudaStream_t st, float w_recip, int w_pow2, DecodeSlice sl) {
    using L = DecodeTiled<R>;
    const uint32_t B = c->P.bucket;
    const uint64_t n_tiles64 = c->P.d / kDecTileElems;
    if ((B & (B - 1)) != 0 || n_tiles64 == 0 || n_tiles64 > 0xFFFFFFFFull) return false;
    const uint32_t gsz = B >= 1024 ? 32 : B / 32;
    if (W > (uint32_t)kDecAreg * gsz) return false;
    if (n_tiles64 * W > 0xFFFFFFFFull) return false;
    static std::once_flag once[kMaxDevices];
    static int occ[kMaxDevices];
    const int dev = c->device;                            // < kMaxDevices: checked at creation
    auto kern = decode_tiled_kernel<R, CARRY>;
    std::call_once(once[dev], [&] {
        int o = 0;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kSmem) ==
                cudaSuccess &&
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o, kern, kDecWarps * 32, L::kSmem) ==
                cudaSuccess)
            occ[dev] = o;
    });
    if (occ[dev] <= 0) return false;
    const uint32_t n_tiles = (uint32_t)n_tiles64;
    const uint32_t full = (uint32_t)(c->sm_count * occ[dev]);
    uint32_t grid = full;
    const uint32_t want = (n_tiles + kDecWarps - 1) / kDecWarps;
    if (grid > want) grid = want;
    if (c->decode_max_ctas && grid > c->decode_max_ctas) grid = c->decode_max_ctas;
    launch_persistent(kern, grid, full, (uint32_t)(kDecWarps * 32), (size_t)L::kSmem, st, c->P, W, tab,
                      out, n_tiles, c->n_words, w_recip, w_pow2, 0x4B000000u, sl);
    return true;
}

// Ring decode (long vectors): returns false when the shape is not covered or the vector is
// too short to give every CTA a few tiles (caller goes on to the warp-tiled kernel).
template <int R, bool CARRY>
bool launch_decode_ring(ecq_ctx* c, uint32_t W, const MessageTable& tab, DecodeOut out,
                        cudaStream_t st, float w_recip, int w_pow2, DecodeSlice sl) {
    using L = DecodeRing<R>;
    const uint32_t B = c->P.bucket;
    const uint64_t n_subs64 = c->P.d / kDecTileElems;
    if ((B & (B - 1)) != 0 || n_subs64 == 0 || n_subs64 > 0xFFFFFFFFull) return false;
    const uint32_t gsz = B >= 1024 ? 32 : B / 32;
    if (W > (uint32_t)kDecAreg * gsz) return false;
    // the kernel stores 32 bytes at a time
    if ((reinterpret_cast<uintptr_t>(out.out) & 31u) || (reinterpret_cast<uintptr_t>(out.params) & 31u))
        return false;
    const uint64_t n_tiles = (n_subs64 + kRingSubs - 1) / kRingSubs;
    if (n_tiles * W > 0xFFFFFFFFull) return false;
    static std::once_flag once[kMaxDevices];
    static int occ[kMaxDevices];
    const int dev = c->device;                            // < kMaxDevices: checked at creation
    auto kern = decode_ring_kernel<R, CARRY>;
    std::call_once(once[dev], [&] {
        int o = 0;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kMaxSmem) ==
                cudaSuccess &&
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o, kern, kRingThreads, L::kMaxSmem) ==
                cudaSuccess)
            occ[dev] = o;
    });
    if (occ[dev] <= 0) return false;
    const RingLayout lay = ring_layout<R>(W, B);
    if (lay.stages < 3) return false;
    const uint32_t full = (uint32_t)(c->sm_count * occ[dev]);
    uint32_t grid = full;
    const uint64_t min_tiles_per_cta = (uint64_t)ring_min_tiles_per_cta(R, W);
    if (c->decode_kernel == ECQ_DECODE_AUTO && (n_tiles < min_tiles_per_cta * grid || R > kRingMaxAutoBits))
        return false;
    if (c->decode_max_ctas && grid > c->decode_max_ctas) grid = c->decode_max_ctas;
    if (grid > n_tiles) grid = (uint32_t)n_tiles;
    launch_persistent(kern, grid, full, (uint32_t)kRingThreads, (size_t)lay.smem, st, c->P, W, tab, out,
                      (uint32_t)n_subs64, c->n_words, w_recip, w_pow2,
                      L::kHalf ? 0x64006400u : 0x4B000000u, c->wait_limit, lay, sl, c->d_status);
    return true;
}

// One launch over the W <= 64 messages of `tab`; w_all is the number of messages of the whole
// mean (the divisor), of which this launch may be one slice (out.first / out.last).
int decode_launch(ecq_ctx* c, uint32_t W, uint32_t w_all, const MessageTable& tab, DecodeOut out,
                  bool first, bool last, cudaStream_t st) {
    const int w_pow2 = (w_all & (w_all - 1)) == 0;
    const float w_recip = 1.0f / (float)w_all;
    const DecodeSlice sl{(float)w_all, first, last};
    bool done = false;
    if (c->decode_kernel != ECQ_DECODE_WARP) switch (c->P.r) {
#define ECQ_CASE(R) case R: done = (first && last)                                                      \
            ? launch_decode_ring<R, false>(c, W, tab, out, st, w_recip, w_pow2, sl)                      \
            : launch_decode_ring<R, true>(c, W, tab, out, st, w_recip, w_pow2, sl); break;
        ECQ_CASE(2) ECQ_CASE(3) ECQ_CASE(4) ECQ_CASE(5) ECQ_CASE(6) ECQ_CASE(7) ECQ_CASE(8) ECQ_CASE(9)
#undef ECQ_CASE
        default: break;
    }
    if (!done) switch (c->P.r) {
#define ECQ_CASE(R) case R: done = (first && last)                                                      \
            ? launch_decode_tiled<R, false>(c, W, tab, out, st, w_recip, w_pow2, sl)                     \
            : launch_decode_tiled<R, true>(c, W, tab, out, st, w_recip, w_pow2, sl); break;
        ECQ_CASE(2) ECQ_CASE(3) ECQ_CASE(4) ECQ_CASE(5) ECQ_CASE(6) ECQ_CASE(7) ECQ_CASE(8) ECQ_CASE(9)
#undef ECQ_CASE
        default: break;
    }
    if (!done) switch (c->P.r) {
#define ECQ_CASE(R) case R: launch_decode<R>(c, W, tab, out, st, w_recip, w_pow2, sl); break;
        ECQ_CASE(2) ECQ_CASE(3) ECQ_CASE(4) ECQ_CASE(5) ECQ_CASE(6) ECQ_CASE(7) ECQ_CASE(8) ECQ_CASE(9)
#undef ECQ_CASE
        default: {
            const uint64_t n_groups = (c->P.d + 31) / 32;
            uint64_t blocks = (n_groups + 255) / 256;
            const uint64_t cap = (uint64_t)c->sm_count * 64;
            if (blocks > cap) blocks = cap;
            decode_mean_generic_kernel<<<(uint32_t)blocks, 256, 0, st>>>(
                c->P, W, tab, out, n_groups, c->n_words, w_recip, w_pow2, sl);
        }
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? ECQ_OK : ECQ_ERR_CUDA;
}

// Eq. 4 over W messages, 64 per launch; between launches the running sums live in `out`.
int decode_impl(ecq_ctx* c, uint32_t W, const uint32_t* const* codes, const float* const* scales,
                float* out, float* params, float neg_eta, cudaStream_t st) {
    if (W > (uint32_t)kMaxBatch && !out) return ECQ_ERR_ARG;
    for (uint32_t w = 0; w < W; ++w)
        if (!codes[w] || !scales[w] || !aligned16(codes[w]) || !aligned4(scales[w]))
            return ECQ_ERR_ARG;
    for (uint32_t w0 = 0; w0 < W; w0 += kMaxBatch) {
        const uint32_t n = std::min<uint32_t>(kMaxBatch, W - w0);
        MessageTable tab;
        std::memset(&tab, 0, sizeof(tab));
        for (uint32_t k = 0; k < n; ++k) {
            tab.codes[k] = codes[w0 + k];
            tab.scales[k] = scales[w0 + k];
        }
        const int rc = decode_launch(c, n, W, tab, DecodeOut{out, params, neg_eta}, w0 == 0,
                                     w0 + n == W, st);
        if (rc != ECQ_OK) return rc;
    }
    return ECQ_OK;
}

inline uint64_t round_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

}  // namespace

extern "C" {

int ecq_create(ecq_ctx** out, uint64_t d, uint32_t bucket, uint32_t levels, float alpha,
               float beta, uint64_t seed) {
    if (!out) return ECQ_ERR_ARG;
    *out = nullptr;
    if (d == 0 || bucket < 32 || bucket % 32 != 0 || levels == 0 || levels > 32767)
        return ECQ_ERR_ARG;
    if (!(alpha >= 0.f) || !(beta >= 0.f) || !(beta <= 1.f) || !(alpha < INFINITY))
        return ECQ_ERR_ARG;
    ecq_ctx* c = new (std::nothrow) ecq_ctx();
    if (!c) return ECQ_ERR_ALLOC;
    CodecParams& P = c->P;
    P.d = d; P.bucket = bucket; P.s = levels; P.mode = 0; P.norm = 0;
    P.alpha = alpha; P.beta = beta; P.sf = (float)levels;
    P.r = 0;
    while ((1ull << P.r) < 2ull * levels + 1ull) ++P.r;
    uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
    for (int i = 0; i < 10; ++i) {
        P.key0[i] = k0; P.key1[i] = k1;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    c->nb = (d + bucket - 1) / bucket;
    c->n_words = (d * P.r + 31) / 32;
    c->tiled_ok = (bucket & (bucket - 1)) == 0 && bucket <= kMaxTiledBucket;
    c->decode_kernel = ECQ_DECODE_AUTO;
    c->decode_max_ctas = 0;
    c->wait_limit = kWaitLimit;
    c->host_ready = false;
    c->d_status = nullptr; c->h_status = nullptr;
    if (cudaGetDevice(&c->device) != cudaSuccess || c->device < 0 || c->device >= kMaxDevices ||
        cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device) != cudaSuccess) {
        delete c; return ECQ_ERR_CUDA;
    }
    if (cudaMalloc(&c->d_status, sizeof(uint32_t)) != cudaSuccess ||
        cudaMallocHost(&c->h_status, sizeof(uint32_t)) != cudaSuccess) {
        if (c->d_status) cudaFree(c->d_status);
        delete c; return ECQ_ERR_ALLOC;
    }
    if (cudaMemset(c->d_status, 0, sizeof(uint32_t)) != cudaSuccess) {
        cudaFree(c->d_status); cudaFreeHost(c->h_status); delete c; return ECQ_ERR_CUDA;
    }
    *out = c;
    return ECQ_OK;
}

void ecq_destroy(ecq_ctx* c) {
    if (!c) return;
    if (c->host_ready) {
        cudaStreamDestroy(c->copy_stream);
        for (int i = 0; i < 2; ++i) { cudaEventDestroy(c->ev_copied[i]); cudaEventDestroy(c->ev_encoded[i]); }
        cudaEventDestroy(c->ev_start);
    }
    if (c->d_status) cudaFree(c->d_status);
    if (c->h_status) cudaFreeHost(c->h_status);
    delete c;
}

int ecq_set_error_mode(ecq_ctx* c, int mode) {
    if (!c || (mode != 0 && mode != 1)) return ECQ_ERR_ARG;
    c->P.mode = mode;
    return ECQ_OK;
}

int ecq_set_decode_plan(ecq_ctx* c, int kernel, uint32_t max_ctas) {
    if (!c || kernel < ECQ_DECODE_AUTO || kernel > ECQ_DECODE_RING) return ECQ_ERR_ARG;
    c->decode_kernel = kernel;
    c->decode_max_ctas = max_ctas;
    return ECQ_OK;
}

int ecq_set_wait_limit(ecq_ctx* c, uint32_t polls) {
    if (!c) return ECQ_ERR_ARG;
    c->wait_limit = polls;
    return ECQ_OK;
}

int ecq_set_norm(ecq_ctx* c, int norm) {
    if (!c || (norm != 0 && norm != 1)) return ECQ_ERR_ARG;
    // the any-shape path sums at most kMaxL2Runs runs of 32 entries per bucket
    if (norm == 1 && !c->tiled_ok && c->P.bucket > 32u * kMaxL2Runs) return ECQ_ERR_ARG;
    c->P.norm = norm;
    return ECQ_OK;
}

uint32_t ecq_code_bits(const ecq_ctx* c) { return c ? c->P.r : 0; }
uint64_t ecq_num_buckets(const ecq_ctx* c) { return c ? c->nb : 0; }
uint64_t ecq_codes_words(const ecq_ctx* c) { return c ? c->n_words : 0; }

int ecq_encode(ecq_ctx* c, uint32_t worker, uint32_t step, const float* grad, float* err,
               uint32_t* codes, float* scales, void* cuda_stream) {
    if (!c || !grad || !err || !codes || !scales) return ECQ_ERR_ARG;
    if (!aligned16(grad) || !aligned16(err) || !aligned16(codes) || !aligned4(scales))
        return ECQ_ERR_ARG;
    return encode_impl(c, worker, step, grad, err, codes, scales,
                       static_cast<cudaStream_t>(cuda_stream));
}

int ecq_encode_batch(ecq_ctx* c, uint32_t W, uint32_t step, const float* const* grads,
                     float* const* errs, uint32_t* const* codes, float* const* scales,
                     void* cuda_stream) {
    if (!c || !grads || !errs || !codes || !scales || W == 0 || W > ECQ_MAX_WORKERS_TOTAL)
        return ECQ_ERR_ARG;
    for (uint32_t w = 0; w < W; ++w) {
        if (!grads[w] || !errs[w] || !codes[w] || !scales[w]) return ECQ_ERR_ARG;
        if (!aligned16(grads[w]) || !aligned16(errs[w]) || !aligned16(codes[w]) || !aligned4(scales[w]))
            return ECQ_ERR_ARG;
    }
    // one launch per ECQ_MAX_WORKERS workers
    for (uint32_t w0 = 0; w0 < W; w0 += ECQ_MAX_WORKERS) {
        const uint32_t n = std::min<uint32_t>(ECQ_MAX_WORKERS, W - w0);
        WorkerBuffers wb[ECQ_MAX_WORKERS];
        for (uint32_t k = 0; k < n; ++k)
            wb[k] = {grads[w0 + k], errs[w0 + k], codes[w0 + k], scales[w0 + k]};
        const int rc = encode_batch_impl(c, w0, n, step, wb, static_cast<cudaStream_t>(cuda_stream));
        if (rc != ECQ_OK) return rc;
    }
    return ECQ_OK;
}

int ecq_decode_mean(ecq_ctx* c, uint32_t W, const uint32_t* const* codes,
                    const float* const* scales, float* out, void* cuda_stream) {
    if (!c || !codes || !scales || !out || W == 0 || W > ECQ_MAX_WORKERS_TOTAL) return ECQ_ERR_ARG;
    if (!aligned16(out)) return ECQ_ERR_ARG;
    return decode_impl(c, W, codes, scales, out, nullptr, 0.f, static_cast<cudaStream_t>(cuda_stream));
}

int ecq_decode_mean_update(ecq_ctx* c, uint32_t W, const uint32_t* const* codes,
                           const float* const* scales, float eta, float* params, float* out,
                           void* cuda_stream) {
    if (!c || !codes || !scales || !params || W == 0 || W > ECQ_MAX_WORKERS_TOTAL) return ECQ_ERR_ARG;
    if (!aligned16(params) || (out && !aligned16(out)) || !(eta == eta) || params == out)
        return ECQ_ERR_ARG;
    return decode_impl(c, W, codes, scales, out, params, -eta, static_cast<cudaStream_t>(cuda_stream));
}

int ecq_code_histogram(ecq_ctx* c, const uint32_t* codes, uint64_t* counts, void* cuda_stream) {
    if (!c || !codes || !counts || !aligned16(codes) ||
        (reinterpret_cast<uintptr_t>(counts) & 7u))
        return ECQ_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const uint32_t nbins = 2 * c->P.s + 1;
    if (cudaMemsetAsync(counts, 0, sizeof(uint64_t) * nbins, st) != cudaSuccess) return ECQ_ERR_CUDA;
    const size_t smem = nbins <= kHistLaneBins ? (size_t)(kHistThreads / 32) * nbins * 32 * 4
                      : nbins <= kHistSharedBins ? (size_t)nbins * 4 : 0;
    const uint64_t rows = (c->P.d + 31) / 32;
    uint64_t blocks = (rows + kHistThreads - 1) / kHistThreads;
    const uint64_t cap = (uint64_t)c->sm_count * 8;
    if (blocks > cap) blocks = cap;
    code_histogram_kernel<<<(uint32_t)blocks, kHistThreads, smem, st>>>(
        c->P, codes, reinterpret_cast<unsigned long long*>(counts));
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? ECQ_OK : ECQ_ERR_CUDA;
}

double ecq_entropy_bound_bits(const uint64_t* counts_host, uint32_t n_bins) {
    if (!counts_host) return 0.0;
    long double total = 0.0L;
    for (uint32_t k = 0; k < n_bins; ++k) total += (long double)counts_host[k];
    double bits = 0.0;
    for (uint32_t k = 0; k < n_bins; ++k)
        if (counts_host[k])
            bits += (double)counts_host[k] * std::log2((double)total / (double)counts_host[k]);
    return bits;
}

// ---- entropy-coded message ---------------------------------------------------------------
// Length-limited Huffman lengths by package-merge, kept as sorted weight lists: level L
// (the deepest) holds the leaves; the list of a level is the merge of the leaves with the
// pairs of the level below.  Only how many of a list's first k entries are leaves is
// needed to read the lengths off: the k_1 = 2n - 2 cheapest entries of the top list
// contain a_1 leaves and k_1 - a_1 packages, which are the first 2 (k_1 - a_1) entries of
// the next list, and so on; the i-th lightest symbol gets one bit per level with a_j > i.
int ecq_huffman_lengths(const ecq_ctx* c, const uint64_t* counts_host, uint8_t* lengths_host) {
    if (!c || !counts_host || !lengths_host) return ECQ_ERR_ARG;
    const uint32_t n_sym = 2 * c->P.s + 1;
    if (n_sym > kHuffMaxSymbols) return ECQ_ERR_ARG;
    std::vector<std::pair<uint64_t, uint32_t>> leaf;          // (count, symbol), ascending
    for (uint32_t k = 0; k < n_sym; ++k) {
        lengths_host[k] = 0;
        if (counts_host[k]) leaf.emplace_back(counts_host[k], k);
    }
    const size_t n = leaf.size();
    if (n == 0) return ECQ_OK;
    if (n == 1) { lengths_host[leaf[0].second] = 1; return ECQ_OK; }
    std::sort(leaf.begin(), leaf.end());
    struct Level { std::vector<uint64_t> weight; std::vector<uint8_t> is_leaf; };
    std::vector<Level> level(kHuffMaxLen);                   // [0] top ... [L-1] deepest
    Level& deepest = level[kHuffMaxLen - 1];
    for (size_t i = 0; i < n; ++i) { deepest.weight.push_back(leaf[i].first); deepest.is_leaf.push_back(1); }
    for (int j = (int)kHuffMaxLen - 2; j >= 0; --j) {
        const Level& below = level[j + 1];
        Level& here = level[j];
        size_t a = 0, b = 0;
        const size_t n_pairs = below.weight.size() / 2;
        while (a < n || b < n_pairs) {
            const uint64_t pw = b < n_pairs ? below.weight[2 * b] + below.weight[2 * b + 1] : 0;
            if (b == n_pairs || (a < n && leaf[a].first <= pw)) {
                here.weight.push_back(leaf[a].first); here.is_leaf.push_back(1); ++a;
            } else {
                here.weight.push_back(pw); here.is_leaf.push_back(0); ++b;
            }
        }
    }
    size_t take = 2 * n - 2;
    for (uint32_t j = 0; j < kHuffMaxLen && take > 0; ++j) {
        size_t leaves = 0;
        for (size_t i = 0; i < take; ++i) leaves += level[j].is_leaf[i];
        for (size_t i = 0; i < leaves; ++i) lengths_host[leaf[i].second] += 1;
        take = 2 * (take - leaves);
    }
    return ECQ_OK;
}

uint64_t ecq_huffman_chunks(const ecq_ctx* c) {
    return c ? (c->P.d + kHuffChunk - 1) / kHuffChunk : 0;
}

uint64_t ecq_huffman_stream_bound(const ecq_ctx* c, const uint64_t* counts_host,
                                  const uint8_t* lengths_host) {
    if (!c || !counts_host || !lengths_host) return 0;
    const uint32_t n_sym = 2 * c->P.s + 1;
    uint64_t bits = 0;
    for (uint32_t k = 0; k < n_sym; ++k) bits += counts_host[k] * lengths_host[k];
    return (bits + 31) / 32 + ecq_huffman_chunks(c);
}

int ecq_huffman_tables(ecq_ctx* c, const uint8_t* lengths_host, void* tables_dev, void* cuda_stream) {
    if (!c || !lengths_host || !tables_dev || !aligned16(tables_dev)) return ECQ_ERR_ARG;
    const uint32_t n_sym = 2 * c->P.s + 1;
    if (n_sym > kHuffMaxSymbols) return ECQ_ERR_ARG;
    // canonical words: within a length in symbol order, the first word of a length is the
    // first unused word of the previous length with a zero appended
    uint32_t per_len[kHuffMaxLen + 2] = {0}, first[kHuffMaxLen + 2] = {0};
    uint64_t kraft = 0;
    for (uint32_t k = 0; k < n_sym; ++k) {
        if (lengths_host[k] > kHuffMaxLen) return ECQ_ERR_ARG;
        if (lengths_host[k]) { per_len[lengths_host[k]] += 1; kraft += 1ull << (kHuffMaxLen - lengths_host[k]); }
    }
    if (kraft > (1ull << kHuffMaxLen)) return ECQ_ERR_ARG;
    for (uint32_t L = 1; L <= kHuffMaxLen; ++L) first[L] = (first[L - 1] + per_len[L - 1]) << 1;
    HuffTables* t = new (std::nothrow) HuffTables;
    if (!t) return ECQ_ERR_ALLOC;
    std::memset(t, 0, sizeof(*t));
    // one word per 12-bit pattern first: symbol << 4 | length
    std::vector<uint16_t> single(1u << kHuffMaxLen, 0);
    for (uint32_t k = 0; k < n_sym; ++k) {
        const uint32_t L = lengths_host[k];
        if (!L) continue;
        const uint32_t word = first[L]++;
        uint32_t rev = 0;                                    // first bit sent -> bit 0
        for (uint32_t b = 0; b < L; ++b) rev |= ((word >> (L - 1 - b)) & 1u) << b;
        t->enc[k] = (L << 16) | rev;
        for (uint32_t hi = 0; hi < (1u << (kHuffMaxLen - L)); ++hi)
            single[(hi << L) | rev] = (uint16_t)((k << 4) | L);
    }
    // the sender's look-ups take k codes at a time: k*r index bits <= 12, k words <= 24 bits
    const uint32_t r = c->P.r;
    uint32_t longest = 1, group = r <= 3 ? 4u : (r <= 6 ? 2u : 1u);
    for (uint32_t k = 0; k < n_sym; ++k) longest = std::max<uint32_t>(longest, lengths_host[k]);
    while (group > 1 && group * longest > 24) group /= 2;
    t->group_syms = group;
    // then all the words that lie wholly inside the pattern
    const uint32_t most = std::min<uint32_t>(kHuffDecMaxSyms, 16 / r);
    for (uint32_t p = 0; p < (1u << kHuffMaxLen); ++p) {
        uint32_t pos = 0, n = 0, syms = 0, first_len = 0;
        while (n < most) {
            const uint16_t e = single[p >> pos];             // the missing high bits read as 0
            const uint32_t L = e & 15u;
            if (L == 0 || pos + L > kHuffMaxLen) break;
            syms |= (uint32_t)(e >> 4) << (n * r);
            if (n == 0) first_len = L;
            pos += L; ++n;
        }
        t->dec[p] = syms | (n << 16) | (pos << 20) | (first_len << 24);
    }
    // pageable source: the copy is staged before the call returns, so `t` can go
    const cudaError_t e = cudaMemcpyAsync(tables_dev, t, sizeof(*t), cudaMemcpyHostToDevice,
                                          static_cast<cudaStream_t>(cuda_stream));
    delete t;
    return e == cudaSuccess ? ECQ_OK : ECQ_ERR_CUDA;
}

int ecq_huffman_encode(ecq_ctx* c, const void* tables_dev, const uint32_t* codes,
                       uint32_t* stream_words, uint64_t capacity_words, uint32_t* offsets,
                       uint16_t* quarters, void* cuda_stream) {
    if (!c || !tables_dev || !codes || !stream_words || !offsets || !quarters ||
        !aligned16(tables_dev) || !aligned16(codes) || !aligned4(stream_words) ||
        !aligned4(offsets) || (reinterpret_cast<uintptr_t>(quarters) & 1u))
        return ECQ_ERR_ARG;
    const uint32_t n_sym = 2 * c->P.s + 1;
    if (n_sym > kHuffMaxSymbols) return ECQ_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const HuffTables* t = static_cast<const HuffTables*>(tables_dev);
    const uint64_t n_chunks = ecq_huffman_chunks(c);
    // contiguous segments of chunks, one per CTA, at least one chunk per warp
    uint64_t blocks = (n_chunks + kHuffWarps - 1) / kHuffWarps;
    const uint64_t cap = (uint64_t)c->sm_count * 8;
    if (blocks > cap) blocks = cap;
    const uint64_t seg = (n_chunks + blocks - 1) / blocks;
    const uint32_t n_seg = (uint32_t)((n_chunks + seg - 1) / seg);
    // shared memory for the largest group table this code width can have
    const uint32_t r = c->P.r, k_most = r <= 3 ? 4u : (r <= 6 ? 2u : 1u);
    const size_t smem_group = (size_t)4 << (k_most * r);
    const size_t smem_write = smem_group +
        (size_t)kHuffWarps * (kHuffChunkWords + 32 + 32 * kHuffRowWords) * 4;
    huff_count_kernel<<<n_seg, kHuffWarps * 32, smem_group, st>>>(
        c->P, t, codes, offsets, c->d_status, n_chunks, seg);
    huff_scan_kernel<<<1, kScanThreads, 0, st>>>(offsets, n_chunks, seg, capacity_words, c->d_status);
    huff_write_kernel<<<n_seg, kHuffWarps * 32, smem_write, st>>>(
        c->P, t, codes, offsets, quarters, stream_words, n_chunks, seg);
    g_launches.fetch_add(3, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? ECQ_OK : ECQ_ERR_CUDA;
}

int ecq_huffman_decode(ecq_ctx* c, const void* tables_dev, const uint32_t* stream_words,
                       uint64_t stream_len_words, const uint32_t* offsets,
                       const uint16_t* quarters, uint32_t* codes, void* cuda_stream) {
    if (!c || !tables_dev || !stream_words || !offsets || !quarters || !codes ||
        !aligned16(tables_dev) || !aligned16(stream_words) || !aligned4(offsets) ||
        (reinterpret_cast<uintptr_t>(quarters) & 1u) || !aligned16(codes))
        return ECQ_ERR_ARG;
    const uint32_t n_sym = 2 * c->P.s + 1;
    if (n_sym > kHuffMaxSymbols) return ECQ_ERR_ARG;
    const uint64_t n_chunks = ecq_huffman_chunks(c);
    uint64_t blocks = (4 * n_chunks + kHuffDecThreads - 1) / kHuffDecThreads;
    const uint64_t cap = (uint64_t)c->sm_count * 16;
    if (blocks > cap) blocks = cap;
    huff_decode_kernel<<<(uint32_t)blocks, kHuffDecThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        c->P, static_cast<const HuffTables*>(tables_dev), stream_words, offsets, quarters, codes, c->d_status,
        n_chunks, c->n_words, stream_len_words);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? ECQ_OK : ECQ_ERR_CUDA;
}

uint64_t ecq_step_host_workspace_bytes(const ecq_ctx* c, uint32_t W) {
    if (!c || W == 0 || W > ECQ_MAX_WORKERS) return 0;
    const uint64_t stage = round_up(c->P.d * 4, 256);
    const uint64_t codes = round_up(c->n_words * 4, 256);
    const uint64_t scales = round_up(c->nb * 4, 256);
    return 2 * stage + W * (codes + scales) + stage;
}

int ecq_step_host(ecq_ctx* c, uint32_t W, uint32_t step, const float* const* grads_host,
                  float* err_dev, void* workspace_dev, uint64_t workspace_bytes, float* out_host,
                  void* cuda_stream) {
    if (!c || !grads_host || !err_dev || !workspace_dev || !out_host || W == 0 ||
        W > ECQ_MAX_WORKERS)
        return ECQ_ERR_ARG;
    if (workspace_bytes < ecq_step_host_workspace_bytes(c, W) ||
        (reinterpret_cast<uintptr_t>(workspace_dev) & 255u) || !aligned16(err_dev) ||
        (c->P.d % 4 != 0 && W > 1))     // worker-major accumulators must stay 16-byte aligned
        return ECQ_ERR_ARG;
    for (uint32_t w = 0; w < W; ++w)
        if (!grads_host[w]) return ECQ_ERR_ARG;
    std::lock_guard<std::mutex> lock(c->host_mu);
    if (!c->host_ready) {
        if (cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking) != cudaSuccess)
            return ECQ_ERR_CUDA;
        for (int i = 0; i < 2; ++i) {
            cudaEventCreateWithFlags(&c->ev_copied[i], cudaEventDisableTiming);
            cudaEventCreateWithFlags(&c->ev_encoded[i], cudaEventDisableTiming);
        }
        cudaEventCreateWithFlags(&c->ev_start, cudaEventDisableTiming);
        c->host_ready = true;
    }
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const uint64_t d = c->P.d;
    const uint64_t stage_b = round_up(d * 4, 256);
    const uint64_t codes_b = round_up(c->n_words * 4, 256);
    const uint64_t scales_b = round_up(c->nb * 4, 256);
    uint8_t* ws = static_cast<uint8_t*>(workspace_dev);
    float* stage[2] = {reinterpret_cast<float*>(ws), reinterpret_cast<float*>(ws + stage_b)};
    uint8_t* msg = ws + 2 * stage_b;
    float* out_dev = reinterpret_cast<float*>(msg + W * (codes_b + scales_b));

    MessageTable tab;
    std::memset(&tab, 0, sizeof(tab));
    // the copy stream must not run ahead of work already queued on the caller's stream
    cudaEventRecord(c->ev_start, st);
    cudaStreamWaitEvent(c->copy_stream, c->ev_start, 0);
    int rc = ECQ_OK;
    for (uint32_t w = 0; w < W && rc == ECQ_OK; ++w) {
        const int sl = w & 1;
        if (w >= 2) cudaStreamWaitEvent(c->copy_stream, c->ev_encoded[sl], 0);
        cudaMemcpyAsync(stage[sl], grads_host[w], d * 4, cudaMemcpyHostToDevice, c->copy_stream);
        cudaEventRecord(c->ev_copied[sl], c->copy_stream);
        cudaStreamWaitEvent(st, c->ev_copied[sl], 0);
        uint32_t* codes = reinterpret_cast<uint32_t*>(msg + w * (codes_b + scales_b));
        float* scales = reinterpret_cast<float*>(msg + w * (codes_b + scales_b) + codes_b);
        tab.codes[w] = codes;
        tab.scales[w] = scales;
        rc = encode_impl(c, w, step, stage[sl], err_dev + (uint64_t)w * d, codes, scales, st);
        cudaEventRecord(c->ev_encoded[sl], st);
    }
    if (rc == ECQ_OK) rc = decode_launch(c, W, W, tab, DecodeOut{out_dev, nullptr, 0.f}, true, true, st);
    if (rc == ECQ_OK &&
        cudaMemcpyAsync(out_host, out_dev, d * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        rc = ECQ_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) rc = ECQ_ERR_CUDA;
    cudaStreamSynchronize(c->copy_stream);
    return rc;
}

int ecq_status(ecq_ctx* c, void* cuda_stream) {
    if (!c) return ECQ_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemcpyAsync(c->h_status, c->d_status, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaMemsetAsync(c->d_status, 0, 4, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return ECQ_ERR_CUDA;
    const uint32_t bits = *c->h_status;
    if (bits & kStatusTimeout) return ECQ_ERR_TIMEOUT;
    if (bits & kStatusNonFinite) return ECQ_ERR_NONFINITE;
    if (bits & kStatusCapacity) return ECQ_ERR_CAPACITY;
    if (bits & kStatusSymbol) return ECQ_ERR_SYMBOL;
    return ECQ_OK;
}

uint64_t ecq_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* ecq_strerror(int status) {
    switch (status) {
        case ECQ_OK: return "ok";
        case ECQ_ERR_ARG: return "invalid argument (null or misaligned pointer, size or range)";
        case ECQ_ERR_CUDA: return "a CUDA call failed";
        case ECQ_ERR_NONFINITE: return "NaN or Inf in a compensated gradient";
        case ECQ_ERR_TIMEOUT: return "an in-kernel wait on an asynchronous copy ran out";
        case ECQ_ERR_ALLOC: return "allocation failed";
        case ECQ_ERR_TOO_LARGE: return "problem too large for the built-in scratch of ecq_step_static";
        case ECQ_ERR_CAPACITY: return "the entropy-coded stream does not fit the given buffer";
        case ECQ_ERR_SYMBOL: return "a level without a code word, or a bit pattern that is no code word";
        default: return "unknown status";
    }
}

}  // extern "C"

// ===========================================================================
// ecq_step_static: the whole iteration without any allocation.  The W messages
// and the status word live in an array compiled into the library.  In host code
// the array's name is only a stand-in; its device address is looked up once per
// device and that pointer is what the kernels get.
// ===========================================================================
static __device__ __align__(256) unsigned char g_static_scratch[ECQ_STATIC_SCRATCH_BYTES];

namespace {

struct StaticScratch {
    std::once_flag once;
    unsigned char* ptr = nullptr;
    cudaError_t err = cudaErrorUnknown;
};
StaticScratch g_static[kMaxDevices];

// Device address of the built-in scratch on the current device (set-up on first use).
unsigned char* static_scratch_ptr(int device) {
    StaticScratch& s = g_static[device];                  // < kMaxDevices: checked by the caller
    std::call_once(s.once, [&] {
        void* p = nullptr;
        s.err = cudaGetSymbolAddress(&p, g_static_scratch);
        if (s.err == cudaSuccess) s.ptr = static_cast<unsigned char*>(p);
    });
    return s.err == cudaSuccess ? s.ptr : nullptr;
}

}  // namespace

extern "C" int ecq_step_static(uint64_t d, uint32_t bucket, uint32_t levels, float alpha,
                               float beta, uint64_t seed, uint32_t W, uint32_t step,
                               const float* const* grads, float* err, float* out,
                               void* cuda_stream) {
    if (!grads || !err || !out || W == 0 || W > ECQ_MAX_WORKERS) return ECQ_ERR_ARG;
    if (d == 0 || bucket < 32 || bucket % 32 != 0 || levels == 0 || levels > 32767)
        return ECQ_ERR_ARG;
    if (!(alpha >= 0.f) || !(beta >= 0.f) || !(beta <= 1.f) || !(alpha < INFINITY))
        return ECQ_ERR_ARG;
    if (!aligned16(err) || !aligned16(out) || (d % 4 != 0 && W > 1)) return ECQ_ERR_ARG;
    for (uint32_t w = 0; w < W; ++w)
        if (!grads[w] || !aligned16(grads[w])) return ECQ_ERR_ARG;

    // a context on the stack: constants only, nothing allocated
    ecq_ctx c;
    CodecParams& P = c.P;
    P.d = d; P.bucket = bucket; P.s = levels; P.mode = 0; P.norm = 0;
    P.alpha = alpha; P.beta = beta; P.sf = (float)levels;
    P.r = 0;
    while ((1ull << P.r) < 2ull * levels + 1ull) ++P.r;
    uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
    for (int i = 0; i < 10; ++i) {
        P.key0[i] = k0; P.key1[i] = k1;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    c.nb = (d + bucket - 1) / bucket;
    c.n_words = (d * P.r + 31) / 32;
    c.tiled_ok = (bucket & (bucket - 1)) == 0 && bucket <= kMaxTiledBucket;
    c.decode_kernel = ECQ_DECODE_AUTO;
    c.decode_max_ctas = 0;
    c.wait_limit = kWaitLimit;
    c.host_ready = false;
    c.h_status = nullptr;

    const uint64_t codes_b = round_up(c.n_words * 4, 256);
    const uint64_t scales_b = round_up(c.nb * 4, 256);
    const uint64_t need = 256 + (uint64_t)W * (codes_b + scales_b);
    if (need > ECQ_STATIC_SCRATCH_BYTES) return ECQ_ERR_TOO_LARGE;

    if (cudaGetDevice(&c.device) != cudaSuccess || c.device < 0 || c.device >= kMaxDevices ||
        cudaDeviceGetAttribute(&c.sm_count, cudaDevAttrMultiProcessorCount, c.device) != cudaSuccess)
        return ECQ_ERR_CUDA;
    unsigned char* scratch = static_scratch_ptr(c.device);
    if (!scratch) return ECQ_ERR_CUDA;
    c.d_status = reinterpret_cast<uint32_t*>(scratch);

    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // the array keeps the previous call's contents: the status word must start at zero
    if (cudaMemsetAsync(c.d_status, 0, sizeof(uint32_t), st) != cudaSuccess) return ECQ_ERR_CUDA;
    MessageTable tab;
    std::memset(&tab, 0, sizeof(tab));
    int rc = ECQ_OK;
    for (uint32_t w = 0; w < W && rc == ECQ_OK; ++w) {
        unsigned char* msg = scratch + 256 + w * (codes_b + scales_b);
        uint32_t* codes = reinterpret_cast<uint32_t*>(msg);
        float* scales = reinterpret_cast<float*>(msg + codes_b);
        tab.codes[w] = codes;
        tab.scales[w] = scales;
        rc = encode_impl(&c, w, step, grads[w], err + (uint64_t)w * d, codes, scales, st);
    }
    if (rc == ECQ_OK) rc = decode_launch(&c, W, W, tab, DecodeOut{out, nullptr, 0.f}, true, true, st);
    uint32_t bits = 0;
    if (cudaMemcpyAsync(&bits, c.d_status, sizeof(bits), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return ECQ_ERR_CUDA;
    if (rc != ECQ_OK) return rc;
    if (bits & kStatusTimeout) return ECQ_ERR_TIMEOUT;
    if (bits & kStatusNonFinite) return ECQ_ERR_NONFINITE;
    if (bits & kStatusCapacity) return ECQ_ERR_CAPACITY;
    if (bits & kStatusSymbol) return ECQ_ERR_SYMBOL;
    return ECQ_OK;
}
