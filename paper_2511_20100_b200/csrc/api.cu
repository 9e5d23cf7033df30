// libmtmcfused: the C-ABI boundary (see include/mtmc_fused.h).  Host side only:
// argument validation, per-device state, TMA descriptor encoding, kernel selection
// by shape and launches.  All arithmetic is in the kernels.
#include "../../include/mtmc_fused.h"

#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "gemm_pair.cuh"
#include "gemm_ksplit.cuh"
#include "gemm_big.cuh"
#include "skinny.cuh"
#include "gemm_mx.cuh"
#include "gemm_mx_pair.cuh"

namespace {

using namespace mtmc;

constexpr int MAX_DEVICES = 64;
constexpr size_t TICKET_BYTES = 64 * 1024;   // library-owned split-K tickets: 16384 tiles
constexpr int SK_MAX_PAIRS = 256;            // stream-K boundaries (pairs of one launch) the flag array covers
constexpr size_t SK_FLAG_BYTES = 2 * SK_MAX_PAIRS * 8 * sizeof(uint32_t);    // one ticket word per (region tile, epilogue warp): fewer than two tiles per pair
constexpr size_t SK_PART_BYTES = 2 * 2 * 4 * 8 * 8 * 32 * sizeof(float4);   // per pair: 2 parts x 2 ranks x 4 quadrants x 32 KiB
#ifndef MTMC_SKINNY_MAX_M
#define MTMC_SKINNY_MAX_M 64
#endif
constexpr int SKINNY_MAX_M = MTMC_SKINNY_MAX_M;   // rows of X the weight-streaming path takes (MMA N = 16, 32 or 64)

struct DeviceState {
    bool ready = false;
    int sm_count = 0;
    uint32_t* status = nullptr;      // device status word (256 bytes reserved)
    // Library-owned scratch is kept per stream, so that calls enqueued on different streams (by one host thread
    // or by several) never share partials or tickets: a slot belongs to the first stream that asked for it.
    struct StreamScratch {
        bool used = false;
        cudaStream_t stream = nullptr;
        uint32_t* tickets = nullptr;     // split-K tickets of the weight-streaming kernel (TICKET_BYTES, allocated on first need)
        void* ws = nullptr;              // workspace (grow-only)
        size_t ws_bytes = 0;
        cudaEvent_t ev0 = nullptr, ev1 = nullptr;    // mtmc_set_timing: around the kernels of the last call on this stream
        bool timed = false;
        uint32_t* sk_flags = nullptr;    // stream-K flag words (SK_FLAG_BYTES, zeroed once: launches tell themselves apart by epoch)
        uint32_t sk_epoch = 0;
    };
    static constexpr int MAX_STREAMS = 32;
    StreamScratch sscratch[MAX_STREAMS];
    // The *_host entry points: a ring of slots, each with device copies of one call's operands and result and
    // the events that order its three phases (copy in, kernels, copy out) across three streams.
    struct HostSlot {
        void* buf[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
        size_t bytes[5] = {0, 0, 0, 0, 0};
        cudaEvent_t in_done = nullptr, k_done = nullptr, out_done = nullptr;
        bool busy = false;
    };
    static constexpr int HOST_SLOTS = 6;
    HostSlot hslot[HOST_SLOTS];
    int hnext = 0;
    size_t hwm[5] = {0, 0, 0, 0, 0};
    cudaStream_t s_in = nullptr, s_out = nullptr;
    int max_pairs = -1;              // co-resident 2-CTA clusters of the skinny kernel (-1: not queried yet)
    int max_gemm_pairs = -1;         // the same for the CTA-pair tiled kernel
    int max_ksplit[6] = {-1, -1, -1, -1, -1, -1};   // co-resident clusters of two / four / eight CTAs of the cluster split-K kernel (256-, then 128-column tiles)
};

std::mutex g_mutex;
DeviceState g_dev[MAX_DEVICES];
std::atomic<long long> g_launches{0};
std::atomic<long long> g_device_allocs{0};     // cudaMalloc calls made by this library (mtmc_device_alloc_count)

// Every device allocation of the library goes through here, so that the count is complete.
cudaError_t counted_malloc(void** ptr, size_t bytes) {
    g_device_allocs.fetch_add(1);
    return cudaMalloc(ptr, bytes);
}

// Status word of the allocation-free entry point on the current device (defined with that entry point, at the
// end of this file): fetches and clears it if that path has been set up on this device; *st = 0 otherwise.
int noalloc_take_status(int dev, uint32_t* st);
bool noalloc_in_use(int dev);

thread_local cudaStream_t t_stream = nullptr;
thread_local void* t_user_ws = nullptr;
thread_local size_t t_user_ws_bytes = 0;
thread_local int t_split_k = 0;
thread_local int t_tile_n = 0;
thread_local int t_cta_pair = 0;   // 0 automatic, 1 force CTA pairs, -1 force single CTAs
thread_local int t_stream_k = 0;   // 0 automatic, 1 stream-K wherever it is legal, -1 never (mtmc_set_schedule)
thread_local int t_static_weights = 0;   // caller's promise that no work in flight writes W (see mtmc_set_static_weights)
thread_local int t_timing = 0;
thread_local unsigned long long* t_trace = nullptr;   // caller's trace buffer (mtmc_set_trace), used by -DMTMC_TRACE builds
thread_local size_t t_trace_bytes = 0;
thread_local char t_error[512] = "";
thread_local char t_last_kernel[96] = "";     // main kernel of the last call of this thread (mtmc_last_kernel_name)

void note_kernel(const char* family, int epi, int detail = 0) {
    static const char* const epi_name[] = {"EPI_ACT", "EPI_SWIGLU", "EPI_LSE", "EPI_ROWMAX", "EPI_XENT", "EPI_SOFTMAX"};
    if (epi >= 0 && detail > 0) snprintf(t_last_kernel, sizeof t_last_kernel, "%s<%s, %d>", family, epi_name[epi], detail);
    else if (epi >= 0) snprintf(t_last_kernel, sizeof t_last_kernel, "%s<%s>", family, epi_name[epi]);
    else snprintf(t_last_kernel, sizeof t_last_kernel, "%s<MX=%d>", family, detail);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

// The trace buffer for a launch of `ctas` CTAs, if the caller gave one that is large enough.
unsigned long long* trace_for(unsigned ctas) {
#ifdef MTMC_TRACE
    if (t_trace && t_trace_bytes >= static_cast<size_t>(ctas) * TRACE_WORDS * sizeof(unsigned long long)) return t_trace;
#endif
    (void)ctas;
    return nullptr;
}

int fail(int code, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(t_error, sizeof t_error, fmt, ap);
    va_end(ap);
    return code;
}

#define CUDA_TRY(expr)                                                                      \
    do {                                                                                    \
        cudaError_t e_ = (expr);                                                            \
        if (e_ != cudaSuccess) return fail(MTMC_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e_)); \
    } while (0)

int get_device(DeviceState** out, int* dev_out = nullptr) {
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= MAX_DEVICES) return fail(MTMC_ERR_UNSUPPORTED_DEVICE, "device index %d out of range", dev);
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceState& d = g_dev[dev];
    if (!d.ready) {
        int major = 0, minor = 0;
        CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
        CUDA_TRY(cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev));
        if (major != 10)
            return fail(MTMC_ERR_UNSUPPORTED_DEVICE, "compute capability %d.%d: this library only runs on 10.x (B200)", major, minor);
        CUDA_TRY(cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev));
        if (!g_encode) {
            void* fn = nullptr;
            cudaDriverEntryPointQueryResult qres;
            CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
            if (!fn || qres != cudaDriverEntryPointSuccess)
                return fail(MTMC_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
            g_encode = reinterpret_cast<EncodeTiledFn>(fn);
        }
        CUDA_TRY(counted_malloc(reinterpret_cast<void**>(&d.status), 256));
        CUDA_TRY(cudaMemset(d.status, 0, 256));
        d.ready = true;
    }
    *out = &d;
    if (dev_out) *dev_out = dev;
    return MTMC_OK;
}

// Tensor-map cache.  A CUtensorMap is a pure function of (address, element type, extents, row pitch, box): it
// holds no reference to the memory, so a cached copy is valid for as long as the key matches, whoever owns the
// buffer now.  Serving loops call with the same few (weight, activation buffer, shape) combinations over and
// over; re-encoding three to five descriptors costs more host time than launching the kernel.  Thread-local,
// direct-mapped, 128 entries.
struct TmapKey {
    const void* ptr; int64_t rows, cols, ld; int box_rows, u8;
    bool operator==(const TmapKey& o) const {
        return ptr == o.ptr && rows == o.rows && cols == o.cols && ld == o.ld && box_rows == o.box_rows && u8 == o.u8;
    }
};
struct TmapEntry { bool valid = false; TmapKey key{}; CUtensorMap map; };
constexpr int TMAP_CACHE_ENTRIES = 128;
thread_local TmapEntry t_tmap_cache[TMAP_CACHE_ENTRIES];
thread_local long long t_tmap_hits = 0, t_tmap_misses = 0;

// 2-D row-major [rows, cols] tensor of bf16 (box = 64 columns x box_rows rows) or of one-byte E4M3 elements
// (box = 128 columns x box_rows rows): one 128-byte swizzle row of K per box row either way.
int encode_2d(CUtensorMap* map, const void* ptr, int64_t rows, int64_t cols, int box_rows, int64_t ld, bool u8) {
    const TmapKey key{ptr, rows, cols, ld > 0 ? ld : cols, box_rows, u8 ? 1 : 0};      // (kind 2: the plain byte maps of encode_bytes_2d)
    uint64_t h = reinterpret_cast<uintptr_t>(ptr) >> 4;
    h = (h ^ static_cast<uint64_t>(rows) * 0x9E3779B97F4A7C15ull ^ static_cast<uint64_t>(key.ld) * 0xC2B2AE3D27D4EB4Full ^
         static_cast<uint64_t>(cols) * 0x165667B19E3779F9ull ^ static_cast<uint64_t>(box_rows * 2 + key.u8)) * 0xD6E8FEB86659FD93ull;
    TmapEntry& e = t_tmap_cache[(h >> 32) % TMAP_CACHE_ENTRIES];
    if (e.valid && e.key == key) { *map = e.map; ++t_tmap_hits; return MTMC_OK; }
    ++t_tmap_misses;
    const size_t esz = u8 ? 1 : 2;
    cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
    cuuint64_t strides[1] = {static_cast<cuuint64_t>(key.ld) * esz};      // row pitch in bytes
    cuuint32_t box[2] = {u8 ? 128u : 64u, static_cast<cuuint32_t>(box_rows)};
    cuuint32_t estr[2] = {1u, 1u};
    CUresult r = g_encode(map, u8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims,
                          strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(MTMC_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d", static_cast<int>(r));
    e.valid = true; e.key = key; e.map = *map;
    return MTMC_OK;
}
// Plain (unswizzled) byte tensor of 256-byte rows, box = 256 bytes x box_rows: the re-arranged MXFP8 scale blocks.
int encode_bytes_2d(CUtensorMap* map, const void* ptr, int64_t rows, int box_rows) {
    cuuint64_t dims[2] = {256u, static_cast<cuuint64_t>(rows)};
    cuuint64_t strides[1] = {256u};
    cuuint32_t box[2] = {256u, static_cast<cuuint32_t>(box_rows)};
    cuuint32_t estr[2] = {1u, 1u};
    CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(MTMC_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d", static_cast<int>(r));
    return MTMC_OK;
}
int encode_bf16_2d(CUtensorMap* map, const void* ptr, int64_t rows, int64_t cols, int box_rows, int64_t ld = 0) {
    return encode_2d(map, ptr, rows, cols, box_rows, ld, false);
}
int encode_u8_2d(CUtensorMap* map, const void* ptr, int64_t rows, int64_t cols, int box_rows, int64_t ld = 0) {
    return encode_2d(map, ptr, rows, cols, box_rows, ld, true);
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_common(const void* X, const void* W, const void* out, int64_t M, int64_t N, int64_t K) {
    if (!X || !W || !out) return fail(MTMC_ERR_INVALID_ARG, "null pointer argument");
    if (M <= 0 || N <= 0 || K <= 0) return fail(MTMC_ERR_INVALID_ARG, "M, N, K must be positive (got %lld, %lld, %lld)",
                                                 (long long)M, (long long)N, (long long)K);
    if (M >= (1ll << 31) || N >= (1ll << 31) || K >= (1ll << 31))
        return fail(MTMC_ERR_UNSUPPORTED_SHAPE, "dimensions must be below 2^31");
    if (K % 8 != 0) return fail(MTMC_ERR_UNSUPPORTED_SHAPE, "K = %lld: K must be a multiple of 8 (16-byte rows for TMA)", (long long)K);
    if (!aligned16(X) || !aligned16(W) || !aligned16(out)) return fail(MTMC_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
    return MTMC_OK;
}

// The scratch slot of the current stream on this device (created on first use).
int get_stream_scratch(DeviceState* d, DeviceState::StreamScratch** out) {
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceState::StreamScratch* free_slot = nullptr;
    for (auto& s : d->sscratch) {
        if (s.used && s.stream == t_stream) { *out = &s; return MTMC_OK; }
        if (!s.used && !free_slot) free_slot = &s;
    }
    if (!free_slot)
        return fail(MTMC_ERR_WORKSPACE, "more than %d streams use library-owned scratch on this device; give the further "
                    "ones their own with mtmc_set_workspace", DeviceState::MAX_STREAMS);
    free_slot->used = true;
    free_slot->stream = t_stream;
    *out = free_slot;
    return MTMC_OK;
}

// Scratch for this call: the caller's if set, else the library's slot for the current stream (grown on demand).
int get_workspace(DeviceState* d, size_t need, void** out) {
    if (need == 0) { *out = nullptr; return MTMC_OK; }
    if (t_user_ws) {
        if (t_user_ws_bytes < need)
            return fail(MTMC_ERR_WORKSPACE, "workspace of %zu bytes given, %zu needed", t_user_ws_bytes, need);
        *out = t_user_ws;
        return MTMC_OK;
    }
    DeviceState::StreamScratch* sc = nullptr;
    if (int rc = get_stream_scratch(d, &sc)) return rc;
    if (sc->ws_bytes < need) {
        // only work on this stream can still be using the old buffer
        if (sc->ws) { CUDA_TRY(cudaStreamSynchronize(t_stream)); CUDA_TRY(cudaFree(sc->ws)); sc->ws = nullptr; sc->ws_bytes = 0; }
        size_t bytes = (need + (1u << 20) - 1) & ~static_cast<size_t>((1u << 20) - 1);
        CUDA_TRY(counted_malloc(&sc->ws, bytes));
        sc->ws_bytes = bytes;
    }
    *out = sc->ws;
    return MTMC_OK;
}

size_t round256(size_t v) { return (v + 255) & ~static_cast<size_t>(255); }

// Scratch of the row reductions: one (max, sum-exp) pair per row and column piece (per epilogue warp share).
// A launch needs n_tiles * tail_split pieces for the plan it picks (lse_partial_bytes); the figure that
// mtmc_workspace_bytes reports covers every plan the library can pick for the shape: 128-column tiles with the
// wave tail cut in four, or 256-column tiles owned by clusters of eight CTAs (eight pieces per tile, also for a
// last tile that lies partly past N).
size_t lse_partial_bytes(const GemmParams& p) {
    return round256(static_cast<size_t>(p.n_tiles) * p.tail_split * EPI_HALVES * static_cast<size_t>(p.M) * sizeof(float2));
}
size_t lse_workspace_bytes(int64_t M, int64_t N) {
    const size_t pieces = std::max(static_cast<size_t>((N + 127) / 128) * 4, static_cast<size_t>((N + 255) / 256) * 8);
    return round256(pieces * EPI_HALVES * static_cast<size_t>(M) * sizeof(float2));
}

int pick_tile_n(int64_t N) {
    if (t_tile_n == 128 || t_tile_n == 256) return t_tile_n;
    return N > 128 ? 256 : 128;
}

int pick_group_m(int m_tiles) { return m_tiles < 16 ? m_tiles : 16; }

struct TimedRegion {
    DeviceState::StreamScratch* sc = nullptr;
    TimedRegion(DeviceState* dev) {
        if (t_timing == 0 || get_stream_scratch(dev, &sc) != MTMC_OK) { sc = nullptr; return; }
        if (!sc->ev0 && (cudaEventCreate(&sc->ev0) != cudaSuccess || cudaEventCreate(&sc->ev1) != cudaSuccess)) { sc = nullptr; return; }
        cudaEventRecord(sc->ev0, t_stream);
    }
    void stop() {
        if (sc) { cudaEventRecord(sc->ev1, t_stream); sc->timed = true; }
    }
};

// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) once per kernel and device instead of per call.
// (Instantiations of one kernel template share a function-pointer type, so the record is keyed
// on the pointer value, not on the type.)
struct SmemAttrRecord { const void* fn; int dev; };
SmemAttrRecord g_smem_attr[256];
int g_smem_attr_count = 0;

template <class Kernel>
int ensure_smem_attr(Kernel kern, int bytes) {
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    const void* key = reinterpret_cast<const void*>(kern);
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        for (int i = 0; i < g_smem_attr_count; ++i)
            if (g_smem_attr[i].fn == key && g_smem_attr[i].dev == dev) return MTMC_OK;
    }
    CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_smem_attr_count < 256) g_smem_attr[g_smem_attr_count++] = SmemAttrRecord{key, dev};
    return MTMC_OK;
}

// Programmatic dependent launch: lets this kernel's set-up overlap the tail of the kernel before
// it in the stream (the kernels block in griddepcontrol.wait before touching global memory).
int pdl_attribute(cudaLaunchAttribute* attr) {
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    return 1;
}

// A small follow-up kernel (merge, scaling pass) as a programmatic dependent of the kernel before it: its blocks are
// placed while that kernel still runs and proceed, from their griddepcontrol.wait, the moment it has completed.
template <class Kern, class... Args>
int launch_follow_up(Kern kern, dim3 grid, unsigned threads, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(threads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = t_stream;
    cudaLaunchAttribute attr[1];
    cfg.attrs = attr;
    cfg.numAttrs = pdl_attribute(attr);
    CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, args...));
    g_launches.fetch_add(1);
    return MTMC_OK;
}

template <int EPI, int BN, bool OUT_BF16>
int launch_tiled(DeviceState* d, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmB2,
                 const CUtensorMap& tmBt, const CUtensorMap& tmB2t, GemmParams p) {
    using Cfg = TileCfg<EPI, BN>;
    auto kern = gemm_tiled_kernel<EPI, BN, OUT_BF16>;
    if (int rc = ensure_smem_attr(kern, Cfg::SMEM_BYTES)) return rc;
    const int grid = p.num_items < d->sm_count ? p.num_items : d->sm_count;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid), 1, 1);
    cfg.blockDim = dim3(Cfg::THREADS, 1, 1);
    cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
    cfg.stream = t_stream;
    cudaLaunchAttribute attr[1];
    cfg.attrs = attr;
    cfg.numAttrs = pdl_attribute(attr);
    CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, tmA, tmB, tmB2, tmBt, tmB2t, p));
    g_launches.fetch_add(1);
    note_kernel("gemm_tiled_kernel", EPI, BN);
    return MTMC_OK;
}

template <int EPI, bool OUT_BF16>
int launch_pair(int clusters, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmB2,
                const CUtensorMap& tmBt, const CUtensorMap& tmB2t, const GemmParams& p) {
    using Cfg = PairCfg<EPI>;
    auto kern = gemm_pair_kernel<EPI, OUT_BF16>;
    if (int rc = ensure_smem_attr(kern, Cfg::SMEM_BYTES)) return rc;
    const int pairs = (p.sk || p.num_items >= clusters) ? clusters : p.num_items;      // stream-K: every pair takes a share
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2u * static_cast<unsigned>(pairs), 1, 1);
    cfg.blockDim = dim3(Cfg::THREADS, 1, 1);
    cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
    cfg.stream = t_stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1 + pdl_attribute(attr + 1);
    GemmParams q = p;
    q.trace = trace_for(cfg.gridDim.x);
    CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, tmA, tmB, tmB2, tmBt, tmB2t, q));
    g_launches.fetch_add(1);
    note_kernel("gemm_pair_kernel", EPI);
    return MTMC_OK;
}

template <int EPI, bool OUT_BF16>
int launch_big(int clusters, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmB2, const GemmParams& p) {
    using Cfg = BigCfg<EPI>;
    auto kern = gemm_big_kernel<EPI, OUT_BF16>;
    constexpr int SMEM = Cfg::smem_bytes(OUT_BF16);
    if (int rc = ensure_smem_attr(kern, SMEM)) return rc;
    const int pairs = p.num_tiles < clusters ? p.num_tiles : clusters;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2u * static_cast<unsigned>(pairs), 1, 1);
    cfg.blockDim = dim3(Cfg::THREADS, 1, 1);
    cfg.dynamicSmemBytes = SMEM;
    cfg.stream = t_stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1 + pdl_attribute(attr + 1);
    GemmParams q = p;
    q.trace = trace_for(cfg.gridDim.x);
    CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, tmA, tmB, tmB2, q));
    g_launches.fetch_add(1);
    note_kernel("gemm_big_kernel", EPI);
    return MTMC_OK;
}

// How many CTA pairs of the pair kernel fit on the device at once (0: clusters unavailable).
int gemm_pairs(DeviceState* d) {
    if (d->max_gemm_pairs < 0) {
        auto kern = gemm_pair_kernel<EPI_ACT, true>;
        int n = 0;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2u * static_cast<unsigned>(d->sm_count), 1, 1);
        cfg.blockDim = dim3(PairCfg<EPI_ACT>::THREADS, 1, 1);
        cfg.dynamicSmemBytes = PairCfg<EPI_ACT>::SMEM_BYTES;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, PairCfg<EPI_ACT>::SMEM_BYTES) != cudaSuccess ||
            cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) {
            (void)cudaGetLastError();
            n = 0;
        }
        d->max_gemm_pairs = n;
    }
    return d->max_gemm_pairs;
}

template <int EPI, bool OUT_BF16, int KS, int BN = 256>
int launch_ksplit_ks(int tiles, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmB2, const GemmParams& p) {
    using Cfg = KSplitCfg<EPI, KS, BN>;
    auto kern = gemm_ksplit_kernel<EPI, OUT_BF16, KS, BN>;
    if (int rc = ensure_smem_attr(kern, Cfg::SMEM_BYTES)) return rc;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(tiles * KS), 1, 1);
    cfg.blockDim = dim3(Cfg::THREADS, 1, 1);
    cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
    cfg.stream = t_stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = KS;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1 + pdl_attribute(attr + 1);
    GemmParams q = p;
    q.trace = trace_for(cfg.gridDim.x);
    CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, tmA, tmB, tmB2, q));
    g_launches.fetch_add(1);
    note_kernel(BN == 128 ? "gemm_ksplit_kernel (128-column tiles)" : "gemm_ksplit_kernel", EPI, KS);
    return MTMC_OK;
}
// ks: cluster size; negative: the same on 128-column tiles (activation epilogues only, clusters of two or four).
template <int EPI, bool OUT_BF16>
int launch_ksplit(int ks, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmB2, const GemmParams& p) {
    if constexpr (EPI == EPI_ACT) {
        if (ks == -4) return launch_ksplit_ks<EPI, OUT_BF16, 4, 128>(p.num_tiles, tmA, tmB, tmB2, p);
        if (ks == -2) return launch_ksplit_ks<EPI, OUT_BF16, 2, 128>(p.num_tiles, tmA, tmB, tmB2, p);
    }
    if constexpr (EPI != EPI_SWIGLU) {
        if (ks == 8) return launch_ksplit_ks<EPI, OUT_BF16, 8>(p.num_tiles, tmA, tmB, tmB2, p);
    }
    return ks == 4 ? launch_ksplit_ks<EPI, OUT_BF16, 4>(p.num_tiles, tmA, tmB, tmB2, p)
                   : launch_ksplit_ks<EPI, OUT_BF16, 2>(p.num_tiles, tmA, tmB, tmB2, p);
}

// How many clusters of `ks` CTAs of the cluster split-K kernel the device holds at once (0: none).
template <int KS, int BN = 256>
int ksplit_clusters_ks(DeviceState* d) {
    int& cached = d->max_ksplit[(BN == 128 ? 3 : 0) + (KS == 8 ? 2 : (KS == 4 ? 1 : 0))];
    if (cached < 0) {
        using Cfg = KSplitCfg<EPI_ACT, KS, BN>;
        auto kern = gemm_ksplit_kernel<EPI_ACT, true, KS, BN>;
        int n = 0;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>(KS * d->sm_count), 1, 1);
        cfg.blockDim = dim3(Cfg::THREADS, 1, 1);
        cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = KS;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM_BYTES) != cudaSuccess ||
            cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) {
            (void)cudaGetLastError();
            n = 0;
        }
        cached = n;
    }
    return cached;
}

// Cluster split-K (2, 4 or 8 CTAs per 128 x 256 tile) for problems of at most half a wave of tiles whose K is
// long enough to cut (at least 8 k-blocks per CTA): the widest cluster whose tiles all run at once.  0: not this path.
// The tuning hook split_k = 1 turns it off; 2 or 4 cap the cluster size.  SwiGLU tiles have four output chunks,
// so their clusters stop at four.
int pick_ksplit(DeviceState* d, int64_t M, int64_t N, int64_t K, int out_tile_n, bool fp8) {
    if (EPI_HALVES != 1 || t_split_k == 1 || t_tile_n != 0 || t_cta_pair > 0) return 0;
    if (N <= 128) return 0;                                   // those take 128-column tiles
    const int64_t tiles = ((M + 127) / 128) * ((N + out_tile_n - 1) / out_tile_n);
    const int64_t k_blocks = (K + (fp8 ? 127 : 63)) / (fp8 ? 128 : 64);
    const int cap = t_split_k > 0 ? t_split_k : 8;
    if (tiles > d->sm_count / 2) return 0;
    if (cap >= 8 && out_tile_n == 256 && k_blocks >= 64 && tiles <= ksplit_clusters_ks<8>(d) && tiles * 8 <= d->sm_count) return 8;
    if (cap >= 4 && k_blocks >= 32 && tiles <= ksplit_clusters_ks<4>(d) && tiles * 4 <= d->sm_count) return 4;
    if (k_blocks >= 16 && tiles <= ksplit_clusters_ks<2>(d)) return 2;
    return 0;
}

// The same for activation epilogues, which also have 128-column tiles (clusters of two or four; returned as -2 / -4).
// With as many CTAs at work the cluster is half as large and a CTA sends a third of the bytes through distributed
// shared memory (48 KiB instead of 112 KiB in place of a cluster of eight), but half of its ring then holds X, so fewer
// bytes of W are in flight per CTA and a long weight stream runs a tenth slower.  Measured (bias + GELU, 128 rows):
// 4096 x 4096 14.2 us against 18.5 us, 8192 x 8192 32.1 us against 31.4 us.  So: in place of clusters of eight
// always, in place of clusters of four when each CTA's walk is short (at most 64 k-blocks in all), and whenever they
// put more CTAs to work.
int pick_ksplit_act(DeviceState* d, int64_t M, int64_t N, int64_t K, bool fp8) {
    const int wide = pick_ksplit(d, M, N, K, 256, fp8);
    if (wide == 0 || t_split_k == 2) return wide;             // (a cap of two is the hook for clusters of two on the wide tiles)
    const int64_t wide_tiles = ((M + 127) / 128) * ((N + 255) / 256);
    const int64_t tiles = ((M + 127) / 128) * ((N + 127) / 128);
    const int64_t k_blocks = (K + (fp8 ? 127 : 63)) / (fp8 ? 128 : 64);
    if (tiles > d->sm_count / 2) return wide;
    int narrow = 0;
    if (k_blocks >= 32 && tiles <= ksplit_clusters_ks<4, 128>(d) && tiles * 4 <= d->sm_count) narrow = 4;
    else if (k_blocks >= 16 && tiles <= ksplit_clusters_ks<2, 128>(d)) narrow = 2;
    if (narrow == 0 || tiles * narrow < wide_tiles * wide) return wide;
    if (tiles * narrow > wide_tiles * wide) return -narrow;   // more CTAs streaming W (e.g. where no cluster of eight can be placed)
    if (wide != 8 && k_blocks > 64) return wide;
    return -narrow;
}

// The schedule of a cluster split-K launch: one whole tile per cluster; row-reduction partials are laid out as
// for a tile cut into `ks` column pieces (each CTA finishes its own columns).
void fill_ksplit(GemmParams& p, int64_t M, int64_t N, int64_t K, int out_tile_n, int ks, bool fp8);

// Large problems go to CTA pairs (256-row tiles); small ones keep single-CTA 128-row tiles.
bool use_pair(DeviceState* d, int64_t M, int64_t N, int64_t K = 1 << 20) {
    if (t_cta_pair < 0 || t_tile_n == 128 || gemm_pairs(d) <= 0) return false;
    if (t_cta_pair > 0) return true;
    if (M * N * K < (1ll << 28)) return false;
    // from a second 128-row block on: even with the pair tile's lower half mostly empty (M = 129) the pair kernel's
    // mainloop makes up for it (129 ... 256 x 32000 x 4096: 62-70 us against 68-78 us on 128-row tiles)
    // (tiny problems, a microsecond of work or less, keep the plain launch: 256-cube 8.1 us against 8.5-9.5 us as a cluster launch)
    return M > 128 && N >= 256;
}

// Waves of 512 x 256 tiles against waves of 256 x 256 tiles, both counted in 256-row tile waves: the large tiles
// must not lose to the last, partial wave more than they gain per FLOP (nothing at moderate K, up to a tenth
// when K is long).  A problem of 32 large tiles on 74 pairs, say, stays on the small ones.
bool big_waves_ok(int64_t M, int64_t N, int pairs, bool long_k) {
    const int64_t n_tiles = (N + 255) / 256;
    const int64_t t_pair = ((M + 255) / 256) * n_tiles, t_big = ((M + 511) / 512) * n_tiles;
    const int64_t w_pair = (t_pair + pairs - 1) / pairs, w_big = 2 * ((t_big + pairs - 1) / pairs);
    return long_k ? 10 * w_big <= 11 * w_pair : w_big <= w_pair;
}

// The 512 x 256 pair tiles (gemm_big.cuh) against the 256 x 256 ones with overlapped epilogues (gemm_pair.cuh).
// Since the pair kernel hands its ring over two k-blocks at a time its mainloop runs close to the tensor pipe's
// pace as well, and its overlapped epilogue then decides: measured on GELU epilogues it is 4-5 % ahead at
// K = 4096 (C2) and K = 14336, level at K = 8192 and 2 % behind at K = 16384; with E4M3 operands 5-15 % ahead up to
// K = 14336; on the logsumexp epilogue 4 % ahead at K = 4096 (C4: 657 against 684 us).  So the large tiles are
// chosen from 256 k-blocks on (K = 16384 in bf16), when their waves cost no more than a tenth above the pair
// kernel's.  Tuning hook: cta_pair = 2 forces them, 1 forces the 256 x 256 pair tiles.
bool use_big(DeviceState* d, int64_t M, int64_t N, int64_t K, bool fp8) {
    const int pairs = gemm_pairs(d);
    if (pairs <= 0 || EPI_HALVES != 1 || t_tile_n != 0 || t_cta_pair < 0 || t_cta_pair == 1) return false;
    if (t_cta_pair == 2) return true;
    if (M < 512 || N < 256) return false;
    const int64_t k_blocks = (K + (fp8 ? 127 : 63)) / (fp8 ? 128 : 64);
    if (k_blocks < 256) return false;
    return big_waves_ok(M, N, pairs, true);
}

// The same choice for the row reductions (logsumexp, row max, cross entropy).
// SwiGLU stays on the 256 x 256 tiles: its epilogue (two MUFU operations per element plus the stores) is too long
// to expose.
bool use_big_rowred(DeviceState* d, int64_t M, int64_t N, int64_t K, bool fp8) { return use_big(d, M, N, K, fp8); }

// SwiGLU on the 512 x 256 tiles: only when the tuning hook forces them (cta_pair = 2); measured slower by default.
bool use_big_swiglu(DeviceState* d, int64_t M, int64_t N, int64_t K, bool fp8) {
    (void)M; (void)N; (void)K; (void)fp8;
    return gemm_pairs(d) > 0 && EPI_HALVES == 1 && t_tile_n == 0 && t_cta_pair == 2;
}

// Tiling of the output and the split of the wave tail.  With G CTAs, the last T % G tiles
// form a partial wave; cutting each of them into `tail_split` column pieces (2 or 4, pieces
// at least 32 columns wide, all pieces fitting one wave) shortens that wave accordingly.
void fill_tiling(GemmParams& p, int64_t M, int64_t N, int64_t K, int out_tile_n, int sm_count, bool split_tail, int bm = 128,
                 bool fp8 = false) {
    p.M = static_cast<int>(M); p.N = static_cast<int>(N); p.K = static_cast<int>(K);
    p.ldo = p.N;
    p.m_tiles = static_cast<int>((M + bm - 1) / bm);
    p.rows_per_tile = bm;
    p.n_tiles = static_cast<int>((N + out_tile_n - 1) / out_tile_n);
    p.num_tiles = p.m_tiles * p.n_tiles;
    p.fp8 = fp8 ? 1 : 0;
    p.bk_elems = fp8 ? 128 : 64;               // one 128-byte swizzle row of K per ring stage
    p.acc_scale = 1.0f;
    p.acc_scale2 = 1.0f;
    p.k_blocks = static_cast<int>((K + p.bk_elems - 1) / p.bk_elems);
    p.group_m = pick_group_m(p.m_tiles);      // 16 row blocks per group measured best for both tile heights
    p.n_full = p.num_tiles; p.num_items = p.num_tiles; p.tail_split = 1; p.tail_width = out_tile_n;
    const int r = p.num_tiles % sm_count;
    if (split_tail && r > 0) {
        int s = 1;
        for (int cand = 4; cand >= 2; cand /= 2)
            if (r * cand <= sm_count && out_tile_n / cand >= 32) { s = cand; break; }
        if (s > 1) {
            p.n_full = p.num_tiles - r;
            p.tail_split = s;
            p.tail_width = out_tile_n / s;
            p.num_items = p.n_full + r * s;
        }
    }
}

void fill_ksplit(GemmParams& p, int64_t M, int64_t N, int64_t K, int out_tile_n, int ks, bool fp8) {
    fill_tiling(p, M, N, K, out_tile_n, 1, false, 128, fp8);
    p.n_full = 0;
    p.tail_split = ks;
    p.early_w = t_static_weights ? 1 : 0;
}

// Stream-K schedule of the pair kernel (see gemm_pair.cuh): the last full wave plus the remainder (everything, when
// there is less than a wave) is dealt by k-blocks, one equal share per pair.  Needs at least one k-block per pair
// in that region (the holders of a tile are then consecutive pairs).
// Only on request (mtmc_set_schedule(1)).  Measured against the default -- whole tiles with the last wave's tiles
// cut into column pieces, and cluster split-K below half a wave -- it is on a par on C2 (3.46 waves: 104.6 against
// 103.3 us), C3 and C4, 3 % behind on 8192 x 4096 x 11008 (6.9 waves), a few per cent ahead at 1.3 waves
// (768 x 8192 x 8192: 108.7 against 113.3 us) and well behind below one wave (128 x 8192 x 8192: 59 against 35 us
// for cluster split-K): the column pieces already recover most of a partial wave, a share runs 4-6 % slower per
// k-block than whole tiles walked side by side, and a hand-over costs its last holder a serial read of the other
// holders' parts (5 us for a writer, up to 20 us for the reader of two parts, exposed when the share has no whole
// tile to hide it under).
bool want_streamk(const GemmParams& p, int clusters) {
    if (EPI_HALVES != 1 || t_stream_k <= 0 || clusters <= 0 || clusters > SK_MAX_PAIRS) return false;
    const int region = p.num_tiles - std::max(0, p.num_tiles / clusters - 1) * clusters;
    return p.num_tiles % clusters != 0 && static_cast<long long>(region) * p.k_blocks >= clusters;
}
size_t streamk_bytes(int clusters) { return SK_FLAG_BYTES + static_cast<size_t>(clusters) * SK_PART_BYTES; }

// Switches `p` (a pair-kernel tiling) to the stream-K schedule and points it at its scratch, which starts
// `offset` bytes into this call's workspace `ws` (flags first with a caller's workspace, cleared per launch;
// the library's own flags live beside its per-stream scratch and are told apart by epoch instead).
int attach_streamk(DeviceState* d, GemmParams& p, int clusters, void* ws, size_t offset) {
    p.sk = 1;
    p.n_full = p.num_tiles; p.num_items = p.num_tiles; p.tail_split = 1;
    p.sk_first_tile = std::max(0, p.num_tiles / clusters - 1) * clusters;     // all full waves but the last are dealt round-robin
    char* base = static_cast<char*>(ws) + offset;
    if (t_user_ws) {
        p.sk_flags = reinterpret_cast<uint32_t*>(base);
        p.sk_partial = reinterpret_cast<float4*>(base + SK_FLAG_BYTES);
        p.sk_epoch = 1;
        CUDA_TRY(cudaMemsetAsync(p.sk_flags, 0, SK_FLAG_BYTES, t_stream));
    } else {
        DeviceState::StreamScratch* sc = nullptr;
        if (int rc = get_stream_scratch(d, &sc)) return rc;
        if (!sc->sk_flags) {
            CUDA_TRY(counted_malloc(reinterpret_cast<void**>(&sc->sk_flags), SK_FLAG_BYTES));
            CUDA_TRY(cudaMemsetAsync(sc->sk_flags, 0, SK_FLAG_BYTES, t_stream));
        }
        sc->sk_epoch = (sc->sk_epoch % 0xfffffeu) + 1;          // 1 .. 2^24 - 2: fits the ticket word's upper 24 bits, never 0
        p.sk_flags = sc->sk_flags;
        p.sk_partial = reinterpret_cast<float4*>(base + SK_FLAG_BYTES);
        p.sk_epoch = sc->sk_epoch;
    }
    return MTMC_OK;
}

// Tiling for the 256-row pair kernel: the stream-K schedule when it pays, else whole tiles with a split wave
// tail.  Returns whether stream-K was chosen; the caller then adds streamk_bytes() to its workspace request
// and calls attach_streamk().
bool plan_pair(DeviceState* d, GemmParams& p, int64_t M, int64_t N, int64_t K, int out_tile_n, bool fp8) {
    const int clusters = gemm_pairs(d);
    fill_tiling(p, M, N, K, out_tile_n, clusters, false, 256, fp8);
    if (want_streamk(p, clusters)) return true;
    fill_tiling(p, M, N, K, out_tile_n, clusters, true, 256, fp8);
    return false;
}
// The workspace of a pair-kernel call with no other scratch: nothing, or the stream-K region.
int pair_scratch(DeviceState* d, GemmParams& p, bool sk) {
    if (!sk) return MTMC_OK;
    const int clusters = gemm_pairs(d);
    void* ws = nullptr;
    if (int rc = get_workspace(d, streamk_bytes(clusters), &ws)) return rc;
    return attach_streamk(d, p, clusters, ws, 0);
}

int skinny_cta_of_unit_host(long long u, long long total, int grid) {
    return static_cast<int>(((u + 1) * grid - 1) / total);
}

struct SkinnyPlan {
    int n_tiles, k_blocks, grid, max_slots, tile_rows, stages, pair, mx;
    long long total;
    size_t ticket_bytes, partial_bytes;
};

// Bands of W rows and the grid.
//  * pair plan (default when W has at least 32 rows per CTA pair): one band per cluster of two
//    CTAs, bands sized so that the clusters cover the SMs; each CTA takes half of K and the
//    pair reduces through distributed shared memory.
//  * ticket plan (few rows, or a forced split): 128-row bands, the (band, k-block) list cut
//    evenly over the SMs or over n_tiles * split_k CTAs; partials and tickets in the workspace.
SkinnyPlan plan_skinny(int sm_count, int pairs, int64_t M, int64_t N, int64_t K, int bk_elems = 64) {
    SkinnyPlan s;
    s.mx = M <= 16 ? 16 : (M <= 32 ? 32 : 64);
    s.k_blocks = static_cast<int>((K + bk_elems - 1) / bk_elems);
    s.tile_rows = 128;
    s.n_tiles = static_cast<int>((N + 127) / 128);
    s.pair = 0;
    long long g = t_split_k > 0 ? static_cast<long long>(s.n_tiles) * t_split_k : sm_count;
    if (t_split_k == 0 && pairs > 0 && s.k_blocks >= 2) {
        int64_t rows = (N + pairs - 1) / pairs;               // rows per band if every pair gets one band
        rows = (rows + 7) / 8 * 8;
        if (rows >= 32 && rows <= 128) {
            s.pair = 1;
            s.tile_rows = static_cast<int>(rows);
            s.n_tiles = static_cast<int>((N + rows - 1) / rows);
            g = 2ll * s.n_tiles;
        }
    }
    s.total = static_cast<long long>(s.n_tiles) * s.k_blocks;
    if (!s.pair) {
        if (g > s.total) g = s.total;
        if (g > 65535 * 16) g = 65535 * 16;
    }
    s.grid = static_cast<int>(g);
    s.stages = s.mx == 16 ? SkinnyCfg<16>::stages_for(s.tile_rows)
                          : (s.mx == 32 ? SkinnyCfg<32>::stages_for(s.tile_rows) : SkinnyCfg<64>::stages_for(s.tile_rows));
    int mx = 1;
    if (!s.pair) {
        for (int t = 0; t < s.n_tiles; ++t) {
            long long first = static_cast<long long>(t) * s.k_blocks;
            int nc = skinny_cta_of_unit_host(first + s.k_blocks - 1, s.total, s.grid) - skinny_cta_of_unit_host(first, s.total, s.grid) + 1;
            if (nc > mx) mx = nc;
        }
    }
    s.max_slots = mx;
    s.ticket_bytes = s.pair ? 0 : round256(static_cast<size_t>(s.n_tiles) * 4);
    s.partial_bytes = mx > 1 ? static_cast<size_t>(s.n_tiles) * s.max_slots * s.mx * 128 * 4 : 0;
    return s;
}

// The weight-streaming kernel takes at most 64 rows of X.  skinny_possible: the shape fits it at all.  prefer_skinny: it is
// the first choice -- when W has at least 64 rows per CTA pair (shorter bands leave its 128-lane MMAs mostly empty and its
// CTAs bound by the k-blocks they issue, not by the bytes they stream: 16 x 4096 x 14336 34.7 us against 27.1 us on the
// cluster split-K kernel, 64 x 1024 x 4096 30.8 against 10.9 us) and, from 17 rows of X on, only on its pair plan
// (N <= 128 x pairs; on the ticket plan its time grows with the rows of X: 64 x 14336 x 4096 40.7 against 29.2 us).
// Shapes it is not preferred for go to the cluster split-K kernel when that applies and come back here otherwise.
int skinny_pairs(DeviceState* d);
bool skinny_possible(int64_t M, int64_t N) { return M <= SKINNY_MAX_M && (N + 31) / 32 <= static_cast<int64_t>(TICKET_BYTES / 4); }
bool prefer_skinny(DeviceState* d, int64_t M, int64_t N) {
    if (!skinny_possible(M, N)) return false;
    if (t_split_k > 0) return true;
    const int pairs = skinny_pairs(d);
    if (pairs <= 0) return M <= 16;
    return N >= 64ll * pairs && (N <= 128ll * pairs || M <= 16);
}

// One thread waits, with a one-millisecond limit, on an mbarrier that nothing ever arrives on:
// the bounded wait gives up, records the status word and the kernel returns normally.
__global__ void timeout_probe_kernel(uint32_t* status) {
    __shared__ __align__(8) unsigned long long bar;
    __shared__ uint32_t abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0u;
        mbar_init(smem_u32(&bar), 1);
        fence_barrier_init();
        mbar_wait(smem_u32(&bar), 0u, &abort_flag, status, STATUS_TIMEOUT_EPILOGUE | 0xEEu, 2000000ll);
    }
}

template <bool OUT_BF16, bool PAIR, int MX, bool FP8>
int launch_skinny(const SkinnyPlan& s, const CUtensorMap& tmW, const CUtensorMap& tmX, const SkinnyParams& p) {
    auto kern = skinny_splitk_kernel<OUT_BF16, PAIR, MX, FP8>;
    if (int rc = ensure_smem_attr(kern, SkinnyCfg<MX>::SMEM_BYTES)) return rc;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(s.grid), 1, 1);
    cfg.blockDim = dim3(192, 1, 1);
    cfg.dynamicSmemBytes = SkinnyCfg<MX>::SMEM_BYTES;
    cfg.stream = t_stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = PAIR ? 2 : 1;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1 + pdl_attribute(attr + 1);
    SkinnyParams q = p;
    q.trace = trace_for(cfg.gridDim.x);
    CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, tmW, tmX, q));
    g_launches.fetch_add(1);
    note_kernel(PAIR ? "skinny_splitk_kernel (pair plan)" : "skinny_splitk_kernel (ticket plan)", -1, MX);
    return MTMC_OK;
}

// How many 2-CTA clusters of the skinny kernel the device can hold at once (0 if clusters
// cannot be scheduled): the pair plan sizes its bands to this.
int skinny_pairs(DeviceState* d) {
    if (d->max_pairs < 0) {
        auto kern = skinny_splitk_kernel<true, true, 16>;
        int n = 0;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2u * static_cast<unsigned>(d->sm_count), 1, 1);
        cfg.blockDim = dim3(192, 1, 1);
        cfg.dynamicSmemBytes = SkinnyCfg<16>::SMEM_BYTES;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SkinnyCfg<16>::SMEM_BYTES) != cudaSuccess ||
            cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) {
            (void)cudaGetLastError();
            n = 0;
        }
        d->max_pairs = n;
    }
    return d->max_pairs;
}

int run_skinny(DeviceState* d, const void* X, const void* W, const float* b, const void* R, int64_t M, int64_t N, int64_t K,
               int act, int out_dtype, void* out, bool fp8 = false, float acc_scale = 1.0f, int64_t ldx = 0, int64_t ldw = 0,
               int64_t ldo = 0) {
    SkinnyPlan s = plan_skinny(d->sm_count, skinny_pairs(d), M, N, K, fp8 ? 128 : 64);
    SkinnyParams p{};
    p.acc_scale = acc_scale;
    p.early_w = t_static_weights;
    p.M = static_cast<int>(M); p.N = static_cast<int>(N); p.K = static_cast<int>(K);
    p.ldo = static_cast<int>(ldo > 0 ? ldo : N);
    p.n_tiles = s.n_tiles; p.k_blocks = s.k_blocks; p.total_units = s.total; p.max_slots = s.max_slots;
    p.tile_rows = s.tile_rows; p.num_stages = s.stages;
    p.act = act; p.bias = b; p.residual = R; p.out = out; p.status = d->status;
    void* ws = nullptr;
    if (t_user_ws) {
        int rc = get_workspace(d, s.ticket_bytes + s.partial_bytes, &ws);
        if (rc) return rc;
        p.tickets = static_cast<uint32_t*>(ws);
        p.partial = reinterpret_cast<float*>(static_cast<char*>(ws) + s.ticket_bytes);
    } else {
        int rc = get_workspace(d, s.partial_bytes, &ws);
        if (rc) return rc;
        p.partial = static_cast<float*>(ws);
        p.tickets = nullptr;
        if (s.ticket_bytes) {
            DeviceState::StreamScratch* sc = nullptr;
            if ((rc = get_stream_scratch(d, &sc))) return rc;
            if (!sc->tickets) CUDA_TRY(counted_malloc(reinterpret_cast<void**>(&sc->tickets), TICKET_BYTES));
            p.tickets = sc->tickets;
        }
    }
    // The tickets of this launch start at zero whatever an earlier launch left behind (one that timed out does
    // not reset its own): a stream-ordered clear of the words in use.  Only the ticket plan pays for it.
    if (s.ticket_bytes) CUDA_TRY(cudaMemsetAsync(p.tickets, 0, s.ticket_bytes, t_stream));
    CUtensorMap tmW, tmX;
    int rc = fp8 ? encode_u8_2d(&tmW, W, N, K, s.tile_rows) : encode_bf16_2d(&tmW, W, N, K, s.tile_rows, ldw);
    if (rc) return rc;
    rc = fp8 ? encode_u8_2d(&tmX, X, M, K, s.mx) : encode_bf16_2d(&tmX, X, M, K, s.mx, ldx);
    if (rc) return rc;
    TimedRegion tr(d);
    const bool bf = out_dtype == MTMC_OUT_BF16;
#define MTMC_SKINNY_DISPATCH(MXV, F8)                                                                         \
    rc = bf ? (s.pair ? launch_skinny<true, true, MXV, F8>(s, tmW, tmX, p) : launch_skinny<true, false, MXV, F8>(s, tmW, tmX, p)) \
            : (s.pair ? launch_skinny<false, true, MXV, F8>(s, tmW, tmX, p) : launch_skinny<false, false, MXV, F8>(s, tmW, tmX, p))
    if (fp8) {
        if (s.mx == 16) { MTMC_SKINNY_DISPATCH(16, true); }
        else if (s.mx == 32) { MTMC_SKINNY_DISPATCH(32, true); }
        else { MTMC_SKINNY_DISPATCH(64, true); }
    } else {
        if (s.mx == 16) { MTMC_SKINNY_DISPATCH(16, false); }
        else if (s.mx == 32) { MTMC_SKINNY_DISPATCH(32, false); }
        else { MTMC_SKINNY_DISPATCH(64, false); }
    }
#undef MTMC_SKINNY_DISPATCH
    tr.stop();
    return rc;
}

// One call through host pointers.  `in[i]` / `out` give host address and size of each operand (a null address
// skips it); `launch` enqueues the device entry point on the compute stream given the device copies.  The copy in
// runs on its own stream, the kernels on the caller's stream, the copy out on a third, chained by events, so
// consecutive calls overlap: the next call's operands travel while this call computes and its result travels
// back.  A slot is reused only after its previous copy out has finished.  blocking: wait for the result.
// Host threads that share a device should not interleave asynchronous calls (they would share slots).
struct HostOperand { const void* host; size_t bytes; };
template <class Launch>
int host_call(const HostOperand (&in)[4], void* out_host, size_t out_bytes, bool blocking, Launch launch) {
    DeviceState* d = nullptr;
    int rc = get_device(&d);
    if (rc) return rc;
    DeviceState::HostSlot* slot = nullptr;
    {   // the ring position is the only state shared between host threads; the device entry point takes the lock itself
        std::lock_guard<std::mutex> lock(g_mutex);
        if (!d->s_in) {
            CUDA_TRY(cudaStreamCreateWithFlags(&d->s_in, cudaStreamNonBlocking));
            CUDA_TRY(cudaStreamCreateWithFlags(&d->s_out, cudaStreamNonBlocking));
        }
        slot = &d->hslot[d->hnext];
        d->hnext = (d->hnext + 1) % DeviceState::HOST_SLOTS;
    }
    DeviceState::HostSlot& s = *slot;
    if (!s.in_done) {
        CUDA_TRY(cudaEventCreateWithFlags(&s.in_done, cudaEventDisableTiming));
        CUDA_TRY(cudaEventCreateWithFlags(&s.k_done, cudaEventDisableTiming));
        CUDA_TRY(cudaEventCreateWithFlags(&s.out_done, cudaEventDisableTiming));
    }
    if (s.busy) { CUDA_TRY(cudaEventSynchronize(s.out_done)); s.busy = false; }
    void* dev[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
    for (int i = 0; i < 5; ++i) {
        const size_t need = i < 4 ? (in[i].host ? in[i].bytes : 0) : out_bytes;
        if (need == 0) continue;
        if (d->hwm[i] < need) d->hwm[i] = need;      // largest operand seen in this position, by any slot
        if (s.bytes[i] < need) {        // the slot is idle: nothing on the device still uses its buffers
            if (s.buf[i]) { CUDA_TRY(cudaFree(s.buf[i])); s.buf[i] = nullptr; s.bytes[i] = 0; }
            CUDA_TRY(counted_malloc(&s.buf[i], d->hwm[i]));     // sized for the largest, so that a steady workload stops reallocating
            s.bytes[i] = d->hwm[i];
        }
        dev[i] = s.buf[i];
    }
    for (int i = 0; i < 4; ++i)
        if (dev[i]) CUDA_TRY(cudaMemcpyAsync(dev[i], in[i].host, in[i].bytes, cudaMemcpyHostToDevice, d->s_in));
    CUDA_TRY(cudaEventRecord(s.in_done, d->s_in));
    CUDA_TRY(cudaStreamWaitEvent(t_stream, s.in_done, 0));
    rc = launch(dev);
    if (rc) return rc;
    CUDA_TRY(cudaEventRecord(s.k_done, t_stream));
    CUDA_TRY(cudaStreamWaitEvent(d->s_out, s.k_done, 0));
    CUDA_TRY(cudaMemcpyAsync(out_host, dev[4], out_bytes, cudaMemcpyDeviceToHost, d->s_out));
    CUDA_TRY(cudaEventRecord(s.out_done, d->s_out));
    s.busy = true;
    if (blocking) { CUDA_TRY(cudaEventSynchronize(s.out_done)); s.busy = false; }
    return MTMC_OK;
}

int fused_linear_host_impl(const void* X, const void* W, const float* b, int64_t M, int64_t N, int64_t K, int act, int out_dtype,
                           void* out, bool blocking);
int swiglu_host_impl(const void* X, const void* Wg, const void* Wu, int64_t M, int64_t N, int64_t K, void* out, bool blocking);
int linear_lse_host_impl(const void* X, const void* W, const float* b, int64_t M, int64_t N, int64_t K, float* lse_out, bool blocking);

// The three row reductions over the never-materialised logits share one driver: a tiled kernel
// leaves one partial per (row, column piece) in the workspace, a merge kernel finishes the rows.
//   EPI_LSE    : out_a = lse                     EPI_ROWMAX : out_a = max, out_i = argmax (may be null)
//   EPI_XENT   : out_b = loss, out_a = lse (may be null); the target logits sit behind the partials
//   EPI_SOFTMAX: prob = the [M,N] probabilities (fp32 / bf16, rows ldo elements apart), out_a = lse (may be null: a merge
//                launch then leaves it behind the partials); the tiled kernel leaves exp(z - max of the piece) in prob,
//                the finishing kernel scales every piece (and merges the partials itself when a row has few of them)
template <int EPI>
int run_row_reduction(const void* X, const void* W, const float* b, const int64_t* targets, int64_t M, int64_t N, int64_t K,
                      float* out_a, float* out_b, int32_t* out_i, bool fp8 = false, float acc_scale = 1.0f, int64_t ldx = 0, int64_t ldw = 0,
                      void* prob = nullptr, int out_dtype = MTMC_OUT_FP32, int64_t ldo = 0) {
    auto encode = fp8 ? encode_u8_2d : encode_bf16_2d;
    if (b && !aligned16(b)) return fail(MTMC_ERR_INVALID_ARG, "bias must be 16-byte aligned");
    DeviceState* d = nullptr;
    int rc = get_device(&d);
    if (rc) return rc;
    // the softmax epilogue runs on the kernels whose pieces the finishing kernel knows: all but the 512 x 256 tiles
    const int ks = pick_ksplit(d, M, N, K, 256, fp8);
    const bool big = EPI != EPI_SOFTMAX && !ks && use_big_rowred(d, M, N, K, fp8);
    const bool pair = !ks && !big && use_pair(d, M, N, K);
    const int bn = (pair || ks || big) ? 256 : pick_tile_n(N);
    GemmParams p{};
    bool sk = false;
    if (ks) fill_ksplit(p, M, N, K, 256, ks, fp8);
    else if (big) fill_tiling(p, M, N, K, 256, gemm_pairs(d), false, 512, fp8);
    else if (pair) sk = plan_pair(d, p, M, N, K, 256, fp8);
    else fill_tiling(p, M, N, K, bn, d->sm_count, true, 128, fp8);
    p.acc_scale = acc_scale;
    const size_t partial_bytes = lse_partial_bytes(p);         // what the chosen plan writes and the merge reads
    const size_t extra = (EPI == EPI_XENT || EPI == EPI_SOFTMAX) ? round256(static_cast<size_t>(M) * sizeof(float)) : 0;
    const int sk_clusters = sk ? gemm_pairs(d) : 0;
    void* ws = nullptr;
    rc = get_workspace(d, partial_bytes + extra + (sk ? streamk_bytes(sk_clusters) : 0), &ws);
    if (rc) return rc;
    if (sk && (rc = attach_streamk(d, p, sk_clusters, ws, partial_bytes + extra))) return rc;
    p.act = ACT_NONE; p.bias = b; p.out = prob; if (ldo > 0) p.ldo = static_cast<int>(ldo); p.lse_partial = static_cast<float2*>(ws); p.status = d->status;
    p.targets = reinterpret_cast<const long long*>(targets);
    p.target_logit = EPI == EPI_XENT ? reinterpret_cast<float*>(static_cast<char*>(ws) + partial_bytes) : nullptr;
    // a target outside [0, N) matches no column: its row's loss comes out as NaN instead of a stale value
    if (EPI == EPI_XENT) CUDA_TRY(cudaMemsetAsync(p.target_logit, 0xFF, static_cast<size_t>(M) * sizeof(float), t_stream));
    CUtensorMap tmA, tmB, tmBt;
    if ((rc = encode(&tmA, X, M, K, big ? 256 : 128, ldx)) || (rc = encode(&tmB, W, N, K, (pair || big) ? 128 : bn, ldw)) ||
        (rc = encode(&tmBt, W, N, K, (pair || big) ? p.tail_width / 2 : p.tail_width, ldw)))
        return rc;
    TimedRegion tr(d);
    if constexpr (EPI == EPI_SOFTMAX) {
        const bool bf = out_dtype == MTMC_OUT_BF16;
        if (ks) rc = bf ? launch_ksplit<EPI, true>(ks, tmA, tmB, tmB, p) : launch_ksplit<EPI, false>(ks, tmA, tmB, tmB, p);
        else if (pair) rc = bf ? launch_pair<EPI, true>(gemm_pairs(d), tmA, tmB, tmB, tmBt, tmBt, p)
                          : launch_pair<EPI, false>(gemm_pairs(d), tmA, tmB, tmB, tmBt, tmBt, p);
        else if (bn == 256) rc = bf ? launch_tiled<EPI, 256, true>(d, tmA, tmB, tmB, tmBt, tmBt, p)
                                    : launch_tiled<EPI, 256, false>(d, tmA, tmB, tmB, tmBt, tmBt, p);
        else rc = bf ? launch_tiled<EPI, 128, true>(d, tmA, tmB, tmB, tmBt, tmBt, p)
                     : launch_tiled<EPI, 128, false>(d, tmA, tmB, tmB, tmBt, tmBt, p);
    } else {
        if (ks) rc = launch_ksplit<EPI, false>(ks, tmA, tmB, tmB, p);
        else if (big) rc = launch_big<EPI, false>(gemm_pairs(d), tmA, tmB, tmB, p);
        else if (pair) rc = launch_pair<EPI, false>(gemm_pairs(d), tmA, tmB, tmB, tmBt, tmBt, p);
        else rc = bn == 256 ? launch_tiled<EPI, 256, false>(d, tmA, tmB, tmB, tmBt, tmBt, p)
                            : launch_tiled<EPI, 128, false>(d, tmA, tmB, tmB, tmBt, tmBt, p);
    }
    tr.stop();
    if (rc) return rc;
    const unsigned blocks = static_cast<unsigned>((M + 7) / 8);      // eight rows per block of the finishing pass
    const dim3 merge_grid(static_cast<unsigned>((M + 31) / 32), 1, 1);
    const unsigned merge_threads = 32u * MERGE_WARPS;
    if constexpr (EPI == EPI_SOFTMAX) {
        // one warp per row and span of eight column tiles: many short blocks, so that the last wave costs little
        const int out_tile_n = (pair || ks || bn == 256) ? 256 : 128;
        const int tiles_per_span = std::max(8, (p.n_tiles + 65534) / 65535);      // grid.y stays within its limit
        const dim3 grid(blocks, static_cast<unsigned>((p.n_tiles + tiles_per_span - 1) / tiles_per_span), 1);
        const bool bf = out_dtype == MTMC_OUT_BF16;
        if (p.n_tiles * p.tail_split <= 256) {      // few pieces per row: every warp of the finishing kernel merges them itself
            auto finish = bf ? softmax_finish_kernel<true, true> : softmax_finish_kernel<false, true>;
            return launch_follow_up(finish, grid, 256u, prob, p.ldo, static_cast<const float2*>(p.lse_partial), out_a, p.M, p.N,
                                    p.rows_per_tile, p.m_tiles, p.n_tiles, p.group_m, p.n_full, p.tail_split, out_tile_n, tiles_per_span);
        }
        float* lse = out_a ? out_a : reinterpret_cast<float*>(static_cast<char*>(ws) + partial_bytes);
        if ((rc = launch_follow_up(lse_merge_rows_kernel, merge_grid, merge_threads, static_cast<const float2*>(p.lse_partial), p.M, p.rows_per_tile,
                                   p.m_tiles, p.n_tiles, p.group_m, p.n_full, p.tail_split, lse, static_cast<const float*>(nullptr),
                                   static_cast<float*>(nullptr))))
            return rc;
        auto finish = bf ? softmax_finish_kernel<true, false> : softmax_finish_kernel<false, false>;
        return launch_follow_up(finish, grid, 256u, prob, p.ldo, static_cast<const float2*>(p.lse_partial), lse, p.M, p.N,
                                p.rows_per_tile, p.m_tiles, p.n_tiles, p.group_m, p.n_full, p.tail_split, out_tile_n, tiles_per_span);
    }
    if (EPI == EPI_ROWMAX)
        return launch_follow_up(rowmax_merge_rows_kernel, merge_grid, merge_threads, static_cast<const float2*>(p.lse_partial), p.M, p.rows_per_tile,
                                p.m_tiles, p.n_tiles, p.group_m, p.n_full, p.tail_split, out_a, out_i);
    return launch_follow_up(lse_merge_rows_kernel, merge_grid, merge_threads, static_cast<const float2*>(p.lse_partial), p.M, p.rows_per_tile,
                            p.m_tiles, p.n_tiles, p.group_m, p.n_full, p.tail_split, out_a, static_cast<const float*>(p.target_logit), out_b);
}

// out = act(X.W^T + b) (+ R): picks the weight-streaming path for decode batches, CTA pairs for
// large shapes and single-CTA tiles otherwise.
int fused_linear_impl(const void* X, const void* W, const float* b, const void* R, int64_t M, int64_t N, int64_t K, int act,
                      int out_dtype, void* out, int64_t ldx = 0, int64_t ldw = 0, int64_t ldo = 0) {
    int rc = check_common(X, W, out, M, N, K);
    if (rc) return rc;
    if (act < 0 || act > 3) return fail(MTMC_ERR_INVALID_ARG, "unknown activation id %d", act);
    if (out_dtype != MTMC_OUT_FP32 && out_dtype != MTMC_OUT_BF16) return fail(MTMC_ERR_INVALID_ARG, "unknown output type id %d", out_dtype);
    if (b && !aligned16(b)) return fail(MTMC_ERR_INVALID_ARG, "bias must be 16-byte aligned");
    DeviceState* d = nullptr;
    rc = get_device(&d);
    if (rc) return rc;
    if (prefer_skinny(d, M, N)) return run_skinny(d, X, W, b, R, M, N, K, act, out_dtype, out, false, 1.0f, ldx, ldw, ldo);

    if (const int ks = pick_ksplit_act(d, M, N, K, false)) {
        GemmParams p{};
        const int bn = ks < 0 ? 128 : 256;
        fill_ksplit(p, M, N, K, bn, ks < 0 ? -ks : ks, false);
        p.act = act; p.bias = b; p.residual = R; p.out = out; if (ldo > 0) p.ldo = static_cast<int>(ldo); p.lse_partial = nullptr; p.status = d->status;
        CUtensorMap tmA, tmB;
        if ((rc = encode_bf16_2d(&tmA, X, M, K, 128, ldx)) || (rc = encode_bf16_2d(&tmB, W, N, K, bn, ldw))) return rc;
        TimedRegion tr(d);
        rc = out_dtype == MTMC_OUT_BF16 ? launch_ksplit<EPI_ACT, true>(ks, tmA, tmB, tmB, p) : launch_ksplit<EPI_ACT, false>(ks, tmA, tmB, tmB, p);
        tr.stop();
        return rc;
    }
    if (skinny_possible(M, N) && t_tile_n == 0 && t_cta_pair <= 0)      // no cluster split-K for the shape (short K, too many tiles): stream the weights after all
        return run_skinny(d, X, W, b, R, M, N, K, act, out_dtype, out, false, 1.0f, ldx, ldw, ldo);
    if (use_big(d, M, N, K, false)) {
        GemmParams p{};
        fill_tiling(p, M, N, K, 256, gemm_pairs(d), false, 512);
        p.act = act; p.bias = b; p.residual = R; p.out = out; if (ldo > 0) p.ldo = static_cast<int>(ldo); p.lse_partial = nullptr; p.status = d->status;
        CUtensorMap tmA, tmB;
        if ((rc = encode_bf16_2d(&tmA, X, M, K, 256, ldx)) || (rc = encode_bf16_2d(&tmB, W, N, K, 128, ldw))) return rc;
        TimedRegion tr(d);
        rc = out_dtype == MTMC_OUT_BF16 ? launch_big<EPI_ACT, true>(gemm_pairs(d), tmA, tmB, tmB, p)
                                        : launch_big<EPI_ACT, false>(gemm_pairs(d), tmA, tmB, tmB, p);
        tr.stop();
        return rc;
    }
    if (use_pair(d, M, N, K)) {
        GemmParams p{};
        const bool sk = plan_pair(d, p, M, N, K, 256, false);
        if ((rc = pair_scratch(d, p, sk))) return rc;
        p.act = act; p.bias = b; p.residual = R; p.out = out; if (ldo > 0) p.ldo = static_cast<int>(ldo); p.lse_partial = nullptr; p.status = d->status;
        CUtensorMap tmA, tmB, tmBt;
        if ((rc = encode_bf16_2d(&tmA, X, M, K, 128, ldx)) || (rc = encode_bf16_2d(&tmB, W, N, K, 128, ldw)) ||
            (rc = encode_bf16_2d(&tmBt, W, N, K, p.tail_width / 2, ldw)))
            return rc;
        TimedRegion tr(d);
        rc = out_dtype == MTMC_OUT_BF16 ? launch_pair<EPI_ACT, true>(gemm_pairs(d), tmA, tmB, tmB, tmBt, tmBt, p)
                                        : launch_pair<EPI_ACT, false>(gemm_pairs(d), tmA, tmB, tmB, tmBt, tmBt, p);
        tr.stop();
        return rc;
    }
    const int bn = pick_tile_n(N);
    GemmParams p{};
    fill_tiling(p, M, N, K, bn, d->sm_count, true);
    p.act = act; p.bias = b; p.residual = R; p.out = out; if (ldo > 0) p.ldo = static_cast<int>(ldo); p.lse_partial = nullptr; p.status = d->status;
    CUtensorMap tmA, tmB, tmBt;
    rc = encode_bf16_2d(&tmA, X, M, K, 128, ldx);
    if (rc) return rc;
    rc = encode_bf16_2d(&tmB, W, N, K, bn, ldw);
    if (rc) return rc;
    rc = encode_bf16_2d(&tmBt, W, N, K, p.tail_width, ldw);
    if (rc) return rc;
    TimedRegion tr(d);
    if (bn == 256) {
        rc = out_dtype == MTMC_OUT_BF16 ? launch_tiled<EPI_ACT, 256, true>(d, tmA, tmB, tmB, tmBt, tmBt, p)
                                        : launch_tiled<EPI_ACT, 256, false>(d, tmA, tmB, tmB, tmBt, tmBt, p);
    } else {
        rc = out_dtype == MTMC_OUT_BF16 ? launch_tiled<EPI_ACT, 128, true>(d, tmA, tmB, tmB, tmBt, tmBt, p)
                                        : launch_tiled<EPI_ACT, 128, false>(d, tmA, tmB, tmB, tmBt, tmBt, p);
    }
    tr.stop();
    return rc;
}
// out = silu(sg * X.Wg^T) * (su * X.Wu^T): bf16 operands (sg = su = 1) or E4M3 operands with the scale products.
int swiglu_impl(const void* X, const void* Wg, const void* Wu, int64_t M, int64_t N, int64_t K, void* out, bool fp8, float sg, float su,
                int64_t ldx = 0, int64_t ldwg = 0, int64_t ldwu = 0, int64_t ldo = 0) {
    auto encode = fp8 ? encode_u8_2d : encode_bf16_2d;
    int rc = check_common(X, Wg, out, M, N, K);
    if (rc) return rc;
    if (!Wu) return fail(MTMC_ERR_INVALID_ARG, "null pointer argument");
    if (!aligned16(Wu)) return fail(MTMC_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
    DeviceState* d = nullptr;
    rc = get_device(&d);
    if (rc) return rc;
    if (const int ks = pick_ksplit(d, M, N, K, 128, fp8)) {
        GemmParams p{};
        fill_ksplit(p, M, N, K, 128, ks, fp8);
        p.acc_scale = sg; p.acc_scale2 = su;
        p.act = ACT_NONE; p.bias = nullptr; p.out = out; if (ldo > 0) p.ldo = static_cast<int>(ldo); p.lse_partial = nullptr; p.status = d->status;
        CUtensorMap tmA, tmG, tmU;
        if ((rc = encode(&tmA, X, M, K, 128, ldx)) || (rc = encode(&tmG, Wg, N, K, 128, ldwg)) ||
            (rc = encode(&tmU, Wu, N, K, 128, ldwu)))
            return rc;
        TimedRegion tr(d);
        rc = launch_ksplit<EPI_SWIGLU, true>(ks, tmA, tmG, tmU, p);
        tr.stop();
        return rc;
    }
    if (use_big_swiglu(d, M, N, K, fp8)) {
        GemmParams p{};
        fill_tiling(p, M, N, K, 128, gemm_pairs(d), false, 512, fp8);
        p.acc_scale = sg; p.acc_scale2 = su;
        p.act = ACT_NONE; p.bias = nullptr; p.out = out; if (ldo > 0) p.ldo = static_cast<int>(ldo); p.lse_partial = nullptr; p.status = d->status;
        CUtensorMap tmA, tmG, tmU;
        if ((rc = encode(&tmA, X, M, K, 256, ldx)) || (rc = encode(&tmG, Wg, N, K, 128, ldwg)) || (rc = encode(&tmU, Wu, N, K, 128, ldwu))) return rc;
        TimedRegion tr(d);
        rc = launch_big<EPI_SWIGLU, true>(gemm_pairs(d), tmA, tmG, tmU, p);
        tr.stop();
        return rc;
    }
    if (use_pair(d, M, N, K)) {
        GemmParams p{};
        const bool sk = plan_pair(d, p, M, N, K, 128, fp8);
        if ((rc = pair_scratch(d, p, sk))) return rc;
        p.acc_scale = sg; p.acc_scale2 = su;
        p.act = ACT_NONE; p.bias = nullptr; p.out = out; if (ldo > 0) p.ldo = static_cast<int>(ldo); p.lse_partial = nullptr; p.status = d->status;
        CUtensorMap tmA, tmG, tmU, tmGt, tmUt;
        if ((rc = encode(&tmA, X, M, K, 128, ldx)) || (rc = encode(&tmG, Wg, N, K, 128, ldwg)) ||
            (rc = encode(&tmU, Wu, N, K, 128, ldwu)) || (rc = encode(&tmGt, Wg, N, K, p.tail_width, ldwg)) ||
            (rc = encode(&tmUt, Wu, N, K, p.tail_width, ldwu)))
            return rc;
        TimedRegion tr(d);
        rc = launch_pair<EPI_SWIGLU, true>(gemm_pairs(d), tmA, tmG, tmU, tmGt, tmUt, p);
        tr.stop();
        return rc;
    }
    GemmParams p{};
    fill_tiling(p, M, N, K, 128, d->sm_count, true, 128, fp8);   // 128 output columns = 128 gate + 128 up accumulator columns
    p.acc_scale = sg; p.acc_scale2 = su;
        p.act = ACT_NONE; p.bias = nullptr; p.out = out; if (ldo > 0) p.ldo = static_cast<int>(ldo); p.lse_partial = nullptr; p.status = d->status;
    CUtensorMap tmA, tmG, tmU, tmGt, tmUt;
    rc = encode(&tmA, X, M, K, 128, ldx);
    if (rc) return rc;
    rc = encode(&tmG, Wg, N, K, 128, ldwg);
    if (rc) return rc;
    rc = encode(&tmU, Wu, N, K, 128, ldwu);
    if (rc) return rc;
    rc = encode(&tmGt, Wg, N, K, p.tail_width, ldwg);
    if (rc) return rc;
    rc = encode(&tmUt, Wu, N, K, p.tail_width, ldwu);
    if (rc) return rc;
    TimedRegion tr(d);
    rc = launch_tiled<EPI_SWIGLU, 256, true>(d, tmA, tmG, tmU, tmGt, tmUt, p);
    tr.stop();
    return rc;
}

int fused_linear_host_impl(const void* X, const void* W, const float* b, int64_t M, int64_t N, int64_t K, int act, int out_dtype,
                           void* out, bool blocking) {
    if (!X || !W || !out) return fail(MTMC_ERR_INVALID_ARG, "null pointer argument");
    if (M <= 0 || N <= 0 || K <= 0) return fail(MTMC_ERR_INVALID_ARG, "M, N, K must be positive");
    if (out_dtype != MTMC_OUT_FP32 && out_dtype != MTMC_OUT_BF16) return fail(MTMC_ERR_INVALID_ARG, "unknown output type id %d", out_dtype);
    const size_t xb = static_cast<size_t>(M) * K * 2, wb = static_cast<size_t>(N) * K * 2, bb = static_cast<size_t>(N) * 4;
    const size_t ob = static_cast<size_t>(M) * N * (out_dtype == MTMC_OUT_BF16 ? 2 : 4);
    const HostOperand in[4] = {{X, xb}, {W, wb}, {nullptr, 0}, {b, bb}};
    return host_call(in, out, ob, blocking, [&](void* const* dev) {
        return mtmc_fused_linear(dev[0], dev[1], static_cast<const float*>(dev[3]), M, N, K, act, out_dtype, dev[4]);
    });
}

int swiglu_host_impl(const void* X, const void* Wg, const void* Wu, int64_t M, int64_t N, int64_t K, void* out, bool blocking) {
    if (!X || !Wg || !Wu || !out) return fail(MTMC_ERR_INVALID_ARG, "null pointer argument");
    if (M <= 0 || N <= 0 || K <= 0) return fail(MTMC_ERR_INVALID_ARG, "M, N, K must be positive");
    const size_t xb = static_cast<size_t>(M) * K * 2, wb = static_cast<size_t>(N) * K * 2, ob = static_cast<size_t>(M) * N * 2;
    const HostOperand in[4] = {{X, xb}, {Wg, wb}, {Wu, wb}, {nullptr, 0}};
    return host_call(in, out, ob, blocking, [&](void* const* dev) { return mtmc_swiglu(dev[0], dev[1], dev[2], M, N, K, dev[4]); });
}

int linear_lse_host_impl(const void* X, const void* W, const float* b, int64_t M, int64_t N, int64_t K, float* lse_out, bool blocking) {
    if (!X || !W || !lse_out) return fail(MTMC_ERR_INVALID_ARG, "null pointer argument");
    if (M <= 0 || N <= 0 || K <= 0) return fail(MTMC_ERR_INVALID_ARG, "M, N, K must be positive");
    const size_t xb = static_cast<size_t>(M) * K * 2, wb = static_cast<size_t>(N) * K * 2, bb = static_cast<size_t>(N) * 4;
    const HostOperand in[4] = {{X, xb}, {W, wb}, {nullptr, 0}, {b, bb}};
    return host_call(in, lse_out, static_cast<size_t>(M) * 4, blocking, [&](void* const* dev) {
        return mtmc_linear_lse(dev[0], dev[1], static_cast<const float*>(dev[3]), M, N, K, static_cast<float*>(dev[4]));
    });
}

// ---------------------------------------------------------------------------- block-scaled E4M3 (MXFP8)
struct MxPlan { bool pair; int out_tile_n; int m_blocks, n_blocks, w_atoms, w_rows_per_block; size_t sfa_bytes, sfb_bytes; };
// Large problems go to CTA pairs with 256 x 224 tiles (SwiGLU: 256 x 96); everything else to single-CTA tiles of
// 128 x 128 (SwiGLU: 128 x 64).
MxPlan plan_mx(DeviceState* d, int epi, int64_t M, int64_t N, int64_t K) {
    MxPlan mp{};
    const size_t stages = static_cast<size_t>((K + 127) / 128);
    const int pair_tile_n = epi == EPI_SWIGLU ? 96 : 224;
    mp.pair = d != nullptr && t_cta_pair >= 0 && gemm_pairs(d) > 0 && (t_cta_pair > 0 || (M >= 512 && N >= pair_tile_n));
    if (mp.pair) {
        mp.out_tile_n = pair_tile_n;
        mp.m_blocks = 2 * static_cast<int>((M + 255) / 256);          // one 128-row block of X scales per CTA of a pair
        mp.n_blocks = static_cast<int>((N + pair_tile_n - 1) / pair_tile_n);
        mp.w_atoms = 2; mp.w_rows_per_block = pair_tile_n;            // SwiGLU: 96 gate rows, then the same 96 up rows
    } else {
        mp.out_tile_n = epi == EPI_SWIGLU ? 64 : 128;
        mp.m_blocks = static_cast<int>((M + 127) / 128);
        mp.n_blocks = static_cast<int>((N + mp.out_tile_n - 1) / mp.out_tile_n);
        mp.w_atoms = 1; mp.w_rows_per_block = epi == EPI_SWIGLU ? 64 : 128;
    }
    mp.sfa_bytes = round256(stages * mp.m_blocks * 512);
    mp.sfb_bytes = round256(stages * mp.n_blocks * mp.w_atoms * 512);
    return mp;
}

int check_mx(const void* X8, const void* SX, const void* W8, const void* SW, const void* out, int64_t M, int64_t N, int64_t K) {
    if (!X8 || !SX || !W8 || !SW || !out) return fail(MTMC_ERR_INVALID_ARG, "null pointer argument");
    if (M <= 0 || N <= 0 || K <= 0) return fail(MTMC_ERR_INVALID_ARG, "M, N, K must be positive");
    if (M >= (1ll << 31) || N >= (1ll << 31) || K >= (1ll << 31)) return fail(MTMC_ERR_UNSUPPORTED_SHAPE, "dimensions must be below 2^31");
    if (K % 32 != 0) return fail(MTMC_ERR_UNSUPPORTED_SHAPE, "K = %lld: K must be a multiple of 32, the scale block of the MX formats", (long long)K);
    if (!aligned16(X8) || !aligned16(W8) || !aligned16(out)) return fail(MTMC_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
    return MTMC_OK;
}

template <int EPI, bool OUT_BF16>
int launch_mx(DeviceState* d, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmB2, const uint8_t* sfa,
              const uint8_t* sfb, const GemmParams& p) {
    using Cfg = MxCfg<EPI>;
    auto kern = gemm_mx_kernel<EPI, OUT_BF16>;
    if (int rc = ensure_smem_attr(kern, Cfg::SMEM_BYTES)) return rc;
    const int grid = p.num_tiles < d->sm_count ? p.num_tiles : d->sm_count;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid), 1, 1);
    cfg.blockDim = dim3(Cfg::THREADS, 1, 1);
    cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
    cfg.stream = t_stream;
    cudaLaunchAttribute attr[1];
    cfg.attrs = attr;
    cfg.numAttrs = pdl_attribute(attr);
    CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, tmA, tmB, tmB2, sfa, sfb, p));
    g_launches.fetch_add(1);
    note_kernel("gemm_mx_kernel", EPI);
    return MTMC_OK;
}

template <int EPI, bool OUT_BF16>
int launch_mx_pair(int clusters, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmB2, const CUtensorMap& tmSFA,
                   const CUtensorMap& tmSFB, const GemmParams& p) {
    using Cfg = MxPairCfg<EPI>;
    auto kern = gemm_mx_pair_kernel<EPI, OUT_BF16>;
    if (int rc = ensure_smem_attr(kern, Cfg::SMEM_BYTES)) return rc;
    const int pairs = p.num_tiles < clusters ? p.num_tiles : clusters;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2u * static_cast<unsigned>(pairs), 1, 1);
    cfg.blockDim = dim3(Cfg::THREADS, 1, 1);
    cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
    cfg.stream = t_stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1 + pdl_attribute(attr + 1);
    GemmParams q = p;
    q.trace = trace_for(cfg.gridDim.x);
    CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, tmA, tmB, tmB2, tmSFA, tmSFB, q));
    g_launches.fetch_add(1);
    note_kernel("gemm_mx_pair_kernel", EPI);
    return MTMC_OK;
}

// Scales into the kernels' block layout (two small launches), then the tiled kernel.  EPI_ACT: out / act / out_dtype;
// EPI_SWIGLU: W = gate, W2 = up with their scales; EPI_LSE: lse_out.
template <int EPI>
int run_mx(const void* X8, const void* SX, const void* W8, const void* SW, const void* W28, const void* SW2, const float* b,
           int64_t M, int64_t N, int64_t K, int act, int out_dtype, void* out, float* lse_out) {
    DeviceState* d = nullptr;
    int rc = get_device(&d);
    if (rc) return rc;
    const MxPlan mp = plan_mx(d, EPI, M, N, K);
    GemmParams p{};
    if (mp.pair) fill_tiling(p, M, N, K, mp.out_tile_n, gemm_pairs(d), false, 256, true);
    else fill_tiling(p, M, N, K, mp.out_tile_n, d->sm_count, false, 128, true);
    p.fp8 = 0;                         // the epilogues see plain fp32 accumulators: the scales are applied inside the MMAs
    const size_t lse_bytes = EPI == EPI_LSE ? lse_partial_bytes(p) : 0;
    void* ws = nullptr;
    if ((rc = get_workspace(d, mp.sfa_bytes + mp.sfb_bytes + lse_bytes, &ws))) return rc;
    uint8_t* sfa = static_cast<uint8_t*>(ws);
    uint8_t* sfb = sfa + mp.sfa_bytes;
    p.act = act; p.bias = b; p.out = out; p.status = d->status;
    p.lse_partial = EPI == EPI_LSE ? reinterpret_cast<float2*>(sfb + mp.sfb_bytes) : nullptr;
    CUtensorMap tmA, tmB, tmB2;
    const int w_box = mp.pair ? (EPI == EPI_SWIGLU ? 96 : 112) : mp.out_tile_n;
    if ((rc = encode_u8_2d(&tmA, X8, M, K, 128)) || (rc = encode_u8_2d(&tmB, W8, N, K, w_box)) ||
        (rc = encode_u8_2d(&tmB2, EPI == EPI_SWIGLU ? W28 : W8, N, K, w_box)))
        return rc;
    const int kb32 = static_cast<int>(K / 32);
    TimedRegion tr(d);
    {
        const long long total_a = static_cast<long long>(p.k_blocks) * mp.m_blocks * 512, total_b = static_cast<long long>(p.k_blocks) * mp.n_blocks * mp.w_atoms * 512;
        const unsigned ga = static_cast<unsigned>(std::min<long long>((total_a + 255) / 256, 4096)), gb = static_cast<unsigned>(std::min<long long>((total_b + 255) / 256, 4096));
        mx_retile_scales_kernel<<<ga, 256, 0, t_stream>>>(static_cast<const uint8_t*>(SX), nullptr, static_cast<int>(M), kb32, mp.m_blocks, p.k_blocks, 128, 1, sfa);
        mx_retile_scales_kernel<<<gb, 256, 0, t_stream>>>(static_cast<const uint8_t*>(SW), EPI == EPI_SWIGLU ? static_cast<const uint8_t*>(SW2) : nullptr,
                                                          static_cast<int>(N), kb32, mp.n_blocks, p.k_blocks, mp.w_rows_per_block, mp.w_atoms, sfb);
        CUDA_TRY(cudaGetLastError());
        g_launches.fetch_add(2);
    }
    if (mp.pair) {
        CUtensorMap tmSFA, tmSFB;
        if ((rc = encode_bytes_2d(&tmSFA, sfa, static_cast<int64_t>(p.k_blocks) * mp.m_blocks * 2, 2)) ||
            (rc = encode_bytes_2d(&tmSFB, sfb, static_cast<int64_t>(p.k_blocks) * mp.n_blocks * 4, 4)))
            return rc;
        if (EPI == EPI_ACT) rc = out_dtype == MTMC_OUT_BF16 ? launch_mx_pair<EPI_ACT, true>(gemm_pairs(d), tmA, tmB, tmB2, tmSFA, tmSFB, p)
                                                           : launch_mx_pair<EPI_ACT, false>(gemm_pairs(d), tmA, tmB, tmB2, tmSFA, tmSFB, p);
        else if (EPI == EPI_SWIGLU) rc = launch_mx_pair<EPI_SWIGLU, true>(gemm_pairs(d), tmA, tmB, tmB2, tmSFA, tmSFB, p);
        else rc = launch_mx_pair<EPI_LSE, false>(gemm_pairs(d), tmA, tmB, tmB2, tmSFA, tmSFB, p);
    } else if (EPI == EPI_ACT) rc = out_dtype == MTMC_OUT_BF16 ? launch_mx<EPI_ACT, true>(d, tmA, tmB, tmB2, sfa, sfb, p) : launch_mx<EPI_ACT, false>(d, tmA, tmB, tmB2, sfa, sfb, p);
    else if (EPI == EPI_SWIGLU) rc = launch_mx<EPI_SWIGLU, true>(d, tmA, tmB, tmB2, sfa, sfb, p);
    else rc = launch_mx<EPI_LSE, false>(d, tmA, tmB, tmB2, sfa, sfb, p);
    tr.stop();
    if (rc) return rc;
    if (EPI == EPI_LSE) {
        return launch_follow_up(lse_merge_rows_kernel, dim3(static_cast<unsigned>((M + 31) / 32), 1, 1), 32u * MERGE_WARPS,
                                static_cast<const float2*>(p.lse_partial), p.M, p.rows_per_tile, p.m_tiles, p.n_tiles, p.group_m, p.n_full,
                                p.tail_split, lse_out, static_cast<const float*>(nullptr), static_cast<float*>(nullptr));
    }
    return MTMC_OK;
}

}  // namespace

extern "C" {

int mtmc_version(void) { return 100; }

int mtmc_set_stream(void* cuda_stream) {
    t_stream = static_cast<cudaStream_t>(cuda_stream);
    return MTMC_OK;
}

int mtmc_set_workspace(void* dptr, size_t bytes) {
    if (dptr == nullptr) { t_user_ws = nullptr; t_user_ws_bytes = 0; return MTMC_OK; }
    if ((reinterpret_cast<uintptr_t>(dptr) & 255u) != 0) return fail(MTMC_ERR_INVALID_ARG, "workspace must be 256-byte aligned");
    t_user_ws = dptr;
    t_user_ws_bytes = bytes;
    return MTMC_OK;
}

int mtmc_set_tuning(int split_k, int tile_n, int cta_pair) {
    if (tile_n > 0 && tile_n != 128 && tile_n != 256) return fail(MTMC_ERR_INVALID_ARG, "tile_n must be 128 or 256");
    t_split_k = split_k > 0 ? split_k : 0;
    t_tile_n = tile_n > 0 ? tile_n : 0;
    t_cta_pair = cta_pair > 1 ? 2 : (cta_pair > 0 ? 1 : (cta_pair < 0 ? -1 : 0));
    return MTMC_OK;
}

int mtmc_trace_enabled(void) {
#ifdef MTMC_TRACE
    return 1;
#else
    return 0;
#endif
}

int mtmc_set_trace(void* dptr, size_t bytes) {
    if (dptr != nullptr && !mtmc_trace_enabled())
        return fail(MTMC_ERR_INVALID_ARG, "this build of the library has no device-side trace (compile with -DMTMC_TRACE)");
    if (dptr != nullptr && (reinterpret_cast<uintptr_t>(dptr) & 7u)) return fail(MTMC_ERR_INVALID_ARG, "trace buffer must be 8-byte aligned");
    t_trace = static_cast<unsigned long long*>(dptr);
    t_trace_bytes = dptr ? bytes : 0;
    return MTMC_OK;
}

int mtmc_set_schedule(int stream_k) {
    t_stream_k = stream_k > 0 ? 1 : (stream_k < 0 ? -1 : 0);
    return MTMC_OK;
}

int mtmc_set_static_weights(int enabled) { t_static_weights = enabled ? 1 : 0; return MTMC_OK; }

int mtmc_set_timing(int enabled) { t_timing = enabled ? 1 : 0; return MTMC_OK; }

float mtmc_last_kernel_ms(void) {
    DeviceState* d = nullptr;
    DeviceState::StreamScratch* sc = nullptr;
    if (get_device(&d) != MTMC_OK || get_stream_scratch(d, &sc) != MTMC_OK || !sc->timed) return -1.0f;
    if (cudaEventSynchronize(sc->ev1) != cudaSuccess) return -1.0f;
    float ms = -1.0f;
    if (cudaEventElapsedTime(&ms, sc->ev0, sc->ev1) != cudaSuccess) return -1.0f;
    return ms;
}

int64_t mtmc_launch_count(void) { return g_launches.load(); }

const char* mtmc_last_error(void) { return t_error; }

const char* mtmc_last_kernel_name(void) { return t_last_kernel; }

size_t mtmc_workspace_bytes(int op, int64_t M, int64_t N, int64_t K) {
    if (M <= 0 || N <= 0 || K <= 0) return static_cast<size_t>(-1);
    if (op < MTMC_OP_FUSED_LINEAR || op > MTMC_OP_LINEAR_SOFTMAX) return static_cast<size_t>(-1);
    if (op >= MTMC_OP_FUSED_LINEAR_MXFP8 && op <= MTMC_OP_LINEAR_LSE_MXFP8) {      // the re-arranged scales (+ the logsumexp partials of 128-column tiles, the most pieces)
        DeviceState* dm = nullptr;
        if (get_device(&dm) != MTMC_OK) return static_cast<size_t>(-1);
        const MxPlan mp = plan_mx(dm, op == MTMC_OP_SWIGLU_MXFP8 ? EPI_SWIGLU : (op == MTMC_OP_LINEAR_LSE_MXFP8 ? EPI_LSE : EPI_ACT), M, N, K);
        const size_t lse = op == MTMC_OP_LINEAR_LSE_MXFP8 ? round256(static_cast<size_t>((N + 127) / 128) * EPI_HALVES * static_cast<size_t>(M) * sizeof(float2)) : 0;
        return mp.sfa_bytes + mp.sfb_bytes + lse;
    }
    DeviceState* d = nullptr;
    if (get_device(&d) != MTMC_OK) return static_cast<size_t>(-1);
    // An upper bound over the kernels the library may pick for the shape under the current tuning: the stream-K
    // region of the pair kernel wherever CTA pairs are possible (whether or not this shape ends up on that schedule).
    const bool pairs_possible = gemm_pairs(d) > 0 && t_stream_k > 0 && t_cta_pair >= 0 && t_tile_n != 128 &&
                                (t_cta_pair > 0 || (M > 128 && N >= 256));
    const size_t sk = pairs_possible ? streamk_bytes(gemm_pairs(d)) : 0;
    switch (op) {
        case MTMC_OP_FUSED_LINEAR: {
            if (!skinny_possible(M, N)) return sk;
            // the larger of the bf16 and the E4M3 plan: mtmc_fused_linear_fp8 shares this op id
            SkinnyPlan s = plan_skinny(d->sm_count, skinny_pairs(d), M, N, K);
            SkinnyPlan s8 = plan_skinny(d->sm_count, skinny_pairs(d), M, N, K, 128);
            return std::max(s.ticket_bytes + s.partial_bytes, s8.ticket_bytes + s8.partial_bytes);
        }
        case MTMC_OP_SWIGLU: return sk;
        case MTMC_OP_LINEAR_LSE: return lse_workspace_bytes(M, N) + sk;
        case MTMC_OP_LINEAR_ROWMAX: return lse_workspace_bytes(M, N) + sk;
        default: return lse_workspace_bytes(M, N) + round256(static_cast<size_t>(M) * sizeof(float)) + sk;
    }
}

int mtmc_selftest_timeout(void) {
    DeviceState* d = nullptr;
    int rc = get_device(&d);
    if (rc) return rc;
    timeout_probe_kernel<<<1, 32, 0, t_stream>>>(d->status);
    CUDA_TRY(cudaGetLastError());
    g_launches.fetch_add(1);
    return MTMC_OK;
}

int mtmc_check_status(void) {
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= MAX_DEVICES) return fail(MTMC_ERR_UNSUPPORTED_DEVICE, "device index %d out of range", dev);
    bool regular = false, noalloc = false;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        regular = g_dev[dev].ready;
    }
    noalloc = noalloc_in_use(dev);
    CUDA_TRY(cudaStreamSynchronize(t_stream));
    uint32_t st = 0, st_noalloc = 0;
    // A process that has only ever used the allocation-free entry point on this device stays allocation-free:
    // the regular per-device state (which owns device memory) is not created just to be found clean.
    if (regular || !noalloc) {
        DeviceState* d = nullptr;
        if (int rc = get_device(&d)) return rc;
        CUDA_TRY(cudaMemcpy(&st, d->status, sizeof st, cudaMemcpyDeviceToHost));
        if (st != 0) CUDA_TRY(cudaMemset(d->status, 0, sizeof st));
    }
    if (noalloc) {
        if (int rc = noalloc_take_status(dev, &st_noalloc)) return rc;
    }
    if (st == 0) st = st_noalloc;
    if ((st & 0xff00u) == STATUS_CHECK_FAILED)
        return fail(MTMC_ERR_DEVICE_CHECK, "a device-side index check of the -DMTMC_CHECKS build failed (status word 0x%x)", st);
    if (st != 0) return fail(MTMC_ERR_DEVICE_TIMEOUT, "a bounded device-side wait expired (status word 0x%x)", st);
    return MTMC_OK;
}

int64_t mtmc_device_alloc_count(void) { return g_device_allocs.load(); }

int mtmc_fused_linear(const void* X, const void* W, const float* b, int64_t M, int64_t N, int64_t K, int act,
                      int out_dtype, void* out) {
    return fused_linear_impl(X, W, b, nullptr, M, N, K, act, out_dtype, out);
}

int mtmc_fused_linear_residual(const void* X, const void* W, const float* b, const void* R, int64_t M, int64_t N,
                               int64_t K, int act, int out_dtype, void* out) {
    if (!R) return fail(MTMC_ERR_INVALID_ARG, "null pointer argument");
    if (!aligned16(R)) return fail(MTMC_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
    return fused_linear_impl(X, W, b, R, M, N, K, act, out_dtype, out);
}

int mtmc_fused_linear_strided(const void* X, int64_t ldx, const void* W, int64_t ldw, const float* b, int64_t M, int64_t N,
                              int64_t K, int act, int out_dtype, void* out, int64_t ldo) {
    if (ldx < K || ldw < K || ldo < N) return fail(MTMC_ERR_INVALID_ARG, "row pitches must cover the rows (ldx, ldw >= K, ldo >= N)");
    if (ldx % 8 != 0 || ldw % 8 != 0) return fail(MTMC_ERR_UNSUPPORTED_SHAPE, "ldx and ldw must be multiples of 8 elements (16-byte rows for TMA)");
    if (ldx >= (1ll << 31) || ldw >= (1ll << 31) || ldo >= (1ll << 31)) return fail(MTMC_ERR_UNSUPPORTED_SHAPE, "row pitches must be below 2^31");
    return fused_linear_impl(X, W, b, nullptr, M, N, K, act, out_dtype, out, ldx, ldw, ldo);
}

int mtmc_fused_linear_fp8(const void* X8, const void* W8, const float* b, float scale_x, float scale_w, int64_t M, int64_t N,
                          int64_t K, int act, int out_dtype, void* out) {
    if (!X8 || !W8 || !out) return fail(MTMC_ERR_INVALID_ARG, "null pointer argument");
    if (M <= 0 || N <= 0 || K <= 0) return fail(MTMC_ERR_INVALID_ARG, "M, N, K must be positive");
    if (M >= (1ll << 31) || N >= (1ll << 31) || K >= (1ll << 31)) return fail(MTMC_ERR_UNSUPPORTED_SHAPE, "dimensions must be below 2^31");
    if (K % 16 != 0) return fail(MTMC_ERR_UNSUPPORTED_SHAPE, "K = %lld: K must be a multiple of 16 for one-byte operands (16-byte rows for TMA)", (long long)K);
    if (!aligned16(X8) || !aligned16(W8) || !aligned16(out) || (b && !aligned16(b))) return fail(MTMC_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
    if (act < 0 || act > 3) return fail(MTMC_ERR_INVALID_ARG, "unknown activation id %d", act);
    if (out_dtype != MTMC_OUT_FP32 && out_dtype != MTMC_OUT_BF16) return fail(MTMC_ERR_INVALID_ARG, "unknown output type id %d", out_dtype);
    DeviceState* d = nullptr;
    int rc = get_device(&d);
    if (rc) return rc;
    if (prefer_skinny(d, M, N)) return run_skinny(d, X8, W8, b, nullptr, M, N, K, act, out_dtype, out, true, scale_x * scale_w);
    if (const int ks = pick_ksplit_act(d, M, N, K, true)) {
        GemmParams p{};
        const int bn = ks < 0 ? 128 : 256;
        fill_ksplit(p, M, N, K, bn, ks < 0 ? -ks : ks, true);
        p.acc_scale = scale_x * scale_w;
        p.act = act; p.bias = b; p.residual = nullptr; p.out = out; p.lse_partial = nullptr; p.status = d->status;
        CUtensorMap tmA, tmB;
        if ((rc = encode_u8_2d(&tmA, X8, M, K, 128)) || (rc = encode_u8_2d(&tmB, W8, N, K, bn))) return rc;
        TimedRegion tr(d);
        rc = out_dtype == MTMC_OUT_BF16 ? launch_ksplit<EPI_ACT, true>(ks, tmA, tmB, tmB, p) : launch_ksplit<EPI_ACT, false>(ks, tmA, tmB, tmB, p);
        tr.stop();
        return rc;
    }
    if (skinny_possible(M, N) && t_tile_n == 0 && t_cta_pair <= 0)
        return run_skinny(d, X8, W8, b, nullptr, M, N, K, act, out_dtype, out, true, scale_x * scale_w);
    if (use_big(d, M, N, K, true)) {
        GemmParams p{};
        fill_tiling(p, M, N, K, 256, gemm_pairs(d), false, 512, true);
        p.acc_scale = scale_x * scale_w;
        p.act = act; p.bias = b; p.residual = nullptr; p.out = out; p.lse_partial = nullptr; p.status = d->status;
        CUtensorMap tmA, tmB;
        if ((rc = encode_u8_2d(&tmA, X8, M, K, 256)) || (rc = encode_u8_2d(&tmB, W8, N, K, 128))) return rc;
        TimedRegion tr(d);
        rc = out_dtype == MTMC_OUT_BF16 ? launch_big<EPI_ACT, true>(gemm_pairs(d), tmA, tmB, tmB, p)
                                        : launch_big<EPI_ACT, false>(gemm_pairs(d), tmA, tmB, tmB, p);
        tr.stop();
        return rc;
    }
    const bool pair = use_pair(d, M, N, K);
    const int bn = pair ? 256 : pick_tile_n(N);
    GemmParams p{};
    if (pair) {
        const bool sk = plan_pair(d, p, M, N, K, 256, true);
        if ((rc = pair_scratch(d, p, sk))) return rc;
    } else {
        fill_tiling(p, M, N, K, bn, d->sm_count, true, 128, true);
    }
    p.acc_scale = scale_x * scale_w;
    p.act = act; p.bias = b; p.residual = nullptr; p.out = out; p.lse_partial = nullptr; p.status = d->status;
    CUtensorMap tmA, tmB, tmBt;
    if ((rc = encode_u8_2d(&tmA, X8, M, K, 128)) || (rc = encode_u8_2d(&tmB, W8, N, K, pair ? 128 : bn)) ||
        (rc = encode_u8_2d(&tmBt, W8, N, K, pair ? p.tail_width / 2 : p.tail_width)))
        return rc;
    const bool bf = out_dtype == MTMC_OUT_BF16;
    TimedRegion tr(d);
    if (pair) rc = bf ? launch_pair<EPI_ACT, true>(gemm_pairs(d), tmA, tmB, tmB, tmBt, tmBt, p)
                      : launch_pair<EPI_ACT, false>(gemm_pairs(d), tmA, tmB, tmB, tmBt, tmBt, p);
    else if (bn == 256) rc = bf ? launch_tiled<EPI_ACT, 256, true>(d, tmA, tmB, tmB, tmBt, tmBt, p)
                                : launch_tiled<EPI_ACT, 256, false>(d, tmA, tmB, tmB, tmBt, tmBt, p);
    else rc = bf ? launch_tiled<EPI_ACT, 128, true>(d, tmA, tmB, tmB, tmBt, tmBt, p)
                 : launch_tiled<EPI_ACT, 128, false>(d, tmA, tmB, tmB, tmBt, tmBt, p);
    tr.stop();
    return rc;
}

int mtmc_fused_linear_mxfp8(const void* X8, const void* SX, const void* W8, const void* SW, const float* b, int64_t M, int64_t N, int64_t K,
                            int act, int out_dtype, void* out) {
    int rc = check_mx(X8, SX, W8, SW, out, M, N, K);
    if (rc) return rc;
    if (act < 0 || act > 3) return fail(MTMC_ERR_INVALID_ARG, "unknown activation id %d", act);
    if (out_dtype != MTMC_OUT_FP32 && out_dtype != MTMC_OUT_BF16) return fail(MTMC_ERR_INVALID_ARG, "unknown output type id %d", out_dtype);
    if (b && !aligned16(b)) return fail(MTMC_ERR_INVALID_ARG, "bias must be 16-byte aligned");
    return run_mx<EPI_ACT>(X8, SX, W8, SW, nullptr, nullptr, b, M, N, K, act, out_dtype, out, nullptr);
}

int mtmc_swiglu_mxfp8(const void* X8, const void* SX, const void* Wg8, const void* SG, const void* Wu8, const void* SU, int64_t M, int64_t N,
                      int64_t K, void* out) {
    int rc = check_mx(X8, SX, Wg8, SG, out, M, N, K);
    if (rc) return rc;
    if (!Wu8 || !SU) return fail(MTMC_ERR_INVALID_ARG, "null pointer argument");
    if (!aligned16(Wu8)) return fail(MTMC_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
    return run_mx<EPI_SWIGLU>(X8, SX, Wg8, SG, Wu8, SU, nullptr, M, N, K, ACT_NONE, MTMC_OUT_BF16, out, nullptr);
}

int mtmc_linear_lse_mxfp8(const void* X8, const void* SX, const void* W8, const void* SW, const float* b, int64_t M, int64_t N, int64_t K,
                          float* lse_out) {
    int rc = check_mx(X8, SX, W8, SW, lse_out, M, N, K);
    if (rc) return rc;
    if (b && !aligned16(b)) return fail(MTMC_ERR_INVALID_ARG, "bias must be 16-byte aligned");
    return run_mx<EPI_LSE>(X8, SX, W8, SW, nullptr, nullptr, b, M, N, K, ACT_NONE, MTMC_OUT_FP32, nullptr, lse_out);
}

int mtmc_swiglu(const void* X, const void* Wg, const void* Wu, int64_t M, int64_t N, int64_t K, void* out) {
    return swiglu_impl(X, Wg, Wu, M, N, K, out, false, 1.0f, 1.0f);
}

int mtmc_swiglu_strided(const void* X, int64_t ldx, const void* Wg, int64_t ldwg, const void* Wu, int64_t ldwu, int64_t M, int64_t N,
                        int64_t K, void* out, int64_t ldo) {
    if (ldx < K || ldwg < K || ldwu < K || ldo < N) return fail(MTMC_ERR_INVALID_ARG, "row pitches must cover the rows (ldx, ldwg, ldwu >= K, ldo >= N)");
    if (ldx % 8 != 0 || ldwg % 8 != 0 || ldwu % 8 != 0)
        return fail(MTMC_ERR_UNSUPPORTED_SHAPE, "ldx, ldwg and ldwu must be multiples of 8 elements (16-byte rows for TMA)");
    if (ldx >= (1ll << 31) || ldwg >= (1ll << 31) || ldwu >= (1ll << 31) || ldo >= (1ll << 31)) return fail(MTMC_ERR_UNSUPPORTED_SHAPE, "row pitches must be below 2^31");
    return swiglu_impl(X, Wg, Wu, M, N, K, out, false, 1.0f, 1.0f, ldx, ldwg, ldwu, ldo);
}

int mtmc_swiglu_fp8(const void* X8, const void* Wg8, const void* Wu8, float scale_x, float scale_g, float scale_u,
                    int64_t M, int64_t N, int64_t K, void* out) {
    if (K % 16 != 0) return fail(MTMC_ERR_UNSUPPORTED_SHAPE, "K = %lld: K must be a multiple of 16 for E4M3 operands", (long long)K);
    return swiglu_impl(X8, Wg8, Wu8, M, N, K, out, true, scale_x * scale_g, scale_x * scale_u);
}

int mtmc_linear_lse(const void* X, const void* W, const float* b, int64_t M, int64_t N, int64_t K, float* lse_out) {
    int rc = check_common(X, W, lse_out, M, N, K);
    if (rc) return rc;
    return run_row_reduction<EPI_LSE>(X, W, b, nullptr, M, N, K, lse_out, nullptr, nullptr);
}

namespace {
int check_row_pitches(int64_t ldx, int64_t ldw, int64_t K) {
    if (ldx < K || ldw < K) return fail(MTMC_ERR_INVALID_ARG, "row pitches must cover the rows (ldx, ldw >= K)");
    if (ldx % 8 != 0 || ldw % 8 != 0) return fail(MTMC_ERR_UNSUPPORTED_SHAPE, "ldx and ldw must be multiples of 8 elements (16-byte rows for TMA)");
    if (ldx >= (1ll << 31) || ldw >= (1ll << 31)) return fail(MTMC_ERR_UNSUPPORTED_SHAPE, "row pitches must be below 2^31");
    return MTMC_OK;
}
}  // namespace

int mtmc_linear_lse_strided(const void* X, int64_t ldx, const void* W, int64_t ldw, const float* b, int64_t M, int64_t N, int64_t K,
                            float* lse_out) {
    int rc = check_common(X, W, lse_out, M, N, K);
    if (rc || (rc = check_row_pitches(ldx, ldw, K))) return rc;
    return run_row_reduction<EPI_LSE>(X, W, b, nullptr, M, N, K, lse_out, nullptr, nullptr, false, 1.0f, ldx, ldw);
}

int mtmc_linear_rowmax_strided(const void* X, int64_t ldx, const void* W, int64_t ldw, const float* b, int64_t M, int64_t N, int64_t K,
                               float* max_out, int32_t* argmax_out) {
    int rc = check_common(X, W, max_out, M, N, K);
    if (rc || (rc = check_row_pitches(ldx, ldw, K))) return rc;
    if (argmax_out && (reinterpret_cast<uintptr_t>(argmax_out) & 3u)) return fail(MTMC_ERR_INVALID_ARG, "argmax_out must be 4-byte aligned");
    return run_row_reduction<EPI_ROWMAX>(X, W, b, nullptr, M, N, K, max_out, nullptr, argmax_out, false, 1.0f, ldx, ldw);
}

int mtmc_linear_cross_entropy_strided(const void* X, int64_t ldx, const void* W, int64_t ldw, const float* b, const int64_t* targets,
                                      int64_t M, int64_t N, int64_t K, float* loss_out, float* lse_out) {
    int rc = check_common(X, W, loss_out, M, N, K);
    if (rc || (rc = check_row_pitches(ldx, ldw, K))) return rc;
    if (!targets) return fail(MTMC_ERR_INVALID_ARG, "null pointer argument");
    if (reinterpret_cast<uintptr_t>(targets) & 7u) return fail(MTMC_ERR_INVALID_ARG, "targets must be 8-byte aligned");
    return run_row_reduction<EPI_XENT>(X, W, b, targets, M, N, K, lse_out, loss_out, nullptr, false, 1.0f, ldx, ldw);
}

int mtmc_linear_lse_fp8(const void* X8, const void* W8, const float* b, float scale_x, float scale_w, int64_t M, int64_t N,
                        int64_t K, float* lse_out) {
    if (K % 16 != 0) return fail(MTMC_ERR_UNSUPPORTED_SHAPE, "K = %lld: K must be a multiple of 16 for E4M3 operands", (long long)K);
    int rc = check_common(X8, W8, lse_out, M, N, K);
    if (rc) return rc;
    return run_row_reduction<EPI_LSE>(X8, W8, b, nullptr, M, N, K, lse_out, nullptr, nullptr, true, scale_x * scale_w);
}

int mtmc_linear_rowmax(const void* X, const void* W, const float* b, int64_t M, int64_t N, int64_t K, float* max_out,
                       int32_t* argmax_out) {
    int rc = check_common(X, W, max_out, M, N, K);
    if (rc) return rc;
    if (argmax_out && (reinterpret_cast<uintptr_t>(argmax_out) & 3u)) return fail(MTMC_ERR_INVALID_ARG, "argmax_out must be 4-byte aligned");
    return run_row_reduction<EPI_ROWMAX>(X, W, b, nullptr, M, N, K, max_out, nullptr, argmax_out);
}

int mtmc_linear_cross_entropy(const void* X, const void* W, const float* b, const int64_t* targets, int64_t M, int64_t N,
                              int64_t K, float* loss_out, float* lse_out) {
    int rc = check_common(X, W, loss_out, M, N, K);
    if (rc) return rc;
    if (!targets) return fail(MTMC_ERR_INVALID_ARG, "null pointer argument");
    if (reinterpret_cast<uintptr_t>(targets) & 7u) return fail(MTMC_ERR_INVALID_ARG, "targets must be 8-byte aligned");
    return run_row_reduction<EPI_XENT>(X, W, b, targets, M, N, K, lse_out, loss_out, nullptr);
}

namespace {
int check_softmax(int64_t N, int out_dtype, const float* lse_out) {
    if (out_dtype != MTMC_OUT_FP32 && out_dtype != MTMC_OUT_BF16) return fail(MTMC_ERR_INVALID_ARG, "unknown output type id %d", out_dtype);
    if (N >= (1ll << 31) - 1024) return fail(MTMC_ERR_UNSUPPORTED_SHAPE, "N = %lld: N must be below 2^31 - 1024", (long long)N);
    if (lse_out && (reinterpret_cast<uintptr_t>(lse_out) & 3u)) return fail(MTMC_ERR_INVALID_ARG, "lse_out must be 4-byte aligned");
    return MTMC_OK;
}
}  // namespace

int mtmc_linear_softmax(const void* X, const void* W, const float* b, int64_t M, int64_t N, int64_t K, int out_dtype,
                        void* prob_out, float* lse_out) {
    int rc = check_common(X, W, prob_out, M, N, K);
    if (rc || (rc = check_softmax(N, out_dtype, lse_out))) return rc;
    return run_row_reduction<EPI_SOFTMAX>(X, W, b, nullptr, M, N, K, lse_out, nullptr, nullptr, false, 1.0f, 0, 0, prob_out, out_dtype);
}

int mtmc_linear_softmax_strided(const void* X, int64_t ldx, const void* W, int64_t ldw, const float* b, int64_t M, int64_t N, int64_t K,
                                int out_dtype, void* prob_out, int64_t ldo, float* lse_out) {
    int rc = check_common(X, W, prob_out, M, N, K);
    if (rc || (rc = check_row_pitches(ldx, ldw, K)) || (rc = check_softmax(N, out_dtype, lse_out))) return rc;
    if (ldo < N) return fail(MTMC_ERR_INVALID_ARG, "row pitches must cover the rows (ldo >= N)");
    if (ldo >= (1ll << 31)) return fail(MTMC_ERR_UNSUPPORTED_SHAPE, "row pitches must be below 2^31");
    return run_row_reduction<EPI_SOFTMAX>(X, W, b, nullptr, M, N, K, lse_out, nullptr, nullptr, false, 1.0f, ldx, ldw, prob_out, out_dtype, ldo);
}

int mtmc_linear_softmax_fp8(const void* X8, const void* W8, const float* b, float scale_x, float scale_w, int64_t M, int64_t N,
                            int64_t K, int out_dtype, void* prob_out, float* lse_out) {
    if (K % 16 != 0) return fail(MTMC_ERR_UNSUPPORTED_SHAPE, "K = %lld: K must be a multiple of 16 for E4M3 operands", (long long)K);
    int rc = check_common(X8, W8, prob_out, M, N, K);
    if (rc || (rc = check_softmax(N, out_dtype, lse_out))) return rc;
    return run_row_reduction<EPI_SOFTMAX>(X8, W8, b, nullptr, M, N, K, lse_out, nullptr, nullptr, true, scale_x * scale_w, 0, 0, prob_out, out_dtype);
}

int mtmc_linear_rowmax_fp8(const void* X8, const void* W8, const float* b, float scale_x, float scale_w, int64_t M, int64_t N,
                           int64_t K, float* max_out, int32_t* argmax_out) {
    if (K % 16 != 0) return fail(MTMC_ERR_UNSUPPORTED_SHAPE, "K = %lld: K must be a multiple of 16 for E4M3 operands", (long long)K);
    int rc = check_common(X8, W8, max_out, M, N, K);
    if (rc) return rc;
    if (argmax_out && (reinterpret_cast<uintptr_t>(argmax_out) & 3u)) return fail(MTMC_ERR_INVALID_ARG, "argmax_out must be 4-byte aligned");
    return run_row_reduction<EPI_ROWMAX>(X8, W8, b, nullptr, M, N, K, max_out, nullptr, argmax_out, true, scale_x * scale_w);
}

int mtmc_linear_cross_entropy_fp8(const void* X8, const void* W8, const float* b, float scale_x, float scale_w,
                                  const int64_t* targets, int64_t M, int64_t N, int64_t K, float* loss_out, float* lse_out) {
    if (K % 16 != 0) return fail(MTMC_ERR_UNSUPPORTED_SHAPE, "K = %lld: K must be a multiple of 16 for E4M3 operands", (long long)K);
    int rc = check_common(X8, W8, loss_out, M, N, K);
    if (rc) return rc;
    if (!targets) return fail(MTMC_ERR_INVALID_ARG, "null pointer argument");
    if (reinterpret_cast<uintptr_t>(targets) & 7u) return fail(MTMC_ERR_INVALID_ARG, "targets must be 8-byte aligned");
    return run_row_reduction<EPI_XENT>(X8, W8, b, targets, M, N, K, lse_out, loss_out, nullptr, true, scale_x * scale_w);
}

}  // extern "C"

// ---------------------------------------------------------------------------- allocation-free variant
// Scratch for mtmc_linear_lse_noalloc: the per-(column tile, row) (max, sum-exp)
// partials and a status word live in the library image itself.  Every GPU that loads
// the library carries these 8 MiB until the process exits.  In host code the names
// below are host-side stand-ins, not device addresses; the device addresses are
// fetched once per device with cudaGetSymbolAddress and cached.
constexpr size_t NOALLOC_MAX_PARTIALS = (1u << 20) * EPI_HALVES;   // float2 entries = 8 MiB with one epilogue warp per quadrant
static __device__ __align__(256) float2 g_noalloc_partials[NOALLOC_MAX_PARTIALS];
static __device__ __align__(256) uint32_t g_noalloc_status[64];

namespace {
struct NoAllocDevice {
    bool ready = false;
    int sm_count = 0;
    float2* partials = nullptr;   // device address of g_noalloc_partials on this device
    uint32_t* status = nullptr;   // device address of g_noalloc_status on this device
};
NoAllocDevice g_noalloc_dev[MAX_DEVICES];

// One-time set-up for the current device.  Queries attributes and symbol addresses only.
int noalloc_device(NoAllocDevice** out) {
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= MAX_DEVICES) return fail(MTMC_ERR_UNSUPPORTED_DEVICE, "device index %d out of range", dev);
    std::lock_guard<std::mutex> lock(g_mutex);
    NoAllocDevice& d = g_noalloc_dev[dev];
    if (!d.ready) {
        int major = 0, minor = 0;
        CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
        CUDA_TRY(cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev));
        if (major != 10)
            return fail(MTMC_ERR_UNSUPPORTED_DEVICE, "compute capability %d.%d: this library only runs on 10.x (B200)", major, minor);
        CUDA_TRY(cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev));
        if (!g_encode) {
            void* fn = nullptr;
            cudaDriverEntryPointQueryResult qres;
            CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
            if (!fn || qres != cudaDriverEntryPointSuccess)
                return fail(MTMC_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
            g_encode = reinterpret_cast<EncodeTiledFn>(fn);
        }
        void* ptr = nullptr;
        CUDA_TRY(cudaGetSymbolAddress(&ptr, g_noalloc_partials));
        d.partials = static_cast<float2*>(ptr);
        CUDA_TRY(cudaGetSymbolAddress(&ptr, g_noalloc_status));
        d.status = static_cast<uint32_t*>(ptr);
        uint32_t zero = 0;
        CUDA_TRY(cudaMemcpy(d.status, &zero, sizeof zero, cudaMemcpyHostToDevice));
        d.ready = true;
    }
    *out = &d;
    return MTMC_OK;
}

bool noalloc_in_use(int dev) {
    std::lock_guard<std::mutex> lock(g_mutex);
    return g_noalloc_dev[dev].ready;
}

int noalloc_take_status(int dev, uint32_t* st) {
    *st = 0;
    uint32_t* word = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        if (g_noalloc_dev[dev].ready) word = g_noalloc_dev[dev].status;
    }
    if (!word) return MTMC_OK;
    CUDA_TRY(cudaMemcpy(st, word, sizeof *st, cudaMemcpyDeviceToHost));
    if (*st != 0) {
        uint32_t zero = 0;
        CUDA_TRY(cudaMemcpy(word, &zero, sizeof zero, cudaMemcpyHostToDevice));
    }
    return MTMC_OK;
}

template <int BN>
int launch_lse_noalloc(NoAllocDevice* d, const CUtensorMap& tmA, const CUtensorMap& tmB, GemmParams p) {
    using Cfg = TileCfg<EPI_LSE, BN>;
    auto kern = gemm_tiled_kernel<EPI_LSE, BN, false>;
    if (int rc = ensure_smem_attr(kern, Cfg::SMEM_BYTES)) return rc;       // a function attribute, set once per device: no allocation
    const int grid = p.num_tiles < d->sm_count ? p.num_tiles : d->sm_count;
    kern<<<grid, Cfg::THREADS, Cfg::SMEM_BYTES, t_stream>>>(tmA, tmB, tmB, tmB, tmB, p);
    CUDA_TRY(cudaGetLastError());
    g_launches.fetch_add(1);
    note_kernel("gemm_tiled_kernel", EPI_LSE, BN);
    return MTMC_OK;
}
}  // namespace

extern "C" int mtmc_linear_lse_noalloc(const void* X, const void* W, const float* b, int64_t M, int64_t N, int64_t K,
                                       float* lse_out) {
    int rc = check_common(X, W, lse_out, M, N, K);
    if (rc) return rc;
    if (b && !aligned16(b)) return fail(MTMC_ERR_INVALID_ARG, "bias must be 16-byte aligned");
    NoAllocDevice* d = nullptr;
    rc = noalloc_device(&d);
    if (rc) return rc;
    const int bn = pick_tile_n(N);
    GemmParams p{};
    fill_tiling(p, M, N, K, bn, d->sm_count, false);      // whole tiles only: one partial per column tile
    const size_t need = EPI_HALVES * static_cast<size_t>(p.n_tiles) * static_cast<size_t>(M);
    if (need > NOALLOC_MAX_PARTIALS)
        return fail(MTMC_ERR_UNSUPPORTED_SHAPE,
                    "mtmc_linear_lse_noalloc: ceil(N/%d) * M = %zu partials exceed the built-in scratch of %zu "
                    "(8 MiB); use mtmc_linear_lse for this shape", bn, need, NOALLOC_MAX_PARTIALS);
    p.act = ACT_NONE; p.bias = b; p.out = nullptr; p.lse_partial = d->partials; p.status = d->status;
    CUtensorMap tmA, tmB;
    rc = encode_bf16_2d(&tmA, X, M, K, 128);
    if (rc) return rc;
    rc = encode_bf16_2d(&tmB, W, N, K, bn);
    if (rc) return rc;
    rc = bn == 256 ? launch_lse_noalloc<256>(d, tmA, tmB, p) : launch_lse_noalloc<128>(d, tmA, tmB, p);
    if (rc) return rc;
    const int rows_per_block = 8;
    lse_merge_kernel<<<static_cast<unsigned>((M + rows_per_block - 1) / rows_per_block), rows_per_block * 32, 0, t_stream>>>(
        p.lse_partial, p.M, p.rows_per_tile, p.m_tiles, p.n_tiles, p.group_m, p.n_full, p.tail_split, lse_out, nullptr, nullptr);
    CUDA_TRY(cudaGetLastError());
    g_launches.fetch_add(1);
    return MTMC_OK;
}

extern "C" {

// ---------------------------------------------------------------------------- host-pointer variants
int mtmc_fused_linear_host(const void* X, const void* W, const float* b, int64_t M, int64_t N, int64_t K, int act,
                           int out_dtype, void* out) {
    return fused_linear_host_impl(X, W, b, M, N, K, act, out_dtype, out, true);
}
int mtmc_swiglu_host(const void* X, const void* Wg, const void* Wu, int64_t M, int64_t N, int64_t K, void* out) {
    return swiglu_host_impl(X, Wg, Wu, M, N, K, out, true);
}
int mtmc_linear_lse_host(const void* X, const void* W, const float* b, int64_t M, int64_t N, int64_t K, float* lse_out) {
    return linear_lse_host_impl(X, W, b, M, N, K, lse_out, true);
}
int mtmc_fused_linear_host_async(const void* X, const void* W, const float* b, int64_t M, int64_t N, int64_t K, int act,
                                 int out_dtype, void* out) {
    return fused_linear_host_impl(X, W, b, M, N, K, act, out_dtype, out, false);
}
int mtmc_swiglu_host_async(const void* X, const void* Wg, const void* Wu, int64_t M, int64_t N, int64_t K, void* out) {
    return swiglu_host_impl(X, Wg, Wu, M, N, K, out, false);
}
int mtmc_linear_lse_host_async(const void* X, const void* W, const float* b, int64_t M, int64_t N, int64_t K, float* lse_out) {
    return linear_lse_host_impl(X, W, b, M, N, K, lse_out, false);
}

int mtmc_host_sync(void) {
    DeviceState* d = nullptr;
    int rc = get_device(&d);
    if (rc) return rc;
    for (auto& s : d->hslot)
        if (s.busy) { CUDA_TRY(cudaEventSynchronize(s.out_done)); s.busy = false; }
    return MTMC_OK;
}

}  // extern "C"
