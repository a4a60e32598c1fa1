// Host-side state of the tdx library: error text, per-device context, TMA descriptor cache, tuning cache.
// Part of the single translation unit tdx_api.cu (everything lives in its anonymous namespace).
#pragma once
#include "tdx.h"

#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <functional>
#include <map>
#include <mutex>
#include <queue>
#include <string>
#include <vector>

#include "simt_kernels.cuh"
#include "umma_conv_halo.cuh"
#include "umma_kernel.cuh"
#include "umma_pair.cuh"

namespace {

using tdx::UmmaParams;

// ------------------------------------------------------------------ errors
thread_local std::string g_err;

int fail(int status, const char* fmt, ...) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    g_err = buf;
    return status;
}

#define TDX_CUDA(expr)                                                                                   \
    do {                                                                                                 \
        cudaError_t e_ = (expr);                                                                         \
        if (e_ != cudaSuccess) return fail(TDX_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e_)); \
    } while (0)

std::atomic<int64_t> g_launches{0};

__device__ int g_device_status_word = 0;

// ------------------------------------------------------------------ per-device state
constexpr int kSmemLimitDefault = 232448;  // 227 KiB opt-in limit of sm_100
constexpr int kStaticSmemReserve = 512;    // barriers and flags declared statically in the kernel
constexpr int kDefaultSmCount = 148;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct DeviceCtx {
    int dev = -1;
    int sm_count = kDefaultSmCount;
    int smem_optin = kSmemLimitDefault;
    int* status_ptr = nullptr;
    EncodeTiledFn encode = nullptr;
    void* ws = nullptr;          // internal split-K workspace
    size_t ws_bytes = 0;
    void* staging[4] = {nullptr, nullptr, nullptr, nullptr};  // host-variant device copies
    size_t staging_bytes[4] = {0, 0, 0, 0};
    void* pieces[2] = {nullptr, nullptr};                     // bf16 pieces of fp32 operands (A, B)
    size_t pieces_bytes[2] = {0, 0};
    // host-buffer entry points: copies in and out run on their own streams, chunk by chunk, around the kernels
    static constexpr int kHostChunks = 8;
    cudaStream_t h2d = nullptr, d2h = nullptr;
    cudaEvent_t ev_start = nullptr, ev_done = nullptr, ev_in[kHostChunks] = {}, ev_out[kHostChunks] = {};
};

std::mutex g_mu;
std::map<int, DeviceCtx> g_ctx;

int get_ctx(DeviceCtx** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return fail(TDX_ERR_NO_DEVICE, "no CUDA device: %s", cudaGetErrorString(e));
    }
    std::lock_guard<std::mutex> lk(g_mu);
    auto it = g_ctx.find(dev);
    if (it != g_ctx.end()) {
        *out = &it->second;
        return TDX_OK;
    }
    cudaDeviceProp prop;
    e = cudaGetDeviceProperties(&prop, dev);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return fail(TDX_ERR_NO_DEVICE, "cudaGetDeviceProperties: %s", cudaGetErrorString(e));
    }
    if (prop.major != 10) return fail(TDX_ERR_NO_DEVICE, "device %d is sm_%d%d, this library is built for sm_100a", dev, prop.major, prop.minor);
    DeviceCtx c;
    c.dev = dev;
    c.sm_count = prop.multiProcessorCount;
    c.smem_optin = static_cast<int>(prop.sharedMemPerBlockOptin);
    void* sym = nullptr;
    e = cudaGetSymbolAddress(&sym, g_device_status_word);
    if (e != cudaSuccess) return fail(TDX_ERR_CUDA, "cudaGetSymbolAddress: %s", cudaGetErrorString(e));
    c.status_ptr = static_cast<int*>(sym);
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    e = cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &qres);
    if (e != cudaSuccess || fn == nullptr || qres != cudaDriverEntryPointSuccess)
        return fail(TDX_ERR_NO_DEVICE, "driver does not export cuTensorMapEncodeTiled");
    c.encode = reinterpret_cast<EncodeTiledFn>(fn);
    e = cudaFuncSetAttribute(tdx::umma_contract_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             c.smem_optin - kStaticSmemReserve);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(tdx::umma_contract_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 c.smem_optin - kStaticSmemReserve);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(tdx::umma_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 c.smem_optin - kStaticSmemReserve);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(tdx::umma_conv_halo_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 c.smem_optin - kStaticSmemReserve);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(tdx::sgemm_small_rowmajor_kernel,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, tdx::kSmallRowmajorSmem);
    if (e != cudaSuccess) return fail(TDX_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    auto ins = g_ctx.emplace(dev, c);
    *out = &ins.first->second;
    return TDX_OK;
}

// ------------------------------------------------------------------ TMA descriptor cache
struct MapKey {
    const void* ptr;
    int rank;
    uint64_t dims[4];
    uint64_t strides[3];
    uint32_t box[4];
    uint32_t estride[4];
    int swizzle;
    bool operator<(const MapKey& o) const { return std::memcmp(this, &o, sizeof(MapKey)) < 0; }
};
std::map<MapKey, CUtensorMap> g_maps;

// bf16 tensor, 128-byte (or 64-byte) swizzle, zero fill outside the tensor.
int get_tensor_map(DeviceCtx* ctx, const void* ptr, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                   const uint32_t* box, CUtensorMap* out, int swizzle_bytes = 128, const uint32_t* elem_strides = nullptr,
                   bool fp32 = false) {
    MapKey key;
    std::memset(&key, 0, sizeof key);
    key.ptr = ptr;
    key.rank = rank;
    key.swizzle = swizzle_bytes + (fp32 ? 1 : 0);        // element type is part of the key
    for (int i = 0; i < rank; ++i) { key.dims[i] = dims[i]; key.box[i] = box[i]; key.estride[i] = elem_strides ? elem_strides[i] : 1; }
    for (int i = 0; i + 1 < rank; ++i) key.strides[i] = strides_bytes[i];
    {
        std::lock_guard<std::mutex> lk(g_mu);
        auto it = g_maps.find(key);
        if (it != g_maps.end()) { *out = it->second; return TDX_OK; }
    }
    cuuint64_t gdim[4], gstr[3];
    cuuint32_t gbox[4], estr[4];
    for (int i = 0; i < rank; ++i) { gdim[i] = dims[i]; gbox[i] = box[i]; estr[i] = elem_strides ? elem_strides[i] : 1; }
    for (int i = 0; i + 1 < rank; ++i) gstr[i] = strides_bytes[i];
    CUtensorMap m;
    CUresult r = ctx->encode(&m, fp32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, static_cast<cuuint32_t>(rank),
                             const_cast<void*>(ptr), gdim, gstr, gbox, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                             swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
        return fail(TDX_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d) rank %d dims %llu %llu box %u %u", (int)r, rank,
                    (unsigned long long)dims[0], (unsigned long long)(rank > 1 ? dims[1] : 0), box[0],
                    rank > 1 ? box[1] : 0);
    {
        std::lock_guard<std::mutex> lk(g_mu);
        if (g_maps.size() > 4096) g_maps.clear();
        g_maps[key] = m;
    }
    *out = m;
    return TDX_OK;
}

// ------------------------------------------------------------------ tuning cache
struct TuneEntry { tdx_config cfg; float us; };
std::map<std::string, TuneEntry> g_tune;

std::string gemm_key(int64_t M, int64_t N, int64_t K, int tA, int tB, int dtype) {
    char b[160];
    snprintf(b, sizeof b, "gemm:%lld:%lld:%lld:%d:%d:%d", (long long)M, (long long)N, (long long)K, tA, tB, dtype);
    return b;
}
std::string conv_key(int64_t N, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int64_t R, int64_t S, int pad,
                     int stride, int dtype) {
    char b[200];
    snprintf(b, sizeof b, "conv:%lld:%lld:%lld:%lld:%lld:%lld:%lld:%d:%d:%d", (long long)N, (long long)H, (long long)W,
             (long long)Cin, (long long)Cout, (long long)R, (long long)S, pad, stride, dtype);
    return b;
}
// every change of the cache bumps the epoch, which invalidates the per-thread memo of the last GEMM query below
std::atomic<unsigned long long> g_tune_epoch{1};
bool tune_lookup(const std::string& key, tdx_config* out) {
    std::lock_guard<std::mutex> lk(g_mu);
    auto it = g_tune.find(key);
    if (it == g_tune.end()) return false;
    *out = it->second.cfg;
    return true;
}
// A stream of calls on one shape asks the same question every time: remember the last answer per thread instead of
// formatting the key and searching the map again (about half a microsecond of a launch-bound call).
bool tune_lookup_gemm(int64_t M, int64_t N, int64_t K, int tA, int tB, int dtype, tdx_config* out) {
    struct Memo { unsigned long long epoch = 0; int64_t M = 0, N = 0, K = 0; int tA = 0, tB = 0, dtype = 0; bool found = false; tdx_config cfg; };
    static thread_local Memo memo;
    const unsigned long long epoch = g_tune_epoch.load(std::memory_order_acquire);
    if (memo.epoch != epoch || memo.M != M || memo.N != N || memo.K != K || memo.tA != tA || memo.tB != tB ||
        memo.dtype != dtype) {
        memo.found = tune_lookup(gemm_key(M, N, K, tA, tB, dtype), &memo.cfg);
        memo.epoch = epoch; memo.M = M; memo.N = N; memo.K = K; memo.tA = tA; memo.tB = tB; memo.dtype = dtype;
    }
    if (memo.found) *out = memo.cfg;
    return memo.found;
}
// TDX_FORCE_CONFIG="tile_m=128,tile_n=128,split_k=6": a partial tile configuration that calls WITHOUT an explicit
// configuration take instead of the automatic choice (tuning cache, cost model) -- for experiments and for pinning a
// deployment to a known configuration without rebuilding the caller.  Read once per process; unknown names or values
// that are not integers make the variable void (reported once on stderr).  Fields not named stay "choose for me".
const tdx_config* forced_config() {
    static tdx_config cfg;
    static int state = 0;            // 0 = not read yet, 1 = none, 2 = valid
    static std::mutex mu;
    std::lock_guard<std::mutex> lk(mu);
    if (state == 0) {
        state = 1;
        const char* env = std::getenv("TDX_FORCE_CONFIG");
        if (env != nullptr && *env != '\0') {
            std::memset(&cfg, 0, sizeof cfg);
            bool ok = true;
            std::string text(env);
            size_t pos = 0;
            while (ok && pos < text.size()) {
                const size_t comma = text.find(',', pos);
                const std::string item = text.substr(pos, comma == std::string::npos ? std::string::npos : comma - pos);
                pos = comma == std::string::npos ? text.size() : comma + 1;
                const size_t eq = item.find('=');
                if (eq == std::string::npos) { ok = false; break; }
                const std::string name = item.substr(0, eq);
                char* end = nullptr;
                const long v = std::strtol(item.c_str() + eq + 1, &end, 10);
                if (end == item.c_str() + eq + 1 || *end != '\0') { ok = false; break; }
                struct { const char* n; int* f; } fields[] = {
                    {"kernel", &cfg.kernel}, {"tile_m", &cfg.tile_m}, {"tile_n", &cfg.tile_n}, {"tile_k", &cfg.tile_k},
                    {"stages", &cfg.stages}, {"cta_pair", &cfg.cta_pair}, {"split_k", &cfg.split_k}, {"store_mode", &cfg.store_mode},
                    {"raster", &cfg.raster}, {"patch_w", &cfg.patch_w}, {"patch_h", &cfg.patch_h}, {"k_stagger", &cfg.k_stagger},
                    {"halo", &cfg.halo}, {"fit", &cfg.fit}};
                bool found = false;
                for (auto& f : fields)
                    if (name == f.n) { *f.f = static_cast<int>(v); found = true; }
                ok = found;
            }
            if (ok) state = 2;
            else fprintf(stderr, "tdx: TDX_FORCE_CONFIG=\"%s\" is not a list of <field>=<integer>; ignored\n", env);
        }
    }
    return state == 2 ? &cfg : nullptr;
}

// TDX_DEBUG_BOUNDS=1: the one-thread-per-output kernels check every index against its operand's extent (read once).
bool debug_bounds_enabled() {
    static const bool on = [] {
        const char* e = std::getenv("TDX_DEBUG_BOUNDS");
        return e != nullptr && *e != '\0' && std::strcmp(e, "0") != 0;
    }();
    return on;
}

void cfg_to_ints(const tdx_config& c, int* v) {
    v[0] = c.kernel; v[1] = c.tile_m; v[2] = c.tile_n; v[3] = c.tile_k; v[4] = c.stages; v[5] = c.cta_pair;
    v[6] = c.split_k; v[7] = c.store_mode; v[8] = c.raster; v[9] = c.patch_w; v[10] = c.patch_h; v[11] = c.k_stagger;
    v[12] = c.halo;
    v[13] = c.fit;
}
void ints_to_cfg(const int* v, tdx_config* c) {
    c->kernel = v[0]; c->tile_m = v[1]; c->tile_n = v[2]; c->tile_k = v[3]; c->stages = v[4]; c->cta_pair = v[5];
    c->split_k = v[6]; c->store_mode = v[7]; c->raster = v[8]; c->patch_w = v[9]; c->patch_h = v[10];
    c->k_stagger = v[11];
    c->halo = v[12];
    c->fit = v[13];
}

}  // namespace
