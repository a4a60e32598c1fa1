// C-ABI of the tdx library: argument validation, kernel choice, TMA descriptor cache,
// launches, the tile-configuration search and its cache.  See include/tdx.h for the contract.
#include "tdx.h"

#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <functional>
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
                   const uint32_t* box, CUtensorMap* out, int swizzle_bytes = 128, const uint32_t* elem_strides = nullptr) {
    MapKey key;
    std::memset(&key, 0, sizeof key);
    key.ptr = ptr;
    key.rank = rank;
    key.swizzle = swizzle_bytes;
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
    CUresult r = ctx->encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, static_cast<cuuint32_t>(rank),
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
bool tune_lookup(const std::string& key, tdx_config* out) {
    std::lock_guard<std::mutex> lk(g_mu);
    auto it = g_tune.find(key);
    if (it == g_tune.end()) return false;
    *out = it->second.cfg;
    return true;
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

// ------------------------------------------------------------------ problem descriptions
struct GemmProblem {
    int64_t M, N, K;
    int transA, transB, dtype;
};
struct ConvProblem {
    int64_t N, H, W, Cin, Cout, R, S;
    int pad, stride, dtype;
    int64_t P, Q;
};

int64_t conv_out_dim(int64_t H, int64_t R, int64_t pad, int64_t stride) {
    const int64_t span = H + 2 * pad - R;
    return span < 0 ? 0 : span / stride + 1;
}
inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// Layout rules of the tensor-core GEMM path: every TMA row pitch must be a multiple of 16 bytes.
bool gemm_umma_layout_ok(const GemmProblem& g) {
    if (g.dtype != TDX_BF16) return false;
    if (g.M >= (1LL << 31) || g.N >= (1LL << 31) || g.K >= (1LL << 31)) return false;
    if (g.transA ? (g.M % 8) : (g.K % 8)) return false;
    if (g.transB ? (g.K % 8) : (g.N % 8)) return false;
    if (ceil_div(g.M, 128) * ceil_div(g.N, 32) * 64 >= (1LL << 31)) return false;
    return true;
}
bool conv_umma_layout_ok(const ConvProblem& c) {
    if (c.dtype != TDX_BF16 || c.stride > 8) return false;      // strided windows: per-tap loads with a traversal stride
    if (c.Cin % 8) return false;
    if (c.N * c.P * c.Q >= (1LL << 31) || c.H * c.W * c.Cin * 2 >= (1LL << 40)) return false;
    if (c.R * c.S >= (1LL << 15) || c.Cout >= (1LL << 31)) return false;
    return true;
}

// Shared memory the staged (TMA-store) epilogue needs: one 32 x 32 bf16 block for each of its 16 warps.
int staging_bytes_for(int /*tile_m*/, int store_mode) { return store_mode == 2 ? 16 * 2048 : 0; }

int umma_max_stages(int tile_m, int tile_n, int smem_limit, int store_mode) {
    const int stage = (tile_m + tile_n) * 128;
    int s = (smem_limit - kStaticSmemReserve - 1024 - staging_bytes_for(tile_m, store_mode)) / stage;
    return std::min(s, tdx::kMaxStages);
}

// Accumulator slots (128 x tile_n each) kept in TMEM: a 256-row tile uses two per tile, and gets four
// when they fit so that the epilogue still overlaps the next tile's main loop.
// Halo-reuse convolution: 8 x 16 output-pixel patches, input window kept in shared memory across the taps.
constexpr int kHaloPatchW = 8, kHaloPatchH = 16, kHaloAStages = 2;
// Stacked images: rows each image takes in the column of all images.  The rows between two images must read as
// zero for both, i.e. be the bottom padding of one and the top padding of the next: H + pad rows per image
// (never fewer than the P output rows).
int64_t stacked_rows_per_image(const ConvProblem& c) { return std::max(c.P, c.H + c.pad); }
// 128-row halves the halo kernel works on: 8 x 16 patches cut per image (halo 2) or from the stacked column (halo 3)
int64_t halo_patches(const ConvProblem& c, int mode) {
    const int64_t pw = ceil_div(c.Q, kHaloPatchW);
    return mode == 3 ? pw * ceil_div(c.N * stacked_rows_per_image(c), kHaloPatchH) : pw * c.N * ceil_div(c.P, kHaloPatchH);
}
int halo_tile_bytes(int64_t R, int64_t S) {
    const int64_t b = (kHaloPatchW + S - 1) * (kHaloPatchH + R - 1) * 128;
    return static_cast<int>((b + 1023) / 1024 * 1024);
}
int halo_max_stages(int tile_m, int tile_n, int64_t R, int64_t S, int smem_limit, int store_mode) {
    const int a = kHaloAStages * (tile_m / 128) * halo_tile_bytes(R, S);
    const int left = smem_limit - kStaticSmemReserve - 1024 - staging_bytes_for(tile_m, store_mode) - a;
    return left <= 0 ? 0 : std::min(left / (tile_n * 128), tdx::kMaxStages);
}

// CTA pair (256 x tile_n per pair): each CTA stages its 128 rows of A and tile_n / 2 columns of B
int pair_max_stages(int tile_n, int smem_limit, int store_mode) {
    const int stage = (128 + tile_n / 2) * 128;
    const int s = (smem_limit - kStaticSmemReserve - 1024 - staging_bytes_for(128, store_mode)) / stage;
    return std::min(s, tdx::kMaxStages);
}

int tmem_slots_for(int tile_m, int bn) {
    const int mh = tile_m / 128;
    int s = std::min(tdx::kMaxSlots, 512 / bn);     // as many as TMEM holds: narrow tiles are short, and the
    s -= s % mh;                                    // epilogue's latency then spans several tiles
    return std::max(s, mh);
}
int tmem_cols_for(int tile_m, int bn) {
    int c = 32;
    while (c < tmem_slots_for(tile_m, bn) * bn) c *= 2;
    return c;
}

// Static feasibility of a fully specified tensor-core configuration (the search-space constraints).
// Returns 0 when feasible, else a short reason.
const char* umma_config_reason(const tdx_config& c, bool b_mn_major, int64_t num_kb, int smem_limit, bool conv,
                               int64_t N, int64_t R = 1, int64_t S = 1, int stride = 1) {
    if (c.tile_m != 128 && c.tile_m != 256) return "tile_m must be 128 or 256";
    if (c.tile_k != 64) return "tile_k must be 64";
    if (c.cta_pair != 1 && c.cta_pair != 2) return "cta_pair must be 1 or 2";
    if (c.cta_pair == 2) {
        if (conv) return "CTA pairs are implemented for the GEMM only";
        if (c.tile_m != 256) return "a CTA pair works on 256-row tiles";
        if (c.split_k != 1) return "CTA pairs have no split-K";
        if (b_mn_major && c.tile_n % 128) return "tile_n must be a multiple of 128 for a CTA pair when B is read N-major";
        if (c.k_stagger) return "CTA pairs have no k_stagger";
    }
    if (c.store_mode != 1 && c.store_mode != 2) return "store_mode must be 1 (direct) or 2 (TMA store)";
    if (c.store_mode == 2) {
        if (N % 8) return "the TMA-store epilogue needs an output row pitch that is a multiple of 16 bytes";
        if (c.split_k > 1) return "split-K writes fp32 partials directly: use store_mode 1";
        if (conv && c.patch_w * c.patch_h < 32) return "the TMA-store epilogue needs patches of at least 32 pixels";
    }
    if (c.tile_n < 32 || c.tile_n > 256 || c.tile_n % 32) return "tile_n must be a multiple of 32 in [32, 256]";
    if (b_mn_major && c.tile_n % 64) return "tile_n must be a multiple of 64 when B is read N-major";
    if (!conv && c.halo > 1) return "halo applies to the convolution only";
    if (conv && (c.halo < 1 || c.halo > 3))
        return "halo must be 1 (per-tap loads), 2 (halo tile kept in shared memory) or 3 (the same over stacked images)";
    if (conv && stride > 1 && (c.patch_w * stride > 256 || c.patch_h * stride > 256))
        return "patch times stride exceeds the 256-element limit of a copy";
    if (conv && c.halo >= 2) {
        if (stride != 1) return "halo reuse needs stride 1";
        if (R * S < 2) return "halo reuse needs a filter with more than one tap";
        if (c.patch_w != kHaloPatchW || c.patch_h != kHaloPatchH) return "halo reuse works on 8 x 16 patches";
        if (kHaloPatchW + S - 1 > 256 || kHaloPatchH + R - 1 > 256) return "filter too large for a halo tile";
        if (c.stages < 2 || c.stages > halo_max_stages(c.tile_m, c.tile_n, R, S, smem_limit, c.store_mode))
            return "stages outside the shared-memory budget";
    } else if (c.cta_pair == 2) {
        if (c.stages < 2 || c.stages > pair_max_stages(c.tile_n, smem_limit, c.store_mode)) return "stages outside the shared-memory budget";
    } else
    if (c.stages < 2 || c.stages > umma_max_stages(c.tile_m, c.tile_n, smem_limit, c.store_mode)) return "stages outside the shared-memory budget";
    if (c.split_k < 1) return "split_k must be >= 1";
    if (conv && c.split_k != 1) return "conv has no split-K";
    if (c.split_k > 1) {
        const int64_t per = ceil_div(num_kb, c.split_k);
        if ((c.split_k - 1) * per >= num_kb) return "split_k leaves an empty K slice";
    }
    if (c.raster < 0) return "raster must be >= 0";
    if (c.fit < 0 || c.fit > 2) return "fit must be 0 (choose), 1 (uniform tiles) or 2 (tile widths fitted to the CTA count)";
    if (c.k_stagger != 0 && c.k_stagger != 1) return "k_stagger must be 0 or 1";
    return nullptr;
}

bool patch_ok(int bw, int bh) {
    const int a = bw * bh;
    return bw >= 8 && bw <= 128 && bh >= 1 && a <= 128 && (a & (a - 1)) == 0 && (bw & (bw - 1)) == 0;
}

// stride: a patch side times the stride must stay within the 256 elements one copy can span
void choose_patch(int64_t P, int64_t Q, int* bw_out, int* bh_out, int stride = 1) {
    int64_t best_cost = -1;
    int best_bw = 8, best_bh = 1;
    for (int bw = 8; bw <= 128 && bw * stride <= 256; bw *= 2) {
        for (int bh = 1; bw * bh <= 128 && bh * stride <= 256; bh *= 2) {
            const int64_t cost = ceil_div(Q, bw) * bw * ceil_div(P, bh) * bh;
            const bool better = best_cost < 0 || cost < best_cost ||
                                (cost == best_cost && (bw * bh > best_bw * best_bh ||
                                                       (bw * bh == best_bw * best_bh && bw > best_bw)));
            if (better) { best_cost = cost; best_bw = bw; best_bh = bh; }
        }
    }
    *bw_out = best_bw;
    *bh_out = best_bh;
}

// Heuristic default (used when neither the caller nor the tuning cache gives a configuration).
void default_umma_config(int64_t tiles_m, int64_t N, int64_t num_kb, bool b_mn_major, int sm_count, int smem_limit,
                         bool allow_split, tdx_config* c) {
    std::memset(c, 0, sizeof *c);
    c->kernel = TDX_KERNEL_UMMA;
    c->tile_m = 128;
    c->tile_k = 64;
    c->cta_pair = 1;
    c->store_mode = 1;
    c->split_k = 1;
    const int min_bn = b_mn_major ? 64 : 32;
    int bn = 0, tm = 128;
    const int64_t n_cap = ceil_div(N, min_bn) * min_bn;   // narrowest tile that covers N at once
    // widest tile that still gives every SM at least one tile; 256-row tiles first (fewest L2 bytes per flop)
    for (int cand_m : {256, 128}) {
        if (bn) break;
        for (int cand : {256, 128, 64, 32}) {
            if (cand < min_bn) continue;
            if (cand_m == 256 && cand < 128) continue;
            if (cand > n_cap && cand / 2 >= n_cap) continue;  // a narrower tile covers N just as well
            if (ceil_div(tiles_m, cand_m / 128) * ceil_div(N, cand) >= sm_count) { bn = cand; tm = cand_m; break; }
        }
    }
    if (bn == 0) {
        bn = N > 64 ? 128 : (N > 32 ? 64 : min_bn);
        const int64_t tiles = tiles_m * ceil_div(N, bn);
        if (allow_split && tiles < sm_count) {
            int64_t s = std::min<int64_t>(ceil_div(sm_count, tiles), std::max<int64_t>(1, num_kb / 4));
            s = std::min<int64_t>(s, 32);
            while (s > 1 && (s - 1) * ceil_div(num_kb, s) >= num_kb) --s;
            c->split_k = static_cast<int>(std::max<int64_t>(1, s));
        }
    }
    c->tile_m = tm;
    c->tile_n = bn;
    // staged epilogue whenever the layout allows it (whole-line writes instead of 16-byte pieces)
    if (c->split_k == 1 && N % 8 == 0) c->store_mode = 2;
    c->stages = std::max(2, umma_max_stages(tm, bn, smem_limit, c->store_mode));
    c->raster = 8;
}


// ------------------------------------------------------------------ tile plan fitted to the number of CTAs
// A uniform grid of T tiles on G persistent CTAs takes ceil(T / G) tile times although it holds only T / G of
// work per CTA (the 4096^3 GEMM: 256 tiles of 256 x 256 on 148 CTAs = 1.73 tile times of work done in 2).  The
// plan keeps the tile height and cuts some row blocks into narrower tiles (widths w < tile_n, both multiples of
// 64) so that every CTA ends at about the same time: tiles are dealt longest first, each to the CTA with the
// least work so far.  The cost model is the measured instruction time of one MMA (N / 2 cycles, at least 60)
// plus a fixed and a per-column epilogue cost.
struct TilePlan {
    std::vector<int4> table;   // [round * grid + cta] = (row block, first column, width, 0)
    int rounds = 0;
    int grid = 0;
    double makespan = 0.0;     // model cycles
    double uniform = 0.0;      // the same for the uniform grid
};

// mmas_per_kb: MMAs one CTA's tensor core runs per 64-deep K block (4 per 128 rows it owns)
double tile_cost_cycles(int mmas_per_kb, int width, int64_t num_kb) {
    const double mma = std::max(width / 2.0, 60.0);
    return static_cast<double>(num_kb) * mmas_per_kb * mma + 1500.0 + 13.0 * width;
}

// makespan of `na` tiles of cost ca and `nb` tiles of cost cb (ca >= cb > 0), dealt longest first on g CTAs, each
// to the CTA with the least work so far (closed form of that greedy rule for two sizes)
double lpt_two_sizes(int64_t na, double ca, int64_t nb, double cb, int g) {
    const int64_t q = na / g, x = na % g;              // x CTAs hold q + 1 wide tiles, g - x hold q
    const double low = ca * static_cast<double>(q), high = x > 0 ? low + ca : low;
    if (nb <= 0) return high;
    if (x == 0) return low + cb * static_cast<double>(ceil_div(nb, g));
    // the g - x lighter CTAs take narrow tiles until they have caught up with the others
    const int64_t catch_up = static_cast<int64_t>(std::ceil(ca / cb - 1e-9));
    const int64_t lighter = g - x;
    if (nb <= catch_up * lighter) return std::max(high, low + cb * static_cast<double>(ceil_div(nb, lighter)));
    const double low2 = low + cb * static_cast<double>(catch_up);      // >= high, by less than cb
    const int64_t rest = nb - catch_up * lighter;
    const int64_t f = rest / g, rem = rest % g;
    if (rem == 0) return low2 + cb * static_cast<double>(f);
    if (rem <= x) return std::max(low2 + cb * static_cast<double>(f), high + cb * static_cast<double>(f + 1));
    return low2 + cb * static_cast<double>(f + 1);
}

// Searches widths and how many row blocks take the narrower cut.  Returns false when nothing beats the uniform grid
// by `min_gain` (relative).
// `g` workers (CTAs, or CTA pairs when pair is set: a pair's two tensor cores share a 256-row tile).
bool plan_fitted_tiles(int64_t M, int64_t N, int64_t num_kb, int bm, int bn, int raster, int g, double min_gain,
                       TilePlan* out, bool pair = false) {
    const int64_t tiles_m = ceil_div(M, bm);
    const int64_t uniform_tiles = tiles_m * ceil_div(N, bn);
    const int mmas = pair ? 4 : 4 * (bm / 128);
    const double c_big = tile_cost_cycles(mmas, bn, num_kb);
    const double uniform = lpt_two_sizes(uniform_tiles, c_big, 0, 0.0, g);
    double best = uniform;
    int best_w = 0;
    int64_t best_b = 0, best_b1 = 0, best_e = 0;
    // pairs: each CTA loads half of a tile's columns, kept a multiple of 64 (one copy per 64 rows)
    const int w_step = pair ? 128 : 64;
    for (int w = bn - w_step; w >= 128; w -= w_step) {
        const double c_small = tile_cost_cycles(mmas, w, num_kb);
        // option b of a row block: b tiles of width w at the high columns, a(b) tiles of width bn before them
        auto bigs_for = [&](int64_t b) { return ceil_div(std::max<int64_t>(0, N - b * w), bn); };
        // options that do not carry a tile more than needed
        std::vector<int64_t> opts;
        for (int64_t b = 0; b <= ceil_div(N, w); ++b)
            if (b == 0 || bigs_for(b) * bn + b * w - N < w) opts.push_back(b);
        for (size_t i = 0; i < opts.size(); ++i)
        for (size_t j = i + 1; j < opts.size(); ++j) {
            const int64_t b0 = opts[i], b1 = opts[j];
            for (int64_t e = 0; e <= tiles_m; ++e) {                            // e row blocks take option b1
                const int64_t na = (tiles_m - e) * bigs_for(b0) + e * bigs_for(b1);
                const int64_t nb = (tiles_m - e) * b0 + e * b1;
                const double m = lpt_two_sizes(na, c_big, nb, c_small, g);
                if (m < best * (1.0 - 1e-9)) { best = m; best_w = w; best_b = b0; best_b1 = b1; best_e = e; }
            }
        }
    }
    out->uniform = uniform;
    out->makespan = best;
    if (best_w == 0 || best > uniform * (1.0 - min_gain)) return false;
    // list the tiles: wide ones first, each group in the panel order of the uniform grid (row blocks fastest
    // inside a panel of `raster` row blocks, then columns, then panels)
    const int w = best_w;
    auto bigs_for = [&](int64_t b) { return ceil_div(std::max<int64_t>(0, N - b * w), static_cast<int64_t>(bn)); };
    struct T { int m, n0, width; };
    std::vector<T> wide, narrow;
    const int64_t panel = raster <= 0 ? tiles_m : std::min<int64_t>(raster, tiles_m);
    for (int64_t m0 = 0; m0 < tiles_m; m0 += panel) {
        const int64_t rows = std::min(panel, tiles_m - m0);
        const int64_t max_cols = ceil_div(N, 64) + 1;
        for (int64_t c = 0; c < max_cols; ++c)          // c-th tile of each row block of the panel
            for (int64_t r = 0; r < rows; ++r) {
                const int64_t m = m0 + r;
                const int64_t b = (m >= tiles_m - best_e) ? best_b1 : best_b;
                const int64_t a = bigs_for(b);
                if (c < a) wide.push_back({static_cast<int>(m), static_cast<int>(c * bn), bn});
                else if (c < a + b) narrow.push_back({static_cast<int>(m), static_cast<int>(a * bn + (c - a) * w), w});
            }
    }
    const int64_t total = static_cast<int64_t>(wide.size() + narrow.size());
    const int grid = static_cast<int>(std::min<int64_t>(total, g));
    std::vector<std::vector<T>> per(grid);
    std::vector<double> load(grid, 0.0);
    const double c_small = tile_cost_cycles(mmas, w, num_kb);
    auto deal = [&](const std::vector<T>& v, double cost) {
        for (const T& t : v) {
            int who = 0;
            for (int i = 1; i < grid; ++i) if (load[i] < load[who] - 1e-6) who = i;
            per[who].push_back(t);
            load[who] += cost;
        }
    };
    deal(wide, c_big);
    deal(narrow, c_small);
    size_t rounds = 0;
    for (auto& v : per) rounds = std::max(rounds, v.size());
    out->grid = grid;
    out->rounds = static_cast<int>(rounds);
    out->table.assign(rounds * grid, make_int4(0, 0, 0, 0));
    for (int i = 0; i < grid; ++i)
        for (size_t k = 0; k < per[i].size(); ++k)
            out->table[k * grid + i] = make_int4(per[i][k].m, per[i][k].n0, per[i][k].width, 0);
    return true;
}

// Device copies of tile plans, one per (shape, tile, CTA count); never freed (a few KB each).
struct PlanKey {
    int64_t M, N, num_kb;
    int bm, bn, raster, g, forced, pair;
    bool operator<(const PlanKey& o) const { return std::memcmp(this, &o, sizeof(PlanKey)) < 0; }
};
struct DevicePlan { int4* dev = nullptr; int rounds = 0, grid = 0; bool fitted = false; };
std::map<PlanKey, DevicePlan> g_plans;

// Looks the plan up (building and uploading it on first use; the upload is ordered on `st` before the kernel).
int get_tile_plan(DeviceCtx* ctx, int64_t M, int64_t N, int64_t num_kb, int bm, int bn, int raster, double min_gain,
                  cudaStream_t st, DevicePlan* out, bool pair = false) {
    PlanKey key;
    std::memset(&key, 0, sizeof key);
    key.M = M; key.N = N; key.num_kb = num_kb; key.bm = bm; key.bn = bn; key.raster = raster; key.g = pair ? ctx->sm_count / 2 : ctx->sm_count; key.forced = min_gain <= 0.0 ? 1 : 0;
    key.pair = pair ? 1 : 0;
    {
        std::lock_guard<std::mutex> lk(g_mu);
        auto it = g_plans.find(key);
        if (it != g_plans.end()) { *out = it->second; return TDX_OK; }
    }
    TilePlan plan;
    DevicePlan d;
    d.fitted = plan_fitted_tiles(M, N, num_kb, bm, bn, raster, key.g, min_gain, &plan, pair);
    if (d.fitted) {
        const size_t bytes = plan.table.size() * sizeof(int4);
        void* dev = nullptr;
        TDX_CUDA(cudaMalloc(&dev, bytes));
        // the table is a std::vector about to go out of scope: copy synchronously (once per shape)
        TDX_CUDA(cudaMemcpy(dev, plan.table.data(), bytes, cudaMemcpyHostToDevice));
        d.dev = static_cast<int4*>(dev);
        d.rounds = plan.rounds;
        d.grid = plan.grid;
    }
    (void)st;
    {
        std::lock_guard<std::mutex> lk(g_mu);
        g_plans[key] = d;
    }
    *out = d;
    return TDX_OK;
}

// ------------------------------------------------------------------ launches
int launch_umma(DeviceCtx* ctx, bool conv, const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc,
                const UmmaParams& p_in, cudaStream_t st, bool halo = false, const CUtensorMap* ma_row = nullptr,
                const CUtensorMap* mc_row = nullptr, int plan_grid = 0) {
    const long long items = static_cast<long long>(p_in.tiles_m) * p_in.tiles_n * p_in.split_k;
    UmmaParams p = p_in;
    if (p.b_box == 0) p.b_box = p.bn;
    const int grid = p.tiles != nullptr ? plan_grid : static_cast<int>(std::min<long long>(items, ctx->sm_count));
    size_t smem = static_cast<size_t>(p.stages) * ((p.bm + p.bn) * 128) + 1024 +
                  staging_bytes_for(p.bm, p.tma_store ? 2 : 1);
    if (halo)
        smem = static_cast<size_t>(p.a_stages) * (p.bm / 128) * p.halo_bytes + static_cast<size_t>(p.stages) * p.bn * 128 +
               1024 + staging_bytes_for(p.bm, p.tma_store ? 2 : 1);
    // producer warp, MMA warp, then 16 epilogue warps (staged epilogue) or 4 per 128-row half (direct)
    const int threads = p.tma_store ? 576 : (p.bm == 256 ? 320 : 192);
    // programmatic stream serialization: the grid may be scheduled while the previous kernel of the stream drains; its
    // set-up then overlaps that tail, and it waits on the device for the predecessor before touching global memory
    cudaLaunchConfig_t lc;
    std::memset(&lc, 0, sizeof lc);
    lc.gridDim = dim3(static_cast<unsigned>(grid));
    lc.blockDim = dim3(static_cast<unsigned>(halo ? threads + 32 : threads));   // halo: one more warp, the halo producer
    lc.dynamicSmemBytes = smem;
    lc.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    if (halo)
        TDX_CUDA(cudaLaunchKernelEx(&lc, tdx::umma_conv_halo_kernel, ma, ma_row ? *ma_row : ma, mb, mc, mc_row ? *mc_row : mc, p));
    else if (conv)
        TDX_CUDA(cudaLaunchKernelEx(&lc, tdx::umma_contract_kernel<true>, ma, mb, mc, p));
    else
        TDX_CUDA(cudaLaunchKernelEx(&lc, tdx::umma_contract_kernel<false>, ma, mb, mc, p));
    TDX_CUDA(cudaGetLastError());
    g_launches.fetch_add(1);
    return TDX_OK;
}

// The reduction is launched with programmatic stream serialization so that its launch latency hides behind
// the tail of the GEMM kernel; it waits on the device for the GEMM grid to complete before reading partials.
int launch_splitk_reduce(int grid, cudaStream_t st, long long MN, int N, int split, const float* partial, float alpha,
                         __nv_bfloat16* out, int vec8, float beta = 0.0f) {
    cudaLaunchConfig_t lc;
    std::memset(&lc, 0, sizeof lc);
    lc.gridDim = dim3(static_cast<unsigned>(grid));
    lc.blockDim = dim3(256);
    lc.dynamicSmemBytes = 0;
    lc.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    const float* bias = nullptr;
    int relu = 0;
    TDX_CUDA(cudaLaunchKernelEx(&lc, tdx::splitk_reduce_kernel, MN, N, split, partial, alpha, bias, relu, out, vec8, beta));
    g_launches.fetch_add(1);
    return TDX_OK;
}

int ensure_ws(DeviceCtx* ctx, size_t bytes, void** out) {
    if (ctx->ws_bytes < bytes) {
        if (ctx->ws) TDX_CUDA(cudaFree(ctx->ws));
        ctx->ws = nullptr;
        ctx->ws_bytes = 0;
        TDX_CUDA(cudaMalloc(&ctx->ws, bytes));
        ctx->ws_bytes = bytes;
    }
    *out = ctx->ws;
    return TDX_OK;
}

int run_gemm_umma(DeviceCtx* ctx, const GemmProblem& g, float alpha, const void* A, const void* B, void* C,
                  const tdx_config& cfg, void* ws, size_t ws_bytes, bool internal_ws, cudaStream_t st, float beta = 0.0f) {
    const int64_t num_kb = ceil_div(g.K, 64);
    UmmaParams p;
    std::memset(&p, 0, sizeof p);
    p.M = static_cast<int>(g.M);
    p.N = static_cast<int>(g.N);
    p.num_kb = static_cast<int>(num_kb);
    p.bm = cfg.tile_m;
    p.slots = tmem_slots_for(cfg.tile_m, cfg.tile_n);
    p.tiles_m = static_cast<int>(ceil_div(g.M, cfg.tile_m));
    p.tiles_n = static_cast<int>(ceil_div(g.N, cfg.tile_n));
    p.panel = cfg.raster == 0 ? p.tiles_m : std::min(cfg.raster, p.tiles_m);
    p.split_k = cfg.split_k;
    p.kb_per_split = static_cast<int>(ceil_div(num_kb, cfg.split_k));
    p.k_stagger = cfg.k_stagger;
    p.bn = cfg.tile_n;
    p.stages = cfg.stages;
    p.tmem_cols = tmem_cols_for(cfg.tile_m, cfg.tile_n);
    p.a_mn_major = g.transA ? 1 : 0;   // A stored K x M: M contiguous
    p.b_mn_major = g.transB ? 0 : 1;   // B stored K x N: N contiguous
    p.alpha = alpha;
    p.beta = beta;
    p.bias = nullptr;
    p.relu = 0;
    p.C = static_cast<__nv_bfloat16*>(C);
    p.ldc = g.N;
    p.status = ctx->status_ptr;
    p.vec_store = (g.N % 8 == 0) && (reinterpret_cast<uintptr_t>(C) % 16 == 0);

    if (cfg.split_k > 1) {
        const size_t need = static_cast<size_t>(cfg.split_k) * g.M * g.N * sizeof(float);
        if (internal_ws) {
            int rc = ensure_ws(ctx, need, &ws);
            if (rc) return rc;
        } else if (ws == nullptr || ws_bytes < need || reinterpret_cast<uintptr_t>(ws) % 256) {
            return fail(TDX_ERR_WORKSPACE, "split_k=%d needs %zu bytes of 256-byte aligned workspace", cfg.split_k, need);
        }
        p.partial = static_cast<float*>(ws);
    }

    CUtensorMap ma, mb;
    int rc;
    if (p.a_mn_major) {
        uint64_t dims[2] = {static_cast<uint64_t>(g.M), static_cast<uint64_t>(g.K)};
        uint64_t str[1] = {static_cast<uint64_t>(g.M) * 2};
        uint32_t box[2] = {64, 64};
        rc = get_tensor_map(ctx, A, 2, dims, str, box, &ma);
    } else {
        uint64_t dims[2] = {static_cast<uint64_t>(g.K), static_cast<uint64_t>(g.M)};
        uint64_t str[1] = {static_cast<uint64_t>(g.K) * 2};
        uint32_t box[2] = {64, 128};
        rc = get_tensor_map(ctx, A, 2, dims, str, box, &ma);
    }
    if (rc) return rc;
    // tile widths fitted to the number of CTAs (see plan_fitted_tiles): B then arrives in 64-row copies
    int plan_grid = 0;
    if (cfg.fit != 1 && cfg.split_k == 1 && cfg.tile_n >= 192 && cfg.tile_n % 64 == 0) {
        DevicePlan dp;
        rc = get_tile_plan(ctx, g.M, g.N, num_kb, cfg.tile_m, cfg.tile_n, cfg.raster, cfg.fit == 2 ? 0.0 : 0.03, st, &dp);
        if (rc) return rc;
        if (dp.fitted) {
            p.tiles = dp.dev;
            p.rounds = dp.rounds;
            p.b_box = 64;
            plan_grid = dp.grid;
        }
    }
    if (p.b_mn_major) {
        uint64_t dims[2] = {static_cast<uint64_t>(g.N), static_cast<uint64_t>(g.K)};
        uint64_t str[1] = {static_cast<uint64_t>(g.N) * 2};
        uint32_t box[2] = {64, 64};
        rc = get_tensor_map(ctx, B, 2, dims, str, box, &mb);
    } else {
        uint64_t dims[2] = {static_cast<uint64_t>(g.K), static_cast<uint64_t>(g.N)};
        uint64_t str[1] = {static_cast<uint64_t>(g.K) * 2};
        uint32_t box[2] = {64, static_cast<uint32_t>(p.tiles ? 64 : cfg.tile_n)};
        rc = get_tensor_map(ctx, B, 2, dims, str, box, &mb);
    }
    if (rc) return rc;

    CUtensorMap mc = ma;   // unused unless the staged epilogue is on
    // the accumulate term is read by the direct-store epilogue (and by the split-K reduction) only
    p.tma_store = (cfg.store_mode == 2 && cfg.split_k == 1 && p.vec_store && beta == 0.0f) ? 1 : 0;
    if (p.tma_store) {
        uint64_t dims[2] = {static_cast<uint64_t>(g.N), static_cast<uint64_t>(g.M)};
        uint64_t str[1] = {static_cast<uint64_t>(g.N) * 2};
        uint32_t box[2] = {32, 32};
        rc = get_tensor_map(ctx, C, 2, dims, str, box, &mc, 64);
        if (rc) return rc;
    }
    rc = launch_umma(ctx, false, ma, mb, mc, p, st, false, nullptr, nullptr, plan_grid);
    if (rc) return rc;
    if (cfg.split_k > 1) {
        const long long MN = static_cast<long long>(g.M) * g.N;
        const int vec8 = p.vec_store ? 1 : 0;
        const long long work = vec8 ? MN / 8 : MN;
        const int grid = static_cast<int>(std::min<long long>(ceil_div(work, 256), 148LL * 16));
        rc = launch_splitk_reduce(std::max(grid, 1), st, MN, static_cast<int>(g.N), cfg.split_k, p.partial, alpha, p.C, vec8, beta);
        if (rc) return rc;
    }
    return TDX_OK;
}

// GEMM on CTA pairs: 256 x tile_n per pair, each CTA loads its 128 rows of A and tile_n / 2 columns of B.
int run_gemm_pair(DeviceCtx* ctx, const GemmProblem& g, float alpha, const void* A, const void* B, void* C,
                  const tdx_config& cfg, cudaStream_t st) {
    const int64_t num_kb = ceil_div(g.K, 64);
    UmmaParams p;
    std::memset(&p, 0, sizeof p);
    p.M = static_cast<int>(g.M);
    p.N = static_cast<int>(g.N);
    p.num_kb = static_cast<int>(num_kb);
    p.bm = 128;                                      // what one CTA of the pair owns (epilogue geometry)
    p.slots = 2 * cfg.tile_n <= 256 ? 4 : 2;
    p.tiles_m = static_cast<int>(ceil_div(g.M, 256));
    p.tiles_n = static_cast<int>(ceil_div(g.N, cfg.tile_n));
    p.panel = cfg.raster == 0 ? p.tiles_m : std::min(cfg.raster, p.tiles_m);
    p.split_k = 1;
    p.kb_per_split = p.num_kb;
    p.bn = cfg.tile_n;
    p.stages = cfg.stages;
    p.tmem_cols = 32;
    while (p.tmem_cols < p.slots * cfg.tile_n) p.tmem_cols *= 2;
    p.a_mn_major = g.transA ? 1 : 0;
    p.b_mn_major = g.transB ? 0 : 1;
    p.alpha = alpha;
    p.C = static_cast<__nv_bfloat16*>(C);
    p.ldc = g.N;
    p.status = ctx->status_ptr;
    p.vec_store = (g.N % 8 == 0) && (reinterpret_cast<uintptr_t>(C) % 16 == 0);
    p.tma_store = (cfg.store_mode == 2 && p.vec_store) ? 1 : 0;

    CUtensorMap ma, mb, mc;
    int rc;
    if (p.a_mn_major) {
        uint64_t dims[2] = {static_cast<uint64_t>(g.M), static_cast<uint64_t>(g.K)};
        uint64_t str[1] = {static_cast<uint64_t>(g.M) * 2};
        uint32_t box[2] = {64, 64};
        rc = get_tensor_map(ctx, A, 2, dims, str, box, &ma);
    } else {
        uint64_t dims[2] = {static_cast<uint64_t>(g.K), static_cast<uint64_t>(g.M)};
        uint64_t str[1] = {static_cast<uint64_t>(g.K) * 2};
        uint32_t box[2] = {64, 128};
        rc = get_tensor_map(ctx, A, 2, dims, str, box, &ma);
    }
    if (rc) return rc;
    // tile widths fitted to the number of pairs; each CTA's half of a tile's B columns then arrives in 64-row copies
    // (K-major B only: an N-major half would have to be a multiple of 64 columns)
    p.b_box = cfg.tile_n / 2;
    int plan_pairs = 0;
    // only on request: a 256 x 128 x 16 pair MMA measured 115 cycles, not 64, so narrow tiles gain nothing here
    if (cfg.fit == 2 && !p.b_mn_major && cfg.tile_n >= 192 && cfg.tile_n % 64 == 0) {
        DevicePlan dp;
        rc = get_tile_plan(ctx, g.M, g.N, num_kb, 256, cfg.tile_n, cfg.raster, 0.0, st, &dp, true);
        if (rc) return rc;
        if (dp.fitted) {
            p.tiles = dp.dev;
            p.rounds = dp.rounds;
            p.b_box = 64;
            plan_pairs = dp.grid;
        }
    }
    if (p.b_mn_major) {
        uint64_t dims[2] = {static_cast<uint64_t>(g.N), static_cast<uint64_t>(g.K)};
        uint64_t str[1] = {static_cast<uint64_t>(g.N) * 2};
        uint32_t box[2] = {64, 64};
        rc = get_tensor_map(ctx, B, 2, dims, str, box, &mb);
    } else {
        uint64_t dims[2] = {static_cast<uint64_t>(g.K), static_cast<uint64_t>(g.N)};
        uint64_t str[1] = {static_cast<uint64_t>(g.K) * 2};
        uint32_t box[2] = {64, static_cast<uint32_t>(p.b_box)};
        rc = get_tensor_map(ctx, B, 2, dims, str, box, &mb);
    }
    if (rc) return rc;
    mc = ma;
    if (p.tma_store) {
        uint64_t dims[2] = {static_cast<uint64_t>(g.N), static_cast<uint64_t>(g.M)};
        uint64_t str[1] = {static_cast<uint64_t>(g.N) * 2};
        uint32_t box[2] = {32, 32};
        rc = get_tensor_map(ctx, C, 2, dims, str, box, &mc, 64);
        if (rc) return rc;
    }
    const long long pair_tiles = static_cast<long long>(p.tiles_m) * p.tiles_n;
    const int pairs = p.tiles ? plan_pairs : static_cast<int>(std::min<long long>(pair_tiles, ctx->sm_count / 2));
    cudaLaunchConfig_t lc;
    std::memset(&lc, 0, sizeof lc);
    lc.gridDim = dim3(static_cast<unsigned>(2 * pairs));
    lc.blockDim = dim3(p.tma_store ? 576 : 192);
    lc.dynamicSmemBytes = static_cast<size_t>(p.stages) * ((128 + p.bn / 2) * 128) + 1024 +
                          staging_bytes_for(128, p.tma_store ? 2 : 1);
    lc.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    TDX_CUDA(cudaLaunchKernelEx(&lc, tdx::umma_pair_kernel, ma, mb, mc, p));
    g_launches.fetch_add(1);
    return TDX_OK;
}

int run_conv_umma(DeviceCtx* ctx, const ConvProblem& c, const void* x, const void* w, const float* bias, int relu,
                  void* y, const tdx_config& cfg, cudaStream_t st, const void* residual = nullptr) {
    const int cchunks = static_cast<int>(ceil_div(c.Cin, 64));
    UmmaParams p;
    std::memset(&p, 0, sizeof p);
    p.bw = cfg.patch_w;
    p.bh = cfg.patch_h;
    p.bm = cfg.tile_m;
    p.slots = tmem_slots_for(cfg.tile_m, cfg.tile_n);
    p.nb = cfg.tile_m / (p.bw * p.bh);
    const bool halo = cfg.halo >= 2;
    const bool stacked = cfg.halo == 3;
    if (halo) {
        p.R = static_cast<int>(c.R);
        p.hpitch = static_cast<int>(kHaloPatchW + c.S - 1);
        p.hrows = static_cast<int>(kHaloPatchH + c.R - 1);
        p.halo_bytes = halo_tile_bytes(c.R, c.S);
        p.a_stages = kHaloAStages;
    }
    p.patches_w = static_cast<int>(ceil_div(c.Q, p.bw));
    p.patches_h = static_cast<int>(ceil_div(c.P, p.bh));
    int64_t total_patches = c.N * p.patches_w * p.patches_h;
    if (stacked) {
        p.Pv = static_cast<int>(stacked_rows_per_image(c));
        p.H = static_cast<int>(c.H);
        p.patches_h = static_cast<int>(ceil_div(c.N * p.Pv, p.bh));      // over the whole column of images
        total_patches = static_cast<int64_t>(p.patches_w) * p.patches_h;
    }
    p.M = static_cast<int>(c.N * c.P * c.Q);
    p.N = static_cast<int>(c.Cout);
    p.num_kb = static_cast<int>(c.R * c.S * cchunks);
    p.tiles_m = static_cast<int>(ceil_div(total_patches, p.nb));
    p.tiles_n = static_cast<int>(ceil_div(c.Cout, cfg.tile_n));
    p.panel = cfg.raster == 0 ? p.tiles_m : std::min(cfg.raster, p.tiles_m);
    p.split_k = 1;
    p.kb_per_split = p.num_kb;
    p.k_stagger = cfg.k_stagger;
    p.bn = cfg.tile_n;
    p.stages = cfg.stages;
    if (halo && cfg.tile_n >= c.Cout) {
        // small filters stay resident: all (chunk, tap) slices of the one column tile fit beside the halo ring,
        // so they are loaded once per CTA and the main loop has no per-tap handshake
        const int64_t slices = c.R * c.S * cchunks;
        const int64_t need = static_cast<int64_t>(p.a_stages) * (cfg.tile_m / 128) * p.halo_bytes + slices * cfg.tile_n * 128 +
                             staging_bytes_for(cfg.tile_m, cfg.store_mode) + 1024;
        if (need <= ctx->smem_optin - kStaticSmemReserve) {
            p.b_resident = 1;
            p.stages = static_cast<int>(slices);
            // spend what is left on more halo tiles in flight (their load latency is what a short tile waits for)
            const int64_t per_stage = static_cast<int64_t>(cfg.tile_m / 128) * p.halo_bytes;
            while (p.a_stages < tdx::kMaxAStages && need + (p.a_stages - kHaloAStages + 1) * per_stage <= ctx->smem_optin - kStaticSmemReserve)
                ++p.a_stages;
        }
    }
    p.tmem_cols = tmem_cols_for(cfg.tile_m, cfg.tile_n);
    p.a_mn_major = 0;
    p.b_mn_major = 0;
    p.alpha = 1.0f;
    p.bias = bias;
    p.residual = static_cast<const __nv_bfloat16*>(residual);
    p.relu = relu;
    p.C = static_cast<__nv_bfloat16*>(y);
    p.ldc = c.Cout;
    p.vec_store = (c.Cout % 8 == 0) && (reinterpret_cast<uintptr_t>(y) % 16 == 0);
    p.P = static_cast<int>(c.P);
    p.Q = static_cast<int>(c.Q);
    p.Nimg = static_cast<int>(c.N);
    p.S = static_cast<int>(c.S);
    p.pad = c.pad;
    p.stride = c.stride;
    p.cchunks = cchunks;
    p.status = ctx->status_ptr;

    CUtensorMap ma, ma_row, mb;
    {
        uint64_t dims[4] = {static_cast<uint64_t>(c.Cin), static_cast<uint64_t>(c.W), static_cast<uint64_t>(c.H),
                            static_cast<uint64_t>(c.N)};
        uint64_t str[3] = {static_cast<uint64_t>(c.Cin) * 2, static_cast<uint64_t>(c.W * c.Cin) * 2,
                           static_cast<uint64_t>(c.H * c.W * c.Cin) * 2};
        uint32_t box[4] = {64, static_cast<uint32_t>(halo ? p.hpitch : p.bw), static_cast<uint32_t>(halo ? p.hrows : p.bh), 1};
        // strided convolution (per-tap loads only): the copy walks the image with the convolution's stride, so a
        // box spanning bw * stride input pixels delivers exactly the bw pixels under one filter tap
        uint32_t estr[4] = {1, static_cast<uint32_t>(c.stride), static_cast<uint32_t>(c.stride), 1};
        if (c.stride > 1) { box[1] *= c.stride; box[2] *= c.stride; }
        int rc = get_tensor_map(ctx, x, 4, dims, str, box, &ma, 128, c.stride > 1 ? estr : nullptr);
        if (rc) return rc;
        ma_row = ma;
        if (stacked) {
            box[2] = 1;              // windows that reach into the next image are copied one row at a time
            rc = get_tensor_map(ctx, x, 4, dims, str, box, &ma_row);
            if (rc) return rc;
        }
    }
    {
        uint64_t dims[3] = {static_cast<uint64_t>(c.Cin), static_cast<uint64_t>(c.R * c.S),
                            static_cast<uint64_t>(c.Cout)};
        uint64_t str[2] = {static_cast<uint64_t>(c.Cin) * 2, static_cast<uint64_t>(c.R * c.S * c.Cin) * 2};
        uint32_t box[3] = {64, 1, static_cast<uint32_t>(cfg.tile_n)};
        int rc = get_tensor_map(ctx, w, 3, dims, str, box, &mb);
        if (rc) return rc;
    }
    CUtensorMap mc = ma, mc_row = ma;
    p.tma_store = (cfg.store_mode == 2 && p.vec_store && p.bw * p.bh >= 32) ? 1 : 0;
    // the staged epilogue reads the residual 16 bytes at a time
    if (reinterpret_cast<uintptr_t>(residual) % 16) p.tma_store = 0;
    if (halo) p.epi_warps = p.tma_store ? 16 : 4 * (cfg.tile_m / 128);
    if (p.tma_store) {
        p.sbx = std::min(p.bw, 32);
        p.sby = 32 / p.sbx;
        uint64_t dims[4] = {static_cast<uint64_t>(c.Cout), static_cast<uint64_t>(c.Q), static_cast<uint64_t>(c.P),
                            static_cast<uint64_t>(c.N)};
        uint64_t str[3] = {static_cast<uint64_t>(c.Cout) * 2, static_cast<uint64_t>(c.Q * c.Cout) * 2,
                           static_cast<uint64_t>(c.P * c.Q * c.Cout) * 2};
        uint32_t box[4] = {32, static_cast<uint32_t>(p.sbx), static_cast<uint32_t>(p.sby), 1};
        int rc = get_tensor_map(ctx, y, 4, dims, str, box, &mc, 64);
        if (rc) return rc;
        mc_row = mc;
        if (stacked) {
            box[2] = 1;              // four pixel rows that cross the seam between two images leave one by one
            rc = get_tensor_map(ctx, y, 4, dims, str, box, &mc_row, 64);
            if (rc) return rc;
        }
    }
    return launch_umma(ctx, true, ma, mb, mc, p, st, halo, &ma_row, &mc_row);
}

void gemm_strides(const GemmProblem& g, long long* sa_i, long long* sa_k, long long* sb_k, long long* sb_j) {
    *sa_i = g.transA ? 1 : g.K;
    *sa_k = g.transA ? g.M : 1;
    *sb_k = g.transB ? 1 : g.N;
    *sb_j = g.transB ? g.K : 1;
}

// batch count, batch strides in elements, and the accumulate factor of tdx_gemm_batched (one batch, beta = 0: tdx_gemm)
struct BatchArgs {
    int64_t batch = 1, stride_a = 0, stride_b = 0, stride_c = 0;
    float beta = 0.0f;
};

int run_gemm_simt_f32(DeviceCtx* ctx, const GemmProblem& g, float alpha, const void* A, const void* B, void* C,
                      cudaStream_t st, const BatchArgs& ba = BatchArgs()) {
    if (g.M >= (1LL << 31) || g.N >= (1LL << 31) || g.K >= (1LL << 31))
        return fail(TDX_ERR_UNSUPPORTED, "fp32 tiled GEMM needs dimensions below 2^31");
    long long sa_i, sa_k, sb_k, sb_j;
    gemm_strides(g, &sa_i, &sa_k, &sb_k, &sb_j);
    const float* a = static_cast<const float*>(A);
    const float* b = static_cast<const float*>(B);
    float* c = static_cast<float*>(C);
    if (ba.batch > 65535) return fail(TDX_ERR_UNSUPPORTED, "fp32 batched GEMM takes at most 65535 batches");
    const unsigned nz = static_cast<unsigned>(ba.batch);
    const bool plain = ba.batch == 1 && ba.beta == 0.0f;
    const int64_t tiles64 = ceil_div(g.M, 64) * ceil_div(g.N, 64) * ba.batch;
    if (tiles64 >= ctx->sm_count) {
        // 64 x 64 tiles (4 x 4 outputs per thread) once there is one per SM; smaller problems take 32 x 32 tiles
        dim3 grid(static_cast<unsigned>(ceil_div(g.N, 64)), static_cast<unsigned>(ceil_div(g.M, 64)), nz);
        tdx::sgemm_ring_kernel<64, 64, 16, 4, 4, 4><<<grid, 256, 0, st>>>((int)g.M, (int)g.N, (int)g.K, sa_i, sa_k, sb_k,
                                                                         sb_j, alpha, a, b, c, ba.beta, ba.stride_a,
                                                                         ba.stride_b, ba.stride_c);
    } else {
        dim3 grid(static_cast<unsigned>(ceil_div(g.N, 32)), static_cast<unsigned>(ceil_div(g.M, 32)), nz);
        const bool rowmajor16 = plain && !g.transA && !g.transB && g.K % 4 == 0 && g.N % 4 == 0 &&
                                reinterpret_cast<uintptr_t>(A) % 16 == 0 && reinterpret_cast<uintptr_t>(B) % 16 == 0;
        if (rowmajor16)
            tdx::sgemm_small_rowmajor_kernel<<<grid, 256, 0, st>>>((int)g.M, (int)g.N, (int)g.K, alpha, a, b, c);
        else
            tdx::sgemm_small_kernel<<<grid, 256, 0, st>>>((int)g.M, (int)g.N, (int)g.K, sa_i, sa_k, sb_k, sb_j, alpha, a, b,
                                                          c, ba.beta, ba.stride_a, ba.stride_b, ba.stride_c);
    }
    TDX_CUDA(cudaGetLastError());
    g_launches.fetch_add(1);
    return TDX_OK;
}

int run_gemm_generic(DeviceCtx* ctx, const GemmProblem& g, float alpha, const void* A, const void* B, void* C,
                     cudaStream_t st, const BatchArgs& ba = BatchArgs()) {
    long long sa_i, sa_k, sb_k, sb_j;
    gemm_strides(g, &sa_i, &sa_k, &sb_k, &sb_j);
    const long long total = g.M * g.N * ba.batch;
    const int grid = static_cast<int>(std::min<long long>(ceil_div(total, 256), static_cast<long long>(ctx->sm_count) * 32));
    if (g.dtype == TDX_F32)
        tdx::gemm_generic_kernel<float, float><<<grid, 256, 0, st>>>(g.M, g.N, g.K, sa_i, sa_k, sb_k, sb_j, alpha,
                                                                    static_cast<const float*>(A),
                                                                    static_cast<const float*>(B), static_cast<float*>(C),
                                                                    ba.beta, ba.batch, ba.stride_a, ba.stride_b, ba.stride_c);
    else
        tdx::gemm_generic_kernel<__nv_bfloat16, __nv_bfloat16><<<grid, 256, 0, st>>>(
            g.M, g.N, g.K, sa_i, sa_k, sb_k, sb_j, alpha, static_cast<const __nv_bfloat16*>(A),
            static_cast<const __nv_bfloat16*>(B), static_cast<__nv_bfloat16*>(C), ba.beta, ba.batch, ba.stride_a,
            ba.stride_b, ba.stride_c);
    TDX_CUDA(cudaGetLastError());
    g_launches.fetch_add(1);
    return TDX_OK;
}

int run_conv_generic(DeviceCtx* ctx, const ConvProblem& c, const void* x, const void* w, const float* bias, int relu,
                     void* y, cudaStream_t st, const void* residual = nullptr) {
    if (c.N >= (1LL << 31) || c.H >= (1LL << 31) || c.W >= (1LL << 31) || c.Cin >= (1LL << 31) ||
        c.Cout >= (1LL << 31) || c.R >= (1LL << 31) || c.S >= (1LL << 31))
        return fail(TDX_ERR_UNSUPPORTED, "conv dimensions must be below 2^31");
    const long long total = c.N * c.P * c.Q * c.Cout;
    const int grid = static_cast<int>(std::min<long long>(ceil_div(total, 256), static_cast<long long>(ctx->sm_count) * 32));
    if (c.dtype == TDX_F32)
        tdx::conv2d_generic_kernel<float, float><<<grid, 256, 0, st>>>(
            (int)c.N, (int)c.H, (int)c.W, (int)c.Cin, (int)c.Cout, (int)c.R, (int)c.S, c.pad, c.stride, (int)c.P,
            (int)c.Q, static_cast<const float*>(x), static_cast<const float*>(w), bias, relu, static_cast<float*>(y),
            static_cast<const float*>(residual));
    else
        tdx::conv2d_generic_kernel<__nv_bfloat16, __nv_bfloat16><<<grid, 256, 0, st>>>(
            (int)c.N, (int)c.H, (int)c.W, (int)c.Cin, (int)c.Cout, (int)c.R, (int)c.S, c.pad, c.stride, (int)c.P,
            (int)c.Q, static_cast<const __nv_bfloat16*>(x), static_cast<const __nv_bfloat16*>(w), bias, relu,
            static_cast<__nv_bfloat16*>(y), static_cast<const __nv_bfloat16*>(residual));
    TDX_CUDA(cudaGetLastError());
    g_launches.fetch_add(1);
    return TDX_OK;
}

// ------------------------------------------------------------------ validation
int validate_gemm(int64_t M, int64_t N, int64_t K, int transA, int transB, int dtype, const void* A, const void* B,
                  const void* C, bool need_ptrs) {
    if (M < 0 || N < 0 || K < 0) return fail(TDX_ERR_INVALID_ARG, "negative dimension (M=%lld N=%lld K=%lld)", (long long)M, (long long)N, (long long)K);
    if ((transA != 0 && transA != 1) || (transB != 0 && transB != 1)) return fail(TDX_ERR_INVALID_ARG, "transA/transB must be 0 or 1");
    if (dtype != TDX_F32 && dtype != TDX_BF16) return fail(TDX_ERR_INVALID_ARG, "unknown dtype %d", dtype);
    if (need_ptrs && M > 0 && N > 0) {
        if (C == nullptr) return fail(TDX_ERR_INVALID_ARG, "C is NULL");
        if (K > 0 && (A == nullptr || B == nullptr)) return fail(TDX_ERR_INVALID_ARG, "A or B is NULL");
        const uintptr_t el = dtype == TDX_F32 ? 4 : 2;
        if (reinterpret_cast<uintptr_t>(A) % el || reinterpret_cast<uintptr_t>(B) % el || reinterpret_cast<uintptr_t>(C) % el)
            return fail(TDX_ERR_ALIGNMENT, "pointer not aligned to its element size");
    }
    return TDX_OK;
}

int validate_conv(int64_t N, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int64_t R, int64_t S, int pad,
                  int stride, int dtype, const void* x, const void* w, const void* y, int relu, bool need_ptrs,
                  ConvProblem* out) {
    if (N < 0 || H < 0 || W < 0 || Cout < 0 || pad < 0) return fail(TDX_ERR_INVALID_ARG, "negative dimension or pad");
    if (Cin <= 0 || R <= 0 || S <= 0) return fail(TDX_ERR_INVALID_ARG, "Cin, R and S must be positive");
    if (stride < 1) return fail(TDX_ERR_INVALID_ARG, "stride must be >= 1");
    if (dtype != TDX_F32 && dtype != TDX_BF16) return fail(TDX_ERR_INVALID_ARG, "unknown dtype %d", dtype);
    if (relu != 0 && relu != 1) return fail(TDX_ERR_INVALID_ARG, "relu must be 0 or 1");
    ConvProblem c{N, H, W, Cin, Cout, R, S, pad, stride, dtype, conv_out_dim(H, R, pad, stride), conv_out_dim(W, S, pad, stride)};
    if (need_ptrs && N > 0 && Cout > 0 && c.P > 0 && c.Q > 0) {
        if (x == nullptr || w == nullptr || y == nullptr) return fail(TDX_ERR_INVALID_ARG, "x, w or y is NULL");
        const uintptr_t el = dtype == TDX_F32 ? 4 : 2;
        if (reinterpret_cast<uintptr_t>(x) % el || reinterpret_cast<uintptr_t>(w) % el || reinterpret_cast<uintptr_t>(y) % el)
            return fail(TDX_ERR_ALIGNMENT, "pointer not aligned to its element size");
    }
    *out = c;
    return TDX_OK;
}

// Fill the zero fields of a (possibly partial) GEMM config and check it.  smem_limit / sm_count come from the
// device when there is one, else from the sm_100 defaults, so the search space can be listed without a GPU.
int resolve_gemm_config(const GemmProblem& g, const tdx_config* user, int sm_count, int smem_limit, tdx_config* out) {
    const bool layout_ok = gemm_umma_layout_ok(g);
    tdx_config c;
    std::memset(&c, 0, sizeof c);
    if (user) c = *user;
    if (c.kernel < 0 || c.kernel > 3) return fail(TDX_ERR_CONFIG, "unknown kernel %d", c.kernel);
    bool from_cache = false;
    if (c.kernel == TDX_KERNEL_AUTO) {
        if (!user) {
            tdx_config cached;
            if (tune_lookup(gemm_key(g.M, g.N, g.K, g.transA, g.transB, g.dtype), &cached)) { c = cached; from_cache = true; }
        }
        if (!from_cache) c.kernel = g.dtype == TDX_F32 ? TDX_KERNEL_SIMT : (layout_ok ? TDX_KERNEL_UMMA : TDX_KERNEL_GENERIC);
    }
    if (c.kernel == TDX_KERNEL_SIMT) {
        if (g.dtype != TDX_F32) return fail(TDX_ERR_CONFIG, "the tiled SIMT kernel is fp32 only");
        *out = c;
        return TDX_OK;
    }
    if (c.kernel == TDX_KERNEL_GENERIC) { *out = c; return TDX_OK; }
    // tensor-core path
    if (g.dtype != TDX_BF16) return fail(TDX_ERR_CONFIG, "the tensor-core kernel is bf16 only");
    if (!layout_ok) return fail(TDX_ERR_ALIGNMENT, "tensor-core path needs 16-byte aligned row pitches (contiguous dims %% 8 == 0)");
    const int64_t num_kb = ceil_div(g.K, 64);
    const bool b_mn = g.transB == 0;
    tdx_config d;
    default_umma_config(ceil_div(g.M, 128), g.N, num_kb, b_mn, sm_count, smem_limit, true, &d);
    if (c.tile_m == 0) c.tile_m = c.cta_pair == 2 ? 256 : ((c.tile_n == 0 || c.tile_n == d.tile_n) ? d.tile_m : 128);
    if (c.tile_k == 0) c.tile_k = d.tile_k;
    if (c.cta_pair == 0) c.cta_pair = d.cta_pair;
    if (c.tile_n == 0) c.tile_n = d.tile_n;
    if (c.split_k == 0) c.split_k = (user && user->cta_pair == 2) ? 1 : (user && user->tile_n != 0 && user->tile_n != d.tile_n) ? 1 : d.split_k;
    if (c.store_mode == 0) {
        c.store_mode = (c.split_k == 1 && g.N % 8 == 0) ? 2 : 1;
        if (c.store_mode == 2 && c.cta_pair != 2 && c.stages > umma_max_stages(c.tile_m, c.tile_n, smem_limit, 2)) c.store_mode = 1;
    }
    if (c.stages == 0)
        c.stages = c.cta_pair == 2 ? std::max(2, pair_max_stages(c.tile_n, smem_limit, c.store_mode))
                                   : std::max(2, umma_max_stages(c.tile_m, c.tile_n, smem_limit, c.store_mode));
    if (!user && !from_cache) c.raster = d.raster;
    const char* why = umma_config_reason(c, b_mn, num_kb, smem_limit, false, g.N);
    if (why) return fail(TDX_ERR_CONFIG, "infeasible config: %s", why);
    *out = c;
    return TDX_OK;
}

int resolve_conv_config(const ConvProblem& cp, const tdx_config* user, int sm_count, int smem_limit, tdx_config* out) {
    const bool layout_ok = conv_umma_layout_ok(cp);
    tdx_config c;
    std::memset(&c, 0, sizeof c);
    if (user) c = *user;
    if (c.kernel < 0 || c.kernel > 3) return fail(TDX_ERR_CONFIG, "unknown kernel %d", c.kernel);
    if (c.kernel == TDX_KERNEL_SIMT) return fail(TDX_ERR_CONFIG, "conv has no tiled SIMT kernel");
    bool from_cache = false;
    if (c.kernel == TDX_KERNEL_AUTO) {
        if (!user) {
            tdx_config cached;
            if (tune_lookup(conv_key(cp.N, cp.H, cp.W, cp.Cin, cp.Cout, cp.R, cp.S, cp.pad, cp.stride, cp.dtype), &cached)) { c = cached; from_cache = true; }
        }
        if (!from_cache) c.kernel = layout_ok ? TDX_KERNEL_UMMA : TDX_KERNEL_GENERIC;
    }
    if (c.kernel == TDX_KERNEL_GENERIC) { *out = c; return TDX_OK; }
    if (cp.dtype != TDX_BF16) return fail(TDX_ERR_CONFIG, "the tensor-core kernel is bf16 only");
    if (!layout_ok) return fail(TDX_ERR_ALIGNMENT, "tensor-core conv needs stride <= 8 and Cin %% 8 == 0");
    const bool halo_auto = c.halo == 0 && !from_cache;
    if (c.halo == 0) {
        // halo reuse unless its fixed 8 x 16 patches waste much more of the image than the best free patch shape
        c.halo = 1;
        if (cp.stride == 1 && cp.R * cp.S > 1 && c.patch_w == 0 && c.patch_h == 0) {
            int bw, bh;
            choose_patch(cp.P, cp.Q, &bw, &bh);
            const int64_t best = ceil_div(cp.Q, bw) * bw * ceil_div(cp.P, bh) * bh;
            const int64_t mine = ceil_div(cp.Q, kHaloPatchW) * kHaloPatchW * ceil_div(cp.P, kHaloPatchH) * kHaloPatchH;
            const int tm = c.tile_m ? c.tile_m : 128, tn = c.tile_n ? c.tile_n : 64;
            if (halo_max_stages(tm, tn, cp.R, cp.S, smem_limit, 2) >= 2) {
                // patches cut from the stacked column of images when that leaves fewer padded rows
                if (halo_patches(cp, 3) < halo_patches(cp, 2)) c.halo = 3;
                else if (mine * 100 <= best * 120) c.halo = 2;
            }
        }
    }
    if (c.halo >= 2 && c.patch_w == 0 && c.patch_h == 0) { c.patch_w = kHaloPatchW; c.patch_h = kHaloPatchH; }
    if (c.patch_w == 0 && c.patch_h == 0) choose_patch(cp.P, cp.Q, &c.patch_w, &c.patch_h, cp.stride);
    if (!patch_ok(c.patch_w, c.patch_h)) return fail(TDX_ERR_CONFIG, "infeasible config: patch %dx%d", c.patch_w, c.patch_h);
    const int nb = 128 / (c.patch_w * c.patch_h);
    const int64_t tiles_m = c.halo >= 2 ? halo_patches(cp, c.halo)
                                        : ceil_div(cp.N * ceil_div(cp.Q, c.patch_w) * ceil_div(cp.P, c.patch_h), nb);
    const int64_t num_kb = cp.R * cp.S * ceil_div(cp.Cin, 64);
    tdx_config d;
    default_umma_config(tiles_m, cp.Cout, num_kb, false, sm_count, smem_limit, false, &d);
    if (c.tile_m == 0) c.tile_m = (c.tile_n == 0 || c.tile_n == d.tile_n) ? d.tile_m : 128;
    if (c.tile_k == 0) c.tile_k = d.tile_k;
    if (c.cta_pair == 0) c.cta_pair = d.cta_pair;
    if (c.tile_n == 0) c.tile_n = d.tile_n;
    if (c.split_k == 0) c.split_k = 1;
    if (c.store_mode == 0) {
        c.store_mode = (cp.Cout % 8 == 0 && c.patch_w * c.patch_h >= 32) ? 2 : 1;
        if (c.store_mode == 2 && c.halo < 2 && c.stages > umma_max_stages(c.tile_m, c.tile_n, smem_limit, 2)) c.store_mode = 1;
    }
    if (c.stages == 0)
        c.stages = c.halo >= 2 ? std::max(2, halo_max_stages(c.tile_m, c.tile_n, cp.R, cp.S, smem_limit, c.store_mode))
                               : std::max(2, umma_max_stages(c.tile_m, c.tile_n, smem_limit, c.store_mode));
    if (!user && !from_cache) c.raster = d.raster;
    const char* why = umma_config_reason(c, false, num_kb, smem_limit, true, cp.Cout, cp.R, cp.S, cp.stride);
    if (why && halo_auto && c.halo >= 2) {
        // the automatic choice of halo reuse did not fit (large filter): fall back to per-tap loads
        tdx_config retry;
        std::memset(&retry, 0, sizeof retry);
        if (user) retry = *user;
        retry.halo = 1;
        return resolve_conv_config(cp, &retry, sm_count, smem_limit, out);
    }
    if (why) return fail(TDX_ERR_CONFIG, "infeasible config: %s", why);
    *out = c;
    return TDX_OK;
}

void device_limits(int* sm_count, int* smem_limit) {
    *sm_count = kDefaultSmCount;
    *smem_limit = kSmemLimitDefault;
    int dev;
    if (cudaGetDevice(&dev) == cudaSuccess) {
        std::lock_guard<std::mutex> lk(g_mu);
        auto it = g_ctx.find(dev);
        if (it != g_ctx.end()) { *sm_count = it->second.sm_count; *smem_limit = it->second.smem_optin; }
    } else {
        cudaGetLastError();
    }
}

int gemm_dispatch(int64_t M, int64_t N, int64_t K, int transA, int transB, float alpha, int dtype, const void* A,
                  const void* B, void* C, void* stream, const tdx_config* cfg, void* ws, size_t ws_bytes,
                  bool internal_ws) {
    int rc = validate_gemm(M, N, K, transA, transB, dtype, A, B, C, true);
    if (rc) return rc;
    if (M == 0 || N == 0) return TDX_OK;
    GemmProblem g{M, N, K, transA, transB, dtype};
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (K == 0) {
        DeviceCtx* ctx0;
        rc = get_ctx(&ctx0);
        if (rc) return rc;
        TDX_CUDA(cudaMemsetAsync(C, 0, static_cast<size_t>(M) * N * (dtype == TDX_F32 ? 4 : 2), st));
        return TDX_OK;
    }
    int sm_count, smem_limit;
    device_limits(&sm_count, &smem_limit);
    // configuration errors are reported before anything touches the device
    tdx_config pre;
    if (cfg) {
        rc = resolve_gemm_config(g, cfg, sm_count, smem_limit, &pre);
        if (rc) return rc;
    }
    DeviceCtx* ctx;
    rc = get_ctx(&ctx);
    if (rc) return rc;
    tdx_config c;
    rc = resolve_gemm_config(g, cfg, ctx->sm_count, ctx->smem_optin, &c);
    if (rc) return rc;
    switch (c.kernel) {
        case TDX_KERNEL_SIMT: return run_gemm_simt_f32(ctx, g, alpha, A, B, C, st);
        case TDX_KERNEL_GENERIC: return run_gemm_generic(ctx, g, alpha, A, B, C, st);
        default:
            if (reinterpret_cast<uintptr_t>(A) % 16 || reinterpret_cast<uintptr_t>(B) % 16) {
                if (cfg && cfg->kernel == TDX_KERNEL_UMMA)
                    return fail(TDX_ERR_ALIGNMENT, "tensor-core path needs 16-byte aligned A and B");
                return run_gemm_generic(ctx, g, alpha, A, B, C, st);
            }
            if (c.cta_pair == 2) return run_gemm_pair(ctx, g, alpha, A, B, C, c, st);
            return run_gemm_umma(ctx, g, alpha, A, B, C, c, ws, ws_bytes, internal_ws, st);
    }
}

int conv_dispatch(int64_t N, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int64_t R, int64_t S, int pad, int stride,
                  int dtype, const void* x, const void* w, const float* bias, int relu, void* y, void* stream,
                  const tdx_config* cfg, const void* residual = nullptr) {
    ConvProblem cp;
    int rc = validate_conv(N, H, W, Cin, Cout, R, S, pad, stride, dtype, x, w, y, relu, true, &cp);
    if (rc) return rc;
    if (reinterpret_cast<uintptr_t>(residual) % (dtype == TDX_F32 ? 4 : 2))
        return fail(TDX_ERR_ALIGNMENT, "residual not aligned to its element size");
    if (N == 0 || Cout == 0 || cp.P == 0 || cp.Q == 0) return TDX_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int sm_count, smem_limit;
    device_limits(&sm_count, &smem_limit);
    tdx_config pre;
    if (cfg) {
        rc = resolve_conv_config(cp, cfg, sm_count, smem_limit, &pre);
        if (rc) return rc;
    }
    DeviceCtx* ctx;
    rc = get_ctx(&ctx);
    if (rc) return rc;
    tdx_config c;
    rc = resolve_conv_config(cp, cfg, ctx->sm_count, ctx->smem_optin, &c);
    if (rc) return rc;
    if (c.kernel == TDX_KERNEL_GENERIC) return run_conv_generic(ctx, cp, x, w, bias, relu, y, st, residual);
    if (reinterpret_cast<uintptr_t>(x) % 16 || reinterpret_cast<uintptr_t>(w) % 16) {
        if (cfg && cfg->kernel == TDX_KERNEL_UMMA) return fail(TDX_ERR_ALIGNMENT, "tensor-core path needs 16-byte aligned x and w");
        return run_conv_generic(ctx, cp, x, w, bias, relu, y, st, residual);
    }
    return run_conv_umma(ctx, cp, x, w, bias, relu, y, c, st, residual);
}

// ------------------------------------------------------------------ search space
void enum_umma_space(bool b_mn, int64_t tiles_m, int64_t N, int64_t num_kb, int sm_count, int smem_limit, bool conv,
                     int patch_w, int patch_h, std::vector<tdx_config>* out, int stride = 1) {
    for (int tm : {256, 128}) {
        const int64_t tiles_m_t = ceil_div(tiles_m, tm / 128);
        for (int bn = 256; bn >= 32; bn -= 32) {
            if (b_mn && bn % 64) continue;
            if (bn > 32 && bn - 32 >= N) continue;        // a narrower tile already covers N
            if (bn != 256 && bn != 128 && bn != 64 && bn != 32 && N % bn && ceil_div(N, bn) == ceil_div(N, bn + 32))
                continue;                                 // odd widths only where they change the tile count
            const int64_t tiles = tiles_m_t * ceil_div(N, bn);
            if (tm == 256 && tiles < sm_count / 2) continue;   // too few tiles to be worth the taller tile
            std::vector<int> splits{1};
            if (!conv && tiles < 2LL * sm_count)
                for (int s : {2, 3, 4, 6, 8, 16})
                    if (num_kb / s >= 2 && tiles * s <= 4LL * sm_count) splits.push_back(s);
            for (int sk : splits)
                for (int sm : {2, 1}) {
                    if (sm == 2 && (sk > 1 || N % 8)) continue;
                    if (sm == 1 && sk == 1 && N % 8 == 0 && tiles * tm * bn > (1 << 22))
                        continue;                          // large outputs: 16-byte scattered stores never win
                    const int max_st = umma_max_stages(tm, bn, smem_limit, sm);
                    if (max_st < 2) continue;
                    std::vector<int> stage_opts;
                    stage_opts.push_back(max_st);
                    if (max_st - 2 >= 3) stage_opts.push_back(max_st - 2);
                    for (int st : stage_opts)
                        for (int raster : {0, 8, 2, 4, 16})
                            for (int stagger : {0, 1}) {
                                if (raster != 0 && tiles_m_t <= raster) continue;
                                tdx_config c;
                                std::memset(&c, 0, sizeof c);
                                c.kernel = TDX_KERNEL_UMMA;
                                c.tile_m = tm; c.tile_n = bn; c.tile_k = 64; c.stages = st; c.cta_pair = 1;
                                c.split_k = sk; c.store_mode = sm; c.raster = raster; c.k_stagger = stagger;
                                c.patch_w = patch_w; c.patch_h = patch_h;
                                c.halo = conv ? 1 : 0;
                                c.fit = conv ? 0 : 1;
                                if (umma_config_reason(c, b_mn, num_kb, smem_limit, conv, N, 3, 3, stride) != nullptr) continue;
                                out->push_back(c);
                                if (!conv && sk == 1 && bn >= 192 && bn % 64 == 0 && stagger == 0) {
                                    // the same tile with widths fitted to the CTA count, where that changes anything
                                    TilePlan plan;
                                    if (plan_fitted_tiles(tiles_m * 128, N, num_kb, tm, bn, raster, sm_count, 0.0, &plan)) {
                                        c.fit = 2;
                                        out->push_back(c);
                                    }
                                }
                            }
                }
        }
    }
}

int write_configs(const std::vector<tdx_config>& v, tdx_config* out, int cap, int* n) {
    if (n) *n = static_cast<int>(v.size());
    if (out)
        for (int i = 0; i < cap && i < static_cast<int>(v.size()); ++i) out[i] = v[i];
    return TDX_OK;
}

int enum_gemm(const GemmProblem& g, int sm_count, int smem_limit, std::vector<tdx_config>* v) {
    if (g.dtype == TDX_F32) {
        tdx_config c;
        std::memset(&c, 0, sizeof c);
        c.kernel = TDX_KERNEL_SIMT;
        v->push_back(c);
        return TDX_OK;
    }
    if (!gemm_umma_layout_ok(g)) {
        tdx_config c;
        std::memset(&c, 0, sizeof c);
        c.kernel = TDX_KERNEL_GENERIC;
        v->push_back(c);
        return TDX_OK;
    }
    enum_umma_space(g.transB == 0, ceil_div(g.M, 128), g.N, ceil_div(g.K, 64), sm_count, smem_limit, false, 0, 0, v);
    // CTA-pair candidates: 256 x tile_n per pair
    const bool b_mn = g.transB == 0;
    const int64_t pair_tiles_m = ceil_div(g.M, 256);
    for (int bn : {256, 192, 128}) {
        if (b_mn && bn % 128) continue;
        if (bn - 64 >= g.N) continue;
        if (pair_tiles_m * ceil_div(g.N, bn) < sm_count / 4) continue;
        const int sm = g.N % 8 == 0 ? 2 : 1;
        const int max_st = pair_max_stages(bn, smem_limit, sm);
        for (int stg : {max_st, max_st - 2})
            for (int raster : {0, 8, 2, 4, 16}) {
                if (stg < 2 || (raster != 0 && pair_tiles_m <= raster)) continue;
                tdx_config c;
                std::memset(&c, 0, sizeof c);
                c.kernel = TDX_KERNEL_UMMA;
                c.tile_m = 256; c.tile_n = bn; c.tile_k = 64; c.stages = stg; c.cta_pair = 2; c.split_k = 1;
                c.store_mode = sm; c.raster = raster; c.fit = 1;
                if (umma_config_reason(c, b_mn, ceil_div(g.K, 64), smem_limit, false, g.N) != nullptr) continue;
                v->push_back(c);
                if (!b_mn && bn >= 192 && bn % 64 == 0) {
                    TilePlan plan;
                    if (plan_fitted_tiles(g.M, g.N, ceil_div(g.K, 64), 256, bn, raster, sm_count / 2, 0.0, &plan, true)) {
                        c.fit = 2;
                        v->push_back(c);
                    }
                }
            }
    }
    return TDX_OK;
}

int enum_conv(const ConvProblem& cp, int sm_count, int smem_limit, std::vector<tdx_config>* v) {
    if (!conv_umma_layout_ok(cp)) {
        tdx_config c;
        std::memset(&c, 0, sizeof c);
        c.kernel = TDX_KERNEL_GENERIC;
        v->push_back(c);
        return TDX_OK;
    }
    // halo-reuse candidates (8 x 16 patches)
    if (cp.R * cp.S > 1 && cp.stride == 1) {
        const int64_t num_kb = cp.R * cp.S * ceil_div(cp.Cin, 64);
        for (int mode : {2, 3})
        for (int tm : {256, 128})
            for (int bn = 256; bn >= 32; bn -= 32) {
                if (mode == 3 && halo_patches(cp, 3) >= halo_patches(cp, 2)) continue;   // stacking saves nothing
                if (bn > 32 && bn - 32 >= cp.Cout) continue;
                if (bn != 256 && bn != 128 && bn != 64 && bn != 32 && cp.Cout % bn) continue;
                const int sm = cp.Cout % 8 == 0 ? 2 : 1;
                const int max_st = halo_max_stages(tm, bn, cp.R, cp.S, smem_limit, sm);
                for (int st : {max_st, max_st - 1, max_st - 2}) {
                    if (st < 2) continue;
                    for (int raster : {0, 8, 2}) {
                        tdx_config c;
                        std::memset(&c, 0, sizeof c);
                        c.kernel = TDX_KERNEL_UMMA;
                        c.tile_m = tm; c.tile_n = bn; c.tile_k = 64; c.stages = st; c.cta_pair = 1; c.split_k = 1;
                        c.store_mode = sm; c.raster = raster; c.patch_w = kHaloPatchW; c.patch_h = kHaloPatchH; c.halo = mode;
                        if (umma_config_reason(c, false, num_kb, smem_limit, true, cp.Cout, cp.R, cp.S) == nullptr) v->push_back(c);
                    }
                }
            }
    }
    // patch shapes: every shape whose padded area is within 15 % of the best one
    int bbw, bbh;
    choose_patch(cp.P, cp.Q, &bbw, &bbh, cp.stride);
    const int64_t best_cost = ceil_div(cp.Q, bbw) * bbw * ceil_div(cp.P, bbh) * bbh;
    for (int bw = 8; bw <= 128; bw *= 2)
        for (int bh = 1; bw * bh <= 128; bh *= 2) {
            if (bw * bh < 32 && !(bw == bbw && bh == bbh)) continue;
            const int64_t cost = ceil_div(cp.Q, bw) * bw * ceil_div(cp.P, bh) * bh;
            if (cost * 100 > best_cost * 115) continue;
            const int nb = 128 / (bw * bh);
            const int64_t tiles_m = ceil_div(cp.N * ceil_div(cp.Q, bw) * ceil_div(cp.P, bh), nb);
            if (bw * cp.stride > 256 || bh * cp.stride > 256) continue;
            enum_umma_space(false, tiles_m, cp.Cout, cp.R * cp.S * ceil_div(cp.Cin, 64), sm_count, smem_limit, true, bw, bh,
                            v, cp.stride);
        }
    return TDX_OK;
}

struct ScratchGuard {
    std::vector<void*> ptrs;
    ~ScratchGuard() { for (void* p : ptrs) if (p) cudaFree(p); }
    int alloc(void** p, size_t bytes) {
        cudaError_t e = cudaMalloc(p, std::max<size_t>(bytes, 256));
        if (e != cudaSuccess) { cudaGetLastError(); return fail(TDX_ERR_CUDA, "cudaMalloc(%zu): %s", bytes, cudaGetErrorString(e)); }
        ptrs.push_back(*p);
        return TDX_OK;
    }
};

int fill_scratch(void* p, size_t elems, uint32_t seed, cudaStream_t st) {
    tdx::fill_pattern_bf16_kernel<<<1184, 256, 0, st>>>(static_cast<__nv_bfloat16*>(p), static_cast<long long>(elems), seed);
    TDX_CUDA(cudaGetLastError());
    return TDX_OK;
}

template <typename Launch>
int time_candidates(const std::vector<tdx_config>& cands, int iters, cudaStream_t st, Launch&& launch, tdx_config* best,
                    float* best_us, tdx_config* tried, float* tried_us, int cap, int* n_tried) {
    cudaEvent_t e0, e1;
    TDX_CUDA(cudaEventCreate(&e0));
    TDX_CUDA(cudaEventCreate(&e1));
    float best_t = -1.0f;
    int count = 0;
    int rc = TDX_OK;
    for (const tdx_config& c : cands) {
        rc = launch(c);              // warm-up (also validates the configuration)
        if (rc == TDX_ERR_CONFIG || rc == TDX_ERR_WORKSPACE) { rc = TDX_OK; continue; }
        if (rc) break;
        rc = launch(c);
        if (rc) break;
        cudaEventRecord(e0, st);
        for (int i = 0; i < iters && rc == TDX_OK; ++i) rc = launch(c);
        cudaEventRecord(e1, st);
        if (rc) break;
        cudaError_t e = cudaEventSynchronize(e1);
        if (e != cudaSuccess) { rc = fail(TDX_ERR_CUDA, "tuning launch failed: %s", cudaGetErrorString(e)); break; }
        float ms = 0.0f;
        cudaEventElapsedTime(&ms, e0, e1);
        const float us = ms * 1000.0f / iters;
        if (tried && tried_us && count < cap) { tried[count] = c; tried_us[count] = us; }
        ++count;
        if (best_t < 0 || us < best_t) { best_t = us; *best = c; }
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (rc) return rc;
    if (best_t < 0) return fail(TDX_ERR_UNSUPPORTED, "no feasible configuration");
    if (best_us) *best_us = best_t;
    if (n_tried) *n_tried = count;
    return TDX_OK;
}

int ensure_staging(DeviceCtx* ctx, int slot, size_t bytes, void** out) {
    bytes = std::max<size_t>(bytes, 256);
    if (ctx->staging_bytes[slot] < bytes) {
        if (ctx->staging[slot]) TDX_CUDA(cudaFree(ctx->staging[slot]));
        ctx->staging[slot] = nullptr;
        ctx->staging_bytes[slot] = 0;
        TDX_CUDA(cudaMalloc(&ctx->staging[slot], bytes));
        ctx->staging_bytes[slot] = bytes;
    }
    *out = ctx->staging[slot];
    return TDX_OK;
}

}  // namespace

// ====================================================================== C ABI
extern "C" {

int tdx_gemm(int64_t M, int64_t N, int64_t K, int transA, int transB, float alpha, int dtype, const void* A,
             const void* B, void* C, void* stream) {
    return gemm_dispatch(M, N, K, transA, transB, alpha, dtype, A, B, C, stream, nullptr, nullptr, 0, true);
}

int tdx_gemm_batched(int64_t batch, int64_t M, int64_t N, int64_t K, int transA, int transB, float alpha, float beta,
                     int dtype, const void* A, int64_t strideA, const void* B, int64_t strideB, void* C, int64_t strideC,
                     void* stream) {
    int rc = validate_gemm(M, N, K, transA, transB, dtype, A, B, C, true);
    if (rc) return rc;
    if (batch < 0) return fail(TDX_ERR_INVALID_ARG, "negative batch count");
    if (strideA < 0 || strideB < 0) return fail(TDX_ERR_INVALID_ARG, "negative batch stride");
    if (batch > 1 && strideC < M * N) return fail(TDX_ERR_INVALID_ARG, "strideC < M * N: the outputs of two batches would overlap");
    if (!(beta == beta) || !(alpha == alpha)) return fail(TDX_ERR_INVALID_ARG, "alpha or beta is NaN");
    if (batch == 0 || M == 0 || N == 0) return TDX_OK;
    if (batch >= (1LL << 31)) return fail(TDX_ERR_UNSUPPORTED, "batch count must be below 2^31");
    DeviceCtx* ctx;
    rc = get_ctx(&ctx);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    GemmProblem g{M, N, K, transA, transB, dtype};
    BatchArgs ba;
    ba.batch = batch; ba.stride_a = strideA; ba.stride_b = strideB; ba.stride_c = strideC; ba.beta = beta;
    if (K == 0) {
        // empty reduction: C = beta * C.  The generic kernel does exactly that (its k loop is empty).
        return run_gemm_generic(ctx, g, alpha, C, C, C, st, ba);
    }
    if (dtype == TDX_F32) return run_gemm_simt_f32(ctx, g, alpha, A, B, C, st, ba);
    // bf16: the tensor-core kernel, one launch per batch, when every batch's operands meet its layout rules
    const bool aligned = gemm_umma_layout_ok(g) && reinterpret_cast<uintptr_t>(A) % 16 == 0 &&
                         reinterpret_cast<uintptr_t>(B) % 16 == 0 && (strideA % 8 == 0) && (strideB % 8 == 0);
    if (!aligned) return run_gemm_generic(ctx, g, alpha, A, B, C, st, ba);
    tdx_config want;
    std::memset(&want, 0, sizeof want);
    if (beta != 0.0f) want.store_mode = 1;          // the accumulate term is read by the direct-store epilogue
    tdx_config cfg;
    rc = resolve_gemm_config(g, beta != 0.0f ? &want : nullptr, ctx->sm_count, ctx->smem_optin, &cfg);
    if (rc) return rc;
    if (cfg.kernel != TDX_KERNEL_UMMA || cfg.cta_pair == 2) return run_gemm_generic(ctx, g, alpha, A, B, C, st, ba);
    for (int64_t b = 0; b < batch; ++b) {
        const char* a = static_cast<const char*>(A) + b * strideA * 2;
        const char* bb = static_cast<const char*>(B) + b * strideB * 2;
        char* c = static_cast<char*>(C) + b * strideC * 2;
        rc = run_gemm_umma(ctx, g, alpha, a, bb, c, cfg, nullptr, 0, true, st, beta);
        if (rc) return rc;
    }
    return TDX_OK;
}

int tdx_add_zero_pad(int64_t N, int64_t H, int64_t W, int64_t C, int pad_top, int pad_bottom, int pad_left, int pad_right,
                     int dtype, const void* x, const void* y, void* out, void* stream) {
    if (N < 0 || H < 0 || W < 0 || C < 0) return fail(TDX_ERR_INVALID_ARG, "negative dimension");
    if (pad_top < 0 || pad_bottom < 0 || pad_left < 0 || pad_right < 0) return fail(TDX_ERR_INVALID_ARG, "negative padding");
    if (dtype != TDX_F32 && dtype != TDX_BF16) return fail(TDX_ERR_INVALID_ARG, "unknown dtype %d", dtype);
    const int64_t Hp = H + pad_top + pad_bottom, Wp = W + pad_left + pad_right;
    const int64_t total = N * Hp * Wp * C;
    if (total == 0) return TDX_OK;
    if (y == nullptr || out == nullptr) return fail(TDX_ERR_INVALID_ARG, "y or out is NULL");
    const int64_t interior = N * H * W * C;
    if (interior > 0 && x == nullptr) return fail(TDX_ERR_INVALID_ARG, "x is NULL");
    const uintptr_t el = dtype == TDX_F32 ? 4 : 2;
    if (reinterpret_cast<uintptr_t>(x) % el || reinterpret_cast<uintptr_t>(y) % el || reinterpret_cast<uintptr_t>(out) % el)
        return fail(TDX_ERR_ALIGNMENT, "pointer not aligned to its element size");
    DeviceCtx* ctx;
    int rc = get_ctx(&ctx);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const long long row_elems = W * C, y_row = Wp * C, y_img = Hp * Wp * C, y_first = (pad_top * Wp + pad_left) * C;
    const int per16 = static_cast<int>(16 / el);
    // 16-byte accesses when every interior row starts on a 16-byte boundary in x, y and out
    const bool vec_ok = row_elems % per16 == 0 && y_row % per16 == 0 && y_img % per16 == 0 && y_first % per16 == 0 &&
                        reinterpret_cast<uintptr_t>(x) % 16 == 0 && reinterpret_cast<uintptr_t>(y) % 16 == 0 &&
                        reinterpret_cast<uintptr_t>(out) % 16 == 0;
    const int vec = vec_ok ? per16 : 1;
    const int max_grid = ctx->sm_count * 16;
    if (out != y) {
        const int grid = static_cast<int>(std::min<long long>(ceil_div(total, 256), max_grid));
        if (dtype == TDX_F32)
            tdx::copy_pad_ring_kernel<float><<<grid, 256, 0, st>>>(total, C, Hp, Wp, pad_top, H, pad_left, W,
                                                                   static_cast<const float*>(y), static_cast<float*>(out));
        else
            tdx::copy_pad_ring_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(total, C, Hp, Wp, pad_top, H, pad_left, W,
                                                                           static_cast<const __nv_bfloat16*>(y),
                                                                           static_cast<__nv_bfloat16*>(out));
        TDX_CUDA(cudaGetLastError());
        g_launches.fetch_add(1);
    }
    if (interior > 0) {
        const long long work = interior / vec;
        const int grid = static_cast<int>(std::min<long long>(ceil_div(work, 256), max_grid));
        if (dtype == TDX_F32)
            tdx::add_zero_pad_kernel<float><<<grid, 256, 0, st>>>(N * H, H, row_elems, y_img, y_row, y_first, vec,
                                                                  static_cast<const float*>(x), static_cast<const float*>(y),
                                                                  static_cast<float*>(out));
        else
            tdx::add_zero_pad_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(
                N * H, H, row_elems, y_img, y_row, y_first, vec, static_cast<const __nv_bfloat16*>(x),
                static_cast<const __nv_bfloat16*>(y), static_cast<__nv_bfloat16*>(out));
        TDX_CUDA(cudaGetLastError());
        g_launches.fetch_add(1);
    }
    return TDX_OK;
}

int tdx_gemm_ex(int64_t M, int64_t N, int64_t K, int transA, int transB, float alpha, int dtype, const void* A,
                const void* B, void* C, void* stream, const tdx_config* cfg, void* workspace, size_t workspace_bytes) {
    // the library's own workspace serves every split-K it chose itself
    const bool internal = (workspace == nullptr) && (cfg == nullptr || cfg->split_k == 0);
    return gemm_dispatch(M, N, K, transA, transB, alpha, dtype, A, B, C, stream, cfg, workspace, workspace_bytes, internal);
}

int tdx_gemm_workspace_size(int64_t M, int64_t N, int64_t K, int dtype, const tdx_config* cfg, size_t* bytes) {
    if (bytes == nullptr) return fail(TDX_ERR_INVALID_ARG, "bytes is NULL");
    if (M < 0 || N < 0 || K < 0) return fail(TDX_ERR_INVALID_ARG, "negative dimension");
    if (dtype != TDX_F32 && dtype != TDX_BF16) return fail(TDX_ERR_INVALID_ARG, "unknown dtype %d", dtype);
    const int split = cfg ? std::max(cfg->split_k, 1) : 1;
    *bytes = split > 1 ? static_cast<size_t>(split) * M * N * sizeof(float) : 0;
    return TDX_OK;
}

int tdx_conv2d_bias_relu(int64_t N, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int64_t R, int64_t S, int pad,
                         int stride, int dtype, const void* x, const void* w, const float* bias, int relu, void* y,
                         void* stream) {
    return conv_dispatch(N, H, W, Cin, Cout, R, S, pad, stride, dtype, x, w, bias, relu, y, stream, nullptr);
}

int tdx_conv2d_bias_add_relu(int64_t N, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int64_t R, int64_t S, int pad,
                             int stride, int dtype, const void* x, const void* w, const float* bias, const void* residual,
                             int relu, void* y, void* stream, const tdx_config* cfg) {
    return conv_dispatch(N, H, W, Cin, Cout, R, S, pad, stride, dtype, x, w, bias, relu, y, stream, cfg, residual);
}

int tdx_conv2d_bias_relu_ex(int64_t N, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int64_t R, int64_t S, int pad,
                            int stride, int dtype, const void* x, const void* w, const float* bias, int relu, void* y,
                            void* stream, const tdx_config* cfg) {
    return conv_dispatch(N, H, W, Cin, Cout, R, S, pad, stride, dtype, x, w, bias, relu, y, stream, cfg);
}

int tdx_gemm_host(int64_t M, int64_t N, int64_t K, int transA, int transB, float alpha, int dtype, const void* A_host,
                  const void* B_host, void* C_host, void* stream) {
    int rc = validate_gemm(M, N, K, transA, transB, dtype, A_host, B_host, C_host, true);
    if (rc) return rc;
    if (M == 0 || N == 0) return TDX_OK;
    DeviceCtx* ctx;
    rc = get_ctx(&ctx);
    if (rc) return rc;
    const size_t el = dtype == TDX_F32 ? 4 : 2;
    const size_t a_bytes = static_cast<size_t>(M) * K * el, b_bytes = static_cast<size_t>(K) * N * el,
                 c_bytes = static_cast<size_t>(M) * N * el;
    void *dA, *dB, *dC;
    if ((rc = ensure_staging(ctx, 0, a_bytes, &dA))) return rc;
    if ((rc = ensure_staging(ctx, 1, b_bytes, &dB))) return rc;
    if ((rc = ensure_staging(ctx, 2, c_bytes, &dC))) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (a_bytes) TDX_CUDA(cudaMemcpyAsync(dA, A_host, a_bytes, cudaMemcpyHostToDevice, st));
    if (b_bytes) TDX_CUDA(cudaMemcpyAsync(dB, B_host, b_bytes, cudaMemcpyHostToDevice, st));
    rc = gemm_dispatch(M, N, K, transA, transB, alpha, dtype, dA, dB, dC, stream, nullptr, nullptr, 0, true);
    if (rc) return rc;
    TDX_CUDA(cudaMemcpyAsync(C_host, dC, c_bytes, cudaMemcpyDeviceToHost, st));
    TDX_CUDA(cudaStreamSynchronize(st));
    return TDX_OK;
}

int tdx_gemm_batched_host(int64_t batch, int64_t M, int64_t N, int64_t K, int transA, int transB, float alpha, float beta,
                          int dtype, const void* A_host, const void* B_host, void* C_host, void* stream) {
    int rc = validate_gemm(M, N, K, transA, transB, dtype, A_host, B_host, C_host, true);
    if (rc) return rc;
    if (batch < 0) return fail(TDX_ERR_INVALID_ARG, "negative batch count");
    if (batch == 0 || M == 0 || N == 0) return TDX_OK;
    DeviceCtx* ctx;
    rc = get_ctx(&ctx);
    if (rc) return rc;
    const size_t el = dtype == TDX_F32 ? 4 : 2;
    const size_t a_bytes = static_cast<size_t>(batch) * M * K * el, b_bytes = static_cast<size_t>(batch) * K * N * el,
                 c_bytes = static_cast<size_t>(batch) * M * N * el;
    void *dA, *dB, *dC;
    if ((rc = ensure_staging(ctx, 0, a_bytes, &dA))) return rc;
    if ((rc = ensure_staging(ctx, 1, b_bytes, &dB))) return rc;
    if ((rc = ensure_staging(ctx, 2, c_bytes, &dC))) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (a_bytes) TDX_CUDA(cudaMemcpyAsync(dA, A_host, a_bytes, cudaMemcpyHostToDevice, st));
    if (b_bytes) TDX_CUDA(cudaMemcpyAsync(dB, B_host, b_bytes, cudaMemcpyHostToDevice, st));
    if (beta != 0.0f) TDX_CUDA(cudaMemcpyAsync(dC, C_host, c_bytes, cudaMemcpyHostToDevice, st));
    rc = tdx_gemm_batched(batch, M, N, K, transA, transB, alpha, beta, dtype, dA, M * K, dB, K * N, dC, M * N, stream);
    if (rc) return rc;
    TDX_CUDA(cudaMemcpyAsync(C_host, dC, c_bytes, cudaMemcpyDeviceToHost, st));
    TDX_CUDA(cudaStreamSynchronize(st));
    return TDX_OK;
}

int tdx_add_zero_pad_host(int64_t N, int64_t H, int64_t W, int64_t C, int pad_top, int pad_bottom, int pad_left,
                          int pad_right, int dtype, const void* x_host, void* y_host, void* stream) {
    if (N < 0 || H < 0 || W < 0 || C < 0 || pad_top < 0 || pad_bottom < 0 || pad_left < 0 || pad_right < 0)
        return fail(TDX_ERR_INVALID_ARG, "negative dimension or padding");
    if (dtype != TDX_F32 && dtype != TDX_BF16) return fail(TDX_ERR_INVALID_ARG, "unknown dtype %d", dtype);
    const size_t el = dtype == TDX_F32 ? 4 : 2;
    const size_t x_bytes = static_cast<size_t>(N) * H * W * C * el;
    const size_t y_bytes = static_cast<size_t>(N) * (H + pad_top + pad_bottom) * (W + pad_left + pad_right) * C * el;
    if (y_bytes == 0) return TDX_OK;
    if (y_host == nullptr || (x_bytes && x_host == nullptr)) return fail(TDX_ERR_INVALID_ARG, "NULL host pointer");
    DeviceCtx* ctx;
    int rc = get_ctx(&ctx);
    if (rc) return rc;
    void *dx, *dy;
    if ((rc = ensure_staging(ctx, 0, x_bytes, &dx))) return rc;
    if ((rc = ensure_staging(ctx, 1, y_bytes, &dy))) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (x_bytes) TDX_CUDA(cudaMemcpyAsync(dx, x_host, x_bytes, cudaMemcpyHostToDevice, st));
    TDX_CUDA(cudaMemcpyAsync(dy, y_host, y_bytes, cudaMemcpyHostToDevice, st));
    rc = tdx_add_zero_pad(N, H, W, C, pad_top, pad_bottom, pad_left, pad_right, dtype, dx, dy, dy, stream);
    if (rc) return rc;
    TDX_CUDA(cudaMemcpyAsync(y_host, dy, y_bytes, cudaMemcpyDeviceToHost, st));
    TDX_CUDA(cudaStreamSynchronize(st));
    return TDX_OK;
}

int tdx_conv2d_bias_relu_host(int64_t N, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int64_t R, int64_t S, int pad,
                              int stride, int dtype, const void* x_host, const void* w_host, const float* bias_host,
                              int relu, void* y_host, void* stream) {
    ConvProblem cp;
    int rc = validate_conv(N, H, W, Cin, Cout, R, S, pad, stride, dtype, x_host, w_host, y_host, relu, true, &cp);
    if (rc) return rc;
    if (N == 0 || Cout == 0 || cp.P == 0 || cp.Q == 0) return TDX_OK;
    DeviceCtx* ctx;
    rc = get_ctx(&ctx);
    if (rc) return rc;
    const size_t el = dtype == TDX_F32 ? 4 : 2;
    const size_t x_bytes = static_cast<size_t>(N) * H * W * Cin * el, w_bytes = static_cast<size_t>(Cout) * R * S * Cin * el,
                 y_bytes = static_cast<size_t>(N) * cp.P * cp.Q * Cout * el, b_bytes = static_cast<size_t>(Cout) * 4;
    void *dx, *dw, *dy, *db = nullptr;
    if ((rc = ensure_staging(ctx, 0, x_bytes, &dx))) return rc;
    if ((rc = ensure_staging(ctx, 1, w_bytes, &dw))) return rc;
    if ((rc = ensure_staging(ctx, 2, y_bytes, &dy))) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (x_bytes) TDX_CUDA(cudaMemcpyAsync(dx, x_host, x_bytes, cudaMemcpyHostToDevice, st));
    TDX_CUDA(cudaMemcpyAsync(dw, w_host, w_bytes, cudaMemcpyHostToDevice, st));
    if (bias_host) {
        if ((rc = ensure_staging(ctx, 3, b_bytes, &db))) return rc;
        TDX_CUDA(cudaMemcpyAsync(db, bias_host, b_bytes, cudaMemcpyHostToDevice, st));
    }
    rc = conv_dispatch(N, H, W, Cin, Cout, R, S, pad, stride, dtype, dx, dw, static_cast<const float*>(db), relu, dy,
                       stream, nullptr);
    if (rc) return rc;
    TDX_CUDA(cudaMemcpyAsync(y_host, dy, y_bytes, cudaMemcpyDeviceToHost, st));
    TDX_CUDA(cudaStreamSynchronize(st));
    return TDX_OK;
}

int tdx_enum_gemm_configs(int64_t M, int64_t N, int64_t K, int transA, int transB, int dtype, tdx_config* out, int cap,
                          int* n) {
    int rc = validate_gemm(M, N, K, transA, transB, dtype, nullptr, nullptr, nullptr, false);
    if (rc) return rc;
    if (cap < 0 || (cap > 0 && out == nullptr)) return fail(TDX_ERR_INVALID_ARG, "bad output list");
    int sm_count, smem_limit;
    device_limits(&sm_count, &smem_limit);
    std::vector<tdx_config> v;
    if (M > 0 && N > 0 && K > 0) enum_gemm(GemmProblem{M, N, K, transA, transB, dtype}, sm_count, smem_limit, &v);
    return write_configs(v, out, cap, n);
}

int tdx_enum_conv2d_configs(int64_t N, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int64_t R, int64_t S, int pad,
                            int stride, int dtype, tdx_config* out, int cap, int* n) {
    ConvProblem cp;
    int rc = validate_conv(N, H, W, Cin, Cout, R, S, pad, stride, dtype, nullptr, nullptr, nullptr, 0, false, &cp);
    if (rc) return rc;
    if (cap < 0 || (cap > 0 && out == nullptr)) return fail(TDX_ERR_INVALID_ARG, "bad output list");
    int sm_count, smem_limit;
    device_limits(&sm_count, &smem_limit);
    std::vector<tdx_config> v;
    if (N > 0 && Cout > 0 && cp.P > 0 && cp.Q > 0) enum_conv(cp, sm_count, smem_limit, &v);
    return write_configs(v, out, cap, n);
}

int tdx_default_gemm_config(int64_t M, int64_t N, int64_t K, int transA, int transB, int dtype, tdx_config* out) {
    int rc = validate_gemm(M, N, K, transA, transB, dtype, nullptr, nullptr, nullptr, false);
    if (rc) return rc;
    if (out == nullptr) return fail(TDX_ERR_INVALID_ARG, "out is NULL");
    if (M == 0 || N == 0 || K == 0) { std::memset(out, 0, sizeof *out); return TDX_OK; }
    int sm_count, smem_limit;
    device_limits(&sm_count, &smem_limit);
    return resolve_gemm_config(GemmProblem{M, N, K, transA, transB, dtype}, nullptr, sm_count, smem_limit, out);
}

int tdx_default_conv2d_config(int64_t N, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int64_t R, int64_t S, int pad,
                              int stride, int dtype, tdx_config* out) {
    ConvProblem cp;
    int rc = validate_conv(N, H, W, Cin, Cout, R, S, pad, stride, dtype, nullptr, nullptr, nullptr, 0, false, &cp);
    if (rc) return rc;
    if (out == nullptr) return fail(TDX_ERR_INVALID_ARG, "out is NULL");
    if (N == 0 || Cout == 0 || cp.P == 0 || cp.Q == 0) { std::memset(out, 0, sizeof *out); return TDX_OK; }
    int sm_count, smem_limit;
    device_limits(&sm_count, &smem_limit);
    return resolve_conv_config(cp, nullptr, sm_count, smem_limit, out);
}

int tdx_tune_gemm(int64_t M, int64_t N, int64_t K, int transA, int transB, int dtype, int iters, tdx_config* best,
                  float* best_us, tdx_config* tried, float* tried_us, int cap, int* n_tried, void* stream) {
    int rc = validate_gemm(M, N, K, transA, transB, dtype, nullptr, nullptr, nullptr, false);
    if (rc) return rc;
    if (best == nullptr || iters < 1 || cap < 0) return fail(TDX_ERR_INVALID_ARG, "best is NULL, iters < 1 or cap < 0");
    if (M == 0 || N == 0 || K == 0) return fail(TDX_ERR_INVALID_ARG, "empty problem");
    DeviceCtx* ctx;
    rc = get_ctx(&ctx);
    if (rc) return rc;
    GemmProblem g{M, N, K, transA, transB, dtype};
    std::vector<tdx_config> cands;
    enum_gemm(g, ctx->sm_count, ctx->smem_optin, &cands);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t el = dtype == TDX_F32 ? 4 : 2;
    ScratchGuard guard;
    void *A, *B, *C, *ws;
    size_t ws_bytes = 0;
    for (const auto& c : cands) ws_bytes = std::max(ws_bytes, c.split_k > 1 ? static_cast<size_t>(c.split_k) * M * N * 4 : 0);
    if ((rc = guard.alloc(&A, M * K * el))) return rc;
    if ((rc = guard.alloc(&B, K * N * el))) return rc;
    if ((rc = guard.alloc(&C, M * N * el))) return rc;
    if ((rc = guard.alloc(&ws, ws_bytes))) return rc;
    // fp32 buffers are filled as pairs of bf16 patterns: finite, varied values either way
    if ((rc = fill_scratch(A, M * K * el / 2, 1u, st))) return rc;
    if ((rc = fill_scratch(B, K * N * el / 2, 2u, st))) return rc;
    auto launch = [&](const tdx_config& c) {
        return gemm_dispatch(M, N, K, transA, transB, 1.0f, dtype, A, B, C, stream, &c, ws, ws_bytes, false);
    };
    rc = time_candidates(cands, iters, st, launch, best, best_us, tried, tried_us, cap, n_tried);
    cudaStreamSynchronize(st);
    if (rc) return rc;
    {
        std::lock_guard<std::mutex> lk(g_mu);
        g_tune[gemm_key(M, N, K, transA, transB, dtype)] = TuneEntry{*best, best_us ? *best_us : 0.0f};
    }
    return TDX_OK;
}

int tdx_tune_conv2d(int64_t N, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int64_t R, int64_t S, int pad,
                    int stride, int dtype, int iters, tdx_config* best, float* best_us, tdx_config* tried,
                    float* tried_us, int cap, int* n_tried, void* stream) {
    ConvProblem cp;
    int rc = validate_conv(N, H, W, Cin, Cout, R, S, pad, stride, dtype, nullptr, nullptr, nullptr, 0, false, &cp);
    if (rc) return rc;
    if (best == nullptr || iters < 1 || cap < 0) return fail(TDX_ERR_INVALID_ARG, "best is NULL, iters < 1 or cap < 0");
    if (N == 0 || Cout == 0 || cp.P == 0 || cp.Q == 0) return fail(TDX_ERR_INVALID_ARG, "empty problem");
    DeviceCtx* ctx;
    rc = get_ctx(&ctx);
    if (rc) return rc;
    std::vector<tdx_config> cands;
    enum_conv(cp, ctx->sm_count, ctx->smem_optin, &cands);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t el = dtype == TDX_F32 ? 4 : 2;
    ScratchGuard guard;
    void *x, *w, *y, *b;
    if ((rc = guard.alloc(&x, N * H * W * Cin * el))) return rc;
    if ((rc = guard.alloc(&w, Cout * R * S * Cin * el))) return rc;
    if ((rc = guard.alloc(&y, N * cp.P * cp.Q * Cout * el))) return rc;
    if ((rc = guard.alloc(&b, Cout * 4))) return rc;
    if ((rc = fill_scratch(x, N * H * W * Cin * el / 2, 3u, st))) return rc;
    if ((rc = fill_scratch(w, Cout * R * S * Cin * el / 2, 4u, st))) return rc;
    TDX_CUDA(cudaMemsetAsync(b, 0, Cout * 4, st));
    auto launch = [&](const tdx_config& c) {
        return conv_dispatch(N, H, W, Cin, Cout, R, S, pad, stride, dtype, x, w, static_cast<const float*>(b), 1, y, stream, &c);
    };
    rc = time_candidates(cands, iters, st, launch, best, best_us, tried, tried_us, cap, n_tried);
    cudaStreamSynchronize(st);
    if (rc) return rc;
    {
        std::lock_guard<std::mutex> lk(g_mu);
        g_tune[conv_key(N, H, W, Cin, Cout, R, S, pad, stride, dtype)] = TuneEntry{*best, best_us ? *best_us : 0.0f};
    }
    return TDX_OK;
}

int tdx_tune_save(const char* json_path) {
    if (json_path == nullptr) return fail(TDX_ERR_INVALID_ARG, "path is NULL");
    FILE* f = fopen(json_path, "w");
    if (!f) return fail(TDX_ERR_INVALID_ARG, "cannot open %s for writing", json_path);
    std::lock_guard<std::mutex> lk(g_mu);
    fprintf(f, "{\"version\": 1, \"entries\": [\n");
    size_t i = 0;
    for (const auto& kv : g_tune) {
        int v[14];
        cfg_to_ints(kv.second.cfg, v);
        fprintf(f, "  {\"key\": \"%s\", \"cfg\": [", kv.first.c_str());
        for (int j = 0; j < 14; ++j) fprintf(f, "%d%s", v[j], j < 13 ? ", " : "");
        fprintf(f, "], \"us\": %.3f}%s\n", kv.second.us, ++i < g_tune.size() ? "," : "");
    }
    fprintf(f, "]}\n");
    fclose(f);
    return TDX_OK;
}

int tdx_tune_load(const char* json_path) {
    if (json_path == nullptr) return fail(TDX_ERR_INVALID_ARG, "path is NULL");
    FILE* f = fopen(json_path, "r");
    if (!f) return fail(TDX_ERR_INVALID_ARG, "cannot open %s", json_path);
    std::string text;
    char buf[4096];
    size_t got;
    while ((got = fread(buf, 1, sizeof buf, f)) > 0) text.append(buf, got);
    fclose(f);
    std::map<std::string, TuneEntry> loaded;
    size_t pos = 0;
    while ((pos = text.find("\"key\"", pos)) != std::string::npos) {
        const size_t q0 = text.find('"', text.find(':', pos) + 1);
        const size_t q1 = q0 == std::string::npos ? q0 : text.find('"', q0 + 1);
        const size_t b0 = q1 == std::string::npos ? q1 : text.find('[', q1);
        const size_t b1 = b0 == std::string::npos ? b0 : text.find(']', b0);
        if (b1 == std::string::npos) return fail(TDX_ERR_INVALID_ARG, "malformed tuning cache %s", json_path);
        const std::string key = text.substr(q0 + 1, q1 - q0 - 1);
        int v[14] = {0};
        int n = 0;
        const char* s = text.c_str() + b0 + 1;
        const char* end = text.c_str() + b1;
        while (s < end && n < 14) {
            char* next;
            long val = strtol(s, &next, 10);
            if (next == s) break;
            v[n++] = static_cast<int>(val);
            s = next;
            while (s < end && (*s == ',' || *s == ' ')) ++s;
        }
        if (n < 11 || n > 14) return fail(TDX_ERR_INVALID_ARG, "malformed cfg list in %s", json_path);
        TuneEntry e;
        ints_to_cfg(v, &e.cfg);
        e.us = 0.0f;
        const size_t u = text.find("\"us\"", b1);
        const size_t nextkey = text.find("\"key\"", b1);
        if (u != std::string::npos && (nextkey == std::string::npos || u < nextkey))
            e.us = static_cast<float>(atof(text.c_str() + text.find(':', u) + 1));
        loaded[key] = e;
        pos = b1;
    }
    std::lock_guard<std::mutex> lk(g_mu);
    for (auto& kv : loaded) g_tune[kv.first] = kv.second;
    return TDX_OK;
}

int tdx_gemm_tile_plan(int64_t M, int64_t N, int64_t K, int tile_m, int tile_n, int raster, int ctas, int* table,
                       int cap_tiles, int* n_rounds, int* n_ctas, double* model_cycles, double* model_cycles_uniform) {
    if (M <= 0 || N <= 0 || K <= 0 || ctas <= 0 || (tile_m != 128 && tile_m != 256) || tile_n < 192 || tile_n > 256 ||
        tile_n % 64 || raster < 0)
        return fail(TDX_ERR_INVALID_ARG, "tdx_gemm_tile_plan: bad argument");
    TilePlan plan;
    const bool fitted = plan_fitted_tiles(M, N, ceil_div(K, 64), tile_m, tile_n, raster, ctas, 0.0, &plan);
    if (model_cycles) *model_cycles = plan.makespan;
    if (model_cycles_uniform) *model_cycles_uniform = plan.uniform;
    if (n_rounds) *n_rounds = fitted ? plan.rounds : 0;
    if (n_ctas) *n_ctas = fitted ? plan.grid : 0;
    if (fitted && table)
        for (size_t i = 0; i < plan.table.size() && static_cast<int>(i) < cap_tiles; ++i) {
            table[3 * i] = plan.table[i].x;
            table[3 * i + 1] = plan.table[i].y;
            table[3 * i + 2] = plan.table[i].z;
        }
    return TDX_OK;
}

int tdx_tune_clear(void) {
    std::lock_guard<std::mutex> lk(g_mu);
    g_tune.clear();
    return TDX_OK;
}

int tdx_check_device_status(void* stream) {
    DeviceCtx* ctx;
    int rc = get_ctx(&ctx);
    if (rc) return rc;
    TDX_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
    int v = 0;
    TDX_CUDA(cudaMemcpy(&v, ctx->status_ptr, sizeof v, cudaMemcpyDeviceToHost));
    if (v != 0) {
        TDX_CUDA(cudaMemset(ctx->status_ptr, 0, sizeof v));
        return fail(TDX_ERR_TIMEOUT, "a kernel abandoned a bounded wait (role code %d)", v);
    }
    return TDX_OK;
}

int tdx_selftest_bounded_wait(int limit_us, void* stream) {
    if (limit_us < 1 || limit_us > 100000) return fail(TDX_ERR_INVALID_ARG, "limit_us must be in [1, 100000]");
    DeviceCtx* ctx;
    int rc = get_ctx(&ctx);
    if (rc) return rc;
    const long long cycles = static_cast<long long>(limit_us) * 2000;   // ~2 GHz: exactness does not matter here
    tdx::bounded_wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(ctx->status_ptr, cycles);
    TDX_CUDA(cudaGetLastError());
    g_launches.fetch_add(1);
    return TDX_OK;
}

int64_t tdx_kernel_launch_count(void) { return g_launches.load(); }

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// tdx_gemm_splitk_static: split-K GEMM whose partial sums live in an array that is part of the
// library image, for callers that must not allocate device memory (see include/tdx.h).
// ---------------------------------------------------------------------------------------------
namespace {

// The scratch itself.  In host code this name is only a handle for the runtime's symbol table, not
// an address a kernel can use; the device address is fetched once per device below.
static __device__ __align__(256) float g_static_splitk_scratch[TDX_STATIC_SCRATCH_BYTES / sizeof(float)];

constexpr int kMaxStaticDevices = 64;
float* g_static_scratch_ptr[kMaxStaticDevices] = {};   // device address of the array, per device ordinal
std::mutex g_static_mu;

// Device address of the scratch array on the current device (looked up on first use, then cached).
int static_scratch_address(int dev, float** out) {
    if (dev < 0 || dev >= kMaxStaticDevices) return fail(TDX_ERR_UNSUPPORTED, "device ordinal %d out of range", dev);
    std::lock_guard<std::mutex> lk(g_static_mu);
    if (g_static_scratch_ptr[dev] == nullptr) {
        float* ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_splitk_scratch);
        if (e != cudaSuccess || ptr == nullptr)
            return fail(TDX_ERR_CUDA, "cudaGetSymbolAddress(static scratch): %s", cudaGetErrorString(e));
        g_static_scratch_ptr[dev] = ptr;
    }
    *out = g_static_scratch_ptr[dev];
    return TDX_OK;
}

// bf16 2-D tensor map, built on the spot (no cache, no heap).
int encode_map_2d(DeviceCtx* ctx, const void* ptr, uint64_t inner, uint64_t outer, uint32_t box_inner,
                  uint32_t box_outer, CUtensorMap* out) {
    cuuint64_t gdim[2] = {inner, outer};
    cuuint64_t gstr[1] = {inner * 2};
    cuuint32_t gbox[2] = {box_inner, box_outer};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = ctx->encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), gdim, gstr, gbox, estr,
                             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(TDX_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d)", static_cast<int>(r));
    return TDX_OK;
}

}  // namespace

extern "C" {

int tdx_gemm_splitk_static(int64_t M, int64_t N, int64_t K, int transA, int transB, float alpha, const void* A,
                           const void* B, void* C, int tile_n, int split_k, void* stream) {
    int rc = validate_gemm(M, N, K, transA, transB, TDX_BF16, A, B, C, true);
    if (rc) return rc;
    if (split_k < 1 || tile_n < 0) return fail(TDX_ERR_INVALID_ARG, "split_k must be >= 1 and tile_n >= 0");
    if (M == 0 || N == 0) return TDX_OK;
    if (K == 0) return fail(TDX_ERR_UNSUPPORTED, "K = 0: use tdx_gemm");
    // size check first: it needs no device
    const double need = static_cast<double>(split_k) * static_cast<double>(M) * static_cast<double>(N) * 4.0;
    if (split_k > 1 && need > static_cast<double>(TDX_STATIC_SCRATCH_BYTES))
        return fail(TDX_ERR_WORKSPACE,
                    "split_k * M * N * 4 = %.0f bytes exceeds the static scratch of %u bytes (TDX_STATIC_SCRATCH_BYTES)",
                    need, TDX_STATIC_SCRATCH_BYTES);
    GemmProblem g{M, N, K, transA, transB, TDX_BF16};
    if (!gemm_umma_layout_ok(g) || reinterpret_cast<uintptr_t>(A) % 16 || reinterpret_cast<uintptr_t>(B) % 16)
        return fail(TDX_ERR_ALIGNMENT, "static split-K GEMM needs 16-byte aligned A, B and contiguous dims %% 8 == 0");
    tdx_config want;
    std::memset(&want, 0, sizeof want);
    want.kernel = TDX_KERNEL_UMMA;
    want.tile_m = 128;
    want.tile_n = tile_n;
    want.split_k = split_k;
    want.store_mode = 1;
    int sm_count, smem_limit;
    device_limits(&sm_count, &smem_limit);
    tdx_config cfg;
    rc = resolve_gemm_config(g, &want, sm_count, smem_limit, &cfg);
    if (rc) return rc;
    DeviceCtx* ctx;
    rc = get_ctx(&ctx);
    if (rc) return rc;
    rc = resolve_gemm_config(g, &want, ctx->sm_count, ctx->smem_optin, &cfg);
    if (rc) return rc;
    float* scratch = nullptr;
    rc = static_scratch_address(ctx->dev, &scratch);
    if (rc) return rc;

    const int64_t num_kb = ceil_div(K, 64);
    UmmaParams p;
    std::memset(&p, 0, sizeof p);
    p.M = static_cast<int>(M);
    p.N = static_cast<int>(N);
    p.num_kb = static_cast<int>(num_kb);
    p.bm = cfg.tile_m;
    p.slots = tmem_slots_for(cfg.tile_m, cfg.tile_n);
    p.tiles_m = static_cast<int>(ceil_div(M, cfg.tile_m));
    p.tiles_n = static_cast<int>(ceil_div(N, cfg.tile_n));
    p.panel = cfg.raster == 0 ? p.tiles_m : std::min(cfg.raster, p.tiles_m);
    p.split_k = cfg.split_k;
    p.kb_per_split = static_cast<int>(ceil_div(num_kb, cfg.split_k));
    p.k_stagger = cfg.k_stagger;
    p.bn = cfg.tile_n;
    p.stages = cfg.stages;
    p.tmem_cols = tmem_cols_for(cfg.tile_m, cfg.tile_n);
    p.a_mn_major = transA ? 1 : 0;
    p.b_mn_major = transB ? 0 : 1;
    p.alpha = alpha;
    p.C = static_cast<__nv_bfloat16*>(C);
    p.ldc = N;
    p.status = ctx->status_ptr;
    p.vec_store = (N % 8 == 0) && (reinterpret_cast<uintptr_t>(C) % 16 == 0);
    p.partial = cfg.split_k > 1 ? scratch : nullptr;

    CUtensorMap ma, mb;
    rc = p.a_mn_major ? encode_map_2d(ctx, A, static_cast<uint64_t>(M), static_cast<uint64_t>(K), 64, 64, &ma)
                      : encode_map_2d(ctx, A, static_cast<uint64_t>(K), static_cast<uint64_t>(M), 64, 128, &ma);
    if (rc) return rc;
    rc = p.b_mn_major ? encode_map_2d(ctx, B, static_cast<uint64_t>(N), static_cast<uint64_t>(K), 64, 64, &mb)
                      : encode_map_2d(ctx, B, static_cast<uint64_t>(K), static_cast<uint64_t>(N), 64,
                                      static_cast<uint32_t>(cfg.tile_n), &mb);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    rc = launch_umma(ctx, false, ma, mb, ma, p, st);   // direct stores: the third map is unused
    if (rc) return rc;
    if (cfg.split_k > 1) {
        const long long MN = static_cast<long long>(M) * N;
        const int vec8 = p.vec_store ? 1 : 0;
        const long long work = vec8 ? MN / 8 : MN;
        const int grid = static_cast<int>(std::min<long long>(ceil_div(work, 256), 148LL * 16));
        tdx::splitk_reduce_kernel<<<std::max(grid, 1), 256, 0, st>>>(MN, static_cast<int>(N), cfg.split_k, scratch, alpha,
                                                                     nullptr, 0, p.C, vec8);
        TDX_CUDA(cudaGetLastError());
        g_launches.fetch_add(1);
    }
    return TDX_OK;
}

const char* tdx_last_error(void) { return g_err.c_str(); }

const char* tdx_version(void) { return "tdx 0.1.0 (sm_100a)"; }

}  // extern "C"
