// Problem descriptions and tile-configuration rules: layout constraints of the tensor-core path, shared-memory and
// TMEM budgets, static feasibility of a configuration (the search-space constraints), heuristic defaults.
#pragma once
#include "host_state.cuh"

namespace {

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
// The cluster reduction (store_mode 3) stages its summed slice the same way: two blocks for each of its four warps per
// 128-row half.
int staging_bytes_for(int tile_m, int store_mode) { return store_mode == 2 ? 16 * 2048 : store_mode == 3 ? (tile_m / 128) * 8 * 2048 : 0; }

// Shared memory for fp32 partial tiles that leave through the copy engine (split-K, K-balanced plan): two 32 x 32 fp32
// blocks for each of the four epilogue warps per 128-row half.  Optional: a configuration whose stages leave no room for
// it stores its partial tiles straight from registers.
int partial_staging_bytes(int tile_m) { return (tile_m / 128) * 4 * 2 * 4096; }
int umma_max_stages_partial(int tile_m, int tile_n, int smem_limit) {
    const int stage = (tile_m + tile_n) * 128;
    return std::min((smem_limit - kStaticSmemReserve - 1024 - partial_staging_bytes(tile_m)) / stage, tdx::kMaxStages);
}

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
    if (c.store_mode < 1 || c.store_mode > 3)
        return "store_mode must be 1 (direct), 2 (TMA store) or 3 (split-K summed inside a thread-block cluster)";
    if (c.store_mode == 3) {
        if (conv || c.cta_pair == 2) return "the cluster reduction is implemented for the single-CTA GEMM only";
        if (c.split_k < 2 || c.split_k > 8) return "the cluster reduction needs split_k in [2, 8] (the cluster size)";
        if (c.tile_n % (32 * c.split_k)) return "the cluster reduction cuts the tile into split_k column slices of a multiple of 32 columns";
        if (c.fit > 1) return "the cluster reduction runs the uniform grid: fit must be 0 or 1";
        // the other ranks' slices are received in the pipeline stages, free by then
        if (static_cast<int64_t>(c.stages) * (c.tile_m + c.tile_n) * 128 < static_cast<int64_t>(c.split_k - 1) * c.tile_m * (c.tile_n / c.split_k) * 4)
            return "the pipeline stages are too small to receive the other ranks' slices";
    }
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
    if (c.fit < 0 || c.fit > 3)
        return "fit must be 0 (choose), 1 (uniform tiles), 2 (tile widths fitted to the CTA count) or 3 (K blocks dealt evenly to all CTAs)";
    if (c.fit == 3) {
        if (conv || c.cta_pair == 2) return "the K-balanced plan is implemented for the single-CTA GEMM only";
        if (c.split_k != 1) return "the K-balanced plan replaces split_k: leave it at 1";
        if (c.store_mode != 1) return "the K-balanced plan writes fp32 partial tiles: use store_mode 1";
        if (num_kb > 4095) return "reduction too long for the K-balanced plan";
        if (c.tile_n % 64) return "the K-balanced plan loads B in 64-row copies: tile_n must be a multiple of 64";
    }
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

// Size heuristic: fills the fields a partial configuration leaves open, and is the automatic choice where the cost
// model does not apply (convolutions, layouts off the tensor-core path).
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

}  // namespace
