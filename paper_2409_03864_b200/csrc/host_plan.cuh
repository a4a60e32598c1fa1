// Tile plan fitted to the number of CTAs: cost model, longest-first dealing, device copies of the tables.
#pragma once
#include "host_config.cuh"

namespace {

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

// mmas_per_kb: MMAs one CTA's tensor core runs per 64-deep K block (4 per 128 rows it owns); b_rows: rows of B the
// CTA loads per K block (the tile's width, half of it in a CTA pair).  A K block costs the MMAs or the time the SM
// needs to take its operand slices in from L2 (about 70 bytes per cycle), whichever is longer: narrow tiles under
// 128 rows of A are bound by the latter (128 x 128: 32 KB per 256 MMA cycles).
double tile_cost_cycles(int mmas_per_kb, int width, int64_t num_kb, int b_rows = -1) {
    const double mma = std::max(width / 2.0, 60.0);
    if (b_rows < 0) b_rows = width;
    const double ingest = (32.0 * mmas_per_kb + b_rows) * 128.0 / 70.0;
    return static_cast<double>(num_kb) * std::max(mmas_per_kb * mma, ingest) + 1500.0 + 13.0 * width;
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
    const double c_big = tile_cost_cycles(mmas, bn, num_kb, pair ? bn / 2 : bn);
    const double uniform = lpt_two_sizes(uniform_tiles, c_big, 0, 0.0, g);
    double best = uniform;
    int best_w = 0;
    int64_t best_b = 0, best_b1 = 0, best_e = 0;
    // pairs: each CTA loads half of a tile's columns, kept a multiple of 64 (one copy per 64 rows)
    const int w_step = pair ? 128 : 64;
    for (int w = bn - w_step; w >= 128; w -= w_step) {
        const double c_small = tile_cost_cycles(mmas, w, num_kb, pair ? w / 2 : w);
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
    const double c_small = tile_cost_cycles(mmas, w, num_kb, pair ? w / 2 : w);
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

// K-balanced plan (fit = 3), for problems with few tiles and a long reduction (the HBM-bound skinny shapes): the
// tiles x K blocks units, tile after tile, are cut into g nearly equal runs, one per CTA, so that every SM streams its
// share of the operands -- a uniform K split leaves SMs idle whenever tiles x splits is no multiple of the SM count
// (128 x 8192 x 8192: 43 tiles x 3 splits = 129 items on 148 SMs).  A run that crosses a tile boundary becomes two
// entries; a boundary that would leave a piece shorter than `min_len` K blocks snaps to the tile boundary (a partial
// tile costs its fp32 store and reload whatever its length).  Every piece writes an fp32 partial tile to its slot
// (ascending K within the tile); nseg[tile] slots are summed by splitk_reduce_var_kernel.
struct KBalancedPlan {
    std::vector<int4> table;   // [round * grid + cta] = (row block, first column, width, kb0 | kb1 << 12 | slot << 24)
    std::vector<int> nseg;     // per tile (row block * tiles_n + column tile)
    int rounds = 0, grid = 0, max_seg = 0, tiles_n = 0;
};
bool plan_k_balanced(int64_t M, int64_t N, int64_t num_kb, int bm, int bn, int g, KBalancedPlan* out, int min_len = 4) {
    const int64_t tiles_m = ceil_div(M, bm), tiles_n = ceil_div(N, bn), T = tiles_m * tiles_n, U = T * num_kb;
    if (num_kb < 1 || num_kb > 4095 || T < 1 || g < 1 || T > (1 << 20)) return false;
    const int64_t G = std::max<int64_t>(1, std::min<int64_t>(g, U / std::max(1, min_len)));      // no run shorter than min_len
    std::vector<int64_t> cut(G + 1);
    for (int64_t c = 0; c <= G; ++c) {
        int64_t b = (c * U + G / 2) / G;                           // even share, rounded
        const int64_t r = b % num_kb;
        if (c > 0 && c < G && r != 0) {                            // keep pieces at least min_len long
            if (r < min_len) b -= r;
            else if (num_kb - r < min_len) b += num_kb - r;
        }
        cut[c] = b;
    }
    std::vector<std::vector<int4>> per(G);
    out->nseg.assign(T, 0);
    for (int64_t c = 0; c < G; ++c) {
        int64_t u = cut[c];
        while (u < cut[c + 1]) {
            const int64_t tile = u / num_kb, kb0 = u % num_kb, kb1 = std::min<int64_t>(num_kb, kb0 + (cut[c + 1] - u));
            const int slot = out->nseg[tile]++;
            if (slot > 127) return false;
            const int64_t m_blk = tile / tiles_n, n_blk = tile % tiles_n;
            const int width = static_cast<int>(std::min<int64_t>(bn, ceil_div(N - n_blk * bn, 64) * 64));
            per[c].push_back(make_int4(static_cast<int>(m_blk), static_cast<int>(n_blk * bn), width,
                                       static_cast<int>(kb0 | (kb1 << 12) | (static_cast<int64_t>(slot) << 24))));
            u += kb1 - kb0;
        }
    }
    size_t rounds = 0;
    for (auto& v : per) rounds = std::max(rounds, v.size());
    out->grid = static_cast<int>(G);
    out->rounds = static_cast<int>(rounds);
    out->tiles_n = static_cast<int>(tiles_n);
    out->max_seg = *std::max_element(out->nseg.begin(), out->nseg.end());
    out->table.assign(rounds * G, make_int4(0, 0, 0, 0));
    for (int64_t c = 0; c < G; ++c)
        for (size_t k = 0; k < per[c].size(); ++k) out->table[k * G + c] = per[c][k];
    return true;
}

// Device copies of tile plans, one per (device, shape, tile, CTA count); never freed (a few KB each).
struct PlanKey {
    int64_t M, N, num_kb;
    int dev, bm, bn, raster, g, forced, pair;
    bool operator<(const PlanKey& o) const { return std::memcmp(this, &o, sizeof(PlanKey)) < 0; }
};
struct DevicePlan {
    int4* dev = nullptr; int rounds = 0, grid = 0; bool fitted = false;
    const int* nseg = nullptr; int max_seg = 0, tiles_n = 0;      // K-balanced plans only (nseg follows the table on the device)
};
std::map<PlanKey, DevicePlan> g_plans;

// Looks the plan up.  First use of a shape on a device builds the plan, allocates its table on that device and
// copies it there synchronously (cudaMalloc + cudaMemcpy: not legal inside a stream capture, so a captured
// call must have been preceded by an eager one for the same shape).
int get_tile_plan(DeviceCtx* ctx, int64_t M, int64_t N, int64_t num_kb, int bm, int bn, int raster, double min_gain,
                  DevicePlan* out, bool pair = false) {
    PlanKey key;
    std::memset(&key, 0, sizeof key);
    key.M = M; key.N = N; key.num_kb = num_kb; key.dev = ctx->dev; key.bm = bm; key.bn = bn; key.raster = raster; key.g = pair ? ctx->sm_count / 2 : ctx->sm_count; key.forced = min_gain <= 0.0 ? 1 : 0;
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
        // the table is a std::vector about to go out of scope: copy synchronously (once per shape and device)
        TDX_CUDA(cudaMemcpy(dev, plan.table.data(), bytes, cudaMemcpyHostToDevice));
        d.dev = static_cast<int4*>(dev);
        d.rounds = plan.rounds;
        d.grid = plan.grid;
    }
    {
        std::lock_guard<std::mutex> lk(g_mu);
        g_plans[key] = d;
    }
    *out = d;
    return TDX_OK;
}

// The K-balanced plan of a shape on this device (built, uploaded and cached like the fitted tile plans).
int get_k_balanced_plan(DeviceCtx* ctx, int64_t M, int64_t N, int64_t num_kb, int bm, int bn, DevicePlan* out) {
    PlanKey key;
    std::memset(&key, 0, sizeof key);
    key.M = M; key.N = N; key.num_kb = num_kb; key.dev = ctx->dev; key.bm = bm; key.bn = bn; key.g = ctx->sm_count;
    key.forced = 3;                                           // plan kind
    {
        std::lock_guard<std::mutex> lk(g_mu);
        auto it = g_plans.find(key);
        if (it != g_plans.end()) { *out = it->second; return TDX_OK; }
    }
    KBalancedPlan plan;
    DevicePlan d;
    d.fitted = plan_k_balanced(M, N, num_kb, bm, bn, ctx->sm_count, &plan);
    if (d.fitted) {
        const size_t tbytes = plan.table.size() * sizeof(int4), nbytes = plan.nseg.size() * sizeof(int);
        void* dev = nullptr;
        TDX_CUDA(cudaMalloc(&dev, tbytes + nbytes));
        TDX_CUDA(cudaMemcpy(dev, plan.table.data(), tbytes, cudaMemcpyHostToDevice));
        TDX_CUDA(cudaMemcpy(static_cast<char*>(dev) + tbytes, plan.nseg.data(), nbytes, cudaMemcpyHostToDevice));
        d.dev = static_cast<int4*>(dev);
        d.nseg = reinterpret_cast<const int*>(static_cast<char*>(dev) + tbytes);
        d.rounds = plan.rounds;
        d.grid = plan.grid;
        d.max_seg = plan.max_seg;
        d.tiles_n = plan.tiles_n;
    }
    {
        std::lock_guard<std::mutex> lk(g_mu);
        g_plans[key] = d;
    }
    *out = d;
    return TDX_OK;
}

// ------------------------------------------------------------------ cost model of a GEMM configuration
// Predicted device time (microseconds) of a fully specified tensor-core configuration; it ranks the candidates of
// the guided search, so only its ordering matters.  Pieces, all from measurements on B200: an MMA of N columns takes
// max(N / 2, 60) cycles; one SM ingests about 70 bytes per cycle from L2; start-up to the first MMA 5500 cycles; the
// staged epilogue about 600 cycles per 32 x 32 block and warp (16 warps), the direct one twice that; an epilogue
// overlaps the next main loop only when TMEM holds more accumulator slots than a tile uses; split-K adds the fp32
// partial traffic and a reduction launch; nothing beats streaming the operands once from HBM.
double model_gemm_us(const GemmProblem& g, const tdx_config& c, int sm_count) {
    const double clk_mhz = 1600.0;
    const int64_t num_kb = ceil_div(g.K, 64);
    const bool pair = c.cta_pair == 2;
    const int workers = pair ? sm_count / 2 : sm_count;
    const int tm = pair ? 256 : c.tile_m, bn = c.tile_n, split = std::max(1, c.split_k);
    const int64_t kb = ceil_div(num_kb, split);
    const int64_t tiles = ceil_div(g.M, tm) * ceil_div(g.N, bn) * split;
    const int halves = pair ? 1 : tm / 128;                                 // 128-row halves one CTA computes
    // a pair's MMA over 256 rows takes 115 cycles or more however narrow it is (measured at 128 columns)
    const double mma = 4.0 * halves * std::max(bn / 2.0, pair ? 115.0 : 60.0);
    // the smaller a K block's copies, the slower the SM takes its operand slices in from L2: about 46 bytes per cycle for
    // 24 KB blocks (128 x 64 tiles: 533 cycles per block), 50 for 32 KB (128 x 128: 655), about 70 from 48 KB on; a pair's
    // CTAs keep up with their MMAs at 32 KB per block (511 cycles measured at 256 columns)
    const double kb_rows = pair ? (128.0 + bn / 2.0) : (tm + static_cast<double>(bn));
    const double l2 = kb_rows * 128.0 / (pair ? 70.0 : kb_rows < 256.0 ? 46.0 : kb_rows < 384.0 ? 50.0 : 70.0);
    const double main_loop = static_cast<double>(kb) * std::max(mma, l2);
    const double blocks = halves * 4.0 * (bn / 32.0);                       // 32 x 32 output blocks per CTA and tile
    double epi = (c.store_mode == 2 ? 600.0 * std::ceil(blocks / 16.0) : 1200.0 * std::ceil(blocks / (4.0 * halves)));
    if (split > 1) epi *= 1.5;                                              // fp32 partials: twice the bytes
    const int slots = pair ? (2 * bn <= 256 ? 4 : 2) : tmem_slots_for(tm, bn);
    const bool overlapped = slots > halves;
    double rounds = std::ceil(static_cast<double>(tiles) / workers);
    double cycles;
    TilePlan plan;
    if (c.fit == 2 && split == 1 && !pair && plan_fitted_tiles(g.M, g.N, num_kb, tm, bn, c.raster, sm_count, 0.0, &plan)) {
        cycles = 5500.0 + plan.makespan;                                    // the plan's own figure includes the epilogues
    } else {
        const double per_tile = overlapped ? std::max(main_loop, epi) : main_loop + epi;
        cycles = 5500.0 + rounds * per_tile + (overlapped ? epi : 0.0) + (pair ? 4000.0 : 0.0);
    }
    // split-K summed inside clusters: one CTA per (tile, K slice), nothing overlaps; after the main loop the ranks
    // exchange (split - 1) / split of a 128 x bn fp32 tile each way through distributed shared memory and store their
    // slice (measured: 6.7 k cycles for 32 KB sent, 9.9 k for 64 KB)
    const bool in_cluster = c.store_mode == 3 && split > 1 && !pair;
    if (in_cluster) {
        const double sent = static_cast<double>(tm) * bn * 4.0 * (split - 1) / split;
        cycles = 5500.0 + rounds * (main_loop + 3400.0 + 0.1 * sent);
    }
    int kbal_slots = 0;
    if (c.fit == 3 && !pair) {
        // K-balanced: every CTA walks its even share of the tiles x K blocks units; a CTA's run touches one or two
        // tiles, each of which costs it a partial-tile epilogue
        KBalancedPlan kp;
        if (plan_k_balanced(g.M, g.N, num_kb, tm, bn, sm_count, &kp)) {
            const double units = static_cast<double>(ceil_div(g.M, tm) * ceil_div(g.N, bn)) * num_kb / kp.grid;
            cycles = 5500.0 + units * std::max(mma, l2) + kp.rounds * 1.5 * 1200.0 * std::ceil(blocks / (4.0 * halves));
            kbal_slots = kp.max_seg;
        }
    }
    double us = cycles / clk_mhz;
    if (kbal_slots > 0) {
        const double tiles_out = static_cast<double>(ceil_div(g.M, tm) * ceil_div(g.N, bn));
        const double avg_seg = (tiles_out + sm_count) / tiles_out;      // each CTA boundary adds one piece
        us += 2.0 + (avg_seg * g.M * g.N * 4.0 * 2.0 + g.M * g.N * 2.0) / 8.0e6;
    }
    // split-K: the reduction kernel's launch hides behind the GEMM's tail and the partial sums are still in L2 when it
    // reads them (128 x 8192 x 8192 in three splits: about 4 us on top of the GEMM kernel)
    if (split > 1 && !in_cluster) us += 2.0 + (static_cast<double>(split) * g.M * g.N * 4.0 * 2.0 + g.M * g.N * 2.0) / 8.0e6;
    const double hbm_us = (static_cast<double>(g.M) * g.K + static_cast<double>(g.K) * g.N + static_cast<double>(g.M) * g.N) * 2.0 / 5.0e6;
    return std::max(us, hbm_us) + 1e-3 * us;      // candidates that all sit on the HBM floor keep the order of their compute estimates
}

// The same kind of model for a convolution configuration (ranks the candidates of the guided convolution search).
// What differs from the GEMM: the rows of a tile are patches of output pixels (rows past the image edge are wasted
// work), the A operand of a K block is an input window -- fetched once per filter tap (per-tap kernel; a strided
// window drags in the pixels between its taps) or once per channel chunk for all taps (halo kernel) -- and a filter
// that fits shared memory is loaded once per CTA.
double model_conv_us(const ConvProblem& cp, const tdx_config& c, int sm_count, int smem_limit) {
    const double clk_mhz = 1600.0;
    const int64_t cchunks = ceil_div(cp.Cin, 64), taps = cp.R * cp.S, num_kb = taps * cchunks;
    const int tm = c.tile_m, bn = c.tile_n, halves = tm / 128;
    int64_t halves_total;
    if (c.halo >= 2) halves_total = halo_patches(cp, c.halo);
    else {
        const int per = std::max(1, c.patch_w * c.patch_h);
        halves_total = ceil_div(cp.N * ceil_div(cp.Q, c.patch_w) * ceil_div(cp.P, c.patch_h), std::max(1, 128 / per));
    }
    const int64_t tiles = ceil_div(halves_total, halves) * ceil_div(cp.Cout, bn);
    // inside the halo kernel an MMA was measured at about 100 cycles however narrow (the issuer advances a window
    // descriptor per tap), so tiles narrower than 200 columns run below the tensor pipe's rate there
    const double mma = 4.0 * halves * std::max(bn / 2.0, c.halo >= 2 ? 100.0 : 60.0);
    double bytes_per_kb, copy_issue = 0.0;
    if (c.halo >= 2) {
        const bool resident = bn >= cp.Cout && static_cast<int64_t>(kHaloAStages) * halves * halo_tile_bytes(cp.R, cp.S) + num_kb * bn * 128 +
                                                    staging_bytes_for(tm, c.store_mode) + 1024 <= smem_limit - kStaticSmemReserve;
        bytes_per_kb = static_cast<double>(halves) * halo_tile_bytes(cp.R, cp.S) / taps + (resident ? 0.0 : bn * 128.0);
    } else {
        bytes_per_kb = tm * 128.0 + bn * 128.0;
        // one copy per patch and tap: small patches mean many copies per K block (measured on the strided
        // 56 x 56 x 256 -> 512 layer: 8 x 4 patches 75.7 us, 16 x 8 patches 62.6 us)
        copy_issue = 45.0 * halves * std::max(1, 128 / std::max(1, c.patch_w * c.patch_h));
    }
    const double l2 = bytes_per_kb / (bn < 128 ? 46.0 : 70.0) + copy_issue;
    const double main_loop = static_cast<double>(num_kb) * std::max(mma, l2);
    const double blocks = halves * 4.0 * (bn / 32.0);
    const double epi = c.store_mode == 2 ? 600.0 * std::ceil(blocks / 16.0) : 1200.0 * std::ceil(blocks / (4.0 * halves));
    const bool overlapped = tmem_slots_for(tm, bn) > halves;
    double rounds = std::ceil(static_cast<double>(tiles) / sm_count);
    const double per_tile = overlapped ? std::max(main_loop, epi) : main_loop + epi;
    // tile widths fitted to the CTA count (streamed filter, tiles of 192 columns or more): the planner's own ratio of
    // the fitted makespan to the uniform grid's
    if (c.fit != 1 && bn >= 192 && bn % 64 == 0 && !(c.halo >= 2 && bytes_per_kb < bn * 128.0)) {
        TilePlan plan;
        if (plan_fitted_tiles(ceil_div(halves_total, halves) * tm, cp.Cout, num_kb, tm, bn, c.raster, sm_count, c.fit == 2 ? 0.0 : 0.03, &plan) &&
            plan.uniform > 0.0)
            rounds *= plan.makespan / plan.uniform;
    }
    // between configurations with the same number of rounds, the one with less work in total (fewer wasted rows) wins
    const double cycles = 5500.0 + rounds * per_tile + (overlapped ? epi : 0.0) + 1e-3 * static_cast<double>(tiles) * per_tile / sm_count;
    // (a strided filter smaller than its stride touches only part of the input.  Candidates that all sit on the HBM floor
    // -- short reductions, where the model's per-tile figures are least reliable -- are told apart only by what is
    // known to matter there: fewer copies per K block and fewer rounds; otherwise the first enumerated, the largest
    // tile, stands: 56 x 56 x 64 -> 256 1 x 1 measured 22.3 us with 256 x 256 tiles, 32.3 with 128 x 128.)
    const double touched = std::min(1.0, static_cast<double>(cp.R) / cp.stride) * std::min(1.0, static_cast<double>(cp.S) / cp.stride);
    const double hbm_us = (static_cast<double>(cp.N) * cp.H * cp.W * cp.Cin * touched + static_cast<double>(cp.Cout) * taps * cp.Cin +
                           static_cast<double>(cp.N) * cp.P * cp.Q * cp.Cout) * 2.0 / 5.0e6;
    return std::max(cycles / clk_mhz, hbm_us) + 1e-3 * (rounds * (1.0 + static_cast<double>(num_kb) * copy_issue / 1000.0));
}

}  // namespace
