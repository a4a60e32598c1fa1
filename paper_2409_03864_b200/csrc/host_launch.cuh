// Kernel launches: parameter blocks, tensor maps and grids of the tensor-core, CUDA-core and generic kernels.
#pragma once
#include "host_plan.cuh"

namespace {

// ------------------------------------------------------------------ launches
int launch_umma(DeviceCtx* ctx, bool conv, const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc,
                const UmmaParams& p_in, cudaStream_t st, bool halo = false, const CUtensorMap* ma_row = nullptr,
                const CUtensorMap* mc_row = nullptr, int plan_grid = 0) {
    const long long items = static_cast<long long>(p_in.tiles_m) * p_in.tiles_n * p_in.split_k * (p_in.batch > 1 ? p_in.batch : 1);
    UmmaParams p = p_in;
    if (p.b_box == 0) p.b_box = p.bn;
    // cluster reduction: one CTA per (tile, K slice), the split_k CTAs of a tile forming one cluster
    const int grid = p.tiles != nullptr ? plan_grid
                                        : static_cast<int>(p.cluster_reduce ? items : std::min<long long>(items, ctx->sm_count));
    size_t smem = static_cast<size_t>(p.stages) * ((p.bm + p.bn) * 128) + 1024 +
                  staging_bytes_for(p.bm, p.tma_store ? 2 : p.cluster_reduce ? 3 : 1) + (p.partial_tma ? partial_staging_bytes(p.bm) : 0);
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
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    if (p.cluster_reduce) {
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = static_cast<unsigned>(p.split_k);
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        lc.numAttrs = 2;
        // a cluster must fit one GPC with this much shared memory per CTA: ask once per shape of launch, so that a
        // configuration the device cannot schedule is refused as a configuration, not as a failed launch
        static std::mutex mu;
        static std::map<std::array<long long, 4>, int> known;
        const std::array<long long, 4> key = {ctx->dev, p.split_k, static_cast<long long>(smem), threads};
        int clusters = -1;
        {
            std::lock_guard<std::mutex> lk(mu);
            auto it = known.find(key);
            if (it != known.end()) clusters = it->second;
        }
        if (clusters < 0) {
            cudaLaunchConfig_t q = lc;
            q.numAttrs = 2;
            q.gridDim = dim3(static_cast<unsigned>(p.split_k));
            TDX_CUDA(cudaOccupancyMaxActiveClusters(&clusters, tdx::umma_contract_kernel<false>, &q));
            std::lock_guard<std::mutex> lk(mu);
            known[key] = clusters;
        }
        if (clusters < 1)
            return fail(TDX_ERR_CONFIG, "a cluster of %d CTAs with %zu bytes of shared memory each cannot be scheduled on this device",
                        p.split_k, smem);
    }
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
                         __nv_bfloat16* out, int vec8, float beta = 0.0f, int batch = 1, long long batch_c = 0) {
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
    TDX_CUDA(cudaLaunchKernelEx(&lc, tdx::splitk_reduce_kernel, MN, N, split, partial, alpha, bias, relu, out, vec8, beta, batch,
                                batch_c));
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

// Operand forms beyond the plain GEMM that run_gemm_umma takes.
//  - fp32 GEMM from bf16 pieces (seg_kb > 0): the operands hold three pieces of `seg_kb` K blocks side by side
//    (cols = 3 * 64 * seg_kb columns), g.K spans the six piece pairs, and C is fp32.
//  - batched (batch > 1): all batches in one launch; batch b of A / B / C starts batch_a / batch_b / batch_c elements
//    after batch b - 1 (batch_a or batch_b = 0: one matrix shared by all batches).
//  - cols > 0: K-major operands whose rows really have `cols` columns (K padded up to the K block).
struct PieceInfo {
    int seg_kb = 0;
    int64_t cols = 0;
    int64_t batch = 1;
    int64_t batch_a = -1, batch_b = -1;   // -1: dense (rows * cols)
    int64_t batch_c = 0;
};

// A K split the library chose itself (batched, accumulate and fp32-result forms) is summed inside clusters whenever the
// configuration allows it: same tile and split, no workspace, one launch less (TDX_FORCE_CONFIG store_mode=1 keeps the
// workspace path).
void prefer_cluster_reduce(const GemmProblem& g, int smem_limit, tdx_config* cfg) {
    // a ranked in-cluster configuration whose K split was changed afterwards may no longer be one
    if (cfg->kernel == TDX_KERNEL_UMMA && cfg->store_mode == 3 &&
        umma_config_reason(*cfg, g.transB == 0, ceil_div(g.K, 64), smem_limit, false, g.N) != nullptr)
        cfg->store_mode = 1;
    if (cfg->kernel != TDX_KERNEL_UMMA || cfg->split_k < 2 || cfg->store_mode != 1 || cfg->fit == 3) return;
    const tdx_config* forced = forced_config();
    if (forced != nullptr && forced->store_mode == 1) return;
    tdx_config c = *cfg;
    c.store_mode = 3;
    c.fit = 1;
    c.stages = std::min(c.stages, umma_max_stages(c.tile_m, c.tile_n, smem_limit, 3));
    if (umma_config_reason(c, g.transB == 0, ceil_div(g.K, 64), smem_limit, false, g.N) == nullptr) *cfg = c;
}

int run_gemm_umma(DeviceCtx* ctx, const GemmProblem& g, float alpha, const void* A, const void* B, void* C,
                  const tdx_config& cfg, void* ws, size_t ws_bytes, bool internal_ws, cudaStream_t st, float beta = 0.0f,
                  const PieceInfo* pieces = nullptr, bool c_f32 = false) {
    // c_f32: bf16 operands, fp32 result (C points to floats); bf16 pieces imply it
    const PieceInfo* form = pieces;                            // any of the forms above
    if (pieces && pieces->seg_kb == 0) pieces = nullptr;       // from here on `pieces` means the fp32 piece form only
    const int64_t num_kb = ceil_div(g.K, 64);
    const int64_t k_cols = (form && form->cols > 0) ? form->cols : g.K;      // columns the K-major operands really have
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
    if (pieces) {
        if (p.a_mn_major || p.b_mn_major) return fail(TDX_ERR_CONFIG, "the fp32 GEMM from bf16 pieces runs K-major operands");
        // smallest terms first, the hi * hi products last: (hi, lo) (lo, hi) (mid, mid) (hi, mid) (mid, hi) (hi, hi)
        const int a_seg[6] = {0, 2, 1, 0, 1, 0}, b_seg[6] = {2, 0, 1, 1, 0, 0};
        for (int i = 0; i < 6; ++i) { p.a_seg[i] = a_seg[i]; p.b_seg[i] = b_seg[i]; }
        p.seg_kb = pieces->seg_kb;
        p.Cf = static_cast<float*>(C);
        p.C = nullptr;
        p.vec_store = (g.N % 4 == 0) && (reinterpret_cast<uintptr_t>(C) % 16 == 0) && (pieces->batch_c % 4 == 0);
        if (pieces->batch > 1) {
            if (static_cast<long long>(pieces->batch) * p.tiles_m * p.tiles_n * cfg.split_k >= (1LL << 31))
                return fail(TDX_ERR_UNSUPPORTED, "too many batched tiles for one launch");
            p.batch = static_cast<int>(pieces->batch);
            p.batch_c = pieces->batch_c;
        }
    }
    const int64_t nbatch = form ? form->batch : 1;
    const long long out_batch_c = form ? static_cast<long long>(form->batch_c) : 0;
    if (!pieces && nbatch > 1) {
        if (static_cast<long long>(nbatch) * p.tiles_m * p.tiles_n * cfg.split_k >= (1LL << 31))
            return fail(TDX_ERR_UNSUPPORTED, "too many batched tiles for one launch");
        p.batch = static_cast<int>(nbatch);
        p.batch_c = out_batch_c;
        if (!c_f32) p.vec_store = p.vec_store && (out_batch_c % 8 == 0);
    }
    // batch strides of the operands (elements); a shared operand is a tensor with a single batch
    const int64_t a_rows_stored = g.transA ? g.K : g.M, a_cols_stored = g.transA ? g.M : k_cols;
    const int64_t b_rows_stored = g.transB ? g.N : g.K, b_cols_stored = g.transB ? k_cols : g.N;
    const int64_t a_bstride = (form && form->batch_a >= 0) ? form->batch_a : a_rows_stored * a_cols_stored;
    const int64_t b_bstride = (form && form->batch_b >= 0) ? form->batch_b : b_rows_stored * b_cols_stored;
    p.a_shared = (nbatch > 1 && a_bstride == 0) ? 1 : 0;
    p.b_shared = (nbatch > 1 && b_bstride == 0) ? 1 : 0;
    const uint64_t a_nb = p.a_shared ? 1 : static_cast<uint64_t>(nbatch), b_nb = p.b_shared ? 1 : static_cast<uint64_t>(nbatch);
    const uint64_t a_bbytes = static_cast<uint64_t>(p.a_shared ? a_rows_stored * a_cols_stored : a_bstride) * 2;
    const uint64_t b_bbytes = static_cast<uint64_t>(p.b_shared ? b_rows_stored * b_cols_stored : b_bstride) * 2;
    if (c_f32 && !pieces) {
        p.Cf = static_cast<float*>(C);
        p.C = nullptr;
        p.vec_store = (g.N % 4 == 0) && (reinterpret_cast<uintptr_t>(C) % 16 == 0);
    }
    const bool f32_result = pieces != nullptr || c_f32;

    // K-balanced plan: the tiles x K blocks units dealt evenly to all CTAs; partial tiles in up to max_seg slots
    DevicePlan kplan;
    const bool k_balanced = cfg.fit == 3 && !f32_result && nbatch == 1 && beta == 0.0f;
    if (cfg.fit == 3 && !k_balanced) return fail(TDX_ERR_CONFIG, "the K-balanced plan serves the plain bf16 GEMM only");
    if (k_balanced) {
        int rcp = get_k_balanced_plan(ctx, g.M, g.N, num_kb, cfg.tile_m, cfg.tile_n, &kplan);
        if (rcp) return rcp;
        if (!kplan.fitted) return fail(TDX_ERR_CONFIG, "no K-balanced plan for this shape");
        const size_t need = static_cast<size_t>(kplan.max_seg) * g.M * g.N * sizeof(float);
        if (internal_ws) {
            int rcw = ensure_ws(ctx, need, &ws);
            if (rcw) return rcw;
        } else if (ws == nullptr || ws_bytes < need || reinterpret_cast<uintptr_t>(ws) % 256) {
            return fail(TDX_ERR_WORKSPACE, "the K-balanced plan needs %zu bytes of 256-byte aligned workspace", need);
        }
        p.partial = static_cast<float*>(ws);
        p.split_k = kplan.max_seg > 1 ? kplan.max_seg : 2;      // > 1: the epilogue writes partial tiles to their slots
        p.kb_per_split = p.num_kb;
        p.tiles = kplan.dev;
        p.rounds = kplan.rounds;
        p.b_box = 64;
    }
    // split-K summed inside clusters: neither workspace nor reduction kernel
    const bool cluster_reduce = cfg.store_mode == 3 && cfg.split_k > 1;
    if (cluster_reduce) {
        if (static_cast<long long>(nbatch) * p.tiles_m * p.tiles_n * cfg.split_k >= (1LL << 31))
            return fail(TDX_ERR_UNSUPPORTED, "too many tiles for one launch");
        p.cluster_reduce = 1;
    }
    if (cfg.split_k > 1 && !cluster_reduce) {
        const size_t need = static_cast<size_t>(cfg.split_k) * g.M * g.N * sizeof(float) * nbatch;
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
    if (p.a_mn_major && nbatch > 1) {
        uint64_t dims[3] = {static_cast<uint64_t>(g.M), static_cast<uint64_t>(g.K), a_nb};
        uint64_t str[2] = {static_cast<uint64_t>(g.M) * 2, a_bbytes};
        uint32_t box[3] = {64, 64, 1};
        rc = get_tensor_map(ctx, A, 3, dims, str, box, &ma);
    } else if (p.a_mn_major) {
        uint64_t dims[2] = {static_cast<uint64_t>(g.M), static_cast<uint64_t>(g.K)};
        uint64_t str[1] = {static_cast<uint64_t>(g.M) * 2};
        uint32_t box[2] = {64, 64};
        rc = get_tensor_map(ctx, A, 2, dims, str, box, &ma);
    } else if (nbatch > 1) {
        uint64_t dims[3] = {static_cast<uint64_t>(k_cols), static_cast<uint64_t>(g.M), a_nb};
        uint64_t str[2] = {static_cast<uint64_t>(k_cols) * 2, a_bbytes};
        uint32_t box[3] = {64, 128, 1};
        rc = get_tensor_map(ctx, A, 3, dims, str, box, &ma);
    } else {
        uint64_t dims[2] = {static_cast<uint64_t>(k_cols), static_cast<uint64_t>(g.M)};
        uint64_t str[1] = {static_cast<uint64_t>(k_cols) * 2};
        uint32_t box[2] = {64, 128};
        rc = get_tensor_map(ctx, A, 2, dims, str, box, &ma);
    }
    if (rc) return rc;
    // tile widths fitted to the number of CTAs (see plan_fitted_tiles): B then arrives in 64-row copies
    int plan_grid = 0;
    if (cfg.fit != 1 && cfg.fit != 3 && cfg.split_k == 1 && cfg.tile_n >= 192 && cfg.tile_n % 64 == 0 && nbatch == 1) {
        DevicePlan dp;
        rc = get_tile_plan(ctx, g.M, g.N, num_kb, cfg.tile_m, cfg.tile_n, cfg.raster, cfg.fit == 2 ? 0.0 : 0.03, &dp);
        if (rc) return rc;
        if (dp.fitted) {
            p.tiles = dp.dev;
            p.rounds = dp.rounds;
            p.b_box = 64;
            plan_grid = dp.grid;
        }
    }
    if (p.b_mn_major && nbatch > 1) {
        uint64_t dims[3] = {static_cast<uint64_t>(g.N), static_cast<uint64_t>(g.K), b_nb};
        uint64_t str[2] = {static_cast<uint64_t>(g.N) * 2, b_bbytes};
        uint32_t box[3] = {64, 64, 1};
        rc = get_tensor_map(ctx, B, 3, dims, str, box, &mb);
    } else if (p.b_mn_major) {
        uint64_t dims[2] = {static_cast<uint64_t>(g.N), static_cast<uint64_t>(g.K)};
        uint64_t str[1] = {static_cast<uint64_t>(g.N) * 2};
        uint32_t box[2] = {64, 64};
        rc = get_tensor_map(ctx, B, 2, dims, str, box, &mb);
    } else if (nbatch > 1) {
        uint64_t dims[3] = {static_cast<uint64_t>(k_cols), static_cast<uint64_t>(g.N), b_nb};
        uint64_t str[2] = {static_cast<uint64_t>(k_cols) * 2, b_bbytes};
        uint32_t box[3] = {64, static_cast<uint32_t>(cfg.tile_n), 1};
        rc = get_tensor_map(ctx, B, 3, dims, str, box, &mb);
    } else {
        uint64_t dims[2] = {static_cast<uint64_t>(k_cols), static_cast<uint64_t>(g.N)};
        uint64_t str[1] = {static_cast<uint64_t>(k_cols) * 2};
        uint32_t box[2] = {64, static_cast<uint32_t>(p.tiles ? 64 : cfg.tile_n)};
        rc = get_tensor_map(ctx, B, 2, dims, str, box, &mb);
    }
    if (rc) return rc;

    CUtensorMap mc = ma;   // unused unless the staged epilogue is on
    // the accumulate term is read by the direct-store epilogue (and by the split-K reduction) only
    p.tma_store = (cfg.store_mode == 2 && cfg.split_k == 1 && p.vec_store && beta == 0.0f && !f32_result && nbatch == 1) ? 1 : 0;
    if (p.tma_store) {
        uint64_t dims[2] = {static_cast<uint64_t>(g.N), static_cast<uint64_t>(g.M)};
        uint64_t str[1] = {static_cast<uint64_t>(g.N) * 2};
        uint32_t box[2] = {32, 32};
        rc = get_tensor_map(ctx, C, 2, dims, str, box, &mc, 64);
        if (rc) return rc;
    }
    if (k_balanced) plan_grid = kplan.grid;
    if (cluster_reduce) {
        // the summed slices leave through the copy engine when the rows of C (and the batches) are 16-byte aligned;
        // else 16-byte (or element-wise) stores from registers
        const uint64_t esz = f32_result ? 4 : 2;
        if (p.vec_store && (nbatch == 1 || (static_cast<uint64_t>(out_batch_c) * esz) % 16 == 0)) {
            uint64_t dims[3] = {static_cast<uint64_t>(g.N), static_cast<uint64_t>(g.M), static_cast<uint64_t>(nbatch)};
            uint64_t str[2] = {static_cast<uint64_t>(g.N) * esz, static_cast<uint64_t>(out_batch_c) * esz};
            uint32_t box[3] = {32, 32, 1};
            rc = get_tensor_map(ctx, C, nbatch > 1 ? 3 : 2, dims, str, box, &mc, f32_result ? 128 : 64, nullptr, f32_result);
            if (rc) return rc;
            p.cluster_tma = f32_result ? 2 : 1;
        }
        return launch_umma(ctx, false, ma, mb, mc, p, st, false, nullptr, nullptr, 0);
    }
    if (p.partial != nullptr && p.split_k > 1) {
        // fp32 partial tiles leave through shared memory and the copy engine (whole 128-byte lines) when the workspace
        // rows allow it and the pipeline leaves room for the staging blocks; else straight from registers
        const size_t room = static_cast<size_t>(ctx->smem_optin - kStaticSmemReserve);
        const size_t want = static_cast<size_t>(p.stages) * ((p.bm + p.bn) * 128) + 1024 + partial_staging_bytes(p.bm);
        if (g.N % 4 == 0 && reinterpret_cast<uintptr_t>(p.partial) % 16 == 0 && want <= room) {
            const uint64_t slots = static_cast<uint64_t>(p.split_k) * static_cast<uint64_t>(nbatch);
            uint64_t dims[3] = {static_cast<uint64_t>(g.N), static_cast<uint64_t>(g.M), slots};
            uint64_t str[2] = {static_cast<uint64_t>(g.N) * 4, static_cast<uint64_t>(g.N) * 4 * static_cast<uint64_t>(g.M)};
            uint32_t box[3] = {32, 32, 1};
            rc = get_tensor_map(ctx, p.partial, 3, dims, str, box, &mc, 128, nullptr, true);
            if (rc) return rc;
            p.partial_tma = 1;
        }
    }
    rc = launch_umma(ctx, false, ma, mb, mc, p, st, false, nullptr, nullptr, plan_grid);
    if (rc) return rc;
    if (k_balanced) {
        const long long MN = static_cast<long long>(g.M) * g.N;
        const int vec8 = (p.vec_store && cfg.tile_n % 8 == 0) ? 1 : 0;
        const long long work = vec8 ? MN / 8 : MN;
        cudaLaunchConfig_t lc;
        std::memset(&lc, 0, sizeof lc);
        lc.gridDim = dim3(static_cast<unsigned>(std::max<long long>(1, std::min<long long>(ceil_div(work, 256), 148LL * 16))));
        lc.blockDim = dim3(256);
        lc.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        lc.attrs = attr;
        lc.numAttrs = 1;
        TDX_CUDA(cudaLaunchKernelEx(&lc, tdx::splitk_reduce_var_kernel, MN, static_cast<int>(g.N), cfg.tile_m, cfg.tile_n, kplan.tiles_n,
                                    kplan.nseg, static_cast<const float*>(p.partial), alpha, p.C, vec8, 0.0f));
        g_launches.fetch_add(1);
        return TDX_OK;
    }
    if (cfg.split_k > 1 && f32_result) {
        // fp32 result: partial sums (fp32, dense) -> alpha * sum + beta * C
        const long long MN = static_cast<long long>(g.M) * g.N;
        const int vec4 = (MN % 4 == 0 && reinterpret_cast<uintptr_t>(C) % 16 == 0 && out_batch_c % 4 == 0) ? 1 : 0;
        const int grid = static_cast<int>(std::min<long long>(ceil_div((vec4 ? MN / 4 : MN) * nbatch, 256), 148LL * 16));
        cudaLaunchConfig_t lc;
        std::memset(&lc, 0, sizeof lc);
        lc.gridDim = dim3(static_cast<unsigned>(std::max(grid, 1)));
        lc.blockDim = dim3(256);
        lc.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        lc.attrs = attr;
        lc.numAttrs = 1;
        TDX_CUDA(cudaLaunchKernelEx(&lc, tdx::splitk_reduce_f32_kernel, MN, cfg.split_k, static_cast<const float*>(p.partial), alpha,
                                    beta, static_cast<float*>(C), vec4, static_cast<int>(nbatch), out_batch_c));
        g_launches.fetch_add(1);
        return TDX_OK;
    }
    if (cfg.split_k > 1) {
        const long long MN = static_cast<long long>(g.M) * g.N;
        const int vec8 = (p.vec_store && MN % 8 == 0) ? 1 : 0;
        const long long work = (vec8 ? MN / 8 : MN) * nbatch;
        const int grid = static_cast<int>(std::min<long long>(ceil_div(work, 256), 148LL * 16));
        rc = launch_splitk_reduce(std::max(grid, 1), st, MN, static_cast<int>(g.N), cfg.split_k, p.partial, alpha, p.C, vec8, beta,
                                  static_cast<int>(nbatch), out_batch_c);
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
        rc = get_tile_plan(ctx, g.M, g.N, num_kb, 256, cfg.tile_n, cfg.raster, 0.0, &dp, true);
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
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;      // as for the single-CTA kernel
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = 2;
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

    // tile widths fitted to the CTA count, as for the GEMM (streamed filter): the filter slices then arrive in 64-row
    // copies
    int plan_grid = 0;
    if (!p.b_resident && cfg.fit != 1 && cfg.tile_n >= 192 && cfg.tile_n % 64 == 0) {
        DevicePlan dp;
        int rcp = get_tile_plan(ctx, static_cast<int64_t>(p.tiles_m) * cfg.tile_m, c.Cout, p.num_kb, cfg.tile_m, cfg.tile_n,
                                cfg.raster, cfg.fit == 2 ? 0.0 : 0.03, &dp);
        if (rcp) return rcp;
        if (dp.fitted) {
            p.tiles = dp.dev;
            p.rounds = dp.rounds;
            p.b_box = 64;
            plan_grid = dp.grid;
        }
    }
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
        uint32_t box[3] = {64, 1, static_cast<uint32_t>(p.tiles ? 64 : cfg.tile_n)};
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
    return launch_umma(ctx, true, ma, mb, mc, p, st, halo, &ma_row, &mc_row, plan_grid);
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
                                reinterpret_cast<uintptr_t>(A) % 16 == 0 && reinterpret_cast<uintptr_t>(B) % 16 == 0 &&
                                reinterpret_cast<uintptr_t>(C) % 16 == 0;
        // small problems are launch-bound: programmatic stream serialization lets a call's launch overlap the
        // previous kernel's tail (the kernels wait on the device before touching memory)
        cudaLaunchConfig_t lc;
        std::memset(&lc, 0, sizeof lc);
        lc.gridDim = grid;
        lc.blockDim = dim3(256);
        lc.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        lc.attrs = attr;
        lc.numAttrs = 1;
        if (rowmajor16) {
            lc.dynamicSmemBytes = tdx::kSmallRowmajorSmem;
            TDX_CUDA(cudaLaunchKernelEx(&lc, tdx::sgemm_small_rowmajor_kernel, (int)g.M, (int)g.N, (int)g.K, alpha, a, b, c));
        } else
            TDX_CUDA(cudaLaunchKernelEx(&lc, tdx::sgemm_small_kernel, (int)g.M, (int)g.N, (int)g.K, sa_i, sa_k, sb_k, sb_j, alpha,
                                        a, b, c, ba.beta, static_cast<long long>(ba.stride_a), static_cast<long long>(ba.stride_b),
                                        static_cast<long long>(ba.stride_c)));
    }
    TDX_CUDA(cudaGetLastError());
    g_launches.fetch_add(1);
    return TDX_OK;
}

// fp32 GEMM on the tensor cores.  Each fp32 operand is cut into three bf16 pieces (hi + mid + lo = the value, all 24
// significand bits), written K-major whatever the operand's own layout, and the tensor-core kernel accumulates the six
// piece pairs that matter ((mid, lo), (lo, mid) and (lo, lo) are below 2^-24 of the product) in fp32 -- six times
// the MMA work of a bf16 GEMM, still several times faster than fp32 FMAs.  Scratch for the pieces is grown on demand.
int ensure_pieces(DeviceCtx* ctx, int slot, size_t bytes, void** out) {
    if (ctx->pieces_bytes[slot] < bytes) {
        if (ctx->pieces[slot]) TDX_CUDA(cudaFree(ctx->pieces[slot]));
        ctx->pieces[slot] = nullptr;
        ctx->pieces_bytes[slot] = 0;
        TDX_CUDA(cudaMalloc(&ctx->pieces[slot], bytes));
        ctx->pieces_bytes[slot] = bytes;
    }
    *out = ctx->pieces[slot];
    return TDX_OK;
}

int resolve_gemm_config(const GemmProblem& g, const tdx_config* user, int sm_count, int smem_limit, tdx_config* out);
bool model_pick_direct_store(const GemmProblem& g, int sm_count, int smem_limit, tdx_config* out);

constexpr size_t kPiecesMaxBytes = size_t(3) << 30;     // per operand; larger problems go batch by batch, or to the CUDA cores

bool gemm_f32_pieces_fit(const GemmProblem& g) {
    if (g.M >= (1LL << 31) || g.N >= (1LL << 31) || g.K >= (1LL << 28)) return false;
    const int64_t Kp = ceil_div(g.K, 64) * 64;
    return static_cast<size_t>(std::max(g.M, g.N)) * 3 * Kp * 2 <= kPiecesMaxBytes;
}

// The automatic choice for fp32: the pieces cost two extra kernels and six times the MMA work, which pays once the
// problem has about 2^28 multiply-adds (measured: 512^3 is still faster on the CUDA cores, 1024^3 and the paper's
// 6 x 196 x 256 x 2305 batch are not; the 256^3 configuration is launch-bound either way).
bool prefer_f32_pieces(const GemmProblem& g, int64_t batch) {
    if (!gemm_f32_pieces_fit(g) || g.M < 64 || g.N < 64 || g.K < 64) return false;
    return static_cast<double>(batch) * g.M * g.N * g.K >= 268435456.0;
}

int run_gemm_f32_pieces(DeviceCtx* ctx, const GemmProblem& g, float alpha, const void* A, const void* B, void* C,
                        cudaStream_t st, const BatchArgs& ba, const tdx_config* user_cfg) {
    if (!gemm_f32_pieces_fit(g)) return fail(TDX_ERR_UNSUPPORTED, "problem too large for the fp32 tensor-core path");
    const int64_t Kp = ceil_div(g.K, 64) * 64;
    const size_t a_one = static_cast<size_t>(g.M) * 3 * Kp * 2, b_one = static_cast<size_t>(g.N) * 3 * Kp * 2;
    // all batches at once when the pieces fit the budget, else one batch at a time; a shared operand (stride 0) once
    const bool a_shared = ba.batch > 1 && ba.stride_a == 0, b_shared = ba.batch > 1 && ba.stride_b == 0;
    int64_t chunk = ba.batch;
    while (chunk > 1 && (a_one * (a_shared ? 1 : chunk) > kPiecesMaxBytes || b_one * (b_shared ? 1 : chunk) > kPiecesMaxBytes))
        chunk = (chunk + 1) / 2;
    if (chunk > 65535) chunk = 65535;
    void *pa, *pb;
    int rc;
    if ((rc = ensure_pieces(ctx, 0, a_one * (a_shared ? 1 : chunk), &pa))) return rc;
    if ((rc = ensure_pieces(ctx, 1, b_one * (b_shared ? 1 : chunk), &pb))) return rc;
    // the tensor-core problem: K-major A'' (M x 3Kp) and B'' (N x 3Kp), six piece pairs of Kp each
    GemmProblem gg{g.M, g.N, 6 * Kp, 0, 1, TDX_BF16};
    tdx_config want;
    std::memset(&want, 0, sizeof want);
    if (user_cfg) want = *user_cfg;
    want.kernel = TDX_KERNEL_UMMA;
    want.store_mode = (user_cfg && user_cfg->store_mode == 3) ? 3 : 1;      // fp32 results: direct stores, or summed inside clusters
    want.cta_pair = 1;          // split_k: the caller's, else chosen like for any GEMM with few tiles and a long reduction
    if (ba.batch == 1 && want.tile_m == 0 && want.tile_n == 0 && want.split_k == 0 && want.stages == 0) {
        // no tile given: the cost model's first choice among the direct-store candidates of the piece problem
        // (for the paper's batch, ranking the problem with all batches' row blocks stacked -- which then sums its K
        // split inside clusters -- measured 40.9 us against 38.8 for the heuristic tile with a reduction launch)
        tdx_config ranked;
        if (model_pick_direct_store(gg, ctx->sm_count, ctx->smem_optin, &ranked)) {
            want.tile_m = ranked.tile_m;
            want.tile_n = ranked.tile_n;
            want.split_k = ranked.split_k;
            want.raster = ranked.raster;
            if (ranked.store_mode == 3) want.store_mode = 3;
        }
    }
    tdx_config cfg;
    rc = resolve_gemm_config(gg, &want, ctx->sm_count, ctx->smem_optin, &cfg);
    if (rc) return rc;
    long long sa_i, sa_k, sb_k, sb_j;
    gemm_strides(g, &sa_i, &sa_k, &sb_k, &sb_j);
    PieceInfo pi;
    pi.seg_kb = static_cast<int>(Kp / 64);
    pi.cols = 3 * Kp;
    const float* a = static_cast<const float*>(A);
    const float* b = static_cast<const float*>(B);
    float* c = static_cast<float*>(C);
    // one launch splits both operands (nb_b == 0: only the first)
    auto split = [&](const float* src_a, int rows_a, long long s_row_a, long long s_k_a, long long bstride_a, int64_t nb_a, void* dst_a,
                     const float* src_b, int rows_b, long long s_row_b, long long s_k_b, long long bstride_b, int64_t nb_b,
                     void* dst_b) -> int {
        const int rows_max = nb_b > 0 ? std::max(rows_a, rows_b) : rows_a;
        dim3 grid(static_cast<unsigned>(ceil_div(Kp, 64)), static_cast<unsigned>(ceil_div(rows_max, 32)),
                  static_cast<unsigned>(nb_a + nb_b));
        if (grid.y > 65535 || nb_a + nb_b > 65535) return fail(TDX_ERR_UNSUPPORTED, "operand too tall for the piece kernel");
        tdx::SplitOperand o0{rows_a, s_row_a, s_k_a, bstride_a, src_a, static_cast<__nv_bfloat16*>(dst_a)};
        tdx::SplitOperand o1{rows_b, s_row_b, s_k_b, bstride_b, src_b, static_cast<__nv_bfloat16*>(dst_b)};
        cudaLaunchConfig_t lc;
        std::memset(&lc, 0, sizeof lc);
        lc.gridDim = grid;
        lc.blockDim = dim3(256);
        lc.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        lc.attrs = attr;
        lc.numAttrs = 1;
        TDX_CUDA(cudaLaunchKernelEx(&lc, tdx::split_f32_bf16x3_kernel, static_cast<int>(g.K), static_cast<int>(Kp),
                                    static_cast<int>(nb_a), o0, o1));
        TDX_CUDA(cudaGetLastError());
        g_launches.fetch_add(1);
        return TDX_OK;
    };
    for (int64_t b0 = 0; b0 < ba.batch; b0 += chunk) {
        const int64_t nb = std::min(chunk, ba.batch - b0);
        // B'' rows are the columns j of op(B): element (j, k) at B[k * sb_k + j * sb_j]
        const bool do_a = !a_shared || b0 == 0, do_b = !b_shared || b0 == 0;
        const float* src_a = a + (a_shared ? 0 : b0 * ba.stride_a);
        const float* src_b = b + (b_shared ? 0 : b0 * ba.stride_b);
        const int64_t nb_a = a_shared ? 1 : nb, nb_b = b_shared ? 1 : nb;
        if (do_a && do_b) {
            if ((rc = split(src_a, static_cast<int>(g.M), sa_i, sa_k, ba.stride_a, nb_a, pa,
                            src_b, static_cast<int>(g.N), sb_j, sb_k, ba.stride_b, nb_b, pb))) return rc;
        } else if (do_a) {
            if ((rc = split(src_a, static_cast<int>(g.M), sa_i, sa_k, ba.stride_a, nb_a, pa, nullptr, 0, 0, 0, 0, 0, nullptr))) return rc;
        } else if (do_b) {
            if ((rc = split(src_b, static_cast<int>(g.N), sb_j, sb_k, ba.stride_b, nb_b, pb, nullptr, 0, 0, 0, 0, 0, nullptr))) return rc;
        }
        if (nb > 1 && !a_shared && !b_shared) {
            // all batches of the chunk in one launch: 3-D operands, items over batch x tiles x splits
            PieceInfo pb_info = pi;
            pb_info.batch = nb;
            pb_info.batch_c = ba.stride_c;
            tdx_config bc = cfg;
            if (!user_cfg || user_cfg->split_k == 0) {
                // the batches already multiply the tiles: split K only as far as it takes to give every SM an item
                const int64_t tiles = nb * ceil_div(g.M, cfg.tile_m) * ceil_div(g.N, cfg.tile_n);
                int64_t sk = std::max<int64_t>(1, std::min<int64_t>({32, ctx->sm_count / std::max<int64_t>(1, tiles), gg.K / 64 / 4}));
                while (sk > 1 && (sk - 1) * ceil_div(gg.K / 64, sk) >= gg.K / 64) --sk;
                bc.split_k = static_cast<int>(sk);
            }
            if (!user_cfg) prefer_cluster_reduce(gg, ctx->smem_optin, &bc);
            rc = run_gemm_umma(ctx, gg, alpha, pa, pb, c + b0 * ba.stride_c, bc, nullptr, 0, true, st, ba.beta, &pb_info);
            if (rc) return rc;
            continue;
        }
        tdx_config one = cfg;
        if (!user_cfg) prefer_cluster_reduce(gg, ctx->smem_optin, &one);
        for (int64_t i = 0; i < nb; ++i) {
            const char* ai = static_cast<const char*>(pa) + (a_shared ? 0 : i * a_one);
            const char* bi = static_cast<const char*>(pb) + (b_shared ? 0 : i * b_one);
            rc = run_gemm_umma(ctx, gg, alpha, ai, bi, c + (b0 + i) * ba.stride_c, one, nullptr, 0, true, st, ba.beta, &pi);
            if (rc) return rc;
        }
    }
    return TDX_OK;
}

// Batched bf16 GEMM with accumulate on the tensor cores, all batches in one launch.
//   direct: every batch's operands meet the copy engine's layout rules as they are -> 3-D tensor maps over the
//           caller's buffers (contiguous dimension, the other one, batch), whatever the transposes.
//   else:   both operands are first copied K-major with K padded to a multiple of 64 (pad_k_bf16_kernel, one launch for
//           both; zeros add nothing to the sums), which removes every alignment rule -- the paper's K = 2305 qualifies --
//           exactly as the fp32 piece path does.
// Tile shape from the cost model's direct-store ranking of one batch's problem; K split only as far as it takes to give
// every SM an item, reduced in a fixed order by one launch for all batches (it also applies beta).
int run_gemm_batched_bf16(DeviceCtx* ctx, const GemmProblem& g, float alpha, float beta, const void* A, int64_t strideA,
                          const void* B, int64_t strideB, void* C, int64_t strideC, int64_t batch, bool direct,
                          cudaStream_t st) {
    GemmProblem gg = g;
    const void *pa = A, *pb = B;
    PieceInfo form;
    form.batch = batch;
    form.batch_c = strideC;
    const bool a_shared = batch > 1 && strideA == 0, b_shared = batch > 1 && strideB == 0;
    if (direct) {
        form.batch_a = strideA;
        form.batch_b = strideB;
    } else {
        const int64_t Kp = ceil_div(g.K, 64) * 64;
        const int64_t nb_a = a_shared ? 1 : batch, nb_b = b_shared ? 1 : batch;
        const size_t a_bytes = static_cast<size_t>(g.M) * Kp * 2 * nb_a, b_bytes = static_cast<size_t>(g.N) * Kp * 2 * nb_b;
        if (a_bytes > kPiecesMaxBytes || b_bytes > kPiecesMaxBytes || nb_a + nb_b > 65535 || ceil_div(std::max(g.M, g.N), 32) > 65535)
            return TDX_ERR_UNSUPPORTED;            // the caller falls back to the generic kernel
        void *da, *db;
        int rc;
        if ((rc = ensure_pieces(ctx, 0, a_bytes, &da))) return rc;
        if ((rc = ensure_pieces(ctx, 1, b_bytes, &db))) return rc;
        long long sa_i, sa_k, sb_k, sb_j;
        gemm_strides(g, &sa_i, &sa_k, &sb_k, &sb_j);
        tdx::PadOperand o0{static_cast<int>(g.M), sa_i, sa_k, strideA, static_cast<const __nv_bfloat16*>(A), static_cast<__nv_bfloat16*>(da)};
        // rows of the copy of B are the columns j of op(B): element (j, k) at B[k * sb_k + j * sb_j]
        tdx::PadOperand o1{static_cast<int>(g.N), sb_j, sb_k, strideB, static_cast<const __nv_bfloat16*>(B), static_cast<__nv_bfloat16*>(db)};
        cudaLaunchConfig_t lc;
        std::memset(&lc, 0, sizeof lc);
        lc.gridDim = dim3(static_cast<unsigned>(Kp / 64), static_cast<unsigned>(ceil_div(std::max(g.M, g.N), 32)),
                          static_cast<unsigned>(nb_a + nb_b));
        lc.blockDim = dim3(256);
        lc.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        lc.attrs = attr;
        lc.numAttrs = 1;
        TDX_CUDA(cudaLaunchKernelEx(&lc, tdx::pad_k_bf16_kernel, static_cast<int>(g.K), static_cast<int>(Kp), static_cast<int>(nb_a), o0, o1));
        TDX_CUDA(cudaGetLastError());
        g_launches.fetch_add(1);
        gg = GemmProblem{g.M, g.N, Kp, 0, 1, TDX_BF16};
        pa = da;
        pb = db;
        form.cols = Kp;
        form.batch_a = a_shared ? 0 : g.M * Kp;
        form.batch_b = b_shared ? 0 : g.N * Kp;
    }
    tdx_config want;
    std::memset(&want, 0, sizeof want);
    want.kernel = TDX_KERNEL_UMMA;
    want.store_mode = 1;          // direct stores: they carry the batch offset and the accumulate term
    want.cta_pair = 1;
    want.fit = 1;
    // The batches multiply the tiles, so the ranking sees them: one problem with the row blocks of all batches stacked
    // (the paper's 6 x 196 x 256 x 2305 batch: 128 x 128 tiles with a K split, 19.4 us; ranked on one batch alone it
    // took 128 x 32 tiles without a split, 28.7 us).  256-row tiles only where they waste no more rows than 128-row ones.
    tdx_config ranked;
    GemmProblem stacked = gg;
    stacked.M = batch * ceil_div(g.M, 128) * 128;
    if (model_pick_direct_store(stacked, ctx->sm_count, ctx->smem_optin, &ranked)) {
        want.tile_m = (ceil_div(g.M, 256) * 256 > ceil_div(g.M, 128) * 128) ? 128 : ranked.tile_m;
        want.tile_n = ranked.tile_n;
        want.raster = ranked.raster;
        want.split_k = ranked.split_k;
        if (ranked.store_mode == 3 && want.tile_m == ranked.tile_m) want.store_mode = 3;
    }
    const tdx_config* forced = forced_config();          // TDX_FORCE_CONFIG: tile shape, depth and K split as given
    if (forced != nullptr) {
        if (forced->tile_m) want.tile_m = forced->tile_m;
        if (forced->tile_n) want.tile_n = forced->tile_n;
        if (forced->stages) want.stages = forced->stages;
        if (forced->split_k) want.split_k = forced->split_k;
        want.raster = forced->raster;
    }
    tdx_config cfg;
    int rc = resolve_gemm_config(gg, &want, ctx->sm_count, ctx->smem_optin, &cfg);
    if (rc) return rc;
    if (batch > 1 && !(forced != nullptr && forced->split_k)) {
        // the ranked K split belongs to the stacked problem; keep it within what gives every SM an item
        const int64_t num_kb = ceil_div(gg.K, 64);
        const int64_t tiles = batch * ceil_div(g.M, cfg.tile_m) * ceil_div(g.N, cfg.tile_n);
        int64_t sk = std::max<int64_t>(1, std::min<int64_t>({32, ceil_div(ctx->sm_count, std::max<int64_t>(1, tiles)), num_kb / 4,
                                                            std::max<int64_t>(1, cfg.split_k)}));
        if (cfg.split_k <= 1) sk = std::max<int64_t>(1, std::min<int64_t>({32, ctx->sm_count / std::max<int64_t>(1, tiles), num_kb / 4}));
        while (sk > 1 && (sk - 1) * ceil_div(num_kb, sk) >= num_kb) --sk;
        cfg.split_k = static_cast<int>(sk);
    }
    prefer_cluster_reduce(gg, ctx->smem_optin, &cfg);
    return run_gemm_umma(ctx, gg, alpha, pa, pb, C, cfg, nullptr, 0, true, st, beta, &form);
}

int run_gemm_generic(DeviceCtx* ctx, const GemmProblem& g, float alpha, const void* A, const void* B, void* C,
                     cudaStream_t st, const BatchArgs& ba = BatchArgs(), bool c_f32 = false,
                     const tdx::BoundsCheck* bounds_override = nullptr) {
    long long sa_i, sa_k, sb_k, sb_j;
    gemm_strides(g, &sa_i, &sa_k, &sb_k, &sb_j);
    const long long total = g.M * g.N * ba.batch;
    const int grid = static_cast<int>(std::min<long long>(ceil_div(total, 256), static_cast<long long>(ctx->sm_count) * 32));
    // debug mode: the extents the caller's shapes and strides imply, checked index by index in the kernel
    tdx::BoundsCheck bc{0, 0, 0, 0, 0, ctx->status_ptr};
    if (bounds_override != nullptr) bc = *bounds_override;
    else if (debug_bounds_enabled()) {
        bc.on = 1;
        bc.a_elems = (ba.batch - 1) * ba.stride_a + g.M * g.K;
        bc.b_elems = (ba.batch - 1) * ba.stride_b + g.K * g.N;
        bc.c_elems = (ba.batch - 1) * ba.stride_c + g.M * g.N;
    }
    if (g.dtype == TDX_BF16 && c_f32)      // bf16 operands, fp32 result
        tdx::gemm_generic_kernel<__nv_bfloat16, float><<<grid, 256, 0, st>>>(
            g.M, g.N, g.K, sa_i, sa_k, sb_k, sb_j, alpha, static_cast<const __nv_bfloat16*>(A),
            static_cast<const __nv_bfloat16*>(B), static_cast<float*>(C), ba.beta, ba.batch, ba.stride_a, ba.stride_b, ba.stride_c, bc);
    else if (g.dtype == TDX_F32)
        tdx::gemm_generic_kernel<float, float><<<grid, 256, 0, st>>>(g.M, g.N, g.K, sa_i, sa_k, sb_k, sb_j, alpha,
                                                                    static_cast<const float*>(A),
                                                                    static_cast<const float*>(B), static_cast<float*>(C),
                                                                    ba.beta, ba.batch, ba.stride_a, ba.stride_b, ba.stride_c, bc);
    else
        tdx::gemm_generic_kernel<__nv_bfloat16, __nv_bfloat16><<<grid, 256, 0, st>>>(
            g.M, g.N, g.K, sa_i, sa_k, sb_k, sb_j, alpha, static_cast<const __nv_bfloat16*>(A),
            static_cast<const __nv_bfloat16*>(B), static_cast<__nv_bfloat16*>(C), ba.beta, ba.batch, ba.stride_a,
            ba.stride_b, ba.stride_c, bc);
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
    tdx::BoundsCheck bc{0, 0, 0, 0, 0, ctx->status_ptr};
    if (debug_bounds_enabled()) {
        bc.on = 1;
        bc.a_elems = c.N * c.H * c.W * c.Cin;
        bc.b_elems = c.Cout * c.R * c.S * c.Cin;
        bc.c_elems = total;
        bc.r_elems = total;
    }
    if (c.dtype == TDX_F32)
        tdx::conv2d_generic_kernel<float, float><<<grid, 256, 0, st>>>(
            (int)c.N, (int)c.H, (int)c.W, (int)c.Cin, (int)c.Cout, (int)c.R, (int)c.S, c.pad, c.stride, (int)c.P,
            (int)c.Q, static_cast<const float*>(x), static_cast<const float*>(w), bias, relu, static_cast<float*>(y),
            static_cast<const float*>(residual), bc);
    else
        tdx::conv2d_generic_kernel<__nv_bfloat16, __nv_bfloat16><<<grid, 256, 0, st>>>(
            (int)c.N, (int)c.H, (int)c.W, (int)c.Cin, (int)c.Cout, (int)c.R, (int)c.S, c.pad, c.stride, (int)c.P,
            (int)c.Q, static_cast<const __nv_bfloat16*>(x), static_cast<const __nv_bfloat16*>(w), bias, relu,
            static_cast<__nv_bfloat16*>(y), static_cast<const __nv_bfloat16*>(residual), bc);
    TDX_CUDA(cudaGetLastError());
    g_launches.fetch_add(1);
    return TDX_OK;
}

}  // namespace
