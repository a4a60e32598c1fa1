// Persistent, warp-specialised tcgen05 contraction kernel (bf16 x bf16 -> fp32 in TMEM).
//
// One CTA owns a stream of BM x BN output tiles (BM = 128 or 256).  Roles:
//   warp 0 (one lane)  TMA producer: fills a ring of shared-memory stages, each holding a
//                      BM x 64 slice of op(A) and a 64 x BN slice of op(B), 128-byte swizzled.
//   warp 1 (one lane)  MMA issuer: per stage and per 128-row half four tcgen05.mma (K = 16
//                      each) into a TMEM accumulator slot; tcgen05.commit releases the stage /
//                      publishes the tile.
//   warps 2..         epilogue: tcgen05.ld the accumulator (one row per thread), apply alpha /
//                      bias / ReLU, convert, and either store 16 bytes at a time from registers
//                      (one warp per 32 rows) or stage 32 x 32 blocks in shared memory (64-byte
//                      swizzled) and let the copy engine write them (TMA store; 16 warps, four per
//                      TMEM lane quarter, so that TMEM-load and store latencies overlap).
// TMEM holds 2 or 4 accumulator slots of 128 x BN; when a tile leaves slots free, the epilogue
// of tile t overlaps the main loop of tile t+1.  A 256-row tile halves the operand bytes fetched
// from L2 per flop (the B slice is shared by both halves), which is what bounds the 128-row tile.
//
// Operand transposes are never materialised: a K-major operand is loaded as one box of
// (64 k) x (rows); an MN-major operand as boxes of (64 mn) x (64 k), and the MMA
// descriptors say which one it is.  For the convolution the A slice of K-step (r, s, c-chunk)
// is the input window shifted by (r - pad, s - pad); out-of-range coordinates are zero-filled
// by the copy engine, which is all the padding there is.
//
// Every wait is bounded: a wait that runs out records a code in the device status word,
// raises a CTA-wide abort flag and all roles leave their loops and free TMEM.
#pragma once
#include <cuda_bf16.h>

#include "ptx_sm100.cuh"

namespace tdx {

constexpr int kHalfM = 128;       // rows of one MMA / one accumulator slot = TMEM lanes
constexpr int kBK = 64;           // K per stage: 64 bf16 = one 128-byte swizzle row
constexpr int kUmmaK = 16;        // K of one tcgen05.mma for 16-bit inputs
constexpr int kMaxStages = 8;
constexpr int kMaxSlots = 8;
constexpr int kHalfABytes = kHalfM * kBK * 2;          // 16 KiB: one 128-row half of the A slice
constexpr long long kWaitLimitCycles = 4000000000LL;  // ~2 s at boost clock

enum : int { kTimeoutProducer = 1, kTimeoutMma = 2, kTimeoutEpilogue = 3 };

struct UmmaParams {
    int M, N;                 // logical output rows / columns
    int num_kb;               // K blocks of 64 in the whole reduction
    int tiles_m, tiles_n, panel;
    int split_k, kb_per_split;
    int k_stagger;            // CTAs start their K loop at different blocks (same products, rotated order)
    int bm, bn, stages, tmem_cols;   // bm = 128 or 256
    int slots;                        // accumulator slots of 128 x bn in TMEM (2 or 4)
    int a_mn_major, b_mn_major;
    float alpha;
    float beta;               // GEMM with accumulate: out = alpha * acc + beta * (what C held); direct stores only
    const float* bias;        // [N] or nullptr
    const __nv_bfloat16* residual;   // convolution: [M][N] added after the bias and before the ReLU, or nullptr
    int relu;
    __nv_bfloat16* C;         // bf16 output, row pitch ldc elements
    long long ldc;
    float* partial;           // split-K: [split][M][N] fp32
    int vec_store;            // rows of C / partial are 16-byte aligned and N % 8 == 0
    int tma_store;            // final output leaves through shared memory + TMA store (needs bn % 64 == 0)
    int partial_tma;          // split-K: fp32 partial tiles leave through shared memory + TMA store (tmC then maps the
                              // workspace as (N, M, batch * split) floats; two 32 x 32 fp32 blocks per epilogue warp)
    int cluster_reduce;       // split-K summed inside a thread-block cluster of split_k CTAs (GEMM, one
                              // tile per CTA): CTA rank s of a cluster reduces K slice s of the cluster's tile, then
                              // the ranks exchange column slices of their partial tiles through distributed shared
                              // memory and rank q writes columns [q, q + 1) * bn / split_k of the result -- no
                              // workspace and no reduction kernel.  The sum runs over the slices in ascending order.
    int cluster_tma;          // cluster reduction: the summed slice leaves as 32 x 32 blocks through shared memory and the
                              // copy engine (1: bf16, 2: fp32; tmC maps C as (N, M) or (N, M, batch)); 0: stores from registers
    int sbx, sby;             // conv TMA-store box: sbx x sby output pixels (sbx * sby = 32)
    // convolution geometry (kConv only)
    int bw, bh, nb;           // spatial patch (bw x bh output pixels), patches per tile = bm / (bw*bh)
    int patches_w, patches_h; // patches per image along Q and P
    int P, Q, Nimg, S, pad, cchunks;
    int stride;               // convolution stride (per-tap loads; the tensor map carries the same traversal stride)
    // halo-reuse convolution (umma_conv_halo_kernel): the input window of an 8 x 16 pixel patch is loaded once
    // per channel chunk and shared by all filter taps
    int R;                    // filter rows (taps = R * S)
    int hpitch, hrows;        // halo tile: (8 + S - 1) pixels wide, (16 + R - 1) pixels high
    int halo_bytes;           // hpitch * hrows * 128 rounded up to 1024
    int a_stages;             // halo tiles in flight per 128-row half
    int b_resident;           // the whole filter (all chunks and taps, one column tile) stays in shared memory:
                              // loaded once per CTA instead of once per tile, no per-tap handshake
    int epi_warps;            // epilogue warps (0: every warp from the third on)
    // Tile table (GEMM, optional): instead of a uniform grid of bm x bn tiles, the output is cut into tiles of
    // bm rows and individually chosen widths (multiples of b_box, at most bn), and the host has already dealt
    // them to the CTAs (CTA pairs for the pair kernel): entry [round * workers + worker] = (row block, first
    // column, width, w); width 0 ends a worker's list.  This is how a tile count that does not fill the last
    // wave of CTAs is evened out.  w = 0: the whole reduction of the tile; otherwise (K-balanced plan, few tiles and
    // a long reduction) K blocks [w & 0xFFF, (w >> 12) & 0xFFF) of it, whose fp32 partial tile goes to slot
    // (w >> 24) & 0x7F of the split-K workspace: the (tile, K block) units are dealt evenly to ALL CTAs, a tile cut
    // by a CTA boundary is completed by the reduction kernel in ascending slot order.
    // fp32 GEMM from bf16 pieces (seg_kb > 0): the operands hold three pieces side by side (seg_kb K blocks each) and the
    // reduction walks six piece pairs: K block kb reads piece a_seg[kb / seg_kb] of A and b_seg[kb / seg_kb] of B.
    // The result is written as fp32 to Cf (direct stores).
    int seg_kb;
    int a_seg[6], b_seg[6];
    float* Cf;
    // batched (pieces path only, batch > 1): the operands are 3-D tensors (K, rows, batch), the items run over
    // batch x tiles x splits, C of batch b starts batch_c elements after that of b - 1, and the split-K partials
    // are laid out [batch][split][M][N]
    int batch;
    long long batch_c;
    int a_shared, b_shared;   // batched: the operand is one matrix shared by all batches (its tensor has one batch)
    const int4* tiles;
    int rounds;
    int b_box;                // rows of one B copy (K-major B); bn when there is no table
    int Pv, H;                // stacked images (Pv > 0): the images of the batch form one column of Nimg * Pv rows,
                              // image n owning rows [n * Pv, n * Pv + P) and the Pv - P rows below it reading as
                              // zero (they are the bottom padding of image n and the top padding of image n + 1);
                              // 16-row patches are cut from that column, so they may straddle two images
    int* status;              // device status word
};

__device__ __forceinline__ bool wait_bounded_for(uint64_t* bar, uint32_t parity, volatile int* s_abort, int* g_status,
                                                 int code, long long limit_cycles) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    uint32_t spins = 0;
    for (;;) {
        if (ptx::mbar_try_wait(bar, parity)) return true;
        if ((++spins & 63u) == 0u) {
            if (*s_abort) return false;
            if (clock64() - t0 > limit_cycles) {
                *s_abort = 1;
                atomicCAS(g_status, 0, code);
                return false;
            }
        }
    }
}
__device__ __forceinline__ bool wait_bounded(uint64_t* bar, uint32_t parity, volatile int* s_abort, int* g_status,
                                             int code) {
    return wait_bounded_for(bar, parity, s_abort, g_status, code, kWaitLimitCycles);
}

// Self-test of the bounded wait: one warp waits on a barrier that nothing ever signals, with a short limit; the wait
// must give up, record `kTimeoutSelfTest` in the status word and let the kernel return normally.
enum : int { kTimeoutSelfTest = 9 };
__global__ void bounded_wait_selftest_kernel(int* status, long long limit_cycles) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int s_abort;
    if (threadIdx.x == 0) {
        ptx::mbar_init(&bar, 1);
        s_abort = 0;
        ptx::fence_barrier_init();
    }
    __syncthreads();
    wait_bounded_for(&bar, 0, &s_abort, status, kTimeoutSelfTest, limit_cycles);
}

struct TileCoord {
    int m_blk, n_blk, kb0, kb1, split;
    int batch;                // batch index (0 unless the launch is batched)
    int n0, bn;               // first output column and width of the tile
};

__device__ __forceinline__ TileCoord decode_item(const UmmaParams& p, int item) {
    TileCoord t;
    t.batch = 0;
    if (p.batch > 1) {
        const int per_batch = p.tiles_m * p.tiles_n * p.split_k;
        t.batch = item / per_batch;
        item -= t.batch * per_batch;
    }
    const int tile = item / p.split_k;
    t.split = item - tile * p.split_k;
    const int per_panel = p.panel * p.tiles_n;
    const int pidx = tile / per_panel;
    const int rem = tile - pidx * per_panel;
    const int m_first = pidx * p.panel;
    const int w = min(p.panel, p.tiles_m - m_first);
    t.n_blk = rem / w;
    t.m_blk = m_first + (rem - t.n_blk * w);
    t.kb0 = t.split * p.kb_per_split;
    t.kb1 = min(p.num_kb, t.kb0 + p.kb_per_split);
    t.n0 = t.n_blk * p.bn;
    t.bn = p.bn;
    return t;
}

// K block a CTA starts a tile's reduction with (k_stagger: CTAs start at different blocks; same terms, rotated order)
__device__ __forceinline__ int first_kblock(const UmmaParams& p, const TileCoord& t) {
    const int nkb = t.kb1 - t.kb0;
    return t.kb0 + (p.k_stagger ? static_cast<int>((static_cast<long long>(blockIdx.x) * nkb) / gridDim.x) : 0);
}

// The `local`-th tile of worker `first_item` of `item_stride` workers (CTAs, or CTA pairs): from the tile table when
// there is one, else item first_item + local * item_stride of the uniform grid.  Returns false when there is none.
__device__ __forceinline__ bool get_tile(const UmmaParams& p, int local, int first_item, int item_stride, int total_items,
                                         TileCoord* t) {
    if (p.tiles != nullptr) {
        if (local >= p.rounds) return false;
        const int4 e = __ldg(p.tiles + static_cast<size_t>(local) * item_stride + first_item);
        if (e.z == 0) return false;
        t->batch = 0;
        t->m_blk = e.x;
        t->n_blk = 0;
        t->n0 = e.y;
        t->bn = e.z;
        t->kb0 = 0;
        t->kb1 = p.num_kb;
        t->split = 0;
        if (e.w != 0) {          // K-balanced plan: this entry is K blocks [kb0, kb1) of the tile, partial sums to slot `split`
            t->kb0 = e.w & 0xFFF;
            t->kb1 = (e.w >> 12) & 0xFFF;
            t->split = (e.w >> 24) & 0x7F;
        }
        return true;
    }
    const int item = first_item + local * item_stride;
    if (item >= total_items) return false;
    *t = decode_item(p, item);
    return true;
}

// The copies of K block `kb` of tile `t` into one pipeline stage: op(A) rows and op(B) columns of that block.
template <bool kConv>
__device__ __forceinline__ void issue_kblock(const UmmaParams& p, const CUtensorMap* tmA, const CUtensorMap* tmB,
                                             const TileCoord& t, int kb, int mh, uint8_t* a_dst, uint8_t* b_dst, uint64_t* bar) {
    auto ld2 = [&](uint8_t* dst, const CUtensorMap* m, int c0, int c1) { ptx::tma_load_2d(dst, m, bar, c0, c1); };
    auto ld3 = [&](uint8_t* dst, const CUtensorMap* m, int c0, int c1, int c2) { ptx::tma_load_3d(dst, m, bar, c0, c1, c2); };
    auto ld4 = [&](uint8_t* dst, const CUtensorMap* m, int c0, int c1, int c2, int c3) {
        ptx::tma_load_4d(dst, m, bar, c0, c1, c2, c3);
    };
    if (kConv) {
        const int tap = kb / p.cchunks;
        const int cc = kb - tap * p.cchunks;
        const int r = tap / p.S;
        const int s = tap - r * p.S;
        const int ppi = p.patches_w * p.patches_h;
        const uint32_t patch_bytes = static_cast<uint32_t>(p.bw * p.bh) * 128u;
        for (int i = 0; i < p.nb; ++i) {
            const int patch = t.m_blk * p.nb + i;
            const int n = patch / ppi;
            const int rem = patch - n * ppi;
            const int ph = rem / p.patches_w;
            const int pw = rem - ph * p.patches_w;
            ld4(a_dst + i * patch_bytes, tmA, cc * kBK, pw * p.bw * p.stride + s - p.pad, ph * p.bh * p.stride + r - p.pad, n);
        }
        // (tiles from a fitted table arrive in 64-row copies, like the GEMM's)
        for (int r0 = 0; r0 < t.bn; r0 += p.b_box) ld3(b_dst + r0 * 128, tmB, cc * kBK, tap, t.n0 + r0);
        return;
    }
    int ka = kb, kbb = kb;                  // K block of A and of B
    if (p.seg_kb > 0) {
        const int sg = kb / p.seg_kb, r = kb - sg * p.seg_kb;
        ka = p.a_seg[sg] * p.seg_kb + r;
        kbb = p.b_seg[sg] * p.seg_kb + r;
    }
    if (p.batch > 1) {
        // batched: 3-D operands (contiguous dimension, the other one, batch); rows past M or N of a batch are
        // zero-filled, never the next batch's
        const int ba = p.a_shared ? 0 : t.batch, bb = p.b_shared ? 0 : t.batch;
        if (p.a_mn_major) {
            for (int i = 0; i < 2 * mh; ++i) ld3(a_dst + i * 8192, tmA, t.m_blk * p.bm + i * 64, ka * kBK, ba);
        } else {
            for (int h = 0; h < mh; ++h) ld3(a_dst + h * kHalfABytes, tmA, ka * kBK, t.m_blk * p.bm + h * kHalfM, ba);
        }
        if (p.b_mn_major) {
            for (int i = 0; i < t.bn / 64; ++i) ld3(b_dst + i * 8192, tmB, t.n0 + i * 64, kbb * kBK, bb);
        } else {
            for (int r0 = 0; r0 < t.bn; r0 += p.b_box) ld3(b_dst + r0 * 128, tmB, kbb * kBK, t.n0 + r0, bb);
        }
        return;
    }
    if (p.a_mn_major) {
        for (int i = 0; i < 2 * mh; ++i) ld2(a_dst + i * 8192, tmA, t.m_blk * p.bm + i * 64, ka * kBK);
    } else {
        for (int h = 0; h < mh; ++h) ld2(a_dst + h * kHalfABytes, tmA, ka * kBK, t.m_blk * p.bm + h * kHalfM);
    }
    if (p.b_mn_major) {
        for (int i = 0; i < t.bn / 64; ++i) ld2(b_dst + i * 8192, tmB, t.n0 + i * 64, kbb * kBK);
    } else {
        for (int r0 = 0; r0 < t.bn; r0 += p.b_box) ld2(b_dst + r0 * 128, tmB, kbb * kBK, t.n0 + r0);
    }
}

// Slot layout of the cluster reduction: a slot holds one rank's bm x slice partial sums for the rank that owns the
// slice, as [32-row group][4-column group][row within the group][16 bytes] (`quarter` = 4 * half + lane quarter): the
// 32 rows of a warp lie side by side (no bank conflicts on either end) and a warp's 32-column step is one contiguous 4 KB.
__device__ __forceinline__ uint32_t cluster_slot_offset(int quarter, int slice, int c_in_slice, int lane) {
    return (static_cast<uint32_t>(quarter * (slice >> 2) + (c_in_slice >> 2)) * 32u + static_cast<uint32_t>(lane)) * 16u;
}

// Epilogue role (all warps from the third on).  With the staged epilogue there are 16 of them (4 per TMEM
// lane quarter) and the warps of a quarter take the 32-column steps round robin; the direct epilogue has one
// warp per quarter and 128-row half.
template <bool kConv>
__device__ __forceinline__ void epilogue_role(const UmmaParams& p, const CUtensorMap* tmC, uint8_t* staging_base,
                                              uint32_t tmem_base, uint64_t* tfull_bar, uint64_t* tempty_bar,
                                              volatile int* abort_flag, int mh, int warp, int lane, int total_items,
                                              int first_item = -1, int item_stride = 0, int m_mul = 1, int m_add = 0,
                                              uint32_t tempty_cluster_addr = 0, const CUtensorMap* tmC_row = nullptr,
                                              const TileCoord* t_first = nullptr, bool have_first = false,
                                              const uint8_t* recv = nullptr, int my_rank = 0) {
    // recv != nullptr (cluster reduction): `t_first` is this rank's column slice of the cluster's tile, its accumulator
    // columns start my_rank * t.bn into the slot, and the other ranks' partial sums of the slice lie in `recv`
    const bool reduce_here = recv != nullptr;
    const int tmem_col_off = reduce_here ? my_rank * t_first->bn : 0;
    // CTA pairs: the pair walks tiles of 256 rows, this CTA owns rows [128 * (2 m + rank), +128) of tile m, and the
    // accumulator-free signal goes to the leader CTA's barrier (tempty_cluster_addr, a shared::cluster address)
    if (first_item < 0) {
        first_item = blockIdx.x;
        item_stride = gridDim.x;
    }
    const int ew = warp - 2;
    const int nwarps_epi = p.epi_warps > 0 ? p.epi_warps : (static_cast<int>(blockDim.x) >> 5) - 2;
    const int ncgrp = nwarps_epi / (4 * mh);      // warps sharing one (half, quarter)
    const int half = (ew >> 2) % mh;              // which 128-row half of the tile this warp drains
    const int cgrp = (ew >> 2) / mh;              // which share of the columns
    const int quarter = warp & 3;                 // TMEM lane quarter this warp may read
    const int row_in_tile = half * kHalfM + quarter * 32 + lane;
    // the caller may have worked out the first tile already (before the grid-dependency wait)
    TileCoord t;
    bool have = have_first;
    if (t_first != nullptr) t = *t_first; else have = get_tile(p, 0, first_item, item_stride, total_items, &t);
    for (int local = 0; have; have = get_tile(p, ++local, first_item, item_stride, total_items, &t)) {
        t.m_blk = t.m_blk * m_mul + m_add;
        const int sidx = local * mh + half;
        const int buf = sidx % p.slots;
        const uint32_t aphase = (sidx / p.slots) & 1;
        // Staged epilogue: lane l fetches the bias of column (step's first column + l) for each of this warp's (at most
        // four) 32-column steps NOW, so that the loads complete while the warp waits for the accumulators -- fetched
        // inside the step, their L2 latency was paid four times per tile (conv 56x56x256: epilogue 3.8 us vs 2.5 for
        // the same tile without bias).  Columns past N are clipped by the store; the index only has to stay in range.
        float bias_pre0 = 0.0f, bias_pre1 = 0.0f, bias_pre2 = 0.0f, bias_pre3 = 0.0f;
        if (p.bias != nullptr && p.tma_store && p.split_k == 1) {
            const int c_first = t.n0 + cgrp * 32 + lane, c_step = ncgrp * 32, last = p.N - 1;
            bias_pre0 = __ldg(p.bias + min(c_first, last));
            bias_pre1 = __ldg(p.bias + min(c_first + c_step, last));
            bias_pre2 = __ldg(p.bias + min(c_first + 2 * c_step, last));
            bias_pre3 = __ldg(p.bias + min(c_first + 3 * c_step, last));
        }
        if (!wait_bounded(&tfull_bar[buf], aphase, abort_flag, p.status, kTimeoutEpilogue)) break;
        ptx::tc_fence_after_sync();

        long long grow;
        bool valid;
        if (kConv) {
            const int per_patch = p.bw * p.bh;
            const int pl = row_in_tile / per_patch;
            const int within = row_in_tile - pl * per_patch;
            const int hl = within / p.bw;
            const int wl = within - hl * p.bw;
            const int patch = t.m_blk * p.nb + pl;
            int n, pp, qq;
            if (p.Pv > 0) {
                const int ph = patch / p.patches_w;
                const int v = ph * p.bh + hl;            // row in the column of stacked images
                n = v / p.Pv;
                pp = v - n * p.Pv;
                qq = (patch - ph * p.patches_w) * p.bw + wl;
            } else {
                const int ppi = p.patches_w * p.patches_h;
                n = patch / ppi;
                const int rem = patch - n * ppi;
                const int ph = rem / p.patches_w;
                const int pw = rem - ph * p.patches_w;
                pp = ph * p.bh + hl;
                qq = pw * p.bw + wl;
            }
            valid = (n < p.Nimg) && (pp < p.P) && (qq < p.Q);
            grow = (static_cast<long long>(n) * p.P + pp) * p.Q + qq;
        } else {
            grow = static_cast<long long>(t.m_blk) * p.bm + row_in_tile;
            valid = grow < p.M;
        }

        if (p.tma_store && p.split_k == 1) {
            // ---- staged path: 32 rows x 32 columns per warp and step, written by the copy engine
            uint8_t* stage_buf = staging_base + (warp - 2) * 2048;
            const int wrow0 = half * kHalfM + quarter * 32;      // first tile row of this warp
            int sc1 = 0, sc2 = 0, sc3 = 0;                       // store coordinates above the column
            bool box_ok;
            // stacked images: the warp's four pixel rows (8 pixels x 32 channels = 512 bytes of the staging block
            // each) leave as one box when they lie in one image; where they cross the seam between two images,
            // lanes 0..3 store one pixel row each
            int nstore = 1;
            const CUtensorMap* store_map = tmC;
            if (kConv && p.Pv > 0) {
                const int pl = wrow0 / kHalfM;
                const int hl0 = (wrow0 - pl * kHalfM) / p.bw;
                const int patch = t.m_blk * p.nb + pl;
                const int ph = patch / p.patches_w;
                const int v0 = ph * p.bh + hl0;
                const int n0 = v0 / p.Pv;
                sc1 = (patch - ph * p.patches_w) * p.bw;
                if (v0 - n0 * p.Pv + 3 < p.P) {
                    sc3 = n0;
                    sc2 = v0 - n0 * p.Pv;
                    box_ok = n0 < p.Nimg;
                } else {
                    const int v = v0 + (lane & 3);
                    sc3 = v / p.Pv;
                    sc2 = v - sc3 * p.Pv;
                    box_ok = (sc3 < p.Nimg) && (sc2 < p.P);
                    nstore = 4;
                    store_map = tmC_row;
                }
            } else if (kConv) {
                const int per_patch = p.bw * p.bh;
                const int pl = wrow0 / per_patch;
                const int within = wrow0 - pl * per_patch;
                const int hl0 = within / p.bw;
                const int wl0 = within - hl0 * p.bw;
                const int patch = t.m_blk * p.nb + pl;
                const int ppi = p.patches_w * p.patches_h;
                const int n = patch / ppi;
                const int rem = patch - n * ppi;
                const int ph = rem / p.patches_w;
                const int pw = rem - ph * p.patches_w;
                sc1 = pw * p.bw + wl0;
                sc2 = ph * p.bh + hl0;
                sc3 = n;
                box_ok = (n < p.Nimg) && (sc2 < p.P) && (sc1 < p.Q);
            } else {
                sc1 = t.m_blk * p.bm + wrow0;
                box_ok = sc1 < p.M;
            }
            // 64-byte swizzle of the staging block: 16-byte slot c of row `lane` lives at slot c ^ ((lane / 2) % 4)
            uint8_t* my_row = stage_buf + lane * 64;
            const int sw = (lane >> 1) & 3;
            const bool plain = (p.bias == nullptr) && (p.relu == 0) && (p.residual == nullptr);
            // Per 32-column step: the accumulators are converted into registers first; then the NEXT step's accumulators
            // are requested from tensor memory, so that their latency passes while this step waits for its staging
            // block (the copy engine may still be reading the previous store), writes it, and hands it to the copy engine.
            int step = 0;
            uint32_t r[32];
            const uint32_t trow = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + static_cast<uint32_t>(buf * p.bn);
            if (cgrp * 32 < t.bn) ptx::tmem_ld_32x32b_x32(trow + static_cast<uint32_t>(cgrp * 32), r);
            for (int c0 = cgrp * 32; c0 < t.bn; c0 += ncgrp * 32, ++step) {
                const int col0 = t.n0 + c0;
                // the bias of column col0 + lane: prefetched above for the first four steps of a warp (all there are
                // with 16 epilogue warps and tiles of up to 256 columns)
                float bias_l = step == 0 ? bias_pre0 : step == 1 ? bias_pre1 : step == 2 ? bias_pre2 : bias_pre3;
                if (step > 3 && p.bias != nullptr) bias_l = __ldg(p.bias + min(col0 + lane, p.N - 1));
                ptx::tmem_ld_wait();
                if (kConv && p.residual != nullptr) {
                    // residual term (convolution only, where alpha is 1): this thread's 32 values of its output row
                    // (64 bytes; the staged epilogue implies N % 8 == 0) join the accumulators before bias and ReLU
                    if (valid) {
                        const uint4* rp = reinterpret_cast<const uint4*>(p.residual + grow * p.ldc + col0);
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
                            if (col0 + g * 8 < p.N) {
                                const uint4 v = __ldg(rp + g);
                                const uint32_t rw[4] = {v.x, v.y, v.z, v.w};      // two bf16 values each
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const int j = g * 8 + e * 2;
                                    r[j] = __float_as_uint(__uint_as_float(r[j]) + __uint_as_float(rw[e] << 16));
                                    r[j + 1] = __float_as_uint(__uint_as_float(r[j + 1]) + __uint_as_float(rw[e] & 0xFFFF0000u));
                                }
                            }
                        }
                    }
                }
                uint32_t pk[16];                                   // the step's 32 outputs as bf16 pairs
                if (plain) {
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        __nv_bfloat162 h2 = __floats2bfloat162_rn(p.alpha * __uint_as_float(r[2 * e]), p.alpha * __uint_as_float(r[2 * e + 1]));
                        pk[e] = *reinterpret_cast<uint32_t*>(&h2);
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        const int j = 2 * e;
                        float x0 = p.alpha * __uint_as_float(r[j]) + __shfl_sync(0xffffffffu, bias_l, j);
                        float x1 = p.alpha * __uint_as_float(r[j + 1]) + __shfl_sync(0xffffffffu, bias_l, j + 1);
                        if (p.relu) {
                            x0 = fmaxf(x0, 0.0f);
                            x1 = fmaxf(x1, 0.0f);
                        }
                        __nv_bfloat162 h2 = __floats2bfloat162_rn(x0, x1);
                        pk[e] = *reinterpret_cast<uint32_t*>(&h2);
                    }
                }
                // r is free again: request the next step's accumulators now
                if (c0 + ncgrp * 32 < t.bn) ptx::tmem_ld_32x32b_x32(trow + static_cast<uint32_t>(c0 + ncgrp * 32), r);
                // the previous store of this warp must have finished reading the staging block
                if (lane < nstore) ptx::tma_store_wait_read<0>();
                __syncwarp();
#pragma unroll
                for (int g = 0; g < 4; ++g)
                    *reinterpret_cast<uint4*>(my_row + ((g ^ sw) << 4)) = make_uint4(pk[4 * g], pk[4 * g + 1], pk[4 * g + 2], pk[4 * g + 3]);
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane < nstore && box_ok && col0 < p.N) {
                    if (kConv)
                        ptx::tma_store_4d(store_map, stage_buf + lane * 512, col0, sc1, sc2, sc3);
                    else
                        ptx::tma_store_2d(tmC, stage_buf, col0, sc1);
                    ptx::tma_store_commit();
                }
                __syncwarp();
            }
        } else
        for (int c0 = 0; c0 < t.bn; c0 += 32) {
            uint32_t r[32];
            const uint32_t taddr =
                tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + static_cast<uint32_t>(buf * p.bn + tmem_col_off + c0);
            ptx::tmem_ld_32x32b_x32(taddr, r);
            ptx::tmem_ld_wait();
            const int col0 = t.n0 + c0;
            if (reduce_here) {
                // slices in ascending order, this rank's own (from tensor memory) in its place: the result does not
                // depend on which rank writes it
                float sum[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) sum[j] = 0.0f;
                const uint32_t slot_bytes = static_cast<uint32_t>(p.bm) * static_cast<uint32_t>(t.bn) * 4u;
                const uint32_t in_slot = cluster_slot_offset(half * 4 + quarter, t.bn, c0, lane);
                for (int s = 0; s < p.split_k; ++s) {
                    if (s == my_rank) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) sum[j] += __uint_as_float(r[j]);
                    } else {
                        const uint8_t* src = recv + static_cast<uint32_t>(s < my_rank ? s : s - 1) * slot_bytes + in_slot;
#pragma unroll
                        for (int g = 0; g < 8; ++g) {
                            const float4 v = *reinterpret_cast<const float4*>(src + g * 512);
                            sum[4 * g] += v.x; sum[4 * g + 1] += v.y; sum[4 * g + 2] += v.z; sum[4 * g + 3] += v.w;
                        }
                    }
                }
#pragma unroll
                for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(sum[j]);
            }
            if (p.split_k > 1 && p.partial_tma && !reduce_here) {
                // fp32 partial tile through shared memory: the thread writes its row's 32 values (128 bytes, 16-byte
                // chunk c at chunk c ^ (row % 8): the 128-byte swizzle of the copy engine) and the copy engine stores
                // the 32 x 32 block as whole 128-byte lines, clipped at the matrix edge; stores straight from registers
                // reach the same lines in 16-byte pieces, eight instructions per line.  Two blocks per warp take turns, so
                // a block is rewritten only after the store issued two steps earlier has read it.
                const int estep = c0 >> 5;
                uint8_t* blk = staging_base + ((warp - 2) * 2 + (estep & 1)) * 4096;
                if (lane == 0) ptx::tma_store_wait_read<1>();
                __syncwarp();
                uint8_t* my_row = blk + lane * 128;
#pragma unroll
                for (int g = 0; g < 8; ++g)
                    *reinterpret_cast<uint4*>(my_row + ((g ^ (lane & 7)) << 4)) = make_uint4(r[g * 4], r[g * 4 + 1], r[g * 4 + 2], r[g * 4 + 3]);
                ptx::fence_proxy_async_smem();
                __syncwarp();
                const int row0 = t.m_blk * p.bm + half * kHalfM + quarter * 32;
                if (lane == 0 && row0 < p.M && col0 < p.N) {
                    ptx::tma_store_3d(tmC, blk, col0, row0, t.batch * p.split_k + t.split);
                    ptx::tma_store_commit();
                }
                __syncwarp();
                continue;
            }
            if (valid && col0 < p.N) {
            if (p.split_k > 1 && !reduce_here) {
                float* dst = p.partial + ((static_cast<long long>(t.batch) * p.split_k + t.split) * p.M + grow) * p.N + col0;
                if (p.vec_store) {
#pragma unroll
                    for (int g = 0; g < 8; ++g) {
                        if (col0 + g * 4 < p.N) {
                            float4 v = make_float4(__uint_as_float(r[g * 4]), __uint_as_float(r[g * 4 + 1]),
                                                   __uint_as_float(r[g * 4 + 2]), __uint_as_float(r[g * 4 + 3]));
                            *reinterpret_cast<float4*>(dst + g * 4) = v;
                        }
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (col0 + j < p.N) dst[j] = __uint_as_float(r[j]);
                }
            } else if (!kConv && p.Cf != nullptr) {
                // fp32 output (the fp32 GEMM from bf16 pieces): out = alpha * acc + beta * (what Cf held)
                float* dst = p.Cf + t.batch * p.batch_c + grow * p.ldc + col0;
                if (p.vec_store) {
#pragma unroll
                    for (int g = 0; g < 8; ++g) {
                        if (col0 + g * 4 < p.N) {
                            float4 v = make_float4(p.alpha * __uint_as_float(r[g * 4]), p.alpha * __uint_as_float(r[g * 4 + 1]),
                                                   p.alpha * __uint_as_float(r[g * 4 + 2]), p.alpha * __uint_as_float(r[g * 4 + 3]));
                            if (p.beta != 0.0f) {
                                const float4 o = *reinterpret_cast<const float4*>(dst + g * 4);
                                v.x = fmaf(p.beta, o.x, v.x); v.y = fmaf(p.beta, o.y, v.y);
                                v.z = fmaf(p.beta, o.z, v.z); v.w = fmaf(p.beta, o.w, v.w);
                            }
                            *reinterpret_cast<float4*>(dst + g * 4) = v;
                        }
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (col0 + j < p.N) {
                            const float x = p.alpha * __uint_as_float(r[j]);
                            dst[j] = p.beta != 0.0f ? fmaf(p.beta, dst[j], x) : x;
                        }
                }
            } else {
                float v[32];
                __nv_bfloat16* const c_row = p.C + t.batch * p.batch_c + grow * p.ldc + col0;
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    float x = p.alpha * __uint_as_float(r[j]);
                    if (p.beta != 0.0f && col0 + j < p.N) x = fmaf(p.beta, __bfloat162float(c_row[j]), x);
                    if (p.bias != nullptr && col0 + j < p.N) x += __ldg(p.bias + col0 + j);
                    if (p.residual != nullptr && col0 + j < p.N) x += __bfloat162float(p.residual[grow * p.ldc + col0 + j]);
                    if (p.relu) x = fmaxf(x, 0.0f);
                    v[j] = x;
                }
                __nv_bfloat16* dst = c_row;
                if (p.vec_store) {
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        if (col0 + g * 8 < p.N) {
                            uint4 pk;
                            __nv_bfloat162 h0 = __floats2bfloat162_rn(v[g * 8 + 0], v[g * 8 + 1]);
                            __nv_bfloat162 h1 = __floats2bfloat162_rn(v[g * 8 + 2], v[g * 8 + 3]);
                            __nv_bfloat162 h2 = __floats2bfloat162_rn(v[g * 8 + 4], v[g * 8 + 5]);
                            __nv_bfloat162 h3 = __floats2bfloat162_rn(v[g * 8 + 6], v[g * 8 + 7]);
                            pk.x = *reinterpret_cast<uint32_t*>(&h0);
                            pk.y = *reinterpret_cast<uint32_t*>(&h1);
                            pk.z = *reinterpret_cast<uint32_t*>(&h2);
                            pk.w = *reinterpret_cast<uint32_t*>(&h3);
                            *reinterpret_cast<uint4*>(dst + g * 8) = pk;
                        }
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (col0 + j < p.N) dst[j] = __float2bfloat16_rn(v[j]);
                }
            }
            }
            __syncwarp();   // reconverge before the next warp-aligned TMEM load
        }
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) {
            if (tempty_cluster_addr != 0)
                ptx::mbar_arrive_cluster(tempty_cluster_addr + static_cast<uint32_t>(buf) * 8u);
            else
                ptx::mbar_arrive(&tempty_bar[buf]);
        }
    }
    // shared memory must stay alive until the copy engine has drained this warp's last store
    if ((p.tma_store || p.partial_tma) && lane < 4) ptx::tma_store_wait_all<0>();
}

// Cluster reduction, first half: every epilogue warp sends its 32 rows of the column slices that other ranks own into
// those ranks' receive slots (slot of this rank) with 16-byte stores through distributed shared memory.  (Staging the
// slices in this CTA's shared memory and sending 4 KB pieces with the copy engine, counted on the receiver's barrier,
// was built and measured too: 29.8 against 28.9 us on the 128 x 8192 x 8192 GEMM, so the stores stayed.)
__device__ __forceinline__ void cluster_push_partials(const UmmaParams& p, uint8_t* recv_base, uint32_t tmem_base, int warp,
                                                      int lane, int me) {
    const int quarter = warp & 3;
    const int half = (warp - 2) >> 2;                  // 256-row tiles: warps 6..9 drain the second accumulator slot
    const int slice = p.bn / p.split_k;
    const uint32_t slot_bytes = static_cast<uint32_t>(p.bm) * static_cast<uint32_t>(slice) * 4u;
    for (int c0 = 0; c0 < p.bn; c0 += 32) {
        const int owner = c0 / slice;
        if (owner == me) continue;
        uint32_t r[32];
        ptx::tmem_ld_32x32b_x32(tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + static_cast<uint32_t>(half * p.bn + c0), r);
        ptx::tmem_ld_wait();
        const uint32_t in_slot = cluster_slot_offset(half * 4 + quarter, slice, c0 - owner * slice, lane);
        const uint32_t there = ptx::smem_u32(recv_base) + static_cast<uint32_t>(me < owner ? me : me - 1) * slot_bytes + in_slot;
        const uint32_t remote = ptx::mapa_u32(there, static_cast<uint32_t>(owner));
#pragma unroll
        for (int g = 0; g < 8; ++g)
            ptx::st_cluster_v4(remote + g * 512, r[4 * g], r[4 * g + 1], r[4 * g + 2], r[4 * g + 3]);
    }
}

// Cluster reduction, second half: each epilogue warp sums its 32 rows of this rank's column slice over the K slices in
// ascending order -- its own from tensor memory, the others' from the receive slots --, applies alpha and the accumulate
// term (beta times what C held, read straight from global memory: a thread's 32 columns are one or two whole lines) and
// hands 32 x 32 blocks to the copy engine: bf16 with the 64-byte swizzle of the staged epilogue, two 2 KB blocks per warp
// taking turns (p.cluster_tma == 1), or fp32 with the 128-byte swizzle, one 4 KB block per warp (== 2).  tmC maps C as
// (N, M) or, batched, (N, M, batch).  Stores straight from registers reach the same lines 16 bytes at a time and cost
// about ten times more.
__device__ __forceinline__ void cluster_reduce_store(const UmmaParams& p, const CUtensorMap* tmC, const uint8_t* recv,
                                                     uint8_t* staging, uint32_t tmem_base, const TileCoord& t, int warp,
                                                     int lane, int me) {
    const int quarter = warp & 3;
    const int half = (warp - 2) >> 2;
    const int slice = p.bn / p.split_k;
    const uint32_t slot_bytes = static_cast<uint32_t>(p.bm) * static_cast<uint32_t>(slice) * 4u;
    const int row0 = t.m_blk * p.bm + half * kHalfM + quarter * 32;
    const long long grow = static_cast<long long>(row0) + lane;
    const bool f32 = p.cluster_tma == 2;
    uint8_t* blocks = staging + (warp - 2) * 4096;
    int step = 0;
    for (int c0 = 0; c0 < slice; c0 += 32, ++step) {
        uint32_t r[32];
        ptx::tmem_ld_32x32b_x32(tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + static_cast<uint32_t>(half * p.bn + me * slice + c0), r);
        ptx::tmem_ld_wait();
        float sum[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) sum[j] = 0.0f;
        const uint32_t in_slot = cluster_slot_offset(half * 4 + quarter, slice, c0, lane);
        for (int s = 0; s < p.split_k; ++s) {
            if (s == me) {
#pragma unroll
                for (int j = 0; j < 32; ++j) sum[j] += __uint_as_float(r[j]);
            } else {
                const uint8_t* src = recv + static_cast<uint32_t>(s < me ? s : s - 1) * slot_bytes + in_slot;
#pragma unroll
                for (int g = 0; g < 8; ++g) {
                    const float4 v = *reinterpret_cast<const float4*>(src + g * 512);
                    sum[4 * g] += v.x; sum[4 * g + 1] += v.y; sum[4 * g + 2] += v.z; sum[4 * g + 3] += v.w;
                }
            }
        }
        const int col0 = t.n0 + me * slice + c0;
#pragma unroll
        for (int j = 0; j < 32; ++j) sum[j] *= p.alpha;
        if (p.beta != 0.0f && grow < p.M) {
            // (rows are 16-byte aligned and N is a multiple of 8 (bf16) or 4 (fp32) here, so groups are all in or all out)
            if (f32) {
                const float* old = p.Cf + t.batch * p.batch_c + grow * p.ldc + col0;
#pragma unroll
                for (int g = 0; g < 8; ++g) {
                    if (col0 + g * 4 < p.N) {
                        const float4 o = *reinterpret_cast<const float4*>(old + g * 4);
                        sum[4 * g] = fmaf(p.beta, o.x, sum[4 * g]); sum[4 * g + 1] = fmaf(p.beta, o.y, sum[4 * g + 1]);
                        sum[4 * g + 2] = fmaf(p.beta, o.z, sum[4 * g + 2]); sum[4 * g + 3] = fmaf(p.beta, o.w, sum[4 * g + 3]);
                    }
                }
            } else {
                const __nv_bfloat16* old = p.C + t.batch * p.batch_c + grow * p.ldc + col0;
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    if (col0 + g * 8 < p.N) {
                        const uint4 o = *reinterpret_cast<const uint4*>(old + g * 8);
                        const uint32_t ow[4] = {o.x, o.y, o.z, o.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            sum[8 * g + 2 * e] = fmaf(p.beta, __uint_as_float(ow[e] << 16), sum[8 * g + 2 * e]);
                            sum[8 * g + 2 * e + 1] = fmaf(p.beta, __uint_as_float(ow[e] & 0xFFFF0000u), sum[8 * g + 2 * e + 1]);
                        }
                    }
                }
            }
        }
        uint8_t* blk = f32 ? blocks : blocks + (step & 1) * 2048;
        // the store that last read this block (the previous one; for bf16 the one before it) must be done with it
        if (lane == 0) { if (f32) ptx::tma_store_wait_read<0>(); else ptx::tma_store_wait_read<1>(); }
        __syncwarp();
        if (f32) {
            uint8_t* my_row = blk + lane * 128;
#pragma unroll
            for (int g = 0; g < 8; ++g)
                *reinterpret_cast<float4*>(my_row + ((g ^ (lane & 7)) << 4)) = make_float4(sum[4 * g], sum[4 * g + 1], sum[4 * g + 2], sum[4 * g + 3]);
        } else {
            uint32_t pk[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                __nv_bfloat162 h2 = __floats2bfloat162_rn(sum[2 * e], sum[2 * e + 1]);
                pk[e] = *reinterpret_cast<uint32_t*>(&h2);
            }
            uint8_t* my_row = blk + lane * 64;
            const int sw = (lane >> 1) & 3;
#pragma unroll
            for (int g = 0; g < 4; ++g)
                *reinterpret_cast<uint4*>(my_row + ((g ^ sw) << 4)) = make_uint4(pk[4 * g], pk[4 * g + 1], pk[4 * g + 2], pk[4 * g + 3]);
        }
        ptx::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0 && row0 < p.M && col0 < p.N) {
            if (p.batch > 1) ptx::tma_store_3d(tmC, blk, col0, row0, t.batch);
            else ptx::tma_store_2d(tmC, blk, col0, row0);
            ptx::tma_store_commit();
        }
        __syncwarp();
    }
    // shared memory must stay alive until the copy engine has drained this warp's last store
    if (lane == 0) ptx::tma_store_wait_all<0>();
}

template <bool kConv>
__global__ void __launch_bounds__(576, 1)
umma_contract_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                     const __grid_constant__ CUtensorMap tmC, const UmmaParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kMaxStages];
    __shared__ __align__(8) uint64_t empty_bar[kMaxStages];
    __shared__ __align__(8) uint64_t tfull_bar[kMaxSlots];
    __shared__ __align__(8) uint64_t tempty_bar[kMaxSlots];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t b_bytes = static_cast<uint32_t>(p.bn) * 128u;
    const int mh = p.bm / kHalfM;                      // 128-row halves per tile
    const uint32_t a_bytes = static_cast<uint32_t>(mh) * kHalfABytes;
    const uint32_t stage_bytes = a_bytes + b_bytes;
    volatile int* abort_flag = &s_abort;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            ptx::mbar_init(&full_bar[s], 1);
            ptx::mbar_init(&empty_bar[s], 1);
        }
        for (int b = 0; b < p.slots; ++b) {
            ptx::mbar_init(&tfull_bar[b], 1);
            ptx::mbar_init(&tempty_bar[b], static_cast<uint32_t>(((blockDim.x >> 5) - 2) / mh));
        }
        s_abort = 0;
        ptx::fence_barrier_init();
        ptx::tma_prefetch_desc(&tmA);
        ptx::tma_prefetch_desc(&tmB);
        if (p.tma_store || p.cluster_tma) ptx::tma_prefetch_desc(&tmC);
    }
    if (warp == 1) {
        __syncwarp();
        ptx::tmem_alloc(&s_tmem_base, static_cast<uint32_t>(p.tmem_cols));
        ptx::tmem_relinquish();
    }
    // What does not depend on the previous grid's results happens BEFORE the dependency wait below, in the microsecond
    // or so between this CTA's start and the predecessor's completion: every role works out its first tile (the tile
    // table was written by the host long before any launch that reads it).  Asking for the first K blocks to be brought
    // into L2 here as well was measured and dropped: the loads after the wait did land 1-2 us sooner, but the wait itself
    // returned later by more than that (1024^3: 11.5 vs 10.2 us per step).
    const int total_items = p.tiles_m * p.tiles_n * p.split_k * (p.batch > 1 ? p.batch : 1);
    TileCoord t_first;
    const bool have_first = get_tile(p, 0, blockIdx.x, gridDim.x, total_items, &t_first);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = s_tmem_base;
    // the next grid in the stream (the split-K reduction, or the next call's kernel) may be scheduled as SMs free up and
    // run its set-up; this grid reads and writes global data only after its own predecessor has completed
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        if (ptx::elect_one()) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            TileCoord t = t_first;
            bool have = have_first;
            for (int local = 0; ok && have; have = get_tile(p, ++local, blockIdx.x, gridDim.x, total_items, &t)) {
                const int nkb = t.kb1 - t.kb0;
                const uint32_t tile_tx = a_bytes + static_cast<uint32_t>(t.bn) * 128u;
                int kb = first_kblock(p, t);
                for (int i = 0; i < nkb; ++i, kb = (kb + 1 == t.kb1) ? t.kb0 : kb + 1) {
                    if (!wait_bounded(&empty_bar[stage], phase ^ 1u, abort_flag, p.status, kTimeoutProducer)) {
                        ok = false;
                        break;
                    }
                    uint64_t* bar = &full_bar[stage];
                    ptx::mbar_arrive_expect_tx(bar, tile_tx);
                    uint8_t* a_dst = smem + static_cast<size_t>(stage) * stage_bytes;
                    issue_kblock<kConv>(p, &tmA, &tmB, t, kb, mh, a_dst, a_dst + a_bytes, bar);
                    if (++stage == p.stages) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
            if (!ok) {
                // let copies that are still in flight land before the CTA goes away
                for (int i = 0; i < 64; ++i) __nanosleep(2000);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (ptx::elect_one()) {
            const uint32_t idesc0 = ptx::make_idesc_bf16_f32(kHalfM, p.bn, p.a_mn_major, p.b_mn_major);
            // K-major: 8-row groups are 1024 B apart (SBO); K advances 32 B inside the swizzle row.
            // MN-major: 64-element groups along MN are one 64 x 64 box (8192 B) apart (LBO),
            //           8-k groups are 1024 B apart (SBO); K advances 16 rows = 2048 B.
            const uint32_t a_lbo = p.a_mn_major ? 8192u : 16u;
            const uint32_t b_lbo = p.b_mn_major ? 8192u : 16u;
            const uint32_t a_kstep = p.a_mn_major ? 2048u : 32u;
            const uint32_t b_kstep = p.b_mn_major ? 2048u : 32u;
            // The issuing thread must spend far fewer cycles per MMA than the MMA takes (128 at N = 256, 32 at
            // N = 64), so the descriptors are built once and only advanced by additions in 16-byte units.
            const uint64_t a_desc0 = ptx::make_smem_desc_sw128(ptx::smem_u32(smem), a_lbo, 1024u);
            const uint64_t b_desc0 = ptx::make_smem_desc_sw128(ptx::smem_u32(smem) + a_bytes, b_lbo, 1024u);
            const uint64_t stage_step = stage_bytes >> 4;
            const uint64_t a_k16 = a_kstep >> 4, b_k16 = b_kstep >> 4;
            uint64_t a_desc = a_desc0, b_desc = b_desc0;       // descriptors of the current stage
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            TileCoord t = t_first;
            bool have = have_first;
            for (int local = 0; ok && have; have = get_tile(p, ++local, blockIdx.x, gridDim.x, total_items, &t)) {
                // N field of the instruction descriptor (bits 17..22) follows the tile's width
                const uint32_t idesc = (idesc0 & ~(0x3Fu << 17)) | (static_cast<uint32_t>(t.bn >> 3) << 17);
                // accumulator slots of this tile: use number u of slot s has barrier phase (u & 1)
                uint32_t d_tmem[2] = {0u, 0u};
                int slot[2] = {0, 0};
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    if (h < mh && ok) {
                        const int idx = local * mh + h;
                        slot[h] = idx % p.slots;
                        const uint32_t aphase = (idx / p.slots) & 1;
                        d_tmem[h] = tmem_base + static_cast<uint32_t>(slot[h] * p.bn);
                        if (!wait_bounded(&tempty_bar[slot[h]], aphase ^ 1u, abort_flag, p.status, kTimeoutMma))
                            ok = false;
                    }
                }
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const int nkb = t.kb1 - t.kb0;
                for (int i = 0; i < nkb; ++i) {
                    if (!wait_bounded(&full_bar[stage], phase, abort_flag, p.status, kTimeoutMma)) {
                        ok = false;
                        break;
                    }
                    ptx::tc_fence_after_sync();
                    const uint32_t first = i > 0 ? 1u : 0u;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        if (h < mh) {
#pragma unroll
                            for (int j = 0; j < kBK / kUmmaK; ++j)
                                ptx::umma_bf16(d_tmem[h], a_desc + (h * (kHalfABytes >> 4) + j * a_k16), b_desc + j * b_k16,
                                               idesc, j > 0 ? 1u : first);
                        }
                    }
                    ptx::umma_commit(&empty_bar[stage]);
                    if (++stage == p.stages) {
                        stage = 0;
                        phase ^= 1u;
                        a_desc = a_desc0;
                        b_desc = b_desc0;
                    } else {
                        a_desc += stage_step;
                        b_desc += stage_step;
                    }
                }
                if (ok) {
                    ptx::umma_commit(&tfull_bar[slot[0]]);
                    if (mh == 2) ptx::umma_commit(&tfull_bar[slot[1]]);
                }
            }
        }
    } else if (!kConv && p.cluster_reduce) {
        // the partial tile of this CTA's K slice is complete once the accumulator barrier (of this warp's 128-row half) flips
        if (have_first) wait_bounded(&tfull_bar[((warp - 2) >> 2) % mh], 0u, abort_flag, p.status, kTimeoutEpilogue);
        ptx::tc_fence_after_sync();
    } else {
        epilogue_role<kConv>(p, &tmC, smem + static_cast<size_t>(p.stages) * stage_bytes, tmem_base, tfull_bar,
                             tempty_bar, abort_flag, mh, warp, lane, total_items, -1, 0, 1, 0, 0, nullptr, &t_first, have_first);
    }
    if (!kConv && p.cluster_reduce) {
        // Every thread of every CTA of the cluster takes part in both barriers, whatever happened in its role.
        // (1) all partial tiles are complete, so every CTA's pipeline stages are free: they become the receive slots;
        // (2) all slices have arrived where they are summed.  After (2) a CTA touches only its own shared memory.
        const int me = static_cast<int>(ptx::cluster_ctarank());
        const bool good = have_first && !*abort_flag;
        ptx::cluster_sync_all();
        if (warp >= 2 && good) cluster_push_partials(p, smem, tmem_base, warp, lane, me);
        ptx::cluster_sync_all();
        if (warp >= 2 && good && p.cluster_tma) {
            cluster_reduce_store(p, &tmC, smem, smem + static_cast<size_t>(p.stages) * stage_bytes, tmem_base, t_first, warp, lane, me);
        } else if (warp >= 2 && good) {
            TileCoord slice = t_first;
            slice.bn = p.bn / p.split_k;
            slice.n0 = t_first.n0 + me * slice.bn;
            epilogue_role<kConv>(p, &tmC, smem + static_cast<size_t>(p.stages) * stage_bytes, tmem_base, tfull_bar, tempty_bar,
                                 abort_flag, mh, warp, lane, total_items, -1, 0, 1, 0, 0, nullptr, &slice, true, smem, me);
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        __syncwarp();
        ptx::tmem_dealloc(tmem_base, static_cast<uint32_t>(p.tmem_cols));
    }
}

}  // namespace tdx
