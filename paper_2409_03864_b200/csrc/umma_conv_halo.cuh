// Convolution kernel that keeps the input halo tile in shared memory across the filter taps.
//
// The per-tap kernel (umma_contract_kernel<true>) fetches the shifted input window again for every
// filter tap: R*S fetches of the same pixels from L2.  Here a 128-row MMA tile is an 8-wide, 16-high
// patch of output pixels; its (8 + S - 1) x (16 + R - 1) input window for one 64-channel chunk is loaded
// ONCE (one TMA box, zero fill outside the image), and tap (r, s) is read straight out of it: output
// pixel (h, w) of the patch needs window pixel (h + r, w + s), i.e. the 8-row groups of the A operand
// start at window row r, column s and are one window row (hpitch * 128 bytes) apart -- exactly what
// the shared-memory descriptor's start address and stride-dimension offset express.
//
// Why a start that is not 1024-byte aligned is legal here.  The copy engine writes the window into a buffer that
// starts on a 1024-byte boundary and applies the 128-byte swizzle as a function of the shared-memory ADDRESS (the
// 16-byte chunk index, address bits 4..6, is XORed with address bits 7..9).  The MMA unit applies the same function of
// the address when it reads.  The descriptor's base-offset field (bits 49..51) exists for a different situation: a
// matrix whose swizzle pattern is shifted against the address because the tile ITSELF was placed at a base that is
// not a multiple of the pattern's 1024-byte period; the field then carries (base >> 7) & 7.  A filter tap does not
// move the tile, it only starts reading further into it, at pixel (r, s) of the window: pattern and address still
// agree, so the field stays 0.  Checked both ways on the device: with the field 0 every halo parity case matches the
// oracle (integer cases bit for bit); with it set to (start >> 7) & 7, as for a shifted tile, 44 of 47 cases fail.
//
// Two rings: halo tiles (a_stages deep, one per channel chunk and 128-row half) and filter slices
// (stages deep, one per (chunk, tap)), each filled by its own warp (the last warp and warp 0), so that a
// halo tile that takes many copies never holds up the filter slices.  Accumulator slots, epilogue and
// bounded waits are those of umma_contract_kernel.
//
// Stacked images (Pv > 0): the 16-row patches are cut from the column formed by all images, Pv = H + pad
// rows per image, so an image height that is no multiple of 16 wastes no rows.  The Pv - P rows between
// two images read as zero: they are the bottom padding of one image and the top padding of the next.
#pragma once
#include "umma_kernel.cuh"

namespace tdx {

constexpr int kMaxAStages = 4;

// output patch of 128-row half `half` of tile `m_blk`: image n and top-left output pixel (p0, q0)
__device__ __forceinline__ void halo_patch_origin(const UmmaParams& p, int m_blk, int half, int mh, int* n, int* p0,
                                                  int* q0) {
    const int patch = m_blk * mh + half;
    if (p.Pv > 0) {
        // stacked images: *p0 is the row in the column of all images, *n is not used
        const int ph = patch / p.patches_w;
        *n = 0;
        *p0 = ph * p.bh;
        *q0 = (patch - ph * p.patches_w) * p.bw;
        return;
    }
    const int ppi = p.patches_w * p.patches_h;
    *n = patch / ppi;
    const int rem = patch - *n * ppi;
    const int ph = rem / p.patches_w;
    *p0 = ph * p.bh;
    *q0 = (rem - ph * p.patches_w) * p.bw;
}

// The input windows of channel chunk `cc` for the 128-row halves of tile `m_blk`, loaded into one halo stage.
__device__ __forceinline__ void issue_halo_windows(const UmmaParams& p, const CUtensorMap* tmA, const CUtensorMap* tmA_row,
                                                   int m_blk, int cc, int mh, uint8_t* stage_dst, uint64_t* bar) {
    auto ld4 = [&](uint8_t* dst, const CUtensorMap* m, int c0, int c1, int c2, int c3) {
        ptx::tma_load_4d(dst, m, bar, c0, c1, c2, c3);
    };
    for (int h = 0; h < mh; ++h) {
        int n, p0, q0;
        halo_patch_origin(p, m_blk, h, mh, &n, &p0, &q0);
        uint8_t* dst = stage_dst + h * p.halo_bytes;
        if (p.Pv > 0) {
            // Row u of the stacked column is row u % Pv of image u / Pv when that is below H, and
            // zero otherwise.  A window that lies inside one image and the zero rows around it is
            // one box (rows outside [0, H) are zero-filled); a window that reaches into the next
            // image is copied row by row.
            const int u = p0 - p.pad;
            int img = u >= 0 ? u / p.Pv : 0;
            int row = u >= 0 ? u - img * p.Pv : u;       // negative: above the first image
            if (row >= p.H) {                            // starts in the zero rows below image img:
                row -= p.Pv;                             // the same rows lie above image img + 1
                ++img;
            }
            if (row + p.hrows <= p.Pv) {
                // img == Nimg happens past the last image: that coordinate is zero-filled too
                ld4(dst, tmA, cc * kBK, q0 - p.pad, row, img);
            } else {
                for (int j = 0; j < p.hrows; ++j) {
                    const bool real = row >= 0 && row < p.H && img < p.Nimg;
                    ld4(dst + j * p.hpitch * 128, tmA_row, cc * kBK, q0 - p.pad, real ? row : p.H, real ? img : 0);
                    if (++row == p.Pv) { row = 0; ++img; }
                }
            }
        } else {
            ld4(dst, tmA, cc * kBK, q0 - p.pad, p0 - p.pad, n);
        }
    }
}

__global__ void __launch_bounds__(608, 1)
umma_conv_halo_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmA_row,
                      const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmC,
                      const __grid_constant__ CUtensorMap tmC_row, const UmmaParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t afull_bar[kMaxAStages];
    __shared__ __align__(8) uint64_t aempty_bar[kMaxAStages];
    __shared__ __align__(8) uint64_t bfull_bar[kMaxStages];
    __shared__ __align__(8) uint64_t bempty_bar[kMaxStages];
    __shared__ __align__(8) uint64_t tfull_bar[kMaxSlots];
    __shared__ __align__(8) uint64_t tempty_bar[kMaxSlots];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int mh = p.bm / kHalfM;
    const uint32_t b_bytes = static_cast<uint32_t>(p.bn) * 128u;
    const uint32_t a_stage_bytes = static_cast<uint32_t>(mh * p.halo_bytes);
    uint8_t* a_ring = smem;
    uint8_t* b_ring = smem + static_cast<size_t>(p.a_stages) * a_stage_bytes;
    uint8_t* staging = b_ring + static_cast<size_t>(p.stages) * b_bytes;
    volatile int* abort_flag = &s_abort;
    const int taps = p.R * p.S;
    const int halo_warp = 2 + p.epi_warps;      // the last warp loads the halo tiles

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.a_stages; ++s) {
            ptx::mbar_init(&afull_bar[s], 1);
            ptx::mbar_init(&aempty_bar[s], 1);
        }
        for (int s = 0; s < (p.b_resident ? 1 : p.stages); ++s) {
            ptx::mbar_init(&bfull_bar[s], 1);
            ptx::mbar_init(&bempty_bar[s], 1);
        }
        for (int b = 0; b < p.slots; ++b) {
            ptx::mbar_init(&tfull_bar[b], 1);
            ptx::mbar_init(&tempty_bar[b], static_cast<uint32_t>(p.epi_warps / mh));
        }
        s_abort = 0;
        ptx::fence_barrier_init();
        ptx::tma_prefetch_desc(&tmA);
        ptx::tma_prefetch_desc(&tmB);
        if (p.Pv > 0) ptx::tma_prefetch_desc(&tmA_row);
        if (p.tma_store) {
            ptx::tma_prefetch_desc(&tmC);
            if (p.Pv > 0) ptx::tma_prefetch_desc(&tmC_row);
        }
    }
    if (warp == 1) {
        __syncwarp();
        ptx::tmem_alloc(&s_tmem_base, static_cast<uint32_t>(p.tmem_cols));
        ptx::tmem_relinquish();
    }
    // before the dependency wait (see umma_contract_kernel): every role works out its first tile
    const int total_items = p.tiles_m * p.tiles_n;
    TileCoord t_first;
    const bool have_first = get_tile(p, 0, blockIdx.x, gridDim.x, total_items, &t_first);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = s_tmem_base;
    ptx::grid_launch_dependents();     // see umma_contract_kernel
    ptx::grid_dependency_wait();

    if (warp == halo_warp) {
        // ------------------------------------------------------------ halo producer: one tile per (item, channel chunk)
        if (ptx::elect_one()) {
            const uint32_t halo_tx = static_cast<uint32_t>(mh * p.hpitch * p.hrows) * 128u;
            int a_buf = 0;
            uint32_t a_phase = 0;
            bool ok = true;
            TileCoord t = t_first;
            bool have = have_first;
            for (int local = 0; ok && have; have = get_tile(p, ++local, blockIdx.x, gridDim.x, total_items, &t)) {
                for (int cc = 0; cc < p.cchunks; ++cc) {
                    if (!wait_bounded(&aempty_bar[a_buf], a_phase ^ 1u, abort_flag, p.status, kTimeoutProducer)) {
                        ok = false;
                        break;
                    }
                    uint64_t* bar = &afull_bar[a_buf];
                    ptx::mbar_arrive_expect_tx(bar, halo_tx);
                    issue_halo_windows(p, &tmA, &tmA_row, t.m_blk, cc, mh, a_ring + static_cast<size_t>(a_buf) * a_stage_bytes, bar);
                    if (++a_buf == p.a_stages) { a_buf = 0; a_phase ^= 1u; }
                }
            }
            if (!ok) {
                for (int i = 0; i < 64; ++i) __nanosleep(2000);
            }
        }
    } else if (warp == 0) {
        // ------------------------------------------------------------ filter producer
        if (ptx::elect_one()) {
            bool ok = true;
            if (p.b_resident) {
                // the whole filter once (slot = chunk * taps + tap)
                ptx::mbar_arrive_expect_tx(&bfull_bar[0], static_cast<uint32_t>(p.cchunks * taps) * b_bytes);
                for (int cc = 0; cc < p.cchunks; ++cc)
                    for (int tap = 0; tap < taps; ++tap)
                        ptx::tma_load_3d(b_ring + static_cast<size_t>(cc * taps + tap) * b_bytes, &tmB, &bfull_bar[0],
                                         cc * kBK, tap, 0);
            } else {
                int b_stage = 0;
                uint32_t b_phase = 0;
                TileCoord t = t_first;
                bool have = have_first;
                for (int local = 0; ok && have; have = get_tile(p, ++local, blockIdx.x, gridDim.x, total_items, &t)) {
                    const uint32_t slice_tx = static_cast<uint32_t>(t.bn) * 128u;     // the tile's width (fitted plans vary it)
                    for (int cc = 0; ok && cc < p.cchunks; ++cc) {
                        for (int tap = 0; tap < taps; ++tap) {
                            if (!wait_bounded(&bempty_bar[b_stage], b_phase ^ 1u, abort_flag, p.status, kTimeoutProducer)) {
                                ok = false;
                                break;
                            }
                            uint64_t* bar = &bfull_bar[b_stage];
                            ptx::mbar_arrive_expect_tx(bar, slice_tx);
                            for (int r0 = 0; r0 < t.bn; r0 += p.b_box)
                                ptx::tma_load_3d(b_ring + static_cast<size_t>(b_stage) * b_bytes + r0 * 128, &tmB, bar, cc * kBK,
                                                 tap, t.n0 + r0);
                            if (++b_stage == p.stages) { b_stage = 0; b_phase ^= 1u; }
                        }
                    }
                }
            }
            if (!ok) {
                for (int i = 0; i < 64; ++i) __nanosleep(2000);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (ptx::elect_one()) {
            const uint32_t idesc0 = ptx::make_idesc_bf16_f32(kHalfM, p.bn, 0, 0);
            const uint32_t a_sbo = static_cast<uint32_t>(p.hpitch) * 128u;     // one window row between 8-row groups
            // descriptors are built once and advanced by additions (16-byte units): the issuing thread has only
            // a few dozen cycles per MMA when the tile is narrow
            const uint64_t halo_desc0 = ptx::make_smem_desc_sw128(ptx::smem_u32(a_ring), 16u, a_sbo);
            const uint64_t b_desc0 = ptx::make_smem_desc_sw128(ptx::smem_u32(b_ring), 16u, 1024u);
            const uint64_t a_stage_step = a_stage_bytes >> 4, b_stage_step = b_bytes >> 4;
            const uint64_t half_step = static_cast<uint64_t>(p.halo_bytes) >> 4;
            uint64_t halo_desc = halo_desc0, b_desc = b_desc0;
            int a_buf = 0, b_stage = 0, local = 0;
            uint32_t a_phase = 0, b_phase = 0;
            bool ok = true;
            if (p.b_resident && !wait_bounded(&bfull_bar[0], 0, abort_flag, p.status, kTimeoutMma)) ok = false;
            TileCoord t = t_first;
            bool have = have_first;
            for (; ok && have; have = get_tile(p, ++local, blockIdx.x, gridDim.x, total_items, &t)) {
                // N field of the instruction descriptor (bits 17..22) follows the tile's width
                const uint32_t idesc = (idesc0 & ~(0x3Fu << 17)) | (static_cast<uint32_t>(t.bn >> 3) << 17);
                uint32_t d_tmem[2] = {0u, 0u};
                int slot[2] = {0, 0};
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    if (h < mh && ok) {
                        const int idx = local * mh + h;
                        slot[h] = idx % p.slots;
                        const uint32_t aphase = (idx / p.slots) & 1;
                        d_tmem[h] = tmem_base + static_cast<uint32_t>(slot[h] * p.bn);
                        if (!wait_bounded(&tempty_bar[slot[h]], aphase ^ 1u, abort_flag, p.status, kTimeoutMma)) ok = false;
                    }
                }
                if (!ok) break;
                ptx::tc_fence_after_sync();
                for (int cc = 0; ok && cc < p.cchunks; ++cc) {
                    if (!wait_bounded(&afull_bar[a_buf], a_phase, abort_flag, p.status, kTimeoutMma)) { ok = false; break; }
                    int r = 0, s = 0;                         // filter tap (r, s), advanced without divisions
                    uint64_t row_desc = halo_desc;            // window row r, column 0 (one pixel = 128 B = 8 units)
                    if (p.b_resident) b_desc = b_desc0 + static_cast<uint64_t>(cc * taps) * b_stage_step;
                    for (int tap = 0; tap < taps; ++tap) {
                        if (!p.b_resident &&
                            !wait_bounded(&bfull_bar[b_stage], b_phase, abort_flag, p.status, kTimeoutMma)) { ok = false; break; }
                        ptx::tc_fence_after_sync();
                        const uint64_t a_tap = row_desc + static_cast<uint64_t>(s) * 8u;
                        const uint32_t first = (cc > 0 || tap > 0) ? 1u : 0u;
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            if (h < mh) {
#pragma unroll
                                for (int j = 0; j < kBK / kUmmaK; ++j)
                                    ptx::umma_bf16(d_tmem[h], a_tap + (h ? half_step : 0) + 2 * j, b_desc + 2 * j, idesc,
                                                   j > 0 ? 1u : first);
                            }
                        }
                        if (p.b_resident) {
                            b_desc += b_stage_step;
                        } else {
                            ptx::umma_commit(&bempty_bar[b_stage]);
                            if (++b_stage == p.stages) { b_stage = 0; b_phase ^= 1u; b_desc = b_desc0; } else { b_desc += b_stage_step; }
                        }
                        if (++s == p.S) { s = 0; ++r; row_desc += static_cast<uint64_t>(p.hpitch) * 8u; }
                    }
                    if (!ok) break;
                    ptx::umma_commit(&aempty_bar[a_buf]);
                    if (++a_buf == p.a_stages) { a_buf = 0; a_phase ^= 1u; halo_desc = halo_desc0; } else { halo_desc += a_stage_step; }
                }
                if (ok) {
                    ptx::umma_commit(&tfull_bar[slot[0]]);
                    if (mh == 2) ptx::umma_commit(&tfull_bar[slot[1]]);
                }
            }
        }
    } else {
        epilogue_role<true>(p, &tmC, staging, tmem_base, tfull_bar, tempty_bar, abort_flag, mh, warp, lane, total_items,
                            -1, 0, 1, 0, 0, &tmC_row, &t_first, have_first);
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
