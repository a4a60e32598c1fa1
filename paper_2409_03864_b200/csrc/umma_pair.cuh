// GEMM kernel on CTA pairs (cluster of two CTAs, tcgen05 cta_group::2).
//
// A pair owns a stream of 256 x BN output tiles.  Each CTA stages only ITS 128 rows of op(A) and ITS BN/2
// columns of op(B) for a K-step (32 KiB per stage at BN = 256, so twice as many stages fit as in the
// single-CTA 256 x 256 tile), one thread of the leader CTA (cluster rank 0) issues MMAs of shape
// 256 x BN x 16 that read both CTAs' shared memory, and each CTA ends up with its own 128 x BN half of the
// accumulator in its own tensor memory.  That half is 256 columns, so two accumulator slots fit again and
// the epilogue of tile t overlaps the main loop of tile t+1 -- which the single-CTA 256 x 256 tile cannot do.
// L2-to-SM traffic per flop equals that of the single-CTA 256 x 256 tile.  No broadcast loads are used.
//
// Synchronisation (leader = rank 0):
//   full[s]    leader's barrier, one arrival (the leader's producer, which also announces the bytes of BOTH
//              CTAs); both producers' TMA loads count their bytes on it.
//   empty[s]   one per CTA; the leader's MMA thread signals both with one commit when a stage has been read.
//   tfull[b]   one per CTA, signalled together by one commit when a tile's accumulators are complete.
//   tempty[b]  leader's barrier; the epilogue warps of both CTAs arrive on it (the peer's through the cluster
//              shared-memory window) when they have drained slot b.
// All waits are bounded as in umma_contract_kernel.
#pragma once
#include "umma_kernel.cuh"

namespace tdx {

__global__ void __launch_bounds__(576, 1)
umma_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
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
    const uint32_t rank = ptx::cluster_ctarank();          // 0 = leader
    const int pair_id = blockIdx.x >> 1;
    const int num_pairs = gridDim.x >> 1;
    const int half_bn = p.bn / 2;
    const uint32_t b_bytes = static_cast<uint32_t>(half_bn) * 128u;   // this CTA's share of the B slice
    const uint32_t stage_bytes = kHalfABytes + b_bytes;
    const int nwarps_epi = (static_cast<int>(blockDim.x) >> 5) - 2;
    volatile int* abort_flag = &s_abort;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            ptx::mbar_init(&full_bar[s], 1);
            ptx::mbar_init(&empty_bar[s], 1);
        }
        for (int b = 0; b < p.slots; ++b) {
            ptx::mbar_init(&tfull_bar[b], 1);
            ptx::mbar_init(&tempty_bar[b], static_cast<uint32_t>(2 * nwarps_epi));   // both CTAs' epilogue warps
        }
        s_abort = 0;
        ptx::fence_barrier_init();
        ptx::tma_prefetch_desc(&tmA);
        ptx::tma_prefetch_desc(&tmB);
        if (p.tma_store) ptx::tma_prefetch_desc(&tmC);
    }
    if (warp == 1) {
        __syncwarp();
        ptx::tmem_alloc_pair(&s_tmem_base, static_cast<uint32_t>(p.tmem_cols));
        ptx::tmem_relinquish_pair();
    }
    // before the dependency wait (see umma_contract_kernel): the pair's first tile
    const int total_items = p.tiles_m * p.tiles_n;     // tiles of 256 rows
    TileCoord t_first;
    const bool have_first = get_tile(p, 0, pair_id, num_pairs, total_items, &t_first);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync_all();          // barriers of both CTAs are initialised before anyone signals across
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = s_tmem_base;
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();

    if (warp == 0) {
        // ------------------------------------------------------------ producer (one per CTA)
        if (ptx::elect_one()) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            TileCoord t = t_first;
            bool have = have_first;
            for (int local = 0; ok && have; have = get_tile(p, ++local, pair_id, num_pairs, total_items, &t)) {
                const int my_bn = t.bn / 2;                                            // this CTA's share of the tile's columns
                const int row0 = t.m_blk * 256 + static_cast<int>(rank) * kHalfM;      // this CTA's rows of op(A)
                const int col0 = t.n0 + static_cast<int>(rank) * my_bn;                // this CTA's columns of op(B)
                const uint32_t pair_tx = 2u * (kHalfABytes + static_cast<uint32_t>(my_bn) * 128u);
                for (int kb = 0; kb < p.num_kb; ++kb) {
                    if (!wait_bounded(&empty_bar[stage], phase ^ 1u, abort_flag, p.status, kTimeoutProducer)) {
                        ok = false;
                        break;
                    }
                    if (rank == 0) ptx::mbar_arrive_expect_tx(&full_bar[stage], pair_tx);
                    const uint32_t bar = ptx::mapa_u32(ptx::smem_u32(&full_bar[stage]), 0);   // the leader's barrier
                    uint8_t* a_dst = smem + static_cast<size_t>(stage) * stage_bytes;
                    uint8_t* b_dst = a_dst + kHalfABytes;
                    if (p.a_mn_major) {
                        ptx::tma_load_2d_pair(a_dst, &tmA, bar, row0, kb * kBK);
                        ptx::tma_load_2d_pair(a_dst + 8192, &tmA, bar, row0 + 64, kb * kBK);
                    } else {
                        ptx::tma_load_2d_pair(a_dst, &tmA, bar, kb * kBK, row0);
                    }
                    if (p.b_mn_major) {
                        for (int i = 0; i < my_bn / 64; ++i)
                            ptx::tma_load_2d_pair(b_dst + i * 8192, &tmB, bar, col0 + i * 64, kb * kBK);
                    } else {
                        for (int r0 = 0; r0 < my_bn; r0 += p.b_box)
                            ptx::tma_load_2d_pair(b_dst + r0 * 128, &tmB, bar, kb * kBK, col0 + r0);
                    }
                    if (++stage == p.stages) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
            if (!ok) {
                for (int i = 0; i < 64; ++i) __nanosleep(2000);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (leader CTA only)
        if (rank == 0 && ptx::elect_one()) {
            const uint32_t idesc0 = ptx::make_idesc_bf16_f32(256, p.bn, p.a_mn_major, p.b_mn_major);
            const uint32_t a_lbo = p.a_mn_major ? 8192u : 16u;
            const uint32_t b_lbo = p.b_mn_major ? 8192u : 16u;
            const uint32_t a_kstep = p.a_mn_major ? 2048u : 32u;
            const uint32_t b_kstep = p.b_mn_major ? 2048u : 32u;
            const uint64_t a_desc0 = ptx::make_smem_desc_sw128(ptx::smem_u32(smem), a_lbo, 1024u);
            const uint64_t b_desc0 = ptx::make_smem_desc_sw128(ptx::smem_u32(smem) + kHalfABytes, b_lbo, 1024u);
            const uint64_t stage_step = stage_bytes >> 4;
            const uint64_t a_k16 = a_kstep >> 4, b_k16 = b_kstep >> 4;
            uint64_t a_desc = a_desc0, b_desc = b_desc0;
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            TileCoord t = t_first;
            bool have = have_first;
            for (int local = 0; ok && have; have = get_tile(p, ++local, pair_id, num_pairs, total_items, &t)) {
                // N field of the instruction descriptor (bits 17..22) follows the tile's width
                const uint32_t idesc = (idesc0 & ~(0x3Fu << 17)) | (static_cast<uint32_t>(t.bn >> 3) << 17);
                const int slot = local % p.slots;
                const uint32_t aphase = (local / p.slots) & 1;
                if (!wait_bounded(&tempty_bar[slot], aphase ^ 1u, abort_flag, p.status, kTimeoutMma)) break;
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(slot * p.bn);
                for (int kb = 0; kb < p.num_kb; ++kb) {
                    if (!wait_bounded(&full_bar[stage], phase, abort_flag, p.status, kTimeoutMma)) {
                        ok = false;
                        break;
                    }
                    ptx::tc_fence_after_sync();
                    const uint32_t first = kb > 0 ? 1u : 0u;
#pragma unroll
                    for (int j = 0; j < kBK / kUmmaK; ++j)
                        ptx::umma_bf16_pair(d_tmem, a_desc + j * a_k16, b_desc + j * b_k16, idesc, j > 0 ? 1u : first);
                    ptx::umma_commit_pair(&empty_bar[stage], 3);      // frees the stage in both CTAs
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
                if (ok) ptx::umma_commit_pair(&tfull_bar[slot], 3);   // accumulators complete in both CTAs
            }
        }
    } else {
        // each CTA drains its own 128 x BN half: rows 128 * (2 m + rank) of the matrix
        const uint32_t leader_tempty = ptx::mapa_u32(ptx::smem_u32(&tempty_bar[0]), 0);
        epilogue_role<false>(p, &tmC, smem + static_cast<size_t>(p.stages) * stage_bytes, tmem_base, tfull_bar, tempty_bar,
                             abort_flag, 1, warp, lane, total_items, pair_id, num_pairs, 2, static_cast<int>(rank),
                             leader_tempty, nullptr, &t_first, have_first);
    }

    // neither CTA may free tensor memory or leave while the other can still touch its memory
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync_all();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        __syncwarp();
        ptx::tmem_dealloc_pair(tmem_base, static_cast<uint32_t>(p.tmem_cols));
    }
}

}  // namespace tdx
