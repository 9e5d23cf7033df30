// The tiled tensor-core path for large problems: CTA pairs (thread-block clusters of two).
//
// A pair owns a 256 x 256 output tile (256 x 128 for SwiGLU).  Each CTA loads its own 128
// rows of X and its own half of the W rows of the tile, so a ring stage is 32 KiB instead of
// 48 KiB: six stages deep instead of four and a third less L2 -> shared-memory traffic per
// FLOP.  The even CTA issues tcgen05.mma.cta_group::2 (M = 256) for both; each CTA keeps the
// accumulator of its own 128 rows in its own TMEM and runs its own epilogue.
//
// Barriers: all TMA bytes of a stage (both CTAs') are counted on the even CTA's `full`
// barrier; tcgen05.commit with a cluster mask frees the stage in both CTAs and publishes
// the accumulator to both; the epilogue warps of both CTAs arrive on the even CTA's
// `accumulator empty` barrier.  No TMA load uses cluster multicast.
#pragma once
#include "gemm_tiled.cuh"

namespace mtmc {

template <int EPI>
struct PairCfg {
    static constexpr int BM = 256;                       // rows per pair tile (128 per CTA)
    static constexpr int BN = 256;                       // accumulator columns
    static constexpr int BK = 64;
    static constexpr int A_BYTES = 128 * BK * 2;         // this CTA's X rows
    static constexpr int B_BYTES = 128 * BK * 2;         // this CTA's half of the W rows (at most)
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int STAGES = 6;
    static constexpr int OUT_TILE_N = (EPI == EPI_SWIGLU) ? BN / 2 : BN;
    static constexpr int TMEM_COLS = 2 * BN;
    static constexpr int NUM_BARRIERS = 2 * STAGES + 4;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_WARPS * EPI_STAGE_BYTES_PER_WARP + NUM_BARRIERS * 8 + 16 + 1024;
    static constexpr int THREADS = 64 + 32 * EPI_WARPS;
};

template <int EPI, bool OUT_BF16>
__global__ void __launch_bounds__(64 + 32 * EPI_WARPS, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                 const __grid_constant__ CUtensorMap tmB2, const __grid_constant__ CUtensorMap tmBt,
                 const __grid_constant__ CUtensorMap tmB2t, const GemmParams p) {
    using Cfg = PairCfg<EPI>;
    constexpr int STAGES = Cfg::STAGES;
    extern __shared__ uint8_t smem_raw[];

    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    const uint32_t epi_stage_base = base + STAGES * Cfg::STAGE_BYTES;        // warp-private store staging
    const uint32_t bar_base = epi_stage_base + EPI_WARPS * EPI_STAGE_BYTES_PER_WARP;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto accf_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + b); };
    auto acce_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + 2 + b); };
    uint8_t* ctrl = smem_raw + (bar_base - raw_addr) + 8 * Cfg::NUM_BARRIERS;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(ctrl);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(ctrl + 4);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();            // 0: issues the MMAs, owns the shared barriers
    const int pair_id = static_cast<int>(blockIdx.x >> 1);
    const int num_pairs = static_cast<int>(gridDim.x >> 1);

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(accf_bar(b), 1); mbar_init(acce_bar(b), 2 * EPI_WARPS); }   // every epilogue warp of both CTAs
        *abort_flag = 0u;
        fence_barrier_init();
        fence_proxy_async_smem();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(rank == 0 ? &tmB : (EPI == EPI_SWIGLU ? &tmB2 : &tmB));
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(tmem_slot)), Cfg::TMEM_COLS);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_arrive();        // both CTAs' barriers are initialised before either side signals the other
    cluster_wait();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_launch_dependents();     // the next kernel in the stream may begin its own set-up
    pdl_wait();                  // everything before this line touched only shared and tensor memory

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            const uint32_t full0_base = cluster_map_shared(full_bar(0), 0);   // the even CTA's full barriers
            for (int t = pair_id; t < p.num_items && ok; t += num_pairs) {
                int mb, nb, sub, width;
                item_coords(p, t, Cfg::OUT_TILE_N, mb, nb, sub, width);
                const bool whole = width == Cfg::OUT_TILE_N;
                const int m0 = mb * Cfg::BM + static_cast<int>(rank) * 128;
                // This CTA's share of the B operand: SwiGLU -> rank 0 the gate rows, rank 1 the up rows of
                // the same columns; otherwise the first / second half of the item's W rows.
                const int b_rows = (EPI == EPI_SWIGLU) ? width : width / 2;
                const int n_row0 = nb * Cfg::OUT_TILE_N + sub * width + ((EPI == EPI_SWIGLU) ? 0 : static_cast<int>(rank) * b_rows);
                const CUtensorMap* mapB = (EPI == EPI_SWIGLU && rank == 1) ? (whole ? &tmB2 : &tmB2t) : (whole ? &tmB : &tmBt);
                const uint32_t cta_bytes = Cfg::A_BYTES + static_cast<uint32_t>(b_rows) * Cfg::BK * 2;
                int kx = 0;                                              // K coordinate of the next k-block
                for (int kb = 0; kb < p.k_blocks; ++kb, kx += p.bk_elems) {
                    if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, p.status, STATUS_TIMEOUT_PRODUCER | 3u)) { ok = false; break; }
                    // loads first, bookkeeping after: the time from "slot free" to "load issued" is on the ring's
                    // critical path (a transaction count may run ahead of its expect_tx within a phase)
                    const uint32_t a_dst = base + s * Cfg::STAGE_BYTES;
                    const uint32_t full0 = full0_base + 8u * s;
                    tma_load_2d_pair(a_dst, &tmA, full0, kx, m0);
                    tma_load_2d_pair(a_dst + Cfg::A_BYTES, mapB, full0, kx, n_row0);
                    if (rank == 0) mbar_expect_tx(full_bar(s), 2u * cta_bytes);     // both CTAs' bytes
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (even CTA only)
        if (lane == 0 && rank == 0) {
            int s = 0;
            uint32_t ph = 0;
            uint32_t acc_ph = 0;
            int it = 0;
            bool ok = true;
            for (int t = pair_id; t < p.num_items && ok; t += num_pairs, ++it) {
                const int buf = it & 1;
                const int width = t < p.n_full ? Cfg::OUT_TILE_N : p.tail_width;
                const int mma_n = EPI == EPI_SWIGLU ? 2 * width : width;
                const uint32_t idesc = p.fp8 ? umma_idesc_e4m3(Cfg::BM, mma_n) : umma_idesc_bf16(Cfg::BM, mma_n);
                if (!mbar_wait_cluster(acce_bar(buf), ((acc_ph >> buf) & 1u) ^ 1u, abort_flag, p.status, STATUS_TIMEOUT_MMA | 5u)) { ok = false; break; }
                acc_ph ^= 1u << buf;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(buf * Cfg::BN);
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    if (!mbar_wait(full_bar(s), ph, abort_flag, p.status, STATUS_TIMEOUT_MMA | 6u)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_src = base + s * Cfg::STAGE_BYTES;
                    const uint64_t a_desc = umma_smem_desc_sw128(a_src);
                    const uint64_t b_desc = umma_smem_desc_sw128(a_src + Cfg::A_BYTES);
                    // four MMAs per 128-byte row either way: 4 x 16 bf16 or 4 x 32 E4M3, 32 bytes apart
                    if (p.fp8) {
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            umma_fp8_pair(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, (kb | k) != 0 ? 1u : 0u);
                    } else {
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            umma_bf16_pair(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, (kb | k) != 0 ? 1u : 0u);
                    }
                    umma_commit_pair(empty_bar(s), 3);           // frees the stage in both CTAs
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                if (ok) umma_commit_pair(accf_bar(buf), 3);      // accumulator complete, in both CTAs
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue (both CTAs)
        const int q = warp & 3;                      // TMEM lane quadrant this warp may read
        const int half = (warp - 2) >> 2;            // which half of the item's columns this warp takes
        const uint32_t lane_base = static_cast<uint32_t>(q * 32) << 16;
        const bool vec_ok = OUT_BF16 ? (p.ldo % 8 == 0) : (p.ldo % 4 == 0);
        uint32_t acc_ph = 0;
        int it = 0;
        bool ok = true;
        for (int t = pair_id; t < p.num_items && ok; t += num_pairs, ++it) {
            const int buf = it & 1;
            int mb, nb, sub, width;
            item_coords(p, t, Cfg::OUT_TILE_N, mb, nb, sub, width);
            const int row = mb * Cfg::BM + static_cast<int>(rank) * 128 + q * 32 + lane;
            const int n_tile0 = nb * Cfg::OUT_TILE_N + sub * width;
            if (!mbar_wait(accf_bar(buf), (acc_ph >> buf) & 1u, abort_flag, p.status, STATUS_TIMEOUT_EPILOGUE | 5u)) { ok = false; break; }
            acc_ph ^= 1u << buf;
            tc_fence_after();
            const uint32_t t_addr = tmem_base + lane_base + static_cast<uint32_t>(buf * Cfg::BN);
            const int chunks = width / 32, split_at = EPI_HALVES == 2 ? (chunks + 1) / 2 : chunks;      // two warps per lane quadrant share the columns
            epilogue_item<EPI, OUT_BF16>(p, t_addr, row, n_tile0, half ? split_at : 0, half ? chunks : split_at, width, nb, sub, half,
                                         vec_ok, smem_raw + (epi_stage_base - raw_addr) + (warp - 2) * EPI_STAGE_BYTES_PER_WARP, lane);
            // this CTA's half of the accumulator is drained: tell the MMA issuer in the even CTA
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_remote(cluster_map_shared(acce_bar(buf), 0));
        }
    }

    // ---------------------------------------------------------------------- teardown
    // Neither CTA may free its TMEM or leave while the other can still touch its memory or barriers.
    tc_fence_before();
    __syncthreads();
    cluster_arrive();
    cluster_wait();
    if (*abort_flag != 0u) {
        const long long t0 = clock64();
        while (clock64() - t0 < 400000ll) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, Cfg::TMEM_COLS);
    }
}

}  // namespace mtmc
