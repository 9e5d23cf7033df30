// Block-scaled E4M3 (MXFP8) on CTA pairs: the cta_group::2 form of gemm_mx.cuh for large problems.
//
// A pair owns a 256 x 224 output tile (SwiGLU: 256 x 96, from 96 gate and 96 up accumulator columns, so that the
// tile is a whole number of 32-column epilogue chunks).  As in gemm_pair.cuh each CTA loads its own 128 rows
// of X and its own half of the tile's W rows (112; SwiGLU: rank 0 the 96 gate rows, rank 1 the 96 up rows), the even CTA issues the MMAs for both
// (tcgen05.mma.cta_group::2.kind::mxf8f6f4.block_scale, M = 256, N = 224, K = 32), and each CTA keeps the
// accumulator of its 128 rows in its own tensor memory, two buffers of 224 columns, so that a tile's epilogue
// runs under the next tile's mainloop.  224 and not 256 columns: the scales need tensor memory too (two sets of
// 4 columns for the X scales and 8 for the W scales), and 2 x 256 accumulator columns would fill all 512.
//
// Scales: a CTA's datapath multiplies its 128 rows with all 224 columns, so its tensor memory needs the scales
// of its own 128 rows of X and of ALL 224 rows of W.  Each CTA therefore loads, per ring stage, its own 512-byte
// block of X scales and the tile's whole 1024-byte block of W scales (the second CTA's copy is an L2 hit), to
// the same shared-memory offsets in both CTAs; one tcgen05.cp.cta_group::2 per block then copies in both CTAs,
// each from its own shared memory to its own tensor memory.  The scale blocks come in by TMA as well (a plain,
// unswizzled byte tensor of 256-byte rows), so that every byte of a stage is counted on the even CTA's `full`
// barrier like the operand tiles.  No load uses cluster multicast.
#pragma once
#include "gemm_mx.cuh"

namespace mtmc {

template <int EPI>
struct MxPairCfg {
    static constexpr int BM = 256;                        // rows per pair tile (128 per CTA)
    static constexpr int BN = (EPI == EPI_SWIGLU) ? 192 : 224;   // accumulator columns (SwiGLU: 96 gate + 96 up)
    static constexpr int BK = 128;                        // E4M3 elements per ring stage: four MMAs of K = 32
    static constexpr int HALF_ROWS = BN / 2;              // W rows each CTA loads
    static constexpr int A_BYTES = 128 * BK;              // 16 KiB
    static constexpr int B_BYTES = HALF_ROWS * BK;        // 14 KiB (SwiGLU: 12 KiB), in a 16 KiB slot
    static constexpr int B_SLOT = 128 * BK;
    static constexpr int SFA_BYTES = 512;                 // scales of this CTA's 128 rows of X x 4 k-blocks
    static constexpr int SFB_BYTES = 1024;                // scales of the tile's 224 or 192 (of 256) accumulator columns x 4 k-blocks
    static constexpr int SF_OFFSET = A_BYTES + B_SLOT;
    static constexpr int SUB_BYTES = 34 * 1024;           // one k-block: operands 32 KiB + scales 1.5 KiB, padded to keep k-blocks 1024-byte aligned
    static constexpr int KB_PER_STAGE = 2;                // two k-blocks per hand-over, as in gemm_pair.cuh: the issuing thread, with three scale copies and
    static constexpr int STAGE_BYTES = KB_PER_STAGE * SUB_BYTES;   // four MMAs per k-block, is what sets the pace, and a wait and a commit per stage come on top
    static constexpr int STAGES = 3;
    static constexpr int OUT_TILE_N = (EPI == EPI_SWIGLU) ? BN / 2 : BN;
    static constexpr int SF_COL0 = 448;                   // after two accumulator buffers: two sets of (4 + 8) scale columns
    static constexpr int TMEM_COLS = 512;
    static constexpr int NUM_BARRIERS = 2 * STAGES + 4;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 4 * EPI_STAGE_BYTES_PER_WARP + NUM_BARRIERS * 8 + 16 + 1024;
    static constexpr int THREADS = 192;
    static_assert(SF_OFFSET + SFA_BYTES + SFB_BYTES <= SUB_BYTES && SMEM_BYTES <= 227 * 1024, "a stage holds operands and scales; six stages fit");
    static_assert(SF_COL0 + 24 <= TMEM_COLS && EPI_HALVES == 1, "accumulators and scale columns fit tensor memory");
    static_assert(2 * BN <= SF_COL0 && OUT_TILE_N % 32 == 0 && HALF_ROWS % 8 == 0, "accumulator buffers below the scale columns; whole epilogue chunks; whole swizzle atoms");
};

__device__ __forceinline__ void tmem_cp_scales_pair(uint32_t taddr, uint64_t sdesc) {
    asm volatile("tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
__device__ __forceinline__ void umma_mxf8_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t sfa_tmem,
                                               uint32_t sfb_tmem, uint32_t accumulate) {
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::mxf8f6f4.block_scale [%0], %1, %2, %3, [%5], [%6], p;\n\t"
        "}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem)
        : "memory");
}

// tmSFA / tmSFB: the re-arranged scales as plain byte tensors of 256-byte rows (two rows per 512-byte block).
template <int EPI, bool OUT_BF16>
__global__ void __launch_bounds__(192, 1)
gemm_mx_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const __grid_constant__ CUtensorMap tmB2, const __grid_constant__ CUtensorMap tmSFA,
                    const __grid_constant__ CUtensorMap tmSFB, const GemmParams p) {
    using Cfg = MxPairCfg<EPI>;
    constexpr int STAGES = Cfg::STAGES;
    extern __shared__ uint8_t smem_raw[];

    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    const uint32_t epi_stage_base = base + STAGES * Cfg::STAGE_BYTES;
    const uint32_t bar_base = epi_stage_base + 4 * EPI_STAGE_BYTES_PER_WARP;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto accf_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + b); };
    auto acce_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + 2 + b); };
    uint8_t* ctrl = smem_raw + (bar_base - raw_addr) + 8 * Cfg::NUM_BARRIERS;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(ctrl);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(ctrl + 4);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int pair_id = static_cast<int>(blockIdx.x >> 1);
    const int num_pairs = static_cast<int>(gridDim.x >> 1);
    const Trace tr(p.trace);

    if (threadIdx.x == 0) {
        tr.stamp(TR_START_NS);
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(accf_bar(b), 1); mbar_init(acce_bar(b), 8); }      // four epilogue warps in each CTA
        *abort_flag = 0u;
        fence_barrier_init();
        fence_proxy_async_smem();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(rank == 0 ? &tmB : (EPI == EPI_SWIGLU ? &tmB2 : &tmB));
        tma_prefetch_desc(&tmSFA);
        tma_prefetch_desc(&tmSFB);
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(tmem_slot)), Cfg::TMEM_COLS);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_arrive();
    cluster_wait();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_launch_dependents();
    pdl_wait();
    if (threadIdx.x == 0) tr.stamp(TR_SETUP_NS);

    if (warp == 0) {
        // ------------------------------------------------------------------ producer (both CTAs)
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            long long t_stall = 0;
            bool t_first = true;
            const uint32_t full0_base = cluster_map_shared(full_bar(0), 0);
            constexpr uint32_t cta_bytes = Cfg::A_BYTES + Cfg::B_BYTES + Cfg::SFA_BYTES + Cfg::SFB_BYTES;
            for (int t = pair_id; t < p.num_tiles && ok; t += num_pairs) {
                int mb, nb;
                tile_coords(p, t, mb, nb);
                const int m0 = mb * Cfg::BM + static_cast<int>(rank) * 128;
                // SwiGLU: rank 0 loads the gate rows, rank 1 the up rows of the tile's columns; otherwise the halves of the W rows
                const int n_row0 = nb * Cfg::OUT_TILE_N + ((EPI == EPI_SWIGLU) ? 0 : static_cast<int>(rank) * Cfg::HALF_ROWS);
                const CUtensorMap* mapB = (EPI == EPI_SWIGLU && rank == 1) ? &tmB2 : &tmB;
                const int m_block = mb * 2 + static_cast<int>(rank);          // this CTA's 128-row block of X scales
                for (int kb = 0; kb < p.k_blocks; kb += Cfg::KB_PER_STAGE) {
                    const int nsub = kb + 1 < p.k_blocks ? 2 : 1;        // an odd walk ends with half a stage
                    const long long tw = tr.now();
                    if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, p.status, STATUS_TIMEOUT_PRODUCER | 0xDu)) { ok = false; break; }
                    t_stall += tr.now() - tw;                 // trace totals live in registers and are written once, after the loop
                    if (t_first) { tr.stamp(TR_PROD_FIRST_NS); t_first = false; }
                    const uint32_t full0 = full0_base + 8u * s;
                    for (int j = 0; j < nsub; ++j) {
                        const uint32_t a_dst = base + s * Cfg::STAGE_BYTES + j * Cfg::SUB_BYTES;
                        tma_load_2d_pair(a_dst, &tmA, full0, (kb + j) * Cfg::BK, m0);
                        tma_load_2d_pair(a_dst + Cfg::A_BYTES, mapB, full0, (kb + j) * Cfg::BK, n_row0);
                        // scale blocks: rows of 256 bytes; block b starts at row 2 b (X: [k-block][row block]) or 4 b (W: [k-block][tile])
                        tma_load_2d_pair(a_dst + Cfg::SF_OFFSET, &tmSFA, full0, 0, 2 * ((kb + j) * (2 * p.m_tiles) + m_block));
                        tma_load_2d_pair(a_dst + Cfg::SF_OFFSET + Cfg::SFA_BYTES, &tmSFB, full0, 0, 4 * ((kb + j) * p.n_tiles + nb));
                    }
                    if (rank == 0) mbar_expect_tx(full_bar(s), 2u * cta_bytes * nsub);
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
            }
            tr.add(TR_PROD_STALL, t_stall);
            tr.stamp(TR_PROD_LAST_NS);
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ scale copies + MMA issue (even CTA)
        if (lane == 0 && rank == 0) {
            int s = 0;
            uint32_t ph = 0, acc_ph = 0;
            int it = 0;
            uint32_t stage_count = 0;
            bool ok = true;
            long long t_data = 0, t_head = 0, t_max = 0, t_acc = 0, t_kb = 0;      // trace totals (dead code without -DMTMC_TRACE)
            bool t_first = true;
            for (int t = pair_id; t < p.num_tiles && ok; t += num_pairs, ++it) {
                const int buf = it & 1;
                const long long ta = tr.now();
                if (!mbar_wait_cluster(acce_bar(buf), ((acc_ph >> buf) & 1u) ^ 1u, abort_flag, p.status, STATUS_TIMEOUT_MMA | 0xDu)) { ok = false; break; }
                t_acc += tr.now() - ta;
                acc_ph ^= 1u << buf;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(buf * Cfg::BN);
                for (int kb = 0; kb < p.k_blocks; kb += Cfg::KB_PER_STAGE) {
                    const int nsub = kb + 1 < p.k_blocks ? 2 : 1;
                    const long long tw = tr.now();
                    if (!mbar_wait(full_bar(s), ph, abort_flag, p.status, STATUS_TIMEOUT_MMA | 0xEu)) { ok = false; break; }
                    { const long long dw = tr.now() - tw; t_data += dw; t_max = dw > t_max ? dw : t_max; if (kb < STAGES * Cfg::KB_PER_STAGE) t_head += dw; }
                    t_kb += nsub;
                    if (t_first) { tr.stamp(TR_MMA_FIRST_NS); t_first = false; }
                    tc_fence_after();
                    for (int j = 0; j < nsub; ++j, ++stage_count) {
                        const uint32_t a_src = base + s * Cfg::STAGE_BYTES + j * Cfg::SUB_BYTES;
                        const uint32_t sf_src = a_src + Cfg::SF_OFFSET;
                        const uint64_t a_desc = umma_smem_desc_sw128(a_src);
                        const uint64_t b_desc = umma_smem_desc_sw128(a_src + Cfg::A_BYTES);
                        // the two sets of scale columns alternate by k-block: the copies of k-block i + 2 are issued after the MMAs of
                        // k-block i and run after them in the same pipe
                        const uint32_t sfa_tmem = tmem_base + static_cast<uint32_t>(Cfg::SF_COL0 + 12 * (stage_count & 1u));
                        const uint32_t sfb_tmem = sfa_tmem + 4u;
                        tmem_cp_scales_pair(sfa_tmem, umma_smem_desc_scales(sf_src));
                        tmem_cp_scales_pair(sfb_tmem, umma_smem_desc_scales(sf_src + Cfg::SFA_BYTES));
                        tmem_cp_scales_pair(sfb_tmem + 4u, umma_smem_desc_scales(sf_src + Cfg::SFA_BYTES + 512));
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            umma_mxf8_pair(d_tmem, a_desc + 2u * k, b_desc + 2u * k, umma_idesc_mxf8(Cfg::BM, Cfg::BN, k), sfa_tmem, sfb_tmem,
                                           (kb | j | k) != 0 ? 1u : 0u);
                    }
                    umma_commit_pair(empty_bar(s), 3);
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                if (ok) umma_commit_pair(accf_bar(buf), 3);
            }
            tr.add(TR_MMA_STALL_DATA, t_data); tr.add(TR_MMA_STALL_HEAD, t_head); tr.max(TR_MMA_STALL_MAX, t_max);
            tr.add(TR_MMA_STALL_ACC, t_acc); tr.add(TR_MMA_KBLOCKS, t_kb);
            tr.stamp(TR_MMA_LAST_NS);
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue (both CTAs)
        const int q = warp & 3;
        const uint32_t lane_base = static_cast<uint32_t>(q * 32) << 16;
        const bool vec_ok = OUT_BF16 ? (p.ldo % 8 == 0) : (p.ldo % 4 == 0);
        uint32_t acc_ph = 0;
        int it = 0;
        bool ok = true;
        for (int t = pair_id; t < p.num_tiles && ok; t += num_pairs, ++it) {
            const int buf = it & 1;
            int mb, nb;
            tile_coords(p, t, mb, nb);
            const int row = mb * Cfg::BM + static_cast<int>(rank) * 128 + q * 32 + lane;
            const bool tracer = warp == 2 && lane == 0;      // one writer for the epilogue's trace words
            const long long tw = tr.now();
            if (!mbar_wait(accf_bar(buf), (acc_ph >> buf) & 1u, abort_flag, p.status, STATUS_TIMEOUT_EPILOGUE | 0xDu)) { ok = false; break; }
            const long long tb = tr.now();
            if (tracer) { tr.add(TR_EPI_STALL, tb - tw); tr.add(TR_EPI_ITEMS, 1); tr.stamp_once(TR_EPI_FIRST_NS); }
            acc_ph ^= 1u << buf;
            tc_fence_after();
            const uint32_t t_addr = tmem_base + lane_base + static_cast<uint32_t>(buf * Cfg::BN);
            epilogue_item<EPI, OUT_BF16>(p, t_addr, row, nb * Cfg::OUT_TILE_N, 0, Cfg::OUT_TILE_N / 32, Cfg::OUT_TILE_N, nb, 0, 0, vec_ok,
                                         smem_raw + (epi_stage_base - raw_addr) + (warp - 2) * EPI_STAGE_BYTES_PER_WARP, lane);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_remote(cluster_map_shared(acce_bar(buf), 0));
            if (tracer) { tr.add(TR_EPI_BUSY, tr.now() - tb); tr.stamp(TR_EPI_END_NS); }
        }
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) tr.stamp(TR_END_NS);
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
