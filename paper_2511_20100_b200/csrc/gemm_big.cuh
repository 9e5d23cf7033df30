// The tiled tensor-core path for large problems with a long K: CTA pairs on 512 x 256 tiles.
//
// gemm_pair.cuh gives each CTA 128 rows of a 256 x 256 pair tile and two accumulator buffers, so
// that a tile's epilogue runs under the next tile's mainloop; a k-block of 32 KiB feeds 512
// clocks of MMA (64 B of shared-memory fill per clock and SM).  Here each CTA owns 256 rows: per 64-wide
// k-block it loads 256 rows of X (32 KiB) and its half of the tile's W rows (16 KiB) and issues the
// MMAs of its two 128-row halves against the same W operand, so 48 KiB feed 1024 clocks of MMA
// (48 B per clock): a quarter less fill per FLOP, from shared memory and from L2.  The price: the
// two accumulators (2 x 256 columns) fill the tensor memory, so the epilogue cannot overlap the
// next tile's mainloop; eight epilogue warps (two per TMEM lane quadrant, one per row half) keep
// it short, and the producer refills the ring meanwhile.  Eight MMAs per wait and commit keep the
// issuing thread well ahead of the tensor pipe; it pays when the k-walk is long against the
// exposed epilogue (measured: from K = 16384 on).
//
// Barriers as in gemm_pair.cuh: all TMA bytes of a stage are counted on the even CTA's `full`
// barrier; tcgen05.commit with a cluster mask frees the stage in both CTAs and publishes the
// accumulators to both; the epilogue warps of both CTAs arrive on the even CTA's `accumulator
// empty` barrier.  No TMA load uses cluster multicast.  Whole tiles only (no tail pieces).
#pragma once
#include "gemm_tiled.cuh"

namespace mtmc {

template <int EPI>
struct BigCfg {
    static constexpr int BM = 512;                       // rows per pair tile (256 per CTA, as two halves of 128)
    static constexpr int BN = 256;                       // accumulator columns per half
    static constexpr int BK = 64;
    static constexpr int A_BYTES = 256 * BK * 2;         // this CTA's X rows: one box of 256 rows
    static constexpr int A_HALF_BYTES = 128 * BK * 2;
    static constexpr int B_BYTES = 128 * BK * 2;         // this CTA's half of the W rows
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int STAGES = 4;
    static constexpr int WARPS_EPI = 8;                  // quadrant = warp % 4, row half = (warp - 2) / 4
    static constexpr int OUT_TILE_N = (EPI == EPI_SWIGLU) ? BN / 2 : BN;
    static constexpr int TMEM_COLS = 2 * BN;             // the two row halves of one tile: all of tensor memory
    static constexpr int NUM_BARRIERS = 2 * STAGES + 3;  // ring, accumulator full, accumulator empty, bias copy written
    static constexpr bool STORES = (EPI == EPI_ACT || EPI == EPI_SWIGLU);
    // Store staging per epilogue warp: a 32 x 32 chunk, 2 KiB as bf16, 4 KiB as fp32.
    __host__ __device__ static constexpr int stage_bytes_per_warp(bool out_bf16) { return out_bf16 ? 2048 : 4096; }
    __host__ __device__ static constexpr int staging_bytes(bool out_bf16) { return STORES ? WARPS_EPI * stage_bytes_per_warp(out_bf16) : 0; }
    // Two copies of the tile's 256 bias values (the tile in its epilogue and the next one), where they fit:
    // not beside the fp32 store staging.
    static constexpr bool HAS_BIAS = (EPI != EPI_SWIGLU);
    __host__ __device__ static constexpr bool bias_in_smem(bool out_bf16) { return HAS_BIAS && (!STORES || out_bf16); }
    __host__ __device__ static constexpr int bias_bytes(bool out_bf16) { return bias_in_smem(out_bf16) ? 2 * BN * 4 : 0; }
    static constexpr int BIAS_OFFSET = (NUM_BARRIERS * 8 + 16 + 15) / 16 * 16;     // from the first barrier
    __host__ __device__ static constexpr int smem_bytes(bool out_bf16) {
        return STAGES * STAGE_BYTES + staging_bytes(out_bf16) + BIAS_OFFSET + bias_bytes(out_bf16) + 1024;
    }
    static constexpr int THREADS = 64 + 32 * WARPS_EPI;
    static_assert(smem_bytes(true) <= 227 * 1024 && smem_bytes(false) <= 227 * 1024, "shared memory per CTA");
    static_assert(EPI_HALVES == 1, "the epilogue's partial layout assumes one warp per quadrant and tile half");
};

template <int EPI, bool OUT_BF16>
__global__ void __launch_bounds__(64 + 32 * BigCfg<EPI>::WARPS_EPI, 1)
gemm_big_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                const __grid_constant__ CUtensorMap tmB2, const GemmParams p) {
    using Cfg = BigCfg<EPI>;
    constexpr int STAGES = Cfg::STAGES;
    extern __shared__ uint8_t smem_raw[];

    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    const uint32_t epi_stage_base = base + STAGES * Cfg::STAGE_BYTES;        // warp-private store staging
    const uint32_t bar_base = epi_stage_base + Cfg::staging_bytes(OUT_BF16);
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    const uint32_t accf_bar = bar_base + 8u * (2 * STAGES);
    const uint32_t acce_bar = bar_base + 8u * (2 * STAGES + 1);
    const uint32_t bias_bar = bar_base + 8u * (2 * STAGES + 2);      // every epilogue warp has written its part of the tile's bias
    uint8_t* ctrl = smem_raw + (bar_base - raw_addr) + 8 * Cfg::NUM_BARRIERS;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(ctrl);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(ctrl + 4);
    // [2][BN] floats if Cfg::bias_in_smem, read as float4: on the next 16-byte boundary after the control words
    float* bias_s = reinterpret_cast<float*>(smem_raw + (bar_base - raw_addr) + Cfg::BIAS_OFFSET);
    static_assert(Cfg::BIAS_OFFSET % 16 == 0 && Cfg::BIAS_OFFSET >= 8 * Cfg::NUM_BARRIERS + 16, "bias copy: aligned, after the control words");

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();            // 0: issues the MMAs, owns the shared barriers
    const int pair_id = static_cast<int>(blockIdx.x >> 1);
    const int num_pairs = static_cast<int>(gridDim.x >> 1);
    const Trace tr(p.trace);

    if (threadIdx.x == 0) {
        tr.stamp(TR_START_NS);
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(accf_bar, 1);
        mbar_init(acce_bar, 2 * Cfg::WARPS_EPI);         // every epilogue warp of both CTAs
        mbar_init(bias_bar, Cfg::WARPS_EPI);
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
    pdl_launch_dependents();
    pdl_wait();
    if (threadIdx.x == 0) tr.stamp(TR_SETUP_NS);

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            long long t_stall = 0;
            bool t_first = true;
            const uint32_t full0_base = cluster_map_shared(full_bar(0), 0);   // the even CTA's full barriers
            for (int t = pair_id; t < p.num_tiles && ok; t += num_pairs) {
                int mb, nb;
                tile_coords(p, t, mb, nb);
                const int m0 = mb * Cfg::BM + static_cast<int>(rank) * 256;
                // SwiGLU: rank 0 loads the gate rows, rank 1 the up rows of the tile's columns; otherwise the
                // first / second half of the tile's W rows.
                const int n_row0 = nb * Cfg::OUT_TILE_N + ((EPI == EPI_SWIGLU) ? 0 : static_cast<int>(rank) * 128);
                const CUtensorMap* mapB = (EPI == EPI_SWIGLU && rank == 1) ? &tmB2 : &tmB;
                int kx = 0;
                for (int kb = 0; kb < p.k_blocks; ++kb, kx += p.bk_elems) {
                    const long long tw = tr.now();
                    if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, p.status, STATUS_TIMEOUT_PRODUCER | 5u)) { ok = false; break; }
                    t_stall += tr.now() - tw;                 // trace totals live in registers and are written once, after the loop
                    if (t_first) { tr.stamp(TR_PROD_FIRST_NS); t_first = false; }
                    const uint32_t a_dst = base + s * Cfg::STAGE_BYTES;
                    const uint32_t full0 = full0_base + 8u * s;
                    tma_load_2d_pair(a_dst, &tmA, full0, kx, m0);
                    tma_load_2d_pair(a_dst + Cfg::A_BYTES, mapB, full0, kx, n_row0);
                    if (rank == 0) mbar_expect_tx(full_bar(s), 2u * Cfg::STAGE_BYTES);       // both CTAs' bytes
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
            }
            tr.add(TR_PROD_STALL, t_stall);
            tr.stamp(TR_PROD_LAST_NS);
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (even CTA only)
        if (lane == 0 && rank == 0) {
            int s = 0;
            uint32_t ph = 0, acc_ph = 0;
            bool ok = true;
            long long t_data = 0, t_head = 0, t_max = 0, t_acc = 0, t_kb = 0;      // trace totals (dead code without -DMTMC_TRACE)
            bool t_first = true;
            const uint32_t idesc = p.fp8 ? umma_idesc_e4m3(256, Cfg::BN) : umma_idesc_bf16(256, Cfg::BN);
            for (int t = pair_id; t < p.num_tiles && ok; t += num_pairs) {
                // the one accumulator set is free again once every epilogue warp of both CTAs has drained it
                const long long ta = tr.now();
                if (!mbar_wait_cluster(acce_bar, acc_ph ^ 1u, abort_flag, p.status, STATUS_TIMEOUT_MMA | 8u)) { ok = false; break; }
                t_acc += tr.now() - ta;
                acc_ph ^= 1u;
                tc_fence_after();
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    const long long tw = tr.now();
                    if (!mbar_wait(full_bar(s), ph, abort_flag, p.status, STATUS_TIMEOUT_MMA | 9u)) { ok = false; break; }
                    { const long long dw = tr.now() - tw; t_data += dw; t_max = dw > t_max ? dw : t_max; if (kb < STAGES) t_head += dw; }
                    ++t_kb;
                    if (t_first) { tr.stamp(TR_MMA_FIRST_NS); t_first = false; }
                    tc_fence_after();
                    const uint32_t a_src = base + s * Cfg::STAGE_BYTES;
                    const uint64_t b_desc = umma_smem_desc_sw128(a_src + Cfg::A_BYTES);
#pragma unroll
                    for (int h = 0; h < 2; ++h) {                // the two 128-row halves share the W operand
                        const uint64_t a_desc = umma_smem_desc_sw128(a_src + h * Cfg::A_HALF_BYTES);
                        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(h * Cfg::BN);
                        if (p.fp8) {
#pragma unroll
                            for (int k = 0; k < 4; ++k)
                                umma_fp8_pair(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, (kb | k) != 0 ? 1u : 0u);
                        } else {
#pragma unroll
                            for (int k = 0; k < 4; ++k)
                                umma_bf16_pair(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, (kb | k) != 0 ? 1u : 0u);
                        }
                    }
                    umma_commit_pair(empty_bar(s), 3);           // frees the stage in both CTAs
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                if (ok) umma_commit_pair(accf_bar, 3);           // both halves complete, in both CTAs
            }
            tr.add(TR_MMA_STALL_DATA, t_data); tr.add(TR_MMA_STALL_HEAD, t_head); tr.max(TR_MMA_STALL_MAX, t_max);
            tr.add(TR_MMA_STALL_ACC, t_acc); tr.add(TR_MMA_KBLOCKS, t_kb);
            tr.stamp(TR_MMA_LAST_NS);
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue (both CTAs, eight warps)
        const int q = warp & 3;                      // TMEM lane quadrant this warp may read
        const int hh = (warp - 2) >> 2;              // row half of the CTA's 256 rows = accumulator column block
        const uint32_t lane_base = static_cast<uint32_t>(q * 32) << 16;
        const uint32_t t_addr = tmem_base + lane_base + static_cast<uint32_t>(hh * Cfg::BN);
        const bool vec_ok = OUT_BF16 ? (p.ldo % 8 == 0) : (p.ldo % 4 == 0);
        constexpr bool BIAS_S = Cfg::bias_in_smem(OUT_BF16);
        const int et = static_cast<int>(threadIdx.x) - 64;       // 0 .. 255: this thread's column of the tile's bias
        uint32_t acc_ph = 0;
        bool ok = true;
        for (int t = pair_id; t < p.num_tiles && ok; t += num_pairs) {
            int mb, nb;
            tile_coords(p, t, mb, nb);
            const int row = mb * Cfg::BM + static_cast<int>(rank) * 256 + hh * 128 + q * 32 + lane;
            float* bias_tile = nullptr;
            if (BIAS_S) {
                // while the mainloop runs: the tile's bias into shared memory (the other copy may still be read by a
                // warp that is finishing the previous tile; nobody gets more than one tile ahead: the wait on `bias_bar`
                // below needs every warp's arrival for this tile)
                bias_tile = bias_s + acc_ph * Cfg::BN;
                const int n = nb * Cfg::OUT_TILE_N + et;
                bias_tile[et] = (p.bias != nullptr && n < p.N) ? __ldg(p.bias + n) : 0.0f;
                __syncwarp();
                if (lane == 0) mbar_arrive(bias_bar);
            }
            const bool tracer = warp == 2 && lane == 0;      // one writer for the epilogue's trace words
            const long long tw = tr.now();
            if (!mbar_wait(accf_bar, acc_ph, abort_flag, p.status, STATUS_TIMEOUT_EPILOGUE | 6u)) { ok = false; break; }
            const long long tb = tr.now();
            if (tracer) { tr.add(TR_EPI_STALL, tb - tw); tr.add(TR_EPI_ITEMS, 1); tr.stamp_once(TR_EPI_FIRST_NS); }
            acc_ph ^= 1u;
            tc_fence_after();
            // the other warps' parts of the bias copy (an mbarrier, so that this wait is bounded like every other)
            if (BIAS_S && !mbar_wait(bias_bar, acc_ph ^ 1u, abort_flag, p.status, STATUS_TIMEOUT_EPILOGUE | 0xAu)) { ok = false; break; }
            epilogue_item<EPI, OUT_BF16>(p, t_addr, row, nb * Cfg::OUT_TILE_N, 0, Cfg::OUT_TILE_N / 32, Cfg::OUT_TILE_N, nb, 0, 0, vec_ok,
                                         smem_raw + (epi_stage_base - raw_addr) + (warp - 2) * Cfg::stage_bytes_per_warp(OUT_BF16), lane,
                                         bias_tile);
            // this warp's share of the accumulators is drained: tell the MMA issuer in the even CTA
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_remote(cluster_map_shared(acce_bar, 0));
            if (tracer) { tr.add(TR_EPI_BUSY, tr.now() - tb); tr.stamp(TR_EPI_END_NS); }
        }
    }

    // ---------------------------------------------------------------------- teardown
    // Neither CTA may free its TMEM or leave while the other can still touch its memory or barriers.
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
