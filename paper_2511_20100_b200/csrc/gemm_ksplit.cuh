// Split-K over a thread-block cluster, for problems with far fewer output tiles than SMs
// (decode / small-prefill batches of 65 ... a few hundred rows against a large weight matrix).
//
// There the tiled kernels leave most SMs idle and every busy CTA walks the whole K range, so
// the time is one CTA's k-walk.  Here a cluster of KS CTAs (2, 4 or 8) owns one 128 x 256 tile:
// CTA r multiplies k-blocks [r KB/KS, (r+1) KB/KS) into its own TMEM accumulator (the same
// TMA ring and tcgen05 mainloop as the tiled kernel), then the cluster does a reduce-scatter
// through distributed shared memory: CTA r receives, from every peer, the peer's partial of
// the 256 / KS accumulator columns that r will finish, adds the KS partials in rank order
// (so the bits do not depend on timing), writes the sum back to its TMEM and runs the usual
// epilogue on its columns.  The partials never touch L2 or HBM and the epilogue is shared
// out over the cluster as well.
//
// The receive buffer is the CTA's TMA ring, idle once its last MMA has completed; a CTA tells
// its peers so (remote arrive on their `ready` barrier) and sends only when every peer is
// ready.  All waits are on CTAs of the same cluster, which the hardware schedules together,
// and all are bounded.
#pragma once
#include "gemm_tiled.cuh"

namespace mtmc {

template <int EPI, int KS, int BN_ = 256>
struct KSplitCfg {
    static_assert(KS == 2 || KS == 4 || KS == 8, "cluster of two, four or eight CTAs (eight: not for SwiGLU, whose tile has four output chunks)");
    static_assert(BN_ == 256 || (BN_ == 128 && KS <= 4 && EPI != EPI_SWIGLU), "128-column tiles: four accumulator chunks, clusters of two or four");
    using Tile = TileCfg<EPI, BN_>;
    static constexpr int BN = BN_;
    // 128-column tiles: twice the tiles, so half the cluster size for the same number of CTAs and a third of the
    // bytes to exchange (a CTA of a cluster of two sends 32 KiB where one of a cluster of four sends 96 KiB); each CTA
    // then walks twice as many, half as heavy k-blocks, and its ring is handed over two k-blocks at a time so that the
    // thread that issues the MMAs keeps ahead of the weight stream (three stages of 2 x 32 KiB).
    static constexpr int KB_PER_STAGE = BN_ == 128 ? 2 : 1;
    static constexpr int SUB_BYTES = Tile::STAGE_BYTES;   // one k-block: X rows, then W rows
    static constexpr int STAGES = Tile::STAGES / KB_PER_STAGE;
    static constexpr int STAGE_BYTES = KB_PER_STAGE * SUB_BYTES;
    static constexpr int OUT_TILE_N = Tile::OUT_TILE_N;
    static constexpr int AC = BN / 32;                    // 32-column chunks of the accumulator
    static constexpr int OC = OUT_TILE_N / 32;            // 32-column chunks of the output tile (SwiGLU: half of AC)
    static constexpr int OWN_OC = OC / KS;                // output chunks this CTA finishes
    static constexpr int OWN_AC = AC / KS;                // accumulator chunks it receives from each peer
    static constexpr int BLOCK_BYTES = 32 * 32 * 4;       // one chunk of one lane quadrant: 32 rows x 128 bytes
    static constexpr int RECV_BYTES = (KS - 1) * OWN_AC * 4 * BLOCK_BYTES;
    static_assert(RECV_BYTES <= STAGES * STAGE_BYTES, "the ring holds the peers' partials");
    // Clusters of two and four send their parts as bulk copies from a staging area behind the receive area (the
    // per-thread stores into a peer's shared memory run at about 16 bytes per cycle and CTA); a cluster of eight
    // would need 2 x 112 KiB for that and keeps the stores.
    static constexpr bool BULK = 2 * RECV_BYTES <= STAGES * STAGE_BYTES;
    static_assert(OWN_OC >= 1, "at least one output chunk per CTA");
    static constexpr int NUM_BARRIERS = 2 * STAGES + 3;   // ring, accumulator full, ready, received
    // Epilogue warps: two per TMEM lane quadrant where the epilogue stores a tile (they share the exchange, the sums and
    // the output chunks: the exchange is the exposed tail of a launch whose CTAs have one work item each); one per
    // quadrant for the row reductions, whose partial per row has one writer.
    static constexpr int EPI_W = (EPI == EPI_ACT || EPI == EPI_SWIGLU) ? 8 : 4;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_W * EPI_STAGE_BYTES_PER_WARP + NUM_BARRIERS * 8 + 16 + 1024;
    static constexpr int THREADS = 64 + 32 * EPI_W;       // producer, MMA issuer, epilogue warps
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory per CTA");
    static constexpr int TMEM_COLS = BN;                  // one accumulator: a CTA has exactly one work item
};

__device__ __forceinline__ void st_shared_cluster_v4(uint32_t caddr, float a, float b, float c, float d) {
    asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(caddr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

template <int EPI, bool OUT_BF16, int KS, int BN = 256>
__global__ void __launch_bounds__(64 + 32 * KSplitCfg<EPI, KS, BN>::EPI_W, 1)
gemm_ksplit_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                   const __grid_constant__ CUtensorMap tmB2, const GemmParams p) {
    using Cfg = KSplitCfg<EPI, KS, BN>;
    using Tile = typename Cfg::Tile;
    constexpr int STAGES = Cfg::STAGES;
    extern __shared__ uint8_t smem_raw[];

    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    const uint32_t epi_stage_base = base + STAGES * Cfg::STAGE_BYTES;
    const uint32_t bar_base = epi_stage_base + Cfg::EPI_W * EPI_STAGE_BYTES_PER_WARP;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    const uint32_t accf_bar = bar_base + 8u * (2 * STAGES);
    const uint32_t ready_bar = bar_base + 8u * (2 * STAGES + 1);      // peers that are ready to receive (their ring is idle)
    const uint32_t recv_bar = bar_base + 8u * (2 * STAGES + 2);       // peers' epilogue warps that have delivered to me
    uint8_t* ctrl = smem_raw + (bar_base - raw_addr) + 8 * Cfg::NUM_BARRIERS;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(ctrl);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(ctrl + 4);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int tile = static_cast<int>(blockIdx.x) / KS;
    const Trace tr(p.trace);

    if (threadIdx.x == 0) {
        tr.stamp(TR_START_NS);
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(accf_bar, 1);
        mbar_init(ready_bar, KS - 1);             // one arrival per peer CTA
        mbar_init(recv_bar, Cfg::BULK ? 1 : (KS - 1) * Cfg::EPI_W);   // bulk copies count bytes; else one arrival per epilogue warp of every peer
        *abort_flag = 0u;
        fence_barrier_init();
        fence_proxy_async_smem();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
        if (EPI == EPI_SWIGLU) tma_prefetch_desc(&tmB2);
        // Static weights: the W loads of the first ring go out now, before the cluster has met and before the wait on the
        // preceding kernel -- they touch only this CTA's shared memory and barriers, which this thread has just initialised,
        // and memory that nothing in flight writes.  The producer loop below adds the X loads of those stages.
        if (p.early_w) {
            int mb_e, nb_e;
            tile_coords(p, tile, mb_e, nb_e);
            const int kb0_e = static_cast<int>(static_cast<long long>(rank) * p.k_blocks / KS);
            const int kb1_e = static_cast<int>(static_cast<long long>(rank + 1) * p.k_blocks / KS);
            constexpr uint32_t b_rows_bytes_e = static_cast<uint32_t>(Cfg::OUT_TILE_N) * Tile::BK * 2;
            constexpr uint32_t tx_e = Tile::A_BYTES + (EPI == EPI_SWIGLU ? 2u : 1u) * b_rows_bytes_e;
            int s = 0;
            for (int kb = kb0_e; kb < kb1_e && s < STAGES; kb += Cfg::KB_PER_STAGE, ++s) {
                const int nsub = (Cfg::KB_PER_STAGE == 2 && kb + 1 < kb1_e) ? 2 : 1;
                mbar_expect_tx(full_bar(s), tx_e * nsub);
                for (int j = 0; j < nsub; ++j) {
                    const uint32_t b_dst = base + s * Cfg::STAGE_BYTES + j * Cfg::SUB_BYTES + Tile::A_BYTES;
                    tma_load_2d(b_dst, &tmB, full_bar(s), (kb + j) * p.bk_elems, nb_e * Cfg::OUT_TILE_N);
                    if (EPI == EPI_SWIGLU) tma_load_2d(b_dst + b_rows_bytes_e, &tmB2, full_bar(s), (kb + j) * p.bk_elems, nb_e * Cfg::OUT_TILE_N);
                }
            }
        }
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), Cfg::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    cluster_arrive();        // every CTA's barriers exist before any peer arrives on them
    cluster_wait();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_launch_dependents();
    pdl_wait();
    if (threadIdx.x == 0) tr.stamp(TR_SETUP_NS);

    int mb, nb;
    tile_coords(p, tile, mb, nb);
    const int kb0 = static_cast<int>(static_cast<long long>(rank) * p.k_blocks / KS);
    const int kb1 = static_cast<int>(static_cast<long long>(rank + 1) * p.k_blocks / KS);

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0;
            const int m0 = mb * 128;
            const int n0 = nb * Cfg::OUT_TILE_N;
            constexpr uint32_t b_rows_bytes = static_cast<uint32_t>(Cfg::OUT_TILE_N) * Tile::BK * 2;
            constexpr uint32_t tx = Tile::A_BYTES + (EPI == EPI_SWIGLU ? 2u : 1u) * b_rows_bytes;
            int begun = p.early_w ? STAGES : 0;          // stages whose bytes are announced and whose W loads are on their way
            for (int kb = kb0; kb < kb1; kb += Cfg::KB_PER_STAGE) {
                const int nsub = (Cfg::KB_PER_STAGE == 2 && kb + 1 < kb1) ? 2 : 1;      // an odd walk ends with half a stage
                const bool early = begun > 0;
                if (early) --begun;
                const long long tw = tr.now();
                if (!early && !mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, p.status, STATUS_TIMEOUT_PRODUCER | 7u)) break;
                tr.add(TR_PROD_STALL, tr.now() - tw);
                tr.stamp_once(TR_PROD_FIRST_NS);
                if (!early) mbar_expect_tx(full_bar(s), tx * nsub);
                for (int j = 0; j < nsub; ++j) {
                    const uint32_t a_dst = base + s * Cfg::STAGE_BYTES + j * Cfg::SUB_BYTES;
                    const uint32_t b_dst = a_dst + Tile::A_BYTES;
                    tma_load_2d(a_dst, &tmA, full_bar(s), (kb + j) * p.bk_elems, m0);
                    if (!early) {
                        tma_load_2d(b_dst, &tmB, full_bar(s), (kb + j) * p.bk_elems, n0);
                        if (EPI == EPI_SWIGLU) tma_load_2d(b_dst + b_rows_bytes, &tmB2, full_bar(s), (kb + j) * p.bk_elems, n0);
                    }
                }
                if (++s == STAGES) { s = 0; ph ^= 1u; }
            }
            tr.stamp(TR_PROD_LAST_NS);
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            const uint32_t idesc = p.fp8 ? umma_idesc_e4m3(128, Cfg::BN) : umma_idesc_bf16(128, Cfg::BN);
            for (int kb = kb0; kb < kb1; kb += Cfg::KB_PER_STAGE) {
                const int nsub = (Cfg::KB_PER_STAGE == 2 && kb + 1 < kb1) ? 2 : 1;
                const long long tw = tr.now();
                if (!mbar_wait(full_bar(s), ph, abort_flag, p.status, STATUS_TIMEOUT_MMA | 7u)) { ok = false; break; }
                tr.add(TR_MMA_STALL_DATA, tr.now() - tw);
                tr.add(TR_MMA_KBLOCKS, nsub);
                tr.stamp_once(TR_MMA_FIRST_NS);
                tc_fence_after();
#pragma unroll
                for (int j = 0; j < Cfg::KB_PER_STAGE; ++j) {
                    if (j < nsub) {
                        const uint32_t a_src = base + s * Cfg::STAGE_BYTES + j * Cfg::SUB_BYTES;
                        const uint64_t a_desc = umma_smem_desc_sw128(a_src);
                        const uint64_t b_desc = umma_smem_desc_sw128(a_src + Tile::A_BYTES);
                        if (p.fp8) {
#pragma unroll
                            for (int k = 0; k < 4; ++k)
                                umma_fp8(tmem_base, a_desc + 2u * k, b_desc + 2u * k, idesc, ((kb - kb0) | j | k) != 0 ? 1u : 0u);
                        } else {
#pragma unroll
                            for (int k = 0; k < 4; ++k)
                                umma_bf16(tmem_base, a_desc + 2u * k, b_desc + 2u * k, idesc, ((kb - kb0) | j | k) != 0 ? 1u : 0u);
                        }
                    }
                }
                umma_commit(empty_bar(s));
                if (++s == STAGES) { s = 0; ph ^= 1u; }
            }
            if (ok) umma_commit(accf_bar);           // my part of the sum is complete and my ring is idle
            tr.stamp(TR_MMA_LAST_NS);
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ reduce-scatter + epilogue
        const int q = warp & 3;                      // TMEM lane quadrant this warp may read
        const int half = (warp - 2) >> 2;            // which of the quadrant's (one or two) warps this is
        constexpr int HALVES = Cfg::EPI_W / 4;
        const uint32_t lane_base = static_cast<uint32_t>(q * 32) << 16;
        const uint32_t t_addr = tmem_base + lane_base;
        const bool vec_ok = OUT_BF16 ? (p.ldo % 8 == 0) : (p.ldo % 4 == 0);
        // Accumulator chunk held at place `loc` of the receive buffer of CTA `owner`: output chunk
        // owner * OWN_OC + loc % OWN_OC of the gate / only half (loc < OWN_OC) or of the up half.
        auto acc_chunk = [&](int owner, int loc) { return (loc / Cfg::OWN_OC) * Cfg::OC + owner * Cfg::OWN_OC + loc % Cfg::OWN_OC; };
        const bool tracer = warp == 2 && lane == 0;
        bool ok = mbar_wait(accf_bar, 0u, abort_flag, p.status, STATUS_TIMEOUT_EPILOGUE | 7u);
        const long long tb = tr.now();
        if (tracer) { tr.stamp(TR_EPI_FIRST_NS); tr.add(TR_EPI_ITEMS, 1); }
        if (ok) {
            tc_fence_after();
            if (Cfg::BULK && warp == 2 && lane == 0) mbar_expect_tx(recv_bar, Cfg::RECV_BYTES);      // what the peers will copy in
            // my ring is idle (every MMA that read it has completed): the peers may write their partials into it
            if (warp == 2 && lane < KS && lane != static_cast<int>(rank)) mbar_arrive_remote(cluster_map_shared(ready_bar, lane));
            ok = mbar_wait_cluster(ready_bar, 0u, abort_flag, p.status, STATUS_TIMEOUT_EPILOGUE | 8u);
        }
        long long tx = tr.now();
        if (tracer) tr.add(TR_XCHG_READY, tx - tb);
        if (ok) {
            // Everything this warp owes its peers goes out first (the TMEM load of the next chunk in flight while one
            // chunk is stored), then ONE fence orders all of it, then the peers are told: a fence per peer would
            // cost a round trip through the cluster each.
            constexpr int SENDS = (KS - 1) * Cfg::OWN_AC;
            // the quadrant's warps share the chunks: the first takes [0, ceil(SENDS / HALVES)), the second the rest
            const int s_begin = HALVES == 2 && half ? (SENDS + 1) / 2 : 0;
            const int s_end = HALVES == 2 && !half ? (SENDS + 1) / 2 : SENDS;
            auto chunk_of = [&](int idx) { return acc_chunk((static_cast<int>(rank) + 1 + idx / Cfg::OWN_AC) % KS, idx % Cfg::OWN_AC); };
            uint32_t r[32];
            if (s_begin < s_end) tmem_ld_32x32b_x32(t_addr + chunk_of(s_begin) * 32, r);
#pragma unroll 1
            for (int idx = s_begin; idx < s_end; ++idx) {
                const int peer = (static_cast<int>(rank) + 1 + idx / Cfg::OWN_AC) % KS;
                const int loc = idx % Cfg::OWN_AC;
                const int sidx = static_cast<int>(rank) < peer ? static_cast<int>(rank) : static_cast<int>(rank) - 1;   // my place among the peer's senders
                tmem_ld_wait();
                float v[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
                if (idx + 1 < s_end) tmem_ld_32x32b_x32(t_addr + chunk_of(idx + 1) * 32, r);
                // the reader is the thread at the same place (quadrant, lane) of the peer, so the layout inside the 4 KiB
                // block is private to the two: each store instruction of the warp writes 512 contiguous bytes
                const uint32_t slot = static_cast<uint32_t>(((sidx * Cfg::OWN_AC + loc) * 4 + q) * Cfg::BLOCK_BYTES);
                if constexpr (Cfg::BULK) {
                    // park the chunk in this CTA's staging area (behind the receive area), then one bulk copy moves it
                    const uint32_t src = base + Cfg::RECV_BYTES + static_cast<uint32_t>((idx * 4 + q) * Cfg::BLOCK_BYTES);
#pragma unroll
                    for (int g = 0; g < 8; ++g)
                        asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(src + g * 512 + lane * 16), "f"(v[4 * g]), "f"(v[4 * g + 1]),
                                     "f"(v[4 * g + 2]), "f"(v[4 * g + 3]) : "memory");
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) bulk_copy_to_peer(cluster_map_shared(base, peer) + slot, src, Cfg::BLOCK_BYTES, cluster_map_shared(recv_bar, peer));
                } else {
                    const uint32_t dst = cluster_map_shared(base, peer) + slot + lane * 16;
#pragma unroll
                    for (int g = 0; g < 8; ++g)
                        st_shared_cluster_v4(dst + g * 512, v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
                }
            }
            if constexpr (!Cfg::BULK) {
                fence_acq_rel_cluster();
                __syncwarp();
                if (lane < KS && lane != static_cast<int>(rank)) mbar_arrive_remote(cluster_map_shared(recv_bar, lane));
            }
            if (tracer) { const long long t1 = tr.now(); tr.add(TR_XCHG_SEND, t1 - tx); tx = t1; }
            ok = mbar_wait_cluster(recv_bar, 0u, abort_flag, p.status, STATUS_TIMEOUT_EPILOGUE | 9u);
            if (tracer) { const long long t1 = tr.now(); tr.add(TR_XCHG_RECV, t1 - tx); tx = t1; }
        }
        // The output chunks this warp finishes: its CTA's OWN_OC chunks, shared between the quadrant's warps.
        const int j_begin = HALVES == 2 && half ? (Cfg::OWN_OC + 1) / 2 : 0;
        const int j_end = HALVES == 2 && !half ? (Cfg::OWN_OC + 1) / 2 : Cfg::OWN_OC;
        if (ok && j_begin < j_end) {
            // sum of the KS partials of those columns (SwiGLU: of their gate and of their up columns), in rank order,
            // back into TMEM
#pragma unroll 1
            for (int part = 0; part < Cfg::OWN_AC / Cfg::OWN_OC; ++part) {
#pragma unroll 1
            for (int j = j_begin; j < j_end; ++j) {
                const int loc = part * Cfg::OWN_OC + j;
                const int a = acc_chunk(static_cast<int>(rank), loc);
                uint32_t r[32];
                tmem_ld_32x32b_x32(t_addr + a * 32, r);
                tmem_ld_wait();
                float acc[32];
#pragma unroll
                for (int s = 0; s < KS; ++s) {
                    if (s == static_cast<int>(rank)) {
#pragma unroll
                        for (int jj = 0; jj < 32; ++jj) acc[jj] = (s == 0) ? __uint_as_float(r[jj]) : acc[jj] + __uint_as_float(r[jj]);
                    } else {
                        const int sidx = s < static_cast<int>(rank) ? s : s - 1;
                        const uint32_t src = base + static_cast<uint32_t>(((sidx * Cfg::OWN_AC + loc) * 4 + q) * Cfg::BLOCK_BYTES + lane * 16);
#pragma unroll
                        for (int g = 0; g < 8; ++g) {
                            const float4 t = ld_shared_v4(src + g * 512);
                            acc[4 * g] = (s == 0) ? t.x : acc[4 * g] + t.x;
                            acc[4 * g + 1] = (s == 0) ? t.y : acc[4 * g + 1] + t.y;
                            acc[4 * g + 2] = (s == 0) ? t.z : acc[4 * g + 2] + t.z;
                            acc[4 * g + 3] = (s == 0) ? t.w : acc[4 * g + 3] + t.w;
                        }
                    }
                }
#pragma unroll
                for (int jj = 0; jj < 32; ++jj) r[jj] = __float_as_uint(acc[jj]);
                tmem_st_32x32b_x32(t_addr + a * 32, r);
            }
            }
            tmem_st_wait();
            if (tracer) { tr.add(TR_XCHG_SUM, tr.now() - tx); tr.add(TR_EPI_HANDOVER, tr.now() - tb); }        // reduce-scatter through distributed shared memory
            const int row = mb * 128 + q * 32 + lane;
            epilogue_item<EPI, OUT_BF16>(p, t_addr, row, nb * Cfg::OUT_TILE_N, static_cast<int>(rank) * Cfg::OWN_OC + j_begin,
                                         static_cast<int>(rank) * Cfg::OWN_OC + j_end, Cfg::OUT_TILE_N, nb, static_cast<int>(rank), 0, vec_ok,
                                         smem_raw + (epi_stage_base - raw_addr) + (warp - 2) * EPI_STAGE_BYTES_PER_WARP, lane);
        }
        if (tracer) { tr.add(TR_EPI_BUSY, tr.now() - tb); tr.stamp(TR_EPI_END_NS); }
    }

    // ---------------------------------------------------------------------- teardown
    // No CTA frees its TMEM or leaves while a peer can still write into its ring or arrive on its barriers.
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
        tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
    }
}

}  // namespace mtmc
