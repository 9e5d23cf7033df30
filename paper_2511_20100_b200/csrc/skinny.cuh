// The skinny (decode-shaped, M <= 16) path: HBM-bound weight streaming with split-K.
//
// The roles are swapped relative to the tiled path ("swap-AB"): the TMEM lanes carry
// rows of W (output columns n), the MMA's N side carries the M <= 16 rows of X.
// W is cut into bands of tile_rows rows (a multiple of 8, at most 128; the MMA is
// always 128 lanes tall, lanes past tile_rows compute on stale shared memory and
// are never read).  Work is the flat list of (band, k-block) units, cut into one
// contiguous, equal share per CTA, so every SM streams the same number of weight
// bytes through a deep TMA ring.  A CTA whose share covers only part of a band's K
// range writes its fp32 partial [16 x 128] to the workspace and takes a ticket; the
// CTA that takes the band's last ticket adds the partials in slot order (so the
// result does not depend on arrival order), applies bias and activation and
// stores.  No CTA ever waits for another.
//
// PAIR mode (the common case: enough rows of W for half the SMs): the K range of every
// band is split over the two CTAs of a thread-block cluster.  The odd CTA sends its
// fp32 partial straight into the even CTA's shared memory (distributed shared memory
// stores + one remote mbarrier arrive); the even CTA adds it to its own registers
// (rank 0 + rank 1, always in that order), applies the epilogue and stores.  No
// global partials, no tickets, no fences to global memory.
//
// What bounds this kernel is per-stage and per-launch overhead, not arithmetic:
//  * a 128x16x16 MMA occupies the tensor pipe for about 70 clocks whatever N is, and
//    the issuing thread spends a few hundred clocks per pipeline hand-off, so one
//    ring stage carries KB_PER_STAGE k-blocks (2 x 16 KiB of W) per hand-off;
//  * k-steps are dealt round-robin onto WAYS independent accumulators;
//  * the producer starts its first loads before the rest of the CTA has finished
//    setting up, and the epilogue fetches its bias before the accumulator is ready.
#pragma once
#include "gemm_tiled.cuh"

namespace mtmc {

struct SkinnyParams {
    int M, N, K;
    int n_tiles, k_blocks;
    int tile_rows;           // W rows per band (multiple of 8, <= 128)
    int num_stages;          // TMA ring depth (<= SkinnyCfg<MX>::MAX_STAGES)
    long long total_units;   // n_tiles * k_blocks
    int max_slots;           // partial slots per band
    int act;
    float acc_scale;         // multiplies the accumulator before the bias (FP8 per-tensor scales; 1 otherwise)
    int early_w;             // 1: W is not written by any work still in flight, so its first ring of loads may
                             // go out before the wait on the preceding kernel (X, bias and outputs still wait)
    const float* bias;
    const void* residual;    // [M,N] in the output's element type, added after the activation, or null
    void* out;
    int ldo;                 // row pitch of out (and of the residual) in elements; N when dense
    float* partial;          // [n_tiles][max_slots][MX][128] fp32
    uint32_t* tickets;       // [n_tiles], zero between launches
    uint32_t* status;
    unsigned long long* trace;   // per-CTA trace records (-DMTMC_TRACE builds, mtmc_set_trace), else null
};

template <int MX_>
struct SkinnyCfg {
    static constexpr int LANES = 128;                     // MMA M = TMEM lanes
    static constexpr int MX = MX_;                        // X rows = MMA N: 16, 32 or 64
    static constexpr int BK = 64;                         // k-block: one 128-byte swizzle row
    static constexpr int KB_PER_STAGE = 2;                // k-blocks per ring stage
    static constexpr int X_BYTES = MX * BK * 2;           // 2 / 4 / 8 KiB per k-block
    static constexpr int MAX_STAGES = 16;
    static constexpr int WAYS = MX == 64 ? 4 : 8;         // independent accumulators
    static constexpr int ACC_COLS = WAYS * MX;            // TMEM columns per accumulator set (128 / 256 / 256)
    static constexpr int TMEM_COLS = 2 * ACC_COLS;        // two sets: MMA on one, epilogue on the other
    static constexpr int NUM_BARRIERS = 2 * MAX_STAGES + 6;   // ring, accumulator sets, pair reduction, store staging
    static constexpr int REDUCE_BYTES = MX * LANES * 4;       // the peer CTA's partial (PAIR mode)
    // One CTA per SM with the whole shared memory: splitting an SM between the running kernel and the next
    // launch (two CTAs of 111 KiB, dependents released after the last load) was measured slower, 28.7-29.2 us
    // against 26.8-27.4 us at 16 x 8192 x 8192, because the ring is then only three stages deep.
    static constexpr int RING_BYTES = 208 * 1024 - REDUCE_BYTES;   // shared memory given to the TMA ring
    static constexpr int SMEM_BYTES = RING_BYTES + REDUCE_BYTES + NUM_BARRIERS * 8 + 16 + 1024;
    static constexpr int stage_bytes(int tile_rows) { return KB_PER_STAGE * (tile_rows * BK * 2 + X_BYTES); }
    // The MMA always reads a 128-row (16 KiB) A tile, also when the band is shorter, so the last W
    // k-block of the last stage must start at least 16 KiB before the end of the ring.
    static constexpr int last_w_end(int tile_rows, int stages) {
        return (stages - 1) * stage_bytes(tile_rows) + (KB_PER_STAGE - 1) * tile_rows * BK * 2 + LANES * BK * 2;
    }
    static constexpr int stages_for(int tile_rows) {
        int s = RING_BYTES / stage_bytes(tile_rows);
        if (s > MAX_STAGES) s = MAX_STAGES;
        while (s > 1 && last_w_end(tile_rows, s) > RING_BYTES) --s;
        return s;
    }
};

// acc[m] += the accumulator ways that were written, in way order (TMEM -> registers).
template <int MX, int WAYS>
__device__ __forceinline__ void skinny_sum_ways(uint32_t set_addr, int ways_used, float (&acc)[MX]) {
#pragma unroll
    for (int l = 0; l < WAYS * MX / 32; ++l) {                // 32 TMEM columns per load
        const int first_way = (32 * l) / MX;
        if (first_way < ways_used) {                          // warp-uniform
            uint32_t r[32];
            tmem_ld_32x32b_x32(set_addr + 32 * l, r);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const int way = (32 * l + j) / MX;            // differs from first_way only when MX == 16
                if (MX >= 32 || way < ways_used) acc[(32 * l + j) % MX] += __uint_as_float(r[j]);
            }
        }
    }
}

__device__ __forceinline__ int skinny_cta_of_unit(long long u, long long total, int grid) {
    return static_cast<int>(((u + 1) * grid - 1) / total);
}

// Stores of one band.  The accumulator leaves the MMA transposed (a thread owns one output column n and all rows m),
// so a direct store would write one 2-byte element per thread and instruction.  Instead every thread parks its
// activated values in shared memory as stage[m][column in band] (fp32), the four epilogue warps meet on a
// bounded barrier, and then the 128 threads write the band row by row with 128-bit stores (eight bf16 or four
// fp32 per thread and instruction; the residual, if any, is read the same way and added here).  `stage` is the
// pair-reduction buffer, free again by now.  Returns false if the wait gave up.
template <bool OUT_BF16, int MX>
__device__ __forceinline__ bool skinny_store_band(const SkinnyParams& p, float* stage, uint32_t stage_bar, uint32_t& stage_phase,
                                                  volatile uint32_t* abort_flag, int nl, int epi_tid, int lane, int n_band0, int band_rows,
                                                  bool row_ok, const float (&y)[MX]) {
    if (row_ok) {
#pragma unroll
        for (int m = 0; m < MX; ++m) stage[m * 128 + nl] = y[m];
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(stage_bar);
    if (!mbar_wait(stage_bar, stage_phase, abort_flag, p.status, STATUS_TIMEOUT_EPILOGUE | 0xFu)) return false;
    stage_phase ^= 1u;
    constexpr int VEC = OUT_BF16 ? 8 : 4;                    // elements per 128-bit store
    constexpr int SEGS = 128 / VEC;
    const bool vec_ok = p.ldo % VEC == 0;                    // 16-byte aligned rows of out (and of the residual)
    const int cols = min(band_rows, p.N - n_band0);          // columns of this band inside the output
    for (int idx = epi_tid; idx < p.M * SEGS; idx += 128) {
        const int m = idx / SEGS, c0 = (idx - m * SEGS) * VEC;
        if (c0 >= cols) continue;
        const float* src = stage + m * 128 + c0;
        const size_t off = static_cast<size_t>(m) * p.ldo + n_band0 + c0;
        float v[VEC];
#pragma unroll
        for (int j = 0; j < VEC; j += 4) {
            const float4 t = *reinterpret_cast<const float4*>(src + j);
            v[j] = t.x; v[j + 1] = t.y; v[j + 2] = t.z; v[j + 3] = t.w;
        }
        if (vec_ok && c0 + VEC <= cols) {
            if (OUT_BF16) {
                if (p.residual) {
                    const uint4 r = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(p.residual) + off);
                    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
                    for (int h = 0; h < 4; ++h) { v[2 * h] += __uint_as_float(w[h] << 16); v[2 * h + 1] += __uint_as_float(w[h] & 0xffff0000u); }
                }
                uint4 q;
                q.x = pack_bf16x2(v[0], v[1]); q.y = pack_bf16x2(v[2], v[3]); q.z = pack_bf16x2(v[4 % VEC], v[5 % VEC]); q.w = pack_bf16x2(v[6 % VEC], v[7 % VEC]);
                *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.out) + off) = q;
            } else {
                if (p.residual) {
                    const float4 r = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(p.residual) + off);
                    v[0] += r.x; v[1] += r.y; v[2] += r.z; v[3] += r.w;
                }
                *reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + off) = make_float4(v[0], v[1], v[2], v[3]);
            }
        } else {
            for (int j = 0; j < VEC && c0 + j < cols; ++j) {
                float t = v[j];
                if (OUT_BF16) {
                    if (p.residual) t += __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p.residual)[off + j]);
                    reinterpret_cast<__nv_bfloat16*>(p.out)[off + j] = __float2bfloat16_rn(t);
                } else {
                    if (p.residual) t += reinterpret_cast<const float*>(p.residual)[off + j];
                    reinterpret_cast<float*>(p.out)[off + j] = t;
                }
            }
        }
    }
    return true;
}

// FP8: E4M3 operands (128 per 128-byte row, K = 32 per MMA) instead of bf16 (64 per row, K = 16);
// the bytes per stage, the ring and the four MMAs per row are the same for both.
template <bool OUT_BF16, bool PAIR, int MX, bool FP8 = false>
__global__ void __launch_bounds__(192, 1)
skinny_splitk_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX,
                     const SkinnyParams p) {
    using Cfg = SkinnyCfg<MX>;
    constexpr int BKE = FP8 ? 128 : 64;                      // elements of K per k-block
    constexpr int MAXS = Cfg::MAX_STAGES;
    constexpr int KPS = Cfg::KB_PER_STAGE;
    const int STAGES = p.num_stages;
    const int R = p.tile_rows;
    const uint32_t w_bytes = static_cast<uint32_t>(R) * Cfg::BK * 2;      // one W k-block; multiple of 1024
    const uint32_t x_off = KPS * w_bytes;                                  // X k-blocks follow the W k-blocks
    const uint32_t stage_bytes = KPS * (w_bytes + Cfg::X_BYTES);
    extern __shared__ uint8_t smem_raw[];

    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    const uint32_t reduce_base = base + Cfg::RING_BYTES;                  // [MX][128] fp32, written by the peer CTA
    const uint32_t bar_base = reduce_base + Cfg::REDUCE_BYTES;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (MAXS + s); };
    auto accf_bar = [&](int b) { return bar_base + 8u * (2 * MAXS + b); };
    auto acce_bar = [&](int b) { return bar_base + 8u * (2 * MAXS + 2 + b); };
    const uint32_t red_bar = bar_base + 8u * (2 * MAXS + 4);
    const uint32_t stage_bar = bar_base + 8u * (2 * MAXS + 5);             // the four epilogue warps have parked their values
    uint8_t* ctrl = smem_raw + (bar_base - raw_addr) + 8 * Cfg::NUM_BARRIERS;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(ctrl);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(ctrl + 4);
    volatile uint32_t* last_flag = reinterpret_cast<volatile uint32_t*>(ctrl + 8);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int KB = p.k_blocks;
    const Trace tr(p.trace);
    if (threadIdx.x == 0) tr.stamp(TR_START_NS);
    // This CTA's share of the unit list.
    int first_tile, first_kb, n_units;
    uint32_t crank = 0;
    if (PAIR) {
        // cluster of two: both CTAs work on band blockIdx.x / 2, each on one half of K
        crank = cluster_ctarank();
        const int half = (KB + 1) >> 1;
        first_tile = static_cast<int>(blockIdx.x >> 1);
        first_kb = crank ? half : 0;
        n_units = crank ? KB - half : half;
    } else {
        long long u_begin, u_end;
        if (p.total_units * gridDim.x < (1ll << 31)) {      // 32-bit arithmetic when it cannot overflow
            const uint32_t tot = static_cast<uint32_t>(p.total_units);
            u_begin = tot * blockIdx.x / gridDim.x;
            u_end = tot * (blockIdx.x + 1u) / gridDim.x;
        } else {
            u_begin = p.total_units * blockIdx.x / gridDim.x;
            u_end = p.total_units * (blockIdx.x + 1) / gridDim.x;
        }
        first_tile = static_cast<int>(u_begin / KB);
        first_kb = static_cast<int>(u_begin - static_cast<long long>(first_tile) * KB);
        n_units = static_cast<int>(u_end - u_begin);
    }

    // The TMA producer's walk over this CTA's k-blocks (one lane of warp 0 runs it).
    //   early = true : only the first ring-full of stages, only their W k-blocks (weights nobody is writing),
    //                  before the wait on the preceding kernel; each stage's full byte count is announced here.
    //   early = false: the whole walk; stages that the early pass already started get only their X k-blocks.
    auto produce = [&](bool early) {
        const uint64_t pol_stream = l2_policy_evict_first();   // W is read exactly once
        const uint64_t pol_keep = l2_policy_evict_last();      // X is re-read by every CTA
        const int pre = p.early_w ? STAGES : 0;                // stages begun by the early pass
        int s = 0, idx = 0;
        uint32_t ph = 0;
        int tile = first_tile, kb = first_kb, left = n_units;
        while (left > 0) {
            int seg = min(KB - kb, left);                      // k-blocks of this band still to load
            left -= seg;
            while (seg > 0) {
                if (early && idx >= pre) return;
                const int nkb = min(KPS, seg);
                const bool begun = !early && idx < pre;        // W already on its way, bytes already announced
                const uint32_t dst = base + s * stage_bytes;
                if (!begun) {
                    const long long tw = tr.now();
                    if (!early && !mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, p.status, STATUS_TIMEOUT_PRODUCER | 2u)) return;
                    tr.add(TR_PROD_STALL, tr.now() - tw);
                    tr.stamp_once(TR_PROD_FIRST_NS);
                    mbar_expect_tx(full_bar(s), nkb * (w_bytes + Cfg::X_BYTES));
                    for (int i = 0; i < nkb; ++i)
                        tma_load_2d_hint(dst + i * w_bytes, &tmW, full_bar(s), (kb + i) * BKE, tile * R, pol_stream);
                }
                if (!early) {
                    for (int i = 0; i < nkb; ++i)
                        tma_load_2d_hint(dst + x_off + i * Cfg::X_BYTES, &tmX, full_bar(s), (kb + i) * BKE, 0, pol_keep);
                }
                kb += nkb;
                seg -= nkb;
                ++idx;
                if (++s == STAGES) { s = 0; ph ^= 1u; }
            }
            ++tile;
            kb = 0;
        }
        if (!early) tr.stamp(TR_PROD_LAST_NS);
    };

    // Set-up.  Warp 0 initialises the barriers and goes straight on to issue loads; it only
    // arrives on the set-up barrier.  The other warps wait there for the barrier
    // initialisation and for warp 1's TMEM allocation.
    if (warp == 0) {
        if (lane == 0) {
            tma_prefetch_desc(&tmW);
            tma_prefetch_desc(&tmX);
            for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
            for (int b = 0; b < 2; ++b) { mbar_init(accf_bar(b), 1); mbar_init(acce_bar(b), 4); }
            mbar_init(red_bar, 4);
            mbar_init(stage_bar, 4);
            *abort_flag = 0u;
            *last_flag = 0u;
            fence_barrier_init();
            fence_proxy_async_smem();
        }
        __syncwarp();
        asm volatile("bar.arrive 2, 192;" ::: "memory");
        if (PAIR) cluster_arrive();          // publishes red_bar's initialisation to the peer; waited for at the end
        if (lane == 0 && p.early_w) produce(true);
        pdl_launch_dependents();
        pdl_wait();                          // before the first load of anything a preceding kernel may have written
        if (lane == 0) tr.stamp(TR_SETUP_NS);
    } else {
        if (warp == 1) {
            tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), Cfg::TMEM_COLS);
            tmem_relinquish();
            tc_fence_before();
        }
        asm volatile("bar.sync 2, 192;" ::: "memory");
        tc_fence_after();
        if (PAIR) cluster_arrive();          // after bar.sync: this CTA's barriers are initialised
        pdl_launch_dependents();
        pdl_wait();                          // before the first access to global memory
    }

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) produce(false);
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        const uint32_t tmem_base = *tmem_slot;
        if (lane == 0) {
            constexpr uint32_t idesc = FP8 ? umma_idesc_e4m3(Cfg::LANES, Cfg::MX) : umma_idesc_bf16(Cfg::LANES, Cfg::MX);
            int s = 0;
            uint32_t ph = 0, acc_ph = 0;                         // bit b of acc_ph: phase of accumulator set b
            int kb = first_kb, left = n_units, seg_idx = 0;
            bool ok = true;
            while (left > 0 && ok) {
                int seg = min(KB - kb, left);
                left -= seg;
                const int buf = seg_idx & 1;
                if (!mbar_wait(acce_bar(buf), ((acc_ph >> buf) & 1u) ^ 1u, abort_flag, p.status, STATUS_TIMEOUT_MMA | 3u)) { ok = false; break; }
                acc_ph ^= 1u << buf;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(buf * Cfg::ACC_COLS);
                uint32_t step = 0;                                // MMA count within this segment
                while (seg > 0) {
                    const int nkb = min(KPS, seg);
                    const long long tw = tr.now();
                    if (!mbar_wait(full_bar(s), ph, abort_flag, p.status, STATUS_TIMEOUT_MMA | 4u)) { ok = false; break; }
                    tr.add(TR_MMA_STALL_DATA, tr.now() - tw);
                    tr.add(TR_MMA_KBLOCKS, nkb);
                    tr.stamp_once(TR_MMA_FIRST_NS);
                    tc_fence_after();
                    const uint32_t src = base + s * stage_bytes;
                    for (int i = 0; i < nkb; ++i) {
                        const uint64_t a_desc = umma_smem_desc_sw128(src + i * w_bytes);
                        const uint64_t b_desc = umma_smem_desc_sw128(src + x_off + i * Cfg::X_BYTES);
#pragma unroll
                        for (int k = 0; k < Cfg::BK / 16; ++k, ++step) {      // four MMAs per 128-byte row either way
                            const uint32_t d = d_tmem + (step % Cfg::WAYS) * Cfg::MX;
                            if constexpr (FP8) umma_fp8(d, a_desc + 2u * k, b_desc + 2u * k, idesc, step >= Cfg::WAYS ? 1u : 0u);
                            else umma_bf16(d, a_desc + 2u * k, b_desc + 2u * k, idesc, step >= Cfg::WAYS ? 1u : 0u);
                        }
                    }
                    umma_commit(empty_bar(s));
                    seg -= nkb;
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                if (ok) umma_commit(accf_bar(buf));
                kb = 0;
                ++seg_idx;
            }
            tr.stamp(TR_MMA_LAST_NS);
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue / fix-up
        const uint32_t tmem_base = *tmem_slot;
        const int q = warp & 3;
        const int nl = q * 32 + lane;                 // row of W inside the band = TMEM lane
        const int epi_tid = (warp - 2) * 32 + lane;
        const uint32_t lane_base = static_cast<uint32_t>(q * 32) << 16;
        uint32_t acc_ph = 0;
        int tile = first_tile, kb0 = first_kb, left = n_units, seg_idx = 0;
        bool ok = true;
        float* stage = reinterpret_cast<float*>(smem_raw + (reduce_base - raw_addr));      // [MX][128] fp32: store staging
        uint32_t stage_phase = 0;
        if (PAIR) {
            left = 0;                                          // the generic loop below is not used
            const int n = first_tile * R + nl;
            const bool row_ok = nl < R && n < p.N;
            const float bn = (crank == 0 && row_ok && p.bias) ? __ldg(p.bias + n) : 0.0f;
            float acc[MX];
#pragma unroll
            for (int m = 0; m < MX; ++m) acc[m] = 0.0f;
            if (n_units > 0) ok = mbar_wait(accf_bar(0), 0u, abort_flag, p.status, STATUS_TIMEOUT_EPILOGUE | 3u);
            if (warp == 2 && lane == 0) tr.stamp(TR_EPI_FIRST_NS);
            if (ok && n_units > 0) {
                tc_fence_after();
                skinny_sum_ways<MX, Cfg::WAYS>(tmem_base + lane_base, min(Cfg::WAYS, n_units * (Cfg::BK / 16)), acc);
                tc_fence_before();
            }
            cluster_wait();                                    // set-up phase: the peer's barriers exist
            if (crank == 1) {
                // hand the partial to the even CTA: [m][lane] floats in its shared memory
                const uint32_t dst = cluster_map_shared(reduce_base, 0) + static_cast<uint32_t>(nl) * 4u;
#pragma unroll
                for (int m = 0; m < MX; ++m) st_shared_cluster_f32(dst + m * (Cfg::LANES * 4), ok ? acc[m] : 0.0f);
                fence_acq_rel_cluster();
                __syncwarp();
                if (lane == 0) mbar_arrive_remote(cluster_map_shared(red_bar, 0));
            } else if (ok) {
                if (mbar_wait_cluster(red_bar, 0u, abort_flag, p.status, STATUS_TIMEOUT_EPILOGUE | 4u)) {
                    const float* peer = reinterpret_cast<const float*>(smem_raw + (reduce_base - raw_addr)) + nl;
#pragma unroll
                    for (int m = 0; m < MX; ++m) acc[m] += peer[m * Cfg::LANES];       // rank 0 + rank 1
#pragma unroll
                    for (int m = 0; m < MX; ++m) acc[m] = apply_act(p.act, FP8 ? fmaf(acc[m], p.acc_scale, bn) : acc[m] + bn);
                    // (each thread overwrites, in the same buffer, exactly the elements it has just read)
                    skinny_store_band<OUT_BF16, MX>(p, stage, stage_bar, stage_phase, abort_flag, nl, epi_tid, lane, first_tile * R, R, row_ok, acc);
                }
            }
        }
        while (left > 0 && ok) {
            const int seg = min(KB - kb0, left);
            left -= seg;
            const int buf = seg_idx & 1;
            const int n = tile * R + nl;
            const bool row_ok = nl < R && n < p.N;
            // fetched before the accumulator is ready so that its latency is off the tail
            const float bn = (row_ok && p.bias) ? __ldg(p.bias + n) : 0.0f;
            if (!mbar_wait(accf_bar(buf), (acc_ph >> buf) & 1u, abort_flag, p.status, STATUS_TIMEOUT_EPILOGUE | 2u)) { ok = false; break; }
            acc_ph ^= 1u << buf;
            tc_fence_after();
            // Sum the accumulator ways that this segment wrote, in way order.
            float acc[MX];
#pragma unroll
            for (int m = 0; m < MX; ++m) acc[m] = 0.0f;
            skinny_sum_ways<MX, Cfg::WAYS>(tmem_base + lane_base + static_cast<uint32_t>(buf * Cfg::ACC_COLS),
                                           min(Cfg::WAYS, seg * (Cfg::BK / 16)), acc);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acce_bar(buf));     // registers hold the band: free the set now

            bool finalize = (seg == KB);                   // this CTA covered the band's whole K range
            if (!finalize) {
                const long long t_first = static_cast<long long>(tile) * KB;
                const int c_first = skinny_cta_of_unit(t_first, p.total_units, gridDim.x);
                const int c_last = skinny_cta_of_unit(t_first + KB - 1, p.total_units, gridDim.x);
                const int n_contrib = c_last - c_first + 1;
                const int slot = static_cast<int>(blockIdx.x) - c_first;
                float* band = p.partial + static_cast<size_t>(tile) * p.max_slots * (MX * 128) + nl;
                float* my = band + static_cast<size_t>(slot) * (MX * 128);
#pragma unroll
                for (int m = 0; m < MX; ++m) __stcg(my + m * 128, acc[m]);
                __threadfence();
                named_barrier_sync(1, 128);
                if (epi_tid == 0) {
                    const uint32_t old = atomicAdd(p.tickets + tile, 1u);
                    const uint32_t last = (old == static_cast<uint32_t>(n_contrib - 1)) ? 1u : 0u;
                    if (last) p.tickets[tile] = 0u;          // ready for the next launch
                    *last_flag = last;
                }
                named_barrier_sync(1, 128);
                if (*last_flag != 0u) {
                    __threadfence();
                    if (n_contrib == 2) {
                        // a + b == b + a exactly: adding the other CTA's partial to the registers gives
                        // the same bits whichever of the two arrives last
                        const float* other = band + static_cast<size_t>(1 - slot) * (MX * 128);
                        float o[MX];
#pragma unroll
                        for (int m = 0; m < MX; ++m) o[m] = __ldcg(other + m * 128);
#pragma unroll
                        for (int m = 0; m < MX; ++m) acc[m] += o[m];
                    } else {
#pragma unroll
                        for (int m = 0; m < MX; ++m) acc[m] = 0.0f;
                        for (int sl = 0; sl < n_contrib; ++sl) {             // slot order
                            float a0[MX];
#pragma unroll
                            for (int m = 0; m < MX; ++m) a0[m] = __ldcg(band + (static_cast<size_t>(sl) * MX + m) * 128);
#pragma unroll
                            for (int m = 0; m < MX; ++m) acc[m] += a0[m];
                        }
                    }
                    finalize = true;
                }
            }
            if (finalize) {                // the same decision in all four epilogue warps
#pragma unroll
                for (int m = 0; m < MX; ++m) acc[m] = apply_act(p.act, FP8 ? fmaf(acc[m], p.acc_scale, bn) : acc[m] + bn);
                if (!skinny_store_band<OUT_BF16, MX>(p, stage, stage_bar, stage_phase, abort_flag, nl, epi_tid, lane, tile * R, R, row_ok, acc)) { ok = false; break; }
                // the next band parks its values in the same buffer: everybody has read this one first
                __syncwarp();
                if (lane == 0) mbar_arrive(stage_bar);
                if (!mbar_wait(stage_bar, stage_phase, abort_flag, p.status, STATUS_TIMEOUT_EPILOGUE | 0xFu)) { ok = false; break; }
                stage_phase ^= 1u;
            }
            ++tile;
            kb0 = 0;
            ++seg_idx;
        }
    }

    if (warp == 2 && lane == 0) tr.stamp(TR_EPI_END_NS);
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) tr.stamp(TR_END_NS);
    if (PAIR) {
        // Neither CTA may leave while its peer can still write into (or arrive on) its shared
        // memory.  The epilogue warps consumed the set-up phase already; the others do it here.
        if (warp < 2) cluster_wait();
        cluster_arrive();
        cluster_wait();
    }
    if (*abort_flag != 0u) {
        const long long t0 = clock64();
        while (clock64() - t0 < 400000ll) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(*tmem_slot, Cfg::TMEM_COLS);
    }
}

}  // namespace mtmc
