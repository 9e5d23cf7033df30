// The skinny (decode-shaped, M <= 16) path: HBM-bound weight streaming with split-K.
//
// The roles are swapped relative to the tiled path ("swap-AB"): the 128 TMEM lanes
// carry 128 rows of W (output columns n), the MMA's N side carries the M <= 16
// rows of X.  Work is the flat list of (n-tile, k-block) units, cut into one
// contiguous, equal share per CTA (stream-K), so every SM streams the same number
// of weight bytes through a deep TMA ring.  A CTA whose share covers only part of
// a tile's K range writes its fp32 partial [16 x 128] to the workspace and takes a
// ticket; the CTA that takes the last ticket of a tile adds the partials in slot
// order (so the result does not depend on arrival order), applies bias and
// activation and stores.  No CTA ever waits for another.
#pragma once
#include "gemm_tiled.cuh"

namespace mtmc {

struct SkinnyParams {
    int M, N, K;
    int n_tiles, k_blocks;
    long long total_units;   // n_tiles * k_blocks
    int max_slots;           // partial slots per tile
    int act;
    const float* bias;
    void* out;
    float* partial;          // [n_tiles][max_slots][16][128] fp32
    uint32_t* tickets;       // [n_tiles], zero between launches
    uint32_t* status;
};

struct SkinnyCfg {
    static constexpr int BNW = 128;                       // W rows per tile = TMEM lanes
    static constexpr int MX = 16;                         // X rows = MMA N
    static constexpr int BK = 64;
    static constexpr int W_BYTES = BNW * BK * 2;          // 16 KiB
    static constexpr int X_BYTES = MX * BK * 2;           // 2 KiB
    static constexpr int STAGE_BYTES = W_BYTES + X_BYTES;
    static constexpr int STAGES = 11;
    static constexpr int TMEM_COLS = 64;                  // two 32-column accumulator buffers
    static constexpr int NUM_BARRIERS = 2 * STAGES + 4;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + NUM_BARRIERS * 8 + 16 + 1024;
};

__device__ __forceinline__ int skinny_cta_of_unit(long long u, long long total, int grid) {
    return static_cast<int>(((u + 1) * grid - 1) / total);
}

template <bool OUT_BF16>
__global__ void __launch_bounds__(192, 1)
skinny_splitk_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX,
                     const SkinnyParams p) {
    using Cfg = SkinnyCfg;
    constexpr int STAGES = Cfg::STAGES;
    extern __shared__ uint8_t smem_raw[];

    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    const uint32_t bar_base = base + STAGES * Cfg::STAGE_BYTES;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto accf_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + b); };
    auto acce_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + 2 + b); };
    uint8_t* ctrl = smem_raw + (bar_base - raw_addr) + 8 * Cfg::NUM_BARRIERS;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(ctrl);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(ctrl + 4);
    volatile uint32_t* last_flag = reinterpret_cast<volatile uint32_t*>(ctrl + 8);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int KB = p.k_blocks;
    const long long u_begin = p.total_units * blockIdx.x / gridDim.x;
    const long long u_end = p.total_units * (blockIdx.x + 1) / gridDim.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(accf_bar(b), 1); mbar_init(acce_bar(b), 4); }
        *abort_flag = 0u;
        *last_flag = 0u;
        fence_barrier_init();
        fence_proxy_async_smem();
        tma_prefetch_desc(&tmW);
        tma_prefetch_desc(&tmX);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), Cfg::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const uint64_t pol_stream = l2_policy_evict_first();   // W is read exactly once
            const uint64_t pol_keep = l2_policy_evict_last();      // X is re-read by every CTA
            int s = 0;
            uint32_t ph = 0;
            for (long long u = u_begin; u < u_end; ++u) {
                const int tile = static_cast<int>(u / KB);
                const int kb = static_cast<int>(u - static_cast<long long>(tile) * KB);
                if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, p.status, STATUS_TIMEOUT_PRODUCER | 2u)) break;
                const uint32_t w_dst = base + s * Cfg::STAGE_BYTES;
                mbar_expect_tx(full_bar(s), Cfg::STAGE_BYTES);
                tma_load_2d_hint(w_dst, &tmW, full_bar(s), kb * Cfg::BK, tile * Cfg::BNW, pol_stream);
                tma_load_2d_hint(w_dst + Cfg::W_BYTES, &tmX, full_bar(s), kb * Cfg::BK, 0, pol_keep);
                if (++s == STAGES) { s = 0; ph ^= 1u; }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(Cfg::BNW, Cfg::MX);
            int s = 0;
            uint32_t ph = 0;
            uint32_t acc_ph[2] = {0u, 0u};
            int seg = 0;
            bool ok = true;
            for (long long u = u_begin; u < u_end && ok; ++seg) {
                const int tile = static_cast<int>(u / KB);
                const int kb0 = static_cast<int>(u - static_cast<long long>(tile) * KB);
                const int kb1 = static_cast<int>(min(static_cast<long long>(KB), kb0 + (u_end - u)));
                const int buf = seg & 1;
                if (!mbar_wait(acce_bar(buf), acc_ph[buf] ^ 1u, abort_flag, p.status, STATUS_TIMEOUT_MMA | 3u)) { ok = false; break; }
                acc_ph[buf] ^= 1u;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(buf * 32);
                for (int kb = kb0; kb < kb1; ++kb) {
                    if (!mbar_wait(full_bar(s), ph, abort_flag, p.status, STATUS_TIMEOUT_MMA | 4u)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t w_src = base + s * Cfg::STAGE_BYTES;
                    const uint64_t a_desc = umma_smem_desc_sw128(w_src);
                    const uint64_t b_desc = umma_smem_desc_sw128(w_src + Cfg::W_BYTES);
#pragma unroll
                    for (int k = 0; k < Cfg::BK / 16; ++k)
                        umma_bf16(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, (kb > kb0 || k > 0) ? 1u : 0u);
                    umma_commit(empty_bar(s));
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                if (ok) umma_commit(accf_bar(buf));
                u += kb1 - kb0;
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue / fix-up
        const int q = warp & 3;
        const int nl = q * 32 + lane;                 // row of W inside the tile = TMEM lane
        const int epi_tid = (warp - 2) * 32 + lane;
        const uint32_t lane_base = static_cast<uint32_t>(q * 32) << 16;
        uint32_t acc_ph[2] = {0u, 0u};
        int seg = 0;
        bool ok = true;
        for (long long u = u_begin; u < u_end && ok; ++seg) {
            const int tile = static_cast<int>(u / KB);
            const int kb0 = static_cast<int>(u - static_cast<long long>(tile) * KB);
            const int kb1 = static_cast<int>(min(static_cast<long long>(KB), kb0 + (u_end - u)));
            const int buf = seg & 1;
            if (!mbar_wait(accf_bar(buf), acc_ph[buf], abort_flag, p.status, STATUS_TIMEOUT_EPILOGUE | 2u)) { ok = false; break; }
            acc_ph[buf] ^= 1u;
            tc_fence_after();
            uint32_t r[16];
            tmem_ld_32x32b_x16(tmem_base + lane_base + static_cast<uint32_t>(buf * 32), r);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acce_bar(buf));     // registers hold the tile: free the buffer now

            float acc[16];
#pragma unroll
            for (int m = 0; m < 16; ++m) acc[m] = __uint_as_float(r[m]);

            bool finalize = (kb0 == 0 && kb1 == KB);       // this CTA covered the tile's whole K range
            if (!finalize) {
                const long long t_first = static_cast<long long>(tile) * KB;
                const int c_first = skinny_cta_of_unit(t_first, p.total_units, gridDim.x);
                const int c_last = skinny_cta_of_unit(t_first + KB - 1, p.total_units, gridDim.x);
                const int n_contrib = c_last - c_first + 1;
                const int slot = static_cast<int>(blockIdx.x) - c_first;
                float* my = p.partial + (static_cast<size_t>(tile) * p.max_slots + slot) * (16 * 128) + nl;
#pragma unroll
                for (int m = 0; m < 16; ++m) __stcg(my + m * 128, acc[m]);
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
                    const float* src = p.partial + static_cast<size_t>(tile) * p.max_slots * (16 * 128) + nl;
#pragma unroll
                    for (int m = 0; m < 16; ++m) acc[m] = 0.0f;
                    for (int sl = 0; sl < n_contrib; ++sl) {
#pragma unroll
                        for (int m = 0; m < 16; ++m) acc[m] += __ldcg(src + (static_cast<size_t>(sl) * 16 + m) * 128);
                    }
                    finalize = true;
                }
            }
            if (finalize) {
                const int n = tile * Cfg::BNW + nl;
                if (n < p.N) {
                    const float bn = p.bias ? __ldg(p.bias + n) : 0.0f;
#pragma unroll
                    for (int m = 0; m < 16; ++m) {
                        if (m < p.M) {
                            const float y = apply_act(p.act, acc[m] + bn);
                            if (OUT_BF16)
                                reinterpret_cast<__nv_bfloat16*>(p.out)[static_cast<size_t>(m) * p.N + n] = __float2bfloat16_rn(y);
                            else
                                reinterpret_cast<float*>(p.out)[static_cast<size_t>(m) * p.N + n] = y;
                        }
                    }
                }
            }
            u += kb1 - kb0;
        }
    }

    tc_fence_before();
    __syncthreads();
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
