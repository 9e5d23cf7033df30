// Block-scaled 8-bit operands (MXFP8): E4M3 elements with one power-of-two scale (UE8M0: 2^(e-127)) per 32
// consecutive elements of K, for X and for W.  The scales cannot be folded into the epilogue like a per-tensor
// scale: they differ from k-block to k-block, so they have to be applied inside the contraction.  The tensor
// core does that itself (tcgen05.mma.kind::mxf8f6f4.block_scale): next to the operand tiles in shared memory it
// takes, per MMA of K = 32, one scale per accumulator row and one per accumulator column from tensor memory.
//
//   warp 0 (one lane)  producer: per ring stage (K = 128 elements = four MMAs) the X tile and the W tile by TMA
//                      (128-byte swizzle, as in the other kernels) and the two matching 512-byte blocks of scales
//                      by bulk copy.  The scales arrive pre-arranged (mx_retile_scales_kernel) as the block that
//                      tcgen05.cp moves in one go: 128 rows x 4 k-blocks, row r0 + 32 r1 at byte 16 r0 + 4 r1 + j.
//   warp 1 (one lane)  per stage: two tcgen05.cp (scales of X and of W, 32 rows x 128 bits broadcast to the four
//                      lane quadrants: four TMEM columns each), then four MMAs; MMA j picks byte j of each column
//                      through the scale ids of its instruction descriptor.  Copies and MMAs execute in issue order,
//                      and consecutive stages alternate between two sets of scale columns.
//   warps 2-5          the epilogues of gemm_tiled.cuh, unchanged (activation, SwiGLU gate, row logsumexp).
//
// Single-CTA tiles of 128 x 128 accumulator columns, two accumulator buffers (the epilogue of a tile runs under
// the next tile's mainloop); tensor memory: 256 columns of accumulators + 16 of scales.
#pragma once
#include "gemm_tiled.cuh"

namespace mtmc {

template <int EPI>
struct MxCfg {
    static constexpr int BM = 128;
    static constexpr int BN = 128;                        // accumulator columns (SwiGLU: 64 gate + 64 up)
    static constexpr int BK = 128;                        // E4M3 elements per ring stage: one 128-byte swizzle row, four MMAs of K = 32
    static constexpr int A_BYTES = BM * BK;
    static constexpr int B_BYTES = BN * BK;
    static constexpr int SF_BYTES = 512;                  // scales of 128 rows x 4 k-blocks
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES + 2 * SF_BYTES;      // 33 KiB: keeps every stage 1024-byte aligned
    static constexpr int STAGES = 6;
    static constexpr int OUT_TILE_N = (EPI == EPI_SWIGLU) ? BN / 2 : BN;
    static constexpr int ACC_COLS = 2 * BN;               // two accumulator buffers
    static constexpr int SF_COL0 = ACC_COLS;              // then 2 sets x (4 columns X scales + 4 columns W scales)
    static constexpr int TMEM_COLS = 512;                 // allocation sizes are powers of two
    static constexpr int NUM_BARRIERS = 2 * STAGES + 4;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 4 * EPI_STAGE_BYTES_PER_WARP + NUM_BARRIERS * 8 + 16 + 1024;
    static constexpr int THREADS = 192;
    static_assert(STAGE_BYTES % 1024 == 0 && SMEM_BYTES <= 227 * 1024, "ring stages stay 1024-byte aligned and fit");
    static_assert(EPI_HALVES == 1, "four epilogue warps");
};

// Shared-memory matrix descriptor of one block of scales: 32 rows of 16 bytes, rows 16 bytes apart, no swizzle
// (groups of eight rows follow each other at 128 bytes).
__device__ __forceinline__ uint64_t umma_smem_desc_scales(uint32_t saddr) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>(128 >> 4) << 32;      // stride byte offset between 8-row groups
    d |= static_cast<uint64_t>(1) << 46;             // descriptor version of sm_100
    return d;
}
// 32 rows x 128 bits from shared memory into four TMEM columns, the same 32 rows to each of the four lane quadrants.
__device__ __forceinline__ void tmem_cp_scales(uint32_t taddr, uint64_t sdesc) {
    asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
// Instruction descriptor of kind::mxf8f6f4 with E4M3 A and B (format code 0, both K-major), UE8M0 scales, fp32 D:
//   bits 4-5 B scale id, 17-22 N >> 3, 23 scale format (1 = UE8M0), 24-28 M >> 4, 29-30 A scale id.
// A scale id says which byte of the 32-bit scale columns this MMA uses: the k-block inside the stage.
__host__ __device__ constexpr uint32_t umma_idesc_mxf8(int m, int n, int scale_id) {
    return (static_cast<uint32_t>(scale_id) << 4) | (static_cast<uint32_t>(n >> 3) << 17) | (1u << 23) |
           (static_cast<uint32_t>(m >> 4) << 24) | (static_cast<uint32_t>(scale_id) << 29);
}
__device__ __forceinline__ void umma_mxf8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t sfa_tmem,
                                          uint32_t sfb_tmem, uint32_t accumulate) {
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale [%0], %1, %2, %3, [%5], [%6], p;\n\t"
        "}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem)
        : "memory");
}

// Re-arranges row-major scales S [rows, kb32] (one byte per row and 32 elements of K) into the blocks the kernels
// copy.  Output: [stage][block][atom] x 512 bytes, an atom holding 128 rows x 4 k-blocks with row r0 + 32 r1, k-block
// j at byte 16 r0 + 4 r1 + j; the neutral scale 127 (2^0) wherever the block has no row of S or K has ended.
//   S2 == null : block b holds rows [b * rows_per_block, (b + 1) * rows_per_block) of S in its first rows_per_block
//                rows (128 of one atom, or 224 of two atoms for the 224-column tiles of the CTA-pair kernel);
//   S2 != null : SwiGLU; rows_per_block rows of S (gate) followed by the same rows of S2 (up), the order of the
//                accumulator columns.
__global__ void mx_retile_scales_kernel(const uint8_t* __restrict__ S, const uint8_t* __restrict__ S2, int rows, int kb32,
                                        int blocks, int stages, int rows_per_block, int atoms, uint8_t* __restrict__ out) {
    const long long total = static_cast<long long>(stages) * blocks * atoms * 512;
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < total; i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int within = static_cast<int>(i & 511);
        const long long at = i >> 9;
        const int atom = static_cast<int>(at % atoms);
        const long long blk = at / atoms;
        const int block = static_cast<int>(blk % blocks), stage = static_cast<int>(blk / blocks);
        const int r0 = within >> 4, r1 = (within >> 2) & 3, j = within & 3;
        const int r = atom * 128 + r0 + 32 * r1;                      // row inside the block
        const uint8_t* src = S;
        int row;
        bool valid;
        if (S2 != nullptr) { src = r < rows_per_block ? S : S2; valid = r < 2 * rows_per_block; row = block * rows_per_block + (r % rows_per_block); }
        else { valid = r < rows_per_block; row = block * rows_per_block + r; }
        const int kb = stage * 4 + j;
        out[i] = (valid && row < rows && kb < kb32) ? src[static_cast<size_t>(row) * kb32 + kb] : static_cast<uint8_t>(127);
    }
}

template <int EPI, bool OUT_BF16>
__global__ void __launch_bounds__(192, 1)
gemm_mx_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmB2, const uint8_t* __restrict__ sfa, const uint8_t* __restrict__ sfb,
               const GemmParams p) {
    using Cfg = MxCfg<EPI>;
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

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(accf_bar(b), 1); mbar_init(acce_bar(b), 4); }
        *abort_flag = 0u;
        fence_barrier_init();
        fence_proxy_async_smem();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
        if (EPI == EPI_SWIGLU) tma_prefetch_desc(&tmB2);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), Cfg::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_launch_dependents();
    pdl_wait();

    const int n_blocks = p.n_tiles;                       // one block of W scales per column tile
    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            constexpr uint32_t b_half_bytes = static_cast<uint32_t>(Cfg::OUT_TILE_N) * Cfg::BK;     // one TMA box of W rows
            constexpr uint32_t tx = Cfg::STAGE_BYTES;
            for (int t = blockIdx.x; t < p.num_tiles && ok; t += gridDim.x) {
                int mb, nb;
                tile_coords(p, t, mb, nb);
                const int m0 = mb * Cfg::BM, n0 = nb * Cfg::OUT_TILE_N;
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, p.status, STATUS_TIMEOUT_PRODUCER | 0xBu)) { ok = false; break; }
                    const uint32_t a_dst = base + s * Cfg::STAGE_BYTES;
                    const uint32_t b_dst = a_dst + Cfg::A_BYTES;
                    const uint32_t sf_dst = b_dst + Cfg::B_BYTES;
                    mbar_expect_tx(full_bar(s), tx);
                    tma_load_2d(a_dst, &tmA, full_bar(s), kb * Cfg::BK, m0);
                    tma_load_2d(b_dst, &tmB, full_bar(s), kb * Cfg::BK, n0);
                    if (EPI == EPI_SWIGLU) tma_load_2d(b_dst + b_half_bytes, &tmB2, full_bar(s), kb * Cfg::BK, n0);
                    bulk_load_1d(sf_dst, sfa + (static_cast<size_t>(kb) * p.m_tiles + mb) * Cfg::SF_BYTES, Cfg::SF_BYTES, full_bar(s));
                    bulk_load_1d(sf_dst + Cfg::SF_BYTES, sfb + (static_cast<size_t>(kb) * n_blocks + nb) * Cfg::SF_BYTES, Cfg::SF_BYTES, full_bar(s));
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ scale copies + MMA issue
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0, acc_ph = 0;
            int it = 0;
            uint32_t stage_count = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < p.num_tiles && ok; t += gridDim.x, ++it) {
                const int buf = it & 1;
                if (!mbar_wait(acce_bar(buf), ((acc_ph >> buf) & 1u) ^ 1u, abort_flag, p.status, STATUS_TIMEOUT_MMA | 0xBu)) { ok = false; break; }
                acc_ph ^= 1u << buf;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(buf * Cfg::BN);
                for (int kb = 0; kb < p.k_blocks; ++kb, ++stage_count) {
                    if (!mbar_wait(full_bar(s), ph, abort_flag, p.status, STATUS_TIMEOUT_MMA | 0xCu)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_src = base + s * Cfg::STAGE_BYTES;
                    const uint32_t sf_src = a_src + Cfg::A_BYTES + Cfg::B_BYTES;
                    const uint64_t a_desc = umma_smem_desc_sw128(a_src);
                    const uint64_t b_desc = umma_smem_desc_sw128(a_src + Cfg::A_BYTES);
                    const uint32_t sfa_tmem = tmem_base + static_cast<uint32_t>(Cfg::SF_COL0 + 8 * (stage_count & 1u));
                    const uint32_t sfb_tmem = sfa_tmem + 4u;
                    tmem_cp_scales(sfa_tmem, umma_smem_desc_scales(sf_src));
                    tmem_cp_scales(sfb_tmem, umma_smem_desc_scales(sf_src + Cfg::SF_BYTES));
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        umma_mxf8(d_tmem, a_desc + 2u * k, b_desc + 2u * k, umma_idesc_mxf8(Cfg::BM, Cfg::BN, k), sfa_tmem, sfb_tmem,
                                  (kb | k) != 0 ? 1u : 0u);
                    umma_commit(empty_bar(s));      // frees the stage once the copies and MMAs have read it
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                if (ok) umma_commit(accf_bar(buf));
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue
        const int q = warp & 3;
        const uint32_t lane_base = static_cast<uint32_t>(q * 32) << 16;
        const bool vec_ok = OUT_BF16 ? (p.ldo % 8 == 0) : (p.ldo % 4 == 0);
        uint32_t acc_ph = 0;
        int it = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < p.num_tiles && ok; t += gridDim.x, ++it) {
            const int buf = it & 1;
            int mb, nb;
            tile_coords(p, t, mb, nb);
            const int row = mb * Cfg::BM + q * 32 + lane;
            if (!mbar_wait(accf_bar(buf), (acc_ph >> buf) & 1u, abort_flag, p.status, STATUS_TIMEOUT_EPILOGUE | 0xBu)) { ok = false; break; }
            acc_ph ^= 1u << buf;
            tc_fence_after();
            const uint32_t t_addr = tmem_base + lane_base + static_cast<uint32_t>(buf * Cfg::BN);
            epilogue_item<EPI, OUT_BF16>(p, t_addr, row, nb * Cfg::OUT_TILE_N, 0, Cfg::OUT_TILE_N / 32, Cfg::OUT_TILE_N, nb, 0, 0, vec_ok,
                                         smem_raw + (epi_stage_base - raw_addr) + (warp - 2) * EPI_STAGE_BYTES_PER_WARP, lane);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acce_bar(buf));
        }
    }

    // ---------------------------------------------------------------------- teardown
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
