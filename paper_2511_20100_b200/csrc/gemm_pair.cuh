// The tiled tensor-core path for large problems: CTA pairs (thread-block clusters of two).
//
// A pair owns a 256 x 256 output tile (256 x 128 for SwiGLU).  Each CTA loads its own 128
// rows of X and its own half of the W rows of the tile, so a k-block is 32 KiB instead of
// 48 KiB (a ring of six k-blocks, handed to the MMA issuer two at a time and back to the producer one by one, instead of four) and a third less L2 -> shared-memory traffic per
// FLOP.  The even CTA issues tcgen05.mma.cta_group::2 (M = 256) for both; each CTA keeps the
// accumulator of its own 128 rows in its own TMEM and runs its own epilogue.
//
// Barriers: all TMA bytes of a stage (both CTAs') are counted on the even CTA's `full`
// barrier; tcgen05.commit with a cluster mask frees the stage in both CTAs and publishes
// the accumulator to both; the epilogue warps of both CTAs arrive on the even CTA's
// `accumulator empty` barrier.  No TMA load uses cluster multicast.
//
// Stream-K schedule (GemmParams::sk).  Whole tiles dealt round-robin leave the last wave partly empty (3.46
// waves of tiles cost 4 tile-times) and a problem of fewer tiles than pairs leaves pairs idle while the others
// walk all of K.  With this schedule the full waves but one are dealt round-robin as before (pairs that run
// together work on neighbouring tiles and share operands in L2), and the rest -- the last full wave plus the
// remainder, or everything when there is less than a wave -- is dealt by k-blocks: the flat list of that region's
// (tile, k-block) units is cut into one contiguous, equal share per pair, so all pairs stream the same number of
// operand bytes and finish together.  A tile whose k-blocks straddle shares has several holders (consecutive
// pairs).  They meet without waiting for one another: each epilogue warp that finishes its part either finds
// all other holders' parts already in global memory, adds them to its accumulator in holder order and runs the
// ordinary epilogue, or leaves its own part there, counts itself in on the tile's ticket word and moves on.  A
// pair works on its pieces of shared tiles first and on its whole tiles after them, so the hand-overs run under
// the mainloop of the tiles that follow.
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
    // A ring stage carries two k-blocks.  The thread that issues the MMAs pays a fixed price per stage (the wait for
    // the stage's data, the commit that frees it) on top of the MMAs themselves, and with one k-block per stage that
    // thread, not the tensor pipe, set the pace: about 700 cycles per k-block against 512 of MMA.
    static constexpr int KB_PER_STAGE = 2;
    static constexpr int SUB_BYTES = A_BYTES + B_BYTES;  // one k-block: this CTA's X rows, then its W rows
    static constexpr int STAGE_BYTES = KB_PER_STAGE * SUB_BYTES;
    static constexpr int STAGES = 3;
    static constexpr int OUT_TILE_N = (EPI == EPI_SWIGLU) ? BN / 2 : BN;
    static constexpr int TMEM_COLS = 2 * BN;
    static constexpr int NUM_BARRIERS = STAGES + KB_PER_STAGE * STAGES + 4;   // full per stage, empty per k-block, accumulators
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_WARPS * EPI_STAGE_BYTES_PER_WARP + NUM_BARRIERS * 8 + 16 + 1024;
    static constexpr int THREADS = 64 + 32 * EPI_WARPS;
};

// One work item of a pair: a whole tile or tail piece (part < 0), or k-blocks [kb0, kb1) of a tile that this pair
// shares with its neighbours under the stream-K schedule (part 0 or 1: which of the pair's two part buffers).
struct PairWork {
    int item, kb0, kb1;
    int part;
};

// Owner of unit x when `total` units are cut into `pairs` contiguous shares [total*p/pairs, total*(p+1)/pairs).
__device__ __forceinline__ int streamk_owner(long long x, long long total, int pairs) {
    return static_cast<int>(((x + 1) * pairs - 1) / total);
}

struct PairWalk {
    int u, dp_end, step;                   // round-robin part: next item, end, stride
    int KB, sk_first;
    int t0, a, t1, b;                      // stream-K share: from k-block a of region tile t0 to k-block b (exclusive) of region tile t1
    int whole, whole_end;                  // whole tiles of the share still to hand out
    int phase;                             // 0 round-robin, 1 first piece, 2 last piece, 3 whole tiles
    bool sk;
    __device__ __forceinline__ PairWalk(const GemmParams& p, int pair, int num_pairs) {
        KB = p.k_blocks; step = num_pairs; sk = p.sk != 0;
        u = pair;
        dp_end = sk ? p.sk_first_tile : p.num_items;
        sk_first = p.sk_first_tile;
        phase = 0;
        t0 = t1 = a = b = 0; whole = whole_end = 0;
        if (sk) {
            const long long U = static_cast<long long>(p.num_items - p.sk_first_tile) * KB;
            const long long su = U * pair / num_pairs, su_end = U * (pair + 1) / num_pairs;
            if (su_end > su) {
                t0 = static_cast<int>(su / KB); a = static_cast<int>(su - static_cast<long long>(t0) * KB);
                t1 = static_cast<int>((su_end - 1) / KB); b = static_cast<int>(su_end - static_cast<long long>(t1) * KB);
                whole = a > 0 ? t0 + 1 : t0;
                whole_end = b < KB ? t1 : t1 + 1;
            } else {
                phase = 4;                 // more pairs than k-blocks: nothing for this one
                sk = false; dp_end = 0;
            }
        }
    }
    // Order inside the share: its pieces of shared tiles first, then its whole tiles, so that the hand-overs (and,
    // where this pair is the last holder to arrive, the tile's completion) run under the mainloop of what follows
    // instead of after the last MMA of the launch.
    __device__ __forceinline__ bool next(PairWork& w) {
        if (phase == 0) {
            if (u < dp_end) { w.item = u; w.kb0 = 0; w.kb1 = KB; w.part = -1; u += step; return true; }
            phase = sk ? 1 : 4;
        }
        if (phase == 1) {
            phase = 2;
            if (a > 0 || (t0 == t1 && b < KB)) {      // the share begins inside tile t0 (or lies inside it altogether)
                w.item = sk_first + t0; w.kb0 = a; w.kb1 = t0 == t1 ? b : KB; w.part = 0;
                return true;
            }
        }
        if (phase == 2) {
            phase = 3;
            if (t1 > t0 && b < KB) { w.item = sk_first + t1; w.kb0 = 0; w.kb1 = b; w.part = 1; return true; }
        }
        if (phase == 3 && whole < whole_end) { w.item = sk_first + whole; w.kb0 = 0; w.kb1 = KB; w.part = -1; ++whole; return true; }
        return false;
    }
};

// Stream-K hand-over for one epilogue warp (CTA `rank` of the pair, TMEM lane quadrant q) whose accumulator holds
// the sum over part of a shared tile's K range.  The holders of a tile are the consecutive pairs whose shares
// meet its k-blocks.  Nobody waits: a warp that finds all other holders' parts in global memory adds them to its
// accumulator, in holder order, and returns true (its accumulator in tensor memory then holds the whole sum and the
// ordinary epilogue follows); otherwise it leaves its own part, counts itself in and returns false.  The sum is
// always formed in holder order, so the bits do not depend on who arrives last.
template <int BN>
__device__ __forceinline__ bool streamk_meet(const GemmParams& p, const PairWork& w, uint32_t t_addr, int pair_id, int num_pairs,
                                             int rank, int q, int lane) {
    constexpr int CHUNKS = BN / 32;
    constexpr size_t WARP_F4 = static_cast<size_t>(CHUNKS) * 8 * 32;           // float4 per warp and part
    const int KB = p.k_blocks;
    const int tt = w.item - p.sk_first_tile;                                   // tile index inside the stream-K region
    const long long U = static_cast<long long>(p.num_items - p.sk_first_tile) * KB;
    const int h_first = streamk_owner(static_cast<long long>(tt) * KB, U, num_pairs);
    const int h_last = streamk_owner(static_cast<long long>(tt + 1) * KB - 1, U, num_pairs);
    const uint32_t holders = static_cast<uint32_t>(h_last - h_first + 1);
    if (!MTMC_CHECK(tt >= 0 && h_first <= pair_id && pair_id <= h_last && holders >= 2u && holders < 256u && (w.part == 0 || w.part == 1),
                    p.status, 3u))
        return false;
    auto part_of = [&](int holder, int which) {
        return p.sk_partial + (((static_cast<size_t>(holder) * 2 + which) * 2 + rank) * 4 + q) * WARP_F4;
    };
    // which of its two part buffers a holder uses for this tile: 0 if its share begins in this tile, else 1
    auto which_of = [&](int holder) { return static_cast<int>((U * holder / num_pairs) / KB) == tt ? 0 : 1; };
    uint32_t* ticket = p.sk_flags + (static_cast<size_t>(tt) * 2 + rank) * 4 + q;
    // ticket word: launch epoch in the upper 24 bits (a word left by an earlier launch counts as zero), arrivals below
    uint32_t seen = 0;
    if (lane == 0) seen = ld_acquire_gpu(ticket);
    seen = __shfl_sync(0xffffffffu, seen, 0);
    uint32_t arrived = (seen >> 8) == p.sk_epoch ? (seen & 0xffu) : 0u;
    if (arrived + 1u < holders) {
        // not everybody else has been here: leave this part (every store instruction of the warp writes 512
        // contiguous bytes; the reader is the thread at the same place of another pair, so the layout is private)
        float4* mine = part_of(pair_id, w.part);
#pragma unroll 1
        for (int c = 0; c < CHUNKS; ++c) {
            uint32_t r[32];
            tmem_ld_32x32b_x32(t_addr + c * 32, r);
            tmem_ld_wait();
#pragma unroll
            for (int v = 0; v < 8; ++v)
                __stcg(mine + (c * 8 + v) * 32 + lane, make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]),
                                                                   __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3])));
        }
        __threadfence();
        __syncwarp();
        if (lane == 0) {
            uint32_t old = seen, now;
            for (;;) {                                       // arrivals + 1 under this launch's epoch (a handful of contenders at most)
                now = (old >> 8) == p.sk_epoch ? old + 1u : ((p.sk_epoch << 8) | 1u);
                const uint32_t prev = atomicCAS(ticket, old, now);
                if (prev == old) break;
                old = prev;
            }
            seen = now;
        }
        seen = __shfl_sync(0xffffffffu, seen, 0);
        arrived = seen & 0xffu;
        if (arrived < holders) return false;                 // somebody is still to come: the last one finishes the tile
    }
    __threadfence();                                         // the other parts were complete before their holders counted themselves in
    // The sum in holder order, chunk by chunk: the other holders' parts from L2 (all loads of a chunk in flight
    // together), this pair's own from tensor memory at its place in the order; back to tensor memory.
#pragma unroll 1
    for (int c = 0; c < CHUNKS; ++c) {
        uint32_t r[32];
        tmem_ld_32x32b_x32(t_addr + c * 32, r);
        float acc[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) acc[j] = 0.0f;          // 0 + x == x: the sum below is part(first) + part(next) + ...
        for (int h = h_first; h <= h_last; ++h) {
            if (h == pair_id) {
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; ++j) acc[j] += __uint_as_float(r[j]);
            } else {
                const float4* src = part_of(h, which_of(h)) + c * 8 * 32 + lane;
                float4 o[8];
#pragma unroll
                for (int v = 0; v < 8; ++v) o[v] = __ldcg(src + v * 32);
#pragma unroll
                for (int v = 0; v < 8; ++v) {
                    acc[4 * v] += o[v].x; acc[4 * v + 1] += o[v].y; acc[4 * v + 2] += o[v].z; acc[4 * v + 3] += o[v].w;
                }
            }
        }
#pragma unroll
        for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(acc[j]);
        tmem_st_32x32b_x32(t_addr + c * 32, r);
    }
    tmem_st_wait();
    return true;
}

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
    // a stage's two k-blocks are handed to the MMA issuer together (one `full` barrier, two arrivals) but handed back
    // one by one (an `empty` barrier each): the first is refilled while the second is still being multiplied
    auto empty_bar = [&](int s, int j) { return bar_base + 8u * (STAGES + Cfg::KB_PER_STAGE * s + j); };
    auto accf_bar = [&](int b) { return bar_base + 8u * ((1 + Cfg::KB_PER_STAGE) * STAGES + b); };
    auto acce_bar = [&](int b) { return bar_base + 8u * ((1 + Cfg::KB_PER_STAGE) * STAGES + 2 + b); };
    uint8_t* ctrl = smem_raw + (bar_base - raw_addr) + 8 * Cfg::NUM_BARRIERS;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(ctrl);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(ctrl + 4);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();            // 0: issues the MMAs, owns the shared barriers
    const int pair_id = static_cast<int>(blockIdx.x >> 1);
    const int num_pairs = static_cast<int>(gridDim.x >> 1);
    const Trace tr(p.trace);

    if (threadIdx.x == 0) {
        tr.stamp(TR_START_NS);
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar(s), Cfg::KB_PER_STAGE);           // one arrival (with its bytes) per k-block
            for (int j = 0; j < Cfg::KB_PER_STAGE; ++j) mbar_init(empty_bar(s, j), 1);
        }
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
            PairWalk walk(p, pair_id, num_pairs);
            PairWork w;
            while (ok && walk.next(w)) {
                int mb, nb, sub, width;
                item_coords(p, w.item, Cfg::OUT_TILE_N, mb, nb, sub, width);
                const bool whole = width == Cfg::OUT_TILE_N;
                const int m0 = mb * Cfg::BM + static_cast<int>(rank) * 128;
                // This CTA's share of the B operand: SwiGLU -> rank 0 the gate rows, rank 1 the up rows of
                // the same columns; otherwise the first / second half of the item's W rows.
                const int b_rows = (EPI == EPI_SWIGLU) ? width : width / 2;
                const int n_row0 = nb * Cfg::OUT_TILE_N + sub * width + ((EPI == EPI_SWIGLU) ? 0 : static_cast<int>(rank) * b_rows);
                const CUtensorMap* mapB = (EPI == EPI_SWIGLU && rank == 1) ? (whole ? &tmB2 : &tmB2t) : (whole ? &tmB : &tmBt);
                const uint32_t cta_bytes = Cfg::A_BYTES + static_cast<uint32_t>(b_rows) * Cfg::BK * 2;
                int kx = w.kb0 * p.bk_elems;                             // K coordinate of the next k-block
                for (int kb = w.kb0; kb < w.kb1; kb += Cfg::KB_PER_STAGE, kx += Cfg::KB_PER_STAGE * p.bk_elems) {
                    const bool two = kb + 1 < w.kb1;                     // an odd walk ends with half a stage
                    const uint32_t full0 = full0_base + 8u * s;
#pragma unroll
                    for (int j = 0; j < Cfg::KB_PER_STAGE; ++j) {
                        const long long tw = tr.now();
                        if (!mbar_wait(empty_bar(s, j), ph ^ 1u, abort_flag, p.status, STATUS_TIMEOUT_PRODUCER | 3u)) { ok = false; break; }
                        t_stall += tr.now() - tw;                 // trace totals live in registers and are written once, after the loop
                        if (t_first) { tr.stamp(TR_PROD_FIRST_NS); t_first = false; }
                        if (j == 0 || two) {
                            // loads first, bookkeeping after: the time from "slot free" to "load issued" is on the ring's
                            // critical path (a transaction count may run ahead of its expect_tx within a phase)
                            const uint32_t a_dst = base + s * Cfg::STAGE_BYTES + j * Cfg::SUB_BYTES;
                            if (!MTMC_CHECK(a_dst + cta_bytes <= epi_stage_base && (kx & 7) == 0 && m0 >= 0 && n_row0 >= 0, p.status, 4u)) { ok = false; break; }
                            tma_load_2d_pair(a_dst, &tmA, full0, kx + j * p.bk_elems, m0);
                            tma_load_2d_pair(a_dst + Cfg::A_BYTES, mapB, full0, kx + j * p.bk_elems, n_row0);
                            if (rank == 0) mbar_expect_tx(full_bar(s), 2u * cta_bytes);     // both CTAs' bytes of this k-block
                        } else if (rank == 0) {
                            mbar_arrive(full_bar(s));                                       // the missing half of an odd walk's last stage
                        }
                    }
                    if (!ok) break;
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
            uint32_t ph = 0;
            uint32_t acc_ph = 0;
            int it = 0;
            bool ok = true;
            long long t_data = 0, t_head = 0, t_max = 0, t_acc = 0, t_kb = 0, t_issue = 0;      // trace totals (dead code without -DMTMC_TRACE)
            bool t_first = true;
            PairWalk walk(p, pair_id, num_pairs);
            PairWork w;
            for (; ok && walk.next(w); ++it) {
                const int buf = it & 1;
                const int width = w.item < p.n_full ? Cfg::OUT_TILE_N : p.tail_width;
                const int mma_n = EPI == EPI_SWIGLU ? 2 * width : width;
                const uint32_t idesc = p.fp8 ? umma_idesc_e4m3(Cfg::BM, mma_n) : umma_idesc_bf16(Cfg::BM, mma_n);
                const long long ta = tr.now();
                if (!mbar_wait_cluster(acce_bar(buf), ((acc_ph >> buf) & 1u) ^ 1u, abort_flag, p.status, STATUS_TIMEOUT_MMA | 5u)) { ok = false; break; }
                t_acc += tr.now() - ta;
                acc_ph ^= 1u << buf;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(buf * Cfg::BN);
                for (int kb = w.kb0; kb < w.kb1; kb += Cfg::KB_PER_STAGE) {
                    const int nsub = kb + 1 < w.kb1 ? 2 : 1;
                    const long long tw = tr.now();
                    if (!mbar_wait(full_bar(s), ph, abort_flag, p.status, STATUS_TIMEOUT_MMA | 6u)) { ok = false; break; }
                    { const long long dw = tr.now() - tw; t_data += dw; t_max = dw > t_max ? dw : t_max; if (kb - w.kb0 < STAGES * Cfg::KB_PER_STAGE) t_head += dw; }
                    t_kb += nsub;
                    if (t_first) { tr.stamp(TR_MMA_FIRST_NS); t_first = false; }
                    tc_fence_after();
                    const uint32_t a_src = base + s * Cfg::STAGE_BYTES;
#pragma unroll
                    for (int j = 0; j < Cfg::KB_PER_STAGE; ++j) {
                        if (j < nsub) {
                            const uint64_t a_desc = umma_smem_desc_sw128(a_src + j * Cfg::SUB_BYTES);
                            const uint64_t b_desc = umma_smem_desc_sw128(a_src + j * Cfg::SUB_BYTES + Cfg::A_BYTES);
                            // four MMAs per 128-byte row either way: 4 x 16 bf16 or 4 x 32 E4M3, 32 bytes apart
                            if (p.fp8) {
#pragma unroll
                                for (int k = 0; k < 4; ++k)
                                    umma_fp8_pair(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, ((kb - w.kb0) | j | k) != 0 ? 1u : 0u);
                            } else {
#pragma unroll
                                for (int k = 0; k < 4; ++k)
                                    umma_bf16_pair(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, ((kb - w.kb0) | j | k) != 0 ? 1u : 0u);
                            }
                        }
                        umma_commit_pair(empty_bar(s, j), 3);    // frees this k-block's half of the stage in both CTAs (also the unused half of an odd walk's end)
                    }
                    t_issue += tr.now() - tw;
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                if (ok) umma_commit_pair(accf_bar(buf), 3);      // accumulator complete, in both CTAs
            }
            tr.add(TR_MMA_STALL_DATA, t_data); tr.add(TR_MMA_STALL_HEAD, t_head); tr.max(TR_MMA_STALL_MAX, t_max);
            tr.add(TR_MMA_STALL_ACC, t_acc); tr.add(TR_MMA_KBLOCKS, t_kb); tr.add(TR_MMA_ISSUE, t_issue - t_data);
            tr.stamp(TR_MMA_LAST_NS);
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
        PairWalk walk(p, pair_id, num_pairs);
        PairWork w;
        for (; ok && walk.next(w); ++it) {
            const int buf = it & 1;
            int mb, nb, sub, width;
            item_coords(p, w.item, Cfg::OUT_TILE_N, mb, nb, sub, width);
            const int row = mb * Cfg::BM + static_cast<int>(rank) * 128 + q * 32 + lane;
            const int n_tile0 = nb * Cfg::OUT_TILE_N + sub * width;
            const bool tracer = warp == 2 && lane == 0;      // one writer for the epilogue's trace words
            const long long tw = tr.now();
            if (!mbar_wait(accf_bar(buf), (acc_ph >> buf) & 1u, abort_flag, p.status, STATUS_TIMEOUT_EPILOGUE | 5u)) { ok = false; break; }
            const long long tb = tr.now();
            if (tracer) { tr.add(TR_EPI_STALL, tb - tw); tr.add(TR_EPI_ITEMS, 1); tr.stamp_once(TR_EPI_FIRST_NS); }
            acc_ph ^= 1u << buf;
            tc_fence_after();
            const uint32_t t_addr = tmem_base + lane_base + static_cast<uint32_t>(buf * Cfg::BN);
            const int chunks = width / 32, split_at = EPI_HALVES == 2 ? (chunks + 1) / 2 : chunks;      // two warps per lane quadrant share the columns
            // part of a shared tile (stream-K): either the whole sum ends up in this accumulator, or the other holder finishes
            const bool finish = w.part < 0 || streamk_meet<Cfg::BN>(p, w, t_addr, pair_id, num_pairs, static_cast<int>(rank), q, lane);
            if (tracer && w.part >= 0) tr.add(TR_EPI_HANDOVER, tr.now() - tb);
            if (finish)
                epilogue_item<EPI, OUT_BF16>(p, t_addr, row, n_tile0, half ? split_at : 0, half ? chunks : split_at, width, nb, sub, half,
                                             vec_ok, smem_raw + (epi_stage_base - raw_addr) + (warp - 2) * EPI_STAGE_BYTES_PER_WARP, lane);
            // this CTA's half of the accumulator is drained: tell the MMA issuer in the even CTA
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_remote(cluster_map_shared(acce_bar(buf), 0));
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
