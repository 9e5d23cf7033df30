// The tiled tensor-core path: persistent, warp-specialised CTAs, one per SM.
//
//   warp 0 (one lane)  TMA producer: X and W tiles, HBM/L2 -> 128B-swizzled shared
//                      memory ring, mbarrier full/empty per stage  (Pipeline principle)
//   warp 1 (one lane)  tcgen05.mma issuer: 128 x BN x 16 bf16 MMAs accumulating fp32
//                      in tensor memory; two accumulator buffers so the next tile's
//                      mainloop overlaps this tile's epilogue     (Tiling principle)
//   warps 2-5          epilogue: tcgen05.ld -> registers -> bias / activation / gate
//                      product / row (max, sum-exp) -> global     (Fusion principle)
//
// Tile order walks M fastest inside groups of group_m row blocks so that the CTAs
// running at the same time share W tiles through L2 (Reordering principle).
#pragma once
#include "ptx.cuh"

namespace mtmc {

enum { EPI_ACT = 0, EPI_SWIGLU = 1, EPI_LSE = 2, EPI_ROWMAX = 3, EPI_XENT = 4, EPI_SOFTMAX = 5 };
enum { ACT_NONE = 0, ACT_RELU = 1, ACT_GELU_TANH = 2, ACT_SILU = 3 };

// Epilogue warps per CTA: EPI_HALVES per TMEM lane quadrant, each draining its share of an item's
// columns.  Measured on C2-C4: eight warps (two per quadrant) shorten the last, exposed epilogue of a
// CTA but cost as much again in the steady state, so the default is one warp per quadrant.
#ifndef MTMC_EPI_WARPS
#define MTMC_EPI_WARPS 4
#endif
constexpr int EPI_WARPS = MTMC_EPI_WARPS;
constexpr int EPI_HALVES = EPI_WARPS / 4;
static_assert(EPI_WARPS == 4 || EPI_WARPS == 8, "one or two epilogue warps per TMEM lane quadrant");
// Bytes of warp-private store staging per epilogue warp: one 32-row x 32-column chunk in fp32.
constexpr int EPI_STAGE_BYTES_PER_WARP = 32 * 32 * 4;

struct GemmParams {
    int M, N, K;
    int m_tiles, n_tiles, num_tiles, k_blocks;
    int rows_per_tile;    // 128 (one CTA per tile) or 256 (CTA pair)
    int group_m;
    // Wave-tail split: the tiles of the last, partial wave (indices >= n_full) are cut into
    // tail_split column pieces of tail_width output columns each, so that the wave fills the
    // SMs with shorter work items.  tail_split == 1: no split, every item is a whole tile.
    int n_full;           // items [0, n_full) are whole tiles
    int num_items;        // n_full + (num_tiles - n_full) * tail_split
    int tail_split;
    int tail_width;       // OUT_TILE_N / tail_split, a multiple of 32
    int act;
    int fp8;              // 0: bf16 operands (64 per 128-byte row, K = 16 per MMA); 1: E4M3 operands (128 per row, K = 32)
    int bk_elems;         // elements of K per ring stage: 64 or 128
    float acc_scale;      // multiplies the accumulator before the bias (product of the FP8 per-tensor scales; 1 otherwise)
    float acc_scale2;     // the same for the up half of a SwiGLU accumulator (acc_scale is then the gate half's)
    const float* bias;    // [N] or null
    const void* residual; // [M,N] in the output's element type, added after the activation, or null (EPI_ACT)
    void* out;            // [M,N] fp32 / bf16 (EPI_ACT, EPI_SWIGLU), rows `ldo` elements apart
    int ldo;              // row pitch of out in elements (N for a dense output)
    float2* lse_partial;  // [n_tiles * tail_split * EPI_HALVES][M] per row, column piece and share of the piece: (max, sum-exp) for EPI_LSE / EPI_XENT,
                          // (max, index bits) for EPI_ROWMAX
    const long long* targets;   // [M] target column per row (EPI_XENT)
    float* target_logit;        // [M] logit at the target column, written by the one piece that holds it (EPI_XENT)
    int early_w;          // 1: W is not written by any work still in flight (mtmc_set_static_weights), so the cluster split-K kernel
                          // sends out its first ring of W loads before it waits for the preceding kernel (X, bias, outputs still wait)
    uint32_t* status;     // device status word
    unsigned long long* trace;   // per-CTA trace records (-DMTMC_TRACE builds, mtmc_set_trace), else null
    // Stream-K schedule of the CTA-pair kernel (gemm_pair.cuh): tiles [0, sk_first_tile) are dealt round-robin; the
    // (tile, k-block) units of the remaining tiles (fewer than two per pair) are cut into one contiguous, equal
    // share per pair, so a tile whose k-blocks straddle shares is finished by the last of its holders to arrive.
    int sk;               // 1: stream-K schedule (whole tiles only: n_full == num_items == num_tiles)
    int sk_first_tile;    // a multiple of the number of pairs
    uint32_t sk_epoch;    // launch counter (24 bits): ticket words left by earlier launches read as zero arrivals
    uint32_t* sk_flags;   // [region tiles][2 ranks][4 lane quadrants] one ticket word per (shared tile, epilogue warp)
    float4* sk_partial;   // [pairs][2 parts][2 ranks][4 quadrants][8 chunks][8][32 lanes] fp32 accumulator parts
};

template <int EPI, int BN>
struct TileCfg {
    static constexpr int BM = 128;                       // accumulator rows = TMEM lanes
    static constexpr int BK = 64;                        // one 128-byte swizzle row of bf16
    static constexpr int A_BYTES = BM * BK * 2;
    static constexpr int B_BYTES = BN * BK * 2;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int STAGES = (BN == 256) ? 4 : 6;
    static constexpr int OUT_TILE_N = (EPI == EPI_SWIGLU) ? BN / 2 : BN;   // output columns per tile
    static constexpr int TMEM_COLS = 2 * BN;             // two accumulator buffers
    static constexpr int NUM_BARRIERS = 2 * STAGES + 4;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_WARPS * EPI_STAGE_BYTES_PER_WARP + NUM_BARRIERS * 8 + 16 + 1024;  // + alignment slack
    static constexpr int THREADS = 64 + 32 * EPI_WARPS;
};

__device__ __forceinline__ void tile_coords(const GemmParams& p, int idx, int& mb, int& nb) {
    const int per_group = p.group_m * p.n_tiles;
    const int g = idx / per_group;
    const int r = idx - g * per_group;
    const int m_first = g * p.group_m;
    const int gm = min(p.group_m, p.m_tiles - m_first);
    nb = r / gm;
    mb = m_first + (r - nb * gm);
}
// The inverse: position of tile (mb, nb) in the walk order.
__device__ __forceinline__ int tile_index(int group_m, int m_tiles, int n_tiles, int mb, int nb) {
    const int g = mb / group_m;
    const int m_first = g * group_m;
    const int gm = min(group_m, m_tiles - m_first);
    return g * group_m * n_tiles + nb * gm + (mb - m_first);
}
// Work item -> row block, column tile, piece within the tile and the piece's width in output columns.
__device__ __forceinline__ void item_coords(const GemmParams& p, int item, int full_width, int& mb, int& nb, int& sub,
                                            int& width) {
    if (item < p.n_full) {
        tile_coords(p, item, mb, nb);
        sub = 0;
        width = full_width;
    } else {
        const int j = item - p.n_full;
        const int parent = p.n_full + j / p.tail_split;
        tile_coords(p, parent, mb, nb);
        sub = j - (j / p.tail_split) * p.tail_split;
        width = p.tail_width;
    }
}

// z / (1 + exp(-z))
__device__ __forceinline__ float silu_f(float z) {
    return z * rcp_approx(1.0f + ex2_approx(-1.4426950408889634f * z));
}
// 0.5 z (1 + tanh(u)) = z * sigmoid(2u),  u = sqrt(2/pi) (z + 0.044715 z^3)
__device__ __forceinline__ float gelu_tanh_f(float z) {
    const float u2 = 1.5957691216057308f * z * fmaf(0.044715f * z, z, 1.0f);   // 2u
    return z * rcp_approx(1.0f + ex2_approx(-1.4426950408889634f * u2));
}
// The same through the hardware tanh (one special-function op instead of two).  Its absolute
// error of about 5e-4 is far inside a bf16 result's rounding, so bf16 outputs use it; fp32
// outputs keep the exp/reciprocal form above.
__device__ __forceinline__ float gelu_tanh_fast(float z) {
    const float u = 0.7978845608028654f * z * fmaf(0.044715f * z, z, 1.0f);
    float t;
    asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(u));
    const float hz = 0.5f * z;
    return fmaf(hz, t, hz);
}
// Two values at once with packed fp32 pairs for the polynomial and the final product: half the issue slots.
__device__ __forceinline__ void gelu_tanh_fast2(float& z0, float& z1) {
    float a0, a1, u0, u1, h0, h1, t0, t1;
    mul_f32x2(a0, a1, z0, z1, 0.044715f, 0.044715f);
    fma_f32x2(a0, a1, a0, a1, z0, z1, 1.0f, 1.0f);                       // 1 + 0.044715 z^2
    mul_f32x2(u0, u1, z0, z1, 0.7978845608028654f, 0.7978845608028654f);
    mul_f32x2(u0, u1, u0, u1, a0, a1);
    asm("tanh.approx.f32 %0, %1;" : "=f"(t0) : "f"(u0));
    asm("tanh.approx.f32 %0, %1;" : "=f"(t1) : "f"(u1));
    mul_f32x2(h0, h1, z0, z1, 0.5f, 0.5f);
    fma_f32x2(z0, z1, h0, h1, t0, t1, h0, h1);
}
__device__ __forceinline__ float apply_act(int act, float z) {
    switch (act) {
        case ACT_RELU: return fmaxf(z, 0.0f);
        case ACT_GELU_TANH: return gelu_tanh_f(z);
        case ACT_SILU: return silu_f(z);
        default: return z;
    }
}

template <bool OUT_BF16>
__device__ __forceinline__ void apply_act_chunk(int act, float (&y)[32]) {
    if (act == ACT_RELU) {
#pragma unroll
        for (int j = 0; j < 32; ++j) y[j] = fmaxf(y[j], 0.0f);
    } else if (act == ACT_GELU_TANH) {
#pragma unroll
        for (int j = 0; j < 32; j += 2) {
            if (OUT_BF16) gelu_tanh_fast2(y[j], y[j + 1]);
            else { y[j] = gelu_tanh_f(y[j]); y[j + 1] = gelu_tanh_f(y[j + 1]); }
        }
    } else if (act == ACT_SILU) {
#pragma unroll
        for (int j = 0; j < 32; ++j) y[j] = silu_f(y[j]);
    }
}

// Stores 32 consecutive columns [n0, n0+32) of one output row; 128-bit stores when
// the row segment is whole and 16-byte aligned, predicated scalar stores otherwise.
template <bool OUT_BF16>
__device__ __forceinline__ void store_row_chunk(void* out, int row, int n0, int N, int ld, const float (&y)[32], bool vec_ok) {
    if (OUT_BF16) {
        __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(out) + static_cast<size_t>(row) * ld + n0;
        if (vec_ok && n0 + 32 <= N) {
            uint4* o4 = reinterpret_cast<uint4*>(o);
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                uint4 q;
                q.x = pack_bf16x2(y[8 * v + 0], y[8 * v + 1]);
                q.y = pack_bf16x2(y[8 * v + 2], y[8 * v + 3]);
                q.z = pack_bf16x2(y[8 * v + 4], y[8 * v + 5]);
                q.w = pack_bf16x2(y[8 * v + 6], y[8 * v + 7]);
                o4[v] = q;
            }
        } else {
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (n0 + j < N) o[j] = __float2bfloat16_rn(y[j]);
        }
    } else {
        float* o = reinterpret_cast<float*>(out) + static_cast<size_t>(row) * ld + n0;
        if (vec_ok && n0 + 32 <= N) {
            float4* o4 = reinterpret_cast<float4*>(o);
#pragma unroll
            for (int v = 0; v < 8; ++v) o4[v] = make_float4(y[4 * v], y[4 * v + 1], y[4 * v + 2], y[4 * v + 3]);
        } else {
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (n0 + j < N) o[j] = y[j];
        }
    }
}

// Coalesced store of one 32-row x 32-column chunk held one row per lane.  The rows are
// exchanged through a warp-private shared-memory buffer (16-byte units, XOR-swizzled so that
// neither side has bank conflicts) so that every 128-bit store instruction of the warp
// writes whole, contiguous row segments: 8 rows x 64 B for bf16, 4 rows x 128 B for fp32.
// Requires the chunk to lie wholly inside [0, N) and 16-byte aligned rows; rows >= M are
// not stored.  `row0` is the output row of lane 0.
template <bool OUT_BF16>
__device__ __forceinline__ void store_chunk_coalesced(uint8_t* stage, void* out, int row0, int n0, int M, int ld,
                                                      const float (&y)[32], int lane) {
    constexpr int UNITS = OUT_BF16 ? 4 : 8;                  // 16-byte units per row of the chunk
    constexpr int ROW_BYTES = UNITS * 16;
    uint4* my_row = reinterpret_cast<uint4*>(stage + lane * ROW_BYTES);
    const int wkey = OUT_BF16 ? ((lane >> 1) & 3) : (lane & 7);
#pragma unroll
    for (int u = 0; u < UNITS; ++u) {
        uint4 q;
        if (OUT_BF16) {
            q.x = pack_bf16x2(y[8 * u + 0], y[8 * u + 1]);
            q.y = pack_bf16x2(y[8 * u + 2], y[8 * u + 3]);
            q.z = pack_bf16x2(y[8 * u + 4], y[8 * u + 5]);
            q.w = pack_bf16x2(y[8 * u + 6], y[8 * u + 7]);
        } else {
            q.x = __float_as_uint(y[4 * u + 0]);
            q.y = __float_as_uint(y[4 * u + 1]);
            q.z = __float_as_uint(y[4 * u + 2]);
            q.w = __float_as_uint(y[4 * u + 3]);
        }
        my_row[u ^ wkey] = q;
    }
    __syncwarp();
    constexpr int ROWS_PER_STORE = 32 / UNITS;
    const int sub_row = lane / UNITS;
    const int unit = lane % UNITS;
    const size_t elem = OUT_BF16 ? 2 : 4;
#pragma unroll
    for (int it = 0; it < UNITS; ++it) {
        const int r = it * ROWS_PER_STORE + sub_row;
        const int rkey = OUT_BF16 ? ((r >> 1) & 3) : (r & 7);
        const uint4 q = *reinterpret_cast<const uint4*>(stage + r * ROW_BYTES + ((unit ^ rkey) * 16));
        if (row0 + r < M) {
            uint8_t* dst = reinterpret_cast<uint8_t*>(out) + (static_cast<size_t>(row0 + r) * ld + n0) * elem + unit * 16;
            *reinterpret_cast<uint4*>(dst) = q;
        }
    }
    __syncwarp();                                            // the buffer is reused by the next chunk
}

// y[j] += R[row][n0 + j] for the 32 columns of one chunk of one row (R in the output's type).
template <bool OUT_BF16>
__device__ __forceinline__ void add_residual_chunk(const void* residual, int row, int n0, int N, float (&y)[32], bool vec_ok) {
    if (OUT_BF16) {
        const __nv_bfloat16* r = reinterpret_cast<const __nv_bfloat16*>(residual) + static_cast<size_t>(row) * N + n0;
        if (vec_ok && n0 + 32 <= N) {
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                const uint4 q = *reinterpret_cast<const uint4*>(r + 8 * v);
                const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    y[8 * v + 2 * h] += __uint_as_float(w[h] << 16);
                    y[8 * v + 2 * h + 1] += __uint_as_float(w[h] & 0xffff0000u);
                }
            }
        } else {
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (n0 + j < N) y[j] += __bfloat162float(r[j]);
        }
    } else {
        const float* r = reinterpret_cast<const float*>(residual) + static_cast<size_t>(row) * N + n0;
        if (vec_ok && n0 + 32 <= N) {
#pragma unroll
            for (int v = 0; v < 8; ++v) {
                const float4 q = *reinterpret_cast<const float4*>(r + 4 * v);
                y[4 * v] += q.x; y[4 * v + 1] += q.y; y[4 * v + 2] += q.z; y[4 * v + 3] += q.w;
            }
        } else {
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (n0 + j < N) y[j] += r[j];
        }
    }
}

// Loads bias[n0 .. n0+32) into registers (zeros past N or without bias).
__device__ __forceinline__ void load_bias_chunk(const float* bias, int n0, int N, float (&b)[32]) {
    if (bias == nullptr) {
#pragma unroll
        for (int j = 0; j < 32; ++j) b[j] = 0.0f;
    } else if (n0 + 32 <= N) {
        const float4* b4 = reinterpret_cast<const float4*>(bias + n0);
#pragma unroll
        for (int v = 0; v < 8; ++v) {
            const float4 t = __ldg(b4 + v);
            b[4 * v] = t.x; b[4 * v + 1] = t.y; b[4 * v + 2] = t.z; b[4 * v + 3] = t.w;
        }
    } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) b[j] = (n0 + j < N) ? __ldg(bias + n0 + j) : 0.0f;
    }
}

// The same from a copy of the tile's bias in shared memory (bias_tile[j] = bias of the tile's column j, zeros
// past N), when the kernel keeps one: a global load costs the exposed epilogue of gemm_big.cuh several hundred
// clocks per chunk, a broadcast shared-memory load a few tens.
__device__ __forceinline__ void tile_bias_chunk(const GemmParams& p, const float* bias_tile, int n_tile0, int n0, float (&b)[32]) {
    if (bias_tile == nullptr) {
        load_bias_chunk(p.bias, n0, p.N, b);
    } else {
        const float4* b4 = reinterpret_cast<const float4*>(bias_tile + (n0 - n_tile0));
#pragma unroll
        for (int v = 0; v < 8; ++v) {
            const float4 t = b4[v];
            b[4 * v] = t.x; b[4 * v + 1] = t.y; b[4 * v + 2] = t.z; b[4 * v + 3] = t.w;
        }
    }
}

// One work item's epilogue for one thread: this thread owns output row `row` (TMEM lane
// of t_addr) and walks chunks [c_begin, c_end) of 32 columns of the item that starts at column n_tile0
// (the other half of the chunks belongs to the second warp of this lane quadrant).
//   EPI_ACT    : + bias, activation, store
//   EPI_SWIGLU : silu(gate) * up with the up columns `width` columns after the gate columns
//   EPI_LSE    : online (max, sum-exp) in base-2 units, one partial per (row, column piece)
//   EPI_XENT   : the same, and the logit at the row's target column is set aside
//   EPI_ROWMAX : running (max, lowest column attaining it), one partial per (row, column piece)
//   EPI_SOFTMAX: the (max, sum-exp) partial of EPI_LSE, and exp(z - max of the piece) stored to out for every column
template <int EPI, bool OUT_BF16>
__device__ __forceinline__ void epilogue_item(const GemmParams& p, uint32_t t_addr, int row, int n_tile0, int c_begin,
                                              int c_end, int width, int nb, int sub, int half, bool vec_ok, uint8_t* stage,
                                              int lane, const float* bias_tile = nullptr) {
    // the chunks lie inside the 512 columns of tensor memory and inside the item; the item starts inside the padded output
    if (!MTMC_CHECK((t_addr & 0xffffu) + static_cast<uint32_t>((EPI == EPI_SWIGLU ? width : 0) + c_end * 32) <= 512u &&
                    c_begin >= 0 && c_end * 32 <= width && n_tile0 >= 0 && n_tile0 < p.N + 256, p.status, 1u)) return;
    if (EPI == EPI_ACT) {
        // Two chunks in flight: while chunk c is being activated and stored, the TMEM load and the
        // bias fetch of chunk c + 1 are already under way.
        int live = c_end;                                    // chunks that start inside [0, N)
        if (n_tile0 + c_end * 32 > p.N) live = (p.N - n_tile0 + 31) / 32;
        uint32_t r[32];
        float bv[32];
        if (c_begin < live) {
            tmem_ld_32x32b_x32(t_addr + c_begin * 32, r);
            tile_bias_chunk(p, bias_tile, n_tile0, n_tile0 + c_begin * 32, bv);
        }
#pragma unroll 1
        for (int c = c_begin; c < live; ++c) {
            const int n0 = n_tile0 + c * 32;
            tmem_ld_wait();                                  // chunk c has landed in r
            float y[32];
#pragma unroll
            for (int j = 0; j < 32; j += 2)
                fma_f32x2(y[j], y[j + 1], __uint_as_float(r[j]), __uint_as_float(r[j + 1]), p.acc_scale, p.acc_scale, bv[j], bv[j + 1]);
            if (c + 1 < live) {                              // r and bv are free again: refill them for chunk c + 1
                tmem_ld_32x32b_x32(t_addr + (c + 1) * 32, r);
                tile_bias_chunk(p, bias_tile, n_tile0, n0 + 32, bv);
            }
            apply_act_chunk<OUT_BF16>(p.act, y);
            if (p.residual != nullptr && row < p.M) add_residual_chunk<OUT_BF16>(p.residual, row, n0, p.N, y, vec_ok);
            if (!MTMC_CHECK(n0 >= 0 && n0 < p.N && p.ldo >= p.N, p.status, 5u)) continue;
            if (vec_ok && n0 + 32 <= p.N) store_chunk_coalesced<OUT_BF16>(stage, p.out, row - lane, n0, p.M, p.ldo, y, lane);
            else if (row < p.M) store_row_chunk<OUT_BF16>(p.out, row, n0, p.N, p.ldo, y, false);
        }
    } else if (EPI == EPI_SWIGLU) {
        // As for the activation epilogue: the gate and up loads of chunk c + 1 go out as soon as chunk c has been
        // combined, so that they are under way during its stores.
        const int live = min(c_end, (p.N - n_tile0 + 31) / 32);
        uint32_t g[32], u[32];
        if (c_begin < live) {
            tmem_ld_32x32b_x32(t_addr + c_begin * 32, g);            // gate columns
            tmem_ld_32x32b_x32(t_addr + width + c_begin * 32, u);    // up columns follow the gate columns
        }
#pragma unroll 1
        for (int c = c_begin; c < live; ++c) {
            const int n0 = n_tile0 + c * 32;
            tmem_ld_wait();
            float y[32];
            if (p.fp8) {                                            // E4M3 operands: the per-tensor scales of gate and up
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    g[j] = __float_as_uint(__uint_as_float(g[j]) * p.acc_scale);
                    u[j] = __float_as_uint(__uint_as_float(u[j]) * p.acc_scale2);
                }
            }
#pragma unroll
            for (int j = 0; j < 32; j += 2) {                       // packed fp32 pairs: half the issue slots of the FP part
                const float g0 = __uint_as_float(g[j]), g1 = __uint_as_float(g[j + 1]);
                float t0, t1, d0, d1, s0, s1;
                mul_f32x2(t0, t1, g0, g1, -1.4426950408889634f, -1.4426950408889634f);
                add_f32x2(d0, d1, ex2_approx(t0), ex2_approx(t1), 1.0f, 1.0f);
                mul_f32x2(s0, s1, g0, g1, rcp_approx(d0), rcp_approx(d1));
                mul_f32x2(y[j], y[j + 1], s0, s1, __uint_as_float(u[j]), __uint_as_float(u[j + 1]));
            }
            if (c + 1 < live) {
                tmem_ld_32x32b_x32(t_addr + (c + 1) * 32, g);
                tmem_ld_32x32b_x32(t_addr + width + (c + 1) * 32, u);
            }
            if (vec_ok && n0 + 32 <= p.N) store_chunk_coalesced<true>(stage, p.out, row - lane, n0, p.M, p.ldo, y, lane);
            else if (row < p.M) store_row_chunk<true>(p.out, row, n0, p.N, p.ldo, y, false);
        }
    } else if (EPI == EPI_ROWMAX) {
        // Four interleaved (max, column) chains per chunk, merged with the tie rule (the lower column wins), and
        // the next chunk's TMEM load in flight meanwhile.
        float mx = -INFINITY;
        int arg = 0x7fffffff;
        const int live = min(c_end, (p.N - n_tile0 + 31) / 32);
        uint32_t r[32];
        if (c_begin < live) tmem_ld_32x32b_x32(t_addr + c_begin * 32, r);
#pragma unroll 1
        for (int c = c_begin; c < live; ++c) {
            const int n0 = n_tile0 + c * 32;
            float bv[32];
            tile_bias_chunk(p, bias_tile, n_tile0, n0, bv);
            tmem_ld_wait();
            float z[32];
#pragma unroll
            for (int j = 0; j < 32; ++j)
                z[j] = (n0 + j < p.N) ? fmaf(__uint_as_float(r[j]), p.acc_scale, bv[j]) : -INFINITY;   // scale 1: the same bits as r + b
            if (c + 1 < live) tmem_ld_32x32b_x32(t_addr + (c + 1) * 32, r);
            float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
            int a4[4] = {0x7fffffff, 0x7fffffff, 0x7fffffff, 0x7fffffff};
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (z[j] > m4[j & 3]) { m4[j & 3] = z[j]; a4[j & 3] = n0 + j; }      // strict: ties keep the lower column of the chain
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (m4[k] > mx || (m4[k] == mx && a4[k] < arg)) { mx = m4[k]; arg = a4[k]; }
        }
        if (row < p.M && MTMC_CHECK((nb * p.tail_split + sub) * EPI_HALVES + half < p.n_tiles * p.tail_split * EPI_HALVES, p.status, 2u))
            p.lse_partial[static_cast<size_t>((nb * p.tail_split + sub) * EPI_HALVES + half) * p.M + row] = make_float2(mx, __int_as_float(arg));
    } else if (EPI == EPI_SOFTMAX) {
        // Two passes over the piece's accumulator columns, which stay in tensor memory meanwhile: first the row's
        // maximum over the piece, then e = 2^(t - max) for every column, stored as the still unnormalised output and
        // summed.  The (max, sum) partial goes the way of EPI_LSE; softmax_finish_kernel multiplies the piece by
        // exp(max - lse) once the row's lse is known.
        constexpr float LOG2E = 1.4426950408889634f;
        const float zscale = LOG2E * p.acc_scale;
        const int live = min(c_end, (p.N - n_tile0 + 31) / 32);
        float mx = -INFINITY, sum = 0.0f;
        uint32_t r[32];
        if (c_begin < live) tmem_ld_32x32b_x32(t_addr + c_begin * 32, r);
#pragma unroll 1
        for (int c = c_begin; c < live; ++c) {
            const int n0 = n_tile0 + c * 32;
            float bv[32];
            tile_bias_chunk(p, bias_tile, n_tile0, n0, bv);
            tmem_ld_wait();
            float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
            const bool ragged = n0 + 32 > p.N;               // columns past N are zero-filled weight rows: masked out
#pragma unroll
            for (int j = 0; j < 32; j += 2) {                // packed fp32 pairs: half the issue slots of the FP part
                float b0, b1, t0, t1;
                mul_f32x2(b0, b1, bv[j], bv[j + 1], LOG2E, LOG2E);
                fma_f32x2(t0, t1, __uint_as_float(r[j]), __uint_as_float(r[j + 1]), zscale, zscale, b0, b1);
                if (ragged) {
                    if (n0 + j >= p.N) t0 = -INFINITY;
                    if (n0 + j + 1 >= p.N) t1 = -INFINITY;
                }
                m4[j & 3] = fmaxf(m4[j & 3], t0);
                m4[(j + 1) & 3] = fmaxf(m4[(j + 1) & 3], t1);
            }
            if (c + 1 < live) tmem_ld_32x32b_x32(t_addr + (c + 1) * 32, r);
            mx = fmaxf(mx, fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3])));
        }
        if (c_begin < live) tmem_ld_32x32b_x32(t_addr + c_begin * 32, r);
#pragma unroll 1
        for (int c = c_begin; c < live; ++c) {
            const int n0 = n_tile0 + c * 32;
            float bv[32], y[32];
            tile_bias_chunk(p, bias_tile, n_tile0, n0, bv);
            tmem_ld_wait();
            float s4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
            const bool ragged = n0 + 32 > p.N;
#pragma unroll
            for (int j = 0; j < 32; j += 2) {
                float b0, b1, t0, t1, d0, d1;
                mul_f32x2(b0, b1, bv[j], bv[j + 1], LOG2E, LOG2E);
                fma_f32x2(t0, t1, __uint_as_float(r[j]), __uint_as_float(r[j + 1]), zscale, zscale, b0, b1);   // the same bits as in the first pass
                add_f32x2(d0, d1, t0, t1, -mx, -mx);
                y[j] = ex2_approx(d0);
                y[j + 1] = ex2_approx(d1);
                if (ragged) {
                    if (n0 + j >= p.N) y[j] = 0.0f;
                    if (n0 + j + 1 >= p.N) y[j + 1] = 0.0f;
                }
                add_f32x2(s4[j & 3], s4[(j + 1) & 3], s4[j & 3], s4[(j + 1) & 3], y[j], y[j + 1]);
            }
            if (c + 1 < live) tmem_ld_32x32b_x32(t_addr + (c + 1) * 32, r);
            sum += (s4[0] + s4[1]) + (s4[2] + s4[3]);
            if (!MTMC_CHECK(n0 >= 0 && n0 < p.N && p.ldo >= p.N, p.status, 5u)) continue;
            if (vec_ok && n0 + 32 <= p.N) store_chunk_coalesced<OUT_BF16>(stage, p.out, row - lane, n0, p.M, p.ldo, y, lane);
            else if (row < p.M) store_row_chunk<OUT_BF16>(p.out, row, n0, p.N, p.ldo, y, false);
        }
        // a piece that lies wholly past N (only possible in the last column tile) stays neutral
        if (row < p.M && MTMC_CHECK((nb * p.tail_split + sub) * EPI_HALVES + half < p.n_tiles * p.tail_split * EPI_HALVES, p.status, 2u))
            p.lse_partial[static_cast<size_t>((nb * p.tail_split + sub) * EPI_HALVES + half) * p.M + row] =
                make_float2(mx * 0.6931471805599453f, sum);
    } else {
        // Online (max, sum-exp) over this tile's columns, in base-2 units: t = z * log2(e).
        constexpr float LOG2E = 1.4426950408889634f;
        const float zscale = LOG2E * p.acc_scale;            // accumulator -> base-2 logit units (acc_scale is 1 for bf16 operands)
        float mx = -INFINITY, sum = 0.0f;
        int tgt = -1;
        float tz = 0.0f;
        bool found = false;
        if (EPI == EPI_XENT && row < p.M) tgt = static_cast<int>(p.targets[row]);
        // Chunks that start inside [0, N); the TMEM load of chunk c + 1 is issued as soon as chunk c has been
        // turned into logits, and the maxima and sums run as four interleaved chains (32-long dependent chains
        // are what an epilogue warp otherwise spends its time on, visibly so when the epilogue is not overlapped).
        int live = min(c_end, (p.N - n_tile0 + 31) / 32);
        uint32_t r[32];
        if (c_begin < live) tmem_ld_32x32b_x32(t_addr + c_begin * 32, r);
#pragma unroll 1
        for (int c = c_begin; c < live; ++c) {
            const int n0 = n_tile0 + c * 32;
            float bv[32], tv[32];
            tile_bias_chunk(p, bias_tile, n_tile0, n0, bv);
            tmem_ld_wait();
            float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int j = 0; j < 32; j += 2) {
                float b0, b1;
                mul_f32x2(b0, b1, bv[j], bv[j + 1], LOG2E, LOG2E);
                fma_f32x2(tv[j], tv[j + 1], __uint_as_float(r[j]), __uint_as_float(r[j + 1]), zscale, zscale, b0, b1);
                m4[j & 3] = fmaxf(m4[j & 3], tv[j]);
                m4[(j + 1) & 3] = fmaxf(m4[(j + 1) & 3], tv[j + 1]);
            }
            if (c + 1 < live) tmem_ld_32x32b_x32(t_addr + (c + 1) * 32, r);      // r is free again
            if (n0 + 32 > p.N) {      // ragged last chunk: columns past N are zero-filled weight rows, mask them out
#pragma unroll
                for (int k = 0; k < 4; ++k) m4[k] = -INFINITY;
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    if (n0 + j >= p.N) tv[j] = -INFINITY;
                    m4[j & 3] = fmaxf(m4[j & 3], tv[j]);
                }
            }
            if (EPI == EPI_XENT) {
                const int rel = tgt - n0;                    // the target's place in this chunk, if it is here
                if (static_cast<unsigned>(rel) < 32u && tgt < p.N) {
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (j == rel) tz = tv[j] * 0.6931471805599453f;
                    found = true;
                }
            }
            const float nm = fmaxf(mx, fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3])));
            float s4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
            for (int j = 0; j < 32; j += 2) {
                float d0, d1;
                add_f32x2(d0, d1, tv[j], tv[j + 1], -nm, -nm);
                add_f32x2(s4[j & 3], s4[(j + 1) & 3], s4[j & 3], s4[(j + 1) & 3], ex2_approx(d0), ex2_approx(d1));
            }
            sum = sum * ex2_approx(mx - nm) + ((s4[0] + s4[1]) + (s4[2] + s4[3]));
            mx = nm;
        }
        // a piece that lies wholly past N (only possible in the last column tile) stays neutral
        if (row < p.M && MTMC_CHECK((nb * p.tail_split + sub) * EPI_HALVES + half < p.n_tiles * p.tail_split * EPI_HALVES, p.status, 2u))
            p.lse_partial[static_cast<size_t>((nb * p.tail_split + sub) * EPI_HALVES + half) * p.M + row] =
                make_float2(mx * 0.6931471805599453f, sum);
        if (EPI == EPI_XENT && found) p.target_logit[row] = tz;
    }
}

template <int EPI, int BN, bool OUT_BF16>
__global__ void __launch_bounds__(64 + 32 * EPI_WARPS, 1)
gemm_tiled_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                  const __grid_constant__ CUtensorMap tmB2, const __grid_constant__ CUtensorMap tmBt,
                  const __grid_constant__ CUtensorMap tmB2t, const GemmParams p) {
    using Cfg = TileCfg<EPI, BN>;
    constexpr int STAGES = Cfg::STAGES;
    extern __shared__ uint8_t smem_raw[];

    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;          // swizzled tiles need 1024-byte alignment
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

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(accf_bar(b), 1); mbar_init(acce_bar(b), EPI_WARPS); }
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
    pdl_launch_dependents();     // the next kernel in the stream may begin its own set-up
    pdl_wait();                  // everything before this line touched only shared and tensor memory

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < p.num_items && ok; t += gridDim.x) {
                int mb, nb, sub, width;
                item_coords(p, t, Cfg::OUT_TILE_N, mb, nb, sub, width);
                const bool whole = width == Cfg::OUT_TILE_N;
                const int m0 = mb * Cfg::BM;
                const int n0 = nb * Cfg::OUT_TILE_N + sub * width;
                const uint32_t b_rows_bytes = static_cast<uint32_t>(width) * Cfg::BK * 2;   // one W box of this item
                const uint32_t tx = Cfg::A_BYTES + (EPI == EPI_SWIGLU ? 2u : 1u) * b_rows_bytes;
                const CUtensorMap* mapB = whole ? &tmB : &tmBt;
                const CUtensorMap* mapB2 = whole ? &tmB2 : &tmB2t;
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, p.status, STATUS_TIMEOUT_PRODUCER | 1u)) { ok = false; break; }
                    const uint32_t a_dst = base + s * Cfg::STAGE_BYTES;
                    const uint32_t b_dst = a_dst + Cfg::A_BYTES;
                    mbar_expect_tx(full_bar(s), tx);
                    tma_load_2d(a_dst, &tmA, full_bar(s), kb * p.bk_elems, m0);
                    tma_load_2d(b_dst, mapB, full_bar(s), kb * p.bk_elems, n0);
                    if (EPI == EPI_SWIGLU)      // the up rows follow the gate rows: one contiguous B operand
                        tma_load_2d(b_dst + b_rows_bytes, mapB2, full_bar(s), kb * p.bk_elems, n0);
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0;
            uint32_t acc_ph = 0;                         // bit b: phase of accumulator buffer b
            int it = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < p.num_items && ok; t += gridDim.x, ++it) {
                const int buf = it & 1;
                const int width = t < p.n_full ? Cfg::OUT_TILE_N : p.tail_width;
                const int mma_n = EPI == EPI_SWIGLU ? 2 * width : width;
                const uint32_t idesc = p.fp8 ? umma_idesc_e4m3(Cfg::BM, mma_n) : umma_idesc_bf16(Cfg::BM, mma_n);
                if (!mbar_wait(acce_bar(buf), ((acc_ph >> buf) & 1u) ^ 1u, abort_flag, p.status, STATUS_TIMEOUT_MMA | 1u)) { ok = false; break; }
                acc_ph ^= 1u << buf;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(buf * BN);
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    if (!mbar_wait(full_bar(s), ph, abort_flag, p.status, STATUS_TIMEOUT_MMA | 2u)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_src = base + s * Cfg::STAGE_BYTES;
                    const uint64_t a_desc = umma_smem_desc_sw128(a_src);
                    const uint64_t b_desc = umma_smem_desc_sw128(a_src + Cfg::A_BYTES);
                    // four MMAs per 128-byte row either way: 4 x 16 bf16 or 4 x 32 E4M3, 32 bytes apart
                    if (p.fp8) {
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            umma_fp8(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, (kb | k) != 0 ? 1u : 0u);
                    } else {
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            umma_bf16(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, (kb | k) != 0 ? 1u : 0u);
                    }
                    umma_commit(empty_bar(s));      // frees the stage once these MMAs have read it
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                if (ok) umma_commit(accf_bar(buf));  // accumulator complete
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue
        const int q = warp & 3;                      // TMEM lane quadrant this warp may read
        const int half = (warp - 2) >> 2;            // which half of the item's columns this warp takes
        const uint32_t lane_base = static_cast<uint32_t>(q * 32) << 16;
        const bool vec_ok = OUT_BF16 ? (p.ldo % 8 == 0) : (p.ldo % 4 == 0);       // 16-byte aligned rows of out (and of a dense residual)
        uint32_t acc_ph = 0;
        int it = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < p.num_items && ok; t += gridDim.x, ++it) {
            const int buf = it & 1;
            int mb, nb, sub, width;
            item_coords(p, t, Cfg::OUT_TILE_N, mb, nb, sub, width);
            const int row = mb * Cfg::BM + q * 32 + lane;
            const int n_tile0 = nb * Cfg::OUT_TILE_N + sub * width;
            const int chunks = width / 32;
            if (!mbar_wait(accf_bar(buf), (acc_ph >> buf) & 1u, abort_flag, p.status, STATUS_TIMEOUT_EPILOGUE | 1u)) { ok = false; break; }
            acc_ph ^= 1u << buf;
            tc_fence_after();
            const uint32_t t_addr = tmem_base + lane_base + static_cast<uint32_t>(buf * BN);

            const int split_at = EPI_HALVES == 2 ? (chunks + 1) / 2 : chunks;   // the warps of a lane quadrant share the columns
            epilogue_item<EPI, OUT_BF16>(p, t_addr, row, n_tile0, half ? split_at : 0, half ? chunks : split_at, width, nb, sub, half,
                                         vec_ok, smem_raw + (epi_stage_base - raw_addr) + (warp - 2) * EPI_STAGE_BYTES_PER_WARP, lane);
            // accumulator buffer drained: hand it back to the MMA warp
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acce_bar(buf));
        }
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (*abort_flag != 0u) {
        // A wait gave up: let copies / MMAs already in flight land before freeing anything.
        const long long t0 = clock64();
        while (clock64() - t0 < 400000ll) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
    }
}

// (m, s) <- (m, s) (+) (om, os):  max of the maxima, sums rescaled to it.  A side that
// has seen nothing yet holds (-inf, 0) and stays neutral.
__device__ __forceinline__ void lse_combine(float& m, float& s, float om, float os) {
    const float nm = fmaxf(m, om);
    const float a = (m == -INFINITY) ? 0.0f : __expf(m - nm);
    const float b = (om == -INFINITY) ? 0.0f : __expf(om - nm);
    s = s * a + os * b;
    m = nm;
}

// Merges the (max, sum-exp) partials of each row, in ascending column order, into
// lse[row] = max + ln(sum).  One warp per row; lanes stride over the column tiles and
// combine with shuffles.  Every piece left EPI_HALVES partials; a whole tile is one piece, a tile
// of the split wave tail is tail_split pieces.  With target_logit / loss given it also writes the
// softmax cross entropy loss[row] = lse[row] - logit[row][target[row]].  (The warp-per-row form: the allocation-free entry
// point launches it with the block size it chose; everything else uses lse_merge_rows_kernel below.)
__global__ void lse_merge_kernel(const float2* __restrict__ partial, int M, int rows_per_tile, int m_tiles, int n_tiles,
                                 int group_m, int n_full, int tail_split, float* __restrict__ lse,
                                 const float* __restrict__ target_logit, float* __restrict__ loss) {
    pdl_launch_dependents();     // the next kernel of this library may set up (and prefetch static weights) beside this one
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= M) return;
    const int mb = row / rows_per_tile;
    float mx = -INFINITY, sum = 0.0f;
    for (int nb = lane; nb < n_tiles; nb += 32) {
        const int pieces = tile_index(group_m, m_tiles, n_tiles, mb, nb) < n_full ? 1 : tail_split;
        for (int sl = 0; sl < EPI_HALVES * pieces; ++sl) {    // ascending columns
            const float2 v = __ldcg(partial + static_cast<size_t>(nb * tail_split * EPI_HALVES + sl) * M + row);
            lse_combine(mx, sum, v.x, v.y);
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const float om = __shfl_xor_sync(0xffffffffu, mx, off);
        const float os = __shfl_xor_sync(0xffffffffu, sum, off);
        lse_combine(mx, sum, om, os);
    }
    if (lane == 0) {
        const float l = mx + __logf(sum);
        if (lse) lse[row] = l;
        if (loss) loss[row] = l - __ldcg(target_logit + row);
    }
}

// The logsumexp merge with the roles of lanes and warps exchanged, and the row-maximum merge (the largest value, ties
// to the lowest column) in the same form: a block owns 32 consecutive rows, lane = row,
// and its warps share out the column tiles (warp w takes tiles w, w + warps, ...).  partial[piece][row] is then read
// as whole 256-byte lines (the warp-per-row form fetches a 32-byte sector for every 8 bytes it uses), four tiles'
// loads are in flight per thread, and warp 0 adds the warps' results in warp order through shared memory, so the
// result does not depend on timing.  Launched with 32 * MERGE_WARPS threads per block and ceil(M / 32) blocks.
constexpr int MERGE_WARPS = 16;

__global__ void __launch_bounds__(32 * MERGE_WARPS)
lse_merge_rows_kernel(const float2* __restrict__ partial, int M, int rows_per_tile, int m_tiles, int n_tiles, int group_m,
                      int n_full, int tail_split, float* __restrict__ lse, const float* __restrict__ target_logit,
                      float* __restrict__ loss) {
    pdl_launch_dependents();     // the next kernel of this library may set up (and prefetch static weights) beside this one
    pdl_wait();                  // launched as a programmatic dependent: the tiled kernel's partials are complete from here on
    __shared__ float2 part[MERGE_WARPS][32];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int row = blockIdx.x * 32 + lane;
    float mx = -INFINITY, sum = 0.0f;
    if (row < M) {
        const int mb = row / rows_per_tile;
        for (int nb0 = w; nb0 < n_tiles; nb0 += 4 * MERGE_WARPS) {
            float2 v[4];
            int more[4];                                      // further partials of the tile (pieces of the wave tail, shares of a piece)
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int nb = nb0 + u * MERGE_WARPS;
                v[u] = make_float2(-INFINITY, 0.0f);
                more[u] = 0;
                if (nb < n_tiles) {
                    const int pieces = tile_index(group_m, m_tiles, n_tiles, mb, nb) < n_full ? 1 : tail_split;
                    more[u] = EPI_HALVES * pieces - 1;
                    v[u] = __ldcg(partial + static_cast<size_t>(nb * tail_split * EPI_HALVES) * M + row);
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                lse_combine(mx, sum, v[u].x, v[u].y);         // (-inf, 0) past the last tile: neutral
                const int nb = nb0 + u * MERGE_WARPS;
                for (int sl = 1; sl <= more[u]; ++sl) {       // ascending columns
                    const float2 x = __ldcg(partial + static_cast<size_t>(nb * tail_split * EPI_HALVES + sl) * M + row);
                    lse_combine(mx, sum, x.x, x.y);
                }
            }
        }
    }
    part[w][lane] = make_float2(mx, sum);
    __syncthreads();
    if (w == 0 && row < M) {
#pragma unroll
        for (int k = 1; k < MERGE_WARPS; ++k) lse_combine(mx, sum, part[k][lane].x, part[k][lane].y);
        const float l = mx + __logf(sum);
        if (lse) lse[row] = l;
        if (loss) loss[row] = l - __ldcg(target_logit + row);
    }
}

__global__ void __launch_bounds__(32 * MERGE_WARPS)
rowmax_merge_rows_kernel(const float2* __restrict__ partial, int M, int rows_per_tile, int m_tiles, int n_tiles, int group_m,
                         int n_full, int tail_split, float* __restrict__ max_out, int* __restrict__ argmax_out) {
    pdl_launch_dependents();
    pdl_wait();
    __shared__ float2 part[MERGE_WARPS][32];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int row = blockIdx.x * 32 + lane;
    float mx = -INFINITY;
    int arg = 0x7fffffff;
    if (row < M) {
        const int mb = row / rows_per_tile;
        for (int nb0 = w; nb0 < n_tiles; nb0 += 4 * MERGE_WARPS) {
            float2 v[4];
            int more[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int nb = nb0 + u * MERGE_WARPS;
                v[u] = make_float2(-INFINITY, __int_as_float(0x7fffffff));
                more[u] = 0;
                if (nb < n_tiles) {
                    const int pieces = tile_index(group_m, m_tiles, n_tiles, mb, nb) < n_full ? 1 : tail_split;
                    more[u] = EPI_HALVES * pieces - 1;
                    v[u] = __ldcg(partial + static_cast<size_t>(nb * tail_split * EPI_HALVES) * M + row);
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                int a = __float_as_int(v[u].y);
                if (v[u].x > mx || (v[u].x == mx && a < arg)) { mx = v[u].x; arg = a; }
                const int nb = nb0 + u * MERGE_WARPS;
                for (int sl = 1; sl <= more[u]; ++sl) {
                    const float2 x = __ldcg(partial + static_cast<size_t>(nb * tail_split * EPI_HALVES + sl) * M + row);
                    a = __float_as_int(x.y);
                    if (x.x > mx || (x.x == mx && a < arg)) { mx = x.x; arg = a; }
                }
            }
        }
    }
    part[w][lane] = make_float2(mx, __int_as_float(arg));
    __syncthreads();
    if (w == 0 && row < M) {
#pragma unroll
        for (int k = 1; k < MERGE_WARPS; ++k) {
            const float om = part[k][lane].x;
            const int oa = __float_as_int(part[k][lane].y);
            if (om > mx || (om == mx && oa < arg)) { mx = om; arg = oa; }
        }
        max_out[row] = mx;
        if (argmax_out) argmax_out[row] = arg;
    }
}

// Finishes EPI_SOFTMAX: turns the unnormalised exponentials in out into probabilities -- every element is multiplied
// by exp(max of its piece - lse of its row), the piece being the (column tile, tail piece, share of the piece) whose
// epilogue thread wrote it.  One warp per row and span of column tiles; 16 bytes per lane and step where the pitch
// allows, four tiles' loads in flight.  MERGE = false: lse_merge_rows_kernel has left the rows' lse in `lse`.
// MERGE = true (rows of few pieces): every warp merges its row's (max, sum-exp) partials itself first, lanes striding
// the column tiles, and the first span's warp writes the lse if the caller wants it -- one launch less.
template <bool OUT_BF16, bool MERGE>
__global__ void softmax_finish_kernel(void* __restrict__ out, int ldo, const float2* __restrict__ partial,
                                      float* __restrict__ lse, int M, int N, int rows_per_tile, int m_tiles, int n_tiles,
                                      int group_m, int n_full, int tail_split, int out_tile_n, int tiles_per_span) {
    pdl_launch_dependents();
    pdl_wait();                  // launched as a programmatic dependent of the kernel that wrote the partials / the lse
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= M) return;
    const int mb = row / rows_per_tile;
    float l;
    if (MERGE) {
        float mx = -INFINITY, sum = 0.0f;
        for (int nb = lane; nb < n_tiles; nb += 32) {
            const int pieces = tile_index(group_m, m_tiles, n_tiles, mb, nb) < n_full ? 1 : tail_split;
            for (int sl = 0; sl < EPI_HALVES * pieces; ++sl) {    // ascending columns
                const float2 v = __ldcg(partial + static_cast<size_t>(nb * tail_split * EPI_HALVES + sl) * M + row);
                lse_combine(mx, sum, v.x, v.y);
            }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float om = __shfl_xor_sync(0xffffffffu, mx, off);
            const float os = __shfl_xor_sync(0xffffffffu, sum, off);
            lse_combine(mx, sum, om, os);
        }
        l = __shfl_sync(0xffffffffu, mx + __logf(sum), 0);
        if (blockIdx.y == 0 && lane == 0 && lse) lse[row] = l;
    } else {
        l = __ldcg(lse + row);
    }

    constexpr int PER = OUT_BF16 ? 8 : 4;                    // elements per 16 bytes
    constexpr int UNROLL = 4;                                // tiles in flight
    constexpr int UPL = OUT_BF16 ? 1 : 2;                    // 16-byte units of a 256-column tile per lane
    const size_t elem = OUT_BF16 ? 2 : 4;
    uint8_t* base = reinterpret_cast<uint8_t*>(out) + static_cast<size_t>(row) * ldo * elem;
    const bool vec = (ldo % PER == 0) && ((reinterpret_cast<uintptr_t>(out) & 15u) == 0);
    const int nb_first = blockIdx.y * tiles_per_span, nb_last = min(n_tiles, nb_first + tiles_per_span);
    const int n_vec = vec ? (N / PER) * PER : 0;             // columns below n_vec travel as whole 16-byte units
    // the partial of the piece of tile nb that holds the tile's column in_tile
    auto piece_of = [&](int nb, int pieces, int in_tile) -> const float2* {
        const int width = out_tile_n / pieces;
        const int sub = in_tile / width;
        const int chunk = (in_tile - sub * width) >> 5, chunks = width >> 5;
        const int half = (EPI_HALVES == 2 && chunk >= (chunks + 1) / 2) ? 1 : 0;
        return partial + static_cast<size_t>((nb * tail_split + sub) * EPI_HALVES + half) * M + row;
    };
    const int units = out_tile_n / PER;                      // 16-byte units per tile: 16, 32 or 64
    for (int nb0 = nb_first; nb0 < nb_last; nb0 += UNROLL) {
        uint4 q[UNROLL][UPL];
        float pm[UNROLL][UPL];                               // the pieces' maxima, fetched while the data is on its way
#pragma unroll
        for (int u = 0; u < UNROLL; ++u)
#pragma unroll
            for (int k = 0; k < UPL; ++k) {
                const int unit = lane + 32 * k, col = (nb0 + u) * out_tile_n + unit * PER;
                if (nb0 + u < nb_last && unit < units && col < n_vec) q[u][k] = __ldcs(reinterpret_cast<const uint4*>(base + col * elem));
            }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int nb = nb0 + u;
            if (nb >= nb_last) break;
            const int pieces = tile_index(group_m, m_tiles, n_tiles, mb, nb) < n_full ? 1 : tail_split;
#pragma unroll
            for (int k = 0; k < UPL; ++k) {
                const int unit = lane + 32 * k;
                if (unit < units && nb * out_tile_n + unit * PER < n_vec) pm[u][k] = __ldcg(piece_of(nb, pieces, unit * PER)).x;   // 16 bytes lie inside one 32-column chunk
            }
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int nb = nb0 + u;
            if (nb >= nb_last) break;
#pragma unroll
            for (int k = 0; k < UPL; ++k) {
                const int unit = lane + 32 * k, col = nb * out_tile_n + unit * PER;
                if (unit >= units || col >= n_vec) continue;
                const float f = __expf(pm[u][k] - l);
                uint32_t w[4] = {q[u][k].x, q[u][k].y, q[u][k].z, q[u][k].w};
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    if (OUT_BF16) w[h] = pack_bf16x2(__uint_as_float(w[h] << 16) * f, __uint_as_float(w[h] & 0xffff0000u) * f);
                    else w[h] = __float_as_uint(__uint_as_float(w[h]) * f);
                }
                *reinterpret_cast<uint4*>(base + col * elem) = make_uint4(w[0], w[1], w[2], w[3]);
            }
        }
    }
    // what does not travel as 16-byte units: the last N mod PER columns, or every column of an unaligned output
    const int c_first = max(n_vec, nb_first * out_tile_n), c_last = min(N, nb_last * out_tile_n);
    for (int c = c_first + lane; c < c_last; c += 32) {
        const int nb = c / out_tile_n;
        const int pieces = tile_index(group_m, m_tiles, n_tiles, mb, nb) < n_full ? 1 : tail_split;
        const float f = __expf(__ldcg(piece_of(nb, pieces, c - nb * out_tile_n)).x - l);
        if (OUT_BF16) {
            __nv_bfloat16* e = reinterpret_cast<__nv_bfloat16*>(base) + c;
            *e = __float2bfloat16_rn(__bfloat162float(*e) * f);
        } else {
            reinterpret_cast<float*>(base)[c] *= f;
        }
    }
}

}  // namespace mtmc
