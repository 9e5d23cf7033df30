// libmtmcref -- the fp64 CPU oracle for the fused-linear hot path.
//
// THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  Only the test-suite, the smoke
// check and the benchmark's cpu_baseline / reference legs may load it.  It shares
// no code, header, table or constant with the CUDA library and includes no CUDA
// header.  It is deliberately plain and slow: every output is the textbook
// definition written out, in double precision, from the same bf16-rounded inputs
// the GPU sees.  Nothing here is blocked, fused or reordered.
//
// What it computes (the operator family the paper's Level-2 "fused ops" class
// stands for -- a GEMM followed by an epilogue, Table "Details of KernelBench and
// TritonBench"; correctness per the paper's Eq. 1 means equality with the
// high-level reference semantics, which for these operators is):
//
//   z[m][n]  = sum_{k=0..K-1} X[m][k] * W[n][k]  (+ b[n])        "X . W^T + b"
//   fused linear :  Y[m][n] = act(z[m][n]),  act in {identity, ReLU, GELU-tanh, SiLU}
//   + residual   :  Y[m][n] = act(z[m][n]) + R[m][n]   (the layer's skip connection joined to the epilogue)
//   FP8 linear   :  Y[m][n] = act( sx*sw * sum_k Xq[m][k] Wq[n][k] + b[n] ),  Xq, Wq 8-bit floats
//                   (E4M3: 1 sign, 4 exponent bits with bias 7, 3 mantissa bits, no infinities),
//                   sx, sw per-tensor scales: the lower-precision variant of the same layer
//   MXFP8 linear :  the same with block scales instead of per-tensor ones (the microscaling format MXFP8):
//                   z[m][n] = sum_k (2^(SX[m][k/32]-127) Xq[m][k]) (2^(SW[n][k/32]-127) Wq[n][k]) + b[n],
//                   Xq, Wq E4M3, SX [M,K/32] and SW [N,K/32] one biased power-of-two exponent (UE8M0) per
//                   32 consecutive elements of K; also as SwiGLU gate and as row logsumexp
//   SwiGLU       :  out[m][n] = silu(g[m][n]) * u[m][n],  g = X.Wg^T, u = X.Wu^T (no bias)
//   row LSE      :  lse[m] = log( sum_n exp(z[m][n]) ), computed two-pass (max, then sum)
//   row max      :  mx[m] = max_n z[m][n], arg[m] = the lowest n attaining it
//                   (the paper's own example of a fusion action joins a linear with a row max,
//                   section "Training Process")
//   cross entropy:  loss[m] = lse[m] - z[m][target[m]]   (softmax cross entropy of the logits row)
//   row softmax  :  P[m][n] = exp(z[m][n] - max_n' z[m][n']) / sum_n' exp(z[m][n'] - max), the normalised
//                   form of the same row reduction (also with E4M3 operands and per-tensor scales)
//
// Layouts: X [M,K], W [N,K], out [M,N]; all dense row-major.  X/W arrive as bf16 bit
// patterns (uint16_t: the upper half of an IEEE-754 binary32), b as binary32 and
// is NOT bf16-rounded.  Outputs are double and are never rounded to the GPU's
// output type: the comparator applies |got - ref| <= atol + rtol*|ref| instead.
//
// Pins (see tests/test_oracle_pins.py): exact rational brute force on tiny
// integer-valued problems, W = I, X = 0, K-split additivity, permutation and
// scaling laws, closed-form activation and logsumexp values, act(z)-act(-z) = z,
// lse(z+c) = lse(z)+c, softmax rows summing to one, softmax of log-integers as exact
// ratios, the two-class softmax as the logistic function, and torch fp64 library
// routines.  No function here is "parity unpinned".
#include <cmath>
#include <cstdint>
#include <cstring>
#include <thread>
#include <vector>
#include <algorithm>
#include <limits>

namespace {

int g_threads = 0;  // 0 = std::thread::hardware_concurrency()

int thread_count() {
    if (g_threads > 0) return g_threads;
    unsigned hc = std::thread::hardware_concurrency();
    return hc == 0 ? 1 : static_cast<int>(hc);
}

// bf16 bit pattern -> double.  Exact: bf16 is the top 16 bits of a binary32.
double bf16_to_double(uint16_t bits) {
    uint32_t u = static_cast<uint32_t>(bits) << 16;
    float f;
    std::memcpy(&f, &u, sizeof f);
    return static_cast<double>(f);
}

// E4M3 bit pattern -> double, exactly.  exponent field 0: subnormal m/8 * 2^-6; otherwise
// (1 + m/8) * 2^(e-7); the pattern S.1111.111 is NaN (the format has no infinities).
double e4m3_to_double(uint8_t bits) {
    const int sign = bits >> 7, e = (bits >> 3) & 15, m = bits & 7;
    double v;
    if (e == 15 && m == 7) v = std::numeric_limits<double>::quiet_NaN();
    else if (e == 0) v = std::ldexp(static_cast<double>(m) / 8.0, -6);
    else v = std::ldexp(1.0 + static_cast<double>(m) / 8.0, e - 7);
    return sign ? -v : v;
}

// UE8M0 scale byte -> double, exactly: an unsigned biased exponent, 2^(e - 127); 255 is NaN.
double e8m0_to_double(uint8_t e) {
    if (e == 255) return std::numeric_limits<double>::quiet_NaN();
    return std::ldexp(1.0, static_cast<int>(e) - 127);
}

// One block-scaled dot product: every element is decoded and multiplied by its block's scale first (exact in
// double: an E4M3 value times a power of two), then the products are summed in ascending k.
double dot_row_mx(const uint8_t* x, const uint8_t* sx, const uint8_t* w, const uint8_t* sw, int64_t K) {
    double acc = 0.0;
    for (int64_t k = 0; k < K; ++k)
        acc += (e8m0_to_double(sx[k / 32]) * e4m3_to_double(x[k])) * (e8m0_to_double(sw[k / 32]) * e4m3_to_double(w[k]));
    return acc;
}

// One pre-activation value: ascending k, one double accumulator, bias added last.
double dot_row(const uint16_t* x, const uint16_t* w, int64_t K) {
    double acc = 0.0;
    for (int64_t k = 0; k < K; ++k) acc += bf16_to_double(x[k]) * bf16_to_double(w[k]);
    return acc;
}

double preact(const uint16_t* X, const uint16_t* W, const float* b, int64_t K, int64_t m, int64_t n) {
    double z = dot_row(X + m * K, W + n * K, K);
    if (b != nullptr) z += static_cast<double>(b[n]);
    return z;
}

// Activations, in double.  GELU is the tanh form (what "GELU-tanh" names):
//   0.5 z (1 + tanh( sqrt(2/pi) (z + 0.044715 z^3) ))
double act_apply(int act, double z) {
    switch (act) {
        case 0: return z;
        case 1: return z > 0.0 ? z : 0.0;
        case 2: {
            const double c0 = std::sqrt(2.0 / M_PI);
            return 0.5 * z * (1.0 + std::tanh(c0 * (z + 0.044715 * z * z * z)));
        }
        case 3: return z / (1.0 + std::exp(-z));
        default: return std::numeric_limits<double>::quiet_NaN();
    }
}

// Run fn(i) for i in [0, count) over the worker threads, contiguous chunks.
template <class F>
void parallel_for(int64_t count, F fn) {
    int nt = thread_count();
    if (count < 2 || nt < 2) {
        for (int64_t i = 0; i < count; ++i) fn(i);
        return;
    }
    if (nt > count) nt = static_cast<int>(count);
    std::vector<std::thread> pool;
    pool.reserve(nt);
    for (int t = 0; t < nt; ++t) {
        int64_t lo = count * t / nt, hi = count * (t + 1) / nt;
        pool.emplace_back([=]() { for (int64_t i = lo; i < hi; ++i) fn(i); });
    }
    for (auto& th : pool) th.join();
}

}  // namespace

extern "C" {

// Number of worker threads (0 restores the default = hardware concurrency).
void mtmc_ref_set_threads(int n) { g_threads = n; }
int mtmc_ref_get_threads(void) { return thread_count(); }

// act ids: 0 identity, 1 ReLU, 2 GELU-tanh, 3 SiLU.  Scalar entry for the pins.
double mtmc_ref_act(int act, double z) { return act_apply(act, z); }

// Y = act(X.W^T + b), full output [M,N] in double.  b may be null (zero bias).
int mtmc_ref_fused_linear(const uint16_t* X, const uint16_t* W, const float* b,
                          int64_t M, int64_t N, int64_t K, int act, double* out) {
    if (!X || !W || !out || M <= 0 || N <= 0 || K <= 0 || act < 0 || act > 3) return 1;
    parallel_for(M, [=](int64_t m) {
        for (int64_t n = 0; n < N; ++n) out[m * N + n] = act_apply(act, preact(X, W, b, K, m, n));
    });
    return 0;
}

// Y = act(X.W^T + b) + R.  R is [M,N], either bf16 bit patterns (r_is_bf16 != 0) or binary32.
int mtmc_ref_fused_linear_residual(const uint16_t* X, const uint16_t* W, const float* b, const void* R, int r_is_bf16,
                                   int64_t M, int64_t N, int64_t K, int act, double* out) {
    if (!X || !W || !R || !out || M <= 0 || N <= 0 || K <= 0 || act < 0 || act > 3) return 1;
    parallel_for(M, [=](int64_t m) {
        for (int64_t n = 0; n < N; ++n) {
            const double r = r_is_bf16 ? bf16_to_double(static_cast<const uint16_t*>(R)[m * N + n])
                                       : static_cast<double>(static_cast<const float*>(R)[m * N + n]);
            out[m * N + n] = act_apply(act, preact(X, W, b, K, m, n)) + r;
        }
    });
    return 0;
}

// Scalar decode of one E4M3 pattern (for the pins).
double mtmc_ref_e4m3(uint8_t bits) { return e4m3_to_double(bits); }

// Y = act(sx*sw * Xq.Wq^T + b) with E4M3 operands (one byte per element), full output in double.
int mtmc_ref_fused_linear_fp8(const uint8_t* X, const uint8_t* W, const float* b, float scale_x, float scale_w,
                              int64_t M, int64_t N, int64_t K, int act, double* out) {
    if (!X || !W || !out || M <= 0 || N <= 0 || K <= 0 || act < 0 || act > 3) return 1;
    const double scale = static_cast<double>(scale_x) * static_cast<double>(scale_w);
    parallel_for(M, [=](int64_t m) {
        for (int64_t n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int64_t k = 0; k < K; ++k) acc += e4m3_to_double(X[m * K + k]) * e4m3_to_double(W[n * K + k]);
            double z = scale * acc;
            if (b) z += static_cast<double>(b[n]);
            out[m * N + n] = act_apply(act, z);
        }
    });
    return 0;
}

// The same at P listed (row, col) positions.
int mtmc_ref_fused_linear_fp8_points(const uint8_t* X, const uint8_t* W, const float* b, float scale_x, float scale_w,
                                     int64_t M, int64_t N, int64_t K, int act,
                                     const int64_t* rows, const int64_t* cols, int64_t P, double* out) {
    if (!X || !W || !out || !rows || !cols || M <= 0 || N <= 0 || K <= 0 || act < 0 || act > 3) return 1;
    for (int64_t p = 0; p < P; ++p)
        if (rows[p] < 0 || rows[p] >= M || cols[p] < 0 || cols[p] >= N) return 1;
    const double scale = static_cast<double>(scale_x) * static_cast<double>(scale_w);
    parallel_for(P, [=](int64_t p) {
        const int64_t m = rows[p], n = cols[p];
        double acc = 0.0;
        for (int64_t k = 0; k < K; ++k) acc += e4m3_to_double(X[m * K + k]) * e4m3_to_double(W[n * K + k]);
        double z = scale * acc;
        if (b) z += static_cast<double>(b[n]);
        out[p] = act_apply(act, z);
    });
    return 0;
}

// The same definition evaluated only at P listed (row, col) positions.
int mtmc_ref_fused_linear_points(const uint16_t* X, const uint16_t* W, const float* b,
                                 int64_t M, int64_t N, int64_t K, int act,
                                 const int64_t* rows, const int64_t* cols, int64_t P, double* out) {
    if (!X || !W || !out || !rows || !cols || M <= 0 || N <= 0 || K <= 0 || act < 0 || act > 3) return 1;
    for (int64_t p = 0; p < P; ++p)
        if (rows[p] < 0 || rows[p] >= M || cols[p] < 0 || cols[p] >= N) return 1;
    parallel_for(P, [=](int64_t p) { out[p] = act_apply(act, preact(X, W, b, K, rows[p], cols[p])); });
    return 0;
}

// out = silu(X.Wg^T) * (X.Wu^T), no bias, full output [M,N] in double.
int mtmc_ref_swiglu(const uint16_t* X, const uint16_t* Wg, const uint16_t* Wu,
                    int64_t M, int64_t N, int64_t K, double* out) {
    if (!X || !Wg || !Wu || !out || M <= 0 || N <= 0 || K <= 0) return 1;
    parallel_for(M, [=](int64_t m) {
        for (int64_t n = 0; n < N; ++n) {
            double g = dot_row(X + m * K, Wg + n * K, K);
            double u = dot_row(X + m * K, Wu + n * K, K);
            out[m * N + n] = act_apply(3, g) * u;
        }
    });
    return 0;
}

int mtmc_ref_swiglu_points(const uint16_t* X, const uint16_t* Wg, const uint16_t* Wu,
                           int64_t M, int64_t N, int64_t K,
                           const int64_t* rows, const int64_t* cols, int64_t P, double* out) {
    if (!X || !Wg || !Wu || !out || !rows || !cols || M <= 0 || N <= 0 || K <= 0) return 1;
    for (int64_t p = 0; p < P; ++p)
        if (rows[p] < 0 || rows[p] >= M || cols[p] < 0 || cols[p] >= N) return 1;
    parallel_for(P, [=](int64_t p) {
        double g = dot_row(X + rows[p] * K, Wg + cols[p] * K, K);
        double u = dot_row(X + rows[p] * K, Wu + cols[p] * K, K);
        out[p] = act_apply(3, g) * u;
    });
    return 0;
}

// out = silu(sx*sg * Xq.Wgq^T) * (sx*su * Xq.Wuq^T) with E4M3 operands: the SwiGLU gate of an FP8 layer whose
// gate and up projections carry their own per-tensor scales.
int mtmc_ref_swiglu_fp8(const uint8_t* X, const uint8_t* Wg, const uint8_t* Wu, float scale_x, float scale_g, float scale_u,
                        int64_t M, int64_t N, int64_t K, double* out) {
    if (!X || !Wg || !Wu || !out || M <= 0 || N <= 0 || K <= 0) return 1;
    const double sg = static_cast<double>(scale_x) * static_cast<double>(scale_g);
    const double su = static_cast<double>(scale_x) * static_cast<double>(scale_u);
    parallel_for(M, [=](int64_t m) {
        for (int64_t n = 0; n < N; ++n) {
            double g = 0.0, u = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                const double x = e4m3_to_double(X[m * K + k]);
                g += x * e4m3_to_double(Wg[n * K + k]);
                u += x * e4m3_to_double(Wu[n * K + k]);
            }
            out[m * N + n] = act_apply(3, sg * g) * (su * u);
        }
    });
    return 0;
}

// One row of logits -> its logsumexp, two passes: the maximum, then the sum of
// exp(z - max) in ascending n, then max + log(sum).
static double lse_of_row(const double* z, int64_t N) {
    double mx = z[0];
    for (int64_t n = 1; n < N; ++n) mx = z[n] > mx ? z[n] : mx;
    double s = 0.0;
    for (int64_t n = 0; n < N; ++n) s += std::exp(z[n] - mx);
    return mx + std::log(s);
}

// lse[m] = log sum_n exp(z[m][n]).  If logits != null the [M,N] pre-activations are
// also written there (for the softmax-sums-to-one check).
int mtmc_ref_linear_lse(const uint16_t* X, const uint16_t* W, const float* b,
                        int64_t M, int64_t N, int64_t K, double* lse, double* logits) {
    if (!X || !W || !lse || M <= 0 || N <= 0 || K <= 0) return 1;
    parallel_for(M, [=](int64_t m) {
        std::vector<double> z(static_cast<size_t>(N));
        for (int64_t n = 0; n < N; ++n) z[n] = preact(X, W, b, K, m, n);
        if (logits) std::copy(z.begin(), z.end(), logits + m * N);
        lse[m] = lse_of_row(z.data(), N);
    });
    return 0;
}

// lse[m] = log sum_n exp(sx*sw * Xq.Wq^T + b) with E4M3 operands; logits as above.
int mtmc_ref_linear_lse_fp8(const uint8_t* X, const uint8_t* W, const float* b, float scale_x, float scale_w,
                            int64_t M, int64_t N, int64_t K, double* lse, double* logits) {
    if (!X || !W || !lse || M <= 0 || N <= 0 || K <= 0) return 1;
    const double scale = static_cast<double>(scale_x) * static_cast<double>(scale_w);
    parallel_for(M, [=](int64_t m) {
        std::vector<double> z(static_cast<size_t>(N));
        for (int64_t n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int64_t k = 0; k < K; ++k) acc += e4m3_to_double(X[m * K + k]) * e4m3_to_double(W[n * K + k]);
            z[n] = scale * acc + (b ? static_cast<double>(b[n]) : 0.0);
        }
        if (logits) std::copy(z.begin(), z.end(), logits + m * N);
        lse[m] = lse_of_row(z.data(), N);
    });
    return 0;
}

// The same for R listed rows only: lse[r] belongs to row rows[r].
int mtmc_ref_linear_lse_rows(const uint16_t* X, const uint16_t* W, const float* b,
                             int64_t M, int64_t N, int64_t K,
                             const int64_t* rows, int64_t R, double* lse) {
    if (!X || !W || !lse || !rows || M <= 0 || N <= 0 || K <= 0) return 1;
    for (int64_t r = 0; r < R; ++r)
        if (rows[r] < 0 || rows[r] >= M) return 1;
    // Columns of one row are spread over the threads; the two-pass reduction runs after.
    for (int64_t r = 0; r < R; ++r) {
        std::vector<double> z(static_cast<size_t>(N));
        double* zp = z.data();
        int64_t m = rows[r];
        parallel_for(N, [=](int64_t n) { zp[n] = preact(X, W, b, K, m, n); });
        lse[r] = lse_of_row(zp, N);
    }
    return 0;
}

// One row of logits -> its softmax by the definition with the maximum taken out first:
// p[n] = exp(z[n] - max) / sum_n' exp(z[n'] - max), the sum in ascending n'.
static void softmax_of_row(const double* z, int64_t N, double* p) {
    double mx = z[0];
    for (int64_t n = 1; n < N; ++n) mx = z[n] > mx ? z[n] : mx;
    double s = 0.0;
    for (int64_t n = 0; n < N; ++n) { p[n] = std::exp(z[n] - mx); s += p[n]; }
    for (int64_t n = 0; n < N; ++n) p[n] /= s;
}

// P[m][n] = softmax over n of z[m][n] = X.W^T + b, all M rows.
int mtmc_ref_linear_softmax(const uint16_t* X, const uint16_t* W, const float* b,
                            int64_t M, int64_t N, int64_t K, double* P) {
    if (!X || !W || !P || M <= 0 || N <= 0 || K <= 0) return 1;
    parallel_for(M, [=](int64_t m) {
        std::vector<double> z(static_cast<size_t>(N));
        for (int64_t n = 0; n < N; ++n) z[n] = preact(X, W, b, K, m, n);
        softmax_of_row(z.data(), N, P + m * N);
    });
    return 0;
}

// The same for R listed rows only: P[r][·] belongs to row rows[r].
int mtmc_ref_linear_softmax_rows(const uint16_t* X, const uint16_t* W, const float* b,
                                 int64_t M, int64_t N, int64_t K,
                                 const int64_t* rows, int64_t R, double* P) {
    if (!X || !W || !P || !rows || M <= 0 || N <= 0 || K <= 0) return 1;
    for (int64_t r = 0; r < R; ++r)
        if (rows[r] < 0 || rows[r] >= M) return 1;
    for (int64_t r = 0; r < R; ++r) {
        std::vector<double> z(static_cast<size_t>(N));
        double* zp = z.data();
        int64_t m = rows[r];
        parallel_for(N, [=](int64_t n) { zp[n] = preact(X, W, b, K, m, n); });
        softmax_of_row(zp, N, P + r * N);
    }
    return 0;
}

// Softmax of a plain vector (for the closed-form pins).
void mtmc_ref_softmax_vector(const double* z, int64_t N, double* p) { softmax_of_row(z, N, p); }

// mx[m] = max_n z[m][n]; arg[m] = lowest column index attaining it.  arg may be null.
int mtmc_ref_linear_rowmax(const uint16_t* X, const uint16_t* W, const float* b,
                           int64_t M, int64_t N, int64_t K, double* mx, int64_t* arg) {
    if (!X || !W || !mx || M <= 0 || N <= 0 || K <= 0) return 1;
    parallel_for(M, [=](int64_t m) {
        double best = preact(X, W, b, K, m, 0);
        int64_t where = 0;
        for (int64_t n = 1; n < N; ++n) {
            double z = preact(X, W, b, K, m, n);
            if (z > best) { best = z; where = n; }
        }
        mx[m] = best;
        if (arg) arg[m] = where;
    });
    return 0;
}

// loss[m] = lse[m] - z[m][target[m]], lse as in mtmc_ref_linear_lse (two-pass).  lse_out may be null.
int mtmc_ref_linear_cross_entropy(const uint16_t* X, const uint16_t* W, const float* b, const int64_t* target,
                                  int64_t M, int64_t N, int64_t K, double* loss, double* lse_out) {
    if (!X || !W || !target || !loss || M <= 0 || N <= 0 || K <= 0) return 1;
    for (int64_t m = 0; m < M; ++m)
        if (target[m] < 0 || target[m] >= N) return 1;
    parallel_for(M, [=](int64_t m) {
        std::vector<double> z(static_cast<size_t>(N));
        for (int64_t n = 0; n < N; ++n) z[n] = preact(X, W, b, K, m, n);
        const double l = lse_of_row(z.data(), N);
        loss[m] = l - z[target[m]];
        if (lse_out) lse_out[m] = l;
    });
    return 0;
}

// One pre-activation of the E4M3 layer: sx*sw * sum_k xq[m][k] wq[n][k] + b[n].
static double preact_fp8(const uint8_t* X, const uint8_t* W, const float* b, double scale, int64_t K, int64_t m, int64_t n) {
    double acc = 0.0;
    for (int64_t k = 0; k < K; ++k) acc += e4m3_to_double(X[m * K + k]) * e4m3_to_double(W[n * K + k]);
    return scale * acc + (b ? static_cast<double>(b[n]) : 0.0);
}

// Row softmax of the E4M3 layer's logits: P[m][n] = softmax over n of sx*sw * Xq.Wq^T + b.
int mtmc_ref_linear_softmax_fp8(const uint8_t* X, const uint8_t* W, const float* b, float scale_x, float scale_w,
                                int64_t M, int64_t N, int64_t K, double* P) {
    if (!X || !W || !P || M <= 0 || N <= 0 || K <= 0) return 1;
    const double scale = static_cast<double>(scale_x) * static_cast<double>(scale_w);
    parallel_for(M, [=](int64_t m) {
        std::vector<double> z(static_cast<size_t>(N));
        for (int64_t n = 0; n < N; ++n) z[n] = preact_fp8(X, W, b, scale, K, m, n);
        softmax_of_row(z.data(), N, P + m * N);
    });
    return 0;
}

// Row maximum and the lowest column attaining it, E4M3 operands.
int mtmc_ref_linear_rowmax_fp8(const uint8_t* X, const uint8_t* W, const float* b, float scale_x, float scale_w,
                               int64_t M, int64_t N, int64_t K, double* mx, int64_t* arg) {
    if (!X || !W || !mx || M <= 0 || N <= 0 || K <= 0) return 1;
    const double scale = static_cast<double>(scale_x) * static_cast<double>(scale_w);
    parallel_for(M, [=](int64_t m) {
        double best = preact_fp8(X, W, b, scale, K, m, 0);
        int64_t where = 0;
        for (int64_t n = 1; n < N; ++n) {
            const double z = preact_fp8(X, W, b, scale, K, m, n);
            if (z > best) { best = z; where = n; }
        }
        mx[m] = best;
        if (arg) arg[m] = where;
    });
    return 0;
}

// loss[m] = lse[m] - z[m][target[m]], E4M3 operands; lse_out may be null.
int mtmc_ref_linear_cross_entropy_fp8(const uint8_t* X, const uint8_t* W, const float* b, float scale_x, float scale_w,
                                      const int64_t* target, int64_t M, int64_t N, int64_t K, double* loss, double* lse_out) {
    if (!X || !W || !target || !loss || M <= 0 || N <= 0 || K <= 0) return 1;
    for (int64_t m = 0; m < M; ++m)
        if (target[m] < 0 || target[m] >= N) return 1;
    const double scale = static_cast<double>(scale_x) * static_cast<double>(scale_w);
    parallel_for(M, [=](int64_t m) {
        std::vector<double> z(static_cast<size_t>(N));
        for (int64_t n = 0; n < N; ++n) z[n] = preact_fp8(X, W, b, scale, K, m, n);
        const double l = lse_of_row(z.data(), N);
        loss[m] = l - z[target[m]];
        if (lse_out) lse_out[m] = l;
    });
    return 0;
}

// logsumexp of a plain vector of doubles (pins: closed forms, shift law).
double mtmc_ref_lse_vector(const double* z, int64_t N) { return lse_of_row(z, N); }

// Scalar decode of one UE8M0 scale byte (for the pins).
double mtmc_ref_e8m0(uint8_t e) { return e8m0_to_double(e); }

// Y = act(z + b) with block-scaled E4M3 operands: X [M,K], SX [M,K/32], W [N,K], SW [N,K/32]; K % 32 == 0.
int mtmc_ref_fused_linear_mxfp8(const uint8_t* X, const uint8_t* SX, const uint8_t* W, const uint8_t* SW, const float* b,
                                int64_t M, int64_t N, int64_t K, int act, double* out) {
    if (!X || !SX || !W || !SW || !out || M <= 0 || N <= 0 || K <= 0 || K % 32 != 0 || act < 0 || act > 3) return 1;
    const int64_t KB = K / 32;
    parallel_for(M, [=](int64_t m) {
        for (int64_t n = 0; n < N; ++n) {
            double z = dot_row_mx(X + m * K, SX + m * KB, W + n * K, SW + n * KB, K);
            if (b) z += static_cast<double>(b[n]);
            out[m * N + n] = act_apply(act, z);
        }
    });
    return 0;
}

// out = silu(z_gate) * z_up with block-scaled E4M3 operands; gate and up weights with their own scales.
int mtmc_ref_swiglu_mxfp8(const uint8_t* X, const uint8_t* SX, const uint8_t* Wg, const uint8_t* SG, const uint8_t* Wu, const uint8_t* SU,
                          int64_t M, int64_t N, int64_t K, double* out) {
    if (!X || !SX || !Wg || !SG || !Wu || !SU || !out || M <= 0 || N <= 0 || K <= 0 || K % 32 != 0) return 1;
    const int64_t KB = K / 32;
    parallel_for(M, [=](int64_t m) {
        for (int64_t n = 0; n < N; ++n) {
            const double g = dot_row_mx(X + m * K, SX + m * KB, Wg + n * K, SG + n * KB, K);
            const double u = dot_row_mx(X + m * K, SX + m * KB, Wu + n * K, SU + n * KB, K);
            out[m * N + n] = act_apply(3, g) * u;
        }
    });
    return 0;
}

// lse[m] = log sum_n exp(z[m][n] + b[n]) with block-scaled E4M3 operands (two passes, as for bf16).
int mtmc_ref_linear_lse_mxfp8(const uint8_t* X, const uint8_t* SX, const uint8_t* W, const uint8_t* SW, const float* b,
                              int64_t M, int64_t N, int64_t K, double* lse) {
    if (!X || !SX || !W || !SW || !lse || M <= 0 || N <= 0 || K <= 0 || K % 32 != 0) return 1;
    const int64_t KB = K / 32;
    parallel_for(M, [=](int64_t m) {
        std::vector<double> z(static_cast<size_t>(N));
        for (int64_t n = 0; n < N; ++n)
            z[n] = dot_row_mx(X + m * K, SX + m * KB, W + n * K, SW + n * KB, K) + (b ? static_cast<double>(b[n]) : 0.0);
        lse[m] = lse_of_row(z.data(), N);
    });
    return 0;
}

// Element-wise comparator.  got/ref are double (the caller widens the GPU result
// exactly).  An element passes when |got-ref| <= atol + rtol*|ref| and both are
// finite.  stats[0] = max |err|, stats[1] = max err/(atol+rtol|ref|),
// stats[2] = index of that worst ratio, stats[3] = number of violations.
// Returns the number of violations (0 = pass), or -1 on bad arguments.
int64_t mtmc_ref_compare(const double* got, const double* ref, int64_t count,
                         double atol, double rtol, double* stats) {
    if (!got || !ref || count < 0) return -1;
    double max_err = 0.0, max_ratio = 0.0;
    int64_t worst = -1, bad = 0;
    for (int64_t i = 0; i < count; ++i) {
        double g = got[i], r = ref[i];
        if (!std::isfinite(g) || !std::isfinite(r)) {
            ++bad;
            worst = worst < 0 ? i : worst;
            max_ratio = std::numeric_limits<double>::infinity();
            continue;
        }
        double err = std::fabs(g - r), bound = atol + rtol * std::fabs(r);
        double ratio = bound > 0.0 ? err / bound : (err > 0.0 ? std::numeric_limits<double>::infinity() : 0.0);
        if (err > max_err) max_err = err;
        if (ratio > max_ratio) { max_ratio = ratio; worst = i; }
        if (err > bound) ++bad;
    }
    if (stats) { stats[0] = max_err; stats[1] = max_ratio; stats[2] = static_cast<double>(worst); stats[3] = static_cast<double>(bad); }
    return bad;
}

}  // extern "C"
