// QLLM quantized-linear oracle  --  TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, single-threaded CPU statement of what the quantized linear
// layer of QLLM (arXiv 2310.08041) computes, written from the paper:
//   LayerNorm -> channel reassembly (Eq. 3 disassembly, Eq. 4 assembly, as a
//   sparse map) -> per-token asymmetric b-bit quantization (Eq. 2) -> integer
//   matmul (Eq. 1 on codes) -> dequantizing epilogue (Eq. 2 inverted),
// plus the offline side: sub-channel counts T = ceil(max|x|/theta) (Sec. 4.1.1),
// bipartite soft matching (Appendix A) and the weight transform
// (Appendix B; quant(W + AB) of Sec. 4.2).
//
// Internals are fp64; stored outputs have the types of the library boundary.
// Nothing here is blocked, fused, vectorised or threaded.  It shares no code
// with the CUDA library and must never be called from the product path: only
// tests, the smoke check and the benchmark's CPU-baseline leg may use it.
//
// Notation: tokens M, input channels C (= K of the GEMM), output channels N.
// (The paper writes M for input channels and N for output channels in Eq. 1.)
//
// Parity pins (tests/test_oracle_pins.py): every function below is pinned to
// something other than itself; none is "parity unpinned".

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <numeric>
#include <vector>

namespace {

inline double widen_bf16(uint16_t h) {
    uint32_t u = static_cast<uint32_t>(h) << 16;
    float f;
    std::memcpy(&f, &u, 4);
    return static_cast<double>(f);
}

inline double load_x(const void* x, int dtype, int64_t idx) {
    if (dtype == 0) return static_cast<double>(static_cast<const float*>(x)[idx]);
    return widen_bf16(static_cast<const uint16_t*>(x)[idx]);
}

// Nearest bfloat16 (round-half-to-even) of a double in the normal range,
// returned as the bit pattern.  Values below the smallest normal flush through
// the float cast (not met by this path's outputs).
uint16_t round_to_bf16(double v) {
    if (std::isnan(v)) return 0x7FC0;
    if (v == 0.0) return std::signbit(v) ? 0x8000 : 0x0000;
    if (std::isinf(v)) return v > 0 ? 0x7F80 : 0xFF80;
    int e;
    double m = std::frexp(v, &e);          // v = m * 2^e, 0.5 <= |m| < 1
    double r = v;
    if (e >= -125)                         // normal bf16: 8 significant bits
        r = std::ldexp(std::nearbyint(std::ldexp(m, 8)), e - 8);
    float f = static_cast<float>(r);
    uint32_t u;
    std::memcpy(&u, &f, 4);
    if (e < -125) {                        // subnormal range: round the float's low half to even
        uint32_t bias = ((u >> 16) & 1u) + 0x7FFFu;
        u += bias;
    }
    return static_cast<uint16_t>(u >> 16);
}

struct Entry {                 // one position of the (expanded / partly merged) channel list
    std::vector<int> members;  // source channels, in entry order
    bool is_sub;               // produced by disassembly (T > 1): never assembled
    int T;                     // split count of the source (1 unless is_sub)
    double m;                  // representative calibration absmax
};

}  // namespace

extern "C" {

// ---------------------------------------------------------------------------
// O1  LayerNorm (the non-linear layer that precedes the reassembly at runtime,
// Sec. 4.3 "Inference efficiency").  Textbook form: biased variance, two passes.
//   y[m][k] = (x[m][k] - mean_m) / sqrt(var_m + eps) * gamma[k] + beta[k]
// x_dtype: 0 = float32, 1 = bfloat16 (widened exactly).  beta may be NULL (= 0).
// ---------------------------------------------------------------------------
int orc_layernorm(const void* x, int x_dtype, int64_t M, int C, const float* gamma,
                  const float* beta, double eps, double* y) {
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        double s = 0.0;
        for (int k = 0; k < C; ++k) s += load_x(x, x_dtype, m * C + k);
        double mean = s / C;
        double v = 0.0;
        for (int k = 0; k < C; ++k) {
            double d = load_x(x, x_dtype, m * C + k) - mean;
            v += d * d;
        }
        double var = v / C;
        double rstd = 1.0 / std::sqrt(var + eps);
        for (int k = 0; k < C; ++k) {
            double d = load_x(x, x_dtype, m * C + k) - mean;
            double b = beta ? static_cast<double>(beta[k]) : 0.0;
            y[m * C + k] = d * rstd * static_cast<double>(gamma[k]) + b;
        }
    }
    return 0;
}

// Per-channel calibration statistic: max over tokens of |y| (Algorithm 1,
// "max value of each channel"), taken on the input of the linear layer.
int orc_channel_absmax(const double* y, int64_t M, int C, float* absmax) {
    for (int k = 0; k < C; ++k) {
        double a = 0.0;
        for (int64_t m = 0; m < M; ++m) a = std::max(a, std::fabs(y[m * C + k]));
        absmax[k] = static_cast<float>(a);
    }
    return 0;
}

// ---------------------------------------------------------------------------
// O2  Reassembly apply.  Output channel c of a token is the weighted sum of the
// LayerNorm outputs listed in row c of the sparse map:
//   x'[c] = sum_{j in [ptr[c], ptr[c+1])} coef[j] * y[src[j]]
// A sub-channel row is (src = i, coef = 1/T_i)  (Eq. 3); a merged row lists the
// members of the set with coef = 1/|S|  (Eq. 4, generalised to a mean).
// ---------------------------------------------------------------------------
int orc_map_apply(const double* y, int64_t M, int C_in, int C_out, const int32_t* ptr,
                  const int32_t* src, const float* coef, double* xr) {
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int c = 0; c < C_out; ++c) {
            double s = 0.0;
            for (int j = ptr[c]; j < ptr[c + 1]; ++j)
                s += static_cast<double>(coef[j]) * y[m * C_in + src[j]];
            xr[m * C_out + c] = s;
        }
    return 0;
}

// ---------------------------------------------------------------------------
// O3  Uniform asymmetric b-bit quantizer of Eq. 2, one parameter pair per row
// (per token for activations, per output channel for weights):
//   alpha = (max - min) / (2^b - 1),  beta = -round(min / alpha),
//   q = clamp(round(v / alpha) + beta, 0, 2^b - 1),   round = half-to-even.
// alpha is stored as float and that stored value is the one used to divide.
// A constant row (max == min = v) takes alpha = |v| (1 if v == 0), so that
// alpha * (q - beta) returns v.
// Outputs: codes (one per byte), scale, zero (integer-valued), code sum per row,
// and optionally the pre-round quotients v/alpha (pre) and min/alpha (zpre).
// ---------------------------------------------------------------------------
int orc_quant_rows(const double* v, int64_t R, int C, int bits, uint8_t* codes, float* scale,
                   float* zero, int32_t* codesum, double* pre, double* zpre) {
    const double qmax = static_cast<double>((1 << bits) - 1);
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < R; ++r) {
        const double* row = v + r * C;
        double lo = row[0], hi = row[0];
        for (int k = 1; k < C; ++k) {
            lo = std::min(lo, row[k]);
            hi = std::max(hi, row[k]);
        }
        double a64 = (hi - lo) / qmax;
        if (!(hi > lo)) a64 = (lo != 0.0) ? std::fabs(lo) : 1.0;
        float a32 = static_cast<float>(a64);
        double alpha = static_cast<double>(a32);
        double zq = lo / alpha;
        double beta = -std::nearbyint(zq);
        int64_t sum = 0;
        for (int k = 0; k < C; ++k) {
            double p = row[k] / alpha;
            double q = std::nearbyint(p) + beta;
            q = std::min(std::max(q, 0.0), qmax);
            codes[r * C + k] = static_cast<uint8_t>(q);
            sum += static_cast<int64_t>(q);
            if (pre) pre[r * C + k] = p;
        }
        scale[r] = a32;
        zero[r] = static_cast<float>(beta);
        if (codesum) codesum[r] = static_cast<int32_t>(sum);
        if (zpre) zpre[r] = zq;
    }
    return 0;
}

// Pack 4-bit codes two per byte: low nibble = even index.
int orc_pack4(const uint8_t* codes, int64_t R, int C, uint8_t* packed) {
    for (int64_t r = 0; r < R; ++r)
        for (int k = 0; k < C / 2; ++k)
            packed[r * (C / 2) + k] =
                static_cast<uint8_t>((codes[r * C + 2 * k] & 0xF) | ((codes[r * C + 2 * k + 1] & 0xF) << 4));
    return 0;
}

// ---------------------------------------------------------------------------
// O4  Offline weight transform.  W is [N][C_in] (output-channel major).
//   W'[n][c] = sum_{j in row c} W[n][src[j]]
// (row duplicated for every sub-channel, Eq. 3 / Appendix B; rows added for a
// merged set, Eq. 4 / Appendix B), then the low-rank pair of Sec. 4.2 is folded
// in, W' += (A B)^T with A [C_out][r], B [r][N] in reassembled channel order.
// The result is fp64, [N][C_out]; quantize it with orc_quant_rows per row n.
// ---------------------------------------------------------------------------
int orc_weight_transform(const float* W, int N, int C_in, int C_out, const int32_t* ptr,
                         const int32_t* src, const float* lrA, const float* lrB, int r,
                         double* Wr) {
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < C_out; ++c) {
            double s = 0.0;
            for (int j = ptr[c]; j < ptr[c + 1]; ++j)
                s += static_cast<double>(W[static_cast<int64_t>(n) * C_in + src[j]]);
            if (lrA && lrB)
                for (int t = 0; t < r; ++t)
                    s += static_cast<double>(lrA[static_cast<int64_t>(c) * r + t]) *
                         static_cast<double>(lrB[static_cast<int64_t>(t) * N + n]);
            Wr[static_cast<int64_t>(n) * C_out + c] = s;
        }
    return 0;
}

// ---------------------------------------------------------------------------
// O5a  Integer matmul on codes (Eq. 1 with quantized operands):
//   acc[m][n] = sum_k qa[m][k] * qw[n][k]
// 64-bit accumulation; returns -1 if any value would not fit an int32.
// ---------------------------------------------------------------------------
int orc_int_matmul(const uint8_t* qa, const uint8_t* qw, int64_t M, int N, int K, int32_t* acc) {
    int overflow = 0;
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int n = 0; n < N; ++n) {
            int64_t s = 0;
            for (int k = 0; k < K; ++k)
                s += static_cast<int64_t>(qa[m * K + k]) * static_cast<int64_t>(qw[static_cast<int64_t>(n) * K + k]);
            if (s > std::numeric_limits<int32_t>::max()) overflow = 1;
            else acc[m * N + n] = static_cast<int32_t>(s);
        }
    return overflow ? -1 : 0;
}

// Same sum for a list of (m, n) pairs only: lets full-size problems be checked
// entry by entry.
int orc_int_matmul_at(const uint8_t* qa, const uint8_t* qw, int K, const int64_t* ms,
                      const int32_t* ns, int64_t count, int32_t* acc) {
    for (int64_t i = 0; i < count; ++i) {
        int64_t s = 0;
        const uint8_t* a = qa + ms[i] * K;
        const uint8_t* w = qw + static_cast<int64_t>(ns[i]) * K;
        for (int k = 0; k < K; ++k) s += static_cast<int64_t>(a[k]) * static_cast<int64_t>(w[k]);
        if (s > std::numeric_limits<int32_t>::max()) return -1;
        acc[i] = static_cast<int32_t>(s);
    }
    return 0;
}

// ---------------------------------------------------------------------------
// O5b  Dequantizing epilogue.  Inverting Eq. 2 on both operands,
//   sum_k a_s (qa - za) * w_s (qw - zw)
//     = a_s w_s (acc - zw * rowsum_a - za * colsum_w + K za zw),
// the bracket being an exact integer I.  out = a_s * w_s * I + bias in fp64.
// ---------------------------------------------------------------------------
int orc_epilogue(const int32_t* acc, int64_t M, int N, int K, const float* a_scale,
                 const float* a_zero, const int32_t* a_rowsum, const float* w_scale,
                 const float* w_zero, const int32_t* w_colsum, const float* bias, double* out) {
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        int64_t za = static_cast<int64_t>(a_zero[m]);
        for (int n = 0; n < N; ++n) {
            int64_t zw = static_cast<int64_t>(w_zero[n]);
            int64_t I = static_cast<int64_t>(acc[m * N + n]) - zw * a_rowsum[m] - za * w_colsum[n] +
                        static_cast<int64_t>(K) * za * zw;
            double o = static_cast<double>(a_scale[m]) * static_cast<double>(w_scale[n]) * static_cast<double>(I);
            if (bias) o += static_cast<double>(bias[n]);
            out[m * N + n] = o;
        }
    }
    return 0;
}

// Casts of the fp64 result to the boundary's output types.
int orc_cast_f32(const double* v, int64_t n, float* out) {
    for (int64_t i = 0; i < n; ++i) out[i] = static_cast<float>(v[i]);
    return 0;
}
int orc_cast_bf16(const double* v, int64_t n, uint16_t* out) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) out[i] = round_to_bf16(v[i]);
    return 0;
}

// Dense fp64 linear layer of Eq. 1 with W stored [N][C]:  out[m][n] = sum_k X[m][k] W[n][k].
int orc_dense_linear(const double* X, const double* W, int64_t M, int N, int C, double* out) {
    for (int64_t m = 0; m < M; ++m)
        for (int n = 0; n < N; ++n) {
            double s = 0.0;
            for (int k = 0; k < C; ++k) s += X[m * C + k] * W[static_cast<int64_t>(n) * C + k];
            out[m * N + n] = s;
        }
    return 0;
}

// ---------------------------------------------------------------------------
// Threshold helpers.
// ---------------------------------------------------------------------------
// Sub-channel count of Sec. 4.1.1, T = ceil(max|x_i| / theta), at least 1.
static int split_count(float m, float theta) {
    double t = std::ceil(static_cast<double>(m) / static_cast<double>(theta));
    if (!(t >= 1.0)) t = 1.0;
    return static_cast<int>(t);
}

int64_t orc_extra_channels(const float* absmax, int C, float theta) {
    int64_t E = 0;
    for (int i = 0; i < C; ++i) E += split_count(absmax[i], theta) - 1;
    return E;
}

// Nearest-rank percentile of the channel maxima: sorted ascending, element
// ceil(pct * C) - 1.
float orc_theta_percentile(const float* absmax, int C, double pct) {
    std::vector<float> s(absmax, absmax + C);
    std::sort(s.begin(), s.end());
    int64_t rank = static_cast<int64_t>(std::ceil(pct * C));
    rank = std::min<int64_t>(std::max<int64_t>(rank, 1), C);
    return s[rank - 1];
}

// A threshold for which disassembly adds exactly `extra` channels.  E(theta) is
// a step function that rises by one each time theta falls below a breakpoint
// m_i / k; with the breakpoints sorted descending b_1 >= b_2 >= ..., E = j on
// [b_{j+1}, b_j).  The midpoint of that interval is returned (0 if the interval
// is empty or the float midpoint does not reproduce `extra`).
float orc_theta_for_extra(const float* absmax, int C, int extra) {
    if (extra < 1) return 0.f;
    std::vector<double> bp;
    for (int i = 0; i < C; ++i)
        for (int k = 1; k <= extra + 1; ++k) bp.push_back(static_cast<double>(absmax[i]) / k);
    std::sort(bp.begin(), bp.end(), [](double a, double b) { return a > b; });
    if (static_cast<int>(bp.size()) < extra + 1) return 0.f;
    double hi = bp[extra - 1], lo = bp[extra];
    float th = static_cast<float>(0.5 * (hi + lo));
    if (!(th > 0.f) || orc_extra_channels(absmax, C, th) != extra) return 0.f;
    return th;
}

// ---------------------------------------------------------------------------
// O6  Reassembly-map builder (a heuristic: steps in the paper's order).
//  1. T_i = max(1, ceil(m_i / theta))                       (Sec. 4.1.1)
//  2. expanded list: channel i contributes T_i consecutive entries, each the
//     sub-channel x_i / T_i (Eq. 3); E = sum (T_i - 1) extra channels.
//  3. entries born from disassembly are never assembled     (Sec. 4.1.2)
//  4. bipartite soft matching (Appendix A): set A = eligible entries at even
//     list positions, set B = those at odd positions; every a in A draws an edge
//     to its most similar b (distance |m_a - m_b| on the calibration maxima;
//     ties: lowest position); the `need` shortest edges are kept (ties: lowest
//     position of a); a joins b's set; the set's feature is the mean of its
//     members (Eq. 4) and it stays at b's position; merged a's are removed.
//  5. if one round cannot supply all E merges it merges every a and runs
//     another round on the shortened list, a merged set counting as one
//     eligible entry with m = mean of its members' maxima.
// Output: CSR with exactly C rows, nnz = C + E.  Returns 0, or -1 when the
// channel count cannot be brought back to C (no eligible pair left), or -2 when
// the caller's buffers are too small (nnz_cap).
// stats[0] = E, stats[1] = rows with more than one member, stats[2] = rounds.
// ---------------------------------------------------------------------------
// dist: optional C x C table of pairwise channel distances (Eq. 5, see orc_channel_distance).  Without it the
// distance between two entries is |m_a - m_b|.  With it the distance between two undivided channels is
// dist[a][b]; a second matching round would need distances between merged sets, which Eq. 5 does not define:
// -4 is returned instead.
static int build_map_impl(const float* absmax, int C, float theta, const double* dist, int32_t* ptr, int32_t* src,
                          float* coef, int64_t nnz_cap, int64_t* stats) {
    if (!(theta > 0.f)) return -3;
    std::vector<Entry> list;
    int64_t E = 0;
    for (int i = 0; i < C; ++i) {
        int T = split_count(absmax[i], theta);
        E += T - 1;
        for (int t = 0; t < T; ++t) {
            Entry e;
            e.members = {i};
            e.is_sub = (T > 1);
            e.T = T;
            e.m = static_cast<double>(absmax[i]);
            list.push_back(e);
        }
    }
    if (C + E > nnz_cap) return -2;
    int64_t need = E;
    int rounds = 0;
    while (need > 0) {
        if (dist && rounds > 0) return -4;
        std::vector<int> A, B;
        for (int p = 0; p < static_cast<int>(list.size()); ++p) {
            if (list[p].is_sub) continue;
            ((p % 2 == 0) ? A : B).push_back(p);
        }
        if (A.empty() || B.empty()) return -1;
        struct Edge { double d; int a; int b; };
        std::vector<Edge> edges;
        for (int a : A) {
            double best = std::numeric_limits<double>::infinity();
            int bb = -1;
            for (int b : B) {
                double d = dist ? dist[static_cast<int64_t>(list[a].members[0]) * C + list[b].members[0]]
                                : std::fabs(list[a].m - list[b].m);
                if (d < best) { best = d; bb = b; }   // B ascending: first minimum = lowest position
            }
            edges.push_back({best, a, bb});
        }
        std::stable_sort(edges.begin(), edges.end(), [](const Edge& x, const Edge& y) {
            if (x.d != y.d) return x.d < y.d;
            return x.a < y.a;
        });
        int64_t keep = std::min<int64_t>(need, static_cast<int64_t>(edges.size()));
        std::vector<Edge> kept(edges.begin(), edges.begin() + keep);
        std::sort(kept.begin(), kept.end(), [](const Edge& x, const Edge& y) { return x.a < y.a; });
        std::vector<char> gone(list.size(), 0);
        for (const Edge& e : kept) {
            for (int s : list[e.a].members) list[e.b].members.push_back(s);
            gone[e.a] = 1;
        }
        for (const Edge& e : kept) {
            double s = 0.0;
            for (int sidx : list[e.b].members) s += static_cast<double>(absmax[sidx]);
            list[e.b].m = s / static_cast<double>(list[e.b].members.size());
        }
        std::vector<Entry> next;
        for (int p = 0; p < static_cast<int>(list.size()); ++p)
            if (!gone[p]) next.push_back(list[p]);
        list.swap(next);
        need -= keep;
        ++rounds;
    }
    if (static_cast<int>(list.size()) != C) return -1;
    int64_t nnz = 0, multi = 0;
    for (int c = 0; c < C; ++c) {
        ptr[c] = static_cast<int32_t>(nnz);
        const Entry& e = list[c];
        double w = e.is_sub ? 1.0 / e.T : 1.0 / static_cast<double>(e.members.size());
        if (e.members.size() > 1) ++multi;
        for (int s : e.members) {
            src[nnz] = s;
            coef[nnz] = static_cast<float>(w);
            ++nnz;
        }
    }
    ptr[C] = static_cast<int32_t>(nnz);
    if (stats) { stats[0] = E; stats[1] = multi; stats[2] = rounds; }
    return 0;
}

int orc_build_map(const float* absmax, int C, float theta, int32_t* ptr, int32_t* src,
                  float* coef, int64_t nnz_cap, int64_t* stats) {
    return build_map_impl(absmax, C, theta, nullptr, ptr, src, coef, nnz_cap, stats);
}

// The same builder with the distance of Eq. 5 between undivided channels, given as a C x C table.
int orc_build_map_dist(const float* absmax, int C, float theta, const double* dist, int32_t* ptr, int32_t* src,
                       float* coef, int64_t nnz_cap, int64_t* stats) {
    if (!dist) return -3;
    return build_map_impl(absmax, C, theta, dist, ptr, src, coef, nnz_cap, stats);
}

// ---------------------------------------------------------------------------
// Eq. 5: the output error of merging channels i and j,
//     D(i, j) = || (x_i (W_i - W_j) + x_j (W_j - W_i)) / 2 ||_F^2 = 1/4 ||x_i - x_j||^2 ||W_i - W_j||^2,
// x_i the column of channel i over the T calibration rows of y (the linear layer's input), W_i the
// weights of input channel i over the N outputs.  Plain definition in fp64.
// y: [T][C], w: [N][C] (output channel major), D: [C][C].
// ---------------------------------------------------------------------------
void orc_channel_distance(const double* y, int64_t T, const float* w, int N, int C, double* D) {
    for (int i = 0; i < C; ++i) {
        for (int j = 0; j < C; ++j) {
            double dx = 0.0, dw = 0.0;
            for (int64_t t = 0; t < T; ++t) {
                const double e = y[t * C + i] - y[t * C + j];
                dx += e * e;
            }
            for (int n = 0; n < N; ++n) {
                const double e = static_cast<double>(w[static_cast<int64_t>(n) * C + i]) -
                                 static_cast<double>(w[static_cast<int64_t>(n) * C + j]);
                dw += e * e;
            }
            D[static_cast<int64_t>(i) * C + j] = 0.25 * dx * dw;
        }
    }
}

}  // extern "C"
