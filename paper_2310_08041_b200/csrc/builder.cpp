// Host-side reassembly builder: calibration maxima + threshold -> sparse map and
// transformed, quantized weights (QLLM Sec. 4.1.1-4.1.2, Appendix A/B, Sec. 4.2).
//
// Data layout.  The channel list is kept as arrays over "slots" (list positions);
// the members of a merged set are chained through `next_member` (one link per
// source channel, since only undivided channels can be merged and each belongs to
// one set).  Nearest-neighbour search over set B uses a (maximum, position)-sorted
// array and binary search, so a matching round costs O(C log C) instead of the
// |A| x |B| distance table; the weight transform is threaded over output channels.

#include <algorithm>
#include <cmath>
#include <cstring>
#include <limits>
#include <thread>
#include <vector>

#include <cuda_runtime.h>

#include "../../include/qllm.h"

namespace qllm {
// channel_distance.cu: nearest channel of B for every channel of A under Eq. 5, on the device
int eq5_nearest_device(const float* y, int64_t T, const float* w, int N, int C, const int* a_idx, int nA,
                       const int* b_idx, int nB, int* best, float* best_d, cudaStream_t st);
}

struct qllm_reassembly {
    int C = 0, N = 0, w_bits = 0;
    int64_t E = 0, merged_rows = 0, rounds = 0;
    std::vector<int32_t> ptr, src;
    std::vector<float> coef;
    std::vector<uint8_t> w_codes;
    std::vector<float> w_scale, w_zero;
    std::vector<int32_t> w_colsum;
};

namespace {

// T = ceil(max|x_i| / theta), at least 1 (Sec. 4.1.1).
inline int sub_channels(float absmax, float theta) {
    double q = std::ceil(double(absmax) / double(theta));
    return q >= 1.0 ? int(q) : 1;
}

struct Slot {
    int head;      // first member (source channel)
    int tail;      // last member
    int count;     // members
    int T;         // split count (sub-channel slots only)
    bool sub;      // born from disassembly: not eligible for assembly
    double m;      // calibration maximum (mean over members for a merged set)
};

// Calibration data on the device for the Eq. 5 distance: y [T][C] (the layer's input), w [N][C].
struct Eq5Device {
    const float* y;
    int64_t T;
    const float* w;
    int N;
    cudaStream_t st;
};

struct BKey {
    double m;
    int pos;
    bool operator<(const BKey& o) const { return m < o.m || (m == o.m && pos < o.pos); }
};

// One round of bipartite soft matching on `slots`; merges up to `need` A-slots into
// their nearest B-slot.  Returns the number of merges done (0 = no eligible pair).
// dist (optional): C x C table of distances between undivided channels; the nearest b of an a is then found by a
// scan over B on that table (the table has no order to search in).  dev (optional): the Eq. 5 distance is
// evaluated on the device from calibration data and only the |A| nearest-neighbour edges come back.
// A negative return is a status code.
int64_t matching_round(std::vector<Slot>& slots, std::vector<int>& next_member,
                       const float* absmax, int64_t need, const float* dist, const Eq5Device* dev, int C) {
    const int L = int(slots.size());
    std::vector<int> A;
    std::vector<BKey> B;
    for (int p = 0; p < L; ++p) {
        if (slots[p].sub) continue;
        if (p & 1) B.push_back({slots[p].m, p}); else A.push_back(p);
    }
    if (A.empty() || B.empty()) return 0;
    std::sort(B.begin(), B.end());
    const int nb = int(B.size());

    struct Edge { double d; int a; int b; };
    std::vector<Edge> edges(A.size());
    if (dev) {
        std::vector<int> Bpos, a_idx, b_idx;              // B in list order: ties go to the lowest position
        for (int p = 1; p < L; p += 2)
            if (!slots[p].sub) { Bpos.push_back(p); b_idx.push_back(slots[p].head); }
        for (int a : A) a_idx.push_back(slots[a].head);
        std::vector<int> best(A.size(), -1);
        std::vector<float> best_d(A.size(), 0.f);
        const int rc = qllm::eq5_nearest_device(dev->y, dev->T, dev->w, dev->N, C, a_idx.data(), int(a_idx.size()),
                                                b_idx.data(), int(b_idx.size()), best.data(), best_d.data(), dev->st);
        if (rc != QLLM_OK) return rc;
        for (size_t i = 0; i < A.size(); ++i) {
            if (best[i] < 0 || !std::isfinite(best_d[i])) return QLLM_ERR_MAP;   // no usable distance in the row
            edges[i] = {double(best_d[i]), A[i], Bpos[size_t(best[i])]};
        }
    } else if (dist) {
        std::vector<int> Bpos;                            // B in list order: ties go to the lowest position
        for (int p = 1; p < L; p += 2)
            if (!slots[p].sub) Bpos.push_back(p);
        for (size_t i = 0; i < A.size(); ++i) {
            const float* row = dist + size_t(slots[A[i]].head) * size_t(C);
            double best = std::numeric_limits<double>::infinity();
            int best_pos = -1;
            for (int p : Bpos) {
                const double d = double(row[slots[p].head]);
                if (d < best) { best = d; best_pos = p; }
            }
            if (best_pos < 0) return QLLM_ERR_MAP;        // every distance of the row is NaN or +inf
            edges[i] = {best, A[i], best_pos};
        }
    }
    for (size_t i = 0; i < A.size() && !dist && !dev; ++i) {
        const int a = A[i];
        const double ma = slots[a].m;
        // first key with m >= ma
        int r = int(std::lower_bound(B.begin(), B.end(), BKey{ma, -1}) - B.begin());
        double best = std::numeric_limits<double>::infinity();
        int best_pos = -1;
        auto consider = [&](int idx) {
            double d = std::fabs(ma - B[idx].m);
            if (d < best || (d == best && B[idx].pos < best_pos)) { best = d; best_pos = B[idx].pos; }
            return d;
        };
        // walk right while the distance does not grow past the best, then left likewise:
        // the distance is monotone in each direction, so only ties extend the walk.
        for (int idx = r; idx < nb; ++idx) { if (consider(idx) > best) break; }
        for (int idx = r - 1; idx >= 0; --idx) { if (consider(idx) > best) break; }
        edges[i] = {best, a, best_pos};
    }
    std::sort(edges.begin(), edges.end(), [](const Edge& x, const Edge& y) {
        return x.d < y.d || (x.d == y.d && x.a < y.a);
    });
    const int64_t keep = std::min<int64_t>(need, int64_t(edges.size()));
    edges.resize(size_t(keep));
    std::sort(edges.begin(), edges.end(), [](const Edge& x, const Edge& y) { return x.a < y.a; });

    std::vector<char> removed(size_t(L), 0);
    for (const Edge& e : edges) {
        Slot& b = slots[e.b];
        const Slot& a = slots[e.a];
        next_member[b.tail] = a.head;
        b.tail = a.tail;
        b.count += a.count;
        removed[e.a] = 1;
    }
    for (const Edge& e : edges) {
        Slot& b = slots[e.b];
        double s = 0.0;
        for (int c = b.head, k = 0; k < b.count; ++k, c = next_member[c]) s += double(absmax[c]);
        b.m = s / double(b.count);
    }
    size_t w = 0;
    for (int p = 0; p < L; ++p)
        if (!removed[p]) slots[w++] = slots[p];
    slots.resize(w);
    return keep;
}

int build_map(const float* absmax, int C, float theta, const float* dist, const Eq5Device* dev, qllm_reassembly& h) {
    std::vector<Slot> slots;
    slots.reserve(size_t(C) + 64);
    int64_t E = 0;
    for (int i = 0; i < C; ++i) {
        const int T = sub_channels(absmax[i], theta);
        E += T - 1;
        if (int64_t(C) + E > (int64_t(1) << 30)) return QLLM_ERR_UNSUPPORTED;
        for (int t = 0; t < T; ++t) slots.push_back({i, i, 1, T, T > 1, double(absmax[i])});
    }
    std::vector<int> next_member(size_t(C), -1);
    int64_t need = E, rounds = 0;
    while (need > 0) {
        if ((dist || dev) && rounds > 0) return QLLM_ERR_UNSUPPORTED;   // Eq. 5 is defined between undivided channels only
        int64_t done = matching_round(slots, next_member, absmax, need, dist, dev, C);
        if (done < 0) return int(done);
        if (done == 0) return QLLM_ERR_INFEASIBLE;
        need -= done;
        ++rounds;
    }
    if (int(slots.size()) != C) return QLLM_ERR_INFEASIBLE;
    h.E = E;
    h.rounds = rounds;
    h.merged_rows = 0;
    h.ptr.resize(size_t(C) + 1);
    h.src.clear(); h.coef.clear();
    h.src.reserve(size_t(C + E)); h.coef.reserve(size_t(C + E));
    for (int c = 0; c < C; ++c) {
        const Slot& s = slots[c];
        h.ptr[c] = int32_t(h.src.size());
        const float w = float(s.sub ? 1.0 / double(s.T) : 1.0 / double(s.count));
        if (s.count > 1) ++h.merged_rows;
        for (int ch = s.head, k = 0; k < s.count; ++k, ch = next_member[ch]) {
            h.src.push_back(ch);
            h.coef.push_back(w);
        }
    }
    h.ptr[C] = int32_t(h.src.size());
    return QLLM_OK;
}

// Eq. 2 on one transformed weight row (K doubles) -> codes, scale, zero, code sum.
void quantize_weight_row(const double* row, int K, int bits, uint8_t* codes_out, float* scale,
                         float* zero, int32_t* colsum) {
    const double qmax = double((1 << bits) - 1);
    double lo = row[0], hi = row[0];
    for (int k = 1; k < K; ++k) { lo = std::min(lo, row[k]); hi = std::max(hi, row[k]); }
    double a = (hi - lo) / qmax;
    if (!(hi > lo)) a = lo != 0.0 ? std::fabs(lo) : 1.0;
    const float a32 = float(a);
    const double alpha = double(a32);
    const double z = -std::nearbyint(lo / alpha);
    int64_t sum = 0;
    auto code_of = [&](double v) {
        double q = std::nearbyint(v / alpha) + z;
        q = q < 0.0 ? 0.0 : (q > qmax ? qmax : q);
        return int(q);
    };
    if (bits == 4) {
        for (int k = 0; k < K; k += 2) {
            int q0 = code_of(row[k]), q1 = code_of(row[k + 1]);
            sum += q0 + q1;
            codes_out[k >> 1] = uint8_t(q0 | (q1 << 4));
        }
    } else {
        for (int k = 0; k < K; ++k) {
            int q = code_of(row[k]);
            sum += q;
            codes_out[k] = uint8_t(q);
        }
    }
    *scale = a32;
    *zero = float(z);
    *colsum = int32_t(sum);
}

void transform_and_quantize(const float* W, int N, int C, const float* lrA, const float* lrB, int r,
                            int bits, qllm_reassembly& h) {
    const int64_t row_bytes = bits == 4 ? C / 2 : C;
    h.w_codes.assign(size_t(row_bytes) * size_t(N), 0);
    h.w_scale.assign(size_t(N), 0.f);
    h.w_zero.assign(size_t(N), 0.f);
    h.w_colsum.assign(size_t(N), 0);
    unsigned hw = std::thread::hardware_concurrency();
    int nthreads = int(std::min<unsigned>(hw ? hw : 1u, 32u));
    nthreads = std::max(1, std::min(nthreads, N));
    auto work = [&](int t) {
        std::vector<double> row(size_t(C), 0.0);
        for (int n = t; n < N; n += nthreads) {
            const float* wn = W + int64_t(n) * C;
            for (int c = 0; c < C; ++c) {
                double s = 0.0;
                for (int j = h.ptr[c]; j < h.ptr[c + 1]; ++j) s += double(wn[h.src[j]]);
                if (lrA && lrB)
                    for (int t2 = 0; t2 < r; ++t2)
                        s += double(lrA[int64_t(c) * r + t2]) * double(lrB[int64_t(t2) * N + n]);
                row[c] = s;
            }
            quantize_weight_row(row.data(), C, bits, h.w_codes.data() + int64_t(n) * row_bytes,
                                &h.w_scale[n], &h.w_zero[n], &h.w_colsum[n]);
        }
    };
    std::vector<std::thread> pool;
    for (int t = 1; t < nthreads; ++t) pool.emplace_back(work, t);
    work(0);
    for (auto& th : pool) th.join();
}

}  // namespace

extern "C" {

static int build_reassembly_impl(const float* calib_absmax, int C, float theta, const float* dist,
                                 const Eq5Device* dev, const float* W,
                                 int N, const float* lr_A, const float* lr_B, int r, int w_bits,
                                 qllm_reassembly_t** out) {
    if (!calib_absmax || !W || !out) return QLLM_ERR_NULL;
    if ((lr_A == nullptr) != (lr_B == nullptr)) return QLLM_ERR_NULL;
    if (C <= 0 || N <= 0 || C > 65536 || (lr_A && r <= 0)) return QLLM_ERR_SHAPE;
    if (!(theta > 0.f) || !std::isfinite(theta)) return QLLM_ERR_SHAPE;
    if (w_bits != 4 && w_bits != 6 && w_bits != 8) return QLLM_ERR_BITS;
    if (w_bits == 4 && (C & 1)) return QLLM_ERR_SHAPE;
    for (int i = 0; i < C; ++i)
        if (!(calib_absmax[i] >= 0.f) || !std::isfinite(calib_absmax[i])) return QLLM_ERR_SHAPE;
    qllm_reassembly* h = new (std::nothrow) qllm_reassembly();
    if (!h) return QLLM_ERR_NOMEM;
    h->C = C; h->N = N; h->w_bits = w_bits;
    int rc;
    try {
        rc = build_map(calib_absmax, C, theta, dist, dev, *h);
        if (rc == QLLM_OK) transform_and_quantize(W, N, C, lr_A, lr_B, r, w_bits, *h);
    } catch (const std::bad_alloc&) {
        rc = QLLM_ERR_NOMEM;
    }
    if (rc != QLLM_OK) { delete h; return rc; }
    *out = h;
    return QLLM_OK;
}

int qllm_build_reassembly(const float* calib_absmax, int C, float theta, const float* W, int N,
                          const float* lr_A, const float* lr_B, int r, int w_bits,
                          qllm_reassembly_t** out) {
    return build_reassembly_impl(calib_absmax, C, theta, nullptr, nullptr, W, N, lr_A, lr_B, r, w_bits, out);
}

int qllm_build_reassembly_dist(const float* calib_absmax, int C, float theta, const float* dist, const float* W,
                               int N, const float* lr_A, const float* lr_B, int r, int w_bits,
                               qllm_reassembly_t** out) {
    if (!dist) return QLLM_ERR_NULL;
    return build_reassembly_impl(calib_absmax, C, theta, dist, nullptr, W, N, lr_A, lr_B, r, w_bits, out);
}

int qllm_build_reassembly_eq5(const float* calib_absmax, int C, float theta, const float* calib_y, int64_t T,
                              const float* W, int N, const float* lr_A, const float* lr_B, int r, int w_bits,
                              void* stream, qllm_reassembly_t** out) {
    if (!calib_y || !W) return QLLM_ERR_NULL;
    if (T <= 0 || C <= 0 || N <= 0) return QLLM_ERR_SHAPE;
    // the weights beside the calibration rows on the device, for the duration of the build
    float* w_dev = nullptr;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMalloc(&w_dev, sizeof(float) * size_t(N) * size_t(C)) != cudaSuccess) { cudaGetLastError(); return QLLM_ERR_NOMEM; }
    if (cudaMemcpyAsync(w_dev, W, sizeof(float) * size_t(N) * size_t(C), cudaMemcpyHostToDevice, st) != cudaSuccess) {
        cudaGetLastError();
        cudaFree(w_dev);
        return QLLM_ERR_CUDA;
    }
    const Eq5Device dev{calib_y, T, w_dev, N, st};
    const int rc = build_reassembly_impl(calib_absmax, C, theta, nullptr, &dev, W, N, lr_A, lr_B, r, w_bits, out);
    cudaStreamSynchronize(st);
    cudaFree(w_dev);
    return rc;
}

void qllm_free_reassembly(qllm_reassembly_t* h) { delete h; }

int qllm_reassembly_map(const qllm_reassembly_t* h, const int32_t** map_ptr, const int32_t** map_src,
                        const float** map_coef, int64_t* nnz) {
    if (!h) return QLLM_ERR_NULL;
    if (map_ptr) *map_ptr = h->ptr.data();
    if (map_src) *map_src = h->src.data();
    if (map_coef) *map_coef = h->coef.data();
    if (nnz) *nnz = int64_t(h->src.size());
    return QLLM_OK;
}

int qllm_reassembly_weights(const qllm_reassembly_t* h, const uint8_t** w_codes, int64_t* w_bytes,
                            const float** w_scale, const float** w_zero, const int32_t** w_colsum) {
    if (!h) return QLLM_ERR_NULL;
    if (w_codes) *w_codes = h->w_codes.data();
    if (w_bytes) *w_bytes = int64_t(h->w_codes.size());
    if (w_scale) *w_scale = h->w_scale.data();
    if (w_zero) *w_zero = h->w_zero.data();
    if (w_colsum) *w_colsum = h->w_colsum.data();
    return QLLM_OK;
}

int qllm_reassembly_stats(const qllm_reassembly_t* h, int64_t stats[6]) {
    if (!h || !stats) return QLLM_ERR_NULL;
    stats[0] = h->E; stats[1] = h->merged_rows; stats[2] = h->rounds;
    stats[3] = h->C; stats[4] = h->N; stats[5] = h->w_bits;
    return QLLM_OK;
}

int qllm_fold_previous(const int32_t* map_ptr, const int32_t* map_src, const float* map_coef, int C,
                       const float* W_prev, const float* bias_prev, int C_in, float* W_out, float* bias_out) {
    if (!map_ptr || !map_src || !map_coef || !W_prev || !W_out) return QLLM_ERR_NULL;
    if (C <= 0 || C_in <= 0) return QLLM_ERR_SHAPE;
    if (bias_prev && !bias_out) return QLLM_ERR_NULL;
    const int rc = qllm_validate_map(map_ptr, map_src, C, map_ptr[C]);
    if (rc != QLLM_OK) return rc;
    // output channel c of the preceding layer = sum_j coef_j * (its output channel src_j): Appendix B's
    // duplication with 1/T for sub-channels and the mean for merged channels, in one pass over the map
    std::vector<double> acc(static_cast<size_t>(C_in));
    for (int c = 0; c < C; ++c) {
        std::fill(acc.begin(), acc.end(), 0.0);
        double b = 0.0;
        for (int j = map_ptr[c]; j < map_ptr[c + 1]; ++j) {
            const double cf = double(map_coef[j]);
            const float* row = W_prev + size_t(map_src[j]) * C_in;
            for (int k = 0; k < C_in; ++k) acc[k] += cf * double(row[k]);
            if (bias_prev) b += cf * double(bias_prev[map_src[j]]);
        }
        float* out = W_out + size_t(c) * C_in;
        for (int k = 0; k < C_in; ++k) out[k] = float(acc[k]);
        if (bias_prev) bias_out[c] = float(b);
    }
    return QLLM_OK;
}

int qllm_validate_map(const int32_t* map_ptr, const int32_t* map_src, int C, int64_t nnz) {
    if (!map_ptr || !map_src) return QLLM_ERR_NULL;
    if (C <= 0 || nnz < C) return QLLM_ERR_MAP;
    if (map_ptr[0] != 0 || int64_t(map_ptr[C]) != nnz) return QLLM_ERR_MAP;
    for (int c = 0; c < C; ++c)
        if (map_ptr[c + 1] <= map_ptr[c]) return QLLM_ERR_MAP;
    for (int64_t j = 0; j < nnz; ++j)
        if (map_src[j] < 0 || map_src[j] >= C) return QLLM_ERR_MAP;
    return QLLM_OK;
}

float qllm_theta_percentile(const float* absmax, int C, double pct) {
    if (!absmax || C <= 0 || !(pct > 0.0) || pct > 1.0) return 0.f;
    std::vector<float> v(absmax, absmax + C);
    int64_t rank = int64_t(std::ceil(pct * double(C)));
    rank = std::max<int64_t>(1, std::min<int64_t>(rank, C));
    std::nth_element(v.begin(), v.begin() + (rank - 1), v.end());
    return v[size_t(rank - 1)];
}

float qllm_theta_for_extra(const float* absmax, int C, int extra) {
    if (!absmax || C <= 0 || extra < 1) return 0.f;
    // Thresholds at which one more sub-channel appears are absmax_i / k.  Pop them from a
    // max-heap: the (extra)-th and (extra+1)-th largest bound the interval with E = extra.
    struct Bp { double v; int i; int k; bool operator<(const Bp& o) const { return v < o.v; } };
    std::vector<Bp> heap;
    heap.reserve(size_t(C));
    for (int i = 0; i < C; ++i) heap.push_back({double(absmax[i]), i, 1});
    std::make_heap(heap.begin(), heap.end());
    double hi = 0.0, lo = 0.0;
    for (int j = 1; j <= extra + 1; ++j) {
        std::pop_heap(heap.begin(), heap.end());
        Bp top = heap.back();
        if (j == extra) hi = top.v;
        if (j == extra + 1) lo = top.v;
        heap.back() = {double(absmax[top.i]) / double(top.k + 1), top.i, top.k + 1};
        std::push_heap(heap.begin(), heap.end());
    }
    const float th = float(0.5 * (hi + lo));
    if (!(th > 0.f)) return 0.f;
    int64_t E = 0;
    for (int i = 0; i < C; ++i) E += sub_channels(absmax[i], th) - 1;
    return E == extra ? th : 0.f;
}

}  // extern "C"
