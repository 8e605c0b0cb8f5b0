// extern "C" entry points of the device side: argument checks, dispatch, the layer
// object, diagnostics.  Every step of the path runs in this library's kernels.

#include <mutex>
#include <new>
#include <vector>

#include "common.h"
#include "reassemble_quant_common.cuh"

namespace qllm {

thread_local int g_last_cuda_error = 0;
std::atomic<int64_t> g_launch_count{0};

// Device-side status word: kernels with bounded waits set it when a wait expires.
__device__ int g_status_word = 0;

int* device_status_word() {
    int* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_status_word);
    if (e != cudaSuccess) { cuda_fail(e); return nullptr; }
    return p;
}

namespace {
std::mutex g_scratch_mu;
struct StreamScratch {
    cudaStream_t st; uint8_t* ptr; size_t cap; uint64_t epoch; cudaEvent_t done;
    unsigned long long done_capture;   // id of the stream capture `done` was last recorded in, 0 = outside any
};
// Id of the capture `st` is part of, 0 when it is not capturing.
unsigned long long capture_id(cudaStream_t st) {
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    unsigned long long id = 0;
    if (cudaStreamGetCaptureInfo(st, &cs, &id) != cudaSuccess) { cudaGetLastError(); return 0; }
    return cs == cudaStreamCaptureStatusActive ? id : 0;
}
std::vector<StreamScratch> g_stream_scratch[kScratchKinds][64];
}  // namespace

int device_sm_count() {
    static std::atomic<int> cache[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    int n = cache[dev].load(std::memory_order_relaxed);
    if (n == 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cache[dev].store(n, std::memory_order_relaxed);
    }
    return n;
}

// Writers of a stream's scratch (the stream itself, or a layer's side stream working ahead for it) take turns:
// scratch_write_begin makes `writer` wait for the previous writer, scratch_write_end records the new contents'
// completion and returns their version.  A holder of data in the scratch (a layer whose expanded weights wait
// there for its GEMM call) compares versions (scratch_version) to see whether the data is still its own.
static StreamScratch* find_scratch(int kind, cudaStream_t st) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64 || kind < 0 || kind >= kScratchKinds) return nullptr;
    for (auto& x : g_stream_scratch[kind][dev])
        if (x.st == st) return &x;
    return nullptr;
}
int scratch_write_begin(int kind, cudaStream_t st, cudaStream_t writer) {
    std::lock_guard<std::mutex> lk(g_scratch_mu);
    StreamScratch* e = find_scratch(kind, st);
    if (!e) return QLLM_ERR_UNSUPPORTED;
    if (!e->done) QLLM_CUDA_TRY(cudaEventCreateWithFlags(&e->done, cudaEventDisableTiming));
    // no-op until a writer has recorded it.  An event recorded inside a stream capture cannot be waited on
    // from outside it, nor the reverse: across that boundary the writers are ordered by the stream itself
    // (the graph runs in stream order, after the work issued before it)
    if (capture_id(writer) == e->done_capture) QLLM_CUDA_TRY(cudaStreamWaitEvent(writer, e->done, 0));
    return QLLM_OK;
}
int scratch_write_end(int kind, cudaStream_t st, cudaStream_t writer, uint64_t* version) {
    std::lock_guard<std::mutex> lk(g_scratch_mu);
    StreamScratch* e = find_scratch(kind, st);
    if (!e || !e->done) return QLLM_ERR_UNSUPPORTED;
    QLLM_CUDA_TRY(cudaEventRecord(e->done, writer));
    e->done_capture = capture_id(writer);
    ++e->epoch;
    if (version) *version = e->epoch;
    return QLLM_OK;
}
uint64_t scratch_version(int kind, cudaStream_t st) {
    std::lock_guard<std::mutex> lk(g_scratch_mu);
    StreamScratch* e = find_scratch(kind, st);
    return e ? e->epoch : 0;
}

int stream_scratch(int kind, cudaStream_t st, size_t bytes, uint8_t** out) {
    int dev = 0;
    QLLM_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64 || kind < 0 || kind >= kScratchKinds) return QLLM_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lk(g_scratch_mu);
    StreamScratch* e = nullptr;
    for (auto& x : g_stream_scratch[kind][dev]) if (x.st == st) e = &x;
    if (!e) { g_stream_scratch[kind][dev].push_back({st, nullptr, 0, 0, nullptr, 0}); e = &g_stream_scratch[kind][dev].back(); }
    if (e->cap < bytes) {
        if (e->ptr) QLLM_CUDA_TRY(cudaFree(e->ptr));
        e->ptr = nullptr; e->cap = 0;
        QLLM_CUDA_TRY(cudaMalloc(&e->ptr, bytes));
        e->cap = bytes;
        ++e->epoch;
        if (kind == kScratchMapImage) QLLM_CUDA_TRY(cudaMemsetAsync(e->ptr, 0, std::min(bytes, kMapScratchHeader), st));
    }
    *out = e->ptr;
    return QLLM_OK;
}

namespace {

// Library-owned scratch for activation row sums when the caller passes none
// (one buffer per device, grown on demand, never shrunk).
struct RowsumScratch {
    int32_t* ptr = nullptr;
    int64_t cap = 0;
};
RowsumScratch g_scratch[64];

int rowsum_scratch(int64_t M, int32_t** out) {
    int dev = 0;
    QLLM_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return QLLM_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lk(g_scratch_mu);
    RowsumScratch& s = g_scratch[dev];
    if (s.cap < M) {
        if (s.ptr) QLLM_CUDA_TRY(cudaFree(s.ptr));
        s.ptr = nullptr; s.cap = 0;
        int64_t want = M < 4096 ? 4096 : M;
        QLLM_CUDA_TRY(cudaMalloc(&s.ptr, size_t(want) * sizeof(int32_t)));
        s.cap = want;
    }
    *out = s.ptr;
    return QLLM_OK;
}

int check_gemm_shape(int64_t M, int N, int K, int a_bits, int w_bits) {
    if (!bits_ok(a_bits) || !bits_ok(w_bits)) return QLLM_ERR_BITS;
    if (M < 0 || N <= 0 || K <= 0) return QLLM_ERR_SHAPE;
    if ((a_bits == 4 || w_bits == 4) && (K & 1)) return QLLM_ERR_SHAPE;
    return QLLM_OK;
}

// Token count from which expanding 4-bit operands to bytes once per call (a bandwidth-bound pre-pass
// over N*K + M*K codes) and running the byte-lane tensor-core kernel beats unpacking every tile in
// shared memory, which caps the tensor pipe near 40 %: more than three 128-row blocks (measured on the 4096- and
// 8192-channel shapes: 129-256 tokens a draw, 257-384 the in-kernel unpack wins, from 385 the expansion).
constexpr int64_t kExpandMinM = 385;
// Fewest tokens per chunk of a chunked host-buffer call.
constexpr int64_t kHostChunkRows = 512;

bool expand_path(int64_t M, int N, int K, int a_bits, int w_bits) {
    return M > 16 && M >= kExpandMinM && (a_bits == 4 || w_bits == 4) && qgemm_tc_supported(M, N, K, a_bits, w_bits);
}

// w_ready: the weight codes already expanded to bytes at the weight slot of this stream's expand scratch
// (done ahead of time on another stream by the layer object), or nullptr.
int dispatch_gemm(const uint8_t* a, const uint8_t* w, int64_t M, int N, int K, int a_bits, int w_bits,
                  const EpilogueArgs& ep, cudaStream_t st, bool may_allocate, const uint8_t* w_ready = nullptr,
                  bool weights_static = false) {
    if (M == 0) return QLLM_OK;
    if (M <= 16 && qgemm_decode_supported(M, N, K, a_bits, w_bits))
        return launch_qgemm_decode(a, w, M, N, K, a_bits, w_bits, ep, st);
    if (qgemm_tc_supported(M, N, K, a_bits, w_bits)) {
        const bool ap = a_bits == 4, wp = w_bits == 4;
        if (may_allocate && (ap || wp) && M >= kExpandMinM) {
            const size_t a_bytes = ap ? size_t(M) * K : 0, w_bytes = wp ? size_t(N) * K : 0;
            uint8_t* buf = nullptr;
            int rc = stream_scratch(kScratchExpand, st, a_bytes + w_bytes, &buf);
            if (rc != QLLM_OK) return rc;
            const bool reuse_w = wp && w_ready == buf + a_bytes;
            const bool writes = ap || (wp && !reuse_w);
            if (writes) { rc = scratch_write_begin(kScratchExpand, st, st); if (rc != QLLM_OK) return rc; }
            if (ap) { rc = launch_expand_codes(a, M, K, buf, st); if (rc != QLLM_OK) return rc; a = buf; }
            if (reuse_w) w = w_ready;
            else if (wp) { rc = launch_expand_codes(w, N, K, buf + a_bytes, st); if (rc != QLLM_OK) return rc; w = buf + a_bytes; }
            if (writes) { rc = scratch_write_end(kScratchExpand, st, st, nullptr); if (rc != QLLM_OK) return rc; }
            return launch_qgemm_tc(a, w, M, N, K, 8, 8, ep, st);
        }
        return launch_qgemm_tc(a, w, M, N, K, a_bits, w_bits, ep, st, weights_static);
    }
    return launch_qgemm_plain(a, w, M, N, K, a_bits, w_bits, ep, st);
}

}  // namespace

// Every argument check of the GEMM entry points, before anything is launched.
int gemm_check_args(const uint8_t* codes, const float* a_scale, const float* a_zero, const uint8_t* w_codes,
                    const float* w_scale, const float* w_zero, const int32_t* w_colsum, const void* out, int64_t M,
                    int N, int K, int a_bits, int w_bits, int out_dtype) {
    const int rc = check_gemm_shape(M, N, K, a_bits, w_bits);
    if (rc != QLLM_OK) return rc;
    if (!dtype_ok(out_dtype)) return QLLM_ERR_DTYPE;
    if (M == 0) return QLLM_OK;
    if (!codes || !a_scale || !a_zero || !w_codes || !w_scale || !w_zero || !w_colsum || !out)
        return QLLM_ERR_NULL;
    if (!aligned16(codes) || !aligned16(w_codes) || !aligned16(out)) return QLLM_ERR_ALIGN;
    return QLLM_OK;
}

int gemm_entry(const uint8_t* codes, const float* a_scale, const float* a_zero, const uint8_t* w_codes,
               const float* w_scale, const float* w_zero, const int32_t* w_colsum, const float* bias, void* out,
               int64_t M, int N, int K, int a_bits, int w_bits, int out_dtype, const int32_t* a_rowsum,
               cudaStream_t st, bool may_allocate, const uint8_t* w_ready, bool weights_static) {
    int rc = gemm_check_args(codes, a_scale, a_zero, w_codes, w_scale, w_zero, w_colsum, out, M, N, K, a_bits, w_bits,
                             out_dtype);
    if (rc != QLLM_OK) return rc;
    if (M == 0) return QLLM_OK;
    if (!a_rowsum) {
        if (!may_allocate) return QLLM_ERR_NULL;
        int32_t* scratch = nullptr;
        rc = rowsum_scratch(M, &scratch);
        if (rc != QLLM_OK) return rc;
        rc = launch_rowsum(codes, M, K, a_bits, scratch, st);
        if (rc != QLLM_OK) return rc;
        a_rowsum = scratch;
    }
    EpilogueArgs ep{a_scale, a_zero, a_rowsum, w_scale, w_zero, w_colsum, bias, out, out_dtype, 0};
    return dispatch_gemm(codes, w_codes, M, N, K, a_bits, w_bits, ep, st, may_allocate, w_ready, weights_static);
}

}  // namespace qllm

using namespace qllm;

struct qllm_layer {
    int C = 0, N = 0, a_bits = 0, w_bits = 0, x_dtype = 0, out_dtype = 0;
    int64_t max_M = 0, nnz = 0;
    float eps = 0.f;
    // device buffers
    float *gamma = nullptr, *beta = nullptr, *bias = nullptr, *coef = nullptr;
    int32_t *ptr = nullptr, *src = nullptr, *w_colsum = nullptr, *a_rowsum = nullptr;
    uint8_t *w_codes = nullptr, *codes = nullptr;
    float *w_scale = nullptr, *w_zero = nullptr, *a_scale = nullptr, *a_zero = nullptr;
    void *x_dev = nullptr, *out_dev = nullptr;   // staging for the host-buffer entry point
    uint8_t* map_image = nullptr;                // reassembly map compiled for the fused kernel (or null)
    MapCounts map_counts;                        // its counts of multi-entry rows
    // The byte expansion of the 4-bit weights that a large-M GEMM needs does not depend on the tokens, so the
    // pre-GEMM call starts it on a side stream; the GEMM call joins it.
    cudaStream_t side = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    // host-buffer calls of many tokens run in chunks so that the copy in, the kernels and the copy out overlap
    static constexpr int kHostChunks = 4;
    cudaStream_t h2d = nullptr, d2h = nullptr;
    cudaEvent_t ev_start = nullptr, ev_in[kHostChunks] = {}, ev_done[kHostChunks] = {};
    const uint8_t* w_ready = nullptr;            // expanded weights in flight / ready for the next GEMM call
    int64_t w_ready_M = -1;
    uint64_t w_epoch = 0;                        // version of the scratch contents when they were written
    // a host-buffer call in chunks expands the weights for its first chunk only: the later chunks read the same bytes
    bool hold_w = false;
    const uint8_t* held_w = nullptr;
    // 4-bit activations of a call that will take the byte-lane GEMM are written one code per byte by the
    // pre-GEMM kernel itself (no expansion pass): lane width of the codes now in the workspace
    int lane_bits = 0;
    // optional resident copy of the 4-bit weights, one code per byte (qllm_layer_keep_byte_weights): large-M calls
    // then widen nothing per call
    uint8_t* w_wide = nullptr;
    std::vector<void*> owned;
};

namespace {
template <typename T>
int dev_alloc(qllm_layer* L, T** p, size_t count) {
    void* q = nullptr;
    cudaError_t e = cudaMalloc(&q, count * sizeof(T) ? count * sizeof(T) : 16);
    if (e != cudaSuccess) { cuda_fail(e); return e == cudaErrorMemoryAllocation ? QLLM_ERR_NOMEM : QLLM_ERR_CUDA; }
    L->owned.push_back(q);
    *p = static_cast<T*>(q);
    return QLLM_OK;
}
template <typename T>
int dev_upload(qllm_layer* L, T** p, const T* host, size_t count) {
    int rc = dev_alloc(L, p, count);
    if (rc != QLLM_OK) return rc;
    QLLM_CUDA_TRY(cudaMemcpy(*p, host, count * sizeof(T), cudaMemcpyHostToDevice));
    return QLLM_OK;
}
}  // namespace

extern "C" {

static int reassemble_entry(const void* x, int x_dtype, int64_t M, int C, const float* ln_gamma,
                            const float* ln_beta, float ln_eps, const int32_t* map_ptr,
                            const int32_t* map_src, const float* map_coef, int bits, const void* map_image,
                            uint8_t* codes, float* a_scale, float* a_zero, int32_t* a_rowsum, void* stream,
                            bool byte_lanes = false, const MapCounts* counts = nullptr, bool share_sm = false) {
    if (!bits_ok(bits)) return QLLM_ERR_BITS;
    if (!dtype_ok(x_dtype)) return QLLM_ERR_DTYPE;
    if (M < 0 || C <= 0 || C > 49152 || (bits == 4 && (C & 1))) return QLLM_ERR_SHAPE;
    if (M == 0) return QLLM_OK;
    if (!x || !map_ptr || !map_src || !map_coef || !codes || !a_scale || !a_zero) return QLLM_ERR_NULL;
    if (!ln_gamma && ln_beta) return QLLM_ERR_NULL;        // no LayerNorm means neither parameter
    if (!aligned16(x) || !aligned16(codes)) return QLLM_ERR_ALIGN;
    return launch_reassemble_quant(x, x_dtype, M, C, ln_gamma, ln_beta, ln_eps, map_ptr, map_src,
                                   map_coef, bits, map_image, codes, a_scale, a_zero, a_rowsum,
                                   static_cast<cudaStream_t>(stream), byte_lanes, counts, share_sm);
}

int qllm_reassemble_quant(const void* x, int x_dtype, int64_t M, int C, const float* ln_gamma,
                          const float* ln_beta, float ln_eps, const int32_t* map_ptr,
                          const int32_t* map_src, const float* map_coef, int bits, uint8_t* codes,
                          float* a_scale, float* a_zero, int32_t* a_rowsum, void* stream) {
    return reassemble_entry(x, x_dtype, M, C, ln_gamma, ln_beta, ln_eps, map_ptr, map_src, map_coef, bits,
                            nullptr, codes, a_scale, a_zero, a_rowsum, stream);
}

int qllm_calib_absmax(const void* x, int x_dtype, int64_t M, int C, const float* ln_gamma,
                      const float* ln_beta, float ln_eps, float* absmax, void* stream) {
    if (!dtype_ok(x_dtype)) return QLLM_ERR_DTYPE;
    if (M < 0 || C <= 0 || C > 24576) return QLLM_ERR_SHAPE;
    if (M == 0) return QLLM_OK;
    if (!x || !ln_gamma || !absmax) return QLLM_ERR_NULL;
    if (!aligned16(x)) return QLLM_ERR_ALIGN;
    return launch_calib_absmax(x, x_dtype, M, C, ln_gamma, ln_beta, ln_eps, absmax,
                               static_cast<cudaStream_t>(stream));
}

int qllm_qgemm(const uint8_t* codes, const float* a_scale, const float* a_zero, const uint8_t* w_codes,
               const float* w_scale, const float* w_zero, const int32_t* w_colsum, const float* bias,
               void* out, int64_t M, int N, int K, int a_bits, int w_bits, int out_dtype,
               const int32_t* a_rowsum, void* stream) {
    return gemm_entry(codes, a_scale, a_zero, w_codes, w_scale, w_zero, w_colsum, bias, out, M, N, K, a_bits,
                      w_bits, out_dtype, a_rowsum, static_cast<cudaStream_t>(stream), true, nullptr);
}

int qllm_qgemm_acc(const uint8_t* codes, const uint8_t* w_codes, int32_t* acc, int64_t M, int N, int K,
                   int a_bits, int w_bits, void* stream) {
    int rc = check_gemm_shape(M, N, K, a_bits, w_bits);
    if (rc != QLLM_OK) return rc;
    if (M == 0) return QLLM_OK;
    if (!codes || !w_codes || !acc) return QLLM_ERR_NULL;
    if (!aligned16(codes) || !aligned16(w_codes) || !aligned16(acc)) return QLLM_ERR_ALIGN;
    EpilogueArgs ep{nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, acc, QLLM_F32, 1};
    return dispatch_gemm(codes, w_codes, M, N, K, a_bits, w_bits, ep, static_cast<cudaStream_t>(stream), true);
}

// ---------------------------------------------------------------------------- layer
int qllm_layer_create(const qllm_reassembly_t* h, const float* ln_gamma, const float* ln_beta,
                      float ln_eps, const float* bias, int a_bits, int x_dtype, int out_dtype,
                      int64_t max_M, qllm_layer_t** out) {
    if (!h || !ln_gamma || !out) return QLLM_ERR_NULL;
    if (!bits_ok(a_bits)) return QLLM_ERR_BITS;
    if (!dtype_ok(x_dtype) || !dtype_ok(out_dtype)) return QLLM_ERR_DTYPE;
    if (max_M <= 0) return QLLM_ERR_SHAPE;
    const int32_t *ptr, *src; const float* coef; int64_t nnz;
    const uint8_t* wc; int64_t wbytes; const float *ws, *wz; const int32_t* wcs;
    int64_t st[6];
    qllm_reassembly_map(h, &ptr, &src, &coef, &nnz);
    qllm_reassembly_weights(h, &wc, &wbytes, &ws, &wz, &wcs);
    qllm_reassembly_stats(h, st);
    const int C = int(st[3]), N = int(st[4]), w_bits = int(st[5]);
    if (a_bits == 4 && (C & 1)) return QLLM_ERR_SHAPE;
    qllm_layer* L = new (std::nothrow) qllm_layer();
    if (!L) return QLLM_ERR_NOMEM;
    L->C = C; L->N = N; L->a_bits = a_bits; L->w_bits = w_bits; L->x_dtype = x_dtype;
    L->out_dtype = out_dtype; L->max_M = max_M; L->nnz = nnz; L->eps = ln_eps;
    int rc = QLLM_OK;
    auto step = [&](int r) { if (rc == QLLM_OK) rc = r; };
    step(dev_upload(L, &L->gamma, ln_gamma, size_t(C)));
    if (ln_beta) step(dev_upload(L, &L->beta, ln_beta, size_t(C)));
    if (bias) step(dev_upload(L, &L->bias, bias, size_t(N)));
    step(dev_upload(L, &L->ptr, ptr, size_t(C) + 1));
    step(dev_upload(L, &L->src, src, size_t(nnz)));
    step(dev_upload(L, &L->coef, coef, size_t(nnz)));
    step(dev_upload(L, &L->w_codes, wc, size_t(wbytes)));
    step(dev_upload(L, &L->w_scale, ws, size_t(N)));
    step(dev_upload(L, &L->w_zero, wz, size_t(N)));
    step(dev_upload(L, &L->w_colsum, wcs, size_t(N)));
    const size_t image_bytes = reassemble_map_image_bytes(C, x_dtype);
    if (image_bytes) {
        step(dev_alloc(L, &L->map_image, image_bytes));
        if (rc == QLLM_OK) step(compile_reassemble_map(C, x_dtype, L->gamma, L->beta, L->ptr, L->src, L->coef, L->map_image, nullptr));
        if (rc == QLLM_OK) step(reassemble_map_counts(C, x_dtype, L->map_image, nullptr, &L->map_counts));
    }
    step(dev_alloc(L, &L->codes, size_t(max_M) * size_t(C)));   // room for one code per byte
    step(dev_alloc(L, &L->a_scale, size_t(max_M)));
    step(dev_alloc(L, &L->a_zero, size_t(max_M)));
    step(dev_alloc(L, &L->a_rowsum, size_t(max_M)));
    const size_t xb = x_dtype == QLLM_F32 ? 4 : 2, ob = out_dtype == QLLM_F32 ? 4 : 2;
    uint8_t *xd = nullptr, *od = nullptr;
    step(dev_alloc(L, &xd, size_t(max_M) * size_t(C) * xb));
    step(dev_alloc(L, &od, size_t(max_M) * size_t(N) * ob));
    L->x_dev = xd; L->out_dev = od;
    if (rc == QLLM_OK && w_bits == 4) {
        if (cudaStreamCreateWithFlags(&L->side, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&L->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&L->ev_join, cudaEventDisableTiming) != cudaSuccess)
            rc = cuda_fail(cudaGetLastError());
    }
    if (rc != QLLM_OK) { qllm_layer_destroy(L); return rc; }
    *out = L;
    return QLLM_OK;
}

void qllm_layer_destroy(qllm_layer_t* L) {
    if (!L) return;
    if (L->side) { cudaStreamSynchronize(L->side); cudaStreamDestroy(L->side); }
    if (L->ev_fork) cudaEventDestroy(L->ev_fork);
    if (L->ev_join) cudaEventDestroy(L->ev_join);
    if (L->h2d) { cudaStreamSynchronize(L->h2d); cudaStreamDestroy(L->h2d); }
    if (L->d2h) { cudaStreamSynchronize(L->d2h); cudaStreamDestroy(L->d2h); }
    if (L->ev_start) cudaEventDestroy(L->ev_start);
    for (cudaEvent_t e : L->ev_in) if (e) cudaEventDestroy(e);
    for (cudaEvent_t e : L->ev_done) if (e) cudaEventDestroy(e);
    for (void* p : L->owned) cudaFree(p);
    if (L->w_wide) cudaFree(L->w_wide);
    delete L;
}

int qllm_layer_reassemble_quant(qllm_layer_t* L, const void* x, int64_t M, void* stream) {
    if (!L || !x) return QLLM_ERR_NULL;
    if (M < 0 || M > L->max_M) return QLLM_ERR_SHAPE;
    L->w_ready = nullptr;
    const bool expand = !L->w_wide && expand_path(M, L->N, L->C, L->a_bits, L->w_bits);
    // 4-bit activations for a tensor-core GEMM (more than 16 tokens) are written one code per byte: the GEMM
    // then expands nothing on the activation side (below kExpandMinM tokens it unpacks only its weight tiles)
    const bool byte_lanes = L->a_bits == 4 && M > 16 && qgemm_tc_supported(M, L->N, L->C, L->a_bits, L->w_bits) &&
                            reassemble_byte_lanes_supported(L->C);
    L->lane_bits = (L->a_bits == 4 && !byte_lanes) ? 4 : 8;
    if (L->side && expand) {
        // start expanding the weights for the coming GEMM on the side stream: it is independent of the tokens
        cudaStream_t st = static_cast<cudaStream_t>(stream);
        const size_t a_bytes = L->lane_bits == 4 ? size_t(M) * L->C : 0, w_bytes = size_t(L->N) * L->C;
        uint8_t* buf = nullptr;
        int rc = stream_scratch(kScratchExpand, st, a_bytes + w_bytes, &buf);
        if (rc != QLLM_OK) return rc;
        if (!(L->hold_w && L->held_w == buf + a_bytes &&
              scratch_version(kScratchExpand, st) == L->w_epoch)) {
            QLLM_CUDA_TRY(cudaEventRecord(L->ev_fork, st));       // earlier users of the scratch are done
            QLLM_CUDA_TRY(cudaStreamWaitEvent(L->side, L->ev_fork, 0));
            rc = scratch_write_begin(kScratchExpand, st, L->side);  // another layer may be expanding there
            if (rc != QLLM_OK) return rc;
            rc = launch_expand_codes(L->w_codes, L->N, L->C, buf + a_bytes, L->side);
            if (rc != QLLM_OK) return rc;
            QLLM_CUDA_TRY(cudaEventRecord(L->ev_join, L->side));
            rc = scratch_write_end(kScratchExpand, st, L->side, &L->w_epoch);
            if (rc != QLLM_OK) return rc;
            if (L->hold_w) L->held_w = buf + a_bytes;
        }
        L->w_ready = buf + a_bytes;
        L->w_ready_M = M;
    }
    return reassemble_entry(x, L->x_dtype, M, L->C, L->gamma, L->beta, L->eps, L->ptr, L->src, L->coef,
                            L->a_bits, L->map_image, L->codes, L->a_scale, L->a_zero, L->a_rowsum, stream,
                            byte_lanes, L->map_image ? &L->map_counts : nullptr, L->w_ready != nullptr);
}

int qllm_layer_qgemm(qllm_layer_t* L, int64_t M, void* out, void* stream) {
    if (!L || !out) return QLLM_ERR_NULL;
    if (M < 0 || M > L->max_M) return QLLM_ERR_SHAPE;
    const uint8_t* w_ready = nullptr;
    if (L->w_ready && L->w_ready_M == M &&
        scratch_version(kScratchExpand, static_cast<cudaStream_t>(stream)) == L->w_epoch) {
        // the expanded weights are still this layer's (another layer or a direct call on the stream would have
        // bumped the version); otherwise the GEMM call expands them again itself
        QLLM_CUDA_TRY(cudaStreamWaitEvent(static_cast<cudaStream_t>(stream), L->ev_join, 0));
        w_ready = L->w_ready;
    }
    L->w_ready = nullptr;
    const int a_lane = L->lane_bits == 8 ? 8 : L->a_bits;
    // the resident byte copy serves every tensor-core call (same codes in 8-bit lanes: nothing is widened per call
    // from 385 tokens, no weight tile is unpacked in shared memory below); decode keeps streaming the 4-bit codes
    if (L->w_wide && M > 16 && qgemm_tc_supported(M, L->N, L->C, a_lane, 8))
        return gemm_entry(L->codes, L->a_scale, L->a_zero, L->w_wide, L->w_scale, L->w_zero, L->w_colsum, L->bias, out, M,
                          L->N, L->C, a_lane, 8, L->out_dtype, L->a_rowsum, static_cast<cudaStream_t>(stream), true,
                          nullptr, true);
    return gemm_entry(L->codes, L->a_scale, L->a_zero, L->w_codes, L->w_scale, L->w_zero, L->w_colsum, L->bias,
                      out, M, L->N, L->C, a_lane, L->w_bits, L->out_dtype, L->a_rowsum,
                      static_cast<cudaStream_t>(stream), true, w_ready, true);   // the layer's weights are written by no kernel
}

int qllm_layer_keep_byte_weights(qllm_layer_t* L, int keep, void* stream) {
    if (!L) return QLLM_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!keep) {
        if (L->w_wide) {
            QLLM_CUDA_TRY(cudaStreamSynchronize(st));             // a GEMM of this layer may still be reading it
            if (L->side) QLLM_CUDA_TRY(cudaStreamSynchronize(L->side));
            QLLM_CUDA_TRY(cudaFree(L->w_wide));
            L->w_wide = nullptr;
        }
        return QLLM_OK;
    }
    if (L->w_bits != 4 || L->w_wide) return QLLM_OK;              // nothing to widen / already there
    void* p = nullptr;
    if (cudaMalloc(&p, size_t(L->N) * size_t(L->C)) != cudaSuccess) { cudaGetLastError(); return QLLM_ERR_NOMEM; }
    int rc = launch_expand_codes(L->w_codes, L->N, L->C, static_cast<uint8_t*>(p), st);
    if (rc == QLLM_OK) {
        const cudaError_t e = cudaStreamSynchronize(st);
        if (e != cudaSuccess) rc = cuda_fail(e);
    }
    if (rc != QLLM_OK) { cudaFree(p); return rc; }
    L->w_wide = static_cast<uint8_t*>(p);
    L->w_ready = nullptr;
    return QLLM_OK;
}

int qllm_layer_forward(qllm_layer_t* L, const void* x, int64_t M, void* out, void* stream) {
    if (!L || !x || !out) return QLLM_ERR_NULL;
    int rc = qllm_layer_reassemble_quant(L, x, M, stream);
    if (rc != QLLM_OK) return rc;
    return qllm_layer_qgemm(L, M, out, stream);
}

int qllm_layer_forward_host(qllm_layer_t* L, const void* x_host, int64_t M, void* out_host, void* stream) {
    if (!L || !x_host || !out_host) return QLLM_ERR_NULL;
    if (M < 0 || M > L->max_M) return QLLM_ERR_SHAPE;
    if (M == 0) return QLLM_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t xb = L->x_dtype == QLLM_F32 ? 4 : 2, ob = L->out_dtype == QLLM_F32 ? 4 : 2;
    constexpr int NC = qllm_layer::kHostChunks;
    const int64_t rows = ((M + NC - 1) / NC + 127) / 128 * 128;      // tokens per chunk
    if (rows < kHostChunkRows || rows >= M) {
        // few tokens: one copy in, the path, one copy out
        QLLM_CUDA_TRY(cudaMemcpyAsync(L->x_dev, x_host, size_t(M) * L->C * xb, cudaMemcpyHostToDevice, st));
        int rc = qllm_layer_forward(L, L->x_dev, M, L->out_dev, stream);
        if (rc != QLLM_OK) return rc;
        QLLM_CUDA_TRY(cudaMemcpyAsync(out_host, L->out_dev, size_t(M) * L->N * ob, cudaMemcpyDeviceToHost, st));
        QLLM_CUDA_TRY(cudaStreamSynchronize(st));
        return QLLM_OK;
    }
    // Many tokens: the copies dominate (x in, out back over the host link), so the call is cut into chunks of
    // token rows: chunk k + 1 is copied in and chunk k - 1 copied out on two copy streams while chunk k runs.
    if (!L->h2d) {
        if (cudaStreamCreateWithFlags(&L->h2d, cudaStreamNonBlocking) != cudaSuccess ||
            cudaStreamCreateWithFlags(&L->d2h, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&L->ev_start, cudaEventDisableTiming) != cudaSuccess)
            return cuda_fail(cudaGetLastError());
        for (int k = 0; k < NC; ++k)
            if (cudaEventCreateWithFlags(&L->ev_in[k], cudaEventDisableTiming) != cudaSuccess ||
                cudaEventCreateWithFlags(&L->ev_done[k], cudaEventDisableTiming) != cudaSuccess)
                return cuda_fail(cudaGetLastError());
    }
    const char* xh = static_cast<const char*>(x_host);
    char* oh = static_cast<char*>(out_host);
    char* xd = static_cast<char*>(L->x_dev);
    char* od = static_cast<char*>(L->out_dev);
    QLLM_CUDA_TRY(cudaEventRecord(L->ev_start, st));                 // earlier work on the caller's stream first
    QLLM_CUDA_TRY(cudaStreamWaitEvent(L->h2d, L->ev_start, 0));
    int nk = 0;
    for (int64_t m0 = 0; m0 < M; m0 += rows, ++nk) {
        const int64_t mk = std::min<int64_t>(rows, M - m0);
        QLLM_CUDA_TRY(cudaMemcpyAsync(xd + size_t(m0) * L->C * xb, xh + size_t(m0) * L->C * xb, size_t(mk) * L->C * xb,
                                      cudaMemcpyHostToDevice, L->h2d));
        QLLM_CUDA_TRY(cudaEventRecord(L->ev_in[nk], L->h2d));
    }
    int rc = QLLM_OK;
    nk = 0;
    L->hold_w = true;                                              // one weight expansion serves all chunks
    L->held_w = nullptr;
    for (int64_t m0 = 0; m0 < M && rc == QLLM_OK; m0 += rows, ++nk) {
        const int64_t mk = std::min<int64_t>(rows, M - m0);
        cudaError_t e = cudaStreamWaitEvent(st, L->ev_in[nk], 0);
        if (e != cudaSuccess) { rc = cuda_fail(e); break; }
        rc = qllm_layer_forward(L, xd + size_t(m0) * L->C * xb, mk, od + size_t(m0) * L->N * ob, stream);
        if (rc != QLLM_OK) break;
        e = cudaEventRecord(L->ev_done[nk], st);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(L->d2h, L->ev_done[nk], 0);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(oh + size_t(m0) * L->N * ob, od + size_t(m0) * L->N * ob, size_t(mk) * L->N * ob,
                                cudaMemcpyDeviceToHost, L->d2h);
        if (e != cudaSuccess) { rc = cuda_fail(e); break; }
    }
    L->hold_w = false;
    L->held_w = nullptr;
    // nothing of this call may be in flight when it returns, whatever happened
    const cudaError_t e1 = cudaStreamSynchronize(L->h2d), e2 = cudaStreamSynchronize(st), e3 = cudaStreamSynchronize(L->d2h);
    if (rc != QLLM_OK) return rc;
    if (e1 != cudaSuccess) return cuda_fail(e1);
    if (e2 != cudaSuccess) return cuda_fail(e2);
    if (e3 != cudaSuccess) return cuda_fail(e3);
    return QLLM_OK;
}

int qllm_layer_workspace(qllm_layer_t* L, uint8_t** codes, float** a_scale, float** a_zero, int32_t** a_rowsum,
                         int* lane_bits) {
    if (!L) return QLLM_ERR_NULL;
    if (lane_bits) *lane_bits = L->lane_bits;
    if (codes) *codes = L->codes;
    if (a_scale) *a_scale = L->a_scale;
    if (a_zero) *a_zero = L->a_zero;
    if (a_rowsum) *a_rowsum = L->a_rowsum;
    return QLLM_OK;
}

// ---------------------------------------------------------------------------- diagnostics
const char* qllm_status_string(int s) {
    switch (s) {
        case QLLM_OK: return "ok";
        case QLLM_ERR_NULL: return "a required pointer is NULL";
        case QLLM_ERR_SHAPE: return "invalid shape";
        case QLLM_ERR_BITS: return "bit-width must be 4, 6 or 8";
        case QLLM_ERR_DTYPE: return "dtype must be QLLM_F32 or QLLM_BF16";
        case QLLM_ERR_MAP: return "malformed reassembly map";
        case QLLM_ERR_INFEASIBLE: return "channel count cannot be restored by assembly";
        case QLLM_ERR_CUDA: return "CUDA error (see qllm_last_cuda_error)";
        case QLLM_ERR_TIMEOUT: return "a bounded device-side wait expired";
        case QLLM_ERR_ALIGN: return "device tensor not 16-byte aligned";
        case QLLM_ERR_UNSUPPORTED: return "size beyond a documented limit";
        case QLLM_ERR_NOMEM: return "out of memory";
        default: return "unknown status";
    }
}

int qllm_last_cuda_error(void) { return g_last_cuda_error; }

int qllm_poll_status(void) {
    int v = 0;
    QLLM_CUDA_TRY(cudaDeviceSynchronize());
    QLLM_CUDA_TRY(cudaMemcpyFromSymbol(&v, g_status_word, sizeof(int)));
    if (v != 0) {
        const int zero = 0;
        QLLM_CUDA_TRY(cudaMemcpyToSymbol(g_status_word, &zero, sizeof(int)));
        return QLLM_ERR_TIMEOUT;
    }
    return QLLM_OK;
}

int64_t qllm_launch_count(void) { return g_launch_count.load(); }

}  // extern "C"
