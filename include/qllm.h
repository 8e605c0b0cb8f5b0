/*
 * qllm.h -- C ABI of the B200 (sm_100a) inference hot path of a QLLM quantized
 * linear layer (QLLM, arXiv 2310.08041).
 *
 * The path:  LayerNorm -> channel reassembly -> per-token asymmetric b-bit
 * quantization  (one fused kernel, qllm_reassemble_quant), then a low-bit
 * integer GEMM against offline-reassembled, per-output-channel quantized
 * weights with a dequantizing epilogue (qllm_qgemm).  The reassembly map and
 * the transformed weights are produced on the host by qllm_build_reassembly.
 *
 * LETTERS.  This header uses GEMM letters: M = tokens, C = K = input channels
 * of the linear layer, N = output channels.  (The paper's Eq. 1 writes M for
 * input channels, N for output channels and L for the sequence length.)
 *
 * CONVENTIONS.  Every function returns an int status: QLLM_OK (0) or a negative
 * QLLM_ERR_* code; nothing throws.  "device" pointers are CUDA global memory of
 * the device that is current when the call is made; "host" pointers are plain
 * host memory.  The caller owns every buffer it passes; the library keeps no
 * caller pointer after a call returns (device work may still be in flight on
 * `stream`, so buffers must stay valid until that stream reaches the call).
 * `stream` is a cudaStream_t passed as void* (NULL = default stream).  Device
 * calls are asynchronous on `stream`, never synchronize, and launch nothing when
 * they return an error found by argument checks.  Main device tensors (x, codes,
 * w_codes, out) must be 16-byte aligned (QLLM_ERR_ALIGN otherwise).  There is
 * no CPU fallback: without a usable CUDA device the device calls fail with
 * QLLM_ERR_CUDA.
 *
 * DEVICE MEMORY.  Which calls may call cudaMalloc / cudaFree:
 *   never      qllm_qgemm_noalloc, qllm_quantize_rows, qllm_calib_absmax, qllm_layernorm_rows,
 *              qllm_channel_distance, qllm_layer_forward / _reassemble_quant / _qgemm / _forward_host (everything a
 *              layer needs is taken in qllm_layer_create and returned in qllm_layer_destroy);
 *   grow-only  qllm_reassemble_quant (compiled-map scratch per (device, stream): grown on the first call
 *              and when C grows), qllm_qgemm and qllm_qgemm_acc (row-sum scratch when a_rowsum = NULL;
 *              widened-code scratch for a 4-bit operand at M >= 385): library-owned buffers, sized by the
 *              largest call so far, kept until the process exits;
 *   always     the offline calls qllm_build_reassembly_eq5 and qllm_search_theta (take and return what
 *              they need inside the call), qllm_layer_create and qllm_layer_keep_byte_weights.
 * qllm_layer_forward_host takes no memory either (its device staging comes from qllm_layer_create); its first
 * chunked call creates two streams and a few events, which the layer keeps.
 * A grow-only call that found its scratch large enough launches kernels only.
 */
#ifndef QLLM_H_
#define QLLM_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- status codes -------------------------------------------------------- */
#define QLLM_OK               0
#define QLLM_ERR_NULL        (-1)  /* a required pointer is NULL                         */
#define QLLM_ERR_SHAPE       (-2)  /* M < 0, C/K/N <= 0, odd channel count for 4-bit ...  */
#define QLLM_ERR_BITS        (-3)  /* bit-width not in {4, 6, 8}                          */
#define QLLM_ERR_DTYPE       (-4)  /* dtype selector not in {QLLM_F32, QLLM_BF16}         */
#define QLLM_ERR_MAP         (-5)  /* reassembly map malformed (host-side checks only)   */
#define QLLM_ERR_INFEASIBLE  (-6)  /* builder cannot bring the channel count back to C   */
#define QLLM_ERR_CUDA        (-7)  /* CUDA runtime error; see qllm_last_cuda_error()      */
#define QLLM_ERR_TIMEOUT     (-8)  /* a bounded device-side wait expired                  */
#define QLLM_ERR_ALIGN       (-9)  /* a main device tensor is not 16-byte aligned         */
#define QLLM_ERR_UNSUPPORTED (-10) /* size beyond a documented limit                      */
#define QLLM_ERR_NOMEM       (-11) /* allocation failed                                   */

#define QLLM_F32  0
#define QLLM_BF16 1

/* ==========================================================================
 * 1. Fused pre-GEMM kernel                        (device, asynchronous)
 * ==========================================================================
 * For every token row m of x[M][C]:
 *
 *   y   = LayerNorm(x_m)            y_k = (x_k - mean) / sqrt(var + ln_eps) * gamma_k + beta_k,
 *                                   biased variance over the C channels.  LayerNorm is the
 *                                   non-linear layer in front of the projection that makes a
 *                                   runtime reassembly step necessary (Sec. 4.3, "Inference
 *                                   efficiency"); fusing it with the reassembly is the
 *                                   paper's stated future work (Sec. 6).
 *   x'_c = sum_{j in [map_ptr[c], map_ptr[c+1])} map_coef[j] * y[map_src[j]],   c = 0..C-1
 *                                   channel disassembly (Eq. 3: an outlier channel becomes T
 *                                   rows (src = i, coef = 1/T)) and channel assembly (Eq. 4:
 *                                   a merged set becomes one row listing its members with
 *                                   coef = 1/|set|) in one sparse map with exactly C rows.
 *   quantize x' per token (Eq. 2):  alpha = (max x' - min x') / (2^bits - 1),
 *                                   zero  = -round(min x' / alpha),
 *                                   q_c   = clamp(round(x'_c / alpha) + zero, 0, 2^bits - 1),
 *                                   round = nearest, ties to even.  A constant row takes
 *                                   alpha = |value| (1 if the value is 0).
 *
 *  x         device, [M][C] row-major, float32 (x_dtype = QLLM_F32) or bfloat16 (QLLM_BF16)
 *  ln_gamma  device float[C];  ln_beta device float[C] or NULL (= 0).  ln_gamma = NULL (then ln_beta
 *            = NULL too): no LayerNorm, x already is the linear layer's input -- the case of Appendix B,
 *            where a preceding linear layer absorbed the map (qllm_fold_previous) and the map passed
 *            here is the identity.  This mode runs on the shape-agnostic kernel.
 *  map_ptr   device int32[C+1], map_src device int32[nnz], map_coef device float[nnz];
 *            rows non-empty, 0 <= src < C.  The map is NOT validated on the device: use
 *            qllm_validate_map on the host copy if it does not come from the builder.
 *  bits      4, 6 or 8
 *  codes     device out.  bits = 4: uint8[M][C/2], byte k holds channel 2k in its low nibble
 *            and channel 2k+1 in its high nibble (C must be even).  bits = 6 or 8: uint8[M][C].
 *  a_scale   device out float[M]  (alpha)
 *  a_zero    device out float[M]  (zero-point, integer-valued)
 *  a_rowsum  device out int32[M] or NULL: sum_c q_c, needed by the GEMM epilogue
 *  M = 0 is a successful no-op.  C <= 49152 (the normalised row is held in shared memory).
 *
 *  Cost of the direct call.  The kernel reads the map in a compiled form (per-source weights, gather positions,
 *  records of the merged rows).  This call receives plain CSR arrays that it may not keep and whose contents the
 *  caller may change between calls.  It therefore keeps the compiled form of the last map used on `stream` in
 *  scratch the library owns per (device, stream), beside a 64-bit hash of everything the form depends on (C, the
 *  three map arrays, ln_gamma, ln_beta: contents, not addresses).  Every call launches one single-CTA kernel ahead
 *  of the main one that hashes the arrays it was given and recompiles only when the hash differs from the one
 *  kept (two different contents share a hash with probability 2^-64).  Bf16 rows of 4096 / 5120 / 8192 channels:
 *  the call also launches the shape-agnostic kernel behind the main one, which returns at once unless the map
 *  is one the main kernel declines (a source channel read with different coefficients: no product of Eq. 3 /
 *  Eq. 4, but a legal argument).  Measured at M = 2048, C = 4096 with a cold L2: 49 us per call with the map
 *  unchanged, 60 us when it is recompiled, against 27 us for the same kernel launched by a layer object
 *  (section 5), which compiles its map once in qllm_layer_create and knows its sizes: use a layer wherever the
 *  map is fixed.
 */
int qllm_reassemble_quant(const void* x, int x_dtype, int64_t M, int C,
                          const float* ln_gamma, const float* ln_beta, float ln_eps,
                          const int32_t* map_ptr, const int32_t* map_src, const float* map_coef,
                          int bits, uint8_t* codes, float* a_scale, float* a_zero,
                          int32_t* a_rowsum, void* stream);

/* The per-token quantizer of Eq. 2 alone (device, asynchronous): alpha, zero-point, codes and code sum of every
 * row of x[M][C], exactly as in qllm_reassemble_quant but with no LayerNorm and no map.  This is the run-time half
 * of the pre-GEMM stage when the reassembly has been folded into the layer that produces x (Appendix B,
 * qllm_fold_previous): that layer already emits the reassembled channels.  Arguments, layouts and errors as in
 * qllm_reassemble_quant.  bf16 rows of up to 8192 channels and fp32 rows of up to 4096 (C a multiple of 256) are
 * read from memory once. */
int qllm_quantize_rows(const void* x, int x_dtype, int64_t M, int C, int bits,
                       uint8_t* codes, float* a_scale, float* a_zero, int32_t* a_rowsum, void* stream);

/* ==========================================================================
 * 2. Low-bit integer GEMM with dequantizing epilogue   (device, asynchronous)
 * ==========================================================================
 * Eq. 1 evaluated on quantized operands, Y = quant(X') quant(W') (Sec. 4.1.3),
 * activations quantized per token and weights per output channel (Sec. 5,
 * implementation details):
 *
 *   acc[m][n] = sum_k qa[m][k] * qw[n][k]                                   (int32, exact)
 *   I[m][n]   = acc - w_zero[n]*a_rowsum[m] - a_zero[m]*w_colsum[n] + K*a_zero[m]*w_zero[n]
 *   out[m][n] = a_scale[m] * w_scale[n] * I[m][n] + bias[n]
 *
 * which is Eq. 2 inverted on both operands: sum_k a_s(qa - za) * w_s(qw - zw).
 *
 *  codes     device, activations as written by qllm_reassemble_quant with bits = a_bits
 *  w_codes   device, [N][K/2] packed like `codes` (w_bits = 4) or uint8[N][K] (6, 8)
 *  w_scale, w_zero   device float[N];  w_colsum device int32[N] = sum_k qw[n][k]
 *  bias      device float[N] or NULL
 *  out       device, [M][N] row-major, float32 or bfloat16 (round to nearest even)
 *  a_rowsum  device int32[M], or NULL: the row sums are then computed by a pre-pass into a
 *            library-owned scratch buffer (grown with cudaMalloc when M exceeds what earlier
 *            calls needed, so pass a_rowsum on allocation-free paths).
 *  K must be even when either operand is 4-bit.  |I| must fit an int32.
 *  Dispatch: M <= 16 takes a weight-streaming kernel (weights read once); larger M takes the
 *  tensor-core kernel when the shape allows it, else a plain kernel.  With a 4-bit operand and
 *  M >= 385 the 4-bit codes are first widened to byte lanes, once per call, into a second
 *  library-owned scratch buffer kept per (device, stream) and grown with cudaMalloc like the
 *  row-sum scratch (N*K + M*K bytes at most); qllm_qgemm_noalloc never does this.
 */
int qllm_qgemm(const uint8_t* codes, const float* a_scale, const float* a_zero,
               const uint8_t* w_codes, const float* w_scale, const float* w_zero,
               const int32_t* w_colsum, const float* bias, void* out,
               int64_t M, int N, int K, int a_bits, int w_bits, int out_dtype,
               const int32_t* a_rowsum, void* stream);

/* Allocation-free variant of qllm_qgemm (the paper has no counterpart; it exists for callers
 * that cannot call cudaMalloc: code inside a caller-managed memory pool or a latency-critical
 * serving loop, where an allocation may synchronise the device or fail, and processes that
 * have given all device memory to another allocator).  It always computes the activation row
 * sums itself, into a fixed array of QLLM_NOALLOC_MAX_M int32 (256 KiB) that is part of the
 * library image: every GPU that loads the library holds it until the process exits.  It calls
 * no cudaMalloc / cudaFree and no allocating library routine.
 *  - M > QLLM_NOALLOC_MAX_M returns QLLM_ERR_UNSUPPORTED; all other arguments and errors are
 *    those of qllm_qgemm (without a_rowsum).
 *  - The first call on a device looks up the array's device address; make that first call
 *    before any stream capture begins.
 *  - All calls on a device share the one array.  Each call overwrites the M entries it uses
 *    before reading them, so nothing from an earlier call leaks in; but two calls whose work
 *    overlaps on the GPU (different streams) race on it: serialise them.
 */
#define QLLM_NOALLOC_MAX_M 65536
int qllm_qgemm_noalloc(const uint8_t* codes, const float* a_scale, const float* a_zero,
                       const uint8_t* w_codes, const float* w_scale, const float* w_zero,
                       const int32_t* w_colsum, const float* bias, void* out,
                       int64_t M, int N, int K, int a_bits, int w_bits, int out_dtype,
                       void* stream);

/* Debug twin of qllm_qgemm: writes the raw int32 accumulators acc[M][N] (same dispatch and
 * kernels, epilogue replaced by a plain store), so that the integer sum can be compared bit
 * for bit with a reference. */
int qllm_qgemm_acc(const uint8_t* codes, const uint8_t* w_codes, int32_t* acc,
                   int64_t M, int N, int K, int a_bits, int w_bits, void* stream);

/* ==========================================================================
 * 3. Calibration statistic                        (device, asynchronous)
 * ==========================================================================
 * absmax[k] = max(absmax[k], max_m |LayerNorm(x_m)_k|): the per-channel maximum of the layer
 * input that Algorithm 1 starts from ("max value of each channel").  absmax must be
 * zero-filled before the first call; calls accumulate, so calibration batches can be streamed.
 * C <= 24576.
 */
int qllm_calib_absmax(const void* x, int x_dtype, int64_t M, int C,
                      const float* ln_gamma, const float* ln_beta, float ln_eps,
                      float* absmax, void* stream);

/* ==========================================================================
 * 4. Offline builder                                   (host only, synchronous)
 * ==========================================================================
 * Turns per-channel calibration maxima into the reassembly map and the transformed,
 * quantized weights of one linear layer:
 *
 *   T_i = max(1, ceil(absmax_i / theta))                     sub-channel count, Sec. 4.1.1
 *   expanded list: channel i -> T_i consecutive entries x_i / T_i (Eq. 3); E = sum(T_i - 1)
 *   E merges by bipartite soft matching (Appendix A): eligible entries (not born from
 *   disassembly, Sec. 4.1.2) at even list positions form set A, at odd positions set B;
 *   each a picks the b with the smallest |absmax_a - absmax_b| (ties: lowest position); the E
 *   shortest edges are kept (ties: lowest a); a joins b's set, which stays at b's position and
 *   carries the mean of its members (Eq. 4); merged a's are removed.  When one round cannot
 *   supply E merges, all of A is merged and further rounds run on the shortened list.
 *   W'[n][c] = sum_{j in row c} W[n][src_j]  (+ (A B)[c][n], the low-rank correction of
 *   Sec. 4.2, folded in before quantization), then Eq. 2 per output channel n.
 *
 *  calib_absmax  host float[C];  theta > 0
 *  W             host float[N][C] (output-channel major); N > 0
 *  lr_A, lr_B    host float[C][r] (reassembled channel order) and float[r][N]; both NULL = none
 *  w_bits        4, 6 or 8
 *  out           receives a handle owned by the caller; release with qllm_free_reassembly
 * Errors: QLLM_ERR_INFEASIBLE when no eligible pair is left before the count is back to C.
 */
typedef struct qllm_reassembly qllm_reassembly_t;

int qllm_build_reassembly(const float* calib_absmax, int C, float theta,
                          const float* W, int N,
                          const float* lr_A, const float* lr_B, int r,
                          int w_bits, qllm_reassembly_t** out);
void qllm_free_reassembly(qllm_reassembly_t* h);

/* The same builder with the distance of Eq. 5 in the bipartite matching (Sec. 4.1.2; the paper names these
 * pairwise distances as the main cost of reassembly): D(i, j) = 1/4 ||y_i - y_j||^2 ||W_i - W_j||^2, y_i the
 * column of channel i over the T calibration rows of the layer's input, W_i the weights of input channel i.
 *  calib_y   DEVICE float[T][C]: the layer's input of the calibration tokens (qllm_layernorm_rows makes it)
 *  W         host float[N][C] as above (copied to the device for the duration of the call)
 *  stream    the device work (nearest-neighbour search: for every entry of set A the nearest entry of set B,
 *            Appendix A step 2) runs there; the call waits for it.  Only those |A| edges come back to the host.
 * Nearest counterpart, tie rules and edge selection are those of qllm_build_reassembly with D(a, b) in place of
 * |m_a - m_b|; D is evaluated in float32.  Eq. 5 is defined between undivided channels, so only one matching
 * round is possible: a threshold that needs a second round returns QLLM_ERR_UNSUPPORTED.  A row of distances
 * without a finite value returns QLLM_ERR_MAP.  Offline step: allocates and frees device memory. */
int qllm_build_reassembly_eq5(const float* calib_absmax, int C, float theta,
                              const float* calib_y, int64_t T,
                              const float* W, int N,
                              const float* lr_A, const float* lr_B, int r,
                              int w_bits, void* stream, qllm_reassembly_t** out);

/* The builder driven by a caller-made distance table: dist is a HOST float[C][C], dist[a][b] takes the place of
 * |m_a - m_b| (same rules, one round only, QLLM_ERR_MAP for a row without a finite value).  qllm_channel_distance
 * makes the Eq. 5 table on the device when the whole table is wanted. */
int qllm_build_reassembly_dist(const float* calib_absmax, int C, float theta, const float* dist,
                               const float* W, int N,
                               const float* lr_A, const float* lr_B, int r,
                               int w_bits, qllm_reassembly_t** out);

/* Build-time device helpers (asynchronous on stream; all pointers DEVICE).
 * qllm_layernorm_rows: y[t][c] = LayerNorm(x[t])[c] as float32, the linear layer's input of the calibration
 * tokens (x [T][C] in x_dtype, ln_beta may be NULL).
 * qllm_channel_distance: D[i][j] of Eq. 5 from y [T][C] and the layer's weights W [N][C] (output channel major,
 * float32), D float[C][C].  The table decides an argmin, so its arithmetic is fixed: float32, rows taken in
 * order with one fused multiply-add each (dx = fma(e, e, dx), e = y[t][i] - y[t][j]; dw likewise over W's rows),
 * D = (0.25f * dx) * dw; the result is bit-reproducible and symmetric. */
int qllm_layernorm_rows(const void* x, int x_dtype, int64_t T, int C, const float* ln_gamma,
                        const float* ln_beta, float ln_eps, float* y, void* stream);
int qllm_channel_distance(const float* y, int64_t T, const float* W, int N, int C, float* D, void* stream);

/* Borrowed host pointers into the handle (valid until qllm_free_reassembly). */
int qllm_reassembly_map(const qllm_reassembly_t* h, const int32_t** map_ptr,
                        const int32_t** map_src, const float** map_coef, int64_t* nnz);
int qllm_reassembly_weights(const qllm_reassembly_t* h, const uint8_t** w_codes, int64_t* w_bytes,
                            const float** w_scale, const float** w_zero,
                            const int32_t** w_colsum);
/* stats[0] = E (channels added by disassembly = merges done), stats[1] = rows with more than
 * one member, stats[2] = matching rounds, stats[3] = C, stats[4] = N, stats[5] = w_bits */
int qllm_reassembly_stats(const qllm_reassembly_t* h, int64_t stats[6]);

/* Appendix B: when the layer in front of the quantized layer is itself linear, the map needs no run-time
 * kernel: it is applied once to that layer's output channels.  W_prev is HOST float[C_src][C_in] (output
 * channel major; C_src = number of source channels the map refers to), bias_prev HOST float[C_src] or NULL;
 * W_out HOST float[C][C_in] and bias_out HOST float[C] receive  row c = sum_j coef_j * row src_j  (a
 * sub-channel becomes the source row divided by T, a merged channel the mean of its members' rows), summed in
 * double in entry order.  x W_out^T + bias_out then equals the map applied to x W_prev^T + bias_prev. */
int qllm_fold_previous(const int32_t* map_ptr, const int32_t* map_src, const float* map_coef, int C,
                       const float* W_prev, const float* bias_prev, int C_in, float* W_out, float* bias_out);

/* Host-side structural check of a map: ptr[0] = 0, rows non-empty and monotone, 0 <= src < C. */
int qllm_validate_map(const int32_t* map_ptr, const int32_t* map_src, int C, int64_t nnz);

/* theta = nearest-rank percentile of the channel maxima: sorted ascending, element
 * ceil(pct * C) - 1.  Returns 0 on bad arguments. */
float qllm_theta_percentile(const float* absmax, int C, double pct);
/* A theta for which disassembly adds exactly `extra` channels: the midpoint of the interval of
 * thresholds on which E(theta) = extra.  Returns 0 when that interval is empty. */
float qllm_theta_for_extra(const float* absmax, int C, int extra);

/* Adaptive threshold search (Algorithm 1; host-orchestrated, offline, waits for the device).
 * For p = 1..P the threshold theta_p = min(m) + p/P (max(m) - min(m)) over the calibration maxima m is tried:
 * the reassembly is built (qllm_build_reassembly, no low-rank term: the search precedes error correction),
 * the calibration tokens run through the reassembled, quantized layer (sections 1 + 2, fp32 output), and the
 * reassembly error  L = || LayerNorm(x) W^T - quant(X^) quant(W^) ||_F^2  (Eq. 6, read on the layer's own
 * output) is summed in fp64 against an fp32 reference product computed once.  *theta_out is the first
 * threshold with the smallest error; losses_out[p-1] (host double[P], may be NULL) receives every error,
 * +inf for a threshold whose map cannot restore the channel count.
 *  calib_x   device [T][C] (x_dtype), 16-byte aligned, T <= 2^24
 *  ln_gamma, ln_beta, calib_absmax, W   HOST (as for qllm_layer_create / qllm_build_reassembly)
 * Allocates device memory for W, the reference and one layer object per candidate and frees it before
 * returning. */
int qllm_search_theta(const void* calib_x, int x_dtype, int64_t T, int C, const float* ln_gamma,
                      const float* ln_beta, float ln_eps, const float* calib_absmax, const float* W, int N,
                      int a_bits, int w_bits, int P, float* theta_out, double* losses_out, void* stream);

/* ==========================================================================
 * 5. Layer object: device-resident map, weights and workspace
 * ==========================================================================
 * Convenience for callers that hold host data: uploads a built reassembly to the current
 * device once and runs sections 1 + 2 back to back.  All allocation happens in
 * qllm_layer_create; the forward calls allocate nothing.
 *  x_dtype/out_dtype  QLLM_F32 or QLLM_BF16;  max_M = largest token count of a forward call
 *  ln_gamma host float[C]; ln_beta host float[C] or NULL; bias host float[N] or NULL
 */
typedef struct qllm_layer qllm_layer_t;

int qllm_layer_create(const qllm_reassembly_t* h, const float* ln_gamma, const float* ln_beta,
                      float ln_eps, const float* bias, int a_bits, int x_dtype, int out_dtype,
                      int64_t max_M, qllm_layer_t** out);
void qllm_layer_destroy(qllm_layer_t* layer);
/* x, out: device.  Asynchronous on stream.
 * Stream capture: once a call of the same M has run on the stream (scratch sized, kernel attributes set), a
 * later call issues only capturable work -- kernel launches and the event fork/join of the internal stream
 * that expands 4-bit weights -- so it may be recorded into a CUDA graph.  The graph holds the scratch
 * pointers of that moment: create every layer that will run on the stream, and run each once at its largest
 * M, before capturing.  Capture whole forwards (both halves inside the capture or both outside it), and do
 * not replay a graph between the two half-step calls of another layer on the same stream. */
int qllm_layer_forward(qllm_layer_t* layer, const void* x, int64_t M, void* out, void* stream);
/* The two halves of qllm_layer_forward, for callers that time or schedule them separately:
 * qllm_layer_reassemble_quant runs the fused pre-GEMM kernel on x[M][C] (device) into the layer's
 * workspace; qllm_layer_qgemm multiplies that workspace (M rows of the last pre-GEMM call) with the
 * layer's weights into out[M][N] (device).  Asynchronous on stream. */
int qllm_layer_reassemble_quant(qllm_layer_t* layer, const void* x, int64_t M, void* stream);
int qllm_layer_qgemm(qllm_layer_t* layer, int64_t M, void* out, void* stream);
/* Memory for time, opt-in: keep != 0 gives a layer with 4-bit weights a second, resident copy of them with one
 * code per byte (N * C bytes of device memory; cudaMalloc + one kernel on stream, the call waits for it).  Calls
 * of 385 tokens and more then skip the per-call widening of the weights (a read of N*C/2 and a write of N*C bytes
 * that runs beside the pre-GEMM kernel: 13-17 us of a 95 us step at M = 2048, C = 4096, N = 12288), calls of 17 to
 * 384 tokens read byte tiles instead of unpacking 4-bit tiles in shared memory (2-3 us of 35); the decode path
 * (M <= 16) keeps streaming the 4-bit codes.  Results are bit-identical either way.  keep = 0 waits for
 * stream and frees the copy.  Not to be called while a forward of this layer is being issued from another thread. */
int qllm_layer_keep_byte_weights(qllm_layer_t* layer, int keep, void* stream);
/* x, out: HOST (pinned memory makes the copies asynchronous).  Copies x to the device, runs the
 * path, copies out back and waits until all of it is done.  Calls of 2048 tokens or more are cut into four
 * chunks of token rows whose copy in, kernels and copy out overlap on two internal copy streams (the host link
 * carries both directions at once); results are those of qllm_layer_forward. */
int qllm_layer_forward_host(qllm_layer_t* layer, const void* x_host, int64_t M, void* out_host,
                            void* stream);
/* Borrowed DEVICE pointers of the layer's quantized-activation workspace of the last forward.
 * *lane_bits (may be NULL) receives how the codes are stored: 4 = two per byte as qllm_reassemble_quant
 * writes 4-bit codes, 8 = one per byte [M][C].  4-bit activations are stored one per byte when the
 * call's GEMM runs on byte lanes (M >= 385 on the tensor-core path): the pre-GEMM kernel then writes
 * the lanes the GEMM reads, which saves a widening pass; the code VALUES are the same. */
int qllm_layer_workspace(qllm_layer_t* layer, uint8_t** codes, float** a_scale, float** a_zero,
                         int32_t** a_rowsum, int* lane_bits);

/* ==========================================================================
 * 6. Diagnostics
 * ========================================================================== */
const char* qllm_status_string(int status);
/* Last cudaError_t seen by this library on the calling thread (0 = none). */
int qllm_last_cuda_error(void);
/* Reads (and clears) the device-side status word of the current device: QLLM_OK, or
 * QLLM_ERR_TIMEOUT if a bounded wait inside a kernel expired since the last poll.
 * Synchronizes the device. */
int qllm_poll_status(void);
/* Exercises the expiry path of the bounded device-side waits (every mbarrier wait of the tensor-core GEMM
 * kernels gives up after ~2^32 cycles, raises the status word and lets its CTA wind down; the paper has no
 * counterpart).  Launches one warp that waits, with the same routine under a limit of 2^20 cycles, for a barrier
 * nobody arrives on: the wait runs out, the status word is set, the kernel returns.  Nothing faults, traps or
 * spins without bound.  *gave_up (device int) becomes 1.  Afterwards qllm_poll_status() returns
 * QLLM_ERR_TIMEOUT once and QLLM_OK again; other calls are unaffected.  Asynchronous on `stream`. */
int qllm_debug_wait_expiry(int* gave_up, void* stream);
/* Number of kernel launches issued by this library in this process (all threads). */
int64_t qllm_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* QLLM_H_ */
