/*
 * qblora.h -- C ABI of the B200 (sm_100a) adapted quantized linear layer of
 * Q-BLoRA / QA-BLoRA (arXiv 2407.17029).
 *
 * Notation.  The paper writes the base weight W as D_in x D_out with y = W^T x
 * (Sec. 3.1).  This library stores it row-major as W_s[o][i] = W[i][o]
 * ("[out][in]", D_in contiguous).  T = tokens, g = block_in, G = D_in / g,
 * P = D_in / lambda_in, Q = D_out / lambda_out, r = adapter inner dimension
 * (the paper's lambda * D_rank, Sec. 3.2).
 *
 * Ownership.  Every pointer in a struct or argument list marked DEVICE is a
 * CUDA device pointer owned by the caller, 16-byte aligned; the library never
 * allocates or frees device memory in these calls.  Pointers marked HOST are
 * ordinary host memory read during the call.  Scratch memory is the caller's
 * `ws` buffer of at least qblora_workspace_bytes(...) bytes; its contents are
 * undefined after a call, and two calls that may run concurrently on the GPU
 * need separate `ws` buffers.
 *
 * Streams.  Work is enqueued on the given stream (a cudaStream_t passed as
 * void*, NULL = default stream), with ONE exception: qblora_linear_bwd runs its
 * adapter-gradient chain on a second stream that the library creates on first
 * use and keeps (one non-blocking stream and three events per host thread and
 * device, never destroyed).  That stream is forked from `stream` at entry and
 * joined back into it before the call returns -- also when the call returns an
 * error after the fork -- so the caller sees ordinary stream semantics, inside a
 * stream capture too.  All caller streams of one host thread share that second
 * stream: do not capture qblora_linear_bwd on one stream while the same thread
 * runs it un-captured on another.
 *
 * State the library keeps between calls (none of it per call):
 *   - the second stream and events above (thread-local);
 *   - per-kernel "shared-memory attribute set" flags and the SM count (atomic,
 *     set once);
 *   - the device address of the built-in scratch of qablora_merge_noalloc, per
 *     device (atomic, set once);
 *   - the launch counter and the armed event pair of the instrumentation calls,
 *     and the values set by the qblora_debug_* test hooks (atomic / thread-local).
 * Every entry point may be called from several host threads at once; calls that
 * share a `ws` buffer, or qablora_merge_noalloc calls on one device, must be
 * serialised by the caller.
 *
 * Errors.  Every call returns a qblora_status; nothing throws or aborts.
 * Argument checks are made on the host before any launch.  Device-side waits
 * are bounded: a kernel that gives up stores QBLORA_ERR_TIMEOUT into the first
 * word of `ws`, which qblora_device_status() reads back.
 *
 * Determinism.  No floating-point atomics: equal inputs give bit-equal outputs.
 */
#ifndef QBLORA_H_
#define QBLORA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  QBLORA_OK = 0,
  QBLORA_ERR_INVALID_ARG = 1, /* null / misaligned pointer, sizes that do not divide, tokens < 1 */
  QBLORA_ERR_UNSUPPORTED = 2, /* valid request the library has no kernel for */
  QBLORA_ERR_WORKSPACE = 3,   /* ws == NULL or ws_bytes too small */
  QBLORA_ERR_CUDA = 4,        /* a CUDA runtime call or launch failed */
  QBLORA_ERR_TIMEOUT = 5,     /* a bounded device-side wait gave up (see qblora_device_status) */
  QBLORA_ERR_TOO_LARGE = 6    /* qablora_merge_noalloc only: the adapter is larger than its built-in scratch */
} qblora_status;

typedef enum {
  /* w~ = alpha * code[c]; alpha = max|w| of the block, no beta.  Sec. 3.2 (the 4-bit
   * normal-quantile base format of Q-BLoRA) with Eq. 1's absmax scaling. */
  QBLORA_FMT_CODEBOOK_ABSMAX = 0,
  /* w~ = alpha * c + beta; alpha = (max - min) / 15, beta = min.  Eq. 1, min-max, N = 4
   * (the format QA-BLoRA merges into, Sec. 3.3). */
  QBLORA_FMT_AFFINE_MINMAX = 1
} qblora_qfmt;

typedef enum { QBLORA_F32 = 0, QBLORA_BF16 = 1 } qblora_dtype;

typedef enum {
  QBLORA_OP_QUANTIZE = 0,
  QBLORA_OP_LINEAR_FWD = 1,
  QBLORA_OP_LINEAR_BWD = 2,
  QBLORA_OP_MERGE = 3,
  QBLORA_OP_LOWBIT_GEMM = 4,
  QBLORA_OP_MERGE_DENSE = 5
} qblora_op;

/* Frozen block-wise 4-bit weight: the triplet (w^, alpha, beta) of Eq. 1 / Sec. 3.3. */
typedef struct {
  int32_t d_in, d_out;         /* paper D_in, D_out */
  int32_t block_in, block_out; /* quantization block: block_out rows x block_in columns of W_s */
  int32_t qfmt;                /* qblora_qfmt */
  float code[16];              /* HOST values, ascending; level table (code-table format only) */
  const uint8_t* codes;        /* DEVICE [d_out][d_in/2]; byte k of row o: low nibble = code(o,2k),
                                  high nibble = code(o,2k+1) */
  const float* alpha;          /* DEVICE [d_out/block_out][d_in/block_in] */
  const float* beta;           /* DEVICE same shape; NULL for the code-table format */
  int32_t code_bits;           /* storage of `codes`: 0 or 4 = one code per nibble, as described above;
                                  2 or 3 = dense N-bit storage (min-max format only, d_in % 32 == 0, every code < 2^N;
                                  Eq. 1 is stated for N bits), written by qblora_pack_codes:
                                    2: DEVICE [d_out][d_in/4],   byte k of row o: code(o,4k+j) in bits 2j..2j+1;
                                    3: DEVICE [d_out][3*d_in/8], codes 8k..8k+7 of row o as the 24-bit number
                                       sum_j code(o,8k+j) << 3j, little-endian in bytes 3k..3k+2.
                                  Calls that read the codes expand such a weight to one code per nibble inside `ws` first
                                  (qblora_workspace_bytes includes the d_out*d_in/2 bytes): the saving is in the memory the
                                  weight occupies at rest, not in the bytes a product streams. */
} qblora_qweight;

/* The parameter-free operator pair that compresses the adapter's input and restores its output
 * size.  The method's own pair is AvgPool & repeat_interleave (Sec. 3.2); the other two are the
 * alternatives of the Sec. 4 ablation on scale operators (the paper finds them clearly worse; they
 * exist here to reproduce that comparison).  With P = d_in / lambda_in, Q = d_out / lambda_out:
 *   AVGPOOL_REPEAT    x'[p] = mean(x[lambda_in p .. lambda_in p + lambda_in - 1]);  y[o] += s y'[o / lambda_out]
 *   TRUNCATE_ZEROPAD  x'[p] = x[p]            (front part kept);   y[o] += s y'[o] for o < Q, nothing beyond
 *   SAMPLE_ZEROFILL   x'[p] = x[lambda_in p]  (regular interval);  y[lambda_out q] += s y'[q], nothing between
 * Only AVGPOOL_REPEAT gives an update that is constant over a quantization block, so qablora_merge
 * and qablora_merge_noalloc return QBLORA_ERR_INVALID_ARG for the other two; qblora_merge_dense takes all. */
typedef enum {
  QBLORA_SCALE_AVGPOOL_REPEAT = 0,
  QBLORA_SCALE_TRUNCATE_ZEROPAD = 1,
  QBLORA_SCALE_SAMPLE_ZEROFILL = 2
} qblora_scale_op;

/* Balanced low-rank adapter (Sec. 3.2): x' = AvgPool_{lambda_in}(x), y' = (A B)^T x',
 * y_adapter = scaling * repeat_interleave_{lambda_out}(y'). */
typedef struct {
  int32_t lambda_in, lambda_out; /* lambda_1 (input pooling), lambda_2 (output repeat) */
  int32_t rank;                  /* r */
  float scaling;                 /* s; multiplies the adapter term only */
  const void* A;                 /* DEVICE bf16 [P][r] */
  const void* B;                 /* DEVICE bf16 [r][Q]; NULL => A is the single matrix H, bf16 [P][Q],
                                    of Sec. 3.3 / Algorithm 2 (rank is then ignored) */
  int32_t scale_op;              /* qblora_scale_op; 0 = the method's AvgPool & repeat_interleave */
} qblora_adapter;

/* Writes the built-in 16-level table (HOST out): nine non-negative levels
 * ppf(1/2 + j/17) / ppf(1/2 + 8/17), j = 0..8, and seven negative levels
 * -ppf(1/2 + j/15) / ppf(1/2 + 7/15), j = 1..7 (ppf = standard normal quantile), ascending,
 * rounded to fp32.  The paper (Sec. 3.2) names a 4-bit normal-quantile type without printing its
 * values; callers that hold another table pass it in qblora_qweight.code instead. */
int qblora_default_code_table(float out[16]);

/* Scratch bytes needed by `op` for this weight / adapter / token count (0 if none).
 * adapter may be NULL.  Returns 0 for invalid arguments as well; the op itself reports those. */
size_t qblora_workspace_bytes(int op, const qblora_qweight* qw, const qblora_adapter* adapter,
                              int64_t tokens);

const char* qblora_status_string(int status);

/* Synchronises `stream` and returns the status word the last call using `ws` left there
 * (QBLORA_OK, or QBLORA_ERR_TIMEOUT if a kernel's bounded wait expired). */
int qblora_device_status(const void* ws, void* stream);

/* Instrumentation for benchmarks (host-side state, per calling thread; no effect on results).
 * qblora_kernel_launches(): number of kernels this library has launched so far in this process.
 * qblora_set_timing_events(start, stop): arms a pair of cudaEvent_t; the next call of
 * qblora_linear_fwd / qblora_linear_bwd / qablora_lowbit_gemm on this thread records `start`
 * immediately before and `stop` immediately after its dominant kernel (the base-weight contraction)
 * on the call's stream, then disarms.  Pass NULL, NULL to disarm.  The paper has no counterpart. */
uint64_t qblora_kernel_launches(void);
int qblora_set_timing_events(void* start_event, void* stop_event);

/* Test hooks for the bounded device-side waits (process-wide host state; the paper has no counterpart).
 * qblora_debug_set_wait_limit(cycles): kernels launched from now on give up a wait after `cycles` SM clock
 *   cycles instead of the default 2 * 10^9 (0 restores the default).
 * qblora_debug_drop_load(iteration): in the NEXT launch of the fused dequant contraction (qblora_linear_fwd /
 *   qblora_linear_bwd / the large-token qablora_lowbit_gemm) the producer of every CTA announces the bytes of
 *   its `iteration`-th weight K-block to the stage's barrier but issues no copy, so that barrier never
 *   completes: every role of the kernel runs into its wait limit, the kernel stores QBLORA_ERR_TIMEOUT in the
 *   status word, releases its tensor memory and returns by itself; the outputs of that call are undefined.
 *   Negative = disarm.  Use together with a short wait limit.
 * qblora_debug_hold_producer(cycles): in the NEXT launch of the fused dequant contraction with an adapter, the
 *   producer of every CTA idles for `cycles` SM clock cycles (at most 10^8, about 50 ms) in front of the first
 *   adapter K-block of its first tile -- what a long wait for the adapter's compressed activation looks like to
 *   the other roles of the kernel.  The results must not change.  0 = disarm. */
int qblora_debug_set_wait_limit(int64_t cycles);
int qblora_debug_drop_load(int32_t iteration);
int qblora_debug_hold_producer(int64_t cycles);

/*
 * Block-wise 4-bit quantization, Eq. 1 (Sec. 3.1).
 *   W       DEVICE [d_out][d_in], fp32 or bf16 (w_dtype); bf16 is promoted exactly.
 *   code    HOST level table (code-table format; ignored for min-max).
 *   codes   DEVICE out, uint8 [d_out][d_in/2];  alpha DEVICE out fp32 [d_out/block_out][d_in/block_in];
 *   beta    DEVICE out, same shape (min-max format); must be NULL for the code-table format.
 * Arithmetic is IEEE fp32, one rounding per operation, so the result is unique:
 *   code table: alpha = max|w|; v = w / alpha; code = #{ j : v > fl32((code[j]+code[j+1])/2) }
 *               (nearest level, ties to the lower index); all-zero block: alpha = 0, code = level 0.0.
 *   min-max:    beta = min; alpha = (max - min) / 15; code = clamp(rint((w - beta) / alpha), 0, 15),
 *               ties to even; constant block: alpha = 0, code = 0.
 * Requires d_in % block_in == 0, d_out % block_out == 0, d_in even.
 */
int qblora_quantize_blockwise(const void* W, int w_dtype, int32_t d_out, int32_t d_in,
                              int32_t block_in, int32_t block_out, int32_t qfmt,
                              const float code[16], uint8_t* codes, float* alpha, float* beta,
                              void* stream);

/*
 * Min-max quantization on an N-bit grid, N = bits in 1..4 (Eq. 1 is stated for N bits; Sec. 3.1):
 *   beta = min; alpha = (max - min) / (2^N - 1); code = clamp(rint((w - beta) / alpha), 0, 2^N - 1), ties to even;
 *   constant block: alpha = 0, code = 0.  Same single-rounding fp32 arithmetic as above; bits = 4 gives exactly
 *   qblora_quantize_blockwise's min-max result.
 * The codes come out one per nibble, codes uint8 [d_out][d_in/2], so the result is an ordinary
 * QBLORA_FMT_AFFINE_MINMAX weight for every other call of this library (forward, backward, both merges, low-bit
 * product); qblora_pack_codes turns 2- and 3-bit codes into dense storage (code_bits of qblora_qweight).
 * Arguments and requirements as for qblora_quantize_blockwise; beta must not be NULL.
 */
int qblora_quantize_minmax_nbit(const void* W, int w_dtype, int32_t d_out, int32_t d_in,
                                int32_t block_in, int32_t block_out, int32_t bits,
                                uint8_t* codes, float* alpha, float* beta, void* stream);

/*
 * Dense storage for N-bit weights, N = bits in {2, 3} (Eq. 1 is stated for N bits; the paper fixes no byte layout --
 * the layout is the one given at qblora_qweight.code_bits).
 *   qblora_pack_codes:   codes DEVICE uint8 [d_out][d_in/2] (one per nibble, e.g. from qblora_quantize_minmax_nbit)
 *                        -> packed DEVICE uint8 [d_out][d_in*bits/8].  ws: at least 256 bytes; qblora_device_status(ws)
 *                        returns QBLORA_ERR_INVALID_ARG afterwards if some code did not fit in `bits` bits.
 *   qblora_unpack_codes: the inverse.
 * Requires d_in % 32 == 0; both buffers 16-byte aligned.
 */
int qblora_pack_codes(const uint8_t* codes, int32_t d_out, int32_t d_in, int32_t bits, uint8_t* packed, void* ws,
                      size_t ws_bytes, void* stream);
int qblora_unpack_codes(const uint8_t* packed, int32_t d_out, int32_t d_in, int32_t bits, uint8_t* codes, void* stream);

/*
 * Forward of the adapted quantized linear (Sec. 3.1 combined formula with the Sec. 3.2 adapter;
 * Algorithm 1's forward read as its prose):
 *   Y[t][o] = sum_i X[t][i] * w~[o][i]  +  s * ((x' A) B)[t][o / lambda_out],
 *   x'[t][p] = (1 / lambda_in) * sum_{j < lambda_in} X[t][lambda_in * p + j].
 * The base weight is dequantized inside the kernel; no dense copy of it is written.
 *   X DEVICE bf16 [tokens][d_in];  Y DEVICE out [tokens][d_out], y_dtype BF16 or F32 (F32 = the
 *   accumulator before the final rounding).  adapter may be NULL (base term only).
 */
int qblora_linear_fwd(const qblora_qweight* qw, const qblora_adapter* adapter, const void* X,
                      int64_t tokens, void* Y, int y_dtype, void* ws, size_t ws_bytes,
                      void* stream);

/*
 * Backward of the same layer with the base weight frozen (Sec. 3.1: only A and B are trained);
 * the paper leaves it to automatic differentiation, so it is the derivative of the forward above:
 *   dv[t][q] = s * sum_{j < lambda_out} dY[t][lambda_out * q + j];   du = dv B^T;
 *   dB = u^T dv  (u = x' A, recomputed from X);   dA = x'^T du;
 *   dX[t][i] = sum_o dY[t][o] * w~[o][i]  +  (du A^T)[t][i / lambda_in] / lambda_in.
 *   dY DEVICE bf16 [tokens][d_out];  dX DEVICE out [tokens][d_in] (dx_dtype BF16 or F32);
 *   dA DEVICE out fp32 [P][r];  dB DEVICE out fp32 [r][Q].  Any of dX, dA, dB may be NULL (skipped).
 *   adapter may be NULL (then dA and dB must be NULL).
 *   Stream: part of the work (the dA / dB chain) is enqueued on a stream the library creates on first
 *   use (per host thread and device); it is ordered after `stream` at entry and joined back into
 *   `stream` before the call returns, so the caller sees ordinary stream semantics (also inside a
 *   stream capture).  Environment QBLORA_NO_OVERLAP=1 keeps everything on `stream`.
 *   Single-matrix adapter (adapter->B == NULL, Sec. 3.3): the adapter term of the forward is
 *   s * (x' H)[t][o / lambda_out]; dA receives dH = x'^T dv as fp32 [P][Q], dB must be NULL, and the
 *   pooled-input gradient is dv H^T.
 */
int qblora_linear_bwd(const qblora_qweight* qw, const qblora_adapter* adapter, const void* X,
                      const void* dY, int64_t tokens, void* dX, int dx_dtype, float* dA, float* dB,
                      void* ws, size_t ws_bytes, void* stream);

/*
 * QA-BLoRA merge (Sec. 3.3; Algorithm 2's new-beta routine): the adapter's equivalent dense
 * update is constant on (lambda_in x lambda_out) tiles (paragraph after Eq. 2), so when every
 * quantization block lies inside one tile it is a shift of that block's beta:
 *   beta'[o/block_out][i/block_in] = beta + s * (A B)[i0 / lambda_in][o0 / lambda_out] / lambda_in.
 * qw must be in the min-max format; codes and alpha are not touched.  beta_out DEVICE fp32, same
 * shape as beta, may alias qw->beta.  Evaluated in fp64 and rounded once to fp32.
 * Requires lambda_in % block_in == 0 and lambda_out % block_out == 0, else QBLORA_ERR_INVALID_ARG.
 * adapter->B == NULL: A is H [P][Q].
 */
int qablora_merge(const qblora_qweight* qw, const qblora_adapter* adapter, float* beta_out,
                  void* ws, size_t ws_bytes, void* stream);

/*
 * Dense 16-bit merge (Sec. 3.1 / 3.2: after fine-tuning the adapter is folded back into a full weight
 * with no inference overhead; Algorithm 1's dense-update routine read as
 * dW[o][i] = (A B)[i / lambda_in][o / lambda_out] / lambda_in):
 *   W_out[o][i] = alpha * level[code] + beta  +  s * dW[o][i]   (A B in fp64, the sum in fp32, then bf16).
 *   W_out DEVICE out bf16 [d_out][d_in] (16-byte aligned, d_in % 8 == 0).  Either format, any block
 *   shape, any (lambda_in, lambda_out).  adapter may be NULL (plain dequantization) and may be the
 *   single matrix H (B == NULL).  The merged weight is then served by qblora_dense_gemm (or any plain bf16 GEMM).
 *   ws: qblora_workspace_bytes(QBLORA_OP_MERGE_DENSE, ...) bytes.
 */
int qblora_merge_dense(const qblora_qweight* qw, const qblora_adapter* adapter, void* W_out, void* ws,
                       size_t ws_bytes, void* stream);

/*
 * Serving product for the 16-bit deployment (Sec. 3.1: the fine-tuned adapter is merged into the weight, W' = W + s A B,
 * "for inference"; Sec. 3.2, "Merging Q-BLoRA": the merged model has no inference overhead):
 *   Y[t][o] = sum_i X[t][i] * W[o][i],  W DEVICE bf16 [d_out][d_in] as written by qblora_merge_dense.
 * A plain bf16 tensor-core GEMM with fp32 accumulation.  X DEVICE bf16 [tokens][d_in]; Y DEVICE out [tokens][d_out],
 * BF16 or F32.  Requires d_in % 8 == 0.  ws: at least 256 bytes (status word only).
 */
int qblora_dense_gemm(const void* W, int32_t d_out, int32_t d_in, const void* X, int64_t tokens, void* Y,
                      int y_dtype, void* ws, size_t ws_bytes, void* stream);

/*
 * The same merge for callers that cannot give the library a workspace.  (The paper has no
 * counterpart; this is a packaging variant of qablora_merge.)
 *
 * Who needs it: code that must not touch the device allocator while it runs -- a serving loop that
 * swaps adapters after start-up with all device memory already committed to weights and caches, a
 * host without a spare allocator context, a plug-in called from inside someone else's stream-ordered
 * pipeline where a cudaMalloc would stall every stream.  qablora_merge needs P * Q fp64 values of
 * scratch for H = A B; here they live in a 2 MiB array that is part of the library image (every GPU
 * that loads the library carries it until the process exits), so the call allocates and frees
 * nothing: no workspace argument, no cudaMalloc / cudaFree, no allocating library routine.
 *
 * Limits and rules:
 *   - P * Q = (d_in / lambda_in) * (d_out / lambda_out) must be <= 262144, else QBLORA_ERR_TOO_LARGE
 *     (the LLaMA-33B shapes of the deploy configuration use 86528 to 232960).
 *   - Inputs, outputs, results and the other error codes are exactly those of qablora_merge.
 *   - The first call on each device looks up the array's device address (with that device current);
 *     make that first call outside any stream capture.
 *   - All calls on a device share the one array, and it keeps the previous call's H.  Each call
 *     overwrites every entry it reads, so nothing carries over between calls; but two calls that
 *     can run concurrently on the same GPU (different streams, different host threads) race on
 *     it -- serialise them.
 */
int qablora_merge_noalloc(const qblora_qweight* qw, const qblora_adapter* adapter, float* beta_out,
                          void* stream);

/*
 * Low-precision inference product on the merged model (Sec. 3.3):
 *   Y[t][o] = sum_i X[t][i] * (alpha[o][i/g] * c[o][i] + beta'[o][i/g]).
 * qw: min-max format.  X DEVICE bf16 [tokens][d_in];  Y DEVICE out [tokens][d_out], BF16 or F32.
 * Small token counts stream the packed weight once (bandwidth-bound); large ones use the same
 * tensor-core mainloop as qblora_linear_fwd.
 */
int qablora_lowbit_gemm(const qblora_qweight* qw, const void* X, int64_t tokens, void* Y,
                        int y_dtype, void* ws, size_t ws_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* QBLORA_H_ */
