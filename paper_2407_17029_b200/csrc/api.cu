// extern "C" entry points declared in include/qblora.h: host-side argument checks, workspace
// accounting and dispatch to the kernels.  No device memory is allocated here.
#include <cmath>
#include <cstdlib>
#include <cstring>

#include "common.cuh"

namespace qb {
namespace {

// Standard normal quantile by safeguarded Newton iteration on 0.5 * (1 + erf(x / sqrt 2)).
double normal_quantile(double p) {
  const double inv_sqrt2 = 0.70710678118654752440, inv_sqrt_2pi = 0.39894228040143267794;
  double lo = -12.0, hi = 12.0, x = 0.0;
  for (int it = 0; it < 200; ++it) {
    const double f = 0.5 * (1.0 + std::erf(x * inv_sqrt2)) - p;
    if (f > 0) hi = x; else lo = x;
    const double d = inv_sqrt_2pi * std::exp(-0.5 * x * x);
    double xn = x - f / d;
    if (!(xn > lo && xn < hi)) xn = 0.5 * (lo + hi);
    if (std::fabs(xn - x) <= 1e-17 * std::fabs(x)) { x = xn; break; }
    x = xn;
  }
  return x;
}

bool force_general() {
  const char* e = std::getenv("QBLORA_FORCE_GENERAL");
  return e && e[0] == '1';
}

// code_bits: 0 or 4 = one code per nibble; 2 or 3 = dense storage (min-max format, d_in a multiple of 32)
bool code_bits_ok(const qblora_qweight* q) {
  if (q->code_bits == 0 || q->code_bits == 4) return true;
  return (q->code_bits == 2 || q->code_bits == 3) && q->qfmt == QBLORA_FMT_AFFINE_MINMAX && q->d_in % 32 == 0;
}

int make_qw(const qblora_qweight* q, QwView* v) {
  if (!q) return QBLORA_ERR_INVALID_ARG;
  if (q->d_in <= 0 || q->d_out <= 0 || q->block_in <= 0 || q->block_out <= 0) return QBLORA_ERR_INVALID_ARG;
  if (q->d_in % 2 || q->d_in % q->block_in || q->d_out % q->block_out) return QBLORA_ERR_INVALID_ARG;
  if (q->qfmt != QBLORA_FMT_CODEBOOK_ABSMAX && q->qfmt != QBLORA_FMT_AFFINE_MINMAX) return QBLORA_ERR_INVALID_ARG;
  if (!q->codes || !q->alpha || !aligned16(q->codes) || !aligned16(q->alpha)) return QBLORA_ERR_INVALID_ARG;
  if (q->qfmt == QBLORA_FMT_AFFINE_MINMAX && (!q->beta || !aligned16(q->beta))) return QBLORA_ERR_INVALID_ARG;
  if (!code_bits_ok(q)) return QBLORA_ERR_INVALID_ARG;
  v->code_bits = q->code_bits == 0 ? 4 : q->code_bits;
  v->d_in = q->d_in; v->d_out = q->d_out; v->block_in = q->block_in; v->block_out = q->block_out;
  v->qfmt = q->qfmt; v->G = q->d_in / q->block_in;
  v->codes = q->codes; v->alpha = q->alpha;
  v->beta = (q->qfmt == QBLORA_FMT_AFFINE_MINMAX) ? q->beta : nullptr;
  for (int j = 0; j < 16; ++j) v->level[j] = (q->qfmt == QBLORA_FMT_CODEBOOK_ABSMAX) ? q->code[j] : (float)j;
  return QBLORA_OK;
}

// geometry-only view for workspace queries (pointers are not needed there)
bool make_qw_geom(const qblora_qweight* q, QwView* v) {
  if (!q || q->d_in <= 0 || q->d_out <= 0 || q->block_in <= 0 || q->block_out <= 0) return false;
  if (q->d_in % 2 || q->d_in % q->block_in || q->d_out % q->block_out) return false;
  if (!code_bits_ok(q)) return false;
  std::memset(v, 0, sizeof(*v));
  v->d_in = q->d_in; v->d_out = q->d_out; v->block_in = q->block_in; v->block_out = q->block_out;
  v->qfmt = q->qfmt; v->G = q->d_in / q->block_in;
  v->code_bits = q->code_bits == 0 ? 4 : q->code_bits;
  return true;
}

int make_ad(const qblora_adapter* a, const QwView& q, bool need_ptrs, AdView* v) {
  if (a->lambda_in < 1 || a->lambda_out < 1) return QBLORA_ERR_INVALID_ARG;
  if (q.d_in % a->lambda_in || q.d_out % a->lambda_out) return QBLORA_ERR_INVALID_ARG;
  if (a->B && a->rank < 1) return QBLORA_ERR_INVALID_ARG;
  if (a->scale_op < QBLORA_SCALE_AVGPOOL_REPEAT || a->scale_op > QBLORA_SCALE_SAMPLE_ZEROFILL) return QBLORA_ERR_INVALID_ARG;
  if (need_ptrs) {
    if (!a->A || !aligned16(a->A)) return QBLORA_ERR_INVALID_ARG;
    if (a->B && !aligned16(a->B)) return QBLORA_ERR_INVALID_ARG;
  }
  v->l1 = a->lambda_in; v->l2 = a->lambda_out; v->r = a->rank; v->s = a->scaling; v->op = a->scale_op;
  v->P = q.d_in / a->lambda_in; v->Q = q.d_out / a->lambda_out;
  v->A = static_cast<const __nv_bfloat16*>(a->A);
  v->B = static_cast<const __nv_bfloat16*>(a->B);
  return QBLORA_OK;
}

bool dtype_ok(int d) { return d == QBLORA_F32 || d == QBLORA_BF16; }

int reset_status(void* ws, cudaStream_t st) {
  QB_CUDA(cudaMemsetAsync(ws, 0, 16, st));
  return QBLORA_OK;
}

// Single-matrix adapters (B == NULL, A is H [P][Q]; Sec. 3.3 / Algorithm 2) train through the same
// kernels as the two-factor form with A := I_P, B := H, r := P: then u = x' I = x' exactly, the adapter
// output is s * repeat(x' H), dB of the factored form is dH = x'^T dv, and du I^T = dv H^T is the
// pooled-input gradient.  The identity lives at the end of the workspace and is written per call.
size_t single_identity_bytes(const AdView& ad) { return align_up((size_t)ad.P * ad.P * 2, 256); }
AdView single_as_factored(const AdView& ad, const __nv_bfloat16* identity) {
  AdView f = ad;
  f.r = ad.P;
  f.B = ad.A;          // H
  f.A = identity;
  return f;
}

// Densely stored codes (code_bits 2 or 3) are expanded to one code per nibble behind the op's own scratch.
size_t expand_bytes(const QwView& q) { return q.code_bits < 4 ? align_up((size_t)q.d_out * q.d_in / 2, 256) : 0; }
size_t with_expansion(size_t need, const QwView& q) { return q.code_bits < 4 ? align_up(need, 256) + expand_bytes(q) : need; }
// Expands into ws + align_up(need, 256) and points the view at the expanded codes.
int expand_codes(QwView* q, size_t need, void* ws, cudaStream_t st) {
  if (q->code_bits >= 4) return QBLORA_OK;
  uint8_t* dst = static_cast<uint8_t*>(ws) + align_up(need, 256);
  const int rc = launch_unpack_codes(q->codes, q->d_out, q->d_in, q->code_bits, dst, st);
  if (rc) return rc;
  q->codes = dst;
  q->code_bits = 4;
  return QBLORA_OK;
}

size_t ws_bytes_impl(int op, const QwView& q, const AdView* ad, int64_t T);
size_t ws_bytes_single(int op, const QwView& q, const AdView& ad, int64_t T) {
  const AdView f = single_as_factored(ad, nullptr);
  return align_up(ws_bytes_impl(op, q, &f, T), 256) + single_identity_bytes(ad);
}

size_t ws_bytes_impl(int op, const QwView& q, const AdView* ad, int64_t T) {
  switch (op) {
    case QBLORA_OP_QUANTIZE: return 0;
    case QBLORA_OP_LINEAR_FWD:
    case QBLORA_OP_LINEAR_BWD:
      if (!force_general() && tc_supported(q, ad, T)) return tc_ws_bytes(op, q, ad, T);
      return simt_ws_bytes(op, q, ad, T);
    case QBLORA_OP_MERGE: return ad ? merge_ws_bytes(q, *ad) : 0;
    case QBLORA_OP_MERGE_DENSE: return merge_dense_ws_bytes(q, ad);
    case QBLORA_OP_LOWBIT_GEMM:
      if (gemv_supported(q, T)) return gemv_ws_bytes(q, T);
      if (!force_general() && tc_supported(q, nullptr, T)) return tc_lowbit_ws_bytes(q, T);
      return simt_ws_bytes(QBLORA_OP_LINEAR_FWD, q, nullptr, T);
    default: return 0;
  }
}

}  // namespace
}  // namespace qb

using namespace qb;

extern "C" {

int qblora_default_code_table(float out[16]) {
  if (!out) return QBLORA_ERR_INVALID_ARG;
  const double pos_den = normal_quantile(0.5 + 8.0 / 17.0), neg_den = normal_quantile(0.5 + 7.0 / 15.0);
  for (int j = 1; j <= 7; ++j) out[7 - j] = (float)(-normal_quantile(0.5 + j / 15.0) / neg_den);
  for (int j = 1; j <= 8; ++j) out[7 + j] = (float)(normal_quantile(0.5 + j / 17.0) / pos_den);
  out[0] = -1.0f; out[7] = 0.0f; out[15] = 1.0f;
  return QBLORA_OK;
}

const char* qblora_status_string(int s) {
  switch (s) {
    case QBLORA_OK: return "ok";
    case QBLORA_ERR_INVALID_ARG: return "invalid argument";
    case QBLORA_ERR_UNSUPPORTED: return "unsupported configuration";
    case QBLORA_ERR_WORKSPACE: return "workspace missing or too small";
    case QBLORA_ERR_CUDA: return "CUDA error";
    case QBLORA_ERR_TIMEOUT: return "device-side wait timed out";
    case QBLORA_ERR_TOO_LARGE: return "problem exceeds the built-in scratch of the no-allocation entry point";
    default: return "unknown status";
  }
}

size_t qblora_workspace_bytes(int op, const qblora_qweight* qw, const qblora_adapter* adapter, int64_t tokens) {
  QwView q;
  if (!make_qw_geom(qw, &q)) return 0;
  AdView ad; const AdView* adp = nullptr;
  if (adapter) {
    if (make_ad(adapter, q, false, &ad) != QBLORA_OK) return 0;
    adp = &ad;
  }
  if (op != QBLORA_OP_MERGE && op != QBLORA_OP_MERGE_DENSE && op != QBLORA_OP_QUANTIZE && tokens < 1) return 0;
  const bool reads_codes = op == QBLORA_OP_LINEAR_FWD || op == QBLORA_OP_LINEAR_BWD || op == QBLORA_OP_MERGE_DENSE ||
                           op == QBLORA_OP_LOWBIT_GEMM;
  size_t need;
  if (adp && !adapter->B && (op == QBLORA_OP_LINEAR_FWD || op == QBLORA_OP_LINEAR_BWD)) need = ws_bytes_single(op, q, ad, tokens);
  else need = ws_bytes_impl(op, q, adp, tokens);
  return reads_codes ? with_expansion(need, q) : need;
}

int qblora_device_status(const void* ws, void* stream) {
  if (!ws) return QBLORA_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  QB_CUDA(cudaStreamSynchronize(st));
  int word = 0;
  QB_CUDA(cudaMemcpy(&word, ws, sizeof(int), cudaMemcpyDeviceToHost));
  return word;
}

int qblora_quantize_blockwise(const void* W, int w_dtype, int32_t d_out, int32_t d_in, int32_t block_in,
                              int32_t block_out, int32_t qfmt, const float code[16], uint8_t* codes,
                              float* alpha, float* beta, void* stream) {
  if (!W || !codes || !alpha || !dtype_ok(w_dtype)) return QBLORA_ERR_INVALID_ARG;
  if (d_in <= 0 || d_out <= 0 || block_in <= 0 || block_out <= 0) return QBLORA_ERR_INVALID_ARG;
  if (d_in % 2 || d_in % block_in || d_out % block_out) return QBLORA_ERR_INVALID_ARG;
  if (!aligned16(W) || !aligned16(codes) || !aligned16(alpha)) return QBLORA_ERR_INVALID_ARG;
  if (qfmt == QBLORA_FMT_CODEBOOK_ABSMAX) {
    if (!code || beta) return QBLORA_ERR_INVALID_ARG;
    for (int j = 0; j < 15; ++j) if (!(code[j] < code[j + 1])) return QBLORA_ERR_INVALID_ARG;
  } else if (qfmt == QBLORA_FMT_AFFINE_MINMAX) {
    if (!beta || !aligned16(beta)) return QBLORA_ERR_INVALID_ARG;
  } else {
    return QBLORA_ERR_INVALID_ARG;
  }
  return launch_quantize(W, w_dtype, d_out, d_in, block_in, block_out, qfmt, 4, code, codes, alpha, beta,
                         static_cast<cudaStream_t>(stream));
}

int qblora_quantize_minmax_nbit(const void* W, int w_dtype, int32_t d_out, int32_t d_in, int32_t block_in,
                                int32_t block_out, int32_t bits, uint8_t* codes, float* alpha, float* beta,
                                void* stream) {
  if (bits < 1 || bits > 4) return QBLORA_ERR_INVALID_ARG;
  if (!W || !codes || !alpha || !beta || !dtype_ok(w_dtype)) return QBLORA_ERR_INVALID_ARG;
  if (d_in <= 0 || d_out <= 0 || block_in <= 0 || block_out <= 0) return QBLORA_ERR_INVALID_ARG;
  if (d_in % 2 || d_in % block_in || d_out % block_out) return QBLORA_ERR_INVALID_ARG;
  if (!aligned16(W) || !aligned16(codes) || !aligned16(alpha) || !aligned16(beta)) return QBLORA_ERR_INVALID_ARG;
  return launch_quantize(W, w_dtype, d_out, d_in, block_in, block_out, QBLORA_FMT_AFFINE_MINMAX, bits, nullptr, codes,
                         alpha, beta, static_cast<cudaStream_t>(stream));
}

int qblora_linear_fwd(const qblora_qweight* qw, const qblora_adapter* adapter, const void* X, int64_t tokens,
                      void* Y, int y_dtype, void* ws, size_t ws_bytes, void* stream) {
  QwView q; int rc = make_qw(qw, &q);
  if (rc) return rc;
  if (!X || !Y || !aligned16(X) || !aligned16(Y) || tokens < 1 || !dtype_ok(y_dtype)) return QBLORA_ERR_INVALID_ARG;
  AdView ad; const AdView* adp = nullptr;
  if (adapter) {
    rc = make_ad(adapter, q, true, &ad);
    if (rc) return rc;
    adp = &ad;
  }
  const bool single = adapter && !adapter->B;
  const size_t need = single ? ws_bytes_single(QBLORA_OP_LINEAR_FWD, q, ad, tokens)
                             : ws_bytes_impl(QBLORA_OP_LINEAR_FWD, q, adp, tokens);
  if (!ws || !aligned16(ws) || ws_bytes < with_expansion(need, q)) return QBLORA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  rc = reset_status(ws, st);
  if (rc) return rc;
  rc = expand_codes(&q, need, ws, st);
  if (rc) return rc;
  if (single) {
    __nv_bfloat16* eye = reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(ws) + need - single_identity_bytes(ad));
    rc = launch_identity(eye, ad.P, st);
    if (rc) return rc;
    ad = single_as_factored(ad, eye);
  }
  const __nv_bfloat16* Xb = static_cast<const __nv_bfloat16*>(X);
  if (!force_general() && tc_supported(q, adp, tokens))
    return tc_linear_fwd(q, adp, Xb, tokens, Y, y_dtype, static_cast<char*>(ws), st);
  return simt_linear_fwd(q, adp, Xb, tokens, Y, y_dtype, static_cast<char*>(ws), st);
}

int qblora_linear_bwd(const qblora_qweight* qw, const qblora_adapter* adapter, const void* X, const void* dY,
                      int64_t tokens, void* dX, int dx_dtype, float* dA, float* dB, void* ws, size_t ws_bytes,
                      void* stream) {
  QwView q; int rc = make_qw(qw, &q);
  if (rc) return rc;
  if (!dY || !aligned16(dY) || tokens < 1 || !dtype_ok(dx_dtype)) return QBLORA_ERR_INVALID_ARG;
  if (dX && !aligned16(dX)) return QBLORA_ERR_INVALID_ARG;
  if ((dA && !aligned16(dA)) || (dB && !aligned16(dB))) return QBLORA_ERR_INVALID_ARG;
  AdView ad; const AdView* adp = nullptr;
  if (adapter) {
    rc = make_ad(adapter, q, true, &ad);
    if (rc) return rc;
    if (!adapter->B && dB) return QBLORA_ERR_INVALID_ARG;   // single matrix: its gradient dH goes to dA
    if (!X || !aligned16(X)) return QBLORA_ERR_INVALID_ARG;
    adp = &ad;
  } else if (dA || dB) {
    return QBLORA_ERR_INVALID_ARG;
  }
  if (!dX && !dA && !dB) return QBLORA_OK;
  const bool single = adapter && !adapter->B;
  const size_t need = single ? ws_bytes_single(QBLORA_OP_LINEAR_BWD, q, ad, tokens)
                             : ws_bytes_impl(QBLORA_OP_LINEAR_BWD, q, adp, tokens);
  if (!ws || !aligned16(ws) || ws_bytes < with_expansion(need, q)) return QBLORA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  rc = reset_status(ws, st);
  if (rc) return rc;
  if (dX) {   // only the dX contraction reads the codes
    rc = expand_codes(&q, need, ws, st);
    if (rc) return rc;
  }
  if (single) {
    __nv_bfloat16* eye = reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(ws) + need - single_identity_bytes(ad));
    rc = launch_identity(eye, ad.P, st);
    if (rc) return rc;
    ad = single_as_factored(ad, eye);
    dB = dA;          // dH = x'^T dv is the factored form's dB
    dA = nullptr;     // the identity is not trained
  }
  const __nv_bfloat16* Xb = static_cast<const __nv_bfloat16*>(X);
  const __nv_bfloat16* dYb = static_cast<const __nv_bfloat16*>(dY);
  if (!force_general() && tc_supported(q, adp, tokens))
    return tc_linear_bwd(q, adp, Xb, dYb, tokens, dX, dx_dtype, dA, dB, static_cast<char*>(ws), st);
  return simt_linear_bwd(q, adp, Xb, dYb, tokens, dX, dx_dtype, dA, dB, static_cast<char*>(ws), st);
}

int qablora_merge(const qblora_qweight* qw, const qblora_adapter* adapter, float* beta_out, void* ws,
                  size_t ws_bytes, void* stream) {
  QwView q; int rc = make_qw(qw, &q);
  if (rc) return rc;
  if (q.qfmt != QBLORA_FMT_AFFINE_MINMAX || !adapter || !beta_out || !aligned16(beta_out)) return QBLORA_ERR_INVALID_ARG;
  AdView ad; rc = make_ad(adapter, q, true, &ad);
  if (rc) return rc;
  // every quantization block must lie inside one (lambda_in x lambda_out) tile of the dense update, and
  // the update must be constant on that tile (only AvgPool & repeat_interleave gives that)
  if (ad.l1 % q.block_in || ad.l2 % q.block_out || ad.op != QBLORA_SCALE_AVGPOOL_REPEAT) return QBLORA_ERR_INVALID_ARG;
  const size_t need = merge_ws_bytes(q, ad);
  if (!ws || !aligned16(ws) || ws_bytes < need) return QBLORA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  rc = reset_status(ws, st);
  if (rc) return rc;
  return launch_merge(q, ad, adapter->B == nullptr, beta_out, static_cast<char*>(ws), st);
}

int qblora_merge_dense(const qblora_qweight* qw, const qblora_adapter* adapter, void* W_out, void* ws,
                       size_t ws_bytes, void* stream) {
  QwView q; int rc = make_qw(qw, &q);
  if (rc) return rc;
  if (!W_out || !aligned16(W_out) || q.d_in % 8) return QBLORA_ERR_INVALID_ARG;
  AdView ad; const AdView* adp = nullptr;
  if (adapter) {
    rc = make_ad(adapter, q, true, &ad);
    if (rc) return rc;
    adp = &ad;
  }
  const size_t need = merge_dense_ws_bytes(q, adp);
  if (!ws || !aligned16(ws) || ws_bytes < with_expansion(need, q)) return QBLORA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  rc = reset_status(ws, st);
  if (rc) return rc;
  rc = expand_codes(&q, need, ws, st);
  if (rc) return rc;
  return launch_merge_dense(q, adp, adapter && adapter->B == nullptr, static_cast<__nv_bfloat16*>(W_out),
                            static_cast<char*>(ws), st);
}

int qblora_pack_codes(const uint8_t* codes, int32_t d_out, int32_t d_in, int32_t bits, uint8_t* packed, void* ws,
                      size_t ws_bytes, void* stream) {
  if (!codes || !packed || !aligned16(codes) || !aligned16(packed)) return QBLORA_ERR_INVALID_ARG;
  if ((bits != 2 && bits != 3) || d_out < 1 || d_in < 32 || d_in % 32) return QBLORA_ERR_INVALID_ARG;
  if (!ws || !aligned16(ws) || ws_bytes < kStatusBytes) return QBLORA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int rc = reset_status(ws, st);
  if (rc) return rc;
  return launch_pack_codes(codes, d_out, d_in, bits, packed, static_cast<int*>(ws), st);
}

int qblora_unpack_codes(const uint8_t* packed, int32_t d_out, int32_t d_in, int32_t bits, uint8_t* codes, void* stream) {
  if (!codes || !packed || !aligned16(codes) || !aligned16(packed)) return QBLORA_ERR_INVALID_ARG;
  if ((bits != 2 && bits != 3) || d_out < 1 || d_in < 32 || d_in % 32) return QBLORA_ERR_INVALID_ARG;
  return launch_unpack_codes(packed, d_out, d_in, bits, codes, static_cast<cudaStream_t>(stream));
}

int qblora_dense_gemm(const void* W, int32_t d_out, int32_t d_in, const void* X, int64_t tokens, void* Y, int y_dtype,
                      void* ws, size_t ws_bytes, void* stream) {
  if (!W || !X || !Y || !aligned16(W) || !aligned16(X) || !aligned16(Y)) return QBLORA_ERR_INVALID_ARG;
  if (d_out < 1 || d_in < 8 || d_in % 8 || tokens < 1 || tokens >= ((int64_t)1 << 31) || !dtype_ok(y_dtype)) return QBLORA_ERR_INVALID_ARG;
  if (!ws || !aligned16(ws) || ws_bytes < dense_gemm_ws_bytes()) return QBLORA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int rc = reset_status(ws, st);
  if (rc) return rc;
  return launch_dense_gemm(static_cast<const __nv_bfloat16*>(W), d_out, d_in, static_cast<const __nv_bfloat16*>(X), tokens, Y,
                           y_dtype, static_cast<int*>(ws), st);
}

int qablora_merge_noalloc(const qblora_qweight* qw, const qblora_adapter* adapter, float* beta_out,
                          void* stream) {
  QwView q; int rc = make_qw(qw, &q);
  if (rc) return rc;
  if (q.qfmt != QBLORA_FMT_AFFINE_MINMAX || !adapter || !beta_out || !aligned16(beta_out)) return QBLORA_ERR_INVALID_ARG;
  AdView ad; rc = make_ad(adapter, q, true, &ad);
  if (rc) return rc;
  if (ad.l1 % q.block_in || ad.l2 % q.block_out || ad.op != QBLORA_SCALE_AVGPOOL_REPEAT) return QBLORA_ERR_INVALID_ARG;
  if ((int64_t)ad.P * ad.Q > merge_noalloc_capacity()) return QBLORA_ERR_TOO_LARGE;
  return launch_merge_noalloc(q, ad, adapter->B == nullptr, beta_out, static_cast<cudaStream_t>(stream));
}

int qablora_lowbit_gemm(const qblora_qweight* qw, const void* X, int64_t tokens, void* Y, int y_dtype,
                        void* ws, size_t ws_bytes, void* stream) {
  QwView q; int rc = make_qw(qw, &q);
  if (rc) return rc;
  if (q.qfmt != QBLORA_FMT_AFFINE_MINMAX) return QBLORA_ERR_INVALID_ARG;
  if (!X || !Y || !aligned16(X) || !aligned16(Y) || tokens < 1 || !dtype_ok(y_dtype)) return QBLORA_ERR_INVALID_ARG;
  const size_t need = ws_bytes_impl(QBLORA_OP_LOWBIT_GEMM, q, nullptr, tokens);
  if (!ws || !aligned16(ws) || ws_bytes < with_expansion(need, q)) return QBLORA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const __nv_bfloat16* Xb = static_cast<const __nv_bfloat16*>(X);
  const bool expanded = q.code_bits < 4;
  rc = expand_codes(&q, need, ws, st);
  if (rc) return rc;
  // the decode kernel clears the status word itself: one launch per call (it is chained to its predecessor as a
  // programmatic dependent unless that predecessor has just written the codes)
  if (gemv_supported(q, tokens)) return launch_lowbit_gemv(q, Xb, tokens, Y, y_dtype, static_cast<int*>(ws), st, !expanded);
  rc = reset_status(ws, st);
  if (rc) return rc;
  if (!force_general() && tc_supported(q, nullptr, tokens))
    return tc_lowbit_gemm(q, Xb, tokens, Y, y_dtype, static_cast<char*>(ws), st);
  return simt_linear_fwd(q, nullptr, Xb, tokens, Y, y_dtype, static_cast<char*>(ws), st);
}

}  // extern "C"
