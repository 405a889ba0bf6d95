// General CUDA-core path of the adapted quantized linear: any quantization block shape and any
// size.  One tiled fp32 GEMM template with operand loaders (bf16 / fp32 matrices with arbitrary
// strides, or the packed 4-bit weight dequantized on the fly) and epilogues.  The tensor-core
// path (tc_gemm.cu) covers the block shape the fine-tuning workloads use; this one covers the rest.
#include "common.cuh"
#include "simt_gemm.cuh"

namespace qb {
using namespace simt;
namespace {

struct SimtWs {
  float *xp, *u, *v, *dv, *du, *dxp;
  size_t bytes;
};

SimtWs carve(int op, const AdView* ad, int64_t T, char* ws) {
  SimtWs w{};
  size_t off = kStatusBytes;
  auto take = [&](size_t n) { char* p = ws ? ws + off : nullptr; off += align_up(n * sizeof(float), 256); return (float*)p; };
  if (ad) {
    w.xp = take((size_t)T * ad->P);
    w.u = take((size_t)T * ad->r);
    if (op == QBLORA_OP_LINEAR_FWD) {
      w.v = take((size_t)T * ad->Q);
    } else {
      w.dv = take((size_t)T * ad->Q);
      w.du = take((size_t)T * ad->r);
      w.dxp = take((size_t)T * ad->P);
    }
  }
  w.bytes = off;
  return w;
}

}  // namespace

size_t simt_ws_bytes(int op, const QwView&, const AdView* ad, int64_t T) {
  return carve(op, ad, T, nullptr).bytes;
}

int simt_linear_fwd(const QwView& qw, const AdView* ad, const __nv_bfloat16* X, int64_t T, void* Y,
                    int y_dtype, char* ws, cudaStream_t st) {
  SimtWs w = carve(QBLORA_OP_LINEAR_FWD, ad, T, ws);
  int rc;
  if (ad) {
    int64_t n = T * ad->P;
    pool_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(X, T, qw.d_in, ad->l1, ad->op, w.xp);
    count_launch();
    QB_CUDA(cudaGetLastError());
    // u = x' A : A is [P][r] -> lb(n = k_rank, k = p) = A[p][k_rank]
    rc = gemm<true, false>(T, ad->r, ad->P, LdF32{w.xp, ad->P, 1}, LdBF16{ad->A, 1, ad->r},
                           EpStoreF32{w.u, ad->r}, st);
    if (rc) return rc;
    // v = u B : B is [r][Q] -> lb(n = q, k) = B[k][q]
    rc = gemm<true, false>(T, ad->Q, ad->r, LdF32{w.u, ad->r, 1}, LdBF16{ad->B, 1, ad->Q},
                           EpStoreF32{w.v, ad->Q}, st);
    if (rc) return rc;
  }
  EpOut ep{Y, y_dtype, qw.d_out, ad ? w.v : nullptr, ad ? ad->Q : 0, ad ? ad->l2 : 1,
           ad ? ad->s : 0.0f, false, ad ? ad->op : 0};
  DominantKernelTimer timer(st);
  return gemm<true, true>(T, qw.d_out, qw.d_in, LdBF16{X, qw.d_in, 1}, LdWq{qw, true}, ep, st);
}

int simt_linear_bwd(const QwView& qw, const AdView* ad, const __nv_bfloat16* X,
                    const __nv_bfloat16* dY, int64_t T, void* dX, int dx_dtype, float* dA, float* dB,
                    char* ws, cudaStream_t st) {
  SimtWs w = carve(QBLORA_OP_LINEAR_BWD, ad, T, ws);
  int rc;
  if (ad) {
    int64_t n = T * ad->P;
    pool_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(X, T, qw.d_in, ad->l1, ad->op, w.xp);
    count_launch();
    QB_CUDA(cudaGetLastError());
    n = T * ad->Q;
    dv_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(dY, T, qw.d_out, ad->l2, ad->op, ad->s, w.dv);
    count_launch();
    QB_CUDA(cudaGetLastError());
    // du = dv B^T : lb(n = k_rank, k = q) = B[k_rank][q]
    rc = gemm<true, true>(T, ad->r, ad->Q, LdF32{w.dv, ad->Q, 1}, LdBF16{ad->B, ad->Q, 1},
                          EpStoreF32{w.du, ad->r}, st);
    if (rc) return rc;
    if (dB) {
      rc = gemm<true, false>(T, ad->r, ad->P, LdF32{w.xp, ad->P, 1}, LdBF16{ad->A, 1, ad->r},
                             EpStoreF32{w.u, ad->r}, st);
      if (rc) return rc;
      // dB[k][q] = sum_t u[t][k] dv[t][q]
      rc = gemm<false, false>(ad->r, ad->Q, T, LdF32{w.u, 1, ad->r}, LdF32{w.dv, 1, ad->Q},
                              EpStoreF32{dB, ad->Q}, st);
      if (rc) return rc;
    }
    if (dA) {
      // dA[p][k] = sum_t x'[t][p] du[t][k]
      rc = gemm<false, false>(ad->P, ad->r, T, LdF32{w.xp, 1, ad->P}, LdF32{w.du, 1, ad->r},
                              EpStoreF32{dA, ad->r}, st);
      if (rc) return rc;
    }
    if (dX) {
      // dx' = du A^T : lb(n = p, k) = A[p][k]
      rc = gemm<true, true>(T, ad->P, ad->r, LdF32{w.du, ad->r, 1}, LdBF16{ad->A, ad->r, 1},
                            EpStoreF32{w.dxp, ad->P}, st);
      if (rc) return rc;
    }
  }
  if (dX) {
    EpOut ep{dX, dx_dtype, qw.d_in, ad ? w.dxp : nullptr, ad ? ad->P : 0, ad ? ad->l1 : 1, 0.0f, true, ad ? ad->op : 0};
    // dX[t][i] = sum_o dY[t][o] w~[o][i] : lb(n = i, k = o)
    DominantKernelTimer timer(st);
    return gemm<true, false>(T, qw.d_in, qw.d_out, LdBF16{dY, qw.d_out, 1}, LdWq{qw, false}, ep, st);
  }
  return QBLORA_OK;
}

namespace {
__global__ void identity_kernel(__nv_bfloat16* out, int n) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx < (int64_t)n * n) out[idx] = __float2bfloat16_rn((idx / n) == (idx % n) ? 1.0f : 0.0f);
}
}  // namespace

int launch_identity(__nv_bfloat16* out, int n, cudaStream_t st) {
  const int64_t total = (int64_t)n * n;
  identity_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(out, n);
  count_launch();
  QB_CUDA(cudaGetLastError());
  return QBLORA_OK;
}

}  // namespace qb
