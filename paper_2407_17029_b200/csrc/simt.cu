// General CUDA-core path of the adapted quantized linear: any quantization block shape and any
// size.  One tiled fp32 GEMM template with operand loaders (bf16 / fp32 matrices with arbitrary
// strides, or the packed 4-bit weight dequantized on the fly) and epilogues.  The tensor-core
// path (tc_gemm.cu) covers the block shape the fine-tuning workloads use; this one covers the rest.
#include "common.cuh"

namespace qb {
namespace {

struct LdF32 {
  const float* p; int64_t s0, s1;  // element (a, b) at p[a*s0 + b*s1]
  __device__ void prepare(float*) const {}
  __device__ float operator()(int a, int b, const float*) const { return p[a * s0 + b * s1]; }
};
struct LdBF16 {
  const __nv_bfloat16* p; int64_t s0, s1;
  __device__ void prepare(float*) const {}
  __device__ float operator()(int a, int b, const float*) const {
    return __bfloat162float(p[a * s0 + b * s1]);
  }
};
// Dequantized weight w~[o][i] = alpha * level[c] (+ beta); `o_first` says whether the loader's first
// index is the output row (forward: B(k = i, n = o) is called as (n, k)) or the input column.
struct LdWq {
  QwView q; bool o_first;
  __device__ void prepare(float* lvl) const {
    if (threadIdx.x < 16) lvl[threadIdx.x] = q.level[threadIdx.x];
  }
  __device__ float operator()(int a, int b, const float* lvl) const {
    const int o = o_first ? a : b, i = o_first ? b : a;
    const uint8_t byte = q.codes[(int64_t)o * (q.d_in >> 1) + (i >> 1)];
    const int c = (i & 1) ? (byte >> 4) : (byte & 15);
    const int64_t bi = (int64_t)(o / q.block_out) * q.G + i / q.block_in;
    const float al = q.alpha[bi];
    return q.beta ? fmaf(al, lvl[c], q.beta[bi]) : al * lvl[c];
  }
};

struct EpStoreF32 {
  float* C; int64_t ld;
  __device__ void operator()(int m, int n, float acc) const { C[m * ld + n] = acc; }
};
struct EpOut {  // out[m][n] = acc + scale * side[m][n / div]   (side may be NULL)
  void* out; int dtype; int64_t ld; const float* side; int side_ld; int div; float scale;
  bool divide;  // true: side / div (backward unpooling), false: side * scale (forward repeat)
  __device__ void operator()(int m, int n, float acc) const {
    if (side) {
      float sv = side[(int64_t)m * side_ld + n / div];
      acc += divide ? __fdiv_rn(sv, (float)div) : scale * sv;
    }
    if (dtype == QBLORA_BF16) reinterpret_cast<__nv_bfloat16*>(out)[m * ld + n] = __float2bfloat16_rn(acc);
    else reinterpret_cast<float*>(out)[m * ld + n] = acc;
  }
};

// C(m, n) = sum_k la(m, k) * lb(n, k), 64 x 64 x 16 tiles, 256 threads, 4 x 4 outputs per thread.
// A_KC / B_KC: whether k is the contiguous index of that operand (picks the coalesced load order).
template <class LA, class LB, class EP, bool A_KC, bool B_KC>
__global__ void __launch_bounds__(256) simt_gemm_kernel(int M, int N, int K, LA la, LB lb, EP ep) {
  __shared__ float As[16][68];
  __shared__ float Bs[16][68];
  __shared__ float lvl[16];
  la.prepare(lvl);
  lb.prepare(lvl);
  __syncthreads();
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  float acc[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += 16) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int idx = tid + e * 256;
      {
        const int k = A_KC ? (idx & 15) : (idx >> 6), m = A_KC ? (idx >> 4) : (idx & 63);
        As[k][m] = (m0 + m < M && k0 + k < K) ? la(m0 + m, k0 + k, lvl) : 0.0f;
      }
      {
        const int k = B_KC ? (idx & 15) : (idx >> 6), n = B_KC ? (idx >> 4) : (idx & 63);
        Bs[k][n] = (n0 + n < N && k0 + k < K) ? lb(n0 + n, k0 + k, lvl) : 0.0f;
      }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = As[k][ty * 4 + i]; b[i] = Bs[k][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int m = m0 + ty * 4 + i, n = n0 + tx * 4 + j;
      if (m < M && n < N) ep(m, n, acc[i][j]);
    }
}

template <bool A_KC, bool B_KC, class LA, class LB, class EP>
int gemm(int64_t M, int64_t N, int64_t K, LA la, LB lb, EP ep, cudaStream_t st) {
  dim3 grid((unsigned)((N + 63) / 64), (unsigned)((M + 63) / 64));
  if (grid.y > 65535) return QBLORA_ERR_UNSUPPORTED;
  simt_gemm_kernel<LA, LB, EP, A_KC, B_KC><<<grid, 256, 0, st>>>((int)M, (int)N, (int)K, la, lb, ep);
  count_launch();
  QB_CUDA(cudaGetLastError());
  return QBLORA_OK;
}

// x'[t][p] = mean of lambda_in consecutive inputs (AvgPool of Sec. 3.2), fp32.
__global__ void pool_kernel(const __nv_bfloat16* __restrict__ X, int64_t T, int d_in, int l1,
                            float* __restrict__ xp) {
  const int P = d_in / l1;
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= T * P) return;
  const int64_t t = idx / P; const int p = (int)(idx % P);
  float s = 0.0f;
  for (int j = 0; j < l1; ++j) s += __bfloat162float(X[t * d_in + (int64_t)p * l1 + j]);
  xp[idx] = __fdiv_rn(s, (float)l1);
}

// dv[t][q] = s * sum of lambda_out consecutive output gradients (adjoint of repeat_interleave).
__global__ void dv_kernel(const __nv_bfloat16* __restrict__ dY, int64_t T, int d_out, int l2, float s,
                          float* __restrict__ dv) {
  const int Q = d_out / l2;
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= T * Q) return;
  const int64_t t = idx / Q; const int q = (int)(idx % Q);
  float a = 0.0f;
  for (int j = 0; j < l2; ++j) a += __bfloat162float(dY[t * d_out + (int64_t)q * l2 + j]);
  dv[idx] = s * a;
}

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
    pool_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(X, T, qw.d_in, ad->l1, w.xp);
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
           ad ? ad->s : 0.0f, false};
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
    pool_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(X, T, qw.d_in, ad->l1, w.xp);
    count_launch();
    QB_CUDA(cudaGetLastError());
    n = T * ad->Q;
    dv_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(dY, T, qw.d_out, ad->l2, ad->s, w.dv);
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
    EpOut ep{dX, dx_dtype, qw.d_in, ad ? w.dxp : nullptr, ad ? ad->P : 0, ad ? ad->l1 : 1, 0.0f, true};
    // dX[t][i] = sum_o dY[t][o] w~[o][i] : lb(n = i, k = o)
    DominantKernelTimer timer(st);
    return gemm<true, false>(T, qw.d_in, qw.d_out, LdBF16{dY, qw.d_out, 1}, LdWq{qw, false}, ep, st);
  }
  return QBLORA_OK;
}

}  // namespace qb
