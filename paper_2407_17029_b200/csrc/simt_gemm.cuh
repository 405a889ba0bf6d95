// CUDA-core building blocks shared by the general path and the adapter side of the tensor-core
// path: a tiled fp32 GEMM template with operand loaders / epilogues, AvgPool and its adjoint.
#pragma once
#include "common.cuh"

namespace qb {
namespace simt {

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
struct EpOut {  // out[m][n] = acc + scale * side[m][src(n)]   (side may be NULL; src = the operator pair's index map)
  void* out; int dtype; int64_t ld; const float* side; int side_ld; int div; float scale;
  bool divide;  // true: side / div (backward un-pooling; no division for the sampling operators), false: side * scale (forward)
  int op;       // qblora_scale_op
  __device__ void operator()(int m, int n, float acc) const {
    if (side) {
      const int j = scale_src(op, n, div, side_ld);
      if (j >= 0) {
        const float sv = side[(int64_t)m * side_ld + j];
        acc += divide ? (op == QBLORA_SCALE_AVGPOOL_REPEAT ? __fdiv_rn(sv, (float)div) : sv) : scale * sv;
      }
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
inline int gemm(int64_t M, int64_t N, int64_t K, LA la, LB lb, EP ep, cudaStream_t st) {
  dim3 grid((unsigned)((N + 63) / 64), (unsigned)((M + 63) / 64));
  if (grid.y > 65535) return QBLORA_ERR_UNSUPPORTED;
  simt_gemm_kernel<LA, LB, EP, A_KC, B_KC><<<grid, 256, 0, st>>>((int)M, (int)N, (int)K, la, lb, ep);
  count_launch();
  QB_CUDA(cudaGetLastError());
  return QBLORA_OK;
}

// x'[t][p] = mean of lambda_in consecutive inputs (AvgPool of Sec. 3.2), fp32; for the alternative operators
// of the Sec. 4 ablation the kept value x[p] (truncation) or the sample x[lambda_in p] (interval sampling).
static __global__ void pool_kernel(const __nv_bfloat16* __restrict__ X, int64_t T, int d_in, int l1, int op,
                            float* __restrict__ xp) {
  const int P = d_in / l1;
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= T * P) return;
  const int64_t t = idx / P; const int p = (int)(idx % P);
  if (op != QBLORA_SCALE_AVGPOOL_REPEAT) {
    xp[idx] = __bfloat162float(X[t * d_in + (op == QBLORA_SCALE_TRUNCATE_ZEROPAD ? p : (int64_t)p * l1)]);
    return;
  }
  float s = 0.0f;
  for (int j = 0; j < l1; ++j) s += __bfloat162float(X[t * d_in + (int64_t)p * l1 + j]);
  xp[idx] = __fdiv_rn(s, (float)l1);
}

// dv[t][q] = s * sum of lambda_out consecutive output gradients (adjoint of repeat_interleave); the adjoint
// of zero padding / zero filling reads the single output the value was written to.
static __global__ void dv_kernel(const __nv_bfloat16* __restrict__ dY, int64_t T, int d_out, int l2, int op, float s,
                          float* __restrict__ dv) {
  const int Q = d_out / l2;
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= T * Q) return;
  const int64_t t = idx / Q; const int q = (int)(idx % Q);
  if (op != QBLORA_SCALE_AVGPOOL_REPEAT) {
    dv[idx] = s * __bfloat162float(dY[t * d_out + (op == QBLORA_SCALE_TRUNCATE_ZEROPAD ? q : (int64_t)q * l2)]);
    return;
  }
  float a = 0.0f;
  for (int j = 0; j < l2; ++j) a += __bfloat162float(dY[t * d_out + (int64_t)q * l2 + j]);
  dv[idx] = s * a;
}


}  // namespace simt
}  // namespace qb
