// Low-bit product for small token counts (decode): Y[t][o] = sum_i X[t][i] (alpha c + beta')[o][i].
// The packed weight is streamed exactly once with 128-bit loads; one warp owns one output row and
// keeps one fp32 accumulator per token.  Per 32-code chunk (half a quantization group) the kernel
// forms sum(c * x) and sum(x) and applies alpha and beta once.
#include "common.cuh"

namespace qb {
namespace {

template <int TT>
__global__ void __launch_bounds__(256) lowbit_gemv_kernel(QwView q, const __nv_bfloat16* __restrict__ X,
                                                          int T, void* __restrict__ Y, int y_dtype) {
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  const int chunks = q.d_in >> 5;  // 16-byte chunks (32 codes) per row
  for (int o = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; o < q.d_out; o += warps) {
    float acc[TT];
#pragma unroll
    for (int t = 0; t < TT; ++t) acc[t] = 0.0f;
    const uint4* row = reinterpret_cast<const uint4*>(q.codes + (int64_t)o * (q.d_in >> 1));
    for (int ch = lane; ch < chunks; ch += 32) {
      const uint4 pk = __ldg(row + ch);
      const float al = __ldg(q.alpha + (int64_t)o * q.G + (ch >> 1));
      const float be = __ldg(q.beta + (int64_t)o * q.G + (ch >> 1));
      const uint32_t w[4] = {pk.x, pk.y, pk.z, pk.w};
#pragma unroll
      for (int t = 0; t < TT; ++t) {
        if (t < T) {
          const uint4* xr = reinterpret_cast<const uint4*>(X + (int64_t)t * q.d_in + ch * 32);
          float dot = 0.0f, sum = 0.0f;
#pragma unroll
          for (int j = 0; j < 4; ++j) {  // word j: codes 8j .. 8j+7 <-> X 8j .. 8j+7 (one uint4)
            const uint4 xv = __ldg(xr + j);
            const uint32_t xs[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float x0 = __uint_as_float(xs[e] << 16);
              const float x1 = __uint_as_float(xs[e] & 0xffff0000u);
              const float c0 = (float)((w[j] >> (8 * e)) & 15u);
              const float c1 = (float)((w[j] >> (8 * e + 4)) & 15u);
              dot = fmaf(c0, x0, dot); dot = fmaf(c1, x1, dot);
              sum += x0 + x1;
            }
          }
          acc[t] = fmaf(al, dot, fmaf(be, sum, acc[t]));
        }
      }
    }
#pragma unroll
    for (int t = 0; t < TT; ++t) {
      float a = acc[t];
#pragma unroll
      for (int s = 16; s > 0; s >>= 1) a += __shfl_xor_sync(0xffffffffu, a, s);
      if (lane == 0 && t < T) {
        if (y_dtype == QBLORA_BF16) reinterpret_cast<__nv_bfloat16*>(Y)[(int64_t)t * q.d_out + o] = __float2bfloat16_rn(a);
        else reinterpret_cast<float*>(Y)[(int64_t)t * q.d_out + o] = a;
      }
    }
  }
}

}  // namespace

bool gemv_supported(const QwView& qw, int64_t T) {
  return qw.block_in == 64 && qw.block_out == 1 && qw.qfmt == QBLORA_FMT_AFFINE_MINMAX && T <= 16;
}

int launch_lowbit_gemv(const QwView& qw, const __nv_bfloat16* X, int64_t T, void* Y, int y_dtype,
                       cudaStream_t st) {
  DominantKernelTimer timer(st);
  count_launch();
  const int rows_per_cta = 8;
  int grid = (qw.d_out + rows_per_cta - 1) / rows_per_cta;
  if (T <= 1) lowbit_gemv_kernel<1><<<grid, 256, 0, st>>>(qw, X, (int)T, Y, y_dtype);
  else if (T <= 2) lowbit_gemv_kernel<2><<<grid, 256, 0, st>>>(qw, X, (int)T, Y, y_dtype);
  else if (T <= 4) lowbit_gemv_kernel<4><<<grid, 256, 0, st>>>(qw, X, (int)T, Y, y_dtype);
  else if (T <= 8) lowbit_gemv_kernel<8><<<grid, 256, 0, st>>>(qw, X, (int)T, Y, y_dtype);
  else lowbit_gemv_kernel<16><<<grid, 256, 0, st>>>(qw, X, (int)T, Y, y_dtype);
  QB_CUDA(cudaGetLastError());
  return QBLORA_OK;
}

}  // namespace qb
