// Low-bit product for small token counts (decode, T <= 16):
//   Y[t][o] = sum_i X[t][i] * (alpha[o][i/64] * c[o][i] + beta'[o][i/64])            (Sec. 3.3)
// The packed weight is streamed exactly once (DRAM traffic = codes + alpha + beta).  Measured: the
// kernel is bound by instruction issue and load latency (about 120 warp instructions per 16 rows x 64
// codes, four warps per scheduler), reaching 25-35 % of the HBM copy bandwidth at T = 1.
//
// Mapping.  A CTA of eight warps owns 16 output rows; warp w takes the w-th eighth of the 64-wide
// quantization groups of those rows, and the eight partial results are summed through shared memory
// in warp order (deterministic).  Inside a warp the work is shaped for mma.sync.m16n8k16 (bf16, fp32
// accumulate): the 16 rows are the M
// side, up to 8 tokens per N tile.  A thread (g = lane / 4, tg = lane % 4) loads, for rows g and
// g + 8, the 8 bytes holding codes 16 tg .. 16 tg + 15 of the current group and turns each 32-bit word
// into four bf16 pairs (128 + c) with one logic op per pair (the nibbles land in the mantissa of
// 128.0).  Because the order of the k index inside an MMA is free as long as both operands agree,
// nibble pairs (e, e + 4) are used as they fall out of the word and the token operand is permuted to
// match with byte permutes.  A second MMA chain with A = 1.0 yields S = sum of x over the group in
// the accumulator layout, and the group contributes
//   alpha * sum((128 + c) x) + (beta - 128 alpha) * S  =  alpha * sum(c x) + beta * S.
#include "common.cuh"

namespace qb {
namespace {

constexpr int GV_WARPS = 8;
constexpr int GV_ROWS = 16;

__device__ __forceinline__ uint32_t gv_prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t r;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
  return r;
}
__device__ __forceinline__ void gv_mma(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                       uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// word of 8 codes -> (128 + c) bf16 pairs: v[e] = (code e, code e + 4), e = 0..3
__device__ __forceinline__ void gv_unpack(uint32_t w, uint32_t (&v)[4]) {
  v[0] = (w & 0x000F000Fu) | 0x43004300u;
  v[1] = ((w >> 4) & 0x000F000Fu) | 0x43004300u;
  v[2] = ((w >> 8) & 0x000F000Fu) | 0x43004300u;
  v[3] = ((w >> 12) & 0x000F000Fu) | 0x43004300u;
}

// Streams NB consecutive groups: all code / scale loads are issued first (constant offsets from the
// running pointers), then each group is unpacked and multiplied.
template <int NT, int NB>
__device__ __forceinline__ void gv_groups(const uint2* __restrict__ c0, const uint2* __restrict__ c1,
                                          const float* __restrict__ al0, const float* __restrict__ al1,
                                          const float* __restrict__ be0, const float* __restrict__ be1,
                                          const uint4* const (&xp)[NT], const bool (&xlive)[NT], float (&y)[NT][4]) {
  uint2 w0[NB], w1[NB];
  float a0[NB], a1[NB], b0[NB], b1[NB];
#pragma unroll
  for (int u = 0; u < NB; ++u) {
    w0[u] = __ldg(c0 + u * 4); w1[u] = __ldg(c1 + u * 4);
    a0[u] = __ldg(al0 + u); a1[u] = __ldg(al1 + u);
    b0[u] = __ldg(be0 + u); b1[u] = __ldg(be1 + u);
  }
  const uint32_t ones = 0x3F803F80u;   // bf16 (1.0, 1.0)
#pragma unroll
  for (int u = 0; u < NB; ++u) {
    uint32_t va[2][4], vb[2][4];      // [word][pair] for rows g (va) and g + 8 (vb)
    gv_unpack(w0[u].x, va[0]); gv_unpack(w0[u].y, va[1]);
    gv_unpack(w1[u].x, vb[0]); gv_unpack(w1[u].y, vb[1]);
    const float s0 = fmaf(-128.0f, a0[u], b0[u]), s1 = fmaf(-128.0f, a1[u], b1[u]);
#pragma unroll
    for (int j = 0; j < NT; ++j) {
      uint4 x0 = make_uint4(0, 0, 0, 0), x1 = make_uint4(0, 0, 0, 0);
      if (xlive[j]) { x0 = __ldg(xp[j] + u * 8); x1 = __ldg(xp[j] + u * 8 + 1); }
      float acc[4] = {0.f, 0.f, 0.f, 0.f}, sum[4] = {0.f, 0.f, 0.f, 0.f};
      const uint32_t xr[2][4] = {{x0.x, x0.y, x0.z, x0.w}, {x1.x, x1.y, x1.z, x1.w}};
#pragma unroll
      for (int wd = 0; wd < 2; ++wd) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          // codes (2h, 2h+4) and (2h+1, 2h+5) of word wd <-> x at the same positions
          const uint32_t bx0 = gv_prmt(xr[wd][h], xr[wd][h + 2], 0x5410u);
          const uint32_t bx1 = gv_prmt(xr[wd][h], xr[wd][h + 2], 0x7632u);
          gv_mma(acc, va[wd][2 * h], vb[wd][2 * h], va[wd][2 * h + 1], vb[wd][2 * h + 1], bx0, bx1);
          gv_mma(sum, ones, ones, ones, ones, bx0, bx1);
        }
      }
      y[j][0] = fmaf(a0[u], acc[0], fmaf(s0, sum[0], y[j][0]));
      y[j][1] = fmaf(a0[u], acc[1], fmaf(s0, sum[1], y[j][1]));
      y[j][2] = fmaf(a1[u], acc[2], fmaf(s1, sum[2], y[j][2]));
      y[j][3] = fmaf(a1[u], acc[3], fmaf(s1, sum[3], y[j][3]));
    }
  }
}

template <int NT>   // NT = number of 8-token tiles (1 or 2)
__global__ void __launch_bounds__(GV_WARPS * 32, 2) lowbit_gemv_kernel(QwView q, const __nv_bfloat16* __restrict__ X, int T,
                                                                       void* __restrict__ Y, int y_dtype) {
  __shared__ float red[GV_WARPS][GV_ROWS][NT * 8];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, tg = lane & 3;
  const int row_base = blockIdx.x * GV_ROWS;
  // rows past the end are clamped for loads and dropped at the store
  const int r0 = min(row_base + g, q.d_out - 1), r1 = min(row_base + g + 8, q.d_out - 1);
  const int per = (q.G + GV_WARPS - 1) / GV_WARPS;
  const int g_begin = min(warp * per, q.G), g_end = min(g_begin + per, q.G);
  // running pointers of this thread, positioned at its first group
  const uint2* c0 = reinterpret_cast<const uint2*>(q.codes + (int64_t)r0 * (q.d_in >> 1)) + tg + g_begin * 4;
  const uint2* c1 = reinterpret_cast<const uint2*>(q.codes + (int64_t)r1 * (q.d_in >> 1)) + tg + g_begin * 4;
  const float* al0 = q.alpha + (int64_t)r0 * q.G + g_begin; const float* al1 = q.alpha + (int64_t)r1 * q.G + g_begin;
  const float* be0 = q.beta + (int64_t)r0 * q.G + g_begin;  const float* be1 = q.beta + (int64_t)r1 * q.G + g_begin;
  const uint4* xp[NT];
  bool xlive[NT];
#pragma unroll
  for (int j = 0; j < NT; ++j) {
    const int t = j * 8 + g;
    xlive[j] = t < T;
    xp[j] = reinterpret_cast<const uint4*>(X + (int64_t)(xlive[j] ? t : 0) * q.d_in) + tg * 2 + g_begin * 8;
  }
  float y[NT][4];
#pragma unroll
  for (int j = 0; j < NT; ++j) { y[j][0] = y[j][1] = y[j][2] = y[j][3] = 0.0f; }

  constexpr int NB = 4;
  int left = g_end - g_begin;
  for (; left >= NB; left -= NB) {
    gv_groups<NT, NB>(c0, c1, al0, al1, be0, be1, xp, xlive, y);
    c0 += NB * 4; c1 += NB * 4; al0 += NB; al1 += NB; be0 += NB; be1 += NB;
#pragma unroll
    for (int j = 0; j < NT; ++j) xp[j] += NB * 8;
  }
  for (; left > 0; --left) {
    gv_groups<NT, 1>(c0, c1, al0, al1, be0, be1, xp, xlive, y);
    c0 += 4; c1 += 4; ++al0; ++al1; ++be0; ++be1;
#pragma unroll
    for (int j = 0; j < NT; ++j) xp[j] += 8;
  }
  // accumulator layout: [0],[1] = row g, tokens 2tg, 2tg+1; [2],[3] = row g + 8
#pragma unroll
  for (int j = 0; j < NT; ++j) {
    red[warp][g][j * 8 + 2 * tg] = y[j][0]; red[warp][g][j * 8 + 2 * tg + 1] = y[j][1];
    red[warp][g + 8][j * 8 + 2 * tg] = y[j][2]; red[warp][g + 8][j * 8 + 2 * tg + 1] = y[j][3];
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < GV_ROWS * NT * 8; idx += GV_WARPS * 32) {
    const int t = idx / GV_ROWS, r = idx % GV_ROWS;     // consecutive threads -> consecutive output rows
    const int o = row_base + r;
    if (t < T && o < q.d_out) {
      float a = 0.0f;
#pragma unroll
      for (int w = 0; w < GV_WARPS; ++w) a += red[w][r][t];
      if (y_dtype == QBLORA_BF16) reinterpret_cast<__nv_bfloat16*>(Y)[(int64_t)t * q.d_out + o] = __float2bfloat16_rn(a);
      else reinterpret_cast<float*>(Y)[(int64_t)t * q.d_out + o] = a;
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
  const int grid = (qw.d_out + GV_ROWS - 1) / GV_ROWS;
  if (T <= 8) lowbit_gemv_kernel<1><<<grid, GV_WARPS * 32, 0, st>>>(qw, X, (int)T, Y, y_dtype);
  else lowbit_gemv_kernel<2><<<grid, GV_WARPS * 32, 0, st>>>(qw, X, (int)T, Y, y_dtype);
  QB_CUDA(cudaGetLastError());
  return QBLORA_OK;
}

}  // namespace qb
