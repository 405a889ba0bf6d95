// Block-wise 4-bit quantizer (Eq. 1).  Every floating-point step is a single IEEE fp32 operation
// (explicit round-to-nearest intrinsics, no fused multiply-add), so codes, alpha and beta are
// uniquely determined by the input.
#include "common.cuh"

namespace qb {
namespace {

struct QuantTable {
  float mid[15];  // fl32 midpoints between adjacent levels
  int zero_idx;   // index of the level closest to 0 (used for all-zero blocks)
  float qmax;     // largest code of the min-max grid: 2^N - 1 (15 for the 4-bit weight)
  int use_lut;    // level table: midpoints far enough apart for the bucket table of code_of_level_lut
};

// Bucket table of the level-table format.  [-1, 1] is covered by 129 equal buckets centred on the multiples of 1/64
// (the table has 256 entries so that any 8-bit index is in range); when adjacent midpoints
// are farther apart than a bucket (plus margins), a bucket, widened by LUT_MARGIN on both sides, sees at most one
// midpoint m, and for every v in it  #{ j : v > mid_j } = base + (v > m),  base = number of midpoints below m (or
// below the bucket when it sees none; m is then a huge value).  An entry is ONE 32-bit word: the float m with its
// four lowest mantissa bits replaced by base.  That moves m by less than 16 ulp < 1e-6, and a value closer than
// LUT_NEAR = 2e-6 to the stored m is decided by the exact quotient anyway, so the comparison with the stored m gives
// the same answer as with m itself everywhere else.  One 4-byte shared-memory load replaces the search.  The bucket
// of v is round(v * 64 + 64), read off the low mantissa bits after adding 2^23 (no conversion instruction, no clamp:
// |v| <= 1 up to rounding, and a non-finite v still gives an index inside the table); a v within rounding of a
// bucket edge may land in the neighbour, whose widened range still covers it.
constexpr int LUT_BUCKETS = 256;
constexpr float LUT_SCALE = 64.0f;       // buckets per unit: bucket of v = round(v * 64 + 64)
constexpr float LUT_NEAR = 2e-6f;        // closer to the stored midpoint than this: the exact quotient decides
constexpr float LUT_MARGIN = 8e-6f;      // > LUT_NEAR + 16 ulp + rounding of the bucket index (1.2e-7)
constexpr float LUT_NONE = 3.0e38f;      // "no midpoint in this bucket"

__device__ __forceinline__ float load_w(const float* W, int64_t i) { return W[i]; }
__device__ __forceinline__ float load_w(const __nv_bfloat16* W, int64_t i) {
  return __bfloat162float(W[i]);
}

__device__ __forceinline__ int code_of_level(float v, const QuantTable& t) {
  int c = 0;
#pragma unroll
  for (int j = 0; j < 15; ++j) c += (v > t.mid[j]) ? 1 : 0;
  return c;
}

// Level-table code without a division per element: code = #{ j : fl32(w / absmax) > mid_j }.
// va = fl32(w * fl32(1 / absmax)) is within 1.2e-7 of the exact quotient (|quotient| <= 1), the rounded quotient
// within 6e-8, and a comparison with mid_j can only differ between the two when the exact quotient lies within one
// ulp of mid_j.  So the position of va among the midpoints (binary search in a shared-memory copy, s_mid[0] = -inf,
// s_mid[1 + j] = mid_j, s_mid[16] = +inf) is the code whenever va is farther than 1e-6 from both neighbouring
// midpoints; otherwise (and for a non-finite va) the exact quotient is compared with all fifteen as before.
__device__ __forceinline__ int code_of_level_fast(float w, float absmax, float inv, const float* s_mid, const QuantTable& t) {
  const float va = __fmul_rn(w, inv);
  int k = 0;
  k += (va > s_mid[k + 8]) ? 8 : 0;
  k += (va > s_mid[k + 4]) ? 4 : 0;
  k += (va > s_mid[k + 2]) ? 2 : 0;
  k += (va > s_mid[k + 1]) ? 1 : 0;
  const float lo = s_mid[k], hi = s_mid[k + 1];
  if ((__fsub_rn(va, lo) > 1e-6f) && (__fsub_rn(hi, va) > 1e-6f)) return k;
  return code_of_level(__fdiv_rn(w, absmax), t);
}

// code = clamp(rint(fl32(fl32(w - beta) / alpha)), 0, qmax), ties to even (Eq. 1), without a division per element.
// inv = fl32(1 / alpha).  qa = fl32(x * inv) is within 2^-23 relative of the exact quotient x / alpha, and so is
// fl32(x / alpha) (within 2^-24); the quotient is at most 15, so both lie within 2e-6 of it.  When qa is farther
// than 1e-5 from every half-integer, rint(qa) and rint(fl32(x / alpha)) are therefore the same integer.  Otherwise
// (about one element in 10^5, and whenever inv overflowed or qa is not finite) the exact quotient decides.
__device__ __forceinline__ int code_of_affine(float w, float beta, float alpha, float inv, float qmax) {
  const float x = __fsub_rn(w, beta);
  const float qa = __fmul_rn(x, inv);
  // adding 2^23 rounds qa (0 <= qa < 16) to the nearest integer, ties to even, and leaves that integer in the low
  // mantissa bits; x lies in [0, max - min], so the integer is already inside [0, qmax] and needs no clamp
  const float m = __fadd_rn(qa, 8388608.0f);
  const float rq = __fsub_rn(m, 8388608.0f);
  if (fabsf(__fsub_rn(qa, rq)) < 0.49999f) return (int)(__float_as_uint(m) & 15u);
  // near a rounding boundary, or qa not finite: the exact quotient decides (ties to even), with the clamp of Eq. 1
  return (int)fminf(fmaxf(rintf(__fdiv_rn(x, alpha)), 0.0f), qmax);
}

// block_in == 64, block_out == 1.  Because d_in is a multiple of 64, block b is the flat element range
// [64 b, 64 b + 64) and its packed codes are bytes [32 b, 32 b + 32).  A warp takes four consecutive
// blocks per step: lane l owns elements 8 (l % 8) .. + 7 of block 4 w + l / 8 (one or two 16-byte loads,
// 1 KB / 512 B per warp and step, contiguous), the block's min / max / absmax come from three shuffle
// rounds inside its eight lanes, and the lane's eight codes leave as one 32-bit store.
template <typename TIn>
__global__ void __launch_bounds__(256) quantize_b64_kernel(const TIn* __restrict__ W, int64_t nblocks,
                                                           int qfmt, QuantTable tab,
                                                           uint8_t* __restrict__ codes,
                                                           float* __restrict__ alpha,
                                                           float* __restrict__ beta) {
  __shared__ float s_mid[17];
  __shared__ uint32_t s_lut[LUT_BUCKETS];
  if (threadIdx.x < 17)
    s_mid[threadIdx.x] = threadIdx.x == 0 ? -INFINITY : threadIdx.x == 16 ? INFINITY : tab.mid[min(max((int)threadIdx.x, 1), 15) - 1];
  if (tab.use_lut && threadIdx.x < LUT_BUCKETS) {
    const float lo = ((float)threadIdx.x - 0.5f) / LUT_SCALE - 1.0f, hi = ((float)threadIdx.x + 0.5f) / LUT_SCALE - 1.0f;   // exact
    float m = LUT_NONE;
    int base = 0, below = 0;
#pragma unroll
    for (int j = 0; j < 15; ++j) {
      if (tab.mid[j] >= lo - LUT_MARGIN && tab.mid[j] < hi + LUT_MARGIN) { m = tab.mid[j]; base = j; }
      below += tab.mid[j] < lo - LUT_MARGIN ? 1 : 0;
    }
    s_lut[threadIdx.x] = (__float_as_uint(m) & ~15u) | (uint32_t)(m == LUT_NONE ? below : base);
  }
  __syncthreads();
  const int lane = threadIdx.x & 31, sub = lane >> 3, part = lane & 7;
  const int64_t warps_per_grid = (int64_t)gridDim.x * (blockDim.x >> 5);
  const int64_t steps = (nblocks + 3) >> 2;
  for (int64_t w = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); w < steps; w += warps_per_grid) {
    const int64_t b = 4 * w + sub;
    const bool live = b < nblocks;
    float v[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) v[e] = 0.0f;
    if (live) {
      if constexpr (sizeof(TIn) == 4) {
        const float4* src = reinterpret_cast<const float4*>(W) + (b * 16 + part * 2);
        const float4 x0 = src[0], x1 = src[1];
        v[0] = x0.x; v[1] = x0.y; v[2] = x0.z; v[3] = x0.w; v[4] = x1.x; v[5] = x1.y; v[6] = x1.z; v[7] = x1.w;
      } else {
        const uint4 x = reinterpret_cast<const uint4*>(W)[b * 8 + part];
        const uint32_t xw[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) { v[2 * e] = __uint_as_float(xw[e] << 16); v[2 * e + 1] = __uint_as_float(xw[e] & 0xffff0000u); }
      }
    }
    float mn = v[0], mx = v[0], am = fabsf(v[0]);
#pragma unroll
    for (int e = 1; e < 8; ++e) { mn = fminf(mn, v[e]); mx = fmaxf(mx, v[e]); am = fmaxf(am, fabsf(v[e])); }
#pragma unroll
    for (int s = 4; s > 0; s >>= 1) {
      mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, s));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, s));
      am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, s));
    }
    uint32_t packed = 0;
    if (qfmt == QBLORA_FMT_CODEBOOK_ABSMAX) {
      const float inv = __frcp_rn(am);
      if (tab.use_lut) {
        // bucket table, no branch per element: the eight codes are formed unconditionally while the smallest distance
        // to a stored midpoint is tracked; a lane that came closer than LUT_NEAR to one (about one lane in 10^4)
        // redoes its eight codes with the exact quotient
        float nearest = INFINITY;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float va = __fmul_rn(v[e], inv);
          const uint32_t b = __float_as_uint(fmaf(va, LUT_SCALE, 8388608.0f + LUT_SCALE)) & (uint32_t)(LUT_BUCKETS - 1);
          const uint32_t en = s_lut[b];
          const float m = __uint_as_float(en);
          nearest = fminf(nearest, fabsf(__fsub_rn(va, m)));
          packed += ((en & 15u) + (va > m ? 1u : 0u)) << (4 * e);
        }
        if (!(nearest > LUT_NEAR) || !(am > 0.0f) || !(inv > 0.0f)) {   // also the all-zero block (va would be NaN) and an absmax whose reciprocal is not finite
          packed = 0;
#pragma unroll
          for (int e = 0; e < 8; ++e)
            packed |= (uint32_t)(am != 0.0f ? code_of_level(__fdiv_rn(v[e], am), tab) : tab.zero_idx) << (4 * e);
        }
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const int c = am != 0.0f ? code_of_level_fast(v[e], am, inv, s_mid, tab) : tab.zero_idx;
          packed |= (uint32_t)c << (4 * e);
        }
      }
      if (live && part == 0) alpha[b] = am;
    } else {
      const float d = __fsub_rn(mx, mn);
      const float a = __fdiv_rn(d, tab.qmax);
      const bool degenerate = (d == 0.0f) || (a == 0.0f);
      const float inv = __frcp_rn(a);
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int c = degenerate ? 0 : code_of_affine(v[e], mn, a, inv, tab.qmax);
        packed |= (uint32_t)c << (4 * e);
      }
      if (live && part == 0) {
        alpha[b] = degenerate ? 0.0f : a;
        beta[b] = mn == 0.0f ? 0.0f : mn;   // a zero minimum is stored as +0, whichever zeros the block holds
      }
    }
    if (live) reinterpret_cast<uint32_t*>(codes)[b * 8 + part] = packed;   // element 2k in the low nibble of byte k
  }
}

// Any block shape with an even block_in: one thread per block, two passes over its elements.
template <typename TIn>
__global__ void quantize_generic_kernel(const TIn* __restrict__ W, int d_out, int d_in, int block_in,
                                        int block_out, int qfmt, QuantTable tab,
                                        uint8_t* __restrict__ codes, float* __restrict__ alpha,
                                        float* __restrict__ beta) {
  const int G = d_in / block_in, R = d_out / block_out;
  int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= (int64_t)G * R) return;
  const int rb = (int)(b / G), gb = (int)(b % G);
  const int o0 = rb * block_out, i0 = gb * block_in;
  float mn = load_w(W, (int64_t)o0 * d_in + i0), mx = mn, am = 0.0f;
  for (int o = o0; o < o0 + block_out; ++o)
    for (int i = i0; i < i0 + block_in; ++i) {
      float w = load_w(W, (int64_t)o * d_in + i);
      mn = fminf(mn, w); mx = fmaxf(mx, w); am = fmaxf(am, fabsf(w));
    }
  float a = 0.0f;
  bool degenerate;
  if (qfmt == QBLORA_FMT_CODEBOOK_ABSMAX) {
    degenerate = (am == 0.0f);
    alpha[b] = am;
  } else {
    float d = __fsub_rn(mx, mn);
    a = __fdiv_rn(d, tab.qmax);
    degenerate = (d == 0.0f) || (a == 0.0f);
    alpha[b] = degenerate ? 0.0f : a;
    beta[b] = mn == 0.0f ? 0.0f : mn;   // a zero minimum is stored as +0
  }
  const float inv = __frcp_rn(a);
  for (int o = o0; o < o0 + block_out; ++o)
    for (int i = i0; i < i0 + block_in; i += 2) {
      int c[2];
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        float w = load_w(W, (int64_t)o * d_in + i + e);
        if (qfmt == QBLORA_FMT_CODEBOOK_ABSMAX)
          c[e] = degenerate ? tab.zero_idx : code_of_level(__fdiv_rn(w, am), tab);
        else
          c[e] = degenerate ? 0 : code_of_affine(w, mn, a, inv, tab.qmax);
      }
      codes[(int64_t)o * (d_in / 2) + i / 2] = (uint8_t)(c[0] | (c[1] << 4));
    }
}

}  // namespace

int launch_quantize(const void* W, int w_dtype, int d_out, int d_in, int block_in, int block_out,
                    int qfmt, int bits, const float* level, uint8_t* codes, float* alpha, float* beta,
                    cudaStream_t st) {
  QuantTable tab;
  tab.zero_idx = 0;
  tab.use_lut = 0;
  tab.qmax = (float)((1 << bits) - 1);
  for (int j = 0; j < 15; ++j) tab.mid[j] = 0.0f;
  if (qfmt == QBLORA_FMT_CODEBOOK_ABSMAX) {
    for (int j = 0; j < 15; ++j)
      tab.mid[j] = (float)(((double)level[j] + (double)level[j + 1]) / 2.0);
    for (int j = 1; j < 16; ++j)
      if (fabs((double)level[j]) < fabs((double)level[tab.zero_idx])) tab.zero_idx = j;
    // bucket table: every pair of adjacent midpoints farther apart than one widened bucket
    tab.use_lut = 1;
    for (int j = 0; j + 1 < 15; ++j)
      if (!(tab.mid[j + 1] - tab.mid[j] > 1.0f / LUT_SCALE + 4.0f * LUT_MARGIN)) tab.use_lut = 0;
    // (midpoints lie strictly inside (-1, 1): the levels are ascending and the caller's table spans [-1, 1])
    for (int j = 0; j < 15; ++j) if (!(fabsf(tab.mid[j]) < 1.0f)) tab.use_lut = 0;
  }
  if (block_in == 64 && block_out == 1) {
    int64_t nblocks = (int64_t)d_out * (d_in / 64);
    int64_t ctas = ((nblocks + 3) / 4 + 7) / 8;      // four blocks per warp and step, eight warps per CTA
    int grid = (int)(ctas < 148 * 16 ? ctas : 148 * 16);
    if (grid < 1) grid = 1;
    if (w_dtype == QBLORA_F32)
      quantize_b64_kernel<float><<<grid, 256, 0, st>>>((const float*)W, nblocks, qfmt, tab, codes, alpha, beta);
    else
      quantize_b64_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)W, nblocks, qfmt, tab, codes, alpha, beta);
  } else {
    if (block_in % 2) return QBLORA_ERR_UNSUPPORTED;
    int64_t nblocks = (int64_t)(d_out / block_out) * (d_in / block_in);
    int grid = (int)((nblocks + 127) / 128);
    if (w_dtype == QBLORA_F32)
      quantize_generic_kernel<float><<<grid, 128, 0, st>>>((const float*)W, d_out, d_in, block_in, block_out, qfmt, tab, codes, alpha, beta);
    else
      quantize_generic_kernel<__nv_bfloat16><<<grid, 128, 0, st>>>((const __nv_bfloat16*)W, d_out, d_in, block_in, block_out, qfmt, tab, codes, alpha, beta);
  }
  count_launch();
  QB_CUDA(cudaGetLastError());
  return QBLORA_OK;
}

}  // namespace qb
