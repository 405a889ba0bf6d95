// Small dense bf16 GEMM on tcgen05 / TMEM / TMA (see tc_small.cuh).  One 128 x bn output tile per
// CTA (bn <= 256), cta_group::1, four TMA-fed stages; warp 0 TMA producer, warp 1 MMA issuer and
// TMEM owner, warps 2-5 epilogue.  Operands may be K-contiguous (K-major) or MN-contiguous
// (MN-major); both are staged in the canonical 128-byte-swizzled layout by TMA.
#include <atomic>

#include "tc_ptx.cuh"
#include "tc_small.cuh"

namespace qb {
using namespace ptx;
namespace {

constexpr int SG_BM = 128, SG_BK = 64, SG_STAGES = 4;
constexpr int SG_A_BYTES = SG_BM * SG_BK * 2;   // 16 KB
constexpr int SG_B_BYTES = 256 * SG_BK * 2;     // 32 KB (bn = 256)
constexpr int SG_THREADS = 192;
constexpr int SG_SMEM = SG_STAGES * (SG_A_BYTES + SG_B_BYTES) + 256 + 1024;
// 193 KB: a CTA of this kernel never shares an SM with a CTA of the fused contraction (218 KB).  That matters for
// tensor memory: this kernel allocates 256 columns, the contraction all 512, and the contraction may be launched
// as this kernel's programmatic dependent and wait for its completion -- on a shared SM either could wait for
// columns the other holds.  Keep the sum of the two footprints above the SM's shared memory.
static_assert(SG_SMEM > 16 * 1024, "see the note on tensor memory above");
constexpr int SG_MAX_SEG = 3;

struct SgMaps {
  CUtensorMap a[SG_MAX_SEG], b[SG_MAX_SEG];
};
struct SgParams {
  int M, N, bn, nseg;
  int kblocks[SG_MAX_SEG];
  int splits;               // gridDim.z; each z takes a contiguous share of every segment's K-blocks
  int64_t split_stride;     // elements between the fp32 partial outputs of consecutive z
  int a_kmajor, b_kmajor;
  SgOut out;
  int* status;
  long long wait_limit;     // cycles after which a device-side wait gives up
};

__global__ void __launch_bounds__(SG_THREADS, 1)
small_gemm_kernel(const __grid_constant__ SgMaps maps, const __grid_constant__ SgParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  const uint32_t sA = base, sB = sA + SG_STAGES * SG_A_BYTES, bars = sB + SG_STAGES * SG_B_BYTES;
  auto full = [&](int s) { return bars + 8u * s; };
  auto empty = [&](int s) { return bars + 8u * (SG_STAGES + s); };
  const uint32_t accfull = bars + 8u * (2 * SG_STAGES);
  const uint32_t tmem_slot = bars + 8u * (2 * SG_STAGES + 1);
  volatile uint32_t* tmem_slot_g = reinterpret_cast<volatile uint32_t*>(smem_raw + (tmem_slot - raw));

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int m0 = blockIdx.y * SG_BM, n0 = blockIdx.x * p.bn;
  // A successor launched as a programmatic dependent (the fused contraction, which needs this product only for
  // its last K-blocks) may start now; it waits for this grid's completion before it reads the result.
  // No effect on ordinary successors.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (tid == 0) {
    for (int s = 0; s < SG_STAGES; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), 1); }
    mbar_init(accfull, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(256) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_g;
  const uint32_t stage_bytes = SG_A_BYTES + (uint32_t)p.bn * SG_BK * 2;

  if (warp == 0) {
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      // launched as a programmatic dependent of the kernel that writes an operand: that kernel is complete after this
      asm volatile("griddepcontrol.wait;" ::: "memory");
      for (int g = 0; g < p.nseg && ok; ++g) {
        const int per = (p.kblocks[g] + p.splits - 1) / p.splits;
        const int kb0 = (int)blockIdx.z * per, kb1 = min(kb0 + per, p.kblocks[g]);
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const int s = it % SG_STAGES;
          const uint32_t ph = (it / SG_STAGES) & 1u;
          if (!mbar_wait(empty(s), ph ^ 1u, p.status, p.wait_limit)) { ok = false; break; }
          mbar_arrive_expect_tx(full(s), stage_bytes);
          const uint32_t a_dst = sA + s * SG_A_BYTES, b_dst = sB + s * SG_B_BYTES;
          if (p.a_kmajor) {
            tma_load_2d(a_dst, &maps.a[g], full(s), kb * SG_BK, m0);
          } else {   // two groups of 64 rows of the output, each [64 k][64 m]
            tma_load_2d(a_dst, &maps.a[g], full(s), m0, kb * SG_BK);
            tma_load_2d(a_dst + 8192, &maps.a[g], full(s), m0 + 64, kb * SG_BK);
          }
          if (p.b_kmajor) {
            tma_load_2d(b_dst, &maps.b[g], full(s), kb * SG_BK, n0);
          } else {
            for (int j = 0; j < p.bn / 64; ++j)
              tma_load_2d(b_dst + j * 8192, &maps.b[g], full(s), n0 + j * 64, kb * SG_BK);
          }
        }
      }
      if (!ok) {
        const uint32_t lo = it > (uint32_t)SG_STAGES ? it - SG_STAGES : 0;
        for (uint32_t j = lo; j < it; ++j) mbar_wait(full(j % SG_STAGES), (j / SG_STAGES) & 1u, p.status, p.wait_limit);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((p.a_kmajor ? 0u : 1u) << 15) |
                             ((p.b_kmajor ? 0u : 1u) << 16) | ((uint32_t)(p.bn >> 3) << 17) |
                             ((uint32_t)(SG_BM >> 4) << 24);
      uint32_t it = 0;
      bool ok = true;
      // launched as a programmatic dependent of the kernel that writes an operand: that kernel is complete after this
      asm volatile("griddepcontrol.wait;" ::: "memory");
      for (int g = 0; g < p.nseg && ok; ++g) {
        const int per = (p.kblocks[g] + p.splits - 1) / p.splits;
        const int kb0 = (int)blockIdx.z * per, kb1 = min(kb0 + per, p.kblocks[g]);
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const int s = it % SG_STAGES;
          const uint32_t ph = (it / SG_STAGES) & 1u;
          if (!mbar_wait(full(s), ph, p.status, p.wait_limit)) { ok = false; break; }
          tc_fence_after();
#pragma unroll
          for (int k = 0; k < SG_BK / 16; ++k) {
            const uint64_t adesc = p.a_kmajor ? smem_desc(sA + s * SG_A_BYTES + k * 32, 16, 1024)
                                              : smem_desc(sA + s * SG_A_BYTES + k * 2048, 8192, 1024);
            const uint64_t bdesc = p.b_kmajor ? smem_desc(sB + s * SG_B_BYTES + k * 32, 16, 1024)
                                              : smem_desc(sB + s * SG_B_BYTES + k * 2048, 8192, 1024);
            tc_mma(tmem_base, adesc, bdesc, idesc, it != 0 || k != 0 ? 1u : 0u);
          }
          tc_commit(empty(s));
        }
      }
      if (ok) tc_commit(accfull);   // (a share with no K-blocks still arrives: nothing was issued)
    }
  } else {
    // epilogue: thread = output row; 32 columns per TMEM load
    const int q = warp & 3;
    const int m = m0 + q * 32 + lane;
    int my_kblocks = 0;   // a share of the split that received no K-block contributes zeros
    for (int g = 0; g < p.nseg; ++g) {
      const int per = (p.kblocks[g] + p.splits - 1) / p.splits;
      const int kb0 = (int)blockIdx.z * per, kb1 = min(kb0 + per, p.kblocks[g]);
      my_kblocks += max(kb1 - kb0, 0);
    }
    if (mbar_wait(accfull, 0, p.status, p.wait_limit)) {
      tc_fence_after();
      for (int c = 0; c < p.bn / 32; ++c) {
        const int nb = n0 + c * 32;
        if (nb >= p.N) break;
        uint32_t v[32];
        tc_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(c * 32), v);
        if (my_kblocks == 0) {
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = 0u;
        }
        if (m >= p.M) continue;
        const SgOut& o = p.out;
        if (o.f32) {
          float* dst = o.f32 + (int64_t)blockIdx.z * p.split_stride + (int64_t)m * o.ld32 + nb;
          if ((o.ld32 & 3) == 0 && nb + 32 <= p.N) {
#pragma unroll
            for (int j = 0; j < 32; j += 4)
              *reinterpret_cast<float4*>(dst + j) = make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]),
                                                                __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) if (nb + j < p.N) dst[j] = __uint_as_float(v[j]);
          }
        }
        if (o.hi || o.lo || o.scaled) {
          const int64_t row = (int64_t)m * o.ld16 + nb;
          if ((o.ld16 & 7) == 0 && nb + 32 <= p.N) {   // 16-byte stores of eight bf16
#pragma unroll
            for (int j = 0; j < 32; j += 8) {
              uint32_t h[4], l[4], sc[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const float x0 = __uint_as_float(v[j + 2 * e]), x1 = __uint_as_float(v[j + 2 * e + 1]);
                const __nv_bfloat162 hh = __floats2bfloat162_rn(x0, x1);
                h[e] = *reinterpret_cast<const uint32_t*>(&hh);
                const __nv_bfloat162 ll = __floats2bfloat162_rn(x0 - __low2float(hh), x1 - __high2float(hh));
                l[e] = *reinterpret_cast<const uint32_t*>(&ll);
                const __nv_bfloat162 ss = o.divide ? __floats2bfloat162_rn(__fdiv_rn(x0, o.scale), __fdiv_rn(x1, o.scale))
                                                   : __floats2bfloat162_rn(x0 * o.scale, x1 * o.scale);
                sc[e] = *reinterpret_cast<const uint32_t*>(&ss);
              }
              if (o.hi) *reinterpret_cast<uint4*>(o.hi + row + j) = make_uint4(h[0], h[1], h[2], h[3]);
              if (o.lo) *reinterpret_cast<uint4*>(o.lo + row + j) = make_uint4(l[0], l[1], l[2], l[3]);
              if (o.scaled) *reinterpret_cast<uint4*>(o.scaled + row + j) = make_uint4(sc[0], sc[1], sc[2], sc[3]);
            }
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              if (nb + j >= p.N) break;
              const float x = __uint_as_float(v[j]);
              const __nv_bfloat16 h = __float2bfloat16_rn(x);
              if (o.hi) o.hi[row + j] = h;
              if (o.lo) o.lo[row + j] = __float2bfloat16_rn(x - __bfloat162float(h));
              if (o.scaled) o.scaled[row + j] = __float2bfloat16_rn(o.divide ? __fdiv_rn(x, o.scale) : x * o.scale);
            }
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(256) : "memory");
  }
}

// out[m][n] = sum over z (in order) of part[z][m][n]
__global__ void reduce_splits_kernel(const float* __restrict__ part, int splits, int64_t MN, int N, float* __restrict__ out,
                                     int64_t ld) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= MN) return;
  float acc = 0.0f;
  for (int z = 0; z < splits; ++z) acc += part[(int64_t)z * MN + idx];
  out[(idx / N) * ld + idx % N] = acc;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess) return nullptr;
    if (q != cudaDriverEntryPointSuccess) return nullptr;
    return reinterpret_cast<EncodeTiledFn>(f);
  }();
  return fn;
}

int operand_map(CUtensorMap* tm, const SgOperand& op, int MN, int K, int box_rows_kmajor) {
  if (op.k_contig)   // rows = mn, inner = k
    return make_tensor_map_2d(tm, false, op.ptr, (uint64_t)K, (uint64_t)MN, (uint64_t)op.ld * 2, SG_BK, box_rows_kmajor, true);
  // rows = k, inner = mn: boxes of 64 mn-elements x 64 k-rows
  return make_tensor_map_2d(tm, false, op.ptr, (uint64_t)MN, (uint64_t)K, (uint64_t)op.ld * 2, 64, SG_BK, true);
}

}  // namespace

int make_tensor_map_2d(void* tm, bool is_u8, const void* ptr, uint64_t inner, uint64_t rows, uint64_t pitch_bytes,
                       uint32_t box_inner, uint32_t box_rows, bool swizzle128) {
  return make_tensor_map_2d_typed(tm, is_u8 ? TM_U8 : TM_BF16, ptr, inner, rows, pitch_bytes, box_inner, box_rows, swizzle128 ? 128 : 0);
}

int make_tensor_map_2d_typed(void* tm, int elem, const void* ptr, uint64_t inner, uint64_t rows, uint64_t pitch_bytes,
                             uint32_t box_inner, uint32_t box_rows, int swizzle_bytes) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return QBLORA_ERR_CUDA;
  cuuint64_t dims[2] = {inner, rows};
  cuuint64_t strides[1] = {pitch_bytes};
  cuuint32_t box[2] = {box_inner, box_rows};
  cuuint32_t estr[2] = {1, 1};
  const CUtensorMapDataType dt = elem == TM_U8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8
                                 : elem == TM_U32 ? CU_TENSOR_MAP_DATA_TYPE_UINT32
                                 : elem == TM_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
  CUresult r = fn(static_cast<CUtensorMap*>(tm), dt,
                  2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                  : swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? QBLORA_OK : QBLORA_ERR_CUDA;
}

int small_gemm_splits(int M, int N, int K) {
  const int n64 = (N + 63) / 64 * 64;
  const int bn = n64 < 256 ? n64 : 256;
  const int tiles = ((N + bn - 1) / bn) * ((M + SG_BM - 1) / SG_BM);
  const int kb = (K + SG_BK - 1) / SG_BK;
  int want = 148 / tiles;
  // at most 16 shares: the gradient products run beside the dX contraction on the few SMs its last wave leaves
  // free, where 32 shares of one K-block each took several rounds (C2 backward call 128 -> 115 us; 8 shares: 113)
  if (want > 16) want = 16;
  if (want > kb) want = kb;
  if (want < 1) want = 1;
  const int per = (kb + want - 1) / want;
  return (kb + per - 1) / per;   // every share owns at least one K-block
}

int small_gemm(int M, int N, const SgSegment* segs, int nseg, const SgOut& out, int* status, cudaStream_t st,
               float* partial, bool dependent, bool wide_tiles) {
  if (nseg < 1 || nseg > SG_MAX_SEG || M < 1 || N < 1) return QBLORA_ERR_INVALID_ARG;
  static std::atomic<bool> attr_set[64];   // per device; atomic: concurrent host threads at worst set it twice
  int dev = 0;
  QB_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return QBLORA_ERR_UNSUPPORTED;
  if (!attr_set[dev].load(std::memory_order_acquire)) {
    QB_CUDA(cudaFuncSetAttribute(small_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SG_SMEM));
    attr_set[dev].store(true, std::memory_order_release);
  }
  SgMaps maps;
  SgParams p{};
  p.M = M; p.N = N; p.nseg = nseg;
  const int n64 = (N + 63) / 64 * 64;
  p.bn = n64 < 256 ? n64 : 256;
  // few row tiles and no split: narrower column tiles put more CTAs to work (the kernel is latency-bound)
  while (!wide_tiles && !partial && p.bn > 64 && ((N + p.bn - 1) / p.bn) * ((M + SG_BM - 1) / SG_BM) < 96 && (p.bn / 2) % 64 == 0) p.bn /= 2;
  p.a_kmajor = segs[0].a.k_contig ? 1 : 0;
  p.b_kmajor = segs[0].b.k_contig ? 1 : 0;
  for (int g = 0; g < nseg; ++g) {
    if ((segs[g].a.k_contig ? 1 : 0) != p.a_kmajor || (segs[g].b.k_contig ? 1 : 0) != p.b_kmajor) return QBLORA_ERR_INVALID_ARG;
    if (segs[g].K < 1 || (segs[g].a.ld & 7) || (segs[g].b.ld & 7) || !aligned16(segs[g].a.ptr) || !aligned16(segs[g].b.ptr))
      return QBLORA_ERR_INVALID_ARG;
    p.kblocks[g] = (segs[g].K + SG_BK - 1) / SG_BK;
    int rc = operand_map(&maps.a[g], segs[g].a, M, segs[g].K, SG_BM);
    if (rc) return rc;
    rc = operand_map(&maps.b[g], segs[g].b, N, segs[g].K, p.bn);
    if (rc) return rc;
  }
  for (int g = nseg; g < SG_MAX_SEG; ++g) { maps.a[g] = maps.a[0]; maps.b[g] = maps.b[0]; p.kblocks[g] = 0; }
  p.out = out;
  p.status = status;
  p.wait_limit = wait_limit_cycles();
  p.splits = 1;
  p.split_stride = 0;
  if (partial) {   // split the contraction; only the fp32 output is supported in this mode
    if (!out.f32 || out.hi || out.lo || out.scaled) return QBLORA_ERR_INVALID_ARG;
    p.splits = small_gemm_splits(M, N, segs[0].K);
    if (p.splits > 1) {
      p.out.f32 = partial;
      p.out.ld32 = N;
      p.split_stride = (int64_t)M * N;
    }
  }
  dim3 grid((unsigned)((N + p.bn - 1) / p.bn), (unsigned)((M + SG_BM - 1) / SG_BM), (unsigned)p.splits);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = dim3(SG_THREADS); cfg.dynamicSmemBytes = SG_SMEM; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = dependent ? 1 : 0;
  QB_CUDA(cudaLaunchKernelEx(&cfg, small_gemm_kernel, maps, p));
  count_launch();
  QB_CUDA(cudaGetLastError());
  if (p.splits > 1) {
    const int64_t MN = (int64_t)M * N;
    reduce_splits_kernel<<<(unsigned)((MN + 255) / 256), 256, 0, st>>>(partial, p.splits, MN, N, out.f32, out.ld32);
    count_launch();
    QB_CUDA(cudaGetLastError());
  }
  return QBLORA_OK;
}

}  // namespace qb
