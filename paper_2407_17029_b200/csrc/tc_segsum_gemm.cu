// The adapter's first product with its compression fused in front (Sec. 3.2), on tcgen05 / TMEM / TMA:
//
//   c[t][w]   = f( sum of lam consecutive src[t][lam w ..] )      f = / lam (AvgPool of the input, forward)
//                                                                 or * scale (adjoint of repeat_interleave, backward)
//   out[t][n] = sum_w c[t][w] * M(n, w)                           M = A^T (u = x' A) or B (du = dv B^T)
//
// One pass over src: eight warps stream a 64-token slab of it, form c in fp32, split it into a bf16 hi + lo pair
// (16 significant bits) and write the pair straight into the MMA's token-side operand tiles in shared memory
// (and, if asked, to global memory for the gradient products that need c itself); the adapter matrix comes by
// TMA; hi and lo share each of its tiles.  The rank index is the MMA's M (one or two 128-row halves, each with
// its own 64-column accumulator), the 64 tokens its N, so a launch has T / 64 CTAs streaming src at once.
// Every mbarrier wait is bounded (status word QBLORA_ERR_TIMEOUT).
#include <atomic>

#include "tc_ptx.cuh"
#include "tc_small.cuh"

namespace qb {
using namespace ptx;
namespace {

constexpr int FG_BT = 64;                        // tokens per CTA
constexpr int FG_BK = 64;                        // compressed columns per stage
constexpr int FG_STAGES = 4;
constexpr int FG_HALF_BYTES = 128 * FG_BK * 2;   // 16 KB: 128 rows of the adapter matrix
constexpr int FG_A_BYTES = 2 * FG_HALF_BYTES;
constexpr int FG_C_BYTES = FG_BT * FG_BK * 2;    // 8 KB: compressed activation, hi or lo
constexpr int FG_WARPS = 8;                      // compression (then epilogue) warps
constexpr int FG_THREADS = (2 + FG_WARPS) * 32;
constexpr int FG_SMEM = FG_STAGES * (FG_A_BYTES + 2 * FG_C_BYTES) + 256 + 1024;
// As for the small product (tc_small_gemm.cu): large enough that a CTA of this kernel never shares an SM with a
// CTA of the fused contraction, which may be its programmatic dependent and holds all of tensor memory.
static_assert(FG_SMEM > 16 * 1024 && FG_SMEM <= 227 * 1024, "shared memory of the fused compression + product");

struct FgParams {
  const __nv_bfloat16* src;
  int64_t T;
  int width, W;             // src row length; compressed columns W = width / lam
  int divide; float scale;  // c = sum / lam, or c = scale * sum
  int N;                    // rows of the adapter matrix as the MMA sees it (the rank), <= 256
  int a_kmajor;             // M(n, w) at ptr[n * ld + w] (true) or ptr[w * ld + n]
  int kblocks;
  __nv_bfloat16 *c_hi, *c_lo; int64_t ld_c;   // optional copy of c
  SgOut out;                // hi / lo / scaled, [T][ld16]
  int* status;
  long long wait_limit;
};

template <int LAM>
__global__ void __launch_bounds__(FG_THREADS, 1)
segsum_gemm_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ FgParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  const uint32_t sA = base, sC = sA + FG_STAGES * FG_A_BYTES, bars = sC + FG_STAGES * 2 * FG_C_BYTES;
  auto full = [&](int s) { return bars + 8u * s; };                     // adapter-matrix tiles landed
  auto ready = [&](int s) { return bars + 8u * (FG_STAGES + s); };      // compressed tiles written
  auto empty = [&](int s) { return bars + 8u * (2 * FG_STAGES + s); };  // the stage's MMAs are done
  const uint32_t accfull = bars + 8u * (3 * FG_STAGES);
  const uint32_t tmem_slot = bars + 8u * (3 * FG_STAGES + 1);
  volatile uint32_t* tmem_slot_g = reinterpret_cast<volatile uint32_t*>(smem_raw + (tmem_slot - raw));

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int64_t t0 = (int64_t)blockIdx.x * FG_BT;
  const int halves = p.N > 128 ? 2 : 1;
  // The fused contraction launched behind this kernel as its programmatic dependent needs the result only for the
  // last K-blocks of a tile; it may set up and start now and waits for this grid's completion before it reads.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (tid == 0) {
    for (int s = 0; s < FG_STAGES; ++s) { mbar_init(full(s), 1); mbar_init(ready(s), FG_WARPS * 32); mbar_init(empty(s), 1); }
    mbar_init(accfull, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(128) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_g;

  if (warp == 0) {
    if (lane == 0) {   // ---------------------------------------------------- TMA producer: adapter-matrix tiles
      bool ok = true;
      int it = 0;
      for (int kb = 0; kb < p.kblocks; ++kb, ++it) {
        const int s = it % FG_STAGES;
        const uint32_t ph = (it / FG_STAGES) & 1u;
        if (!mbar_wait(empty(s), ph ^ 1u, p.status, p.wait_limit)) { ok = false; break; }
        mbar_arrive_expect_tx(full(s), (uint32_t)halves * FG_HALF_BYTES);
        const uint32_t a_dst = sA + s * FG_A_BYTES;
        for (int h = 0; h < halves; ++h) {
          if (p.a_kmajor) {
            tma_load_2d(a_dst + h * FG_HALF_BYTES, &tm_a, full(s), kb * FG_BK, h * 128);
          } else {   // two groups of 64 rank indices, each [64 w][64 n]
            tma_load_2d(a_dst + h * FG_HALF_BYTES, &tm_a, full(s), h * 128, kb * FG_BK);
            tma_load_2d(a_dst + h * FG_HALF_BYTES + 8192, &tm_a, full(s), h * 128 + 64, kb * FG_BK);
          }
        }
      }
      if (!ok) {   // give copies already in flight a bounded chance to land before the CTA exits
        const int lo = it > FG_STAGES ? it - FG_STAGES : 0;
        for (int j = lo; j < it; ++j) mbar_wait(full(j % FG_STAGES), (uint32_t)(j / FG_STAGES) & 1u, p.status, p.wait_limit);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {   // ---------------------------------------------------- MMA issuer
      // D fp32, A / B bf16, B (tokens) K-major, A K- or MN-major, M = 128, N = 64
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((p.a_kmajor ? 0u : 1u) << 15) |
                             ((uint32_t)(FG_BT >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
      bool ok = true;
      for (int kb = 0; kb < p.kblocks; ++kb) {
        const int s = kb % FG_STAGES;
        const uint32_t ph = (uint32_t)(kb / FG_STAGES) & 1u;
        if (!mbar_wait(full(s), ph, p.status, p.wait_limit) || !mbar_wait(ready(s), ph, p.status, p.wait_limit)) { ok = false; break; }
        tc_fence_after();
        for (int h = 0; h < halves; ++h) {
          const uint32_t a_tile = sA + s * FG_A_BYTES + h * FG_HALF_BYTES;
#pragma unroll
          for (int seg = 0; seg < 2; ++seg) {   // hi, lo: the same adapter-matrix tile
            const uint32_t c_tile = sC + s * 2 * FG_C_BYTES + seg * FG_C_BYTES;
#pragma unroll
            for (int k = 0; k < FG_BK / 16; ++k) {
              const uint64_t adesc = p.a_kmajor ? smem_desc(a_tile + k * 32, 16, 1024) : smem_desc(a_tile + k * 2048, 8192, 1024);
              const uint64_t bdesc = smem_desc(c_tile + k * 32, 16, 1024);
              tc_mma(tmem_base + (uint32_t)(h * FG_BT), adesc, bdesc, idesc, (kb | seg | k) != 0 ? 1u : 0u);
            }
          }
        }
        tc_commit(empty(s));
      }
      if (ok) tc_commit(accfull);
    }
  } else {
    // -------------------------------------------------------------------------- compression warps, then epilogue
    // Warp wv takes tokens 8 wv .. 8 wv + 7 of the slab.  Per token and K-block: 64 windows = 64 LAM elements =
    // 8 LAM 16-byte chunks, LAM / 4 per lane (consecutive lanes read consecutive chunks); a window is LAM / 8
    // consecutive lanes, reduced with shuffles.
    constexpr int L = LAM / 4;        // loads per lane, token and K-block
    constexpr int G = LAM / 8;        // lanes per window
    const int wv = warp - 2;
    bool ok = true;
    for (int kb = 0; kb < p.kblocks && ok; ++kb) {
      const int s = kb % FG_STAGES;
      const uint32_t ph = (uint32_t)(kb / FG_STAGES) & 1u;
      const uint32_t c_hi_tile = sC + s * 2 * FG_C_BYTES, c_lo_tile = c_hi_tile + FG_C_BYTES;
      bool slot_free = false;
#pragma unroll 1
      for (int b = 0; b < L && ok; ++b) {       // batches of eight loads in flight per lane
        uint4 v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int qi = b * 8 + i, tl = qi / L, j = qi % L;
          const int64_t t = t0 + wv * 8 + tl;
          const int ch = j * 32 + lane;
          const int64_t col = (int64_t)kb * FG_BK * LAM + ch * 8;
          v[i] = make_uint4(0, 0, 0, 0);
          if (t < p.T && col < p.width) v[i] = __ldg(reinterpret_cast<const uint4*>(p.src + t * p.width + col));
        }
        if (!slot_free) {   // the loads above are in flight while this waits for the stage
          // (one outcome for the whole warp: the shuffles below need all 32 lanes)
          if (!__all_sync(0xffffffffu, mbar_wait(empty(s), ph ^ 1u, p.status, p.wait_limit))) { ok = false; break; }
          slot_free = true;
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int qi = b * 8 + i, tl = qi / L, j = qi % L;
          const int row = wv * 8 + tl;                 // token within the slab
          const int64_t t = t0 + row;
          const uint32_t w4[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
          float e[8];
#pragma unroll
          for (int k = 0; k < 4; ++k) { e[2 * k] = __uint_as_float(w4[k] << 16); e[2 * k + 1] = __uint_as_float(w4[k] & 0xffff0000u); }
          float sacc = ((e[0] + e[1]) + (e[2] + e[3])) + ((e[4] + e[5]) + (e[6] + e[7]));
#pragma unroll
          for (int off = 1; off < G; off <<= 1) sacc += __shfl_xor_sync(0xffffffffu, sacc, off);
          if ((lane & (G - 1)) == 0) {
            const int wl = (j * 32 + lane) / G;        // window within the K-block
            const float c = p.divide ? __fdiv_rn(sacc, (float)LAM) : p.scale * sacc;
            const __nv_bfloat16 hi = __float2bfloat16_rn(c);
            const __nv_bfloat16 lo = __float2bfloat16_rn(c - __bfloat162float(hi));
            // K-major tile [64 tokens][64 w], 128-byte rows, 16-byte chunks XOR-swizzled with the row
            const uint32_t off = (uint32_t)row * 128u + ((((uint32_t)wl >> 3) ^ ((uint32_t)row & 7u)) << 4) + ((uint32_t)wl & 7u) * 2u;
            asm volatile("st.shared.b16 [%0], %1;" ::"r"(c_hi_tile + off), "h"(__bfloat16_as_ushort(hi)) : "memory");
            asm volatile("st.shared.b16 [%0], %1;" ::"r"(c_lo_tile + off), "h"(__bfloat16_as_ushort(lo)) : "memory");
            const int w = kb * FG_BK + wl;
            if (p.c_hi && t < p.T && w < p.W) {
              p.c_hi[t * p.ld_c + w] = hi;
              p.c_lo[t * p.ld_c + w] = lo;
            }
          }
        }
      }
      if (!ok) break;
      fence_async_proxy();   // generic-proxy stores -> visible to the tensor core's async proxy
      mbar_arrive(ready(s));
    }
    // epilogue: warp group h = wv / 4 drains accumulator half h; thread = rank index, registers = tokens
    const int q = warp & 3, h = wv >> 2;
    if (ok && h < halves && __all_sync(0xffffffffu, mbar_wait(accfull, 0, p.status, p.wait_limit))) {
      tc_fence_after();
      const int n = h * 128 + q * 32 + lane;
      const SgOut& o = p.out;
      for (int c2 = 0; c2 < FG_BT / 32; ++c2) {
        uint32_t v[32];
        tc_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(h * FG_BT + c2 * 32), v);
        if (n >= p.N) continue;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const int64_t t = t0 + c2 * 32 + j;
          if (t >= p.T) break;
          const float x = __uint_as_float(v[j]);
          const __nv_bfloat16 hi = __float2bfloat16_rn(x);
          const int64_t idx = t * o.ld16 + n;
          if (o.hi) o.hi[idx] = hi;
          if (o.lo) o.lo[idx] = __float2bfloat16_rn(x - __bfloat162float(hi));
          if (o.scaled) o.scaled[idx] = __float2bfloat16_rn(o.divide ? __fdiv_rn(x, o.scale) : x * o.scale);
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(128) : "memory");
  }
}

template <int LAM>
int launch_fg(const CUtensorMap& tm, const FgParams& p, int dev, int slot, cudaStream_t st) {
  static std::atomic<bool> attr_set[64][4];   // per device and instantiation; atomic: host threads at worst set it twice
  if (!attr_set[dev][slot].load(std::memory_order_acquire)) {
    QB_CUDA(cudaFuncSetAttribute(segsum_gemm_kernel<LAM>, cudaFuncAttributeMaxDynamicSharedMemorySize, FG_SMEM));
    attr_set[dev][slot].store(true, std::memory_order_release);
  }
  segsum_gemm_kernel<LAM><<<(unsigned)((p.T + FG_BT - 1) / FG_BT), FG_THREADS, FG_SMEM, st>>>(tm, p);
  count_launch();
  QB_CUDA(cudaGetLastError());
  return QBLORA_OK;
}

}  // namespace

bool segsum_gemm_ok(int width, int lam, int N) {
  return (lam == 8 || lam == 16 || lam == 32 || lam == 64) && width % lam == 0 && N >= 8 && N <= 256 && N % 8 == 0;
}

int segsum_gemm(const SegGemm& a, int* status, cudaStream_t st) {
  if (!segsum_gemm_ok(a.width, a.lam, a.N) || a.T < 1 || !a.src || !aligned16(a.src) || !aligned16(a.m.ptr) || (a.m.ld & 7) ||
      a.out.ld16 < a.N || (a.c_hi != nullptr) != (a.c_lo != nullptr))
    return QBLORA_ERR_INVALID_ARG;
  int dev = 0;
  QB_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return QBLORA_ERR_UNSUPPORTED;
  FgParams p{};
  p.src = a.src; p.T = a.T; p.width = a.width; p.W = a.width / a.lam;
  p.divide = a.divide ? 1 : 0; p.scale = a.scale;
  p.N = a.N; p.a_kmajor = a.m.k_contig ? 1 : 0;
  p.kblocks = (p.W + FG_BK - 1) / FG_BK;
  p.c_hi = a.c_hi; p.c_lo = a.c_lo; p.ld_c = a.ld_c;
  p.out = a.out;
  p.status = status;
  p.wait_limit = wait_limit_cycles();
  CUtensorMap tm;
  int rc = a.m.k_contig
      ? make_tensor_map_2d(&tm, false, a.m.ptr, (uint64_t)p.W, (uint64_t)a.N, (uint64_t)a.m.ld * 2, FG_BK, 128, true)
      : make_tensor_map_2d(&tm, false, a.m.ptr, (uint64_t)a.N, (uint64_t)p.W, (uint64_t)a.m.ld * 2, 64, FG_BK, true);
  if (rc) return rc;
  switch (a.lam) {
    case 8: return launch_fg<8>(tm, p, dev, 0, st);
    case 16: return launch_fg<16>(tm, p, dev, 1, st);
    case 32: return launch_fg<32>(tm, p, dev, 2, st);
    default: return launch_fg<64>(tm, p, dev, 3, st);
  }
}

}  // namespace qb
