// Tensor-core path of the adapted quantized linear for sm_100a: a persistent, warp-specialised
// tcgen05 GEMM whose weight operand is unpacked from 4-bit codes and block-dequantized inside the
// mainloop (Sec. 3.1 / Algorithm 1's "dequantize then matmul", fused), with the adapter branch of
// Sec. 3.2 appended as extra K-blocks of the same accumulation:
//
//   forward : Y^T[o][t]  = sum_i w~[o][i] X[t][i]   + sum_k B[k][o/l2]      (s u)[t][k]
//   backward: dX^T[i][t] = sum_o w~[o][i] dY[t][o]  + sum_k A[i/l1][k]      (du/l1)[t][k]
//
// Two CTAs on the two SMs of a TPC form a cluster and issue tcgen05.mma with cta_group::2: the
// pair computes a 256 (weight rows) x 256 (tokens) tile.  Each CTA dequantizes its own 128 weight
// rows into shared memory (the MMA's A operand, canonical 128-byte-swizzled layout: K-major in the
// forward, MN-major in the backward, so the same [o][i]-packed codes serve both) and stages half of
// the token tile by TMA (the B operand; no multicast), which halves the shared-memory traffic per
// MMA cycle compared with a single-CTA tile -- the resource that bounds this kernel.  Accumulators
// live in TMEM (2 x 256 columns, double-buffered so the epilogue of one tile overlaps the mainloop
// of the next).
//
// Warp roles (448 threads per CTA): warp 0 TMA producer; warp 1 MMA issuer (leader CTA only) and
// TMEM owner; warps 2-9 two dequant groups taking alternate K-blocks (those of the other CTA report
// each finished stage to the leader's barrier); warps 10-13 epilogue.  Every mbarrier wait is bounded;
// on expiry the kernel stores QBLORA_ERR_TIMEOUT in the workspace status word and every role
// leaves its loop.
#include <cuda.h>

#include "common.cuh"
#include "simt_gemm.cuh"

namespace qb {
using namespace simt;
namespace {

constexpr int BM = 128;        // rows of the weight-side operand per CTA (256 per CTA pair)
constexpr int BN = 256;        // tokens per tile (each CTA of the pair stages 128 of them)
constexpr int BN_HALF = BN / 2;
constexpr int BK = 64;         // contraction elements per stage = one quantization block
constexpr int STAGES = 6;
constexpr int A_BYTES = BM * BK * 2;        // 16 KB dequantized weight tile
constexpr int B_BYTES = BN_HALF * BK * 2;   // 16 KB: this CTA's half of the token tile
constexpr int P_BYTES = BM * BK / 2;        // 4 KB packed codes
constexpr int NUM_THREADS = 448;            // 14 warps, see roles above
constexpr int SMEM_BYTES = STAGES * (A_BYTES + B_BYTES + P_BYTES) + 512 + 1024;
constexpr long long WAIT_LIMIT_CYCLES = 2000000000LL;  // ~1 s: far beyond any legitimate wait

struct TcParams {
  int M;                    // output rows of the tile grid: d_out (forward) / d_in (backward)
  int kb_base, kb_extra;    // K-blocks from the quantized weight / from the adapter
  int T;
  int m_tiles, n_tiles;     // tiles of 256 rows x 256 tokens (one per CTA pair)
  int d_in, d_out, G;
  const float* alpha;
  const float* beta;
  float level[16];
  const __nv_bfloat16* ex;  // forward: B^T [Q][r_pad]; backward: A^T [r_pad][P]
  int ex_ld, lam;           // leading dimension of ex; forward lambda_out, backward lambda_in
  void* out;                // forward Y [T][d_out]; backward dX [T][d_in]
  int out_dtype;
  int* status;
};

// ------------------------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// arrive on a barrier of another CTA of the cluster (address from map_to_cta)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: false (and the status word set) if the phase did not complete in time.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > WAIT_LIMIT_CYCLES) {
      atomicExch(status, (int)QBLORA_ERR_TIMEOUT);
      return false;
    }
  }
  return true;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// completion of all prior MMAs of the pair -> one arrival on the barrier at this offset in both CTAs
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(bar), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle.  `lbo`/`sbo` in bytes.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo >> 4) & 0x3FFFu) << 32;
  d |= (uint64_t)1 << 46;   // descriptor version (sm_100)
  d |= (uint64_t)2 << 61;   // 128-byte swizzle
  return d;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
// Eight 4-bit codes (one 32-bit word, code e in bits 4e..4e+3) -> eight bf16 values alpha*level+beta.
// `tabv` holds level[lane & 15] in every lane, so a warp shuffle indexed by the raw shifted word
// (the source lane is taken modulo 32, and lanes 16-31 mirror lanes 0-15) is the table lookup.
// The product is formed in fp32 and rounded once to bf16.
__device__ __forceinline__ void dequant_word(uint32_t w, float tabv, float alpha, float beta, uint32_t (&o)[4]) {
  float v[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    const float lv = __shfl_sync(0xffffffffu, tabv, (int)(w >> (4 * e)));
    v[e] = fmaf(alpha, lv, beta);
  }
#pragma unroll
  for (int e = 0; e < 4; ++e) o[e] = pack_bf16x2(v[2 * e], v[2 * e + 1]);
}

template <int MODE>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
tc_dq_gemm_kernel(const __grid_constant__ CUtensorMap tm_b, const __grid_constant__ CUtensorMap tm_bx,
                  const __grid_constant__ CUtensorMap tm_p, const __grid_constant__ TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  const uint32_t sA = base, sB = sA + STAGES * A_BYTES, sP = sB + STAGES * B_BYTES;
  const uint32_t bars = sP + STAGES * P_BYTES;
  const uint8_t* gP = smem_raw + (sP - raw);
  auto full = [&](int s) { return bars + 8u * s; };                      // TMA bytes landed (local)
  auto aready = [&](int s) { return bars + 8u * (STAGES + s); };          // dequantized tile written (local)
  auto empty = [&](int s) { return bars + 8u * (2 * STAGES + s); };       // MMAs reading the stage are done
  auto peer = [&](int s) { return bars + 8u * (3 * STAGES + s); };        // leader only: the other CTA's stage is ready
  auto accfull = [&](int a) { return bars + 8u * (4 * STAGES + a); };
  auto accempty = [&](int a) { return bars + 8u * (4 * STAGES + 2 + a); };  // leader only: both epilogues drained
  const uint32_t tmem_slot = bars + 8u * (4 * STAGES + 4);
  volatile uint32_t* tmem_slot_g = reinterpret_cast<volatile uint32_t*>(smem_raw + (tmem_slot - raw));

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();       // 0 = leader (issues the MMAs of the pair)
  const int num_clusters = gridDim.x >> 1, cluster_id = blockIdx.x >> 1;

  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full(s), 1); mbar_init(aready(s), 128); mbar_init(empty(s), 1); mbar_init(peer(s), 4);
    }
    for (int a = 0; a < 2; ++a) { mbar_init(accfull(a), 1); mbar_init(accempty(a), 256); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {  // the same warp of both CTAs allocates the pair's tensor memory
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();   // barriers of both CTAs are initialised before any remote arrival
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_g;

  const int num_tiles = p.m_tiles * p.n_tiles;
  const int kb_total = p.kb_base + p.kb_extra;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (one lane)
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters) {
        const int m0 = (tile % p.m_tiles) * (2 * BM) + (int)rank * BM;
        const int t0 = (tile / p.m_tiles) * BN + (int)rank * BN_HALF;
        for (int kb = 0; kb < kb_total; ++kb, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1u;
          if (!mbar_wait(empty(s), ph ^ 1u, p.status)) { ok = false; break; }
          if (kb < p.kb_base) {
            mbar_arrive_expect_tx(full(s), B_BYTES + P_BYTES);
            tma_load_2d(sB + s * B_BYTES, &tm_b, full(s), kb * BK, t0);
            if (MODE == 0) {
              tma_load_2d(sP + s * P_BYTES, &tm_p, full(s), kb * (BK / 2), m0);
            } else {   // two boxes of 64 rows x 32 bytes: packed[ng][k][32 B]
              tma_load_2d(sP + s * P_BYTES, &tm_p, full(s), m0 / 2, kb * BK);
              tma_load_2d(sP + s * P_BYTES + P_BYTES / 2, &tm_p, full(s), m0 / 2 + 32, kb * BK);
            }
          } else {
            mbar_arrive_expect_tx(full(s), B_BYTES);
            tma_load_2d(sB + s * B_BYTES, &tm_bx, full(s), (kb - p.kb_base) * BK, t0);
          }
        }
      }
      if (!ok) {  // give copies already in flight a bounded chance to land before the CTA exits
        const uint32_t lo = it > (uint32_t)STAGES ? it - STAGES : 0;
        for (uint32_t j = lo; j < it; ++j) mbar_wait(full(j % STAGES), (j / STAGES) & 1u, p.status);
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      // ------------------------------------------------------------------ MMA issuer (leader CTA, one lane)
      // instruction descriptor: D fp32, A/B bf16, B K-major, A K-major (forward) or MN-major (backward),
      // M = 256 and N = 256 across the CTA pair
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((MODE == 1 ? 1u : 0u) << 15) |
                             ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((2 * BM) >> 4) << 24);
      uint32_t it = 0;
      bool ok = true;
      int lt = 0;
      for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters, ++lt) {
        const int a = lt & 1;
        const uint32_t aph = (lt >> 1) & 1u;
        if (!mbar_wait(accempty(a), aph ^ 1u, p.status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(a * BN);
        for (int kb = 0; kb < kb_total; ++kb, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1u;
          if (!mbar_wait(full(s), ph, p.status) || !mbar_wait(aready(s), ph, p.status) ||
              !mbar_wait(peer(s), ph, p.status)) { ok = false; break; }
          tc_fence_after();
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            uint64_t adesc, bdesc;
            if (MODE == 0) adesc = smem_desc(sA + s * A_BYTES + k * 32, 16, 1024);
            else           adesc = smem_desc(sA + s * A_BYTES + k * 2048, 8192, 1024);
            bdesc = smem_desc(sB + s * B_BYTES + k * 32, 16, 1024);
            tc_mma_pair(d_tmem, adesc, bdesc, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          tc_commit_pair(empty(s));
        }
        if (ok) tc_commit_pair(accfull(a));
      }
    }
  } else if (warp < 10) {
    // ------------------------------------------------------------------ dequant warps: two groups of 128
    // threads; group g fills the stages of K-blocks with (global index & 1) == g.  Thread d owns one
    // quantization block (64 codes, one alpha/beta) of the tile per K-block.
    const int g = (warp - 2) >> 2;
    const int d = tid - 64 - 128 * g;
    const float tabv = p.level[lane & 15];
    const uint32_t leader_peer = map_to_cta(peer(0), 0);
    bool ok = true;
    uint32_t it = 0;
    for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters) {
      const int m0 = (tile % p.m_tiles) * (2 * BM) + (int)rank * BM;
      for (int kb = 0; kb < kb_total; ++kb, ++it) {
        if ((int)(it & 1u) != g) continue;
        const int s = it % STAGES;
        const uint32_t ph = (it / STAGES) & 1u;
        const uint32_t a_stage = sA + s * A_BYTES;
        uint32_t dst, xr;   // address of this thread's 128-byte row (before the chunk XOR) and XOR pattern
        if (MODE == 0) { dst = a_stage + d * 128; xr = d & 7; }
        else           { dst = a_stage + (d >> 6) * 8192 + (d & 63) * 128; xr = d & 7; }
        if (kb < p.kb_base) {
          float al = 0.0f, be = 0.0f;
          if (MODE == 0) {
            const int row = m0 + d;
            if (row < p.d_out) {
              al = __ldg(p.alpha + (int64_t)row * p.G + kb);
              if (p.beta) be = __ldg(p.beta + (int64_t)row * p.G + kb);
            }
          } else {
            const int o = kb * BK + (d & 63), blk = (m0 >> 6) + (d >> 6);
            if (o < p.d_out && blk < p.G) {
              al = __ldg(p.alpha + (int64_t)o * p.G + blk);
              if (p.beta) be = __ldg(p.beta + (int64_t)o * p.G + blk);
            }
          }
          const bool landed = mbar_wait(full(s), ph, p.status) && mbar_wait(empty(s), ph ^ 1u, p.status);
          if (!__all_sync(0xffffffffu, landed)) { ok = false; break; }   // keep the warp together for the shuffles
          const uint8_t* src = gP + s * P_BYTES + d * 32;
          const uint4 q0 = *reinterpret_cast<const uint4*>(src);
          const uint4 q1 = *reinterpret_cast<const uint4*>(src + 16);
          const uint32_t w[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            uint32_t o4[4];
            dequant_word(w[j], tabv, al, be, o4);
            st_shared_v4(dst + (((uint32_t)j ^ xr) << 4), o4[0], o4[1], o4[2], o4[3]);
          }
        } else {
          // adapter K-blocks carry no packed codes, but the other CTA still vouches for its token half
          if (!mbar_wait(empty(s), ph ^ 1u, p.status) || (rank != 0 && !mbar_wait(full(s), ph, p.status))) { ok = false; break; }
          const int kk = (kb - p.kb_base) * BK;
          if (MODE == 0) {
            // A[m = o][k] = B[kk + k][o / lambda_out], read from the transposed copy (row = q)
            const int row = m0 + d;
            if (row < p.d_out) {
              const uint4* src = reinterpret_cast<const uint4*>(p.ex + (int64_t)(row / p.lam) * p.ex_ld + kk);
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                const uint4 v = __ldg(src + j);
                st_shared_v4(dst + (((uint32_t)j ^ xr) << 4), v.x, v.y, v.z, v.w);
              }
            } else {
#pragma unroll
              for (int j = 0; j < 8; ++j) st_shared_v4(dst + (((uint32_t)j ^ xr) << 4), 0, 0, 0, 0);
            }
          } else {
            // A[m = i][k] = A_adapter[i / lambda_in][kk + k], read from the transposed copy (row = kk + k)
            const unsigned short* src = reinterpret_cast<const unsigned short*>(p.ex + (int64_t)(kk + (d & 63)) * p.ex_ld);
            const int i0 = m0 + (d >> 6) * 64;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              uint32_t o4[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const int ia = i0 + j * 8 + 2 * e, ib = ia + 1;
                const uint32_t lo = ia < p.d_in ? (uint32_t)__ldg(src + ia / p.lam) : 0u;
                const uint32_t hi = ib < p.d_in ? (uint32_t)__ldg(src + ib / p.lam) : 0u;
                o4[e] = lo | (hi << 16);
              }
              st_shared_v4(dst + (((uint32_t)j ^ xr) << 4), o4[0], o4[1], o4[2], o4[3]);
            }
          }
        }
        fence_async_proxy();   // generic-proxy stores -> visible to the tensor core's async proxy
        if (rank == 0) {
          mbar_arrive(aready(s));
        } else {
          // this CTA's stage (token half landed, weight tile written) is ready: tell the leader, once per warp
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(leader_peer + 8u * s);
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps (128 threads)
    const int q = warp & 3;                       // TMEM lane quadrant this warp may read
    const uint32_t leader_accempty0 = map_to_cta(accempty(0), 0), leader_accempty1 = map_to_cta(accempty(1), 0);
    bool ok = true;
    int lt = 0;
    for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters, ++lt) {
      const int a = lt & 1;
      const uint32_t aph = (lt >> 1) & 1u;
      const int m = (tile % p.m_tiles) * (2 * BM) + (int)rank * BM + q * 32 + lane;
      const int t0 = (tile / p.m_tiles) * BN;
      if (!mbar_wait(accfull(a), aph, p.status)) { ok = false; break; }
      tc_fence_after();
      for (int c = 0; c < BN / 32; ++c) {
        if (t0 + c * 32 >= p.T) break;
        uint32_t v[32];
        tc_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(a * BN + c * 32), v);
        if (m < p.M) {
          if (p.out_dtype == QBLORA_BF16) {
            __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(p.out);
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const int t = t0 + c * 32 + j;
              if (t < p.T) out[(int64_t)t * p.M + m] = __float2bfloat16_rn(__uint_as_float(v[j]));
            }
          } else {
            float* out = reinterpret_cast<float*>(p.out);
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const int t = t0 + c * 32 + j;
              if (t < p.T) out[(int64_t)t * p.M + m] = __uint_as_float(v[j]);
            }
          }
        }
      }
      tc_fence_before();
      mbar_arrive_cluster(a == 0 ? leader_accempty0 : leader_accempty1);
    }
  }

  // Neither CTA may leave (or free tensor memory) while its partner can still reach into it.
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}

// -------------------------------------------------------------------------------- adapter helpers
// dst[c][rw] = src[rw][c] for rw < rows, zero for rows <= rw < rows_pad (dst leading dimension rows_pad).
__global__ void transpose_pad_cols_kernel(const __nv_bfloat16* __restrict__ src, int rows, int cols, int rows_pad,
                                          __nv_bfloat16* __restrict__ dst) {
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)cols * rows_pad) return;
  const int c = (int)(idx / rows_pad), rw = (int)(idx % rows_pad);
  dst[idx] = rw < rows ? src[(int64_t)rw * cols + c] : __float2bfloat16_rn(0.0f);
}
// dst[rw][c] = src[c][rw] for rw < rows_src... : A^T with zero rows appended: dst [r_pad][P], src A [P][r].
__global__ void transpose_pad_rows_kernel(const __nv_bfloat16* __restrict__ A, int P, int r, int r_pad,
                                          __nv_bfloat16* __restrict__ dst) {
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)r_pad * P) return;
  const int k = (int)(idx / P), pp = (int)(idx % P);
  dst[idx] = k < r ? A[(int64_t)pp * r + k] : __float2bfloat16_rn(0.0f);
}

struct EpBf16Scaled {  // C16[m][n] = bf16(scale * acc); optional fp32 copy of acc
  __nv_bfloat16* C16; int64_t ld16; float scale; bool divide; float* C32; int64_t ld32;
  __device__ void operator()(int m, int n, float acc) const {
    if (C32) C32[m * ld32 + n] = acc;
    const float v = divide ? __fdiv_rn(acc, scale) : acc * scale;
    C16[m * ld16 + n] = __float2bfloat16_rn(v);
  }
};

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

// 2-D tensor map: `inner` contiguous elements per row, `rows` rows, row pitch `pitch_bytes`.
int make_map(CUtensorMap* tm, CUtensorMapDataType dt, int elem_bytes, const void* ptr, uint64_t inner,
             uint64_t rows, uint64_t pitch_bytes, uint32_t box_inner, uint32_t box_rows, bool swizzle128) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return QBLORA_ERR_CUDA;
  cuuint64_t dims[2] = {inner, rows};
  cuuint64_t strides[1] = {pitch_bytes};
  cuuint32_t box[2] = {box_inner, box_rows};
  cuuint32_t estr[2] = {1, 1};
  (void)elem_bytes;
  CUresult r = fn(tm, dt, 2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? QBLORA_OK : QBLORA_ERR_CUDA;
}

int num_sms() {
  static int n = []() {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) return 148;
    return v;
  }();
  return n;
}

struct TcWs {
  float *xp, *u32, *dv, *du32;
  __nv_bfloat16 *u16, *bt, *du16, *at;
  int r_pad;
  size_t bytes;
};

TcWs carve(int op, const AdView* ad, int64_t T, char* ws) {
  TcWs w{};
  size_t off = kStatusBytes;
  auto take = [&](size_t nbytes) { char* ptr = ws ? ws + off : nullptr; off += align_up(nbytes, 256); return ptr; };
  if (ad) {
    w.r_pad = (ad->r + BK - 1) / BK * BK;
    w.xp = (float*)take((size_t)T * ad->P * 4);
    w.u32 = (float*)take((size_t)T * ad->r * 4);
    if (op == QBLORA_OP_LINEAR_FWD) {
      w.u16 = (__nv_bfloat16*)take((size_t)T * w.r_pad * 2);
      w.bt = (__nv_bfloat16*)take((size_t)ad->Q * w.r_pad * 2);
    } else {
      w.dv = (float*)take((size_t)T * ad->Q * 4);
      w.du32 = (float*)take((size_t)T * ad->r * 4);
      w.du16 = (__nv_bfloat16*)take((size_t)T * w.r_pad * 2);
      w.at = (__nv_bfloat16*)take((size_t)w.r_pad * ad->P * 2);
    }
  }
  w.bytes = off;
  return w;
}

int launch_main(int mode, const QwView& qw, const AdView* ad, const __nv_bfloat16* Bop, const __nv_bfloat16* Bx,
                int r_pad, const __nv_bfloat16* ex, int64_t T, void* out, int out_dtype, int* status,
                cudaStream_t st) {
  static bool attr_set[2] = {false, false};
  if (!attr_set[mode]) {
    cudaError_t e = mode == 0
        ? cudaFuncSetAttribute(tc_dq_gemm_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES)
        : cudaFuncSetAttribute(tc_dq_gemm_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) return QBLORA_ERR_CUDA;
    attr_set[mode] = true;
  }
  TcParams p{};
  p.M = mode == 0 ? qw.d_out : qw.d_in;
  const int Kq = mode == 0 ? qw.d_in : qw.d_out;
  p.kb_base = (Kq + BK - 1) / BK;
  p.kb_extra = ad ? r_pad / BK : 0;
  p.T = (int)T;
  p.m_tiles = (p.M + 2 * BM - 1) / (2 * BM);
  p.n_tiles = (int)((T + BN - 1) / BN);
  p.d_in = qw.d_in; p.d_out = qw.d_out; p.G = qw.G;
  p.alpha = qw.alpha; p.beta = qw.beta;
  for (int j = 0; j < 16; ++j) p.level[j] = qw.level[j];
  p.ex = ex;
  p.ex_ld = ad ? (mode == 0 ? r_pad : ad->P) : 0;
  p.lam = ad ? (mode == 0 ? ad->l2 : ad->l1) : 1;
  p.out = out; p.out_dtype = out_dtype; p.status = status;

  CUtensorMap tm_b, tm_bx, tm_p;
  int rc = make_map(&tm_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Bop, (uint64_t)Kq, (uint64_t)T, (uint64_t)Kq * 2, BK, BN_HALF, true);
  if (rc) return rc;
  if (ad) rc = make_map(&tm_bx, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Bx, (uint64_t)r_pad, (uint64_t)T, (uint64_t)r_pad * 2, BK, BN_HALF, true);
  else tm_bx = tm_b;
  if (rc) return rc;
  if (mode == 0) rc = make_map(&tm_p, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, qw.codes, (uint64_t)qw.d_in / 2, (uint64_t)qw.d_out, (uint64_t)qw.d_in / 2, BK / 2, BM, false);
  else rc = make_map(&tm_p, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, qw.codes, (uint64_t)qw.d_in / 2, (uint64_t)qw.d_out, (uint64_t)qw.d_in / 2, BK / 2, BK, false);
  if (rc) return rc;

  const int tiles = p.m_tiles * p.n_tiles;                      // one tile per CTA pair
  const int pairs = num_sms() / 2;
  const int grid = 2 * (tiles < pairs ? tiles : pairs);
  {
    DominantKernelTimer timer(st);
    if (mode == 0) tc_dq_gemm_kernel<0><<<grid, NUM_THREADS, SMEM_BYTES, st>>>(tm_b, tm_bx, tm_p, p);
    else tc_dq_gemm_kernel<1><<<grid, NUM_THREADS, SMEM_BYTES, st>>>(tm_b, tm_bx, tm_p, p);
    count_launch();
  }
  QB_CUDA(cudaGetLastError());
  return QBLORA_OK;
}

}  // namespace

bool tc_supported(const QwView& qw, const AdView*, int64_t T) {
  return qw.block_in == BK && qw.block_out == 1 && qw.d_in % BK == 0 && qw.d_out % 8 == 0 && T >= 1 &&
         T < (int64_t)1 << 31;
}

size_t tc_ws_bytes(int op, const QwView&, const AdView* ad, int64_t T) { return carve(op, ad, T, nullptr).bytes; }

int tc_linear_fwd(const QwView& qw, const AdView* ad, const __nv_bfloat16* X, int64_t T, void* Y, int y_dtype,
                  char* ws, cudaStream_t st) {
  TcWs w = carve(QBLORA_OP_LINEAR_FWD, ad, T, ws);
  int rc;
  if (ad) {
    int64_t n = T * ad->P;
    pool_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(X, T, qw.d_in, ad->l1, w.xp);
    count_launch();
    QB_CUDA(cudaGetLastError());
    if (w.r_pad != ad->r) QB_CUDA(cudaMemsetAsync(w.u16, 0, (size_t)T * w.r_pad * 2, st));
    // u16 = bf16(s * x' A): the scaling rides on the compressed activation, B stays exact
    rc = gemm<true, false>(T, ad->r, ad->P, LdF32{w.xp, ad->P, 1}, LdBF16{ad->A, 1, ad->r},
                           EpBf16Scaled{w.u16, w.r_pad, ad->s, false, nullptr, 0}, st);
    if (rc) return rc;
    n = (int64_t)ad->Q * w.r_pad;
    transpose_pad_cols_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(ad->B, ad->r, ad->Q, w.r_pad, w.bt);
    count_launch();
    QB_CUDA(cudaGetLastError());
  }
  return launch_main(0, qw, ad, X, w.u16, w.r_pad, w.bt, T, Y, y_dtype, reinterpret_cast<int*>(ws), st);
}

int tc_linear_bwd(const QwView& qw, const AdView* ad, const __nv_bfloat16* X, const __nv_bfloat16* dY, int64_t T,
                  void* dX, int dx_dtype, float* dA, float* dB, char* ws, cudaStream_t st) {
  TcWs w = carve(QBLORA_OP_LINEAR_BWD, ad, T, ws);
  int rc;
  if (ad) {
    int64_t n = T * ad->Q;
    dv_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(dY, T, qw.d_out, ad->l2, ad->s, w.dv);
    count_launch();
    QB_CUDA(cudaGetLastError());
    if (dX && w.r_pad != ad->r) QB_CUDA(cudaMemsetAsync(w.du16, 0, (size_t)T * w.r_pad * 2, st));
    // du = dv B^T (fp32 for dA) and du16 = bf16(du / lambda_in) for the dX contraction
    rc = gemm<true, true>(T, ad->r, ad->Q, LdF32{w.dv, ad->Q, 1}, LdBF16{ad->B, ad->Q, 1},
                          EpBf16Scaled{w.du16, w.r_pad, (float)ad->l1, true, w.du32, ad->r}, st);
    if (rc) return rc;
    if (dA || dB) {
      n = T * ad->P;
      pool_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(X, T, qw.d_in, ad->l1, w.xp);
      count_launch();
      QB_CUDA(cudaGetLastError());
    }
    if (dB) {
      rc = gemm<true, false>(T, ad->r, ad->P, LdF32{w.xp, ad->P, 1}, LdBF16{ad->A, 1, ad->r},
                             EpStoreF32{w.u32, ad->r}, st);
      if (rc) return rc;
      rc = gemm<false, false>(ad->r, ad->Q, T, LdF32{w.u32, 1, ad->r}, LdF32{w.dv, 1, ad->Q},
                              EpStoreF32{dB, ad->Q}, st);
      if (rc) return rc;
    }
    if (dA) {
      rc = gemm<false, false>(ad->P, ad->r, T, LdF32{w.xp, 1, ad->P}, LdF32{w.du32, 1, ad->r},
                              EpStoreF32{dA, ad->r}, st);
      if (rc) return rc;
    }
    if (dX) {
      n = (int64_t)w.r_pad * ad->P;
      transpose_pad_rows_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(ad->A, ad->P, ad->r, w.r_pad, w.at);
      count_launch();
      QB_CUDA(cudaGetLastError());
    }
  }
  if (!dX) return QBLORA_OK;
  return launch_main(1, qw, ad, dY, w.du16, w.r_pad, w.at, T, dX, dx_dtype, reinterpret_cast<int*>(ws), st);
}

}  // namespace qb
