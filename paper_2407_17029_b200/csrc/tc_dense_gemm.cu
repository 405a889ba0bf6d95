// Serving product for the 16-bit deployment (Sec. 3.1 / 3.2: after fine-tuning the adapter is merged into a
// full-precision weight "with no inference overhead"):  Y[t][o] = sum_i X[t][i] W'[o][i],  W' bf16 [d_out][d_in]
// as written by qblora_merge_dense.
//
// A plain bf16 tcgen05 GEMM: persistent, one 256 (weight rows) x 256 (tokens) tile per CTA pair
// (cta_group::2), both operands staged by TMA (each CTA loads its own 128 weight rows and its own half of the
// token tile; no multicast), fp32 accumulators in TMEM, double-buffered so the epilogue of one tile overlaps the
// mainloop of the next.  It is the fused contraction of tc_gemm.cu without the dequant warps.
//
// Warp roles (256 threads per CTA): warp 0 TMA producer; warp 1 MMA issuer (leader CTA only) and TMEM owner;
// warp 2 relay (other CTA only: tells the leader when this CTA's half of a stage has landed); warps 4-7 epilogue.
// Every mbarrier wait is bounded; on expiry the kernel stores QBLORA_ERR_TIMEOUT in the status word and every
// role leaves its loop.
#include <cuda.h>

#include <atomic>

#include "common.cuh"
#include "tc_ptx.cuh"
#include "tc_small.cuh"

namespace qb {
using namespace ptx;
namespace {

constexpr int DG_BM = 128;         // weight rows per CTA (256 per pair)
constexpr int DG_BN = 256;         // tokens per tile (each CTA stages 128 of them)
constexpr int DG_BK = 64;
constexpr int DG_STAGES = 6;
constexpr int DG_A_BYTES = DG_BM * DG_BK * 2;        // 16 KB
constexpr int DG_B_BYTES = (DG_BN / 2) * DG_BK * 2;  // 16 KB
constexpr int DG_THREADS = 256;
constexpr int DG_SMEM = DG_STAGES * (DG_A_BYTES + DG_B_BYTES) + 512 + 1024;

// Tile order: groups of DG_GROUP_M row tiles, token tiles outer inside a group.  The 74 tiles in flight then span
// 8 row tiles x ~9 token tiles, so every operand panel they read is shared by several of them and stays in L2
// (with the row tiles simply running fastest, a 13824 x 5120 weight is streamed from HBM once per token tile).
constexpr int DG_GROUP_M = 8;
__device__ __forceinline__ void dg_tile_coords(int tile, int m_tiles, int n_tiles, int& mt, int& nt) {
  const int per_group = DG_GROUP_M * n_tiles;
  const int g = tile / per_group, r = tile - g * per_group;
  const int first = g * DG_GROUP_M;
  const int gm = min(DG_GROUP_M, m_tiles - first);
  nt = r / gm;
  mt = first + (r - nt * gm);
}

struct DgParams {
  int M, T, kb_total, m_tiles, n_tiles;
  void* out;
  int out_dtype;
  int* status;
  long long wait_limit;
};

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(DG_THREADS, 1)
tc_dense_gemm_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_x,
                     const __grid_constant__ DgParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  const uint32_t sA = base, sB = sA + DG_STAGES * DG_A_BYTES;
  const uint32_t bars = sB + DG_STAGES * DG_B_BYTES;
  auto full = [&](int s) { return bars + 8u * s; };                        // this CTA's TMA bytes landed
  auto empty = [&](int s) { return bars + 8u * (DG_STAGES + s); };          // MMAs reading the stage are done
  auto peer = [&](int s) { return bars + 8u * (2 * DG_STAGES + s); };       // leader only: the other CTA's half landed
  auto accfull = [&](int a) { return bars + 8u * (3 * DG_STAGES + a); };
  auto accempty = [&](int a) { return bars + 8u * (3 * DG_STAGES + 2 + a); };   // leader only: both epilogues drained
  const uint32_t tmem_slot = bars + 8u * (3 * DG_STAGES + 4);
  volatile uint32_t* tmem_slot_g = reinterpret_cast<volatile uint32_t*>(smem_raw + (tmem_slot - raw));

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();
  const int num_clusters = gridDim.x >> 1, cluster_id = blockIdx.x >> 1;

  if (tid == 0) {
    for (int s = 0; s < DG_STAGES; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), 1); mbar_init(peer(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(accfull(a), 1); mbar_init(accempty(a), 256); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_g;
  const int num_tiles = p.m_tiles * p.n_tiles;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (one lane)
    if (lane == 0) {
      uint32_t it = 0, ph = 0;
      int s = 0;
      bool ok = true;
      for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters) {
        int mt, nt;
        dg_tile_coords(tile, p.m_tiles, p.n_tiles, mt, nt);
        const int m0 = mt * (2 * DG_BM) + (int)rank * DG_BM;
        const int t0 = nt * DG_BN + (int)rank * (DG_BN / 2);
        for (int kb = 0; kb < p.kb_total; ++kb, ++it) {
          if (!mbar_wait(empty(s), ph ^ 1u, p.status, p.wait_limit)) { ok = false; break; }
          mbar_arrive_expect_tx(full(s), DG_A_BYTES + DG_B_BYTES);
          tma_load_2d(sA + s * DG_A_BYTES, &tm_w, full(s), kb * DG_BK, m0);
          tma_load_2d(sB + s * DG_B_BYTES, &tm_x, full(s), kb * DG_BK, t0);
          if (++s == DG_STAGES) { s = 0; ph ^= 1u; }
        }
      }
      if (!ok) {  // give copies already in flight a bounded chance to land before the CTA exits
        const uint32_t lo = it > (uint32_t)DG_STAGES ? it - DG_STAGES : 0;
        for (uint32_t j = lo; j < it; ++j) mbar_wait(full(j % DG_STAGES), (j / DG_STAGES) & 1u, p.status, p.wait_limit);
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      // ------------------------------------------------------------------ MMA issuer (leader CTA, one lane)
      // instruction descriptor: D fp32, A/B bf16, both K-major, M = 256 and N = 256 across the CTA pair
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(DG_BN >> 3) << 17) |
                             ((uint32_t)((2 * DG_BM) >> 4) << 24);
      const uint64_t dhi = smem_desc(0, 16, 1024);
      const uint32_t a_lo0 = (sA & 0x3FFFFu) >> 4, b_lo0 = (sB & 0x3FFFFu) >> 4;
      bool ok = true;
      int lt = 0, s = 0;
      uint32_t ph = 0;
      for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters, ++lt) {
        const int a = lt & 1;
        const uint32_t aph = (lt >> 1) & 1u;
        if (!mbar_wait(accempty(a), aph ^ 1u, p.status, p.wait_limit)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(a * DG_BN);
        uint32_t acc = 0;
        for (int kb = 0; kb < p.kb_total; ++kb) {
          if (!mbar_wait(full(s), ph, p.status, p.wait_limit) || !mbar_wait(peer(s), ph, p.status, p.wait_limit)) { ok = false; break; }
          tc_fence_after();
          const uint64_t adesc = dhi | (uint64_t)(a_lo0 + (uint32_t)s * (DG_A_BYTES >> 4));
          const uint64_t bdesc = dhi | (uint64_t)(b_lo0 + (uint32_t)s * (DG_B_BYTES >> 4));
#pragma unroll
          for (int k = 0; k < DG_BK / 16; ++k) {
            tc_mma_pair(d_tmem, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc, acc);
            acc = 1u;
          }
          tc_commit_pair(empty(s));
          if (++s == DG_STAGES) { s = 0; ph ^= 1u; }
        }
        if (ok) tc_commit_pair(accfull(a));
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------------ relay (other CTA, one lane): its half of the
    // stage has landed -> one arrival on the leader's barrier for that stage
    if (lane == 0 && rank != 0) {
      const uint32_t leader_peer = map_to_cta(peer(0), 0);
      int s = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters) {
        for (int kb = 0; kb < p.kb_total; ++kb) {
          if (!mbar_wait(full(s), ph, p.status, p.wait_limit)) { ok = false; break; }
          mbar_arrive_cluster(leader_peer + 8u * s);
          if (++s == DG_STAGES) { s = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------------ epilogue warps (128 threads)
    const int q = warp & 3;                       // TMEM lane quadrant this warp may read
    const uint32_t leader_accempty0 = map_to_cta(accempty(0), 0), leader_accempty1 = map_to_cta(accempty(1), 0);
    bool ok = true;
    int lt = 0;
    for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters, ++lt) {
      const int a = lt & 1;
      const uint32_t aph = (lt >> 1) & 1u;
      int mt, nt;
      dg_tile_coords(tile, p.m_tiles, p.n_tiles, mt, nt);
      const int m = mt * (2 * DG_BM) + (int)rank * DG_BM + q * 32 + lane;
      const int t0 = nt * DG_BN;
      if (!mbar_wait(accfull(a), aph, p.status, p.wait_limit)) { ok = false; break; }
      tc_fence_after();
      for (int c = 0; c < DG_BN / 32; ++c) {
        if (t0 + c * 32 >= p.T) break;
        uint32_t v[32];
        tc_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(a * DG_BN + c * 32), v);
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

}  // namespace

size_t dense_gemm_ws_bytes() { return kStatusBytes; }

int launch_dense_gemm(const __nv_bfloat16* W, int d_out, int d_in, const __nv_bfloat16* X, int64_t T, void* Y,
                      int y_dtype, int* status, cudaStream_t st) {
  static std::atomic<bool> attr_set[64];
  int dev = 0;
  QB_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return QBLORA_ERR_UNSUPPORTED;
  if (!attr_set[dev].load(std::memory_order_acquire)) {
    QB_CUDA(cudaFuncSetAttribute(tc_dense_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, DG_SMEM));
    attr_set[dev].store(true, std::memory_order_release);
  }
  DgParams p{};
  p.M = d_out; p.T = (int)T;
  p.kb_total = (d_in + DG_BK - 1) / DG_BK;
  p.m_tiles = (d_out + 2 * DG_BM - 1) / (2 * DG_BM);
  p.n_tiles = (int)((T + DG_BN - 1) / DG_BN);
  p.out = Y; p.out_dtype = y_dtype; p.status = status;
  p.wait_limit = wait_limit_cycles();
  CUtensorMap tm_w, tm_x;
  int rc = make_tensor_map_2d(&tm_w, false, W, (uint64_t)d_in, (uint64_t)d_out, (uint64_t)d_in * 2, DG_BK, DG_BM, true);
  if (rc) return rc;
  rc = make_tensor_map_2d(&tm_x, false, X, (uint64_t)d_in, (uint64_t)T, (uint64_t)d_in * 2, DG_BK, DG_BN / 2, true);
  if (rc) return rc;
  int sms = 148;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int tiles = p.m_tiles * p.n_tiles, pairs = sms / 2;
  const int grid = 2 * (tiles < pairs ? tiles : pairs);
  {
    DominantKernelTimer timer(st);
    tc_dense_gemm_kernel<<<grid, DG_THREADS, DG_SMEM, st>>>(tm_w, tm_x, p);
    count_launch();
  }
  QB_CUDA(cudaGetLastError());
  return QBLORA_OK;
}

}  // namespace qb
