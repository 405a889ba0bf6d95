// Tensor-core path of the adapted quantized linear for sm_100a: a persistent, warp-specialised
// tcgen05 GEMM whose weight operand is unpacked from 4-bit codes and block-dequantized inside the
// mainloop (Sec. 3.1 / Algorithm 1's "dequantize then matmul", fused), with the adapter branch of
// Sec. 3.2 appended as extra K-blocks of the same accumulation:
//
//   forward : Y^T[o][t]  = sum_i w~[o][i] X[t][i]   + sum_k B[k][o/l2]      (s u)[t][k]
//   backward: dX^T[i][t] = sum_o w~[o][i] dY[t][o]  + sum_k A[i/l1][k]      (du/l1)[t][k]
//
// Two CTAs on the two SMs of a TPC form a cluster and issue tcgen05.mma with cta_group::2: one MMA covers
// 256 weight rows x 256 tokens.  Each CTA dequantizes its own 128 weight rows into shared memory (the MMA's A
// operand, canonical 128-byte-swizzled layout: K-major in the forward, MN-major in the backward, so the same
// [o][i]-packed codes serve both) and stages its half of every 256-token group by TMA (the B operand; no
// multicast).  Accumulators live in TMEM (2 x 256 columns).  Two tile shapes (Shape<NH>): 256 x 256 with the
// two TMEM halves double-buffering the accumulator, and 256 x 512, where one dequantized weight stage feeds the
// MMAs of two token groups -- half the dequantization work, shared-memory stores and ALU time per flop, which
// is what bounds this kernel -- and the tile's epilogue runs on eight warps without a mainloop beside it.
//
// Warp roles: warp 0 TMA producer; warp 1 MMA issuer (leader CTA only) and TMEM owner; then the dequant
// groups of four warps each, taking the K-blocks in turn (two groups in the forward, three in the backward;
// those of the other CTA report each finished stage to the leader's barrier); the last four (eight) warps are
// the epilogue.  Every mbarrier wait is bounded; on expiry the kernel stores QBLORA_ERR_TIMEOUT in the workspace
// status word and every role leaves its loop.
#include <cuda.h>

#include <atomic>
#include <cstdlib>

#include "common.cuh"
#include "simt_gemm.cuh"
#include "tc_ptx.cuh"
#include "tc_small.cuh"

namespace qb {
using namespace simt;
using namespace ptx;
namespace {

constexpr int BM = 128;        // rows of the weight-side operand per CTA (256 per CTA pair)
constexpr int BN = 256;        // tokens per MMA (each CTA of the pair stages 128 of them)
constexpr int BN_HALF = BN / 2;
constexpr int BK = 64;         // contraction elements per stage = one quantization block
constexpr int A_BYTES = BM * BK * 2;        // 16 KB dequantized weight tile
constexpr int BH_BYTES = BN_HALF * BK * 2;  // 16 KB: this CTA's half of one 256-token group
constexpr int P_BYTES = BM * BK / 2;        // 4 KB packed codes

// Tile shape.  NH = 1: a 256 x 256 tile per CTA pair, the two halves of tensor memory double-buffer the
// accumulator (the epilogue of one tile overlaps the mainloop of the next).  NH = 2: a 256 x 512 tile, both
// halves of tensor memory hold the one tile's accumulators and every dequantized weight stage feeds two MMA
// groups (tokens [0, 256) and [256, 512) of the tile), which halves the dequantization work, its shared-memory
// stores and its ALU time per flop; the price is an epilogue that no longer overlaps a mainloop (eight
// epilogue warps drain both halves at once) and coarser tiles.  The host picks per launch (tile_halves()).
template <int NH>
struct Shape {
  static constexpr int STAGES = NH == 2 ? 4 : 6;
  static constexpr int TILE_N = NH * BN;
  static constexpr int B_BYTES = NH * BH_BYTES;
  static constexpr int SMEM_BYTES = STAGES * (A_BYTES + B_BYTES + P_BYTES) + 512 + 1024;
};
static_assert(Shape<1>::SMEM_BYTES <= 227 * 1024 && Shape<2>::SMEM_BYTES <= 227 * 1024, "shared memory of the fused contraction");

// Warp roles.  Dequant groups of 128 threads take the K-blocks in turn (group g: index % NG == g).  The forward
// runs two groups; the backward three: its scale loads touch a new row of alpha / beta in every K-block (the
// forward walks along a row and mostly hits the L1), so one of its groups spends longer per K-block and two of
// them could not keep the tensor pipe fed (C4 shapes, kernel alone: backward 950 -> 1100 TFLOP/s with three
// groups and the scales of a group's next K-block loaded one K-block ahead; the forward measured the same with
// two or three groups and slower with the early load).
template <int MODE, int NH>
struct Roles {
  static constexpr int NG = MODE == 0 ? 2 : 3;
  static constexpr int EPI_WARP0 = 2 + 4 * NG;            // the epilogue warps (four per accumulator half in use at once) come last
  static constexpr int NUM_THREADS = (EPI_WARP0 + 4 * NH) * 32;
  static constexpr bool SCALES_AHEAD = MODE == 1;
};

struct TcParams {
  int M;                    // output rows of the tile grid: d_out (forward) / d_in (backward)
  int kb_base, kb_extra;    // K-blocks from the quantized weight / from the adapter
  int T;
  int m_tiles, n_tiles;     // tiles of 256 rows x 256 tokens (one per CTA pair)
  int d_in, d_out, G;
  int block_in, block_out;  // quantization block
  int direct;               // min-max format: form alpha * c + beta directly instead of through the per-block table
  const float* alpha;
  const float* beta;
  float level[16];
  const __nv_bfloat16* ex;  // adapter matrix feeding the extra K-blocks: forward B [r][Q], backward A [P][r]
  int ex_ld, ex_rows, lam;  // its leading dimension; the rank r; forward lambda_out, backward lambda_in
  int op, n_small;          // operator pair (qblora_scale_op) and the compressed size on that side (forward Q, backward P)
  // Low-bit product (Sec. 3.3) only: the per-block offsets as their own K-blocks.  The weight tile then holds
  // bf16(alpha * c + beta_c) with beta_c = -alpha * (mid code of the block), and the rest of the offset,
  // gamma = beta' - beta_c, multiplies the group sums of x: three K-segments of ng_blocks K-blocks each,
  // (gamma_hi, S_hi), (gamma_lo, S_hi), (gamma_hi, S_lo), with hi + lo the bf16 split of an fp32 value.
  int kb_gamma, ng_blocks;
  const __nv_bfloat16 *gam_h, *gam_l;   // [d_out][gam_ld], columns beyond G are zero
  int gam_ld;
  void* out;                // forward Y [T][d_out]; backward dX [T][d_in]
  int out_dtype;
  int* status;
  long long wait_limit;     // cycles after which a device-side wait gives up
  int drop_load;            // test hook: the producers leave out the loads of this K-block iteration (-1: none)
  long long hold_producer;  // test hook: the producers idle this many cycles in front of their first adapter K-block
};

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t r;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
  return r;
}

// Per-block dequantization table kept in registers.  The sixteen values bf16(alpha * level[c] + beta)
// of one quantization block (fp32 product, one rounding) are split into a low-byte plane and a
// high-byte plane of four registers each; a 4-bit code then selects its two bytes with byte-permute
// instructions only.  Measured on this part a byte permute issues at the rate of any integer ALU
// operation (2 cycles per warp instruction per scheduler) while a warp shuffle takes 4 and occupies
// the shared-memory data pipe the tensor core's operand fetch needs, so this lookup (21 ALU ops per
// 8 codes, table build amortised over 64) beats a shuffle-indexed table (8 shuffles + 7 shifts +
// 8 FMAs + 4 conversions per 8 codes).
struct BlockTable {
  uint32_t lp[4], hp[4];
  __device__ __forceinline__ void build(const float (&level)[16], float alpha, float beta) {
#pragma unroll
    for (int m = 0; m < 4; ++m) {
      const uint32_t p0 = pack_bf16x2(fmaf(alpha, level[4 * m + 0], beta), fmaf(alpha, level[4 * m + 1], beta));
      const uint32_t p1 = pack_bf16x2(fmaf(alpha, level[4 * m + 2], beta), fmaf(alpha, level[4 * m + 3], beta));
      lp[m] = prmt(p0, p1, 0x6420u);
      hp[m] = prmt(p0, p1, 0x7531u);
    }
  }
  // four codes in the low 16 bits of `a` (each masked to 3 bits) / `s2` (merge selector) -> 4 bf16
  __device__ __forceinline__ void half(uint32_t a, uint32_t s2, uint32_t& o01, uint32_t& o23) const {
    const uint32_t lo = prmt(prmt(lp[0], lp[1], a), prmt(lp[2], lp[3], a), s2);
    const uint32_t hi = prmt(prmt(hp[0], hp[1], a), prmt(hp[2], hp[3], a), s2);
    o01 = prmt(lo, hi, 0x5140u);
    o23 = prmt(lo, hi, 0x7362u);
  }
  // eight codes (code e in bits 4e..4e+3 of w) -> eight bf16 values in element order
  // m4 = 0x44444444 and c3210 = 0x32103210 come in registers: (x & literal) | literal compiles to
  // two logic ops, the explicit three-input form to one
  __device__ __forceinline__ void lookup8(uint32_t w, uint32_t (&o)[4], uint32_t m4, uint32_t c3210) const {
    const uint32_t a = w & 0x77777777u;                               // index within an 8-entry half
    uint32_t s2;                                                      // byte j: j + 4 * (code >> 3)
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(s2) : "r"(w >> 1), "r"(m4), "r"(c3210));
    half(a, s2, o[0], o[1]);
    half(a >> 16, s2 >> 16, o[2], o[3]);
  }
};

// Min-max format with quantization blocks narrower than a K-block (the paper's native 8 x 8 and 4 x 8
// blocks, Sec. 3.3): the 64 codes a dequant thread owns span 64 / BI (alpha, beta) pairs, so instead of
// a per-block table the value alpha * c + beta is formed directly.  A nibble OR-ed into the mantissa of
// 2^23 is the float 2^23 + c; one exact subtraction and one fused multiply-add (both on the FMA pipe)
// give the fp32 value, which is rounded once to bf16.  ab = this thread's alpha / beta entries.
template <int BI>
__device__ __forceinline__ void dequant_direct8(uint32_t w, int word, const float* al, const float* be, uint32_t (&o)[4]) {
  float v[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    const int sc = (word * 8 + e) / BI;                       // compile-time after unrolling
    const float c = __uint_as_float(((w >> (4 * e)) & 0xFu) | 0x4B000000u) - 8388608.0f;
    v[e] = fmaf(al[sc], c, be[sc]);
  }
#pragma unroll
  for (int e = 0; e < 4; ++e) o[e] = pack_bf16x2(v[2 * e], v[2 * e + 1]);
}

template <int MODE, int NH>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(Roles<MODE, NH>::NUM_THREADS, 1)
tc_dq_gemm_kernel(const __grid_constant__ CUtensorMap tm_b, const __grid_constant__ CUtensorMap tm_bx,
                  const __grid_constant__ CUtensorMap tm_p, const __grid_constant__ CUtensorMap tm_s,
                  const __grid_constant__ CUtensorMap tm_sl, const __grid_constant__ TcParams p) {
  constexpr int NG = Roles<MODE, NH>::NG, EPI_WARP0 = Roles<MODE, NH>::EPI_WARP0;
  constexpr int STAGES = Shape<NH>::STAGES, B_BYTES = Shape<NH>::B_BYTES, TILE_N = Shape<NH>::TILE_N;
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
  const int kb_total = p.kb_base + p.kb_extra + p.kb_gamma;
  const int kb_gamma0 = p.kb_base + p.kb_extra;   // first K-block of the offset term

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (one lane)
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      bool adapter_input_ready = false;
      for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters) {
        const int m0 = (tile % p.m_tiles) * (2 * BM) + (int)rank * BM;
        const int tt0 = (tile / p.m_tiles) * TILE_N;            // first token of the tile
        const int t0 = tt0 + (int)rank * BN_HALF;               // this CTA's 128 tokens of the first 256-token group
        const bool two = NH == 2 && tt0 + BN < p.T;             // the tile's second 256-token group holds tokens
        const uint32_t b_bytes = two ? 2 * BH_BYTES : BH_BYTES;
        for (int kb = 0; kb < kb_total; ++kb, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1u;
          if (!mbar_wait(empty(s), ph ^ 1u, p.status, p.wait_limit)) { ok = false; break; }
          if (kb < p.kb_base) {
            mbar_arrive_expect_tx(full(s), b_bytes + P_BYTES);
            // test hook (qblora_debug_drop_load): the bytes are announced and never sent, so this stage's
            // barrier cannot complete and every role has to run into its wait limit and leave by itself
            if ((int)it != p.drop_load) {
              tma_load_2d(sB + s * B_BYTES, &tm_b, full(s), kb * BK, t0);
              if (two) tma_load_2d(sB + s * B_BYTES + BH_BYTES, &tm_b, full(s), kb * BK, t0 + BN);
              if (MODE == 0) {
                tma_load_2d(sP + s * P_BYTES, &tm_p, full(s), kb * (BK / 2), m0);
              } else {   // two boxes of 64 rows x 32 bytes: packed[ng][k][32 B]
                tma_load_2d(sP + s * P_BYTES, &tm_p, full(s), m0 / 2, kb * BK);
                tma_load_2d(sP + s * P_BYTES + P_BYTES / 2, &tm_p, full(s), m0 / 2 + 32, kb * BK);
              }
            }
          } else {
            // The compressed adapter activation is written by the kernel launched just before this one.  With the
            // programmatic-dependent launch this grid started while that kernel was still running (everything up
            // to here reads only the caller's inputs); its result is complete and visible after this wait.
            if (!adapter_input_ready) {
              asm volatile("griddepcontrol.wait;" ::: "memory");
              adapter_input_ready = true;
              // test hook (qblora_debug_hold_producer): as if that wait had taken this much longer
              if (p.hold_producer > 0) { const long long h0 = clock64(); while (clock64() - h0 < p.hold_producer) {} }
            }
            mbar_arrive_expect_tx(full(s), b_bytes);
            if (kb < kb_gamma0) {
              tma_load_2d(sB + s * B_BYTES, &tm_bx, full(s), (kb - p.kb_base) * BK, t0);
              if (two) tma_load_2d(sB + s * B_BYTES + BH_BYTES, &tm_bx, full(s), (kb - p.kb_base) * BK, t0 + BN);
            } else {   // group sums of x: hi for the first two segments, lo for the third
              const int kg = kb - kb_gamma0, seg = kg / p.ng_blocks, blk = kg - seg * p.ng_blocks;
              tma_load_2d(sB + s * B_BYTES, seg == 2 ? &tm_sl : &tm_s, full(s), blk * BK, t0);
              if (two) tma_load_2d(sB + s * B_BYTES + BH_BYTES, seg == 2 ? &tm_sl : &tm_s, full(s), blk * BK, t0 + BN);
            }
          }
        }
      }
      if (!ok) {  // give copies already in flight a bounded chance to land before the CTA exits
        const uint32_t lo = it > (uint32_t)STAGES ? it - STAGES : 0;
        for (uint32_t j = lo; j < it; ++j) mbar_wait(full(j % STAGES), (j / STAGES) & 1u, p.status, p.wait_limit);
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      // ------------------------------------------------------------------ MMA issuer (leader CTA, one lane)
      // instruction descriptor: D fp32, A/B bf16, B K-major, A K-major (forward) or MN-major (backward),
      // M = 256 and N = 256 across the CTA pair
      const uint32_t idesc_common = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) |
                                    ((uint32_t)((2 * BM) >> 4) << 24);
      const uint32_t idesc_kmajor = idesc_common, idesc_mnmajor = idesc_common | (1u << 15);
      // One thread issues every MMA of the pair, so its instruction count per K-block is on the critical path:
      // the shared-memory descriptors are kept as running 64-bit values (constant upper half; the 14-bit start
      // address field moves by 2 per 32 bytes), the stage index and phase are counters, and the weight and
      // adapter K-blocks have loops of their own.
      const uint64_t dhi_k = smem_desc(0, 16, 1024), dhi_mn = smem_desc(0, 8192, 1024);   // upper halves (address 0)
      const uint32_t a_lo0 = (sA & 0x3FFFFu) >> 4, b_lo0 = (sB & 0x3FFFFu) >> 4;
      bool ok = true;
      int lt = 0, s = 0;
      uint32_t ph = 0;
      for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters, ++lt) {
        // NH == 1: the tile's accumulator is half (lt & 1) of tensor memory, used every other tile.  NH == 2: the
        // tile's two 256-token groups take both halves, every tile (a half without tokens gets no MMAs but still
        // goes through its full / empty hand-over, so the phases stay in step).
        const int a = NH == 2 ? 0 : (lt & 1);
        const uint32_t aph = NH == 2 ? (lt & 1u) : ((lt >> 1) & 1u);
        if (!mbar_wait(accempty(a), aph ^ 1u, p.status, p.wait_limit)) { ok = false; break; }
        if (NH == 2 && !mbar_wait(accempty(1), aph ^ 1u, p.status, p.wait_limit)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(a * BN);
        const bool two = NH == 2 && (tile / p.m_tiles) * TILE_N + BN < p.T;
        uint32_t acc = 0;   // the first MMA of a tile overwrites the accumulator
        // weight K-blocks [0, kb_base): K-major tile in the forward, MN-major in the backward; adapter K-blocks
        // [kb_base, kb_gamma0): the other way round (see the dequant warps); offset-term K-blocks: K-major
        for (int part = 0; part < 3 && ok; ++part) {
          const int n_kb = part == 0 ? p.kb_base : part == 1 ? p.kb_extra : p.kb_gamma;
          const bool a_kmajor = part == 2 || (MODE == 0) == (part == 0);
          const uint64_t dhi_a = a_kmajor ? dhi_k : dhi_mn;
          const uint32_t a_step = a_kmajor ? 2u : 128u;      // 32 bytes / 2048 bytes per K = 16, in 16-byte units
          const uint32_t idesc = a_kmajor ? idesc_kmajor : idesc_mnmajor;
          for (int kb = 0; kb < n_kb; ++kb) {
            if (!mbar_wait(full(s), ph, p.status, p.wait_limit) || !mbar_wait(aready(s), ph, p.status, p.wait_limit) ||
                !mbar_wait(peer(s), ph, p.status, p.wait_limit)) { ok = false; break; }
            tc_fence_after();
            const uint64_t adesc = dhi_a | (uint64_t)(a_lo0 + (uint32_t)s * (A_BYTES >> 4));
            const uint64_t bdesc = dhi_k | (uint64_t)(b_lo0 + (uint32_t)s * (B_BYTES >> 4));
#pragma unroll
            for (int k = 0; k < BK / 16; ++k)
              tc_mma_pair(d_tmem, adesc + (uint64_t)(k * a_step), bdesc + (uint64_t)(k * 2), idesc, k == 0 ? acc : 1u);
            if (two) {   // the same weight stage against the tile's second token group
#pragma unroll
              for (int k = 0; k < BK / 16; ++k)
                tc_mma_pair(d_tmem + BN, adesc + (uint64_t)(k * a_step), bdesc + (uint64_t)((BH_BYTES >> 4) + k * 2), idesc, k == 0 ? acc : 1u);
            }
            acc = 1u;
            tc_commit_pair(empty(s));
            if (++s == STAGES) { s = 0; ph ^= 1u; }
          }
        }
        if (ok) {
          tc_commit_pair(accfull(a));
          if (NH == 2) tc_commit_pair(accfull(1));
        }
      }
    }
  } else if (warp < EPI_WARP0) {
    // ------------------------------------------------------------------ dequant warps: NG groups of 128
    // threads; group g fills the stages of K-blocks with (global index % NG) == g.  Thread d owns one
    // quantization block (64 codes, one alpha/beta) of the tile per K-block.
    const int g = (warp - 2) >> 2;
    const int d = tid - 64 - 128 * g;
    const uint32_t leader_peer = map_to_cta(peer(0), 0);
    uint32_t k_m4 = 0x44444444u, k_c3210 = 0x32103210u;   // constants of lookup8, pinned to registers
    asm volatile("" : "+r"(k_m4), "+r"(k_c3210));
    // low-bit product: the per-block table offsets (and gamma) come from the kernel launched just before this one,
    // which may still be running when this grid starts as its programmatic dependent
    if (p.kb_gamma) asm volatile("griddepcontrol.wait;" ::: "memory");
    bool ok = true;
    uint32_t it = 0;
    float al_next = 0.0f, be_next = 0.0f;   // scale and offset of this group's next weight K-block of the tile,
    bool have_next = false;                 // loaded one K-block ahead (the load's latency hides under the look-ups)
    for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters) {
      const int m0 = (tile % p.m_tiles) * (2 * BM) + (int)rank * BM;
      // (alpha, beta) of this thread's quantization block in weight K-block kb
      auto load_scale = [&](int kb, float& al, float& be) {
        al = 0.0f; be = 0.0f;
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
      };
      for (int kb = 0; kb < kb_total; ++kb, ++it) {
        if ((int)(it % (uint32_t)NG) != g) continue;
        const int s = it % STAGES;
        const uint32_t ph = (it / STAGES) & 1u;
        const uint32_t a_stage = sA + s * A_BYTES;
        // K-major tile: thread d owns row d (64 K elements = 128 bytes).  MN-major tile: thread d owns
        // K-row (d & 63) of the 64-row group (d >> 6).  Either way a 128-byte row whose 16-byte chunks
        // are XOR-swizzled with (d & 7).
        const bool a_kmajor = kb >= kb_gamma0 || (MODE == 0) == (kb < p.kb_base);
        const uint32_t dst = a_kmajor ? a_stage + d * 128 : a_stage + (d >> 6) * 8192 + (d & 63) * 128;
        const uint32_t xr = d & 7;
        if (kb < p.kb_base && p.direct) {
          // ---- 2-D min-max blocks: the 64 codes of this thread lie in row o, columns i0 .. i0 + 63
          const int o = MODE == 0 ? m0 + d : kb * BK + (d & 63);
          const int i0 = MODE == 0 ? kb * BK : m0 + (d >> 6) * 64;
          float al[16], be[16];
#pragma unroll
          for (int k = 0; k < 16; ++k) { al[k] = 0.0f; be[k] = 0.0f; }
          if (o < p.d_out && i0 < p.d_in) {
            const int gi = p.d_in / p.block_in;
            const float4* ap = reinterpret_cast<const float4*>(p.alpha + (int64_t)(o / p.block_out) * gi + i0 / p.block_in);
            const float4* bp = reinterpret_cast<const float4*>(p.beta + (int64_t)(o / p.block_out) * gi + i0 / p.block_in);
            const int n4 = (BK / p.block_in) >> 2;             // 2 (block_in 8) or 4 (block_in 4) float4 each
#pragma unroll
            for (int k = 0; k < 4; ++k)
              if (k < n4) {
                const float4 a4 = __ldg(ap + k), b4 = __ldg(bp + k);
                al[4 * k] = a4.x; al[4 * k + 1] = a4.y; al[4 * k + 2] = a4.z; al[4 * k + 3] = a4.w;
                be[4 * k] = b4.x; be[4 * k + 1] = b4.y; be[4 * k + 2] = b4.z; be[4 * k + 3] = b4.w;
              }
          }
          // slot first, then its bytes (see the note on the wait order at the end of this loop body)
          if (!mbar_wait(empty(s), ph ^ 1u, p.status, p.wait_limit)) { ok = false; break; }
          if (!mbar_wait(full(s), ph, p.status, p.wait_limit)) { ok = false; break; }
          const uint8_t* src = gP + s * P_BYTES + d * 32;
          const uint4 q0 = *reinterpret_cast<const uint4*>(src);
          const uint4 q1 = *reinterpret_cast<const uint4*>(src + 16);
          const uint32_t w[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            uint32_t o4[4];
            if (p.block_in == 8) dequant_direct8<8>(w[j], j, al, be, o4);
            else dequant_direct8<4>(w[j], j, al, be, o4);
            st_shared_v4(dst + (((uint32_t)j ^ xr) << 4), o4[0], o4[1], o4[2], o4[3]);
          }
        } else if (kb < p.kb_base) {
          float al, be;
          if (have_next) { al = al_next; be = be_next; } else load_scale(kb, al, be);
          have_next = Roles<MODE, NH>::SCALES_AHEAD && kb + NG < p.kb_base;
          if (have_next) load_scale(kb + NG, al_next, be_next);
          BlockTable tab;
          tab.build(p.level, al, be);
          // slot first, then its bytes (see the note on the wait order at the end of this loop body)
          if (!mbar_wait(empty(s), ph ^ 1u, p.status, p.wait_limit)) { ok = false; break; }
          if (!mbar_wait(full(s), ph, p.status, p.wait_limit)) { ok = false; break; }
          const uint8_t* src = gP + s * P_BYTES + d * 32;
          const uint4 q0 = *reinterpret_cast<const uint4*>(src);
          const uint4 q1 = *reinterpret_cast<const uint4*>(src + 16);
          const uint32_t w[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            uint32_t o4[4];
            tab.lookup8(w[j], o4, k_m4, k_c3210);
            st_shared_v4(dst + (((uint32_t)j ^ xr) << 4), o4[0], o4[1], o4[2], o4[3]);
          }
        } else if (kb >= kb_gamma0) {
          // offset term of the low-bit product: K-major tile A[m = o][k = group] = gamma_hi (segments 0, 2) or
          // gamma_lo (segment 1); thread = output row o, reading 128 contiguous bytes of that row (the loads are
          // issued before the wait for the slot, so their latency hides under it)
          const int kg = kb - kb_gamma0, seg = kg / p.ng_blocks, g0 = (kg - seg * p.ng_blocks) * BK;
          const int o = m0 + d;
          const uint4* src = reinterpret_cast<const uint4*>((seg == 1 ? p.gam_l : p.gam_h) + (int64_t)(o < p.d_out ? o : 0) * p.gam_ld + g0);
          uint4 v[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            v[j] = make_uint4(0, 0, 0, 0);
            if (o < p.d_out && g0 + j * 8 < p.gam_ld) v[j] = __ldg(src + j);
          }
          if (!mbar_wait(empty(s), ph ^ 1u, p.status, p.wait_limit)) { ok = false; break; }
#pragma unroll
          for (int j = 0; j < 8; ++j) st_shared_v4(dst + (((uint32_t)j ^ xr) << 4), v[j].x, v[j].y, v[j].z, v[j].w);
        } else {
          // adapter K-blocks carry no packed codes
          const int kk = (kb - p.kb_base) * BK;
          if (MODE == 0) {
            // MN-major tile: A[m = o][k] = B[kk + k][o / lambda_out]; thread = (K-row, 64-wide output group),
            // reading a contiguous run of row kk + k of B.  Loads first, then the wait for the slot, then the stores.
            const int krow = kk + (d & 63);
            const int o0 = m0 + (d >> 6) * 64;
            const unsigned short* src = reinterpret_cast<const unsigned short*>(p.ex) + (int64_t)krow * p.ex_ld;
            const bool live = krow < p.ex_rows;
            uint4 v[8];
            if ((p.lam & 7) == 0 && p.op == QBLORA_SCALE_AVGPOOL_REPEAT) {   // a 16-byte chunk (8 outputs) repeats a single element of B
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                const int o = o0 + j * 8;
                uint32_t e = (live && o < p.d_out) ? (uint32_t)__ldg(src + o / p.lam) : 0u;
                e |= e << 16;
                v[j] = make_uint4(e, e, e, e);
              }
            } else if (p.op == QBLORA_SCALE_TRUNCATE_ZEROPAD) {
              // the first Q outputs take B's row as it is (Q is a multiple of 8: whole aligned 16-byte chunks), the rest nothing
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                const int o = o0 + j * 8;
                v[j] = make_uint4(0, 0, 0, 0);
                if (live && o < p.n_small) v[j] = __ldg(reinterpret_cast<const uint4*>(src + o));
              }
            } else if ((p.lam & 7) == 0) {
              // zero fill with a factor that is a multiple of 8: only the first output of a chunk can be a sampled one
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                const int o = o0 + j * 8;
                const uint32_t e = (live && o < p.d_out && o % p.lam == 0) ? (uint32_t)__ldg(src + o / p.lam) : 0u;
                v[j] = make_uint4(e, 0u, 0u, 0u);
              }
            } else {
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                uint32_t o4[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  const int oa = o0 + j * 8 + 2 * e, ob = oa + 1;
                  // column of B that the operator pair ties this output to (none: the output gets no adapter term)
                  const int qa = scale_src(p.op, oa, p.lam, p.n_small), qb_ = scale_src(p.op, ob, p.lam, p.n_small);
                  const uint32_t lo = (live && oa < p.d_out && qa >= 0) ? (uint32_t)__ldg(src + qa) : 0u;
                  const uint32_t hi = (live && ob < p.d_out && qb_ >= 0) ? (uint32_t)__ldg(src + qb_) : 0u;
                  o4[e] = lo | (hi << 16);
                }
                v[j] = make_uint4(o4[0], o4[1], o4[2], o4[3]);
              }
            }
            if (!mbar_wait(empty(s), ph ^ 1u, p.status, p.wait_limit)) { ok = false; break; }
#pragma unroll
            for (int j = 0; j < 8; ++j) st_shared_v4(dst + (((uint32_t)j ^ xr) << 4), v[j].x, v[j].y, v[j].z, v[j].w);
          } else {
            // K-major tile: A[m = i][k] = A_adapter[i / lambda_in][kk + k]; thread = input column i,
            // reading 128 contiguous bytes of a row of A_adapter (rank is a multiple of 8)
            const int i = m0 + d;
            const int prow = i < p.d_in ? scale_src(p.op, i, p.lam, p.n_small) : -1;   // -1: input not seen by the adapter
            const uint4* src = reinterpret_cast<const uint4*>(p.ex + (int64_t)(prow < 0 ? 0 : prow) * p.ex_ld + kk);
            uint4 v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              v[j] = make_uint4(0, 0, 0, 0);
              if (prow >= 0 && kk + j * 8 < p.ex_rows) v[j] = __ldg(src + j);
            }
            if (!mbar_wait(empty(s), ph ^ 1u, p.status, p.wait_limit)) { ok = false; break; }
#pragma unroll
            for (int j = 0; j < 8; ++j) st_shared_v4(dst + (((uint32_t)j ^ xr) << 4), v[j].x, v[j].y, v[j].z, v[j].w);
          }
        }
        // Wait order.  A parity wait tells "the phase with this parity is over", which is only the phase meant
        // while the waiter is less than one turn of the ring ahead of whoever completes it.  Every dequant thread
        // therefore waits for the producer's bytes of EVERY K-block it handles -- also of the adapter and
        // offset-term K-blocks, whose weight tile needs nothing from the producer: a thread that has seen full(it)
        // knows that the producer has passed it, hence (the producer waits for empty in order, and a group's next
        // K-block is at most NG <= STAGES further) that the MMAs of it + NG - 2 STAGES are done, so its next wait
        // for an empty slot means the right phase; and a weight K-block waits for the slot before the bytes: the
        // slot is free only after the MMAs of it - STAGES, which had waited for full(it - STAGES), so the wait
        // for full(it) cannot be answered by the previous turn's phase.  (Without this a producer held up for
        // long in griddepcontrol.wait let the dequant threads run a whole turn ahead through the adapter
        // K-blocks, and the next tile's first weight tiles were built from the previous turn's codes.)
        // In the other CTA of the pair the same wait also vouches for its token half of the stage.
        if (kb >= p.kb_base && !mbar_wait(full(s), ph, p.status, p.wait_limit)) { ok = false; break; }
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
    const int h = NH == 2 ? (warp - EPI_WARP0) >> 2 : 0;   // NH == 2: which 256-token group of the tile this warp drains
    const uint32_t leader_accempty0 = map_to_cta(accempty(0), 0), leader_accempty1 = map_to_cta(accempty(1), 0);
    bool ok = true;
    int lt = 0;
    for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters, ++lt) {
      const int a = NH == 2 ? h : (lt & 1);
      const uint32_t aph = NH == 2 ? (lt & 1u) : ((lt >> 1) & 1u);
      const int m = (tile % p.m_tiles) * (2 * BM) + (int)rank * BM + q * 32 + lane;
      const int t0 = (tile / p.m_tiles) * TILE_N + h * BN;
      if (!mbar_wait(accfull(a), aph, p.status, p.wait_limit)) { ok = false; break; }
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
__device__ __forceinline__ void store_split(float x, __nv_bfloat16* hi, __nv_bfloat16* lo, int64_t idx) {
  const __nv_bfloat16 h = __float2bfloat16_rn(x);
  hi[idx] = h;
  lo[idx] = __float2bfloat16_rn(x - __bfloat162float(h));
}
// Fast path of both segment sums below: out[t][w] = f(sum of `lam` consecutive bf16 of row t), f = /lam
// (AvgPool) or *scale (adjoint of repeat_interleave), written as a bf16 hi + lo pair.  One 16-byte load
// (8 elements) per thread; windows wider than a chunk are finished with warp shuffles.  Needs width % 8
// == 0 and lam in {1, 2, 4} or 8 * 2^k <= 256 with chunks-per-row % (lam / 8) == 0 (true when lam | width).
// 16-byte loads in flight per thread.  Two, at 32 registers per thread, measured best inside a step (C2 forward
// call 110 -> 107 us against four loads at 48 registers, 113 us with eight, 109 us with one): a 256-thread CTA of
// this kernel then fits on an SM beside a CTA of the fused contraction (448 x 128 registers), so the contraction,
// launched as a programmatic dependent further down the chain, can move in while the last CTAs here drain.
constexpr int SEGSUM_UNROLL = 2;
template <bool DIVIDE>
__device__ __forceinline__ void segsum_split_body(int64_t block, const __nv_bfloat16* __restrict__ src, int64_t rows, int width,
                                                  int lam, float scale, int ld_out,
                                                  __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo) {
  constexpr int UNROLL = SEGSUM_UNROLL;   // 16-byte loads in flight per thread (the kernel is a pure stream)
  const int chunks_per_row = width >> 3;
  const int64_t total = rows * chunks_per_row;
  uint4 q4[UNROLL];
  int64_t tt[UNROLL]; int cc[UNROLL]; bool lv[UNROLL];
#pragma unroll
  for (int k = 0; k < UNROLL; ++k) {
    const int64_t idx = (block * UNROLL + k) * blockDim.x + threadIdx.x;
    lv[k] = idx < total;
    tt[k] = 0; cc[k] = 0;
    q4[k] = make_uint4(0, 0, 0, 0);
    if (lv[k]) {
      if (total < (1ll << 31)) { const uint32_t i32 = (uint32_t)idx; tt[k] = i32 / (uint32_t)chunks_per_row; }
      else tt[k] = idx / chunks_per_row;
      cc[k] = (int)(idx - tt[k] * chunks_per_row);
      q4[k] = __ldg(reinterpret_cast<const uint4*>(src + tt[k] * width) + cc[k]);
    }
  }
#pragma unroll
  for (int k = 0; k < UNROLL; ++k) {
    const bool live = lv[k];
    const int64_t t = tt[k];
    const int c = cc[k];
    float v[8];
    const uint32_t w[4] = {q4[k].x, q4[k].y, q4[k].z, q4[k].w};
#pragma unroll
    for (int e = 0; e < 4; ++e) { v[2 * e] = __uint_as_float(w[e] << 16); v[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u); }
    if (lam >= 8) {
      float sacc = ((v[0] + v[1]) + (v[2] + v[3])) + ((v[4] + v[5]) + (v[6] + v[7]));
      const int lanes = lam >> 3;   // power of two, <= 32; windows never straddle a warp (256 % lanes == 0, rows aligned)
      for (int off = 1; off < lanes; off <<= 1) sacc += __shfl_xor_sync(0xffffffffu, sacc, off);
      if (live && (c & (lanes - 1)) == 0) {
        const float r = DIVIDE ? __fdiv_rn(sacc, (float)lam) : scale * sacc;
        store_split(r, hi, lo, t * ld_out + c / lanes);
      }
    } else if (live) {
      const int per = 8 / lam;      // windows inside this chunk
      for (int j = 0; j < per; ++j) {
        float sacc = 0.0f;
        for (int e = 0; e < lam; ++e) sacc += v[j * lam + e];
        const float r = DIVIDE ? __fdiv_rn(sacc, (float)lam) : scale * sacc;
        store_split(r, hi, lo, t * ld_out + c * per + j);
      }
    }
  }
}
template <bool DIVIDE>
__global__ void __launch_bounds__(256, 8) segsum_split_kernel(const __nv_bfloat16* __restrict__ src, int64_t rows, int width,
                                                           int lam, float scale, int ld_out,
                                                           __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the small product that follows may set up now
  segsum_split_body<DIVIDE>(blockIdx.x, src, rows, width, lam, scale, ld_out, hi, lo);
}
inline bool segsum_fast_ok(int width, int lam) {
  if (width % 8) return false;
  if (lam == 1 || lam == 2 || lam == 4) return true;
  if (lam % 8) return false;
  const int lanes = lam / 8;
  return lanes <= 32 && (lanes & (lanes - 1)) == 0 && (width / 8) % lanes == 0;
}

// x'[t][p] = AvgPool_{lambda_in}(X) (Sec. 3.2) as a bf16 hi + lo pair (hi + lo carries ~16 mantissa bits)
__global__ void pool_split_kernel(const __nv_bfloat16* __restrict__ X, int64_t T, int d_in, int l1, int ldp,
                                  __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the small product that follows may set up now
  const int P = d_in / l1;
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= T * P) return;
  const int64_t t = idx / P; const int pp = (int)(idx % P);
  const __nv_bfloat16* src = X + t * d_in + (int64_t)pp * l1;
  float s = 0.0f;
  if ((l1 & 7) == 0) {
    for (int j = 0; j < l1; j += 8) {
      const uint4 v = __ldg(reinterpret_cast<const uint4*>(src + j));
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) s += __uint_as_float(w[e] << 16) + __uint_as_float(w[e] & 0xffff0000u);
    }
  } else {
    for (int j = 0; j < l1; ++j) s += __bfloat162float(src[j]);
  }
  store_split(__fdiv_rn(s, (float)l1), hi, lo, t * ldp + pp);
}
// dv[t][q] = s * sum of lambda_out consecutive output gradients (adjoint of repeat_interleave), hi + lo
__global__ void dv_split_kernel(const __nv_bfloat16* __restrict__ dY, int64_t T, int d_out, int l2, float scaling,
                                int ldq, __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the small product that follows may set up now
  const int Q = d_out / l2;
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= T * Q) return;
  const int64_t t = idx / Q; const int q = (int)(idx % Q);
  const __nv_bfloat16* src = dY + t * d_out + (int64_t)q * l2;
  float a = 0.0f;
  if ((l2 & 7) == 0) {
    for (int j = 0; j < l2; j += 8) {
      const uint4 v = __ldg(reinterpret_cast<const uint4*>(src + j));
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) a += __uint_as_float(w[e] << 16) + __uint_as_float(w[e] & 0xffff0000u);
    }
  } else {
    for (int j = 0; j < l2; ++j) a += __bfloat162float(src[j]);
  }
  store_split(scaling * a, hi, lo, t * ldq + q);
}

// The alternative operator pairs of the Sec. 4 ablation read single values: out[t][j] = scale * src[t][j * stride]
// (stride 1 = truncation, lambda = interval sampling; scale = 1 for x', s for dv), stored as a hi + lo pair.
__global__ void sample_split_kernel(const __nv_bfloat16* __restrict__ src, int64_t T, int width, int n_small, int stride,
                                    float scale, int ld_out, __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the small product that follows may set up now
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= T * n_small) return;
  const int64_t t = idx / n_small; const int j = (int)(idx - t * n_small);
  store_split(scale * __bfloat162float(src[t * width + (int64_t)j * stride]), hi, lo, t * ld_out + j);
}

// Low-bit product, one thread per quantization block (64 codes = 32 bytes): splits the block's offset beta' into
// beta_c = -alpha * c_mid, which stays inside the bf16 weight operand (c_mid = middle of the codes the block
// uses, so alpha * c + beta_c is centred on zero and its bf16 rounding error is that of the weight's own spread,
// whatever shift a merge has put into beta'), and gamma = beta' - beta_c, kept as a bf16 hi + lo pair for the
// offset-term K-blocks.  The last block of a row also zeroes the row's padding columns.
__device__ __forceinline__ void lowbit_center_body(int64_t block, const uint8_t* __restrict__ codes, const float* __restrict__ alpha,
                                                   const float* __restrict__ beta, int64_t nblocks, int G, int ldg,
                                                   float* __restrict__ beta_c, __nv_bfloat16* __restrict__ gam_h,
                                                   __nv_bfloat16* __restrict__ gam_l) {
  const int64_t b = block * blockDim.x + threadIdx.x;
  if (b >= nblocks) return;
  const uint4* src = reinterpret_cast<const uint4*>(codes + b * 32);
  const uint4 q0 = __ldg(src), q1 = __ldg(src + 1);
  const uint32_t w[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
  uint32_t mn = 0x0F0F0F0Fu, mx = 0u;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const uint32_t lo = w[j] & 0x0F0F0F0Fu, hi = (w[j] >> 4) & 0x0F0F0F0Fu;
    mn = __vminu4(mn, __vminu4(lo, hi));
    mx = __vmaxu4(mx, __vmaxu4(lo, hi));
  }
  mn = __vminu4(mn, mn >> 16); mn = __vminu4(mn, mn >> 8);
  mx = __vmaxu4(mx, mx >> 16); mx = __vmaxu4(mx, mx >> 8);
  const float c_mid = 0.5f * (float)((mn & 0xFFu) + (mx & 0xFFu));
  const float bc = -__fmul_rn(__ldg(alpha + b), c_mid);
  const float gm = __fsub_rn(__ldg(beta + b), bc);
  beta_c[b] = bc;
  const int64_t row = b / G;
  const int g = (int)(b - row * G);
  store_split(gm, gam_h, gam_l, row * ldg + g);
  if (g == G - 1)
    for (int k = G; k < ldg; ++k) { gam_h[row * ldg + k] = __float2bfloat16_rn(0.0f); gam_l[row * ldg + k] = __float2bfloat16_rn(0.0f); }
}

// The two preparations of the low-bit product in ONE launch (they are independent and each is too small to fill the
// GPU for long): CTAs [0, center_ctas) split the offsets, the rest form the group sums of x.
__global__ void __launch_bounds__(256, 8) lowbit_prepare_kernel(int center_ctas, const uint8_t* __restrict__ codes,
                                                               const float* __restrict__ alpha, const float* __restrict__ beta,
                                                               int64_t nblocks, int G, int ldg, float* __restrict__ beta_c,
                                                               __nv_bfloat16* __restrict__ gam_h, __nv_bfloat16* __restrict__ gam_l,
                                                               const __nv_bfloat16* __restrict__ X, int64_t T, int d_in,
                                                               __nv_bfloat16* __restrict__ s_h, __nv_bfloat16* __restrict__ s_l) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the contraction that follows may set up now
  if ((int)blockIdx.x < center_ctas) lowbit_center_body(blockIdx.x, codes, alpha, beta, nblocks, G, ldg, beta_c, gam_h, gam_l);
  else segsum_split_body<false>((int64_t)blockIdx.x - center_ctas, X, T, d_in, BK, 1.0f, ldg, s_h, s_l);
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

inline int round8(int x) { return (x + 7) / 8 * 8; }

struct TcWs {
  __nv_bfloat16 *xh, *xl, *u16, *dvh, *dvl, *duh, *dul, *du16, *uh, *ul;
  float* partial;   // split-K scratch shared by the dA and dB products
  int ldp, ldq, ldr;
  size_t bytes;
};

TcWs carve(int op, const AdView* ad, int64_t T, char* ws) {
  TcWs w{};
  size_t off = kStatusBytes;
  auto take = [&](size_t elems) { char* ptr = ws ? ws + off : nullptr; off += align_up(elems * 2, 256); return (__nv_bfloat16*)ptr; };
  if (ad) {
    w.ldp = round8(ad->P); w.ldq = round8(ad->Q); w.ldr = round8(ad->r);
    w.xh = take((size_t)T * w.ldp); w.xl = take((size_t)T * w.ldp);
    if (op == QBLORA_OP_LINEAR_FWD) {
      w.u16 = take((size_t)T * w.ldr);
    } else {
      w.dvh = take((size_t)T * w.ldq); w.dvl = take((size_t)T * w.ldq);
      w.duh = take((size_t)T * w.ldr); w.dul = take((size_t)T * w.ldr); w.du16 = take((size_t)T * w.ldr);
      w.uh = take((size_t)T * w.ldr); w.ul = take((size_t)T * w.ldr);
      const size_t pa = (size_t)small_gemm_splits(ad->P, ad->r, (int)T) * ad->P * ad->r;
      const size_t pb = (size_t)small_gemm_splits(ad->r, ad->Q, (int)T) * ad->r * ad->Q;
      w.partial = (float*)take(2 * (pa > pb ? pa : pb));
    }
  }
  w.bytes = off;
  return w;
}

// QBLORA_NO_PDL=1 launches the fused contraction as an ordinary kernel (for A/B timing).
bool overlap_adapter_prologue() {
  static const bool on = []() { const char* v = getenv("QBLORA_NO_PDL"); return !(v && v[0] == '1'); }();
  return on;
}

// Launches the fused-dequant GEMM.  Bop: X (forward) / dY (backward); Bx: the compressed adapter
// activation [T][ldx] feeding the extra K-blocks (s * x' A forward, dv B^T / lambda_in backward).
// Offset term of the low-bit product (see TcParams): per-block table offsets beta_c [d_out][G], gamma = beta' - beta_c
// as bf16 hi / lo [d_out][ldg], and the group sums of x as bf16 hi / lo [T][ldg].
struct LowbitTerm {
  const float* beta_c;
  const __nv_bfloat16 *gam_h, *gam_l, *s_h, *s_l;
  int ldg;
};

// Tile shape of a launch (Shape<NH>): 512-token tiles when the problem has more than one 256-token group and the
// coarser tiles do not cost more in idle CTA pairs of the last round than they save per tile.  A 512-token tile
// is costed at kWideTileCost 256-token tiles.  QBLORA_TILE_HALVES=1|2 forces a shape (for A/B timing).
constexpr double kWideTileCost = 1.5;
int tile_halves(int m_tiles, int64_t T, int pairs) {
  static const int forced = []() { const char* v = getenv("QBLORA_TILE_HALVES"); return v ? atoi(v) : 0; }();
  if (T <= BN) return 1;
  if (forced == 1 || forced == 2) return forced;
  const int64_t tiles1 = (int64_t)m_tiles * ((T + BN - 1) / BN), tiles2 = (int64_t)m_tiles * ((T + 2 * BN - 1) / (2 * BN));
  const double cost1 = (double)((tiles1 + pairs - 1) / pairs), cost2 = kWideTileCost * (double)((tiles2 + pairs - 1) / pairs);
  return cost2 <= cost1 ? 2 : 1;
}

int launch_main(int mode, const QwView& qw, const AdView* ad, const __nv_bfloat16* Bop, const __nv_bfloat16* Bx,
                int ldx, int64_t T, void* out, int out_dtype, int* status, cudaStream_t st,
                const LowbitTerm* lb = nullptr) {
  // the shared-memory opt-in is a per-device function attribute: set once per device and kernel (the flags are
  // atomic, so concurrent host threads at worst set it twice)
  static std::atomic<bool> attr_set[64][2][2];
  int dev = 0;
  QB_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return QBLORA_ERR_UNSUPPORTED;
  TcParams p{};
  p.M = mode == 0 ? qw.d_out : qw.d_in;
  const int Kq = mode == 0 ? qw.d_in : qw.d_out;
  const int pairs = num_sms() / 2;
  const int nh = tile_halves((p.M + 2 * BM - 1) / (2 * BM), T, pairs);
  const void* kernel = mode == 0 ? (nh == 2 ? (const void*)tc_dq_gemm_kernel<0, 2> : (const void*)tc_dq_gemm_kernel<0, 1>)
                                 : (nh == 2 ? (const void*)tc_dq_gemm_kernel<1, 2> : (const void*)tc_dq_gemm_kernel<1, 1>);
  const int smem_bytes = nh == 2 ? Shape<2>::SMEM_BYTES : Shape<1>::SMEM_BYTES;
  const int threads = mode == 0 ? (nh == 2 ? Roles<0, 2>::NUM_THREADS : Roles<0, 1>::NUM_THREADS)
                                : (nh == 2 ? Roles<1, 2>::NUM_THREADS : Roles<1, 1>::NUM_THREADS);
  if (!attr_set[dev][mode][nh - 1].load(std::memory_order_acquire)) {
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes) != cudaSuccess) return QBLORA_ERR_CUDA;
    attr_set[dev][mode][nh - 1].store(true, std::memory_order_release);
  }
  p.kb_base = (Kq + BK - 1) / BK;
  p.kb_extra = ad ? (ad->r + BK - 1) / BK : 0;
  p.T = (int)T;
  p.m_tiles = (p.M + 2 * BM - 1) / (2 * BM);
  p.n_tiles = (int)((T + nh * BN - 1) / (nh * BN));
  p.d_in = qw.d_in; p.d_out = qw.d_out; p.G = qw.G;
  p.block_in = qw.block_in; p.block_out = qw.block_out;
  p.direct = qw.block_in != BK ? 1 : 0;   // (for 64 x 1 blocks the table is faster: 883 vs 702 TFLOP/s on the C5 up shape)
  p.alpha = qw.alpha; p.beta = qw.beta;
  for (int j = 0; j < 16; ++j) p.level[j] = qw.level[j];
  p.ex = ad ? (mode == 0 ? ad->B : ad->A) : nullptr;
  p.ex_ld = ad ? (mode == 0 ? ad->Q : ad->r) : 0;
  p.ex_rows = ad ? ad->r : 0;
  p.lam = ad ? (mode == 0 ? ad->l2 : ad->l1) : 1;
  p.op = ad ? ad->op : 0;
  p.n_small = ad ? (mode == 0 ? ad->Q : ad->P) : 0;
  p.out = out; p.out_dtype = out_dtype; p.status = status;
  p.wait_limit = wait_limit_cycles();
  p.drop_load = take_dropped_load();
  p.hold_producer = ad ? take_producer_hold() : 0;
  if (lb) {
    p.beta = lb->beta_c;
    p.ng_blocks = (qw.G + BK - 1) / BK;
    p.kb_gamma = 3 * p.ng_blocks;
    p.gam_h = lb->gam_h; p.gam_l = lb->gam_l; p.gam_ld = lb->ldg;
  }

  CUtensorMap tm_b, tm_bx, tm_p, tm_s, tm_sl;
  int rc = make_tensor_map_2d(&tm_b, false, Bop, (uint64_t)Kq, (uint64_t)T, (uint64_t)Kq * 2, BK, BN_HALF, true);
  if (rc) return rc;
  if (ad) rc = make_tensor_map_2d(&tm_bx, false, Bx, (uint64_t)ad->r, (uint64_t)T, (uint64_t)ldx * 2, BK, BN_HALF, true);
  else tm_bx = tm_b;
  if (rc) return rc;
  if (mode == 0) rc = make_tensor_map_2d(&tm_p, true, qw.codes, (uint64_t)qw.d_in / 2, (uint64_t)qw.d_out, (uint64_t)qw.d_in / 2, BK / 2, BM, false);
  else rc = make_tensor_map_2d(&tm_p, true, qw.codes, (uint64_t)qw.d_in / 2, (uint64_t)qw.d_out, (uint64_t)qw.d_in / 2, BK / 2, BK, false);
  if (rc) return rc;
  if (lb) {
    rc = make_tensor_map_2d(&tm_s, false, lb->s_h, (uint64_t)qw.G, (uint64_t)T, (uint64_t)lb->ldg * 2, BK, BN_HALF, true);
    if (rc) return rc;
    rc = make_tensor_map_2d(&tm_sl, false, lb->s_l, (uint64_t)qw.G, (uint64_t)T, (uint64_t)lb->ldg * 2, BK, BN_HALF, true);
    if (rc) return rc;
  } else {
    tm_s = tm_b; tm_sl = tm_b;
  }

  const int tiles = p.m_tiles * p.n_tiles;                      // one tile per CTA pair
  const int grid = 2 * (tiles < pairs ? tiles : pairs);
  // With an adapter the kernel in front of this one on the stream is the small product that writes Bx, and only
  // the last K-blocks of a tile read it: launch as its programmatic dependent, so that the weight K-blocks run
  // while that product finishes (the producer warp waits for it before the first adapter K-block).  Without an
  // adapter the predecessor is the caller's own work and the launch is an ordinary one.
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid); cfg.blockDim = dim3((unsigned)threads); cfg.dynamicSmemBytes = (size_t)smem_bytes; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = ((ad || lb) && overlap_adapter_prologue()) ? 1 : 0;
  cudaError_t le;
  {
    DominantKernelTimer timer(st);
    void* args[6] = {&tm_b, &tm_bx, &tm_p, &tm_s, &tm_sl, &p};
    le = cudaLaunchKernelExC(&cfg, kernel, args);
    count_launch();
  }
  QB_CUDA(le);
  QB_CUDA(cudaGetLastError());
  return QBLORA_OK;
}

int launch_pool(const QwView& qw, const AdView& ad, const __nv_bfloat16* X, int64_t T, const TcWs& w, cudaStream_t st) {
  const int64_t n = T * ad.P;
  if (ad.op != QBLORA_SCALE_AVGPOOL_REPEAT) {
    sample_split_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(
        X, T, qw.d_in, ad.P, ad.op == QBLORA_SCALE_TRUNCATE_ZEROPAD ? 1 : ad.l1, 1.0f, w.ldp, w.xh, w.xl);
  } else if (segsum_fast_ok(qw.d_in, ad.l1)) {
    const int64_t chunks = T * (qw.d_in / 8);
    segsum_split_kernel<true><<<(unsigned)((chunks + 256 * SEGSUM_UNROLL - 1) / (256 * SEGSUM_UNROLL)), 256, 0, st>>>(X, T, qw.d_in, ad.l1, 0.0f, w.ldp, w.xh, w.xl);
  } else {
    pool_split_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(X, T, qw.d_in, ad.l1, w.ldp, w.xh, w.xl);
  }
  count_launch();
  QB_CUDA(cudaGetLastError());
  return QBLORA_OK;
}

// u = x' A with x' = xh + xl: two K-segments against the same (exact, bf16) A
int launch_u_gemm(const AdView& ad, int64_t T, const TcWs& w, const SgOut& out, int* status, cudaStream_t st,
                  bool before_contraction) {
  const SgOperand a_mat{ad.A, ad.r, false};   // (n = rank index, k = p) at A[k * r + n]
  SgSegment segs[2] = {{{w.xh, w.ldp, true}, a_mat, ad.P}, {{w.xl, w.ldp, true}, a_mat, ad.P}};
  // directly behind the compression kernel on the same stream: its programmatic dependent
  return small_gemm((int)T, ad.r, segs, 2, out, status, st, nullptr, overlap_adapter_prologue(), before_contraction);
}

}  // namespace

bool tc_supported(const QwView& qw, const AdView* ad, int64_t T) {
  // block 64 x 1 (either format), or the min-max format with 8- or 4-wide blocks of any height
  const bool block_ok = (qw.block_in == BK && qw.block_out == 1) ||
                        (qw.qfmt == QBLORA_FMT_AFFINE_MINMAX && (qw.block_in == 8 || qw.block_in == 4) &&
                         qw.d_out % qw.block_out == 0);
  if (!(block_ok && qw.d_in % BK == 0 && qw.d_out % 8 == 0 && T >= 1 && T < (int64_t)1 << 31))
    return false;
  // TMA over the adapter matrices needs 16-byte row pitches
  return !ad || (ad->r % 8 == 0 && ad->Q % 8 == 0);
}

size_t tc_ws_bytes(int op, const QwView&, const AdView* ad, int64_t T) { return carve(op, ad, T, nullptr).bytes; }

int tc_linear_fwd(const QwView& qw, const AdView* ad, const __nv_bfloat16* X, int64_t T, void* Y, int y_dtype,
                  char* ws, cudaStream_t st) {
  TcWs w = carve(QBLORA_OP_LINEAR_FWD, ad, T, ws);
  int* status = reinterpret_cast<int*>(ws);
  if (ad) {
    int rc = launch_pool(qw, *ad, X, T, w, st);
    if (rc) return rc;
    // u16 = bf16(s * x' A): the scaling rides on the compressed activation, B stays exact
    SgOut out{};
    out.scaled = w.u16; out.ld16 = w.ldr; out.scale = ad->s; out.divide = false;
    rc = launch_u_gemm(*ad, T, w, out, status, st, true);
    if (rc) return rc;
  }
  return launch_main(0, qw, ad, X, w.u16, w.ldr, T, Y, y_dtype, status, st);
}

// Low-bit product for more than a handful of tokens (Sec. 3.3), 64 x 1 blocks:
//   Y[t][o] = sum_i x[t][i] bf16(alpha c + beta_c)[o][i] + sum_g gamma[o][g] S[t][g],  S[t][g] = sum of x over group g.
// Keeping gamma (which carries the merged adapter's shift) out of the bf16 weight operand makes the merged
// layer agree with the unmerged one to the accuracy of the base weight's own rounding (the merge identity).
namespace {
struct LowbitWs {
  float* beta_c; __nv_bfloat16 *gam_h, *gam_l, *s_h, *s_l; int ldg; size_t bytes;
};
LowbitWs carve_lowbit(const QwView& qw, int64_t T, char* ws) {
  LowbitWs w{};
  w.ldg = round8(qw.G);
  size_t off = kStatusBytes;
  auto take = [&](size_t bytes) { char* ptr = ws ? ws + off : nullptr; off += align_up(bytes, 256); return ptr; };
  w.beta_c = (float*)take((size_t)qw.d_out * qw.G * 4);
  w.gam_h = (__nv_bfloat16*)take((size_t)qw.d_out * w.ldg * 2);
  w.gam_l = (__nv_bfloat16*)take((size_t)qw.d_out * w.ldg * 2);
  w.s_h = (__nv_bfloat16*)take((size_t)T * w.ldg * 2);
  w.s_l = (__nv_bfloat16*)take((size_t)T * w.ldg * 2);
  w.bytes = off;
  return w;
}
}  // namespace

bool tc_lowbit_split_offsets(const QwView& qw) {
  return qw.qfmt == QBLORA_FMT_AFFINE_MINMAX && qw.block_in == BK && qw.block_out == 1;
}
size_t tc_lowbit_ws_bytes(const QwView& qw, int64_t T) {
  return tc_lowbit_split_offsets(qw) ? carve_lowbit(qw, T, nullptr).bytes : tc_ws_bytes(QBLORA_OP_LINEAR_FWD, qw, nullptr, T);
}
int tc_lowbit_gemm(const QwView& qw, const __nv_bfloat16* X, int64_t T, void* Y, int y_dtype, char* ws, cudaStream_t st) {
  int* status = reinterpret_cast<int*>(ws);
  if (!tc_lowbit_split_offsets(qw)) return launch_main(0, qw, nullptr, X, nullptr, 0, T, Y, y_dtype, status, st);
  const LowbitWs w = carve_lowbit(qw, T, ws);
  const int64_t nblocks = (int64_t)qw.d_out * qw.G;
  // offsets split per block and group sums of x (d_in is a multiple of 64 here, so the one-load-per-thread
  // segment sum applies), in one launch
  const int64_t chunks = T * (qw.d_in / 8);
  const int center_ctas = (int)((nblocks + 255) / 256);
  const int64_t sum_ctas = (chunks + 256 * SEGSUM_UNROLL - 1) / (256 * SEGSUM_UNROLL);
  lowbit_prepare_kernel<<<(unsigned)(center_ctas + sum_ctas), 256, 0, st>>>(center_ctas, qw.codes, qw.alpha, qw.beta, nblocks, qw.G,
                                                                          w.ldg, w.beta_c, w.gam_h, w.gam_l, X, T, qw.d_in, w.s_h, w.s_l);
  count_launch();
  QB_CUDA(cudaGetLastError());
  const LowbitTerm lb{w.beta_c, w.gam_h, w.gam_l, w.s_h, w.s_l, w.ldg};
  return launch_main(0, qw, nullptr, X, nullptr, 0, T, Y, y_dtype, status, st, &lb);
}

namespace {
// Second stream for the backward's adapter-gradient chain, so that it runs beside the dX contraction
// (whose last wave leaves SMs idle) instead of in front of it.  Created on first use, per host thread
// and device; the events only order work (no timing).
struct SideLane {
  cudaStream_t stream = nullptr;
  cudaEvent_t fork = nullptr, du_done = nullptr, join = nullptr;
  bool ok = false, tried = false;
};
SideLane* side_lane() {
  static thread_local SideLane lanes[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  SideLane& l = lanes[dev];
  if (!l.tried) {
    l.tried = true;
    const char* off = getenv("QBLORA_NO_OVERLAP");
    if (!(off && off[0] == '1') &&
        cudaStreamCreateWithFlags(&l.stream, cudaStreamNonBlocking) == cudaSuccess &&
        cudaEventCreateWithFlags(&l.fork, cudaEventDisableTiming) == cudaSuccess &&
        cudaEventCreateWithFlags(&l.du_done, cudaEventDisableTiming) == cudaSuccess &&
        cudaEventCreateWithFlags(&l.join, cudaEventDisableTiming) == cudaSuccess)
      l.ok = true;
  }
  return l.ok ? &l : nullptr;
}
}  // namespace

int tc_linear_bwd(const QwView& qw, const AdView* ad, const __nv_bfloat16* X, const __nv_bfloat16* dY, int64_t T,
                  void* dX, int dx_dtype, float* dA, float* dB, char* ws, cudaStream_t st) {
  TcWs w = carve(QBLORA_OP_LINEAR_BWD, ad, T, ws);
  int* status = reinterpret_cast<int*>(ws);
  if (!ad) return dX ? launch_main(1, qw, ad, dY, w.du16, w.ldr, T, dX, dx_dtype, status, st) : QBLORA_OK;
  // Two chains: (a) dv -> du, which the dX contraction needs; (b) pooled x -> u -> dB, dA, which
  // nothing else needs.  With a side lane (b) runs on it: it starts together with (a), waits for du
  // before the gradient products, and is joined at the end; the caller's stream goes straight from
  // (a) to the dX contraction.
  SideLane* lane = (dX && (dA || dB)) ? side_lane() : nullptr;
  cudaStream_t sb = lane ? lane->stream : st;
  if (lane) {
    QB_CUDA(cudaEventRecord(lane->fork, st));
    QB_CUDA(cudaStreamWaitEvent(lane->stream, lane->fork, 0));
  }
  // From here on the side lane may hold work of this call (and, inside a stream capture, is part of the capture):
  // whatever happens below, it is joined back into the caller's stream before the call returns.
  const int rc = [&]() -> int {
    int rc;
    const int64_t n = T * ad->Q;
    if (ad->op != QBLORA_SCALE_AVGPOOL_REPEAT) {
      sample_split_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(
          dY, T, qw.d_out, ad->Q, ad->op == QBLORA_SCALE_TRUNCATE_ZEROPAD ? 1 : ad->l2, ad->s, w.ldq, w.dvh, w.dvl);
    } else if (segsum_fast_ok(qw.d_out, ad->l2)) {
      const int64_t chunks = T * (qw.d_out / 8);
      segsum_split_kernel<false><<<(unsigned)((chunks + 256 * SEGSUM_UNROLL - 1) / (256 * SEGSUM_UNROLL)), 256, 0, st>>>(dY, T, qw.d_out, ad->l2, ad->s, w.ldq, w.dvh, w.dvl);
    } else {
      dv_split_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(dY, T, qw.d_out, ad->l2, ad->s, w.ldq, w.dvh, w.dvl);
    }
    count_launch();
    QB_CUDA(cudaGetLastError());
    {  // du = dv B^T (hi + lo for dA) and du16 = bf16(du / lambda_in) for the dX contraction
      const SgOperand b_mat{ad->B, ad->Q, true};   // (n = rank index, k = q) at B[n * Q + k]
      SgSegment segs[2] = {{{w.dvh, w.ldq, true}, b_mat, ad->Q}, {{w.dvl, w.ldq, true}, b_mat, ad->Q}};
      SgOut out{};
      out.hi = w.duh; out.lo = w.dul; out.scaled = w.du16; out.ld16 = w.ldr; out.divide = true;
      out.scale = ad->op == QBLORA_SCALE_AVGPOOL_REPEAT ? (float)ad->l1 : 1.0f;   // only the average carries 1 / lambda_in
      rc = small_gemm((int)T, ad->r, segs, 2, out, status, st, nullptr, overlap_adapter_prologue(), false);   // behind dv's kernel (narrow tiles: wide ones start the contraction earlier, which costs the gradient chain beside it more than it saves: C2 backward 115 vs 119 us)
      if (rc) return rc;
    }
    if (lane) QB_CUDA(cudaEventRecord(lane->du_done, st));
    if (dA || dB) {
      rc = launch_pool(qw, *ad, X, T, w, sb);
      if (rc) return rc;
    }
    if (dB) {
      SgOut uo{};
      uo.hi = w.uh; uo.lo = w.ul; uo.ld16 = w.ldr;
      rc = launch_u_gemm(*ad, T, w, uo, status, sb, false);
      if (rc) return rc;
    }
    if (lane) QB_CUDA(cudaStreamWaitEvent(lane->stream, lane->du_done, 0));   // dv and du are complete
    if (dB) {
      // dB[k][q] = sum_t u[t][k] dv[t][q]: both operands token-major, i.e. MN-contiguous
      const SgOperand uh{w.uh, w.ldr, false}, ul{w.ul, w.ldr, false}, dh{w.dvh, w.ldq, false}, dl{w.dvl, w.ldq, false};
      SgSegment segs[3] = {{uh, dh, (int)T}, {ul, dh, (int)T}, {uh, dl, (int)T}};
      SgOut out{};
      out.f32 = dB; out.ld32 = ad->Q;
      rc = small_gemm(ad->r, ad->Q, segs, 3, out, status, sb, w.partial);
      if (rc) return rc;
    }
    if (dA) {
      // dA[p][k] = sum_t x'[t][p] du[t][k]
      const SgOperand xh{w.xh, w.ldp, false}, xl{w.xl, w.ldp, false}, dh{w.duh, w.ldr, false}, dl{w.dul, w.ldr, false};
      SgSegment segs[3] = {{xh, dh, (int)T}, {xl, dh, (int)T}, {xh, dl, (int)T}};
      SgOut out{};
      out.f32 = dA; out.ld32 = ad->r;
      rc = small_gemm(ad->P, ad->r, segs, 3, out, status, sb, w.partial);
      if (rc) return rc;
    }
    return dX ? launch_main(1, qw, ad, dY, w.du16, w.ldr, T, dX, dx_dtype, status, st) : QBLORA_OK;
  }();
  if (lane) {   // the call's work is complete when st is; on an error path this also closes a capture's fork
    const bool joined = cudaEventRecord(lane->join, lane->stream) == cudaSuccess &&
                        cudaStreamWaitEvent(st, lane->join, 0) == cudaSuccess;
    if (!joined && rc == QBLORA_OK) return QBLORA_ERR_CUDA;
  }
  return rc;
}

}  // namespace qb
