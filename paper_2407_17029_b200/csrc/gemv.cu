// Low-bit product for small token counts (decode, T <= 16):
//   Y[t][o] = sum_i X[t][i] * (alpha[o][i/64] * c[o][i] + beta'[o][i/64])            (Sec. 3.3)
// The packed weight is streamed exactly once (DRAM traffic = codes + alpha + beta).
//
// Structure.  One persistent CTA per SM.  A producer thread streams tiles of 32 output rows x 16
// quantization groups (16 KB of codes as four 128-byte-swizzled TMA boxes, plus the 32 x 16 alpha
// and beta values) through a shared-memory ring guarded by mbarriers, so no compute warp ever waits
// on DRAM latency or does global address arithmetic for the weight.  Each of the sixteen compute
// warps owns one of the tile's 16 groups and all 32 rows (two MMA row tiles).  Partial sums stay in
// registers across the K tiles and are summed through shared memory in warp order at the end
// (deterministic).
//
// Arithmetic.  The work of a warp is shaped for mma.sync.m16n8k16 (fp16 operands, fp32 accumulate):
// 16 rows are the M side, up to 8 tokens per N tile.  A thread (g = lane / 4, tg = lane % 4) reads,
// for rows g + 8 q (q = 0..3), the 8 bytes holding codes 16 tg .. 16 tg + 15 of the group and turns
// each 32-bit word into four fp16 pairs with one three-input logic op per pair: the nibbles are OR-ed
// into the mantissa of 1024.0, and because fp16's mantissa holds two neighbouring nibbles a word
// needs one shift only; odd nibbles come out as 1024 + 16 c and the token operand carries 1/16 at
// those positions.  The order of the k index inside an MMA is free as long as both operands agree,
// so nibble pairs (e, e + 4) are used as they fall out of the word and the token fragments are laid
// out to match.  x (bf16) is converted to fp16 after a power-of-two prescale 2^-e of its own for
// every 64-value slice (group, token).  With P = sum of the fragment values and R = sum of the
// scaled x over a group, the group contributes  2^e (alpha (acc - 1024 P) + beta R).
//
// Two kernels: one token (fragments of x resident in shared memory, row blocks outer) and 2..16
// tokens (K tiles outer, fragments prepared once in the workspace and streamed per K tile).
#include <cstdlib>
#include <atomic>
#include "tc_ptx.cuh"
#include "tc_small.cuh"

namespace qb {
using namespace ptx;
namespace {

constexpr int GT_ROWS = 32;            // rows per tile (two MMA row tiles)
constexpr int GT_GROUPS = 16;          // quantization groups per tile (1024 codes per row), one per warp
constexpr int GT_WARPS = 16;           // compute warps; warp 16 is the producer
constexpr int GT_THREADS = (GT_WARPS + 1) * 32;
constexpr int KO_THREADS = (GT_WARPS + 2) * 32;   // K-outer kernel: a second helper warp loads the token fragments
constexpr int GT_CODE_BYTES = GT_ROWS * GT_GROUPS * 32;   // 16 KB = four boxes of [32 rows][128 B]
constexpr int GT_SCALE_BYTES = GT_ROWS * GT_GROUPS * 4;   // 2 KB each for alpha and beta
constexpr int GT_STAGE_BYTES = GT_CODE_BYTES + 2 * GT_SCALE_BYTES;

// (w & m) | c as ONE three-input logic op.  Mask and magic are passed in registers: written with two
// literals the compiler emits two logic ops (one literal each), which costs a third of the kernel.
__device__ __forceinline__ uint32_t gv_and_or(uint32_t w, uint32_t m, uint32_t c) {
  uint32_t v;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(v) : "r"(w), "r"(m), "r"(c));
  return v;
}
// constants of the unpackers, kept in registers (see gv_and_or)
struct GvConst {
  uint32_t m0, m1, c;
  __device__ __forceinline__ GvConst(uint32_t m0_, uint32_t m1_, uint32_t c_) : m0(m0_), m1(m1_), c(c_) {
    asm volatile("" : "+r"(m0), "+r"(m1), "+r"(c));
  }
};
// Word of 8 codes -> four fp16 pairs for the A fragments (k.m0 = 0x000F000F, k.m1 = 0x00F000F0,
// k.c = 0x64006400 = fp16 1024.0 twice).
// With a 10-bit mantissa two neighbouring nibbles fit below the magic exponent, so a word needs one
// shift instead of three: v[0], v[2] = 1024 + c for codes (0,4), (2,6); v[1], v[3] = 1024 + 16 c for
// codes (1,5), (3,7).  The token operand carries 1/16 at the odd positions to match.
__device__ __forceinline__ void gv_unpack_h(uint32_t w, uint32_t (&v)[4], const GvConst& k) {
  const uint32_t t = w >> 8;
  v[0] = gv_and_or(w, k.m0, k.c);
  v[1] = gv_and_or(w, k.m1, k.c);
  v[2] = gv_and_or(t, k.m0, k.c);
  v[3] = gv_and_or(t, k.m1, k.c);
}
__device__ __forceinline__ void gv_mma_h(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void gv_mma0_h(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                          uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
      : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.0f));
}
__device__ __forceinline__ uint32_t gv_pack_h2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ float gv_h_lo(uint32_t v) { return __half2float(__ushort_as_half((unsigned short)(v & 0xFFFFu))); }
__device__ __forceinline__ float gv_h_hi(uint32_t v) { return __half2float(__ushort_as_half((unsigned short)(v >> 16))); }
__device__ __forceinline__ float gv_absmax8(const uint4& x, float m) {
  const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    m = fmaxf(m, fabsf(__uint_as_float(w[i] << 16)));
    m = fmaxf(m, fabsf(__uint_as_float(w[i] & 0xFFFF0000u)));
  }
  return m;
}

// shared-memory loads with 32-bit shared-space addresses (immediate offset OFF)
template <int OFF>
__device__ __forceinline__ uint2 gv_lds2(uint32_t addr) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0, %1}, [%2 + %3];" : "=r"(v.x), "=r"(v.y) : "r"(addr), "n"(OFF));
  return v;
}
template <int OFF>
__device__ __forceinline__ uint4 gv_lds4(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4 + %5];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr), "n"(OFF));
  return v;
}
template <int OFF>
__device__ __forceinline__ float gv_ldsf(uint32_t addr) {
  float v;
  asm volatile("ld.shared.f32 %0, [%1 + %2];" : "=f"(v) : "r"(addr), "n"(OFF));
  return v;
}
template <int OFF>
__device__ __forceinline__ float2 gv_ldsf2(uint32_t addr) {
  float2 v;
  asm volatile("ld.shared.v2.f32 {%0, %1}, [%2 + %3];" : "=f"(v.x), "=f"(v.y) : "r"(addr), "n"(OFF));
  return v;
}
template <int OFF>
__device__ __forceinline__ float4 gv_ldsf4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4 + %5];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr), "n"(OFF));
  return v;
}

// Release of a shared-memory buffer to the producer: one mbarrier arrival per warp, issued by lane 0 after
// __syncwarp().  What has to hold: every lane's ld.shared from the buffer has returned its data before the
// arrival is performed, because the arrival (release) is what the producer's try_wait (acquire) pairs with
// before it lets the async proxy (TMA / bulk copy) overwrite the buffer.  Program order alone does not give
// that to the assembler -- a load that is merely issued may still be in flight -- so the arrival's address
// operand is made to depend on `dep`, a value computed FROM the loaded registers (the sums they fed, see the
// call sites) and and-ed with a kernel parameter that is zero at run time but unknown at compile time.  The
// arrival therefore cannot issue before those registers are written, whatever the scheduling.
__device__ __forceinline__ uint32_t gv_dep(float a, float b, float c, float d, uint32_t zero) {
  return (__float_as_uint(a) ^ __float_as_uint(b) ^ __float_as_uint(c) ^ __float_as_uint(d)) & zero;
}
__device__ __forceinline__ void gv_release(uint32_t bar, uint32_t dep) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar + dep) : "memory");
}

// Waits of this kernel pass a suspend-time hint so that a waiting warp sleeps in hardware until the
// phase completes instead of polling: polling takes issue slots and ALU cycles from the warps of the
// same scheduler that still have work.  Still bounded: gives up after the cycle limit.
__device__ __forceinline__ bool gv_try_wait_hint(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(bar), "r"(parity), "r"(100000u) : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool gv_wait(uint32_t bar, uint32_t parity, int* status, long long limit) {
  if (gv_try_wait_hint(bar, parity)) return true;
  const long long t0 = clock64();
  while (!gv_try_wait_hint(bar, parity)) {
    if (clock64() - t0 > limit) {
      atomicExch(status, (int)QBLORA_ERR_TIMEOUT);
      return false;
    }
  }
  return true;
}

struct GtParams {
  int d_in, d_out, G, T;
  int n_rb, n_kc;            // row blocks of 32 rows, K tiles of 16 groups
  int stages;                // depth of the shared-memory ring (as many as fit)
  const __nv_bfloat16* X;
  void* Y;
  int y_dtype;
  int* status;
  // one-token kernel, split tail (see T1Walk): row blocks done whole, ways the rest is split, hand-over area
  int tail_first, tail_split;
  long long wait_limit;      // cycles after which a device-side wait gives up
  uint32_t zero;             // always 0; unknown to the compiler (see gv_release)
  uint32_t epoch;            // value a hand-over flag takes in this launch (never 0, differs from launch to launch)
  float* tail_partial;       // [tail row block][part][32 rows] fp32
  uint32_t* tail_flags;      // [tail row block][part]
};

// Row blocks of one CTA in the one-token kernel.  Whole row blocks b, b + G, ... below tail_first; then,
// when the remaining row blocks would occupy at most half of the CTAs, each of them is split along K
// into tail_split parts given to different CTAs (unit u = blockIdx.x: row block tail_first + u /
// split, part u % split), so the last round takes 1 / split of a round instead of a whole one.  Part
// 0 owns the row block: it adds the other parts' sums (handed over through global memory) and stores.
struct T1Walk {
  int rb, kc0, kc1, part;
  bool tail;
  int next_full, done_tail;
  __device__ T1Walk() : next_full((int)blockIdx.x), done_tail(0) {}
  __device__ bool next(const GtParams& p) {
    if (next_full < p.tail_first) {
      rb = next_full; kc0 = 0; kc1 = p.n_kc; part = 0; tail = false;
      next_full += gridDim.x;
      return true;
    }
    if (done_tail) return false;
    done_tail = 1;
    if (p.tail_split <= 1) {        // the rest as whole row blocks (at most one more per CTA)
      rb = next_full; kc0 = 0; kc1 = p.n_kc; part = 0; tail = false;
      return rb < p.n_rb;
    }
    const int u = (int)blockIdx.x;
    rb = p.tail_first + u / p.tail_split;
    part = u % p.tail_split;
    if (rb >= p.n_rb) return false;
    kc0 = p.n_kc * part / p.tail_split; kc1 = p.n_kc * (part + 1) / p.tail_split;
    tail = true;
    return true;
  }
};

// ---------------------------------------------------------------------------------------------------
// One token.  x is converted once per CTA into fp16 fragments in shared memory (each group of 64 values
// with its own power-of-two prescale), the row blocks are the outer loop and only column 0 of the
// accumulator tile is kept.
constexpr int T1_RED_BYTES = GT_WARPS * GT_ROWS * 4;        // [16 warps][32 rows]
constexpr int T1_MAX_STAGES = 10;

__global__ void __launch_bounds__(GT_THREADS, 1)
lowbit_gemv_t1_kernel(const __grid_constant__ CUtensorMap tm_c, const __grid_constant__ CUtensorMap tm_a,
                      const __grid_constant__ CUtensorMap tm_b, const __grid_constant__ GtParams p) {
  const int STAGES = p.stages;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gbase = smem_raw + (base - raw);
  const uint32_t red_off = STAGES * GT_STAGE_BYTES;
  float* red = reinterpret_cast<float*>(gbase + red_off);                 // [16 warps][32 rows]
  const uint32_t bar_off = red_off + T1_RED_BYTES;
  const uint32_t bars = base + bar_off;
  auto full = [&](int s) { return bars + 8u * s; };
  auto empty = [&](int s) { return bars + 8u * (STAGES + s); };
  const uint32_t red_done = bars + 8u * (2 * STAGES);       // all 16 warps have written their sums of the row block
  const uint32_t red_free = bars + 8u * (2 * STAGES + 1);   // the summing warp has read them
  // ss[G] = (1024 P 2^e, R 2^e, 2^e, -) per group (P = sum of the fp16 fragment values, R = sum of the
  // scaled x, 2^-e the group's prescale), then
  // xs[G][4 tg][8 words] = fp16 fragments, then 128 zero bytes
  const uint32_t ss_off = bar_off + 256;
  float* ss = reinterpret_cast<float*>(gbase + ss_off);
  const uint32_t xs_off = ss_off + (uint32_t)p.G * 16;
  uint4* xs = reinterpret_cast<uint4*>(gbase + xs_off);
  const uint32_t zero_off = xs_off + (uint32_t)p.G * 128;

  // a successor launched as a programmatic dependent may start on every SM this grid has left
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    if (blockIdx.x == 0) *p.status = 0;   // any give-up below is written at least a wait limit later
    for (int s = 0; s < STAGES; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), GT_WARPS); }
    mbar_init(red_done, GT_WARPS);
    mbar_init(red_free, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  if (warp == GT_WARPS) {
    // ------------------------------------------------------------------ producer (one lane)
    if (lane == 0) {
      uint32_t it = 0, ph = 0;
      int s = 0;
      bool ok = true;
      T1Walk walk;
      while (ok && walk.next(p)) {
        const int rb = walk.rb;
        for (int kc = walk.kc0; kc < walk.kc1; ++kc, ++it) {
          if (!gv_wait(empty(s), ph ^ 1u, p.status, p.wait_limit)) { ok = false; break; }
          const uint32_t st = base + s * GT_STAGE_BYTES;
          mbar_arrive_expect_tx(full(s), GT_STAGE_BYTES);
#pragma unroll
          for (int j = 0; j < 4; ++j)   // four groups = 128 bytes = 32 u32 per row and box
            tma_load_2d(st + j * 4096, &tm_c, full(s), (kc * GT_GROUPS + j * 4) * 8, rb * GT_ROWS);
          tma_load_2d(st + GT_CODE_BYTES, &tm_a, full(s), kc * GT_GROUPS, rb * GT_ROWS);
          tma_load_2d(st + GT_CODE_BYTES + GT_SCALE_BYTES, &tm_b, full(s), kc * GT_GROUPS, rb * GT_ROWS);
          if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
      }
      if (!ok) {   // give copies already in flight a bounded chance to land before the CTA exits
        const uint32_t lo = it > (uint32_t)STAGES ? it - STAGES : 0;
        for (uint32_t j = lo; j < it; ++j) gv_wait(full(j % STAGES), (j / STAGES) & 1u, p.status, p.wait_limit);
      }
    }
  } else {
    // ------------------------------------------------------------------ compute warps
    const int g = lane >> 2, tg = lane & 3;
    // The weights are constants, x and Y are not: in a chain of launches (one decode step) this kernel may
    // have been started before its predecessor finished (programmatic dependent launch), so the producer
    // streams weights at once while everything that reads x or writes results waits here.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // ---- once per CTA, while the first tiles are in flight: fragments and group sums of x.
    // Item = (group, tg): 16 values of x; the four tg lanes of an item are neighbours.  Every group's
    // 64 values get their own power-of-two prescale 2^-e (max |x| 2^-e in [2^14, 2^15)), so no pass over
    // all of x and no CTA-wide reduction is needed first.
    const int items = p.G * 4;
    if (tid < 32) reinterpret_cast<uint32_t*>(gbase + zero_off)[tid] = 0u;
    for (int i0 = 0; i0 < items; i0 += GT_WARPS * 32) {
      const int idx = i0 + tid;
      const bool live = idx < items;
      const int q = live ? idx : 0;
      const uint4* src = reinterpret_cast<const uint4*>(p.X + q * 16);
      const uint4 x0 = __ldg(src), x1 = __ldg(src + 1);
      float am = gv_absmax8(x1, gv_absmax8(x0, 0.0f));
      am = fmaxf(am, __shfl_xor_sync(0xFFFFFFFFu, am, 1));
      am = fmaxf(am, __shfl_xor_sync(0xFFFFFFFFu, am, 2));
      int e = (int)((__float_as_uint(am) >> 23) & 0xFFu) - 127 - 14;
      e = e < -100 ? -100 : (e > 120 ? 120 : e);
      const float up = __uint_as_float((uint32_t)(127 + e) << 23);
      const float in_scale = __uint_as_float((uint32_t)(127 - e) << 23), in_scale16 = in_scale * 0.0625f;
      const uint32_t xw[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
      uint32_t f[8];
      float ps = 0.0f, rs = 0.0f;   // sum of fragment values; sum of scaled x as the fragments hold it
#pragma unroll
      for (int wd = 0; wd < 2; ++wd)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          // word wd holds x at positions 0..7 as pairs (2j, 2j+1) in xw[4 wd + j]; fragment register
          // 2 (2 wd + h) pairs positions (2h, 2h+4), the next one (2h+1, 2h+5) scaled by 1/16
          const uint32_t wa = xw[4 * wd + h], wb = xw[4 * wd + h + 2];
          const uint32_t ev = gv_pack_h2(__uint_as_float(wa << 16) * in_scale, __uint_as_float(wb << 16) * in_scale);
          const uint32_t od = gv_pack_h2(__uint_as_float(wa & 0xFFFF0000u) * in_scale16,
                                         __uint_as_float(wb & 0xFFFF0000u) * in_scale16);
          f[2 * (2 * wd + h)] = ev;
          f[2 * (2 * wd + h) + 1] = od;
          const float se = gv_h_lo(ev) + gv_h_hi(ev), so = gv_h_lo(od) + gv_h_hi(od);
          ps += se + so;
          rs += se + 16.0f * so;
        }
      ps += __shfl_xor_sync(0xFFFFFFFFu, ps, 1); rs += __shfl_xor_sync(0xFFFFFFFFu, rs, 1);
      ps += __shfl_xor_sync(0xFFFFFFFFu, ps, 2); rs += __shfl_xor_sync(0xFFFFFFFFu, rs, 2);
      if (live) {
        if ((q & 3) == 0) *reinterpret_cast<float4*>(ss + (q >> 2) * 4) = make_float4(1024.0f * ps * up, rs * up, up, 0.0f);
        xs[q * 2] = make_uint4(f[0], f[1], f[2], f[3]);
        xs[q * 2 + 1] = make_uint4(f[4], f[5], f[6], f[7]);
      }
    }
    asm volatile("bar.sync 1, 512;" ::: "memory");

    // byte offsets inside a stage that do not depend on the stage: the thread's 8 bytes of codes of the
    // warp's group in row g (rows g + 8 q: + 1024 q, same swizzle phase) and its scale entries (rows g + 8 q: + 512 q)
    const uint32_t code_off = ((uint32_t)warp >> 2) * 4096u + (uint32_t)g * 128u +
                              ((((((uint32_t)warp & 3u) << 1) | ((uint32_t)tg >> 1)) ^ (uint32_t)g) << 4) +
                              (((uint32_t)tg & 1u) << 3);
    // alpha / beta tiles are [32 rows][16 groups] fp32 with the 64-byte swizzle (16-byte chunk index
    // xor (row / 2) % 4), which spreads the eight rows a warp reads at once over eight banks
    const uint32_t scale_off = GT_CODE_BYTES + (uint32_t)g * 64u +
                               ((((uint32_t)warp >> 2) ^ (((uint32_t)g >> 1) & 3u)) << 4) + ((uint32_t)warp & 3u) * 4u;
    // B fragment column = token: only the lanes with g == 0 hold the token, the others read the zero
    // block (stride 0) instead of selecting zeros
    const uint32_t xs_addr = base + (g == 0 ? xs_off : zero_off) + (uint32_t)tg * 32u;
    const uint32_t xs_stride = g == 0 ? 128u : 0u;
    const uint32_t ss_addr = base + ss_off;
    uint32_t rph = 0, rcount = 0;   // phase of the reduction barriers; row blocks done
    const GvConst kc_(0x000F000Fu, 0x00F000F0u, 0x64006400u);
    bool ok = true;        // after a timed-out wait the warp keeps walking its loops (so the CTA
                           // barriers still match) but no longer waits or computes
    int s = 0;
    uint32_t ph = 0;
    T1Walk walk;
    while (walk.next(p)) {
      const int rb = walk.rb;
      float y[2][2] = {{0.0f, 0.0f}, {0.0f, 0.0f}};    // [row tile][row g, row g + 8], token 0 (lanes tg == 0)
      for (int kc = walk.kc0; kc < walk.kc1; ++kc) {
        if (ok && !gv_wait(full(s), ph, p.status, p.wait_limit)) ok = false;
        const int grp = kc * GT_GROUPS + warp;
        if (ok) {
          if (grp < p.G) {                                   // warp-uniform
            const uint32_t sb = base + (uint32_t)s * GT_STAGE_BYTES;
            const uint32_t ca = sb + code_off, sa = sb + scale_off;
            const float4 sg = gv_ldsf4<0>(ss_addr + (uint32_t)grp * 16u);     // (1024 P 2^e, R 2^e, 2^e, -) of the group
            const uint32_t xa = xs_addr + (uint32_t)grp * xs_stride;
            const uint4 x0 = gv_lds4<0>(xa), x1 = gv_lds4<16>(xa);
            // all shared-memory loads of the group first (they stay in program order), then the math
            uint2 w0[2], w1[2];
            float a0[2], a1[2], b0[2], b1[2];
            w0[0] = gv_lds2<0>(ca); w1[0] = gv_lds2<1024>(ca); w0[1] = gv_lds2<2048>(ca); w1[1] = gv_lds2<3072>(ca);
            a0[0] = gv_ldsf<0>(sa); a1[0] = gv_ldsf<512>(sa); a0[1] = gv_ldsf<1024>(sa); a1[1] = gv_ldsf<1536>(sa);
            b0[0] = gv_ldsf<GT_SCALE_BYTES>(sa); b1[0] = gv_ldsf<GT_SCALE_BYTES + 512>(sa);
            b0[1] = gv_ldsf<GT_SCALE_BYTES + 1024>(sa); b1[1] = gv_ldsf<GT_SCALE_BYTES + 1536>(sa);
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
              uint32_t va[2][4], vb[2][4];      // [word][pair] for rows g + 16 mt (va) and g + 16 mt + 8 (vb)
              gv_unpack_h(w0[mt].x, va[0], kc_); gv_unpack_h(w0[mt].y, va[1], kc_);
              gv_unpack_h(w1[mt].x, vb[0], kc_); gv_unpack_h(w1[mt].y, vb[1], kc_);
              float acc[4];
              gv_mma0_h(acc, va[0][0], vb[0][0], va[0][1], vb[0][1], x0.x, x0.y);
              gv_mma_h(acc, va[0][2], vb[0][2], va[0][3], vb[0][3], x0.z, x0.w);
              gv_mma_h(acc, va[1][0], vb[1][0], va[1][1], vb[1][1], x1.x, x1.y);
              gv_mma_h(acc, va[1][2], vb[1][2], va[1][3], vb[1][3], x1.z, x1.w);
              // alpha (2^e acc - 1024 P 2^e) + beta R 2^e; column 0 of the accumulator tile is held by the tg == 0 lanes
              y[mt][0] = fmaf(a0[mt], fmaf(acc[0], sg.z, -sg.x), fmaf(b0[mt], sg.y, y[mt][0]));
              y[mt][1] = fmaf(a1[mt], fmaf(acc[2], sg.z, -sg.x), fmaf(b1[mt], sg.y, y[mt][1]));
            }
          }
          __syncwarp();
          // y[][] are sums over everything this lane loaded from the stage (codes through the MMAs, alpha, beta)
          if (lane == 0) gv_release(empty(s), gv_dep(y[0][0], y[0][1], y[1][0], y[1][1], p.zero));
        }
        if (++s == STAGES) { s = 0; ph ^= 1u; }
      }
      // End of the row block, without a CTA-wide barrier.  Every warp writes its partial sums into its
      // slot (once the warp that summed the previous row block has let go of the buffer) and arrives
      // on red_done; the sixteen slots are then summed in slot order (deterministic) and stored by
      // warp (row block count) % 16, which is the only warp that waits for the others.
      if (ok && !gv_wait(red_free, rph ^ 1u, p.status, p.wait_limit)) ok = false;
      float* my_red = red + warp * GT_ROWS;
      if (tg == 0) {
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) { my_red[mt * 16 + g] = y[mt][0]; my_red[mt * 16 + g + 8] = y[mt][1]; }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(red_done);
      if (warp == (int)(rcount & 15u)) {
        if (ok && !gv_wait(red_done, rph, p.status, p.wait_limit)) ok = false;
        float a = 0.0f;
#pragma unroll
        for (int ww = 0; ww < GT_WARPS; ++ww) a += red[ww * GT_ROWS + lane];
        __syncwarp();
        if (lane == 0) gv_release(red_free, gv_dep(a, a, a, 0.0f, p.zero));
        if (walk.tail) {
          const int slot = (rb - p.tail_first) * p.tail_split;
          if (walk.part != 0) {
            // hand this K range's sums to the owner: stores, fence, then the flag (this launch's epoch)
            p.tail_partial[(slot + walk.part) * GT_ROWS + lane] = a;
            __threadfence();
            __syncwarp();
            if (lane == 0) atomicExch(p.tail_flags + slot + walk.part, p.epoch);
            ++rcount; rph ^= 1u;
            continue;
          }
          for (int part = 1; part < p.tail_split; ++part) {      // bounded wait, then add in part order
            uint32_t seen = p.epoch;
            if (lane == 0 && ok) {
              const long long w0 = clock64();
              while ((seen = *reinterpret_cast<volatile uint32_t*>(p.tail_flags + slot + part)) != p.epoch) {
                __nanosleep(100);
                if (clock64() - w0 > p.wait_limit) { atomicExch(p.status, (int)QBLORA_ERR_TIMEOUT); break; }
              }
            }
            seen = __shfl_sync(0xFFFFFFFFu, seen, 0);
            if (seen != p.epoch) ok = false;
            __threadfence();
            a += __ldcg(p.tail_partial + (slot + part) * GT_ROWS + lane);
            // Consumed: put the flag back to 0, which is never an epoch.  A launch replayed from a CUDA graph
            // carries the epoch it was captured with, so without this the flag left by the previous replay
            // would already match and the owner would read sums that are not there yet.  The next writer of
            // this flag is a later launch, whose compute warps start only after this grid has completed.
            if (lane == 0) atomicExch(p.tail_flags + slot + part, 0u);
          }
        }
        const int o = rb * GT_ROWS + lane;                // lane = row of the block
        if (o < p.d_out) {
          if (p.y_dtype == QBLORA_BF16) reinterpret_cast<__nv_bfloat16*>(p.Y)[o] = __float2bfloat16_rn(a);
          else reinterpret_cast<float*>(p.Y)[o] = a;
        }
      }
      ++rcount;
      rph ^= 1u;
    }
  }
  __syncthreads();
}

constexpr size_t GT_SMEM_MAX = 227 * 1024;
// dynamic shared memory besides the stage ring: alignment slack, reduction buffer, barriers, group
// sums, fragments, zero block
size_t t1_fixed_smem(int G) { return 1024 + T1_RED_BYTES + 256 + (size_t)G * 16 + (size_t)G * 128 + 128; }
int t1_stages(int G) {   // ring depth that fits; 0 if fewer than six stages would be left
  const size_t fixed = t1_fixed_smem(G);
  if (fixed + 6 * (size_t)GT_STAGE_BYTES > GT_SMEM_MAX) return 0;
  const int n = (int)((GT_SMEM_MAX - fixed) / GT_STAGE_BYTES);
  return n < T1_MAX_STAGES ? n : T1_MAX_STAGES;
}
int t1_launch(const CUtensorMap& tm_c, const CUtensorMap& tm_a, const CUtensorMap& tm_b, GtParams p, int grid,
              cudaStream_t st, bool chain) {
  p.stages = t1_stages(p.G);
  const size_t smem = t1_fixed_smem(p.G) + (size_t)p.stages * GT_STAGE_BYTES;
  QB_CUDA(cudaFuncSetAttribute(lowbit_gemv_t1_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)grid); cfg.blockDim = dim3(GT_THREADS); cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = chain ? 1 : 0;
  QB_CUDA(cudaLaunchKernelEx(&cfg, lowbit_gemv_t1_kernel, tm_c, tm_a, tm_b, p));
  return QBLORA_OK;
}

// ---------------------------------------------------------------------------------------------------
// K-outer variant for 2..16 tokens (and for one token when its fragments do not fit shared memory).  A small kernel first turns x into fp16 MMA fragments in the
// workspace: per K tile a contiguous block [16 groups][NTOK tokens][4 quarters][32 B] plus, per group
// and token, (1024 P 2^e, R 2^e, 2^e, 0), where 2^-e is that 64-value slice's own power-of-two
// prescale, P the sum of the fragment values and R the sum of the scaled x (so no pass over all of x
// is needed and tokens of very different magnitude do not share a scale).  The main kernel makes the
// K tiles the OUTER loop: a loader warp brings a K tile's fragment block into shared memory once
// (bulk copy, double-buffered) while the producer warp streams the weight tiles of the CTA's RB row
// blocks for that K tile through the ring; the two never wait for each other, so the ring stays full
// across K tiles (with one lane doing both, the look-ahead was one K tile: 40 -> 32 us at 16 tokens).
// A warp takes its group's fragments into registers once per K tile and reuses them for the RB row
// blocks, so the main loop has no global loads, no byte permutes and the cheaper fp16 unpack, and x
// crosses L2 -> SM once per RB row blocks.  The RB accumulators stay in registers.
template <int NT>
struct KoCfg {
  static constexpr int NTOK = NT * 8;
  static constexpr int RB = NT == 1 ? 4 : 2;                       // row blocks per pass (register budget)
  static constexpr int XBUF_BYTES = GT_GROUPS * NTOK * 128;        // fragments of one K tile
  static constexpr int SBUF_BYTES = GT_GROUPS * NTOK * 16;         // float4 per group and token
  static constexpr int KT_BYTES = XBUF_BYTES + SBUF_BYTES;         // one K tile's block in the workspace
  static constexpr int RED_BYTES = GT_WARPS * GT_ROWS * NTOK * 4;
  static constexpr int FIXED = 1024 + 2 * KT_BYTES + RED_BYTES + 512;
};

__device__ __forceinline__ void gv_bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// one thread per (K tile, group, token, quarter): 16 values of x -> 32 bytes of fragments
template <int NT>
__global__ void __launch_bounds__(256) x_prepare_kernel(const __nv_bfloat16* __restrict__ X, int T, int d_in, int G,
                                                        int n_kc, uint8_t* __restrict__ out) {
  using Cfg = KoCfg<NT>;
  constexpr int NTOK = Cfg::NTOK;
  // the main kernel is launched as a programmatic dependent: it may start (set up, stream weights) now and
  // waits for this grid's completion only before it reads the fragments
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // In a chain of launches this grid may itself have started early: the previous launch may still read
  // the fragment area (same workspace) and may still be producing x.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int idx = blockIdx.x * 256 + threadIdx.x;
  const int total = n_kc * GT_GROUPS * NTOK * 4;
  const bool in_range = idx < total;
  const int q = in_range ? idx : 0;
  const int tg = q & 3, t = (q >> 2) % NTOK, gl = ((q >> 2) / NTOK) % GT_GROUPS, kc = (q >> 2) / (NTOK * GT_GROUPS);
  const int grp = kc * GT_GROUPS + gl;
  uint4 xa = make_uint4(0, 0, 0, 0), xb = make_uint4(0, 0, 0, 0);
  if (in_range && t < T && grp < G) {
    const uint4* src = reinterpret_cast<const uint4*>(X + (int64_t)t * d_in + grp * 64 + tg * 16);
    xa = __ldg(src); xb = __ldg(src + 1);
  }
  float am = gv_absmax8(xb, gv_absmax8(xa, 0.0f));
  am = fmaxf(am, __shfl_xor_sync(0xFFFFFFFFu, am, 1));
  am = fmaxf(am, __shfl_xor_sync(0xFFFFFFFFu, am, 2));
  int e = (int)((__float_as_uint(am) >> 23) & 0xFFu) - 127 - 14;     // max |x| 2^-e in [2^14, 2^15)
  e = e < -100 ? -100 : (e > 120 ? 120 : e);
  const float up = __uint_as_float((uint32_t)(127 + e) << 23), dn = __uint_as_float((uint32_t)(127 - e) << 23);
  const float dn16 = dn * 0.0625f;
  const uint32_t xw[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
  uint32_t f[8];
  float ps = 0.0f, rs = 0.0f;   // sum of fragment values; sum of scaled x as the fragments hold it
#pragma unroll
  for (int wd = 0; wd < 2; ++wd)
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const uint32_t wa = xw[4 * wd + h], wb = xw[4 * wd + h + 2];
      const uint32_t ev = gv_pack_h2(__uint_as_float(wa << 16) * dn, __uint_as_float(wb << 16) * dn);
      const uint32_t od = gv_pack_h2(__uint_as_float(wa & 0xFFFF0000u) * dn16, __uint_as_float(wb & 0xFFFF0000u) * dn16);
      f[2 * (2 * wd + h)] = ev;
      f[2 * (2 * wd + h) + 1] = od;
      const float se = gv_h_lo(ev) + gv_h_hi(ev), so = gv_h_lo(od) + gv_h_hi(od);
      ps += se + so;
      rs += se + 16.0f * so;
    }
  ps += __shfl_xor_sync(0xFFFFFFFFu, ps, 1); rs += __shfl_xor_sync(0xFFFFFFFFu, rs, 1);
  ps += __shfl_xor_sync(0xFFFFFFFFu, ps, 2); rs += __shfl_xor_sync(0xFFFFFFFFu, rs, 2);
  if (in_range) {
    uint8_t* blk = out + (size_t)kc * Cfg::KT_BYTES;
    const uint32_t item = (uint32_t)(gl * NTOK + t);
    uint4* dst = reinterpret_cast<uint4*>(blk + item * 128u + (uint32_t)tg * 32u);
    dst[0] = make_uint4(f[0], f[1], f[2], f[3]);
    dst[1] = make_uint4(f[4], f[5], f[6], f[7]);
    if (tg == 0) *reinterpret_cast<float4*>(blk + Cfg::XBUF_BYTES + item * 16u) = make_float4(1024.0f * ps * up, rs * up, up, 0.0f);
  }
}

template <int NT>
__global__ void __launch_bounds__(KO_THREADS, 1)
lowbit_gemv_ko_kernel(const __grid_constant__ CUtensorMap tm_c, const __grid_constant__ CUtensorMap tm_a,
                      const __grid_constant__ CUtensorMap tm_b, const __grid_constant__ GtParams p,
                      const uint8_t* __restrict__ xfrag) {
  using Cfg = KoCfg<NT>;
  constexpr int NTOK = Cfg::NTOK, RB = Cfg::RB;
  const int STAGES = p.stages;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gbase = smem_raw + (base - raw);
  const uint32_t xbuf_off = STAGES * GT_STAGE_BYTES;                    // [2] x (fragments, then float4 per group, token)
  const uint32_t red_off = xbuf_off + 2 * Cfg::KT_BYTES;
  float* red = reinterpret_cast<float*>(gbase + red_off);               // [16 warps][32 rows][NTOK]
  const uint32_t bars = base + red_off + Cfg::RED_BYTES;
  auto full = [&](int s) { return bars + 8u * s; };
  auto empty = [&](int s) { return bars + 8u * (STAGES + s); };
  const uint32_t red_done = bars + 8u * (2 * STAGES);
  const uint32_t red_free = bars + 8u * (2 * STAGES + 1);
  auto xfull = [&](uint32_t b) { return bars + 8u * (2 * STAGES + 2 + b); };
  auto xempty = [&](uint32_t b) { return bars + 8u * (2 * STAGES + 4 + b); };

  // a successor launched as a programmatic dependent may start on every SM this grid has left
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    if (blockIdx.x == 0) *p.status = 0;   // any give-up below is written at least a wait limit later
    for (int s = 0; s < STAGES; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), GT_WARPS); }
    mbar_init(red_done, GT_WARPS);
    mbar_init(red_free, p.T);
    for (uint32_t b = 0; b < 2; ++b) { mbar_init(xfull(b), 1); mbar_init(xempty(b), GT_WARPS); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  const int n_pass = (p.n_rb + gridDim.x * RB - 1) / (gridDim.x * RB);   // passes of RB row blocks per CTA

  if (warp == GT_WARPS) {
    // ------------------------------------------------------------------ weight producer (one lane)
    // The weights do not depend on the kernel that prepares the fragments, and the ring never waits
    // for a fragment buffer: all of its stages stay in flight whatever the state of the K tile.
    if (lane == 0) {
      uint32_t it = 0, ph = 0;
      int s = 0;
      bool ok = true;
      for (int pass = 0; pass < n_pass && ok; ++pass) {
        if (pass * RB * (int)gridDim.x + (int)blockIdx.x >= p.n_rb) break;   // no row block left for this CTA
        for (int kc = 0; kc < p.n_kc && ok; ++kc) {
          for (int j = 0; j < RB; ++j) {
            const int rb = (pass * RB + j) * gridDim.x + blockIdx.x;
            if (rb >= p.n_rb) break;
            if (!gv_wait(empty(s), ph ^ 1u, p.status, p.wait_limit)) { ok = false; break; }
            const uint32_t st = base + s * GT_STAGE_BYTES;
            mbar_arrive_expect_tx(full(s), GT_STAGE_BYTES);
#pragma unroll
            for (int q = 0; q < 4; ++q)
              tma_load_2d(st + q * 4096, &tm_c, full(s), (kc * GT_GROUPS + q * 4) * 8, rb * GT_ROWS);
            tma_load_2d(st + GT_CODE_BYTES, &tm_a, full(s), kc * GT_GROUPS, rb * GT_ROWS);
            tma_load_2d(st + GT_CODE_BYTES + GT_SCALE_BYTES, &tm_b, full(s), kc * GT_GROUPS, rb * GT_ROWS);
            ++it;
            if (++s == STAGES) { s = 0; ph ^= 1u; }
          }
        }
      }
      if (!ok) {   // give copies already in flight a bounded chance to land before the CTA exits
        const uint32_t lo = it > (uint32_t)STAGES ? it - STAGES : 0;
        for (uint32_t j = lo; j < it; ++j) gv_wait(full(j % STAGES), (j / STAGES) & 1u, p.status, p.wait_limit);
      }
    }
  } else if (warp == GT_WARPS + 1) {
    // ------------------------------------------------------------------ fragment loader (one lane)
    if (lane == 0) {
      asm volatile("griddepcontrol.wait;" ::: "memory");   // the fragments are complete and visible
      uint32_t xit = 0;
      bool ok = true;
      for (int pass = 0; pass < n_pass && ok; ++pass) {
        if (pass * RB * (int)gridDim.x + (int)blockIdx.x >= p.n_rb) break;
        for (int kc = 0; kc < p.n_kc; ++kc, ++xit) {
          const uint32_t xb = xit & 1u;
          if (!gv_wait(xempty(xb), ((xit >> 1) & 1u) ^ 1u, p.status, p.wait_limit)) { ok = false; break; }
          mbar_arrive_expect_tx(xfull(xb), Cfg::KT_BYTES);
          gv_bulk_load(base + xbuf_off + xb * Cfg::KT_BYTES, xfrag + (size_t)kc * Cfg::KT_BYTES, Cfg::KT_BYTES, xfull(xb));
        }
      }
      if (!ok) {
        const uint32_t xlo = xit > 2u ? xit - 2u : 0u;
        for (uint32_t j = xlo; j < xit; ++j) gv_wait(xfull(j & 1u), (j >> 1) & 1u, p.status, p.wait_limit);
      }
    }
  } else {
    // ------------------------------------------------------------------ compute warps
    const int g = lane >> 2, tg = lane & 3;
    const uint32_t code_off = ((uint32_t)warp >> 2) * 4096u + (uint32_t)g * 128u +
                              ((((((uint32_t)warp & 3u) << 1) | ((uint32_t)tg >> 1)) ^ (uint32_t)g) << 4) +
                              (((uint32_t)tg & 1u) << 3);
    const uint32_t scale_off = GT_CODE_BYTES + (uint32_t)g * 64u +
                               ((((uint32_t)warp >> 2) ^ (((uint32_t)g >> 1) & 3u)) << 4) + ((uint32_t)warp & 3u) * 4u;
    const GvConst kc_(0x000F000Fu, 0x00F000F0u, 0x64006400u);
    // B fragment of lane (g, tg) = token g (+ 8 n), quarter tg, of this warp's group
    const uint32_t xrd = base + xbuf_off + ((uint32_t)warp * NTOK + (uint32_t)g) * 128u + (uint32_t)tg * 32u;
    const uint32_t srd = base + xbuf_off + Cfg::XBUF_BYTES + ((uint32_t)warp * NTOK + 2u * (uint32_t)tg) * 16u;
    bool ok = true;
    int s = 0;
    uint32_t ph = 0, rph = 0, rcount = 0, xit = 0;
    for (int pass = 0; pass < n_pass; ++pass) {
      if (pass * RB * (int)gridDim.x + (int)blockIdx.x >= p.n_rb) break;
      float y[RB][NT][2][4];
#pragma unroll
      for (int j = 0; j < RB; ++j)
#pragma unroll
        for (int n = 0; n < NT; ++n)
#pragma unroll
          for (int mt = 0; mt < 2; ++mt) { y[j][n][mt][0] = y[j][n][mt][1] = y[j][n][mt][2] = y[j][n][mt][3] = 0.0f; }
      for (int kc = 0; kc < p.n_kc; ++kc, ++xit) {
        // ---- this warp's group of the K tile: fragments and offsets into registers, once for all row blocks
        const uint32_t xb = xit & 1u;
        if (ok && !gv_wait(xfull(xb), (xit >> 1) & 1u, p.status, p.wait_limit)) ok = false;
        uint32_t f[NT][8];
        float4 sg[NT][2];
#pragma unroll
        for (int n = 0; n < NT; ++n) {
          const uint32_t xa_ = xrd + xb * Cfg::KT_BYTES + (uint32_t)n * (8u * 128u);
          const uint4 x0 = gv_lds4<0>(xa_), x1 = gv_lds4<16>(xa_);
          f[n][0] = x0.x; f[n][1] = x0.y; f[n][2] = x0.z; f[n][3] = x0.w;
          f[n][4] = x1.x; f[n][5] = x1.y; f[n][6] = x1.z; f[n][7] = x1.w;
          const uint32_t sa_ = srd + xb * Cfg::KT_BYTES + (uint32_t)n * (8u * 16u);
          sg[n][0] = gv_ldsf4<0>(sa_); sg[n][1] = gv_ldsf4<16>(sa_);
        }
        __syncwarp();
        const bool group_live = kc * GT_GROUPS + warp < p.G;
#pragma unroll
        for (int j = 0; j < RB; ++j) {
          const int rb = (pass * RB + j) * gridDim.x + blockIdx.x;
          if (rb >= p.n_rb) break;
          if (ok && !gv_wait(full(s), ph, p.status, p.wait_limit)) ok = false;
          if (ok) {
            if (group_live) {
              const uint32_t sb = base + (uint32_t)s * GT_STAGE_BYTES;
              const uint32_t ca = sb + code_off, sa = sb + scale_off;
              uint2 w0[2], w1[2];
              float a0[2], a1[2], b0[2], b1[2];
              w0[0] = gv_lds2<0>(ca); w1[0] = gv_lds2<1024>(ca); w0[1] = gv_lds2<2048>(ca); w1[1] = gv_lds2<3072>(ca);
              a0[0] = gv_ldsf<0>(sa); a1[0] = gv_ldsf<512>(sa); a0[1] = gv_ldsf<1024>(sa); a1[1] = gv_ldsf<1536>(sa);
              b0[0] = gv_ldsf<GT_SCALE_BYTES>(sa); b1[0] = gv_ldsf<GT_SCALE_BYTES + 512>(sa);
              b0[1] = gv_ldsf<GT_SCALE_BYTES + 1024>(sa); b1[1] = gv_ldsf<GT_SCALE_BYTES + 1536>(sa);
#pragma unroll
              for (int mt = 0; mt < 2; ++mt) {
                uint32_t va[2][4], vb[2][4];
                gv_unpack_h(w0[mt].x, va[0], kc_); gv_unpack_h(w0[mt].y, va[1], kc_);
                gv_unpack_h(w1[mt].x, vb[0], kc_); gv_unpack_h(w1[mt].y, vb[1], kc_);
#pragma unroll
                for (int n = 0; n < NT; ++n) {
                  float acc[4];
                  gv_mma0_h(acc, va[0][0], vb[0][0], va[0][1], vb[0][1], f[n][0], f[n][1]);
                  gv_mma_h(acc, va[0][2], vb[0][2], va[0][3], vb[0][3], f[n][2], f[n][3]);
                  gv_mma_h(acc, va[1][0], vb[1][0], va[1][1], vb[1][1], f[n][4], f[n][5]);
                  gv_mma_h(acc, va[1][2], vb[1][2], va[1][3], vb[1][3], f[n][6], f[n][7]);
                  // alpha (2^e acc - 1024 P 2^e) + beta R 2^e for tokens 2tg (sg[n][0]) and 2tg+1 (sg[n][1])
                  y[j][n][mt][0] = fmaf(a0[mt], fmaf(acc[0], sg[n][0].z, -sg[n][0].x), fmaf(b0[mt], sg[n][0].y, y[j][n][mt][0]));
                  y[j][n][mt][1] = fmaf(a0[mt], fmaf(acc[1], sg[n][1].z, -sg[n][1].x), fmaf(b0[mt], sg[n][1].y, y[j][n][mt][1]));
                  y[j][n][mt][2] = fmaf(a1[mt], fmaf(acc[2], sg[n][0].z, -sg[n][0].x), fmaf(b1[mt], sg[n][0].y, y[j][n][mt][2]));
                  y[j][n][mt][3] = fmaf(a1[mt], fmaf(acc[3], sg[n][1].z, -sg[n][1].x), fmaf(b1[mt], sg[n][1].y, y[j][n][mt][3]));
                }
              }
            }
            __syncwarp();
            // sums over everything this lane loaded from the stage: rows g (…[0]) and g + 8 (…[2]) of both row tiles
            if (lane == 0) gv_release(empty(s), gv_dep(y[j][0][0][0], y[j][0][0][2], y[j][0][1][0], y[j][0][1][2], p.zero));
          }
          if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
        // The fragment buffer is released here, after the K tile's row blocks.  The arrival depends on the
        // first row block's sums of every token tile (they consumed f[n][0..7] through the MMAs and both
        // sg[n][] entries) and, for a warp whose group lies beyond G and did no arithmetic, on the last loaded
        // registers themselves.
        __syncwarp();
        if (ok && lane == 0) {
          uint32_t dep = __float_as_uint(sg[0][1].w) ^ __float_as_uint(sg[NT - 1][1].w) ^ f[0][7] ^ f[NT - 1][7];
#pragma unroll
          for (int n = 0; n < NT; ++n) dep ^= __float_as_uint(y[0][n][0][0]) ^ __float_as_uint(y[0][n][0][1]);
          gv_release(xempty(xb), dep & p.zero);
        }
      }
      // ---- end of the pass: the RB row blocks are summed over the warps one after the other
#pragma unroll
      for (int j = 0; j < RB; ++j) {
        const int rb = (pass * RB + j) * gridDim.x + blockIdx.x;
        if (rb >= p.n_rb) break;
        if (ok && !gv_wait(red_free, rph ^ 1u, p.status, p.wait_limit)) ok = false;
        float* my_red = red + warp * GT_ROWS * NTOK;
#pragma unroll
        for (int n = 0; n < NT; ++n)
#pragma unroll
          for (int mt = 0; mt < 2; ++mt) {
            // slot layout [token][row ^ 8 (token / 2 mod 4)]: these stores and the sums below are free of bank conflicts
            float* r0 = my_red + (n * 8 + 2 * tg) * GT_ROWS;
            const int ra = (mt * 16 + g) ^ (tg << 3), rc = ra ^ 8;   // rows g and g + 8 of the row tile
            r0[ra] = y[j][n][mt][0]; r0[GT_ROWS + ra] = y[j][n][mt][1];
            r0[rc] = y[j][n][mt][2]; r0[GT_ROWS + rc] = y[j][n][mt][3];
          }
        __syncwarp();
        if (lane == 0) mbar_arrive(red_done);
        const int t = (warp - (int)(rcount & 15u)) & 15;    // the token this warp sums (if it exists)
        if (t < p.T) {
          if (ok && !gv_wait(red_done, rph, p.status, p.wait_limit)) ok = false;
          float a = 0.0f;
#pragma unroll
          for (int ww = 0; ww < GT_WARPS; ++ww) a += red[(ww * NTOK + t) * GT_ROWS + (lane ^ (((t >> 1) & 3) << 3))];
          __syncwarp();
          if (lane == 0) gv_release(red_free, gv_dep(a, a, a, 0.0f, p.zero));
          const int o = rb * GT_ROWS + lane;                // lane = row of the block
          if (o < p.d_out) {
            if (p.y_dtype == QBLORA_BF16) reinterpret_cast<__nv_bfloat16*>(p.Y)[(int64_t)t * p.d_out + o] = __float2bfloat16_rn(a);
            else reinterpret_cast<float*>(p.Y)[(int64_t)t * p.d_out + o] = a;
          }
        }
        ++rcount;
        rph ^= 1u;
      }
    }
  }
  __syncthreads();
}

template <int NT>
int ko_stages() {
  const int n = (int)((GT_SMEM_MAX - KoCfg<NT>::FIXED) / GT_STAGE_BYTES);
  return n < 10 ? n : 10;
}
template <int NT>
int ko_launch(const CUtensorMap& tm_c, const CUtensorMap& tm_a, const CUtensorMap& tm_b, GtParams p, int grid,
              uint8_t* xfrag, cudaStream_t st, bool chain) {
  p.stages = ko_stages<NT>();
  const int items = p.n_kc * GT_GROUPS * KoCfg<NT>::NTOK * 4;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  {
    cudaLaunchConfig_t pc{};
    pc.gridDim = dim3((unsigned)((items + 255) / 256)); pc.blockDim = dim3(256); pc.dynamicSmemBytes = 0; pc.stream = st;
    pc.attrs = attr; pc.numAttrs = chain ? 1 : 0;
    QB_CUDA(cudaLaunchKernelEx(&pc, x_prepare_kernel<NT>, p.X, p.T, p.d_in, p.G, p.n_kc, xfrag));
  }
  count_launch();
  const size_t smem = KoCfg<NT>::FIXED + (size_t)p.stages * GT_STAGE_BYTES;
  QB_CUDA(cudaFuncSetAttribute(lowbit_gemv_ko_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)grid); cfg.blockDim = dim3(KO_THREADS); cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cfg.attrs = attr; cfg.numAttrs = chain ? 1 : 0;
  const uint8_t* xf = xfrag;
  QB_CUDA(cudaLaunchKernelEx(&cfg, lowbit_gemv_ko_kernel<NT>, tm_c, tm_a, tm_b, p, xf));
  return QBLORA_OK;
}

}  // namespace

bool gemv_supported(const QwView& qw, int64_t T) {
  // TMA over alpha / beta rows needs a 16-byte row pitch: G % 4 == 0
  return qw.block_in == 64 && qw.block_out == 1 && qw.qfmt == QBLORA_FMT_AFFINE_MINMAX && T <= 16 && qw.G % 4 == 0 && qw.G <= 1024;
}

constexpr int T1_TAIL_MAX_BLOCKS = 128, T1_TAIL_MAX_SPLIT = 4;   // row blocks in a split tail, parts each
constexpr size_t T1_TAIL_HALF = (size_t)T1_TAIL_MAX_BLOCKS * T1_TAIL_MAX_SPLIT * (GT_ROWS * 4 + 4);
constexpr size_t T1_TAIL_BYTES = 2 * T1_TAIL_HALF;   // two areas, used by alternate launches (launches of a chain may overlap)

size_t gemv_ws_bytes(const QwView& qw, int64_t T) {
  // status word, then either the token fragments of the K-outer kernel (one K tile after the other)
  // or the hand-over area of the one-token kernel's split tail (sums, then flags)
  const size_t n_kc = (size_t)(qw.G + GT_GROUPS - 1) / GT_GROUPS;
  const size_t frag = n_kc * (T <= 8 ? (size_t)KoCfg<1>::KT_BYTES : (size_t)KoCfg<2>::KT_BYTES);
  return kStatusBytes + (frag > T1_TAIL_BYTES ? frag : T1_TAIL_BYTES);
}

// `chain`: launch as programmatic dependents (the weight stream starts while the predecessor drains).  false when the
// weight itself was written by the kernel in front (densely stored codes just expanded into the workspace).
int launch_lowbit_gemv(const QwView& qw, const __nv_bfloat16* X, int64_t T, void* Y, int y_dtype, int* status,
                       cudaStream_t st, bool chain) {
  uint8_t* xfrag = reinterpret_cast<uint8_t*>(status) + kStatusBytes;   // fragments of x (see gemv_ws_bytes)
  GtParams p{};
  p.d_in = qw.d_in; p.d_out = qw.d_out; p.G = qw.G; p.T = (int)T;
  p.n_rb = (qw.d_out + GT_ROWS - 1) / GT_ROWS;
  p.n_kc = (qw.G + GT_GROUPS - 1) / GT_GROUPS;
  p.X = X; p.Y = Y; p.y_dtype = y_dtype; p.status = status;
  p.wait_limit = wait_limit_cycles();
  CUtensorMap tm_c, tm_a, tm_b;
  // codes as 32-bit words: [d_out][d_in / 8], boxes of 32 words (four groups) x 32 rows, 128-byte swizzle
  int rc = make_tensor_map_2d_typed(&tm_c, TM_U32, qw.codes, (uint64_t)qw.d_in / 8, (uint64_t)qw.d_out,
                                    (uint64_t)qw.d_in / 2, 32, GT_ROWS, 128);
  if (rc) return rc;
  rc = make_tensor_map_2d_typed(&tm_a, TM_F32, qw.alpha, (uint64_t)qw.G, (uint64_t)qw.d_out, (uint64_t)qw.G * 4,
                                GT_GROUPS, GT_ROWS, 64);
  if (rc) return rc;
  rc = make_tensor_map_2d_typed(&tm_b, TM_F32, qw.beta, (uint64_t)qw.G, (uint64_t)qw.d_out, (uint64_t)qw.G * 4,
                                GT_GROUPS, GT_ROWS, 64);
  if (rc) return rc;
  int sms = 148;
  { int dev = 0; if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev); }
  int grid = p.n_rb < sms ? p.n_rb : sms;
  const bool one_token = T == 1 && t1_stages(p.G) > 0;
  p.tail_first = p.n_rb; p.tail_split = 1;
  if (one_token) {
    // Split tail (see T1Walk): the row blocks left after the whole rounds, when they would keep at most
    // half of the CTAs busy, are cut along K so that all CTAs share them.
    static std::atomic<uint32_t> launches{0};
    const int whole = p.n_rb >= sms ? (p.n_rb / sms) * sms : 0;
    const int rem = p.n_rb - whole;
    int split = rem > 0 ? sms / rem : 1;
    if (split > T1_TAIL_MAX_SPLIT) split = T1_TAIL_MAX_SPLIT;
    if (split > p.n_kc) split = p.n_kc;
    // the hand-over costs about as much as three tiles: split only when it saves clearly more
    if (split >= 2 && rem <= T1_TAIL_MAX_BLOCKS && p.n_kc - p.n_kc / split >= 8) {
      p.tail_first = whole; p.tail_split = split;
      if (whole == 0) grid = rem * split;
      uint32_t e = launches.fetch_add(1) + 1;
      p.epoch = e == 0 ? launches.fetch_add(1) + 1 : e;
      uint8_t* area = xfrag + (p.epoch & 1u) * T1_TAIL_HALF;
      p.tail_partial = reinterpret_cast<float*>(area);
      p.tail_flags = reinterpret_cast<uint32_t*>(area + (size_t)T1_TAIL_MAX_BLOCKS * T1_TAIL_MAX_SPLIT * GT_ROWS * 4);
    }
  }
  {
    DominantKernelTimer timer(st);
    count_launch();
    if (one_token) rc = t1_launch(tm_c, tm_a, tm_b, p, grid, st, chain);
    else if (T <= 8) rc = ko_launch<1>(tm_c, tm_a, tm_b, p, grid, xfrag, st, chain);
    else rc = ko_launch<2>(tm_c, tm_a, tm_b, p, grid, xfrag, st, chain);
    if (rc) return rc;
  }
  QB_CUDA(cudaGetLastError());
  return QBLORA_OK;
}

}  // namespace qb
