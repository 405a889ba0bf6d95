// Small dense bf16 GEMM on tcgen05 for the adapter branch (Sec. 3.2): C[m][n] = sum over segments of
// sum_k A_seg(m, k) * B_seg(n, k), fp32 accumulation in TMEM.  Several K-segments let a caller feed
// "hi + lo" bf16 splits of fp32 operands (A_hi B_hi + A_lo B_hi + A_hi B_lo) so the adapter
// gradients keep fp32-grade accuracy while running on the tensor cores.
#pragma once
#include "common.cuh"

namespace qb {

// A matrix seen as (mn, k).  k_contig: element at ptr[mn * ld + k]; otherwise ptr[k * ld + mn].
// ptr 16-byte aligned, ld a multiple of 8 elements.
struct SgOperand {
  const __nv_bfloat16* ptr;
  int64_t ld;
  bool k_contig;
};
struct SgSegment {
  SgOperand a, b;
  int K;
};
// Any subset of the outputs may be requested.  f32: C.  hi/lo: bf16(C) and bf16(C - hi).
// scaled: bf16(C * scale) or bf16(C / scale) when divide.
struct SgOut {
  float* f32; int64_t ld32;
  __nv_bfloat16 *hi, *lo, *scaled; int64_t ld16;
  float scale; bool divide;
};

// All segments must use the same operand majors.  `status` = device status word (bounded waits).
// `partial` (optional, fp32 output only): scratch of small_gemm_splits(M, N, K) * M * N floats; the
// contraction is then split over that many CTAs per output tile and summed in a fixed order.
// `dependent`: the kernel in front of this one on `st` is one of this library's that signals
// griddepcontrol.launch_dependents and writes an operand; this product is then launched as its programmatic
// dependent (set-up overlaps that kernel's tail; the operand loads wait for its completion).
// `wide_tiles`: keep 256-wide column tiles even when that leaves few CTAs.  For a product that sits in front of the
// fused contraction: each of its CTAs keeps a CTA of the contraction off its SM until it is done, so few CTAs
// delay fewer tiles (C2 forward call 108 -> 103.5 us).
int small_gemm(int M, int N, const SgSegment* segs, int nseg, const SgOut& out, int* status, cudaStream_t st,
               float* partial = nullptr, bool dependent = false, bool wide_tiles = false);
int small_gemm_splits(int M, int N, int K);

// Encodes a 2-D tensor map (shared with the main kernel's host code).
int make_tensor_map_2d(void* tm, bool is_u8, const void* ptr, uint64_t inner, uint64_t rows, uint64_t pitch_bytes,
                       uint32_t box_inner, uint32_t box_rows, bool swizzle128);

// Same with an explicit element type and shared-memory swizzle span (0, 64 or 128 bytes).
enum { TM_BF16 = 0, TM_U8 = 1, TM_U32 = 2, TM_F32 = 3 };
int make_tensor_map_2d_typed(void* tm, int elem, const void* ptr, uint64_t inner, uint64_t rows, uint64_t pitch_bytes,
                             uint32_t box_inner, uint32_t box_rows, int swizzle_bytes);

}  // namespace qb
