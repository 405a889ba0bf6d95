// Shared declarations of the CUDA library behind include/qblora.h.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "qblora.h"

#define QB_CUDA(call)                                   \
  do {                                                  \
    if ((call) != cudaSuccess) return QBLORA_ERR_CUDA;  \
  } while (0)

namespace qb {

// Device-side view of a frozen quantized weight (pointers are device pointers).
struct QwView {
  int d_in, d_out, block_in, block_out, qfmt, G;  // G = d_in / block_in
  int code_bits;   // storage of the codes: 4 = one per nibble; 2, 3 = dense (pack.cu), expanded into the workspace before use
  const uint8_t* codes;
  const float* alpha;
  const float* beta;
  float level[16];  // level table (code-table format) or 0..15 (min-max format)
};

struct AdView {
  int l1, l2, r, P, Q;
  int op;  // qblora_scale_op
  float s;
  const __nv_bfloat16* A;
  const __nv_bfloat16* B;
};

// Index map of the adapter's parameter-free operator pair (Sec. 3.2 and the scale-operator ablation of
// Sec. 4): the compressed index that full-size index `idx` is tied to, or -1 for none.  `lam` is the
// factor of that side, `n_small` the compressed size.  The tie's coefficient is 1 / lam on the input side
// of AvgPool & repeat_interleave and 1 everywhere else.
__host__ __device__ __forceinline__ int scale_src(int op, int idx, int lam, int n_small) {
  if (op == QBLORA_SCALE_AVGPOOL_REPEAT) return idx / lam;
  if (op == QBLORA_SCALE_TRUNCATE_ZEROPAD) return idx < n_small ? idx : -1;
  return (idx % lam == 0) ? idx / lam : -1;
}

constexpr size_t kStatusBytes = 256;  // first bytes of every workspace: device status word

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ---- instrumentation (instrument.cu) ------------------------------------------------------------
void count_launch(int n = 1);
// Device-side waits give up after this many cycles (~1 s: far beyond any legitimate wait) unless
// qblora_debug_set_wait_limit has set another value; every launch passes the current value to its kernel.
constexpr long long kDefaultWaitLimitCycles = 2000000000LL;
long long wait_limit_cycles();
// Test hook armed by qblora_debug_drop_load: returns the armed producer iteration once (then -1 again).
int take_dropped_load();
// Test hook armed by qblora_debug_hold_producer: returns the armed number of cycles once (then 0 again).
long long take_producer_hold();
// Brackets the dominant kernel of a call with the armed event pair (if any), then disarms.
struct DominantKernelTimer {
  cudaStream_t st; cudaEvent_t stop;
  explicit DominantKernelTimer(cudaStream_t s);
  ~DominantKernelTimer();
};

// ---- entry points of the individual translation units (host side) ----------------------------
int launch_quantize(const void* W, int w_dtype, int d_out, int d_in, int block_in, int block_out,
                    int qfmt, int bits, const float* level, uint8_t* codes, float* alpha, float* beta,
                    cudaStream_t st);

// General path (any block shape, any size): CUDA-core kernels.
size_t simt_ws_bytes(int op, const QwView& qw, const AdView* ad, int64_t T);
int simt_linear_fwd(const QwView& qw, const AdView* ad, const __nv_bfloat16* X, int64_t T, void* Y,
                    int y_dtype, char* ws, cudaStream_t st);
int simt_linear_bwd(const QwView& qw, const AdView* ad, const __nv_bfloat16* X,
                    const __nv_bfloat16* dY, int64_t T, void* dX, int dx_dtype, float* dA, float* dB,
                    char* ws, cudaStream_t st);

size_t merge_ws_bytes(const QwView& qw, const AdView& ad);
int launch_merge(const QwView& qw, const AdView& ad, bool single_matrix, float* beta_out, char* ws,
                 cudaStream_t st);

int64_t merge_noalloc_capacity();   // P * Q entries the built-in scratch of the no-alloc merge holds
int launch_merge_noalloc(const QwView& qw, const AdView& ad, bool single_matrix, float* beta_out,
                         cudaStream_t st);

// Bandwidth-bound low-bit product for small token counts (block_out == 1, block_in == 64).
size_t merge_dense_ws_bytes(const QwView& qw, const AdView* ad);
int launch_merge_dense(const QwView& qw, const AdView* ad, bool single_matrix, __nv_bfloat16* W, char* ws, cudaStream_t st);
int launch_identity(__nv_bfloat16* out, int n, cudaStream_t st);   // bf16 identity [n][n]
bool gemv_supported(const QwView& qw, int64_t T);
size_t gemv_ws_bytes(const QwView& qw, int64_t T);   // status word + (T > 1) token fragments
int launch_lowbit_gemv(const QwView& qw, const __nv_bfloat16* X, int64_t T, void* Y, int y_dtype,
                       int* status, cudaStream_t st, bool chain = true);

// Dense 2- / 3-bit code storage (pack.cu); d_in % 32 == 0.
int launch_pack_codes(const uint8_t* nibble, int64_t d_out, int64_t d_in, int bits, uint8_t* packed, int* bad, cudaStream_t st);
int launch_unpack_codes(const uint8_t* packed, int64_t d_out, int64_t d_in, int bits, uint8_t* nibble, cudaStream_t st);

// Plain bf16 tcgen05 GEMM serving a dense merged weight: Y = X W^T, W bf16 [d_out][d_in] (d_in % 8 == 0).
size_t dense_gemm_ws_bytes();
int launch_dense_gemm(const __nv_bfloat16* W, int d_out, int d_in, const __nv_bfloat16* X, int64_t T, void* Y,
                      int y_dtype, int* status, cudaStream_t st);

// Tensor-core path (tcgen05 / TMEM / TMA): block_in == 64, block_out == 1.
bool tc_supported(const QwView& qw, const AdView* ad, int64_t T);
size_t tc_ws_bytes(int op, const QwView& qw, const AdView* ad, int64_t T);
int tc_linear_fwd(const QwView& qw, const AdView* ad, const __nv_bfloat16* X, int64_t T, void* Y,
                  int y_dtype, char* ws, cudaStream_t st);
// Low-bit product on the tensor-core path (any token count; the caller sends small ones to the decode kernels).
size_t tc_lowbit_ws_bytes(const QwView& qw, int64_t T);
int tc_lowbit_gemm(const QwView& qw, const __nv_bfloat16* X, int64_t T, void* Y, int y_dtype, char* ws, cudaStream_t st);
int tc_linear_bwd(const QwView& qw, const AdView* ad, const __nv_bfloat16* X,
                  const __nv_bfloat16* dY, int64_t T, void* dX, int dx_dtype, float* dA, float* dB,
                  char* ws, cudaStream_t st);

}  // namespace qb
