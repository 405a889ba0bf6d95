// QA-BLoRA merge (Sec. 3.3): fold the adapter into the per-block beta of the min-max format.
// Two small kernels: H = A B in fp64 (P x Q values), then beta' = beta + s * H / lambda_in.
#include <atomic>

#include "common.cuh"

namespace qb {
namespace {

__global__ void merge_h_kernel(const __nv_bfloat16* __restrict__ A, const __nv_bfloat16* __restrict__ B,
                               int P, int Q, int r, bool single, double* __restrict__ H) {
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)P * Q) return;
  const int p = (int)(idx / Q), q = (int)(idx % Q);
  double h = 0.0;
  if (single) {
    h = (double)__bfloat162float(A[idx]);
  } else {
    // bf16 x bf16 products are exact in fp64 (16 significant bits), so the fused multiply-add rounds
    // exactly like a separate multiply and add; the sum runs in index order.  (fp64 throughput bounds
    // this kernel: eight chains per thread with 16-byte loads of B measured slower.)
    for (int k = 0; k < r; ++k)
      h = __fma_rn((double)__bfloat162float(A[(int64_t)p * r + k]), (double)__bfloat162float(B[(int64_t)k * Q + q]), h);
  }
  H[idx] = h;
}

__global__ void merge_beta_kernel(const float* __restrict__ beta, const double* __restrict__ H, int R,
                                  int G, int Q, int block_in, int block_out, int l1, int l2, double s,
                                  float* __restrict__ beta_out) {
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)R * G) return;
  const int rb = (int)(idx / G), gb = (int)(idx % G);
  const int p = (gb * block_in) / l1, q = (rb * block_out) / l2;
  const double h = H[(int64_t)p * Q + q];
  beta_out[idx] = (float)__dadd_rn((double)beta[idx], __ddiv_rn(__dmul_rn(s, h), (double)l1));
}

// Dense 16-bit merge (Sec. 3.1 / 3.2: the adapter folded back into a full-precision weight):
//   W'[o][i] = alpha * level[c] + beta  +  s * H[i / lambda_in][o / lambda_out] / lambda_in,   rounded to bf16.
// A thread produces eight consecutive i of one row (four packed bytes in, one 16-byte store out).
struct Level16 { float v[16]; };
__global__ void __launch_bounds__(256) merge_dense_kernel(const uint8_t* __restrict__ codes, const float* __restrict__ alpha,
                                                          const float* __restrict__ beta, int d_out, int d_in,
                                                          int block_in, int block_out, const Level16 level16,
                                                          const double* __restrict__ H, int P, int Q, int l1, int l2,
                                                          int op, double s_over_l1, __nv_bfloat16* __restrict__ W) {
  __shared__ float lev[16];
  if (threadIdx.x < 16) lev[threadIdx.x] = level16.v[threadIdx.x];
  __syncthreads();
  const int chunks = d_in >> 3;
  const int ch = (int)(blockIdx.x * blockDim.x + threadIdx.x);     // grid: x over the row's 8-element chunks, y = row
  if (ch >= chunks) return;
  const int i0 = ch * 8;
  for (int o = (int)blockIdx.y; o < d_out; o += (int)gridDim.y) {
    const uint32_t w = *reinterpret_cast<const uint32_t*>(codes + (int64_t)o * (d_in >> 1) + (i0 >> 1));
    const int gi = d_in / block_in;
    const float* arow = alpha + (int64_t)(o / block_out) * gi;
    const float* brow = beta ? beta + (int64_t)(o / block_out) * gi : nullptr;
    // fp32 is enough before the single rounding to bf16; the adapter term s * H / lambda_in is taken from the
    // fp64 H once per pooling window
    uint32_t out[4];
    // running block / window indices instead of a division per element
    int b = i0 / block_in, brem = i0 - b * block_in;
    int win = i0 / l1, wrem = i0 - win * l1;
    // AvgPool & repeat_interleave: constant per pooling window.  The alternative operator pairs place
    // s * H on single kept / sampled positions (s_over_l1 is then s itself) and are looked up per element.
    const int hq = H ? scale_src(op, o, l2, Q) : -1;
    const double* hcol = hq >= 0 ? H + hq : nullptr;
    float delta = (hcol && op == QBLORA_SCALE_AVGPOOL_REPEAT) ? (float)(hcol[(int64_t)win * Q] * s_over_l1) : 0.0f;
    float al = arow[b], be = brow ? brow[b] : 0.0f;
    float v[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int c = (w >> (4 * e)) & 15;
      if (op != QBLORA_SCALE_AVGPOOL_REPEAT) {
        const int hp = hcol ? scale_src(op, i0 + e, l1, P) : -1;
        delta = hp >= 0 ? (float)(hcol[(int64_t)hp * Q] * s_over_l1) : 0.0f;
      }
      v[e] = fmaf(al, lev[c], be) + delta;
      if (++brem == block_in && e < 7) { brem = 0; ++b; al = arow[b]; be = brow ? brow[b] : 0.0f; }
      if (++wrem == l1 && e < 7) {
        wrem = 0; ++win;
        if (hcol && op == QBLORA_SCALE_AVGPOOL_REPEAT) delta = (float)(hcol[(int64_t)win * Q] * s_over_l1);
      }
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const __nv_bfloat162 pk = __floats2bfloat162_rn(v[2 * e], v[2 * e + 1]);
      out[e] = *reinterpret_cast<const uint32_t*>(&pk);
    }
    *reinterpret_cast<uint4*>(W + (int64_t)o * d_in + i0) = make_uint4(out[0], out[1], out[2], out[3]);
  }
}

// Scratch of qablora_merge_noalloc: the P x Q matrix H = A B in fp64.  It is part of the loaded
// library image, so every GPU that loads the library holds these 2 MiB until the process exits.
constexpr int64_t kStaticMergeElems = 262144;
static __device__ __align__(256) double g_merge_scratch[kStaticMergeElems];

}  // namespace

size_t merge_dense_ws_bytes(const QwView&, const AdView* ad) {
  return kStatusBytes + 256 + (ad ? align_up((size_t)ad->P * ad->Q * sizeof(double), 256) : 0);
}

int launch_merge_dense(const QwView& qw, const AdView* ad, bool single, __nv_bfloat16* W, char* ws, cudaStream_t st) {
  Level16 lev;
  for (int j = 0; j < 16; ++j) lev.v[j] = qw.level[j];
  double* H = nullptr;
  if (ad) {
    H = reinterpret_cast<double*>(ws + kStatusBytes + 256);
    const int64_t n = (int64_t)ad->P * ad->Q;
    merge_h_kernel<<<(unsigned)((n + 127) / 128), 128, 0, st>>>(ad->A, ad->B, ad->P, ad->Q, ad->r, single, H);
    count_launch();
    QB_CUDA(cudaGetLastError());
  }
  const dim3 grid((unsigned)((qw.d_in / 8 + 255) / 256), (unsigned)(qw.d_out < 65535 ? qw.d_out : 65535));
  merge_dense_kernel<<<grid, 256, 0, st>>>(qw.codes, qw.alpha, qw.beta, qw.d_out, qw.d_in, qw.block_in,
                                                                qw.block_out, lev, H, ad ? ad->P : 1, ad ? ad->Q : 1, ad ? ad->l1 : 1,
                                                                ad ? ad->l2 : 1, ad ? ad->op : 0,
                                                                !ad ? 0.0 : ad->op == QBLORA_SCALE_AVGPOOL_REPEAT ? (double)ad->s / (double)ad->l1 : (double)ad->s, W);
  count_launch();
  QB_CUDA(cudaGetLastError());
  return QBLORA_OK;
}

size_t merge_ws_bytes(const QwView&, const AdView& ad) {
  return kStatusBytes + align_up((size_t)ad.P * ad.Q * sizeof(double), 256);
}

int launch_merge(const QwView& qw, const AdView& ad, bool single, float* beta_out, char* ws,
                 cudaStream_t st) {
  double* H = reinterpret_cast<double*>(ws + kStatusBytes);
  int64_t n = (int64_t)ad.P * ad.Q;
  merge_h_kernel<<<(unsigned)((n + 127) / 128), 128, 0, st>>>(ad.A, ad.B, ad.P, ad.Q, ad.r, single, H);
  count_launch();
  QB_CUDA(cudaGetLastError());
  const int R = qw.d_out / qw.block_out;
  n = (int64_t)R * qw.G;
  merge_beta_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(qw.beta, H, R, qw.G, ad.Q, qw.block_in,
                                                               qw.block_out, ad.l1, ad.l2, (double)ad.s,
                                                               beta_out);
  count_launch();
  QB_CUDA(cudaGetLastError());
  return QBLORA_OK;
}

int64_t merge_noalloc_capacity() { return kStaticMergeElems; }

// Same two kernels as launch_merge, with H in the static device array above.  In host code the
// array's name is only a host-side handle, so its device address is looked up (once per device, with
// that device current) and cached; that lookup is the only set-up this path needs.
int launch_merge_noalloc(const QwView& qw, const AdView& ad, bool single, float* beta_out, cudaStream_t st) {
  constexpr int kMaxDevices = 64;
  static std::atomic<double*> scratch_of_device[kMaxDevices];   // atomic: host threads may race to fill an entry (same value)
  int dev = -1;
  QB_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return QBLORA_ERR_UNSUPPORTED;
  double* H = scratch_of_device[dev].load(std::memory_order_acquire);
  if (!H) {
    double* ptr = nullptr;
    QB_CUDA(cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_merge_scratch));
    if (!ptr) return QBLORA_ERR_CUDA;
    scratch_of_device[dev].store(ptr, std::memory_order_release);
    H = ptr;
  }
  // every one of the P * Q entries read below is written first, so nothing has to be cleared
  int64_t n = (int64_t)ad.P * ad.Q;
  merge_h_kernel<<<(unsigned)((n + 127) / 128), 128, 0, st>>>(ad.A, ad.B, ad.P, ad.Q, ad.r, single, H);
  count_launch();
  QB_CUDA(cudaGetLastError());
  const int R = qw.d_out / qw.block_out;
  n = (int64_t)R * qw.G;
  merge_beta_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(qw.beta, H, R, qw.G, ad.Q, qw.block_in,
                                                               qw.block_out, ad.l1, ad.l2, (double)ad.s,
                                                               beta_out);
  count_launch();
  QB_CUDA(cudaGetLastError());
  return QBLORA_OK;
}

}  // namespace qb
