// QA-BLoRA merge (Sec. 3.3): fold the adapter into the per-block beta of the min-max format.
// Two small kernels: H = A B in fp64 (P x Q values), then beta' = beta + s * H / lambda_in.
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
    // bf16 x bf16 products are exact in fp64; the sum runs in index order
    for (int k = 0; k < r; ++k)
      h = __dadd_rn(h, __dmul_rn((double)__bfloat162float(A[(int64_t)p * r + k]),
                                 (double)__bfloat162float(B[(int64_t)k * Q + q])));
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

// Scratch of qablora_merge_noalloc: the P x Q matrix H = A B in fp64.  It is part of the loaded
// library image, so every GPU that loads the library holds these 2 MiB until the process exits.
constexpr int64_t kStaticMergeElems = 262144;
static __device__ __align__(256) double g_merge_scratch[kStaticMergeElems];

}  // namespace

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
  static double* scratch_of_device[kMaxDevices] = {};
  int dev = -1;
  QB_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return QBLORA_ERR_UNSUPPORTED;
  if (!scratch_of_device[dev]) {
    double* ptr = nullptr;
    QB_CUDA(cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_merge_scratch));
    if (!ptr) return QBLORA_ERR_CUDA;
    scratch_of_device[dev] = ptr;
  }
  double* H = scratch_of_device[dev];
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
