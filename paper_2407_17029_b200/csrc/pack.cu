// Dense storage of N-bit codes, N = 2 or 3 (Eq. 1 is stated for N bits; the paper fixes no byte layout):
//   N = 2: byte k of a row holds codes 4k .. 4k+3, code 4k+j in bits 2j .. 2j+1 (d_in / 4 bytes per row);
//   N = 3: codes 8k .. 8k+7 form the 24-bit number sum_j code(8k+j) << 3j, little-endian in bytes 3k .. 3k+2
//          (3 d_in / 8 bytes per row).
// The kernels of this library work on one code per nibble; a densely stored weight is expanded into the caller's
// workspace at the start of a call (one pass: N/8 bytes read and 1/2 byte written per weight), so what is saved
// is the memory the model occupies at rest, not the bytes a product streams.
// A thread converts 32 codes: four nibble words <-> two (N = 2) or three (N = 3) dense words.
#include "common.cuh"

namespace qb {
namespace {

__device__ __forceinline__ uint32_t squeeze2(uint32_t w) {   // eight nibbles -> eight 2-bit fields (16 bits)
  uint32_t x = w & 0x33333333u;
  x = (x | (x >> 2)) & 0x0F0F0F0Fu;
  x = (x | (x >> 4)) & 0x00FF00FFu;
  return (x | (x >> 8)) & 0x0000FFFFu;
}
__device__ __forceinline__ uint32_t spread2(uint32_t x) {    // 16 bits -> eight nibbles
  x = (x | (x << 8)) & 0x00FF00FFu;
  x = (x | (x << 4)) & 0x0F0F0F0Fu;
  return (x | (x << 2)) & 0x33333333u;
}
__device__ __forceinline__ uint32_t squeeze3(uint32_t w) {   // eight nibbles -> eight 3-bit fields (24 bits)
  uint32_t x = w & 0x77777777u;
  x = (x & 0x07070707u) | ((x & 0x70707070u) >> 1);
  x = (x & 0x003F003Fu) | ((x & 0x3F003F00u) >> 2);
  return (x & 0x00000FFFu) | ((x >> 4) & 0x00FFF000u);
}
__device__ __forceinline__ uint32_t spread3(uint32_t g) {    // 24 bits -> eight nibbles
  uint32_t x = (g & 0x00000FFFu) | ((g & 0x00FFF000u) << 4);
  x = (x & 0x003F003Fu) | ((x & 0x0FC00FC0u) << 2);
  return (x & 0x07070707u) | ((x & 0x38383838u) << 1);
}

template <int BITS>
__global__ void __launch_bounds__(256) pack_codes_kernel(const uint4* __restrict__ nibble, int64_t n32, uint32_t* __restrict__ packed,
                                                         int* __restrict__ bad) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n32) return;
  const uint4 v = nibble[i];
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
  const uint32_t over = BITS == 2 ? 0xCCCCCCCCu : 0x88888888u;      // bits a code of N bits must not have
  if (bad && ((w[0] | w[1] | w[2] | w[3]) & over)) atomicExch(bad, (int)QBLORA_ERR_INVALID_ARG);
  if (BITS == 2) {
    packed[2 * i] = squeeze2(w[0]) | (squeeze2(w[1]) << 16);
    packed[2 * i + 1] = squeeze2(w[2]) | (squeeze2(w[3]) << 16);
  } else {
    const uint32_t g0 = squeeze3(w[0]), g1 = squeeze3(w[1]), g2 = squeeze3(w[2]), g3 = squeeze3(w[3]);
    packed[3 * i] = g0 | (g1 << 24);
    packed[3 * i + 1] = (g1 >> 8) | (g2 << 16);
    packed[3 * i + 2] = (g2 >> 16) | (g3 << 8);
  }
}

template <int BITS>
__global__ void __launch_bounds__(256) unpack_codes_kernel(const uint32_t* __restrict__ packed, int64_t n32, uint4* __restrict__ nibble) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n32) return;
  uint4 out;
  if (BITS == 2) {
    const uint32_t a = packed[2 * i], b = packed[2 * i + 1];
    out = make_uint4(spread2(a & 0xFFFFu), spread2(a >> 16), spread2(b & 0xFFFFu), spread2(b >> 16));
  } else {
    const uint32_t a = packed[3 * i], b = packed[3 * i + 1], c = packed[3 * i + 2];
    out = make_uint4(spread3(a & 0xFFFFFFu), spread3((a >> 24) | ((b & 0xFFFFu) << 8)), spread3((b >> 16) | ((c & 0xFFu) << 16)),
                     spread3(c >> 8));
  }
  nibble[i] = out;
}

}  // namespace

// `bad` (optional, device int): set to QBLORA_ERR_INVALID_ARG when a code does not fit in `bits` bits.
int launch_pack_codes(const uint8_t* nibble, int64_t d_out, int64_t d_in, int bits, uint8_t* packed, int* bad, cudaStream_t st) {
  const int64_t n32 = d_out * d_in / 32;
  const unsigned grid = (unsigned)((n32 + 255) / 256);
  if (bits == 2) pack_codes_kernel<2><<<grid, 256, 0, st>>>(reinterpret_cast<const uint4*>(nibble), n32, reinterpret_cast<uint32_t*>(packed), bad);
  else pack_codes_kernel<3><<<grid, 256, 0, st>>>(reinterpret_cast<const uint4*>(nibble), n32, reinterpret_cast<uint32_t*>(packed), bad);
  count_launch();
  QB_CUDA(cudaGetLastError());
  return QBLORA_OK;
}

int launch_unpack_codes(const uint8_t* packed, int64_t d_out, int64_t d_in, int bits, uint8_t* nibble, cudaStream_t st) {
  const int64_t n32 = d_out * d_in / 32;
  const unsigned grid = (unsigned)((n32 + 255) / 256);
  if (bits == 2) unpack_codes_kernel<2><<<grid, 256, 0, st>>>(reinterpret_cast<const uint32_t*>(packed), n32, reinterpret_cast<uint4*>(nibble));
  else unpack_codes_kernel<3><<<grid, 256, 0, st>>>(reinterpret_cast<const uint32_t*>(packed), n32, reinterpret_cast<uint4*>(nibble));
  count_launch();
  QB_CUDA(cudaGetLastError());
  return QBLORA_OK;
}

}  // namespace qb
