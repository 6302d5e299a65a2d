// kmq_pack / kmq_unpack: canonical LSB-first bit-packing of centroid indices
// along K (uint32 words, 32/bits fields per word).
#include "kmq_common.cuh"

namespace kmq {
namespace {

// One thread builds one output word from 32/BITS consecutive index bytes.
// The bytes of one word are contiguous and 32/BITS-byte aligned, so they are
// fetched as 8-, 16- or 2x16-byte vectors.
template <int BITS>
__global__ void __launch_bounds__(256) pack_kernel(const uint8_t* __restrict__ idx, uint32_t* __restrict__ packed,
                                                   int64_t total_words) {
  constexpr int PER = 32 / BITS;
  constexpr uint32_t MASK = (1u << BITS) - 1u;
  int64_t w = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (; w < total_words; w += stride) {
    const uint8_t* src = idx + w * PER;
    uint32_t out = 0;
    if constexpr (BITS == 4) {
      uint2 v = *reinterpret_cast<const uint2*>(src);
      uint32_t r[2] = {v.x, v.y};
#pragma unroll
      for (int i = 0; i < 8; ++i) out |= ((r[i >> 2] >> ((i & 3) * 8)) & MASK) << (i * 4);
    } else if constexpr (BITS == 2) {
      uint4 v = *reinterpret_cast<const uint4*>(src);
      uint32_t r[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int i = 0; i < 16; ++i) out |= ((r[i >> 2] >> ((i & 3) * 8)) & MASK) << (i * 2);
    } else {
      uint4 a = *reinterpret_cast<const uint4*>(src);
      uint4 b = *reinterpret_cast<const uint4*>(src + 16);
      uint32_t r[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 32; ++i) out |= ((r[i >> 2] >> ((i & 3) * 8)) & MASK) << i;
    }
    packed[w] = out;
  }
}

template <int BITS>
__global__ void __launch_bounds__(256) unpack_kernel(const uint32_t* __restrict__ packed, uint8_t* __restrict__ idx,
                                                     int64_t total_words) {
  constexpr int PER = 32 / BITS;
  constexpr uint32_t MASK = (1u << BITS) - 1u;
  int64_t w = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (; w < total_words; w += stride) {
    const uint32_t word = packed[w];
    uint32_t r[PER / 4];
#pragma unroll
    for (int q = 0; q < PER / 4; ++q) {
      uint32_t v = 0;
#pragma unroll
      for (int i = 0; i < 4; ++i) v |= ((word >> ((q * 4 + i) * BITS)) & MASK) << (i * 8);
      r[q] = v;
    }
    uint32_t* dst = reinterpret_cast<uint32_t*>(idx + w * PER);
#pragma unroll
    for (int q = 0; q < PER / 4; ++q) dst[q] = r[q];
  }
}

inline int grid_for(int64_t items, int threads, int sm_count) {
  int64_t blocks = (items + threads - 1) / threads;
  int64_t cap = (int64_t)sm_count * 16;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  return (int)blocks;
}

}  // namespace

cudaError_t launch_pack(const uint8_t* idx, int64_t N, int64_t K, int bits, uint32_t* packed, cudaStream_t s) {
  const DeviceInfo* di = device_info();
  if (!di) return cudaGetLastError();
  const int64_t words = N * (K / (32 / bits));
  const int grid = grid_for(words, 256, di->sm_count);
  if (bits == 1) pack_kernel<1><<<grid, 256, 0, s>>>(idx, packed, words);
  else if (bits == 2) pack_kernel<2><<<grid, 256, 0, s>>>(idx, packed, words);
  else pack_kernel<4><<<grid, 256, 0, s>>>(idx, packed, words);
  return cudaGetLastError();
}

cudaError_t launch_unpack(const uint32_t* packed, int64_t N, int64_t K, int bits, uint8_t* idx, cudaStream_t s) {
  const DeviceInfo* di = device_info();
  if (!di) return cudaGetLastError();
  const int64_t words = N * (K / (32 / bits));
  const int grid = grid_for(words, 256, di->sm_count);
  if (bits == 1) unpack_kernel<1><<<grid, 256, 0, s>>>(packed, idx, words);
  else if (bits == 2) unpack_kernel<2><<<grid, 256, 0, s>>>(packed, idx, words);
  else unpack_kernel<4><<<grid, 256, 0, s>>>(packed, idx, words);
  return cudaGetLastError();
}

}  // namespace kmq
