// kmq_pack / kmq_unpack: bit-packing of centroid indices along K (uint32 words, 32/bits fields per word), in the
// canonical layout (row-major, fields LSB first), the tuned tile-major layout, or the bit-plane layout of the
// activation-table kernel.
#include "kmq_common.cuh"
#include "kmq_table_layout.cuh"

namespace kmq {
namespace {

// One thread builds one output word from 32/BITS consecutive index bytes (contiguous and 32/BITS-byte aligned,
// fetched as 8-, 16- or 2x16-byte vectors).  In the tuned layout the output words are enumerated in storage order
// and the padding words (rows >= N, words >= wpr) are written as zero.
template <int BITS, bool TUNED>
__global__ void __launch_bounds__(256) pack_kernel(const uint8_t* __restrict__ idx, uint32_t* __restrict__ packed,
                                                   int64_t N, int64_t wpr, int64_t total_words) {
  constexpr int PER = 32 / BITS;
  constexpr uint32_t MASK = (1u << BITS) - 1u;
  const int64_t steps = tuned_steps(wpr);
  int64_t w = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (; w < total_words; w += stride) {
    int64_t src_word = w;
    if constexpr (TUNED) {
      const int64_t wi = w & 15, r = (w >> 4) & 15, blk = w >> 8;
      const int64_t n = (blk / steps) * kTileRows + r, j = (blk % steps) * 16 + wi;
      if (n >= N || j >= wpr) {
        packed[w] = 0;
        continue;
      }
      src_word = n * wpr + j;
    }
    const uint8_t* src = idx + src_word * PER;
    uint32_t out = 0;
    if constexpr (BITS == 4) {
      uint2 v = *reinterpret_cast<const uint2*>(src);
      uint32_t r[2] = {v.x, v.y};
#pragma unroll
      for (int i = 0; i < 8; ++i) out |= ((r[i >> 2] >> ((i & 3) * 8)) & MASK) << field_pos<BITS>(i, TUNED);
    } else if constexpr (BITS == 2) {
      uint4 v = *reinterpret_cast<const uint4*>(src);
      uint32_t r[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int i = 0; i < 16; ++i) out |= ((r[i >> 2] >> ((i & 3) * 8)) & MASK) << field_pos<BITS>(i, TUNED);
    } else {
      uint4 a = *reinterpret_cast<const uint4*>(src);
      uint4 b = *reinterpret_cast<const uint4*>(src + 16);
      uint32_t r[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 32; ++i) out |= ((r[i >> 2] >> ((i & 3) * 8)) & MASK) << field_pos<BITS>(i, TUNED);
    }
    packed[w] = out;
  }
}

// One thread expands word j of row n into 32/BITS index bytes.
template <int BITS, bool TUNED>
__global__ void __launch_bounds__(256) unpack_kernel(const uint32_t* __restrict__ packed, uint8_t* __restrict__ idx,
                                                     int64_t wpr, int64_t total_words) {
  constexpr int PER = 32 / BITS;
  constexpr uint32_t MASK = (1u << BITS) - 1u;
  const int64_t steps = tuned_steps(wpr);
  int64_t w = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (; w < total_words; w += stride) {
    const uint32_t word = TUNED ? packed[tuned_word_index(w / wpr, w % wpr, steps)] : packed[w];
    uint32_t r[PER / 4];
#pragma unroll
    for (int q = 0; q < PER / 4; ++q) {
      uint32_t v = 0;
#pragma unroll
      for (int i = 0; i < 4; ++i) v |= ((word >> field_pos<BITS>(q * 4 + i, TUNED)) & MASK) << (i * 8);
      r[q] = v;
    }
    uint32_t* dst = reinterpret_cast<uint32_t*>(idx + w * PER);
#pragma unroll
    for (int q = 0; q < PER / 4; ++q) dst[q] = r[q];
  }
}

// Table layout: one thread builds one 32-bit word = bytes 4q .. 4q+3 of one lane of one 512-byte unit, i.e. one
// bit plane of four groups of 8 weights of one row.  Padding (rows >= N, groups beyond K) is written as zero.
template <int BITS>
__global__ void __launch_bounds__(256) pack_table_kernel(const uint8_t* __restrict__ idx, uint32_t* __restrict__ packed,
                                                         int64_t N, int64_t K, int64_t chunks, int64_t total_words) {
  int64_t w = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (; w < total_words; w += stride) {
    const int64_t unit = w >> 7;                  // 128 words per unit
    const int lane = (int)(w & 127) >> 2, q = (int)(w & 3);
    const int plane = (int)(unit % BITS);
    const int64_t tc = unit / BITS, tile = tc / chunks, chunk = tc % chunks;
    uint32_t out = 0;
#pragma unroll
    for (int bi = 0; bi < 4; ++bi) {
      int r, gl;
      table_unit_coords(lane, 4 * q + bi, r, gl);
      const int64_t n = tile * 16 + r, k0 = (chunk * 32 + gl) * 8;
      if (n < N && k0 < K) {
        const uint2 v = *reinterpret_cast<const uint2*>(idx + n * K + k0);
        const uint32_t e[2] = {v.x, v.y};
        uint32_t byte = 0;
#pragma unroll
        for (int t = 0; t < 8; ++t) byte |= ((e[t >> 2] >> ((t & 3) * 8 + plane)) & 1u) << t;
        out |= byte << (8 * bi);
      }
    }
    packed[w] = out;
  }
}

// Table layout: one thread restores the 8 indices of one group of one row.
template <int BITS>
__global__ void __launch_bounds__(256) unpack_table_kernel(const uint32_t* __restrict__ packed, uint8_t* __restrict__ idx,
                                                           int64_t K, int64_t chunks, int64_t total_groups) {
  const uint8_t* bytes = reinterpret_cast<const uint8_t*>(packed);
  const int64_t gpr = K >> 3;
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (; i < total_groups; i += stride) {
    const int64_t n = i / gpr, g = i % gpr;
    uint32_t e[2] = {0, 0};
#pragma unroll
    for (int p = 0; p < BITS; ++p) {
      const uint32_t byte = bytes[table_byte_offset(n, g, p, chunks, BITS)];
#pragma unroll
      for (int t = 0; t < 8; ++t) e[t >> 2] |= ((byte >> t) & 1u) << ((t & 3) * 8 + p);
    }
    *reinterpret_cast<uint2*>(idx + n * K + g * 8) = make_uint2(e[0], e[1]);
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

cudaError_t launch_pack(const uint8_t* idx, int64_t N, int64_t K, int bits, int layout, uint32_t* packed,
                        cudaStream_t s) {
  const DeviceInfo* di = device_info();
  if (!di) return cudaErrorInvalidDevice;
  const int64_t wpr = K / (32 / bits);
  if (layout == KMQ_LAYOUT_TABLE && bits != 4) {
    const int64_t chunks = table_chunks(K), words = table_total_bytes(N, K, bits) / 4;
    const int grid = grid_for(words, 256, di->sm_count);
    if (bits == 1) pack_table_kernel<1><<<grid, 256, 0, s>>>(idx, packed, N, K, chunks, words);
    else pack_table_kernel<2><<<grid, 256, 0, s>>>(idx, packed, N, K, chunks, words);
    return cudaGetLastError();
  }
  const bool tuned = layout != KMQ_LAYOUT_CANONICAL;
  const int64_t words = tuned ? tuned_total_words(N, wpr) : N * wpr;
  const int grid = grid_for(words, 256, di->sm_count);
  if (bits == 1 && tuned) pack_kernel<1, true><<<grid, 256, 0, s>>>(idx, packed, N, wpr, words);
  else if (bits == 1) pack_kernel<1, false><<<grid, 256, 0, s>>>(idx, packed, N, wpr, words);
  else if (bits == 2 && tuned) pack_kernel<2, true><<<grid, 256, 0, s>>>(idx, packed, N, wpr, words);
  else if (bits == 2) pack_kernel<2, false><<<grid, 256, 0, s>>>(idx, packed, N, wpr, words);
  else if (tuned) pack_kernel<4, true><<<grid, 256, 0, s>>>(idx, packed, N, wpr, words);
  else pack_kernel<4, false><<<grid, 256, 0, s>>>(idx, packed, N, wpr, words);
  return cudaGetLastError();
}

cudaError_t launch_unpack(const uint32_t* packed, int64_t N, int64_t K, int bits, int layout, uint8_t* idx,
                          cudaStream_t s) {
  const DeviceInfo* di = device_info();
  if (!di) return cudaErrorInvalidDevice;
  const int64_t wpr = K / (32 / bits);
  if (layout == KMQ_LAYOUT_TABLE && bits != 4) {
    const int64_t groups = N * (K >> 3);
    const int grid = grid_for(groups, 256, di->sm_count);
    if (bits == 1) unpack_table_kernel<1><<<grid, 256, 0, s>>>(packed, idx, K, table_chunks(K), groups);
    else unpack_table_kernel<2><<<grid, 256, 0, s>>>(packed, idx, K, table_chunks(K), groups);
    return cudaGetLastError();
  }
  const int64_t words = N * wpr;
  const bool tuned = layout != KMQ_LAYOUT_CANONICAL;
  const int grid = grid_for(words, 256, di->sm_count);
  if (bits == 1 && tuned) unpack_kernel<1, true><<<grid, 256, 0, s>>>(packed, idx, wpr, words);
  else if (bits == 1) unpack_kernel<1, false><<<grid, 256, 0, s>>>(packed, idx, wpr, words);
  else if (bits == 2 && tuned) unpack_kernel<2, true><<<grid, 256, 0, s>>>(packed, idx, wpr, words);
  else if (bits == 2) unpack_kernel<2, false><<<grid, 256, 0, s>>>(packed, idx, wpr, words);
  else if (tuned) unpack_kernel<4, true><<<grid, 256, 0, s>>>(packed, idx, wpr, words);
  else unpack_kernel<4, false><<<grid, 256, 0, s>>>(packed, idx, wpr, words);
  return cudaGetLastError();
}

}  // namespace kmq
