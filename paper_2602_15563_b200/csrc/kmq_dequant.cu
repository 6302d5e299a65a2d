// kmq_dequant_to_bf16: W^[n,k] = C_n[idx[n,k]] as a dense bf16 matrix.
// The kernel is bound by the 2-byte-per-weight output stream, so every thread
// produces exactly one 16-byte store (8 weights) from 8*BITS packed bits and
// consecutive threads write consecutive 16-byte pieces.
#include "kmq_common.cuh"

namespace kmq {
namespace {

// The 8*BITS bits that hold weights 8c .. 8c+7 of row n, fields LSB first.
template <int BITS, bool TUNED>
__device__ __forceinline__ uint32_t load_chunk_bits(const uint32_t* __restrict__ packed, int64_t n, int64_t wpr,
                                                    int64_t steps, int64_t c) {
  if constexpr (TUNED) {
    // the fields of a chunk are spread over its word: permute the word back, then cut the chunk out
    constexpr int CPW = 4 / BITS;   // 8-weight chunks per word
    const uint32_t w = canonical_from_tuned<BITS>(__ldg(packed + tuned_word_index(n, c / CPW, steps)));
    if constexpr (BITS == 4) return w;
    return (w >> ((int)(c % CPW) * 8 * BITS)) & ((1u << (8 * BITS)) - 1u);
  } else if constexpr (BITS == 4) {
    return __ldg(packed + n * wpr + c);
  } else if constexpr (BITS == 2) {
    return __ldg(reinterpret_cast<const uint16_t*>(packed + n * wpr) + c);
  } else {
    return __ldg(reinterpret_cast<const uint8_t*>(packed + n * wpr) + c);
  }
}

template <int BITS, bool TUNED>
__global__ void __launch_bounds__(256) dequant_kernel(const uint32_t* __restrict__ packed,
                                                      const uint16_t* __restrict__ cb, uint16_t* __restrict__ W,
                                                      int64_t N, int64_t K) {
  constexpr int Q = 1 << BITS;
  const int64_t cpr = K >> 3;            // 8-weight chunks per row
  const int64_t wpr = K / (32 / BITS);   // words per row
  const int64_t steps = tuned_steps(wpr);
  const int64_t total = N * cpr;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t chunk = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; chunk < total; chunk += stride) {
    const int64_t n = chunk / cpr;
    const int64_t c = chunk - n * cpr;
    const uint32_t v = load_chunk_bits<BITS, TUNED>(packed, n, wpr, steps, c);
    uint32_t o[4];
    if constexpr (BITS == 1) {
      // codebook = 4 bytes {c0, c1}; a selector nibble pair picks bytes (2i, 2i+1)
      const uint32_t cw = __ldg(reinterpret_cast<const uint32_t*>(cb + n * Q));
#pragma unroll
      for (int p = 0; p < 4; ++p) {
        const uint32_t i0 = (v >> (2 * p)) & 1u, i1 = (v >> (2 * p + 1)) & 1u;
        o[p] = __byte_perm(cw, cw, 0x1010u + i0 * 0x22u + i1 * 0x2200u);
      }
    } else if constexpr (BITS == 2) {
      // codebook = 8 bytes {c0,c1 | c2,c3}: byte pair (2i, 2i+1) of the two words
      const uint2 cw = __ldg(reinterpret_cast<const uint2*>(cb + n * Q));
#pragma unroll
      for (int p = 0; p < 4; ++p) {
        const uint32_t i0 = (v >> (4 * p)) & 3u, i1 = (v >> (4 * p + 2)) & 3u;
        o[p] = __byte_perm(cw.x, cw.y, 0x1010u + i0 * 0x22u + i1 * 0x2200u);
      }
    } else {
      const uint16_t* row_cb = cb + n * Q;
#pragma unroll
      for (int p = 0; p < 4; ++p) {
        const uint32_t i0 = (v >> (8 * p)) & 15u, i1 = (v >> (8 * p + 4)) & 15u;
        o[p] = (uint32_t)__ldg(row_cb + i0) | ((uint32_t)__ldg(row_cb + i1) << 16);
      }
    }
    stg_stream_u4(reinterpret_cast<uint4*>(W + n * K + c * 8), make_uint4(o[0], o[1], o[2], o[3]));
  }
}

}  // namespace

cudaError_t launch_dequant(const uint32_t* packed, const uint16_t* cb, uint16_t* W, int64_t N, int64_t K, int bits,
                           int layout, cudaStream_t s) {
  const DeviceInfo* di = device_info();
  if (!di) return cudaGetLastError();
  const int64_t total = N * (K >> 3);
  int64_t blocks = (total + 255) / 256;
  const int64_t cap = (int64_t)di->sm_count * 32;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  const bool tuned = layout == KMQ_LAYOUT_TUNED;
  if (bits == 1 && tuned) dequant_kernel<1, true><<<(int)blocks, 256, 0, s>>>(packed, cb, W, N, K);
  else if (bits == 1) dequant_kernel<1, false><<<(int)blocks, 256, 0, s>>>(packed, cb, W, N, K);
  else if (bits == 2 && tuned) dequant_kernel<2, true><<<(int)blocks, 256, 0, s>>>(packed, cb, W, N, K);
  else if (bits == 2) dequant_kernel<2, false><<<(int)blocks, 256, 0, s>>>(packed, cb, W, N, K);
  else if (tuned) dequant_kernel<4, true><<<(int)blocks, 256, 0, s>>>(packed, cb, W, N, K);
  else dequant_kernel<4, false><<<(int)blocks, 256, 0, s>>>(packed, cb, W, N, K);
  return cudaGetLastError();
}

}  // namespace kmq
