// kmq_dequant_to_bf16: W^[n,k] = C_n[idx[n,k]] as a dense bf16 matrix.
// The kernel is bound by the 2-byte-per-weight output stream, so every thread
// produces exactly one 16-byte store (8 weights) from 8*BITS packed bits and
// consecutive threads write consecutive 16-byte pieces.
#include "kmq_common.cuh"
#include "kmq_table_layout.cuh"

namespace kmq {
namespace {

// 8 weights (8*BITS index bits, fields LSB first) -> 8 bf16 = one 16-byte value.
template <int BITS>
__device__ __forceinline__ uint4 decode8(uint32_t v, uint32_t c0, uint32_t c1, const uint16_t* __restrict__ row_cb) {
  uint32_t o[4];
  if constexpr (BITS == 1) {
    // codebook = 4 bytes {c0, c1}; a selector nibble pair picks bytes (2i, 2i+1)
#pragma unroll
    for (int p = 0; p < 4; ++p) {
      const uint32_t i0 = (v >> (2 * p)) & 1u, i1 = (v >> (2 * p + 1)) & 1u;
      o[p] = __byte_perm(c0, c0, 0x1010u + i0 * 0x22u + i1 * 0x2200u);
    }
  } else if constexpr (BITS == 2) {
    // codebook = 8 bytes {c0,c1 | c2,c3}: byte pair (2i, 2i+1) of the two words
#pragma unroll
    for (int p = 0; p < 4; ++p) {
      const uint32_t i0 = (v >> (4 * p)) & 3u, i1 = (v >> (4 * p + 2)) & 3u;
      o[p] = __byte_perm(c0, c1, 0x1010u + i0 * 0x22u + i1 * 0x2200u);
    }
  } else {
    // c0 = this lane's share of the row's codebook: centroid (lane % 16) in the low half word.  A lookup is a
    // shuffle from the lane that holds the entry (all 32 lanes of the warp must be here); two lookups are packed
    // by one PRMT.  This keeps the 16 entries out of the load path, which the packed words and the stores need.
    (void)row_cb;
#pragma unroll
    for (int p = 0; p < 4; ++p) {
      const uint32_t i0 = (v >> (8 * p)) & 15u, i1 = (v >> (8 * p + 4)) & 15u;
      const uint32_t lo = __shfl_sync(0xFFFFFFFFu, c0, (int)i0), hi = __shfl_sync(0xFFFFFFFFu, c0, (int)i1);
      o[p] = __byte_perm(lo, hi, 0x5410u);
    }
  }
  return make_uint4(o[0], o[1], o[2], o[3]);
}

template <int BITS>
__device__ __forceinline__ void load_codebook(const uint16_t* __restrict__ row_cb, uint32_t& c0, uint32_t& c1) {
  c0 = c1 = 0;
  if constexpr (BITS == 1) c0 = __ldg(reinterpret_cast<const uint32_t*>(row_cb));
  if constexpr (BITS == 2) {
    const uint2 cw = __ldg(reinterpret_cast<const uint2*>(row_cb));
    c0 = cw.x;
    c1 = cw.y;
  }
  if constexpr (BITS == 4) c0 = __ldg(row_cb + (threadIdx.x & 15));
}

// One CTA walks rows (grid-stride); inside a row every thread turns 8 weights into one 16-byte streaming store,
// consecutive threads writing consecutive pieces.  In the tuned layout the row's words come in 64-byte runs, one
// per 1 KB step of its tile, and the 8 fields of a chunk are cut out of the word after one shift.
template <int BITS, bool TUNED>
__global__ void __launch_bounds__(256) dequant_rows_kernel(const uint32_t* __restrict__ packed,
                                                           const uint16_t* __restrict__ cb, uint16_t* __restrict__ W,
                                                           int64_t N, int64_t K) {
  constexpr int Q = 1 << BITS;
  constexpr int CPW = 4 / BITS;                  // 8-weight chunks per word
  const int cpr = (int)(K >> 3);                 // 8-weight chunks per row
  const int64_t wpr = K / (32 / BITS);           // words per row
  const int64_t steps = tuned_steps(wpr);
  for (int64_t n = blockIdx.x; n < N; n += gridDim.x) {
    const uint32_t* row_words =
        TUNED ? packed + ((n >> 4) * steps * kTileRows + (n & 15)) * 16 : packed + n * wpr;
    const uint16_t* row_cb = cb + n * Q;
    uint32_t c0, c1;
    load_codebook<BITS>(row_cb, c0, c1);
    uint4* out = reinterpret_cast<uint4*>(W + n * K);
    // b = 4 looks its centroids up by warp shuffles, so there whole warps stay in the loop (lanes past the end of
    // the row decode a zero word and store nothing)
    const int cend = BITS == 4 ? (cpr + 31) & ~31 : cpr;
    for (int c = threadIdx.x; c < cend; c += 256) {
      const bool live = BITS != 4 || c < cpr;
      uint32_t v = 0;
      if (!live) {
      } else if constexpr (TUNED) {
        const int j = c / CPW, q = c % CPW;
        const uint32_t t = __ldg(row_words + (int64_t)(j >> 4) * 256 + (j & 15));
        if constexpr (BITS == 4) {
          v = t;
        } else if constexpr (BITS == 2) {
          // field 4p + c' at bits 2p + 8c'; chunk q holds p = 2q, 2q+1: shift them down to p = 0, 1
          const uint32_t u = t >> (4 * q);
          v = 0;
#pragma unroll
          for (int i = 0; i < 8; ++i) v |= ((u >> field_pos<2>(i, true)) & 3u) << (2 * i);
        } else {
          // field 2c' at bit 15 - c', field 2c'+1 at bit 31 - c'; chunk q holds c' = 4q .. 4q+3
          const uint32_t u = t << (4 * q);
          v = 0;
#pragma unroll
          for (int i = 0; i < 8; ++i) v |= ((u >> field_pos<1>(i, true)) & 1u) << i;
        }
      } else if constexpr (BITS == 4) {
        v = __ldg(row_words + c);
      } else if constexpr (BITS == 2) {
        v = __ldg(reinterpret_cast<const uint16_t*>(row_words) + c);
      } else {
        v = __ldg(reinterpret_cast<const uint8_t*>(row_words) + c);
      }
      const uint4 w8 = decode8<BITS>(v, c0, c1, row_cb);
      if (live) stg_stream_u4(out + c, w8);
    }
  }
}

// Table (bit-plane) layout: a thread gathers the plane bytes of one group of 8 weights, interleaves them into
// LSB-first index fields and stores the 8 decoded weights as one 16-byte piece.
template <int BITS>
__global__ void __launch_bounds__(256) dequant_table_kernel(const uint32_t* __restrict__ packed,
                                                            const uint16_t* __restrict__ cb, uint16_t* __restrict__ W,
                                                            int64_t N, int64_t K) {
  constexpr int Q = 1 << BITS;
  const uint8_t* bytes = reinterpret_cast<const uint8_t*>(packed);
  const int gpr = (int)(K >> 3);
  const int64_t chunks = table_chunks(K);
  for (int64_t n = blockIdx.x; n < N; n += gridDim.x) {
    const uint16_t* row_cb = cb + n * Q;
    uint32_t c0, c1;
    load_codebook<BITS>(row_cb, c0, c1);
    uint4* out = reinterpret_cast<uint4*>(W + n * K);
    for (int g = threadIdx.x; g < gpr; g += 256) {
      uint32_t v = __ldg(bytes + table_byte_offset(n, g, 0, chunks, BITS));
      if constexpr (BITS == 2) {
        const uint32_t hi = __ldg(bytes + table_byte_offset(n, g, 1, chunks, BITS));
        uint32_t z = 0;
#pragma unroll
        for (int t = 0; t < 8; ++t) z |= (((v >> t) & 1u) | (((hi >> t) & 1u) << 1)) << (2 * t);
        v = z;
      }
      stg_stream_u4(out + g, decode8<BITS>(v, c0, c1, row_cb));
    }
  }
}

}  // namespace

cudaError_t launch_dequant(const uint32_t* packed, const uint16_t* cb, uint16_t* W, int64_t N, int64_t K, int bits,
                           int layout, cudaStream_t s) {
  const DeviceInfo* di = device_info();
  if (!di) return cudaErrorInvalidDevice;
  const bool tuned = layout != KMQ_LAYOUT_CANONICAL;
  int64_t blocks = N;
  const int64_t cap = (int64_t)di->sm_count * 8;   // 8 resident CTAs of 256 threads per SM
  if (blocks > cap) blocks = cap;
  if (layout == KMQ_LAYOUT_TABLE && bits != 4) {
    if (bits == 1) dequant_table_kernel<1><<<(int)blocks, 256, 0, s>>>(packed, cb, W, N, K);
    else dequant_table_kernel<2><<<(int)blocks, 256, 0, s>>>(packed, cb, W, N, K);
    return cudaGetLastError();
  }
  if (bits == 1 && tuned) dequant_rows_kernel<1, true><<<(int)blocks, 256, 0, s>>>(packed, cb, W, N, K);
  else if (bits == 1) dequant_rows_kernel<1, false><<<(int)blocks, 256, 0, s>>>(packed, cb, W, N, K);
  else if (bits == 2 && tuned) dequant_rows_kernel<2, true><<<(int)blocks, 256, 0, s>>>(packed, cb, W, N, K);
  else if (bits == 2) dequant_rows_kernel<2, false><<<(int)blocks, 256, 0, s>>>(packed, cb, W, N, K);
  else if (tuned) dequant_rows_kernel<4, true><<<(int)blocks, 256, 0, s>>>(packed, cb, W, N, K);
  else dequant_rows_kernel<4, false><<<(int)blocks, 256, 0, s>>>(packed, cb, W, N, K);
  return cudaGetLastError();
}

}  // namespace kmq
