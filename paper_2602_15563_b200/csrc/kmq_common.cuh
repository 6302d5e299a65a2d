// Shared device/host helpers for libkmq (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "kmq.h"

namespace kmq {

constexpr int kWarp = 32;
constexpr int kTileRows = 16;   // rows of one tile of the tuned layout (= rows of one MMA tile)

__host__ __device__ constexpr int fields_per_word(int bits) { return 32 / bits; }

// bf16 bit pattern -> fp32 (exact).
__device__ __forceinline__ float bf16_bits_to_float(uint32_t b) { return __uint_as_float(b << 16); }

// fp32 -> bf16 bit pattern, round-to-nearest-even (finite inputs).
__device__ __forceinline__ uint32_t float_to_bf16_bits(float f) {
  uint32_t u = __float_as_uint(f);
  u += 0x7FFFu + ((u >> 16) & 1u);
  return u >> 16;
}

__device__ __forceinline__ uint4 ldg_stream_u4(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

__device__ __forceinline__ void stg_stream_u4(uint4* p, uint4 v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
               : "memory");
}

// ---------------------------------------------------------------------------
// Packed layouts.  Word j of row n holds the indices idx[n, j*(32/bits) + i].
//   canonical: word (n, j) at n * wpr + j, field i at bits [i*bits, (i+1)*bits).
//   tuned:     tile-major.  Rows are grouped in tiles of 16 and a row's words in steps of 16 words (64 bytes);
//              step s of tile T is one contiguous 1 KB block holding the 64 bytes of each of the 16 rows, row
//              after row; every row is zero-padded to whole steps and N to whole tiles.  Inside a word the
//              fields sit where the tensor-core kernels extract four consecutive weights most cheaply.
// ---------------------------------------------------------------------------
template <int BITS>
__host__ __device__ constexpr int field_pos(int i, bool tuned) {
  if (!tuned || BITS == 4) return i * BITS;
  if (BITS == 2) return 2 * (i >> 2) + 8 * (i & 3);
  return (i & 1) ? 31 - (i >> 1) : 15 - (i >> 1);
}

// Word in the tuned layout -> the same fields in canonical order.
template <int BITS>
__device__ __forceinline__ uint32_t canonical_from_tuned(uint32_t t) {
  if constexpr (BITS == 4) {
    return t;
  } else {
    constexpr uint32_t MASK = (1u << BITS) - 1u;
    uint32_t w = 0;
#pragma unroll
    for (int i = 0; i < 32 / BITS; ++i) w |= ((t >> field_pos<BITS>(i, true)) & MASK) << (i * BITS);
    return w;
  }
}

__host__ __device__ inline int64_t tuned_steps(int64_t wpr) { return (wpr + 15) >> 4; }

// Index (in 32-bit words) of word j of row n in the tuned layout.
__host__ __device__ inline int64_t tuned_word_index(int64_t n, int64_t j, int64_t steps) {
  return ((((n >> 4) * steps + (j >> 4)) * kTileRows + (n & 15)) << 4) + (j & 15);
}

__host__ __device__ inline int64_t tuned_total_words(int64_t N, int64_t wpr) {
  return ((N + kTileRows - 1) / kTileRows) * tuned_steps(wpr) * 256;
}

struct DeviceInfo {
  int sm_count;
  int max_smem_optin;
};
const DeviceInfo* device_info();  // cached per device; nullptr on CUDA error

// Launchers implemented in the kernel files (return cudaError_t of the launch).
cudaError_t launch_pack(const uint8_t* idx, int64_t N, int64_t K, int bits, int layout, uint32_t* packed,
                        cudaStream_t s);
cudaError_t launch_unpack(const uint32_t* packed, int64_t N, int64_t K, int bits, int layout, uint8_t* idx,
                          cudaStream_t s);
cudaError_t launch_dequant(const uint32_t* packed, const uint16_t* cb, uint16_t* W, int64_t N, int64_t K, int bits,
                           int layout, cudaStream_t s);

struct LinearPlan {
  int variant;        // index into the variant table
  int launches;       // kernels launched per call
  size_t workspace;   // bytes of scratch
  int split_k;        // K slices (1 = none)
  const char* name;
};
LinearPlan plan_linear(int64_t N, int64_t K, int bits, int64_t M, int layout);
cudaError_t launch_linear(const LinearPlan& plan, const uint32_t* packed, const uint16_t* cb, const uint16_t* x,
                          uint16_t* y, int64_t N, int64_t K, int bits, int64_t M, int layout, void* workspace,
                          cudaStream_t s);

}  // namespace kmq
