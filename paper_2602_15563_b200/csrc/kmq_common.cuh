// Shared device/host helpers for libkmq (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "kmq.h"

namespace kmq {

constexpr int kWarp = 32;

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

struct DeviceInfo {
  int sm_count;
  int max_smem_optin;
};
const DeviceInfo* device_info();  // cached per device; nullptr on CUDA error

// Launchers implemented in the kernel files (return cudaError_t of the launch).
cudaError_t launch_pack(const uint8_t* idx, int64_t N, int64_t K, int bits, uint32_t* packed, cudaStream_t s);
cudaError_t launch_unpack(const uint32_t* packed, int64_t N, int64_t K, int bits, uint8_t* idx, cudaStream_t s);
cudaError_t launch_dequant(const uint32_t* packed, const uint16_t* cb, uint16_t* W, int64_t N, int64_t K, int bits,
                           cudaStream_t s);

struct LinearPlan {
  int variant;        // index into the variant table
  int launches;       // kernels launched per call
  size_t workspace;   // bytes of scratch
  int split_k;        // K slices (1 = none)
  const char* name;
};
LinearPlan plan_linear(int64_t N, int64_t K, int bits, int64_t M);
cudaError_t launch_linear(const LinearPlan& plan, const uint32_t* packed, const uint16_t* cb, const uint16_t* x,
                          uint16_t* y, int64_t N, int64_t K, int bits, int64_t M, void* workspace, cudaStream_t s);

}  // namespace kmq
