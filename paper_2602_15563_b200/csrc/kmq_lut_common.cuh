// Device helpers shared by the activation-table kernels (per-row codebooks: kmq_linear_lut.cu; block format:
// kmq_block_lut.cu): absolute shared-memory addressing of the tables, bulk asynchronous copies with mbarriers and
// time-bounded waits, the 16-lookup step.
#pragma once
#include "kmq_common.cuh"
#include "kmq_mma_common.cuh"

namespace kmq {

constexpr uint32_t kLutTableBase = 65536;   // absolute shared-memory byte address of table slot 0

// Offset of table slot q from slot 0.  The lookup addresses carry kLutTableBase in their registers, so that the
// immediate of a lookup is only this.
__host__ __device__ constexpr uint32_t lut_slot_offset(int q) {
  return (uint32_t)(q >> 1) * 65536u + (uint32_t)(q & 1) * 128u;
}

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

template <uint32_t IMM>
__device__ __forceinline__ float lds_f32(uint32_t addr) {
  float v;
  asm volatile("ld.shared.f32 %0, [%1+%2];" : "=f"(v) : "r"(addr), "n"(IMM));
  return v;
}

__device__ __forceinline__ uint4 lds_u4(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}

__device__ __forceinline__ void sts_f32(uint32_t addr, float v) {
  asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}

template <int LUT>
__device__ __forceinline__ uint32_t lop3(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, %4;" : "=r"(d) : "r"(a), "r"(b), "r"(c), "n"(LUT));
  return d;
}

// ---- mbarrier + bulk copy ----
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// global -> shared bulk copy; `bytes` a multiple of 16, both addresses 16-byte aligned; local memory only
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Wait for phase `parity` of an mbarrier, at most about kWaitNs: false when the time ran out.
constexpr uint64_t kWaitNs = 100ull * 1000 * 1000;
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(done)
      : "r"(bar), "r"(parity)
      : "memory");
  return done != 0;
}
static __device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity) {
  uint64_t t0 = 0;
  for (uint32_t i = 0;; ++i) {
    if (mbar_try(bar, parity)) return true;
    if ((i & 31u) == 31u) {
      const uint64_t now = global_timer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > kWaitNs) return false;
    }
  }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  return mbar_try(bar, parity) || mbar_wait_slow(bar, parity);
}

// 16 lookups of one 16-byte plane piece: byte k of word i -> table column of step 4i + k.
template <uint32_t IMM>
__device__ __forceinline__ void lookup16(const uint32_t (&w)[4], const uint32_t (&base)[16], float& acc0, float& acc1) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    acc0 += lds_f32<IMM>(prmt(w[i], base[4 * i + 0], 0x7604u));
    acc1 += lds_f32<IMM>(prmt(w[i], base[4 * i + 1], 0x7614u));
    acc0 += lds_f32<IMM>(prmt(w[i], base[4 * i + 2], 0x7624u));
    acc1 += lds_f32<IMM>(prmt(w[i], base[4 * i + 3], 0x7634u));
  }
}

// The same in table slot q.  The slot offset must be an immediate: q is a compile-time constant wherever this is
// called (an unrolled loop index), so the switch folds away.
__device__ __forceinline__ void lookup16_slot(int q, const uint32_t (&w)[4], const uint32_t (&base)[16], float& acc0,
                                              float& acc1) {
  switch (q) {
    case 0: lookup16<lut_slot_offset(0)>(w, base, acc0, acc1); break;
    case 1: lookup16<lut_slot_offset(1)>(w, base, acc0, acc1); break;
    case 2: lookup16<lut_slot_offset(2)>(w, base, acc0, acc1); break;
    default: lookup16<lut_slot_offset(3)>(w, base, acc0, acc1); break;
  }
}

constexpr unsigned int kErrWait = 1u, kErrWindow = 2u;   // bits of the device error word

// Device address of the table kernels' sticky error word (defined in kmq_linear_lut.cu), looked up once per device.
unsigned int* lut_error_word(cudaError_t* e);

}  // namespace kmq
