// Device helpers shared by the tensor-core kmq_linear kernels.
#pragma once
#include "kmq_common.cuh"

namespace kmq {

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}

// (a & b) | c in one LOP3 (the compiler does not merge an AND and an OR that both take immediates).
__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}

// b = 1: the two centroids of one row as bf16 pairs (c0, c0) and (c0 ^ c1, c0 ^ c1).  select() turns a word whose
// bits 15 and 31 are two index bits into the two weights, each a bit copy of a stored centroid: a sign-replicating
// PRMT spreads each bit over its half word, one LOP3 flips c0 into c1 where the bit is set.
struct Dec1 {
  uint32_t c00, dd;
  __device__ __forceinline__ void init(const uint16_t* __restrict__ cb_row) {
    const uint32_t c = __ldg(reinterpret_cast<const uint32_t*>(cb_row));
    c00 = prmt(c, c, 0x1010u);
    dd = c00 ^ prmt(c, c, 0x3232u);
  }
  __device__ __forceinline__ uint32_t select(uint32_t v) const {
    const uint32_t mask = prmt(v, v, 0xBB99u);
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0x6C;" : "=r"(d) : "r"(mask), "r"(c00), "r"(dd));   // c00 ^ (mask & dd)
    return d;
  }
};

// Powers of two read from constant memory: a multiply by one of these is a left shift that issues on the
// FMA pipe (IMAD) instead of the half-rate integer pipe that the decode saturates.
static __constant__ uint32_t kPow2[16] = {1u << 0, 1u << 1, 1u << 2,  1u << 3,  1u << 4,  1u << 5,  1u << 6,  1u << 7,
                                          1u << 8, 1u << 9, 1u << 10, 1u << 11, 1u << 12, 1u << 13, 1u << 14, 1u << 15};

// b = 2: byte tables {lo bytes of c0..c3}, {hi bytes of c0..c3} of one row
struct Dec2 {
  uint32_t lo, hi;
  __device__ __forceinline__ void init(const uint16_t* __restrict__ cb_row) {
    const uint2 c = __ldg(reinterpret_cast<const uint2*>(cb_row));
    lo = prmt(c.x, c.y, 0x6420u);
    hi = prmt(c.x, c.y, 0x7531u);
  }
  // phase q of a word: fields q, q+4, q+8, q+12 -> (W_q, W_q+4) and (W_q+8, W_q+12)
  __device__ __forceinline__ void pair(uint32_t w, int q, uint32_t& a_first, uint32_t& a_second) const {
    const uint32_t f = (w >> (2 * q)) & 0x03030303u;
    const uint32_t sel = f * 0x11u + 0x40404040u;   // per byte: nibbles (i, 4 + i) select (lo_i, hi_i)
    a_first = prmt(lo, hi, sel);
    a_second = prmt(lo, hi, sel >> 16);
  }
};

}  // namespace kmq
