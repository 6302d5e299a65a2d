// Generic kmq_linear kernel: any legal shape, one warp per output row, CUDA-core
// FMAs.  It is the fallback for shapes the tuned kernels do not cover.
#include "kmq_common.cuh"
#include "kmq_linear_variants.cuh"

namespace kmq {
namespace {

constexpr int kWarpsPerCta = 8;

template <int BITS, int MB, bool TUNED>
__global__ void __launch_bounds__(kWarpsPerCta * 32) linear_generic_kernel(
    const uint32_t* __restrict__ packed, const uint16_t* __restrict__ cb, const uint16_t* __restrict__ x,
    uint16_t* __restrict__ y, int64_t N, int64_t K, int64_t M) {
  constexpr int PER = 32 / BITS;
  constexpr int Q = 1 << BITS;
  constexpr uint32_t MASK = Q - 1;
  __shared__ float cbs[kWarpsPerCta][Q];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t n = (int64_t)blockIdx.x * kWarpsPerCta + warp;
  if (n >= N) return;  // whole warp leaves together; only warp-level syncs below
  if (lane < Q) cbs[warp][lane] = bf16_bits_to_float(cb[n * Q + lane]);
  __syncwarp();

  const int64_t wpr = K / PER;
  const uint32_t* row = packed + n * wpr;   // canonical layout only
  const int64_t steps = tuned_steps(wpr);
  for (int64_t m0 = 0; m0 < M; m0 += MB) {
    float acc[MB];
#pragma unroll
    for (int mm = 0; mm < MB; ++mm) acc[mm] = 0.f;
    for (int64_t j = lane; j < wpr; j += 32) {
      const uint32_t word =
          TUNED ? canonical_from_tuned<BITS>(__ldg(packed + tuned_word_index(n, j, steps))) : __ldg(row + j);
#pragma unroll
      for (int q = 0; q < PER / 8; ++q) {
        float wv[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) wv[i] = cbs[warp][(word >> ((q * 8 + i) * BITS)) & MASK];
#pragma unroll
        for (int mm = 0; mm < MB; ++mm) {
          if (m0 + mm < M) {
            const uint4 xv = __ldg(reinterpret_cast<const uint4*>(x + (m0 + mm) * K + j * PER + q * 8));
            const uint32_t xr[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
            for (int p = 0; p < 4; ++p) {
              acc[mm] = fmaf(wv[2 * p], __uint_as_float(xr[p] << 16), acc[mm]);
              acc[mm] = fmaf(wv[2 * p + 1], __uint_as_float(xr[p] & 0xFFFF0000u), acc[mm]);
            }
          }
        }
      }
    }
#pragma unroll
    for (int mm = 0; mm < MB; ++mm) {
      float v = acc[mm];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
      if (lane == 0 && m0 + mm < M) y[(m0 + mm) * N + n] = (uint16_t)float_to_bf16_bits(v);
    }
  }
}

}  // namespace

cudaError_t launch_linear_generic(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
                                  int64_t K, int bits, int64_t M, int layout, cudaStream_t s) {
  const unsigned grid = (unsigned)((N + kWarpsPerCta - 1) / kWarpsPerCta);
  const int threads = kWarpsPerCta * 32;
  const bool tuned = layout == KMQ_LAYOUT_TUNED;
  if (bits == 1 && tuned) linear_generic_kernel<1, 4, true><<<grid, threads, 0, s>>>(packed, cb, x, y, N, K, M);
  else if (bits == 1) linear_generic_kernel<1, 4, false><<<grid, threads, 0, s>>>(packed, cb, x, y, N, K, M);
  else if (bits == 2 && tuned) linear_generic_kernel<2, 4, true><<<grid, threads, 0, s>>>(packed, cb, x, y, N, K, M);
  else if (bits == 2) linear_generic_kernel<2, 4, false><<<grid, threads, 0, s>>>(packed, cb, x, y, N, K, M);
  else if (tuned) linear_generic_kernel<4, 4, true><<<grid, threads, 0, s>>>(packed, cb, x, y, N, K, M);
  else linear_generic_kernel<4, 4, false><<<grid, threads, 0, s>>>(packed, cb, x, y, N, K, M);
  return cudaGetLastError();
}

}  // namespace kmq
