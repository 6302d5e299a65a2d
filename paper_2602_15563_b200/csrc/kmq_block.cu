// The paper's own k-means block format: one codebook of 2^b centroids per weight tensor, one bf16 scale per block
// of 64 consecutive inputs of a row, indices packed along the input dimension into bytes (8 / b per byte, LSB
// first), b = 1, 2, 4, 8:   W^[n, k] = scale[n, k / 64] * c[idx[n, k]],   P_w = b + 0.25 bits per weight.
//
// kmq_block_linear: a CTA owns 8 or 16 output rows and walks K in slices of 32 blocks; a lane owns whole blocks (block
// g = lane of the slice: 8 b bytes, loaded as 8-, 16-byte or several 16-byte words, neighbouring lanes neighbouring blocks),
// so a block's 64 products stay in one thread and the block scale is applied either to every weight ("direct", the
// paper's first listing) or once to the block's sum ("deferred scaling", its second listing), both in fp32.  The
// codebook is a table in shared memory with one copy per lane bank (a lookup never conflicts); the activations of a
// slice are staged in shared memory once per CTA.  The 32 lanes' sums are added by shuffles, the result is rounded
// to bf16.
#include "kmq_common.cuh"

namespace kmq {
namespace {

constexpr int kBlock = 64;          // inputs per scale
constexpr int kBWarps = 8;

template <int BITS>
struct BGeo {
  static constexpr int kEntries = 1 << BITS;
  static constexpr int kBlockBytes = kBlock * BITS / 8;            // 8, 16, 32, 64
  static constexpr int kWords = kBlockBytes / 4;                   // 32-bit words of packed indices per block
  static constexpr int kPerWord = 32 / BITS;
  static constexpr int kTableBytes = kEntries * 32 * 4;            // fp32, entry e of lane l at (e * 32 + l) * 4
};

template <int WORDS>
__device__ __forceinline__ void load_words(const uint8_t* p, uint32_t (&w)[WORDS]) {
  if constexpr (WORDS == 2) {
    const uint2 v = __ldg(reinterpret_cast<const uint2*>(p));
    w[0] = v.x;
    w[1] = v.y;
  } else {
#pragma unroll
    for (int i = 0; i < WORDS / 4; ++i) {
      const uint4 v = ldg_stream_u4(reinterpret_cast<const uint4*>(p) + i);
      w[4 * i] = v.x;
      w[4 * i + 1] = v.y;
      w[4 * i + 2] = v.z;
      w[4 * i + 3] = v.w;
    }
  }
}

// Activations of one slice of 32 blocks (2048 inputs) in shared memory: block g of batch row m at
// (m * 32 + g) * kXBlockStride bytes; the 16 bytes of padding per block make the lanes' 128-bit reads (lane = block)
// conflict-free.
constexpr int kSliceBlocks = 32;
constexpr int kXBlockStride = kBlock * 2 + 16;

// A CTA of 8 warps owns 8 * ROWS consecutive output rows and walks K in slices of 32 blocks: the slice of x is copied
// to shared memory once per CTA (coalesced, double buffered), then lane g of every warp handles block g of the slice
// for the warp's ROWS rows.
template <int BITS, int MB, bool DEFER, int ROWS>
__global__ void __launch_bounds__(kBWarps * 32) block_linear_kernel(const uint8_t* __restrict__ wq,
                                                                    const uint16_t* __restrict__ scales,
                                                                    const uint16_t* __restrict__ codebook,
                                                                    const uint16_t* __restrict__ x,
                                                                    uint16_t* __restrict__ y, int64_t N, int64_t K,
                                                                    int M) {
  using G = BGeo<BITS>;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* const table = reinterpret_cast<float*>(smem_raw);
  unsigned char* const xs = smem_raw + G::kTableBytes;   // [2 buffers][MB][32 blocks][kXBlockStride]
  constexpr int kXBuf = MB * kSliceBlocks * kXBlockStride;
  for (int i = threadIdx.x; i < G::kEntries * 32; i += blockDim.x) table[i] = bf16_bits_to_float(__ldg(codebook + (i >> 5)));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const float* const tl = table + lane;
  const int64_t blocks = K / kBlock, row_bytes = K * BITS / 8;
  const int64_t n0 = ((int64_t)blockIdx.x * kBWarps + warp) * ROWS;
  const int slices = (int)((blocks + kSliceBlocks - 1) / kSliceBlocks);

  // 16-byte piece `threadIdx.x` of the slice of every batch row: block threadIdx.x / 8, piece threadIdx.x % 8
  auto stage = [&](int sl) {
    const int64_t g = (int64_t)sl * kSliceBlocks + (threadIdx.x >> 3);
#pragma unroll
    for (int m = 0; m < MB; ++m) {
      uint4 q = make_uint4(0, 0, 0, 0);
      if (m < M && g < blocks) q = __ldg(reinterpret_cast<const uint4*>(x + (int64_t)m * K + g * kBlock) + (threadIdx.x & 7));
      *reinterpret_cast<uint4*>(xs + (sl & 1) * kXBuf + (m * kSliceBlocks + (threadIdx.x >> 3)) * kXBlockStride +
                                (threadIdx.x & 7) * 16) = q;
    }
  };
  stage(0);
  float acc[ROWS][MB];
#pragma unroll
  for (int r = 0; r < ROWS; ++r)
#pragma unroll
    for (int m = 0; m < MB; ++m) acc[r][m] = 0.f;

  for (int sl = 0; sl < slices; ++sl) {
    __syncthreads();   // slice sl is staged (and the table, the first time); everybody is done with slice sl - 1
    if (sl + 1 < slices) stage(sl + 1);
    const int64_t g = (int64_t)sl * kSliceBlocks + lane;
    if (g < blocks && n0 < N) {
      uint32_t w[ROWS][G::kWords];
      float s[ROWS];
#pragma unroll
      for (int r = 0; r < ROWS; ++r) {
        const int64_t n = n0 + r < N ? n0 + r : N - 1;   // a row past the end re-reads the last one; it is not stored
        load_words<G::kWords>(wq + n * row_bytes + g * G::kBlockBytes, w[r]);
        s[r] = bf16_bits_to_float(__ldg(scales + n * blocks + g));
      }
      float part[ROWS][MB];
#pragma unroll
      for (int r = 0; r < ROWS; ++r)
#pragma unroll
        for (int m = 0; m < MB; ++m) part[r][m] = 0.f;
      const unsigned char* const xb = xs + (sl & 1) * kXBuf + lane * kXBlockStride;
#pragma unroll
      for (int p = 0; p < kBlock / 8; ++p) {   // 8 inputs at a time: one 16-byte piece of x per batch row
        float xv[MB][8];
#pragma unroll
        for (int m = 0; m < MB; ++m) {
          const uint4 q = *reinterpret_cast<const uint4*>(xb + m * kSliceBlocks * kXBlockStride + p * 16);
          const uint32_t qq[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            xv[m][2 * i] = __uint_as_float(qq[i] << 16);
            xv[m][2 * i + 1] = __uint_as_float(qq[i] & 0xFFFF0000u);
          }
        }
#pragma unroll
        for (int r = 0; r < ROWS; ++r) {
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int k = p * 8 + i;   // weight k of the block: field k % per of word k / per, LSB first
            const uint32_t idx = (w[r][k / G::kPerWord] >> ((k % G::kPerWord) * BITS)) & (G::kEntries - 1);
            float c = tl[idx * 32];
            if constexpr (!DEFER) c *= s[r];
#pragma unroll
            for (int m = 0; m < MB; ++m) part[r][m] = fmaf(xv[m][i], c, part[r][m]);
          }
        }
      }
#pragma unroll
      for (int r = 0; r < ROWS; ++r)
#pragma unroll
        for (int m = 0; m < MB; ++m) acc[r][m] = DEFER ? fmaf(s[r], part[r][m], acc[r][m]) : acc[r][m] + part[r][m];
    }
  }
#pragma unroll
  for (int r = 0; r < ROWS; ++r)
#pragma unroll
    for (int m = 0; m < MB; ++m) {
      float v = acc[r][m];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
      if (lane == 0 && m < M && n0 + r < N) y[(int64_t)m * N + n0 + r] = (uint16_t)float_to_bf16_bits(v);
    }
}

// W[n, k] = bf16(scale * centroid): the product of two bf16 numbers is exact in fp32, one rounding to nearest even.
template <int BITS>
__global__ void __launch_bounds__(256) block_dequant_kernel(const uint8_t* __restrict__ wq,
                                                            const uint16_t* __restrict__ scales,
                                                            const uint16_t* __restrict__ codebook,
                                                            uint16_t* __restrict__ W, int64_t N, int64_t K) {
  constexpr int E = 1 << BITS;
  __shared__ float table[E];
  for (int i = threadIdx.x; i < E; i += blockDim.x) table[i] = bf16_bits_to_float(__ldg(codebook + i));
  __syncthreads();
  const int64_t groups = N * (K / 8);   // 8 weights = BITS bytes in, 16 bytes out
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < groups; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t n = i / (K / 8), k0 = (i % (K / 8)) * 8;
    const uint8_t* src = wq + n * (K * BITS / 8) + k0 * BITS / 8;
    uint64_t bits8 = 0;
#pragma unroll
    for (int b = 0; b < BITS; ++b) bits8 |= (uint64_t)__ldg(src + b) << (8 * b);
    const float s = bf16_bits_to_float(__ldg(scales + n * (K / kBlock) + k0 / kBlock));
    uint32_t o[4];
#pragma unroll
    for (int p = 0; p < 4; ++p) {
      const uint32_t i0 = (uint32_t)(bits8 >> (2 * p * BITS)) & (E - 1), i1 = (uint32_t)(bits8 >> ((2 * p + 1) * BITS)) & (E - 1);
      o[p] = float_to_bf16_bits(s * table[i0]) | (float_to_bf16_bits(s * table[i1]) << 16);
    }
    stg_stream_u4(reinterpret_cast<uint4*>(W + n * K + k0), make_uint4(o[0], o[1], o[2], o[3]));
  }
}

// idx uint8 [N, K] -> bytes [N, K * BITS / 8], fields LSB first; one thread per output byte.
template <int BITS>
__global__ void __launch_bounds__(256) block_pack_kernel(const uint8_t* __restrict__ idx, uint8_t* __restrict__ wq,
                                                         int64_t total_bytes) {
  constexpr int PER = 8 / BITS;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total_bytes; i += (int64_t)gridDim.x * blockDim.x) {
    uint32_t out = 0;
#pragma unroll
    for (int f = 0; f < PER; ++f) out |= (uint32_t)(idx[i * PER + f] & ((1u << BITS) - 1u)) << (f * BITS);
    wq[i] = (uint8_t)out;
  }
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

kmq_status check_block_shape(int64_t N, int64_t K, int bits, int64_t M) {
  if (bits != 1 && bits != 2 && bits != 4 && bits != 8) return KMQ_ERR_BITS;
  if (N < 1 || M < 1 || K < kBlock || (K % kBlock) != 0) return KMQ_ERR_SHAPE;
  if (N > (int64_t(1) << 31) || K > (int64_t(1) << 31) || M > (int64_t(1) << 24)) return KMQ_ERR_SHAPE;
  return KMQ_OK;
}

template <int BITS, int MB, int ROWS>
cudaError_t launch_block_mb(const uint8_t* wq, const uint16_t* scales, const uint16_t* cb, const uint16_t* x, uint16_t* y,
                            int64_t N, int64_t K, int M, bool defer, int sm_count, cudaStream_t s) {
  constexpr int smem = BGeo<BITS>::kTableBytes + 2 * MB * kSliceBlocks * kXBlockStride;
  (void)sm_count;
  const int64_t grid = (N + kBWarps * ROWS - 1) / (kBWarps * ROWS);
  static bool configured[64][2] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !configured[dev][defer]) {
    cudaError_t e = defer ? cudaFuncSetAttribute(block_linear_kernel<BITS, MB, true, ROWS>,
                                                 cudaFuncAttributeMaxDynamicSharedMemorySize, smem)
                          : cudaFuncSetAttribute(block_linear_kernel<BITS, MB, false, ROWS>,
                                                 cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    configured[dev][defer] = true;
  }
  if (defer)
    block_linear_kernel<BITS, MB, true, ROWS><<<(int)grid, kBWarps * 32, smem, s>>>(wq, scales, cb, x, y, N, K, M);
  else
    block_linear_kernel<BITS, MB, false, ROWS><<<(int)grid, kBWarps * 32, smem, s>>>(wq, scales, cb, x, y, N, K, M);
  return cudaGetLastError();
}

template <int BITS, int MB>
cudaError_t launch_block_rows(const uint8_t* wq, const uint16_t* scales, const uint16_t* cb, const uint16_t* x,
                              uint16_t* y, int64_t N, int64_t K, int M, bool defer, int sm_count, cudaStream_t s) {
  // two rows per warp only where that still gives every SM four CTAs
  if (N >= (int64_t)sm_count * 4 * kBWarps * 2)
    return launch_block_mb<BITS, MB, 2>(wq, scales, cb, x, y, N, K, M, defer, sm_count, s);
  return launch_block_mb<BITS, MB, 1>(wq, scales, cb, x, y, N, K, M, defer, sm_count, s);
}

template <int BITS>
cudaError_t launch_block_bits(const uint8_t* wq, const uint16_t* scales, const uint16_t* cb, const uint16_t* x,
                              uint16_t* y, int64_t N, int64_t K, int64_t M, bool defer, cudaStream_t s) {
  const DeviceInfo* di = device_info();
  if (!di) return cudaErrorInvalidDevice;
  const int grid = di->sm_count;
  for (int64_t m0 = 0; m0 < M; m0 += 4) {   // up to 4 batch rows per pass
    const int mc = (int)(M - m0 < 4 ? M - m0 : 4);
    const uint16_t* xp = x + m0 * K;
    uint16_t* yp = y + m0 * N;
    cudaError_t e = mc == 1   ? launch_block_rows<BITS, 1>(wq, scales, cb, xp, yp, N, K, mc, defer, grid, s)
                    : mc == 2 ? launch_block_rows<BITS, 2>(wq, scales, cb, xp, yp, N, K, mc, defer, grid, s)
                              : launch_block_rows<BITS, 4>(wq, scales, cb, xp, yp, N, K, mc, defer, grid, s);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace
}  // namespace kmq

using namespace kmq;

extern "C" {

size_t kmq_block_packed_bytes(int64_t N, int64_t K, int bits) {
  return check_block_shape(N, K, bits, 1) == KMQ_OK ? (size_t)N * (size_t)K * bits / 8 : 0;
}

kmq_status kmq_block_pack(const uint8_t* idx, int64_t N, int64_t K, int bits, uint8_t* wq, void* stream) {
  if (!idx || !wq) return KMQ_ERR_NULL;
  if (kmq_status s = check_block_shape(N, K, bits, 1)) return s;
  if (!aligned16(idx) || !aligned16(wq)) return KMQ_ERR_ALIGN;
  const DeviceInfo* di = device_info();
  if (!di) return KMQ_ERR_CUDA;
  const int64_t total = N * K * bits / 8;
  int64_t grid = (total + 255) / 256;
  if (grid > (int64_t)di->sm_count * 16) grid = (int64_t)di->sm_count * 16;
  cudaStream_t s = (cudaStream_t)stream;
  if (bits == 1) block_pack_kernel<1><<<(int)grid, 256, 0, s>>>(idx, wq, total);
  else if (bits == 2) block_pack_kernel<2><<<(int)grid, 256, 0, s>>>(idx, wq, total);
  else if (bits == 4) block_pack_kernel<4><<<(int)grid, 256, 0, s>>>(idx, wq, total);
  else block_pack_kernel<8><<<(int)grid, 256, 0, s>>>(idx, wq, total);
  return cudaGetLastError() == cudaSuccess ? KMQ_OK : KMQ_ERR_CUDA;
}

kmq_status kmq_block_linear(const uint8_t* wq, const uint16_t* scales, const uint16_t* codebook, const uint16_t* x,
                            uint16_t* y, int64_t N, int64_t K, int bits, int64_t M, int scale_order, void* stream) {
  if (!wq || !scales || !codebook || !x || !y) return KMQ_ERR_NULL;
  if (kmq_status s = check_block_shape(N, K, bits, M)) return s;
  if (scale_order != KMQ_SCALE_DIRECT && scale_order != KMQ_SCALE_DEFERRED) return KMQ_ERR_LAYOUT;
  if (!aligned16(wq) || !aligned16(scales) || !aligned16(codebook) || !aligned16(x) || !aligned16(y)) return KMQ_ERR_ALIGN;
  const bool defer = scale_order == KMQ_SCALE_DEFERRED;
  cudaStream_t s = (cudaStream_t)stream;
  cudaError_t e = bits == 1   ? launch_block_bits<1>(wq, scales, codebook, x, y, N, K, M, defer, s)
                  : bits == 2 ? launch_block_bits<2>(wq, scales, codebook, x, y, N, K, M, defer, s)
                  : bits == 4 ? launch_block_bits<4>(wq, scales, codebook, x, y, N, K, M, defer, s)
                              : launch_block_bits<8>(wq, scales, codebook, x, y, N, K, M, defer, s);
  return e == cudaSuccess ? KMQ_OK : KMQ_ERR_CUDA;
}

kmq_status kmq_block_dequant_to_bf16(const uint8_t* wq, const uint16_t* scales, const uint16_t* codebook, uint16_t* W,
                                     int64_t N, int64_t K, int bits, void* stream) {
  if (!wq || !scales || !codebook || !W) return KMQ_ERR_NULL;
  if (kmq_status s = check_block_shape(N, K, bits, 1)) return s;
  if (!aligned16(wq) || !aligned16(scales) || !aligned16(codebook) || !aligned16(W)) return KMQ_ERR_ALIGN;
  const DeviceInfo* di = device_info();
  if (!di) return KMQ_ERR_CUDA;
  int64_t grid = (N * (K / 8) + 255) / 256;
  if (grid > (int64_t)di->sm_count * 16) grid = (int64_t)di->sm_count * 16;
  cudaStream_t s = (cudaStream_t)stream;
  if (bits == 1) block_dequant_kernel<1><<<(int)grid, 256, 0, s>>>(wq, scales, codebook, W, N, K);
  else if (bits == 2) block_dequant_kernel<2><<<(int)grid, 256, 0, s>>>(wq, scales, codebook, W, N, K);
  else if (bits == 4) block_dequant_kernel<4><<<(int)grid, 256, 0, s>>>(wq, scales, codebook, W, N, K);
  else block_dequant_kernel<8><<<(int)grid, 256, 0, s>>>(wq, scales, codebook, W, N, K);
  return cudaGetLastError() == cudaSuccess ? KMQ_OK : KMQ_ERR_CUDA;
}

}  // extern "C"
