// kmq_linear on the canonical packed layout, batch rows M <= 8 per pass: one CTA per 16 output rows, the
// warps of the CTA split K, every warp streams its slices of the packed rows
// with 128-bit loads (several in flight per lane), rebuilds the bf16 weights
// in registers directly in the operand layout of mma.sync.m16n8k16 (weights
// are the 16-row A operand, the batch is the 8-column B operand, fp32
// accumulators), and the partial sums of the warps are added through shared
// memory before the bf16 store.
//
// The integer pipe (64 lane-ops/clk/SM) and the shared-memory port
// (32 lanes/clk/SM) bound this kernel long before the FMA units do, so each
// bit width uses the cheapest exact decode that fits them:
//   b = 2  the row's 4 centroids are 8 bytes = the two source registers of
//          one byte-permute (PRMT); one PRMT yields two weights.
//   b = 4  a per-row table of all 256 (centroid, centroid) pairs in shared
//          memory, one copy per lane bank so lookups never conflict; one
//          32-bit LDS yields two weights.
//   b = 1  a shift puts two index bits on bits 15 and 31, a sign-replicating
//          PRMT spreads them over their half words and one LOP3 selects c0 or
//          c1: bit copies of the stored centroids.
// The order in which a word's fields reach the k-slots of an MMA is whatever
// is cheapest to extract; the activations are staged in shared memory in that
// same order, so the canonical packed layout is consumed as is.
#include "kmq_common.cuh"
#include "kmq_linear_variants.cuh"
#include "kmq_mma_common.cuh"

namespace kmq {
namespace {

constexpr int kWarps = 8;          // warps per CTA, all on the same 16 rows, K split between them
constexpr int kThreads = kWarps * 32;
constexpr int kStages = 4;         // 16-byte loads in flight per lane and row
constexpr int kRows = 16;          // output rows per CTA (one MMA tile)
constexpr int kPairTableBytes = 32768;  // 256 entries x 32 lane banks x 4 B
constexpr int kRedBytes = kWarps * 32 * 16;  // per warp: 32 lanes x 4 floats

template <int BITS>
struct Geo {
  static constexpr int kMmaPerWord = 8 / BITS;          // 16 k-slots per MMA = 4 lanes x 4 weights
  static constexpr int kSlots = 4 * kMmaPerWord;        // MMAs per step (a lane owns 4 words per step)
  static constexpr int kStepK = 512 / BITS;             // weights of one row consumed per step
  static constexpr int kWordK = 32 / BITS;
  static constexpr int kRowStride = kSlots * 32 + 32;   // bytes of staged activations per batch row (+pad)
  static constexpr int kTableBytes = BITS == 4 ? 2 * kPairTableBytes : 0;
};

template <int BITS, int MMAX>
constexpr int smem_bytes() {
  return Geo<BITS>::kTableBytes + kWarps * MMAX * Geo<BITS>::kRowStride + kRedBytes;
}

// ---------------------------------------------------------------------------
// Activation staging.  One step of one warp covers kStepK consecutive k; lane
// (g, t) of the MMA owns the 16-byte chunk t of that range, i.e. words j =
// 0..3 of kWordK weights each.  The activations of batch row m are stored as
// 8-byte units [slot = j*kMmaPerWord + q][t] holding the four k-slots lane t
// feeds to MMA (j, q), in the order the weight decode produces them.
// ---------------------------------------------------------------------------
template <int BITS>
__device__ __forceinline__ void stage_block(const uint16_t* __restrict__ xrow, int64_t k0, bool valid,
                                            unsigned char* dst) {
  // dst: unit [slot = j*kMmaPerWord][t] of this batch row; consecutive MMAs of the word are 32 bytes apart
  constexpr int Q = Geo<BITS>::kMmaPerWord;
  if constexpr (BITS == 4) {
    uint4 v = make_uint4(0, 0, 0, 0);
    if (valid) v = __ldg(reinterpret_cast<const uint4*>(xrow + k0));
    *reinterpret_cast<uint2*>(dst) = make_uint2(v.x, v.y);        // weights 0..3 of the word
    *reinterpret_cast<uint2*>(dst + 32) = make_uint2(v.z, v.w);   // weights 4..7
  } else if constexpr (BITS == 2) {
    uint32_t r[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (valid) {
      const uint4 v0 = __ldg(reinterpret_cast<const uint4*>(xrow + k0));
      const uint4 v1 = __ldg(reinterpret_cast<const uint4*>(xrow + k0 + 8));
      r[0] = v0.x; r[1] = v0.y; r[2] = v0.z; r[3] = v0.w; r[4] = v1.x; r[5] = v1.y; r[6] = v1.z; r[7] = v1.w;
    }
    // MMA q takes weights (q, q+4 | q+8, q+12) of the 16-weight word
#pragma unroll
    for (int q = 0; q < Q; ++q) {
      const uint32_t sel = (q & 1) ? 0x7632u : 0x5410u;
      const int base = q >> 1;
      *reinterpret_cast<uint2*>(dst + q * 32) =
          make_uint2(prmt(r[base], r[base + 2], sel), prmt(r[base + 4], r[base + 6], sel));
    }
  } else {
    uint32_t r[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) r[i] = 0;
    if (valid) {
#pragma unroll
      for (int v = 0; v < 4; ++v) {
        const uint4 u = __ldg(reinterpret_cast<const uint4*>(xrow + k0 + 8 * v));
        r[4 * v] = u.x; r[4 * v + 1] = u.y; r[4 * v + 2] = u.z; r[4 * v + 3] = u.w;
      }
    }
    // MMA e takes weights (15-2e, 31-2e | 14-2e, 30-2e) of the 32-weight word
#pragma unroll
    for (int e = 0; e < Q; ++e)
      *reinterpret_cast<uint2*>(dst + e * 32) =
          make_uint2(prmt(r[7 - e], r[15 - e], 0x7632u), prmt(r[7 - e], r[15 - e], 0x5410u));
  }
}

template <int BITS>
__device__ __forceinline__ void stage_step(const uint16_t* __restrict__ x, int64_t K, int M, int64_t step,
                                           unsigned char* xs_warp, int lane) {
  using G = Geo<BITS>;
  const int blk = lane & 15;                 // 16 word blocks per batch row: chunk t = blk / 4, word j = blk % 4
  const int t = blk >> 2, j = blk & 3;
  const int64_t k0 = step * G::kStepK + (int64_t)blk * G::kWordK;
  const bool in_k = k0 < K;
  for (int m = lane >> 4; m < M; m += 2)
    stage_block<BITS>(x + (int64_t)m * K, k0, in_k, xs_warp + m * G::kRowStride + j * G::kMmaPerWord * 32 + t * 8);
}

template <int BITS, int MMAX>
__global__ void __launch_bounds__(kThreads) linear_mma_kernel(const uint32_t* __restrict__ packed,
                                                              const uint16_t* __restrict__ cb,
                                                              const uint16_t* __restrict__ x, uint16_t* __restrict__ y,
                                                              int64_t N, int64_t K, int M) {
  using G = Geo<BITS>;
  constexpr int Q = G::kMmaPerWord;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  // [pair tables (b = 4)] [staged activations: kWarps x MMAX rows] [warp partials]
  unsigned char* const tables = smem_raw;
  unsigned char* const xs_all = smem_raw + G::kTableBytes;
  float* const red = reinterpret_cast<float*>(xs_all + kWarps * MMAX * G::kRowStride);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int64_t row0 = (int64_t)blockIdx.x * kRows;
  const int64_t wpr = K / G::kWordK;              // words per packed row
  const int64_t chunks = wpr >> 2;                // 16-byte chunks per row
  const int64_t steps = (chunks + 3) >> 2;
  const int64_t rg = min(row0 + g, N - 1), rh = min(row0 + g + 8, N - 1);   // clamped: loads stay inside the matrix
  const uint4* __restrict__ pg = reinterpret_cast<const uint4*>(packed + rg * wpr);
  const uint4* __restrict__ ph = reinterpret_cast<const uint4*>(packed + rh * wpr);
  unsigned char* const xs_warp = xs_all + warp * (MMAX * G::kRowStride);

  // ---- weight loads of the first kStages steps go out before anything else ----
  uint4 qa[kStages], qb[kStages];
#pragma unroll
  for (int d = 0; d < kStages; ++d) {
    const int64_t c = 4 * ((int64_t)warp + (int64_t)d * kWarps) + t;
    qa[d] = qb[d] = make_uint4(0, 0, 0, 0);
    if (c < chunks) {
      qa[d] = ldg_stream_u4(pg + c);
      qb[d] = ldg_stream_u4(ph + c);
    }
  }

  // ---- per-row decode state ----
  Dec1 sg, sh;
  if constexpr (BITS == 1) {
    sg.init(cb + rg * 2);
    sh.init(cb + rh * 2);
  }
  Dec2 dg, dh;
  if constexpr (BITS == 2) {
    dg.init(cb + rg * 4);
    dh.init(cb + rh * 4);
  }
  if constexpr (BITS == 4) {
    // entry e of row r: (C_r[e & 15], C_r[e >> 4]); the 4 lanes that share a row get one bank each.
    // Byte address of (half, e, lane) = half * 32 KB + e * 128 + lane * 4, lane = 4 * (r % 8) + t.
    const int r8 = threadIdx.x & 7, half = (threadIdx.x >> 3) & 1;
    const int64_t rr = min(row0 + r8 + 8 * half, N - 1);
    const uint16_t* crow = cb + rr * 16;
    for (int e = threadIdx.x >> 4; e < 256; e += kThreads / 16) {
      const uint32_t v = (uint32_t)__ldg(crow + (e & 15)) | ((uint32_t)__ldg(crow + (e >> 4)) << 16);
      *reinterpret_cast<uint4*>(tables + half * kPairTableBytes + e * 128 + r8 * 16) = make_uint4(v, v, v, v);
    }
    __syncthreads();
  }
  const uint32_t lane4 = lane * 4;

  float acc[4] = {0.f, 0.f, 0.f, 0.f};

  const unsigned char* const xb_lane = xs_warp + g * G::kRowStride + t * 8;   // B fragments: batch row g, chunk t
  const bool has_col = g < M;

  for (int64_t s0 = warp; s0 < steps; s0 += (int64_t)kStages * kWarps) {
#pragma unroll
    for (int d = 0; d < kStages; ++d) {
      const int64_t s = s0 + (int64_t)d * kWarps;
      if (s < steps) {   // warp-uniform
        __syncwarp();
        stage_step<BITS>(x, K, M, s, xs_warp, lane);
        __syncwarp();
        const uint32_t wa[4] = {qa[d].x, qa[d].y, qa[d].z, qa[d].w};
        const uint32_t wb[4] = {qb[d].x, qb[d].y, qb[d].z, qb[d].w};
        {  // refill this stage for the step kStages rounds ahead
          const int64_t c = 4 * (s + (int64_t)kStages * kWarps) + t;
          if (c < chunks) {
            qa[d] = ldg_stream_u4(pg + c);
            qb[d] = ldg_stream_u4(ph + c);
          }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
#pragma unroll
          for (int q = 0; q < Q; ++q) {
            uint2 b = make_uint2(0, 0);
            if (has_col) b = *reinterpret_cast<const uint2*>(xb_lane + (j * Q + q) * 32);
            uint32_t a0, a1, a2, a3;
            if constexpr (BITS == 2) {
              dg.pair(wa[j], q, a0, a2);
              dh.pair(wb[j], q, a1, a3);
            } else if constexpr (BITS == 4) {
              // bytes 2q and 2q+1 of the word hold weights (4q, 4q+1) and (4q+2, 4q+3)
              constexpr uint32_t kMask = 0x7F80u;
              const uint32_t oa0 = ((q == 0 ? (wa[j] << 7) : (wa[j] >> 9)) & kMask) | lane4;
              const uint32_t oa1 = ((q == 0 ? (wa[j] >> 1) : (wa[j] >> 17)) & kMask) | lane4;
              const uint32_t ob0 = ((q == 0 ? (wb[j] << 7) : (wb[j] >> 9)) & kMask) | lane4;
              const uint32_t ob1 = ((q == 0 ? (wb[j] >> 1) : (wb[j] >> 17)) & kMask) | lane4;
              a0 = *reinterpret_cast<const uint32_t*>(tables + oa0);
              a2 = *reinterpret_cast<const uint32_t*>(tables + oa1);
              a1 = *reinterpret_cast<const uint32_t*>(tables + kPairTableBytes + ob0);
              a3 = *reinterpret_cast<const uint32_t*>(tables + kPairTableBytes + ob1);
            } else {
              // pair c = 2q: weights (15-2q | 31-2q); pair c = 2q+1: weights (14-2q | 30-2q) on bits 15 and 31
              a0 = sg.select(wa[j] << (2 * q));
              a2 = sg.select(wa[j] << (2 * q + 1));
              a1 = sh.select(wb[j] << (2 * q));
              a3 = sh.select(wb[j] << (2 * q + 1));
            }
            mma_bf16_16816(acc, a0, a1, a2, a3, b.x, b.y);
          }
        }
      }
    }
  }

  // ---- add the partial sums of the warps, store ----
  *reinterpret_cast<float4*>(red + (warp * 32 + lane) * 4) = make_float4(acc[0], acc[1], acc[2], acc[3]);
  __syncthreads();
  if (threadIdx.x < kRows * 8) {
    const int r = threadIdx.x & 15, m = threadIdx.x >> 4;   // consecutive threads -> consecutive output rows
    const int64_t n = row0 + r;
    if (m < M && n < N) {
      const int src_lane = (r & 7) * 4 + (m >> 1), src_reg = (r >> 3) * 2 + (m & 1);
      float v = 0.f;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) v += red[(w * 32 + src_lane) * 4 + src_reg];
      y[(int64_t)m * N + n] = (uint16_t)float_to_bf16_bits(v);
    }
  }
}

template <int BITS, int MMAX>
cudaError_t launch_one(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
                       int64_t K, int M, cudaStream_t s) {
  constexpr int smem = smem_bytes<BITS, MMAX>();
  static bool configured[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(linear_mma_kernel<BITS, MMAX>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  const unsigned grid = (unsigned)((N + kRows - 1) / kRows);
  linear_mma_kernel<BITS, MMAX><<<grid, kThreads, smem, s>>>(packed, cb, x, y, N, K, M);
  return cudaGetLastError();
}

template <int BITS>
cudaError_t launch_bits(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
                        int64_t K, int M, cudaStream_t s) {
  if (M == 1) return launch_one<BITS, 1>(packed, cb, x, y, N, K, M, s);
  if (M == 2) return launch_one<BITS, 2>(packed, cb, x, y, N, K, M, s);
  if (M <= 4) return launch_one<BITS, 4>(packed, cb, x, y, N, K, M, s);
  return launch_one<BITS, 8>(packed, cb, x, y, N, K, M, s);
}

}  // namespace

bool linear_mma_supports(int64_t N, int64_t K, int bits, int64_t M) {
  (void)M;
  return (K * bits) % 128 == 0 && K <= (int64_t(1) << 30) && (N + kRows - 1) / kRows <= 0x7FFFFFFF;
}

// Batches larger than 8 are processed 8 rows at a time (one launch each).
cudaError_t launch_linear_mma(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
                              int64_t K, int bits, int64_t M, cudaStream_t s) {
  for (int64_t m0 = 0; m0 < M; m0 += 8) {
    const int mc = (int)(M - m0 < 8 ? M - m0 : 8);
    const uint16_t* xp = x + m0 * K;
    uint16_t* yp = y + m0 * N;
    cudaError_t e;
    if (bits == 1) e = launch_bits<1>(packed, cb, xp, yp, N, K, mc, s);
    else if (bits == 2) e = launch_bits<2>(packed, cb, xp, yp, N, K, mc, s);
    else e = launch_bits<4>(packed, cb, xp, yp, N, K, mc, s);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace kmq
