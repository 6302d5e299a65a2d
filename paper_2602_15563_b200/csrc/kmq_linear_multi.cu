// kmq_linear on the tuned (tile-major) layout for batches of up to 64 rows per launch (chosen from 4, 5 or 9 rows
// on, see linear_multi_min_rows): the tiles of a CTA share the staged activations, and the decode of a weight
// fragment is paid once and reused by up to 8 MMAs (one per group of 8 batch rows).
//
// One CTA owns TPC = 4 (or 2) tiles of 16 output rows.  Its 8 warps are 8 / TPC K-groups of TPC warps; warp
// (group, i) owns tile i and the steps s = group, group + 8 / TPC, ... of it.  The warps of a K-group walk the
// same steps together and share the activations under a step: they are copied global -> shared with cp.async, double buffered, one named barrier per
// step.  Per step a warp decodes its 1 KB of packed indices (two 128-bit loads issued one step earlier) into
// mma.sync.m16n8k16 A fragments and multiplies each fragment with the NT B fragments (batch rows 8 nt .. 8 nt + 7)
// read from shared memory.  At the end the other K-groups hand their accumulators to the first through shared
// memory, which adds them, applies the b = 1 codebook and stores bf16.
//
// b = 4 uses single-entry per-row tables here (16 entries x 32 lane banks, 4 KB per tile; one LDS per weight and a
// PRMT per pair): the 64 KB pair tables of the GEMV kernel would not fit for 4 tiles, and the decode is amortised
// over NT MMAs anyway.
#include "kmq_common.cuh"
#include "kmq_linear_variants.cuh"
#include "kmq_mma_common.cuh"

namespace kmq {
namespace {

constexpr int kTableBytesPerTile = 2 * 16 * 32 * 4;   // b = 4: [half][entry][lane] words
constexpr int kMaxSmem = 200 * 1024;                  // dynamic shared memory a variant may ask for

template <int BITS>
struct MGeo {
  static constexpr int kMmaPerWord = 8 / BITS;
  static constexpr int kStepK = 512 / BITS;
  static constexpr int kWordK = 32 / BITS;
  static constexpr int kChunkXBytes = 4 * kWordK * 2;     // activations under one 16-byte chunk of a row
  static constexpr int kChunkStride = kChunkXBytes + 16;  // +16 bytes: conflict-free 16-byte B-fragment loads
  static constexpr int kRowStride = 4 * kChunkStride;     // one batch row of one step
  static constexpr int kPiecesPerRow = kStepK / 8;        // 16-byte pieces per batch row and step
};

// TPC tiles per CTA (2 or 4), W warps -> W / TPC K-groups of TPC warps
template <int BITS, int NT, int TPC, int W = 8>
struct MSmem {
  using G = MGeo<BITS>;
  static constexpr int kGroups = W / TPC;
  static constexpr int kTableBytes = BITS == 4 ? TPC * kTableBytesPerTile : 0;
  static constexpr int kBuf = 8 * NT * G::kRowStride;                 // one x buffer: 8 NT batch rows of one step
  static constexpr int kX = kGroups * 2 * kBuf;                       // double buffered, per K-group
  static constexpr int kRed = (kGroups - 1) * TPC * 32 * NT * 4 * 4;  // accumulators of K-groups 1.. (aliases x)
  static constexpr int kTotal = kTableBytes + (kX > kRed ? kX : kRed);
};

template <int BITS>
__device__ __forceinline__ int piece_offset(int w) {
  using G = MGeo<BITS>;
  constexpr int kPiecesPerChunk = G::kChunkXBytes / 16;
  return (w / kPiecesPerChunk) * G::kChunkStride + (w % kPiecesPerChunk) * 16;
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src, bool valid) {
  const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
  const int bytes = valid ? 16 : 0;   // 0 source bytes: the 16 destination bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(gmem_src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void group_barrier(int group, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(group + 1), "r"(threads) : "memory");
}

template <int BITS, int NT, int TPC, int W = 8>
__global__ void __launch_bounds__(W * 32, (W == 8 && NT <= 2 && TPC == 2) ? 2 : 1) linear_multi_kernel(const uint32_t* __restrict__ packed,
                                                                    const uint16_t* __restrict__ cb,
                                                                    const uint16_t* __restrict__ x,
                                                                    uint16_t* __restrict__ y, int64_t N, int64_t K,
                                                                    int M) {
  using G = MGeo<BITS>;
  using SM = MSmem<BITS, NT, TPC, W>;
  constexpr int kThreads = W * 32;
  constexpr int Q = G::kMmaPerWord;
  constexpr int kGroups = SM::kGroups, kGroupThreads = TPC * 32;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  unsigned char* const tables = smem_raw;
  unsigned char* const xbase = smem_raw + SM::kTableBytes;
  float* const red = reinterpret_cast<float*>(xbase);                       // reused after the main loop

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int wt = warp % TPC, group = warp / TPC;       // tile inside the CTA, K-group
  const int gtid = threadIdx.x - group * kGroupThreads;  // thread inside the K-group
  const int64_t tiles = (N + kTileRows - 1) / kTileRows;
  const int64_t tile_id = (int64_t)blockIdx.x * TPC + wt;
  const bool has_tile = tile_id < tiles;               // warp-uniform; such a warp still stages x and joins barriers
  const int64_t row0 = tile_id * kTileRows;
  const int chunks = (int)(K / (4 * G::kWordK));
  const int steps = (chunks + 3) >> 2;
  const uint4* __restrict__ tile =
      reinterpret_cast<const uint4*>(packed) + (has_tile ? tile_id : 0) * (int64_t)steps * 64 + lane;
  unsigned char* const xgroup = xbase + group * 2 * SM::kBuf;

  // copy the activations under step s into buffer `buf` of this K-group (zeros past K; rows >= M are not touched:
  // their MMA columns are never stored)
  auto stage = [&](int s, int buf) {
    unsigned char* dst = xgroup + buf * SM::kBuf;
    const int total = M * G::kPiecesPerRow;
    for (int p = gtid; p < total; p += kGroupThreads) {
      const int m = p / G::kPiecesPerRow, w = p % G::kPiecesPerRow;
      const int64_t k = (int64_t)s * G::kStepK + w * 8;
      const bool ok = k < K;
      cp_async16(dst + m * G::kRowStride + piece_offset<BITS>(w), x + (int64_t)m * K + (ok ? k : 0), ok);
    }
    cp_async_commit();
  };

  // ---- first loads: weights of this warp's first two steps, activations of the group's first step ----
  uint4 qa[2], qb[2];
#pragma unroll
  for (int d = 0; d < 2; ++d) {
    const int s = group + d * kGroups;
    qa[d] = qb[d] = make_uint4(0, 0, 0, 0);
    if (has_tile && s < steps) {
      qa[d] = ldg_stream_u4(tile + (int64_t)s * 64);
      qb[d] = ldg_stream_u4(tile + (int64_t)s * 64 + 32);
    }
  }
  // ---- per-row decode state ----
  Dec1 sg, sh;
  if constexpr (BITS == 1) {
    sg.init(cb + min(row0 + g, N - 1) * 2);
    sh.init(cb + min(row0 + g + 8, N - 1) * 2);
  }
  Dec2 dg, dh;
  if constexpr (BITS == 2) {
    dg.init(cb + min(row0 + g, N - 1) * 4);
    dh.init(cb + min(row0 + g + 8, N - 1) * 4);
  }
  if constexpr (BITS == 4) {
    // word (tile, half, entry e, lane) = C_row[e] in both halves, row = 16 tile + 8 half + lane / 4
    for (int i = threadIdx.x; i < TPC * 2 * 16 * 32; i += kThreads) {
      const int ln = i & 31, e = (i >> 5) & 15, half = (i >> 9) & 1, tl = i >> 10;
      const int64_t r = min(((int64_t)blockIdx.x * TPC + tl) * kTileRows + 8 * half + (ln >> 2), N - 1);
      const uint32_t c = __ldg(cb + r * 16 + e);
      reinterpret_cast<uint32_t*>(tables)[i] = c | (c << 16);
    }
    __syncthreads();
  }
  // Programmatic dependent launch: up to here only the packed indices and the codebooks were read (constants of the
  // layer); the activations may come from the previous kernel on the stream and are read only once it has completed.
  // At b = 4, where the set-up of a CTA is long (its tables), the next kernel is released at once so that its CTAs
  // set up under this grid's MMAs; otherwise just before the partial sums are exchanged (measured, 4096 x 4096 M = 16:
  // b = 4 9.7 -> 8.3 us early, 8.7 late; b = 2 6.4 -> 6.3 / 6.5; 8192 x 8192 b = 2 M = 32 20.1 -> 20.1 / 19.5).
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if constexpr (BITS == 4) asm volatile("griddepcontrol.launch_dependents;");
  if (group < steps) stage(group, 0);
  const unsigned char* const tab_g = tables + wt * kTableBytesPerTile;   // rows g; rows g + 8 are 2 KB further
  const uint32_t lane4 = lane * 4;

  float acc[NT][4];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;

  for (int s0 = group; s0 < steps; s0 += 2 * kGroups) {   // uniform over the K-group
#pragma unroll
   for (int buf = 0; buf < 2; ++buf) {                     // buffer index = parity of the group's step count
    const int s = s0 + buf * kGroups;
    if (s >= steps) break;
    cp_async_wait_all();
    group_barrier(group, kGroupThreads);   // x of step s is in place, and every warp of the group is done with step s - 2
    if (s + kGroups < steps) stage(s + kGroups, buf ^ 1);
    const unsigned char* const xs = xgroup + buf * SM::kBuf;
    if (has_tile) {
      const uint4 va = qa[buf], vb = qb[buf];
      const uint32_t wa[4] = {va.x, va.y, va.z, va.w};
      const uint32_t wb[4] = {vb.x, vb.y, vb.z, vb.w};
      if (s + 2 * kGroups < steps) {   // refill for the step after next
        qa[buf] = ldg_stream_u4(tile + (int64_t)(s + 2 * kGroups) * 64);
        qb[buf] = ldg_stream_u4(tile + (int64_t)(s + 2 * kGroups) * 64 + 32);
      }
      const unsigned char* const xb = xs + g * G::kRowStride + t * G::kChunkStride;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
#pragma unroll
        for (int q2 = 0; q2 < Q; q2 += 2) {
          uint4 xv[NT];   // 16 bytes of x per batch row = the k-slots of two consecutive MMAs
#pragma unroll
          for (int nt = 0; nt < NT; ++nt)
            xv[nt] = *reinterpret_cast<const uint4*>(xb + nt * 8 * G::kRowStride + (j * Q + q2) * 8);
#pragma unroll
          for (int qq = 0; qq < 2; ++qq) {
            const int q = q2 + qq;
            uint32_t a0, a1, a2, a3;
            if constexpr (BITS == 2) {
              dg.pair(wa[j], q, a0, a2);
              dh.pair(wb[j], q, a1, a3);
            } else if constexpr (BITS == 4) {
              // nibbles 4q .. 4q+3 of the word: weights (4q, 4q+1 | 4q+2, 4q+3); offset = (nibble << 7) | lane * 4
              uint32_t lo[4], hi[4];
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const int sh = 4 * (4 * q + i) - 7;
                const uint32_t ua = sh < 0 ? (wa[j] << -sh) : (wa[j] >> sh);
                const uint32_t ub = sh < 0 ? (wb[j] << -sh) : (wb[j] >> sh);
                lo[i] = *reinterpret_cast<const uint32_t*>(tab_g + and_or(ua, 0x780u, lane4));
                hi[i] = *reinterpret_cast<const uint32_t*>(tab_g + 2048 + and_or(ub, 0x780u, lane4));
              }
              a0 = prmt(lo[0], lo[1], 0x7610u);
              a2 = prmt(lo[2], lo[3], 0x7610u);
              a1 = prmt(hi[0], hi[1], 0x7610u);
              a3 = prmt(hi[2], hi[3], 0x7610u);
            } else {
              const uint32_t m0 = kPow2[2 * q], m1 = kPow2[2 * q + 1];
              a0 = sg.select(wa[j] * m0);
              a2 = sg.select(wa[j] * m1);
              a1 = sh.select(wb[j] * m0);
              a3 = sh.select(wb[j] * m1);
            }
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
              mma_bf16_16816(acc[nt], a0, a1, a2, a3, qq ? xv[nt].z : xv[nt].x, qq ? xv[nt].w : xv[nt].y);
          }
        }
      }
    }
   }
  }

  // ---- K-groups 1.. hand their partial sums to K-group 0, which adds and stores ----
  asm volatile("griddepcontrol.launch_dependents;");
  __syncthreads();   // every warp is done with the x buffers; `red` aliases them
  if (group > 0) {
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
      *reinterpret_cast<float4*>(red + ((((group - 1) * TPC + wt) * NT + nt) * 32 + lane) * 4) =
          make_float4(acc[nt][0], acc[nt][1], acc[nt][2], acc[nt][3]);
  }
  __syncthreads();
  if (group == 0 && has_tile) {
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      float v[4] = {acc[nt][0], acc[nt][1], acc[nt][2], acc[nt][3]};
#pragma unroll
      for (int gq = 1; gq < kGroups; ++gq) {
        const float4 o =
            *reinterpret_cast<const float4*>(red + ((((gq - 1) * TPC + wt) * NT + nt) * 32 + lane) * 4);
        v[0] += o.x; v[1] += o.y; v[2] += o.z; v[3] += o.w;
      }
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int m = nt * 8 + 2 * t + (r & 1);
        const int64_t n = row0 + g + 8 * (r >> 1);
        if (m < M && n < N) y[(int64_t)m * N + n] = (uint16_t)float_to_bf16_bits(v[r]);
      }
    }
  }
}

template <int BITS, int NT, int TPC, int W = 8>
cudaError_t launch_nt(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N, int64_t K,
                      int M, cudaStream_t s) {
  constexpr int smem = MSmem<BITS, NT, TPC, W>::kTotal;
  static bool configured[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    cudaError_t e =
        cudaFuncSetAttribute(linear_multi_kernel<BITS, NT, TPC, W>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  const int64_t tiles = (N + kTileRows - 1) / kTileRows;
  const unsigned grid = (unsigned)((tiles + TPC - 1) / TPC);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(W * 32);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, linear_multi_kernel<BITS, NT, TPC, W>, packed, cb, x, y, N, K, M);
}

template <int BITS>
cudaError_t launch_bits(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
                        int64_t K, int M, cudaStream_t s) {
  // Tiles per CTA: 4 share the staged activations among more warps, 2 give twice as many CTAs.  Measured: 2 wins
  // when 4 would leave more than half of the SMs without a CTA, and for b = 2, 4 at up to 16 rows (two CTAs then fit an SM).
  const DeviceInfo* di = device_info();
  const int64_t tiles = (N + kTileRows - 1) / kTileRows;
  const bool few = (tiles + 3) / 4 <= (di ? di->sm_count : 148) / 2;
  const bool fits_one_wave = (tiles + 3) / 4 <= (di ? di->sm_count : 148);   // CTAs of 4 tiles <= SMs
  // few tiles and a long K: 2 tiles x 8 K-groups (16 warps) while each K-group still gets 4 steps or more
  // (4096 x 11008, b = 2, M = 16: 13.4 -> 12.3 us; 4096 x 4096: b = 4 11.5 -> 9.8 us, b = 2 (16 steps) 6.4 -> 6.9 us)
  const bool few16 = few && (tiles + 1) / 2 <= (di ? di->sm_count : 148) && (K * BITS / 128 + 3) / 4 >= 32;
  if (M <= 8) {
    // same shape of CTA for up to 8 batch rows (8192 x 28672, b = 1, M = 4: 35.0 -> 23.5 us; 8192 x 8192, b = 2,
    // M = 8: 12.7 -> 11.7 us)
    if (!few && fits_one_wave) return launch_nt<BITS, 1, 4, 16>(packed, cb, x, y, N, K, M, s);
    if constexpr (MSmem<BITS, 1, 2, 16>::kTotal <= kMaxSmem) {
      if (few16) return launch_nt<BITS, 1, 2, 16>(packed, cb, x, y, N, K, M, s);
    }
    if (few || BITS != 1) return launch_nt<BITS, 1, 2>(packed, cb, x, y, N, K, M, s);
    return launch_nt<BITS, 1, 4>(packed, cb, x, y, N, K, M, s);
  }
  if (M <= 16) {
    // 4 tiles x 4 K-groups (16 warps) when that grid gives every SM at most one CTA: 8192 x 8192, b = 2, M = 16:
    // 16.1 -> 14.4 us; 8192 x 28672, M = 16: b = 1 47.9 -> 40.1 us, b = 4 85.2 -> 76.6 us
    if (!few && fits_one_wave) return launch_nt<BITS, 2, 4, 16>(packed, cb, x, y, N, K, M, s);
    if constexpr (MSmem<BITS, 2, 2, 16>::kTotal <= kMaxSmem) {
      if (few16) return launch_nt<BITS, 2, 2, 16>(packed, cb, x, y, N, K, M, s);
    }
    if (few || BITS != 1) return launch_nt<BITS, 2, 2>(packed, cb, x, y, N, K, M, s);
    return launch_nt<BITS, 2, 4>(packed, cb, x, y, N, K, M, s);
  }
  if (M <= 32) {
    if constexpr (MSmem<BITS, 4, 2>::kTotal <= kMaxSmem) {
      if (few) return launch_nt<BITS, 4, 2>(packed, cb, x, y, N, K, M, s);
    }
    // when every SM gets at most one CTA anyway: 4 K-groups, i.e. 16 warps per CTA instead of 8 (8192 x 8192,
    // b = 2, M = 32: 22.6 -> 20.3 us; with more CTAs than SMs two 8-warp CTAs share an SM and that is faster)
    if constexpr (MSmem<BITS, 4, 4, 16>::kTotal <= kMaxSmem) {
      if (fits_one_wave) return launch_nt<BITS, 4, 4, 16>(packed, cb, x, y, N, K, M, s);
    }
    return launch_nt<BITS, 4, 4>(packed, cb, x, y, N, K, M, s);
  }
  if constexpr (BITS == 1) {
    return cudaErrorInvalidValue;   // unreachable: b = 1 is launched in passes of at most 32 rows
  } else {
    if constexpr (MSmem<BITS, 8, 2>::kTotal <= kMaxSmem) {
      if (few) return launch_nt<BITS, 8, 2>(packed, cb, x, y, N, K, M, s);
    }
    return launch_nt<BITS, 8, 4>(packed, cb, x, y, N, K, M, s);
  }
}

}  // namespace

// Batch rows per launch of the multi-tile kernel: 64, or 32 for b = 1 (its x buffers are twice as large).
int linear_multi_rows_per_launch(int bits) { return bits == 1 ? 32 : 64; }

// Smallest batch that goes to the multi-tile kernel.  The GEMV kernel stages the activations of a step once per
// warp and tile; at b = 1 a step spans 512 activations per batch row against 1 KB of packed words, so from 3 batch
// rows on sharing the staged activations among the tiles of a CTA wins (8192 x 28672: 33 -> 23 us at M = 3,
// 88 -> 25 us at M = 8), from 2 rows on when the GEMV grid would not fit the SMs in one wave of CTAs.  At b = 2, 4 it
// only wins on such shapes, from 5 and 4 rows on.
int linear_multi_min_rows(int bits, int64_t N) {
  const DeviceInfo* di = device_info();
  const int64_t tiles = (N + kTileRows - 1) / kTileRows;
  const bool waves = di && tiles > (int64_t)di->sm_count * 3;
  if (bits == 1) return waves ? 2 : 3;
  return waves ? (bits == 2 ? 5 : 4) : 9;
}

cudaError_t launch_linear_multi(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
                                int64_t K, int bits, int64_t M, cudaStream_t s) {
  const int64_t per = linear_multi_rows_per_launch(bits);
  for (int64_t m0 = 0; m0 < M; m0 += per) {
    const int mc = (int)(M - m0 < per ? M - m0 : per);
    const uint16_t* xp = x + m0 * K;
    uint16_t* yp = y + m0 * N;
    cudaError_t e;
    if (mc < linear_multi_min_rows(bits, N)) e = launch_linear_tiled(packed, cb, xp, yp, N, K, bits, mc, s);   // a short tail
    else if (bits == 1) e = launch_bits<1>(packed, cb, xp, yp, N, K, mc, s);
    else if (bits == 2) e = launch_bits<2>(packed, cb, xp, yp, N, K, mc, s);
    else e = launch_bits<4>(packed, cb, xp, yp, N, K, mc, s);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace kmq
