// kmq_linear on the tuned (tile-major) packed layout, small batches (M <= 8; larger ones, and from
// linear_multi_min_rows() batch rows on also smaller ones, go to the multi-tile kernel).
//
// One CTA owns one tile of 16 output rows; its 8 warps split K step by step (a step = 64 packed bytes of each
// row = 1 KB of the tile, stored contiguously).  Per step a warp
//   - has the step's 1 KB of packed indices in registers: two 512-byte coalesced 128-bit loads issued several
//     steps earlier (a ring of kStages steps per warp),
//   - copies the activations under the step into its own slice of shared memory (prefetched into registers
//     together with the weights), so that the B fragments are conflict-free 16-byte shared loads,
//   - rebuilds the bf16 weights in registers in the A-operand layout of mma.sync.m16n8k16 (weights are the 16-row
//     A operand, the batch is the 8-column B operand, fp32 accumulators) and issues the MMAs.
// The decode per bit width is the cheapest exact one for the half-rate integer pipe and the shared-memory port:
//   b = 4  per-row table of all 256 (centroid, centroid) pairs in shared memory, one copy per lane bank; the
//          byte offset of a lookup is one PRMT of the packed word, one 32-bit LDS yields two weights.
//   b = 2  the row's 4 centroids are the 8 source bytes of one PRMT; one PRMT yields two weights.
//   b = 1  a shift (as a multiply on the FMA pipe) puts two index bits on bits 15 and 31, a sign-replicating PRMT
//          spreads them over their half words and one LOP3 selects c0 or c1: bit copies of the stored centroids.
#include "kmq_common.cuh"
#include "kmq_linear_variants.cuh"
#include "kmq_mma_common.cuh"

namespace kmq {
namespace {

constexpr int kWarps = 8;
constexpr int kMinCtasPerSm = 3;   // register budget of the launch bounds
constexpr int kThreads = kWarps * 32;
constexpr int kRows = kTileRows;
constexpr int kPairEntryStride = 256;   // b = 4 tables: entry e, half h, lane l at e * 256 + h * 128 + l * 4
constexpr int kTableBytes4 = 256 * kPairEntryStride;

template <int BITS>
struct TGeo {
  static constexpr int kMmaPerWord = 8 / BITS;            // 16 k-slots per MMA = 4 lanes x 4 weights
  static constexpr int kStepK = 512 / BITS;               // weights of one row per step
  static constexpr int kWordK = 32 / BITS;
  static constexpr int kChunkXBytes = 4 * kWordK * 2;     // activations under one 16-byte chunk of a row
  static constexpr int kChunkStride = kChunkXBytes + 16;  // staged with 16 bytes of padding: no bank conflicts
  static constexpr int kRowStride = 4 * kChunkStride;     // one batch row of one step
  static constexpr int kPiecesPerRow = kStepK / 8;        // 16-byte pieces of x per batch row and step
  static constexpr int kTableBytes = BITS == 4 ? kTableBytes4 : 0;
  static constexpr int kStages = 2;                       // steps in flight per warp (deeper rings measured slower)
};

template <int BITS, int MMAX>
struct TSmem {
  using G = TGeo<BITS>;
  static constexpr int kXs = kWarps * MMAX * G::kRowStride;
  static constexpr int kRed = kWarps * 32 * 16;
  static constexpr int kTotal = G::kTableBytes + kXs + kRed;
};

// shared-memory byte offset (within one batch row of a warp's slice) of 16-byte piece `w` of a step
template <int BITS>
__device__ __forceinline__ int piece_offset(int w) {
  using G = TGeo<BITS>;
  constexpr int kPiecesPerChunk = G::kChunkXBytes / 16;
  return (w / kPiecesPerChunk) * G::kChunkStride + (w % kPiecesPerChunk) * 16;
}

// Steps [sa, sb) of tile `tile_id`, all 8 warps of the CTA: on return thread i < 128 holds in `v` the sum over those
// steps for output row i % 16 and batch row i / 16.  May be called several times by one CTA; shared memory is reused
// from call to call.
template <int BITS, int MMAX>
__device__ __forceinline__ void tile_segment(const uint32_t* __restrict__ packed, const uint16_t* __restrict__ cb,
                                             const uint16_t* __restrict__ x, int64_t N, int64_t K, int M,
                                             int64_t tile_id, int sa, int sb, bool wait_for_x, bool early_trigger,
                                             float& v) {
  using G = TGeo<BITS>;
  using SM = TSmem<BITS, MMAX>;
  constexpr int Q = G::kMmaPerWord;
  constexpr int STAGES = G::kStages;
  // 16-byte pieces of x per lane and step, and whether they ride in the register ring with the weights
  constexpr int kPieces = MMAX * G::kPiecesPerRow;
  constexpr int NP = (kPieces + 31) / 32;
  constexpr bool kPrefetchX = NP <= 2;

  extern __shared__ __align__(128) unsigned char smem_raw[];
  unsigned char* const tables = smem_raw;
  unsigned char* const xs_warp = smem_raw + G::kTableBytes + (threadIdx.x >> 5) * (MMAX * G::kRowStride);
  float* const red = reinterpret_cast<float*>(smem_raw + G::kTableBytes + SM::kXs);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int64_t row0 = tile_id * kRows;
  const int chunks = (int)(K / (4 * G::kWordK));   // 16-byte chunks per row
  const int steps = (chunks + 3) >> 2;             // the layout pads every row to whole steps
  // step s of this tile: 64 16-byte units, unit h * 32 + lane = row (g + 8h), chunk t
  const uint4* __restrict__ tile = reinterpret_cast<const uint4*>(packed) + tile_id * steps * 64 + lane;
  __syncthreads();   // a previous segment's readers of the tables and of `red` are done

  // ---- x pieces of this lane: piece p = lane + 32 i -> batch row p / kPiecesPerRow, piece p % kPiecesPerRow
  int px_k[NP], px_sm[NP];
  const uint16_t* px_src[NP];
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    const int p = lane + 32 * i;
    const int m = p / G::kPiecesPerRow, w = p % G::kPiecesPerRow;
    px_k[i] = (p < kPieces && m < M) ? w * 8 : -1;   // k offset inside the step, or -1: nothing to copy
    px_sm[i] = m * G::kRowStride + piece_offset<BITS>(w);
    px_src[i] = x + (int64_t)m * K + w * 8;
  }
  auto load_x = [&](int s, uint4 (&v)[NP]) {
#pragma unroll
    for (int i = 0; i < NP; ++i) {
      v[i] = make_uint4(0, 0, 0, 0);
      if (px_k[i] >= 0 && (int64_t)s * G::kStepK + px_k[i] < K)
        v[i] = __ldg(reinterpret_cast<const uint4*>(px_src[i] + (int64_t)s * G::kStepK));
    }
  };

  // ---- ring: weights (and x pieces) of this warp's next kStages steps ----
  constexpr int XS = kPrefetchX ? STAGES : 1;   // without prefetch one buffer, filled just before use
  uint4 qa[STAGES], qb[STAGES], qx[XS][NP];
#pragma unroll
  for (int d = 0; d < STAGES; ++d) {
    const int s = sa + warp + d * kWarps;
    qa[d] = qb[d] = make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int i = 0; i < NP; ++i) qx[kPrefetchX ? d : 0][i] = make_uint4(0, 0, 0, 0);
    if (s < sb) {
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
    // entry e of row r: (C_r[e & 15], C_r[e >> 4]); the 4 lanes that share a row get one bank each.
    // A thread owns one row and one low index: it fetches the row's 16 centroids once (32 bytes) and writes the
    // 16 entries e = low + 16 * high with no further loads.
    const int r8 = threadIdx.x & 7, half = (threadIdx.x >> 3) & 1, low = (threadIdx.x >> 4) & 15;
    constexpr int kParts = kThreads / 256;   // threads beyond the first 256 take a share of the high indices
    const int part = threadIdx.x >> 8;
    const uint16_t* crow = cb + min(row0 + r8 + 8 * half, N - 1) * 16;
    const uint4 ca = __ldg(reinterpret_cast<const uint4*>(crow)), cc = __ldg(reinterpret_cast<const uint4*>(crow) + 1);
    const uint32_t lo = __ldg(crow + low);
    const uint32_t c2[8] = {ca.x, ca.y, ca.z, ca.w, cc.x, cc.y, cc.z, cc.w};
    unsigned char* dst = tables + low * kPairEntryStride + half * 128 + r8 * 16;
#pragma unroll
    for (int hi = 0; hi < 16; ++hi) {
      if (kParts > 1 && (hi % kParts) != part) continue;
      const uint32_t v = prmt(lo, c2[hi >> 1], (hi & 1) ? 0x7610u : 0x5410u);   // (C[low], C[hi])
      *reinterpret_cast<uint4*>(dst + hi * 16 * kPairEntryStride) = make_uint4(v, v, v, v);
    }
    __syncthreads();
  }
  const uint32_t lane4 = lane * 4;

  // Programmatic dependent launch: up to here only the packed indices and the codebooks were read, which are
  // constants of the layer; the activations may come from the previous kernel on the stream, so they are read
  // only once that kernel is known to have completed.  A CTA that became resident early has its first weights
  // under way (and, for b = 4, its tables built) by then.
  if (wait_for_x) {
    // a hint only (it binds no value): the first few CTAs pull the activations towards L2 while waiting
    if (blockIdx.x < 4) {
      for (int64_t o = ((int64_t)blockIdx.x * kThreads + threadIdx.x) * 64; o < (int64_t)M * K; o += 4 * kThreads * 64)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(x + o));
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // Where it pays (see early_trigger()), the next kernel on the stream may become resident from here on: its CTAs
    // read their packed words and build their tables in the SM slots this grid leaves free, while this one computes.
    if (early_trigger) asm volatile("griddepcontrol.launch_dependents;");
  }
  if constexpr (kPrefetchX) {
#pragma unroll
    for (int d = 0; d < STAGES; ++d) {
      const int s = sa + warp + d * kWarps;
      if (s < sb) load_x(s, qx[d]);
    }
  }

  float acc[4] = {0.f, 0.f, 0.f, 0.f};

  // B fragments: lane (g, t) supplies batch row g; the columns of an MMA are independent, so lanes with
  // g >= M re-read the last real row and their columns are never stored.
  const unsigned char* const xb = xs_warp + min(g, M - 1) * G::kRowStride + t * G::kChunkStride;

  for (int s0 = sa + warp; s0 < sb; s0 += STAGES * kWarps) {
#pragma unroll
    for (int d = 0; d < STAGES; ++d) {
      const int s = s0 + d * kWarps;
      if (s < sb) {   // warp-uniform
        // stage the activations under this step (zeros past K)
        if constexpr (!kPrefetchX) load_x(s, qx[0]);
        __syncwarp();
#pragma unroll
        for (int i = 0; i < NP; ++i)
          if (px_k[i] >= 0) *reinterpret_cast<uint4*>(xs_warp + px_sm[i]) = qx[kPrefetchX ? d : 0][i];
        __syncwarp();

        const uint32_t wa[4] = {qa[d].x, qa[d].y, qa[d].z, qa[d].w};
        const uint32_t wb[4] = {qb[d].x, qb[d].y, qb[d].z, qb[d].w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
#pragma unroll
          for (int q2 = 0; q2 < Q; q2 += 2) {
            // 16 bytes of x = the 8 weights of two consecutive MMAs
            // b = 4 is bound by the shared-memory pipe: there only the lanes of real batch rows read (a 128-bit
            // load takes one pass per quarter warp that has an active lane); elsewhere the predicate costs more
            uint4 xv = make_uint4(0, 0, 0, 0);
            if (BITS != 4 || g < M) xv = *reinterpret_cast<const uint4*>(xb + (j * Q + q2) * 8);
#pragma unroll
            for (int qq = 0; qq < 2; ++qq) {
              const int q = q2 + qq;
              uint32_t a0, a1, a2, a3;
              if constexpr (BITS == 2) {
                dg.pair(wa[j], q, a0, a2);
                dh.pair(wb[j], q, a1, a3);
              } else if constexpr (BITS == 4) {
                // index byte k of the word -> byte offset (byte << 8) | lane * 4: result bytes (lane4, byte k, 0, 0)
                const uint32_t s0b = 0x5504u | ((2 * q) << 4), s1b = 0x5504u | ((2 * q + 1) << 4);
                a0 = *reinterpret_cast<const uint32_t*>(tables + prmt(wa[j], lane4, s0b));
                a2 = *reinterpret_cast<const uint32_t*>(tables + prmt(wa[j], lane4, s1b));
                a1 = *reinterpret_cast<const uint32_t*>(tables + 128 + prmt(wb[j], lane4, s0b));
                a3 = *reinterpret_cast<const uint32_t*>(tables + 128 + prmt(wb[j], lane4, s1b));
              } else {
                // shift by c puts weights (2c, 2c+1) of the word on the two sign bits; c = 2q and 2q + 1
                const uint32_t m0 = kPow2[2 * q], m1 = kPow2[2 * q + 1];
                a0 = sg.select(wa[j] * m0);
                a2 = sg.select(wa[j] * m1);
                a1 = sh.select(wb[j] * m0);
                a3 = sh.select(wb[j] * m1);
              }
              mma_bf16_16816(acc, a0, a1, a2, a3, qq ? xv.z : xv.x, qq ? xv.w : xv.y);
            }
          }
        }
        // refill this stage for the step kStages rounds ahead
        const int s2 = s + STAGES * kWarps;
        if (s2 < sb) {
          qa[d] = ldg_stream_u4(tile + (int64_t)s2 * 64);
          qb[d] = ldg_stream_u4(tile + (int64_t)s2 * 64 + 32);
          if constexpr (kPrefetchX) load_x(s2, qx[kPrefetchX ? d : 0]);
        }
      }
    }
  }

  // ---- add the partial sums of the warps ----
  *reinterpret_cast<float4*>(red + (warp * 32 + lane) * 4) = make_float4(acc[0], acc[1], acc[2], acc[3]);
  __syncthreads();
  v = 0.f;
  if (threadIdx.x < kRows * 8) {
    const int r = threadIdx.x & 15, m = threadIdx.x >> 4;   // consecutive threads -> consecutive output rows
    const int src_lane = (r & 7) * 4 + (m >> 1), src_reg = (r >> 3) * 2 + (m & 1);
#pragma unroll
    for (int w = 0; w < kWarps; ++w) v += red[(w * 32 + src_lane) * 4 + src_reg];
  }
}

// Thread i < 128: store the finished sum of output row row0 + i % 16, batch row i / 16, as bf16.
__device__ __forceinline__ void store_output(float v, uint16_t* __restrict__ y, int64_t N, int M, int64_t row0) {
  if (threadIdx.x < kRows * 8) {
    const int r = threadIdx.x & 15, m = threadIdx.x >> 4;
    const int64_t n = row0 + r;
    if (m < M && n < N) y[(int64_t)m * N + n] = (uint16_t)float_to_bf16_bits(v);
  }
}

// One CTA per tile.
template <int BITS, int MMAX>
__global__ void __launch_bounds__(kThreads, kMinCtasPerSm) linear_tiled_kernel(const uint32_t* __restrict__ packed,
                                                                    const uint16_t* __restrict__ cb,
                                                                    const uint16_t* __restrict__ x,
                                                                    uint16_t* __restrict__ y, int64_t N, int64_t K,
                                                                    int M, int early) {
  const int steps = (int)((K / (4 * TGeo<BITS>::kWordK) + 3) >> 2);
  const int64_t row0 = (int64_t)blockIdx.x * kRows;
  float v;
  tile_segment<BITS, MMAX>(packed, cb, x, N, K, M, blockIdx.x, 0, steps, true, early != 0, v);
  // Programmatic dependent launch: from here on at the latest the next kernel on the stream may become resident; it
  // reads nothing but constants of its layer until this kernel has completed (see tile_segment), so its first
  // weights are under way while this one stores and drains.
  asm volatile("griddepcontrol.launch_dependents;");
  store_output(v, y, N, M, row0);
}

// ---------------------------------------------------------------------------
// Balanced variant for more tiles than resident CTA slots.  The tiles * steps step-units, in tile-major order, are
// cut into gridDim.x equal contiguous ranges, one per CTA (all CTAs resident at once, so no second wave).  A range
// is longer than a tile, so a CTA finishes the tiles that lie wholly inside its range and owns at most two partial
// tiles, one at each end; their sums go to scratch slot [cta][0] (range starts inside the tile) or [cta][1] (range
// ends inside it).  Every cut therefore has exactly two contributors, which the fix-up kernel adds in a fixed order.
// ---------------------------------------------------------------------------
constexpr int kSlotFloats = kRows * 8 + 8;   // 128 sums (+ 8 unused: keeps the slots 32-byte aligned)

template <int BITS, int MMAX>
__global__ void __launch_bounds__(kThreads, kMinCtasPerSm) linear_split_kernel(const uint32_t* __restrict__ packed,
                                                                    const uint16_t* __restrict__ cb,
                                                                    const uint16_t* __restrict__ x,
                                                                    uint16_t* __restrict__ y, int64_t N, int64_t K,
                                                                    int M, float* __restrict__ scratch) {
  const int64_t steps = (K / (4 * TGeo<BITS>::kWordK) + 3) >> 2;
  const int64_t units = ((N + kRows - 1) / kRows) * steps;
  const int64_t u0 = units * blockIdx.x / gridDim.x, u1 = units * (blockIdx.x + 1) / gridDim.x;
  bool first = true;   // the first segment waits for the previous kernel on the stream before it reads x
  for (int64_t tile = u0 / steps; tile * steps < u1; ++tile) {
    const int64_t base = tile * steps;
    const int sa = (int)(u0 > base ? u0 - base : 0), sb = (int)(u1 - base < steps ? u1 - base : steps);
    float v;
    tile_segment<BITS, MMAX>(packed, cb, x, N, K, M, tile, sa, sb, first, false, v);
    first = false;
    if (sa == 0 && sb == steps) {
      store_output(v, y, N, M, tile * kRows);
    } else if (threadIdx.x < kRows * 8) {
      float* slot = scratch + ((int64_t)blockIdx.x * 2 + (sa == 0 ? 1 : 0)) * kSlotFloats;
      slot[threadIdx.x] = v;
    }
  }
  asm volatile("griddepcontrol.launch_dependents;");
}

// Block c adds the two halves of the tile that the cut between CTA c and CTA c + 1 falls into.
template <int BITS>
__global__ void __launch_bounds__(kRows * 8) linear_split_fixup_kernel(const float* __restrict__ scratch,
                                                                       const uint16_t* __restrict__ cb,
                                                                       uint16_t* __restrict__ y, int64_t N, int64_t K,
                                                                       int M, int ctas) {
  const int64_t steps = (K / (4 * TGeo<BITS>::kWordK) + 3) >> 2;
  const int64_t units = ((N + kRows - 1) / kRows) * steps;
  const int64_t cut = units * (blockIdx.x + 1) / ctas;
  if (cut % steps == 0) return;   // the cut is a tile boundary: nothing was left partial
  asm volatile("griddepcontrol.wait;" ::: "memory");   // the slots are the previous kernel's output
  asm volatile("griddepcontrol.launch_dependents;");
  const int64_t row0 = (cut / steps) * kRows;
  const float* end_of_c = scratch + ((int64_t)blockIdx.x * 2 + 1) * kSlotFloats;
  const float* start_of_next = scratch + ((int64_t)(blockIdx.x + 1) * 2) * kSlotFloats;
  const float v = end_of_c[threadIdx.x] + start_of_next[threadIdx.x];
  store_output(v, y, N, M, row0);
}

// Whether the CTAs of linear_tiled_kernel release the next kernel on the stream right after their own wait instead of
// just before their store.  The next call's CTAs then take the SM slots this grid leaves free and do their set-up
// (packed words, b = 4 tables) under this grid's MMAs, at the price of competing with them.  Measured on B200 at
// batch 1 over N = 2048 .. 16384, K = 2048 .. 11264 (us per call, late / early release):
//   b = 2: faster nearly everywhere (4096 x 4096 3.64 / 3.25, 3072 x 3072 2.94 / 2.68, 8192 x 8192 10.4 / 9.9) except
//          with between two and three CTAs per SM (5120 x 4096 4.68 / 4.99, 6144 x 4096 4.83 / 5.08);
//   b = 4: faster (5120 x 4096 6.61 / 5.46, 3072 x 3072 4.03 / 3.46, 8192 x 8192 16.1 / 15.4) except when the grid
//          nearly fills two CTA slots of every SM and tiles are long (4096 x 4096 4.92 / 5.13, 4096 x 8192 8.06 / 8.92);
//   b = 1: no gain or a loss (4096 x 4096 3.14 / 3.90) except on long tiles away from that window (3072 x 8192
//          5.15 / 4.83, 8192 x 8192 9.09 / 8.48).
bool early_trigger(int bits, int64_t tiles, int64_t steps, int sm_count) {
  const int64_t two = 2 * (int64_t)sm_count, three = 3 * (int64_t)sm_count;
  const bool nearly_two = 5 * tiles > 4 * two && tiles <= two;   // more than 0.8 of two CTAs per SM, at most two
  if (bits == 2) return !(tiles > two && tiles < three);
  if (bits == 4) return !(nearly_two && steps >= 32);
  return steps >= 16 && !(10 * tiles > 7 * two && tiles <= two);
}

template <int BITS, int MMAX>
cudaError_t launch_one(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
                       int64_t K, int M, cudaStream_t s) {
  constexpr int smem = TSmem<BITS, MMAX>::kTotal;
  static bool configured[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    cudaError_t e =
        cudaFuncSetAttribute(linear_tiled_kernel<BITS, MMAX>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((N + kRows - 1) / kRows));
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const DeviceInfo* di = device_info();
  const int64_t steps = (K / (4 * TGeo<BITS>::kWordK) + 3) >> 2;
  const int early = di && early_trigger(BITS, (N + kRows - 1) / kRows, steps, di->sm_count) ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, linear_tiled_kernel<BITS, MMAX>, packed, cb, x, y, N, K, M, early);
}

template <int BITS>
cudaError_t launch_bits(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
                        int64_t K, int M, cudaStream_t s) {
  if (M == 1) return launch_one<BITS, 1>(packed, cb, x, y, N, K, M, s);
  if (M == 2) return launch_one<BITS, 2>(packed, cb, x, y, N, K, M, s);
  if (M <= 4) return launch_one<BITS, 4>(packed, cb, x, y, N, K, M, s);
  if constexpr (BITS == 1) {
    return cudaErrorInvalidValue;   // unreachable: b = 1 goes to the multi-tile kernel from 4 batch rows on
  } else {
    return launch_one<BITS, 8>(packed, cb, x, y, N, K, M, s);
  }
}

template <int BITS, int MMAX>
cudaError_t launch_split_one(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
                             int64_t K, int M, float* scratch, int ctas, cudaStream_t s) {
  constexpr int smem = TSmem<BITS, MMAX>::kTotal;
  static bool configured[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    cudaError_t e =
        cudaFuncSetAttribute(linear_split_kernel<BITS, MMAX>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)ctas);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, linear_split_kernel<BITS, MMAX>, packed, cb, x, y, N, K, M, scratch);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t fix = {};
  fix.gridDim = dim3((unsigned)(ctas - 1));
  fix.blockDim = dim3(kRows * 8);
  fix.stream = s;
  fix.attrs = attr;
  fix.numAttrs = 1;
  return cudaLaunchKernelEx(&fix, linear_split_fixup_kernel<BITS>, (const float*)scratch, cb, y, N, K, M, ctas);
}

template <int BITS>
cudaError_t launch_split_bits(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
                              int64_t K, int M, float* scratch, int ctas, cudaStream_t s) {
  if (M == 1) return launch_split_one<BITS, 1>(packed, cb, x, y, N, K, M, scratch, ctas, s);
  if (M == 2) return launch_split_one<BITS, 2>(packed, cb, x, y, N, K, M, scratch, ctas, s);
  if (M <= 4) return launch_split_one<BITS, 4>(packed, cb, x, y, N, K, M, scratch, ctas, s);
  return cudaErrorInvalidValue;   // unreachable: with more tiles than CTA slots, 5 rows and more go to the multi-tile kernel
}

}  // namespace

// Tuned layout.  Batches larger than 8 are processed 8 rows at a time (one launch each).
cudaError_t launch_linear_tiled(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
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

namespace kmq {

// CTAs of the balanced variant (0 = use one CTA per tile): all resident slots when there are more tiles than slots.
// Every range restarts the load pipeline and the decode set-up once or twice more than a whole tile would, so this
// only pays when a tile is long: at least kSplitMinSteps steps (measured: 8192 x 28672, b = 4, 224 steps, 55 -> 44 us;
// with 16..56 steps per tile the per-tile grid is faster).
constexpr int64_t kSplitMinSteps = 128;

namespace {

// CTAs of linear_split_kernel<BITS, MMAX> that fit one SM (registers and shared memory), asked from the runtime
// once per device and instantiation.
template <int BITS, int MMAX>
int split_ctas_per_sm() {
  static int cached[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  if (cached[dev] == 0) {
    constexpr int smem = TSmem<BITS, MMAX>::kTotal;
    int n = 0;
    if (cudaFuncSetAttribute(linear_split_kernel<BITS, MMAX>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) !=
            cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, linear_split_kernel<BITS, MMAX>, kThreads, smem) !=
            cudaSuccess)
      return 0;
    cached[dev] = n > 0 ? n : -1;
  }
  return cached[dev] > 0 ? cached[dev] : 0;
}

template <int BITS>
int split_ctas_per_sm_bits(int64_t M) {
  return M == 1 ? split_ctas_per_sm<BITS, 1>() : M == 2 ? split_ctas_per_sm<BITS, 2>() : split_ctas_per_sm<BITS, 4>();
}

}  // namespace

int linear_split_ctas(int64_t N, int64_t K, int bits, int64_t M) {
  const DeviceInfo* di = device_info();
  if (!di || M > 4 || M >= linear_multi_min_rows(bits, N)) return 0;
  // one CTA per resident slot of the instantiation that will run, so that there is no second wave
  const int per_sm = bits == 1 ? split_ctas_per_sm_bits<1>(M) : bits == 2 ? split_ctas_per_sm_bits<2>(M)
                                                                            : split_ctas_per_sm_bits<4>(M);
  if (per_sm <= 0) return 0;
  const int64_t slots = (int64_t)di->sm_count * per_sm;
  const int64_t tiles = (N + kRows - 1) / kRows;
  const int64_t steps = (K * bits / 128 + 3) / 4;
  return (tiles > slots && steps >= kSplitMinSteps) ? (int)slots : 0;
}

size_t linear_split_scratch_bytes(int ctas) { return (size_t)ctas * 2 * kSlotFloats * sizeof(float); }

cudaError_t launch_linear_split(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
                                int64_t K, int bits, int64_t M, void* scratch, int ctas, cudaStream_t s) {
  float* sc = static_cast<float*>(scratch);
  if (bits == 1) return launch_split_bits<1>(packed, cb, x, y, N, K, (int)M, sc, ctas, s);
  if (bits == 2) return launch_split_bits<2>(packed, cb, x, y, N, K, (int)M, sc, ctas, s);
  return launch_split_bits<4>(packed, cb, x, y, N, K, (int)M, sc, ctas, s);
}

}  // namespace kmq
