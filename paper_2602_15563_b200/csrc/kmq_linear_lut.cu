// kmq_linear on KMQ_LAYOUT_TABLE for b = 1, 2 and small batches: the activation-table kernel.
//
// With a per-row codebook the weight side has nothing to share between rows, but the activation side has: for a
// group of 8 consecutive inputs every row needs the sum of the activations selected by 8 index bits, and there are
// only 256 such sums.  A CTA therefore builds, for its slice of K, the table  T_g[e] = sum_t bit_t(e) * x[8g + t]
// (fp32) of every group g in shared memory once and then streams the packed bit planes of many rows through it:
// one shared-memory lookup and one fp32 add per 8 weights and bit-plane class, no multiply, no per-weight integer
// work.  The layer is evaluated as
//     y[n] = c_s * S + sum_{j != s} (c_j - c_s) * A_j[n],     A_j[n] = sum_{k : idx[n,k] = j} x[k],   S = sum_k x[k]
// with s the centroid of smallest magnitude of row n.  This is the definition regrouped by index value; leaving out
// the class of the smallest centroid (instead of always class 0) keeps the rounding error of every term relative to
// |c_j| * sum_{idx = j} |x|, i.e. inside the stated tolerance for any finite codebook, not just balanced ones.
//   b = 1: one class (the centroid of larger magnitude): one lookup per byte of the bit plane, XORed with the
//          row's mask when that centroid is index 0.
//   b = 2: three classes, selected from the two bit planes by three LOP3 per 32 weights.
//
// Shared-memory table: entry e of group column c of table slot q at byte  65536 + (q >> 1) * 65536 + e * 256 +
// (q & 1) * 128 + c * 4  (absolute shared address): the entry index is byte 1 of the address, so one PRMT turns a
// byte of packed bits into the address, and slot and parity are an immediate offset.  32 columns x 4 bytes = all 32
// banks, and the layout's row rotation (kmq_table_layout.cuh) makes the 32 lanes of a warp use 32 different columns in
// every lookup: no bank conflicts by construction.  A slot holds one chunk (256 weights); up to 4 slots = 128 KB.
//
// Work split: CTA (s, rb) owns K slice s (NL chunks) and row block rb; warp w owns the 16-row tiles rb0 + w,
// rb0 + w + W, ...  The packed bits of a tile reach the warp through its own ring of shared-memory stages filled by
// bulk asynchronous copies (cp.async.bulk, completion on an mbarrier per stage): no registers and no scoreboard
// slots are tied up by loads in flight, so up to 32 warps of 64 registers run per SM.  A lane owns one row of the
// tile and every second group, keeps its running sums in registers over the NL chunks and adds the two lanes of a row
// with one shuffle.  With a single slice the warp applies the codebook and stores its rows directly.  With 2, 4 or 8
// slices that fit the machine as thread-block clusters, the slices of a row block are one cluster: the sums stay in
// each CTA's shared memory and, after a cluster barrier, CTA s adds its share of the rows over all slices out of the
// other CTAs' shared memory (fixed order), applies the codebook and stores.  Otherwise the per-slice sums go to
// scratch [slice][class][row] and a second kernel adds the slices in a fixed order, applies the codebook and stores.
//
// Programmatic dependent launch: the CTA may start while the previous kernel on the stream is still running.  Until
// griddepcontrol.wait returns it only sets up its barriers, starts the first copies of packed indices (constants of
// the layer) and hints x towards L2; x, y and the scratch are touched only afterwards.
#include <mutex>

#include "kmq_common.cuh"
#include "kmq_linear_variants.cuh"
#include "kmq_lut_common.cuh"
#include "kmq_table_layout.cuh"

namespace kmq {
namespace {

// Geometry of one instantiation: NL chunks per K slice.
//   piece  = what one bulk copy brings: all planes of PC consecutive chunks of one tile (contiguous in the layout)
//   stages = pieces in flight per warp; the first kStagesHigh of a warp sit above the tables, the rest below them
template <int BITS, int NL>
struct LutGeo {
  static constexpr int kClasses = BITS == 1 ? 1 : 3;
  static constexpr int kPieceChunks = (BITS == 1 && NL % 2 == 0) ? 2 : 1;
  static constexpr int kPieces = NL / kPieceChunks;                      // pieces per tile
  static constexpr int kPieceBytes = kPieceChunks * BITS * kTableUnitBytes;   // 512 or 1024
  static constexpr uint32_t kTableEnd = kLutTableBase + (uint32_t)((NL + 1) / 2) * 65536u;
  static constexpr int kWarps = NL <= 2 ? 32 : NL == 3 ? 24 : 20;
  static constexpr int kStagesHigh = NL <= 2 ? 3 : 1;
  static constexpr int kStagesLow = NL <= 2 ? 1 : NL == 3 ? 2 : 3;
  static constexpr int kStages = kStagesHigh + kStagesLow;               // a multiple of kPieces
  static constexpr int kTasksPerRound = kStages / kPieces;               // tiles whose pieces fill the ring once
  static constexpr uint32_t kSumBase = 1152;                             // 16 floats: sum of x per chunk
  static constexpr uint32_t kBarBase = 1216;                             // mbarriers: 8 bytes per warp and stage
  static constexpr uint32_t kLowBase = 2304;                             // low stages: [kLowBase, kLutTableBase)
  static constexpr uint32_t kHighEnd = kTableEnd + (uint32_t)(kWarps * kStagesHigh * kPieceBytes);
  // cluster variant: the CTA's partial sums [class][row of the block] sit between the low stages and the tables
  static constexpr uint32_t kPartBase = kLowBase + (uint32_t)(kWarps * kStagesLow * kPieceBytes);
  static constexpr int kPartFloats = (int)(kLutTableBase - kPartBase) / 4;
  static constexpr uint32_t kSxWord = kSumBase + 40;                     // a free word of the sum area: sum of x
  static_assert(kBarBase + kWarps * kStages * 8 <= kLowBase, "mbarriers must fit below the low stages");
  static_assert(kLowBase + kWarps * kStagesLow * kPieceBytes <= kLutTableBase, "low stages overlap the tables");
  static_assert(kHighEnd <= 227 * 1024 + 1024, "stages exceed the shared memory of an SM");
  static_assert(NL >= 1 && NL <= 4 && (BITS == 1 || NL <= 3), "unsupported slice length");
  static_assert(kStages % kPieces == 0, "the ring must hold whole tiles");
};

// ---- thread-block cluster: barrier and loads from another CTA's shared memory ----
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// `saddr`: an address in this CTA's shared-memory window; the value at the same place of the CTA of rank `rank`.
__device__ __forceinline__ float ld_cluster_f32(uint32_t saddr, uint32_t rank) {
  uint32_t ra;
  float v;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(saddr), "r"(rank));
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(ra) : "memory");
  return v;
}

// Index of the centroid of smallest magnitude (lowest index on ties); `c` = the row's codebook as bf16 pairs.
template <int BITS>
__device__ __forceinline__ int smallest_centroid(const uint32_t (&c)[2]) {
  const uint32_t m0 = c[0] & 0x7FFFu, m1 = (c[0] >> 16) & 0x7FFFu;
  if constexpr (BITS == 1) {
    return m1 < m0 ? 1 : 0;
  } else {
    const uint32_t m2 = c[1] & 0x7FFFu, m3 = (c[1] >> 16) & 0x7FFFu;
    int s = 0;
    uint32_t best = m0;
    if (m1 < best) { best = m1; s = 1; }
    if (m2 < best) { best = m2; s = 2; }
    if (m3 < best) { best = m3; s = 3; }
    return s;
  }
}

template <int BITS>
__device__ __forceinline__ void load_row_codebook(const uint16_t* __restrict__ cb, int64_t n, uint32_t (&c)[2]) {
  if constexpr (BITS == 1) {
    c[0] = __ldg(reinterpret_cast<const uint32_t*>(cb + n * 2));
    c[1] = 0;
  } else {
    const uint2 v = __ldg(reinterpret_cast<const uint2*>(cb + n * 4));
    c[0] = v.x;
    c[1] = v.y;
  }
}

// Scratch: partial[slice][class][rows_pad] fp32, then sx[slice] (sum of the activations of the slice).
__host__ __device__ inline size_t lut_scratch_floats(int slices, int classes, int64_t rows_pad) {
  return (size_t)slices * classes * rows_pad + slices;
}


template <int BITS, int NL>
__global__ void __launch_bounds__(LutGeo<BITS, NL>::kWarps * 32, 1)
    linear_lut_kernel(const unsigned char* __restrict__ packed, const uint16_t* __restrict__ cb,
                      const uint16_t* __restrict__ x, uint16_t* __restrict__ y, float* __restrict__ scratch, int64_t N,
                      int64_t K, int slices, int row_blocks, unsigned int* __restrict__ err, int in_cluster) {
  using G = LutGeo<BITS, NL>;
  constexpr int CL = G::kClasses, S = G::kStages, P = G::kPieces, PC = G::kPieceChunks, TPR = G::kTasksPerRound;
  extern __shared__ __align__(128) unsigned char smem_raw[];

  // ================= before the previous kernel on the stream is known to have finished =================
  // Only the packed indices and codebooks (constants of the layer) and this CTA's own shared memory are touched here.
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  const int slice = blockIdx.x % slices, rb = blockIdx.x / slices;
  const int chunks = (int)table_chunks(K);
  const int tiles = (int)table_tiles(N);
  const int64_t rows_pad = (int64_t)tiles * 16;
  const int chunk0 = slice * NL;
  const int t0 = (int)((int64_t)tiles * rb / row_blocks), t1 = (int)((int64_t)tiles * (rb + 1) / row_blocks);
  const int rows_blk = (t1 - t0) * 16;   // rows of this row block, padding included

  // Tables, stages and barriers sit at absolute shared-memory addresses: the dynamic shared memory of this CTA must
  // cover [kSumBase, kHighEnd).
  // In a cluster launch the shared-memory window of the CTA of rank r starts at r << 24 of the shared address space
  // (0 without a cluster); every absolute address below carries this base.  It leaves bits 8..15 alone, which the
  // lookups overwrite with the table entry.
  const uint32_t wb = smem_addr(smem_raw) & 0xFF000000u;
  {
    const uint32_t s0 = smem_addr(smem_raw) - wb;
    uint32_t dyn;
    asm("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn));
    if (s0 > G::kSumBase || s0 + dyn < G::kHighEnd) {   // the same in every CTA of the grid: all of them leave here
      asm volatile("griddepcontrol.wait;" ::: "memory");
      if (threadIdx.x == 0) atomicOr(err, kErrWindow);
      return;
    }
  }

  // ---- this warp's ring: stage st < kStagesHigh above the tables, the others below.  Stage tt * P + pc holds
  //      piece pc of the warp's tile number ti with ti % TPR = tt; round number ti / TPR gives the mbarrier phase ----
  const uint32_t bar0 = wb + G::kBarBase + (uint32_t)(warp * S) * 8u;
  const uint32_t high0 = wb + G::kTableEnd + (uint32_t)(warp * G::kStagesHigh * G::kPieceBytes);
  const uint32_t low0 = wb + G::kLowBase + (uint32_t)(warp * G::kStagesLow * G::kPieceBytes);
  auto stage_addr = [&](int st) -> uint32_t {   // st is a compile-time constant wherever this is called
    return st < G::kStagesHigh ? high0 + (uint32_t)(st * G::kPieceBytes)
                               : low0 + (uint32_t)((st - G::kStagesHigh) * G::kPieceBytes);
  };
  if (lane == 0) {
#pragma unroll
    for (int st = 0; st < S; ++st) mbar_init(bar0 + 8 * st, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  // the warp's tiles are t0 + warp + nwarps * ti, ti < my_tiles.  Chunks beyond K are not copied (bytes of piece
  // pc: piece_bytes[pc], 0 = the piece is skipped altogether); the tables of chunks beyond K are all zero, so the
  // stale bits looked up for the uncopied part of a piece add nothing.
  const int my_tiles = t1 > t0 + warp ? (t1 - t0 - warp + nwarps - 1) / nwarps : 0;
  uint32_t piece_bytes[P];
#pragma unroll
  for (int pc = 0; pc < P; ++pc)
    piece_bytes[pc] = (uint32_t)max(0, min(PC, chunks - (chunk0 + pc * PC))) * (BITS * kTableUnitBytes);
  const unsigned char* src_task = packed + ((int64_t)(t0 + warp) * chunks + chunk0) * (BITS * kTableUnitBytes);
  const int64_t tile_stride = (int64_t)nwarps * chunks * (BITS * kTableUnitBytes);
  auto issue = [&](int st, int pc, const unsigned char* task_src) {   // lane 0 only; st, pc compile-time constants
    if (piece_bytes[pc] != 0) {
      mbar_expect_tx(bar0 + 8 * st, piece_bytes[pc]);
      bulk_load(stage_addr(st), task_src + pc * G::kPieceBytes, piece_bytes[pc], bar0 + 8 * st);
    }
  };
  if (lane == 0) {
#pragma unroll
    for (int tt = 0; tt < TPR; ++tt)
      if (tt < my_tiles) {
#pragma unroll
        for (int pc = 0; pc < P; ++pc) issue(tt * P + pc, pc, src_task + tt * tile_stride);
      }
  }
  // Pull this slice of x towards L2 (a hint: it binds no value, so it is harmless should x still be changing).
  if (warp == 0 && lane < NL * 4) {
    const int64_t k0 = (int64_t)chunk0 * kTableChunkK + lane * 64;
    if (k0 < K) asm volatile("prefetch.global.L2 [%0];" ::"l"(x + k0));
  }
  // per-lane table columns: step i of a 16-byte piece addresses column a + 2 * ((r + i) % 16)
  uint32_t base[16];
  {
    const int a = lane & 1, r = lane >> 1;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      // through an opaque move: the 16 values must stay in registers
      asm volatile("mov.u32 %0, %1;" : "=r"(base[i]) : "r"(wb | kLutTableBase | ((uint32_t)(a + 2 * ((r + i) & 15)) << 2)));
    }
  }
  auto row_codebook = [&](int ti, uint32_t (&c)[2]) {   // codebook of this lane's row of the warp's tile number ti
    const int64_t n = (int64_t)(t0 + warp + ti * nwarps) * 16 + (lane >> 1);
    load_row_codebook<BITS>(cb, n < N ? n : N - 1, c);
  };
  uint32_t cnext[2] = {0, 0};
  if (my_tiles > 0) row_codebook(0, cnext);
  float* part = scratch + (size_t)slice * CL * rows_pad + (size_t)(t0 + warp) * 16 + (lane >> 1);

  // ================= everything below may depend on the previous kernel (x, y, scratch) =================
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;");

  // ---- build the tables of this slice: item (j, h) = entries 16 h .. 16 h + 15 of every group of chunk j; the warps
  //      take the 16 NL items in turn, all loads of x first ----
  {
    constexpr int kItems = 16 * NL, kMaxPerWarp = (kItems + 15) / 16;   // at least 16 warps
    uint4 xv[kMaxPerWarp];
#pragma unroll
    for (int u = 0; u < kMaxPerWarp; ++u) {
      const int item = warp + u * nwarps;
      const int64_t k0 = ((int64_t)(chunk0 + (item >> 4)) * 32 + lane) * 8;
      xv[u] = make_uint4(0, 0, 0, 0);
      if (item < kItems && k0 < K) xv[u] = __ldg(reinterpret_cast<const uint4*>(x + k0));
    }
#pragma unroll
    for (int u = 0; u < kMaxPerWarp; ++u) {
      const int item = warp + u * nwarps;
      if (item < kItems) {   // warp-uniform
        const int j = item >> 4, h = item & 15;
        const float x0 = __uint_as_float(xv[u].x << 16), x1 = __uint_as_float(xv[u].x & 0xFFFF0000u);
        const float x2 = __uint_as_float(xv[u].y << 16), x3 = __uint_as_float(xv[u].y & 0xFFFF0000u);
        const float x4 = __uint_as_float(xv[u].z << 16), x5 = __uint_as_float(xv[u].z & 0xFFFF0000u);
        const float x6 = __uint_as_float(xv[u].w << 16), x7 = __uint_as_float(xv[u].w & 0xFFFF0000u);
        float hs = 0.f;   // inputs 4..7 selected by the high nibble h (warp-uniform)
        if (h & 1) hs += x4;
        if (h & 2) hs += x5;
        if (h & 4) hs += x6;
        if (h & 8) hs += x7;
        float l[16];
        l[0] = 0.f;  l[1] = x0;  l[2] = x1;  l[3] = x0 + x1;
        l[4] = x2;   l[5] = x0 + x2;  l[6] = x1 + x2;  l[7] = l[3] + x2;
#pragma unroll
        for (int i = 0; i < 8; ++i) l[8 + i] = l[i] + x3;
        const uint32_t dst = wb + kLutTableBase + lut_slot_offset(j) + (uint32_t)h * 16u * 256u + (uint32_t)lane * 4u;
#pragma unroll
        for (int i = 0; i < 16; ++i) sts_f32(dst + i * 256, l[i] + hs);
        // entry 255 = the sum of all 8 inputs of the group: summed over the chunk's groups by the warp of item (j, 15)
        if (h == 15) {
          float v = l[15] + hs;
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
          if (lane == 0) sts_f32(wb + G::kSumBase + 4 * j, v);
        }
      }
    }
  }
  __syncthreads();
  float sx_slice = 0.f;   // sum of the activations of this slice, chunk by chunk
#pragma unroll
  for (int j = 0; j < NL; ++j) sx_slice += lds_f32<0>(wb + G::kSumBase + 4 * j);
  if (threadIdx.x == 0 && slices > 1) {
    if (in_cluster) sts_f32(wb + G::kSxWord, sx_slice);
    else if (rb == 0) scratch[(size_t)slices * CL * rows_pad + slice] = sx_slice;
  }

  bool ok = true;
  for (int ti0 = 0; ti0 < my_tiles && ok; ti0 += TPR) {
    const uint32_t parity = (uint32_t)(ti0 / TPR) & 1u;
#pragma unroll
    for (int tt = 0; tt < TPR; ++tt) {
      const int ti = ti0 + tt;
      if (ti < my_tiles && ok) {   // warp-uniform
        const uint32_t ccur[2] = {cnext[0], cnext[1]};
        const int s = smallest_centroid<BITS>(ccur);
        const uint32_t mlo = (s & 1) ? 0xFFFFFFFFu : 0u, mhi = (s & 2) ? 0xFFFFFFFFu : 0u;
        if (ti + 1 < my_tiles) row_codebook(ti + 1, cnext);
        float acc[CL][2];
#pragma unroll
        for (int q = 0; q < CL; ++q) acc[q][0] = acc[q][1] = 0.f;
#pragma unroll
        for (int pc = 0; pc < P; ++pc) {
          const int st = tt * P + pc;
          if (piece_bytes[pc] != 0 && ok) {   // uniform over the CTA
            if (!mbar_wait(bar0 + 8 * st, parity)) ok = false;
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (ok) {
              const uint32_t sa = stage_addr(st) + lane * 16;
#pragma unroll
              for (int u = 0; u < PC; ++u) {   // chunk pc * PC + u of the slice sits in table slot pc * PC + u
                const uint4 r0 = lds_u4(sa + u * BITS * kTableUnitBytes);
                const uint32_t lo[4] = {r0.x ^ mlo, r0.y ^ mlo, r0.z ^ mlo, r0.w ^ mlo};
                if constexpr (BITS == 1) {
                  lookup16_slot(pc * PC + u, lo, base, acc[0][0], acc[0][1]);
                } else {
                  const uint4 r1 = lds_u4(sa + u * BITS * kTableUnitBytes + kTableUnitBytes);
                  const uint32_t hi[4] = {r1.x, r1.y, r1.z, r1.w};
                  uint32_t i1[4], i2[4], i3[4];
#pragma unroll
                  for (int i = 0; i < 4; ++i) {
                    i1[i] = lop3<0x90>(lo[i], hi[i], mhi);   // p & ~q   (p = lo ^ mlo, q = hi ^ mhi): index s ^ 1
                    i2[i] = lop3<0x06>(lo[i], hi[i], mhi);   // ~p & q: index s ^ 2
                    i3[i] = lop3<0x60>(lo[i], hi[i], mhi);   // p & q:  index s ^ 3
                  }
                  lookup16_slot(pc * PC + u, i1, base, acc[0][0], acc[0][1]);
                  lookup16_slot(pc * PC + u, i2, base, acc[CL - 2][0], acc[CL - 2][1]);
                  lookup16_slot(pc * PC + u, i3, base, acc[CL - 1][0], acc[CL - 1][1]);
                }
              }
              // every lane has used what it read from the stage: refill it with the same piece of the tile one
              // ring round ahead
              __syncwarp();
              if (lane == 0 && ti + TPR < my_tiles) issue(st, pc, src_task + TPR * tile_stride);
            }
          }
        }
        // the two lanes of a row hold its even and odd groups
        const int tile = t0 + warp + ti * nwarps;
        float v[CL];
#pragma unroll
        for (int q = 0; q < CL; ++q) {
          v[q] = acc[q][0] + acc[q][1];
          v[q] += __shfl_xor_sync(0xFFFFFFFFu, v[q], 1);
        }
        if (slices == 1) {
          // the whole of K is in this slice: apply the codebook and store
          const int64_t n = (int64_t)tile * 16 + (lane >> 1);
          if ((lane & 1) == 0 && n < N && ok) {
            auto cent = [&](int i) { return bf16_bits_to_float((ccur[i >> 1] >> ((i & 1) * 16)) & 0xFFFFu); };
            const float cs = cent(s);
            float out = cs * sx_slice;
#pragma unroll
            for (int q = 0; q < CL; ++q) out = fmaf(cent(s ^ (q + 1)) - cs, v[q], out);
            y[n] = (uint16_t)float_to_bf16_bits(out);
          }
        } else if (in_cluster) {
          // this CTA's share of the rows' sums stays in its shared memory for the reduction over the cluster
          if ((lane & 1) == 0) {
            const int row_local = (tile - t0) * 16 + (lane >> 1);
#pragma unroll
            for (int q = 0; q < CL; ++q)
              sts_f32(wb + G::kPartBase + 4u * (uint32_t)(q * rows_blk + row_local), ok ? v[q] : 0.f);
          }
        } else if (ok && (lane & 1) == 0) {
#pragma unroll
          for (int q = 0; q < CL; ++q) part[(size_t)q * rows_pad] = v[q];
        }
        part += nwarps * 16;
        src_task += tile_stride;
      }
    }
  }
  if (!ok) {
    // A copy did not arrive in time: report it.  The copies still under way get one more bounded wait each before
    // the CTA gives its shared memory back (phase parities alternate, so waiting for both covers every stage).
    if (lane == 0) atomicOr(err, kErrWait);
    for (int st = 0; st < S; ++st) {
      if (!mbar_try(bar0 + 8 * st, 0)) (void)mbar_wait_slow(bar0 + 8 * st, 1);
    }
  }
  if (!in_cluster) return;

  // ---- reduction over the cluster: the `slices` CTAs of a row block are one thread-block cluster (rank = slice:
  //      the grid is slice-major in x and the cluster spans `slices` CTAs in x).  No CTA leaves the kernel between
  //      its start and here except through the window check above, which fails in all CTAs or in none; so every CTA
  //      reaches both barriers.  After the first, CTA `slice` adds, for its share of the block's rows, the sums of
  //      all slices in slice order straight out of the other CTAs' shared memory, applies the codebook and stores;
  //      the second keeps every CTA's shared memory alive until all have read it.
  __syncthreads();
  cluster_sync_all();
  {
    const int share = (rows_blk + slices - 1) / slices;
    const int r_begin = slice * share, r_end = min(rows_blk, r_begin + share);
    float sx = 0.f;
    for (int s2 = 0; s2 < slices; ++s2) sx += ld_cluster_f32(wb + G::kSxWord, (uint32_t)s2);
    for (int row_local = r_begin + (int)threadIdx.x; row_local < r_end; row_local += (int)blockDim.x) {
      const int64_t n = (int64_t)t0 * 16 + row_local;
      if (n >= N) break;
      uint32_t c[2];
      load_row_codebook<BITS>(cb, n, c);
      float a[CL];
#pragma unroll
      for (int q = 0; q < CL; ++q) a[q] = 0.f;
      for (int s2 = 0; s2 < slices; ++s2) {
#pragma unroll
        for (int q = 0; q < CL; ++q)
          a[q] += ld_cluster_f32(wb + G::kPartBase + 4u * (uint32_t)(q * rows_blk + row_local), (uint32_t)s2);
      }
      const int sm = smallest_centroid<BITS>(c);
      auto cent = [&](int i) { return bf16_bits_to_float((c[i >> 1] >> ((i & 1) * 16)) & 0xFFFFu); };
      const float cs = cent(sm);
      float out = cs * sx;
#pragma unroll
      for (int q = 0; q < CL; ++q) out = fmaf(cent(sm ^ (q + 1)) - cs, a[q], out);
      y[n] = (uint16_t)float_to_bf16_bits(out);
    }
  }
  cluster_sync_all();
}

// Second kernel (more than one slice): adds the slices of every row in a fixed order, applies the codebook and stores
// bf16.  A CTA of 8 warps owns 32 rows (lane = row); warp w adds the slices w, w + 8, ... of its rows (independent
// loads: one trip to L2), then warp 0 adds the 8 partial sums in order.
constexpr int kFinWarps = 8;

template <int BITS>
__global__ void __launch_bounds__(kFinWarps * 32)
    linear_lut_finish_kernel(const float* __restrict__ scratch, const uint16_t* __restrict__ cb,
                             uint16_t* __restrict__ y, int64_t N, int slices) {
  constexpr int CL = BITS == 1 ? 1 : 3;
  __shared__ float part[kFinWarps][CL + 1][32];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t rows_pad = table_tiles(N) * 16;
  const int64_t n = (int64_t)blockIdx.x * 32 + lane;
  const bool in_pad = n < rows_pad;
  uint32_t c[2] = {0, 0};
  if (warp == 0 && n < N) load_row_codebook<BITS>(cb, n, c);   // a constant of the layer: before the wait
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;");
  const float* sxp = scratch + (size_t)slices * CL * rows_pad;
  float a[CL], sx = 0.f;
#pragma unroll
  for (int q = 0; q < CL; ++q) a[q] = 0.f;
  for (int s0 = warp; s0 < slices; s0 += 4 * kFinWarps) {
    float v[4][CL], vs[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int s = s0 + u * kFinWarps;
      const bool ok = s < slices && in_pad;
#pragma unroll
      for (int q = 0; q < CL; ++q) v[u][q] = ok ? __ldcg(scratch + ((size_t)s * CL + q) * rows_pad + n) : 0.f;
      vs[u] = s < slices ? __ldcg(sxp + s) : 0.f;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
#pragma unroll
      for (int q = 0; q < CL; ++q) a[q] += v[u][q];
      sx += vs[u];
    }
  }
#pragma unroll
  for (int q = 0; q < CL; ++q) part[warp][q][lane] = a[q];
  part[warp][CL][lane] = sx;
  __syncthreads();
  if (warp != 0 || n >= N) return;
#pragma unroll
  for (int w = 1; w < kFinWarps; ++w) {
#pragma unroll
    for (int q = 0; q < CL; ++q) a[q] += part[w][q][lane];
    sx += part[w][CL][lane];
  }
  const int s = smallest_centroid<BITS>(c);
  auto cent = [&](int i) { return bf16_bits_to_float((c[i >> 1] >> ((i & 1) * 16)) & 0xFFFFu); };
  const float cs = cent(s);
  float v = cs * sx;
#pragma unroll
  for (int q = 0; q < CL; ++q) v = fmaf(cent(s ^ (q + 1)) - cs, a[q], v);
  y[n] = (uint16_t)float_to_bf16_bits(v);
}

__device__ unsigned int g_lut_error;   // sticky: bit 1 = the kernel found its shared-memory window misplaced

}  // namespace

// Device address of the error word, looked up once per device.
unsigned int* lut_error_word(cudaError_t* e) {
  static unsigned int* addr[64] = {};
  static std::mutex mu;
  int dev = 0;
  *e = cudaGetDevice(&dev);
  if (*e != cudaSuccess) return nullptr;
  if (dev < 0 || dev >= 64) {
    *e = cudaErrorInvalidDevice;
    return nullptr;
  }
  std::lock_guard<std::mutex> lock(mu);
  if (!addr[dev]) {
    void* p = nullptr;
    *e = cudaGetSymbolAddress(&p, g_lut_error);
    if (*e != cudaSuccess) return nullptr;
    addr[dev] = static_cast<unsigned int*>(p);
  }
  return addr[dev];
}

namespace {

struct LutPlan {
  int nl, slices, row_blocks, warps;
  int cluster;   // 1: the slices of a row block form a thread-block cluster and are added through its shared memory
};

constexpr int lut_max_warps(int nl) { return nl <= 2 ? 32 : nl == 3 ? 24 : 20; }

// How many clusters of `csize` CTAs of linear_lut_kernel<BITS, NL> can be resident at once (0: none, or the query
// failed).
template <int BITS, int NL>
int lut_cluster_capacity_one(int csize) {
  using G = LutGeo<BITS, NL>;
  constexpr int smem = (int)G::kHighEnd - 1024;
  if (cudaFuncSetAttribute(linear_lut_kernel<BITS, NL>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
    return 0;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)csize;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(csize * 64));
  cfg.blockDim = dim3((unsigned)(G::kWarps * 32));
  cfg.dynamicSmemBytes = smem;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, linear_lut_kernel<BITS, NL>, &cfg) != cudaSuccess) {
    (void)cudaGetLastError();
    return 0;
  }
  return n;
}

int lut_cluster_capacity(int bits, int nl, int csize) {
  static int cache[64][3][5][4];   // [device][bits][nl][log2 csize]; 0 = not asked yet, -1 = none
  static std::mutex mu;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  const int lg = csize == 2 ? 1 : csize == 4 ? 2 : csize == 8 ? 3 : 0;
  if (lg == 0 || nl < 1 || nl > 4 || (bits != 1 && bits != 2) || (bits == 2 && nl > 3)) return 0;
  std::lock_guard<std::mutex> lock(mu);
  int& c = cache[dev][bits][nl][lg];
  if (c == 0) {
    int n = 0;
    if (bits == 1) n = nl == 1 ? lut_cluster_capacity_one<1, 1>(csize) : nl == 2 ? lut_cluster_capacity_one<1, 2>(csize)
                     : nl == 3 ? lut_cluster_capacity_one<1, 3>(csize) : lut_cluster_capacity_one<1, 4>(csize);
    else n = nl == 1 ? lut_cluster_capacity_one<2, 1>(csize) : nl == 2 ? lut_cluster_capacity_one<2, 2>(csize)
                     : lut_cluster_capacity_one<2, 3>(csize);
    c = n > 0 ? n : -1;
  }
  return c > 0 ? c : 0;
}

// Floats of partial sums a CTA can keep for the reduction over its cluster.
int lut_part_floats(int bits, int nl) {
  if (bits == 1) return nl == 1 ? LutGeo<1, 1>::kPartFloats : nl == 2 ? LutGeo<1, 2>::kPartFloats
                        : nl == 3 ? LutGeo<1, 3>::kPartFloats : LutGeo<1, 4>::kPartFloats;
  return nl == 1 ? LutGeo<2, 1>::kPartFloats : nl == 2 ? LutGeo<2, 2>::kPartFloats : LutGeo<2, 3>::kPartFloats;
}

// Chunks per slice: the choice that minimises the shared-memory work of the busiest CTA (table build: 256 cycles per
// chunk; lookups: 16 cycles per tile, chunk and class) with all CTAs resident at once; then as many warps as give
// every warp the same number of tiles (at least 16: the table build needs them).  Adding the slices costs a second
// kernel (about 5000 cycles with its two kernel-to-kernel transitions) unless the 2, 4 or 8 slices of a row block can
// run as one cluster (about 1000 cycles for its two barriers and the loads from the other CTAs' shared memory).
LutPlan plan_lut(int64_t N, int64_t K, int bits, int sm_count) {
  const int64_t chunks = table_chunks(K), tiles = table_tiles(N);
  const int classes = bits == 1 ? 1 : 3;
  LutPlan best = {1, (int)chunks, 1, 16, 0};
  double best_cost = 1e30;
  auto consider = [&](int nl, int64_t slices, int64_t rb, int cluster) {
    const int64_t tiles_cta = (tiles + rb - 1) / rb;
    const int64_t waves = (slices * rb + sm_count - 1) / sm_count;
    const int64_t tasks_warp = (tiles_cta + lut_max_warps(nl) - 1) / lut_max_warps(nl);
    int64_t warps = (tiles_cta + tasks_warp - 1) / tasks_warp;
    if (warps < 16) warps = 16;
    const double cost = (double)waves * (256.0 * nl + (16.0 * classes + 4.0) * nl * (double)(tasks_warp * warps) + 600.0) +
                        8.0 * slices + (slices == 1 ? 0.0 : cluster ? 1000.0 : 5000.0);
    if (cost < best_cost) {
      best_cost = cost;
      best = {nl, (int)slices, (int)rb, (int)warps, cluster};
    }
  };
  for (int nl = 1; nl <= (bits == 1 ? 4 : 3); ++nl) {
    const int64_t slices = (chunks + nl - 1) / nl;
    int64_t rb = sm_count / slices;
    if (rb < 1) rb = 1;
    if (rb > tiles) rb = tiles;
    consider(nl, slices, rb, 0);
    if (slices == 2 || slices == 4 || slices == 8) {
      int64_t rbc = lut_cluster_capacity(bits, nl, (int)slices);
      if (rbc > tiles) rbc = tiles;
      if (rbc >= 1 && ((tiles + rbc - 1) / rbc) * 16 * classes <= lut_part_floats(bits, nl)) consider(nl, slices, rbc, 1);
    }
  }
  return best;
}

template <int BITS, int NL>
cudaError_t launch_lut_one(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
                           int64_t K, const LutPlan& p, float* scratch, unsigned int* err, cudaStream_t s) {
  using G = LutGeo<BITS, NL>;
  constexpr int smem = (int)G::kHighEnd - 1024;   // dynamic shared memory starts at or below byte 1024 of the window
  static bool configured[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(linear_lut_kernel<BITS, NL>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;   // CTAs slice 0 .. slices-1 of a row block are consecutive in x
  attr[1].val.clusterDim.x = (unsigned)p.slices;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(p.slices * p.row_blocks));
  cfg.blockDim = dim3((unsigned)(p.warps * 32));
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = p.cluster ? 2 : 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, linear_lut_kernel<BITS, NL>, reinterpret_cast<const unsigned char*>(packed),
                                     cb, x, y, scratch, N, K, p.slices, p.row_blocks, err, p.cluster);
  if (e != cudaSuccess || p.slices == 1 || p.cluster) return e;
  cudaLaunchConfig_t fin = {};
  fin.gridDim = dim3((unsigned)((N + 31) / 32));
  fin.blockDim = dim3(kFinWarps * 32);
  fin.stream = s;
  fin.attrs = attr;
  fin.numAttrs = 1;
  return cudaLaunchKernelEx(&fin, linear_lut_finish_kernel<BITS>, (const float*)scratch, cb, y, N, p.slices);
}

template <int BITS>
cudaError_t launch_lut_bits(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
                            int64_t K, const LutPlan& p, float* scratch, unsigned int* err, cudaStream_t s) {
  switch (p.nl) {
    case 1: return launch_lut_one<BITS, 1>(packed, cb, x, y, N, K, p, scratch, err, s);
    case 2: return launch_lut_one<BITS, 2>(packed, cb, x, y, N, K, p, scratch, err, s);
    case 3: return launch_lut_one<BITS, 3>(packed, cb, x, y, N, K, p, scratch, err, s);
    default: break;
  }
  if constexpr (BITS == 1) {
    if (p.nl == 4) return launch_lut_one<BITS, 4>(packed, cb, x, y, N, K, p, scratch, err, s);
  }
  return cudaErrorInvalidValue;   // unreachable: plan_lut only picks the slice lengths instantiated here
}

}  // namespace

bool linear_lut_supports(int64_t N, int64_t K, int bits, int64_t M) {
  (void)N;
  (void)M;
  const DeviceInfo* di = device_info();
  // tables and stages sit at fixed shared-memory addresses and take almost all of a 228 KB SM
  return di && (bits == 1 || bits == 2) && (K % 8) == 0 && di->max_smem_optin >= 227 * 1024;
}

// Where the table kernel is the faster one.  It costs one pass per batch row (the tensor-core kernels cost about the
// same for 1 to 8 rows) and a fixed few microseconds (its CTAs take a whole SM each, so consecutive calls do not
// overlap; the table build; the second kernel or the cluster reduction), so it pays at batch 1 on large 1-bit
// layers.  Measured on B200, table against tensor-core kernel, b = 1, us per call: 8192 x 28672: 14.8 / 27.9;
// 6144 x 20480: 10.0 / 15.9; 20480 x 6144: 10.6 / 14.6; 8192 x 8192: 8.0 / 9.1; at 50 to 59 M weights about equal
// (4096 x 14336: 7.8 / 8.2; 14336 x 4096: 8.5 / 8.3; 8192 x 6144: 7.2 / 7.1; 16384 x 3072: 6.8 / 7.9); below, the
// tensor-core kernel (6144 x 6144: 6.8 / 5.7; 4096 x 4096: 5.5 / 3.2).  b = 2 never: 8192 x 8192: 12.0 / 10.4.
bool linear_lut_preferred(int64_t N, int64_t K, int bits, int64_t M) {
  return linear_lut_supports(N, K, bits, M) && bits == 1 && M == 1 && N * K >= (int64_t(1) << 26);
}

size_t linear_lut_scratch_bytes(int64_t N, int64_t K, int bits) {
  const DeviceInfo* di = device_info();
  if (!di) return 0;
  const LutPlan p = plan_lut(N, K, bits, di->sm_count);
  if (p.slices == 1 || p.cluster) return 0;   // the whole of K in one CTA, or the slices added inside a cluster
  return lut_scratch_floats(p.slices, bits == 1 ? 1 : 3, table_tiles(N) * 16) * sizeof(float);
}

// One batch row per pass (two kernels each unless the slice is the whole of K); the scratch is reused from pass to pass.
cudaError_t launch_linear_lut(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
                              int64_t K, int bits, int64_t M, void* scratch, cudaStream_t s) {
  const DeviceInfo* di = device_info();
  if (!di) return cudaErrorInvalidDevice;
  const LutPlan p = plan_lut(N, K, bits, di->sm_count);
  cudaError_t e = cudaSuccess;
  unsigned int* err = lut_error_word(&e);
  if (!err) return e;
  for (int64_t m = 0; m < M; ++m) {
    e = bits == 1 ? launch_lut_bits<1>(packed, cb, x + m * K, y + m * N, N, K, p, (float*)scratch, err, s)
                  : launch_lut_bits<2>(packed, cb, x + m * K, y + m * N, N, K, p, (float*)scratch, err, s);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

cudaError_t read_lut_error_flags(unsigned int* flags) {
  *flags = 0;
  cudaError_t e = cudaMemcpyFromSymbol(flags, g_lut_error, sizeof(unsigned int));
  if (e != cudaSuccess) return e;
  if (*flags) {
    const unsigned int zero = 0;
    e = cudaMemcpyToSymbol(g_lut_error, &zero, sizeof(unsigned int));
  }
  return e;
}

}  // namespace kmq
