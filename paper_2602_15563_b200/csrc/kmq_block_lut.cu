// The paper's block format (shared codebook of 2^b centroids, bf16 scale per block of 64) through an activation
// table: kmq_block_table_pack / _unpack / _linear, b = 1, 2, 4, decode batches (one pass per batch row).
//
// Because the codebook is shared by all rows, a table over the activations can hold finished partial dot products:
// for the group of 8 / b inputs that one byte of packed indices covers,
//     U_g[e] = sum_t x[g * (8/b) + t] * c[(e >> (t * b)) & (2^b - 1)],        e = 0 .. 255
// (the paper's 256-entry byte table, Appendix "Benchmarking", "Kernel implementations", moved from the weights to
// the activations), and the layer with deferred scaling becomes
//     y[n] = sum_blocks scale[n, blk] * sum_{g in blk} U_g[byte[n, g]]:
// one shared-memory lookup and one fp32 add per byte of weights, one multiply-add per block.  Every entry is a sum of
// the selected products themselves (no differences of centroids), so its rounding error is relative to the terms it
// stands for whatever the codebook.
//
// A CTA (slice s, row block rb) builds the tables of its K slice (NL chunks of 32 groups, 32 KB each) once and streams
// the units of its rows' tiles through them (layout: kmq_table_layout.cuh; bulk asynchronous copies into a ring of
// two stages per warp, one mbarrier each, time-bounded waits).  A lane owns one row of the tile and every second
// group; the layout's rotation keeps the 32 lookups of a step on 32 different banks and whole runs of steps inside
// one block.  With one slice the warp stores its rows; otherwise the slice sums go to scratch [slice][row] and a
// second kernel adds them in a fixed order.
//
// Programmatic dependent launch as in the per-row table kernel: before griddepcontrol.wait only the packed table and
// the codebook (constants of the layer) and the CTA's own shared memory are touched.
#include "kmq_common.cuh"
#include "kmq_lut_common.cuh"
#include "kmq_table_layout.cuh"

namespace kmq {
namespace {

constexpr uint32_t kSmemEnd = 227 * 1024 + 1024;   // end of the shared-memory window of a CTA (absolute address)

template <int BITS, int NL>
struct BGeo {
  static constexpr int kUnit = btl_unit_bytes(BITS);
  static constexpr int kStageBytes = NL * kUnit;                 // one tile's share of the slice = one bulk copy
  static constexpr uint32_t kCbBase = 1152;                      // 16 floats: the codebook
  static constexpr uint32_t kBarBase = 1216;                     // mbarriers, 8 bytes per stage
  static constexpr uint32_t kLowBase = 2304;                     // stages below the tables: [kLowBase, kLutTableBase)
  static constexpr uint32_t kTableEnd = kLutTableBase + (uint32_t)((NL + 1) / 2) * 65536u;
  static constexpr int kLowStages = (int)((kLutTableBase - kLowBase) / kStageBytes);
  static constexpr int kHighStages = (int)((kSmemEnd - kTableEnd) / kStageBytes);
  static constexpr int kStagesPerWarp = 2;
  static constexpr int kWarpsFit = (kLowStages + kHighStages) / kStagesPerWarp;
  static constexpr int kWarps = kWarpsFit > 20 ? 20 : kWarpsFit;
  static constexpr uint32_t kHighEnd = kTableEnd + (uint32_t)(kHighStages * kStageBytes);
  static_assert(kWarps >= 16, "the table build needs 16 warps");
  static_assert(kBarBase + kWarps * kStagesPerWarp * 8 <= kLowBase, "mbarriers must fit below the stages");
  static_assert(kStageBytes % 16 == 0, "bulk copies move multiples of 16 bytes");
  static_assert(NL >= 1 && NL <= 4, "unsupported slice length");
};

__device__ __forceinline__ uint32_t lds_b32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint2 lds_b64(uint32_t addr) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint32_t lds_b16(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}

// One lookup: byte k of `w` is the entry, `base` carries the table base and the column.
template <uint32_t IMM, int KBYTE>
__device__ __forceinline__ float lookup1(uint32_t w, uint32_t base) {
  return lds_f32<IMM>(prmt(w, base, 0x7604u | (uint32_t)(KBYTE << 4)));
}

// Steps [I0, I0 + CNT) of a lane's 16 bytes (CNT a multiple of 4, I0 too): sum of the CNT lookups in table slot Q.
template <int Q, int I0, int CNT>
__device__ __forceinline__ float run_sum(const uint32_t (&w)[4], const uint32_t (&base)[16]) {
  constexpr uint32_t IMM = lut_slot_offset(Q);
  float a0 = 0.f, a1 = 0.f;
#pragma unroll
  for (int i = I0; i < I0 + CNT; i += 4) {
    a0 += lookup1<IMM, 0>(w[i >> 2], base[i + 0]);
    a1 += lookup1<IMM, 1>(w[i >> 2], base[i + 1]);
    a0 += lookup1<IMM, 2>(w[i >> 2], base[i + 2]);
    a1 += lookup1<IMM, 3>(w[i >> 2], base[i + 3]);
  }
  return a0 + a1;
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// One chunk of one tile: the lane's 16 lookups of table slot Q, block by block, each block's sum times its scale.
template <int BITS, int Q>
__device__ __forceinline__ float chunk_sum(uint32_t unit_addr, int lane, const uint32_t (&base)[16]) {
  const uint4 r0 = lds_u4(unit_addr + lane * 16);
  const uint32_t w[4] = {r0.x, r0.y, r0.z, r0.w};
  const int r = lane >> 1;
  if constexpr (BITS == 4) {
    const float s = bf16_lo(lds_b16(unit_addr + 512 + r * 2));
    return s * run_sum<Q, 0, 16>(w, base);
  } else if constexpr (BITS == 2) {
    // two blocks; the run j of row r is block (j + r / 8) % 2: swap the halves for the rows 8..15
    uint32_t sc = lds_b32(unit_addr + 512 + r * 4);
    sc = prmt(sc, sc, (r & 8) ? 0x1032u : 0x3210u);
    float v = bf16_lo(sc) * run_sum<Q, 0, 8>(w, base);
    return fmaf(bf16_hi(sc), run_sum<Q, 8, 8>(w, base), v);
  } else {
    // four blocks; run j of row r is block (j + r / 4) % 4: rotate the four scales right by r / 4 places
    uint2 sc = lds_b64(unit_addr + 512 + r * 8);
    if (r & 8) {
      const uint32_t t = sc.x;
      sc.x = sc.y;
      sc.y = t;
    }
    if (r & 4) {
      const uint32_t lo = __funnelshift_r(sc.x, sc.y, 16), hi = __funnelshift_r(sc.y, sc.x, 16);
      sc.x = lo;
      sc.y = hi;
    }
    float v = bf16_lo(sc.x) * run_sum<Q, 0, 4>(w, base);
    v = fmaf(bf16_hi(sc.x), run_sum<Q, 4, 4>(w, base), v);
    v = fmaf(bf16_lo(sc.y), run_sum<Q, 8, 4>(w, base), v);
    return fmaf(bf16_hi(sc.y), run_sum<Q, 12, 4>(w, base), v);
  }
}

template <int BITS, int NL>
__global__ void __launch_bounds__(BGeo<BITS, NL>::kWarps * 32, 1)
    block_lut_kernel(const unsigned char* __restrict__ tab, const uint16_t* __restrict__ codebook,
                     const uint16_t* __restrict__ x, uint16_t* __restrict__ y, float* __restrict__ scratch, int64_t N,
                     int64_t K, int slices, int row_blocks, unsigned int* __restrict__ err) {
  using G = BGeo<BITS, NL>;
  constexpr int S = G::kStagesPerWarp, UB = G::kUnit, GW = 8 / BITS;   // GW = weights per group
  extern __shared__ __align__(128) unsigned char smem_raw[];

  // ================= before the previous kernel on the stream is known to have finished =================
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  const int slice = blockIdx.x % slices, rb = blockIdx.x / slices;
  const int chunks = (int)btl_chunks(K, BITS);
  const int tiles = (int)table_tiles(N);
  const int64_t rows_pad = (int64_t)tiles * 16;
  const int chunk0 = slice * NL;
  const int nvalid = min(NL, chunks - chunk0);   // chunks of this slice that exist
  const int t0 = (int)((int64_t)tiles * rb / row_blocks), t1 = (int)((int64_t)tiles * (rb + 1) / row_blocks);
  {
    const uint32_t s0 = smem_addr(smem_raw);
    uint32_t dyn;
    asm("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn));
    if (s0 > G::kCbBase || s0 + dyn < G::kHighEnd) {
      asm volatile("griddepcontrol.wait;" ::: "memory");
      if (threadIdx.x == 0) atomicOr(err, kErrWindow);
      return;
    }
  }
  // this warp's two stages: slot ids warp * S + st, the first kLowStages slots below the tables, the rest above
  uint32_t stage[S], bar[S];
#pragma unroll
  for (int st = 0; st < S; ++st) {
    const int sid = warp * S + st;
    stage[st] = sid < G::kLowStages ? G::kLowBase + (uint32_t)(sid * G::kStageBytes)
                                    : G::kTableEnd + (uint32_t)((sid - G::kLowStages) * G::kStageBytes);
    bar[st] = G::kBarBase + (uint32_t)sid * 8u;
  }
  if (lane == 0) {
#pragma unroll
    for (int st = 0; st < S; ++st) mbar_init(bar[st], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  const int my_tiles = t1 > t0 + warp ? (t1 - t0 - warp + nwarps - 1) / nwarps : 0;
  const uint32_t piece_bytes = (uint32_t)(nvalid * UB);
  const unsigned char* src_task = tab + ((int64_t)(t0 + warp) * chunks + chunk0) * UB;
  const int64_t tile_stride = (int64_t)nwarps * chunks * UB;
  if (lane == 0) {
#pragma unroll
    for (int st = 0; st < S; ++st)
      if (st < my_tiles) {
        mbar_expect_tx(bar[st], piece_bytes);
        bulk_load(stage[st], src_task + st * tile_stride, piece_bytes, bar[st]);
      }
  }
  if (warp == 0 && lane < NL * 4) {   // a hint: pull this slice of x towards L2
    const int64_t k0 = (int64_t)chunk0 * btl_chunk_k(BITS) + lane * (btl_chunk_k(BITS) / 4);
    if (k0 < K) asm volatile("prefetch.global.L2 [%0];" ::"l"(x + k0));
  }
  if (threadIdx.x < (1 << BITS)) sts_f32(G::kCbBase + 4 * threadIdx.x, bf16_bits_to_float(__ldg(codebook + threadIdx.x)));
  uint32_t base[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    // through an opaque move: the 16 values must stay in registers
    asm volatile("mov.u32 %0, %1;" : "=r"(base[i]) : "r"(kLutTableBase | ((uint32_t)btl_group_of(lane, i, BITS) << 2)));
  }
  float* part = scratch + (size_t)slice * rows_pad + (size_t)(t0 + warp) * 16 + (lane >> 1);
  __syncthreads();   // the codebook is in shared memory

  // ================= everything below may depend on the previous kernel (x, y, scratch) =================
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;");

  // ---- tables of this slice: item (j, h) = entries 16 h .. 16 h + 15 of every group of chunk j; lane = group ----
  {
    constexpr int kItems = 16 * NL, kMaxPerWarp = (kItems + 15) / 16;
    uint4 xv[kMaxPerWarp];
#pragma unroll
    for (int u = 0; u < kMaxPerWarp; ++u) {
      const int item = warp + u * nwarps;
      const int64_t k0 = ((int64_t)(chunk0 + (item >> 4)) * 32 + lane) * GW;
      xv[u] = make_uint4(0, 0, 0, 0);
      if (item < kItems && k0 < K) {
        if constexpr (BITS == 1) xv[u] = __ldg(reinterpret_cast<const uint4*>(x + k0));
        else if constexpr (BITS == 2) {
          const uint2 t = __ldg(reinterpret_cast<const uint2*>(x + k0));
          xv[u].x = t.x;
          xv[u].y = t.y;
        } else xv[u].x = __ldg(reinterpret_cast<const uint32_t*>(x + k0));
      }
    }
#pragma unroll
    for (int u = 0; u < kMaxPerWarp; ++u) {
      const int item = warp + u * nwarps;
      if (item < kItems) {   // warp-uniform
        const int j = item >> 4, h = item & 15;
        float l[16], hs;
        if constexpr (BITS == 1) {
          const float c0 = lds_f32<0>(G::kCbBase), c1 = lds_f32<4>(G::kCbBase);
          const uint32_t xw[4] = {xv[u].x, xv[u].y, xv[u].z, xv[u].w};
          float p[8][2];
#pragma unroll
          for (int t = 0; t < 8; ++t) {
            const float xt = (t & 1) ? bf16_hi(xw[t >> 1]) : bf16_lo(xw[t >> 1]);
            p[t][0] = xt * c0;
            p[t][1] = xt * c1;
          }
          float A[4], B[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            A[e] = p[0][e & 1] + p[1][e >> 1];
            B[e] = p[2][e & 1] + p[3][e >> 1];
          }
#pragma unroll
          for (int e = 0; e < 16; ++e) l[e] = A[e & 3] + B[e >> 2];
          hs = (((h & 1) ? p[4][1] : p[4][0]) + ((h & 2) ? p[5][1] : p[5][0])) +
               (((h & 4) ? p[6][1] : p[6][0]) + ((h & 8) ? p[7][1] : p[7][0]));
        } else if constexpr (BITS == 2) {
          float c[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) c[q] = lds_f32<0>(G::kCbBase + 4 * q);
          const float x0 = bf16_lo(xv[u].x), x1 = bf16_hi(xv[u].x), x2 = bf16_lo(xv[u].y), x3 = bf16_hi(xv[u].y);
#pragma unroll
          for (int e = 0; e < 16; ++e) l[e] = x0 * c[e & 3] + x1 * c[e >> 2];
          hs = x2 * lds_f32<0>(G::kCbBase + 4 * (h & 3)) + x3 * lds_f32<0>(G::kCbBase + 4 * (h >> 2));
        } else {
          const float x0 = bf16_lo(xv[u].x), x1 = bf16_hi(xv[u].x);
#pragma unroll
          for (int e = 0; e < 16; ++e) l[e] = x0 * lds_f32<0>(G::kCbBase + 4 * e);
          hs = x1 * lds_f32<0>(G::kCbBase + 4 * h);
        }
        const uint32_t dst = kLutTableBase + lut_slot_offset(j) + (uint32_t)h * 16u * 256u + (uint32_t)lane * 4u;
#pragma unroll
        for (int e = 0; e < 16; ++e) sts_f32(dst + e * 256, l[e] + hs);
      }
    }
  }
  __syncthreads();

  bool ok = true;
  for (int ti0 = 0; ti0 < my_tiles && ok; ti0 += S) {
    const uint32_t parity = (uint32_t)(ti0 / S) & 1u;
#pragma unroll
    for (int st = 0; st < S; ++st) {
      const int ti = ti0 + st;
      if (ti < my_tiles && ok) {   // warp-uniform
        if (!mbar_wait(bar[st], parity)) ok = false;
        ok = __all_sync(0xFFFFFFFFu, ok);
        float v = 0.f;
        if (ok) {
          v = chunk_sum<BITS, 0>(stage[st], lane, base);
          if constexpr (NL > 1) {
            if (nvalid > 1) v += chunk_sum<BITS, 1>(stage[st] + UB, lane, base);
          }
          if constexpr (NL > 2) {
            if (nvalid > 2) v += chunk_sum<BITS, 2>(stage[st] + 2 * UB, lane, base);
          }
          if constexpr (NL > 3) {
            if (nvalid > 3) v += chunk_sum<BITS, 3>(stage[st] + 3 * UB, lane, base);
          }
          // every lane has used what it read from the stage: refill it with the tile one ring round ahead
          __syncwarp();
          if (lane == 0 && ti + S < my_tiles) {
            mbar_expect_tx(bar[st], piece_bytes);
            bulk_load(stage[st], src_task + S * tile_stride, piece_bytes, bar[st]);
          }
        }
        v += __shfl_xor_sync(0xFFFFFFFFu, v, 1);   // the two lanes of a row hold its even and odd groups
        if (ok && (lane & 1) == 0) {
          if (slices == 1) {
            const int64_t n = (int64_t)(t0 + warp + ti * nwarps) * 16 + (lane >> 1);
            if (n < N) y[n] = (uint16_t)float_to_bf16_bits(v);
          } else {
            *part = v;
          }
        }
        part += nwarps * 16;
        src_task += tile_stride;
      }
    }
  }
  if (!ok) {
    // A copy did not arrive in time: report it, and give the copies still under way one more bounded wait each
    // before the CTA gives its shared memory back (waiting for both phase parities covers every stage).
    if (lane == 0) atomicOr(err, kErrWait);
#pragma unroll
    for (int st = 0; st < S; ++st) {
      if (!mbar_try(bar[st], 0)) (void)mbar_wait_slow(bar[st], 1);
    }
  }
}

// Second kernel (more than one slice): y[n] = the slices of row n added in a fixed order.  8 warps per 32 rows: warp w
// adds the slices w, w + 8, ... (independent loads), warp 0 then adds the 8 partial sums in order.
constexpr int kFinWarps = 8;

__global__ void __launch_bounds__(kFinWarps * 32)
    block_lut_finish_kernel(const float* __restrict__ scratch, uint16_t* __restrict__ y, int64_t N, int slices) {
  __shared__ float part[kFinWarps][32];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t rows_pad = table_tiles(N) * 16;
  const int64_t n = (int64_t)blockIdx.x * 32 + lane;
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;");
  float a = 0.f;
  for (int s0 = warp; s0 < slices; s0 += 4 * kFinWarps) {
    float v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int s = s0 + u * kFinWarps;
      v[u] = (s < slices && n < rows_pad) ? __ldcg(scratch + (size_t)s * rows_pad + n) : 0.f;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) a += v[u];
  }
  part[warp][lane] = a;
  __syncthreads();
  if (warp != 0 || n >= N) return;
#pragma unroll
  for (int w = 1; w < kFinWarps; ++w) a += part[w][lane];
  y[n] = (uint16_t)float_to_bf16_bits(a);
}

// ---------------------------------------------------------------------------------------------------------------
// Layout conversion.  One thread per 32-bit word of the table: the first 128 words of a unit are index bytes, the
// rest scales (two per word).
// ---------------------------------------------------------------------------------------------------------------
template <int BITS>
__global__ void __launch_bounds__(256) block_table_pack_kernel(const uint8_t* __restrict__ wq,
                                                               const uint16_t* __restrict__ scales,
                                                               uint32_t* __restrict__ tab, int64_t N, int64_t K,
                                                               int64_t chunks, int64_t total_words) {
  constexpr int UW = btl_unit_bytes(BITS) / 4, BPC = btl_blocks_per_chunk(BITS);
  const int64_t row_bytes = K * BITS / 8, row_blocks = K / 64;
  int64_t w = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (; w < total_words; w += stride) {
    const int64_t unit = w / UW;
    const int uw = (int)(w % UW);
    const int64_t tile = unit / chunks, chunk = unit % chunks;
    uint32_t out = 0;
    if (uw < 128) {
      const int lane = uw >> 2;
      const int64_t n = tile * 16 + (lane >> 1);
#pragma unroll
      for (int bi = 0; bi < 4; ++bi) {
        const int64_t g = chunk * 32 + btl_group_of(lane, 4 * (uw & 3) + bi, BITS);
        if (n < N && g < row_bytes) out |= (uint32_t)wq[n * row_bytes + g] << (8 * bi);
      }
    } else {
#pragma unroll
      for (int hlf = 0; hlf < 2; ++hlf) {
        const int e = (uw - 128) * 2 + hlf;                 // scale number r * BPC + q of the unit
        const int64_t n = tile * 16 + e / BPC, blk = chunk * BPC + e % BPC;
        if (n < N && blk < row_blocks) out |= (uint32_t)scales[n * row_blocks + blk] << (16 * hlf);
      }
    }
    tab[w] = out;
  }
}

template <int BITS>
__global__ void __launch_bounds__(256) block_table_unpack_kernel(const uint8_t* __restrict__ tab,
                                                                 uint8_t* __restrict__ wq,
                                                                 uint16_t* __restrict__ scales, int64_t N, int64_t K,
                                                                 int64_t chunks) {
  const int64_t row_bytes = K * BITS / 8, row_blocks = K / 64;
  const int64_t total = N * row_bytes;
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (; i < total; i += stride) {
    const int64_t n = i / row_bytes, g = i % row_bytes;
    wq[i] = tab[btl_byte_offset(n, g, chunks, BITS)];
    if (g < row_blocks)
      scales[n * row_blocks + g] = *reinterpret_cast<const uint16_t*>(tab + btl_scale_offset(n, g, chunks, BITS));
  }
}

struct BlutPlan {
  int nl, slices, row_blocks, warps;
};

template <int BITS>
constexpr int blut_max_warps(int nl) {
  return nl == 1 ? BGeo<BITS, 1>::kWarps : nl == 2 ? BGeo<BITS, 2>::kWarps : nl == 3 ? BGeo<BITS, 3>::kWarps
                                                                                     : BGeo<BITS, 4>::kWarps;
}

// Chunks per slice: the choice that minimises the shared-memory work of the busiest CTA (table build: 256 cycles per
// chunk; lookups and their scale: about 20 cycles per tile and chunk) with all CTAs resident at once; then as many
// warps as give every warp the same number of tiles (at least 16: the table build needs them).
template <int BITS>
BlutPlan plan_blut(int64_t N, int64_t K, int sm_count) {
  const int64_t chunks = btl_chunks(K, BITS), tiles = table_tiles(N);
  BlutPlan best = {1, (int)chunks, 1, 16};
  double best_cost = 1e30;
  for (int nl = 1; nl <= 4; ++nl) {
    const int64_t slices = (chunks + nl - 1) / nl;
    int64_t rb = sm_count / slices;
    if (rb < 1) rb = 1;
    if (rb > tiles) rb = tiles;
    const int64_t tiles_cta = (tiles + rb - 1) / rb;
    const int64_t waves = (slices * rb + sm_count - 1) / sm_count;
    const int maxw = blut_max_warps<BITS>(nl);
    const int64_t tasks_warp = (tiles_cta + maxw - 1) / maxw;
    int64_t warps = (tiles_cta + tasks_warp - 1) / tasks_warp;
    if (warps < 16) warps = 16;
    const double cost = (double)waves * (256.0 * nl + 20.0 * nl * (double)(tasks_warp * warps) + 600.0) + 8.0 * slices;
    if (cost < best_cost) {
      best_cost = cost;
      best = {nl, (int)slices, (int)rb, (int)warps};
    }
  }
  return best;
}

template <int BITS, int NL>
cudaError_t launch_blut_one(const uint8_t* tab, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N, int64_t K,
                            const BlutPlan& p, float* scratch, unsigned int* err, cudaStream_t s) {
  using G = BGeo<BITS, NL>;
  constexpr int smem = (int)G::kHighEnd - 1024;   // dynamic shared memory starts at or below byte 1024 of the window
  if (cudaError_t e = cudaFuncSetAttribute(block_lut_kernel<BITS, NL>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem))
    return e;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(p.slices * p.row_blocks));
  cfg.blockDim = dim3((unsigned)(p.warps * 32));
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, block_lut_kernel<BITS, NL>, reinterpret_cast<const unsigned char*>(tab), cb, x,
                                     y, scratch, N, K, p.slices, p.row_blocks, err);
  if (e != cudaSuccess || p.slices == 1) return e;
  cudaLaunchConfig_t fin = {};
  fin.gridDim = dim3((unsigned)((N + 31) / 32));
  fin.blockDim = dim3(kFinWarps * 32);
  fin.stream = s;
  fin.attrs = attr;
  fin.numAttrs = 1;
  return cudaLaunchKernelEx(&fin, block_lut_finish_kernel, (const float*)scratch, y, N, p.slices);
}

template <int BITS>
cudaError_t launch_blut_bits(const uint8_t* tab, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N, int64_t K,
                             int64_t M, float* scratch, cudaStream_t s) {
  const DeviceInfo* di = device_info();
  if (!di) return cudaErrorInvalidDevice;
  const BlutPlan p = plan_blut<BITS>(N, K, di->sm_count);
  cudaError_t e = cudaSuccess;
  unsigned int* err = lut_error_word(&e);
  if (!err) return e;
  for (int64_t m = 0; m < M; ++m) {
    const uint16_t* xm = x + m * K;
    uint16_t* ym = y + m * N;
    switch (p.nl) {
      case 1: e = launch_blut_one<BITS, 1>(tab, cb, xm, ym, N, K, p, scratch, err, s); break;
      case 2: e = launch_blut_one<BITS, 2>(tab, cb, xm, ym, N, K, p, scratch, err, s); break;
      case 3: e = launch_blut_one<BITS, 3>(tab, cb, xm, ym, N, K, p, scratch, err, s); break;
      default: e = launch_blut_one<BITS, 4>(tab, cb, xm, ym, N, K, p, scratch, err, s); break;
    }
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

inline bool al16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

kmq_status check_table_shape(int64_t N, int64_t K, int bits, int64_t M) {
  if (bits != 1 && bits != 2 && bits != 4) return KMQ_ERR_BITS;
  if (N < 1 || M < 1 || K < 64 || (K % 64) != 0) return KMQ_ERR_SHAPE;
  if (N > (int64_t(1) << 31) || K > (int64_t(1) << 31) || M > (int64_t(1) << 24)) return KMQ_ERR_SHAPE;
  return KMQ_OK;
}

size_t blut_scratch_bytes(int64_t N, int64_t K, int bits) {
  const DeviceInfo* di = device_info();
  if (!di) return 0;
  const BlutPlan p = bits == 1 ? plan_blut<1>(N, K, di->sm_count)
                   : bits == 2 ? plan_blut<2>(N, K, di->sm_count)
                               : plan_blut<4>(N, K, di->sm_count);
  return p.slices == 1 ? 0 : (size_t)p.slices * (size_t)(table_tiles(N) * 16) * sizeof(float);
}

inline int grid_for_items(int64_t items, int sm_count) {
  int64_t blocks = (items + 255) / 256;
  const int64_t cap = (int64_t)sm_count * 16;
  if (blocks > cap) blocks = cap;
  return (int)(blocks < 1 ? 1 : blocks);
}

}  // namespace
}  // namespace kmq

using namespace kmq;

extern "C" {

size_t kmq_block_table_bytes(int64_t N, int64_t K, int bits) {
  if (check_table_shape(N, K, bits, 1) != KMQ_OK) return 0;
  return (size_t)btl_total_bytes(N, K, bits);
}

int64_t kmq_block_table_index_offset(int64_t n, int64_t k, int64_t N, int64_t K, int bits) {
  if (check_table_shape(N, K, bits, 1) != KMQ_OK || n < 0 || n >= N || k < 0 || k >= K) return -1;
  return btl_byte_offset(n, k / (8 / bits), btl_chunks(K, bits), bits);
}

int64_t kmq_block_table_scale_offset(int64_t n, int64_t k, int64_t N, int64_t K, int bits) {
  if (check_table_shape(N, K, bits, 1) != KMQ_OK || n < 0 || n >= N || k < 0 || k >= K) return -1;
  return btl_scale_offset(n, k / 64, btl_chunks(K, bits), bits);
}

kmq_status kmq_block_table_pack(const uint8_t* wq, const uint16_t* scales, int64_t N, int64_t K, int bits, uint8_t* table,
                                void* stream) {
  if (!wq || !scales || !table) return KMQ_ERR_NULL;
  if (kmq_status s = check_table_shape(N, K, bits, 1)) return s;
  if (!al16(wq) || !al16(scales) || !al16(table)) return KMQ_ERR_ALIGN;
  const DeviceInfo* di = device_info();
  if (!di) return KMQ_ERR_CUDA;
  const int64_t chunks = btl_chunks(K, bits), words = btl_total_bytes(N, K, bits) / 4;
  const int grid = grid_for_items(words, di->sm_count);
  cudaStream_t s = (cudaStream_t)stream;
  uint32_t* t32 = reinterpret_cast<uint32_t*>(table);
  if (bits == 1) block_table_pack_kernel<1><<<grid, 256, 0, s>>>(wq, scales, t32, N, K, chunks, words);
  else if (bits == 2) block_table_pack_kernel<2><<<grid, 256, 0, s>>>(wq, scales, t32, N, K, chunks, words);
  else block_table_pack_kernel<4><<<grid, 256, 0, s>>>(wq, scales, t32, N, K, chunks, words);
  return cudaGetLastError() == cudaSuccess ? KMQ_OK : KMQ_ERR_CUDA;
}

kmq_status kmq_block_table_unpack(const uint8_t* table, int64_t N, int64_t K, int bits, uint8_t* wq, uint16_t* scales,
                                  void* stream) {
  if (!wq || !scales || !table) return KMQ_ERR_NULL;
  if (kmq_status s = check_table_shape(N, K, bits, 1)) return s;
  if (!al16(wq) || !al16(scales) || !al16(table)) return KMQ_ERR_ALIGN;
  const DeviceInfo* di = device_info();
  if (!di) return KMQ_ERR_CUDA;
  const int64_t chunks = btl_chunks(K, bits);
  const int grid = grid_for_items(N * (K * bits / 8), di->sm_count);
  cudaStream_t s = (cudaStream_t)stream;
  if (bits == 1) block_table_unpack_kernel<1><<<grid, 256, 0, s>>>(table, wq, scales, N, K, chunks);
  else if (bits == 2) block_table_unpack_kernel<2><<<grid, 256, 0, s>>>(table, wq, scales, N, K, chunks);
  else block_table_unpack_kernel<4><<<grid, 256, 0, s>>>(table, wq, scales, N, K, chunks);
  return cudaGetLastError() == cudaSuccess ? KMQ_OK : KMQ_ERR_CUDA;
}

size_t kmq_block_table_workspace_bytes(int64_t N, int64_t K, int bits) {
  if (check_table_shape(N, K, bits, 1) != KMQ_OK) return 0;
  return blut_scratch_bytes(N, K, bits);
}

kmq_status kmq_block_table_linear(const uint8_t* table, const uint16_t* codebook, const uint16_t* x, uint16_t* y,
                                  int64_t N, int64_t K, int bits, int64_t M, void* workspace, size_t workspace_bytes,
                                  void* stream) {
  if (!table || !codebook || !x || !y) return KMQ_ERR_NULL;
  if (kmq_status s = check_table_shape(N, K, bits, M)) return s;
  if (!al16(table) || !al16(codebook) || !al16(x) || !al16(y)) return KMQ_ERR_ALIGN;
  const DeviceInfo* di = device_info();
  if (!di || di->max_smem_optin < 227 * 1024) return KMQ_ERR_CUDA;   // the tables take almost all of a 228 KB SM
  const size_t need = blut_scratch_bytes(N, K, bits);
  if (need > 0) {
    if (!workspace || workspace_bytes < need) return KMQ_ERR_WORKSPACE;
    if (!al16(workspace)) return KMQ_ERR_ALIGN;
  }
  cudaStream_t s = (cudaStream_t)stream;
  const cudaError_t e = bits == 1   ? launch_blut_bits<1>(table, codebook, x, y, N, K, M, (float*)workspace, s)
                        : bits == 2 ? launch_blut_bits<2>(table, codebook, x, y, N, K, M, (float*)workspace, s)
                                    : launch_blut_bits<4>(table, codebook, x, y, N, K, M, (float*)workspace, s);
  return e == cudaSuccess ? KMQ_OK : KMQ_ERR_CUDA;
}

}  // extern "C"
