// kmq_linear on the tuned (tile-major) layout for batches of 16 rows and more: the 5th-generation tensor core
// (tcgen05.mma, accumulator in tensor memory) multiplies dequantised bf16 weight tiles with the activations.
//
// One CTA owns 128 output rows = 8 tiles of 16; warp w decodes tile w.  K is walked in stages of 128 weights per
// row.  Per stage
//   * every lane rebuilds 2 x 32 weights (rows r and r + 8 of its tile, r = lane % 8, 16-byte chunk t = lane / 8
//     of the step) as bf16 and stores them, 8 weights per 128-bit store, into the A buffer of the stage in the
//     K-major core-matrix layout the tensor core reads: 8 rows x 16 bytes contiguous, the next 8 weights of the same
//     rows kLBO bytes further, the next 8 rows kSBO bytes further (a quarter warp fills one core matrix, so the
//     stores have no bank conflicts);
//   * the activations under the stage (NB batch rows, zero-filled past M and past K) are copied global -> shared
//     with cp.async into the B buffer in the same layout;
//   * after a CTA barrier one thread issues 8 tcgen05.mma (128 x NB x 16 each) that add into the accumulator
//     D[128 output rows][NB batch rows] in tensor memory, and commits them to the mbarrier of the buffer.
// Two buffers: the warps decode stage i + 1 while the tensor core works on stage i.  At the end the accumulator is read
// with tcgen05.ld (lane = output row, column = batch row), rounded to bf16 and stored.
//
// Inside a stage the order of the weights of a row is (chunk t, then the 32 weights of this stage in the chunk);
// A and B use the same order, and a sum does not depend on the order of its terms.
//
// Every wait on an mbarrier is bounded; when it runs out the CTA stops, sets bit 0 of the device error word, frees its
// tensor memory and returns.
#include "kmq_common.cuh"
#include "kmq_linear_variants.cuh"
#include "kmq_mma_common.cuh"

namespace kmq {

__device__ unsigned int g_device_error_flags = 0;   // sticky; read and cleared by kmq_device_error_flags()

namespace {

constexpr int kBlockRows = 128;                          // rows of the MMA (UMMA M)
constexpr int kStageK = 128;                             // weights of a row per stage
constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kLBO = 128;                                // bytes between core matrices that are neighbours in K
constexpr int kSBO = (kStageK / 8) * kLBO;               // bytes between groups of 8 rows
constexpr int kAStageBytes = kBlockRows * kStageK * 2;   // 32 KB
constexpr int kKSlices = kStageK / 16;                   // MMAs per stage
constexpr uint32_t kWaitLimit = 1u << 20;                // polls of an mbarrier (about 20 ns apart) before giving up

template <int BITS>
struct UGeo {
  static constexpr int kWordK = 32 / BITS;
  static constexpr int kStepK = 512 / BITS;                    // weights of a row per 1 KB step of a tile
  static constexpr int kChunkK = kStepK / 4;                   // weights under one 16-byte chunk
  static constexpr int kStagesPerStep = kStepK / kStageK;      // 1, 2, 4 for b = 4, 2, 1
  static constexpr int kTableBytes = BITS == 4 ? kWarps * 2 * 16 * 128 : 0;   // b = 4: [tile][half][entry][lane]
};

template <int BITS, int NB>
struct USmem {
  static constexpr int kBStageBytes = NB * kStageK * 2;
  static constexpr int kA = 0;
  static constexpr int kB = 2 * kAStageBytes;
  static constexpr int kTables = kB + 2 * kBStageBytes;
  static constexpr int kBars = kTables + UGeo<BITS>::kTableBytes;   // two mbarriers, then the tensor-memory address
  static constexpr int kTotal = kBars + 32;
};

// Shared-memory matrix descriptor: K-major, no swizzle, strides kLBO / kSBO, descriptor version of sm_100.
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(kLBO >> 4) << 16) | ((uint64_t)(kSBO >> 4) << 32) |
         ((uint64_t)1 << 46);
}

// Instruction descriptor of kind::f16: D fp32, A and B bf16, both K-major, M = 128, N = NB.
template <int NB>
__device__ __forceinline__ uint32_t instr_desc() {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NB >> 3) << 17) | ((uint32_t)(kBlockRows >> 4) << 24);
}

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      :
      : "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void async_proxy_fence() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void cp_async16(uint32_t smem_dst, const void* gmem_src, bool valid) {
  const int bytes = valid ? 16 : 0;   // 0 source bytes: the 16 destination bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_dst), "l"(gmem_src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
  asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
}

// Bounded wait for the phase of parity `parity` of an mbarrier.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < kWaitLimit; ++i) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    if (done) return true;
    __nanosleep(20);
  }
  return false;
}

// Per-row decode state of a lane: rows r (h = 0) and r + 8 (h = 1) of its tile.
template <int BITS>
struct RowState;
template <>
struct RowState<2> {
  Dec2 d;
  __device__ __forceinline__ void init(const uint16_t* cb_row, const unsigned char*, int) { d.init(cb_row); }
};
template <>
struct RowState<1> {
  uint32_t base, diff;   // (c0, c0) and (c0 ^ c1, c0 ^ c1)
  __device__ __forceinline__ void init(const uint16_t* cb_row, const unsigned char*, int) {
    const uint32_t c = __ldg(reinterpret_cast<const uint32_t*>(cb_row));
    base = prmt(c, c, 0x1010u);
    diff = base ^ prmt(c, c, 0x3232u);
  }
};
template <>
struct RowState<4> {
  const unsigned char* tab;   // this lane's bank of the [entry][lane] table of its tile half
  __device__ __forceinline__ void init(const uint16_t*, const unsigned char* table_half, int lane) {
    tab = table_half + lane * 4;
  }
};

// The 32 weights of stage U (of its step) in one lane's chunk `v` of one row -> four 128-bit stores of 8 bf16 each,
// kLBO bytes apart.
template <int BITS, int U>
__device__ __forceinline__ void decode_store(const uint4& v, const RowState<BITS>& st, unsigned char* dst) {
  const uint32_t w4[4] = {v.x, v.y, v.z, v.w};
  if constexpr (BITS == 4) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint32_t e[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {   // nibble i -> byte offset nibble * 128 of the lane's table bank
        const int sh = 4 * i - 7;
        const uint32_t u = sh < 0 ? (w4[j] << -sh) : (w4[j] >> sh);
        e[i] = *reinterpret_cast<const uint32_t*>(st.tab + (u & 0x780u));
      }
      *reinterpret_cast<uint4*>(dst + j * kLBO) = make_uint4(prmt(e[0], e[1], 0x7610u), prmt(e[2], e[3], 0x7610u),
                                                             prmt(e[4], e[5], 0x7610u), prmt(e[6], e[7], 0x7610u));
    }
  } else if constexpr (BITS == 2) {
#pragma unroll
    for (int jj = 0; jj < 2; ++jj) {
      const uint32_t w = w4[2 * U + jj];
      uint32_t a[8];
#pragma unroll
      for (int q = 0; q < 4; ++q) st.d.pair(w, q, a[2 * q], a[2 * q + 1]);   // weights 4q .. 4q + 3
      *reinterpret_cast<uint4*>(dst + (2 * jj) * kLBO) = make_uint4(a[0], a[1], a[2], a[3]);
      *reinterpret_cast<uint4*>(dst + (2 * jj + 1) * kLBO) = make_uint4(a[4], a[5], a[6], a[7]);
    }
  } else {
    const uint32_t w = w4[U];
#pragma unroll
    for (int kg = 0; kg < 4; ++kg) {
      uint32_t a[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        // shift c puts weights (2c, 2c + 1) on bits 15 and 31; PRMT in sign-replicate mode turns them into
        // 16-bit masks; masked XOR picks c0 or c1 bit-exactly
        const uint32_t sh = w * kPow2[4 * kg + i];
        const uint32_t sel = prmt(sh, sh, 0xBB99u);
        asm("lop3.b32 %0, %1, %2, %3, 0x6A;" : "=r"(a[i]) : "r"(sel), "r"(st.diff), "r"(st.base));
      }
      *reinterpret_cast<uint4*>(dst + kg * kLBO) = make_uint4(a[0], a[1], a[2], a[3]);
    }
  }
}

template <int BITS, int NB>
__global__ void __launch_bounds__(kThreads, 1) linear_umma_kernel(const uint32_t* __restrict__ packed,
                                                                  const uint16_t* __restrict__ cb,
                                                                  const uint16_t* __restrict__ x,
                                                                  uint16_t* __restrict__ y, int64_t N, int64_t K,
                                                                  int M) {
  using G = UGeo<BITS>;
  using SM = USmem<BITS, NB>;
  constexpr int SPS = G::kStagesPerStep;
  constexpr uint32_t kTmemCols = NB <= 32 ? 32 : 64;   // a power of two >= 32
  extern __shared__ __align__(128) unsigned char smem_raw[];
  unsigned char* const a_buf = smem_raw + SM::kA;
  unsigned char* const tables = smem_raw + SM::kTables;
  const uint32_t smem_base = (uint32_t)__cvta_generic_to_shared(smem_raw);
  const uint32_t a_addr = smem_base + SM::kA, b_addr = smem_base + SM::kB, bar_addr = smem_base + SM::kBars;
  volatile uint32_t* const tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_raw + SM::kBars + 16);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = lane & 7, t = lane >> 3;
  const int64_t tiles = (N + kTileRows - 1) / kTileRows;
  const int64_t tile_id = (int64_t)blockIdx.x * kWarps + warp;
  const bool has_tile = tile_id < tiles;   // warp-uniform; a warp without a tile leaves its A rows as they are
  const int64_t row0 = tile_id * kTileRows;
  const int chunks = (int)(K / (4 * G::kWordK));
  const int steps = (chunks + 3) >> 2;
  // step s of the tile: 64 16-byte units, unit h * 32 + row * 4 + chunk holds chunk `chunk` of row (row + 8h)
  const uint4* __restrict__ tile =
      reinterpret_cast<const uint4*>(packed) + (has_tile ? tile_id : 0) * (int64_t)steps * 64 + r * 4 + t;

  // ---- set-up: mbarriers, tensor memory, decode state ----
  if (threadIdx.x == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_addr) : "memory");
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_addr + 8) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(bar_addr + 16), "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if constexpr (BITS == 4) {
    // word [tile][half][entry e][lane] = (C_row[e], C_row[e]), row = 16 tile + 8 half + lane % 8
    for (int i = threadIdx.x; i < kWarps * 2 * 16 * 32; i += kThreads) {
      const int ln = i & 31, e = (i >> 5) & 15, half = (i >> 9) & 1, tl = i >> 10;
      const int64_t row = min(((int64_t)blockIdx.x * kWarps + tl) * kTileRows + 8 * half + (ln & 7), N - 1);
      const uint32_t c = __ldg(cb + row * 16 + e);
      reinterpret_cast<uint32_t*>(tables)[i] = c | (c << 16);
    }
  }
  RowState<BITS> st0, st1;
  st0.init(cb + min(row0 + r, N - 1) * (1 << BITS), tables + (warp * 2 + 0) * 2048, lane);
  st1.init(cb + min(row0 + r + 8, N - 1) * (1 << BITS), tables + (warp * 2 + 1) * 2048, lane);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_d = *tmem_slot;

  // this lane's 16-byte slots in an A buffer: row group 2 warp + h, core matrices 4t .. 4t + 3, row r
  unsigned char* const a_lane = a_buf + (2 * warp) * kSBO + (4 * t) * kLBO + r * 16;
  const uint32_t idesc = instr_desc<NB>();

  uint4 na = make_uint4(0, 0, 0, 0), nb = na;
  if (has_tile && steps > 0) {
    na = ldg_stream_u4(tile);
    nb = ldg_stream_u4(tile + 32);
  }
  int stage = 0;
  bool ok = true;
  for (int s = 0; s < steps && ok; ++s) {
    const uint4 va = na, vb = nb;
    if (has_tile && s + 1 < steps) {
      na = ldg_stream_u4(tile + (int64_t)(s + 1) * 64);
      nb = ldg_stream_u4(tile + (int64_t)(s + 1) * 64 + 32);
    }
#pragma unroll
    for (int u = 0; u < SPS; ++u) {
      if (!ok) break;
      const int buf = stage & 1;
      if (stage >= 2) {   // the MMAs that read this buffer two stages ago are done
        ok = mbar_wait(bar_addr + 8 * buf, ((stage >> 1) - 1) & 1);
        ok = __syncthreads_and(ok);
        if (!ok) break;
      }
      // activations: piece p = (batch row m, core matrix kg); bits of p: kg0 | m0..2 | kg1..3 | m3..
#pragma unroll
      for (int i = 0; i < NB / 16; ++i) {
        const int p = threadIdx.x + kThreads * i;
        const int kg = (p & 1) | ((p >> 3) & 14), m = ((p >> 1) & 7) | ((p >> 7) << 3);
        const int64_t k = (int64_t)s * G::kStepK + (kg >> 2) * G::kChunkK + u * 32 + (kg & 3) * 8;
        const bool valid = m < M && k < K;
        cp_async16(b_addr + buf * SM::kBStageBytes + (m >> 3) * kSBO + kg * kLBO + (m & 7) * 16,
                   x + (valid ? (int64_t)m * K + k : 0), valid);
      }
      if (has_tile) {
        unsigned char* const dst = a_lane + buf * kAStageBytes;
        if (u == 0) { decode_store<BITS, 0>(va, st0, dst); decode_store<BITS, 0>(vb, st1, dst + kSBO); }
        if (SPS > 1 && u == 1) { decode_store<BITS, 1 % SPS>(va, st0, dst); decode_store<BITS, 1 % SPS>(vb, st1, dst + kSBO); }
        if (SPS > 2 && u == 2) { decode_store<BITS, 2 % SPS>(va, st0, dst); decode_store<BITS, 2 % SPS>(vb, st1, dst + kSBO); }
        if (SPS > 2 && u == 3) { decode_store<BITS, 3 % SPS>(va, st0, dst); decode_store<BITS, 3 % SPS>(vb, st1, dst + kSBO); }
      }
      cp_async_wait_all();
      async_proxy_fence();   // the stores above become visible to the tensor core's reads of shared memory
      __syncthreads();
      if (threadIdx.x == 0) {
        tc_fence_after_sync();
#pragma unroll
        for (int ks = 0; ks < kKSlices; ++ks)
          umma_bf16(tmem_d, smem_desc(a_addr + buf * kAStageBytes + ks * 2 * kLBO),
                    smem_desc(b_addr + buf * SM::kBStageBytes + ks * 2 * kLBO), idesc, (stage | ks) != 0);
        umma_commit(bar_addr + 8 * buf);
      }
      ++stage;
    }
  }
  // ---- all MMAs done -> read the accumulator, round, store ----
  if (ok && stage > 0) {
    const int last = stage - 1;
    ok = mbar_wait(bar_addr + 8 * (last & 1), (last >> 1) & 1);
    ok = __syncthreads_and(ok);
  }
  if (ok) {
    tc_fence_after_sync();
    const int q = warp & 3, half = warp >> 2;   // a warp reads the 32 lanes of its quarter; the two halves split the columns
    const int64_t n = (int64_t)blockIdx.x * kBlockRows + q * 32 + lane;
#pragma unroll
    for (int c0 = 0; c0 < NB / 2; c0 += 8) {
      const int col = half * (NB / 2) + c0;
      uint32_t v[8];
      if (stage > 0) {
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                     : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                     : "r"(tmem_d + ((uint32_t)(q * 32) << 16) + col));
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = 0;
      }
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (col + j < M && n < N) y[(int64_t)(col + j) * N + n] = (uint16_t)float_to_bf16_bits(__uint_as_float(v[j]));
    }
  } else if (threadIdx.x == 0) {
    atomicOr(&g_device_error_flags, 1u);
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(kTmemCols) : "memory");
}


}  // namespace

namespace {

template <int BITS, int NB>
cudaError_t launch_nb(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N, int64_t K,
                      int M, cudaStream_t s) {
  constexpr int smem = USmem<BITS, NB>::kTotal;
  static bool configured[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(linear_umma_kernel<BITS, NB>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  const unsigned grid = (unsigned)((N + kBlockRows - 1) / kBlockRows);
  linear_umma_kernel<BITS, NB><<<grid, kThreads, smem, s>>>(packed, cb, x, y, N, K, M);
  return cudaGetLastError();
}

template <int BITS>
cudaError_t launch_bits(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
                        int64_t K, int M, cudaStream_t s) {
  if (M <= 16) return launch_nb<BITS, 16>(packed, cb, x, y, N, K, M, s);
  if (M <= 32) return launch_nb<BITS, 32>(packed, cb, x, y, N, K, M, s);
  if (M <= 48) return launch_nb<BITS, 48>(packed, cb, x, y, N, K, M, s);
  return launch_nb<BITS, 64>(packed, cb, x, y, N, K, M, s);
}

}  // namespace

#ifndef KMQ_UMMA_MIN_ROWS
#define KMQ_UMMA_MIN_ROWS (1 << 30)   // not selected yet: correct, but slower than the multi-tile kernel
#endif
int linear_umma_min_rows() { return KMQ_UMMA_MIN_ROWS; }
int linear_umma_rows_per_launch() { return 64; }

cudaError_t launch_linear_umma(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
                               int64_t K, int bits, int64_t M, cudaStream_t s) {
  const int64_t per = linear_umma_rows_per_launch();
  for (int64_t m0 = 0; m0 < M; m0 += per) {
    const int mc = (int)(M - m0 < per ? M - m0 : per);
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

// Reads and clears the device error word (synchronises the device).
cudaError_t read_device_error_flags(unsigned int* flags) {
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return e;
  e = cudaMemcpyFromSymbol(flags, g_device_error_flags, sizeof(unsigned int));
  if (e != cudaSuccess) return e;
  const unsigned int zero = 0;
  return cudaMemcpyToSymbol(g_device_error_flags, &zero, sizeof(unsigned int));
}


}  // namespace kmq
