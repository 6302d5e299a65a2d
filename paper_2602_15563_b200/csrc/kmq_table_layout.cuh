// KMQ_LAYOUT_TABLE: the packed layout read by the activation-table kernel (b = 1, 2; b = 4 is stored as in the
// tuned layout).
//
// The index bits are stored as bit planes, one byte per group of 8 consecutive weights of a row: bit t of the byte
// of plane p, row n, group g is bit p of idx[n, 8g + t].  Rows are grouped in tiles of 16 and a row's groups in
// chunks of 32 (256 weights); plane p of chunk c of tile T is one contiguous 512-byte unit at byte offset
//   ((T * chunks + c) * bits + p) * 512,          chunks = ceil(K / 256),
// so a tile's whole K range is contiguous.  Inside a unit, lane L = 2 * (n % 16) + (g % 2) of a warp owns the 16
// bytes [16 L, 16 L + 16): byte i of lane (a, r) = (L & 1, L >> 1) holds group  a + 2 * ((r + i) % 16)  of the
// chunk.  The rotation by the row makes the 32 lanes of a warp address 32 different groups at every step i, which is
// what keeps the kernel's table lookups free of shared-memory bank conflicts.  Rows beyond N and groups beyond K are
// zero padding.
#pragma once
#include <stdint.h>

namespace kmq {

constexpr int kTableChunkK = 256;     // weights of one row per chunk
constexpr int kTableUnitBytes = 512;  // one plane of one chunk of one 16-row tile

__host__ __device__ inline int64_t table_chunks(int64_t K) { return (K + kTableChunkK - 1) / kTableChunkK; }
__host__ __device__ inline int64_t table_tiles(int64_t N) { return (N + 15) >> 4; }
__host__ __device__ inline int64_t table_total_bytes(int64_t N, int64_t K, int bits) {
  return table_tiles(N) * table_chunks(K) * bits * kTableUnitBytes;
}

// Byte offset of the byte that holds plane `plane` of weights 8g .. 8g+7 of row n (g = k / 8).
__host__ __device__ inline int64_t table_byte_offset(int64_t n, int64_t g, int plane, int64_t chunks, int bits) {
  const int64_t tile = n >> 4, chunk = g >> 5;
  const int r = (int)(n & 15), gl = (int)(g & 31);
  const int a = gl & 1, t = gl >> 1;
  const int lane = 2 * r + a, i = (t - r) & 15;
  return ((tile * chunks + chunk) * bits + plane) * kTableUnitBytes + lane * 16 + i;
}

// Inverse, inside a unit: byte `i` of lane `lane` -> row within the tile and group within the chunk.
__host__ __device__ inline void table_unit_coords(int lane, int i, int& row_in_tile, int& group_in_chunk) {
  const int a = lane & 1, r = lane >> 1;
  row_in_tile = r;
  group_in_chunk = a + 2 * ((r + i) & 15);
}

// ---------------------------------------------------------------------------------------------------------------
// Block-format table layout: what the activation-table kernel of the paper's block format reads (b = 1, 2, 4).
//
// A group is one byte of the packed indices (8 / bits consecutive weights, fields LSB first), a chunk 32 groups of a
// row (256 / bits weights = 4 / bits blocks of 64), a tile 16 rows.  Chunk c of tile T is one contiguous unit of
//   512 + 32 * (4 / bits)  bytes  at byte offset  (T * chunks + c) * unit_bytes,     chunks = ceil(K / (256 / bits)):
// 512 index bytes, then the bf16 scales of the unit's blocks, scale[row r][block q of the chunk] at byte
// 512 + (r * (4 / bits) + q) * 2.  Lane L = 2 r + a of a warp owns the index bytes [16 L, 16 L + 16).  With
// S = 4 * bits (bytes of a lane per block), r = r_hi * S + r_lo, byte i = S * j + f of the lane holds group
//   (8 * bits) * ((j + r_hi) % (4 / bits))  +  a  +  2 * ((f + r_lo) % S)
// of the chunk: at every step i the 32 lanes address 32 different groups (no shared-memory bank conflicts in the
// table lookups), and S consecutive steps of a lane stay inside one block, so that the block's scale is applied once
// per S lookups.  Rows beyond N and groups beyond K hold zero bytes and zero scales.
// ---------------------------------------------------------------------------------------------------------------
__host__ __device__ constexpr int btl_blocks_per_chunk(int bits) { return 4 / bits; }
__host__ __device__ constexpr int btl_unit_bytes(int bits) { return 512 + 32 * (4 / bits); }
__host__ __device__ constexpr int btl_chunk_k(int bits) { return 256 / bits; }
__host__ __device__ inline int64_t btl_chunks(int64_t K, int bits) {
  return (K + btl_chunk_k(bits) - 1) / btl_chunk_k(bits);
}
__host__ __device__ inline int64_t btl_total_bytes(int64_t N, int64_t K, int bits) {
  return table_tiles(N) * btl_chunks(K, bits) * btl_unit_bytes(bits);
}

// Group (0..31) of the chunk held by byte i of lane `lane`, and the block (0 .. 4/bits - 1) it lies in.
__host__ __device__ inline int btl_group_of(int lane, int i, int bits) {
  const int S = 4 * bits, bpc = 4 / bits;
  const int a = lane & 1, r = lane >> 1, r_hi = r / S, r_lo = r % S, j = i / S, f = i % S;
  return (8 * bits) * ((j + r_hi) % bpc) + a + 2 * ((f + r_lo) % S);
}

// Byte offset of the index byte of group g (= k / (8 / bits)) of row n.
__host__ __device__ inline int64_t btl_byte_offset(int64_t n, int64_t g, int64_t chunks, int bits) {
  const int S = 4 * bits, bpc = 4 / bits;
  const int64_t tile = n >> 4, chunk = g >> 5;
  const int r = (int)(n & 15), gl = (int)(g & 31);
  const int q = gl / (8 * bits), w = gl % (8 * bits), a = w & 1, m = w >> 1;
  const int r_hi = r / S, r_lo = r % S;
  const int j = (q - r_hi + bpc) % bpc, f = (m - r_lo + S) % S;
  return (tile * chunks + chunk) * btl_unit_bytes(bits) + (2 * r + a) * 16 + S * j + f;
}

// Byte offset of the bf16 scale of block `blk` (= k / 64) of row n.
__host__ __device__ inline int64_t btl_scale_offset(int64_t n, int64_t blk, int64_t chunks, int bits) {
  const int bpc = 4 / bits;
  return ((n >> 4) * chunks + blk / bpc) * btl_unit_bytes(bits) + 512 + ((n & 15) * bpc + blk % bpc) * 2;
}

}  // namespace kmq
