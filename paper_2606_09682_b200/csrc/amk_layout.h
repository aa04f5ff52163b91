// Packed-weight geometry shared by the host packer and the device kernel.
//
// A matrix-vector product y = W x (W: [rows][K]) is split by rows across the persistent blocks; block
// `slot` owns a contiguous run of "units" (1 row, or 2 rows where rows must stay together).  Inside a
// block the rows are processed in passes of at most kPassRows rows.  In a pass the consumer warps form
// a Wr x Wk grid: row-warp wr owns G <= 16 consecutive rows (one m16 tensor-core tile), k-warp wk owns
// every Wk-th column block (64 columns for bf16; 128 for the integer dtypes = one quantisation group; an int8 matrix
// whose K is 64 short of a multiple of 128 gets its last block filled up with zero codes).  The bytes of a pass are
// stored block-major: for column block b, the work units (b, wr = 0..Wr-1) one after another.  A work
// unit -- the rows of one row-warp in one column block -- is contiguous, and a ring tile is a run of
// `upt` consecutive units, so each block's weight stream is a sequence of contiguous byte runs that one
// producer thread fetches with bulk copies, never waiting on a data dependency.
//
// Inside a unit the bytes are ordered for ldmatrix: 16-byte chunk c (8 bf16 / 16 int8 / 32 int4 codes
// along K) of row r sits at (c * rows + r) * 16, so the eight rows of an 8x8 matrix are 128 contiguous
// bytes (no bank conflicts).  The k order inside a block is permuted (col_of_k) so that the activation
// values one lane feeds to the tensor core -- its B fragments for every k step of the block -- are
// contiguous in the natural column order.  An int4 / grouped-int8 unit ends with {fp16 scale, 16-bit zero point
// (0 for grouped int8)} per row (its block is one group).
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define AMK_HD __host__ __device__ __forceinline__
#else
#define AMK_HD inline
#endif

namespace amk {

constexpr int kConsumerWarps = 11;            // consumer warps per block (+1 producer warp = 384 threads, 168 registers each)
constexpr int kThreads = 32 * (kConsumerWarps + 1);
constexpr int kConsumerThreads = 32 * kConsumerWarps;
constexpr int kGMax = 16;                     // rows per row-warp: one m16n8 tile
constexpr int kPassRows = kConsumerWarps * kGMax;
constexpr int kMaxStages = 16;
constexpr int kMaxRep = 16;                   // q heads per kv head
constexpr int kAttnMinChunk = 32;             // fewest cache positions per split-K chunk
constexpr int kMaxChunks = 64;
constexpr int kChunkCap = 24;                 // chunks per kv group: beyond this the exchange and the combine of the partials cost
                                              // more than the shorter chunks save (TinyLlama shape, position 1024: 33 -> 22
                                              // chunks, 584 -> 579 us; 18 and 12 chunks measured slower again)

enum OpKind : int { OP_QKV = 0, OP_O = 1, OP_GATEUP = 2, OP_DOWN = 3, OP_LMHEAD = 4 };
enum WDtype : int { W_BF16 = 0, W_INT8 = 1, W_INT4 = 2, W_INT8G = 3 };
AMK_HD constexpr bool grouped(int wdtype) { return wdtype == W_INT4 || wdtype == W_INT8G; }   // scales inside the units

AMK_HD int ceil_div(int a, int b) { return (a + b - 1) / b; }

AMK_HD constexpr int block_cols(int wdtype) { return wdtype == W_BF16 ? 64 : 128; }   // columns per column block
AMK_HD int block_chunks(int wdtype) { return wdtype == W_INT4 ? 4 : 8; }           // 16-byte chunks per row per block
// bytes of a work unit holding `rows` rows (grouped: codes, then 4 bytes {scale, zero} per row, padded to 16)
AMK_HD int unit_bytes(int wdtype, int rows) {
  if (wdtype == W_BF16) return rows * 128;
  if (wdtype == W_INT8) return rows * 128;
  if (wdtype == W_INT8G) return (rows * 132 + 15) & ~15;
  return (rows * 68 + 15) & ~15;
}

// Logical k index inside a block (what the tensor-core fragments see) -> natural column inside the block.
// Lane-quad q of a warp supplies, for k step s (bf16 k16, int8 k32, int4: k32 after nibble expansion) and
// fragment half h, the values j; its whole supply for a block is the contiguous column run starting at
// q * (block_cols / 4).
//   bf16: k = 16 s + 8 h + 2 q + j  (s<4, h<2, q<4, j<2)  ->  col 16 q + 4 s + 2 h + j
//   int8, int4, grouped int8: k = 32 s + 16 h + 4 q + j (s<4, h<2, q<4, j<4)  ->  col 32 q + 8 s + 4 h + j
AMK_HD int col_of_k(int wdtype, int k) {
  if (wdtype == W_BF16) {
    const int s = k >> 4, h = (k >> 3) & 1, q = (k >> 1) & 3, j = k & 1;
    return 16 * q + 4 * s + 2 * h + j;
  }
  const int s = k >> 5, h = (k >> 4) & 1, q = (k >> 2) & 3, j = k & 3;
  return 32 * q + 8 * s + 4 * h + j;
}

// Where logical k of a row is stored inside its unit: the 16-byte chunk, and the element inside the chunk
// (bf16: 2-byte element; int8: byte; int4: nibble, low nibble of a byte first).
//   bf16 / int8 / grouped int8: k-major.   int4: one ldmatrix word (8 nibbles) of chunk 2 (s >> 1) + h expands into the
//   fragment registers of k steps s = 2x (even nibbles) and s = 2x + 1 (odd nibbles).
AMK_HD void place_of_k(int wdtype, int k, int* chunk, int* elem) {
  if (wdtype == W_BF16) { *chunk = k >> 3; *elem = k & 7; return; }
  if (wdtype == W_INT8 || wdtype == W_INT8G) { *chunk = k >> 4; *elem = k & 15; return; }
  const int s = k >> 5, h = (k >> 4) & 1, q = (k >> 2) & 3, j = k & 3;
  *chunk = 2 * (s >> 1) + h;
  *elem = 8 * q + 2 * j + (s & 1);
}

// Rows owned by slot s.  The split of an op's units over the slots is a table: bounds[s] .. bounds[s+1] are
// slot s's units (n_slots + 1 entries, bounds[0] = 0, bounds[n_slots] = units).  The host builds it in
// proportion to what each SM was measured to stream, so that all blocks finish an op together.
struct Slice { int row0; int rows; };
AMK_HD Slice slot_slice(const int* bounds, int unit_rows, int s) {
  Slice r; r.row0 = bounds[s] * unit_rows; r.rows = (bounds[s + 1] - bounds[s]) * unit_rows;
  return r;
}
// Inverse: which slot owns a row (the last slot whose first unit is not beyond the row's unit).
AMK_HD int slot_of_row(const int* bounds, int unit_rows, int n_slots, int row) {
  const int u = row / unit_rows;
  int lo = 0, hi = n_slots - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (bounds[mid] <= u) lo = mid; else hi = mid - 1;
  }
  return lo;
}
// (host only) Unit boundaries for `units` units over n_slots slots with relative weights w (nullptr: equal shares).
inline void make_bounds(int units, int n_slots, const double* w, int* bounds) {
  double total = 0.0;
  for (int s = 0; s < n_slots; s++) total += w ? w[s] : 1.0;
  double cum = 0.0;
  bounds[0] = 0;
  for (int s = 0; s < n_slots; s++) {
    cum += w ? w[s] : 1.0;
    int b = (int)(units * (cum / total) + 0.5);
    if (b < bounds[s]) b = bounds[s];
    if (b > units) b = units;
    bounds[s + 1] = b;
  }
  bounds[n_slots] = units;
}

// Geometry of one pass of R rows over K columns.
struct PassGeom {
  int R;        // rows in the pass
  int G;        // rows per row-warp (the last row-warp has g_last)
  int g_last;
  int Wr;       // row-warps
  int Wk;       // k-warps
  int nblk;     // column blocks
  int n_units;  // Wr * nblk work units, ordered (b, wr)
  int upt;      // work units per ring tile
  int n_tiles;
  int ub_full;  // bytes of a unit of G rows
  int ub_last;  // bytes of the last row-warp's unit
  int bb;       // bytes of one column block = (Wr - 1) * ub_full + ub_last
};

AMK_HD PassGeom pass_geom(int R, int K, int wdtype, int stage_bytes) {
  PassGeom g;
  g.R = R;
  // fewest row-warps that keep G <= kGMax; if at most half the warps are needed, several k-warps share a
  // row group and the row-warps are spread over what the k split leaves; otherwise every warp is a row-warp.
  const int wr_min = ceil_div(R, kGMax);
  int wr;
  if (2 * wr_min > kConsumerWarps) wr = kConsumerWarps;
  else wr = kConsumerWarps / (kConsumerWarps / wr_min);
  const int G = ceil_div(R, wr);
  g.G = G;
  g.Wr = ceil_div(R, G);
  g.g_last = R - (g.Wr - 1) * G;
  g.Wk = kConsumerWarps / g.Wr;
  g.nblk = ceil_div(K, block_cols(wdtype));
  if (g.Wk > g.nblk) g.Wk = g.nblk;
  g.n_units = g.Wr * g.nblk;
  g.ub_full = unit_bytes(wdtype, G);
  g.ub_last = unit_bytes(wdtype, g.g_last);
  g.bb = (g.Wr - 1) * g.ub_full + g.ub_last;
  g.upt = stage_bytes / g.ub_full;
  if (g.upt < 1) g.upt = 1;
  g.n_tiles = ceil_div(g.n_units, g.upt);
  return g;
}

// Byte offset of work unit (column block b, row-warp r) from the start of the pass.
AMK_HD int64_t unit_off_br(const PassGeom& g, int b, int r) { return (int64_t)b * g.bb + (int64_t)r * g.ub_full; }
AMK_HD int64_t pass_bytes(const PassGeom& g) { return (int64_t)g.nblk * g.bb; }
// Byte offset of work unit u (= b * Wr + r); u >= n_units gives the pass size.
AMK_HD int64_t unit_off(const PassGeom& g, int u) {
  if (u >= g.n_units) return pass_bytes(g);
  int b = u / g.Wr;
  return unit_off_br(g, b, u - b * g.Wr);
}

AMK_HD int n_passes(int rows) { return ceil_div(rows, kPassRows); }
AMK_HD int pass_rows(int rows, int p) { int left = rows - p * kPassRows; return left < kPassRows ? left : kPassRows; }

// Packed bytes of a slice of `rows` rows.
AMK_HD int64_t slice_bytes(int rows, int K, int wdtype, int stage_bytes) {
  int64_t t = 0;
  for (int p = 0; p < n_passes(rows); p++) t += pass_bytes(pass_geom(pass_rows(rows, p), K, wdtype, stage_bytes));
  return t;
}

// Split-K plan of the attention over positions [0, n_pos): chunk length and count.
AMK_HD void attn_chunks(int n_pos, int n_blocks, int n_kv, int* chunk_len, int* n_chunks) {
  int cmax = n_blocks / n_kv;
  if (cmax > kMaxChunks) cmax = kMaxChunks;
  if (cmax > kChunkCap) cmax = kChunkCap;
  if (cmax < 1) cmax = 1;
  int lc = ceil_div(n_pos, cmax);
  if (lc < kAttnMinChunk) lc = kAttnMinChunk;
  *chunk_len = lc;
  *n_chunks = ceil_div(n_pos, lc);
}

// One matrix-vector product kind of a model (the same for every layer).
struct OpShape {
  int32_t K, rows, unit_rows, wdtype;
};

}  // namespace amk
