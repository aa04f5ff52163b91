// Packed-weight geometry shared by the host packer and the device kernel.
//
// A matrix-vector product y = W x (W: [rows][K]) is split by rows across the persistent blocks; block
// `slot` owns a contiguous run of "units" (1 row, or 2 rows where rows must stay together).  Inside a
// block the rows are processed in passes of at most kPassRows rows.  In a pass the consumer warps form
// a W_r x W_k grid: row-warp wr owns G consecutive rows, k-warp wk owns every W_k-th 256-column block.
// The bytes of a pass are stored block-major: for column block b, rows 0..R-1, each row's 256 columns
// (the last block may be narrower).  A "work unit" (b, wr) -- G rows of one column block -- is therefore
// contiguous, and a ring tile is a run of consecutive work units, so each block's whole weight stream is
// one contiguous byte range that a single producer thread can fetch with bulk copies, never waiting on
// a data dependency.
//
// Column order inside a 256-column block of width Wd: lane l (< Wd/8) holds columns
// {4l..4l+3} and {Wd/2 + 4l .. Wd/2 + 4l + 3}, so its activation reads are two conflict-free 16-byte
// shared-memory loads and, for int4 (Wd = 256, groups of 128), its first four codes belong to group 2b
// and its last four to group 2b+1.
//
// Bytes per row per full column block: bf16 512, int8 256, int4 128 + 8 (fp16 scale and zero point of
// its two groups follow the 128 code bytes of the same row).
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define AMK_HD __host__ __device__ __forceinline__
#else
#define AMK_HD inline
#endif

namespace amk {

constexpr int kConsumerWarps = 15;            // consumer warps per block (+1 producer warp = 512 threads)
constexpr int kThreads = 32 * (kConsumerWarps + 1);
constexpr int kConsumerThreads = 32 * kConsumerWarps;
constexpr int kGMax = 8;                      // rows per row-warp
constexpr int kPassRows = kConsumerWarps * kGMax;
constexpr int kBlockCols = 256;               // columns per column block
constexpr int kMaxStages = 16;
constexpr int kMaxRep = 16;                   // q heads per kv head
constexpr int kAttnMinChunk = 32;             // fewest cache positions per split-K chunk
constexpr int kMaxChunks = 64;

enum OpKind : int { OP_QKV = 0, OP_O = 1, OP_GATEUP = 2, OP_DOWN = 3, OP_LMHEAD = 4 };
enum WDtype : int { W_BF16 = 0, W_INT8 = 1, W_INT4 = 2 };

// One matrix-vector product of the step.  Lives in device memory (table built by amk_create).
struct OpDesc {
  int32_t kind;          // OpKind
  int32_t layer;
  int32_t K;             // input length
  int32_t rows;          // output rows (virtual rows: QKV = q|k|v rows, GATEUP = g0,u0,g1,u1,...)
  int32_t unit_rows;     // rows per ownership unit (1, or 2)
  int32_t wdtype;        // WDtype of this op (LM head is always bf16)
  int32_t rot;           // slot rotation: block c takes slot (c + rot) % n_blocks
  int32_t pad;
  uint64_t packed_off;   // byte offset of this op's region in the packed buffer
  uint64_t scale_off;    // int8: byte offset of the fp16 row scales (virtual row order); else 0
};

AMK_HD int ceil_div(int a, int b) { return (a + b - 1) / b; }

// bytes of one row inside a column block of width wd
AMK_HD int rowchunk_bytes(int wdtype, int wd) {
  return wdtype == W_BF16 ? wd * 2 : (wdtype == W_INT8 ? wd : (wd / 2 + 8 * (wd / kBlockCols)));
}
AMK_HD int64_t row_bytes(int wdtype, int K) {
  int nbf = K / kBlockCols, tail = K % kBlockCols;
  return (int64_t)nbf * rowchunk_bytes(wdtype, kBlockCols) + (tail ? rowchunk_bytes(wdtype, tail) : 0);
}

// Rows owned by slot s: units are dealt as evenly as possible, the first (units % n) slots get one more.
struct Slice { int row0; int rows; };
AMK_HD Slice slot_slice(int total_rows, int unit_rows, int n_slots, int s) {
  int units = total_rows / unit_rows;
  int q = units / n_slots, rem = units % n_slots;
  int u0 = s * q + (s < rem ? s : rem);
  int nu = q + (s < rem ? 1 : 0);
  Slice r; r.row0 = u0 * unit_rows; r.rows = nu * unit_rows;
  return r;
}
// Inverse: which slot owns a row.
AMK_HD int slot_of_row(int total_rows, int unit_rows, int n_slots, int row) {
  int units = total_rows / unit_rows;
  int q = units / n_slots, rem = units % n_slots;
  int u = row / unit_rows;
  int big = rem * (q + 1);
  if (u < big) return u / (q + 1);
  return q ? rem + (u - big) / q : n_slots - 1;
}

// Geometry of one pass of R rows over K columns.
struct PassGeom {
  int R;        // rows in the pass
  int G;        // rows per row-warp (the last row-warp may have fewer)
  int Wr;       // row-warps
  int Wk;       // k-warps
  int nblk;     // column blocks (the last may be narrower)
  int tail;     // width of the last block if narrower than 256, else 0
  int n_units;  // Wr * nblk work units
  int upt;      // work units per ring tile
  int n_tiles;
  int rc_full;  // bytes of one row in a full block
  int rc_tail;  // bytes of one row in the tail block
};

AMK_HD PassGeom pass_geom(int R, int K, int wdtype, int stage_bytes) {
  PassGeom g;
  g.R = R;
  const int galign = (wdtype == W_INT4) ? 2 : 1;     // int4 row chunks are 136 B: keep unit offsets 16-byte aligned
  // fewest row-warps that keep G <= kGMax; if at most half the warps are needed, several k-warps share a
  // row group and the row-warps are spread over what the k split leaves; otherwise every warp is a row-warp.
  const int wr_min = ceil_div(R, kGMax);
  int wr;
  if (2 * wr_min > kConsumerWarps) wr = kConsumerWarps;
  else wr = kConsumerWarps / (kConsumerWarps / wr_min);
  int G = ceil_div(R, wr);
  G = ceil_div(G, galign) * galign;
  if (G > kGMax) G = kGMax;
  g.G = G;
  g.Wr = ceil_div(R, G);
  g.Wk = kConsumerWarps / g.Wr;
  g.nblk = ceil_div(K, kBlockCols);
  g.tail = K % kBlockCols;
  if (g.Wk > g.nblk) g.Wk = g.nblk;
  g.n_units = g.Wr * g.nblk;
  g.rc_full = rowchunk_bytes(wdtype, kBlockCols);
  g.rc_tail = g.tail ? rowchunk_bytes(wdtype, g.tail) : g.rc_full;
  int ub = G * g.rc_full;
  g.upt = stage_bytes / ub;
  if (g.upt < 1) g.upt = 1;
  g.n_tiles = ceil_div(g.n_units, g.upt);
  return g;
}

// Byte offset of work unit (column block b, row-warp r) from the start of the pass.
AMK_HD int64_t unit_off_br(const PassGeom& g, int b, int r) {
  int rc = (g.tail && b == g.nblk - 1) ? g.rc_tail : g.rc_full;
  return (int64_t)b * g.R * g.rc_full + (int64_t)r * g.G * rc;   // every block before b is full
}
// Total bytes of the pass.
AMK_HD int64_t pass_bytes(const PassGeom& g) {
  int nbf = g.nblk - (g.tail ? 1 : 0);
  return (int64_t)nbf * g.R * g.rc_full + (g.tail ? (int64_t)g.R * g.rc_tail : 0);
}
// Byte offset of work unit u (= b * Wr + r); u == n_units gives the pass size.
AMK_HD int64_t unit_off(const PassGeom& g, int u) {
  if (u >= g.n_units) return pass_bytes(g);
  int b = u / g.Wr;
  return unit_off_br(g, b, u - b * g.Wr);
}

// Number of passes for a slice of `rows` rows and the rows of pass p.
AMK_HD int n_passes(int rows) { return ceil_div(rows, kPassRows); }
AMK_HD int pass_rows(int rows, int p) { int left = rows - p * kPassRows; return left < kPassRows ? left : kPassRows; }

// Column held at element e (0..7) of lane l in a block of width wd.
AMK_HD int lane_col(int wd, int lane, int e) { return (e < 4) ? 4 * lane + e : wd / 2 + 4 * lane + (e - 4); }

// Split-K plan of the attention over positions [0, n_pos): chunk length and count.
AMK_HD void attn_chunks(int n_pos, int n_blocks, int n_kv, int* chunk_len, int* n_chunks) {
  int cmax = n_blocks / n_kv;
  if (cmax > kMaxChunks) cmax = kMaxChunks;
  if (cmax < 1) cmax = 1;
  int lc = ceil_div(n_pos, cmax);
  if (lc < kAttnMinChunk) lc = kAttnMinChunk;
  *chunk_len = lc;
  *n_chunks = ceil_div(n_pos, lc);
}

}  // namespace amk
