// Host-side exhaustive check of the packed-weight geometry (amk_layout.h): for one op it replays what the
// packer writes, what the producer copies and what every consumer warp reads, and verifies that
//   * every (row, column) of the matrix is read exactly once, with the activation index it belongs to,
//   * every ring tile is 16-byte aligned, fits the stage, and tiles are contiguous and cover the slice,
//   * every work unit a consumer warp touches lies inside the tile it waits for.
// Usage: layout_check rows K wdtype unit_rows n_blocks stage_bytes   -> prints "ok" or a diagnostic.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <vector>

#include "amk_layout.h"
using namespace amk;

int main(int argc, char** argv) {
  if (argc < 7) return 2;
  const int rows = atoi(argv[1]), K = atoi(argv[2]), wd = atoi(argv[3]), unit_rows = atoi(argv[4]);
  const int N = atoi(argv[5]), stage = atoi(argv[6]);
  const int64_t rb = row_bytes(wd, K);
  const int64_t total = (int64_t)rows * rb;
  // packer: for each element, the byte offset (and nibble for int4) where it lands; record owner (row, col)
  // granularity: one entry per 8-element lane chunk start offset -> (row, c0, c1)
  std::vector<int> seen((size_t)rows * K, 0);
  std::vector<unsigned char> owner_mark((size_t)total, 0);
  int64_t covered = 0;
  for (int slot = 0; slot < N; slot++) {
    const Slice sl = slot_slice(rows, unit_rows, N, slot);
    for (int r = sl.row0; r < sl.row0 + sl.rows; r++)
      if (slot_of_row(rows, unit_rows, N, r) != slot) { printf("slot_of_row mismatch row %d\n", r); return 1; }
    const int64_t base = (int64_t)sl.row0 * rb;
    const int np = n_passes(sl.rows);
    int64_t slice_bytes = 0;
    for (int ps = 0; ps < np; ps++) {
      const int R = pass_rows(sl.rows, ps);
      const PassGeom g = pass_geom(R, K, wd, stage);
      if (g.G < 1 || g.G > kGMax || g.Wr * g.Wk > kConsumerWarps || g.Wr < 1 || g.Wk < 1) { printf("bad geom R=%d G=%d Wr=%d Wk=%d\n", R, g.G, g.Wr, g.Wk); return 1; }
      if ((g.Wr - 1) * g.G >= R || g.Wr * g.G < R) { printf("row split wrong R=%d G=%d Wr=%d\n", R, g.G, g.Wr); return 1; }
      const int64_t pbase = base + (int64_t)ps * kPassRows * rb;
      if (pass_bytes(g) != (int64_t)R * rb) { printf("pass bytes %lld != %lld\n", (long long)pass_bytes(g), (long long)R * rb); return 1; }
      // producer tiles
      int64_t prev_end = 0;
      for (int t = 0; t < g.n_tiles; t++) {
        const int u0 = t * g.upt;
        const int64_t o0 = unit_off(g, u0), o1 = unit_off(g, u0 + g.upt);
        if (o0 != prev_end) { printf("tile gap\n"); return 1; }
        if ((o1 - o0) > stage || (o1 - o0) <= 0 || ((pbase + o0) & 15) || ((o1 - o0) & 15)) {
          printf("tile size/alignment: R=%d K=%d t=%d o0=%lld o1=%lld\n", R, K, t, (long long)o0, (long long)o1); return 1;
        }
        prev_end = o1;
      }
      if (prev_end != pass_bytes(g)) { printf("tiles do not cover the pass\n"); return 1; }
      slice_bytes += prev_end;
      // consumers
      for (int warp = 0; warp < kConsumerWarps; warp++) {
        const int wr = warp % g.Wr, wk = warp / g.Wr;
        if (wk >= g.Wk) continue;
        const int my_rows = (g.R - wr * g.G) < g.G ? (g.R - wr * g.G) : g.G;
        for (int t = 0; t < g.n_tiles; t++) {
          const int u0 = t * g.upt, u1 = (u0 + g.upt < g.n_units) ? u0 + g.upt : g.n_units;
          const int64_t t0 = unit_off(g, u0), t1 = unit_off(g, u0 + g.upt);
          int b = (u0 > wr) ? (u0 - wr + g.Wr - 1) / g.Wr : 0;
          b += ((wk - b) % g.Wk + g.Wk) % g.Wk;
          for (; b * g.Wr + wr < u1; b += g.Wk) {
            const bool is_tail = g.tail && (b == g.nblk - 1);
            const int wdt = is_tail ? g.tail : kBlockCols;
            const int rc = is_tail ? g.rc_tail : g.rc_full;
            const int64_t uo = unit_off_br(g, b, wr);
            if (uo < t0 || uo + (int64_t)my_rows * rc > t1) { printf("unit outside its tile\n"); return 1; }
            for (int i = 0; i < my_rows; i++) {
              const int row = sl.row0 + ps * kPassRows + wr * g.G + i;
              for (int lane = 0; lane < wdt / 8; lane++) {
                const int64_t off = pbase + uo + (int64_t)i * rc + lane * (wd == W_BF16 ? 16 : (wd == W_INT8 ? 8 : 4));
                if (off < 0 || off >= total) { printf("offset out of range\n"); return 1; }
                if (owner_mark[off]) { printf("byte read twice: off %lld\n", (long long)off); return 1; }
                owner_mark[off] = 1;
                for (int e = 0; e < 8; e++) {
                  const int col = b * kBlockCols + lane_col(wdt, lane, e);
                  if (col >= K) { printf("column out of range\n"); return 1; }
                  seen[(size_t)row * K + col]++;
                }
              }
            }
          }
        }
      }
    }
    if (slice_bytes != (int64_t)sl.rows * rb) { printf("slice bytes mismatch\n"); return 1; }
    covered += sl.rows;
  }
  if (covered != rows) { printf("rows covered %lld of %d\n", (long long)covered, rows); return 1; }
  for (size_t i = 0; i < seen.size(); i++)
    if (seen[i] != 1) { printf("element (%zu,%zu) read %d times\n", i / K, i % K, seen[i]); return 1; }
  printf("ok\n");
  return 0;
}
