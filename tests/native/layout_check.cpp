// Host-side exhaustive check of the packed-weight geometry (amk_layout.h): for one op it replays where the
// packer puts every weight, what the producer copies and which work units every consumer warp reads, and
// verifies that
//   * every (row, column) of the matrix lands in exactly one place, and every stored element is read by
//     exactly one warp (its row group, its column blocks),
//   * inside a block, logical k -> (chunk, element) and logical k -> natural column are bijections, and the
//     columns one lane quad supplies to the tensor core for a block are one contiguous run,
//   * every ring tile is 16-byte aligned, fits the stage, and the tiles of a pass are contiguous and cover it,
//   * every work unit a consumer warp touches lies inside the tile it waits for.
// Usage: layout_check rows K wdtype unit_rows n_blocks stage_bytes [skew]  -> prints "ok" or a diagnostic.
// skew > 0 gives the slots unequal weights (1 + skew * (slot % 7) / 7), as a measured-bandwidth split would.
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
  const double skew = argc > 7 ? atof(argv[7]) : 0.0;
  std::vector<double> wts(N);
  for (int i = 0; i < N; i++) wts[i] = 1.0 + skew * (i % 7) / 7.0;
  std::vector<int> bounds(N + 1);
  make_bounds(rows / unit_rows, N, wts.data(), bounds.data());
  if (bounds[0] != 0 || bounds[N] != rows / unit_rows) { printf("bad bounds\n"); return 1; }
  const int bc = block_cols(wd), cpb = block_chunks(wd);
  const int epc = bc / cpb;                     // elements per 16-byte chunk
  if (K % bc && !(wd == W_INT8 && K % bc == 64)) { printf("K not a multiple of the column block\n"); return 1; }
  // the in-block permutation
  {
    std::vector<int> col_seen(bc, 0), place_seen(bc, 0);
    for (int k = 0; k < bc; k++) {
      int ch, el;
      place_of_k(wd, k, &ch, &el);
      const int col = col_of_k(wd, k);
      if (col < 0 || col >= bc || ch < 0 || ch >= cpb || el < 0 || el >= epc) { printf("k map out of range\n"); return 1; }
      col_seen[col]++;
      place_seen[ch * epc + el]++;
    }
    for (int i = 0; i < bc; i++) if (col_seen[i] != 1 || place_seen[i] != 1) { printf("k map not a bijection\n"); return 1; }
    // lane quad q supplies, for every step and half, consecutive columns starting at q * bc / 4
    const int per_q = bc / 4, jn = (wd == W_BF16) ? 2 : 4, kstep = (wd == W_BF16) ? 16 : 32;
    for (int k = 0; k < bc; k++) {
      const int q = (wd == W_BF16) ? ((k >> 1) & 3) : ((k >> 2) & 3);
      const int s = k / kstep, h = (k / (kstep / 2)) & 1, j = k % jn;
      const int expect = q * per_q + (s * 2 + h) * jn + j;
      if (col_of_k(wd, k) != expect) { printf("lane supply not contiguous at k=%d\n", k); return 1; }
    }
  }
  std::vector<int> seen((size_t)rows * K, 0);
  long long covered = 0;
  for (int slot = 0; slot < N; slot++) {
    const Slice sl = slot_slice(bounds.data(), unit_rows, slot);
    for (int r = sl.row0; r < sl.row0 + sl.rows; r++)
      if (slot_of_row(bounds.data(), unit_rows, N, r) != slot) { printf("slot_of_row mismatch row %d\n", r); return 1; }
    const int np = n_passes(sl.rows);
    long long sbytes = 0;
    for (int ps = 0; ps < np; ps++) {
      const int R = pass_rows(sl.rows, ps);
      const PassGeom g = pass_geom(R, K, wd, stage);
      if (g.G < 1 || g.G > kGMax || g.Wr * g.Wk > kConsumerWarps || g.Wr < 1 || g.Wk < 1 || g.g_last < 1 || g.g_last > g.G ||
          (g.Wr - 1) * g.G + g.g_last != R) {
        printf("bad geom R=%d G=%d g_last=%d Wr=%d Wk=%d\n", R, g.G, g.g_last, g.Wr, g.Wk);
        return 1;
      }
      std::vector<unsigned char> mark((size_t)pass_bytes(g), 0);
      // producer tiles
      long long prev_end = 0;
      for (int t = 0; t < g.n_tiles; t++) {
        const long long o0 = unit_off(g, t * g.upt), o1 = unit_off(g, (t + 1) * g.upt);
        if (o0 != prev_end) { printf("tile gap\n"); return 1; }
        if ((o1 - o0) > stage || (o1 - o0) <= 0 || ((sbytes + o0) & 15) || ((o1 - o0) & 15)) {
          printf("tile size/alignment: R=%d K=%d t=%d o0=%lld o1=%lld\n", R, K, t, o0, o1);
          return 1;
        }
        prev_end = o1;
      }
      if (prev_end != pass_bytes(g)) { printf("tiles do not cover the pass\n"); return 1; }
      // consumers: the incremental walk of the kernel
      for (int warp = 0; warp < kConsumerWarps; warp++) {
        const int wr = warp % g.Wr, wk = warp / g.Wr;
        if (wk >= g.Wk) continue;
        const int urows = (wr == g.Wr - 1) ? g.g_last : g.G;
        int next_b = wk, t_b = 0, t_r = 0;
        const int step_b = g.upt / g.Wr, step_r = g.upt - step_b * g.Wr;
        for (int t = 0; t < g.n_tiles; t++) {
          const long long tile_off = (long long)t_b * g.bb + (long long)t_r * g.ub_full;
          if (tile_off != unit_off(g, t * g.upt)) { printf("tile walk drifted\n"); return 1; }
          const long long tile_end = unit_off(g, (t + 1) * g.upt);
          int n_b = t_b + step_b, n_r = t_r + step_r;
          if (n_r >= g.Wr) { n_r -= g.Wr; n_b++; }
          while (next_b < g.nblk && (next_b < n_b || (next_b == n_b && wr < n_r))) {
            const long long uo = (long long)next_b * g.bb + (long long)wr * g.ub_full;
            if (uo < tile_off || uo + unit_bytes(wd, urows) > tile_end) { printf("unit outside its tile\n"); return 1; }
            // every element of the unit: row i, chunk c, element e  ->  (row, column)
            for (int i = 0; i < urows; i++) {
              const int row = sl.row0 + ps * kPassRows + wr * g.G + i;
              for (int k = 0; k < bc; k++) {
                int ch, el;
                place_of_k(wd, k, &ch, &el);
                const long long byte = uo + ((long long)ch * urows + i) * 16 + (wd == W_BF16 ? el * 2 : (wd == W_INT4 ? el / 2 : el));
                if (byte >= (long long)mark.size()) { printf("element outside the pass\n"); return 1; }
                mark[byte] = 1;
                if (wd == W_BF16) mark[byte + 1] = 1;
                if (next_b * bc + col_of_k(wd, k) >= K) continue;         // (zero fill of an int8 matrix's half-full last block)
                seen[(size_t)row * K + (size_t)next_b * bc + col_of_k(wd, k)]++;
              }
              if (grouped(wd)) {
                const long long sz = uo + (long long)urows * (wd == W_INT4 ? 64 : 128) + i * 4;
                for (int e = 0; e < 4; e++) mark[sz + e] = 1;
              }
            }
            next_b += g.Wk;
          }
          t_b = n_b;
          t_r = n_r;
        }
        if (next_b < g.nblk) { printf("a warp did not reach all its blocks\n"); return 1; }
      }
      // every byte except unit padding is used
      long long used = 0;
      for (unsigned char m : mark) used += m;
      const long long expect = (long long)R * g.nblk * (wd == W_INT4 ? 68 : (wd == W_INT8G ? 132 : 128));
      if (used != expect) { printf("bytes used %lld, expected %lld\n", used, expect); return 1; }
      sbytes += pass_bytes(g);
    }
    if (sbytes != slice_bytes(sl.rows, K, wd, stage)) { printf("slice bytes mismatch\n"); return 1; }
    covered += sl.rows;
  }
  if (covered != rows) { printf("rows covered %lld of %d\n", covered, rows); return 1; }
  for (size_t i = 0; i < seen.size(); i++)
    if (seen[i] != 1) { printf("element (%zu,%zu) read %d times\n", i / K, i % K, seen[i]); return 1; }
  printf("ok\n");
  return 0;
}
