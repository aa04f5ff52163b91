"""Independent decision procedure for the tables a decode step runs from (test infrastructure only).

The library's static check (amk_plan_check, after the paper's validate(), Section 4, Table 2) is judged
against this file the way the paper judges its validator against an independent oracle (Section 5, "Validator
soundness"): every tampered table this oracle finds unsafe must be rejected, every real table accepted.  It
shares no code with the library: the packed layout is restated here from its description, and the dependency
model is decided by brute force -- an explicit graph of (task, block) events for a few blocks and plain
reachability -- instead of the checker's rule about all-to-all joins.

is_safe(words, model) -> (bool, reason).  `model` is a dict with hidden, n_layers, n_q_heads, n_kv_heads,
head_dim, mlp, vocab, wdtype (0 bf16, 1 int8, 2 int4, 3 grouped int8), stage_bytes, n_blocks, and optionally lm_wdtype (the LM
head's dtype when it is quantised like the layers; 0 otherwise).
"""
from collections import deque

MAGIC = 0x314E414C504B4D41
WARPS, GMAX = 11, 16                 # consumer warps per block; rows per row-warp (one m16 tile)
PASS_ROWS = WARPS * GMAX
# buffers of the dependency model
XA, QKV, O, XB, M, KVROW, OUT, MAXB, PART = 1, 2, 4, 8, 16, 32, 64, 128, 256


def _cdiv(a, b):
    return -(-a // b)


def _unit_bytes(wd, rows):
    """A work unit = the rows of one row-warp over one column block (64 columns for bf16; 128 for the integer dtypes,
    an int8 matrix's last block zero-filled when K is 64 short of a multiple of 128)."""
    if wd == 0:
        return rows * 128                      # 64 bf16
    if wd == 1:
        return rows * 128                      # 128 int8
    if wd == 3:
        return (rows * 132 + 15) // 16 * 16    # 128 int8 + {fp16 scale, pad} per row, padded to 16 bytes
    return (rows * 68 + 15) // 16 * 16         # 128 nibbles + {scale, zero} fp16 per row, padded to 16 bytes


def _pass_tiles(rows, k, wd, stage):
    """[(offset in the pass, bytes)] of the ring tiles of one pass of `rows` rows, and the pass size.
    Row groups of at most 16 rows; as few row-warps as that allows, unless more than half the warps are needed,
    in which case all; units ordered (column block, row-warp); a tile holds stage // (bytes of a full unit)
    consecutive units."""
    wr_min = _cdiv(rows, GMAX)
    wr = WARPS if 2 * wr_min > WARPS else WARPS // (WARPS // wr_min)
    g = _cdiv(rows, wr)
    wr = _cdiv(rows, g)
    g_last = rows - (wr - 1) * g
    nblk = _cdiv(k, 64 if wd == 0 else 128)
    ub, ubl = _unit_bytes(wd, g), _unit_bytes(wd, g_last)
    block_bytes = (wr - 1) * ub + ubl
    n_units = wr * nblk
    upt = max(1, stage // ub)

    def off(u):
        if u >= n_units:
            return nblk * block_bytes
        b, r = divmod(u, wr)
        return b * block_bytes + r * ub
    tiles = []
    for t in range(_cdiv(n_units, upt)):
        o0, o1 = off(t * upt), off((t + 1) * upt)
        tiles.append((o0, o1 - o0))
    return tiles, nblk * block_bytes


def _slice_tiles(rows, k, wd, stage):
    out, base = [], 0
    for p in range(_cdiv(rows, PASS_ROWS)):
        r = min(PASS_ROWS, rows - p * PASS_ROWS)
        tiles, size = _pass_tiles(r, k, wd, stage)
        out += [(base + o, n) for o, n in tiles]
        base += size
    return out, base


def _schedule_safe(rows):
    """Brute force over an explicit event graph: 3 blocks, 3 layer cycles + head.  A task that does not run on
    every block runs on one, a different one each layer and for each task kind (nothing may be assumed about
    which blocks two such tasks share).  Nodes: (task index, block).  Edges: program order on a block; writer(block b')
    -> reader(block b) for every buffer the reader reads whole (b' over the writer's participants), and
    writer(b) -> reader(b) for buffers it reads in part (its own rows)."""
    if len(rows) != 6:
        return False, "schedule rows"
    nb, cycles = 3, 3
    seq = []
    for cyc in range(cycles):
        for r in range(5):
            seq.append((rows[r], cyc))
    seq.append((rows[5], cycles))
    for i, (row, _) in enumerate(seq):
        if row[0] != (i % 5 if i < 5 * cycles else 5):
            return False, "task kinds out of place"

    def parts(i):
        row, cyc = seq[i]
        return list(range(nb)) if (row[3] & 1) else [(cyc + row[0]) % nb]
    n = len(seq)
    succ = {(i, b): set() for i in range(n) for b in range(nb)}
    for b in range(nb):
        mine = [i for i in range(n) if b in parts(i)]
        for a, c in zip(mine, mine[1:]):
            succ[(a, b)].add((c, b))
    last_writer = {}
    reads_of = {}          # buffer -> [(reader task, version = writer task)]
    for i, (row, _) in enumerate(seq):
        reads, writes, full = row[1], row[2], row[3] >> 8
        if full & ~reads:
            return False, "reads whole what it does not read"
        for buf in (XA, QKV, O, XB, M, MAXB, PART):
            if not reads & buf:
                continue
            w = i if (buf == PART and writes & buf) else last_writer.get(buf)
            if w is None:
                if buf == XA:
                    continue                   # the embedding row: enters from outside
                return False, f"task {i} waits for buffer {buf} nobody wrote"
            reads_of.setdefault(buf, []).append((i, w))
            if w != i:
                for b in parts(i):
                    srcs = parts(w) if (full & buf) else ([b] if b in parts(w) else parts(w))
                    for bw in srcs:
                        succ[(w, bw)].add((i, b))
        for buf in (XA, QKV, O, XB, M, MAXB, PART):
            if writes & buf:
                last_writer[buf] = i
    if not seq[-1][0][2] & OUT:
        return False, "no output"

    def reach(src, dst):
        seen, dq = {src}, deque([src])
        while dq:
            u = dq.popleft()
            if u == dst:
                return True
            for v in succ[u]:
                if v not in seen:
                    seen.add(v)
                    dq.append(v)
        return False
    # an overwrite must come after every read of the previous version, on every pair of blocks
    writers = {}
    for i, (row, _) in enumerate(seq):
        for buf in (XA, QKV, O, XB, M, MAXB, PART):
            if row[2] & buf:
                writers.setdefault(buf, []).append(i)
    for buf, ws in writers.items():
        for w_prev, w_next in zip(ws, ws[1:]):
            for (r, ver) in reads_of.get(buf, []):
                if ver != w_prev or r >= w_next:
                    continue
                for br in parts(r):
                    for bw in parts(w_next):
                        if not reach((r, br), (w_next, bw)):
                            return False, f"task {w_next} may overwrite buffer {buf} under task {r}"
    return True, ""


def is_safe(words, model):
    w = [int(x) for x in words]
    if len(w) < 8 or w[0] != MAGIC:
        return False, "magic"
    nb, L, n_ops, stage, wbytes, n_tiles, n_sched = w[1:8]
    if nb != model["n_blocks"] or L != model["n_layers"] or n_ops != 4 * L + 1 or stage != model["stage_bytes"]:
        return False, "header"
    if n_sched > 64 or len(w) != 8 + n_ops * 8 + 5 * (nb + 1) + (nb + 1) + n_tiles + n_sched * 4:
        return False, "length"
    p = 8
    ops = [w[p + 8 * i: p + 8 * i + 8] for i in range(n_ops)]
    p += 8 * n_ops
    bounds = [w[p + k * (nb + 1): p + (k + 1) * (nb + 1)] for k in range(5)]
    p += 5 * (nb + 1)
    tbeg = w[p: p + nb + 1]
    p += nb + 1
    tiles = w[p: p + n_tiles]
    p += n_tiles
    sched = [tuple(w[p + 4 * i: p + 4 * i + 4]) for i in range(n_sched)]

    H, I, V, wd = model["hidden"], model["mlp"], model["vocab"], model["wdtype"]
    qd, kvd = model["n_q_heads"] * model["head_dim"], model["n_kv_heads"] * model["head_dim"]
    # (the LM head is bf16 unless the model says it is quantised like the layers)
    shape = [(H, qd + 2 * kvd, 1, wd), (qd, H, 1, wd), (H, 2 * I, 2, wd), (I, H, 1, wd), (H, V, 1, model.get("lm_wdtype", 0))]
    # every row of every GEMV: exactly one producer
    for k in range(5):
        units = shape[k][1] // shape[k][2]
        b = bounds[k]
        if b[0] != 0 or b[nb] != units or any(b[s + 1] < b[s] for s in range(nb)):
            return False, f"bounds of kind {k}"
    if tbeg[0] != 0 or tbeg[nb] != n_tiles or any(tbeg[s + 1] < tbeg[s] for s in range(nb)):
        return False, "tile index"
    # what each block's consumers will wait for, op by op, against what its producer will issue
    expect = [[] for _ in range(nb)]
    covered_end = 0
    for i, op in enumerate(ops):
        kind = 4 if i == n_ops - 1 else i % 4
        layer = i // 4
        K, rows, ur, dt = shape[kind]
        if op[:6] != [kind, layer, K, rows, ur, dt]:
            return False, f"op {i}"
        off, nbytes = op[6], op[7]
        if off < covered_end or off % 16 or off + nbytes > wbytes:
            return False, f"region of op {i}"
        covered_end = off + nbytes
        task = 5 * L if kind == 4 else 5 * layer + (0 if kind == 0 else kind + 1)
        pos = off
        for s in range(nb):
            srows = (bounds[kind][s + 1] - bounds[kind][s]) * ur
            tl, size = _slice_tiles(srows, K, dt, stage)
            for o, n in tl:
                if n <= 0 or n > stage or n % 16 or (pos + o) % 16 or pos + o + n > wbytes:
                    return False, "tile shape"
                expect[s].append((pos + o, n, task))
            pos += size
            if kind == 0:
                expect[s].append((0, 0, 5 * layer + 1))        # attention marker
        if pos - off != nbytes:
            return False, f"region size of op {i}"
    for s in range(nb):
        got = []
        for e in tiles[tbeg[s]: tbeg[s + 1]]:
            nby = ((e >> 40) & 0x1FFF) << 4
            got.append((((e & ((1 << 40) - 1)) << 4) if nby else 0, nby, e >> 53))
        if got != expect[s]:
            return False, f"queue of block {s}"
    return _schedule_safe(sched)
