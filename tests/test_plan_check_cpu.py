"""The static check of the tables a step runs from (amk_plan_check; the paper's validate(), Section 4, Table 2)
against an independent brute-force oracle, the way the paper measures its validator (Section 5, "Validator
soundness"): real plans are accepted by both; tampered plans of several unsafe classes -- the paper's cycle /
drop-wait / out-of-bounds / capacity classes restated for ring-tile queues, row bounds and the dependency model
-- that the oracle finds unsafe must all be rejected (no false accept), and whatever the oracle finds safe must
be accepted (no false reject).  CPU only: neither side touches a GPU."""
import numpy as np
import pytest

from oracle import plan_oracle
from paper_2606_09682_b200 import binding as amk
from paper_2606_09682_b200 import inputs as inp

WD = {"bf16": 0, "int8": 1, "int4": 2, "int8g": 3}
CASES = [("mini", "bf16", 148), ("mini_ragged", "int8", 132), ("mini_hd128", "int4", 7), ("mini_wide", "int4", 148),
         ("tinyllama_1b", "int8", 148), ("smollm2_135m", "bf16", 148), ("llama3_8b", "bf16", 148),
         ("mini_wide", "int8g", 148), ("tinyllama_1b", "int8g", 148)]
QHEAD_CASES = [("mini_ragged", "int8", 132), ("mini_wide", "int4", 148), ("tinyllama_1b", "int8", 148),
               ("mini_hd128", "int8g", 148)]


def _plan(name, wdtype, n_blocks, **kw):
    shape = inp.SHAPES[name]
    cfg = amk.make_config(shape, wdtype, n_blocks=n_blocks, **kw)
    words = amk.amk_plan_export(cfg)
    model = dict(hidden=shape.hidden, n_layers=shape.n_layers, n_q_heads=shape.n_q_heads, n_kv_heads=shape.n_kv_heads,
                 head_dim=shape.head_dim, mlp=shape.mlp, vocab=shape.vocab, wdtype=WD[wdtype],
                 stage_bytes=int(words[4]), n_blocks=n_blocks,
                 lm_wdtype=WD[wdtype] if kw.get("quantize_lm_head") else 0)
    return cfg, words, model


def _sections(words):
    nb, n_ops, n_tiles, n_sched = int(words[1]), int(words[3]), int(words[6]), int(words[7])
    ops = 8
    bounds = ops + 8 * n_ops
    tbeg = bounds + 5 * (nb + 1)
    tiles = tbeg + nb + 1
    sched = tiles + n_tiles
    return dict(nb=nb, n_ops=n_ops, n_tiles=n_tiles, ops=ops, bounds=bounds, tbeg=tbeg, tiles=tiles, sched=sched)


@pytest.mark.parametrize("name,wdtype,n_blocks", CASES)
def test_real_plans_are_accepted_by_checker_and_oracle(name, wdtype, n_blocks):
    cfg, words, model = _plan(name, wdtype, n_blocks)
    st, why = amk.amk_plan_check(cfg, words)
    assert st == amk.AMK_OK, why
    ok, why = plan_oracle.is_safe(words, model)
    assert ok, why


@pytest.mark.parametrize("name,wdtype,n_blocks", QHEAD_CASES)
def test_plans_with_a_quantised_lm_head(name, wdtype, n_blocks):
    cfg, words, model = _plan(name, wdtype, n_blocks, quantize_lm_head=True)
    st, why = amk.amk_plan_check(cfg, words)
    assert st == amk.AMK_OK, why
    ok, why = plan_oracle.is_safe(words, model)
    assert ok, why
    # the same tables are not those of the bf16-head model, for either judge
    cfg0, words0, model0 = _plan(name, wdtype, n_blocks)
    assert amk.amk_plan_check(cfg0, words)[0] != amk.AMK_OK
    assert not plan_oracle.is_safe(words, model0)[0]


def test_other_stage_sizes_are_accepted():
    for sb in (16384, 24576, 65536):
        cfg, words, model = _plan("mini_wide", "int8", 37, stage_bytes=sb)
        assert amk.amk_plan_check(cfg, words)[0] == amk.AMK_OK
        assert plan_oracle.is_safe(words, model)[0]


# ---- mutation classes ------------------------------------------------------------------------------------
def _tile_fields(e):
    e = int(e)
    return e & ((1 << 40) - 1), (e >> 40) & 0x1FFF, e >> 53


def _make_tile(off16, n16, task):
    return np.uint64(off16 | (n16 << 40) | (task << 53))


def m_drop_tile(w, s, rng):          # a consumer waits for a tile its producer never issues (deadlock)
    i = int(rng.integers(s["n_tiles"]))
    out = np.delete(w, s["tiles"] + i)
    out[6] -= 1
    blk = np.searchsorted(w[s["tbeg"]: s["tbeg"] + s["nb"] + 1], i, side="right") - 1
    out[s["tbeg"] + blk + 1: s["tbeg"] + s["nb"] + 1] -= 1
    return out


def m_dup_tile(w, s, rng):           # a tile nobody waits for shifts everything behind it
    i = int(rng.integers(s["n_tiles"]))
    out = np.insert(w, s["tiles"] + i, w[s["tiles"] + i])
    out[6] += 1
    blk = np.searchsorted(w[s["tbeg"]: s["tbeg"] + s["nb"] + 1], i, side="right") - 1
    out[s["tbeg"] + blk + 1: s["tbeg"] + s["nb"] + 1] += 1
    return out


def m_swap_tiles(w, s, rng):         # queue order differs from the consumers' order
    out = w.copy()
    for _ in range(100):
        i = int(rng.integers(s["n_tiles"] - 1))
        a, b = out[s["tiles"] + i], out[s["tiles"] + i + 1]
        if a != b:
            out[s["tiles"] + i], out[s["tiles"] + i + 1] = b, a
            return out
    return out


def m_oob_offset(w, s, rng):         # a copy from outside the weight area
    out = w.copy()
    for _ in range(100):
        i = int(rng.integers(s["n_tiles"]))
        off, n, task = _tile_fields(out[s["tiles"] + i])
        if n:
            out[s["tiles"] + i] = _make_tile((int(w[5]) >> 4) + int(rng.integers(1, 1000)), n, task)
            return out
    return out


def m_oversize(w, s, rng):           # more bytes than a ring stage holds / a tile of the wrong size
    out = w.copy()
    for _ in range(100):
        i = int(rng.integers(s["n_tiles"]))
        off, n, task = _tile_fields(out[s["tiles"] + i])
        if n:
            n2 = int(rng.choice([n + 1, max(1, n - 1), (int(w[4]) >> 4) + 1]))
            out[s["tiles"] + i] = _make_tile(off, n2, task)
            return out
    return out


def m_wrong_task(w, s, rng):         # a tile tagged with another task (the join it belongs to changes)
    out = w.copy()
    i = int(rng.integers(s["n_tiles"]))
    off, n, task = _tile_fields(out[s["tiles"] + i])
    out[s["tiles"] + i] = _make_tile(off, n, task + int(rng.choice([1, 2, 5])))
    return out


def m_bounds(w, s, rng):             # rows with no producer (waited for, never written) or with two
    out = w.copy()
    k = int(rng.integers(5))
    j = int(rng.integers(1, s["nb"]))
    out[s["bounds"] + k * (s["nb"] + 1) + j] += np.uint64(int(rng.choice([1, 3])))
    return out


def m_bounds_end(w, s, rng):         # the last rows of an op have no producer
    out = w.copy()
    k = int(rng.integers(5))
    out[s["bounds"] + k * (s["nb"] + 1) + s["nb"]] -= np.uint64(1)
    return out


def m_marker(w, s, rng):             # the attention marker turned into a weight tile / moved to another layer
    out = w.copy()
    idx = [i for i in range(s["n_tiles"]) if _tile_fields(out[s["tiles"] + i])[1] == 0]
    i = idx[int(rng.integers(len(idx)))]
    off, n, task = _tile_fields(out[s["tiles"] + i])
    out[s["tiles"] + i] = _make_tile(0, 0, task + 5) if rng.integers(2) else _make_tile(0, 4, task)
    return out


def m_region(w, s, rng):             # two ops' regions overlap / an op's shape is not the model's
    out = w.copy()
    i = int(rng.integers(1, s["n_ops"]))
    if rng.integers(2):
        out[s["ops"] + 8 * i + 6] -= np.uint64(256)
    else:
        out[s["ops"] + 8 * i + 3] += np.uint64(1)
    return out


def m_sched_drop_write(w, s, rng):   # a buffer that is waited for is never written (unsatisfiable wait)
    out = w.copy()
    r = int(rng.choice([0, 2, 3, 4]))
    out[s["sched"] + 4 * r + 2] = np.uint64(0)
    return out


def m_sched_partial_join(w, s, rng): # a join that no longer covers all blocks: overwrites race with late readers
    out = w.copy()
    for r in rng.choice([0, 2, 3, 4], size=int(rng.integers(1, 3)), replace=False):
        if rng.integers(2):
            out[s["sched"] + 4 * int(r) + 3] &= np.uint64(0xFF)              # reads nothing whole any more
        else:
            out[s["sched"] + 4 * int(r) + 3] &= np.uint64(~1 & 0xFFFFFF)     # only some blocks take part
    return out


def m_sched_swap(w, s, rng):         # two tasks exchanged in the order
    out = w.copy()
    a, b = (int(x) for x in rng.choice(5, size=2, replace=False))
    ra = out[s["sched"] + 4 * a: s["sched"] + 4 * a + 4].copy()
    out[s["sched"] + 4 * a: s["sched"] + 4 * a + 4] = out[s["sched"] + 4 * b: s["sched"] + 4 * b + 4]
    out[s["sched"] + 4 * b: s["sched"] + 4 * b + 4] = ra
    return out


def m_truncate(w, s, rng):           # a table cut short
    return w[: len(w) - int(rng.integers(1, 50))].copy()


MUTATIONS = [m_drop_tile, m_dup_tile, m_swap_tiles, m_oob_offset, m_oversize, m_wrong_task, m_bounds, m_bounds_end,
             m_marker, m_region, m_sched_drop_write, m_sched_partial_join, m_sched_swap, m_truncate]


@pytest.mark.parametrize("mutation", MUTATIONS, ids=lambda f: f.__name__[2:])
def test_no_false_accept_and_no_false_reject(mutation):
    """30 mutants per class over three plans: whatever the oracle finds unsafe the checker must reject (as in the
    paper's soundness table: no false accept), and the class must actually produce unsafe tables (else the
    test would prove nothing)."""
    rng = np.random.default_rng(1234)
    unsafe = 0
    for name, wdtype, nb in [("mini_ragged", "int8", 13), ("mini_hd128", "int4", 7), ("mini", "bf16", 148)]:
        cfg, words, model = _plan(name, wdtype, nb)
        s = _sections(words)
        for _ in range(10):
            mutant = mutation(words, s, rng)
            ok, why_o = plan_oracle.is_safe(mutant, model)
            st, why_c = amk.amk_plan_check(cfg, mutant)
            if not ok:
                assert st != amk.AMK_OK, ("false accept", mutation.__name__, why_o)
            elif not mutation.__name__.startswith("m_sched"):
                # queues, bounds, regions: the two decide the same property, so they agree both ways; on the
                # dependency model the checker's rule may refuse an edit the three-block instance survives
                assert st == amk.AMK_OK, ("false reject", mutation.__name__, why_c)
            unsafe += not ok
    assert unsafe >= 5, unsafe                       # (the step has redundant joins: many single edits stay safe)


def test_reject_reason_is_reported():
    cfg, words, model = _plan("mini", "bf16", 148)
    s = _sections(words)
    mutant = m_drop_tile(words, s, np.random.default_rng(5))
    st, why = amk.amk_plan_check(cfg, mutant)
    assert st != amk.AMK_OK and "block" in why
