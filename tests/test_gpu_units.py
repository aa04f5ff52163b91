"""GPU checks of the integer / byte work and of the failure path, through the C ABI:
quantiser codes and scales bit-exact against the oracle's quantiser, the packed layout's inverse
bit-exact against the canonical inputs, the bounded-wait status, argument errors, and the
device-resident greedy loop against single steps."""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2606_09682_b200 import inputs as inp

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def amk():
    from paper_2606_09682_b200 import binding
    return binding


def _rand_bf16(rows, cols, seed, std=0.02):
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    w = (torch.randn(rows, cols, generator=g, device="cuda") * std).to(torch.bfloat16)
    return w


@pytest.mark.parametrize("rows,cols", [(37, 256), (300, 1024), (64, 5632)])
def test_quantisers_bit_exact_against_oracle(amk, rows, cols):
    w = _rand_bf16(rows, cols, 31)
    w[3] = 0                       # all-zero row
    w[5, :128] = w[5, :128].abs()  # all-positive group
    w[7, 1] = 3.0                  # outlier
    wb = inp.bits(w)
    q, s = amk.amk_quantize_int8(w)
    qo, so = orc.quantize_int8(wb)
    assert np.array_equal(q.cpu().numpy(), qo)
    assert np.array_equal(inp.bits(s), so)
    qg, sg = amk.amk_quantize_int8_grouped(w)
    qgo, sgo = orc.quantize_int8_grouped(wb, 128)
    assert np.array_equal(qg.cpu().numpy(), qgo)
    assert np.array_equal(inp.bits(sg), sgo)
    p, s4, z4 = amk.amk_quantize_int4(w)
    po, s4o, z4o = orc.quantize_int4(wb, 128)
    assert np.array_equal(p.cpu().numpy(), po)
    assert np.array_equal(inp.bits(s4), s4o)
    assert np.array_equal(inp.bits(z4), z4o)


@pytest.mark.parametrize("name,wdtype", [("mini_wide", "bf16"), ("mini_ragged", "bf16"), ("mini_wide", "int8"),
                                         ("mini_ragged", "int8"), ("mini_wide", "int4"), ("mini_hd128", "int4"),
                                         ("mini_wide", "int8g"), ("mini_hd128", "int8g")])
def test_packed_layout_unpacks_bit_exact(amk, name, wdtype):
    shape = inp.SHAPES[name]
    w = inp.make_weights(shape, 41, device="cuda")
    wq = amk.quantize_weights(w, wdtype)
    dec = amk.Decoder(shape, wq, wdtype)
    which_of = {"wq": 0, "wk": 1, "wv": 2, "wo": 3, "wgate": 4, "wup": 5, "wdown": 6}
    for l in range(shape.n_layers):
        for kind, which in which_of.items():
            out, sc, zr = dec.amk_debug_unpack(l, which)
            assert torch.equal(out.view(torch.uint8), wq[kind][l].view(torch.uint8)), (l, kind)
            if wdtype != "bf16":
                assert torch.equal(sc.view(torch.int16), wq[kind + "_scale"][l].view(torch.int16)), (l, kind)
            if wdtype == "int4":
                assert torch.equal(zr.view(torch.int16), wq[kind + "_zero"][l].view(torch.int16)), (l, kind)
    out, _, _ = dec.amk_debug_unpack(0, amk.AMK_LIN_LM_HEAD)
    head = w["embed"] if shape.tied else w["lm_head"]
    assert torch.equal(out.view(torch.int16), head.view(torch.int16))
    dec.close()


@pytest.mark.parametrize("name,wdtype", [("mini_ragged", "int8"), ("mini_wide", "int4")])
def test_quantised_lm_head_unpacks_bit_exact(amk, name, wdtype):
    """With quantize_lm_head the packed LM head holds the codes, scales and zero points it was given -- which are
    the oracle quantiser's, bit for bit, of the LM head matrix (of the embedding matrix for the tied shape)."""
    shape = inp.SHAPES[name]
    w = inp.make_weights(shape, 52, device="cuda")
    wq = amk.quantize_lm_head(amk.quantize_weights(w, wdtype), wdtype, shape.tied)
    dec = amk.Decoder(shape, wq, wdtype, quantize_lm_head=True)
    out, sc, zr = dec.amk_debug_unpack(0, amk.AMK_LIN_LM_HEAD)
    assert torch.equal(out.view(torch.uint8), wq["lm_head_q"].view(torch.uint8))
    assert torch.equal(sc.view(torch.int16), wq["lm_head_scale"].view(torch.int16))
    head = inp.bits(w["embed"] if shape.tied else w["lm_head"])
    if wdtype == "int8":
        qo, so = orc.quantize_int8(head)
    else:
        qo, so, zo = orc.quantize_int4(head, 128)
        assert torch.equal(zr.view(torch.int16), wq["lm_head_zero"].view(torch.int16))
        assert np.array_equal(inp.bits(zr), zo)
    assert np.array_equal(out.cpu().numpy().view(qo.dtype), qo) and np.array_equal(inp.bits(sc), so)
    dec.close()


def test_bounded_wait_reports_timeout_and_recovers(amk):
    """A signal that never comes: every waiter gives up after the time limit, the status says which join,
    and the following step is correct again.  Nothing traps or hangs."""
    shape = inp.SHAPES["mini"]
    w = inp.make_weights(shape, 42, device="cuda")
    dec = amk.Decoder(shape, w, "bf16", wait_timeout_us=3000)
    kv = dec.new_cache()
    dec.amk_decode_step(5, 0, kv)
    assert dec.amk_last_status()[0] == amk.AMK_OK
    good = dec.logits.clone()
    dec.amk_debug_drop_signal(phase=7, block=3)
    dec.amk_decode_step(5, 0, kv)
    st, msg = dec.amk_last_status()
    assert st == amk.AMK_ERR_TIMEOUT and "join 7" in msg, (st, msg)
    dec.amk_decode_step(5, 0, kv)
    st, msg = dec.amk_last_status()
    assert st == amk.AMK_OK, msg
    assert torch.equal(dec.logits, good)
    dec.close()


def test_argument_errors(amk):
    shape = inp.SHAPES["mini"]
    w = inp.make_weights(shape, 43, device="cuda")
    dec = amk.Decoder(shape, w, "bf16")
    kv = dec.new_cache()
    for tok, pos, code in ((0, -1, amk.AMK_ERR_BAD_POS), (0, shape.max_seq, amk.AMK_ERR_BAD_POS),
                           (-1, 0, amk.AMK_ERR_BAD_TOKEN), (shape.vocab, 0, amk.AMK_ERR_BAD_TOKEN)):
        with pytest.raises(amk.AmkError) as e:
            dec.amk_decode_step(tok, pos, kv)
        assert e.value.code == code
    assert amk.lib.amk_decode_step(dec.h, 0, 0, None, None, None, None) == amk.AMK_ERR_INVALID_ARG
    # a packed buffer that is too small is refused
    cfg = amk.make_config(shape, "bf16")
    h = C.c_void_p()
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    ws = torch.empty(amk.amk_workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    wts = amk.amk_weights()
    assert amk.lib.amk_create(C.byref(cfg), C.byref(wts), small.data_ptr(), small.numel(), ws.data_ptr(), ws.numel(),
                              None, C.byref(h)) == amk.AMK_ERR_INVALID_ARG
    dec.close()


def test_misaligned_buffers_are_refused_on_the_host(amk):
    """The kernel fetches cache rows with 16-byte bulk copies and writes 4-byte words: a misaligned pointer is an
    argument error, never a device fault."""
    shape = inp.SHAPES["mini"]
    w = inp.make_weights(shape, 45, device="cuda")
    dec = amk.Decoder(shape, w, "bf16")
    kv = dec.new_cache()
    big = torch.zeros(kv.numel() + 64, dtype=torch.bfloat16, device="cuda")
    odd = torch.zeros(shape.vocab * 4 + 16, dtype=torch.uint8, device="cuda")
    call = amk.lib.amk_decode_step
    assert call(dec.h, 1, 0, big.data_ptr() + 2, dec.logits.data_ptr(), dec.next_token.data_ptr(), None) == amk.AMK_ERR_INVALID_ARG
    assert call(dec.h, 1, 0, big.data_ptr() + 8, dec.logits.data_ptr(), dec.next_token.data_ptr(), None) == amk.AMK_ERR_INVALID_ARG
    assert call(dec.h, 1, 0, kv.data_ptr(), odd.data_ptr() + 2, dec.next_token.data_ptr(), None) == amk.AMK_ERR_INVALID_ARG
    assert call(dec.h, 1, 0, kv.data_ptr(), dec.logits.data_ptr(), odd.data_ptr() + 1, None) == amk.AMK_ERR_INVALID_ARG
    toks = torch.zeros(8, dtype=torch.int32, device="cuda")
    assert amk.lib.amk_decode_greedy(dec.h, 1, 0, 4, big.data_ptr() + 4, toks.data_ptr(), None, None) == amk.AMK_ERR_INVALID_ARG
    assert call(dec.h, 1, 0, big.data_ptr() + 16, dec.logits.data_ptr(), dec.next_token.data_ptr(), None) == amk.AMK_OK
    assert dec.amk_last_status()[0] == amk.AMK_OK
    dec.close()


def test_sequence_numbers_cross_their_wrap(amk):
    """Every published activation carries steps * (5 L + 1) + task + 1 in 32 bits.  Near 2^32 the library clears
    the activation area on the stream and restarts the count: steps on both sides of that point, and across it
    inside one device-resident run, give what a fresh handle gives."""
    shape = inp.SHAPES["mini_wide"]
    w = inp.make_weights(shape, 46, device="cuda", std=0.05)
    ref = amk.Decoder(shape, w, "bf16")
    dec = amk.Decoder(shape, w, "bf16")
    per = 5 * shape.n_layers + 1
    limit = (1 << 32) // per
    n = 12
    kv_r, kv_d = ref.new_cache(), dec.new_cache()
    want = ref.amk_decode_greedy(9, 0, n, kv_r).cpu().tolist()
    want_logits = ref.logits.clone()
    dec.amk_debug_set_step_count(limit - 6)                   # the wrap falls inside the 12-step run
    got = dec.amk_decode_greedy(9, 0, n, kv_d).cpu().tolist()
    assert dec.amk_last_status()[0] == amk.AMK_OK
    assert got == want and torch.equal(kv_d, kv_r) and torch.equal(dec.logits, want_logits)
    # single steps right at the boundary, with stale activations of the highest sequence numbers in the workspace
    for start in (limit - 3, limit - 2, limit - 1):
        dec.amk_debug_set_step_count(start)
        kv1, kv2 = dec.new_cache(), ref.new_cache()
        tok = 9
        for pos in range(4):
            dec.amk_decode_step(tok, pos, kv1)
            ref.amk_decode_step(tok, pos, kv2)
            assert dec.amk_last_status()[0] == amk.AMK_OK
            assert torch.equal(dec.logits, ref.logits) and int(dec.next_token.item()) == int(ref.next_token.item())
            tok = int(ref.next_token.item())
        assert torch.equal(kv1, kv2)
    ref.close()
    dec.close()


@pytest.mark.parametrize("wdtype,pos", [("bf16", 0), ("int8", 70), ("int4", 33)])
def test_guard_bands_around_every_caller_buffer_stay_intact(amk, wdtype, pos):
    """Stand-in for a memory checker (none can be run here): the packed buffer, the workspace, the logits and the
    KV cache sit between bands of a fixed pattern; create, the decode step, the device-resident loop and the
    debugging read-backs must leave the bands untouched."""
    shape = inp.SHAPES["mini_ragged" if wdtype != "int4" else "mini_wide"]
    w = inp.make_weights(shape, 47, device="cuda")
    wq = amk.quantize_weights(w, wdtype)
    dec = amk.Decoder(shape, wq, wdtype, flags=amk.AMK_FLAG_DEBUG_HIDDEN | amk.AMK_FLAG_TRACE, guard_bytes=4096)
    kv = dec.new_cache()
    kv.view(torch.int16)[:] = inp.make_kv_prefill(shape, 48, pos, device="cuda").view(torch.int16)
    assert dec.guards_intact()
    dec.amk_decode_step(3, pos, kv)
    assert dec.amk_last_status()[0] == amk.AMK_OK
    dec.amk_decode_greedy(3, pos, min(8, shape.max_seq - pos), kv)
    assert dec.amk_last_status()[0] == amk.AMK_OK
    dec.amk_debug_hidden()
    dec.amk_debug_trace()
    torch.cuda.synchronize()
    assert dec.guards_intact()
    dec.close()


@pytest.mark.parametrize("cycles", [False, True])
def test_trace_stamps_are_ordered_within_every_task(amk, cycles):
    """amk_debug_trace: within a block every matrix-vector task's stamps follow the order of its stages, tasks
    follow each other, and the producer issued a task's first tile no later than its last."""
    shape = inp.SHAPES["mini_wide"]
    w = inp.make_weights(shape, 49, device="cuda")
    flags = amk.AMK_FLAG_TRACE | (amk.AMK_FLAG_TRACE_CYCLES if cycles else 0)
    dec = amk.Decoder(shape, w, "bf16", flags=flags)
    kv = inp.make_kv_prefill(shape, 50, 40, device="cuda")
    for pos in (0, 40):
        dec.amk_decode_step(7, pos, kv)
        assert dec.amk_last_status()[0] == amk.AMK_OK
        tr = dec.amk_debug_trace().numpy()                    # [blocks][5 L + 1][events]
        nb, nt, _ = tr.shape
        order = [0, 1, 2, 8, 9, 10, 7, 3]                     # enter, joined, loaded, pass begin, first tile, tiles done, reduced, computed
        p = dec.plan()
        for b in range(nb):
            prev_end = 0
            for t in range(nt):
                if t % 5 == 1 and t != nt - 1:
                    continue                                  # attention tasks stamp a different set of stages
                e = tr[b, t]
                if e[3] == 0 or e[1] == 0:
                    continue                                  # a block without rows of this product
                seq = [int(e[i]) for i in order]
                assert all(x > 0 for x in seq), (b, t, seq)
                assert all(x <= y for x, y in zip(seq, seq[1:])), (b, t, seq)
                assert seq[0] >= prev_end, (b, t)
                prev_end = seq[-1]
                if e[5]:
                    assert e[5] <= e[6], (b, t)
    dec.close()


def test_greedy_loop_equals_single_steps(amk):
    shape = inp.SHAPES["mini_wide"]
    w = inp.make_weights(shape, 44, device="cuda", std=0.05)
    dec = amk.Decoder(shape, w, "bf16")
    kv1, kv2 = dec.new_cache(), dec.new_cache()
    n = 24
    toks = dec.amk_decode_greedy(17, 0, n, kv1)
    torch.cuda.synchronize()
    last_logits = dec.logits.clone()
    tok, single = 17, []
    for pos in range(n):
        dec.amk_decode_step(tok, pos, kv2)
        tok = int(dec.next_token.item())
        single.append(tok)
    assert toks.cpu().tolist() == single
    assert torch.equal(kv1, kv2) and torch.equal(last_logits, dec.logits)
    assert dec.amk_last_status()[0] == amk.AMK_OK
    dec.close()


def test_knob_search_on_a_small_grid(amk):
    """The search with the real effects: every point passes the correctness gate (the knobs do not change the
    arithmetic: logits bit-equal to the default configuration's), no latency is below the floor."""
    from paper_2606_09682_b200 import autotune as at
    shape = inp.SHAPES["mini_wide"]
    w = inp.make_weights(shape, 51, device="cuda")
    build, correct, measure, release, floor_us = at.gpu_effects(shape, w, "bf16", pos=3)
    grid = [at.Knobs(16384, 2, 2), at.Knobs(24576, 3, 6), at.Knobs(65536, 2, 2)]
    res = at.tune(build, correct, measure, release, floor_us, grid=grid, steps=10, ab_rounds=3)
    assert len(res["trials"]) == 4
    for t in res["trials"]:
        assert t.verdict in ("kept", "reverted") or t.verdict.startswith("rejected: build"), t
        if t.latency_us is not None:
            assert t.latency_us >= floor_us
    assert res["best_us"] >= floor_us


def test_handles_with_different_shared_memory_plans_coexist(amk):
    """A handle created later with a smaller shared-memory plan (smaller ring stages) must not break an earlier
    handle's launches: both step, alternately, and each repeats its own result bit for bit."""
    shape = inp.SHAPES["mini_wide"]
    w = inp.make_weights(shape, 61, device="cuda")
    wq = amk.quantize_weights(w, "int4")
    big = amk.Decoder(shape, wq, "int4")
    small = amk.Decoder(shape, wq, "int4", stage_bytes=8192, n_stages=2)
    assert small.plan().smem_bytes < big.plan().smem_bytes
    kv_b, kv_s = big.new_cache(), small.new_cache()
    outs = []
    for _ in range(2):
        for dec, kv in ((big, kv_b), (small, kv_s)):
            dec.amk_decode_step(7, 0, kv)
            st, msg = dec.amk_last_status()
            assert st == 0, msg
            outs.append(dec.logits.clone())
    assert torch.equal(outs[0], outs[2]) and torch.equal(outs[1], outs[3])
    assert torch.allclose(outs[0], outs[1], rtol=0, atol=1e-3 * float(outs[0].abs().max()))
    big.close()
    small.close()
