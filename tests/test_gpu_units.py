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
    p, s4, z4 = amk.amk_quantize_int4(w)
    po, s4o, z4o = orc.quantize_int4(wb, 128)
    assert np.array_equal(p.cpu().numpy(), po)
    assert np.array_equal(inp.bits(s4), s4o)
    assert np.array_equal(inp.bits(z4), z4o)


@pytest.mark.parametrize("name,wdtype", [("mini_wide", "bf16"), ("mini_ragged", "bf16"), ("mini_wide", "int8"),
                                         ("mini_ragged", "int8"), ("mini_wide", "int4"), ("mini_hd128", "int4")])
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
