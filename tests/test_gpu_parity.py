"""GPU parity: the CUDA decode step against the CPU oracle, element by element, on small seeded models
whose sizes span several ring tiles, several passes and ragged tails.  Calls go through the C ABI."""
import numpy as np
import pytest
import torch

from paper_2606_09682_b200 import inputs as inp

pytestmark = pytest.mark.gpu

import gpu_common as gc  # noqa: E402


def _setup(name, wdtype, seed, std=0.05, norm_jitter=0.1, quantize_lm_head=False, kv_dtype="bf16", **kw):
    from paper_2606_09682_b200 import binding as amk
    shape = inp.SHAPES[name]
    w = inp.make_weights(shape, seed, device="cuda", std=std, norm_jitter=norm_jitter)
    wq = amk.quantize_weights(w, wdtype)
    if quantize_lm_head:
        wq = amk.quantize_lm_head(wq, wdtype, shape.tied)
    dec = amk.Decoder(shape, wq, wdtype, flags=amk.AMK_FLAG_DEBUG_HIDDEN, quantize_lm_head=quantize_lm_head,
                      kv_dtype=kv_dtype, **kw)
    model, _ = gc.oracle_model(shape, w, wdtype, quantize_lm_head, kv_dtype)
    return shape, dec, model


@pytest.mark.parametrize("name,wdtype", [
    ("mini", "bf16"), ("mini_ragged", "bf16"), ("mini_hd128", "bf16"), ("mini_wide", "bf16"),
    ("mini", "int8"), ("mini_ragged", "int8"), ("mini_hd128", "int8"),
    ("mini", "int4"), ("mini_hd128", "int4"), ("mini_wide", "int4"),
    ("mini", "int8g"), ("mini_hd128", "int8g"), ("mini_wide", "int8g"),
])
def test_multi_step_decode_matches_oracle(name, wdtype):
    shape, dec, model = _setup(name, wdtype, seed=21)
    kv_g = dec.new_cache()
    kv_c = model.new_cache()
    rng = np.random.default_rng(3)
    worst = {"logits": 0.0, "hidden_max": 0.0}
    for pos in range(6):
        tok = int(rng.integers(0, shape.vocab))
        r = gc.compare_step(shape, dec, model, tok, pos, kv_g, kv_c)
        worst = {k: max(worst[k], r[k]) for k in worst}
    print(name, wdtype, worst)
    dec.close()


@pytest.mark.parametrize("name,wdtype", [("mini", "int8"), ("mini_ragged", "int8"), ("mini_wide", "int4"),
                                         ("mini_hd128", "int4"), ("mini_wide", "int8g")])
def test_quantised_lm_head(name, wdtype):
    """quantize_lm_head = 1: the LM head GEMV streams codes quantised like the layers (a quantised copy of the
    embedding matrix for the tied mini_ragged shape), against the oracle with the same reading switched on."""
    shape, dec, model = _setup(name, wdtype, seed=27, quantize_lm_head=True)
    kv_g, kv_c = dec.new_cache(), model.new_cache()
    rng = np.random.default_rng(4)
    for pos in range(4):
        tok = int(rng.integers(0, shape.vocab))
        r = gc.compare_step(shape, dec, model, tok, pos, kv_g, kv_c)
        print(name, wdtype, "quantised head", pos, r)
    dec.close()


@pytest.mark.parametrize("name,wdtype", [("mini", "bf16"), ("mini_ragged", "bf16"), ("mini_hd128", "int8"), ("mini_wide", "int4")])
def test_fp8_cache_multi_step_and_prefilled(name, wdtype):
    """kv_dtype = fp8 (e4m3): appended rows are the oracle's e4m3 roundings or their neighbours, attention reads the
    8-bit entries -- from an empty cache over a few positions, then on a pre-filled cache with several chunks, a
    ragged tail, a chunk boundary and the last slot."""
    shape, dec, model = _setup(name, wdtype, seed=28, kv_dtype="fp8")
    kv_g, kv_c = dec.new_cache(), model.new_cache()
    rng = np.random.default_rng(5)
    for pos in range(5):
        tok = int(rng.integers(0, shape.vocab))
        r = gc.compare_step(shape, dec, model, tok, pos, kv_g, kv_c)
        print(name, wdtype, "fp8 cache", pos, r)
    tok = inp.make_token(shape, 12)
    for pos in (31, 32, 77, 200 if shape.max_seq > 200 else shape.max_seq - 2, shape.max_seq - 1):
        kv_g = inp.make_kv_prefill(shape, 13, pos, device="cuda", kv_dtype="fp8")
        kv_c = gc.kv_words(kv_g).copy()
        r = gc.compare_step(shape, dec, model, tok, pos, kv_g, kv_c)
        print(name, wdtype, "fp8 cache, pre-filled", pos, r)
    dec.close()


@pytest.mark.parametrize("name,pos", [("mini", 100), ("mini_hd128", 200), ("mini_wide", 301), ("mini_ragged", 95)])
def test_prefilled_cache_split_k(name, pos):
    """A pre-filled N(0,1) cache long enough for several split-K chunks with a ragged last chunk."""
    shape, dec, model = _setup(name, "bf16", seed=22)
    kv_g = inp.make_kv_prefill(shape, 5, pos, device="cuda")
    kv_c = inp.bits(kv_g).copy()
    tok = inp.make_token(shape, 5)
    for p in (pos, pos + 1) if pos + 1 < shape.max_seq else (pos,):
        r = gc.compare_step(shape, dec, model, tok, p, kv_g, kv_c)
        print(name, p, r)
    dec.close()


@pytest.mark.parametrize("name,wdtype", [("mini", "bf16"), ("mini_hd128", "int8"), ("mini_ragged", "bf16"), ("mini_wide", "int4"),
                                         ("mini_hd128", "int8g")])
def test_chunk_boundaries_and_last_position(name, wdtype):
    """Positions around the 32-position chunk boundary -- a last chunk that holds nothing but the new row
    (pos = 32, 64), chunks that end exactly at the boundary (pos = 31, 63), one position only in the cache
    (pos = 1) -- and the last position the cache has room for."""
    shape, dec, model = _setup(name, wdtype, seed=24)
    tok = inp.make_token(shape, 6)
    for pos in (1, 31, 32, 33, 63, 64, shape.max_seq - 1):
        kv_g = inp.make_kv_prefill(shape, 7, pos, device="cuda")
        kv_c = inp.bits(kv_g).copy()
        r = gc.compare_step(shape, dec, model, tok, pos, kv_g, kv_c)
        print(name, wdtype, pos, r)
    dec.close()


@pytest.mark.parametrize("name,wdtype", [("mini", "bf16"), ("mini_hd128", "int8"), ("mini_wide", "int4")])
def test_counter_joins(name, wdtype):
    """sync_mode 2: the paper's synchronisation model on top -- a release-increment of one counter per task and
    an acquire-spin on it before the next (Section 4, "Synchronization model") -- gives the same results."""
    shape, dec, model = _setup(name, wdtype, seed=25, sync_mode=2)
    tok = inp.make_token(shape, 8)
    for pos in (0, 1, 40, 100):
        kv_g = inp.make_kv_prefill(shape, 9, pos, device="cuda")
        kv_c = inp.bits(kv_g).copy()
        r = gc.compare_step(shape, dec, model, tok, pos, kv_g, kv_c)
        print(name, wdtype, "counters", pos, r)
    dec.close()


@pytest.mark.parametrize("n_blocks", [148, 101, 37])
def test_block_counts(n_blocks):
    """The split of every product's rows over the blocks (and with it the order of the partial sums) follows the
    block count; the results stay within the same bar for every split, and each split repeats bit for bit."""
    shape, dec, model = _setup("mini_wide", "int8", seed=26, n_blocks=n_blocks)
    tok = inp.make_token(shape, 10)
    for pos in (0, 50):
        kv_g = inp.make_kv_prefill(shape, 11, pos, device="cuda")
        kv_c = inp.bits(kv_g).copy()
        r = gc.compare_step(shape, dec, model, tok, pos, kv_g, kv_c)
        first = dec.logits.clone()
        dec.amk_decode_step(tok, pos, kv_g)
        torch.cuda.synchronize()
        assert torch.equal(dec.logits, first)
        print("blocks", n_blocks, pos, r)
    dec.close()


def test_deterministic_repeat():
    shape, dec, model = _setup("mini_wide", "bf16", seed=23)
    kv = inp.make_kv_prefill(shape, 6, 77, device="cuda")
    ref = None
    for _ in range(20):
        dec.amk_decode_step(11, 77, kv)
        torch.cuda.synchronize()
        cur = (dec.logits.clone(), int(dec.next_token.item()), dec.amk_debug_hidden().clone())
        if ref is None:
            ref = cur
        assert torch.equal(cur[0], ref[0]) and cur[1] == ref[1] and torch.equal(cur[2], ref[2])
    dec.close()
