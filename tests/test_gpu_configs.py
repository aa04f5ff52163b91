"""GPU parity at the full sizes of the measured workloads, in the launch configuration the benchmark
times (one block per SM, automatic plan).

SmolLM2-135M and TinyLlama-1.1B shapes: the whole step against the whole oracle step.
Llama-3-8B shape: the whole step as well, layer by layer so that only one layer's weights are on the host at
a time -- the oracle applies all 32 layers in turn to its OWN residual stream (starting from the embedding row)
and then the LM head, and every layer's stream, the appended cache rows and the logits are compared with the
CUDA path's.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2606_09682_b200 import inputs as inp

pytestmark = pytest.mark.gpu

import gpu_common as gc  # noqa: E402


@pytest.fixture(scope="module")
def amk():
    from paper_2606_09682_b200 import binding
    return binding


def _build(amk, name, wdtype, seed, quantize_lm_head=False, **kw):
    shape = inp.SHAPES[name]
    w = inp.make_weights(shape, seed, device="cuda")
    wq = amk.quantize_weights(w, wdtype)
    if quantize_lm_head:
        wq = amk.quantize_lm_head(wq, wdtype, shape.tied)
    dec = amk.Decoder(shape, wq, wdtype, flags=amk.AMK_FLAG_DEBUG_HIDDEN, quantize_lm_head=quantize_lm_head, **kw)
    return shape, w, wq, dec


def test_smollm2_shape_one_step_pos0(amk):
    """Config: SmolLM2-135M shape, bf16, one decode step at position 0."""
    shape, w, _, dec = _build(amk, "smollm2_135m", "bf16", 0xA3C0)
    model, _ = gc.oracle_model(shape, w, "bf16")
    kv_g, kv_c = dec.new_cache(), model.new_cache()
    r = gc.compare_step(shape, dec, model, inp.make_token(shape, 0xA3C0), 0, kv_g, kv_c)
    print("smollm2 pos0", r)
    dec.close()


def test_smollm2_shape_measured_split(amk):
    """AMK_FLAG_MEASURED_SPLIT: amk_create measures what every SM streams and gives each block its share of the
    rows (blocks are then identified by SM id): same bar as the equal split, and the same result every time."""
    shape = inp.SHAPES["smollm2_135m"]
    w = inp.make_weights(shape, 0xA3C0, device="cuda")
    dec = amk.Decoder(shape, w, "bf16", flags=amk.AMK_FLAG_DEBUG_HIDDEN | amk.AMK_FLAG_MEASURED_SPLIT)
    model, _ = gc.oracle_model(shape, w, "bf16")
    tok = inp.make_token(shape, 0xA3C0)
    for pos in (0, 37):
        kv_g = inp.make_kv_prefill(shape, 0xA3C0, pos, device="cuda")
        kv_c = inp.bits(kv_g).copy()
        r = gc.compare_step(shape, dec, model, tok, pos, kv_g, kv_c)
        first = dec.logits.clone()
        dec.amk_decode_step(tok, pos, kv_g)
        torch.cuda.synchronize()
        assert torch.equal(dec.logits, first)
        print("smollm2 measured split", pos, r)
    dec.close()


def test_smollm2_shape_256_greedy_steps(amk):
    """Config: 256 consecutive steps from position 0 with a growing cache.  Teacher-forced on the oracle's
    greedy tokens (so every step is compared like with like), then free-running on the device-resident
    loop, reporting where the two token streams first differ."""
    shape, w, _, dec = _build(amk, "smollm2_135m", "bf16", 0xA3C1)
    model, _ = gc.oracle_model(shape, w, "bf16")
    kv_g, kv_c = dec.new_cache(), model.new_cache()
    tok = inp.make_token(shape, 0xA3C1)
    first = tok
    oracle_tokens, oracle_logits, soft = [], [], 0
    worst = {"logits": 0.0, "hidden_max": 0.0}
    for pos in range(256):
        check_hidden = pos % 16 == 0 or pos == 255           # the hidden read-back is the slow part
        r = gc.compare_step(shape, dec, model, tok, pos, kv_g, kv_c, check_hidden=check_hidden)
        worst["logits"] = max(worst["logits"], r["logits"])
        if check_hidden:
            worst["hidden_max"] = max(worst["hidden_max"], r["hidden_max"])
        soft += r["argmax"] == "soft"
        # next input token: the oracle's greedy choice (recomputed from the oracle's logits of this step)
        tok = int(np.argmax(gc.LAST["logits_oracle"]))
        oracle_tokens.append(tok)
        oracle_logits.append(gc.LAST["logits_oracle"])
    kv_free = dec.new_cache()
    toks = dec.amk_decode_greedy(first, 0, 256, kv_free).cpu().tolist()
    div = next((i for i in range(256) if toks[i] != oracle_tokens[i]), 256)
    print("smollm2 256 steps", worst, "soft matches", soft, "free-run agrees with the oracle for", div, "tokens")
    assert dec.amk_last_status()[0] == 0
    # up to the first divergence the free run must be the oracle's stream; a divergence must be at a near-tie:
    # the token the free run chose there has to be within the soft-match gap of the oracle's maximum at that step
    assert div >= 1
    if div < 256:
        lo = oracle_logits[div]
        assert lo[toks[div]] >= lo.max() - gc.ARGMAX_GAP, (div, toks[div], float(lo[toks[div]]), float(lo.max()))
    dec.close()


@pytest.mark.parametrize("wdtype,pos", [("bf16", 0), ("bf16", 1024), ("int8", 0), ("int8", 512), ("int4", 0), ("int4", 512),
                                        ("int8g", 0), ("int8g", 300)])
def test_tinyllama_shape(amk, wdtype, pos):
    shape, w, _, dec = _build(amk, "tinyllama_1b", wdtype, 0xA3C2)
    model, _ = gc.oracle_model(shape, w, wdtype)
    kv_g = inp.make_kv_prefill(shape, 0xA3C2, pos, device="cuda")
    kv_c = inp.bits(kv_g).copy()
    r = gc.compare_step(shape, dec, model, inp.make_token(shape, 0xA3C2), pos, kv_g, kv_c)
    print("tinyllama", wdtype, pos, r)
    dec.close()


@pytest.mark.parametrize("wdtype,pos", [("bf16", 1024), ("int8", 0), ("int4", 300)])
def test_tinyllama_shape_fp8_cache(amk, wdtype, pos):
    """The TinyLlama shape with an fp8 (e4m3) KV cache: the whole step against the oracle with the same cache type."""
    shape, w, _, dec = _build(amk, "tinyllama_1b", wdtype, 0xA3C7, kv_dtype="fp8")
    model, _ = gc.oracle_model(shape, w, wdtype, kv_dtype="fp8")
    kv_g = inp.make_kv_prefill(shape, 0xA3C7, pos, device="cuda", kv_dtype="fp8")
    kv_c = gc.kv_words(kv_g).copy()
    r = gc.compare_step(shape, dec, model, inp.make_token(shape, 0xA3C7), pos, kv_g, kv_c)
    print("tinyllama fp8 cache", wdtype, pos, r)
    dec.close()


@pytest.mark.parametrize("wdtype,pos", [("int8", 0), ("int4", 200), ("int8g", 0)])
def test_tinyllama_shape_quantised_lm_head(amk, wdtype, pos):
    shape, w, _, dec = _build(amk, "tinyllama_1b", wdtype, 0xA3C2, quantize_lm_head=True)
    model, _ = gc.oracle_model(shape, w, wdtype, quantize_lm_head=True)
    kv_g = inp.make_kv_prefill(shape, 0xA3C2, pos, device="cuda")
    kv_c = inp.bits(kv_g).copy()
    r = gc.compare_step(shape, dec, model, inp.make_token(shape, 0xA3C2), pos, kv_g, kv_c)
    print("tinyllama quantised head", wdtype, pos, r)
    dec.close()


@pytest.mark.parametrize("wdtype,pos", [("bf16", 0), ("int8", 77), ("int4", 0)])
def test_paper_small_shape(amk, wdtype, pos):
    """The paper's 4-layer hidden-2048 "small" model (vocabulary assumed: see the shape record): the whole step."""
    shape, w, _, dec = _build(amk, "paper_small", wdtype, 0xA3C6)
    model, _ = gc.oracle_model(shape, w, wdtype)
    kv_g = inp.make_kv_prefill(shape, 0xA3C6, pos, device="cuda")
    kv_c = inp.bits(kv_g).copy()
    r = gc.compare_step(shape, dec, model, inp.make_token(shape, 0xA3C6), pos, kv_g, kv_c)
    print("paper_small", wdtype, pos, r)
    dec.close()


@pytest.mark.parametrize("wdtype,pos", [("bf16", 0), ("int8", 0), ("int4", 300)])
def test_llama32_1b_shape(amk, wdtype, pos):
    """The paper's 16-layer "b1" shape (Llama-3.2-1B dimensions, untied head): the whole step against the oracle."""
    shape, w, _, dec = _build(amk, "llama32_1b", wdtype, 0xA3C5)
    model, _ = gc.oracle_model(shape, w, wdtype)
    kv_g = inp.make_kv_prefill(shape, 0xA3C5, pos, device="cuda")
    kv_c = inp.bits(kv_g).copy()
    r = gc.compare_step(shape, dec, model, inp.make_token(shape, 0xA3C5), pos, kv_g, kv_c)
    print("llama32_1b", wdtype, pos, r)
    dec.close()


@pytest.mark.parametrize("wdtype,pos", [("bf16", 0), ("bf16", 4096), ("int8", 0), ("int8", 4096), ("int4", 0), ("int4", 2500),
                                        ("int8g", 0)])
def test_llama3_8b_shape_whole_step_layer_by_layer(amk, wdtype, pos):
    shape, w, wq, dec = _build(amk, "llama3_8b", wdtype, 0xA3C4)
    kv_g = inp.make_kv_prefill(shape, 0xA3C4, pos, device="cuda")
    kv_before = kv_g.clone()
    tok = inp.make_token(shape, 0xA3C4)
    dec.amk_decode_step(tok, pos, kv_g)
    st, msg = dec.amk_last_status()
    assert st == 0, msg
    hidden = dec.amk_debug_hidden().numpy()
    logits_g = dec.logits.cpu().numpy()
    tok_g = int(dec.next_token.item())
    L, G, S, hd = shape.n_layers, shape.n_kv_heads, shape.max_seq, shape.head_dim
    s1 = shape.with_(n_layers=1)
    wdt = gc.WD[wdtype]
    kvb = kv_before.view(2, L, G, S, hd)
    kva = kv_g.view(2, L, G, S, hd)
    x = w["embed"][tok].float().cpu().numpy()               # the oracle's own stream, from the embedding row on
    assert np.array_equal(hidden[0], x)
    worst = {"hidden": 0.0, "hidden_elem": 0.0, "kv_ulp": 0, "kv_one_step_frac": 0.0, "kv_far": 0}
    mask = np.ones(S, dtype=bool)
    mask[pos] = False
    for l in range(L):
        wl = {"embed": np.zeros((1, shape.hidden), dtype=np.uint16), "lm_head": np.zeros((1, shape.hidden), dtype=np.uint16),
              "final_norm": inp.bits(w["final_norm"]),
              "attn_norm": [inp.bits(w["attn_norm"][l])], "mlp_norm": [inp.bits(w["mlp_norm"][l])]}
        for k in inp.KINDS:
            wl[k] = [inp.bits(w[k][l])]
        wl = orc.quantize_weights(wl, wdt, 128)               # the oracle's own quantiser, every layer
        if wdtype != "bf16" and l in (0, L // 2, L - 1):
            # ... which agrees bit for bit with the device quantiser used for the CUDA path
            assert np.array_equal(wl["wdown"][0], wq["wdown"][l].cpu().numpy())
            assert np.array_equal(wl["wdown_scale"][0], inp.bits(wq["wdown_scale"][l]))
        model = orc.Model(s1.with_(vocab=1), wl, wdtype=wdt, group=128)
        kv_l = inp.bits(kvb[:, l].contiguous()).reshape(-1).copy()          # [2][1][G][S][hd]
        kvg = inp.bits(kva[:, l].contiguous()).reshape(2, G, S, hd)
        rows_gpu = np.ascontiguousarray(kvg[:, :, pos, :])
        x = model.layer_step(0, pos, x, kv_l, rows_pref=rows_gpu)
        e, em = gc.rel_l2(hidden[l + 1], x), gc.max_err(hidden[l + 1], x)
        assert e <= gc.HIDDEN_TOL and em <= gc.ELEM_TOL, (l, e, em)
        # the cache: slot `pos` only was written, with the oracle's own roundings or their neighbours
        assert np.array_equal(kvg[:, :, mask, :], inp.bits(kvb[:, l].contiguous()).reshape(2, G, S, hd)[:, :, mask, :])
        u, f1, far = gc.check_kv_rows(rows_gpu, model.rows_own.reshape(rows_gpu.shape))
        worst = {"hidden": max(worst["hidden"], e), "hidden_elem": max(worst["hidden_elem"], em),
                 "kv_ulp": max(worst["kv_ulp"], u), "kv_one_step_frac": max(worst["kv_one_step_frac"], f1),
                 "kv_far": worst["kv_far"] + far}
        del model, wl
    # LM head on the oracle's own final stream: the logits of the whole step
    head_w = {"embed": np.zeros((1, shape.hidden), dtype=np.uint16), "lm_head": inp.bits(w["lm_head"]),
              "final_norm": inp.bits(w["final_norm"]), "attn_norm": [inp.bits(w["attn_norm"][0])],
              "mlp_norm": [inp.bits(w["mlp_norm"][0])]}
    for k in inp.KINDS:
        head_w[k] = [np.zeros((1, 1), dtype=np.uint16)]
    hm = orc.Model(s1.with_(tied=False), head_w)
    logits_o, tok_o = hm.head_step(x)
    el, elm = gc.rel_l2(logits_g, logits_o), gc.max_err(logits_g, logits_o)
    assert el <= gc.LOGITS_TOL and elm <= gc.ELEM_TOL, (el, elm)
    kind = gc.check_argmax(logits_o, tok_g)
    print("llama3_8b", wdtype, pos, worst, {"logits": el, "logits_elem": elm, "argmax": kind})
    dec.close()
