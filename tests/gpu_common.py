"""Helpers shared by the GPU parity tests: run the CUDA path and the CPU oracle on the same seeded
inputs and compare them with the tolerances of the acceptance bar."""
import numpy as np
import torch

from oracle import oracle as orc
from paper_2606_09682_b200 import inputs as inp

HIDDEN_TOL = 5e-3      # rel-L2 per layer hidden state
LOGITS_TOL = 1e-2      # rel-L2 on logits
ARGMAX_GAP = 1e-2      # the greedy token must match bit-exactly when the oracle's top-2 gap exceeds this
WD = {"bf16": orc.W_BF16, "int8": orc.W_INT8, "int4": orc.W_INT4, "int8g": orc.W_INT8G}
LAST = {}                # the last compared step's raw outputs, for callers that need them


def rel_l2(a, b):
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-30))


def bf16_f32(bits):
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def bf16_ulp_distance(a_bits, b_bits):
    """Distance in bf16 steps between two arrays of bit patterns (sign-magnitude -> ordered integers)."""
    def key(x):
        x = np.asarray(x, dtype=np.uint16).astype(np.int32)
        return np.where(x & 0x8000, -(x & 0x7FFF), x & 0x7FFF)
    return np.abs(key(a_bits) - key(b_bits))


def kv_words(kv_gpu):
    """The cache as the oracle keeps it: one 16-bit word per element (a bf16 bit pattern, or an e4m3 code)."""
    if kv_gpu.dtype == torch.uint8:
        return kv_gpu.cpu().numpy().astype(np.uint16)
    return kv_gpu.view(torch.int16).cpu().numpy().view(np.uint16)


def e4m3_f32(codes):
    c = torch.from_numpy(np.ascontiguousarray(codes).astype(np.uint8))
    return c.view(torch.float8_e4m3fn).to(torch.float32).numpy()


def oracle_model(shape, weights_gpu, wdtype, quantize_lm_head=False, kv_dtype="bf16"):
    """The oracle's model of the same seeded bf16 weights, quantised by the oracle's own quantiser."""
    wnp = inp.weights_to_numpy(weights_gpu)
    wq = orc.quantize_weights(wnp, WD[wdtype], 128)
    if quantize_lm_head:
        wq = orc.quantize_lm_head(wq, WD[wdtype], 128, tied=shape.tied)
    return orc.Model(shape, wq, wdtype=WD[wdtype], group=128, quantize_lm_head=quantize_lm_head,
                     kv_dtype=orc.KV_E4M3 if kv_dtype == "fp8" else orc.KV_BF16), wq


def check_argmax(logits_oracle, tok_gpu):
    order = np.argsort(-logits_oracle, kind="stable")
    top, second = logits_oracle[order[0]], logits_oracle[order[1]]
    if top - second > ARGMAX_GAP:
        assert tok_gpu == int(order[0]), (tok_gpu, int(order[0]), float(top - second))
        return "exact"
    assert logits_oracle[tok_gpu] >= top - ARGMAX_GAP, (tok_gpu, float(logits_oracle[tok_gpu]), float(top))
    return "soft"


ELEM_TOL = 1e-3        # element-wise: |gpu - oracle| <= ELEM_TOL * max|oracle| on the logits and on every hidden row
KV_NEAR_ZERO = 1e-4    # a cached value more than one bf16 step off must be within this fraction of its row's maximum


def max_err(a, b):
    """Largest element-wise deviation relative to the reference row's largest magnitude."""
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    return float(np.abs(a - b).max() / max(np.abs(b).max(), 1e-30))


def check_kv_rows(rows_gpu, rows_own, fp8=False):
    """The appended K / V rows of both sides, as bf16 bit patterns (e4m3 codes) of the same shape [..., hd].  They are roundings
    of fp32 values that agree to ~1e-6, so they are equal or neighbours -- except where the value itself is
    rounding noise around zero (there a bf16 step is far smaller than that 1e-6): such entries must be tiny
    against their row.  Returns (largest distance in bf16 steps, fraction one step apart, number further apart)."""
    if fp8:
        key = lambda x: np.where(x & 0x80, -(x & 0x7F).astype(np.int32), (x & 0x7F).astype(np.int32))
        d = np.abs(key(np.asarray(rows_gpu)) - key(np.asarray(rows_own)))
        g_f, o_f = e4m3_f32(rows_gpu), e4m3_f32(rows_own)
    else:
        d = bf16_ulp_distance(rows_gpu, rows_own)
        g_f, o_f = bf16_f32(rows_gpu), bf16_f32(rows_own)
    row_scale = np.abs(o_f).max(axis=-1, keepdims=True)
    far = d > 1
    assert not (far & (np.abs(g_f - o_f) > KV_NEAR_ZERO * row_scale)).any(), (int(d.max()), int(far.sum()))
    return int(d.max()), float((d == 1).mean()), int(far.sum())


def compare_step(shape, dec, model, token, pos, kv_gpu, kv_cpu, check_hidden=True):
    """One step on both sides; asserts the acceptance bar; returns a dict of measured errors.

    The CUDA path runs first.  The oracle then takes the step with the CUDA path's appended cache rows as its
    preference: where such an entry neighbours the oracle's own rounding (both are valid roundings of fp32 values
    that differ in the last bits) the oracle continues from it, so that everything downstream of the cache is
    compared like with like and the element-wise bound can be tight."""
    L, G, S, hd = shape.n_layers, shape.n_kv_heads, shape.max_seq, shape.head_dim
    kv_before = kv_cpu.copy()
    dec.amk_decode_step(token, pos, kv_gpu)
    st, msg = dec.amk_last_status()
    assert st == 0, msg
    kvg = kv_words(kv_gpu).reshape(2, L, G, S, hd)
    rows_gpu = np.ascontiguousarray(kvg[:, :, :, pos, :])
    logits_o, tok_o, hidden_o = model.decode_step(token, pos, kv_cpu, want_hidden=check_hidden, rows_pref=rows_gpu)
    logits_g = dec.logits.cpu().numpy()
    tok_g = int(dec.next_token.item())
    LAST["logits_oracle"], LAST["logits_gpu"], LAST["token_gpu"] = logits_o, logits_g, tok_g
    out = {"logits": rel_l2(logits_g, logits_o), "logits_max": max_err(logits_g, logits_o)}
    assert np.isfinite(logits_g).all()
    if check_hidden:
        hidden_g = dec.amk_debug_hidden().numpy()
        errs = [rel_l2(hidden_g[l], hidden_o[l]) for l in range(L + 1)]
        out["hidden_max"] = max(errs)
        out["hidden_elem_max"] = max(max_err(hidden_g[l], hidden_o[l]) for l in range(L + 1))
        assert errs[0] == 0.0, "embedding row must be exact"
        assert max(errs) <= HIDDEN_TOL, errs
        assert out["hidden_elem_max"] <= ELEM_TOL, out
    assert out["logits"] <= LOGITS_TOL, out
    assert out["logits_max"] <= ELEM_TOL, out
    out["argmax"] = check_argmax(logits_o, tok_g)
    assert tok_g == int(np.argmax(logits_g)) or logits_g[tok_g] == logits_g.max()
    # KV cache: exactly slot `pos` of every layer / kv head changed ...
    kvb = kv_before.reshape(2, L, G, S, hd)
    mask = np.ones(S, dtype=bool)
    mask[pos] = False
    assert np.array_equal(kvg[:, :, :, mask, :], kvb[:, :, :, mask, :]), "a slot other than pos changed"
    # ... and the new rows are the oracle's own roundings or their neighbours
    out["kv_ulp_max"], out["kv_one_step_frac"], out["kv_far"] = check_kv_rows(
        rows_gpu, model.rows_own.reshape(rows_gpu.shape), fp8=kv_gpu.dtype == torch.uint8)
    # keep both caches identical from here on so later steps compare like with like
    kv_cpu[:] = kv_words(kv_gpu)
    return out
