"""Whole-step pins for the CPU oracle.

1. A second, independent statement of the model: a dense float64 recomputation over the whole prefix
   (explicit causal score matrix, no cache, nothing incremental), written here with numpy matrices.
   Decoding with the cache must reproduce its last row at every step.
2. A library special case: a random-init transformers ``LlamaForCausalLM`` on the toy shape (fp32,
   eager attention).  This fixes the conventions the paper leaves to "HuggingFace Llama-family":
   half-split rotary pairing, grouped-query head mapping, pre-norm residual layout, SwiGLU order.
3. Quantised variants against the same dense recomputation fed with dequantised matrices.
"""
import math

import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2606_09682_b200 import inputs as inp


def f64(bits):
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def round_bf16(x64):
    """fp64 -> fp32 -> bf16 -> fp64 through torch's conversions."""
    t = torch.tensor(np.asarray(x64, dtype=np.float64)).to(torch.float32).to(torch.bfloat16)
    return t.to(torch.float64).numpy()


def e4m3_codes(x64):
    """fp64 -> fp32 -> e4m3 codes through torch's conversion (round to nearest even; callers stay below 448)."""
    t = torch.tensor(np.asarray(x64, dtype=np.float64)).to(torch.float32).to(torch.float8_e4m3fn)
    return t.view(torch.uint8).numpy()


def e4m3_values(codes):
    return torch.from_numpy(np.ascontiguousarray(codes, dtype=np.uint8)).view(torch.float8_e4m3fn).to(torch.float64).numpy()


def dense_forward(shape, W, tokens, round_kv=True, e4m3_cache=None):
    """Logits [T][V] and hidden [T][L+1][H] for the whole token prefix, recomputed from scratch.
    W: dict of float64 matrices (already dequantised).
    ``e4m3_cache``: the step-by-step implementation's fp8 cache as codes [2][L][n_kv][S][hd].  fp8 steps are coarse
    (2^-4 relative), so two correct computations of a key that differ in the last fp32 bits may round to neighbouring
    codes and then differ visibly downstream; here each cached code must be this dense form's own rounding of its own
    fp64 key / value or a neighbour of it, and the dense form then carries on with the cached code's value."""
    T = len(tokens)
    H, nq, nkv, hd = shape.hidden, shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    n_rep = nq // nkv
    X = W["embed"][tokens]                                           # [T][H]
    hidden = [X.copy()]
    pos = np.arange(T)[:, None]
    inv_freq = shape.rope_theta ** (-2.0 * np.arange(hd // 2) / hd)  # [hd/2]
    ang = pos * inv_freq[None, :]
    cos, sin = np.cos(ang), np.sin(ang)                              # [T][hd/2]

    def norm(X, g):
        return X / np.sqrt((X ** 2).mean(axis=1, keepdims=True) + shape.rms_eps) * g[None, :]

    def rot(U):                                                      # U [T][heads][hd]
        a, b = U[..., :hd // 2], U[..., hd // 2:]
        c, s = cos[:, None, :], sin[:, None, :]
        return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)

    causal = np.tril(np.ones((T, T), dtype=bool))
    for l in range(shape.n_layers):
        A = norm(X, W["attn_norm"][l])
        Q = rot((A @ W["wq"][l].T).reshape(T, nq, hd))
        K = rot((A @ W["wk"][l].T).reshape(T, nkv, hd))
        Vv = (A @ W["wv"][l].T).reshape(T, nkv, hd)
        if e4m3_cache is not None:
            for which, U in ((0, K), (1, Vv)):
                got = np.transpose(e4m3_cache[which, l, :, :T, :], (1, 0, 2)).astype(np.uint8)      # [T][n_kv][hd]
                own = e4m3_codes(U)
                mag = lambda c: np.where(c & 0x80, -(c & 0x7F).astype(np.int32), (c & 0x7F).astype(np.int32))
                apart = np.abs(mag(got) - mag(own))
                assert apart.max() <= 1, (l, which, int(apart.max()))
                assert (apart != 0).mean() < 0.01                     # neighbours are the rare exception
                U[...] = e4m3_values(got)
        elif round_kv:
            K, Vv = round_bf16(K), round_bf16(Vv)
        O = np.zeros((T, nq, hd))
        for h in range(nq):
            g = h // n_rep
            S = (Q[:, h, :] @ K[:, g, :].T) / math.sqrt(hd)          # [T][T]
            S = np.where(causal, S, -np.inf)
            P = np.exp(S - S.max(axis=1, keepdims=True))
            P /= P.sum(axis=1, keepdims=True)
            O[:, h, :] = P @ Vv[:, g, :]
        X = X + O.reshape(T, nq * hd) @ W["wo"][l].T
        B = norm(X, W["mlp_norm"][l])
        G, U = B @ W["wgate"][l].T, B @ W["wup"][l].T
        X = X + ((G / (1.0 + np.exp(-G))) * U) @ W["wdown"][l].T
        hidden.append(X.copy())
    Y = norm(X, W["final_norm"])
    head = W["lm_head_deq"] if W.get("lm_head_deq") is not None else (W["embed"] if shape.tied else W["lm_head"])
    return Y @ head.T, np.stack(hidden, axis=1)


def to_f64(wnp, shape, wdtype=orc.W_BF16, group=128):
    out = {"embed": f64(wnp["embed"]), "final_norm": f64(wnp["final_norm"]),
           "lm_head": None if shape.tied else f64(wnp["lm_head"]),
           "attn_norm": [f64(a) for a in wnp["attn_norm"]], "mlp_norm": [f64(a) for a in wnp["mlp_norm"]]}
    for kind in orc.KINDS:
        mats = []
        for l in range(shape.n_layers):
            if wdtype == orc.W_BF16:
                mats.append(f64(wnp[kind][l]))
            elif wdtype == orc.W_INT8:
                s = wnp[kind + "_scale"][l].view(np.float16).astype(np.float64)
                mats.append(wnp[kind][l].astype(np.float64) * s[:, None])
            elif wdtype == orc.W_INT8G:
                s = wnp[kind + "_scale"][l].view(np.float16).astype(np.float64)
                mats.append(wnp[kind][l].astype(np.float64) * np.repeat(s, group, axis=1))
            else:
                q = orc.unpack_int4(wnp[kind][l]).astype(np.float64)
                s = wnp[kind + "_scale"][l].view(np.float16).astype(np.float64)
                z = wnp[kind + "_zero"][l].view(np.float16).astype(np.float64)
                mats.append((q - np.repeat(z, group, axis=1)) * np.repeat(s, group, axis=1))
        out[kind] = mats
    if "lm_head_q" in wnp:                                           # a quantised LM head: its dequantised matrix
        if wdtype == orc.W_INT8:
            s = wnp["lm_head_scale"].view(np.float16).astype(np.float64)
            out["lm_head_deq"] = wnp["lm_head_q"].astype(np.float64) * s[:, None]
        elif wdtype == orc.W_INT8G:
            s = wnp["lm_head_scale"].view(np.float16).astype(np.float64)
            out["lm_head_deq"] = wnp["lm_head_q"].astype(np.float64) * np.repeat(s, group, axis=1)
        else:
            q = orc.unpack_int4(wnp["lm_head_q"]).astype(np.float64)
            s = wnp["lm_head_scale"].view(np.float16).astype(np.float64)
            z = wnp["lm_head_zero"].view(np.float16).astype(np.float64)
            out["lm_head_deq"] = (q - np.repeat(z, group, axis=1)) * np.repeat(s, group, axis=1)
    return out


def rel_l2(a, b):
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-30))


def greedy_tokens(n, vocab, seed):
    rng = np.random.default_rng(seed)
    return [int(t) for t in rng.integers(0, vocab, size=n)]


@pytest.mark.parametrize("name,norm_jitter", [("toy", 0.0), ("toy", 0.1), ("toy_ragged", 0.1)])
def test_decode_with_cache_equals_dense_recompute(name, norm_jitter):
    shape = inp.SHAPES[name]
    w = inp.make_weights(shape, seed=11, std=0.25 if name == "toy" else 0.08, norm_jitter=norm_jitter)
    wnp = inp.weights_to_numpy(w)
    model = orc.Model(shape, wnp)
    toks = greedy_tokens(9, shape.vocab, 5)
    logits_d, hidden_d = dense_forward(shape, to_f64(wnp, shape), toks)
    kv = model.new_cache()
    for t, tok in enumerate(toks):
        logits, nxt, hidden = model.decode_step(tok, t, kv)
        assert rel_l2(hidden, hidden_d[t]) < 2e-5
        assert rel_l2(logits, logits_d[t]) < 2e-5
        gap = np.sort(logits_d[t])[-1] - np.sort(logits_d[t])[-2]
        if gap > 1e-4:
            assert nxt == int(np.argmax(logits_d[t]))
    # the cache slots beyond the last position were never written
    S, hd = shape.max_seq, shape.head_dim
    kvv = kv.reshape(2, shape.n_layers, shape.n_kv_heads, S, hd)
    assert not kvv[:, :, :, len(toks):, :].any()
    assert kvv[:, :, :, :len(toks), :].any()


@pytest.mark.parametrize("name,wdtype", [("toy", orc.W_BF16), ("toy_ragged", orc.W_BF16), ("toy", orc.W_INT8)])
def test_fp8_cache_decode_equals_dense_recompute_on_the_cached_codes(name, wdtype):
    """kv_dtype = e4m3: every appended cache entry is the e4m3 rounding (torch's, on an independent fp64 forward)
    of the rotated key / the value or its neighbour; attention reads the decoded codes; everything downstream
    equals the dense form computed from those codes.  The cache differs from the bf16 cache's values."""
    shape = inp.SHAPES[name]
    group = 32 if name == "toy" else 8
    w = inp.make_weights(shape, seed=19, std=0.25 if name == "toy" else 0.08, norm_jitter=0.1)
    wq = orc.quantize_weights(inp.weights_to_numpy(w), wdtype, group)
    model = orc.Model(shape, wq, wdtype=wdtype, group=group, kv_dtype=orc.KV_E4M3)
    model16 = orc.Model(shape, wq, wdtype=wdtype, group=group)
    toks = greedy_tokens(8, shape.vocab, 9)
    kv, kv16 = model.new_cache(), model16.new_cache()
    outs = []
    for t, tok in enumerate(toks):
        outs.append(model.decode_step(tok, t, kv))
        l16, _, h16 = model16.decode_step(tok, t, kv16)
    assert kv.max() <= 0xFF                                          # codes in the low byte
    L, G, S, hd = shape.n_layers, shape.n_kv_heads, shape.max_seq, shape.head_dim
    codes = kv.reshape(2, L, G, S, hd)
    logits_d, hidden_d = dense_forward(shape, to_f64(wq, shape, wdtype, group), toks, e4m3_cache=codes)
    for t in range(len(toks)):
        logits, nxt, hidden = outs[t]
        assert rel_l2(hidden, hidden_d[t]) < 2e-5
        assert rel_l2(logits, logits_d[t]) < 2e-5
    assert not codes[:, :, :, len(toks):, :].any()                   # slots beyond the last position untouched
    assert rel_l2(outs[-1][0], l16) > 1e-3                           # not the bf16 cache's result
    # position 0 of layer 0: the attention output is the decoded cached v (softmax over one position)
    assert np.array_equal(orc.e4m3_to_f32(codes[1, 0, :, 0, :].astype(np.uint8)),
                          e4m3_values(codes[1, 0, :, 0, :]).astype(np.float32))


@pytest.mark.parametrize("wdtype", [orc.W_INT8, orc.W_INT4, orc.W_INT8G])
def test_quantised_decode_equals_dense_on_dequantised_matrices(wdtype):
    shape = inp.SHAPES["toy"]
    group = 32                                                       # hidden 64 -> 2 groups, mlp 128 -> 4 groups
    w = inp.make_weights(shape, seed=12, std=0.25, norm_jitter=0.1)
    wq = orc.quantize_weights(inp.weights_to_numpy(w), wdtype, group)
    model = orc.Model(shape, wq, wdtype=wdtype, group=group)
    toks = greedy_tokens(6, shape.vocab, 6)
    logits_d, hidden_d = dense_forward(shape, to_f64(wq, shape, wdtype, group), toks)
    kv = model.new_cache()
    for t, tok in enumerate(toks):
        logits, nxt, hidden = model.decode_step(tok, t, kv)
        assert rel_l2(hidden, hidden_d[t]) < 2e-5
        assert rel_l2(logits, logits_d[t]) < 2e-5


@pytest.mark.parametrize("wdtype", [orc.W_INT8, orc.W_INT4, orc.W_INT8G])
@pytest.mark.parametrize("name", ["toy", "toy_ragged"])
def test_quantised_lm_head_equals_dense_on_its_dequantised_matrix(wdtype, name):
    """quantize_lm_head = 1: the LM head (the embedding matrix when tied) is quantised like the layers; the
    embedding gather keeps reading bf16.  The logits must be those of the dense form with the dequantised head, and
    must differ from the bf16-head logits (so the flag is not a no-op)."""
    shape = inp.SHAPES[name]
    group = 32 if name == "toy" else 8                               # toy_ragged: hidden 192, mlp 328 -> groups of 8
    # (grouped int8 takes another seed: with seed 15 one cached K element of the toy model sits on a bf16 rounding
    #  tie that the fp64 dense form and the fp32 step resolve differently, a 2^-9 step on that element)
    seed = 16 if wdtype == orc.W_INT8G else 15
    w = inp.make_weights(shape, seed=seed, std=0.25 if name == "toy" else 0.08, norm_jitter=0.1)
    wq = orc.quantize_weights(inp.weights_to_numpy(w), wdtype, group)
    wq = orc.quantize_lm_head(wq, wdtype, group, tied=shape.tied)
    model = orc.Model(shape, wq, wdtype=wdtype, group=group, quantize_lm_head=True)
    plain = orc.Model(shape, wq, wdtype=wdtype, group=group)
    toks = greedy_tokens(4, shape.vocab, 7)
    logits_d, hidden_d = dense_forward(shape, to_f64(wq, shape, wdtype, group), toks)
    kv, kv2 = model.new_cache(), plain.new_cache()
    for t, tok in enumerate(toks):
        logits, nxt, hidden = model.decode_step(tok, t, kv)
        logits_p, _, hidden_p = plain.decode_step(tok, t, kv2)
        assert rel_l2(logits, logits_d[t]) < 2e-5
        assert np.array_equal(hidden, hidden_p)                      # the layers and the embedding row are untouched
        assert rel_l2(logits, logits_p) > 1e-3
        lg, nx = model.head_step(hidden[-1])
        assert np.array_equal(lg, logits) and nx == nxt


def test_layer_and_head_steps_compose_to_the_full_step():
    shape = inp.SHAPES["toy_ragged"]
    wnp = inp.weights_to_numpy(inp.make_weights(shape, seed=13, std=0.08, norm_jitter=0.1))
    model = orc.Model(shape, wnp)
    kv_a, kv_b = model.new_cache(), model.new_cache()
    for pos, tok in enumerate([3, 77, 500]):
        logits, nxt, hidden = model.decode_step(tok, pos, kv_a)
        x = hidden[0].copy()
        for l in range(shape.n_layers):
            x = model.layer_step(l, pos, x, kv_b)
            assert np.array_equal(x, hidden[l + 1])
        lg, nx = model.head_step(x)
        assert np.array_equal(lg, logits) and nx == nxt
    assert np.array_equal(kv_a, kv_b)


def test_pos0_attention_output_is_cached_v():
    """At position 0 the softmax has one entry, so layer 0's attention output is the rounded V row:
    x_1 = x_0 + Wo * bf16(v) exactly as the dense form with a 1x1 score matrix says."""
    shape = inp.SHAPES["toy"]
    wnp = inp.weights_to_numpy(inp.make_weights(shape, seed=14, std=0.25))
    model = orc.Model(shape, wnp)
    kv = model.new_cache()
    tok = 42
    logits, nxt, hidden = model.decode_step(tok, 0, kv)
    W = to_f64(wnp, shape)
    x0 = W["embed"][tok]
    a = x0 / np.sqrt((x0 ** 2).mean() + shape.rms_eps)
    v = round_bf16(a @ W["wv"][0].T)                                  # [nkv*hd]
    n_rep = shape.n_q_heads // shape.n_kv_heads
    o = np.concatenate([v.reshape(shape.n_kv_heads, -1)[h // n_rep] for h in range(shape.n_q_heads)])
    x_attn = x0 + o @ W["wo"][0].T
    b = x_attn / np.sqrt((x_attn ** 2).mean() + shape.rms_eps)
    G, U = b @ W["wgate"][0].T, b @ W["wup"][0].T
    x1 = x_attn + ((G / (1 + np.exp(-G))) * U) @ W["wdown"][0].T
    assert rel_l2(hidden[1], x1) < 1e-5
    S, hd = shape.max_seq, shape.head_dim
    kvv = kv.reshape(2, shape.n_layers, shape.n_kv_heads, S, hd)
    assert np.array_equal(f64(kvv[1, 0, :, 0, :]).ravel(), v)


def _bump(bits, steps):
    """bf16 bit patterns moved `steps` representable values away from zero (finite, non-zero inputs)."""
    return (np.asarray(bits, dtype=np.uint16) + np.uint16(steps)).astype(np.uint16)


@pytest.mark.parametrize("kv_dtype", [orc.KV_BF16, orc.KV_E4M3])
def test_preferred_cache_rows_are_adopted_only_next_to_the_own_rounding(kv_dtype):
    """decode_step(rows_pref=...): another implementation's appended rows are taken where they are the oracle's
    own rounding or a neighbouring bf16 (e4m3) value, and attention then reads them; anything further away is
    refused.  Pinned at position 0, where the attention output is the cached V row, against the dense form."""
    shape = inp.SHAPES["toy"]
    wnp = inp.weights_to_numpy(inp.make_weights(shape, seed=14, std=0.25))
    model = orc.Model(shape, wnp, kv_dtype=kv_dtype)
    tok = 42
    L, G, S, hd = shape.n_layers, shape.n_kv_heads, shape.max_seq, shape.head_dim
    kv0 = model.new_cache()
    logits0, nxt0, hidden0 = model.decode_step(tok, 0, kv0)
    own = kv0.reshape(2, L, G, S, hd)[:, :, :, 0, :].copy()                  # [2][L][G][hd]
    # 1. preferring the oracle's own rows changes nothing
    kv1 = model.new_cache()
    logits1, nxt1, hidden1 = model.decode_step(tok, 0, kv1, rows_pref=own)
    assert model.n_adopted == 0 and np.array_equal(model.rows_own.reshape(own.shape), own)
    assert np.array_equal(kv1, kv0) and np.array_equal(logits1, logits0) and np.array_equal(hidden1, hidden0)
    # 2. layer 0: every third V entry one step away (adopted), every fifth K entry two steps away (refused)
    pref = own.copy()
    pref[1, 0].reshape(-1)[::3] = _bump(own[1, 0].reshape(-1)[::3], 1)
    pref[0, 0].reshape(-1)[::5] = _bump(own[0, 0].reshape(-1)[::5], 2)
    kv2 = model.new_cache()
    logits2, nxt2, hidden2 = model.decode_step(tok, 0, kv2, rows_pref=pref)
    got = kv2.reshape(2, L, G, S, hd)[:, :, :, 0, :]
    own2 = model.rows_own.reshape(own.shape)
    assert np.array_equal(own2[:, 0], own[:, 0])                              # layer 0's own roundings are as before
    assert np.array_equal(got[1, 0], pref[1, 0]) and np.array_equal(got[0, 0], own[0, 0])
    # (later layers see a changed stream: there the first run's rows are adopted wherever they are neighbours)
    assert model.n_adopted == int((got != own2).sum()) >= len(own[1, 0].reshape(-1)[::3])
    # the dense form of layer 0 with the adopted V row
    W = to_f64(wnp, shape)
    x0 = W["embed"][tok]
    v = (f64(pref[1, 0]) if kv_dtype == orc.KV_BF16 else e4m3_values(pref[1, 0])).reshape(G, hd)
    n_rep = shape.n_q_heads // G
    o = np.concatenate([v[h // n_rep] for h in range(shape.n_q_heads)])
    x_attn = x0 + o @ W["wo"][0].T
    b = x_attn / np.sqrt((x_attn ** 2).mean() + shape.rms_eps)
    Gt, U = b @ W["wgate"][0].T, b @ W["wup"][0].T
    x1 = x_attn + ((Gt / (1 + np.exp(-Gt))) * U) @ W["wdown"][0].T
    assert rel_l2(hidden2[1], x1) < 1e-5
    assert rel_l2(hidden0[1], x1) > 1e-4                                     # (the bumped entries do matter)
    # 3. the single-layer form agrees with the full step
    kv3 = model.new_cache()
    x = model.layer_step(0, 0, hidden2[0], kv3, rows_pref=pref[:, 0])
    assert np.array_equal(x, hidden2[1]) and model.n_adopted == len(own[1, 0].reshape(-1)[::3])


def test_against_transformers_llama():
    tr = pytest.importorskip("transformers")
    shape = inp.SHAPES["toy"]
    w = inp.make_weights(shape, seed=15, std=0.25, norm_jitter=0.1)
    wnp = inp.weights_to_numpy(w)
    kwargs = dict(hidden_size=shape.hidden, intermediate_size=shape.mlp, num_hidden_layers=shape.n_layers,
                  num_attention_heads=shape.n_q_heads, num_key_value_heads=shape.n_kv_heads,
                  head_dim=shape.head_dim, vocab_size=shape.vocab, rms_norm_eps=shape.rms_eps,
                  max_position_embeddings=shape.max_seq, tie_word_embeddings=False, attention_bias=False,
                  mlp_bias=False, hidden_act="silu", attention_dropout=0.0)
    try:
        cfg = tr.LlamaConfig(rope_theta=shape.rope_theta, **kwargs)
    except TypeError:
        cfg = tr.LlamaConfig(rope_parameters={"rope_type": "default", "rope_theta": shape.rope_theta}, **kwargs)
    cfg._attn_implementation = "eager"
    torch.manual_seed(0)
    m = tr.LlamaForCausalLM(cfg).to(torch.float32).eval()
    sd = m.state_dict()

    def put(name, t):
        assert sd[name].shape == t.shape, (name, sd[name].shape, t.shape)
        sd[name].copy_(t.float())

    with torch.no_grad():
        put("model.embed_tokens.weight", w["embed"])
        put("lm_head.weight", w["lm_head"])
        put("model.norm.weight", w["final_norm"])
        names = {"wq": "self_attn.q_proj", "wk": "self_attn.k_proj", "wv": "self_attn.v_proj",
                 "wo": "self_attn.o_proj", "wgate": "mlp.gate_proj", "wup": "mlp.up_proj", "wdown": "mlp.down_proj"}
        for l in range(shape.n_layers):
            put(f"model.layers.{l}.input_layernorm.weight", w["attn_norm"][l])
            put(f"model.layers.{l}.post_attention_layernorm.weight", w["mlp_norm"][l])
            for k, n in names.items():
                put(f"model.layers.{l}.{n}.weight", w[k][l])
    toks = greedy_tokens(8, shape.vocab, 7)
    with torch.no_grad():
        ref = m(torch.tensor([toks])).logits[0].double().numpy()       # [T][V]
    model = orc.Model(shape, wnp, round_kv=False)
    kv = model.new_cache()
    kv32 = np.zeros(kv.size, dtype=np.float32)
    for t, tok in enumerate(toks):
        logits, nxt, _ = model.decode_step(tok, t, kv, kv_f32=kv32)
        assert rel_l2(logits, ref[t]) < 1e-5, t
    assert not kv.any()                                               # the bf16 cache is untouched in this mode
