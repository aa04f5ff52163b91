"""Pins for the CPU oracle's pieces: each test checks the oracle against something it does not compute
itself -- a closed form, a hand value, an invariant, an exhaustive integer round trip, or an
independent library routine (numpy float16, torch bfloat16)."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_numbers.txt")


def bf16_bits(x):
    """bf16 bit patterns through torch's own conversion (independent of the oracle's)."""
    t = torch.tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def bf16_val(bits):
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


ONE = bf16_bits([1.0])[0]


# ------------------------------------------------------------------------------------------------
# 16-bit formats
# ------------------------------------------------------------------------------------------------

def test_f16_to_f32_exhaustive_vs_numpy():
    allbits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    ref = allbits.view(np.float16).astype(np.float32)
    got = orc.f16_to_f32(allbits)
    same = (got.view(np.uint32) == ref.view(np.uint32)) | (np.isnan(got) & np.isnan(ref))
    assert same.all()


def test_bf16_to_f32_exhaustive_vs_torch():
    allbits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    ref = torch.from_numpy(allbits.view(np.int16)).view(torch.bfloat16).float().numpy()
    got = orc.bf16_to_f32(allbits)
    same = (got.view(np.uint32) == ref.view(np.uint32)) | (np.isnan(got) & np.isnan(ref))
    assert same.all()


def _f32_samples():
    rng = np.random.default_rng(1)
    x = np.concatenate([
        rng.standard_normal(20000).astype(np.float32) * np.float32(0.02),
        rng.standard_normal(20000).astype(np.float32) * np.float32(100.0),
        (rng.standard_normal(5000) * 1e-6).astype(np.float32),             # fp16 subnormal range
        np.array([0.0, -0.0, 1.0, -1.0, 65504.0, 65519.9, 65520.0, 70000.0, 2.0 ** -24, 2.0 ** -25,
                  1.5 * 2.0 ** -25, 2.0 ** -14, 6.1e-5, np.inf, -np.inf], dtype=np.float32),
        # exact ties: 1 + (2k+1) * 2^-11 sits halfway between two fp16 values; 1 + (2k+1)*2^-8 between two bf16
        (1.0 + (2 * np.arange(64) + 1) * 2.0 ** -11).astype(np.float32),
        (1.0 + (2 * np.arange(64) + 1) * 2.0 ** -8).astype(np.float32),
    ])
    return x


def test_f32_to_f16_vs_numpy():
    x = _f32_samples()
    with np.errstate(over="ignore"):
        ref = x.astype(np.float16).view(np.uint16)
    assert np.array_equal(orc.f32_to_f16(x), ref)


def test_f32_to_bf16_vs_torch():
    x = _f32_samples()
    assert np.array_equal(orc.f32_to_bf16(x), bf16_bits(x))


# ------------------------------------------------------------------------------------------------
# RMSNorm
# ------------------------------------------------------------------------------------------------

def test_rmsnorm_hand_values():
    g = np.full(2, ONE, dtype=np.uint16)
    out = orc.rmsnorm([3.0, 4.0], g, 0.0)                   # mean square 12.5 -> [3, 4] / sqrt(12.5)
    assert np.allclose(out, [0.8485281, 1.1313708], rtol=0, atol=2e-7)
    out = orc.rmsnorm([3.0, 4.0], g, 1e-5)
    assert abs(out[0] - 3.0 / math.sqrt(12.5 + 1e-5)) < 1e-7
    assert abs(out[0] - 0.8485278) < 2e-7


def test_rmsnorm_constant_vector_closed_form():
    H, c, eps = 96, 0.37, 1e-5
    gvals = np.linspace(0.5, 1.5, H).astype(np.float32)
    g = bf16_bits(gvals)
    out = orc.rmsnorm(np.full(H, c, dtype=np.float32), g, eps)
    expect = np.float32(c) / math.sqrt(float(np.float32(c)) ** 2 + eps) * bf16_val(g).astype(np.float64)
    assert np.allclose(out, expect, rtol=2e-7, atol=0)


def test_rmsnorm_unit_weight_mean_square_and_scale_invariance():
    rng = np.random.default_rng(2)
    H, eps = 576, 1e-5
    x = rng.standard_normal(H).astype(np.float32)
    g = np.full(H, ONE, dtype=np.uint16)
    a = orc.rmsnorm(x, g, eps).astype(np.float64)
    ms = float(np.mean(x.astype(np.float64) ** 2))
    assert abs(np.mean(a ** 2) - ms / (ms + eps)) < 1e-6          # mean(a^2) = ms / (ms + eps)
    b = orc.rmsnorm(7.0 * x, g, 0.0)
    a0 = orc.rmsnorm(x, g, 0.0)
    assert np.allclose(a0, b, rtol=3e-7, atol=0)                   # a(alpha x) = a(x) when eps = 0


# ------------------------------------------------------------------------------------------------
# RoPE
# ------------------------------------------------------------------------------------------------

def test_rope_pos0_is_identity_bit_for_bit():
    rng = np.random.default_rng(3)
    u = rng.standard_normal(64).astype(np.float32)
    assert np.array_equal(orc.rope(u, 0, 10000.0).view(np.uint32), u.view(np.uint32))


def test_rope_hand_values():
    # hd = 2: one pair, frequency 1, position 1: (1, 0) -> (cos 1, sin 1)
    out = orc.rope([1.0, 0.0], 1, 123.0)
    assert np.allclose(out, [0.5403023, 0.8414710], atol=1e-7)
    # hd = 4, theta = 1e4, pos = 3: pairs (0,2) and (1,3) with frequencies 1 and 0.01
    out = orc.rope([1.0, 2.0, 3.0, 4.0], 3, 10000.0)
    c0, s0, c1, s1 = math.cos(3.0), math.sin(3.0), math.cos(0.03), math.sin(0.03)
    expect = [1 * c0 - 3 * s0, 2 * c1 - 4 * s1, 3 * c0 + 1 * s0, 4 * c1 + 2 * s1]
    assert np.allclose(out, expect, atol=1e-6)
    assert np.allclose(out, [-1.4133525, 1.8791181, -2.8288575, 4.0581911], atol=1e-6)


def test_rope_preserves_pair_norms_and_relative_angle():
    rng = np.random.default_rng(4)
    hd = 128
    q = rng.standard_normal(hd).astype(np.float32)
    k = rng.standard_normal(hd).astype(np.float32)
    for pos in (1, 17, 4095):
        r = orc.rope(q, pos, 500000.0).astype(np.float64)
        n0 = q[:hd // 2].astype(np.float64) ** 2 + q[hd // 2:].astype(np.float64) ** 2
        n1 = r[:hd // 2] ** 2 + r[hd // 2:] ** 2
        assert np.allclose(n0, n1, rtol=1e-6)
    # <R_m q, R_n k> depends on m - n only
    d1 = float(np.dot(orc.rope(q, 10, 1e4).astype(np.float64), orc.rope(k, 3, 1e4).astype(np.float64)))
    d2 = float(np.dot(orc.rope(q, 110, 1e4).astype(np.float64), orc.rope(k, 103, 1e4).astype(np.float64)))
    assert abs(d1 - d2) < 1e-4


def test_rope_distinguishes_half_split_from_interleaved():
    # unit vector on dim 1: half-split pairs it with dim 1 + hd/2 at frequency theta^(-2/hd);
    # an interleaved convention would pair it with dim 0 at frequency 1.
    hd, theta, pos = 8, 10000.0, 5
    u = np.zeros(hd, dtype=np.float32)
    u[1] = 1.0
    out = orc.rope(u, pos, theta)
    phi = pos * theta ** (-2.0 / hd)
    expect = np.zeros(hd)
    expect[1], expect[1 + hd // 2] = math.cos(phi), math.sin(phi)
    assert np.allclose(out, expect, atol=1e-7)


# ------------------------------------------------------------------------------------------------
# softmax attention and the split-K combine
# ------------------------------------------------------------------------------------------------

def test_attention_hand_value_and_split_combine():
    # one head, hd = 1, q = 1: scores = K / sqrt(1).  K = [0, ln2, ln3, 0], V = [1,2,3,4]
    # (K and V chosen exactly representable or rounded first) -> weights [1,2,3,1]/7, output 18/7.
    K = bf16_bits([0.0, math.log(2.0), math.log(3.0), 0.0]).reshape(4, 1)
    V = bf16_bits([1.0, 2.0, 3.0, 4.0]).reshape(4, 1)
    kv = bf16_val(K).astype(np.float64).ravel()
    w_expect = np.exp(kv) / np.exp(kv).sum()
    o, w = orc.attention_head([1.0], K, V, 0, 4, want_weights=True)
    assert abs(w.sum() - 1.0) < 1e-12
    assert np.allclose(w, w_expect, atol=1e-12)
    assert np.allclose(w, [1 / 7, 2 / 7, 3 / 7, 1 / 7], atol=2e-3)       # bf16(ln2), bf16(ln3) are 3-digit values
    assert abs(o[0] - float((w_expect * [1, 2, 3, 4]).sum())) < 1e-6
    assert abs(o[0] - 18 / 7) < 5e-3
    p0 = orc.attention_partial([1.0], K, V, 0, 2)
    p1 = orc.attention_partial([1.0], K, V, 2, 4)
    oc = orc.attention_combine([p0[0], p1[0]], [p0[1], p1[1]], [p0[2], p1[2]])
    assert abs(oc[0] - o[0]) < 1e-7


def test_attention_single_position_returns_v_exactly():
    rng = np.random.default_rng(5)
    hd = 64
    q = rng.standard_normal(hd).astype(np.float32) * 5
    K = bf16_bits(rng.standard_normal((1, hd)))
    V = bf16_bits(rng.standard_normal((1, hd)))
    o = orc.attention_head(q, K, V, 0, 1)
    assert np.array_equal(o.view(np.uint32), bf16_val(V).ravel().view(np.uint32))


def test_attention_equal_keys_gives_mean_and_dominant_key_gives_its_row():
    rng = np.random.default_rng(6)
    hd, n = 16, 9
    q = rng.standard_normal(hd).astype(np.float32)
    krow = bf16_bits(rng.standard_normal(hd))
    K = np.tile(krow, (n, 1))
    V = bf16_bits(rng.standard_normal((n, hd)))
    o, w = orc.attention_head(q, K, V, 0, n, want_weights=True)
    assert np.allclose(w, 1.0 / n, atol=1e-15)
    assert np.allclose(o, bf16_val(V).astype(np.float64).mean(axis=0), atol=1e-6)
    # one key aligned with q and scaled so its score exceeds the rest by > 50
    K2 = np.zeros((n, hd), dtype=np.uint16)
    qn = q / np.linalg.norm(q)
    K2[4] = bf16_bits(qn * 60.0 * math.sqrt(hd) / np.linalg.norm(q))
    o2 = orc.attention_head(q, K2, V, 0, n)
    assert np.allclose(o2, bf16_val(V)[4], atol=1e-6)


@pytest.mark.parametrize("chunk", [1, 7, 64, 200])
def test_split_k_combine_equals_unsplit(chunk):
    rng = np.random.default_rng(7)
    hd, n = 32, 200
    q = rng.standard_normal(hd).astype(np.float32)
    K = bf16_bits(rng.standard_normal((n, hd)))
    V = bf16_bits(rng.standard_normal((n, hd)))
    full = orc.attention_head(q, K, V, 0, n)
    parts = [orc.attention_partial(q, K, V, a, min(n, a + chunk)) for a in range(0, n, chunk)]
    comb = orc.attention_combine([p[0] for p in parts], [p[1] for p in parts], [p[2] for p in parts])
    assert np.allclose(comb, full, atol=1e-6, rtol=1e-6)


def test_attention_respects_range_bounds():
    rng = np.random.default_rng(8)
    hd, n = 16, 12
    q = rng.standard_normal(hd).astype(np.float32)
    K = bf16_bits(rng.standard_normal((n, hd)))
    V = bf16_bits(rng.standard_normal((n, hd)))
    a = orc.attention_head(q, K, V, 0, 5)
    b = orc.attention_head(q, K[:5].copy(), V[:5].copy(), 0, 5)
    assert np.array_equal(a, b)
    Kf, Vf = bf16_val(K).astype(np.float64), bf16_val(V).astype(np.float64)
    s = Kf[:5] @ q.astype(np.float64) / math.sqrt(hd)
    w = np.exp(s - s.max())
    w /= w.sum()
    assert np.allclose(a, w @ Vf[:5], atol=1e-6)


# ------------------------------------------------------------------------------------------------
# GEMV, SiLU, argmax
# ------------------------------------------------------------------------------------------------

def test_gemv_exact_integer_cases():
    rng = np.random.default_rng(9)
    rows, cols = 13, 40
    x = rng.integers(-8, 9, size=cols).astype(np.float32)
    # identity-like: row o selects column o
    W = np.zeros((rows, cols), dtype=np.float32)
    for o in range(rows):
        W[o, (3 * o) % cols] = 1.0
    y = orc.gemv(orc.W_BF16, bf16_bits(W), x)
    assert np.array_equal(y, x[[(3 * o) % cols for o in range(rows)]])
    # +-1 matrix: exact integer dot products; a transposed operand or dropped column would change them
    Wpm = rng.choice([-1.0, 1.0], size=(rows, cols)).astype(np.float32)
    y = orc.gemv(orc.W_BF16, bf16_bits(Wpm), x)
    assert np.array_equal(y, (Wpm.astype(np.int64) @ x.astype(np.int64)).astype(np.float32))
    # int8 with scale 2^-3 and int4 with scale 2^-2, zero 5: still exact
    q8 = rng.integers(-127, 128, size=(rows, cols)).astype(np.int8)
    s8 = np.full(rows, np.float16(0.125).view(np.uint16), dtype=np.uint16)
    y = orc.gemv(orc.W_INT8, q8, x, scale=s8)
    assert np.array_equal(y, (q8.astype(np.int64) @ x.astype(np.int64)).astype(np.float32) * 0.125)
    cols4, group = 64, 32
    x4 = rng.integers(-8, 9, size=cols4).astype(np.float32)
    q4 = rng.integers(0, 16, size=(rows, cols4)).astype(np.uint8)
    packed = (q4[:, 0::2] | (q4[:, 1::2] << 4)).astype(np.uint8)
    s4 = np.full((rows, cols4 // group), np.float16(0.25).view(np.uint16), dtype=np.uint16)
    zvals = rng.integers(0, 16, size=(rows, cols4 // group))
    z4 = zvals.astype(np.float16).view(np.uint16)
    y = orc.gemv(orc.W_INT4, packed, x4, scale=s4, zero=z4, group=group)
    ref = ((q4.astype(np.int64) - np.repeat(zvals, group, axis=1)) * x4.astype(np.int64)).sum(axis=1) * 0.25
    assert np.array_equal(y, ref.astype(np.float32))
    assert np.array_equal(orc.unpack_int4(packed), q4)
    # grouped int8: a different power-of-two scale per (row, group); a scale taken from the wrong row or group, or
    # applied per row, changes the integers
    ng = cols4 // group
    q8g = rng.integers(-127, 128, size=(rows, cols4)).astype(np.int8)
    exps = rng.integers(-6, 3, size=(rows, ng))
    s8g = (2.0 ** exps).astype(np.float16).view(np.uint16)
    y = orc.gemv(orc.W_INT8G, q8g, x4, scale=s8g, group=group)
    ref = ((q8g.astype(np.int64) * x4.astype(np.int64)).reshape(rows, ng, group).sum(axis=2) * 2.0 ** exps).sum(axis=1)
    assert np.array_equal(y, ref.astype(np.float32))


def test_silu_values():
    assert orc.silu(0.0) == 0.0
    assert abs(orc.silu(1.0) - 0.7310586) < 1e-7
    assert abs(orc.silu(-1.0) + 0.2689414) < 1e-7
    for z in (0.3, 2.5, 11.0):
        assert abs((orc.silu(z) - orc.silu(-z)) - z) < 1e-6          # silu(z) - silu(-z) = z
    assert abs(orc.silu(40.0) - 40.0) < 1e-6 and abs(orc.silu(-40.0)) < 1e-12


def test_argmax_lowest_index_on_tie():
    v = np.array([0.5, 2.0, -1.0, 2.0, 2.0, 1.0], dtype=np.float32)
    assert orc.argmax(v) == 1
    assert orc.argmax(np.array([-3.0, -3.0], dtype=np.float32)) == 0


# ------------------------------------------------------------------------------------------------
# quantisers
# ------------------------------------------------------------------------------------------------

def test_int4_pack_unpack_all_byte_values():
    allb = np.arange(256, dtype=np.uint8).reshape(1, 256)
    codes = orc.unpack_int4(allb)
    assert np.array_equal(codes[0, 0::2], np.arange(256) & 15)
    assert np.array_equal(codes[0, 1::2], np.arange(256) >> 4)
    # oracle's own dequant reads the same nibble order: scale 1, zero 0 -> value = code
    s = np.full((1, 4), np.float16(1.0).view(np.uint16), dtype=np.uint16)
    z = np.zeros((1, 4), dtype=np.uint16)
    d = orc.dequant(orc.W_INT4, allb, s, z, group=128)
    assert np.array_equal(d[0], codes[0].astype(np.float32))


def test_int8_quantiser_hand_row():
    W = np.array([[0x3DCD, 0xBD4D, 0x3CCD, 0x0000]], dtype=np.uint16)   # 0.10009766 -0.05004883 0.02502441 0
    q, s = orc.quantize_int8(W)
    assert s[0] == 0x1275                                              # fp16(0.10009766 / 127)
    assert q.tolist() == [[127, -63, 32, 0]]
    d = orc.dequant(orc.W_INT8, q, s)
    assert np.allclose(d[0], [0.10010290, -0.04965734, 0.02522278, 0.0], atol=1e-8)


def test_grouped_int8_quantiser_hand_groups():
    # two groups of four with very different ranges: each gets the per-row rule on its own
    W = np.array([[0x3DCD, 0xBD4D, 0x3CCD, 0x0000, 0x3A83, 0xBA03, 0x0000, 0x3983]], dtype=np.uint16)
    q, s = orc.quantize_int8_grouped(W, group=4)
    assert s.shape == (1, 2) and s[0, 0] == 0x1275                     # fp16(0.10009766 / 127), as the per-row pin
    assert q[0, :4].tolist() == [127, -63, 32, 0]
    # second group: 0x3A83 = 0.0010004044 is its maximum -> code 127; half of it -> -63 or -64; a quarter -> 32
    assert q[0, 4] == 127 and q[0, 5] in (-63, -64) and q[0, 6] == 0 and q[0, 7] in (31, 32)
    assert s[0, 1] == np.float16(np.float32(0.0010004044) / np.float32(127)).view(np.uint16)
    d = orc.dequant(orc.W_INT8G, q, s, group=4)
    assert np.allclose(d[0, :4], [0.10010290, -0.04965734, 0.02522278, 0.0], atol=1e-8)


def test_int4_quantiser_hand_group():
    vals = np.array([[-0.03002930, 0.0, 0.01501465, 0.04492188]], dtype=np.float32)
    W = bf16_bits(vals)
    p, s, z = orc.quantize_int4(W, group=4)
    assert s[0, 0] == 0x1D1E                                           # fp16((mx - mn) / 15)
    assert np.float16(6.0).view(np.uint16) == z[0, 0]
    assert p.tolist() == [[0x60, 0xF9]]                                # codes 0,6 | 9,15
    d = orc.dequant(orc.W_INT4, p, s, z, group=4)
    assert np.allclose(d[0], [-0.02998352, 0.0, 0.01499176, 0.04497528], atol=1e-8)


def test_quantisers_vs_numpy_float16_and_error_bounds():
    rng = np.random.default_rng(10)
    rows, cols, group = 24, 256, 128
    Wf = (rng.standard_normal((rows, cols)) * 0.02).astype(np.float32)
    Wf[3] = 0.0                                                         # all-zero row -> scale 1
    Wf[5, :128] = np.abs(Wf[5, :128])                                   # all-positive group -> zero point 0
    W = bf16_bits(Wf)
    Wv = bf16_val(W)
    q, s = orc.quantize_int8(W)
    amax = np.abs(Wv).max(axis=1)
    s_ref = np.where(amax == 0, np.float16(1.0), (amax / np.float32(127)).astype(np.float16))
    assert np.array_equal(s, s_ref.view(np.uint16))
    sf = s_ref.astype(np.float32)
    assert np.array_equal(q, np.clip(np.rint(Wv / sf[:, None]), -127, 127).astype(np.int8))
    d = orc.dequant(orc.W_INT8, q, s)
    assert (np.abs(d - Wv) <= sf[:, None] * 0.5 * (1 + 1e-6)).all()
    # grouped int8: the per-row rule per (row, group); with one group per row it IS the per-row quantiser
    qg, sg = orc.quantize_int8_grouped(W, group)
    Wg = Wv.reshape(rows, cols // group, group)
    amaxg = np.abs(Wg).max(axis=2)
    sg_ref = np.where(amaxg == 0, np.float16(1.0), (amaxg / np.float32(127)).astype(np.float16))
    assert np.array_equal(sg, sg_ref.view(np.uint16))
    sgf = sg_ref.astype(np.float32)
    assert np.array_equal(qg.reshape(Wg.shape), np.clip(np.rint(Wg / sgf[:, :, None]), -127, 127).astype(np.int8))
    dg = orc.dequant(orc.W_INT8G, qg, sg, group=group).reshape(Wg.shape)
    assert (np.abs(dg - Wg) <= sgf[:, :, None] * 0.5 * (1 + 1e-6)).all()
    q1, s1 = orc.quantize_int8_grouped(W, cols)
    assert np.array_equal(q1, q) and np.array_equal(s1[:, 0], s)
    p, s4, z4 = orc.quantize_int4(W, group)
    codes = orc.unpack_int4(p)
    mn = np.minimum(Wg.min(axis=2), 0)
    mx = np.maximum(Wg.max(axis=2), 0)
    s4_ref = np.where(mx == mn, np.float16(1.0), ((mx - mn) / np.float32(15)).astype(np.float16))
    assert np.array_equal(s4, s4_ref.view(np.uint16))
    s4f = s4_ref.astype(np.float32)
    z_ref = np.clip(np.rint(-mn / s4f), 0, 15)
    assert np.array_equal(orc.f16_to_f32(z4), z_ref.astype(np.float32))
    c_ref = np.clip(np.rint(Wg / s4f[:, :, None]) + z_ref[:, :, None], 0, 15).astype(np.uint8)
    assert np.array_equal(codes.reshape(rows, cols // group, group), c_ref)
    assert z_ref[5, 0] == 0
    # bit patterns, not only values: a zero point of an all-positive group is -mn / s = -0.0 before the clamp and
    # is stored as +0 (0x0000); no stored zero point ever carries a sign bit
    assert z4[5, 0] == 0x0000
    assert not (z4 & 0x8000).any()
    d4 = orc.dequant(orc.W_INT4, p, s4, z4, group).reshape(rows, cols // group, group)
    # inside the representable range the error is at most half a step (plus the zero point's own rounding)
    assert (np.abs(d4 - Wg) <= s4f[:, :, None] * 1.0 * (1 + 1e-6)).all()
    inside = (np.rint(Wg / s4f[:, :, None]) + z_ref[:, :, None] >= 0) & (np.rint(Wg / s4f[:, :, None]) + z_ref[:, :, None] <= 15)
    assert (np.abs(d4 - Wg)[inside] <= s4f[:, :, None].repeat(group, axis=2)[inside] * 0.5 * (1 + 1e-6)).all()


# ------------------------------------------------------------------------------------------------
# shapes and byte accounting against the numbers the paper prints
# ------------------------------------------------------------------------------------------------

def _golden():
    out = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v, tol = line.split()[:3]
            out[k] = (float(v), float(tol))
    return out


def test_parameter_counts_and_byte_ratios_match_paper():
    from paper_2606_09682_b200.inputs import SHAPES, streamed_bytes
    g = _golden()
    smol, tiny = SHAPES["smollm2_135m"], SHAPES["tinyllama_1b"]
    assert smol.n_params() == 134_515_008 and tiny.n_params() == 1_100_048_384
    v, tol = g["smollm2_135m_params_M"]
    assert abs(smol.n_params() / 1e6 - v) <= tol
    v, tol = g["tinyllama_1b_params_M"]
    assert abs(tiny.n_params() / 1e6 - v) <= tol
    v, tol = g["smollm2_135m_fp32_MB"]
    assert abs(smol.n_params() * 4 / 1e6 - v) <= tol
    v, tol = g["llama32_1b_bf16_MB"]
    assert abs(SHAPES["llama32_1b"].n_params() * 2 / 1e6 - v) <= tol
    v, tol = g["paper_small_bf16_MB"]
    assert abs(SHAPES["paper_small"].n_params() * 2 / 1e6 - v) <= tol

    def wbytes(dt):
        b = streamed_bytes(smol, dt, 0)
        return b["weights"] + b["scales"]
    r8, r4 = wbytes("int8") / wbytes("bf16"), wbytes("int4") / wbytes("bf16")
    v, tol = g["int8_byte_ratio"]
    assert abs(r8 - v) <= tol
    v, tol = g["int4_byte_ratio"]
    assert abs(r4 - v) <= tol
    v, tol = g["int4_floor_drop"]
    assert abs(1 / r4 - v) <= tol


def test_streamed_bytes_table():
    from paper_2606_09682_b200.inputs import SHAPES, streamed_bytes
    b = streamed_bytes(SHAPES["tinyllama_1b"], "bf16", 0)
    assert abs((b["weights"] + b["scales"]) / 1e6 - 2069.03) < 0.01
    b = streamed_bytes(SHAPES["llama3_8b"], "int8", 4096)
    assert abs((b["weights"] + b["scales"]) / 1e6 - 8033.29) < 0.01
    assert abs(2.0 * 32 * 8 * 128 * 2 * 4096 / 1e6 - 536.87) < 0.01


# ------------------------------------------------------------------------------------------------
# fp8 e4m3 (the element type of the optional 8-bit KV cache)
# ------------------------------------------------------------------------------------------------

def test_e4m3_to_f32_exhaustive_vs_torch():
    codes = np.arange(256, dtype=np.uint8)
    ours = orc.e4m3_to_f32(codes)
    ref = torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn).to(torch.float32).numpy()
    nan = np.isnan(ref)
    assert nan.sum() == 2 and nan[0x7F] and nan[0xFF] and np.isnan(ours[nan]).all()
    assert np.array_equal(ours[~nan].view(np.uint32), ref[~nan].view(np.uint32))       # bit for bit, -0 included
    assert ours[0x7E] == 448.0 and ours[0x01] == 2.0 ** -9 and ours[0x08] == 2.0 ** -6


def test_f32_to_e4m3_vs_torch_ties_and_saturation():
    rng = np.random.default_rng(77)
    vals = [rng.standard_normal(20000).astype(np.float32) * s for s in (1e-3, 1e-2, 1.0, 30.0, 200.0)]
    # every representable value, every midpoint between neighbours (ties), and values a hair to either side
    rep = orc.e4m3_to_f32(np.arange(0x7F, dtype=np.uint8)).astype(np.float64)
    mid = (rep[:-1] + rep[1:]) / 2
    edge = np.concatenate([rep, mid, mid * (1 + 1e-6), mid * (1 - 1e-6)]).astype(np.float32)
    x = np.concatenate(vals + [edge, -edge, np.array([0.0, -0.0], dtype=np.float32)])
    x = x[np.abs(x) <= 464.0]                         # beyond the tie above 448 torch gives NaN, the contract here saturates
    ours = orc.f32_to_e4m3(x)
    ref = torch.from_numpy(x.copy()).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(ours, ref)
    # round trip of every finite code, ties to even at hand-worked midpoints, saturation, NaN
    codes = np.array([c for c in range(256) if (c & 0x7F) != 0x7F], dtype=np.uint8)
    assert np.array_equal(orc.f32_to_e4m3(orc.e4m3_to_f32(codes)), codes)
    assert orc.f32_to_e4m3(np.float32(2.0 ** -10))[()] == 0x00            # half the smallest subnormal: tie -> even (0)
    assert orc.f32_to_e4m3(np.float32(3 * 2.0 ** -10))[()] == 0x02        # 1.5 subnormal steps: tie -> even (2)
    assert orc.f32_to_e4m3(np.float32(1.0625))[()] == 0x38                # 1 + 1/16: tie between 1.0 and 1.125 -> 1.0
    assert orc.f32_to_e4m3(np.float32(1.1875))[()] == 0x3A                # tie between 1.125 and 1.25 -> 1.25 (even)
    assert orc.f32_to_e4m3(np.float32(464.0))[()] == 0x7E and orc.f32_to_e4m3(np.float32(465.0))[()] == 0x7E
    assert orc.f32_to_e4m3(np.float32(1e30))[()] == 0x7E and orc.f32_to_e4m3(np.float32(-np.inf))[()] == 0xFE
    assert orc.f32_to_e4m3(np.float32(np.nan))[()] & 0x7F == 0x7F
