"""ctypes/numpy front end of the CPU oracle (``oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the benchmark's CPU-baseline
leg.  The CUDA library and its Python binding never import this module, and it never imports them.

All 16-bit floating-point data crosses this boundary as ``numpy.uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

KINDS = ("wq", "wk", "wv", "wo", "wgate", "wup", "wdown")
W_BF16, W_INT8, W_INT4, W_INT8G = 0, 1, 2, 3
KV_BF16, KV_E4M3 = 0, 1      # cache element type; the cache array holds 16-bit words either way (an e4m3 code in the low byte)


def build(force: bool = False) -> str:
    """Compile ``oracle.c`` with gcc (OpenMP, no fast-math, no contraction) if it is stale."""
    if (not force) and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC):
        return _LIB
    cmd = ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
           "-fno-fast-math", "-o", _LIB, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return _LIB


class _Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("hidden", "n_layers", "n_q_heads", "n_kv_heads", "head_dim",
                                         "mlp", "vocab", "max_seq", "tied_embeddings")] + [
        ("rms_eps", C.c_float), ("rope_theta", C.c_float),
        ("wdtype", C.c_int32), ("group_size", C.c_int32), ("round_kv", C.c_int32), ("quantize_lm_head", C.c_int32),
        ("kv_dtype", C.c_int32)]


_PP = C.POINTER(C.c_void_p)


class _Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p),
                ("attn_norm", _PP), ("mlp_norm", _PP),
                ("w", _PP * 7), ("scale", _PP * 7), ("zero", _PP * 7),
                ("lm_head_q", C.c_void_p), ("lm_head_scale", C.c_void_p), ("lm_head_zero", C.c_void_p)]


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        L = _lib
        L.orc_bf16_to_f32.restype = C.c_float
        L.orc_bf16_to_f32.argtypes = [C.c_uint16]
        L.orc_f32_to_bf16.restype = C.c_uint16
        L.orc_f32_to_bf16.argtypes = [C.c_float]
        L.orc_f16_to_f32.restype = C.c_float
        L.orc_f16_to_f32.argtypes = [C.c_uint16]
        L.orc_f32_to_f16.restype = C.c_uint16
        L.orc_f32_to_f16.argtypes = [C.c_float]
        L.orc_e4m3_to_f32.restype = C.c_float
        L.orc_e4m3_to_f32.argtypes = [C.c_uint8]
        L.orc_f32_to_e4m3.restype = C.c_uint8
        L.orc_f32_to_e4m3.argtypes = [C.c_float]
        L.orc_silu.restype = C.c_float
        L.orc_silu.argtypes = [C.c_float]
        L.orc_argmax.restype = C.c_int
        L.orc_dequant.restype = C.c_float
        L.orc_num_threads.restype = C.c_int
        L.orc_decode_step.restype = C.c_int
        L.orc_layer_step.restype = C.c_int
        L.orc_decode_step_rows.restype = C.c_int
        L.orc_layer_step_rows.restype = C.c_int
        L.orc_head_step.restype = C.c_int
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _c(a, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


# ------------------------------------------------------------------------------------------------
# scalar / vector pieces
# ------------------------------------------------------------------------------------------------

def bf16_to_f32(bits) -> np.ndarray:
    b = np.asarray(bits, dtype=np.uint16)
    out = np.empty(b.shape, dtype=np.float32)
    f = lib().orc_bf16_to_f32
    flat_in, flat_out = b.ravel(), out.ravel()
    for i in range(flat_in.size):
        flat_out[i] = f(int(flat_in[i]))
    return out


def f32_to_bf16(x) -> np.ndarray:
    v = np.asarray(x, dtype=np.float32)
    out = np.empty(v.shape, dtype=np.uint16)
    f = lib().orc_f32_to_bf16
    fi, fo = v.ravel(), out.ravel()
    for i in range(fi.size):
        fo[i] = f(float(fi[i]))
    return out


def e4m3_to_f32(codes) -> np.ndarray:
    b = np.asarray(codes, dtype=np.uint8)
    out = np.empty(b.shape, dtype=np.float32)
    f = lib().orc_e4m3_to_f32
    fi, fo = b.ravel(), out.ravel()
    for i in range(fi.size):
        fo[i] = f(int(fi[i]))
    return out


def f32_to_e4m3(x) -> np.ndarray:
    v = np.asarray(x, dtype=np.float32)
    out = np.empty(v.shape, dtype=np.uint8)
    f = lib().orc_f32_to_e4m3
    fi, fo = v.ravel(), out.ravel()
    for i in range(fi.size):
        fo[i] = f(float(fi[i]))
    return out


def f16_to_f32(bits) -> np.ndarray:
    b = np.asarray(bits, dtype=np.uint16)
    out = np.empty(b.shape, dtype=np.float32)
    f = lib().orc_f16_to_f32
    fi, fo = b.ravel(), out.ravel()
    for i in range(fi.size):
        fo[i] = f(int(fi[i]))
    return out


def f32_to_f16(x) -> np.ndarray:
    v = np.asarray(x, dtype=np.float32)
    out = np.empty(v.shape, dtype=np.uint16)
    f = lib().orc_f32_to_f16
    fi, fo = v.ravel(), out.ravel()
    for i in range(fi.size):
        fo[i] = f(float(fi[i]))
    return out


def rmsnorm(x, g_bf16, eps: float) -> np.ndarray:
    x = _c(x, np.float32)
    g = _c(g_bf16, np.uint16)
    out = np.empty_like(x)
    lib().orc_rmsnorm(_p(x), _p(g), C.c_int(x.size), C.c_float(eps), _p(out))
    return out


def rope(u, pos: int, theta: float) -> np.ndarray:
    u = _c(u, np.float32).copy()
    lib().orc_rope(_p(u), C.c_int(u.size), C.c_int(pos), C.c_double(theta))
    return u


def silu(z: float) -> float:
    return float(lib().orc_silu(C.c_float(z)))


def argmax(v) -> int:
    v = _c(v, np.float32)
    return int(lib().orc_argmax(_p(v), C.c_int(v.size)))


def gemv(wdtype: int, W, x, scale=None, zero=None, group: int = 128) -> np.ndarray:
    """y = deq(W) x.  W: uint16 [rows][cols] (bf16 bits), int8 [rows][cols] (per-row or grouped scales) or uint8
    [rows][cols/2]."""
    x = _c(x, np.float32)
    cols = x.size
    if wdtype == W_BF16:
        W = _c(W, np.uint16)
    elif wdtype in (W_INT8, W_INT8G):
        W = _c(W, np.int8)
    else:
        W = _c(W, np.uint8)
    rows = W.shape[0]
    scale = None if scale is None else _c(scale, np.uint16)
    zero = None if zero is None else _c(zero, np.uint16)
    y = np.empty(rows, dtype=np.float32)
    lib().orc_gemv(C.c_int(wdtype), _p(W), _p(scale), _p(zero), C.c_int(group), C.c_int(rows), C.c_int(cols),
                   _p(x), _p(y))
    return y


def dequant(wdtype: int, W, scale=None, zero=None, group: int = 128) -> np.ndarray:
    """Dense fp32 matrix of dequantised weights (small matrices only: one call per element)."""
    if wdtype == W_BF16:
        W = _c(W, np.uint16)
        rows, cols = W.shape
    elif wdtype in (W_INT8, W_INT8G):
        W = _c(W, np.int8)
        rows, cols = W.shape
    else:
        W = _c(W, np.uint8)
        rows, cols = W.shape[0], W.shape[1] * 2
    scale = None if scale is None else _c(scale, np.uint16)
    zero = None if zero is None else _c(zero, np.uint16)
    out = np.empty((rows, cols), dtype=np.float32)
    f = lib().orc_dequant
    for o in range(rows):
        for j in range(cols):
            out[o, j] = f(C.c_int(wdtype), _p(W), _p(scale), _p(zero), C.c_int(group), C.c_int(cols),
                          C.c_int(o), C.c_int(j))
    return out


def quantize_int8(W_bf16):
    W = _c(W_bf16, np.uint16)
    rows, cols = W.shape
    q = np.empty((rows, cols), dtype=np.int8)
    s = np.empty(rows, dtype=np.uint16)
    lib().orc_quantize_int8(_p(W), C.c_int(rows), C.c_int(cols), _p(q), _p(s))
    return q, s


def quantize_int8_grouped(W_bf16, group: int = 128):
    W = _c(W_bf16, np.uint16)
    rows, cols = W.shape
    assert cols % group == 0
    q = np.empty((rows, cols), dtype=np.int8)
    s = np.empty((rows, cols // group), dtype=np.uint16)
    lib().orc_quantize_int8_grouped(_p(W), C.c_int(rows), C.c_int(cols), C.c_int(group), _p(q), _p(s))
    return q, s


def quantize_int4(W_bf16, group: int = 128):
    W = _c(W_bf16, np.uint16)
    rows, cols = W.shape
    assert cols % group == 0 and cols % 2 == 0
    packed = np.zeros((rows, cols // 2), dtype=np.uint8)
    s = np.empty((rows, cols // group), dtype=np.uint16)
    z = np.empty((rows, cols // group), dtype=np.uint16)
    lib().orc_quantize_int4(_p(W), C.c_int(rows), C.c_int(cols), C.c_int(group), _p(packed), _p(s), _p(z))
    return packed, s, z


def unpack_int4(packed) -> np.ndarray:
    """Integer codes 0..15, element j of a row taken from byte j//2 (even j: low nibble)."""
    p = np.asarray(packed, dtype=np.uint8)
    out = np.empty(p.shape[:-1] + (p.shape[-1] * 2,), dtype=np.uint8)
    out[..., 0::2] = p & 0x0F
    out[..., 1::2] = p >> 4
    return out


def attention_head(q, K_bf16, V_bf16, j0: int, j1: int, want_weights: bool = False):
    q = _c(q, np.float32)
    K = _c(K_bf16, np.uint16)
    V = _c(V_bf16, np.uint16)
    hd = q.size
    o = np.empty(hd, dtype=np.float32)
    w = np.empty(j1 - j0, dtype=np.float64) if want_weights else None
    lib().orc_attention_head(_p(q), _p(K), _p(V), C.c_int(hd), C.c_int(j0), C.c_int(j1), _p(o), _p(w))
    return (o, w) if want_weights else o


def attention_partial(q, K_bf16, V_bf16, j0: int, j1: int):
    q = _c(q, np.float32)
    K = _c(K_bf16, np.uint16)
    V = _c(V_bf16, np.uint16)
    hd = q.size
    m = C.c_double()
    l = C.c_double()
    acc = np.empty(hd, dtype=np.float64)
    lib().orc_attention_partial(_p(q), _p(K), _p(V), C.c_int(hd), C.c_int(j0), C.c_int(j1),
                                C.byref(m), C.byref(l), _p(acc))
    return m.value, l.value, acc


def attention_combine(ms: Sequence[float], ls: Sequence[float], accs: Sequence[np.ndarray]) -> np.ndarray:
    m = _c(ms, np.float64)
    l = _c(ls, np.float64)
    acc = _c(np.stack(accs), np.float64)
    n, hd = acc.shape
    o = np.empty(hd, dtype=np.float32)
    lib().orc_attention_combine(_p(m), _p(l), _p(acc), C.c_int(n), C.c_int(hd), _p(o))
    return o


# ------------------------------------------------------------------------------------------------
# whole step
# ------------------------------------------------------------------------------------------------

@dataclass
class Shape:
    hidden: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    mlp: int
    vocab: int
    max_seq: int
    tied: bool
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0

    @classmethod
    def of(cls, s) -> "Shape":
        """Accept any object with the same attribute names (e.g. the input module's shape record)."""
        return cls(hidden=s.hidden, n_layers=s.n_layers, n_q_heads=s.n_q_heads, n_kv_heads=s.n_kv_heads,
                   head_dim=s.head_dim, mlp=s.mlp, vocab=s.vocab, max_seq=s.max_seq, tied=bool(s.tied),
                   rms_eps=float(s.rms_eps), rope_theta=float(s.rope_theta))


def kv_elems(s) -> int:
    """Elements in the whole cache buffer (K then V)."""
    return 2 * s.n_layers * s.n_kv_heads * s.max_seq * s.head_dim


class Model:
    """Holds numpy views of the canonical weights and the C structs pointing at them.

    ``weights``: dict with ``embed`` [V][H] uint16, ``lm_head`` (or None), ``final_norm`` [H] uint16,
    ``attn_norm`` / ``mlp_norm``: lists of [H] uint16, and for each kind in KINDS a list over layers of
    the weight array (uint16 bf16 bits, int8, or packed uint8) plus, when quantised, ``<kind>_scale`` and
    (int4) ``<kind>_zero`` lists of uint16 arrays.
    """

    def __init__(self, shape, weights: Dict, wdtype: int = W_BF16, group: int = 128, round_kv: bool = True,
                 quantize_lm_head: bool = False, kv_dtype: int = KV_BF16):
        """``kv_dtype``: KV_BF16, or KV_E4M3 (cache entries rounded to fp8 e4m3; the cache array then holds the codes).
        ``quantize_lm_head``: the LM head is read from ``weights["lm_head_q"]`` / ``["lm_head_scale"]`` /
        ``["lm_head_zero"]`` (see ``quantize_lm_head``), quantised like the layers."""
        self.shape = Shape.of(shape)
        s = self.shape
        self.wdtype, self.group = wdtype, group
        self._keep: List[np.ndarray] = []
        qlm = bool(quantize_lm_head) and wdtype != W_BF16
        self.cfg = _Config(s.hidden, s.n_layers, s.n_q_heads, s.n_kv_heads, s.head_dim, s.mlp, s.vocab,
                           s.max_seq, int(s.tied), s.rms_eps, s.rope_theta, wdtype, group, int(round_kv), int(qlm),
                           int(kv_dtype))
        w = _Weights()
        w.embed = self._hold(weights["embed"], np.uint16)
        w.lm_head = None if s.tied else self._hold(weights["lm_head"], np.uint16)
        w.final_norm = self._hold(weights["final_norm"], np.uint16)
        w.attn_norm = self._ptr_array(weights["attn_norm"], np.uint16)
        w.mlp_norm = self._ptr_array(weights["mlp_norm"], np.uint16)
        wdt = {W_BF16: np.uint16, W_INT8: np.int8, W_INT4: np.uint8, W_INT8G: np.int8}[wdtype]
        for i, kind in enumerate(KINDS):
            w.w[i] = self._ptr_array(weights[kind], wdt)
            if wdtype != W_BF16:
                w.scale[i] = self._ptr_array(weights[kind + "_scale"], np.uint16)
            if wdtype == W_INT4:
                w.zero[i] = self._ptr_array(weights[kind + "_zero"], np.uint16)
        if qlm:
            w.lm_head_q = self._hold(weights["lm_head_q"], wdt)
            w.lm_head_scale = self._hold(weights["lm_head_scale"], np.uint16)
            if wdtype == W_INT4:
                w.lm_head_zero = self._hold(weights["lm_head_zero"], np.uint16)
        self.w = w

    def _hold(self, a, dtype) -> int:
        a = np.ascontiguousarray(a, dtype=dtype)
        self._keep.append(a)
        return a.ctypes.data

    def _ptr_array(self, arrays, dtype):
        ptrs = (C.c_void_p * len(arrays))()
        for i, a in enumerate(arrays):
            ptrs[i] = self._hold(a, dtype)
        self._keep.append(ptrs)
        return C.cast(ptrs, _PP)

    def new_cache(self) -> np.ndarray:
        return np.zeros(kv_elems(self.shape), dtype=np.uint16)

    def decode_step(self, token: int, pos: int, kv: np.ndarray, kv_f32: Optional[np.ndarray] = None,
                    want_hidden: bool = True, rows_pref: Optional[np.ndarray] = None):
        """Returns (logits fp32 [V], next_token, hidden fp32 [L+1][H] or None); updates ``kv`` in place.

        ``rows_pref`` (uint16 [2][L][n_kv][hd]): another implementation's appended cache rows.  An entry is
        adopted where it is the oracle's own rounding or a neighbouring bf16 value (both are valid roundings of
        fp32 values that differ in the last bits); the oracle's own rows and the number of adopted entries are
        then left in ``self.rows_own`` / ``self.n_adopted``."""
        s = self.shape
        assert kv.dtype == np.uint16 and kv.size == kv_elems(s) and kv.flags["C_CONTIGUOUS"]
        logits = np.empty(s.vocab, dtype=np.float32)
        nxt = C.c_int(-1)
        hidden = np.empty((s.n_layers + 1, s.hidden), dtype=np.float32) if want_hidden else None
        if rows_pref is None:
            rc = lib().orc_decode_step(C.byref(self.cfg), C.byref(self.w), C.c_int(token), C.c_int(pos),
                                       _p(kv), _p(kv_f32), _p(logits), C.byref(nxt), _p(hidden))
        else:
            rows_pref = _c(rows_pref, np.uint16)
            assert rows_pref.size == 2 * s.n_layers * s.n_kv_heads * s.head_dim
            self.rows_own = np.empty(rows_pref.size, dtype=np.uint16)
            n = C.c_int(0)
            rc = lib().orc_decode_step_rows(C.byref(self.cfg), C.byref(self.w), C.c_int(token), C.c_int(pos),
                                            _p(kv), _p(kv_f32), _p(logits), C.byref(nxt), _p(hidden),
                                            _p(rows_pref), _p(self.rows_own), C.byref(n))
            self.n_adopted = int(n.value)
        if rc != 0:
            raise ValueError("oracle: bad argument (token/pos/head shape)")
        return logits, int(nxt.value), hidden

    def layer_step(self, layer: int, pos: int, x_in, kv: np.ndarray, rows_pref: Optional[np.ndarray] = None) -> np.ndarray:
        """One decoder layer on a given residual stream.  ``rows_pref`` (uint16 [2][n_kv][hd]): see decode_step."""
        s = self.shape
        x_in = _c(x_in, np.float32)
        out = np.empty(s.hidden, dtype=np.float32)
        if rows_pref is None:
            rc = lib().orc_layer_step(C.byref(self.cfg), C.byref(self.w), C.c_int(layer), C.c_int(pos), _p(x_in),
                                      _p(kv), _p(out))
        else:
            rows_pref = _c(rows_pref, np.uint16)
            assert rows_pref.size == 2 * s.n_kv_heads * s.head_dim
            self.rows_own = np.empty(rows_pref.size, dtype=np.uint16)
            n = C.c_int(0)
            rc = lib().orc_layer_step_rows(C.byref(self.cfg), C.byref(self.w), C.c_int(layer), C.c_int(pos), _p(x_in),
                                           _p(kv), _p(out), _p(rows_pref), _p(self.rows_own), C.byref(n))
            self.n_adopted = int(n.value)
        if rc != 0:
            raise ValueError("oracle: bad argument")
        return out

    def head_step(self, x_in):
        s = self.shape
        x_in = _c(x_in, np.float32)
        logits = np.empty(s.vocab, dtype=np.float32)
        nxt = C.c_int(-1)
        lib().orc_head_step(C.byref(self.cfg), C.byref(self.w), _p(x_in), _p(logits), C.byref(nxt))
        return logits, int(nxt.value)


def quantize_weights(weights: Dict, wdtype: int, group: int = 128) -> Dict:
    """Apply the oracle's own quantiser to the seven per-layer linears of a bf16 weight dict."""
    if wdtype == W_BF16:
        return weights
    out = {k: v for k, v in weights.items() if k not in KINDS}
    for kind in KINDS:
        qs, ss, zs = [], [], []
        for W in weights[kind]:
            if wdtype in (W_INT8, W_INT8G):
                q, s = quantize_int8(W) if wdtype == W_INT8 else quantize_int8_grouped(W, group)
                qs.append(q)
                ss.append(s)
            else:
                q, s, z = quantize_int4(W, group)
                qs.append(q)
                ss.append(s)
                zs.append(z)
        out[kind] = qs
        out[kind + "_scale"] = ss
        if wdtype == W_INT4:
            out[kind + "_zero"] = zs
    return out


def quantize_lm_head(weights: Dict, wdtype: int, group: int = 128, tied: bool = False) -> Dict:
    """Adds ``lm_head_q`` / ``lm_head_scale`` (/ ``lm_head_zero``): the oracle's own quantiser applied to the LM head
    matrix (the embedding matrix when tied).  The bf16 matrices stay in the dict."""
    out = dict(weights)
    W = weights["embed"] if (tied or weights.get("lm_head") is None) else weights["lm_head"]
    if wdtype == W_INT8:
        out["lm_head_q"], out["lm_head_scale"] = quantize_int8(W)
    elif wdtype == W_INT8G:
        out["lm_head_q"], out["lm_head_scale"] = quantize_int8_grouped(W, group)
    elif wdtype == W_INT4:
        out["lm_head_q"], out["lm_head_scale"], out["lm_head_zero"] = quantize_int4(W, group)
    return out


def num_threads() -> int:
    return int(lib().orc_num_threads())
