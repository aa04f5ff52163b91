"""Seeded synthetic inputs: model shapes, random-init weights, tokens and pre-filled KV caches.

This module holds none of the decode arithmetic.  It only draws numbers: it serves both the CUDA path
and the CPU oracle so that each sees exactly the same tensors.  The paper's speed studies use
random-initialised weights at real Llama shapes at decode position 0 (Section 5, "Beating cuBLAS with
int8"); the shapes below are those of the workloads this repository measures.

Everything 16-bit is produced as a ``torch.bfloat16`` tensor; ``bits()`` gives the ``numpy.uint16``
view a CPU consumer wants.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, List, Optional

import numpy as np
import torch

KINDS = ("wq", "wk", "wv", "wo", "wgate", "wup", "wdown")


@dataclass(frozen=True)
class ModelShape:
    name: str
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

    def linear_dims(self, kind: str):
        """(rows, cols) = (out, in) of one per-layer linear."""
        H, q, kv, I = self.hidden, self.n_q_heads * self.head_dim, self.n_kv_heads * self.head_dim, self.mlp
        return {"wq": (q, H), "wk": (kv, H), "wv": (kv, H), "wo": (H, q),
                "wgate": (I, H), "wup": (I, H), "wdown": (H, I)}[kind]

    def n_params(self) -> int:
        per_layer = sum(r * c for r, c in (self.linear_dims(k) for k in KINDS)) + 2 * self.hidden
        head = 0 if self.tied else self.vocab * self.hidden
        return self.vocab * self.hidden + self.n_layers * per_layer + self.hidden + head

    def with_(self, **kw) -> "ModelShape":
        return replace(self, **kw)


SHAPES: Dict[str, ModelShape] = {
    # 2-layer hidden-64 toy used for brute-force checks
    "toy": ModelShape("toy", 64, 2, 4, 2, 16, 128, 97, 64, False),
    # a slightly larger toy with ragged sizes (rows not multiples of anything convenient)
    "toy_ragged": ModelShape("toy_ragged", 192, 3, 6, 2, 32, 328, 1003, 96, True),
    # small shapes the CUDA kernel accepts (head_dim 64 / 128), spanning several tiles and ragged tails
    "mini": ModelShape("mini", 256, 2, 4, 2, 64, 512, 1000, 128, False),
    "mini_ragged": ModelShape("mini_ragged", 192, 3, 3, 1, 64, 320, 1003, 96, True),
    "mini_hd128": ModelShape("mini_hd128", 512, 2, 8, 2, 128, 1024, 2048, 256, False, rope_theta=500000.0),
    "mini_wide": ModelShape("mini_wide", 1024, 2, 16, 2, 64, 2816, 5000, 512, False),
    "smollm2_135m": ModelShape("smollm2_135m", 576, 30, 9, 3, 64, 1536, 49152, 2048, True),
    "tinyllama_1b": ModelShape("tinyllama_1b", 2048, 22, 32, 4, 64, 5632, 32000, 2048, False),
    "llama3_8b": ModelShape("llama3_8b", 4096, 32, 32, 8, 128, 14336, 128256, 8192, False,
                            rope_theta=500000.0),
    # the paper's 16-layer "b1" shape (Section 5, Tables 7-8: 2997.0 MB of bf16 weights): Llama-3.2-1B dimensions
    # with an untied LM head
    "llama32_1b": ModelShape("llama32_1b", 2048, 16, 32, 8, 64, 8192, 128256, 2048, False,
                             rope_theta=500000.0),
    # the paper's 4-layer hidden-2048 "small" model (Section 5, Tables 7-8: 622.9 MB of bf16 weights).  The paper gives
    # its layer count, hidden size and weight bytes only; taken here as four layers of the b1 dimensions with a tied
    # embedding of 33280 rows, the vocabulary at which the bf16 bytes come to the paper's 622.9 MB (an assumption)
    "paper_small": ModelShape("paper_small", 2048, 4, 32, 8, 64, 8192, 33280, 2048, True, rope_theta=500000.0),
}


def _gen(seed: int, stream: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((int(seed) * 1000003 + int(stream)) & 0x7FFFFFFFFFFFFFFF)
    return g


def _normal_bf16(shape, std: float, seed: int, stream: int, device) -> torch.Tensor:
    g = _gen(seed, stream, device)
    n = 1
    for d in shape:
        n *= d
    out = torch.empty(n, dtype=torch.bfloat16, device=device)
    step = 1 << 26                      # draw in fp32 chunks so the largest tensors never need 4 bytes/elem at once
    for a in range(0, n, step):
        b = min(n, a + step)
        out[a:b] = (torch.randn(b - a, generator=g, device=device, dtype=torch.float32) * std).to(torch.bfloat16)
    return out.view(*shape)


def make_weights(shape: ModelShape, seed: int, device="cpu", std: float = 0.02,
                 norm_jitter: float = 0.0) -> Dict:
    """Random-init bf16 weights: every linear / embedding / LM-head entry i.i.d. N(0, std^2) rounded to
    bf16; norm weights exactly 1.0 (or 1 + N(0, norm_jitter^2) when a test wants them to matter)."""
    dev = torch.device(device)
    w: Dict = {}
    w["embed"] = _normal_bf16((shape.vocab, shape.hidden), std, seed, 1, dev)
    w["lm_head"] = None if shape.tied else _normal_bf16((shape.vocab, shape.hidden), std, seed, 2, dev)

    def norm(stream):
        if norm_jitter == 0.0:
            return torch.ones(shape.hidden, dtype=torch.bfloat16, device=dev)
        g = _gen(seed, stream, dev)
        return (1.0 + norm_jitter * torch.randn(shape.hidden, generator=g, device=dev)).to(torch.bfloat16)

    w["final_norm"] = norm(3)
    w["attn_norm"] = [norm(100 + 16 * l) for l in range(shape.n_layers)]
    w["mlp_norm"] = [norm(101 + 16 * l) for l in range(shape.n_layers)]
    for i, kind in enumerate(KINDS):
        w[kind] = [_normal_bf16(shape.linear_dims(kind), std, seed, 102 + 16 * l + i, dev)
                   for l in range(shape.n_layers)]
    return w


def make_token(shape: ModelShape, seed: int) -> int:
    g = _gen(seed, 7, "cpu")
    return int(torch.randint(0, shape.vocab, (1,), generator=g).item())


def make_kv_prefill(shape: ModelShape, seed: int, pos: int, device="cpu", std: float = 1.0,
                    kv_dtype: str = "bf16") -> torch.Tensor:
    """The whole cache buffer (K then V, each [L][n_kv][max_seq][hd] bf16) with positions [0, pos) drawn
    i.i.d. N(0, std^2) and every other slot zero.  ``kv_dtype="fp8"``: the same draws as e4m3 codes (uint8; torch's
    conversion -- any valid code is a valid input)."""
    dev = torch.device(device)
    L, g_, S, hd = shape.n_layers, shape.n_kv_heads, shape.max_seq, shape.head_dim
    kv = torch.zeros((2, L, g_, S, hd), dtype=torch.bfloat16, device=dev)
    if pos > 0:
        kv[:, :, :, :pos, :] = _normal_bf16((2, L, g_, pos, hd), std, seed, 9, dev)
    if kv_dtype == "fp8":
        return kv.to(torch.float32).to(torch.float8_e4m3fn).view(torch.uint8).view(-1)
    return kv.view(-1)


def bits(t: Optional[torch.Tensor]) -> Optional[np.ndarray]:
    """numpy.uint16 bit view of a bf16/fp16 tensor (copied to host if needed)."""
    if t is None:
        return None
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def weights_to_numpy(w: Dict) -> Dict:
    """Host bit-pattern view of a bf16 weight dict, in the form the CPU oracle takes."""
    out: Dict = {}
    for k, v in w.items():
        if isinstance(v, list):
            out[k] = [bits(t) for t in v]
        else:
            out[k] = bits(v)
    return out


def streamed_bytes(shape: ModelShape, wdtype: str = "bf16", pos: int = 0, group: int = 128,
                   quantize_lm_head: bool = False, kv_dtype: str = "bf16") -> Dict[str, float]:
    """Algorithmic bytes one decode step must move: weights + scales + KV read/write + activations.
    ``quantize_lm_head``: the LM head is streamed at the layers' width (with its scales) instead of as bf16."""
    H, L, I, V = shape.hidden, shape.n_layers, shape.mlp, shape.vocab
    nq, nkv, hd = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    lin = sum(r * c for r, c in (shape.linear_dims(k) for k in KINDS))
    rows = sum(r for r, _ in (shape.linear_dims(k) for k in KINDS))
    if wdtype == "bf16":
        wl, sc = 2.0 * lin, 0.0
    elif wdtype == "int8":
        wl, sc = 1.0 * lin, 2.0 * rows
    elif wdtype == "int4":
        wl, sc = 0.5 * lin, 4.0 * lin / group
    elif wdtype == "int8g":                                          # grouped int8: {fp16 scale, pad} per row and group
        wl, sc = 1.0 * lin, 4.0 * lin / group
    else:
        raise ValueError(wdtype)
    head, head_sc = 2.0 * V * H, 0.0
    if quantize_lm_head and wdtype == "int8":
        head, head_sc = 1.0 * V * H, 2.0 * V
    elif quantize_lm_head and wdtype == "int4":
        head, head_sc = 0.5 * V * H, 4.0 * V * H / group
    elif quantize_lm_head and wdtype == "int8g":
        head, head_sc = 1.0 * V * H, 4.0 * V * H / group
    weights = L * wl + head + 2.0 * (2 * L + 1) * H + 2.0 * H            # linears + LM head + norms + one embedding row
    scales = L * sc + head_sc
    kv_esz = 1.0 if kv_dtype == "fp8" else 2.0
    kv = 2.0 * L * nkv * hd * kv_esz * pos + 2.0 * L * nkv * hd * kv_esz
    act = 4.0 * (L * (4 * H + (nq + 2 * nkv) * hd + nq * hd + 2 * I) + 2 * H) + 4.0 * V
    return {"weights": weights, "scales": scales, "kv": kv, "act": act, "total": weights + scales + kv + act}
