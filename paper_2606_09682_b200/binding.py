"""ctypes binding of the C-ABI library (``include/amk.h``): same names, argument marshalling only.

Every step of the decode path runs inside the library's CUDA kernels.  PyTorch is used here for device
memory (``torch.empty``), streams and nothing else.  If the shared library is missing this module raises
at import: there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("AMK_LIB") or os.path.join(_HERE, "libamk.so")      # AMK_LIB: another build of the library

AMK_ABI_VERSION = 3
AMK_OK, AMK_ERR_INVALID_ARG, AMK_ERR_UNSUPPORTED, AMK_ERR_CUDA, AMK_ERR_OOM = 0, 1, 2, 3, 4
AMK_ERR_TIMEOUT, AMK_ERR_ABORTED, AMK_ERR_BAD_POS, AMK_ERR_BAD_TOKEN = 5, 6, 7, 8
AMK_W_BF16, AMK_W_INT8, AMK_W_INT4, AMK_W_INT8_GROUPED = 0, 1, 2, 3
AMK_KV_BF16, AMK_KV_FP8_E4M3 = 0, 1
KVDTYPES = {"bf16": AMK_KV_BF16, "fp8": AMK_KV_FP8_E4M3}
AMK_FLAG_DEBUG_HIDDEN = 1
AMK_FLAG_TRACE = 2
AMK_FLAG_MEASURED_SPLIT = 4
AMK_FLAG_TRACE_CYCLES = 8
AMK_TRACE_EVENTS = 12
AMK_LIN_Q, AMK_LIN_K, AMK_LIN_V, AMK_LIN_O, AMK_LIN_GATE, AMK_LIN_UP, AMK_LIN_DOWN, AMK_LIN_LM_HEAD = range(8)
KINDS = ("wq", "wk", "wv", "wo", "wgate", "wup", "wdown")
WDTYPES = {"bf16": AMK_W_BF16, "int8": AMK_W_INT8, "int4": AMK_W_INT4, "int8g": AMK_W_INT8_GROUPED}


class amk_config(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in ("struct_size", "abi_version", "hidden", "n_layers", "n_q_heads",
                                          "n_kv_heads", "head_dim", "mlp", "vocab", "max_seq",
                                          "tied_embeddings")] + [
        ("rms_eps", C.c_float), ("rope_theta", C.c_float)] + [
        (n, C.c_uint32) for n in ("wdtype", "group_size", "quantize_lm_head", "wait_timeout_us", "flags",
                                  "stage_bytes", "n_stages", "max_inflight", "sync_mode", "n_blocks", "l2_ahead", "kv_dtype")]


_PP = C.POINTER(C.c_void_p)


class amk_weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p),
                ("attn_norm", _PP), ("mlp_norm", _PP),
                ("linear", _PP * 7), ("scale", _PP * 7), ("zero", _PP * 7),
                ("lm_head_q", C.c_void_p), ("lm_head_scale", C.c_void_p), ("lm_head_zero", C.c_void_p)]


class amk_plan(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in ("n_blocks", "threads", "smem_bytes", "stage_bytes", "n_stages",
                                          "max_inflight", "l2_ahead", "n_gemv_ops", "n_phases")] + [
        (n, C.c_uint64) for n in ("packed_bytes", "workspace_bytes", "kv_bytes", "weight_stream_bytes")]


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2606_09682_b200.build` "
                          "(there is no fallback path)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    cfgp = C.POINTER(amk_config)
    sigs = {
        "amk_status_str": (C.c_char_p, [C.c_int]),
        "amk_packed_bytes": (C.c_int, [cfgp, C.POINTER(sz)]),
        "amk_workspace_bytes": (C.c_int, [cfgp, C.POINTER(sz)]),
        "amk_kv_bytes": (C.c_int, [cfgp, C.POINTER(sz)]),
        "amk_create": (C.c_int, [cfgp, C.POINTER(amk_weights), vp, sz, vp, sz, vp, C.POINTER(vp)]),
        "amk_decode_step": (C.c_int, [vp, i32, i32, vp, vp, vp, vp]),
        "amk_decode_greedy": (C.c_int, [vp, i32, i32, i32, vp, vp, vp, vp]),
        "amk_last_status": (C.c_int, [vp, C.POINTER(C.c_int), C.c_char_p, sz]),
        "amk_plan_info": (C.c_int, [vp, C.POINTER(amk_plan)]),
        "amk_debug_hidden": (C.c_int, [vp, vp]),
        "amk_debug_trace": (C.c_int, [vp, vp, sz]),
        "amk_debug_unpack": (C.c_int, [vp, C.c_int, C.c_int, vp, vp, vp, vp]),
        "amk_debug_drop_signal": (C.c_int, [vp, C.c_int, C.c_int]),
        "amk_debug_set_step_count": (C.c_int, [vp, C.c_uint32]),
        "amk_last_kernel_ns": (C.c_int, [vp, C.POINTER(C.c_uint64)]),
        "amk_destroy": (C.c_int, [vp]),
        "amk_quantize_int8": (C.c_int, [vp, i64, i64, vp, vp, vp]),
        "amk_quantize_int8_grouped": (C.c_int, [vp, i64, i64, vp, vp, vp]),
        "amk_quantize_int4": (C.c_int, [vp, i64, i64, vp, vp, vp, vp]),
        "amk_argmax_static": (C.c_int, [vp, i64, vp, C.c_char_p, sz, vp]),
        "amk_plan_export": (C.c_int, [C.POINTER(amk_config), vp, sz, C.POINTER(sz)]),
        "amk_plan_check": (C.c_int, [C.POINTER(amk_config), vp, sz, C.c_char_p, sz]),
    }
    for name, (res, args) in sigs.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    return lib


lib = _load()
EXPORTS = ("amk_status_str", "amk_packed_bytes", "amk_workspace_bytes", "amk_kv_bytes", "amk_create",
           "amk_decode_step", "amk_decode_greedy", "amk_last_status", "amk_plan_info", "amk_debug_hidden",
           "amk_debug_trace", "amk_debug_unpack", "amk_debug_drop_signal", "amk_debug_set_step_count", "amk_last_kernel_ns", "amk_destroy", "amk_quantize_int8", "amk_quantize_int8_grouped", "amk_quantize_int4",
           "amk_argmax_static", "amk_plan_export", "amk_plan_check")


class AmkError(RuntimeError):
    def __init__(self, code: int, what: str = ""):
        self.code = code
        super().__init__(f"{what}: {lib.amk_status_str(code).decode()} ({code})")


def _check(code: int, what: str):
    if code != AMK_OK:
        raise AmkError(code, what)


def make_config(shape, wdtype: str = "bf16", flags: int = 0, wait_timeout_us: int = 0, stage_bytes: int = 0,
                n_stages: int = 0, max_inflight: int = 0, group_size: int = 128, sync_mode: int = 1,
                n_blocks: int = 0, l2_ahead: int = 0, quantize_lm_head: bool = False,
                kv_dtype: str = "bf16") -> amk_config:
    """``shape``: any object with hidden, n_layers, n_q_heads, n_kv_heads, head_dim, mlp, vocab, max_seq,
    tied, rms_eps, rope_theta attributes."""
    c = amk_config()
    c.struct_size, c.abi_version = C.sizeof(amk_config), AMK_ABI_VERSION
    c.hidden, c.n_layers, c.n_q_heads, c.n_kv_heads = shape.hidden, shape.n_layers, shape.n_q_heads, shape.n_kv_heads
    c.head_dim, c.mlp, c.vocab, c.max_seq = shape.head_dim, shape.mlp, shape.vocab, shape.max_seq
    c.tied_embeddings = int(shape.tied)
    c.rms_eps, c.rope_theta = shape.rms_eps, shape.rope_theta
    c.wdtype = WDTYPES[wdtype]
    c.group_size = group_size if wdtype in ("int4", "int8g") else 0
    c.wait_timeout_us, c.flags = wait_timeout_us, flags
    c.stage_bytes, c.n_stages, c.max_inflight = stage_bytes, n_stages, max_inflight
    c.sync_mode, c.n_blocks, c.l2_ahead = sync_mode, n_blocks, l2_ahead
    c.quantize_lm_head = int(bool(quantize_lm_head))
    c.kv_dtype = KVDTYPES[kv_dtype]
    return c


def amk_packed_bytes(cfg: amk_config) -> int:
    n = C.c_size_t()
    _check(lib.amk_packed_bytes(C.byref(cfg), C.byref(n)), "amk_packed_bytes")
    return n.value


def amk_workspace_bytes(cfg: amk_config) -> int:
    n = C.c_size_t()
    _check(lib.amk_workspace_bytes(C.byref(cfg), C.byref(n)), "amk_workspace_bytes")
    return n.value


def amk_kv_bytes(cfg: amk_config) -> int:
    n = C.c_size_t()
    _check(lib.amk_kv_bytes(C.byref(cfg), C.byref(n)), "amk_kv_bytes")
    return n.value


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def amk_quantize_int8(w: torch.Tensor):
    """bf16 [rows][cols] (cuda) -> (int8 [rows][cols], fp16 [rows])."""
    assert w.is_cuda and w.dtype == torch.bfloat16 and w.is_contiguous()
    rows, cols = w.shape
    q = torch.empty((rows, cols), dtype=torch.int8, device=w.device)
    s = torch.empty((rows,), dtype=torch.float16, device=w.device)
    _check(lib.amk_quantize_int8(w.data_ptr(), rows, cols, q.data_ptr(), s.data_ptr(), _stream()), "amk_quantize_int8")
    return q, s


def amk_quantize_int8_grouped(w: torch.Tensor):
    """bf16 [rows][cols] (cuda) -> (int8 [rows][cols], fp16 scale [rows][cols/128])."""
    assert w.is_cuda and w.dtype == torch.bfloat16 and w.is_contiguous()
    rows, cols = w.shape
    q = torch.empty((rows, cols), dtype=torch.int8, device=w.device)
    s = torch.empty((rows, cols // 128), dtype=torch.float16, device=w.device)
    _check(lib.amk_quantize_int8_grouped(w.data_ptr(), rows, cols, q.data_ptr(), s.data_ptr(), _stream()),
           "amk_quantize_int8_grouped")
    return q, s


def amk_quantize_int4(w: torch.Tensor):
    """bf16 [rows][cols] (cuda) -> (uint8 [rows][cols/2], fp16 scale [rows][cols/128], fp16 zero same)."""
    assert w.is_cuda and w.dtype == torch.bfloat16 and w.is_contiguous()
    rows, cols = w.shape
    p = torch.empty((rows, cols // 2), dtype=torch.uint8, device=w.device)
    s = torch.empty((rows, cols // 128), dtype=torch.float16, device=w.device)
    z = torch.empty((rows, cols // 128), dtype=torch.float16, device=w.device)
    _check(lib.amk_quantize_int4(w.data_ptr(), rows, cols, p.data_ptr(), s.data_ptr(), z.data_ptr(), _stream()),
           "amk_quantize_int4")
    return p, s, z


AMK_ARGMAX_STATIC_MAX_N = 1 << 20


def amk_plan_export(cfg: amk_config):
    """The tables a step runs from, as a numpy uint64 array (host only; no GPU needed when cfg.n_blocks is set)."""
    import numpy as np
    need = C.c_size_t()
    _check(lib.amk_plan_export(C.byref(cfg), None, 0, C.byref(need)), "amk_plan_export")
    out = np.zeros(need.value, dtype=np.uint64)
    _check(lib.amk_plan_export(C.byref(cfg), out.ctypes.data, out.size, C.byref(need)), "amk_plan_export")
    return out


def amk_plan_check(cfg: amk_config, tables):
    """(status, reason) of the static check over an exported -- or tampered with -- table array."""
    import numpy as np
    t = np.ascontiguousarray(tables, dtype=np.uint64)
    msg = C.create_string_buffer(256)
    st = lib.amk_plan_check(C.byref(cfg), t.ctypes.data, t.size, msg, 256)
    return st, msg.value.decode()


def amk_argmax_static(x: torch.Tensor, token: torch.Tensor, n: int = -1) -> None:
    """fp32 vector (cuda) -> token[0] (int32, cuda) = index of its maximum; library-owned scratch, no allocation.
    ``n`` overrides the element count handed to the library (for argument-checking tests)."""
    assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous()
    assert token.is_cuda and token.dtype == torch.int32 and token.numel() >= 1
    assert token.device == x.device, "x and token must live on the same device"
    msg = C.create_string_buffer(256)
    with torch.cuda.device(x.device):          # the library uses the scratch array of the current device
        code = lib.amk_argmax_static(x.data_ptr(), x.numel() if n < 0 else n, token.data_ptr(), msg, 256, _stream())
    if code != AMK_OK:
        raise AmkError(code, msg.value.decode() or "amk_argmax_static")


def quantize_weights(weights: Dict, wdtype: str) -> Dict:
    """Run the library's quantiser over the seven per-layer linears of a bf16 weight dict (cuda tensors)."""
    if wdtype == "bf16":
        return weights
    out = {k: v for k, v in weights.items() if k not in KINDS}
    for kind in KINDS:
        qs, ss, zs = [], [], []
        for w in weights[kind]:
            if wdtype == "int8":
                q, s = amk_quantize_int8(w)
            elif wdtype == "int8g":
                q, s = amk_quantize_int8_grouped(w)
            else:
                q, s, z = amk_quantize_int4(w)
                zs.append(z)
            qs.append(q)
            ss.append(s)
        out[kind], out[kind + "_scale"] = qs, ss
        if wdtype == "int4":
            out[kind + "_zero"] = zs
    return out


def quantize_lm_head(weights: Dict, wdtype: str, tied: bool) -> Dict:
    """Adds ``lm_head_q`` / ``lm_head_scale`` (/ ``lm_head_zero``): the library's quantiser applied to the LM head
    matrix (the embedding matrix when tied), for a decoder created with ``quantize_lm_head=True``."""
    out = dict(weights)
    w = weights["embed"] if (tied or weights.get("lm_head") is None) else weights["lm_head"]
    if wdtype == "int8":
        out["lm_head_q"], out["lm_head_scale"] = amk_quantize_int8(w)
    elif wdtype == "int8g":
        out["lm_head_q"], out["lm_head_scale"] = amk_quantize_int8_grouped(w)
    elif wdtype == "int4":
        out["lm_head_q"], out["lm_head_scale"], out["lm_head_zero"] = amk_quantize_int4(w)
    return out


def _ptr_array(tensors: Sequence[torch.Tensor], keep: List):
    arr = (C.c_void_p * len(tensors))()
    for i, t in enumerate(tensors):
        assert t.is_cuda and t.is_contiguous()
        arr[i] = t.data_ptr()
    keep.append(arr)
    return C.cast(arr, _PP)


class Decoder:
    """Owns the caller-side device buffers (torch tensors) of one handle and forwards to the C ABI."""

    def __init__(self, shape, weights: Dict, wdtype: str = "bf16", flags: int = 0, wait_timeout_us: int = 0,
                 stage_bytes: int = 0, n_stages: int = 0, max_inflight: int = 0, sync_mode: int = 1,
                 n_blocks: int = 0, l2_ahead: int = 0, device="cuda", guard_bytes: int = 0,
                 quantize_lm_head: bool = False, kv_dtype: str = "bf16"):
        """``guard_bytes`` (a multiple of 256): the packed buffer, the workspace and the logits get that many bytes
        of a fixed pattern in front and behind, which ``guards_intact()`` checks -- a stand-in for a memory checker."""
        self.shape, self.wdtype = shape, wdtype
        self.device = torch.device(device)
        self.cfg = make_config(shape, wdtype, flags, wait_timeout_us, stage_bytes, n_stages, max_inflight,
                               sync_mode=sync_mode, n_blocks=n_blocks, l2_ahead=l2_ahead,
                               quantize_lm_head=quantize_lm_head, kv_dtype=kv_dtype)
        self.kv_dtype = kv_dtype
        self.quantize_lm_head = bool(quantize_lm_head)
        assert guard_bytes % 256 == 0
        self._guard = guard_bytes
        self._guarded: List[torch.Tensor] = []
        self.packed = self._alloc(amk_packed_bytes(self.cfg))
        self.workspace = self._alloc(amk_workspace_bytes(self.cfg))
        keep: List = []
        w = amk_weights()
        w.embed = weights["embed"].data_ptr()
        w.lm_head = None if shape.tied else weights["lm_head"].data_ptr()
        if quantize_lm_head:
            w.lm_head_q = weights["lm_head_q"].data_ptr()
            w.lm_head_scale = weights["lm_head_scale"].data_ptr()
            w.lm_head_zero = weights["lm_head_zero"].data_ptr() if wdtype == "int4" else None
        w.final_norm = weights["final_norm"].data_ptr()
        w.attn_norm = _ptr_array(weights["attn_norm"], keep)
        w.mlp_norm = _ptr_array(weights["mlp_norm"], keep)
        for i, kind in enumerate(KINDS):
            w.linear[i] = _ptr_array(weights[kind], keep)
            if wdtype != "bf16":
                w.scale[i] = _ptr_array(weights[kind + "_scale"], keep)
            if wdtype == "int4":
                w.zero[i] = _ptr_array(weights[kind + "_zero"], keep)
        h = C.c_void_p()
        _check(lib.amk_create(C.byref(self.cfg), C.byref(w), self.packed.data_ptr(), self.packed.numel(),
                              self.workspace.data_ptr(), self.workspace.numel(), _stream(), C.byref(h)), "amk_create")
        self.h = h
        torch.cuda.current_stream().synchronize()      # the canonical weights may be freed from here on
        self.logits = self._alloc(4 * shape.vocab).view(torch.float32)
        self.next_token = torch.empty(1, dtype=torch.int32, device=self.device)

    def _alloc(self, n_bytes: int) -> torch.Tensor:
        """uint8 device buffer of n_bytes (256-byte aligned), with guard bands around it if asked for."""
        g = self._guard
        if not g:
            return torch.empty(n_bytes, dtype=torch.uint8, device=self.device)
        inner = (n_bytes + 255) // 256 * 256
        whole = torch.full((inner + 2 * g,), 0xA5, dtype=torch.uint8, device=self.device)
        self._guarded.append((whole, inner))
        return whole[g:g + n_bytes]

    def guards_intact(self) -> bool:
        g = self._guard
        return all(bool((w[:g] == 0xA5).all()) and bool((w[g + inner:] == 0xA5).all()) for w, inner in self._guarded)

    def new_cache(self) -> torch.Tensor:
        n = amk_kv_bytes(self.cfg)
        fp8 = self.kv_dtype == "fp8"
        if not self._guard:
            return torch.zeros(n if fp8 else n // 2, dtype=torch.uint8 if fp8 else torch.bfloat16, device=self.device)
        buf = self._alloc(n)
        buf.zero_()
        return buf if fp8 else buf.view(torch.bfloat16)

    def plan(self) -> amk_plan:
        p = amk_plan()
        _check(lib.amk_plan_info(self.h, C.byref(p)), "amk_plan_info")
        return p

    def amk_decode_step(self, token: int, pos: int, kv: torch.Tensor, want_logits: bool = True) -> None:
        _check(lib.amk_decode_step(self.h, token, pos, kv.data_ptr(), self.logits.data_ptr() if want_logits else None,
                                   self.next_token.data_ptr(), _stream()), "amk_decode_step")

    def amk_decode_greedy(self, first_token: int, pos0: int, n_steps: int, kv: torch.Tensor) -> torch.Tensor:
        toks = torch.empty(n_steps, dtype=torch.int32, device=self.device)
        _check(lib.amk_decode_greedy(self.h, first_token, pos0, n_steps, kv.data_ptr(), toks.data_ptr(),
                                     self.logits.data_ptr(), _stream()), "amk_decode_greedy")
        return toks

    def amk_last_status(self):
        st = C.c_int()
        msg = C.create_string_buffer(256)
        _check(lib.amk_last_status(self.h, C.byref(st), msg, 256), "amk_last_status")
        return st.value, msg.value.decode()

    def amk_debug_hidden(self) -> torch.Tensor:
        out = torch.empty((self.shape.n_layers + 1, self.shape.hidden), dtype=torch.float32)
        _check(lib.amk_debug_hidden(self.h, out.data_ptr()), "amk_debug_hidden")
        return out

    def amk_debug_trace(self) -> torch.Tensor:
        """int64 nanosecond stamps [n_blocks][5 L + 1][AMK_TRACE_EVENTS] of the last step."""
        nb, nt = self.plan().n_blocks, 5 * self.shape.n_layers + 1
        out = torch.zeros((nb, nt, AMK_TRACE_EVENTS), dtype=torch.int64)
        _check(lib.amk_debug_trace(self.h, out.data_ptr(), out.numel()), "amk_debug_trace")
        return out

    def amk_debug_unpack(self, layer: int, which: int):
        """Returns (codes, scale, zero) rebuilt from the packed buffer, canonical layouts."""
        s = self.shape
        qd, kvd = s.n_q_heads * s.head_dim, s.n_kv_heads * s.head_dim
        dims = [(qd, s.hidden), (kvd, s.hidden), (kvd, s.hidden), (s.hidden, qd), (s.mlp, s.hidden),
                (s.mlp, s.hidden), (s.hidden, s.mlp), (s.vocab, s.hidden)][which]
        wd = "bf16" if (which == AMK_LIN_LM_HEAD and not self.quantize_lm_head) else self.wdtype
        rows, cols = dims
        scale = zero = None
        if wd == "bf16":
            out = torch.zeros((rows, cols), dtype=torch.bfloat16, device=self.device)
        elif wd == "int8":
            out = torch.zeros((rows, cols), dtype=torch.int8, device=self.device)
            scale = torch.zeros((rows,), dtype=torch.float16, device=self.device)
        elif wd == "int8g":
            out = torch.zeros((rows, cols), dtype=torch.int8, device=self.device)
            scale = torch.zeros((rows, cols // 128), dtype=torch.float16, device=self.device)
        else:
            out = torch.zeros((rows, cols // 2), dtype=torch.uint8, device=self.device)
            scale = torch.zeros((rows, cols // 128), dtype=torch.float16, device=self.device)
            zero = torch.zeros((rows, cols // 128), dtype=torch.float16, device=self.device)
        _check(lib.amk_debug_unpack(self.h, layer, which, out.data_ptr(),
                                    None if scale is None else scale.data_ptr(),
                                    None if zero is None else zero.data_ptr(), _stream()), "amk_debug_unpack")
        return out, scale, zero

    def amk_debug_drop_signal(self, phase: int, block: int) -> None:
        _check(lib.amk_debug_drop_signal(self.h, phase, block), "amk_debug_drop_signal")

    def amk_last_kernel_ns(self) -> int:
        """Kernel-only nanoseconds of the last step (first block start to last block end); synchronises."""
        ns = C.c_uint64()
        _check(lib.amk_last_kernel_ns(self.h, C.byref(ns)), "amk_last_kernel_ns")
        return int(ns.value)

    def amk_debug_set_step_count(self, steps: int) -> None:
        _check(lib.amk_debug_set_step_count(self.h, steps), "amk_debug_set_step_count")

    def close(self) -> None:
        if getattr(self, "h", None):
            lib.amk_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
