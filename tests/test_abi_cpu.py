"""CPU-only checks of the boundary: the shared library loads, exports every symbol the header declares,
the Python mirror of the POD structs matches the C layout, the size queries and argument checks work
without a GPU, and the packed-weight geometry covers every matrix element exactly once."""
import ctypes as C
import os
import re
import subprocess

import pytest

from paper_2606_09682_b200 import build as amk_build
from paper_2606_09682_b200 import inputs as inp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "amk.h")


@pytest.fixture(scope="module")
def amk():
    amk_build.build()
    from paper_2606_09682_b200 import binding
    return binding


def header_functions():
    src = open(HEADER).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(amk_[a-z0-9_]+)\s*\(", src)))


def test_library_exports_every_declared_symbol(amk):
    names = header_functions()
    assert len(names) >= 15
    for n in names:
        assert hasattr(amk.lib, n), n
    assert sorted(amk.EXPORTS) == names


def test_struct_mirror_matches_header(amk, tmp_path):
    """Compile a tiny C program against the header and compare sizeof/offsetof with the ctypes mirror."""
    fields = [f for f, _ in amk.amk_config._fields_]
    plan_fields = [f for f, _ in amk.amk_plan._fields_]
    prog = ['#include <stdio.h>', '#include <stddef.h>', '#include "amk.h"', 'int main(void){',
            'printf("%zu %zu %zu\\n", sizeof(amk_config), sizeof(amk_weights), sizeof(amk_plan));']
    for f in fields:
        prog.append(f'printf("%zu\\n", offsetof(amk_config, {f}));')
    for f in plan_fields:
        prog.append(f'printf("%zu\\n", offsetof(amk_plan, {f}));')
    prog.append("return 0;}")
    src = tmp_path / "t.c"
    src.write_text("\n".join(prog))
    exe = tmp_path / "t"
    subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), "-o", str(exe), str(src)], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split()
    assert [int(x) for x in out[:3]] == [C.sizeof(amk.amk_config), C.sizeof(amk.amk_weights), C.sizeof(amk.amk_plan)]
    offs = [int(x) for x in out[3:]]
    assert offs[:len(fields)] == [getattr(amk.amk_config, f).offset for f in fields]
    assert offs[len(fields):] == [getattr(amk.amk_plan, f).offset for f in plan_fields]


def test_size_queries_and_argument_checks(amk):
    for name in ("smollm2_135m", "tinyllama_1b", "llama3_8b"):
        s = inp.SHAPES[name]
        for wd in ("bf16", "int8", "int4", "int8g"):
            cfg = amk.make_config(s, wd)
            if wd in ("int4", "int8g") and name == "smollm2_135m":       # hidden 576 is not a multiple of the group size 128
                with pytest.raises(amk.AmkError) as e:
                    amk.amk_packed_bytes(cfg)
                assert e.value.code == amk.AMK_ERR_UNSUPPORTED
                continue
            pb = amk.amk_packed_bytes(cfg)
            b = inp.streamed_bytes(s, wd, 0)
            # packed buffer = streamed weights and scales + a canonical embedding copy (+ alignment padding)
            expect = b["weights"] + b["scales"] - 2.0 * s.hidden + 2.0 * s.vocab * s.hidden
            if wd == "int8":
                # int8 rows are stored in whole blocks of 128 columns: an input length 64 short of a multiple of 128
                # is filled up with zero codes
                pad = lambda k: -(-k // 128) * 128 - k
                expect += s.n_layers * sum(r * pad(c) for r, c in (s.linear_dims(k) for k in inp.KINDS))
            slack = 0.02 if wd in ("int4", "int8g") else 1e-3        # units with scales inside are padded to 16 bytes
            assert 0 <= pb - expect < slack * expect + 1e6, (name, wd, pb, expect)
            assert amk.amk_kv_bytes(cfg) == 2 * s.n_layers * s.n_kv_heads * s.max_seq * s.head_dim * 2
            assert amk.amk_workspace_bytes(cfg) > 0
    cfg = amk.make_config(inp.SHAPES["mini"], "bf16")
    n = C.c_size_t()
    assert amk.lib.amk_packed_bytes(None, C.byref(n)) == amk.AMK_ERR_INVALID_ARG
    assert amk.lib.amk_packed_bytes(C.byref(cfg), None) == amk.AMK_ERR_INVALID_ARG
    cfg.struct_size = 12
    assert amk.lib.amk_packed_bytes(C.byref(cfg), C.byref(n)) == amk.AMK_ERR_INVALID_ARG
    cfg = amk.make_config(inp.SHAPES["mini"], "bf16")
    cfg.abi_version = 99
    assert amk.lib.amk_kv_bytes(C.byref(cfg), C.byref(n)) == amk.AMK_ERR_INVALID_ARG
    for field, val in (("head_dim", 48), ("n_q_heads", 3), ("quantize_lm_head", 1)):     # (a bf16 model has nothing to quantise its head like)
        cfg = amk.make_config(inp.SHAPES["mini"], "bf16")
        setattr(cfg, field, val)
        assert amk.lib.amk_packed_bytes(C.byref(cfg), C.byref(n)) == amk.AMK_ERR_UNSUPPORTED, field
    cfg = amk.make_config(inp.SHAPES["mini"], "int8", quantize_lm_head=True)
    assert amk.lib.amk_packed_bytes(C.byref(cfg), C.byref(n)) == amk.AMK_OK
    cfg.quantize_lm_head = 2
    assert amk.lib.amk_packed_bytes(C.byref(cfg), C.byref(n)) == amk.AMK_ERR_INVALID_ARG
    # limits of the plan: a task id is kept in 11 bits; sync_mode is 0 (automatic), 1 or 2
    cfg = amk.make_config(inp.SHAPES["mini"], "bf16")
    cfg.n_layers = 410
    assert amk.lib.amk_packed_bytes(C.byref(cfg), C.byref(n)) == amk.AMK_ERR_UNSUPPORTED
    cfg = amk.make_config(inp.SHAPES["mini"], "bf16", sync_mode=3)
    assert amk.lib.amk_packed_bytes(C.byref(cfg), C.byref(n)) == amk.AMK_ERR_INVALID_ARG
    for mode in (0, 1, 2):
        cfg = amk.make_config(inp.SHAPES["mini"], "bf16", sync_mode=mode)
        assert amk.lib.amk_packed_bytes(C.byref(cfg), C.byref(n)) == amk.AMK_OK
    # amk_create refuses buffers that are not 256-byte aligned before it touches the device
    cfg = amk.make_config(inp.SHAPES["mini"], "bf16")
    w = amk.amk_weights()
    h = C.c_void_p()
    for packed, ws in ((0x10000100 + 16, 0x20000000), (0x10000100 - 0x100, 0x20000000 + 128)):
        assert amk.lib.amk_create(C.byref(cfg), C.byref(w), packed, 1 << 30, ws, 1 << 30, None,
                                  C.byref(h)) == amk.AMK_ERR_INVALID_ARG
        assert not h.value
    # calls on a NULL handle fail cleanly
    assert amk.lib.amk_decode_step(None, 0, 0, None, None, None, None) == amk.AMK_ERR_INVALID_ARG
    assert amk.lib.amk_destroy(None) == amk.AMK_ERR_INVALID_ARG
    assert amk.lib.amk_status_str(amk.AMK_ERR_TIMEOUT) == b"device-side wait timed out"


@pytest.fixture(scope="module")
def layout_check(tmp_path_factory):
    exe = tmp_path_factory.mktemp("native") / "layout_check"
    subprocess.run(["g++", "-O2", "-std=c++17", "-I", os.path.join(ROOT, "paper_2606_09682_b200", "csrc"),
                    "-o", str(exe), os.path.join(ROOT, "tests", "native", "layout_check.cpp")], check=True)
    return str(exe)


@pytest.mark.parametrize("rows,K,wd,unit,nblk", [
    (2560, 2048, 0, 1, 148), (2048, 2048, 0, 1, 148), (11264, 2048, 0, 2, 148), (2048, 5632, 0, 1, 148),   # TinyLlama bf16
    (960, 576, 0, 1, 148), (3072, 576, 0, 2, 148), (576, 1536, 0, 1, 148),                                  # SmolLM2 shape
    (6144, 4096, 1, 1, 148), (28672, 4096, 1, 2, 148), (4096, 14336, 1, 1, 148),                            # Llama-3-8B int8
    (2560, 2048, 2, 1, 148), (11264, 2048, 2, 2, 148), (2048, 5632, 2, 1, 148),                             # TinyLlama int4
    (2560, 2048, 3, 1, 148), (11264, 2048, 3, 2, 148), (2048, 5632, 3, 1, 148), (300, 384, 3, 1, 132),      # grouped int8
    (1003, 192, 0, 1, 148), (7, 64, 0, 1, 148), (300, 320, 1, 1, 132), (5000, 1024, 0, 1, 7),               # odd cases
    (128256, 4096, 0, 1, 148), (49152, 576, 0, 1, 148),                                                     # LM heads
])
def test_packed_geometry_covers_every_element_once(layout_check, rows, K, wd, unit, nblk):
    for stage in (32768, 16384):
        r = subprocess.run([layout_check, str(rows), str(K), str(wd), str(unit), str(nblk), str(stage)],
                           capture_output=True, text=True)
        assert r.stdout.strip() == "ok", (r.stdout, r.stderr)
