"""GPU check of amk_argmax_static, the token selection whose scratch memory is a fixed array inside the
library.  Collected last (file name), passes alone and after the other GPU tests.  It is compared with the
existing entry point: amk_decode_step returns the logits and the token its own LM-head tail chose, and the
static-scratch call must choose the same token from those logits, on two steps in a row and on two calls
in a row with nothing in between (the arrival counter has to be back at zero each time)."""
import numpy as np
import pytest
import torch

from paper_2606_09682_b200 import inputs as inp

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def amk():
    from paper_2606_09682_b200 import binding
    return binding


@pytest.mark.parametrize("name", ["mini_ragged", "mini_wide"])
def test_static_argmax_matches_decode_step_token_on_consecutive_calls(amk, name):
    shape = inp.SHAPES[name]
    w = inp.make_weights(shape, 77, device="cuda", norm_jitter=0.1)
    dec = amk.Decoder(shape, w, "bf16")
    kv = inp.make_kv_prefill(shape, 78, 0, device="cuda")
    tok = torch.full((4,), -1, dtype=torch.int32, device="cuda")
    token = inp.make_token(shape, 79)
    for pos in range(2):                      # two decode steps in a row, each followed by two static calls
        dec.amk_decode_step(token, pos, kv)
        st, msg = dec.amk_last_status()
        assert st == 0, msg
        amk.amk_argmax_static(dec.logits, tok[2 * pos:])
        amk.amk_argmax_static(dec.logits, tok[2 * pos + 1:])
        torch.cuda.synchronize()
        want = int(dec.next_token.item())
        assert int(tok[2 * pos].item()) == want and int(tok[2 * pos + 1].item()) == want, (pos, tok.tolist(), want)
        logits = dec.logits.cpu().numpy()
        assert want == int(np.argmax(logits))          # lowest index among equal maxima, as numpy
        token = want


@pytest.mark.parametrize("n", [1, 31, 2048, 2049, 32000, 128256, 1 << 20])
def test_static_argmax_sizes_ties_and_back_to_back_calls(amk, n):
    g = torch.Generator(device="cuda")
    g.manual_seed(n)
    x = torch.randn(n, generator=g, device="cuda")
    tok = torch.full((3,), -1, dtype=torch.int32, device="cuda")
    amk.amk_argmax_static(x, tok[0:])
    y = x.clone()
    top = float(x.max().item()) + 1.0
    y[n - 1] = top                            # the maximum twice: the lower index wins
    y[n // 2] = top
    amk.amk_argmax_static(y, tok[1:])
    amk.amk_argmax_static(x, tok[2:])         # and the first input again, straight after
    torch.cuda.synchronize()
    assert int(tok[0].item()) == int(torch.argmax(x).item())
    assert int(tok[1].item()) == n // 2
    assert int(tok[2].item()) == int(tok[0].item())


def test_static_argmax_rejects_sizes_beyond_its_scratch(amk):
    x = torch.zeros(16, device="cuda")
    tok = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    with pytest.raises(amk.AmkError) as e:
        amk.amk_argmax_static(x, tok, n=amk.AMK_ARGMAX_STATIC_MAX_N + 1)     # rejected before anything is read
    assert e.value.code == amk.AMK_ERR_UNSUPPORTED and "exceeds AMK_ARGMAX_STATIC_MAX_N" in str(e.value)
    with pytest.raises(amk.AmkError) as e:
        amk.amk_argmax_static(x, tok, n=0)
    assert e.value.code == amk.AMK_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert int(tok.item()) == -7
    amk.amk_argmax_static(x, tok)             # still usable afterwards; all equal -> index 0
    torch.cuda.synchronize()
    assert int(tok.item()) == 0


def test_static_argmax_nan_and_infinite_inputs(amk):
    """NaN elements are never chosen; nothing but NaNs gives index 0; -inf everywhere gives the lowest index."""
    tok = torch.full((3,), -1, dtype=torch.int32, device="cuda")
    x = torch.full((5000,), float("nan"), device="cuda")
    amk.amk_argmax_static(x, tok[0:])
    x2 = x.clone()
    x2[4097] = -3.0
    amk.amk_argmax_static(x2, tok[1:])
    amk.amk_argmax_static(torch.full((5000,), float("-inf"), device="cuda"), tok[2:])
    torch.cuda.synchronize()
    assert tok.tolist() == [0, 4097, 0]


def test_static_argmax_allocates_nothing_after_its_first_call(amk):
    """The point of the entry point: once the per-device set-up has run, a call takes no device memory -- neither
    through torch's allocator nor from the driver."""
    x = torch.randn(128256, device="cuda")
    tok = torch.zeros(1, dtype=torch.int32, device="cuda")
    amk.amk_argmax_static(x, tok)             # first call on the device: set-up
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for _ in range(20):
        amk.amk_argmax_static(x, tok)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == (alloc0, reserved0)
    assert free1 == free0, (free0, free1)
    assert int(tok.item()) == int(torch.argmax(x).item())


def test_static_argmax_rejects_host_memory(amk):
    import ctypes as C
    host = torch.zeros(16)
    tok = torch.zeros(1, dtype=torch.int32, device="cuda")
    msg = C.create_string_buffer(256)
    code = amk.lib.amk_argmax_static(host.data_ptr(), 16, tok.data_ptr(), msg, 256, None)
    assert code == amk.AMK_ERR_INVALID_ARG and b"not device memory" in msg.value
