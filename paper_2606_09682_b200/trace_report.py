"""Per-task time breakdown of a decode step from the kernel's own trace (AMK_FLAG_TRACE, amk_debug_trace).

    python -m paper_2606_09682_b200.trace_report --shape tinyllama_1b --wdtype bf16 --pos 0

Every block stamps the global timer (a quarter-microsecond clock) at the stages of every task; this prints, for a
layer in the middle of the model and for the LM head, the medians over blocks of the time between consecutive
stages, the skew between blocks, and when the block's producer issued the task's ring tiles relative to the moment
its consumers reached the task (negative: the weights were in shared memory or on their way before they were
needed).  With --cycles the stamps are SM cycle counters instead (differences within a block only) and the
figures are averages over all middle layers: finer, but each stamp costs the stamping warp ~100 cycles.
"""
from __future__ import annotations

import argparse

import numpy as np
import torch

from . import binding as amk
from . import inputs as inp

EV = dict(enter=0, joined=1, loaded=2, computed=3, signalled=4, prod_first=5, prod_last=6, reduced=7, pass_begin=8,
          first_tile=9, tiles_done=10, polls=11)
NAMES = ["QKV", "ATT", "O", "GU", "DOWN"]
CHAIN = ["enter", "joined", "loaded", "pass_begin", "first_tile", "tiles_done", "reduced", "computed"]
ATT_CHAIN = ["enter", "joined", "loaded", "pass_begin", "first_tile", "tiles_done", "reduced", "computed"]
ATT_LABEL = ["enter", "joined", "q gathered", "scores", "softmax", "P V", "partials in", "computed"]


def collect(shape, wdtype, pos, cycles, **knobs):
    w = amk.quantize_weights(inp.make_weights(shape, 7, device="cuda"), wdtype)
    flags = amk.AMK_FLAG_TRACE | (amk.AMK_FLAG_TRACE_CYCLES if cycles else 0)
    dec = amk.Decoder(shape, w, wdtype, flags=flags, **knobs)
    kv = inp.make_kv_prefill(shape, 5, pos, device="cuda")
    tok = inp.make_token(shape, 5)
    for _ in range(5):
        dec.amk_decode_step(tok, pos, kv)
    st, msg = dec.amk_last_status()
    if st != 0:
        raise RuntimeError(msg)
    tr = dec.amk_debug_trace().numpy().astype(np.float64)
    dec.close()
    return tr


def med(e, a, b):
    return float(np.median(e[:, EV[b]] - e[:, EV[a]]))


def report(tr, shape, pos, cycles):
    L = shape.n_layers
    unit = "cycles" if cycles else "ns"
    layers = list(range(2, L - 1)) if cycles else [L // 2]
    if not cycles:
        t0 = tr[:, 0, 0].min()
        total = tr[:, 5 * L, EV["computed"]].max() - t0
        per_layer = (tr[:, 5 * (L - 1) + 4, 3].max() - tr[:, 4, 3].max()) / (L - 1)
        print(f"step {total / 1e3:.1f} us; per layer {per_layer / 1e3:.2f} us")
    for k in (0, 2, 3, 4):
        acc = np.zeros(len(CHAIN) - 1)
        extra = []
        for l in layers:
            e = tr[:, 5 * l + k, :]
            acc += np.array([med(e, CHAIN[i], CHAIN[i + 1]) for i in range(len(CHAIN) - 1)])
            if not cycles:
                extra.append((e[:, 0].max() - np.median(e[:, 0]), e[:, 3].max() - np.median(e[:, 3]),
                              np.median(e[:, EV["polls"]]), med(e, "enter", "prod_first"), med(e, "enter", "prod_last")))
        acc /= len(layers)
        line = "  ".join(f"{CHAIN[i + 1]} +{acc[i]:.0f}" for i in range(len(acc)))
        print(f"{NAMES[k]:5s} ({unit}): {line}   total {acc.sum():.0f}")
        if extra:
            x = np.mean(np.array(extra), axis=0)
            print(f"        enter skew max-median {x[0]:.0f}, computed skew {x[1]:.0f}, gather rounds {x[2]:.0f}, "
                  f"producer issued first / last tile at {x[3]:+.0f} / {x[4]:+.0f} from enter")
    if pos > 0:
        acc = np.zeros(len(ATT_CHAIN) - 1)
        n = 0
        for l in layers:
            e = tr[:, 5 * l + 1, :]
            e = e[e[:, EV["computed"]] > 0]
            if len(e) == 0:
                continue
            acc += np.array([med(e, ATT_CHAIN[i], ATT_CHAIN[i + 1]) for i in range(len(ATT_CHAIN) - 1)])
            n += 1
        if n:
            acc /= n
            line = "  ".join(f"{ATT_LABEL[i + 1]} +{acc[i]:.0f}" for i in range(len(acc)))
            print(f"ATT   ({unit}): {line}   total {acc.sum():.0f}")
    e = tr[:, 5 * L, :]
    print(f"LM head ({unit}): joined +{med(e, 'enter', 'joined'):.0f}  loaded +{med(e, 'joined', 'loaded'):.0f}  "
          f"computed +{med(e, 'loaded', 'computed'):.0f}")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--shape", default="tinyllama_1b", choices=sorted(inp.SHAPES))
    ap.add_argument("--wdtype", default="bf16", choices=["bf16", "int8", "int4", "int8g"])
    ap.add_argument("--pos", type=int, default=0)
    ap.add_argument("--cycles", action="store_true")
    ap.add_argument("--sync-mode", type=int, default=1)
    a = ap.parse_args()
    shape = inp.SHAPES[a.shape]
    tr = collect(shape, a.wdtype, a.pos, a.cycles, sync_mode=a.sync_mode)
    print(f"{a.shape} {a.wdtype} pos {a.pos}" + (" (counter joins)" if a.sync_mode == 2 else ""))
    report(tr, shape, a.pos, a.cycles)
    torch.cuda.synchronize()


if __name__ == "__main__":
    main()
