"""Knob search for the decode kernel with the paper's guards (Section 5, "Self-improving autoresearch"):

    candidate -> amk_create (which runs the static plan check) -> correctness gate -> CUDA-event median latency,
    never recorded without a correctness PASS -> keep / revert decided by an interleaved back-to-back A/B
    re-measurement against the incumbent (a candidate that only met a cooler clock is reverted) -> a
    physical-floor guard that withholds any latency below bytes / peak bandwidth as an artifact.

The search logic takes its three effects as callables -- `build(knobs)`, `correct(handle)`, `measure(handle, n)` --
so that it can be exercised without a GPU; `gpu_effects` supplies the real ones.  The knobs are the ones
amk_config exposes: ring stage size, copies in flight, L2 look-ahead (they change neither the arithmetic nor its
order, so the default correctness gate is bit-equality of logits and token with the default configuration's).

    python -m paper_2606_09682_b200.autotune --shape tinyllama_1b --wdtype bf16
"""
from __future__ import annotations

import argparse
import dataclasses
import itertools
import json
import statistics
from typing import Callable, Dict, Iterable, List, Optional


@dataclasses.dataclass(frozen=True)
class Knobs:
    stage_bytes: int = 0          # 0: the library's default
    max_inflight: int = 0
    l2_ahead: int = 0

    def kwargs(self) -> Dict[str, int]:
        return dataclasses.asdict(self)


@dataclasses.dataclass
class Trial:
    knobs: Knobs
    verdict: str                              # kept / reverted / rejected: <why>
    latency_us: Optional[float] = None        # only ever set after a correctness PASS and above the floor
    ab_us: Optional[List[float]] = None       # [candidate median, incumbent median] of the interleaved rounds


def default_grid() -> List[Knobs]:
    return [Knobs(s, i, a) for s, i, a in itertools.product((16384, 24576, 32768, 49152), (2, 3, 4), (2, 6))]


def tune(build: Callable[[Knobs], object], correct: Callable[[object], bool], measure: Callable[[object, int], float],
         release: Callable[[object], None], floor_us: float, grid: Optional[Iterable[Knobs]] = None,
         steps: int = 20, ab_rounds: int = 5, min_gain: float = 0.01, max_trials: int = 64) -> Dict:
    """Returns {"best": Knobs, "best_us": float, "trials": [Trial]}.  The incumbent starts as Knobs() (defaults).

    build    knobs -> handle, or raises (an infeasible point: rejected)
    correct  handle -> bool
    measure  (handle, steps) -> median microseconds per step
    floor_us bytes streamed per step / peak bandwidth: nothing real is faster
    """
    trials: List[Trial] = []
    inc_knobs = Knobs()
    inc = build(inc_knobs)
    if not correct(inc):
        release(inc)
        raise RuntimeError("the default configuration fails the correctness gate: nothing to tune against")
    inc_us = measure(inc, steps)
    if inc_us < floor_us:
        release(inc)
        raise RuntimeError(f"default configuration measured {inc_us:.1f} us, below the {floor_us:.1f} us floor: "
                           "the measurement is not to be trusted")
    trials.append(Trial(inc_knobs, "kept", inc_us))
    for knobs in itertools.islice((k for k in (grid if grid is not None else default_grid()) if k != Knobs()), max_trials):
        try:
            cand = build(knobs)
        except Exception as e:                     # infeasible point (e.g. the ring does not fit)
            trials.append(Trial(knobs, f"rejected: build ({e})"))
            continue
        try:
            if not correct(cand):
                trials.append(Trial(knobs, "rejected: correctness"))          # no latency without a PASS
                continue
            single = measure(cand, steps)
            if single < floor_us:
                trials.append(Trial(knobs, f"rejected: {single:.1f} us is below the physical floor {floor_us:.1f} us"))
                continue
            if single >= inc_us * (1.0 - min_gain):
                trials.append(Trial(knobs, "reverted", single))
                continue
            # looks faster: decide on interleaved back-to-back rounds, candidate and incumbent alternating
            c_us, i_us = [], []
            for _ in range(ab_rounds):
                c_us.append(measure(cand, steps))
                i_us.append(measure(inc, steps))
            c_med, i_med = statistics.median(c_us), statistics.median(i_us)
            if min(c_us) < floor_us:
                trials.append(Trial(knobs, "rejected: below the physical floor in the A/B rounds", None, [c_med, i_med]))
                continue
            if c_med < i_med * (1.0 - min_gain):
                trials.append(Trial(knobs, "kept", c_med, [c_med, i_med]))
                release(inc)
                inc, inc_knobs, inc_us, cand = cand, knobs, c_med, None
            else:
                trials.append(Trial(knobs, "reverted", c_med, [c_med, i_med]))
        finally:
            if cand is not None:
                release(cand)
    release(inc)
    return {"best": inc_knobs, "best_us": inc_us, "trials": trials}


def gpu_effects(shape, weights, wdtype: str, pos: int = 0, device="cuda", seed: int = 1):
    """(build, correct, measure, release, floor_us) on the current GPU.  The gate compares logits and token bit for
    bit with the default configuration's (the knobs change neither the arithmetic nor its order)."""
    import json as _json
    import os

    import numpy as np
    import torch

    from . import binding as amk
    from . import inputs as inp

    tok = inp.make_token(shape, seed)
    ref = {}

    def fresh_kv():
        return inp.make_kv_prefill(shape, seed + 1, pos, device=device)

    def build(knobs: Knobs):
        dec = amk.Decoder(shape, weights, wdtype, device=device, **knobs.kwargs())
        dec._kv = fresh_kv()
        return dec

    def correct(dec) -> bool:
        dec.amk_decode_step(tok, pos, dec._kv)
        st, _ = dec.amk_last_status()
        if st != 0:
            return False
        out = (dec.logits.clone(), int(dec.next_token.item()))
        if not ref:
            ref["out"] = out
            return bool(torch.isfinite(out[0]).all())
        return bool(torch.equal(out[0], ref["out"][0]) and out[1] == ref["out"][1])

    def measure(dec, steps: int) -> float:
        for _ in range(3):
            dec.amk_decode_step(tok, pos, dec._kv)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        ev[0].record()
        for i in range(steps):
            dec.amk_decode_step(tok, pos, dec._kv)
            ev[i + 1].record()
        torch.cuda.synchronize()
        return float(np.median([ev[i].elapsed_time(ev[i + 1]) * 1e3 for i in range(steps)]))

    def release(dec):
        dec.close()

    peak = 6544.7                                        # GB/s; replaced by the measured figure when present
    path = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            peak = float(_json.load(open(path))["hbm_gbs"])
        except Exception:
            pass
    # a pure read stream measures up to ~1.12x the copy figure on this part: the floor leaves that room
    floor_us = inp.streamed_bytes(shape, wdtype, pos)["total"] / (peak * 1.15 * 1e9) * 1e6
    return build, correct, measure, release, floor_us


def main():
    import torch

    from . import binding as amk
    from . import inputs as inp

    ap = argparse.ArgumentParser()
    ap.add_argument("--shape", default="tinyllama_1b", choices=sorted(inp.SHAPES))
    ap.add_argument("--wdtype", default="bf16", choices=["bf16", "int8", "int4", "int8g"])
    ap.add_argument("--pos", type=int, default=0)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--max-trials", type=int, default=24)
    a = ap.parse_args()
    shape = inp.SHAPES[a.shape]
    w = amk.quantize_weights(inp.make_weights(shape, 1, device="cuda"), a.wdtype)
    res = tune(*gpu_effects(shape, w, a.wdtype, a.pos), steps=a.steps, max_trials=a.max_trials)
    for t in res["trials"]:
        print(json.dumps({"knobs": t.knobs.kwargs(), "verdict": t.verdict, "us": t.latency_us, "ab": t.ab_us}))
    print(json.dumps({"best": res["best"].kwargs(), "best_us": res["best_us"]}))
    torch.cuda.synchronize()


if __name__ == "__main__":
    main()
