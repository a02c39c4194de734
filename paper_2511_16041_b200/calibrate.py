"""Calibration of the tiling-selection model on the GPU at hand.

The constants of ``atb_hw_params_b200`` were fitted on one B200.  This module repeats that procedure
(the paper's Section 7 names automatic calibration and search as future work): it times ``atb_gemm``
for a set of tilings on a set of shapes, then searches a grid of model constants for the set under
which ``atb_select_tiling`` picks, shape by shape, a tiling as close as possible to the fastest one
measured.  The result is a plain dict / JSON file that ``load_hw_params`` turns back into the
structure ``atb_select_tiling`` accepts.

    python -m paper_2511_16041_b200.calibrate --out atb_hw_params.json            # full: ~1 minute
    python -m paper_2511_16041_b200.calibrate --quick --out atb_hw_params.json    # 5 shapes

Only ``measure`` needs a GPU; ``fit`` is host arithmetic on the records.
"""
from __future__ import annotations

import argparse
import itertools
import json
import math
from typing import Dict, Iterable, List, Optional, Sequence, Tuple

from . import (atb_hw_params_b200, atb_hw_params_t, atb_select_tiling, atb_tiling_supported)

Shape = Tuple[int, int, int]
TilingT = Tuple[int, int, int, int]

# The constants the search moves, with the values it tries.  Everything else keeps its preset value.
DEFAULT_GRID: Dict[str, Sequence[float]] = {
    "convert_cycles": (300.0, 400.0),
    "convert_exposed_cycles": (20.0, 45.0),
    "convert_latency_cycles": (700.0, 1200.0),
    "load_latency_cycles": (800.0, 1200.0, 1600.0),
    "delta_cycles": (20.0, 45.0, 90.0),
    "pair_efficiency": (0.95, 1.0),
    "tile_fixed_cycles": (1000.0, 3000.0),
    "drain_cycles_per_column": (2.0, 4.0),
    "pair_tile_cycles": (2000.0, 4000.0),
    "thin_slab_cost": (0.3, 0.6),
}

FULL_SHAPES: List[Shape] = [
    (2048, 2048, 2048), (4096, 4096, 4096), (8192, 8192, 8192), (16384, 16384, 4096), (8192, 8192, 1024),
    (8192, 8192, 2048), (4096, 14336, 4096), (4096, 4096, 14336), (1024, 4096, 4096), (16384, 2048, 8192),
    (2048, 16384, 8192), (4096, 8192, 16384), (3000, 5000, 7008), (8192, 1024, 4096), (1024, 8192, 2048),
]
QUICK_SHAPES: List[Shape] = [(2048, 2048, 2048), (4096, 4096, 4096), (8192, 8192, 2048), (4096, 4096, 14336),
                             (1024, 8192, 2048)]


def all_tilings() -> List[TilingT]:
    """Every tiling ``atb_gemm`` accepts."""
    return [(ma, mc, k, n) for mc in (128, 256, 384) for n in (64, 128, 256, 512) for k in (64, 128)
            for ma in (32, 64, 128, 256) if ma <= mc and mc % ma == 0 and atb_tiling_supported(ma, mc, k, n)]


def measure(shapes: Iterable[Shape], tilings: Optional[Iterable[TilingT]] = None, reps: int = 5,
            device: str = "cuda:0") -> List[dict]:
    """Times ``atb_gemm`` (best of ``reps`` launches, CUDA events) for every tiling on every shape.
    Operands are random BFP16 planes and a random BF16 matrix: the rate does not depend on the values."""
    import torch
    from . import atb_bfp16_exp_bytes, atb_device_status, atb_gemm

    shapes = list(shapes)
    tilings = list(tilings) if tilings is not None else all_tilings()
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(1)
    mk = max(m * k for m, _, k in shapes)
    kn = max(k * n for _, n, k in shapes)
    mn = max(m * n for m, n, _ in shapes)
    exp_bytes = max(atb_bfp16_exp_bytes(m, k) for m, _, k in shapes)
    mant = torch.randint(-127, 128, (mk,), dtype=torch.int8, device=dev, generator=g)
    expp = torch.randint(125, 130, (exp_bytes,), dtype=torch.uint8, device=dev, generator=g)
    B = torch.randn((kn,), device=dev, generator=g).to(torch.bfloat16)
    C = torch.empty((mn,), dtype=torch.bfloat16, device=dev)
    def time_one(M, N, K, til, n):
        for _ in range(2):
            atb_gemm(M, N, K, *til, mant, expp, B, C, ldb=N, ldc=N)
        events = []
        for _ in range(n):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            atb_gemm(M, N, K, *til, mant, expp, B, C, ldb=N, ldc=N)
            b.record()
            events.append((a, b))
        torch.cuda.synchronize()
        return min(a.elapsed_time(b) for a, b in events)

    # The rate a tiling shows depends a little on what ran just before it (power state), so every shape is
    # walked twice, in opposite orders, and a tiling keeps its better time.
    records = []
    for (M, N, K) in shapes:
        best = {}
        for order in (tilings, tilings[::-1]):
            for til in order:
                ms = time_one(M, N, K, til, max(reps // 2, 2))
                best[til] = min(ms, best.get(til, ms))
        for til in tilings:
            records.append({"M": M, "N": N, "K": K, "tiling": list(til), "ms": best[til],
                            "tflops": 2.0 * M * N * K / best[til] / 1e9})
    atb_device_status()
    return records


def make_hw(values: Optional[Dict[str, float]] = None) -> atb_hw_params_t:
    """The B200 preset with ``values`` written over it."""
    hw = atb_hw_params_b200()
    for name, v in (values or {}).items():
        if not hasattr(hw, name):
            raise KeyError("atb_hw_params_t has no field %r" % name)
        setattr(hw, name, type(getattr(hw, name))(v))
    return hw


def hw_to_dict(hw: atb_hw_params_t) -> Dict[str, float]:
    return {name: getattr(hw, name) for name, _ in hw._fields_}


def load_hw_params(path: str) -> atb_hw_params_t:
    """Reads a JSON file written by this module (or any dict of field values) into the structure."""
    with open(path) as f:
        data = json.load(f)
    return make_hw(data.get("hw_params", data))


def _by_shape(records: Iterable[dict]) -> Dict[Shape, Dict[TilingT, float]]:
    out: Dict[Shape, Dict[TilingT, float]] = {}
    for r in records:
        out.setdefault((r["M"], r["N"], r["K"]), {})[tuple(r["tiling"])] = r["tflops"]
    return out


def evaluate(hw: atb_hw_params_t, records: Iterable[dict]) -> Dict[str, float]:
    """How well the selection does under ``hw``: for each shape, the measured rate of the best-scored
    measured tiling over the best measured rate ("pick quality", 1 = the model finds the fastest), and
    the r.m.s. error of log(predicted / measured)."""
    quality, sq = [], []
    for shape, meas in _by_shape(records).items():
        _, scores = atb_select_tiling(*shape, hw=hw, max_scores=256)
        ranked = [(s.t.T_MA, s.t.T_MC, s.t.T_K, s.t.T_N) for s in scores]      # the selection's own order
        pred = {t: s.predicted_flops / 1e12 for t, s in zip(ranked, scores)}
        known = {t: v for t, v in meas.items() if t in pred}
        if not known:
            continue
        pick = next(t for t in ranked if t in known)
        quality.append(known[pick] / max(known.values()))
        sq += [(math.log(pred[t]) - math.log(v)) ** 2 for t, v in known.items() if v > 0 and pred[t] > 0]
    return {"pick_quality_mean": sum(quality) / len(quality), "pick_quality_min": min(quality),
            "rms_log_error": math.sqrt(sum(sq) / len(sq)), "shapes": len(quality)}


def fit(records: Iterable[dict], grid: Optional[Dict[str, Sequence[float]]] = None) -> Tuple[Dict[str, float], Dict[str, float]]:
    """Exhaustive search of ``grid`` (name -> candidate values).  Objective: mean pick quality, then the
    worst shape's, then the absolute error - the selection is rated by what it picks, the absolute
    prediction only breaks ties.  Returns (best values, their evaluation)."""
    records = list(records)
    grid = dict(grid or DEFAULT_GRID)
    names = list(grid)
    best_key, best_vals, best_eval = None, None, None
    for combo in itertools.product(*(grid[n] for n in names)):
        vals = dict(zip(names, combo))
        ev = evaluate(make_hw(vals), records)
        key = (round(ev["pick_quality_mean"] + 0.3 * ev["pick_quality_min"], 6), -ev["rms_log_error"])
        if best_key is None or key > best_key:
            best_key, best_vals, best_eval = key, vals, ev
    return best_vals, best_eval


def main(argv: Optional[Sequence[str]] = None) -> int:
    ap = argparse.ArgumentParser(description=__doc__.split("\n\n")[0])
    ap.add_argument("--out", default="atb_hw_params.json")
    ap.add_argument("--quick", action="store_true", help="5 shapes instead of 15")
    ap.add_argument("--records", default=None, help="fit these records (JSON lines) instead of measuring")
    ap.add_argument("--reps", type=int, default=5)
    args = ap.parse_args(argv)
    if args.records:
        with open(args.records) as f:
            records = [json.loads(line) for line in f if line.strip()]
    else:
        records = measure(QUICK_SHAPES if args.quick else FULL_SHAPES, reps=args.reps)
    before = evaluate(atb_hw_params_b200(), records)
    values, after = fit(records)
    with open(args.out, "w") as f:
        json.dump({"hw_params": hw_to_dict(make_hw(values)), "fitted": values, "evaluation": after,
                   "preset_evaluation": before, "records": len(records)}, f, indent=1)
    print("preset : %s" % before)
    print("fitted : %s" % after)
    print("values : %s" % values)
    print("written: %s" % args.out)
    return 0


if __name__ == "__main__":
    raise SystemExit(main())
