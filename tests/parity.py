"""Parity bookkeeping for the GPU tests: every comparison with the oracle is recorded, and only
comparisons named on an explicit allow-list may use anything but the stated tolerance.

Stated tolerances (relative L2 per tensor):
    strict fp32 mode : 1e-4 everywhere
    bf16 mode        : block outputs / logits 2e-2, gradients 5e-2

Two rules, chosen per comparison by the CALLER, never by the outcome:

  "stated"  the error must not exceed the stated tolerance.  Every block-level case, every stored
            transition, the per-block checks inside the full-size networks and the forward
            quantities use it.

  "floor"   for END-TO-END gradients of a deep BN-ReLU stack only.  Those are discontinuous in the
            activations (an element whose pre-activation changes sign moves a term in or out of
            every sum behind it), so the oracle's own gradients move when its input is perturbed by
            the size of the rounding differences between any two implementations.  The test
            measures that movement ("floor": input times 1 +- 1e-6, and one grid step on a
            fixed-point state) and accepts an error up to FLOOR_FACTOR x floor, never more than
            MAX_BOUND.  MAX_BOUND = 0.7 keeps the cosine between the two tensors above 0.71 and
            rejects a zero tensor (error 1.0), an uncorrelated one (1.41) and a wrong sign (2.0).

Each record says which rule applied and whether the stated tolerance was met anyway.  The session
writes them to the JSON file named by REVNET_PARITY_REPORT (if set) and prints a summary.
"""
import fnmatch
import json
import os

import numpy as np

from tests import helpers as hp

TOL = {1: dict(out=1e-4, grad=1e-4), 0: dict(out=2e-2, grad=5e-2)}
RECON = 1e-3
FLOOR_FACTOR = 3.0
MAX_BOUND = 0.7

RECORDS = []


def cosine(a, b):
    a = np.asarray(a, np.float64).ravel(); b = np.asarray(b, np.float64).ravel()
    d = np.linalg.norm(a) * np.linalg.norm(b)
    return float(a @ b / d) if d > 0 else 1.0


def check(case, got, ref, tol, floor_fn=None, floor_allowed=()):
    """Compare dicts of tensors.  A tensor whose name matches a pattern in `floor_allowed` is held to
    max(tol, FLOOR_FACTOR x floor) <= MAX_BOUND, everything else to `tol`.  floor_fn() returns a list
    of dicts: the oracle's outputs for perturbed inputs (called only if some allowed tensor misses tol).
    Returns (worst error, worst floor)."""
    assert set(ref) <= set(got), (case, sorted(set(ref) - set(got)))
    errs = {k: hp.rel_l2(got[k], ref[k]) for k in ref}
    allowed = {k for k in ref if any(fnmatch.fnmatchcase(k, p) for p in floor_allowed)}
    floors = {}
    if floor_fn is not None and any(errs[k] > tol for k in allowed):
        for alt in floor_fn():
            for k in allowed:
                floors[k] = max(floors.get(k, 0.0), hp.rel_l2(alt[k], ref[k]))
    bad = {}
    for k, e in errs.items():
        if k in allowed:
            fl = floors.get(k, 0.0)
            bound = min(MAX_BOUND, max(tol, FLOOR_FACTOR * fl))
            rule = "floor"
        else:
            fl, bound, rule = None, tol, "stated"
        RECORDS.append(dict(case=case, tensor=k, err=e, tol=tol, rule=rule, floor=fl, bound=bound,
                            met_stated=bool(e <= tol), cos=cosine(got[k], ref[k]), ok=bool(e <= bound)))
        if not e <= bound:
            bad[k] = (e, bound)
    assert not bad, f"{case}: (error, bound) {bad}"
    return max(errs.values()), max(floors.values(), default=0.0)


def summary():
    """One line per case: tensors compared, how many by each rule, worst error and where."""
    by = {}
    for r in RECORDS:
        c = by.setdefault(r["case"], dict(n=0, stated=0, floor=0, floor_used=0, worst=0.0, worst_t="", tol=r["tol"], worst_floor=0.0, min_cos=1.0))
        c["n"] += 1
        c[r["rule"]] += 1
        if r["rule"] == "floor" and not r["met_stated"]:
            c["floor_used"] += 1
            c["worst_floor"] = max(c["worst_floor"], r["floor"] or 0.0)
        if r["err"] >= c["worst"]:
            c["worst"], c["worst_t"] = r["err"], r["tensor"]
        c["min_cos"] = min(c["min_cos"], r["cos"])
    return by


def write_report():
    path = os.environ.get("REVNET_PARITY_REPORT")
    if not RECORDS:
        return
    by = summary()
    lines = ["case | tensors | held to stated tol | floor rule allowed | needed the floor | worst err (tensor) | stated tol | worst floor | min cos"]
    for c, v in by.items():
        lines.append(f"{c} | {v['n']} | {v['stated']} | {v['floor']} | {v['floor_used']} | {v['worst']:.3e} ({v['worst_t']}) | {v['tol']:g} | "
                     f"{v['worst_floor']:.3e} | {v['min_cos']:.4f}")
    text = "\n".join(lines)
    print("\n" + text)
    if path:
        os.makedirs(os.path.dirname(os.path.abspath(path)), exist_ok=True)
        with open(path, "w") as f:
            json.dump(dict(records=RECORDS, summary=by), f)
        with open(os.path.splitext(path)[0] + ".txt", "w") as f:
            f.write(text + "\n")
