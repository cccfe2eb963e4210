"""Tolerance rule of the parity tests.

Target: max-abs error 2e-3 and max-rel error 1e-2 against the fp64 oracle for
16-bit inputs with fp32 accumulation.  A correctly rounded bf16 OUTPUT alone
has an error of up to 2^-9 relative (3.9e-3 absolute for values in [1, 2)),
and a relative error is meaningless next to zero, so:
  * fp32 output: max-abs <= 2e-3 and, over elements with |ref| >= 1e-2,
    max-rel <= 1e-2, both outright;
  * output in the storage type: no element may fail
    (abs err <= 2e-3) or (abs err <= 1e-2 * |ref|).
"""
import numpy as np

ABS_TOL = 2e-3
REL_TOL = 1e-2


def parity_report(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    err = np.abs(got - ref)
    big = np.abs(ref) >= 1e-2
    max_rel = float((err[big] / np.abs(ref[big])).max()) if big.any() else 0.0
    fails = int((~((err <= ABS_TOL) | (err <= REL_TOL * np.abs(ref)))).sum())
    return {"max_abs": float(err.max()) if err.size else 0.0, "max_rel": max_rel, "fails": fails}


def assert_parity(got, ref, native_out: bool, what=""):
    assert np.all(np.isfinite(np.asarray(got, dtype=np.float64))), f"{what}: non-finite output"
    r = parity_report(got, ref)
    if native_out:
        assert r["fails"] == 0, f"{what}: {r}"
    else:
        assert r["max_abs"] <= ABS_TOL and r["max_rel"] <= REL_TOL, f"{what}: {r}"
    return r
