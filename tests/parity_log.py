"""Observed maximum errors of the GPU parity tests, kept per test and written out at the end of the
session, so that the margins to the stated tolerances can be read and not only the pass/fail.

Keys name the path and the quantity (``dense_O``, ``decode_lse`` ...); values are max-abs errors against the
fp64 oracle.  Not a test module.
"""
from __future__ import annotations

import json
from pathlib import Path


class ErrorLog:
    def __init__(self):
        self.rows = []

    def add(self, test: str, **values):
        self.rows.append({"test": test, **{k: float(v) for k, v in values.items()}})

    def worst(self) -> dict:
        out = {}
        for r in self.rows:
            for k, v in r.items():
                if k != "test":
                    out[k] = max(out.get(k, 0.0), v)
        return out

    def dump(self, path: Path):
        if not self.rows:
            return
        try:
            path.parent.mkdir(exist_ok=True)
            path.write_text(json.dumps({"worst": self.worst(), "rows": self.rows}, indent=1))
        except OSError:
            pass


LOG = ErrorLog()

# Empirical ceilings, asserted beside the stated tolerances (2e-2 bf16 / 1e-4 fp32 on O, 1e-3 on the log-sum-exp).
# Log-sum-exp: fp32 arithmetic on both kernel families; the largest value seen over all tests is 4e-6.
LSE_CEILING = 2e-5
# O in bf16 is dominated by the one rounding of the output (relative 2^-9) plus, on the tensor-core kernel, the
# rounding of the weights P to bf16: measured against 2^-8 |O_ref| + 1e-3 per element, see rel_error().
REL_CEILING = 2.0


def rel_error(got, ref) -> float:
    """max over elements of |got - ref| / (2^-8 |ref| + 1e-3): the error in units of what two bf16 roundings of
    a value of that size may cost (plus a small absolute floor for values near zero)."""
    import numpy as np
    return float(np.max(np.abs(got - ref) / (np.abs(ref) / 256.0 + 1e-3)))
