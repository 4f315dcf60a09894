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
# O in bf16: the one rounding of the output costs up to 2^-9 |O|, and on the tensor-core kernel the rounding of
# every weight P to bf16 costs up to 2^-9 sum p |v| / sum p, about 2^-9 for value rows of unit scale: the error
# is measured in units of (|O_ref| + 1) / 256 per element, see rel_error().
REL_CEILING = 1.5


def rel_error(got, ref) -> float:
    """max over elements of |got - ref| / ((|ref| + 1) / 256): the error in units of what the bf16 roundings of
    an output of that size, made from value rows of unit scale, may cost."""
    import numpy as np
    return float(np.max(np.abs(got - ref) / ((np.abs(ref) + 1.0) / 256.0)))
