"""What the needle inputs of the GPU parity tests can see, shown on the CPU oracle: a mistake is planted
in the oracle's input (a whole 64-key tile dropped, or counted twice) and the result is compared with the
correct one.  With needle inputs either mistake moves the output far beyond the attention tolerances; with
the Gaussian inputs of the other tests the same mistakes stay below the bf16 tolerance, which is why the
needle tests exist."""
import numpy as np
import torch

import needle
from paper_2310_02409_b200 import inputs


def _run(oracle, c, drop=None, twice=None):
    """Oracle on batch c (one sequence, nuggets only) with the nugget rows [drop) removed or [twice) repeated."""
    n = inputs.to_numpy
    cK, cV, cpos = n(c["cK"]), n(c["cV"]), c["cpos"]
    keep = np.arange(int(c["clen"][0]))
    if drop is not None:
        keep = np.concatenate([keep[:drop[0]], keep[drop[1]:]])
    if twice is not None:
        keep = np.concatenate([keep, np.arange(*twice)])
    return oracle.attend(n(c["Q"]), int(c["q_pos0"][0]), c["scale"], np.ascontiguousarray(cK[keep]),
                         np.ascontiguousarray(cV[keep]), np.ascontiguousarray(cpos[keep]), len(keep), None, None, 0, 0)


def test_a_lost_or_doubled_tile_is_visible_with_needles_and_not_without(oracle):
    H, dh, n_keys = 2, 128, 16896                     # the longest list of the workloads (13B shape, r = 1)
    j = 64 * 100 + 63                                 # last key of tile 100
    tile = (64 * 100, 64 * 101)
    c = needle.batch(torch.bfloat16, H, dh, [4], [n_keys], [0], {(0, 0): j, (0, 1): j}, ("needle-cpu",),
                     q_pos0=[n_keys])
    O, lse = _run(oracle, c)
    O_drop, lse_drop = _run(oracle, c, drop=tile)
    O_twice, lse_twice = _run(oracle, c, twice=tile)
    assert np.max(np.abs(O - O_drop)) > 0.2 and np.min(np.abs(lse - lse_drop)) > 0.5
    assert np.max(np.abs(O - O_twice)) > 0.05 and np.min(np.abs(lse - lse_twice)) > 0.3
    # another tile than the needle's: its 64 keys still carry 64/n of the remaining weight against the needle
    other = (64 * 7, 64 * 8)
    _, lse_other = _run(oracle, c, drop=other)
    assert np.min(np.abs(lse - lse_other)) > 1e-3
    # the same mistakes on Gaussian inputs hide inside the bf16 tolerance on O
    g = dict(c)
    for name in ("Q", "cK", "cV"):
        g[name] = inputs.randn(tuple(c[name].shape), "needle-cpu", "gauss", name, dtype=torch.bfloat16)
    Og, lg = _run(oracle, g)
    Og_drop, lg_drop = _run(oracle, g, drop=tile)
    assert np.max(np.abs(Og - Og_drop)) < 2e-2
    assert np.max(np.abs(lg - lg_drop)) > 1e-3         # ... but not on the log-sum-exp


def test_needle_positions_cover_every_tile_edge():
    p = needle.positions(130, 70, 64)
    assert p == [0, 63, 64, 127, 128, 129, 130, 193, 194, 199]
    calls = list(needle.sweep([(0, 0), (0, 1), (1, 0)], {0: [1, 2, 3], 1: [7]}))
    assert calls == [{(0, 0): 1, (0, 1): 2, (1, 0): 7}, {(0, 0): 3, (0, 1): 1, (1, 0): 7}]
