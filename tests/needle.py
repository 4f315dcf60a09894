"""Needle inputs for the attention parity tests.  Not a test module.

With Gaussian keys every key carries about 1/n of the softmax weight, so on a long list a whole tile of
keys can go missing (or be counted twice) and move the output by less than the bf16 tolerance.  Here all
keys of a (sequence, head) have logits near zero except one, the needle, whose logit is ln(n) + 0.5: it
carries about 60 % of the weight.  Losing the needle's tile, or any tile's worth of the remaining weight
mis-scaled against it, moves O by a tenth and more and the log-sum-exp by far more than 1e-3.  Sweeping
the needle over the first and last key of every tile gives every tile and every cut between thread
blocks, key chunks and segments its turn.

Layout of a batch: nuggets of sequence b sit at positions 0 .. clen_b - 1, its local tokens follow at
clen_b .. clen_b + llen_b - 1, and its tq_b queries are the last tq_b local tokens unless q_pos0 says
otherwise (so a block of queries attends itself causally, Eq. 13, behind nuggets and local context, Eq. 9).
"""
from __future__ import annotations

import math

import numpy as np
import torch

from paper_2310_02409_b200 import inputs


def positions(n_c: int, n_l: int, tile: int) -> list[int]:
    """First and last key of every `tile`-key tile of the nugget segment and of the local segment
    (tiles restart at the segment boundary), as indices into the list [nuggets ; local]."""
    out = set()
    for base, n in ((0, n_c), (n_c, n_l)):
        for t0 in range(0, n, tile):
            out.add(base + t0)
            out.add(base + min(n, t0 + tile) - 1)
    return sorted(out)


def batch(dtype, H, dh, tqs, clens, llens, needles, tag, q_pos0=None, slack=3):
    """Host tensors and tables of one ragged batch.  needles: {(b, h): index into [nuggets ; local] of b}."""
    B = len(tqs)
    scale = dh ** -0.5
    q_off = inputs.offsets(tqs)
    cache_off = inputs.offsets([c + slack for c in clens])
    loc_off = inputs.offsets([l + slack for l in llens])
    T, C, Lr = max(int(q_off[-1]), 1), max(int(cache_off[-1]), 1), max(int(loc_off[-1]), 1)
    Q = inputs.randn((T, H, dh), tag, "nQ", std=0.25)
    cK = inputs.randn((C, H, dh), tag, "ncK", std=0.25)
    lK = inputs.randn((Lr, H, dh), tag, "nlK", std=0.25)
    cV = inputs.randn((C, H, dh), tag, "ncV")
    lV = inputs.randn((Lr, H, dh), tag, "nlV")
    Q[..., 0] = 4.0
    cK[..., 0] = 0.0
    lK[..., 0] = 0.0
    for (b, h), j in needles.items():
        n = clens[b] + llens[b]
        assert 0 <= j < n
        lift = (math.log(n) + 0.5) / (4.0 * scale)
        if j < clens[b]:
            cK[int(cache_off[b]) + j, h, 0] = lift
        else:
            lK[int(loc_off[b]) + j - clens[b], h, 0] = lift
    cpos = np.full(C, 2 ** 30, np.int32)                 # slack rows carry junk positions
    for b in range(B):
        cpos[cache_off[b]:cache_off[b] + clens[b]] = np.arange(clens[b])
    loc_pos0 = np.asarray(clens, np.int32)
    qp0 = np.asarray([clens[b] + llens[b] - tqs[b] for b in range(B)], np.int32) if q_pos0 is None \
        else np.asarray(q_pos0, np.int32)
    cast = lambda t: t.to(dtype)
    return dict(Q=cast(Q), cK=cast(cK), cV=cast(cV), lK=cast(lK), lV=cast(lV), cpos=cpos, q_off=q_off, q_pos0=qp0,
                cache_off=cache_off, clen=np.asarray(clens, np.int32), loc_off=loc_off[:-1].copy(),
                llen=np.asarray(llens, np.int32), loc_pos0=loc_pos0, scale=scale, H=H, dh=dh, T=int(q_off[-1]))


def oracle_result(oracle, c):
    """(O, lse) of the fp64 oracle for a batch made by batch()."""
    n = inputs.to_numpy
    return oracle.attend_ragged(n(c["Q"]), c["q_off"], c["q_pos0"], c["scale"], n(c["cK"]), n(c["cV"]), c["cpos"],
                                c["cache_off"], c["clen"], n(c["lK"]), n(c["lV"]), c["loc_off"], c["llen"], c["loc_pos0"])


def sweep(units, pos_lists):
    """Deal the positions of every sequence out over its heads, call after call.

    units: [(b, h)]; pos_lists: {b: [positions]}.  Yields one needles dict per call until every position of
    every sequence has been used once."""
    heads = {}
    for b, h in units:
        heads.setdefault(b, []).append(h)
    calls = max(math.ceil(len(pos_lists[b]) / len(hs)) for b, hs in heads.items())
    for c in range(calls):
        needles = {}
        for b, hs in heads.items():
            for i, h in enumerate(hs):
                at = c * len(hs) + i
                needles[(b, h)] = pos_lists[b][at % len(pos_lists[b])]
        yield needles


def max_errors(O: torch.Tensor, lse: torch.Tensor, ref, T: int):
    """max-abs error of O, of the finite log-sum-exps (-inf must match exactly), and the error of O in units
    of two bf16 roundings of the reference value (parity_log.rel_error)."""
    import parity_log
    got = O.float().cpu().numpy().astype(np.float64)[:T]
    gl = lse.cpu().numpy().astype(np.float64)[:T]
    Oo, lo = ref
    assert np.array_equal(np.isneginf(gl), np.isneginf(lo))
    fin = np.isfinite(lo)
    return (float(np.max(np.abs(got - Oo))), (float(np.max(np.abs(gl[fin] - lo[fin]))) if fin.any() else 0.0),
            parity_log.rel_error(got, Oo))
