"""GPU parity of dodo_attend on needle inputs (see needle.py): cases that the attention tolerance cannot
mask.  One key per (sequence, head) carries most of the softmax weight, and it is moved over the first and
last key of every key tile, so a tile that a kernel skipped, read twice, masked wrongly or merged with the
wrong scale shows as an error of a tenth and more in O and of far more than 1e-3 in the log-sum-exp.

Covered: the tensor-core kernel in its plain form and in both balanced forms (every cut between thread
blocks falls next to a swept key), on a list long enough that the default rule balances; the streaming
kernel without split, with its chunks merged in a thread-block cluster and merged through tickets, at one,
two and four queries per block, bf16 and fp32; compressor mode (a block attends itself causally behind the
nuggets, Eq. 13) and mixed resolution (nuggets plus an uncompressed window, Eq. 9).
"""
import numpy as np
import pytest
import torch

import needle
import parity_log

pytestmark = pytest.mark.gpu

TOL = {torch.bfloat16: 2e-2, torch.float32: 1e-4}


def _dev(x):
    return x.cuda() if isinstance(x, torch.Tensor) else torch.from_numpy(np.ascontiguousarray(x)).cuda()


def _gpu(dodo, c, ws):
    O = torch.full((max(c["T"], 1), c["H"], c["dh"]), float("nan"), dtype=c["Q"].dtype, device="cuda")
    lse = torch.full((max(c["T"], 1), c["H"]), float("nan"), device="cuda")
    dodo.attend(_dev(c["Q"]), c["q_off"], c["q_pos0"], c["scale"], _dev(c["cK"]), _dev(c["cV"]), _dev(c["cpos"]),
                c["cache_off"], c["clen"], _dev(c["lK"]), _dev(c["lV"]), c["loc_off"], c["llen"], c["loc_pos0"], O, lse, ws)
    torch.cuda.synchronize()
    return O, lse


def _sweep_case(dodo, oracle, dtype, H, dh, tqs, clens, llens, tile, tag, settings, q_pos0=None):
    """Every needle position of every sequence once; each call is run under every tuning in `settings`
    (a list of (knob, value) lists) against one oracle result.  Returns the worst (O, lse) errors."""
    from paper_2310_02409_b200 import api
    B = len(tqs)
    ws = torch.empty(dodo.attend_workspace_bytes(dh), dtype=torch.uint8, device="cuda")
    units = [(b, h) for b in range(B) for h in range(H) if tqs[b] > 0]
    pos = {b: needle.positions(clens[b], llens[b], tile) for b in range(B) if tqs[b] > 0}
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    defaults = {api.TUNE_ATTEND_TARGET_BLOCKS: 2 * sms, api.TUNE_DENSE_BALANCE: 0, api.TUNE_DENSE_MIN_QUERIES: 32}
    worst_o = worst_l = worst_r = 0.0
    ncalls = 0
    for needles in needle.sweep(units, pos):
        c = needle.batch(dtype, H, dh, tqs, clens, llens, needles, (tag, ncalls), q_pos0=q_pos0)
        ref = needle.oracle_result(oracle, c)
        for knobs in settings:
            try:
                for knob, value in knobs:
                    dodo.set_tuning(knob, value)
                O, lse = _gpu(dodo, c, ws)
            finally:
                for knob, value in defaults.items():
                    dodo.set_tuning(knob, value)
            eo, el, er = needle.max_errors(O, lse, ref, c["T"])
            assert eo <= TOL[dtype] and el <= 1e-3, (tag, needles, knobs, eo, el)          # the stated tolerances
            assert el <= parity_log.LSE_CEILING and er <= parity_log.REL_CEILING, (tag, needles, knobs, el, er)   # where the kernels sit
            worst_o, worst_l, worst_r = max(worst_o, eo), max(worst_l, el), max(worst_r, er)
        ncalls += 1
    assert dodo.device_status() == 0
    return worst_o, worst_l, worst_r, ncalls


def _balance_modes():
    from paper_2310_02409_b200 import api
    return [[(api.TUNE_DENSE_BALANCE, m)] for m in (0, 1, 2, 3)]


@pytest.mark.parametrize("name,H,tqs,clens,llens", [
    # compressor mode (Eq. 13): the block's own K/V are the local segment; two and three query tiles, ragged tails
    ("eq13", 4, [300, 129], [500, 52], [300, 129]),
    # mixed resolution (Eq. 9) at the shape of the autoregressive workload: 717 nuggets, a 1024-token window, the block
    ("eq9", 4, [256, 256], [717, 717], [1280, 1280]),
])
def test_dense_needle_every_tile(dodo, oracle, name, H, tqs, clens, llens):
    eo, el, er, n = _sweep_case(dodo, oracle, torch.bfloat16, H, 128, tqs, clens, llens, 64, ("needle-dense", name),
                                _balance_modes())
    parity_log.LOG.add(f"needle dense {name} ({n} calls x 4 balance modes)", needle_dense_O=eo, needle_dense_lse=el,
                       needle_dense_rel=er)


def test_dense_needle_long_list_default_balance(dodo, oracle):
    # 6200 nuggets = 97 key tiles per unit, 16 units for 296 resident blocks: the default rule (mode 0) balances
    # and keeps the two query tiles of a head in step; every unit is cut about 18 times
    eo, el, er, n = _sweep_case(dodo, oracle, torch.bfloat16, 8, 128, [256], [6200], [296], 64, ("needle-dense", "long"),
                                _balance_modes())
    parity_log.LOG.add(f"needle dense long list ({n} calls x 4 balance modes)", needle_dense_O=eo, needle_dense_lse=el,
                       needle_dense_rel=er)


def _targets(*values):
    from paper_2310_02409_b200 import api
    return [[(api.TUNE_ATTEND_TARGET_BLOCKS, v)] for v in values]


@pytest.mark.parametrize("name,dtype,H,dh,tqs,clens,llens,targets", [
    # the decode workload's shape (205 nuggets + a 64-token window): no split at the default target when the
    # heads fill the device, three chunks in a cluster otherwise, one granule per block at the largest target
    ("c2", torch.bfloat16, 8, 128, [1] * 8, [205] * 8, [64] * 8, (1, 296, 4096)),
    # one sequence, 40 heads (13B shape, r = 10): six chunks as one cluster; 4096: merged through tickets
    ("c4r10", torch.bfloat16, 40, 128, [1], [1639], [5], (296, 4096)),
    # ragged batch: chunk counts differ per sequence -> partial results and tickets
    ("ragged", torch.bfloat16, 4, 128, [1, 1, 1], [1000, 333, 64], [64, 0, 200], (1, 296, 4096)),
    ("ragged64", torch.bfloat16, 4, 64, [1, 1, 1], [1000, 333, 64], [64, 0, 200], (296, 4096)),
    # two and four queries per block, fp32, causal inside the block
    ("qt2", torch.float32, 4, 64, [2, 2], [900, 900], [40, 40], (296, 4096)),
    ("qt4", torch.float32, 2, 128, [4, 3], [1200, 700], [4, 9], (1, 296, 4096)),
])
def test_decode_needle_every_granule(dodo, oracle, name, dtype, H, dh, tqs, clens, llens, targets):
    from paper_2310_02409_b200 import api
    # (query blocks of up to four tokens stay on the streaming kernel whatever the threshold)
    eo, el, er, n = _sweep_case(dodo, oracle, dtype, H, dh, tqs, clens, llens, 64, ("needle-decode", name), _targets(*targets))
    kind = "needle_decode" if dtype == torch.bfloat16 else "needle_fp32"
    parity_log.LOG.add(f"needle decode {name} ({n} calls x {len(targets)} split targets)",
                       **{kind + "_O": eo, kind + "_lse": el, kind + "_rel": er})
