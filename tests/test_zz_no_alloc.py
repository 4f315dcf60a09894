"""dodo_attend_noalloc: the attention entry point for callers that may not allocate device memory.

Such callers (a plug-in inside an engine whose pool owns the device, a path that cannot tolerate
cudaMalloc's synchronisation) cannot create a context or a workspace, so this entry point keeps its
scratch in a fixed device array inside the library.  The test calls it through the C ABI twice in a
row on different inputs -- the second call finds the first call's leftovers in the shared array --
and checks each result against the fp64 oracle within the attention tolerance of the other tests, and
against dodo_attend's as a second assertion.
Collected last on purpose: a run that stops at the first failure has then run everything else.
"""
import numpy as np
import pytest
import torch

from paper_2310_02409_b200 import inputs

pytestmark = pytest.mark.gpu

TOL = {torch.bfloat16: 2e-2, torch.float32: 1e-4}


def _batch(dtype, H, dh, clens, llens, tag, tqs=None):
    B = len(clens)
    tqs = [1] * B if tqs is None else tqs
    cache_off = inputs.offsets([c + 2 for c in clens])
    loc_off = inputs.offsets(llens)
    q_off = inputs.offsets(tqs)
    g = lambda rows, name: inputs.randn((max(rows, 1), H, dh), *tag, name, dtype=dtype).cuda()
    cK, cV = g(int(cache_off[-1]), "cK"), g(int(cache_off[-1]), "cV")
    lK, lV = g(int(loc_off[-1]), "lK"), g(int(loc_off[-1]), "lV")
    Q = g(int(q_off[-1]), "Q")
    cpos = np.zeros(max(int(cache_off[-1]), 1), np.int32)
    for b in range(B):
        cpos[cache_off[b]:cache_off[b] + clens[b]] = np.arange(clens[b]) * 2
    loc_pos0 = np.array([2 * c for c in clens], np.int32)
    # one query: every key is visible; several: they are the last local tokens and see each other causally
    q_pos0 = loc_pos0 + np.array(llens, np.int32) - np.array([t - 1 if t > 1 else 0 for t in tqs], np.int32)
    return dict(Q=Q, q_off=q_off, q_pos0=q_pos0, scale=dh ** -0.5, cK=cK, cV=cV, cpos_host=cpos,
                cpos=torch.from_numpy(cpos).cuda(), cache_off=cache_off, clen=np.array(clens, np.int32),
                lK=lK, lV=lV, loc_off=loc_off[:-1], llen=np.array(llens, np.int32), loc_pos0=loc_pos0)


def _oracle(oracle, c):
    n = inputs.to_numpy
    return oracle.attend_ragged(n(c["Q"]), c["q_off"], c["q_pos0"], c["scale"], n(c["cK"]), n(c["cV"]), c["cpos_host"],
                                c["cache_off"], c["clen"], n(c["lK"]), n(c["lV"]), c["loc_off"], c["llen"], c["loc_pos0"])


@pytest.mark.parametrize("dtype,dh", [(torch.bfloat16, 128), (torch.float32, 64)])
def test_noalloc_matches_oracle_and_attend_on_two_calls_in_a_row(dodo, oracle, dtype, dh):
    from paper_2310_02409_b200 import api
    H = 8
    ws = torch.empty(dodo.attend_workspace_bytes(dh), dtype=torch.uint8, device="cuda")
    cases = [_batch(dtype, H, dh, [205, 700, 13, 0], [64, 0, 7, 30], ("noalloc", 1, str(dtype))),
             _batch(dtype, H, dh, [90, 1500, 333], [5, 64, 0], ("noalloc", 2, str(dtype))),
             # query blocks of two and of seven tokens over long caches: two and four queries per thread block,
             # partial results per query row in the shared array
             _batch(dtype, H, dh, [1200, 40], [2, 9], ("noalloc", 3, str(dtype)), tqs=[2, 2]),
             _batch(dtype, H, dh, [2000, 900, 5], [7, 30, 8], ("noalloc", 4, str(dtype)), tqs=[7, 1, 3])]
    for c in cases:   # back to back: each call reuses the array the one before dirtied
        T = int(c["q_off"][-1])
        out = torch.full_like(c["Q"], float("nan"))
        out_lse = torch.full(c["Q"].shape[:2], float("nan"), device="cuda")
        api.attend_noalloc(c["Q"], c["q_off"], c["q_pos0"], c["scale"], c["cK"], c["cV"], c["cpos"], c["cache_off"],
                           c["clen"], c["lK"], c["lV"], c["loc_off"], c["llen"], c["loc_pos0"], out, out_lse)
        ref = torch.full_like(c["Q"], float("nan"))
        ref_lse = torch.full(c["Q"].shape[:2], float("nan"), device="cuda")
        dodo.attend(c["Q"], c["q_off"], c["q_pos0"], c["scale"], c["cK"], c["cV"], c["cpos"], c["cache_off"],
                    c["clen"], c["lK"], c["lV"], c["loc_off"], c["llen"], c["loc_pos0"], ref, ref_lse, ws)
        torch.cuda.synchronize()
        # first against the oracle ...
        Oo, lo = _oracle(oracle, c)
        err = float(np.max(np.abs(out.float().cpu().numpy().astype(np.float64)[:T] - Oo)))
        err_l = float(np.max(np.abs(out_lse.cpu().numpy().astype(np.float64)[:T] - lo)))
        assert err <= TOL[dtype] and err_l <= 1e-3, (err, err_l)
        # ... then against the entry point that takes a context and a workspace
        assert float((out.float() - ref.float()).abs().max()) <= TOL[dtype]
        assert float((out_lse - ref_lse).abs().max()) <= 1e-3


def test_noalloc_rejects_what_does_not_fit(dodo):
    from paper_2310_02409_b200 import api
    c = _batch(torch.bfloat16, 2, 128, [10] * 65, [0] * 65, ("noalloc", "big"))
    out = torch.zeros_like(c["Q"])
    with pytest.raises(api.DodoError) as e:      # more sequences than one call may carry
        api.attend_noalloc(c["Q"], c["q_off"], c["q_pos0"], c["scale"], c["cK"], c["cV"], c["cpos"], c["cache_off"],
                           c["clen"], c["lK"], c["lV"], c["loc_off"], c["llen"], c["loc_pos0"], out, None)
    assert e.value.status == api.ERR_CAPACITY and "64" in str(e.value)
    # (The other refusal, a split plan larger than the array, cannot be provoked on this device: a split happens
    # only below 2 x SMs (query tile, head) units and then writes at most 16 x 2 x SMs partial rows, 2.5 MB at
    # head size 128 on 148 SMs.  The check guards devices with more than about 250 SMs.)
