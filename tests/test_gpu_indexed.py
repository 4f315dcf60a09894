"""GPU parity of dodo_attend_indexed: a query block attends the selected rows straight out of the uncompressed
K / V (row-gather tensor copies inside the tensor-core kernel), with no nugget cache in between.  The oracle is
the definition: gather the rows idx names (Eq. 5), then attend (Eq. 13 / Eq. 9).  Beside the tolerance against
the oracle, the result must equal, bit for bit, what dodo_gather_kv followed by dodo_attend gives on the same
inputs: the two paths put the same rows into the same tiles of the same kernel.
"""
import numpy as np
import pytest
import torch

import needle
import parity_log
from paper_2310_02409_b200 import inputs

pytestmark = pytest.mark.gpu

BF = torch.bfloat16


def _dev(x):
    return x.cuda() if isinstance(x, torch.Tensor) else torch.from_numpy(np.ascontiguousarray(x)).cuda()


def _case(dodo, oracle, H, tqs, ns, ks, llens, tag, q_pos0=None, pos_base=None, with_cache_path=True):
    """Ragged batch: sequence b has ns[b] context tokens of which ks[b] are selected (sorted random positions),
    llens[b] local tokens after the context, tqs[b] queries (the last local tokens unless q_pos0 says otherwise)."""
    dh, B = 128, len(tqs)
    scale = dh ** -0.5
    seq_off, nug_off, q_off = inputs.offsets(ns), inputs.offsets(ks), inputs.offsets(tqs)
    loc_off = inputs.offsets([l + 2 for l in llens])
    N, Kt, T, Lr = max(int(seq_off[-1]), 1), int(nug_off[-1]), max(int(q_off[-1]), 1), max(int(loc_off[-1]), 1)
    K = inputs.randn((N, H, dh), tag, "K", dtype=BF)
    V = inputs.randn((N, H, dh), tag, "V", dtype=BF)
    Q = inputs.randn((T, H, dh), tag, "Q", dtype=BF)
    lK = inputs.randn((Lr, H, dh), tag, "lK", dtype=BF)
    lV = inputs.randn((Lr, H, dh), tag, "lV", dtype=BF)
    rs = np.random.RandomState(inputs.seed_for(tag) % 2 ** 32)
    idx = np.concatenate([np.sort(rs.choice(ns[b], ks[b], replace=False)) for b in range(B)] + [np.zeros(0, np.int64)]).astype(np.int32)
    pb = np.zeros(B, np.int32) if pos_base is None else np.asarray(pos_base, np.int32)
    loc_pos0 = pb + np.asarray(ns, np.int32)
    qp0 = np.asarray([loc_pos0[b] + llens[b] - tqs[b] for b in range(B)], np.int32) if q_pos0 is None else np.asarray(q_pos0, np.int32)
    llen = np.asarray(llens, np.int32)
    ws = torch.empty(dodo.attend_workspace_bytes(dh), dtype=torch.uint8, device="cuda")
    Kd, Vd, Qd, lKd, lVd, idx_d = _dev(K), _dev(V), _dev(Q), _dev(lK), _dev(lV), _dev(idx if Kt else np.zeros(1, np.int32))
    O = torch.full((T, H, dh), float("nan"), dtype=BF, device="cuda")
    lse = torch.full((T, H), float("nan"), device="cuda")
    dodo.attend_indexed(Qd, q_off, qp0, scale, Kd, Vd, seq_off, idx_d, nug_off, pb, lKd, lVd, loc_off[:-1], llen, loc_pos0, O, lse, ws)
    torch.cuda.synchronize()
    # oracle: gather, then attend
    cK = np.zeros((max(Kt, 1), H, dh), np.uint16); cV = np.zeros_like(cK); cpos = np.zeros(max(Kt, 1), np.int32)
    lens = oracle.gather_ragged(inputs.to_numpy(K), inputs.to_numpy(V), seq_off, idx, nug_off, pb, cK, cV, cpos, nug_off, [0] * B)
    Oo, lo = oracle.attend_ragged(inputs.to_numpy(Q), q_off, qp0, scale, cK, cV, cpos, nug_off, lens, inputs.to_numpy(lK),
                                  inputs.to_numpy(lV), loc_off[:-1], llen, loc_pos0)
    Tn = int(q_off[-1])
    got, gl = O.float().cpu().numpy().astype(np.float64)[:Tn], lse.cpu().numpy().astype(np.float64)[:Tn]
    assert np.array_equal(np.isneginf(gl), np.isneginf(lo))
    fin = np.isfinite(lo)
    eo = float(np.max(np.abs(got - Oo))) if Tn else 0.0
    el = float(np.max(np.abs(gl[fin] - lo[fin]))) if fin.any() else 0.0
    parity_log.LOG.add(f"indexed attend {tag}", indexed_O=eo, indexed_lse=el)
    assert eo <= 2e-2 and el <= 1e-3, (tag, eo, el)
    assert el <= parity_log.LSE_CEILING, (tag, el)
    if with_cache_path:
        # the same call through a materialised cache: same tiles, same kernel -> the same bits
        cKd = torch.zeros((max(Kt, 1), H, dh), dtype=BF, device="cuda"); cVd = torch.zeros_like(cKd)
        cpd = torch.zeros(max(Kt, 1), dtype=torch.int32, device="cuda")
        clen = np.zeros(B, np.int32)
        dodo.gather_kv(Kd, Vd, seq_off, idx_d, nug_off, pb, cKd, cVd, cpd, nug_off, clen)
        O2 = torch.full_like(O, float("nan")); lse2 = torch.full_like(lse, float("nan"))
        # (query blocks shorter than the tensor-core threshold would go to the streaming kernel: force the same kernel)
        from paper_2310_02409_b200 import api
        dodo.set_tuning(api.TUNE_DENSE_MIN_QUERIES, 1)
        try:
            dodo.attend(Qd, q_off, qp0, scale, cKd, cVd, cpd, nug_off, clen, lKd, lVd, loc_off[:-1], llen, loc_pos0, O2, lse2, ws)
        finally:
            dodo.set_tuning(api.TUNE_DENSE_MIN_QUERIES, 32)
        torch.cuda.synchronize()
        assert torch.equal(O[:Tn], O2[:Tn]) and torch.equal(lse[:Tn], lse2[:Tn])
    return eo, el


@pytest.mark.parametrize("mode", [0, 1, 2, 3])
@pytest.mark.parametrize("H,tqs,ns,ks,llens", [
    (4, [128], [640], [64], [128]),                                     # exactly one tile of everything
    (4, [256, 37, 130], [7000, 500, 90], [717, 52, 0], [300, 37, 200]),  # ragged tails (717 = 11 tiles + 13 rows), no selection at all
    (2, [17, 231], [231, 878], [24, 88], [17, 231]),                   # the paper's one-shot sizes: 231- and 878-token documents
    (3, [300], [20000], [5003], [300]),                                # long list: 79 tiles, tail of 11 rows (not a multiple of 4)
])
def test_indexed_attend_matches_gather_then_attend(dodo, oracle, mode, H, tqs, ns, ks, llens):
    from paper_2310_02409_b200 import api
    dodo.set_tuning(api.TUNE_DENSE_BALANCE, mode)
    try:
        _case(dodo, oracle, H, tqs, ns, ks, llens, ("indexed", mode, tuple(ks)))
    finally:
        dodo.set_tuning(api.TUNE_DENSE_BALANCE, 0)
    assert dodo.device_status() == 0


def test_indexed_attend_masks_by_position(dodo, oracle):
    # queries inside the compressed region: selected tokens at later positions are invisible, the earliest queries
    # see nothing (O = 0, lse = -inf); positions are pos_base + idx
    _case(dodo, oracle, 2, [140, 40], [900, 300], [300, 64], [0, 50], "indexed-mask", q_pos0=[1000 - 2, 5000 + 150],
          pos_base=[1000, 5000])
    assert dodo.device_status() == 0


def test_indexed_attend_many_sequences(dodo, oracle):
    # more sequences than one launch group; some without queries, some without selection
    rs = np.random.RandomState(5)
    B = 70
    ns = [int(rs.randint(40, 400)) for _ in range(B)]
    ks = [0 if b % 11 == 3 else int(rs.randint(1, ns[b] // 3 + 2)) for b in range(B)]
    tqs = [0 if b % 9 == 4 else int(rs.randint(1, 150)) for b in range(B)]
    llens = [t + int(rs.randint(0, 30)) for t in tqs]
    _case(dodo, oracle, 2, tqs, ns, ks, llens, "indexed-many")
    assert dodo.device_status() == 0


def test_indexed_attend_needle_every_tile(dodo, oracle):
    # needle inputs (see needle.py) through the gathered path: the rows of a needle batch's cache are scattered over an
    # uncompressed array three times as long whose other rows would wreck the result if one of them were fetched
    H, tqs, clens, llens = 4, [200], [1300], [200]
    ws = torch.empty(dodo.attend_workspace_bytes(128), dtype=torch.uint8, device="cuda")
    units = [(0, h) for h in range(H)]
    pos = {0: needle.positions(clens[0], llens[0], 64)}
    n = 3 * clens[0]
    rs = np.random.RandomState(9)
    worst_o = worst_l = 0.0
    for call, needles in enumerate(needle.sweep(units, pos)):
        c = needle.batch(BF, H, 128, tqs, clens, llens, needles, ("indexed-needle", call))
        idx = np.sort(rs.choice(n, clens[0], replace=False)).astype(np.int32)
        K = torch.full((n, H, 128), 30.0, dtype=BF)            # a stray row would dominate every softmax
        V = torch.full((n, H, 128), -100.0, dtype=BF)
        K[idx] = c["cK"][:clens[0]]
        V[idx] = c["cV"][:clens[0]]
        pb = np.array([-n], np.int32)                          # all selected positions lie before the local tokens
        c["cpos"][:clens[0]] = pb[0] + idx
        ref = needle.oracle_result(oracle, c)
        O = torch.full((tqs[0], H, 128), float("nan"), dtype=BF, device="cuda")
        lse = torch.full((tqs[0], H), float("nan"), device="cuda")
        dodo.attend_indexed(_dev(c["Q"]), c["q_off"], c["q_pos0"], c["scale"], _dev(K), _dev(V), [0, n], _dev(idx), [0, clens[0]], pb,
                            _dev(c["lK"]), _dev(c["lV"]), c["loc_off"], c["llen"], c["loc_pos0"], O, lse, ws)
        torch.cuda.synchronize()
        eo, el, er = needle.max_errors(O, lse, ref, c["T"])
        assert eo <= 2e-2 and el <= 1e-3 and el <= parity_log.LSE_CEILING and er <= parity_log.REL_CEILING, (needles, eo, el, er)
        worst_o, worst_l = max(worst_o, eo), max(worst_l, el)
    parity_log.LOG.add("indexed attend, needle sweep", indexed_O=worst_o, indexed_lse=worst_l)
    assert dodo.device_status() == 0


def test_indexed_attend_reports_bad_indices_and_refuses_other_shapes(libdodo):
    from paper_2310_02409_b200 import api
    ctx = api.Dodo(0)
    try:
        H, dh, n = 2, 128, 100
        K = inputs.randn((2 * n, H, dh), "indexed-bad", "K", dtype=BF).cuda()
        V = inputs.randn((2 * n, H, dh), "indexed-bad", "V", dtype=BF).cuda()
        Q = inputs.randn((40, H, dh), "indexed-bad", "Q", dtype=BF).cuda()
        O = torch.zeros_like(Q)
        ws = torch.empty(ctx.attend_workspace_bytes(dh), dtype=torch.uint8, device="cuda")
        idx = torch.tensor([3, 7, n, 50], dtype=torch.int32, device="cuda")     # n is outside sequence 0 (but inside K: sequence 1's row 0)
        ctx.attend_indexed(Q, [0, 40, 40], [n, n], dh ** -0.5, K, V, [0, n, 2 * n], idx, [0, 4, 4], [0, 0], None, None, None, None, None,
                           O, None, ws)
        torch.cuda.synchronize()
        assert ctx.device_status() == api.DEV_BAD_INDEX and bool(torch.isfinite(O.float()).all())
        ctx.reset()
        with pytest.raises(api.DodoError) as e:        # fp32 is not served by the tensor-core kernel
            ctx.attend_indexed(Q.float(), [0, 40], [n], dh ** -0.5, K.float(), V.float(), [0, n], idx, [0, 4], [0], None, None, None, None,
                               None, O.float(), None, ws)
        assert e.value.status == api.ERR_UNSUPPORTED
        with pytest.raises(api.DodoError) as e:        # more selected rows than tokens
            ctx.attend_indexed(Q, [0, 40], [n], dh ** -0.5, K, V, [0, 3], idx, [0, 4], [0], None, None, None, None, None, O, None, ws)
        assert e.value.status == api.ERR_INVALID_ARG
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
    finally:
        ctx.close()
