"""GPU parity at the full sizes of the LLaMA-shaped workloads (one layer each), in the launch
configuration the measurements use (`workloads.py`), against the fp64 CPU oracle.

Whatever the oracle finishes in seconds is compared in full: scores, indices, cache contents,
positions, single-token decode steps.  The query blocks (up to 512 queries over up to 16,896 keys
and 40 heads) and the 64-sequence ragged batch are compared on sampled outputs that the oracle
computes one by one: query rows on both sides of every 128-row tile boundary plus seeded random
ones, all heads; the shortest, the longest and seeded other sequences of the ragged batch.
"""
import numpy as np
import pytest
import torch

import parity_log
from paper_2310_02409_b200 import inputs

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2          # the stated tolerances
TOL_LSE = 1e-3
# Where the kernels sit on these shapes (Gaussian values, lists of 52 to 16,896 keys: outputs are small, so the
# one rounding to bf16 costs little): asserted beside the tolerances.  Largest seen: 1.9e-3 on the ragged batch
# (its shortest sequence has 52 nuggets), 7.5e-4 on the other configurations.
CEIL_O_LONG = 1.5e-3     # lists of at least 820 keys (the AR and the ratio-sweep configurations)
CEIL_O_RAGGED = 4e-3


def _host(t):
    return inputs.to_numpy(t)


def _f64(t):
    return t.float().cpu().numpy().astype(np.float64)


def _check_compress_full(oracle, inst):
    """Scores inside the fp32 band of fp64, indices bit-exact against TopK of the GPU's own scores,
    k = ceil(n/r), cache rows and positions bit-exact.  Returns the oracle's caches."""
    wl = inst.wl
    X, w = _host(inst.X), _host(inst.w)
    s_gpu = inst.scores.cpu().numpy()
    s64 = oracle.score(X, w, 0.0)
    mag = (inst.X.float().abs() @ inst.w.float().abs()).double().cpu().numpy()   # size of the band only
    assert np.all(np.abs(s_gpu.astype(np.float64) - s64) <= 1e-5 * (1.0 + 1.001 * mag))
    idx_o = oracle.select_ragged(s_gpu, inst.seq_off, inst.nug_off, 0)
    assert np.array_equal(inst.idx.cpu().numpy()[:int(inst.nug_off[-1])], idx_o)
    for b in range(wl.B):
        assert inst.nug_off[b + 1] - inst.nug_off[b] == oracle.num_nuggets(int(inst.n[b]), inst.r)
    cK = np.zeros_like(_host(inst.cacheK)); cV = np.zeros_like(cK)
    cpos = np.zeros(cK.shape[0], np.int32)
    lens = oracle.gather_ragged(_host(inst.K), _host(inst.V), inst.seq_off, idx_o, inst.nug_off,
                                np.zeros(wl.B, np.int32), cK, cV, cpos, inst.cache_off, [0] * wl.B)
    assert lens == inst.cache_len.tolist()
    assert np.array_equal(_host(inst.cacheK), cK) and np.array_equal(_host(inst.cacheV), cV)
    assert np.array_equal(inst.cache_pos.cpu().numpy(), cpos)
    return cK, cV, cpos, lens


def _sample_rows(tq, extra, *tags):
    """Query rows next to every 128-row tile boundary, the first and the last, plus seeded random ones."""
    rows = {0, tq - 1}
    for e in range(128, tq, 128):
        rows |= {e - 1, e}
    rs = np.random.RandomState(inputs.seed_for("rows", tq, *tags) % (2 ** 32))
    rows |= set(int(x) for x in rs.randint(0, tq, size=extra))
    return sorted(rows)


def _check_block_sampled(oracle, inst, caches, rows, tags, errlog):
    """Sampled rows of the query block, all heads, each computed by the oracle on its own: O and lse."""
    cK, cV, cpos, lens = caches
    loc_off, loc_len, loc_pos0, q_pos0 = inst.block_tables()
    Qb, Ob, Lb = _host(inst.Qb), _f64(inst.Ob), inst.lse_b.cpu().numpy().astype(np.float64)
    lK, lV = _host(inst.locK), _host(inst.locV)
    worst, worst_l = 0.0, 0.0
    for b in range(inst.wl.B):
        c0, l0 = int(inst.cache_off[b]), int(loc_off[b])
        for i in rows:
            row = int(inst.qb_off[b]) + i
            ref, ref_l = oracle.attend(Qb[row:row + 1], int(q_pos0[b]) + i, inst.sm_scale,
                                       cK[c0:c0 + lens[b]], cV[c0:c0 + lens[b]], cpos[c0:c0 + lens[b]], lens[b],
                                       lK[l0:l0 + int(loc_len[b])], lV[l0:l0 + int(loc_len[b])], int(loc_len[b]),
                                       int(loc_pos0[b]))
            worst = max(worst, float(np.max(np.abs(Ob[row] - ref[0]))))
            worst_l = max(worst_l, float(np.max(np.abs(Lb[row] - ref_l[0]))))
    errlog.add(f"fullsize query block {tags}", dense_O=worst, dense_lse=worst_l)
    assert worst <= TOL_BF16 and worst_l <= TOL_LSE, (tags, worst, worst_l)
    assert worst <= CEIL_O_LONG and worst_l <= parity_log.LSE_CEILING, (tags, worst, worst_l)
    return worst


def _check_decode_steps(oracle, inst, caches, steps, tags, errlog):
    cK, cV, cpos, lens = caches
    for s in steps:
        loc_off, loc_len, loc_pos0, q_pos0 = inst.window(s)
        ref, ref_l = oracle.attend_ragged(_host(inst.Qd[s]), inst.q_off, q_pos0, inst.sm_scale, cK, cV, cpos, inst.cache_off,
                                          lens, _host(inst.locK), _host(inst.locV), loc_off, loc_len, loc_pos0)
        err = float(np.max(np.abs(_f64(inst.Od[s]) - ref)))
        err_l = float(np.max(np.abs(inst.lse_d[s].cpu().numpy().astype(np.float64) - ref_l)))
        errlog.add(f"fullsize decode {tags} step {s}", decode_O=err, decode_lse=err_l)
        assert err <= TOL_BF16 and err_l <= TOL_LSE, (s, err, err_l)
        assert err <= CEIL_O_LONG and err_l <= parity_log.LSE_CEILING, (s, err, err_l)


def test_c3_llama7b_ar_full_size_one_layer(dodo, oracle, errlog):
    # 4 x 7168 compressed tokens -> 717 nuggets each, 1024 uncompressed, a 256-token query block on the
    # tensor-core kernel, then decode tokens with a growing window (first and last of the 64)
    from paper_2310_02409_b200.workloads import CompressDecode
    wl = inputs.WORKLOADS["c3_llama7b_ar"]
    inst = CompressDecode(dodo, wl, 10, ("c3-full",), with_lse=True)
    assert inst.k.tolist() == [717] * 4
    inst.compress()
    inst.query_block()
    steps = [0, wl.decode_steps - 1]
    for s in steps:
        inst.decode_step(s)
    torch.cuda.synchronize()
    caches = _check_compress_full(oracle, inst)
    _check_block_sampled(oracle, inst, caches, _sample_rows(wl.tq_dense, 6, "c3"), "c3", errlog)
    _check_decode_steps(oracle, inst, caches, steps, "c3", errlog)
    assert dodo.device_status() == 0


@pytest.mark.parametrize("r", [1, 5, 10, 20])
def test_c4_llama13b_ratio_sweep_full_size_one_layer(dodo, oracle, r, errlog):
    # one sequence of 16,384 tokens at 40 heads x 128, 512-token query block, 128 decode tokens
    from paper_2310_02409_b200.workloads import CompressDecode
    wl = inputs.WORKLOADS["c4_llama13b_sweep"]
    inst = CompressDecode(dodo, wl, r, ("c4-full", r), with_lse=True)
    assert int(inst.k[0]) == {1: 16384, 5: 3277, 10: 1639, 20: 820}[r]
    inst.compress()
    inst.query_block()
    steps = [0, wl.decode_steps - 1]
    for s in steps:
        inst.decode_step(s)
    torch.cuda.synchronize()
    caches = _check_compress_full(oracle, inst)
    rows = _sample_rows(wl.tq_dense, 4, "c4", r)
    _check_block_sampled(oracle, inst, caches, rows, ("c4", r), errlog)
    _check_decode_steps(oracle, inst, caches, steps, ("c4", r), errlog)
    if r == 1:
        # every token is a nugget: the block must equal full causal attention (Eq. 3) over
        # [context ; block], here by a library routine on the sampled rows
        assert np.array_equal(inst.idx.cpu().numpy(), np.arange(16384, dtype=np.int32))
        n, tq = 16384, wl.tq_dense
        k = torch.cat([inst.K, inst.locK[:tq]]).cpu().double().permute(1, 0, 2)
        v = torch.cat([inst.V, inst.locV[:tq]]).cpu().double().permute(1, 0, 2)
        q = inst.Qb[rows].cpu().double().permute(1, 0, 2)
        key_pos = torch.arange(n + tq)
        mask = key_pos[None, :] <= (n + torch.tensor(rows))[:, None]
        full = torch.nn.functional.scaled_dot_product_attention(q[None], k[None], v[None], attn_mask=mask, scale=inst.sm_scale)
        full = full[0].permute(1, 0, 2).numpy()
        assert np.max(np.abs(_f64(inst.Ob[rows]) - full)) <= TOL_BF16
    assert dodo.device_status() == 0


def test_c5_ragged_serving_full_size_one_layer(dodo, oracle, errlog):
    # 64 sequences, lengths log-uniform in [512, 32768] (489 k tokens), 256 decode steps with the
    # segment appends at steps 127, 191, 255.  Indices of every sequence are checked; scores, cache
    # contents and attention outputs on six sequences replayed by the oracle one by one.
    from paper_2310_02409_b200.workloads import RaggedServing
    wl = inputs.WORKLOADS["c5_ragged_serving"]
    lengths = list(wl.n_ctx)
    H, dh, S, r = wl.H, wl.dh, 64, 10
    srv = RaggedServing(dodo, lengths, wl.d, H, dh, r, wl.decode_steps, ("c5-full",), with_lse=True)
    B, st = srv.B, srv.steps
    srv.compress_context()
    torch.cuda.synchronize()
    N = int(srv.seq_off[-1])
    s_gpu = srv.scores.cpu().numpy()[:N].copy()
    idx_gpu = srv.idx.cpu().numpy()[:int(srv.nug_off0[-1])].copy()
    assert np.array_equal(idx_gpu, oracle.select_ragged(s_gpu, srv.seq_off, srv.nug_off0, 0))
    for b in range(B):
        assert srv.k0[b] == oracle.num_nuggets(lengths[b], r)

    rs = np.random.RandomState(inputs.seed_for("c5-full", "sample") % (2 ** 32))
    sample = sorted({int(np.argmin(lengths)), int(np.argmax(lengths))} | set(int(x) for x in rs.choice(B, 4, replace=False)))
    w = _host(srv.w)
    state = {}
    for b in sample:
        s0, s1 = int(srv.seq_off[b]), int(srv.seq_off[b + 1])
        s64 = oracle.score(_host(srv.X[s0:s1]), w, 0.0)
        mag = (srv.X[s0:s1].float().abs() @ srv.w.float().abs()).double().cpu().numpy()
        assert np.all(np.abs(s_gpu[s0:s1].astype(np.float64) - s64) <= 1e-5 * (1.0 + 1.001 * mag))
        cap = int(srv.cache_off[b + 1] - srv.cache_off[b])
        cK = np.zeros((cap, H, dh), np.uint16); cV = np.zeros_like(cK); cpos = np.zeros(cap, np.int32)
        ib = idx_gpu[srv.nug_off0[b]:srv.nug_off0[b + 1]]
        oracle.gather(_host(srv.K[s0:s1]), ib, 0, cK, cpos, 0)
        ln = oracle.gather(_host(srv.V[s0:s1]), ib, 0, cV, None, 0)
        state[b] = [cK, cV, cpos, ln]
    decX, decK, decV = _host(srv.decX), _host(srv.decK), _host(srv.decV)

    check = {0, 126, 127, 128, 191, 192, 255}
    win0, appended = 0, []
    for s in range(st):
        did = srv.decode_step(s)
        if s in check:
            torch.cuda.synchronize()
            Q, O, Ls = _host(srv.Qd[s]), _f64(srv.Od[s]), srv.lse_d[s].cpu().numpy().astype(np.float64)
            for b in sample:
                cK, cV, cpos, ln = state[b]
                ll = s + 1 - win0
                ref, ref_l = oracle.attend(Q[b:b + 1], lengths[b] + s, srv.sm_scale, cK, cV, cpos, ln,
                                           decK[b, win0:s + 1], decV[b, win0:s + 1], ll, lengths[b] + win0)
                err = float(np.max(np.abs(O[b] - ref[0])))
                err_l = float(np.max(np.abs(Ls[b] - ref_l[0])))
                errlog.add(f"fullsize c5 step {s} sequence {b}", decode_O=err, decode_lse=err_l)
                assert err <= TOL_BF16 and err_l <= TOL_LSE, (s, b, err, err_l)
                assert err <= CEIL_O_RAGGED and err_l <= parity_log.LSE_CEILING, (s, b, err, err_l)
        if did:
            appended.append(s)
            torch.cuda.synchronize()
            sg = srv.scores.cpu().numpy()[:B * S].copy()
            ig = srv.idx.cpu().numpy()[:B * srv.kS].copy()
            assert np.array_equal(ig, oracle.select_ragged(sg, srv.seg_off, srv.seg_nug_off, 0))
            for b in sample:
                cK, cV, cpos, ln = state[b]
                s64 = oracle.score(np.ascontiguousarray(decX[b, win0:win0 + S]), w, 0.0)
                assert np.max(np.abs(sg[b * S:(b + 1) * S] - s64)) < 1e-3
                ib = ig[b * srv.kS:(b + 1) * srv.kS]
                oracle.gather(np.ascontiguousarray(decK[b, win0:win0 + S]), ib, lengths[b] + win0, cK, cpos, ln)
                state[b][3] = oracle.gather(np.ascontiguousarray(decV[b, win0:win0 + S]), ib, lengths[b] + win0, cV, None, ln)
            win0 += S
    assert appended == [127, 191, 255]
    for b in range(B):
        assert srv.cache_len[b] == oracle.num_nuggets(lengths[b], r) + 3 * oracle.num_nuggets(S, r)
    for b in sample:
        cK, cV, cpos, ln = state[b]
        c0 = int(srv.cache_off[b])
        assert ln == srv.cache_len[b]
        assert np.array_equal(_host(srv.cacheK[c0:c0 + ln]), cK[:ln]) and np.array_equal(_host(srv.cacheV[c0:c0 + ln]), cV[:ln])
        assert np.array_equal(srv.cache_pos[c0:c0 + ln].cpu().numpy(), cpos[:ln])
    assert dodo.device_status() == 0
