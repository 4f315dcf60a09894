"""Seeded random shapes through the C ABI against the fp64 oracle: ragged batches whose sizes are drawn
rather than picked by hand, so that tile boundaries, empty pieces, launch-group cuts, split plans and
the choice between the streaming and the tensor-core attend kernel are hit in combinations no
hand-written case lists.  Every case is reproducible from its number.
"""
import numpy as np
import pytest
import torch

from paper_2310_02409_b200 import inputs
from test_gpu_parity import ATTEND_TOL, _attend_case, _select_gpu, dev

pytestmark = pytest.mark.gpu


def _rs(*tags):
    return np.random.RandomState(inputs.seed_for("random-shapes", *tags) % (2 ** 32))


def _length(rs, hi):
    """A length in [0, hi]: mostly log-uniform, sometimes 0 or right at a power of two (tile edges)."""
    p = rs.rand()
    if p < 0.12:
        return 0
    if p < 0.30:
        e = 2 ** rs.randint(0, int(np.log2(max(hi, 2))) + 1)
        return int(min(hi, max(0, e + rs.randint(-1, 2))))
    return int(np.exp(rs.uniform(0.0, np.log(hi + 1))) - 1 + 0.5)


@pytest.mark.parametrize("case", range(24))
def test_select_random_ragged_batches(dodo, oracle, case):
    rs = _rs("select", case)
    B = int(rs.choice([1, 2, 7, 64, 65, 130]))
    hi = int(rs.choice([40, 600, 5000, 40000])) if B <= 7 else int(rs.choice([40, 600, 3000]))
    lens = [_length(rs, hi) for _ in range(B)]
    ks = []
    for n in lens:
        mode = rs.randint(0, 4)
        ks.append(0 if n == 0 else [oracle.num_nuggets(n, int(rs.choice([1, 2, 5, 10, 20]))), n, 1,
                                    int(rs.randint(0, n + 1))][mode])
    kind = inputs.STRESS_KINDS[rs.randint(0, len(inputs.STRESS_KINDS))]
    flags = int(rs.randint(0, 2))
    seq_off, nug_off = inputs.offsets(lens), inputs.offsets(ks)
    s = inputs.stress_scores(kind, max(int(seq_off[-1]), 1), "random-shapes", case)[:int(seq_off[-1])]
    if len(s) == 0:
        s = np.zeros(1, np.float32)
    got = _select_gpu(dodo, s, seq_off, nug_off, flags)
    assert np.array_equal(got, oracle.select_ragged(s, seq_off, nug_off, flags)), (case, kind, flags)


@pytest.mark.parametrize("case", range(16))
def test_fused_score_select_gather_random(dodo, oracle, case):
    # score + select in one launch, then gather appended behind rows already in the cache
    rs = _rs("compress", case)
    dtype = [torch.bfloat16, torch.float32][rs.randint(0, 2)]
    d = int(rs.choice([64, 256, 1000, 4096]))
    H, dh = [(1, 64), (2, 64), (4, 128), (3, 128)][rs.randint(0, 4)]
    B = int(rs.choice([1, 3, 9, 66]))
    hi = 5000 if B <= 3 else (900 if B <= 9 else 120)
    lens = [_length(rs, hi) for _ in range(B)]
    r = int(rs.choice([1, 3, 10, 20]))
    ks = [oracle.num_nuggets(n, r) for n in lens]
    flags = int(rs.randint(0, 2))
    seq_off, nug_off = inputs.offsets(lens), inputs.offsets(ks)
    N, Kt = int(seq_off[-1]), int(nug_off[-1])
    X = inputs.randn((max(N, 1), d), "rs-compress", case, "X", dtype=dtype)
    w = inputs.randn((d,), "rs-compress", case, "w", std=d ** -0.5, dtype=dtype)
    K = inputs.randn((max(N, 1), H, dh), "rs-compress", case, "K", dtype=dtype)
    V = inputs.randn((max(N, 1), H, dh), "rs-compress", case, "V", dtype=dtype)
    scores = torch.full((max(N, 1),), float("nan"), device="cuda")
    idx = torch.full((max(Kt, 1),), -3, dtype=torch.int32, device="cuda")
    bias = float(rs.randn())
    dodo.score_select(dev(X), dev(w), bias, seq_off, nug_off, flags, scores, idx)
    torch.cuda.synchronize()
    s_gpu = scores.cpu().numpy()[:N]
    s64 = oracle.score(inputs.to_numpy(X)[:N], inputs.to_numpy(w), bias)
    band = 1e-5 * (1.0 + abs(bias) + X[:N].double().abs().numpy() @ w.double().abs().numpy())
    assert np.all(np.abs(s_gpu.astype(np.float64) - s64) <= band)
    idx_o = oracle.select_ragged(s_gpu if N else np.zeros(1, np.float32), seq_off, nug_off, flags)
    assert np.array_equal(idx.cpu().numpy()[:Kt], idx_o)

    used = [int(rs.randint(0, 4)) for _ in range(B)]               # rows already in each cache region
    cache_off = inputs.offsets([u + k + int(rs.randint(0, 3)) for u, k in zip(used, ks)])
    cap = max(int(cache_off[-1]), 1)
    cK0 = inputs.randn((cap, H, dh), "rs-compress", case, "cK", dtype=dtype)
    cV0 = inputs.randn((cap, H, dh), "rs-compress", case, "cV", dtype=dtype)
    cpos0 = np.full(cap, -9, np.int32)
    cKd, cVd, cpd = dev(cK0), dev(cV0), dev(cpos0)
    len_g = np.array(used, np.int32)
    pos_base = rs.randint(0, 1000, size=B).astype(np.int32)
    dodo.gather_kv(dev(K), dev(V), seq_off, idx, nug_off, pos_base, cKd, cVd, cpd, cache_off, len_g)
    torch.cuda.synchronize()
    cKo, cVo, cpo = inputs.to_numpy(cK0).copy(), inputs.to_numpy(cV0).copy(), cpos0.copy()
    len_o = oracle.gather_ragged(inputs.to_numpy(K), inputs.to_numpy(V), seq_off, idx_o, nug_off, pos_base,
                                 cKo, cVo, cpo, cache_off, used)
    assert len_g.tolist() == len_o
    assert np.array_equal(inputs.to_numpy(cKd), cKo) and np.array_equal(inputs.to_numpy(cVd), cVo)
    assert np.array_equal(cpd.cpu().numpy(), cpo)


@pytest.mark.parametrize("case", range(36))
def test_attend_random_ragged_batches(dodo, oracle, case):
    from paper_2310_02409_b200 import api
    rs = _rs("attend", case)
    family = ["decode", "small_block", "dense", "mixed"][case % 4]
    dtype = torch.bfloat16 if family == "dense" or rs.rand() < 0.6 else torch.float32
    dh = 128 if family == "dense" or rs.rand() < 0.6 else 64
    H = int(rs.choice([1, 2, 3, 5, 8]))
    B = int(rs.choice([1, 2, 5, 9])) if family != "decode" else int(rs.choice([1, 3, 8, 70]))
    tqs, clens, llens, qp0 = [], [], [], []
    for b in range(B):
        if family == "decode":
            tq = int(rs.rand() < 0.9)
        elif family == "small_block":
            tq = int(rs.randint(0, 9))
        elif family == "dense":
            tq = int(rs.choice([0, 32, 33, 100, 128, 129, 200, 257]))
        else:
            tq = int(rs.choice([0, 1, 4, 40, 130]))
        c = _length(rs, 700 if B <= 9 else 150)
        extra = _length(rs, 300 if B <= 9 else 60)
        # usually the queries are the last tq local tokens; sometimes the block sits elsewhere, so that
        # some queries see only part of the nuggets, or nothing at all
        llens.append(tq + extra)
        tqs.append(tq)
        clens.append(c)
        split = 3 * c + 7
        where = rs.rand()
        if where < 0.7:
            qp0.append(split + extra)
        elif where < 0.85:
            qp0.append(int(rs.randint(0, split + 1)))          # inside the compressed region
        else:
            qp0.append(split + extra + int(rs.randint(1, 50)))   # beyond every key
    default_target = 2 * torch.cuda.get_device_properties(0).multi_processor_count
    target = int(rs.choice([default_target, default_target, 1, 64, 600, 4096]))
    balance = int(rs.choice([0, 0, 1, 2, 3]))
    dodo.set_tuning(api.TUNE_ATTEND_TARGET_BLOCKS, target)
    dodo.set_tuning(api.TUNE_DENSE_BALANCE, balance)
    try:
        eo, el = _attend_case(dodo, oracle, dtype, H, dh, tqs, clens, llens, tag=("rs-attend", case), q_pos0=qp0,
                              shuffle_pos=bool(rs.rand() < 0.3), with_lse=bool(rs.rand() < 0.7),
                              cache_slack=int(rs.randint(0, 6)))
    finally:
        dodo.set_tuning(api.TUNE_ATTEND_TARGET_BLOCKS, default_target)
        dodo.set_tuning(api.TUNE_DENSE_BALANCE, 0)
    assert eo <= ATTEND_TOL[dtype] and el <= 2e-3, (case, family, eo, el)
    assert dodo.device_status() == 0
