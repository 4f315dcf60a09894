"""GPU parity: every C-ABI entry point against the fp64 CPU oracle on the same seeded inputs.

Bit-exact for indices and cache contents; attention within 2e-2 (bf16) / 1e-4 (fp32) max-abs of the
fp64 oracle; scores within the fp32-accumulation band 1e-5 * (1 + sum |x_c w_c|).
"""
import math

import numpy as np
import pytest
import torch

import parity_log
from paper_2310_02409_b200 import inputs

pytestmark = pytest.mark.gpu

ATTEND_TOL = {torch.bfloat16: 2e-2, torch.float32: 1e-4}


def dev(x):
    return x.cuda() if isinstance(x, torch.Tensor) else torch.from_numpy(np.ascontiguousarray(x)).cuda()


# --------------------------------------------------------------------------------------- select

def _select_gpu(dodo, scores_np, seq_off, nug_off, flags=0):
    s = dev(scores_np.astype(np.float32))
    idx = torch.full((max(int(nug_off[-1]), 1),), -7, dtype=torch.int32, device="cuda")
    dodo.select(s, seq_off, nug_off, flags, idx)
    torch.cuda.synchronize()
    return idx.cpu().numpy()[:int(nug_off[-1])]


@pytest.mark.parametrize("kind", inputs.STRESS_KINDS)
@pytest.mark.parametrize("n", [1, 2, 31, 33, 1000, 4096, 4097, 20000, 40000])
def test_select_bit_exact_single_sequence(dodo, oracle, kind, n):
    s = inputs.stress_scores(kind, n, "gpu-select")
    for r in (1, 3, 10, 20):
        k = oracle.num_nuggets(n, r)
        for flags in (0, oracle.FORCE_LAST):
            seq_off, nug_off = inputs.offsets([n]), inputs.offsets([k])
            got = _select_gpu(dodo, s, seq_off, nug_off, flags)
            assert np.array_equal(got, oracle.select(s, k, flags)), (kind, n, r, flags)


def test_select_ragged_batch_with_empty_sequences(dodo, oracle):
    lens = [0, 5, 777, 0, 4096, 1, 12345, 64]
    ks = [oracle.num_nuggets(n, 10) for n in lens]
    ks[2] = 0            # k = 0 on a non-empty sequence is allowed
    seq_off, nug_off = inputs.offsets(lens), inputs.offsets(ks)
    s = inputs.stress_scores("quantised8", int(seq_off[-1]), "ragged")
    got = _select_gpu(dodo, s, seq_off, nug_off)
    assert np.array_equal(got, oracle.select_ragged(s, seq_off, nug_off))


@pytest.mark.parametrize("flags", [0, 1])
@pytest.mark.parametrize("lens,kind", [
    ([9000, 32768, 8193, 20001, 300], "quantised8"),     # long sequences take a cluster each, the short one a block
    ([8193, 70000], "normal"),                           # slices longer than the usual key cache
    ([9000] * 40 + [10], "all_equal"),                   # more long sequences than clusters of 8 fit at once
])
def test_select_long_sequences_in_clusters(dodo, oracle, lens, kind, flags):
    ks = [oracle.num_nuggets(n, 10) for n in lens]
    ks[0] = lens[0]      # keep everything
    ks[-1] = 1
    seq_off, nug_off = inputs.offsets(lens), inputs.offsets(ks)
    s = inputs.stress_scores(kind, int(seq_off[-1]), "longsel", len(lens))
    got = _select_gpu(dodo, s, seq_off, nug_off, flags)
    assert np.array_equal(got, oracle.select_ragged(s, seq_off, nug_off, flags))


def test_select_more_sequences_than_one_launch_group(dodo, oracle):
    lens = inputs.loguniform_lengths(150, 1, 600, "many")
    ks = [oracle.num_nuggets(n, 7) for n in lens]
    seq_off, nug_off = inputs.offsets(lens), inputs.offsets(ks)
    s = inputs.stress_scores("normal", int(seq_off[-1]), "many")
    got = _select_gpu(dodo, s, seq_off, nug_off, oracle.FORCE_LAST)
    assert np.array_equal(got, oracle.select_ragged(s, seq_off, nug_off, oracle.FORCE_LAST))


def test_select_rejects_bad_arguments(dodo):
    from paper_2310_02409_b200 import api
    s = torch.zeros(10, device="cuda")
    idx = torch.zeros(20, dtype=torch.int32, device="cuda")
    with pytest.raises(api.DodoError) as e:
        dodo.select(s, [0, 10], [0, 11], 0, idx)          # k > n
    assert e.value.status == api.ERR_INVALID_ARG
    with pytest.raises(api.DodoError):
        dodo.select(s, [1, 10], [0, 1], 0, idx)           # offsets must start at 0
    with pytest.raises(api.DodoError):
        dodo.select(s, [0, 10], [0, 1], 8, idx)           # unknown flag


# --------------------------------------------------------------------------------------- score

def _score_band(X, w):
    """fp32-accumulation tolerance band per row: 1e-5 * (1 + sum_c |x_c w_c|)."""
    return 1e-5 * (1.0 + (X.double().abs() @ w.double().abs()).numpy())


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("d", [256, 4096, 5120, 72])
def test_score_matches_oracle(dodo, oracle, dtype, d):
    lens = [37, 0, 130, 1]
    seq_off = inputs.offsets(lens)
    N = int(seq_off[-1])
    X = inputs.randn((N, d), "score", d, "X", dtype=dtype)
    w = inputs.randn((d,), "score", d, "w", std=d ** -0.5, dtype=dtype)
    out = torch.full((N,), float("nan"), device="cuda")
    dodo.score(dev(X), dev(w), 0.125, seq_off, out)
    torch.cuda.synchronize()
    ref = oracle.score(inputs.to_numpy(X), inputs.to_numpy(w), 0.125)
    assert np.all(np.abs(out.cpu().numpy().astype(np.float64) - ref) <= _score_band(X, w))


def test_score_exact_on_power_of_two_inputs(dodo, oracle):
    # sums of small powers of two are exact in fp32 in any order: the result must equal fp64
    rs = np.random.RandomState(5)
    N, d = 70, 512
    X = torch.from_numpy((2.0 ** rs.randint(-3, 4, size=(N, d)) * rs.choice([-1, 1], size=(N, d))).astype(np.float32))
    w = torch.from_numpy((2.0 ** rs.randint(-3, 4, size=d)).astype(np.float32))
    for dtype in (torch.float32, torch.bfloat16):
        out = torch.empty(N, device="cuda")
        dodo.score(dev(X.to(dtype)), dev(w.to(dtype)), 0.0, [0, N], out)
        ref = oracle.score(inputs.to_numpy(X.to(dtype)), inputs.to_numpy(w.to(dtype)))
        assert np.array_equal(out.cpu().numpy().astype(np.float64), ref)


@pytest.mark.parametrize("dtype,d,lens", [
    (torch.float32, 256, [512]),
    (torch.bfloat16, 4096, [2048, 100, 0, 33, 1000]),
    (torch.bfloat16, 1024, inputs.loguniform_lengths(70, 1, 3000, "ss")),
])
@pytest.mark.parametrize("flags", [0, 1])
def test_fused_score_select(dodo, oracle, dtype, d, lens, flags):
    seq_off = inputs.offsets(lens)
    ks = [oracle.num_nuggets(n, 10) for n in lens]
    nug_off = inputs.offsets(ks)
    N = int(seq_off[-1])
    X = inputs.randn((N, d), "fused", d, "X", dtype=dtype)
    w = inputs.randn((d,), "fused", d, "w", std=d ** -0.5, dtype=dtype)
    Xd, wd = dev(X), dev(w)
    s_fused = torch.full((N,), float("nan"), device="cuda")
    idx = torch.full((int(nug_off[-1]),), -1, dtype=torch.int32, device="cuda")
    dodo.score_select(Xd, wd, 0.0, seq_off, nug_off, flags, s_fused, idx)
    s_plain = torch.empty(N, device="cuda")
    dodo.score(Xd, wd, 0.0, seq_off, s_plain)
    torch.cuda.synchronize()
    # the hand-over buffer holds exactly what dodo_score writes
    assert torch.equal(s_fused, s_plain)
    # scores -> indices is bit-exact: the oracle's stable-sort TopK on the very same fp32 scores
    s_np = s_fused.cpu().numpy()
    assert np.array_equal(idx.cpu().numpy(), oracle.select_ragged(s_np, seq_off, nug_off, flags))
    # end to end against the all-fp64 pipeline: any disagreement must sit inside the score band
    s64 = oracle.score(inputs.to_numpy(X), inputs.to_numpy(w))
    idx64 = oracle.select_ragged(s64, seq_off, nug_off, flags)
    band = _score_band(X, w)
    got = idx.cpu().numpy()
    for b in range(len(lens)):
        a = set(got[nug_off[b]:nug_off[b + 1]].tolist())
        c = set(idx64[nug_off[b]:nug_off[b + 1]].tolist())
        if a != c:
            sb = s64[seq_off[b]:seq_off[b + 1]]
            kth = np.sort(sb)[::-1][ks[b] - 1]
            for i in a ^ c:
                assert abs(sb[i] - kth) <= 2 * band[seq_off[b] + i]


# --------------------------------------------------------------------------------------- gather

@pytest.mark.parametrize("dtype,H,dh", [(torch.bfloat16, 32, 128), (torch.float32, 4, 64), (torch.bfloat16, 3, 8)])
def test_gather_bit_exact_and_append(dodo, oracle, dtype, H, dh):
    lens = [100, 0, 37, 260]
    seq_off = inputs.offsets(lens)
    N = int(seq_off[-1])
    K = inputs.randn((N, H, dh), "gather", "K", dtype=dtype)
    V = inputs.randn((N, H, dh), "gather", "V", dtype=dtype)
    caps = [40, 3, 20, 95]
    cache_off = inputs.offsets(caps)
    cap = int(cache_off[-1])
    pad = 4     # canary rows after the last region
    cK = torch.full((cap + pad, H, dh), 7.0, dtype=dtype)
    cV = torch.full((cap + pad, H, dh), 9.0, dtype=dtype)
    cpos = torch.full((cap + pad,), -5, dtype=torch.int32)
    cK_d, cV_d, cpos_d = dev(cK), dev(cV), dev(cpos)
    cK_o, cV_o, cpos_o = inputs.to_numpy(cK).copy(), inputs.to_numpy(cV).copy(), cpos.numpy().copy()
    Kd, Vd = dev(K), dev(V)
    Kn, Vn = inputs.to_numpy(K), inputs.to_numpy(V)
    len_g = np.zeros(4, np.int32)
    len_o = [0, 0, 0, 0]
    for rnd, r in enumerate((10, 4)):     # two appends into the same regions
        ks = [oracle.num_nuggets(n, r) for n in lens]
        nug_off = inputs.offsets(ks)
        s = inputs.stress_scores("normal", N, "gather", rnd)
        idx = oracle.select_ragged(s, seq_off, nug_off)
        pos_base = np.array([1000 * rnd + 10 * b for b in range(4)], np.int32)
        dodo.gather_kv(Kd, Vd, seq_off, dev(idx), nug_off, pos_base, cK_d, cV_d, cpos_d, cache_off, len_g)
        len_o = oracle.gather_ragged(Kn, Vn, seq_off, idx, nug_off, pos_base, cK_o, cV_o, cpos_o, cache_off, len_o)
        torch.cuda.synchronize()
        assert len_g.tolist() == len_o
        assert np.array_equal(inputs.to_numpy(cK_d), cK_o)
        assert np.array_equal(inputs.to_numpy(cV_d), cV_o)
        assert np.array_equal(cpos_d.cpu().numpy(), cpos_o)
    # a third append overflows sequence 0's region: refused before any launch, nothing changes
    from paper_2310_02409_b200 import api
    ks = [30, 0, 0, 0]
    nug_off = inputs.offsets(ks)
    with pytest.raises(api.DodoError) as e:
        dodo.gather_kv(Kd, Vd, seq_off, dev(np.arange(30, dtype=np.int32)), nug_off, np.zeros(4, np.int32),
                       cK_d, cV_d, cpos_d, cache_off, len_g)
    assert e.value.status == api.ERR_CAPACITY and len_g.tolist() == len_o
    assert np.array_equal(inputs.to_numpy(cK_d), cK_o)


@pytest.mark.parametrize("dtype,H,dh,L", [(torch.bfloat16, 32, 128, 3), (torch.float32, 4, 64, 1), (torch.bfloat16, 3, 8, 70)])
def test_gather_layers_equals_one_gather_per_layer(dodo, oracle, dtype, H, dh, L):
    # one shared selection (Sec. 2.1), L layers in one call (70 layers: more than one launch), two appends;
    # every layer's cache must equal the oracle's gather of that layer, the positions are written once
    lens = [100, 0, 37, 260]
    B, seq_off = len(lens), inputs.offsets(lens)
    N = int(seq_off[-1])
    caps = [40, 3, 20, 95]
    cache_off = inputs.offsets(caps)
    cap, pad = int(cache_off[-1]), 4
    Ks = [inputs.randn((N, H, dh), "gatherL", l, "K", dtype=dtype) for l in range(L)]
    Vs = [inputs.randn((N, H, dh), "gatherL", l, "V", dtype=dtype) for l in range(L)]
    cKs = [torch.full((cap + pad, H, dh), 7.0 + l, dtype=dtype) for l in range(L)]
    cVs = [torch.full((cap + pad, H, dh), -9.0 - l, dtype=dtype) for l in range(L)]
    cpos = torch.full((cap + pad,), -5, dtype=torch.int32)
    Kd, Vd, cKd, cVd, cpos_d = [dev(t) for t in Ks], [dev(t) for t in Vs], [dev(t) for t in cKs], [dev(t) for t in cVs], dev(cpos)
    cKo = [inputs.to_numpy(t).copy() for t in cKs]
    cVo = [inputs.to_numpy(t).copy() for t in cVs]
    cpos_o = [cpos.numpy().copy() for _ in range(L)]
    len_g, len_o = np.zeros(B, np.int32), [[0] * B for _ in range(L)]
    for rnd, r in enumerate((10, 4)):
        ks = [oracle.num_nuggets(n, r) for n in lens]
        nug_off = inputs.offsets(ks)
        idx = oracle.select_ragged(inputs.stress_scores("normal", N, "gatherL", rnd), seq_off, nug_off)
        pos_base = np.array([1000 * rnd + 10 * b for b in range(B)], np.int32)
        dodo.gather_kv_layers(Kd, Vd, seq_off, dev(idx), nug_off, pos_base, cKd, cVd, cpos_d, cache_off, len_g)
        torch.cuda.synchronize()
        for l in range(L):
            len_o[l] = oracle.gather_ragged(inputs.to_numpy(Ks[l]), inputs.to_numpy(Vs[l]), seq_off, idx, nug_off, pos_base,
                                            cKo[l], cVo[l], cpos_o[l], cache_off, len_o[l])
            assert len_g.tolist() == len_o[l]
            assert np.array_equal(inputs.to_numpy(cKd[l]), cKo[l]) and np.array_equal(inputs.to_numpy(cVd[l]), cVo[l])
            assert np.array_equal(cpos_d.cpu().numpy(), cpos_o[l])
    # overflow: refused before any launch; mismatched layer lists and a missing layer pointer are refused too
    from paper_2310_02409_b200 import api
    nug_off = inputs.offsets([30, 0, 0, 0])
    before = len_g.copy()
    with pytest.raises(api.DodoError) as e:
        dodo.gather_kv_layers(Kd, Vd, seq_off, dev(np.arange(30, dtype=np.int32)), nug_off, np.zeros(B, np.int32),
                              cKd, cVd, cpos_d, cache_off, len_g)
    assert e.value.status == api.ERR_CAPACITY and np.array_equal(len_g, before)
    assert np.array_equal(inputs.to_numpy(cKd[0]), cKo[0])
    with pytest.raises(ValueError):
        dodo.gather_kv_layers(Kd, Vd[:-1] if L > 1 else [], seq_off, dev(np.arange(30, dtype=np.int32)), nug_off,
                              np.zeros(B, np.int32), cKd, cVd, cpos_d, cache_off, len_g)


def test_gather_reports_an_index_outside_its_sequence(libdodo):
    # an index that is not a position of its sequence is not followed: that row of the cache and its position
    # stay as they were, every other row is copied, and the device status word says so.  The bad values still
    # point inside the K/V allocation (sequence 0's n_0 is sequence 1's first token), so no read could leave it
    # even if the check were not there.  Own context: the shared one must end the session with a clean status.
    from paper_2310_02409_b200 import api
    ctx = api.Dodo(0)
    try:
        lens, H, dh = [40, 50], 2, 64
        seq_off = inputs.offsets(lens)
        K = inputs.randn((90, H, dh), "badidx", "K", dtype=torch.bfloat16)
        V = inputs.randn((90, H, dh), "badidx", "V", dtype=torch.bfloat16)
        idx = np.array([3, 40, 7, -1, 5, 49], np.int32)          # 40 = n_0 and -1 are outside sequence 0
        nug_off = inputs.offsets([4, 2])
        cK = torch.full((6, H, dh), 7.0, dtype=torch.bfloat16, device="cuda")
        cV = torch.full((6, H, dh), 9.0, dtype=torch.bfloat16, device="cuda")
        cpos = torch.full((6,), -5, dtype=torch.int32, device="cuda")
        clen = np.zeros(2, np.int32)
        ctx.gather_kv(dev(K), dev(V), seq_off, dev(idx), nug_off, [100, 200], cK, cV, cpos, nug_off, clen)
        torch.cuda.synchronize()
        assert ctx.device_status() == api.DEV_BAD_INDEX
        want_K = torch.full((6, H, dh), 7.0, dtype=torch.bfloat16)
        want_V = torch.full((6, H, dh), 9.0, dtype=torch.bfloat16)
        want_pos = np.full(6, -5, np.int32)
        for slot, (b, i) in {0: (0, 3), 2: (0, 7), 4: (1, 5), 5: (1, 49)}.items():
            want_K[slot], want_V[slot] = K[seq_off[b] + i], V[seq_off[b] + i]
            want_pos[slot] = (100, 200)[b] + i
        assert torch.equal(cK.cpu(), want_K) and torch.equal(cV.cpu(), want_V)
        assert np.array_equal(cpos.cpu().numpy(), want_pos)
        ctx.reset()
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        # the multi-layer form checks the same way
        ctx.gather_kv_layers([dev(K)], [dev(V)], seq_off, dev(idx), nug_off, [100, 200], [cK], [cV], cpos, nug_off,
                             np.zeros(2, np.int32))
        torch.cuda.synchronize()
        assert ctx.device_status() == api.DEV_BAD_INDEX
        ctx.reset()
    finally:
        ctx.close()


def test_results_are_reproducible_bit_for_bit(dodo, oracle):
    # the same call twice gives the same bits: select and gather (integer work), and the attend paths whose
    # merge order could depend on block timing if it were written carelessly -- chunks merged in a cluster,
    # chunks merged by whichever block draws the last ticket, cut units of the tensor-core kernel
    from paper_2310_02409_b200 import api
    lens = [9000, 300, 20001, 0, 4096]
    ks = [oracle.num_nuggets(n, 10) for n in lens]
    seq_off, nug_off = inputs.offsets(lens), inputs.offsets(ks)
    s = dev(inputs.stress_scores("quantised8", int(seq_off[-1]), "twice"))
    idx = [torch.full((int(nug_off[-1]),), -1, dtype=torch.int32, device="cuda") for _ in range(2)]
    for t in idx:
        dodo.select(s, seq_off, nug_off, 0, t)
    assert torch.equal(idx[0], idx[1])
    H, dh = 4, 128
    K = dev(inputs.randn((int(seq_off[-1]), H, dh), "twice", "K", dtype=torch.bfloat16))
    V = dev(inputs.randn((int(seq_off[-1]), H, dh), "twice", "V", dtype=torch.bfloat16))
    caches = []
    for _ in range(2):
        cK = torch.zeros((int(nug_off[-1]), H, dh), dtype=torch.bfloat16, device="cuda")
        cV, cpos = torch.zeros_like(cK), torch.zeros(int(nug_off[-1]), dtype=torch.int32, device="cuda")
        dodo.gather_kv(K, V, seq_off, idx[0], nug_off, np.zeros(5, np.int32), cK, cV, cpos, nug_off, np.zeros(5, np.int32))
        caches.append((cK, cV, cpos))
    assert all(torch.equal(a, b) for a, b in zip(*caches))
    cK, cV, cpos = caches[0]
    ws = torch.empty(dodo.attend_workspace_bytes(dh), dtype=torch.uint8, device="cuda")
    clen = np.asarray(ks, np.int32)

    def attend(Q, q_off, q_pos0):
        outs = []
        for _ in range(2):
            O = torch.full_like(Q, float("nan"))
            lse = torch.full(Q.shape[:2], float("nan"), device="cuda")
            dodo.attend(Q, q_off, q_pos0, dh ** -0.5, cK, cV, cpos, nug_off, clen, None, None, None, None, None, O, lse, ws)
            outs.append((O, lse))
        torch.cuda.synchronize()
        assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])

    big = np.asarray([10 ** 6] * 5, np.int32)
    Q1 = dev(inputs.randn((4, H, dh), "twice", "Q1", dtype=torch.bfloat16))
    attend(Q1, np.array([0, 1, 2, 3, 3, 4], np.int32), big)                     # ragged: chunks meet through tickets
    dodo.set_tuning(api.TUNE_DENSE_BALANCE, 1)
    try:
        Qb = dev(inputs.randn((5 * 130, H, dh), "twice", "Qb", dtype=torch.bfloat16))
        attend(Qb, np.arange(6, dtype=np.int32) * 130, big)                     # tensor-core kernel, cut units
    finally:
        dodo.set_tuning(api.TUNE_DENSE_BALANCE, 0)
    # equal sequences: the chunks of a head form one cluster
    cK2 = dev(inputs.randn((1400, H, dh), "twice", "cK2", dtype=torch.bfloat16))
    cV2 = dev(inputs.randn((1400, H, dh), "twice", "cV2", dtype=torch.bfloat16))
    cpos2 = torch.arange(1400, dtype=torch.int32, device="cuda")
    Q2 = dev(inputs.randn((2, H, dh), "twice", "Q2", dtype=torch.bfloat16))
    outs = []
    for _ in range(2):
        O = torch.full_like(Q2, float("nan"))
        dodo.attend(Q2, [0, 1, 2], [5000, 5000], dh ** -0.5, cK2, cV2, cpos2, [0, 700, 1400], [700, 700], None, None, None,
                    None, None, O, None, None)
        outs.append(O)
    torch.cuda.synchronize()
    assert torch.equal(outs[0], outs[1]) and not torch.isnan(outs[0].float()).any()


# --------------------------------------------------------------------------------------- attend

def _attend_case(dodo, oracle, dtype, H, dh, tqs, clens, llens, *, tag, scale=None, q_pos0=None,
                 cache_slack=5, with_lse=True, shuffle_pos=False, workspace=True):
    """Build a ragged batch, run dodo_attend and the oracle, return max-abs errors (O, lse)."""
    B = len(tqs)
    scale = scale if scale is not None else dh ** -0.5
    q_off = inputs.offsets(tqs)
    cache_off = inputs.offsets([c + cache_slack for c in clens])
    loc_off = inputs.offsets([l + 3 for l in llens])
    T, C, Lr = int(q_off[-1]), int(cache_off[-1]), int(loc_off[-1])
    Q = inputs.randn((max(T, 1), H, dh), tag, "Q", dtype=dtype)
    cK = inputs.randn((max(C, 1), H, dh), tag, "cK", dtype=dtype)
    cV = inputs.randn((max(C, 1), H, dh), tag, "cV", dtype=dtype)
    lK = inputs.randn((max(Lr, 1), H, dh), tag, "lK", dtype=dtype)
    lV = inputs.randn((max(Lr, 1), H, dh), tag, "lV", dtype=dtype)
    # nugget positions: ascending picks from the compressed region [0, split); local follows
    rs = np.random.RandomState(inputs.seed_for(tag) % 2 ** 32)
    cpos = np.full(max(C, 1), 2 ** 30, np.int32)    # slack rows carry junk positions
    loc_pos0 = np.zeros(B, np.int32)
    qp0 = np.zeros(B, np.int32)
    for b in range(B):
        split = 3 * clens[b] + 7
        p = np.sort(rs.choice(split, clens[b], replace=False)).astype(np.int32)
        if shuffle_pos:
            rs.shuffle(p)
        cpos[cache_off[b]:cache_off[b] + clens[b]] = p
        loc_pos0[b] = split
        # default: the queries are the last tq local tokens (they see themselves causally)
        qp0[b] = split + llens[b] - tqs[b] if q_pos0 is None else q_pos0[b]
    O = torch.full((max(T, 1), H, dh), float("nan"), dtype=dtype, device="cuda")
    lse = torch.full((max(T, 1), H), float("nan"), device="cuda") if with_lse else None
    ws = torch.empty(dodo.attend_workspace_bytes(dh), dtype=torch.uint8, device="cuda") if workspace else None
    dodo.attend(dev(Q), q_off, qp0, scale, dev(cK), dev(cV), dev(cpos), cache_off, np.array(clens, np.int32),
                dev(lK), dev(lV), loc_off[:-1], np.array(llens, np.int32), loc_pos0, O, lse, ws)
    torch.cuda.synchronize()
    Oo, lo = oracle.attend_ragged(inputs.to_numpy(Q), q_off, qp0, scale, inputs.to_numpy(cK), inputs.to_numpy(cV),
                                  cpos, cache_off, clens, inputs.to_numpy(lK), inputs.to_numpy(lV),
                                  loc_off[:-1], llens, loc_pos0)
    if T == 0:
        return 0.0, 0.0
    got = O.float().cpu().numpy().astype(np.float64)[:T]
    err_o = float(np.max(np.abs(got - Oo)))
    err_l = 0.0
    if with_lse:
        gl = lse.cpu().numpy().astype(np.float64)[:T]
        fin = np.isfinite(lo)
        assert np.array_equal(np.isneginf(gl), np.isneginf(lo))
        err_l = float(np.max(np.abs(gl[fin] - lo[fin]))) if fin.any() else 0.0
    # which kernel family served the call (the library's shape rule, for the error log's key only)
    kind = "fp32" if dtype == torch.float32 else "dense" if (dh == 128 and max(tqs) >= 32) else \
        "decode" if max(tqs) == 1 else "block"
    err_r = parity_log.rel_error(got, Oo)
    parity_log.LOG.add(f"attend case {tag}", **{kind + "_O": err_o, kind + "_lse": err_l, kind + "_rel": err_r})
    # where the kernels sit, beside the stated tolerances the callers assert
    assert err_l <= parity_log.LSE_CEILING and (dtype == torch.float32 or err_r <= parity_log.REL_CEILING), (tag, err_l, err_r)
    return err_o, err_l


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("dh", [64, 128])
def test_attend_decode_ragged(dodo, oracle, dtype, dh):
    # one query token per sequence; nugget counts span several tiles and ragged tails; one sequence
    # has no nuggets, one no local tokens, one is empty altogether
    tqs = [1, 1, 1, 1, 1, 0, 1]
    clens = [205, 13, 0, 700, 64, 10, 1]
    llens = [64, 1, 40, 0, 130, 5, 1]
    eo, el = _attend_case(dodo, oracle, dtype, 8, dh, tqs, clens, llens, tag=("dec", str(dtype), dh))
    assert eo <= ATTEND_TOL[dtype] and el <= 1e-3


@pytest.mark.parametrize("target", [1, 64, 600, 4096])
def test_attend_split_invariance(dodo, oracle, target):
    # any chunking of the keys (none, a few, one granule per block) gives the same result within tolerance
    from paper_2310_02409_b200 import api
    dodo.set_tuning(api.TUNE_ATTEND_TARGET_BLOCKS, target)
    try:
        eo, el = _attend_case(dodo, oracle, torch.bfloat16, 4, 128, [1, 1, 1], [1000, 333, 64], [64, 0, 200],
                              tag=("split", target))
        assert eo <= 2e-2 and el <= 1e-3
        eo, el = _attend_case(dodo, oracle, torch.float32, 2, 64, [3, 1], [500, 90], [70, 9],
                              tag=("split32", target))
        assert eo <= 1e-4 and el <= 1e-4
    finally:
        dodo.set_tuning(api.TUNE_ATTEND_TARGET_BLOCKS, 2 * torch.cuda.get_device_properties(0).multi_processor_count)


@pytest.mark.parametrize("dtype,H,dh,tqs,clens,llens,kw", [
    # one sequence, 40 heads: 7 chunks by the split rule, 6 as clusters that are all resident at once
    (torch.bfloat16, 40, 128, [1], [1639], [5], {}),
    # equal sequences, few heads: as many chunks as key granules; no workspace is needed for this merge
    (torch.bfloat16, 8, 128, [1, 1], [700, 700], [64, 64], {"workspace": False}),
    # query tiles of 2 and of 4 tokens, a sequence without queries between the others, no lse
    (torch.float32, 4, 64, [2, 0, 2], [900, 900, 900], [40, 40, 40], {"with_lse": False}),
    (torch.float32, 2, 128, [4, 4], [1200, 1200], [4, 4], {}),
    # queries early in the compressed region, nuggets in arbitrary order: whole chunks see nothing
    (torch.bfloat16, 4, 64, [1, 1], [1500, 1500], [0, 0], {"q_pos0": [40, 2000], "shuffle_pos": True}),
    # no key at all is visible: O = 0, lse = -inf out of the merge
    (torch.float32, 4, 64, [1], [600], [0], {"q_pos0": [-1]}),
])
def test_attend_split_merged_in_cluster(dodo, oracle, dtype, H, dh, tqs, clens, llens, kw):
    # batches in which every sequence is cut into the same number of chunks: the chunks of a (query tile, head)
    # run as one thread-block cluster and merge in shared memory
    eo, el = _attend_case(dodo, oracle, dtype, H, dh, tqs, clens, llens,
                          tag=("cluster", str(dtype), H, dh, tuple(tqs), tuple(clens)), **kw)
    assert eo <= ATTEND_TOL[dtype] and el <= 1e-3


@pytest.mark.parametrize("dtype,dh", [(torch.float32, 64), (torch.bfloat16, 128), (torch.float32, 128), (torch.bfloat16, 64)])
@pytest.mark.parametrize("tq", [2, 3, 4, 16, 37])
def test_attend_query_block_causal(dodo, oracle, dtype, dh, tq):
    # compressor mode (Eq. 13): a block of queries sees all nuggets and, causally, itself
    eo, el = _attend_case(dodo, oracle, dtype, 4, dh, [tq, tq + 1], [52, 130], [tq, tq + 9],
                          tag=("blk", str(dtype), dh, tq))
    assert eo <= ATTEND_TOL[dtype] and el <= 1e-3


def test_attend_masks_by_position(dodo, oracle):
    # queries in the middle of the compressed region: nuggets at later positions are invisible;
    # the first query sees nothing at all (O = 0, lse = -inf); cache order is arbitrary
    eo, el = _attend_case(dodo, oracle, torch.float32, 2, 64, [40, 5], [90, 30], [0, 12],
                          tag="maskpos", q_pos0=[-1, 20], shuffle_pos=True)
    assert eo <= 1e-4 and el <= 1e-4


def test_attend_without_lse_and_many_sequences(dodo, oracle):
    lens = inputs.loguniform_lengths(130, 1, 400, "manyseq")
    eo, _ = _attend_case(dodo, oracle, torch.bfloat16, 2, 128, [1] * 130, lens, [l % 70 for l in lens],
                         tag="manyseq", with_lse=False)
    assert eo <= 2e-2


def test_attend_r1_equals_full_attention(dodo, oracle):
    # r = 1 keeps every token as a nugget: nugget attention must equal full causal attention (Eq. 3)
    n, m, H, dh = 300, 8, 4, 64
    q = inputs.randn((n + m, H, dh), "r1gpu", "q")
    k = inputs.randn((n + m, H, dh), "r1gpu", "k")
    v = inputs.randn((n + m, H, dh), "r1gpu", "v")
    scale = dh ** -0.5
    qh, kh, vh = (x.double().permute(1, 0, 2).unsqueeze(0) for x in (q, k, v))
    full = torch.nn.functional.scaled_dot_product_attention(qh, kh, vh, is_causal=True, scale=scale)[0].permute(1, 0, 2)
    seq_off, nug_off = inputs.offsets([n]), inputs.offsets([dodo.num_nuggets(n, 1)])
    s = dev(inputs.stress_scores("normal", n, "r1gpu"))
    idx = torch.empty(n, dtype=torch.int32, device="cuda")
    dodo.select(s, seq_off, nug_off, 0, idx)
    cK = torch.zeros((n, H, dh), device="cuda")
    cV = torch.zeros((n, H, dh), device="cuda")
    cpos = torch.zeros(n, dtype=torch.int32, device="cuda")
    clen = np.zeros(1, np.int32)
    dodo.gather_kv(dev(k[:n]), dev(v[:n]), seq_off, idx, nug_off, [0], cK, cV, cpos, [0, n], clen)
    O = torch.empty((m, H, dh), device="cuda")
    ws = torch.empty(dodo.attend_workspace_bytes(dh), dtype=torch.uint8, device="cuda")
    dodo.attend(dev(q[n:]), [0, m], [n], scale, cK, cV, cpos, [0, n], clen,
                dev(k[n:]), dev(v[n:]), [0], [m], [n], O, None, ws)
    torch.cuda.synchronize()
    assert float((O.cpu().double() - full[n:]).abs().max()) <= 1e-4


def test_attend_rejects_bad_arguments(dodo):
    from paper_2310_02409_b200 import api
    Q = torch.zeros((1, 2, 32), device="cuda")
    with pytest.raises(api.DodoError) as e:
        dodo.attend(Q, [0, 1], [0], 1.0, None, None, None, None, None, None, None, None, None, None, Q, None, None)
    assert e.value.status == api.ERR_UNSUPPORTED       # head size 32
    Q = torch.zeros((1, 2, 64), device="cuda")
    K = torch.zeros((10, 2, 64), device="cuda")
    with pytest.raises(api.DodoError) as e:            # cache_len beyond its region
        dodo.attend(Q, [0, 1], [0], 1.0, K, K, torch.zeros(10, dtype=torch.int32, device="cuda"), [0, 10], [11],
                    None, None, None, None, None, Q, None, None)
    assert e.value.status == api.ERR_INVALID_ARG
    with pytest.raises(api.DodoError) as e:            # split needed but no workspace
        Kb = torch.zeros((5000, 2, 64), device="cuda")
        dodo.attend(Q, [0, 1], [0], 1.0, Kb, Kb, torch.zeros(5000, dtype=torch.int32, device="cuda"), [0, 5000],
                    [5000], None, None, None, None, None, Q, None, None)
    assert e.value.status == api.ERR_CAPACITY


def test_attend_sees_rows_appended_just_before_it(dodo, oracle):
    # a gather appends to the nugget cache directly before every attend, many times over, with no host
    # synchronisation between: each attend must see the rows and positions its predecessor wrote.  (The attend
    # kernel may start while the gather drains; it reads no cache row ahead of its dependency wait unless the
    # launch before it was an attend.)  Between two appends a second attend runs, which may read ahead.
    H, dh, n, rounds, per = 8, 128, 4096, 24, 40
    B = 4
    seq_off = inputs.offsets([n] * B)
    K = inputs.randn((B * n, H, dh), "append", "K", dtype=torch.bfloat16)
    V = inputs.randn((B * n, H, dh), "append", "V", dtype=torch.bfloat16)
    Kd, Vd = dev(K), dev(V)
    cap = rounds * per
    cache_off = inputs.offsets([cap] * B)
    # stale contents that would poison the result if an attend read a row before its append landed
    cK = torch.full((B * cap, H, dh), 50.0, dtype=torch.bfloat16, device="cuda")
    cV = torch.full((B * cap, H, dh), -300.0, dtype=torch.bfloat16, device="cuda")
    cpos = torch.zeros(B * cap, dtype=torch.int32, device="cuda")
    clen = np.zeros(B, np.int32)
    rs = np.random.RandomState(3)
    order = np.stack([rs.permutation(n)[:cap] for _ in range(B)])              # tokens appended, round by round
    Q = inputs.randn((2 * rounds, B, H, dh), "append", "Q", dtype=torch.bfloat16)
    Qd = dev(Q)
    O = torch.full((2 * rounds, B, H, dh), float("nan"), dtype=torch.bfloat16, device="cuda")
    nug_off = inputs.offsets([per] * B)
    q_off, q_pos0 = np.arange(B + 1, dtype=np.int32), np.full(B, n, np.int32)
    idx_all = [dev(np.sort(order[:, r * per:(r + 1) * per], axis=1).reshape(-1).astype(np.int32)) for r in range(rounds)]
    ws = torch.empty(dodo.attend_workspace_bytes(dh), dtype=torch.uint8, device="cuda")
    for r in range(rounds):
        dodo.gather_kv(Kd, Vd, seq_off, idx_all[r], nug_off, np.zeros(B, np.int32), cK, cV, cpos, cache_off, clen)
        for rep in range(2):
            dodo.attend(Qd[2 * r + rep], q_off, q_pos0, dh ** -0.5, cK, cV, cpos, cache_off, clen, None, None, None, None,
                        None, O[2 * r + rep], None, ws)
    torch.cuda.synchronize()
    Kn, Vn = inputs.to_numpy(K), inputs.to_numpy(V)
    cKo = np.zeros((B * cap, H, dh), np.uint16); cVo = np.zeros_like(cKo); cpo = np.zeros(B * cap, np.int32)
    lens = [0] * B
    worst = 0.0
    for r in range(rounds):
        lens = oracle.gather_ragged(Kn, Vn, seq_off, idx_all[r].cpu().numpy(), nug_off, np.zeros(B, np.int32), cKo, cVo, cpo,
                                    cache_off, lens)
        for rep in range(2):
            ref = oracle.attend_ragged(inputs.to_numpy(Q[2 * r + rep]), q_off, q_pos0, dh ** -0.5, cKo, cVo, cpo, cache_off,
                                       lens, None, None, None, None, None)[0]
            worst = max(worst, float(np.max(np.abs(O[2 * r + rep].float().cpu().numpy().astype(np.float64) - ref))))
    parity_log.LOG.add("attend directly after an append, 24 rounds", decode_O=worst)
    assert worst <= 2e-2, worst
    assert np.array_equal(inputs.to_numpy(cK), cKo) and np.array_equal(cpos.cpu().numpy(), cpo)


# ------------------------------------------------------------------------- attend, tensor-core path

@pytest.mark.parametrize("tqs,clens,llens", [
    ([128], [128], [128]),                       # exactly one tile of everything
    ([256, 37, 130], [717, 52, 0], [300, 37, 200]),   # several query and key tiles, ragged tails, no nuggets
    ([64, 200], [1000, 90], [0, 0]),             # nuggets only
])
def test_attend_dense_query_blocks(dodo, oracle, tqs, clens, llens):
    # bf16, head size 128, query blocks of 32+ tokens: tcgen05 kernel (P is rounded to bf16 there)
    llens = [max(l, 0) for l in llens]
    q_pos0 = None if all(l >= t for l, t in zip(llens, tqs)) else [3 * c + 7 + l for c, l in zip(clens, llens)]
    eo, el = _attend_case(dodo, oracle, torch.bfloat16, 4, 128, tqs, clens, llens, tag=("dense", tuple(tqs)),
                          q_pos0=q_pos0)
    assert eo <= 2e-2 and el <= 1e-3


def test_attend_dense_masks_by_position(dodo, oracle):
    # queries in the middle of the compressed region, cache rows in arbitrary order: only keys at
    # positions <= the query's are visible; the earliest queries see nothing (O = 0, lse = -inf)
    eo, el = _attend_case(dodo, oracle, torch.bfloat16, 2, 128, [140, 40], [300, 64], [0, 50],
                          tag="densemask", q_pos0=[-2, 30], shuffle_pos=True)
    assert eo <= 2e-2 and el <= 1e-3


@pytest.mark.parametrize("tqs,clens,llens,q_pos0,shuffle", [
    ([256, 37, 130], [717, 52, 0], [300, 37, 200], None, False),   # units of 17, 2 and 4 key tiles cut at every tile
    ([64, 128], [0, 300], [0, 64], [5, 1000], False),             # a unit without any key sits between the others
    ([140, 190], [300, 64], [0, 50], [-2, 30], True),              # position masks, rows that see nothing; two query tiles each
    ([300], [5000], [300], None, False),                           # long list: blocks hold many tiles of one unit
    ([257, 384], [900, 0], [400, 384], None, False),               # three query tiles each, one sequence without nuggets
])
@pytest.mark.parametrize("mode", [1, 3])
def test_attend_dense_balanced_units(dodo, oracle, tqs, clens, llens, q_pos0, shuffle, mode):
    # key tiles spread evenly over the thread blocks whatever unit they belong to: units cut by a block
    # boundary are finished through partial results and a last-arriver merge; same tolerance.  Mode 1 keeps
    # the query tiles of a head in step where every sequence has the same number of them (the last case, and
    # the third), mode 3 never does.
    from paper_2310_02409_b200 import api
    dodo.set_tuning(api.TUNE_DENSE_BALANCE, mode)
    try:
        eo, el = _attend_case(dodo, oracle, torch.bfloat16, 4, 128, tqs, clens, llens, tag=("balanced", tuple(tqs)),
                              q_pos0=q_pos0, shuffle_pos=shuffle)
        eo2, el2 = _attend_case(dodo, oracle, torch.bfloat16, 4, 128, tqs, clens, llens, tag=("balanced", tuple(tqs)),
                                q_pos0=q_pos0, shuffle_pos=shuffle)     # counters were left clean
    finally:
        dodo.set_tuning(api.TUNE_DENSE_BALANCE, 0)
    assert eo <= 2e-2 and el <= 1e-3 and eo2 == eo and el2 == el
    assert dodo.device_status() == 0


@pytest.mark.parametrize("mode", [0, 1, 3])
def test_attend_dense_many_sequences_and_empty_blocks(dodo, oracle, mode):
    # more sequences than one launch group holds (the second launch reuses counters and workspace), some of
    # them without queries, all others with two query tiles (so that mode 1 keeps them in step)
    from paper_2310_02409_b200 import api
    rs = np.random.RandomState(11)
    B = 70
    tqs = [0 if b % 9 == 4 else int(rs.randint(129, 200)) for b in range(B)]
    clens = [int(rs.randint(0, 150)) for _ in range(B)]
    llens = [t + int(rs.randint(0, 40)) for t in tqs]
    dodo.set_tuning(api.TUNE_DENSE_BALANCE, mode)
    try:
        eo, el = _attend_case(dodo, oracle, torch.bfloat16, 2, 128, tqs, clens, llens, tag=("dense-many", mode))
    finally:
        dodo.set_tuning(api.TUNE_DENSE_BALANCE, 0)
    assert eo <= 2e-2 and el <= 1e-3
    assert dodo.device_status() == 0


def test_attend_dense_equals_streaming_kernel(dodo, oracle):
    # the same call through both kernels (shape rule overridden): results agree within tolerance
    from paper_2310_02409_b200 import api
    args = (dodo, oracle, torch.bfloat16, 4, 128, [96, 33], [205, 500], [96, 40])
    e_dense, _ = _attend_case(*args, tag="both")
    dodo.set_tuning(api.TUNE_DENSE_MIN_QUERIES, 1 << 30)
    try:
        e_simt, _ = _attend_case(*args, tag="both")
    finally:
        dodo.set_tuning(api.TUNE_DENSE_MIN_QUERIES, 32)
    assert e_dense <= 2e-2 and e_simt <= 2e-2
