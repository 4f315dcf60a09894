"""Pins for the CPU oracle: every oracle function is checked against something other than itself
(values the paper prints, brute force, closed forms, library routines, invariants)."""
import itertools
import math
from pathlib import Path

import numpy as np
import pytest
import torch

from paper_2310_02409_b200 import inputs

GOLDEN = Path(__file__).resolve().parent / "golden"


# --------------------------------------------------------------------------- k = ceil(n / r)

def _golden_counts():
    rows = []
    for line in (GOLDEN / "nugget_counts.txt").read_text().splitlines():
        line = line.split("#")[0].strip()
        if line:
            rows.append(tuple(int(x) for x in line.split()))
    return rows


@pytest.mark.parametrize("n,r,k", _golden_counts())
def test_num_nuggets_printed_values(oracle, n, r, k):
    assert oracle.num_nuggets(n, r) == k


def test_num_nuggets_is_smallest_k_covering_n(oracle):
    # k is the least integer with k * r >= n
    for n in range(0, 300):
        for r in (1, 2, 3, 5, 7, 10, 20, 64):
            k = oracle.num_nuggets(n, r)
            assert k * r >= n and (k - 1) * r < n


# --------------------------------------------------------------------------- score

def test_score_closed_forms(oracle):
    d = 64
    w = np.arange(d, dtype=np.float32) - 10.0
    # rows of the identity pick out single weights; a row of ones sums them
    X = np.concatenate([np.eye(d, dtype=np.float32), np.ones((1, d), np.float32)])
    s = oracle.score(X, w, bias=0.5)
    assert np.array_equal(s[:d], w.astype(np.float64) + 0.5)
    assert s[d] == float(w.sum()) + 0.5


def test_score_bf16_bit_patterns(oracle):
    # bf16 bits: 0x3F80 = 1, 0xC000 = -2, 0x3F00 = 0.5, 0x4049 = 3.140625
    X = np.array([[0x3F80, 0xC000, 0x3F00, 0x4049]], dtype=np.uint16)
    w = np.array([0x3F80, 0x3F80, 0xC000, 0x3F80], dtype=np.uint16)
    assert oracle.score(X, w)[0] == 1.0 - 2.0 - 1.0 + 3.140625


def test_score_matches_library_dot(oracle):
    X = inputs.randn((37, 256), "pin", "X").numpy()
    w = inputs.randn((256,), "pin", "w", std=1 / 16).numpy()
    ref = X.astype(np.float64) @ w.astype(np.float64) - 0.25
    np.testing.assert_allclose(oracle.score(X, w, -0.25), ref, rtol=0, atol=1e-12)


def test_score_not_transposed(oracle):
    # a [rows, d] array read as [d, rows] would mix rows; one hot row shows it
    X = np.zeros((3, 5), np.float32)
    X[1, 4] = 2.0
    w = np.array([1, 10, 100, 1000, 10000], np.float32)
    assert oracle.score(X, w).tolist() == [0.0, 20000.0, 0.0]


# --------------------------------------------------------------------------- select (TopK)

def _precedes(s, i, j):
    """Total order of the paper's TopK with ties to the lower position; NaN after everything."""
    a, b = s[i], s[j]
    an, bn = math.isnan(a), math.isnan(b)
    if an != bn:
        return bn
    if not an and a != b:
        return a > b
    return i < j


def _brute_force_topk(s, k):
    n = len(s)
    hits = []
    for sub in itertools.combinations(range(n), k):
        inside = set(sub)
        outside = [j for j in range(n) if j not in inside]
        if all(_precedes(s, i, j) for i in sub for j in outside):
            hits.append(list(sub))
    assert len(hits) == 1, "the tie-break makes the answer unique"
    return hits[0]


@pytest.mark.parametrize("kind", ["normal", "quantised8", "two_valued", "all_equal", "specials",
                                  "signed_zeros"])
def test_select_brute_force_small(oracle, kind):
    for n in range(1, 13):
        s = inputs.stress_scores(kind, n, "bf")
        for k in range(0, n + 1):
            got = oracle.select(s, k).tolist()
            assert got == _brute_force_topk([float(x) for x in s], k), (kind, n, k, s)


def test_select_brute_force_n16(oracle):
    s = inputs.stress_scores("quantised8", 16, "bf16")
    for k in (1, 2, 8, 15):
        assert oracle.select(s, k).tolist() == _brute_force_topk([float(x) for x in s], k)


@pytest.mark.parametrize("kind", ["normal", "quantised8", "two_valued", "ascending", "descending",
                                  "denormals"])
@pytest.mark.parametrize("n", [1, 2, 31, 512, 2048, 5000])
def test_select_matches_library_stable_argsort(oracle, kind, n):
    s = inputs.stress_scores(kind, n, "lib")
    for r in (1, 3, 10, 20):
        k = -(-n // r)
        order = np.argsort(-s.astype(np.float64), kind="stable")
        assert oracle.select(s, k).tolist() == sorted(order[:k].tolist())


def test_select_invariants_and_special_cases(oracle):
    n, k = 1000, 100
    s = inputs.stress_scores("normal", n, "inv")
    idx = oracle.select(s, k)
    assert len(idx) == k and np.all(np.diff(idx) > 0) and idx.min() >= 0 and idx.max() < n
    rest = np.setdiff1d(np.arange(n), idx)
    assert s[idx].min() >= s[rest].max()
    # all scores equal: the lowest k positions win
    assert oracle.select(np.full(50, 3.0, np.float32), 7).tolist() == list(range(7))
    # duplicates straddling the k-th place: of the three 5.0's only the two lowest positions fit
    s2 = np.array([1, 5, 9, 5, 0, 5, 9], np.float32)
    assert oracle.select(s2, 4).tolist() == [1, 2, 3, 6]
    # -0.0 ties with +0.0
    assert oracle.select(np.array([-0.0, 0.0, -0.0], np.float32), 2).tolist() == [0, 1]
    # NaN ranks below -inf and is taken only when k forces it
    s3 = np.array([np.nan, -np.inf, 1.0, np.nan], np.float32)
    assert oracle.select(s3, 2).tolist() == [1, 2]
    assert oracle.select(s3, 3).tolist() == [0, 1, 2]
    # k = n keeps everything, k = 0 nothing
    assert oracle.select(s2, 7).tolist() == list(range(7))
    assert oracle.select(s2, 0).tolist() == []
    with pytest.raises(ValueError):
        oracle.select(s2, 8)


def test_select_force_last(oracle):
    # footnote to Eq. 14: the last token is always a nugget; k is unchanged
    s = np.array([3, 9, 1, 7, -5], np.float32)
    assert oracle.select(s, 2).tolist() == [1, 3]
    assert oracle.select(s, 2, oracle.FORCE_LAST).tolist() == [1, 4]
    assert oracle.select(s, 1, oracle.FORCE_LAST).tolist() == [4]
    assert oracle.select(s, 5, oracle.FORCE_LAST).tolist() == [0, 1, 2, 3, 4]
    # when the last token is already among the best, forcing changes nothing
    s[4] = 100
    assert oracle.select(s, 3, oracle.FORCE_LAST).tolist() == oracle.select(s, 3).tolist()


def test_select_depends_only_on_ranking(oracle):
    # Eq. 6: p = sigmoid(score) is monotone, so TopK on scores and on probabilities agree
    s = inputs.stress_scores("normal", 777, "sig").astype(np.float64)
    p = 1.0 / (1.0 + np.exp(-s))
    assert len(np.unique(p)) == len(np.unique(s))
    assert oracle.select(s, 78).tolist() == oracle.select(p, 78).tolist()


# --------------------------------------------------------------------------- gather

@pytest.mark.parametrize("dtype", [np.float32, np.uint16])
def test_gather_is_a_row_copy(oracle, dtype):
    rs = np.random.RandomState(0)
    n, H, dh, cap = 40, 3, 8, 20
    src = rs.randint(0, 60000, size=(n, H, dh)).astype(dtype)
    cache = np.full((cap, H, dh), 7, dtype=dtype)
    pos = np.full(cap, -1, np.int32)
    idx1 = np.array([0, 5, 6, 39], np.int32)
    length = oracle.gather(src, idx1, 100, cache, pos, 0)
    assert length == 4
    idx2 = np.array([2, 3], np.int32)
    before = cache[:4].copy()
    length = oracle.gather(src, idx2, 500, cache, pos, length)
    assert length == 6
    assert np.array_equal(cache[:4], before) and np.array_equal(cache[:4], src[idx1])
    assert np.array_equal(cache[4:6], src[idx2])
    assert np.all(cache[6:] == 7) and np.all(pos[6:] == -1)
    assert pos[:6].tolist() == [100, 105, 106, 139, 502, 503]
    with pytest.raises(ValueError):
        oracle.gather(src, np.arange(15, dtype=np.int32), 0, cache, pos, length)


# --------------------------------------------------------------------------- attend

def _bits(t):
    return inputs.to_numpy(t)


def _sdpa_full_causal(q, k, v, scale):
    """Library full causal attention (Eq. 3) in fp64.  q, k, v: [T, H, dh] over one whole sequence."""
    qh, kh, vh = (x.double().permute(1, 0, 2).unsqueeze(0) for x in (q, k, v))
    o = torch.nn.functional.scaled_dot_product_attention(qh, kh, vh, is_causal=True, scale=scale)
    return o[0].permute(1, 0, 2).numpy()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_attend_r1_equals_full_causal_attention(oracle, dtype):
    # compression ratio 1 keeps every token, so Eq. 13 over nuggets must equal Eq. 3
    n, m, H, dh = 50, 9, 3, 16
    scale = 0.37
    q = inputs.randn((n + m, H, dh), "r1", "q", dtype=dtype)
    k = inputs.randn((n + m, H, dh), "r1", "k", dtype=dtype)
    v = inputs.randn((n + m, H, dh), "r1", "v", dtype=dtype)
    full = _sdpa_full_causal(q, k, v, scale)
    idx = oracle.select(inputs.stress_scores("normal", n, "r1"), oracle.num_nuggets(n, 1))
    assert idx.tolist() == list(range(n))
    o, lse = oracle.attend(_bits(q[n:]), n, scale, _bits(k[:n])[idx], _bits(v[:n])[idx], idx, n,
                           _bits(k[n:]), _bits(v[n:]), m, n)
    np.testing.assert_allclose(o, full[n:], rtol=0, atol=1e-12)
    logits = torch.einsum("thc,shc->hts", q.double(), k.double()) * scale
    mask = torch.tril(torch.ones(n + m, n + m, dtype=torch.bool))
    ref_lse = torch.logsumexp(logits.masked_fill(~mask, -math.inf), dim=-1).T.numpy()
    np.testing.assert_allclose(lse, ref_lse[n:], rtol=0, atol=1e-12)


def test_attend_masks_future_nuggets_by_position(oracle):
    # every token is in the cache, queries sit in the middle of the sequence: a key is visible
    # only if its position is <= the query's, which is again full causal attention
    n, H, dh = 40, 2, 8
    q = inputs.randn((n, H, dh), "mask", "q")
    k = inputs.randn((n, H, dh), "mask", "k")
    v = inputs.randn((n, H, dh), "mask", "v")
    full = _sdpa_full_causal(q, k, v, 0.5)
    perm = np.random.RandomState(1).permutation(n)     # cache order must not matter, positions do
    o, _ = oracle.attend(_bits(q[10:25]), 10, 0.5, _bits(k)[perm], _bits(v)[perm],
                         perm.astype(np.int32), n, None, None, 0, 0)
    np.testing.assert_allclose(o, full[10:25], rtol=0, atol=1e-12)
    # the same through the local segment alone (positions lpos0 + j)
    o2, _ = oracle.attend(_bits(q[10:25]), 10, 0.5, None, None, None, 0, _bits(k), _bits(v), n, 0)
    np.testing.assert_allclose(o2, full[10:25], rtol=0, atol=1e-12)


def test_attend_closed_forms(oracle):
    H, dh = 2, 4
    q = np.zeros((1, H, dh), np.float32)
    q[0, 0, 0] = 2.0
    q[0, 1, 1] = 1.0
    K = np.zeros((2, H, dh), np.float32)
    K[0, 0, 0] = math.log(3.0)      # head 0: logits scale*2*ln3 and 0
    K[1, 1, 1] = math.log(7.0)      # head 1: logits 0 and scale*ln7
    V = np.zeros((2, H, dh), np.float32)
    V[0, :, :] = 1.0
    V[1, :, :] = 5.0
    pos = np.array([0, 1], np.int32)
    o, lse = oracle.attend(q, 5, 0.5, K, V, pos, 2, None, None, 0, 0)
    l3 = float(np.float32(math.log(3.0)))
    l7 = float(np.float32(math.log(7.0)))
    w0 = math.exp(l3) / (math.exp(l3) + 1.0)                      # ~3/4 on key 0
    w1 = math.exp(0.5 * l7) / (math.exp(0.5 * l7) + 1.0)          # ~sqrt7/(1+sqrt7) on key 1
    np.testing.assert_allclose(o[0, 0], np.full(dh, w0 * 1.0 + (1 - w0) * 5.0), atol=1e-14)
    np.testing.assert_allclose(o[0, 1], np.full(dh, (1 - w1) * 1.0 + w1 * 5.0), atol=1e-14)
    np.testing.assert_allclose(lse[0], [math.log(math.exp(l3) + 1), math.log(math.exp(0.5 * l7) + 1)],
                               atol=1e-14)
    # zero queries: uniform weights, o = mean(V), lse = log(#keys)
    n = 11
    Kr = inputs.randn((n, H, dh), "cf", "k").numpy()
    Vr = inputs.randn((n, H, dh), "cf", "v").numpy()
    o, lse = oracle.attend(np.zeros((1, H, dh), np.float32), 99, 1.0, Kr, Vr,
                           np.arange(n, dtype=np.int32), n, None, None, 0, 0)
    np.testing.assert_allclose(o[0], Vr.astype(np.float64).mean(0), atol=1e-14)
    np.testing.assert_allclose(lse, math.log(n), atol=1e-14)
    # a single visible key returns its value row; nothing visible returns zeros and -inf
    o, lse = oracle.attend(np.ones((1, H, dh), np.float32), 0, 1.0, Kr, Vr,
                           np.arange(n, dtype=np.int32), n, None, None, 0, 0)
    assert np.array_equal(o[0], Vr[0].astype(np.float64))
    o, lse = oracle.attend(np.ones((1, H, dh), np.float32), -1, 1.0, Kr, Vr,
                           np.arange(n, dtype=np.int32), n, None, None, 0, 0)
    assert np.all(o == 0) and np.all(np.isneginf(lse))


def test_attend_brute_force_python(oracle):
    Tq, H, dh, c, l = 3, 2, 4, 5, 4
    Q = inputs.randn((Tq, H, dh), "py", "q").numpy()
    cK = inputs.randn((c, H, dh), "py", "ck").numpy()
    cV = inputs.randn((c, H, dh), "py", "cv").numpy()
    lK = inputs.randn((l, H, dh), "py", "lk").numpy()
    lV = inputs.randn((l, H, dh), "py", "lv").numpy()
    cpos = np.array([0, 3, 4, 9, 12], np.int32)
    q0, l0, scale = 11, 10, 0.7
    o, lse = oracle.attend(Q, q0, scale, cK, cV, cpos, c, lK, lV, l, l0)
    for t in range(Tq):
        for h in range(H):
            keys = [(cK[j, h], cV[j, h]) for j in range(c) if cpos[j] <= q0 + t]
            keys += [(lK[j, h], lV[j, h]) for j in range(l) if l0 + j <= q0 + t]
            lg = [scale * sum(float(a) * float(b) for a, b in zip(Q[t, h], kk)) for kk, _ in keys]
            z = sum(math.exp(x) for x in lg)
            ref = [sum(math.exp(x) / z * float(vv[cdim]) for x, (_, vv) in zip(lg, keys))
                   for cdim in range(dh)]
            np.testing.assert_allclose(o[t, h], ref, atol=1e-13)
            assert abs(lse[t, h] - math.log(z)) < 1e-13


def test_attend_invariants(oracle):
    Tq, H, dh, c, l = 4, 3, 8, 30, 12
    Q = inputs.randn((Tq, H, dh), "iv", "q").numpy()
    cK = inputs.randn((c, H, dh), "iv", "ck").numpy()
    cV = inputs.randn((c, H, dh), "iv", "cv").numpy()
    lK = inputs.randn((l, H, dh), "iv", "lk").numpy()
    lV = inputs.randn((l, H, dh), "iv", "lv").numpy()
    cpos = np.sort(np.random.RandomState(3).choice(100, c, replace=False)).astype(np.int32)
    o, lse = oracle.attend(Q, 108, 0.3, cK, cV, cpos, c, lK, lV, l, 100)
    # convex combination of the visible value rows
    allV = np.concatenate([cV, lV]).astype(np.float64)
    assert np.all(o <= allV.max(0) + 1e-12) and np.all(o >= allV.min(0) - 1e-12)
    # attending [A ; B] equals the log-sum-exp merge of attending A and B separately
    oa, la = oracle.attend(Q, 108, 0.3, cK, cV, cpos, c, None, None, 0, 0)
    ob, lb = oracle.attend(Q, 108, 0.3, None, None, None, 0, lK, lV, l, 100)
    m = np.maximum(la, lb)
    wa, wb = np.exp(la - m), np.exp(lb - m)
    merged = (oa * wa[..., None] + ob * wb[..., None]) / (wa + wb)[..., None]
    np.testing.assert_allclose(o, merged, atol=1e-12)
    np.testing.assert_allclose(lse, m + np.log(wa + wb), atol=1e-12)
    # constant value rows come back unchanged
    oc, _ = oracle.attend(Q, 108, 0.3, cK, np.full_like(cV, 2.5), cpos, c, None, None, 0, 0)
    np.testing.assert_allclose(oc, 2.5, atol=1e-13)


def test_ragged_helpers_match_per_sequence_calls(oracle):
    lens = [5, 0, 17]
    seq_off = inputs.offsets(lens)
    ks = [oracle.num_nuggets(n, 4) for n in lens]
    nug_off = inputs.offsets(ks)
    s = inputs.stress_scores("quantised8", int(seq_off[-1]), "rag")
    idx = oracle.select_ragged(s, seq_off, nug_off)
    for b in range(3):
        assert idx[nug_off[b]:nug_off[b + 1]].tolist() == \
            oracle.select(s[seq_off[b]:seq_off[b + 1]], ks[b]).tolist()


def test_gather_ragged_matches_per_sequence_calls(oracle):
    # a ragged batch with an empty sequence and caches that already hold rows: the batch loop must equal one
    # plain row copy per sequence (numpy fancy indexing), appended after the rows in use, positions = base + idx
    lens = [9, 0, 30, 4]
    H, dh = 2, 4
    seq_off = inputs.offsets(lens)
    ks = [3, 0, 7, 4]
    nug_off = inputs.offsets(ks)
    used = [2, 0, 5, 0]                       # rows already in each cache region
    caps = [6, 1, 13, 4]
    cache_off = inputs.offsets(caps)
    N, cap = int(seq_off[-1]), int(cache_off[-1])
    K = inputs.randn((N, H, dh), "grag", "K").numpy()
    V = inputs.randn((N, H, dh), "grag", "V").numpy()
    rs = np.random.RandomState(17)
    idx = np.concatenate([np.sort(rs.choice(n, k, replace=False)) for n, k in zip(lens, ks)]).astype(np.int32)
    pos_base = np.array([100, 200, 300, 400], np.int32)
    cK = np.full((cap, H, dh), -7.0, np.float32); cV = np.full((cap, H, dh), -9.0, np.float32)
    cpos = np.full(cap, -5, np.int32)
    want_K, want_V, want_pos = cK.copy(), cV.copy(), cpos.copy()
    new_len = oracle.gather_ragged(K, V, seq_off, idx, nug_off, pos_base, cK, cV, cpos, cache_off, used)
    assert new_len == [u + k for u, k in zip(used, ks)]
    for b in range(4):
        ib = idx[nug_off[b]:nug_off[b + 1]]
        at = int(cache_off[b]) + used[b]
        want_K[at:at + ks[b]] = K[seq_off[b]:seq_off[b + 1]][ib]
        want_V[at:at + ks[b]] = V[seq_off[b]:seq_off[b + 1]][ib]
        want_pos[at:at + ks[b]] = pos_base[b] + ib
    assert np.array_equal(cK, want_K) and np.array_equal(cV, want_V) and np.array_equal(cpos, want_pos)
    # a region that cannot take its sequence's rows is refused
    with pytest.raises(ValueError):
        oracle.gather_ragged(K, V, seq_off, idx, nug_off, pos_base, cK, cV, cpos, cache_off, [4, 0, 5, 0])


def test_attend_ragged_matches_per_sequence_calls(oracle):
    # ragged batch: a sequence without queries, one without local tokens, one without nuggets, caches only
    # partly in use (rows past cache_len must not be looked at), local windows at non-zero offsets
    H, dh = 2, 8
    tqs = [3, 0, 1, 2]
    clen = [5, 4, 0, 9]
    caps = [7, 4, 2, 9]
    llen = [4, 2, 6, 0]
    q_off, cache_off = inputs.offsets(tqs), inputs.offsets(caps)
    loc_off = np.array([1, 6, 9, 0], np.int32)          # rows 0, 5 and 8 are gaps
    Q = inputs.randn((int(q_off[-1]), H, dh), "arag", "Q").numpy()
    cK = inputs.randn((int(cache_off[-1]), H, dh), "arag", "cK").numpy()
    cV = inputs.randn((int(cache_off[-1]), H, dh), "arag", "cV").numpy()
    lK = inputs.randn((16, H, dh), "arag", "lK").numpy()
    lV = inputs.randn((16, H, dh), "arag", "lV").numpy()
    cpos = np.full(int(cache_off[-1]), 10 ** 6, np.int32)     # unused rows carry junk positions
    for b in range(4):
        cpos[cache_off[b]:cache_off[b] + clen[b]] = np.arange(clen[b]) * 3
    loc_pos0 = np.array([20, 15, 2, 0], np.int32)
    q_pos0 = np.array([21, 0, 7, 12], np.int32)               # sequence 0: causal inside its local tokens
    O, lse = oracle.attend_ragged(Q, q_off, q_pos0, 0.4, cK, cV, cpos, cache_off, clen, lK, lV, loc_off, llen, loc_pos0)
    assert O.shape == Q.shape and lse.shape == Q.shape[:2]
    for b in range(4):
        if tqs[b] == 0:
            continue
        c0, l0 = int(cache_off[b]), int(loc_off[b])
        o, l = oracle.attend(Q[q_off[b]:q_off[b + 1]], int(q_pos0[b]), 0.4, cK[c0:c0 + clen[b]], cV[c0:c0 + clen[b]],
                             cpos[c0:c0 + clen[b]], clen[b], lK[l0:l0 + llen[b]], lV[l0:l0 + llen[b]], llen[b],
                             int(loc_pos0[b]))
        assert np.array_equal(O[q_off[b]:q_off[b + 1]], o) and np.array_equal(lse[q_off[b]:q_off[b + 1]], l)
    # ... and against the definition written out for one (query, head): softmax over the visible keys only
    b, t, h = 3, 1, 1
    q = Q[q_off[b] + t, h].astype(np.float64)
    vis = [j for j in range(clen[b]) if cpos[cache_off[b] + j] <= q_pos0[b] + t]
    assert vis == [0, 1, 2, 3, 4]                              # positions 0, 3, ..., 12 <= 13; 15 and up are hidden
    logit = np.array([0.4 * float(q @ cK[cache_off[b] + j, h].astype(np.float64)) for j in vis])
    p = np.exp(logit - logit.max()); p /= p.sum()
    ref = sum(pj * cV[cache_off[b] + j, h].astype(np.float64) for pj, j in zip(p, vis))
    np.testing.assert_allclose(O[q_off[b] + t, h], ref, atol=1e-13)
    # loc_len = None means no local tokens anywhere
    O2, _ = oracle.attend_ragged(Q, q_off, q_pos0, 0.4, cK, cV, cpos, cache_off, clen, None, None, None, None, None)
    o3, _ = oracle.attend(Q[q_off[3]:q_off[4]], int(q_pos0[3]), 0.4, cK[cache_off[3]:], cV[cache_off[3]:], cpos[cache_off[3]:],
                          clen[3], None, None, 0, 0)
    assert np.array_equal(O2[q_off[3]:q_off[4]], o3)


# --------------------------------------------------------------------------- threshold selection (Eq. 8)

@pytest.mark.parametrize("kind", inputs.STRESS_KINDS)
def test_select_threshold_brute_force(oracle, kind):
    s = inputs.stress_scores(kind, 257, "thr")
    finite = s[np.isfinite(s)]
    for lam in [-np.inf, np.inf, np.nan, 0.0, -0.0] + ([float(np.median(finite)), float(finite.max()), float(finite.min())] if finite.size else []):
        want = [i for i in range(len(s)) if float(s[i]) > lam]      # IEEE: NaN on either side is never "above"
        assert oracle.select_threshold(s, lam).tolist() == want


def test_select_threshold_agrees_with_topk(oracle):
    # Distinct scores: keeping what lies above the (k+1)-th largest score is keeping the k largest (Eq. 8 vs Eq. 14).
    s = np.random.RandomState(5).permutation(400).astype(np.float32) * 0.37 - 60.0
    order = np.sort(s)[::-1]
    for k in (1, 7, 40, 399):
        assert oracle.select_threshold(s, float(order[k])).tolist() == oracle.select(s, k).tolist()
    assert oracle.select_threshold(s, float(order[0])).tolist() == []
    # ties: the strict test keeps none of the scores equal to Lambda, TopK keeps the lowest positions of them
    t = np.array([1.0, 2.0, 2.0, 3.0, 2.0], np.float32)
    assert oracle.select_threshold(t, 2.0).tolist() == [3]
    assert oracle.select(t, 2).tolist() == [1, 3]


def test_select_threshold_monotone_in_lambda(oracle):
    s = inputs.stress_scores("normal", 500, "mono")
    prev = set(range(500))
    for lam in np.linspace(-3, 3, 25):
        cur = set(oracle.select_threshold(s, float(lam)).tolist())
        assert cur <= prev
        prev = cur


@pytest.mark.parametrize("m,r", [(100, 10), (101, 10), (64, 1), (7, 20), (1, 1), (1000, 3)])
def test_estimate_threshold_against_library_sort(oracle, m, r):
    s = np.random.RandomState(m * 31 + r).standard_normal(m).astype(np.float32)     # distinct with probability 1
    lam = oracle.estimate_threshold(s, r)
    k = -(-m // r)
    if k >= m:
        assert lam == -np.inf and len(oracle.select_threshold(s, lam)) == m
    else:
        assert lam == float(np.sort(s)[::-1][k])                    # the (k+1)-th largest, by numpy's sort
        assert len(oracle.select_threshold(s, lam)) == k            # exactly k of the sample pass: about m / r (text after Eq. 8)
        assert abs(k - m / r) < 1


def test_estimate_threshold_special_values(oracle):
    s = np.array([np.nan, 1.0, -np.inf, np.inf, 0.0, -0.0, np.nan, 2.0], np.float32)
    # ranking: inf, 2, 1, 0 (= -0), -0, -inf, nan, nan
    assert oracle.estimate_threshold(s, 8) == 2.0                   # k = 1 -> second largest
    assert oracle.estimate_threshold(s, 2) == 0.0                   # k = 4 -> fifth largest: one of the zeros
    assert oracle.estimate_threshold(s, 4 / 3 if False else 1) == -np.inf
    lam = oracle.estimate_threshold(s[[0, 6, 1]], 2)                # k = 2 of 3 -> third largest is a NaN
    assert math.isnan(lam) and oracle.select_threshold(s, lam).tolist() == []


# --------------------------------------------------------------------------- two-layer Scorer (Eq. 6, App. B.3)

def test_score_mlp_reduces_to_linear_scorer(oracle):
    # identity first layer, identity activation: s = w2 . x + b2, the linear Scorer
    d = 48
    X = inputs.randn((21, d), "mlp", "X").numpy()
    w2 = inputs.randn((d,), "mlp", "w2", std=0.2).numpy()
    s = oracle.score_mlp(X, np.eye(d, dtype=np.float32), np.zeros(d, np.float32), w2, 0.75, oracle.ACT_IDENTITY)
    np.testing.assert_allclose(s, oracle.score(X, w2, 0.75), rtol=0, atol=1e-13)


@pytest.mark.parametrize("act", [0, 1, 2])
def test_score_mlp_matches_library_matmul(oracle, act):
    rows, d, dh = 19, 40, 56                                     # not square: a transposed W1 cannot pass
    X = inputs.randn((rows, d), "mlp2", "X").numpy()
    W1 = inputs.randn((dh, d), "mlp2", "W1", std=d ** -0.5).numpy()
    b1 = inputs.randn((dh,), "mlp2", "b1", std=0.3).numpy()
    w2 = inputs.randn((dh,), "mlp2", "w2", std=dh ** -0.5).numpy()
    pre = X.astype(np.float64) @ W1.astype(np.float64).T + b1.astype(np.float64)
    if act == 1:
        h = np.maximum(pre, 0.0)
    elif act == 2:
        h = 0.5 * pre * (1.0 + np.tanh(math.sqrt(2.0 / math.pi) * (pre + 0.044715 * pre ** 3)))
    else:
        h = pre
    ref = h @ w2.astype(np.float64) - 1.5
    np.testing.assert_allclose(oracle.score_mlp(X, W1, b1, w2, -1.5, act), ref, rtol=0, atol=1e-12)


def test_score_mlp_closed_forms_and_parameter_count(oracle):
    d = 8
    X = np.array([[1, -2, 3, -4, 5, -6, 7, -8]], np.float32)
    # ReLU keeps the positive coordinates, the bias shifts the kink, w2 sums what is left
    s = oracle.score_mlp(X, np.eye(d, dtype=np.float32), np.full(d, 0.5, np.float32), np.ones(d, np.float32), 0.0, oracle.ACT_RELU)
    assert s[0] == (1 + 3 + 5 + 7) + 4 * 0.5
    # GELU at 0 is 0, and far from 0 it is the identity / zero
    g = oracle.score_mlp(np.array([[0.0, 30.0, -30.0]], np.float32), np.eye(3, dtype=np.float32), np.zeros(3, np.float32),
                         np.array([1.0, 1.0, 1.0], np.float32), 0.0, oracle.ACT_GELU_TANH)
    assert abs(g[0] - 30.0) < 1e-12
    # bf16 storage: exact widening (0x3F80 = 1, 0xC000 = -2, 0x3F00 = 0.5)
    Xb = np.array([[0x3F80, 0xC000]], np.uint16)
    Wb = np.array([[0x3F80, 0x3F00], [0xC000, 0x3F80]], np.uint16)         # h = (1 - 1, -2 - 2) = (0, -4)
    assert oracle.score_mlp(Xb, Wb, np.array([1.0, 5.0], np.float32), np.array([0x3F80, 0x3F00], np.uint16), 0.0, 1)[0] == 1.0 + 0.5
    # the shape the paper's parameter count fixes (Table 5: 16.8M Scorer parameters at d = 4096)
    dd = 4096
    assert dd * dd + dd + dd + 1 == 16_785_409


# --------------------------------------------------------------------------- mean pooling of even chunks (Sec. 5.1 baseline)

@pytest.mark.parametrize("n,r", [(320, 10), (37, 5), (7, 10), (64, 1), (1, 3)])
def test_pool_matches_library_mean(oracle, n, r):
    x = inputs.randn((n, 3, 4), "pool", n, r, "x").numpy()
    out, pos = oracle.pool(x, r, pos_base=1000)
    k = -(-n // r)
    assert out.shape == (k, 3, 4) and pos.shape == (k,)
    for j in range(k):
        seg = x[j * r:(j + 1) * r].astype(np.float64)               # numpy slicing stops at n by itself
        np.testing.assert_allclose(out[j], seg.mean(axis=0), rtol=0, atol=1e-15)
        assert pos[j] == 1000 + min((j + 1) * r, n) - 1
    # the printed budgets: 320 / 640 / 1280 tokens of history pooled at ratio 10 give 32 / 64 / 128 states (Table 1)
    assert [len(oracle.pool(np.zeros((m, 2), np.float32), 10)[1]) for m in (320, 640, 1280)] == [32, 64, 128]


def test_pool_special_cases(oracle):
    # r = 1: every token is its own segment -- the identity, at the tokens' own positions
    x = inputs.randn((9, 5), "pool1", "x").numpy()
    out, pos = oracle.pool(x, 1, pos_base=7)
    assert np.array_equal(out, x.astype(np.float64)) and pos.tolist() == list(range(7, 16))
    # constant segments come back unchanged; a sign error or a wrong divisor (r instead of the short last segment's 2) would not
    y = np.repeat(np.array([[2.0], [-3.0], [5.0]], np.float32), 4, axis=0)[:10]        # segments of 4, 4, 2 rows
    out, pos = oracle.pool(y, 4)
    assert out[:, 0].tolist() == [2.0, -3.0, 5.0] and pos.tolist() == [3, 7, 9]
    # bf16 storage widens exactly: 0x3F80 = 1, 0x4000 = 2, 0x4040 = 3 -> mean 2
    b = np.array([[0x3F80], [0x4000], [0x4040]], np.uint16)
    assert oracle.pool(b, 3)[0][0, 0] == 2.0
