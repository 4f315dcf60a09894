"""GPU parity of threshold selection (Eq. 8) and of the threshold estimate against the CPU oracle:
counts and positions bit-exact, Lambda equal as a number, and one streaming pass through
score -> estimate -> count -> select -> gather -> attend."""
import math

import numpy as np
import pytest
import torch

from paper_2310_02409_b200 import inputs

pytestmark = pytest.mark.gpu


def dev(x):
    return x.cuda() if isinstance(x, torch.Tensor) else torch.from_numpy(np.ascontiguousarray(x)).cuda()


def _threshold_gpu(dodo, s_np, seq_off, lam, regions=None):
    """counts, then positions laid out from the counts (or into the given regions)."""
    B = len(seq_off) - 1
    s = dev(s_np.astype(np.float32))
    counts = torch.full((max(B, 1),), -7, dtype=torch.int32, device="cuda")
    dodo.count_threshold(s, seq_off, lam, counts)
    c = counts.cpu().numpy()[:B]                    # the one device-to-host read of this mode
    nug_off = inputs.offsets(c if regions is None else regions)
    idx = torch.full((max(int(nug_off[-1]), 1),), -7, dtype=torch.int32, device="cuda")
    dodo.select_threshold(s, seq_off, nug_off, lam, idx)
    torch.cuda.synchronize()
    return c, idx.cpu().numpy()[:int(nug_off[-1])], nug_off


def _lambdas(s):
    fin = s[np.isfinite(s)]
    out = [-np.inf, np.inf, float("nan"), 0.0]
    if fin.size:
        out += [float(np.median(fin)), float(fin.max()), float(fin.min()), float(np.float32(np.percentile(fin, 90)))]
    return out


@pytest.mark.parametrize("kind", inputs.STRESS_KINDS)
@pytest.mark.parametrize("n", [1, 31, 1000, 1024, 1025, 40000])
def test_threshold_bit_exact_single_sequence(dodo, oracle, kind, n):
    s = inputs.stress_scores(kind, n, "gpu-thr")
    for lam in _lambdas(s):
        lam32 = float(np.float32(lam))
        want = oracle.select_threshold(s, lam32)
        c, got, _ = _threshold_gpu(dodo, s, inputs.offsets([n]), lam32)
        assert c.tolist() == [len(want)] and np.array_equal(got, want), (kind, n, lam)


def test_threshold_ragged_batch_and_regions(dodo, oracle):
    lens = [0, 5, 777, 0, 4096, 1, 12345, 64] + list(inputs.loguniform_lengths(120, 1, 600, "thr-many"))   # > one launch group
    seq_off = inputs.offsets(lens)
    s = inputs.stress_scores("quantised8", int(seq_off[-1]), "thr-ragged")
    lam = 0.25
    want = [oracle.select_threshold(s[seq_off[b]:seq_off[b + 1]], lam) for b in range(len(lens))]
    c, got, nug_off = _threshold_gpu(dodo, s, seq_off, lam)
    assert c.tolist() == [len(w) for w in want]
    assert np.array_equal(got, np.concatenate(want))
    # regions that do not match the counts: a short one keeps the lowest positions, a long one keeps its tail
    regions = [max(0, len(w) - 2) if b % 2 else min(lens[b], len(w) + 3) for b, w in enumerate(want)]
    _, got2, off2 = _threshold_gpu(dodo, s, seq_off, lam, regions)
    for b, w in enumerate(want):
        r = got2[off2[b]:off2[b + 1]]
        m = min(len(w), len(r))
        assert np.array_equal(r[:m], w[:m]) and np.all(r[m:] == -7)


@pytest.mark.parametrize("kind", ["normal", "quantised8", "specials", "signed_zeros", "all_equal"])
@pytest.mark.parametrize("m", [1, 100, 4096, 4097, 50000])
def test_estimate_threshold_equals_oracle(dodo, oracle, kind, m):
    s = inputs.stress_scores(kind, m, "gpu-est")
    out = torch.zeros(1, device="cuda")
    for r in (1, 2, 10, 20, 1000):
        dodo.estimate_threshold(dev(s.astype(np.float32)), r, out)
        got, want = float(out.cpu()[0]), oracle.estimate_threshold(s, r)
        assert (math.isnan(got) and math.isnan(want)) or got == want, (kind, m, r, got, want)


def test_threshold_rejects_bad_arguments(dodo):
    from paper_2310_02409_b200 import api
    s = torch.zeros(10, device="cuda")
    out = torch.zeros(4, dtype=torch.int32, device="cuda")
    with pytest.raises(api.DodoError):
        dodo.count_threshold(s, [1, 10], 0.0, out)               # offsets must start at 0
    with pytest.raises(api.DodoError):
        dodo.select_threshold(s, [0, 10], [0, 11], 0.0, out)      # a region longer than its sequence
    with pytest.raises(api.DodoError) as e:
        dodo.estimate_threshold(s, 0, torch.zeros(1, device="cuda"))
    assert e.value.status == api.ERR_INVALID_ARG


def test_streaming_threshold_path(dodo, oracle):
    """Contexts arrive, Lambda comes from a sample of their scores, nuggets are whatever passes; then the
    cache is attended.  Selection is checked on the GPU's own fp32 scores, attention against fp64."""
    dt, H, dh, d, r = torch.float32, 4, 64, 256, 8
    lens = [300, 41, 0, 1500]
    B, seq_off = len(lens), inputs.offsets(lens)
    N = int(seq_off[-1])
    X = inputs.randn((N, d), "stream", "X", dtype=dt)
    w = inputs.randn((d,), "stream", "w", std=d ** -0.5, dtype=dt)
    K = inputs.randn((N, H, dh), "stream", "K", dtype=dt)
    V = inputs.randn((N, H, dh), "stream", "V", dtype=dt)
    scores = torch.empty(N, device="cuda")
    dodo.score(dev(X), dev(w), 0.0, seq_off, scores)
    lam_d = torch.zeros(1, device="cuda")
    dodo.estimate_threshold(scores[:1024], r, lam_d)             # "sampled tokens": the first 1024 scores
    lam = float(lam_d.cpu()[0])
    s_np = scores.cpu().numpy()
    assert lam == oracle.estimate_threshold(s_np[:1024], r)
    counts = torch.zeros(B, dtype=torch.int32, device="cuda")
    dodo.count_threshold(scores, seq_off, lam, counts)
    c = counts.cpu().numpy()
    assert abs(int(c.sum()) - N / r) < 0.25 * N / r               # about one token in r (text after Eq. 8)
    nug_off = inputs.offsets(c)
    idx = torch.zeros(max(int(nug_off[-1]), 1), dtype=torch.int32, device="cuda")
    dodo.select_threshold(scores, seq_off, nug_off, lam, idx)
    want = [oracle.select_threshold(s_np[seq_off[b]:seq_off[b + 1]], lam) for b in range(B)]
    assert np.array_equal(idx.cpu().numpy()[:int(nug_off[-1])], np.concatenate(want))
    # gather and attend exactly as after TopK
    cache_off = inputs.offsets(c + 2)
    cap = int(cache_off[-1])
    cK = torch.zeros((cap, H, dh), device="cuda"); cV = torch.zeros_like(cK)
    cpos = torch.zeros(cap, dtype=torch.int32, device="cuda")
    cache_len = np.zeros(B, np.int32)
    dodo.gather_kv(dev(K), dev(V), seq_off, idx, nug_off, np.zeros(B, np.int32), cK, cV, cpos, cache_off, cache_len)
    assert cache_len.tolist() == c.tolist()
    tq = [3, 1, 2, 5]
    q_off = inputs.offsets(tq)
    Q = inputs.randn((int(q_off[-1]), H, dh), "stream", "Q", dtype=dt)
    q_pos0 = np.asarray(lens, np.int32)                           # the queries follow their contexts
    lK = inputs.randn((int(q_off[-1]), H, dh), "stream", "lK", dtype=dt)
    lV = inputs.randn((int(q_off[-1]), H, dh), "stream", "lV", dtype=dt)
    O = torch.zeros((int(q_off[-1]), H, dh), device="cuda")
    ws = torch.empty(dodo.attend_workspace_bytes(dh), dtype=torch.uint8, device="cuda")
    dodo.attend(dev(Q), q_off, q_pos0, dh ** -0.5, cK, cV, cpos, cache_off, cache_len, dev(lK), dev(lV), q_off[:-1],
                np.asarray(tq, np.int32), q_pos0, O, None, ws)
    torch.cuda.synchronize()
    cKo, cVo = np.zeros((cap, H, dh), np.float32), np.zeros((cap, H, dh), np.float32)
    cpo = np.zeros(cap, np.int32)
    oracle.gather_ragged(inputs.to_numpy(K), inputs.to_numpy(V), seq_off, np.concatenate(want).astype(np.int32), nug_off,
                         np.zeros(B, np.int32), cKo, cVo, cpo, cache_off, np.zeros(B, np.int32))
    assert np.array_equal(cKo, cK.cpu().numpy()) and np.array_equal(cpo, cpos.cpu().numpy())
    ref, _ = oracle.attend_ragged(inputs.to_numpy(Q), q_off, q_pos0, dh ** -0.5, cKo, cVo, cpo, cache_off, c,
                                  inputs.to_numpy(lK), inputs.to_numpy(lV), q_off[:-1], tq, q_pos0)
    assert np.max(np.abs(O.cpu().numpy().astype(np.float64) - ref)) <= 1e-4
