"""GPU parity of dodo_compress (score, TopK and gather in one call; Eq. 14 then Eq. 5) against the oracle and
against the two calls it stands for.

Checked per case: the scores lie in the fp32 accumulation band of the fp64 oracle; the indices are the oracle's
TopK of the very scores the GPU wrote (bit-exact, ties to the lower position); the cache rows, positions and
lengths are the oracle's gather of those indices (bit-exact), rows outside the appended range untouched; and
scores, indices and caches equal dodo_score_select + dodo_gather_kv bit for bit.  The shapes cover the overlapped
form (up to 64 sequences of up to 4096 tokens: the gather follows each sequence's selection through a flag), its
edges (empty sequences, k = 0, a ragged last block of rows, the last token forced, a second append behind the
first, calls back to back on one context) and the batches that run as the two plain calls (more than 64
sequences, a longer sequence).
"""
import numpy as np
import pytest
import torch

from paper_2310_02409_b200 import inputs

pytestmark = pytest.mark.gpu


def dev(x):
    return x.cuda() if isinstance(x, torch.Tensor) else torch.from_numpy(np.ascontiguousarray(x)).cuda()


def _band(X, w):
    return 1e-5 * (1.0 + (X.double().abs() @ w.double().abs()).numpy())


class _Case:
    """One batch: inputs on both sides, caches with canary rows, oracle-side mirrors."""

    def __init__(self, dtype, d, H, dh, lens, ks, tag, pre=None):
        self.lens, self.ks = lens, ks
        B = len(lens)
        self.seq_off, self.nug_off = inputs.offsets(lens), inputs.offsets(ks)
        N = max(int(self.seq_off[-1]), 1)
        self.X = inputs.randn((N, d), "compress", tag, "X", dtype=dtype)
        self.w = inputs.randn((d,), "compress", tag, "w", std=d ** -0.5, dtype=dtype)
        self.K = inputs.randn((N, H, dh), "compress", tag, "K", dtype=dtype)
        self.V = inputs.randn((N, H, dh), "compress", tag, "V", dtype=dtype)
        pre = pre or [0] * B
        self.pre = pre
        caps = [k + p + (b % 3) for b, (k, p) in enumerate(zip(ks, pre))]     # some slack rows per region
        self.cache_off = inputs.offsets(caps)
        cap = int(self.cache_off[-1]) + 2                                        # canary rows behind the last region
        self.cK = torch.full((cap, H, dh), 7.0, dtype=dtype)
        self.cV = torch.full((cap, H, dh), 9.0, dtype=dtype)
        self.cpos = torch.full((cap,), -5, dtype=torch.int32)
        self.pos_base = np.array([100 * b + 3 for b in range(B)], np.int32)
        self.Xd, self.wd, self.Kd, self.Vd = dev(self.X), dev(self.w), dev(self.K), dev(self.V)

    def fresh(self):
        return dev(self.cK), dev(self.cV), dev(self.cpos), np.array(self.pre, np.int32)


def _run(dodo, c, flags, bias, one_call):
    N = max(int(c.seq_off[-1]), 1)
    scores = torch.full((N,), float("nan"), device="cuda")
    idx = torch.full((max(int(c.nug_off[-1]), 1),), -1, dtype=torch.int32, device="cuda")
    cK, cV, cpos, clen = c.fresh()
    if one_call:
        dodo.compress(c.Xd, c.wd, bias, c.Kd, c.Vd, c.seq_off, c.nug_off, c.pos_base, flags, scores, idx, cK, cV, cpos,
                      c.cache_off, clen)
    else:
        dodo.score_select(c.Xd, c.wd, bias, c.seq_off, c.nug_off, flags, scores, idx)
        dodo.gather_kv(c.Kd, c.Vd, c.seq_off, idx, c.nug_off, c.pos_base, cK, cV, cpos, c.cache_off, clen)
    torch.cuda.synchronize()
    return scores, idx, cK, cV, cpos, clen


def _check(dodo, oracle, c, flags=0, bias=0.25):
    n_seq, n_nug = int(c.seq_off[-1]), int(c.nug_off[-1])
    scores, idx, cK, cV, cpos, clen = _run(dodo, c, flags, bias, True)
    assert dodo.device_status() == 0
    s_np = scores.cpu().numpy()[:n_seq]
    # scores: inside the fp32 accumulation band of the fp64 oracle, every element written
    ref = oracle.score(inputs.to_numpy(c.X)[:n_seq], inputs.to_numpy(c.w), bias)
    assert np.all(np.abs(s_np.astype(np.float64) - ref) <= _band(c.X[:n_seq], c.w))
    # indices: the oracle's TopK of exactly these scores
    want_idx = oracle.select_ragged(s_np, c.seq_off, c.nug_off, flags)
    got_idx = idx.cpu().numpy()[:n_nug]
    assert np.array_equal(got_idx, want_idx)
    # caches: the oracle's gather of those indices into the same pre-filled regions
    cK_o, cV_o, cpos_o = inputs.to_numpy(c.cK).copy(), inputs.to_numpy(c.cV).copy(), c.cpos.numpy().copy()
    len_o = oracle.gather_ragged(inputs.to_numpy(c.K), inputs.to_numpy(c.V), c.seq_off, want_idx, c.nug_off, c.pos_base,
                                 cK_o, cV_o, cpos_o, c.cache_off, list(c.pre))
    assert clen.tolist() == list(len_o)
    assert np.array_equal(inputs.to_numpy(cK), cK_o) and np.array_equal(inputs.to_numpy(cV), cV_o)
    assert np.array_equal(cpos.cpu().numpy(), cpos_o)
    # and the two calls it stands for give the same bits
    s2, i2, cK2, cV2, cpos2, clen2 = _run(dodo, c, flags, bias, False)
    assert torch.equal(scores[:n_seq], s2[:n_seq]) and torch.equal(idx[:n_nug], i2[:n_nug])
    assert torch.equal(cK, cK2) and torch.equal(cV, cV2) and torch.equal(cpos, cpos2) and clen.tolist() == clen2.tolist()
    return scores, idx, cK, cV


@pytest.mark.parametrize("name,dtype,d,H,dh,lens,r,flags", [
    # the decode workload's shape at a quarter of its width: 8 sequences, 64 score items each, 205 nuggets each
    ("c2", torch.bfloat16, 1024, 8, 128, [2048] * 8, 10, 0),
    # ragged: an empty sequence, a one-token sequence, lengths that end inside a block of rows and inside a group
    # of four nuggets; the last token forced into the selection
    ("ragged", torch.bfloat16, 512, 4, 64, [100, 0, 37, 1, 1000, 33, 2047], 10, 1),
    ("fp32", torch.float32, 256, 2, 64, [517, 64, 3], 4, 0),
    # r = 1: every token is a nugget (k = n), 16-byte rows
    ("r1", torch.bfloat16, 72, 1, 8, [130, 70], 1, 0),
    # the longest sequences the overlapped form takes, beside a short one (its gather waits for the long TopK)
    ("long", torch.bfloat16, 256, 2, 64, [4096, 40, 4095], 20, 0),
    # a sequence of the longest kind whose scores start off a 16-byte boundary: its selection streams them in two tiles
    ("long-unaligned", torch.bfloat16, 128, 1, 64, [3, 4096, 2, 4094], 10, 1),
    # one sequence
    ("single", torch.bfloat16, 256, 2, 64, [3000], 10, 0),
    # 64 sequences: the most one launch holds
    ("b64", torch.bfloat16, 128, 1, 64, inputs.loguniform_lengths(64, 1, 600, "compress-b64"), 5, 0),
])
def test_compress_overlapped(dodo, oracle, name, dtype, d, H, dh, lens, r, flags):
    ks = [oracle.num_nuggets(n, r) for n in lens]
    _check(dodo, oracle, _Case(dtype, d, H, dh, lens, ks, name), flags)


def test_compress_k_zero_and_append_behind_earlier_rows(dodo, oracle):
    # sequences that keep nothing (their flags are still raised, nothing waits on them), regions that already
    # hold rows: the new rows land behind them and the old ones stay
    lens = [300, 200, 0, 64]
    c = _Case(torch.bfloat16, 256, 2, 64, lens, [30, 0, 0, 7], "append", pre=[5, 2, 0, 1])
    _check(dodo, oracle, c)


def test_compress_back_to_back_calls_leave_the_context_clean(dodo, oracle):
    # the flags, the exit counter and the tickets return to zero inside the launches: different shapes in a row,
    # then the first one again with identical bits
    a = _Case(torch.bfloat16, 512, 4, 64, [700, 33, 1500], [70, 4, 150], "again-a")
    b = _Case(torch.bfloat16, 256, 2, 64, [64] * 40, [7] * 40, "again-b")
    first = _check(dodo, oracle, a)
    _check(dodo, oracle, b)
    again = _check(dodo, oracle, a)
    for x, y in zip(first, again):
        assert torch.equal(x, y)


@pytest.mark.parametrize("name,lens", [
    ("65-sequences", [40 + b for b in range(65)]),  # more than one launch's argument holds
    ("too-long", [4097, 100]),                     # selected by a launch of its own
    ("longer", [16384, 7168, 12288, 9000]),        # ... by thread-block clusters
])
def test_compress_batches_that_run_as_two_calls(dodo, oracle, name, lens):
    ks = [oracle.num_nuggets(n, 10) for n in lens]
    _check(dodo, oracle, _Case(torch.bfloat16, 256, 2, 64, lens, ks, name))


def test_compress_rejects_bad_arguments(dodo):
    from paper_2310_02409_b200 import api
    c = _Case(torch.bfloat16, 256, 2, 64, [100, 50], [10, 5], "bad")
    scores = torch.empty(150, device="cuda")
    idx = torch.empty(15, dtype=torch.int32, device="cuda")
    cK, cV, cpos, clen = c.fresh()
    with pytest.raises(api.DodoError) as e:      # k exceeds n
        dodo.compress(c.Xd, c.wd, 0.0, c.Kd, c.Vd, c.seq_off, inputs.offsets([101, 5]), c.pos_base, 0, scores, idx, cK, cV,
                      cpos, c.cache_off, clen)
    assert e.value.status == api.ERR_INVALID_ARG
    with pytest.raises(api.DodoError) as e:      # a region too small for its nuggets: nothing is launched
        dodo.compress(c.Xd, c.wd, 0.0, c.Kd, c.Vd, c.seq_off, c.nug_off, c.pos_base, 0, scores, idx, cK, cV, cpos,
                      inputs.offsets([9, 9]), clen)
    assert e.value.status == api.ERR_CAPACITY and clen.tolist() == [0, 0]
    assert torch.equal(cK, dev(c.cK))


@pytest.mark.parametrize("kind", inputs.STRESS_KINDS)
@pytest.mark.parametrize("flags", [0, 1])
def test_compress_on_stress_scores(dodo, oracle, kind, flags):
    """Scores that stress the selection (ties, constants, signed zeros, infinities and NaNs, denormals) reach the
    fused selection exactly: X carries the wanted score in its first feature and w = (1, 0, 0, ...), so that the
    pre-counted first radix pass, the early exit to direct ranking (or its absence, with more than 512 equal keys)
    and the flag-following gather all see them.  Lengths: within one register tile, the longest fused length, and
    the longest one starting off a 16-byte boundary (streamed in two tiles)."""
    lens = [700, 3, 4096, 1, 2048, 4096]
    seq_off = inputs.offsets(lens)
    ks = [oracle.num_nuggets(n, 7) for n in lens]
    nug_off = inputs.offsets(ks)
    N, d, H, dh = int(seq_off[-1]), 8, 1, 8
    want = np.concatenate([inputs.stress_scores(kind, n, "compress-stress", b) for b, n in enumerate(lens)])
    X = torch.zeros((N, d), dtype=torch.float32)
    X[:, 0] = torch.from_numpy(want)
    w = torch.zeros(d, dtype=torch.float32)
    w[0] = 1.0
    K = inputs.randn((N, H, dh), "compress-stress", "K")
    V = inputs.randn((N, H, dh), "compress-stress", "V")
    scores = torch.full((N,), 123.0, device="cuda")
    idx = torch.full((int(nug_off[-1]),), -1, dtype=torch.int32, device="cuda")
    cK = torch.zeros((int(nug_off[-1]), H, dh), device="cuda")
    cV = torch.zeros_like(cK)
    cpos = torch.full((int(nug_off[-1]),), -1, dtype=torch.int32, device="cuda")
    clen = np.zeros(len(lens), np.int32)
    dodo.compress(dev(X), dev(w), 0.0, dev(K), dev(V), seq_off, nug_off, np.zeros(len(lens), np.int32), flags, scores, idx,
                  cK, cV, cpos, nug_off, clen)
    torch.cuda.synchronize()
    assert dodo.device_status() == 0
    got = scores.cpu().numpy()
    # the scores arrive bit for bit (NaN payloads aside; -0 + 0 bias gives +0, which ranks the same)
    both_nan = np.isnan(got) & np.isnan(want)
    assert np.all(both_nan | (got == want))
    want_idx = oracle.select_ragged(got, seq_off, nug_off, flags)
    assert np.array_equal(idx.cpu().numpy(), want_idx)
    rows = np.concatenate([seq_off[b] + want_idx[nug_off[b]:nug_off[b + 1]] for b in range(len(lens))])
    assert np.array_equal(cK.cpu().numpy(), K.numpy()[rows]) and np.array_equal(cV.cpu().numpy(), V.numpy()[rows])
    assert np.array_equal(cpos.cpu().numpy(), want_idx) and clen.tolist() == ks


@pytest.mark.parametrize("kind", inputs.STRESS_KINDS)
@pytest.mark.parametrize("flags", [0, 1])
def test_score_select_long_on_stress_scores(dodo, oracle, kind, flags):
    """The same stress scores through the long-sequence form of dodo_score_select: the score launch counts the top
    key digits, the selection launched behind it (one block of 1024 threads up to 8192 tokens, a thread-block cluster
    beyond) starts from those counts and clears them; a second call on the same context must find them cleared."""
    lens = [9000, 5000, 16384, 8192]
    seq_off = inputs.offsets(lens)
    ks = [oracle.num_nuggets(n, 9) for n in lens]
    nug_off = inputs.offsets(ks)
    N, d = int(seq_off[-1]), 8
    want = np.concatenate([inputs.stress_scores(kind, n, "select-long-stress", b) for b, n in enumerate(lens)])
    X = torch.zeros((N, d), dtype=torch.float32)
    X[:, 0] = torch.from_numpy(want)
    w = torch.zeros(d, dtype=torch.float32)
    w[0] = 1.0
    Xd, wd = dev(X), dev(w)
    for _ in range(2):
        scores = torch.full((N,), 123.0, device="cuda")
        idx = torch.full((int(nug_off[-1]),), -1, dtype=torch.int32, device="cuda")
        dodo.score_select(Xd, wd, 0.0, seq_off, nug_off, flags, scores, idx)
        torch.cuda.synchronize()
        assert dodo.device_status() == 0
        got = scores.cpu().numpy()
        assert np.all((np.isnan(got) & np.isnan(want)) | (got == want))
        assert np.array_equal(idx.cpu().numpy(), oracle.select_ragged(got, seq_off, nug_off, flags))
