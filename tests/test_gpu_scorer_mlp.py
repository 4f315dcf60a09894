"""GPU parity of the two-layer Scorer (Eq. 6, App. B.3) against the fp64 oracle, and its hand-over to TopK."""
import numpy as np
import pytest
import torch

from paper_2310_02409_b200 import inputs

pytestmark = pytest.mark.gpu


def dev(x):
    return x.cuda() if isinstance(x, torch.Tensor) else torch.from_numpy(np.ascontiguousarray(x)).cuda()


def _case(rows, d, dh, tag):
    bf = torch.bfloat16
    X = inputs.randn((rows, d), tag, "X", dtype=bf)
    W1 = inputs.randn((dh, d), tag, "W1", std=d ** -0.5, dtype=bf)
    b1 = inputs.randn((dh,), tag, "b1", std=0.5)
    w2 = inputs.randn((dh,), tag, "w2", std=dh ** -0.5, dtype=bf)
    return X, W1, b1, w2


def _tolerance(X, W1, b1, w2, rows_idx):
    """fp32 accumulation of products of bf16 pairs (exact in fp32) over d terms, then over dh terms:
    1e-5 of the sum of the magnitudes that enter a score, the same band as for the linear Scorer
    (the activations used are 1-Lipschitz, so first-layer errors pass through undamped at most)."""
    Xf, Wf = inputs.to_numpy(X).astype(np.uint32) << 16, inputs.to_numpy(W1).astype(np.uint32) << 16
    Xf, Wf = Xf.view(np.float32).astype(np.float64), Wf.view(np.float32).astype(np.float64)
    w2f = (inputs.to_numpy(w2).astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    mag = (np.abs(Xf[rows_idx]) @ np.abs(Wf).T + np.abs(b1.numpy().astype(np.float64))) @ np.abs(w2f)
    return 1e-5 * (1.0 + mag)


@pytest.mark.parametrize("act", [0, 1, 2])
@pytest.mark.parametrize("rows,d,dh", [(1, 64, 256), (300, 256, 256), (700, 320, 768), (513, 1024, 1024)])
def test_score_mlp_matches_oracle(dodo, oracle, rows, d, dh, act):
    X, W1, b1, w2 = _case(rows, d, dh, ("mlp", rows, d, dh))
    scores = torch.full((rows,), float("nan"), device="cuda")
    ws = torch.empty(dodo.score_mlp_workspace_bytes(rows, dh), dtype=torch.uint8, device="cuda")
    dodo.score_mlp(dev(X), dev(W1), dev(b1), dev(w2), -0.25, act, [0, rows], scores, ws)
    torch.cuda.synchronize()
    assert dodo.device_status() == 0
    ref = oracle.score_mlp(inputs.to_numpy(X), inputs.to_numpy(W1), b1.numpy(), inputs.to_numpy(w2), -0.25, act)
    got = scores.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - ref) <= _tolerance(X, W1, b1, w2, np.arange(rows))), float(np.max(np.abs(got - ref)))


def test_score_mlp_ragged_batch_reproducible_and_selected(dodo, oracle):
    lens = [0, 130, 1, 700, 256]
    seq_off = inputs.offsets(lens)
    rows, d, dh = int(seq_off[-1]), 256, 512
    X, W1, b1, w2 = _case(rows, d, dh, "mlp-ragged")
    ws = torch.empty(dodo.score_mlp_workspace_bytes(rows, dh), dtype=torch.uint8, device="cuda")
    s1 = torch.zeros(rows, device="cuda"); s2 = torch.zeros(rows, device="cuda")
    dodo.score_mlp(dev(X), dev(W1), dev(b1), dev(w2), 0.0, 1, seq_off, s1, ws)
    dodo.score_mlp(dev(X), dev(W1), dev(b1), dev(w2), 0.0, 1, seq_off, s2, ws)
    torch.cuda.synchronize()
    assert torch.equal(s1, s2)                                     # bit for bit, run to run
    ks = [oracle.num_nuggets(n, 10) for n in lens]
    nug_off = inputs.offsets(ks)
    idx = torch.zeros(int(nug_off[-1]), dtype=torch.int32, device="cuda")
    dodo.select(s1, seq_off, nug_off, 0, idx)                      # TopK on the GPU's own fp32 scores
    torch.cuda.synchronize()
    assert np.array_equal(idx.cpu().numpy(), oracle.select_ragged(s1.cpu().numpy(), seq_off, nug_off))


def test_score_mlp_llama_shape_sampled_rows(dodo, oracle):
    # d = dh = 4096 (the shape the paper's 16.8M parameters fix), 2,500 tokens; the oracle checks sampled rows,
    # among them the first and last of the ragged last block of 256
    rows, d, dh = 2500, 4096, 4096
    X, W1, b1, w2 = _case(rows, d, dh, "mlp-7b")
    scores = torch.full((rows,), float("nan"), device="cuda")
    ws = torch.empty(dodo.score_mlp_workspace_bytes(rows, dh), dtype=torch.uint8, device="cuda")
    dodo.score_mlp(dev(X), dev(W1), dev(b1), dev(w2), 0.5, 1, [0, 1000, rows], scores, ws)
    torch.cuda.synchronize()
    assert dodo.device_status() == 0 and bool(torch.isfinite(scores).all())
    pick = np.array([0, 1, 127, 128, 255, 256, 1000, 2047, 2303, 2304, 2400, 2499])
    ref = oracle.score_mlp(inputs.to_numpy(X)[pick], inputs.to_numpy(W1), b1.numpy(), inputs.to_numpy(w2), 0.5, 1)
    got = scores.cpu().numpy().astype(np.float64)[pick]
    assert np.all(np.abs(got - ref) <= _tolerance(X, W1, b1, w2, pick)), float(np.max(np.abs(got - ref)))


def test_score_mlp_rejects_bad_arguments(dodo):
    from paper_2310_02409_b200 import api
    X = torch.zeros((10, 64), dtype=torch.bfloat16, device="cuda")
    W = torch.zeros((256, 64), dtype=torch.bfloat16, device="cuda")
    b1 = torch.zeros(256, device="cuda"); w2 = torch.zeros(256, dtype=torch.bfloat16, device="cuda")
    s = torch.zeros(10, device="cuda")
    ws = torch.empty(dodo.score_mlp_workspace_bytes(10, 256), dtype=torch.uint8, device="cuda")
    with pytest.raises(api.DodoError) as e:
        dodo.score_mlp(X.float(), W.float(), b1, w2.float(), 0.0, 1, [0, 10], s, ws)           # fp32 inputs
    assert e.value.status == api.ERR_UNSUPPORTED
    with pytest.raises(api.DodoError) as e:
        dodo.score_mlp(X, W[:100], b1[:100], w2[:100], 0.0, 1, [0, 10], s, ws)                   # dh not a multiple of 256
    assert e.value.status == api.ERR_UNSUPPORTED
    with pytest.raises(api.DodoError) as e:
        dodo.score_mlp(X, W, b1, w2, 0.0, 7, [0, 10], s, ws)                                     # unknown activation
    assert e.value.status == api.ERR_INVALID_ARG
    with pytest.raises(api.DodoError) as e:
        dodo.score_mlp(X, W, b1, w2, 0.0, 1, [0, 10], s, ws[:8])                                 # workspace too small
    assert e.value.status == api.ERR_CAPACITY


@pytest.mark.parametrize("flags", [0, 1])
@pytest.mark.parametrize("lens", [[0, 130, 1, 700, 256], [2048] * 3 + [513], inputs.loguniform_lengths(70, 1, 1500, "mlp-fused"),
                                  [4096, 4500, 90]])
def test_score_mlp_select_fused(dodo, oracle, lens, flags):
    # the two-layer Scorer with its TopK fused into the reduction (the last case has a sequence beyond the fused limit and
    # takes the separate select launch; the 70-sequence one more than one launch group): the hand-over buffer holds
    # exactly what dodo_score_mlp writes, and the indices are the oracle's TopK of those scores, bit for bit
    seq_off = inputs.offsets(lens)
    rows, d, dh = int(seq_off[-1]), 256, 512
    X, W1, b1, w2 = _case(rows, d, dh, ("mlp-fused", len(lens), rows))
    ks = [oracle.num_nuggets(n, 10) for n in lens]
    nug_off = inputs.offsets(ks)
    ws = torch.empty(dodo.score_mlp_workspace_bytes(rows, dh), dtype=torch.uint8, device="cuda")
    Xd, W1d, b1d, w2d = dev(X), dev(W1), dev(b1), dev(w2)
    s_plain = torch.full((rows,), float("nan"), device="cuda")
    dodo.score_mlp(Xd, W1d, b1d, w2d, 0.125, 1, seq_off, s_plain, ws)
    for _ in range(2):          # twice: the arrival counters were left clean
        s_fused = torch.full((rows,), float("nan"), device="cuda")
        idx = torch.full((max(int(nug_off[-1]), 1),), -1, dtype=torch.int32, device="cuda")
        dodo.score_mlp_select(Xd, W1d, b1d, w2d, 0.125, 1, seq_off, nug_off, flags, s_fused, idx, ws)
        torch.cuda.synchronize()
        assert torch.equal(s_fused, s_plain)
        want = oracle.select_ragged(s_fused.cpu().numpy(), seq_off, nug_off, flags)
        assert np.array_equal(idx.cpu().numpy()[:int(nug_off[-1])], want)
    assert dodo.device_status() == 0
