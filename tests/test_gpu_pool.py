"""GPU parity of dodo_pool_kv, the mean-pooling comparison system (Sec. 5.1): pooled K/V rows and their positions
against the fp64 oracle, appends into partly filled caches, and attention over the pooled cache through
dodo_attend against the oracle's attention over the same rows."""
import numpy as np
import pytest
import torch

import parity_log
from paper_2310_02409_b200 import inputs

pytestmark = pytest.mark.gpu


def _dev(x):
    return x.cuda() if isinstance(x, torch.Tensor) else torch.from_numpy(np.ascontiguousarray(x)).cuda()


@pytest.mark.parametrize("dtype,H,dh,r", [(torch.bfloat16, 32, 128, 10), (torch.float32, 4, 64, 10), (torch.bfloat16, 3, 8, 4),
                                          (torch.bfloat16, 40, 128, 1), (torch.float32, 2, 64, 20)])
def test_pool_matches_oracle_and_appends(dodo, oracle, dtype, H, dh, r):
    lens = [320, 0, 37, 261, 5]
    B, seq_off = len(lens), inputs.offsets(lens)
    N = int(seq_off[-1])
    K = inputs.randn((N, H, dh), "pool", r, "K", dtype=dtype)
    V = inputs.randn((N, H, dh), "pool", r, "V", dtype=dtype)
    ks = [oracle.num_nuggets(n, r) for n in lens]
    used = [3, 0, 1, 0, 2]                                   # rows already in each region stay untouched
    cache_off = inputs.offsets([k + u + 1 for k, u in zip(ks, used)])
    cap = int(cache_off[-1])
    cK = torch.full((cap + 2, H, dh), 7.0, dtype=dtype); cV = torch.full((cap + 2, H, dh), -9.0, dtype=dtype)
    cpos = torch.full((cap + 2,), -5, dtype=torch.int32)
    cKd, cVd, cpd = _dev(cK), _dev(cV), _dev(cpos)
    clen = np.asarray(used, np.int32)
    pos_base = np.array([100 * b for b in range(B)], np.int32)
    dodo.pool_kv(_dev(K), _dev(V), seq_off, r, pos_base, cKd, cVd, cpd, cache_off, clen)
    torch.cuda.synchronize()
    assert clen.tolist() == [u + k for u, k in zip(used, ks)]
    gotK, gotV, gotp = cKd.cpu(), cVd.cpu(), cpd.cpu().numpy()
    Kn, Vn = inputs.to_numpy(K), inputs.to_numpy(V)
    touched = np.zeros(cap + 2, bool)
    worst = 0.0
    for b in range(B):
        mk, pk = oracle.pool(Kn[seq_off[b]:seq_off[b + 1]], r, int(pos_base[b])) if lens[b] else (np.zeros((0, H, dh)), np.zeros(0, np.int32))
        mv, _ = oracle.pool(Vn[seq_off[b]:seq_off[b + 1]], r, int(pos_base[b])) if lens[b] else (np.zeros((0, H, dh)), None)
        at = int(cache_off[b]) + used[b]
        touched[at:at + ks[b]] = True
        assert np.array_equal(gotp[at:at + ks[b]], pk)
        for got, ref in ((gotK, mk), (gotV, mv)):
            g = got[at:at + ks[b]].double().numpy()
            # fp32 sums of r terms, one rounding to the storage type
            tol = (2.0 ** -8 if dtype == torch.bfloat16 else 2.0 ** -22) * np.abs(ref) + 1e-6
            assert np.all(np.abs(g - ref) <= tol)
            worst = max(worst, float(np.max(np.abs(g - ref))) if ks[b] else 0.0)
    # nothing else was written: earlier rows, slack rows and the canary rows keep their fill
    assert bool((gotK[~touched].float() == 7.0).all()) and bool((gotV[~touched].float() == -9.0).all())
    assert np.all(gotp[~touched] == -5)
    parity_log.LOG.add(f"pool {dtype} r={r}", pool_abs=worst)
    if r == 1:      # every token is its own segment: the pooled cache is the K/V themselves
        for b in range(B):
            at = int(cache_off[b]) + used[b]
            assert torch.equal(gotK[at:at + ks[b]], K[seq_off[b]:seq_off[b + 1]])
    # a region too small for its sequence's segments is refused before any launch
    from paper_2310_02409_b200 import api
    with pytest.raises(api.DodoError) as e:
        dodo.pool_kv(_dev(K), _dev(V), seq_off, r, pos_base, cKd, cVd, cpd, cache_off, clen)
    assert e.value.status == api.ERR_CAPACITY


def test_attend_over_pooled_cache(dodo, oracle):
    # the comparison system end to end: 320 / 640 tokens of history pooled at ratio 10 into 32 / 64 states, then a decode
    # token and a block of queries attend the pooled states plus a window of recent tokens (the budgets of Table 1)
    H, dh, r = 8, 128, 10
    lens, tqs, llens = [320, 640, 77], [1, 40, 3], [32, 64, 3]
    B, seq_off = 3, inputs.offsets(lens)
    K = inputs.randn((int(seq_off[-1]), H, dh), "pool-att", "K", dtype=torch.bfloat16)
    V = inputs.randn((int(seq_off[-1]), H, dh), "pool-att", "V", dtype=torch.bfloat16)
    ks = [oracle.num_nuggets(n, r) for n in lens]
    assert ks[:2] == [32, 64]
    cache_off = inputs.offsets(ks)
    cK = torch.zeros((int(cache_off[-1]), H, dh), dtype=torch.bfloat16, device="cuda"); cV = torch.zeros_like(cK)
    cpos = torch.zeros(int(cache_off[-1]), dtype=torch.int32, device="cuda")
    clen = np.zeros(B, np.int32)
    dodo.pool_kv(_dev(K), _dev(V), seq_off, r, np.zeros(B, np.int32), cK, cV, cpos, cache_off, clen)
    q_off, loc_off = inputs.offsets(tqs), inputs.offsets(llens)
    Q = inputs.randn((int(q_off[-1]), H, dh), "pool-att", "Q", dtype=torch.bfloat16)
    lK = inputs.randn((int(loc_off[-1]), H, dh), "pool-att", "lK", dtype=torch.bfloat16)
    lV = inputs.randn((int(loc_off[-1]), H, dh), "pool-att", "lV", dtype=torch.bfloat16)
    loc_pos0 = np.asarray(lens, np.int32)
    q_pos0 = loc_pos0 + np.asarray(llens, np.int32) - np.asarray(tqs, np.int32)
    O = torch.full((int(q_off[-1]), H, dh), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((int(q_off[-1]), H), float("nan"), device="cuda")
    ws = torch.empty(dodo.attend_workspace_bytes(dh), dtype=torch.uint8, device="cuda")
    dodo.attend(_dev(Q), q_off, q_pos0, dh ** -0.5, cK, cV, cpos, cache_off, clen, _dev(lK), _dev(lV), loc_off[:-1],
                np.asarray(llens, np.int32), loc_pos0, O, lse, ws)
    torch.cuda.synchronize()
    # the oracle attends the pooled rows as the kernel stored them (their rounding is checked above), at the positions it computes itself
    pos_ref = np.concatenate([oracle.pool(inputs.to_numpy(K[seq_off[b]:seq_off[b + 1]]), r)[1] for b in range(B)])
    assert np.array_equal(cpos.cpu().numpy(), pos_ref)
    Oo, lo = oracle.attend_ragged(inputs.to_numpy(Q), q_off, q_pos0, dh ** -0.5, inputs.to_numpy(cK), inputs.to_numpy(cV), pos_ref,
                                  cache_off, ks, inputs.to_numpy(lK), inputs.to_numpy(lV), loc_off[:-1], llens, loc_pos0)
    eo = float(np.max(np.abs(O.float().cpu().numpy().astype(np.float64) - Oo)))
    el = float(np.max(np.abs(lse.cpu().numpy().astype(np.float64) - lo)))
    parity_log.LOG.add("attend over a pooled cache", decode_O=eo, decode_lse=el)
    assert eo <= 2e-2 and el <= 1e-3
