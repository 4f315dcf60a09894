"""GPU parity on the workload configurations, driven through the same plumbing (`workloads.py`) and
launch configuration the benchmark times, against the fp64 CPU oracle."""
import numpy as np
import pytest
import torch

from paper_2310_02409_b200 import inputs

pytestmark = pytest.mark.gpu

TOL = {torch.bfloat16: 2e-2, torch.float32: 1e-4}


def _host(t):
    return inputs.to_numpy(t)


def _check_compress(oracle, inst):
    """Indices bit-exact against the oracle's TopK on the GPU's own fp32 scores, scores within the
    fp32 band of fp64, cache contents and positions bit-exact.  Returns the oracle's caches."""
    wl = inst.wl
    X, w = _host(inst.X), _host(inst.w)
    s_gpu = inst.scores.cpu().numpy()
    s64 = oracle.score(X, w, 0.0)
    band = 1e-5 * (1.0 + inst.X.cpu().double().abs().numpy() @ inst.w.cpu().double().abs().numpy())
    assert np.all(np.abs(s_gpu.astype(np.float64) - s64) <= band)
    idx_o = oracle.select_ragged(s_gpu, inst.seq_off, inst.nug_off, 0)
    Kt = int(inst.nug_off[-1])
    assert np.array_equal(inst.idx.cpu().numpy()[:Kt], idx_o)
    for b in range(wl.B):
        assert inst.nug_off[b + 1] - inst.nug_off[b] == oracle.num_nuggets(int(inst.n[b]), inst.r)
    cK = np.zeros_like(_host(inst.cacheK)); cV = np.zeros_like(cK)
    cpos = np.zeros(cK.shape[0], np.int32)
    lens = oracle.gather_ragged(_host(inst.K), _host(inst.V), inst.seq_off, idx_o, inst.nug_off,
                                np.zeros(wl.B, np.int32), cK, cV, cpos, inst.cache_off, [0] * wl.B)
    assert lens == inst.cache_len.tolist()
    assert np.array_equal(_host(inst.cacheK), cK) and np.array_equal(_host(inst.cacheV), cV)
    assert np.array_equal(inst.cache_pos.cpu().numpy(), cpos)
    # every nugget lies inside its sequence's compressed context
    for b in range(wl.B):
        p = cpos[inst.cache_off[b]:inst.cache_off[b] + lens[b]]
        assert np.all(np.diff(p) > 0) and p.min() >= 0 and p.max() < inst.n[b]
    return cK, cV, cpos, lens, s64


def _oracle_attend(oracle, inst, Q, q_off, tables, caches):
    cK, cV, cpos, lens = caches
    loc_off, loc_len, loc_pos0, q_pos0 = tables
    return oracle.attend_ragged(_host(Q), q_off, q_pos0, inst.sm_scale, cK, cV, cpos, inst.cache_off, lens,
                                _host(inst.locK), _host(inst.locV), loc_off, loc_len, loc_pos0)


def _errs(O, lse, ref):
    """max-abs errors of an output tensor and its log-sum-exp against the oracle's pair (O, lse)."""
    eo = float(np.max(np.abs(O.float().cpu().numpy().astype(np.float64) - ref[0])))
    el = float(np.max(np.abs(lse.cpu().numpy().astype(np.float64).reshape(ref[1].shape) - ref[1])))
    return eo, el


def test_c1_tiny_fp32_whole_path(dodo, oracle, errlog):
    from paper_2310_02409_b200.workloads import CompressDecode
    wl = inputs.WORKLOADS["c1_tiny_fp32"]
    inst = CompressDecode(dodo, wl, 10, ("seed", 0), gen_device="cpu", with_lse=True)
    inst.compress()
    inst.query_block()
    torch.cuda.synchronize()
    assert int(inst.k[0]) == 52
    cK, cV, cpos, lens, s64 = _check_compress(oracle, inst)
    # on this seeded input the all-fp64 pipeline selects the very same nuggets
    assert np.array_equal(oracle.select(s64, 52), inst.idx.cpu().numpy())
    ref = _oracle_attend(oracle, inst, inst.Qb, inst.qb_off, inst.block_tables(), (cK, cV, cpos, lens))
    err, err_l = _errs(inst.Ob, inst.lse_b, ref)
    errlog.add("c1 tiny fp32 query block", fp32_O=err, fp32_lse=err_l)
    assert err <= 1e-4 and err_l <= 1e-4, (err, err_l)


def test_c2_llama7b_decode_full_size(dodo, oracle, errlog):
    from paper_2310_02409_b200.workloads import CompressDecode
    wl = inputs.WORKLOADS["c2_llama7b_decode"]
    inst = CompressDecode(dodo, wl, 10, ("c2-parity",), gen_device="cpu", with_lse=True)
    assert inst.k.tolist() == [205] * 8
    inst.compress()
    steps = [0, 1, 63, 127]
    for s in steps:
        inst.decode_step(s)
    torch.cuda.synchronize()
    cK, cV, cpos, lens, _ = _check_compress(oracle, inst)
    for s in steps:
        ref = _oracle_attend(oracle, inst, inst.Qd[s], inst.q_off, inst.window(s), (cK, cV, cpos, lens))
        err, err_l = _errs(inst.Od[s], inst.lse_d[s], ref)
        errlog.add(f"c2 decode step {s}", decode_O=err, decode_lse=err_l)
        assert err <= 2e-2 and err_l <= 1e-3, (s, err, err_l)


@pytest.mark.parametrize("r", [1, 5, 10, 20])
def test_c4_shapes_ratio_sweep_scaled(dodo, oracle, r, errlog):
    # LLaMA-13B head geometry (40 x 128, d = 5120) at a context the oracle finishes in seconds; the
    # query block and two decode tokens; at r = 1 the result must equal full causal attention
    wl = inputs.Workload("c4_scaled", torch.bfloat16, (1500,), 5120, 40, 128, ratios=(r,), tq_dense=24,
                         decode_steps=2, layers=1)
    from paper_2310_02409_b200.workloads import CompressDecode
    inst = CompressDecode(dodo, wl, r, ("c4", r), gen_device="cpu", with_lse=True)
    inst.compress()
    inst.query_block()
    for s in range(2):
        inst.decode_step(s)
    torch.cuda.synchronize()
    assert int(inst.k[0]) == {1: 1500, 5: 300, 10: 150, 20: 75}[r]
    cK, cV, cpos, lens, _ = _check_compress(oracle, inst)
    ref = _oracle_attend(oracle, inst, inst.Qb, inst.qb_off, inst.block_tables(), (cK, cV, cpos, lens))
    got = inst.Ob.float().cpu().numpy().astype(np.float64)
    err, err_l = _errs(inst.Ob, inst.lse_b, ref)
    errlog.add(f"c4 scaled r={r} query block (24 queries)", block_O=err, block_lse=err_l)
    assert err <= 2e-2 and err_l <= 1e-3, (err, err_l)
    for s in range(2):
        ref_s = _oracle_attend(oracle, inst, inst.Qd[s], inst.q_off, inst.window(s), (cK, cV, cpos, lens))
        err, err_l = _errs(inst.Od[s], inst.lse_d[s], ref_s)
        errlog.add(f"c4 scaled r={r} decode step {s}", decode_O=err, decode_lse=err_l)
        assert err <= 2e-2 and err_l <= 1e-3, (s, err, err_l)
    if r == 1:
        # Eq. 3: full causal attention over [context ; block] by an independent library routine
        n, tq, H, dh = 1500, 24, 40, 128
        k = torch.cat([inst.K.cpu(), inst.locK.cpu()[:tq]]).double()
        v = torch.cat([inst.V.cpu(), inst.locV.cpu()[:tq]]).double()
        q = torch.cat([torch.zeros(n, H, dh, dtype=torch.float64), inst.Qb.cpu().double()])
        qh, kh, vh = (x.permute(1, 0, 2).unsqueeze(0) for x in (q, k, v))
        full = torch.nn.functional.scaled_dot_product_attention(qh, kh, vh, is_causal=True, scale=inst.sm_scale)
        full = full[0].permute(1, 0, 2)[n:].numpy()
        assert np.max(np.abs(got - full)) <= 2e-2


def test_c5_ragged_serving_with_appends_scaled(dodo, oracle, errlog):
    # 64 sequences, context lengths log-uniform (scaled down 16x so the oracle finishes in seconds),
    # one token per sequence per step, segments of 64 decoded tokens compressed and appended to the
    # nugget caches at steps 127, 191 and 255; checked at the first step, around every append and at
    # the last step
    from paper_2310_02409_b200.workloads import RaggedServing
    lengths = inputs.loguniform_lengths(64, 32, 2048, "c5-scaled")
    srv = RaggedServing(dodo, lengths, 512, 4, 128, 10, 256, ("c5",), gen_device="cpu", with_lse=True)
    srv.compress_context()
    torch.cuda.synchronize()
    # oracle state
    X, w, K, V = (_host(t) for t in (srv.X, srv.w, srv.K, srv.V))
    decX, decK, decV = _host(srv.decX), _host(srv.decK), _host(srv.decV)
    B, st = srv.B, srv.steps
    s_gpu = srv.scores.cpu().numpy()[:X.shape[0]]
    idx_o = oracle.select_ragged(s_gpu, srv.seq_off, srv.nug_off0, 0)
    assert np.array_equal(srv.idx.cpu().numpy()[:len(idx_o)], idx_o)
    cK = np.zeros_like(_host(srv.cacheK)); cV = np.zeros_like(cK)
    cpos = np.zeros(cK.shape[0], np.int32)
    lens = oracle.gather_ragged(K, V, srv.seq_off, idx_o, srv.nug_off0, np.zeros(B, np.int32), cK, cV, cpos,
                                srv.cache_off, [0] * B)
    win0 = 0
    check = {0, 126, 127, 128, 190, 191, 192, 254, 255}
    appended = []
    for s in range(st):
        tables = srv.window(s)
        did = srv.decode_step(s)
        if s in check:
            torch.cuda.synchronize()
            ref = oracle.attend_ragged(_host(srv.Qd[s]), srv.q_off, tables[3], srv.sm_scale, cK, cV, cpos, srv.cache_off,
                                       lens, decK.reshape(B * st, 4, 128), decV.reshape(B * st, 4, 128),
                                       tables[0], tables[1], tables[2])
            err, err_l = _errs(srv.Od[s], srv.lse_d[s], ref)
            errlog.add(f"c5 scaled step {s}", decode_O=err, decode_lse=err_l)
            assert err <= 2e-2 and err_l <= 1e-3, (s, err, err_l)
        if did:
            appended.append(s)
            torch.cuda.synchronize()
            # replay the append in the oracle: TopK of the segment's GPU scores, gather, positions
            segX = np.ascontiguousarray(decX[:, win0:win0 + 64]).reshape(B * 64, -1)
            sg = srv.scores.cpu().numpy()[:B * 64]
            s64 = oracle.score(segX, w, 0.0)
            assert np.max(np.abs(sg - s64)) < 1e-3
            io = oracle.select_ragged(sg, srv.seg_off, srv.seg_nug_off, 0)
            assert np.array_equal(srv.idx.cpu().numpy()[:len(io)], io)
            segK = np.ascontiguousarray(decK[:, win0:win0 + 64]).reshape(B * 64, 4, 128)
            segV = np.ascontiguousarray(decV[:, win0:win0 + 64]).reshape(B * 64, 4, 128)
            lens = oracle.gather_ragged(segK, segV, srv.seg_off, io, srv.seg_nug_off, srv.n + win0, cK, cV, cpos,
                                        srv.cache_off, lens)
            win0 += 64
            assert lens == srv.cache_len.tolist()
            assert np.array_equal(_host(srv.cacheK), cK) and np.array_equal(_host(srv.cacheV), cV)
            assert np.array_equal(srv.cache_pos.cpu().numpy(), cpos)
    assert appended == [127, 191, 255]
    assert all(lens[b] == oracle.num_nuggets(lengths[b], 10) + 3 * 7 for b in range(B))


def test_c3_ar_mode_scaled_two_layers(dodo, oracle, errlog):
    # autoregressive mode: compressed past + uncompressed recent tokens, a 256-token query block (the
    # tensor-core kernel) and then decode tokens with a growing window; two independent layers
    # (own X, w, K, V, Q, hence own nugget sets), context scaled so the oracle finishes in seconds
    from paper_2310_02409_b200.workloads import CompressDecode
    wl = inputs.Workload("c3_scaled", torch.bfloat16, (896,) * 4, 1024, 8, 128, local=128, tq_dense=256,
                         decode_steps=3, layers=2)
    picked = []
    for layer in range(wl.layers):
        inst = CompressDecode(dodo, wl, 10, ("c3", layer), gen_device="cpu", with_lse=True)
        assert not inst.sliding
        inst.compress()
        inst.query_block()
        for s in range(3):
            inst.decode_step(s)
        torch.cuda.synchronize()
        assert inst.k.tolist() == [90] * 4
        cK, cV, cpos, lens, _ = _check_compress(oracle, inst)
        picked.append(inst.idx.cpu().numpy().copy())
        ref = _oracle_attend(oracle, inst, inst.Qb, inst.qb_off, inst.block_tables(), (cK, cV, cpos, lens))
        err, err_l = _errs(inst.Ob, inst.lse_b, ref)
        errlog.add(f"c3 scaled layer {layer} query block", dense_O=err, dense_lse=err_l)
        assert err <= 2e-2 and err_l <= 1e-3, (err, err_l)
        for s in range(3):
            ref_s = _oracle_attend(oracle, inst, inst.Qd[s], inst.q_off, inst.window(s), (cK, cV, cpos, lens))
            err, err_l = _errs(inst.Od[s], inst.lse_d[s], ref_s)
            errlog.add(f"c3 scaled layer {layer} decode step {s}", decode_O=err, decode_lse=err_l)
            assert err <= 2e-2 and err_l <= 1e-3, (s, err, err_l)
    assert not np.array_equal(picked[0], picked[1])     # per-layer selection really is independent


@pytest.mark.parametrize("pinned_kv", [True, False])
def test_host_buffer_entry_point_matches_oracle(dodo, oracle, pinned_kv):
    # dodo_compress_decode_host: the same path fed from host memory in one call; pinned K/V are read in
    # place by the gather (only the nuggets' rows cross the bus), pageable K/V are uploaded whole
    from paper_2310_02409_b200 import api
    lens, d, H, dh, r, local, steps = [300, 77, 1000], 512, 4, 128, 10, 16, 5
    B = len(lens)
    seq_off = inputs.offsets(lens)
    ks = [oracle.num_nuggets(n, r) for n in lens]
    nug_off = inputs.offsets(ks)
    N = int(seq_off[-1])
    g = lambda shape, name, std=1.0: inputs.randn(shape, "hostpath", name, std=std, dtype=torch.bfloat16).pin_memory()
    hX, hw = g((N, d), "X"), g((d,), "w", d ** -0.5)
    hK, hV = g((N, H, dh), "K"), g((N, H, dh), "V")
    if not pinned_kv:
        hK, hV = hK.clone(), hV.clone()      # ordinary pageable copies
        assert not hK.is_pinned() and not hV.is_pinned()
    hLK, hLV = g((B, local + steps, H, dh), "lK"), g((B, local + steps, H, dh), "lV")
    hQ = g((steps, B, H, dh), "Q")
    hO = torch.zeros_like(hQ).pin_memory()
    arena = torch.empty(dodo.host_arena_bytes(api.BF16, d, H, dh, N, int(nug_off[-1]), B, local, steps),
                        dtype=torch.uint8, device="cuda")
    dodo.compress_decode_host(hX, hw, hK, hV, seq_off, nug_off, hLK, hLV, local, hQ, dh ** -0.5, hO, arena)
    torch.cuda.synchronize()
    assert dodo.device_status() == 0
    # oracle, all in fp64 (on these inputs the fp32 and fp64 score rankings agree)
    s64 = oracle.score(_host(hX), _host(hw))
    idx = oracle.select_ragged(s64.astype(np.float32), seq_off, nug_off)
    Kt = int(nug_off[-1])
    cK = np.zeros((Kt, H, dh), np.uint16); cV = np.zeros_like(cK); cpos = np.zeros(Kt, np.int32)
    clen = oracle.gather_ragged(_host(hK), _host(hV), seq_off, idx, nug_off, np.zeros(B, np.int32), cK, cV, cpos,
                                nug_off, [0] * B)
    lK, lV = _host(hLK).reshape(-1, H, dh), _host(hLV).reshape(-1, H, dh)
    n = np.asarray(lens, np.int32)
    base = np.arange(B, dtype=np.int32) * (local + steps)
    worst = 0.0
    for t in range(steps):
        ref = oracle.attend_ragged(_host(hQ[t]), np.arange(B + 1, dtype=np.int32), n + local + t, dh ** -0.5, cK, cV,
                                   cpos, nug_off, clen, lK, lV, base + t + 1, np.full(B, local, np.int32), n + t + 1)[0]
        worst = max(worst, float(np.max(np.abs(hO[t].float().numpy().astype(np.float64) - ref))))
    assert worst <= 2e-2, worst


def test_shared_indices_across_layers(dodo, oracle):
    """The paper's Sec. 2.1 form: the Scorer reads one layer's hidden states and the same token positions are
    kept at every layer.  One fused score+select, ONE gather for all layers, then one attend per layer."""
    dt, H, dh, d, r, L = torch.bfloat16, 4, 128, 512, 10, 3
    lens = [333, 1024, 77]
    B, seq_off = len(lens), inputs.offsets(lens)
    N = int(seq_off[-1])
    ks = np.asarray([oracle.num_nuggets(n, r) for n in lens], np.int32)
    nug_off = inputs.offsets(ks)
    X = inputs.randn((N, d), "shared", "X", dtype=dt)
    w = inputs.randn((d,), "shared", "w", std=d ** -0.5, dtype=dt)
    scores = torch.empty(N, device="cuda")
    idx = torch.empty(int(nug_off[-1]), dtype=torch.int32, device="cuda")
    dodo.score_select(X.cuda(), w.cuda(), 0.0, seq_off, nug_off, 0, scores, idx)
    torch.cuda.synchronize()
    idx_ref = oracle.select_ragged(scores.cpu().numpy(), seq_off, nug_off)
    assert np.array_equal(idx.cpu().numpy(), idx_ref)
    tq = [2, 1, 3]
    q_off = inputs.offsets(tq)
    q_pos0 = np.asarray(lens, np.int32)
    ws = torch.empty(dodo.attend_workspace_bytes(dh), dtype=torch.uint8, device="cuda")
    cap = int(nug_off[-1])
    Ks = [inputs.randn((N, H, dh), "shared", layer, "K", dtype=dt) for layer in range(L)]
    Vs = [inputs.randn((N, H, dh), "shared", layer, "V", dtype=dt) for layer in range(L)]
    cKs = [torch.zeros((cap, H, dh), dtype=dt, device="cuda") for _ in range(L)]
    cVs = [torch.zeros((cap, H, dh), dtype=dt, device="cuda") for _ in range(L)]
    cpos = torch.zeros(cap, dtype=torch.int32, device="cuda")
    cache_len = np.zeros(B, np.int32)
    dodo.gather_kv_layers([t.cuda() for t in Ks], [t.cuda() for t in Vs], seq_off, idx, nug_off, np.zeros(B, np.int32),
                          cKs, cVs, cpos, nug_off, cache_len)
    assert np.array_equal(cache_len, ks)
    for layer in range(L):
        Q = inputs.randn((int(q_off[-1]), H, dh), "shared", layer, "Q", dtype=dt)
        lK = inputs.randn((int(q_off[-1]), H, dh), "shared", layer, "lK", dtype=dt)
        lV = inputs.randn((int(q_off[-1]), H, dh), "shared", layer, "lV", dtype=dt)
        O = torch.zeros((int(q_off[-1]), H, dh), dtype=dt, device="cuda")
        dodo.attend(Q.cuda(), q_off, q_pos0, dh ** -0.5, cKs[layer], cVs[layer], cpos, nug_off, cache_len, lK.cuda(),
                    lV.cuda(), q_off[:-1], np.asarray(tq, np.int32), q_pos0, O, None, ws)
        torch.cuda.synchronize()
        Kn, Vn = inputs.to_numpy(Ks[layer]), inputs.to_numpy(Vs[layer])
        cKo, cVo = np.zeros((cap, H, dh), Kn.dtype), np.zeros((cap, H, dh), Vn.dtype)
        cpo = np.zeros(cap, np.int32)
        oracle.gather_ragged(Kn, Vn, seq_off, idx_ref, nug_off, np.zeros(B, np.int32), cKo, cVo, cpo, nug_off, np.zeros(B, np.int32))
        assert np.array_equal(cKo, inputs.to_numpy(cKs[layer].cpu())) and np.array_equal(cVo, inputs.to_numpy(cVs[layer].cpu()))
        assert np.array_equal(cpo, cpos.cpu().numpy())          # the same positions at every layer
        ref, _ = oracle.attend_ragged(inputs.to_numpy(Q), q_off, q_pos0, dh ** -0.5, cKo, cVo, cpo, nug_off, ks,
                                      inputs.to_numpy(lK), inputs.to_numpy(lV), q_off[:-1], tq, q_pos0)
        assert np.max(np.abs(O.float().cpu().numpy().astype(np.float64) - ref)) <= 2e-2
