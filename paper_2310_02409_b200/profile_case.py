"""A small, self-ending run of the hot path for profilers (timing lives in bench.py): R layer instances of a
workload, compressed once, then a few decode steps launched eagerly (no CUDA graph), interleaved over the
instances so that every attend launch reads its keys from HBM; optionally the workload's query block, the
two-layer Scorer, the multi-layer gather, or a one-shot query by index.

    python -m paper_2310_02409_b200.profile_case --instances 4 --decode-steps 4
"""
from __future__ import annotations

import argparse

import torch

from . import api, build, inputs
from .workloads import CompressDecode


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c2_llama7b_decode")
    ap.add_argument("--instances", type=int, default=4)
    ap.add_argument("--decode-steps", type=int, default=4)
    ap.add_argument("--ratio", type=int, default=10)
    ap.add_argument("--target-blocks", type=int, default=0)
    ap.add_argument("--dense-balance", type=int, default=0, help="0 auto, 1 always, 2 never")
    ap.add_argument("--scorer-mlp", type=int, default=0, metavar="ROWS",
                    help="instead: the two-layer Scorer (d -> d -> 1, ReLU) of the workload's width over ROWS tokens, timed")
    ap.add_argument("--gather-layers", type=int, default=0, metavar="L",
                    help="instead: one selection shared by L layers of the workload's shape, gathered by one call and by L calls, timed")
    ap.add_argument("--indexed", action="store_true",
                    help="instead: a one-shot query by index (dodo_attend_indexed), 8 documents of 878 tokens at ratio 10, 17 query tokens")
    ap.add_argument("--pool", action="store_true",
                    help="instead: mean pooling of the workload's K/V at the ratio (dodo_pool_kv), a few launches")
    ap.add_argument("--select", action="store_true",
                    help="instead: the stand-alone TopK (dodo_select) over Gaussian scores of the workload's lengths, a few launches")
    ap.add_argument("--query-block-reps", type=int, default=0,
                    help="also run the workload's query block this many times and report its rate")
    args = ap.parse_args()
    build.build()
    dodo = api.Dodo(0)
    if args.target_blocks:
        dodo.set_tuning(api.TUNE_ATTEND_TARGET_BLOCKS, args.target_blocks)
    if args.dense_balance:
        dodo.set_tuning(api.TUNE_DENSE_BALANCE, args.dense_balance)
    wl = inputs.WORKLOADS[args.workload]
    if args.scorer_mlp:
        scorer_mlp(dodo, wl.d, args.scorer_mlp)
        return
    if args.gather_layers:
        gather_layers(dodo, wl, args.ratio, args.gather_layers)
        return
    if args.indexed:
        one_shot_indexed(dodo, wl)
        return
    if args.pool or args.select:
        pool_or_select(dodo, wl, args.ratio, args.instances, args.pool)
        return
    if args.workload == "c5_ragged_serving":
        ragged_serving(dodo, wl, args.ratio)
        return
    insts = [CompressDecode(dodo, wl, args.ratio, ("profile", i), steps=args.decode_steps)
             for i in range(args.instances)]
    for it in insts:
        it.compress()
    for s in range(args.decode_steps):
        for it in insts:
            it.decode_step(s)
    if args.query_block_reps and wl.tq_dense:
        for it in insts:
            it.query_block()
        torch.cuda.synchronize()
        # as a CUDA graph, so that the host side of the calls (five tensor maps each) does not bound the rate
        side, gr = torch.cuda.Stream(), torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr, stream=side):
            for _ in range(args.query_block_reps):
                for it in insts:
                    it.query_block()
        gr.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        gr.replay()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / (args.query_block_reps * len(insts))
        fl = insts[0].flops_query_block()
        print(f"query block: {ms * 1e3:.1f} us per launch, {fl / 1e9:.2f} GFLOP, {fl / ms / 1e9:.1f} TFLOP/s")
    torch.cuda.synchronize()
    assert dodo.device_status() == 0
    print(f"ok: {args.instances} instances, {args.decode_steps} decode steps, "
          f"{sum(i.device_bytes() for i in insts) / 1e9:.2f} GB on the device")


def pool_or_select(dodo, wl, r, instances, pool, reps=3):
    """dodo_pool_kv (or dodo_select) on `instances` seeded layer instances of the workload's shape, in rotation."""
    import numpy as np
    insts = [CompressDecode(dodo, wl, r, ("profile", "ps", i), steps=1) for i in range(instances)]
    for _ in range(reps):
        for it in insts:
            if pool:
                it.cache_len[:] = 0
                dodo.pool_kv(it.K, it.V, it.seq_off, r, it.pos_base, it.cacheK, it.cacheV, it.cache_pos, it.cache_off, it.cache_len)
            else:
                dodo.select(it.scores.normal_(), it.seq_off, it.nug_off, 0, it.idx)
    torch.cuda.synchronize()
    assert dodo.device_status() == 0
    print(f"ok: {'pool_kv' if pool else 'select'} x {reps} on {instances} instances of {wl.name}, ratio {r}")


def scorer_mlp(dodo, d, rows, reps=5):
    """dodo_score_mlp on seeded inputs of width d = dh over `rows` tokens: device time and tensor rate."""
    bf = torch.bfloat16
    X = inputs.randn((rows, d), "profile", "mlpX", dtype=bf, device="cuda")
    W1 = inputs.randn((d, d), "profile", "mlpW1", std=d ** -0.5, dtype=bf, device="cuda")
    b1 = inputs.randn((d,), "profile", "mlpb1", std=0.5, device="cuda")
    w2 = inputs.randn((d,), "profile", "mlpw2", std=d ** -0.5, dtype=bf, device="cuda")
    scores = torch.zeros(rows, device="cuda")
    ws = torch.empty(dodo.score_mlp_workspace_bytes(rows, d), dtype=torch.uint8, device="cuda")
    run = lambda: dodo.score_mlp(X, W1, b1, w2, 0.0, api.ACT_RELU, [0, rows], scores, ws)
    run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        run()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / reps
    fl = 2.0 * rows * d * d
    print(f"two-layer Scorer: {rows} tokens, d = dh = {d}: {ms * 1e3:.1f} us per call, {fl / 1e9:.1f} GFLOP, {fl / ms / 1e9:.1f} TFLOP/s")
    assert dodo.device_status() == 0


def gather_layers(dodo, wl, r, L, reps=5):
    """dodo_gather_kv_layers against L calls of dodo_gather_kv on seeded K/V of the workload's shape, one shared
    selection (random positions, ascending per sequence): device times from CUDA-graph replays, results compared."""
    import numpy as np
    n = np.asarray(wl.n_ctx, dtype=np.int32)
    B, H, dh = len(n), wl.H, wl.dh
    seq_off = inputs.offsets(n)
    k = np.asarray([dodo.num_nuggets(int(x), r) for x in n], dtype=np.int32)
    nug_off = inputs.offsets(k)
    N, Kt = int(seq_off[-1]), int(nug_off[-1])
    bf = torch.bfloat16
    Ks = [inputs.randn((N, H, dh), "profile", "gl", l, "K", dtype=bf, device="cuda") for l in range(L)]
    Vs = [inputs.randn((N, H, dh), "profile", "gl", l, "V", dtype=bf, device="cuda") for l in range(L)]
    cKs = [torch.zeros((Kt, H, dh), dtype=bf, device="cuda") for _ in range(L)]
    cVs = [torch.zeros((Kt, H, dh), dtype=bf, device="cuda") for _ in range(L)]
    cpos = torch.zeros(Kt, dtype=torch.int32, device="cuda")
    rs = np.random.RandomState(inputs.seed_for(("profile", "gl", "idx")) % 2 ** 32)
    idx = np.concatenate([np.sort(rs.choice(int(n[b]), int(k[b]), replace=False)) for b in range(B)]).astype(np.int32)
    idx = torch.from_numpy(idx).cuda()
    pos_base = np.zeros(B, np.int32)

    def one_call():
        dodo.gather_kv_layers(Ks, Vs, seq_off, idx, nug_off, pos_base, cKs, cVs, cpos, nug_off, np.zeros(B, np.int32))

    def per_layer():
        for l in range(L):
            dodo.gather_kv(Ks[l], Vs[l], seq_off, idx, nug_off, pos_base, cKs[l], cVs[l], cpos, nug_off, np.zeros(B, np.int32))

    nbytes = L * Kt * 4 * H * dh * 2 + Kt * 8
    for name, fn in (("one call", one_call), ("a call per layer", per_layer)):
        fn()
        torch.cuda.synchronize()
        side, gr = torch.cuda.Stream(), torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr, stream=side):
            fn()
        gr.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            gr.replay()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        print(f"gather of {Kt} nuggets x {L} layers, {name}: {ms * 1e3:.1f} us, {nbytes / 1e6:.0f} MB, {nbytes / ms / 1e6:.0f} GB/s")
        if name == "one call":
            ref = [c.clone() for c in cKs + cVs]
            for c in cKs + cVs:
                c.zero_()
    assert all(torch.equal(a, b) for a, b in zip(ref, cKs + cVs))
    assert dodo.device_status() == 0


def ragged_serving(dodo, wl, r):
    """The ragged serving layer at full size: compress all contexts, then every decode step with its appends, the
    decode loop as one CUDA graph.  Prints device times and rates."""
    from .workloads import RaggedServing
    rs = RaggedServing(dodo, wl.n_ctx, wl.d, wl.H, wl.dh, r, wl.decode_steps, ("profile", "c5"))
    rs.compress_context()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    rs.compress_context()
    e1.record()
    torch.cuda.synchronize()
    ms_c = e0.elapsed_time(e1)
    e = rs.X.element_size()
    by_c = int(rs.n.sum()) * (rs.d * e + 4) + int(rs.k0.sum()) * (4 * rs.H * rs.dh * e + 8)
    print(f"compress: {ms_c:.3f} ms for {int(rs.n.sum())} tokens -> {int(rs.k0.sum())} nuggets, {by_c / ms_c / 1e6:.0f} GB/s; "
          f"imbalance max k / mean k = {rs.k0.max() / rs.k0.mean():.2f}")
    keys = []

    def decode():
        rs.compress_context()      # (host tables back to the state after the context; cheap beside 256 steps)
        for s in range(rs.steps):
            keys.append(rs.keys_per_step(s))
            rs.decode_step(s)

    decode()
    torch.cuda.synchronize()
    total_keys = sum(keys)
    del keys[:]
    side, gr = torch.cuda.Stream(), torch.cuda.CUDAGraph()
    with torch.cuda.graph(gr, stream=side):
        decode()
    gr.replay()
    torch.cuda.synchronize()
    e0.record()
    gr.replay()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) - ms_c
    by = 2 * total_keys * rs.H * rs.dh * e
    print(f"decode: {rs.steps} steps (appends at 128, 192, 256) in {ms:.2f} ms = {ms * 1e3 / rs.steps:.1f} us per step, "
          f"{by / rs.steps / 1e6:.0f} MB of K/V per step, {by / ms / 1e6:.0f} GB/s, {rs.B * rs.steps / ms * 1e3:.0f} tokens/s per layer")
    torch.cuda.synchronize()
    assert dodo.device_status() == 0


def one_shot_indexed(dodo, wl, B=8, n=878, r=10, tq=17, instances=6):
    """dodo_attend_indexed once per instance: tq query tokens over the k selected rows of an n-token document."""
    import numpy as np
    H, dh, k = wl.H, wl.dh, -(-n // r)
    bf = torch.bfloat16
    seq_off, nug_off, q_off = inputs.offsets([n] * B), inputs.offsets([k] * B), inputs.offsets([tq] * B)
    ws = torch.empty(dodo.attend_workspace_bytes(dh), dtype=torch.uint8, device="cuda")
    for i in range(instances):
        g = lambda shape, nm: inputs.randn(shape, "profile", "indexed", i, nm, dtype=bf, device="cuda")
        K, V, Q, lK, lV = g((B * n, H, dh), "K"), g((B * n, H, dh), "V"), g((B * tq, H, dh), "Q"), g((B * tq, H, dh), "lK"), g((B * tq, H, dh), "lV")
        rs = np.random.RandomState(i)
        idx = torch.from_numpy(np.concatenate([np.sort(rs.choice(n, k, replace=False)) for _ in range(B)]).astype(np.int32)).cuda()
        O = torch.zeros_like(Q)
        dodo.attend_indexed(Q, q_off, np.full(B, n, np.int32), dh ** -0.5, K, V, seq_off, idx, nug_off, np.zeros(B, np.int32), lK, lV,
                            np.arange(B, dtype=np.int32) * tq, np.full(B, tq, np.int32), np.full(B, n, np.int32), O, None, ws)
    torch.cuda.synchronize()
    assert dodo.device_status() == 0
    print(f"ok: {instances} one-shot queries by index, {B} documents of {n} tokens, {k} selected, {tq} query tokens")


if __name__ == "__main__":
    main()
