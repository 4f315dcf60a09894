"""Benchmark of the compressed-context hot path on B200.

Headline workload: the LLaMA-7B-shaped single-layer decode configuration (bf16, batch 8, d = 4096,
32 heads x 128, context 2048 -> 205 nuggets per sequence at ratio 10, 128 decode steps, each attending
the nuggets plus a 64-token local window).  One benchmark step is one pass of the whole path:
score+select and gather for every sequence, then all 128 decode steps.  A single layer's K/V
(35 MB) would sit in the 126 MB L2, so R independent instances of the layer are interleaved step
by step; every attend launch then reads its keys from HBM, as it would in a multi-layer model.

Prints ONE JSON line.  Beside the headline it carries `roofline` (the dominant kernel against the
measured HBM peak), `e2e` (the same metric through the host-buffer entry point), `cpu_baseline` (the fp64
oracle on the host cores) and, at one GPU, `configs`: the other workload configurations at full size, one
layer each, with the compress step, the dense query block and the decode launches timed separately
(CUDA-graph replays, one CUDA-event pair per replay, 20 replays: mean, median, best) and each against its
own roofline.  `--impl reference` times the fp64 CPU oracle on the host cores instead.

`--gpus N` with N > 1 runs N independent replicas, one process per GPU; started without a launcher it
re-executes itself under torch.distributed.run.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

# DRAM bytes of one attend launch on this workload from an ncu capture (dram__bytes_read.sum +
# dram__bytes_write.sum, see profiles/attend_kernel_c2_decode.md), valid only for the kernel source
# it was taken on: reported as null once csrc/attend.cu has changed since.
ATTEND_TRAFFIC = {"bytes": 35381504, "attend_cu_sha1": "40189a9563c3a4cd124c98e0661e5ff706ec8f9b"}

METRIC = "nugget-attention decode tokens/s"
UNIT = "tokens/s"
WORKLOAD = "c2_llama7b_decode"
RATIO = 10


def workload_config(wl, nuggets_per_seq: int, instances: int, world: int) -> dict:
    """The `config` object of the JSON line: the workload as both arms define it (the reference arm computes a
    stated sample of it and scales).  Same keys and values from either arm."""
    row = wl.H * wl.dh * 2
    kv_mb = instances * 2 * wl.B * (nuggets_per_seq + wl.local) * row / 1e6
    return {"workload": WORKLOAD, "batch": wl.B, "context": wl.n_ctx[0], "ratio": RATIO,
            "nuggets_per_seq": nuggets_per_seq, "decode_steps": wl.decode_steps, "local_window": wl.local,
            "heads": wl.H, "head_dim": wl.dh, "d": wl.d, "instances": instances,
            "l2": f"cold: {instances} independent layer instances interleaved per decode step "
                  f"({kv_mb:.0f} MB of K/V between reuses, L2 is 126 MB)",
            "parallelism": f"replicas x{world}, no collective"}


def attend_traffic():
    import hashlib
    src = ROOT / "paper_2310_02409_b200" / "csrc" / "attend.cu"
    try:
        if hashlib.sha1(src.read_bytes()).hexdigest() == ATTEND_TRAFFIC["attend_cu_sha1"]:
            return ATTEND_TRAFFIC["bytes"]
    except OSError:
        pass
    return None


def measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            return json.loads(p.read_text()), "measured"
        except Exception:
            pass
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}, "fallback"


class ClockSampler:
    """nvidia-smi clock/throttle samples taken while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        sel = str(device_index)
        try:
            import torch
            sel = "GPU-" + str(torch.cuda.get_device_properties(device_index).uuid)
        except Exception:
            pass
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", sel, f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=self.tmp, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
        self.tmp.flush()
        rows = [l.strip().split(", ") for l in Path(self.tmp.name).read_text().splitlines() if l.strip()]
        try:
            os.unlink(self.tmp.name)
        except OSError:
            pass
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0])); smax.append(float(r[1]))
            except ValueError:
                continue
            for name, v in zip(names, r[3:7]):
                if v.strip() == "Active":
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
# CPU oracle legs
# ------------------------------------------------------------------------------------------------

def oracle_pass(host, decode_steps_sample: int):
    """One pass of the path by the CPU oracle on host copies of an instance's inputs.

    Compression runs in full; only `decode_steps_sample` evenly spaced decode steps are computed and
    their time is scaled to all steps.  Returns (estimated seconds for the full pass, seconds spent).
    """
    import numpy as np
    import oracle
    n, B, steps, L = host["n"], host["B"], host["steps"], host["local"]
    t0 = time.perf_counter()
    s64 = oracle.score(host["X"], host["w"], 0.0)
    s32 = s64.astype(np.float32)
    idx = oracle.select_ragged(s32, host["seq_off"], host["nug_off"], 0)
    cK, cV = np.zeros_like(host["cacheK"]), np.zeros_like(host["cacheV"])
    cpos = np.zeros(cK.shape[0], np.int32)
    clen = oracle.gather_ragged(host["K"], host["V"], host["seq_off"], idx, host["nug_off"], np.zeros(B, np.int32),
                                cK, cV, cpos, host["cache_off"], [0] * B)
    t1 = time.perf_counter()
    pick = np.unique(np.linspace(0, steps - 1, decode_steps_sample).astype(int))
    q_off = np.arange(B + 1, dtype=np.int32)
    for s in pick:
        base = np.arange(B, dtype=np.int32) * host["loc_cap"]
        oracle.attend_ragged(host["Qd"][s], q_off, n + L + s, host["scale"], cK, cV, cpos, host["cache_off"], clen,
                             host["locK"], host["locV"], base + s + 1, np.full(B, L, np.int32), n + s + 1)
    t2 = time.perf_counter()
    est = (t1 - t0) + (t2 - t1) * steps / len(pick)
    return est, t2 - t0, len(pick)


def host_copy(inst):
    from paper_2310_02409_b200 import inputs
    wl = inst.wl
    return {"X": inputs.to_numpy(inst.X), "w": inputs.to_numpy(inst.w), "K": inputs.to_numpy(inst.K),
            "V": inputs.to_numpy(inst.V), "locK": inputs.to_numpy(inst.locK), "locV": inputs.to_numpy(inst.locV),
            "Qd": inputs.to_numpy(inst.Qd), "cacheK": inputs.to_numpy(inst.cacheK), "cacheV": inputs.to_numpy(inst.cacheV),
            "seq_off": inst.seq_off, "nug_off": inst.nug_off, "cache_off": inst.cache_off, "n": inst.n.copy(),
            "B": wl.B, "steps": inst.steps, "local": wl.local, "loc_cap": inst.loc_cap, "scale": inst.sm_scale}


def host_inputs_cpu(wl, r):
    """The same instance layout drawn on the CPU (for the reference arm, which has no GPU work)."""
    import numpy as np
    import oracle
    from paper_2310_02409_b200 import inputs
    B, H, dh, d, steps = wl.B, wl.H, wl.dh, wl.d, wl.decode_steps
    n = np.asarray(wl.n_ctx, np.int32)
    k = np.asarray([oracle.num_nuggets(int(x), r) for x in n], np.int32)
    N, Kt = int(n.sum()), int(k.sum())
    loc_cap = wl.local + steps
    tag = ("bench-ref",)
    g = lambda shape, name, std=1.0: inputs.to_numpy(inputs.randn(shape, *tag, name, std=std, dtype=wl.dtype))
    return {"X": g((N, d), "X"), "w": g((d,), "w", d ** -0.5), "K": g((N, H, dh), "K"), "V": g((N, H, dh), "V"),
            "locK": g((B * loc_cap, H, dh), "locK"), "locV": g((B * loc_cap, H, dh), "locV"),
            "Qd": g((steps, B, H, dh), "Qd"), "cacheK": np.zeros((Kt, H, dh), np.uint16),
            "cacheV": np.zeros((Kt, H, dh), np.uint16), "seq_off": inputs.offsets(n), "nug_off": inputs.offsets(k),
            "cache_off": inputs.offsets(k), "n": n, "B": B, "steps": steps, "local": wl.local, "loc_cap": loc_cap,
            "scale": dh ** -0.5}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2310_02409_b200 import inputs
    wl = inputs.WORKLOADS[WORKLOAD]
    host = host_inputs_cpu(wl, RATIO)
    sample_steps = 16
    for _ in range(min(args.warmup, 1)):
        oracle_pass(host, sample_steps)
    t0 = time.perf_counter()
    est_total = 0.0
    for _ in range(args.steps):
        est, _, used = oracle_pass(host, sample_steps)
        est_total += est
    wall = time.perf_counter() - t0
    tokens = wl.B * wl.decode_steps * args.steps
    value = tokens / est_total
    sample = (f"per step: one of the workload's {args.instances} identical layer instances (tokens/s does not depend on "
              f"their number): full score+select+gather of {wl.B}x{wl.n_ctx[0]} tokens, {used} of {wl.decode_steps} decode "
              f"steps computed and scaled to all of them; {args.steps} steps, {wall:.1f} s of CPU work")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * est_total / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(wl, oracle.num_nuggets(wl.n_ctx[0], RATIO), args.instances,
                                      int(os.environ.get("WORLD_SIZE", "1"))),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
# CUDA arm
# ------------------------------------------------------------------------------------------------

def max_over_ranks(values, world: int, device):
    """Every rank's device-measured times -> their maximum over the ranks (what the job really took)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(values, dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def job_throughput(units_per_rank_per_step: int, steps: int, world: int, max_ms: float) -> float:
    """Weak scaling, no collective on the data path: every rank does the same work on its own replica;
    the job's throughput is all ranks' units over the slowest rank's time."""
    return world * units_per_rank_per_step * steps / (max_ms * 1e-3)


def check_world(gpus_asked: int, world: int) -> None:
    """`--gpus N` and the number of ranks actually running must agree: a job that was asked for N GPUs never
    reports fewer."""
    if gpus_asked != world:
        raise SystemExit(f"bench.py: --gpus {gpus_asked} but {world} rank(s) are running (WORLD_SIZE); "
                         "start it as `python bench.py --gpus N` or under torch.distributed.run with N ranks")


def launcher_command(gpus: int, argv: list[str], port: int) -> list[str]:
    """The command that runs this script as `gpus` ranks on this node, one per GPU."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(gpus),
            "--master-addr", "127.0.0.1", "--master-port", str(port), str(Path(__file__).resolve()), *argv]


def respawn_under_launcher(gpus: int, argv: list[str]) -> int:
    """`python bench.py --gpus N` without a launcher: run the same command line as N ranks."""
    import socket
    with socket.socket() as so:
        so.bind(("127.0.0.1", 0))
        port = so.getsockname()[1]
    return subprocess.call(launcher_command(gpus, argv, port))


def spread(ms_list, per: float = 1.0) -> dict:
    """mean / median / best of per-replay device times (ms), each divided by `per`, in microseconds."""
    us = sorted(1e3 * m / per for m in ms_list)
    return {"mean": sum(us) / len(us), "median": us[len(us) // 2] if len(us) % 2 else 0.5 * (us[len(us) // 2 - 1] + us[len(us) // 2]),
            "best": us[0], "reps": len(us)}


def time_graph(fn, reps: int):
    """Capture fn() (library calls on the current stream) as one CUDA graph; three warm-up replays, then `reps`
    replays each bracketed by its own CUDA-event pair.  Returns the per-replay times in ms."""
    import torch
    side, gr = torch.cuda.Stream(), torch.cuda.CUDAGraph()
    with torch.cuda.graph(gr, stream=side):
        fn()
    for _ in range(3):
        gr.replay()
    torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
    for a, b in ev:
        a.record(); gr.replay(); b.record()
    torch.cuda.synchronize()
    return [a.elapsed_time(b) for a, b in ev]


def roofline_of(bound: str, work_per_launch: float, us: dict, peaks: dict, peak_kind: str) -> dict:
    """achieved = algorithmic bytes (or flops) per launch / mean device time per launch, against the measured peak:
    the copy bandwidth for an HBM-bound part, the burst bf16 rate (a kernel timed alone) for a contraction."""
    if bound == "hbm":
        achieved, peak, unit = work_per_launch / (us["mean"] * 1e-6) / 1e9, peaks["hbm_gbs"], "GB/s"
        note = f"of {peak_kind} copy bandwidth"
    else:
        achieved, peak, unit = work_per_launch / (us["mean"] * 1e-6) / 1e12, peaks["bf16_tflops"], "TFLOP/s"
        note = f"of {peak_kind} bf16 burst rate (kernel timed alone)"
    return {"bound": bound, "achieved": achieved, "peak": peak, "unit": unit, "frac": achieved / peak,
            "frac_best": achieved * us["mean"] / us["best"] / peak, "peak_kind": note}


def config_compress_decode(dodo, wl, r: int, tag, peaks, peak_kind, reps: int) -> dict:
    """One layer of a CompressDecode workload at full size: the compress step (fused score+select, gather), the
    dense query block and the decode launches, each timed on its own.  Enough independent instances of the
    layer are rotated that a decode round's K/V exceed twice the L2."""
    import torch
    from paper_2310_02409_b200.workloads import CompressDecode
    probe_bytes = 2 * (sum(-(-n // r) for n in wl.n_ctx) + wl.B * (wl.local + wl.tq_dense)) * wl.H * wl.dh * 2
    R = max(1, min(10, -(-256_000_000 // probe_bytes)))
    insts = [CompressDecode(dodo, wl, r, (*tag, i)) for i in range(R)]
    steps = insts[0].steps
    for it in insts:
        it.compress()
        if wl.tq_dense:
            it.query_block()
    for s in range(steps):
        for it in insts:
            it.decode_step(s)
    torch.cuda.synchronize()
    rec = {"ratio": r, "nuggets_per_seq": int(insts[0].k[0]), "instances": R, "layers_timed": 1,
           "l2": f"cold: {R} layer instance(s) in rotation, {R * probe_bytes / 1e6:.0f} MB of K/V between reuses"}

    def compress():
        for it in insts:
            it.compress()
    us = spread(time_graph(compress, reps), R)
    by = insts[0].bytes_score() + insts[0].bytes_gather()
    rec["compress"] = {"us_per_instance": us, "bytes": by, "roofline": roofline_of("hbm", by, us, peaks, peak_kind)}
    if wl.tq_dense:
        def block():
            for it in insts:
                it.query_block()
        us = spread(time_graph(block, reps), R)
        fl = insts[0].flops_query_block()
        rec["query_block"] = {"queries": wl.tq_dense, "us_per_launch": us, "flops": fl,
                              "roofline": roofline_of("tensor", fl, us, peaks, peak_kind)}

    def decode():
        for s in range(steps):
            for it in insts:
                it.decode_step(s)
    ms = time_graph(decode, reps)
    us = spread(ms, R * steps)
    by = sum(insts[0].bytes_decode_step(s) for s in range(steps)) / steps
    rec["decode"] = {"steps": steps, "us_per_launch": us, "bytes_per_launch": by,
                     "tokens_per_s_per_layer": wl.B * steps * R / (sum(ms) / len(ms) * 1e-3),
                     "roofline": roofline_of("hbm", by, us, peaks, peak_kind)}
    assert dodo.device_status() == 0
    return rec


def config_ragged_serving(dodo, wl, r: int, peaks, peak_kind, reps: int) -> dict:
    """One layer of the ragged serving workload at full size: compression of all contexts, then every decode
    step with its segment appends as one CUDA graph."""
    import torch
    from paper_2310_02409_b200.workloads import RaggedServing
    rs = RaggedServing(dodo, wl.n_ctx, wl.d, wl.H, wl.dh, r, wl.decode_steps, ("bench", "c5"))
    e = rs.X.element_size()
    row = rs.H * rs.dh * e
    rs.compress_context()
    keys = []
    for s in range(rs.steps):
        keys.append(rs.keys_per_step(s))
        rs.decode_step(s)
    torch.cuda.synchronize()
    rec = {"ratio": r, "sequences": rs.B, "tokens": int(rs.n.sum()), "nuggets": int(rs.k0.sum()),
           "imbalance_max_k_over_mean_k": float(rs.k0.max() / rs.k0.mean()), "layers_timed": 1,
           "l2": "cold by size: every launch moves far more than the 126 MB L2"}
    us = spread(time_graph(rs.compress_context, reps))
    by = int(rs.n.sum()) * (rs.d * e + 4) + int(rs.k0.sum()) * (4 * row + 8)
    rec["compress"] = {"us": us, "bytes": by, "roofline": roofline_of("hbm", by, us, peaks, peak_kind)}

    def decode():
        rs.rewind()
        for s in range(rs.steps):
            rs.decode_step(s)
    ms = time_graph(decode, reps)
    us = spread(ms, rs.steps)
    by = (2 * sum(keys) * row + 2 * rs.B * row * rs.steps) / rs.steps
    rec["decode"] = {"steps": rs.steps, "appends_at_steps": [s + 1 for s in range(rs.steps) if (s + 1) % rs.S == 0 and s + 1 >= 2 * rs.S],
                     "us_per_step": us, "bytes_per_step": by,
                     "tokens_per_s_per_layer": rs.B * rs.steps / (sum(ms) / len(ms) * 1e-3),
                     "note": "a step is one attend launch over all 64 sequences; the three append steps add staging copies, a "
                             "fused score+select and a gather, inside the timed graph",
                     "roofline": roofline_of("hbm", by, us, peaks, peak_kind)}
    assert dodo.device_status() == 0
    return rec


def config_scorer_mlp(dodo, rows: int, d: int, peaks, peak_kind, reps: int) -> dict:
    """The two-layer Scorer (d -> d -> 1, ReLU) over `rows` tokens."""
    import torch
    from paper_2310_02409_b200 import api, inputs
    bf = torch.bfloat16
    X = inputs.randn((rows, d), "bench", "mlpX", dtype=bf, device="cuda")
    W1 = inputs.randn((d, d), "bench", "mlpW1", std=d ** -0.5, dtype=bf, device="cuda")
    b1 = inputs.randn((d,), "bench", "mlpb1", std=0.5, device="cuda")
    w2 = inputs.randn((d,), "bench", "mlpw2", std=d ** -0.5, dtype=bf, device="cuda")
    scores = torch.zeros(rows, device="cuda")
    ws = torch.empty(dodo.score_mlp_workspace_bytes(rows, d), dtype=torch.uint8, device="cuda")
    run = lambda: dodo.score_mlp(X, W1, b1, w2, 0.0, api.ACT_RELU, [0, rows], scores, ws)
    run()
    torch.cuda.synchronize()
    us = spread(time_graph(run, reps))
    fl = 2.0 * rows * d * d
    assert dodo.device_status() == 0
    return {"tokens": rows, "d": d, "hidden": d, "activation": "relu", "us_per_call": us, "flops": fl,
            "l2": "X (134 MB) exceeds the L2; W1 (34 MB) is meant to stay in it",
            "roofline": roofline_of("tensor", fl, us, peaks, peak_kind)}


def config_mlp_compress(dodo, wl, r: int, peaks, peak_kind, reps: int) -> dict:
    """The compress step with the two-layer Scorer (d -> d -> 1, ReLU) in place of the linear one: tensor-core pass,
    reduction fused with the TopK, gather.  The first layer's 2 d^2 flop per token dominate."""
    import torch
    from paper_2310_02409_b200 import api, inputs
    from paper_2310_02409_b200.workloads import CompressDecode
    insts = [CompressDecode(dodo, wl, r, ("bench", "mlpc", i), steps=1) for i in range(2)]
    d = wl.d
    W1 = inputs.randn((d, d), "bench", "mlpc", "W1", std=d ** -0.5, dtype=torch.bfloat16, device="cuda")
    b1 = inputs.randn((d,), "bench", "mlpc", "b1", std=0.5, device="cuda")
    w2 = inputs.randn((d,), "bench", "mlpc", "w2", std=d ** -0.5, dtype=torch.bfloat16, device="cuda")
    rows = int(insts[0].seq_off[-1])
    ws = torch.empty(dodo.score_mlp_workspace_bytes(rows, d), dtype=torch.uint8, device="cuda")

    def run(it):
        it.cache_len[:] = 0
        dodo.score_mlp_select(it.X, W1, b1, w2, 0.0, api.ACT_RELU, it.seq_off, it.nug_off, 0, it.scores, it.idx, ws)
        dodo.gather_kv(it.K, it.V, it.seq_off, it.idx, it.nug_off, it.pos_base, it.cacheK, it.cacheV, it.cache_pos, it.cache_off,
                       it.cache_len)
    for it in insts:
        run(it)
    torch.cuda.synchronize()
    us = spread(time_graph(lambda: [run(it) for it in insts], reps), len(insts))
    fl = 2.0 * rows * d * d
    assert dodo.device_status() == 0
    return {"workload_shape": wl.name, "ratio": r, "tokens": rows, "hidden": d, "activation": "relu", "us_per_instance": us, "flops": fl,
            "launches_per_instance": 3, "roofline": roofline_of("tensor", fl, us, peaks, peak_kind)}


def config_mean_pool(dodo, wl, r: int, peaks, peak_kind, reps: int) -> dict:
    """The comparison system's compression (Sec. 5.1): K/V of every even chunk of r tokens pooled by their mean into
    one cache row.  Reads every K and V row once; instances rotate so that they come from HBM."""
    import numpy as np
    import torch
    from paper_2310_02409_b200 import inputs
    B, H, dh = wl.B, wl.H, wl.dh
    n = np.asarray(wl.n_ctx, np.int32)
    seq_off = inputs.offsets(n)
    ks = np.asarray([dodo.num_nuggets(int(x), r) for x in n], np.int32)
    cache_off = inputs.offsets(ks)
    N, Kt = int(seq_off[-1]), int(cache_off[-1])
    row = H * dh * 2
    inst = max(2, min(8, -(-256_000_000 // (2 * N * row))))
    S = [dict(K=inputs.randn((N, H, dh), "bench", "pool", i, "K", dtype=torch.bfloat16, device="cuda"),
              V=inputs.randn((N, H, dh), "bench", "pool", i, "V", dtype=torch.bfloat16, device="cuda"),
              cK=torch.zeros((Kt, H, dh), dtype=torch.bfloat16, device="cuda"), cV=torch.zeros((Kt, H, dh), dtype=torch.bfloat16, device="cuda"),
              cp=torch.zeros(Kt, dtype=torch.int32, device="cuda")) for i in range(inst)]

    def run(s):
        dodo.pool_kv(s["K"], s["V"], seq_off, r, np.zeros(B, np.int32), s["cK"], s["cV"], s["cp"], cache_off, np.zeros(B, np.int32))
    for s in S:
        run(s)
    torch.cuda.synchronize()
    us = spread(time_graph(lambda: [run(s) for s in S], reps), inst)
    by = 2 * N * row + 2 * Kt * row + 4 * Kt
    assert dodo.device_status() == 0
    return {"workload_shape": wl.name, "ratio": r, "tokens": N, "pooled_rows": Kt, "instances": inst, "us_per_instance": us, "bytes": by,
            "roofline": roofline_of("hbm", by, us, peaks, peak_kind)}


def config_one_shot(dodo, name: str, B: int, H: int, n: int, r: int, tq: int, reps: int) -> dict:
    """A one-shot query over a compressed document (compressor mode, Eq. 13): tq query tokens attend the k selected
    tokens of an n-token document and, causally, themselves.  Two routes to the same bits: gather the selected rows
    into a nugget cache, then attend (two launches); or attend straight over the uncompressed K/V by index (one
    launch, no cache).  Random ascending indices stand in for a selection; instances rotate so that K/V come from HBM."""
    import numpy as np
    import torch
    from paper_2310_02409_b200 import api, inputs
    dh, k = 128, -(-n // r)
    inst = max(2, min(16, -(-256_000_000 // (2 * B * n * H * dh * 2))))
    seq_off, nug_off, q_off = inputs.offsets([n] * B), inputs.offsets([k] * B), inputs.offsets([tq] * B)
    loc_off = np.arange(B, dtype=np.int32) * tq
    pb, llen, lp0, qp0 = np.zeros(B, np.int32), np.full(B, tq, np.int32), np.full(B, n, np.int32), np.full(B, n, np.int32)
    bf = torch.bfloat16
    S = []
    for i in range(inst):
        g = lambda shape, nm: inputs.randn(shape, "bench", name, i, nm, dtype=bf, device="cuda")
        rs = np.random.RandomState(inputs.seed_for("bench", name, i) % 2 ** 32)
        idx = np.concatenate([np.sort(rs.choice(n, k, replace=False)) for _ in range(B)]).astype(np.int32)
        S.append(dict(K=g((B * n, H, dh), "K"), V=g((B * n, H, dh), "V"), Q=g((B * tq, H, dh), "Q"), lK=g((B * tq, H, dh), "lK"),
                      lV=g((B * tq, H, dh), "lV"), idx=torch.from_numpy(idx).cuda(),
                      cK=torch.zeros((B * k, H, dh), dtype=bf, device="cuda"), cV=torch.zeros((B * k, H, dh), dtype=bf, device="cuda"),
                      cp=torch.zeros(B * k, dtype=torch.int32, device="cuda"), O=torch.zeros((B * tq, H, dh), dtype=bf, device="cuda"),
                      O2=torch.zeros((B * tq, H, dh), dtype=bf, device="cuda")))
    ws = torch.empty(dodo.attend_workspace_bytes(dh), dtype=torch.uint8, device="cuda")

    def through_cache(s):
        clen = np.zeros(B, np.int32)
        dodo.gather_kv(s["K"], s["V"], seq_off, s["idx"], nug_off, pb, s["cK"], s["cV"], s["cp"], nug_off, clen)
        dodo.attend(s["Q"], q_off, qp0, dh ** -0.5, s["cK"], s["cV"], s["cp"], nug_off, clen, s["lK"], s["lV"], loc_off, llen, lp0,
                    s["O"], None, ws)

    def by_index(s):
        dodo.attend_indexed(s["Q"], q_off, qp0, dh ** -0.5, s["K"], s["V"], seq_off, s["idx"], nug_off, pb, s["lK"], s["lV"],
                            loc_off, llen, lp0, s["O2"], None, ws)

    # both routes on the tensor-core kernel (a block of 17 queries would otherwise take the streaming kernel in dodo_attend)
    dodo.set_tuning(api.TUNE_DENSE_MIN_QUERIES, 1)
    try:
        for s in S:
            through_cache(s); by_index(s)
        torch.cuda.synchronize()
        same = all(torch.equal(s["O"], s["O2"]) for s in S)
        us_c = spread(time_graph(lambda: [through_cache(s) for s in S], reps), inst)
        us_i = spread(time_graph(lambda: [by_index(s) for s in S], reps), inst)
    finally:
        dodo.set_tuning(api.TUNE_DENSE_MIN_QUERIES, 32)
    assert dodo.device_status() == 0
    return {"batch": B, "heads": H, "document_tokens": n, "ratio": r, "nuggets": k, "query_tokens": tq, "instances": inst,
            "gather_then_attend_us": us_c, "attend_indexed_us": us_i, "indexed_speedup": us_c["mean"] / us_i["mean"],
            "outputs_bit_equal": bool(same)}


def other_configs(dodo, peaks, peak_kind, reps: int) -> dict:
    """The workload configurations beside the headline one, each at full size, one layer."""
    import torch
    from paper_2310_02409_b200 import inputs
    out = {}

    def freed(fn):
        rec = fn()
        torch.cuda.synchronize()
        torch.cuda.empty_cache()
        return rec

    wl3 = inputs.WORKLOADS["c3_llama7b_ar"]
    out["c3_llama7b_ar"] = freed(lambda: config_compress_decode(dodo, wl3, 10, ("bench", "c3"), peaks, peak_kind, reps))
    wl4 = inputs.WORKLOADS["c4_llama13b_sweep"]
    out["c4_llama13b_sweep"] = {f"r{r}": freed(lambda r=r: config_compress_decode(dodo, wl4, r, ("bench", "c4", r), peaks, peak_kind, reps))
                                for r in wl4.ratios}
    wl5 = inputs.WORKLOADS["c5_ragged_serving"]
    out["c5_ragged_serving"] = freed(lambda: config_ragged_serving(dodo, wl5, 10, peaks, peak_kind, reps))
    out["scorer_mlp_16k_tokens"] = freed(lambda: config_scorer_mlp(dodo, 16384, 4096, peaks, peak_kind, reps))
    wl2 = inputs.WORKLOADS[WORKLOAD]
    out["mlp_scored_compress_c2_shape"] = freed(lambda: config_mlp_compress(dodo, wl2, RATIO, peaks, peak_kind, reps))
    out["mean_pool_baseline_c2_shape"] = freed(lambda: config_mean_pool(dodo, wl2, RATIO, peaks, peak_kind, reps))
    # one-shot queries over a compressed document at the sizes the paper works through (a 231-token document with a
    # 17-token query, an 878-token document), LLaMA-7B heads, batch 8; and a shape where the index route loses
    out["one_shot_query"] = {
        "doc231_r5": freed(lambda: config_one_shot(dodo, "doc231", 8, 32, 231, 5, 17, reps)),
        "doc878_r10": freed(lambda: config_one_shot(dodo, "doc878", 8, 32, 878, 10, 17, reps)),
        "13b_16k_r10_block512": freed(lambda: config_one_shot(dodo, "c4r10", 1, 40, 16384, 10, 512, reps)),
    }
    return out


def run_cuda(args):
    import numpy as np
    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    check_world(args.gpus, world)
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    from paper_2310_02409_b200 import build
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    from paper_2310_02409_b200 import api, inputs
    from paper_2310_02409_b200.workloads import CompressDecode

    wl = inputs.WORKLOADS[WORKLOAD]
    dodo = api.Dodo(local_rank)
    if args.target_blocks:
        dodo.set_tuning(api.TUNE_ATTEND_TARGET_BLOCKS, args.target_blocks)
    R = args.instances
    insts = [CompressDecode(dodo, wl, RATIO, ("bench", rank, i)) for i in range(R)]
    steps = insts[0].steps

    def compress_all():
        for it in insts:
            it.compress()

    def decode_all():
        for s in range(steps):
            for it in insts:
                it.decode_step(s)

    # eager once (loads the kernels), then capture the two halves of a step as CUDA graphs so the
    # 1000+ launches of a step are not bound by Python
    compress_all(); decode_all()
    torch.cuda.synchronize()
    assert dodo.device_status() == 0
    side = torch.cuda.Stream()
    gA, gB = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
    with torch.cuda.graph(gA, stream=side):
        compress_all()
    with torch.cuda.graph(gB, stream=side):
        decode_all()
    launches_per_step = R * 2 + R * steps     # per instance: fused score + TopK, the gather that follows its flags, then the attends

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        gA.replay(); gB.replay()
    barrier()
    sampler = ClockSampler(local_rank) if rank == 0 else None
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    barrier()
    for i in range(args.steps):
        ev[i][0].record(); gA.replay(); ev[i][1].record(); gB.replay(); ev[i][2].record()
    barrier()
    total_ms = ev[0][0].elapsed_time(ev[-1][2])
    compress_ms = sum(e[0].elapsed_time(e[1]) for e in ev) / args.steps
    decode_ms = sum(e[1].elapsed_time(e[2]) for e in ev) / args.steps
    step_ms = [e[0].elapsed_time(e[2]) for e in ev]                   # per step: mean, median and best are reported
    decode_step_ms = [e[1].elapsed_time(e[2]) for e in ev]
    compress_step_ms = [e[0].elapsed_time(e[1]) for e in ev]
    assert dodo.device_status() == 0

    # the workload as stated, one layer instance on its own: its 35 MB of K/V stay in L2 from one decode
    # step to the next (reported beside the cold figure, not part of `value`)
    gW = torch.cuda.CUDAGraph()
    with torch.cuda.graph(gW, stream=side):
        for s in range(steps):
            insts[0].decode_step(s)
    gW.replay()
    torch.cuda.synchronize()
    w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    w0.record()
    for _ in range(3):
        gW.replay()
    w1.record()
    torch.cuda.synchronize()
    warm_us = w0.elapsed_time(w1) * 1e3 / (3 * steps)

    # the compress step as the two calls it replaces (the gather waits for the whole score + select launch), same
    # instances in the same rotation: reported beside the one-call figure, not part of `value`
    def compress_two_calls():
        for it in insts:
            it.cache_len[:] = 0
            dodo.score_select(it.X, it.w, 0.0, it.seq_off, it.nug_off, 0, it.scores, it.idx)
            dodo.gather_kv(it.K, it.V, it.seq_off, it.idx, it.nug_off, it.pos_base, it.cacheK, it.cacheV, it.cache_pos,
                           it.cache_off, it.cache_len)
    two_call_us = spread(time_graph(compress_two_calls, 20), R)
    compress_all()   # (leave the caches as the one-call step fills them; same contents)
    torch.cuda.synchronize()

    # end to end: every step uploads its inputs from pinned host memory and downloads the outputs
    e2e_steps = max(1, min(args.steps, 5))
    h2d = d2h = 0
    e2e_ms = float("nan")
    if not args.no_e2e:
        # one dodo_compress_decode_host call per layer instance: inputs start in pinned HOST memory,
        # outputs end there; the copies, the compression and all decode steps are inside the call
        names = ["X", "w", "K", "V", "locK", "locV", "Qd"]
        pinned = [{nm: getattr(it, nm).cpu().pin_memory() for nm in names} for it in insts]
        out_host = [torch.empty_like(it.Od, device="cpu").pin_memory() for it in insts]
        # bytes that cross the bus per step: X, w, the local rows and the queries are uploaded whole; of the
        # context's K and V (pinned, visible to the device) the gather reads only the nuggets' rows in place
        row_bytes = wl.H * wl.dh * pinned[0]["K"].element_size()
        h2d = sum(t.numel() * t.element_size() for p in pinned for nm, t in p.items() if nm not in ("K", "V"))
        h2d += sum(2 * int(it.nug_off[-1]) * row_bytes for it in insts)
        d2h = sum(t.numel() * t.element_size() for t in out_host)
        it0 = insts[0]
        # two lanes (a stream, an arena and a library context each: a context's counters serve one stream at a time)
        # take the instances alternately: the calls are asynchronous, so one instance's copies cross PCIe while the
        # previous one computes
        arena_bytes = dodo.host_arena_bytes(api.BF16, wl.d, wl.H, wl.dh, int(it0.seq_off[-1]), int(it0.nug_off[-1]),
                                            wl.B, wl.local, steps)
        lanes = [(torch.cuda.Stream(), torch.empty(arena_bytes, dtype=torch.uint8, device="cuda"), ctx_)
                 for ctx_ in (dodo, api.Dodo(local_rank))]

        def e2e_step():
            main = torch.cuda.current_stream()
            for side, _, _ in lanes:
                side.wait_stream(main)
            for i, (it, p, o) in enumerate(zip(insts, pinned, out_host)):
                side, arena, lane_ctx = lanes[i % 2]
                with torch.cuda.stream(side):
                    lane_ctx.compress_decode_host(p["X"], p["w"], p["K"], p["V"], it.seq_off, it.nug_off, p["locK"], p["locV"],
                                              wl.local, p["Qd"], it.sm_scale, o, arena)
            for side, _, _ in lanes:
                main.wait_stream(side)

        e2e_step()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(e2e_steps):
            e2e_step()
        e1.record()
        barrier()
        e2e_ms = e0.elapsed_time(e1)
    clocks = sampler.stop() if sampler else None

    total_ms, e2e_ms, decode_ms, compress_ms = max_over_ranks([total_ms, e2e_ms, decode_ms, compress_ms], world, "cuda")

    tokens_per_step = R * wl.B * steps
    if rank == 0:
        peaks, peak_kind = measured_peaks()
        value = job_throughput(tokens_per_step, args.steps, world, total_ms)
        e2e_value = job_throughput(tokens_per_step, e2e_steps, world, e2e_ms)
        attend_bytes = insts[0].bytes_decode_step(0)
        attend_us = decode_ms * 1e3 / (R * steps)
        achieved = attend_bytes / (attend_us * 1e-6) / 1e9
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": workload_config(wl, int(insts[0].k[0]), R, world),
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": e2e_steps},
            "gpu_launches": launches_per_step * args.steps,
            "clocks": clocks,
            "roofline": {"kernel": "attend_kernel<bf16,128,QT=1,U=4> (split-K flash-decode)", "bound": "hbm",
                         "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": achieved / peaks["hbm_gbs"], "peak_kind": f"of {peak_kind}",
                         "frac_of_nominal_8TBs": achieved / 8000.0, "traffic": attend_traffic(),
                         "bytes_per_launch": attend_bytes, "us_per_launch": attend_us},
            "spread": {"ms_per_step": {k: (v / 1e3 if k != "reps" else v) for k, v in spread(step_ms).items()},
                       "attend_us_per_launch": spread(decode_step_ms, R * steps),
                       "compress_us_per_instance": spread(compress_step_ms, R),
                       "tokens_per_s_median": world * tokens_per_step / (spread(step_ms)["median"] * 1e-6),
                       "tokens_per_s_best": world * tokens_per_step / (spread(step_ms)["best"] * 1e-6),
                       "note": "this rank's per-step device times (one CUDA-event pair per step); `value` is from the "
                               "max over ranks of the whole timed region"},
            "breakdown": {"compress_ms_per_step": compress_ms, "decode_ms_per_step": decode_ms,
                          "decode_only_tokens_per_s": tokens_per_step / (decode_ms * 1e-3),
                          "attend_us_per_launch_l2_warm_single_instance": warm_us,
                          "compress_us_per_instance_as_two_waiting_launches": two_call_us,
                          "compress_GBs": R * (insts[0].bytes_score() + insts[0].bytes_gather()) / (compress_ms * 1e-3) / 1e9},
        }
        if world == 1 and not args.no_cpu_baseline:
            import oracle
            # whole instances (compression and all decode steps, nothing scaled) until about 10 s are spent
            spent_total, done = 0.0, 0
            for it in insts:
                est, spent, used = oracle_pass(host_copy(it), steps)
                spent_total += spent
                done += 1
                if spent_total >= 10.0:
                    break
            cores = oracle.threads()
            line["cpu_baseline"] = {
                "value": done * wl.B * steps / spent_total, "unit": UNIT, "cores": cores, "kind": "oracle",
                "sample": f"{done} of the {R} layer instances in full (score+select+gather of {wl.B}x{wl.n_ctx[0]} tokens, "
                          f"all {steps} decode steps): {spent_total:.1f} s of CPU work"}
            # the same oracle on one thread: one instance, compression in full, 8 decode steps scaled to all
            oracle.set_threads(1)
            try:
                est1, spent1, used1 = oracle_pass(host_copy(insts[0]), 8)
            finally:
                oracle.set_threads(cores)
            line["cpu_baseline"]["single_thread"] = {
                "value": wl.B * steps / est1, "unit": UNIT, "cores": 1,
                "sample": f"one layer instance, score+select+gather in full, {used1} of {steps} decode steps scaled to "
                          f"all: {spent1:.1f} s of CPU work"}
        if world == 1 and not args.no_configs:
            # the other configurations, full size, one layer each (the headline instances are released first)
            del insts, gA, gB, gW
            if not args.no_e2e:
                del lanes, pinned, out_host
            torch.cuda.synchronize()
            torch.cuda.empty_cache()
            line["configs"] = other_configs(dodo, peaks, peak_kind, max(20, args.steps))
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--instances", type=int, default=8)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (tuning sweeps)")
    ap.add_argument("--no-configs", action="store_true", help="skip the other workload configurations (tuning sweeps)")
    ap.add_argument("--target-blocks", type=int, default=0, help="override the split-K block target")
    args = ap.parse_args()
    if args.gpus < 1:
        raise SystemExit("bench.py: --gpus must be at least 1")
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(respawn_under_launcher(args.gpus, sys.argv[1:]))
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
