"""Benchmark of the compressed-context hot path on B200.

Workload: the LLaMA-7B-shaped single-layer decode configuration (bf16, batch 8, d = 4096, 32 heads
x 128, context 2048 -> 205 nuggets per sequence at ratio 10, 128 decode steps, each attending the
nuggets plus a 64-token local window).  One benchmark step is one pass of the whole path:
score+select and gather for every sequence, then all 128 decode steps.  A single layer's K/V
(35 MB) would sit in the 126 MB L2, so R independent instances of the layer are interleaved step
by step; every attend launch then reads its keys from HBM, as it would in a multi-layer model.

Prints ONE JSON line (see README/DESIGN for the keys).  `--impl reference` times the fp64 CPU oracle
on the host cores instead.
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
ATTEND_TRAFFIC = {"bytes": 35380992, "attend_cu_sha1": "1322e8197c56fce1dc04ee7d1f9b006b5ef2f70b"}

METRIC = "nugget-attention decode tokens/s"
UNIT = "tokens/s"
WORKLOAD = "c2_llama7b_decode"
RATIO = 10


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
    sample = (f"per step: full score+select+gather of {wl.B}x{wl.n_ctx[0]} tokens, {used} of {wl.decode_steps} decode "
              f"steps computed and scaled to all of them; {args.steps} steps, {wall:.1f} s of CPU work")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * est_total / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "batch": wl.B, "context": wl.n_ctx[0], "ratio": RATIO,
                       "decode_steps": wl.decode_steps, "local_window": wl.local},
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


def run_cuda(args):
    import numpy as np
    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
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
    if args.stages:
        dodo.set_tuning(api.TUNE_ATTEND_STAGES, args.stages)
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
    launches_per_step = R * 2 + R * steps

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
            "config": {"workload": WORKLOAD, "batch": wl.B, "context": wl.n_ctx[0], "ratio": RATIO,
                       "nuggets_per_seq": int(insts[0].k[0]), "decode_steps": steps, "local_window": wl.local,
                       "heads": wl.H, "head_dim": wl.dh, "d": wl.d, "instances": R,
                       "l2": f"cold: {R} independent layer instances interleaved per decode step "
                             f"({R * attend_bytes / 1e6:.0f} MB of K/V between reuses, L2 is 126 MB)",
                       "parallelism": f"replicas x{world}, no collective"},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": e2e_steps},
            "gpu_launches": launches_per_step * args.steps,
            "clocks": clocks,
            "roofline": {"kernel": "attend_kernel<bf16,128,QT=1,U=4> (split-K flash-decode)", "bound": "hbm",
                         "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": achieved / peaks["hbm_gbs"], "peak_kind": f"of {peak_kind}",
                         "frac_of_nominal_8TBs": achieved / 8000.0, "traffic": attend_traffic(),
                         "bytes_per_launch": attend_bytes, "us_per_launch": attend_us},
            "breakdown": {"compress_ms_per_step": compress_ms, "decode_ms_per_step": decode_ms,
                          "decode_only_tokens_per_s": tokens_per_step / (decode_ms * 1e-3),
                          "attend_us_per_launch_l2_warm_single_instance": warm_us,
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
    ap.add_argument("--target-blocks", type=int, default=0, help="override the split-K block target")
    ap.add_argument("--stages", type=int, default=0, help="override the shared-memory stage count")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
