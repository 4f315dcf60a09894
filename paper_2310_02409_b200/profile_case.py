"""A small, self-ending run of the hot path for profilers: R layer instances of the LLaMA-7B decode
workload, compressed once, then a few decode steps launched eagerly (no CUDA graph), interleaved over
the instances so that every attend launch reads its keys from HBM.

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
    ap.add_argument("--stages", type=int, default=0)
    ap.add_argument("--dense-balance", type=int, default=0, help="0 auto, 1 always, 2 never")
    ap.add_argument("--query-block-reps", type=int, default=0,
                    help="also run the workload's query block this many times and report its rate")
    args = ap.parse_args()
    build.build()
    dodo = api.Dodo(0)
    if args.target_blocks:
        dodo.set_tuning(api.TUNE_ATTEND_TARGET_BLOCKS, args.target_blocks)
    if args.dense_balance:
        dodo.set_tuning(api.TUNE_DENSE_BALANCE, args.dense_balance)
    if args.stages:
        dodo.set_tuning(api.TUNE_ATTEND_STAGES, args.stages)
    wl = inputs.WORKLOADS[args.workload]
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
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.query_block_reps):
            for it in insts:
                it.query_block()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / (args.query_block_reps * len(insts))
        fl = insts[0].flops_query_block()
        print(f"query block: {ms * 1e3:.1f} us per launch, {fl / 1e9:.2f} GFLOP, {fl / ms / 1e9:.1f} TFLOP/s")
    torch.cuda.synchronize()
    assert dodo.device_status() == 0
    print(f"ok: {args.instances} instances, {args.decode_steps} decode steps, "
          f"{sum(i.device_bytes() for i in insts) / 1e9:.2f} GB on the device")


if __name__ == "__main__":
    main()
