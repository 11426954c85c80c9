#!/usr/bin/env python
"""Run a few denoise steps of one workload shape, for profilers and quick timing.

  python profile_step.py --workload c2 --layers 4 --steps 3

The model has the workload's architecture with ``--layers`` layers (default: all) and seeded random
weights; the prompt is the workload's.  After prefill the script runs ``--steps`` denoise steps on a
fully masked block (threshold 2.0, so that only the forced position commits and every step does the
same work) and prints the mean step time from CUDA events.  With few layers the whole process holds
a few GB on the device, which keeps profiler captures short.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import sys

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def main() -> int:
    import numpy as np
    import torch

    from paper_2601_07568_b200 import binding as d3
    from paper_2601_07568_b200 import build as d3build
    from paper_2601_07568_b200 import synth_inputs as si

    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c2", choices=sorted(si.WORKLOADS))
    ap.add_argument("--layers", type=int, default=0, help="number of layers (0 = the workload's)")
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=1)
    ap.add_argument("--prefix", type=int, default=0, help="override the cached prefix length (0 = after prefill)")
    ap.add_argument("--no-chain", action="store_true", help="one kernel per matmul instead of the chain launch")
    args = ap.parse_args()

    d3build.build()
    w = si.WORKLOADS[args.workload]
    shape = w.model
    if args.layers > 0:
        shape = dataclasses.replace(shape, n_layers=args.layers)
    torch.cuda.set_device(0)
    dev = "cuda:0"
    W = si.gen_weights(shape)
    cfg = d3.make_config(shape, block=w.block, max_batch=w.batch, max_seq=w.max_seq,
                         max_prefill_rows=w.batch * w.prompt_max)
    ctx = d3.d3_create(cfg)
    d3.d3_load_weights(ctx, d3.weights_from_numpy(shape, W), shape.n_layers)
    del W
    ids_np, lens_np = si.gen_prompts(w)
    d3.d3_prefill(ctx, torch.from_numpy(ids_np).to(dev), torch.from_numpy(lens_np).to(dev))
    if args.no_chain:
        d3.d3_set_tuning(ctx, chain=0)
    if args.prefix > 0:
        d3.d3_set_state(ctx, torch.full((w.batch,), args.prefix, dtype=torch.int32, device=dev))
    bs, B = w.batch, w.block
    ids = torch.full((bs, B), shape.mask_id, dtype=torch.int32, device=dev)
    mask = torch.ones((bs, B), dtype=torch.uint8, device=dev)
    pos = torch.zeros((bs, B), dtype=torch.int32, device=dev)
    oid = torch.zeros((bs, B), dtype=torch.int32, device=dev)
    cnt = torch.zeros(bs, dtype=torch.int32, device=dev)

    def step():
        ids.fill_(shape.mask_id)
        mask.fill_(1)
        d3.d3_denoise_step(ctx, ids, mask, 2.0, pos, oid, cnt)

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    l0 = d3.d3_launch_count(ctx)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / max(args.steps, 1)
    launches = (d3.d3_launch_count(ctx) - l0) // max(args.steps, 1)
    err = d3.d3_get_error_word(ctx)
    d3.d3_destroy(ctx)
    print(json.dumps({"workload": w.name, "layers": shape.n_layers, "rows": bs * B, "ms_per_step": ms,
                      "launches_per_step": launches, "device_error_word": err,
                      "committed": int(cnt.sum().item())}))
    return 0 if err == 0 else 1


if __name__ == "__main__":
    sys.exit(main())
