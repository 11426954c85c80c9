#!/usr/bin/env python
"""Writes tests/golden/c2_oracle_trace.json: the CPU oracle's own free-running decode of the c2 request
(LLaDA-8B-shaped random-init model, batch 1, prompt 256, generate 256 tokens in blocks of 32,
threshold 0.9).  Calls nothing but oracle/ and the seeded input generators; takes tens of minutes on a
few host cores and about 40 GB of memory, which is why its result is stored.

Stored per denoise step: block, step, the mask before the step, and for every position of the block the
oracle's confidence, entropy, arg-max token and top-2 probability gap (the quantities the parity rule
of the decoding tests is stated in), and the positions committed.  Stored per request: the tokens, the
step at which each position was committed, and the forward counts.

  python tests/golden/make_c2_oracle_trace.py [--workload c2] [--out tests/golden/c2_oracle_trace.json]
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import time

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from oracle import d3_oracle as o  # noqa: E402
from paper_2601_07568_b200 import synth_inputs as si  # noqa: E402


def main() -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--out", default=os.path.join(ROOT, "tests", "golden", "c2_oracle_trace.json"))
    ap.add_argument("--mirror", type=int, default=1, help="1: activations rounded to bf16 where a bf16 pipeline stores them")
    args = ap.parse_args()
    w = si.WORKLOADS[args.workload]
    assert w.batch == 1, "one sequence"
    t0 = time.time()
    W = si.gen_weights(w.model)
    ids, lens = si.gen_prompts(w)
    model = o.model_from_shape(w.model, W, np.float32, mirror_bf16=bool(args.mirror))
    prompt = ids[0, :lens[0]]

    # the oracle's generate loop, step by step, so that the top-2 gap of every step can be kept
    state = model.prefill(prompt)
    n_blocks = w.gen_len // w.block
    tokens = np.full(w.gen_len, w.model.mask_id, dtype=np.int32)
    commit_step = np.zeros(w.gen_len, dtype=np.int32)
    steps = []
    n_denoise = n_finalize = 0
    for j in range(n_blocks):
        blk = np.full(w.block, w.model.mask_id, dtype=np.int32)
        mask = np.ones(w.block, dtype=bool)
        step = 0
        while mask.any():
            step += 1
            lg, conf, tok, ent = model.denoise_forward(state, blk)
            p, _, _, _ = o.softmax_stats(lg, w.model.mask_id)
            part = np.partition(p, -2, axis=-1)
            gap = part[:, -1] - part[:, -2]
            commit = o.decide(conf, ent, mask, w.threshold, o.MODE_CONFIDENCE)
            steps.append(dict(block=j, step=step, mask_in=mask.astype(int).tolist(), conf=[float(x) for x in conf],
                              ent=[float(x) for x in ent], tok=[int(x) for x in tok], gap=[float(x) for x in gap],
                              commit=np.flatnonzero(commit).tolist()))
            blk[commit] = tok[commit]
            mask[commit] = False
            commit_step[j * w.block:(j + 1) * w.block][commit] = step
            n_denoise += 1
            print(f"block {j} step {step}: committed {int(commit.sum())}, {int(mask.sum())} left, {time.time() - t0:.0f} s", flush=True)
        state = model.finalize_block(state, blk)
        n_finalize += 1
        tokens[j * w.block:(j + 1) * w.block] = blk
    out = dict(workload=w.name, model=w.model.name, threshold=w.threshold, block=w.block, gen_len=w.gen_len,
               prompt_len=int(lens[0]), mirror_bf16=bool(args.mirror), arithmetic="float32 on bf16-valued weights",
               n_denoise=n_denoise, n_finalize=n_finalize, tokens=[int(x) for x in tokens],
               commit_step=[int(x) for x in commit_step], steps=steps, seconds=round(time.time() - t0, 1),
               written_by="tests/golden/make_c2_oracle_trace.py (oracle only)")
    with open(args.out, "w") as f:
        json.dump(out, f)
    print("wrote", args.out, "denoise", n_denoise, "finalize", n_finalize)
    return 0


if __name__ == "__main__":
    sys.exit(main())
