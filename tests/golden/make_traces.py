#!/usr/bin/env python
"""Writes the oracle's free-running traces of the benchmark configurations that fit host memory, for the GPU
parity tests to compare whole runs against (tests/golden/<config>_trace.json).  Calls only oracle/ and synth/.

    python tests/golden/make_traces.py c2            # config 2: 7B shape, 512-token prompt, 256 greedy tokens (about 15 min on 8 cores)

A trace holds vanilla greedy decoding (tokens and the top-1/top-2 margin of every step) and the SWIFT run with the
config's fixed skip set (per round: start position, draft tokens, their margins, target arg maxes and margins,
accepted length, next token), keyed by a hash of the configuration and of the oracle's and the generator's sources:
a test skips a trace whose key no longer matches."""
import hashlib
import json
import os
import sys
import time

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import torch  # noqa: E402

import synth  # noqa: E402
from oracle import swift_oracle as so  # noqa: E402

HERE = os.path.dirname(os.path.abspath(__file__))


def trace_key(name: str) -> str:
    model_name, run = synth.RUNS[name]
    h = hashlib.sha256()
    h.update(repr((synth.MODELS[model_name], run)).encode())
    for rel in ("oracle/swift_oracle.py", "synth/__init__.py", "synth/synth_cpu.c"):
        h.update(open(os.path.join(ROOT, rel), "rb").read())
    return h.hexdigest()[:16]


def make(name: str) -> dict:
    model_name, run = synth.RUNS[name]
    cfg = synth.MODELS[model_name]
    assert run.mode == "greedy" and not run.optimise, "free-running traces cover the greedy, fixed-skip-set configurations"
    w = synth.make_weights(cfg)
    w = {k: (v.to(torch.float32) if torch.is_tensor(v) else [{n: t.to(torch.float32) for n, t in blk.items()} for blk in v]) for k, v in w.items()}
    z = [int(v) for v in synth.block_mask(cfg, synth.draft_blocks(cfg, run.n_skip_blocks))]
    prompt = synth.prompt(cfg, run.prompt_len)
    cap = run.prompt_len + run.max_new + 32
    t0 = time.time()
    van, margins = so.vanilla_generate(so.Oracle(so.Shape.of(cfg), w, dtype=torch.float32, max_positions=cap), prompt, run.max_new)
    t1 = time.time()
    out, rounds, stats = so.swift_generate(so.Oracle(so.Shape.of(cfg), w, dtype=torch.float32, max_positions=cap), prompt, z,
                                           so.GenParams(max_new=run.max_new, max_draft=run.max_draft, stop_conf=run.stop_conf))
    t2 = time.time()
    assert out == van, "the oracle's SWIFT run must reproduce vanilla greedy decoding (Section 3.1)"
    return {"config": name, "key": trace_key(name), "oracle_dtype": "float32", "seconds": {"vanilla": t1 - t0, "swift": t2 - t1},
            "prompt_len": run.prompt_len, "skip_mask": z, "tokens": van, "margins": margins, "stats": stats,
            "rounds": [{"n_start": r.n_start, "draft": r.draft, "draft_margin": r.draft_margin, "conf": r.conf,
                        "target_argmax": r.target_argmax, "target_margin": r.target_margin, "accepted": r.accepted,
                        "next_token": r.next_token} for r in rounds]}


if __name__ == "__main__":
    torch.set_num_threads(os.cpu_count() or 1)
    for name in sys.argv[1:] or ["c2"]:
        tr = make(name)
        path = os.path.join(HERE, f"{name}_trace.json")
        json.dump(tr, open(path, "w"))
        print(f"{path}: {len(tr['tokens'])} tokens, {len(tr['rounds'])} rounds, M {tr['stats']['M']:.2f}, alpha {tr['stats']['alpha']:.2f}, "
              f"{tr['seconds']['vanilla'] + tr['seconds']['swift']:.0f} s")
