#!/usr/bin/env python
"""Benchmark of the SWIFT decoding hot path on B200.

One step = one complete run of the workload through the C boundary: prefill of the synthetic prompt,
then draft / verify / accept rounds until max_new tokens are out (all with host buffers in and out).
`value` is decode tokens/s with everything resident in HBM (CUDA-event time of the decode part, on the
library's stream); `e2e` is tokens/s of the whole call (prefill and host<->device copies included) by
the host clock.  Inputs are synthetic LLaMA-shaped models (see synth/), far larger than L2, so no L2
flush is needed between steps.  Multi-GPU: replicas only (batch-1 decoding is one dependent chain);
each rank decodes its own sequence on its own GPU and `value` sums them.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

import synth  # noqa: E402

METRIC = "batch-1 decode tokens/s (SWIFT self-speculative decoding)"
UNIT = "tokens/s"
PAPER_CONTEXT = "paper: 1.3x-1.6x over vanilla on 4x RTX A6000, FP16, HF transformers (context only)"


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def tensor_peak_tflops():
    """Dense bf16 throughput sustained over a long loop (the many-row GEMMs run inside long steps)."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d.get("bf16_tflops_sustained", d.get("bf16_tflops", 1400.0)))
    return 1400.0


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def __exit__(self, *a):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()

    def summary(self):
        sm, mx, reasons = [], 0.0, set()
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx = max(mx, float(r[1]))
            except (ValueError, IndexError):
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx or None, "reasons": sorted(reasons),
                "samples": len(sm)}


def aggregate_replicas(tokens: int, decode_ms: float, total_ms: float, wall_s: float, world: int, device=None):
    """Whole-job numbers of N independent replicas: every rank decoded `tokens` tokens of its own sequence; the job
    takes as long as its slowest rank (max over ranks), and its throughput is all ranks' tokens over that time.
    Returns (decode tokens/s, max decode ms, max total ms, max wall s).  Uses the default process group when world > 1."""
    if world > 1:
        import torch.distributed as dist
        t = torch.tensor([decode_ms, total_ms, wall_s], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        decode_ms, total_ms, wall_s = t.tolist()
    return world * tokens / (decode_ms * 1e-3), decode_ms, total_ms, wall_s


def config_of(desc: str, kv_dtype: str):
    """The `config` object of the JSON line; both arms (this library, the CPU oracle) print the same keys and values."""
    return {"workload": desc, "l2": "inputs (weights) far larger than L2; no flush", "parallelism": "replicas only",
            "kv_cache": kv_dtype, "e2e_note": "whole swift_generate call incl. prefill and host copies, host clock",
            "context": PAPER_CONTEXT}


def profile_traffic(shape: str, rows: int):
    """DRAM bytes per launch of the gate/up GEMM from the ncu capture summarised under profiles/ (a line
    `traffic: <shape> <rows> rows = <bytes> bytes per launch` in the summary that names its command), or None."""
    path = os.path.join(ROOT, "profiles", "gemm_tc_gate_up_9rows.md")
    try:
        for line in open(path):
            parts = line.split()
            if len(parts) >= 7 and parts[0] == "traffic:" and parts[1] == shape and parts[2] == str(rows):
                return float(parts[5])
    except OSError:
        pass
    return None


def workload(name: str):
    model_name, run = synth.RUNS[name]
    cfg = synth.MODELS[model_name]
    z = synth.block_mask(cfg, synth.draft_blocks(cfg, run.n_skip_blocks))
    return cfg, run, z


def oracle_sample(cfg, run, z, weights, n_ctx, k=None, n_vanilla=3):
    """The CPU oracle, as it stands, on a bounded slice of the workload at its final context length n_ctx: n_vanilla
    vanilla steps and one SWIFT round (k drafts + verify + accept) behind a cache of n_ctx positions.  The cache is
    filled with seeded random K,V instead of a prefill of n_ctx tokens (a forward's cost does not depend on the cached
    values; the prefill alone would take minutes on host cores).  Returns tokens/s of both."""
    from oracle import swift_oracle as so
    k = run.max_draft if k is None else k
    dtype = torch.float64 if cfg.dtype == "f32" else torch.float32
    o = so.Oracle(so.Shape.of(cfg), weights, dtype=dtype, max_positions=n_ctx + n_vanilla + k + 8)
    g = torch.Generator().manual_seed(1234)
    for b in range(cfg.n_blocks):
        o.K[b][:n_ctx] = torch.randn(n_ctx, cfg.n_kv_heads, cfg.head_dim, generator=g, dtype=dtype)
        o.V[b][:n_ctx] = torch.randn(n_ctx, cfg.n_kv_heads, cfg.head_dim, generator=g, dtype=dtype)
    o.n, o.tokens = n_ctx, synth.prompt(cfg, n_ctx + 1)
    t0 = time.perf_counter()
    for _ in range(n_vanilla):
        row = o.forward_rows([o.tokens[-1]], o.n)[0]
        o.commit([], so.argmax_lowest(row))
    t1 = time.perf_counter()
    d_tok, _, _ = o.draft(list(z), k)
    tl = o.verify(d_tok)
    a, nxt = so.accept_greedy(d_tok, tl)
    o.commit(d_tok[:a], nxt)
    t2 = time.perf_counter()
    return {"vanilla": n_vanilla / (t1 - t0), "swift": (a + 1) / (t2 - t1), "seconds": t2 - t0, "accepted": a, "k": k}


def oracle_model(cfg, run, z, weights=None):
    """The model the CPU baseline runs: the workload's own when its widened copy fits comfortably in host memory,
    else an 8-block copy with the same widths (its throughput is scaled by depth and labelled as extrapolated)."""
    small = cfg if cfg.n_blocks * cfg.block_params() < 8e9 else cfg.with_blocks(8)
    if small is cfg:
        return cfg, z, (weights if weights is not None else synth.make_weights(cfg)), 1.0
    zz = synth.block_mask(small, synth.draft_blocks(small, max(1, run.n_skip_blocks * 8 // cfg.n_blocks)))
    return small, zz, synth.make_weights(small), small.n_blocks / cfg.n_blocks


def sample_text(cfg, small, run, n_ctx, seconds=None):
    return (f"3 vanilla steps and one SWIFT round of {run.max_draft} drafts + verify + accept behind {n_ctx} cached positions "
            f"(the workload's final context length; cache filled with seeded random K,V)"
            + (f", {seconds:.1f} s of CPU work" if seconds is not None else "")
            + ("" if small is cfg else "; on an 8-block copy of the model, scaled by depth (extrapolated)"))


def stream_mode(model, cfg, run, z, gp, args, max_new, desc, hbm_peak):
    """A stream of inputs with the skip set carried over: input i starts from the set input i-1 ended with
    (swift_final_skip_mask) and keeps optimising it until an input ends above the matchness threshold; after that the
    set is used as it is.  One vanilla run per input gives the reference speed on the same prompt."""
    import dataclasses
    from paper_2410_06916_b200 import GenParams
    carry, optimising, rows = z, run.optimise, []
    model.generate(synth.prompt(cfg, 64), GenParams(max_new=8, vanilla=True))          # warm-up
    tot_tokens = tot_ms = van_ms = 0.0
    for i in range(args.stream):
        prompt = synth.prompt(cfg, run.prompt_len, stream=100 + i)
        gpi = dataclasses.replace(gp, skip_mask=carry, n_opt_rounds=gp.n_opt_rounds if optimising else 0)
        out, st, _ = model.generate(prompt, gpi)
        carry = model.final_skip_mask()                  # (before the vanilla run, which ends with the empty set)
        van, vst, _ = model.generate(prompt, GenParams(max_new=max_new, vanilla=True))
        if st.opt_rounds > 0 and st.best_matchness > run.stop_matchness:
            optimising = False
        rows.append({"input": i, "tokens_per_s": (st.tokens - 1) / (st.ms_decode * 1e-3), "vanilla_tokens_per_s": (vst.tokens - 1) / (vst.ms_decode * 1e-3),
                     "alpha": st.accepted / max(st.drafted, 1), "M": (st.tokens - 1) / st.rounds, "opt_rounds": st.opt_rounds,
                     "best_matchness": st.best_matchness, "ms_score": st.ms_score, "equals_vanilla": out == van,
                     "skipped_blocks": [int(b) for b in range(cfg.n_blocks) if carry[2 * b] and carry[2 * b + 1]]})
        tot_tokens += st.tokens - 1; tot_ms += st.ms_decode; van_ms += vst.ms_decode
    print(json.dumps({"metric": METRIC, "value": tot_tokens / (tot_ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.stream, "warmup": 1,
                      "ms_per_step": tot_ms / args.stream, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                      "dtype": "bf16" if cfg.dtype == "bf16" else "f32", "data": "synthetic",
                      "config": config_of(desc + f"; stream of {args.stream} inputs, skip set carried over", args.kv_dtype),
                      "vanilla_tokens_per_s": tot_tokens / (van_ms * 1e-3), "speedup_vs_vanilla": van_ms / tot_ms, "stream": rows}))


def micro(cfg, run, args, hbm_peak, tensor_peak):
    """Each GEMM shape of the walk, alone, on a 4-block copy of the model (weights still several times L2)."""
    from paper_2410_06916_b200 import SwiftModel
    small = cfg.with_blocks(4)
    model = SwiftModel(small, max_positions=64, max_draft=run.max_draft, kv_dtype=args.kv_dtype)
    model.load_weights(synth.iter_tensors(small))
    names = ["qkv", "o_proj", "gate_up", "down", "lm_head"]
    out = {"micro": small.name, "peak_gbs": hbm_peak, "gemms": {}}
    for which, name in enumerate(names):
        for rows in (1, run.max_draft + 1):
            ms, nbytes = model.time_gemm(which, rows, args.micro_iters)
            out["gemms"][f"{name}/{rows}"] = {"us": round(ms * 1e3, 2), "MB": round(nbytes / 1e6, 1),
                                              "gbs": round(nbytes / ms * 1e-6, 1), "frac": round(nbytes / ms * 1e-6 / hbm_peak, 3)}
        if args.micro_many_rows and (which != 2 or 2 * small.ffn <= small.vocab):
            # the many-row form: tensor-bound; two bf16 products per weight (hi and lo activation planes)
            ms, nbytes = model.time_gemm(which, 128, args.micro_iters)
            tflops = 2 * 2.0 * 128 * (nbytes / 2) / ms * 1e-9
            out["gemms"][f"{name}/128"] = {"us": round(ms * 1e3, 2), "MB": round(nbytes / 1e6, 1), "tflops_hi_lo": round(tflops, 1),
                                           "frac_tensor": round(tflops / tensor_peak, 3)}
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    # defaults: long enough for the optimising workload (the default) to have settled on its layer set before the timed steps
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3", choices=sorted(synth.RUNS))
    ap.add_argument("--max-new", type=int, default=0, help="override the number of generated tokens")
    ap.add_argument("--prompt-len", type=int, default=0, help="override the prompt length (profiling runs)")
    ap.add_argument("--kv-dtype", default="f32", choices=["f32", "bf16"], help="storage of cached K,V")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--stream", type=int, default=0,
                    help="run the workload as a stream of this many inputs (different prompts), each starting from the skip set "
                         "the previous one ended with (the dynamic input streams of the paper's Section 5.3); prints one JSON line")
    ap.add_argument("--micro", action="store_true",
                    help="time each weight-streaming GEMM of the model alone on a few-block copy (profiling aid); prints one JSON line")
    ap.add_argument("--micro-iters", type=int, default=40)
    ap.add_argument("--micro-score", action="store_true", help="with --micro-forward: also two rounds of candidate scoring")
    ap.add_argument("--micro-many-rows", action="store_true", help="with --micro: also the 128-row form of each GEMM")
    ap.add_argument("--micro-forward", action="store_true",
                    help="a few decode rounds on a 4-block copy of the model at the workload's context length (profiling aid)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    cfg, run, z = workload(args.workload)
    if args.prompt_len:
        import dataclasses
        run = dataclasses.replace(run, prompt_len=args.prompt_len)
    max_new = args.max_new or run.max_new
    hbm_peak, peak_kind = peaks()
    tensor_peak = tensor_peak_tflops()
    sampling = run.mode == "sampling"
    desc = (f"{args.workload}: {cfg.name}-shaped decoder ({cfg.n_blocks} blocks, d {cfg.d_model}, {cfg.dtype}), "
            f"prompt {run.prompt_len}, {max_new} {run.mode} tokens, {run.n_skip_blocks} blocks skipped, max draft {run.max_draft}"
            + (f", temperature {run.temperature}, top_p {run.top_p}" if sampling and (run.temperature != 1.0 or run.top_p != 1.0) else "")
            + (f", on-the-fly optimisation ({run.n_candidates} proposals per round, at most {run.max_opt_rounds} rounds per input); the steps "
               "form a stream of different inputs: skip set and proposal engine carry over from step to step, warm-up steps included" if run.optimise else ""))

    if args.impl == "reference":
        if rank != 0:
            return
        torch.set_num_threads(os.cpu_count() or 1)
        small, zz, w, scale = oracle_model(cfg, run, z)
        n_ctx = run.prompt_len + max_new
        vals = []
        for i in range(args.warmup + args.steps):
            s = oracle_sample(small, run, zz, w, n_ctx)
            if i >= args.warmup:
                vals.append(s)
        v = statistics.mean(x["swift"] for x in vals) * scale
        sample = "per step: " + sample_text(cfg, small, run, n_ctx)
        print(json.dumps({"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": 0, "steps": args.steps,
                          "warmup": args.warmup, "ms_per_step": 1e3 * statistics.mean(x["seconds"] for x in vals),
                          "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                          "config": config_of(desc, args.kv_dtype),
                          "cpu_baseline": {"value": v, "unit": UNIT, "cores": torch.get_num_threads(), "kind": "oracle", "sample": sample},
                          "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))
        return

    from paper_2410_06916_b200 import GenParams, SwiftModel
    torch.cuda.set_device(local)
    if args.micro:
        micro(cfg, run, args, hbm_peak, tensor_peak)
        return
    if args.micro_forward:
        small = cfg.with_blocks(4)
        zz = synth.block_mask(small, synth.draft_blocks(small, 2))
        model = SwiftModel(small, max_positions=run.prompt_len + 64, max_draft=run.max_draft, kv_dtype=args.kv_dtype)
        model.load_weights(synth.iter_tensors(small))
        prompt = synth.prompt(small, run.prompt_len)
        outs = {}
        for name, gp in (("vanilla", GenParams(max_new=4, vanilla=True)),
                         ("swift", GenParams(max_new=2 * (run.max_draft + 1) + 1, max_draft=run.max_draft, skip_mask=zz))):
            _, st, _ = model.generate(prompt, gp)
            outs[name] = {"ms_decode": st.ms_decode, "tokens": st.tokens, "rounds": st.rounds, "launches": st.kernel_launches}
        if args.micro_score:          # plus two rounds of candidate scoring (32 proposals, half of the sub-layers skipped)
            rng = np.random.default_rng(5)
            masks = (rng.random((32, 2 * small.n_blocks)) < 0.45).astype(np.uint8)
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            for _ in range(2):
                ev0.record(model.stream)
                model.score_skipsets(masks, 32)
                ev1.record(model.stream)
                torch.cuda.synchronize()
            outs["scoring_round_ms"] = ev0.elapsed_time(ev1)
        print(json.dumps({"micro_forward": small.name, "prompt": run.prompt_len, **outs}))
        return
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    weights = synth.make_weights(cfg) if cfg.n_blocks * cfg.block_params() < 40e9 else None
    model = SwiftModel(cfg, max_positions=run.prompt_len + max_new + 32, max_draft=run.max_draft, device=f"cuda:{local}",
                       kv_dtype=args.kv_dtype)
    if weights is not None:
        model.load_weights((n, -1, weights[n]) for n in ("embed", "lm_head", "final_norm"))
        model.load_weights((n, b, t) for b, wb in enumerate(weights["blocks"]) for n, t in wb.items())
    else:
        model.load_weights(synth.iter_tensors(cfg))
    if sampling:
        model.set_sampling(True, run.temperature, run.rng_seed, run.top_p)
    prompt = synth.prompt(cfg, run.prompt_len, stream=rank)
    if run.optimise:
        # config 3 as written: start from the uniform pattern; every optimisation round the library proposes the candidates
        # itself (random search, a Gaussian-process proposal every 25th step: Section 4.1, Appendix B.2) and scores them
        # together with the set in use; it stops above matchness 0.95, after the round cap, or after 300 proposals in a
        # row without a better set (Appendix B.2's patience, in rounds of n_candidates proposals)
        z = synth.block_mask(cfg, synth.uniform_blocks(cfg.n_blocks, run.n_skip_blocks))
    gp = GenParams(max_new=max_new, max_draft=run.max_draft, stop_conf=run.stop_conf, skip_mask=z, gamma=run.gamma,
                   n_opt_rounds=run.max_opt_rounds if run.optimise else 0, stop_matchness=run.stop_matchness,
                   n_candidates=run.n_candidates if run.optimise else 0, opt_skip_blocks=run.n_skip_blocks, opt_beta=25,
                   opt_seed=cfg.seed, opt_patience=-(-300 // run.n_candidates))

    if args.stream > 0:
        stream_mode(model, cfg, run, z, gp, args, max_new, desc, hbm_peak)
        return

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # With on-the-fly optimisation the steps form a stream, as in the paper (the optimisation phase runs until it has
    # converged and its cost is spread over the inputs that follow): a step starts from the skip set the previous step
    # ended with, the library's proposal engine keeps what it has learnt, and once a step ends with its set above the
    # matchness threshold the later steps use that set as it is.  The warm-up steps are the first inputs of that stream.
    import dataclasses
    opt_log = []

    def one_step():
        nonlocal gp, prompt
        if run.optimise:                                     # every step of the stream is another input
            prompt = synth.prompt(cfg, run.prompt_len, stream=1000 * rank + len(opt_log))
        tok, st, _ = model.generate(prompt, gp)
        if run.optimise:
            opt_log.append({"opt_rounds": st.opt_rounds, "best_matchness": st.best_matchness, "ms_score": st.ms_score,
                            "tokens_per_s": (st.tokens - 1) / (st.ms_decode * 1e-3), "alpha": st.accepted / max(st.drafted, 1)})
            done = st.opt_rounds > 0 and st.best_matchness > run.stop_matchness
            gp = dataclasses.replace(gp, skip_mask=model.final_skip_mask(), n_opt_rounds=0 if (done or gp.n_opt_rounds == 0) else gp.n_opt_rounds)
        return st

    for _ in range(args.warmup):
        one_step()
    launches0 = model.launches
    stats = []
    barrier()
    with ClockSampler(local) as clk:
        t0 = time.perf_counter()
        for _ in range(args.steps):
            stats.append(one_step())
        torch.cuda.synchronize()
        wall = time.perf_counter() - t0
    barrier()
    launches = model.launches - launches0
    dec_ms = sum(s.ms_decode for s in stats)
    tot_ms = sum(s.ms_decode + s.ms_prefill for s in stats)
    tokens = sum(s.tokens - 1 for s in stats)            # the first token comes out of prefill
    value, dec_ms, tot_ms, wall = aggregate_replicas(tokens, dec_ms, tot_ms, wall, world, device="cuda")
    e2e = world * sum(s.tokens for s in stats) / wall

    def dist_of(ms, nbytes, keep):
        """min / median / max over rounds of the achieved fraction of the HBM roofline (first round left out: warm-up)."""
        f = [b / (t * 1e-3) * 1e-9 / hbm_peak for t, b, k in list(zip(ms, nbytes, keep))[1:] if k and t > 0]
        if not f:
            return None
        return {"min": min(f), "p50": statistics.median(f), "max": max(f), "rounds": len(f)}

    # vanilla decoding of the same model for the comparison the metric names
    swift_tokens = model.generate(prompt, gp)[0]
    z_final = model.final_skip_mask()
    md, mv, bd, bv, kd = model.round_times()
    sbd, sbv = model.round_bytes_stored()
    fdist = {"draft_frac": dist_of(md, bd, kd > 0), "verify_frac": dist_of(mv, bv, kd == run.max_draft)}
    # the same rounds with cached K,V counted as they are stored (fp32 by default): what the implementation moves
    fdist_stored = {"draft_frac": dist_of(md, sbd, kd > 0), "verify_frac": dist_of(mv, sbv, kd == run.max_draft)}
    stored_ratio = {"draft": float(sbd[kd > 0].sum() / max(bd[kd > 0].sum(), 1.0)) if (kd > 0).any() else None,
                    "verify": float(sbv.sum() / max(bv.sum(), 1.0))}
    # expected speedup of Eq. 5 (Appendix B.3) with the measured cost ratio c = one draft forward / one verification
    full = kd == run.max_draft
    c_meas = float(np.median(md[full] / kd[full]) / np.median(mv[full])) if full.any() and run.max_draft > 0 else None
    model.generate(prompt[:64], GenParams(max_new=8, vanilla=True))
    if sampling:
        model.set_sampling(False)
    v_tokens, vst, _ = model.generate(prompt, GenParams(max_new=max_new, vanilla=True))
    vanilla = (vst.tokens - 1) / (vst.ms_decode * 1e-3)
    lossless = None if sampling else (swift_tokens == v_tokens)   # greedy SWIFT must reproduce vanilla decoding
    _, vmv, _, vbv, _ = model.round_times()
    _, vsbv = model.round_bytes_stored()
    fdist["vanilla_frac"] = dist_of(vmv, vbv, np.ones(len(vmv), dtype=bool))
    fdist_stored["vanilla_frac"] = dist_of(vmv, vsbv, np.ones(len(vmv), dtype=bool))
    stored_ratio["vanilla"] = float(vsbv.sum() / max(vbv.sum(), 1.0))

    s0 = stats[-1]
    n_ctx = run.prompt_len + max_new // 2
    fw = {"draft_gbs": sum(s.bytes_draft for s in stats) / max(sum(s.ms_draft for s in stats), 1e-9) * 1e-6,
          "verify_gbs": sum(s.bytes_verify for s in stats) / max(sum(s.ms_verify for s in stats), 1e-9) * 1e-6,
          "vanilla_gbs": vst.bytes_verify / (vst.ms_decode * 1e-3) * 1e-9,
          "draft_bytes": model.forward_bytes(z, 1, n_ctx), "verify_bytes": model.forward_bytes(None, run.max_draft + 1, n_ctx)}
    fw["draft_frac"], fw["verify_frac"], fw["vanilla_frac"] = (fw[k] / hbm_peak for k in ("draft_gbs", "verify_gbs", "vanilla_gbs"))
    fw["bytes"] = "algorithmic: weights of the kept sub-layers + output head + cached K,V at 2 bytes per element + rows in/out"
    # the same sums with the cache counted as stored (stored / algorithmic bytes of the same forwards)
    fw["stored_bytes_ratio"] = stored_ratio
    fw["draft_frac_stored_bytes"] = fw["draft_frac"] * stored_ratio["draft"] if stored_ratio["draft"] else None
    fw["verify_frac_stored_bytes"] = fw["verify_frac"] * stored_ratio["verify"]
    fw["vanilla_frac_stored_bytes"] = fw["vanilla_frac"] * stored_ratio["vanilla"]

    # dominant kernel: the weight-streaming GEMM (largest instance: fused gate/up), timed alone with CUDA events
    g_ms, g_bytes = model.time_gemm(2, run.max_draft + 1, 200)
    g1_ms, _ = model.time_gemm(2, 1, 200)
    achieved = g_bytes / (g_ms * 1e-3) * 1e-9
    # DRAM bytes per launch of that kernel (read + write, mean of two launches) from the ncu captures summarised in
    # the profiles folder (7B and 13B widths, 9 rows); other shapes have no capture of their own
    traffic = profile_traffic(cfg.name.split("-")[0], run.max_draft + 1)        # keyed by the widths (13b-graded has the 13b shapes)
    roofline = {"bound": "hbm", "kernel": "skinny GEMM, fused gate/up projection, %d rows" % (run.max_draft + 1),
                "achieved": achieved, "peak": hbm_peak, "peak_kind": f"{peak_kind} copy bandwidth (burst)", "unit": "GB/s",
                "frac": achieved / hbm_peak, "traffic": traffic, "bytes_per_launch": g_bytes, "ms_per_launch": g_ms,
                "one_row_frac": g_bytes / (g1_ms * 1e-3) * 1e-9 / hbm_peak,
                # whole forwards (every kernel of the walk), worst round of the run, algorithmic bytes: the target quantity
                "forward_draft_frac": fdist["draft_frac"]["min"] if fdist["draft_frac"] else None,
                "forward_verify_frac": fdist["verify_frac"]["min"] if fdist["verify_frac"] else None,
                "forward_draft_frac_stored_bytes": fdist_stored["draft_frac"]["min"] if fdist_stored["draft_frac"] else None,
                "forward_verify_frac_stored_bytes": fdist_stored["verify_frac"]["min"] if fdist_stored["verify_frac"] else None}

    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
           "ms_per_step": tot_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
           "dtype": "bf16" if cfg.dtype == "bf16" else "f32", "data": "synthetic",
           "config": config_of(desc, args.kv_dtype),
           "vanilla_tokens_per_s": vanilla, "swift_equals_vanilla": lossless, "speedup_vs_vanilla": value / world / vanilla,
           "M": (s0.tokens - 1) / s0.rounds, "alpha": s0.accepted / max(s0.drafted, 1), "rounds": s0.rounds,
           "ms_prefill": s0.ms_prefill, "forwards": fw, "forwards_per_round": fdist, "forwards_per_round_stored_bytes": fdist_stored, "roofline": roofline,
           "e2e": {"value": e2e, "unit": UNIT, "h2d_bytes_per_step": s0.h2d_bytes, "d2h_bytes_per_step": s0.d2h_bytes},
           "gpu_launches": launches, "clocks": clk.summary()}

    if cfg.dtype == "bf16" and cfg.head_dim == 128:
        # Prefill runs in 128-row chunks through the many-row form of the GEMM: tensor work, two bf16 products (hi and lo
        # activation planes) per weight of every block per prompt token (the output head sees one row only).
        pf_flops = 2 * 2.0 * run.prompt_len * cfg.n_blocks * cfg.block_params()
        pf_tflops = pf_flops / (s0.ms_prefill * 1e-3) * 1e-12
        out["prefill"] = {"ms": s0.ms_prefill, "tokens": run.prompt_len, "bound": "tensor (128 rows per weight tile, hi and lo bf16 products)",
                          "tflops_hi_lo": pf_tflops, "peak_tflops": tensor_peak, "frac": pf_tflops / tensor_peak}

    # Dynamic verification (Section 4.2): the same run with the skip set the main run ended with, verifying the chain alone
    # and verifying a token tree of up to 16 rows (greedy decoding only)
    if not sampling and run.max_draft > 0:
        import dataclasses
        gp_fix = dataclasses.replace(gp, skip_mask=z_final, n_opt_rounds=0)
        c_tok, c_st, _ = model.generate(prompt, gp_fix)
        model.set_tree(16)
        t_tok, t_st, _ = model.generate(prompt, gp_fix)
        model.set_tree(0)
        out["dynamic_verification"] = {
            "tree_rows": 16, "M_chain": (c_st.tokens - 1) / c_st.rounds, "M_tree": (t_st.tokens - 1) / t_st.rounds,
            "tokens_per_s_chain": (c_st.tokens - 1) / (c_st.ms_decode * 1e-3), "tokens_per_s_tree": (t_st.tokens - 1) / (t_st.ms_decode * 1e-3),
            "alpha_chain": c_st.accepted / max(c_st.drafted, 1), "tree_equals_vanilla": t_tok == v_tokens,
            "tokens_differing_from_vanilla": sum(int(a != b) for a, b in zip(t_tok, v_tokens))}

    # Candidate scoring (Eq. 2-3), for every shape: one round of the workload's candidate count on the last gamma generated
    # tokens of the run that just ended, timed with CUDA events on the library's stream.  Bytes: what the method needs if
    # every kept sub-layer's weights are streamed once per candidate (each candidate is one draft-model forward of gamma rows).
    n_cand = run.n_candidates
    probe = synth.candidate_masks(cfg, max(1, run.n_skip_blocks), n_cand, 0)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    model.score_skipsets(probe[:2], run.gamma)                       # warm-up
    with torch.cuda.stream(model.stream):
        ev0.record(model.stream)
        model.score_skipsets(probe, run.gamma)
        ev1.record(model.stream)
    torch.cuda.synchronize()
    ms_round = ev0.elapsed_time(ev1)
    n_end = run.prompt_len + max_new
    sc_bytes = sum(model.forward_bytes(probe[c], run.gamma, n_end - run.gamma) for c in range(n_cand))
    sc_gbs = sc_bytes / (ms_round * 1e-3) * 1e-9
    # With the candidates side by side (128 rows per GEMM launch) a round is tensor work: two bf16 products (hi and lo
    # activation planes) per weight of every kept sub-layer and of the output head, per row.
    shp = cfg.shapes()
    p_attn = sum(int(np.prod(shp[k])) for k in ("wq", "wk", "wv", "wo"))
    p_mlp = sum(int(np.prod(shp[k])) for k in ("wgate", "wup", "wdown"))
    kept = lambda c: sum((p_mlp if i % 2 else p_attn) for i in range(2 * cfg.n_blocks) if not probe[c][i])
    sc_flops = sum(2 * 2.0 * run.gamma * (kept(c) + cfg.vocab * cfg.d_model) for c in range(n_cand))
    sc_tflops = sc_flops / (ms_round * 1e-3) * 1e-12
    out["scoring"] = {"candidates_per_round": n_cand, "gamma": run.gamma, "ms_per_round": ms_round,
                      "bound": "tensor (candidates side by side: 128 rows per weight tile, hi and lo bf16 products)",
                      "tflops_hi_lo": sc_tflops, "peak_tflops": tensor_peak, "frac": sc_tflops / tensor_peak,
                      "gbs_if_streamed_per_candidate": sc_gbs, "frac_hbm_if_streamed_per_candidate": sc_gbs / hbm_peak,
                      "vs_one_vanilla_step": ms_round / (1e3 / vanilla)}
    if run.optimise:
        # the optimisation phase as it went over the warm-up and timed steps (step 0 is config 3 as written: one input,
        # from the uniform pattern, its optimisation rounds inside its decode time)
        out["optimisation"] = {"steps": opt_log, "rounds_total": sum(x["opt_rounds"] for x in opt_log),
                               "converged_at_step": next((i for i, x in enumerate(opt_log) if x["best_matchness"] > run.stop_matchness), None),
                               "first_step_tokens_per_s": opt_log[0]["tokens_per_s"] if opt_log else None,
                               "skipped_blocks": [int(b) for b in range(cfg.n_blocks) if z_final[2 * b] and z_final[2 * b + 1]],
                               "planted_blocks": synth.planted_blocks(cfg)}
    if run.optimise and s0.opt_rounds > 0:
        out["scoring"].update({"opt_rounds": s0.opt_rounds, "ms_per_round_in_run": s0.ms_score / s0.opt_rounds,
                               "best_matchness": s0.best_matchness, "share_of_decode": s0.ms_score / s0.ms_decode})
    if c_meas is not None:
        M_, a_ = out["M"], out["alpha"]
        out["eq5"] = {"c_measured": c_meas, "expected_speedup": M_ * a_ / ((M_ - 1) * c_meas + a_) if a_ > 0 else None,
                      "achieved_speedup": out["speedup_vs_vanilla"]}

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        model.close()
        small, zz, w, scale = oracle_model(cfg, run, z, weights)
        torch.set_num_threads(os.cpu_count() or 1)
        n_ctx = run.prompt_len + max_new
        s = oracle_sample(small, run, zz, w, n_ctx)
        out["cpu_baseline"] = {"value": s["swift"] * scale, "unit": UNIT, "cores": torch.get_num_threads(), "kind": "oracle",
                               "vanilla_value": s["vanilla"] * scale, "sample": sample_text(cfg, small, run, n_ctx, s["seconds"])}
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
