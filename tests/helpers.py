"""Shared by the GPU parity tests: build the same synthetic model on both sides and walk them in step."""
from __future__ import annotations

from typing import List, Sequence

import numpy as np
import torch

import synth
from oracle import swift_oracle as so

LOGIT_TOL = 2e-2        # max |dlogit| / std(oracle row)
MARGIN = 0.05           # tokens must agree wherever the oracle's top-1/top-2 gap exceeds this


def make_pair(cfg, max_positions=256, page_size=16, max_draft=15, oracle_dtype=None, kv_dtype="f32", widen=True):
    """(oracle, gpu model) over identical synthetic weights.  widen=False keeps the oracle's copy in the storage type
    (it widens a tensor whenever it applies it): half the host memory of an fp32 copy, for the multi-billion shapes."""
    from paper_2410_06916_b200 import SwiftModel
    w = synth.make_weights(cfg)
    gpu = SwiftModel(cfg, max_positions=max_positions, page_size=page_size, max_draft=max_draft, kv_dtype=kv_dtype)
    gpu.pack("embed", -1, w["embed"]); gpu.pack("lm_head", -1, w["lm_head"]); gpu.pack("final_norm", -1, w["final_norm"])
    for b, wb in enumerate(w["blocks"]):
        for name, t in wb.items():
            gpu.pack(name, b, t)
    if oracle_dtype is None:
        oracle_dtype = torch.float64 if cfg.dtype == "f32" else torch.float32
    if cfg.dtype == "bf16" and widen:    # widen once (exact) so the oracle does not convert on every call
        w = {k: (v.to(oracle_dtype) if torch.is_tensor(v) else [{n: t.to(oracle_dtype) for n, t in blk.items()} for blk in v])
             for k, v in w.items()}
    o = so.Oracle(so.Shape.of(cfg), w, dtype=oracle_dtype, max_positions=max_positions)
    return o, gpu


class LazyBlocks:
    """Per-block weights generated from the seed when a block is asked for and dropped afterwards, so that the
    oracle can walk a model whose widened weights would not fit host memory (its forward takes each block once)."""

    def __init__(self, cfg):
        self.cfg = cfg
        self.planted = set(synth.planted_blocks(cfg))

    def __len__(self):
        return self.cfg.n_blocks

    def __getitem__(self, b):
        return _LazyBlock(self.cfg, b, b in self.planted)


class _LazyBlock:
    """One block's tensors, each generated when it is asked for (a skipped sub-layer's weights never are)."""

    def __init__(self, cfg, b, planted):
        self.cfg, self.b, self.planted = cfg, b, planted

    def __getitem__(self, name):
        return synth.make_tensor(self.cfg, name, self.b, planted=self.planted)


def make_streamed_pair(cfg, max_positions=256, page_size=16, max_draft=15, kv_dtype="f32"):
    """(oracle, gpu model) over identical synthetic weights, neither side holding a host copy of the blocks:
    the GPU is filled tensor by tensor, the oracle regenerates a block whenever its forward reaches it."""
    from paper_2410_06916_b200 import SwiftModel
    gpu = SwiftModel(cfg, max_positions=max_positions, page_size=page_size, max_draft=max_draft, kv_dtype=kv_dtype)
    gpu.load_weights(synth.iter_tensors(cfg))
    w = {name: synth.make_tensor(cfg, name) for name in ("embed", "lm_head", "final_norm")}
    w["blocks"] = LazyBlocks(cfg)
    o = so.Oracle(so.Shape.of(cfg), w, dtype=torch.float32, max_positions=max_positions)
    return o, gpu


def logit_err(got: np.ndarray, ref: torch.Tensor) -> float:
    """max over rows of max|got - ref| / std(ref row)."""
    ref = ref.to(torch.float64).numpy()
    got = np.asarray(got, dtype=np.float64)
    return float((np.abs(got - ref).max(axis=-1) / ref.std(axis=-1)).max())


def resync(gpu, o: so.Oracle, rounds_done: int = -1):
    """Put the GPU context in the oracle's committed state (tokens, pending token, round counter)."""
    gpu.prefill(o.tokens[:-1])
    gpu.set_pending(o.tokens[-1], rounds_done)
    assert gpu.n == o.n


def walk_rounds(o: so.Oracle, gpu, z, n_rounds: int, max_k: int, stop_conf: float = 0.0, sampling=False,
                temperature=1.0, seed=0, first_round=1, dec_tol=1e-3, top_p=1.0, greedy_draft=False):
    """Runs n_rounds of draft -> verify -> accept on both sides from the same state and compares every
    intermediate the oracle exposes, exempting only decisions the oracle marks as near a boundary.
    Returns counters for the caller to assert on."""
    stats = dict(rounds=0, draft_cmp=0, draft_exempt=0, accept_cmp=0, accept_exempt=0, resyncs=0, max_logit_err=0.0,
                 accepted=0, drafted=0)
    for r in range(first_round, first_round + n_rounds):
        assert gpu.n == o.n
        q_rows: List[torch.Tensor] = []
        dec_margins: List[float] = []
        if sampling:
            def sampler(j, q, _r=r):
                if greedy_draft:                       # arg max of the draft; q is the point mass on it
                    tok = so.argmax_lowest(q)
                    q_rows.append(so.point_mass(q.numel(), tok))
                    top2 = torch.topk(q, 2).values
                    dec_margins.append(float(top2[0] - top2[1]) / float(top2[0]))   # relative gap of the two best
                    return tok
                q_rows.append(q)
                tok, dist = so.categorical(q, so.uniform(seed, _r, j, so.DRAW_DRAFT))
                dec_margins.append(dist)
                return tok
            d_tok, d_conf, d_rows = o.draft(z, max_k, stop_conf, sampler, temperature, top_p)
        else:
            d_tok, d_conf, d_rows = o.draft(z, max_k, stop_conf)
            dec_margins = [so.top2_margin(x) for x in d_rows]
        g_tok, g_conf = gpu.draft(z, max_k, stop_conf)
        same_draft = True
        for j in range(min(len(d_tok), len(g_tok))):
            near = dec_margins[j] <= (dec_tol if sampling else MARGIN)
            if g_tok[j] != d_tok[j]:
                assert near, f"round {r} draft {j}: gpu {g_tok[j]} oracle {d_tok[j]} margin {dec_margins[j]}"
                stats["draft_exempt"] += 1
                same_draft = False
                break
            stats["draft_cmp"] += 1
            assert abs(g_conf[j] - d_conf[j]) <= 0.02 * d_conf[j] + 1e-6, (g_conf[j], d_conf[j])
        if same_draft and len(g_tok) != len(d_tok):     # early stop decided differently: must be at the threshold
            jj = min(len(g_tok), len(d_tok)) - 1
            assert abs(d_conf[jj] - stop_conf) <= 0.02 * stop_conf + 1e-6
            same_draft = False
        if sampling and not same_draft:
            # the draft distributions kept on the GPU belong to another prefix: start this round over
            tl = o.verify(d_tok)
            a, nxt, _ = so.accept_sampling(d_tok, q_rows, tl, temperature, seed, r, top_p)
            o.commit(d_tok[:a], nxt)
            gpu.verify(); gpu.accept()                  # close the GPU's round on its own drafts, then start over
            resync(gpu, o, r)
            stats["resyncs"] += 1
            continue
        tl = o.verify(d_tok)
        g_am, g_logits = gpu.verify(d_tok)             # teacher-forced with the oracle's drafts
        rows = len(d_tok) + 1
        err = logit_err(g_logits[:rows], tl)
        stats["max_logit_err"] = max(stats["max_logit_err"], err)
        assert err <= LOGIT_TOL, f"round {r}: logits off by {err} sigma"
        t_margin = [so.top2_margin(tl[i]) for i in range(rows)]
        t_am = [so.argmax_lowest(tl[i]) for i in range(rows)]
        for i in range(rows):
            if t_margin[i] > MARGIN:
                assert int(g_am[i]) == t_am[i], f"round {r} row {i}"
        if sampling:
            a, nxt, dec = so.accept_sampling(d_tok, q_rows, tl, temperature, seed, r, top_p)
            exempt = any(d["margin"] <= dec_tol for d in dec)
        else:
            a, nxt = so.accept_greedy(d_tok, tl)
            exempt = any(m <= MARGIN for m in t_margin[:a + 1])
        g_a, g_next = gpu.accept()
        o.commit(d_tok[:a], nxt)
        stats["rounds"] += 1
        stats["accepted"] += a
        stats["drafted"] += len(d_tok)
        if (g_a, g_next) == (a, nxt):
            stats["accept_cmp"] += 1
        else:
            assert exempt, f"round {r}: gpu accepted {g_a}, next {g_next}; oracle {a}, {nxt}"
            stats["accept_exempt"] += 1
            resync(gpu, o, r)
            stats["resyncs"] += 1
    return stats


def compare_free_running(gpu_tokens: Sequence[int], ref_tokens: Sequence[int], ref_margins: Sequence[float]):
    """Free-running sequences must agree up to the first position where the oracle's margin is small."""
    for i, (g, t) in enumerate(zip(gpu_tokens, ref_tokens)):
        if g != t:
            assert ref_margins[i] <= MARGIN, f"token {i}: gpu {g} oracle {t} margin {ref_margins[i]}"
            return i
    return len(ref_tokens)
