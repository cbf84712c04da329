"""Pins for the oracle's SWIFT steps: what the paper and the mathematics fix, independent of the oracle."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

import synth
from oracle import swift_oracle as so

HERE = os.path.dirname(os.path.abspath(__file__))


def _oracle(cfg, weights, max_positions=160):
    return so.Oracle(so.Shape.of(cfg), weights, dtype=torch.float64, max_positions=max_positions)


def _masks(cfg):
    L = 2 * cfg.n_blocks
    rng = np.random.default_rng(5)
    out = [[0] * L, [1] * L, list(synth.block_mask(cfg, synth.planted_blocks(cfg)))]
    out += [list(rng.integers(0, 2, L)) for _ in range(3)]          # sub-layer granularity
    return out


# ------------------------------------------------------------------------------ losslessness
@pytest.mark.parametrize("stop_conf", [0.0, 0.05])
def test_greedy_swift_equals_vanilla_for_every_skip_set(small_cfg, small_weights, stop_conf):
    """Section 3.1: verification by the full model keeps the output unchanged, whatever z is."""
    prompt = synth.prompt(small_cfg, 9)
    ref, _ = so.vanilla_generate(_oracle(small_cfg, small_weights), prompt, 25)
    for z in _masks(small_cfg):
        out, rounds, stats = so.swift_generate(_oracle(small_cfg, small_weights), prompt, z,
                                               so.GenParams(max_new=25, max_draft=4, stop_conf=stop_conf))
        assert out == ref, z
        assert len(out) == 25 and stats["tokens"] == 25
        assert sum(r.accepted + 1 for r in rounds) == 24          # first token comes from prefill


def test_empty_skip_set_accepts_everything(small_cfg, small_weights):
    """z = 0 makes the draft model the target itself: alpha = 1, every round accepts all k."""
    prompt = synth.prompt(small_cfg, 9)
    _, rounds, stats = so.swift_generate(_oracle(small_cfg, small_weights), prompt, [0] * 8,
                                         so.GenParams(max_new=21, max_draft=4))
    assert stats["alpha"] == 1.0 and all(r.accepted == len(r.draft) for r in rounds)
    assert [len(r.draft) for r in rounds] == [4, 4, 4, 4]        # 1 + 4*(4+1) = 21
    assert abs(stats["M"] - 5.0) < 1e-12


def test_exactly_zero_planted_blocks_are_free_to_skip(small_cfg):
    """With the planted residual branches scaled to exactly 0, skipping them changes nothing."""
    cfg = synth.ModelConfig(**{**small_cfg.__dict__, "planted_scale": 0.0})
    w = synth.make_weights(cfg)
    z = list(synth.block_mask(cfg, synth.planted_blocks(cfg)))
    assert sum(z) == 4
    prompt = synth.prompt(cfg, 40)
    o = _oracle(cfg, w)
    _, rounds, stats = so.swift_generate(o, prompt, z, so.GenParams(max_new=41, max_draft=3))
    assert stats["alpha"] == 1.0
    scores, _ = o.score_skipsets([z, [0] * 8], 32)
    assert scores == [1.0, 1.0]


def test_early_stop_keeps_the_low_confidence_token(small_cfg, small_weights):
    o = _oracle(small_cfg, small_weights)
    o.prefill(synth.prompt(small_cfg, 9))
    toks, confs, _ = o.draft([0] * 8, 6, stop_conf=2.0)           # every confidence is below 2
    assert len(toks) == 1 and len(confs) == 1
    toks, confs, _ = o.draft([0] * 8, 6, stop_conf=0.0)
    assert len(toks) == 6 and all(0.0 < c <= 1.0 for c in confs)


def test_kv_after_rollback_equals_fresh_prefill(small_cfg, small_weights):
    """After accept + rollback, cached K,V of the kept positions are the full model's."""
    prompt = synth.prompt(small_cfg, 9)
    z = [1, 1, 0, 0, 1, 0, 0, 1]
    o = _oracle(small_cfg, small_weights)
    so.swift_generate(o, prompt, z, so.GenParams(max_new=17, max_draft=4))
    fresh = _oracle(small_cfg, small_weights)
    fresh.forward_rows(o.tokens[:o.n], 0)
    for b in range(small_cfg.n_blocks):
        assert torch.allclose(o.K[b][:o.n], fresh.K[b][:o.n], atol=1e-10)
        assert torch.allclose(o.V[b][:o.n], fresh.V[b][:o.n], atol=1e-10)


# ------------------------------------------------------------------------------ matchness (Eq. 2-3)
def test_matchness_by_brute_force(small_cfg, small_weights):
    """Eq. 2: y'_i is the draft model's prediction for context token i given the true prefix.
    Brute force: gamma separate passes, each over the whole sequence up to that token, where the
    prefix before the window uses the full model's K,V and the window uses the draft's."""
    prompt = synth.prompt(small_cfg, 12)
    o = _oracle(small_cfg, small_weights)
    so.vanilla_generate(o, prompt, 12)
    gamma, n, T = 8, o.n, o.tokens
    masks = _masks(small_cfg)
    scores, preds = o.score_skipsets(masks, gamma)
    assert scores[0] == 1.0                                        # empty set reproduces the model
    assert all(abs(s * gamma - round(s * gamma)) < 1e-12 and 0.0 <= s <= 1.0 for s in scores)
    for z, s, pr in zip(masks, scores, preds):
        hits = 0
        for i in range(gamma):
            b = _oracle(small_cfg, small_weights)
            b.forward_rows(T[:n - gamma], 0)                       # target K,V for the prefix
            row = b.forward_rows(T[n - gamma:n - gamma + i + 1], n - gamma, z)[-1]
            y = int(torch.argmax(row))
            assert y == pr[i]
            hits += int(y == T[n - gamma + i + 1])
        assert abs(hits / gamma - s) < 1e-12


def test_optimisation_keeps_strictly_better_candidates(small_cfg, small_weights):
    """Section 4.1: the highest-scoring set is retained.  The set in use is scored on the same window as the
    proposals (entry 0) and is replaced only by a proposal that beats it there; earliest among equals."""
    prompt = synth.prompt(small_cfg, 8)
    cands = lambda r: synth.candidate_masks(small_cfg, 2, 4, r)
    gp = so.GenParams(max_new=30, max_draft=3, gamma=8, max_opt_rounds=3, stop_matchness=2.0)
    z0 = list(synth.block_mask(small_cfg, synth.uniform_blocks(4, 2)))
    out, rounds, _ = so.swift_generate(_oracle(small_cfg, small_weights), prompt, z0, gp, cands)
    ref, _ = so.vanilla_generate(_oracle(small_cfg, small_weights), prompt, 30)
    assert out == ref
    scored = [r for r in rounds if r.matchness is not None]
    assert len(scored) == 3 and all(len(r.matchness) == 5 for r in scored)
    z = z0
    for i, r in enumerate(scored):
        pool = [z] + [list(m) for m in cands(i)]
        best = max(r.matchness)
        z = pool[r.matchness.index(best)]                         # lowest index among equals; index 0 = the set in use
        assert r.z == z
    assert rounds[-1].z == z
    first = rounds.index(scored[0])
    assert all(r.z == z0 for r in rounds[:first])


def test_optimisation_never_drops_a_set_no_proposal_beats(small_cfg):
    """With the planted residual branches scaled to exactly 0 the planted set re-predicts every context token
    (matchness 1), so no proposal can score strictly higher: it must survive every optimisation round, and a
    run that starts elsewhere must not end on anything worse than what it held on the way."""
    cfg = synth.ModelConfig(**{**small_cfg.__dict__, "planted_scale": 0.0})
    w = synth.make_weights(cfg)
    planted = list(synth.block_mask(cfg, synth.planted_blocks(cfg)))
    prompt = synth.prompt(cfg, 10)
    cands = lambda r: synth.candidate_masks(cfg, 2, 6, r)
    gp = so.GenParams(max_new=40, max_draft=3, gamma=8, max_opt_rounds=4, stop_matchness=2.0)
    _, rounds, stats = so.swift_generate(_oracle(cfg, w), prompt, planted, gp, cands)
    scored = [r for r in rounds if r.matchness is not None]
    assert len(scored) == 4 and all(r.matchness[0] == 1.0 for r in scored)
    assert all(r.z == planted for r in rounds) and stats["alpha"] == 1.0
    # patience: two rounds in a row without a replacement end the optimisation
    gp2 = so.GenParams(max_new=40, max_draft=3, gamma=8, max_opt_rounds=4, stop_matchness=2.0, patience=2)
    _, rounds2, _ = so.swift_generate(_oracle(cfg, w), prompt, planted, gp2, cands)
    assert sum(r.matchness is not None for r in rounds2) == 2
    # the score threshold ends it after the first round (1.0 > 0.95)
    gp3 = so.GenParams(max_new=40, max_draft=3, gamma=8, max_opt_rounds=4)
    _, rounds3, _ = so.swift_generate(_oracle(cfg, w), prompt, planted, gp3, cands)
    assert sum(r.matchness is not None for r in rounds3) == 1


# ------------------------------------------------------------------------------ sampling acceptance
def _first_token_histogram(p, q, trials, seed, one_hot_draft=False):
    V = p.numel()
    counts = np.zeros(V)
    accepted = 0
    tl = torch.log(p)[None].repeat(2, 1)
    for t in range(trials):
        y = so.categorical(q, so.uniform(seed, t, 1, so.DRAW_DRAFT))[0]
        a, nxt, _ = so.accept_sampling([y], [q], tl, 1.0, seed, t)
        accepted += a
        counts[y if a == 1 else nxt] += 1
    return counts, accepted


@pytest.mark.parametrize("case", ["generic", "q_with_zeros", "one_hot_q", "p_equals_q"])
def test_speculative_sampling_reproduces_target_distribution(case):
    """The acceptance rule must leave the emitted token distributed exactly as p (chi-squared), and
    accept with probability sum_i min(p_i, q_i)."""
    g = torch.Generator().manual_seed(3)
    V = 12
    p = torch.softmax(torch.randn(V, generator=g, dtype=torch.float64) * 1.5, 0)
    q = torch.softmax(torch.randn(V, generator=g, dtype=torch.float64) * 1.5, 0)
    if case == "q_with_zeros":
        q[::3] = 0
        q /= q.sum()
    elif case == "one_hot_q":
        q = torch.zeros(V, dtype=torch.float64)
        q[int(torch.argmax(p))] = 1.0
    elif case == "p_equals_q":
        q = p.clone()
    trials = 100_000
    counts, accepted = _first_token_histogram(p, q, trials, seed=17)
    expect = p.numpy() * trials
    chi2 = float(((counts - expect) ** 2 / expect).sum())
    assert chi2 < 40.0, chi2                    # 11 dof: P(chi2 > 40) ~ 3e-5
    rate = float(torch.minimum(p, q).sum())
    assert abs(accepted / trials - rate) < 5.0 * np.sqrt(max(rate * (1 - rate), 1e-9) / trials) + 1e-12
    if case == "p_equals_q":
        assert accepted == trials


# ------------------------------------------------------------------------------ nucleus (top-p) filtering
def test_nucleus_worked_example_and_limits():
    """By hand: p = (0.5, 0.3, 0.15, 0.05).  top_p 0.9 needs three tokens (0.8 < 0.9 <= 0.95); top_p 0.5 is reached
    by the first token alone; top_p 1 changes nothing; a tiny top_p leaves the arg max (greedy)."""
    p = torch.tensor([0.15, 0.5, 0.05, 0.3], dtype=torch.float64)
    f, margin = so.nucleus(p, 0.9)
    assert torch.allclose(f, torch.tensor([0.15, 0.5, 0.0, 0.3], dtype=torch.float64) / 0.95)
    assert margin == pytest.approx(0.05)                      # 0.95 - 0.9; the other side (0.8) is 0.1 away
    assert torch.allclose(so.nucleus(p, 0.5)[0], torch.tensor([0.0, 1.0, 0.0, 0.0], dtype=torch.float64))
    assert torch.allclose(so.nucleus(p, 0.51)[0], torch.tensor([0.0, 0.625, 0.0, 0.375], dtype=torch.float64))
    assert so.nucleus(p, 1.0)[0] is p
    assert torch.equal(so.nucleus(p, 1e-9)[0], torch.tensor([0.0, 1.0, 0.0, 0.0], dtype=torch.float64))
    # equal probabilities are kept together
    t = torch.tensor([0.4, 0.2, 0.2, 0.2], dtype=torch.float64)
    assert torch.allclose(so.nucleus(t, 0.5)[0], t)


def test_nucleus_is_the_smallest_set_of_most_probable_tokens_by_brute_force():
    """Among all token subsets whose mass reaches top_p, the kept set is one of minimum size, and of those the one
    of maximum mass (checked by enumerating every subset of a 10-token vocabulary)."""
    import itertools
    g = torch.Generator().manual_seed(8)
    for trial in range(20):
        p = torch.softmax(torch.randn(10, generator=g, dtype=torch.float64) * 1.3, 0)
        top_p = float(torch.rand(1, generator=g, dtype=torch.float64)) * 0.98 + 0.01
        f, _ = so.nucleus(p, top_p)
        kept = set(torch.nonzero(f).flatten().tolist())
        best = None
        for size in range(1, 11):
            ok = [c for c in itertools.combinations(range(10), size) if float(p[list(c)].sum()) >= top_p]
            if ok:
                best = set(max(ok, key=lambda c: float(p[list(c)].sum())))
                break
        assert kept == best, (trial, top_p)
        assert torch.allclose(f[list(kept)], p[list(kept)] / p[list(kept)].sum())


def test_nucleus_keeps_the_tokens_huggingface_keeps():
    """The library the paper ran (Appendix B.2) filters with TopPLogitsWarper: same kept set on random logits."""
    from transformers.generation.logits_process import TopPLogitsWarper
    g = torch.Generator().manual_seed(12)
    for top_p in (0.95, 0.6, 0.3):
        logits = torch.randn(5, 300, generator=g, dtype=torch.float64) * 2.0
        warped = TopPLogitsWarper(top_p=top_p)(None, logits.clone())
        for r in range(5):
            f, margin = so.nucleus(torch.softmax(logits[r], -1), top_p)
            if margin > 1e-9:
                assert torch.equal(f > 0, torch.isfinite(warped[r])), (top_p, r)


def test_speculative_sampling_with_nucleus_reproduces_the_filtered_target():
    """With top_p < 1 the emitted token must follow nucleus(p) (tokens outside it never appear), whatever q."""
    g = torch.Generator().manual_seed(5)
    V, top_p, trials, seed = 12, 0.8, 60_000, 23
    p = torch.softmax(torch.randn(V, generator=g, dtype=torch.float64) * 1.5, 0)
    q_full = torch.softmax(torch.randn(V, generator=g, dtype=torch.float64) * 1.5, 0)
    pf, q = so.nucleus(p, top_p)[0], so.nucleus(q_full, top_p)[0]
    assert 0 < int((pf == 0).sum()) < V - 1
    tl = torch.log(p)[None].repeat(2, 1)
    counts = np.zeros(V)
    for t in range(trials):
        y = so.categorical(q, so.uniform(seed, t, 1, so.DRAW_DRAFT))[0]
        a, nxt, _ = so.accept_sampling([y], [q], tl, 1.0, seed, t, top_p)
        counts[y if a == 1 else nxt] += 1
    assert counts[(pf == 0).numpy()].sum() == 0
    live = (pf > 0).numpy()
    expect = pf.numpy()[live] * trials
    chi2 = float(((counts[live] - expect) ** 2 / expect).sum())
    assert chi2 < 40.0, chi2


def test_wrong_acceptance_rules_fail_the_chi_squared():
    """Guard on the guard: always accepting the draft gives q, not p, and the statistic explodes."""
    g = torch.Generator().manual_seed(3)
    p = torch.softmax(torch.randn(12, generator=g, dtype=torch.float64) * 1.5, 0)
    q = torch.softmax(torch.randn(12, generator=g, dtype=torch.float64) * 1.5, 0)
    trials = 20_000
    counts = np.zeros(12)
    for t in range(trials):
        counts[so.categorical(q, so.uniform(1, t, 1, so.DRAW_DRAFT))[0]] += 1
    expect = p.numpy() * trials
    assert float(((counts - expect) ** 2 / expect).sum()) > 200.0


@pytest.mark.parametrize("greedy_draft", [False, True], ids=["sampled_drafts", "argmax_drafts"])
def test_whole_round_sampling_is_lossless_on_a_tiny_model(greedy_draft):
    """Second emitted token of SWIFT in sampling mode: its law, given the first token, is the target's, whether the
    drafts are drawn from the draft distribution or chosen by arg max (Eq. 4) with a point-mass q."""
    cfg = synth.ModelConfig("micro", n_blocks=2, d_model=16, n_heads=2, n_kv_heads=1, head_dim=8, ffn=24,
                            vocab=6, dtype="f32", seed=5, n_planted=1, init_std=0.6)
    w = synth.make_weights(cfg)
    prompt = synth.prompt(cfg, 4)
    z = [0, 1, 1, 0]
    base = _oracle(cfg, w, 32)
    l0 = base.prefill(prompt)[-1]
    p1 = torch.softmax(l0, 0)
    # exact law of token 2 under the target: sum_t1 p(t1) p(t2 | t1)
    law = torch.zeros(cfg.vocab, dtype=torch.float64)
    for t1 in range(cfg.vocab):
        b = _oracle(cfg, w, 32)
        b.prefill(prompt, first_token=t1)
        law += p1[t1] * torch.softmax(b.forward_rows([t1], b.n)[0], 0)
    trials = 6000
    counts = np.zeros(cfg.vocab)
    for t in range(trials):
        out, _, _ = so.swift_generate(_oracle(cfg, w, 32), prompt, z,
                                      so.GenParams(max_new=3, max_draft=2, mode="sampling", rng_seed=1000 + t,
                                                   greedy_draft=greedy_draft))
        counts[out[1]] += 1
    expect = law.numpy() * trials
    chi2 = float(((counts - expect) ** 2 / expect).sum())
    assert chi2 < 30.0, chi2                    # 5 dof: P(chi2 > 30) ~ 1.5e-5


def test_categorical_is_inverse_cdf_in_index_order():
    w = torch.tensor([0.0, 2.0, 0.0, 1.0, 1.0], dtype=torch.float64)
    assert so.categorical(w, 0.0)[0] == 1
    assert so.categorical(w, 0.49)[0] == 1
    assert so.categorical(w, 0.51)[0] == 3
    assert so.categorical(w, 0.76)[0] == 4
    assert so.categorical(w, 1.0 - 2 ** -24)[0] == 4


def test_greedy_accept_prefix_rule():
    V = 5
    tl = torch.full((4, V), -1.0, dtype=torch.float64)
    for r, t in enumerate([2, 4, 1, 3]):
        tl[r, t] = 1.0
    assert so.accept_greedy([2, 4, 1], tl) == (3, 3)             # all accepted, bonus from last row
    assert so.accept_greedy([2, 0, 1], tl) == (1, 4)             # later matches do not count
    assert so.accept_greedy([0, 4, 1], tl) == (0, 2)
    tl[0, 0] = 1.0                                               # tie: lowest id wins
    assert so.accept_greedy([0], tl[:2]) == (1, 4)


# ------------------------------------------------------------------------------ Philox, Eq. 5
def test_philox_matches_an_independent_library_implementation():
    """Triton ships Philox4x32-10 as tl.philox_impl; its CPU interpreter evaluates it without a GPU."""
    pytest.importorskip("triton")
    rng = np.random.default_rng(0)
    cases = [[0] * 6, [0xFFFFFFFF] * 6] + [list(map(int, rng.integers(0, 2 ** 32, 6))) for _ in range(6)]
    code = r"""
import sys, json, torch, triton, triton.language as tl
@triton.jit
def k(out, c0, c1, c2, c3, k0, k1):
    a = tl.full((1,), 0, tl.uint32)
    r0, r1, r2, r3 = tl.philox_impl(a + c0, a + c1, a + c2, a + c3, a + k0, a + k1, 10)
    i = tl.arange(0, 1)
    tl.store(out + i, r0); tl.store(out + 1 + i, r1); tl.store(out + 2 + i, r2); tl.store(out + 3 + i, r3)
res = []
for c in json.loads(sys.argv[1]):
    o = torch.zeros(4, dtype=torch.int32)
    k[(1,)](o, *[torch.tensor([v], dtype=torch.int64).to(torch.int32).item() if v < 2**31 else v - 2**32 for v in c])
    res.append([int(x) & 0xFFFFFFFF for x in o])
print(json.dumps(res))
"""
    import json
    env = dict(os.environ, TRITON_INTERPRET="1")
    r = subprocess.run([sys.executable, "-c", code, json.dumps(cases)], capture_output=True, text=True, env=env,
                       timeout=600)
    if r.returncode != 0:
        pytest.skip("triton interpreter unavailable: " + r.stderr[-300:])
    ref = json.loads(r.stdout.strip().splitlines()[-1])
    for c, want in zip(cases, ref):
        assert list(so.philox4x32_10(c[:4], c[4:])) == want
        assert list(synth.philox4x32_10(c[:4], c[4:])) == want


def test_uniform_is_24_bit_and_in_range():
    us = [so.uniform(9, r, 1, so.DRAW_ACCEPT) for r in range(2000)]
    assert all(0.0 <= u < 1.0 and (u * 2 ** 24).is_integer() for u in us)
    assert abs(np.mean(us) - 0.5) < 0.03
    assert so.uniform(9, 1, 1, so.DRAW_ACCEPT) != so.uniform(9, 1, 1, so.DRAW_RESAMPLE)


def test_expected_speedup_matches_table_5():
    """Eq. 5 evaluated at the (M, alpha, c) triples of Table 5 gives the speedups printed there."""
    rows = [l.split() for l in open(os.path.join(HERE, "golden", "table5_expected_speedup.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 9
    for *_, M, alpha, c, printed in rows:
        assert abs(so.expected_speedup(float(M), float(alpha), float(c)) - float(printed)) < 0.0051
    assert so.expected_speedup(1.0, 0.7, 0.55) == 1.0            # one token per round: no gain, no loss


# ------------------------------------------------------------------------------ dynamic verification (token tree)
def test_tree_width_bins_are_the_papers():
    """Section 4.2: k = 10, 5, 3, 1 for p in (0, 0.5], (0.5, 0.8], (0.8, 0.95], (0.95, 1]."""
    for p, k in ((1e-6, 10), (0.3, 10), (0.5, 10), (0.5000001, 5), (0.8, 5), (0.81, 3), (0.95, 3), (0.9500001, 1), (1.0, 1)):
        assert so.tree_width(p) == k, p


def test_tree_shape_and_row_budget():
    rows = [torch.tensor([0.0, 5.0, 4.0, 3.0, 2.0, 1.0, 0.5, 0.4, 0.3, 0.2, 0.1, -1.0]),
            torch.tensor([9.0, 1.0, 8.0, 7.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0])]
    tree = so.build_tree(7, [1, 0], rows, [0.7, 0.9], row_budget=64)           # widths 5 and 3
    assert tree.tokens == [7, 1, 0, 2, 3, 4, 5, 2, 3]                           # chain first, then alternatives depth by depth
    assert tree.depth == [0, 1, 2, 1, 1, 1, 1, 2, 2]
    assert tree.parent == [-1, 0, 1, 0, 0, 0, 0, 1, 1]
    sees = tree.sees()
    assert sees[2].tolist() == [True, True, True] + [False] * 6                 # y'_2 sees t*, y'_1, itself
    assert sees[4].tolist() == [True, False, False, False, True, False, False, False, False]   # an alternative of y'_1: t* and itself
    assert sees[8].tolist() == [True, True, False, False, False, False, False, False, True]    # an alternative of y'_2: t*, y'_1, itself
    tight = so.build_tree(7, [1, 0], rows, [0.7, 0.9], row_budget=5)           # 3 chain rows + 2: the first position takes both
    assert tight.tokens == [7, 1, 0, 2, 3] and tight.depth == [0, 1, 2, 1, 1]
    assert so.build_tree(7, [1, 0], rows, [0.99, 0.96], row_budget=64).tokens == [7, 1, 0]     # confident drafts: the chain alone
    # equal logits rank by token id
    assert so.ranked_tokens(torch.tensor([1.0, 3.0, 3.0, 2.0, 3.0]), 4) == [1, 2, 4, 3]


def test_tree_rows_equal_separate_causal_forwards(small_cfg, small_weights):
    """Brute force: verifying the linearised tree in one masked forward gives every node the logits a plain causal
    forward over its root-to-node path gives."""
    o = _oracle(small_cfg, small_weights)
    o.prefill(synth.prompt(small_cfg, 11))
    z = [1, 1, 0, 0, 1, 0, 0, 1]
    d_tok, d_conf, d_rows = o.draft(z, 4)
    tree = so.build_tree(o.tokens[-1], d_tok, d_rows, [0.4, 0.7, 0.9, 0.99], row_budget=32)    # widths 10, 5, 3, 1
    assert len(tree.tokens) == 5 + 9 + 4 + 2
    tl = o.verify_tree(tree)
    for node in range(len(tree.tokens)):
        path = []
        j = node
        while j >= 0:
            path.append(j)
            j = tree.parent[j]
        path.reverse()
        b = _oracle(small_cfg, small_weights)
        b.forward_rows(o.tokens[:o.n], 0)
        ref = b.forward_rows([tree.tokens[r] for r in path], o.n, write_kv=False)[-1]
        assert torch.allclose(tl[node], ref, atol=1e-9, rtol=0), node


@pytest.mark.parametrize("stop_conf", [0.0, 0.05])
def test_tree_verification_is_lossless_and_never_shorter(small_cfg, small_weights, stop_conf):
    """Section 3.1 / 4.2: with the tree every emitted token is still the target's arg max, so the output equals
    vanilla greedy decoding for every skip set; and from the same state a tree round accepts at least as many
    tokens as the chain alone."""
    prompt = synth.prompt(small_cfg, 9)
    ref, _ = so.vanilla_generate(_oracle(small_cfg, small_weights), prompt, 30)
    gains = 0
    for z in _masks(small_cfg):
        o = _oracle(small_cfg, small_weights)
        out, rounds, stats = so.swift_generate(o, prompt, z, so.GenParams(max_new=30, max_draft=4, stop_conf=stop_conf, tree_rows=16))
        assert out == ref and len(out) == 30, z
        fresh = _oracle(small_cfg, small_weights)
        fresh.forward_rows(o.tokens[:o.n], 0)
        for b in range(small_cfg.n_blocks):                       # accepted alternatives were moved to their slots
            assert torch.allclose(o.K[b][:o.n], fresh.K[b][:o.n], atol=1e-10) and torch.allclose(o.V[b][:o.n], fresh.V[b][:o.n], atol=1e-10)
        for r in rounds:
            assert len(r.tree.tokens) <= max(16, len(r.draft) + 1) and r.tree.tokens[1:len(r.draft) + 1] == r.draft
            chain_a, _ = so.accept_greedy(r.draft, torch.stack([torch.nn.functional.one_hot(torch.tensor(t), small_cfg.vocab).double()
                                                                for t in r.target_argmax[:len(r.draft) + 1]]))
            assert r.accepted >= chain_a
            gains += r.accepted - chain_a
    assert gains > 0                                              # some alternative was accepted somewhere
