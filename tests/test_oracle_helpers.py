"""Pins for the small oracle helpers the GPU parity harness leans on: the top-1/top-2 margin that decides
which token mismatches are exempt, the plain projection that checks the GEMM kernels, the draft confidence
p_j of Section 4.2, and the distances to a decision boundary that speculative-sampling comparisons use.
Every expected value below is worked out by hand or follows from a property, not from the helper's formula."""
import math

import pytest
import torch

import synth
from oracle import swift_oracle as so


# ------------------------------------------------------------------------------ top2_margin
def test_top2_margin_on_hand_written_rows():
    assert so.top2_margin(torch.tensor([1.0, 3.5, 3.0, -2.0])) == pytest.approx(0.5, abs=1e-12)       # best 3.5, runner-up 3.0
    assert so.top2_margin(torch.tensor([2.0, 2.0, 1.0])) == 0.0                                       # a tie
    assert so.top2_margin(torch.tensor([-7.0, -1.0, -4.0])) == pytest.approx(3.0, abs=1e-12)          # all negative
    assert so.top2_margin(torch.tensor([0.0, 10.0, 0.0, 9.75, 0.0])) == pytest.approx(0.25, abs=1e-12)  # not adjacent, not first
    # the runner-up is the second largest entry, not the smallest and not the mean
    assert so.top2_margin(torch.tensor([5.0, 1.0, 4.0, -100.0])) == pytest.approx(1.0, abs=1e-12)
    # fp32 input is widened before the subtraction: 1 + 2^-23 and 1 differ by exactly 2^-23
    row = torch.tensor([1.0 + 2.0 ** -23, 1.0, 0.0], dtype=torch.float32)
    assert so.top2_margin(row) == 2.0 ** -23


def test_top2_margin_is_what_exempts_a_flip():
    """Adding less than the margin to the runner-up keeps the arg max, adding more flips it."""
    g = torch.Generator().manual_seed(3)
    for _ in range(20):
        row = torch.randn(50, generator=g, dtype=torch.float64)
        m = so.top2_margin(row)
        best = so.argmax_lowest(row)
        second = int(torch.topk(row, 2).indices[1])
        lo, hi = row.clone(), row.clone()
        lo[second] += 0.99 * m
        hi[second] += 1.01 * m
        assert so.argmax_lowest(lo) == best and so.argmax_lowest(hi) == second


# ------------------------------------------------------------------------------ linear
def test_linear_is_x_times_w_transposed():
    x = torch.tensor([[1.0, 2.0, 3.0], [0.0, -1.0, 2.0]])                       # [2 rows, 3 inputs]
    W = torch.tensor([[1.0, 0.0, 2.0], [-1.0, 3.0, 1.0], [0.5, 0.5, 0.5], [0.0, 0.0, -1.0]])   # [4 outputs, 3 inputs]
    y = so.linear(x, W)
    assert y.dtype == torch.float64 and tuple(y.shape) == (2, 4)
    # by hand: row 0 = (1+0+6, -1+6+3, 3, -3), row 1 = (0+0+4, 0-3+2, 0.5, -2)
    assert y.tolist() == [[7.0, 8.0, 3.0, -3.0], [4.0, -1.0, 0.5, -2.0]]


def test_linear_widens_bf16_weights_exactly():
    W = torch.tensor([[0.3, -1.7], [2.2, 0.01], [5.0, 9.0]]).to(torch.bfloat16)   # [3 outputs, 2 inputs]
    x = torch.tensor([[1.0, 1.0]])
    y = so.linear(x, W)
    exact = [float(W[i, 0].to(torch.float64) + W[i, 1].to(torch.float64)) for i in range(3)]
    assert y[0].tolist() == exact


# ------------------------------------------------------------------------------ draft confidence (Section 4.2)
class _FixedLogits(so.Oracle):
    """An oracle whose forward returns hand-written logits, so that the drafting bookkeeping can be checked
    without a model in the way."""

    def __init__(self, rows):
        self.rows = [torch.tensor(r, dtype=torch.float64) for r in rows]
        self.calls = 0
        self.tokens, self.n = [0], 5

    def forward_rows(self, row_tokens, pos0, z=None, write_kv=True):
        r = self.rows[self.calls]
        self.calls += 1
        return r[None, :]


@pytest.mark.parametrize("temperature,top_p", [(1.0, 1.0), (0.5, 1.0), (1.0, 0.5), (0.6, 0.95), (2.0, 0.3)])
def test_draft_confidence_is_max_softmax_at_temperature_one(temperature, top_p):
    """p_j = max P(. | ...) of the draft model (Section 4.2): the plain soft-max of the draft's logits, whatever
    temperature and nucleus cut the sampling distributions use.  Logits (0, ln 3): soft-max (1/4, 3/4); at
    temperature 1/2 it would be (1/10, 9/10), after a nucleus cut at 0.5 it would be (0, 1)."""
    rows = [[0.0, math.log(3.0)], [math.log(2.0), 0.0, 0.0]]              # second step: (1/2, 1/4, 1/4)
    o = _FixedLogits(rows)
    picked = []
    toks, confs, _ = o.draft([0, 0], 2, 0.0, sampler=lambda j, q: picked.append(q) or so.argmax_lowest(q),
                             temperature=temperature, top_p=top_p)
    assert confs == pytest.approx([0.75, 0.5], abs=1e-12)
    assert toks == [1, 0]
    # ... while the distribution handed to the sampler does follow the temperature
    if top_p == 1.0:
        w = 3.0 ** (1.0 / temperature)
        assert picked[0].tolist() == pytest.approx([1.0 / (1.0 + w), w / (1.0 + w)], abs=1e-12)
    # greedy drafting reports the same confidences
    o2 = _FixedLogits(rows)
    toks2, confs2, _ = o2.draft([0, 0], 2, 0.0)
    assert toks2 == [1, 0] and confs2 == pytest.approx([0.75, 0.5], abs=1e-12)


def test_early_stop_compares_that_confidence():
    rows = [[0.0, math.log(3.0)], [math.log(2.0), 0.0, 0.0], [0.0, 5.0]]
    assert len(_FixedLogits(rows).draft([0, 0], 3, 0.6)[0]) == 2         # 0.75 >= 0.6 continues, 0.5 < 0.6 stops (token kept)
    assert len(_FixedLogits(rows).draft([0, 0], 3, 0.8)[0]) == 1         # 0.75 < 0.8 stops at once
    assert len(_FixedLogits(rows).draft([0, 0], 3, 0.5)[0]) == 3         # 0.5 is not below 0.5


# ------------------------------------------------------------------------------ categorical: index and distance
def test_categorical_worked_example():
    w = torch.tensor([1.0, 2.0, 1.0])                                     # running sums 1, 3, 4
    i, d = so.categorical(w, 0.3)                                         # 1.2 falls in (1, 3): 0.2 above the lower edge
    assert i == 1 and d == pytest.approx(0.05, abs=1e-12)
    i, d = so.categorical(w, 0.76)                                        # 3.04 falls in (3, 4): 0.04 above the lower edge
    assert i == 2 and d == pytest.approx(0.01, abs=1e-12)
    i, d = so.categorical(w, 0.25)                                        # exactly on an edge: the bin that starts there
    assert i == 1 and d == 0.0
    i, d = so.categorical(w, 0.0)
    assert i == 0 and d == 0.0
    i, d = so.categorical(torch.tensor([0.0, 0.0, 4.0, 0.0]), 0.5)        # empty bins are never drawn
    assert i == 2 and d == pytest.approx(0.5, abs=1e-12)


def test_categorical_distance_bounds_the_shift_that_changes_the_draw():
    g = torch.Generator().manual_seed(8)
    for _ in range(50):
        w = torch.rand(12, generator=g, dtype=torch.float64) + 0.01
        u = float(torch.rand(1, generator=g, dtype=torch.float64)) * 0.98 + 0.01
        i, d = so.categorical(w, u)
        assert so.categorical(w, u + 0.99 * d)[0] == i and so.categorical(w, u - 0.99 * d)[0] == i
        up, down = u + 1.01 * d + 1e-12, u - 1.01 * d - 1e-12
        if up >= 1.0 or down < 0.0:                                       # the nearest edge is an end of [0, 1): nothing beyond it
            continue
        assert {so.categorical(w, up)[0], so.categorical(w, down)[0]} != {i}   # one of the two directions leaves the bin


# ------------------------------------------------------------------------------ accept_sampling: margins
def _find_seed(lo, hi, slot=1, purpose=so.DRAW_ACCEPT, round_index=1):
    for seed in range(10000):
        u = so.uniform(seed, round_index, slot, purpose)
        if lo < u < hi:
            return seed, u
    raise AssertionError("no seed found")


def test_accept_margin_worked_example():
    """p = (0.5, 0.3, 0.2), q = (0.2, 0.6, 0.2), draft token 1: accepted iff u * 0.6 < 0.3, i.e. u < 1/2."""
    logits = torch.log(torch.tensor([[0.5, 0.3, 0.2], [0.1, 0.1, 0.8]], dtype=torch.float64))
    q = torch.tensor([0.2, 0.6, 0.2], dtype=torch.float64)
    seed, u = _find_seed(0.20, 0.30)                                      # accepted: u * 0.6 is 0.12 .. 0.18 against 0.3
    a, tok, log = so.accept_sampling([1], [q], logits, 1.0, seed, 1)
    assert a == 1 and log[0]["kind"] == "accept" and log[0]["u"] == u
    assert log[0]["margin"] == pytest.approx(1.0 - 2.0 * u, abs=1e-9)     # (0.3 - 0.6 u) / 0.3
    assert log[1]["kind"] == "bonus" and log[1]["j"] == 2
    seed, u = _find_seed(0.70, 0.90)                                      # rejected: u * 0.6 is 0.42 .. 0.54 against 0.3
    a, tok, log = so.accept_sampling([1], [q], logits, 1.0, seed, 1)
    assert a == 0 and log[0]["margin"] == pytest.approx(1.0 - 0.5 / u, abs=1e-9)   # (0.6 u - 0.3) / (0.6 u)
    assert log[1]["kind"] == "resample" and tok == 0                      # max(0, p - q) = (0.3, 0, 0): only token 0 is left
    # the resample's distance: the residual has one bin, [0, 0.3), and u' * 0.3 sits min(u', 1 - u') of its width from an edge
    u2 = so.uniform(seed, 1, 1, so.DRAW_RESAMPLE)
    assert log[1]["margin"] == pytest.approx(min(u2, 1.0 - u2), abs=1e-9)


def test_accept_margin_is_the_relative_change_that_flips_the_decision():
    g = torch.Generator().manual_seed(2)
    flips = 0
    for trial in range(40):
        V = 9
        logits = torch.randn(2, V, generator=g, dtype=torch.float64)
        q = torch.softmax(torch.randn(V, generator=g, dtype=torch.float64), 0)
        y = int(torch.randint(0, V, (1,), generator=g))
        a, _, log = so.accept_sampling([y], [q], logits, 0.8, trial, 3)
        m = log[0]["margin"]
        if not 1e-6 < m < 0.9:
            continue
        accepted = a == 1
        for f, expect_flip in ((0.99, False), (1.01, True)):
            q2 = q.clone()
            # an accepted draft is rejected once u * q(y) grows past p(y); a rejected one is accepted once it shrinks below
            q2[y] = q[y] / (1.0 - f * m) if accepted else q[y] * (1.0 - f * m)
            a2, _, _ = so.accept_sampling([y], [q2], logits, 0.8, trial, 3)
            assert ((a2 == 1) != accepted) == expect_flip, (trial, f, m)
            flips += int(expect_flip)
    assert flips >= 10
