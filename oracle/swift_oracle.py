"""CPU oracle for SWIFT's decoding hot path (arXiv 2410.06916).  TEST INFRASTRUCTURE ONLY.

A plain, slow, obviously-correct restatement of what the path computes, in ordinary PyTorch CPU
ops (fp64 by default; fp32 for the multi-billion-parameter shapes that do not fit host RAM in
fp64).  It shares no code with the CUDA library and must never be imported by it: only tests, the
smoke check and the benchmark's CPU-baseline leg use this file.

What is pinned by tests independent of this file: the decoder forward against the Huggingface LLaMA
implementation the paper ran (Appendix B.2) and against torch's fused attention; greedy
losslessness against vanilla decoding (Section 3.1); sampling acceptance by chi-squared and the
closed-form acceptance rate; nucleus filtering by a worked example, subset enumeration and the
Huggingface warper; matchness (Eq. 3) by brute force; Eq. 5 against the values printed in
Table 5; Philox against an independent library implementation.

Parity unpinned by the paper (readings, fixed by convention only): RMSNorm eps 1e-5, RoPE theta
1e4 with rotate-half pairing, argmax tie rule (lowest id), the random-number stream layout.

Notation follows the paper: z in {0,1}^L is the skipped sub-layer set over L = 2*n_blocks sub-layers
ordered [attn_0, mlp_0, attn_1, ...]; y'_j are draft tokens, p_j their confidence, gamma the context
window, N_D the maximum draft length, epsilon the early-stop threshold.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import torch

_MASK32 = 0xFFFFFFFF


# =============================================================================== random numbers
def philox4x32_10(ctr: Sequence[int], key: Sequence[int]) -> Tuple[int, int, int, int]:
    """Philox4x32-10 (Salmon et al., SC'11): ten rounds of two 32x32->64 multiplies and xors."""
    c = [int(v) & _MASK32 for v in ctr]
    k = [int(v) & _MASK32 for v in key]
    for _ in range(10):
        prod0 = 0xD2511F53 * c[0]
        prod1 = 0xCD9E8D57 * c[2]
        c = [((prod1 >> 32) ^ c[1] ^ k[0]) & _MASK32, prod1 & _MASK32,
             ((prod0 >> 32) ^ c[3] ^ k[1]) & _MASK32, prod0 & _MASK32]
        k = [(k[0] + 0x9E3779B9) & _MASK32, (k[1] + 0xBB67AE85) & _MASK32]
    return tuple(c)


# purposes of a random draw inside one decoding round (counter word 2)
DRAW_DRAFT, DRAW_ACCEPT, DRAW_RESAMPLE, DRAW_BONUS = 0, 1, 2, 3


def uniform(seed: int, round_index: int, slot: int, purpose: int) -> float:
    """u in [0,1): top 24 bits of the first Philox word at counter (round, slot, purpose, 0)."""
    w = philox4x32_10((round_index, slot, purpose, 0), (seed & _MASK32, (seed >> 32) & _MASK32))
    return (w[0] >> 8) * (2.0 ** -24)


def categorical(weights: torch.Tensor, u: float) -> Tuple[int, float]:
    """Smallest index i whose running sum (taken in index order) exceeds u * total.

    Returns (i, relative distance of u*total to the nearest edge of bin i) so a comparison with
    another implementation can exempt draws that sit on a bin edge.
    """
    w = weights.to(torch.float64)
    cs = torch.cumsum(w, 0)
    total = float(cs[-1])
    t = u * total
    i = int(torch.searchsorted(cs, torch.tensor(t, dtype=torch.float64), right=True))
    i = min(i, w.numel() - 1)
    while float(w[i]) == 0.0 and i > 0:   # only reachable through rounding at the very top
        i -= 1
    lo = float(cs[i - 1]) if i > 0 else 0.0
    dist = min(t - lo, float(cs[i]) - t) / total
    return i, dist


# =============================================================================== model pieces
def nucleus(prob: torch.Tensor, top_p: float) -> Tuple[torch.Tensor, float]:
    """Nucleus (top-p) filter, the sampling setting of Appendix B.2 (temperature 0.6, top_p 0.95).

    Tokens are taken in order of decreasing probability until their total mass first reaches top_p times
    the whole; every token at least as probable as the last one taken is kept (equal probabilities are
    kept or dropped together), the others get probability 0, and the kept ones are renormalised.
    top_p >= 1 returns the distribution unchanged.  Also returns how far the cut was from falling one
    token earlier or later: min(|mass before the last token - top_p|, |mass with it - top_p|) as a
    fraction of the whole."""
    if top_p >= 1.0:
        return prob, float("inf")
    p = prob.to(torch.float64)
    order = torch.sort(p, descending=True, stable=True).indices
    cs = torch.cumsum(p[order], dim=0)
    total = float(cs[-1])
    goal = top_p * total
    m = int(torch.searchsorted(cs, torch.tensor(goal, dtype=torch.float64)))     # first m with cs[m] >= goal
    m = min(m, p.numel() - 1)
    thr = p[order[m]]
    kept = torch.where(p >= thr, p, torch.zeros_like(p))
    before = float(cs[m - 1]) if m > 0 else 0.0
    margin = min(abs(float(cs[m]) - goal), abs(before - goal)) / total
    return kept / kept.sum(), margin


def rmsnorm(x: torch.Tensor, g: torch.Tensor, eps: float) -> torch.Tensor:
    """x * g / sqrt(mean(x^2) + eps), row-wise."""
    return x * torch.rsqrt((x * x).mean(dim=-1, keepdim=True) + eps) * g.to(x.dtype)


def rope(x: torch.Tensor, positions: torch.Tensor, theta: float) -> torch.Tensor:
    """Rotary embedding, rotate-half pairing: dim i is paired with dim i + d_h/2.

    x: [M, heads, d_h]; positions: [M] absolute indices from 0.
    """
    M, _, dh = x.shape
    half = dh // 2
    inv_freq = theta ** (-torch.arange(half, dtype=torch.float64) * 2.0 / dh)
    ang = positions.to(torch.float64)[:, None] * inv_freq[None, :]          # [M, half]
    cos, sin = torch.cos(ang).to(x.dtype)[:, None, :], torch.sin(ang).to(x.dtype)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return torch.cat([x1 * cos - x2 * sin, x2 * cos + x1 * sin], dim=-1)


def attention(q: torch.Tensor, K: torch.Tensor, V: torch.Tensor, allowed: torch.Tensor) -> torch.Tensor:
    """softmax(q K^T / sqrt(d_h)) V per head, with an explicit boolean mask.

    q: [M, H, d_h]; K, V: [n, H_kv, d_h]; allowed: [M, n].  Query head h reads KV head h // (H/H_kv).
    """
    M, H, dh = q.shape
    Hkv = K.shape[1]
    group = H // Hkv
    out = torch.empty_like(q)
    for h in range(H):
        kh, vh = K[:, h // group, :], V[:, h // group, :]
        s = (q[:, h, :] @ kh.T) / math.sqrt(dh)
        s = s.masked_fill(~allowed, float("-inf"))
        out[:, h, :] = torch.softmax(s, dim=-1) @ vh
    return out


def linear(x: torch.Tensor, W: torch.Tensor) -> torch.Tensor:
    """y = x W^T in fp64: the projection every sub-layer applies (weights stored [out, in])."""
    return x.to(torch.float64) @ W.to(torch.float64).T


def swiglu(gate: torch.Tensor, up: torch.Tensor) -> torch.Tensor:
    return gate * torch.sigmoid(gate) * up


def argmax_lowest(row: torch.Tensor) -> int:
    """argmax with ties broken towards the lowest token id."""
    m = row.max()
    return int(torch.nonzero(row == m)[0])


def top2_margin(row: torch.Tensor) -> float:
    v = torch.topk(row.to(torch.float64), 2).values
    return float(v[0] - v[1])


@dataclass
class Shape:
    n_blocks: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    vocab: int
    rope_theta: float = 10000.0
    rms_eps: float = 1e-5

    @staticmethod
    def of(cfg) -> "Shape":
        return Shape(cfg.n_blocks, cfg.d_model, cfg.n_heads, cfg.n_kv_heads, cfg.head_dim, cfg.ffn,
                     cfg.vocab, cfg.rope_theta, cfg.rms_eps)


# =============================================================================== decoder forward
class Oracle:
    """The target model, its KV cache and the committed sequence.

    State after prefill: `tokens` = prompt + generated tokens including the pending token t* (whose
    K,V are not in the cache yet); `n` = number of cached positions = len(tokens) - 1.
    """

    def __init__(self, shape: Shape, weights: Dict[str, object], dtype=torch.float64, max_positions: int = 4096):
        self.s = shape
        self.w = weights
        self.dtype = dtype
        self.max_positions = max_positions
        s = shape
        self.K = [torch.zeros(max_positions, s.n_kv_heads, s.head_dim, dtype=dtype) for _ in range(s.n_blocks)]
        self.V = [torch.zeros(max_positions, s.n_kv_heads, s.head_dim, dtype=dtype) for _ in range(s.n_blocks)]
        self.tokens: List[int] = []
        self.n = 0

    # ---- one weight application; weights may be stored in a narrower type and are widened exactly
    def _lin(self, x: torch.Tensor, W: torch.Tensor) -> torch.Tensor:
        return x @ W.to(self.dtype).T

    def forward_rows(self, row_tokens: Sequence[int], pos0: int, z: Optional[Sequence[int]] = None,
                     write_kv: bool = True, depth: Optional[Sequence[int]] = None,
                     sees: Optional[torch.Tensor] = None) -> torch.Tensor:
        """Logits [M, V] for M new rows at positions pos0..pos0+M-1 under skipped sub-layer set z.

        Every row attends to cached positions [0, pos0) and causally to the new rows.  A skipped
        sub-layer is the identity on the residual stream (Section 3.1): its norm, projections and,
        for attention, its K,V computation are all left out.  K,V of the new rows are stored in the
        cache for non-skipped attention sub-layers when write_kv is set.

        A token tree (Section 4.2, dynamic verification) is a set of rows that are not one sequence:
        `depth[i]` puts row i at sequence position pos0 + depth[i] and `sees` [M, M] says which of the
        new rows row i attends to (its ancestors and itself).  Row i's K,V still go to cache slot pos0 + i.
        """
        s = self.s
        M = len(row_tokens)
        z = [0] * (2 * s.n_blocks) if z is None else [int(v) for v in z]
        assert len(z) == 2 * s.n_blocks and pos0 + M <= self.max_positions
        pos = torch.arange(pos0, pos0 + M) if depth is None else pos0 + torch.tensor(list(depth), dtype=torch.long)
        h = self.w["embed"][torch.tensor(list(row_tokens), dtype=torch.long)].to(self.dtype)
        # row i may read cache position j < pos0 always, and new row j' <= i (or the rows `sees` names)
        among = torch.tril(torch.ones(M, M, dtype=torch.bool)) if sees is None else sees.to(torch.bool)
        allowed = torch.cat([torch.ones(M, pos0, dtype=torch.bool), among], dim=1)
        for b in range(s.n_blocks):
            wb = self.w["blocks"][b]
            if not z[2 * b]:
                x = rmsnorm(h, wb["attn_norm"], s.rms_eps)
                q = self._lin(x, wb["wq"]).view(M, s.n_heads, s.head_dim)
                k = self._lin(x, wb["wk"]).view(M, s.n_kv_heads, s.head_dim)
                v = self._lin(x, wb["wv"]).view(M, s.n_kv_heads, s.head_dim)
                q, k = rope(q, pos, s.rope_theta), rope(k, pos, s.rope_theta)
                Kall = torch.cat([self.K[b][:pos0], k], dim=0)
                Vall = torch.cat([self.V[b][:pos0], v], dim=0)
                a = attention(q, Kall, Vall, allowed).reshape(M, s.n_heads * s.head_dim)
                h = h + self._lin(a, wb["wo"])
                if write_kv:
                    self.K[b][pos0:pos0 + M] = k
                    self.V[b][pos0:pos0 + M] = v
            if not z[2 * b + 1]:
                x = rmsnorm(h, wb["mlp_norm"], s.rms_eps)
                h = h + self._lin(swiglu(self._lin(x, wb["wgate"]), self._lin(x, wb["wup"])), wb["wdown"])
        return self._lin(rmsnorm(h, self.w["final_norm"], s.rms_eps), self.w["lm_head"])

    # ---- the steps of the method ---------------------------------------------------------
    def prefill(self, prompt: Sequence[int], first_token: Optional[int] = None) -> torch.Tensor:
        """Full model over the prompt; caches K,V for [0, len(prompt)); t* = argmax of the last row
        unless the caller supplies it (sampling mode draws it outside).  Returns the logits."""
        logits = self.forward_rows(prompt, 0)
        self.n = len(prompt)
        t = argmax_lowest(logits[-1]) if first_token is None else int(first_token)
        self.tokens = list(prompt) + [t]
        return logits

    def draft(self, z: Sequence[int], max_k: int, stop_conf: float = 0.0,
              sampler=None, temperature: float = 1.0, top_p: float = 1.0) -> Tuple[List[int], List[float], List[torch.Tensor]]:
        """Autoregressive drafting with the layer-skipped model (Eq. 4) and early stopping.

        Step j feeds t* (j = 1) or y'_{j-1} at position n+j-1.  y'_j = argmax of the draft logits,
        p_j = max softmax (T = 1).  The token that falls below epsilon is kept, then drafting stops.
        With `sampler(j, q_j) -> token`, y'_j is drawn from q_j = nucleus(softmax(draft logits / T), top_p) instead.
        Returns (draft tokens, confidences, draft logits rows).
        """
        toks, confs, rows = [], [], []
        inp = self.tokens[-1]
        for j in range(1, max_k + 1):
            logit = self.forward_rows([inp], self.n + j - 1, z)[0]
            prob = torch.softmax(logit.to(torch.float64), dim=-1)
            if sampler is None:
                y = argmax_lowest(logit)
            else:
                y = int(sampler(j, nucleus(torch.softmax(logit.to(torch.float64) / temperature, dim=-1), top_p)[0]))
            toks.append(y)
            confs.append(float(prob.max()))
            rows.append(logit)
            inp = y
            if confs[-1] < stop_conf:
                break
        return toks, confs, rows

    def verify(self, draft_tokens: Sequence[int]) -> torch.Tensor:
        """Full model on rows [t*, y'_1..y'_k] at positions n..n+k; K,V written for every layer."""
        return self.forward_rows([self.tokens[-1]] + list(draft_tokens), self.n)

    def verify_tree(self, tree: "TokenTree") -> torch.Tensor:
        """Full model on all rows of a token tree at once (Section 4.2, dynamic verification): row i sits at position
        n + depth[i], attends to the cache and to its own ancestors, and leaves its K,V in slot n + i."""
        assert tree.tokens[0] == self.tokens[-1]
        return self.forward_rows(tree.tokens, self.n, depth=tree.depth, sees=tree.sees())

    def commit_path(self, tree: "TokenTree", path: Sequence[int], next_token: int) -> None:
        """KV rollback after a verified tree: the accepted node of depth j must end up in slot n + j; chain nodes are
        there already, an accepted alternative is moved there from the slot it was verified in."""
        for j, row in enumerate(path, start=1):
            assert tree.depth[row] == j
            if row != j:
                for b in range(self.s.n_blocks):
                    self.K[b][self.n + j] = self.K[b][self.n + row]
                    self.V[b][self.n + j] = self.V[b][self.n + row]
        self.commit([tree.tokens[r] for r in path], next_token)

    def commit(self, accepted: Sequence[int], next_token: int) -> None:
        """KV rollback: keep positions [0, n + a + 1); positions beyond are dropped (left stale)."""
        self.n += len(accepted) + 1
        self.tokens += list(accepted) + [int(next_token)]

    def score_skipsets(self, masks: Sequence[Sequence[int]], gamma: int) -> Tuple[List[float], List[List[int]]]:
        """matchness (Eq. 2-3) of every candidate z_c on the last gamma generated tokens.

        Rows are the inputs tokens[n-gamma .. n-1] at those positions; their known successors are
        tokens[n-gamma+1 .. n].  The prefix [0, n-gamma) comes from the target's cache; the window's
        K,V are the candidate's own and are never stored.
        """
        n, T = self.n, self.tokens
        assert gamma <= n and len(T) == n + 1
        scores, preds = [], []
        for z in masks:
            logits = self.forward_rows(T[n - gamma:n], n - gamma, z, write_kv=False)
            y = [argmax_lowest(logits[i]) for i in range(gamma)]
            preds.append(y)
            scores.append(sum(int(y[i] == T[n - gamma + 1 + i]) for i in range(gamma)) / gamma)
        return scores, preds


# =============================================================================== acceptance
def accept_greedy(draft_tokens: Sequence[int], target_logits: torch.Tensor) -> Tuple[int, int]:
    """Greedy verification: a = longest prefix with y'_j == argmax(target row j-1); the next token
    is the target's argmax on row a (the correction, or the bonus token when a = k)."""
    a = 0
    for j, y in enumerate(draft_tokens):
        if argmax_lowest(target_logits[j]) != int(y):
            break
        a += 1
    return a, argmax_lowest(target_logits[a])


def point_mass(n: int, y: int) -> torch.Tensor:
    """The distribution of a draft token chosen by arg max (Eq. 4): all mass on y."""
    q = torch.zeros(n, dtype=torch.float64)
    q[y] = 1.0
    return q


def accept_sampling(draft_tokens: Sequence[int], q_rows: Sequence[torch.Tensor], target_logits: torch.Tensor,
                    temperature: float, seed: int, round_index: int, top_p: float = 1.0) -> Tuple[int, int, List[dict]]:
    """Speculative-sampling verification (the acceptance strategy of Appendix B.2, after Leviathan et al.).

    p_j = nucleus(softmax(target row j-1 / T), top_p): the distribution plain sampling from the target would
    use; q_j = the distribution y'_j was drawn from.  For j = 1..k draw
    u_j and accept iff u_j * q_j(y'_j) < p_j(y'_j)  (i.e. u < min(1, p/q)).  On the first rejection
    draw the replacement from max(0, p_j - q_j) renormalised; if nothing is rejected draw a bonus token
    from p_{k+1}.  Returns (a, next token, per-decision records for boundary-aware comparison).
    """
    k = len(draft_tokens)
    P = torch.softmax(target_logits.to(torch.float64) / temperature, dim=-1)
    if top_p < 1.0:
        P = torch.stack([nucleus(P[i], top_p)[0] for i in range(P.shape[0])])
    log: List[dict] = []
    for j in range(1, k + 1):
        y = int(draft_tokens[j - 1])
        p, q = P[j - 1], q_rows[j - 1].to(torch.float64)
        u = uniform(seed, round_index, j, DRAW_ACCEPT)
        lhs, rhs = u * float(q[y]), float(p[y])
        log.append({"kind": "accept", "j": j, "u": u, "margin": abs(lhs - rhs) / max(rhs, lhs, 1e-300)})
        if not lhs < rhs:
            resid = torch.clamp(p - q, min=0.0)
            if float(resid.sum()) <= 0.0:      # p == q everywhere: no residual mass, fall back to p
                resid = p
            tok, dist = categorical(resid, uniform(seed, round_index, j, DRAW_RESAMPLE))
            log.append({"kind": "resample", "j": j, "margin": dist})
            return j - 1, tok, log
    tok, dist = categorical(P[k], uniform(seed, round_index, k + 1, DRAW_BONUS))
    log.append({"kind": "bonus", "j": k + 1, "margin": dist})
    return k, tok, log


# =============================================================================== dynamic verification (token tree)
def tree_width(p: float) -> int:
    """How many of the draft model's top predictions stand in for a draft token of confidence p (Section 4.2):
    10, 5, 3, 1 for p in (0, 0.5], (0.5, 0.8], (0.8, 0.95], (0.95, 1]."""
    return 10 if p <= 0.5 else 5 if p <= 0.8 else 3 if p <= 0.95 else 1


@dataclass
class TokenTree:
    """The draft candidates of one round, linearised: row 0 is the pending token t*, rows 1..k the drafted chain
    y'_1..y'_k, then, depth by depth, the alternatives of each draft position (the draft model's next-best
    predictions at that step).  An alternative of depth j hangs off chain row j-1 and has no children: drafting
    went on from y'_j only."""
    tokens: List[int]
    depth: List[int]
    parent: List[int]

    def sees(self) -> torch.Tensor:
        """[M, M]: row i attends to its ancestors and itself (the 'special causal attention mask' of Section 4.2)."""
        M = len(self.tokens)
        a = torch.zeros(M, M, dtype=torch.bool)
        for i in range(M):
            j = i
            while j >= 0:
                a[i, j] = True
                j = self.parent[j]
        return a

    def children(self, node: int) -> List[int]:
        return [c for c, p in enumerate(self.parent) if p == node]


def ranked_tokens(row: torch.Tensor, n: int) -> List[int]:
    """The n best token ids of a logits row, best first; equal logits in order of token id."""
    idx = torch.sort(row.to(torch.float64), descending=True, stable=True).indices   # stable: equal values keep index order
    return [int(i) for i in idx[:n]]


def build_tree(pending: int, draft_tokens: Sequence[int], draft_rows: Sequence[torch.Tensor], conf: Sequence[float],
               row_budget: int) -> TokenTree:
    """Extends every draft position j with the draft model's top-k predictions at that step, k = tree_width(p_j).
    The paper sets no limit on the rows verified at once; here the forward takes row_budget rows, so the chain
    (1 + k rows) is placed first and the alternatives are handed out from the first draft position on until the
    rows run out (an earlier position decides whether the later ones matter at all)."""
    k = len(draft_tokens)
    assert row_budget >= k + 1
    tokens, depth, parent = [int(pending)] + [int(t) for t in draft_tokens], list(range(k + 1)), list(range(-1, k))
    for j in range(1, k + 1):
        extra = min(tree_width(conf[j - 1]) - 1, row_budget - len(tokens))
        if extra <= 0:
            continue
        best = ranked_tokens(draft_rows[j - 1], extra + 1)
        alts = [t for t in best if t != tokens[j]][:extra]            # the chain token is the best one under greedy drafting
        for t in alts:
            tokens.append(t); depth.append(j); parent.append(j - 1)
    return TokenTree(tokens, depth, parent)


def accept_tree(tree: TokenTree, target_logits: torch.Tensor) -> Tuple[List[int], int]:
    """Greedy verification of a token tree: from t*, follow the child whose token is the target's arg max at the
    current node; where no child matches, that arg max is the next token.  Returns (rows of the accepted nodes in
    order, next token): every emitted token is what vanilla greedy decoding would have produced."""
    node, path = 0, []
    while True:
        gold = argmax_lowest(target_logits[node])
        hit = [c for c in tree.children(node) if tree.tokens[c] == gold]
        if not hit:
            return path, gold
        node = hit[0]
        path.append(node)


# =============================================================================== whole runs
@dataclass
class GenParams:
    max_new: int
    max_draft: int = 8            # N_D
    stop_conf: float = 0.0        # epsilon
    mode: str = "greedy"          # or "sampling"
    temperature: float = 1.0
    top_p: float = 1.0
    greedy_draft: bool = False    # sampling mode with drafts chosen by arg max (Eq. 4 as written): q_j = point mass on y'_j
    rng_seed: int = 0
    gamma: int = 32
    stop_matchness: float = 0.95
    max_opt_rounds: int = 0       # 0 = skip set fixed
    patience: int = 0             # stop optimising after this many rounds in a row that kept the incumbent (0 = never)
    tree_rows: int = 0            # dynamic verification: rows one verification may hold (0 = the drafted chain only)


@dataclass
class Round:
    n_start: int
    draft: List[int]
    conf: List[float]
    draft_margin: List[float]
    target_argmax: List[int]
    target_margin: List[float]
    accepted: int
    next_token: int
    decisions: List[dict] = field(default_factory=list)
    matchness: Optional[List[float]] = None
    z: Optional[List[int]] = None
    tree: Optional[TokenTree] = None       # dynamic verification: the rows that were verified and the accepted path
    path: Optional[List[int]] = None


def vanilla_generate(o: Oracle, prompt: Sequence[int], max_new: int, mode: str = "greedy",
                     temperature: float = 1.0, rng_seed: int = 0, top_p: float = 1.0) -> Tuple[List[int], List[float]]:
    """Plain autoregressive decoding of the full model: the definition SWIFT must reproduce."""
    logits = o.prefill(prompt)
    margins = [top2_margin(logits[-1])]
    if mode == "sampling":
        p = nucleus(torch.softmax(logits[-1].to(torch.float64) / temperature, -1), top_p)[0]
        o.tokens[-1] = categorical(p, uniform(rng_seed, 0, 0, DRAW_BONUS))[0]
    step = 0
    while len(o.tokens) - len(prompt) < max_new:
        step += 1
        row = o.forward_rows([o.tokens[-1]], o.n)[0]
        margins.append(top2_margin(row))
        if mode == "sampling":
            p = nucleus(torch.softmax(row.to(torch.float64) / temperature, -1), top_p)[0]
            t = categorical(p, uniform(rng_seed, step, 0, DRAW_BONUS))[0]
        else:
            t = argmax_lowest(row)
        o.commit([], t)
    return o.tokens[len(prompt):], margins


def swift_generate(o: Oracle, prompt: Sequence[int], z0: Sequence[int], gp: GenParams,
                   candidates=None, optimizer: "Optional[LayerSetOptimizer]" = None,
                   n_candidates: int = 0) -> Tuple[List[int], List[Round], dict]:
    """Draft-then-verify decoding with skipped sub-layer set z (Sections 4.1-4.2).

    Each round: [optionally score candidates on the last gamma generated tokens and keep the best] ->
    draft at most N_D tokens (stop early below epsilon) -> verify with the full model -> accept ->
    roll the KV cache back.  Emits exactly gp.max_new tokens: the draft length is capped at
    remaining - 1, and with one token left a plain full-model step is taken.
    `candidates(round) -> masks [C, L]` supplies the proposals of one optimisation round; alternatively `optimizer`
    (a LayerSetOptimizer) proposes n_candidates sets per round and is told every score of the round.

    An optimisation round scores the set in use together with the proposals on the same window (the set in
    use is entry 0 of the round's `matchness`) and keeps the highest-scoring one (Section 4.1), the earliest
    among equals: the set in use is replaced only by a proposal that beats it on the tokens both were scored
    on.  Optimisation ends once the kept set scores above gp.stop_matchness, after gp.max_opt_rounds rounds,
    or after gp.patience rounds in a row without a replacement (the stop rules of Appendix B.2).
    """
    sampling = gp.mode == "sampling"
    logits = o.prefill(prompt)
    if sampling:
        p = nucleus(torch.softmax(logits[-1].to(torch.float64) / gp.temperature, -1), gp.top_p)[0]
        o.tokens[-1] = categorical(p, uniform(gp.rng_seed, 0, 0, DRAW_BONUS))[0]
    z = [int(v) for v in z0]
    best_score, opt_rounds, optimising, stale = -1.0, 0, gp.max_opt_rounds > 0, 0
    rounds: List[Round] = []
    n_prompt = len(prompt)
    r = 0
    while len(o.tokens) - n_prompt < gp.max_new:
        r += 1
        remaining = gp.max_new - (len(o.tokens) - n_prompt)
        scores = None
        if optimising and len(o.tokens) - n_prompt >= gp.gamma and (candidates is not None or optimizer is not None):
            if optimizer is not None:
                proposals = [optimizer.mask(optimizer.suggest()) for _ in range(n_candidates)]
            else:
                proposals = [[int(v) for v in m] for m in candidates(opt_rounds)]
            masks = [list(z)] + proposals
            scores, _ = o.score_skipsets(masks, gp.gamma)
            if optimizer is not None:
                for mk, sc in zip(masks, scores):
                    optimizer.observe([b for b in range(o.s.n_blocks) if mk[2 * b] and mk[2 * b + 1]], sc)
            c_best = max(range(len(scores)), key=lambda c: (scores[c], -c))   # entry 0, the set in use, wins ties
            best_score, z = scores[c_best], masks[c_best]
            stale = 0 if c_best != 0 else stale + 1
            opt_rounds += 1
            if best_score > gp.stop_matchness or opt_rounds >= gp.max_opt_rounds or (gp.patience > 0 and stale >= gp.patience):
                optimising = False
        k_max = min(gp.max_draft, remaining - 1)
        q_rows: List[torch.Tensor] = []
        if k_max > 0:
            if sampling:
                def sampler(j, prob, _r=r):
                    if gp.greedy_draft:
                        y = argmax_lowest(prob)
                        q_rows.append(point_mass(prob.numel(), y))
                        return y
                    q_rows.append(prob)
                    return categorical(prob, uniform(gp.rng_seed, _r, j, DRAW_DRAFT))[0]
                d_tok, d_conf, d_rows = o.draft(z, k_max, gp.stop_conf, sampler, gp.temperature, gp.top_p)
            else:
                d_tok, d_conf, d_rows = o.draft(z, k_max, gp.stop_conf)
        else:
            d_tok, d_conf, d_rows = [], [], []
        if gp.tree_rows > 0 and not sampling:
            # dynamic verification: the chain plus the draft model's next-best predictions, verified as one tree
            tree = build_tree(o.tokens[-1], d_tok, d_rows, d_conf, max(gp.tree_rows, len(d_tok) + 1))
            tl = o.verify_tree(tree)
            path, nxt = accept_tree(tree, tl)
            M = len(tree.tokens)
            rounds.append(Round(o.n, d_tok, d_conf, [top2_margin(x) for x in d_rows], [argmax_lowest(tl[i]) for i in range(M)],
                                [top2_margin(tl[i]) for i in range(M)], len(path), nxt, [], scores, list(z), tree, list(path)))
            o.commit_path(tree, path, nxt)
            continue
        tl = o.verify(d_tok)
        if sampling:
            a, nxt, dec = accept_sampling(d_tok, q_rows, tl, gp.temperature, gp.rng_seed, r, gp.top_p)
        else:
            (a, nxt), dec = accept_greedy(d_tok, tl), []
        rounds.append(Round(o.n, d_tok, d_conf, [top2_margin(x) for x in d_rows],
                            [argmax_lowest(tl[i]) for i in range(len(d_tok) + 1)],
                            [top2_margin(tl[i]) for i in range(len(d_tok) + 1)], a, nxt, dec, scores, list(z)))
        o.commit(d_tok[:a], nxt)
    out = o.tokens[n_prompt:]
    n_draft = sum(len(x.draft) for x in rounds)
    stats = {"rounds": len(rounds), "tokens": len(out), "drafted": n_draft,
             "accepted": sum(x.accepted for x in rounds),
             "M": (len(out) - 1) / max(len(rounds), 1),    # tokens per target forward (prefill's token excluded)
             "alpha": sum(x.accepted for x in rounds) / max(n_draft, 1)}
    return out, rounds, stats


def expected_speedup(M: float, alpha: float, c: float) -> float:
    """Eq. 5: E(Spd.) = M*alpha / ((M-1)*c + alpha), c = 1 - r the draft/target cost ratio."""
    return M * alpha / ((M - 1.0) * c + alpha)


# =============================================================================== layer set suggestion (Section 4.1)
class LayerSetOptimizer:
    """Proposes skipped-layer sets for the on-the-fly optimisation (Section 4.1, 'Efficient Layer Set Suggestion').

    The input space is all sets of m of the n_blocks blocks (skip ratio r = m / n_blocks fixed).  Optimisation step o
    (counted from 1) proposes a uniformly random set, except every beta-th step, which asks a Gaussian-process model of
    matchness over the sets seen so far for the set with the highest upper confidence bound (Bayesian optimisation).
    The paper delegates that part to a third-party package and prints no formulas; this is the textbook form:

      * a set is its indicator vector x in {0,1}^n_blocks; the squared distance of two sets is their Hamming distance;
      * mean function: ridge regression of the standardised scores on the indicators, w = (X^T X + ridge I)^-1 X^T t, over
        all evaluated sets (how much each block costs when skipped: the additive part of matchness);
      * on the residuals of the `gp_window` most recent evaluations: zero-mean GP, Matern-5/2 covariance
        k(d) = (1 + s + s^2/3) exp(-s), s = sqrt(5) d / ell, observation noise `noise`; ell is the one of `ells` with the
        highest marginal likelihood; posterior mean and variance by a Cholesky factorisation of K + noise * I;
      * acquisition mu + kappa * sigma, maximised over a pool: `pool` random sets, every set one swap away from the best
        set seen, the m blocks with the smallest regression cost, and every set one swap away from that; sets already
        evaluated are left out.

    Random draws come from Philox4x32-10 keyed by `seed`: counter (index, 0, stream, 0x4F5054), one word per draw.
    """

    def __init__(self, n_blocks: int, m: int, beta: int = 25, seed: int = 0, pool: int = 512, kappa: float = 2.576,
                 noise: float = 1e-2, ells: Sequence[float] = (1.0, 2.0, 4.0), ridge: float = 1.0, gp_window: int = 256):
        assert 0 < m < n_blocks
        self.nb, self.m, self.beta, self.seed, self.pool, self.kappa, self.noise, self.ells = n_blocks, m, beta, seed, pool, kappa, noise, tuple(ells)
        self.ridge, self.gp_window = ridge, gp_window
        self.step = 0                       # optimisation steps taken (= proposals made)
        self.draws = 0                      # random words consumed
        self.X: List[Tuple[int, ...]] = []  # evaluated sets (sorted block tuples) ...
        self.y: List[float] = []            # ... and their matchness

    # ---- random sets
    def _word(self) -> int:
        w = philox4x32_10((self.draws & _MASK32, self.draws >> 32, 7, 0x4F5054), (self.seed & _MASK32, (self.seed >> 32) & _MASK32))[0]
        self.draws += 1
        return w

    def random_set(self) -> Tuple[int, ...]:
        """m blocks by a partial Fisher-Yates shuffle: position i swaps with i + word mod (n - i)."""
        idx = list(range(self.nb))
        for i in range(self.m):
            j = i + self._word() % (self.nb - i)
            idx[i], idx[j] = idx[j], idx[i]
        return tuple(sorted(idx[:self.m]))

    # ---- Gaussian process
    @staticmethod
    def matern52(d2, ell: float):
        import numpy as np
        s = np.sqrt(5.0 * np.asarray(d2, dtype=np.float64)) / ell
        return (1.0 + s + s * s / 3.0) * np.exp(-s)

    def _indicator(self, sets):
        import numpy as np
        X = np.zeros((len(sets), self.nb))
        for i, s in enumerate(sets):
            X[i, list(s)] = 1.0
        return X

    def fit(self):
        """Standardises the scores and picks ell by marginal likelihood.  Returns what predict() needs."""
        import numpy as np
        Xall = self._indicator(self.X)
        y = np.asarray(self.y, dtype=np.float64)
        mu, sd = y.mean(), y.std()
        sd = sd if sd > 1e-12 else 1.0
        t_all = (y - mu) / sd
        w = np.linalg.solve(Xall.T @ Xall + self.ridge * np.eye(self.nb), Xall.T @ t_all)     # mean function
        X = Xall[-self.gp_window:]
        t = (t_all - Xall @ w)[-self.gp_window:]                                              # the GP models what is left
        d2 = (X[:, None, :] != X[None, :, :]).sum(-1).astype(np.float64)
        best = None
        for ell in self.ells:
            K = self.matern52(d2, ell) + self.noise * np.eye(len(t))
            Lc = np.linalg.cholesky(K)
            a = np.linalg.solve(Lc.T, np.linalg.solve(Lc, t))
            lml = -0.5 * float(t @ a) - float(np.log(np.diag(Lc)).sum()) - 0.5 * len(t) * math.log(2.0 * math.pi)
            if best is None or lml > best[0]:
                best = (lml, ell, Lc, a)
        return {"X": X, "mu": mu, "sd": sd, "ell": best[1], "L": best[2], "alpha": best[3], "lml": best[0], "w": w, "resid": t}

    def predict(self, model, sets):
        """Posterior mean and standard deviation of matchness at `sets` (in matchness units)."""
        import numpy as np
        Z = self._indicator(sets)
        d2 = (Z[:, None, :] != model["X"][None, :, :]).sum(-1).astype(np.float64)
        Ks = self.matern52(d2, model["ell"])
        mean = Z @ model["w"] + Ks @ model["alpha"]
        v = np.linalg.solve(model["L"], Ks.T)
        var = np.maximum(1.0 - (v * v).sum(0), 0.0)
        return model["mu"] + model["sd"] * mean, model["sd"] * np.sqrt(var)

    # ---- proposals
    def best_set(self) -> Optional[Tuple[int, ...]]:
        """The evaluated set with the highest matchness (the earliest among equals)."""
        if not self.y:
            return None
        return self.X[max(range(len(self.y)), key=lambda i: (self.y[i], -i))]

    def bayesian_set(self) -> Tuple[Tuple[int, ...], dict]:
        """The unevaluated set with the highest mu + kappa * sigma among `pool` random sets and the one-swap
        neighbours of the best set seen (pool order, earliest among equals)."""
        cand: List[Tuple[int, ...]] = [self.random_set() for _ in range(self.pool)]

        def with_swaps(base):
            out = [tuple(base)]
            outside = [b for b in range(self.nb) if b not in base]
            for out_b in base:
                for in_b in outside:
                    out.append(tuple(sorted((set(base) - {out_b}) | {in_b})))
            return out

        inc = self.best_set()
        model = self.fit() if self.X else None
        if inc is not None:
            cand += with_swaps(inc)[1:]
            # the m blocks that cost least to skip according to the regression: largest weights, compared to six decimals
            # (blocks that were always skipped together get the same weight up to rounding), lowest index among equals
            order = sorted(range(self.nb), key=lambda b: (-math.floor(float(model["w"][b]) * 1e6 + 0.5), b))
            cand += with_swaps(tuple(sorted(order[:self.m])))
        seen = set(self.X)
        cand = [c for c in dict.fromkeys(cand) if c not in seen]
        if not cand or not self.X:
            return (cand[0] if cand else self.random_set()), {}
        mean, std = self.predict(model, cand)
        ucb = mean + self.kappa * std
        i = max(range(len(cand)), key=lambda j: (float(ucb[j]), -j))
        return cand[i], {"ucb": float(ucb[i]), "candidates": cand, "ucb_all": ucb, "model": model}

    def suggest(self) -> Tuple[int, ...]:
        """The next proposal: Bayesian every beta-th step once something has been evaluated, random otherwise."""
        self.step += 1
        if self.beta > 0 and self.step % self.beta == 0 and self.X:
            return self.bayesian_set()[0]
        return self.random_set()

    def observe(self, blocks: Sequence[int], matchness: float) -> None:
        self.X.append(tuple(sorted(int(b) for b in blocks)))
        self.y.append(float(matchness))

    def mask(self, blocks: Sequence[int]) -> List[int]:
        """Sub-layer mask [attn_0, mlp_0, ...] that skips both sub-layers of every block in `blocks`."""
        z = [0] * (2 * self.nb)
        for b in blocks:
            z[2 * b] = z[2 * b + 1] = 1
        return z
