"""Seeded synthetic inputs: model shapes, weights, planted blocks, prompts, candidate masks.

Input generation only.  Nothing here belongs to the decoding method; the CPU oracle and
the CUDA library are both fed from this module so that they see bit-identical inputs.

The synthetic models stand in for the LLaMA-2 7B / 13B / 70B checkpoints and the few-shot
prompts the paper evaluates on (Section 5.1, Appendix B.1/B.2): same tensor shapes, random
N(0, 0.02) weights, uniform random prompt ids, and "planted" layer sparsity (a seeded set of
blocks whose residual-branch output projections are scaled down) so that a good skip set
exists for the method to exploit.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, replace
from typing import Dict, Iterator, List, Tuple

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "_synth_cpu.so")
_SRC_PATH = os.path.join(_HERE, "synth_cpu.c")
_TAG = 0x53594E54
_MASK32 = 0xFFFFFFFF

# tensor ids (counter word 2)
TID_EMBED, TID_LM_HEAD, TID_FINAL_NORM = 0, 1, 2
TID_BLOCK_BASE, TID_BLOCK_STRIDE = 16, 16
_BLOCK_TENSORS = ("wq", "wk", "wv", "wo", "wgate", "wup", "wdown", "attn_norm", "mlp_norm")
TID_PROMPT, TID_SHUFFLE, TID_MASKS = 3, 4, 5


@dataclass(frozen=True)
class ModelConfig:
    name: str
    n_blocks: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    vocab: int
    dtype: str  # "f32" or "bf16": storage type of the weights
    seed: int
    n_planted: int
    planted_scale: float = 0.01
    init_std: float = 0.02
    gain_std: float = 0.0  # norm gains = 1 + gain_std * N(0,1); the paper-shaped configs use 1
    embed_std: float = 0.0      # standard deviation of the token embedding; 0 = init_std
    branch_scale: float = 1.0   # factor on every block's residual-branch output projections (wo, wdown), planted or not
    rope_theta: float = 10000.0
    rms_eps: float = 1e-5

    @property
    def n_sublayers(self) -> int:
        return 2 * self.n_blocks

    @property
    def q_dim(self) -> int:
        return self.n_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    def shapes(self) -> Dict[str, Tuple[int, ...]]:
        d = self.d_model
        return {
            "wq": (self.q_dim, d), "wk": (self.kv_dim, d), "wv": (self.kv_dim, d),
            "wo": (d, self.q_dim), "wgate": (self.ffn, d), "wup": (self.ffn, d),
            "wdown": (d, self.ffn), "attn_norm": (d,), "mlp_norm": (d,),
            "embed": (self.vocab, d), "lm_head": (self.vocab, d), "final_norm": (d,),
        }

    def block_params(self) -> int:
        s = self.shapes()
        return sum(int(np.prod(s[k])) for k in ("wq", "wk", "wv", "wo", "wgate", "wup", "wdown"))

    def with_blocks(self, n_blocks: int, n_planted: int | None = None, name: str | None = None) -> "ModelConfig":
        """Same widths, fewer blocks: a reduced-depth copy the oracle finishes in seconds."""
        if n_planted is None:
            n_planted = (self.n_planted * n_blocks) // self.n_blocks
        return replace(self, n_blocks=n_blocks, n_planted=n_planted,
                       name=name or f"{self.name}-{n_blocks}blk")


@dataclass(frozen=True)
class RunConfig:
    prompt_len: int
    max_new: int
    max_draft: int
    stop_conf: float = 0.0
    n_skip_blocks: int = 0       # blocks skipped by the draft model (both sub-layers)
    mode: str = "greedy"         # "greedy" or "sampling"
    temperature: float = 1.0
    top_p: float = 1.0           # nucleus filtering of the sampling distributions (1 = none)
    rng_seed: int = 0
    optimise: bool = False       # on-the-fly skip-set optimisation (Section 4.1)
    gamma: int = 32              # context window
    n_candidates: int = 32       # candidates scored per optimisation round
    max_opt_rounds: int = 16
    stop_matchness: float = 0.95


# The five benchmark shapes.  Seeds other than the first are this repository's choice: the lowest
# seed whose planted set leaves the first three blocks alone.  With N(0, 0.02) everywhere the token
# embedding is small (0.02 per element) next to a block's output (order 1), so a planted block at the
# very start still contributes as much as the embedding itself and skipping it is not "nearly free".
MODELS: Dict[str, ModelConfig] = {
    "tiny": ModelConfig("tiny", 8, 256, 4, 4, 64, 688, 2048, "f32", seed=0, n_planted=4),
    "7b": ModelConfig("7b", 32, 4096, 32, 32, 128, 11008, 32000, "bf16", seed=2, n_planted=14),
    "13b": ModelConfig("13b", 40, 5120, 40, 40, 128, 13824, 32000, "bf16", seed=3, n_planted=18),
    "70b": ModelConfig("70b", 80, 8192, 64, 8, 128, 28672, 32000, "bf16", seed=6, n_planted=36),
    # a 34B-class backbone (the paper also runs 33B/34B models, Section 5.2, without giving their shapes): 60 blocks, 56 query
    # heads on 8 KV heads (7 per group, not a power of two), vocabulary 64000 (twice the others'), skip ratio 0.5
    "34b": ModelConfig("34b", 60, 7168, 56, 8, 128, 20480, 64000, "bf16", seed=12, n_planted=30),
    # The 13B shape with layers that behave like a trained model's for the purposes of layer skipping: with N(0, 0.02)
    # everywhere a block's output is as large as the whole residual stream, and skipping any single block that is not
    # planted already destroys the prediction (measured: matchness <= 0.16), so no search over skip sets can be
    # guided by matchness.  Here the token embedding carries the stream (std 0.9) and every block adds a modest
    # increment (output projections x 0.05, planted ones x 0.01 on top): matchness then falls gradually with every
    # non-planted block skipped, as the paper's models do.  Config 3 (on-the-fly optimisation) runs on this one.
    "13b-graded": ModelConfig("13b-graded", 40, 5120, 40, 40, 128, 13824, 32000, "bf16", seed=3, n_planted=18,
                              embed_std=0.9, branch_scale=0.05),
}
RUNS: Dict[str, Tuple[str, RunConfig]] = {
    "c1": ("tiny", RunConfig(32, 64, 4, stop_conf=0.8, n_skip_blocks=4)),
    "c2": ("7b", RunConfig(512, 256, 8, n_skip_blocks=14)),
    # (up to 32 optimisation rounds per input: Appendix B.2's S = 1000 proposals at 32 proposals per round)
    "c3": ("13b-graded", RunConfig(1024, 512, 8, n_skip_blocks=18, optimise=True, max_opt_rounds=32)),
    "c3-flat": ("13b", RunConfig(1024, 512, 8, n_skip_blocks=18, optimise=True, max_opt_rounds=32)),     # the same on the all-N(0, 0.02) model
    "c3-fixed": ("13b", RunConfig(1024, 512, 8, n_skip_blocks=18)),     # config 3's shape with the planted set held fixed
    "c4": ("13b", RunConfig(1024, 512, 8, n_skip_blocks=20, mode="sampling", rng_seed=4)),
    # config 4 with the sampling setting the paper uses on code generation (Appendix B.2)
    "c4-nucleus": ("13b", RunConfig(1024, 512, 8, n_skip_blocks=20, mode="sampling", temperature=0.6, top_p=0.95, rng_seed=4)),
    "c5": ("70b", RunConfig(2048, 512, 12, n_skip_blocks=36)),
    "w34": ("34b", RunConfig(1024, 512, 8, n_skip_blocks=30)),            # second workload shape: 34B class, r = 0.5
}


# ----------------------------------------------------------------------------- Philox (scalar)
def philox4x32_10(ctr, key):
    """Philox4x32-10 from its published definition, on Python ints (small counts only)."""
    c0, c1, c2, c3 = (int(x) & _MASK32 for x in ctr)
    k0, k1 = (int(x) & _MASK32 for x in key)
    for _ in range(10):
        p0 = 0xD2511F53 * c0
        p1 = 0xCD9E8D57 * c2
        c0, c1, c2, c3 = ((p1 >> 32) ^ c1 ^ k0) & _MASK32, p1 & _MASK32, \
                         ((p0 >> 32) ^ c3 ^ k1) & _MASK32, p0 & _MASK32
        k0 = (k0 + 0x9E3779B9) & _MASK32
        k1 = (k1 + 0xBB67AE85) & _MASK32
    return c0, c1, c2, c3


def _word(seed: int, tid: int, index: int) -> int:
    """32-bit word number `index` of the stream (seed, tid): word index%4 of Philox block index//4."""
    blk, lane = divmod(index, 4)
    out = philox4x32_10((blk & _MASK32, blk >> 32, tid, _TAG), (seed & _MASK32, seed >> 32))
    return out[lane]


# ----------------------------------------------------------------------------- native bulk fill
_lib = None


def build(force: bool = False) -> str:
    """Compile the CPU generator with gcc (in-tree)."""
    if force or not os.path.exists(_LIB_PATH) or os.path.getmtime(_LIB_PATH) < os.path.getmtime(_SRC_PATH):
        tmp = _LIB_PATH + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O3", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC_PATH])
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB_PATH)
        lib.synth_fill.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_uint64,
                                   ctypes.c_uint32, ctypes.c_float, ctypes.c_float, ctypes.c_void_p,
                                   ctypes.c_int]
        lib.synth_fill.restype = None
        lib.synth_philox.argtypes = [ctypes.c_void_p] * 3
        lib.synth_philox.restype = None
        _lib = lib
    return _lib


_Z = None


def normal_table() -> np.ndarray:
    """Z[i] = inverse standard-normal CDF at (i + 0.5) / 65536, computed in double, stored fp32."""
    global _Z
    if _Z is None:
        from scipy.special import ndtri
        _Z = np.ascontiguousarray(ndtri((np.arange(65536, dtype=np.float64) + 0.5) / 65536.0).astype(np.float32))
    return _Z


def fill(shape, seed: int, tensor_id: int, scale: float, dtype: str, scale2: float = 1.0,
         out: torch.Tensor | None = None) -> torch.Tensor:
    """Tensor of `shape` with elements (scale * Z[u16]) * scale2, stored as fp32 or bf16."""
    n = int(np.prod(shape))
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    if out is None:
        out = torch.empty(n, dtype=tdt)
    assert out.is_contiguous() and out.numel() == n and out.dtype == tdt and out.device.type == "cpu"
    Z = normal_table()
    _load().synth_fill(out.data_ptr(), 0, n, seed, tensor_id, scale, scale2, Z.ctypes.data,
                       0 if dtype == "f32" else 1)
    return out.view(*shape)


# ----------------------------------------------------------------------------- model pieces
def planted_blocks(cfg: ModelConfig) -> List[int]:
    """First n_planted entries of a Philox-keyed Fisher-Yates shuffle of the block indices."""
    return _subset(cfg.seed, TID_SHUFFLE, 0, cfg.n_blocks, cfg.n_planted)


def _subset(seed: int, tid: int, stream_offset: int, n: int, m: int) -> List[int]:
    idx = list(range(n))
    for i in range(min(m, n - 1)):
        j = i + _word(seed, tid, stream_offset + i) % (n - i)
        idx[i], idx[j] = idx[j], idx[i]
    return sorted(idx[:m])


def tensor_id(name: str, block: int = -1) -> int:
    if name == "embed":
        return TID_EMBED
    if name == "lm_head":
        return TID_LM_HEAD
    if name == "final_norm":
        return TID_FINAL_NORM
    return TID_BLOCK_BASE + TID_BLOCK_STRIDE * block + _BLOCK_TENSORS.index(name)


def make_tensor(cfg: ModelConfig, name: str, block: int = -1, planted: bool | None = None,
                out: torch.Tensor | None = None) -> torch.Tensor:
    """One weight tensor of the synthetic model (CPU).  Norm gains are always fp32."""
    shape = cfg.shapes()[name]
    tid = tensor_id(name, block)
    if name.endswith("norm"):
        if cfg.gain_std == 0.0:
            return torch.ones(shape, dtype=torch.float32)
        return 1.0 + fill(shape, cfg.seed, tid, cfg.gain_std, "f32")
    if planted is None:
        planted = block in planted_blocks(cfg)
    s2 = 1.0
    if name in ("wo", "wdown"):
        s2 = cfg.branch_scale * (cfg.planted_scale if planted else 1.0)
    std = cfg.embed_std if (name == "embed" and cfg.embed_std > 0.0) else cfg.init_std
    return fill(shape, cfg.seed, tid, std, cfg.dtype, s2, out=out)


def iter_tensors(cfg: ModelConfig) -> Iterator[Tuple[str, int, torch.Tensor]]:
    """Yield (name, block, tensor) one at a time, so a model larger than host RAM can be streamed."""
    planted = set(planted_blocks(cfg))
    yield "embed", -1, make_tensor(cfg, "embed")
    for b in range(cfg.n_blocks):
        for name in _BLOCK_TENSORS:
            yield name, b, make_tensor(cfg, name, b, planted=b in planted)
    yield "final_norm", -1, make_tensor(cfg, "final_norm")
    yield "lm_head", -1, make_tensor(cfg, "lm_head")


def make_weights(cfg: ModelConfig) -> Dict[str, object]:
    """All weights on the host: {'embed', 'lm_head', 'final_norm', 'blocks': [ {name: tensor} ]}."""
    w: Dict[str, object] = {"blocks": [dict() for _ in range(cfg.n_blocks)]}
    for name, b, t in iter_tensors(cfg):
        if b < 0:
            w[name] = t
        else:
            w["blocks"][b][name] = t
    return w


def prompt(cfg: ModelConfig, n: int, stream: int = 0) -> List[int]:
    """n uniform token ids in [0, vocab)."""
    return [_word(cfg.seed, TID_PROMPT, stream * (1 << 20) + i) % cfg.vocab for i in range(n)]


def block_mask(cfg: ModelConfig, blocks) -> np.ndarray:
    """uint8[2*n_blocks], order [attn_0, mlp_0, attn_1, ...], 1 = skip; both sub-layers of each block."""
    z = np.zeros(2 * cfg.n_blocks, dtype=np.uint8)
    for b in blocks:
        z[2 * b] = z[2 * b + 1] = 1
    return z


def draft_blocks(cfg: ModelConfig, n_skip: int) -> List[int]:
    """The fixed draft skip set: the planted blocks, topped up (or cut) to n_skip blocks by a seeded draw."""
    planted = planted_blocks(cfg)
    if n_skip <= len(planted):
        return planted[:n_skip]
    rest = [b for b in range(cfg.n_blocks) if b not in planted]
    extra = _subset(cfg.seed, TID_SHUFFLE, 1 << 16, len(rest), n_skip - len(planted))
    return sorted(planted + [rest[i] for i in extra])


def uniform_blocks(n_blocks: int, m: int) -> List[int]:
    """Evenly spread set of m blocks: block b is in it iff floor((b+1)m/nb) > floor(b m/nb)."""
    return [b for b in range(n_blocks) if ((b + 1) * m) // n_blocks > (b * m) // n_blocks]


def candidate_masks(cfg: ModelConfig, n_skip: int, count: int, round_index: int = 0) -> np.ndarray:
    """Random-search proposals: `count` uniform subsets of n_skip blocks, as sub-layer masks [count, 2*nb]."""
    out = np.zeros((count, 2 * cfg.n_blocks), dtype=np.uint8)
    for c in range(count):
        off = ((round_index * count + c) << 10)
        out[c] = block_mask(cfg, _subset(cfg.seed, TID_MASKS, off, cfg.n_blocks, n_skip))
    return out
