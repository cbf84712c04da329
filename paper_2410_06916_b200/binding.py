"""ctypes binding of include/swift.h.  Argument marshalling only: every step of the decoding path
runs inside the CUDA library; torch supplies device memory and the stream.  There is no fallback:
if the library cannot be built or loaded, importing callers get an exception."""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Iterable, List, Optional, Sequence, Tuple

import numpy as np
import torch

from . import build as _build

MAX_ROWS = 16
_KINDS = {"embed": 0, "lm_head": 1, "final_norm": 2, "wq": 3, "wk": 4, "wv": 5, "wo": 6, "wgate": 7,
          "wup": 8, "wdown": 9, "attn_norm": 10, "mlp_norm": 11}
_STATUS = {0: "OK", 1: "EINVAL", 2: "ESTATE", 3: "ECAPACITY", 4: "ECUDA", 5: "ETIMEOUT", 6: "EUNSUPPORTED"}


class SwiftError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"SWIFT_{_STATUS.get(status, status)}: {message}")
        self.status = status


class _Desc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_blocks", "d_model", "n_heads", "n_kv_heads", "head_dim", "ffn", "vocab",
                                         "dtype")] + \
               [("rope_theta", C.c_float), ("rms_eps", C.c_float)] + \
               [(n, C.c_int32) for n in ("max_positions", "page_size", "max_draft", "kv_dtype")]


class _DevBuf(C.Structure):
    _fields_ = [("dptr", C.c_void_p), ("bytes", C.c_size_t)]


class _GenParams(C.Structure):
    _fields_ = [("max_new", C.c_int32), ("max_draft", C.c_int32), ("stop_conf", C.c_float), ("vanilla", C.c_int32),
                ("gamma", C.c_int32), ("n_candidates", C.c_int32), ("n_opt_rounds", C.c_int32),
                ("stop_matchness", C.c_float), ("opt_patience", C.c_int32), ("opt_skip_blocks", C.c_int32),
                ("opt_beta", C.c_int32), ("opt_seed", C.c_uint64), ("skip_mask", C.c_void_p), ("candidate_masks", C.c_void_p)]


class _Stats(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("tokens", "rounds", "drafted", "accepted", "opt_rounds", "reserved")] + \
               [(n, C.c_float) for n in ("best_matchness", "ms_prefill", "ms_decode", "ms_draft", "ms_verify", "ms_score")] + \
               [("bytes_draft", C.c_double), ("bytes_verify", C.c_double), ("kernel_launches", C.c_int64),
                ("h2d_bytes", C.c_int64), ("d2h_bytes", C.c_int64)]


# every symbol include/swift.h declares
SYMBOLS = ("swift_weights_bytes", "swift_kv_bytes", "swift_workspace_bytes", "swift_load", "swift_free",
           "swift_last_error", "swift_pack_tensor", "swift_set_sampling", "swift_set_top_p", "swift_set_greedy_draft", "swift_forward_rows", "swift_prefill",
           "swift_set_pending", "swift_draft", "swift_verify", "swift_accept", "swift_score_skipsets", "swift_generate",
           "swift_committed_length", "swift_launch_count", "swift_round_times", "swift_round_bytes_stored", "swift_final_skip_mask", "swift_forward_bytes", "swift_read_kv", "swift_time_gemm", "swift_set_gemm_impl", "swift_gemm", "swift_gemm_static",
           "swift_gemm_static_error", "swift_probe_wait_limit", "swift_many_row_schedule", "swift_set_tree", "swift_verify_tree", "swift_tree_rows", "swift_opt_create", "swift_opt_free", "swift_opt_suggest", "swift_opt_observe")

_lib = None


def load_library(path: Optional[str] = None) -> C.CDLL:
    """Builds (if stale) and loads libswift_b200.so; raises if that is not possible."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or _build.build()
    lib = C.CDLL(p)
    vp, i32, u64, f32 = C.c_void_p, C.c_int32, C.c_uint64, C.c_float
    for name in ("swift_weights_bytes", "swift_kv_bytes", "swift_workspace_bytes"):
        getattr(lib, name).argtypes = [C.POINTER(_Desc)]
        getattr(lib, name).restype = C.c_size_t
    lib.swift_load.argtypes = [C.POINTER(_Desc), _DevBuf, _DevBuf, _DevBuf, vp, C.POINTER(vp)]
    lib.swift_free.argtypes = [vp]
    lib.swift_last_error.argtypes = [vp]
    lib.swift_last_error.restype = C.c_char_p
    lib.swift_pack_tensor.argtypes = [vp, i32, i32, vp, C.c_size_t]
    lib.swift_set_sampling.argtypes = [vp, i32, f32, u64]
    lib.swift_set_top_p.argtypes = [vp, f32]
    lib.swift_set_greedy_draft.argtypes = [vp, i32]
    lib.swift_forward_rows.argtypes = [vp, vp, i32, i32, vp, i32, vp, vp]
    lib.swift_prefill.argtypes = [vp, vp, i32, vp]
    lib.swift_set_pending.argtypes = [vp, i32, i32]
    lib.swift_draft.argtypes = [vp, vp, i32, f32, vp, vp, vp]
    lib.swift_verify.argtypes = [vp, vp, i32, vp, vp]
    lib.swift_accept.argtypes = [vp, vp, vp]
    lib.swift_score_skipsets.argtypes = [vp, vp, i32, i32, vp]
    lib.swift_generate.argtypes = [vp, C.POINTER(_GenParams), vp, i32, vp, vp, vp, C.POINTER(_Stats)]
    lib.swift_committed_length.argtypes = [vp]
    lib.swift_launch_count.argtypes = [vp]
    lib.swift_launch_count.restype = C.c_int64
    lib.swift_final_skip_mask.argtypes = [vp, vp]
    lib.swift_final_skip_mask.restype = C.c_int32
    lib.swift_round_times.argtypes = [vp, i32, vp, vp, vp, vp, vp]
    lib.swift_round_times.restype = C.c_int32
    lib.swift_probe_wait_limit.argtypes = [vp, i32]
    lib.swift_many_row_schedule.argtypes = [i32, i32, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    lib.swift_set_tree.argtypes = [vp, i32]
    lib.swift_verify_tree.argtypes = [vp, vp, vp, i32, vp, vp]
    lib.swift_tree_rows.argtypes = [vp, vp, vp, vp]
    lib.swift_tree_rows.restype = C.c_int32
    lib.swift_opt_create.argtypes = [i32, i32, i32, C.c_uint64, i32]
    lib.swift_opt_create.restype = vp
    lib.swift_opt_free.argtypes = [vp]
    lib.swift_opt_free.restype = None
    lib.swift_opt_suggest.argtypes = [vp, vp, vp]
    lib.swift_opt_observe.argtypes = [vp, vp, C.c_float]
    lib.swift_round_bytes_stored.argtypes = [vp, i32, vp, vp]
    lib.swift_round_bytes_stored.restype = C.c_int32
    lib.swift_forward_bytes.argtypes = [vp, vp, i32, i32, i32]
    lib.swift_forward_bytes.restype = C.c_double
    lib.swift_set_gemm_impl.argtypes = [vp, i32]
    lib.swift_gemm_static.argtypes = [vp, i32, i32, i32, vp, i32, vp, vp]
    lib.swift_gemm_static_error.argtypes = []
    lib.swift_gemm_static_error.restype = C.c_char_p
    lib.swift_gemm.argtypes = [vp, i32, i32, vp, i32, vp]
    lib.swift_time_gemm.argtypes = [vp, i32, i32, i32, vp, vp]
    lib.swift_read_kv.argtypes = [vp, i32, i32, i32, i32, vp]
    for name in SYMBOLS:
        fn = getattr(lib, name)          # AttributeError if a declared symbol is missing
        if fn.restype is C.c_int:
            fn.restype = C.c_int32
    if path is None:
        _lib = lib
    return lib


def lib() -> C.CDLL:
    return load_library()


@dataclass
class GenParams:
    max_new: int
    max_draft: int = 8
    stop_conf: float = 0.0
    vanilla: bool = False
    gamma: int = 32
    n_opt_rounds: int = 0
    stop_matchness: float = 0.95
    opt_patience: int = 0                             # optimisation rounds without a replacement before it stops (0 = no rule)
    n_candidates: int = 0                             # proposals per round when the library makes them itself (candidate_masks None)
    opt_skip_blocks: int = 0                          # ... sets of this many whole blocks,
    opt_beta: int = 25                                # ... a Gaussian-process proposal every opt_beta-th one (0 = random search only)
    opt_seed: int = 0
    skip_mask: Optional[np.ndarray] = None            # uint8 [2*n_blocks]
    candidate_masks: Optional[np.ndarray] = None      # uint8 [n_opt_rounds, C, 2*n_blocks]


@dataclass
class GenStats:
    tokens: int
    rounds: int
    drafted: int
    accepted: int
    opt_rounds: int
    best_matchness: float
    ms_prefill: float
    ms_decode: float
    ms_draft: float
    ms_verify: float
    ms_score: float
    bytes_draft: float
    bytes_verify: float
    kernel_launches: int
    h2d_bytes: int = 0
    d2h_bytes: int = 0


STATIC_SCRATCH_BYTES = 8 * 1024 * 1024


class LayerSetOptimizer:
    """The library's proposal engine for the on-the-fly optimisation (Section 4.1), usable on its own: host code
    only, no device needed.  suggest() -> (mask uint8[2*n_blocks], came from the Gaussian-process step); observe(mask, score)."""

    def __init__(self, n_blocks: int, n_skip_blocks: int, beta: int = 25, seed: int = 0, pool: int = 512):
        self._lib = load_library()
        self.n_sub = 2 * n_blocks
        self._h = self._lib.swift_opt_create(n_blocks, n_skip_blocks, beta, seed, pool)
        if not self._h:
            raise ValueError("swift_opt_create rejected the arguments")

    def suggest(self) -> Tuple[np.ndarray, bool]:
        m = np.zeros(self.n_sub, dtype=np.uint8)
        b = C.c_int32()
        if self._lib.swift_opt_suggest(self._h, _ptr(m), C.byref(b)) != 0:
            raise SwiftError("swift_opt_suggest failed")
        return m, bool(b.value)

    def observe(self, mask, matchness: float) -> None:
        if self._lib.swift_opt_observe(self._h, _ptr(_u8(mask)), float(matchness)) != 0:
            raise SwiftError("swift_opt_observe failed")

    def close(self) -> None:
        if self._h:
            self._lib.swift_opt_free(self._h)
            self._h = None

    def __del__(self):
        self.close()


def many_row_schedule(n: int, k: int) -> Tuple[int, int]:
    """(grid, largest number of CTAs sharing one output tile) of the many-row GEMM for an [n][k] weight; host only."""
    grid, share = C.c_int32(), C.c_int32()
    st = lib().swift_many_row_schedule(n, k, C.byref(grid), C.byref(share))
    if st != 0:
        raise SwiftError(f"swift_many_row_schedule({n}, {k}): status {st}")
    return grid.value, share.value


def gemm_static(w: torch.Tensor, x: torch.Tensor, y: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> None:
    """y = x @ w.T through swift_gemm_static: w [N, K] fp32 or bf16, x [rows <= 16, K] fp32, y [rows, N] fp32, all
    contiguous CUDA tensors the caller made beforehand.  The call itself allocates nothing (its scratch is an
    array inside the library) and only enqueues work on `stream` (default: the current stream)."""
    if not (w.is_cuda and x.is_cuda and y.is_cuda and w.is_contiguous() and x.is_contiguous() and y.is_contiguous()):
        raise ValueError("w, x, y must be contiguous CUDA tensors")
    if x.dtype != torch.float32 or y.dtype != torch.float32 or w.dtype not in (torch.float32, torch.bfloat16):
        raise TypeError("x, y fp32; w fp32 or bf16")
    if w.dim() != 2 or x.dim() != 2 or x.shape[1] != w.shape[1] or tuple(y.shape) != (x.shape[0], w.shape[0]):
        raise ValueError("shape mismatch")
    s = stream if stream is not None else torch.cuda.current_stream(w.device)
    with torch.cuda.device(w.device):
        st = lib().swift_gemm_static(C.c_void_p(w.data_ptr()), 1 if w.dtype == torch.bfloat16 else 0, w.shape[0], w.shape[1],
                                     C.c_void_p(x.data_ptr()), x.shape[0], C.c_void_p(y.data_ptr()), C.c_void_p(s.cuda_stream))
    if st != 0:
        raise SwiftError(st, lib().swift_gemm_static_error().decode())


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _u8(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.uint8))


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


class SwiftModel:
    """One model + KV cache + workspace on one GPU, driven through the C boundary."""

    def __init__(self, cfg, max_positions: int, page_size: int = 16, max_draft: int = 15, device: str = "cuda:0",
                 kv_dtype: str = "f32"):
        """kv_dtype: storage of cached K,V: "f32" (default: keeps the logits within the parity tolerance) or
        "bf16" (halves the cache and its traffic; fp32 models always use "f32")."""
        if not torch.cuda.is_available():
            raise RuntimeError("paper_2410_06916_b200 needs a CUDA device (B200); there is no CPU path")
        self._lib = lib()
        self.cfg = cfg
        self.device = torch.device(device)
        max_positions = (max_positions + page_size - 1) // page_size * page_size
        self.desc = _Desc(cfg.n_blocks, cfg.d_model, cfg.n_heads, cfg.n_kv_heads, cfg.head_dim, cfg.ffn, cfg.vocab,
                          1 if cfg.dtype == "bf16" else 0, cfg.rope_theta, cfg.rms_eps, max_positions, page_size,
                          max_draft, 1 if (kv_dtype == "bf16" and cfg.dtype == "bf16") else 0)
        sizes = [self._lib.swift_weights_bytes(C.byref(self.desc)), self._lib.swift_kv_bytes(C.byref(self.desc)),
                 self._lib.swift_workspace_bytes(C.byref(self.desc))]
        if 0 in sizes:
            raise SwiftError(1, "invalid model description")
        self.ctx = C.c_void_p()
        with torch.cuda.device(self.device):
            self.stream = torch.cuda.Stream(device=self.device)
            self._bufs = [torch.empty(s + 256, dtype=torch.uint8, device=self.device) for s in sizes]
            devbufs = []
            for b, s in zip(self._bufs, sizes):
                p = (b.data_ptr() + 255) // 256 * 256
                devbufs.append(_DevBuf(p, s))
            st = self._lib.swift_load(C.byref(self.desc), *devbufs, C.c_void_p(self.stream.cuda_stream), C.byref(self.ctx))
        if st != 0:
            raise SwiftError(st, self._lib.swift_last_error(None).decode())
        self.weight_bytes, self.kv_bytes, self.workspace_bytes = sizes
        self.vocab, self.n_sub = cfg.vocab, 2 * cfg.n_blocks

    # ------------------------------------------------------------------ plumbing
    def _check(self, st: int):
        if st != 0:
            raise SwiftError(st, self._lib.swift_last_error(self.ctx).decode())

    def close(self):
        if getattr(self, "ctx", None) and self.ctx.value:
            self._lib.swift_free(self.ctx)
            self.ctx = C.c_void_p()
            self._bufs = []

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def pack(self, name: str, block: int, t: torch.Tensor):
        want = torch.float32 if name.endswith("norm") or self.cfg.dtype == "f32" else torch.bfloat16
        t = t.detach().to("cpu").contiguous()
        if t.dtype != want:
            raise TypeError(f"{name}: expected {want}, got {t.dtype}")
        with torch.cuda.device(self.device):
            self._check(self._lib.swift_pack_tensor(self.ctx, _KINDS[name], block, C.c_void_p(t.data_ptr()),
                                                    t.numel() * t.element_size()))

    def load_weights(self, tensors: Iterable[Tuple[str, int, torch.Tensor]]):
        for name, block, t in tensors:
            self.pack(name, block, t)

    def set_sampling(self, sampling: bool, temperature: float = 1.0, seed: int = 0, top_p: float = 1.0,
                     greedy_draft: bool = False):
        self._check(self._lib.swift_set_sampling(self.ctx, 1 if sampling else 0, temperature, seed))
        self._check(self._lib.swift_set_top_p(self.ctx, top_p))
        self._check(self._lib.swift_set_greedy_draft(self.ctx, 1 if greedy_draft else 0))

    @property
    def n(self) -> int:
        return self._lib.swift_committed_length(self.ctx)

    @property
    def launches(self) -> int:
        return self._lib.swift_launch_count(self.ctx)

    def forward_bytes(self, skip_mask, n_rows: int, n_context: int, kv_elem_bytes: int = 2) -> float:
        """HBM bytes one forward must move; cached K,V counted at kv_elem_bytes per element (0 = as this context stores them)."""
        m = None if skip_mask is None else _u8(skip_mask)
        return self._lib.swift_forward_bytes(self.ctx, _ptr(m), n_rows, n_context, kv_elem_bytes)

    # ------------------------------------------------------------------ the steps
    def forward_rows(self, tokens: Sequence[int], pos0: int, skip_mask=None, write_kv: bool = True,
                     want_logits: bool = True) -> Tuple[Optional[np.ndarray], np.ndarray]:
        t = _i32(tokens)
        m = None if skip_mask is None else _u8(skip_mask)
        logits = np.empty((len(t), self.vocab), dtype=np.float32) if want_logits else None
        am = np.empty(len(t), dtype=np.int32)
        with torch.cuda.device(self.device):
            self._check(self._lib.swift_forward_rows(self.ctx, _ptr(t), len(t), pos0, _ptr(m), 1 if write_kv else 0,
                                                     _ptr(logits), _ptr(am)))
        return logits, am

    def prefill(self, tokens: Sequence[int]) -> int:
        t = _i32(tokens)
        first = C.c_int32()
        with torch.cuda.device(self.device):
            self._check(self._lib.swift_prefill(self.ctx, _ptr(t), len(t), C.byref(first)))
        return first.value

    def set_pending(self, token: int, rounds_done: int = -1):
        self._check(self._lib.swift_set_pending(self.ctx, int(token), int(rounds_done)))

    def draft(self, skip_mask, max_k: int, stop_conf: float = 0.0) -> Tuple[List[int], List[float]]:
        m = _u8(skip_mask)
        toks = np.zeros(max(max_k, 1), dtype=np.int32)
        conf = np.zeros(max(max_k, 1), dtype=np.float32)
        k = C.c_int32()
        with torch.cuda.device(self.device):
            self._check(self._lib.swift_draft(self.ctx, _ptr(m), max_k, stop_conf, _ptr(toks), _ptr(conf), C.byref(k)))
        return toks[:k.value].tolist(), conf[:k.value].tolist()

    def verify(self, tokens: Optional[Sequence[int]] = None, want_logits: bool = True):
        t = None if tokens is None else _i32(tokens)
        k = 0 if t is None else len(t)
        am = np.zeros(MAX_ROWS, dtype=np.int32)
        logits = np.empty((MAX_ROWS, self.vocab), dtype=np.float32) if want_logits else None
        tp = None if t is None else (_ptr(t) if k > 0 else C.c_void_p(am.ctypes.data))  # non-null marks "tokens given"
        with torch.cuda.device(self.device):
            self._check(self._lib.swift_verify(self.ctx, tp, k, _ptr(am), _ptr(logits)))
        return am, logits

    def probe_wait_limit(self, limit_us: int = 1000) -> None:
        """Lets one bounded device-side wait run out (harmlessly); raises SwiftError(ETIMEOUT), after which the model works on."""
        with torch.cuda.device(self.device):
            self._check(self._lib.swift_probe_wait_limit(self.ctx, limit_us))

    def set_tree(self, tree_rows: int) -> None:
        """Dynamic verification (Section 4.2): rows one verification of the device's own drafts may hold (0 = the chain only)."""
        self._check(self._lib.swift_set_tree(self.ctx, tree_rows))

    def verify_tree(self, tokens: Sequence[int], parent: Sequence[int], want_logits: bool = True):
        t, p = _i32(tokens), _i32(parent)
        am = np.zeros(MAX_ROWS, dtype=np.int32)
        logits = np.empty((MAX_ROWS, self.vocab), dtype=np.float32) if want_logits else None
        with torch.cuda.device(self.device):
            self._check(self._lib.swift_verify_tree(self.ctx, _ptr(t), _ptr(p), len(t), _ptr(am), _ptr(logits)))
        return am[:len(t)], (logits[:len(t)] if want_logits else None)

    def tree_rows(self):
        """(tokens, parent, depth) of the tree the last verification held (empty for a plain chain)."""
        t, p, d = (np.zeros(MAX_ROWS, dtype=np.int32) for _ in range(3))
        n = self._lib.swift_tree_rows(self.ctx, _ptr(t), _ptr(p), _ptr(d))
        return t[:n].tolist(), p[:n].tolist(), d[:n].tolist()

    def accept(self) -> Tuple[int, int]:
        a, nxt = C.c_int32(), C.c_int32()
        with torch.cuda.device(self.device):
            self._check(self._lib.swift_accept(self.ctx, C.byref(a), C.byref(nxt)))
        return a.value, nxt.value

    def score_skipsets(self, masks, gamma: int) -> np.ndarray:
        m = _u8(masks).reshape(-1, self.n_sub)
        out = np.zeros(m.shape[0], dtype=np.float32)
        with torch.cuda.device(self.device):
            self._check(self._lib.swift_score_skipsets(self.ctx, _ptr(m), m.shape[0], gamma, _ptr(out)))
        return out

    def generate(self, prompt: Sequence[int], gp: GenParams) -> Tuple[List[int], GenStats, np.ndarray]:
        p = _i32(prompt)
        skip = None if gp.skip_mask is None else _u8(gp.skip_mask)
        cands = None if gp.candidate_masks is None else _u8(gp.candidate_masks)
        n_cand = gp.n_candidates if cands is None else cands.reshape(gp.n_opt_rounds, -1, self.n_sub).shape[1]
        own = cands is None and gp.n_candidates > 0 and gp.opt_skip_blocks > 0      # the library proposes the candidates
        cp = _GenParams(gp.max_new, gp.max_draft, gp.stop_conf, 1 if gp.vanilla else 0, gp.gamma, n_cand,
                        gp.n_opt_rounds if (cands is not None or own) else 0, gp.stop_matchness, gp.opt_patience,
                        gp.opt_skip_blocks, gp.opt_beta, gp.opt_seed, _ptr(skip), _ptr(cands))
        out = np.zeros(gp.max_new, dtype=np.int32)
        trace = np.zeros((gp.max_new, 4), dtype=np.int32)
        n_out = C.c_int32()
        st = _Stats()
        with torch.cuda.device(self.device):
            self._check(self._lib.swift_generate(self.ctx, C.byref(cp), _ptr(p), len(p), _ptr(out), C.byref(n_out),
                                                 _ptr(trace), C.byref(st)))
        stats = GenStats(**{f: getattr(st, f) for f in GenStats.__dataclass_fields__})
        return out[:n_out.value].tolist(), stats, trace[:stats.rounds]

    def final_skip_mask(self) -> Optional[np.ndarray]:
        """The skip set the last generate() ended with (to seed the next input of a stream), or None."""
        m = np.zeros(self.n_sub, dtype=np.uint8)
        return m if self._lib.swift_final_skip_mask(self.ctx, _ptr(m)) == self.n_sub else None

    def round_times(self):
        """Per round of the last generate(): (ms_draft, ms_verify, bytes_draft, bytes_verify, drafted) arrays."""
        n = self._lib.swift_round_times(self.ctx, 0, None, None, None, None, None)
        md, mv = np.zeros(n, dtype=np.float32), np.zeros(n, dtype=np.float32)
        bd, bv = np.zeros(n, dtype=np.float64), np.zeros(n, dtype=np.float64)
        k = np.zeros(n, dtype=np.int32)
        self._lib.swift_round_times(self.ctx, n, _ptr(md), _ptr(mv), _ptr(bd), _ptr(bv), _ptr(k))
        return md, mv, bd, bv, k

    def round_bytes_stored(self):
        """Per round of the last generate(): (bytes_draft, bytes_verify) with cached K,V counted as stored."""
        n = self._lib.swift_round_bytes_stored(self.ctx, 0, None, None)
        bd, bv = np.zeros(n, dtype=np.float64), np.zeros(n, dtype=np.float64)
        self._lib.swift_round_bytes_stored(self.ctx, n, _ptr(bd), _ptr(bv))
        return bd, bv

    def set_gemm_impl(self, tensor_cores: bool):
        self._check(self._lib.swift_set_gemm_impl(self.ctx, 1 if tensor_cores else 0))

    def gemm(self, which: int, block: int, x: np.ndarray) -> np.ndarray:
        """y = x @ W^T for one stored weight (fused / interleaved row order), through the library's GEMM kernel."""
        x = np.ascontiguousarray(x, dtype=np.float32)
        c = self.cfg
        n = [c.q_dim + 2 * c.kv_dim, c.d_model, 2 * c.ffn, c.d_model, c.vocab][which]
        y = np.empty((x.shape[0], n), dtype=np.float32)
        with torch.cuda.device(self.device):
            self._check(self._lib.swift_gemm(self.ctx, which, block, _ptr(x), x.shape[0], _ptr(y)))
        return y

    def time_gemm(self, which: int, n_rows: int, iters: int) -> Tuple[float, float]:
        """(ms per launch, weight bytes per launch) of one weight-streaming GEMM of the walk."""
        ms, nbytes = C.c_float(), C.c_double()
        with torch.cuda.device(self.device):
            self._check(self._lib.swift_time_gemm(self.ctx, which, n_rows, iters, C.byref(ms), C.byref(nbytes)))
        return ms.value, nbytes.value

    def read_kv(self, block: int, which: int, pos0: int, count: int) -> np.ndarray:
        out = np.empty((count, self.cfg.n_kv_heads, self.cfg.head_dim), dtype=np.float32)
        with torch.cuda.device(self.device):
            self._check(self._lib.swift_read_kv(self.ctx, block, which, pos0, count, _ptr(out)))
        return out
