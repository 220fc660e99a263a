"""Seeded synthetic inputs for the verify-and-judge step.

This module only draws numbers and lays them out in memory.  It holds none of the
method's arithmetic (no projection, no argmax, no judge, no prefix walk), so that both
the CPU oracle's tests and the CUDA library's tests and benchmark can share it.

The shapes follow Llama-3.x draft/target pairs (Section 4 of the paper: Llama-3.2-1B /
Llama-3.1-8B and Llama-3.1-8B / Llama-3.1-70B, bfloat16).  The values are i.i.d.
Gaussians: the paper's datasets and weights are not available, only their shapes are used.

Every tensor has its own Philox stream keyed by (seed, tensor id), so a tensor's values
do not depend on which other tensors were drawn or in what order.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np

GENERATOR_VERSION = "aj_inputs/1"

BF16 = 0  # storage: uint16 holding the upper half of an IEEE fp32
F32 = 1

_T_W, _T_HT, _T_HD, _T_JW, _T_RATE, _T_TOK, _T_LRX, _T_LRU, _T_LRN = range(9)


@dataclass(frozen=True)
class Config:
    name: str
    B: int
    K: int
    d: int
    d_draft: int
    V: int
    dtype: int = BF16
    sigma_W: float = 0.02
    sigma_h: float = 1.0
    sigma_w: float = 0.02
    judge_b: float = 0.0
    tau: float = 0.5
    match_lo: float = 0.7  # per-sequence match rate ~ U(match_lo, match_hi)
    match_hi: float = 0.7
    seed: int = 0

    @property
    def M(self) -> int:
        return self.B * (self.K + 1)

    @property
    def F(self) -> int:
        return self.d_draft + self.d


# The five workloads named by the benchmark definition.
C1 = Config("c1_tiny_f32", B=1, K=4, d=256, d_draft=128, V=1000, dtype=F32, sigma_w=0.05)
C2 = Config("c2_8b_b1_k16", B=1, K=16, d=4096, d_draft=2048, V=128256)
C3 = Config("c3_8b_b64_k32", B=64, K=32, d=4096, d_draft=2048, V=128256, match_lo=0.5, match_hi=0.95)
C4 = Config("c4_70b_b32_k64", B=32, K=64, d=8192, d_draft=4096, V=128256, match_lo=0.6, match_hi=0.6)
C2_TAUS = (0.0, 0.5, 1.0)
C4_TAUS = tuple(round(0.1 * i, 1) for i in range(1, 10))
SWEEP_B = (1, 8, 64, 256)
SWEEP_K = (8, 16, 32, 64)


def sweep_config(B: int, K: int) -> Config:
    return Config(f"c5_8b_b{B}_k{K}", B=B, K=K, d=4096, d_draft=2048, V=128256)


CONFIGS = {c.name: c for c in (C1, C2, C3, C4)}


def scaled(cfg: Config, **kw) -> Config:
    """A copy of cfg with some fields replaced (used for cut-down test shapes)."""
    return replace(cfg, **kw)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bfloat16 (nearest, ties to even); returns the 16 stored bits."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def to_f64(a: np.ndarray, dtype: int) -> np.ndarray:
    """Exact widening of a stored tensor to float64 (for checks that need the values)."""
    return (bf16_bits_to_f32(a) if dtype == BF16 else a).astype(np.float64)


def _rng(seed: int, tensor_id: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed, tensor_id]))


def _normal(seed: int, tensor_id: int, shape, sigma: float, dtype: int, chunk: int = 1 << 24) -> np.ndarray:
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.uint16 if dtype == BF16 else np.float32)
    g = _rng(seed, tensor_id)
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        x = g.standard_normal(e - s, dtype=np.float32) * np.float32(sigma)
        out[s:e] = f32_to_bf16_bits(x) if dtype == BF16 else x
    return out.reshape(shape)


def make_W(cfg: Config, layout: int = 0) -> np.ndarray:
    """LM head.  layout 0: row-major [V, d] (one row per vocabulary entry); 1: row-major [d, V]."""
    W = _normal(cfg.seed, _T_W, (cfg.V, cfg.d), cfg.sigma_W, cfg.dtype)
    return W if layout == 0 else np.ascontiguousarray(W.T)


def make_hidden(cfg: Config):
    """(h_target [B,K+1,d], h_draft [B,K+1,d_draft] or None)."""
    ht = _normal(cfg.seed, _T_HT, (cfg.B, cfg.K + 1, cfg.d), cfg.sigma_h, cfg.dtype)
    hd = None
    if cfg.d_draft > 0:
        hd = _normal(cfg.seed, _T_HD, (cfg.B, cfg.K + 1, cfg.d_draft), cfg.sigma_h, cfg.dtype)
    return ht, hd


def make_judge(cfg: Config) -> np.ndarray:
    """Classifier weights, fp32, ordered [draft features ; target features]."""
    return _normal(cfg.seed, _T_JW, (cfg.F,), cfg.sigma_w, F32)


def match_rates(cfg: Config) -> np.ndarray:
    return _rng(cfg.seed, _T_RATE).uniform(cfg.match_lo, cfg.match_hi, size=cfg.B)


def plant_draft_tokens(cfg: Config, y: np.ndarray, rows=None) -> np.ndarray:
    """Draft tokens planted against given target tokens y [n, K+1] (int).

    Position i copies y[:, i] with the sequence's match rate, else takes a token drawn
    uniformly from the other V-1 ids.  `rows` names which sequences of the batch the n
    rows of y are (default: the first n); each sequence has its own stream, so a
    sequence's draft tokens do not depend on which others are planted.
    """
    y = np.asarray(y)
    n = y.shape[0]
    rows = list(range(n)) if rows is None else list(rows)
    rates = match_rates(cfg)
    out = np.empty((n, cfg.K), dtype=np.int32)
    for r, b in enumerate(rows):
        g = np.random.Generator(np.random.Philox(key=[cfg.seed, (_T_TOK << 32) + b]))
        keep = g.random(cfg.K) < rates[b]
        other = g.integers(0, cfg.V - 1, size=cfg.K)
        other = other + (other >= y[r, : cfg.K])  # skip the true token
        out[r] = np.where(keep, y[r, : cfg.K], other).astype(np.int32)
    return out


def random_draft_tokens(cfg: Config) -> np.ndarray:
    """Draft tokens drawn without reference to any target token (almost all mismatch)."""
    return _rng(cfg.seed, _T_TOK).integers(0, cfg.V, size=(cfg.B, cfg.K)).astype(np.int32)


def make_labelled_features(n: int, F: int, dtype: int = BF16, seed: int = 1234, important: float = 0.2, noise: float = 1.0):
    """A synthetic training set for the classifier: n feature rows [n, F] (i.i.d. unit Gaussians in the given
    storage, like the hidden states above) and labels [n] uint8, 1 = "important".  A row is labelled important
    when its projection on a random unit direction plus Gaussian noise of the given size is among the largest
    `important` share (the paper reports about 20 % important among the mismatches it mines, Section 4.1), so
    the labels are learnable but not separable."""
    X = _normal(seed, _T_LRX, (n, F), 1.0, dtype)
    u = _rng(seed, _T_LRU).standard_normal(F)
    u /= np.linalg.norm(u)
    score = to_f64(X, dtype) @ u + noise * _rng(seed, _T_LRN).standard_normal(n)
    cut = np.quantile(score, 1.0 - important)
    return X, (score > cut).astype(np.uint8)
