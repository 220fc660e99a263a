"""ctypes loader for the CPU oracle (oracle/aj_oracle.c).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's cpu-baseline / reference arms may
import this module.  It never imports the CUDA package and shares nothing with it.
"""
from __future__ import annotations

import ctypes
import hashlib
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "aj_oracle.c")
_LIB = None


def _cpu_tag() -> tuple[str, list[str]]:
    flags: set[str] = set()
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    flags = set(line.split(":", 1)[1].split())
                    break
    except OSError:
        pass
    if {"avx2", "fma"} <= flags:
        return "avx2", ["-mavx2", "-mfma"]
    return "generic", []


def lib_path() -> str:
    tag, _ = _cpu_tag()
    h = hashlib.sha1(open(_SRC, "rb").read()).hexdigest()[:10]
    return os.path.join(_HERE, f"libaj_oracle_{tag}_{h}.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP); the file name carries the ISA tag and source hash."""
    out = lib_path()
    if force or not os.path.exists(out):
        _, isa = _cpu_tag()
        tmp = f"{out}.{os.getpid()}.tmp"
        cmd = ["gcc", "-O3", "-fopenmp", "-fPIC", "-shared", "-std=c11", *isa, "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, out)
    return out


def _lib():
    global _LIB
    if _LIB is None:
        L = ctypes.CDLL(build())
        vp, ip, dp, fp = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p
        ci, cf = ctypes.c_int, ctypes.c_float
        L.ajo_num_threads.restype = ci
        L.ajo_logits.argtypes = [vp, vp, ci, ci, ci, ci, ci, dp]
        L.ajo_logits.restype = ci
        L.ajo_argmax.argtypes = [dp, ci, ip, dp, dp]
        L.ajo_argmax.restype = None
        L.ajo_judge_p.argtypes = [vp, vp, ci, fp, cf, ci, ci]
        L.ajo_judge_p.restype = ctypes.c_double
        L.ajo_verify.argtypes = [vp, vp, vp, ip, fp, cf, cf, ci, ci, ci, ci, ci, ci, ci, ci, ip, ip, ip, dp, dp, dp]
        L.ajo_verify.restype = ci
        u64 = ctypes.c_uint64
        L.ajo_verify_sampled.argtypes = [vp, vp, vp, ip, fp, cf, cf, ci, ci, ci, ci, ci, ci, ci, ci, ctypes.c_double, u64, u64, ci,
                                         ip, ip, ip, dp, dp, dp]
        L.ajo_verify_sampled.restype = ci
        L.ajo_philox4x32_10.argtypes = [vp, vp, vp]
        L.ajo_philox4x32_10.restype = None
        L.ajo_noise_uniform.argtypes = [u64, u64, ci, ci]
        L.ajo_noise_uniform.restype = ctypes.c_double
        L.ajo_gumbel.argtypes = [u64, u64, ci, ci]
        L.ajo_gumbel.restype = ctypes.c_double
        L.ajo_rank.argtypes = [dp, ci, ci, ctypes.c_double, ip]
        L.ajo_rank.restype = ci
        L.ajo_verify_topk.argtypes = [vp, vp, ip, ci, ctypes.c_double, ci, ci, ci, ci, ci, ci, ip, ip, ip, dp, dp, ip, ip]
        L.ajo_verify_topk.restype = ci
        _LIB = L
    return _LIB


def num_threads() -> int:
    return int(_lib().ajo_num_threads())


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _check_storage(a: np.ndarray, dtype: int, name: str) -> np.ndarray:
    want = np.uint16 if dtype == 0 else np.float32
    if a.dtype != want:
        raise TypeError(f"{name}: expected {want} storage for dtype {dtype}, got {a.dtype}")
    return np.ascontiguousarray(a)


def logits(h: np.ndarray, W: np.ndarray, dtype: int, w_layout: int = 0) -> np.ndarray:
    """fp64 logits [R, V] of R rows h [R, d] against the LM head."""
    h = _check_storage(h, dtype, "h")
    W = _check_storage(W, dtype, "W")
    R, d = h.shape
    V = W.shape[0] if w_layout == 0 else W.shape[1]
    assert (W.shape[1] if w_layout == 0 else W.shape[0]) == d
    out = np.empty((R, V), dtype=np.float64)
    rc = _lib().ajo_logits(_ptr(h), _ptr(W), dtype, w_layout, R, d, V, _ptr(out))
    if rc:
        raise RuntimeError(f"ajo_logits failed: {rc}")
    return out


def argmax(row: np.ndarray):
    """(lowest index of the maximum, the maximum, distance to the best other index)."""
    row = np.ascontiguousarray(row, dtype=np.float64)
    y = ctypes.c_int32()
    t = ctypes.c_double()
    g = ctypes.c_double()
    _lib().ajo_argmax(_ptr(row), row.shape[0], ctypes.byref(y), ctypes.byref(t), ctypes.byref(g))
    return int(y.value), float(t.value), float(g.value)


def judge_p(h_draft_row, h_target_row, dtype: int, judge_w: np.ndarray, judge_b: float) -> float:
    """P(important) for one position from [h_draft_row ; h_target_row]."""
    ht = _check_storage(h_target_row, dtype, "h_target_row")
    hd = None if h_draft_row is None else _check_storage(h_draft_row, dtype, "h_draft_row")
    w = np.ascontiguousarray(judge_w, dtype=np.float32)
    d = ht.shape[0]
    dd = 0 if hd is None else hd.shape[0]
    assert w.shape[0] == d + dd
    return float(_lib().ajo_judge_p(_ptr(hd), _ptr(ht), dtype, _ptr(w), float(judge_b), dd, d))


@dataclass
class OracleResult:
    accept_len: np.ndarray  # [B] int32
    next_tok: np.ndarray  # [B] int32
    target_tok: np.ndarray  # [B, K+1] int32
    top1: np.ndarray  # [B, K+1] float64
    gap: np.ndarray  # [B, K+1] float64
    judge_p: np.ndarray  # [B, K] float64, NaN where the draft token matched


def tree_accept(tok, parent, y, p, tau):
    """The acceptance rule on a draft tree (one sequence): (accept_len, best_node, next_tok)."""
    tok = np.ascontiguousarray(tok, dtype=np.int32)
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    y = np.ascontiguousarray(y, dtype=np.int32)
    p = np.ascontiguousarray(p, dtype=np.float64)
    N = tok.shape[0]
    assert parent.shape == (N,) and y.shape == (N + 1,) and p.shape == (N,)
    out = [ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()]
    L = _lib()
    L.ajo_tree_accept.argtypes = [ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_float,
                                  ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
    L.ajo_tree_accept.restype = None
    L.ajo_tree_accept(N, _ptr(tok), _ptr(parent), _ptr(y), _ptr(p), float(tau), *[ctypes.byref(o) for o in out])
    return tuple(int(o.value) for o in out)


def verify_tree(h_target, h_draft, W, draft_tok, parent, judge_w, judge_b, tau, dtype: int, w_layout: int = 0,
                temperature: float = 0.0, seed: int = 0, step: int = 0, row0: int = 0) -> OracleResult:
    """The whole step for tree drafts: h_target [B, N+1, d], draft_tok and parent [B, N]; the result also has best_node [B]."""
    ht = np.ascontiguousarray(h_target)
    B, R, d = ht.shape
    N = R - 1
    hd = None if h_draft is None else np.ascontiguousarray(h_draft)
    dd = 0 if hd is None else hd.shape[2]
    W = np.ascontiguousarray(W)
    V = W.shape[0] if w_layout == 0 else W.shape[1]
    tok = np.ascontiguousarray(draft_tok, dtype=np.int32)
    par = np.ascontiguousarray(parent, dtype=np.int32)
    assert tok.shape == (B, N) and par.shape == (B, N)
    w = np.ascontiguousarray(judge_w, dtype=np.float32)
    assert w.shape == (dd + d,)
    res = OracleResult(np.empty(B, np.int32), np.empty(B, np.int32), np.empty((B, R), np.int32), np.empty((B, R), np.float64),
                       np.empty((B, R), np.float64), np.empty((B, N), np.float64))
    best = np.empty(B, np.int32)
    L = _lib()
    vp, ci, u64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_uint64
    L.ajo_verify_tree.argtypes = [vp, vp, vp, vp, vp, vp, ctypes.c_float, ctypes.c_float, ci, ci, ci, ci, ci, ci, ci,
                                  ctypes.c_double, u64, u64, ci, vp, vp, vp, vp, vp, vp, vp]
    L.ajo_verify_tree.restype = ci
    rc = L.ajo_verify_tree(_ptr(ht), _ptr(hd), _ptr(W), _ptr(tok), _ptr(par), _ptr(w), float(judge_b), float(tau), dtype, w_layout,
                           B, N, d, dd, V, float(temperature), int(seed), int(step), int(row0), _ptr(res.accept_len), _ptr(res.next_tok),
                           _ptr(best), _ptr(res.target_tok), _ptr(res.top1), _ptr(res.gap), _ptr(res.judge_p))
    if rc:
        raise RuntimeError(f"ajo_verify_tree failed ({rc})")
    res.best_node = best
    return res


def philox4x32_10(ctr, key):
    """Philox4x32-10: four 32-bit counter words and two key words in, four words out."""
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.empty(4, dtype=np.uint32)
    _lib().ajo_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def noise_uniform(seed: int, step: int, j: int, v: int) -> float:
    return float(_lib().ajo_noise_uniform(seed, step, j, v))


def gumbel(seed: int, step: int, j: int, v: int) -> float:
    return float(_lib().ajo_gumbel(seed, step, j, v))


def verify(h_target, h_draft, W, draft_tok, judge_w, judge_b, tau, dtype: int, w_layout: int = 0,
           extra_row: bool = True, temperature: float = 0.0, seed: int = 0, step: int = 0, row0: int = 0) -> OracleResult:
    """The whole verify-and-judge step for B sequences (see aj_oracle.c for the definition).

    extra_row=False: the hidden states have K rows, not K + 1 (the last draft token is not encoded)."""
    ht = _check_storage(h_target, dtype, "h_target")
    hd = None if h_draft is None else _check_storage(h_draft, dtype, "h_draft")
    W = _check_storage(W, dtype, "W")
    tok = np.ascontiguousarray(draft_tok, dtype=np.int32)
    w = np.ascontiguousarray(judge_w, dtype=np.float32)
    B, R, d = ht.shape
    K = R - 1 if extra_row else R
    dd = 0 if hd is None else hd.shape[2]
    V = W.shape[0] if w_layout == 0 else W.shape[1]
    assert tok.shape == (B, K) and w.shape == (d + dd,)
    assert (W.shape[1] if w_layout == 0 else W.shape[0]) == d
    res = OracleResult(
        np.empty(B, np.int32), np.empty(B, np.int32), np.empty((B, R), np.int32),
        np.empty((B, R), np.float64), np.empty((B, R), np.float64), np.empty((B, K), np.float64),
    )
    rc = _lib().ajo_verify_sampled(
        _ptr(ht), _ptr(hd), _ptr(W), _ptr(tok), _ptr(w), float(judge_b), float(tau), dtype, w_layout,
        B, K, d, dd, V, 1 if extra_row else 0, float(temperature), int(seed), int(step), int(row0), _ptr(res.accept_len), _ptr(res.next_tok), _ptr(res.target_tok),
        _ptr(res.top1), _ptr(res.gap), _ptr(res.judge_p),
    )
    if rc:
        raise RuntimeError(f"ajo_verify failed: {rc}")
    return res


def rewalk(target_tok, draft_tok, judge_p_all, tau):
    """Steps 3-5 again for another tau from a stored result (no projection is redone).

    This calls back into nothing: it replays the accept walk on the oracle's own y and p
    so that tau sweeps over one (h, W) do not repeat the fp64 projection.
    """
    target_tok = np.asarray(target_tok)
    draft_tok = np.asarray(draft_tok)
    B, K = draft_tok.shape
    acc = np.empty(B, np.int32)
    nxt = np.empty(B, np.int32)
    for b in range(B):
        n = 0
        while n < K:
            if draft_tok[b, n] != target_tok[b, n]:
                p = judge_p_all[b, n]
                ok = False if tau <= 0 else True if tau >= 1 else bool(np.float32(p) < np.float32(tau))
                if not ok:
                    break
            n += 1
        acc[b] = n
        nxt[b] = target_tok[b, n]
    return acc, nxt


def rank(row: np.ndarray, tok: int, band: float = 0.0):
    """(rank of entry tok by decreasing logit, ties by index; number of other entries within band of it)."""
    row = np.ascontiguousarray(row, dtype=np.float64)
    near = ctypes.c_int32()
    r = _lib().ajo_rank(_ptr(row), row.shape[0], int(tok), float(band), ctypes.byref(near))
    return int(r), int(near.value)


@dataclass
class TopKResult:
    accept_len: np.ndarray  # [B]
    next_tok: np.ndarray  # [B]
    target_tok: np.ndarray  # [B, K+1]
    top1: np.ndarray  # [B, K+1]
    gap: np.ndarray  # [B, K+1]
    rank: np.ndarray  # [B, K]: -1 where the draft token matched
    near: np.ndarray  # [B, K]


def verify_topk(h_target, W, draft_tok, top_k: int, dtype: int, w_layout: int = 0, band: float = 1e-2) -> TopKResult:
    """The step under the top-K rule of Section 4.1 (see aj_oracle.c)."""
    ht = _check_storage(h_target, dtype, "h_target")
    W = _check_storage(W, dtype, "W")
    tok = np.ascontiguousarray(draft_tok, dtype=np.int32)
    B, R, d = ht.shape
    K = R - 1
    V = W.shape[0] if w_layout == 0 else W.shape[1]
    res = TopKResult(np.empty(B, np.int32), np.empty(B, np.int32), np.empty((B, R), np.int32), np.empty((B, R), np.float64),
                     np.empty((B, R), np.float64), np.empty((B, K), np.int32), np.empty((B, K), np.int32))
    rc = _lib().ajo_verify_topk(_ptr(ht), _ptr(W), _ptr(tok), int(top_k), float(band), dtype, w_layout, B, K, d, V,
                                _ptr(res.accept_len), _ptr(res.next_tok), _ptr(res.target_tok), _ptr(res.top1), _ptr(res.gap),
                                _ptr(res.rank), _ptr(res.near))
    if rc:
        raise RuntimeError(f"ajo_verify_topk failed: {rc}")
    return res
