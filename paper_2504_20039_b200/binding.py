"""ctypes binding of the aj_verify C-ABI (include/aj_verify.h).

Argument marshalling only: every step of the verify-and-judge cycle runs in the CUDA library.
There is no CPU fallback; loading fails loudly if the library has not been built.
torch is used by callers for device memory and streams; this module only needs `data_ptr()`.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libaj_verify.so")

AJ_OK, AJ_ERR_INVALID_ARG, AJ_ERR_UNSUPPORTED, AJ_ERR_WORKSPACE, AJ_ERR_CUDA, AJ_ERR_TIMEOUT, AJ_ERR_NOT_SM100 = range(7)
AJ_BF16, AJ_F32 = 0, 1
AJ_W_VD, AJ_W_DV = 0, 1
AJ_FLAG_FORCE_SIMT, AJ_FLAG_TIME_KERNELS, AJ_FLAG_ONE_SM, AJ_FLAG_NO_EXTRA_ROW = 1, 2, 8, 16

EXPORTS = (
    "aj_create", "aj_verify", "aj_verify_host", "aj_last_status", "aj_last_gemm_ms", "aj_gemm_ms_stats", "aj_last_launch_count",
    "aj_last_gemm_path", "aj_pair_schedule", "aj_destroy", "aj_set_top_k", "aj_set_sampling", "aj_verify_tree", "aj_lr_fit", "aj_shard_exchange_bytes", "aj_shard_exchange_alloc", "aj_shard_exchange_free", "aj_shard_range", "aj_create_sharded",
    "aj_shard_project", "aj_shard_finish", "aj_ipc_export", "aj_ipc_import", "aj_ipc_close", "aj_status_string", "aj_version", "aj_verify_static",
    "aj_fuse_judge", "aj_lr_release",
)

_lib = None


class AjError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {status_string(status)} ({status})")


def lib() -> ctypes.CDLL:
    """The loaded CUDA library; raises if it has not been built (python -m paper_2504_20039_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build the CUDA library first "
                "(python __graft_entry__.py build, or python paper_2504_20039_b200/build.py)"
            )
        L = ctypes.CDLL(LIB_PATH)
        vp, ci, cf, cu = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_uint
        L.aj_create.argtypes = [ctypes.POINTER(vp), ci, ci, ci, ci, ci, ci, ci, ci, cu]
        L.aj_create.restype = ci
        L.aj_verify.argtypes = [vp, vp, vp, vp, vp, vp, cf, cf, ci, ci, ci, ci, vp, vp, vp, vp, vp, vp]
        L.aj_verify.restype = ci
        L.aj_verify_tree.argtypes = [vp, vp, vp, vp, vp, vp, vp, cf, cf, ci, ci, ci, ci, vp, vp, vp, vp, vp, vp, vp]
        L.aj_verify_tree.restype = ci
        L.aj_lr_fit.argtypes = [ci, vp, vp, ctypes.c_longlong, ci, ci, cf, ci, cf, vp, ctypes.POINTER(ctypes.c_float),
                                ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_float), vp]
        L.aj_lr_fit.restype = ci
        L.aj_verify_host.argtypes = [vp, vp, vp, vp, vp, vp, cf, cf, ci, ci, ci, ci, vp, vp, vp, vp]
        L.aj_verify_host.restype = ci
        L.aj_last_status.argtypes = [vp]
        L.aj_last_status.restype = ci
        L.aj_last_gemm_ms.argtypes = [vp, ctypes.POINTER(cf)]
        L.aj_last_gemm_ms.restype = ci
        L.aj_gemm_ms_stats.argtypes = [vp, ctypes.POINTER(cf), ctypes.POINTER(cf), ctypes.POINTER(ci)]
        L.aj_gemm_ms_stats.restype = ci
        L.aj_last_launch_count.argtypes = [vp]
        L.aj_last_launch_count.restype = ci
        L.aj_last_gemm_path.argtypes = [vp]
        L.aj_last_gemm_path.restype = ctypes.c_char_p
        L.aj_destroy.argtypes = [vp]
        L.aj_destroy.restype = ci
        L.aj_status_string.argtypes = [ci]
        L.aj_status_string.restype = ctypes.c_char_p
        L.aj_verify_static.argtypes = [vp, vp, vp, vp, vp, cf, cf, ci, ci, ci, ci, ci, ci, ci, vp, vp, vp, vp, vp, vp, vp]
        L.aj_verify_static.restype = ci
        L.aj_pair_schedule.argtypes = [ci, ci, ci, ctypes.POINTER(ctypes.c_int32)]
        L.aj_pair_schedule.restype = ci
        L.aj_shard_exchange_bytes.argtypes = [ci, ci, ci]
        L.aj_shard_exchange_bytes.restype = ctypes.c_size_t
        L.aj_shard_exchange_alloc.argtypes = [ci, ci, ci, ctypes.POINTER(vp)]
        L.aj_shard_exchange_alloc.restype = ci
        L.aj_shard_exchange_free.argtypes = [vp]
        L.aj_shard_exchange_free.restype = ci
        L.aj_shard_range.argtypes = [ci, ci, ci, ctypes.POINTER(ci), ctypes.POINTER(ci)]
        L.aj_shard_range.restype = ci
        L.aj_create_sharded.argtypes = [ctypes.POINTER(vp), ci, ci, ci, ci, ci, ci, ci, ci, cu, ci, ci, ci, ci, ctypes.POINTER(vp)]
        L.aj_create_sharded.restype = ci
        L.aj_shard_project.argtypes = [vp, vp, vp, ci, ci, vp]
        L.aj_shard_project.restype = ci
        L.aj_shard_finish.argtypes = [vp, vp, vp, vp, vp, cf, cf, ci, ci, vp, vp, vp, vp, vp, vp]
        L.aj_shard_finish.restype = ci
        L.aj_ipc_export.argtypes = [vp, ctypes.c_char_p]
        L.aj_ipc_export.restype = ci
        L.aj_ipc_import.argtypes = [ctypes.c_char_p, ctypes.POINTER(vp)]
        L.aj_ipc_import.restype = ci
        L.aj_ipc_close.argtypes = [vp]
        L.aj_ipc_close.restype = ci
        L.aj_lr_release.argtypes = [ci]
        L.aj_lr_release.restype = ci
        L.aj_fuse_judge.argtypes = [vp, vp, vp]
        L.aj_fuse_judge.restype = ci
        L.aj_set_top_k.argtypes = [vp, ci]
        L.aj_set_top_k.restype = ci
        L.aj_set_sampling.argtypes = [vp, ctypes.c_float, ctypes.c_uint64, ctypes.c_uint64]
        L.aj_set_sampling.restype = ci
        L.aj_version.argtypes = []
        L.aj_version.restype = ctypes.c_char_p
        _lib = L
    return _lib


def lr_fit(device: int, X, labels, n: int, F: int, dtype: int, C: float, w_out, max_iter: int = 500, tol: float = 1e-4,
           stream: int = 0, check: bool = True):
    """aj_lr_fit: fit the classifier on device-resident features; returns (status, b, iterations, evaluations, max |grad|);
    the kernel milliseconds of the fit are left in lr_fit.kernel_ms."""
    b = ctypes.c_float()
    it = (ctypes.c_int * 2)()
    stats = (ctypes.c_float * 2)()
    st = lib().aj_lr_fit(device, _ptr(X), _ptr(labels), n, F, dtype, float(C), max_iter, float(tol), _ptr(w_out),
                         ctypes.byref(b), it, stats, stream or None)
    if check and st != AJ_OK:
        raise AjError(st, "aj_lr_fit")
    lr_fit.kernel_ms = stats[1]
    return st, b.value, it[0], it[1], stats[0]


def lr_release(device: int = -1) -> int:
    """aj_lr_release: free the workspace aj_lr_fit keeps between fits."""
    return lib().aj_lr_release(device)


def status_string(status: int) -> str:
    return lib().aj_status_string(int(status)).decode()


def version() -> str:
    return lib().aj_version().decode()


def _ptr(t):
    """Device or host address of a torch tensor / numpy array / int / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    return t.ctypes.data


AJ_STATIC_MAX_ROWS = 32768


def pair_schedule(M: int, d: int, V: int) -> dict:
    """aj_pair_schedule: how the two-SM kernel tiles M rows against V vocabulary entries (host arithmetic)."""
    out = (ctypes.c_int32 * 10)()
    st = lib().aj_pair_schedule(M, d, V, out)
    if st != AJ_OK:
        raise AjError(st, "aj_pair_schedule")
    keys = ("n_v", "n_n", "u_base", "u_rem", "box_rows", "n_groups", "g_base", "g_rem", "dual", "stages")
    return dict(zip(keys, (int(x) for x in out)))


def verify_static(h_target, h_draft, W_lm, draft_tok, judge_w, judge_b: float, tau: float, B: int, K: int, d: int,
                  d_draft: int, V: int, dtype: int, layout: int, accept_len, next_tok, target_tok=None, top1_val=None,
                  judge_p=None, dev_status=None, stream: int = 0, check: bool = True) -> int:
    """aj_verify_static: one cycle on the current device without a handle and without any allocation.

    For callers that cannot call cudaMalloc (all memory already in their own pool, audited or frozen
    allocators): the scratch lives in a fixed array inside the library.  At most AJ_STATIC_MAX_ROWS
    rows (B*(K+1)); calls that overlap on the GPU race on that array.
    """
    st = lib().aj_verify_static(_ptr(h_target), _ptr(h_draft), _ptr(W_lm), _ptr(draft_tok), _ptr(judge_w), float(judge_b),
                                float(tau), B, K, d, d_draft, V, dtype, layout, _ptr(accept_len), _ptr(next_tok),
                                _ptr(target_tok), _ptr(top1_val), _ptr(judge_p), _ptr(dev_status), stream or None)
    if check and st != AJ_OK:
        raise AjError(st, "aj_verify_static")
    return st


def shard_exchange_bytes(max_B: int, max_K: int, world: int) -> int:
    """aj_shard_exchange_bytes: size of one GPU's exchange buffer for a vocabulary-parallel group."""
    return int(lib().aj_shard_exchange_bytes(max_B, max_K, world))


def shard_exchange_alloc(max_B: int, max_K: int, world: int) -> int:
    """aj_shard_exchange_alloc: a zero-filled exchange buffer on the current device (its device address)."""
    out = ctypes.c_void_p()
    st = lib().aj_shard_exchange_alloc(max_B, max_K, world, ctypes.byref(out))
    if st != AJ_OK:
        raise AjError(st, "aj_shard_exchange_alloc")
    return int(out.value)


def shard_exchange_free(device_ptr: int) -> None:
    st = lib().aj_shard_exchange_free(device_ptr)
    if st != AJ_OK:
        raise AjError(st, "aj_shard_exchange_free")


def shard_range(V: int, world: int, rank: int):
    """aj_shard_range: (v_begin, v_count) of rank `rank` among `world` GPUs."""
    b, n = ctypes.c_int(), ctypes.c_int()
    st = lib().aj_shard_range(V, world, rank, ctypes.byref(b), ctypes.byref(n))
    if st != AJ_OK:
        raise AjError(st, "aj_shard_range")
    return int(b.value), int(n.value)


def ipc_export(device_ptr) -> bytes:
    """aj_ipc_export: 64 opaque bytes another process of this node can import."""
    buf = ctypes.create_string_buffer(64)
    st = lib().aj_ipc_export(_ptr(device_ptr), buf)
    if st != AJ_OK:
        raise AjError(st, "aj_ipc_export")
    return buf.raw


def ipc_import(handle: bytes) -> int:
    """aj_ipc_import: the device address at which this process sees the exported memory."""
    out = ctypes.c_void_p()
    st = lib().aj_ipc_import(ctypes.create_string_buffer(bytes(handle), 64), ctypes.byref(out))
    if st != AJ_OK:
        raise AjError(st, "aj_ipc_import")
    return int(out.value)


def ipc_close(device_ptr: int) -> None:
    st = lib().aj_ipc_close(device_ptr)
    if st != AJ_OK:
        raise AjError(st, "aj_ipc_close")


class Handle:
    """aj_create / aj_destroy as an object; methods mirror the C entry points.

    With `shard=(rank, world, v_begin, v_count, exchange)` the handle is one GPU of a vocabulary-parallel
    group (aj_create_sharded); `exchange` lists every rank's exchange buffer (tensors or addresses)."""

    def __init__(self, device: int, max_B: int, max_K: int, d: int, d_draft: int, V: int,
                 dtype: int = AJ_BF16, layout: int = AJ_W_VD, flags: int = 0, shard=None):
        self._h = ctypes.c_void_p()
        if shard is None:
            st = lib().aj_create(ctypes.byref(self._h), device, max_B, max_K, d, d_draft, V, dtype, layout, flags)
        else:
            rank, world, v_begin, v_count, exchange = shard
            ptrs = (ctypes.c_void_p * len(exchange))(*[_ptr(e) for e in exchange])
            st = lib().aj_create_sharded(ctypes.byref(self._h), device, max_B, max_K, d, d_draft, V, dtype, layout, flags,
                                         rank, world, v_begin, v_count, ptrs)
        if st != AJ_OK:
            self._h = ctypes.c_void_p()
            raise AjError(st, "aj_create" if shard is None else "aj_create_sharded")
        self.d, self.V, self.d_draft = d, V, d_draft

    def shard_project(self, h_target, W_shard, B: int, K: int, stream: int = 0, check: bool = True) -> int:
        """aj_shard_project: this GPU's projection + exchange of one cycle."""
        st = lib().aj_shard_project(self._h, _ptr(h_target), _ptr(W_shard), B, K, stream or None)
        if check and st != AJ_OK:
            raise AjError(st, "aj_shard_project")
        return st

    def shard_finish(self, h_target, h_draft, draft_tok, judge_w, judge_b: float, tau: float, B: int, K: int,
                     accept_len, next_tok, target_tok=None, top1_val=None, judge_p=None, stream: int = 0,
                     check: bool = True) -> int:
        """aj_shard_finish: wait for every GPU's keys, then judge + prefix scan."""
        st = lib().aj_shard_finish(self._h, _ptr(h_target), _ptr(h_draft), _ptr(draft_tok), _ptr(judge_w), float(judge_b),
                                   float(tau), B, K, _ptr(accept_len), _ptr(next_tok), _ptr(target_tok), _ptr(top1_val),
                                   _ptr(judge_p), stream or None)
        if check and st != AJ_OK:
            raise AjError(st, "aj_shard_finish")
        return st

    def verify(self, h_target, h_draft, W_lm, draft_tok, judge_w, judge_b: float, tau: float, B: int, K: int,
               accept_len, next_tok, target_tok=None, top1_val=None, judge_p=None, stream: int = 0, check: bool = True) -> int:
        """aj_verify: device tensors in, device tensors out, asynchronous on `stream` (a cudaStream_t as int)."""
        st = lib().aj_verify(self._h, _ptr(h_target), _ptr(h_draft), _ptr(W_lm), _ptr(draft_tok), _ptr(judge_w),
                             float(judge_b), float(tau), B, K, self.d, self.V, _ptr(accept_len), _ptr(next_tok),
                             _ptr(target_tok), _ptr(top1_val), _ptr(judge_p), stream or None)
        if check and st != AJ_OK:
            raise AjError(st, "aj_verify")
        return st

    def verify_tree(self, h_target, h_draft, W_lm, draft_tok, parent, judge_w, judge_b: float, tau: float, B: int, N: int,
                    accept_len, next_tok, best_node=None, target_tok=None, top1_val=None, judge_p=None, stream: int = 0,
                    check: bool = True) -> int:
        """aj_verify_tree: the cycle for tree drafts (parent [B, N], -1 = child of the root; row n + 1 encodes node n)."""
        st = lib().aj_verify_tree(self._h, _ptr(h_target), _ptr(h_draft), _ptr(W_lm), _ptr(draft_tok), _ptr(parent), _ptr(judge_w),
                                  float(judge_b), float(tau), B, N, self.d, self.V, _ptr(accept_len), _ptr(next_tok),
                                  _ptr(best_node), _ptr(target_tok), _ptr(top1_val), _ptr(judge_p), stream or None)
        if check and st != AJ_OK:
            raise AjError(st, "aj_verify_tree")
        return st

    def verify_host(self, h_target, h_draft, W_lm, draft_tok, judge_w, judge_b: float, tau: float, B: int, K: int,
                    accept_len, next_tok, target_tok=None, stream: int = 0, check: bool = True) -> int:
        """aj_verify_host: per-cycle tensors in host memory, W_lm and judge_w on the device; synchronous."""
        st = lib().aj_verify_host(self._h, _ptr(h_target), _ptr(h_draft), _ptr(W_lm), _ptr(draft_tok), _ptr(judge_w),
                                  float(judge_b), float(tau), B, K, self.d, self.V, _ptr(accept_len), _ptr(next_tok),
                                  _ptr(target_tok), stream or None)
        if check and st != AJ_OK:
            raise AjError(st, "aj_verify_host")
        return st

    def fuse_judge(self, judge_w=None, stream: int = 0, check: bool = True) -> int:
        """aj_fuse_judge: compute the classifier's target half in the projection kernel (None: back to the judge kernel)."""
        st = lib().aj_fuse_judge(self._h, _ptr(judge_w), stream or None)
        if check and st != AJ_OK:
            raise AjError(st, "aj_fuse_judge")
        return st

    def set_top_k(self, top_k: int, check: bool = True) -> int:
        """aj_set_top_k: accept a mismatch iff the draft token is among the target's top_k (0: back to the classifier)."""
        st = lib().aj_set_top_k(self._h, int(top_k))
        if check and st != AJ_OK:
            raise AjError(st, "aj_set_top_k")
        return st

    def set_sampling(self, temperature: float, seed: int = 0, step: int = 0, check: bool = True) -> int:
        """aj_set_sampling: draw the target's tokens from softmax(logit / temperature) by the Gumbel-max trick
        (0: back to greedy); `step` is the next cycle's counter and advances by one per cycle."""
        st = lib().aj_set_sampling(self._h, float(temperature), int(seed) & (2**64 - 1), int(step) & (2**64 - 1))
        if check and st != AJ_OK:
            raise AjError(st, "aj_set_sampling")
        return st

    def last_status(self) -> int:
        return lib().aj_last_status(self._h)

    def last_gemm_ms(self) -> float:
        ms = ctypes.c_float()
        st = lib().aj_last_gemm_ms(self._h, ctypes.byref(ms))
        if st != AJ_OK:
            raise AjError(st, "aj_last_gemm_ms")
        return float(ms.value)

    def gemm_ms_stats(self):
        """(mean ms, min ms, calls) of the projection kernel since the previous read-out."""
        mean, lo, n = ctypes.c_float(), ctypes.c_float(), ctypes.c_int()
        st = lib().aj_gemm_ms_stats(self._h, ctypes.byref(mean), ctypes.byref(lo), ctypes.byref(n))
        if st != AJ_OK:
            raise AjError(st, "aj_gemm_ms_stats")
        return float(mean.value), float(lo.value), int(n.value)

    def last_launch_count(self) -> int:
        return lib().aj_last_launch_count(self._h)

    def last_gemm_path(self) -> str:
        return lib().aj_last_gemm_path(self._h).decode()

    def destroy(self) -> None:
        if self._h:
            lib().aj_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass
