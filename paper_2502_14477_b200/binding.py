"""ctypes binding of the ESA C ABI (same names as ``include/esa.h``).

Argument marshalling only: tensors are checked (device, dtype, contiguity,
shape) and passed as raw device pointers; every step of the path runs in the
library's kernels.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np
import torch

from .build import LIB_PATH

STATUS_NAMES = {
    0: "ESA_OK", 1: "ESA_ERR_INVALID_ARG", 2: "ESA_ERR_SHAPE", 3: "ESA_ERR_CAPACITY",
    4: "ESA_ERR_CUDA", 5: "ESA_ERR_TIMEOUT", 6: "ESA_ERR_UNSUPPORTED", 7: "ESA_ERR_STATE",
    8: "ESA_ERR_INDEX",
}


class EsaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__(f"{where}: {STATUS_NAMES.get(int(status), status)}")


class _CConfig(C.Structure):
    _fields_ = [
        ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("d_c", C.c_int32),
        ("l_init", C.c_int32), ("l_local", C.c_int32), ("top_k", C.c_int32), ("eps", C.c_int32),
        ("max_chunk", C.c_int32), ("max_batch", C.c_int32), ("max_tokens", C.c_int64),
        ("softmax_scale", C.c_float),
    ]


@dataclass
class EsaConfig:
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_c: int
    l_init: int
    l_local: int
    top_k: int
    eps: int
    max_chunk: int
    max_batch: int
    max_tokens: int
    softmax_scale: float = 0.0

    def to_c(self) -> _CConfig:
        return _CConfig(self.n_q_heads, self.n_kv_heads, self.head_dim, self.d_c, self.l_init, self.l_local,
                        self.top_k, self.eps, self.max_chunk, self.max_batch, self.max_tokens,
                        self.softmax_scale)


_lib = None

_PROTOS = {
    "esa_status_string": (C.c_char_p, [C.c_int]),
    "esa_workspace_bytes": (C.c_size_t, [C.POINTER(_CConfig)]),
    "esa_create": (C.c_int, [C.POINTER(_CConfig), C.POINTER(C.c_void_p)]),
    "esa_destroy": (C.c_int, [C.c_void_p]),
    "esa_set_compressors": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "esa_append_kv": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p,
                                C.c_void_p, C.c_void_p]),
    "esa_append_kv_async": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p,
                                      C.c_void_p, C.c_void_p, C.c_void_p]),
    "esa_compress_keys": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]),
    "esa_compress_keys_async": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p,
                                          C.c_void_p, C.c_void_p]),
    "esa_select": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p,
                             C.c_void_p, C.c_void_p]),
    "esa_select_async": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p,
                                   C.c_void_p, C.c_void_p, C.c_void_p]),
    "esa_select_full": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32,
                                  C.c_void_p, C.c_void_p]),
    "esa_select_full_async": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32,
                                        C.c_void_p, C.c_void_p, C.c_void_p]),
    "esa_attend": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p,
                             C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "esa_attend_async": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p,
                                   C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "esa_attend_two_position": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p,
                                          C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "esa_attend_two_position_async": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p,
                                                C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                                C.c_void_p]),
    "esa_attend_host_kv": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                     C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]),
    "esa_attend_host_kv_async": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                           C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p,
                                           C.c_void_p]),
    "esa_attend_noalloc": (C.c_int, [C.POINTER(_CConfig), C.c_int32, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p,
                                     C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "esa_fit_create": (C.c_int, [C.POINTER(_CConfig), C.c_int32, C.c_float, C.POINTER(C.c_void_p)]),
    "esa_fit_destroy": (C.c_int, [C.c_void_p]),
    "esa_fit_set_weights": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "esa_fit_get_weights": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "esa_fit_step_async": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]),
    "esa_fit_launch_count": (C.c_int64, [C.c_void_p]),
    "esa_read_pooled_scores": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_int64, C.c_void_p]),
    "esa_read_compressed_queries": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]),
    "esa_debug_wait_timeout": (C.c_int, [C.c_void_p, C.c_int64, C.c_void_p]),
    "esa_kernel_class_count": (C.c_int32, []),
    "esa_kernel_class_name": (C.c_char_p, [C.c_int32]),
    "esa_set_profiling": (C.c_int, [C.c_void_p, C.c_int32]),
    "esa_read_profile": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]),
    "esa_launch_count": (C.c_int64, [C.c_void_p]),
    "esa_last_device_status": (C.c_int, [C.c_void_p, C.c_void_p]),
}

EXPORTED_SYMBOLS = tuple(_PROTOS)


def library_path() -> str:
    return LIB_PATH


def load_library():
    """dlopen the built CUDA library.  Raises if it has not been built: there is no
    fallback implementation."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2502_14477_b200.build` "
            "(needs nvcc, targets sm_100a). The ESA path has no CPU or PyTorch fallback.")
    lib = C.CDLL(LIB_PATH)
    for name, (res, args) in _PROTOS.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    _lib = lib
    return lib


def _ptr(t: Optional[torch.Tensor]):
    return 0 if t is None else t.data_ptr()


def _check(t: torch.Tensor, name: str, dtype, shape=None):
    # kept cheap: it runs for every tensor of every call
    if not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype:
        raise TypeError(f"{name} must have dtype {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if shape is not None and t.shape != shape:
        raise ValueError(f"{name} must have shape {tuple(shape)}, got {tuple(t.shape)}")


def _stream_ptr(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


class Esa:
    """One ESA context (device workspace + compressors).  Methods mirror the C entry
    points; by default they enqueue on torch's current stream (the ``*_async`` calls),
    ``sync=True`` uses the blocking variants on the legacy default stream."""

    def __init__(self, cfg: EsaConfig):
        self.lib = load_library()
        self.cfg = cfg
        self._c = cfg.to_c()
        h = C.c_void_p()
        st = self.lib.esa_create(C.byref(self._c), C.byref(h))
        if st != 0:
            raise EsaError(st, "esa_create")
        self._h = h

    # ------------------------------------------------------------------ admin
    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            self.lib.esa_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def workspace_bytes(self) -> int:
        return int(self.lib.esa_workspace_bytes(C.byref(self._c)))

    @property
    def launch_count(self) -> int:
        return int(self.lib.esa_launch_count(self._h))

    def last_device_status(self, stream=None) -> int:
        return int(self.lib.esa_last_device_status(self._h, _stream_ptr(stream)))

    def set_compressors(self, Wq, bq, Wk, bk):
        c = self.cfg
        wq = np.ascontiguousarray(np.asarray(Wq, dtype=np.float32))
        wk = np.ascontiguousarray(np.asarray(Wk, dtype=np.float32))
        if wq.shape != (c.d_c, c.n_q_heads * c.head_dim) or wk.shape != (c.d_c, c.n_kv_heads * c.head_dim):
            raise ValueError("compressor weights must be [d_c, H*d] and [d_c, H_G*d]")
        b_q = None if bq is None else np.ascontiguousarray(np.asarray(bq, dtype=np.float32))
        b_k = None if bk is None else np.ascontiguousarray(np.asarray(bk, dtype=np.float32))
        for b in (b_q, b_k):
            if b is not None and b.shape != (c.d_c,):
                raise ValueError("bias must be [d_c]")
        st = self.lib.esa_set_compressors(
            self._h, wq.ctypes.data_as(C.c_void_p), None if b_q is None else b_q.ctypes.data_as(C.c_void_p),
            wk.ctypes.data_as(C.c_void_p), None if b_k is None else b_k.ctypes.data_as(C.c_void_p))
        if st != 0:
            raise EsaError(st, "esa_set_compressors")

    @staticmethod
    def _nprev(n_prev: Sequence[int], B: int):
        """Host int64[B] for the C call (a ctypes array: cheaper to build than a numpy one)."""
        if len(n_prev) != B:
            raise ValueError("n_prev must have one entry per sequence")
        return (C.c_int64 * B)(*[int(x) for x in n_prev])

    # ------------------------------------------------------------ entry points
    def append_kv(self, K_new, V_new, K_cache, V_cache, n_prev, stream=None, sync=False):
        c = self.cfg
        B, n_new = K_new.shape[0], K_new.shape[1]
        _check(K_new, "K_new", torch.bfloat16, (B, n_new, c.n_kv_heads, c.head_dim))
        _check(V_new, "V_new", torch.bfloat16, (B, n_new, c.n_kv_heads, c.head_dim))
        _check(K_cache, "K_cache", torch.bfloat16, (B, c.max_tokens, c.n_kv_heads, c.head_dim))
        _check(V_cache, "V_cache", torch.bfloat16, (B, c.max_tokens, c.n_kv_heads, c.head_dim))
        npv = self._nprev(n_prev, B)
        if sync:
            st = self.lib.esa_append_kv(self._h, B, _ptr(K_new), _ptr(V_new), n_new, _ptr(K_cache),
                                        _ptr(V_cache), npv)
        else:
            st = self.lib.esa_append_kv_async(self._h, B, _ptr(K_new), _ptr(V_new), n_new, _ptr(K_cache),
                                              _ptr(V_cache), npv,
                                              _stream_ptr(stream))
        if st != 0:
            raise EsaError(st, "esa_append_kv")

    def compress_keys(self, K_new, kc_cache, n_prev, stream=None, sync=False):
        c = self.cfg
        B, n_new = K_new.shape[0], K_new.shape[1]
        _check(K_new, "K_new", torch.bfloat16, (B, n_new, c.n_kv_heads, c.head_dim))
        _check(kc_cache, "kc_cache", torch.bfloat16, (B, c.max_tokens, c.d_c))
        npv = self._nprev(n_prev, B)
        if sync:
            st = self.lib.esa_compress_keys(self._h, B, _ptr(K_new), n_new, _ptr(kc_cache),
                                            npv)
        else:
            st = self.lib.esa_compress_keys_async(self._h, B, _ptr(K_new), n_new, _ptr(kc_cache),
                                                  npv, _stream_ptr(stream))
        if st != 0:
            raise EsaError(st, "esa_compress_keys")

    def select(self, Q_cur, kc_cache, n_prev, idx_out, n_sel_out, stream=None, sync=False):
        c = self.cfg
        B, l_C = Q_cur.shape[0], Q_cur.shape[1]
        _check(Q_cur, "Q_cur", torch.bfloat16, (B, l_C, c.n_q_heads, c.head_dim))
        _check(kc_cache, "kc_cache", torch.bfloat16, (B, c.max_tokens, c.d_c))
        _check(idx_out, "idx_out", torch.int32, (B, c.top_k))
        _check(n_sel_out, "n_sel_out", torch.int32, (B,))
        npv = self._nprev(n_prev, B)
        if sync:
            st = self.lib.esa_select(self._h, B, _ptr(Q_cur), l_C, _ptr(kc_cache),
                                     npv, _ptr(idx_out), _ptr(n_sel_out))
        else:
            st = self.lib.esa_select_async(self._h, B, _ptr(Q_cur), l_C, _ptr(kc_cache),
                                           npv, _ptr(idx_out), _ptr(n_sel_out),
                                           _stream_ptr(stream))
        if st != 0:
            raise EsaError(st, "esa_select")

    def select_full(self, Q_cur, K_cache, n_prev, idx_out, n_sel_out, per_head=False, stream=None, sync=False):
        """``esa_select_full``: selection on full-dimension scores (Eq. 3) or the per-head vote."""
        c = self.cfg
        B, l_C = Q_cur.shape[0], Q_cur.shape[1]
        _check(Q_cur, "Q_cur", torch.bfloat16, (B, l_C, c.n_q_heads, c.head_dim))
        _check(K_cache, "K_cache", torch.bfloat16, (B, c.max_tokens, c.n_kv_heads, c.head_dim))
        _check(idx_out, "idx_out", torch.int32, (B, c.top_k))
        _check(n_sel_out, "n_sel_out", torch.int32, (B,))
        npv = self._nprev(n_prev, B)
        mode = 1 if per_head else 0
        if sync:
            st = self.lib.esa_select_full(self._h, B, _ptr(Q_cur), l_C, _ptr(K_cache), npv, mode, _ptr(idx_out),
                                          _ptr(n_sel_out))
        else:
            st = self.lib.esa_select_full_async(self._h, B, _ptr(Q_cur), l_C, _ptr(K_cache), npv, mode, _ptr(idx_out),
                                                _ptr(n_sel_out), _stream_ptr(stream))
        if st != 0:
            raise EsaError(st, "esa_select_full")

    def attend(self, Q_cur, K_cache, V_cache, n_prev, idx, n_sel, O, stream=None, sync=False):
        c = self.cfg
        B, l_C = Q_cur.shape[0], Q_cur.shape[1]
        _check(Q_cur, "Q_cur", torch.bfloat16, (B, l_C, c.n_q_heads, c.head_dim))
        _check(K_cache, "K_cache", torch.bfloat16, (B, c.max_tokens, c.n_kv_heads, c.head_dim))
        _check(V_cache, "V_cache", torch.bfloat16, (B, c.max_tokens, c.n_kv_heads, c.head_dim))
        _check(idx, "idx", torch.int32, (B, c.top_k))
        _check(n_sel, "n_sel", torch.int32, (B,))
        _check(O, "O", torch.bfloat16, (B, l_C, c.n_q_heads, c.head_dim))
        npv = self._nprev(n_prev, B)
        if sync:
            st = self.lib.esa_attend(self._h, B, _ptr(Q_cur), l_C, _ptr(K_cache), _ptr(V_cache),
                                     npv, _ptr(idx), _ptr(n_sel), _ptr(O))
        else:
            st = self.lib.esa_attend_async(self._h, B, _ptr(Q_cur), l_C, _ptr(K_cache), _ptr(V_cache),
                                           npv, _ptr(idx), _ptr(n_sel), _ptr(O),
                                           _stream_ptr(stream))
        if st != 0:
            raise EsaError(st, "esa_attend")

    def attend_two_position(self, Q_cur, Q_far, K_cache, K_far_cache, V_cache, n_prev, idx, n_sel, O, stream=None,
                            sync=False):
        """``esa_attend_two_position``: Q_far / K_far_cache (either may be None) are read for I and M_k."""
        c = self.cfg
        B, l_C = Q_cur.shape[0], Q_cur.shape[1]
        _check(Q_cur, "Q_cur", torch.bfloat16, (B, l_C, c.n_q_heads, c.head_dim))
        if Q_far is not None:
            _check(Q_far, "Q_far", torch.bfloat16, (B, l_C, c.n_q_heads, c.head_dim))
        _check(K_cache, "K_cache", torch.bfloat16, (B, c.max_tokens, c.n_kv_heads, c.head_dim))
        if K_far_cache is not None:
            _check(K_far_cache, "K_far_cache", torch.bfloat16, (B, c.max_tokens, c.n_kv_heads, c.head_dim))
        _check(V_cache, "V_cache", torch.bfloat16, (B, c.max_tokens, c.n_kv_heads, c.head_dim))
        _check(idx, "idx", torch.int32, (B, c.top_k))
        _check(n_sel, "n_sel", torch.int32, (B,))
        _check(O, "O", torch.bfloat16, (B, l_C, c.n_q_heads, c.head_dim))
        npv = self._nprev(n_prev, B)
        if sync:
            st = self.lib.esa_attend_two_position(self._h, B, _ptr(Q_cur), _ptr(Q_far), l_C, _ptr(K_cache),
                                                  _ptr(K_far_cache), _ptr(V_cache), npv, _ptr(idx), _ptr(n_sel), _ptr(O))
        else:
            st = self.lib.esa_attend_two_position_async(self._h, B, _ptr(Q_cur), _ptr(Q_far), l_C, _ptr(K_cache),
                                                        _ptr(K_far_cache), _ptr(V_cache), npv, _ptr(idx), _ptr(n_sel),
                                                        _ptr(O), _stream_ptr(stream))
        if st != 0:
            raise EsaError(st, "esa_attend_two_position")

    def attend_host_kv(self, Q_cur, K_host, V_host, n_prev, idx, n_sel, K_stage, V_stage, O, stream=None, sync=False):
        """``esa_attend_host_kv``: K_host / V_host are pinned host tensors [B, max_tokens, H_G, d]; K_stage / V_stage
        device scratch [B, stage_rows, H_G, d]."""
        c = self.cfg
        B, l_C = Q_cur.shape[0], Q_cur.shape[1]
        _check(Q_cur, "Q_cur", torch.bfloat16, (B, l_C, c.n_q_heads, c.head_dim))
        for t, name in ((K_host, "K_host"), (V_host, "V_host")):
            if t.is_cuda or not t.is_pinned():
                raise TypeError(f"{name} must be a pinned host tensor")
            if t.dtype != torch.bfloat16 or not t.is_contiguous() or t.shape != (B, c.max_tokens, c.n_kv_heads, c.head_dim):
                raise ValueError(f"{name} must be contiguous bf16 [B, max_tokens, H_G, d]")
        stage_rows = K_stage.shape[1]
        _check(K_stage, "K_stage", torch.bfloat16, (B, stage_rows, c.n_kv_heads, c.head_dim))
        _check(V_stage, "V_stage", torch.bfloat16, (B, stage_rows, c.n_kv_heads, c.head_dim))
        _check(idx, "idx", torch.int32, (B, c.top_k))
        _check(n_sel, "n_sel", torch.int32, (B,))
        _check(O, "O", torch.bfloat16, (B, l_C, c.n_q_heads, c.head_dim))
        npv = self._nprev(n_prev, B)
        if sync:
            st = self.lib.esa_attend_host_kv(self._h, B, _ptr(Q_cur), l_C, K_host.data_ptr(), V_host.data_ptr(), npv, _ptr(idx),
                                             _ptr(n_sel), _ptr(K_stage), _ptr(V_stage), stage_rows, _ptr(O))
        else:
            st = self.lib.esa_attend_host_kv_async(self._h, B, _ptr(Q_cur), l_C, K_host.data_ptr(), V_host.data_ptr(), npv,
                                                   _ptr(idx), _ptr(n_sel), _ptr(K_stage), _ptr(V_stage), stage_rows, _ptr(O),
                                                   _stream_ptr(stream))
        if st != 0:
            raise EsaError(st, "esa_attend_host_kv")

    def read_pooled_scores(self, b: int, n: int, stream=None) -> np.ndarray:
        out = np.empty(n, dtype=np.float32)
        st = self.lib.esa_read_pooled_scores(self._h, b, out.ctypes.data_as(C.c_void_p), n, _stream_ptr(stream))
        if st != 0:
            raise EsaError(st, "esa_read_pooled_scores")
        return out


    def read_compressed_queries(self, n_rows: int, stream=None) -> np.ndarray:
        """q' of the last scoring selection as bf16 bit patterns, uint16 [n_rows, d_c]."""
        out = np.empty((n_rows, self.cfg.d_c), dtype=np.uint16)
        st = self.lib.esa_read_compressed_queries(self._h, out.ctypes.data_as(C.c_void_p), n_rows, _stream_ptr(stream))
        if st != 0:
            raise EsaError(st, "esa_read_compressed_queries")
        return out

    def set_profiling(self, on: bool):
        st = self.lib.esa_set_profiling(self._h, 1 if on else 0)
        if st != 0:
            raise EsaError(st, "esa_set_profiling")

    def read_profile(self) -> dict:
        """{kernel class name: (launches, total ms)} of the launches profiled since the last read."""
        n = int(self.lib.esa_kernel_class_count())
        cnt = (C.c_int64 * n)()
        ms = (C.c_double * n)()
        st = self.lib.esa_read_profile(self._h, n, cnt, ms)
        if st != 0:
            raise EsaError(st, "esa_read_profile")
        return {self.lib.esa_kernel_class_name(i).decode(): (int(cnt[i]), float(ms[i])) for i in range(n) if cnt[i]}

    def debug_wait_timeout(self, limit_cycles: int, stream=None):
        st = self.lib.esa_debug_wait_timeout(self._h, int(limit_cycles), _stream_ptr(stream))
        if st != 0:
            raise EsaError(st, "esa_debug_wait_timeout")


class EsaFit:
    """Trainer of the two compressors (Eq. 7): ``esa_fit_*``.  Marshalling only."""

    def __init__(self, cfg: EsaConfig, batch: int, lr: float = 5e-4):
        self.lib = load_library()
        self.cfg, self.batch = cfg, batch
        self._c = cfg.to_c()
        h = C.c_void_p()
        st = self.lib.esa_fit_create(C.byref(self._c), batch, lr, C.byref(h))
        if st != 0:
            raise EsaError(st, "esa_fit_create")
        self._h = h

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            self.lib.esa_fit_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def launch_count(self) -> int:
        return int(self.lib.esa_fit_launch_count(self._h))

    def set_weights(self, Wq, bq, Wk, bk):
        arr = [None if a is None else np.ascontiguousarray(np.asarray(a, dtype=np.float32)) for a in (Wq, bq, Wk, bk)]
        st = self.lib.esa_fit_set_weights(self._h, *[None if a is None else a.ctypes.data_as(C.c_void_p) for a in arr])
        if st != 0:
            raise EsaError(st, "esa_fit_set_weights")

    def get_weights(self):
        c = self.cfg
        out = (np.empty((c.d_c, c.n_q_heads * c.head_dim), np.float32), np.empty(c.d_c, np.float32),
               np.empty((c.d_c, c.n_kv_heads * c.head_dim), np.float32), np.empty(c.d_c, np.float32))
        st = self.lib.esa_fit_get_weights(self._h, *[a.ctypes.data_as(C.c_void_p) for a in out])
        if st != 0:
            raise EsaError(st, "esa_fit_get_weights")
        return out

    def step(self, Q_batch, K_batch, loss_out=None, stream=None):
        c = self.cfg
        n = Q_batch.shape[0]
        _check(Q_batch, "Q_batch", torch.bfloat16, (n, c.n_q_heads, c.head_dim))
        _check(K_batch, "K_batch", torch.bfloat16, (n, c.n_kv_heads, c.head_dim))
        if loss_out is not None:
            _check(loss_out, "loss_out", torch.float32, (1,))
        st = self.lib.esa_fit_step_async(self._h, _ptr(Q_batch), _ptr(K_batch), n, _ptr(loss_out), _stream_ptr(stream))
        if st != 0:
            raise EsaError(st, "esa_fit_step_async")


def attend_noalloc(cfg: EsaConfig, Q_cur, K_cache, V_cache, n_prev, idx, n_sel, O, stream=None):
    """``esa_attend_noalloc``: attention of a small chunk (decode) without a context and without
    any device allocation -- the split partials live in a fixed array inside the library.  For
    callers that must not allocate once running (see ``include/esa.h``).  Calls on one device
    share that array and must be ordered with respect to each other."""
    lib = load_library()
    B, l_C = Q_cur.shape[0], Q_cur.shape[1]
    _check(Q_cur, "Q_cur", torch.bfloat16, (B, l_C, cfg.n_q_heads, cfg.head_dim))
    _check(K_cache, "K_cache", torch.bfloat16, (B, cfg.max_tokens, cfg.n_kv_heads, cfg.head_dim))
    _check(V_cache, "V_cache", torch.bfloat16, (B, cfg.max_tokens, cfg.n_kv_heads, cfg.head_dim))
    _check(idx, "idx", torch.int32, (B, cfg.top_k))
    _check(n_sel, "n_sel", torch.int32, (B,))
    _check(O, "O", torch.bfloat16, (B, l_C, cfg.n_q_heads, cfg.head_dim))
    npv = Esa._nprev(n_prev, B)
    c = cfg.to_c()
    st = lib.esa_attend_noalloc(C.byref(c), B, _ptr(Q_cur), l_C, _ptr(K_cache), _ptr(V_cache),
                                npv, _ptr(idx), _ptr(n_sel), _ptr(O), _stream_ptr(stream))
    if st != 0:
        raise EsaError(st, "esa_attend_noalloc")
