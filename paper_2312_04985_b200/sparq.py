"""Thin ctypes binding over the C ABI of ``include/sparq.h``.

Argument marshalling only: every step of the path runs in the CUDA kernels of
``libsparq_b200.so``.  PyTorch supplies device memory (``tensor.data_ptr()``) and the current
stream.  There is no CPU fallback: a missing library or a missing GPU raises.

Function names, argument order and semantics are those of the header; tensors replace the
pointer arguments and shapes are read from them.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from . import build as _build

OK = 0
ERR_NULL_POINTER, ERR_BAD_SHAPE, ERR_BAD_RK, ERR_WORKSPACE, ERR_TOO_LONG, ERR_CUDA, ERR_STATIC_SCRATCH = 1, 2, 3, 4, 5, 6, 7
ERR_ALIGNMENT = 8
ERR_BAD_OPTION = 9
TAU_L1, TAU_SQRT_D, TAU_SQRT_R = 0, 1, 2
STATIC_SCRATCH_BYTES = 8 << 20
DEV_BAD_SEQ_LEN, DEV_CACHE_FULL, DEV_TIMEOUT = 16, 17, 18
K_MAX = 1024
HEAD_DIM = 128

EXPORTS = ("sparq_status_string", "sparq_max_seq_len", "sparq_cache_build", "sparq_cache_append", "sparq_decode",
           "sparq_workspace_bytes", "dense_decode", "dense_workspace_bytes", "dense_decode_static", "sparq_step_host",
           "sparq_step_host_staging_bytes", "sparq_decode_grouped", "sparq_grouped_workspace_bytes",
           "sparq_decode_1xk", "sparq_1xk_workspace_bytes", "sparq_decode_opt", "sparq_decode_grouped_opt")


class SparqError(RuntimeError):
    def __init__(self, fn: str, code: int):
        self.code = code
        super().__init__("%s failed: %s (%d)" % (fn, status_string(code), code))


_lib = None


def lib() -> ctypes.CDLL:
    """Load ``libsparq_b200.so`` (built in-tree by ``build.build()``); raise if it is missing."""
    global _lib
    if _lib is None:
        path = _build.LIB_PATH
        if not os.path.exists(path):
            raise ImportError("CUDA library %s not built: run `python -m paper_2312_04985_b200.build` "
                              "or __graft_entry__.build()" % path)
        L = ctypes.CDLL(path)
        vp, i, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
        L.sparq_status_string.restype = ctypes.c_char_p
        L.sparq_status_string.argtypes = [i]
        L.sparq_max_seq_len.restype = i
        L.sparq_max_seq_len.argtypes = []
        L.sparq_cache_build.restype = i
        L.sparq_cache_build.argtypes = [vp] * 6 + [i] * 4 + [vp, vp]
        L.sparq_cache_append.restype = i
        L.sparq_cache_append.argtypes = [vp] * 8 + [i] * 4 + [vp, vp]
        L.sparq_decode.restype = i
        L.sparq_decode.argtypes = [vp] * 6 + [i] * 7 + [vp] * 4 + [vp, sz, vp, vp]
        L.sparq_decode_opt.restype = i
        L.sparq_decode_opt.argtypes = [vp] * 6 + [i] * 10 + [vp] * 4 + [vp, sz, vp, vp]
        L.sparq_workspace_bytes.restype = sz
        L.sparq_workspace_bytes.argtypes = [i] * 7
        L.dense_decode.restype = i
        L.dense_decode.argtypes = [vp] * 4 + [i] * 5 + [vp, vp, sz, vp, vp]
        L.dense_workspace_bytes.restype = sz
        L.dense_workspace_bytes.argtypes = [i] * 5
        L.dense_decode_static.restype = i
        L.dense_decode_static.argtypes = [vp] * 4 + [i] * 5 + [vp, vp, vp]
        L.sparq_step_host.restype = i
        L.sparq_step_host.argtypes = [vp] * 9 + [i] * 7 + [vp, vp, sz, vp, vp]
        L.sparq_step_host_staging_bytes.restype = sz
        L.sparq_step_host_staging_bytes.argtypes = [i] * 7
        L.sparq_decode_grouped.restype = i
        L.sparq_decode_grouped.argtypes = [vp] * 6 + [i] * 8 + [vp] * 4 + [vp, sz, vp, vp]
        L.sparq_decode_grouped_opt.restype = i
        L.sparq_decode_grouped_opt.argtypes = [vp] * 6 + [i] * 10 + [vp] * 4 + [vp, sz, vp, vp]
        L.sparq_grouped_workspace_bytes.restype = sz
        L.sparq_grouped_workspace_bytes.argtypes = [i] * 5
        L.sparq_decode_1xk.restype = i
        L.sparq_decode_1xk.argtypes = [vp] * 5 + [i] * 7 + [vp] * 4 + [vp, sz, vp, vp]
        L.sparq_1xk_workspace_bytes.restype = sz
        L.sparq_1xk_workspace_bytes.argtypes = [i] * 5
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().sparq_status_string(int(code)).decode()


def _dev(t: Optional[torch.Tensor], dtype, name: str):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("%s must be a CUDA tensor (there is no CPU path)" % name)
    if t.dtype != dtype or not t.is_contiguous():
        raise ValueError("%s must be a contiguous %s tensor" % (name, dtype))
    return t.data_ptr()


def _stream(ref: torch.Tensor) -> int:
    return torch.cuda.current_stream(ref.device).cuda_stream


def _check(fn: str, rc: int):
    if rc != OK:
        raise SparqError(fn, rc)


def sparq_max_seq_len() -> int:
    return int(lib().sparq_max_seq_len())


def sparq_workspace_bytes(B, Hq, Hkv, d, S_max, r, k) -> int:
    return int(lib().sparq_workspace_bytes(B, Hq, Hkv, d, S_max, r, k))


def dense_workspace_bytes(B, Hq, Hkv, d, S_max) -> int:
    return int(lib().dense_workspace_bytes(B, Hq, Hkv, d, S_max))


def sparq_step_host_staging_bytes(B, Hq, Hkv, d, S_max, r, k) -> int:
    return int(lib().sparq_step_host_staging_bytes(B, Hq, Hkv, d, S_max, r, k))


def sparq_cache_build(K, V, seq_lens, Kt, vsum, vbar, status=None):
    B, Hkv, S_max, d = K.shape
    with torch.cuda.device(K.device):
        rc = lib().sparq_cache_build(_dev(K, torch.float16, "K"), _dev(V, torch.float16, "V"),
                                     _dev(seq_lens, torch.int32, "seq_lens"), _dev(Kt, torch.float16, "Kt"),
                                     _dev(vsum, torch.float32, "vsum"), _dev(vbar, torch.float16, "vbar"),
                                     B, Hkv, d, S_max, _dev(status, torch.int32, "status"), _stream(K))
    _check("sparq_cache_build", rc)


def sparq_cache_append(k_new, v_new, K, Kt, V, vsum, vbar, seq_lens, status=None):
    B, Hkv, S_max, d = K.shape
    with torch.cuda.device(K.device):
        rc = lib().sparq_cache_append(_dev(k_new, torch.float16, "k_new"), _dev(v_new, torch.float16, "v_new"),
                                      _dev(K, torch.float16, "K"), _dev(Kt, torch.float16, "Kt"),
                                      _dev(V, torch.float16, "V"), _dev(vsum, torch.float32, "vsum"),
                                      _dev(vbar, torch.float16, "vbar"), _dev(seq_lens, torch.int32, "seq_lens"),
                                      B, Hkv, d, S_max, _dev(status, torch.int32, "status"), _stream(K))
    _check("sparq_cache_append", rc)


def sparq_decode(q, K, Kt, V, vbar, seq_lens, r, k, out, idx_r=None, idx_k=None, alpha=None, workspace=None,
                 status=None):
    B, Hq, d = q.shape
    Hkv, S_max = K.shape[1], K.shape[2]
    with torch.cuda.device(q.device):
        rc = lib().sparq_decode(_dev(q, torch.float16, "q"), _dev(K, torch.float16, "K"),
                                _dev(Kt, torch.float16, "Kt"), _dev(V, torch.float16, "V"),
                                _dev(vbar, torch.float16, "vbar"), _dev(seq_lens, torch.int32, "seq_lens"),
                                B, Hq, Hkv, d, S_max, int(r), int(k), _dev(out, torch.float16, "out"),
                                _dev(idx_r, torch.int32, "idx_r"), _dev(idx_k, torch.int32, "idx_k"),
                                _dev(alpha, torch.float32, "alpha"),
                                None if workspace is None else workspace.data_ptr(),
                                0 if workspace is None else workspace.numel() * workspace.element_size(),
                                _dev(status, torch.int32, "status"), _stream(q))
    _check("sparq_decode", rc)
    return out


def sparq_decode_opt(q, K, Kt, V, vbar, seq_lens, r, k, out, tau_mode=TAU_L1, realloc=True, window=0, idx_r=None,
                     idx_k=None, alpha=None, workspace=None, status=None):
    B, Hq, d = q.shape
    Hkv, S_max = K.shape[1], K.shape[2]
    with torch.cuda.device(q.device):
        rc = lib().sparq_decode_opt(_dev(q, torch.float16, "q"), _dev(K, torch.float16, "K"),
                                    _dev(Kt, torch.float16, "Kt"), _dev(V, torch.float16, "V"),
                                    _dev(vbar, torch.float16, "vbar"), _dev(seq_lens, torch.int32, "seq_lens"),
                                    B, Hq, Hkv, d, S_max, int(r), int(k), int(tau_mode), 1 if realloc else 0, int(window),
                                    _dev(out, torch.float16, "out"), _dev(idx_r, torch.int32, "idx_r"),
                                    _dev(idx_k, torch.int32, "idx_k"), _dev(alpha, torch.float32, "alpha"),
                                    None if workspace is None else workspace.data_ptr(),
                                    0 if workspace is None else workspace.numel() * workspace.element_size(),
                                    _dev(status, torch.int32, "status"), _stream(q))
    _check("sparq_decode_opt", rc)
    return out


def sparq_grouped_workspace_bytes(B, Hq, Hkv, d, S_max) -> int:
    return int(lib().sparq_grouped_workspace_bytes(B, Hq, Hkv, d, S_max))


def sparq_decode_grouped(q, K, Kt, V, vbar, seq_lens, r, k, out, workspace, realloc=True, idx_r=None, idx_k=None,
                         alpha=None, status=None):
    B, Hq, d = q.shape
    Hkv, S_max = K.shape[1], K.shape[2]
    with torch.cuda.device(q.device):
        rc = lib().sparq_decode_grouped(_dev(q, torch.float16, "q"), _dev(K, torch.float16, "K"),
                                        _dev(Kt, torch.float16, "Kt"), _dev(V, torch.float16, "V"),
                                        _dev(vbar, torch.float16, "vbar"), _dev(seq_lens, torch.int32, "seq_lens"),
                                        B, Hq, Hkv, d, S_max, int(r), int(k), 1 if realloc else 0,
                                        _dev(out, torch.float16, "out"), _dev(idx_r, torch.int32, "idx_r"),
                                        _dev(idx_k, torch.int32, "idx_k"), _dev(alpha, torch.float32, "alpha"),
                                        None if workspace is None else workspace.data_ptr(),
                                        0 if workspace is None else workspace.numel() * workspace.element_size(),
                                        _dev(status, torch.int32, "status"), _stream(q))
    _check("sparq_decode_grouped", rc)
    return out


def sparq_decode_grouped_opt(q, K, Kt, V, vbar, seq_lens, r, k, out, workspace, tau_mode=TAU_L1, realloc=True, window=0,
                             idx_r=None, idx_k=None, alpha=None, status=None):
    B, Hq, d = q.shape
    Hkv, S_max = K.shape[1], K.shape[2]
    with torch.cuda.device(q.device):
        rc = lib().sparq_decode_grouped_opt(_dev(q, torch.float16, "q"), _dev(K, torch.float16, "K"),
                                            _dev(Kt, torch.float16, "Kt"), _dev(V, torch.float16, "V"),
                                            _dev(vbar, torch.float16, "vbar"), _dev(seq_lens, torch.int32, "seq_lens"),
                                            B, Hq, Hkv, d, S_max, int(r), int(k), int(tau_mode), 1 if realloc else 0,
                                            int(window), _dev(out, torch.float16, "out"), _dev(idx_r, torch.int32, "idx_r"),
                                            _dev(idx_k, torch.int32, "idx_k"), _dev(alpha, torch.float32, "alpha"),
                                            None if workspace is None else workspace.data_ptr(),
                                            0 if workspace is None else workspace.numel() * workspace.element_size(),
                                            _dev(status, torch.int32, "status"), _stream(q))
    _check("sparq_decode_grouped_opt", rc)
    return out


def sparq_1xk_workspace_bytes(B, Hq, Hkv, d, S_max) -> int:
    return int(lib().sparq_1xk_workspace_bytes(B, Hq, Hkv, d, S_max))


def sparq_decode_1xk(q, K, V, vbar, seq_lens, r, k, out, workspace, idx_r=None, idx_k=None, alpha=None, status=None):
    B, Hq, d = q.shape
    Hkv, S_max = K.shape[1], K.shape[2]
    with torch.cuda.device(q.device):
        rc = lib().sparq_decode_1xk(_dev(q, torch.float16, "q"), _dev(K, torch.float16, "K"), _dev(V, torch.float16, "V"),
                                    _dev(vbar, torch.float16, "vbar"), _dev(seq_lens, torch.int32, "seq_lens"),
                                    B, Hq, Hkv, d, S_max, int(r), int(k), _dev(out, torch.float16, "out"),
                                    _dev(idx_r, torch.int32, "idx_r"), _dev(idx_k, torch.int32, "idx_k"),
                                    _dev(alpha, torch.float32, "alpha"),
                                    None if workspace is None else workspace.data_ptr(),
                                    0 if workspace is None else workspace.numel() * workspace.element_size(),
                                    _dev(status, torch.int32, "status"), _stream(q))
    _check("sparq_decode_1xk", rc)
    return out


def dense_decode(q, K, V, seq_lens, out, workspace=None, status=None):
    B, Hq, d = q.shape
    Hkv, S_max = K.shape[1], K.shape[2]
    with torch.cuda.device(q.device):
        rc = lib().dense_decode(_dev(q, torch.float16, "q"), _dev(K, torch.float16, "K"),
                                _dev(V, torch.float16, "V"), _dev(seq_lens, torch.int32, "seq_lens"),
                                B, Hq, Hkv, d, S_max, _dev(out, torch.float16, "out"),
                                None if workspace is None else workspace.data_ptr(),
                                0 if workspace is None else workspace.numel() * workspace.element_size(),
                                _dev(status, torch.int32, "status"), _stream(q))
    _check("dense_decode", rc)
    return out


def dense_decode_static(q, K, V, seq_lens, out, status=None):
    """dense_decode on the library's built-in scratch: no workspace argument, nothing allocated by the
    call.  Raises SparqError(ERR_STATIC_SCRATCH) when the problem needs more than STATIC_SCRATCH_BYTES.
    Calls on one device share that scratch: keep them ordered on one stream."""
    B, Hq, d = q.shape
    Hkv, S_max = K.shape[1], K.shape[2]
    with torch.cuda.device(q.device):
        rc = lib().dense_decode_static(_dev(q, torch.float16, "q"), _dev(K, torch.float16, "K"),
                                       _dev(V, torch.float16, "V"), _dev(seq_lens, torch.int32, "seq_lens"),
                                       B, Hq, Hkv, d, S_max, _dev(out, torch.float16, "out"),
                                       _dev(status, torch.int32, "status"), _stream(q))
    _check("dense_decode_static", rc)
    return out


def sparq_step_host(q_host, k_new_host, v_new_host, K, Kt, V, vsum, vbar, seq_lens, r, k, out_host, staging,
                    status=None):
    """Host-buffer step: q_host, k_new_host, v_new_host, out_host are CPU (pinned) fp16 tensors.
    With k_new_host = v_new_host = None, q_host is a flat buffer holding q [B,Hq,d], k_new and
    v_new [B,Hkv,d] back to back (one copy to the device instead of three)."""
    Hkv, S_max, d = K.shape[1], K.shape[2], K.shape[3]
    B = out_host.shape[0]
    Hq = out_host.shape[1]
    packed = k_new_host is None and v_new_host is None
    if packed and q_host.numel() != B * (Hq + 2 * Hkv) * d:
        raise ValueError("packed q_host must hold B*(Hq + 2*Hkv)*d elements")
    for t, name in ((q_host, "q_host"), (k_new_host, "k_new_host"), (v_new_host, "v_new_host"),
                    (out_host, "out_host")):
        if t is None and packed:
            continue
        if t is None or t.is_cuda or t.dtype != torch.float16 or not t.is_contiguous():
            raise ValueError("%s must be a contiguous CPU float16 tensor" % name)
    with torch.cuda.device(K.device):
        rc = lib().sparq_step_host(q_host.data_ptr(), None if packed else k_new_host.data_ptr(),
                                   None if packed else v_new_host.data_ptr(),
                                   _dev(K, torch.float16, "K"), _dev(Kt, torch.float16, "Kt"),
                                   _dev(V, torch.float16, "V"), _dev(vsum, torch.float32, "vsum"),
                                   _dev(vbar, torch.float16, "vbar"), _dev(seq_lens, torch.int32, "seq_lens"),
                                   B, Hq, Hkv, d, S_max, int(r), int(k), out_host.data_ptr(), staging.data_ptr(),
                                   staging.numel() * staging.element_size(), _dev(status, torch.int32, "status"),
                                   _stream(K))
    _check("sparq_step_host", rc)
    return out_host
