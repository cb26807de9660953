"""ctypes binding of the batch-invariant linear layer and RMS normalisation
(``include/vosti_linear.h``): argument marshalling only."""
from __future__ import annotations

import ctypes

import torch

import os

from . import binding as _vb

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libvosti_linear.so")
if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2609_38981_b200.build` "
        "(the linear layer has no fallback)")
_lib = ctypes.CDLL(LIB_PATH)
_vp = ctypes.c_void_p

EXPORTS = ("vosti_linear_tile_shape", "vosti_linear_segments", "vosti_linear_workspace_bytes", "vosti_linear",
           "vosti_linear_ex", "vosti_rmsnorm", "vosti_linear_poll_status", "vosti_linear_fingerprint", "vosti_linear_contract")

_lib.vosti_linear_tile_shape.restype = ctypes.c_int
_lib.vosti_linear_tile_shape.argtypes = [ctypes.c_int64, ctypes.c_int64] + [ctypes.POINTER(ctypes.c_int32)] * 3
_lib.vosti_linear.restype = ctypes.c_int
_lib.vosti_linear.argtypes = [_vp, _vp, _vp, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, _vp, ctypes.c_size_t, _vp]
_lib.vosti_linear_ex.restype = ctypes.c_int
_lib.vosti_linear_ex.argtypes = [_vp, _vp, _vp, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, _vp, ctypes.c_size_t,
                                 ctypes.c_int32, _vp]
_lib.vosti_linear_segments.restype = ctypes.c_int
_lib.vosti_linear_segments.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.POINTER(ctypes.c_int32)]
_lib.vosti_linear_workspace_bytes.restype = ctypes.c_size_t
_lib.vosti_linear_workspace_bytes.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_int64]
_lib.vosti_rmsnorm.restype = ctypes.c_int
_lib.vosti_rmsnorm.argtypes = [_vp, _vp, _vp, ctypes.c_int64, ctypes.c_int64, ctypes.c_float, _vp]
_lib.vosti_linear_fingerprint.restype = ctypes.c_uint64
_lib.vosti_linear_fingerprint.argtypes = []
_lib.vosti_linear_contract.restype = ctypes.c_int32
_lib.vosti_linear_contract.argtypes = [ctypes.POINTER(ctypes.c_uint32), ctypes.c_int32]
_lib.vosti_linear_poll_status.restype = ctypes.c_int
_lib.vosti_linear_poll_status.argtypes = [_vp]


def vosti_linear_tile_shape(N: int, K: int):
    """(B_M, B_N, B_K) for an (N, K) weight: a function of N and K only."""
    v = [ctypes.c_int32() for _ in range(3)]
    _vb._check(_lib.vosti_linear_tile_shape(int(N), int(K), *[ctypes.byref(x) for x in v]),
               "vosti_linear_tile_shape")
    return tuple(x.value for x in v)


def vosti_linear_segments(N: int, K: int) -> int:
    v = ctypes.c_int32()
    _vb._check(_lib.vosti_linear_segments(int(N), int(K), ctypes.byref(v)), "vosti_linear_segments")
    return v.value


def vosti_linear_workspace_bytes(M: int, N: int, K: int) -> int:
    return int(_lib.vosti_linear_workspace_bytes(int(M), int(N), int(K)))


def _bf16_cuda(t: torch.Tensor, ndim: int) -> torch.Tensor:
    assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous() and t.ndim == ndim
    return t


VOSTI_LINEAR_AUTO = 0
VOSTI_LINEAR_WHOLE_TILES = 1
VOSTI_LINEAR_SPLIT_WORKSPACE = 2
VOSTI_LINEAR_SPLIT_CLUSTER = 3
VOSTI_LINEAR_PAIRS = 4


def vosti_linear(x: torch.Tensor, w: torch.Tensor, y: torch.Tensor = None, workspace: torch.Tensor = None,
                 stream=None, schedule: int = VOSTI_LINEAR_AUTO) -> torch.Tensor:
    """y [M, N] = x [M, K] @ w [N, K]^T; tensors are CUDA bf16, contiguous.  workspace: an optional
    CUDA byte tensor (see vosti_linear_workspace_bytes) for the split schedule that needs one.
    schedule: VOSTI_LINEAR_AUTO, or one of the schedules by name (vosti_linear_ex)."""
    x, w = _bf16_cuda(x, 2), _bf16_cuda(w, 2)
    M, K = x.shape
    N = w.shape[0]
    assert w.shape[1] == K
    if y is None:
        y = torch.empty((M, N), dtype=torch.bfloat16, device=x.device)
    _bf16_cuda(y, 2)
    assert y.shape == (M, N)
    ws_ptr, ws_bytes = (0, 0) if workspace is None else (workspace.data_ptr(), workspace.numel() * workspace.element_size())
    if schedule == VOSTI_LINEAR_AUTO:
        _vb._check(_lib.vosti_linear(_vb._dev(x), _vb._dev(w), _vb._dev(y), M, N, K, ws_ptr, ws_bytes,
                                     _vb._stream(stream)), "vosti_linear")
    else:
        _vb._check(_lib.vosti_linear_ex(_vb._dev(x), _vb._dev(w), _vb._dev(y), M, N, K, ws_ptr, ws_bytes,
                                        int(schedule), _vb._stream(stream)), "vosti_linear_ex")
    return y


def vosti_rmsnorm(x: torch.Tensor, weight: torch.Tensor, eps: float, y: torch.Tensor = None,
                  stream=None) -> torch.Tensor:
    x, weight = _bf16_cuda(x, 2), _bf16_cuda(weight, 1)
    M, K = x.shape
    assert weight.shape == (K,)
    if y is None:
        y = torch.empty_like(x)
    _vb._check(_lib.vosti_rmsnorm(_vb._dev(x), _vb._dev(weight), _vb._dev(y), M, K, float(eps),
                                  _vb._stream(stream)), "vosti_rmsnorm")
    return y


def vosti_linear_poll_status(stream=None) -> int:
    return int(_lib.vosti_linear_poll_status(_vb._stream(stream)))


def vosti_linear_fingerprint() -> int:
    return int(_lib.vosti_linear_fingerprint())


def vosti_linear_contract():
    buf = (ctypes.c_uint32 * 16)()
    n = _lib.vosti_linear_contract(buf, 16)
    return [int(x) for x in buf[:n]]
