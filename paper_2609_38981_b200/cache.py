"""ctypes binding of the prefix-cache manager (``include/vosti_cache.h``):
argument marshalling only.  The manager is host-side C++ inside libvosti."""
from __future__ import annotations

import ctypes
from typing import List, Sequence, Tuple

import numpy as np

from . import binding as _vb

_lib = _vb._lib
_vp = ctypes.c_void_p
_i32p = ctypes.POINTER(ctypes.c_int32)
_i64p = ctypes.POINTER(ctypes.c_int64)

EXPORTS = (
    "vosti_cache_create", "vosti_cache_destroy", "vosti_cache_admit", "vosti_cache_append",
    "vosti_cache_computed", "vosti_cache_step_boundary", "vosti_cache_finish", "vosti_cache_block_table",
    "vosti_cache_stats", "vosti_cache_check", "vosti_cache_page_info", "vosti_cache_debug_set_hash_mask",
)

_lib.vosti_cache_create.restype = ctypes.c_int
_lib.vosti_cache_create.argtypes = [ctypes.POINTER(_vp), ctypes.c_int64, ctypes.c_int32]
_lib.vosti_cache_destroy.restype = ctypes.c_int
_lib.vosti_cache_destroy.argtypes = [_vp]
_lib.vosti_cache_admit.restype = ctypes.c_int
_lib.vosti_cache_admit.argtypes = [_vp, ctypes.c_int64, _i32p, ctypes.c_int64, _i64p]
_lib.vosti_cache_append.restype = ctypes.c_int
_lib.vosti_cache_append.argtypes = [_vp, ctypes.c_int64, _i32p, ctypes.c_int64]
_lib.vosti_cache_computed.restype = ctypes.c_int
_lib.vosti_cache_computed.argtypes = [_vp, ctypes.c_int64, ctypes.c_int64]
_lib.vosti_cache_step_boundary.restype = ctypes.c_int
_lib.vosti_cache_step_boundary.argtypes = [_vp]
_lib.vosti_cache_finish.restype = ctypes.c_int
_lib.vosti_cache_finish.argtypes = [_vp, ctypes.c_int64]
_lib.vosti_cache_block_table.restype = ctypes.c_int
_lib.vosti_cache_block_table.argtypes = [_vp, ctypes.c_int64, _i32p, ctypes.c_int64, _i64p]
_lib.vosti_cache_stats.restype = ctypes.c_int
_lib.vosti_cache_stats.argtypes = [_vp, _i64p, _i64p, _i64p, _i64p, _i64p]
_lib.vosti_cache_check.restype = ctypes.c_int
_lib.vosti_cache_check.argtypes = [_vp, ctypes.POINTER(ctypes.c_char_p)]
_lib.vosti_cache_page_info.restype = ctypes.c_int
_lib.vosti_cache_page_info.argtypes = [_vp, ctypes.c_int32, _i32p, _i32p, _i32p, _i32p]
_lib.vosti_cache_debug_set_hash_mask.restype = ctypes.c_int
_lib.vosti_cache_debug_set_hash_mask.argtypes = [_vp, ctypes.c_uint64]


def _tok(tokens) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))


class PrefixCache:
    """Owns a vosti_cache handle."""

    def __init__(self, num_pages: int, page_size: int):
        h = _vp()
        _vb._check(_lib.vosti_cache_create(ctypes.byref(h), int(num_pages), int(page_size)), "vosti_cache_create")
        self.handle = h
        self.page_size = page_size
        self.num_pages = num_pages

    def close(self):
        if self.handle:
            _lib.vosti_cache_destroy(self.handle)
            self.handle = None

    def __del__(self):
        self.close()

    def admit(self, request_id: int, tokens) -> int:
        """Returns the number of leading tokens already cached."""
        t = _tok(tokens)
        n = ctypes.c_int64()
        _vb._check(_lib.vosti_cache_admit(self.handle, int(request_id), t.ctypes.data_as(_i32p), len(t),
                                          ctypes.byref(n)), "vosti_cache_admit")
        return n.value

    def append(self, request_id: int, tokens) -> None:
        t = _tok(tokens)
        _vb._check(_lib.vosti_cache_append(self.handle, int(request_id), t.ctypes.data_as(_i32p), len(t)),
                   "vosti_cache_append")

    def computed(self, request_id: int, upto: int) -> None:
        _vb._check(_lib.vosti_cache_computed(self.handle, int(request_id), int(upto)), "vosti_cache_computed")

    def step_boundary(self) -> None:
        _vb._check(_lib.vosti_cache_step_boundary(self.handle), "vosti_cache_step_boundary")

    def finish(self, request_id: int) -> None:
        _vb._check(_lib.vosti_cache_finish(self.handle, int(request_id)), "vosti_cache_finish")

    def block_table(self, request_id: int) -> List[int]:
        n = ctypes.c_int64()
        _vb._check(_lib.vosti_cache_block_table(self.handle, int(request_id), None, 0, ctypes.byref(n)),
                   "vosti_cache_block_table")
        out = np.zeros(max(n.value, 1), dtype=np.int32)
        _vb._check(_lib.vosti_cache_block_table(self.handle, int(request_id), out.ctypes.data_as(_i32p),
                                                n.value, ctypes.byref(n)), "vosti_cache_block_table")
        return out[:n.value].tolist()

    def stats(self) -> dict:
        v = [ctypes.c_int64() for _ in range(5)]
        _vb._check(_lib.vosti_cache_stats(self.handle, *[ctypes.byref(x) for x in v]), "vosti_cache_stats")
        return dict(zip(("free", "retained", "live", "hit_pages", "evicted_pages"), (x.value for x in v)))

    def check(self) -> str:
        """'' when every bookkeeping invariant holds, else the violated condition."""
        what = ctypes.c_char_p()
        rc = _lib.vosti_cache_check(self.handle, ctypes.byref(what))
        return "" if rc == 0 else (what.value or b"?").decode()

    def page_info(self, page: int):
        """(depth, parent, refs, children) of a registered page, or None."""
        v = [ctypes.c_int32() for _ in range(4)]
        rc = _lib.vosti_cache_page_info(self.handle, int(page), *[ctypes.byref(x) for x in v])
        return None if rc != 0 else tuple(x.value for x in v)

    def debug_set_hash_mask(self, mask: int) -> None:
        _vb._check(_lib.vosti_cache_debug_set_hash_mask(self.handle, int(mask)), "vosti_cache_debug_set_hash_mask")
