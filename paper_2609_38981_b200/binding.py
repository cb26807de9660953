"""ctypes binding of libvosti (``include/vosti.h``): argument marshalling only.

Every step of the path runs in the library's CUDA kernels; this module turns
torch tensors into device pointers and numpy arrays into host pointers.  There
is no fallback: if the built library is missing, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libvosti.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2609_38981_b200.build` "
        "(nvcc, sm_100a).  There is no CPU or PyTorch fallback.")

_lib = ctypes.CDLL(LIB_PATH)

VOSTI_OK, VOSTI_ERR_INVALID_ARG, VOSTI_ERR_UNSUPPORTED_CONFIG, VOSTI_ERR_OUT_OF_RANGE, \
    VOSTI_ERR_WORKSPACE, VOSTI_ERR_CUDA, VOSTI_ERR_TIMEOUT = range(7)
VOSTI_FLAG_CHECK_WRITE_SLOTS = 1
VOSTI_FLAG_PACK_SHARED_SPLITS = 2
VOSTI_FLAG_PACK_THROUGH_TILES = 4
VOSTI_FLAG_NO_OVERLAP = 8
VOSTI_HOST_STEPS_IN_FLIGHT = 3

EXPORTS = (
    "vosti_workspace_bytes", "vosti_plan", "vosti_plan_ex", "vosti_create", "vosti_destroy", "vosti_kv_append",
    "vosti_paged_attention", "vosti_paged_attention_ex", "vosti_paged_attention_noalloc", "vosti_noalloc_poll_status",
    "vosti_noalloc_selftest_bounded_wait", "vosti_cp_partial", "vosti_cp_segments",
    "vosti_cp_combine", "vosti_step_host", "vosti_step_host_async", "vosti_step_host_wait",
    "vosti_device_plan_bytes", "vosti_plan_device", "vosti_kv_append_planned", "vosti_paged_attention_planned",
    "vosti_poll_device_status",
    "vosti_selftest_bounded_wait", "vosti_selftest_mma", "vosti_profile_enable", "vosti_profile_read", "vosti_launch_count",
    "vosti_last_schedule", "vosti_fingerprint", "vosti_contract", "vosti_host_time",
    "vosti_constants", "vosti_status_string",
)


class vosti_config(ctypes.Structure):
    _fields_ = [
        ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32), ("page_size", ctypes.c_int32),
        ("num_pages", ctypes.c_int64), ("kv_pool", ctypes.c_void_p),
        ("max_batch", ctypes.c_int32), ("max_total_q", ctypes.c_int64),
        ("max_seq_len", ctypes.c_int64), ("workspace", ctypes.c_void_p),
        ("workspace_bytes", ctypes.c_size_t), ("flags", ctypes.c_uint32),
    ]


class vosti_work_item(ctypes.Structure):
    _fields_ = [("req", ctypes.c_int32), ("row_group", ctypes.c_int32),
                ("split_begin", ctypes.c_int32), ("split_end", ctypes.c_int32)]


_i32p = ctypes.c_void_p  # int32* arguments: passed as raw addresses (see _ip)
_cfgp = ctypes.POINTER(vosti_config)
_vp = ctypes.c_void_p

_lib.vosti_workspace_bytes.restype = ctypes.c_size_t
_lib.vosti_workspace_bytes.argtypes = [_cfgp]
_lib.vosti_plan.restype = ctypes.c_int
_lib.vosti_plan.argtypes = [_cfgp, _i32p, _i32p, _i32p, ctypes.c_int32,
                            ctypes.POINTER(vosti_work_item), ctypes.c_int64,
                            ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int64),
                            ctypes.POINTER(ctypes.c_int64)]
_lib.vosti_plan_ex.restype = ctypes.c_int
_lib.vosti_plan_ex.argtypes = [_cfgp, _i32p, _i32p, _i32p, ctypes.c_int32, ctypes.c_int32,
                               ctypes.POINTER(vosti_work_item), ctypes.c_int64,
                               ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int64),
                               ctypes.POINTER(ctypes.c_int64)]
_lib.vosti_create.restype = ctypes.c_int
_lib.vosti_create.argtypes = [ctypes.POINTER(_vp), _cfgp]
_lib.vosti_destroy.restype = ctypes.c_int
_lib.vosti_destroy.argtypes = [_vp]
_lib.vosti_kv_append.restype = ctypes.c_int
_lib.vosti_kv_append.argtypes = [_vp, _vp, _vp, _i32p, _i32p, _i32p, ctypes.c_int32,
                                 ctypes.c_int32, _vp]
_lib.vosti_paged_attention.restype = ctypes.c_int
_lib.vosti_paged_attention.argtypes = [_vp, _vp, _vp, _i32p, _i32p, _i32p, _i32p, ctypes.c_int32,
                                       ctypes.c_int32, ctypes.c_float, _vp]
_lib.vosti_paged_attention_ex.restype = ctypes.c_int
_lib.vosti_paged_attention_ex.argtypes = [_vp, _vp, _vp, _vp, _i32p, _i32p, _i32p, _i32p, ctypes.c_int32,
                                          ctypes.c_int32, ctypes.c_float, ctypes.c_int32, _vp]
_szp = ctypes.POINTER(ctypes.c_size_t)
_lib.vosti_cp_partial.restype = ctypes.c_int
_lib.vosti_cp_partial.argtypes = [_vp, _vp, _i32p, _i32p, _i32p, _i32p, ctypes.c_int32, ctypes.c_int32,
                                  ctypes.c_float, ctypes.c_int32, ctypes.c_int32, _szp, _szp, _szp, _szp, _vp]
_lib.vosti_cp_segments.restype = ctypes.c_int
_lib.vosti_cp_segments.argtypes = [_cfgp, _i32p, _i32p, _i32p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                   ctypes.c_void_p, ctypes.c_int64, ctypes.POINTER(ctypes.c_int64),
                                   ctypes.POINTER(ctypes.c_int64)]
_lib.vosti_cp_combine.restype = ctypes.c_int
_lib.vosti_cp_combine.argtypes = [_vp, _vp, _vp, _i32p, _i32p, _i32p, ctypes.c_int32, _vp]
_lib.vosti_paged_attention_noalloc.restype = ctypes.c_int
_lib.vosti_paged_attention_noalloc.argtypes = [
    ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, _vp, ctypes.c_int64, _vp, _vp,
    _i32p, _i32p, _i32p, _i32p, ctypes.c_int32, ctypes.c_int32, ctypes.c_float, _vp]
_lib.vosti_noalloc_poll_status.restype = ctypes.c_int
_lib.vosti_noalloc_poll_status.argtypes = [_vp]
_lib.vosti_noalloc_selftest_bounded_wait.restype = ctypes.c_int
_lib.vosti_noalloc_selftest_bounded_wait.argtypes = [ctypes.c_uint32, _vp]
_lib.vosti_step_host.restype = ctypes.c_int
_lib.vosti_step_host.argtypes = [_vp, _vp, _vp, _vp, _vp, _i32p, _i32p, _i32p, _i32p,
                                 ctypes.c_int32, ctypes.c_int32, ctypes.c_float, _vp]
_lib.vosti_step_host_async.restype = ctypes.c_int
_lib.vosti_step_host_async.argtypes = _lib.vosti_step_host.argtypes + [ctypes.POINTER(ctypes.c_int64)]
_lib.vosti_step_host_wait.restype = ctypes.c_int
_lib.vosti_step_host_wait.argtypes = [_vp, ctypes.c_int64]
_lib.vosti_device_plan_bytes.restype = ctypes.c_size_t
_lib.vosti_device_plan_bytes.argtypes = [_cfgp]
_lib.vosti_plan_device.restype = ctypes.c_int
_lib.vosti_plan_device.argtypes = [_vp, _vp, _vp, _vp, _vp, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                   ctypes.c_int32, _vp]
_lib.vosti_kv_append_planned.restype = ctypes.c_int
_lib.vosti_kv_append_planned.argtypes = [_vp, _vp, _vp, _vp, _vp, ctypes.c_int32, ctypes.c_int32, _vp]
_lib.vosti_paged_attention_planned.restype = ctypes.c_int
_lib.vosti_paged_attention_planned.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, ctypes.c_int32, ctypes.c_int32,
                                               ctypes.c_float, ctypes.c_int32, _vp]
_lib.vosti_poll_device_status.restype = ctypes.c_int
_lib.vosti_poll_device_status.argtypes = [_vp, _vp]
_lib.vosti_selftest_bounded_wait.restype = ctypes.c_int
_lib.vosti_selftest_bounded_wait.argtypes = [_vp, ctypes.c_uint32, _vp]
_lib.vosti_profile_enable.restype = ctypes.c_int
_lib.vosti_profile_enable.argtypes = [_vp, ctypes.c_int32]
_lib.vosti_profile_read.restype = ctypes.c_int
_lib.vosti_profile_read.argtypes = [_vp, ctypes.POINTER(ctypes.c_double),
                                    ctypes.POINTER(ctypes.c_int64)]
_lib.vosti_launch_count.restype = ctypes.c_int64
_lib.vosti_launch_count.argtypes = [_vp]
_lib.vosti_last_schedule.restype = ctypes.c_int
_lib.vosti_last_schedule.argtypes = [_vp, ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int64),
                                     ctypes.POINTER(ctypes.c_int64)]
_lib.vosti_fingerprint.restype = ctypes.c_uint64
_lib.vosti_fingerprint.argtypes = [_vp]
_lib.vosti_selftest_mma.restype = ctypes.c_int
_lib.vosti_selftest_mma.argtypes = [_vp, _vp, _vp, ctypes.c_int32, _vp, _vp, _vp]
_lib.vosti_host_time.restype = ctypes.c_int
_lib.vosti_host_time.argtypes = [_vp, ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int64), ctypes.c_int32]
_lib.vosti_contract.restype = ctypes.c_int32
_lib.vosti_contract.argtypes = [ctypes.POINTER(ctypes.c_uint32), ctypes.c_int32]
_lib.vosti_constants.restype = None
_lib.vosti_constants.argtypes = [_i32p, _i32p, _i32p]
_lib.vosti_status_string.restype = ctypes.c_char_p
_lib.vosti_status_string.argtypes = [ctypes.c_int]


class VostiError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {vosti_status_string(status)} ({status})")


def _check(status: int, where: str) -> None:
    if status != VOSTI_OK:
        raise VostiError(status, where)


def _host_i32(a) -> np.ndarray:
    if type(a) is np.ndarray and a.dtype == np.int32 and a.flags.c_contiguous:
        return a                      # the common case of a serving loop: nothing to convert
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _ip(a: np.ndarray) -> int:
    """Host address of an int32 array (the array must outlive the call).  A plain integer:
    building a typed ctypes pointer costs several microseconds per argument."""
    return a.ctypes.data


def _dev(t) -> int:
    """Device (or host) address of a contiguous torch tensor, or a raw int."""
    if t is None:
        return 0
    if isinstance(t, int):
        return t
    assert t.is_contiguous()
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return int(getattr(stream, "cuda_stream", stream))


def vosti_status_string(status: int) -> str:
    return _lib.vosti_status_string(int(status)).decode()


def vosti_constants():
    a, b, c = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
    _lib.vosti_constants(ctypes.byref(a), ctypes.byref(b), ctypes.byref(c))
    return {"key_tile": a.value, "split_len": b.value, "rows_per_group": c.value}


def make_config(n_q_heads, n_kv_heads, head_dim, page_size, num_pages, max_batch, max_total_q,
                max_seq_len, kv_pool=0, workspace=0, workspace_bytes=0, flags=0) -> vosti_config:
    return vosti_config(n_q_heads, n_kv_heads, head_dim, page_size, num_pages, _dev(kv_pool),
                        max_batch, max_total_q, max_seq_len, _dev(workspace), workspace_bytes, flags)


def vosti_workspace_bytes(cfg: vosti_config) -> int:
    return int(_lib.vosti_workspace_bytes(ctypes.byref(cfg)))


def vosti_plan(cfg: vosti_config, q_lens, start_pos, seq_lens):
    """Host-only planning.  Returns (items [n,4] int32, n_split, n_partial_rows)."""
    q, s, n = _host_i32(q_lens), _host_i32(start_pos), _host_i32(seq_lens)
    cnt, nsp, npr = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int64()
    _check(_lib.vosti_plan(ctypes.byref(cfg), _ip(q), _ip(s), _ip(n), len(q), None, 0,
                           ctypes.byref(cnt), ctypes.byref(nsp), ctypes.byref(npr)), "vosti_plan")
    items = (vosti_work_item * max(cnt.value, 1))()
    _check(_lib.vosti_plan(ctypes.byref(cfg), _ip(q), _ip(s), _ip(n), len(q), items, cnt.value,
                           ctypes.byref(cnt), ctypes.byref(nsp), ctypes.byref(npr)), "vosti_plan")
    arr = np.array([[it.req, it.row_group, it.split_begin, it.split_end]
                    for it in items[:cnt.value]], dtype=np.int32).reshape(-1, 4)
    return arr, nsp.value, npr.value


def vosti_plan_ex(cfg: vosti_config, q_lens, start_pos, seq_lens, window: int):
    """Host-only planning under a sliding window.  Returns like vosti_plan."""
    q, s, n = _host_i32(q_lens), _host_i32(start_pos), _host_i32(seq_lens)
    cnt, nsp, npr = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int64()
    _check(_lib.vosti_plan_ex(ctypes.byref(cfg), _ip(q), _ip(s), _ip(n), len(q), int(window), None, 0,
                              ctypes.byref(cnt), ctypes.byref(nsp), ctypes.byref(npr)), "vosti_plan_ex")
    items = (vosti_work_item * max(cnt.value, 1))()
    _check(_lib.vosti_plan_ex(ctypes.byref(cfg), _ip(q), _ip(s), _ip(n), len(q), int(window), items,
                              cnt.value, ctypes.byref(cnt), ctypes.byref(nsp), ctypes.byref(npr)),
           "vosti_plan_ex")
    arr = np.array([[it.req, it.row_group, it.split_begin, it.split_end]
                    for it in items[:cnt.value]], dtype=np.int32).reshape(-1, 4)
    return arr, nsp.value, npr.value


def vosti_fingerprint(ctx=None) -> int:
    return int(_lib.vosti_fingerprint(ctx.handle if ctx is not None else None))


def vosti_selftest_mma(ctx: "Context", a, b, mode: int, d_tc, d_warp, stream=None) -> None:
    """One [128 x 64] product by tcgen05.mma (d_tc) and by mma.sync (d_warp); see include/vosti.h."""
    _check(_lib.vosti_selftest_mma(ctx.handle, _dev(a), _dev(b), int(mode), _dev(d_tc), _dev(d_warp),
                                   _stream(stream)), "vosti_selftest_mma")


def vosti_host_time(ctx: "Context", reset: bool = False):
    """(nanoseconds, calls) the library spent on the host in append / attention calls of ctx."""
    ns, calls = ctypes.c_int64(), ctypes.c_int64()
    _check(_lib.vosti_host_time(ctx.handle, ctypes.byref(ns), ctypes.byref(calls), int(reset)), "vosti_host_time")
    return ns.value, calls.value


def vosti_contract():
    """The words vosti_fingerprint hashes (version, frozen sizes, rule ids), in order."""
    buf = (ctypes.c_uint32 * 32)()
    n = _lib.vosti_contract(buf, 32)
    return [int(x) for x in buf[:n]]


class Context:
    """Owns a vosti_ctx handle and keeps the pool / workspace tensors alive."""

    def __init__(self, cfg: vosti_config, keep=()):
        self.cfg = cfg
        self._keep = tuple(keep)
        self.workspace = keep[1] if len(keep) > 1 else None   # the torch tensor behind cfg.workspace
        h = _vp()
        _check(_lib.vosti_create(ctypes.byref(h), ctypes.byref(cfg)), "vosti_create")
        self.handle = h

    def close(self):
        if getattr(self, "handle", None):
            _lib.vosti_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def vosti_create(n_q_heads, n_kv_heads, head_dim, page_size, kv_pool, max_batch, max_total_q,
                 max_seq_len, flags=0, workspace=None) -> Context:
    """kv_pool: torch uint8/int16/bf16 CUDA tensor holding the whole pool.  The
    workspace is allocated with torch (device memory is torch's job here)
    unless one is passed in."""
    import torch
    page_bytes = n_kv_heads * 2 * page_size * head_dim * 2
    num_pages = kv_pool.numel() * kv_pool.element_size() // page_bytes
    cfg = make_config(n_q_heads, n_kv_heads, head_dim, page_size, num_pages, max_batch,
                      max_total_q, max_seq_len, flags=flags)
    need = vosti_workspace_bytes(cfg)
    if need == 0:
        raise VostiError(VOSTI_ERR_UNSUPPORTED_CONFIG, "vosti_workspace_bytes")
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=kv_pool.device)
    cfg.kv_pool = kv_pool.data_ptr()
    cfg.workspace = workspace.data_ptr()
    cfg.workspace_bytes = workspace.numel() * workspace.element_size()
    return Context(cfg, keep=(kv_pool, workspace))


def vosti_destroy(ctx: Context) -> None:
    ctx.close()


def vosti_kv_append(ctx: Context, k_new, v_new, q_lens, start_pos, block_tables,
                    stream=None) -> None:
    q, s = _host_i32(q_lens), _host_i32(start_pos)
    bt = _host_i32(block_tables)
    assert bt.ndim == 2 and bt.shape[0] == len(q)
    _check(_lib.vosti_kv_append(ctx.handle, _dev(k_new), _dev(v_new), _ip(q), _ip(s), _ip(bt),
                                bt.shape[1], len(q), _stream(stream)), "vosti_kv_append")


def vosti_paged_attention(ctx: Context, q, out, q_lens, start_pos, seq_lens, block_tables,
                          softmax_scale: float, stream=None) -> None:
    ql, s, n = _host_i32(q_lens), _host_i32(start_pos), _host_i32(seq_lens)
    bt = _host_i32(block_tables)
    assert bt.ndim == 2 and bt.shape[0] == len(ql)
    _check(_lib.vosti_paged_attention(ctx.handle, _dev(q), _dev(out), _ip(ql), _ip(s), _ip(n),
                                      _ip(bt), bt.shape[1], len(ql), float(softmax_scale),
                                      _stream(stream)), "vosti_paged_attention")


def vosti_paged_attention_ex(ctx: Context, q, out, lse, q_lens, start_pos, seq_lens, block_tables,
                             softmax_scale: float, window: int = 0, stream=None) -> None:
    """With a sliding window and / or the log-sum-exp output (lse: fp32 [T, Hq] or None)."""
    ql, s, n = _host_i32(q_lens), _host_i32(start_pos), _host_i32(seq_lens)
    bt = _host_i32(block_tables)
    assert bt.ndim == 2 and bt.shape[0] == len(ql)
    _check(_lib.vosti_paged_attention_ex(ctx.handle, _dev(q), _dev(out), _dev(lse) if lse is not None else None,
                                         _ip(ql), _ip(s), _ip(n), _ip(bt), bt.shape[1], len(ql),
                                         float(softmax_scale), int(window), _stream(stream)),
           "vosti_paged_attention_ex")


def vosti_cp_partial(ctx: Context, q, q_lens, start_pos, seq_lens, block_tables, softmax_scale: float,
                     cp_rank: int, cp_world: int, stream=None):
    """Context-parallel phase 1.  Returns the two fp32 views of the context's workspace
    (partial U rows, partial (m, z) pairs) that the caller sums over ranks in place."""
    import torch
    ql, s, n = _host_i32(q_lens), _host_i32(start_pos), _host_i32(seq_lens)
    bt = _host_i32(block_tables)
    assert bt.ndim == 2 and bt.shape[0] == len(ql)
    v = [ctypes.c_size_t() for _ in range(4)]
    _check(_lib.vosti_cp_partial(ctx.handle, _dev(q), _ip(ql), _ip(s), _ip(n), _ip(bt), bt.shape[1], len(ql),
                                 float(softmax_scale), int(cp_rank), int(cp_world),
                                 *[ctypes.byref(x) for x in v], _stream(stream)), "vosti_cp_partial")
    ws = ctx._keep[1]
    assert ws.dtype == torch.uint8
    u = ws[v[0].value:v[0].value + v[1].value].view(torch.float32)
    mz = ws[v[2].value:v[2].value + v[3].value].view(torch.float32)
    return u, mz


def vosti_cp_segments(cfg: vosti_config, q_lens, start_pos, seq_lens, cp_rank: int, cp_world: int):
    """Host-only: the partial rows rank cp_rank owns, as an int64 array [n, 2] of (first row,
    rows), and the total number of partial rows of the call."""
    ql, s, n = _host_i32(q_lens), _host_i32(start_pos), _host_i32(seq_lens)
    cnt, rows = ctypes.c_int64(), ctypes.c_int64()
    _check(_lib.vosti_cp_segments(ctypes.byref(cfg), _ip(ql), _ip(s), _ip(n), len(ql), cp_rank, cp_world,
                                  None, 0, ctypes.byref(cnt), ctypes.byref(rows)), "vosti_cp_segments")
    seg = np.zeros((max(cnt.value, 1), 2), dtype=np.int64)
    _check(_lib.vosti_cp_segments(ctypes.byref(cfg), _ip(ql), _ip(s), _ip(n), len(ql), cp_rank, cp_world,
                                  seg.ctypes.data, cnt.value, ctypes.byref(cnt), ctypes.byref(rows)),
           "vosti_cp_segments")
    return seg[:cnt.value], rows.value


def vosti_cp_combine(ctx: Context, out, lse, q_lens, start_pos, seq_lens, stream=None) -> None:
    """Context-parallel phase 2: the fold over all splits (after the sum over ranks)."""
    ql, s, n = _host_i32(q_lens), _host_i32(start_pos), _host_i32(seq_lens)
    _check(_lib.vosti_cp_combine(ctx.handle, _dev(out), _dev(lse) if lse is not None else None, _ip(ql), _ip(s),
                                 _ip(n), len(ql), _stream(stream)), "vosti_cp_combine")


def vosti_paged_attention_noalloc(n_q_heads, n_kv_heads, head_dim, page_size, kv_pool, q, out,
                                  q_lens, start_pos, seq_lens, block_tables,
                                  softmax_scale: float, stream=None) -> None:
    """Context-free variant that allocates nothing (see include/vosti.h for its
    limits).  kv_pool is the torch tensor holding the whole pool."""
    ql, s, n = _host_i32(q_lens), _host_i32(start_pos), _host_i32(seq_lens)
    bt = _host_i32(block_tables)
    assert bt.ndim == 2 and bt.shape[0] == len(ql)
    page_bytes = n_kv_heads * 2 * page_size * head_dim * 2
    num_pages = kv_pool.numel() * kv_pool.element_size() // page_bytes
    _check(_lib.vosti_paged_attention_noalloc(
        n_q_heads, n_kv_heads, head_dim, page_size, _dev(kv_pool), num_pages, _dev(q), _dev(out),
        _ip(ql), _ip(s), _ip(n), _ip(bt), bt.shape[1], len(ql), float(softmax_scale),
        _stream(stream)), "vosti_paged_attention_noalloc")


def vosti_noalloc_poll_status(stream=None) -> int:
    """Reads and clears the status word of the allocation-free entry point (current device)."""
    return _lib.vosti_noalloc_poll_status(_stream(stream))


def vosti_noalloc_selftest_bounded_wait(limit_us: int, stream=None) -> None:
    _check(_lib.vosti_noalloc_selftest_bounded_wait(int(limit_us), _stream(stream)),
           "vosti_noalloc_selftest_bounded_wait")


def vosti_step_host(ctx: Context, q_host, out_host, k_new_host, v_new_host, q_lens, start_pos,
                    seq_lens, block_tables, softmax_scale: float, stream=None) -> None:
    ql, s, n = _host_i32(q_lens), _host_i32(start_pos), _host_i32(seq_lens)
    bt = _host_i32(block_tables)
    _check(_lib.vosti_step_host(ctx.handle, _dev(q_host), _dev(out_host), _dev(k_new_host),
                                _dev(v_new_host), _ip(ql), _ip(s), _ip(n), _ip(bt), bt.shape[1],
                                len(ql), float(softmax_scale), _stream(stream)), "vosti_step_host")


def vosti_step_host_async(ctx: Context, q_host, out_host, k_new_host, v_new_host, q_lens, start_pos,
                          seq_lens, block_tables, softmax_scale: float, stream=None) -> int:
    """Returns the step's ticket; the host buffers belong to the library until it is waited for."""
    ql, s, n = _host_i32(q_lens), _host_i32(start_pos), _host_i32(seq_lens)
    bt = _host_i32(block_tables)
    ticket = ctypes.c_int64(-1)
    _check(_lib.vosti_step_host_async(ctx.handle, _dev(q_host), _dev(out_host), _dev(k_new_host),
                                      _dev(v_new_host), _ip(ql), _ip(s), _ip(n), _ip(bt), bt.shape[1],
                                      len(ql), float(softmax_scale), _stream(stream), ctypes.byref(ticket)),
           "vosti_step_host_async")
    return ticket.value


def vosti_step_host_wait(ctx: Context, ticket: int) -> None:
    _check(_lib.vosti_step_host_wait(ctx.handle, int(ticket)), "vosti_step_host_wait")


def vosti_device_plan_bytes(ctx: Context) -> int:
    return int(_lib.vosti_device_plan_bytes(ctypes.byref(ctx.cfg)))


def vosti_plan_device(ctx: Context, plan, q_lens_dev, start_pos_dev, block_tables_dev, max_q_len: int,
                      stream=None, window: int = 0) -> None:
    """All array arguments are int32 CUDA tensors; `plan` a CUDA byte tensor of vosti_device_plan_bytes."""
    _check(_lib.vosti_plan_device(ctx.handle, _dev(plan), _dev(q_lens_dev), _dev(start_pos_dev),
                                  _dev(block_tables_dev), block_tables_dev.shape[1], q_lens_dev.shape[0],
                                  int(max_q_len), int(window), _stream(stream)), "vosti_plan_device")


def vosti_kv_append_planned(ctx: Context, plan, k_new, v_new, block_tables_dev, max_q_len: int,
                            stream=None) -> None:
    _check(_lib.vosti_kv_append_planned(ctx.handle, _dev(plan), _dev(k_new), _dev(v_new), _dev(block_tables_dev),
                                        block_tables_dev.shape[0], int(max_q_len), _stream(stream)),
           "vosti_kv_append_planned")


def vosti_paged_attention_planned(ctx: Context, plan, q, out, lse, block_tables_dev, max_q_len: int,
                                  softmax_scale: float, stream=None, window: int = 0) -> None:
    _check(_lib.vosti_paged_attention_planned(ctx.handle, _dev(plan), _dev(q), _dev(out), _dev(lse),
                                              _dev(block_tables_dev), block_tables_dev.shape[0], int(max_q_len),
                                              float(softmax_scale), int(window), _stream(stream)),
           "vosti_paged_attention_planned")


def vosti_poll_device_status(ctx: Context, stream=None) -> int:
    return int(_lib.vosti_poll_device_status(ctx.handle, _stream(stream)))


def vosti_selftest_bounded_wait(ctx: Context, limit_us: int, stream=None) -> None:
    _check(_lib.vosti_selftest_bounded_wait(ctx.handle, int(limit_us), _stream(stream)),
           "vosti_selftest_bounded_wait")


def vosti_profile_enable(ctx: Context, mode: int) -> None:
    _check(_lib.vosti_profile_enable(ctx.handle, int(mode)), "vosti_profile_enable")


def vosti_profile_read(ctx: Context):
    ms, n = ctypes.c_double(), ctypes.c_int64()
    _check(_lib.vosti_profile_read(ctx.handle, ctypes.byref(ms), ctypes.byref(n)),
           "vosti_profile_read")
    return ms.value, n.value


def vosti_last_schedule(ctx: "Context"):
    """(split-parallel items, packed items among them, tile items) of the last attention call."""
    a, b, c = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int64()
    _check(_lib.vosti_last_schedule(ctx.handle, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)),
           "vosti_last_schedule")
    return a.value, b.value, c.value


def vosti_launch_count(ctx: Context) -> int:
    return int(_lib.vosti_launch_count(ctx.handle))
