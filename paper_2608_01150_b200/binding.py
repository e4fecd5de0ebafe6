"""ctypes binding of libzellige.so -- same names as the C ABI in include/zellige.h.

Argument marshalling only.  Tensors are torch CUDA tensors (device memory and streams come
from PyTorch); the functions pass their data pointers and the current stream to the
library.  Raw-pointer entry points (``*_ptr``) take integers so that callers holding host
buffers can drive the same C calls.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence, Tuple

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libzellige.so")

STATUS_NAMES = {0: "ZL_OK", 1: "ZL_ERR_INVALID_ARG", 2: "ZL_ERR_OVERLAP", 3: "ZL_ERR_UNSUPPORTED",
                4: "ZL_ERR_WORKSPACE", 5: "ZL_ERR_CUDA", 6: "ZL_ERR_TIMEOUT"}


KERNEL_NAMES = ("fwd", "merge", "bwd_pre", "bwd_main", "bwd_post")


class ZlError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {STATUS_NAMES.get(status, status)}")


class ShardDesc(ctypes.Structure):
    _fields_ = [("q_off", ctypes.c_int32), ("q_len", ctypes.c_int32), ("kv_off", ctypes.c_int32),
                ("kv_len", ctypes.c_int32), ("seq_id", ctypes.c_int32)]


class WholeDesc(ctypes.Structure):
    _fields_ = [("off", ctypes.c_int32), ("len", ctypes.c_int32), ("head_begin", ctypes.c_int32),
                ("head_count", ctypes.c_int32)]


class HeadRange(ctypes.Structure):
    _fields_ = [("head_begin", ctypes.c_int32), ("head_count", ctypes.c_int32)]


class TasksInfo(ctypes.Structure):
    _fields_ = [("n_tasks", ctypes.c_int32), ("n_merge_groups", ctypes.c_int32),
                ("n_kv_groups", ctypes.c_int32), ("n_fwd_items", ctypes.c_int32),
                ("n_bwd_items", ctypes.c_int32), ("partial_rows", ctypes.c_int64),
                ("o_partial_bytes", ctypes.c_size_t), ("lse_partial_bytes", ctypes.c_size_t),
                ("bwd_workspace_bytes", ctypes.c_size_t), ("n_fused_ranges", ctypes.c_int32)]


def library_path() -> str:
    return _LIB_PATH


def _load():
    if not os.path.exists(_LIB_PATH):
        raise ImportError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2608_01150_b200.build` "
            "(nvcc, sm_100a). There is no fallback path.")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, i32, i64p = ctypes.c_void_p, ctypes.c_int32, ctypes.POINTER(ctypes.c_int64)
    lib.zl_build_tasks.restype = ctypes.c_int
    lib.zl_build_tasks.argtypes = [vp, i32, vp, i32, i32, i32, i32, i32, vp, ctypes.POINTER(vp)]
    lib.zl_build_tasks_ex.restype = ctypes.c_int
    lib.zl_build_tasks_ex.argtypes = [vp, i32, vp, i32, i32, i32, i32, i32, ctypes.c_uint32, vp, ctypes.POINTER(vp)]
    lib.zl_build_tasks_heads.restype = ctypes.c_int
    lib.zl_build_tasks_heads.argtypes = [vp, i32, vp, vp, i32, i32, i32, i32, i32, ctypes.c_uint32, vp, ctypes.POINTER(vp)]
    lib.zl_tasks_get_info.restype = ctypes.c_int
    lib.zl_tasks_get_info.argtypes = [vp, ctypes.POINTER(TasksInfo)]
    lib.zl_tasks_get_partial_slot.restype = ctypes.c_int
    lib.zl_tasks_get_partial_slot.argtypes = [vp, i32, i64p, i64p]
    for name in ("zl_tasks_get_fwd_items", "zl_tasks_get_bwd_items"):
        getattr(lib, name).restype = ctypes.c_int
        getattr(lib, name).argtypes = [vp, vp, i32, ctypes.POINTER(i32)]
    lib.zl_free_tasks.restype = None
    lib.zl_free_tasks.argtypes = [vp]
    lib.zl_coalesced_attn_fwd.restype = ctypes.c_int
    lib.zl_coalesced_attn_fwd.argtypes = [vp, vp, vp, vp, ctypes.c_float, vp, vp, vp, vp, vp]
    lib.zl_coalesced_attn_fwd_packed.restype = ctypes.c_int
    lib.zl_coalesced_attn_fwd_packed.argtypes = [vp, vp, ctypes.c_float, vp, vp, vp, vp, vp]
    lib.zl_coalesced_attn_bwd_packed.restype = ctypes.c_int
    lib.zl_coalesced_attn_bwd_packed.argtypes = [vp, vp, vp, vp, vp, ctypes.c_float, vp, vp, ctypes.c_size_t, vp]
    lib.zl_lse_merge.restype = ctypes.c_int
    lib.zl_lse_merge.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.zl_coalesced_attn_bwd.restype = ctypes.c_int
    lib.zl_coalesced_attn_bwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, ctypes.c_float, vp, vp, vp, vp,
                                          ctypes.c_size_t, vp]
    for name in ("zl_set_fwd_phases", "zl_set_bwd_phases"):
        getattr(lib, name).restype = ctypes.c_int
        getattr(lib, name).argtypes = [vp, vp, vp, i32, vp]
    lib.zl_coalesced_attn_fwd_phase.restype = ctypes.c_int
    lib.zl_coalesced_attn_fwd_phase.argtypes = [vp, i32, vp, vp, vp, ctypes.c_float, vp, vp, vp, vp, vp]
    lib.zl_coalesced_attn_bwd_phase.restype = ctypes.c_int
    lib.zl_coalesced_attn_bwd_phase.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp, ctypes.c_float, vp, vp, vp, vp,
                                                ctypes.c_size_t, vp]
    lib.zl_phase_info.restype = ctypes.c_int
    lib.zl_phase_info.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(i32)]
    lib.zl_set_sm_margin.restype = ctypes.c_int
    lib.zl_set_sm_margin.argtypes = [vp, i32]
    lib.zl_coalesced_attn_bwd_noalloc.restype = ctypes.c_int
    lib.zl_coalesced_attn_bwd_noalloc.argtypes = [vp, vp, vp, vp, vp, vp, vp, ctypes.c_float, vp, vp, vp, vp]
    lib.zl_last_device_status.restype = ctypes.c_int
    lib.zl_last_device_status.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(i32)]
    lib.zl_set_kernel_timing.restype = ctypes.c_int
    lib.zl_set_kernel_timing.argtypes = [vp, i32]
    lib.zl_get_kernel_timing.restype = ctypes.c_int
    lib.zl_get_kernel_timing.argtypes = [vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(i32)]
    lib.zl_debug_set_fwd_order.restype = ctypes.c_int
    lib.zl_debug_set_fwd_order.argtypes = [vp, i32, vp]
    lib.zl_set_bwd_kernel.restype = ctypes.c_int
    lib.zl_set_bwd_kernel.argtypes = [vp, i32]
    lib.zl_selftest_bounded_wait.restype = ctypes.c_int
    lib.zl_selftest_bounded_wait.argtypes = [vp, i32, vp]
    lib.zl_status_str.restype = ctypes.c_char_p
    lib.zl_status_str.argtypes = [ctypes.c_int]
    lib.zl_launch_count.restype = ctypes.c_int64
    lib.zl_launch_count.argtypes = []
    return lib


_lib = _load()


def lib():
    return _lib


def _check(status: int, what: str):
    if status != 0:
        raise ZlError(status, what)


def _stream_ptr(stream=None) -> int:
    import torch
    if stream is None:
        if not torch.cuda.is_available():
            return 0
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream) if hasattr(stream, "cuda_stream") else int(stream)


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


class TaskHandle:
    """Owns a ``zl_tasks*``.  Built once per placement, reused for every layer and step."""

    def __init__(self, ptr: int, n_heads: int, head_dim: int, total_q: int, total_kv: int, n_shards: int):
        self._ptr = ctypes.c_void_p(ptr)
        self.n_heads, self.head_dim, self.total_q, self.total_kv = n_heads, head_dim, total_q, total_kv
        self.n_shards = n_shards
        info = TasksInfo()
        _check(_lib.zl_tasks_get_info(self._ptr, ctypes.byref(info)), "zl_tasks_get_info")
        self.info = info

    @property
    def ptr(self):
        return self._ptr

    def partial_slot(self, shard_idx: int) -> Tuple[int, int]:
        a, b = ctypes.c_int64(), ctypes.c_int64()
        _check(_lib.zl_tasks_get_partial_slot(self._ptr, shard_idx, ctypes.byref(a), ctypes.byref(b)),
               "zl_tasks_get_partial_slot")
        return a.value, b.value

    def _items(self, fn) -> List[Tuple[int, int, int, int]]:
        n = ctypes.c_int32()
        _check(fn(self._ptr, None, 0, ctypes.byref(n)), "items count")
        buf = (ctypes.c_int32 * (4 * max(1, n.value)))()
        _check(fn(self._ptr, buf, n.value, ctypes.byref(n)), "items")
        return [tuple(buf[4 * i:4 * i + 4]) for i in range(n.value)]

    def fwd_items(self):
        return self._items(_lib.zl_tasks_get_fwd_items)

    def bwd_items(self):
        return self._items(_lib.zl_tasks_get_bwd_items)

    def last_device_status(self) -> Tuple[int, int]:
        c, w = ctypes.c_int32(), ctypes.c_int32()
        _check(_lib.zl_last_device_status(self._ptr, ctypes.byref(c), ctypes.byref(w)), "zl_last_device_status")
        return c.value, w.value

    def set_kernel_timing(self, enable: bool):
        _check(_lib.zl_set_kernel_timing(self._ptr, 1 if enable else 0), "zl_set_kernel_timing")

    def get_kernel_timing(self):
        """{kernel name: (total ms, launches)} since the last read; synchronises the device."""
        ms = (ctypes.c_float * len(KERNEL_NAMES))()
        n = (ctypes.c_int32 * len(KERNEL_NAMES))()
        _check(_lib.zl_get_kernel_timing(self._ptr, ms, n), "zl_get_kernel_timing")
        return {name: (float(ms[i]), int(n[i])) for i, name in enumerate(KERNEL_NAMES)}

    def set_fwd_order(self, mode: int, stream=None):
        """0 longest-first (default), 1 placement order, 2 shortest-first (measurement aid)."""
        _check(_lib.zl_debug_set_fwd_order(self._ptr, mode, _stream_ptr(stream)), "zl_debug_set_fwd_order")

    @staticmethod
    def _phase_array(values):
        if values is None:
            return None, None
        arr = (ctypes.c_int32 * max(1, len(values)))(*[int(v) for v in values])
        return arr, ctypes.cast(arr, ctypes.c_void_p)

    def set_fwd_phases(self, whole_phase, shard_phase, n_phases: int, stream=None):
        """zl_set_fwd_phases: one phase number per whole sequence / per shard (None = all zero)."""
        a, ap = self._phase_array(whole_phase)
        b, bp = self._phase_array(shard_phase)
        _check(_lib.zl_set_fwd_phases(self._ptr, ap, bp, n_phases, _stream_ptr(stream)), "zl_set_fwd_phases")

    def set_bwd_phases(self, whole_phase, shard_phase, n_phases: int, stream=None):
        """zl_set_bwd_phases."""
        a, ap = self._phase_array(whole_phase)
        b, bp = self._phase_array(shard_phase)
        _check(_lib.zl_set_bwd_phases(self._ptr, ap, bp, n_phases, _stream_ptr(stream)), "zl_set_bwd_phases")

    def phase_info(self):
        """zl_phase_info: (forward items per phase, backward items per phase)."""
        nf, nb = ctypes.c_int32(0), ctypes.c_int32(0)
        fi, bi = (ctypes.c_int32 * MAX_PHASES)(), (ctypes.c_int32 * MAX_PHASES)()
        _check(_lib.zl_phase_info(self._ptr, ctypes.byref(nf), ctypes.byref(nb), fi, bi), "zl_phase_info")
        return list(fi[:nf.value]), list(bi[:nb.value])

    def set_sm_margin(self, n_sms: int):
        """zl_set_sm_margin: SMs the persistent kernels leave free for kernels of other streams."""
        _check(_lib.zl_set_sm_margin(self._ptr, n_sms), "zl_set_sm_margin")

    def set_bwd_kernel(self, kernel: int):
        """0 library default, 1 one CTA per key tile, 2 CTA pairs (head_dim 128)."""
        _check(_lib.zl_set_bwd_kernel(self._ptr, kernel), "zl_set_bwd_kernel")

    def selftest_bounded_wait(self, limit_us: int = 1000, stream=None):
        """Launches a kernel whose bounded wait must expire; read the outcome with last_device_status()."""
        _check(_lib.zl_selftest_bounded_wait(self._ptr, limit_us, _stream_ptr(stream)), "zl_selftest_bounded_wait")

    def close(self):
        if self._ptr:
            _lib.zl_free_tasks(self._ptr)
            self._ptr = ctypes.c_void_p(0)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


BUILD_FUSE_LOCAL_CHUNKS = 1
MAX_PHASES = 64  # ZL_MAX_PHASES


def build_tasks(cu_seqlens: Sequence[int], shards: Sequence[Sequence[int]], total_q: int, total_kv: int,
                n_heads: int, head_dim: int, stream=None, flags: int = 0) -> TaskHandle:
    """zl_build_tasks / zl_build_tasks_ex: placement (cu_seqlens + shard descriptors) -> task handle.
    flags: 0 or BUILD_FUSE_LOCAL_CHUNKS."""
    n_whole = max(0, len(cu_seqlens) - 1)
    cu = (ctypes.c_int32 * max(1, len(cu_seqlens)))(*[int(c) for c in cu_seqlens])
    sh = (ShardDesc * max(1, len(shards)))(*[ShardDesc(*[int(v) for v in s]) for s in shards])
    out = ctypes.c_void_p()
    cu_p = ctypes.cast(cu, ctypes.c_void_p) if len(cu_seqlens) else None
    sh_p = ctypes.cast(sh, ctypes.c_void_p) if len(shards) else None
    if flags:
        st = _lib.zl_build_tasks_ex(cu_p, n_whole, sh_p, len(shards), total_q, total_kv, n_heads, head_dim,
                                    ctypes.c_uint32(flags), _stream_ptr(stream), ctypes.byref(out))
    else:
        st = _lib.zl_build_tasks(cu_p, n_whole, sh_p, len(shards), total_q, total_kv, n_heads, head_dim,
                                 _stream_ptr(stream), ctypes.byref(out))
    _check(st, "zl_build_tasks")
    return TaskHandle(out.value, n_heads, head_dim, total_q, total_kv, len(shards))


def build_tasks_heads(whole: Sequence[Sequence[int]], shards: Sequence[Sequence[int]],
                      shard_heads: Optional[Sequence[Sequence[int]]], total_q: int, total_kv: int,
                      n_heads: int, head_dim: int, stream=None, flags: int = 0) -> TaskHandle:
    """zl_build_tasks_heads: whole = (off, len, head_begin, head_count) per whole sequence, shards =
    (q_off, q_len, kv_off, kv_len, seq_id) per shard, shard_heads = (head_begin, head_count) per shard or
    None for all heads."""
    wd = (WholeDesc * max(1, len(whole)))(*[WholeDesc(*[int(v) for v in w]) for w in whole])
    sh = (ShardDesc * max(1, len(shards)))(*[ShardDesc(*[int(v) for v in s[:5]]) for s in shards])
    hr = None
    if shard_heads is not None:
        assert len(shard_heads) == len(shards)
        hr = (HeadRange * max(1, len(shards)))(*[HeadRange(int(a), int(b)) for a, b in shard_heads])
    out = ctypes.c_void_p()
    st = _lib.zl_build_tasks_heads(ctypes.cast(wd, ctypes.c_void_p) if len(whole) else None, len(whole),
                                   ctypes.cast(sh, ctypes.c_void_p) if len(shards) else None,
                                   ctypes.cast(hr, ctypes.c_void_p) if hr is not None and len(shards) else None,
                                   len(shards), total_q, total_kv, n_heads, head_dim, ctypes.c_uint32(flags),
                                   _stream_ptr(stream), ctypes.byref(out))
    _check(st, "zl_build_tasks_heads")
    return TaskHandle(out.value, n_heads, head_dim, total_q, total_kv, len(shards))


def coalesced_attn_fwd(tasks: TaskHandle, q, k, v, scale: float, o, lse, o_partial=None, lse_partial=None,
                       stream=None):
    """zl_coalesced_attn_fwd.  Tensors: torch CUDA tensors or raw device pointers (int)."""
    _check(_lib.zl_coalesced_attn_fwd(tasks.ptr, _ptr(q), _ptr(k), _ptr(v), ctypes.c_float(scale), _ptr(o),
                                      _ptr(lse), _ptr(o_partial), _ptr(lse_partial), _stream_ptr(stream)),
           "zl_coalesced_attn_fwd")


def coalesced_attn_fwd_phase(tasks: TaskHandle, phase: int, q, k, v, scale: float, o, lse, o_partial=None,
                             lse_partial=None, stream=None):
    """zl_coalesced_attn_fwd_phase: the tasks of one launch phase."""
    _check(_lib.zl_coalesced_attn_fwd_phase(tasks.ptr, phase, _ptr(q), _ptr(k), _ptr(v), ctypes.c_float(scale), _ptr(o),
                                            _ptr(lse), _ptr(o_partial), _ptr(lse_partial), _stream_ptr(stream)),
           "zl_coalesced_attn_fwd_phase")


def coalesced_attn_bwd_phase(tasks: TaskHandle, phase: int, q, k, v, o, lse, d_o, scale: float, dq, dk, dv, workspace,
                             workspace_bytes: Optional[int] = None, stream=None):
    """zl_coalesced_attn_bwd_phase: phases 0 .. n-1 in order, same arguments."""
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    _check(_lib.zl_coalesced_attn_bwd_phase(tasks.ptr, phase, _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(d_o),
                                            ctypes.c_float(scale), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(workspace),
                                            ctypes.c_size_t(workspace_bytes), _stream_ptr(stream)),
           "zl_coalesced_attn_bwd_phase")


def lse_merge(tasks: TaskHandle, o_partial, lse_partial, o, lse, stream=None):
    """zl_lse_merge."""
    _check(_lib.zl_lse_merge(tasks.ptr, _ptr(o_partial), _ptr(lse_partial), _ptr(o), _ptr(lse),
                             _stream_ptr(stream)), "zl_lse_merge")


def coalesced_attn_bwd(tasks: TaskHandle, q, k, v, o, lse, d_o, scale: float, dq, dk, dv, workspace,
                       workspace_bytes: Optional[int] = None, stream=None):
    """zl_coalesced_attn_bwd."""
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    _check(_lib.zl_coalesced_attn_bwd(tasks.ptr, _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(d_o),
                                      ctypes.c_float(scale), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(workspace),
                                      ctypes.c_size_t(workspace_bytes), _stream_ptr(stream)),
           "zl_coalesced_attn_bwd")


def coalesced_attn_fwd_packed(tasks: TaskHandle, qkv, scale: float, o, lse, o_partial=None, lse_partial=None,
                              stream=None):
    """zl_coalesced_attn_fwd_packed: qkv is [T, 3, H, d] bf16 (total_q == total_kv == T)."""
    _check(_lib.zl_coalesced_attn_fwd_packed(tasks.ptr, _ptr(qkv), ctypes.c_float(scale), _ptr(o), _ptr(lse),
                                             _ptr(o_partial), _ptr(lse_partial), _stream_ptr(stream)),
           "zl_coalesced_attn_fwd_packed")


def coalesced_attn_bwd_packed(tasks: TaskHandle, qkv, o, lse, d_o, scale: float, dqkv, workspace,
                              workspace_bytes: Optional[int] = None, stream=None):
    """zl_coalesced_attn_bwd_packed: reads qkv [T, 3, H, d], writes dqkv [T, 3, H, d]."""
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    _check(_lib.zl_coalesced_attn_bwd_packed(tasks.ptr, _ptr(qkv), _ptr(o), _ptr(lse), _ptr(d_o),
                                             ctypes.c_float(scale), _ptr(dqkv), _ptr(workspace),
                                             ctypes.c_size_t(workspace_bytes), _stream_ptr(stream)),
           "zl_coalesced_attn_bwd_packed")


NOALLOC_SCRATCH_BYTES = 64 * 1024 * 1024


def coalesced_attn_bwd_noalloc(tasks: TaskHandle, q, k, v, o, lse, d_o, scale: float, dq, dk, dv, stream=None):
    """zl_coalesced_attn_bwd_noalloc: the backward for callers that cannot allocate device memory
    (no workspace argument; the scratch is a fixed 64 MiB array inside the library).  Raises
    ZL_ERR_WORKSPACE for placements that need more scratch than that.  Calls must not overlap on
    the GPU, and the first call on a device should be made outside stream capture."""
    _check(_lib.zl_coalesced_attn_bwd_noalloc(tasks.ptr, _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(d_o),
                                              ctypes.c_float(scale), _ptr(dq), _ptr(dk), _ptr(dv),
                                              _stream_ptr(stream)), "zl_coalesced_attn_bwd_noalloc")


def launch_count() -> int:
    return int(_lib.zl_launch_count())
