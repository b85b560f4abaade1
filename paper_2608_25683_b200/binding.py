"""ctypes binding of libpsrl.so: same names as the C ABI, argument marshalling only.

Every step of the path runs inside the library's kernels.  The binding raises
if the library has not been built; there is no fallback of any kind.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpsrl.so")

PSRL_OK = 0
STATUS_NAMES = [
    "PSRL_OK", "PSRL_ERR_INVALID_ARG", "PSRL_ERR_BAD_TREE", "PSRL_ERR_BAD_BLOCK_SIZE", "PSRL_ERR_SHAPE",
    "PSRL_ERR_UNSUPPORTED", "PSRL_ERR_POOL_FULL", "PSRL_ERR_WORKSPACE", "PSRL_ERR_HOST_OOM", "PSRL_ERR_CUDA",
    "PSRL_ERR_TIMEOUT", "PSRL_ERR_INTERNAL",
]
PSRL_F32, PSRL_BF16 = 0, 1
BWD_STATIC_SCRATCH_BYTES = 16 * 1024 * 1024 + 256   # PSRL_BWD_STATIC_SCRATCH_BYTES of include/psrl.h
SEG_HAS_Q, SEG_SAMPLE_END = 1, 2

EXPORTS = [
    "psrl_plan_build", "psrl_plan_view", "psrl_plan_device_bytes", "psrl_plan_upload",
    "psrl_fwd_workspace_bytes", "psrl_bwd_workspace_bytes", "psrl_tree_attn_fwd", "psrl_tree_attn_bwd",
    "psrl_device_status", "psrl_last_cuda_error", "psrl_plan_destroy", "psrl_status_string",
    "psrl_bench_bwd_phases", "psrl_tree_attn_bwd_static", "psrl_launch_count", "psrl_plan_schedule",
    "psrl_cache_create", "psrl_cache_begin", "psrl_cache_end", "psrl_cache_stats", "psrl_cache_refcounts",
    "psrl_cache_destroy",
    "psrl_kv_scatter", "psrl_kv_gather",
    "psrl_cost_sequence", "psrl_group_workloads", "psrl_place_groups", "psrl_microbatch_tokens",
]

_I32P = C.POINTER(C.c_int32)


class TreeDesc(C.Structure):
    _fields_ = [
        ("n_segments", C.c_int32), ("parent", _I32P), ("seg_len", _I32P), ("seg_flags", C.POINTER(C.c_uint8)),
        ("group_block_size", _I32P), ("n_groups", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
        ("head_dim", C.c_int32), ("dtype", C.c_int), ("free_extents", _I32P), ("n_free", C.c_int32),
        ("seg_slot_base", _I32P),
    ]


class CostModel(C.Structure):
    _fields_ = [("a1", C.c_double), ("a2", C.c_double), ("a3", C.c_double)]


class CacheDesc(C.Structure):
    _fields_ = [
        ("n_segments", C.c_int32), ("parent", _I32P), ("seg_len", _I32P), ("seg_flags", C.POINTER(C.c_uint8)),
        ("group_block_size", _I32P), ("n_groups", C.c_int32), ("n_microbatches", C.c_int32), ("mb_of_seg", _I32P),
        ("capacity_slots", C.c_int64),
    ]


class CacheStep(C.Structure):
    _fields_ = [
        ("n_segments", C.c_int32), ("seg_id", _I32P), ("parent", _I32P), ("seg_len", _I32P),
        ("seg_flags", C.POINTER(C.c_uint8)), ("group_block_size", _I32P), ("n_groups", C.c_int32),
        ("seg_slot_base", _I32P), ("n_new", C.c_int32), ("n_reload", C.c_int32), ("n_evict", C.c_int32),
        ("new_seg", _I32P), ("reload_seg", _I32P), ("evict_seg", _I32P), ("evict_base", _I32P),
        ("live_slots", C.c_int64), ("pool_slots", C.c_int64),
    ]


class CacheStats(C.Structure):
    _fields_ = [("peak_slots", C.c_int64), ("evicted_slots", C.c_int64), ("reloaded_slots", C.c_int64),
                ("pool_high_water", C.c_int64), ("total_slots", C.c_int64)]


_VIEW_SCALARS32 = ["n_seg", "n_groups", "n_pages", "n_samples", "max_depth", "T", "T_q", "pool_slots"]
_VIEW_SCALARS64 = ["flat_tokens", "tree_pairs", "flat_pairs"]
_VIEW_ARRAYS = [
    "canon_of_input", "input_of_canon", "seg_group", "seg_bs", "seg_parent", "seg_len", "seg_flags", "seg_depth",
    "seg_anc_tokens", "seg_sub_end", "seg_tok_off", "seg_q_off", "seg_refcount", "anc_off", "anc_list",
    "seg_first_page", "seg_n_pages", "page_seg", "page_bs", "page_valid", "page_pos", "page_refcount", "page_slot",
    "bt_off", "bt_pages", "tok_slot", "sample_end_seg", "sample_len",
]


class PlanView(C.Structure):
    _fields_ = (
        [(n, C.c_int32) for n in _VIEW_SCALARS32]
        + [(n, C.c_int64) for n in _VIEW_SCALARS64]
        + [("n_anc", C.c_int32), ("n_bt", C.c_int32)]
        + [(n, _I32P) for n in _VIEW_ARRAYS]
    )


class PsrlError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{where}: {name}{(' (' + detail + ')') if detail else ''}")
        self.status = status
        self.name = name


_lib = None


def lib() -> C.CDLL:
    """Load libpsrl.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2608_25683_b200.build` "
            "(there is no fallback path)")
    L = C.CDLL(LIB_PATH)
    L.psrl_plan_build.argtypes = [C.POINTER(TreeDesc), C.POINTER(C.c_void_p)]
    L.psrl_plan_build.restype = C.c_int
    L.psrl_plan_view.argtypes = [C.c_void_p, C.POINTER(PlanView)]
    L.psrl_plan_view.restype = C.c_int
    L.psrl_plan_device_bytes.argtypes = [C.c_void_p]
    L.psrl_plan_device_bytes.restype = C.c_size_t
    L.psrl_plan_upload.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    L.psrl_plan_upload.restype = C.c_int
    for f in (L.psrl_fwd_workspace_bytes, L.psrl_bwd_workspace_bytes):
        f.argtypes = [C.c_void_p]
        f.restype = C.c_size_t
    L.psrl_tree_attn_fwd.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p,
                                     C.c_void_p, C.c_float, C.c_void_p, C.c_size_t, C.c_void_p]
    L.psrl_tree_attn_fwd.restype = C.c_int
    L.psrl_tree_attn_bwd.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p,
                                     C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_float,
                                     C.c_void_p, C.c_size_t, C.c_void_p]
    L.psrl_tree_attn_bwd.restype = C.c_int
    L.psrl_device_status.argtypes = [C.c_void_p, C.c_void_p]
    L.psrl_device_status.restype = C.c_int
    L.psrl_tree_attn_bwd_static.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p,
                                            C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_float,
                                            C.POINTER(C.c_void_p), C.c_void_p]
    L.psrl_tree_attn_bwd_static.restype = C.c_int
    L.psrl_bench_bwd_phases.argtypes = L.psrl_tree_attn_bwd.argtypes + [C.c_int]
    L.psrl_bench_bwd_phases.restype = C.c_int
    L.psrl_plan_schedule.argtypes = [C.c_void_p, C.POINTER(_I32P), C.POINTER(C.c_size_t)]
    L.psrl_plan_schedule.restype = C.c_int
    _F64P = C.POINTER(C.c_double)
    _U8P = C.POINTER(C.c_uint8)
    L.psrl_cost_sequence.argtypes = [C.POINTER(CostModel), C.c_int64, C.c_int64]
    L.psrl_cost_sequence.restype = C.c_double
    L.psrl_group_workloads.argtypes = [C.c_int32, _I32P, _I32P, _U8P, C.POINTER(CostModel), C.c_int32, _F64P]
    L.psrl_group_workloads.restype = C.c_int
    L.psrl_place_groups.argtypes = [C.c_int32, _F64P, C.c_int32, _I32P, _F64P]
    L.psrl_place_groups.restype = C.c_int
    L.psrl_microbatch_tokens.argtypes = [C.c_int32, _I32P, _I32P, _U8P, C.POINTER(CostModel), C.c_int32, C.c_int32,
                                         _I32P, _I32P, _I32P, _I32P, _I32P, _I32P, _F64P]
    L.psrl_microbatch_tokens.restype = C.c_int
    L.psrl_kv_scatter.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]
    L.psrl_kv_scatter.restype = C.c_int
    L.psrl_kv_gather.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p]
    L.psrl_kv_gather.restype = C.c_int
    L.psrl_cache_create.argtypes = [C.POINTER(CacheDesc), C.POINTER(C.c_void_p)]
    L.psrl_cache_create.restype = C.c_int
    L.psrl_cache_begin.argtypes = [C.c_void_p, C.c_int32, C.POINTER(CacheStep)]
    L.psrl_cache_begin.restype = C.c_int
    L.psrl_cache_end.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.c_int32), C.POINTER(_I32P), C.POINTER(C.c_int64)]
    L.psrl_cache_end.restype = C.c_int
    L.psrl_cache_stats.argtypes = [C.c_void_p, C.POINTER(CacheStats)]
    L.psrl_cache_stats.restype = C.c_int
    L.psrl_cache_refcounts.argtypes = [C.c_void_p, C.POINTER(_I32P)]
    L.psrl_cache_refcounts.restype = C.c_int
    L.psrl_cache_destroy.argtypes = [C.c_void_p]
    L.psrl_cache_destroy.restype = None
    L.psrl_launch_count.argtypes = [C.c_void_p, C.c_int]
    L.psrl_launch_count.restype = C.c_int
    L.psrl_last_cuda_error.restype = C.c_char_p
    L.psrl_plan_destroy.argtypes = [C.c_void_p]
    L.psrl_plan_destroy.restype = None
    L.psrl_status_string.argtypes = [C.c_int]
    L.psrl_status_string.restype = C.c_char_p
    _lib = L
    return L


def _check(status: int, where: str):
    if status != PSRL_OK:
        detail = ""
        if status == 9:
            detail = lib().psrl_last_cuda_error().decode()
        raise PsrlError(status, where, detail)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


class Plan:
    """Owner of a psrl_plan_t.  `view` holds numpy copies of the canonical arrays."""

    def __init__(self, parent: Sequence[int], seg_len: Sequence[int], group_block_size: Sequence[int],
                 n_q_heads: int, n_kv_heads: int, head_dim: int, dtype: str,
                 seg_flags: Optional[Sequence[int]] = None, free_extents=None, seg_slot_base=None):
        self._h = C.c_void_p()
        self._dev = None
        self._ws = {}
        L = lib()
        p, l, g = _i32(parent), _i32(seg_len), _i32(group_block_size)
        d = TreeDesc()
        d.n_segments = len(p)
        d.parent = p.ctypes.data_as(_I32P)
        d.seg_len = l.ctypes.data_as(_I32P)
        fl = None
        if seg_flags is not None:
            fl = np.ascontiguousarray(np.asarray(seg_flags, dtype=np.uint8))
            d.seg_flags = fl.ctypes.data_as(C.POINTER(C.c_uint8))
        d.group_block_size = g.ctypes.data_as(_I32P)
        d.n_groups = len(g)
        d.n_q_heads, d.n_kv_heads, d.head_dim = int(n_q_heads), int(n_kv_heads), int(head_dim)
        d.dtype = {"f32": PSRL_F32, "bf16": PSRL_BF16}.get(dtype, 99)
        fe = None
        if free_extents is not None:
            fe = _i32(np.asarray(free_extents, dtype=np.int64).reshape(-1))
            d.free_extents = fe.ctypes.data_as(_I32P)
            d.n_free = len(fe) // 2
        sb = None
        if seg_slot_base is not None:
            sb = _i32(seg_slot_base)
            if len(sb) != len(p):
                raise ValueError("seg_slot_base needs one entry per segment")
            d.seg_slot_base = sb.ctypes.data_as(_I32P)
        _check(L.psrl_plan_build(C.byref(d), C.byref(self._h)), "psrl_plan_build")
        self.n_q_heads, self.n_kv_heads, self.head_dim, self.dtype = int(n_q_heads), int(n_kv_heads), int(head_dim), dtype
        v = PlanView()
        _check(L.psrl_plan_view(self._h, C.byref(v)), "psrl_plan_view")
        self.view = self._copy_view(v)

    @staticmethod
    def _copy_view(v: PlanView) -> dict:
        out = {n: int(getattr(v, n)) for n in _VIEW_SCALARS32 + _VIEW_SCALARS64}
        n_seg, n_pages = out["n_seg"], out["n_pages"]
        sizes = {n: n_seg for n in _VIEW_ARRAYS}
        sizes.update(anc_off=n_seg + 1, anc_list=int(v.n_anc), bt_off=n_seg + 1, bt_pages=int(v.n_bt),
                     tok_slot=out["T"], sample_end_seg=out["n_samples"], sample_len=out["n_samples"])
        for n in ("page_seg", "page_bs", "page_valid", "page_pos", "page_refcount", "page_slot"):
            sizes[n] = n_pages
        for n in _VIEW_ARRAYS:
            sz = sizes[n]
            ptr = getattr(v, n)
            out[n] = np.ctypeslib.as_array(ptr, shape=(sz,)).copy() if sz > 0 else np.zeros(0, dtype=np.int32)
        return out

    @property
    def handle(self):
        return self._h

    def schedule(self) -> np.ndarray:
        """Copy of the device work schedule (int32 words) for host-side checks."""
        words, n = _I32P(), C.c_size_t()
        _check(lib().psrl_plan_schedule(self._h, C.byref(words), C.byref(n)), "psrl_plan_schedule")
        return np.ctypeslib.as_array(words, shape=(n.value,)).copy()

    def device_bytes(self) -> int:
        return int(lib().psrl_plan_device_bytes(self._h))

    def fwd_workspace_bytes(self) -> int:
        return int(lib().psrl_fwd_workspace_bytes(self._h))

    def bwd_workspace_bytes(self) -> int:
        return int(lib().psrl_bwd_workspace_bytes(self._h))

    def upload(self, device="cuda", stream=None):
        """Allocate the device mirror with torch and upload the schedule."""
        import torch

        buf = torch.empty(self.device_bytes() + 256, dtype=torch.uint8, device=device)
        ptr = (buf.data_ptr() + 255) // 256 * 256
        s = _stream_ptr(stream)
        _check(lib().psrl_plan_upload(self._h, C.c_void_p(ptr), self.device_bytes(), s), "psrl_plan_upload")
        self._dev = buf
        return self

    def workspace(self, kind: str, device="cuda"):
        """A cached torch workspace of the right size ('fwd' | 'bwd'); returns (ptr, bytes)."""
        import torch

        need = self.fwd_workspace_bytes() if kind == "fwd" else self.bwd_workspace_bytes()
        key = (kind, str(torch.device(device if self._dev is None else self._dev.device)))
        if key not in self._ws:
            self._ws[key] = torch.empty(need + 256, dtype=torch.uint8, device=device)
        buf = self._ws[key]
        return (buf.data_ptr() + 255) // 256 * 256, need

    def close(self):
        if self._h:
            lib().psrl_plan_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def _stream_ptr(stream) -> C.c_void_p:
    if stream is None:
        import torch

        if torch.cuda.is_available():
            return C.c_void_p(torch.cuda.current_stream().cuda_stream)
        return C.c_void_p(0)
    if hasattr(stream, "cuda_stream"):
        return C.c_void_p(stream.cuda_stream)
    return C.c_void_p(int(stream))


def psrl_tree_attn_fwd(plan: Plan, q, k_pool, v_pool, softmax_scale: float, o=None, lse=None, stream=None,
                       workspace=None):
    """Forward.  q [T_q,Hq,d], pools [Hkv,capacity,d] torch CUDA tensors of the
    plan's dtype.  Returns (o, lse); both are allocated with torch if not given."""
    import torch

    V = plan.view
    assert q.is_contiguous() and k_pool.is_contiguous() and v_pool.is_contiguous()
    assert tuple(q.shape) == (V["T_q"], plan.n_q_heads, plan.head_dim), q.shape
    assert k_pool.shape == v_pool.shape and k_pool.shape[0] == plan.n_kv_heads and k_pool.shape[2] == plan.head_dim
    _check_dtype(plan, q, k_pool, v_pool)
    if o is None:
        o = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((plan.n_q_heads, V["T_q"]), dtype=torch.float32, device=q.device)
    ws, wsb = workspace if workspace is not None else plan.workspace("fwd", q.device)
    st = lib().psrl_tree_attn_fwd(plan.handle, q.data_ptr(), k_pool.data_ptr(), v_pool.data_ptr(),
                                  int(k_pool.shape[1]), o.data_ptr(), lse.data_ptr(), float(softmax_scale),
                                  C.c_void_p(ws), wsb, _stream_ptr(stream))
    _check(st, "psrl_tree_attn_fwd")
    return o, lse


def psrl_tree_attn_bwd(plan: Plan, q, k_pool, v_pool, o, lse, d_o, softmax_scale: float, d_q=None, dk_pool=None,
                       dv_pool=None, stream=None, workspace=None):
    """Backward.  Returns (d_q, dk_pool, dv_pool).  dk/dv pools are allocated
    zero-filled if not given (the library itself only writes the plan's pages)."""
    import torch

    _check_dtype(plan, q, k_pool, v_pool, o, d_o)
    assert d_o.is_contiguous() and o.is_contiguous() and lse.is_contiguous()
    if d_q is None:
        d_q = torch.empty_like(q)
    if dk_pool is None:
        dk_pool = torch.zeros_like(k_pool)
    if dv_pool is None:
        dv_pool = torch.zeros_like(v_pool)
    ws, wsb = workspace if workspace is not None else plan.workspace("bwd", q.device)
    st = lib().psrl_tree_attn_bwd(plan.handle, q.data_ptr(), k_pool.data_ptr(), v_pool.data_ptr(),
                                  int(k_pool.shape[1]), o.data_ptr(), lse.data_ptr(), d_o.data_ptr(), d_q.data_ptr(),
                                  dk_pool.data_ptr(), dv_pool.data_ptr(), float(softmax_scale), C.c_void_p(ws), wsb,
                                  _stream_ptr(stream))
    _check(st, "psrl_tree_attn_bwd")
    return d_q, dk_pool, dv_pool


def psrl_device_status(plan: Plan, kind: str = "fwd", stream=None, device="cuda") -> int:
    ws, _ = plan.workspace(kind, device)
    return int(lib().psrl_device_status(C.c_void_p(ws), _stream_ptr(stream)))


def psrl_tree_attn_bwd_static(plan: Plan, q, k_pool, v_pool, o, lse, d_o, softmax_scale: float, d_q, dk_pool,
                              dv_pool, stream=None) -> int:
    """Backward without any device allocation: for callers that may not touch
    the CUDA allocator (see include/psrl.h).  Unlike psrl_tree_attn_bwd this
    wrapper allocates nothing either, so every output tensor must be passed in.
    The library's built-in scratch array serves as workspace; it is shared by
    all calls on the device, so calls must not overlap on the GPU, and its size
    caps the problem: plan.bwd_workspace_bytes() (header + D, one float per query
    row and head, + slabs of split KV tiles + partial dQ rows) must not exceed
    BWD_STATIC_SCRATCH_BYTES = 16 MiB + 256 (PSRL_ERR_WORKSPACE beyond).
    Returns the device address of the status header (for psrl_device_status)."""
    _check_dtype(plan, q, k_pool, v_pool, o, d_o, d_q, dk_pool, dv_pool)
    ws = C.c_void_p()
    st = lib().psrl_tree_attn_bwd_static(plan.handle, q.data_ptr(), k_pool.data_ptr(), v_pool.data_ptr(),
                                         int(k_pool.shape[1]), o.data_ptr(), lse.data_ptr(), d_o.data_ptr(),
                                         d_q.data_ptr(), dk_pool.data_ptr(), dv_pool.data_ptr(),
                                         float(softmax_scale), C.byref(ws), _stream_ptr(stream))
    _check(st, "psrl_tree_attn_bwd_static")
    return int(ws.value or 0)


def psrl_bench_bwd_phases(plan: Plan, q, k_pool, v_pool, o, lse, d_o, softmax_scale: float, d_q, dk_pool, dv_pool,
                          phases: int, stream=None, workspace=None):
    """Benchmark aid: the backward with a mask of the kernels to launch (bit 0 D pre-pass, bit 1 dQ,
    bit 2 dK/dV), so that each can be timed on its own.  Outputs must be passed in."""
    _check_dtype(plan, q, k_pool, v_pool, o, d_o, d_q, dk_pool, dv_pool)
    ws, wsb = workspace if workspace is not None else plan.workspace("bwd", q.device)
    st = lib().psrl_bench_bwd_phases(plan.handle, q.data_ptr(), k_pool.data_ptr(), v_pool.data_ptr(),
                                     int(k_pool.shape[1]), o.data_ptr(), lse.data_ptr(), d_o.data_ptr(),
                                     d_q.data_ptr(), dk_pool.data_ptr(), dv_pool.data_ptr(), float(softmax_scale),
                                     C.c_void_p(ws), wsb, _stream_ptr(stream), int(phases))
    _check(st, "psrl_bench_bwd_phases")


def psrl_kv_scatter(plan: Plan, k_tok, v_tok, k_pool, v_pool, stream=None):
    """Token-major K, V [T, Hkv, d] -> slots tok_slot[t] of the pools [Hkv, capacity, d] (in place)."""
    _check_dtype(plan, k_tok, v_tok, k_pool, v_pool)
    T, Hkv, d = plan.view["T"], plan.n_kv_heads, plan.head_dim
    for t in (k_tok, v_tok):
        if tuple(t.shape) != (T, Hkv, d) or not t.is_contiguous():
            raise ValueError("k_tok / v_tok must be contiguous [T, Hkv, d]")
    if k_pool.shape != v_pool.shape or k_pool.shape[0] != Hkv or k_pool.shape[2] != d or not k_pool.is_contiguous():
        raise ValueError("pools must be contiguous [Hkv, capacity, d]")
    _check(lib().psrl_kv_scatter(plan._h, k_tok.data_ptr(), v_tok.data_ptr(), k_pool.data_ptr(), v_pool.data_ptr(),
                                 int(k_pool.shape[1]), _stream_ptr(stream)), "psrl_kv_scatter")


def psrl_kv_gather(plan: Plan, k_pool, v_pool, k_tok=None, v_tok=None, stream=None):
    """The inverse read: pools -> token-major [T, Hkv, d] (e.g. dK, dV back to the projections)."""
    import torch

    _check_dtype(plan, k_pool, v_pool)
    T, Hkv, d = plan.view["T"], plan.n_kv_heads, plan.head_dim
    if k_tok is None:
        k_tok = torch.empty((T, Hkv, d), dtype=k_pool.dtype, device=k_pool.device)
    if v_tok is None:
        v_tok = torch.empty((T, Hkv, d), dtype=v_pool.dtype, device=v_pool.device)
    _check(lib().psrl_kv_gather(plan._h, k_pool.data_ptr(), v_pool.data_ptr(), int(k_pool.shape[1]), k_tok.data_ptr(),
                                v_tok.data_ptr(), _stream_ptr(stream)), "psrl_kv_gather")
    return k_tok, v_tok


def _flags_ptr(seg_flags):
    if seg_flags is None:
        return None, None
    fl = np.ascontiguousarray(np.asarray(seg_flags, dtype=np.uint8))
    return fl, fl.ctypes.data_as(C.POINTER(C.c_uint8))


def psrl_cost_sequence(alpha, l: int, h: int) -> float:
    """Eq. 1 for one sequence of length l with a cached prefix of h tokens."""
    m = CostModel(*[float(a) for a in alpha])
    return float(lib().psrl_cost_sequence(C.byref(m), int(l), int(h)))


def psrl_group_workloads(parent, seg_len, alpha, seg_flags=None):
    """Workload of every prefix group (sum of Eq. 1 over its samples)."""
    p, l = _i32(parent), _i32(seg_len)
    n_groups = int((p == -1).sum())
    out = np.zeros(n_groups, dtype=np.float64)
    m = CostModel(*[float(a) for a in alpha])
    keep, fp = _flags_ptr(seg_flags)
    _check(lib().psrl_group_workloads(len(p), p.ctypes.data_as(_I32P), l.ctypes.data_as(_I32P), fp, C.byref(m), n_groups,
                                      out.ctypes.data_as(C.POINTER(C.c_double))), "psrl_group_workloads")
    return out


def psrl_place_groups(workload, n_workers: int):
    """Longest-processing-time-first placement: (worker of every group, load of every worker)."""
    w = np.ascontiguousarray(np.asarray(workload, dtype=np.float64))
    worker = np.zeros(len(w), dtype=np.int32)
    load = np.zeros(int(n_workers), dtype=np.float64)
    _check(lib().psrl_place_groups(len(w), w.ctypes.data_as(C.POINTER(C.c_double)), int(n_workers),
                                   worker.ctypes.data_as(_I32P), load.ctypes.data_as(C.POINTER(C.c_double))),
           "psrl_place_groups")
    return worker, load


def psrl_microbatch_tokens(parent, seg_len, alpha, n_microbatches: int, seg_flags=None):
    """Token-wise micro-batching: the forest of pieces as a dict of arrays (parent, seg_len, mb, seg, begin)
    plus the per-micro-batch budget."""
    p, l = _i32(parent), _i32(seg_len)
    cap = len(p) + int(n_microbatches)
    outs = [np.zeros(cap, dtype=np.int32) for _ in range(5)]
    n, budget = C.c_int32(), C.c_double()
    m = CostModel(*[float(a) for a in alpha])
    keep, fp = _flags_ptr(seg_flags)
    _check(lib().psrl_microbatch_tokens(len(p), p.ctypes.data_as(_I32P), l.ctypes.data_as(_I32P), fp, C.byref(m),
                                        int(n_microbatches), cap, C.byref(n), *[o.ctypes.data_as(_I32P) for o in outs],
                                        C.byref(budget)), "psrl_microbatch_tokens")
    k = n.value
    return dict(parent=outs[0][:k].copy(), seg_len=outs[1][:k].copy(), mb=outs[2][:k].copy(), seg=outs[3][:k].copy(),
                begin=outs[4][:k].copy(), budget=float(budget.value))


class Cache:
    """Owner of a psrl_cache_t (Dynamic Block Caching over an ordered list of micro-batches).
    begin(m) returns the micro-batch's tree as plain lists, ready for Plan(..., seg_slot_base=...)."""

    def __init__(self, parent, seg_len, group_block_size, mb_of_seg, n_microbatches: int, seg_flags=None,
                 capacity_slots: int = 0):
        self._h = C.c_void_p()
        p, l, g, mb = _i32(parent), _i32(seg_len), _i32(group_block_size), _i32(mb_of_seg)
        d = CacheDesc()
        d.n_segments = len(p)
        d.parent, d.seg_len = p.ctypes.data_as(_I32P), l.ctypes.data_as(_I32P)
        fl = None
        if seg_flags is not None:
            fl = np.ascontiguousarray(np.asarray(seg_flags, dtype=np.uint8))
            d.seg_flags = fl.ctypes.data_as(C.POINTER(C.c_uint8))
        d.group_block_size, d.n_groups = g.ctypes.data_as(_I32P), len(g)
        d.n_microbatches = int(n_microbatches)
        if len(mb) != len(p) or len(l) != len(p):
            raise ValueError("parent, seg_len and mb_of_seg need one entry per segment")
        d.mb_of_seg = mb.ctypes.data_as(_I32P)
        d.capacity_slots = int(capacity_slots)
        self.n_segments = len(p)
        _check(lib().psrl_cache_create(C.byref(d), C.byref(self._h)), "psrl_cache_create")

    def begin(self, m: int) -> dict:
        st = CacheStep()
        _check(lib().psrl_cache_begin(self._h, int(m), C.byref(st)), "psrl_cache_begin")
        arr = lambda ptr, k: [int(ptr[i]) for i in range(k)]
        k = st.n_segments
        return dict(seg_id=arr(st.seg_id, k), parent=arr(st.parent, k), seg_len=arr(st.seg_len, k),
                    seg_flags=arr(st.seg_flags, k), group_block_size=arr(st.group_block_size, st.n_groups),
                    seg_slot_base=arr(st.seg_slot_base, k), new=arr(st.new_seg, st.n_new),
                    reload=arr(st.reload_seg, st.n_reload),
                    evict=list(zip(arr(st.evict_seg, st.n_evict), arr(st.evict_base, st.n_evict))),
                    live_slots=int(st.live_slots), pool_slots=int(st.pool_slots))

    def end(self, m: int) -> dict:
        nf, ptr, live = C.c_int32(), _I32P(), C.c_int64()
        _check(lib().psrl_cache_end(self._h, int(m), C.byref(nf), C.byref(ptr), C.byref(live)), "psrl_cache_end")
        return dict(freed=[int(ptr[i]) for i in range(nf.value)], live_slots=int(live.value))

    def stats(self) -> dict:
        s = CacheStats()
        _check(lib().psrl_cache_stats(self._h, C.byref(s)), "psrl_cache_stats")
        return {n: int(getattr(s, n)) for n, _ in CacheStats._fields_}

    def refcounts(self):
        ptr = _I32P()
        _check(lib().psrl_cache_refcounts(self._h, C.byref(ptr)), "psrl_cache_refcounts")
        return [int(ptr[i]) for i in range(self.n_segments)]

    def __del__(self):
        if getattr(self, "_h", None) and self._h.value:
            lib().psrl_cache_destroy(self._h)
            self._h = C.c_void_p()


def psrl_launch_count(plan: Plan, backward: bool) -> int:
    """Kernels one forward (backward=False) or backward call launches for this plan."""
    return int(lib().psrl_launch_count(plan._h, int(bool(backward))))


def _check_dtype(plan: Plan, *tensors):
    import torch

    want = torch.float32 if plan.dtype == "f32" else torch.bfloat16
    for t in tensors:
        if t.dtype != want:
            raise TypeError(f"tensor dtype {t.dtype} does not match the plan's {want}")
        if not t.is_cuda:
            raise RuntimeError("tensors must live on a CUDA device: this library has no CPU path")
