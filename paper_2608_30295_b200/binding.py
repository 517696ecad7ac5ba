"""ctypes binding of libcatekv.so: argument marshalling only.

Every step of the hot path runs in the library's CUDA kernels; PyTorch is used
here for device memory and the current stream.  The entry points carry the
names of the C ABI (include/catekv.h).  There is no CPU fallback: importing
this module without the built library raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# CATEKV_LIBRARY selects another build of the same library (the checked build, libcatekv_checked.so)
LIB_PATH = os.environ.get("CATEKV_LIBRARY") or os.path.join(_HERE, "libcatekv.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_CAPACITY, ERR_WORKSPACE, ERR_CUDA, ERR_DEVICE = 0, -1, -2, -3, -4, -5, -6
STATUS_BYTES = 256
STATUS_WAIT_EXPIRED, STATUS_CAPACITY, STATUS_INDEX_RANGE = 1, 2, 4
POOL_NONE, POOL_CHUNK, POOL_SLIDING = 0, 1, 2
OUT_BF16, OUT_FP32 = 0, 1
SEG_ALIGN = 128


class CatekvError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = _lib.catekv_error_string(code).decode()
        if code == ERR_CUDA:
            msg += f" (cudaError {_lib.catekv_last_cuda_error()})"
        super().__init__(f"{where}: {msg} [{code}]")


class PagesStruct(C.Structure):
    _fields_ = [("max_pages", C.c_int32), ("n_pages", C.c_int32), ("next_free", C.c_int32), ("reserved", C.c_int32),
                ("k_ovf", C.c_void_p), ("v_ovf", C.c_void_p), ("table_dev", C.c_void_p), ("table", C.c_void_p),
                ("seg_pages", C.c_void_p), ("seg_cap_dev", C.c_void_p)]


class CacheStruct(C.Structure):
    _fields_ = [("B", C.c_int32), ("Hkv", C.c_int32), ("d", C.c_int32), ("reserved", C.c_int32),
                ("total_rows", C.c_int64), ("k_pool", C.c_void_p), ("v_pool", C.c_void_p),
                ("seg_off_dev", C.c_void_p), ("seg_len_dev", C.c_void_p),
                ("seg_off", C.c_void_p), ("seg_cap", C.c_void_p), ("seg_len", C.c_void_p),
                ("pages", C.POINTER(PagesStruct)), ("seg_cap_dev", C.c_void_p)]


class StatusStruct(C.Structure):
    _fields_ = [("flags", C.c_int32), ("kernel", C.c_int32), ("segment", C.c_int32), ("index", C.c_int32)]


PAGE_ROWS = 64


class SelectParams(C.Structure):
    _fields_ = [("B", C.c_int32), ("Hq", C.c_int32), ("Hkv", C.c_int32), ("d", C.c_int32),
                ("L_obs", C.c_int32), ("sink", C.c_int32), ("local", C.c_int32), ("budget_consistent", C.c_int32),
                ("eta_adaptive", C.c_float), ("pool_mode", C.c_int32), ("pool_param", C.c_int32),
                ("reserved", C.c_int32),
                ("q_win", C.c_void_p), ("k", C.c_void_p), ("v", C.c_void_p),
                ("kv_stride_b", C.c_int64), ("kv_stride_h", C.c_int64), ("kv_stride_t", C.c_int64),
                ("seq_len", C.c_void_p), ("head_mask", C.c_void_p), ("row_lse_scored", C.c_void_p)]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2608_30295_b200.build` "
                          "(there is no fallback path)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, f32, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_float, C.c_size_t
    sig = {
        "catekv_version": (C.c_int, []),
        "catekv_error_string": (C.c_char_p, [C.c_int]),
        "catekv_last_cuda_error": (C.c_int, []),
        "catekv_cache_layout": (C.c_int, [i32, i32, vp, i32, vp, vp, C.POINTER(i64)]),
        "catekv_head_cv_workspace_bytes": (sz, [i32, i32, i32, i32, i32, i32, i32]),
        "catekv_head_cv": (C.c_int, [vp, vp, i64, i64, i64, vp, i32, i32, i32, i32, i32, i32, i32, f32, f32, i32,
                                     vp, vp, sz, vp]),
        "catekv_classify_heads": (C.c_int, [vp, i32, i32, f32, vp]),
        "catekv_select_workspace_bytes": (sz, [i32, i32, i32, i32, i32]),
        "catekv_select_compact": (C.c_int, [C.POINTER(SelectParams), C.POINTER(CacheStruct), vp, i64, vp, sz, vp]),
        "catekv_append": (C.c_int, [C.POINTER(CacheStruct), vp, vp, vp]),
        "catekv_cache_advance": (C.c_int, [C.POINTER(CacheStruct), i32]),
        "catekv_cache_regrow": (C.c_int, [C.POINTER(CacheStruct), C.POINTER(CacheStruct), vp]),
        "catekv_pages_reserve": (C.c_int, [C.POINTER(CacheStruct), i32, vp]),
        "catekv_decode_num_ctas": (C.c_int, []),
        "catekv_decode_plan_bytes": (sz, [i32, i32, i32]),
        "catekv_decode_workspace_bytes": (sz, [i32, i32, i32]),
        "catekv_decode_plan": (C.c_int, [C.POINTER(CacheStruct), i32, vp, vp, sz, vp]),
        "catekv_decode_attn": (C.c_int, [C.POINTER(CacheStruct), vp, i32, f32, vp, i32, vp, vp, vp, sz, vp, sz, vp]),
        "catekv_decode_partials": (C.c_int, [C.POINTER(CacheStruct), vp, i32, f32, vp, i32, vp, vp, vp, sz, vp, sz, vp]),
        "catekv_decode_combine": (C.c_int, [C.POINTER(CacheStruct), vp, i32, f32, vp, i32, vp, vp, vp, sz, vp, sz, vp]),
        "catekv_append_decode_attn": (C.c_int, [C.POINTER(CacheStruct), vp, vp, vp, i32, f32, vp, i32, vp, vp, vp, sz,
                                                vp, sz, vp]),
        "catekv_attention_recall": (C.c_int, [vp, vp, vp, i32, vp]),
        "catekv_retrieval_meta_bytes": (sz, [C.POINTER(CacheStruct), i32]),
        "catekv_retrieval_build": (C.c_int, [C.POINTER(CacheStruct), i32, vp, vp]),
        "catekv_retrieval_append": (C.c_int, [C.POINTER(CacheStruct), i32, vp, vp, vp]),
        "catekv_append_retrieval": (C.c_int, [C.POINTER(CacheStruct), vp, vp, i32, vp, vp]),
        "catekv_retrieve_workspace_bytes": (sz, [i32, i32, i32]),
        "catekv_retrieve_compact": (C.c_int, [C.POINTER(CacheStruct), vp, i32, vp, i32, vp, i32, i32, i32,
                                              C.POINTER(CacheStruct), vp, i64, vp, sz, vp]),
        "catekv_retrieve_select": (C.c_int, [C.POINTER(CacheStruct), vp, i32, vp, i32, vp, i32, i32, i32, vp, i64, vp,
                                             vp, sz, vp]),
        "catekv_retrieve_lengths": (C.c_int, [C.POINTER(CacheStruct), i32, vp, i32, i32, i32, vp]),
        "catekv_decode_attn_indexed": (C.c_int, [C.POINTER(CacheStruct), vp, i64, vp, vp, i32, f32, vp, i32, vp, vp, vp,
                                                 sz, vp, sz, vp]),
        "catekv_decode_attn_noalloc": (C.c_int, [C.POINTER(CacheStruct), vp, i32, f32, vp, i32, vp, vp, vp, sz, vp]),
        "catekv_workspace_status": (C.c_int, [vp, C.POINTER(StatusStruct), i32, vp]),
        "catekv_checked_build": (C.c_int, []),
        "catekv_checked_status": (C.c_int, [C.POINTER(StatusStruct), i32]),
        "catekv_test_expire_score_waits": (None, [i32]),
        "catekv_cache_sync_lengths": (C.c_int, [C.POINTER(CacheStruct), vp]),
        "catekv_window_attn_workspace_bytes": (sz, [i32, i32, i32, i32, i32]),
        "catekv_window_attn": (C.c_int, [vp, vp, vp, i64, i64, i64, vp, i32, i32, i32, i32, i32, vp, i32, vp, vp, vp, sz, vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    return lib, tuple(sig)


_lib, EXPORTS = _load()


def _check(rc: int, where: str):
    if rc != OK:
        raise CatekvError(rc, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _np_ptr(a: np.ndarray) -> int:
    return a.ctypes.data


def _dev_ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def catekv_version() -> int:
    return _lib.catekv_version()


def catekv_cache_layout(B: int, Hkv: int, len0, max_new: int):
    """-> (seg_off int32[B*Hkv], seg_cap int32[B*Hkv], total_rows)."""
    len0 = np.ascontiguousarray(len0, dtype=np.int32).reshape(-1)
    off = np.zeros(B * Hkv, dtype=np.int32)
    cap = np.zeros(B * Hkv, dtype=np.int32)
    total = C.c_int64(0)
    _check(_lib.catekv_cache_layout(B, Hkv, _np_ptr(len0), max_new, _np_ptr(off), _np_ptr(cap), C.byref(total)),
           "catekv_cache_layout")
    return off, cap, int(total.value)


class Cache:
    """Device pools and segment tables of one layer's hybrid cache (memory only)."""

    def __init__(self, B: int, Hkv: int, len0, max_new: int, device="cuda", d: int = 128):
        self.B, self.Hkv, self.d = B, Hkv, d
        self.seg_off, self.seg_cap, self.total_rows = catekv_cache_layout(B, Hkv, len0, max_new)
        self.seg_len = np.zeros(B * Hkv, dtype=np.int32)
        self.device = torch.device(device)
        rows = max(self.total_rows, 1)
        self.k_pool = torch.empty((rows, d), dtype=torch.bfloat16, device=device)
        self.v_pool = torch.empty((rows, d), dtype=torch.bfloat16, device=device)
        self.seg_off_dev = torch.from_numpy(self.seg_off).to(device)
        self.seg_len_dev = torch.zeros(B * Hkv, dtype=torch.int32, device=device)
        self.seg_cap_dev = torch.from_numpy(self.seg_cap).to(device)
        self.struct = CacheStruct(B, Hkv, d, 0, self.total_rows, self.k_pool.data_ptr(), self.v_pool.data_ptr(),
                                  self.seg_off_dev.data_ptr(), self.seg_len_dev.data_ptr(),
                                  _np_ptr(self.seg_off), _np_ptr(self.seg_cap), _np_ptr(self.seg_len), None,
                                  self.seg_cap_dev.data_ptr())
        self.pages = None

    def attach_pages(self, n_pages: int, max_pages: int) -> "Pages":
        """Give the cache overflow pools of n_pages pages of 64 rows (memory only; catekv_pages_reserve hands
        the pages out).  The segments keep what they hold."""
        self.pages = Pages(self, n_pages, max_pages)
        self.struct.pages = C.pointer(self.pages.struct)
        return self.pages

    def set_lengths(self, lens):
        """Set host mirror and device lengths (used when rows are written by the caller)."""
        self.seg_len[:] = np.asarray(lens, dtype=np.int32).reshape(-1)
        self.seg_len_dev.copy_(torch.from_numpy(self.seg_len))

    def kept_rows(self) -> int:
        return int(self.seg_len.sum())


class Pages:
    """Overflow pools, page table (device + host mirror) and per-segment page counts of one cache (memory only)."""

    def __init__(self, cache: Cache, n_pages: int, max_pages: int):
        n = cache.B * cache.Hkv
        self.k_ovf = torch.empty((max(n_pages, 1) * PAGE_ROWS, cache.d), dtype=torch.bfloat16, device=cache.device)
        self.v_ovf = torch.empty_like(self.k_ovf)
        self.table = np.full((n, max_pages), -1, dtype=np.int32)
        self.table_dev = torch.full((n, max_pages), -1, dtype=torch.int32, device=cache.device)
        self.seg_pages = np.zeros(n, dtype=np.int32)
        self.seg_cap_dev = cache.seg_cap_dev
        self.struct = PagesStruct(max_pages, n_pages, 0, 0, self.k_ovf.data_ptr(), self.v_ovf.data_ptr(),
                                  self.table_dev.data_ptr(), _np_ptr(self.table), _np_ptr(self.seg_pages),
                                  self.seg_cap_dev.data_ptr())


def catekv_append(cache: Cache, k_new: torch.Tensor, v_new: torch.Tensor):
    assert k_new.is_contiguous() and v_new.is_contiguous()
    _check(_lib.catekv_append(C.byref(cache.struct), k_new.data_ptr(), v_new.data_ptr(), _stream()), "catekv_append")


def catekv_cache_sync_lengths(cache: Cache):
    """Fetch the device's segment lengths into the host mirror (synchronises the current stream)."""
    _check(_lib.catekv_cache_sync_lengths(C.byref(cache.struct), _stream()), "catekv_cache_sync_lengths")


def catekv_workspace_status(ws: torch.Tensor, clear: bool = False, raise_on_error: bool = True) -> dict:
    """Read the status block at the start of a select / head_cv / retrieval workspace (synchronises the current
    stream).  -> {"flags", "kernel", "segment", "index"}; raises CatekvError(ERR_DEVICE) when a flag is set."""
    st = StatusStruct()
    rc = _lib.catekv_workspace_status(ws.data_ptr(), C.byref(st), 1 if clear else 0, _stream())
    if rc != OK and (raise_on_error or rc != ERR_DEVICE):
        raise CatekvError(rc, "catekv_workspace_status")
    return {"flags": st.flags, "kernel": st.kernel, "segment": st.segment, "index": st.index}


def catekv_checked_build() -> bool:
    return bool(_lib.catekv_checked_build())


def catekv_checked_status(clear: bool = False) -> dict:
    """Checked build only: the library's own status block (device-wide synchronisation); never raises on flags."""
    st = StatusStruct()
    rc = _lib.catekv_checked_status(C.byref(st), 1 if clear else 0)
    if rc not in (OK, ERR_DEVICE):
        raise CatekvError(rc, "catekv_checked_status")
    return {"flags": st.flags, "kernel": st.kernel, "segment": st.segment, "index": st.index}


def catekv_test_expire_score_waits(n_launches: int):
    """Test hook: the next n_launches scoring launches run with an idle producer lane and a 512-poll wait limit."""
    _lib.catekv_test_expire_score_waits(int(n_launches))


def retrieve_workspace(cache: Cache) -> torch.Tensor:
    """A retrieval workspace for `cache` with its status block zeroed (memory only)."""
    ws = torch.empty(_lib.catekv_retrieve_workspace_bytes(cache.B, cache.Hkv, int(cache.seg_cap.max())),
                     dtype=torch.uint8, device=cache.device)
    ws[:STATUS_BYTES].zero_()
    return ws


def catekv_cache_advance(cache: Cache, n_tokens: int = 1):
    """Host mirror only: account for appends that a replayed CUDA graph performs on the device."""
    _check(_lib.catekv_cache_advance(C.byref(cache.struct), n_tokens), "catekv_cache_advance")


def catekv_pages_reserve(cache: Cache, n_new: int):
    """Make sure every segment can take n_new more rows (hands out overflow pages where the capacity is short)."""
    _check(_lib.catekv_pages_reserve(C.byref(cache.struct), n_new, _stream()), "catekv_pages_reserve")


def catekv_cache_regrow(src: Cache, max_new: int) -> Cache:
    """A new cache with room for max_new more rows per segment, holding src's rows (device copy)."""
    dst = Cache(src.B, src.Hkv, src.seg_len, max_new, src.device, src.d)
    _check(_lib.catekv_cache_regrow(C.byref(src.struct), C.byref(dst.struct), _stream()), "catekv_cache_regrow")
    return dst


def catekv_decode_num_ctas() -> int:
    n = _lib.catekv_decode_num_ctas()
    if n < 0:
        raise CatekvError(n, "catekv_decode_num_ctas")
    return n


class DecodePlan:
    """Plan and workspace buffers of catekv_decode_attn for one cache (memory only)."""

    def __init__(self, cache: Cache, num_ctas: int):
        self.num_ctas = num_ctas
        self.bytes = _lib.catekv_decode_plan_bytes(cache.B, cache.Hkv, num_ctas)
        self.host = torch.empty(self.bytes, dtype=torch.uint8).pin_memory()
        self.dev = torch.empty(self.bytes, dtype=torch.uint8, device=cache.device)
        self.ws_bytes = _lib.catekv_decode_workspace_bytes(cache.B, cache.Hkv, num_ctas)
        self.ws = torch.empty(self.ws_bytes, dtype=torch.uint8, device=cache.device)


def catekv_decode_plan(cache: Cache, plan: DecodePlan):
    _check(_lib.catekv_decode_plan(C.byref(cache.struct), plan.num_ctas, plan.host.data_ptr(), plan.dev.data_ptr(),
                                   plan.bytes, _stream()), "catekv_decode_plan")


def plan_header(plan: DecodePlan) -> dict:
    h = plan.host[:48].numpy().view(np.int32)
    return {"num_ctas": int(h[1]), "n_segs": int(h[2]), "n_items": int(h[3]), "n_slots": int(h[4]),
            "tile": int(h[5]), "total_rows": int(plan.host[24:32].numpy().view(np.int64)[0]),
            "max_pieces": int(h[11])}


def _decode_call(fn, name, cache, q, plan, out, lse_out, sm_scale):
    assert q.is_contiguous() and out.is_contiguous() and q.dtype == torch.bfloat16
    Hq = q.shape[1]
    if out.dtype == torch.bfloat16:
        od = OUT_BF16
    elif out.dtype == torch.float32:
        od = OUT_FP32
    else:
        raise TypeError("out must be bf16 or fp32")
    _check(fn(C.byref(cache.struct), q.data_ptr(), Hq, sm_scale, out.data_ptr(), od, _dev_ptr(lse_out),
              plan.host.data_ptr(), plan.dev.data_ptr(), plan.bytes, plan.ws.data_ptr(), plan.ws_bytes, _stream()), name)


def catekv_decode_attn(cache: Cache, q: torch.Tensor, plan: DecodePlan, out: torch.Tensor,
                       lse_out: Optional[torch.Tensor] = None, sm_scale: float = 0.0):
    _decode_call(_lib.catekv_decode_attn, "catekv_decode_attn", cache, q, plan, out, lse_out, sm_scale)


def catekv_decode_partials(cache: Cache, q: torch.Tensor, plan: DecodePlan, out: torch.Tensor,
                           lse_out: Optional[torch.Tensor] = None, sm_scale: float = 0.0):
    _decode_call(_lib.catekv_decode_partials, "catekv_decode_partials", cache, q, plan, out, lse_out, sm_scale)


def catekv_decode_combine(cache: Cache, q: torch.Tensor, plan: DecodePlan, out: torch.Tensor,
                          lse_out: Optional[torch.Tensor] = None, sm_scale: float = 0.0):
    _decode_call(_lib.catekv_decode_combine, "catekv_decode_combine", cache, q, plan, out, lse_out, sm_scale)


def catekv_append_decode_attn(cache: Cache, k_new: torch.Tensor, v_new: torch.Tensor, q: torch.Tensor,
                              plan: DecodePlan, out: torch.Tensor, lse_out: Optional[torch.Tensor] = None,
                              sm_scale: float = 0.0):
    assert q.is_contiguous() and out.is_contiguous() and k_new.is_contiguous() and v_new.is_contiguous()
    od = OUT_BF16 if out.dtype == torch.bfloat16 else OUT_FP32
    assert out.dtype in (torch.bfloat16, torch.float32) and q.dtype == torch.bfloat16
    _check(_lib.catekv_append_decode_attn(C.byref(cache.struct), k_new.data_ptr(), v_new.data_ptr(), q.data_ptr(),
                                          q.shape[1], sm_scale, out.data_ptr(), od, _dev_ptr(lse_out),
                                          plan.host.data_ptr(), plan.dev.data_ptr(), plan.bytes, plan.ws.data_ptr(),
                                          plan.ws_bytes, _stream()), "catekv_append_decode_attn")


def catekv_attention_recall(lse_kept: torch.Tensor, lse_full: torch.Tensor) -> torch.Tensor:
    """-> recall float32, same shape: exp(lse_kept - lse_full), computed on the device."""
    assert lse_kept.is_contiguous() and lse_full.is_contiguous() and lse_kept.shape == lse_full.shape
    assert lse_kept.dtype == torch.float32 and lse_full.dtype == torch.float32
    out = torch.empty_like(lse_kept)
    _check(_lib.catekv_attention_recall(lse_kept.data_ptr(), lse_full.data_ptr(), out.data_ptr(), lse_kept.numel(),
                                        _stream()), "catekv_attention_recall")
    return out


def catekv_retrieval_meta(cache: Cache, chunk_size: int) -> torch.Tensor:
    """An uninitialised metadata buffer of the right size for `cache` (memory only)."""
    n = _lib.catekv_retrieval_meta_bytes(C.byref(cache.struct), chunk_size)
    if n == 0:
        raise CatekvError(ERR_UNSUPPORTED, "catekv_retrieval_meta_bytes")
    return torch.empty(n, dtype=torch.uint8, device=cache.device)


def catekv_retrieval_build(cache: Cache, chunk_size: int, meta: torch.Tensor):
    _check(_lib.catekv_retrieval_build(C.byref(cache.struct), chunk_size, meta.data_ptr(), _stream()),
           "catekv_retrieval_build")


def catekv_retrieval_append(cache: Cache, chunk_size: int, k_new: torch.Tensor, meta: torch.Tensor):
    assert k_new.is_contiguous()
    _check(_lib.catekv_retrieval_append(C.byref(cache.struct), chunk_size, k_new.data_ptr(), meta.data_ptr(), _stream()),
           "catekv_retrieval_append")


def catekv_retrieve_compact(cache: Cache, meta: torch.Tensor, chunk_size: int, q: torch.Tensor, retrieval_mask,
                            budget: int, sink: int, local: int, step_cache: Cache,
                            idx_out: Optional[torch.Tensor] = None, ws: Optional[torch.Tensor] = None):
    assert q.is_contiguous() and q.dtype == torch.bfloat16
    retrieval_mask = np.ascontiguousarray(retrieval_mask, dtype=np.uint8).reshape(-1)
    if ws is None:
        ws = retrieve_workspace(cache)
    stride = 0 if idx_out is None else idx_out.stride(0)
    _check(_lib.catekv_retrieve_compact(C.byref(cache.struct), meta.data_ptr(), chunk_size, q.data_ptr(), q.shape[1],
                                        _np_ptr(retrieval_mask), budget, sink, local, C.byref(step_cache.struct),
                                        _dev_ptr(idx_out), stride, ws.data_ptr(), ws.numel(), _stream()),
           "catekv_retrieve_compact")
    return ws


def catekv_append_retrieval(cache: Cache, k_new: torch.Tensor, v_new: torch.Tensor, chunk_size: int,
                            meta: torch.Tensor):
    assert k_new.is_contiguous() and v_new.is_contiguous()
    _check(_lib.catekv_append_retrieval(C.byref(cache.struct), k_new.data_ptr(), v_new.data_ptr(), chunk_size,
                                        meta.data_ptr(), _stream()), "catekv_append_retrieval")


def catekv_retrieve_lengths(cache: Cache, chunk_size: int, retrieval_mask, budget: int, sink: int, local: int):
    """Host only: rows every segment is attended over under query-aware retrieval with these parameters."""
    retrieval_mask = np.ascontiguousarray(retrieval_mask, dtype=np.uint8).reshape(-1)
    lens = np.zeros(cache.B * cache.Hkv, dtype=np.int32)
    _check(_lib.catekv_retrieve_lengths(C.byref(cache.struct), chunk_size, _np_ptr(retrieval_mask), budget, sink,
                                        local, _np_ptr(lens)), "catekv_retrieve_lengths")
    return lens


class CacheView:
    """The pools, offsets and capacities of `cache` under other host lengths: what catekv_decode_plan needs to
    plan catekv_decode_attn_indexed (lens = catekv_retrieve_lengths).  Memory only; shares the device arrays."""

    def __init__(self, cache: Cache, lens):
        self.B, self.Hkv, self.d, self.device = cache.B, cache.Hkv, cache.d, cache.device
        self.base = cache
        self.seg_off, self.seg_cap = cache.seg_off, cache.seg_cap
        self.seg_len = np.ascontiguousarray(lens, dtype=np.int32).reshape(-1).copy()
        b = cache.struct
        self.struct = CacheStruct(b.B, b.Hkv, b.d, 0, b.total_rows, b.k_pool, b.v_pool, b.seg_off_dev, b.seg_len_dev,
                                  b.seg_off, b.seg_cap, _np_ptr(self.seg_len), None, b.seg_cap_dev)


def catekv_retrieve_select(cache: Cache, meta: torch.Tensor, chunk_size: int, q: torch.Tensor, retrieval_mask,
                           budget: int, sink: int, local: int, idx: torch.Tensor, sel_len: torch.Tensor,
                           ws: Optional[torch.Tensor] = None):
    assert q.is_contiguous() and q.dtype == torch.bfloat16
    assert idx.dtype == torch.int32 and sel_len.dtype == torch.int32 and idx.stride(1) == 1
    retrieval_mask = np.ascontiguousarray(retrieval_mask, dtype=np.uint8).reshape(-1)
    if ws is None:
        ws = retrieve_workspace(cache)
    _check(_lib.catekv_retrieve_select(C.byref(cache.struct), meta.data_ptr(), chunk_size, q.data_ptr(), q.shape[1],
                                       _np_ptr(retrieval_mask), budget, sink, local, idx.data_ptr(), idx.stride(0),
                                       sel_len.data_ptr(), ws.data_ptr(), ws.numel(), _stream()),
           "catekv_retrieve_select")
    return ws


def catekv_decode_attn_indexed(cache: Cache, idx: torch.Tensor, sel_len: torch.Tensor, q: torch.Tensor,
                               plan: DecodePlan, out: torch.Tensor, lse_out: Optional[torch.Tensor] = None,
                               sm_scale: float = 0.0):
    assert q.is_contiguous() and out.is_contiguous() and q.dtype == torch.bfloat16
    assert idx.dtype == torch.int32 and sel_len.dtype == torch.int32 and idx.stride(1) == 1
    if out.dtype == torch.bfloat16:
        od = OUT_BF16
    elif out.dtype == torch.float32:
        od = OUT_FP32
    else:
        raise TypeError("out must be bf16 or fp32")
    _check(_lib.catekv_decode_attn_indexed(C.byref(cache.struct), idx.data_ptr(), idx.stride(0), sel_len.data_ptr(),
                                           q.data_ptr(), q.shape[1], sm_scale, out.data_ptr(), od, _dev_ptr(lse_out),
                                           plan.host.data_ptr(), plan.dev.data_ptr(), plan.bytes, plan.ws.data_ptr(),
                                           plan.ws_bytes, _stream()), "catekv_decode_attn_indexed")


NOALLOC_SCRATCH_BYTES = 4 << 20


def catekv_decode_attn_noalloc(cache: Cache, q: torch.Tensor, plan: DecodePlan, out: torch.Tensor,
                               lse_out: Optional[torch.Tensor] = None, sm_scale: float = 0.0):
    """catekv_decode_attn with the partials in the library's own fixed 4 MiB array instead of plan.ws: for
    callers that may not allocate device memory (a host that owns the whole GPU arena, or a request path that
    cannot afford cudaMalloc's device-wide synchronisation).  Nothing is allocated by this call; plans with
    more than 1016 partial slots are refused (ERR_WORKSPACE).  Calls share the array: keep them ordered."""
    assert q.is_contiguous() and out.is_contiguous() and q.dtype == torch.bfloat16
    if out.dtype == torch.bfloat16:
        od = OUT_BF16
    elif out.dtype == torch.float32:
        od = OUT_FP32
    else:
        raise TypeError("out must be bf16 or fp32")
    _check(_lib.catekv_decode_attn_noalloc(C.byref(cache.struct), q.data_ptr(), q.shape[1], sm_scale,
                                           out.data_ptr(), od, _dev_ptr(lse_out), plan.host.data_ptr(),
                                           plan.dev.data_ptr(), plan.bytes, _stream()), "catekv_decode_attn_noalloc")


def catekv_select_workspace_bytes(B, Hq, Hkv, n_max, L_obs) -> int:
    return _lib.catekv_select_workspace_bytes(B, Hq, Hkv, n_max, L_obs)


def catekv_select_compact(q_win: torch.Tensor, k: torch.Tensor, v: torch.Tensor, seq_len, head_mask, cache: Cache,
                          budget_consistent: int, eta_adaptive: float, sink: int, local: int, pool_mode: int,
                          pool_param: int, ws: Optional[torch.Tensor] = None,
                          idx_out: Optional[torch.Tensor] = None, row_lse_scored: Optional[torch.Tensor] = None):
    """q_win [B,Hq,L_obs,d] bf16 contiguous; k, v [B,Hkv,n_max,d] bf16 (any strides, d contiguous).
    row_lse_scored: float32 [B,Hq,L_obs] from catekv_window_attn (the call then skips its first pass over K)."""
    B, Hq, L_obs, d = q_win.shape
    Hkv, n_max = k.shape[1], k.shape[2]
    assert q_win.is_contiguous() and k.stride(3) == 1 and v.stride() == k.stride()
    seq_len = np.ascontiguousarray(seq_len, dtype=np.int32).reshape(-1)
    head_mask = np.ascontiguousarray(head_mask, dtype=np.uint8).reshape(-1)
    if ws is None:
        ws = torch.empty(catekv_select_workspace_bytes(B, Hq, Hkv, n_max, L_obs), dtype=torch.uint8, device=k.device)
    p = SelectParams(B, Hq, Hkv, d, L_obs, sink, local, budget_consistent, eta_adaptive, pool_mode, pool_param, 0,
                     q_win.data_ptr(), k.data_ptr(), v.data_ptr(), k.stride(0), k.stride(1), k.stride(2),
                     _np_ptr(seq_len), _np_ptr(head_mask), _dev_ptr(row_lse_scored))
    if row_lse_scored is not None:
        assert row_lse_scored.dtype == torch.float32 and row_lse_scored.is_contiguous()
        assert tuple(row_lse_scored.shape) == (B, Hq, L_obs)
    stride = 0 if idx_out is None else idx_out.stride(0)
    _check(_lib.catekv_select_compact(C.byref(p), C.byref(cache.struct), _dev_ptr(idx_out), stride, ws.data_ptr(),
                                      ws.numel(), _stream()), "catekv_select_compact")
    return ws


def catekv_window_attn(q_win: torch.Tensor, k: torch.Tensor, v: torch.Tensor, seq_len, out_dtype=torch.float32,
                       ws: Optional[torch.Tensor] = None):
    """-> (out [B,Hq,L_obs,d], lse [B,Hq,L_obs], lse_scored [B,Hq,L_obs]) on the device: the causal attention rows of
    the last L_obs queries, their log-sum-exp, and the log-sum-exp over the scored keys [0, n - L_obs) alone."""
    B, Hq, L_obs, d = q_win.shape
    Hkv, n_max = k.shape[1], k.shape[2]
    assert q_win.is_contiguous() and k.stride(3) == 1 and v.stride() == k.stride()
    seq_len = np.ascontiguousarray(seq_len, dtype=np.int32).reshape(-1)
    if ws is None:
        ws = torch.empty(_lib.catekv_window_attn_workspace_bytes(B, Hq, Hkv, n_max, L_obs), dtype=torch.uint8,
                         device=k.device)
    out = torch.empty((B, Hq, L_obs, d), dtype=out_dtype, device=k.device)
    lse = torch.empty((B, Hq, L_obs), dtype=torch.float32, device=k.device)
    lse_scored = torch.empty_like(lse)
    od = OUT_BF16 if out_dtype == torch.bfloat16 else OUT_FP32
    assert out_dtype in (torch.bfloat16, torch.float32)
    _check(_lib.catekv_window_attn(q_win.data_ptr(), k.data_ptr(), v.data_ptr(), k.stride(0), k.stride(1), k.stride(2),
                                   _np_ptr(seq_len), B, Hq, Hkv, d, L_obs, out.data_ptr(), od, lse.data_ptr(),
                                   lse_scored.data_ptr(), ws.data_ptr(), ws.numel(), _stream()), "catekv_window_attn")
    return out, lse, lse_scored


def catekv_head_cv_workspace_bytes(B, Hq, Hkv, n_max, L_obs, L_init, L_rec) -> int:
    return _lib.catekv_head_cv_workspace_bytes(B, Hq, Hkv, n_max, L_obs, L_init, L_rec)


def catekv_head_cv(q_win: torch.Tensor, k: torch.Tensor, seq_len, L_init: int, L_rec: int, quantile_k: float,
                   alpha: float, causal: bool, ws: Optional[torch.Tensor] = None) -> torch.Tensor:
    """-> cv float32 [B, Hkv] on the device."""
    B, Hq, L_obs, d = q_win.shape
    Hkv, n_max = k.shape[1], k.shape[2]
    assert q_win.is_contiguous() and k.stride(3) == 1
    seq_len = np.ascontiguousarray(seq_len, dtype=np.int32).reshape(-1)
    if ws is None:
        ws = torch.empty(catekv_head_cv_workspace_bytes(B, Hq, Hkv, n_max, L_obs, L_init, L_rec), dtype=torch.uint8,
                         device=k.device)
    cv = torch.empty((B, Hkv), dtype=torch.float32, device=k.device)
    _check(_lib.catekv_head_cv(q_win.data_ptr(), k.data_ptr(), k.stride(0), k.stride(1), k.stride(2),
                               _np_ptr(seq_len), B, Hq, Hkv, d, L_obs, L_init, L_rec, quantile_k, alpha,
                               1 if causal else 0, cv.data_ptr(), ws.data_ptr(), ws.numel(), _stream()),
           "catekv_head_cv")
    return cv


def catekv_classify_heads(cv, r: float) -> np.ndarray:
    cv = np.ascontiguousarray(cv, dtype=np.float32)
    n_samples, n_heads = cv.shape
    mask = np.zeros(n_heads, dtype=np.uint8)
    _check(_lib.catekv_classify_heads(_np_ptr(cv), n_samples, n_heads, r, _np_ptr(mask)), "catekv_classify_heads")
    return mask
