"""Thin ctypes binding over ``libenl.so``: same names as the C ABI, argument marshalling only.

Every step of the path (page scatter, gather plan upload, attention, split merge) runs inside the
library; nothing here computes.  There is no fallback: if the library is missing, loading raises.
Tensors are torch CUDA tensors (device memory and streams are torch's); index lists are host arrays.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libenl.so")

ENL_BF16 = 1
ENL_DEVICE_NONE = -1
ENL_REPLACE, ENL_APPEND = 0, 1
ENL_PLAN_ONLY, ENL_MASS_ONLY = 1, 2
ENL_OK, ENL_E_INVAL, ENL_E_NOGROUP, ENL_E_NOMEM, ENL_E_CUDA, ENL_E_TIMEOUT, ENL_E_LIMIT, ENL_E_EVICTED, ENL_E_CORRUPT = 0, -1, -2, -3, -4, -5, -6, -8, -9
ENL_STATIC_MAX_SEGMENTS, ENL_STATIC_MAX_KEYS, ENL_STATIC_SCRATCH_BYTES = 255, 65536, 4 << 20

EXPORTS = ("enl_cache_create", "enl_group_store", "enl_attend", "enl_cache_free", "enl_strerror",
           "enl_group_store_all_layers", "enl_group_len", "enl_cache_status", "enl_cache_selfcheck", "enl_plan_inspect", "enl_attend_static", "enl_cluster_assign",
           "enl_cluster_assign_sums", "enl_select_knapsack", "enl_rope_rotate", "enl_tier_enable", "enl_group_evict", "enl_step_prepare", "enl_group_resident")


class CacheDesc(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("page_tokens", ctypes.c_int32), ("max_groups", ctypes.c_int32),
                ("max_tokens", ctypes.c_int64), ("dtype", ctypes.c_int32), ("device", ctypes.c_int32),
                ("max_batch", ctypes.c_int32), ("max_q_tokens", ctypes.c_int32), ("scratch_bytes", ctypes.c_int64)]


class AttendArgs(ctypes.Structure):
    _fields_ = [("layer", ctypes.c_int32), ("batch", ctypes.c_int32),
                ("sel_ids", ctypes.c_void_p), ("cu_sel", ctypes.c_void_p), ("cu_q", ctypes.c_void_p),
                ("cu_new", ctypes.c_void_p),
                ("n_sel", ctypes.c_int32), ("n_q", ctypes.c_int32), ("n_new", ctypes.c_int32),
                ("q", ctypes.c_void_p), ("k_new", ctypes.c_void_p), ("v_new", ctypes.c_void_p),
                ("out", ctypes.c_void_p), ("group_mass", ctypes.c_void_p), ("mass_stride", ctypes.c_int32),
                ("sel_off_out", ctypes.c_void_p), ("split_hint", ctypes.c_int32), ("flags", ctypes.c_uint32),
                ("group_mass_sum", ctypes.c_void_p), ("sum_stride", ctypes.c_int32), ("n_obj", ctypes.c_int32),
                ("obj_off", ctypes.c_void_p)]


class StaticArgs(ctypes.Structure):
    _fields_ = [("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("n_seg", ctypes.c_int32), ("seg_len", ctypes.c_void_p), ("n_new", ctypes.c_int32),
                ("q", ctypes.c_void_p), ("k", ctypes.c_void_p), ("v", ctypes.c_void_p), ("out", ctypes.c_void_p),
                ("group_mass", ctypes.c_void_p)]


class ClusterArgs(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int32), ("mass", ctypes.c_void_p), ("n_q", ctypes.c_int32),
                ("n_q_heads", ctypes.c_int32), ("mass_stride", ctypes.c_int32), ("n_groups", ctypes.c_int32),
                ("n_obj", ctypes.c_int32), ("obj_off", ctypes.c_void_p), ("threshold", ctypes.c_float),
                ("avg", ctypes.c_void_p), ("assign", ctypes.c_void_p)]


class PrepareStats(ctypes.Structure):
    _fields_ = [("n_hit", ctypes.c_int32), ("n_miss", ctypes.c_int32), ("n_evicted", ctypes.c_int32),
                ("bytes_h2d", ctypes.c_int64), ("bytes_d2h", ctypes.c_int64)]


class EnlError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {strerror(code)} ({code})")
        self.code = code


_lib = None
_n_layers = {}          # cache handle -> layer count (the all-layers store takes one pointer per layer)


def lib() -> ctypes.CDLL:
    """Loads the library (raises OSError if it has not been built: there is no other path)."""
    global _lib
    if _lib is None:
        L = ctypes.CDLL(LIB_PATH)
        L.enl_cache_create.argtypes = [ctypes.POINTER(CacheDesc), ctypes.POINTER(ctypes.c_void_p)]
        L.enl_cache_create.restype = ctypes.c_int
        L.enl_group_store.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                      ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p]
        L.enl_group_store.restype = ctypes.c_int
        L.enl_group_store_all_layers.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p,
                                                 ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p]
        L.enl_group_store_all_layers.restype = ctypes.c_int
        L.enl_attend.argtypes = [ctypes.c_void_p, ctypes.POINTER(AttendArgs), ctypes.c_void_p]
        L.enl_attend.restype = ctypes.c_int
        L.enl_cache_free.argtypes = [ctypes.c_void_p]
        L.enl_cache_free.restype = ctypes.c_int
        L.enl_strerror.argtypes = [ctypes.c_int]
        L.enl_strerror.restype = ctypes.c_char_p
        L.enl_group_len.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32]
        L.enl_group_len.restype = ctypes.c_int32
        L.enl_cache_status.argtypes = [ctypes.c_void_p]
        L.enl_cache_status.restype = ctypes.c_int
        L.enl_cache_selfcheck.argtypes = [ctypes.c_void_p]
        L.enl_cache_selfcheck.restype = ctypes.c_int
        L.enl_plan_inspect.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p,
                                       ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p,
                                       ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        L.enl_plan_inspect.restype = ctypes.c_int
        L.enl_attend_static.argtypes = [ctypes.POINTER(StaticArgs), ctypes.c_void_p]
        L.enl_attend_static.restype = ctypes.c_int
        L.enl_cluster_assign.argtypes = [ctypes.POINTER(ClusterArgs), ctypes.c_void_p]
        L.enl_cluster_assign.restype = ctypes.c_int
        L.enl_cluster_assign_sums.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p,
                                              ctypes.c_int32, ctypes.c_int32, ctypes.c_float, ctypes.c_void_p, ctypes.c_void_p,
                                              ctypes.c_void_p]
        L.enl_cluster_assign_sums.restype = ctypes.c_int
        L.enl_select_knapsack.argtypes = [ctypes.c_int32, ctypes.c_void_p, ctypes.c_float, ctypes.c_void_p,
                                          ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p]
        L.enl_select_knapsack.restype = ctypes.c_int
        L.enl_rope_rotate.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p,
                                      ctypes.c_int32, ctypes.c_double, ctypes.c_int32, ctypes.c_void_p]
        L.enl_rope_rotate.restype = ctypes.c_int
        L.enl_tier_enable.argtypes = [ctypes.c_void_p, ctypes.c_int64]
        L.enl_tier_enable.restype = ctypes.c_int
        L.enl_group_evict.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p]
        L.enl_group_evict.restype = ctypes.c_int
        L.enl_step_prepare.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p,
                                       ctypes.POINTER(PrepareStats)]
        L.enl_step_prepare.restype = ctypes.c_int
        L.enl_group_resident.argtypes = [ctypes.c_void_p, ctypes.c_int32]
        L.enl_group_resident.restype = ctypes.c_int
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().enl_strerror(int(code)).decode()


def _ptr(t) -> Optional[int]:
    return None if t is None else int(t.data_ptr())


def _i32(a) -> Optional[np.ndarray]:
    return None if a is None else np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _np_ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def enl_cache_create(n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int, max_groups: int,
                     max_tokens: int, device: int = 0, max_batch: int = 0, max_q_tokens: int = 0,
                     scratch_bytes: int = 0, page_tokens: int = 0, dtype: int = ENL_BF16) -> int:
    """Returns the opaque cache handle."""
    d = CacheDesc(n_layers, n_q_heads, n_kv_heads, head_dim, page_tokens, max_groups, max_tokens, dtype,
                  device, max_batch, max_q_tokens, scratch_bytes)
    h = ctypes.c_void_p()
    rc = lib().enl_cache_create(ctypes.byref(d), ctypes.byref(h))
    if rc != ENL_OK:
        raise EnlError(rc, "enl_cache_create")
    _n_layers[int(h.value)] = int(n_layers)
    return h.value


def enl_group_store(cache: int, group_id: int, layer: int, k, v, mode: int = ENL_REPLACE,
                    stream: int = 0, n_tokens: Optional[int] = None) -> None:
    """``k``/``v``: ``[n, Hkv, D]`` bf16 CUDA tensors (or None with ``n_tokens`` on a bookkeeping cache)."""
    n = int(k.shape[0]) if k is not None else int(n_tokens)
    rc = lib().enl_group_store(cache, group_id, layer, n, _ptr(k), _ptr(v), mode, stream or None)
    if rc != ENL_OK:
        raise EnlError(rc, "enl_group_store")


def enl_group_store_all_layers(cache: int, group_id: int, ks, vs, mode: int = ENL_REPLACE, stream: int = 0,
                               n_tokens: Optional[int] = None, n_layers: Optional[int] = None) -> None:
    """``ks``/``vs``: one ``[n, Hkv, D]`` bf16 CUDA tensor per layer (or None with ``n_tokens`` on a bookkeeping
    cache).  Every layer of the group is written by one launch."""
    if ks is None:
        n, kp, vp = int(n_tokens), None, None
    else:
        n = int(ks[0].shape[0])
        if any(int(t.shape[0]) != n for t in list(ks) + list(vs)):
            raise ValueError("every layer must bring the same number of rows")
        n_layers = _n_layers.get(int(cache), n_layers)
        if n_layers is not None and (len(ks) != n_layers or len(vs) != n_layers):
            raise ValueError("one K and one V tensor per layer of the cache")
        kp = (ctypes.c_void_p * len(ks))(*[_ptr(t) for t in ks])
        vp = (ctypes.c_void_p * len(vs))(*[_ptr(t) for t in vs])
    rc = lib().enl_group_store_all_layers(cache, group_id, n, kp, vp, mode, stream or None)
    if rc != ENL_OK:
        raise EnlError(rc, "enl_group_store_all_layers")


def enl_attend(cache: int, layer: int, sel_ids: Sequence[int], q, k_new, v_new, out, group_mass=None,
               cu_sel=None, cu_q=None, cu_new=None, n_q: Optional[int] = None, n_new: Optional[int] = None,
               mass_stride: Optional[int] = None, want_sel_off: bool = False, split_hint: int = 0,
               flags: int = 0, stream: int = 0, group_mass_sum=None, obj_off=None):
    """One attend call.  Returns ``sel_off`` (numpy int32 ``[n_sel + batch]``) when asked, else None.
    ``group_mass_sum``: fp32 CUDA tensor ``[n_obj, stride]`` the call adds per-object mass sums to, with
    ``obj_off`` the ``n_obj + 1`` row offsets of the objects."""
    sel = _i32(sel_ids)
    cs, cq, cn = _i32(cu_sel), _i32(cu_q), _i32(cu_new)
    batch = 1 if cq is None else len(cq) - 1
    nq = int(n_q) if n_q is not None else int(q.shape[0])
    nn = int(n_new) if n_new is not None else int(k_new.shape[0])
    so = np.zeros(len(sel) + batch, np.int32) if want_sel_off else None
    a = AttendArgs()
    a.layer, a.batch = layer, batch
    a.sel_ids, a.cu_sel, a.cu_q, a.cu_new = _np_ptr(sel), _np_ptr(cs), _np_ptr(cq), _np_ptr(cn)
    a.n_sel, a.n_q, a.n_new = len(sel), nq, nn
    a.q, a.k_new, a.v_new, a.out = _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out)
    a.group_mass = _ptr(group_mass)
    a.mass_stride = int(mass_stride) if mass_stride is not None else (
        int(group_mass.shape[-1]) if group_mass is not None else 0)
    a.sel_off_out = _np_ptr(so)
    a.split_hint, a.flags = split_hint, flags
    oo = _i32(obj_off)
    a.group_mass_sum = _ptr(group_mass_sum)
    a.sum_stride = int(group_mass_sum.shape[-1]) if group_mass_sum is not None else 0
    a.n_obj = (len(oo) - 1) if oo is not None else 0
    a.obj_off = _np_ptr(oo)
    rc = lib().enl_attend(cache, ctypes.byref(a), stream or None)
    if rc != ENL_OK:
        raise EnlError(rc, "enl_attend")
    return so


def enl_attend_static(seg_len: Sequence[int], n_new: int, q, k, v, out, group_mass=None, stream: int = 0) -> None:
    """One query token over contiguous caller-owned K/V, for callers that must not allocate: the library
    keeps its split-KV partials in a fixed built-in device array instead of allocated scratch.
    ``q``/``out``: ``[Hq, D]`` bf16; ``k``/``v``: ``[sum(seg_len) + n_new, Hkv, D]`` bf16;
    ``group_mass``: ``[Hq, len(seg_len) + 1]`` fp32 or None.  Calls share the built-in array, so issue
    them on one stream (or order them); sizes beyond the fixed maxima raise ``ENL_E_LIMIT``."""
    sl = _i32(seg_len)
    a = StaticArgs()
    a.n_q_heads, a.n_kv_heads, a.head_dim = int(q.shape[-2]), int(k.shape[-2]), int(q.shape[-1])
    a.n_seg, a.seg_len, a.n_new = len(sl), _np_ptr(sl) if len(sl) else None, int(n_new)
    a.q, a.k, a.v, a.out, a.group_mass = _ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(group_mass)
    rc = lib().enl_attend_static(ctypes.byref(a), stream or None)
    if rc != ENL_OK:
        raise EnlError(rc, "enl_attend_static")


def enl_cluster_assign(masses: Sequence, obj_off: Sequence[int], n_groups: int, threshold: float, avg, assign,
                       stream: int = 0) -> None:
    """``masses``: one fp32 CUDA tensor ``[n_q, Hq, stride]`` per scored layer (the group_mass of the scoring
    attend); ``avg``: fp32 ``[n_obj, n_groups]``, ``assign``: int32 ``[n_obj]`` CUDA tensors (outputs)."""
    ptrs = (ctypes.c_void_p * len(masses))(*[int(m.data_ptr()) for m in masses])
    off = _i32(obj_off)
    a = ClusterArgs()
    a.n_layers, a.mass = len(masses), ctypes.cast(ptrs, ctypes.c_void_p)
    a.n_q, a.n_q_heads, a.mass_stride = int(masses[0].shape[0]), int(masses[0].shape[1]), int(masses[0].shape[2])
    a.n_groups, a.n_obj, a.obj_off, a.threshold = int(n_groups), len(off) - 1, _np_ptr(off), float(threshold)
    a.avg, a.assign = _ptr(avg), _ptr(assign)
    rc = lib().enl_cluster_assign(ctypes.byref(a), stream or None)
    if rc != ENL_OK:
        raise EnlError(rc, "enl_cluster_assign")


def enl_cluster_assign_sums(mass_sum, obj_off: Sequence[int], n_groups: int, n_q_heads: int, n_layers: int,
                            threshold: float, avg, assign, stream: int = 0) -> None:
    """``mass_sum``: fp32 CUDA tensor ``[n_obj, stride]`` that the scoring attends added to (group_mass_sum);
    ``avg``: fp32 ``[n_obj, n_groups]``, ``assign``: int32 ``[n_obj]`` CUDA tensors (outputs)."""
    off = _i32(obj_off)
    rc = lib().enl_cluster_assign_sums(_ptr(mass_sum), int(mass_sum.shape[-1]), int(n_groups), len(off) - 1, _np_ptr(off),
                                       int(n_q_heads), int(n_layers), float(threshold), _ptr(avg), _ptr(assign),
                                       stream or None)
    if rc != ENL_OK:
        raise EnlError(rc, "enl_cluster_assign_sums")


def enl_select_knapsack(prob: Sequence[float], threshold: float, mem_bytes: Sequence[int], budget_bytes: int,
                        quantum: int = 1 << 20) -> np.ndarray:
    """Host-only.  Returns the selected group indices (ascending, int32)."""
    pr = np.ascontiguousarray(np.asarray(prob, dtype=np.float32))
    mb = np.ascontiguousarray(np.asarray(mem_bytes, dtype=np.int64))
    out = np.zeros(max(len(pr), 1), np.int32)
    rc = lib().enl_select_knapsack(len(pr), _np_ptr(pr), float(threshold), _np_ptr(mb), int(budget_bytes),
                                   int(quantum), _np_ptr(out))
    if rc < 0:
        raise EnlError(rc, "enl_select_knapsack")
    return out[:rc].copy()


def enl_rope_rotate(rows, positions=None, first_pos: int = 0, base: float = 10000.0, interleaved: bool = False,
                    stream: int = 0) -> None:
    """Rotates ``rows`` (device bf16 [n][heads][D]) in place; ``positions`` is a device int32 tensor [n] or None."""
    n, heads, d = (int(x) for x in rows.shape)
    rc = lib().enl_rope_rotate(_ptr(rows), n, heads, d, _ptr(positions), int(first_pos), float(base),
                               1 if interleaved else 0, stream or None)
    if rc != ENL_OK:
        raise EnlError(rc, "enl_rope_rotate")


def enl_tier_enable(cache: int, host_tokens: int) -> None:
    rc = lib().enl_tier_enable(cache, int(host_tokens))
    if rc != ENL_OK:
        raise EnlError(rc, "enl_tier_enable")


def enl_group_evict(cache: int, group_id: int, stream: int = 0) -> None:
    rc = lib().enl_group_evict(cache, int(group_id), stream or None)
    if rc != ENL_OK:
        raise EnlError(rc, "enl_group_evict")


def enl_step_prepare(cache: int, sel_ids: Sequence[int], stream: int = 0) -> dict:
    """Makes the selected groups device-resident; returns hits, misses, evictions and bytes moved."""
    sel = _i32(sel_ids)
    st = PrepareStats()
    rc = lib().enl_step_prepare(cache, _np_ptr(sel) if len(sel) else None, len(sel), stream or None, ctypes.byref(st))
    if rc != ENL_OK:
        raise EnlError(rc, "enl_step_prepare")
    return dict(n_hit=st.n_hit, n_miss=st.n_miss, n_evicted=st.n_evicted, bytes_h2d=st.bytes_h2d, bytes_d2h=st.bytes_d2h)


def enl_group_resident(cache: int, group_id: int) -> int:
    return int(lib().enl_group_resident(cache, int(group_id)))


def enl_cache_free(cache: int) -> None:
    _n_layers.pop(int(cache), None)
    lib().enl_cache_free(cache)


def enl_group_len(cache: int, group_id: int, layer: int) -> int:
    return int(lib().enl_group_len(cache, group_id, layer))


def enl_cache_status(cache: int) -> int:
    return int(lib().enl_cache_status(cache))


def enl_cache_selfcheck(cache: int) -> int:
    """ENL_OK, or ENL_E_CORRUPT when a guard page of the pool is no longer all zero."""
    return int(lib().enl_cache_selfcheck(cache))


def enl_plan_inspect(cache: int, cap_entries: int = 1 << 16, cap_batch: int = 256):
    """Host copy of the last gather plan: dict with stream pages/meta, per-episode offsets, splits, items and
    how the splits are merged (0 none, 1 merge kernel, 2 CTA pairs inside the attention kernel, 3 decode kernel)."""
    pages = np.zeros(cap_entries, np.int32)
    meta = np.zeros(cap_entries, np.int32)
    off = np.zeros(cap_batch, np.int32)
    tiles = np.zeros(cap_batch, np.int32)
    ne, ns, ni, mk = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
    rc = lib().enl_plan_inspect(cache, cap_entries, _np_ptr(pages), _np_ptr(meta), ctypes.byref(ne), cap_batch,
                                _np_ptr(off), _np_ptr(tiles), ctypes.byref(ns), ctypes.byref(ni), ctypes.byref(mk))
    if rc != ENL_OK:
        raise EnlError(rc, "enl_plan_inspect")
    n = min(ne.value, cap_entries)
    return dict(pages=pages[:n], meta=meta[:n], n_entries=ne.value, ep_stream_off=off, ep_cached_tiles=tiles,
                n_splits=ns.value, n_items=ni.value, merge_kind=mk.value)
