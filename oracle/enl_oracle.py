"""Python front end of the float64 CPU oracle (``enl_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the benchmark's
CPU-baseline leg.  The product package never imports this module, and this module never
imports the product package.

The oracle keeps its own group container (a dict of plain arrays, no pages): one entry per
(group id, layer), rows in stored order; an append concatenates at the end (paper, Sec. 3.2:
new objects are concatenated at the end of their group, existing K/V is untouched).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "enl_oracle.c")
_LIB = os.path.join(_HERE, "libenl_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP, -O2, no fast-math) into ``libenl_oracle.so``."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        lib.enl_oracle_threads.restype = ctypes.c_int
        lib.enl_oracle_sel_off.restype = None
        lib.enl_oracle_attend.restype = ctypes.c_int
        _lib = lib
    return _lib


def threads() -> int:
    """Number of OpenMP threads the oracle will use."""
    return int(_load().enl_oracle_threads())


def _bits(x) -> np.ndarray:
    """bf16 tensor / uint16 array -> contiguous uint16 bit patterns (exact, no rounding)."""
    if isinstance(x, np.ndarray):
        if x.dtype != np.uint16:
            raise TypeError("numpy inputs must already be uint16 bf16 bit patterns")
        return np.ascontiguousarray(x)
    import torch  # local: only tensors need it

    if x.dtype != torch.bfloat16:
        raise TypeError("tensor inputs must be bfloat16")
    return np.ascontiguousarray(x.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16))


def sel_off(sel_len: Sequence[int]) -> np.ndarray:
    """Exclusive prefix sum of the selected groups' lengths, length n_sel + 1 (int64)."""
    n = len(sel_len)
    a = np.ascontiguousarray(np.asarray(sel_len, dtype=np.int32))
    out = np.zeros(n + 1, dtype=np.int64)
    _load().enl_oracle_sel_off(
        ctypes.c_int(n), a.ctypes.data_as(ctypes.c_void_p), out.ctypes.data_as(ctypes.c_void_p)
    )
    return out


def attend_slots(
    n_q_heads: int,
    n_kv_heads: int,
    head_dim: int,
    slots_k: Sequence,
    slots_v: Sequence,
    q,
    k_new,
    v_new,
    rows: Optional[Sequence[int]] = None,
    want_mass: bool = True,
) -> Tuple[np.ndarray, Optional[np.ndarray]]:
    """Attention of one episode over explicit slot arrays.

    ``slots_k[s]`` / ``slots_v[s]``: ``[len_s, Hkv, D]`` bf16; ``q``: ``[n_q, Hq, D]``;
    ``k_new`` / ``v_new``: ``[n_new, Hkv, D]``.  Returns ``(out [n_rows, Hq, D] f64,
    mass [n_rows, Hq, n_sel + 1] f64)``; ``rows`` picks query rows (default: all).
    """
    lib = _load()
    n_sel = len(slots_k)
    kb = [_bits(k) for k in slots_k]
    vb = [_bits(v) for v in slots_v]
    lens = np.asarray([k.shape[0] if k.ndim == 3 else 0 for k in kb], dtype=np.int32)
    for k, v in zip(kb, vb):
        assert k.shape == v.shape
        assert k.shape[0] == 0 or k.shape[1:] == (n_kv_heads, head_dim)
    qb, knb, vnb = _bits(q), _bits(k_new), _bits(v_new)
    n_q, n_new = qb.shape[0], knb.shape[0]
    assert qb.shape[1:] == (n_q_heads, head_dim)
    assert knb.shape == vnb.shape and (n_new == 0 or knb.shape[1:] == (n_kv_heads, head_dim))
    if rows is None:
        rows_a = np.arange(n_q, dtype=np.int32)
    else:
        rows_a = np.ascontiguousarray(np.asarray(rows, dtype=np.int32))
    n_rows = int(rows_a.shape[0])
    out = np.zeros((n_rows, n_q_heads, head_dim), dtype=np.float64)
    mass = np.zeros((n_rows, n_q_heads, n_sel + 1), dtype=np.float64) if want_mass else None
    PtrArr = ctypes.c_void_p * max(n_sel, 1)
    kp = PtrArr(*[k.ctypes.data for k in kb]) if n_sel else PtrArr()
    vp = PtrArr(*[v.ctypes.data for v in vb]) if n_sel else PtrArr()
    rc = lib.enl_oracle_attend(
        ctypes.c_int(n_q_heads), ctypes.c_int(n_kv_heads), ctypes.c_int(head_dim),
        ctypes.c_int(n_sel), lens.ctypes.data_as(ctypes.c_void_p), kp, vp,
        ctypes.c_int(n_q), ctypes.c_int(n_new),
        qb.ctypes.data_as(ctypes.c_void_p), knb.ctypes.data_as(ctypes.c_void_p),
        vnb.ctypes.data_as(ctypes.c_void_p),
        ctypes.c_int(n_rows), rows_a.ctypes.data_as(ctypes.c_void_p),
        out.ctypes.data_as(ctypes.c_void_p),
        mass.ctypes.data_as(ctypes.c_void_p) if mass is not None else None,
    )
    if rc != 0:
        raise ValueError("enl_oracle_attend rejected its arguments")
    return out, mass


class OracleCache:
    """The oracle's own group store: ``(group, layer) -> (K bits, V bits)``, no pages."""

    def __init__(self, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int):
        self.n_layers, self.n_q_heads = n_layers, n_q_heads
        self.n_kv_heads, self.head_dim = n_kv_heads, head_dim
        self._g: Dict[Tuple[int, int], Tuple[np.ndarray, np.ndarray]] = {}

    def group_store(self, group_id: int, layer: int, k, v, append: bool = False) -> None:
        kb, vb = _bits(k), _bits(v)
        kb = kb.reshape(-1, self.n_kv_heads, self.head_dim)
        vb = vb.reshape(-1, self.n_kv_heads, self.head_dim)
        key = (int(group_id), int(layer))
        if append and key in self._g:
            k0, v0 = self._g[key]
            kb, vb = np.concatenate([k0, kb], axis=0), np.concatenate([v0, vb], axis=0)
        self._g[key] = (kb, vb)

    def group_len(self, group_id: int, layer: int) -> int:
        return int(self._g[(int(group_id), int(layer))][0].shape[0])

    def attend(
        self,
        layer: int,
        sel_ids: Sequence[int],
        q,
        k_new,
        v_new,
        rows: Optional[Sequence[int]] = None,
        want_mass: bool = True,
    ):
        """One episode.  Returns ``(out, mass, sel_off)``; slots follow ``sel_ids`` order."""
        ks = [self._g[(int(g), int(layer))][0] for g in sel_ids]
        vs = [self._g[(int(g), int(layer))][1] for g in sel_ids]
        out, mass = attend_slots(self.n_q_heads, self.n_kv_heads, self.head_dim, ks, vs,
                                 q, k_new, v_new, rows=rows, want_mass=want_mass)
        return out, mass, sel_off([k.shape[0] for k in ks])


# ---- clustering reduce and retrieval knapsack (the consumers / producers around the attention) ----

def cluster_assign(masses: Sequence[np.ndarray], obj_off: Sequence[int], n_groups: int, threshold: float):
    """Sec. 3.3: average attention between each new object and each existing group, and the decision.

    ``masses``: one ``[n_q, Hq, >= n_groups]`` array per scored layer (the per-slot mass of the scoring
    attend); object o owns query rows ``obj_off[o]:obj_off[o+1]``.  The average runs over the object's
    rows, all q heads and all layers (float64).  Returns ``(avg [n_obj, n_groups], assign [n_obj])`` with
    ``assign = argmax`` (lowest index on ties) where the largest average exceeds the threshold, else -1."""
    n_obj = len(obj_off) - 1
    avg = np.zeros((n_obj, n_groups), dtype=np.float64)
    assign = np.full(n_obj, -1, dtype=np.int64)
    for o in range(n_obj):
        r0, r1 = int(obj_off[o]), int(obj_off[o + 1])
        total = np.zeros(n_groups, dtype=np.float64)
        count = 0
        for m in masses:
            blk = np.asarray(m, dtype=np.float64)[r0:r1, :, :n_groups]
            total += blk.sum(axis=(0, 1))
            count += blk.shape[0] * blk.shape[1]
        if count:
            avg[o] = total / count
        g = int(np.argmax(avg[o]))
        if avg[o, g] > threshold:
            assign[o] = g
    return avg, assign


def knapsack_bruteforce(prob: Sequence[float], threshold: float, mem_bytes: Sequence[int], budget_bytes: int,
                        quantum: int):
    """Sec. 3.4, Eq. 1-2 by enumeration: max sum (P_i - threshold) x_i  s.t.  sum M_i x_i <= M, x_i in {0,1},
    with M_i rounded up and M rounded down to multiples of ``quantum``.  Returns ``(best value, best subsets)``:
    every subset (as a sorted tuple) that reaches the best value within 1e-12.  Small n only."""
    n = len(prob)
    w = [-(-int(m) // int(quantum)) for m in mem_bytes]
    cap = int(budget_bytes) // int(quantum)
    best, arg = 0.0, [()]
    for mask in range(1, 1 << n):
        idx = tuple(i for i in range(n) if mask >> i & 1)
        if sum(w[i] for i in idx) > cap:
            continue
        v = float(sum(float(np.float32(prob[i])) - float(np.float32(threshold)) for i in idx))
        if v > best + 1e-12:
            best, arg = v, [idx]
        elif abs(v - best) <= 1e-12:
            arg.append(idx)
    return best, arg


def rope_rotate(rows: np.ndarray, positions: Sequence[int], base: float, interleaved: bool) -> np.ndarray:
    """Rotary position embedding as published (Su et al., "RoFormer"; Sec. 3.2 of the paper only cites it): in every
    head, channel pair j -- (2j, 2j+1) when ``interleaved``, else (j, j + D/2) -- of the row at position pos is turned
    by the angle pos * base^(-2j/D).  ``rows`` is float64 [n][heads][D]; returns a new array."""
    x = np.asarray(rows, dtype=np.float64)
    n, heads, d = x.shape
    out = np.empty_like(x)
    for i in range(n):
        for j in range(d // 2):
            ang = float(positions[i]) * float(base) ** (-2.0 * j / d)
            cs, sn = np.cos(ang), np.sin(ang)
            i1, i2 = (2 * j, 2 * j + 1) if interleaved else (j, j + d // 2)
            out[i, :, i1] = x[i, :, i1] * cs - x[i, :, i2] * sn
            out[i, :, i2] = x[i, :, i2] * cs + x[i, :, i1] * sn
    return out


class TierModel:
    """Residency book-keeping of the slow tier (Sec. 3.2 / 3.4): which groups are in device memory, under a
    device budget in pages, with least-recently-selected eviction.  Plain Python; the reference for the hit /
    miss / eviction counts of enl_step_prepare."""

    def __init__(self, device_pages: int, page_tokens: int = 16):
        self.free = int(device_pages)
        self.page_tokens = page_tokens
        self.pages: Dict[int, int] = {}          # group -> pages
        self.resident: Dict[int, bool] = {}
        self.last_use: Dict[int, int] = {}
        self.tick = 0

    def store(self, gid: int, n_tokens: int) -> None:
        need = -(-n_tokens // self.page_tokens)
        have = self.pages.get(gid, 0)
        assert self.resident.get(gid, True)
        self.free -= need - have
        assert self.free >= 0
        self.pages[gid] = need
        self.resident[gid] = True
        self.last_use.setdefault(gid, 0)

    def evict(self, gid: int) -> None:
        if self.resident[gid]:
            self.free += self.pages[gid]
            self.resident[gid] = False

    def prepare(self, sel: Sequence[int]):
        self.tick += 1
        uniq = list(dict.fromkeys(int(g) for g in sel))
        hits = [g for g in uniq if self.resident[g]]
        misses = [g for g in uniq if not self.resident[g]]
        need = sum(self.pages[g] for g in misses)
        evicted = []
        if self.free < need:
            cand = sorted((g for g in self.pages if self.resident[g] and self.pages[g] > 0 and g not in uniq),
                          key=lambda g: (self.last_use[g], g))
            for g in cand:
                if self.free >= need:
                    break
                self.evict(g)
                evicted.append(g)
            assert self.free >= need
        for g in misses:
            self.free -= self.pages[g]
            self.resident[g] = True
        for g in uniq:
            self.last_use[g] = self.tick
        return hits, misses, evicted
