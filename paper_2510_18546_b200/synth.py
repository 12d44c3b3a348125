"""Seeded synthetic workloads shaped like the paper's planner prompts.

This module holds NO arithmetic of the method: it only draws shapes (group lengths, select
lists, new-token counts) and bf16 values from seeded generators.  Both the CUDA path and the
CPU oracle are fed from it, by the tests and the benchmark.

Shapes follow the paper: a navigation map split into object groups of tens to hundreds of
tokens (App. C), prompts of up to thousands of tokens (Sec. 3.1), new tokens = instruction
plus trajectory (App. C), about 40-128 decoded tokens per planning step (Sec. 3.2), 40
layers for the 11B planner (App. D).  Values are N(0, sigma^2) rounded to bf16.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Tuple

import numpy as np
import torch


@dataclass
class Workload:
    name: str
    seed: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    sigma: float
    pool_lens: List[np.ndarray]          # per episode: length of every pool group
    sel_local: List[np.ndarray]          # per episode: selected groups, indices into that pool
    n_q: List[int]                       # per episode: query rows
    n_new: List[int]                     # per episode: new-token keys
    decode_steps: int = 0                # > 0: n_q = 1 per step, n_new = t + 1
    group_base: List[int] = field(default_factory=list)   # global id of each episode's group 0

    def __post_init__(self):
        base, acc = [], 0
        for lens in self.pool_lens:
            base.append(acc)
            acc += len(lens)
        self.group_base = base

    # ---- shapes -------------------------------------------------------------------------
    @property
    def batch(self) -> int:
        return len(self.pool_lens)

    @property
    def n_groups(self) -> int:
        return int(sum(len(x) for x in self.pool_lens))

    @property
    def pool_tokens(self) -> int:
        return int(sum(int(x.sum()) for x in self.pool_lens))

    def sel_ids(self) -> np.ndarray:
        """Concatenated global group ids of every episode's select list (int32)."""
        return np.concatenate([self.sel_local[b].astype(np.int32) + self.group_base[b]
                               for b in range(self.batch)]).astype(np.int32)

    def cu(self) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
        """(cu_sel, cu_q, cu_new): per-episode prefix counts, each of length batch + 1."""
        cs = np.zeros(self.batch + 1, np.int32)
        cq = np.zeros(self.batch + 1, np.int32)
        cn = np.zeros(self.batch + 1, np.int32)
        for b in range(self.batch):
            cs[b + 1] = cs[b] + len(self.sel_local[b])
            cq[b + 1] = cq[b] + self.n_q[b]
            cn[b + 1] = cn[b] + self.n_new[b]
        return cs, cq, cn

    def selected_tokens(self, b: int) -> int:
        return int(self.pool_lens[b][self.sel_local[b]].sum())

    # ---- values -------------------------------------------------------------------------
    def _gen(self, layer: int, episode: int, kind: int, device) -> torch.Generator:
        g = torch.Generator(device=device)
        g.manual_seed((((self.seed * 1000 + layer) * 4096 + episode) * 8 + kind) & 0x7FFFFFFFFFFF)
        return g

    def _randn_bf16(self, shape, gen, device) -> torch.Tensor:
        x = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
        return (x * self.sigma).to(torch.bfloat16)

    def pool_kv(self, layer: int, episode: int, device="cpu") -> Tuple[torch.Tensor, torch.Tensor]:
        """K, V of one episode's whole pool for one layer: ``[pool tokens, Hkv, D]`` bf16.
        Group i occupies rows ``offs[i]:offs[i+1]`` with ``offs = cumsum(pool_lens)``."""
        n = int(self.pool_lens[episode].sum())
        shape = (n, self.n_kv_heads, self.head_dim)
        k = self._randn_bf16(shape, self._gen(layer, episode, 0, device), device)
        v = self._randn_bf16(shape, self._gen(layer, episode, 1, device), device)
        return k, v

    def pool_offsets(self, episode: int) -> np.ndarray:
        return np.concatenate([[0], np.cumsum(self.pool_lens[episode])]).astype(np.int64)

    def new_qkv(self, layer: int, device="cpu"):
        """q ``[sum n_q, Hq, D]``, k_new / v_new ``[sum n_new, Hkv, D]`` for the whole batch.
        For a decode workload these are the full buffers of all steps (``decode_steps`` rows);
        step t uses q row t and new keys 0..t."""
        if self.decode_steps:
            tq, tn = self.decode_steps, self.decode_steps
        else:
            tq, tn = int(sum(self.n_q)), int(sum(self.n_new))
        q = self._randn_bf16((tq, self.n_q_heads, self.head_dim), self._gen(layer, 0, 2, device), device)
        k = self._randn_bf16((tn, self.n_kv_heads, self.head_dim), self._gen(layer, 0, 3, device), device)
        v = self._randn_bf16((tn, self.n_kv_heads, self.head_dim), self._gen(layer, 0, 4, device), device)
        return q, k, v


def _lens(g: torch.Generator, n: int, lo: int, hi: int) -> np.ndarray:
    return torch.randint(lo, hi + 1, (n,), generator=g).numpy().astype(np.int32)


def _pick(g: torch.Generator, pool: int, k: int) -> np.ndarray:
    return torch.randperm(pool, generator=g)[:k].numpy().astype(np.int32)


def make(name: str) -> Workload:
    """The five benchmark workloads (plus the all-groups scoring pass of the long episode)."""
    planner = dict(n_q_heads=32, n_kv_heads=8, head_dim=128, sigma=0.5)
    if name == "tiny":
        g = torch.Generator().manual_seed(0)
        return Workload("tiny", 0, 1, 8, 2, 64, 1.0, [np.full(16, 32, np.int32)],
                        [_pick(g, 16, 4)], [64], [64])
    if name == "planner":
        g = torch.Generator().manual_seed(1)
        lens = _lens(g, 200, 40, 120)
        return Workload("planner", 1, 40, pool_lens=[lens], sel_local=[_pick(g, 200, 24)],
                        n_q=[512], n_new=[512], **planner)
    if name in ("long", "long_scoring"):
        g = torch.Generator().manual_seed(2)
        lens = _lens(g, 1000, 20, 200)
        sel = _pick(g, 1000, 64)
        if name == "long":
            return Workload("long", 2, 40, pool_lens=[lens], sel_local=[sel],
                            n_q=[1024], n_new=[1024], **planner)
        # clustering pass: every pool group is scored, on the first ceil(40/10) layers
        return Workload("long_scoring", 2, 4, pool_lens=[lens],
                        sel_local=[np.arange(1000, dtype=np.int32)],
                        n_q=[1024], n_new=[1024], **planner)
    if name == "concurrent":
        g = torch.Generator().manual_seed(3)
        pools, sels, nq = [], [], []
        for _ in range(16):
            pools.append(_lens(g, 300, 40, 160))
            sels.append(_pick(g, 300, 32))
            nq.append(int(torch.randint(256, 769, (1,), generator=g).item()))
        return Workload("concurrent", 3, 40, pool_lens=pools, sel_local=sels,
                        n_q=nq, n_new=list(nq), **planner)
    if name == "decode":
        g = torch.Generator().manual_seed(4)
        lens = _lens(g, 128, 256, 426)
        return Workload("decode", 4, 40, pool_lens=[lens], sel_local=[_pick(g, 128, 96)],
                        n_q=[1], n_new=[1], decode_steps=128, **planner)
    raise KeyError(name)


def make_small(seed: int, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int,
               pool_lens, sel_local, n_q, n_new, sigma: float = 1.0, name: str = "custom") -> Workload:
    """A hand-specified workload for tests (lists per episode)."""
    return Workload(name, seed, n_layers, n_q_heads, n_kv_heads, head_dim, sigma,
                    [np.asarray(x, np.int32) for x in pool_lens],
                    [np.asarray(x, np.int32) for x in sel_local], list(n_q), list(n_new))


NAMES = ("tiny", "planner", "long", "long_scoring", "concurrent", "decode")
