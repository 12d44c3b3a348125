"""Shared test plumbing: run one workload through the CUDA library and through the CPU oracle
on the same seeded tensors, and compare.  No arithmetic of the method lives here."""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

from oracle import enl_oracle as orc
from paper_2510_18546_b200 import enl
from paper_2510_18546_b200.synth import Workload

# tolerances of the parity bar: bf16 outputs and fp32 masses against the float64 oracle
OUT_MAX_ABS, OUT_MEAN_ABS, MASS_MAX_ABS = 2e-2, 2e-3, 1e-3


class Session:
    """A cache on the GPU filled with a workload's pool for the given layers.
    Cache layer index i holds workload layer ``layers[i]``."""

    def __init__(self, wl: Workload, layers: Sequence[int], device: str = "cuda:0", scratch_bytes: int = 0,
                 extra_tokens: int = 0, extra_groups: int = 0):
        self.wl, self.layers, self.device = wl, list(layers), torch.device(device)
        tq = wl.decode_steps if wl.decode_steps else int(sum(wl.n_q))
        self.cache = enl.enl_cache_create(len(self.layers), wl.n_q_heads, wl.n_kv_heads, wl.head_dim,
                                          max_groups=wl.n_groups + extra_groups,
                                          max_tokens=wl.pool_tokens + extra_tokens,
                                          device=self.device.index or 0, max_batch=max(wl.batch, 1),
                                          max_q_tokens=max(tq, 1), scratch_bytes=scratch_bytes)
        self.host_kv: Dict = {}
        for li, layer in enumerate(self.layers):
            for b in range(wl.batch):
                k, v = wl.pool_kv(layer, b, self.device)
                offs = wl.pool_offsets(b)
                for g in range(len(wl.pool_lens[b])):
                    enl.enl_group_store(self.cache, wl.group_base[b] + g, li, k[offs[g]:offs[g + 1]],
                                        v[offs[g]:offs[g + 1]])
                # the oracle only ever needs the selected groups: keep those on the host
                sel = wl.sel_local[b]
                self.host_kv[(li, b)] = ([k[offs[g]:offs[g + 1]].cpu() for g in sel],
                                         [v[offs[g]:offs[g + 1]].cpu() for g in sel])
        torch.cuda.synchronize(self.device)

    def close(self):
        if self.cache:
            try:
                # the two pages no group owns (one at either end of every layer's pool) must still be all zero
                assert enl.enl_cache_selfcheck(self.cache) == enl.ENL_OK, "a kernel wrote outside its pages"
            finally:
                enl.enl_cache_free(self.cache)
                self.cache = None

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()

    # ---- CUDA path ------------------------------------------------------------------------
    def attend(self, li: int, q, k_new, v_new, n_q: Optional[List[int]] = None, n_new: Optional[List[int]] = None,
               split_hint: int = 0, want_mass: bool = True, sel_override=None):
        wl = self.wl
        n_q = list(n_q) if n_q is not None else list(wl.n_q)
        n_new = list(n_new) if n_new is not None else list(wl.n_new)
        sel = wl.sel_ids() if sel_override is None else np.asarray(sel_override, np.int32)
        cs, _, _ = wl.cu()
        cq = np.concatenate([[0], np.cumsum(n_q)]).astype(np.int32)
        cn = np.concatenate([[0], np.cumsum(n_new)]).astype(np.int32)
        max_slots = int(np.max(np.diff(cs))) if len(sel) else 0
        out = torch.empty(int(cq[-1]), wl.n_q_heads, wl.head_dim, dtype=torch.bfloat16, device=self.device)
        mass = None
        if want_mass:
            mass = torch.full((int(cq[-1]), wl.n_q_heads, max_slots + 1), float("nan"),
                              dtype=torch.float32, device=self.device)
        sel_off = enl.enl_attend(self.cache, li, sel, q, k_new, v_new, out, mass,
                                 cu_sel=cs if wl.batch > 1 else None, cu_q=cq if wl.batch > 1 else None,
                                 cu_new=cn if wl.batch > 1 else None, n_q=int(cq[-1]), n_new=int(cn[-1]),
                                 want_sel_off=True, split_hint=split_hint,
                                 stream=torch.cuda.current_stream(self.device).cuda_stream)
        return out, mass, sel_off

    # ---- oracle ---------------------------------------------------------------------------
    def oracle(self, li: int, b: int, q, k_new, v_new, rows=None):
        """Episode b through the float64 oracle; q/k_new/v_new are that episode's own rows."""
        ks, vs = self.host_kv[(li, b)]
        wl = self.wl
        out, mass = orc.attend_slots(wl.n_q_heads, wl.n_kv_heads, wl.head_dim, ks, vs,
                                     q.cpu(), k_new.cpu(), v_new.cpu(), rows=rows)
        return out, mass, orc.sel_off([k.shape[0] for k in ks])


def check_close(out_gpu: torch.Tensor, out_ref: np.ndarray, mass_gpu: Optional[torch.Tensor],
                mass_ref: Optional[np.ndarray], what: str = ""):
    """The parity bar: max abs <= 2e-2 and mean abs <= 2e-3 on bf16 outputs, 1e-3 on masses."""
    og = out_gpu.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(og).all(), f"{what}: non-finite output"
    err = np.abs(og - out_ref)
    assert err.max() <= OUT_MAX_ABS, f"{what}: out max abs {err.max():.3e}"
    assert err.mean() <= OUT_MEAN_ABS, f"{what}: out mean abs {err.mean():.3e}"
    res = dict(out_max=float(err.max()), out_mean=float(err.mean()))
    if mass_ref is not None:
        mg = mass_gpu.cpu().numpy().astype(np.float64)[..., :mass_ref.shape[-1]]
        assert np.isfinite(mg).all(), f"{what}: non-finite mass"
        me = np.abs(mg - mass_ref)
        assert me.max() <= MASS_MAX_ABS, f"{what}: mass max abs {me.max():.3e}"
        res["mass_max"] = float(me.max())
    return res


def sample_rows(n_q: int, seed: int, extra: int = 24) -> List[int]:
    """Fixed rows around tile edges plus seeded random rows."""
    fixed = [0, 1, 31, 32, 63, 64, 127, 128, n_q // 2, n_q - 1]
    rng = np.random.default_rng(seed)
    rows = set(r for r in fixed if 0 <= r < n_q)
    rows.update(int(x) for x in rng.integers(0, n_q, size=extra))
    return sorted(rows)
