"""GPU parity at the full benchmark sizes, in the launch configuration the benchmark times (library-chosen
KV splits, varlen batch layout): sampled query rows of sampled layers against the float64 oracle, plus
properties that hold at any size (mass rows sum to 1, prefix sums bit-exact)."""
import numpy as np
import pytest
import torch

from paper_2510_18546_b200 import enl, synth
from tests.helpers import Session, check_close, sample_rows

pytestmark = pytest.mark.gpu


def layers_of(wl):
    return sorted({0, wl.n_layers // 2, wl.n_layers - 1})


@pytest.mark.parametrize("name", ["planner", "long", "long_scoring", "concurrent"])
def test_prefill_workloads_sampled_rows(name):
    wl = synth.make(name)
    layers = layers_of(wl) if name != "concurrent" else [0, wl.n_layers - 1]
    with Session(wl, layers) as s:
        cs, cq, cn = wl.cu()
        for li, layer in enumerate(layers):
            q, kn, vn = wl.new_qkv(layer, s.device)
            out, mass, sel_off = s.attend(li, q, kn, vn)
            torch.cuda.synchronize()
            assert enl.enl_cache_status(s.cache) == enl.ENL_OK
            assert torch.isfinite(out.float()).all()
            so = 0
            episodes = range(wl.batch) if wl.batch <= 4 else [0, 5, wl.batch - 1]
            offs_per_ep = {}
            for b in range(wl.batch):
                G = len(wl.sel_local[b])
                offs_per_ep[b] = sel_off[so:so + G + 1]
                so += G + 1
                rs = mass[cq[b]:cq[b + 1], :, :G + 1].sum(-1)
                assert (rs - 1).abs().max().item() < 1e-3, f"{name} layer {layer} ep {b}: mass rows must sum to 1"
                assert mass[cq[b]:cq[b + 1], :, :G + 1].min().item() >= 0
            for b in episodes:
                G = len(wl.sel_local[b])
                rows = sample_rows(wl.n_q[b], seed=layer * 100 + b)
                qo, mo, off = s.oracle(li, b, q[cq[b]:cq[b + 1]], kn[cn[b]:cn[b + 1]], vn[cn[b]:cn[b + 1]], rows=rows)
                idx = torch.as_tensor(rows, device=s.device) + int(cq[b])
                check_close(out[idx], qo, mass[idx][:, :, :G + 1], mo, what=f"{name} layer {layer} ep {b}")
                assert list(offs_per_ep[b]) == [int(x) for x in off]


def test_decode_workload_steps():
    """One query per step over ~32k cached tokens plus the grown new-token buffer; steps 0, 63 and 127."""
    wl = synth.make("decode")
    layers = layers_of(wl)
    with Session(wl, layers) as s:
        G = len(wl.sel_local[0])
        for li, layer in enumerate(layers):
            q, kn, vn = wl.new_qkv(layer, s.device)
            for t in (0, 63, 127):
                out, mass, sel_off = s.attend(li, q[t:t + 1], kn[:t + 1], vn[:t + 1], n_q=[1], n_new=[t + 1])
                torch.cuda.synchronize()
                assert enl.enl_cache_status(s.cache) == enl.ENL_OK
                qo, mo, off = s.oracle(li, 0, q[t:t + 1], kn[:t + 1], vn[:t + 1])
                check_close(out, qo, mass[:, :, :G + 1], mo, what=f"decode layer {layer} step {t}")
                assert list(sel_off) == [int(x) for x in off]
                assert (mass[:, :, :G + 1].sum(-1) - 1).abs().max().item() < 1e-3


def test_decode_step_equals_prefill_row():
    """App. A: decoding concatenates the new token's K/V; step t equals row t of a prefill over the same keys."""
    wl = synth.make_small(21, 1, 32, 8, 128, [[300, 17, 256, 90]], [[0, 1, 2, 3]], [40], [40], sigma=0.5, name="dec_eq")
    with Session(wl, [0]) as s:
        q, kn, vn = wl.new_qkv(0, s.device)
        o_all, m_all, _ = s.attend(0, q, kn, vn)
        for t in (0, 17, 39):
            o1, m1, _ = s.attend(0, q[t:t + 1], kn[:t + 1], vn[:t + 1], n_q=[1], n_new=[t + 1])
            torch.cuda.synchronize()
            assert (o1.float() - o_all[t:t + 1].float()).abs().max().item() <= 2e-2
            assert (m1 - m_all[t:t + 1]).abs().max().item() <= 1e-3


def test_indicator_values_tie_output_to_mass():
    """With V = indicator of the slot, output channel s equals mass slot s (bf16 rounding apart)."""
    wl = synth.make_small(22, 1, 8, 2, 128, [[50, 33, 70]], [[0, 1, 2]], [96], [96], name="tie")
    with Session(wl, [0]) as s:
        k, v = wl.pool_kv(0, 0, s.device)
        offs = wl.pool_offsets(0)
        v = torch.zeros_like(v)
        for g in range(3):
            v[offs[g]:offs[g + 1], :, g] = 1
            enl.enl_group_store(s.cache, g, 0, k[offs[g]:offs[g + 1]], v[offs[g]:offs[g + 1]])
        q, kn, vn = wl.new_qkv(0, s.device)
        vn = torch.zeros_like(vn)
        vn[:, :, 3] = 1
        out, mass, _ = s.attend(0, q, kn, vn)
        torch.cuda.synchronize()
        assert (out[:, :, :4].float() - mass[:, :, :4]).abs().max().item() <= 8e-3
        assert out[:, :, 4:].float().abs().max().item() == 0.0
