"""Pins for the float64 oracle: each test ties it to something other than itself.

The paper prints no numeric worked example for the attention (App. A gives the formula,
App. C a prompt layout), so the pins are: an independent library routine, an independent
brute force, closed forms, and invariants that the definition implies.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import enl_oracle as orc

HERE = os.path.dirname(os.path.abspath(__file__))


def bf16(x: torch.Tensor) -> torch.Tensor:
    return x.to(torch.bfloat16)


def rand_case(seed, Hq, Hkv, D, lens, n_q, n_new, sigma=1.0):
    g = torch.Generator().manual_seed(seed)
    ks = [bf16(torch.randn(n, Hkv, D, generator=g) * sigma) for n in lens]
    vs = [bf16(torch.randn(n, Hkv, D, generator=g) * sigma) for n in lens]
    q = bf16(torch.randn(n_q, Hq, D, generator=g) * sigma)
    kn = bf16(torch.randn(n_new, Hkv, D, generator=g) * sigma)
    vn = bf16(torch.randn(n_new, Hkv, D, generator=g) * sigma)
    return ks, vs, q, kn, vn


def sdpa_reference(Hq, Hkv, D, ks, vs, q, kn, vn):
    """Dense masked attention over the concatenation through torch's SDPA in float64:
    the first S columns are visible to every row, the rest causally (bottom-right aligned)."""
    rep = Hq // Hkv
    K = torch.cat(list(ks) + [kn], 0).double()            # [S + n_new, Hkv, D]
    V = torch.cat(list(vs) + [vn], 0).double()
    S = K.shape[0] - kn.shape[0]
    n_q, n_new = q.shape[0], kn.shape[0]
    Kh = K.permute(1, 0, 2).repeat_interleave(rep, 0)      # [Hq, T, D]
    Vh = V.permute(1, 0, 2).repeat_interleave(rep, 0)
    Qh = q.double().permute(1, 0, 2)                        # [Hq, n_q, D]
    mask = torch.zeros(n_q, S + n_new, dtype=torch.bool)
    mask[:, :S] = True
    for r in range(n_q):
        mask[r, S:S + (n_new - n_q) + r + 1] = True
    o = torch.nn.functional.scaled_dot_product_attention(Qh, Kh, Vh, attn_mask=mask)
    return o.permute(1, 0, 2).numpy()                       # [n_q, Hq, D]


def brute_force_longdouble(Hq, Hkv, D, ks, vs, q, kn, vn):
    """A second, deliberately different formulation: exp / sum with NO max subtraction,
    numpy extended precision, one key at a time."""
    rep = Hq // Hkv
    n_q, n_new = q.shape[0], kn.shape[0]
    f = lambda t: t.float().numpy().astype(np.longdouble)
    ks_, vs_ = [f(k) for k in ks], [f(v) for v in vs]
    q_, kn_, vn_ = f(q), f(kn), f(vn)
    out = np.zeros((n_q, Hq, D), np.longdouble)
    mass = np.zeros((n_q, Hq, len(ks) + 1), np.longdouble)
    for r in range(n_q):
        c = n_new - n_q + r
        for h in range(Hq):
            kv = h // rep
            num = np.zeros(D, np.longdouble)
            den = np.longdouble(0)
            w = np.zeros(len(ks) + 1, np.longdouble)
            for s in range(len(ks)):
                for t in range(ks_[s].shape[0]):
                    e = np.exp(np.dot(q_[r, h], ks_[s][t, kv]) / np.sqrt(np.longdouble(D)))
                    num += e * vs_[s][t, kv]
                    den += e
                    w[s] += e
            for t in range(c + 1):
                e = np.exp(np.dot(q_[r, h], kn_[t, kv]) / np.sqrt(np.longdouble(D)))
                num += e * vn_[t, kv]
                den += e
                w[-1] += e
            out[r, h] = num / den
            mass[r, h] = w / den
    return out.astype(np.float64), mass.astype(np.float64)


# ---- 1. reduces to a library routine ------------------------------------------------------
@pytest.mark.parametrize("Hq,Hkv,D,lens,n_q,n_new", [
    (8, 2, 64, [32, 32, 32, 32], 64, 64),
    (4, 4, 16, [5, 1, 9], 7, 7),
    (6, 2, 32, [3, 17], 4, 11),          # n_q < n_new: queries align with the last new keys
    (4, 1, 8, [], 9, 9),                 # empty select list: plain causal attention
])
def test_matches_sdpa_float64(Hq, Hkv, D, lens, n_q, n_new):
    ks, vs, q, kn, vn = rand_case(11, Hq, Hkv, D, lens, n_q, n_new)
    out, mass = orc.attend_slots(Hq, Hkv, D, ks, vs, q, kn, vn)
    ref = sdpa_reference(Hq, Hkv, D, ks, vs, q, kn, vn)
    assert np.abs(out - ref).max() < 1e-12
    assert np.abs(mass.sum(-1) - 1).max() < 1e-12


def test_empty_select_is_causal_sdpa():
    Hq, Hkv, D = 4, 2, 16
    _, _, q, kn, vn = rand_case(5, Hq, Hkv, D, [], 12, 12)
    out, mass = orc.attend_slots(Hq, Hkv, D, [], [], q, kn, vn)
    Qh = q.double().permute(1, 0, 2)
    Kh = kn.double().permute(1, 0, 2).repeat_interleave(2, 0)
    Vh = vn.double().permute(1, 0, 2).repeat_interleave(2, 0)
    ref = torch.nn.functional.scaled_dot_product_attention(Qh, Kh, Vh, is_causal=True)
    assert np.abs(out - ref.permute(1, 0, 2).numpy()).max() < 1e-12
    assert mass.shape[-1] == 1 and np.abs(mass - 1).max() < 1e-12


# ---- 8. brute force on tiny inputs, different formulation ---------------------------------
@pytest.mark.parametrize("seed", range(6))
def test_brute_force_tiny(seed):
    rng = np.random.default_rng(seed)
    Hkv = int(rng.integers(1, 3))
    Hq = Hkv * int(rng.integers(1, 4))
    D = 8
    lens = [int(x) for x in rng.integers(1, 6, size=int(rng.integers(1, 5)))]
    n_new = int(rng.integers(1, 6))
    n_q = int(rng.integers(1, n_new + 1))
    ks, vs, q, kn, vn = rand_case(100 + seed, Hq, Hkv, D, lens, n_q, n_new)
    out, mass = orc.attend_slots(Hq, Hkv, D, ks, vs, q, kn, vn)
    bo, bm = brute_force_longdouble(Hq, Hkv, D, ks, vs, q, kn, vn)
    assert np.abs(out - bo).max() < 1e-13
    assert np.abs(mass - bm).max() < 1e-13


def test_brute_force_tiny_config_rows():
    """The Tiny benchmark shape (8/2 heads, D=64, 4 groups of 32, 64 new tokens), a few rows."""
    ks, vs, q, kn, vn = rand_case(0, 8, 2, 64, [32] * 4, 64, 64)
    rows = [0, 1, 31, 63]
    out, mass = orc.attend_slots(8, 2, 64, ks, vs, q, kn, vn, rows=rows)
    bo, bm = brute_force_longdouble(8, 2, 64, ks, vs, q, kn, vn)
    assert np.abs(out - bo[rows]).max() < 1e-12
    assert np.abs(mass - bm[rows]).max() < 1e-12


# ---- 2./3./4. invariants ------------------------------------------------------------------
def test_mass_rows_sum_to_one_and_nonnegative():
    ks, vs, q, kn, vn = rand_case(3, 8, 2, 32, [7, 40, 1, 19], 20, 33)
    _, mass = orc.attend_slots(8, 2, 32, ks, vs, q, kn, vn)
    assert mass.min() >= 0
    assert np.abs(mass.sum(-1) - 1).max() < 1e-12


def test_select_order_permutation():
    lens = [7, 40, 1, 19, 12]
    ks, vs, q, kn, vn = rand_case(4, 8, 2, 32, lens, 10, 10)
    out, mass = orc.attend_slots(8, 2, 32, ks, vs, q, kn, vn)
    perm = [3, 0, 4, 2, 1]
    out2, mass2 = orc.attend_slots(8, 2, 32, [ks[i] for i in perm], [vs[i] for i in perm], q, kn, vn)
    assert np.abs(out - out2).max() < 1e-12
    assert np.abs(mass[..., perm] - mass2[..., :5]).max() < 1e-12
    assert np.abs(mass[..., 5] - mass2[..., 5]).max() < 1e-12
    assert list(orc.sel_off([lens[i] for i in perm])) == [0, 19, 26, 38, 39, 79]


def test_group_split_additivity():
    ks, vs, q, kn, vn = rand_case(6, 4, 2, 16, [11, 30, 5], 6, 6)
    out, mass = orc.attend_slots(4, 2, 16, ks, vs, q, kn, vn)
    ks2 = [ks[0], ks[1][:13], ks[1][13:], ks[2]]
    vs2 = [vs[0], vs[1][:13], vs[1][13:], vs[2]]
    out2, mass2 = orc.attend_slots(4, 2, 16, ks2, vs2, q, kn, vn)
    assert np.abs(out - out2).max() < 1e-12
    assert np.abs(mass[..., 1] - (mass2[..., 1] + mass2[..., 2])).max() < 1e-12
    assert np.abs(mass[..., [0, 2, 3]] - mass2[..., [0, 3, 4]]).max() < 1e-12


# ---- 5. closed forms ----------------------------------------------------------------------
def test_zero_query_is_uniform():
    lens = [3, 10, 6]
    ks, vs, q, kn, vn = rand_case(7, 4, 2, 16, lens, 5, 8)
    q = torch.zeros_like(q)
    out, mass = orc.attend_slots(4, 2, 16, ks, vs, q, kn, vn)
    S = sum(lens)
    Vcat = torch.cat(vs, 0).double()
    for r in range(5):
        c = 8 - 5 + r
        n = S + c + 1
        for s, L in enumerate(lens):
            assert np.allclose(mass[r, :, s], L / n, atol=1e-14)
        assert np.allclose(mass[r, :, 3], (c + 1) / n, atol=1e-14)
        for h in range(4):
            mean = (Vcat[:, h // 2].sum(0) + vn[:c + 1, h // 2].double().sum(0)) / n
            assert np.abs(out[r, h] - mean.numpy()).max() < 1e-13


def test_two_way_softmax():
    D = 16
    ks, vs, q, kn, vn = rand_case(8, 1, 1, D, [1], 1, 1)
    out, mass = orc.attend_slots(1, 1, D, ks, vs, q, kn, vn)
    sg = float((q[0, 0].double() * ks[0][0, 0].double()).sum()) / math.sqrt(D)
    sn = float((q[0, 0].double() * kn[0, 0].double()).sum()) / math.sqrt(D)
    pg = 1.0 / (1.0 + math.exp(sn - sg))
    assert abs(mass[0, 0, 0] - pg) < 1e-14 and abs(mass[0, 0, 1] - (1 - pg)) < 1e-14
    ref = pg * vs[0][0, 0].double().numpy() + (1 - pg) * vn[0, 0].double().numpy()
    assert np.abs(out[0, 0] - ref).max() < 1e-14


def test_one_hot_when_one_score_dominates():
    D = 4
    q = bf16(torch.tensor([[[64.0, 0, 0, 0]]]))                        # [1, 1, 4]
    kg = bf16(torch.tensor([[[0.0, 1, 0, 0]], [[32.0, 0, 0, 0]], [[0.0, 0, 1, 0]]]))  # key 1: score 1024
    vg = bf16(torch.tensor([[[1.0, 2, 3, 4]], [[5.0, 6, 7, 8]], [[9.0, 10, 11, 12]]]))
    kn = bf16(torch.zeros(1, 1, D))
    vn = bf16(torch.ones(1, 1, D))
    out, mass = orc.attend_slots(1, 1, D, [kg[:1], kg[1:]], [vg[:1], vg[1:]], q, kn, vn)
    assert np.array_equal(out[0, 0], np.array([5.0, 6, 7, 8]))
    assert np.array_equal(mass[0, 0], np.array([0.0, 1.0, 0.0]))


# ---- 6. O <-> mass tie --------------------------------------------------------------------
def test_indicator_values_tie_output_to_mass():
    lens = [4, 9, 2]
    D = 8
    ks, vs, q, kn, vn = rand_case(9, 4, 2, D, lens, 6, 6)
    vs = [torch.zeros_like(v) for v in vs]
    for s in range(3):
        vs[s][:, :, s] = 1
    vn = torch.zeros_like(vn)
    vn[:, :, 3] = 1
    out, mass = orc.attend_slots(4, 2, D, ks, vs, q, kn, vn)
    assert np.abs(out[:, :, :4] - mass).max() < 1e-14
    assert np.abs(out[:, :, 4:]).max() == 0


# ---- 7. prefill row == decode call --------------------------------------------------------
def test_prefill_row_equals_decode_call():
    ks, vs, q, kn, vn = rand_case(10, 8, 2, 32, [6, 20], 9, 9)
    out, mass = orc.attend_slots(8, 2, 32, ks, vs, q, kn, vn)
    for r in (0, 4, 8):
        o1, m1 = orc.attend_slots(8, 2, 32, ks, vs, q[r:r + 1], kn[:r + 1], vn[:r + 1])
        assert np.abs(o1[0] - out[r]).max() < 1e-14
        assert np.abs(m1[0] - mass[r]).max() < 1e-14


def test_row_subset_equals_full():
    ks, vs, q, kn, vn = rand_case(12, 4, 2, 16, [6, 20], 9, 12)
    out, mass = orc.attend_slots(4, 2, 16, ks, vs, q, kn, vn)
    rows = [8, 0, 3]
    o2, m2 = orc.attend_slots(4, 2, 16, ks, vs, q, kn, vn, rows=rows)
    assert np.array_equal(o2, out[rows]) and np.array_equal(m2, mass[rows])


# ---- GQA mapping, scaling and transposition would each break these ------------------------
def test_gqa_head_mapping_is_contiguous_blocks():
    """q heads 0..rep-1 read kv head 0, the next rep read kv head 1 (h // rep)."""
    Hq, Hkv, D = 4, 2, 8
    ks, vs, q, kn, vn = rand_case(13, Hq, Hkv, D, [5], 3, 3)
    out, _ = orc.attend_slots(Hq, Hkv, D, ks, vs, q, kn, vn)
    for h in range(Hq):
        kv = h // 2
        o1, _ = orc.attend_slots(1, 1, D, [ks[0][:, kv:kv + 1]], [vs[0][:, kv:kv + 1]],
                                 q[:, h:h + 1], kn[:, kv:kv + 1], vn[:, kv:kv + 1])
        assert np.abs(o1[:, 0] - out[:, h]).max() < 1e-14


# ---- 9. book-keeping ----------------------------------------------------------------------
def test_sel_off_against_handwritten_prefix():
    assert list(orc.sel_off([])) == [0]
    assert list(orc.sel_off([5])) == [0, 5]
    assert list(orc.sel_off([40, 120, 0, 77])) == [0, 40, 160, 160, 237]


def test_appendix_c_layout_fixture():
    """App. C: a map of 3 object groups of which groups 2 and 3 are selected, followed by the
    instruction and trajectory.  The paper gives the layout, not token counts; the lengths in
    the fixture are made up.  Values were written by tests/golden/make_golden.py (oracle only)."""
    path = os.path.join(HERE, "golden", "appc_3groups.txt")
    vals = {}
    with open(path) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            k, v = line.split("=", 1)
            vals[k.strip()] = v.strip()
    from tests.golden.make_golden import appc_case
    cache, sel, q, kn, vn = appc_case()
    out, mass, off = cache.attend(0, sel, q, kn, vn)
    assert sel == [1, 2]                                   # zero-based ids of "Group 2, Group 3"
    assert [int(x) for x in vals["sel_off"].split()] == list(off)
    assert mass.shape[-1] == 3                             # two groups + the new tokens
    got = np.array([float.fromhex(x) for x in vals["mass_row_last_head0"].split()])
    assert np.array_equal(got, mass[-1, 0])
    got = np.array([float.fromhex(x) for x in vals["out_row_last_head0_first4"].split()])
    assert np.array_equal(got, out[-1, 0, :4])


def test_append_concatenates_at_end():
    """Sec. 3.2: new objects are concatenated at the end of the group; old rows untouched."""
    c = orc.OracleCache(1, 2, 1, 8)
    g = torch.Generator().manual_seed(1)
    k1, v1 = bf16(torch.randn(3, 1, 8, generator=g)), bf16(torch.randn(3, 1, 8, generator=g))
    k2, v2 = bf16(torch.randn(2, 1, 8, generator=g)), bf16(torch.randn(2, 1, 8, generator=g))
    q, kn, vn = (bf16(torch.randn(2, 2, 8, generator=g)), bf16(torch.randn(2, 1, 8, generator=g)),
                 bf16(torch.randn(2, 1, 8, generator=g)))
    c.group_store(0, 0, k1, v1)
    c.group_store(0, 0, k2, v2, append=True)
    assert c.group_len(0, 0) == 5
    o, m, off = c.attend(0, [0], q, kn, vn)
    o2, m2 = orc.attend_slots(2, 1, 8, [torch.cat([k1, k2])], [torch.cat([v1, v2])], q, kn, vn)
    assert np.array_equal(o, o2) and np.array_equal(m, m2) and list(off) == [0, 5]
