"""GPU parity, small shapes: the CUDA library (through the C ABI) against the float64 oracle,
element by element, on sizes that span several tiles and ragged tails."""
import numpy as np
import pytest
import torch

from paper_2510_18546_b200 import enl, synth
from tests.helpers import Session, check_close

pytestmark = pytest.mark.gpu


def run_case(wl, split_hint=0, layer=0, expect_merge=None):
    with Session(wl, [layer]) as s:
        q, kn, vn = wl.new_qkv(layer, s.device)
        out, mass, sel_off = s.attend(0, q, kn, vn, split_hint=split_hint)
        torch.cuda.synchronize()
        assert enl.enl_cache_status(s.cache) == enl.ENL_OK
        if expect_merge is not None:
            assert enl.enl_plan_inspect(s.cache)["merge_kind"] == expect_merge
        cs, cq, cn = wl.cu()
        so = 0
        for b in range(wl.batch):
            qo, mo, off = s.oracle(0, b, q[cq[b]:cq[b + 1]], kn[cn[b]:cn[b + 1]], vn[cn[b]:cn[b + 1]])
            G = len(wl.sel_local[b])
            check_close(out[cq[b]:cq[b + 1]], qo, mass[cq[b]:cq[b + 1], :, :G + 1], mo,
                        what=f"{wl.name} ep{b} split{split_hint}")
            assert list(sel_off[so:so + G + 1]) == [int(x) for x in off]      # bit-exact book-keeping
            so += G + 1
            rs = mass[cq[b]:cq[b + 1], :, :G + 1].sum(-1)
            assert (rs - 1).abs().max().item() < 1e-3


def test_tiny_config():
    run_case(synth.make("tiny"))


@pytest.mark.parametrize("split", [2, 3])
def test_tiny_config_kv_split(split):
    run_case(synth.make("tiny"), split_hint=split)


SMALL = {
    # ragged groups, several tiles, rows not a multiple of the CTA's 64 tokens
    "ragged_d128": dict(Hq=8, Hkv=2, D=128, pool=[[1, 50, 16, 33, 7, 120, 15, 17]], sel=[[5, 0, 3, 7, 1]],
                        n_q=[77], n_new=[77]),
    "ragged_d64": dict(Hq=8, Hkv=2, D=64, pool=[[9, 31, 64, 2]], sel=[[3, 2, 1, 0]], n_q=[130], n_new=[130]),
    # queries aligned with the LAST new keys (chunked prefill / multi-token decode)
    "nq_lt_nnew": dict(Hq=8, Hkv=2, D=128, pool=[[40, 41, 42]], sel=[[2, 0]], n_q=[5], n_new=[200]),
    "empty_select": dict(Hq=4, Hkv=1, D=128, pool=[[10]], sel=[[]], n_q=[150], n_new=[150]),
    "one_decode_token": dict(Hq=32, Hkv=8, D=128, pool=[[300, 17, 256]], sel=[[0, 1, 2]], n_q=[1], n_new=[1]),
    "decode_grown": dict(Hq=32, Hkv=8, D=128, pool=[[300, 17, 256]], sel=[[2, 0]], n_q=[1], n_new=[37]),
    "rep1": dict(Hq=2, Hkv=2, D=64, pool=[[20, 20]], sel=[[1, 0]], n_q=[140], n_new=[140]),
    "rep8": dict(Hq=8, Hkv=1, D=128, pool=[[20, 45]], sel=[[0, 1]], n_q=[40], n_new=[40]),
    # one query token per episode: the streaming decode kernel
    "decode_batch": dict(Hq=8, Hkv=2, D=128, pool=[[30, 60, 90], [5, 5, 5, 5], [200]],
                         sel=[[2, 0], [0, 1, 2, 3], []], n_q=[1, 1, 1], n_new=[1, 10, 129]),
    "decode_d64_rep8": dict(Hq=8, Hkv=1, D=64, pool=[[20, 45, 300]], sel=[[0, 1, 2]], n_q=[1], n_new=[33]),
    "decode_rep1": dict(Hq=2, Hkv=2, D=64, pool=[[20, 0, 20]], sel=[[2, 1, 0]], n_q=[1], n_new=[16]),
    "decode_many_pages": dict(Hq=16, Hkv=4, D=128, pool=[[1500, 700, 16, 1, 2300]], sel=[[4, 3, 0, 2, 1]],
                              n_q=[1], n_new=[17]),
    "varlen_batch": dict(Hq=8, Hkv=2, D=128, pool=[[30, 60, 90], [5, 5, 5, 5], [200]],
                         sel=[[2, 0], [0, 1, 2, 3], []], n_q=[70, 3, 129], n_new=[70, 10, 129]),
}


@pytest.mark.parametrize("name", sorted(SMALL))
@pytest.mark.parametrize("split", [0, 2, 5])
def test_small_shapes(name, split):
    c = SMALL[name]
    wl = synth.make_small(7, 1, c["Hq"], c["Hkv"], c["D"], c["pool"], c["sel"], c["n_q"], c["n_new"], name=name)
    run_case(wl, split_hint=split)


# Two KV splits of a head_dim-128 call are merged by pairs of CTAs inside the attention kernel.  The slot in which
# the splits meet is credited by both: inside a group, on a group boundary, inside the new tokens.
PAIR = {
    "meet_inside_slot": dict(Hq=8, Hkv=2, D=128, pool=[[300, 40]], sel=[[0, 1]], n_q=[64], n_new=[64]),
    "meet_on_boundary": dict(Hq=8, Hkv=2, D=128, pool=[[128, 128, 5]], sel=[[0, 1]], n_q=[30], n_new=[30]),
    "meet_in_new_tokens": dict(Hq=8, Hkv=2, D=128, pool=[[100]], sel=[[0]], n_q=[400], n_new=[400]),
    "one_q_tile_zero_len_group": dict(Hq=8, Hkv=2, D=128, pool=[[128, 0, 130]], sel=[[0, 1, 2]], n_q=[20], n_new=[20]),
    "rep1_many_rows": dict(Hq=2, Hkv=2, D=128, pool=[[70, 90, 11]], sel=[[2, 1, 0]], n_q=[300], n_new=[333]),
    "batch_of_three": dict(Hq=8, Hkv=2, D=128, pool=[[30, 60, 90], [5, 5, 250], [200]],
                           sel=[[2, 0], [0, 1, 2], [0]], n_q=[70, 3, 129], n_new=[70, 10, 129]),
}


@pytest.mark.parametrize("name", sorted(PAIR))
def test_pair_merge(name):
    c = PAIR[name]
    wl = synth.make_small(11, 1, c["Hq"], c["Hkv"], c["D"], c["pool"], c["sel"], c["n_q"], c["n_new"], name=name)
    run_case(wl, split_hint=2, expect_merge=2)


def test_pair_merge_without_mass_and_twice_in_a_row():
    """No mass buffer: the slot book-keeping of the pair has nowhere to write.  The second call reuses the plan and
    the barriers' fresh state of a new launch."""
    c = PAIR["meet_inside_slot"]
    wl = synth.make_small(12, 1, c["Hq"], c["Hkv"], c["D"], c["pool"], c["sel"], c["n_q"], c["n_new"], name="pair_nomass")
    with Session(wl, [0]) as s:
        q, kn, vn = wl.new_qkv(0, s.device)
        qo, _, _ = s.oracle(0, 0, q, kn, vn)
        for _ in range(2):
            out, mass, _ = s.attend(0, q, kn, vn, split_hint=2, want_mass=False)
            torch.cuda.synchronize()
            assert mass is None and enl.enl_cache_status(s.cache) == enl.ENL_OK
            assert enl.enl_plan_inspect(s.cache)["merge_kind"] == 2
            check_close(out, qo, None, None, what="pair merge without mass")


def test_split_merge_kinds():
    c = SMALL["ragged_d128"]
    wl = synth.make_small(7, 1, c["Hq"], c["Hkv"], c["D"], c["pool"], c["sel"], c["n_q"], c["n_new"], name="kinds")
    run_case(wl, split_hint=1, expect_merge=0)
    run_case(wl, split_hint=3, expect_merge=1)
    c = SMALL["empty_select"]                       # one tile only: nothing for a second CTA of a pair to do
    wl = synth.make_small(7, 1, c["Hq"], c["Hkv"], c["D"], c["pool"], c["sel"], c["n_q"], c["n_new"], name="kinds1")
    run_case(wl, split_hint=2, expect_merge=0)
    c = SMALL["decode_grown"]
    wl = synth.make_small(7, 1, c["Hq"], c["Hkv"], c["D"], c["pool"], c["sel"], c["n_q"], c["n_new"], name="kinds2")
    run_case(wl, split_hint=0, expect_merge=3)


def test_store_all_layers_equals_layer_by_layer_stores():
    """Every layer of a group written by one launch (replace, then append) reads back exactly as the same rows
    written layer by layer."""
    wl = synth.make_small(21, 3, 8, 2, 128, [[70, 33, 5]], [[1, 0, 2]], [40], [40], name="all_layers")
    dev = torch.device("cuda:0")
    caches = [enl.enl_cache_create(3, 8, 2, 128, wl.n_groups, wl.pool_tokens + 64, device=0, max_batch=1,
                                   max_q_tokens=40) for _ in range(2)]
    try:
        kv = [wl.pool_kv(layer, 0, dev) for layer in range(3)]
        offs = wl.pool_offsets(0)
        for g in range(3):
            a, b = int(offs[g]), int(offs[g + 1])
            cut = a + (b - a) // 2                      # first half stored, second half appended
            for layer in range(3):
                enl.enl_group_store(caches[0], g, layer, kv[layer][0][a:cut], kv[layer][1][a:cut])
                enl.enl_group_store(caches[0], g, layer, kv[layer][0][cut:b], kv[layer][1][cut:b], mode=enl.ENL_APPEND)
            enl.enl_group_store_all_layers(caches[1], g, [kv[l][0][a:cut] for l in range(3)],
                                           [kv[l][1][a:cut] for l in range(3)])
            enl.enl_group_store_all_layers(caches[1], g, [kv[l][0][cut:b] for l in range(3)],
                                           [kv[l][1][cut:b] for l in range(3)], mode=enl.ENL_APPEND)
        sel = wl.sel_ids()
        for layer in range(3):
            q, kn, vn = wl.new_qkv(layer, dev)
            res = []
            for c in caches:
                out = torch.empty_like(q)
                mass = torch.full((40, 8, len(sel) + 1), float("nan"), dtype=torch.float32, device=dev)
                enl.enl_attend(c, layer, sel, q, kn, vn, out, mass)
                res.append((out, mass))
            torch.cuda.synchronize()
            assert torch.equal(res[0][0], res[1][0]) and torch.equal(res[0][1], res[1][1])
            assert [enl.enl_group_len(caches[1], g, layer) for g in range(3)] == [70, 33, 5]
    finally:
        for c in caches:
            enl.enl_cache_free(c)


def test_store_all_layers_beyond_one_launch():
    """More than 64 pages and more than 64 layers: the store is cut into several launches."""
    n_layers, n_tok = 66, 1100
    dev = torch.device("cuda:0")
    gen = torch.Generator(device=dev).manual_seed(5)
    ks = [torch.randn(n_tok, 1, 64, generator=gen, device=dev).to(torch.bfloat16) for _ in range(n_layers)]
    vs = [torch.randn(n_tok, 1, 64, generator=gen, device=dev).to(torch.bfloat16) for _ in range(n_layers)]
    q = torch.randn(7, 2, 64, generator=gen, device=dev).to(torch.bfloat16)
    kn = torch.randn(7, 1, 64, generator=gen, device=dev).to(torch.bfloat16)
    vn = torch.randn(7, 1, 64, generator=gen, device=dev).to(torch.bfloat16)
    caches = [enl.enl_cache_create(n_layers, 2, 1, 64, 2, 1200, device=0, max_batch=1, max_q_tokens=7) for _ in range(2)]
    try:
        for layer in range(n_layers):
            enl.enl_group_store(caches[0], 1, layer, ks[layer], vs[layer])
        enl.enl_group_store_all_layers(caches[1], 1, ks, vs)
        for layer in (0, 63, 64, 65):
            res = []
            for c in caches:
                out = torch.empty_like(q)
                mass = torch.full((7, 2, 2), float("nan"), dtype=torch.float32, device=dev)
                enl.enl_attend(c, layer, [1], q, kn, vn, out, mass)
                res.append((out, mass))
            torch.cuda.synchronize()
            assert torch.equal(res[0][0], res[1][0]) and torch.equal(res[0][1], res[1][1])
            assert torch.isfinite(res[1][1]).all()
    finally:
        for c in caches:
            enl.enl_cache_free(c)


def test_zero_length_group_has_zero_mass():
    wl = synth.make_small(8, 1, 8, 2, 64, [[12, 0, 20]], [[0, 1, 2]], [33], [33], name="zero_len")
    with Session(wl, [0]) as s:
        q, kn, vn = wl.new_qkv(0, s.device)
        out, mass, sel_off = s.attend(0, q, kn, vn)
        torch.cuda.synchronize()
        assert list(sel_off) == [0, 12, 12, 32]
        assert mass[:, :, 1].abs().max().item() == 0.0
        qo, mo, _ = s.oracle(0, 0, q, kn, vn)
        check_close(out, qo, mass, mo, what="zero_len")


def test_select_order_permutes_mass_only():
    wl = synth.make_small(9, 1, 8, 2, 128, [[33, 70, 18, 5]], [[0, 1, 2, 3]], [64], [64], name="perm")
    with Session(wl, [0]) as s:
        q, kn, vn = wl.new_qkv(0, s.device)
        o1, m1, _ = s.attend(0, q, kn, vn)
        perm = [2, 0, 3, 1]
        o2, m2, off2 = s.attend(0, q, kn, vn, sel_override=perm)
        torch.cuda.synchronize()
        assert list(off2) == [0, 18, 51, 56, 126]
        assert (o1.float() - o2.float()).abs().max().item() <= 2e-2
        assert (m1[..., perm] - m2[..., :4]).abs().max().item() <= 1e-3
        assert (m1[..., 4] - m2[..., 4]).abs().max().item() <= 1e-3


def test_append_keeps_existing_rows():
    """Sec. 3.2: rows appended at the end of a group; a later attend sees old + new rows in order."""
    wl = synth.make_small(10, 1, 8, 2, 128, [[45, 30]], [[0, 1]], [20], [20], name="append")
    with Session(wl, [0], extra_tokens=64) as s:
        g = torch.Generator(device=s.device).manual_seed(3)
        ka = (torch.randn(21, 2, 128, generator=g, device=s.device)).to(torch.bfloat16)
        va = (torch.randn(21, 2, 128, generator=g, device=s.device)).to(torch.bfloat16)
        enl.enl_group_store(s.cache, 0, 0, ka, va, mode=enl.ENL_APPEND)
        assert enl.enl_group_len(s.cache, 0, 0) == 66
        ks, vs = s.host_kv[(0, 0)]
        s.host_kv[(0, 0)] = ([torch.cat([ks[0], ka.cpu()]), ks[1]], [torch.cat([vs[0], va.cpu()]), vs[1]])
        q, kn, vn = wl.new_qkv(0, s.device)
        out, mass, sel_off = s.attend(0, q, kn, vn)
        torch.cuda.synchronize()
        assert list(sel_off) == [0, 66, 96]
        qo, mo, _ = s.oracle(0, 0, q, kn, vn)
        check_close(out, qo, mass, mo, what="append")


def _crafted_jump(k_second: float):
    """Two 128-token groups: zero keys in the first, constant keys in the second, so that every score of the
    second KV tile exceeds every score of the first by q.k/sqrt(D) = 16 * k_second * 128 / sqrt(128)."""
    dev = torch.device("cuda:0")
    Hq, Hkv, D, n = 8, 2, 128, 40
    g = torch.Generator(device=dev).manual_seed(5)
    k0 = torch.zeros(128, Hkv, D, dtype=torch.bfloat16, device=dev)
    k1 = torch.full((128, Hkv, D), k_second, dtype=torch.bfloat16, device=dev)
    v0 = torch.randn(128, Hkv, D, generator=g, device=dev).to(torch.bfloat16)
    v1 = torch.randn(128, Hkv, D, generator=g, device=dev).to(torch.bfloat16)
    q = torch.full((n, Hq, D), 16.0, dtype=torch.bfloat16, device=dev)
    kn = torch.zeros(n, Hkv, D, dtype=torch.bfloat16, device=dev)
    vn = torch.randn(n, Hkv, D, generator=g, device=dev).to(torch.bfloat16)
    cache = enl.enl_cache_create(1, Hq, Hkv, D, 2, 256, device=0, max_q_tokens=64)
    try:
        enl.enl_group_store(cache, 0, 0, k0, v0)
        enl.enl_group_store(cache, 1, 0, k1, v1)
        out = torch.empty_like(q)
        mass = torch.zeros(n, Hq, 3, dtype=torch.float32, device=dev)
        enl.enl_attend(cache, 0, [0, 1], q, kn, vn, out, mass)
        torch.cuda.synchronize()
        status = enl.enl_cache_status(cache)
    finally:
        enl.enl_cache_free(cache)
    from oracle import enl_oracle as orc
    ro, rm = orc.attend_slots(Hq, Hkv, D, [k0.cpu(), k1.cpu()], [v0.cpu(), v1.cpu()], q.cpu(), kn.cpu(), vn.cpu())
    return status, out, mass, ro, rm


@pytest.mark.parametrize("k_second,jump", [(0.25, 65), (0.5, 130)])
def test_a_large_jump_of_the_row_maximum_is_exact(k_second, jump):
    """The second key tile beats the first by 65 / 130 log2 units: far beyond the lazy-rescale threshold (and, at
    130, beyond what one fp32 rescale factor can carry: the first tile's contribution underflows to exactly 0, as
    it does in the float64 oracle to within 1e-39)."""
    status, out, mass, ro, rm = _crafted_jump(k_second)     # 16 * k * 128 / sqrt(128) * log2(e) = 65.3 / 130.6
    assert status == enl.ENL_OK
    check_close(out, ro, mass, rm, what=f"jump {jump}")
    assert mass[:, :, 0].abs().max().item() < 1e-6 and (mass[:, :, 1] - 1).abs().max().item() < 1e-3


def test_padding_left_by_a_longer_version_of_the_group_is_harmless():
    """ENL_REPLACE to a shorter length leaves the group's last page partly used.  Whatever the longer version held
    in the rows behind the new end (here NaN bit patterns) must not reach the result: padded keys get probability
    0, and 0 x NaN would still be NaN inside the P V product, so the store clears those rows."""
    wl = synth.make_small(61, 1, 8, 2, 128, [[37, 50]], [[0, 1]], [40], [40], name="stale_padding")
    with Session(wl, [0], extra_tokens=64) as s:
        dev = s.device
        poison = torch.full((48, 2, 128), float("nan"), dtype=torch.bfloat16, device=dev)
        k, v = wl.pool_kv(0, 0, dev)
        offs = wl.pool_offsets(0)
        for g in range(2):                                   # a longer, all-NaN version first, then the real rows
            enl.enl_group_store(s.cache, g, 0, poison, poison)
            enl.enl_group_store(s.cache, g, 0, k[offs[g]:offs[g + 1]], v[offs[g]:offs[g + 1]])
        assert [enl.enl_group_len(s.cache, g, 0) for g in range(2)] == [37, 50]
        q, kn, vn = wl.new_qkv(0, dev)
        for split in (0, 2):                                 # the direct path and the pair merge
            out, mass, _ = s.attend(0, q, kn, vn, split_hint=split)
            torch.cuda.synchronize()
            assert enl.enl_cache_status(s.cache) == enl.ENL_OK
            ro, rm, _ = s.oracle(0, 0, q, kn, vn)
            check_close(out, ro, mass, rm, what=f"stale padding split {split}")
        out1, mass1, _ = s.attend(0, q[-1:], kn, vn, n_q=[1], n_new=[40])      # the one-token decode kernel
        torch.cuda.synchronize()
        ro1, rm1, _ = s.oracle(0, 0, q[-1:], kn, vn)
        check_close(out1, ro1, mass1, rm1, what="stale padding decode")
        # append into the partly used page: the rows behind the new end are cleared again
        enl.enl_group_store(s.cache, 0, 0, poison, poison)
        enl.enl_group_store(s.cache, 0, 0, k[offs[0]:offs[0] + 20], v[offs[0]:offs[0] + 20])
        enl.enl_group_store(s.cache, 0, 0, k[offs[0] + 20:offs[1]], v[offs[0] + 20:offs[1]], mode=enl.ENL_APPEND)
        out, mass, _ = s.attend(0, q, kn, vn)
        torch.cuda.synchronize()
        check_close(out, ro, mass, rm, what="stale padding after append")


def test_split_that_sees_no_key_after_calls_that_left_other_data_in_the_scratch():
    """Eight zero-length groups come first, so the first 128-key tile of the stream holds no key at all, and with
    three splits over five tiles the first split is exactly that tile: its log-sum-exp is -inf and its weight in
    the merge is 0.  The scratch buffer is never cleared; the calls before (another split count, a one-token decode
    call) leave -inf and unrelated partial results where this call's partial outputs go."""
    wl = synth.make_small(71, 1, 8, 2, 128, [[0] * 8 + [300, 40]], [list(range(10))], [64], [64], name="empty_split")
    with Session(wl, [0]) as s:
        q, kn, vn = wl.new_qkv(0, s.device)
        ro, rm, _ = s.oracle(0, 0, q, kn, vn)
        ro1, rm1, _ = s.oracle(0, 0, q[-1:], kn, vn)
        for split in (5, 1):
            out, mass, _ = s.attend(0, q, kn, vn, split_hint=split)
            torch.cuda.synchronize()
            check_close(out, ro, mass, rm, what=f"empty first tile, split {split}")
        out1, mass1, _ = s.attend(0, q[-1:], kn, vn, n_q=[1], n_new=[64])
        torch.cuda.synchronize()
        check_close(out1, ro1, mass1, rm1, what="empty first tile, decode")
        out, mass, _ = s.attend(0, q, kn, vn, split_hint=3)
        torch.cuda.synchronize()
        assert enl.enl_cache_status(s.cache) == enl.ENL_OK
        p = enl.enl_plan_inspect(s.cache)
        assert p["merge_kind"] == 1 and p["n_splits"] == 3
        check_close(out, ro, mass, rm, what="empty first tile, split 3")
        assert mass[:, :, :8].abs().max().item() == 0.0          # zero-length groups: mass exactly 0
