"""The rows next to the hot path: the clustering reduce that consumes the group mass (Sec. 3.3), the retrieval
knapsack that produces the select list (Sec. 3.4, Eq. 1-2), and the group-append compute step (Sec. 3.2)."""
import itertools
import math

import numpy as np
import pytest
import torch

from oracle import enl_oracle as orc
from paper_2510_18546_b200 import build as enl_build
from paper_2510_18546_b200 import enl


@pytest.fixture(scope="module", autouse=True)
def _built():
    enl_build.build_library()


# ---- oracle pins (CPU) ---------------------------------------------------------------------------
def test_cluster_oracle_closed_forms():
    rng = np.random.default_rng(0)
    n_q, Hq, G = 12, 4, 5
    # uniform mass 1/(G+1) on every slot: every average equals it, nothing beats a threshold above it
    m = np.full((n_q, Hq, G + 1), 1.0 / (G + 1))
    avg, asg = orc.cluster_assign([m, m], [0, 5, 12], G, 0.5)
    assert np.allclose(avg, 1.0 / (G + 1), atol=1e-15) and list(asg) == [-1, -1]
    # all mass of object 0 on group 3, of object 1 on group 1
    m = np.zeros((n_q, Hq, G + 1))
    m[:5, :, 3] = 1.0
    m[5:, :, 1] = 0.75
    m[5:, :, G] = 0.25                                     # the new-token slot is ignored
    avg, asg = orc.cluster_assign([m], [0, 5, 12], G, 0.6)
    assert avg[0, 3] == 1.0 and avg[1, 1] == 0.75 and list(asg) == [3, 1]
    assert list(orc.cluster_assign([m], [0, 5, 12], G, 0.75)[1]) == [3, -1]      # "exceeds": strictly greater
    # the mean is over rows, heads and layers alike: hand-written loop
    masses = [rng.random((n_q, Hq, G + 2)) for _ in range(3)]
    avg, _ = orc.cluster_assign(masses, [0, 2, 2, 9], G, 2.0)
    want = np.zeros(G)
    for layer in masses:
        for r in range(2, 9):
            for h in range(Hq):
                want += layer[r, h, :G]
    assert np.allclose(avg[2], want / (3 * 7 * Hq), atol=1e-14)
    assert np.all(avg[1] == 0)                             # an object without tokens
    assert np.allclose(orc.cluster_assign(masses[::-1], [0, 2, 2, 9], G, 2.0)[0], avg, atol=1e-14)   # layer order


def test_knapsack_bruteforce_small_cases_by_hand():
    # Eq. 1-2 with threshold 0.5 (values exact in binary): 0.375, 0.25, 0.125, -0.25; sizes 3, 2, 2, 1 MiB
    mib = 1 << 20
    best, arg = orc.knapsack_bruteforce([0.875, 0.75, 0.625, 0.25], 0.5, [3 * mib, 2 * mib, 2 * mib, mib], 4 * mib, mib)
    assert best == 0.375 and set(arg) == {(0,), (1, 2)}            # budget 4 MiB: two ways to the same value
    best, arg = orc.knapsack_bruteforce([0.875, 0.75, 0.625, 0.25], 0.5, [3 * mib, 2 * mib, 2 * mib, mib], 5 * mib, mib)
    assert best == 0.625 and arg == [(0, 1)]
    # sizes round up, the budget rounds down
    best, arg = orc.knapsack_bruteforce([0.9, 0.9], 0.5, [mib + 1, mib], 2 * mib + mib // 2, mib)
    assert arg == [(0,)] or set(arg) == {(0,), (1,)}


# ---- the library against the oracle ------------------------------------------------------------------
@pytest.mark.parametrize("seed", range(8))
def test_knapsack_matches_bruteforce(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 13))
    prob = rng.random(n).astype(np.float32)
    mem = (rng.integers(1, 40, size=n) * 163840).astype(np.int64)       # tokens x 160 KiB per token (40 layers)
    budget = int(rng.integers(0, int(mem.sum()) + 1))
    quantum = 1 << 18
    sel = enl.enl_select_knapsack(prob, 0.45, mem, budget, quantum)
    best, arg = orc.knapsack_bruteforce(prob, 0.45, mem, budget, quantum)
    assert list(sel) == sorted(set(int(x) for x in sel))                # ascending, each group once (x_i in {0,1})
    assert sum(-(-int(mem[i]) // quantum) for i in sel) <= budget // quantum
    val = float(sum(float(prob[i]) - float(np.float32(0.45)) for i in sel))
    assert abs(val - best) < 1e-9
    assert all(prob[i] > np.float32(0.45) for i in sel)


def test_knapsack_edges():
    assert len(enl.enl_select_knapsack([], 0.5, [], 100)) == 0
    assert len(enl.enl_select_knapsack([0.9], 0.5, [10 << 20], 5 << 20)) == 0          # does not fit
    assert list(enl.enl_select_knapsack([0.9, 0.2, 0.8], 0.5, [1 << 20] * 3, 64 << 20)) == [0, 2]
    with pytest.raises(enl.EnlError):
        enl.enl_select_knapsack([0.9], 0.5, [-1], 10)
    with pytest.raises(enl.EnlError):
        enl.enl_select_knapsack([0.9], 0.5, [1], 10, quantum=0)


@pytest.mark.gpu
@pytest.mark.parametrize("n_groups,stride,n_layers", [(5, 6, 1), (24, 25, 4), (130, 131, 2), (1000, 1001, 2)])
def test_cluster_assign_matches_oracle(n_groups, stride, n_layers):
    dev = torch.device("cuda:0")
    g = torch.Generator(device=dev).manual_seed(n_groups)
    n_q, Hq = 96, 8
    masses = []
    for _ in range(n_layers):
        x = torch.rand(n_q, Hq, stride, generator=g, device=dev) ** 4
        masses.append((x / x.sum(-1, keepdim=True)).contiguous())
    obj_off = [0, 7, 7, 40, 41, 96]
    # give two objects a clear winner
    for m in masses:
        m[0:7, :, 3 % n_groups] += 0.5
        m[41:96, :, n_groups - 1] += 0.4
    n_obj = len(obj_off) - 1
    avg = torch.full((n_obj, n_groups), float("nan"), dtype=torch.float32, device=dev)
    asg = torch.full((n_obj,), -7, dtype=torch.int32, device=dev)
    thr = 0.3
    enl.enl_cluster_assign(masses, obj_off, n_groups, thr, avg, asg, stream=torch.cuda.current_stream(dev).cuda_stream)
    torch.cuda.synchronize()
    ravg, rasg = orc.cluster_assign([m.cpu().numpy() for m in masses], obj_off, n_groups, thr)
    assert np.abs(avg.cpu().numpy() - ravg).max() < 2e-6               # fp32 sums of <= 55*8*4 values in [0, 1.5]
    got = asg.cpu().numpy()
    for o in range(n_obj):
        top = np.sort(ravg[o])[::-1]
        clear = abs(top[0] - thr) > 1e-4 and (len(top) < 2 or top[0] - top[1] > 1e-4)
        if clear:
            assert got[o] == rasg[o], (o, got[o], rasg[o])
        else:                                                           # a tie or a value at the threshold: any valid answer
            assert got[o] == -1 or ravg[o, got[o]] >= top[0] - 1e-4
    assert got[0] == 3 % n_groups and got[4] == n_groups - 1 and got[1] == -1


@pytest.mark.gpu
def test_cluster_assign_argument_errors():
    dev = torch.device("cuda:0")
    m = torch.zeros(4, 2, 6, device=dev)
    avg = torch.zeros(1, 5, device=dev)
    asg = torch.zeros(1, dtype=torch.int32, device=dev)
    with pytest.raises(enl.EnlError) as e:
        enl.enl_cluster_assign([m], [0, 9], 5, 0.1, avg, asg)            # span beyond n_q
    assert e.value.code == enl.ENL_E_INVAL
    with pytest.raises(enl.EnlError) as e:
        enl.enl_cluster_assign([m], [3, 1], 5, 0.1, avg, asg)            # descending
    assert e.value.code == enl.ENL_E_INVAL
    with pytest.raises(enl.EnlError) as e:
        enl.enl_cluster_assign([m] * 17, [0, 4], 5, 0.1, avg, asg)       # too many layers for one call
    assert e.value.code == enl.ENL_E_LIMIT
    with pytest.raises(enl.EnlError) as e:
        enl.enl_cluster_assign([m], [0, 4], 7, 0.1, avg, asg)            # more groups than the stride holds
    assert e.value.code == enl.ENL_E_INVAL


@pytest.mark.gpu
def test_group_append_compute_step():
    """Sec. 3.2: "we concatenate the information of new objects at the end of the group ... compute their KV
    cache when the group is selected": the appended tokens attend over the group's existing K/V plus their own
    causal K/V (enl_attend with select = {g}), then their K/V is appended; the existing rows stay untouched,
    which shows as an unchanged result for a query that sees only them."""
    from tests.helpers import Session, check_close
    from paper_2510_18546_b200 import synth
    wl = synth.make_small(41, 1, 8, 2, 128, [[70, 33]], [[0]], [19], [19], name="append_compute")
    with Session(wl, [0], extra_tokens=64) as s:
        q, kn, vn = wl.new_qkv(0, s.device)                  # the 19 appended tokens: their Q and their own K/V
        out, mass, off = s.attend(0, q, kn, vn, sel_override=[0])
        torch.cuda.synchronize()
        ro, rm, roff = s.oracle(0, 0, q, kn, vn)
        check_close(out, ro, mass[:, :, :2], rm, what="append compute")
        assert list(off) == [0, 70]
        # a probe that sees the old rows only: before and after the append of the new K/V
        probe_q, probe_k, probe_v = q[:1], kn[:1] * 0, vn[:1] * 0
        before, _, _ = s.attend(0, probe_q, probe_k, probe_v, n_q=[1], n_new=[1], sel_override=[0])
        enl.enl_group_store(s.cache, 0, 0, kn, vn, mode=enl.ENL_APPEND)
        assert enl.enl_group_len(s.cache, 0, 0) == 89
        after, mass_after, off2 = s.attend(0, probe_q, probe_k, probe_v, n_q=[1], n_new=[1], sel_override=[0])
        torch.cuda.synchronize()
        assert list(off2) == [0, 89]
        ks, vs = s.host_kv[(0, 0)]
        s.host_kv[(0, 0)] = ([torch.cat([ks[0], kn.cpu()])], [torch.cat([vs[0], vn.cpu()])])
        ro2, rm2, _ = s.oracle(0, 0, probe_q, probe_k, probe_v)
        check_close(after, ro2, mass_after[:, :, :2], rm2, what="after append")
        # the first 70 rows still hold what they held: the group's own attention over them has not moved
        wl1 = s.host_kv[(0, 0)]
        ro_old, _ = orc.attend_slots(8, 2, 128, [wl1[0][0][:70]], [wl1[1][0][:70]], probe_q.cpu(), probe_k.cpu(), probe_v.cpu())
        assert np.abs(before.float().cpu().numpy() - ro_old).max() <= 2e-2


@pytest.mark.gpu
@pytest.mark.parametrize("shape", ["few_slots", "many_slots", "batch"])
def test_mass_sums_from_the_attention_kernel_match_the_oracle(shape):
    """Sec. 3.3 consumes only the average mass over an object's tokens, the q heads and the scored layers:
    enl_attend adds the per-object sums itself (group_mass_sum), enl_cluster_assign_sums turns them into
    averages and decisions.  Checked against the oracle's attention + oracle.cluster_assign, over two layers."""
    from tests.helpers import Session
    from paper_2510_18546_b200 import synth
    if shape == "few_slots":            # slots parked in shared memory, one thread per row converts
        wl = synth.make_small(51, 2, 8, 2, 128, [[40, 17, 90, 33]], [[2, 0, 3]], [70], [70], name="sum_few")
        obj_off = [0, 9, 9, 41, 70]
    elif shape == "many_slots":         # slots parked in the mass buffer, the warp converts row by row
        pool = [[5 + (i * 7) % 23 for i in range(40)]]
        wl = synth.make_small(52, 2, 8, 2, 128, pool, [list(range(40))], [100], [100], name="sum_many")
        obj_off = [3, 10, 64, 65, 97]   # rows 0-2 and 97-99 belong to no object
    else:                               # objects of two episodes
        wl = synth.make_small(53, 2, 8, 2, 128, [[30, 60], [5, 5, 250]], [[1, 0], [2, 0]], [40, 50], [40, 50], name="sum_batch")
        obj_off = [0, 40, 60, 90]
    n_obj = len(obj_off) - 1
    with Session(wl, [0, 1]) as s:
        cs, cq, cn = wl.cu()
        G = int(max(len(x) for x in wl.sel_local))
        dev = s.device
        sums = torch.zeros(n_obj, G + 1, dtype=torch.float32, device=dev)
        ref_masses = []
        for li in range(2):
            q, kn, vn = wl.new_qkv(li, dev)
            out = torch.empty_like(q)
            mass = torch.full((q.shape[0], wl.n_q_heads, G + 1), float("nan"), dtype=torch.float32, device=dev)
            enl.enl_attend(s.cache, li, wl.sel_ids(), q, kn, vn, out if li == 0 else None, mass,
                           cu_sel=cs if wl.batch > 1 else None, cu_q=cq if wl.batch > 1 else None,
                           cu_new=cn if wl.batch > 1 else None, n_q=int(cq[-1]), n_new=int(cn[-1]),
                           flags=0 if li == 0 else enl.ENL_MASS_ONLY, group_mass_sum=sums, obj_off=obj_off)
            torch.cuda.synchronize()
            assert enl.enl_cache_status(s.cache) == enl.ENL_OK
            assert enl.enl_plan_inspect(s.cache)["n_splits"] == 1
            rm = np.zeros((q.shape[0], wl.n_q_heads, G + 1))
            for b in range(wl.batch):
                ro, mo, _ = s.oracle(li, b, q[cq[b]:cq[b + 1]], kn[cn[b]:cn[b + 1]], vn[cn[b]:cn[b + 1]])
                rm[cq[b]:cq[b + 1], :, :mo.shape[-1]] = mo
                if li == 0:             # the output is still written without ENL_MASS_ONLY
                    assert np.abs(out[cq[b]:cq[b + 1]].float().cpu().numpy() - ro).max() <= 2e-2
                gm = mass[cq[b]:cq[b + 1], :, :mo.shape[-1]].cpu().numpy()
                assert np.abs(gm - mo).max() <= 1e-3
            ref_masses.append(rm)
        n_groups = G                    # the new-token slot is not a group
        avg = torch.full((n_obj, n_groups), float("nan"), dtype=torch.float32, device=dev)
        asg = torch.full((n_obj,), -7, dtype=torch.int32, device=dev)
        thr = 0.05
        enl.enl_cluster_assign_sums(sums, obj_off, n_groups, wl.n_q_heads, 2, thr, avg, asg)
        torch.cuda.synchronize()
        ravg, rasg = orc.cluster_assign(ref_masses, obj_off, n_groups, thr)
        assert np.abs(avg.cpu().numpy() - ravg).max() < 1e-4, np.abs(avg.cpu().numpy() - ravg).max()
        got = asg.cpu().numpy()
        for o in range(n_obj):
            top = np.sort(ravg[o])[::-1]
            if abs(top[0] - thr) > 1e-3 and (len(top) < 2 or top[0] - top[1] > 1e-3):
                assert got[o] == rasg[o], (o, got[o], rasg[o])


@pytest.mark.gpu
def test_mass_only_and_sum_argument_errors():
    from tests.helpers import Session
    from paper_2510_18546_b200 import synth
    wl = synth.make_small(54, 1, 8, 2, 128, [[40, 17]], [[1, 0]], [20], [20], name="sum_err")
    with Session(wl, [0]) as s:
        q, kn, vn = wl.new_qkv(0, s.device)
        out = torch.empty_like(q)
        mass = torch.zeros(20, 8, 3, dtype=torch.float32, device=s.device)
        sums = torch.zeros(2, 3, dtype=torch.float32, device=s.device)
        with pytest.raises(enl.EnlError) as e:      # ENL_MASS_ONLY without a mass buffer
            enl.enl_attend(s.cache, 0, wl.sel_ids(), q, kn, vn, None, None, flags=enl.ENL_MASS_ONLY)
        assert e.value.code == enl.ENL_E_INVAL
        with pytest.raises(enl.EnlError) as e:      # sums without the per-row masses
            enl.enl_attend(s.cache, 0, wl.sel_ids(), q, kn, vn, out, None, group_mass_sum=sums, obj_off=[0, 5, 20])
        assert e.value.code == enl.ENL_E_INVAL
        with pytest.raises(enl.EnlError) as e:      # spans beyond the query rows
            enl.enl_attend(s.cache, 0, wl.sel_ids(), q, kn, vn, out, mass, group_mass_sum=sums, obj_off=[0, 5, 21])
        assert e.value.code == enl.ENL_E_INVAL
        with pytest.raises(enl.EnlError) as e:      # descending spans
            enl.enl_attend(s.cache, 0, wl.sel_ids(), q, kn, vn, out, mass, group_mass_sum=sums, obj_off=[0, 9, 5])
        assert e.value.code == enl.ENL_E_INVAL


# ---- rotary position helper (Sec. 3.2 cites the embedding; base and pairing are the caller's) ----

def test_rope_oracle_pins():
    """What the mathematics fixes: position 0 is the identity; a pair's norm is kept; the first pair (frequency 1)
    turns by the position itself, counter-clockwise; pair j turns by pos * base^(-2j/D); rotations add up; and the
    property the embedding exists for: <R_m q, R_n k> depends on m - n only."""
    rng = np.random.default_rng(3)
    d = 16
    x = rng.standard_normal((5, 2, d))
    for inter in (False, True):
        pair = (lambda j: (2 * j, 2 * j + 1)) if inter else (lambda j: (j, j + d // 2))
        assert np.array_equal(orc.rope_rotate(x, [0] * 5, 10000.0, inter), x)
        y = orc.rope_rotate(x, [3, 1, 4, 1, 5], 10000.0, inter)
        for j in range(d // 2):
            i1, i2 = pair(j)
            assert np.allclose(y[..., i1] ** 2 + y[..., i2] ** 2, x[..., i1] ** 2 + x[..., i2] ** 2, rtol=1e-12)
        # unit vector along the first channel of a pair: the angle it ends at
        e = np.zeros((1, 1, d))
        for j in (0, 3, d // 2 - 1):
            i1, i2 = pair(j)
            e[:] = 0.0
            e[0, 0, i1] = 1.0
            r = orc.rope_rotate(e, [7], 100.0, inter)
            want = (7.0 * 100.0 ** (-2.0 * j / d)) % (2 * math.pi)
            assert math.isclose(math.atan2(r[0, 0, i2], r[0, 0, i1]) % (2 * math.pi), want, abs_tol=1e-12)
            assert np.count_nonzero(np.abs(r) > 1e-15) <= 2
        a = orc.rope_rotate(orc.rope_rotate(x, [2] * 5, 50.0, inter), [9] * 5, 50.0, inter)
        assert np.allclose(a, orc.rope_rotate(x, [11] * 5, 50.0, inter), atol=1e-12)
        q, k = rng.standard_normal((1, 1, d)), rng.standard_normal((1, 1, d))
        dots = [float((orc.rope_rotate(q, [m], 10000.0, inter) * orc.rope_rotate(k, [n], 10000.0, inter)).sum())
                for m, n in ((5, 2), (13, 10), (3, 0))]
        assert max(dots) - min(dots) < 1e-12
    # the two pairings differ (a transposed pairing would not pass both branches above with the same data)
    assert not np.allclose(orc.rope_rotate(x, [3] * 5, 10000.0, False), orc.rope_rotate(x, [3] * 5, 10000.0, True))


def test_rope_argument_errors():
    enl_build.build_library()
    L = enl.lib()
    assert L.enl_rope_rotate(None, 1, 1, 64, None, 0, 10000.0, 0, None) == enl.ENL_E_INVAL
    assert L.enl_rope_rotate(16, 1, 1, 63, None, 0, 10000.0, 0, None) == enl.ENL_E_INVAL      # odd head_dim
    assert L.enl_rope_rotate(16, 1, 0, 64, None, 0, 10000.0, 0, None) == enl.ENL_E_INVAL
    assert L.enl_rope_rotate(16, 1, 1, 64, None, 0, 0.0, 0, None) == enl.ENL_E_INVAL          # base must be positive
    assert L.enl_rope_rotate(16, 1, 1, 512, None, 0, 10000.0, 0, None) == enl.ENL_E_LIMIT
    assert L.enl_rope_rotate(16, 0, 1, 64, None, 0, 10000.0, 0, None) == enl.ENL_OK           # nothing to do


@pytest.mark.gpu
@pytest.mark.parametrize("d,heads,inter", [(128, 8, False), (128, 8, True), (64, 2, False), (32, 3, True)])
def test_rope_rotate_matches_oracle(d, heads, inter):
    """Rows rotated by the library against the float64 oracle: contiguous positions from a large offset (the angle
    must be reduced in double) and a position list; then stored and attended like any other K."""
    dev = torch.device("cuda:0")
    g = torch.Generator().manual_seed(5)
    n = 77
    x = (torch.randn(n, heads, d, generator=g) * 0.5).to(torch.bfloat16)
    for positions, first in ((None, 100000), (torch.randint(0, 4096, (n,), generator=g).to(torch.int32), 0)):
        rows = x.clone().to(dev)
        pos_host = list(range(first, first + n)) if positions is None else positions.tolist()
        enl.enl_rope_rotate(rows, None if positions is None else positions.to(dev), first_pos=first, base=10000.0,
                            interleaved=inter)
        torch.cuda.synchronize()
        want = orc.rope_rotate(x.double().numpy(), pos_host, 10000.0, inter)
        got = rows.float().cpu().numpy().astype(np.float64)
        # one bf16 rounding of a value of that size, plus fp32 sine / cosine
        assert np.all(np.abs(got - want) <= np.abs(want) * 2.0 ** -8 + 1e-5), np.abs(got - want).max()
