"""The slow tier (Sec. 3.2: all group K/V lives in slow memory, the selected groups are loaded once per planning
step; Sec. 3.4: groups selected in two adjacent steps are already loaded = cache hits)."""
import numpy as np
import pytest
import torch

from oracle import enl_oracle as orc
from paper_2510_18546_b200 import build as enl_build
from paper_2510_18546_b200 import enl


@pytest.fixture(scope="module", autouse=True)
def _built():
    enl_build.build_library()


def test_tier_model_by_hand():
    """The reference model itself, on a trace worked out by hand: six device pages, groups of two pages."""
    m = orc.TierModel(6)
    m.store(0, 32), m.store(1, 32), m.store(2, 20)
    assert m.free == 0
    assert m.prepare([0, 1]) == ([0, 1], [], [])                       # both resident: two hits
    m.evict(1)
    m.store(3, 30)
    assert m.free == 0 and not m.resident[1]
    # group 1 must come back: 0 was selected in step 1, 2 and 3 never -> the lower id of those goes first
    assert m.prepare([1]) == ([], [1], [2])
    assert m.prepare([2, 0]) == ([0], [2], [3])                        # 1 was used more recently than 3
    assert [m.resident[g] for g in range(4)] == [True, True, True, False]


def test_residency_counts_follow_the_model():
    """Book-keeping only (no device): hits, misses, LRU evictions and bytes equal the plain model step by step."""
    rng = np.random.default_rng(3)
    n_groups = 12
    lens = [int(x) for x in rng.integers(10, 90, size=n_groups)]
    pages = [-(-n // 16) for n in lens]
    max_tokens = 16 * (sum(sorted(pages)[-5:]) - n_groups + 2)           # room for about five groups
    dev_pages = -(-max_tokens // 16) + n_groups                          # the pool: ceil(max_tokens / 16) + max_groups pages
    c = enl.enl_cache_create(1, 8, 2, 64, max_groups=n_groups, max_tokens=max_tokens, device=enl.ENL_DEVICE_NONE)
    model = orc.TierModel(dev_pages)
    page_bytes = 2 * 16 * 64 * 2                                         # kv heads x tokens x head_dim x bf16
    try:
        enl.enl_tier_enable(c, sum(lens))
        for g, n in enumerate(lens):
            while model.free < pages[g]:                                  # make room the way a caller would
                victim = min(x for x in model.pages if model.resident[x])
                model.evict(victim)
                enl.enl_group_evict(c, victim)
            enl.enl_group_store(c, g, 0, None, None, n_tokens=n)
            model.store(g, n)
        total_hits = total_sel = 0
        for step in range(60):
            k = int(rng.integers(1, 5))
            sel = [int(x) for x in rng.choice(n_groups, size=k, replace=False)]
            hits, misses, evicted = model.prepare(sel)
            got = enl.enl_step_prepare(c, sel)
            assert (got["n_hit"], got["n_miss"], got["n_evicted"]) == (len(hits), len(misses), len(evicted)), (step, sel)
            assert [enl.enl_group_resident(c, g) for g in range(n_groups)] == [int(model.resident[g]) for g in range(n_groups)]
            assert got["bytes_h2d"] == 2 * page_bytes * sum(pages[g] for g in misses)
            off = enl.enl_attend(c, 0, sel, None, None, None, None, n_q=1, n_new=1, want_sel_off=True, flags=enl.ENL_PLAN_ONLY)
            assert list(off) == [int(x) for x in orc.sel_off([lens[g] for g in sel])]
            total_hits += len(hits)
            total_sel += len(sel)
        assert 0 < total_hits < total_sel                                 # the trace has both hits and misses
    finally:
        enl.enl_cache_free(c)


def test_evicted_group_is_refused_until_prepared():
    c = enl.enl_cache_create(1, 8, 2, 64, max_groups=4, max_tokens=200, device=enl.ENL_DEVICE_NONE)
    try:
        with pytest.raises(enl.EnlError):
            enl.enl_group_evict(c, 0)                                     # no slow tier yet
        enl.enl_tier_enable(c, 200)
        enl.enl_group_store(c, 0, 0, None, None, n_tokens=50)
        enl.enl_group_store(c, 1, 0, None, None, n_tokens=30)
        enl.enl_group_evict(c, 0)
        assert enl.enl_group_resident(c, 0) == 0 and enl.enl_group_resident(c, 1) == 1
        for call in (lambda: enl.enl_attend(c, 0, [0], None, None, None, None, n_q=1, n_new=1, flags=enl.ENL_PLAN_ONLY),
                     lambda: enl.enl_group_store(c, 0, 0, None, None, mode=enl.ENL_APPEND, n_tokens=3)):
            with pytest.raises(enl.EnlError) as e:
                call()
            assert e.value.code == enl.ENL_E_EVICTED
        st = enl.enl_step_prepare(c, [0, 1])
        assert (st["n_hit"], st["n_miss"], st["n_evicted"]) == (1, 1, 0)
        assert st["bytes_h2d"] == 4 * (2 * 16 * 64 * 2) * 2 and st["bytes_d2h"] == 0
        enl.enl_group_store(c, 0, 0, None, None, mode=enl.ENL_APPEND, n_tokens=3)
        assert enl.enl_group_len(c, 0, 0) == 53
        with pytest.raises(enl.EnlError) as e:
            enl.enl_step_prepare(c, [3])                                  # never stored
        assert e.value.code == enl.ENL_E_NOGROUP
    finally:
        enl.enl_cache_free(c)


@pytest.mark.gpu
def test_evict_and_reload_give_identical_results():
    """Pages travel device -> pinned host -> (other) device pages; attention over the reloaded groups is bit-identical,
    also after an append made while the group was resident, and a hit moves no bytes."""
    from paper_2510_18546_b200 import synth
    from tests.helpers import Session, check_close
    wl = synth.make_small(51, 2, 8, 2, 128, [[45, 100, 33, 70, 16, 5]], [[1, 3, 0, 5]], [48], [48], name="tier")
    with Session(wl, [0, 1], extra_tokens=64) as s:
        enl.enl_tier_enable(s.cache, 600)
        q, kn, vn = wl.new_qkv(0, s.device)
        ref = [s.attend(li, q, kn, vn) for li in (0, 1)]
        torch.cuda.synchronize()
        for g in (3, 1, 5, 2):
            enl.enl_group_evict(s.cache, g)
        assert [enl.enl_group_resident(s.cache, g) for g in range(6)] == [1, 0, 0, 0, 1, 0]
        with pytest.raises(enl.EnlError) as e:
            s.attend(0, q, kn, vn)
        assert e.value.code == enl.ENL_E_EVICTED
        # something else takes the freed pages, so the reload lands on different ones
        g0 = torch.Generator(device=s.device).manual_seed(1)
        kx = torch.randn(60, 2, 128, generator=g0, device=s.device).to(torch.bfloat16)
        enl.enl_group_store(s.cache, 4, 0, kx, kx)
        enl.enl_group_store(s.cache, 4, 1, kx, kx)
        st = enl.enl_step_prepare(s.cache, wl.sel_ids())
        assert (st["n_hit"], st["n_miss"]) == (1, 3)
        pages = sum(-(-int(wl.pool_lens[0][g]) // 16) for g in (1, 3, 5))
        assert st["bytes_h2d"] == pages * (2 * 16 * 128 * 2) * 2 * 2          # pages x page bytes x (K, V) x 2 layers
        for li in (0, 1):
            out, mass, off = s.attend(li, q, kn, vn)
            torch.cuda.synchronize()
            assert torch.equal(out, ref[li][0]) and torch.equal(mass, ref[li][1]) and list(off) == list(ref[li][2])
        st = enl.enl_step_prepare(s.cache, wl.sel_ids())
        assert (st["n_hit"], st["n_miss"], st["bytes_h2d"], st["bytes_d2h"]) == (4, 0, 0, 0)
        # against the oracle as well
        qo, mo, _ = s.oracle(0, 0, q, kn, vn)
        check_close(s.attend(0, q, kn, vn)[0], qo, s.attend(0, q, kn, vn)[1][:, :, :5], mo, what="tier reload")
        assert enl.enl_cache_status(s.cache) == enl.ENL_OK
