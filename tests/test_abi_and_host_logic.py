"""CPU-only tests of the boundary and of the integer book-keeping: the C-ABI library loads and
exports every symbol that include/enl.h declares, and a bookkeeping-only cache (no device)
reproduces the page table, the select-list prefix sums and the gather plan exactly."""
import os
import re

import numpy as np
import pytest

from oracle import enl_oracle as orc
from paper_2510_18546_b200 import build as enl_build
from paper_2510_18546_b200 import enl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    enl_build.build_library()


def declared_symbols():
    with open(os.path.join(ROOT, "include", "enl.h")) as f:
        text = f.read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(enl_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    L = enl.lib()
    names = declared_symbols()
    assert {"enl_cache_create", "enl_group_store", "enl_attend", "enl_cache_free"} <= set(names)
    for n in names:
        assert hasattr(L, n), f"libenl.so does not export {n}"
    assert set(names) == set(enl.EXPORTS)


def test_strerror_texts():
    assert enl.strerror(enl.ENL_OK) == "ok"
    for code in (enl.ENL_E_INVAL, enl.ENL_E_NOGROUP, enl.ENL_E_NOMEM, enl.ENL_E_CUDA, enl.ENL_E_TIMEOUT):
        assert enl.strerror(code) and enl.strerror(code) != "unknown error"


def host_cache(**kw):
    args = dict(n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=128, max_groups=8, max_tokens=400,
                device=enl.ENL_DEVICE_NONE, max_batch=4, max_q_tokens=1024)
    args.update(kw)
    return enl.enl_cache_create(**args)


def plan(cache, layer, sel, n_q, n_new, **kw):
    return enl.enl_attend(cache, layer, sel, None, None, None, None, n_q=n_q, n_new=n_new,
                          want_sel_off=True, flags=enl.ENL_PLAN_ONLY, **kw)


def test_create_rejects_bad_shapes():
    for kw in (dict(n_q_heads=6), dict(head_dim=96), dict(n_layers=0), dict(max_groups=0), dict(max_tokens=0),
               dict(page_tokens=32), dict(n_q_heads=64, n_kv_heads=2), dict(dtype=7)):
        with pytest.raises(enl.EnlError) as e:
            host_cache(**kw)
        assert e.value.code == enl.ENL_E_INVAL


def test_store_lengths_append_and_replace():
    c = host_cache()
    try:
        assert enl.enl_group_len(c, 3, 0) == -1
        enl.enl_group_store(c, 3, 0, None, None, n_tokens=45)
        assert enl.enl_group_len(c, 3, 0) == 45 and enl.enl_group_len(c, 3, 1) == -1
        enl.enl_group_store(c, 3, 0, None, None, mode=enl.ENL_APPEND, n_tokens=21)      # Sec. 3.2: append at the end
        assert enl.enl_group_len(c, 3, 0) == 66
        enl.enl_group_store(c, 3, 0, None, None, mode=enl.ENL_REPLACE, n_tokens=5)
        assert enl.enl_group_len(c, 3, 0) == 5
        enl.enl_group_store(c, 3, 0, None, None, mode=enl.ENL_APPEND, n_tokens=0)
        assert enl.enl_group_len(c, 3, 0) == 5
        assert enl.enl_group_len(c, 99, 0) == enl.ENL_E_NOGROUP
        with pytest.raises(enl.EnlError) as e:
            enl.enl_group_store(c, 8, 0, None, None, n_tokens=1)
        assert e.value.code == enl.ENL_E_NOGROUP
        with pytest.raises(enl.EnlError) as e:
            enl.enl_group_store(c, 0, 2, None, None, n_tokens=1)
        assert e.value.code == enl.ENL_E_INVAL
    finally:
        enl.enl_cache_free(c)


def test_pool_exhaustion_leaves_state_unchanged():
    c = host_cache(max_tokens=64, max_groups=2)          # 64/16 + 2 groups = 6 usable pages
    try:
        enl.enl_group_store(c, 0, 0, None, None, n_tokens=64)
        with pytest.raises(enl.EnlError) as e:
            enl.enl_group_store(c, 1, 0, None, None, n_tokens=64)
        assert e.value.code == enl.ENL_E_NOMEM
        assert enl.enl_group_len(c, 1, 0) == -1 and enl.enl_group_len(c, 0, 0) == 64
        enl.enl_group_store(c, 1, 0, None, None, n_tokens=32)               # what is left still fits
        enl.enl_group_store(c, 0, 0, None, None, mode=enl.ENL_REPLACE, n_tokens=16)   # frees three pages
        enl.enl_group_store(c, 1, 0, None, None, mode=enl.ENL_APPEND, n_tokens=48)
        assert enl.enl_group_len(c, 1, 0) == 80
    finally:
        enl.enl_cache_free(c)


def test_sel_off_is_the_oracles_prefix_sum_and_follows_list_order():
    c = host_cache()
    lens = [40, 120, 0, 77, 16, 1]
    try:
        for g, n in enumerate(lens):
            for layer in range(2):
                enl.enl_group_store(c, g, layer, None, None, n_tokens=n)
        for sel in ([0, 1, 2, 3], [3, 1], [5, 4, 3, 2, 1, 0], []):
            got = plan(c, 1, sel, 3, 7)
            want = orc.sel_off([lens[g] for g in sel])
            assert got.dtype == np.int32 and list(got) == [int(x) for x in want]
    finally:
        enl.enl_cache_free(c)


def test_gather_plan_stream_matches_page_table_by_hand():
    """Stream entries are (page, slot << 8 | valid tokens) in list order, one null entry for an empty
    group, and null padding up to a multiple of eight entries (one 128-key tile)."""
    c = host_cache()
    try:
        for g, n in enumerate([33, 0, 16, 130]):
            enl.enl_group_store(c, g, 0, None, None, n_tokens=n)
        plan(c, 0, [3, 1, 0], 5, 5)
        p = enl.enl_plan_inspect(c)
        slots = [m >> 8 for m in p["meta"]]
        valid = [m & 0xff for m in p["meta"]]
        # group 3: 130 tokens = 8 full pages + 2; group 1: empty; group 0: 33 = 2 full + 1
        assert valid[:13] == [16] * 8 + [2] + [0] + [16, 16, 1]
        assert slots[:13] == [0] * 9 + [1] + [2] * 3
        assert p["n_entries"] == 16 and valid[13:] == [0, 0, 0] and slots[13:] == [2, 2, 2]
        assert list(p["pages"][13:]) == [0, 0, 0] and p["pages"][9] == 0          # the all-zero page
        used = [int(x) for x in p["pages"][:9]] + [int(x) for x in p["pages"][10:13]]
        assert len(set(used)) == len(used) and 0 not in used                      # distinct real pages
        assert p["ep_cached_tiles"][0] == 2 and p["ep_stream_off"][0] == 0
        # a second group's pages never alias the first's
        plan(c, 0, [2], 5, 5)
        p2 = enl.enl_plan_inspect(c)
        assert p2["n_entries"] == 8 and int(p2["pages"][0]) not in used
    finally:
        enl.enl_cache_free(c)


def test_varlen_batch_plan_and_prefixes():
    c = host_cache()
    lens = [30, 60, 90, 5, 7, 200]
    try:
        for g, n in enumerate(lens):
            enl.enl_group_store(c, g, 0, None, None, n_tokens=n)
        sel = [2, 0, 3, 4, 5]
        got = plan(c, 0, sel, 70 + 3 + 129, 70 + 10 + 129, cu_sel=[0, 2, 4, 5], cu_q=[0, 70, 73, 202],
                   cu_new=[0, 70, 80, 209])
        assert list(got) == [0, 90, 120, 0, 5, 12, 0, 200]
        p = enl.enl_plan_inspect(c)
        assert list(p["ep_stream_off"][:3]) == [0, 8, 16]
        assert list(p["ep_cached_tiles"][:3]) == [1, 1, 2]
        # CTAs: ceil(n_q / 64 tokens) per kv head per episode (rep = 4 -> 32 tokens per Q tile, two tiles)
        assert p["n_items"] == (2 + 1 + 3) * 2 * p["n_splits"]
    finally:
        enl.enl_cache_free(c)


def test_attend_argument_errors():
    c = host_cache()
    try:
        enl.enl_group_store(c, 0, 0, None, None, n_tokens=10)
        enl.enl_group_store(c, 1, 0, None, None, n_tokens=10)
        bad = [
            (dict(sel=[0, 0], n_q=1, n_new=1), enl.ENL_E_INVAL),        # Sec. 3.4: x_i is 0 or 1
            (dict(sel=[7], n_q=1, n_new=1), enl.ENL_E_NOGROUP),         # never stored
            (dict(sel=[8], n_q=1, n_new=1), enl.ENL_E_NOGROUP),         # out of range
            (dict(sel=[0], n_q=5, n_new=4), enl.ENL_E_INVAL),           # more queries than new keys
            (dict(sel=[0], n_q=0, n_new=4), enl.ENL_E_INVAL),
            (dict(sel=[0], n_q=2000, n_new=2000), enl.ENL_E_INVAL),     # beyond max_q_tokens
        ]
        for kw, code in bad:
            with pytest.raises(enl.EnlError) as e:
                plan(c, 0, kw["sel"], kw["n_q"], kw["n_new"])
            assert e.value.code == code, kw
        with pytest.raises(enl.EnlError) as e:                            # stored for layer 0 only
            plan(c, 1, [0], 1, 1)
        assert e.value.code == enl.ENL_E_NOGROUP
        with pytest.raises(enl.EnlError) as e:                            # a GPU call on a bookkeeping cache
            enl.enl_attend(c, 0, [0], None, None, None, None, n_q=1, n_new=1)
        assert e.value.code == enl.ENL_E_CUDA
        # the same id in two different episodes is fine
        got = plan(c, 0, [0, 1, 0], 4, 4, cu_sel=[0, 2, 3], cu_q=[0, 2, 4], cu_new=[0, 2, 4])
        assert list(got) == [0, 10, 20, 0, 10]
    finally:
        enl.enl_cache_free(c)


def test_plan_is_reused_until_a_store_changes_the_cache():
    c = host_cache()
    try:
        for g in range(3):
            for layer in range(2):
                enl.enl_group_store(c, g, layer, None, None, n_tokens=20 + g)
        plan(c, 0, [0, 1], 4, 4)
        p1 = enl.enl_plan_inspect(c)
        plan(c, 1, [0, 1], 4, 4)                                          # other layer, same plan
        p2 = enl.enl_plan_inspect(c)
        assert np.array_equal(p1["pages"], p2["pages"]) and np.array_equal(p1["meta"], p2["meta"])
        enl.enl_group_store(c, 0, 0, None, None, mode=enl.ENL_APPEND, n_tokens=30)
        enl.enl_group_store(c, 0, 1, None, None, mode=enl.ENL_APPEND, n_tokens=30)
        got = plan(c, 1, [0, 1], 4, 4)
        assert list(got) == [0, 50, 71]
        p3 = enl.enl_plan_inspect(c)
        assert p3["n_entries"] == 8 and [m & 0xff for m in p3["meta"][:6]] == [16, 16, 16, 2, 16, 5]
    finally:
        enl.enl_cache_free(c)


def test_merge_kind_follows_splits_shape_and_tile_count():
    """Two splits of a head_dim-128 call go to CTA pairs (kind 2) only when every CTA has a tile of its own;
    other split counts use the scratch buffer and the merge kernel (1); one query token per episode is the decode
    kernel's business (3)."""
    c = host_cache()
    try:
        for g, n in enumerate([300, 40, 7]):
            enl.enl_group_store(c, g, 0, None, None, n_tokens=n)
        plan(c, 0, [0, 1], 64, 64, split_hint=1)
        assert enl.enl_plan_inspect(c)["merge_kind"] == 0
        plan(c, 0, [0, 1], 64, 64, split_hint=2)
        p = enl.enl_plan_inspect(c)
        assert p["merge_kind"] == 2 and p["n_splits"] == 2 and p["n_items"] % 2 == 0
        plan(c, 0, [0, 1], 64, 64, split_hint=3)
        assert enl.enl_plan_inspect(c)["merge_kind"] == 1
        plan(c, 0, [], 64, 64, split_hint=2)                    # one tile in all: a second CTA would have nothing to do
        p = enl.enl_plan_inspect(c)
        assert p["merge_kind"] == 0 and p["n_splits"] == 1      # the hint is clamped: no CTA without a tile
        plan(c, 0, [0, 1], 1, 9)
        assert enl.enl_plan_inspect(c)["merge_kind"] == 3
    finally:
        enl.enl_cache_free(c)
    c = host_cache(head_dim=64)
    try:
        enl.enl_group_store(c, 0, 0, None, None, n_tokens=300)
        plan(c, 0, [0], 64, 64, split_hint=2)
        assert enl.enl_plan_inspect(c)["merge_kind"] == 1
    finally:
        enl.enl_cache_free(c)


def test_store_all_layers_moves_every_layer_together_or_not_at_all():
    c = host_cache()                                    # two layers
    try:
        enl.enl_group_store_all_layers(c, 2, None, None, n_tokens=40)
        assert [enl.enl_group_len(c, 2, l) for l in range(2)] == [40, 40]
        enl.enl_group_store_all_layers(c, 2, None, None, mode=enl.ENL_APPEND, n_tokens=9)      # Sec. 3.2: append
        assert [enl.enl_group_len(c, 2, l) for l in range(2)] == [49, 49]
        got = plan(c, 1, [2], 3, 3)
        assert list(got) == [0, 49]
        enl.enl_group_store(c, 2, 0, None, None, mode=enl.ENL_APPEND, n_tokens=1)              # layers now disagree
        with pytest.raises(enl.EnlError) as e:
            enl.enl_group_store_all_layers(c, 2, None, None, mode=enl.ENL_APPEND, n_tokens=5)
        assert e.value.code == enl.ENL_E_INVAL
        assert [enl.enl_group_len(c, 2, l) for l in range(2)] == [50, 49]                      # nothing moved
        enl.enl_group_store(c, 2, 1, None, None, mode=enl.ENL_APPEND, n_tokens=1)
        enl.enl_group_store_all_layers(c, 2, None, None, mode=enl.ENL_REPLACE, n_tokens=0)     # an empty group
        assert [enl.enl_group_len(c, 2, l) for l in range(2)] == [0, 0]
        with pytest.raises(enl.EnlError) as e:
            enl.enl_group_store_all_layers(c, 99, None, None, n_tokens=1)
        assert e.value.code == enl.ENL_E_NOGROUP
        with pytest.raises(enl.EnlError) as e:
            enl.enl_group_store_all_layers(c, 3, None, None, n_tokens=100000)                  # more than the pool holds
        assert e.value.code == enl.ENL_E_NOMEM and enl.enl_group_len(c, 3, 0) == -1
    finally:
        enl.enl_cache_free(c)
