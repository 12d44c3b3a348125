"""The entry point for callers that may not allocate (enl_attend_static): a robot's planner tick that
runs with memory fixed at start-up, or code hosted inside another runtime that owns the device heap,
cannot create a cache, so it hands the library one contiguous K/V buffer and the library keeps its
split-KV partials in a device array that is part of the library image.  Its result must equal what the
allocating path (enl_attend with one query token over the same groups) returns, call after call: the
built-in array is shared by all calls and still holds the previous call's partials."""
import numpy as np
import pytest
import torch

from oracle import enl_oracle as orc
from paper_2510_18546_b200 import enl, synth
from tests.helpers import MASS_MAX_ABS, OUT_MAX_ABS, OUT_MEAN_ABS, Session, check_close

pytestmark = pytest.mark.gpu


def both_paths(s, wl, sel, t, want_mass=True):
    """(out, mass) of enl_attend (n_q = 1, n_new = t + 1) and of enl_attend_static on the same keys."""
    q, kn, vn = wl.new_qkv(0, s.device)
    out_a, mass_a, _ = s.attend(0, q[t:t + 1], kn[:t + 1], vn[:t + 1], n_q=[1], n_new=[t + 1], sel_override=sel)
    k, v = wl.pool_kv(0, 0, s.device)
    offs = wl.pool_offsets(0)
    ks = [k[offs[g]:offs[g + 1]] for g in sel] + [kn[:t + 1]]
    vs = [v[offs[g]:offs[g + 1]] for g in sel] + [vn[:t + 1]]
    kc, vc = torch.cat(ks).contiguous(), torch.cat(vs).contiguous()
    out_s = torch.full((wl.n_q_heads, wl.head_dim), float("nan"), dtype=torch.bfloat16, device=s.device)
    mass_s = torch.full((wl.n_q_heads, len(sel) + 1), float("nan"), dtype=torch.float32, device=s.device) if want_mass else None
    enl.enl_attend_static([int(wl.pool_lens[0][g]) for g in sel], t + 1, q[t], kc, vc, out_s, mass_s,
                          stream=torch.cuda.current_stream(s.device).cuda_stream)
    torch.cuda.synchronize()
    # the float64 oracle on the same contiguous keys, the segments as its slots: a mistake shared by the two
    # one-token CUDA paths would pass a comparison of one with the other
    ro, rm = orc.attend_slots(wl.n_q_heads, wl.n_kv_heads, wl.head_dim, [x.cpu() for x in ks[:-1]],
                              [x.cpu() for x in vs[:-1]], q[t:t + 1].cpu(), kn[:t + 1].cpu(), vn[:t + 1].cpu())
    check_close(out_s[None], ro, mass_s[None] if want_mass else None, rm if want_mass else None, "static vs oracle")
    return out_a[0], (mass_a[0, :, :len(sel) + 1] if want_mass else None), out_s, mass_s


def assert_same(out_a, mass_a, out_s, mass_s):
    err = (out_a.float() - out_s.float()).abs()
    assert torch.isfinite(out_s.float()).all()
    assert err.max().item() <= OUT_MAX_ABS and err.mean().item() <= OUT_MEAN_ABS
    if mass_a is not None:
        assert torch.isfinite(mass_s).all()
        assert (mass_a - mass_s).abs().max().item() <= MASS_MAX_ABS
        assert (mass_s.sum(-1) - 1).abs().max().item() <= MASS_MAX_ABS


def test_two_calls_in_a_row_match_the_allocating_path():
    wl = synth.make_small(31, 1, 32, 8, 128, [[300, 17, 256, 90, 0, 1200]], [[0, 1, 2, 3, 4, 5]], [40], [40],
                          sigma=0.5, name="static")
    with Session(wl, [0]) as s:
        # first call: many keys, many splits; second call: fewer segments and keys, so stale partials of the
        # first call sit right behind what the second one writes
        assert_same(*both_paths(s, wl, [5, 0, 4, 2, 1, 3], 39))
        assert_same(*both_paths(s, wl, [1, 3], 0))
        assert_same(*both_paths(s, wl, [], 7))
        assert_same(*both_paths(s, wl, [5, 2], 20, want_mass=False))


def test_head_dim_64_and_other_head_ratios():
    wl = synth.make_small(32, 1, 8, 2, 64, [[33, 70, 18, 5]], [[0, 1, 2, 3]], [12], [12], name="static64")
    with Session(wl, [0]) as s:
        assert_same(*both_paths(s, wl, [2, 0, 3, 1], 11))
        assert_same(*both_paths(s, wl, [3], 0))


def test_limits_are_reported_not_enqueued():
    dev = torch.device("cuda:0")
    q = torch.zeros(32, 128, dtype=torch.bfloat16, device=dev)
    kv = torch.zeros(64, 8, 128, dtype=torch.bfloat16, device=dev)
    out = torch.zeros_like(q)
    with pytest.raises(enl.EnlError) as e:       # more keys than ENL_STATIC_MAX_KEYS (sizes only; nothing is read)
        enl.enl_attend_static([enl.ENL_STATIC_MAX_KEYS], 1, q, kv, kv, out)
    assert e.value.code == enl.ENL_E_LIMIT
    with pytest.raises(enl.EnlError) as e:       # more segments than ENL_STATIC_MAX_SEGMENTS
        enl.enl_attend_static([0] * (enl.ENL_STATIC_MAX_SEGMENTS + 1), 1, q, kv, kv, out)
    assert e.value.code == enl.ENL_E_LIMIT
    q16 = torch.zeros(32, 128, dtype=torch.bfloat16, device=dev)
    kv1 = torch.zeros(64, 2, 128, dtype=torch.bfloat16, device=dev)
    with pytest.raises(enl.EnlError) as e:       # 16 q heads per kv head
        enl.enl_attend_static([10], 1, q16, kv1, kv1, out)
    assert e.value.code == enl.ENL_E_LIMIT
    with pytest.raises(enl.EnlError) as e:
        enl.enl_attend_static([10], 0, q, kv, kv, out)
    assert e.value.code == enl.ENL_E_INVAL
