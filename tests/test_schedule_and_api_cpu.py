"""Host logic: the scale-block scheduler against the oracle's explicit mask, the C ABI's symbol
table against include/hmar.h, and argument validation (which runs before any device is touched)."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2506_04421_b200 as hmar
from oracle import hmar_oracle as orc
from workloads import CONFIGS

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SIDE_LISTS = [
    (1,), (1, 1), (3, 11), (12, 12), (1, 2, 3, 4), (2, 1, 3, 1, 2), (11, 12), (12, 11, 1),
    CONFIGS["256_d16_fwd"].side_lens, CONFIGS["512_d24_train"].side_lens, (1, 2, 4, 8, 16, 32, 64),
]


WINDOWS = [("markov", hmar.HMAR_WINDOW_MARKOV), ("causal", hmar.HMAR_WINDOW_CAUSAL), ("self", hmar.HMAR_WINDOW_SELF),
           ("prev", hmar.HMAR_WINDOW_PREV)]


@pytest.mark.parametrize("window", WINDOWS, ids=[w[0] for w in WINDOWS])
@pytest.mark.parametrize("sides", SIDE_LISTS)
@pytest.mark.parametrize("direction", [0, 1])
def test_tiles_cover_exactly_the_live_blocks(sides, direction, window):
    M = orc.window_mask(sides, window[0])
    if direction == 1:
        M = M.T            # rows = keys, columns = the queries that see them
    L = M.shape[0]
    tiles = hmar.hmar_schedule_tiles(sides, direction, window=window[1])
    seen = np.zeros(L, dtype=int)
    for t in tiles:
        r0, rc = t["row_begin"], t["row_count"]
        assert 0 < rc <= 128 and 0 <= r0 and r0 + rc <= L
        seen[r0:r0 + rc] += 1
        sub = M[r0:r0 + rc]
        cols = np.nonzero(sub.any(axis=0))[0]
        if len(cols) == 0:
            # keys that no query sees (the last scale under the preceding-scale mask): an empty partner range
            assert direction == 1 and window[0] == "prev" and t["partner_begin"] == t["partner_end"] and t["cost"] == 0
            continue
        # the partner range is the tight hull of what the tile's rows may touch
        assert cols.min() == t["partner_begin"] and cols.max() + 1 == t["partner_end"]
        # every row's support is one contiguous run inside that range (or empty)
        for row in sub:
            idx = np.nonzero(row)[0]
            assert len(idx) == 0 or idx[-1] - idx[0] + 1 == len(idx)
        full = bool(sub[:, t["partner_begin"]:t["partner_end"]].all())
        assert full == bool(t["uniform"])
        assert t["cost"] == -(-(t["partner_end"] - t["partner_begin"]) // 128)
    assert (seen == 1).all()              # every row in exactly one tile
    costs = [t["cost"] for t in tiles]
    assert costs == sorted(costs, reverse=True)


def test_tile_counts_for_paper_shapes():
    # 512x512 schedule: scales 1-5 packed (66 rows), scale 6 alone, then 2+3+5+8 full-scale tiles
    t = hmar.hmar_schedule_tiles(CONFIGS["512_d24_train"].side_lens, 0)
    assert len(t) == 20 and sum(x["uniform"] == 0 for x in t) == 1
    t = hmar.hmar_schedule_tiles(CONFIGS["256_d16_fwd"].side_lens, 0)
    assert len(t) == 7


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "hmar.h")).read()
    declared = set(re.findall(r"\b(hmar_[a-z0-9_]+)\s*\(", header))
    declared -= {"hmar_status"}
    assert declared == set(hmar.EXPORTED_SYMBOLS)
    L = hmar.lib()
    for name in declared:
        assert getattr(L, name) is not None


def _call_fwd(q=1 << 12, k=1 << 12, v=1 << 12, out=1 << 12, lse=1 << 12, B=1, H=1, D=64, sides=(1, 2),
              scale=0.125):
    arr = (ctypes.c_int * max(len(sides), 1))(*sides)
    vp = ctypes.c_void_p
    return hmar.lib().hmar_attn_fwd(vp(q), vp(k), vp(v), vp(out), vp(lse), B, H, D, len(sides), arr,
                                    scale, None)


def test_argument_errors_are_reported_before_any_launch():
    # pointers are fake but never dereferenced: validation fails first
    assert _call_fwd(q=0) == hmar.HMAR_ERR_BAD_ARG
    assert _call_fwd(q=(1 << 12) + 4) == hmar.HMAR_ERR_BAD_ARG          # misaligned
    assert _call_fwd(B=0) == hmar.HMAR_ERR_BAD_ARG
    assert _call_fwd(D=48) == hmar.HMAR_ERR_UNSUPPORTED                # head dimensions are 32, 64 or 128
    assert _call_fwd(sides=()) == hmar.HMAR_ERR_BAD_ARG
    assert _call_fwd(sides=(1, 0, 2)) == hmar.HMAR_ERR_BAD_ARG
    assert _call_fwd(sides=(1, -3)) == hmar.HMAR_ERR_BAD_ARG
    assert _call_fwd(sides=tuple([1] * 65)) == hmar.HMAR_ERR_BAD_ARG
    assert _call_fwd(B=70000) == hmar.HMAR_ERR_BAD_ARG
    assert _call_fwd(scale=0.0) == hmar.HMAR_ERR_BAD_ARG
    assert _call_fwd(scale=-0.125) == hmar.HMAR_ERR_BAD_ARG
    assert _call_fwd(scale=float("inf")) == hmar.HMAR_ERR_BAD_ARG
    assert _call_fwd(scale=float("nan")) == hmar.HMAR_ERR_BAD_ARG
    assert hmar.hmar_attn_bwd_workspace_bytes(1, 1, 48, (1, 2)) == 0
    assert hmar.hmar_attn_bwd_workspace_bytes(2, 3, 64, (1, 2)) >= 2 * 3 * 5 * (64 + 1) * 4
    with pytest.raises(hmar.HmarError):
        hmar.hmar_schedule_tiles((1, 0), 0)
    assert hmar.status_string(hmar.HMAR_ERR_WORKSPACE) == "workspace missing or too small"
    vp = ctypes.c_void_p
    # scale step: k_prev must be NULL exactly when side_prev == 0
    f = hmar.lib().hmar_attn_scale_step
    p = vp(1 << 12)
    assert f(p, None, None, p, p, p, None, 1, 1, 64, 2, 3, 0.125, None) == hmar.HMAR_ERR_BAD_ARG
    assert f(p, p, p, p, p, p, None, 1, 1, 64, 0, 3, 0.125, None) == hmar.HMAR_ERR_BAD_ARG
    assert f(p, p, p, p, p, p, None, 1, 1, 64, 2, 0, 0.125, None) == hmar.HMAR_ERR_BAD_ARG


def test_packed_forward_argument_errors():
    vp = ctypes.c_void_p
    f = hmar.lib().hmar_attn_fwd_packed
    p = vp(1 << 12)
    sides = (ctypes.c_int * 2)(1, 2)
    assert f(None, p, p, 1, 1, 64, 2, sides, 0.125, None) == hmar.HMAR_ERR_BAD_ARG
    assert f(vp((1 << 12) + 2), p, p, 1, 1, 64, 2, sides, 0.125, None) == hmar.HMAR_ERR_BAD_ARG
    assert f(p, p, p, 1, 1, 32, 2, sides, 0.125, None) == hmar.HMAR_ERR_UNSUPPORTED
    assert f(p, p, p, 1, 1, 64, 0, sides, 0.125, None) == hmar.HMAR_ERR_BAD_ARG
    assert f(p, p, p, 1, 1, 64, 2, sides, -1.0, None) == hmar.HMAR_ERR_BAD_ARG


def test_valid_call_without_a_device_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    assert _call_fwd() in (hmar.HMAR_ERR_CUDA, hmar.HMAR_ERR_UNSUPPORTED)


def test_argument_errors_of_the_added_entry_points():
    """Validation runs before any device is touched (the pointers are fake and never dereferenced)."""
    L = hmar.lib()
    p = ctypes.c_void_p(1 << 12)
    sides = (ctypes.c_int * 2)(1, 2)
    # packed backward
    f = L.hmar_attn_bwd_packed
    assert f(None, p, p, p, p, p, 1 << 20, 1, 1, 64, 2, sides, 0.125, None) == hmar.HMAR_ERR_BAD_ARG
    assert f(p, p, p, p, p, p, 1 << 20, 1, 1, 128, 2, sides, 0.125, None) == hmar.HMAR_ERR_UNSUPPORTED
    assert f(p, p, p, p, p, None, 0, 1, 1, 64, 2, sides, 0.125, None) == hmar.HMAR_ERR_WORKSPACE
    assert f(p, p, p, p, p, p, 16, 1, 1, 64, 2, sides, 0.125, None) == hmar.HMAR_ERR_WORKSPACE
    # the fourth window is accepted by the scheduler, a fifth is not
    assert L.hmar_schedule_tiles_window(2, sides, hmar.HMAR_WINDOW_PREV, 1, None, 0) > 0
    assert L.hmar_schedule_tiles_window(2, sides, 4, 1, None, 0) == hmar.HMAR_ERR_BAD_ARG
    # reconstruction step
    g = L.hmar_recon_accumulate
    assert g(None, p, None, p, None, None, 1, 32, 4096, 4, 32, None) == hmar.HMAR_ERR_BAD_ARG        # no xhat
    assert g(p, p, None, p, None, None, 1, 32, 4096, 33, 32, None) == hmar.HMAR_ERR_BAD_ARG          # would shrink the map
    assert g(p, p, None, p, p, None, 1, 32, 4096, 4, 32, None) == hmar.HMAR_ERR_BAD_ARG              # mask without old tokens
    assert g(p, p, p, p, p, p, 1, 32, 4096, 4, 32, None) == hmar.HMAR_ERR_BAD_ARG                    # tokens_out aliases an input
    assert g(p, p, None, p, None, None, 0, 32, 4096, 4, 32, None) == hmar.HMAR_ERR_BAD_ARG
    d = L.hmar_recon_downsample
    q2 = ctypes.c_void_p(p.value + 4096)
    assert d(None, q2, 1, 32, 32, 13, None) == hmar.HMAR_ERR_BAD_ARG                                 # no input
    assert d(p, None, 1, 32, 32, 13, None) == hmar.HMAR_ERR_BAD_ARG                                  # no output
    assert d(p, p, 1, 32, 32, 13, None) == hmar.HMAR_ERR_BAD_ARG                                     # in place
    assert d(p, q2, 1, 32, 13, 32, None) == hmar.HMAR_ERR_BAD_ARG                                    # would enlarge
    assert d(p, q2, 1, 32, 32, 0, None) == hmar.HMAR_ERR_BAD_ARG


def test_prev_window_backward_tiles_leave_out_nothing_but_the_last_scale():
    # under the preceding-scale mask the only key rows without queries are those of the last scale
    for sides in ((3, 11, 12), (1, 2, 3, 4, 6, 9, 13, 18), (12, 12, 12)):
        tiles = hmar.hmar_schedule_tiles(sides, 1, window=hmar.HMAR_WINDOW_PREV)
        empty = [t for t in tiles if t["partner_begin"] == t["partner_end"]]
        L_total = sum(s * s for s in sides)
        last_begin = L_total - sides[-1] ** 2
        assert all(t["row_begin"] >= last_begin for t in empty)
        covered = sum(t["row_count"] for t in empty)
        assert covered <= sides[-1] ** 2


def test_backward_full_tile_share_picks_the_instantiation():
    """The share of a head's backward steps in full tiles, recomputed here from the exported tile list, and on
    which side of the 60 % line the paper's two training resolutions fall (Sec. 5: 256 x 256 has L = 680,
    512 x 512 has L = 2240): the short list runs the one-variant backward, the long one the three-variant one."""
    def share(side_lens, window=hmar.HMAR_WINDOW_MARKOV):
        plain = total = 0
        for t in hmar.hmar_schedule_tiles(side_lens, 1, window=window):
            steps = (t["partner_end"] - t["partner_begin"] + 127) // 128
            total += steps
            if t["uniform"] and t["row_count"] == 128:
                plain += steps
        return plain * 1000 // total
    short, long_ = CONFIGS["256_d30_train"].side_lens, CONFIGS["512_d24_train"].side_lens
    for sides in (short, long_, (1, 2), (16, 16), (12, 12, 12)):
        assert hmar.hmar_schedule_bwd_full_tile_share(sides) == share(sides), sides
    for window in (hmar.HMAR_WINDOW_CAUSAL, hmar.HMAR_WINDOW_SELF, hmar.HMAR_WINDOW_PREV):
        assert hmar.hmar_schedule_bwd_full_tile_share(long_, window) == share(long_, window)
    assert hmar.hmar_schedule_bwd_full_tile_share(short) < 600 <= hmar.hmar_schedule_bwd_full_tile_share(long_)
    # (16, 16): four full tiles of 128 keys (two per scale), seen by 512 and by 256 queries: every step is plain
    assert hmar.hmar_schedule_bwd_full_tile_share((16, 16)) == 1000
    # (1, 2): one packed tile of 5 key rows, never full
    assert hmar.hmar_schedule_bwd_full_tile_share((1, 2)) == 0
    with pytest.raises(hmar.HmarError):
        hmar.hmar_schedule_bwd_full_tile_share((1, 0))
