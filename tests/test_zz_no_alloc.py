"""The backward entry point that allocates nothing, against the regular backward.

hmar_attn_bwd_noalloc exists for callers that may not allocate device memory when they need a
backward pass (all memory belongs to someone else's pool, the process must not grow after start-up,
or nothing that may synchronise the device is allowed).  It keeps its scratch in a fixed array inside
the library, so what has to be shown is that it gives the regular entry point's result, and that it
still does on a second call, when the shared array holds the first call's leftovers.  The result is also
compared with the CPU oracle, so that it does not rest on the other entry point being right, and the
defining property is checked directly: free device memory does not change over the calls, and the call works
with the regular entry points' plan cache released.

This file is named so that pytest collects it last.
"""
import ctypes

import numpy as np
import pytest
import torch

import paper_2506_04421_b200 as hmar
from oracle import hmar_oracle as orc
from workloads import training_inputs
from workloads.device import to_device

pytestmark = pytest.mark.gpu


class _Wl:
    def __init__(self, sides, B, H, seed):
        self.B, self.H, self.D, self.side_lens, self.softmax_scale = B, H, 64, tuple(sides), 0.125
        self.seed, self.L = seed, sum(s * s for s in sides)


def _case(wl):
    q, k, v, do = training_inputs(wl)
    tq, tk, tv, tdo = (to_device(x, wl.B, wl.H, torch.bfloat16) for x in (q, k, v, do))
    out, lse = hmar.hmar_attn_fwd(tq, tk, tv, wl.side_lens, wl.softmax_scale)
    ref = hmar.hmar_attn_bwd(tq, tk, tv, out, lse, tdo, wl.side_lens, wl.softmax_scale)
    # the caller owns every output; poison them so a call that wrote nothing cannot pass
    dq, dk, dv = (torch.full_like(tq, float("nan")) for _ in range(3))
    hmar.hmar_attn_bwd_noalloc(tq, tk, tv, out, lse, tdo, wl.side_lens, wl.softmax_scale, dq, dk, dv)
    torch.cuda.synchronize()
    # dk and dv are accumulated in a fixed order: identical.  dq is summed by reductions into global memory in
    # both entry points (the order varies), so it is compared with the bf16 tolerance the parity tests use.
    assert torch.equal(dk, ref[1]) and torch.equal(dv, ref[2])
    err = (dq.float() - ref[0].float()).abs()
    assert err.max().item() <= 2e-2 and err.mean().item() <= 2e-3
    assert torch.isfinite(dq).all()
    # and against the oracle, with the parity tests' tolerances
    for name, g, r in zip(("dq", "dk", "dv"), (dq, dk, dv), orc.attn_bwd(q, k, v, do, wl.side_lens, wl.softmax_scale)):
        d = np.abs(g.double().cpu().numpy().reshape(r.shape) - r)
        assert d.max() <= 2e-2 and d.mean() <= 2e-3, f"{name}: max {d.max():.3e} mean {d.mean():.3e}"


def test_noalloc_backward_matches_regular_backward_twice_in_a_row():
    # first call: several scales, ragged tiles, 2 x 3 heads
    _case(_Wl((1, 2, 3, 4, 6, 9, 13), B=2, H=3, seed=9001))
    # second call right after it, other shape and data: the shared scratch still holds the first
    # call's work list, delta and accumulator, all of which must be replaced or cleared
    _case(_Wl((3, 11, 5), B=1, H=2, seed=9002))
    # and the first shape again, so that a stale accumulator of the same size would show
    _case(_Wl((1, 2, 3, 4, 6, 9, 13), B=2, H=3, seed=9003))


def test_noalloc_backward_allocates_nothing():
    """Free device memory (cudaMemGetInfo) is the same before and after calls on side lists the library has
    never seen, and the entry point does not depend on the plan cache of the regular entry points."""
    cases = []
    for n, sides in enumerate(((2, 7, 5), (4, 4, 9), (1, 3, 12))):
        wl = _Wl(sides, B=1, H=2, seed=9100 + n)
        q, k, v, do = training_inputs(wl)
        tq, tk, tv, tdo = (to_device(x, wl.B, wl.H, torch.bfloat16) for x in (q, k, v, do))
        out, lse = hmar.hmar_attn_fwd(tq, tk, tv, wl.side_lens, wl.softmax_scale)
        ref = orc.attn_bwd(q, k, v, do, wl.side_lens, wl.softmax_scale)
        cases.append((wl, tq, tk, tv, out, lse, tdo, [torch.empty_like(tq) for _ in range(3)], ref))
    # warm-up on another list: the first call on a device looks the scratch address up
    w = cases[0]
    hmar.hmar_attn_bwd_noalloc(w[1], w[2], w[3], w[4], w[5], w[6], (2, 7, 5), 0.125, *w[7])
    hmar.hmar_shutdown()                   # the regular entry points' plans are gone
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for wl, tq, tk, tv, out, lse, tdo, grads, _ in cases:
        hmar.hmar_attn_bwd_noalloc(tq, tk, tv, out, lse, tdo, wl.side_lens, wl.softmax_scale, *grads)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    for wl, _, _, _, _, _, _, grads, ref in cases:
        for g, r in zip(grads, ref):
            d = np.abs(g.double().cpu().numpy().reshape(r.shape) - r)
            assert d.max() <= 2e-2 and d.mean() <= 2e-3


def test_noalloc_backward_rejects_problems_beyond_its_fixed_scratch():
    sides = (16, 32)                      # L = 1280
    B, H = 2, 13                          # 33280 rows > HMAR_NOALLOC_MAX_ROWS
    assert B * H * 1280 > hmar.HMAR_NOALLOC_MAX_ROWS
    t = torch.zeros((B, H, 1280, 64), dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros((B, H, 1280), dtype=torch.float32, device="cuda")
    sentinel = torch.full_like(t, 7.0)
    with pytest.raises(hmar.HmarError) as e:
        hmar.hmar_attn_bwd_noalloc(t, t, t, t, lse, t, sides, 0.125, sentinel, sentinel, sentinel)
    assert e.value.status == hmar.HMAR_ERR_WORKSPACE
    torch.cuda.synchronize()
    assert (sentinel == 7.0).all()        # nothing was launched
    # one batch less fits
    B = 1
    t = torch.randn((B, H, 1280, 64), device="cuda").to(torch.bfloat16)
    out, lse = hmar.hmar_attn_fwd(t, t, t, sides, 0.125)
    dq, dk, dv = (torch.empty_like(t) for _ in range(3))
    hmar.hmar_attn_bwd_noalloc(t, t, t, out, lse, t, sides, 0.125, dq, dk, dv)
    ref = hmar.hmar_attn_bwd(t, t, t, out, lse, t, sides, 0.125)
    assert torch.equal(dk, ref[1]) and torch.equal(dv, ref[2])


def test_noalloc_backward_argument_errors():
    p = ctypes.c_void_p(1 << 12)
    sides = (ctypes.c_int * 2)(1, 2)
    f = hmar.lib().hmar_attn_bwd_noalloc
    assert f(None, p, p, p, p, p, p, p, p, 1, 1, 64, 2, sides, 0.125, None) == hmar.HMAR_ERR_BAD_ARG
    assert f(p, p, p, p, p, p, p, p, p, 1, 1, 32, 2, sides, 0.125, None) == hmar.HMAR_ERR_UNSUPPORTED
    assert f(p, p, p, p, p, p, p, p, p, 1, 1, 64, 0, sides, 0.125, None) == hmar.HMAR_ERR_BAD_ARG
