"""Parity of the CUDA path (through the C ABI) with the fp64 CPU oracle, element by element.

Tolerances (written here, derived from the arithmetic):
  * bf16 entry points: inputs are bf16 (shared with the oracle, so input rounding cancels), products
    are exact in fp32, the softmax is fp32, P and dS are rounded to bf16 before the second matrix
    product and the outputs are rounded to bf16 (relative 2^-9).  For N(0,1) inputs the outputs are
    O(1), giving max |err| <= 2e-2 and mean |err| <= 2e-3 on out, dq, dk, dv; lse is fp32 and must
    agree to 1e-3.
  * fp32 debug entry points: <= 1e-5 on everything.
  * inputs that are not N(0,1) (the stress cases): dK = scale * dS^T Q is linear in Q, so its tolerance
    follows the factor put on Q; the fp32 build's error is the rounding of s - lse at |s| ~ 30, which grows
    with the logits.  The bf16 dQ gets no such factor: it is held to the element-wise first-order bound of
    its own roundings (`_bf16_dq_bound`) and to the unscaled mean.
"""
import numpy as np
import pytest
import torch

import paper_2506_04421_b200 as hmar
from oracle import hmar_oracle as orc
from workloads import CONFIGS, scale_step_inputs, training_inputs
from workloads.device import bulk_normal, to_device, training_tensors

pytestmark = pytest.mark.gpu

BF16_MAX, BF16_MEAN, LSE_TOL, F32_TOL = 2e-2, 2e-3, 1e-3, 1e-5


def _err(gpu, ref):
    d = np.abs(gpu.detach().double().cpu().numpy().reshape(ref.shape) - ref)
    return float(d.max()), float(d.mean())


def _assert_close(name, gpu, ref, is_f32, magnitude=1.0):
    """`magnitude` rescales the absolute tolerances for tensors whose entries are not O(1)."""
    mx, mean = _err(gpu, ref)
    mx, mean = mx / magnitude, mean / magnitude
    if is_f32:
        assert mx <= F32_TOL, f"{name}: max abs err {mx:.3e} > {F32_TOL}"
    else:
        assert mx <= BF16_MAX, f"{name}: max abs err {mx:.3e} > {BF16_MAX}"
        assert mean <= BF16_MEAN, f"{name}: mean abs err {mean:.3e} > {BF16_MEAN}"


def _assert_lse(gpu, ref, is_f32):
    mx, _ = _err(gpu, ref)
    assert mx <= (F32_TOL if is_f32 else LSE_TOL), f"lse: max abs err {mx:.3e}"


def _bf16_dq_bound(q, k, v, do, side_lens, scale, window="markov"):
    """Element-wise first-order bound on |dq_gpu - dq_exact| of the bf16 path, from its stated roundings
    (u = 2^-8 is the unit roundoff of bf16): the result is rounded to bf16 (u |dQ|); dS is rounded to bf16
    before dQ = scale * dS K (scale * u * |dS| |K|); delta = rowsum(dO o O) is formed from the bf16-rounded
    O (|d delta| <= u * rowsum |dO||O|, which reaches dQ through scale * P |K|).  Everything else (fp32
    accumulation, ex2.approx on an fp32 argument of size <= 2^6) is below 2^-17 relative and is covered by the
    absolute slack.  The terms are worst-case sums, so a correct kernel sits well inside."""
    u = 2.0 ** -8
    q, k, v, do = (np.asarray(x, dtype=np.float64) for x in (q, k, v, do))
    P, _ = orc.attention_probs(q, k, orc.window_mask(side_lens, window), scale)
    dP = do @ np.swapaxes(v, -1, -2)
    delta = (P * dP).sum(axis=-1, keepdims=True)
    dS = P * (dP - delta)
    ak = np.abs(k)
    d_delta = u * (np.abs(do) * np.abs(P @ v)).sum(axis=-1, keepdims=True)
    return u * np.abs(scale * (dS @ k)) + scale * u * (np.abs(dS) @ ak) + scale * d_delta * (P @ ak) + 1e-3


def _assert_bf16_dq(name, dq, ref, bound, max_factor=1.0):
    """bf16 dQ of a stress case: inside the derived element-wise bound, and inside the N(0,1) tolerances
    (`max_factor` only where the reference dQ itself is larger than O(1))."""
    d = np.abs(dq.detach().double().cpu().numpy().reshape(ref.shape) - ref)
    mx, mean, worst = float(d.max()), float(d.mean()), float((d / bound).max())
    msg = (f"{name}: max abs err {mx:.3e}, mean abs err {mean:.3e}, max err/bound {worst:.3f}, "
           f"max |ref| {np.abs(ref).max():.2f}")
    assert worst <= 1.0, msg
    assert mx <= BF16_MAX * max_factor and mean <= BF16_MEAN * max_factor, msg


def _guarded(shape, dtype, guards, pad=512):
    """An output tensor with `pad` canary elements before and after it in the same allocation; appends to
    `guards` a function that says whether the canaries are still intact."""
    n = int(np.prod(shape))
    flat = torch.full((n + 2 * pad,), 77.0, dtype=dtype, device="cuda")
    guards.append(lambda: bool((flat[:pad] == 77.0).all() and (flat[pad + n:] == 77.0).all()))
    return flat[pad:pad + n].view(*shape)


def _no_device_error():
    status, detail = hmar.hmar_device_status()
    assert status == hmar.HMAR_OK, f"device status {status} detail {detail:#x}"


class _Wl:
    """Ad-hoc workload for the edge-case side lists."""
    def __init__(self, sides, B=1, H=2, seed=777, D=64):
        self.B, self.H, self.D, self.side_lens, self.softmax_scale = B, H, D, tuple(sides), 0.125
        self.seed = seed + sum((i + 1) * s for i, s in enumerate(sides))
        self.L = sum(s * s for s in sides)


def _run_training(wl, dtype, gain=1.0, backward=True, simt=False):
    # q scaled by `gain` makes dK (= scale * dS^T Q) grow by the same factor; in the fp32 build the rounding
    # of s - lse, which feeds every P and dS, grows with the logits.  The bf16 dQ has neither excuse.
    mag_k = max(1.0, gain)
    is_f32 = dtype == torch.float32
    q, k, v, do = training_inputs(wl, bf16=not is_f32, gain=gain)
    prev = hmar.hmar_debug_force_simt(simt)
    try:
        tq, tk, tv, tdo = (to_device(x, wl.B, wl.H, dtype) for x in (q, k, v, do))
        # every output sits between canary stretches that the kernels must leave alone
        guards = []
        out, lse = _guarded(tq.shape, dtype, guards), _guarded(tq.shape[:3], torch.float32, guards)
        hmar.hmar_attn_fwd(tq, tk, tv, wl.side_lens, wl.softmax_scale, out=out, lse=lse)
        ref_out, ref_lse = orc.attn_fwd(q, k, v, wl.side_lens, wl.softmax_scale)
        _assert_close("out", out, ref_out, is_f32)
        _assert_lse(lse, ref_lse, is_f32)
        if backward:
            dq, dk, dv = (_guarded(tq.shape, dtype, guards) for _ in range(3))
            hmar.hmar_attn_bwd(tq, tk, tv, out, lse, tdo, wl.side_lens, wl.softmax_scale, dq=dq, dk=dk, dv=dv)
            rq, rk, rv = orc.attn_bwd(q, k, v, do, wl.side_lens, wl.softmax_scale)
            if is_f32 or gain == 1.0:
                _assert_close("dq", dq, rq, is_f32, mag_k)
            else:
                _assert_bf16_dq("dq", dq, rq, _bf16_dq_bound(q, k, v, do, wl.side_lens, wl.softmax_scale))
            _assert_close("dk", dk, rk, is_f32, mag_k)
            _assert_close("dv", dv, rv, is_f32)
        _no_device_error()
        assert all(intact() for intact in guards), "a kernel wrote outside its output tensor"
    finally:
        hmar.hmar_debug_force_simt(prev)


EDGE_SIDES = [(1,), (1, 1), (3, 11), (12, 12), (11, 12), (2, 1, 3, 1, 2), (12, 11, 1), (1, 2, 3, 4, 5, 6, 8, 10, 13, 16),
              (16, 3, 17), (1, 23)]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_config1_tiny_fwd_bwd(dtype):
    _run_training(CONFIGS["tiny"], dtype)


@pytest.mark.parametrize("sides", EDGE_SIDES)
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_edge_side_lists_fwd_bwd(sides, dtype):
    _run_training(_Wl(sides), dtype)


@pytest.mark.parametrize("sides", [(1, 2, 3, 4), (3, 11), (1, 2, 3, 4, 5, 6, 8, 10, 13, 16)])
def test_bf16_simt_fallback_kernels(sides):
    _run_training(_Wl(sides), torch.bfloat16, simt=True)


@pytest.mark.parametrize("D", [32, 128])
@pytest.mark.parametrize("sides", [(1, 2, 3, 4), (3, 11), (2, 1, 3, 1, 2), (1, 2, 3, 4, 5, 6, 8, 10, 13, 16)])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_other_head_dimensions_through_the_plain_kernels(sides, dtype, D):
    """Head dimensions 32 and 128 (the tensor-core kernels are D = 64 only): forward, backward and the inference
    step on the plain-FMA kernels, same tolerances."""
    wl = _Wl(sides, D=D)
    wl.softmax_scale = D ** -0.5
    _run_training(wl, dtype)
    is_f32 = dtype == torch.float32
    s = len(sides) - 1
    q, kp, vp, kc, vc = scale_step_inputs(wl, s, 0, bf16=not is_f32)
    dev = [to_device(x, wl.B, wl.H, dtype) for x in (q, kp, vp, kc, vc)]
    out, lse = hmar.hmar_attn_scale_step(*dev, sides[s - 1], sides[s], wl.softmax_scale)
    ref_out, ref_lse = orc.scale_step(q, kp, vp, kc, vc, wl.softmax_scale)
    _assert_close("step out", out, ref_out, is_f32)
    _assert_lse(lse, ref_lse, is_f32)
    _no_device_error()


def test_large_logits_exercise_running_max():
    # q scaled by 8: logits ~ N(0, 8^2), the running maximum moves often and P is peaked
    _run_training(_Wl((1, 2, 3, 4, 6, 9, 13, 18)), torch.bfloat16, gain=8.0)
    _run_training(_Wl((1, 2, 3, 4, 6, 9, 13, 18)), torch.float32, gain=8.0)


def test_rows_past_a_partial_key_tile_cannot_reach_dq():
    # Scale 2 has 81 keys: its key tile is loaded 128 rows high, so rows 81..127 hold the first keys of
    # scale 3, which the tile's queries of scale 2 must not see.  Those keys are made 16 times larger
    # (a power of two: still exact in bf16), so that a logit against them is worth e^40 and more: if such
    # a row leaked into dQ = dS K the result would be off by many orders of magnitude.
    wl = _Wl((1, 9, 13, 5))
    q, k, v, do = training_inputs(wl, bf16=True)
    n = [s * s for s in wl.side_lens]
    k = k.copy()
    k[:, n[0] + n[1]:n[0] + n[1] + n[2], :] *= 16.0
    tq, tk, tv, tdo = (to_device(x, wl.B, wl.H, torch.bfloat16) for x in (q, k, v, do))
    out, lse = hmar.hmar_attn_fwd(tq, tk, tv, wl.side_lens, wl.softmax_scale)
    ref_out, ref_lse = orc.attn_fwd(q, k, v, wl.side_lens, wl.softmax_scale)
    _assert_close("out", out, ref_out, False)
    _assert_lse(lse, ref_lse, False)
    dq, dk, dv = hmar.hmar_attn_bwd(tq, tk, tv, out, lse, tdo, wl.side_lens, wl.softmax_scale)
    rq, rk, rv = orc.attn_bwd(q, k, v, do, wl.side_lens, wl.softmax_scale)
    assert torch.isfinite(dq).all() and torch.isfinite(dk).all() and torch.isfinite(dv).all()
    # the queries that see the large keys have dQ = scale * dS K with |K| up to 16 x 4: dQ itself is 16 times
    # larger there, so the absolute tolerances are too, and every element stays inside its derived bound
    _assert_bf16_dq("dq", dq, rq, _bf16_dq_bound(q, k, v, do, wl.side_lens, wl.softmax_scale), max_factor=16.0)
    # dK_j = scale * sum_i dS_ij Q_i and dV_j = sum_i P_ij dO_i: with logits this large several queries put P
    # close to 1 on the same key, and the bf16 roundings of those dS and P (2^-8 relative, times |Q|, |dO| up
    # to 4) add up, so twice the usual bound for both
    _assert_close("dk", dk, rk, False, 2.0)
    _assert_close("dv", dv, rv, False, 2.0)
    # the rows the test is about: queries of scale 2 see keys of scales 1 and 2 only, all of them O(1)
    lo, hi = n[0], n[0] + n[1]
    d = np.abs(dq.detach().double().cpu().numpy().reshape(rq.shape)[:, lo:hi] - rq[:, lo:hi])
    assert d.max() <= BF16_MAX, f"dq of the tile's own queries: max abs err {d.max():.3e}"
    _no_device_error()


@pytest.mark.parametrize("sides,B,H", [((1, 2, 3, 4, 6, 9, 13), 2, 3), ((3, 11), 1, 2), ((16, 3, 17), 3, 1)])
def test_packed_qkv_forward(sides, B, H):
    # qkv [B, L, 3, H, D] (the projection's layout), out [B, L, H, D]; the oracle sees the same values as
    # [B*H, L, D] tensors
    wl = _Wl(sides, B=B, H=H)
    q, k, v = training_inputs(wl, bf16=True, with_dout=False)
    L, D = wl.L, wl.D
    packed = np.stack([x.reshape(B, H, L, D) for x in (q, k, v)], axis=0)          # [3, B, H, L, D]
    packed = np.ascontiguousarray(packed.transpose(1, 3, 0, 2, 4))                 # [B, L, 3, H, D]
    t = torch.from_numpy(packed).to(device="cuda", dtype=torch.bfloat16)
    out, lse = hmar.hmar_attn_fwd_packed(t, wl.side_lens, wl.softmax_scale)
    assert out.shape == (B, L, H, D) and lse.shape == (B, H, L)
    ref_out, ref_lse = orc.attn_fwd(q, k, v, wl.side_lens, wl.softmax_scale)
    _assert_close("out", out.permute(0, 2, 1, 3).contiguous(), ref_out, False)
    _assert_lse(lse, ref_lse, False)
    # the same values through the contiguous entry point give the same bits
    tq, tk, tv = (to_device(x, B, H, torch.bfloat16) for x in (q, k, v))
    out_c, lse_c = hmar.hmar_attn_fwd(tq, tk, tv, wl.side_lens, wl.softmax_scale)
    assert torch.equal(out_c, out.permute(0, 2, 1, 3)) and torch.equal(lse_c, lse)
    _no_device_error()


@pytest.mark.parametrize("sides,B,H", [((1, 2, 3, 4, 6, 9, 13), 2, 3), ((3, 11), 1, 2), ((16, 3, 17), 3, 1), ((1, 2, 3, 4, 5, 6, 8, 10, 13, 16), 2, 2)])
def test_packed_qkv_backward(sides, B, H):
    """Backward on qkv / dqkv [B,L,3,H,D] and out / dout [B,L,H,D]: against the oracle, and dk, dv bit for bit against
    the contiguous entry point on the same values (dq is summed in an order that varies: tolerance)."""
    wl = _Wl(sides, B=B, H=H)
    q, k, v, do = training_inputs(wl, bf16=True)
    L, D = wl.L, wl.D
    packed = np.stack([x.reshape(B, H, L, D) for x in (q, k, v)], axis=0)          # [3, B, H, L, D]
    t = torch.from_numpy(np.ascontiguousarray(packed.transpose(1, 3, 0, 2, 4))).to(device="cuda", dtype=torch.bfloat16)
    tdo = torch.from_numpy(np.ascontiguousarray(do.reshape(B, H, L, D).transpose(0, 2, 1, 3))).to(device="cuda", dtype=torch.bfloat16)
    out, lse = hmar.hmar_attn_fwd_packed(t, wl.side_lens, wl.softmax_scale)
    guards = []
    dqkv = _guarded(t.shape, torch.bfloat16, guards)
    hmar.hmar_attn_bwd_packed(t, out, lse, tdo, wl.side_lens, wl.softmax_scale, dqkv=dqkv)
    refs = orc.attn_bwd(q, k, v, do, wl.side_lens, wl.softmax_scale)
    got = [dqkv[:, :, i].permute(0, 2, 1, 3).contiguous() for i in range(3)]      # [B, H, L, D]
    for nm, g, r in zip(("dq", "dk", "dv"), got, refs):
        _assert_close(nm, g, r, False)
    tq, tk, tv, tdo_c = (to_device(x, B, H, torch.bfloat16) for x in (q, k, v, do))
    out_c, lse_c = hmar.hmar_attn_fwd(tq, tk, tv, wl.side_lens, wl.softmax_scale)
    dq_c, dk_c, dv_c = hmar.hmar_attn_bwd(tq, tk, tv, out_c, lse_c, tdo_c, wl.side_lens, wl.softmax_scale)
    assert torch.equal(dk_c, got[1]) and torch.equal(dv_c, got[2])
    assert (dq_c.float() - got[0].float()).abs().max().item() <= BF16_MAX
    assert all(intact() for intact in guards)
    _no_device_error()


def test_packed_qkv_forward_full_size_matches_contiguous_bits():
    # the headline shape as bench.py's packed leg runs it: the packed entry point must give the very bits
    # of the contiguous one (which the sampled-head tests compare with the oracle at this size)
    wl = CONFIGS["512_d24_train"]
    B, H, L, D = wl.B, wl.H, wl.L, wl.D
    qkv = bulk_normal(wl.seed, 9, B, L, 3 * H, D, torch.bfloat16, "cuda").view(B, L, 3, H, D)
    out, lse = hmar.hmar_attn_fwd_packed(qkv, wl.side_lens, wl.softmax_scale)
    q, k, v = (qkv[:, :, i].permute(0, 2, 1, 3).contiguous() for i in range(3))
    out_c, lse_c = hmar.hmar_attn_fwd(q, k, v, wl.side_lens, wl.softmax_scale)
    assert torch.equal(out_c, out.permute(0, 2, 1, 3)) and torch.equal(lse_c, lse)
    _no_device_error()


@pytest.mark.parametrize("sides", [(12, 13, 14), (13, 12, 15), (16, 13, 19, 12)])
def test_forward_ignores_non_finite_values_outside_a_rows_window(sides):
    """Key tiles are fetched 64 rows at a time, so the tail of a scale's last tile holds rows of the next scale.
    Those keys are masked, but a masked P of exactly 0 times a non-finite V would still be NaN: the forward
    clears such V rows, and a NaN logit is replaced, not scaled.  With K and V of one scale set to NaN / Inf,
    every row that cannot see that scale must come out exactly as without them.  (Scales of at least 128 tokens:
    a tile that packs several small scales gives its rows different windows over the same V rows, and there the
    inputs have to be finite.)"""
    wl = _Wl(sides)
    q, k, v = training_inputs(wl, bf16=True, with_dout=False)
    n = [s * s for s in wl.side_lens]
    start = np.concatenate([[0], np.cumsum(n)])
    tq, tk, tv = (to_device(x, wl.B, wl.H, torch.bfloat16) for x in (q, k, v))
    clean, clean_lse = hmar.hmar_attn_fwd(tq, tk, tv, wl.side_lens, wl.softmax_scale)
    for bad_scale in range(1, len(sides)):
        tk2, tv2 = tk.clone(), tv.clone()
        tk2[:, :, start[bad_scale]:start[bad_scale + 1]] = float("nan")
        tv2[:, :, start[bad_scale]:start[bad_scale + 1]] = float("inf")
        out, lse = hmar.hmar_attn_fwd(tq, tk2, tv2, wl.side_lens, wl.softmax_scale)
        # rows of scales bad_scale and bad_scale + 1 see the poisoned keys; all others must be untouched
        keep = np.ones(wl.L, dtype=bool)
        keep[start[bad_scale]:start[min(bad_scale + 2, len(sides))]] = False
        idx = torch.from_numpy(np.nonzero(keep)[0]).cuda()
        assert torch.equal(out[:, :, idx], clean[:, :, idx]) and torch.equal(lse[:, :, idx], clean_lse[:, :, idx])
    _no_device_error()


def test_fp32_debug_build_512_shape_one_head():
    _run_training(_Wl(CONFIGS["512_d24_train"].side_lens, B=1, H=1), torch.float32)


WINDOWS = [("causal", hmar.HMAR_WINDOW_CAUSAL), ("self", hmar.HMAR_WINDOW_SELF), ("prev", hmar.HMAR_WINDOW_PREV)]


@pytest.mark.parametrize("window", WINDOWS, ids=[w[0] for w in WINDOWS])
@pytest.mark.parametrize("sides", [(1, 2, 3, 4), (3, 11), (12, 11, 1), (2, 1, 3, 1, 2), (1, 2, 3, 4, 5, 6, 8, 10, 13, 16), (16, 3, 17), (5,), (1, 1), (9, 13, 18)])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_other_block_masks_fwd_bwd(sides, dtype, window):
    """VAR's block-causal mask, the block-diagonal mask and the preceding-scale mask (whose last scale's keys have
    no queries: dK = dV = 0 there) through the *_window entry points."""
    wl = _Wl(sides)
    is_f32 = dtype == torch.float32
    q, k, v, do = training_inputs(wl, bf16=not is_f32)
    tq, tk, tv, tdo = (to_device(x, wl.B, wl.H, dtype) for x in (q, k, v, do))
    out, lse = hmar.hmar_attn_fwd(tq, tk, tv, wl.side_lens, wl.softmax_scale, window=window[1])
    ref_out, ref_lse = orc.attn_fwd(q, k, v, wl.side_lens, wl.softmax_scale, window=window[0])
    _assert_close("out", out, ref_out, is_f32)
    _assert_lse(lse, ref_lse, is_f32)
    dq, dk, dv = hmar.hmar_attn_bwd(tq, tk, tv, out, lse, tdo, wl.side_lens, wl.softmax_scale, window=window[1])
    rq, rk, rv = orc.attn_bwd(q, k, v, do, wl.side_lens, wl.softmax_scale, window=window[0])
    # Under the narrow masks a one-token scale is the only key of every query of the next scale: P = 1 for all of
    # them, and that key's dK, dV are plain sums over those queries, several times larger than O(1).  A bf16
    # result cannot be closer than its unit roundoff 2^-8 |x|, so where the oracle's largest entry exceeds
    # 2e-2 / 2^-8 = 5.1 the absolute limits grow in proportion (factor 1 otherwise, and always 1 for fp32).
    def mag(ref):
        return 1.0 if is_f32 else max(1.0, float(np.abs(ref).max()) * 2.0 ** -8 / BF16_MAX)
    _assert_close("dq", dq, rq, is_f32, mag(rq))
    _assert_close("dk", dk, rk, is_f32, mag(rk))
    _assert_close("dv", dv, rv, is_f32, mag(rv))
    if window[0] == "prev" and len(sides) > 1:
        n_last = sides[-1] ** 2                        # nobody looks at the last scale's keys: exact zeros
        assert not dk[:, :, -n_last:].any() and not dv[:, :, -n_last:].any()
    _no_device_error()


def _sample_heads(BH, n=6):
    rng = np.random.default_rng(BH)
    inner = rng.permutation(np.arange(1, BH - 1))[:max(0, min(n, BH) - 2)]
    return sorted({0, BH - 1} | set(int(x) for x in inner))


def _partition_heads(wl, n, window=hmar.HMAR_WINDOW_MARKOV):
    """Heads for the full-size comparisons, taken from the backward's own partition of the work.

    The backward runs one persistent block per SM; block b takes the items (head, key tile) whose cost, in the
    head-by-head order of the item list, lies in [total * b / blocks, total * (b + 1) / blocks), a tile costing
    its 128-query steps plus two.  The hand-over between two items of different heads, and the first and last
    item of a block, are the places where a mistake would hide from a comparison of whole heads chosen at
    random, so the heads picked are those in which a block's run starts strictly inside the head, spread over
    the blocks, always with the first and the last head.  (For sequences cut into several runs per head every
    head has such boundaries.)"""
    BH = wl.B * wl.H
    tiles = hmar.hmar_schedule_tiles(wl.side_lens, 1, window)
    head_cost = sum((t["partner_end"] - t["partner_begin"] + 127) // 128 + 2 for t in tiles)
    blocks = torch.cuda.get_device_properties(0).multi_processor_count
    total = BH * head_cost
    inside = sorted({(total * b // blocks) // head_cost for b in range(1, blocks) if (total * b // blocks) % head_cost})
    inside = [h for h in inside if 0 < h < BH - 1] or list(range(1, BH - 1))
    step = max(1, len(inside) // max(1, n - 2))
    return sorted({0, BH - 1} | set(inside[::step][:max(0, n - 2)]))


def _check_sampled(wl, heads, window_id, window_name, backward, chunk):
    """Forward (and backward) at full size; the oracle checks `heads` element by element, `chunk` at a time."""
    dev, host = training_tensors(wl, heads, with_dout=backward)
    out, lse = hmar.hmar_attn_fwd(dev["q"], dev["k"], dev["v"], wl.side_lens, wl.softmax_scale, window=window_id)
    grads = None
    if backward:
        grads = hmar.hmar_attn_bwd(dev["q"], dev["k"], dev["v"], out, lse, dev["dout"], wl.side_lens, wl.softmax_scale,
                                   window=window_id)
        for g in grads:
            assert torch.isfinite(g).all()
    for lo in range(0, len(heads), chunk):
        sl = slice(lo, lo + chunk)
        idx = torch.as_tensor(heads[sl], device="cuda")
        hq, hk, hv = host["q"][sl], host["k"][sl], host["v"][sl]
        ref_out, ref_lse = orc.attn_fwd(hq, hk, hv, wl.side_lens, wl.softmax_scale, window=window_name)
        _assert_close(f"out[heads {heads[sl]}]", out.view(-1, wl.L, wl.D)[idx], ref_out, False)
        _assert_lse(lse.view(-1, wl.L)[idx], ref_lse, False)
        if backward:
            refs = orc.attn_bwd(hq, hk, hv, host["dout"][sl], wl.side_lens, wl.softmax_scale, window=window_name)
            for nm, g, r in zip(("dq", "dk", "dv"), grads, refs):
                _assert_close(f"{nm}[heads {heads[sl]}]", g.view(-1, wl.L, wl.D)[idx], r, False)
    return dev, out, lse, grads


def test_block_causal_full_size_sampled_heads():
    """The paper's comparison workload (VAR's block-causal mask, App. B.4) on the 512x512 d24 shape."""
    wl = CONFIGS["512_d24_train"]
    heads = _partition_heads(wl, 32, hmar.HMAR_WINDOW_CAUSAL)
    assert len(heads) >= 32
    _check_sampled(wl, heads, hmar.HMAR_WINDOW_CAUSAL, "causal", True, 4)
    _no_device_error()


@pytest.mark.parametrize("name", ["256_d16_fwd", "256_d30_train", "512_d24_train", "1024_d24_train"])
def test_full_size_configs_sampled_heads(name):
    """Configs 2-4 (and the 1024 shape) at their full sizes, in the launch shape the benchmark times; the oracle
    checks a sample of heads element by element: at least 32 (8 at L = 9451, where one head costs the oracle
    several seconds and gigabytes), chosen where the backward's blocks change heads."""
    wl = CONFIGS[name]
    backward = "bwd" in wl.passes
    n_heads = 8 if wl.L > 4000 else 32
    heads = _partition_heads(wl, n_heads) if backward else _sample_heads(wl.B * wl.H, n_heads)
    assert len(heads) >= min(n_heads, wl.B * wl.H // 4)
    dev, out, lse, grads = _check_sampled(wl, heads, hmar.HMAR_WINDOW_MARKOV, "markov", backward,
                                          1 if wl.L > 4000 else (4 if wl.L > 1000 else 16))
    # properties that hold for every head: finite outputs, |out| bounded by max |v| of the head
    assert torch.isfinite(out).all() and torch.isfinite(lse).all()
    assert (out.float().abs().amax(dim=(2, 3)) <= dev["v"].float().abs().amax(dim=(2, 3)) * 1.01).all()
    if backward:
        # column sums of dV equal column sums of dO for every head (rows of P sum to one)
        s_dv = grads[2].float().sum(dim=2)
        s_do = dev["dout"].float().sum(dim=2)
        assert (s_dv - s_do).abs().max().item() < 0.5     # sums of L bf16-rounded terms
    _no_device_error()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_scale_step_small_batch_all_scales(dtype):
    wl = CONFIGS["512_d24_infer"]
    is_f32 = dtype == torch.float32
    heads = [0, 1, 700, wl.B * wl.H - 1]
    B, H = 2, 2
    for s, side in enumerate(wl.side_lens):
        for sub in (0, 3):
            q, kp, vp, kc, vc = scale_step_inputs(wl, s, sub, bf16=not is_f32, heads=heads)
            dev = [None if x is None else to_device(x, B, H, dtype) for x in (q, kp, vp, kc, vc)]
            side_prev = wl.side_lens[s - 1] if s else 0
            out, lse = hmar.hmar_attn_scale_step(*dev, side_prev, side, wl.softmax_scale)
            ref_out, ref_lse = orc.scale_step(q, kp, vp, kc, vc, wl.softmax_scale)
            _assert_close(f"out[scale {s}]", out, ref_out, is_f32)
            _assert_lse(lse, ref_lse, is_f32)
            out2, none = hmar.hmar_attn_scale_step(*dev, side_prev, side, wl.softmax_scale, want_lse=False)
            assert none is None and torch.equal(out2, out)
    _no_device_error()


@pytest.mark.parametrize("sub", [0, 3])
def test_scale_step_full_batch_all_scales_sampled_heads(sub):
    """Config 5 at B=64, H=24, every scale, first and last masked sub-step; sampled heads against the oracle.
    Scales 1-6 (windows of at most 128 keys) run in the small-window kernel, 7-10 in the tcgen05 kernel."""
    wl = CONFIGS["512_d24_infer"]
    BH = wl.B * wl.H
    heads = _sample_heads(BH, 6)
    idx = torch.as_tensor(heads, device="cuda")
    for s in range(len(wl.side_lens)):
        side, side_prev = wl.side_lens[s], (wl.side_lens[s - 1] if s else 0)
        host = scale_step_inputs(wl, s, sub, bf16=True, heads=heads)
        dev = []
        for sid, h in enumerate(host):
            if h is None:
                dev.append(None)
                continue
            t = bulk_normal(wl.seed + s, sid, wl.B, wl.H, h.shape[1], wl.D)
            t.view(BH, h.shape[1], wl.D)[idx] = torch.from_numpy(h).to(device="cuda", dtype=torch.bfloat16)
            dev.append(t)
        out, lse = hmar.hmar_attn_scale_step(*dev, side_prev, side, wl.softmax_scale)
        ref_out, ref_lse = orc.scale_step(*host, wl.softmax_scale)
        _assert_close(f"out[scale {s}]", out.view(BH, -1, wl.D)[idx], ref_out, False)
        _assert_lse(lse.view(BH, -1)[idx], ref_lse, False)
        assert torch.isfinite(out).all() and torch.isfinite(lse).all()
    _no_device_error()


@pytest.mark.parametrize("sides", [(1, 2), (3, 4, 6), (9, 13), (13, 18), (18, 24), (5, 14)])
def test_scale_step_on_a_kv_ring_matches_dense_tensors_bits(sides):
    """K and V of the previous and the current scale adjacent in one ring buffer [B,H,ring_rows,D], q and out
    as slices of wider buffers: the strided entry point must give the oracle's result and the very bits of
    the dense entry point (both kernels: windows below and above 128 keys)."""
    wl = _Wl(sides, B=2, H=3)
    B, H, D = wl.B, wl.H, wl.D
    for s in range(1, len(sides)):
        n_prev, n_cur = sides[s - 1] ** 2, sides[s] ** 2
        q, kp, vp, kc, vc = scale_step_inputs(wl, s, 0, bf16=True)
        ring_rows = n_prev + n_cur + 24
        ring_k = torch.full((B, H, ring_rows, D), float("nan"), dtype=torch.bfloat16, device="cuda")
        ring_v = torch.full_like(ring_k, float("nan"))
        a = 8
        for ring, prev, cur in ((ring_k, kp, kc), (ring_v, vp, vc)):
            ring[:, :, a:a + n_prev] = to_device(prev, B, H, torch.bfloat16)
            ring[:, :, a + n_prev:a + n_prev + n_cur] = to_device(cur, B, H, torch.bfloat16)
        q_wide = torch.zeros((B, H, n_cur + 8, D), dtype=torch.bfloat16, device="cuda")
        q_wide[:, :, :n_cur] = to_device(q, B, H, torch.bfloat16)
        out_wide = torch.full((B, H, n_cur + 16, D), 7.0, dtype=torch.bfloat16, device="cuda")
        out, lse = hmar.hmar_attn_scale_step_strided(
            q_wide[:, :, :n_cur], ring_k[:, :, a:a + n_prev], ring_v[:, :, a:a + n_prev],
            ring_k[:, :, a + n_prev:a + n_prev + n_cur], ring_v[:, :, a + n_prev:a + n_prev + n_cur],
            sides[s - 1], sides[s], wl.softmax_scale, out=out_wide[:, :, :n_cur])
        ref_out, ref_lse = orc.scale_step(q, kp, vp, kc, vc, wl.softmax_scale)
        _assert_close("out", out_wide[:, :, :n_cur].contiguous(), ref_out, False)
        _assert_lse(lse, ref_lse, False)
        assert (out_wide[:, :, n_cur:] == 7.0).all()                     # nothing written past the head's rows
        dense = [to_device(x, B, H, torch.bfloat16) for x in (q, kp, vp, kc, vc)]
        out_d, lse_d = hmar.hmar_attn_scale_step(*dense, sides[s - 1], sides[s], wl.softmax_scale)
        assert torch.equal(out_d, out_wide[:, :, :n_cur]) and torch.equal(lse_d, lse)
    _no_device_error()


def test_scale_step_strided_argument_errors():
    import ctypes
    p = ctypes.c_void_p(1 << 12)
    f = hmar.lib().hmar_attn_scale_step_strided
    ok_strides = (16 * 64, 4 * 64, 16 * 64, 16 * 64)
    assert f(p, p, p, p, p, p, None, 1, 1, 64, 2, 4, 16 * 64 - 8, *ok_strides[1:], 0.125, None) == hmar.HMAR_ERR_BAD_ARG   # head shorter than its rows
    assert f(p, p, p, p, p, p, None, 1, 1, 64, 2, 4, 16 * 64 + 4, *ok_strides[1:], 0.125, None) == hmar.HMAR_ERR_BAD_ARG   # heads off the 16-byte grid
    assert f(p, None, None, p, p, p, None, 1, 1, 64, 2, 4, *ok_strides, 0.125, None) == hmar.HMAR_ERR_BAD_ARG              # prev missing


def test_full_size_forward_and_scale_step_repeat_bit_identical():
    """The forward paths have no atomics, so two runs on the same inputs must agree bit for bit, at the
    sizes where thousands of blocks start and finish at different times (a warp that reads its output
    accumulator before the last product has landed shows up here)."""
    wl = CONFIGS["512_d24_infer"]
    s = len(wl.side_lens) - 1
    side, side_prev = wl.side_lens[s], wl.side_lens[s - 1]
    t = [bulk_normal(wl.seed, i, wl.B, wl.H, (side_prev if i in (1, 2) else side) ** 2, wl.D) for i in range(5)]
    first, _ = hmar.hmar_attn_scale_step(*t, side_prev, side, wl.softmax_scale)
    for _ in range(4):
        again, _ = hmar.hmar_attn_scale_step(*t, side_prev, side, wl.softmax_scale)
        assert torch.equal(first, again)
    wt = CONFIGS["512_d24_train"]
    q, k, v = (bulk_normal(wt.seed, i, wt.B, wt.H, wt.L, wt.D) for i in range(3))
    o1, l1 = hmar.hmar_attn_fwd(q, k, v, wt.side_lens, wt.softmax_scale)
    for _ in range(3):
        o2, l2 = hmar.hmar_attn_fwd(q, k, v, wt.side_lens, wt.softmax_scale)
        assert torch.equal(o1, o2) and torch.equal(l1, l2)
    _no_device_error()


def test_scale_step_matches_training_forward_rows():
    """The inference step of scale k equals the scale-k rows of the training forward (same kernels'
    arithmetic, different entry point)."""
    wl = _Wl((2, 5, 12, 3))
    q, k, v, _ = training_inputs(wl, bf16=True)
    tq, tk, tv = (to_device(x, wl.B, wl.H, torch.bfloat16) for x in (q, k, v))
    out, lse = hmar.hmar_attn_fwd(tq, tk, tv, wl.side_lens, wl.softmax_scale)
    starts = np.concatenate([[0], np.cumsum([s * s for s in wl.side_lens])])
    for s, side in enumerate(wl.side_lens):
        cur = slice(starts[s], starts[s + 1])
        prev = slice(starts[s - 1], starts[s]) if s else None
        o, l = hmar.hmar_attn_scale_step(
            tq[:, :, cur].contiguous(),
            None if prev is None else tk[:, :, prev].contiguous(),
            None if prev is None else tv[:, :, prev].contiguous(),
            tk[:, :, cur].contiguous(), tv[:, :, cur].contiguous(),
            wl.side_lens[s - 1] if s else 0, side, wl.softmax_scale)
        assert (o.float() - out[:, :, cur].float()).abs().max().item() <= 1e-2
        assert (l - lse[:, :, cur]).abs().max().item() <= 1e-4


def test_bounded_wait_runs_out_reports_and_leaves_the_context_usable():
    """A kernel whose bounded wait runs out (a barrier nothing arrives on, 1 ms limit, the kernels' own wait
    and report routines) returns by itself; the status word reports it once; while the word is latched the
    tensor-core kernels return without writing; after the poll everything works again."""
    hmar.hmar_device_status()                                   # clear whatever earlier tests left
    hmar.hmar_selftest_bounded_wait()
    assert hmar.hmar_device_status() == (hmar.HMAR_ERR_DEVICE_TIMEOUT, 0xD1A6)
    assert hmar.hmar_device_status() == (hmar.HMAR_OK, 0)       # reported once, then clear
    wl = _Wl((3, 11, 5))
    q, k, v, do = training_inputs(wl, bf16=True)
    tq, tk, tv, tdo = (to_device(x, wl.B, wl.H, torch.bfloat16) for x in (q, k, v, do))
    hmar.hmar_selftest_bounded_wait()
    out = torch.full_like(tq, 7.0)
    hmar.hmar_attn_fwd(tq, tk, tv, wl.side_lens, wl.softmax_scale, out=out)      # launched while the word is latched
    torch.cuda.synchronize()
    assert (out == 7.0).all()
    assert hmar.hmar_device_status()[0] == hmar.HMAR_ERR_DEVICE_TIMEOUT
    _run_training(wl, torch.bfloat16)                           # and the library is back to normal


def test_bad_workspace_is_rejected():
    wl = CONFIGS["tiny"]
    q, k, v, do = training_inputs(wl)
    tq, tk, tv, tdo = (to_device(x, wl.B, wl.H, torch.bfloat16) for x in (q, k, v, do))
    out, lse = hmar.hmar_attn_fwd(tq, tk, tv, wl.side_lens, wl.softmax_scale)
    small = torch.empty(64, dtype=torch.uint8, device="cuda")
    with pytest.raises(hmar.HmarError) as e:
        hmar.hmar_attn_bwd(tq, tk, tv, out, lse, tdo, wl.side_lens, wl.softmax_scale, workspace=small)
    assert e.value.status == hmar.HMAR_ERR_WORKSPACE


def test_repeat_calls_are_stable():
    wl = _Wl((1, 2, 3, 4, 6, 9, 13))
    q, k, v, do = training_inputs(wl)
    tq, tk, tv, tdo = (to_device(x, wl.B, wl.H, torch.bfloat16) for x in (q, k, v, do))
    o1, l1 = hmar.hmar_attn_fwd(tq, tk, tv, wl.side_lens, wl.softmax_scale)
    o2, l2 = hmar.hmar_attn_fwd(tq, tk, tv, wl.side_lens, wl.softmax_scale)
    assert torch.equal(o1, o2) and torch.equal(l1, l2)     # the forward is deterministic
    g1 = hmar.hmar_attn_bwd(tq, tk, tv, o1, l1, tdo, wl.side_lens, wl.softmax_scale)
    g2 = hmar.hmar_attn_bwd(tq, tk, tv, o1, l1, tdo, wl.side_lens, wl.softmax_scale)
    assert torch.equal(g1[1], g2[1]) and torch.equal(g1[2], g2[2])        # dk, dv deterministic
    assert (g1[0].float() - g2[0].float()).abs().max().item() <= 2e-2     # dq: atomics, order may differ
    assert hmar.hmar_launch_count() > 0


@pytest.mark.parametrize("side,out_side,B,C,V", [(1, 32, 3, 32, 4096), (6, 32, 2, 32, 4096), (13, 32, 2, 32, 4096), (32, 32, 2, 32, 4096),
                                                  (3, 7, 2, 5, 17), (16, 16, 65, 32, 4096), (5, 16, 2, 40, 33), (40, 48, 1, 8, 50),
                                                  (8, 48, 2, 16, 100), (24, 64, 1, 8, 64), (8, 80, 1, 8, 30)])
@pytest.mark.parametrize("masked", [False, True])
def test_recon_accumulate_matches_oracle(side, out_side, B, C, V, masked):
    """The sampler's neighbour step (Alg. 2 lines 7-8 with the sub-step's token selection, Sec. 4.2) on a synthetic
    codebook: fp32 on the GPU against the fp64 oracle, and the selected token map bit for bit.  Maps of at most
    32 x 32 tokens and reconstructions of at most 64 x 64 take the staged kernel (also with more than 32 channels,
    and with more than 32 output columns), the 40 x 40 map and the 80 x 80 reconstruction the plain one."""
    rng = np.random.default_rng(1000 * side + out_side + int(masked))
    codebook = rng.standard_normal((V, C)).astype(np.float32)
    old = rng.integers(0, V, (B, side, side)).astype(np.int32)
    new = rng.integers(0, V, (B, side, side)).astype(np.int32)
    mask = rng.integers(0, 2, (B, side, side)).astype(np.uint8)
    x0 = rng.standard_normal((B, C, out_side, out_side)).astype(np.float32)
    dev = lambda a: torch.from_numpy(a).cuda()
    guards = []
    xhat = _guarded(x0.shape, torch.float32, guards)
    xhat.copy_(dev(x0))
    t_out = torch.full((B, side, side), -1, dtype=torch.int32, device="cuda")
    hmar.hmar_recon_accumulate(xhat, dev(codebook), dev(new), dev(old) if masked else None, dev(mask) if masked else None, t_out)
    sel = orc.select_tokens(old, new, mask) if masked else new
    ref = orc.recon_accumulate(x0, codebook, sel, out_side)
    assert torch.equal(t_out.cpu(), torch.from_numpy(sel.astype(np.int32)))
    err = np.abs(xhat.double().cpu().numpy() - ref)
    assert err.max() <= 1e-5 * max(1.0, np.abs(ref).max()), f"max abs err {err.max():.3e}"
    assert all(intact() for intact in guards)


@pytest.mark.parametrize("S,s,B,C", [(32, 1, 3, 5), (32, 13, 2, 32), (32, 16, 9, 8), (32, 32, 2, 4), (16, 6, 2, 7), (7, 3, 1, 3),
                                     (64, 24, 2, 3), (64, 64, 1, 2), (80, 9, 1, 2), (5, 5, 1, 1)])
def test_recon_downsample_matches_oracle(S, s, B, C):
    """The running reconstruction brought down to a scale's resolution (Sec. 4.1) by area interpolation: fp32 on the
    GPU against the fp64 oracle.  Planes of at most 64 x 64 take the staged kernel, the 80 x 80 case the plain one;
    the output sits between canaries."""
    rng = np.random.default_rng(100 * S + s)
    x = rng.standard_normal((B, C, S, S)).astype(np.float32)
    guards = []
    out = _guarded((B, C, s, s), torch.float32, guards)
    xg = torch.from_numpy(x).cuda()
    res = hmar.hmar_recon_downsample(xg, s, out=out)
    assert res is out
    ref = orc.area_downsample(x, s)
    err = np.abs(out.double().cpu().numpy() - ref)
    assert err.max() <= 1e-5 * max(1.0, np.abs(ref).max()), f"max abs err {err.max():.3e}"
    assert torch.equal(xg.cpu(), torch.from_numpy(x))           # the input is read only
    assert all(intact() for intact in guards)


def test_recon_accumulate_codebook_off_16_byte_alignment():
    """A codebook whose base address is not a multiple of 16 bytes takes the staged kernel's one-value-at-a-time
    gather; same result as the oracle."""
    rng = np.random.default_rng(77)
    V, C, side, out_side, B = 40, 8, 6, 16, 2
    codebook = rng.standard_normal((V, C)).astype(np.float32)
    new = rng.integers(0, V, (B, side, side)).astype(np.int32)
    x0 = rng.standard_normal((B, C, out_side, out_side)).astype(np.float32)
    buf = torch.zeros(V * C + 1, dtype=torch.float32, device="cuda")
    cb = buf[1:].view(V, C)
    cb.copy_(torch.from_numpy(codebook))
    assert cb.data_ptr() % 16 == 4
    xhat = torch.from_numpy(x0).cuda()
    hmar.hmar_recon_accumulate(xhat, cb, torch.from_numpy(new).cuda())
    ref = orc.recon_accumulate(x0, codebook, new, out_side)
    err = np.abs(xhat.double().cpu().numpy() - ref)
    assert err.max() <= 1e-5 * max(1.0, np.abs(ref).max()), f"max abs err {err.max():.3e}"


def test_edge_cases_through_the_checking_build():
    """The library compiled with -DHMAR_BOUNDS_CHECK compares every address its kernels form by their own
    arithmetic (plain loads and stores; TMA copies are clipped by the hardware) with the extent of its tensor and
    records HMAR_ERR_BOUNDS instead of accessing.  The edge-case side lists, the packed layouts, the K/V ring and
    the small-window step run through it in a fresh process; _no_device_error() in those tests fails on any
    recorded code, and the results still have to match the oracle."""
    import os
    import subprocess
    import sys
    from paper_2506_04421_b200 import build as b
    lib_path = b.build(checked=True)
    env = dict(os.environ, HMAR_LIBRARY=lib_path)
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    sel = "test_edge_side_lists_fwd_bwd or test_config1 or test_packed_qkv_backward or test_scale_step_on_a_kv_ring or " \
          "test_scale_step_small_batch_all_scales or test_other_block_masks_fwd_bwd"
    res = subprocess.run([sys.executable, "-m", "pytest", os.path.join(root, "tests", "test_gpu_parity.py"), "-x", "-q", "-m", "gpu",
                          "-k", sel, "-p", "no:cacheprovider"], env=env, capture_output=True, text=True, cwd=root, timeout=900)
    assert res.returncode == 0, res.stdout[-3000:] + res.stderr[-1000:]
    assert " passed" in res.stdout
