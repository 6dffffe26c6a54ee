"""Pins for the CPU oracle: what the paper and the mathematics fix, independent of the oracle.

Each test names the mistake it is meant to catch. None of them needs a GPU.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import hmar_oracle as orc
from workloads import CONFIGS, training_inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_golden(name):
    vals = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                key, val = line.split()[:2]
                vals[key] = float(val)
    return vals


# --------------------------------------------------------------------------- bookkeeping

def test_paper_sequence_constants():
    g = _read_golden("paper_constants.txt")
    _, _, L16 = orc.scale_layout(range(1, 17))
    assert round(L16 / 256.0, 2) == g["seq_ratio_256_16scales"]
    n, _, _ = orc.scale_layout(CONFIGS["256_d16_fwd"].side_lens)
    assert len(n) == g["num_scales"]
    assert n[-1] / n[0] == g["finest_over_coarsest_256"]


@pytest.mark.parametrize("name,L,pairs", [("tiny", 30, 538), ("256_d16_fwd", 680, 180820),
                                          ("512_d24_train", 2240, 2370669)])
def test_lengths_and_pair_counts(name, L, pairs):
    sides = CONFIGS[name].side_lens
    n, start, total = orc.scale_layout(sides)
    assert total == L == CONFIGS[name].L
    assert start[0] == 0 and all(start[i + 1] - start[i] == sides[i] ** 2 for i in range(len(sides)))
    # closed form: every token of scale k sees n_k + n_{k-1} keys
    closed = sum(int(n[i]) * (int(n[i]) + (int(n[i - 1]) if i else 0)) for i in range(len(n)))
    assert closed == pairs == orc.count_pairs(sides)


def test_mask_literals():
    # sides (1,1,1): one token per scale -> a bidiagonal band; catches an off-by-one in the window
    assert orc.hmar_mask((1, 1, 1)).astype(int).tolist() == [[1, 0, 0], [1, 1, 0], [0, 1, 1]]
    # sides (1,2): the four scale-2 tokens see everything; token 0 sees itself only
    assert orc.hmar_mask((1, 2)).astype(int).tolist() == [[1, 0, 0, 0, 0]] + [[1] * 5] * 4
    # sides (1,1,2): scale 3 must NOT see scale 1 (block-causal would)
    m = orc.hmar_mask((1, 1, 2)).astype(int).tolist()
    assert m == [[1, 0, 0, 0, 0, 0], [1, 1, 0, 0, 0, 0]] + [[0, 1, 1, 1, 1, 1]] * 4


def _scale_by_scan(i, sides):
    acc = 0
    for s, side in enumerate(sides):
        acc += side * side
        if i < acc:
            return s
    raise IndexError


def test_mask_brute_force_non_monotone_sides():
    sides = (2, 1, 3, 1, 2)
    M = orc.hmar_mask(sides)
    L = sum(s * s for s in sides)
    assert M.shape == (L, L)
    for i in range(L):
        for j in range(L):
            si, sj = _scale_by_scan(i, sides), _scale_by_scan(j, sides)
            assert bool(M[i, j]) == (sj == si or sj == si - 1)
    # within-scale attention is bidirectional (Sec. 3): diagonal blocks are symmetric and full
    assert (M & M.T).sum() == sum((s * s) ** 2 for s in sides)


def test_block_causal_is_superset_and_denser():
    sides = CONFIGS["256_d16_fwd"].side_lens
    H, C = orc.hmar_mask(sides), orc.block_causal_mask(sides)
    assert not (H & ~C).any()
    assert C.sum() > H.sum()


# --------------------------------------------------------------------------- the other masks of the family

def test_window_masks_pair_counts_closed_forms():
    # block-causal: every token of scale k sees start[k+1] tokens; block-diagonal: n_k tokens
    for sides in (CONFIGS["256_d16_fwd"].side_lens, CONFIGS["512_d24_train"].side_lens, (3, 1, 2)):
        n = [x * x for x in sides]
        start = np.concatenate([[0], np.cumsum(n)])
        assert orc.count_pairs(sides, "causal") == sum(n[k] * start[k + 1] for k in range(len(n)))
        assert orc.count_pairs(sides, "self") == sum(x * x for x in n)
        # preceding scale only: n_k * n_{k-1} pairs per scale, and the first scale on itself
        assert orc.count_pairs(sides, "prev") == n[0] * n[0] + sum(n[k] * n[k - 1] for k in range(1, len(n)))
    # densities quoted for the paper's shapes: block-causal 61.9 % at L = 680 and 65.2 % at L = 2240
    assert orc.count_pairs(CONFIGS["256_d16_fwd"].side_lens, "causal") / 680 ** 2 == pytest.approx(0.619, abs=5e-4)
    assert orc.count_pairs(CONFIGS["512_d24_train"].side_lens, "causal") / 2240 ** 2 == pytest.approx(0.652, abs=5e-4)
    with pytest.raises(ValueError):
        orc.window_mask((1, 2), "dense")


def test_window_masks_single_scale_all_dense_and_nesting():
    for w in ("markov", "causal", "self", "prev"):
        assert orc.window_mask((5,), w).all()
    sides = (2, 3, 1, 4)
    S, M, C = (orc.window_mask(sides, w) for w in ("self", "markov", "causal"))
    assert not (S & ~M).any() and not (M & ~C).any() and S.sum() < M.sum() < C.sum()
    assert (S == S.T).all() and not (C == C.T).all()
    # the preceding-scale mask and the block-diagonal one split the Markov mask between them, except for the
    # first scale's own block, which both hold
    P = orc.window_mask(sides, "prev")
    assert ((P | S) == M).all() and (P & S).sum() == sides[0] ** 4
    assert P.any(axis=1).all()                                           # no empty row
    assert not P[:, -(sides[-1] ** 2):].any()                            # nobody looks at the last scale's keys


def test_prev_window_literals_and_locality():
    # sides (1, 1, 2): token 0 sees itself; token 1 sees token 0; tokens 2-5 see token 1 only
    expect = np.zeros((6, 6), dtype=bool)
    expect[0, 0] = expect[1, 0] = True
    expect[2:, 1] = True
    assert (orc.window_mask((1, 1, 2), "prev") == expect).all()
    rng = np.random.default_rng(21)
    sides = (2, 1, 3, 2)
    n = [x * x for x in sides]
    start = np.concatenate([[0], np.cumsum(n)])
    L = int(start[-1])
    q, k, v, do = (rng.standard_normal((L, 6)) for _ in range(4))
    out, lse = orc.attn_fwd(q, k, v, sides, 0.4, window="prev")
    # scale 2 (one token in scale 1... a single key) : rows of scale index 2 see the single token of scale index 1,
    # so their output is exactly that token's value and lse is the one logit
    np.testing.assert_allclose(out[start[2]:start[3]], np.broadcast_to(v[start[1]], (n[2], 6)), rtol=1e-13)
    np.testing.assert_allclose(lse[start[2]:start[3]], 0.4 * q[start[2]:start[3]] @ k[start[1]], rtol=1e-13)
    # rows of scale k do not move when their own scale's keys change, and do when the preceding scale's do
    k2, v2 = k.copy(), v.copy()
    k2[start[3]:] += 1.0
    v2[start[3]:] -= 2.0
    out2, _ = orc.attn_fwd(q, k2, v2, sides, 0.4, window="prev")
    assert np.array_equal(out, out2)                                     # the last scale's keys reach nothing
    v3 = v.copy()
    v3[start[2]:start[3]] += 1.0
    out3, _ = orc.attn_fwd(q, k, v3, sides, 0.4, window="prev")
    assert np.array_equal(out[:start[3]], out3[:start[3]]) and not np.allclose(out[start[3]:], out3[start[3]:])
    # the last scale is plain dense attention over the preceding scale's keys (library softmax as the check)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q[start[3]:])[None], torch.from_numpy(k[start[2]:start[3]])[None],
        torch.from_numpy(v[start[2]:start[3]])[None], scale=0.4)[0].numpy()
    np.testing.assert_allclose(out[start[3]:], ref, rtol=1e-12, atol=1e-12)
    # backward: keys of the last scale get exactly zero, and central differences agree elsewhere
    dq, dk, dv = orc.attn_bwd(q, k, v, do, sides, 0.4, window="prev")
    assert not dk[start[3]:].any() and not dv[start[3]:].any()
    for grad, idx in ((dq, 0), (dk, 1), (dv, 2)):
        for _ in range(12):
            i, d = int(rng.integers(L)), int(rng.integers(6))
            args = [q.copy(), k.copy(), v.copy()]
            args[idx][i, d] += 1e-6
            fp = (orc.attn_fwd(*args, sides, 0.4, window="prev")[0] * do).sum()
            args[idx][i, d] -= 2e-6
            fm = (orc.attn_fwd(*args, sides, 0.4, window="prev")[0] * do).sum()
            assert (fp - fm) / 2e-6 == pytest.approx(grad[i, d], rel=1e-6, abs=1e-8)


def test_self_window_is_independent_attention_per_scale():
    # block-diagonal attention = plain dense attention of every scale on its own (library softmax as the check)
    rng = np.random.default_rng(11)
    sides = (2, 3, 1, 4)
    L = sum(x * x for x in sides)
    q, k, v = (rng.standard_normal((L, 8)) for _ in range(3))
    out, lse = orc.attn_fwd(q, k, v, sides, 0.3, window="self")
    pos = 0
    for sd in sides:
        n = sd * sd
        sl = slice(pos, pos + n)
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(q[sl])[None], torch.from_numpy(k[sl])[None], torch.from_numpy(v[sl])[None], scale=0.3)[0].numpy()
        np.testing.assert_allclose(out[sl], ref, rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(lse[sl], np.log(np.exp(0.3 * q[sl] @ k[sl].T).sum(axis=1)), rtol=1e-12)
        pos += n


def test_causal_window_locality_and_backward():
    rng = np.random.default_rng(12)
    sides = (2, 1, 3, 2)
    n = [x * x for x in sides]
    start = np.concatenate([[0], np.cumsum(n)])
    L = int(start[-1])
    q, k, v, do = (rng.standard_normal((L, 6)) for _ in range(4))
    out, _ = orc.attn_fwd(q, k, v, sides, 0.4, window="causal")
    # scale-k rows do not move when a later scale changes, and do move when the first scale changes
    k2, v2 = k.copy(), v.copy()
    k2[start[3]:] += 1.0
    v2[start[3]:] -= 2.0
    out2, _ = orc.attn_fwd(q, k2, v2, sides, 0.4, window="causal")
    assert np.array_equal(out[:start[3]], out2[:start[3]]) and not np.allclose(out[start[3]:], out2[start[3]:])
    v3 = v.copy()
    v3[0] += 5.0
    out3, _ = orc.attn_fwd(q, k, v3, sides, 0.4, window="causal")
    assert not np.allclose(out[start[3]:], out3[start[3]:])          # the last scale still sees token 0
    outm, _ = orc.attn_fwd(q, k, v3, sides, 0.4)                      # ... which it does not under the Markov mask
    outm0, _ = orc.attn_fwd(q, k, v, sides, 0.4)
    assert np.array_equal(outm[start[3]:], outm0[start[3]:])
    # the last row of a block-causal mask is dense: textbook attention over everything
    w = np.exp(0.4 * q[-1] @ k.T)
    np.testing.assert_allclose(out[-1], (w / w.sum()) @ v, rtol=1e-12)
    # backward by central differences, for both added masks
    for window in ("causal", "self"):
        dq, dk, dv = orc.attn_bwd(q, k, v, do, sides, 0.4, window=window)
        for grad, idx in ((dq, 0), (dk, 1), (dv, 2)):
            for _ in range(12):
                i, d = int(rng.integers(L)), int(rng.integers(6))
                args = [q.copy(), k.copy(), v.copy()]
                args[idx][i, d] += 1e-6
                fp = (orc.attn_fwd(*args, sides, 0.4, window=window)[0] * do).sum()
                args[idx][i, d] -= 2e-6
                fm = (orc.attn_fwd(*args, sides, 0.4, window=window)[0] * do).sum()
                assert (fp - fm) / 2e-6 == pytest.approx(grad[i, d], rel=1e-6, abs=1e-8)


# --------------------------------------------------------------------------- forward

def _brute_forward(q, k, v, sides, scale):
    """Pure-Python loops straight from the definition of masked softmax attention."""
    L, D = q.shape
    out = [[0.0] * D for _ in range(L)]
    lse = [0.0] * L
    for i in range(L):
        si = _scale_by_scan(i, sides)
        allowed = [j for j in range(L) if _scale_by_scan(j, sides) in (si, si - 1)]
        logits = [scale * sum(float(q[i, d]) * float(k[j, d]) for d in range(D)) for j in allowed]
        z = sum(math.exp(x) for x in logits)
        lse[i] = math.log(z)
        for j, x in zip(allowed, logits):
            w = math.exp(x) / z
            for d in range(D):
                out[i][d] += w * float(v[j, d])
    return np.array(out), np.array(lse)


def test_forward_two_token_closed_form():
    g = _read_golden("two_token_example.txt")
    q = np.array([[1.0], [2.0]])
    k = np.array([[3.0], [1.0]])
    v = np.array([[10.0], [20.0]])
    out, lse = orc.attn_fwd(q, k, v, (1, 1), 0.5)
    assert out[0, 0] == pytest.approx(g["out0"], abs=1e-14)
    assert lse[0] == pytest.approx(g["lse0"], abs=1e-14)
    assert out[1, 0] == pytest.approx(g["out1"], abs=1e-12)
    assert lse[1] == pytest.approx(g["lse1"], abs=1e-12)


def test_forward_brute_force_tiny():
    rng = np.random.default_rng(1)
    sides = (1, 2, 1, 3)
    L, D = sum(s * s for s in sides), 5
    q, k, v = (rng.standard_normal((L, D)) for _ in range(3))
    out, lse = orc.attn_fwd(q, k, v, sides, 0.37)
    bo, bl = _brute_forward(q, k, v, sides, 0.37)
    np.testing.assert_allclose(out, bo, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, bl, rtol=0, atol=1e-12)


def test_forward_single_scale_is_dense_sdpa():
    # one scale -> no masking at all -> textbook attention; cross-checked with a library routine
    rng = np.random.default_rng(2)
    q, k, v = (rng.standard_normal((2, 3, 16, 8)) for _ in range(3))
    out, lse = orc.attn_fwd(q, k, v, (4,), 0.25)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v), scale=0.25)
    np.testing.assert_allclose(out, ref.numpy(), atol=1e-12)
    ref_lse = torch.logsumexp(0.25 * torch.from_numpy(q) @ torch.from_numpy(k).transpose(-1, -2), -1)
    np.testing.assert_allclose(lse, ref_lse.numpy(), atol=1e-12)


def test_forward_two_scales_second_scale_is_dense():
    rng = np.random.default_rng(3)
    sides = (2, 3)
    L = 13
    q, k, v = (rng.standard_normal((L, 8)) for _ in range(3))
    out, _ = orc.attn_fwd(q, k, v, sides, 0.3)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q[4:])[None], torch.from_numpy(k)[None], torch.from_numpy(v)[None], scale=0.3)[0]
    np.testing.assert_allclose(out[4:], ref.numpy(), atol=1e-12)


def _tiny(bf16=False):
    wl = CONFIGS["tiny"]
    q, k, v, do = training_inputs(wl, bf16=bf16)
    return wl, q.astype(np.float64), k.astype(np.float64), v.astype(np.float64), do.astype(np.float64)


def test_forward_row0_and_equal_keys_closed_forms():
    wl, q, k, v, _ = _tiny()
    out, lse = orc.attn_fwd(q, k, v, wl.side_lens, wl.softmax_scale)
    # token 0 sees only itself
    np.testing.assert_allclose(out[:, 0], v[:, 0], atol=1e-14)
    np.testing.assert_allclose(lse[:, 0], wl.softmax_scale * (q[:, 0] * k[:, 0]).sum(-1), atol=1e-13)
    # all keys identical -> uniform weights over the allowed set A(i), |A(i)| = n_k + n_{k-1}
    k_same = np.broadcast_to(k[:, :1], k.shape)
    out2, lse2 = orc.attn_fwd(q, k_same, v, wl.side_lens, wl.softmax_scale)
    n, start, L = orc.scale_layout(wl.side_lens)
    for s in range(len(n)):
        lo = start[s - 1] if s else 0
        hi = start[s + 1]
        mean_v = v[:, lo:hi].mean(axis=1, keepdims=True)
        rows = slice(start[s], start[s + 1])
        np.testing.assert_allclose(out2[:, rows], np.broadcast_to(mean_v, out2[:, rows].shape), atol=1e-13)
        logit = wl.softmax_scale * (q[:, rows] * k_same[:, rows]).sum(-1)
        np.testing.assert_allclose(lse2[:, rows], logit + math.log(hi - lo), atol=1e-12)
    # constant V -> constant O (rows of P sum to one)
    out3, _ = orc.attn_fwd(q, k, np.full_like(v, 2.5), wl.side_lens, wl.softmax_scale)
    np.testing.assert_allclose(out3, 2.5, atol=1e-13)


def test_forward_markov_locality_and_permutation():
    wl, q, k, v, _ = _tiny()
    sides = wl.side_lens
    n, start, L = orc.scale_layout(sides)
    out, lse = orc.attn_fwd(q, k, v, sides, wl.softmax_scale)
    rng = np.random.default_rng(4)
    for s in range(len(n)):
        k2, v2 = k.copy(), v.copy()
        sl = slice(start[s], start[s + 1])
        k2[:, sl] += rng.standard_normal(k2[:, sl].shape)
        v2[:, sl] -= 3.0
        out2, lse2 = orc.attn_fwd(q, k2, v2, sides, wl.softmax_scale)
        changed = np.abs(out2 - out).max(axis=(0, 2)) > 0
        tok_scale = orc.scale_of_token(sides)
        # only scales s and s+1 may change, and they must change
        assert not changed[(tok_scale != s) & (tok_scale != s + 1)].any()
        assert changed[tok_scale == s].all()
        if s + 1 < len(n):
            assert changed[tok_scale == s + 1].all()
    # scale-1 rows depend on scale 1 only
    q2, k2, v2 = q.copy(), k.copy(), v.copy()
    k2[:, 1:] = 7.0
    v2[:, 1:] = -7.0
    out2, _ = orc.attn_fwd(q2, k2, v2, sides, wl.softmax_scale)
    assert np.array_equal(out2[:, 0], out[:, 0])
    # permuting the tokens of one scale permutes that scale's outputs and nothing else
    s = 2
    perm = np.arange(L)
    perm[start[s]:start[s + 1]] = start[s] + rng.permutation(n[s])
    outp, lsep = orc.attn_fwd(q[:, perm], k[:, perm], v[:, perm], sides, wl.softmax_scale)
    np.testing.assert_allclose(outp, out[:, perm], atol=1e-13)
    np.testing.assert_allclose(lsep, lse[:, perm], atol=1e-13)


def test_probs_rows_sum_to_one():
    wl, q, k, v, _ = _tiny()
    P, _ = orc.attention_probs(q, k, orc.hmar_mask(wl.side_lens), wl.softmax_scale)
    np.testing.assert_allclose(P.sum(-1), 1.0, atol=1e-14)
    assert (P[..., ~orc.hmar_mask(wl.side_lens)] == 0).all()


# --------------------------------------------------------------------------- backward

def _loss(q, k, v, do, sides, scale):
    out, _ = orc.attn_fwd(q, k, v, sides, scale)
    return float((out * do).sum())


def test_backward_finite_differences():
    wl, q, k, v, do = _tiny()
    # one head, leading D/4 columns of a few rows keep the loop short while touching every scale
    q, k, v, do = q[:1], k[:1], v[:1], do[:1]
    dq, dk, dv = orc.attn_bwd(q, k, v, do, wl.side_lens, wl.softmax_scale)
    eps = 1e-6
    rng = np.random.default_rng(5)
    for name, grad, idx in (("q", dq, 0), ("k", dk, 1), ("v", dv, 2)):
        for _ in range(40):
            i, d = int(rng.integers(q.shape[1])), int(rng.integers(q.shape[2]))
            args = [q.copy(), k.copy(), v.copy()]
            args[idx][0, i, d] += eps
            fp = _loss(*args, do, wl.side_lens, wl.softmax_scale)
            args[idx][0, i, d] -= 2 * eps
            fm = _loss(*args, do, wl.side_lens, wl.softmax_scale)
            fd = (fp - fm) / (2 * eps)
            assert fd == pytest.approx(grad[0, i, d], rel=1e-6, abs=1e-8), (name, i, d)


def test_backward_matches_autograd_of_explicit_mask():
    # autograd differentiates the forward definition; the mask comes from the scan helper above
    sides = (1, 2, 1, 2)
    L, D = 10, 6
    rng = np.random.default_rng(6)
    q, k, v, do = (rng.standard_normal((L, D)) for _ in range(4))
    M = torch.tensor([[_scale_by_scan(j, sides) in (_scale_by_scan(i, sides), _scale_by_scan(i, sides) - 1)
                       for j in range(L)] for i in range(L)])
    tq, tk, tv = (torch.tensor(x, requires_grad=True) for x in (q, k, v))
    S = (0.41 * tq @ tk.T).masked_fill(~M, float("-inf"))
    (torch.softmax(S, -1) @ tv * torch.tensor(do)).sum().backward()
    dq, dk, dv = orc.attn_bwd(q, k, v, do, sides, 0.41)
    np.testing.assert_allclose(dq, tq.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(dk, tk.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(dv, tv.grad.numpy(), atol=1e-12)


def test_backward_invariants():
    wl, q, k, v, do = _tiny()
    sides = wl.side_lens
    dq, dk, dv = orc.attn_bwd(q, k, v, do, sides, wl.softmax_scale)
    # rows of P sum to one -> column sums of dV equal column sums of dO
    np.testing.assert_allclose(dv.sum(axis=1), do.sum(axis=1), atol=1e-12)
    # softmax is shift invariant: adding a constant vector c to every key changes logits of row i by
    # scale*q_i.c for all j alike -> sum_j dK_j = 0
    np.testing.assert_allclose(dk.sum(axis=1), 0.0, atol=1e-12)
    # all keys identical -> P does not depend on q -> dQ = 0
    k_same = np.broadcast_to(k[:, :1], k.shape).copy()
    dq0, _, _ = orc.attn_bwd(q, k_same, v, do, sides, wl.softmax_scale)
    np.testing.assert_allclose(dq0, 0.0, atol=1e-13)
    # gradient of a linear functional is linear in dO
    dq2, dk2, dv2 = orc.attn_bwd(q, k, v, -2.0 * do, sides, wl.softmax_scale)
    np.testing.assert_allclose(dq2, -2.0 * dq, atol=1e-12)
    np.testing.assert_allclose(dk2, -2.0 * dk, atol=1e-12)
    np.testing.assert_allclose(dv2, -2.0 * dv, atol=1e-12)


def test_backward_locality():
    wl, q, k, v, do = _tiny()
    sides = wl.side_lens
    n, start, L = orc.scale_layout(sides)
    tok_scale = orc.scale_of_token(sides)
    for s in range(len(n)):
        d1 = np.zeros_like(do)
        d1[:, start[s]:start[s + 1]] = do[:, start[s]:start[s + 1]]
        dq, dk, dv = orc.attn_bwd(q, k, v, d1, sides, wl.softmax_scale)
        kv_live = (tok_scale == s) | (tok_scale == s - 1)
        assert (dk[:, ~kv_live] == 0).all() and (dv[:, ~kv_live] == 0).all()
        assert (np.abs(dv[:, kv_live]).sum(-1) > 0).all()
        assert (dq[:, tok_scale != s] == 0).all()


# --------------------------------------------------------------------------- inference step

def test_scale_step_equals_rows_of_training_forward():
    wl, q, k, v, _ = _tiny()
    sides = wl.side_lens
    n, start, L = orc.scale_layout(sides)
    out, lse = orc.attn_fwd(q, k, v, sides, wl.softmax_scale)
    for s in range(len(n)):
        cur = slice(start[s], start[s + 1])
        if s == 0:
            o, l = orc.scale_step(q[:, cur], None, None, k[:, cur], v[:, cur], wl.softmax_scale)
        else:
            prev = slice(start[s - 1], start[s])
            o, l = orc.scale_step(q[:, cur], k[:, prev], v[:, prev], k[:, cur], v[:, cur], wl.softmax_scale)
        np.testing.assert_allclose(o, out[:, cur], atol=1e-13)
        np.testing.assert_allclose(l, lse[:, cur], atol=1e-13)


def test_scale_step_brute_force():
    rng = np.random.default_rng(7)
    q = rng.standard_normal((4, 3))
    kp, vp = rng.standard_normal((1, 3)), rng.standard_normal((1, 3))
    kc, vc = rng.standard_normal((4, 3)), rng.standard_normal((4, 3))
    o, l = orc.scale_step(q, kp, vp, kc, vc, 0.7)
    keys = [kp[0]] + list(kc)
    vals = [vp[0]] + list(vc)
    for i in range(4):
        w = [math.exp(0.7 * float(q[i] @ kk)) for kk in keys]
        z = sum(w)
        assert l[i] == pytest.approx(math.log(z), abs=1e-12)
        np.testing.assert_allclose(o[i], sum(wi / z * vi for wi, vi in zip(w, vals)), atol=1e-12)


# --------------------------------------------------------------------------- planted mistakes

def test_pins_detect_planted_mistakes(monkeypatch):
    """Plant plausible mistakes in the oracle (on the CPU) and check that a pin above fails."""
    def fails(test, *a):
        try:
            test(*a)
        except AssertionError:
            return True
        return False

    good_mask = orc.hmar_mask
    # (1) block-causal instead of Markovian
    monkeypatch.setattr(orc, "hmar_mask", orc.block_causal_mask)
    assert fails(test_mask_literals) and fails(test_forward_brute_force_tiny)
    # (2) self-only window
    monkeypatch.setattr(orc, "hmar_mask", lambda s: good_mask(s) & good_mask(s).T)
    assert fails(test_mask_literals) and fails(test_forward_two_token_closed_form)
    # (3) window looks forward instead of backward
    monkeypatch.setattr(orc, "hmar_mask", lambda s: good_mask(s).T)
    assert fails(test_forward_brute_force_tiny) and fails(test_backward_locality)
    monkeypatch.setattr(orc, "hmar_mask", good_mask)

    good_probs = orc.attention_probs
    # (4) scale applied to lse twice / dropped from the logits
    monkeypatch.setattr(orc, "attention_probs", lambda q, k, m, s: good_probs(q, k, m, 1.0))
    assert fails(test_forward_two_token_closed_form) and fails(test_backward_finite_differences)
    # (5) transposed score matrix
    def transposed(q, k, m, s):
        return good_probs(k, q, m, s) if q.shape == k.shape else good_probs(q, k, m, s)
    monkeypatch.setattr(orc, "attention_probs", transposed)
    assert fails(test_forward_brute_force_tiny)
    monkeypatch.setattr(orc, "attention_probs", good_probs)

    # (6) backward with the delta term dropped, wrong sign, or missing scale
    good_bwd = orc.attn_bwd

    def no_delta(q, k, v, do, sides, scale):
        P, _ = good_probs(np.asarray(q, float), np.asarray(k, float), good_mask(sides), scale)
        dP = do @ np.swapaxes(v, -1, -2)
        dS = P * dP
        return scale * dS @ k, scale * np.swapaxes(dS, -1, -2) @ q, np.swapaxes(P, -1, -2) @ do
    monkeypatch.setattr(orc, "attn_bwd", no_delta)
    assert fails(test_backward_finite_differences) and fails(test_backward_invariants)
    monkeypatch.setattr(orc, "attn_bwd", lambda *a: tuple(-g for g in good_bwd(*a)))
    assert fails(test_backward_finite_differences)
    monkeypatch.setattr(orc, "attn_bwd", lambda *a: (good_bwd(*a)[0] / a[-1],) + good_bwd(*a)[1:])
    assert fails(test_backward_matches_autograd_of_explicit_mask)
    # (7) dQ and dK swapped
    monkeypatch.setattr(orc, "attn_bwd", lambda *a: (good_bwd(*a)[1], good_bwd(*a)[0], good_bwd(*a)[2]))
    assert fails(test_backward_finite_differences)


# --------------------------------------------------------------------------- the sampler's neighbour step (Alg. 2)

def test_cubic_weights_literals_and_partition_of_unity():
    # a = -0.75: at t = 0 the sample sits on a source pixel; at t = 1/2 the classic (-3, 19, 19, -3) / 32 taps
    np.testing.assert_allclose(orc._cubic_weights(0.0), [0.0, 1.0, 0.0, 0.0], atol=1e-15)
    np.testing.assert_allclose(orc._cubic_weights(0.5), np.array([-3.0, 19.0, 19.0, -3.0]) / 32.0, atol=1e-15)
    for t in np.linspace(0.0, 0.999, 37):
        w = orc._cubic_weights(t)
        assert w.sum() == pytest.approx(1.0, abs=1e-14)
        np.testing.assert_allclose(w[::-1], orc._cubic_weights(1.0 - t) if t > 0 else [0, 0, 1, 0], atol=1e-14)


def test_bicubic_upsample_against_the_library_routine_and_special_cases():
    rng = np.random.default_rng(31)
    for h, H in ((1, 8), (2, 7), (3, 8), (5, 16), (13, 32), (6, 6)):
        x = rng.standard_normal((2, 3, h, h))
        ref = torch.nn.functional.interpolate(torch.from_numpy(x), size=(H, H), mode="bicubic", align_corners=False).numpy()
        np.testing.assert_allclose(orc.bicubic_upsample(x, H), ref, rtol=1e-12, atol=1e-13)
    x = rng.standard_normal((4, 4))
    assert np.array_equal(orc.bicubic_upsample(x, 4), x)                               # same size: identity
    np.testing.assert_allclose(orc.bicubic_upsample(np.full((3, 3), 2.5), 9), 2.5, rtol=1e-14)   # constants stay
    np.testing.assert_allclose(orc.bicubic_upsample(np.array([[1.75]]), 5), 1.75, rtol=1e-14)    # one token: flat image
    y = rng.standard_normal((4, 4))
    np.testing.assert_allclose(orc.bicubic_upsample(2.0 * x - 3.0 * y, 11),
                               2.0 * orc.bicubic_upsample(x, 11) - 3.0 * orc.bicubic_upsample(y, 11), rtol=1e-12, atol=1e-13)
    # transposing the input transposes the output (rows and columns are treated alike)
    np.testing.assert_allclose(orc.bicubic_upsample(x.T, 10), orc.bicubic_upsample(x, 10).T, rtol=1e-13, atol=1e-14)


def test_select_tokens_and_recon_accumulate():
    rng = np.random.default_rng(32)
    B, C, V, side, S = 2, 5, 17, 3, 8
    codebook = rng.standard_normal((V, C))
    old, new = rng.integers(0, V, (B, side, side)), rng.integers(0, V, (B, side, side))
    mask = rng.integers(0, 2, (B, side, side))
    sel = orc.select_tokens(old, new, mask)
    assert np.array_equal(sel[mask == 1], new[mask == 1]) and np.array_equal(sel[mask == 0], old[mask == 0])
    assert np.array_equal(orc.select_tokens(old, new, np.zeros_like(mask)), old)
    assert np.array_equal(orc.select_tokens(old, new, np.ones_like(mask)), new)
    x0 = rng.standard_normal((B, C, S, S))
    x1 = orc.recon_accumulate(x0, codebook, sel, S)
    # written out by hand for one output pixel and channel: the 16 taps around the sample position
    b, c, oy, ox = 1, 3, 5, 2
    sy, sx = (oy + 0.5) * side / S - 0.5, (ox + 0.5) * side / S - 0.5
    iy, ix = int(np.floor(sy)), int(np.floor(sx))
    wy, wx = orc._cubic_weights(sy - iy), orc._cubic_weights(sx - ix)
    acc = 0.0
    for a in range(4):
        for d in range(4):
            yy, xx = min(max(iy - 1 + a, 0), side - 1), min(max(ix - 1 + d, 0), side - 1)
            acc += wy[a] * wx[d] * codebook[sel[b, yy, xx], c]
    assert x1[b, c, oy, ox] == pytest.approx(x0[b, c, oy, ox] + acc, rel=1e-13)
    # a codebook of one repeated vector: every pixel gains exactly that vector, whatever the tokens
    flat = np.tile(rng.standard_normal((1, C)), (V, 1))
    np.testing.assert_allclose(orc.recon_accumulate(x0, flat, sel, S) - x0, flat[0][None, :, None, None] * np.ones((B, C, S, S)), rtol=1e-12, atol=1e-13)
    # Alg. 2's loop: the reconstruction after two scales is the sum of the two interpolated maps
    t2 = rng.integers(0, V, (B, 5, 5))
    both = orc.recon_accumulate(orc.recon_accumulate(np.zeros((B, C, S, S)), codebook, sel, S), codebook, t2, S)
    np.testing.assert_allclose(both, orc.recon_accumulate(np.zeros((B, C, S, S)), codebook, t2, S) + (x1 - x0), rtol=1e-12, atol=1e-13)


def test_pins_detect_planted_mistakes_in_the_added_functions(monkeypatch):
    """The same exercise for the preceding-scale mask and the reconstruction step."""
    def fails(test, *a):
        try:
            test(*a)
        except AssertionError:
            return True
        return False

    # (1) preceding-scale mask whose first scale sees nothing / which also sees the own scale
    good_prev = orc.previous_scale_mask
    monkeypatch.setattr(orc, "previous_scale_mask", lambda s: good_prev(s) & ~orc.block_diagonal_mask(s))
    assert fails(test_window_masks_single_scale_all_dense_and_nesting) and fails(test_window_masks_pair_counts_closed_forms)
    monkeypatch.setattr(orc, "previous_scale_mask", lambda s: orc.hmar_mask(s))
    assert fails(test_prev_window_literals_and_locality) and fails(test_window_masks_pair_counts_closed_forms)
    monkeypatch.setattr(orc, "previous_scale_mask", good_prev)

    # (2) another cubic kernel parameter; taps in reverse order
    good_w = orc._cubic_weights
    monkeypatch.setattr(orc, "_cubic_weights", lambda t: good_w(t, a=-0.5))
    assert fails(test_cubic_weights_literals_and_partition_of_unity) and fails(test_bicubic_upsample_against_the_library_routine_and_special_cases)
    monkeypatch.setattr(orc, "_cubic_weights", lambda t: good_w(t)[::-1])
    assert fails(test_cubic_weights_literals_and_partition_of_unity) and fails(test_bicubic_upsample_against_the_library_routine_and_special_cases)
    monkeypatch.setattr(orc, "_cubic_weights", good_w)

    # (3) sample positions without the half-pixel shift (corner-aligned instead)
    good_up = orc.bicubic_upsample

    def corner_aligned(x, out_side):
        x = np.asarray(x, dtype=np.float64)
        h = x.shape[-1]
        if h == out_side or h == 1:
            return good_up(x, out_side)
        big = good_up(x, out_side)
        return np.roll(big, 1, axis=-1)          # any systematic shift of the sampling grid
    monkeypatch.setattr(orc, "bicubic_upsample", corner_aligned)
    assert fails(test_bicubic_upsample_against_the_library_routine_and_special_cases) and fails(test_select_tokens_and_recon_accumulate)
    monkeypatch.setattr(orc, "bicubic_upsample", good_up)

    # (4) the selection inverted; the accumulation replaced by an overwrite
    good_sel = orc.select_tokens
    monkeypatch.setattr(orc, "select_tokens", lambda o, n, m: good_sel(n, o, m))
    assert fails(test_select_tokens_and_recon_accumulate)
    monkeypatch.setattr(orc, "select_tokens", good_sel)
    good_acc = orc.recon_accumulate
    monkeypatch.setattr(orc, "recon_accumulate", lambda x, cb, t, s: good_acc(np.zeros_like(np.asarray(x, dtype=np.float64)), cb, t, s))
    assert fails(test_select_tokens_and_recon_accumulate)


def test_area_downsample_against_the_library_routine_closed_forms_and_a_planted_mistake():
    """Pins of the oracle's area interpolation: the library's routine in fp64, block means where the sizes divide,
    a hand-computed 3 -> 2 case (bins {0, 1} and {1, 2}), identity, constants, the global mean at size 1, and a
    planted mistake (ceil taken as floor for the bin's end) that the library comparison catches."""
    rng = np.random.default_rng(35)
    for h, s in ((32, 1), (32, 13), (32, 16), (32, 32), (16, 6), (7, 3), (9, 4), (64, 24), (5, 5)):
        x = rng.standard_normal((2, 3, h, h))
        ref = torch.nn.functional.interpolate(torch.from_numpy(x), size=(s, s), mode="area").numpy()
        np.testing.assert_allclose(orc.area_downsample(x, s), ref, rtol=1e-12, atol=1e-13)
    x = rng.standard_normal((3, 12, 12))
    np.testing.assert_allclose(orc.area_downsample(x, 4), x.reshape(3, 4, 3, 4, 3).mean(axis=(2, 4)), rtol=1e-13)   # block means
    np.testing.assert_allclose(orc.area_downsample(x, 1)[:, 0, 0], x.mean(axis=(1, 2)), rtol=1e-13)
    assert np.array_equal(orc.area_downsample(x, 12), x)
    np.testing.assert_allclose(orc.area_downsample(np.full((9, 9), -1.25), 4), -1.25, rtol=1e-15)
    y = np.arange(9.0).reshape(3, 3)          # rows {0,1} / {1,2} and the like columns
    np.testing.assert_allclose(orc.area_downsample(y, 2), [[(0 + 1 + 3 + 4) / 4, (1 + 2 + 4 + 5) / 4],
                                                           [(3 + 4 + 6 + 7) / 4, (4 + 5 + 7 + 8) / 4]], rtol=1e-15)
    np.testing.assert_allclose(orc.area_downsample(y.T, 2), orc.area_downsample(y, 2).T, rtol=1e-15)

    def planted(x, s):                        # end of the bin rounded down: drops the shared row / column
        h = x.shape[-1]
        out = np.zeros(x.shape[:-2] + (s, s))
        for i in range(s):
            r0, r1 = (i * h) // s, max(((i + 1) * h) // s, (i * h) // s + 1)
            for j in range(s):
                c0, c1 = (j * h) // s, max(((j + 1) * h) // s, (j * h) // s + 1)
                out[..., i, j] = x[..., r0:r1, c0:c1].mean(axis=(-2, -1))
        return out
    z = rng.standard_normal((7, 7))
    ref = torch.nn.functional.interpolate(torch.from_numpy(z)[None, None], size=(3, 3), mode="area").numpy()[0, 0]
    assert np.abs(planted(z, 3) - ref).max() > 1e-3
    np.testing.assert_allclose(orc.area_downsample(z, 3), ref, rtol=1e-12, atol=1e-13)
