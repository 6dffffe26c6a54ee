"""CPU oracle for HMAR's Markovian masked attention.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain statement of what the attention path computes. It is used by
the tests, by the smoke check and by the benchmark's CPU-baseline leg, and by nothing else;
the CUDA library never imports or links it, and it shares no code with the CUDA library.

Everything is float64 numpy. The explicit L x L mask is materialised per call. numpy's
matmul is the only library primitive used; there is no tiling, fusion or reordering.

What it follows:
  * the mask: Sec. 4.1 ("Markovian" next-scale prediction: scale k is conditioned on its
    immediate predecessor only), Fig. attn-mask / App. B.3 (block-diagonal, windowed
    pattern versus VAR's block-causal one), Sec. 3 (tokens inside one scale attend to each
    other bidirectionally). Reading used here: a token of scale k attends to every token
    of scales k-1 and k, and the first scale attends to itself only.
  * the arithmetic: Sec. 4.1 says the kernel extends FlashAttention, i.e. it is exact
    softmax attention; the paper prints no formula, so the textbook definition
    O = softmax(scale * Q K^T + mask) V and its analytic gradient are written out.
  * the inference step: Sec. 4.1 / Sec. 4.4 (only the previous scale is kept; every
    masked refinement sub-step is conditioned on the previous scale and on the tokens of
    the current scale): Q = current scale, K/V = previous scale followed by current scale.

Parity pins: every function here is pinned by tests/test_oracle_pins.py (closed forms,
brute force, invariants, finite differences, a library cross-check on the dense special
case). Nothing in this file is "parity unpinned".
"""
import numpy as np


def scale_layout(side_lens):
    """Token counts n_k = side_k^2, start offsets and total length of the flattened sequence.

    Sec. 3: the K token maps r_1..r_K of h_k x w_k tokens are flattened scale after scale.
    Returns (n, start, L) with start of length K+1 (start[K] == L).
    """
    sides = [int(s) for s in side_lens]
    if len(sides) == 0 or any(s <= 0 for s in sides):
        raise ValueError("side_lens must be a non-empty list of positive integers")
    n = np.array([s * s for s in sides], dtype=np.int64)
    start = np.concatenate([[0], np.cumsum(n)]).astype(np.int64)
    return n, start, int(start[-1])


def scale_of_token(side_lens):
    """scale(i) (0-based) for every flattened token index i."""
    n, _, _ = scale_layout(side_lens)
    return np.repeat(np.arange(len(n), dtype=np.int64), n)


def hmar_mask(side_lens):
    """Boolean [L, L] mask, M[i, j] = True iff scale(j) in {scale(i) - 1, scale(i)}.

    Sec. 4.1 and Fig. attn-mask (Markovian / windowed block pattern).
    """
    s = scale_of_token(side_lens)
    si = s[:, None]
    sj = s[None, :]
    return (sj == si) | (sj == si - 1)


def block_causal_mask(side_lens):
    """VAR's block-causal mask (Sec. 3): scale k attends to all scales <= k."""
    s = scale_of_token(side_lens)
    return s[None, :] <= s[:, None]


def block_diagonal_mask(side_lens):
    """Scale k attends to scale k only: the literal block-diagonal pattern of Sec. 1 / App. B.3."""
    s = scale_of_token(side_lens)
    return s[None, :] == s[:, None]


def previous_scale_mask(side_lens):
    """Scale k attends to scale k-1 only (App. B.3 read literally: "only the immediately preceding scale");
    the first scale has no predecessor and attends to itself, so that no row is empty."""
    s = scale_of_token(side_lens)
    si = s[:, None]
    sj = s[None, :]
    return (sj == si - 1) | ((si == 0) & (sj == 0))


def window_mask(side_lens, window="markov"):
    """The mask of the family named by `window`: "markov" (HMAR, scales k-1 and k), "causal" (VAR's
    block-causal mask, Sec. 3), "self" (block-diagonal) or "prev" (the preceding scale only)."""
    if window == "markov":
        return hmar_mask(side_lens)
    if window == "causal":
        return block_causal_mask(side_lens)
    if window == "self":
        return block_diagonal_mask(side_lens)
    if window == "prev":
        return previous_scale_mask(side_lens)
    raise ValueError("window must be 'markov', 'causal', 'self' or 'prev'")


def count_pairs(side_lens, window="markov"):
    """Number of unmasked (i, j) pairs per head under the mask."""
    return int(window_mask(side_lens, window).sum())


def _masked_softmax(S, M):
    """Row softmax of S restricted to M; returns (P, lse) with natural-log lse."""
    S = np.where(M, S, -np.inf)
    m = S.max(axis=-1, keepdims=True)
    E = np.exp(S - m)
    l = E.sum(axis=-1, keepdims=True)
    P = E / l
    lse = (m + np.log(l))[..., 0]
    return P, lse


def attention_probs(q, k, mask, softmax_scale):
    """P [.., Lq, Lk] and lse [.., Lq] for one masked softmax attention (float64)."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    S = softmax_scale * (q @ np.swapaxes(k, -1, -2))
    return _masked_softmax(S, mask)


def attn_fwd(q, k, v, side_lens, softmax_scale, window="markov"):
    """Training forward. q, k, v: [..., L, D]. Returns out [..., L, D], lse [..., L] (float64).

    lse_i = ln sum_j exp(softmax_scale * q_i . k_j) over the allowed j.
    """
    v = np.asarray(v, dtype=np.float64)
    M = window_mask(side_lens, window)
    if q.shape[-2] != M.shape[0]:
        raise ValueError("sequence length does not match side_lens")
    P, lse = attention_probs(q, k, M, softmax_scale)
    return P @ v, lse


def attn_bwd(q, k, v, dout, side_lens, softmax_scale, window="markov"):
    """Training backward: gradients of sum(out * dout) w.r.t. q, k, v (float64).

    dV = P^T dO;  dP = dO V^T;  delta_i = sum_j P_ij dP_ij;  dS = P o (dP - delta);
    dQ = scale * dS K;  dK = scale * dS^T Q.
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    dout = np.asarray(dout, dtype=np.float64)
    M = window_mask(side_lens, window)
    P, _ = attention_probs(q, k, M, softmax_scale)
    dV = np.swapaxes(P, -1, -2) @ dout
    dP = dout @ np.swapaxes(v, -1, -2)
    delta = (P * dP).sum(axis=-1, keepdims=True)
    dS = P * (dP - delta)
    dQ = softmax_scale * (dS @ k)
    dK = softmax_scale * (np.swapaxes(dS, -1, -2) @ q)
    return dQ, dK, dV


def scale_step(q, k_prev, v_prev, k_cur, v_cur, softmax_scale):
    """Inference step of one scale: Q [.., n_cur, D] over K/V = prev followed by cur, no mask.

    k_prev / v_prev are None at the first scale (it has no predecessor).
    Returns out [.., n_cur, D], lse [.., n_cur].
    """
    k_cur = np.asarray(k_cur, dtype=np.float64)
    v_cur = np.asarray(v_cur, dtype=np.float64)
    if k_prev is None:
        kk, vv = k_cur, v_cur
    else:
        kk = np.concatenate([np.asarray(k_prev, dtype=np.float64), k_cur], axis=-2)
        vv = np.concatenate([np.asarray(v_prev, dtype=np.float64), v_cur], axis=-2)
    M = np.ones((q.shape[-2], kk.shape[-2]), dtype=bool)
    P, lse = attention_probs(q, kk, M, softmax_scale)
    return P @ vv, lse


# ----------------------------------------------------------------------------------------------
# The sampler's steps on either side of the attention at inference (Alg. 2, "Multi-scale VQ-VAE
# Reconstruction"; Sec. 4.2, the masked refinement sub-steps).  The paper writes
#     x~_k = interpolate(lookup(V, r_k), H_K, W_K),   x~_{1:k} = x~_{1:k-1} + x~_k
# and, inside a scale, regenerates only the positions chosen by the sub-step's mask.  It does not say
# which interpolation; reading used here: bicubic convolution with the kernel parameter a = -0.75 and
# half-pixel sample positions, source indices clamped at the border (what the VAR tokenizer family that
# HMAR builds on uses to bring a coarse token map to the final resolution).

def select_tokens(tokens_old, tokens_new, mask):
    """Sec. 4.2: positions where `mask` is nonzero take the newly generated token, the others keep theirs."""
    return np.where(np.asarray(mask) != 0, np.asarray(tokens_new), np.asarray(tokens_old))


def _cubic_weights(t, a=-0.75):
    """Weights of the four taps at offsets -1, 0, 1, 2 for a sample at fractional position t in [0, 1)."""
    def near(x):      # |x| <= 1
        return ((a + 2.0) * x - (a + 3.0)) * x * x + 1.0

    def far(x):       # 1 < |x| < 2
        return ((a * x - 5.0 * a) * x + 8.0 * a) * x - 4.0 * a
    return np.array([far(t + 1.0), near(t), near(1.0 - t), far(2.0 - t)])


def bicubic_upsample(x, out_side):
    """x: [..., h, w] float64 -> [..., out_side, out_side], plain loops over the output pixels."""
    x = np.asarray(x, dtype=np.float64)
    h, w = x.shape[-2], x.shape[-1]
    out = np.zeros(x.shape[:-2] + (out_side, out_side), dtype=np.float64)
    for oy in range(out_side):
        sy = (oy + 0.5) * h / out_side - 0.5
        iy = int(np.floor(sy))
        wy = _cubic_weights(sy - iy)
        for ox in range(out_side):
            sx = (ox + 0.5) * w / out_side - 0.5
            ix = int(np.floor(sx))
            wx = _cubic_weights(sx - ix)
            acc = 0.0
            for a in range(4):
                yy = min(max(iy - 1 + a, 0), h - 1)
                for b in range(4):
                    xx = min(max(ix - 1 + b, 0), w - 1)
                    acc = acc + wy[a] * wx[b] * x[..., yy, xx]
            out[..., oy, ox] = acc
    return out


def recon_accumulate(xhat, codebook, tokens, out_side):
    """One pass of Alg. 2's loop body: xhat [B, C, out_side, out_side] + interpolate(lookup(codebook, tokens)).

    codebook: [V, C]; tokens: [B, side, side] integer ids.  Returns the new running reconstruction (float64)."""
    codebook = np.asarray(codebook, dtype=np.float64)
    tokens = np.asarray(tokens)
    looked = codebook[tokens]                                   # [B, side, side, C]
    coarse = np.moveaxis(looked, -1, 1)                         # [B, C, side, side]
    return np.asarray(xhat, dtype=np.float64) + bicubic_upsample(coarse, out_side)


def area_downsample(x, out_side):
    """The running reconstruction brought down to a scale's resolution (Sec. 4.1: the interpolation of Alg. 1's
    loop maps x~_{1:k-1} to an H_k x W_k image, which the scale is conditioned on).  The paper does not name the
    interpolation; reading used here, the counterpart of the bicubic enlargement above in the VAR tokenizer family:
    area interpolation, i.e. output pixel (i, j) is the plain mean of the input pixels whose rows lie in
    [floor(i * h / out), ceil((i + 1) * h / out)) and whose columns lie in the like range.

    x: [..., h, w] float64 -> [..., out_side, out_side]; out_side <= h, w."""
    x = np.asarray(x, dtype=np.float64)
    h, w = x.shape[-2], x.shape[-1]
    out = np.zeros(x.shape[:-2] + (out_side, out_side), dtype=np.float64)
    for i in range(out_side):
        r0, r1 = (i * h) // out_side, -((-(i + 1) * h) // out_side)
        for j in range(out_side):
            c0, c1 = (j * w) // out_side, -((-(j + 1) * w) // out_side)
            acc = 0.0
            for r in range(r0, r1):
                for c in range(c0, c1):
                    acc = acc + x[..., r, c]
            out[..., i, j] = acc / ((r1 - r0) * (c1 - c0))
    return out
