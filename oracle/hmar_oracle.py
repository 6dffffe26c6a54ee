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
