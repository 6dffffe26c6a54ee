"""Counter-based seeded generators for Q/K/V/dOut tensors.

Values are i.i.d. N(0,1) drawn from numpy's Philox generator keyed by (seed, stream), so
any (batch, head) slice can be regenerated on its own without materialising the rest of
the tensor: head `bh` of a tensor is always the `bh`-th block of the same Philox stream.
For bf16 workloads the values are rounded to bf16 once here (round-to-nearest-even) and
returned widened to float32, so every consumer sees bit-identical inputs.
"""
import numpy as np

_STREAMS = {"q": 0, "k": 1, "v": 2, "dout": 3, "k_cur": 4, "v_cur": 5}


def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result stays float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    r = (u + bias) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def _head_block(seed: int, stream: int, bh: int, rows: int, D: int) -> np.ndarray:
    # One independent Philox key per (seed, stream, head): reproducible for any subset.
    bitgen = np.random.Philox(key=[np.uint64(seed), np.uint64((stream << 32) | bh)])
    return np.random.Generator(bitgen).standard_normal((rows, D), dtype=np.float32)


def normal_tensor(seed: int, name: str, BH: int, rows: int, D: int, bf16: bool = True,
                  heads=None, gain: float = 1.0) -> np.ndarray:
    """[len(heads) or BH, rows, D] float32 N(0, gain^2) tensor for stream `name`."""
    stream = _STREAMS[name] if isinstance(name, str) else int(name)
    idx = range(BH) if heads is None else heads
    out = np.empty((len(idx), rows, D), dtype=np.float32)
    for n, bh in enumerate(idx):
        out[n] = _head_block(seed, stream, bh, rows, D)
    if gain != 1.0:
        out *= np.float32(gain)
    return bf16_round(out) if bf16 else out


def training_inputs(wl, bf16: bool = True, heads=None, with_dout: bool = True, gain: float = 1.0):
    """q, k, v (and dout) of shape [BH', L, D] for a training workload.

    `heads` selects flattened (b*H + h) indices; None means all B*H heads.
    `gain` scales q only (used to stress the running-max path of the softmax).
    """
    BH, L, D = wl.B * wl.H, wl.L, wl.D
    q = normal_tensor(wl.seed, "q", BH, L, D, bf16, heads, gain)
    k = normal_tensor(wl.seed, "k", BH, L, D, bf16, heads)
    v = normal_tensor(wl.seed, "v", BH, L, D, bf16, heads)
    if not with_dout:
        return q, k, v
    dout = normal_tensor(wl.seed, "dout", BH, L, D, bf16, heads)
    return q, k, v, dout


def scale_step_inputs(wl, scale_idx: int, sub_step: int, bf16: bool = True, heads=None):
    """Inputs of one inference sub-step at 0-based scale `scale_idx`.

    The previous scale's K/V stay fixed over the sub-steps of a scale (they are the cached
    tokens); Q and the scale's own K/V are fresh for every sub-step.
    Returns q, k_prev, v_prev, k_cur, v_cur with k_prev/v_prev None at the first scale.
    """
    BH, D = wl.B * wl.H, wl.D
    n_cur = wl.side_lens[scale_idx] ** 2
    base = wl.seed * 1000 + scale_idx * 16
    fresh = base + 1 + sub_step
    q = normal_tensor(fresh, "q", BH, n_cur, D, bf16, heads)
    k_cur = normal_tensor(fresh, "k_cur", BH, n_cur, D, bf16, heads)
    v_cur = normal_tensor(fresh, "v_cur", BH, n_cur, D, bf16, heads)
    if scale_idx == 0:
        return q, None, None, k_cur, v_cur
    n_prev = wl.side_lens[scale_idx - 1] ** 2
    k_prev = normal_tensor(base, "k", BH, n_prev, D, bf16, heads)
    v_prev = normal_tensor(base, "v", BH, n_prev, D, bf16, heads)
    return q, k_prev, v_prev, k_cur, v_cur
