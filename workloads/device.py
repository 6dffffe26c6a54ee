"""Device-side helpers for full-size workloads (torch used as a buffer allocator and RNG only).

At the benchmark sizes, generating every head on the host would take minutes, so the bulk of a
tensor is filled by torch's seeded device generator and only the heads that a test compares with
the CPU oracle are overwritten with the host generator's values (workloads.gen).
"""
import numpy as np
import torch

from . import gen


def to_device(arr, B, H, dtype, device="cuda"):
    """[BH, rows, D] float32 numpy -> [B, H, rows, D] device tensor of `dtype`."""
    t = torch.from_numpy(np.ascontiguousarray(arr)).to(device=device, dtype=dtype)
    return t.view(B, H, arr.shape[1], arr.shape[2]).contiguous()


def bulk_normal(seed, stream_id, B, H, rows, D, dtype=torch.bfloat16, device="cuda"):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) * 16 + int(stream_id))
    return torch.randn((B, H, rows, D), generator=g, device=device, dtype=torch.float32).to(dtype)


def training_tensors(wl, sample_heads, dtype=torch.bfloat16, device="cuda", with_dout=True):
    """Full [B,H,L,D] device tensors plus the host copies of `sample_heads` (flattened b*H+h).

    Returns (dev, host): dicts keyed 'q','k','v'[,'dout']; host[name] is [len(sample_heads), L, D]
    float32 holding exactly the values stored on the device for those heads.
    """
    names = ["q", "k", "v"] + (["dout"] if with_dout else [])
    bf16 = dtype == torch.bfloat16
    dev, host = {}, {}
    for sid, name in enumerate(names):
        t = bulk_normal(wl.seed, sid, wl.B, wl.H, wl.L, wl.D, dtype, device)
        h = gen.normal_tensor(wl.seed, name, wl.B * wl.H, wl.L, wl.D, bf16, list(sample_heads))
        flat = t.view(wl.B * wl.H, wl.L, wl.D)
        flat[torch.as_tensor(list(sample_heads), device=device)] = torch.from_numpy(h).to(device=device, dtype=dtype)
        dev[name], host[name] = t, h
    return dev, host
