#!/usr/bin/env python
"""Benchmark of the HMAR Markovian block-sparse attention path on B200.

A step is one pass of the whole hot path on the 512x512 HMAR-d24 training shape (B=16, H=24,
L=2240, D=64): forward, then backward, through the C ABI on bf16 device tensors.  The metric is
useful TFLOP/s: only the unmasked (query, key) pairs count, 4*pairs*D for the forward and
10*pairs*D for the backward, per head.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With N > 1 (launched by torch.distributed.run) every rank runs the same shape on its own tensors
(the path has no exchange step: independent replicas, weak scaling); the time is the maximum over
ranks.  `--impl reference` times the CPU oracle, as it stands, on a bounded sample of heads.
"""
import argparse
import json
import os
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

WORKLOAD = "512_d24_train"
METRIC = "useful_tflops_fwd_bwd_512x512_d24"
UNIT = "TFLOP/s"

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu
# capture summarised under profiles/ (None until a capture exists for the current kernel).
# The captures are of the batch-4 case (traffic grows in proportion to the heads), scaled by 4 to the full batch.
NCU_TRAFFIC_BYTES = {"hmar_bwd": 4 * (230900224 + 111457792), "hmar_fwd": 4 * (82932224 + 9546496)}


def pairs_per_head(side_lens):
    n = [s * s for s in side_lens]
    return sum(n[i] * (n[i] + (n[i - 1] if i else 0)) for i in range(len(n)))


def useful_flops(wl):
    p = pairs_per_head(wl.side_lens) * wl.B * wl.H * wl.D
    return 4 * p, 10 * p


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"bf16_tflops": d["bf16_tflops"], "bf16_tflops_sustained": d.get("bf16_tflops_sustained"),
                "hbm_gbs": d["hbm_gbs"], "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, sm_max, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                sm_max.append(float(f[2]))
            except ValueError:
                continue
            for nm, val in zip(names, f[5:9]):
                if val.lower() == "active":
                    reasons.add(nm)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(sm_max)), "reasons": sorted(reasons),
                "samples": len(sm)}


def time_oracle(wl, n_heads, steps, warmup):
    """Times the CPU oracle (forward + backward) on `n_heads` heads of the workload per step."""
    from threadpoolctl import threadpool_info

    from oracle import hmar_oracle as orc
    from workloads import training_inputs
    heads = sorted({0, wl.B * wl.H - 1} | set(range(1, n_heads - 1)))[:n_heads]
    q, k, v, do = training_inputs(wl, bf16=True, heads=heads)
    times = []
    for it in range(warmup + steps):
        t0 = time.perf_counter()
        orc.attn_fwd(q, k, v, wl.side_lens, wl.softmax_scale)
        orc.attn_bwd(q, k, v, do, wl.side_lens, wl.softmax_scale)
        dt = time.perf_counter() - t0
        if it >= warmup:
            times.append(dt)
    flops = 14 * pairs_per_head(wl.side_lens) * wl.D * len(heads)
    cores = max([p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"] or [1])
    sec = float(np.mean(times))
    return {"value": flops / sec / 1e12, "unit": UNIT, "cores": int(cores), "kind": "oracle",
            "sample": f"{len(heads)} of {wl.B * wl.H} heads (first, last and the heads between), fwd+bwd, "
                      f"{sec * 1e3:.0f} ms per sample; numpy fp64 with an explicit {wl.L}x{wl.L} mask"}, sec


def time_dense_masked(wl, q, k, v, do, reps=3):
    """Dense masked attention of the same shape on the same GPU (torch SDPA with the explicit boolean HMAR
    mask, forward + backward): the comparison the paper's App. B.4 makes.  Library kernels, timed outside
    the benchmark's own timed region; reported as context only."""
    import torch
    import torch.nn.functional as F
    n = [s * s for s in wl.side_lens]
    scale_of = torch.repeat_interleave(torch.arange(len(n)), torch.tensor(n)).to(q.device)
    mask = (scale_of[None, :] == scale_of[:, None]) | (scale_of[None, :] == scale_of[:, None] - 1)
    qq, kk, vv = (t.detach().clone().requires_grad_(True) for t in (q, k, v))

    def step():
        out = F.scaled_dot_product_attention(qq, kk, vv, attn_mask=mask, scale=wl.softmax_scale)
        out.backward(do)
        qq.grad = kk.grad = vv.grad = None

    step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        step()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


L2_BYTES = 126 * 1024 * 1024


def _rotating_sets(bytes_per_set, cap=12):
    """How many copies of a leg's tensors to cycle through so that consecutive iterations do not find their
    inputs in L2 (the sets together hold more than twice the L2, up to `cap` sets)."""
    return int(max(2, min(cap, -(-2 * L2_BYTES // max(1, bytes_per_set)))))


def time_scale_steps(hmar, wl_inf, dev, peaks, reps=6):
    """Every scale of the 512x512 d24 inference sweep (B=64, H=24; one call is one masked sub-step: fresh Q and
    own-scale K/V, the previous scale's K/V kept).  Per scale: ms per call (CUDA events around `reps` calls that
    cycle through several input sets, so the inputs come from HBM), achieved GB/s on the algorithmic bytes
    (Q, O, K/V of both scales once) and useful TFLOP/s, each as a fraction of its measured peak."""
    import torch
    from workloads.device import bulk_normal
    B, H, D = wl_inf.B, wl_inf.H, wl_inf.D
    rows = []
    for s, side in enumerate(wl_inf.side_lens):
        side_prev = wl_inf.side_lens[s - 1] if s else 0
        nc, npv = side * side, side_prev * side_prev
        byt = B * H * (2 * nc + 2 * (nc + npv)) * D * 2
        flops = 4 * B * H * nc * (nc + npv) * D
        n_sets = _rotating_sets(byt)
        sets = []
        for k in range(n_sets):
            sets.append([bulk_normal(wl_inf.seed + s + 100 * k, i, B, H, (side_prev if i in (1, 2) else side) ** 2, D,
                                     torch.bfloat16, dev) if (s or i not in (1, 2)) else None for i in range(5)])
        o = torch.empty_like(sets[0][0])
        for k in range(min(3, n_sets)):
            hmar.hmar_attn_scale_step(*sets[k], side_prev, side, wl_inf.softmax_scale, out=o, want_lse=False)
        n_calls = reps * n_sets if byt < (8 << 20) else max(reps, n_sets)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for it in range(n_calls):
            hmar.hmar_attn_scale_step(*sets[it % n_sets], side_prev, side, wl_inf.softmax_scale, out=o, want_lse=False)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / n_calls
        gbs, tf = byt / ms / 1e6, flops / ms / 1e9
        rows.append({"scale": s + 1, "side": side, "ms": round(ms, 4), "gbs": round(gbs, 1),
                     "frac_hbm": round(gbs / peaks["hbm_gbs"], 4), "tflops": round(tf, 1),
                     "frac_tensor": round(tf / peaks["bf16_tflops"], 4), "input_sets": n_sets,
                     "bound": "tensor" if flops / byt > 250 else ("hbm" if byt > (16 << 20) else "launch latency")})
        del sets
        torch.cuda.empty_cache()
    return rows


def time_small_config(hmar, wl_x, dev, peaks, reps=4):
    """A 256x256 (L = 680) config at its full batch: forward, and backward if the config has one.  The tensors of
    these configs fit in L2, so the calls cycle through several input sets.  Reports ms, useful TFLOP/s, and GB/s
    on the algorithmic bytes (fwd: Q, K, V, O + LSE; bwd: Q, K, V, O, dO, LSE in, dQ, dK, dV out) against the
    measured HBM copy bandwidth: these shapes are HBM-bound (arithmetic intensity 130-150 FLOP/B)."""
    import torch
    from workloads.device import bulk_normal
    B, H, L, D = wl_x.B, wl_x.H, wl_x.L, wl_x.D
    backward = "bwd" in wl_x.passes
    elem = B * H * L * D * 2
    fwd_bytes = 4 * elem + 4 * B * H * L
    bwd_bytes = 8 * elem + 4 * B * H * L
    n_sets = _rotating_sets(fwd_bytes + (bwd_bytes if backward else 0), cap=8)
    sets = [[bulk_normal(wl_x.seed + 100 * k, i, B, H, L, D, torch.bfloat16, dev) for i in range(4 if backward else 3)]
            for k in range(n_sets)]
    out = torch.empty_like(sets[0][0])
    lse = torch.empty((B, H, L), dtype=torch.float32, device=dev)
    dq, dk, dv = (torch.empty_like(out) for _ in range(3)) if backward else (None, None, None)
    ws = torch.empty(hmar.hmar_attn_bwd_workspace_bytes(B, H, D, wl_x.side_lens), dtype=torch.uint8, device=dev) if backward else None

    def one(t):
        hmar.hmar_attn_fwd(t[0], t[1], t[2], wl_x.side_lens, wl_x.softmax_scale, out=out, lse=lse)
        if backward:
            hmar.hmar_attn_bwd(t[0], t[1], t[2], out, lse, t[3], wl_x.side_lens, wl_x.softmax_scale, dq=dq, dk=dk, dv=dv,
                               workspace=ws)

    for t in sets[:2]:
        one(t)
    torch.cuda.synchronize()
    n_calls = reps * n_sets
    hmar.hmar_profile_begin()
    for it in range(n_calls):
        one(sets[it % n_sets])
    kern = hmar.hmar_profile_end()
    f_ms = kern["hmar_fwd_tc_kernel"][1] / n_calls
    f_fl, b_fl = useful_flops(wl_x)
    res = {"B": B, "H": H, "L": L, "input_sets": n_sets,
           "fwd": {"ms": round(f_ms, 4), "tflops": round(f_fl / f_ms / 1e9, 1), "gbs": round(fwd_bytes / f_ms / 1e6, 1),
                   "frac_hbm": round(fwd_bytes / f_ms / 1e6 / peaks["hbm_gbs"], 4), "algorithmic_bytes": fwd_bytes}}
    if backward:
        b_ms = sum(v[1] for k, v in kern.items() if "bwd" in k) / n_calls
        res["bwd"] = {"ms": round(b_ms, 4), "tflops": round(b_fl / b_ms / 1e9, 1), "gbs": round(bwd_bytes / b_ms / 1e6, 1),
                      "frac_hbm": round(bwd_bytes / b_ms / 1e6 / peaks["hbm_gbs"], 4), "algorithmic_bytes": bwd_bytes,
                      "kernels_ms": {k: round(v[1] / n_calls, 4) for k, v in kern.items() if "bwd" in k}}
    res["timing"] = "sum of the library's per-kernel CUDA events over the calls"
    return res


def time_recon(hmar, dev, peaks, reps=20):
    """The sampler's neighbour step (Alg. 2 lines 7-8 fused with the sub-step's token selection) on a synthetic
    codebook (V = 4096, C = 32), latent 32 x 32: at the sampler's batch (64) and at a batch whose reconstruction
    exceeds L2 (2048: 268 MB), for the last scale (32 -> 32) and a middle one (13 -> 32).  GB/s on the algorithmic
    bytes (the reconstruction read and written once) against the measured HBM bandwidth.  Then the other neighbour,
    the area interpolation of the reconstruction down to those two sizes (Sec. 4.1; algorithmic bytes: the
    reconstruction read once plus the small image written)."""
    import torch
    rows = []
    g = torch.Generator(device=dev)
    g.manual_seed(4421)
    V, C, S = 4096, 32, 32
    codebook = torch.randn((V, C), generator=g, device=dev)
    for B in (64, 2048):
        xhat = torch.zeros((B, C, S, S), device=dev)
        for side in (13, 32):
            old = torch.randint(0, V, (B, side, side), generator=g, device=dev, dtype=torch.int32)
            new = torch.randint(0, V, (B, side, side), generator=g, device=dev, dtype=torch.int32)
            mask = torch.randint(0, 2, (B, side, side), generator=g, device=dev, dtype=torch.uint8)
            sel = torch.empty_like(old)
            for _ in range(3):
                hmar.hmar_recon_accumulate(xhat, codebook, new, old, mask, sel)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                hmar.hmar_recon_accumulate(xhat, codebook, new, old, mask, sel)
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / reps
            byt = 2 * xhat.numel() * 4
            rows.append({"op": "accumulate", "B": B, "side": side, "ms": round(ms, 4), "gbs": round(byt / ms / 1e6, 1),
                         "frac_hbm": round(byt / ms / 1e6 / peaks["hbm_gbs"], 4), "algorithmic_bytes": byt})
        for side in (13, 32):                              # the other neighbour: area interpolation down to a scale
            out = torch.empty((B, C, side, side), device=dev)
            for _ in range(3):
                hmar.hmar_recon_downsample(xhat, side, out=out)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                hmar.hmar_recon_downsample(xhat, side, out=out)
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / reps
            byt = (xhat.numel() + out.numel()) * 4
            rows.append({"op": "downsample", "B": B, "side": side, "ms": round(ms, 4), "gbs": round(byt / ms / 1e6, 1),
                         "frac_hbm": round(byt / ms / 1e6 / peaks["hbm_gbs"], 4), "algorithmic_bytes": byt})
        del xhat
        torch.cuda.empty_cache()
    return rows


def oracle_errors(hmar, dev):
    """Max / mean abs error against the CPU oracle of one head per config, the head placed in an otherwise
    device-generated full-size problem (outside every timed region)."""
    import torch
    from oracle import hmar_oracle as orc
    from workloads import CONFIGS, scale_step_inputs
    from workloads.device import bulk_normal, training_tensors
    res = {}

    def err(g, r):
        d = np.abs(g.detach().double().cpu().numpy().reshape(r.shape) - r)
        return [float(f"{d.max():.3e}"), float(f"{d.mean():.3e}")]

    for name in ("256_d16_fwd", "256_d30_train", "512_d24_train"):
        wl_x = CONFIGS[name]
        head = (wl_x.B * wl_x.H) // 3
        backward = "bwd" in wl_x.passes
        d, h = training_tensors(wl_x, [head], with_dout=backward)
        out, lse = hmar.hmar_attn_fwd(d["q"], d["k"], d["v"], wl_x.side_lens, wl_x.softmax_scale)
        ro, rl = orc.attn_fwd(h["q"], h["k"], h["v"], wl_x.side_lens, wl_x.softmax_scale)
        e = {"head": head, "out": err(out.view(-1, wl_x.L, wl_x.D)[head], ro[0]), "lse": err(lse.view(-1, wl_x.L)[head], rl[0])}
        if backward:
            g = hmar.hmar_attn_bwd(d["q"], d["k"], d["v"], out, lse, d["dout"], wl_x.side_lens, wl_x.softmax_scale)
            r = orc.attn_bwd(h["q"], h["k"], h["v"], h["dout"], wl_x.side_lens, wl_x.softmax_scale)
            for nm, gg, rr in zip(("dq", "dk", "dv"), g, r):
                e[nm] = err(gg.view(-1, wl_x.L, wl_x.D)[head], rr[0])
        res[name] = e
        del d
        torch.cuda.empty_cache()
    wl_i = CONFIGS["512_d24_infer"]
    BH, head = wl_i.B * wl_i.H, (wl_i.B * wl_i.H) // 3
    worst = [0.0, 0.0]
    for s_, side in enumerate(wl_i.side_lens):
        sp = wl_i.side_lens[s_ - 1] if s_ else 0
        host = scale_step_inputs(wl_i, s_, 1, bf16=True, heads=[head])
        devt = []
        for sid, hh in enumerate(host):
            if hh is None:
                devt.append(None)
                continue
            t = bulk_normal(wl_i.seed + s_, sid, wl_i.B, wl_i.H, hh.shape[1], wl_i.D)
            t.view(BH, hh.shape[1], wl_i.D)[head] = torch.from_numpy(hh[0]).to(device=dev, dtype=torch.bfloat16)
            devt.append(t)
        o, _ = hmar.hmar_attn_scale_step(*devt, sp, side, wl_i.softmax_scale)
        ro, _ = orc.scale_step(*host, wl_i.softmax_scale)
        e = err(o.view(BH, -1, wl_i.D)[head], ro[0])
        worst = [max(worst[0], e[0]), max(worst[1], e[1])]
    res["512_d24_infer"] = {"head": head, "out_worst_scale": worst}
    res["what"] = "[max abs, mean abs] against the fp64 oracle, one head per config"
    return res


def time_training_shape(hmar, wl_x, dev, window, reps=3):
    """ms of forward and of backward on another training shape / mask of the family (context legs)."""
    import torch
    from workloads.device import bulk_normal
    B, H, L, D = wl_x.B, wl_x.H, wl_x.L, wl_x.D
    q, k, v, do = (bulk_normal(wl_x.seed, i, B, H, L, D, torch.bfloat16, dev) for i in range(4))
    out = torch.empty_like(q)
    lse = torch.empty((B, H, L), dtype=torch.float32, device=dev)
    dq, dk, dv = (torch.empty_like(q) for _ in range(3))
    ws = torch.empty(hmar.hmar_attn_bwd_workspace_bytes(B, H, D, wl_x.side_lens), dtype=torch.uint8, device=dev)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    f_ms = b_ms = 0.0
    for it in range(reps + 1):
        ev[0].record()
        hmar.hmar_attn_fwd(q, k, v, wl_x.side_lens, wl_x.softmax_scale, out=out, lse=lse, window=window)
        ev[1].record()
        hmar.hmar_attn_bwd(q, k, v, out, lse, do, wl_x.side_lens, wl_x.softmax_scale, dq=dq, dk=dk, dv=dv,
                           workspace=ws, window=window)
        ev[2].record()
        torch.cuda.synchronize()
        if it:
            f_ms += ev[0].elapsed_time(ev[1]) / reps
            b_ms += ev[1].elapsed_time(ev[2]) / reps
    return f_ms, b_ms


def time_packed_step(hmar, wl_x, dev, reps=5):
    """ms of forward and backward on the packed projection layouts (qkv, dqkv [B,L,3,H,D]; out, dout [B,L,H,D]), and
    of the transposing copies that the contiguous entry points would need around them for the same data: three in
    and one out for the forward, one more in (dout) and three out (dq, dk, dv) for the backward (context leg)."""
    import torch
    from workloads.device import bulk_normal
    B, H, L, D = wl_x.B, wl_x.H, wl_x.L, wl_x.D
    qkv = bulk_normal(wl_x.seed, 9, B, L, 3 * H, D, torch.bfloat16, dev).view(B, L, 3, H, D)
    dout = bulk_normal(wl_x.seed, 10, B, L, H, D, torch.bfloat16, dev)
    out = torch.empty((B, L, H, D), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((B, H, L), dtype=torch.float32, device=dev)
    dqkv = torch.empty_like(qkv)
    ws = torch.empty(hmar.hmar_attn_bwd_workspace_bytes(B, H, D, wl_x.side_lens), dtype=torch.uint8, device=dev)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    f_ms = b_ms = c_ms = 0.0
    for it in range(reps + 1):
        ev[0].record()
        hmar.hmar_attn_fwd_packed(qkv, wl_x.side_lens, wl_x.softmax_scale, out=out, lse=lse)
        ev[1].record()
        hmar.hmar_attn_bwd_packed(qkv, out, lse, dout, wl_x.side_lens, wl_x.softmax_scale, dqkv=dqkv, workspace=ws)
        ev[2].record()
        q, k, v = (qkv[:, :, i].permute(0, 2, 1, 3).contiguous() for i in range(3))
        do_c = dout.permute(0, 2, 1, 3).contiguous()
        q.permute(0, 2, 1, 3).contiguous()                  # out back to [B,L,H,D]
        for i in range(3):
            dqkv[:, :, i].copy_(q.permute(0, 2, 1, 3))      # dq, dk, dv into the packed gradient
        ev[3].record()
        torch.cuda.synchronize()
        del q, k, v, do_c
        if it:
            f_ms += ev[0].elapsed_time(ev[1]) / reps
            b_ms += ev[1].elapsed_time(ev[2]) / reps
            c_ms += ev[2].elapsed_time(ev[3]) / reps
    return f_ms, b_ms, c_ms


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_heads = 4
    base, sec = time_oracle(wl, n_heads, args.steps, min(args.warmup, 1))
    line = {
        "impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": min(args.warmup, 1), "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "B": wl.B, "H": wl.H, "L": wl.L, "D": wl.D,
                   "side_lens": list(wl.side_lens), "note": "CPU oracle; each step is the bounded sample below"},
        "cpu_baseline": base,
        "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def run_ours(args, wl):
    import torch
    import torch.distributed as dist

    import paper_2506_04421_b200 as hmar
    from workloads.device import bulk_normal

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the HMAR library has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    B, H, L, D = wl.B, wl.H, wl.L, wl.D
    sides, scale = wl.side_lens, wl.softmax_scale
    seed = wl.seed + 1000 * rank
    q, k, v, do = (bulk_normal(seed, i, B, H, L, D, torch.bfloat16, dev) for i in range(4))
    out = torch.empty_like(q)
    lse = torch.empty((B, H, L), dtype=torch.float32, device=dev)
    dq, dk, dv = (torch.empty_like(q) for _ in range(3))
    ws = torch.empty(hmar.hmar_attn_bwd_workspace_bytes(B, H, D, sides), dtype=torch.uint8, device=dev)

    def step():
        hmar.hmar_attn_fwd(q, k, v, sides, scale, out=out, lse=lse)
        hmar.hmar_attn_bwd(q, k, v, out, lse, do, sides, scale, dq=dq, dk=dk, dv=dv, workspace=ws)

    for _ in range(args.warmup):
        step()
    barrier()

    # ---- device-resident timing: K steps between two events, plus per-call events for the roofline
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches0 = hmar.hmar_launch_count()
    barrier()
    hmar.hmar_profile_begin()          # per-kernel CUDA events on the launch stream, inside the timed region
    t_begin = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    t_begin.record()
    for i in range(args.steps):
        ev[i][0].record()
        hmar.hmar_attn_fwd(q, k, v, sides, scale, out=out, lse=lse)
        ev[i][1].record()
        hmar.hmar_attn_bwd(q, k, v, out, lse, do, sides, scale, dq=dq, dk=dk, dv=dv, workspace=ws)
        ev[i][2].record()
    t_end.record()
    barrier()
    kernels = hmar.hmar_profile_end()
    launches = hmar.hmar_launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    total_ms = t_begin.elapsed_time(t_end)
    fwd_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in ev]))
    bwd_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in ev]))
    status, detail = hmar.hmar_device_status()
    if status != 0:
        raise RuntimeError(f"device status {status} detail {detail:#x}")

    # ---- context legs, outside the timed region (rank 0 only): dense masked comparison, inference sweep
    extras = {}
    if rank == 0 and not args.no_extras:
        try:
            dense_ms = time_dense_masked(wl, q, k, v, do)
            extras["dense_masked_sdpa"] = {"ms_fwd_bwd": dense_ms, "speedup_over_it": dense_ms / (total_ms / args.steps),
                                           "what": "torch SDPA with the explicit boolean mask, same shape, same GPU"}
        except Exception as e:     # the comparison is context; its failure must not lose the benchmark line
            extras["dense_masked_sdpa"] = {"error": str(e)[:200]}
        torch.cuda.empty_cache()
        if args.batch == 0:
            from workloads import CONFIGS
            peaks = measured_peaks()
            rows = time_scale_steps(hmar, CONFIGS["512_d24_infer"], dev, peaks)
            ms = [r["ms"] for r in rows]
            extras["scale_step_ms"] = {"workload": "512_d24_infer, B=64 H=24, one sub-step per call", "per_scale": ms,
                                       "sweep_4_sub_steps": round(4 * sum(ms), 4), "roofline_per_scale": rows,
                                       "peaks": {"hbm_gbs": peaks["hbm_gbs"], "bf16_tflops": peaks["bf16_tflops"], "source": peaks["source"]}}
            torch.cuda.empty_cache()
            # the two 256 x 256 configs (L = 680): HBM-bound shapes, achieved GB/s against the measured copy bandwidth
            for nm in ("256_d16_fwd", "256_d30_train"):
                extras[nm] = time_small_config(hmar, CONFIGS[nm], dev, peaks)
                torch.cuda.empty_cache()
            extras["recon_accumulate"] = {"workload": "synthetic codebook V=4096 C=32, latent 32x32", "rows": time_recon(hmar, dev, peaks)}
            try:
                extras["oracle_errors"] = oracle_errors(hmar, dev)
            except Exception as e:     # context; its failure must not lose the benchmark line
                extras["oracle_errors"] = {"error": str(e)[:200]}
            torch.cuda.empty_cache()
            # VAR's block-causal mask on the same shape and kernels: the workload the paper's speedups are against
            cf, cb = time_training_shape(hmar, wl, dev, hmar.HMAR_WINDOW_CAUSAL)
            extras["block_causal_same_kernels"] = {"fwd_ms": round(cf, 4), "bwd_ms": round(cb, 4),
                                                   "markov_speedup_fwd": round(cf / fwd_ms, 3),
                                                   "markov_speedup_bwd": round(cb / bwd_ms, 3)}
            torch.cuda.empty_cache()
            # forward on the packed QKV projection output, and the transposing copies it makes unnecessary
            pf, pb, cp = time_packed_step(hmar, wl, dev)
            extras["packed_qkv_step"] = {"fwd_ms": round(pf, 4), "bwd_ms": round(pb, 4), "contiguous_fwd_ms": round(fwd_ms, 4),
                                         "contiguous_bwd_ms": round(bwd_ms, 4), "transposes_avoided_ms": round(cp, 4),
                                         "layout": "qkv, dqkv [B,L,3,H,D]; out, dout [B,L,H,D]"}
            torch.cuda.empty_cache()
            # 1024 x 1024 (synthetic 14-scale schedule ending at 64 x 64, L = 9451), Markov mask
            wl_big = CONFIGS["1024_d24_train"]
            bf, bb = time_training_shape(hmar, wl_big, dev, hmar.HMAR_WINDOW_MARKOV, reps=2)
            fl_f, fl_b = useful_flops(wl_big)
            extras["1024_d24_train"] = {"L": wl_big.L, "fwd_ms": round(bf, 4), "bwd_ms": round(bb, 4),
                                        "useful_tflops": round((fl_f + fl_b) / ((bf + bb) * 1e-3) / 1e12, 1),
                                        "schedule": "synthetic: " + str(list(wl_big.side_lens))}
            torch.cuda.empty_cache()
    args.extras = extras

    # ---- end to end: pinned host tensors in, results back to the host, inside the timed region
    if args.no_e2e:
        return _finish(args, wl, world, rank, dev, total_ms, float("nan"), fwd_ms, bwd_ms, launches, clocks, kernels)
    hq, hk, hv, hdo = (t.cpu().pin_memory() for t in (q, k, v, do))
    h_out, h_dq, h_dk, h_dv = (torch.empty_like(hq).pin_memory() for _ in range(4))
    h_lse = torch.empty((B, H, L), dtype=torch.float32).pin_memory()

    # The batch is cut into chunks; chunk c is copied in on one stream, computed on a second and copied out on a
    # third, so the host-to-device copies, the kernels and the device-to-host copies of different chunks overlap
    # (PCIe carries both directions at once).  Every call goes through the C ABI on the chunk's own slices.
    n_chunks = 8 if B % 8 == 0 else (4 if B % 4 == 0 else 1)     # measured at B = 16: 11.8-12.1 ms with 4, 10.7-11.2 with 8
    cb = B // n_chunks
    s_in, s_run, s_out = (torch.cuda.Stream(device=dev) for _ in range(3))
    ws_c = [torch.empty(hmar.hmar_attn_bwd_workspace_bytes(cb, H, D, sides), dtype=torch.uint8, device=dev) for _ in range(2)]
    ev_in = [torch.cuda.Event() for _ in range(n_chunks)]
    ev_run = [torch.cuda.Event() for _ in range(n_chunks)]
    ev_free = [torch.cuda.Event() for _ in range(n_chunks)]     # the chunk's results have left the device

    def e2e_step():
        for c in range(n_chunks):
            sl = slice(c * cb, (c + 1) * cb)
            with torch.cuda.stream(s_in):
                for d_t, h_t in ((q, hq), (k, hk), (v, hv), (do, hdo)):
                    d_t[sl].copy_(h_t[sl], non_blocking=True)
                ev_in[c].record(s_in)
            with torch.cuda.stream(s_run):
                s_run.wait_event(ev_in[c])
                if c >= 2:
                    s_run.wait_event(ev_free[c - 2])           # the workspace of chunk c - 2 is reused
                hmar.hmar_attn_fwd(q[sl], k[sl], v[sl], sides, scale, out=out[sl], lse=lse[sl], stream=s_run)
                hmar.hmar_attn_bwd(q[sl], k[sl], v[sl], out[sl], lse[sl], do[sl], sides, scale, dq=dq[sl], dk=dk[sl], dv=dv[sl],
                                   workspace=ws_c[c % 2], stream=s_run)
                ev_run[c].record(s_run)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_run[c])
                for h_t, d_t in ((h_out, out), (h_lse, lse), (h_dq, dq), (h_dk, dk), (h_dv, dv)):
                    h_t[sl].copy_(d_t[sl], non_blocking=True)
                ev_free[c].record(s_out)
        cur = torch.cuda.current_stream()
        cur.wait_stream(s_out)
        cur.wait_stream(s_run)
        cur.wait_stream(s_in)

    e2e_steps = max(2, min(args.steps, 5))
    e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for st_ in (s_in, s_run, s_out):
        st_.wait_stream(torch.cuda.current_stream())
    e0.record()
    for _ in range(e2e_steps):
        for st_ in (s_in, s_run, s_out):
            st_.wait_stream(torch.cuda.current_stream())      # a step starts after the previous one has ended
        e2e_step()
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps
    args.e2e_note = f"{n_chunks} batch chunks on three streams (copy in, compute, copy out), pinned host buffers"
    return _finish(args, wl, world, rank, dev, total_ms, e2e_ms, fwd_ms, bwd_ms, launches, clocks, kernels)


def _finish(args, wl, world, rank, dev, total_ms, e2e_ms, fwd_ms, bwd_ms, launches, clocks, kernels):
    import torch
    import torch.distributed as dist
    B, H, L, D = wl.B, wl.H, wl.L, wl.D
    sides, scale = wl.side_lens, wl.softmax_scale
    times = torch.tensor([total_ms, e2e_ms, fwd_ms, bwd_ms], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(times, op=dist.ReduceOp.MAX)
    total_ms, e2e_ms, fwd_ms, bwd_ms = times.tolist()
    ms_per_step = total_ms / args.steps
    f_fwd, f_bwd = useful_flops(wl)
    value = world * (f_fwd + f_bwd) / (ms_per_step * 1e-3) / 1e12
    e2e_value = world * (f_fwd + f_bwd) / (e2e_ms * 1e-3) / 1e12

    if rank == 0:
        peaks = measured_peaks()
        bwd_tf = f_bwd / (bwd_ms * 1e-3) / 1e12
        fwd_tf = f_fwd / (fwd_ms * 1e-3) / 1e12
        # the dominant kernel: average launch duration from the library's own events in the timed region
        per_kernel = {name: {"launches": n, "avg_ms": ms / n, "share": ms / (ms_per_step * args.steps)}
                      for name, (n, ms) in kernels.items()}
        dom = "hmar_bwd_tc_kernel"
        dom_ms = per_kernel[dom]["avg_ms"]
        dom_tf = f_bwd / (dom_ms * 1e-3) / 1e12
        cpu_base = None if args.no_cpu else time_oracle(wl, min(24, B * H), 2, 0)[0]
        elem = 2 * B * H * L * D
        import paper_2506_04421_b200 as hmar
        ws_bytes = hmar.hmar_attn_bwd_workspace_bytes(B, H, D, sides)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD + (f" (batch reduced to {B})" if args.batch > 0 else ""),
                       "B": B, "H": H, "L": L, "D": D, "side_lens": list(sides), "softmax_scale": scale, "passes": "fwd+bwd", "parallelism": f"replicas x{world}",
                       "l2": f"tensors larger than L2 (8 x {elem / 1e6:.0f} MB + {ws_bytes / 1e6:.0f} MB workspace per step), no flush"},
            "fraction_of_peak": {"burst": value / world / peaks["bf16_tflops"],
                                 "sustained": value / world / (peaks["bf16_tflops_sustained"] or float("nan")),
                                 "nominal_2250": value / world / 2250.0, "peaks": peaks["source"]},
            "phases": {"fwd_ms": fwd_ms, "bwd_ms": bwd_ms, "fwd_tflops": fwd_tf, "bwd_tflops": bwd_tf},
            "roofline": {"bound": "tensor", "kernel": dom, "achieved": dom_tf, "peak": peaks["bf16_tflops"],
                         "unit": "TFLOP/s", "frac": dom_tf / peaks["bf16_tflops"],
                         "peak_source": peaks["source"] + " burst", "avg_launch_ms": dom_ms,
                         "algorithmic_flops_per_launch": f_bwd,
                         "traffic": NCU_TRAFFIC_BYTES["hmar_bwd"] * B // 16},
            "kernels": per_kernel,
            "cpu_baseline": cpu_base,
            "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": 4 * elem, "d2h_bytes_per_step": 4 * elem + 4 * B * H * L,
                    "how": getattr(args, "e2e_note", "")},
            "gpu_launches": int(launches),
            "clocks": clocks,
        }
        line.update(getattr(args, "extras", {}))
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_case(args):
    """A named side case run a few times (for profiling one kernel on a workload that is not the headline's):
    `256_d30_train` = forward + backward of the L = 680 training config at its full batch; `infer_scale7` = the
    inference step of scale 7 (169 queries, 250 keys) at B = 64, H = 24; `recon_b2048` = the sampler's neighbour step
    on a 32 x 32 x 32 reconstruction at B = 2048 (268 MB), a 13 x 13 map then the 32 x 32 one per repetition, each
    followed by the area interpolation down to 13 x 13 and to 32 x 32.
    Prints a small JSON line."""
    import torch

    import paper_2506_04421_b200 as hmar
    from workloads import CONFIGS
    from workloads.device import bulk_normal
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    reps = max(1, args.steps)
    hmar.hmar_profile_begin()
    if args.case == "256_d30_train":
        wl_x = CONFIGS["256_d30_train"]
        q, k, v, do = (bulk_normal(wl_x.seed, i, wl_x.B, wl_x.H, wl_x.L, wl_x.D, torch.bfloat16, dev) for i in range(4))
        for _ in range(args.warmup + reps):
            out, lse = hmar.hmar_attn_fwd(q, k, v, wl_x.side_lens, wl_x.softmax_scale)
            hmar.hmar_attn_bwd(q, k, v, out, lse, do, wl_x.side_lens, wl_x.softmax_scale)
    elif args.case == "recon_b2048":
        g = torch.Generator(device=dev)
        g.manual_seed(4421)
        V, C, S, B = 4096, 32, 32, 2048
        codebook = torch.randn((V, C), generator=g, device=dev)
        xhat = torch.zeros((B, C, S, S), device=dev)
        maps = {side: [torch.randint(0, V, (B, side, side), generator=g, device=dev, dtype=torch.int32) for _ in range(2)] +
                      [torch.randint(0, 2, (B, side, side), generator=g, device=dev, dtype=torch.uint8),
                       torch.empty((B, side, side), device=dev, dtype=torch.int32)] for side in (13, 32)}
        for _ in range(args.warmup + reps):
            for side in (13, 32):
                new, old, mask, sel = maps[side]
                hmar.hmar_recon_accumulate(xhat, codebook, new, old, mask, sel)
            for side in (13, 32):
                hmar.hmar_recon_downsample(xhat, side)
    else:
        wl_x = CONFIGS["512_d24_infer"]
        s_ = 6
        side, sp = wl_x.side_lens[s_], wl_x.side_lens[s_ - 1]
        t = [bulk_normal(wl_x.seed + s_, i, wl_x.B, wl_x.H, (sp if i in (1, 2) else side) ** 2, wl_x.D, torch.bfloat16, dev) for i in range(5)]
        for _ in range(args.warmup + reps):
            hmar.hmar_attn_scale_step(*t, sp, side, wl_x.softmax_scale, want_lse=False)
    kern = hmar.hmar_profile_end()
    print(json.dumps({"case": args.case, "calls": args.warmup + reps,
                      "kernels_avg_ms": {k_: round(v_[1] / v_[0], 4) for k_, v_ in kern.items()}}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--batch", type=int, default=0,
                    help="override the batch size (profiling on a reduced case; named in config.workload)")
    ap.add_argument("--case", choices=["256_d30_train", "infer_scale7", "recon_b2048"], default=None,
                    help="run a named side case a few times instead of the benchmark (profiling)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle baseline leg")
    ap.add_argument("--no-extras", action="store_true", help="skip the dense masked comparison and the inference sweep")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    from workloads import CONFIGS
    wl = CONFIGS[WORKLOAD]
    if args.batch > 0:
        import dataclasses
        wl = dataclasses.replace(wl, B=args.batch)
    if args.case is not None:
        run_case(args)
    elif args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
