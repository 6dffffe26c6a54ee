"""ctypes binding of libhmar.so: argument marshalling only.

Every function here has the name and argument order of the C entry point it wraps (see
include/hmar.h). Tensors are torch CUDA tensors used purely as device buffers; all of the
arithmetic runs inside the library's kernels. There is no CPU fallback: if the shared library
is missing or fails to load, importing this module raises.
"""
import ctypes
import os

import torch

from . import build as _build

_LIB = None

HMAR_OK = 0
HMAR_ERR_BAD_ARG = -1
HMAR_ERR_UNSUPPORTED = -2
HMAR_ERR_CUDA = -3
HMAR_ERR_WORKSPACE = -4
HMAR_ERR_DEVICE_TIMEOUT = -5
HMAR_ERR_BOUNDS = -6

HMAR_WINDOW_MARKOV = 0      # scales k-1 and k (HMAR)
HMAR_WINDOW_CAUSAL = 1      # scales 1..k (VAR's block-causal mask)
HMAR_WINDOW_SELF = 2        # scale k only (block-diagonal)
HMAR_WINDOW_PREV = 3        # scale k-1 only; the first scale attends to itself

EXPORTED_SYMBOLS = (
    "hmar_attn_fwd", "hmar_attn_fwd_f32", "hmar_attn_fwd_window", "hmar_attn_fwd_window_f32", "hmar_attn_fwd_packed", "hmar_attn_bwd_packed",
    "hmar_attn_bwd_workspace_bytes", "hmar_attn_bwd", "hmar_attn_bwd_f32", "hmar_attn_bwd_window",
    "hmar_attn_bwd_window_f32", "hmar_schedule_tiles_window", "hmar_attn_bwd_noalloc", "hmar_attn_scale_step", "hmar_attn_scale_step_f32", "hmar_attn_scale_step_strided", "hmar_schedule_tiles", "hmar_schedule_bwd_full_tile_share",
    "hmar_recon_accumulate", "hmar_recon_downsample", "hmar_device_status", "hmar_selftest_bounded_wait", "hmar_profile_begin", "hmar_profile_end", "hmar_debug_force_simt", "hmar_launch_count", "hmar_shutdown",
    "hmar_status_string",
)


class HmarError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


def lib():
    """Load (building first if the sources are newer) the in-tree shared library."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = _build.LIB_PATH                 # libhmar.so, or the library named by the HMAR_LIBRARY environment variable
    if os.path.abspath(path) == os.path.abspath(_build.CHECKED_LIB_PATH):
        if _build.needs_build(path):
            path = _build.build(checked=True)
    elif "HMAR_LIBRARY" not in os.environ and _build.needs_build():
        path = _build.build()
    L = ctypes.CDLL(path)
    vp, ip, fp = ctypes.c_void_p, ctypes.POINTER(ctypes.c_int), ctypes.c_float
    i = ctypes.c_int
    L.hmar_attn_fwd.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, ip, fp, vp]
    L.hmar_attn_fwd_f32.argtypes = L.hmar_attn_fwd.argtypes
    L.hmar_attn_fwd_window.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, ip, i, fp, vp]
    L.hmar_attn_fwd_window_f32.argtypes = L.hmar_attn_fwd_window.argtypes
    L.hmar_attn_fwd_packed.argtypes = [vp, vp, vp, i, i, i, i, ip, fp, vp]
    L.hmar_attn_bwd_packed.argtypes = [vp] * 5 + [vp, ctypes.c_size_t, i, i, i, i, ip, fp, vp]
    L.hmar_attn_bwd_workspace_bytes.argtypes = [i, i, i, i, ip]
    L.hmar_attn_bwd_workspace_bytes.restype = ctypes.c_size_t
    L.hmar_attn_bwd.argtypes = [vp] * 9 + [vp, ctypes.c_size_t, i, i, i, i, ip, fp, vp]
    L.hmar_attn_bwd_f32.argtypes = L.hmar_attn_bwd.argtypes
    L.hmar_attn_bwd_window.argtypes = [vp] * 9 + [vp, ctypes.c_size_t, i, i, i, i, ip, i, fp, vp]
    L.hmar_attn_bwd_window_f32.argtypes = L.hmar_attn_bwd_window.argtypes
    L.hmar_schedule_tiles_window.argtypes = [i, ip, i, i, ctypes.POINTER(ctypes.c_int32), i]
    L.hmar_schedule_bwd_full_tile_share.argtypes = [i, ip, i]
    L.hmar_attn_bwd_noalloc.argtypes = [vp] * 9 + [i, i, i, i, ip, fp, vp]
    L.hmar_attn_scale_step.argtypes = [vp] * 7 + [i, i, i, i, i, fp, vp]
    L.hmar_attn_scale_step_f32.argtypes = L.hmar_attn_scale_step.argtypes
    ll = ctypes.c_longlong
    L.hmar_attn_scale_step_strided.argtypes = [vp] * 7 + [i, i, i, i, i, ll, ll, ll, ll, fp, vp]
    L.hmar_schedule_tiles.argtypes = [i, ip, i, ctypes.POINTER(ctypes.c_int32), i]
    L.hmar_recon_accumulate.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, i, vp]
    L.hmar_recon_downsample.argtypes = [vp, vp, i, i, i, i, vp]
    L.hmar_device_status.argtypes = [ip]
    L.hmar_selftest_bounded_wait.argtypes = [vp]
    L.hmar_profile_begin.restype = None
    L.hmar_profile_end.argtypes = [ctypes.c_char_p, ctypes.c_size_t]
    L.hmar_debug_force_simt.argtypes = [i]
    L.hmar_launch_count.restype = ctypes.c_longlong
    L.hmar_shutdown.restype = None
    L.hmar_status_string.argtypes = [i]
    L.hmar_status_string.restype = ctypes.c_char_p
    for name in EXPORTED_SYMBOLS:
        getattr(L, name)                     # a missing symbol fails here, at load time
    _LIB = L
    return L


def status_string(status):
    return lib().hmar_status_string(int(status)).decode()


def _sides(side_lens):
    arr = (ctypes.c_int * len(side_lens))(*[int(s) for s in side_lens])
    return arr, len(side_lens)


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _check(status, where):
    if status != HMAR_OK:
        raise HmarError(status, where)


def _is_f32(t):
    if t.dtype == torch.float32:
        return True
    if t.dtype == torch.bfloat16:
        return False
    raise TypeError("tensors must be bfloat16 or float32")


def _need(*tensors):
    for t in tensors:
        if t is not None and (not t.is_cuda or not t.is_contiguous()):
            raise ValueError("tensors must be contiguous CUDA tensors")


def hmar_attn_fwd(q, k, v, side_lens, softmax_scale, out=None, lse=None, stream=None, window=HMAR_WINDOW_MARKOV):
    """Training forward. q, k, v: [B,H,L,D]. Returns (out [B,H,L,D], lse [B,H,L] fp32).
    `window` other than HMAR_WINDOW_MARKOV goes through hmar_attn_fwd_window."""
    _need(q, k, v, out, lse)
    B, H, L, D = q.shape
    if out is None:
        out = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((B, H, L), dtype=torch.float32, device=q.device)
    sides, n = _sides(side_lens)
    if window != HMAR_WINDOW_MARKOV:
        fn = lib().hmar_attn_fwd_window_f32 if _is_f32(q) else lib().hmar_attn_fwd_window
        _check(fn(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(lse), B, H, D, n, sides, int(window),
                  float(softmax_scale), _stream(stream)), "hmar_attn_fwd_window")
        return out, lse
    fn = lib().hmar_attn_fwd_f32 if _is_f32(q) else lib().hmar_attn_fwd
    _check(fn(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(lse), B, H, D, n, sides,
              float(softmax_scale), _stream(stream)), "hmar_attn_fwd")
    return out, lse


def hmar_attn_fwd_packed(qkv, side_lens, softmax_scale, out=None, lse=None, stream=None):
    """Training forward on the packed projection output. qkv: [B,L,3,H,D] bf16.
    Returns (out [B,L,H,D], lse [B,H,L] fp32)."""
    _need(qkv, out, lse)
    B, L, three, H, D = qkv.shape
    if three != 3:
        raise ValueError("qkv must be [B, L, 3, H, D]")
    if out is None:
        out = torch.empty((B, L, H, D), dtype=qkv.dtype, device=qkv.device)
    if lse is None:
        lse = torch.empty((B, H, L), dtype=torch.float32, device=qkv.device)
    sides, n = _sides(side_lens)
    _check(lib().hmar_attn_fwd_packed(_ptr(qkv), _ptr(out), _ptr(lse), B, H, D, n, sides, float(softmax_scale),
                                      _stream(stream)), "hmar_attn_fwd_packed")
    return out, lse


def hmar_attn_bwd_packed(qkv, out, lse, dout, side_lens, softmax_scale, dqkv=None, workspace=None, stream=None):
    """Training backward on the packed layouts. qkv [B,L,3,H,D], out and dout [B,L,H,D], lse [B,H,L].
    Returns dqkv [B,L,3,H,D]."""
    _need(qkv, out, lse, dout, dqkv, workspace)
    B, L, three, H, D = qkv.shape
    if three != 3 or _is_f32(qkv):
        raise ValueError("qkv must be bfloat16 [B, L, 3, H, D]")
    dqkv = torch.empty_like(qkv) if dqkv is None else dqkv
    if workspace is None:
        workspace = torch.empty(hmar_attn_bwd_workspace_bytes(B, H, D, side_lens), dtype=torch.uint8, device=qkv.device)
    sides, n = _sides(side_lens)
    _check(lib().hmar_attn_bwd_packed(_ptr(qkv), _ptr(out), _ptr(lse), _ptr(dout), _ptr(dqkv), _ptr(workspace),
                                      workspace.numel(), B, H, D, n, sides, float(softmax_scale), _stream(stream)),
           "hmar_attn_bwd_packed")
    return dqkv


def hmar_attn_bwd_workspace_bytes(B, H, D, side_lens):
    sides, n = _sides(side_lens)
    return int(lib().hmar_attn_bwd_workspace_bytes(B, H, D, n, sides))


def hmar_attn_bwd(q, k, v, out, lse, dout, side_lens, softmax_scale, dq=None, dk=None, dv=None,
                  workspace=None, stream=None, window=HMAR_WINDOW_MARKOV):
    """Training backward. Returns (dq, dk, dv), each [B,H,L,D].
    `window` other than HMAR_WINDOW_MARKOV goes through hmar_attn_bwd_window."""
    _need(q, k, v, out, lse, dout, dq, dk, dv, workspace)
    B, H, L, D = q.shape
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(q) if dk is None else dk
    dv = torch.empty_like(q) if dv is None else dv
    if workspace is None:
        workspace = torch.empty(hmar_attn_bwd_workspace_bytes(B, H, D, side_lens), dtype=torch.uint8,
                                device=q.device)
    sides, n = _sides(side_lens)
    if window != HMAR_WINDOW_MARKOV:
        fn = lib().hmar_attn_bwd_window_f32 if _is_f32(q) else lib().hmar_attn_bwd_window
        _check(fn(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(lse), _ptr(dout), _ptr(dq), _ptr(dk), _ptr(dv),
                  _ptr(workspace), workspace.numel() * workspace.element_size(), B, H, D, n, sides, int(window),
                  float(softmax_scale), _stream(stream)), "hmar_attn_bwd_window")
        return dq, dk, dv
    fn = lib().hmar_attn_bwd_f32 if _is_f32(q) else lib().hmar_attn_bwd
    _check(fn(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(lse), _ptr(dout), _ptr(dq), _ptr(dk), _ptr(dv),
              _ptr(workspace), workspace.numel() * workspace.element_size(), B, H, D, n, sides,
              float(softmax_scale), _stream(stream)), "hmar_attn_bwd")
    return dq, dk, dv


HMAR_NOALLOC_MAX_ROWS = 32768


def hmar_attn_bwd_noalloc(q, k, v, out, lse, dout, side_lens, softmax_scale, dq, dk, dv, stream=None):
    """Backward through the entry point that allocates nothing: for callers that may not touch the
    device allocator (memory owned by someone else's pool, no growth after start-up, no call that may
    synchronise). The caller passes every output tensor; neither this wrapper nor the library
    allocates. B*H*L must not exceed HMAR_NOALLOC_MAX_ROWS, and calls must not overlap on the GPU."""
    _need(q, k, v, out, lse, dout, dq, dk, dv)
    if _is_f32(q):
        raise TypeError("hmar_attn_bwd_noalloc takes bfloat16 tensors")
    B, H, L, D = q.shape
    sides, n = _sides(side_lens)
    _check(lib().hmar_attn_bwd_noalloc(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(lse), _ptr(dout), _ptr(dq),
                                       _ptr(dk), _ptr(dv), B, H, D, n, sides, float(softmax_scale),
                                       _stream(stream)), "hmar_attn_bwd_noalloc")
    return dq, dk, dv


def hmar_attn_scale_step(q, k_prev, v_prev, k_cur, v_cur, side_prev, side_cur, softmax_scale,
                         out=None, lse=None, want_lse=True, stream=None):
    """Inference step of one scale. q, k_cur, v_cur: [B,H,side_cur^2,D]; k_prev, v_prev:
    [B,H,side_prev^2,D] or None when side_prev == 0. Returns (out, lse or None)."""
    _need(q, k_prev, v_prev, k_cur, v_cur, out, lse)
    B, H, n_cur, D = q.shape
    if out is None:
        out = torch.empty_like(q)
    if lse is None and want_lse:
        lse = torch.empty((B, H, n_cur), dtype=torch.float32, device=q.device)
    fn = lib().hmar_attn_scale_step_f32 if _is_f32(q) else lib().hmar_attn_scale_step
    _check(fn(_ptr(q), _ptr(k_prev), _ptr(v_prev), _ptr(k_cur), _ptr(v_cur), _ptr(out), _ptr(lse),
              B, H, D, int(side_prev), int(side_cur), float(softmax_scale), _stream(stream)),
           "hmar_attn_scale_step")
    return out, lse


def hmar_attn_scale_step_strided(q, k_prev, v_prev, k_cur, v_cur, side_prev, side_cur, softmax_scale,
                                 out=None, lse=None, want_lse=True, stream=None):
    """Inference step on views whose heads are not packed back to back, e.g. slices of one K/V ring
    [B,H,ring_rows,D] (k_prev = ring[:, :, a:a+n_prev], k_cur = ring[:, :, a+n_prev:a+n_prev+n_cur]).
    Every tensor is a [B,H,rows,D] view with contiguous rows and heads a constant stride apart."""
    B, H, n_cur, D = q.shape

    def head_stride(t):
        if t is None:
            return 0
        if not t.is_cuda or t.stride(3) != 1 or t.stride(2) != D or (t.shape[1] > 1 and t.shape[0] > 1 and t.stride(0) != H * t.stride(1)):
            raise ValueError("views must have contiguous rows and evenly spaced heads")
        return t.stride(1) if t.shape[1] > 1 else (t.stride(0) if t.shape[0] > 1 else t.shape[2] * D)

    if _is_f32(q):
        raise TypeError("hmar_attn_scale_step_strided takes bfloat16 tensors")
    if out is None:
        out = torch.empty((B, H, n_cur, D), dtype=q.dtype, device=q.device)
    if lse is None and want_lse:
        lse = torch.empty((B, H, n_cur), dtype=torch.float32, device=q.device)
    _check(lib().hmar_attn_scale_step_strided(
        _ptr(q), _ptr(k_prev), _ptr(v_prev), _ptr(k_cur), _ptr(v_cur), _ptr(out), _ptr(lse), B, H, D, int(side_prev),
        int(side_cur), head_stride(q), head_stride(k_prev), head_stride(k_cur), head_stride(out), float(softmax_scale),
        _stream(stream)), "hmar_attn_scale_step_strided")
    return out, lse


def hmar_recon_accumulate(xhat, codebook, tokens_new, tokens_old=None, mask=None, tokens_out=None, stream=None):
    """xhat [B,C,S,S] fp32 += bicubic(lookup(codebook [V,C], selected tokens [B,s,s])); returns xhat.
    `mask` (uint8 [B,s,s]) chooses tokens_new over tokens_old per position; `tokens_out` receives the selection."""
    _need(xhat, codebook, tokens_new, tokens_old, mask, tokens_out)
    if xhat.dtype != torch.float32 or codebook.dtype != torch.float32 or tokens_new.dtype != torch.int32:
        raise TypeError("xhat and codebook must be float32, tokens int32")
    if mask is not None and mask.dtype != torch.uint8:
        raise TypeError("mask must be uint8")
    B, C, S, _ = xhat.shape
    V = codebook.shape[0]
    side = tokens_new.shape[1]
    _check(lib().hmar_recon_accumulate(_ptr(xhat), _ptr(codebook), _ptr(tokens_old), _ptr(tokens_new), _ptr(mask),
                                       _ptr(tokens_out), B, C, V, side, S, _stream(stream)), "hmar_recon_accumulate")
    return xhat


def hmar_recon_downsample(xhat, out_side, out=None, stream=None):
    """Area interpolation of xhat [B,C,S,S] fp32 down to [B,C,out_side,out_side]; returns the result."""
    _need(xhat, out)
    if xhat.dtype != torch.float32:
        raise TypeError("xhat must be float32")
    B, C, S, _ = xhat.shape
    if out is None:
        out = torch.empty((B, C, out_side, out_side), dtype=torch.float32, device=xhat.device)
    elif out.dtype != torch.float32 or tuple(out.shape) != (B, C, out_side, out_side):
        raise ValueError("out must be float32 [B, C, out_side, out_side]")
    _check(lib().hmar_recon_downsample(_ptr(xhat), _ptr(out), B, C, S, int(out_side), _stream(stream)), "hmar_recon_downsample")
    return out


def hmar_schedule_tiles(side_lens, direction, window=HMAR_WINDOW_MARKOV):
    """Work list of one head as a list of dicts (host only; needs no GPU)."""
    sides, n = _sides(side_lens)
    count = lib().hmar_schedule_tiles_window(n, sides, int(window), int(direction), None, 0)
    if count < 0:
        raise HmarError(count, "hmar_schedule_tiles")
    buf = (ctypes.c_int32 * (6 * count))()
    lib().hmar_schedule_tiles_window(n, sides, int(window), int(direction), buf, count)
    keys = ("row_begin", "row_count", "partner_begin", "partner_end", "uniform", "cost")
    return [dict(zip(keys, buf[6 * t:6 * t + 6])) for t in range(count)]


def hmar_schedule_bwd_full_tile_share(side_lens, window=HMAR_WINDOW_MARKOV):
    """Thousandths of a head's backward steps that lie in full tiles (host only; needs no GPU)."""
    sides, n = _sides(side_lens)
    share = lib().hmar_schedule_bwd_full_tile_share(n, sides, int(window))
    if share < 0:
        raise HmarError(share, "hmar_schedule_bwd_full_tile_share")
    return share


def hmar_device_status():
    """(status, detail) recorded by the kernels since the last call; synchronises the device."""
    detail = ctypes.c_int(0)
    status = lib().hmar_device_status(ctypes.byref(detail))
    return status, detail.value


def hmar_selftest_bounded_wait(stream=None):
    """Launches the one-block kernel whose bounded wait must run out (see include/hmar.h)."""
    _check(lib().hmar_selftest_bounded_wait(_stream(stream)), "hmar_selftest_bounded_wait")


def hmar_profile_begin():
    lib().hmar_profile_begin()


def hmar_profile_end():
    """{kernel name: (launches, total_ms)} for the kernels launched since hmar_profile_begin()."""
    buf = ctypes.create_string_buffer(8192)
    _check(lib().hmar_profile_end(buf, len(buf)), "hmar_profile_end")
    out = {}
    for line in buf.value.decode().splitlines():
        name, count, ms = line.split()
        out[name] = (int(count), float(ms))
    return out


def hmar_debug_force_simt(enable):
    return lib().hmar_debug_force_simt(1 if enable else 0)


def hmar_launch_count():
    return int(lib().hmar_launch_count())


def hmar_shutdown():
    lib().hmar_shutdown()
