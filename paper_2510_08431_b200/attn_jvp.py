"""Thin Python binding of the C ABI in include/attn_jvp.h (argument marshalling only).

Every step of the computation runs inside the CUDA library; PyTorch is used for
device memory and streams.  There is no CPU or eager fallback: if the library is
missing or the device is not sm_100, calls raise.
"""
from __future__ import annotations

import ctypes
import math
import os
import threading

import torch

KV_TANGENT_FREE = 0x1
FWD_ONLY = 0x2

ERR_NULL, ERR_SHAPE, ERR_UNSUPPORTED_D, ERR_ALIGN, ERR_FLAGS = 1, 2, 3, 4, 5
ERR_SCALE, ERR_ALIAS, ERR_ARCH, ERR_CUDA, ERR_DEVICE_TIMEOUT, ERR_DEVICE_LAYOUT, ERR_WORKSPACE = 6, 7, 8, 9, 10, 11, 12
ERR_STATIC_SCRATCH = 13
STATIC_SCRATCH_BYTES = 32 * 1024 * 1024

EXPORTS = ("attn_jvp_fwd", "attn_jvp_fwd_stream", "attn_jvp_fwd_mu", "attn_jvp_splitkv_workspace_bytes",
           "attn_jvp_suggest_splits", "attn_jvp_fwd_splitkv", "attn_jvp_fwd_splitkv_static", "attn_jvp_host_workspace_bytes",
           "attn_jvp_fwd_host", "attn_jvp_qknorm_fwd", "attn_jvp_set_tuning", "attn_jvp_debug_timeout_info", "attn_jvp_selftest_bounded_wait", "attn_jvp_set_stream", "attn_jvp_device_status", "attn_jvp_strerror",
           "attn_jvp_version")

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libattn_jvp.so")
_lock = threading.Lock()
_lib = None


class AttnJvpError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"attn_jvp error {code}: {msg}")
        self.code = code


def library_path() -> str:
    return _LIB_PATH


def load():
    """Loads libattn_jvp.so (built in-tree by paper_2510_08431_b200.build); raises if it is missing."""
    global _lib
    with _lock:
        if _lib is None:
            if not os.path.exists(_LIB_PATH):
                raise RuntimeError(
                    f"{_LIB_PATH} is missing: build it with `python -m paper_2510_08431_b200.build` "
                    "(there is no fallback path)")
            lib = ctypes.CDLL(_LIB_PATH)
            vp, ci, cu, cf = ctypes.c_void_p, ctypes.c_int, ctypes.c_uint, ctypes.c_float
            common = [vp] * 9 + [ci] * 5 + [cf, cu]
            lib.attn_jvp_fwd.argtypes = common
            lib.attn_jvp_fwd.restype = ci
            lib.attn_jvp_fwd_stream.argtypes = common + [vp]
            lib.attn_jvp_fwd_stream.restype = ci
            lib.attn_jvp_fwd_mu.argtypes = [vp] * 10 + [ci] * 5 + [cf, cu, vp]
            lib.attn_jvp_fwd_mu.restype = ci
            lib.attn_jvp_splitkv_workspace_bytes.argtypes = [ci] * 6
            lib.attn_jvp_splitkv_workspace_bytes.restype = ctypes.c_size_t
            lib.attn_jvp_suggest_splits.argtypes = [ci] * 5
            lib.attn_jvp_suggest_splits.restype = ci
            lib.attn_jvp_fwd_splitkv.argtypes = [vp] * 10 + [ci] * 5 + [cf, cu, ci, vp, ctypes.c_size_t, vp]
            lib.attn_jvp_fwd_splitkv.restype = ci
            lib.attn_jvp_fwd_splitkv_static.argtypes = [vp] * 10 + [ci] * 5 + [cf, cu, ci, vp]
            lib.attn_jvp_fwd_splitkv_static.restype = ci
            lib.attn_jvp_host_workspace_bytes.argtypes = [ci] * 6
            lib.attn_jvp_host_workspace_bytes.restype = ctypes.c_size_t
            lib.attn_jvp_fwd_host.argtypes = [vp] * 9 + [ci] * 5 + [cf, cu, ci, vp, ctypes.c_size_t, vp]
            lib.attn_jvp_fwd_host.restype = ci
            lib.attn_jvp_qknorm_fwd.argtypes = [vp] * 5 + [ctypes.c_longlong, ci, cf, vp]
            lib.attn_jvp_qknorm_fwd.restype = ci
            lib.attn_jvp_selftest_bounded_wait.argtypes = [vp]
            lib.attn_jvp_selftest_bounded_wait.restype = ci
            lib.attn_jvp_set_tuning.argtypes = [ci, ci]
            lib.attn_jvp_set_tuning.restype = ci
            lib.attn_jvp_set_stream.argtypes = [vp]
            lib.attn_jvp_set_stream.restype = ci
            lib.attn_jvp_device_status.argtypes = []
            lib.attn_jvp_device_status.restype = ci
            lib.attn_jvp_strerror.argtypes = [ci]
            lib.attn_jvp_strerror.restype = ctypes.c_char_p
            lib.attn_jvp_version.argtypes = []
            lib.attn_jvp_version.restype = ci
            # benchmarking aid: ATTN_JVP_SOFTMAX_GROUPS=1|2 forces the kernel variant for the whole process
            forced = os.environ.get("ATTN_JVP_SOFTMAX_GROUPS")
            if forced:
                lib.attn_jvp_set_tuning(TUNE_SOFTMAX_GROUPS, int(forced))
            forced = os.environ.get("ATTN_JVP_CTA_PAIR")
            if forced:
                lib.attn_jvp_set_tuning(TUNE_CTA_PAIR, int(forced))
            _lib = lib
    return _lib


def _ptr(x):
    if x is None:
        return None
    if isinstance(x, torch.Tensor):
        return x.data_ptr()
    return int(x)


def attn_jvp_strerror(code: int) -> str:
    return load().attn_jvp_strerror(int(code)).decode()


def attn_jvp_version() -> int:
    return int(load().attn_jvp_version())


TUNE_SOFTMAX_GROUPS = 1
TUNE_CTA_PAIR = 2


def attn_jvp_debug_timeout_info():
    """After ERR_DEVICE_TIMEOUT: (barrier smem address, parity, threadIdx.x, blockIdx.x) of the first wait that
    gave up on the current device, or None."""
    buf = (ctypes.c_uint * 4)()
    lib = load()
    lib.attn_jvp_debug_timeout_info.argtypes = [ctypes.POINTER(ctypes.c_uint)]
    lib.attn_jvp_debug_timeout_info.restype = ctypes.c_int
    return tuple(buf) if lib.attn_jvp_debug_timeout_info(buf) == 1 else None


def attn_jvp_set_tuning(knob: int, value: int) -> int:
    """Process-wide tuning knob (see include/attn_jvp.h); returns the library's return code."""
    return int(load().attn_jvp_set_tuning(int(knob), int(value)))


def attn_jvp_set_stream(cuda_stream) -> int:
    return int(load().attn_jvp_set_stream(_ptr(cuda_stream)))


def attn_jvp_selftest_bounded_wait(cuda_stream=None) -> int:
    """Enqueues the bounded-wait self-test kernel (its wait expires after about 2 s); see include/attn_jvp.h."""
    return int(load().attn_jvp_selftest_bounded_wait(_ptr(cuda_stream)))


def attn_jvp_device_status() -> int:
    return int(load().attn_jvp_device_status())


def attn_jvp_fwd(q, k, v, tq, tk, tv, o, to, lse, B, H, Lq, Lk, D, scale, flags=0) -> int:
    """Raw call: tensors (or integer device addresses) in, return code out.  See include/attn_jvp.h."""
    return int(load().attn_jvp_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(tq), _ptr(tk), _ptr(tv), _ptr(o), _ptr(to),
                                   _ptr(lse), B, H, Lq, Lk, D, float(scale), int(flags)))


def attn_jvp_fwd_stream(q, k, v, tq, tk, tv, o, to, lse, B, H, Lq, Lk, D, scale, flags, cuda_stream) -> int:
    return int(load().attn_jvp_fwd_stream(_ptr(q), _ptr(k), _ptr(v), _ptr(tq), _ptr(tk), _ptr(tv), _ptr(o),
                                          _ptr(to), _ptr(lse), B, H, Lq, Lk, D, float(scale), int(flags),
                                          _ptr(cuda_stream)))


def attn_jvp_fwd_mu(q, k, v, tq, tk, tv, o, to, lse, mu, B, H, Lq, Lk, D, scale, flags, cuda_stream) -> int:
    return int(load().attn_jvp_fwd_mu(_ptr(q), _ptr(k), _ptr(v), _ptr(tq), _ptr(tk), _ptr(tv), _ptr(o), _ptr(to),
                                      _ptr(lse), _ptr(mu), B, H, Lq, Lk, D, float(scale), int(flags),
                                      _ptr(cuda_stream)))


def attn_jvp_splitkv_workspace_bytes(B, H, Lq, Lk, D, splits) -> int:
    return int(load().attn_jvp_splitkv_workspace_bytes(B, H, Lq, Lk, D, splits))


def attn_jvp_suggest_splits(B, H, Lq, Lk, D) -> int:
    return int(load().attn_jvp_suggest_splits(B, H, Lq, Lk, D))


def attn_jvp_fwd_splitkv(q, k, v, tq, tk, tv, o, to, lse, mu, B, H, Lq, Lk, D, scale, flags, splits, workspace,
                         workspace_bytes, cuda_stream) -> int:
    return int(load().attn_jvp_fwd_splitkv(_ptr(q), _ptr(k), _ptr(v), _ptr(tq), _ptr(tk), _ptr(tv), _ptr(o),
                                           _ptr(to), _ptr(lse), _ptr(mu), B, H, Lq, Lk, D, float(scale), int(flags),
                                           int(splits), _ptr(workspace), int(workspace_bytes), _ptr(cuda_stream)))


def attn_jvp_fwd_splitkv_static(q, k, v, tq, tk, tv, o, to, lse, mu, B, H, Lq, Lk, D, scale, flags, splits,
                                cuda_stream) -> int:
    """Split-KV for callers that may not allocate GPU memory (serving loops whose memory was fixed at start-up,
    processes where a framework allocator owns every byte): the chunk partials go to a 32 MiB buffer built into the library instead of
    a caller-provided workspace.  Calls larger than that are refused (ERR_STATIC_SCRATCH); calls that overlap on
    the GPU race on the shared buffer.  Raw call: tensors or device addresses in, return code out."""
    return int(load().attn_jvp_fwd_splitkv_static(_ptr(q), _ptr(k), _ptr(v), _ptr(tq), _ptr(tk), _ptr(tv), _ptr(o),
                                                  _ptr(to), _ptr(lse), _ptr(mu), B, H, Lq, Lk, D, float(scale),
                                                  int(flags), int(splits), _ptr(cuda_stream)))


def attn_jvp_qknorm_fwd(x, tx, w, y, ty, rows, D, eps, cuda_stream) -> int:
    """Raw call of the RMS-norm JVP kernel: tensors or device addresses in, return code out."""
    return int(load().attn_jvp_qknorm_fwd(_ptr(x), _ptr(tx), _ptr(w), _ptr(y), _ptr(ty), int(rows), int(D),
                                          float(eps), _ptr(cuda_stream)))


def qknorm_jvp(x, tx, w, eps=1e-6):
    """y = w . x / rms(x) over the last dimension and its tangent ty for tangent tx (None: primal only).

    x, tx: contiguous CUDA bf16 tensors [..., D]; w: CUDA fp32 [D].  Returns (y, ty)."""
    if not (x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous()):
        raise ValueError("x must be a contiguous CUDA bf16 tensor")
    if tx is not None and not (tx.is_cuda and tx.dtype == torch.bfloat16 and tx.is_contiguous() and tx.shape == x.shape):
        raise ValueError("tx must match x")
    D = x.shape[-1]
    if not (w.is_cuda and w.dtype == torch.float32 and w.is_contiguous() and tuple(w.shape) == (D,)):
        raise ValueError("w must be a contiguous CUDA fp32 tensor of shape [D]")
    y = torch.empty_like(x)
    ty = None if tx is None else torch.empty_like(x)
    with torch.cuda.device(x.device):
        rc = attn_jvp_qknorm_fwd(x, tx, w, y, ty, x.numel() // D, D, eps, torch.cuda.current_stream().cuda_stream)
    if rc != 0:
        raise AttnJvpError(rc, attn_jvp_strerror(rc))
    return y, ty


def _check(t, name, shape):
    if not t.is_cuda or t.dtype != torch.bfloat16 or tuple(t.shape) != shape or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous CUDA bf16 tensor of shape {shape}")


def attention_jvp(q, k, v, tq=None, tk=None, tv=None, scale=None, fwd_only=False, out=None,
                  return_mu=False, splits=1, workspace=None):
    """O, tO, LSE of Algorithm 2 for [B][L][H][D] bf16 CUDA tensors, on torch's current stream.

    ``tk is None and tv is None`` selects the tangent-free K/V path (cross-attention on a constant
    context); ``fwd_only`` runs the plain forward (returns tO = None).  ``out`` may supply
    preallocated (o, to, lse).  ``return_mu`` adds mu = rowsum(P . tS) (the tangent of LSE) as a fourth
    result.  ``splits`` > 1 cuts the keys into chunks processed by independent CTAs and merged by a
    second kernel (for few queries and many keys), ``splits=0`` lets the library choose
    (``attn_jvp_suggest_splits``); ``workspace`` may supply its scratch (a CUDA uint8
    tensor of at least attn_jvp_splitkv_workspace_bytes), else it is allocated here with torch.
    Returns (o, to, lse) or (o, to, lse, mu).
    """
    B, Lq, H, D = q.shape
    Lk = k.shape[1]
    _check(q, "q", (B, Lq, H, D)); _check(k, "k", (B, Lk, H, D)); _check(v, "v", (B, Lk, H, D))
    flags = 0
    if fwd_only:
        flags |= FWD_ONLY
        tq = tk = tv = None
    else:
        _check(tq, "tq", (B, Lq, H, D))
        if tk is None and tv is None:
            flags |= KV_TANGENT_FREE
        else:
            _check(tk, "tk", (B, Lk, H, D)); _check(tv, "tv", (B, Lk, H, D))
    if scale is None:
        scale = 1.0 / math.sqrt(D)
    if out is None:
        o = torch.empty_like(q)
        to = None if fwd_only else torch.empty_like(q)
        lse = torch.empty((B, H, Lq), dtype=torch.float32, device=q.device)
    else:
        o, to, lse = out
    mu = torch.empty((B, H, Lq), dtype=torch.float32, device=q.device) if return_mu else None
    with torch.cuda.device(q.device):
        stream = torch.cuda.current_stream().cuda_stream
        if splits == 0:
            splits = attn_jvp_suggest_splits(B, H, Lq, Lk, D)
        if splits > 1:
            need = attn_jvp_splitkv_workspace_bytes(B, H, Lq, Lk, D, splits)
            if workspace is None and need > 0:
                workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
            nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
            rc = attn_jvp_fwd_splitkv(q, k, v, tq, tk, tv, o, to, lse, mu, B, H, Lq, Lk, D, scale, flags, splits,
                                      workspace, nbytes, stream)
        elif return_mu:
            rc = attn_jvp_fwd_mu(q, k, v, tq, tk, tv, o, to, lse, mu, B, H, Lq, Lk, D, scale, flags, stream)
        else:
            rc = attn_jvp_fwd_stream(q, k, v, tq, tk, tv, o, to, lse, B, H, Lq, Lk, D, scale, flags, stream)
    if rc != 0:
        raise AttnJvpError(rc, attn_jvp_strerror(rc))
    return (o, to, lse, mu) if return_mu else (o, to, lse)


def attn_jvp_host_workspace_bytes(B, H, Lq, Lk, D, heads_per_stage=0) -> int:
    return int(load().attn_jvp_host_workspace_bytes(B, H, Lq, Lk, D, int(heads_per_stage)))


def attn_jvp_fwd_host(q, k, v, tq, tk, tv, o, to, lse, B, H, Lq, Lk, D, scale, flags, heads_per_stage, workspace,
                      workspace_bytes, cuda_stream) -> int:
    """Raw call on HOST tensors (or integer host addresses); ``workspace`` is device memory.  See include/attn_jvp.h."""
    return int(load().attn_jvp_fwd_host(_ptr(q), _ptr(k), _ptr(v), _ptr(tq), _ptr(tk), _ptr(tv), _ptr(o), _ptr(to),
                                        _ptr(lse), B, H, Lq, Lk, D, float(scale), int(flags), int(heads_per_stage),
                                        _ptr(workspace), int(workspace_bytes), _ptr(cuda_stream)))


def attention_jvp_host(q, k, v, tq=None, tk=None, tv=None, scale=None, fwd_only=False, device="cuda:0", out=None,
                       workspace=None, heads_per_stage=0, synchronize=True):
    """Host-to-host call: CPU bf16 tensors [B][L][H][D] in (pinned memory lets the copies overlap the kernel),
    CPU tensors out.

    The library pipelines groups of heads: copy in, kernel, copy out (``attn_jvp_fwd_host``).  ``out`` = (o, to,
    lse) CPU tensors to fill (allocated pinned if omitted; ``to`` is None with ``fwd_only``); ``workspace`` = a
    uint8 CUDA tensor of at least ``attn_jvp_host_workspace_bytes(...)`` bytes (allocated if omitted).  With
    ``synchronize=False`` the call returns once everything is enqueued on the current stream of ``device``.
    Returns (o, to, lse) on the CPU.
    """
    dev = torch.device(device)
    for name, t in (("q", q), ("k", k), ("v", v), ("tq", tq), ("tk", tk), ("tv", tv)):
        if t is not None:
            if t.device.type != "cpu" or t.dtype != torch.bfloat16 or not t.is_contiguous() or t.dim() != 4:
                raise ValueError(f"{name} must be a contiguous CPU bf16 tensor [B][L][H][D]")
    B, Lq, H, D = q.shape
    Lk = k.shape[1]
    if k.shape != (B, Lk, H, D) or v.shape != k.shape:
        raise ValueError("k and v must be [B][Lk][H][D] with the B, H, D of q")
    flags = 0
    if fwd_only:
        flags |= FWD_ONLY
        tq = tk = tv = None
    else:
        if tq is None or tq.shape != q.shape:
            raise ValueError("tq (shape of q) is required unless fwd_only")
        if tk is None and tv is None:
            flags |= KV_TANGENT_FREE
        elif tk is None or tv is None or tk.shape != k.shape or tv.shape != k.shape:
            raise ValueError("tk and tv must both be given (shape of k) or both be None")
    if scale is None:
        scale = 1.0 / math.sqrt(D)
    if out is None:
        o = torch.empty((B, Lq, H, D), dtype=torch.bfloat16, pin_memory=True)
        to = None if fwd_only else torch.empty((B, Lq, H, D), dtype=torch.bfloat16, pin_memory=True)
        lse = torch.empty((B, H, Lq), dtype=torch.float32, pin_memory=True)
    else:
        o, to, lse = out
    need = attn_jvp_host_workspace_bytes(B, H, Lq, Lk, D, heads_per_stage)
    with torch.cuda.device(dev):
        if workspace is None:
            workspace = torch.empty(need, dtype=torch.uint8, device=dev)
        stream = torch.cuda.current_stream(dev)
        rc = attn_jvp_fwd_host(q, k, v, tq, tk, tv, o, to, lse, B, H, Lq, Lk, D, scale, flags, heads_per_stage,
                               workspace, workspace.numel() * workspace.element_size(), stream.cuda_stream)
        if rc != 0:
            raise AttnJvpError(rc, attn_jvp_strerror(rc))
        if synchronize:
            stream.synchronize()
            st = attn_jvp_device_status()
            if st != 0:
                raise AttnJvpError(st, attn_jvp_strerror(st))
    return o, to, lse
