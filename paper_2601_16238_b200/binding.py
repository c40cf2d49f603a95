"""ctypes binding of ``libvtattn.so``: argument marshalling only.

Every function here has the name of the C entry point it forwards to (see
``include/vt_attn.h``) and takes torch tensors purely as owners of device (or
pinned host) memory; no attention arithmetic happens in Python.  If the shared
library has not been built the loader raises: there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libvtattn.so")
_lib = None

OK = 0
ERR_INVALID_ARGUMENT = -1
ERR_UNSUPPORTED = -2
ERR_WORKSPACE_TOO_SMALL = -3
ERR_CUDA = -4
ERR_DEVICE_TIMEOUT = -5
ERR_STATIC_SCRATCH_TOO_SMALL = -6
STATIC_SCRATCH_ROWS = 1 << 20

_vp, _i, _f, _sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
_DIMS = [_i] * 6

EXPORTS = {
    "vt_attn_abi_version": (_i, []),
    "vt_attn_status_string": (ctypes.c_char_p, [_i]),
    "vt_attn_last_cuda_error": (ctypes.c_char_p, []),
    "vt_attn_fwd": (_i, [_vp] * 5 + _DIMS + [_i, _f, _vp]),
    "vt_attn_fwd_rope": (_i, [_vp] * 7 + _DIMS + [_i, _f, _i, _i, _vp]),
    "vt_attn_fwd_dv": (_i, [_vp] * 5 + _DIMS + [_i, _i, _f, _vp]),
    "vt_attn_fwd_dv_f16": (_i, [_vp] * 5 + _DIMS + [_i, _i, _f, _vp]),
    "vt_attn_fwd_kernel_kind": (_i, _DIMS + [_i]),
    "vt_attn_fwd_f16": (_i, [_vp] * 5 + _DIMS + [_i, _f, _vp]),
    "vt_attn_bwd_f16": (_i, [_vp] * 9 + _DIMS + [_i, _f, _vp, _sz, _vp]),
    "vt_attn_bwd_dv": (_i, [_vp] * 9 + _DIMS + [_i, _i, _f, _vp, _sz, _vp]),
    "vt_attn_bwd_dv_f16": (_i, [_vp] * 9 + _DIMS + [_i, _i, _f, _vp, _sz, _vp]),
    "vt_attn_bwd_workspace_bytes": (_sz, _DIMS),
    "vt_attn_bwd_kernel_kind": (_i, _DIMS),
    "vt_attn_bwd": (_i, [_vp] * 9 + _DIMS + [_i, _f, _vp, _sz, _vp]),
    "vt_attn_bwd_static_scratch": (_i, [_vp] * 9 + _DIMS + [_i, _f, _vp]),
    "vt_attn_bwd_static_scratch_f16": (_i, [_vp] * 9 + _DIMS + [_i, _f, _vp]),
    "vt_attn_fwd_varlen": (_i, [_vp] * 7 + [_i] * 8 + [_i, _f, _vp]),
    "vt_attn_fwd_varlen_f16": (_i, [_vp] * 7 + [_i] * 8 + [_i, _f, _vp]),
    "vt_attn_fwd_splitkv_workspace_bytes": (_sz, _DIMS + [_i]),
    "vt_attn_fwd_splitkv": (_i, [_vp] * 5 + _DIMS + [_i, _f, _i, _vp, _sz, _vp]),
    "vt_attn_fwd_splitkv_f16": (_i, [_vp] * 5 + _DIMS + [_i, _f, _i, _vp, _sz, _vp]),
    "vt_attn_fwd_splitkv_plan": (_i, _DIMS + [_i, ctypes.POINTER(_i), ctypes.POINTER(_i)]),
    "vt_attn_fwd_splitkv_varlen_workspace_bytes": (_sz, [_i] * 8),
    "vt_attn_fwd_splitkv_varlen": (_i, [_vp] * 7 + [_i] * 8 + [_i, _f, _i, _vp, _sz, _vp]),
    "vt_attn_fwd_splitkv_varlen_f16": (_i, [_vp] * 7 + [_i] * 8 + [_i, _f, _i, _vp, _sz, _vp]),
    "vt_attn_fwd_splitkv_varlen_plan": (_i, [_i] * 8 + [ctypes.POINTER(_i), ctypes.POINTER(_i)]),
    "vt_attn_merge_partial": (_i, [_vp] * 4 + [ctypes.c_longlong, _i, _i, _vp]),
    "vt_attn_merge_finish": (_i, [_vp] * 2 + [ctypes.c_longlong, _i, _vp]),
    "vt_attn_accumulate_partial": (_i, [_vp] * 2 + [ctypes.c_longlong, _i, _i, _vp]),
    "vt_attn_bwd_varlen_workspace_bytes": (_sz, [_i, _i]),
    "vt_attn_bwd_varlen": (_i, [_vp] * 11 + [_i] * 8 + [_i, _f, _vp, _sz, _vp]),
    "vt_attn_bwd_varlen_f16": (_i, [_vp] * 11 + [_i] * 8 + [_i, _f, _vp, _sz, _vp]),
    "vt_attn_host_staging_bytes": (_sz, _DIMS + [_i]),
    "vt_attn_fwd_host": (_i, [_vp] * 5 + _DIMS + [_i, _f, _vp, _sz, _vp]),
    "vt_attn_fwd_bwd_host": (_i, [_vp] * 9 + _DIMS + [_i, _f, _vp, _sz, _vp]),
    "vt_attn_fwd_host_f16": (_i, [_vp] * 5 + _DIMS + [_i, _f, _vp, _sz, _vp]),
    "vt_attn_fwd_bwd_host_f16": (_i, [_vp] * 9 + _DIMS + [_i, _f, _vp, _sz, _vp]),
    "vt_attn_device_status": (_i, [ctypes.POINTER(ctypes.c_uint), _vp]),
    "vt_attn_device_status_async": (_i, [_vp, _vp]),
    "vt_attn_device_status_clear": (_i, [_vp]),
    "vt_attn_get_info": (_i, [ctypes.POINTER(_i), _i]),
    "vt_attn_selftest_tile": (_i, [_vp] * 5 + [_i, _f, _vp]),
    "vt_attn_selftest_timeout": (_i, [ctypes.c_uint, _vp]),
}


class VtAttnError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(what)


def load_library(path: str | None = None):
    """Load the shared library (once) and declare its prototypes.  Raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    path = path or LIB_PATH
    if not os.path.exists(path):
        raise FileNotFoundError(
            f"{path} not found: build it with `python -m paper_2601_16238_b200.build` "
            "(there is no fallback path)")
    lib = ctypes.CDLL(path)
    for name, (res, args) in EXPORTS.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    if lib.vt_attn_abi_version() != 1:
        raise RuntimeError("libvtattn.so ABI version mismatch")
    _lib = lib
    return lib


def _check(rc: int, what: str):
    if rc != OK:
        lib = load_library()
        msg = lib.vt_attn_status_string(rc).decode()
        detail = lib.vt_attn_last_cuda_error().decode() if rc == ERR_CUDA else ""
        raise VtAttnError(rc, f"{what}: {msg}" + (f" ({detail})" if detail else ""))


def _stream(stream, device=None):
    import torch
    if stream is None:
        stream = torch.cuda.current_stream(device)
    return stream.cuda_stream         # a plain int: ctypes converts it through the declared c_void_p argtype


def _call(device, fn, *args):
    """Run the C entry point with `device` current: the library launches on the current device."""
    import torch
    if device.type == "cuda" and device.index is not None and device.index != torch.cuda.current_device():
        with torch.cuda.device(device):
            return fn(*args)
    return fn(*args)


def _p(t):
    return t.data_ptr()               # plain int, converted by the declared argtypes (cheaper than a c_void_p object)


def _require(t, dtype, name, device_type="cuda", shape=None, device=None):
    """Raise ValueError unless `t` is a contiguous tensor of `dtype` on a `device_type` device (the very `device`, if
    given) with exactly `shape` (if given).  Every tensor is checked BEFORE the library is entered: the kernels trust the
    sizes they are told, and a short tensor would be read or written past its end on the GPU."""
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name}: expected shape {tuple(shape)}, got {tuple(t.shape)}")
    if t.dtype != dtype or not t.is_contiguous() or t.device.type != device_type:
        raise ValueError(f"{name}: expected a contiguous {dtype} tensor on {device_type}")
    if device is not None and t.device != device:
        raise ValueError(f"{name}: on {t.device}, the other tensors are on {device}")


def _dims(q, k, v=None, own_dv=False):
    """(B, Hq, Hkv, Sq, Sk, D) after checking that q, k (and v) are 4-d tensors whose shapes agree with one another."""
    if q.dim() != 4 or k.dim() != 4:
        raise ValueError("q and k must be [B, H, S, D]")
    B, Hq, Sq, D = (int(x) for x in q.shape)
    Bk, Hkv, Sk, Dk = (int(x) for x in k.shape)
    if Bk != B or Dk != D:
        raise ValueError(f"q {tuple(q.shape)} and k {tuple(k.shape)} disagree on the batch or the head dimension")
    if Hkv <= 0 or Hq % Hkv != 0:
        raise ValueError(f"Hq = {Hq} is not a multiple of Hkv = {Hkv}")
    if v is not None and (v.dim() != 4 or tuple(v.shape[:3]) != (B, Hkv, Sk) or (not own_dv and int(v.shape[3]) != D)):
        raise ValueError(f"v {tuple(v.shape)} does not match k {tuple(k.shape)}")
    return B, Hq, Hkv, Sq, Sk, D


def _inputs(dtype, device_type, q, **others):
    """dtype / contiguity / device of the input tensors (their shapes were checked by _dims)."""
    _require(q, dtype, "q", device_type)
    for name, t in others.items():
        _require(t, dtype, name, device_type, device=q.device)


def _mask_mode(causal) -> int:
    """False/0: no mask; True/1: causal, top-left aligned; 2: causal, bottom-right aligned."""
    mode = int(causal)
    if mode not in (0, 1, 2):
        raise ValueError("causal must be False/0, True/1 (top-left aligned) or 2 (bottom-right aligned)")
    return mode


def _outputs_fwd(q, o, lse, o_shape, lse_shape):
    import torch
    if o is None:
        o = torch.empty(o_shape, dtype=q.dtype, device=q.device)
    else:
        _require(o, q.dtype, "o", shape=o_shape, device=q.device)
    if lse is None:
        lse = torch.empty(lse_shape, dtype=torch.float32, device=q.device)
    else:
        _require(lse, torch.float32, "lse", shape=lse_shape, device=q.device)
    return o, lse


def _fwd(entry: str, dtype, q, k, v, causal, scale, o, lse, stream):
    lib = load_library()
    dims = _dims(q, k, v)
    o, lse = _outputs_fwd(q, o, lse, q.shape, q.shape[:3])
    _inputs(dtype, "cuda", q, k=k, v=v)
    rc = _call(q.device, getattr(lib, entry), _p(q), _p(k), _p(v), _p(o), _p(lse), *dims, _mask_mode(causal), float(scale),
               _stream(stream, q.device))
    _check(rc, entry)
    return o, lse


def vt_attn_fwd(q, k, v, causal: bool, scale: float, o=None, lse=None, stream=None):
    """Forward attention on device tensors [B,H,S,D] (bf16).  Returns (O bf16, LSE fp32)."""
    import torch
    return _fwd("vt_attn_fwd", torch.bfloat16, q, k, v, causal, scale, o, lse, stream)


def vt_attn_fwd_rope(q, k_rotated, v, rope_cos, rope_sin, causal, scale: float, q_pos0: int = 0, o=None, lse=None, stream=None):
    """vt_attn_fwd with the rotary embedding of the queries applied inside the kernel: q unrotated, k_rotated already
    rotated; rope_cos / rope_sin fp32 [positions, D/2].  Returns (O bf16, LSE fp32)."""
    import torch
    lib = load_library()
    dims = _dims(q, k_rotated, v)
    half = dims[5] // 2
    if rope_cos.dim() != 2 or int(rope_cos.shape[1]) != half or rope_sin.shape != rope_cos.shape:
        raise ValueError(f"rope_cos / rope_sin: expected [positions, {half}] tensors of the same shape")
    o, lse = _outputs_fwd(q, o, lse, q.shape, q.shape[:3])
    _inputs(torch.bfloat16, "cuda", q, k=k_rotated, v=v)
    _require(rope_cos, torch.float32, "rope_cos", device=q.device)
    _require(rope_sin, torch.float32, "rope_sin", device=q.device)
    rc = _call(q.device, lib.vt_attn_fwd_rope, _p(q), _p(k_rotated), _p(v), _p(rope_cos), _p(rope_sin), _p(o), _p(lse), *dims,
               _mask_mode(causal), float(scale), int(q_pos0), int(rope_cos.shape[0]), _stream(stream, q.device))
    _check(rc, "vt_attn_fwd_rope")
    return o, lse


def _fwd_dv(name, dtype, q, k, v, causal, scale, o, lse, stream):
    lib = load_library()
    dims = _dims(q, k, v, own_dv=True)
    Dv = int(v.shape[-1])
    o, lse = _outputs_fwd(q, o, lse, tuple(q.shape[:3]) + (Dv,), q.shape[:3])
    _inputs(dtype, "cuda", q, k=k, v=v)
    rc = _call(q.device, getattr(lib, name), _p(q), _p(k), _p(v), _p(o), _p(lse), *dims, Dv, _mask_mode(causal), float(scale),
               _stream(stream, q.device))
    _check(rc, name)
    return o, lse


def vt_attn_fwd_dv(q, k, v, causal, scale: float, o=None, lse=None, stream=None):
    """Forward attention with V (and O) of their own head dimension: q, k [B,H,S,D], v [B,Hkv,Sk,Dv] (bf16).
    Returns (O [B,Hq,Sq,Dv] bf16, LSE fp32)."""
    import torch
    return _fwd_dv("vt_attn_fwd_dv", torch.bfloat16, q, k, v, causal, scale, o, lse, stream)


def vt_attn_fwd_dv_f16(q, k, v, causal, scale: float, o=None, lse=None, stream=None):
    """vt_attn_fwd_dv on fp16 tensors."""
    import torch
    return _fwd_dv("vt_attn_fwd_dv_f16", torch.float16, q, k, v, causal, scale, o, lse, stream)


def vt_attn_fwd_kernel_kind(B, Hq, Hkv, Sq, Sk, D, causal) -> int:
    """0: one query tile per block; 1: the two-tile kernel for long D = 128 sequences; 2: a long and a short query
    tile per block, one after the other (causal shapes whose blocks fill the SMs in one even wave)."""
    rc = load_library().vt_attn_fwd_kernel_kind(B, Hq, Hkv, Sq, Sk, D, _mask_mode(causal))
    if rc < 0:
        _check(rc, "vt_attn_fwd_kernel_kind")
    return rc


def vt_attn_fwd_f16(q, k, v, causal: bool, scale: float, o=None, lse=None, stream=None):
    """Forward attention on fp16 device tensors [B,H,S,D].  Returns (O fp16, LSE fp32)."""
    import torch
    return _fwd("vt_attn_fwd_f16", torch.float16, q, k, v, causal, scale, o, lse, stream)


def vt_attn_bwd_workspace_bytes(B, Hq, Hkv, Sq, Sk, D) -> int:
    return int(load_library().vt_attn_bwd_workspace_bytes(B, Hq, Hkv, Sq, Sk, D))


def vt_attn_bwd_kernel_kind(B, Hq, Hkv, Sq, Sk, D) -> int:
    """0: Delta + one kernel for dK / dV + one for dQ; 1: the single-pass backward (one kernel forms dK, dV and adds its
    share of dQ into a fixed-point accumulator, a last pass rounds dQ)."""
    rc = load_library().vt_attn_bwd_kernel_kind(B, Hq, Hkv, Sq, Sk, D)
    if rc < 0:
        _check(rc, "vt_attn_bwd_kernel_kind")
    return rc


def vt_attn_fwd_splitkv_plan(B, Hq, Hkv, Sq, Sk, D, n_splits=0):
    """(chunks used, heads of a KV group share a tile) for a shape; host-only."""
    lib = load_library()
    used, share = _i(0), _i(0)
    _check(lib.vt_attn_fwd_splitkv_plan(B, Hq, Hkv, Sq, Sk, D, n_splits, ctypes.byref(used), ctypes.byref(share)),
           "vt_attn_fwd_splitkv_plan")
    return used.value, bool(share.value)


def _workspace(workspace, need, device):
    import torch
    if workspace is None:
        return torch.empty(max(256, int(need)), dtype=torch.uint8, device=device)
    if not workspace.is_contiguous() or workspace.device != device:
        raise ValueError(f"workspace: expected a contiguous tensor on {device}")
    return workspace


def _splitkv(entry: str, dtype, q, k, v, causal, scale, n_splits, o, lse, workspace, stream):
    lib = load_library()
    dims = _dims(q, k, v)
    o, lse = _outputs_fwd(q, o, lse, q.shape, q.shape[:3])
    _inputs(dtype, "cuda", q, k=k, v=v)
    workspace = _workspace(workspace, 0 if workspace is not None else lib.vt_attn_fwd_splitkv_workspace_bytes(*dims, int(n_splits)), q.device)
    rc = _call(q.device, getattr(lib, entry), _p(q), _p(k), _p(v), _p(o), _p(lse), *dims, _mask_mode(causal), float(scale),
               int(n_splits), _p(workspace), workspace.numel() * workspace.element_size(), _stream(stream, q.device))
    _check(rc, entry)
    return o, lse


def vt_attn_fwd_splitkv(q, k, v, causal, scale: float, n_splits: int = 0, o=None, lse=None, workspace=None, stream=None):
    """Same result as vt_attn_fwd, keys cut into ``n_splits`` chunks (0: library's choice) merged afterwards."""
    import torch
    return _splitkv("vt_attn_fwd_splitkv", torch.bfloat16, q, k, v, causal, scale, n_splits, o, lse, workspace, stream)


def vt_attn_fwd_splitkv_f16(q, k, v, causal, scale: float, n_splits: int = 0, o=None, lse=None, workspace=None, stream=None):
    """vt_attn_fwd_splitkv on fp16 tensors."""
    import torch
    return _splitkv("vt_attn_fwd_splitkv_f16", torch.float16, q, k, v, causal, scale, n_splits, o, lse, workspace, stream)


def _shapes(*items):
    """(tensor or None, name, shape) triples: every tensor given has exactly that shape."""
    for t, name, shape in items:
        if t is not None and tuple(t.shape) != tuple(shape):
            raise ValueError(f"{name}: expected shape {tuple(shape)}, got {tuple(t.shape)}")


def _grad_out(t, like, name):
    import torch
    if t is None:
        return torch.empty_like(like)
    _require(t, like.dtype, name, shape=like.shape, device=like.device)
    return t


def _bwd(entry: str, dtype, q, k, v, o, d_o, lse, causal, scale, dq, dk, dv, workspace, stream):
    import torch
    lib = load_library()
    dims = _dims(q, k, v)
    _shapes((o, "o", q.shape), (d_o, "d_o", q.shape), (lse, "lse", q.shape[:3]), (dq, "dq", q.shape), (dk, "dk", k.shape),
            (dv, "dv", v.shape))
    _inputs(dtype, "cuda", q, k=k, v=v, o=o, d_o=d_o)
    _require(lse, torch.float32, "lse", device=q.device)
    dq, dk, dv = _grad_out(dq, q, "dq"), _grad_out(dk, k, "dk"), _grad_out(dv, v, "dv")
    workspace = _workspace(workspace, 0 if workspace is not None else lib.vt_attn_bwd_workspace_bytes(*dims), q.device)
    rc = _call(q.device, getattr(lib, entry), _p(q), _p(k), _p(v), _p(o), _p(d_o), _p(lse), _p(dq), _p(dk), _p(dv), *dims,
               _mask_mode(causal), float(scale), _p(workspace), workspace.numel() * workspace.element_size(),
               _stream(stream, q.device))
    _check(rc, entry)
    return dq, dk, dv


def vt_attn_bwd(q, k, v, o, d_o, lse, causal: bool, scale: float, dq=None, dk=None, dv=None,
                workspace=None, stream=None):
    """Backward attention.  Returns (dQ, dK, dV) in bf16."""
    import torch
    return _bwd("vt_attn_bwd", torch.bfloat16, q, k, v, o, d_o, lse, causal, scale, dq, dk, dv, workspace, stream)


def vt_attn_bwd_f16(q, k, v, o, d_o, lse, causal: bool, scale: float, dq=None, dk=None, dv=None,
                    workspace=None, stream=None):
    """Backward attention on fp16 tensors.  Returns (dQ, dK, dV) in fp16."""
    import torch
    return _bwd("vt_attn_bwd_f16", torch.float16, q, k, v, o, d_o, lse, causal, scale, dq, dk, dv, workspace, stream)


def _bwd_dv(entry: str, dtype, q, k, v, o, d_o, lse, causal, scale, dq, dk, dv, workspace, stream):
    import torch
    lib = load_library()
    dims = _dims(q, k, v, own_dv=True)
    Dv = int(v.shape[-1])
    o_shape = tuple(q.shape[:3]) + (Dv,)
    _shapes((o, "o", o_shape), (d_o, "d_o", o_shape), (lse, "lse", q.shape[:3]), (dq, "dq", q.shape), (dk, "dk", k.shape), (dv, "dv", v.shape))
    _inputs(dtype, "cuda", q, k=k, v=v, o=o, d_o=d_o)
    _require(lse, torch.float32, "lse", device=q.device)
    dq, dk, dv = _grad_out(dq, q, "dq"), _grad_out(dk, k, "dk"), _grad_out(dv, v, "dv")
    workspace = _workspace(workspace, 0 if workspace is not None else lib.vt_attn_bwd_workspace_bytes(*dims), q.device)
    rc = _call(q.device, getattr(lib, entry), _p(q), _p(k), _p(v), _p(o), _p(d_o), _p(lse), _p(dq), _p(dk), _p(dv), *dims, Dv,
               _mask_mode(causal), float(scale), _p(workspace), workspace.numel() * workspace.element_size(), _stream(stream, q.device))
    _check(rc, entry)
    return dq, dk, dv


def vt_attn_bwd_dv(q, k, v, o, d_o, lse, causal, scale: float, dq=None, dk=None, dv=None, workspace=None, stream=None):
    """Backward of vt_attn_fwd_dv: q, k [B,H,S,D], v, o, d_o [.., Dv] (bf16).  Returns (dQ, dK, dV)."""
    import torch
    return _bwd_dv("vt_attn_bwd_dv", torch.bfloat16, q, k, v, o, d_o, lse, causal, scale, dq, dk, dv, workspace, stream)


def vt_attn_bwd_dv_f16(q, k, v, o, d_o, lse, causal, scale: float, dq=None, dk=None, dv=None, workspace=None, stream=None):
    """vt_attn_bwd_dv on fp16 tensors."""
    import torch
    return _bwd_dv("vt_attn_bwd_dv_f16", torch.float16, q, k, v, o, d_o, lse, causal, scale, dq, dk, dv, workspace, stream)


def _bwd_static(name, dtype, q, k, v, o, d_o, lse, causal, scale, dq, dk, dv, stream):
    import torch
    lib = load_library()
    dims = _dims(q, k, v)
    _shapes((o, "o", q.shape), (d_o, "d_o", q.shape), (lse, "lse", q.shape[:3]), (dq, "dq", q.shape), (dk, "dk", k.shape),
            (dv, "dv", v.shape))
    _inputs(dtype, "cuda", q, k=k, v=v, o=o, d_o=d_o, dq=dq, dk=dk, dv=dv)
    _require(lse, torch.float32, "lse", device=q.device)
    rc = _call(q.device, getattr(lib, name), _p(q), _p(k), _p(v), _p(o), _p(d_o), _p(lse), _p(dq), _p(dk), _p(dv), *dims,
               _mask_mode(causal), float(scale), _stream(stream, q.device))
    _check(rc, name)
    return dq, dk, dv


def vt_attn_bwd_static_scratch(q, k, v, o, d_o, lse, causal: bool, scale: float, dq, dk, dv, stream=None):
    """Backward for callers that cannot allocate: the Delta scratch is a fixed array inside the
    library, so this wrapper allocates nothing either; dq, dk, dv must be passed in.  Needs
    B * Hq * Sq <= STATIC_SCRATCH_ROWS.  Calls that may overlap on the GPU race on the shared array."""
    import torch
    return _bwd_static("vt_attn_bwd_static_scratch", torch.bfloat16, q, k, v, o, d_o, lse, causal, scale, dq, dk, dv, stream)


def vt_attn_bwd_static_scratch_f16(q, k, v, o, d_o, lse, causal: bool, scale: float, dq, dk, dv, stream=None):
    """vt_attn_bwd_static_scratch on fp16 tensors."""
    import torch
    return _bwd_static("vt_attn_bwd_static_scratch_f16", torch.float16, q, k, v, o, d_o, lse, causal, scale, dq, dk, dv, stream)


def _varlen_dims(q, k, v, cu_q, cu_k, max_sq, max_sk, dtype, **more):
    """(n_seqs, Hq, Hkv, total_q, total_k, max_sq, max_sk, D) after checking the packed tensors against one another.
    `more`: name -> (tensor or None, shape) of further tensors whose shapes are checked before any dtype / device."""
    import torch
    if q.dim() != 3 or k.dim() != 3:
        raise ValueError("packed q and k must be [total, H, D]")
    total_q, Hq, D = (int(x) for x in q.shape)
    total_k, Hkv, Dk = (int(x) for x in k.shape)
    if Dk != D:
        raise ValueError("q and k disagree on the head dimension")
    if Hkv <= 0 or Hq % Hkv != 0:
        raise ValueError(f"Hq = {Hq} is not a multiple of Hkv = {Hkv}")
    if cu_q.dim() != 1 or cu_q.numel() < 1 or cu_k.shape != cu_q.shape:
        raise ValueError("cu_seqlens_q and cu_seqlens_k must be 1-d with n_seqs + 1 entries each")
    _shapes((v, "v", k.shape), *((t, n, shp) for n, (t, shp) in more.items()))
    _inputs(dtype, "cuda", q, k=k, v=v)
    _require(cu_q, torch.int32, "cu_seqlens_q", device=q.device)
    _require(cu_k, torch.int32, "cu_seqlens_k", device=q.device)
    return int(cu_q.numel()) - 1, Hq, Hkv, total_q, total_k, int(max_sq), int(max_sk), D


def _fwd_varlen(entry: str, dtype, q, k, v, cu_seqlens_q, cu_seqlens_k, max_sq, max_sk, causal, scale, o, lse, stream):
    lib = load_library()
    dims = _varlen_dims(q, k, v, cu_seqlens_q, cu_seqlens_k, max_sq, max_sk, dtype,
                        o=(o, q.shape), lse=(lse, (q.shape[1], q.shape[0])))
    o, lse = _outputs_fwd(q, o, lse, q.shape, (q.shape[1], q.shape[0]))
    rc = _call(q.device, getattr(lib, entry), _p(q), _p(k), _p(v), _p(o), _p(lse), _p(cu_seqlens_q), _p(cu_seqlens_k), *dims,
               _mask_mode(causal), float(scale), _stream(stream, q.device))
    _check(rc, entry)
    return o, lse


def vt_attn_fwd_varlen(q, k, v, cu_seqlens_q, cu_seqlens_k, max_sq: int, max_sk: int, causal: bool, scale: float,
                       o=None, lse=None, stream=None):
    """Packed forward: q [total_q,Hq,D], k, v [total_k,Hkv,D] (bf16), cu_seqlens_* int32 device tensors.
    Returns (O [total_q,Hq,D] bf16, LSE [Hq,total_q] fp32)."""
    import torch
    return _fwd_varlen("vt_attn_fwd_varlen", torch.bfloat16, q, k, v, cu_seqlens_q, cu_seqlens_k, max_sq, max_sk, causal, scale, o, lse, stream)


def vt_attn_fwd_varlen_f16(q, k, v, cu_seqlens_q, cu_seqlens_k, max_sq: int, max_sk: int, causal: bool, scale: float,
                           o=None, lse=None, stream=None):
    """vt_attn_fwd_varlen on fp16 tensors."""
    import torch
    return _fwd_varlen("vt_attn_fwd_varlen_f16", torch.float16, q, k, v, cu_seqlens_q, cu_seqlens_k, max_sq, max_sk, causal, scale, o, lse, stream)


def vt_attn_fwd_splitkv_varlen_plan(n_seqs, Hq, Hkv, total_k, max_sq, max_sk, D, n_splits=0):
    """(chunks used, heads of a KV group share a tile) for a packed batch; host-only."""
    lib = load_library()
    used, share = _i(0), _i(0)
    _check(lib.vt_attn_fwd_splitkv_varlen_plan(n_seqs, Hq, Hkv, total_k, max_sq, max_sk, D, n_splits, ctypes.byref(used), ctypes.byref(share)),
           "vt_attn_fwd_splitkv_varlen_plan")
    return used.value, bool(share.value)


def _splitkv_varlen(name, dtype, q, k, v, cu_seqlens_q, cu_seqlens_k, max_sq, max_sk, causal, scale, n_splits, o, lse, workspace, stream):
    lib = load_library()
    dims = _varlen_dims(q, k, v, cu_seqlens_q, cu_seqlens_k, max_sq, max_sk, dtype,      # n_seqs, Hq, Hkv, total_q, total_k, max_sq, max_sk, D
                        o=(o, q.shape), lse=(lse, (q.shape[1], q.shape[0])))
    o, lse = _outputs_fwd(q, o, lse, q.shape, (q.shape[1], q.shape[0]))
    need = 0 if workspace is not None else lib.vt_attn_fwd_splitkv_varlen_workspace_bytes(dims[0], dims[1], dims[2], dims[3], dims[5], dims[6], dims[7], int(n_splits))
    workspace = _workspace(workspace, need, q.device)
    rc = _call(q.device, getattr(lib, name), _p(q), _p(k), _p(v), _p(o), _p(lse), _p(cu_seqlens_q), _p(cu_seqlens_k), *dims,
               _mask_mode(causal), float(scale), int(n_splits), _p(workspace),
               workspace.numel() * workspace.element_size(), _stream(stream, q.device))
    _check(rc, name)
    return o, lse


def vt_attn_fwd_splitkv_varlen(q, k, v, cu_seqlens_q, cu_seqlens_k, max_sq: int, max_sk: int, causal, scale: float, n_splits: int = 0,
                               o=None, lse=None, workspace=None, stream=None):
    """vt_attn_fwd_varlen with the keys cut into chunks (0: library's choice) that are merged afterwards."""
    import torch
    return _splitkv_varlen("vt_attn_fwd_splitkv_varlen", torch.bfloat16, q, k, v, cu_seqlens_q, cu_seqlens_k, max_sq, max_sk, causal, scale,
                           n_splits, o, lse, workspace, stream)


def vt_attn_fwd_splitkv_varlen_f16(q, k, v, cu_seqlens_q, cu_seqlens_k, max_sq: int, max_sk: int, causal, scale: float, n_splits: int = 0,
                                   o=None, lse=None, workspace=None, stream=None):
    """vt_attn_fwd_splitkv_varlen on fp16 tensors."""
    import torch
    return _splitkv_varlen("vt_attn_fwd_splitkv_varlen_f16", torch.float16, q, k, v, cu_seqlens_q, cu_seqlens_k, max_sq, max_sk, causal, scale,
                           n_splits, o, lse, workspace, stream)


def vt_attn_merge_partial(o_acc, lse_acc, o_part, lse_part, first: bool, stream=None):
    """Fold one partial forward result (bf16 O, fp32 LSE over one block of keys) into the fp32 running result."""
    import torch
    if o_part.dim() < 2:
        raise ValueError("o_part must be [..., rows, D]")
    _shapes((o_acc, "o_acc", o_part.shape), (lse_part, "lse_part", o_part.shape[:-1]), (lse_acc, "lse_acc", o_part.shape[:-1]))
    _require(o_part, torch.bfloat16, "o_part")
    _require(o_acc, torch.float32, "o_acc", shape=o_part.shape, device=o_part.device)
    _require(lse_part, torch.float32, "lse_part", shape=o_part.shape[:-1], device=o_part.device)
    _require(lse_acc, torch.float32, "lse_acc", shape=o_part.shape[:-1], device=o_part.device)
    D = int(o_part.shape[-1])
    rc = _call(o_part.device, load_library().vt_attn_merge_partial, _p(o_acc), _p(lse_acc), _p(o_part), _p(lse_part),
               o_part.numel() // D, D, int(bool(first)), _stream(stream, o_part.device))
    _check(rc, "vt_attn_merge_partial")


def vt_attn_accumulate_partial(acc, part, first: bool, stream=None):
    """acc (fp32) += part (bf16); acc = part when ``first``."""
    import torch
    _require(part, torch.bfloat16, "part")
    _require(acc, torch.float32, "acc", shape=part.shape, device=part.device)
    D = int(part.shape[-1])
    rc = _call(part.device, load_library().vt_attn_accumulate_partial, _p(acc), _p(part), part.numel() // D, D,
               int(bool(first)), _stream(stream, part.device))
    _check(rc, "vt_attn_accumulate_partial")


def vt_attn_merge_finish(o_acc, o=None, stream=None):
    """Round the fp32 running result to bf16."""
    import torch
    _require(o_acc, torch.float32, "o_acc")
    if o is None:
        o = torch.empty(o_acc.shape, dtype=torch.bfloat16, device=o_acc.device)
    else:
        _require(o, torch.bfloat16, "o", shape=o_acc.shape, device=o_acc.device)
    D = int(o_acc.shape[-1])
    rc = _call(o_acc.device, load_library().vt_attn_merge_finish, _p(o_acc), _p(o), o_acc.numel() // D, D,
               _stream(stream, o_acc.device))
    _check(rc, "vt_attn_merge_finish")
    return o


def vt_attn_bwd_varlen_workspace_bytes(Hq, total_q) -> int:
    return int(load_library().vt_attn_bwd_varlen_workspace_bytes(Hq, total_q))


def _bwd_varlen(entry: str, dtype, q, k, v, o, d_o, lse, cu_seqlens_q, cu_seqlens_k, max_sq, max_sk, causal, scale, dq, dk, dv,
                workspace, stream):
    import torch
    lib = load_library()
    lse_shape = (q.shape[1], q.shape[0]) if q.dim() == 3 else None
    dims = _varlen_dims(q, k, v, cu_seqlens_q, cu_seqlens_k, max_sq, max_sk, dtype, o=(o, q.shape), d_o=(d_o, q.shape),
                        lse=(lse, lse_shape), dq=(dq, q.shape), dk=(dk, k.shape), dv=(dv, k.shape))
    _require(o, dtype, "o", shape=q.shape, device=q.device)
    _require(d_o, dtype, "d_o", shape=q.shape, device=q.device)
    _require(lse, torch.float32, "lse", shape=(q.shape[1], q.shape[0]), device=q.device)
    dq, dk, dv = _grad_out(dq, q, "dq"), _grad_out(dk, k, "dk"), _grad_out(dv, v, "dv")
    workspace = _workspace(workspace, 0 if workspace is not None else lib.vt_attn_bwd_varlen_workspace_bytes(dims[1], dims[3]), q.device)
    rc = _call(q.device, getattr(lib, entry), _p(q), _p(k), _p(v), _p(o), _p(d_o), _p(lse), _p(dq), _p(dk), _p(dv),
               _p(cu_seqlens_q), _p(cu_seqlens_k), *dims, _mask_mode(causal), float(scale), _p(workspace),
               workspace.numel() * workspace.element_size(), _stream(stream, q.device))
    _check(rc, entry)
    return dq, dk, dv


def vt_attn_bwd_varlen(q, k, v, o, d_o, lse, cu_seqlens_q, cu_seqlens_k, max_sq: int, max_sk: int, causal: bool,
                       scale: float, dq=None, dk=None, dv=None, workspace=None, stream=None):
    """Packed backward.  Returns (dQ, dK, dV) in bf16, laid out like q, k, v."""
    import torch
    return _bwd_varlen("vt_attn_bwd_varlen", torch.bfloat16, q, k, v, o, d_o, lse, cu_seqlens_q, cu_seqlens_k, max_sq, max_sk, causal, scale,
                       dq, dk, dv, workspace, stream)


def vt_attn_bwd_varlen_f16(q, k, v, o, d_o, lse, cu_seqlens_q, cu_seqlens_k, max_sq: int, max_sk: int, causal: bool,
                           scale: float, dq=None, dk=None, dv=None, workspace=None, stream=None):
    """vt_attn_bwd_varlen on fp16 tensors."""
    import torch
    return _bwd_varlen("vt_attn_bwd_varlen_f16", torch.float16, q, k, v, o, d_o, lse, cu_seqlens_q, cu_seqlens_k, max_sq, max_sk, causal,
                       scale, dq, dk, dv, workspace, stream)


def vt_attn_host_staging_bytes(B, Hq, Hkv, Sq, Sk, D, with_backward: bool) -> int:
    return int(load_library().vt_attn_host_staging_bytes(B, Hq, Hkv, Sq, Sk, D, int(bool(with_backward))))


def _fwd_host(name, dtype, q, k, v, o, lse, causal, scale, staging, stream):
    import torch
    lib = load_library()
    dims = _dims(q, k, v)
    _shapes((o, "o", q.shape), (lse, "lse", q.shape[:3]))
    _inputs(dtype, "cpu", q, k=k, v=v, o=o)
    _require(lse, torch.float32, "lse", "cpu")
    _require(staging, torch.uint8, "staging")
    rc = _call(staging.device, getattr(lib, name), _p(q), _p(k), _p(v), _p(o), _p(lse), *dims, _mask_mode(causal), float(scale),
               _p(staging), staging.numel(), _stream(stream, staging.device))
    _check(rc, name)


def _fwd_bwd_host(name, dtype, q, k, v, d_o, o, lse, dq, dk, dv, causal, scale, staging, stream):
    import torch
    lib = load_library()
    dims = _dims(q, k, v)
    _shapes((d_o, "d_o", q.shape), (o, "o", q.shape), (dq, "dq", q.shape), (dk, "dk", k.shape), (dv, "dv", v.shape),
            (lse, "lse", q.shape[:3]))
    _inputs(dtype, "cpu", q, k=k, v=v, d_o=d_o, o=o, dq=dq, dk=dk, dv=dv)
    _require(lse, torch.float32, "lse", "cpu")
    _require(staging, torch.uint8, "staging")
    rc = _call(staging.device, getattr(lib, name), _p(q), _p(k), _p(v), _p(d_o), _p(o), _p(lse), _p(dq), _p(dk), _p(dv), *dims,
               _mask_mode(causal), float(scale), _p(staging), staging.numel(), _stream(stream, staging.device))
    _check(rc, name)


def vt_attn_fwd_host(q, k, v, o, lse, causal: bool, scale: float, staging, stream=None):
    """Forward on (pinned) bf16 host tensors; ``staging`` is a device uint8 tensor.  Asynchronous."""
    import torch
    _fwd_host("vt_attn_fwd_host", torch.bfloat16, q, k, v, o, lse, causal, scale, staging, stream)


def vt_attn_fwd_host_f16(q, k, v, o, lse, causal: bool, scale: float, staging, stream=None):
    """vt_attn_fwd_host on fp16 host tensors."""
    import torch
    _fwd_host("vt_attn_fwd_host_f16", torch.float16, q, k, v, o, lse, causal, scale, staging, stream)


def vt_attn_fwd_bwd_host(q, k, v, d_o, o, lse, dq, dk, dv, causal: bool, scale: float, staging, stream=None):
    """Forward + backward on (pinned) bf16 host tensors.  Asynchronous."""
    import torch
    _fwd_bwd_host("vt_attn_fwd_bwd_host", torch.bfloat16, q, k, v, d_o, o, lse, dq, dk, dv, causal, scale, staging, stream)


def vt_attn_fwd_bwd_host_f16(q, k, v, d_o, o, lse, dq, dk, dv, causal: bool, scale: float, staging, stream=None):
    """vt_attn_fwd_bwd_host on fp16 host tensors."""
    import torch
    _fwd_bwd_host("vt_attn_fwd_bwd_host_f16", torch.float16, q, k, v, d_o, o, lse, dq, dk, dv, causal, scale, staging, stream)


def vt_attn_device_status(stream=None):
    """(status, detail word).  Synchronises the stream."""
    lib = load_library()
    detail = ctypes.c_uint(0)
    rc = lib.vt_attn_device_status(ctypes.byref(detail), _stream(stream))
    return int(rc), int(detail.value)


def vt_attn_device_status_async(word_host, stream=None):
    """Enqueue a copy of the status word into ``word_host`` (a pinned int32 host tensor of one element).  No
    synchronisation: the value is valid after the caller has synchronised the stream (0: no wait expired)."""
    import torch
    if word_host.is_cuda or word_host.dtype != torch.int32 or word_host.numel() != 1:
        raise ValueError("word_host: expected a one-element int32 host tensor")
    _check(load_library().vt_attn_device_status_async(_p(word_host), _stream(stream)), "vt_attn_device_status_async")


def vt_attn_device_status_clear(stream=None):
    """Enqueue the reset of the status word.  No synchronisation."""
    _check(load_library().vt_attn_device_status_clear(_stream(stream)), "vt_attn_device_status_clear")


def vt_attn_get_info():
    lib = load_library()
    arr = (ctypes.c_int * 8)()
    n = lib.vt_attn_get_info(arr, 8)
    return list(arr)[:n]


def vt_attn_selftest_tile(q, k, v, p_scale: float, stream=None):
    """One-tile building-block check.  q, k, v: bf16 [128, D] on the device."""
    import torch
    lib = load_library()
    D = int(q.shape[1])
    s_out = torch.empty(128, 128, dtype=torch.float32, device=q.device)
    o_out = torch.empty(128, D, dtype=torch.float32, device=q.device)
    rc = lib.vt_attn_selftest_tile(_p(q), _p(k), _p(v), _p(s_out), _p(o_out), D, float(p_scale), _stream(stream))
    _check(rc, "vt_attn_selftest_tile")
    return s_out, o_out


def vt_attn_selftest_timeout(limit_ms: int, stream=None):
    rc = load_library().vt_attn_selftest_timeout(int(limit_ms), _stream(stream))
    _check(rc, "vt_attn_selftest_timeout")
