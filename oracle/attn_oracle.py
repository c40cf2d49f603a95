"""ctypes wrapper around the fp64 CPU oracle (``attn_oracle.c``).

TEST INFRASTRUCTURE ONLY: the oracle defines what "correct" means for the GPU
library and is timed as the reported CPU baseline.  Nothing in the product path
may import this module, and this module imports nothing from the product.

The operation is the one the paper benchmarks as "Attention (fwd)" and
"Attention (bwd)" against torch scaled_dot_product_attention (kernel
microbenchmark table); the formulas are written out at the top of
``attn_oracle.c``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "attn_oracle.c")
_LIB = os.path.join(_HERE, "libattn_oracle.so")
_lock = threading.Lock()
_lib = None

_DP = ctypes.POINTER(ctypes.c_double)


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP, -O3) if the shared object is stale."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-std=c11", "-fPIC", "-shared",
                   "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        dims = [ctypes.c_int] * 6
        lib.attn_oracle_num_threads.restype = ctypes.c_int
        lib.attn_oracle_set_num_threads.restype = ctypes.c_int
        lib.attn_oracle_set_num_threads.argtypes = [ctypes.c_int]
        lib.attn_oracle_fwd.restype = ctypes.c_int
        lib.attn_oracle_fwd.argtypes = [_DP] * 5 + dims + [ctypes.c_int, ctypes.c_double]
        lib.attn_oracle_probs.restype = ctypes.c_int
        lib.attn_oracle_probs.argtypes = ([_DP] * 3 + dims + [ctypes.c_int, ctypes.c_double,
                                                              ctypes.c_int, ctypes.c_int])
        lib.attn_oracle_bwd.restype = ctypes.c_int
        lib.attn_oracle_bwd.argtypes = [_DP] * 8 + dims + [ctypes.c_int, ctypes.c_double]
        _lib = lib
    return _lib


def num_threads() -> int:
    """Threads the oracle's OpenMP loops will use."""
    return int(_load().attn_oracle_num_threads())


def set_num_threads(n: int) -> int:
    """Use ``n`` OpenMP threads from now on; returns the number in force."""
    return int(_load().attn_oracle_set_num_threads(int(n)))


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns (uint16) to float64 exactly."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen IEEE half bit patterns (uint16) to float64 exactly."""
    return np.ascontiguousarray(bits, dtype=np.uint16).view(np.float16).astype(np.float64)


def _f64(x: np.ndarray) -> np.ndarray:
    if x.dtype == np.uint16:
        return bf16_bits_to_f64(x)
    return np.ascontiguousarray(x, dtype=np.float64)


def _ptr(x: np.ndarray):
    return x.ctypes.data_as(_DP)


def _mask_mode(causal) -> int:
    """False/0: no mask; True/1: causal, top-left aligned; 2: causal, bottom-right aligned."""
    mode = int(causal)
    if mode not in (0, 1, 2):
        raise ValueError("causal must be False/0, True/1 (top-left) or 2 (bottom-right)")
    return mode


def _dims(q, k):
    B, Hq, Sq, D = q.shape
    Bk, Hkv, Sk, Dk = k.shape
    if Bk != B or Dk != D:
        raise ValueError("q and k disagree on batch or head dim")
    return B, Hq, Hkv, Sq, Sk, D


def attn_fwd(q, k, v, causal, scale: float):
    """O [B,Hq,Sq,D] and LSE [B,Hq,Sq] in fp64.  Inputs: float64, or uint16 bf16 bits.

    ``causal``: False/0 none, True/1 top-left aligned, 2 bottom-right aligned (see attn_oracle.c)."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    B, Hq, Hkv, Sq, Sk, D = _dims(q, k)
    if v.shape != k.shape:
        raise ValueError("k and v shapes differ")
    o = np.empty((B, Hq, Sq, D), dtype=np.float64)
    lse = np.empty((B, Hq, Sq), dtype=np.float64)
    rc = _load().attn_oracle_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse),
                                 B, Hq, Hkv, Sq, Sk, D, _mask_mode(causal), float(scale))
    if rc != 0:
        raise ValueError(f"attn_oracle_fwd failed with status {rc}")
    return o, lse


def attn_probs(q, k, causal: bool, scale: float, b: int, h: int):
    """Dense softmax probabilities [Sq, Sk] of one head (masked entries are 0)."""
    q, k = _f64(q), _f64(k)
    B, Hq, Hkv, Sq, Sk, D = _dims(q, k)
    p = np.empty((Sq, Sk), dtype=np.float64)
    rc = _load().attn_oracle_probs(_ptr(q), _ptr(k), _ptr(p), B, Hq, Hkv, Sq, Sk, D,
                                   _mask_mode(causal), float(scale), int(b), int(h))
    if rc != 0:
        raise ValueError(f"attn_oracle_probs failed with status {rc}")
    return p


def attn_bwd(q, k, v, d_o, causal: bool, scale: float, return_delta: bool = False):
    """dQ, dK, dV in fp64 (plus Delta = rowsum(dO * O) on request)."""
    q, k, v, d_o = _f64(q), _f64(k), _f64(v), _f64(d_o)
    B, Hq, Hkv, Sq, Sk, D = _dims(q, k)
    if v.shape != k.shape or d_o.shape != q.shape:
        raise ValueError("shape mismatch")
    dq = np.empty_like(q)
    dk = np.empty_like(k)
    dv = np.empty_like(v)
    delta = np.empty((B, Hq, Sq), dtype=np.float64)
    rc = _load().attn_oracle_bwd(_ptr(q), _ptr(k), _ptr(v), _ptr(d_o),
                                 _ptr(dq), _ptr(dk), _ptr(dv), _ptr(delta),
                                 B, Hq, Hkv, Sq, Sk, D, _mask_mode(causal), float(scale))
    if rc != 0:
        raise ValueError(f"attn_oracle_bwd failed with status {rc}")
    if return_delta:
        return dq, dk, dv, delta
    return dq, dk, dv


# --------------------------------------------------------------------------------------------
# Variable-length (packed) batches.  Not a new definition: sequence i owns the token rows
# [cu[i], cu[i+1]) of the packed tensors and is attended on its own with the formulas above,
# causal masking aligned (top-left or bottom-right, as `causal` says) inside the sequence.  Packed layouts: q, o, dO, dQ
# [total_q, Hq, D]; k, v, dK, dV [total_k, Hkv, D]; LSE [Hq, total_q].  A sequence with no keys
# has an empty softmax: its O rows are 0 and its LSE is -inf (and all its gradients are 0).
# --------------------------------------------------------------------------------------------
def _seq_slices(cu):
    cu = np.asarray(cu, dtype=np.int64)
    if cu.ndim != 1 or cu.size < 1 or cu[0] != 0 or np.any(np.diff(cu) < 0):
        raise ValueError("cu_seqlens must start at 0 and be non-decreasing")
    return [(int(cu[i]), int(cu[i + 1])) for i in range(cu.size - 1)]


def attn_fwd_varlen(q, k, v, cu_q, cu_k, causal: bool, scale: float):
    """Packed forward: returns O [total_q, Hq, D] and LSE [Hq, total_q] in fp64."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    sq, sk = _seq_slices(cu_q), _seq_slices(cu_k)
    if len(sq) != len(sk) or sq[-1][1] != q.shape[0] or sk[-1][1] != k.shape[0]:
        raise ValueError("cu_seqlens do not match the packed tensors")
    o = np.zeros_like(q)
    lse = np.full((q.shape[1], q.shape[0]), -np.inf)
    for (a, b), (c, d) in zip(sq, sk):
        if b == a or d == c:
            continue
        oi, li = attn_fwd(q[a:b].transpose(1, 0, 2)[None], k[c:d].transpose(1, 0, 2)[None],
                          v[c:d].transpose(1, 0, 2)[None], causal, scale)
        o[a:b] = oi[0].transpose(1, 0, 2)
        lse[:, a:b] = li[0]
    return o, lse


def attn_bwd_varlen(q, k, v, d_o, cu_q, cu_k, causal: bool, scale: float):
    """Packed backward: dQ [total_q, Hq, D], dK and dV [total_k, Hkv, D] in fp64."""
    q, k, v, d_o = _f64(q), _f64(k), _f64(v), _f64(d_o)
    sq, sk = _seq_slices(cu_q), _seq_slices(cu_k)
    if len(sq) != len(sk) or sq[-1][1] != q.shape[0] or sk[-1][1] != k.shape[0]:
        raise ValueError("cu_seqlens do not match the packed tensors")
    dq, dk, dv = np.zeros_like(q), np.zeros_like(k), np.zeros_like(v)
    for (a, b), (c, d) in zip(sq, sk):
        if b == a or d == c:
            continue
        gq, gk, gv = attn_bwd(q[a:b].transpose(1, 0, 2)[None], k[c:d].transpose(1, 0, 2)[None],
                              v[c:d].transpose(1, 0, 2)[None], d_o[a:b].transpose(1, 0, 2)[None], causal, scale)
        dq[a:b] = gq[0].transpose(1, 0, 2)
        dk[c:d] = gk[0].transpose(1, 0, 2)
        dv[c:d] = gv[0].transpose(1, 0, 2)
    return dq, dk, dv
