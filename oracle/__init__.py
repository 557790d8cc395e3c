"""CPU oracle for the TLinFormer attention hot path -- TEST INFRASTRUCTURE ONLY.

Imported by ``tests/``, by ``__graft_entry__.smoke()`` and by the CPU-baseline /
reference legs of ``bench.py``.  The product package never imports it, and it
never imports the product package.  ``tlin_oracle.c`` is the implementation;
this file compiles it with gcc and marshals numpy / torch-CPU arrays to it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tlin_oracle.c")
_LIB = os.path.join(_HERE, "libtlin_oracle.so")
_lib = None

BF16, F32 = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP) if the shared object is stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
                               _SRC, "-o", _LIB, "-lm"])
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, dp, i32, i64 = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int64
        lib.tlin_ref_attn_forward.argtypes = [vp, vp, vp, i32, dp, dp, i32, i32, i64, i64, i32, i32]
        lib.tlin_ref_attn_backward.argtypes = [vp, vp, vp, vp, i32, dp, dp, dp, i32, i32, i64, i64, i32, i32]
        lib.tlin_ref_decode_step.argtypes = [vp, vp, vp, vp, vp, i32, dp, dp, i32, i32, i64, i64, i32]
        lib.tlin_ref_merge_lse.argtypes = [dp, dp, dp, dp, dp, dp, i64, i32]
        lib.tlin_ref_decode_step_fp8.argtypes = [vp, vp, vp, vp, vp, vp, vp, dp, dp, i32, i32, i64, i64, i32]
        lib.tlin_ref_e4m3_decode.argtypes = [ctypes.c_uint8]
        lib.tlin_ref_e4m3_decode.restype = ctypes.c_double
        lib.tlin_ref_e4m3_encode.argtypes = [ctypes.c_float]
        lib.tlin_ref_e4m3_encode.restype = ctypes.c_uint8
        lib.tlin_ref_allowed.argtypes = [i64, i64, i64, i64, i32]
        lib.tlin_ref_num_threads.argtypes = []
        _lib = lib
    return _lib


def _as_elems(x):
    """(contiguous numpy array of uint16 or float32, elem_type) from numpy or torch CPU input."""
    if hasattr(x, "detach"):  # torch tensor
        import torch
        x = x.detach()
        if x.device.type != "cpu":
            raise ValueError("the oracle takes host tensors")
        x = x.contiguous()
        if x.dtype == torch.bfloat16:
            return x.view(torch.int16).numpy().view(np.uint16), BF16
        if x.dtype == torch.float32:
            return x.numpy(), F32
        raise TypeError(f"unsupported dtype {x.dtype}")
    x = np.ascontiguousarray(x)
    if x.dtype == np.uint16:
        return x, BF16
    if x.dtype == np.float32:
        return x, F32
    raise TypeError(f"unsupported dtype {x.dtype}; pass bf16 bits as uint16 or float32")


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def num_threads() -> int:
    return int(_load().tlin_ref_num_threads())


def allowed(i: int, j: int, N: int, W: int, causal_window: int) -> bool:
    """Mask predicate: may query i (of W) use key j (of N)?"""
    return bool(_load().tlin_ref_allowed(i, j, N, W, int(causal_window)))


def attn_forward(q, k, v, causal_window: int):
    """q:[B,H,W,d], k,v:[B,H,N,d] (bf16 bits/torch bf16 or float32) -> (out f64 [B,H,W,d], lse f64 [B,H,W])."""
    qa, tq = _as_elems(q)
    ka, tk = _as_elems(k)
    va, tv = _as_elems(v)
    if not (tq == tk == tv):
        raise TypeError("q, k, v must share one element type")
    B, H, W, d = qa.shape
    Bk, Hk, N, dk = ka.shape
    if (Bk, Hk, dk) != (B, H, d) or va.shape != ka.shape:
        raise ValueError("shape mismatch")
    out = np.empty((B, H, W, d), dtype=np.float64)
    lse = np.empty((B, H, W), dtype=np.float64)
    rc = _load().tlin_ref_attn_forward(_ptr(qa), _ptr(ka), _ptr(va), tq, _ptr(out), _ptr(lse),
                                       B, H, N, W, d, int(causal_window))
    if rc != 0:
        raise ValueError(f"tlin_ref_attn_forward rejected its arguments (rc={rc})")
    return out, lse


def attn_backward(q, k, v, dout, causal_window: int):
    """Gradients of ``attn_forward`` for a loss with dL/dout = dout (and no dependence on lse).

    q,dout:[B,H,W,d], k,v:[B,H,N,d] (one element type) -> (dq [B,H,W,d], dk, dv [B,H,N,d]), all float64.
    """
    qa, tq = _as_elems(q)
    ka, tk = _as_elems(k)
    va, tv = _as_elems(v)
    da, td = _as_elems(dout)
    if not (tq == tk == tv == td):
        raise TypeError("q, k, v, dout must share one element type")
    B, H, W, d = qa.shape
    Bk, Hk, N, dk_ = ka.shape
    if (Bk, Hk, dk_) != (B, H, d) or va.shape != ka.shape or da.shape != qa.shape:
        raise ValueError("shape mismatch")
    dq = np.empty((B, H, W, d), dtype=np.float64)
    dk = np.empty((B, H, N, d), dtype=np.float64)
    dv = np.empty((B, H, N, d), dtype=np.float64)
    rc = _load().tlin_ref_attn_backward(_ptr(qa), _ptr(ka), _ptr(va), _ptr(da), tq, _ptr(dq), _ptr(dk), _ptr(dv),
                                        B, H, N, W, d, int(causal_window))
    if rc != 0:
        raise ValueError(f"tlin_ref_attn_backward rejected its arguments (rc={rc})")
    return dq, dk, dv


def decode_step(q_new, k_new, v_new, k_cache, v_cache, pos: int):
    """Append k_new,v_new at row ``pos`` of the caches (in place), attend q_new over rows [0,pos].

    k_cache, v_cache must be writable contiguous arrays ([B,H,Ncap,d]); torch CPU
    tensors are modified through their shared memory.  Returns (out f64 [B,H,1,d], lse f64 [B,H]).
    """
    qa, tq = _as_elems(q_new)
    kn, tk = _as_elems(k_new)
    vn, tv = _as_elems(v_new)
    kc, tkc = _as_elems(k_cache)
    vc, tvc = _as_elems(v_cache)
    if len({tq, tk, tv, tkc, tvc}) != 1:
        raise TypeError("all tensors must share one element type")
    B, H, Ncap, d = kc.shape
    for a in (qa, kn, vn):
        if a.shape != (B, H, 1, d):
            raise ValueError("new-token tensors must be [B,H,1,d]")
    if hasattr(k_cache, "detach"):
        if not k_cache.is_contiguous() or not v_cache.is_contiguous():
            raise ValueError("caches must be contiguous to be updated in place")
    out = np.empty((B, H, 1, d), dtype=np.float64)
    lse = np.empty((B, H), dtype=np.float64)
    rc = _load().tlin_ref_decode_step(_ptr(qa), _ptr(kn), _ptr(vn), _ptr(kc), _ptr(vc), tq,
                                      _ptr(out), _ptr(lse), B, H, Ncap, int(pos), d)
    if rc != 0:
        raise ValueError(f"tlin_ref_decode_step rejected its arguments (rc={rc})")
    return out, lse


def e4m3_decode(code: int) -> float:
    """Value of an E4M3 code (0..255); NaN for 0x7f and 0xff."""
    return float(_load().tlin_ref_e4m3_decode(int(code) & 0xFF))


def e4m3_encode(x: float) -> int:
    """Nearest finite E4M3 code of an fp32 value (ties to even, saturating at +-448)."""
    return int(_load().tlin_ref_e4m3_encode(float(np.float32(x))))


def decode_step_fp8(q_new, k_new, v_new, k_cache, v_cache, k_scale, v_scale, pos: int):
    """Cached decode step over an 8-bit (E4M3) cache; value = decode(code) * scale[b,h].

    q_new,k_new,v_new: bf16 [B,H,1,d]; k_cache,v_cache: uint8 [B,H,Ncap,d], updated in place at row ``pos``;
    k_scale,v_scale: float32 [B,H].  Returns (out f64 [B,H,1,d], lse f64 [B,H])."""
    qa, tq = _as_elems(q_new)
    kn, tk = _as_elems(k_new)
    vn, tv = _as_elems(v_new)
    if not (tq == tk == tv == BF16):
        raise TypeError("q_new, k_new, v_new must be bf16")

    def bytes_of(c):
        if hasattr(c, "detach"):
            if not c.is_contiguous():
                raise ValueError("caches must be contiguous to be updated in place")
            c = c.numpy()
        if c.dtype != np.uint8 or not c.flags["C_CONTIGUOUS"]:
            raise TypeError("caches are contiguous uint8 arrays")
        return c

    kc, vc = bytes_of(k_cache), bytes_of(v_cache)
    ks = np.ascontiguousarray(k_scale.numpy() if hasattr(k_scale, "detach") else k_scale, dtype=np.float32)
    vs = np.ascontiguousarray(v_scale.numpy() if hasattr(v_scale, "detach") else v_scale, dtype=np.float32)
    B, H, Ncap, d = kc.shape
    out = np.empty((B, H, 1, d), dtype=np.float64)
    lse = np.empty((B, H), dtype=np.float64)
    rc = _load().tlin_ref_decode_step_fp8(_ptr(qa), _ptr(kn), _ptr(vn), _ptr(kc), _ptr(vc), _ptr(ks), _ptr(vs),
                                          _ptr(out), _ptr(lse), B, H, Ncap, int(pos), d)
    if rc != 0:
        raise ValueError(f"tlin_ref_decode_step_fp8 rejected its arguments (rc={rc})")
    return out, lse


def merge_lse(out_a, lse_a, out_b, lse_b):
    """Exact merge of two partial attention results over disjoint key sets (all float64)."""
    oa = np.ascontiguousarray(out_a, dtype=np.float64)
    ob = np.ascontiguousarray(out_b, dtype=np.float64)
    la = np.ascontiguousarray(lse_a, dtype=np.float64)
    lb = np.ascontiguousarray(lse_b, dtype=np.float64)
    d = oa.shape[-1]
    rows = oa.size // d
    out = np.empty_like(oa)
    lse = np.empty_like(la)
    rc = _load().tlin_ref_merge_lse(_ptr(oa), _ptr(la), _ptr(ob), _ptr(lb), _ptr(out), _ptr(lse), rows, d)
    if rc != 0:
        raise ValueError("tlin_ref_merge_lse rejected its arguments")
    return out, lse
