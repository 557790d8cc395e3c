"""ctypes binding over the C-ABI declared in include/tlin.h.

Argument marshalling only: every function takes torch tensors (device memory, streams) and hands
raw pointers and sizes to libtlin.so.  No attention arithmetic happens here and there is no
fallback: if the shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtlin.so")

TLIN_OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_ARCH = -1, -2, -3, -4, -5, -6


class TlinError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


class FwdPlan(ctypes.Structure):
    _fields_ = [("tile_m", ctypes.c_int32), ("tile_n", ctypes.c_int32), ("q_tiles", ctypes.c_int32),
                ("key_tiles", ctypes.c_int32), ("n_groups", ctypes.c_int32), ("n_ctas", ctypes.c_int32),
                ("total_units", ctypes.c_int64), ("uses_workspace", ctypes.c_int32),
                ("tensor_path", ctypes.c_int32), ("workspace_bytes", ctypes.c_int64),
                ("schedule", ctypes.c_int32), ("causal_window", ctypes.c_int32),
                ("n_keys", ctypes.c_int32), ("n_queries", ctypes.c_int32)]


class Problem(ctypes.Structure):
    _fields_ = [("q", ctypes.c_void_p), ("k", ctypes.c_void_p), ("v", ctypes.c_void_p), ("out", ctypes.c_void_p),
                ("lse", ctypes.c_void_p), ("BH", ctypes.c_int32), ("n_keys", ctypes.c_int32), ("kv_rows", ctypes.c_int32),
                ("n_queries", ctypes.c_int32), ("causal_window", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class DecodeProblem(ctypes.Structure):
    _fields_ = [("q_new", ctypes.c_void_p), ("k_new", ctypes.c_void_p), ("v_new", ctypes.c_void_p), ("k_cache", ctypes.c_void_p),
                ("v_cache", ctypes.c_void_p), ("out", ctypes.c_void_p), ("lse", ctypes.c_void_p), ("BH", ctypes.c_int32),
                ("Ncap", ctypes.c_int32), ("pos", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class DecodePlan(ctypes.Structure):
    _fields_ = [("splits", ctypes.c_int32), ("keys_per_split", ctypes.c_int32), ("n_ctas", ctypes.c_int32),
                ("workspace_bytes", ctypes.c_int64)]


_vp, _i, _i64, _sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_size_t

# name -> (restype, argtypes); mirrors include/tlin.h one to one
SIGNATURES = {
    "tlin_attn_forward": (_i, [_vp] * 5 + [_i] * 6 + [_vp]),
    "tlin_attn_forward_f32": (_i, [_vp] * 5 + [_i] * 6 + [_vp]),
    "tlin_attn_forward_prefixes": (_i, [_vp] * 5 + [_i] * 6 + [_vp, _i, _vp]),
    "tlin_attn_forward_host": (_i, [_vp] * 10 + [_i] * 6 + [_vp]),
    "tlin_attn_forward_batched": (_i, [_vp, _i, _i, _vp]),
    "tlin_plan_batched": (_i, [_vp, _i, _i, _vp, _vp]),
    "tlin_attn_forward_cache": (_i, [_vp] * 5 + [_i] * 7 + [_vp]),
    "tlin_attn_backward": (_i, [_vp] * 9 + [_i] * 6 + [_vp]),
    "tlin_attn_backward_f32": (_i, [_vp] * 9 + [_i] * 6 + [_vp]),
    "tlin_decode_step": (_i, [_vp] * 7 + [_i] * 5 + [_vp]),
    "tlin_decode_step_host": (_i, [_vp] * 12 + [_i] * 5 + [_vp]),
    "tlin_decode_step_batched": (_i, [_vp, _i, _i, _vp]),
    "tlin_decode_step_static": (_i, [_vp] * 7 + [_i] * 5 + [_vp]),
    "tlin_decode_step_ragged": (_i, [_vp] * 7 + [_i] * 3 + [_vp, _i, _i, _vp]),
    "tlin_decode_step_fp8": (_i, [_vp] * 9 + [_i] * 5 + [_vp]),
    "tlin_merge_lse": (_i, [_vp] * 6 + [_i64, _i, _vp]),
    "tlin_merge_lse_f32": (_i, [_vp] * 6 + [_i64, _i, _vp]),
    "tlin_workspace_bytes_forward": (_sz, [_i] * 6),
    "tlin_workspace_bytes_decode": (_sz, [_i] * 4),
    "tlin_workspace_bytes_forward_prefixes": (_sz, [_i] * 5 + [_vp, _i]),
    "tlin_workspace_bytes_backward": (_sz, [_i] * 5),
    "tlin_set_workspace": (_i, [_vp, _sz]),
    "tlin_plan_forward": (_i, [_i] * 8 + [ctypes.POINTER(FwdPlan)]),
    "tlin_plan_decode": (_i, [_i] * 5 + [ctypes.POINTER(DecodePlan)]),
    "tlin_plan_group_start": (_i64, [ctypes.POINTER(FwdPlan), _i]),
    "tlin_plan_backward_share_start": (_i64, [_i] * 7),
    "tlin_allowed": (_i, [_i64] * 4 + [_i]),
    "tlin_tile_class": (_i, [_i64, _i64, _i, _i, _i, _i, _i]),
    "tlin_get_status": (_i, [_vp]),
    "tlin_debug_wait_expires": (_i, [ctypes.c_longlong, _vp, _vp]),
    "tlin_status_string": (ctypes.c_char_p, [_i]),
    "tlin_version": (ctypes.c_char_p, []),
    "tlin_set_forward_impl": (_i, [_i]),
    "tlin_set_backward_impl": (_i, [_i]),
    "tlin_backward_arrangement": (_i, [_i, _i, _i, _i, _i]),
    "tlin_last_launch_count": (_i, []),
}

_lib = None
_workspace_tensor = None  # keeps the registered workspace alive


def lib():
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2508_20407_b200.build` "
                               "(there is no CPU fallback)")
        l = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(l, name)
            fn.restype, fn.argtypes = res, args
        _lib = l
    return _lib


def status_string(status: int) -> str:
    return lib().tlin_status_string(status).decode()


def version() -> str:
    return lib().tlin_version().decode()


def _check(rc: int, where: str):
    if rc != TLIN_OK:
        raise TlinError(rc, where)


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _dev(t, dtype, shape, name):
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype or tuple(t.shape) != tuple(shape) or not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous {dtype} of shape {tuple(shape)}, got {t.dtype} {tuple(t.shape)}")


# ------------------------------------------------------------------ workspace
def workspace_bytes_forward(B, H, N, W, d, causal_window) -> int:
    return int(lib().tlin_workspace_bytes_forward(B, H, N, W, d, int(causal_window)))


def workspace_bytes_decode(B, H, Ncap, d) -> int:
    return int(lib().tlin_workspace_bytes_decode(B, H, Ncap, d))


def workspace_bytes_backward(B, H, N, W, d) -> int:
    return int(lib().tlin_workspace_bytes_backward(B, H, N, W, d))


def set_workspace(t: torch.Tensor | None):
    """Registers a device buffer (any dtype) as split-K scratch; the tensor is kept alive here."""
    global _workspace_tensor
    if t is None:
        _check(lib().tlin_set_workspace(None, 0), "tlin_set_workspace")
    else:
        if not t.is_cuda or not t.is_contiguous():
            raise ValueError("workspace must be a contiguous CUDA tensor")
        _check(lib().tlin_set_workspace(_ptr(t), t.numel() * t.element_size()), "tlin_set_workspace")
    _workspace_tensor = t


def ensure_workspace(nbytes: int, device="cuda"):
    """Grows the registered workspace to at least ``nbytes`` (allocation happens here, in torch)."""
    global _workspace_tensor
    cur = 0 if _workspace_tensor is None else _workspace_tensor.numel()
    if nbytes > cur or (_workspace_tensor is not None and str(_workspace_tensor.device) != str(torch.device(device)) and torch.device(device).index is not None):
        set_workspace(torch.empty(max(nbytes, 1 << 20), dtype=torch.uint8, device=device))
    return _workspace_tensor


# ------------------------------------------------------------------ compute
def tlin_attn_forward(q, k, v, out=None, lse=None, causal_window=1, stream=None):
    """bf16 forward.  q [B,H,W,d], k,v [B,H,N,d] -> (out [B,H,W,d] bf16, lse [B,H,W] fp32)."""
    B, H, W, d = q.shape
    N = k.shape[2]
    _dev(q, torch.bfloat16, (B, H, W, d), "q")
    _dev(k, torch.bfloat16, (B, H, N, d), "k")
    _dev(v, torch.bfloat16, (B, H, N, d), "v")
    if out is None:
        out = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((B, H, W), dtype=torch.float32, device=q.device)
    _dev(out, torch.bfloat16, (B, H, W, d), "out")
    _dev(lse, torch.float32, (B, H, W), "lse")
    ensure_workspace(workspace_bytes_forward(B, H, N, W, d, causal_window), q.device)
    _check(lib().tlin_attn_forward(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(lse), B, H, N, W, d,
                                   int(causal_window), _stream(stream)), "tlin_attn_forward")
    return out, lse


def tlin_attn_forward_prefixes(q, k, v, n_keys, out=None, lse=None, causal_window=1, stream=None):
    """Chunk-scheduled forward: q [C,B,H,W,d], shared k,v [B,H,L,d], chunk c uses the first n_keys[c] key rows.

    Returns (out [C,B,H,W,d] bf16, lse [C,B,H,W] fp32)."""
    C, B, H, W, d = q.shape
    L = k.shape[2]
    n_keys = [int(x) for x in n_keys]
    if len(n_keys) != C:
        raise ValueError("one key count per chunk")
    _dev(q, torch.bfloat16, (C, B, H, W, d), "q")
    _dev(k, torch.bfloat16, (B, H, L, d), "k")
    _dev(v, torch.bfloat16, (B, H, L, d), "v")
    if out is None:
        out = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((C, B, H, W), dtype=torch.float32, device=q.device)
    _dev(out, torch.bfloat16, (C, B, H, W, d), "out")
    _dev(lse, torch.float32, (C, B, H, W), "lse")
    arr = (ctypes.c_int32 * C)(*n_keys)
    ensure_workspace(int(lib().tlin_workspace_bytes_forward_prefixes(B, H, W, d, C, arr, int(causal_window))), q.device)
    _check(lib().tlin_attn_forward_prefixes(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(lse), B, H, L, W, d, C, arr,
                                            int(causal_window), _stream(stream)), "tlin_attn_forward_prefixes")
    return out, lse


def tlin_attn_forward_cache(q, k_cache, v_cache, n_keys, out=None, lse=None, causal_window=1, stream=None):
    """Cache-miss forward over the first ``n_keys`` rows of decode caches [B,H,Ncap,d], in place."""
    B, H, W, d = q.shape
    Ncap = k_cache.shape[2]
    _dev(q, torch.bfloat16, (B, H, W, d), "q")
    _dev(k_cache, torch.bfloat16, (B, H, Ncap, d), "k_cache")
    _dev(v_cache, torch.bfloat16, (B, H, Ncap, d), "v_cache")
    if out is None:
        out = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((B, H, W), dtype=torch.float32, device=q.device)
    _dev(out, torch.bfloat16, (B, H, W, d), "out")
    _dev(lse, torch.float32, (B, H, W), "lse")
    ensure_workspace(workspace_bytes_forward(B, H, int(n_keys), W, d, causal_window), q.device)
    _check(lib().tlin_attn_forward_cache(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(out), _ptr(lse), B, H, Ncap, int(n_keys),
                                         W, d, int(causal_window), _stream(stream)), "tlin_attn_forward_cache")
    return out, lse


def make_problem_table(problems):
    """ctypes array of Problem from dicts/tuples (q, k, v, out, lse, n_keys, causal_window): q [B,H,W,d] (or [BH,W,d]),
    k, v [B,H,rows,d] with rows >= n_keys (n_keys None: all rows)."""
    arr = (Problem * len(problems))()
    keep = []
    for i, (q, k, v, out, lse, n_keys, causal) in enumerate(problems):
        d = q.shape[-1]
        W = q.shape[-2]
        bh = q.numel() // (W * d)
        rows = k.shape[-2]
        n_keys = rows if n_keys is None else int(n_keys)
        for t, name in ((q, "q"), (k, "k"), (v, "v"), (out, "out")):
            if not t.is_cuda or t.dtype != torch.bfloat16 or not t.is_contiguous():
                raise ValueError(f"problem {i}: {name} must be a contiguous bf16 CUDA tensor")
        if k.numel() != bh * rows * d or v.shape != k.shape or out.shape != q.shape:
            raise ValueError(f"problem {i}: shape mismatch")
        if lse is not None and (lse.dtype != torch.float32 or lse.numel() != bh * W or not lse.is_contiguous()):
            raise ValueError(f"problem {i}: lse must be contiguous fp32 of {bh * W} elements")
        arr[i] = Problem(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), None if lse is None else lse.data_ptr(),
                         bh, n_keys, rows if rows != n_keys else 0, W, int(causal), 0)
        keep.append((q, k, v, out, lse))
    return arr, keep


def tlin_attn_forward_batched(problems, stream=None):
    """One launch for a list of problems (q, k, v, out, lse, n_keys, causal_window) sharing one head size."""
    arr, _keep = make_problem_table(problems)
    d = problems[0][0].shape[-1]
    _check(lib().tlin_attn_forward_batched(ctypes.cast(arr, ctypes.c_void_p), len(problems), d, _stream(stream)), "tlin_attn_forward_batched")


def tlin_plan_batched(problem_array, num_sms=0):
    """(starts list of n_ctas + 1 entries) for a ctypes Problem array."""
    starts = (ctypes.c_int64 * 200)()
    n = ctypes.c_int32(0)
    _check(lib().tlin_plan_batched(ctypes.cast(problem_array, ctypes.c_void_p), len(problem_array), num_sms,
                                   ctypes.cast(starts, ctypes.c_void_p), ctypes.cast(ctypes.pointer(n), ctypes.c_void_p)), "tlin_plan_batched")
    return [int(starts[i]) for i in range(n.value + 1)]


def tlin_attn_forward_f32(q, k, v, out=None, lse=None, causal_window=1, stream=None):
    """fp32 forward (CUDA-core kernel)."""
    B, H, W, d = q.shape
    N = k.shape[2]
    _dev(q, torch.float32, (B, H, W, d), "q")
    _dev(k, torch.float32, (B, H, N, d), "k")
    _dev(v, torch.float32, (B, H, N, d), "v")
    if out is None:
        out = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((B, H, W), dtype=torch.float32, device=q.device)
    _dev(out, torch.float32, (B, H, W, d), "out")
    _dev(lse, torch.float32, (B, H, W), "lse")
    _check(lib().tlin_attn_forward_f32(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(lse), B, H, N, W, d,
                                       int(causal_window), _stream(stream)), "tlin_attn_forward_f32")
    return out, lse


def _backward(fn_name, dtype, q, k, v, out, lse, dout, dq, dk, dv, causal_window, stream):
    B, H, W, d = q.shape
    N = k.shape[2]
    for t, shape, name in ((q, (B, H, W, d), "q"), (k, (B, H, N, d), "k"), (v, (B, H, N, d), "v"),
                           (out, (B, H, W, d), "out"), (dout, (B, H, W, d), "dout")):
        _dev(t, dtype, shape, name)
    _dev(lse, torch.float32, (B, H, W), "lse")
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(k) if dk is None else dk
    dv = torch.empty_like(v) if dv is None else dv
    _dev(dq, dtype, (B, H, W, d), "dq")
    _dev(dk, dtype, (B, H, N, d), "dk")
    _dev(dv, dtype, (B, H, N, d), "dv")
    ensure_workspace(workspace_bytes_backward(B, H, N, W, d), q.device)
    _check(getattr(lib(), fn_name)(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(lse), _ptr(dout), _ptr(dq), _ptr(dk),
                                   _ptr(dv), B, H, N, W, d, int(causal_window), _stream(stream)), fn_name)
    return dq, dk, dv


def tlin_attn_backward(q, k, v, out, lse, dout, dq=None, dk=None, dv=None, causal_window=1, stream=None):
    """bf16 backward of ``tlin_attn_forward``: (dq [B,H,W,d], dk, dv [B,H,N,d]) for the loss gradient ``dout``.

    ``out`` and ``lse`` are the forward's results for the same q, k, v and causal_window."""
    return _backward("tlin_attn_backward", torch.bfloat16, q, k, v, out, lse, dout, dq, dk, dv, causal_window, stream)


def tlin_attn_backward_f32(q, k, v, out, lse, dout, dq=None, dk=None, dv=None, causal_window=1, stream=None):
    """fp32 backward of ``tlin_attn_forward_f32`` (CUDA-core kernels)."""
    return _backward("tlin_attn_backward_f32", torch.float32, q, k, v, out, lse, dout, dq, dk, dv, causal_window, stream)


def tlin_attn_forward_host(q_h, k_h, v_h, out_h, lse_h, q_d, k_d, v_d, out_d, lse_d, causal_window=1, stream=None):
    """Forward with HOST (pinned) q/k/v/out/lse and caller-supplied device staging tensors."""
    B, H, W, d = q_d.shape
    N = k_d.shape[2]
    for t, n in ((q_h, "q_h"), (k_h, "k_h"), (v_h, "v_h"), (out_h, "out_h"), (lse_h, "lse_h")):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError(f"{n} must be a contiguous host tensor")
    ensure_workspace(workspace_bytes_forward(B, H, N, W, d, causal_window), q_d.device)
    _check(lib().tlin_attn_forward_host(_ptr(q_h), _ptr(k_h), _ptr(v_h), _ptr(out_h), _ptr(lse_h),
                                        _ptr(q_d), _ptr(k_d), _ptr(v_d), _ptr(out_d), _ptr(lse_d),
                                        B, H, N, W, d, int(causal_window), _stream(stream)), "tlin_attn_forward_host")
    return out_h, lse_h


def tlin_decode_step(q_new, k_new, v_new, k_cache, v_cache, pos, out=None, lse=None, stream=None):
    """One cached decode step: appends k_new/v_new at row pos, attends q_new over rows [0,pos]."""
    B, H, Ncap, d = k_cache.shape
    for t, n in ((q_new, "q_new"), (k_new, "k_new"), (v_new, "v_new")):
        _dev(t, torch.bfloat16, (B, H, 1, d), n)
    _dev(k_cache, torch.bfloat16, (B, H, Ncap, d), "k_cache")
    _dev(v_cache, torch.bfloat16, (B, H, Ncap, d), "v_cache")
    if out is None:
        out = torch.empty_like(q_new)
    if lse is None:
        lse = torch.empty((B, H), dtype=torch.float32, device=q_new.device)
    ensure_workspace(workspace_bytes_decode(B, H, Ncap, d), q_new.device)
    _check(lib().tlin_decode_step(_ptr(q_new), _ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache),
                                  _ptr(out), _ptr(lse), B, H, Ncap, int(pos), d, _stream(stream)), "tlin_decode_step")
    return out, lse


def tlin_decode_step_fp8(q_new, k_new, v_new, k_cache, v_cache, k_scale, v_scale, pos, out=None, lse=None, stream=None):
    """Decode step over an 8-bit cache: k_cache, v_cache are uint8 [B,H,Ncap,d] (E4M3 codes), value = code * scale[b,h];
    k_scale, v_scale fp32 device tensors [B,H]."""
    B, H, Ncap, d = k_cache.shape
    for t, n in ((q_new, "q_new"), (k_new, "k_new"), (v_new, "v_new")):
        _dev(t, torch.bfloat16, (B, H, 1, d), n)
    _dev(k_cache, torch.uint8, (B, H, Ncap, d), "k_cache")
    _dev(v_cache, torch.uint8, (B, H, Ncap, d), "v_cache")
    _dev(k_scale, torch.float32, (B, H), "k_scale")
    _dev(v_scale, torch.float32, (B, H), "v_scale")
    if out is None:
        out = torch.empty_like(q_new)
    if lse is None:
        lse = torch.empty((B, H), dtype=torch.float32, device=q_new.device)
    ensure_workspace(workspace_bytes_decode(B, H, Ncap, d), q_new.device)
    _check(lib().tlin_decode_step_fp8(_ptr(q_new), _ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache), _ptr(k_scale),
                                      _ptr(v_scale), _ptr(out), _ptr(lse), B, H, Ncap, int(pos), d, _stream(stream)),
           "tlin_decode_step_fp8")
    return out, lse


def tlin_decode_step_ragged(q_new, k_new, v_new, k_cache, v_cache, pos, max_pos, out=None, lse=None, stream=None):
    """Decode step with one cache length per sequence: ``pos`` is an int32 device tensor of shape [B],
    ``max_pos`` a host-side upper bound of its entries."""
    B, H, Ncap, d = k_cache.shape
    for t, n in ((q_new, "q_new"), (k_new, "k_new"), (v_new, "v_new")):
        _dev(t, torch.bfloat16, (B, H, 1, d), n)
    _dev(k_cache, torch.bfloat16, (B, H, Ncap, d), "k_cache")
    _dev(v_cache, torch.bfloat16, (B, H, Ncap, d), "v_cache")
    _dev(pos, torch.int32, (B,), "pos")
    if out is None:
        out = torch.empty_like(q_new)
    if lse is None:
        lse = torch.empty((B, H), dtype=torch.float32, device=q_new.device)
    ensure_workspace(workspace_bytes_decode(B, H, Ncap, d), q_new.device)
    _check(lib().tlin_decode_step_ragged(_ptr(q_new), _ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache),
                                         _ptr(out), _ptr(lse), B, H, Ncap, _ptr(pos), int(max_pos), d, _stream(stream)),
           "tlin_decode_step_ragged")
    return out, lse


def tlin_decode_step_batched(problems, stream=None):
    """One launch for a list of decode problems (q_new, k_new or None, v_new or None, k_cache, v_cache, pos, out, lse)."""
    arr = (DecodeProblem * len(problems))()
    for i, (q_new, k_new, v_new, k_cache, v_cache, pos, out, lse) in enumerate(problems):
        d = k_cache.shape[-1]
        Ncap = k_cache.shape[-2]
        bh = k_cache.numel() // (Ncap * d)
        for t, name in ((q_new, "q_new"), (out, "out")) + (((k_new, "k_new"), (v_new, "v_new")) if k_new is not None else ()):
            if not t.is_cuda or t.dtype != torch.bfloat16 or not t.is_contiguous() or t.numel() != bh * d:
                raise ValueError(f"problem {i}: {name} must be contiguous bf16 [BH,1,d]")
        for t, name in ((k_cache, "k_cache"), (v_cache, "v_cache")):
            if not t.is_cuda or t.dtype != torch.bfloat16 or not t.is_contiguous() or t.numel() != bh * Ncap * d:
                raise ValueError(f"problem {i}: {name} must be contiguous bf16 [BH,Ncap,d]")
        if lse is not None and (lse.dtype != torch.float32 or lse.numel() != bh or not lse.is_contiguous()):
            raise ValueError(f"problem {i}: lse must be contiguous fp32 [BH]")
        arr[i] = DecodeProblem(q_new.data_ptr(), None if k_new is None else k_new.data_ptr(), None if v_new is None else v_new.data_ptr(),
                               k_cache.data_ptr(), v_cache.data_ptr(), out.data_ptr(), None if lse is None else lse.data_ptr(),
                               bh, Ncap, int(pos), 0)
    d = problems[0][3].shape[-1]
    _check(lib().tlin_decode_step_batched(ctypes.cast(arr, ctypes.c_void_p), len(problems), d, _stream(stream)), "tlin_decode_step_batched")


def tlin_decode_step_static(q_new, k_new, v_new, k_cache, v_cache, pos, out, lse, stream=None):
    """tlin_decode_step without any allocation: scratch is the library's built-in array, and ``out``
    ([B,H,1,d] bf16) and ``lse`` ([B,H] fp32) must be supplied by the caller."""
    B, H, Ncap, d = k_cache.shape
    for t, n in ((q_new, "q_new"), (k_new, "k_new"), (v_new, "v_new"), (out, "out")):
        _dev(t, torch.bfloat16, (B, H, 1, d), n)
    _dev(lse, torch.float32, (B, H), "lse")
    _check(lib().tlin_decode_step_static(_ptr(q_new), _ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache),
                                         _ptr(out), _ptr(lse), B, H, Ncap, int(pos), d, _stream(stream)),
           "tlin_decode_step_static")
    return out, lse


def tlin_decode_step_host(q_new_h, k_new_h, v_new_h, out_h, lse_h, q_new_d, k_new_d, v_new_d, out_d, lse_d,
                          k_cache, v_cache, pos, stream=None):
    B, H, Ncap, d = k_cache.shape
    ensure_workspace(workspace_bytes_decode(B, H, Ncap, d), k_cache.device)
    _check(lib().tlin_decode_step_host(_ptr(q_new_h), _ptr(k_new_h), _ptr(v_new_h), _ptr(out_h), _ptr(lse_h),
                                       _ptr(q_new_d), _ptr(k_new_d), _ptr(v_new_d), _ptr(out_d), _ptr(lse_d),
                                       _ptr(k_cache), _ptr(v_cache), B, H, Ncap, int(pos), d, _stream(stream)),
           "tlin_decode_step_host")
    return out_h, lse_h


def tlin_merge_lse(out_a, lse_a, out_b, lse_b, out=None, lse=None, stream=None):
    """Exact merge of two results over disjoint key sets (bf16 or fp32 outputs, fp32 lse)."""
    d = out_a.shape[-1]
    rows = out_a.numel() // d
    if out is None:
        out = torch.empty_like(out_a)
    if lse is None:
        lse = torch.empty_like(lse_a)
    fn = lib().tlin_merge_lse_f32 if out_a.dtype == torch.float32 else lib().tlin_merge_lse
    _check(fn(_ptr(out_a), _ptr(lse_a), _ptr(out_b), _ptr(lse_b), _ptr(out), _ptr(lse), rows, d, _stream(stream)),
           "tlin_merge_lse")
    return out, lse


# ------------------------------------------------------------------ host logic
def tlin_plan_forward(B, H, N, W, d, causal_window, is_f32=False, num_sms=0) -> FwdPlan:
    p = FwdPlan()
    _check(lib().tlin_plan_forward(B, H, N, W, d, int(causal_window), int(is_f32), num_sms, ctypes.byref(p)), "tlin_plan_forward")
    return p


def tlin_plan_decode(B, H, L, d, num_sms=0) -> DecodePlan:
    p = DecodePlan()
    _check(lib().tlin_plan_decode(B, H, L, d, num_sms, ctypes.byref(p)), "tlin_plan_decode")
    return p


def tlin_plan_group_start(plan: FwdPlan, g: int) -> int:
    return int(lib().tlin_plan_group_start(ctypes.byref(plan), g))


def tlin_allowed(i, j, N, W, causal_window) -> int:
    return int(lib().tlin_allowed(i, j, N, W, int(causal_window)))


def tlin_tile_class(N, W, causal_window, tile_m, tile_n, qt, kt) -> int:
    return int(lib().tlin_tile_class(N, W, int(causal_window), tile_m, tile_n, qt, kt))


def tlin_get_status(stream=None) -> int:
    return int(lib().tlin_get_status(_stream(stream)))


def tlin_debug_wait_expires(limit_cycles: int, waited=None, stream=None) -> None:
    """Launches the diagnostic kernel whose bounded wait runs out; ``waited`` is an optional int64 device tensor."""
    _check(lib().tlin_debug_wait_expires(int(limit_cycles), _ptr(waited), _stream(stream)), "tlin_debug_wait_expires")


def tlin_set_forward_impl(impl: int) -> int:
    return int(lib().tlin_set_forward_impl(impl))


def tlin_set_backward_impl(impl: int) -> int:
    """0: the library chooses (one kernel while the fp32 dQ buffer is at most 64 MiB), 1: two kernels (dK/dV, then dQ;
    bitwise repeatable), 2: one kernel (d = 128; dQ summed by reductions in L2, repeatable up to the order of fp32
    additions).  Returns the previous setting."""
    return int(lib().tlin_set_backward_impl(int(impl)))


def tlin_backward_arrangement(B, H, N, W, d) -> int:
    """1 (two kernels) or 2 (one kernel): what a bf16 backward call of these sizes gets under the current setting."""
    return int(lib().tlin_backward_arrangement(B, H, N, W, d))


def tlin_last_launch_count() -> int:
    return int(lib().tlin_last_launch_count())


# ------------------------------------------------------------------ autograd glue (marshalling only)
class _AttentionFunction(torch.autograd.Function):
    """Lets PyTorch's autograd call the library's forward and backward entry points; nothing is computed here."""

    @staticmethod
    def forward(ctx, q, k, v, causal_window):
        f32 = q.dtype == torch.float32
        q, k, v = q.contiguous(), k.contiguous(), v.contiguous()
        out, lse = (tlin_attn_forward_f32 if f32 else tlin_attn_forward)(q, k, v, causal_window=causal_window)
        ctx.save_for_backward(q, k, v, out, lse)
        ctx.causal_window = int(causal_window)
        ctx.f32 = f32
        ctx.mark_non_differentiable(lse)
        return out, lse

    @staticmethod
    def backward(ctx, dout, _dlse):
        q, k, v, out, lse = ctx.saved_tensors
        fn = tlin_attn_backward_f32 if ctx.f32 else tlin_attn_backward
        dq, dk, dv = fn(q, k, v, out, lse, dout.contiguous(), causal_window=ctx.causal_window)
        return dq, dk, dv, None


def attention(q, k, v, causal_window=1):
    """Differentiable attention for PyTorch training code: (out, lse) = tlin_attn_forward(q, k, v); gradients of `out`
    with respect to q, k, v come from tlin_attn_backward (lse is returned for merging and is not differentiable).
    bf16 or fp32 tensors, shapes as in tlin_attn_forward."""
    return _AttentionFunction.apply(q, k, v, causal_window)
