"""Seeded synthetic inputs for the TLinFormer attention hot path.

This module only manufactures input tensors.  It holds none of the method's
arithmetic (no scores, softmax, masks or merges) and is the one piece of code
that both the CPU oracle's tests and the CUDA path's tests may share.

Values are drawn from a counter-based generator: element ``i`` of tensor
``tensor_id`` under ``seed`` is ``BoxMuller(splitmix64(key, 2i), splitmix64(key,
2i+1))`` evaluated in float64 and rounded to the requested dtype.  Because the
value depends only on (seed, tensor_id, flat index) the same tensor can be made
in chunks, on the host or on a GPU.  Whenever a CPU oracle is compared with a
GPU result the oracle is handed a host copy of the exact bits the kernel read,
so an ulp-level difference between host and device ``log``/``cos`` can never
turn into a disagreement about the inputs.

The paper's own inference benchmark feeds random token tensors of shape (1, N)
(Section 6.3); these generators stand in for already-projected q/k/v of the same
shapes.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import torch

_M64 = (1 << 64) - 1


def _s64(x: int) -> int:
    """Two's-complement reinterpretation of an unsigned 64-bit constant."""
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


_GOLDEN = _s64(0x9E3779B97F4A7C15)
_MUL1 = _s64(0xBF58476D1CE4E5B9)
_MUL2 = _s64(0x94D049BB133111EB)


def _lshr(z: torch.Tensor, s: int) -> torch.Tensor:
    return (z >> s) & ((1 << (64 - s)) - 1)


def _splitmix64(x: torch.Tensor) -> torch.Tensor:
    """splitmix64 finaliser on an int64 tensor holding uint64 bit patterns."""
    z = x + _GOLDEN
    z = (z ^ _lshr(z, 30)) * _MUL1
    z = (z ^ _lshr(z, 27)) * _MUL2
    return z ^ _lshr(z, 31)


def _splitmix64_int(x: int) -> int:
    z = (x + 0x9E3779B97F4A7C15) & _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def stream_key(seed: int, tensor_id: int) -> int:
    """One 64-bit key per (seed, tensor_id) stream."""
    return _splitmix64_int(_splitmix64_int(seed & _M64) ^ ((tensor_id * 0xD6E8FEB86659FD93) & _M64))


def _uniform53(bits: torch.Tensor) -> torch.Tensor:
    """(0,1) float64 from the top 53 bits, never 0 or 1."""
    return (_lshr(bits, 11).to(torch.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal_flat(seed: int, tensor_id: int, start: int, count: int, device="cpu") -> torch.Tensor:
    """float64 N(0,1) values for flat indices [start, start+count) of one stream."""
    key = _s64(stream_key(seed, tensor_id))
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    c0 = _splitmix64((idx * 2) ^ key)
    c1 = _splitmix64((idx * 2 + 1) ^ key)
    u1 = _uniform53(c0)
    u2 = _uniform53(c1)
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)


def row_hash_mod(seed: int, tensor_id: int, start_row: int, rows: int, modulus: int, device="cpu") -> torch.Tensor:
    """splitmix64(key ^ row) mod modulus for rows [start_row, start_row+rows) (non-negative int64)."""
    key = _s64(stream_key(seed, tensor_id + 1000))
    idx = torch.arange(start_row, start_row + rows, dtype=torch.int64, device=device)
    h = _lshr(_splitmix64(idx ^ key), 1)  # 63 bits, non-negative
    return h % modulus


def normal_tensor(seed: int, tensor_id: int, shape, dtype=torch.bfloat16, device="cpu", scale: float = 1.0,
                  peaky_rows: tuple[int, float] | None = None, chunk_elems: int = 1 << 26) -> torch.Tensor:
    """Tensor of ``shape`` with entries ``scale * N(0,1)``, rounded to ``dtype``.

    ``peaky_rows=(modulus, factor)`` multiplies whole rows (last dim = one row) by
    ``factor`` when the row's hash is 0 mod ``modulus`` -- the recipe of the
    "1 % of key rows scaled x8" workload.  Generated chunk by chunk so that the
    float64 temporaries stay small next to the result.
    """
    shape = tuple(int(s) for s in shape)
    total = 1
    for s in shape:
        total *= s
    out = torch.empty(total, dtype=dtype, device=device)
    rowlen = shape[-1] if shape else 1
    chunk = max(rowlen, (chunk_elems // rowlen) * rowlen)
    for start in range(0, total, chunk):
        n = min(chunk, total - start)
        x = normal_flat(seed, tensor_id, start, n, device=device)
        if scale != 1.0:
            x = x * scale
        if peaky_rows is not None:
            modulus, factor = peaky_rows
            r0, nr = start // rowlen, n // rowlen
            hit = row_hash_mod(seed, tensor_id, r0, nr, modulus, device=device) == 0
            x = x.view(nr, rowlen) * torch.where(hit, float(factor), 1.0).to(torch.float64)[:, None]
            x = x.reshape(-1)
        out[start:start + n] = x.to(dtype)
    return out.view(shape)


@dataclass(frozen=True)
class Workload:
    """One of the benchmark/parity configurations (shapes follow [B,H,rows,d])."""
    name: str
    B: int
    H: int
    d: int
    N: int          # key/value rows (forward) or rows already cached before step 0 (decode)
    W: int          # query rows (forward) or number of decode steps
    seed: int
    causal_window: int = 1
    scale: float = 1.0
    peaky: tuple[int, float] | None = None
    decode: bool = False


def _w(name, B, H, d, N, W, seed, **kw):
    return Workload(name=name, B=B, H=H, d=d, N=N, W=W, seed=seed, **kw)


WORKLOADS = {
    # tiny forward, oracle-scale; q,k,v ~ N(0,1)/sqrt(d)
    "cfg1_tiny": _w("cfg1_tiny", 1, 4, 64, 1024, 128, 0, scale=1.0 / 8.0),
    # mid forward
    "cfg2_mid": _w("cfg2_mid", 4, 16, 64, 8192, 256, 1),
    # long forward, 1 % of key rows x8
    "cfg3_long": _w("cfg3_long", 1, 32, 128, 32768, 512, 2, peaky=(100, 8.0)),
    # very long forward
    "cfg4_vlong": _w("cfg4_vlong", 1, 32, 128, 131072, 1024, 3),
    # cached decode: 65536 cached rows + 256 single-token steps
    "cfg5_decode": _w("cfg5_decode", 8, 32, 128, 65536, 256, 4, decode=True),
    # --- the other attention layers of a block, at the sizes of the very long configuration (W_oh = W_og = 1024) ---
    # restoring cross-attention: every history token queries the W_oh summary tokens (unmasked)
    "restore_vlong": _w("restore_vlong", 1, 32, 128, 1024, 131072 - 1024, 5, causal_window=0),
    # inner context layer: self-attention among the W_oh summary tokens (unmasked)
    "inner_self": _w("inner_self", 1, 32, 128, 1024, 1024, 6, causal_window=0),
    # inner generation layer: W_og window queries over [summary tokens; window], causal inside the window
    "inner_gen": _w("inner_gen", 1, 32, 128, 2048, 1024, 7, causal_window=1),
    # --- training (forward + backward): the last of the 8 windows of a sliding-window pass (stride W_og = 1024) over
    # sequences of 8192 tokens: W_og window queries over the whole sequence so far, causal inside the window
    "train_chunk": _w("train_chunk", 4, 32, 128, 8192, 1024, 8, causal_window=1),
    # plain causal attention of a whole 4096-token sequence over itself (N = W): the layer of the standard architecture
    # the paper compares with, and the window rule at its widest (half of the rectangle is masked)
    "train_seq": _w("train_seq", 4, 32, 128, 4096, 4096, 10, causal_window=1),
}

Q_ID, K_ID, V_ID, QNEW_ID, KNEW_ID, VNEW_ID = 0, 1, 2, 3, 4, 5


def forward_inputs(wl: Workload, device="cpu", dtype=torch.bfloat16):
    """(q [B,H,W,d], k [B,H,N,d], v [B,H,N,d]) for a forward workload."""
    q = normal_tensor(wl.seed, Q_ID, (wl.B, wl.H, wl.W, wl.d), dtype, device, wl.scale)
    k = normal_tensor(wl.seed, K_ID, (wl.B, wl.H, wl.N, wl.d), dtype, device, wl.scale, peaky_rows=wl.peaky)
    v = normal_tensor(wl.seed, V_ID, (wl.B, wl.H, wl.N, wl.d), dtype, device, wl.scale)
    return q, k, v


def decode_inputs(wl: Workload, device="cpu", dtype=torch.bfloat16, steps: int | None = None):
    """Cache prefix and per-step tokens for a decode workload.

    Returns (k_cache, v_cache) of shape [B,H,Ncap,d] with the first N rows filled
    and the rest zero, Ncap = N + steps, and (q_new, k_new, v_new) of shape
    [steps,B,H,1,d].
    """
    steps = wl.W if steps is None else steps
    ncap = wl.N + steps
    k_cache = torch.zeros((wl.B, wl.H, ncap, wl.d), dtype=dtype, device=device)
    v_cache = torch.zeros((wl.B, wl.H, ncap, wl.d), dtype=dtype, device=device)
    # fill per (b,h) so that element counters do not depend on Ncap
    for b in range(wl.B):
        for h in range(wl.H):
            tid = 16 + 2 * (b * wl.H + h)
            k_cache[b, h, :wl.N] = normal_tensor(wl.seed, tid, (wl.N, wl.d), dtype, device, wl.scale)
            v_cache[b, h, :wl.N] = normal_tensor(wl.seed, tid + 1, (wl.N, wl.d), dtype, device, wl.scale)
    shp = (steps, wl.B, wl.H, 1, wl.d)
    q_new = normal_tensor(wl.seed, QNEW_ID, shp, dtype, device, wl.scale)
    k_new = normal_tensor(wl.seed, KNEW_ID, shp, dtype, device, wl.scale)
    v_new = normal_tensor(wl.seed, VNEW_ID, shp, dtype, device, wl.scale)
    return (k_cache, v_cache), (q_new, k_new, v_new)


def forward_inputs_head(wl: Workload, b: int, h: int, device="cpu", dtype=torch.bfloat16, q_rows: slice | None = None):
    """The (b,h) slice of ``forward_inputs(wl)``: (q [W',d], k [N,d], v [N,d]), made without the rest.

    Uses the same counters as the full tensors, so the values agree with a slice of them (up to the
    host/device libm note in the module docstring).
    """
    bh = b * wl.H + h
    r0, r1 = (0, wl.W) if q_rows is None else (q_rows.start or 0, wl.W if q_rows.stop is None else q_rows.stop)

    def rows(tid, first_row, n_rows, peaky):
        x = normal_flat(wl.seed, tid, first_row * wl.d, n_rows * wl.d, device=device)
        if wl.scale != 1.0:
            x = x * wl.scale
        if peaky is not None:
            hit = row_hash_mod(wl.seed, tid, first_row, n_rows, peaky[0], device=device) == 0
            x = (x.view(n_rows, wl.d) * torch.where(hit, float(peaky[1]), 1.0).to(torch.float64)[:, None]).reshape(-1)
        return x.to(dtype).view(n_rows, wl.d)

    q = rows(Q_ID, bh * wl.W + r0, r1 - r0, None)
    k = rows(K_ID, bh * wl.N, wl.N, wl.peaky)
    v = rows(V_ID, bh * wl.N, wl.N, None)
    return q, k, v
