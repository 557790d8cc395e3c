"""Pins for the CPU oracle: every expectation here comes from the paper's formula
worked by other means (explicit probability matrices, closed forms, invariants,
a textbook library routine, hand-derived fixtures), never from the oracle itself."""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from oracle import cost_model
from paper_2508_20407_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
rng = np.random.default_rng(1234)


def brute_force(q, k, v, causal_window):
    """Explicit-matrix attention, written independently of the oracle: returns (out, lse, P)."""
    q, k, v = (np.asarray(a, dtype=np.float64) for a in (q, k, v))
    B, H, W, d = q.shape
    N = k.shape[2]
    S = np.einsum("bhid,bhjd->bhij", q, k) / math.sqrt(d)
    if causal_window:
        i = np.arange(W)[:, None]
        j = np.arange(N)[None, :]
        S = np.where(j <= (N - W) + i, S, -np.inf)
    E = np.exp(S - S.max(axis=-1, keepdims=True))
    P = E / E.sum(axis=-1, keepdims=True)
    lse = np.log(np.exp(S).sum(axis=-1))
    return np.einsum("bhij,bhjd->bhid", P, v), lse, P


def rand(*shape):
    return rng.standard_normal(shape).astype(np.float32)


# ---------------------------------------------------------------- brute force / library
@pytest.mark.parametrize("B,H,N,W,d,causal", [
    (1, 1, 8, 4, 4, 1), (1, 1, 8, 4, 4, 0), (2, 3, 7, 7, 3, 1), (1, 2, 5, 1, 2, 1),
    (1, 1, 1, 1, 1, 1), (2, 2, 33, 9, 8, 1), (1, 2, 33, 40, 8, 0), (1, 1, 6, 6, 5, 0),
])
def test_brute_force_tiny(B, H, N, W, d, causal):
    q, k, v = rand(B, H, W, d), rand(B, H, N, d), rand(B, H, N, d)
    out, lse = oracle.attn_forward(q, k, v, causal)
    ref, ref_lse, P = brute_force(q, k, v, causal)
    assert np.abs(P.sum(-1) - 1).max() < 1e-14
    assert np.abs(out - ref).max() < 1e-13
    assert np.abs(lse - ref_lse).max() < 1e-13


def test_hand_derived_fixture():
    vals = {}
    consts = {"LN3": math.log(3.0), "LN4": math.log(4.0), "LN8": math.log(8.0)}
    for line in open(os.path.join(GOLDEN, "attention_two_keys.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        name, *nums = line.split()
        vals[name] = np.array([consts[x] if x in consts else float(x) for x in nums])
    q = vals["q"].astype(np.float32).reshape(1, 1, 1, 4)
    for nk, o_name, l_name in ((2, "out2", "lse2"), (3, "out3", "lse3")):
        k = np.stack([vals[f"k{j}"] for j in range(nk)]).astype(np.float32).reshape(1, 1, nk, 4)
        v = np.stack([vals[f"v{j}"] for j in range(nk)]).astype(np.float32).reshape(1, 1, nk, 4)
        out, lse = oracle.attn_forward(q, k, v, 0)
        assert np.abs(out.ravel() - vals[o_name]).max() < 2e-6
        assert abs(lse.item() - vals[l_name].item()) < 1e-6


def test_reduces_to_textbook_causal_when_history_empty():
    # First training chunk has an empty history (Section 5.1): N == W, plain causal attention.
    q, k, v = rand(2, 2, 17, 8), rand(2, 2, 17, 8), rand(2, 2, 17, 8)
    out, _ = oracle.attn_forward(q, k, v, 1)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q).double(), torch.from_numpy(k).double(), torch.from_numpy(v).double(), is_causal=True)
    assert np.abs(out - ref.numpy()).max() < 1e-13


def test_reduces_to_textbook_self_attention():
    # Self attention (Section 3): Q = K = V = X, unmasked.
    x = rand(1, 3, 19, 8)
    out, _ = oracle.attn_forward(x, x, x, 0)
    xt = torch.from_numpy(x).double()
    ref = torch.nn.functional.scaled_dot_product_attention(xt, xt, xt)
    assert np.abs(out - ref.numpy()).max() < 1e-13


def test_window_rows_equal_last_rows_of_full_causal_attention():
    # One softmax over history + window == the last W rows of causal attention over the whole sequence.
    N, W, d = 40, 12, 8
    x_q, k, v = rand(1, 2, N, d), rand(1, 2, N, d), rand(1, 2, N, d)
    full = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(x_q).double(), torch.from_numpy(k).double(), torch.from_numpy(v).double(), is_causal=True)
    out, _ = oracle.attn_forward(x_q[:, :, N - W:], k, v, 1)
    assert np.abs(out - full.numpy()[:, :, N - W:]).max() < 1e-13


# ---------------------------------------------------------------- closed forms
def test_constant_values_give_constant_output():
    q, k = rand(1, 2, 5, 4), rand(1, 2, 11, 4)
    v = np.ones((1, 2, 11, 4), dtype=np.float32)
    for causal in (0, 1):
        out, _ = oracle.attn_forward(q, k, v, causal)
        assert np.abs(out - 1.0).max() < 1e-15


@pytest.mark.parametrize("N,W", [(11, 5), (6, 6), (9, 1)])
def test_zero_query_gives_mean_and_log_count(N, W):
    q = np.zeros((1, 1, W, 4), dtype=np.float32)
    k, v = rand(1, 1, N, 4), rand(1, 1, N, 4)
    out, lse = oracle.attn_forward(q, k, v, 1)
    for i in range(W):
        cnt = N - W + i + 1
        assert abs(lse[0, 0, i] - math.log(cnt)) < 1e-14
        assert np.abs(out[0, 0, i] - v[0, 0, :cnt].astype(np.float64).mean(0)).max() < 1e-14
    out, lse = oracle.attn_forward(q, k, v, 0)
    assert np.abs(lse - math.log(N)).max() < 1e-14
    assert np.abs(out - v.astype(np.float64).mean(2, keepdims=True)).max() < 1e-14


def test_identical_keys_shift_lse_only():
    d, N, W = 4, 9, 3
    q, v = rand(1, 1, W, d), rand(1, 1, N, d)
    k0 = rand(d)
    k = np.broadcast_to(k0, (1, 1, N, d)).copy()
    out, lse = oracle.attn_forward(q, k, v, 0)
    s = (q[0, 0].astype(np.float64) @ k0.astype(np.float64)) / math.sqrt(d)
    assert np.abs(lse[0, 0] - (s + math.log(N))).max() < 1e-13
    assert np.abs(out[0, 0] - v[0, 0].astype(np.float64).mean(0)).max() < 1e-13


def test_dominant_key_selects_its_value():
    d, N = 4, 12
    q, k, v = rand(1, 1, 1, d), 0.01 * rand(1, 1, N, d), rand(1, 1, N, d)
    k[0, 0, 7] = 200.0 * q[0, 0, 0] / np.linalg.norm(q[0, 0, 0])
    out, _ = oracle.attn_forward(q, k, v, 0)
    assert np.abs(out[0, 0, 0] - v[0, 0, 7]).max() < 1e-12


def test_key_shift_moves_lse_by_q_dot_c():
    d, N, W = 8, 10, 4
    # dyadic values keep k + c exact in fp32
    q = np.round(rand(1, 1, W, d) * 8) / 8
    k = np.round(rand(1, 1, N, d) * 8) / 8
    v = rand(1, 1, N, d)
    c = (np.round(rand(d) * 8) / 8).astype(np.float32)
    out0, lse0 = oracle.attn_forward(q.astype(np.float32), k.astype(np.float32), v, 1)
    out1, lse1 = oracle.attn_forward(q.astype(np.float32), (k + c).astype(np.float32), v, 1)
    shift = (q[0, 0].astype(np.float64) @ c.astype(np.float64)) / math.sqrt(d)
    assert np.abs(out1 - out0).max() < 1e-12
    assert np.abs((lse1 - lse0)[0, 0] - shift).max() < 1e-12


def test_key_permutation_invariance_without_mask():
    q, k, v = rand(1, 2, 3, 4), rand(1, 2, 13, 4), rand(1, 2, 13, 4)
    perm = rng.permutation(13)
    out0, lse0 = oracle.attn_forward(q, k, v, 0)
    out1, lse1 = oracle.attn_forward(q, k[:, :, perm].copy(), v[:, :, perm].copy(), 0)
    assert np.abs(out1 - out0).max() < 1e-13 and np.abs(lse1 - lse0).max() < 1e-13


def test_scale_is_inverse_sqrt_of_head_dim():
    # single key pair: lse difference between two keys' scores isolates the 1/sqrt(d) factor
    d = 16
    q = np.zeros((1, 1, 1, d), np.float32); q[..., 0] = 4.0
    k = np.zeros((1, 1, 1, d), np.float32); k[..., 0] = 3.0
    v = rand(1, 1, 1, d)
    _, lse = oracle.attn_forward(q, k, v, 0)
    assert abs(lse.item() - 12.0 / 4.0) < 1e-14


# ---------------------------------------------------------------- mask and causality
def test_mask_predicate_exhaustive_small():
    for N in range(1, 9):
        for W in range(1, N + 1):
            cnt = 0
            for i in range(W):
                for j in range(-1, N + 1):
                    exp = (0 <= j < N) and (j <= N - W + i)
                    assert oracle.allowed(i, j, N, W, 1) == exp
                    cnt += exp
                    assert oracle.allowed(i, j, N, W, 0) == (0 <= j < N)
            assert cnt == cost_model.allowed_pairs(N, W, 1) == W * (N - W) + W * (W + 1) // 2


def test_future_tokens_do_not_change_earlier_rows_bitwise():
    N, W, d = 24, 10, 8
    q, k, v = rand(1, 2, W, d), rand(1, 2, N, d), rand(1, 2, N, d)
    out0, lse0 = oracle.attn_forward(q, k, v, 1)
    for i in (0, 3, 8):
        k2, v2 = k.copy(), v.copy()
        k2[:, :, N - W + i + 1:] += 5.0
        v2[:, :, N - W + i + 1:] -= 3.0
        out1, lse1 = oracle.attn_forward(q, k2, v2, 1)
        assert np.array_equal(out1[:, :, :i + 1], out0[:, :, :i + 1])
        assert np.array_equal(lse1[:, :, :i + 1], lse0[:, :, :i + 1])
        if i + 1 < W:
            assert not np.array_equal(out1[:, :, i + 1:], out0[:, :, i + 1:])


def test_rejects_window_longer_than_sequence():
    with pytest.raises(ValueError):
        oracle.attn_forward(rand(1, 1, 5, 4), rand(1, 1, 4, 4), rand(1, 1, 4, 4), 1)


# ---------------------------------------------------------------- element types
def test_bf16_inputs_are_widened_exactly():
    q = torch.randn(1, 2, 5, 8, generator=torch.Generator().manual_seed(3)).bfloat16()
    k = torch.randn(1, 2, 9, 8, generator=torch.Generator().manual_seed(4)).bfloat16()
    v = torch.randn(1, 2, 9, 8, generator=torch.Generator().manual_seed(5)).bfloat16()
    out_b, lse_b = oracle.attn_forward(q, k, v, 1)
    ref, ref_lse, _ = brute_force(q.float().numpy(), k.float().numpy(), v.float().numpy(), 1)
    assert np.abs(out_b - ref).max() < 1e-13 and np.abs(lse_b - ref_lse).max() < 1e-13
    bits = k.view(torch.int16).numpy().view(np.uint16)
    out_u, _ = oracle.attn_forward(q.view(torch.int16).numpy().view(np.uint16), bits,
                                   v.view(torch.int16).numpy().view(np.uint16), 1)
    assert np.array_equal(out_u, out_b)


# ---------------------------------------------------------------- split / merge
def merge_by_definition(oa, la, ob, lb):
    za, zb = np.exp(la), np.exp(lb)
    return (za[..., None] * oa + zb[..., None] * ob) / (za + zb)[..., None], np.log(za + zb)


@pytest.mark.parametrize("split", [1, 5, 12])
def test_attention_over_union_equals_merge_of_parts(split):
    N, W, d = 13, 4, 8
    q, k, v = rand(1, 2, W, d), rand(1, 2, N, d), rand(1, 2, N, d)
    full, full_lse, _ = brute_force(q, k, v, 0)
    oa, la, _ = brute_force(q, k[:, :, :split], v[:, :, :split], 0)
    ob, lb, _ = brute_force(q, k[:, :, split:], v[:, :, split:], 0)
    out, lse = oracle.merge_lse(oa, la, ob, lb)
    assert np.abs(out - full).max() < 1e-12 and np.abs(lse - full_lse).max() < 1e-12
    out_d, lse_d = merge_by_definition(oa, la, ob, lb)
    assert np.abs(out - out_d).max() < 1e-12 and np.abs(lse - lse_d).max() < 1e-12


def test_merge_with_empty_side_and_large_lse():
    oa, ob = rng.standard_normal((3, 4)), rng.standard_normal((3, 4))
    la = np.array([0.3, -np.inf, 900.0])
    lb = np.array([-np.inf, -np.inf, 899.0])
    out, lse = oracle.merge_lse(oa, la, ob, lb)
    assert np.array_equal(out[0], oa[0]) and lse[0] == 0.3
    assert lse[1] == -np.inf and np.array_equal(out[1], np.zeros(4))
    w = 1.0 / (1.0 + math.exp(-1.0))
    assert np.abs(out[2] - (w * oa[2] + (1 - w) * ob[2])).max() < 1e-14
    assert abs(lse[2] - (900.0 + math.log1p(math.exp(-1.0)))) < 1e-12


def test_history_plus_window_decomposition_matches_single_softmax():
    # "combined" read as one softmax over history (unmasked) and window (causal): equals the
    # merge of a focused call on the history and a plain causal call on the window.
    N, W, d = 29, 7, 8
    q, k, v = rand(1, 2, W, d), rand(1, 2, N, d), rand(1, 2, N, d)
    joint, joint_lse = oracle.attn_forward(q, k, v, 1)
    oh, lh = oracle.attn_forward(q, k[:, :, :N - W].copy(), v[:, :, :N - W].copy(), 0)
    ow, lw = oracle.attn_forward(q, k[:, :, N - W:].copy(), v[:, :, N - W:].copy(), 1)
    out, lse = merge_by_definition(oh, lh, ow, lw)
    assert np.abs(out - joint).max() < 1e-12 and np.abs(lse - joint_lse).max() < 1e-12


# ---------------------------------------------------------------- decode
def test_decode_steps_equal_rows_of_full_forward_and_cache_bookkeeping():
    B, H, N0, T, d = 2, 2, 11, 5, 8
    Ncap = N0 + T + 2
    canary = np.float32(-777.0)
    k_cache = np.full((B, H, Ncap, d), canary, dtype=np.float32)
    v_cache = np.full((B, H, Ncap, d), canary, dtype=np.float32)
    k_hist, v_hist = rand(B, H, N0, d), rand(B, H, N0, d)
    k_cache[:, :, :N0], v_cache[:, :, :N0] = k_hist, v_hist
    qn, kn, vn = rand(T, B, H, 1, d), rand(T, B, H, 1, d), rand(T, B, H, 1, d)
    k_all = np.concatenate([k_hist] + [kn[t] for t in range(T)], axis=2)
    v_all = np.concatenate([v_hist] + [vn[t] for t in range(T)], axis=2)
    q_all = np.concatenate([qn[t] for t in range(T)], axis=2)
    full, full_lse, _ = brute_force(q_all, k_all, v_all, 1)
    for t in range(T):
        out, lse = oracle.decode_step(qn[t], kn[t], vn[t], k_cache, v_cache, N0 + t)
        assert np.abs(out[:, :, 0] - full[:, :, t]).max() < 1e-13
        assert np.abs(lse - full_lse[:, :, t]).max() < 1e-13
        assert np.array_equal(k_cache[:, :, :N0 + t + 1], k_all[:, :, :N0 + t + 1])
        assert np.array_equal(v_cache[:, :, :N0 + t + 1], v_all[:, :, :N0 + t + 1])
        assert (k_cache[:, :, N0 + t + 1:] == canary).all() and (v_cache[:, :, N0 + t + 1:] == canary).all()


def test_decode_matches_forward_oracle_rows_bf16():
    wl = synth.Workload("t", 1, 2, 16, 37, 4, seed=9, decode=True)
    (kc, vc), (qn, kn, vn) = synth.decode_inputs(wl)
    k_all = torch.cat([kc[:, :, :wl.N]] + [kn[t] for t in range(wl.W)], dim=2)
    v_all = torch.cat([vc[:, :, :wl.N]] + [vn[t] for t in range(wl.W)], dim=2)
    q_all = torch.cat([qn[t] for t in range(wl.W)], dim=2)
    full, full_lse = oracle.attn_forward(q_all, k_all, v_all, 1)
    for t in range(wl.W):
        out, lse = oracle.decode_step(qn[t], kn[t], vn[t], kc, vc, wl.N + t)
        assert np.abs(out[:, :, 0] - full[:, :, t]).max() < 1e-13
        assert np.abs(lse - full_lse[:, :, t]).max() < 1e-13
    assert torch.equal(kc, k_all) and torch.equal(vc, v_all)


def test_decode_rejects_bad_position():
    z = np.zeros((1, 1, 1, 4), np.float32)
    c = np.zeros((1, 1, 3, 4), np.float32)
    for pos in (-1, 3):
        with pytest.raises(ValueError):
            oracle.decode_step(z, z, z, c, c.copy(), pos)


# ---------------------------------------------------------------- the paper's cost model
def test_cost_model_closed_forms_are_identities():
    r = np.random.default_rng(7)
    for _ in range(200):
        W_oh, W_og, Hd, D = (int(r.integers(1, 300)), int(r.integers(1, 300)), int(r.integers(0, 9)), int(r.integers(1, 600)))
        N = W_og + int(r.integers(1, 5000))
        assert D * cost_model.pairs(cost_model.miss_layers(N, W_oh, W_og, Hd)) == cost_model.miss_closed_form(N, W_oh, W_og, Hd, D)
        hit = cost_model.hit_layers(N, W_oh, W_og, Hd)
        assert D * cost_model.pairs(hit) == cost_model.hit_closed_form(N, W_oh, W_og, Hd, D)
        # slope/intercept form, Eq. (total cost = C1 N + C0)
        c1 = D * (2 * W_oh + W_og)
        c0 = D * (Hd * (W_oh ** 2 + W_og ** 2 + W_og * W_oh) + W_og ** 2 - W_og * W_oh)
        assert c1 * N + c0 == cost_model.miss_closed_form(N, W_oh, W_og, Hd, D)


def test_cost_model_hand_worked_examples():
    for line in open(os.path.join(GOLDEN, "cost_model_examples.txt")):
        if line.startswith("#") or not line.strip():
            continue
        N, W_oh, W_og, Hd, D, miss, hit = (int(x) for x in line.split())
        assert D * cost_model.pairs(cost_model.miss_layers(N, W_oh, W_og, Hd)) == miss
        assert cost_model.miss_closed_form(N, W_oh, W_og, Hd, D) == miss
        assert D * cost_model.pairs(cost_model.hit_layers(N, W_oh, W_og, Hd)) == hit
        assert cost_model.hit_closed_form(N, W_oh, W_og, Hd, D) == hit


# ---------------------------------------------------------------- the comparison gates themselves
def test_gates_reject_zero_output_and_accept_rounding_noise():
    import parity
    wl = synth.WORKLOADS["cfg1_tiny"]
    q, k, v = synth.forward_inputs(wl)
    ref, ref_lse = oracle.attn_forward(q, k, v, 1)
    with pytest.raises(AssertionError):
        parity.check(np.zeros_like(ref), ref_lse, ref, ref_lse, "bf16", "zero control")
    rounded = torch.from_numpy(ref).bfloat16().double().numpy()
    parity.check(rounded, ref_lse.astype(np.float32), ref, ref_lse, "bf16", "bf16 rounding")
    with pytest.raises(AssertionError):
        parity.check(rounded, ref_lse + 0.01, ref, ref_lse, "bf16", "lse control")


def test_stored_oracle_rows_have_not_drifted():
    wl = synth.WORKLOADS["cfg1_tiny"]
    q, k, v = synth.forward_inputs(wl)
    out, lse = oracle.attn_forward(q, k, v, wl.causal_window)
    n = 0
    for line in open(os.path.join(GOLDEN, "oracle_cfg1_rows.txt")):
        if line.startswith("#"):
            continue
        parts = line.split()
        b, h, i = (int(x) for x in parts[:3])
        vals = np.array([float(x) for x in parts[3:]])
        assert abs(lse[b, h, i] - vals[0]) < 1e-9
        assert np.abs(out[b, h, i, :8] - vals[1:]).max() < 1e-9
        n += 1
    assert n == 4


# ----------------------------------------------------------------------------- backward oracle
# The gradient of the Section 3 attention formula.  None of these pins calls attn_backward for its expectation.
def _rand_problem(seed, B, H, N, W, d):
    rng = np.random.default_rng(seed)
    mk = lambda *s: rng.standard_normal(s).astype(np.float32)
    return mk(B, H, W, d), mk(B, H, N, d), mk(B, H, N, d), mk(B, H, W, d)


@pytest.mark.parametrize("B,H,N,W,d,causal", [(1, 1, 6, 3, 4, 1), (1, 2, 7, 7, 3, 1), (2, 1, 5, 2, 2, 0), (1, 1, 4, 6, 4, 0)])
def test_backward_matches_central_differences_of_the_forward(B, H, N, W, d, causal):
    """dL/dx for L = sum(out * g), by central differences of the forward oracle (itself pinned above)."""
    q, k, v, g = _rand_problem(40 + N, B, H, N, W, d)
    dq, dk, dv = oracle.attn_backward(q, k, v, g, causal)

    def loss(q_, k_, v_):
        out, _ = oracle.attn_forward(q_, k_, v_, causal)
        return float((out * g.astype(np.float64)).sum())

    eps = 1e-3          # inputs are float32: the step has to survive the cast; the forward is smooth, error O(eps^2)
    for name, x, grad in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        rng = np.random.default_rng(7)
        for _ in range(12):
            idx = tuple(int(rng.integers(0, n)) for n in x.shape)
            xp, xm = x.copy(), x.copy()
            xp[idx] += eps
            xm[idx] -= eps
            args_p = {"q": (xp, k, v), "k": (q, xp, v), "v": (q, k, xp)}[name]
            args_m = {"q": (xm, k, v), "k": (q, xm, v), "v": (q, k, xm)}[name]
            step = float(xp[idx]) - float(xm[idx])          # the step actually taken after rounding to float32
            fd = (loss(*args_p) - loss(*args_m)) / step
            assert abs(fd - grad[idx]) <= 2e-5 * max(1.0, abs(fd)), (name, idx, fd, grad[idx])


@pytest.mark.parametrize("N,W,causal", [(9, 5, 1), (6, 6, 1), (8, 3, 0)])
def test_backward_matches_autograd_of_the_textbook_formula(N, W, causal):
    """torch autograd (fp64, CPU) through softmax(QK^T/sqrt(d) + mask)V written with library ops."""
    B, H, d = 2, 2, 8
    q, k, v, g = _rand_problem(50 + N, B, H, N, W, d)
    tq, tk, tv = (torch.tensor(x, dtype=torch.float64, requires_grad=True) for x in (q, k, v))
    s = tq @ tk.transpose(-1, -2) / d ** 0.5
    if causal:
        keep = torch.arange(N)[None, :] <= (N - W) + torch.arange(W)[:, None]
        s = s.masked_fill(~keep, float("-inf"))
    (torch.softmax(s, -1) @ tv * torch.tensor(g, dtype=torch.float64)).sum().backward()
    dq, dk, dv = oracle.attn_backward(q, k, v, g, causal)
    assert np.abs(dq - tq.grad.numpy()).max() < 1e-12
    assert np.abs(dk - tk.grad.numpy()).max() < 1e-12
    assert np.abs(dv - tv.grad.numpy()).max() < 1e-12


def test_backward_closed_forms():
    """q = 0: uniform probabilities over the allowed keys, so dv_j = sum_i dout_i / n_i over the rows that see j,
    and dk = 0 (ds multiplies q = 0); dq_i = sum_j ds_ij k_j / sqrt(d) with ds_ij = (dout_i.v_j - mean_j')/n_i."""
    B, H, N, W, d = 1, 1, 6, 3, 4
    _, k, v, g = _rand_problem(3, B, H, N, W, d)
    q = np.zeros((B, H, W, d), dtype=np.float32)
    dq, dk, dv = oracle.attn_backward(q, k, v, g, 1)
    assert np.abs(dk).max() == 0.0
    n_i = np.array([N - W + i + 1 for i in range(W)], dtype=np.float64)
    exp_dv = np.zeros((N, d))
    exp_dq = np.zeros((W, d))
    for i in range(W):
        n = int(n_i[i])
        exp_dv[:n] += g[0, 0, i].astype(np.float64) / n
        dp = v[0, 0, :n].astype(np.float64) @ g[0, 0, i].astype(np.float64)
        ds = (dp - dp.mean()) / n
        exp_dq[i] = ds @ k[0, 0, :n].astype(np.float64) / np.sqrt(d)
    assert np.abs(dv[0, 0] - exp_dv).max() < 1e-13 and np.abs(dq[0, 0] - exp_dq).max() < 1e-13
    # the rows of ds sum to zero: adding the same vector to every allowed key leaves dq's projection ... and
    # a constant added to dout along v-directions: sum_j dv_j = sum_i dout_i (probabilities sum to one)
    q2, k2, v2, g2 = _rand_problem(4, 1, 2, 7, 4, 3)
    _, _, dv2 = oracle.attn_backward(q2, k2, v2, g2, 0)
    assert np.abs(dv2.sum(axis=2) - g2.astype(np.float64).sum(axis=2)).max() < 1e-12


def test_backward_respects_the_causal_window():
    """Keys beyond a row's limit get no gradient from that row: with only the first window row carrying dout,
    dk and dv vanish exactly for j > N - W, and dq of the other rows is zero."""
    B, H, N, W, d = 1, 1, 8, 4, 4
    q, k, v, g = _rand_problem(9, B, H, N, W, d)
    g[:, :, 1:] = 0.0
    dq, dk, dv = oracle.attn_backward(q, k, v, g, 1)
    assert (dk[0, 0, N - W + 1:] == 0).all() and (dv[0, 0, N - W + 1:] == 0).all()
    assert (dq[0, 0, 1:] == 0).all() and np.abs(dq[0, 0, 0]).max() > 0
    assert np.abs(dv[0, 0, :N - W + 1]).min() > 0


# ---------------------------------------------------------------------------------------------------------------
# 8-bit (E4M3) key/value cache: the codec against the published format and a library conversion, the decode step
# against a probability matrix written out in numpy over values dequantised by the library conversion.
def test_e4m3_decode_table_matches_the_format_and_the_library_view():
    assert oracle.e4m3_decode(0x00) == 0.0 and oracle.e4m3_decode(0x38) == 1.0 and oracle.e4m3_decode(0x40) == 2.0
    assert oracle.e4m3_decode(0x7E) == 448.0 and oracle.e4m3_decode(0x01) == 2.0 ** -9 and oracle.e4m3_decode(0x08) == 2.0 ** -6
    assert oracle.e4m3_decode(0xC0) == -2.0 and np.isnan(oracle.e4m3_decode(0x7F)) and np.isnan(oracle.e4m3_decode(0xFF))
    mine = np.array([oracle.e4m3_decode(c) for c in range(256)])
    assert np.all(np.diff(mine[:0x7F]) > 0)                       # codes order the non-negative values
    lib = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).float().numpy()
    assert np.all((mine == lib) | (np.isnan(mine) & np.isnan(lib)))


def test_e4m3_encode_rounds_to_nearest_even_and_saturates():
    for c in list(range(0x7F)) + list(range(0x80, 0xFF)):
        assert oracle.e4m3_encode(oracle.e4m3_decode(c)) == c      # every finite code is a fixed point (signed zero too)
    assert oracle.e4m3_encode(1.0625) == 0x38 and oracle.e4m3_encode(1.1875) == 0x3A       # ties go to the even mantissa
    assert oracle.e4m3_encode(2.0 ** -10) == 0x00 and oracle.e4m3_encode(3 * 2.0 ** -10) == 0x02   # ties among subnormals
    assert oracle.e4m3_encode(449.0) == 0x7E and oracle.e4m3_encode(1e30) == 0x7E and oracle.e4m3_encode(-1e30) == 0xFE
    assert oracle.e4m3_encode(float("nan")) == 0x7F
    g = torch.Generator().manual_seed(0)
    x = torch.cat([torch.randn(20000, generator=g) * s for s in (1e-3, 0.1, 3.0, 100.0)])
    x = x[x.abs() <= 448.0]                                        # the library conversion does not saturate beyond
    lib = x.to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    mine = np.array([oracle.e4m3_encode(float(v)) for v in x.numpy()], dtype=np.uint8)
    assert np.array_equal(lib, mine)


def test_fp8_decode_step_against_numpy_over_library_dequantised_values():
    B, H, Ncap, d, pos = 2, 3, 20, 16, 11
    g = torch.Generator().manual_seed(5)
    k_scale = (torch.rand(B, H, generator=g) * 0.05 + 0.01).float()
    v_scale = (torch.rand(B, H, generator=g) * 0.05 + 0.01).float()
    kc = (torch.randn(B, H, Ncap, d, generator=g) / k_scale[:, :, None, None]).to(torch.float8_e4m3fn).view(torch.uint8).contiguous()
    vc = (torch.randn(B, H, Ncap, d, generator=g) / v_scale[:, :, None, None]).to(torch.float8_e4m3fn).view(torch.uint8).contiguous()
    q, kn, vn = (torch.randn(B, H, 1, d, generator=g).to(torch.bfloat16) for _ in range(3))
    kc0, vc0 = kc.clone(), vc.clone()
    out, lse = oracle.decode_step_fp8(q, kn, vn, kc, vc, k_scale, v_scale, pos)
    # the appended row: fp32 division, then the library's conversion; nothing else changed
    want_k = (kn.float() / k_scale[:, :, None, None]).to(torch.float8_e4m3fn).view(torch.uint8)[:, :, 0]
    want_v = (vn.float() / v_scale[:, :, None, None]).to(torch.float8_e4m3fn).view(torch.uint8)[:, :, 0]
    assert torch.equal(kc[:, :, pos], want_k) and torch.equal(vc[:, :, pos], want_v)
    keep = [j for j in range(Ncap) if j != pos]
    assert torch.equal(kc[:, :, keep], kc0[:, :, keep]) and torch.equal(vc[:, :, keep], vc0[:, :, keep])
    # attention over the dequantised rows [0, pos], written out
    kd = kc.view(torch.float8_e4m3fn).double().numpy() * k_scale.double().numpy()[:, :, None, None]
    vd = vc.view(torch.float8_e4m3fn).double().numpy() * v_scale.double().numpy()[:, :, None, None]
    s = np.einsum("bhqc,bhjc->bhqj", q.double().numpy(), kd[:, :, :pos + 1]) / np.sqrt(d)
    p = np.exp(s - s.max(-1, keepdims=True))
    want = np.einsum("bhqj,bhjc->bhqc", p / p.sum(-1, keepdims=True), vd[:, :, :pos + 1])
    assert np.abs(out - want).max() < 1e-12
    assert np.abs(lse - (np.log(p.sum(-1)) + s.max(-1))[:, :, 0]).max() < 1e-12
