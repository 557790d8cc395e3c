"""GPU parity of the backward entry point against the CPU oracle's fp64 chain rule, element by element on the
same seeded bf16 inputs.  The forward results the backward needs (out, lse) come from the library's own forward,
as they do in training.

Gates (bf16 in, fp32 arithmetic, bf16 out): per gradient tensor, relative L2 error <= 2e-2 and
max|err| <= 2e-2 * max|reference| -- the forward's absolute gates, scaled by the gradient's own magnitude, because a
gradient has no natural unit scale (it is linear in dout).  Where the exact gradient is identically zero (a single
visible key makes the softmax constant, so dq = dk = 0) the fp32 difference dp - delta leaves rounding noise of a few
1e-7 on unit-scale inputs: an absolute floor of 1e-5 covers it."""
import numpy as np
import pytest
import torch

import oracle
import parity
from guards import Guarded
from paper_2508_20407_b200 import binding as tl
from paper_2508_20407_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda"
REL_L2, REL_MAX, ABS_FLOOR = 2e-2, 2e-2, 1e-5


IMPLS = [0, 1]      # 0: tensor-core kernels, 1: CUDA-core kernels (the same switch as the forward's)


def grads(q, k, v, dout, causal, impl=0, guarded=False, arrangement=1):
    """Gradients through the C-ABI.  guarded: dq, dk, dv and the workspace sit inside buffers of exactly the documented
    sizes with filled guard regions on both sides, which must come back untouched.  arrangement: tlin_set_backward_impl
    (1, the two kernels, unless a test asks for the one kernel or for the library's own choice)."""
    out, lse = tl.tlin_attn_forward(q, k, v, causal_window=causal)
    prev = tl.tlin_set_forward_impl(impl)
    prev_arr = tl.tlin_set_backward_impl(arrangement)
    saved = tl._workspace_tensor
    gs = []
    try:
        dq = dk = dv = None
        if guarded:
            B, H, W, d = q.shape
            gq, gk, gv = Guarded(q.shape, q.dtype, DEV), Guarded(k.shape, k.dtype, DEV), Guarded(v.shape, v.dtype, DEV)
            gw = Guarded((max(tl.workspace_bytes_backward(B, H, k.shape[2], W, d), 16),), torch.uint8, DEV)
            gs = [(gq, "dq"), (gk, "dk"), (gv, "dv"), (gw, "workspace")]
            tl.set_workspace(gw.t)
            dq, dk, dv = gq.t, gk.t, gv.t
        dq, dk, dv = tl.tlin_attn_backward(q, k, v, out, lse, dout, dq, dk, dv, causal_window=causal)
        torch.cuda.synchronize()
        assert tl.tlin_get_status() == 0
        assert tl.tlin_last_launch_count() >= 3
        if guarded:
            assert tl._workspace_tensor is gw.t
    finally:
        tl.tlin_set_forward_impl(prev)
        tl.tlin_set_backward_impl(prev_arr)
        if guarded:
            tl.set_workspace(saved)
    for g, name in gs:
        g.check(f"backward impl={impl} {name}")
    return dq, dk, dv


def compare(got, ref, what):
    got = got.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all(), f"{what}: non-finite gradient"
    e = parity.errors(got, ref)
    scale = float(np.abs(ref).max())
    if scale > 1e-3:
        assert e["rel_l2"] <= REL_L2, f"{what}: rel L2 {e['rel_l2']:.3e}"
    assert e["max_abs"] <= REL_MAX * scale + ABS_FLOOR, f"{what}: max|err| {e['max_abs']:.3e} vs max|ref| {scale:.3e}"
    return e


def run_case(B, H, N, W, d, causal, seed, peaky=False, impl=0, guarded=False, arrangement=1):
    wl = synth.Workload("bwd", B, H, d, N, W, seed=seed, causal_window=causal)
    q, k, v = synth.forward_inputs(wl, device=DEV, dtype=torch.bfloat16)
    if peaky:
        q = (q.float() * 6.0).to(torch.bfloat16)
    g = torch.Generator(device="cpu").manual_seed(seed + 7)
    dout = torch.randn(q.shape, generator=g, dtype=torch.float32).to(torch.bfloat16).to(DEV)
    dq, dk, dv = grads(q, k, v, dout, causal, impl, guarded, arrangement)
    rq, rk, rv = oracle.attn_backward(q.cpu(), k.cpu(), v.cpu(), dout.cpu(), causal)
    tag = f"B{B} H{H} N{N} W{W} d{d} causal{causal} impl{impl} arrangement{arrangement}"
    compare(dq, rq, tag + " dq")
    compare(dk, rk, tag + " dk")
    compare(dv, rv, tag + " dv")
    return dq, dk, dv


SHAPES = [  # B, H, N, W, d, causal: single elements, ragged tails on both axes, several key slices, both masks
    (1, 1, 1, 1, 64, 1), (1, 2, 33, 1, 128, 1), (2, 1, 64, 64, 64, 1), (1, 2, 300, 300, 128, 1),
    (1, 3, 1000, 77, 128, 1), (2, 2, 515, 130, 64, 0), (1, 2, 257, 255, 128, 0), (1, 1, 100, 300, 128, 0),
    (1, 1, 4096, 96, 128, 1), (3, 2, 1111, 200, 64, 1), (1, 1, 2049, 31, 64, 0),
]


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("B,H,N,W,d,causal", SHAPES)
def test_backward_elementwise(B, H, N, W, d, causal, impl):
    run_case(B, H, N, W, d, causal, seed=300 + N + W, impl=impl, guarded=True)


@pytest.mark.parametrize("seed", [21, 22, 23])
def test_backward_random_shapes_against_the_oracle(seed):
    # seeded shapes nobody picked by hand (the forward tests' generator, smaller: the fp64 chain rule costs more)
    from test_gpu_forward import random_shapes
    for (B, H, N, W, d, causal) in random_shapes(seed, 6, budget=1.5e9):
        run_case(B, H, N, W, d, causal, seed=seed * 1000 + N + W, impl=0, guarded=True)


# the one-kernel arrangement (d = 128): the same element-by-element gates, guarded buffers, poisoned workspace
ONE_KERNEL = [s for s in SHAPES if s[4] == 128] + [(1, 2, 40000, 300, 128, 1), (1, 1, 30000, 1024, 128, 0), (2, 40, 1600, 1500, 128, 1),
                                                   (1, 1, 2048, 512, 128, 1), (1, 3, 2560, 768, 128, 1), (1, 5, 4000, 1000, 128, 1)]


@pytest.mark.parametrize("B,H,N,W,d,causal", ONE_KERNEL)
def test_backward_one_kernel_arrangement(B, H, N, W, d, causal):
    assert tl.workspace_bytes_backward(B, H, N, W, d) >= B * H * (-(-W // 128) * 128) * (d + 2) * 4
    run_case(B, H, N, W, d, causal, seed=600 + N + W, impl=0, guarded=True, arrangement=2)


def test_backward_one_kernel_arrangement_repeats_dk_dv_bitwise_and_dq_within_fp32_addition_order():
    wl = synth.Workload("bwd", 1, 2, 128, 30000, 300, seed=9, causal_window=1)
    q, k, v = synth.forward_inputs(wl, device=DEV, dtype=torch.bfloat16)
    dout = torch.randn(q.shape, device=DEV).to(torch.bfloat16)
    a = grads(q, k, v, dout, 1, 0, arrangement=2)
    b = grads(q, k, v, dout, 1, 0, arrangement=2)
    assert torch.equal(a[1], b[1]) and torch.equal(a[2], b[2])
    diff = (a[0].float() - b[0].float()).abs()
    assert float(diff.max()) <= 2.0 ** -7 * float(a[0].float().abs().max())
    two = grads(q, k, v, dout, 1, 0, arrangement=1)
    assert torch.equal(a[1], two[1]) and torch.equal(a[2], two[2])      # dK, dV: the same products in the same order


@pytest.mark.parametrize("B,H,N,W,d,causal", [(1, 2, 4000, 300, 128, 1), (2, 2, 515, 130, 128, 0), (1, 3, 1000, 77, 64, 1)])
def test_backward_with_the_arrangement_the_library_chooses(B, H, N, W, d, causal):
    # setting 0: fp32 dQ buffers up to 64 MiB take the one kernel at d = 128, everything else the two kernels
    prev = tl.tlin_set_backward_impl(0)
    try:
        assert tl.tlin_backward_arrangement(B, H, N, W, d) == (2 if d == 128 else 1)
        assert tl.tlin_backward_arrangement(4, 32, 4096, 4096, 128) == 1        # 256 MiB of fp32 dQ
        assert tl.tlin_backward_arrangement(4, 32, 8192, 1024, 128) == 2        # 64 MiB
        assert tl.tlin_backward_arrangement(1, 32, 32768, 512, 128) == 2        # 8 MiB
        assert tl.tlin_backward_arrangement(1, 1, 1, 1, 36) < 0 and tl.tlin_backward_arrangement(0, 1, 1, 1, 128) < 0
        tl.tlin_set_backward_impl(1)
        assert tl.tlin_backward_arrangement(B, H, N, W, d) == 1
    finally:
        tl.tlin_set_backward_impl(prev)
    run_case(B, H, N, W, d, causal, seed=650 + N + W, impl=0, guarded=True, arrangement=0)


def test_backward_arrangement_switch_rejects_other_values_and_other_head_sizes_keep_two_kernels():
    assert tl.tlin_set_backward_impl(0) in (0, 1, 2)
    assert tl.tlin_set_backward_impl(3) < 0 and tl.tlin_set_backward_impl(-1) < 0
    run_case(1, 2, 515, 130, 64, 1, seed=4, impl=0, guarded=True, arrangement=2)     # d = 64
    assert tl.tlin_last_launch_count() >= 3


@pytest.mark.parametrize("impl", IMPLS)
def test_backward_cfg1_tiny(impl):
    wl = synth.WORKLOADS["cfg1_tiny"]
    run_case(wl.B, wl.H, wl.N, wl.W, wl.d, wl.causal_window, seed=wl.seed, impl=impl)


@pytest.mark.parametrize("impl", IMPLS)
def test_backward_peaked_softmax(impl):
    # scores large enough that most rows put nearly all weight on one key: exercises exp(s - lse) near 1 and near 0
    run_case(1, 2, 700, 96, 128, 1, seed=11, peaky=True, impl=impl)


# many CTAs per (b,h) on the dQ side (key range split between groups, partial sums added by the reduce kernel), several
# key tiles per CTA on the dK/dV side, both schedules of the plan
BIG = [(1, 2, 40000, 300, 128, 1), (2, 3, 20000, 520, 64, 1), (1, 160, 384, 512, 64, 0), (6, 16, 1024, 1000, 64, 1),
       (1, 1, 30000, 1024, 128, 0),
       # the dQ kernel on a plan whose CTAs share whole problems by cost (window rule, >= three problems per CTA)
       (2, 40, 1600, 1500, 128, 1), (3, 50, 900, 900, 64, 1)]


@pytest.mark.parametrize("B,H,N,W,d,causal", BIG)
def test_backward_tensor_core_schedules(B, H, N, W, d, causal):
    run_case(B, H, N, W, d, causal, seed=500 + N + W, impl=0)


def segments_without_a_visible_key_tile(plan, N, W):
    """(group, bh, q tile) of every partial segment of the dQ kernel's plan in which the window rule hides all key tiles
    from the whole 256-row query tile: the segment runs no MMA, yet its partial slot is summed by the reduce kernel."""
    T = plan.key_tiles
    starts = [tl.tlin_plan_group_start(plan, g) for g in range(plan.n_groups + 1)]
    found = []
    for g in range(plan.n_groups):
        u = starts[g]
        while u < starts[g + 1]:
            bh, tb = divmod(u, T)
            te = min(T, tb + (starts[g + 1] - u))
            if not (tb == 0 and te == T):
                for qt in range(plan.q_tiles):
                    visible = -(-min(N, N - W + qt * plan.tile_m + plan.tile_m) // plan.tile_n)
                    if visible <= tb:
                        found.append((g, bh, qt))
            u += te - tb
    return found


# window rule, key range of a (b,h) split between groups, and a group whose share of the keys lies wholly behind the
# window of the first query tiles: those (group, query tile) pairs have nothing to compute for the shared (b,h)
HIDDEN_TAIL = [(1, 1, 2048, 512, 128), (1, 1, 1536, 1024, 64), (1, 3, 2560, 768, 128), (2, 2, 3000, 700, 64),
               (1, 5, 4000, 1000, 128)]


@pytest.mark.parametrize("B,H,N,W,d", HIDDEN_TAIL)
def test_backward_split_keys_with_segments_hidden_by_the_window(B, H, N, W, d):
    prev = tl.tlin_set_forward_impl(0)
    try:
        plan = tl.tlin_plan_forward(B, H, N, W, d, 1)
    finally:
        tl.tlin_set_forward_impl(prev)
    assert plan.tensor_path and plan.schedule == 0 and plan.uses_workspace
    assert segments_without_a_visible_key_tile(plan, N, W), "the shape no longer reaches the case this test is for"
    run_case(B, H, N, W, d, 1, seed=800 + N + W, impl=0, guarded=True)


@pytest.mark.parametrize("impl", IMPLS)
def test_backward_keys_outside_every_window_get_zero_gradient(impl):
    # with the window rule the last key is visible to the last query only; a key count N == W makes key j invisible
    # to queries i < j.  Zero dout rows for the queries that see the tail => exact zeros in dk, dv there.
    B, H, N, W, d = 1, 2, 160, 160, 64
    wl = synth.Workload("bwd", B, H, d, N, W, seed=5, causal_window=1)
    q, k, v = synth.forward_inputs(wl, device=DEV, dtype=torch.bfloat16)
    dout = torch.randn(q.shape, device=DEV).to(torch.bfloat16)
    dout[:, :, 100:, :] = 0
    _, dk, dv = grads(q, k, v, dout, 1, impl)
    assert float(dk[:, :, 100:, :].float().abs().max()) == 0.0
    assert float(dv[:, :, 100:, :].float().abs().max()) == 0.0
    assert float(dk[:, :, :100, :].float().abs().max()) > 0.0


def test_backward_tensor_core_path_is_bitwise_repeatable():
    wl = synth.Workload("bwd", 1, 2, 128, 30000, 300, seed=9, causal_window=1)
    q, k, v = synth.forward_inputs(wl, device=DEV, dtype=torch.bfloat16)
    dout = torch.randn(q.shape, device=DEV).to(torch.bfloat16)
    a = grads(q, k, v, dout, 1, 0)
    b = grads(q, k, v, dout, 1, 0)
    assert all(torch.equal(x, y) for x, y in zip(a, b))


def test_backward_cuda_core_path_is_deterministic_up_to_the_dq_sum_order():
    # dk, dv have one owner per element: bitwise repeatable.  dq is summed over key slices with atomics: equal within
    # fp32 rounding, so the rounded bf16 values differ by at most a last place of the largest elements.
    wl = synth.Workload("bwd", 1, 2, 128, 3000, 64, seed=9, causal_window=1)
    q, k, v = synth.forward_inputs(wl, device=DEV, dtype=torch.bfloat16)
    dout = torch.randn(q.shape, device=DEV).to(torch.bfloat16)
    a = grads(q, k, v, dout, 1, 1)
    b = grads(q, k, v, dout, 1, 1)
    assert torch.equal(a[1], b[1]) and torch.equal(a[2], b[2])
    diff = (a[0].float() - b[0].float()).abs()
    assert float(diff.max()) <= 2.0 ** -7 * float(a[0].float().abs().max())


def test_backward_argument_errors():
    q = torch.zeros(1, 1, 32, 64, dtype=torch.bfloat16, device=DEV)
    k = torch.zeros(1, 1, 16, 64, dtype=torch.bfloat16, device=DEV)
    lse = torch.zeros(1, 1, 32, dtype=torch.float32, device=DEV)
    with pytest.raises(tl.TlinError):        # N < W with the window rule
        tl.tlin_attn_backward(q, k, k, q, lse, q, causal_window=1)
    q100 = torch.zeros(1, 1, 8, 100, dtype=torch.bfloat16, device=DEV)
    lse8 = torch.zeros(1, 1, 8, dtype=torch.float32, device=DEV)
    with pytest.raises(tl.TlinError):        # bf16 head sizes are multiples of 8
        tl.tlin_attn_backward(q100, q100, q100, q100, lse8, q100, causal_window=0)


ODD = [(1, 2, 300, 77, 40, 1), (2, 1, 515, 130, 96, 0), (1, 1, 200, 64, 256, 1), (1, 2, 129, 33, 8, 1)]


@pytest.mark.parametrize("B,H,N,W,d,causal", ODD)
def test_backward_other_head_sizes_bf16(B, H, N, W, d, causal):
    # head sizes outside {64, 128} are served by the CUDA-core kernels whatever the switch says
    run_case(B, H, N, W, d, causal, seed=700 + N + d, impl=0)


F32 = [(1, 2, 300, 77, 36, 1), (2, 1, 515, 130, 64, 0), (1, 1, 1000, 200, 128, 1), (1, 3, 97, 97, 100, 1), (1, 1, 1, 1, 4, 1)]


@pytest.mark.parametrize("B,H,N,W,d,causal", F32)
def test_backward_f32(B, H, N, W, d, causal):
    # fp32 tensors, fp32 arithmetic (the paper's own model has d = 36): gates of the fp32 forward, relative to the
    # gradient's magnitude
    wl = synth.Workload("bwd32", B, H, d, N, W, seed=900 + N + d, causal_window=causal)
    q, k, v = synth.forward_inputs(wl, device=DEV, dtype=torch.float32)
    g = torch.Generator(device="cpu").manual_seed(3)
    dout = torch.randn(q.shape, generator=g, dtype=torch.float32).to(DEV)
    out, lse = tl.tlin_attn_forward_f32(q, k, v, causal_window=causal)
    dq, dk, dv = tl.tlin_attn_backward_f32(q, k, v, out, lse, dout, causal_window=causal)
    torch.cuda.synchronize()
    assert tl.tlin_get_status() == 0
    refs = oracle.attn_backward(q.cpu(), k.cpu(), v.cpu(), dout.cpu(), causal)
    for got, ref, name in zip((dq, dk, dv), refs, ("dq", "dk", "dv")):
        e = parity.errors(got.cpu().numpy(), ref)
        scale = float(np.abs(ref).max())
        assert e["max_abs"] <= 1e-4 * scale + 1e-6, f"{name}: max|err| {e['max_abs']:.3e} vs max|ref| {scale:.3e}"
        if scale > 1e-3:
            assert e["rel_l2"] <= 1e-4, f"{name}: rel L2 {e['rel_l2']:.3e}"


@pytest.mark.parametrize("name,heads,arrangement", [("train_chunk", ((0, 0), (1, 16), (3, 31)), 1), ("train_seq", ((2, 9),), 1),
                                                    ("train_chunk", ((0, 5), (2, 0), (3, 30)), 0)])
def test_backward_at_the_benchmarked_training_shapes_on_sampled_heads(name, heads, arrangement):
    # the full workloads bench.py times (train_chunk: B4 H32 N8192 W1024, the last window of a sliding-window pass;
    # train_seq: B4 H32 N=W=4096, a whole sequence over itself, where the CTAs share whole problems by cost); the
    # oracle recomputes whole (b,h) pairs, which are independent problems: the first, a middle and the last one
    wl = synth.WORKLOADS[name]
    q, k, v = synth.forward_inputs(wl, device=DEV, dtype=torch.bfloat16)
    g = torch.Generator(device="cpu").manual_seed(wl.seed + 99)
    dout = torch.randn(q.shape, generator=g, dtype=torch.float32).to(torch.bfloat16).to(DEV)
    dq, dk, dv = grads(q, k, v, dout, wl.causal_window, 0, arrangement=arrangement)   # 0: what bench.py times (the library's choice)
    for b, h in heads:
        sl = (slice(b, b + 1), slice(h, h + 1))
        rq, rk, rv = oracle.attn_backward(q[sl].cpu(), k[sl].cpu(), v[sl].cpu(), dout[sl].cpu(), wl.causal_window)
        compare(dq[sl], rq, f"{name} b{b} h{h} dq")
        compare(dk[sl], rk, f"{name} b{b} h{h} dk")
        compare(dv[sl], rv, f"{name} b{b} h{h} dv")


@pytest.mark.parametrize("dtype,d", [(torch.bfloat16, 128), (torch.float32, 36)])
def test_autograd_glue_matches_pytorch_autograd_of_the_textbook_formula(dtype, d):
    # tl.attention plugs the two entry points into torch.autograd; the reference differentiates the formula itself in fp64
    B, H, N, W, causal = 2, 2, 300, 130, 1
    g = torch.Generator(device="cpu").manual_seed(17)
    mk = lambda *s: (torch.randn(*s, generator=g) / 3).to(dtype).to(DEV).requires_grad_(True)
    q, k, v = mk(B, H, W, d), mk(B, H, N, d), mk(B, H, N, d)
    w = torch.randn(B, H, W, d, generator=g).to(DEV)
    out, lse = tl.attention(q, k, v, causal_window=causal)
    (out.float() * w).sum().backward()
    qd, kd, vd = (t.detach().double().cpu().requires_grad_(True) for t in (q, k, v))
    s = qd @ kd.transpose(-1, -2) / d ** 0.5
    i = torch.arange(W)[:, None]
    j = torch.arange(N)[None, :]
    s = s.masked_fill(j > (N - W) + i, float("-inf"))
    ref = torch.softmax(s, -1) @ vd
    (ref * w.double().cpu()).sum().backward()
    tol = 2e-2 if dtype == torch.bfloat16 else 1e-4
    for got, want, name in ((q.grad, qd.grad, "dq"), (k.grad, kd.grad, "dk"), (v.grad, vd.grad, "dv")):
        err = float((got.double().cpu() - want).abs().max())
        assert err <= tol * float(want.abs().max()) + 1e-6, f"{name}: {err:.3e}"
    assert not lse.requires_grad


@pytest.mark.parametrize("name", ["train_chunk", "train_seq"])
def test_backward_invariants_on_every_head_at_the_benchmarked_shapes(name):
    """Properties of the exact gradients that hold at any size, checked on ALL (b,h) of the full workloads (the oracle
    recomputes only a few heads there): every softmax row sums to one, so sum_j dv_j = sum_i dout_i, and sum_j ds_ij = 0
    for every query i, so sum_j dk_j = 0.  The stored gradients are rounded to bf16: the sums of n rounded values are
    compared within sqrt(n) rounding errors of their typical magnitude (six standard deviations)."""
    wl = synth.WORKLOADS[name]
    q, k, v = synth.forward_inputs(wl, device=DEV, dtype=torch.bfloat16)
    g = torch.Generator(device="cpu").manual_seed(wl.seed + 99)
    dout = torch.randn(q.shape, generator=g, dtype=torch.float32).to(torch.bfloat16).to(DEV)
    dq, dk, dv = grads(q, k, v, dout, wl.causal_window, 0)
    assert torch.isfinite(dq.float()).all() and torch.isfinite(dk.float()).all() and torch.isfinite(dv.float()).all()
    n = wl.N
    # sum over keys of dv against sum over queries of dout, per (b,h) and column
    lhs, rhs = dv.double().sum(dim=2), dout.double().sum(dim=2)
    scale_v = dv.double().abs().mean(dim=2) * (n ** 0.5) * 2.0 ** -8 * 6 + 1e-6
    assert bool(((lhs - rhs).abs() <= scale_v + 2e-3 * rhs.abs()).all()), float(((lhs - rhs).abs() / (scale_v + 2e-3 * rhs.abs())).max())
    # sum over keys of dk is zero up to rounding, per (b,h) and column.  delta_i = dout_i . out_i is formed from the
    # stored bf16 out, whose rounding (2^-9 relative per element) leaves sum_j ds_ij = delta_i(exact) - delta_i(used) =: e_i
    # and so sum_j dk_j = scale * sum_i e_i q_i: that term is estimated from the data and allowed as well
    out, _ = tl.tlin_attn_forward(q, k, v, causal_window=wl.causal_window)
    e2 = (dout.double() * out.double()).pow(2).sum(dim=3, keepdim=True) * 2.0 ** -18          # per query row
    delta_term = (q.double().pow(2) * e2).sum(dim=2).sqrt() / wl.d ** 0.5
    s = dk.double().sum(dim=2).abs()
    scale_k = dk.double().abs().mean(dim=2) * (n ** 0.5) * 2.0 ** -8 * 6 + 6 * delta_term + 1e-6
    assert bool((s <= scale_k).all()), float((s / scale_k).max())


def test_backward_both_kernel_families_agree_on_every_head_of_the_training_chunk():
    """dq has no closed-form invariant, so on the full train_chunk workload every (b,h) of the tensor-core gradients is
    compared with the CUDA-core kernels' (which the small cases pin to the oracle element by element): two independent
    implementations of the same chain rule, both storing bf16.  Gate per (b,h): the oracle gates of this file with the
    other family as the reference, plus one bf16 last place for the second rounding."""
    wl = synth.WORKLOADS["train_chunk"]
    q, k, v = synth.forward_inputs(wl, device=DEV, dtype=torch.bfloat16)
    g = torch.Generator(device="cpu").manual_seed(wl.seed + 99)
    dout = torch.randn(q.shape, generator=g, dtype=torch.float32).to(torch.bfloat16).to(DEV)
    tc = grads(q, k, v, dout, wl.causal_window, 0)
    cc = grads(q, k, v, dout, wl.causal_window, 1)
    one = grads(q, k, v, dout, wl.causal_window, 0, arrangement=2)
    assert torch.equal(one[1], tc[1]) and torch.equal(one[2], tc[2])
    for a, b, name in list(zip(tc, cc, ("dq", "dk", "dv"))) + [(one[0], cc[0], "dq (one kernel)")]:
        a, b = a.float(), b.float()
        assert torch.isfinite(a).all() and torch.isfinite(b).all(), name
        diff = (a - b).abs()
        scale = b.abs().amax(dim=(2, 3))                                   # per (b,h)
        worst = diff.amax(dim=(2, 3))
        gate = (REL_MAX + 2.0 ** -7) * scale + ABS_FLOOR
        assert bool((worst <= gate).all()), f"{name}: worst (b,h) ratio {float((worst / gate).max()):.3f}"
        rel = (diff.double().pow(2).sum(dim=(2, 3)) / b.double().pow(2).sum(dim=(2, 3)).clamp_min(1e-30)).sqrt()
        assert bool((rel <= REL_L2).all()), f"{name}: rel L2 {float(rel.max()):.3e}"
