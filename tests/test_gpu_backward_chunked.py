"""GPU parity of the O(T) two-pass backward (kata_bwd_chunked) against the fp64 oracle's gradients of the definition.

The three forms of the forward are one function, so `ko.kata_quadratic_bwd` is the reference on short sequences;
on long ones `ko.kata_bwd_rows` gives the same gradients for sampled tokens (pinned against `kata_quadratic_bwd`
in the CPU tests), and the quadratic-form backward kernel gives every element.

Tolerance: max |g - r| <= tol * max(1, max |r|) per gradient tensor, tol = 1e-4 for fp32 inputs and 2e-2 for bf16
inputs (the arithmetic is fp32 either way; bf16 gradients are rounded once on store)."""
import numpy as np
import pytest

from oracle import kata_oracle as ko
from paper_2607_17419_b200 import binding as kb
from paper_2607_17419_b200 import inputs

from helpers import dev_tensors, to_numpy64
from test_gpu_backward import TOL, dout_for

pytestmark = pytest.mark.gpu


def run_bwd(w, seed=5, **kw):
    import torch
    q, k, v = dev_tensors(w)
    g_dev, g_ref = dout_for(w, seed)
    dq, dk, dv = kb.kata_bwd_chunked(q, k, v, g_dev, **kw)
    torch.cuda.synchronize()
    assert kb.kata_last_impl() == kb.KATA_IMPL_SIMT
    # two normalisations, the forward sweep, dq, the reverse sweep, dk
    assert kb.kata_last_launch_count() == 6
    return (q, k, v, g_dev), g_ref, (dq, dk, dv)


def close(got, ref, tol, what):
    assert np.all(np.isfinite(got)), what
    err = np.max(np.abs(got - ref))
    assert err <= tol * max(1.0, np.abs(ref).max()), f"{what}: {err:.3e} vs scale {np.abs(ref).max():.3e}"


@pytest.mark.parametrize("dtype,dk,dv", [("f32", 16, 16), ("f32", 32, 64), ("f32", 64, 8), ("f32", 64, 64),
                                         ("bf16", 64, 64), ("bf16", 32, 16), ("bf16", 16, 64)])
@pytest.mark.parametrize("T", [1, 63, 64, 65, 200, 449])
def test_backward_chunked_short(dtype, dk, dv, T):
    w = inputs.gaussian_workload(f"bwdc_{dtype}_{dk}_{dv}_{T}", dtype, 1, 2, T, dk, dv, 64, 1800 + T + dk)
    _, g_ref, grads = run_bwd(w)
    for b in range(w.B):
        for h in range(w.H):
            ref = ko.kata_quadratic_bwd(w.q_ref[b, h], w.k_ref[b, h], w.v_ref[b, h], g_ref[b, h])
            for name, got, r in zip(("dq", "dk", "dv"), grads, ref):
                close(to_numpy64(got[b, h]), r, TOL[dtype], f"{name} ({b},{h}) T={T}")


def test_backward_chunked_degenerate_rows():
    """Zero key rows and zero query rows (zero feature, zero gradient), a first key of zero (normaliser 0 on the
    first row: out = 0 there and nothing flows back), repeated keys."""
    w = inputs.gaussian_workload("bwdc_degenerate", "f32", 1, 1, 130, 64, 64, 64, 1999)
    for arr in (w.k_ref, w.k_dev):
        arr[0, 0, 0] = 0
        arr[0, 0, 70] = 0
        arr[0, 0, 100] = arr[0, 0, 99]
    for arr in (w.q_ref, w.q_dev):
        arr[0, 0, 64] = 0
    _, g_ref, grads = run_bwd(w)
    ref = ko.kata_quadratic_bwd(w.q_ref[0, 0], w.k_ref[0, 0], w.v_ref[0, 0], g_ref[0, 0])
    for name, got, r in zip(("dq", "dk", "dv"), grads, ref):
        close(to_numpy64(got[0, 0]), r, TOL["f32"], name)
    assert np.all(to_numpy64(grads[1][0, 0])[[0, 70]] == 0) and np.all(to_numpy64(grads[0][0, 0])[64] == 0)
    assert np.all(to_numpy64(grads[0][0, 0])[0] == 0), "row 0 has a zero normaliser"


def test_backward_chunked_is_reproducible_and_batched():
    import torch
    w = inputs.gaussian_workload("bwdc_batch", "bf16", 3, 5, 300, 64, 64, 64, 2024)
    _, g_ref, a = run_bwd(w)
    _, _, b = run_bwd(w)
    for x, y in zip(a, b):
        assert torch.equal(x, y)
    for bb, h in ((0, 0), (2, 4), (1, 3)):
        ref = ko.kata_quadratic_bwd(w.q_ref[bb, h], w.k_ref[bb, h], w.v_ref[bb, h], g_ref[bb, h])
        for name, got, r in zip(("dq", "dk", "dv"), a, ref):
            close(to_numpy64(got[bb, h]), r, TOL["bf16"], f"{name} ({bb},{h})")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_backward_chunked_T32768_full_heads(dtype):
    """T = 32768: every element of both heads against the quadratic-form backward kernel (an independent kernel,
    itself checked against the oracle), 128 sampled tokens of head 0 against the oracle."""
    import torch
    T = 32768
    w = inputs.gaussian_workload(f"bwdc_long_{dtype}", dtype, 1, 2, T, 64, 64, 64, 3100)
    (q, k, v, g_dev), g_ref, grads = run_bwd(w)
    quad = kb.kata_bwd_quadratic(q, k, v, g_dev)
    torch.cuda.synchronize()
    tol = TOL[dtype]
    for name, got, other in zip(("dq", "dk", "dv"), grads, quad):
        close(to_numpy64(got), to_numpy64(other), 2 * tol if dtype == "bf16" else tol, f"{name} vs quadratic backward")
    r = np.random.default_rng(5)
    rows = sorted(set([0, 1, 63, 64, T - 1, T - 64, T - 65] + [int(x) for x in r.integers(T, size=121)]))
    rq, rk, rv = ko.kata_bwd_rows(w.q_ref[0, 0], w.k_ref[0, 0], w.v_ref[0, 0], g_ref[0, 0], rows, rows)
    for name, got, ref in zip(("dq", "dk", "dv"), grads, (rq, rk, rv)):
        close(to_numpy64(got[0, 0])[rows], ref, tol, f"{name} sampled rows")


def test_backward_chunked_config4_sampled_rows():
    """Config 4 at T = 131072 (16 heads, bf16): sampled tokens of one head against the oracle."""
    T = 131072
    w = inputs.config(4, T)
    _, g_ref, grads = run_bwd(w)
    h = 9
    r = np.random.default_rng(11)
    rows = sorted(set([0, 64, T - 1, T - 100] + [int(x) for x in r.integers(T, size=44)]))
    rq, rk, rv = ko.kata_bwd_rows(w.q_ref[0, h], w.k_ref[0, h], w.v_ref[0, h], g_ref[0, h], rows, rows)
    for name, got, ref in zip(("dq", "dk", "dv"), grads, (rq, rk, rv)):
        g = to_numpy64(got[0, h])
        assert np.all(np.isfinite(to_numpy64(got)))
        close(g[rows], ref, TOL["bf16"], f"{name} sampled rows")


def test_backward_chunked_rejects_what_it_does_not_do():
    import torch
    w = inputs.gaussian_workload("bwdc_reject", "f32", 1, 1, 64, 64, 64, 64, 1)
    q, k, v = dev_tensors(w)
    for kw in (dict(feature_order=1), dict(feature_groups=2), dict(impl=kb.KATA_IMPL_TENSOR), dict(C=128)):
        with pytest.raises(kb.KataError):
            kb.kata_bwd_chunked(q, k, v, torch.zeros_like(v), **kw)
