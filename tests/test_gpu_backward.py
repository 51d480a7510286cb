"""GPU parity of the backward pass (kata_bwd_quadratic) against the fp64 oracle's gradients of the definition.

Tolerance: max |g - r| <= tol * max(1, max |r|) per gradient tensor, tol = 1e-4 for fp32 inputs and 2e-2 for bf16
inputs (the gradients are sums of signed terms, so the error is measured against the largest entry)."""
import numpy as np
import pytest

from oracle import kata_oracle as ko
from paper_2607_17419_b200 import binding as kb
from paper_2607_17419_b200 import inputs

from helpers import dev_tensors, to_numpy64, to_torch

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-4, "bf16": 2e-2}


def dout_for(w, seed):
    """Seeded upstream gradient in the workload's dtype: device tensor and its exact fp64 value."""
    d = inputs.normal(seed, 7, w.B * w.H * w.T * w.d_v).reshape(w.B, w.H, w.T, w.d_v)
    if w.dtype == "bf16":
        bits = inputs.f32_to_bf16_bits(d.astype(np.float32)).reshape(d.shape)
        return to_torch(bits, "bf16"), inputs.bf16_bits_to_f64(bits)
    d32 = d.astype(np.float32)
    return to_torch(d32, "f32"), d32.astype(np.float64)


def check_grads(w, feature, seed=5, **kw):
    import torch
    q, k, v = dev_tensors(w)
    g_dev, g_ref = dout_for(w, seed)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    dq, dk, dv = kb.kata_bwd_quadratic(q, k, v, g_dev, device_status=st, **kw)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    # tensor-core kernels for bf16 and the full rank-one feature (pre-pass, dq with the row scalars, dk/dv); rows
    # narrower than 64 are zero-padded (four copies in, three out)
    tensor = (w.dtype == "bf16" and kw.get("impl", kb.KATA_IMPL_AUTO) != kb.KATA_IMPL_SIMT and
              (feature == "psd_direct" or (feature.startswith("psd_direct:g") and w.d_k == 64 and w.d_v == 64)))
    padded = tensor and (w.d_k < 64 or w.d_v < 64)
    assert kb.kata_last_impl() == (kb.KATA_IMPL_TENSOR if tensor else kb.KATA_IMPL_SIMT)
    assert kb.kata_last_launch_count() == (10 if padded else 3 if tensor else 2)
    tol = TOL[w.dtype]
    for b in range(w.B):
        for h in range(w.H):
            rq, rk, rv = ko.kata_quadratic_bwd(w.q_ref[b, h], w.k_ref[b, h], w.v_ref[b, h], g_ref[b, h], feature)
            for name, got, ref in (("dq", dq, rq), ("dk", dk, rk), ("dv", dv, rv)):
                g = to_numpy64(got[b, h])
                assert np.all(np.isfinite(g)), name
                err = np.max(np.abs(g - ref))
                assert err <= tol * max(1.0, np.abs(ref).max()), f"{name} ({b},{h}) {feature}: {err:.3e}"
    return dq, dk, dv


@pytest.mark.parametrize("dtype,dk,dv", [("f32", 16, 16), ("f32", 32, 64), ("f32", 64, 32), ("f32", 64, 64),
                                         ("bf16", 64, 64), ("bf16", 32, 16), ("bf16", 16, 64), ("bf16", 32, 32)])
@pytest.mark.parametrize("T", [1, 63, 64, 65, 200])
def test_backward_psd(dtype, dk, dv, T):
    w = inputs.gaussian_workload(f"bwd_{dtype}_{dk}_{dv}_{T}", dtype, 1, 2, T, dk, dv, 64, 800 + T + dk)
    check_grads(w, "psd_direct")


@pytest.mark.parametrize("T", [1, 2, 63, 64, 65, 127, 128, 129, 191, 192, 193, 257, 600])
def test_backward_tensor_tile_boundaries(T):
    """Tensor-core kernels: fixed tiles of 128 rows, streamed tiles of 64; and the fp32 kernels on the same inputs."""
    w = inputs.gaussian_workload(f"bwd_tc_{T}", "bf16", 1, 2, T, 64, 64, 64, 860 + T)
    a = check_grads(w, "psd_direct")
    b = check_grads(w, "psd_direct", impl=kb.KATA_IMPL_SIMT)
    for x, y in zip(a, b):
        assert float((x.float() - y.float()).abs().max()) <= 4e-2 * max(1.0, float(y.float().abs().max()))


def test_backward_tensor_zero_rows():
    import torch
    T = 300
    w = inputs.gaussian_workload("bwd_tc_zero", "bf16", 1, 1, T, 64, 64, 64, 870)
    for t in (0, 1, 64, 127, 128, 200):
        w.k_dev[0, 0, t] = 0
        w.k_ref[0, 0, t] = 0
    for t in (0, 5, 128, 256):
        w.q_dev[0, 0, t] = 0
        w.q_ref[0, 0, t] = 0
    dq, dk, dv = check_grads(w, "psd_direct")
    assert torch.all(dk[0, 0, [0, 1, 64, 127, 128, 200]] == 0) and torch.all(dv[0, 0, [0, 1, 64, 127, 128, 200]] == 0)
    assert torch.all(dq[0, 0, [0, 1, 5, 128, 256]] == 0)
    dq2, dk2, dv2 = check_grads(w, "psd_direct")
    assert torch.equal(dq, dq2) and torch.equal(dk, dk2) and torch.equal(dv, dv2)      # fixed summation order


@pytest.mark.parametrize("g", [2, 4])
@pytest.mark.parametrize("T", [1, 63, 64, 65, 128, 129, 200, 257, 600])
def test_backward_blockwise_tensor_tile_boundaries(g, T):
    """Blockwise map on the tensor-core backward kernels (bf16, d = 64), and the fp32 kernels on the same inputs."""
    w = inputs.gaussian_workload(f"bwd_tc_mg_{T}", "bf16", 1, 2, T, 64, 64, 64, 880 + T + g)
    a = check_grads(w, f"psd_direct:g{g}", feature_groups=g)
    b = check_grads(w, f"psd_direct:g{g}", feature_groups=g, impl=kb.KATA_IMPL_SIMT)
    for x, y in zip(a, b):
        assert float((x.float() - y.float()).abs().max()) <= 4e-2 * max(1.0, float(y.float().abs().max()))


@pytest.mark.parametrize("g", [2, 4])
@pytest.mark.parametrize("dtype,d", [("f32", 16), ("f32", 64), ("bf16", 64)])
def test_backward_blockwise(g, dtype, d):
    w = inputs.gaussian_workload(f"bwd_mg_{dtype}_{d}_{g}", dtype, 2, 2, 150, d, d, 64, 820 + d + g)
    check_grads(w, f"psd_direct:g{g}", feature_groups=g)


@pytest.mark.parametrize("dtype,d", [("f32", 32), ("bf16", 64)])
def test_backward_first_order(dtype, d):
    w = inputs.nonnegative_workload(f"bwd_o1_{dtype}_{d}", dtype, 1, 2, 180, d, d, 64, 830 + d)
    check_grads(w, "identity", feature_order=1)


def test_backward_zero_rows_and_reproducibility():
    import torch
    T, d = 140, 32
    w = inputs.gaussian_workload("bwd_zero", "f32", 1, 1, T, d, d, 64, 840)
    w.k_dev[0, 0, [0, 1, 64, 70]] = 0
    w.q_dev[0, 0, [0, 5, 65]] = 0
    w.k_ref[0, 0, [0, 1, 64, 70]] = 0
    w.q_ref[0, 0, [0, 5, 65]] = 0
    dq, dk, dv = check_grads(w, "psd_direct")
    assert torch.all(dk[0, 0, [0, 1, 64, 70]] == 0) and torch.all(dq[0, 0, [0, 1, 5, 65]] == 0)
    assert torch.all(dv[0, 0, [0, 1, 64, 70]] == 0)
    dq2, dk2, dv2 = check_grads(w, "psd_direct")
    assert torch.equal(dq, dq2) and torch.equal(dk, dk2) and torch.equal(dv, dv2)      # fixed summation order


def test_backward_is_the_gradient_of_the_gpu_forward():
    """Directional derivative of the GPU forward (fp32 kernels) along a random direction against <grad, direction>."""
    import torch
    w = inputs.gaussian_workload("bwd_dir", "f32", 1, 2, 96, 32, 32, 64, 850)
    q, k, v = dev_tensors(w)
    g_dev, _ = dout_for(w, 9)
    dq, dk, dv = kb.kata_bwd_quadratic(q, k, v, g_dev)
    gen = torch.Generator(device="cuda").manual_seed(1)
    uq, uk, uv = (torch.randn(x.shape, device="cuda", generator=gen) for x in (q, k, v))
    h = 2e-3
    lp = (kb.kata_fwd_quadratic(q + h * uq, k + h * uk, v + h * uv).double() * g_dev.double()).sum()
    lm = (kb.kata_fwd_quadratic(q - h * uq, k - h * uk, v - h * uv).double() * g_dev.double()).sum()
    num = float((lp - lm) / (2 * h))
    ana = float((dq.double() * uq).sum() + (dk.double() * uk).sum() + (dv.double() * uv).sum())
    assert abs(num - ana) <= 2e-3 * max(1.0, abs(ana))


def test_backward_argument_checks():
    import torch
    w = inputs.gaussian_workload("bwd_args", "bf16", 1, 1, 64, 64, 64, 64, 1)
    q, k, v = dev_tensors(w)
    with pytest.raises(kb.KataError):
        kb.kata_bwd_quadratic(q, k, v, v, impl=kb.KATA_IMPL_TENSOR, feature_order=1)     # fp32 kernels only
    with pytest.raises(kb.KataError):
        kb.kata_bwd_quadratic(q, k, v, v, feature_groups=3)


def test_backward_config2_full_size_heads():
    """The benchmark shape (B=4, H=16, T=4096, d=64, bf16): every row of two heads against the oracle."""
    import torch
    w = inputs.config(2)
    q, k, v = dev_tensors(w)
    g_dev, g_ref = dout_for(w, 11)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    dq, dk, dv = kb.kata_bwd_quadratic(q, k, v, g_dev, device_status=st)
    torch.cuda.synchronize()
    assert kb.kata_last_impl() == kb.KATA_IMPL_TENSOR and int(st.item()) == 0
    for b, h in ((0, 0), (3, 15)):
        rq, rk, rv = ko.kata_quadratic_bwd(w.q_ref[b, h], w.k_ref[b, h], w.v_ref[b, h], g_ref[b, h])
        for name, got, ref in (("dq", dq, rq), ("dk", dk, rk), ("dv", dv, rv)):
            gg = to_numpy64(got[b, h])
            assert np.all(np.isfinite(gg))
            err = np.max(np.abs(gg - ref))
            assert err <= 2e-2 * max(1.0, np.abs(ref).max()), f"{name} ({b},{h}): {err:.3e}"
