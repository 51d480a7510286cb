"""GPU parity of the zero-padded tensor-core path: bf16 inputs whose rows are narrower than 64 entries are padded
to 64 (dot products, norms and the kept output columns are unchanged) and run on the d = 64 kernels."""
import numpy as np
import pytest

from oracle import kata_oracle as ko
from paper_2607_17419_b200 import binding as kb
from paper_2607_17419_b200 import inputs

from helpers import check, dev_tensors, to_numpy64

pytestmark = pytest.mark.gpu

FORMS = {
    "quadratic": lambda q, k, v, **kw: kb.kata_fwd_quadratic(q, k, v, **kw),
    "chunked_seq": lambda q, k, v, **kw: kb.kata_fwd_chunked(q, k, v, inter_chunk=kb.KATA_SEQUENTIAL, **kw),
    "chunked_scan": lambda q, k, v, **kw: kb.kata_fwd_chunked(q, k, v, inter_chunk=kb.KATA_SCAN, **kw),
    "state_scan": lambda q, k, v, **kw: kb.kata_chunk_state_scan(q, k, v, **kw),
}
SHAPES = [(16, 16), (32, 32), (32, 64), (64, 16), (16, 64), (64, 32)]


@pytest.mark.parametrize("form", list(FORMS))
@pytest.mark.parametrize("dk,dv", SHAPES)
def test_padded_psd(form, dk, dv):
    import torch
    w = inputs.gaussian_workload(f"pad_{dk}_{dv}", "bf16", 2, 2, 333, dk, dv, 64, 900 + dk + dv)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    o = FORMS[form](*dev_tensors(w), device_status=st)
    torch.cuda.synchronize()
    assert kb.kata_last_impl() == kb.KATA_IMPL_TENSOR and int(st.item()) == 0
    assert tuple(o.shape) == (2, 2, 333, dv)
    g = to_numpy64(o)
    for b in range(w.B):
        for h in range(w.H):
            ref = ko.kata_quadratic(w.q_ref[b, h], w.k_ref[b, h], w.v_ref[b, h])[0]
            check(g[b, h], ref, "bf16", f"padded {dk}x{dv}/{form} ({b},{h})")
    # the fp32 kernels on the same inputs
    o2 = FORMS[form](*dev_tensors(w), impl=kb.KATA_IMPL_SIMT)
    torch.cuda.synchronize()
    assert kb.kata_last_impl() == kb.KATA_IMPL_SIMT
    assert float((o.float() - o2.float()).abs().max()) <= 4e-2


@pytest.mark.parametrize("form", ["chunked_seq", "chunked_scan", "state_scan"])
@pytest.mark.parametrize("dk,dv", [(32, 32), (16, 64)])
def test_padded_first_order(form, dk, dv):
    import torch
    w = inputs.nonnegative_workload(f"pad_o1_{dk}_{dv}", "bf16", 1, 2, 400, dk, dv, 64, 950 + dk)
    o = FORMS[form](*dev_tensors(w), feature_order=1)
    torch.cuda.synchronize()
    assert kb.kata_last_impl() == kb.KATA_IMPL_TENSOR
    g = to_numpy64(o)
    for h in range(w.H):
        ref = ko.kata_quadratic(w.q_ref[0, h], w.k_ref[0, h], w.v_ref[0, h], "identity")[0]
        check(g[0, h], ref, "bf16", f"padded first order {dk}x{dv}/{form} head {h}")


def test_padding_is_not_used_where_the_width_matters():
    """Feature blocks and state layouts depend on the true width: those calls stay on the fp32 kernels."""
    import torch
    w = inputs.gaussian_workload("pad_not", "bf16", 1, 1, 128, 32, 32, 64, 5)
    q, k, v = dev_tensors(w)
    kb.kata_fwd_quadratic(q, k, v, feature_groups=2)
    assert kb.kata_last_impl() == kb.KATA_IMPL_SIMT
    n = kb.decode_n_psi(32)
    S, Z = torch.empty(1, 1, n, 32, device="cuda"), torch.empty(1, 1, n, device="cuda")
    kb.kata_fwd_chunked(q, k, v, s_pre=S, z_pre=Z)
    assert kb.kata_last_impl() == kb.KATA_IMPL_SIMT
    with pytest.raises(kb.KataError):
        kb.kata_fwd_quadratic(q, k, v, feature_groups=2, impl=kb.KATA_IMPL_TENSOR)


def test_padded_host_io_entry_matches_device_entry():
    """Host buffers in, host buffer out, rows padded inside the workspace: the same bits as the device entry."""
    import torch
    w = inputs.gaussian_workload("pad_host", "bf16", 2, 2, 300, 32, 16, 64, 61)
    q, k, v = dev_tensors(w)
    for fn, call in ((kb.KATA_FN_QUADRATIC, kb.kata_fwd_quadratic), (kb.KATA_FN_CHUNKED, kb.kata_fwd_chunked),
                     (kb.KATA_FN_CHUNK_STATE_SCAN, kb.kata_chunk_state_scan)):
        ref = call(q, k, v)
        assert kb.kata_last_impl() == kb.KATA_IMPL_TENSOR
        hq, hk, hv = (t.cpu().pin_memory() for t in (q, k, v))
        ho = torch.empty_like(hv).pin_memory()
        kb.kata_fwd_host(fn, hq, hk, hv, ho)
        torch.cuda.synchronize()
        assert kb.kata_last_impl() == kb.KATA_IMPL_TENSOR
        assert torch.equal(ho, ref.cpu())
