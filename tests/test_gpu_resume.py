"""GPU parity of the state hand-off of the sequential chunked forward: a sequence fed in pieces, each call
starting from the state the previous call left (``s_init/z_init`` <- ``s_pre/z_pre``), gives the outputs of the
definition on the whole sequence; the last state equals the sum of the lifted keys."""
import numpy as np
import pytest

from oracle import kata_oracle as ko
from paper_2607_17419_b200 import binding as kb
from paper_2607_17419_b200 import inputs

from helpers import check, dev_tensors, to_numpy64

pytestmark = pytest.mark.gpu


def run_pieces(w, cuts, layout, g=0, in_place=False, impl=kb.KATA_IMPL_AUTO):
    import torch
    q, k, v = dev_tensors(w)
    code = kb.KATA_LAYOUT_PACKED if layout == "psd_packed" else kb.KATA_LAYOUT_DIRECT
    n = kb.decode_n_psi(w.d_k, 2, code, g)
    S = [torch.zeros(w.B, w.H, n, w.d_v, device="cuda") for _ in range(2)]
    Z = [torch.zeros(w.B, w.H, n, device="cuda") for _ in range(2)]
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    outs, impls = [], set()
    edges = [0] + list(cuts) + [w.T]
    cur = 0
    for i in range(len(edges) - 1):
        a, b = edges[i], edges[i + 1]
        nxt = cur if in_place else 1 - cur
        kw = dict(s_pre=S[nxt], z_pre=Z[nxt], state_layout=code, feature_groups=g, device_status=st, impl=impl)
        if i > 0:                       # the first piece starts from the zero state (no s_init)
            kw.update(s_init=S[cur], z_init=Z[cur])
        outs.append(kb.kata_fwd_chunked(q[:, :, a:b].contiguous(), k[:, :, a:b].contiguous(),
                                        v[:, :, a:b].contiguous(), **kw))
        impls.add(kb.kata_last_impl())
        cur = nxt
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    return torch.cat(outs, dim=2), S[cur], Z[cur], impls


def check_against_definition(w, o, S, Z, feat):
    gpu = to_numpy64(o)
    for b in range(w.B):
        for h in range(w.H):
            ref = ko.kata_quadratic(w.q_ref[b, h], w.k_ref[b, h], w.v_ref[b, h], feat)[0]
            check(gpu[b, h], ref, w.dtype, f"pieces ({b},{h}) {feat}")
            fk = ko.apply_feature(w.k_ref[b, h], feat)
            Sr, Zr = fk.T @ w.v_ref[b, h], fk.sum(axis=0)
            tol = 1e-4 if w.dtype == "f32" else 2e-2
            assert np.max(np.abs(to_numpy64(S[b, h]) - Sr)) <= tol * max(1.0, np.abs(Sr).max())
            assert np.max(np.abs(to_numpy64(Z[b, h]) - Zr)) <= tol * max(1.0, np.abs(Zr).max())


@pytest.mark.parametrize("layout", ["psd_direct", "psd_packed"])
@pytest.mark.parametrize("cuts", [(128,), (1,), (100, 101, 390), (64, 257, 511)])
def test_resume_tensor(layout, cuts):
    """bf16, d = 64: the tensor-core kernel loads the state into its TMEM accumulators before the first tile."""
    w = inputs.gaussian_workload("resume_tc", "bf16", 1, 2, 700, 64, 64, 64, 41)
    o, S, Z, impls = run_pieces(w, cuts, layout)
    assert impls == {kb.KATA_IMPL_TENSOR}
    check_against_definition(w, o, S, Z, layout)


@pytest.mark.parametrize("in_place", [False, True])
def test_resume_tensor_in_place_and_simt_agree(in_place):
    w = inputs.gaussian_workload("resume_tc2", "bf16", 2, 2, 450, 64, 64, 64, 43)
    o, S, Z, impls = run_pieces(w, (200, 333), "psd_packed", in_place=in_place)
    assert impls == {kb.KATA_IMPL_TENSOR}
    check_against_definition(w, o, S, Z, "psd_packed")
    o2, S2, Z2, impls2 = run_pieces(w, (200, 333), "psd_packed", in_place=in_place, impl=kb.KATA_IMPL_SIMT)
    assert impls2 == {kb.KATA_IMPL_SIMT}
    assert float((o.float() - o2.float()).abs().max()) <= 4e-2
    assert float((S - S2).abs().max()) <= 2e-2 * max(1.0, float(S2.abs().max()))


@pytest.mark.parametrize("dtype,dk,dv,g", [("f32", 16, 16, 0), ("f32", 32, 64, 0), ("f32", 64, 32, 0), ("f32", 32, 16, 2),
                                           ("f32", 64, 16, 4), ("bf16", 32, 32, 0), ("bf16", 32, 64, 2)])
@pytest.mark.parametrize("layout", ["psd_direct", "psd_packed"])
def test_resume_simt(dtype, dk, dv, g, layout):
    """fp32 kernels (every shape; the blockwise map hands its state over through them)."""
    w = inputs.gaussian_workload("resume_simt", dtype, 1, 2, 230, dk, dv, 64, 47 + dk + g)
    o, S, Z, impls = run_pieces(w, (64, 65, 150), layout, g=g, in_place=(dk == 32))
    assert impls == {kb.KATA_IMPL_SIMT}
    feat = layout + (f":g{g}" if g else "")
    check_against_definition(w, o, S, Z, feat)


def test_resume_then_decode_matches_one_call():
    """Prefill in two pieces, then decode steps: the same outputs as one chunked call over everything."""
    import torch
    w = inputs.gaussian_workload("resume_dec", "bf16", 1, 2, 300, 64, 64, 64, 53)
    q, k, v = dev_tensors(w)
    o, S, Z, _ = run_pieces(inputs.gaussian_workload("resume_dec", "bf16", 1, 2, 300, 64, 64, 64, 53), (129,), "psd_direct")
    # the state after 300 tokens continues with decode steps on fresh tokens
    w2 = inputs.gaussian_workload("resume_dec_tail", "bf16", 1, 2, 8, 64, 64, 64, 54)
    q2, k2, v2 = dev_tensors(w2)
    outs = [kb.kata_decode_step(q2[:, :, t].contiguous(), k2[:, :, t].contiguous(), v2[:, :, t].contiguous(), S, Z).float()
            for t in range(8)]
    torch.cuda.synchronize()
    dec = torch.stack(outs, dim=2).cpu().numpy().astype(np.float64)
    for h in range(2):
        qq = np.concatenate([w.q_ref[0, h], w2.q_ref[0, h]])
        kk = np.concatenate([w.k_ref[0, h], w2.k_ref[0, h]])
        vv = np.concatenate([w.v_ref[0, h], w2.v_ref[0, h]])
        ref = ko.kata_quadratic(qq, kk, vv)[0]
        check(to_numpy64(o)[0, h], ref[:300], "bf16", "prefill in pieces")
        check(dec[0, h], ref[300:], "bf16", "decode after pieces")


def test_resume_argument_checks():
    import torch
    w = inputs.gaussian_workload("resume_args", "f32", 1, 1, 64, 16, 16, 64, 1)
    q, k, v = dev_tensors(w)
    n = kb.decode_n_psi(16)
    S, Z = torch.zeros(1, 1, n, 16, device="cuda"), torch.zeros(1, 1, n, device="cuda")
    with pytest.raises(kb.KataError):
        kb.kata_fwd_chunked(q, k, v, s_init=S)                                   # both or neither
    with pytest.raises(kb.KataError):
        kb.kata_fwd_chunked(q, k, v, s_init=S, z_init=Z, inter_chunk=kb.KATA_SCAN)
    with pytest.raises(kb.KataError):
        kb.kata_fwd_quadratic(q, k, v, s_init=S, z_init=Z)
    with pytest.raises(kb.KataError):
        kb.kata_chunk_state_scan(q, k, v, s_init=S, z_init=Z)
    with pytest.raises(kb.KataError):
        kb.kata_fwd_chunked(q, k, v, s_init=S, z_init=Z, feature_order=1)


def test_resume_in_place_many_heads():
    """More CTAs than SMs (64 heads x 8 value slices): the slices of a head start at different times, and the
    state advanced in place must still be read before it is written."""
    import torch
    w = inputs.gaussian_workload("resume_many", "bf16", 4, 16, 384, 64, 64, 64, 59)
    a = run_pieces(w, (128, 256), "psd_direct", in_place=False)
    b = run_pieces(w, (128, 256), "psd_direct", in_place=True)
    assert a[3] == b[3] == {kb.KATA_IMPL_TENSOR}
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1]) and torch.equal(a[2], b[2])
    gpu = to_numpy64(b[0])
    for bb, h in ((0, 0), (3, 15)):
        ref = ko.kata_quadratic(w.q_ref[bb, h], w.k_ref[bb, h], w.v_ref[bb, h])[0]
        check(gpu[bb, h], ref, "bf16", f"in place, many heads ({bb},{h})")
