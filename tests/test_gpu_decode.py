"""GPU parity of kata_decode_step against the fp64 oracle: from a zero state, resumed from an exported prefix
state (prefill -> decode hand-off), zero rows, every state layout."""
import numpy as np
import pytest

from oracle import kata_oracle as ko
from paper_2607_17419_b200 import binding as kb
from paper_2607_17419_b200 import inputs

from helpers import TOL, check, dev_tensors, to_numpy64

pytestmark = pytest.mark.gpu

FEATURES = {"psd_direct": dict(feature_order=2, state_layout=kb.KATA_LAYOUT_DIRECT),
            "psd_packed": dict(feature_order=2, state_layout=kb.KATA_LAYOUT_PACKED),
            "identity": dict(feature_order=1)}


def decode_all(q, k, v, S, Z, t0, t1, **opts):
    """Feed tokens t0..t1-1 of [B,H,T,d] tensors one by one; returns [B,H,t1-t0,d_v] (float64)."""
    import torch
    outs = []
    for t in range(t0, t1):
        o = kb.kata_decode_step(q[:, :, t].contiguous(), k[:, :, t].contiguous(), v[:, :, t].contiguous(), S, Z, **opts)
        outs.append(o.float())
    torch.cuda.synchronize()
    return torch.stack(outs, dim=2).cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("feature", list(FEATURES))
@pytest.mark.parametrize("dtype,dk,dv", [("f32", 16, 16), ("f32", 32, 64), ("f32", 64, 64), ("bf16", 64, 64), ("bf16", 32, 16)])
def test_decode_from_zero_state(feature, dtype, dk, dv):
    import torch
    B, H, T = 2, 3, 40
    w = (inputs.nonnegative_workload if feature == "identity" else inputs.gaussian_workload)(
        f"dec_{feature}_{dtype}_{dk}_{dv}", dtype, B, H, T, dk, dv, 64, 50 + dk + dv)
    q, k, v = dev_tensors(w)
    n = kb.decode_n_psi(dk, **FEATURES[feature])
    S = torch.zeros(B, H, n, dv, device="cuda")
    Z = torch.zeros(B, H, n, device="cuda")
    g = decode_all(q, k, v, S, Z, 0, T, **FEATURES[feature])
    for b in range(B):
        for h in range(H):
            ref = ko.kata_quadratic(w.q_ref[b, h], w.k_ref[b, h], w.v_ref[b, h], feature)[0]
            check(g[b, h], ref, dtype, f"decode/{feature} ({b},{h})")
            # the state after T tokens is the plain sum of feature-value outer products (fp32 accumulation)
            fk = ko.apply_feature(w.k_ref[b, h], feature)
            Sr, Zr = fk.T @ w.v_ref[b, h], fk.sum(axis=0)
            assert np.max(np.abs(to_numpy64(S[b, h]) - Sr)) <= 1e-4 * max(1.0, np.abs(Sr).max())
            assert np.max(np.abs(to_numpy64(Z[b, h]) - Zr)) <= 1e-4 * max(1.0, np.abs(Zr).max())


@pytest.mark.parametrize("layout", ["psd_direct", "psd_packed"])
def test_prefill_then_decode(layout):
    """Resume from the prefix state that the scan pipeline exports for a chunk and decode that chunk's tokens:
    the outputs are those of the forward pass over the whole sequence."""
    import torch
    w = inputs.gaussian_workload("handoff", "f32", 1, 2, 200, 32, 32, 64, 77)
    q, k, v = dev_tensors(w)
    NC = (w.T + 63) // 64
    n = kb.decode_n_psi(32, **FEATURES[layout])
    s_pre = torch.empty(1, 2, NC, n, 32, device="cuda")
    z_pre = torch.empty(1, 2, NC, n, device="cuda")
    fwd = kb.kata_chunk_state_scan(q, k, v, s_pre=s_pre, z_pre=z_pre, state_layout=FEATURES[layout]["state_layout"])
    c = NC - 1                                   # the last (ragged) chunk: tokens 192..199
    S, Z = s_pre[:, :, c].contiguous(), z_pre[:, :, c].contiguous()
    g = decode_all(q, k, v, S, Z, 64 * c, w.T, **FEATURES[layout])
    for h in range(2):
        ref = ko.kata_quadratic(w.q_ref[0, h], w.k_ref[0, h], w.v_ref[0, h])[0][64 * c:]
        check(g[0, h], ref, "f32", f"hand-off/{layout} head {h}")
        assert np.max(np.abs(g[0, h] - to_numpy64(fwd)[0, h, 64 * c:])) <= 2 * TOL["f32"]


def test_decode_zero_rows_and_determinism():
    import torch
    B, H, d = 1, 2, 64
    r = np.random.default_rng(5)
    q = torch.from_numpy(r.standard_normal((B, H, d)).astype(np.float32)).cuda()
    k = torch.from_numpy(r.standard_normal((B, H, d)).astype(np.float32)).cuda()
    v = torch.from_numpy(r.standard_normal((B, H, d)).astype(np.float32)).cuda()
    S = torch.zeros(B, H, d * d, d, device="cuda")
    Z = torch.zeros(B, H, d * d, device="cuda")
    # zero key on an empty state: nothing is added, the denominator is 0, the output is 0 (never NaN)
    o = kb.kata_decode_step(q, torch.zeros_like(k), v, S, Z)
    assert torch.all(o == 0) and torch.all(S == 0) and torch.all(Z == 0)
    o1 = kb.kata_decode_step(q, k, v, S, Z)
    # a zero query reads 0 and still updates the state
    S2, Z2 = S.clone(), Z.clone()
    o2 = kb.kata_decode_step(torch.zeros_like(q), k, v, S2, Z2)
    assert torch.all(o2 == 0) and not torch.equal(S2, S)
    # first real token: o = v (weight 1 on itself), whatever q is, as long as q is not orthogonal to k
    assert torch.allclose(o1, v, atol=1e-5)
    # same call, same state: identical bits
    Sa, Za, Sb, Zb = S.clone(), Z.clone(), S.clone(), Z.clone()
    oa, ob = kb.kata_decode_step(q, k, v, Sa, Za), kb.kata_decode_step(q, k, v, Sb, Zb)
    torch.cuda.synchronize()
    assert torch.equal(oa, ob) and torch.equal(Sa, Sb) and torch.equal(Za, Zb)


@pytest.mark.parametrize("dtype,impl", [("f32", "simt"), ("bf16", "tensor"), ("bf16", "simt")])
@pytest.mark.parametrize("layout", ["psd_direct", "psd_packed"])
def test_final_state_of_the_chunked_forward(dtype, impl, layout):
    """kata_fwd_chunked (sequential) exports the state after the last token; decoding on from it gives the
    forward pass over the longer sequence."""
    import torch
    B, H, T, Tp, d = 1, 2, 300, 270, 64           # prefill 270 tokens (ragged: 2 tiles + 14), decode 30 more
    w = inputs.gaussian_workload("prefill", dtype, B, H, T, d, d, 64, 91)
    q, k, v = dev_tensors(w)
    n = kb.decode_n_psi(d, **FEATURES[layout])
    S = torch.full((B, H, n, d), float("nan"), device="cuda")
    Z = torch.full((B, H, n), float("nan"), device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    o = kb.kata_fwd_chunked(q[:, :, :Tp].contiguous(), k[:, :, :Tp].contiguous(), v[:, :, :Tp].contiguous(),
                            s_pre=S, z_pre=Z, state_layout=FEATURES[layout]["state_layout"], device_status=st,
                            impl=kb.KATA_IMPL_SIMT if impl == "simt" else kb.KATA_IMPL_TENSOR)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    assert (kb.kata_last_impl() == kb.KATA_IMPL_TENSOR) == (impl == "tensor")
    g_pre = to_numpy64(o)
    # bf16 W rows on the tensor path: the state carries the rounding of the per-token products
    tol_state = 1e-4 if dtype == "f32" else 1e-2
    for h in range(H):
        ref = ko.kata_quadratic(w.q_ref[0, h], w.k_ref[0, h], w.v_ref[0, h])[0]
        check(g_pre[0, h], ref[:Tp], dtype, f"prefill {impl}/{layout}")
        fk = ko.apply_feature(w.k_ref[0, h, :Tp], layout)
        Sr, Zr = fk.T @ w.v_ref[0, h, :Tp], fk.sum(axis=0)
        assert np.all(np.isfinite(to_numpy64(S[0, h]))) and np.all(np.isfinite(to_numpy64(Z[0, h])))
        assert np.max(np.abs(to_numpy64(S[0, h]) - Sr)) <= tol_state * max(1.0, np.abs(Sr).max())
        assert np.max(np.abs(to_numpy64(Z[0, h]) - Zr)) <= tol_state * max(1.0, np.abs(Zr).max())
    g = decode_all(q, k, v, S, Z, Tp, T, **FEATURES[layout])
    for h in range(H):
        ref = ko.kata_quadratic(w.q_ref[0, h], w.k_ref[0, h], w.v_ref[0, h])[0]
        check(g[0, h], ref[Tp:], dtype, f"decode after prefill {impl}/{layout}")
