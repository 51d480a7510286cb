"""GPU parity of the blockwise PSD map (KATA-Mg, g = 2 or 4) against the fp64 oracle: every form, the exported
prefix states, the final state and the decode step."""
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
CASES = [("f32", 16, 16, 2), ("f32", 16, 32, 4), ("f32", 32, 16, 4), ("f32", 64, 64, 2), ("bf16", 64, 64, 2),
         ("bf16", 64, 64, 4), ("bf16", 32, 64, 2)]


@pytest.mark.parametrize("form", list(FORMS))
@pytest.mark.parametrize("dtype,dk,dv,g", CASES)
def test_blockwise_forms(form, dtype, dk, dv, g):
    import torch
    w = inputs.gaussian_workload(f"mg_{dtype}_{dk}_{dv}_{g}", dtype, 2, 2, 333, dk, dv, 64, 300 + dk + g)
    o = FORMS[form](*dev_tensors(w), feature_groups=g)
    torch.cuda.synchronize()
    # tensor-core kernels for the blockwise map (bf16, d = 64), every form
    tensor = (dtype, dk, dv) == ("bf16", 64, 64)
    assert kb.kata_last_impl() == (kb.KATA_IMPL_TENSOR if tensor else kb.KATA_IMPL_SIMT)
    gpu = to_numpy64(o)
    for b in range(w.B):
        for h in range(w.H):
            ref = ko.kata_quadratic(w.q_ref[b, h], w.k_ref[b, h], w.v_ref[b, h], f"psd_direct:g{g}")[0]
            check(gpu[b, h], ref, dtype, f"M{g}/{form} ({b},{h})")
    # g = 1 given explicitly is the plain feature
    o1, o0 = FORMS[form](*dev_tensors(w), feature_groups=1), FORMS[form](*dev_tensors(w))
    torch.cuda.synchronize()
    assert torch.equal(o1, o0)


@pytest.mark.parametrize("g", [2, 4])
@pytest.mark.parametrize("T", [1, 31, 32, 33, 64, 65, 127, 128, 129, 257, 640])
def test_blockwise_quadratic_tensor_tiles(g, T):
    """Tensor-core quadratic kernel: key tiles of 128 / g keys, the last g of them masked on the diagonal."""
    import torch
    w = inputs.gaussian_workload(f"mg_tc_{T}", "bf16", 1, 2, T, 64, 64, 64, 500 + T + g)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    o = kb.kata_fwd_quadratic(*dev_tensors(w), feature_groups=g, device_status=st)
    torch.cuda.synchronize()
    assert kb.kata_last_impl() == kb.KATA_IMPL_TENSOR and int(st.item()) == 0
    gpu = to_numpy64(o)
    for h in range(w.H):
        ref = ko.kata_quadratic(w.q_ref[0, h], w.k_ref[0, h], w.v_ref[0, h], f"psd_direct:g{g}")[0]
        check(gpu[0, h], ref, "bf16", f"M{g} tensor quadratic T={T} head {h}")
    # the fp32 SIMT kernel on the same inputs agrees to the bf16 tolerance
    o2 = kb.kata_fwd_quadratic(*dev_tensors(w), feature_groups=g, impl=kb.KATA_IMPL_SIMT)
    torch.cuda.synchronize()
    assert kb.kata_last_impl() == kb.KATA_IMPL_SIMT
    assert float((o.float() - o2.float()).abs().max()) <= 4e-2


@pytest.mark.parametrize("g", [2, 4])
@pytest.mark.parametrize("T", [1, 15, 16, 17, 33, 64, 127, 128, 129, 255, 256, 257, 385, 640, 1100])
def test_blockwise_chunked_tensor_tiles(g, T):
    """Tensor-core one-pass chunked kernel with the state blocks of the g feature groups only."""
    import torch
    w = inputs.gaussian_workload(f"mg_tcs_{T}", "bf16", 1, 2, T, 64, 64, 64, 600 + T + g)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    o = kb.kata_fwd_chunked(*dev_tensors(w), feature_groups=g, device_status=st)
    torch.cuda.synchronize()
    assert kb.kata_last_impl() == kb.KATA_IMPL_TENSOR and int(st.item()) == 0
    gpu = to_numpy64(o)
    for h in range(w.H):
        ref = ko.kata_quadratic(w.q_ref[0, h], w.k_ref[0, h], w.v_ref[0, h], f"psd_direct:g{g}")[0]
        check(gpu[0, h], ref, "bf16", f"M{g} tensor chunked T={T} head {h}")


@pytest.mark.parametrize("g,B,H,T", [(2, 1, 3, 1000), (2, 2, 16, 700), (2, 1, 14, 515), (4, 1, 2, 1300), (4, 3, 9, 520),
                                     (4, 2, 16, 900)])
def test_blockwise_chunked_head_layouts(g, B, H, T):
    """The feature-split kernel with the blockwise map: block pairs inside a feature group only, dealt to ten CTAs of
    two per head while ten per head fit the GPU in one wave (g = 2, B*H <= 14), to five of four beyond, to six of two
    for g = 4; CTAs of the five- and six-CTA layouts weigh two 16-key runs of a tile.  Several tiles, a ragged tail,
    grids of one and of several waves; and the same result run after run."""
    import torch
    w = inputs.gaussian_workload(f"mg_split_{g}_{B}_{H}_{T}", "bf16", B, H, T, 64, 64, 64, 4100 + T + g)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    o = kb.kata_fwd_chunked(*dev_tensors(w), feature_groups=g, device_status=st)
    torch.cuda.synchronize()
    assert kb.kata_last_impl() == kb.KATA_IMPL_TENSOR and int(st.item()) == 0
    assert kb.kata_last_launch_count() == 2, "the key-scale pre-pass and the feature-split kernel"
    o2 = kb.kata_fwd_chunked(*dev_tensors(w), feature_groups=g)
    torch.cuda.synchronize()
    assert torch.equal(o, o2)
    gpu = to_numpy64(o)
    for b in range(B):
        for h in range(0, H, max(1, H // 3)):
            ref = ko.kata_quadratic(w.q_ref[b, h], w.k_ref[b, h], w.v_ref[b, h], f"psd_direct:g{g}")[0]
            check(gpu[b, h], ref, "bf16", f"M{g} feature-split B{B} H{H} T={T} head ({b},{h})")


@pytest.mark.parametrize("form", ["quadratic", "chunked_seq"])
@pytest.mark.parametrize("g", [2, 4])
def test_blockwise_tensor_degenerate(form, g):
    """Zero keys and queries: zero feature, output 0 where the normaliser is 0."""
    T = 300
    w = inputs.gaussian_workload("mg_tc_deg", "bf16", 1, 1, T, 64, 64, 64, 77 + g)
    q, k, v = w.q_dev.copy(), w.k_dev.copy(), w.v_dev.copy()
    for t in (0, 1, 31, 32, 127, 128, 299):
        k[0, 0, t] = 0
    for t in (0, 5, 64, 128, 256):
        q[0, 0, t] = 0
    # one key that lives in a single block of the split: its other blocks are zero vectors
    k[0, 0, 40, 64 // g:] = 0
    from helpers import to_torch
    qr, kr, vr = (inputs.bf16_bits_to_f64(a[0, 0]) for a in (q, k, v))
    ref = ko.kata_quadratic(qr, kr, vr, f"psd_direct:g{g}")[0]
    o = FORMS[form](*(to_torch(a, "bf16") for a in (q, k, v)), feature_groups=g)
    assert kb.kata_last_impl() == kb.KATA_IMPL_TENSOR
    gpu = to_numpy64(o)
    check(gpu[0, 0], ref, "bf16", f"M{g} degenerate/{form}")
    assert np.all(gpu[0, 0, [0, 1, 5, 64, 128, 256]] == 0)


@pytest.mark.parametrize("layout", ["psd_direct", "psd_packed"])
@pytest.mark.parametrize("g", [2, 4])
def test_blockwise_states_and_decode(layout, g):
    """Exported prefix states, the final state of the sequential form, and decoding on from it."""
    import torch
    B, H, T, Tp, d, dv = 1, 2, 200, 150, 32, 16
    w = inputs.gaussian_workload("mg_state", "f32", B, H, T, d, dv, 64, 400 + g)
    q, k, v = dev_tensors(w)
    code = kb.KATA_LAYOUT_PACKED if layout == "psd_packed" else kb.KATA_LAYOUT_DIRECT
    feat = f"{layout}:g{g}"
    n = kb.decode_n_psi(d, 2, code, g)
    assert n == ko.feature_dim(d, feat)
    NC = (T + 63) // 64
    s_pre = torch.empty(B, H, NC, n, dv, device="cuda")
    z_pre = torch.empty(B, H, NC, n, device="cuda")
    kb.kata_chunk_state_scan(q, k, v, s_pre=s_pre, z_pre=z_pre, state_layout=code, feature_groups=g)
    S = torch.empty(B, H, n, dv, device="cuda")
    Z = torch.empty(B, H, n, device="cuda")
    kb.kata_fwd_chunked(q[:, :, :Tp].contiguous(), k[:, :, :Tp].contiguous(), v[:, :, :Tp].contiguous(),
                        s_pre=S, z_pre=Z, state_layout=code, feature_groups=g)
    torch.cuda.synchronize()
    for h in range(H):
        _, rs, rz = ko.kata_scan(w.q_ref[0, h], w.k_ref[0, h], w.v_ref[0, h], 64, feat)
        assert np.max(np.abs(to_numpy64(s_pre[0, h]) - rs)) <= 1e-5 * max(1.0, np.abs(rs).max())
        assert np.max(np.abs(to_numpy64(z_pre[0, h]) - rz)) <= 1e-5 * max(1.0, np.abs(rz).max())
        fk = ko.apply_feature(w.k_ref[0, h, :Tp], feat)
        Sr, Zr = fk.T @ w.v_ref[0, h, :Tp], fk.sum(axis=0)
        assert np.max(np.abs(to_numpy64(S[0, h]) - Sr)) <= 1e-4 * max(1.0, np.abs(Sr).max())
        assert np.max(np.abs(to_numpy64(Z[0, h]) - Zr)) <= 1e-4 * max(1.0, np.abs(Zr).max())
    outs = []
    for t in range(Tp, T):
        outs.append(kb.kata_decode_step(q[:, :, t].contiguous(), k[:, :, t].contiguous(), v[:, :, t].contiguous(), S, Z,
                                        state_layout=code, feature_groups=g).float())
    torch.cuda.synchronize()
    gdec = torch.stack(outs, dim=2).cpu().numpy().astype(np.float64)
    for h in range(H):
        ref = ko.kata_quadratic(w.q_ref[0, h], w.k_ref[0, h], w.v_ref[0, h], feat)[0][Tp:]
        check(gdec[0, h], ref, "f32", f"M{g} decode after prefill/{layout}")


@pytest.mark.parametrize("g", [2, 4])
def test_blockwise_full_size_sampled_rows(g):
    """The benchmark shapes: one-pass chunked form at T = 131072 (c4) and the quadratic form on c2, rows sampled
    from the definition."""
    import torch
    from helpers import oracle_rows, sample_picks
    feat = f"psd_direct:g{g}"
    for w, form in ((inputs.config(4, 131072), "chunked_seq"), (inputs.config(2), "quadratic")):
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        o = FORMS[form](*dev_tensors(w), feature_groups=g, device_status=st)
        torch.cuda.synchronize()
        assert kb.kata_last_impl() == kb.KATA_IMPL_TENSOR and int(st.item()) == 0
        gpu = to_numpy64(o)
        assert np.all(np.isfinite(gpu))
        picks = sample_picks(w, 128, 7 + g)
        ref = oracle_rows(w, picks, feat)
        got = np.stack([gpu[b, h, t] for b, h, t in picks])
        check(got, ref, "bf16", f"M{g} {form} {w.name} sampled rows")
        del o, gpu


@pytest.mark.parametrize("g", [2, 4])
@pytest.mark.parametrize("scan_group", [0, 2, 3, 8])
def test_blockwise_groupings_tensor(g, scan_group):
    """Scan forms of the blockwise map on the tensor-core kernels: groups of tiles, restart from the scanned prefix."""
    import torch
    w = inputs.gaussian_workload("mg_grouped", "bf16", 1, 2, 1100, 64, 64, 64, 77 + g)
    for form in ("chunked_scan", "state_scan"):
        o = FORMS[form](*dev_tensors(w), feature_groups=g, scan_group=scan_group)
        torch.cuda.synchronize()
        assert kb.kata_last_impl() == kb.KATA_IMPL_TENSOR
        gpu = to_numpy64(o)
        for h in range(w.H):
            ref = ko.kata_quadratic(w.q_ref[0, h], w.k_ref[0, h], w.v_ref[0, h], f"psd_direct:g{g}")[0]
            check(gpu[0, h], ref, "bf16", f"M{g} {form} scan_group={scan_group} head {h}")


@pytest.mark.parametrize("layout", ["psd_direct", "psd_packed"])
@pytest.mark.parametrize("g", [2, 4])
def test_blockwise_state_hand_off_tensor(layout, g):
    """Final state, restart from it (in pieces, in place) and decode steps, bf16 d = 64 on the tensor-core kernel."""
    import torch
    B, H, T, d = 1, 2, 420, 64
    w = inputs.gaussian_workload("mg_state_tc", "bf16", B, H, T, d, d, 64, 460 + g)
    q, k, v = dev_tensors(w)
    code = kb.KATA_LAYOUT_PACKED if layout == "psd_packed" else kb.KATA_LAYOUT_DIRECT
    feat = f"{layout}:g{g}"
    n = kb.decode_n_psi(d, 2, code, g)
    S = torch.zeros(B, H, n, d, device="cuda")
    Z = torch.zeros(B, H, n, device="cuda")
    outs = []
    cuts = [0, 130, 257, 400]
    for i in range(3):
        a, b = cuts[i], cuts[i + 1]
        kw = dict(s_pre=S, z_pre=Z, state_layout=code, feature_groups=g)
        if i > 0:
            kw.update(s_init=S, z_init=Z)                      # advanced in place
        outs.append(kb.kata_fwd_chunked(q[:, :, a:b].contiguous(), k[:, :, a:b].contiguous(), v[:, :, a:b].contiguous(), **kw))
        assert kb.kata_last_impl() == kb.KATA_IMPL_TENSOR
    for t in range(400, T):
        outs.append(kb.kata_decode_step(q[:, :, t].contiguous(), k[:, :, t].contiguous(), v[:, :, t].contiguous(), S, Z,
                                        state_layout=code, feature_groups=g).unsqueeze(2))
    torch.cuda.synchronize()
    gpu = to_numpy64(torch.cat(outs, dim=2))
    for h in range(H):
        ref = ko.kata_quadratic(w.q_ref[0, h], w.k_ref[0, h], w.v_ref[0, h], feat)[0]
        check(gpu[0, h], ref, "bf16", f"M{g} hand-off/{layout} head {h}")
        fk = ko.apply_feature(w.k_ref[0, h], feat)
        Sr, Zr = fk.T @ w.v_ref[0, h], fk.sum(axis=0)
        assert np.max(np.abs(to_numpy64(S[0, h]) - Sr)) <= 2e-2 * max(1.0, np.abs(Sr).max())
        assert np.max(np.abs(to_numpy64(Z[0, h]) - Zr)) <= 2e-2 * max(1.0, np.abs(Zr).max())


def test_blockwise_argument_checks():
    import torch
    w = inputs.gaussian_workload("mg_args", "f32", 1, 1, 64, 16, 16, 64, 1)
    q, k, v = dev_tensors(w)
    with pytest.raises(kb.KataError):
        kb.kata_fwd_quadratic(q, k, v, feature_groups=3)
    with pytest.raises(kb.KataError):
        kb.kata_fwd_quadratic(q, k, v, feature_groups=2, feature_order=1)
    wb = inputs.gaussian_workload("mg_args_bf16", "bf16", 1, 1, 64, 64, 64, 64, 1)
    with pytest.raises(kb.KataError):
        wn = inputs.gaussian_workload("mg_args_narrow", "bf16", 1, 1, 64, 32, 32, 64, 1)
        kb.kata_fwd_chunked(*dev_tensors(wn), feature_groups=2, impl=kb.KATA_IMPL_TENSOR)   # blocks of a narrower row: fp32 kernels
