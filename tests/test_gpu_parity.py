"""GPU parity: the CUDA path (through the C ABI) against the fp64 oracle, element by element."""
import numpy as np
import pytest

from oracle import kata_oracle as ko
from paper_2607_17419_b200 import binding as kb
from paper_2607_17419_b200 import inputs

from helpers import (TOL, check, dev_tensors, elem_err, oracle_full, oracle_rows, row_err, sample_picks,
                     to_numpy64)

pytestmark = pytest.mark.gpu

FORMS = {
    "quadratic": lambda q, k, v, **kw: kb.kata_fwd_quadratic(q, k, v, **kw),
    "chunked_seq": lambda q, k, v, **kw: kb.kata_fwd_chunked(q, k, v, inter_chunk=kb.KATA_SEQUENTIAL, **kw),
    "chunked_scan": lambda q, k, v, **kw: kb.kata_fwd_chunked(q, k, v, inter_chunk=kb.KATA_SCAN, **kw),
    "state_scan": lambda q, k, v, **kw: kb.kata_chunk_state_scan(q, k, v, **kw),
}
IMPLS = {"simt": kb.KATA_IMPL_SIMT, "auto": kb.KATA_IMPL_AUTO}


def run_form(form, w, impl="auto", **kw):
    import torch
    q, k, v = dev_tensors(w)
    o = FORMS[form](q, k, v, impl=IMPLS[impl], **kw)
    torch.cuda.synchronize()
    return to_numpy64(o)


def full_check(w, form, impl="auto", feature="psd_direct", **kw):
    g = run_form(form, w, impl, **kw)
    ref = oracle_full(w, feature)
    for (b, h), r in ref.items():
        check(g[b, h], r, w.dtype, f"{w.name}/{form}/{impl} head ({b},{h})")
    return g


# ---------------------------------------------------------------------------
# config 1: tiny fp32, all forms, states
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("form", list(FORMS))
def test_config1_all_forms(form):
    full_check(inputs.config(1), form)


@pytest.mark.parametrize("layout", ["psd_direct", "psd_packed"])
def test_config1_exported_prefix_states(layout):
    import torch
    w = inputs.config(1)
    q, k, v = dev_tensors(w)
    NC = -(-w.T // w.C)
    n = ko.feature_dim(w.d_k, layout)
    s_pre = torch.full((w.B, w.H, NC, n, w.d_v), float("nan"), device="cuda")
    z_pre = torch.full((w.B, w.H, NC, n), float("nan"), device="cuda")
    code = kb.KATA_LAYOUT_DIRECT if layout == "psd_direct" else kb.KATA_LAYOUT_PACKED
    o = kb.kata_chunk_state_scan(q, k, v, s_pre=s_pre, z_pre=z_pre, state_layout=code)
    torch.cuda.synchronize()
    for h in range(w.H):
        ro, rs, rz = ko.kata_scan(w.q_ref[0, h], w.k_ref[0, h], w.v_ref[0, h], w.C, layout)
        check(to_numpy64(o)[0, h], ro, "f32", "scan output")
        gs, gz = to_numpy64(s_pre)[0, h], to_numpy64(z_pre)[0, h]
        assert np.all(gs[0] == 0) and np.all(gz[0] == 0)
        scale = max(1.0, np.abs(rs).max())
        assert np.max(np.abs(gs - rs)) / scale < 1e-5
        assert np.max(np.abs(gz - rz)) / max(1.0, np.abs(rz).max()) < 1e-5


# ---------------------------------------------------------------------------
# small shapes spanning several tiles and ragged tails, every supported (d_k, d_v)
# ---------------------------------------------------------------------------

SMALL = [
    ("f32", 1, 1, 1, 16, 16), ("f32", 1, 2, 63, 64, 64), ("f32", 2, 1, 65, 32, 64), ("f32", 1, 3, 333, 64, 16),
    ("bf16", 1, 1, 1, 64, 64), ("bf16", 2, 3, 333, 64, 64), ("bf16", 1, 2, 64, 64, 64),
    ("bf16", 1, 2, 129, 32, 32), ("bf16", 1, 1, 200, 16, 64), ("bf16", 1, 2, 1000, 64, 32),
]


@pytest.mark.parametrize("form", list(FORMS))
@pytest.mark.parametrize("dtype,B,H,T,dk,dv", SMALL)
def test_small_shapes(form, dtype, B, H, T, dk, dv):
    w = inputs.gaussian_workload(f"s_{dtype}_{T}_{dk}_{dv}", dtype, B, H, T, dk, dv, 64, 100 + T + dk)
    for impl in ("simt", "auto"):
        full_check(w, form, impl)


def test_scan_group_sizes_agree():
    w = inputs.gaussian_workload("groups", "bf16", 1, 2, 1500, 64, 64, 64, 7)
    ref = oracle_full(w)
    for sg in (1, 2, 5, 24, 100):
        g = run_form("chunked_scan", w, scan_group=sg)
        for (b, h), r in ref.items():
            check(g[b, h], r, "bf16", f"scan_group={sg}")


def test_inter_chunk_auto_takes_the_scan_form_for_one_long_head():
    """One head of 6000 tokens: AUTO runs the grouped passes and equals the oracle; sixteen such
    heads fill the GPU and stay on the single sequential pass."""
    import torch
    w = inputs.gaussian_workload("auto_scan", "bf16", 1, 1, 6000, 64, 64, 64, 21)
    q, k, v = dev_tensors(w)
    o = kb.kata_fwd_chunked(q, k, v, inter_chunk=kb.KATA_INTER_AUTO)
    torch.cuda.synchronize()
    # groups of a few tiles: the state-only pass, the scan rounds, the restarted pass
    ng, _, rounds = kb.kata_scan_plan(kb.KATA_FN_CHUNKED, 1, 1, 6000, 64, 64, 64, kb.make_opts(kb.KATA_BF16, inter_chunk=kb.KATA_INTER_AUTO))
    assert ng >= 8 and rounds >= 3
    assert kb.kata_last_launch_count() == 2 + rounds and kb.kata_last_impl() == 2
    for (b, h), r in oracle_full(w).items():
        check(to_numpy64(o)[b, h], r, "bf16", "auto -> scan")
    w = inputs.gaussian_workload("auto_seq", "bf16", 1, 16, 1000, 64, 64, 64, 22)
    q, k, v = dev_tensors(w)
    o = kb.kata_fwd_chunked(q, k, v, inter_chunk=kb.KATA_INTER_AUTO)
    torch.cuda.synchronize()
    # the sequential walk of the feature-split kernel: the key-scale pre-pass and the kernel
    assert kb.kata_last_launch_count() == 2
    for (b, h), r in oracle_full(w, heads=[(0, 3)]).items():
        check(to_numpy64(o)[b, h], r, "bf16", "auto -> sequential")


def test_degenerate_rows():
    """Zero keys/queries and D = 0 rows give 0, never NaN (reading: readout defined only for D > 0)."""
    import torch
    T, d = 130, 64
    w = inputs.gaussian_workload("degenerate", "f32", 1, 1, T, d, d, 64, 9)
    q, k, v = w.q_dev.copy(), w.k_dev.copy(), w.v_dev.copy()
    k[0, 0, 0] = 0.0          # first key zero -> D_0 = 0
    k[0, 0, 70] = 0.0
    q[0, 0, 5] = 0.0          # zero query -> 0
    q[0, 0, 100] = 0.0
    ref = ko.kata_quadratic(q[0, 0].astype(np.float64), k[0, 0].astype(np.float64), v[0, 0].astype(np.float64))[0]
    assert np.all(ref[0] == 0) and np.all(ref[5] == 0) and np.all(ref[100] == 0)
    tq, tk, tv = (torch.from_numpy(a).cuda() for a in (q, k, v))
    for form in FORMS:
        for impl in ("simt", "auto"):
            g = to_numpy64(FORMS[form](tq, tk, tv, impl=IMPLS[impl]))
            check(g[0, 0], ref, "f32", f"degenerate/{form}/{impl}")
            assert np.all(g[0, 0, [0, 5, 100]] == 0)


def test_sequential_mode_is_deterministic():
    import torch
    w = inputs.gaussian_workload("det", "bf16", 1, 4, 700, 64, 64, 64, 11)
    q, k, v = dev_tensors(w)
    a = kb.kata_fwd_chunked(q, k, v).clone()
    b = kb.kata_fwd_chunked(q, k, v).clone()
    c = kb.kata_fwd_quadratic(q, k, v).clone()
    d = kb.kata_fwd_quadratic(q, k, v).clone()
    torch.cuda.synchronize()
    assert torch.equal(a, b) and torch.equal(c, d)


def test_host_io_entry_matches_device_entry():
    import torch
    w = inputs.gaussian_workload("hostio", "bf16", 1, 2, 300, 64, 64, 64, 12)
    q, k, v = dev_tensors(w)
    ref = kb.kata_fwd_chunked(q, k, v)
    hq, hk, hv = (t.cpu().pin_memory() for t in (q, k, v))
    ho = torch.empty_like(hv).pin_memory()
    kb.kata_fwd_host(kb.KATA_FN_CHUNKED, hq, hk, hv, ho)
    torch.cuda.synchronize()
    assert torch.equal(ho, ref.cpu())
    ho2 = torch.empty_like(hv).pin_memory()
    kb.kata_fwd_host(kb.KATA_FN_CHUNK_STATE_SCAN, hq, hk, hv, ho2)
    torch.cuda.synchronize()
    check(to_numpy64(ho2)[0, 0], oracle_full(w, heads=[(0, 0)])[(0, 0)], "bf16", "host scan")


@pytest.mark.parametrize("B,H,T,groups", [(1, 2, 33000, 0), (2, 1, 40000, 2), (1, 1, 70001, 0)])
def test_host_io_long_sequence_in_pieces(B, H, T, groups):
    """Long sequences through the host-buffer entry are copied and computed piece by piece (state handed from
    piece to piece, copies overlapped with the kernels): the result equals the device entry's within the bf16
    tolerance and the oracle on sampled rows; the ragged last piece and a second call on the same buffers too."""
    import torch
    w = inputs.gaussian_workload("hostpipe", "bf16", B, H, T, 64, 64, 64, 31 + T)
    q, k, v = dev_tensors(w)
    ref = to_numpy64(kb.kata_fwd_chunked(q, k, v, feature_groups=groups))
    hq, hk, hv = (t.cpu().pin_memory() for t in (q, k, v))
    ho = torch.empty_like(hv).pin_memory()
    for rep in range(2):
        ho.zero_()
        kb.kata_fwd_host(kb.KATA_FN_CHUNKED, hq, hk, hv, ho, feature_groups=groups)
        torch.cuda.synchronize()
        assert kb.kata_last_launch_count() >= 4          # one kernel (and a state copy) per piece
        g = to_numpy64(ho)
        assert elem_err(g, ref) <= TOL["bf16"] and row_err(g, ref) <= TOL["bf16"]
    picks = sample_picks(w, 96, T) + [(B - 1, H - 1, T - 1), (0, 0, 0)]
    feature = "psd_direct" if groups == 0 else f"psd_direct:g{groups}"
    got = np.stack([g[b, h, t] for b, h, t in picks])
    check(got, oracle_rows(w, picks, feature), "bf16", "host pieces, sampled rows")


# ---------------------------------------------------------------------------
# first-order features (rows used as they are), nonnegative inputs so that D > 0
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("form", list(FORMS))
@pytest.mark.parametrize("dtype,T,dk,dv", [("f32", 300, 64, 64), ("bf16", 257, 64, 64), ("f32", 100, 16, 32)])
def test_first_order_features(form, dtype, T, dk, dv):
    w = inputs.nonnegative_workload("o1", dtype, 1, 2, T, dk, dv, 64, 21)
    full_check(w, form, feature="identity", feature_order=1)


def test_first_order_states():
    import torch
    w = inputs.nonnegative_workload("o1s", "f32", 1, 2, 300, 64, 64, 64, 22)
    q, k, v = dev_tensors(w)
    NC = -(-w.T // 64)
    s_pre = torch.empty((1, 2, NC, 64, 64), device="cuda")
    z_pre = torch.empty((1, 2, NC, 64), device="cuda")
    kb.kata_chunk_state_scan(q, k, v, s_pre=s_pre, z_pre=z_pre, feature_order=1)
    for h in range(2):
        _, rs, rz = ko.kata_scan(w.q_ref[0, h], w.k_ref[0, h], w.v_ref[0, h], 64, "identity")
        assert np.max(np.abs(to_numpy64(s_pre)[0, h] - rs)) / np.abs(rs).max() < 1e-5
        assert np.max(np.abs(to_numpy64(z_pre)[0, h] - rz)) / np.abs(rz).max() < 1e-5


# ---------------------------------------------------------------------------
# the benchmark configurations at full size
# ---------------------------------------------------------------------------

def test_config2_quadratic_full():
    full_check(inputs.config(2), "quadratic")


def test_config3_chunked_full_size():
    w = inputs.config(3)
    g = run_form("chunked_seq", w)
    heads = [(0, 0), (3, 7), (7, 15), (5, 2)]
    for (b, h), r in oracle_full(w, heads=heads).items():
        check(g[b, h], r, "bf16", f"c3 head ({b},{h})")
    picks = sample_picks(w, 256, 33)
    ref = oracle_rows(w, picks)
    got = np.stack([g[b, h, t] for b, h, t in picks])
    check(got, ref, "bf16", "c3 sampled rows")


def test_config5_recall_full():
    w = inputs.config(5)
    g = full_check(w, "chunked_seq")
    gq = run_form("quadratic", w)
    assert elem_err(gq, g) <= TOL["bf16"]


def test_config4_scan_forms_in_sixteen_groups():
    """Config 4 at T = 131072 with the chunk axis cut into 16 groups of 128 chunks: the state-only pass, four rounds
    of the Hillis-Steele scan over the group states (section "Tree-scan inter-chunk reduction", appendix
    "Associative-scan kernel"), the restarted pass.  Both scan entry points against the definition on sampled rows
    and against the sequential walk on every element."""
    T = 131072
    w = inputs.config(4, T)
    sg = (T // 64) // 16
    for fn, mode in ((kb.KATA_FN_CHUNKED, kb.KATA_SCAN), (kb.KATA_FN_CHUNK_STATE_SCAN, kb.KATA_SEQUENTIAL)):
        ng, cpg, rounds = kb.kata_scan_plan(fn, w.B, w.H, T, 64, 64, 64, kb.make_opts(kb.KATA_BF16, inter_chunk=mode, scan_group=sg))
        assert ng == 16 and cpg == sg and rounds == 4
    seq = run_form("chunked_seq", w)
    picks = sample_picks(w, 192, 777)
    ref = oracle_rows(w, picks)
    for form in ("chunked_scan", "state_scan"):
        g = run_form(form, w, scan_group=sg)
        assert kb.kata_last_impl() == kb.KATA_IMPL_TENSOR
        assert kb.kata_last_launch_count() >= 2 + 4, "state-only pass, four scan rounds, restarted pass"
        assert np.all(np.isfinite(g))
        assert elem_err(g, seq) <= TOL["bf16"] and row_err(g, seq) <= TOL["bf16"], form
        got = np.stack([g[b, h, t] for b, h, t in picks])
        check(got, ref, "bf16", f"c4 T={T} {form} in 16 groups, sampled rows")


@pytest.mark.parametrize("T", [8192, 32768, 131072])
def test_config4_long_context(T):
    w = inputs.config(4, T)
    seq = run_form("chunked_seq", w)
    scan = run_form("chunked_scan", w)
    pipe = run_form("state_scan", w)
    assert np.all(np.isfinite(seq)) and np.all(np.isfinite(scan)) and np.all(np.isfinite(pipe))
    # scan forms equal the sequential recurrence within tolerance, on every element
    assert elem_err(scan, seq) <= TOL["bf16"] and row_err(scan, seq) <= TOL["bf16"]
    assert elem_err(pipe, seq) <= TOL["bf16"] and row_err(pipe, seq) <= TOL["bf16"]
    if T == 8192:
        for (b, h), r in oracle_full(w, heads=[(0, 0), (0, 9)]).items():
            for name, g in (("seq", seq), ("scan", scan), ("pipe", pipe)):
                check(g[b, h], r, "bf16", f"c4 T={T} {name} head {h}")
    picks = sample_picks(w, 256, T)
    ref = oracle_rows(w, picks)
    for name, g in (("seq", seq), ("scan", scan), ("pipe", pipe)):
        got = np.stack([g[b, h, t] for b, h, t in picks])
        check(got, ref, "bf16", f"c4 T={T} {name} sampled rows")
    # convexity: every output coordinate lies within the running min/max of the values seen so far
    v = w.v_ref
    lo, hi = np.minimum.accumulate(v, axis=2), np.maximum.accumulate(v, axis=2)
    slack = 2e-2 * np.maximum(1.0, np.abs(v).max())
    assert np.all(seq >= lo - slack) and np.all(seq <= hi + slack)


def test_more_heads_than_one_grid_axis():
    """65537 heads: a kernel takes at most 65535 at a time, the forward entries run the rest as a second slab on the
    same stream and in the same scratch.  Heads on both sides of the cut against the definition; a call with state
    pointers keeps the limit."""
    import torch
    B, H, T, d = 65537, 1, 3, 16
    w = inputs.gaussian_workload("many_heads", "f32", B, H, T, d, d, 64, 91)
    q, k, v = dev_tensors(w)
    heads = [0, 1, 65533, 65534, 65535, 65536]
    ref = {b: ko.kata_quadratic(w.q_ref[b, 0], w.k_ref[b, 0], w.v_ref[b, 0])[0] for b in heads}
    for form in ("quadratic", "chunked_seq", "chunked_scan", "state_scan"):
        g = run_form(form, w)
        assert np.all(np.isfinite(g))
        for b in heads:
            check(g[b, 0], ref[b], "f32", f"{form}, head {b} of {B}")
        assert kb.kata_last_launch_count() >= 2, "two slabs of heads"
    S = torch.zeros(B, H, kb.decode_n_psi(d), d, device="cuda")
    Z = torch.zeros(B, H, kb.decode_n_psi(d), device="cuda")
    with pytest.raises(kb.KataError) as e:
        kb.kata_fwd_chunked(q, k, v, s_init=S, z_init=Z)
    assert e.value.status == kb.KATA_ERR_UNSUPPORTED_SHAPE
