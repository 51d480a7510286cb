"""GPU parity of the first-order tensor-core kernel (bf16, d_k = d_v = 64; rows of q, k used as features, the
setting of the paper's scan benchmark with matched d x d states): every form, chunk sizes 64 and 128, group
sizes, tile boundaries, the benchmark shape by sampled rows.  Non-negative features so that the normaliser is
positive (with signed features it can vanish)."""
import numpy as np
import pytest

from oracle import kata_oracle as ko
from paper_2607_17419_b200 import binding as kb
from paper_2607_17419_b200 import inputs

from helpers import check, dev_tensors, oracle_rows, sample_picks, to_numpy64, to_torch

pytestmark = pytest.mark.gpu

FORMS = {
    "chunked_seq": lambda q, k, v, **kw: kb.kata_fwd_chunked(q, k, v, inter_chunk=kb.KATA_SEQUENTIAL, **kw),
    "chunked_scan": lambda q, k, v, **kw: kb.kata_fwd_chunked(q, k, v, inter_chunk=kb.KATA_SCAN, **kw),
    "state_scan": lambda q, k, v, **kw: kb.kata_chunk_state_scan(q, k, v, **kw),
}


def run(form, q, k, v, **kw):
    import torch
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    o = FORMS[form](q, k, v, feature_order=1, device_status=st, **kw)
    torch.cuda.synchronize()
    assert kb.kata_last_impl() == kb.KATA_IMPL_TENSOR, "the tensor-core path must be the one that ran"
    assert int(st.item()) == 0, "device status"
    return to_numpy64(o)


def reference(w, b, h):
    return ko.kata_quadratic(w.q_ref[b, h], w.k_ref[b, h], w.v_ref[b, h], "identity")[0]


@pytest.mark.parametrize("form", list(FORMS))
@pytest.mark.parametrize("T", [1, 2, 127, 128, 129, 255, 256, 257, 385, 640, 1500])
def test_tile_boundaries(form, T):
    w = inputs.nonnegative_workload(f"o1_{T}", "bf16", 1, 2, T, 64, 64, 64, 700 + T)
    g = run(form, *dev_tensors(w))
    for h in range(w.H):
        check(g[0, h], reference(w, 0, h), "bf16", f"order 1 T={T}/{form} head {h}")


@pytest.mark.parametrize("form", ["chunked_scan", "state_scan"])
@pytest.mark.parametrize("C,scan_group", [(64, 1), (64, 2), (64, 5), (64, 16), (128, 1), (128, 2), (128, 3), (128, 64)])
def test_groupings(form, C, scan_group):
    """Every grouping of the chunk axis gives the same result (groups are rounded up to whole 128-token tiles)."""
    w = inputs.nonnegative_workload("o1_groups", "bf16", 2, 2, 1100, 64, 64, C, 31)
    g = run(form, *dev_tensors(w), C=C, scan_group=scan_group)
    ng, cpg, rounds = kb.kata_scan_plan(kb.KATA_FN_CHUNKED if form == "chunked_scan" else kb.KATA_FN_CHUNK_STATE_SCAN,
                                        2, 2, 1100, 64, 64, C,
                                        kb.make_opts(kb.KATA_BF16, feature_order=1, inter_chunk=kb.KATA_SCAN, scan_group=scan_group))
    assert (cpg * C) % 128 == 0 or ng == 1
    assert ng == -(-(-(-1100 // C)) // cpg)
    for b in range(w.B):
        for h in range(w.H):
            check(g[b, h], reference(w, b, h), "bf16", f"order 1 C={C} group={scan_group}/{form} ({b},{h})")


def test_zero_rows_and_signed_values():
    """Zero query rows give 0 (normaliser 0), zero keys contribute nothing; values are signed."""
    T = 300
    w = inputs.nonnegative_workload("o1_zero", "bf16", 1, 1, T, 64, 64, 64, 37)
    q, k, v = w.q_dev.copy(), w.k_dev.copy(), w.v_dev.copy()
    for t in (0, 1, 127, 128, 200):
        k[0, 0, t] = 0
    for t in (0, 5, 128, 256):
        q[0, 0, t] = 0
    qr, kr, vr = (inputs.bf16_bits_to_f64(a[0, 0]) for a in (q, k, v))
    ref = ko.kata_quadratic(qr, kr, vr, "identity")[0]
    for form in FORMS:
        g = run(form, *(to_torch(a, "bf16") for a in (q, k, v)))
        check(g[0, 0], ref, "bf16", f"order 1 zero rows/{form}")
        assert np.all(g[0, 0, [0, 5, 128, 256]] == 0)


def test_matches_fp32_kernel():
    import torch
    w = inputs.nonnegative_workload("o1_simt", "bf16", 2, 3, 777, 64, 64, 64, 41)
    q, k, v = dev_tensors(w)
    g = run("state_scan", q, k, v)
    o2 = kb.kata_chunk_state_scan(q, k, v, feature_order=1, impl=kb.KATA_IMPL_SIMT)
    torch.cuda.synchronize()
    assert kb.kata_last_impl() == kb.KATA_IMPL_SIMT
    assert np.max(np.abs(g - to_numpy64(o2))) <= 2e-2


def test_chunk_128_needs_the_tensor_path():
    w = inputs.nonnegative_workload("o1_c128", "f32", 1, 1, 256, 16, 16, 64, 43)
    with pytest.raises(kb.KataError):
        kb.kata_chunk_state_scan(*dev_tensors(w), feature_order=1, C=128)
    wb = inputs.nonnegative_workload("o1_c128b", "bf16", 1, 1, 256, 64, 64, 64, 43)
    with pytest.raises(kb.KataError):
        kb.kata_fwd_chunked(*dev_tensors(wb), C=128)                      # PSD feature: C = 64 only


@pytest.mark.parametrize("B,T", [(1, 131072), (4, 8192)])
def test_scan_benchmark_shapes_sampled_rows(B, T):
    """Shapes of the paper's B x T grid (H = 16, d = 64, bf16, C = 128): rows sampled from the definition."""
    w = inputs.nonnegative_workload(f"o1_bench_{B}_{T}", "bf16", B, 16, T, 64, 64, 128, 47)
    q, k, v = dev_tensors(w)
    picks = sample_picks(w, 96, B + T)
    ref = oracle_rows(w, picks, "identity")
    outs = {}
    for form in FORMS:
        g = run(form, q, k, v, C=128)
        assert np.all(np.isfinite(g))
        got = np.stack([g[b, h, t] for b, h, t in picks])
        check(got, ref, "bf16", f"order 1 B={B} T={T}/{form} sampled rows")
        outs[form] = g
    assert np.max(np.abs(outs["chunked_scan"] - outs["chunked_seq"])) <= 2e-2
    assert np.max(np.abs(outs["state_scan"] - outs["chunked_seq"])) <= 2e-2


@pytest.mark.parametrize("n_groups", [8, 9, 10, 16, 17, 18, 33])
def test_anchor_boundaries_of_the_chained_scan(n_groups):
    """Single-launch scan form with one tile per group: group counts on both sides of the anchors (every eighth
    group publishes the sum of everything up to itself), a ragged last tile, more (group, head) tickets than SMs."""
    T = 128 * n_groups - 5
    w = inputs.nonnegative_workload(f"o1_anchor_{n_groups}", "bf16", 2, 3, T, 64, 64, 128, 900 + n_groups)
    q, k, v = dev_tensors(w)
    ng, cpg, hops = kb.kata_scan_plan(kb.KATA_FN_CHUNK_STATE_SCAN, 2, 3, T, 64, 64, 128,
                                      kb.make_opts(kb.KATA_BF16, feature_order=1, scan_group=1))
    assert (ng, cpg) == (n_groups, 1) and hops == (n_groups - 2) // 8 + 1
    g = run("state_scan", q, k, v, C=128, scan_group=1)
    assert kb.kata_last_launch_count() == 1
    g2 = run("state_scan", q, k, v, C=128, scan_group=1)
    assert np.array_equal(g, g2), "the sum over the group states has a fixed order"
    for b in range(w.B):
        for h in range(w.H):
            check(g[b, h], reference(w, b, h), "bf16", f"order 1, {n_groups} groups ({b},{h})")


def test_more_tickets_than_sms():
    """32 heads x 12 groups = 384 (group, head) tickets for 148 persistent CTAs."""
    w = inputs.nonnegative_workload("o1_tickets", "bf16", 2, 16, 3000, 64, 64, 128, 53)
    g = run("state_scan", *dev_tensors(w), C=128, scan_group=2)
    for b, h in ((0, 0), (0, 15), (1, 7), (1, 15)):
        check(g[b, h], reference(w, b, h), "bf16", f"order 1, 384 tickets ({b},{h})")
