"""GPU parity, tensor-core kernels (bf16, d_k = d_v = 64): tile boundaries, degenerate rows, value structure.

The tensor-core kernels work in tiles of 128 tokens (quadratic form: 128 queries x 128 keys; chunked form: 128
tokens per state update), so the ragged cases sit around multiples of 128.
"""
import numpy as np
import pytest

from oracle import kata_oracle as ko
from paper_2607_17419_b200 import binding as kb
from paper_2607_17419_b200 import inputs

from helpers import check, dev_tensors, oracle_full, to_numpy64, to_torch

pytestmark = pytest.mark.gpu

FORMS = {
    "quadratic": lambda q, k, v, **kw: kb.kata_fwd_quadratic(q, k, v, **kw),
    "chunked_seq": lambda q, k, v, **kw: kb.kata_fwd_chunked(q, k, v, inter_chunk=kb.KATA_SEQUENTIAL, **kw),
    "chunked_scan": lambda q, k, v, **kw: kb.kata_fwd_chunked(q, k, v, inter_chunk=kb.KATA_SCAN, **kw),
}


def run(form, q, k, v, **kw):
    import torch
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    o = FORMS[form](q, k, v, device_status=st, **kw)
    torch.cuda.synchronize()
    assert kb.kata_last_impl() == kb.KATA_IMPL_TENSOR, "the tensor-core path must be the one that ran"
    assert int(st.item()) == 0, "device status"
    return to_numpy64(o)


@pytest.mark.parametrize("form", list(FORMS))
@pytest.mark.parametrize("T", [2, 17, 127, 128, 129, 255, 256, 257, 385, 640])
def test_tile_boundaries(form, T):
    w = inputs.gaussian_workload(f"edge_{T}", "bf16", 1, 2, T, 64, 64, 64, 900 + T)
    g = run(form, *dev_tensors(w))
    for (b, h), r in oracle_full(w).items():
        check(g[b, h], r, "bf16", f"T={T}/{form} head ({b},{h})")


@pytest.mark.parametrize("form", list(FORMS))
def test_degenerate_rows_bf16(form):
    """Zero keys and queries on and around tile boundaries: zero feature, output 0 where D = 0, never NaN."""
    T, d = 300, 64
    w = inputs.gaussian_workload("degenerate_bf16", "bf16", 1, 1, T, d, d, 64, 19)
    q, k, v = w.q_dev.copy(), w.k_dev.copy(), w.v_dev.copy()
    for t in (0, 1, 127, 128, 200, 299):
        k[0, 0, t] = 0
    for t in (0, 5, 127, 128, 256):
        q[0, 0, t] = 0
    qr, kr, vr = (inputs.bf16_bits_to_f64(a[0, 0]) for a in (q, k, v))
    ref = ko.kata_quadratic(qr, kr, vr)[0]
    assert np.all(ref[[0, 1, 5, 127, 128, 256]] == 0)        # rows 0, 1: no live key yet; the others: zero query
    g = run(form, *(to_torch(a, "bf16") for a in (q, k, v)))
    check(g[0, 0], ref, "bf16", f"degenerate/{form}")
    assert np.all(g[0, 0, [0, 1, 5, 127, 128, 256]] == 0)


@pytest.mark.parametrize("form", list(FORMS))
@pytest.mark.parametrize("scale", [1.0 / 64, 16.0])
def test_input_scale(form, scale):
    """The weights depend on directions only; the output scales with v.  Large and small q, k norms."""
    w = inputs.gaussian_workload("scale", "bf16", 1, 2, 400, 64, 64, 64, 23)
    q, k, v = dev_tensors(w)
    base = run(form, q, k, v)
    g = run(form, (q.float() * scale).to(q.dtype), (k.float() * scale).to(k.dtype), v)
    # powers of two: the bf16 inputs scale exactly, and so do all products before the normalisation
    for (b, h), r in oracle_full(w).items():
        check(g[b, h], r, "bf16", f"scale={scale}/{form}")
    assert np.max(np.abs(g - base)) <= 2e-2


@pytest.mark.parametrize("form", list(FORMS))
def test_nonnegative_values_stay_in_hull(form):
    """Proposition 1 (convex gate): each output row is a convex combination of earlier value rows."""
    w = inputs.nonnegative_workload("hull", "bf16", 1, 2, 700, 64, 64, 64, 29)
    g = run(form, *dev_tensors(w))
    vmax = np.maximum.accumulate(w.v_ref, axis=2)
    vmin = np.minimum.accumulate(w.v_ref, axis=2)
    slack = 2e-2 * np.maximum(1.0, np.maximum(np.abs(vmax), np.abs(vmin)))
    assert np.all(g <= vmax + slack) and np.all(g >= vmin - slack)
    for (b, h), r in oracle_full(w).items():
        check(g[b, h], r, "bf16", f"hull/{form}")


def test_bounded_waits_time_out_cleanly_and_the_stream_stays_usable():
    """The error contract of the tensor-core kernels (`KATA_ERR_DEVICE_TIMEOUT` in `*device_status`): a wait that
    nothing satisfies gives up on its own limit, the kernel writes the status and returns, and the next call on the
    same stream is correct.  Run on a test-only kernel of one warp (no TMEM, MMA or TMA in flight)."""
    import torch
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    rep = torch.full((8,), -1, dtype=torch.int32, device="cuda")
    rep[7] = 0                                               # the flag in global memory
    assert kb.kata_selftest_wait_timeout(st, rep, max_polls=2000) == kb.KATA_OK
    torch.cuda.synchronize()
    assert int(st.item()) == kb.KATA_ERR_DEVICE_TIMEOUT
    assert rep.tolist()[:3] == [1, 1, 1], "both barrier waits gave up and raised the abort flag"
    # the wait on a flag of another CTA: gives up when nobody sets it, returns when it is set, gives up at once on poison
    assert rep.tolist()[3:7] == [1, 1, 1, 1]
    assert kb.kata_selftest_wait_timeout(st, rep, max_polls=0) == kb.KATA_ERR_INVALID_ARG
    # the next ordinary call on the same stream
    w = inputs.gaussian_workload("after_timeout", "bf16", 1, 2, 300, 64, 64, 64, 4242)
    for form in FORMS:
        g = run(form, *dev_tensors(w))
        for (b, h), r in oracle_full(w).items():
            check(g[b, h], r, "bf16", f"after a timed-out launch/{form} head ({b},{h})")


@pytest.mark.parametrize("form", list(FORMS))
def test_queries_nearly_orthogonal_to_every_key(form):
    """Small normalisers: probe queries whose cosine to every key (their own included) is about a tenth of a
    typical one, so the normaliser is about a hundredth of its usual size while the output stays of order one.  The
    kernels read the state and the weights through bf16 operands; the output must still match the definition, and
    it must not have fallen into the `normaliser <= 0 -> out = 0` branch."""
    T, every = 1500, 97
    w = inputs.near_orthogonal_workload("near_orth", "bf16", 1, 2, T, 64, 64, 64, 606, every=every)
    probes = np.arange(every - 1, T, every)
    ref = oracle_full(w)
    D = {bh: ko.kata_quadratic(w.q_ref[bh], w.k_ref[bh], w.v_ref[bh])[2] for bh in ref}
    g = run(form, *dev_tensors(w))
    for (b, h), r in ref.items():
        d = D[(b, h)]
        others = np.setdiff1d(np.arange(200, T), probes)
        assert np.median(d[probes[2:]] / (probes[2:] + 1)) < 0.1 * np.median(d[others] / (others + 1)), "the probes are not small"
        check(g[b, h], r, "bf16", f"near-orthogonal/{form} head ({b},{h})")
        check(g[b, h][probes], r[probes], "bf16", f"near-orthogonal/{form} probe rows, head ({b},{h})")
        assert np.all(np.abs(g[b, h][probes]).max(axis=1) > 0), "a probe row came out as 0: its normaliser was lost"
