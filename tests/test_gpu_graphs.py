"""The device entry points allocate nothing and never synchronise, so a call can be captured into a CUDA graph and
replayed: the replay must give what the plain call gives, bit for bit, on every route (several launches, a memset,
programmatic dependent launches)."""
import pytest

from paper_2607_17419_b200 import binding as kb
from paper_2607_17419_b200 import inputs

from helpers import check, dev_tensors, oracle_full, to_numpy64

pytestmark = pytest.mark.gpu

CASES = {
    "chunked_seq": (lambda q, k, v, o, **kw: kb.kata_fwd_chunked(q, k, v, o, inter_chunk=kb.KATA_SEQUENTIAL, **kw), {}),
    "chunked_scan": (lambda q, k, v, o, **kw: kb.kata_fwd_chunked(q, k, v, o, inter_chunk=kb.KATA_SCAN, **kw), dict(scan_group=4)),
    "quadratic": (lambda q, k, v, o, **kw: kb.kata_fwd_quadratic(q, k, v, o, **kw), {}),
    "state_scan": (lambda q, k, v, o, **kw: kb.kata_chunk_state_scan(q, k, v, o, **kw), dict(scan_group=4)),
    "order1_scan": (lambda q, k, v, o, **kw: kb.kata_chunk_state_scan(q, k, v, o, **kw), dict(feature_order=1, C=128, scan_group=2)),
}


@pytest.mark.parametrize("case", list(CASES))
def test_a_call_replays_from_a_cuda_graph(case):
    import torch
    fn, kw = CASES[case]
    order1 = kw.get("feature_order") == 1
    make = inputs.nonnegative_workload if order1 else inputs.gaussian_workload
    w = make(f"graph_{case}", "bf16", 2, 3, 1500, 64, 64, kw.get("C", 64), 61)
    q, k, v = dev_tensors(w)
    ws = kb.Workspace()
    plain = torch.empty_like(v)
    fn(q, k, v, plain, workspace=ws, **kw)                     # also sizes the workspace before the capture
    torch.cuda.synchronize()
    launches = kb.kata_last_launch_count()
    out = torch.zeros_like(v)
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            fn(q, k, v, out, workspace=ws, **kw)
        assert kb.kata_last_launch_count() == launches
        for _ in range(3):
            out.zero_()
            graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, plain), "replay differs from the plain call"
    if not order1:
        for (b, h), r in oracle_full(w, heads=[(1, 2)]).items():
            check(to_numpy64(out)[b, h], r, "bf16", f"{case} replayed")
