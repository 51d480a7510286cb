"""The allocation-free scan entry point (collected last on purpose).

Some callers may not call cudaMalloc at all -- a plugin inside a framework that owns device memory, or
a serving path that must not disturb the allocator -- so ``kata_chunk_state_scan_static`` keeps its
scan scratch in a fixed device array inside the library.  Here it is called through the C ABI, twice
in a row (the second call finds the first call's leftovers in the array), and both results are
compared with the ordinary ``kata_chunk_state_scan`` entry point.
"""
import ctypes

import numpy as np
import pytest

from paper_2607_17419_b200 import binding as kb
from paper_2607_17419_b200 import build as kbuild
from paper_2607_17419_b200 import inputs

from helpers import TOL, check, dev_tensors, elem_err, oracle_full, row_err, to_numpy64

pytestmark = pytest.mark.gpu


def call_static(q, k, v, out, B, H, T, d, **opt_kw):
    import torch
    opts = kb.make_opts(kb.KATA_BF16 if q.dtype == torch.bfloat16 else kb.KATA_F32,
                        stream=torch.cuda.current_stream().cuda_stream, **opt_kw)
    return kb.lib().kata_chunk_state_scan_static(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), B, H, T, d, d,
                                                 64, ctypes.byref(opts))


@pytest.mark.parametrize("dtype,B,H,T,d", [("bf16", 1, 4, 3000, 64), ("f32", 1, 2, 700, 16)])
def test_static_scratch_matches_workspace_entry_point(dtype, B, H, T, d):
    import torch
    kbuild.build()
    w = inputs.gaussian_workload("noalloc", dtype, B, H, T, d, d, 64, 31)
    q, k, v = dev_tensors(w)
    ref = kb.kata_chunk_state_scan(q, k, v)
    torch.cuda.synchronize()
    r = to_numpy64(ref)
    oracle = oracle_full(w)
    outs = [torch.full_like(v, float("nan")) for _ in range(3)]
    free = []
    for attempt, out in enumerate(outs):          # calls in a row share the one scratch array
        assert call_static(q, k, v, out, B, H, T, d) == 0
        torch.cuda.synchronize()
        free.append(torch.cuda.mem_get_info()[0])
    # the central claim: no device memory is taken by the second and later calls (the first may load the module)
    assert free[1] == free[2], free
    for attempt, out in enumerate(outs):
        g = to_numpy64(out)
        assert np.all(np.isfinite(g)), attempt
        assert elem_err(g, r) <= TOL[dtype] and row_err(g, r) <= TOL[dtype], attempt
        for (b, h), ref_bh in oracle.items():     # and against the definition, not only against its sibling
            check(g[b, h], ref_bh, dtype, f"static entry, call {attempt}, head ({b},{h})")
    # a different problem in between, then the first one again
    w2 = inputs.gaussian_workload("noalloc2", dtype, 1, 3, 1111, d, d, 64, 32)
    q2, k2, v2 = dev_tensors(w2)
    out2 = torch.empty_like(v2)
    assert call_static(q2, k2, v2, out2, 1, 3, 1111, d) == 0
    torch.cuda.synchronize()
    r2 = to_numpy64(kb.kata_chunk_state_scan(q2, k2, v2))
    assert elem_err(to_numpy64(out2), r2) <= TOL[dtype]
    out = torch.empty_like(v)
    assert call_static(q, k, v, out, B, H, T, d, scan_group=16) == 0       # an explicit group size that fits
    torch.cuda.synchronize()
    assert elem_err(to_numpy64(out), r) <= TOL[dtype]


def test_static_scratch_rejects_what_does_not_fit():
    import torch
    kbuild.build()
    w = inputs.gaussian_workload("noalloc3", "bf16", 1, 2, 256, 64, 64, 64, 33)
    q, k, v = dev_tensors(w)
    out = torch.empty_like(v)
    # pretend sizes whose scratch cannot fit 32 MiB even with the coarsest grouping: nothing is launched
    assert call_static(q, k, v, out, 64, 64, 1 << 20, 64) == -4
    # one chunk per group on a long sequence does not fit either
    assert call_static(q, k, v, out, 8, 16, 1 << 17, 64, scan_group=1) == -4
    # state export is not offered by this entry point
    assert call_static(q, k, v, out, 1, 2, 256, 64, s_pre=4096, z_pre=8192) == -1
    # invalid arguments come back with the codes of kata_chunk_state_scan, before the scratch is looked up
    assert call_static(q, k, v, out, 1, 2, 0, 64) == -1          # T = 0
    assert call_static(q, k, v, out, 1, 2, 256, 48) == -2         # unsupported row width
    # and a normal call still works afterwards
    assert call_static(q, k, v, out, 1, 2, 256, 64) == 0
    torch.cuda.synchronize()
    assert elem_err(to_numpy64(out), to_numpy64(kb.kata_chunk_state_scan(q, k, v))) <= TOL["bf16"]
