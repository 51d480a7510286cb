"""Shared helpers of the GPU parity tests: tensors from workloads, error gates, oracle sampling."""
import numpy as np

from oracle import kata_oracle as ko

# Tolerances: max-abs-relative error against the fp64 oracle, 1e-4 for fp32 inputs and 2e-2 for
# bf16 inputs (fp32 accumulation).  "Relative" is read as |g-r| / max(|r|, 1) element-wise (values
# have unit scale) together with the per-row relative L2 error ||g_t - r_t|| / ||r_t||.
TOL = {"f32": 1e-4, "bf16": 2e-2}


def to_torch(arr, dtype, device="cuda"):
    import torch
    if dtype == "bf16":
        t = torch.from_numpy(np.ascontiguousarray(arr).view(np.int16)).view(torch.bfloat16)
    else:
        t = torch.from_numpy(np.ascontiguousarray(arr))
    return t.to(device) if device else t


def dev_tensors(w, device="cuda"):
    return tuple(to_torch(a, w.dtype, device) for a in (w.q_dev, w.k_dev, w.v_dev))


def to_numpy64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def elem_err(g, r):
    return float(np.max(np.abs(g - r) / np.maximum(np.abs(r), 1.0))) if g.size else 0.0


def row_err(g, r):
    nr = np.linalg.norm(r, axis=-1)
    ng = np.linalg.norm(g - r, axis=-1)
    live = nr > 0
    return float(np.max(ng[live] / nr[live])) if np.any(live) else 0.0


def check(g, r, dtype, what=""):
    e, rr = elem_err(g, r), row_err(g, r)
    tol = TOL[dtype]
    assert np.all(np.isfinite(g)), f"{what}: non-finite output"
    assert e <= tol, f"{what}: element error {e:.3e} > {tol}"
    assert rr <= tol, f"{what}: row-relative L2 error {rr:.3e} > {tol}"
    return e, rr


def oracle_full(w, feature="psd_direct", heads=None):
    """Definition (quadratic form) for all or selected (b,h); returns dict {(b,h): o}."""
    out = {}
    sel = heads if heads is not None else [(b, h) for b in range(w.B) for h in range(w.H)]
    for b, h in sel:
        out[(b, h)] = ko.kata_quadratic(w.q_ref[b, h], w.k_ref[b, h], w.v_ref[b, h], feature)[0]
    return out


def oracle_rows(w, picks, feature="psd_direct"):
    """picks: list of (b,h,t); returns [len(picks), d_v] from the definition, row by row."""
    out = np.zeros((len(picks), w.d_v))
    by_head = {}
    for j, (b, h, t) in enumerate(picks):
        by_head.setdefault((b, h), []).append((j, t))
    for (b, h), lst in by_head.items():
        rows = [t for _, t in lst]
        res = ko.kata_rows(w.q_ref[b, h], w.k_ref[b, h], w.v_ref[b, h], rows, feature)
        for (j, _), r in zip(lst, res):
            out[j] = r
    return out


def sample_picks(w, n, seed):
    r = np.random.default_rng(seed)
    picks = [(int(r.integers(w.B)), int(r.integers(w.H)), int(r.integers(w.T))) for _ in range(n)]
    # always include the first rows (smallest denominators) and the very last row
    picks += [(0, 0, t) for t in range(min(8, w.T))] + [(w.B - 1, w.H - 1, w.T - 1)]
    return picks
