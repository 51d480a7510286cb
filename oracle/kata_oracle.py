"""fp64 CPU oracle for the KATA forward pass (TEST INFRASTRUCTURE ONLY).

This file is the slow, plain statement of what the CUDA kernels must compute.
It is imported only by the tests, by the smoke check and by the benchmark's
CPU-baseline leg; the product path never touches it and it shares no code with
the CUDA sources.  Everything is numpy float64, one head at a time, with no
blocking or fusion beyond what the cited definition itself states.

What is computed (one head; q,k in R^{T x d}, v in R^{T x d_v}):

  * rows are projected to the unit sphere, u_hat = u/||u||  (explicit l2
    normalisation of the method summary; a zero row stays zero);
  * the feature is the rank-one PSD lift psi(u) = u u^T ("Rank-one packing into
    the PSD cone"), either as the d^2 direct outer-product layout or as the
    d(d+1)/2 packed symmetric coordinates ("From rank-one rays to low-rank PSD
    packing"), so <psi(q),psi(k)> = (q_hat . k_hat)^2;
  * the causal normalised readout of Eq. (2) (linearised attention):
        z_t = psi(q_t)^T S_t / psi(q_t)^T Z_t,
        S_t = sum_{i<=t} psi(k_i) v_i^T,  Z_t = sum_{i<=t} psi(k_i);
    z_t := 0 when the denominator is 0 (the paper defines the readout only for
    a positive denominator; this is the reading both sides use).

Forms, all of which must agree to rounding:

  kata_quadratic   the definition: dense causal weights w_ti = (q_hat_t.k_hat_i)^2
  kata_recurrent   token recurrence of Eq. (2) on the explicit feature vectors
  kata_chunked     Algorithm 1 with the chunk equations (chunk state update,
                   masked intra-chunk scores, chunk output)
  kata_scan        the three-stage pipeline of the associative-scan appendix:
                   chunk-local states, exclusive prefix (running sum or
                   log-depth doubling), chunk output
  gate_decomposition   Proposition 1 (output-level gating)
  kata_quadratic_bwd   gradients of the definition with respect to q, k, v (chain rule
                   through o = N/D, the weights and the normalisation)
  kata_bwd_rows    the same gradients for selected tokens only (long sequences)

feature="identity" treats the rows of q,k as already-mapped features (the
setting the scan appendix analyses): no normalisation, no lift.

Parity pins: every function here is pinned by tests/test_oracle_pins.py
(closed forms, printed numbers, invariances, brute force); none is unpinned.
"""
from __future__ import annotations

import math

import numpy as np

FEATURES = ("psd_direct", "psd_packed", "identity")


# ---------------------------------------------------------------------------
# feature maps
# ---------------------------------------------------------------------------

def normalize_rows(x: np.ndarray) -> np.ndarray:
    """u_hat = u / ||u||_2 per row; an all-zero row maps to zero."""
    x = np.asarray(x, dtype=np.float64)
    n = np.sqrt(np.sum(x * x, axis=-1, keepdims=True))
    out = np.zeros_like(x)
    np.divide(x, n, out=out, where=n > 0)
    return out


def psi_direct(u: np.ndarray) -> np.ndarray:
    """vec(u u^T): row (a*d+b) holds u_a u_b.  u: [..., d] -> [..., d*d]."""
    u = np.asarray(u, dtype=np.float64)
    return (u[..., :, None] * u[..., None, :]).reshape(*u.shape[:-1], u.shape[-1] ** 2)


def packed_index(d: int):
    """Upper-triangle (a<=b) index pairs in row-major order; d(d+1)/2 of them."""
    a, b = np.triu_indices(d)
    return a, b


def psi_packed(u: np.ndarray) -> np.ndarray:
    """Isometric symmetric packing of u u^T: diagonal u_a^2, off-diagonal sqrt(2) u_a u_b (a<b)."""
    u = np.asarray(u, dtype=np.float64)
    a, b = packed_index(u.shape[-1])
    scale = np.where(a == b, 1.0, math.sqrt(2.0))
    return u[..., a] * u[..., b] * scale


def split_feature(feature: str):
    """'psd_direct', 'psd_packed', 'identity', or a PSD name with a block suffix ':g2' / ':g4' (KATA-Mg).

    Returns (base name, g)."""
    base, _, suf = feature.partition(":")
    g = 1
    if suf:
        if not (suf.startswith("g") and suf[1:].isdigit()):
            raise ValueError(feature)
        g = int(suf[1:])
    if base not in FEATURES or (g != 1 and base == "identity") or g < 1:
        raise ValueError(feature)
    return base, g


def feature_dim(d: int, feature: str) -> int:
    base, g = split_feature(feature)
    if d % g != 0:
        raise ValueError(f"d={d} is not divisible by g={g}")
    m = d // g
    if base == "psd_direct":
        return g * m * m
    if base == "psd_packed":
        return g * (m * (m + 1) // 2)
    return d


def apply_feature(x: np.ndarray, feature: str) -> np.ndarray:
    """Row-wise Psi(X).  PSD features: the row is l2-normalised, then lifted; with a ':g' suffix the
    normalised row is cut into g blocks of d/g entries and each block is lifted on its own (the blockwise PSD
    map psi_Mg(u) = (u_1 u_1^T, ..., u_g u_g^T), whose inner product is sum_a (q_a . k_a)^2), blocks
    concatenated in order."""
    base, g = split_feature(feature)
    if base == "identity":
        return np.asarray(x, dtype=np.float64)
    u = normalize_rows(x)
    d = u.shape[-1]
    if d % g != 0:
        raise ValueError(f"d={d} is not divisible by g={g}")
    m = d // g
    lift = psi_direct if base == "psd_direct" else psi_packed
    return np.concatenate([lift(u[..., a * m:(a + 1) * m]) for a in range(g)], axis=-1)


def _safe_div(n: np.ndarray, d: np.ndarray) -> np.ndarray:
    """n / d row-wise with the D=0 reading: output 0 where the denominator is 0."""
    out = np.zeros_like(n)
    np.divide(n, d[..., None], out=out, where=(d != 0)[..., None])
    return out


# ---------------------------------------------------------------------------
# form Q: the definition
# ---------------------------------------------------------------------------

def _block_kernel(qh: np.ndarray, kh: np.ndarray, g: int) -> np.ndarray:
    """sum over the g blocks of (q_a . k_a)^2 for normalised rows qh [Tq,d], kh [Tk,d]  ->  [Tq,Tk].

    g = 1 is the full rank-one lift (q_hat . k_hat)^2; g > 1 the blockwise PSD map of KATA-Mg."""
    d = qh.shape[-1]
    if d % g != 0:
        raise ValueError(f"d={d} is not divisible by g={g}")
    m = d // g
    out = np.zeros((qh.shape[0], kh.shape[0]))
    for a in range(g):
        out += (qh[:, a * m:(a + 1) * m] @ kh[:, a * m:(a + 1) * m].T) ** 2
    return out


def causal_weights(q: np.ndarray, k: np.ndarray, feature: str = "psd_direct") -> np.ndarray:
    """w[t,i] = <psi(q_t), psi(k_i)> for i<=t, else 0, from the closed form of the inner product
    (dot products of the rows, never the lifted features).  [T,T]."""
    base, g = split_feature(feature)
    if base == "identity":
        s = np.asarray(q, np.float64) @ np.asarray(k, np.float64).T
    else:
        s = _block_kernel(normalize_rows(q), normalize_rows(k), g)
    return np.tril(s)


def kata_quadratic(q, k, v, feature: str = "psd_direct"):
    """o_t = sum_{i<=t} w_ti v_i / sum_{i<=t} w_ti.  Returns (o, N, D)."""
    w = causal_weights(q, k, feature)
    v = np.asarray(v, dtype=np.float64)
    N = w @ v
    D = w.sum(axis=1)
    return _safe_div(N, D), N, D


def kata_rows(q, k, v, rows, feature: str = "psd_direct") -> np.ndarray:
    """The definition evaluated for selected output rows only (for long sequences)."""
    q = np.asarray(q, np.float64)
    k = np.asarray(k, np.float64)
    v = np.asarray(v, np.float64)
    out = np.zeros((len(rows), v.shape[1]))
    base, g = split_feature(feature)
    kh = k if base == "identity" else normalize_rows(k)
    for j, t in enumerate(rows):
        if base == "identity":
            w = kh[: t + 1] @ q[t]
        else:
            w = _block_kernel(normalize_rows(q[t][None]), kh[: t + 1], g)[0]
        D = w.sum()
        if D != 0:
            out[j] = (w @ v[: t + 1]) / D
    return out


# ---------------------------------------------------------------------------
# form R: token recurrence, Eq. (2)
# ---------------------------------------------------------------------------

def kata_recurrent(q, k, v, feature: str = "psd_direct"):
    """S_t = S_{t-1} + psi(k_t) v_t^T, Z_t = Z_{t-1} + psi(k_t), z_t = psi(q_t)^T S_t / psi(q_t)^T Z_t."""
    fq = apply_feature(q, feature)
    fk = apply_feature(k, feature)
    v = np.asarray(v, dtype=np.float64)
    T, n = fk.shape
    S = np.zeros((n, v.shape[1]))
    Z = np.zeros(n)
    o = np.zeros_like(v)
    for t in range(T):
        S += np.outer(fk[t], v[t])
        Z += fk[t]
        den = fq[t] @ Z
        if den != 0:
            o[t] = (fq[t] @ S) / den
    return o


# ---------------------------------------------------------------------------
# backward of the definition (vector-Jacobian product)
# ---------------------------------------------------------------------------

def kata_quadratic_bwd(q, k, v, dout, feature: str = "psd_direct"):
    """Gradients of L = sum(dout * o) for o = kata_quadratic(q, k, v, feature)[0], by the chain rule through the
    definition in the order it is written: o = N / D, N = W V, D = W 1, W = tril(<psi(q_hat), psi(k_hat)>),
    x_hat = x / ||x||.  Returns (dq, dk, dv).  Rows with D = 0 have o = 0 identically in a neighbourhood of
    the inputs that keeps D = 0 and contribute nothing; a zero row of q or k has a zero feature and gets a zero
    gradient (the reading of the forward: the feature of a zero row is the constant 0)."""
    q = np.asarray(q, np.float64)
    k = np.asarray(k, np.float64)
    v = np.asarray(v, np.float64)
    dout = np.asarray(dout, np.float64)
    base, g = split_feature(feature)
    W = causal_weights(q, k, feature)
    D = W.sum(axis=1)
    o = _safe_div(W @ v, D)
    live = D != 0
    invD = np.zeros_like(D)
    invD[live] = 1.0 / D[live]
    # o_t = sum_i W_ti v_i / D_t:  dL/dW_ti = dout_t . (v_i - o_t) / D_t  (i <= t),  dL/dv_i = sum_t (W_ti / D_t) dout_t
    G = np.tril((dout @ v.T - np.sum(dout * o, axis=1)[:, None]) * invD[:, None])
    dv = (W * invD[:, None]).T @ dout
    if base == "identity":
        return G @ k, G.T @ q, dv          # W_ti = q_t . k_i
    qh, kh = normalize_rows(q), normalize_rows(k)
    d = q.shape[1]
    m = d // g
    dqh, dkh = np.zeros_like(q), np.zeros_like(k)
    for a in range(g):                      # W_ti = sum_a (qh_t,a . kh_i,a)^2
        sl = slice(a * m, (a + 1) * m)
        E = 2.0 * G * (qh[:, sl] @ kh[:, sl].T)
        dqh[:, sl] = E @ kh[:, sl]
        dkh[:, sl] = E.T @ qh[:, sl]

    def through_normalisation(x, xh, dxh):  # x_hat = x/||x||:  dx = (dx_hat - x_hat (x_hat . dx_hat)) / ||x||
        n = np.sqrt(np.sum(x * x, axis=1))
        out = np.zeros_like(x)
        nz = n > 0
        proj = dxh - xh * np.sum(xh * dxh, axis=1, keepdims=True)
        out[nz] = proj[nz] / n[nz, None]
        return out

    return through_normalisation(q, qh, dqh), through_normalisation(k, kh, dkh), dv


def kata_bwd_rows(q, k, v, dout, rows_q, rows_k, C: int = 256):
    """Rows of the gradients of `kata_quadratic_bwd` (feature 'psd_direct') for long sequences: dq for the tokens in
    rows_q, dk and dv for the tokens in rows_k.  o_t and D_t of every token come from Algorithm 1 (chunk equations,
    one chunk of features at a time); each requested row is then the sum the chain rule states, written out over
    all the tokens it couples to:
        u_t = dout_t / D_t,  c_t = (dout_t . o_t) / D_t,  s_ti = q_hat_t . k_hat_i,
        dq_hat_t = 2 sum_{i<=t} s_ti (u_t . v_i - c_t) k_hat_i,
        dk_hat_i = 2 sum_{t>=i} s_ti (u_t . v_i - c_t) q_hat_t,   dv_i = sum_{t>=i} s_ti^2 u_t,
        dx = (dx_hat - x_hat (x_hat . dx_hat)) / ||x||.
    Returns (dq [len(rows_q), d], dk [len(rows_k), d], dv [len(rows_k), d_v])."""
    q = np.asarray(q, np.float64)
    k = np.asarray(k, np.float64)
    v = np.asarray(v, np.float64)
    dout = np.asarray(dout, np.float64)
    T, d = q.shape
    qh, kh = normalize_rows(q), normalize_rows(k)
    o = np.zeros_like(v)
    D = np.zeros(T)
    S = np.zeros((d * d, v.shape[1]))
    Z = np.zeros(d * d)
    for t0 in range(0, T, C):
        sl = slice(t0, min(T, t0 + C))
        FQ, FK = psi_direct(qh[sl]), psi_direct(kh[sl])
        o[sl], _, D[sl] = chunk_output(FQ, FK, v[sl], S, Z)
        S = S + FK.T @ v[sl]
        Z = Z + FK.sum(axis=0)
    invD = np.zeros(T)
    invD[D != 0] = 1.0 / D[D != 0]
    u = dout * invD[:, None]
    c = np.sum(dout * o, axis=1) * invD

    def through_normalisation(x, xh, dxh):
        n = math.sqrt(float(np.sum(x * x)))
        return (dxh - xh * np.dot(xh, dxh)) / n if n > 0 else np.zeros_like(x)

    dq = np.zeros((len(rows_q), d))
    for j, t in enumerate(rows_q):
        s = kh[:t + 1] @ qh[t]
        e = v[:t + 1] @ u[t] - c[t]
        dq[j] = through_normalisation(q[t], qh[t], 2.0 * (s * e) @ kh[:t + 1])
    dk = np.zeros((len(rows_k), d))
    dv = np.zeros((len(rows_k), v.shape[1]))
    for j, i in enumerate(rows_k):
        s = qh[i:] @ kh[i]
        e = u[i:] @ v[i] - c[i:]
        dk[j] = through_normalisation(k[i], kh[i], 2.0 * (s * e) @ qh[i:])
        dv[j] = (s * s) @ u[i:]
    return dq, dk, dv


def kata_decode_step(S, Z, q, k, v, feature: str = "psd_direct"):
    """One token of the recurrent form ("Linear attention as a recurrence": S_t = S_{t-1} + psi(k_t) v_t^T,
    Z_t = Z_{t-1} + psi(k_t), readout psi(q_t)^T S_t / psi(q_t)^T Z_t; 0 where the denominator is 0).

    S [n_psi, d_v], Z [n_psi], q, k [d_k], v [d_v].  Returns (o, S_new, Z_new); the inputs are not modified.
    """
    fq = apply_feature(np.asarray(q, dtype=np.float64)[None, :], feature)[0]
    fk = apply_feature(np.asarray(k, dtype=np.float64)[None, :], feature)[0]
    v = np.asarray(v, dtype=np.float64)
    S_new = np.asarray(S, dtype=np.float64) + np.outer(fk, v)
    Z_new = np.asarray(Z, dtype=np.float64) + fk
    den = fq @ Z_new
    o = (fq @ S_new) / den if den != 0 else np.zeros_like(v)
    return o, S_new, Z_new


# ---------------------------------------------------------------------------
# form C: Algorithm 1 (chunkwise forward)
# ---------------------------------------------------------------------------

def _pad_chunks(x: np.ndarray, C: int) -> np.ndarray:
    T = x.shape[0]
    NC = -(-T // C)
    out = np.zeros((NC * C,) + x.shape[1:])
    out[:T] = x
    return out.reshape((NC, C) + x.shape[1:])


def chunk_output(FQ, FK, V, S, Z):
    """Chunk-output equations: P=(Psi(Q)Psi(K)^T) o M; N=Psi(Q)S+PV; D=Psi(Q)Z+P1; O=diag(D)^-1 N."""
    C = FQ.shape[0]
    M = np.tril(np.ones((C, C)))
    P = (FQ @ FK.T) * M
    N = FQ @ S + P @ V
    D = FQ @ Z + P @ np.ones(C)
    return _safe_div(N, D), N, D


def kata_chunked(q, k, v, C: int, feature: str = "psd_direct"):
    """Algorithm 1: pad, S_[0]=0, Z_[0]=0, per chunk output then state update; truncate to T."""
    T = q.shape[0]
    FQ = _pad_chunks(apply_feature(q, feature), C)
    FK = _pad_chunks(apply_feature(k, feature), C)
    V = _pad_chunks(np.asarray(v, np.float64), C)
    NC, _, n = FK.shape
    S = np.zeros((n, V.shape[2]))
    Z = np.zeros(n)
    o = np.zeros((NC, C, V.shape[2]))
    for c in range(NC):
        o[c], _, _ = chunk_output(FQ[c], FK[c], V[c], S, Z)
        S = S + FK[c].T @ V[c]
        Z = Z + FK[c].T @ np.ones(C)
    return o.reshape(NC * C, -1)[:T]


# ---------------------------------------------------------------------------
# form S: chunk-state -> exclusive prefix -> chunk-output
# ---------------------------------------------------------------------------

def chunk_local_states(k, v, C: int, feature: str = "psd_direct"):
    """Stage (i): S_loc^(c) = Psi(K_[c])^T V_[c], Z_loc^(c) = 1^T Psi(K_[c]) for every chunk."""
    FK = _pad_chunks(apply_feature(k, feature), C)
    V = _pad_chunks(np.asarray(v, np.float64), C)
    S_loc = np.einsum("ctn,ctv->cnv", FK, V)
    Z_loc = FK.sum(axis=1)
    return S_loc, Z_loc


def scan_rounds(NC: int) -> int:
    """ceil(log2 N_C) rounds of the log-depth exclusive scan."""
    return 0 if NC <= 1 else int(math.ceil(math.log2(NC)))


def exclusive_prefix_running(x: np.ndarray) -> np.ndarray:
    """pre[c] = sum_{c'<c} x[c'] by a plain running sum; pre[0] = 0."""
    pre = np.zeros_like(x)
    acc = np.zeros_like(x[0])
    for c in range(x.shape[0]):
        pre[c] = acc
        acc = acc + x[c]
    return pre


def exclusive_prefix_doubling(x: np.ndarray):
    """Same prefix in ceil(log2 N_C) rounds: inclusive doubling scan, then shift by one chunk.

    Returns (pre, rounds).
    """
    NC = x.shape[0]
    inc = x.copy()
    rounds = 0
    step = 1
    while step < NC:
        nxt = inc.copy()
        nxt[step:] = inc[step:] + inc[:-step]
        inc = nxt
        step *= 2
        rounds += 1
    pre = np.zeros_like(x)
    pre[1:] = inc[:-1]
    return pre, rounds


def kata_scan(q, k, v, C: int, feature: str = "psd_direct", prefix: str = "doubling"):
    """Three-stage pipeline.  Returns (o, S_pre, Z_pre) with S_pre[0]=0, Z_pre[0]=0."""
    T = q.shape[0]
    S_loc, Z_loc = chunk_local_states(k, v, C, feature)
    if prefix == "doubling":
        S_pre, _ = exclusive_prefix_doubling(S_loc)
        Z_pre, _ = exclusive_prefix_doubling(Z_loc)
    elif prefix == "running":
        S_pre = exclusive_prefix_running(S_loc)
        Z_pre = exclusive_prefix_running(Z_loc)
    else:
        raise ValueError(prefix)
    FQ = _pad_chunks(apply_feature(q, feature), C)
    FK = _pad_chunks(apply_feature(k, feature), C)
    V = _pad_chunks(np.asarray(v, np.float64), C)
    NC = FK.shape[0]
    o = np.zeros((NC, C, V.shape[2]))
    for c in range(NC):
        o[c], _, _ = chunk_output(FQ[c], FK[c], V[c], S_pre[c], Z_pre[c])
    return o.reshape(NC * C, -1)[:T], S_pre, Z_pre


# ---------------------------------------------------------------------------
# Proposition 1: the normaliser as a convex output gate
# ---------------------------------------------------------------------------

def gate_decomposition(q, k, v, feature: str = "psd_direct"):
    """Per token: D_{t-1} = psi(q_t)^T Z_{t-1}, c_t = psi(q_t)^T psi(k_t), D_t = D_{t-1}+c_t,
    alpha = D_{t-1}/D_t, beta = c_t/D_t, z_t = alpha * zbar_{t|t-1} + beta * v_t,
    zbar_{t|t-1} = psi(q_t)^T S_{t-1} / D_{t-1};  D_{t-1}=0 gives (alpha,beta)=(0,1), z_t=v_t.

    Returns dict(alpha, beta, D_prev, c, o) with o built only from the gate formula.
    """
    fq = apply_feature(q, feature)
    fk = apply_feature(k, feature)
    v = np.asarray(v, dtype=np.float64)
    T, n = fk.shape
    S = np.zeros((n, v.shape[1]))
    Z = np.zeros(n)
    alpha = np.zeros(T)
    beta = np.zeros(T)
    Dp = np.zeros(T)
    cc = np.zeros(T)
    o = np.zeros_like(v)
    for t in range(T):
        Dp[t] = fq[t] @ Z
        cc[t] = fq[t] @ fk[t]
        Dt = Dp[t] + cc[t]
        if Dt != 0:
            alpha[t] = Dp[t] / Dt
            beta[t] = cc[t] / Dt
            if Dp[t] != 0:
                o[t] = alpha[t] * ((fq[t] @ S) / Dp[t]) + beta[t] * v[t]
            else:
                o[t] = v[t]
        S += np.outer(fk[t], v[t])
        Z += fk[t]
    return dict(alpha=alpha, beta=beta, D_prev=Dp, c=cc, o=o)


# ---------------------------------------------------------------------------
# batched wrappers ([B,H,T,d] layouts)
# ---------------------------------------------------------------------------

def batched(fn, q, k, v, *args, **kw) -> np.ndarray:
    """Apply a per-head form returning o (or a tuple whose first item is o) over [B,H,...]."""
    B, H = q.shape[:2]
    out = np.zeros(v.shape, dtype=np.float64)
    for b in range(B):
        for h in range(H):
            r = fn(q[b, h], k[b, h], v[b, h], *args, **kw)
            out[b, h] = r[0] if isinstance(r, tuple) else r
    return out
