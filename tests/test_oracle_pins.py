"""Pins for the fp64 oracle: things the paper and the mathematics fix, none of which
re-types the oracle's own formula.  CPU only."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import kata_oracle as ko

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def golden(name):
    out = {}
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            out[key] = float(vals[0])
    return out


def rng(seed):
    return np.random.default_rng(seed)


def rand_qkv(seed, T, d, dv):
    r = rng(seed)
    return r.standard_normal((T, d)), r.standard_normal((T, d)), r.standard_normal((T, dv))


# ---------------------------------------------------------------------------
# printed numbers
# ---------------------------------------------------------------------------

def test_rope_worked_example_weight():
    g = golden("rope_kernel_ratio.txt")
    ang = g["omega_delta"]
    q = np.array([[1.0, 0.0]])
    k = np.array([[math.cos(ang), math.sin(ang)]])
    w = ko.causal_weights(3.7 * q, 0.2 * k)[0, 0]       # scale must not matter
    assert round(w, 4) == g["r_kata"]
    assert abs(w - math.cos(ang) ** 2) < 1e-15
    # the companion softmax number, to check the fixture was read in the right way
    assert round(math.exp((math.cos(ang) - 1.0) / g["tau"]), 4) == g["r_softmax"]


def test_feature_widths_printed():
    g = golden("feature_widths.txt")
    d = int(g["d"])
    u = rng(0).standard_normal((3, d))
    assert ko.psi_direct(u).shape[-1] == g["direct"] == ko.feature_dim(d, "psd_direct")
    assert ko.psi_packed(u).shape[-1] == g["packed"] == ko.feature_dim(d, "psd_packed")


def test_state_entries_table():
    g = golden("state_entries_kata_m1.txt")
    d, dv = int(g["d"]), int(g["d_v"])
    k, v = rng(1).standard_normal((5, d)), rng(2).standard_normal((5, dv))
    S_loc, Z_loc = ko.chunk_local_states(k, v, 5, "psd_packed")
    assert g["layers"] * S_loc[0].size == g["state_entries"]
    assert Z_loc[0].size == d * (d + 1) // 2


def test_scan_rounds_printed():
    g = golden("scan_rounds.txt")
    NC = -(-int(g["T"]) // int(g["C"]))
    assert NC == g["n_chunks"]
    assert ko.scan_rounds(NC) == g["rounds"]
    x = rng(3).standard_normal((NC, 4, 3))
    pre, rounds = ko.exclusive_prefix_doubling(x)
    assert rounds == g["rounds"]
    assert np.all(pre[0] == 0)
    for n, r in [(1, 0), (2, 1), (3, 2), (5, 3), (128, 7), (512, 9), (2048, 11), (2049, 12)]:
        assert ko.scan_rounds(n) == r
        assert ko.exclusive_prefix_doubling(np.ones((n, 1)))[1] == r


def test_psnr_simplex_closed_form():
    g = golden("psnr_welch.txt")
    p, T = int(g["p"]), int(g["T"])
    # regular simplex: centre the T standard basis vectors of R^T, express in the (T-1)-dim span
    E = np.eye(T) - 1.0 / T
    U, s, _ = np.linalg.svd(E)
    keys = (U[:, :p] * s[:p])
    keys /= np.linalg.norm(keys, axis=1, keepdims=True)
    G = keys @ keys.T
    assert np.allclose(G[~np.eye(T, dtype=bool)], -1.0 / p, atol=1e-12)
    v = np.eye(T)                       # orthonormal values: coefficients are read off directly
    for j in range(T):
        q = np.tile(keys[j], (T, 1))
        o, _, _ = ko.kata_quadratic(q, keys, v)
        coef = o[T - 1]                 # a_i at the last position
        expected = np.full(T, p ** -2.0) / (1 + (T - 1) * p ** -2.0)
        expected[j] = 1.0 / (1 + (T - 1) * p ** -2.0)
        assert np.allclose(coef, expected, atol=1e-14)
        psnr = coef[j] ** 2 / np.sum(np.delete(coef, j) ** 2)
        assert abs(psnr - g["psnr"]) < 1e-9
        assert abs(psnr - p ** 2 * (T - 1) / (T - p) ** 2) < 1e-9


# ---------------------------------------------------------------------------
# kernel identity and packing
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("d", [1, 2, 3, 16, 64])
def test_kernel_identity(d):
    r = rng(d)
    u = ko.normalize_rows(r.standard_normal((7, d)))
    w = ko.normalize_rows(r.standard_normal((9, d)))
    ref = (u @ w.T) ** 2
    assert np.allclose(ko.psi_direct(u) @ ko.psi_direct(w).T, ref, atol=1e-14)
    assert np.allclose(ko.psi_packed(u) @ ko.psi_packed(w).T, ref, atol=1e-14)
    # unit Frobenius norm of the lift
    assert np.allclose(np.linalg.norm(ko.psi_direct(u), axis=1), 1.0, atol=1e-14)
    assert np.allclose(np.linalg.norm(ko.psi_packed(u), axis=1), 1.0, atol=1e-14)


def test_direct_layout_is_row_major_outer_product():
    u = np.array([2.0, 3.0, 5.0])
    f = ko.psi_direct(u)
    assert f.tolist() == [4, 6, 10, 6, 9, 15, 10, 15, 25]
    p = ko.psi_packed(u)
    s = math.sqrt(2.0)
    assert np.allclose(p, [4, 6 * s, 10 * s, 9, 15 * s, 25])


def test_normalize_zero_row():
    x = np.array([[0.0, 0.0], [3.0, 4.0]])
    assert ko.normalize_rows(x).tolist() == [[0.0, 0.0], [0.6, 0.8]]


# ---------------------------------------------------------------------------
# the forms agree
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("feature", ["psd_direct", "psd_packed", "identity"])
@pytest.mark.parametrize("T,d,dv", [(37, 5, 3), (64, 8, 8), (130, 4, 6)])
def test_forms_agree(feature, T, d, dv):
    q, k, v = rand_qkv(T * 100 + d, T, d, dv)
    if feature == "identity":
        q, k = np.abs(q), np.abs(k)
    oq, _, _ = ko.kata_quadratic(q, k, v, feature)
    orr = ko.kata_recurrent(q, k, v, feature)
    assert np.max(np.abs(oq - orr)) < 1e-10
    for C in (1, 2, 7, 64, T, T + 5):
        oc = ko.kata_chunked(q, k, v, C, feature)
        assert oc.shape == oq.shape
        assert np.max(np.abs(oq - oc)) < 1e-10, C
        for prefix in ("running", "doubling"):
            os_, S_pre, Z_pre = ko.kata_scan(q, k, v, C, feature, prefix)
            assert np.max(np.abs(oq - os_)) < 1e-10, (C, prefix)
            assert np.all(S_pre[0] == 0) and np.all(Z_pre[0] == 0)
    rows = [0, 1, T // 2, T - 1]
    assert np.max(np.abs(ko.kata_rows(q, k, v, rows, feature) - oq[rows])) < 1e-12


def test_config1_forms_agree_full_size():
    """B=1,H=2,T=512,d=16,C=64 (the tiny config), all forms."""
    from paper_2607_17419_b200 import inputs
    w = inputs.config(1)
    for h in range(w.H):
        q, k, v = w.q_ref[0, h], w.k_ref[0, h], w.v_ref[0, h]
        oq, _, _ = ko.kata_quadratic(q, k, v)
        assert np.max(np.abs(ko.kata_recurrent(q, k, v, "psd_packed") - oq)) < 1e-10
        assert np.max(np.abs(ko.kata_chunked(q, k, v, w.C, "psd_direct") - oq)) < 1e-10
        assert np.max(np.abs(ko.kata_scan(q, k, v, w.C, "psd_packed")[0] - oq)) < 1e-10


def test_prefix_two_ways_and_against_cumsum():
    x = rng(5).standard_normal((37, 6, 2))
    a = ko.exclusive_prefix_running(x)
    b, _ = ko.exclusive_prefix_doubling(x)
    c = np.concatenate([np.zeros((1, 6, 2)), np.cumsum(x, axis=0)[:-1]])
    assert np.allclose(a, c, atol=1e-12) and np.allclose(b, c, atol=1e-12)


def test_scan_states_match_running_state():
    q, k, v = rand_qkv(11, 50, 4, 3)
    C = 8
    _, S_pre, Z_pre = ko.kata_scan(q, k, v, C, "psd_direct")
    fk = ko.psi_direct(ko.normalize_rows(k))
    for c in range(S_pre.shape[0]):
        S = sum((np.outer(fk[i], v[i]) for i in range(c * C)), np.zeros((16, 3)))
        assert np.allclose(S_pre[c], S, atol=1e-12)
        assert np.allclose(Z_pre[c], fk[: c * C].sum(axis=0), atol=1e-12)


# ---------------------------------------------------------------------------
# brute force, written independently (scalar loops straight from the sums)
# ---------------------------------------------------------------------------

def brute(q, k, v):
    T, d, dv = len(q), len(q[0]), len(v[0])
    out = [[0.0] * dv for _ in range(T)]
    for t in range(T):
        nq = math.sqrt(sum(x * x for x in q[t]))
        num = [0.0] * dv
        den = 0.0
        for i in range(t + 1):
            nk = math.sqrt(sum(x * x for x in k[i]))
            if nq == 0 or nk == 0:
                w = 0.0
            else:
                w = (sum(q[t][a] * k[i][a] for a in range(d)) / (nq * nk)) ** 2
            den += w
            for j in range(dv):
                num[j] += w * v[i][j]
        if den != 0:
            out[t] = [x / den for x in num]
    return np.array(out)


@pytest.mark.parametrize("T,d,dv", [(1, 1, 1), (5, 2, 3), (8, 3, 2)])
def test_brute_force_tiny(T, d, dv):
    q, k, v = rand_qkv(T + 10 * d, T, d, dv)
    ref = brute(q.tolist(), k.tolist(), v.tolist())
    for feature in ("psd_direct", "psd_packed"):
        assert np.allclose(ko.kata_quadratic(q, k, v, feature)[0], ref, atol=1e-13)
        assert np.allclose(ko.kata_recurrent(q, k, v, feature), ref, atol=1e-13)
        assert np.allclose(ko.kata_chunked(q, k, v, 3, feature), ref, atol=1e-13)
        assert np.allclose(ko.kata_scan(q, k, v, 3, feature)[0], ref, atol=1e-13)


def test_zero_rows_and_zero_denominator():
    # first key zero -> D_0 = 0 -> o_0 = 0; orthogonal query/keys -> 0; zero query -> 0
    k = np.array([[0.0, 0.0], [1.0, 0.0], [1.0, 0.0], [0.0, 2.0]])
    q = np.array([[1.0, 1.0], [0.0, 1.0], [0.0, 0.0], [1.0, 1.0]])
    v = np.array([[1.0], [2.0], [4.0], [8.0]])
    ref = brute(q.tolist(), k.tolist(), v.tolist())
    assert ref[:3].tolist() == [[0.0], [0.0], [0.0]]
    assert abs(ref[3, 0] - (0.5 * 2 + 0.5 * 4 + 0.5 * 8) / 1.5) < 1e-15
    for C in (1, 2, 3, 4):
        assert np.allclose(ko.kata_chunked(q, k, v, C), ref, atol=1e-15)
        assert np.allclose(ko.kata_scan(q, k, v, C, "psd_packed")[0], ref, atol=1e-15)
    assert np.allclose(ko.kata_quadratic(q, k, v)[0], ref, atol=1e-15)
    assert np.allclose(ko.kata_recurrent(q, k, v), ref, atol=1e-15)


# ---------------------------------------------------------------------------
# textbook reductions and invariances
# ---------------------------------------------------------------------------

def test_dk1_is_running_mean():
    T = 40
    r = rng(7)
    q, k = r.standard_normal((T, 1)), r.standard_normal((T, 1))
    v = r.standard_normal((T, 3))
    mean = np.cumsum(v, axis=0) / np.arange(1, T + 1)[:, None]
    for o in (ko.kata_quadratic(q, k, v)[0], ko.kata_recurrent(q, k, v), ko.kata_chunked(q, k, v, 8),
              ko.kata_scan(q, k, v, 8)[0]):
        assert np.allclose(o, mean, atol=1e-13)


def test_orthonormal_keys_exact_retrieval():
    d = 6
    k = np.eye(d)
    v = rng(8).standard_normal((d, 4))
    for j in range(d):
        q = np.tile(k[j], (d, 1))
        o = ko.kata_chunked(q, k, v, 4)
        for t in range(j, d):
            assert np.allclose(o[t], v[j], atol=1e-15)
        assert np.all(o[:j] == 0)          # key j not yet seen: all weights 0 -> D = 0 -> 0


def test_first_row_is_first_value_and_constant_values():
    q, k, v = rand_qkv(9, 30, 5, 4)
    o, _, _ = ko.kata_quadratic(q, k, v)
    assert np.allclose(o[0], v[0], atol=1e-15)
    vc = np.tile(np.array([[1.5, -2.0]]), (30, 1))
    assert np.allclose(ko.kata_chunked(q, k, vc, 7), vc, atol=1e-13)


def test_convex_hull_and_nonnegative_weights():
    q, k, v = rand_qkv(10, 60, 4, 3)
    w = ko.causal_weights(q, k)
    assert np.all(w >= 0) and np.all(np.triu(w, 1) == 0)
    o = ko.kata_scan(q, k, v, 16)[0]
    lo = np.minimum.accumulate(v, axis=0)
    hi = np.maximum.accumulate(v, axis=0)
    assert np.all(o >= lo - 1e-12) and np.all(o <= hi + 1e-12)


def test_invariances():
    T, d, dv = 33, 6, 4
    q, k, v = rand_qkv(12, T, d, dv)
    r = rng(13)
    base = ko.kata_chunked(q, k, v, 8)
    cq = r.uniform(0.1, 5.0, (T, 1)) * r.choice([-1.0, 1.0], (T, 1))
    ck = r.uniform(0.1, 5.0, (T, 1)) * r.choice([-1.0, 1.0], (T, 1))
    assert np.allclose(ko.kata_chunked(q * cq, k * ck, v, 8), base, atol=1e-12)
    R, _ = np.linalg.qr(r.standard_normal((d, d)))
    assert np.allclose(ko.kata_chunked(q @ R, k @ R, v, 8), base, atol=1e-12)
    A, b = r.standard_normal((dv, 2)), r.standard_normal(2)
    assert np.allclose(ko.kata_chunked(q, k, v @ A + b, 8), base @ A + b, atol=1e-12)


def test_dense_matmul_definition():
    """tril((Q K^T)^2) V / rowsum with library matmuls on independently normalised rows."""
    q, k, v = rand_qkv(14, 48, 8, 5)
    qh = q / np.linalg.norm(q, axis=1, keepdims=True)
    kh = k / np.linalg.norm(k, axis=1, keepdims=True)
    W = np.tril(np.square(qh @ kh.T))
    ref = (W @ v) / W.sum(axis=1, keepdims=True)
    assert np.allclose(ko.kata_recurrent(q, k, v, "psd_packed"), ref, atol=1e-12)
    assert np.allclose(ko.kata_chunked(q, k, v, 16), ref, atol=1e-12)


def test_identity_feature_is_plain_linear_attention():
    q, k, v = rand_qkv(15, 40, 6, 3)
    q, k = np.abs(q), np.abs(k)
    W = np.tril(q @ k.T)
    ref = (W @ v) / W.sum(axis=1, keepdims=True)
    assert np.allclose(ko.kata_scan(q, k, v, 8, "identity")[0], ref, atol=1e-12)
    S_loc, Z_loc = ko.chunk_local_states(k, v, 8, "identity")
    assert np.allclose(S_loc[1], k[8:16].T @ v[8:16], atol=1e-13)
    assert np.allclose(Z_loc[4], k[32:40].sum(axis=0), atol=1e-13)


# ---------------------------------------------------------------------------
# Proposition 1: the normaliser is a convex gate
# ---------------------------------------------------------------------------

def test_gate_decomposition():
    q, k, v = rand_qkv(16, 45, 5, 3)
    k[0] = 0.0                                   # D_0 = 0 and D_1 = c_1 only
    g = ko.gate_decomposition(q, k, v)
    o = ko.kata_quadratic(q, k, v)[0]
    assert np.all(g["alpha"] >= 0) and np.all(g["beta"] >= 0)
    live = (g["D_prev"] + g["c"]) > 0
    assert np.allclose((g["alpha"] + g["beta"])[live], 1.0, atol=1e-14)
    assert np.allclose(g["o"], o, atol=1e-12)
    assert g["alpha"][1] == 0.0 and g["beta"][1] == 1.0 and np.allclose(o[1], v[1])
    assert np.all(o[0] == 0)
    # D_{t-1} uses the *current* query against the previous state
    w = ko.causal_weights(q, k)
    assert np.allclose(g["D_prev"], w.sum(axis=1) - np.diag(w), atol=1e-13)
    assert np.allclose(g["c"], np.diag(w), atol=1e-15)


def test_batched_wrapper():
    r = rng(17)
    q, k = r.standard_normal((2, 3, 20, 4)), r.standard_normal((2, 3, 20, 4))
    v = r.standard_normal((2, 3, 20, 5))
    ob = ko.batched(ko.kata_chunked, q, k, v, 8)
    for b, h in itertools.product(range(2), range(3)):
        assert np.array_equal(ob[b, h], ko.kata_chunked(q[b, h], k[b, h], v[b, h], 8))
    ob2 = ko.batched(ko.kata_quadratic, q, k, v)
    assert np.allclose(ob, ob2, atol=1e-12)


# ---------------------------------------------------------------------------
# decode step (the recurrence taken one token at a time)
# ---------------------------------------------------------------------------

def _decode_all(q, k, v, feature):
    n = ko.feature_dim(q.shape[1], feature)
    S, Z = np.zeros((n, v.shape[1])), np.zeros(n)
    out = []
    for t in range(q.shape[0]):
        o, S, Z = ko.kata_decode_step(S, Z, q[t], k[t], v[t], feature)
        out.append(o)
    return np.array(out), S, Z


@pytest.mark.parametrize("feature", ["psd_direct", "psd_packed", "identity"])
def test_decode_steps_from_zero_state_give_the_definition(feature):
    # brute force (pure Python loops over the definition) for the PSD features; for the identity feature the
    # weights are plain dot products, checked against a dense masked matmul
    q, k, v = rand_qkv(31, 7, 3, 2)
    o, S, Z = _decode_all(q, k, v, feature)
    if feature == "identity":
        w = np.tril(q @ k.T)
        ref = (w @ v) / w.sum(axis=1, keepdims=True)
    else:
        ref = brute(q.tolist(), k.tolist(), v.tolist())
    assert np.allclose(o, ref, atol=1e-12)
    # the state is the plain sum of feature-value outer products; its row sums against ones give Z
    fk = ko.apply_feature(k, feature)
    assert np.allclose(S, fk.T @ v, atol=1e-13) and np.allclose(Z, fk.sum(axis=0), atol=1e-13)


def test_decode_step_special_cases():
    # d_k = 1: every weight is 1, so the outputs are the running mean of v
    r = rng(33)
    q, k, v = r.standard_normal((9, 1)), r.standard_normal((9, 1)), r.standard_normal((9, 3))
    o, _, Z = _decode_all(q, k, v, "psd_direct")
    assert np.allclose(o, np.cumsum(v, axis=0) / np.arange(1, 10)[:, None], atol=1e-13)
    assert np.allclose(Z, [9.0])
    # zero key leaves the state unchanged; zero query reads 0; the inputs are not modified
    S0, Z0 = np.ones((4, 2)), np.ones(4)
    o, S1, Z1 = ko.kata_decode_step(S0, Z0, [1.0, 2.0], [0.0, 0.0], [5.0, 6.0])
    assert np.array_equal(S1, S0) and np.array_equal(Z1, Z0) and np.all(S0 == 1)
    o, _, _ = ko.kata_decode_step(S0, Z0, [0.0, 0.0], [1.0, 0.0], [5.0, 6.0])
    assert np.all(o == 0)
    # resuming from the exclusive-prefix state of a chunk reproduces the rest of the sequence
    q, k, v = rand_qkv(35, 12, 3, 2)
    full = ko.kata_quadratic(q, k, v)[0]
    _, S_pre, Z_pre = ko.kata_scan(q, k, v, 4)
    S, Z = S_pre[2], Z_pre[2]
    for t in range(8, 12):
        o, S, Z = ko.kata_decode_step(S, Z, q[t], k[t], v[t])
        assert np.allclose(o, full[t], atol=1e-12)


# ---------------------------------------------------------------------------
# blockwise PSD map (KATA-Mg)
# ---------------------------------------------------------------------------

def brute_mg(q, k, v, g):
    """Definition with the blockwise kernel sum_a (q_hat_a . k_hat_a)^2, plain Python loops."""
    T, d, dv = len(q), len(q[0]), len(v[0])
    m = d // g

    def unit(x):
        n = math.sqrt(sum(t * t for t in x))
        return [t / n for t in x] if n > 0 else [0.0] * len(x)

    qh, kh = [unit(r) for r in q], [unit(r) for r in k]
    out = []
    for t in range(T):
        num, den = [0.0] * dv, 0.0
        for i in range(t + 1):
            w = 0.0
            for a in range(g):
                dot = sum(qh[t][a * m + e] * kh[i][a * m + e] for e in range(m))
                w += dot * dot
            den += w
            for c in range(dv):
                num[c] += w * v[i][c]
        out.append([x / den if den != 0 else 0.0 for x in num])
    return np.array(out)


@pytest.mark.parametrize("g", [1, 2, 4])
def test_blockwise_feature_against_brute_force(g):
    q, k, v = rand_qkv(60 + g, 9, 4, 3)
    ref = brute_mg(q.tolist(), k.tolist(), v.tolist(), g)
    if g == 1:
        assert np.allclose(ref, brute(q.tolist(), k.tolist(), v.tolist()), atol=1e-14)
    for base in ("psd_direct", "psd_packed"):
        f = f"{base}:g{g}"
        assert np.allclose(ko.kata_quadratic(q, k, v, f)[0], ref, atol=1e-13)
        assert np.allclose(ko.kata_recurrent(q, k, v, f), ref, atol=1e-13)
        assert np.allclose(ko.kata_chunked(q, k, v, 4, f), ref, atol=1e-13)
        assert np.allclose(ko.kata_scan(q, k, v, 4, f)[0], ref, atol=1e-13)
    # g = 1 with the suffix is the plain feature
    assert np.array_equal(ko.apply_feature(q, "psd_direct:g1"), ko.apply_feature(q, "psd_direct"))


def test_blockwise_feature_sizes_and_kernel():
    # state entries d (d/g + 1) / 2 * d_v: the paper's 266,240 (M1) and 135,168 (M2) at d = 64, d_v = 128
    assert ko.feature_dim(64, "psd_packed") * 128 == 266240
    assert ko.feature_dim(64, "psd_packed:g2") * 128 == 135168
    assert ko.feature_dim(64, "psd_direct:g4") == 4 * 16 * 16
    # kernel identity <psi(q), psi(k)> = sum_a (q_a . k_a)^2 on the normalised rows, both packings
    r = rng(71)
    q, k = r.standard_normal((5, 8)), r.standard_normal((6, 8))
    qh, kh = ko.normalize_rows(q), ko.normalize_rows(k)
    for g in (2, 4):
        m = 8 // g
        want = sum((qh[:, a * m:(a + 1) * m] @ kh[:, a * m:(a + 1) * m].T) ** 2 for a in range(g))
        for base in ("psd_direct", "psd_packed"):
            got = ko.apply_feature(q, f"{base}:g{g}") @ ko.apply_feature(k, f"{base}:g{g}").T
            assert np.allclose(got, want, atol=1e-14)
    # g = d: every block is one coordinate, the kernel is sum_a q_a^2 k_a^2
    got = ko.apply_feature(q, "psd_direct:g8") @ ko.apply_feature(k, "psd_direct:g8").T
    assert np.allclose(got, (qh ** 2) @ (kh ** 2).T, atol=1e-14)
    with pytest.raises(ValueError):
        ko.apply_feature(q, "psd_direct:g3")
    with pytest.raises(ValueError):
        ko.apply_feature(q, "identity:g2")


# ---------------------------------------------------------------------------
# backward of the definition
# ---------------------------------------------------------------------------

def _loss(q, k, v, dout, feature):
    return float(np.sum(dout * ko.kata_quadratic(q, k, v, feature)[0]))


@pytest.mark.parametrize("feature", ["psd_direct", "psd_direct:g2", "psd_packed:g4", "identity"])
def test_backward_matches_central_differences(feature):
    """Every entry of dq, dk, dv against (L(x + h e) - L(x - h e)) / 2h of the forward definition."""
    r = np.random.default_rng(71)
    T, d, dv = 9, 8, 5
    q, k, v, dout = r.normal(size=(T, d)), r.normal(size=(T, d)), r.normal(size=(T, dv)), r.normal(size=(T, dv))
    if feature == "identity":
        q, k = np.abs(q) + 0.1, np.abs(k) + 0.1          # keep the normaliser away from 0
    dq, dk, dvv = ko.kata_quadratic_bwd(q, k, v, dout, feature)
    h = 1e-6
    for name, x, grad in (("q", q, dq), ("k", k, dk), ("v", v, dvv)):
        num = np.zeros_like(x)
        for idx in np.ndindex(*x.shape):
            old = x[idx]
            x[idx] = old + h
            lp = _loss(q, k, v, dout, feature)
            x[idx] = old - h
            lm = _loss(q, k, v, dout, feature)
            x[idx] = old
            num[idx] = (lp - lm) / (2 * h)
        assert np.max(np.abs(num - grad)) <= 2e-7 * max(1.0, np.abs(grad).max()), name


def test_backward_invariants():
    r = np.random.default_rng(72)
    T, d, dv = 40, 16, 12
    q, k, v, dout = r.normal(size=(T, d)), r.normal(size=(T, d)), r.normal(size=(T, dv)), r.normal(size=(T, dv))
    for feature in ("psd_direct", "psd_direct:g2", "psd_direct:g4"):
        dq, dk, dvv = ko.kata_quadratic_bwd(q, k, v, dout, feature)
        # o does not change when a query or a key row is rescaled (degree 0): Euler's relation per row
        assert np.max(np.abs(np.sum(dq * q, axis=1))) <= 1e-12
        assert np.max(np.abs(np.sum(dk * k, axis=1))) <= 1e-12
        # adding one vector c to every value row adds c to every output row: sum_i dv_i = sum_t dout_t
        assert np.max(np.abs(dvv.sum(axis=0) - dout.sum(axis=0))) <= 1e-12
        # packed and direct coordinates are the same function of q, k
        dq2, dk2, dv2 = ko.kata_quadratic_bwd(q, k, v, dout, feature.replace("direct", "packed"))
        assert np.max(np.abs(dq - dq2)) <= 1e-13 and np.max(np.abs(dk - dk2)) <= 1e-13 and np.max(np.abs(dvv - dv2)) <= 1e-13
    # first-order feature: degree 0 in the common scale of ALL keys only (one relation in total)
    qp, kp = np.abs(q) + 0.1, np.abs(k) + 0.1
    dq, dk, dvv = ko.kata_quadratic_bwd(qp, kp, v, dout, "identity")
    assert abs(np.sum(dk * kp)) <= 1e-10 and np.max(np.abs(np.sum(dq * qp, axis=1))) <= 1e-10
    # token 0 sees only itself: o_0 = v_0 whatever q_0, k_0 are
    dq, dk, dvv = ko.kata_quadratic_bwd(q[:1], k[:1], v[:1], dout[:1])
    assert np.max(np.abs(dq)) <= 1e-12 and np.max(np.abs(dk)) <= 1e-12 and np.allclose(dvv, dout[:1])


def test_backward_zero_rows_and_dead_denominators():
    r = np.random.default_rng(73)
    T, d, dv = 12, 8, 4
    q, k, v, dout = r.normal(size=(T, d)), r.normal(size=(T, d)), r.normal(size=(T, dv)), r.normal(size=(T, dv))
    k[0] = 0
    k[1] = 0            # rows 0, 1 have D = 0
    k[5] = 0
    q[7] = 0
    dq, dk, dvv = ko.kata_quadratic_bwd(q, k, v, dout)
    assert np.all(np.isfinite(dq)) and np.all(np.isfinite(dk)) and np.all(np.isfinite(dvv))
    assert np.all(dk[[0, 1, 5]] == 0) and np.all(dq[[0, 1, 7]] == 0) and np.all(dvv[[0, 1, 5]] == 0)
    # rows 0, 1 are dead as keys (zero feature) and as queries (D = 0): the rest is the problem without them
    keep = list(range(2, T))
    dq2, dk2, dv2 = ko.kata_quadratic_bwd(q[keep], k[keep], v[keep], dout[keep])
    assert np.allclose(dq[keep], dq2, atol=1e-13) and np.allclose(dk[keep], dk2, atol=1e-13)
    assert np.allclose(dvv[keep], dv2, atol=1e-13)
    # a key with a zero feature carries zero weight: its value row does not matter to anything
    v2 = v.copy()
    v2[5] += 100.0
    dq3, dk3, dv3 = ko.kata_quadratic_bwd(q, k, v2, dout)
    assert np.allclose(dq3, dq, atol=1e-12) and np.allclose(dk3, dk, atol=1e-12) and np.allclose(dv3, dvv, atol=1e-12)


def test_backward_rows_equal_the_backward_of_the_definition():
    """`kata_bwd_rows` (the long-sequence helper: forward by the chunk equations, then each requested row as the sum
    the chain rule states) against `kata_quadratic_bwd` on every row of a short sequence, including a zero key row,
    a zero query row and a ragged last chunk; and against central differences of the definition for one row."""
    rng = np.random.default_rng(77)
    T, d, dv = 150, 8, 5
    q, k, v, dout = (rng.standard_normal((T, n)) for n in (d, d, dv, dv))
    k[3] = 0.0
    q[10] = 0.0
    rq, rk, rv = ko.kata_quadratic_bwd(q, k, v, dout)
    rows = list(range(T))
    for C in (64, 256, 7):
        dq, dk, dvv = ko.kata_bwd_rows(q, k, v, dout, rows, rows, C=C)
        for got, ref in ((dq, rq), (dk, rk), (dvv, rv)):
            assert np.max(np.abs(got - ref)) <= 1e-10 * max(1.0, np.abs(ref).max())
    # a subset in arbitrary order
    sel = [149, 0, 64, 63, 3]
    dq, dk, dvv = ko.kata_bwd_rows(q, k, v, dout, sel, sel[::-1])
    assert np.allclose(dq, rq[sel], atol=1e-10) and np.allclose(dk, rk[sel[::-1]], atol=1e-10)
    assert np.allclose(dvv, rv[sel[::-1]], atol=1e-10)
    # central differences of L = sum(dout * o) in k[40]
    L = lambda kk: float(np.sum(dout * ko.kata_quadratic(q, kk, v)[0]))
    eps = 1e-6
    num = np.zeros(d)
    for a in range(d):
        kp, km = k.copy(), k.copy()
        kp[40, a] += eps
        km[40, a] -= eps
        num[a] = (L(kp) - L(km)) / (2 * eps)
    assert np.allclose(ko.kata_bwd_rows(q, k, v, dout, [], [40])[1][0], num, rtol=1e-5, atol=1e-7)
