"""Seeded synthetic inputs for the KATA forward (host side, numpy only).

This module holds none of the method's arithmetic: it only draws numbers.  The
CPU oracle and the CUDA path are both fed from the arrays produced here, so the
two sides always see bit-identical inputs.

Generator.  Every element is a pure function of (seed, stream, flat index):
a 64-bit counter ``seed * 2**40 + stream * 2**36 + index`` style key is mixed
with the splitmix64 finaliser, two such words give two uniforms and a
Box-Muller transform turns them into one N(0,1) sample.  Nothing depends on
numpy's own bit generators, so values are stable across numpy versions.

Streams: 0 = q, 1 = k, 2 = v, 3.. = auxiliary draws of the recall workload.

bf16 workloads hand out *both* the uint16 bit patterns (what the GPU reads)
and the exact float64 values of those bit patterns (what the oracle reads).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

_MASK = np.uint64(0xFFFFFFFFFFFFFFFF)


def _splitmix64(x: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser on uint64 arrays (wrapping arithmetic)."""
    with np.errstate(over="ignore"):
        z = (x + np.uint64(0x9E3779B97F4A7C15)) & _MASK
        z = ((z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _MASK
        z = ((z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _MASK
        return z ^ (z >> np.uint64(31))


def _words(seed: int, stream: int, lane: int, n: int, start: int = 0) -> np.ndarray:
    """n 64-bit words for flat indices start..start+n-1 of (seed, stream, lane)."""
    with np.errstate(over="ignore"):
        key = _splitmix64(
            np.array([(seed & 0xFFFFFFFF) * 0x100000000 + (stream & 0xFFFF) * 0x10000 + (lane & 0xFFFF)],
                     dtype=np.uint64)
        )[0]
        idx = np.arange(start, start + n, dtype=np.uint64)
        return _splitmix64((idx * np.uint64(0xD1342543DE82EF95) + key) & _MASK)


def uniform01(seed: int, stream: int, n: int, lane: int = 0, start: int = 0) -> np.ndarray:
    """n doubles in the open interval (0,1)."""
    w = _words(seed, stream, lane, n, start)
    return ((w >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal(seed: int, stream: int, n: int, start: int = 0) -> np.ndarray:
    """n iid N(0,1) doubles (Box-Muller on two independent uniform lanes)."""
    out = np.empty(n, dtype=np.float64)
    blk = 1 << 22
    for s in range(0, n, blk):
        m = min(blk, n - s)
        u1 = uniform01(seed, stream, m, lane=0, start=start + s)
        u2 = uniform01(seed, stream, m, lane=1, start=start + s)
        out[s:s + m] = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    return out


def randint(seed: int, stream: int, n: int, high: np.ndarray | int) -> np.ndarray:
    """n integers, element i uniform on {0..high_i-1} (high scalar or array)."""
    u = uniform01(seed, stream, n, lane=2)
    return np.minimum((u * high).astype(np.int64), np.asarray(high, dtype=np.int64) - 1)


# ---------------------------------------------------------------------------
# bf16 helpers (storage format conversion only)
# ---------------------------------------------------------------------------

def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even); returns uint16 bits."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    """Exact float64 value of bfloat16 bit patterns."""
    u = b.astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    u = b.astype(np.uint32) << np.uint32(16)
    return u.view(np.float32)


# ---------------------------------------------------------------------------
# workloads
# ---------------------------------------------------------------------------

@dataclass
class Workload:
    """One synthetic problem instance.

    q, k: [B,H,T,d_k]; v: [B,H,T,d_v].  ``*_dev`` is what is copied to the GPU
    (float32 arrays for dtype "f32", uint16 bf16 bit patterns for "bf16");
    ``*_ref`` is the exact float64 value of the same numbers for the oracle.
    """
    name: str
    dtype: str
    B: int
    H: int
    T: int
    d_k: int
    d_v: int
    C: int
    seed: int
    q_dev: np.ndarray
    k_dev: np.ndarray
    v_dev: np.ndarray
    q_ref: np.ndarray
    k_ref: np.ndarray
    v_ref: np.ndarray


def _finish(name, dtype, B, H, T, d_k, d_v, C, seed, q, k, v) -> Workload:
    q = q.astype(np.float32).reshape(B, H, T, d_k)
    k = k.astype(np.float32).reshape(B, H, T, d_k)
    v = v.astype(np.float32).reshape(B, H, T, d_v)
    if dtype == "f32":
        dev = (q, k, v)
        ref = tuple(a.astype(np.float64) for a in dev)
    elif dtype == "bf16":
        dev = tuple(f32_to_bf16_bits(a).reshape(a.shape) for a in (q, k, v))
        ref = tuple(bf16_bits_to_f64(a) for a in dev)
    else:
        raise ValueError(f"dtype {dtype!r}")
    return Workload(name, dtype, B, H, T, d_k, d_v, C, seed, *dev, *ref)


def gaussian_workload(name: str, dtype: str, B: int, H: int, T: int, d_k: int, d_v: int,
                      C: int, seed: int) -> Workload:
    """q, k, v iid N(0,1); generation order q, k, v; index order [B,H,T,d]."""
    q = normal(seed, 0, B * H * T * d_k)
    k = normal(seed, 1, B * H * T * d_k)
    v = normal(seed, 2, B * H * T * d_v)
    return _finish(name, dtype, B, H, T, d_k, d_v, C, seed, q, k, v)


def recall_workload(name: str, dtype: str, B: int, H: int, T: int, d_k: int, d_v: int,
                    C: int, seed: int, n_keys: int = 256, noise_sigma: float = 0.1) -> Workload:
    """Repeated-key recall pattern.

    Per (b,h): a dictionary of ``n_keys`` random unit vectors; position t holds
    dictionary entry id_t (uniform); the value is a one-hot row with a uniform
    index; the query at t is the key stored at a uniformly chosen earlier (or
    the same) position s_t in {0..t} plus N(0, noise_sigma^2) noise per
    component (variance 0.01 by default).
    """
    BH = B * H
    dic = normal(seed, 3, BH * n_keys * d_k).reshape(BH, n_keys, d_k)
    dic /= np.linalg.norm(dic, axis=-1, keepdims=True)
    ids = randint(seed, 4, BH * T, n_keys).reshape(BH, T)
    k = np.take_along_axis(dic, ids[:, :, None], axis=1)            # [BH,T,d_k]
    hot = randint(seed, 5, BH * T, d_v).reshape(BH, T)
    v = np.zeros((BH, T, d_v), dtype=np.float64)
    np.put_along_axis(v, hot[:, :, None], 1.0, axis=2)
    tpos = np.tile(np.arange(T, dtype=np.int64) + 1, BH)
    src = randint(seed, 6, BH * T, tpos).reshape(BH, T)
    q = np.take_along_axis(k, src[:, :, None], axis=1)
    q = q + noise_sigma * normal(seed, 0, BH * T * d_k).reshape(BH, T, d_k)
    return _finish(name, dtype, B, H, T, d_k, d_v, C, seed, q, k, v)


def near_orthogonal_workload(name: str, dtype: str, B: int, H: int, T: int, d_k: int, d_v: int, C: int, seed: int,
                             span: int = 48, every: int = 97, eps: float = 0.125) -> Workload:
    """Gaussian rows whose keys live in the first ``span`` coordinates; every ``every``-th query ("probe" rows
    t = every - 1, 2 every - 1, ...) has its part inside that span scaled by ``eps`` (a power of two), so that it is
    nearly orthogonal to every key up to and including its own: small normaliser, output still of order one."""
    q = normal(seed, 0, B * H * T * d_k).reshape(B, H, T, d_k)
    k = normal(seed, 1, B * H * T * d_k).reshape(B, H, T, d_k)
    v = normal(seed, 2, B * H * T * d_v)
    k[..., span:] = 0.0
    probes = np.arange(every - 1, T, every)
    if dtype == "bf16":                      # scale the rounded values, so that the scaling is exact
        q = bf16_bits_to_f64(f32_to_bf16_bits(q.astype(np.float32)).reshape(q.shape))
    q[:, :, probes, :span] *= eps
    return _finish(name, dtype, B, H, T, d_k, d_v, C, seed, q.reshape(-1), k.reshape(-1), v)


def nonnegative_workload(name: str, dtype: str, B: int, H: int, T: int, d_k: int, d_v: int,
                         C: int, seed: int) -> Workload:
    """|N(0,1)| features for q,k (already-mapped first-order features), N(0,1) values."""
    q = np.abs(normal(seed, 0, B * H * T * d_k))
    k = np.abs(normal(seed, 1, B * H * T * d_k))
    v = normal(seed, 2, B * H * T * d_v)
    return _finish(name, dtype, B, H, T, d_k, d_v, C, seed, q, k, v)


def config(idx: int, T: int | None = None) -> Workload:
    """The five benchmark configurations (1-based, as listed in the baseline file)."""
    if idx == 1:
        return gaussian_workload("c1_tiny_f32", "f32", 1, 2, 512, 16, 16, 64, 0)
    if idx == 2:
        return gaussian_workload("c2_quadratic_bf16", "bf16", 4, 16, 4096, 64, 64, 64, 1)
    if idx == 3:
        return gaussian_workload("c3_chunked_bf16", "bf16", 8, 16, 4096, 64, 64, 64, 2)
    if idx == 4:
        T = 131072 if T is None else T
        return gaussian_workload(f"c4_long_bf16_T{T}", "bf16", 1, 16, T, 64, 64, 64, 3)
    if idx == 5:
        return recall_workload("c5_recall_bf16", "bf16", 16, 8, 2048, 32, 32, 64, 4)
    raise ValueError(f"no config {idx}")
