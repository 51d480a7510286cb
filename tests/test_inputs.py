"""The seeded generators: determinism, distribution sanity, bf16 rounding, recall structure."""
import numpy as np

from paper_2607_17419_b200 import inputs


def test_deterministic_and_windowed():
    a = inputs.normal(3, 1, 1000)
    b = inputs.normal(3, 1, 1000)
    assert np.array_equal(a, b)
    assert np.array_equal(inputs.normal(3, 1, 100, start=400), a[400:500])
    assert not np.array_equal(a, inputs.normal(4, 1, 1000))
    assert not np.array_equal(a, inputs.normal(3, 2, 1000))


def test_normal_moments():
    x = inputs.normal(0, 0, 1 << 20)
    assert abs(x.mean()) < 5e-3 and abs(x.std() - 1.0) < 5e-3
    assert abs(np.mean(x ** 3)) < 2e-2 and abs(np.mean(x ** 4) - 3.0) < 5e-2
    assert abs(np.corrcoef(x[:-1], x[1:])[0, 1]) < 5e-3


def test_bf16_rounding_rne():
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 0.0, 3.0e38, 1e-40], dtype=np.float32)
    bits = inputs.f32_to_bf16_bits(x)
    back = inputs.bf16_bits_to_f32(bits)
    # 1 + 2^-8 is a tie between 1.0 and 1+2^-7 -> even (1.0); 1 + 3*2^-8 ties to 1+2^-6
    assert back[0] == 1.0 and back[1] == 1.0 and back[2] == np.float32(1.015625)
    assert back[3] == -2.5 and back[4] == 0.0
    import torch
    t = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(back, t)
    r = inputs.normal(5, 0, 4096).astype(np.float32)
    assert np.array_equal(inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(r)),
                          torch.from_numpy(r).to(torch.bfloat16).to(torch.float32).numpy())
    assert np.array_equal(inputs.bf16_bits_to_f64(bits), back.astype(np.float64))


def test_config1_shapes():
    w = inputs.config(1)
    assert (w.B, w.H, w.T, w.d_k, w.d_v, w.C, w.dtype) == (1, 2, 512, 16, 16, 64, "f32")
    assert w.q_dev.dtype == np.float32 and w.q_dev.shape == (1, 2, 512, 16)
    assert np.array_equal(w.q_ref, w.q_dev.astype(np.float64))


def test_recall_structure():
    w = inputs.recall_workload("r", "bf16", 2, 2, 256, 32, 32, 64, 4)
    assert w.k_dev.dtype == np.uint16
    k = w.k_ref.reshape(4, 256, 32)
    assert np.allclose(np.linalg.norm(k, axis=-1), 1.0, atol=1e-2)
    for h in range(4):
        assert len(np.unique(k[h], axis=0)) <= 256
        assert len(np.unique(k[h], axis=0)) < 256          # repeats exist at T = 256 draws of 256
    v = w.v_ref.reshape(4, 256, 32)
    assert np.all(v.sum(axis=-1) == 1.0) and np.all((v == 0) | (v == 1))
    # each query is close to some key at an earlier-or-equal position
    q = w.q_ref.reshape(4, 256, 32)
    for t in (0, 5, 100, 255):
        dist = np.linalg.norm(k[0, : t + 1] - q[0, t], axis=-1).min()
        assert dist < 0.1 * np.sqrt(32) * 2.0
