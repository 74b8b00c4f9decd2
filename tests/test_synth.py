"""The seeded generator: reproducible, right distributions, right shapes."""

import numpy as np
import pytest

from paper_2504_08838_b200 import synth


def test_splitmix64_known_values():
    # first outputs of splitmix64 seeded with 0 (published test vector of the algorithm)
    z = synth.splitmix64(0, 3)
    assert [int(v) for v in z] == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]


def test_streams_are_reproducible_and_offsettable():
    a = synth.splitmix64(123, 100)
    b = synth.splitmix64(123, 40, offset=60)
    assert np.array_equal(a[60:], b)
    assert not np.array_equal(synth.splitmix64(124, 100), a)


def test_normal_moments_and_bf16_roundtrip():
    x = synth.normal(7, 200_000, 0.02)
    assert abs(x.mean()) < 3e-4 and abs(x.std() - 0.02) < 3e-4
    bits = synth.normal_bf16(7, (200_000,), 0.02)
    back = synth.bf16_bits_to_f32(bits)
    assert np.all(np.abs(back - x.astype(np.float32)) <= np.abs(x) * 2.0 ** -8 + 1e-30)
    assert np.array_equal(synth.f32_to_bf16_bits(back), bits)


def test_bernoulli_density():
    m = synth.bernoulli_mask(9, (512, 512), 0.3)
    assert abs(m.mean() - 0.3) < 0.01
    assert set(np.unique(m)) <= {0, 1}


def test_magnitude_mask_keeps_largest_per_row():
    M, K = 64, 256
    w = synth.normal_bf16(10, (M, K), 0.02)
    mask = synth.magnitude_mask(w, 11, 0.5)
    d_r = synth.row_densities(11, M, 0.5)
    assert np.all((d_r > 0) & (d_r < 1))
    keep = np.floor(d_r * K + 0.5).astype(int)
    assert np.array_equal(mask.sum(axis=1), keep)
    mag = (w & 0x7FFF).astype(np.int32)
    for r in range(M):
        if 0 < keep[r] < K:
            assert mag[r][mask[r] == 1].min() >= mag[r][mask[r] == 0].max()
    assert abs(mask.mean() - 0.5) < 0.05
    # 70 % sparsity: densities spread over (0, 0.6)
    d7 = synth.row_densities(12, 4096, 0.3)
    assert d7.min() > 0 and d7.max() < 0.6 and abs(d7.mean() - 0.3) < 0.01


def test_two_four_mask_keeps_two_largest_of_every_four():
    w = synth.normal_bf16(77, (37, 64), 0.02)
    m = synth.two_four_mask(w)
    assert m.shape == w.shape and m.dtype == np.uint8
    g = m.reshape(37, 16, 4)
    assert (g.sum(axis=2) == 2).all()
    mag = (w & np.uint16(0x7FFF)).astype(np.int32).reshape(37, 16, 4)
    kept_min = np.where(g == 1, mag, 1 << 20).min(axis=2)
    dropped_max = np.where(g == 0, mag, -1).max(axis=2)
    assert (kept_min >= dropped_max).all()
    # ties go to the lower column
    t = np.full((1, 4), 0x3C00, np.uint16)
    assert synth.two_four_mask(t).tolist() == [[1, 1, 0, 0]]
    with pytest.raises(ValueError):
        synth.two_four_mask(np.zeros((2, 6), np.uint16))
    w2, m2 = synth.make_linear(2, 0, 4, 8, 32, 0.5, "2:4")
    assert np.array_equal(m2, synth.two_four_mask(w2))


def test_drafter_shapes():
    assert [(n, m, k) for n, m, k in synth.LLAMA_1B.linears()] == [
        ("q", 2048, 2048), ("k", 512, 2048), ("v", 512, 2048), ("o", 2048, 2048),
        ("gate", 8192, 2048), ("up", 8192, 2048), ("down", 2048, 8192)]
    assert synth.QWEN_1P5B.linears()[6] == ("down", 1536, 8960)
    assert synth.LLAMA_3B.linears()[1] == ("k", 1024, 3072)
    w, mask = synth.make_linear(2, 0, 1, 512, 2048, 0.5)
    assert w.shape == mask.shape == (512, 2048) and w.dtype == np.uint16 and mask.dtype == np.uint8
    w2, _ = synth.make_linear(2, 1, 1, 512, 2048, 0.5)
    assert not np.array_equal(w, w2)
