"""The seeded input generator: published test vector, statistics, bf16 rounding, slicing."""
import numpy as np
import pytest

from paper_2410_09397_b200 import inputs


def test_splitmix64_published_vector():
    # first outputs of splitmix64 seeded with 0 (reference implementation by S. Vigna)
    with np.errstate(over="ignore"):
        z = inputs._mix(np.arange(1, 4, dtype=np.uint64) * inputs.GOLDEN)
    assert [int(v) for v in z] == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]


def test_normal_statistics_and_streams_differ():
    x = inputs.normal_f32(3, 0, 1 << 20).astype(np.float64)
    assert abs(x.mean()) < 5e-3 and abs(x.var() - 1) < 1e-2
    assert abs((x ** 3).mean()) < 2e-2 and abs((x ** 4).mean() - 3) < 5e-2
    y = inputs.normal_f32(4, 0, 1 << 20).astype(np.float64)
    assert abs(np.corrcoef(x, y)[0, 1]) < 5e-3
    assert abs(np.corrcoef(x[:-1], x[1:])[0, 1]) < 5e-3


def test_slices_are_addressable():
    full = inputs.normal_f32(9, 0, 5000, chunk=777)
    part = inputs.normal_f32(9, 1234, 1000, chunk=333)
    assert np.array_equal(full[1234:2234], part)
    w = inputs.WORKLOADS["C2"]
    t = w.tensors(head_slice=(5, 7))
    one = inputs.normal_tensor(w.seed, inputs.TENSOR_K, (1, w.n, w.d), bf16=True, start=6 * w.n * w.d)
    assert np.array_equal(t["K"][1:2], one)


def test_bf16_rounding_matches_torch():
    torch = pytest.importorskip("torch")
    x = inputs.normal_f32(1, 0, 100000)
    x = np.concatenate([x, np.array([1.00390625, 1.01171875, -1.00390625, 0.0, 3.0e38], np.float32)])
    bits = inputs.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16)
    assert np.array_equal(bits.view(np.int16), ref.view(torch.int16).numpy())
    assert np.array_equal(inputs.bf16_bits_to_f32(bits), ref.float().numpy())


def test_block_mask_recipe():
    m = inputs.block_mask(5, 256, 0.1)
    assert m.shape == (1, 256, 256) and m.dtype == np.uint8
    assert np.all(np.diagonal(m[0]) == 1)
    off = m[0].sum() - 256
    assert abs(off / (256 * 255) - 0.1) < 0.01
    assert np.array_equal(m, inputs.block_mask(5, 256, 0.1))
    assert not np.array_equal(m, inputs.block_mask(6, 256, 0.1))
