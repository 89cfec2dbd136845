"""The seeded input generators: formats, distributions, determinism, outlier channels."""
import numpy as np

from paper_2606_11357_b200 import workloads as wl
from helpers import bf16_bits_to_f64


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.00390625, 1.01171875, 1.0 + 2**-8 + 2**-20, -3.0e38, 1e-40], dtype=np.float32)
    # 1 + 2^-8 is a tie between 0x3F80 and 0x3F81 -> even (0x3F80); 1 + 3*2^-8 ties to 0x3F82
    bits = wl.f32_to_bf16_bits(x)
    assert bits[:4].tolist() == [0x3F80, 0x3F80, 0x3F82, 0x3F81]
    back = bf16_bits_to_f64(bits)
    assert np.all(np.abs(back[:5] - x[:5].astype(np.float64)) <= np.abs(x[:5]) * 2.0**-8)


def test_w4_problem_formats_and_ranges():
    p = wl.make_w4(4, 512, 72, seed=1, keep_raw=True)
    assert p.a_bf16.shape == (4, 512) and p.a_bf16.dtype == np.uint16
    assert p.qweight.shape == (512, 9) and p.qweight.dtype == np.uint32
    assert p.qzeros.shape == (4, 9) and p.scales_f16.shape == (4, 72)
    assert p.scales_f16.dtype == np.float16
    s = p.scales_f16.astype(np.float64)
    assert s.min() >= 0.001 - 1e-6 and s.max() <= 0.02 + 1e-5
    assert set(np.unique(p.raw["q"])) == set(range(16))
    a = bf16_bits_to_f64(p.a_bf16)
    assert abs(a.mean()) < 0.1 and 0.9 < a.std() < 1.1


def test_w8_problem_formats_and_ranges():
    p = wl.make_w8(2, 256, 40, seed=2)
    assert p.w_i8.dtype == np.int8 and p.w_i8.shape == (256, 40)
    assert p.w_i8.min() >= -127 and p.w_i8.max() <= 127
    s = p.scales_f16.astype(np.float64)
    assert s.min() >= 0.0005 - 1e-6 and s.max() <= 0.005 + 1e-5
    assert p.qweight is None and p.qzeros is None


def test_seed_names_the_inputs():
    a, b, c = wl.make_w4(1, 128, 8, 5), wl.make_w4(1, 128, 8, 5), wl.make_w4(1, 128, 8, 6)
    assert np.array_equal(a.qweight, b.qweight) and np.array_equal(a.a_bf16, b.a_bf16)
    assert not np.array_equal(a.qweight, c.qweight)


def test_outlier_channels():
    p = wl.make_w4(64, 4096, 8, seed=2, outlier_frac=0.01)
    a = bf16_bits_to_f64(p.a_bf16)
    col_std = a.std(axis=0)
    big = np.sort(np.nonzero(col_std > 8.0)[0])
    assert len(big) == 41                                  # round(0.01 * 4096)
    assert np.all(col_std[big] > 12.0) and np.median(col_std) < 1.3


def test_config_shapes():
    p = wl.config0()
    assert (p.M, p.K, p.N, p.bits, p.seed) == (1, 4096, 4096, 4, 0)
    p = wl.config1(4, 4096, 1024)
    assert (p.M, p.K, p.N) == (4, 4096, 1024)
