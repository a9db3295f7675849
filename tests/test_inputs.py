"""Host side of the seeded input generators (no method arithmetic in that module)."""
import math

import numpy as np
import pytest

from paper_1906_12043_b200 import inputs as I


def test_generator_is_a_pure_function_of_its_counters():
    a = I.gaussian(7, I.STREAM_GRAD, 3, 11, 1000, 257, 0.01)
    b = I.gaussian(7, I.STREAM_GRAD, 3, 11, 0, 2000, 0.01)[1000:1257]
    np.testing.assert_array_equal(a, b)                      # random access by element index
    cols = np.array([5, 1999, 0, 1000])
    np.testing.assert_array_equal(I.gaussian_at(7, I.STREAM_GRAD, 3, 11, cols, 0.01), b_full(cols))
    for other in [(8, I.STREAM_GRAD, 3, 11), (7, I.STREAM_X0, 3, 11), (7, I.STREAM_GRAD, 4, 11),
                  (7, I.STREAM_GRAD, 3, 12)]:
        assert not np.array_equal(I.gaussian(*other, 1000, 257, 0.01), a)


def b_full(cols):
    return I.gaussian(7, I.STREAM_GRAD, 3, 11, 0, 2000, 0.01)[cols]


def test_values_are_gaussian_with_the_stated_sigma():
    z = I.gaussian(0, I.STREAM_GRAD, 0, 0, 0, 1_000_000, 0.01).astype(np.float64) / 0.01
    assert abs(z.mean()) < 4e-3
    assert abs(z.var() - 1) < 6e-3
    assert abs((z ** 3).mean()) < 2e-2
    assert abs((z ** 4).mean() - 3) < 5e-2
    assert 4.0 < np.abs(z).max() < 6.7
    # independent across workers and steps
    z2 = I.gaussian(0, I.STREAM_GRAD, 1, 0, 0, 1_000_000, 0.01).astype(np.float64) / 0.01
    z3 = I.gaussian(0, I.STREAM_GRAD, 0, 1, 0, 1_000_000, 0.01).astype(np.float64) / 0.01
    assert abs((z * z2).mean()) < 5e-3 and abs((z * z3).mean()) < 5e-3


def test_polynomial_log_and_cosine_track_the_library_functions():
    key = I.stream_key(1, 2, 3, 4)
    h = I.element_bits(key, np.arange(200_000, dtype=np.uint64))
    z = I.std_normal_from_bits(h)
    u1 = ((h >> np.uint64(32)) + np.uint64(1)).astype(np.float64) / 2 ** 32
    u2 = (h & np.uint64(0xFFFFFFFF)).astype(np.float64) / 2 ** 32
    ref = np.sqrt(-2 * np.log(u1)) * np.cos(2 * np.pi * u2)
    assert np.abs(z - ref).max() < 2e-14
    # every octant and both extremes of u1
    hh = np.array([(0xFFFFFFFF << 32) | (o << 29) | r for o in range(8) for r in (0, 1, (1 << 29) - 1)]
                  + [0, 1 << 32], dtype=np.uint64)
    zz = I.std_normal_from_bits(hh)
    u1 = ((hh >> np.uint64(32)) + np.uint64(1)).astype(np.float64) / 2 ** 32
    u2 = (hh & np.uint64(0xFFFFFFFF)).astype(np.float64) / 2 ** 32
    rr = np.sqrt(-2 * np.log(u1)) * np.cos(2 * np.pi * u2)
    assert np.all(np.isfinite(zz)) and np.abs(zz - rr).max() < 1e-13


def test_mixer_matches_between_python_int_and_numpy():
    for z in (0, 1, I.GOLDEN, I.MASK64, 123456789123456789):
        assert int(I._mix64_np(np.array([z], dtype=np.uint64))[0]) == I.mix64_int(z)


def test_workload_recipes():
    x0 = I.initial_point(1000)
    assert x0.dtype == np.float32 and x0.shape == (1000,)
    np.testing.assert_array_equal(I.initial_point(1000, cols=np.array([3, 999])), x0[[3, 999]])
    g = I.gradients(3, 500, step=4)
    assert g.shape == (3, 500) and g.dtype == np.float32
    np.testing.assert_array_equal(I.gradients(3, 500, step=4, cols=np.array([0, 77]))[:, 1], g[:, 77])
    assert not np.array_equal(g[0], g[1])


@pytest.mark.parametrize("P,world", [(100_000, 2), (11_689_512, 8), (63, 4), (1, 2), (4096, 3)])
def test_shard_columns_tiles_the_vector(P, world):
    edges = [I.shard_columns(P, r, world) for r in range(world)]
    assert edges[0][0] == 0 and edges[-1][1] == P
    for (a, b), (c, d) in zip(edges, edges[1:]):
        assert b == c and a <= b
    for a, b in edges[:-1]:
        assert b % 64 == 0 or b == P
