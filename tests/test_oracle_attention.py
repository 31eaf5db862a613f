"""Pins of the oracle's attention proposal (Sec. 4.5): pixelwise entropy of the softmax over the channels of
the last convolutional layer, hard threshold at the image's mean entropy, the mask reused at every
resolution."""
import numpy as np
from scipy import special, stats


def test_entropy_against_a_library_routine_and_closed_forms(oracle):
    rng = np.random.default_rng(1)
    q = rng.integers(0, 16, size=(2, 3, 4, 37)).astype(np.uint8)
    step = 0.37
    h = oracle.attention_entropy(q, step)
    ref = stats.entropy(special.softmax(q.astype(np.float64) * step, axis=-1), axis=-1)
    assert np.allclose(h, ref, rtol=1e-12, atol=1e-14)
    # equal activations: the uniform distribution, log C; adding a constant to every channel changes nothing
    assert np.allclose(oracle.attention_entropy(np.full((1, 1, 1, 64), 9, np.uint8), 0.5), np.log(64))
    assert np.allclose(oracle.attention_entropy(q + 7, step), h, rtol=1e-12)
    # one channel far above the rest: nearly zero; two equal channels far above the rest: log 2
    one = np.zeros((1, 1, 1, 100), np.uint8); one[..., 3] = 255
    assert oracle.attention_entropy(one, 1.0) < 1e-100
    two = np.zeros((1, 1, 1, 100), np.uint8); two[..., [3, 70]] = 255
    assert np.allclose(oracle.attention_entropy(two, 1.0), np.log(2))
    # signed codes
    s = rng.integers(-15, 16, size=(1, 2, 2, 9)).astype(np.int8)
    assert np.allclose(oracle.attention_entropy(s, 0.2), stats.entropy(special.softmax(s * 0.2, axis=-1), axis=-1))


def test_mask_thresholds_at_the_image_mean_and_is_sampled_by_nearest_neighbour(oracle):
    rng = np.random.default_rng(2)
    h = rng.random((3, 7, 7))
    h[1] = np.arange(49).reshape(7, 7)                      # image 1: entropy grows with the pixel index
    maps, mean = oracle.attention_maps(h, 3, 4, [7, 14, 28, 5, 10])
    assert np.allclose(mean, h.reshape(3, -1).mean(1))
    assert set(np.unique(maps[7])) == {3, 4}
    assert np.array_equal(maps[7][1].reshape(-1), np.where(np.arange(49) > 24, 4, 3))      # mean of 0..48 is 24
    for n in range(3):
        assert np.array_equal(maps[7][n] == 4, h[n] > mean[n])
    # integer factors: every location of the small map becomes a block
    assert np.array_equal(maps[14], maps[7].repeat(2, 1).repeat(2, 2))
    assert np.array_equal(maps[28], maps[7].repeat(4, 1).repeat(4, 2))
    # other sizes: location (y, x) reads floor(y * 7 / r), floor(x * 7 / r)
    for r in (5, 10):
        for y in range(r):
            for x in range(r):
                assert np.array_equal(maps[r][:, y, x], maps[7][:, y * 7 // r, x * 7 // r])
    # a constant image: nothing is above the mean
    maps, _ = oracle.attention_maps(np.full((1, 4, 4), 2.5), 3, 4, [4])
    assert (maps[4] == 3).all()
