"""Pins of the oracle's max pooling: a hand-worked case and a library routine."""
import numpy as np
import pytest

import oracle


def test_hand_worked_3x3_stride2_pad1():
    # 1 channel, 4x4 image 0..15 row-major: windows clipped at the borders
    x = np.arange(16, dtype=np.float32).reshape(1, 4, 4, 1)
    y = oracle.maxpool2d(x, (3, 3), (2, 2), (1, 1))
    # output (0,0): rows -1..1, cols -1..1 -> max(0,1,4,5) = 5; (0,1): cols 1..3 -> 7; (1,0): rows 1..3 -> 13; (1,1) -> 15
    assert y.reshape(2, 2).tolist() == [[5.0, 7.0], [13.0, 15.0]]


def test_negative_values_are_not_beaten_by_padding():
    x = -np.ones((1, 3, 3, 2), dtype=np.float32)
    assert (oracle.maxpool2d(x, (3, 3), (2, 2), (1, 1)) == -1.0).all()     # padding is ignored, not zero


@pytest.mark.parametrize("kernel,stride,pad", [((3, 3), (2, 2), (1, 1)), ((2, 2), (2, 2), (0, 0)), ((3, 2), (1, 2), (1, 0))])
def test_equals_library_max_pool(kernel, stride, pad):
    torch = pytest.importorskip("torch")
    x = np.random.default_rng(3).standard_normal((2, 11, 9, 8)).astype(np.float32)
    want = torch.nn.functional.max_pool2d(torch.from_numpy(x).permute(0, 3, 1, 2), kernel, stride, pad).permute(0, 2, 3, 1).numpy()
    assert np.array_equal(oracle.maxpool2d(x, kernel, stride, pad), want)


def test_rejects_padding_as_large_as_the_window():
    with pytest.raises(ValueError):
        oracle.maxpool2d(np.zeros((1, 4, 4, 4), dtype=np.float32), (2, 2), (2, 2), (2, 2))
