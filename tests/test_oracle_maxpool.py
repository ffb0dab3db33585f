"""Pins for the oracle's max-pool (used to check the pooled tensor of the layer stack).

Max-pooling is not in the paper; the stack of ResNet-50 shapes needs it between the first layer and
the first bottleneck.  Definition: the maximum over the window positions that lie inside the image
(padding never wins, also when every value is negative).
"""
import numpy as np
import torch

import oracle


def test_hand_made_4x4_with_negative_values():
    # 1 image, 4x4, 1 channel, 3x3 window, stride 2, pad 1 -> 2x2 outputs.  All values negative, so a
    # padding value of 0 taken into the maximum would show up.  Windows (rows x cols of the image):
    #   (0,0): rows 0..1, cols 0..1   (0,1): rows 0..1, cols 1..3
    #   (1,0): rows 1..3, cols 0..1   (1,1): rows 1..3, cols 1..3
    x = np.array([[-9., -2., -7., -8.],
                  [-3., -6., -5., -4.],
                  [-8., -9., -9., -7.],
                  [-1., -5., -6., -9.]]).reshape(1, 4, 4, 1)
    y = oracle.maxpool2d(x, R=3, stride=2, pad=1)
    assert y.shape == (1, 2, 2, 1)
    assert y[0, :, :, 0].tolist() == [[-2., -2.], [-1., -4.]]


def test_window_of_one_pixel_and_no_padding():
    x = np.arange(2 * 5 * 5 * 3, dtype=np.float64).reshape(2, 5, 5, 3) * (-1.0) ** np.arange(3)
    assert np.array_equal(oracle.maxpool2d(x, R=1, stride=1, pad=0), x)          # identity
    y = oracle.maxpool2d(x, R=2, stride=2, pad=0)                                 # plain 2x2 blocks
    want = x[:, :4, :4].reshape(2, 2, 2, 2, 2, 3).max(axis=(2, 4))
    assert np.array_equal(y, want)


def test_against_library_max_pool_fp64():
    rng = np.random.default_rng(11)
    for (N, H, W, C, R, stride, pad) in [(2, 9, 7, 5, 3, 2, 1), (1, 12, 12, 8, 3, 2, 1), (3, 6, 11, 2, 3, 1, 1),
                                         (1, 8, 8, 4, 2, 2, 0), (2, 7, 7, 3, 5, 2, 2)]:
        x = rng.standard_normal((N, H, W, C)) - 3.0        # mostly negative
        y = oracle.maxpool2d(x, R=R, stride=stride, pad=pad)
        t = torch.nn.functional.max_pool2d(torch.from_numpy(x).permute(0, 3, 1, 2), R, stride, pad)
        assert np.array_equal(y, t.permute(0, 2, 3, 1).numpy())
