"""Pins for the oracle's convolution and linear layers (Appendix F.1/F.2 geometry)."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import hts_oracle as orc


def test_output_extents_match_paper_geometry():
    # 8x8/4, 4x4/2, 3x3/1 on 84x84 and on 72x96, no padding, floor
    assert [orc.conv_out(84, 8, 4), orc.conv_out(20, 4, 2), orc.conv_out(9, 3, 1)] == [20, 9, 7]
    assert [orc.conv_out(72, 8, 4), orc.conv_out(17, 4, 2), orc.conv_out(7, 3, 1)] == [17, 7, 5]
    assert [orc.conv_out(96, 8, 4), orc.conv_out(23, 4, 2), orc.conv_out(10, 3, 1)] == [23, 10, 8]
    assert orc.lib().hts_oracle_flat_features(84, 84) == 3136
    assert orc.lib().hts_oracle_flat_features(72, 96) == 2560


def test_all_ones_kernel_gives_window_sums():
    x = np.arange(64, dtype=np.float64).reshape(1, 8, 8)
    w = np.ones((1, 1, 4, 4))
    y = orc.conv2d(x, w, np.zeros(1), stride=2, relu=False)
    assert y.shape == (1, 3, 3)
    for i in range(3):
        for j in range(3):
            assert y[0, i, j] == x[0, 2 * i:2 * i + 4, 2 * j:2 * j + 4].sum()


def test_hand_computed_tiny_case():
    # 1 channel 3x3 input, 2x2 kernel, stride 1: four outputs written out by hand
    x = np.array([[[1., 2., 3.], [4., 5., 6.], [7., 8., 9.]]])
    w = np.array([[[[1., -1.], [2., 0.5]]]])
    y = orc.conv2d(x, w, np.array([0.25]), 1, False)
    exp = np.array([[1 - 2 + 8 + 2.5, 2 - 3 + 10 + 3], [4 - 5 + 14 + 4, 5 - 6 + 16 + 4.5]]) + 0.25
    assert np.array_equal(y[0], exp)


def test_one_by_one_kernel_is_a_matrix_product():
    g = np.random.default_rng(1)
    x = g.standard_normal((5, 6, 7))
    w = g.standard_normal((3, 5, 1, 1))
    b = g.standard_normal(3)
    y = orc.conv2d(x, w, b, 1, False)
    exp = (w[:, :, 0, 0] @ x.reshape(5, -1)).reshape(3, 6, 7) + b[:, None, None]
    np.testing.assert_allclose(y, exp, rtol=1e-13, atol=1e-13)


def test_impulse_returns_unflipped_kernel():
    g = np.random.default_rng(2)
    C, H, W, O, k, s = 3, 11, 13, 2, 4, 1
    w = g.standard_normal((O, C, k, k))
    x = np.zeros((C, H, W))
    c0, i0, j0 = 1, 6, 7
    x[c0, i0, j0] = 1.0
    y = orc.conv2d(x, w, np.zeros(O), s, False)
    for o in range(O):
        for i in range(y.shape[1]):
            for j in range(y.shape[2]):
                u, v = i0 - i, j0 - j
                exp = w[o, c0, u, v] if 0 <= u < k and 0 <= v < k else 0.0
                assert y[o, i, j] == exp


@pytest.mark.parametrize("C,H,W,O,k,s", [(4, 20, 28, 5, 8, 4), (3, 9, 11, 6, 4, 2), (2, 7, 9, 3, 3, 1)])
def test_matches_library_cross_correlation(C, H, W, O, k, s):
    g = np.random.default_rng(3)
    x, w, b = g.standard_normal((C, H, W)), g.standard_normal((O, C, k, k)), g.standard_normal(O)
    y = orc.conv2d(x, w, b, s, True)
    ref = F.relu(F.conv2d(torch.from_numpy(x)[None], torch.from_numpy(w), torch.from_numpy(b), stride=s))[0]
    np.testing.assert_allclose(y, ref.numpy(), rtol=1e-12, atol=1e-12)
    assert (y >= 0).all() and (y == 0).any()


@pytest.mark.parametrize("k,s", [(8, 4), (4, 2)])
def test_space_to_depth_identity(k, s):
    # a k x k / s convolution with k = 2s equals a 2x2/1 convolution on the
    # space-to-depth(s) rearrangement of input and kernel
    g = np.random.default_rng(4)
    C, H, W, O = 3, 6 * s, 7 * s, 4
    x, w, b = g.standard_normal((C, H, W)), g.standard_normal((O, C, k, k)), g.standard_normal(O)
    y = orc.conv2d(x, w, b, s, False)
    xs = x.reshape(C, H // s, s, W // s, s).transpose(0, 2, 4, 1, 3).reshape(C * s * s, H // s, W // s)
    ws = w.reshape(O, C, 2, s, 2, s).transpose(0, 1, 3, 5, 2, 4).reshape(O, C * s * s, 2, 2)
    y2 = orc.conv2d(xs, ws, b, 1, False)
    np.testing.assert_allclose(y, y2, rtol=1e-12, atol=1e-12)


def test_linear_matches_matrix_product_and_relu():
    g = np.random.default_rng(5)
    x, w, b = g.standard_normal(37), g.standard_normal((11, 37)), g.standard_normal(11)
    np.testing.assert_allclose(orc.linear(x, w, b, False), w @ x + b, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(orc.linear(x, w, b, True), np.maximum(w @ x + b, 0), rtol=1e-13, atol=1e-13)
