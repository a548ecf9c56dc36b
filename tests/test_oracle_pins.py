"""Pins for the CPU oracle: the convolution it computes is checked against things other than itself --
a library convolution in float64, a brute-force textbook loop, and closed forms.  CPU only."""
import itertools

import numpy as np
import pytest
import torch

import oracle
from paper_2001_00138_b200 import synth


def _random_pruned(F, C, seed, n_patterns=8, prune=0.3):
    rng = np.random.Generator(np.random.PCG64(seed))
    pats = synth.pattern_set(n_patterns)
    w = rng.standard_normal((F, C, 3, 3)).astype(np.float32)
    pid = rng.integers(0, n_patterns, size=(F, C)).astype(np.int32)
    pid[rng.random((F, C)) < prune] = -1
    return w, synth.mask_from_pid(pid, pats), pid, pats


def _textbook(x, wm, bias, relu):
    """out = act(b + sum_{c,r,s} w[f,c,r,s] * xpad[n,c,y+r,x+s]) with explicit zero padding, pure Python."""
    N, C, H, W = x.shape
    F = wm.shape[0]
    xp = np.zeros((N, C, H + 2, W + 2), dtype=np.float64)
    xp[:, :, 1:-1, 1:-1] = x
    out = np.zeros((N, F, H, W), dtype=np.float64)
    for n, f, y, xx in itertools.product(range(N), range(F), range(H), range(W)):
        acc = 0.0 if bias is None else float(bias[f])
        for c, r, s in itertools.product(range(C), range(3), range(3)):
            acc += float(wm[f, c, r, s]) * xp[n, c, y + r, xx + s]
        out[n, f, y, xx] = max(acc, 0.0) if relu else acc
    return out


@pytest.mark.parametrize("shape", [(2, 3, 4, 5, 5), (2, 3, 4, 7, 6), (1, 5, 2, 1, 1), (1, 2, 3, 2, 9)])
@pytest.mark.parametrize("relu", [False, True])
def test_matches_library_conv2d_float64(shape, relu):
    N, C, F, H, W = shape
    w, mask, _, _ = _random_pruned(F, C, seed=11 + H * W)
    rng = np.random.Generator(np.random.PCG64(5))
    x = rng.standard_normal((N, C, H, W)).astype(np.float32)
    bias = rng.standard_normal(F).astype(np.float32)
    got = oracle.conv3x3(x, w, mask, bias, relu)
    ref = torch.nn.functional.conv2d(torch.from_numpy(x).double(), torch.from_numpy(w * mask).double(),
                                     torch.from_numpy(bias).double(), stride=1, padding=1)
    if relu:
        ref = torch.relu(ref)
    np.testing.assert_allclose(got, ref.numpy().astype(np.float32), rtol=1e-6, atol=1e-6)


@pytest.mark.parametrize("relu", [False, True])
def test_matches_textbook_loops(relu):
    N, C, F, H, W = 2, 3, 4, 5, 4
    w, mask, _, _ = _random_pruned(F, C, seed=3)
    rng = np.random.Generator(np.random.PCG64(8))
    x = rng.standard_normal((N, C, H, W)).astype(np.float32)
    bias = rng.standard_normal(F).astype(np.float32)
    got = oracle.conv3x3(x, w, mask, bias, relu)
    ref = _textbook(x, (w * mask), bias, relu)
    np.testing.assert_allclose(got, ref.astype(np.float32), rtol=1e-6, atol=1e-6)
    got_nobias = oracle.conv3x3(x, w, mask, None, relu)
    np.testing.assert_allclose(got_nobias, _textbook(x, w * mask, None, relu).astype(np.float32), rtol=1e-6, atol=1e-6)


def test_values_outside_the_mask_are_ignored():
    w, mask, _, _ = _random_pruned(3, 4, seed=21)
    x = np.random.Generator(np.random.PCG64(2)).standard_normal((1, 4, 6, 5)).astype(np.float32)
    a = oracle.conv3x3(x, w, mask, None, False)
    w2 = np.where(mask == 1, w, np.float32(123.0))
    b = oracle.conv3x3(x, w2, mask, None, False)
    assert np.array_equal(a, b)


@pytest.mark.parametrize("tap", range(9))
def test_single_tap_is_a_shift(tap):
    """A kernel with weight 1 at tap (r,s) copies the input shifted by (r-1, s-1): cross-correlation, no flip."""
    H, W = 5, 7
    x = np.arange(H * W, dtype=np.float32).reshape(1, 1, H, W) + 1
    w = np.zeros((1, 1, 3, 3), dtype=np.float32)
    mask = np.zeros((1, 1, 3, 3), dtype=np.uint8)
    r, s = divmod(tap, 3)
    w[0, 0, r, s] = 1.0
    mask[0, 0, r, s] = 1
    got = oracle.conv3x3(x, w, mask, None, False)[0, 0]
    exp = np.zeros((H, W), dtype=np.float32)
    for y in range(H):
        for xx in range(W):
            yy, xs = y + r - 1, xx + s - 1
            if 0 <= yy < H and 0 <= xs < W:
                exp[y, xx] = x[0, 0, yy, xs]
    assert np.array_equal(got, exp)


def test_all_ones_counts_in_bounds_taps():
    """All-ones input and all-ones kept weights: the output counts the kept taps that fall inside the image."""
    F, C, H, W = 3, 5, 6, 4
    _, mask, pid, pats = _random_pruned(F, C, seed=33, prune=0.4)
    w = np.ones((F, C, 3, 3), dtype=np.float32)
    x = np.ones((1, C, H, W), dtype=np.float32)
    got = oracle.conv3x3(x, w, mask, None, False)
    for f in range(F):
        kept = [int(pats[p]) for p in pid[f] if p >= 0]
        assert got[0, f, 2, 2] == 4 * len(kept)                      # interior pixel: every tap lands inside
        corner = sum(1 for m in kept for t in synth.mask_to_taps(m) if t // 3 >= 1 and t % 3 >= 1)
        assert got[0, f, 0, 0] == corner                             # top-left pixel: rows/cols -1 are padding
        bottom = sum(1 for m in kept for t in synth.mask_to_taps(m) if t // 3 <= 1)
        assert got[0, f, H - 1, 1] == bottom


def test_bias_relu_and_double_accumulation():
    # three channels, centre weight 1 each: 1e8 + 1 - 1e8 is exactly 1 in double, 0 in a float running sum
    x = np.zeros((1, 3, 3, 3), dtype=np.float32)
    x[0, :, 1, 1] = [1e8, 1.0, -1e8]
    w = np.zeros((2, 3, 3, 3), dtype=np.float32)
    mask = np.zeros_like(w, dtype=np.uint8)
    w[:, :, 1, 1] = 1.0
    mask[:, :, 1, 1] = 1
    bias = np.asarray([0.5, -2.0], dtype=np.float32)
    out = oracle.conv3x3(x, w, mask, bias, False)
    assert out[0, 0, 1, 1] == 1.5 and out[0, 1, 1, 1] == -1.0
    out = oracle.conv3x3(x, w, mask, bias, True)
    assert out[0, 0, 1, 1] == 1.5 and out[0, 1, 1, 1] == 0.0
    assert out[0, 1, 0, 0] == 0.0 and out[0, 0, 0, 0] == 0.5          # relu(bias) where no input reaches


def test_empty_filter_outputs_activated_bias():
    w, mask, _, _ = _random_pruned(3, 4, seed=5)
    mask[1] = 0
    x = np.random.Generator(np.random.PCG64(1)).standard_normal((2, 4, 4, 4)).astype(np.float32)
    bias = np.asarray([0.1, 0.7, -0.3], dtype=np.float32)
    out = oracle.conv3x3(x, w, mask, bias, True)
    assert np.all(out[:, 1] == np.float32(0.7))


def test_point_function_agrees_with_full_tensor():
    w, mask, _, _ = _random_pruned(4, 6, seed=9)
    rng = np.random.Generator(np.random.PCG64(4))
    x = rng.standard_normal((2, 6, 7, 5)).astype(np.float32)
    bias = rng.standard_normal(4).astype(np.float32)
    full = oracle.conv3x3(x, w, mask, bias, True)
    for n, f, y, xx in [(0, 0, 0, 0), (1, 3, 6, 4), (1, 2, 3, 0), (0, 1, 0, 4)]:
        assert np.float32(oracle.conv3x3_point(x, w, mask, bias, True, n, f, y, xx)) == full[n, f, y, xx]


@pytest.mark.parametrize("hw", [(6, 8), (7, 9), (5, 3), (13, 9), (2, 2), (3, 2), (14, 15)])
def test_maxpool_matches_library(hw):
    """2x2 / stride-2 maximum with floor extents: an odd last row or column is dropped, as the library pool does."""
    H, W = hw
    x = np.random.Generator(np.random.PCG64(6 + H * W)).standard_normal((2, 3, H, W)).astype(np.float32)
    ref = torch.nn.functional.max_pool2d(torch.from_numpy(x), 2).numpy()
    got = oracle.maxpool2x2(x)
    assert got.shape == (2, 3, H // 2, W // 2)
    assert np.array_equal(got, ref)


def test_maxpool_closed_form_on_a_ramp():
    """On a ramp that grows along rows and columns every window's maximum is its bottom-right element."""
    H, W = 7, 5
    x = (np.arange(H)[:, None] * 100 + np.arange(W)[None, :]).astype(np.float32).reshape(1, 1, H, W)
    got = oracle.maxpool2x2(x)[0, 0]
    exp = x[0, 0, 1:2 * (H // 2):2, 1:2 * (W // 2):2]
    assert np.array_equal(got, exp)


def test_threads_do_not_change_the_result():
    L = synth.config1()
    oracle.set_num_threads(1)
    a = oracle.conv3x3(L.x, L.weights, L.mask, L.bias, True)
    oracle.set_num_threads(max(2, oracle.num_threads()))
    b = oracle.conv3x3(L.x, L.weights, L.mask, L.bias, True)
    assert np.array_equal(a, b)
