"""The sampled references of tests/netcheck.py (used only where the oracle needs minutes for a whole tensor: the
ResNet-50-shaped net at batch 1024) are pinned here to the oracle functions they stand for, element by element, on
stride-1 and stride-2 problems with 3x3 and 1x1 filters."""
import numpy as np
import pytest

import oracle
from netcheck import _conv_samples, _dgrad_samples, _wgrad_samples

CASES = [  # N, H, W, C, K, R, stride
    (2, 8, 8, 5, 7, 3, 1),
    (3, 8, 6, 4, 6, 3, 2),
    (2, 4, 4, 6, 5, 1, 1),
    (2, 8, 8, 3, 4, 1, 2),
]


@pytest.mark.parametrize("case", CASES)
def test_sampled_references_equal_the_oracle(case):
    N, H, W, C, K, R, stride = case
    pad = (R - 1) // 2
    rng = np.random.default_rng(sum(case))
    x = rng.standard_normal((N, H, W, C))
    w = rng.standard_normal((K, R, R, C))
    y = oracle.conv2d_fwd(x, w, stride, pad)
    dy = rng.standard_normal(y.shape)
    # enough draws to hit every border row/column and every tap of these small problems
    idx, got = _conv_samples(np.random.default_rng(1), x, w, y.shape, stride, pad, 400)
    np.testing.assert_allclose(got, y[tuple(idx.T)], rtol=1e-12, atol=1e-12)
    dx = oracle.conv2d_dgrad(dy, w, x.shape, stride, pad)
    idx, got = _dgrad_samples(np.random.default_rng(2), dy, w, x.shape, stride, pad, 400)
    np.testing.assert_allclose(got, dx[tuple(idx.T)], rtol=1e-12, atol=1e-12)
    dw = oracle.conv2d_wgrad(dy, x, R, R, stride, pad)
    idx, got = _wgrad_samples(np.random.default_rng(3), dy, x, R, stride, pad, 200)
    np.testing.assert_allclose(got, dw[tuple(idx.T)], rtol=1e-12, atol=1e-12)
    # the draws covered the corners: first and last output row/column, every filter tap
    assert {0, y.shape[1] - 1} <= set(_conv_samples(np.random.default_rng(1), x, w, y.shape, stride, pad, 400)[0][:, 1])
    assert len({(r, s) for _, r, s, _ in idx}) == R * R
