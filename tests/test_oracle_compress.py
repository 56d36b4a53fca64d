"""Pins for the oracle's parameter-free visual compression (no GPU needed)."""

import numpy as np
import torch

import oracle


def test_pool_against_torch_avg_pool_and_tail_window():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((2, 576, 12))
    for ratio in (2, 3, 4, 20):
        got = oracle.visual_pool(x, ratio)
        full = 576 // ratio
        ref = torch.nn.functional.avg_pool1d(torch.from_numpy(x).transpose(1, 2), ratio, ratio).transpose(1, 2).numpy()
        assert got.shape == (2, -(-576 // ratio), 12)
        assert np.abs(got[:, :full] - ref).max() < 1e-12            # library routine on the full windows
        if 576 % ratio:
            assert np.abs(got[:, -1] - x[:, full * ratio:].mean(axis=1)).max() < 1e-15
    # closed form: pooling a ramp by r gives the window mid-points; ratio 1 is the identity
    ramp = np.arange(12.0).reshape(1, 12, 1)
    assert oracle.visual_pool(ramp, 4)[0, :, 0].tolist() == [1.5, 5.5, 9.5]
    assert oracle.visual_pool(ramp, 5)[0, :, 0].tolist() == [2.0, 7.0, 10.5]
    assert np.array_equal(oracle.visual_pool(x, 1), x)


def test_prune_is_row_selection():
    x = np.arange(2 * 6 * 3).reshape(2, 6, 3)
    got = oracle.visual_prune(x, np.array([[0, 2, 5], [4, 1, 1]]))
    assert got[0].tolist() == [x[0, 0].tolist(), x[0, 2].tolist(), x[0, 5].tolist()]
    assert got[1].tolist() == [x[1, 4].tolist(), x[1, 1].tolist(), x[1, 1].tolist()]
