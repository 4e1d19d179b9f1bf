"""Pins of the thinning oracle (paper, Implementation, "Network Thinning"; Evaluation,
Objective 1) against facts that do not depend on it: removing zero structures
leaves the network's function unchanged (checked with torch's CPU convolution),
removal followed by re-insertion of zeros restores the tensor, and hand cases."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle


def _zero_some(rng, w, frac):
    """Zero a random subset of leading-index slices (what structure pruning leaves)."""
    dead = rng.random(w.shape[0]) < frac
    w = w.copy()
    w[dead] = 0.0
    return w, dead


def test_flags_hand_case_and_signed_zero():
    x = np.zeros((3, 2, 2), dtype=np.float32)
    x[0, 1, 0] = 5.0
    x[2, 0, 1] = -0.0                       # a negative zero is still a zero
    assert oracle.thin_flags(x, 0).tolist() == [1, 0, 0]
    assert oracle.thin_flags(x, 1).tolist() == [0, 1]
    x[1, 0, 0] = np.float32(1e-45)          # a subnormal is not
    assert oracle.thin_flags(x, 0).tolist() == [1, 1, 0]
    assert oracle.thin_flags(x, 1).tolist() == [1, 1]
    x[2, 1, 1] = np.nan
    assert oracle.thin_flags(x, 0).tolist() == [1, 1, 1]


def test_compact_hand_case():
    x = np.arange(2 * 3 * 2, dtype=np.float32).reshape(2, 3, 2)
    out = oracle.thin_compact(x, np.array([0, 1], np.uint8), np.array([1, 0, 1], np.uint8))
    assert out.shape == (1, 2, 2)
    assert out.reshape(-1).tolist() == [6.0, 7.0, 10.0, 11.0]
    assert oracle.thin_compact(x, None, None).tolist() == x.tolist()
    assert oracle.thin_compact(x, np.zeros(2, np.uint8), None).shape == (0, 3, 2)


def test_reinsertion_restores_the_tensor():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((13, 7, 9)).astype(np.float32)
    x[rng.random(13) < 0.4] = 0.0
    x[:, rng.random(7) < 0.4] = 0.0
    k0, k1 = oracle.thin_flags(x, 0), oracle.thin_flags(x, 1)
    out = oracle.thin_compact(x, k0, k1)
    assert out.shape == (int(k0.sum()), int(k1.sum()), 9)
    back = np.zeros_like(x)
    back[np.ix_(np.flatnonzero(k0), np.flatnonzero(k1))] = out
    assert np.array_equal(back, x)
    # every removed value was a zero, so the count of non-zeros is unchanged
    assert oracle.count_nonzero([x])[-1] == oracle.count_nonzero([out])[-1]


def test_thinned_network_computes_the_same_function():
    """conv -> relu -> conv -> relu -> flatten -> fc without biases: dropping the
    zero filters of a layer and the matching input channels of the next one
    (the thinning strategy for a chain) leaves the output unchanged."""
    rng = np.random.default_rng(11)
    w1, dead1 = _zero_some(rng, rng.standard_normal((12, 3, 3, 3)).astype(np.float32), 0.4)
    w2, dead2 = _zero_some(rng, rng.standard_normal((10, 12, 3, 3)).astype(np.float32), 0.4)
    hw = 6 * 6
    w3 = rng.standard_normal((5, 10 * hw)).astype(np.float32)
    x = torch.from_numpy(rng.standard_normal((2, 3, 6, 6)).astype(np.float32)).double()

    def net(a, b, c):
        h = F.relu(F.conv2d(x, torch.from_numpy(a).double(), padding=1))
        h = F.relu(F.conv2d(h, torch.from_numpy(b).double(), padding=1))
        return h.flatten(1) @ torch.from_numpy(c).double().t()

    k1 = oracle.thin_flags(w1.reshape(12, 3, 9), 0)
    k2 = oracle.thin_flags(w2.reshape(10, 12, 9), 0)
    assert np.array_equal(k1 == 0, dead1) and np.array_equal(k2 == 0, dead2)
    t1 = oracle.thin_compact(w1.reshape(12, 3, 9), k1, None).reshape(-1, 3, 3, 3)
    t2 = oracle.thin_compact(w2.reshape(10, 12, 9), k2, k1).reshape(-1, t1.shape[0], 3, 3)
    # the fc layer sees channel c at columns [c*hw, (c+1)*hw): view [5][10][hw], drop along axis 1
    t3 = oracle.thin_compact(w3.reshape(5, 10, hw), None, k2).reshape(5, -1)
    assert t1.shape[0] == int(k1.sum()) < 12 and t2.shape[0] == int(k2.sum()) < 10
    y_full, y_thin = net(w1, w2, w3), net(t1, t2, t3)
    assert torch.allclose(y_full, y_thin, rtol=1e-12, atol=1e-12)


def test_count_nonzero_and_footprint():
    a = np.array([0.0, -0.0, 1.0, np.float32(1e-45), -2.0], dtype=np.float32)
    b = np.zeros(7, dtype=np.float32)
    c = np.ones((2, 3), dtype=np.float32)
    assert oracle.count_nonzero([a, b, c]).tolist() == [3, 0, 6, 9]
    assert oracle.footprint_bytes([a, b, c], 2) == 18
    # magnitude pruning at sparsity s keeps n - round(s n) values: the footprint follows
    rng = np.random.default_rng(5)
    w = rng.standard_normal(1000).astype(np.float32)
    out = oracle.cstep_prune([w], [None], 0.9, 1e-3)
    assert oracle.footprint_bytes(out.theta, 4) == 4 * 100


@pytest.mark.parametrize("axis", [0, 1])
def test_flags_agree_with_elementwise_scan(axis):
    rng = np.random.default_rng(17 + axis)
    x = rng.standard_normal((9, 11, 4)).astype(np.float32)
    x[rng.random(x.shape) < 0.7] = 0.0
    x[2] = 0.0
    x[:, 5] = 0.0
    want = np.zeros(x.shape[axis], np.uint8)
    for i in range(9):
        for j in range(11):
            for r in range(4):
                if x[i, j, r] != 0:
                    want[(i, j)[axis]] = 1
    assert np.array_equal(oracle.thin_flags(x, axis), want)
