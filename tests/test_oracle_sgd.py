"""Pins of the oracle's parameter update (Algorithm 1, UpdateParameters: SGD with momentum and L2
weight decay on the fp32 master weights).  CPU only."""
import numpy as np
import pytest
import torch

import oracle
from paper_1605_04711_b200 import datagen as dg


def test_hand_worked_step():
    # g = 0.5 + 0.1*2 = 0.7;  v' = 0.9*1 + 0.7 = 1.6;  w' = 2 - 0.25*1.6 = 1.6
    w, v = oracle.sgd_update(np.array([2.0], np.float32), np.array([0.5], np.float32), np.array([1.0], np.float32),
                             0.25, 0.9, 0.1)
    assert w[0] == pytest.approx(1.6, rel=1e-6) and v[0] == pytest.approx(1.6, rel=1e-6)
    # no momentum, no decay: plain gradient descent, exact in binary
    w, v = oracle.sgd_update(np.array([1.0, -3.0], np.float32), np.array([0.5, -1.0], np.float32),
                             np.zeros(2, np.float32), 0.5, 0.0, 0.0)
    assert w.tolist() == [0.75, -2.5] and v.tolist() == [0.5, -1.0]


def test_matches_torch_sgd_over_several_steps():
    # an independent implementation of the same rule (dampening 0, no Nesterov); torch may fuse a
    # multiply and an add, so the comparison allows a few units in the last place
    n = 4096
    W0 = dg.he_normal(51, "sgd-w", 1, n).reshape(-1)
    p = torch.nn.Parameter(torch.from_numpy(W0.copy()))
    opt = torch.optim.SGD([p], lr=0.1, momentum=0.9, weight_decay=1e-4)
    W, V = W0.copy(), np.zeros(n, np.float32)
    for step in range(5):
        g = dg.draw(51, f"sgd-g{step}", n, "normal", 0.0, 0.05)
        p.grad = torch.from_numpy(g.copy())
        opt.step()
        W, V = oracle.sgd_update(W, g, V, 0.1, 0.9, 1e-4)
        assert np.allclose(W, p.detach().numpy(), rtol=0, atol=4 * np.finfo(np.float32).eps * np.abs(W).max())
    buf = opt.state[p]["momentum_buffer"].numpy()
    assert np.allclose(V, buf, rtol=1e-5, atol=1e-7)


def test_fp32_result_is_the_rounded_exact_result_up_to_the_rounding_of_its_steps():
    n = 10000
    W = dg.he_normal(52, "sgd-w2", 1, n).reshape(-1)
    g = dg.draw(52, "sgd-g2", n, "normal", 0.0, 0.05)
    V = dg.draw(52, "sgd-v2", n, "normal", 0.0, 0.05)
    w32, v32 = oracle.sgd_update(W, g, V, 0.1, 0.9, 1e-4)
    lr, mu, wd = (float(np.float32(x)) for x in (0.1, 0.9, 1e-4))
    v64 = mu * V.astype(np.float64) + (g.astype(np.float64) + wd * W.astype(np.float64))
    w64 = W.astype(np.float64) - lr * v64
    eps = np.finfo(np.float32).eps
    # four roundings on the way to V' (product, sum, product, sum), two more to W'
    verr = 4 * eps * (np.abs(V) + np.abs(g) + wd * np.abs(W) + 1e-30)
    assert np.all(np.abs(v32 - v64) <= verr)
    assert np.all(np.abs(w32 - w64) <= lr * verr + 2 * eps * (np.abs(W) + lr * np.abs(v64) + 1e-30))


def test_threshold_of_the_updated_weights_follows_the_update():
    # the next iteration's ternarization (Algorithm 1, first loop) sees the updated weights
    W = dg.he_normal(53, "sgd-w3", 64, 576)
    g = dg.draw(53, "sgd-g3", W.size, "normal", 0.0, 0.01).reshape(W.shape)
    w1, _ = oracle.sgd_update(W, g, np.zeros_like(W), 0.1, 0.9, 1e-4)
    st0, _ = oracle.ternarize(W, 0.7)
    st1, _ = oracle.ternarize(w1, 0.7)
    assert st1.delta == pytest.approx(0.7 * np.abs(w1.astype(np.float64)).mean(), rel=1e-13)
    assert st1.delta != st0.delta
