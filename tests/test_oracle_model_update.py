"""Pins for the oracle's model update (Eq. 1 / Algorithm 1, momentum of Sec. 6.1): exact small cases,
closed forms of the recursion, and the optimiser of the framework the paper trained with."""
import numpy as np
import torch

import oracle


def test_plain_step_on_exact_values():
    # Eq. (1) with dyadic numbers: every product and difference is exact in single precision
    w = np.array([1.0, -2.0, 0.5, 8.0], np.float32)
    g = np.array([4.0, -1.0, 0.0, 0.25], np.float32)
    got, v = oracle.model_update(w, g, 0.5)
    assert v is None
    assert got.tolist() == [-1.0, -1.5, 0.5, 7.875]
    # the inputs are not modified
    assert w.tolist() == [1.0, -2.0, 0.5, 8.0]


def test_zero_rate_and_zero_momentum():
    rng = np.random.default_rng(0)
    w, g, v = (rng.standard_normal(1000).astype(np.float32) for _ in range(3))
    w1, v1 = oracle.model_update(w, g, 0.0, v, 0.9)
    assert np.array_equal(w1, w)                      # eta = 0: parameters stay
    assert np.allclose(v1, 0.9 * v + g, rtol=1e-6, atol=1e-7)
    w2, v2 = oracle.model_update(w, g, 0.1, v, 0.0)
    assert np.array_equal(v2, g)                      # mu = 0: the velocity is the gradient
    w3, _ = oracle.model_update(w, g, 0.1)
    assert np.array_equal(w2, w3)                     # and the step is the plain one


def test_quadratic_contracts_geometrically():
    # f(w) = |w|^2 / 2 has gradient w: the plain step gives w_t = (1 - eta)^t w_0
    w0 = np.linspace(-3, 3, 13).astype(np.float32)
    w = w0.copy()
    for _ in range(20):
        w, _ = oracle.model_update(w, w, 0.25)
    assert np.allclose(w, 0.75 ** 20 * w0.astype(np.float64), rtol=1e-5, atol=0)


def test_constant_gradient_closed_form():
    # v_t = g (1 - mu^t) / (1 - mu),  w_t = w_0 - eta g sum_{s<=t} (1 - mu^s) / (1 - mu)
    g = np.array([1.0, -0.5, 3.0], np.float32)
    w = np.zeros(3, np.float32)
    v = np.zeros(3, np.float32)
    eta, mu, T = 0.01, 0.9, 30
    for _ in range(T):
        w, v = oracle.model_update(w, g, eta, v, mu)
    mu64, eta64 = float(np.float32(mu)), float(np.float32(eta))
    vt = g.astype(np.float64) * (1 - mu64 ** T) / (1 - mu64)
    wt = -eta64 * g.astype(np.float64) * sum((1 - mu64 ** s) / (1 - mu64) for s in range(1, T + 1))
    assert np.allclose(v, vt, rtol=1e-5)
    assert np.allclose(w, wt, rtol=1e-5)


def test_against_library_optimiser():
    # torch.optim.SGD with momentum, no dampening, no Nesterov, no weight decay
    rng = np.random.default_rng(1)
    d = 4096
    w0 = rng.standard_normal(d).astype(np.float32)
    p = torch.nn.Parameter(torch.from_numpy(w0.copy()))
    opt = torch.optim.SGD([p], lr=0.05, momentum=0.9)
    w, v = w0.copy(), np.zeros(d, np.float32)
    for step in range(6):
        g = rng.standard_normal(d).astype(np.float32)
        p.grad = torch.from_numpy(g.copy())
        opt.step()
        w, v = oracle.model_update(w, g, 0.05, v, 0.9)
        assert np.allclose(w, p.detach().numpy(), rtol=2e-6, atol=2e-6), step
    buf = opt.state[p]["momentum_buffer"].numpy()
    assert np.allclose(v, buf, rtol=2e-6, atol=2e-6)
    # a Nesterov or dampened variant is a different sequence: the pin would see it
    q = torch.nn.Parameter(torch.from_numpy(w0.copy()))
    opt2 = torch.optim.SGD([q], lr=0.05, momentum=0.9, nesterov=True)
    rng = np.random.default_rng(1)
    rng.standard_normal(d)
    for step in range(2):
        q.grad = torch.from_numpy(rng.standard_normal(d).astype(np.float32))
        opt2.step()
    w2, v2 = w0.copy(), np.zeros(d, np.float32)
    rng = np.random.default_rng(1)
    rng.standard_normal(d)
    for step in range(2):
        w2, v2 = oracle.model_update(w2, rng.standard_normal(d).astype(np.float32), 0.05, v2, 0.9)
    assert not np.allclose(w2, q.detach().numpy(), rtol=1e-4, atol=1e-4)
