"""Pins for the oracle's first-order local steps (plain SGD, Eqs. 2-3; momentum in
velocity form) used by the EASGD / EAMSGD comparison methods of Sec. VI."""
import numpy as np
import torch

from oracle import OracleState


def _state(K, P, seed, scale=1.0):
    rng = np.random.default_rng(seed)
    st = OracleState((rng.standard_normal(P) * scale).astype(np.float32), K, [(0, P, 1)])
    return st, rng


def test_sgd_constant_gradient_closed_form_exact(orc):
    # dyadic values keep every operation exact: x_T = x_0 - T eta g (Eq. 3 iterated)
    K, P, T = 2, 16, 8
    st = OracleState(np.full(P, 4.0, np.float32), K, [(0, P, 1)])
    g = np.zeros((K, P), np.float32)
    g[0], g[1] = 2.0, -0.5
    for _ in range(T):
        st.sgd_step(g, lr=0.25)
    assert np.all(st.x[0] == 4.0 - T * 0.25 * 2.0) and np.all(st.x[1] == 4.0 + T * 0.25 * 0.5)
    assert np.all(st.m == 0.0)                               # plain SGD keeps no velocity
    assert st.step.tolist() == [T, T]


def test_sgd_on_quadratic_is_geometric(orc):
    # f = h x^2 / 2, g = h x: x_T = (1 - eta h)^T x_0
    P, T, eta = 64, 30, 0.05
    st, rng = _state(1, P, 31)
    h = rng.uniform(0.1, 10, P)
    x0 = st.x[0].astype(np.float64)
    for _ in range(T):
        g = (h * st.x[0].astype(np.float64)).astype(np.float32)[None]
        st.sgd_step(np.ascontiguousarray(g), lr=eta)
    assert np.allclose(st.x[0], (1 - eta * h) ** T * x0, rtol=2e-5, atol=1e-7)


def test_momentum_constant_gradient_closed_form(orc):
    # u_t = -eta g (1 - delta^t) / (1 - delta);  x_T = x_0 + sum_t u_t
    K, P, T, eta, delta = 1, 8, 12, 0.125, 0.5
    st = OracleState(np.zeros(P, np.float32), K, [(0, P, 1)])
    g = np.full((K, P), 3.0, np.float32)
    for _ in range(T):
        st.sgd_step(g, lr=eta, momentum=delta)
    u = [-eta * 3.0 * (1 - delta ** t) / (1 - delta) for t in range(1, T + 1)]
    assert np.allclose(st.m[0], u[-1], rtol=1e-6)
    assert np.allclose(st.x[0], sum(u), rtol=1e-6)
    # first step by hand: u = 0.5 * 0 - 0.125 * 3 = -0.375, x = -0.375 (exact)
    st2 = OracleState(np.zeros(P, np.float32), K, [(0, P, 1)])
    st2.sgd_step(g, lr=eta, momentum=delta)
    assert np.all(st2.m[0] == -0.375) and np.all(st2.x[0] == -0.375)


def test_sgd_and_momentum_match_library_optimizer(orc):
    # torch.optim.SGD (CPU, double): buf = delta buf + g, x -= eta buf  ==  velocity form
    # with u = -eta buf for a constant learning rate
    K, P, T, eta = 3, 200, 25, 0.01
    for delta in (0.0, 0.5, 0.9):
        st, rng = _state(K, P, 32)
        xt = torch.tensor(st.x.astype(np.float64), requires_grad=True)
        opt = torch.optim.SGD([xt], lr=eta, momentum=delta)
        for _ in range(T):
            g = rng.standard_normal((K, P)).astype(np.float32)
            st.sgd_step(g, lr=eta, momentum=delta)
            xt.grad = torch.tensor(g.astype(np.float64))
            opt.step()
        assert np.allclose(st.x, xt.detach().numpy(), rtol=1e-5, atol=2e-6), delta


def test_sgd_inactive_worker_and_row_stride(orc):
    K, P, ld = 3, 10, 16
    st, rng = _state(K, P, 33)
    x0, m0 = st.x.copy(), st.m.copy()
    g = np.full((K, ld), np.nan, np.float32)                  # padding columns are never read
    g[:, :P] = rng.standard_normal((K, P)).astype(np.float32)
    st.sgd_step(g, lr=0.1, momentum=0.5, active=np.array([1, 0, 1], np.uint8))
    assert np.array_equal(st.x[1], x0[1]) and np.array_equal(st.m[1], m0[1])
    assert st.step.tolist() == [1, 0, 1]
    assert np.allclose(st.x[0], x0[0] - 0.1 * g[0, :P], rtol=1e-6, atol=1e-7)
    assert np.all(np.isfinite(st.x))
