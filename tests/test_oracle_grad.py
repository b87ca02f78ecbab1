"""Pins for the oracle's analytic gradients: central finite differences of the
oracle's own fp64 forward, plus identities the chain rule fixes."""
import numpy as np
import pytest
import torch

from oracle import cp_head
from paper_2410_17765_b200 import synth


def problem(seed=2, N=4, d=5, V=7, n=2, r=3):
    inp = synth.make_inputs(synth.Shape(N, d, V, n, r), seed=seed, weight_scale=20.0)
    # finite differences need fp64 operands that can move by 1e-6
    return dict(h=inp.h.double().numpy().copy(), W_head=inp.W_head.double().numpy().copy(),
                E=inp.E.double().numpy().copy(), W_g=inp.W_g.double().numpy().copy(),
                x=inp.x.numpy().copy()), inp.shape


def objective(p, s, aux, up):
    fw = cp_head.forward(p["h"], p["W_head"], p["E"], p["W_g"], p["x"], s.n, s.r, aux_coef=aux)
    if up is None:
        return fw.loss
    return float(np.dot(up, fw.logp) + aux * np.sum(fw.wbar ** 2))


@pytest.mark.parametrize("aux,custom_up", [(0.0, False), (1.5, False), (0.7, True)])
def test_gradients_match_central_differences(aux, custom_up):
    p, s = problem()
    up = np.linspace(-0.5, 0.8, s.N) if custom_up else None
    g = cp_head.backward(p["h"], p["W_head"], p["E"], p["W_g"], p["x"], s.n, s.r,
                         aux_coef=aux, dloss_dlogp=up)
    eps = 1e-6
    rng = np.random.default_rng(0)
    for name, grad in [("h", g.dh), ("W_head", g.dW_head), ("E", g.dE), ("W_g", g.dW_g)]:
        arr = p[name]
        flat_idx = rng.choice(arr.size, size=min(arr.size, 25), replace=False)
        for fi in flat_idx:
            idx = np.unravel_index(fi, arr.shape)
            old = arr[idx]
            arr[idx] = old + eps
            fp = objective(p, s, aux, up)
            arr[idx] = old - eps
            fm = objective(p, s, aux, up)
            arr[idx] = old
            num = (fp - fm) / (2 * eps)
            assert abs(num - grad[idx]) <= 1e-6 * max(1.0, abs(num)) + 1e-8, (name, idx, num, grad[idx])


def test_gate_logit_gradient_sums_to_zero_and_aux_forms_agree():
    p, s = problem(seed=5, r=4)
    g = cp_head.backward(p["h"], p["W_head"], p["E"], p["W_g"], p["x"], s.n, s.r, aux_coef=2.0)
    assert np.allclose(g.dg.sum(axis=1), 0.0, atol=1e-15)
    assert np.allclose(g.c.sum(axis=1), -1.0 / s.N, atol=1e-15)
    # gradient of sum (wbar - 1/r)^2 w.r.t. W_g by finite differences equals that of sum wbar^2
    g0 = cp_head.backward(p["h"], p["W_head"], p["E"], p["W_g"], p["x"], s.n, s.r, aux_coef=0.0)
    aux_grad = (g.dW_g - g0.dW_g) / 2.0
    eps = 1e-6
    for idx in [(0, 0), (1, 3), (3, 2)]:
        vals = []
        for sign in (+1, -1):
            Wg = p["W_g"].copy()
            Wg[idx] += sign * eps
            w = np.exp(cp_head.gate_log_weights(p["h"], Wg)).mean(axis=0)
            vals.append(np.sum((w - 1.0 / s.r) ** 2))
        assert abs((vals[0] - vals[1]) / (2 * eps) - aux_grad[idx]) < 1e-8


def test_rank1_gradient_matches_torch_autograd_cross_entropy():
    inp = synth.make_inputs(synth.Shape(6, 8, 9, 3, 1), seed=8, weight_scale=20.0)
    s = inp.shape
    g = cp_head.backward(inp.h, inp.W_head, inp.E, inp.W_g, inp.x, s.n, s.r)
    h = inp.h.double().requires_grad_()
    Wh = inp.W_head.double().requires_grad_()
    E = inp.E.double().requires_grad_()
    loss = 0.0
    for t in range(s.n):
        logits = (h @ Wh[t].T) @ E.T
        loss = loss + torch.nn.functional.cross_entropy(logits, inp.x[:, t].long(), reduction="sum") / s.N
    loss.backward()
    assert np.allclose(g.dh, h.grad.numpy(), atol=1e-13)
    assert np.allclose(g.dW_head, Wh.grad.numpy(), atol=1e-13)
    assert np.allclose(g.dE, E.grad.numpy(), atol=1e-13)
    assert np.allclose(g.dW_g, 0.0, atol=1e-15)


def test_gradients_are_additive_over_position_chunks():
    p, s = problem(seed=6, N=6)
    up = np.full(s.N, -1.0 / s.N)
    full = cp_head.backward(p["h"], p["W_head"], p["E"], p["W_g"], p["x"], s.n, s.r)
    acc = np.zeros_like(full.dE)
    for lo, hi in [(0, 2), (2, 6)]:
        part = cp_head.backward(p["h"][lo:hi], p["W_head"], p["E"], p["W_g"], p["x"][lo:hi], s.n, s.r,
                                dloss_dlogp=up[lo:hi])
        acc += part.dE
        assert np.allclose(part.dh, full.dh[lo:hi], atol=1e-15)
    assert np.allclose(acc, full.dE, atol=1e-15)


def test_per_token_objective_gradients_match_finite_differences():
    # objective sum_i sum_s up[i, s] * log P(x_1..x_{s+1}) + aux: e.g. a discounted per-token cross-entropy
    p, s = problem(seed=11, N=3, n=3, r=2)
    rng = np.random.default_rng(3)
    ups = rng.normal(size=(s.N, s.n))
    aux = 0.8

    def f():
        fw = cp_head.forward(p["h"], p["W_head"], p["E"], p["W_g"], p["x"], s.n, s.r, aux_coef=aux)
        return float(np.sum(ups * cp_head.prefix_log_probs(fw)) + aux * np.sum(fw.wbar ** 2))

    g = cp_head.backward(p["h"], p["W_head"], p["E"], p["W_g"], p["x"], s.n, s.r, aux_coef=aux, dloss_dprefix=ups)
    for name, grad in [("h", g.dh), ("W_head", g.dW_head), ("E", g.dE), ("W_g", g.dW_g)]:
        arr = p[name]
        for fi in rng.choice(arr.size, size=min(arr.size, 20), replace=False):
            idx = np.unravel_index(fi, arr.shape)
            old = arr[idx]
            arr[idx] = old + 1e-6
            fp = f()
            arr[idx] = old - 1e-6
            fm = f()
            arr[idx] = old
            assert abs((fp - fm) / 2e-6 - grad[idx]) <= 1e-6 * max(1.0, abs(grad[idx])) + 1e-8, (name, idx)
    # weights on the last prefix only reproduce the plain objective
    last = np.zeros((s.N, s.n))
    last[:, -1] = -1.0 / s.N
    a = cp_head.backward(p["h"], p["W_head"], p["E"], p["W_g"], p["x"], s.n, s.r, dloss_dprefix=last)
    b = cp_head.backward(p["h"], p["W_head"], p["E"], p["W_g"], p["x"], s.n, s.r)
    assert np.allclose(a.dE, b.dE, atol=1e-15) and np.allclose(a.dh, b.dh, atol=1e-15)
    # discounted cross-entropy: sum_k gamma^k CE_k with CE_k = prefix_{k-1} - prefix_k is such a weighting
    gamma = 0.7
    wts = np.zeros((s.N, s.n))
    for k in range(s.n):
        wts[:, k] -= gamma ** k / s.N
        if k > 0:
            wts[:, k - 1] += gamma ** k / s.N
    fw = cp_head.forward(p["h"], p["W_head"], p["E"], p["W_g"], p["x"], s.n, s.r)
    pre = cp_head.prefix_log_probs(fw)
    ce = -np.diff(pre, axis=1, prepend=0.0)                      # CE_k = -log p(x_k | x_<k)
    assert abs(np.sum(wts * pre) - np.sum((gamma ** np.arange(s.n))[None, :] * ce) / s.N) < 1e-12
