"""Pins for the oracle of the fine-tuning (distillation) objective, Eq. 14: special cases that
reduce to library routines, brute-force conditionals of the joint of Eq. 9, invariants, and
central finite differences for the gradient."""
import itertools

import numpy as np
import pytest
import torch
from scipy.special import rel_entr

from oracle import cp_head, distill
from paper_2410_17765_b200 import synth


def problem(seed=3, N=4, d=5, V=7, n=3, r=3, scale=20.0):
    inp = synth.make_inputs(synth.Shape(N, d, V, n, r), seed=seed, weight_scale=scale)
    T = synth.make_teacher_logits(inp.shape, inp.x, seed=seed)
    p = dict(h=inp.h.double().numpy().copy(), W_head=inp.W_head.double().numpy().copy(),
             E=inp.E.double().numpy().copy(), W_g=inp.W_g.double().numpy().copy(),
             x=inp.x.numpy().copy(), T=T.double().numpy().copy())
    return p, inp.shape


def test_rank1_matches_library_kl_and_cross_entropy():
    p, s = problem(r=1)
    out = distill.forward(p["h"], p["W_head"], p["E"], p["W_g"], p["x"], p["T"], s.n, 1, beta=0.9, gamma=0.8)
    for k in range(s.n):
        S = torch.from_numpy((p["h"] @ p["W_head"][k].T) @ p["E"].T)
        pd = torch.softmax(S, dim=1).numpy()
        pc = torch.softmax(torch.from_numpy(p["T"][:, k, :]), dim=1).numpy()
        assert np.allclose(out.kl[:, k], rel_entr(pd, pc).sum(axis=1), atol=1e-12)
        ce = torch.nn.functional.cross_entropy(S, torch.from_numpy(p["x"][:, k]).long(), reduction="none").numpy()
        assert np.allclose(out.ce[:, k], ce, atol=1e-12)
    disc = 0.8 ** np.arange(s.n)
    want = np.sum(disc * (0.9 * out.kl + 0.1 * out.ce)) / s.N
    assert abs(out.loss - want) < 1e-12


def test_conditionals_match_brute_force_marginals_of_the_joint():
    """p^d_k(v) = P(x_1..x_{k-1}, v) / P(x_1..x_{k-1}), both sides summed out of the full joint tensor
    built from cp_head.forward (itself pinned separately)."""
    p, s = problem(seed=6, N=2, V=5, n=3, r=3)
    logpd, logpi, _ = distill.conditional_log_probs(p["h"], p["W_head"], p["E"], p["W_g"], p["x"], s.n, s.r)
    joint = np.empty((s.N,) + (s.V,) * s.n)
    for tup in itertools.product(range(s.V), repeat=s.n):
        xs = np.tile(np.array(tup, dtype=np.int64), (s.N, 1))
        joint[(slice(None),) + tup] = np.exp(
            cp_head.forward(p["h"], p["W_head"], p["E"], p["W_g"], xs, s.n, s.r).logp)
    assert np.allclose(joint.reshape(s.N, -1).sum(axis=1), 1.0, atol=1e-12)
    for i in range(s.N):
        x = p["x"][i]
        m1 = joint[i].sum(axis=(1, 2))
        assert np.allclose(np.exp(logpd[i, 0]), m1, atol=1e-12)
        m2 = joint[i, x[0]].sum(axis=1)
        assert np.allclose(np.exp(logpd[i, 1]), m2 / m2.sum(), atol=1e-12)
        m3 = joint[i, x[0], x[1]]
        assert np.allclose(np.exp(logpd[i, 2]), m3 / m3.sum(), atol=1e-12)
    assert np.allclose(np.exp(logpi).sum(axis=2), 1.0, atol=1e-12)
    assert np.allclose(np.exp(logpd).sum(axis=2), 1.0, atol=1e-12)


def test_teacher_equal_to_own_conditionals_gives_zero_kl_and_is_shift_invariant():
    p, s = problem(seed=4)
    logpd, _, _ = distill.conditional_log_probs(p["h"], p["W_head"], p["E"], p["W_g"], p["x"], s.n, s.r)
    out = distill.forward(p["h"], p["W_head"], p["E"], p["W_g"], p["x"], logpd + 3.25, s.n, s.r)
    assert np.allclose(out.kl, 0.0, atol=1e-13)
    # prefix agrees with the forward oracle's prefix scores; CE telescopes
    fw = cp_head.forward(p["h"], p["W_head"], p["E"], p["W_g"], p["x"], s.n, s.r)
    assert np.allclose(out.prefix, cp_head.prefix_log_probs(fw), atol=1e-12)
    assert np.allclose(out.ce.sum(axis=1), -fw.logp, atol=1e-12)
    a = distill.forward(p["h"], p["W_head"], p["E"], p["W_g"], p["x"], p["T"], s.n, s.r)
    shift = np.linspace(-2, 5, s.N * s.n).reshape(s.N, s.n, 1)
    b = distill.forward(p["h"], p["W_head"], p["E"], p["W_g"], p["x"], p["T"] + shift, s.n, s.r)
    assert np.allclose(a.kl, b.kl, atol=1e-12)
    assert (a.kl > 0).all()


def test_loss_weights_reproduce_the_loss():
    p, s = problem(seed=9, r=2)
    beta, gamma, aux = 0.7, 0.6, 0.4
    out = distill.forward(p["h"], p["W_head"], p["E"], p["W_g"], p["x"], p["T"], s.n, s.r, beta=beta,
                          gamma=gamma, aux_coef=aux)
    up, uk = distill.loss_weights(s.N, s.n, beta, gamma)
    wbar = np.exp(cp_head.gate_log_weights(p["h"], p["W_g"])).mean(axis=0)
    assert abs(np.sum(up * out.prefix) + np.sum(uk * out.kl) + aux * np.sum(wbar ** 2) - out.loss) < 1e-13


@pytest.mark.parametrize("beta,gamma,aux,custom", [(0.9, 0.8, 0.0, False), (0.5, 1.0, 1.2, False),
                                                   (0.9, 0.8, 0.3, True), (1.0, 0.9, 0.0, False)])
def test_gradient_matches_central_differences(beta, gamma, aux, custom):
    p, s = problem(seed=11)
    rng = np.random.default_rng(1)
    up = rng.normal(size=(s.N, s.n)) if custom else None
    uk = rng.normal(size=(s.N, s.n)) if custom else None

    def objective():
        out = distill.forward(p["h"], p["W_head"], p["E"], p["W_g"], p["x"], p["T"], s.n, s.r, beta=beta,
                              gamma=gamma, aux_coef=aux)
        if not custom:
            return out.loss
        wbar = np.exp(cp_head.gate_log_weights(p["h"], p["W_g"])).mean(axis=0)
        return float(np.sum(up * out.prefix) + np.sum(uk * out.kl) + aux * np.sum(wbar ** 2))

    g = distill.backward(p["h"], p["W_head"], p["E"], p["W_g"], p["x"], p["T"], s.n, s.r, beta=beta, gamma=gamma,
                         aux_coef=aux, dloss_dprefix=up, dloss_dkl=uk)
    eps = 1e-6
    for name, grad in [("h", g.dh), ("W_head", g.dW_head), ("E", g.dE), ("W_g", g.dW_g)]:
        arr = p[name]
        for fi in rng.choice(arr.size, size=min(arr.size, 20), replace=False):
            idx = np.unravel_index(fi, arr.shape)
            old = arr[idx]
            arr[idx] = old + eps
            fp = objective()
            arr[idx] = old - eps
            fm = objective()
            arr[idx] = old
            num = (fp - fm) / (2 * eps)
            assert abs(num - grad[idx]) <= 2e-6 * max(1.0, abs(num)) + 1e-8, (name, idx, num, grad[idx])
    assert np.allclose(g.dg.sum(axis=1), 0.0, atol=1e-14)


def test_beta_zero_reduces_to_the_per_token_cross_entropy_gradient():
    p, s = problem(seed=12, r=2)
    up, _ = distill.loss_weights(s.N, s.n, 0.0, 0.7)
    a = distill.backward(p["h"], p["W_head"], p["E"], p["W_g"], p["x"], p["T"], s.n, s.r, beta=0.0, gamma=0.7)
    b = cp_head.backward(p["h"], p["W_head"], p["E"], p["W_g"], p["x"], s.n, s.r, dloss_dprefix=up)
    for name in ("dh", "dW_head", "dE", "dW_g"):
        assert np.allclose(getattr(a, name), getattr(b, name), atol=1e-14)
