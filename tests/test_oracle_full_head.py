"""Pins for the oracle's full-head variant (Eq. 6 as printed)."""
import numpy as np
import torch

from oracle import cp_head
from paper_2410_17765_b200 import synth


def problem(N=5, d=6, V=9, n=2, r=3, seed=31):
    inp = synth.make_inputs(synth.Shape(N, d, V, n, r), seed=seed, weight_scale=20.0)
    g = torch.Generator().manual_seed(seed + 1)
    W_full = (torch.randn((n * r, V, d), generator=g) * 0.4).to(torch.bfloat16)
    return inp, W_full


def test_shared_head_is_the_special_case_W_full_equals_E_times_W_head():
    # the fine-tuning section's construction W^(s)_alpha = W x w^(s)_alpha
    inp, _ = problem()
    s = inp.shape
    W_full = np.stack([inp.E.double().numpy() @ inp.W_head[k].double().numpy() for k in range(s.K)])
    a = cp_head.forward(inp.h, inp.W_head, inp.E, inp.W_g, inp.x, s.n, s.r, aux_coef=0.5)
    b = cp_head.forward_full(inp.h, W_full, inp.W_g, inp.x, s.n, s.r, aux_coef=0.5)
    assert np.allclose(a.logp, b.logp, atol=1e-12) and abs(a.loss - b.loss) < 1e-12
    ga = cp_head.backward(inp.h, inp.W_head, inp.E, inp.W_g, inp.x, s.n, s.r, aux_coef=0.5)
    gb = cp_head.backward_full(inp.h, W_full, inp.W_g, inp.x, s.n, s.r, aux_coef=0.5)
    assert np.allclose(ga.dh, gb.dh, atol=1e-13) and np.allclose(ga.dW_g, gb.dW_g, atol=1e-13)
    # chain rule back to the factors: dE = sum_k dW_full[k] W_head[k]^T, dW_head[k] = E^T dW_full[k]
    dE = sum(gb.dW_full[k] @ inp.W_head[k].double().numpy().T for k in range(s.K))
    assert np.allclose(dE, ga.dE, atol=1e-13)
    for k in range(s.K):
        assert np.allclose(inp.E.double().numpy().T @ gb.dW_full[k], ga.dW_head[k], atol=1e-13)


def test_rank1_full_head_is_independent_cross_entropies():
    inp, W_full = problem(N=6, d=8, V=10, n=3, r=1, seed=5)
    s = inp.shape
    fw = cp_head.forward_full(inp.h, W_full, inp.W_g, inp.x, s.n, s.r)
    h = inp.h.double().requires_grad_()
    Wf = W_full.double().requires_grad_()
    total = 0.0
    for t in range(s.n):
        total = total + torch.nn.functional.cross_entropy(h @ Wf[t].T, inp.x[:, t].long(), reduction="none")
    assert np.allclose(fw.logp, -total.detach().numpy(), atol=1e-12)
    (total.sum() / s.N).backward()
    g = cp_head.backward_full(inp.h, W_full, inp.W_g, inp.x, s.n, s.r)
    assert np.allclose(g.dh, h.grad.numpy(), atol=1e-13)
    assert np.allclose(g.dW_full, Wf.grad.numpy(), atol=1e-13)


def test_full_head_gradients_match_finite_differences():
    inp, W_full = problem(N=4, d=5, V=7, n=2, r=2, seed=9)
    s = inp.shape
    p = dict(h=inp.h.double().numpy().copy(), W=W_full.double().numpy().copy(), Wg=inp.W_g.double().numpy().copy())
    aux = 1.3

    def f():
        return cp_head.forward_full(p["h"], p["W"], p["Wg"], inp.x, s.n, s.r, aux_coef=aux).loss

    g = cp_head.backward_full(p["h"], p["W"], p["Wg"], inp.x, s.n, s.r, aux_coef=aux)
    rng = np.random.default_rng(1)
    for name, grad in (("h", g.dh), ("W", g.dW_full), ("Wg", g.dW_g)):
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
