"""Pins for the fp64 oracle's forward: things the paper and the mathematics fix
independently of the oracle's own code path."""
import itertools
import math

import numpy as np
import pytest
import torch

from oracle import cp_head
from paper_2410_17765_b200 import synth


def small(N=5, d=6, V=8, n=3, r=3, seed=1, scale=20.0):
    """fp64 random problem with O(1) logits (weights scaled up from 0.02)."""
    inp = synth.make_inputs(synth.Shape(N, d, V, n, r), seed=seed, weight_scale=scale)
    return inp


def run(inp, **kw):
    s = inp.shape
    return cp_head.forward(inp.h, inp.W_head, inp.E, inp.W_g, inp.x, s.n, s.r, **kw)


def test_rank1_is_sum_of_independent_cross_entropies():
    # Eq. 1: at r = 1 the joint is the product of n independent softmax heads.
    inp = small(N=7, d=16, V=11, n=4, r=1)
    fw = run(inp)
    h = inp.h.double()
    E = inp.E.double()
    total = torch.zeros(7, dtype=torch.float64)
    for s in range(4):
        logits = (h @ inp.W_head[s].double().T) @ E.T
        total -= torch.nn.functional.cross_entropy(logits, inp.x[:, s].long(), reduction="none")
    assert np.allclose(fw.logp, total.numpy(), rtol=0, atol=1e-12)
    assert np.all(fw.logw == 0.0)


@pytest.mark.parametrize("r", [1, 3, 5])
def test_joint_sums_to_one_over_all_tuples(r):
    # Eq. 3 + Eq. 5: sum over all V^n tuples of exp(logP) = 1.
    V, n = 8, 3
    base = small(N=1, d=6, V=V, n=n, r=r, seed=3)
    tuples = torch.tensor(list(itertools.product(range(V), repeat=n)), dtype=torch.int32)
    rep = synth.Inputs(shape=synth.Shape(V ** n, 6, V, n, r), h=base.h.expand(V ** n, -1).contiguous(),
                       W_head=base.W_head, E=base.E, W_g=base.W_g, x=tuples)
    fw = run(rep)
    assert abs(np.exp(fw.logp).sum() - 1.0) < 1e-12
    # marginalising the last token out of the n-head joint gives the (n-1)-head joint
    fw_prefix = cp_head.prefix_log_probs(fw)
    joint = np.exp(fw.logp).reshape(V, V, V)
    assert np.allclose(joint.sum(axis=2).reshape(-1), np.exp(fw_prefix[::V, 1]), atol=1e-13)
    assert np.allclose(joint.sum(axis=(1, 2)), np.exp(fw_prefix[::V * V, 0]), atol=1e-13)
    assert np.allclose(fw_prefix[:, 2], fw.logp, atol=1e-14)


def test_gate_weights_on_simplex():
    inp = small(N=50, d=32, V=8, n=2, r=7, scale=50.0)
    w = np.exp(cp_head.gate_log_weights(inp.h, inp.W_g))
    assert np.all(w >= 0)
    assert np.all(np.abs(w.sum(axis=1) - 1.0) <= 1e-15 * 7 * 4)


def test_matches_naive_product_form_with_python_loops():
    # Eq. 2 evaluated literally with probabilities and explicit loops.
    inp = small(N=3, d=4, V=5, n=2, r=3, seed=9)
    s = inp.shape
    h = inp.h.double().tolist()
    Wh = inp.W_head.double().tolist()
    E = inp.E.double().tolist()
    Wg = inp.W_g.double().tolist()
    x = inp.x.tolist()
    fw = run(inp)
    for i in range(s.N):
        g = [sum(Wg[a][m] * h[i][m] for m in range(s.d)) for a in range(s.r)]
        zg = sum(math.exp(v) for v in g)
        w = [math.exp(v) / zg for v in g]
        total = 0.0
        for a in range(s.r):
            prod = w[a]
            for t in range(s.n):
                k = t * s.r + a
                z = [sum(Wh[k][j][m] * h[i][m] for m in range(s.d)) for j in range(s.d)]
                logits = [sum(E[v][j] * z[j] for j in range(s.d)) for v in range(s.V)]
                den = sum(math.exp(l) for l in logits)
                prod *= math.exp(logits[x[i][t]]) / den
            total += prod
        assert abs(math.log(total) - fw.logp[i]) < 1e-12


def test_closed_forms():
    inp = small(N=6, d=8, V=13, n=3, r=4)
    s = inp.shape
    zero_heads = synth.Inputs(s, inp.h, torch.zeros_like(inp.W_head), inp.E, inp.W_g, inp.x)
    assert np.allclose(run(zero_heads).logp, -s.n * math.log(s.V), atol=1e-13)
    zero_E = synth.Inputs(s, inp.h, inp.W_head, torch.zeros_like(inp.E), inp.W_g, inp.x)
    assert np.allclose(run(zero_E).logp, -s.n * math.log(s.V), atol=1e-13)
    zero_gate = synth.Inputs(s, inp.h, inp.W_head, inp.E, torch.zeros_like(inp.W_g), inp.x)
    fw = run(zero_gate, aux_coef=1.0)
    assert np.allclose(np.exp(fw.logw), 1.0 / s.r, atol=1e-15)
    assert abs((fw.loss + fw.logp.mean()) - 1.0 / s.r) < 1e-14
    # identical experts: the mixture collapses to the rank-1 value for any gate
    same = inp.W_head.view(s.n, s.r, s.d, s.d)[:, :1].expand(-1, s.r, -1, -1).reshape(s.K, s.d, s.d).contiguous()
    fw_same = run(synth.Inputs(s, inp.h, same, inp.E, inp.W_g, inp.x))
    r1 = synth.Inputs(synth.Shape(s.N, s.d, s.V, s.n, 1), inp.h, same.view(s.n, s.r, s.d, s.d)[:, 0].contiguous(),
                      inp.E, inp.W_g[:1].contiguous(), inp.x)
    assert np.allclose(fw_same.logp, run(r1).logp, atol=1e-12)


def test_invariants():
    inp = small(N=9, d=8, V=10, n=2, r=5, seed=4)
    s = inp.shape
    fw = run(inp, aux_coef=0.5)
    perm = torch.tensor([3, 0, 4, 1, 2])
    Wp = inp.W_head.view(s.n, s.r, s.d, s.d)[:, perm].reshape(s.K, s.d, s.d).contiguous()
    fwp = run(synth.Inputs(s, inp.h, Wp, inp.E, inp.W_g[perm].contiguous(), inp.x), aux_coef=0.5)
    assert np.allclose(fw.logp, fwp.logp, atol=1e-13)
    assert abs(fw.loss - fwp.loss) < 1e-13
    amax = fw.a.max(axis=1)
    assert np.all(fw.logp >= amax - 1e-15) and np.all(fw.logp <= amax + math.log(s.r) + 1e-15)
    assert np.allclose(fw.q.sum(axis=1), 1.0, atol=1e-14)
    assert abs(fw.wbar.sum() - 1.0) < 1e-14
    assert fw.counts.sum() == s.N
    assert np.all(fw.C <= 0)
    # soft balance term vs the (wbar - 1/r)^2 form of Eq. 10
    assert abs(np.sum((fw.wbar - 1 / s.r) ** 2) - (np.sum(fw.wbar ** 2) - 1 / s.r)) < 1e-15


def test_first_token_marginal_is_mixture_of_first_factors():
    # Eq. 11 by explicit probabilities.
    inp = small(N=4, d=8, V=9, n=3, r=3, seed=12)
    s = inp.shape
    fw = run(inp)
    pre = cp_head.prefix_log_probs(fw)
    w = np.exp(fw.logw)
    h = inp.h.double().numpy()
    E = inp.E.double().numpy()
    for i in range(s.N):
        p = 0.0
        for a in range(s.r):
            logits = E @ (inp.W_head[a].double().numpy() @ h[i])
            sm = np.exp(logits) / np.exp(logits).sum()
            p += w[i, a] * sm[inp.x[i, 0]]
        assert abs(math.log(p) - pre[i, 0]) < 1e-12


def test_hard_counts_ties_go_to_lowest_index():
    inp = small(N=4, d=8, V=9, n=1, r=3)
    s = inp.shape
    fw = run(synth.Inputs(s, inp.h, inp.W_head, inp.E, torch.zeros_like(inp.W_g), inp.x))
    assert fw.counts.tolist() == [4, 0, 0]


def test_stable_for_large_logits():
    inp = small(N=4, d=16, V=12, n=2, r=2, scale=2000.0)
    fw = run(inp)
    assert np.all(np.isfinite(fw.logp)) and np.all(fw.logp <= 0)


def test_bf16_rounding_helper_matches_torch():
    g = torch.Generator().manual_seed(0)
    v = torch.randn(10000, generator=g, dtype=torch.float64) * 3
    v[:4] = torch.tensor([1.00390625, 1.01171875, -1.00390625, 0.0], dtype=torch.float64)  # ties
    ours = cp_head.round_to_bf16(v.numpy())
    ref = v.float().to(torch.bfloat16).double().numpy()
    assert np.array_equal(ours, ref)


def test_contract_mode_is_close_but_not_identical():
    inp = synth.make_inputs(synth.Shape(8, 256, 512, 2, 2), seed=5)
    a = run(inp)
    b = run(inp, round_z=True)
    diff = np.abs(a.logp - b.logp).max()
    assert 0 < diff < 1e-2
