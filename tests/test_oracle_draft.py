"""Pins for the oracle's draft generation (sampling section), independent of its code path:
brute-force marginals of the joint tensor, the likelihood function, and sampling statistics."""
import itertools

import numpy as np
import torch

from oracle import cp_head
from paper_2410_17765_b200 import synth


def problem(N=3, d=6, V=6, n=3, r=3, seed=21):
    return synth.make_inputs(synth.Shape(N, d, V, n, r), seed=seed, weight_scale=25.0)


def joint_tensor(inp, i):
    """Full joint P(x_1..x_n) for position i by evaluating the likelihood on all V^n tuples."""
    s = inp.shape
    tuples = torch.tensor(list(itertools.product(range(s.V), repeat=s.n)), dtype=torch.int32)
    T = tuples.shape[0]
    fw = cp_head.forward(inp.h[i:i + 1].expand(T, -1).contiguous(), inp.W_head, inp.E, inp.W_g, tuples, s.n, s.r)
    return np.exp(fw.logp).reshape((s.V,) * s.n)


def test_greedy_draft_follows_brute_force_conditionals():
    inp = problem()
    s = inp.shape
    dr = cp_head.draft(inp.h, inp.W_head, inp.E, inp.W_g, s.n, s.r, topk=3)
    for i in range(s.N):
        A = joint_tensor(inp, i)
        prefix = ()
        for t in range(s.n):
            # marginal over the tokens after t, conditioned on the drafted prefix
            marg = A[prefix].sum(axis=tuple(range(1, s.n - t))) if t < s.n - 1 else A[prefix]
            cond = marg / marg.sum()
            assert int(np.argmax(cond)) == dr.tokens[i, t]
            best3 = np.argsort(-cond, kind="stable")[:3]
            assert list(best3) == list(dr.topk_tokens[i, t])
            assert np.allclose(np.log(cond[best3]), dr.topk_logp[i, t], atol=1e-10)
            # mix is the log joint of (prefix, v)
            assert np.allclose(np.exp(dr.mix[i, t]), marg, atol=1e-12)
            prefix = prefix + (int(dr.tokens[i, t]),)
        assert abs(np.log(A[prefix]) - dr.logp_joint[i]) < 1e-10


def test_draft_logp_matches_likelihood_of_the_drafted_tokens():
    inp = problem(N=5, d=8, V=11, n=4, r=2, seed=4)
    s = inp.shape
    g = torch.Generator().manual_seed(3)
    u = torch.rand((s.N, s.n, s.V), generator=g, dtype=torch.float64).clamp_(1e-12, 1 - 1e-12)
    for uniform in (None, u):
        dr = cp_head.draft(inp.h, inp.W_head, inp.E, inp.W_g, s.n, s.r, uniform=uniform)
        fw = cp_head.forward(inp.h, inp.W_head, inp.E, inp.W_g, torch.from_numpy(dr.tokens), s.n, s.r)
        assert np.allclose(dr.logp_joint, fw.logp, atol=1e-12)
        pre = cp_head.prefix_log_probs(fw)
        # sum_v exp(mix[s, v]) = P(prefix before s)
        tot = cp_head.logsumexp(dr.mix, axis=2)
        assert np.allclose(tot[:, 0], 0.0, atol=1e-12)
        assert np.allclose(tot[:, 1:], pre[:, :-1], atol=1e-12)


def test_first_token_distribution_is_eq11():
    inp = problem(N=2, d=6, V=7, n=2, r=3, seed=8)
    s = inp.shape
    dr = cp_head.draft(inp.h, inp.W_head, inp.E, inp.W_g, s.n, s.r)
    w = np.exp(cp_head.gate_log_weights(inp.h, inp.W_g))
    for i in range(s.N):
        p = np.zeros(s.V)
        for a in range(s.r):
            logits = inp.E.double().numpy() @ (inp.W_head[a].double().numpy() @ inp.h[i].double().numpy())
            e = np.exp(logits - logits.max())
            p += w[i, a] * e / e.sum()
        assert np.allclose(np.exp(dr.mix[i, 0]), p, atol=1e-13)


def test_gumbel_max_sampling_frequencies_match_the_joint():
    # 4000 independent draws of a 2-token draft at one position: empirical pair frequencies vs the joint.
    inp = problem(N=1, d=6, V=4, n=2, r=3, seed=5)
    s = inp.shape
    A = joint_tensor(inp, 0)
    draws = 4000
    rep = synth.Inputs(shape=synth.Shape(draws, s.d, s.V, s.n, s.r), h=inp.h.expand(draws, -1).contiguous(),
                       W_head=inp.W_head, E=inp.E, W_g=inp.W_g, x=inp.x.expand(draws, -1).contiguous())
    g = torch.Generator().manual_seed(11)
    u = torch.rand((draws, s.n, s.V), generator=g, dtype=torch.float64).clamp_(1e-12, 1 - 1e-12)
    dr = cp_head.draft(rep.h, rep.W_head, rep.E, rep.W_g, s.n, s.r, uniform=u)
    freq = np.zeros((s.V, s.V))
    for a, b in dr.tokens:
        freq[a, b] += 1.0 / draws
    # standard error of a frequency <= 0.5/sqrt(draws) = 0.008; allow 5 sigma
    assert np.max(np.abs(freq - A)) < 0.04
    # temperature -> 0 reproduces the greedy draft
    cold = cp_head.draft(inp.h, inp.W_head, inp.E, inp.W_g, s.n, s.r, uniform=u[:1], temperature=1e-6)
    greedy = cp_head.draft(inp.h, inp.W_head, inp.E, inp.W_g, s.n, s.r)
    assert np.array_equal(cold.tokens, greedy.tokens)


def test_forced_prefix_gives_the_conditionals_of_that_path():
    """With every token forced the joint score is the likelihood of that sequence (Eq. 9), and the candidates
    of step s are the brute-force conditionals given the forced prefix; -1 entries fall back to the selection."""
    import itertools

    inp = synth.make_inputs(synth.Shape(3, 6, 5, 3, 3), seed=21, weight_scale=30.0)
    s = inp.shape
    args = (inp.h, inp.W_head, inp.E, inp.W_g)
    rng = np.random.default_rng(3)
    forced = rng.integers(0, s.V, size=(s.N, s.n))
    out = cp_head.draft(*args, s.n, s.r, topk=s.V, forced=forced)
    assert (out.tokens == forced).all()
    fw = cp_head.forward(*args, forced.astype(np.int32), s.n, s.r)
    assert np.allclose(out.logp_joint, fw.logp, atol=1e-12)
    joint = np.empty((s.N,) + (s.V,) * s.n)
    for tup in itertools.product(range(s.V), repeat=s.n):
        xs = np.tile(np.array(tup, dtype=np.int32), (s.N, 1))
        joint[(slice(None),) + tup] = np.exp(cp_head.forward(*args, xs, s.n, s.r).logp)
    for i in range(s.N):
        cond = joint[i, forced[i, 0], forced[i, 1]]
        cond = cond / cond.sum()
        order = out.topk_tokens[i, 2]
        assert np.allclose(np.exp(out.topk_logp[i, 2]), cond[order], atol=1e-12)
    partly = forced.copy()
    partly[:, 1:] = -1
    free = cp_head.draft(*args, s.n, s.r, topk=1, forced=partly)
    assert (free.tokens[:, 0] == forced[:, 0]).all()
    assert (free.tokens[:, 1] == out.topk_tokens[:, 1, 0]).all()   # greedy continuation of the forced first token
