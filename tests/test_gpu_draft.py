"""GPU parity of draft generation (cpmtp_sample_draft) against the fp64 oracle.

A drafted token is an argmax, so a near-tie may legitimately resolve differently in
fp32: tokens are compared exactly where the oracle's margin is clear, and otherwise
the GPU's choice must be within the tolerance of the oracle's best score.  What is
unique is compared outright: the joint log-probability of the GPU's own draft (the
oracle's likelihood of those tokens) and the candidates' conditional log-probabilities."""
import numpy as np
import pytest
import torch

from oracle import cp_head
from paper_2410_17765_b200 import synth

pytestmark = pytest.mark.gpu

LOGP_TOL = 2e-3


def to_dev(inp):
    return [t.cuda() for t in (inp.h, inp.W_head, inp.E, inp.W_g)]


def check_against_oracle(inp, out, ref, topk, uniform=None, temperature=1.0):
    s = inp.shape
    draft = out["draft"].cpu().numpy().astype(np.int64)
    assert draft.min() >= 0 and draft.max() < s.V
    # 1. joint log-probability of the GPU's own draft
    fw = cp_head.forward(inp.h, inp.W_head, inp.E, inp.W_g, torch.from_numpy(draft), s.n, s.r)
    assert np.max(np.abs(out["logp_joint"].cpu().numpy() - fw.logp)) <= LOGP_TOL
    # 2. tokens: follow the oracle position by position while the prefixes agree
    tk = out["topk_tokens"].cpu().numpy()
    tl = out["topk_logp"].cpu().numpy()
    same_prefix = np.ones(s.N, dtype=bool)
    agree = 0
    for t in range(s.n):
        mix = ref.mix[:, t, :]
        norm = cp_head.logsumexp(mix, axis=1) if t == 0 else None
        for i in np.nonzero(same_prefix)[0]:
            if uniform is None:
                score = mix[i]
            else:
                cond = mix[i] - cp_head.logsumexp(ref.mix[i, t][None, :], axis=1)[0]
                score = cond / temperature - np.log(-np.log(uniform[i, t].double().numpy()))
            best = score.max()
            assert score[draft[i, t]] >= best - 2 * LOGP_TOL / min(1.0, temperature), (i, t)
            if draft[i, t] == ref.tokens[i, t]:
                agree += 1
                # candidates of this conditional: same scores (the order of near-equal ones may differ)
                want = ref.topk_logp[i, t]
                assert np.max(np.abs(np.sort(tl[i, t])[::-1] - want)) <= 3 * LOGP_TOL, (i, t)
                cond_all = mix[i] - cp_head.logsumexp(mix[i][None, :], axis=1)[0]
                assert np.max(np.abs(cond_all[tk[i, t]] - tl[i, t])) <= LOGP_TOL
                assert len(set(tk[i, t].tolist())) == topk
            else:
                same_prefix[i] = False
    return agree / (s.N * s.n)


@pytest.mark.parametrize("N,V,d,n,r,topk", [(8, 5000, 256, 4, 8, 5), (1, 3000, 512, 3, 4, 1), (64, 2500, 128, 2, 3, 8),
                                            (5, 130, 64, 8, 32, 2)])
def test_greedy_draft_matches_oracle(N, V, d, n, r, topk):
    from paper_2410_17765_b200 import binding

    shape = synth.Shape(N=N, d=d, V=V, n=n, r=r)
    inp = synth.make_inputs(shape, seed=7, weight_scale=2.0)
    ref = cp_head.draft(inp.h, inp.W_head, inp.E, inp.W_g, n, r, topk=topk)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = binding.sample_draft(*to_dev(inp), n, topk=topk, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    frac = check_against_oracle(inp, out, ref, topk)
    assert frac >= 0.9
    # greedy: the first candidate is the drafted token
    assert torch.equal(out["topk_tokens"][:, :, 0], out["draft"])


def test_sampled_draft_matches_oracle():
    from paper_2410_17765_b200 import binding

    shape = synth.Shape(N=16, d=256, V=4000, n=3, r=4)
    inp = synth.make_inputs(shape, seed=9, weight_scale=2.0)
    g = torch.Generator().manual_seed(5)
    u = torch.rand((shape.N, shape.n, shape.V), generator=g, dtype=torch.float32).clamp_(1e-7, 1 - 1e-7)
    for temperature in (1.0, 0.5):
        ref = cp_head.draft(inp.h, inp.W_head, inp.E, inp.W_g, shape.n, shape.r, topk=4, uniform=u,
                            temperature=temperature)
        out = binding.sample_draft(*to_dev(inp), shape.n, uniform=u.cuda(), temperature=temperature, topk=4)
        torch.cuda.synchronize()
        frac = check_against_oracle(inp, out, ref, 4, uniform=u, temperature=temperature)
        assert frac >= 0.9
    # sampling spreads over tokens: not every position takes the most likely one
    assert not torch.equal(out["topk_tokens"][:, :, 0], out["draft"])


def test_draft_is_deterministic_and_validates_arguments():
    from paper_2410_17765_b200 import binding

    shape = synth.Shape(N=4, d=128, V=900, n=2, r=2)
    inp = synth.make_inputs(shape, seed=2)
    dev = to_dev(inp)
    a = binding.sample_draft(*dev, shape.n, topk=3)
    b = binding.sample_draft(*dev, shape.n, topk=3)
    torch.cuda.synchronize()
    assert torch.equal(a["draft"], b["draft"]) and torch.equal(a["topk_logp"], b["topk_logp"])
    with pytest.raises(binding.CpmtpError):
        binding.sample_draft(*dev, shape.n, topk=9)
    with pytest.raises(binding.CpmtpError):
        binding.sample_draft(*dev, shape.n, uniform=torch.rand((4, 2, 900), device="cuda"), temperature=0.0)


def test_long_runs_of_equal_scores_go_to_the_lowest_ids():
    """Whole stretches of the vocabulary with exactly equal scores (here: identical rows of E, so identical logits
    for every expert) are more ties than the candidate array of the selection holds, so the exhaustive merge runs;
    the result is still the oracle's: ties resolve to the lowest token id."""
    from paper_2410_17765_b200 import binding

    shape = synth.Shape(N=3, d=128, V=5000, n=2, r=4)
    inp = synth.make_inputs(shape, seed=3, weight_scale=2.0)
    E = inp.E.clone()
    E[:] = E[0]                       # every token the same: all scores equal
    E[4000:4003] = inp.E[1] * 4       # three tokens that stand out, inside a later chunk
    ref = cp_head.draft(inp.h, inp.W_head, E, inp.W_g, shape.n, shape.r, topk=8)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = binding.sample_draft(inp.h.cuda(), inp.W_head.cuda(), E.cuda(), inp.W_g.cuda(), shape.n, topk=8, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    tk = out["topk_tokens"].cpu().numpy()
    # the equal-score tokens that fill the remaining places are the lowest ids, in order
    for i in range(shape.N):
        for t in range(shape.n):
            rest = [v for v in tk[i, t].tolist() if not 4000 <= v < 4003]
            assert rest == list(range(len(rest))), (i, t, tk[i, t])
            assert set(tk[i, t].tolist()) == set(ref.topk_tokens[i, t].tolist())
    assert np.max(np.abs(np.sort(out["topk_logp"].cpu().numpy(), axis=2) - np.sort(ref.topk_logp, axis=2))) <= LOGP_TOL


def test_vocabulary_of_more_chunks_than_threads():
    """V > 2048 * 256: the merging block's threads each hold the candidate lists of several chunks."""
    from paper_2410_17765_b200 import binding

    shape = synth.Shape(N=2, d=64, V=2048 * 256 + 5000, n=2, r=2)
    inp = synth.make_inputs(shape, seed=13, weight_scale=8.0)
    ref = cp_head.draft(inp.h, inp.W_head, inp.E, inp.W_g, shape.n, shape.r, topk=4)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = binding.sample_draft(*to_dev(inp), shape.n, topk=4, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    frac = check_against_oracle(inp, out, ref, 4)
    assert frac >= 0.75


def test_verify_draft_matches_oracle():
    from paper_2410_17765_b200 import binding

    g = torch.Generator().manual_seed(0)
    N, n = 1000, 4
    draft = torch.randint(0, 3, (N, n), generator=g, dtype=torch.int32)
    base = torch.randint(0, 3, (N, n), generator=g, dtype=torch.int32)
    got = binding.verify_draft(draft.cuda(), base.cuda())
    assert np.array_equal(got.cpu().numpy(), cp_head.accepted_prefix_greedy(draft, base))
    # probabilistic rule: draft-side conditionals from cumulative sums, base side arbitrary
    cond = -torch.rand((N, n), generator=g) * 3
    pre = torch.cumsum(cond, dim=1).float()
    lb = (cond + torch.randn((N, n), generator=g)).float()
    u = torch.rand((N, n), generator=g).float()
    got = binding.verify_draft(logp_prefix=pre.cuda(), logp_base=lb.cuda(), uniform=u.cuda()).cpu().numpy()
    want = cp_head.accepted_prefix_sampled(pre, lb, u)
    # a decision within fp32 rounding of its threshold may go either way: compare where the margin is clear
    ratio = np.minimum(1.0, np.exp(lb.double().numpy() - np.diff(pre.double().numpy(), axis=1, prepend=0.0)))
    clear = np.all(np.abs(u.double().numpy() - ratio) > 1e-5, axis=1)
    assert clear.mean() > 0.99
    assert np.array_equal(got[clear], want[clear])
    assert got.min() >= 0 and got.max() <= n


def test_forced_tokens_walk_a_draft_tree():
    """Forced entries replace the selection; the reported candidates are the conditionals given the forced path
    and the joint score is the likelihood of the path; -1 entries are left to the sampler."""
    from paper_2410_17765_b200 import binding

    shape = synth.Shape(N=6, d=256, V=1500, n=3, r=4)
    inp = synth.make_inputs(shape, seed=11, weight_scale=2.0)
    dev = to_dev(inp)
    g = torch.Generator().manual_seed(5)
    forced = torch.randint(0, shape.V, (shape.N, shape.n), generator=g, dtype=torch.int32)
    forced[::2, 1:] = -1                     # every other position: only the first token is given
    ref = cp_head.draft(inp.h, inp.W_head, inp.E, inp.W_g, shape.n, shape.r, topk=4, forced=forced)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = binding.sample_draft(*dev, shape.n, topk=4, forced=forced.cuda(), dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    draft = out["draft"].cpu()
    given = forced >= 0
    assert torch.equal(draft[given], forced[given])
    assert np.array_equal(draft.numpy(), ref.tokens)
    assert np.max(np.abs(out["logp_joint"].cpu().numpy() - ref.logp_joint)) <= 2e-3
    assert np.array_equal(out["topk_tokens"].cpu().numpy(), ref.topk_tokens)
    assert np.max(np.abs(out["topk_logp"].cpu().numpy() - ref.topk_logp)) <= 2e-3
    # a token beyond the vocabulary is clamped and reported
    bad = forced.clone()
    bad[0, 0] = shape.V + 7
    out2 = binding.sample_draft(*dev, shape.n, topk=1, forced=bad.cuda(), dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 1 and int(out2["draft"][0, 0].item()) == shape.V - 1
