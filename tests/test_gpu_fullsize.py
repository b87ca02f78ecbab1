"""GPU parity at the full workload sizes, in the launch configuration bench.py times.

The fp64 oracle is far too slow for whole batches at these sizes, but positions are
independent: log P and dh are checked on sampled positions of the full-batch run
(oracle evaluated on just those positions, with the full batch's -1/N upstream
gradient), and the weight gradients, which sum over all positions, are checked by
additivity over disjoint position chunks plus a direct comparison at a small N with
the full d, V, n, r.
"""
import functools

import numpy as np
import pytest
import torch

from oracle import cp_head
from paper_2410_17765_b200 import synth
from parity_checks import assert_expert_counts

pytestmark = pytest.mark.gpu

LOGP_TOL = 2e-3
GRAD_TOL = 1e-2


@functools.lru_cache(maxsize=1)
def inputs_for(name, targets="uniform"):
    return synth.make_inputs(synth.CONFIGS[name], seed=0, targets=targets)


def to_dev(inp):
    return [t.cuda() for t in (inp.h, inp.W_head, inp.E, inp.W_g, inp.x)]


def rel_l2(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def sample_positions(N, count, seed=0):
    g = torch.Generator().manual_seed(seed)
    idx = torch.randperm(N, generator=g)[:count].sort().values
    return idx


def test_train_fwd_full_size_sampled_logp():
    from paper_2410_17765_b200 import binding

    inp = inputs_for("train_fwd")
    s = inp.shape
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = binding.forward(*to_dev(inp), dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    logp = out["logp"].cpu().numpy()
    assert np.all(np.isfinite(logp)) and np.all(logp < 0)
    idx = sample_positions(s.N, 12)
    sub = synth.subsample_positions(inp, idx)
    ref = cp_head.forward(sub.h, sub.W_head, sub.E, sub.W_g, sub.x, s.n, s.r)
    assert np.max(np.abs(logp[idx.numpy()] - ref.logp)) <= LOGP_TOL
    # loss is the mean of -logP over all positions (the device reduction, checked against the host sum)
    assert abs(float(out["loss"].item()) + float(logp.astype(np.float64).mean())) <= 1e-4


def test_train_fwd_bwd_full_size_sampled_and_additive():
    from paper_2410_17765_b200 import binding

    inp = inputs_for("train_fwd_bwd")
    s = inp.shape
    dev = to_dev(inp)
    cs = binding.make_shape(s.N, s.d, s.V, s.n, s.r)
    saved = binding.Saved.alloc(cs)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = binding.alloc_workspace(binding.workspace_bytes(cs, binding.OP_BACKWARD))
    fwd = binding.forward(*dev, saved=saved, dev_status=st)
    full = binding.backward(*dev, saved, workspace=ws, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    # sampled positions: logP and dh against the oracle with the full batch's upstream gradient -1/N
    idx = sample_positions(s.N, 3)
    sub = synth.subsample_positions(inp, idx)
    up = np.full(len(idx), -1.0 / s.N)
    ref = cp_head.backward(sub.h, sub.W_head, sub.E, sub.W_g, sub.x, s.n, s.r, dloss_dlogp=up)
    reff = cp_head.forward(sub.h, sub.W_head, sub.E, sub.W_g, sub.x, s.n, s.r)
    assert np.max(np.abs(fwd["logp"].cpu().numpy()[idx.numpy()] - reff.logp)) <= LOGP_TOL
    got_dh = full["dh"][idx.cuda()].float().cpu().numpy()
    assert rel_l2(got_dh, ref.dh) <= GRAD_TOL
    # additivity of the weight gradients over two disjoint halves of the batch (same -1/N weights)
    acc = {k: torch.zeros_like(full[k], dtype=torch.float32) for k in ("dW_head", "dE", "dW_g")}
    half = s.N // 2
    upd = torch.full((half,), -1.0 / s.N, dtype=torch.float32, device="cuda")
    h, W, E, Wg, x = dev
    cs_h = binding.make_shape(half, s.d, s.V, s.n, s.r)
    saved_h = binding.Saved.alloc(cs_h)
    for lo in (0, half):
        hh, xx = h[lo:lo + half].contiguous(), x[lo:lo + half].contiguous()
        binding.forward(hh, W, E, Wg, xx, saved=saved_h, dev_status=st)
        part = binding.backward(hh, W, E, Wg, xx, saved_h, dloss_dlogp=upd, workspace=ws, dev_status=st)
        torch.cuda.synchronize()
        for k in acc:
            acc[k] += part[k].float()
        del part
    assert int(st.item()) == 0
    for k in acc:
        num = torch.linalg.vector_norm(acc[k] - full[k].float()).item()
        den = torch.linalg.vector_norm(full[k].float()).item()
        assert num / den <= GRAD_TOL, (k, num / den)


def test_weight_gradients_at_full_width_small_batch():
    """dE, dW_head, dW_g against the oracle at N=6 with the full d, V, n, r of the training shape."""
    from paper_2410_17765_b200 import binding

    big = inputs_for("train_fwd_bwd")
    s = big.shape
    sub = synth.subsample_positions(big, torch.arange(6))
    ref = cp_head.backward(sub.h, sub.W_head, sub.E, sub.W_g, sub.x, s.n, s.r, aux_coef=1.0)
    dev = to_dev(sub)
    saved = binding.Saved.alloc(binding.make_shape(6, s.d, s.V, s.n, s.r))
    binding.forward(*dev, aux_coef=1.0, saved=saved)
    g = binding.backward(*dev, saved, aux_coef=1.0)
    torch.cuda.synchronize()
    for key, want in (("dh", ref.dh), ("dW_head", ref.dW_head), ("dE", ref.dE), ("dW_g", ref.dW_g)):
        assert rel_l2(g[key].float().cpu().numpy(), want) <= GRAD_TOL, key


@pytest.mark.parametrize("name,count", [("decode_1", 1), ("decode_8", 3), ("decode_64", 3)])
def test_decode_full_size(name, count):
    from paper_2410_17765_b200 import binding

    inp = inputs_for(name)
    s = inp.shape
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = binding.score_draft(*to_dev(inp), dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    idx = sample_positions(s.N, count)
    sub = synth.subsample_positions(inp, idx)
    ref = cp_head.forward(sub.h, sub.W_head, sub.E, sub.W_g, sub.x, s.n, s.r)
    assert np.max(np.abs(out["logp_joint"].cpu().numpy()[idx.numpy()] - ref.logp)) <= LOGP_TOL
    pre = cp_head.prefix_log_probs(ref)
    assert np.max(np.abs(out["logp_prefix"].cpu().numpy()[idx.numpy()] - pre)) <= LOGP_TOL


def test_draft_generation_full_decode_size():
    """Greedy draft with 5 candidates at the decode shape (N=8, d=4096, V=128256, n=4, r=8)."""
    from paper_2410_17765_b200 import binding

    inp = inputs_for("decode_8")
    s = inp.shape
    ref = cp_head.draft(inp.h, inp.W_head, inp.E, inp.W_g, s.n, s.r, topk=5)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    h, W, E, Wg, _ = to_dev(inp)
    out = binding.sample_draft(h, W, E, Wg, s.n, topk=5, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    draft = out["draft"].cpu().numpy().astype(np.int64)
    fw = cp_head.forward(inp.h, inp.W_head, inp.E, inp.W_g, torch.from_numpy(draft), s.n, s.r)
    assert np.max(np.abs(out["logp_joint"].cpu().numpy() - fw.logp)) <= LOGP_TOL
    tl = out["topk_logp"].cpu().numpy()
    agree = 0
    for i in range(s.N):
        for t in range(s.n):
            # the drafted token is the oracle's argmax or within tolerance of it
            assert ref.mix[i, t, draft[i, t]] >= ref.mix[i, t].max() - 5 * LOGP_TOL
            if draft[i, t] != ref.tokens[i, t]:
                break
            agree += 1
            # candidate values are exact (unrounded z); the candidate *set* is selected on bf16-z logits,
            # so the last place may go to a token within the selection's resolution of the true k-th
            assert np.max(np.abs(np.sort(tl[i, t])[::-1] - ref.topk_logp[i, t])) <= 5 * LOGP_TOL
            cond = ref.mix[i, t] - cp_head.logsumexp(ref.mix[i, t][None, :], axis=1)[0]
            tk = out["topk_tokens"][i, t].cpu().numpy()
            assert np.max(np.abs(cond[tk] - tl[i, t])) <= LOGP_TOL
    assert agree >= 0.75 * s.N * s.n


def test_bigvocab_full_size_forward_and_backward_sampled():
    from paper_2410_17765_b200 import binding

    inp = inputs_for("bigvocab_fwd_bwd", "zipf")
    s = inp.shape
    dev = to_dev(inp)
    cs = binding.make_shape(s.N, s.d, s.V, s.n, s.r, 1.0)
    saved = binding.Saved.alloc(cs)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    fwd = binding.forward(*dev, aux_coef=1.0, saved=saved, want_counts=True, dev_status=st)
    g = binding.backward(*dev, saved, aux_coef=1.0, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    idx = sample_positions(s.N, 2)
    sub = synth.subsample_positions(inp, idx)
    reff = cp_head.forward(sub.h, sub.W_head, sub.E, sub.W_g, sub.x, s.n, s.r)
    assert np.max(np.abs(fwd["logp"].cpu().numpy()[idx.numpy()] - reff.logp)) <= LOGP_TOL
    # gate statistics over the whole batch: cheap for the oracle (no vocabulary work)
    logw = cp_head.gate_log_weights(inp.h, inp.W_g)
    wbar = np.exp(logw).mean(axis=0)
    assert np.max(np.abs(saved.wbar[: s.r].cpu().numpy() - wbar)) <= 1e-5
    assert_expert_counts(fwd["counts"].cpu().numpy(), logw)
    loss_ref = -float(fwd["logp"].double().mean().item()) + float(np.sum(wbar ** 2))
    assert abs(float(fwd["loss"].item()) - loss_ref) <= 1e-4
    # gradients: finite, and the hot target rows of dE (Zipf head) are where the mass is
    for k in ("dh", "dW_head", "dE", "dW_g"):
        assert bool(torch.isfinite(g[k].float()).all()), k
    row_norm = torch.linalg.vector_norm(g["dE"].float(), dim=1)
    assert int(torch.argmax(row_norm).item()) < 16
    # dh of the sampled positions against the oracle (upstream -1/N; the balance term's u uses the full-batch wbar,
    # so compare with aux off on both sides by subtracting nothing: run a second backward without aux)
    g0 = binding.backward(*dev, saved, aux_coef=None, dev_status=st)
    torch.cuda.synchronize()
    up = np.full(len(idx), -1.0 / s.N)
    ref = cp_head.backward(sub.h, sub.W_head, sub.E, sub.W_g, sub.x, s.n, s.r, dloss_dlogp=up)
    assert rel_l2(g0["dh"][idx.cuda()].float().cpu().numpy(), ref.dh) <= GRAD_TOL


def rel_l2_blocked(got_dev, want):
    """Relative L2 error of a bf16 device tensor against an fp64 array, one slice of the first axis at a time
    (the weight gradients at this size are several GB in fp64)."""
    num = den = 0.0
    for j in range(want.shape[0]):
        g = got_dev[j].double().cpu().numpy()
        num += float(np.sum((g - want[j]) ** 2))
        den += float(np.sum(want[j] ** 2))
    return (num / max(den, 1e-300)) ** 0.5


def test_bigvocab_small_batch_gradients():
    """Every gradient against the oracle at the full width of the big-vocabulary training step
    (d = 4096, V = 128256, n = 4, r = 16, Zipf targets, balance term on): a batch of 3 positions, which the
    fp64 oracle finishes in about a minute.  The weight gradients sum over positions and the balance term's
    gradient depends on the batch's mean gate weights, so they need a batch the oracle can run whole."""
    from paper_2410_17765_b200 import binding

    big = inputs_for("bigvocab_fwd_bwd", "zipf")
    s = big.shape
    sub = synth.subsample_positions(big, torch.tensor([0, 1, 2]))
    ref = cp_head.backward(sub.h, sub.W_head, sub.E, sub.W_g, sub.x, s.n, s.r, aux_coef=1.0)
    dev = to_dev(sub)
    saved = binding.Saved.alloc(binding.make_shape(3, s.d, s.V, s.n, s.r))
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    fwd = binding.forward(*dev, aux_coef=1.0, saved=saved, want_counts=True, dev_status=st)
    g = binding.backward(*dev, saved, aux_coef=1.0, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    reff = cp_head.forward(sub.h, sub.W_head, sub.E, sub.W_g, sub.x, s.n, s.r, aux_coef=1.0)
    assert np.max(np.abs(fwd["logp"].cpu().numpy() - reff.logp)) <= LOGP_TOL
    assert abs(float(fwd["loss"].item()) - reff.loss) <= LOGP_TOL
    assert_expert_counts(fwd["counts"].cpu().numpy(), reff.logw)
    assert rel_l2(g["dh"].float().cpu().numpy(), ref.dh) <= GRAD_TOL
    assert rel_l2(g["dW_g"].float().cpu().numpy(), ref.dW_g) <= GRAD_TOL
    # the gate gradient with the balance term really in it: it differs from the plain one
    plain = cp_head._coefficients(reff, 3, 0.0, None, None)[1]
    assert np.linalg.norm(ref.dg - plain) > 1e-3 * np.linalg.norm(plain)
    assert rel_l2_blocked(g["dW_head"], ref.dW_head) <= GRAD_TOL
    err_dE = rel_l2_blocked(g["dE"].view(64, -1, s.d), ref.dE.reshape(64, -1, s.d))
    assert err_dE <= GRAD_TOL, err_dE


def test_distill_full_size_sampled_kl_and_dh():
    """Eq. 14 at the fine-tuning size the benchmark times (N = 8192, d = 4096, V = 32000, n = 4, r = 8):
    KL terms, prefix scores and dh on sampled positions against the oracle run on just those positions
    with the full batch's weights; the loss against a host sum of the device's own per-position terms."""
    from oracle import distill
    from paper_2410_17765_b200 import binding

    inp = inputs_for("train_fwd_bwd")
    s = inp.shape
    T = synth.make_teacher_logits(s, inp.x, seed=0)
    dev = to_dev(inp) + [T.cuda()]
    cs = binding.make_shape(s.N, s.d, s.V, s.n, s.r)
    saved, dsaved = binding.Saved.alloc(cs), binding.DistillSaved.alloc(cs)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    beta, gamma = 0.9, 0.8
    out = binding.distill_forward(*dev, saved, dsaved, beta=beta, gamma=gamma, dev_status=st)
    g = binding.distill_backward(*dev, saved, dsaved, beta=beta, gamma=gamma, dev_status=st, skip=("dE",))
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    kl = out["kl"].cpu().numpy()
    prefix = out["logp_prefix"].cpu().numpy()
    assert np.all(np.isfinite(kl)) and np.all(kl > -1e-4)
    idx = sample_positions(s.N, 6, seed=3)
    sub = synth.subsample_positions(inp, idx)
    Tsub = T[idx]
    ref = distill.forward(sub.h, sub.W_head, sub.E, sub.W_g, sub.x, Tsub, s.n, s.r, beta=beta, gamma=gamma)
    assert np.max(np.abs(kl[idx.numpy()] - ref.kl)) <= LOGP_TOL
    assert np.max(np.abs(prefix[idx.numpy()] - ref.prefix)) <= LOGP_TOL
    disc = gamma ** np.arange(s.n)
    ce = -np.diff(np.concatenate([np.zeros((s.N, 1)), prefix.astype(np.float64)], axis=1), axis=1)
    want = float(np.sum(disc * (beta * kl.astype(np.float64) + (1 - beta) * ce)) / s.N)
    assert abs(float(out["loss"].item()) - want) <= 1e-4
    # dh of a position depends on that position only: oracle on the sample with the full batch's 1/N weights
    up, uk = distill.loss_weights(s.N, s.n, beta, gamma)
    gr = distill.backward(sub.h, sub.W_head, sub.E, sub.W_g, sub.x, Tsub, s.n, s.r, dloss_dprefix=up[: len(idx)],
                          dloss_dkl=uk[: len(idx)])
    assert rel_l2(g["dh"][idx.cuda()].float().cpu().numpy(), gr.dh) <= GRAD_TOL
