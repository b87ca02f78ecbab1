"""Seeded random shapes through every likelihood entry point, against the oracle: ragged N, V, d
(multiples of 64), all n and several r, uniform and Zipf targets, chunked and unchunked backward."""

import numpy as np
import pytest
import torch

from oracle import cp_head
from paper_2410_17765_b200 import synth
from parity_checks import assert_expert_counts

pytestmark = pytest.mark.gpu


def rel_l2(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def random_case(it):
    rng = np.random.default_rng(1000 + it)
    d = int(rng.choice([64, 128, 192, 256, 320, 512, 1024]))
    n = int(rng.integers(1, 5))
    r = int(rng.choice([1, 2, 3, 4, 8, 16]))
    N = int(rng.choice([1, 2, 7, 33, 128, 129, 300, 700]))
    V = int(rng.integers(2, 3000))
    cost = n * r * (d * d + V * d)
    if N * cost > 1.5e10:
        N = max(1, int(1.5e10 / cost))
    return synth.Shape(N, d, V, n, r), str(rng.choice(["uniform", "zipf"])), float(rng.choice([0.0, 1.0])), \
        int(rng.choice([0, 128, 256, 1024]))


@pytest.mark.parametrize("it", range(12))
def test_random_shape(it):
    from paper_2410_17765_b200 import binding

    shape, targets, aux, chunk = random_case(it)
    n, r = shape.n, shape.r
    inp = synth.make_inputs(shape, seed=it, targets=targets)
    ref = cp_head.forward(inp.h, inp.W_head, inp.E, inp.W_g, inp.x, n, r, aux_coef=aux)
    refg = cp_head.backward(inp.h, inp.W_head, inp.E, inp.W_g, inp.x, n, r, aux_coef=aux)
    W_full = synth.make_full_head(shape, seed=it, weight_scale=3.0)
    reff = cp_head.forward_full(inp.h, W_full, inp.W_g, inp.x, n, r)
    reffg = cp_head.backward_full(inp.h, W_full, inp.W_g, inp.x, n, r)
    dev = [t.cuda() for t in (inp.h, inp.W_head, inp.E, inp.W_g, inp.x)]
    cs = binding.make_shape(shape.N, shape.d, shape.V, n, r)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    with binding.knobs(CPMTP_BWD_CHUNK_ROWS=chunk or None):
        saved = binding.Saved.alloc(cs)
        f = binding.forward(*dev, aux_coef=aux if aux else None, saved=saved, want_counts=True, dev_status=st)
        g = binding.backward(*dev, saved, aux_coef=aux if aux else None, dev_status=st)
    sc = binding.score_draft(*dev, dev_status=st)
    saved_f = binding.Saved.alloc_full(cs)
    ff = binding.forward_full(dev[0], W_full.cuda(), dev[3], dev[4], saved=saved_f, dev_status=st)
    gf = binding.backward_full(dev[0], W_full.cuda(), dev[3], dev[4], saved_f, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0, shape
    assert np.abs(f["logp"].cpu().numpy() - ref.logp).max() <= 2e-3, shape
    assert np.abs(sc["logp_joint"].cpu().numpy() - ref.logp).max() <= 2e-3, shape
    assert abs(float(f["loss"].item()) - ref.loss) <= 2e-3, shape
    assert np.abs(ff["logp"].cpu().numpy() - reff.logp).max() <= 2e-3, shape
    assert_expert_counts(f["counts"].cpu().numpy(), ref.logw)
    assert_expert_counts(ff["counts"].cpu().numpy(), reff.logw)
    for key, want in (("dh", refg.dh), ("dW_head", refg.dW_head), ("dE", refg.dE), ("dW_g", refg.dW_g)):
        if np.linalg.norm(want) > 0:
            assert rel_l2(g[key].float().cpu().numpy(), want) <= 1e-2, (shape, key)
    for key, want in (("dh", reffg.dh), ("dW_full", reffg.dW_full), ("dW_g", reffg.dW_g)):
        if np.linalg.norm(want) > 0:
            assert rel_l2(gf[key].float().cpu().numpy(), want) <= 1e-2, (shape, key)


def random_distill_case(it):
    rng = np.random.default_rng(5000 + it)
    d = int(rng.choice([64, 128, 192, 256, 512, 1024]))
    n = int(rng.integers(1, 5))
    r = int(rng.choice([1, 2, 3, 4, 5, 6, 7, 8, 12, 16, 32]))
    N = int(rng.choice([1, 2, 7, 33, 128, 129, 300]))
    V = int(rng.integers(2, 2500))
    if rng.random() < 0.4:
        V = (V + 7) // 8 * 8          # vector teacher loads
    cost = n * r * (d * d + V * d)
    if N * cost > 8e9:
        N = max(1, int(8e9 / cost))
    mem = N * n * r * V * 8 * 3       # the oracle keeps [N, n, r, V] fp64 arrays
    if mem > 2e9:
        N = max(1, int(N * 2e9 / mem))
    return synth.Shape(N, d, V, n, r), float(rng.choice([0.0, 0.5, 0.9, 1.0])), float(rng.choice([0.7, 1.0])), \
        float(rng.choice([0.0, 1.0])), int(rng.choice([0, 96, 256, 1024]))


@pytest.mark.parametrize("it", range(10))
def test_random_distill_shape(it):
    """Eq. 14 on random shapes: every padded-rank instantiation, ragged groups and vocabularies, both teacher
    load paths, chunked backward."""
    from oracle import distill
    from paper_2410_17765_b200 import binding

    shape, beta, gamma, aux, chunk = random_distill_case(it)
    n, r = shape.n, shape.r
    inp = synth.make_inputs(shape, seed=100 + it, weight_scale=2.0 if shape.d <= 512 else 1.0)
    T = synth.make_teacher_logits(shape, inp.x, seed=it)
    ref = distill.forward(inp.h, inp.W_head, inp.E, inp.W_g, inp.x, T, n, r, beta=beta, gamma=gamma, aux_coef=aux)
    refg = distill.backward(inp.h, inp.W_head, inp.E, inp.W_g, inp.x, T, n, r, beta=beta, gamma=gamma, aux_coef=aux)
    dev = [t.cuda() for t in (inp.h, inp.W_head, inp.E, inp.W_g, inp.x, T)]
    cs = binding.make_shape(shape.N, shape.d, shape.V, n, r)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    saved, dsaved = binding.Saved.alloc(cs), binding.DistillSaved.alloc(cs)
    with binding.knobs(CPMTP_BWD_CHUNK_ROWS=chunk or None):
        out = binding.distill_forward(*dev, saved, dsaved, beta=beta, gamma=gamma, aux_coef=aux if aux else None,
                                      dev_status=st)
        g = binding.distill_backward(*dev, saved, dsaved, beta=beta, gamma=gamma, aux_coef=aux if aux else None,
                                     dev_status=st)
        torch.cuda.synchronize()
    assert int(st.item()) == 0, shape
    assert np.abs(out["kl"].cpu().numpy() - ref.kl).max() <= 2e-3, shape
    assert np.abs(out["logp_prefix"].cpu().numpy() - ref.prefix).max() <= 2e-3, shape
    assert abs(float(out["loss"].item()) - ref.loss) <= 2e-3, shape
    for key, want in (("dh", refg.dh), ("dW_head", refg.dW_head), ("dE", refg.dE), ("dW_g", refg.dW_g)):
        if np.linalg.norm(want) > 0:
            assert rel_l2(g[key].float().cpu().numpy(), want) <= 1e-2, (shape, key)
