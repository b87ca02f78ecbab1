"""CPU oracle for the fine-tuning (distillation) objective of the CP head (fp64, numpy).

TEST INFRASTRUCTURE ONLY, like oracle/cp_head.py: never imported by the product package.

The fine-tuning section trains only the head against a frozen model whose own next-token
distributions p^c are available.  For the k-th predicted token it forms (Eq. 14)

    L_k = beta * KL(p^d_{t+k}, p^c_{t+k}) + (1 - beta) * CE(p^d_{t+k}, x_{t+k})

and sums the L_k with a discount gamma, plus the balance term.  Readings taken here:
  * p^d_{t+k} is the head's distribution of token k GIVEN the tokens before it, taken from the
    training sequence: sum_a pi_{k,a} P^(k)(v | a) with pi_{k,a} proportional to
    w_a * prod_{t<k} P^(t)(x_t | a)  (the conditional of the sampling section, teacher-forced).
    The printed conditioning "p^c_{t+1:t_k-1}" is garbled; the sequence's own tokens stand in.
  * KL(p, q) = sum_v p(v) log(p(v) / q(v)), arguments in the printed order (head first).
  * CE(p^d_{t+k}, x_{t+k}) = -log p^d_{t+k}(x_{t+k}) = prefix_{k-1} - prefix_k with
    prefix_k = log P(x_{t+1..t+k}).
  * The sum after Eq. 14 is printed with limits 0..d; it is read as sum_{k=1..n} gamma^{k-1} L_k,
    averaged over the positions.
  * p^c is given as logits T[i, k, :] (any additive constant per row is irrelevant).

Parity pins (tests/test_oracle_distill.py): rank 1 against scipy's rel_entr and a library
cross-entropy; teacher equal to the head's own conditional gives KL = 0; the conditionals against
brute-force marginals of the joint of Eq. 9; invariance to a shift of the teacher logits; the
gradient against central finite differences of `forward`.  Nothing here is "parity unpinned".
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

from . import cp_head as cp


def conditional_log_probs(h, W_head, E, W_g, x, n: int, r: int, *, round_z: bool = False):
    """log p^d[i, k, v] and log pi[i, k, a] (mixture weights before token k), teacher-forced on x.

    Also returns log P^(k)(v | a) as logP[i, k, a, v] for the gradient.  round_z rounds the projected
    hidden states to bf16 first (explanatory mode only, as in cp_head.factor_log_probs)."""
    hd, Ed, xi = cp._f64(h), cp._f64(E), cp._i64(x)
    N = hd.shape[0]
    V = Ed.shape[0]
    logw = cp.gate_log_weights(h, W_g)
    logP = np.empty((N, n, r, V))
    for k in range(n * r):
        s, a = divmod(k, r)
        z = cp.head_projection(hd, W_head[k])
        if round_z:
            z = cp.round_to_bf16(z)
        S = z @ Ed.T
        logP[:, s, a, :] = S - cp.logsumexp(S, axis=1)[:, None]
    rows = np.arange(N)
    lb = logw.copy()
    logpi = np.empty((N, n, r))
    logpd = np.empty((N, n, V))
    for s in range(n):
        logpi[:, s, :] = lb - cp.logsumexp(lb, axis=1)[:, None]
        logpd[:, s, :] = cp.logsumexp(logpi[:, s, :, None] + logP[:, s, :, :], axis=1)
        lb = lb + logP[rows, s, :, xi[:, s]]
    return logpd, logpi, logP


@dataclass
class Distill:
    kl: np.ndarray       # [N, n]  KL(p^d_k, p^c_k)
    ce: np.ndarray       # [N, n]  -log p^d_k(x_k)
    prefix: np.ndarray   # [N, n]  log P(x_1..x_k)
    loss: float          # (1/N) sum_i sum_k gamma^k (beta KL + (1-beta) CE) + aux_coef sum_a wbar_a^2


def forward(h, W_head, E, W_g, x, teacher, n: int, r: int, *, beta: float = 0.9, gamma: float = 1.0,
            aux_coef: float = 0.0, round_z: bool = False) -> Distill:
    """Eq. 14 and the discounted sum after it."""
    logpd, _, _ = conditional_log_probs(h, W_head, E, W_g, x, n, r, round_z=round_z)
    T = cp._f64(teacher)
    logpc = T - cp.logsumexp(T, axis=2)[:, :, None]
    pd = np.exp(logpd)
    kl = np.sum(pd * (logpd - logpc), axis=2)
    xi = cp._i64(x)
    N = xi.shape[0]
    ce = -np.take_along_axis(logpd, xi[:, :, None], axis=2)[:, :, 0]
    prefix = -np.cumsum(ce, axis=1)
    disc = gamma ** np.arange(n)
    wbar = np.exp(cp.gate_log_weights(h, W_g)).mean(axis=0)
    loss = float(np.sum(disc[None, :] * (beta * kl + (1.0 - beta) * ce)) / N + aux_coef * np.sum(wbar * wbar))
    return Distill(kl=kl, ce=ce, prefix=prefix, loss=loss)


def loss_weights(N: int, n: int, beta: float, gamma: float):
    """Upstream gradients that make  sum up*prefix + sum uk*kl  equal the data part of the loss:
    uk[i, k] = beta gamma^k / N;  CE_k = prefix_{k-1} - prefix_k  gives
    up[i, k] = (1 - beta) (gamma^{k+1} [k+1 < n] - gamma^k) / N."""
    disc = gamma ** np.arange(n + 1)
    disc[n] = 0.0
    uk = np.tile(beta * disc[:n] / N, (N, 1))
    up = np.tile((1.0 - beta) * (disc[1:] - disc[:n]) / N, (N, 1))
    return up, uk


def backward(h, W_head, E, W_g, x, teacher, n: int, r: int, *, beta: float = 0.9, gamma: float = 1.0,
             aux_coef: float = 0.0, dloss_dprefix=None, dloss_dkl=None) -> cp.Gradients:
    """Gradient of  sum_i sum_k (up[i,k] prefix[i,k] + uk[i,k] kl[i,k]) + aux_coef sum_a wbar_a^2;
    up / uk default to loss_weights(beta, gamma), i.e. the loss of `forward`.

    With P = P^(k)(. | a), e = pi_{k,a} P, l(v) = log(p^d_k(v) / p^c_k(v)), pm_{k,a} = sum_v e(v) l(v):
      d kl_k / d S[k, a, u]      = e(u) l(u) - P(u) pm_{k,a}
      d kl_k / d log b_{k, a}    = pm_{k,a} - pi_{k,a} kl_k          (b = unnormalised pi)
    and log b_{k,a} = log w_a + sum_{t<k} C[t, a] carries the second line to the gate and to the
    earlier heads' target terms, where it joins the coefficients of the cross-entropy part."""
    hd, Ed, Wg, xi = cp._f64(h), cp._f64(E), cp._f64(W_g), cp._i64(x)
    N, d = hd.shape
    V = Ed.shape[0]
    K = n * r
    up_def, uk_def = loss_weights(N, n, beta, gamma)
    up = up_def if dloss_dprefix is None else cp._f64(dloss_dprefix)
    uk = uk_def if dloss_dkl is None else cp._f64(dloss_dkl)
    fw = cp.forward(h, W_head, E, W_g, x, n, r, aux_coef=aux_coef)
    c3, dg = cp._coefficients(fw, N, aux_coef, None, up)          # cross-entropy part
    logpd, logpi, logP = conditional_log_probs(h, W_head, E, W_g, x, n, r)
    T = cp._f64(teacher)
    ell = logpd - (T - cp.logsumexp(T, axis=2)[:, :, None])       # [N, n, V]
    pi = np.exp(logpi)
    e = pi[:, :, :, None] * np.exp(logP)                          # [N, n, r, V]
    pm = np.sum(e * ell[:, :, None, :], axis=3)                   # [N, n, r]
    kl = pm.sum(axis=2)
    tb = uk[:, :, None] * (pm - pi * kl[:, :, None])              # d obj / d log b_{k,a}
    c3 = c3.copy()
    for k in range(n):
        c3[:, :k, :] += tb[:, k, None, :]                         # heads before k
    w = np.exp(fw.logw)
    D = tb.sum(axis=1)                                            # d obj / d log w from the KL part
    dg = dg + D - w * D.sum(axis=1, keepdims=True)

    dh = dg @ Wg
    dW_g = dg.T @ hd
    dE = np.zeros((V, d))
    dW_head = np.empty((K, d, d))
    rows = np.arange(N)
    for k in range(K):
        s, a = divmod(k, r)
        Wk = cp._f64(W_head[k])
        z = hd @ Wk.T
        P = np.exp(logP[:, s, a, :])
        G = -c3[:, s, a][:, None] * P
        G[rows, xi[:, s]] += c3[:, s, a]
        G += uk[:, s][:, None] * (e[:, s, a, :] * ell[:, s, :] - P * pm[:, s, a][:, None])
        dz = G @ Ed
        dE += G.T @ z
        dW_head[k] = dz.T @ hd
        dh += dz @ Wk
    return cp.Gradients(dh=dh, dW_head=dW_head, dE=dE, dW_g=dW_g, dg=dg, c=c3)
