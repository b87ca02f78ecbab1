"""CPU oracle for the rank-r CP multi-token head log-likelihood (fp64, numpy).

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of the
paper's definitions that the CUDA library is judged against.  It shares no code
with the CUDA path and must never be imported by the product package; only the
tests, the smoke check and the benchmark's CPU-baseline leg call it.

Every operand is widened exactly to float64 before any arithmetic (bf16 and
fp32 values are exactly representable), so the result is the paper's definition
evaluated on the given bit patterns, up to fp64 rounding.

Notation (paper name -> name here): embedding e_t -> h[i, :]; shared head
matrix W of the fine-tuning section -> E[V, d]; the small per-(s, alpha)
matrices w^(s)_alpha of that section -> W_head[k, :, :] with k = s*r + alpha,
indexed [out][in]; gate matrix W_h of Eq. 7 -> W_g[r, d]; targets
x_{t+1..t+n} -> x[i, 0..n-1].

Readings of the paper taken here:
  * The per-head matrix of the fine-tuning section is printed with shape
    V x E, which cannot be multiplied on the right of W (V x E) and would not
    be "smaller"; it is read as E x E (d x d) and the factor logits are
    E . (W_head[s, alpha] . h).
  * No bias, no temperature, natural logarithms.
  * Loss = mean over positions of -log P, plus aux_coef * sum_alpha wbar_alpha^2
    where wbar is the mean gate weight over positions (the differentiable form
    of the balance penalty of Eq. 10: replacing the hard fraction n_alpha / N
    by wbar_alpha, sum (wbar - 1/r)^2 = sum wbar^2 - 1/r).

Parity pins: every function below is pinned by tests/test_oracle_*.py
(closed forms, brute-force normalisation, the rank-1 reduction to independent
cross-entropies, finite differences; for draft generation the brute-force
conditionals of the full joint tensor and sampling frequencies).  Nothing here
is "parity unpinned".
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


def _f64(a) -> np.ndarray:
    """Exact widening to float64 of a numpy array or a torch CPU tensor."""
    if hasattr(a, "detach"):  # torch tensor (bf16 has no numpy dtype: go through torch)
        import torch

        return a.detach().to("cpu").to(torch.float64).numpy()
    return np.asarray(a, dtype=np.float64)


def _i64(a) -> np.ndarray:
    if hasattr(a, "detach"):
        return a.detach().to("cpu").numpy().astype(np.int64)
    return np.asarray(a, dtype=np.int64)


def logsumexp(a: np.ndarray, axis: int) -> np.ndarray:
    """log sum exp along ``axis`` with the maximum subtracted first."""
    m = np.max(a, axis=axis, keepdims=True)
    return (m + np.log(np.sum(np.exp(a - m), axis=axis, keepdims=True))).squeeze(axis)


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float64 values to the nearest bf16 (ties to even), returned as float64.

    Used only by the explanatory "contract" mode that mimics storing z in bf16.
    """
    f = np.asarray(a, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    u = (u + 0x7FFF + lsb) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64)


def gate_log_weights(h, W_g) -> np.ndarray:
    """log w[i, alpha], w = softmax(W_g h) (Eq. 7)."""
    g = _f64(h) @ _f64(W_g).T
    return g - logsumexp(g, axis=1)[:, None]


def head_projection(h, W_head_k) -> np.ndarray:
    """z[i, :] = W_head[k] . h[i, :] for one head k (reduced head of the
    fine-tuning section: W^(s)_alpha = W x w^(s)_alpha applied right to left)."""
    return _f64(h) @ _f64(W_head_k).T


def factor_log_probs(h, W_head, E, x, n: int, r: int, *, round_z: bool = False):
    """C[i, s, alpha] = log P^(s)(x[i, s] | alpha) (Eq. 6 with Eq. 8).

    Returns (C, lse, tgt): lse[i, k] = logsumexp_v S[i, k, v] and
    tgt[i, k] = S[i, k, x[i, s]], with S[i, k, :] = E . z[i, k, :].
    """
    hd, Ed, xi = _f64(h), _f64(E), _i64(x)
    N = hd.shape[0]
    K = n * r
    lse = np.empty((N, K))
    tgt = np.empty((N, K))
    rows = np.arange(N)
    for k in range(K):
        s = k // r
        z = head_projection(hd, W_head[k])
        if round_z:
            z = round_to_bf16(z)
        S = z @ Ed.T  # [N, V]
        lse[:, k] = logsumexp(S, axis=1)
        tgt[:, k] = S[rows, xi[:, s]]
    C = (tgt - lse).reshape(N, n, r)
    return C, lse, tgt


@dataclass
class Forward:
    logp: np.ndarray   # [N]     log P(x_{t+1..t+n} | ctx)          (Eq. 9)
    logw: np.ndarray   # [N, r]  log mixture weights                (Eq. 7)
    C: np.ndarray      # [N, n, r] factor log-probabilities         (Eq. 8)
    lse: np.ndarray    # [N, n*r]
    tgt: np.ndarray    # [N, n*r]
    a: np.ndarray      # [N, r]  log w_alpha + sum_s C[s, alpha]
    q: np.ndarray      # [N, r]  posterior over experts exp(a - logp)
    wbar: np.ndarray   # [r]     mean gate weight
    counts: np.ndarray  # [r]    n_alpha of Eq. 10: positions whose largest weight is alpha
    loss: float


def forward(h, W_head, E, W_g, x, n: int, r: int, *, aux_coef: float = 0.0,
            round_z: bool = False) -> Forward:
    """Joint log-likelihood per position in the log domain (last line of Eq. 9)."""
    logw = gate_log_weights(h, W_g)
    C, lse, tgt = factor_log_probs(h, W_head, E, x, n, r, round_z=round_z)
    a = logw + C.sum(axis=1)
    logp = logsumexp(a, axis=1)
    q = np.exp(a - logp[:, None])
    w = np.exp(logw)
    wbar = w.mean(axis=0)
    counts = np.bincount(np.argmax(w, axis=1), minlength=r).astype(np.int64)
    loss = float(-logp.mean() + aux_coef * np.sum(wbar * wbar))
    return Forward(logp=logp, logw=logw, C=C, lse=lse, tgt=tgt, a=a, q=q, wbar=wbar,
                   counts=counts, loss=loss)


def prefix_log_probs(fw: Forward) -> np.ndarray:
    """log P(x_{t+1..t+s}) for s = 1..n: the mixture with only the first s
    factors folded into the expert weights (sampling section; s = 1 is Eq. 11)."""
    partial = np.cumsum(fw.C, axis=1)                      # [N, n, r]
    return logsumexp(fw.logw[:, None, :] + partial, axis=2)  # [N, n]


@dataclass
class Gradients:
    dh: np.ndarray       # [N, d]
    dW_head: np.ndarray  # [n*r, d, d]
    dE: np.ndarray       # [V, d]
    dW_g: np.ndarray     # [r, d]
    dg: np.ndarray       # [N, r]  gradient w.r.t. the gate logits W_g h
    c: np.ndarray        # [N, r]  gradient w.r.t. every C[i, s, alpha] (same for all s)


def _coefficients(fw: Forward, N: int, aux_coef: float, dloss_dlogp, dloss_dprefix):
    """Gradient of the objective w.r.t. every C[i, s, alpha] (returned as c3 [N, n, r]) and w.r.t. the
    gate logits (dg [N, r]).

    Plain objective  sum_i up_i logp_i:  c3[i, s, :] = up_i q[i, :] for every s.
    Per-token objective  sum_i sum_s up[i, s] * prefix[i, s]  with prefix[i, s] = log P(x_1..x_{s+1}), e.g. the
    discounted cross-entropy part of the fine-tuning loss (Eq. 14 and the sum after it: CE_k = prefix_{k-1} -
    prefix_k):  prefix_s depends on C[t, :] for t <= s through its own expert posterior q_s, hence
      c3[i, t, :] = sum_{s >= t} up[i, s] q_s[i, :],   dg = sum_s up[i, s] (q_s - w)."""
    w = np.exp(fw.logw)
    u = 2.0 * aux_coef * fw.wbar / N
    aux_dg = w * (u[None, :] - (w @ u)[:, None])
    n = fw.C.shape[1]
    if dloss_dprefix is None:
        up = np.full(N, -1.0 / N) if dloss_dlogp is None else _f64(dloss_dlogp)
        c = up[:, None] * fw.q
        return np.repeat(c[:, None, :], n, axis=1), up[:, None] * (fw.q - w) + aux_dg
    ups = _f64(dloss_dprefix)                                   # [N, n]
    a_s = fw.logw[:, None, :] + np.cumsum(fw.C, axis=1)         # [N, n, r]
    q_s = np.exp(a_s - logsumexp(a_s, axis=2)[:, :, None])
    weighted = ups[:, :, None] * q_s
    c3 = np.cumsum(weighted[:, ::-1, :], axis=1)[:, ::-1, :]    # suffix sums over s
    dg = (weighted - ups[:, :, None] * w[:, None, :]).sum(axis=1) + aux_dg
    return c3, dg


def backward(h, W_head, E, W_g, x, n: int, r: int, *, aux_coef: float = 0.0,
             dloss_dlogp=None, dloss_dprefix=None) -> Gradients:
    """Gradient of  loss = sum_i up_i * logp_i + aux_coef * sum_alpha wbar_alpha^2
    with up_i = dloss_dlogp[i] (default -1/N, the mean negative log-likelihood); or, with
    dloss_dprefix [N, n], of  sum_i sum_s dloss_dprefix[i, s] * log P(x_1..x_{s+1})  (see _coefficients).

    Chain rule through Eq. 9, Eq. 8 and Eq. 7:
      d loss / d a[i, alpha]      = up_i * q[i, alpha]            (softmax of the outer logsumexp)
      d loss / d C[i, s, alpha]   = up_i * q[i, alpha]            (a is linear in C)
      d loss / d S[i, k, v]       = c[i, alpha(k)] * (1[v = x[i, s(k)]] - softmax(S[i, k])_v)
      d loss / d logw[i, alpha]   = up_i * q[i, alpha]
      d loss / d g[i, beta]       = up_i * (q[i, beta] - w[i, beta])              (log-softmax Jacobian)
                                    + w[i, beta] * (u_beta - sum_gamma w[i, gamma] u_gamma),
                                    u_beta = 2 aux_coef wbar_beta / N             (softmax Jacobian)
    then plain matrix calculus for z = W_head[k] h, S = E z, g = W_g h.
    """
    hd, Ed, Wg, xi = _f64(h), _f64(E), _f64(W_g), _i64(x)
    N, d = hd.shape
    V = Ed.shape[0]
    K = n * r
    fw = forward(h, W_head, E, W_g, x, n, r, aux_coef=aux_coef)
    c3, dg = _coefficients(fw, N, aux_coef, dloss_dlogp, dloss_dprefix)
    c = c3[:, -1, :] if dloss_dprefix is None else c3

    dh = dg @ Wg
    dW_g = dg.T @ hd
    dE = np.zeros((V, d))
    dW_head = np.empty((K, d, d))
    rows = np.arange(N)
    for k in range(K):
        s, alpha = divmod(k, r)
        Wk = _f64(W_head[k])
        z = hd @ Wk.T
        S = z @ Ed.T
        P = np.exp(S - fw.lse[:, k][:, None])
        G = -c3[:, s, alpha][:, None] * P
        G[rows, xi[:, s]] += c3[:, s, alpha]
        dz = G @ Ed
        dE += G.T @ z
        dW_head[k] = dz.T @ hd
        dh += dz @ Wk
    return Gradients(dh=dh, dW_head=dW_head, dE=dE, dW_g=dW_g, dg=dg, c=c)


@dataclass
class Draft:
    tokens: np.ndarray       # [N, n]      drafted tokens x_{t+1..t+n}
    logp_joint: np.ndarray   # [N]         log P(tokens) under the CP head (Eq. 9 at the drafted tokens)
    topk_tokens: np.ndarray  # [N, n, k]   most likely next tokens given the drafted prefix, best first
    topk_logp: np.ndarray    # [N, n, k]   their conditional log-probabilities
    mix: np.ndarray          # [N, n, V]   log P(x_{t+1..t+s-1} = drafted prefix, x_{t+s} = v)


def draft(h, W_head, E, W_g, n: int, r: int, *, topk: int = 1, uniform=None,
          temperature: float = 1.0, forced=None) -> Draft:
    """Sequential draft generation from the factors (sampling section).

    The first token comes from the marginal of Eq. 11; for every later token the
    expert weights are multiplied by the factors of the tokens already drawn
    (b_alpha = w_alpha * prod_{t<s} P^(t)(x_t | alpha), the prose under Eq. 12)
    and the next token is drawn from  sum_alpha b_alpha P^(s)(v | alpha) / sum_alpha b_alpha
    (the printed Eq. 12 / Eq. 13 omit the s-th factor and the normaliser; this is the
    reading their surrounding text describes).

    uniform=None: temperature 0, the most likely token is taken (ties -> lowest id).
    uniform [N, n, V] in (0, 1): the token is drawn exactly from the conditional
    distribution, sharpened by 1/temperature, with the Gumbel-max rule
    argmax_v( log p(v) / temperature - log(-log u[v]) ).
    topk: the k most likely tokens of each conditional (unperturbed), best first.
    forced [N, n] int or None: entries >= 0 are taken as the drafted token of that step instead of the
    selection (the candidates are still those of the conditional); -1 leaves the step to the sampler.  This is
    how a caller walks a draft tree: the conditionals of a node are those given its path.
    """
    hd, Ed = _f64(h), _f64(E)
    N = hd.shape[0]
    V = Ed.shape[0]
    logw = gate_log_weights(h, W_g)
    logP = np.empty((N, n, r, V))
    for k in range(n * r):
        s, alpha = divmod(k, r)
        S = head_projection(hd, W_head[k]) @ Ed.T
        logP[:, s, alpha, :] = S - logsumexp(S, axis=1)[:, None]
    lb = logw.copy()                                   # log b_alpha
    rows = np.arange(N)
    tokens = np.empty((N, n), dtype=np.int64)
    top_t = np.empty((N, n, topk), dtype=np.int64)
    top_lp = np.empty((N, n, topk))
    mixes = np.empty((N, n, V))
    u = None if uniform is None else _f64(uniform)
    for s in range(n):
        mix = logsumexp(lb[:, :, None] + logP[:, s, :, :], axis=1)      # [N, V]
        norm = logsumexp(lb, axis=1)                                    # log sum_alpha b_alpha
        mixes[:, s, :] = mix
        order = np.argsort(-mix, axis=1, kind="stable")[:, :topk]
        top_t[:, s, :] = order
        top_lp[:, s, :] = np.take_along_axis(mix, order, axis=1) - norm[:, None]
        if u is None:
            x_s = order[:, 0]
        else:
            x_s = np.argmax((mix - norm[:, None]) / temperature - np.log(-np.log(u[:, s, :])), axis=1)
        if forced is not None:
            f = _i64(forced)[:, s]
            x_s = np.where(f >= 0, f, x_s)
        tokens[:, s] = x_s
        lb = lb + logP[rows, s, :, x_s]
    return Draft(tokens=tokens, logp_joint=logsumexp(lb, axis=1), topk_tokens=top_t, topk_logp=top_lp,
                 mix=mixes)


# ---------------------------------------------------------------------------
# Full head (Eq. 6 as printed): one unembedding W^(s)_alpha in R^{V x d} per (token, expert),
# stacked as W_full[k, V, d] with k = s*r + alpha.  The shared-head form above is the special
# case W_full[k] = E . W_head[k].


def factor_log_probs_full(h, W_full, x, n: int, r: int):
    """C, lse, tgt as in factor_log_probs, with logits S[i, k, :] = W_full[k] . h[i] (Eq. 6, Eq. 8)."""
    hd, xi = _f64(h), _i64(x)
    N = hd.shape[0]
    K = n * r
    lse = np.empty((N, K))
    tgt = np.empty((N, K))
    rows = np.arange(N)
    for k in range(K):
        S = hd @ _f64(W_full[k]).T
        lse[:, k] = logsumexp(S, axis=1)
        tgt[:, k] = S[rows, xi[:, k // r]]
    return (tgt - lse).reshape(N, n, r), lse, tgt


def forward_full(h, W_full, W_g, x, n: int, r: int, *, aux_coef: float = 0.0) -> Forward:
    """Eq. 9 with the full head of Eq. 6."""
    logw = gate_log_weights(h, W_g)
    C, lse, tgt = factor_log_probs_full(h, W_full, x, n, r)
    a = logw + C.sum(axis=1)
    logp = logsumexp(a, axis=1)
    q = np.exp(a - logp[:, None])
    w = np.exp(logw)
    wbar = w.mean(axis=0)
    counts = np.bincount(np.argmax(w, axis=1), minlength=r).astype(np.int64)
    loss = float(-logp.mean() + aux_coef * np.sum(wbar * wbar))
    return Forward(logp=logp, logw=logw, C=C, lse=lse, tgt=tgt, a=a, q=q, wbar=wbar, counts=counts, loss=loss)


@dataclass
class GradientsFull:
    dh: np.ndarray       # [N, d]
    dW_full: np.ndarray  # [n*r, V, d]
    dW_g: np.ndarray     # [r, d]


def backward_full(h, W_full, W_g, x, n: int, r: int, *, aux_coef: float = 0.0, dloss_dlogp=None,
                  dloss_dprefix=None) -> GradientsFull:
    """Gradient of the same objective as `backward`, for the full head:
    dS as there; dW_full[k] = dS[:, k, :]^T h, dh = sum_k dS[:, k, :] W_full[k] + dg W_g."""
    hd, Wg, xi = _f64(h), _f64(W_g), _i64(x)
    N, d = hd.shape
    K = n * r
    fw = forward_full(h, W_full, W_g, x, n, r, aux_coef=aux_coef)
    c3, dg = _coefficients(fw, N, aux_coef, dloss_dlogp, dloss_dprefix)
    dh = dg @ Wg
    dW_g = dg.T @ hd
    V = _f64(W_full[0]).shape[0]
    dW_full = np.empty((K, V, d))
    rows = np.arange(N)
    for k in range(K):
        s, alpha = divmod(k, r)
        Wk = _f64(W_full[k])
        S = hd @ Wk.T
        G = -c3[:, s, alpha][:, None] * np.exp(S - fw.lse[:, k][:, None])
        G[rows, xi[:, s]] += c3[:, s, alpha]
        dW_full[k] = G.T @ hd
        dh += G @ Wk
    return GradientsFull(dh=dh, dW_full=dW_full, dW_g=dW_g)


def accepted_prefix_greedy(draft_tokens, base_tokens) -> np.ndarray:
    """Draft-then-verify with greedy decoding (Preliminaries): the number of leading draft tokens that
    equal the base model's tokens, i.e. the length of the longest common prefix, per position."""
    d, b = _i64(draft_tokens), _i64(base_tokens)
    out = np.zeros(d.shape[0], dtype=np.int64)
    for i in range(d.shape[0]):
        k = 0
        while k < d.shape[1] and d[i, k] == b[i, k]:
            k += 1
        out[i] = k
    return out


def accepted_prefix_sampled(logp_draft_prefix, logp_base, uniform) -> np.ndarray:
    """Probabilistic verification (the generalisation the Preliminaries mention): draft token s, drawn
    with conditional probability q_s = exp(prefix[s] - prefix[s-1]), is kept with probability
    min(1, p_s / q_s), p_s = exp(logp_base[s]) the base model's probability of that token; the accepted
    length is the number of tokens kept before the first rejection (uniform[i, s] decides token s)."""
    pre, lb, u = _f64(logp_draft_prefix), _f64(logp_base), _f64(uniform)
    N, n = pre.shape
    out = np.zeros(N, dtype=np.int64)
    for i in range(N):
        k = 0
        prev = 0.0
        while k < n:
            logq = pre[i, k] - prev
            if not (u[i, k] < min(1.0, np.exp(lb[i, k] - logq))):
                break
            prev = pre[i, k]
            k += 1
        out[i] = k
    return out
