"""fp64 CPU oracle for the GRADIENT of the MtPC head's window log-likelihood: TEST INFRASTRUCTURE, not a product path.

Training minimises the negative log-likelihood of the observed windows (Sec. 4.1, Eq. 6); its gradient with
respect to the hidden states and to the head's parameters is the derivative of
    L = sum_t weight[t] * log q(x_{t,1..n} | h_t)
through the circuit (Eq. CP / Eq. HMM / Eq. BTree), the softmaxes of Sec. 3.3 and the two projections. The oracle
does not derive that gradient by hand: it writes the forward DEFINITION out once more with plain PyTorch CPU ops in
float64 (matmul, log_softmax, gather, logsumexp - the same steps, in the same order, as oracle/mtpc_oracle.py) and
lets reverse-mode differentiation of exactly those steps produce it. It shares no code with the CUDA library and is
only called by the tests, the smoke check and the benchmark's CPU legs.

composite_loss_grad does the same for the training loss itself (Eq. 6: per-slot conditionals, valid-token normalisation,
discount gamma).

Pins (tests/test_oracle_grad.py): the torch forward equals the numpy oracle's forward to 1e-12; every gradient
equals central finite differences of the NUMPY oracle's log-likelihood (an independent route: no autograd, no torch);
closed forms (CP with r = 1: d/dlogit = weight * (onehot - softmax); a masked byte has zero gradient; gradients of
a normalised circuit's weights sum to zero within each sum unit); the Eq. 6 loss equals the numpy oracle's
composite_loss and its gradient equals central finite differences of that; with gamma = 1 and every byte valid it is
the gradient of the mean joint negative log-likelihood. lowrank_grad (App. G, shared unembeddings with low-rank
adaptors) is pinned by central finite differences of the numpy oracle's lowrank_unembedding and by the closed forms
dW_base = sum_j dU_ij, and dA = 0 where B = 0. No function here is left unpinned.
"""
from __future__ import annotations

import numpy as np
import torch

CP, HMM, BTREE, HMM_CTX = 0, 1, 2, 3


def _lse(x, dim):
    return torch.logsumexp(x, dim=dim)


def _evidence(logphi, x):
    """g[t, i, k] = log phi[t, i, k, x_ti]; a negative target marginalises the byte (the unit outputs one)."""
    T, n, r, v = logphi.shape
    safe = torch.clamp(x, min=0)
    idx = safe[:, :, None, None].expand(T, n, r, 1)
    g = torch.gather(logphi, 3, idx)[..., 0]
    return torch.where((x < 0)[:, :, None], torch.zeros_like(g), g)


def _btree_product(j, lo, hi, logw, g, r):
    mid = lo + (hi - lo) // 2
    out = 0.0
    for child, (a, b) in ((2 * j + 1, (lo, mid)), (2 * j + 2, (mid, hi))):
        if b - a == 1:
            out = out + g[:, a, :]
        else:
            below = _btree_product(child, a, b, logw, g, r)
            rows = 1 + (child - 1) * r
            out = out + _lse(logw[:, rows:rows + r, :] + below[:, None, :], dim=-1)
    return out


def forward(family: int, h, W_emit, W_sum, T_static, targets):
    """log q of every window, [T], from torch float64 tensors; the definition, step by step (Sec. 3.3, Eq. CP / HMM /
    BTree). T_static: static transition logits (HMM), the transition bias (HMM_CTX, may be None), else None."""
    n, r, v, d = W_emit.shape
    T = h.shape[0]
    logits = (h @ W_emit.reshape(n * r * v, d).T).reshape(T, n, r, v)
    slog = (h @ W_sum.T).reshape(T, W_sum.shape[0] // r, r)
    return forward_from_logits(family, logits, slog, T_static, targets)


def forward_from_logits(family: int, logits, slog, T_static, targets):
    """The same definition from the two projections on: logits [T, n, r, v] of the input units, slog [T, S, r] of the sum
    units (Sec. 3.3), then the softmaxes and the circuit."""
    T, n, r, v = logits.shape
    logphi = torch.log_softmax(logits, dim=-1)
    if family == HMM_CTX and T_static is not None:
        slog = torch.cat([slog[:, :1, :], slog[:, 1:, :] + T_static.reshape(1, -1, r)], dim=1)
    logw = torch.log_softmax(slog, dim=-1)
    g = _evidence(logphi, targets)
    if family == CP:
        return _lse(logw[:, 0, :] + g.sum(dim=1), dim=-1)
    if family == HMM:
        logA = torch.log_softmax(T_static, dim=-1)
        alpha = logw[:, 0, :] + g[:, 0, :]
        for i in range(1, n):
            alpha = g[:, i, :] + _lse(alpha[:, :, None] + logA[i - 1][None, :, :], dim=1)
        return _lse(alpha, dim=-1)
    if family == HMM_CTX:
        alpha = logw[:, 0, :] + g[:, 0, :]
        for i in range(1, n):
            alpha = g[:, i, :] + _lse(alpha[:, :, None] + logw[:, 1 + (i - 1) * r:1 + i * r, :], dim=1)
        return _lse(alpha, dim=-1)
    if family == BTREE:
        return _lse(logw[:, 0, :] + _btree_product(0, 0, n, logw, g, r), dim=-1)
    raise ValueError(family)


def window_logprob_logit_grad(family: int, h, W_emit, W_sum, T_static, targets, weight):
    """Gradient of L = sum_t weight[t] * log q_t with respect to the two projections themselves: dlogit [T, n, r, v]
    (input units) and dslog [T, S, r] (sum units), numpy float64. By the chain rule through the projections,
    dW_emit = dlogit^T h, dW_sum = dslog^T h and dh = dlogit W_emit + dslog W_sum (pinned that way); a test uses the
    magnitudes |dlogit|, |dslog| to bound, entry by entry, what rounding dlogit to 16 bits may cost a gradient."""
    th = torch.tensor(np.asarray(h, dtype=np.float64))
    tW = torch.tensor(np.asarray(W_emit, dtype=np.float64))
    tR = torch.tensor(np.asarray(W_sum, dtype=np.float64))
    n, r, v, d = tW.shape
    T = th.shape[0]
    logits = (th @ tW.reshape(n * r * v, d).T).reshape(T, n, r, v).requires_grad_(True)
    slog = (th @ tR.T).reshape(T, tR.shape[0] // r, r).requires_grad_(True)
    tT = None
    if T_static is not None and family in (HMM, HMM_CTX):
        tT = torch.tensor(np.asarray(T_static, dtype=np.float64))
    tx = torch.tensor(np.asarray(targets, dtype=np.int64))
    tw = torch.tensor(np.asarray(weight, dtype=np.float64))
    lp = forward_from_logits(family, logits, slog, tT, tx)
    (lp * tw).sum().backward()
    return dict(dlogit=logits.grad.numpy(), dslog=np.zeros(tuple(slog.shape)) if slog.grad is None else slog.grad.numpy())


def window_logprob_grad(family: int, h, W_emit, W_sum, T_static, targets, weight):
    """Gradient of L = sum_t weight[t] * log q_t with respect to h [T, d], W_emit [n, r, v, d], W_sum [S r, d] and
    T_static (static logits or contextual bias; None if the head has none). numpy in, numpy float64 out:
    dict(logprob [T], dh, dW_emit, dW_sum, dT_static)."""
    th = torch.tensor(np.asarray(h, dtype=np.float64), requires_grad=True)
    tW = torch.tensor(np.asarray(W_emit, dtype=np.float64), requires_grad=True)
    tR = torch.tensor(np.asarray(W_sum, dtype=np.float64), requires_grad=True)
    tT = None
    if T_static is not None and family in (HMM, HMM_CTX):
        tT = torch.tensor(np.asarray(T_static, dtype=np.float64), requires_grad=True)
    tx = torch.tensor(np.asarray(targets, dtype=np.int64))
    tw = torch.tensor(np.asarray(weight, dtype=np.float64))
    lp = forward(family, th, tW, tR, tT, tx)
    (lp * tw).sum().backward()
    zero = lambda t: np.zeros(tuple(t.shape)) if t.grad is None else t.grad.numpy()
    return dict(logprob=lp.detach().numpy(), dh=zero(th), dW_emit=zero(tW), dW_sum=zero(tR),
                dT_static=None if tT is None else zero(tT))


def composite_loss_grad(family: int, h, W_emit, W_sum, T_static, targets, num_sequences: int, gamma: float):
    """Eq. (6) and its gradient: L = sum_j gamma^(j-1) L_j with L_j = -(1/N) sum_i (1/V_ij) sum_t log p(x_{t+j} | x_{<t+j}),
    the conditional of slot j being the ratio of consecutive prefix marginals of the window's circuit. Written as
    that definition (one masked evaluation of the circuit per prefix length, then the sums of Eq. 6 with explicit
    loops over slots and sequences) and differentiated by reverse mode.
    Returns dict(slot_loss [n], loss, dh, dW_emit, dW_sum, dT_static)."""
    th = torch.tensor(np.asarray(h, dtype=np.float64), requires_grad=True)
    tW = torch.tensor(np.asarray(W_emit, dtype=np.float64), requires_grad=True)
    tR = torch.tensor(np.asarray(W_sum, dtype=np.float64), requires_grad=True)
    tT = None
    if T_static is not None and family in (HMM, HMM_CTX):
        tT = torch.tensor(np.asarray(T_static, dtype=np.float64), requires_grad=True)
    tx = torch.tensor(np.asarray(targets, dtype=np.int64))
    T, n = tx.shape
    N = num_sequences
    L = T // N
    prefix = []
    for j in range(n):
        masked = tx.clone()
        masked[:, j + 1:] = -1
        prefix.append(forward(family, th, tW, tR, tT, masked))
    slot = []
    total = 0.0
    for j in range(n):
        cond = prefix[j] - (prefix[j - 1] if j > 0 else 0.0)
        acc = 0.0
        for i in range(N):
            rows = slice(i * L, (i + 1) * L)
            valid = tx[rows, j] >= 0
            V = int(valid.sum())
            if V:
                acc = acc + cond[rows][valid].sum() / V
        Lj = -acc / N
        slot.append(Lj)
        total = total + gamma ** j * Lj
    total.backward()
    zero = lambda t: np.zeros(tuple(t.shape)) if t.grad is None else t.grad.numpy()
    return dict(slot_loss=np.array([float(s.detach()) for s in slot]), loss=float(total.detach()), dh=zero(th), dW_emit=zero(tW),
                dW_sum=zero(tR), dT_static=None if tT is None else zero(tT))


def lowrank_grad(W_base, A, B, dU):
    """App. G, U[i, j] = W_base[i] + A[i, j] B[i, j]: given the gradient dU [n, r, v, d] of a scalar with respect to
    the composed unembeddings, its gradient with respect to W_base [n, v, d], A [n, r, v, k] and B [n, r, k, d], by reverse
    mode through the definition. Returns dict(U, dW_base, dA, dB), numpy float64."""
    tW = torch.tensor(np.asarray(W_base, dtype=np.float64), requires_grad=True)
    tA = torch.tensor(np.asarray(A, dtype=np.float64), requires_grad=True)
    tB = torch.tensor(np.asarray(B, dtype=np.float64), requires_grad=True)
    U = tW[:, None, :, :] + torch.matmul(tA, tB)
    (U * torch.tensor(np.asarray(dU, dtype=np.float64))).sum().backward()
    return dict(U=U.detach().numpy(), dW_base=tW.grad.numpy(), dA=tA.grad.numpy(), dB=tB.grad.numpy())
