"""Pins for the gradient oracle (oracle/mtpc_oracle_grad.py). Its torch forward is compared with the numpy oracle's
forward (two transcriptions of the definition), and every gradient with central finite differences of the NUMPY
oracle's log-likelihood - a route with no automatic differentiation in it - plus closed forms."""
import numpy as np
import pytest
import scipy.special
import torch

from oracle import mtpc_oracle as orc
from oracle import mtpc_oracle_grad as og

CP, HMM, BTREE, HMM_CTX = orc.CP, orc.HMM, orc.BTREE, orc.HMM_CTX


def tiny(rng, family, n, r, v, d=4, T=3):
    S = orc.num_sum_units(family, n, r)
    h = rng.normal(size=(T, d))
    W = rng.normal(size=(n, r, v, d))
    R = rng.normal(size=(S * r, d))
    Ts = rng.normal(size=(n - 1, r, r)) if family in (HMM, HMM_CTX) else None
    x = rng.integers(0, v, size=(T, n))
    wt = rng.normal(size=T)
    return h, W, R, Ts, x, wt


CASES = [(CP, 3, 3, 4), (CP, 2, 1, 3), (HMM, 3, 2, 3), (HMM, 4, 3, 2), (HMM_CTX, 3, 2, 3), (BTREE, 4, 2, 3), (BTREE, 2, 3, 3),
         (BTREE, 8, 2, 2)]


@pytest.mark.parametrize("family,n,r,v", CASES)
def test_torch_forward_equals_numpy_forward(family, n, r, v):
    rng = np.random.default_rng(900 + 10 * family + n)
    h, W, R, Ts, x, wt = tiny(rng, family, n, r, v)
    x[0, n - 1] = -1                                          # a marginalised byte
    got = og.window_logprob_grad(family, h, W, R, Ts, x, wt)["logprob"]
    np.testing.assert_allclose(got, orc.window_logprob(family, h, W, R, Ts, x), atol=1e-12)


def loss_numpy(family, h, W, R, Ts, x, wt):
    return float((orc.window_logprob(family, h, W, R, Ts, x) * wt).sum())


def finite_difference(fn, arr, eps=1e-6, sample=None, rng=None):
    """Central differences of fn() with respect to entries of `arr` (modified in place and restored)."""
    flat = arr.reshape(-1)
    idx = np.arange(flat.size) if sample is None or flat.size <= sample else rng.choice(flat.size, sample, replace=False)
    out = np.zeros(len(idx))
    for q, e in enumerate(idx):
        keep = flat[e]
        flat[e] = keep + eps
        up = fn()
        flat[e] = keep - eps
        dn = fn()
        flat[e] = keep
        out[q] = (up - dn) / (2 * eps)
    return idx, out


@pytest.mark.parametrize("family,n,r,v", CASES)
def test_gradients_equal_finite_differences_of_the_numpy_oracle(family, n, r, v):
    rng = np.random.default_rng(910 + 10 * family + n)
    h, W, R, Ts, x, wt = tiny(rng, family, n, r, v)
    x[1, 0] = -1
    g = og.window_logprob_grad(family, h, W, R, Ts, x, wt)
    fn = lambda: loss_numpy(family, h, W, R, Ts, x, wt)
    for name, arr in (("dh", h), ("dW_emit", W), ("dW_sum", R), ("dT_static", Ts)):
        if arr is None:
            assert g[name] is None
            continue
        idx, fd = finite_difference(fn, arr, sample=60, rng=rng)
        np.testing.assert_allclose(g[name].reshape(-1)[idx], fd, atol=2e-7, err_msg=name)
        assert np.abs(fd).max() > 1e-4 or (name == "dW_sum" and r == 1)   # not vacuous (one unit: softmax of one logit)


def test_rank_one_mixture_has_the_softmax_gradient():
    # CP with r = 1 is fully factorised: d log q / d logit[i, b] = onehot(x_i) - softmax(logit[i]); with W = identity
    # blocks the logits are the hidden state itself, so dh is that expression laid out along d.
    n, v = 3, 4
    d = n * v
    W = np.eye(d).reshape(n, 1, v, d)
    R = np.zeros((1, d))
    rng = np.random.default_rng(5)
    h = rng.normal(size=(2, d))
    x = np.array([[1, 3, 0], [2, -1, 2]])
    wt = np.array([0.5, -2.0])
    g = og.window_logprob_grad(CP, h, W, R, None, x, wt)
    want = np.zeros((2, n, v))
    for t in range(2):
        for i in range(n):
            if x[t, i] >= 0:
                want[t, i] = -scipy.special.softmax(h[t].reshape(n, v)[i])
                want[t, i, x[t, i]] += 1.0
    np.testing.assert_allclose(g["dh"], (want * wt[:, None, None]).reshape(2, d), atol=1e-12)
    assert np.abs(g["dh"].reshape(2, n, v)[1, 1]).max() == 0   # the marginalised byte


@pytest.mark.parametrize("family,n,r,v", [(CP, 3, 3, 4), (HMM_CTX, 3, 2, 3), (BTREE, 4, 2, 3)])
def test_sum_unit_logit_gradients_sum_to_zero_per_unit(family, n, r, v):
    # softmax is shift-invariant: adding a constant to the r logits of one sum unit changes nothing, so the gradient
    # with respect to those logits sums to zero. With d = S r and W_sum = identity the logits are the hidden state.
    S = orc.num_sum_units(family, n, r)
    d = S * r + 1
    rng = np.random.default_rng(920 + family)
    W = np.zeros((n, r, v, d))
    W[..., d - 1] = rng.normal(size=(n, r, v))                 # the emissions see the last hidden column only
    R = np.concatenate([np.eye(S * r), np.zeros((S * r, 1))], axis=1)
    h = rng.normal(size=(2, d))
    x = rng.integers(0, v, size=(2, n))
    g = og.window_logprob_grad(family, h, W, R, None, x, np.array([1.0, -0.7]))
    dlogit = g["dh"][:, :S * r].reshape(2, S, r)               # = d loss / d (sum-unit logits)
    assert np.abs(dlogit).max() > 1e-3
    assert np.abs(dlogit.sum(axis=-1)).max() < 1e-12


# ------------------------------------------------------------------ Eq. (6) and its gradient
def loss6_numpy(family, h, W, R, Ts, x, N, gamma):
    pre = orc.window_prefix_logprob(family, h, W, R, Ts, x)
    return orc.composite_loss(pre, x, N, gamma)


@pytest.mark.parametrize("family,n,r,v", [(CP, 3, 3, 4), (HMM, 3, 2, 3), (HMM_CTX, 3, 2, 3), (BTREE, 4, 2, 3)])
def test_eq6_loss_and_gradient_against_the_numpy_oracle(family, n, r, v):
    rng = np.random.default_rng(950 + family)
    N, L = 2, 4
    h, W, R, Ts, x, _ = tiny(rng, family, n, r, v, T=N * L)
    for j in range(1, n):                                     # windows running past the end of their sequence
        x.reshape(N, L, n)[:, L - j:, j] = -1
    x[0, 0] = -1                                              # and a hole at the front of one window
    gamma = 0.8
    g = og.composite_loss_grad(family, h, W, R, Ts, x, N, gamma)
    slot, total = loss6_numpy(family, h, W, R, Ts, x, N, gamma)
    np.testing.assert_allclose(g["slot_loss"], slot, atol=1e-12)
    assert abs(g["loss"] - total) < 1e-12
    fn = lambda: loss6_numpy(family, h, W, R, Ts, x, N, gamma)[1]
    for name, arr in (("dh", h), ("dW_emit", W), ("dW_sum", R), ("dT_static", Ts)):
        if arr is None:
            continue
        idx, fd = finite_difference(fn, arr, sample=40, rng=rng)
        np.testing.assert_allclose(g[name].reshape(-1)[idx], fd, atol=2e-7, err_msg=name)
        assert np.abs(fd).max() > 1e-4


@pytest.mark.parametrize("family", [CP, HMM, BTREE])
def test_undiscounted_eq6_gradient_is_the_mean_nll_gradient(family):
    rng = np.random.default_rng(960 + family)
    n, r, v, N, L = 4, 2, 3, 2, 3
    h, W, R, Ts, x, _ = tiny(rng, family, n, r, v, T=N * L)
    g6 = og.composite_loss_grad(family, h, W, R, Ts, x, N, 1.0)
    gj = og.window_logprob_grad(family, h, W, R, Ts, x, np.full(N * L, -1.0 / (N * L)))
    for name in ("dh", "dW_emit", "dW_sum"):
        np.testing.assert_allclose(g6[name], gj[name], atol=1e-12)


@pytest.mark.parametrize("family,n,r,v", CASES)
def test_logit_gradients_chain_to_the_parameter_gradients(family, n, r, v):
    """window_logprob_logit_grad: pushed through the two projections by hand (dW = dlogit^T h, dh = dlogit W + dslog R), the
    gradients with respect to the logits must give the parameter gradients that finite differences already pin; and
    for a rank-one mixture they have the closed form weight * (onehot - softmax)."""
    rng = np.random.default_rng(1700 + 10 * family + n)
    h, W, R, Ts, x, wt = tiny(rng, family, n, r, v)
    x[1, 0] = -1
    full = og.window_logprob_grad(family, h, W, R, Ts, x, wt)
    lg = og.window_logprob_logit_grad(family, h, W, R, Ts, x, wt)
    T, d = h.shape
    dl = lg["dlogit"].reshape(T, n * r * v)
    ds = lg["dslog"].reshape(T, -1)
    np.testing.assert_allclose(dl.T @ h, full["dW_emit"].reshape(n * r * v, d), atol=1e-12)
    np.testing.assert_allclose(ds.T @ h, full["dW_sum"], atol=1e-12)
    np.testing.assert_allclose(dl @ W.reshape(n * r * v, d) + ds @ R, full["dh"], atol=1e-12)
    assert np.abs(lg["dlogit"][1, 0]).max() == 0.0            # the marginalised byte: no gradient into its logits
    if family == CP and r == 1:
        logits = np.einsum("td,nvd->tnv", h, W[:, 0])
        soft = scipy.special.softmax(logits, axis=-1)
        onehot = np.zeros_like(soft)
        for t in range(T):
            for i in range(n):
                if x[t, i] >= 0:
                    onehot[t, i, x[t, i]] = 1.0
        want = wt[:, None, None] * (onehot - soft) * (x >= 0)[:, :, None]
        np.testing.assert_allclose(lg["dlogit"][:, :, 0, :], want, atol=1e-12)
