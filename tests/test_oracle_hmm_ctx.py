"""Pins for the oracle's contextual HMM (App. H: transitions produced from the hidden state, plus a bias). Checked
against literal path enumeration with each position's own tables, against the static HMM and the mixture it reduces
to, by brute-force normalisation and by the sampler's frequencies - never against itself."""
import itertools
import math

import numpy as np
import pytest
import scipy.special
import scipy.stats

from oracle import mtpc_oracle as orc

CP, HMM, HMM_CTX = orc.CP, orc.HMM, orc.HMM_CTX


def head(rng, n, r, v, d=5, trans_scale=1.0):
    W = rng.normal(size=(n, r, v, d))
    R = rng.normal(size=((1 + (n - 1) * r) * r, d))
    R[r:] *= trans_scale
    bias = rng.normal(size=(n - 1, r, r))
    return W, R, bias


def enum_paths(pi, A, phi, x):
    n, r = len(x), len(pi)
    total = 0.0
    for zs in itertools.product(range(r), repeat=n):
        p = pi[zs[0]] * phi[0][zs[0]][x[0]]
        for i in range(1, n):
            p *= A[i - 1][zs[i - 1]][zs[i]] * phi[i][zs[i]][x[i]]
        total += p
    return total


@pytest.mark.parametrize("n,r,v", [(1, 3, 4), (2, 2, 3), (3, 3, 3), (4, 2, 3)])
def test_contextual_hmm_equals_path_enumeration_with_per_position_tables(n, r, v):
    rng = np.random.default_rng(800 + n)
    W, R, bias = head(rng, n, r, v)
    T = 3
    h = rng.normal(size=(T, 5))
    logits = h @ R.T
    for t in range(T):
        pi = scipy.special.softmax(logits[t, :r])
        A = scipy.special.softmax(logits[t, r:].reshape(n - 1, r, r) + bias, axis=-1) if n > 1 else None
        phi = scipy.special.softmax(np.einsum("nrvd,d->nrv", W, h[t]), axis=-1)
        for x in list(itertools.product(range(v), repeat=n))[::3]:
            got = orc.window_logprob(HMM_CTX, h[t:t + 1], W, R, bias, np.array([x]))[0]
            assert abs(got - math.log(enum_paths(pi, A, phi, x))) < 1e-12
    assert n == 1 or not np.allclose(logits[0, r:], logits[1, r:])   # the tables really differ between positions


def test_zero_transition_rows_reduce_to_the_static_hmm_and_identity_bias_to_cp():
    rng = np.random.default_rng(810)
    n, r, v = 4, 3, 4
    W, R, bias = head(rng, n, r, v, trans_scale=0.0)               # transitions come from the bias alone
    h = rng.normal(size=(5, 5))
    x = rng.integers(0, v, size=(5, n))
    np.testing.assert_allclose(orc.window_logprob(HMM_CTX, h, W, R, bias, x),
                               orc.window_logprob(HMM, h, W, R[:r], bias, x), atol=1e-12)
    ident = np.where(np.eye(r, dtype=bool), 0.0, -1e4)[None].repeat(n - 1, axis=0)
    np.testing.assert_allclose(orc.window_logprob(HMM_CTX, h, W, R, ident, x),
                               orc.window_logprob(CP, h, W, R[:r], None, x), atol=1e-12)
    # no bias at all is a zero bias
    W2, R2, _ = head(rng, n, r, v)
    np.testing.assert_allclose(orc.window_logprob(HMM_CTX, h, W2, R2, None, x),
                               orc.window_logprob(HMM_CTX, h, W2, R2, np.zeros((n - 1, r, r)), x), atol=1e-12)


@pytest.mark.parametrize("n,r,v", [(3, 3, 3), (4, 2, 3)])
def test_contextual_hmm_is_normalised_and_marginalises(n, r, v):
    rng = np.random.default_rng(820 + n)
    W, R, bias = head(rng, n, r, v)
    h = rng.normal(size=(1, 5))
    xs = np.array(list(itertools.product(range(v), repeat=n)))
    lp = orc.window_logprob(HMM_CTX, np.repeat(h, len(xs), axis=0), W, R, bias, xs)
    assert abs(np.exp(lp).sum() - 1.0) < 1e-12
    table = np.exp(lp).reshape((v,) * n)
    x = xs[len(xs) // 2]
    pre = orc.window_prefix_logprob(HMM_CTX, h, W, R, bias, x[None])[0]
    for i in range(n):
        assert abs(pre[i] - math.log(table[tuple(x[:i + 1])].sum())) < 1e-12


def test_contextual_hmm_sampler_follows_the_exact_joint_and_the_chain_direction():
    rng = np.random.default_rng(830)
    n, r, v = 3, 3, 3
    W, R, bias = head(rng, n, r, v)
    W *= 1.5
    h = rng.normal(size=(1, 5))
    draws = 200_000
    u = np.random.default_rng(9).random(size=(draws, 2 * n))
    out = orc.draft_sample(HMM_CTX, h, W, R, bias, draws, u)
    xs = np.array(list(itertools.product(range(v), repeat=n)))
    exact = np.exp(orc.window_logprob(HMM_CTX, np.repeat(h, len(xs), axis=0), W, R, bias, xs))
    codes = (out["bytes"] * (v ** np.arange(n - 1, -1, -1))).sum(axis=1)
    assert scipy.stats.chisquare(np.bincount(codes, minlength=len(xs)), exact * draws).pvalue > 1e-3
    np.testing.assert_allclose(out["logprob"], np.log(exact)[codes], atol=1e-12)
    # pairs of consecutive states follow pi[a] A_1[a, b]
    logits = (h @ R.T)[0]
    pi = scipy.special.softmax(logits[:r])
    A1 = scipy.special.softmax(logits[r:r + r * r].reshape(r, r) + bias[0], axis=-1)
    pair = np.bincount(out["unit"][:, 0] * r + out["unit"][:, 1], minlength=r * r)
    assert scipy.stats.chisquare(pair, (pi[:, None] * A1).reshape(-1) * draws).pvalue > 1e-3
    # deterministic chain through the bias: a transposed table would walk it backwards
    det = np.full((3, r, r), -1e5)
    for a in range(r):
        det[:, a, (a + 1) % r] = 0.0
    Rz = np.zeros(((1 + 3 * r) * r, 2))
    Rz[0, 0] = 50.0
    logw = orc.sum_unit_logw(np.array([[1.0, 0.0]]), Rz, r, bias=det)
    unit, _ = orc.sample_latents(HMM_CTX, logw, None, 1, np.full((1, 8), 0.5), 4)
    assert unit.tolist() == [[0, 1, 2, 0]]


def test_sum_unit_count_matches_the_complexity_table():
    # Table 3, HMM rows (r = 32, v = 320): 89,120 and 179,232 circuit parameters = n r v + (1 + (n-1) r) r
    assert 8 * 32 * 320 + orc.num_sum_units(HMM_CTX, 8, 32) * 32 == 89120
    assert 16 * 32 * 320 + orc.num_sum_units(HMM_CTX, 16, 32) * 32 == 179232
