"""Pins for the oracle's prefix marginals and acceptance stage (Algorithm 3). Nothing here compares the oracle with
itself or with the CUDA path: prefix marginals are checked against explicit sums of the joint over the later bytes,
the conditional against the chain rule, the acceptance stage against an example worked by hand from the algorithm's
formulas, and its output against the theorem the algorithm rests on - the emitted bytes follow the TARGET model's
distribution whatever the draft distribution is."""
import itertools
import math

import numpy as np
import pytest
import scipy.stats

from oracle import mtpc_oracle as orc

CP, HMM, BTREE = orc.CP, orc.HMM, orc.BTREE


def _tiny_head(rng, family, n, r, v, d=5):
    S = orc.num_sum_units(family, n, r)
    W, R = rng.normal(size=(n, r, v, d)), rng.normal(size=(S * r, d))
    Ts = rng.normal(size=(n - 1, r, r)) if family == HMM else None
    return W, R, Ts


def _all_strings(v, n):
    return np.array(list(itertools.product(range(v), repeat=n)))


@pytest.mark.parametrize("family,n,r,v", [(CP, 3, 3, 3), (CP, 4, 1, 2), (HMM, 4, 2, 3), (HMM, 3, 3, 2), (BTREE, 4, 3, 3),
                                           (BTREE, 8, 2, 2), (BTREE, 2, 3, 4)])
def test_prefix_marginals_equal_sums_of_the_joint_over_later_bytes(family, n, r, v):
    rng = np.random.default_rng(300 + 10 * family + n)
    W, R, Ts = _tiny_head(rng, family, n, r, v)
    h = rng.normal(size=(1, 5))
    xs = _all_strings(v, n)
    joint = np.exp(orc.window_logprob(family, np.repeat(h, len(xs), axis=0), W, R, Ts, xs))
    table = joint.reshape((v,) * n)
    some = xs[rng.choice(len(xs), size=min(len(xs), 12), replace=False)]
    got = orc.window_prefix_logprob(family, np.repeat(h, len(some), axis=0), W, R, Ts, some)
    assert got.shape == (len(some), n)
    for row, x in zip(got, some):
        for i in range(n):
            want = table[tuple(x[:i + 1])].sum()          # explicit sum over x_{i+2}..x_n
            assert abs(row[i] - math.log(want)) < 1e-12
        assert abs(row[n - 1] - math.log(table[tuple(x)])) < 1e-12
        assert (np.diff(row) <= 1e-15).all()             # a longer prefix is never more probable


@pytest.mark.parametrize("family,n,r,v", [(CP, 3, 2, 4), (HMM, 3, 3, 3), (BTREE, 4, 2, 3)])
def test_next_byte_conditional_is_normalised_and_chains_to_the_joint(family, n, r, v):
    rng = np.random.default_rng(400 + family)
    W, R, Ts = _tiny_head(rng, family, n, r, v)
    h = rng.normal(size=(2, 5))
    logphi = orc.emission_logphi(h, W)
    logw = orc.sum_unit_logw(h, R, r)
    x = rng.integers(0, v, size=(2, n))
    joint = orc.window_logprob(family, h, W, R, Ts, x)
    chain = np.zeros(2)
    xs = _all_strings(v, n)
    for s in range(n):
        cond = orc.next_byte_logprob(family, logw, logphi, Ts, x, np.full(2, s))
        assert cond.shape == (2, v)
        np.testing.assert_allclose(np.exp(cond).sum(axis=-1), 1.0, atol=1e-12)
        chain += cond[np.arange(2), x[:, s]]
        # against the explicit ratio of sums of the joint, first position only
        table = np.exp(orc.window_logprob(family, np.repeat(h[:1], len(xs), axis=0), W, R, Ts, xs)).reshape((v,) * n)
        sub = table[tuple(x[0, :s])] if s else table
        want = sub.reshape(v, -1).sum(axis=1) / sub.sum()
        np.testing.assert_allclose(np.exp(cond[0]), want, atol=1e-12)
    np.testing.assert_allclose(chain, joint, atol=1e-12)
    # windows may sit at different prefix lengths in one call
    mixed = orc.next_byte_logprob(family, logw, logphi, Ts, x, np.array([0, n - 1]))
    np.testing.assert_allclose(mixed[0], orc.next_byte_logprob(family, logw, logphi, Ts, x, np.array([0, 0]))[0])
    np.testing.assert_allclose(mixed[1], orc.next_byte_logprob(family, logw, logphi, Ts, x, np.array([n - 1] * 2))[1])


def _never(rows, s):
    raise AssertionError("no byte was rejected: the draft's conditional must not be needed")


def test_acceptance_example_worked_by_hand():
    """n = 2, v = 3. Draft x = (1, 2) with q(x_1 = 1) = 0.7 and q(x_1 = 1, x_2 = 2) = 0.7 * 0.5.
    Target p(X_1) = (0.5, 0.3, 0.2), p(X_2 | 1) = (0.1, 0.3, 0.6), p(X_3 | 1, 2) = (0.2, 0.2, 0.6)."""
    x = np.array([[1, 2]])
    prefix = np.log(np.array([[0.7, 0.35]]))
    p = np.array([[[0.5, 0.3, 0.2], [0.1, 0.3, 0.6], [0.2, 0.2, 0.6]]])
    q_first = np.log(np.array([[0.2, 0.7, 0.1]]))        # q(X_1)
    q_second = np.log(np.array([[0.25, 0.25, 0.5]]))     # q(X_2 | x_1 = 1)

    # byte 1: ratio 0.3 / 0.7 = 0.4286. alpha = 0.5 rejects it. Residual max(0, p - q) = (0.3, 0, 0.1) / 0.4 =
    # (0.75, 0, 0.25); u = 0.8 falls in the last cell, u = 0.7 in the first.
    for u_last, want in [(0.8, 2), (0.7, 0), (0.75, 2)]:
        out = orc.speculative_accept(prefix, x, p, np.array([[0.5, 0.0, u_last]]), lambda rows, s: q_first)
        assert out["accepted"].tolist() == [0] and out["next_byte"].tolist() == [want]
    # alpha = 0.4 accepts byte 1. Byte 2: q(x_2 | x_1) = 0.35 / 0.7 = 0.5, ratio 0.6 / 0.5 = 1.2: always accepted.
    # All n accepted: the extra byte comes from p(X_3 | 1, 2) = (0.2, 0.2, 0.6): u = 0.39 -> 1.
    out = orc.speculative_accept(prefix, x, p, np.array([[0.4, 0.999, 0.39]]), _never)
    assert out["accepted"].tolist() == [2] and out["next_byte"].tolist() == [1]
    out = orc.speculative_accept(prefix, x, p, np.array([[0.4, 0.999, 0.15]]), _never)   # p(X_2 | 1) would give 1
    assert out["accepted"].tolist() == [2] and out["next_byte"].tolist() == [0]
    # a draft whose second byte is over-confident: x = (1, 0): q(0 | 1) = 0.25, p = 0.1, ratio 0.4; alpha 0.41 rejects.
    # Residual max(0, (0.1, 0.3, 0.6) - (0.25, 0.25, 0.5)) = (0, 0.05, 0.1) / 0.15 = (0, 1/3, 2/3).
    x2 = np.array([[1, 0]])
    prefix2 = np.log(np.array([[0.7, 0.7 * 0.25]]))
    seen = {}

    def cond(rows, s):
        seen["s"] = s.tolist()
        return q_second

    out = orc.speculative_accept(prefix2, x2, p, np.array([[0.1, 0.41, 0.3]]), cond)
    assert out["accepted"].tolist() == [1] and out["next_byte"].tolist() == [1] and seen["s"] == [1]
    out = orc.speculative_accept(prefix2, x2, p, np.array([[0.1, 0.41, 0.34]]), cond)
    assert out["next_byte"].tolist() == [2]
    assert abs(out["margin"][0] - min(0.41 - 0.4, abs(1 / 3 - 0.34))) < 1e-12
    out = orc.speculative_accept(prefix2, x2, p, np.array([[0.1, 0.39, 0.34]]), _never)
    assert out["accepted"].tolist() == [2]


@pytest.mark.parametrize("family", [CP, HMM, BTREE])
def test_target_equal_to_draft_accepts_everything(family):
    rng = np.random.default_rng(500 + family)
    n, r, v = 4, 3, 4
    W, R, Ts = _tiny_head(rng, family, n, r, v)
    h = rng.normal(size=(3, 5))
    wpp = 5
    u = rng.random(size=(3 * wpp, 2 * n))
    d = orc.draft_sample(family, h, W, R, Ts, wpp, u)
    pos = np.repeat(np.arange(3), wpp)
    logphi, logw = orc.emission_logphi(h, W), orc.sum_unit_logw(h, R, r)
    prefix = orc.prefix_logprob(family, logw, logphi, Ts, d["bytes"], pos)
    np.testing.assert_allclose(prefix[:, -1], d["logprob"], atol=1e-12)
    p = np.zeros((3 * wpp, n + 1, v))
    for s in range(n):
        p[:, s, :] = np.exp(orc.next_byte_logprob(family, logw, logphi, Ts, d["bytes"], np.full(3 * wpp, s), pos))
    p[:, n, :] = np.array([0.1, 0.2, 0.3, 0.4])
    ua = rng.random(size=(3 * wpp, n + 1)) * 0.999
    out = orc.speculative_accept(prefix, d["bytes"], p, ua, _never)
    assert (out["accepted"] == n).all()
    want = (np.cumsum([0.1, 0.2, 0.3, 0.4])[None, :] <= ua[:, n:n + 1]).sum(axis=1)
    assert out["next_byte"].tolist() == want.tolist()


@pytest.mark.parametrize("family,n,r,v", [(CP, 2, 3, 3), (HMM, 2, 3, 3), (BTREE, 2, 2, 3), (HMM, 3, 2, 2)])
def test_emitted_bytes_follow_the_target_model(family, n, r, v):
    """Speculative sampling is exact: the bytes a cycle emits are distributed as the autoregressive target model
    would have produced them, for ANY draft distribution. Target: random tables p(X_1), p(X_2 | x_1), ...; draft:
    a random tiny head. Chi-squared on byte 1, on byte 2 given byte 1, and on the byte after a fully accepted window."""
    rng = np.random.default_rng(600 + 7 * family + n)
    W, R, Ts = _tiny_head(rng, family, n, r, v)
    h = rng.normal(size=(1, 5))
    draws = 150_000
    u = np.random.default_rng(11).random(size=(draws, 2 * n))
    d = orc.draft_sample(family, h, W, R, Ts, draws, u)
    x = d["bytes"]
    pos = np.zeros(draws, dtype=np.int64)
    logphi, logw = orc.emission_logphi(h, W), orc.sum_unit_logw(h, R, r)
    prefix = orc.prefix_logprob(family, logw, logphi, Ts, x, pos)
    # target model: table[i] has shape (v,)*i + (v,) and gives p(X_{i+1} | first i bytes)
    tables = []
    for i in range(n + 1):
        t = rng.gamma(0.8, size=(v,) * (i + 1)) + 0.02
        tables.append(t / t.sum(axis=-1, keepdims=True))
    p = np.zeros((draws, n + 1, v))
    for i in range(n + 1):
        p[:, i, :] = tables[i][tuple(x[:, j] for j in range(i))]
    ua = np.random.default_rng(12).random(size=(draws, n + 1))
    out = orc.speculative_accept(prefix, x, p, ua,
                                 lambda rows, s: orc.next_byte_logprob(family, logw, logphi, Ts, x[rows], s, pos[rows]))
    acc, nb = out["accepted"], out["next_byte"]
    assert acc.min() == 0 and acc.max() == n                    # the test exercises rejection and full acceptance
    emitted = np.concatenate([x, np.zeros((draws, 1), dtype=np.int64)], axis=1)
    emitted[np.arange(draws), acc] = nb                          # bytes 0..acc-1 are the draft's, byte acc is the extra one
    # byte 1
    c1 = np.bincount(emitted[:, 0], minlength=v)
    assert scipy.stats.chisquare(c1, tables[0] * draws).pvalue > 1e-3
    # byte i+1 given the bytes before it, over the cycles that emitted it
    for i in range(1, n + 1):
        have = acc >= i
        for ctx in itertools.product(range(v), repeat=i):
            sel = have & (emitted[:, :i] == np.array(ctx)).all(axis=1)
            if sel.sum() < 200:
                continue
            ci = np.bincount(emitted[sel, i], minlength=v)
            assert scipy.stats.chisquare(ci, tables[i][ctx] * sel.sum()).pvalue > 1e-4, (i, ctx)


def test_acceptance_uses_one_uniform_per_test_in_order():
    # q = p except on the second byte, where the ratio is 0.5: only column 1 of the uniforms can reject
    x = np.array([[0, 0, 0]])
    prefix = np.log(np.array([[0.5, 0.25, 0.125]]))
    p = np.full((1, 4, 2), 0.5)
    p[0, 1, 0] = 0.25
    p[0, 1, 1] = 0.75
    q_half = np.log(np.array([[0.5, 0.5]]))
    for u in ([0.9, 0.49, 0.9, 0.1], [0.0, 0.5, 0.0, 0.1]):
        out = orc.speculative_accept(prefix, x, p, np.array([u]), _never)
        assert out["accepted"].tolist() == [3]
    out = orc.speculative_accept(prefix, x, p, np.array([[0.1, 0.51, 0.1, 0.1]]), lambda rows, s: q_half)
    assert out["accepted"].tolist() == [1]
    # residual = max(0, (0.25, 0.75) - (0.5, 0.5)) = (0, 0.25) -> byte 1 whatever the uniform
    assert out["next_byte"].tolist() == [1]


# ------------------------------------------------------------------ Eq. (6)
def test_loss_example_worked_by_hand():
    """N = 2 sequences of L = 2 positions, n = 2. Conditionals (probabilities) per position and slot:
         seq 0: t0 (1/2, 1/4)  t1 (1/8, masked)      seq 1: t0 (1/2, 1/2)  t1 (masked, masked)
    L_1 = -(1/2) [ (ln 1/2 + ln 1/8) / 2 + (ln 1/2) / 1 ] = (1/2)(2 ln 2 + ln 2) = 1.5 ln 2
    L_2 = -(1/2) [ (ln 1/4) / 1 + (ln 1/2) / 1 ] = 1.5 ln 2;  L = L_1 + gamma L_2."""
    ln = math.log
    prefix = np.array([[ln(1 / 2), ln(1 / 8)], [ln(1 / 8), ln(1 / 8)], [ln(1 / 2), ln(1 / 4)], [0.0, 0.0]])
    targets = np.array([[3, 1], [0, -1], [2, 2], [-1, -1]])
    slot, total = orc.composite_loss(prefix, targets, 2, 0.8)
    np.testing.assert_allclose(slot, [1.5 * ln(2), 1.5 * ln(2)], atol=1e-12)
    assert abs(total - 1.5 * ln(2) * 1.8) < 1e-12
    # a sequence whose slot has no valid byte adds nothing, but still counts in N
    targets2 = targets.copy()
    targets2[2, 1] = -1
    slot2, _ = orc.composite_loss(prefix, targets2, 2, 0.8)
    assert abs(slot2[1] - ln(4) / 2) < 1e-12


@pytest.mark.parametrize("family", [CP, HMM, BTREE])
def test_undiscounted_loss_with_all_bytes_valid_is_the_mean_joint_nll(family):
    rng = np.random.default_rng(700 + family)
    n, r, v, N, L = 4, 3, 5, 3, 6
    W, R, Ts = _tiny_head(rng, family, n, r, v)
    h = rng.normal(size=(N * L, 5))
    x = rng.integers(0, v, size=(N * L, n))
    prefix = orc.window_prefix_logprob(family, h, W, R, Ts, x)
    slot, total = orc.composite_loss(prefix, x, N, 1.0)
    joint = orc.window_logprob(family, h, W, R, Ts, x)
    assert abs(total + joint.mean()) < 1e-12            # sum_j L_j = -(1/(N L)) sum_t log q(window)
    # slot terms are per-slot means of conditionals; discounting weights them by gamma^j
    _, disc = orc.composite_loss(prefix, x, N, 0.5)
    assert abs(disc - sum(0.5 ** j * slot[j] for j in range(n))) < 1e-12
    # masking the tail of a window leaves the earlier slots' terms unchanged
    xm = x.copy()
    xm[L - 1, 2:] = -1
    pm = orc.window_prefix_logprob(family, h, W, R, Ts, xm)
    slot_m, _ = orc.composite_loss(pm, xm, N, 1.0)
    np.testing.assert_allclose(slot_m[:2], slot[:2], atol=1e-12)
    assert abs(slot_m[2] - slot[2]) > 1e-6
