"""Pins for the fp64 oracle: it is checked against what the paper and the mathematics fix, never against
itself and never against the CUDA path. Enumerations below are literal transcriptions of the defining sums
(Eq. CP, Eq. HMM, Eq. BTree) in the probability domain with explicit loops."""
import itertools
import math
import os

import numpy as np
import pytest
import scipy.special
import scipy.stats

from oracle import mtpc_oracle as orc

CP, HMM, BTREE = orc.CP, orc.HMM, orc.BTREE
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ helpers (test-local, probability domain)
def rand_simplex(rng, *shape):
    x = rng.gamma(0.7, size=shape) + 1e-3
    return x / x.sum(axis=-1, keepdims=True)


def enum_cp(omega, phi, x):
    n = len(x)
    return sum(omega[z] * math.prod(phi[i][z][x[i]] for i in range(n)) for z in range(len(omega)))


def enum_hmm(pi, A, phi, x):
    n, r = len(x), len(pi)
    total = 0.0
    for zs in itertools.product(range(r), repeat=n):
        p = pi[zs[0]] * phi[0][zs[0]][x[0]]
        for i in range(1, n):
            p *= A[i - 1][zs[i - 1]][zs[i]] * phi[i][zs[i]][x[i]]
        total += p
    return total


def tree_structure(n):
    """Recursive halving: node j covers tokens [lo, hi); children 2j+1 (left half) and 2j+2 (right half);
    a half of one token is a layer of input units indexed by node j's latent. Returns (parent of each
    internal node, owner node of each token)."""
    parent, owner = {}, {}

    def build(j, lo, hi, par):
        parent[j] = par
        mid = lo + (hi - lo) // 2
        for c, (a, b) in ((2 * j + 1, (lo, mid)), (2 * j + 2, (mid, hi))):
            if b - a == 1:
                owner[a] = j
            else:
                build(c, a, b, j)

    build(0, 0, n, None)
    return parent, owner


def enum_btree(omega_root, Omega, phi, x):
    """Omega[j][a][b] = q(z_j = b | z_parent(j) = a)."""
    n, r = len(x), len(omega_root)
    parent, owner = tree_structure(n)
    nodes = sorted(parent)
    total = 0.0
    for zs in itertools.product(range(r), repeat=len(nodes)):
        z = dict(zip(nodes, zs))
        p = omega_root[z[0]]
        for j in nodes[1:]:
            p *= Omega[j][z[parent[j]]][z[j]]
        for i in range(n):
            p *= phi[i][z[owner[i]]][x[i]]
        total += p
    return total


def btree_logw(omega_root, Omega, n, r):
    """Pack root weights and per-node conditional tables into the [1 + (n-2) r, r] group layout."""
    logw = np.zeros((1 + (n - 2) * r, r))
    logw[0] = np.log(omega_root)
    for j in range(1, n - 1):
        logw[1 + (j - 1) * r: 1 + j * r] = np.log(Omega[j])
    return logw


# ------------------------------------------------------------------ softmax / head projections
def test_logsumexp_and_log_softmax_against_library():
    rng = np.random.default_rng(0)
    x = rng.normal(size=(5, 7, 11)) * 30
    np.testing.assert_allclose(orc.logsumexp(x, axis=1), scipy.special.logsumexp(x, axis=1), rtol=0, atol=1e-12)
    np.testing.assert_allclose(orc.log_softmax(x, axis=-1), scipy.special.log_softmax(x, axis=-1), atol=1e-12)
    np.testing.assert_allclose(np.exp(orc.log_softmax(x, axis=0)).sum(axis=0), 1.0, atol=1e-12)


def test_emission_hand_example():
    # one position, one slot, one unit, v = 3, d = 2: logits are (a, b, a + b) for h = (a, b)
    a, b = 0.5, -1.25
    W = np.array([[1.0, 0.0], [0.0, 1.0], [1.0, 1.0]]).reshape(1, 1, 3, 2)
    got = orc.emission_logphi(np.array([[a, b]]), W)[0, 0, 0]
    z = math.log(math.exp(a) + math.exp(b) + math.exp(a + b))
    np.testing.assert_allclose(got, [a - z, b - z, a + b - z], atol=1e-14)


def test_emission_closed_forms_and_index_order():
    rng = np.random.default_rng(1)
    T, n, r, v = 3, 2, 3, 5
    d = n * r * v
    # one-hot rows: logit[t, i, k, b] = h[t, (i*r + k)*v + b]  -> any transposed/misindexed operand shows up
    W = np.eye(d).reshape(n, r, v, d)
    h = rng.normal(size=(T, d))
    want = scipy.special.log_softmax(h.reshape(T, n, r, v), axis=-1)
    np.testing.assert_allclose(orc.emission_logphi(h, W), want, atol=1e-13)
    # zero hidden state -> uniform categoricals
    np.testing.assert_allclose(orc.emission_logphi(np.zeros((2, d)), rng.normal(size=(n, r, v, d))), -math.log(v), atol=1e-14)
    # v = 2 is a logistic: p(1) = sigmoid((w1 - w0) . h)
    W2 = rng.normal(size=(1, 1, 2, 4))
    h2 = rng.normal(size=(6, 4))
    s = h2 @ (W2[0, 0, 1] - W2[0, 0, 0])
    np.testing.assert_allclose(np.exp(orc.emission_logphi(h2, W2)[:, 0, 0, 1]), 1 / (1 + np.exp(-s)), atol=1e-14)


def test_sum_unit_groups_are_consecutive_rows():
    rng = np.random.default_rng(2)
    r, S, d = 3, 4, 12
    R = np.eye(d)                                   # logit[t, s, k] = h[t, s*r + k]
    h = rng.normal(size=(5, d))
    want = scipy.special.log_softmax(h.reshape(5, S, r), axis=-1)
    np.testing.assert_allclose(orc.sum_unit_logw(h, R, r), want, atol=1e-13)


def test_evidence_gathers_and_marginalises():
    rng = np.random.default_rng(3)
    logphi = np.log(rand_simplex(rng, 4, 3, 2, 5))
    x = np.array([[0, 4, 2], [1, -1, 3], [-1, -1, -1], [4, 4, 4]])
    g = orc.evidence(logphi, x)
    for t in range(4):
        for i in range(3):
            for k in range(2):
                assert g[t, i, k] == (0.0 if x[t, i] < 0 else logphi[t, i, k, x[t, i]])


# ------------------------------------------------------------------ circuit evaluation vs literal enumeration
@pytest.mark.parametrize("n,r,v", [(1, 3, 4), (3, 1, 4), (3, 3, 3), (4, 2, 3)])
def test_cp_equals_enumeration(n, r, v):
    rng = np.random.default_rng(10 + n)
    omega, phi = rand_simplex(rng, r), rand_simplex(rng, n, r, v)
    for x in itertools.product(range(v), repeat=n):
        g = orc.evidence(np.log(phi)[None], np.array([x]))
        got = orc.cp_eval(np.log(omega)[None], g)[0]
        assert abs(got - math.log(enum_cp(omega, phi, x))) < 1e-12


@pytest.mark.parametrize("n,r,v", [(1, 3, 4), (2, 2, 3), (3, 3, 3), (4, 2, 3), (5, 2, 2)])
def test_hmm_forward_equals_path_enumeration(n, r, v):
    rng = np.random.default_rng(20 + n)
    pi, A, phi = rand_simplex(rng, r), rand_simplex(rng, max(n - 1, 0), r, r), rand_simplex(rng, n, r, v)
    for x in itertools.product(range(v), repeat=n):
        g = orc.evidence(np.log(phi)[None], np.array([x]))
        got = orc.hmm_eval(np.log(pi)[None], np.log(A), g)[0]
        assert abs(got - math.log(enum_hmm(pi, A, phi, x))) < 1e-12


@pytest.mark.parametrize("n,r,v", [(2, 3, 3), (4, 2, 3), (4, 3, 2), (8, 2, 2)])
def test_btree_equals_latent_tree_enumeration(n, r, v):
    rng = np.random.default_rng(30 + n + r)
    omega_root = rand_simplex(rng, r)
    Omega = {j: rand_simplex(rng, r, r) for j in range(1, n - 1)}
    phi = rand_simplex(rng, n, r, v)
    logw = btree_logw(omega_root, Omega, n, r)[None]
    strings = list(itertools.product(range(v), repeat=n))
    if len(strings) > 40:
        strings = [strings[i] for i in np.random.default_rng(0).choice(len(strings), 40, replace=False)]
    for x in strings:
        g = orc.evidence(np.log(phi)[None], np.array([x]))
        got = orc.btree_eval(logw, g)[0]
        assert abs(got - math.log(enum_btree(omega_root, Omega, phi, x))) < 1e-12


def test_btree_rejects_non_power_of_two():
    with pytest.raises(ValueError):
        orc.btree_eval(np.zeros((1, 1 + 4 * 2, 2)), np.zeros((1, 6, 2)))


# ------------------------------------------------------------------ reductions between families
def test_cp_rank_one_is_fully_factorised():
    rng = np.random.default_rng(40)
    T, n, v, d = 6, 5, 7, 9
    h, W, R = rng.normal(size=(T, d)), rng.normal(size=(n, 1, v, d)), rng.normal(size=(1, d))
    x = rng.integers(0, v, size=(T, n))
    got = orc.window_logprob(CP, h, W, R, None, x)
    want = np.zeros(T)
    for t in range(T):
        for i in range(n):
            want[t] += scipy.special.log_softmax(W[i, 0] @ h[t])[x[t, i]]
    np.testing.assert_allclose(got, want, atol=1e-12)


def test_hmm_with_identity_transitions_is_cp():
    rng = np.random.default_rng(41)
    T, n, r, v, d = 5, 4, 3, 6, 8
    h, W, R = rng.normal(size=(T, d)), rng.normal(size=(n, r, v, d)), rng.normal(size=(r, d))
    x = rng.integers(0, v, size=(T, n))
    ident = np.where(np.eye(r, dtype=bool), 0.0, -1e5)[None].repeat(n - 1, axis=0)   # softmax -> I exactly in fp64
    np.testing.assert_allclose(orc.window_logprob(HMM, h, W, R, ident, x),
                               orc.window_logprob(CP, h, W, R, None, x), atol=1e-12)


def test_hmm_single_step_is_a_mixture():
    rng = np.random.default_rng(42)
    h, W, R = rng.normal(size=(4, 5)), rng.normal(size=(1, 3, 6, 5)), rng.normal(size=(3, 5))
    x = rng.integers(0, 6, size=(4, 1))
    np.testing.assert_allclose(orc.window_logprob(HMM, h, W, R, np.zeros((0, 3, 3)), x),
                               orc.window_logprob(CP, h, W, R, None, x), atol=1e-12)


def test_btree_two_tokens_is_cp_and_identity_tables_are_cp():
    rng = np.random.default_rng(43)
    T, r, v, d = 4, 3, 5, 7
    h = rng.normal(size=(T, d))
    W2, R2 = rng.normal(size=(2, r, v, d)), rng.normal(size=(r, d))
    x2 = rng.integers(0, v, size=(T, 2))
    np.testing.assert_allclose(orc.window_logprob(BTREE, h, W2, R2, None, x2),
                               orc.window_logprob(CP, h, W2, R2, None, x2), atol=1e-12)
    # n = 4 with every child latent forced equal to its parent's: one shared latent = CP
    n = 4
    phi, omega = rand_simplex(rng, n, r, v), rand_simplex(rng, r)
    with np.errstate(divide="ignore"):
        logw = btree_logw(omega, {j: np.eye(r) for j in range(1, n - 1)}, n, r)[None]
    for x in [(0, 1, 2, 3), (4, 4, 0, 1)]:
        g = orc.evidence(np.log(phi)[None], np.array([x]))
        assert abs(orc.btree_eval(logw, g)[0] - math.log(enum_cp(omega, phi, x))) < 1e-12


# ------------------------------------------------------------------ normalisation and marginals, whole path
def _tiny_head(rng, family, n, r, v, d=5):
    S = orc.num_sum_units(family, n, r)
    W, R = rng.normal(size=(n, r, v, d)), rng.normal(size=(S * r, d))
    Ts = rng.normal(size=(n - 1, r, r)) if family == HMM else None
    return W, R, Ts


@pytest.mark.parametrize("family,n,r,v", [(CP, 4, 3, 3), (CP, 3, 1, 4), (CP, 2, 2, 5), (HMM, 4, 3, 3), (HMM, 3, 2, 4),
                                           (BTREE, 4, 3, 3), (BTREE, 2, 2, 5), (BTREE, 8, 2, 2)])
def test_window_probabilities_sum_to_one(family, n, r, v):
    rng = np.random.default_rng(50 + family + n)
    W, R, Ts = _tiny_head(rng, family, n, r, v)
    h = rng.normal(size=(1, 5))
    xs = np.array(list(itertools.product(range(v), repeat=n)))
    lp = orc.window_logprob(family, np.repeat(h, len(xs), axis=0), W, R, Ts, xs)
    assert abs(np.exp(lp).sum() - 1.0) < 1e-12


@pytest.mark.parametrize("family", [CP, HMM, BTREE])
def test_negative_target_sums_the_byte_out(family):
    rng = np.random.default_rng(60 + family)
    n, r, v = 4, 3, 3
    W, R, Ts = _tiny_head(rng, family, n, r, v)
    h = rng.normal(size=(1, 5))
    for masked in [(1,), (0, 3), (0, 1, 2, 3)]:
        x = np.array([2, 0, 1, 2])
        x[list(masked)] = -1
        got = orc.window_logprob(family, h, W, R, Ts, x[None])[0]
        total = 0.0
        for fill in itertools.product(range(v), repeat=len(masked)):
            y = x.copy()
            y[list(masked)] = fill
            total += math.exp(orc.window_logprob(family, h, W, R, Ts, y[None])[0])
        assert abs(got - math.log(total)) < 1e-12
    # everything marginalised: the partition function of a normalised circuit is 1


# ------------------------------------------------------------------ sampling
def test_inverse_cdf_rule():
    logp = np.log(np.array([[0.25, 0.5, 0.25]] * 6))
    u = np.array([0.0, 0.2499, 0.25, 0.7499, 0.75, 0.999999])
    idx, margin = orc.inv_cdf(logp, u)
    assert idx.tolist() == [0, 0, 1, 1, 2, 2]
    np.testing.assert_allclose(margin, [0.25, 0.0001, 0.0, 0.0001, 0.0, 0.249999], atol=1e-12)
    # rounding leaves no index: fall back to the last one
    idx, _ = orc.inv_cdf(np.log(np.array([[0.5, 0.4999999]])), np.array([0.99999999]))
    assert idx.tolist() == [1]


@pytest.mark.parametrize("family,n,r,v", [(CP, 3, 3, 3), (HMM, 3, 3, 3), (BTREE, 4, 3, 2)])
def test_sampled_windows_follow_the_exact_joint(family, n, r, v):
    rng = np.random.default_rng(70 + family)
    W, R, Ts = _tiny_head(rng, family, n, r, v)
    W *= 1.5
    h = rng.normal(size=(1, 5))
    draws = 200_000
    u = np.random.default_rng(7).random(size=(draws, 2 * n))
    out = orc.draft_sample(family, h, W, R, Ts, draws, u)
    xs = np.array(list(itertools.product(range(v), repeat=n)))
    exact = np.exp(orc.window_logprob(family, np.repeat(h, len(xs), axis=0), W, R, Ts, xs))
    codes = (out["bytes"] * (v ** np.arange(n - 1, -1, -1))).sum(axis=1)
    counts = np.bincount(codes, minlength=len(xs))
    assert scipy.stats.chisquare(counts, exact * draws).pvalue > 1e-3
    # draft log-prob is the joint marginal of the drafted string
    np.testing.assert_allclose(out["logprob"], np.log(exact)[codes], atol=1e-12)
    # first latent follows the root / initial / mixture weights
    if family != BTREE:         # (token 0 of a tree hangs under a deeper latent, not under the root's)
        omega = np.exp(orc.sum_unit_logw(h, R, r))[0, 0]
        first_unit = out["unit"][:, 0]
        assert scipy.stats.chisquare(np.bincount(first_unit, minlength=r), omega * draws).pvalue > 1e-3


def test_hmm_sampler_uses_row_of_previous_state():
    # deterministic chain 0 -> 1 -> 2 -> 0 ...: a transposed transition table would walk it backwards
    r, n = 3, 4
    Ts = np.full((n - 1, r, r), -1e5)
    for a in range(r):
        Ts[:, a, (a + 1) % r] = 0.0
    logw = np.log(np.array([[[1.0 - 2e-9, 1e-9, 1e-9]]]))
    unit, _ = orc.sample_latents(HMM, logw, Ts, 1, np.full((1, 2 * n), 0.5), n)
    assert unit.tolist() == [[0, 1, 2, 0]]


def test_btree_sampler_token_owners():
    # child latents copy the parent's (identity tables): every token must use the root's draw
    n, r = 8, 3
    with np.errstate(divide="ignore"):
        logw = btree_logw(np.array([0.2, 0.5, 0.3]), {j: np.eye(r) for j in range(1, n - 1)}, n, r)[None]
    unit, _ = orc.sample_latents(BTREE, logw, None, 3, np.array([[0.1] * 16, [0.5] * 16, [0.9] * 16]), n)
    assert unit.tolist() == [[0] * 8, [1] * 8, [2] * 8]
    # distinct deterministic tables: node j sends parent value a to (a + j) mod r
    Omega = {}
    for j in range(1, n - 1):
        t = np.zeros((r, r))
        for a in range(r):
            t[a, (a + j) % r] = 1.0
        Omega[j] = t
    with np.errstate(divide="ignore"):
        logw = btree_logw(np.array([1.0, 0.0, 0.0]), Omega, n, r)[None]
    unit, _ = orc.sample_latents(BTREE, logw, None, 1, np.full((1, 16), 0.5), n)
    parent, owner = tree_structure(n)
    z = {0: 0}
    for j in range(1, n - 1):
        z[j] = (z[parent[j]] + j) % r
    assert unit[0].tolist() == [z[owner[i]] for i in range(n)]


# ------------------------------------------------------------------ structure counts printed by the paper
def test_counts_reproduce_the_complexity_table():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "table3_counts.txt")) if l.strip() and not l.startswith("#")]
    assert len(rows) == 8
    for n, fam, flops, params, gflops, mparams in rows:
        c = orc.circuit_counts(fam, int(n), 32, 320, 4096)
        assert c["circuit_params"] == int(params), (fam, n)
        if fam in ("hmm", "btree"):
            assert abs(c["circuit_flops"] - int(flops)) <= 50, (fam, n)       # printed as x.y K
        else:
            assert abs(c["circuit_flops"] - int(flops)) <= 1, (fam, n)        # the table prints 2r + 1 for CP
        assert abs(c["head_params"] / 1e6 - float(mparams)) <= 0.51, (fam, n)
        assert abs(c["head_flops"] / 1e9 - float(gflops)) <= 0.0051, (fam, n)
