"""The pins must be sharp: a plausible mistake planted in the oracle (a transposed table, a dropped term, a wrong
child or slot index, a non-strict comparison) has to break at least one of them. Each mutant is the oracle's
own source with one textual edit, executed as a throw-away module on the CPU; the pin is a literal enumeration
or a closed form from test_oracle_pins.py, never the oracle itself."""
import importlib.util
import itertools
import math
import os
import types

import numpy as np
import pytest

HERE = os.path.dirname(os.path.abspath(__file__))
ORACLE_SRC = os.path.join(os.path.dirname(HERE), "oracle", "mtpc_oracle.py")

_spec = importlib.util.spec_from_file_location("pins_for_mutants", os.path.join(HERE, "test_oracle_pins.py"))
pins = importlib.util.module_from_spec(_spec)
_spec.loader.exec_module(pins)


def mutant(old: str, new: str) -> types.ModuleType:
    src = open(ORACLE_SRC).read()
    assert src.count(old) == 1, f"mutation site not unique or missing: {old!r}"
    mod = types.ModuleType("oracle_mutant")
    exec(compile(src.replace(old, new), "oracle_mutant", "exec"), mod.__dict__)
    return mod


def cp_gap(orc):
    rng = np.random.default_rng(1)
    n, r, v = 3, 3, 3
    omega, phi = pins.rand_simplex(rng, r), pins.rand_simplex(rng, n, r, v)
    gap = 0.0
    for x in itertools.product(range(v), repeat=n):
        g = orc.evidence(np.log(phi)[None], np.array([x]))
        gap = max(gap, abs(orc.cp_eval(np.log(omega)[None], g)[0] - math.log(pins.enum_cp(omega, phi, x))))
    return gap


def hmm_gap(orc):
    rng = np.random.default_rng(2)
    n, r, v = 3, 3, 3
    pi, A, phi = pins.rand_simplex(rng, r), pins.rand_simplex(rng, n - 1, r, r), pins.rand_simplex(rng, n, r, v)
    gap = 0.0
    for x in itertools.product(range(v), repeat=n):
        g = orc.evidence(np.log(phi)[None], np.array([x]))
        gap = max(gap, abs(orc.hmm_eval(np.log(pi)[None], np.log(A), g)[0] - math.log(pins.enum_hmm(pi, A, phi, x))))
    return gap


def btree_gap(orc, n=8, r=2, v=2):
    rng = np.random.default_rng(3)
    omega_root = pins.rand_simplex(rng, r)
    Omega = {j: pins.rand_simplex(rng, r, r) for j in range(1, n - 1)}
    phi = pins.rand_simplex(rng, n, r, v)
    logw = pins.btree_logw(omega_root, Omega, n, r)[None]
    gap = 0.0
    for x in list(itertools.product(range(v), repeat=n))[::7]:
        g = orc.evidence(np.log(phi)[None], np.array([x]))
        gap = max(gap, abs(orc.btree_eval(logw, g)[0] - math.log(pins.enum_btree(omega_root, Omega, phi, x))))
    return gap


def emission_gap(orc):
    rng = np.random.default_rng(4)
    T, n, r, v = 3, 2, 3, 5
    d = n * r * v
    W = np.eye(d).reshape(n, r, v, d)
    h = rng.normal(size=(T, d))
    import scipy.special
    want = scipy.special.log_softmax(h.reshape(T, n, r, v), axis=-1)
    return float(np.abs(orc.emission_logphi(h, W) - want).max())


def inv_cdf_wrong(orc):
    idx, _ = orc.inv_cdf(np.log(np.array([[0.25, 0.5, 0.25]] * 3)), np.array([0.25, 0.75, 0.1]))
    return 0.0 if idx.tolist() == [1, 2, 0] else 1.0


def hmm_sampler_wrong(orc):
    r, n = 3, 4
    Ts = np.full((n - 1, r, r), -1e5)
    for a in range(r):
        Ts[:, a, (a + 1) % r] = 0.0
    logw = np.log(np.array([[[1.0 - 2e-9, 1e-9, 1e-9]]]))
    unit, _ = orc.sample_latents(orc.HMM, logw, Ts, 1, np.full((1, 2 * n), 0.5), n)
    return 0.0 if unit.tolist() == [[0, 1, 2, 0]] else 1.0


def btree_sampler_wrong(orc):
    n, r = 8, 3
    Omega = {}
    for j in range(1, n - 1):
        t = np.zeros((r, r))
        for a in range(r):
            t[a, (a + j) % r] = 1.0
        Omega[j] = t
    with np.errstate(divide="ignore"):
        logw = pins.btree_logw(np.array([1.0, 0.0, 0.0]), Omega, n, r)[None]
    unit, _ = orc.sample_latents(orc.BTREE, logw, None, 1, np.full((1, 16), 0.5), n)
    parent, owner = pins.tree_structure(n)
    z = {0: 0}
    for j in range(1, n - 1):
        z[j] = (z[parent[j]] + j) % r
    return 0.0 if unit[0].tolist() == [z[owner[i]] for i in range(n)] else 1.0


def masked_gap(orc):
    rng = np.random.default_rng(5)
    logphi = np.log(pins.rand_simplex(rng, 1, 2, 2, 3))
    g = orc.evidence(logphi, np.array([[-1, 2]]))
    return float(np.abs(g[0, 0]).max() + np.abs(g[0, 1] - logphi[0, 1, :, 2]).max())


def prefix_gap(orc):
    """Prefix marginals against explicit sums of the joint over the later bytes (tiny HMM)."""
    rng = np.random.default_rng(6)
    n, r, v = 3, 2, 3
    pi, A, phi = pins.rand_simplex(rng, r), pins.rand_simplex(rng, n - 1, r, r), pins.rand_simplex(rng, n, r, v)
    table = np.zeros((v,) * n)
    for x in itertools.product(range(v), repeat=n):
        table[x] = pins.enum_hmm(pi, A, phi, x)
    x = np.array([[2, 0, 1]])
    with np.errstate(divide="ignore"):
        got = orc.prefix_logprob(orc.HMM, np.log(pi)[None, None], np.log(phi)[None], np.log(A), x)
    # np.log(A) are already log-probabilities: log_softmax leaves them unchanged
    want = [table[2].sum(), table[2, 0].sum(), table[2, 0, 1]]
    return float(np.abs(got[0] - np.log(want)).max())


def conditional_gap(orc):
    rng = np.random.default_rng(7)
    n, r, v = 3, 2, 3
    omega, phi = pins.rand_simplex(rng, r), pins.rand_simplex(rng, n, r, v)
    table = np.zeros((v,) * n)
    for x in itertools.product(range(v), repeat=n):
        table[x] = pins.enum_cp(omega, phi, x)
    x = np.array([[1, 2, 0]])
    got = orc.next_byte_logprob(orc.CP, np.log(omega)[None, None], np.log(phi)[None], None, x, np.array([1]))
    want = table[1].sum(axis=1) / table[1].sum()
    return float(np.abs(np.exp(got[0]) - want).max())


def accept_wrong(orc):
    """The example worked by hand in test_oracle_speculative.py, plus a full acceptance."""
    p = np.array([[[0.5, 0.3, 0.2], [0.1, 0.3, 0.6], [0.2, 0.2, 0.6]]])
    q_first = np.log(np.array([[0.2, 0.7, 0.1]]))
    q_second = np.log(np.array([[0.25, 0.25, 0.5]]))
    bad = 0.0
    out = orc.speculative_accept(np.log(np.array([[0.7, 0.35]])), np.array([[1, 2]]), p, np.array([[0.5, 0.0, 0.8]]),
                                 lambda rows, s: q_first)
    bad += out["accepted"].tolist() != [0] or out["next_byte"].tolist() != [2]
    out = orc.speculative_accept(np.log(np.array([[0.7, 0.35]])), np.array([[1, 2]]), p, np.array([[0.4, 0.999, 0.15]]),
                                 lambda rows, s: q_second)
    bad += out["accepted"].tolist() != [2] or out["next_byte"].tolist() != [0]    # p(X_3 | 1, 2) = (0.2, 0.2, 0.6)
    out = orc.speculative_accept(np.log(np.array([[0.7, 0.175]])), np.array([[1, 0]]), p, np.array([[0.1, 0.41, 0.3]]),
                                 lambda rows, s: q_second)
    bad += out["accepted"].tolist() != [1] or out["next_byte"].tolist() != [1]
    out = orc.speculative_accept(np.log(np.array([[0.7, 0.175]])), np.array([[1, 0]]), p, np.array([[0.1, 0.39, 0.3]]),
                                 lambda rows, s: q_second)
    bad += out["accepted"].tolist() != [2] or out["next_byte"].tolist() != [1]
    return float(bad)


def hmm_ctx_gap(orc):
    """Contextual HMM against path enumeration with each position's own tables (softmax taken here with scipy)."""
    import scipy.special
    rng = np.random.default_rng(8)
    n, r, v, d, T = 3, 2, 3, 4, 2
    h = rng.normal(size=(T, d))
    R = rng.normal(size=((1 + (n - 1) * r) * r, d))
    bias = rng.normal(size=(n - 1, r, r))
    phi = pins.rand_simplex(rng, T, n, r, v)
    logits = h @ R.T
    gap = 0.0
    for t in range(T):
        pi = scipy.special.softmax(logits[t, :r])
        A = scipy.special.softmax(logits[t, r:].reshape(n - 1, r, r) + bias, axis=-1)
        for x in itertools.product(range(v), repeat=n):
            g = orc.evidence(np.log(phi[t])[None], np.array([x]))
            logw = orc.sum_unit_logw(h[t:t + 1], R, r, bias=bias)
            got = orc.circuit_eval(orc.HMM_CTX, logw, g)[0]
            gap = max(gap, abs(got - math.log(pins.enum_hmm(pi, A, phi[t], x))))
    return gap


def hmm_ctx_sampler_wrong(orc):
    # deterministic chain through the bias (R = 0): 0 -> 1 -> 2 -> 0; a transposed table walks it backwards
    r, n = 3, 4
    bias = np.full((n - 1, r, r), -1e5)
    for a in range(r):
        bias[:, a, (a + 1) % r] = 0.0
    R = np.zeros(((1 + (n - 1) * r) * r, 2))
    R[0, 0] = 50.0                                      # initial state 0
    logw = orc.sum_unit_logw(np.array([[1.0, 0.0]]), R, r, bias=bias)
    unit, _ = orc.sample_latents(orc.HMM_CTX, logw, None, 1, np.full((1, 2 * n), 0.5), n)
    return 0.0 if unit.tolist() == [[0, 1, 2, 0]] else 1.0


def loss_gap(orc):
    ln = math.log
    prefix = np.array([[ln(1 / 2), ln(1 / 8)], [ln(1 / 8), ln(1 / 8)], [ln(1 / 2), ln(1 / 4)], [0.0, 0.0]])
    targets = np.array([[3, 1], [0, -1], [2, 2], [-1, -1]])
    slot, total = orc.composite_loss(prefix, targets, 2, 0.8)
    return float(np.abs(slot - 1.5 * ln(2)).max() + abs(total - 1.5 * ln(2) * 1.8))


def lowrank_gap(orc):
    """Hand example and the scalar formula of App. G's U_ij = W_i + A_ij B_ij, with distinct slots and components."""
    rng = np.random.default_rng(11)
    n, r, v, d, k = 2, 3, 4, 5, 2
    W, A, B = rng.normal(size=(n, v, d)), rng.normal(size=(n, r, v, k)), rng.normal(size=(n, r, k, d))
    U = orc.lowrank_unembedding(W, A, B)
    gap = 0.0
    for i in range(n):
        for j in range(r):
            for b in range(v):
                for c in range(d):
                    want = W[i, b, c] + sum(A[i, j, b, q] * B[i, j, q, c] for q in range(k))
                    gap = max(gap, abs(U[i, j, b, c] - want))
    return gap


MUTANTS = [
    # (what is planted, old text, new text, pin that must notice)
    ("mixture weights dropped from Eq. CP", "logsumexp(logw + g.sum(axis=1), axis=-1)", "logsumexp(g.sum(axis=1), axis=-1)", cp_gap),
    ("product over slots replaced by the first slot", "logw + g.sum(axis=1)", "logw + g[:, 0, :]", cp_gap),
    ("transition table transposed", "alpha[:, :, None] + logA[i - 1][None, :, :], axis=1)",
     "alpha[:, :, None] + logA[i - 1].T[None, :, :], axis=1)", hmm_gap),
    ("forward sum taken over the new state", "logA[i - 1][None, :, :], axis=1)", "logA[i - 1][None, :, :], axis=2)", hmm_gap),
    ("transition of the wrong step", "alpha[:, :, None] + logA[i - 1]", "alpha[:, :, None] + logA[(i - 1) // 2]", hmm_gap),
    ("initial weights forgotten", "alpha = logpi + g[:, 0, :]", "alpha = g[:, 0, :]", hmm_gap),
    ("right child uses the left child's table", "rows = 1 + (child - 1) * r", "rows = 1 + (2 * j + 1 - 1) * r", btree_gap),
    ("child table transposed", "logsumexp(logOmega + below[:, None, :], axis=-1)",
     "logsumexp(logOmega + below[:, :, None], axis=1)", btree_gap),
    ("halves split off centre", "mid = lo + (hi - lo) // 2", "mid = lo + max((hi - lo) // 2 - 1, 1)", btree_gap),
    ("root weights forgotten", "logsumexp(logw[:, 0, :] + _btree_product", "logsumexp(_btree_product", btree_gap),
    ("softmax over the units instead of the vocabulary", "return log_softmax(logits, axis=-1)\n\n\ndef sum_unit_logw",
     "return log_softmax(logits, axis=-2)\n\n\ndef sum_unit_logw", emission_gap),
    ("non-strict CDF comparison", "(cdf <= u[:, None])", "(cdf < u[:, None])", inv_cdf_wrong),
    ("sampler walks the transposed chain", "inv_cdf(logA[i - 1][z, :], u[:, i])", "inv_cdf(logA[i - 1][:, z].T, u[:, i])",
     hmm_sampler_wrong),
    ("tree sampler conditions on the wrong parent", "parent = (j - 1) // 2", "parent = max(j - 2, 0) // 2", btree_sampler_wrong),
    ("tree sampler gives tokens to the wrong node", "zs[:, n // 2 - 1 + i // 2]", "zs[:, n // 2 - 1 + (i + 1) // 2 % (n // 2)]",
     btree_sampler_wrong),
    ("marginalised byte not set to one", "return np.where((x < 0)[:, :, None], 0.0, g)", "return g", masked_gap),
    ("prefix of length i keeps byte i+1", "masked[:, i + 1:] = -1", "masked[:, i + 2:] = -1", prefix_gap),
    ("prefix of length i drops byte i", "masked[:, i + 1:] = -1", "masked[:, i:] = -1", prefix_gap),
    ("conditional not divided by the prefix marginal", "evidence(logphi, ext, pos), T_static) - denom",
     "evidence(logphi, ext, pos), T_static)", conditional_gap),
    ("conditional places the byte one slot late", "ext = np.where(cols == s[:, None], b, base)",
     "ext = np.where(cols == s[:, None] + 1, b, base)", conditional_gap),
    ("acceptance uses the joint prefix instead of the conditional", "lq = prefix_lq[w, s] - (prefix_lq[w, s - 1] if s > 0 else 0.0)",
     "lq = prefix_lq[w, s]", accept_wrong),
    ("acceptance ratio inverted", "ratio = p[w, s, x[w, s]] / np.exp(lq)", "ratio = np.exp(lq) / p[w, s, x[w, s]]", accept_wrong),
    ("acceptance test reversed", "if alpha > ratio:", "if alpha < ratio:", accept_wrong),
    ("residual taken as q - p", "m = np.maximum(0.0, p[rej, accepted[rej], :] - qn)", "m = np.maximum(0.0, qn - p[rej, accepted[rej], :])",
     accept_wrong),
    ("residual not clipped at zero", "m = np.maximum(0.0, p[rej, accepted[rej], :] - qn)", "m = np.abs(p[rej, accepted[rej], :] - qn)",
     accept_wrong),
    ("residual uses the target row of the first byte", "m = np.maximum(0.0, p[rej, accepted[rej], :] - qn)",
     "m = np.maximum(0.0, p[rej, 0, :] - qn)", accept_wrong),
    ("byte after a full acceptance drawn from the wrong target row", "inv_cdf(np.log(np.maximum(p[full, n, :], 1e-300)), u[full, n])",
     "inv_cdf(np.log(np.maximum(p[full, n - 1, :], 1e-300)), u[full, n])", accept_wrong),
    ("acceptance test uses the last uniform", "alpha = u[w, s]", "alpha = u[w, n]", accept_wrong),
    ("contextual table of the wrong step", "logA = logw[:, 1 + (i - 1) * r:1 + i * r, :]", "logA = logw[:, 1:1 + r, :]", hmm_ctx_gap),
    ("contextual table transposed", "alpha = g[:, i, :] + logsumexp(alpha[:, :, None] + logA, axis=1)",
     "alpha = g[:, i, :] + logsumexp(alpha[:, None, :] + logA, axis=2)", hmm_ctx_gap),
    ("transition bias dropped", "logits[:, 1:, :] += np.asarray(bias, dtype=np.float64).reshape(1, -1, r)",
     "logits[:, 1:, :] += 0.0", hmm_ctx_gap),
    ("transition bias also added to the initial unit", "logits[:, 1:, :] += np.asarray(bias, dtype=np.float64).reshape(1, -1, r)",
     "logits[:, :-1, :] += np.asarray(bias, dtype=np.float64).reshape(1, -1, r)", hmm_ctx_gap),
    ("contextual sampler ignores the previous state", "inv_cdf(logw[pos, 1 + (i - 1) * r + z, :], u[:, i])",
     "inv_cdf(logw[pos, 1 + (i - 1) * r, :], u[:, i])", hmm_ctx_sampler_wrong),
    ("loss normalised by the sequence length instead of the valid count", "acc += cond[rows, j][valid].sum() / V",
     "acc += cond[rows, j][valid].sum() / L", loss_gap),
    ("loss counts invalid bytes", "valid = tg[rows, j] >= 0", "valid = tg[rows, j] >= -1", loss_gap),
    ("loss uses the prefix marginal instead of the conditional", "cond = pre - np.concatenate([np.zeros((T, 1)), pre[:, :-1]], axis=1)",
     "cond = pre", loss_gap),
    ("discount starts at gamma instead of one", "sum(gamma ** j * slot[j] for j in range(n))",
     "sum(gamma ** (j + 1) * slot[j] for j in range(n))", loss_gap),
    ("loss not averaged over the sequences", "slot[j] = -acc / N", "slot[j] = -acc", loss_gap),
    ("adaptor added to the base matrix of the wrong slot", "U[i, j] = W_base[i] + A[i, j] @ B[i, j]",
     "U[i, j] = W_base[0] + A[i, j] @ B[i, j]", lowrank_gap),
    ("adaptor shared by the components", "U[i, j] = W_base[i] + A[i, j] @ B[i, j]", "U[i, j] = W_base[i] + A[i, 0] @ B[i, 0]",
     lowrank_gap),
    ("adaptor dropped", "U[i, j] = W_base[i] + A[i, j] @ B[i, j]", "U[i, j] = W_base[i]", lowrank_gap),
]


def test_every_pin_passes_on_the_real_oracle():
    orc = mutant("CP, HMM, BTREE, HMM_CTX = 0, 1, 2, 3", "CP, HMM, BTREE, HMM_CTX = 0, 1, 2, 3")   # unmodified copy
    for pin in {m[3] for m in MUTANTS}:
        assert pin(orc) < 1e-12, pin.__name__


@pytest.mark.parametrize("what,old,new,pin", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistake_breaks_a_pin(what, old, new, pin):
    try:
        gap = pin(mutant(old, new))
    except Exception:
        return                      # a mutant that cannot even run is caught too
    assert gap > 1e-6, f"the pins do not notice: {what}"
