"""fp64 CPU oracle for the MtPC head: TEST INFRASTRUCTURE, not a product path.

Plain, slow, step-by-step numpy (float64) statement of what the head computes, written from the paper's
definitions. It shares no code with the CUDA library and must never be imported by it; only the tests,
the smoke check and the benchmark's CPU-baseline leg call it.

What follows which passage:
  emission_logphi   Sec. 3.3 "Input unit distributions": phi_tij = softmax(W_ij e_t)
  sum_unit_logw     Sec. 3.3 "Sum unit parameters":      omega_ti = softmax(R_i e_t)
  evidence          Sec. 3.1 (input units) + App. B.1 (a marginalised input unit integrates to 1)
  cp_eval           Eq. (CP)
  hmm_eval          Eq. (HMM), evaluated layer by layer (one sum + one product layer per window step)
  hmm_ctx_eval      the same with contextual transitions (App. H): tables produced from the hidden state
  btree_eval        Eq. (BTree), recursive halving with a latent per internal node
  draft_sample      App. B.2, Algorithm 1 (ancestral sampling), with inverse-CDF categorical draws
  circuit_counts    App. C, Table 3 (sizes of the circuits and of the linear head)
  prefix_logprob    Algorithm 3, "compute marginals": q(x_1..x_i) for i = 1..n, by summing the later bytes out
  next_byte_logprob the conditional q(X_{s+1} | x_1..x_s) as a ratio of two such marginals
  speculative_accept Algorithm 3, acceptance loop and the last byte (residual or target distribution)
  composite_loss    Eq. (6): per-slot negative log-likelihood with valid-token normalisation and discount gamma
  lowrank_unembedding  App. G, "Unembedding parameter sharing": U_ij = W_i + A_ij B_ij

Readings taken where the paper is silent or garbled:
  * BTree: the left half is the first floor(n/2) tokens; a child latent depends on its parent's latent
    only; products are element-wise in the latent; n must be a power of two here. Internal nodes are in
    heap order (root 0, children 2j+1 and 2j+2); the deepest internal node n/2-1+m owns tokens 2m, 2m+1.
    Table 3's parameter counts fix the number of sum units at 1 + (n-2) r, each of fan-in r.
  * HMM: T_static[i-1, a, b] is the logit of z_i = b given z_{i-1} = a (softmax over b); only the initial
    distribution is contextual here (the paper's "non-contextual" transition variant).
  * HMM_CTX (the paper's best configuration, App. H): transition logits = rows of R applied to the hidden state
    plus a bias [n-1, r, r] (the "bias term" that allows the identity initialisation), softmax over the new state.
  * sampleCategorical is inverse-CDF: the smallest index j with u < p_0 + ... + p_j (last index if none).
  * The draft log-prob is the joint marginal log q(x_1..x_n) (latents summed out), as verification needs.
  * No bias and no temperature in either projection.

Pins (tests/test_oracle_*.py): brute-force normalisation over all v^n strings; CP with r=1 equals the
product of marginals; CP/HMM/BTree equal literal enumeration over latent assignments; HMM with identity
transitions equals CP; BTree with n=2 equals CP; masked targets equal brute-force marginals; closed-form
softmax cases; sampled frequencies match the exact joint (chi-squared); Table 3 counts; prefix marginals equal
brute-force sums over the later bytes; the conditional sums to one and chains back to the joint; the
acceptance stage reproduces a hand-computed example, accepts everything when target and draft agree, and its
output bytes follow the TARGET model's distribution (chi-squared) whatever the draft is; the loss reproduces a
hand-computed example and, with gamma = 1 and every byte valid, the mean joint negative log-likelihood. No
function here is left unpinned.
"""
from __future__ import annotations

import numpy as np

CP, HMM, BTREE, HMM_CTX = 0, 1, 2, 3     # HMM_CTX: HMM whose transitions depend on the hidden state (App. H)


# ----------------------------------------------------------------------------------------------------
# elementary pieces
# ----------------------------------------------------------------------------------------------------
def logsumexp(x: np.ndarray, axis: int = -1) -> np.ndarray:
    m = np.max(x, axis=axis, keepdims=True)
    return np.squeeze(m, axis=axis) + np.log(np.sum(np.exp(x - m), axis=axis))


def log_softmax(x: np.ndarray, axis: int = -1) -> np.ndarray:
    return x - np.expand_dims(logsumexp(x, axis=axis), axis)


def num_sum_units(family: int, n: int, r: int, contextual_transitions: bool = False) -> int:
    """How many sum units the head parameterises from the hidden state (the z of R in R^{z x r x d})."""
    if family == CP:
        return 1
    if family == HMM:
        return 1 + (n - 1) * r if contextual_transitions else 1
    if family == HMM_CTX:
        return 1 + (n - 1) * r
    if family == BTREE:
        return 1 + (n - 2) * r
    raise ValueError(family)


def circuit_counts(family: str, n: int, r: int, v: int, d: int) -> dict:
    """Parameter and FLOP counts in the convention of Table 3 (contextual HMM transitions, as the paper's
    experiments use). A sum unit of fan-in r costs 2r FLOPs; FF is n input units and one product."""
    if family == "ff":
        return dict(circuit_params=n * v, circuit_flops=n - 1, head_params=n * v * d, head_flops=2 * n * v * d)
    fam = {"cp": CP, "hmm": HMM, "btree": BTREE}[family]
    S = num_sum_units(fam, n, r, contextual_transitions=True)
    circuit_params = n * r * v + S * r
    head_params = circuit_params * d
    return dict(circuit_params=circuit_params, circuit_flops=2 * r * S, head_params=head_params,
                head_flops=2 * head_params)


# ----------------------------------------------------------------------------------------------------
# head: hidden state -> circuit parameters (Sec. 3.3)
# ----------------------------------------------------------------------------------------------------
def emission_logphi(h: np.ndarray, W_emit: np.ndarray) -> np.ndarray:
    """log phi[t, i, k, :] = log softmax(W_emit[i, k] @ h[t]);  h [T, d], W_emit [n, r, v, d] -> [T, n, r, v]."""
    h = np.asarray(h, dtype=np.float64)
    W = np.asarray(W_emit, dtype=np.float64)
    n, r, v, d = W.shape
    logits = (h @ W.reshape(n * r * v, d).T).reshape(h.shape[0], n, r, v)
    return log_softmax(logits, axis=-1)


def sum_unit_logw(h: np.ndarray, W_sum: np.ndarray, r: int, bias: np.ndarray | None = None) -> np.ndarray:
    """log omega[t, s, :] = log softmax(W_sum[s*r:(s+1)*r] @ h[t]);  -> [T, S, r].
    `bias` (contextual HMM, App. H "adding a bias term"): [n-1, r, r] logits added to the sum units after the
    first one, in row order, before the softmax; bias[i-1, a, :] belongs to the unit of z_i given z_{i-1} = a."""
    h = np.asarray(h, dtype=np.float64)
    R = np.asarray(W_sum, dtype=np.float64)
    logits = (h @ R.T).reshape(h.shape[0], R.shape[0] // r, r)
    if bias is not None:
        logits = logits.copy()
        logits[:, 1:, :] += np.asarray(bias, dtype=np.float64).reshape(1, -1, r)
    return log_softmax(logits, axis=-1)


def evidence(logphi: np.ndarray, targets: np.ndarray, pos: np.ndarray | None = None) -> np.ndarray:
    """g[w, i, k] = log phi[pos[w], i, k, x_wi]; a negative target marginalises the byte: the unit
    outputs 1 (log 0 = 0 contribution). `pos` maps each window to its position (identity if None)."""
    T, n, r, v = logphi.shape
    x = np.asarray(targets).reshape(-1, n)
    if pos is None:
        pos = np.arange(T)
    safe = np.where(x < 0, 0, x)
    g = logphi[pos[:, None, None], np.arange(n)[None, :, None], np.arange(r)[None, None, :], safe[:, :, None]]
    return np.where((x < 0)[:, :, None], 0.0, g)


# ----------------------------------------------------------------------------------------------------
# circuit evaluation (log space)
# ----------------------------------------------------------------------------------------------------
def cp_eval(logw: np.ndarray, g: np.ndarray) -> np.ndarray:
    """Eq. (CP): sum_z q(z) prod_i q(x_i | z);  logw [T, r], g [T, n, r] -> [T]."""
    return logsumexp(logw + g.sum(axis=1), axis=-1)


def hmm_eval(logpi: np.ndarray, logA: np.ndarray, g: np.ndarray) -> np.ndarray:
    """Eq. (HMM). logpi [T, r]; logA [n-1, r, r] with logA[i-1, a, b] = log q(z_i = b | z_{i-1} = a);
    g [T, n, r]. alpha_1(z) = q(z) q(x_1|z); alpha_i(b) = q(x_i|b) sum_a alpha_{i-1}(a) q(b|a)."""
    T, n, r = g.shape
    alpha = logpi + g[:, 0, :]
    for i in range(1, n):
        alpha = g[:, i, :] + logsumexp(alpha[:, :, None] + logA[i - 1][None, :, :], axis=1)
    return logsumexp(alpha, axis=-1)


def _btree_product(j: int, lo: int, hi: int, logw: np.ndarray, g: np.ndarray, r: int) -> np.ndarray:
    """log of the product unit under latent z_j over tokens [lo, hi): [T, r] indexed by the value of z_j."""
    mid = lo + (hi - lo) // 2
    out = 0.0
    for child, (a, b) in ((2 * j + 1, (lo, mid)), (2 * j + 2, (mid, hi))):
        if b - a == 1:
            out = out + g[:, a, :]                       # input units of token a, one per value of z_j
        else:
            below = _btree_product(child, a, b, logw, g, r)            # [T, r] over z_child
            rows = 1 + (child - 1) * r                                  # sum units of node `child`
            logOmega = logw[:, rows:rows + r, :]                        # [T, z_j, z_child]
            out = out + logsumexp(logOmega + below[:, None, :], axis=-1)
    return out


def btree_eval(logw: np.ndarray, g: np.ndarray) -> np.ndarray:
    """Eq. (BTree). logw [T, 1 + (n-2) r, r]: group 0 = root weights; group 1 + (j-1) r + a = weights of
    node j's latent given its parent's latent = a.  g [T, n, r]."""
    T, n, r = g.shape
    if n < 2 or (n & (n - 1)):
        raise ValueError("binary-tree head: n must be a power of two >= 2")
    return logsumexp(logw[:, 0, :] + _btree_product(0, 0, n, logw, g, r), axis=-1)


def hmm_ctx_eval(logw: np.ndarray, g: np.ndarray) -> np.ndarray:
    """Eq. (HMM) with contextual, inhomogeneous transitions (App. H): every position has its own tables.
    logw [T, 1 + (n-1) r, r]: unit 0 = initial distribution; unit 1 + (i-1) r + a = log q(z_i = . | z_{i-1} = a)."""
    T, n, r = g.shape
    alpha = logw[:, 0, :] + g[:, 0, :]
    for i in range(1, n):
        logA = logw[:, 1 + (i - 1) * r:1 + i * r, :]                   # [T, a, b]
        alpha = g[:, i, :] + logsumexp(alpha[:, :, None] + logA, axis=1)
    return logsumexp(alpha, axis=-1)


def static_log_transitions(T_static: np.ndarray) -> np.ndarray:
    return log_softmax(np.asarray(T_static, dtype=np.float64), axis=-1)


def circuit_eval(family: int, logw: np.ndarray, g: np.ndarray, T_static: np.ndarray | None = None) -> np.ndarray:
    if family == CP:
        return cp_eval(logw[:, 0, :], g)
    if family == HMM:
        return hmm_eval(logw[:, 0, :], static_log_transitions(T_static), g)
    if family == BTREE:
        return btree_eval(logw, g)
    if family == HMM_CTX:
        return hmm_ctx_eval(logw, g)
    raise ValueError(family)


def head_logw(family: int, h, W_sum, T_static, r: int) -> np.ndarray:
    """Sum-unit log-weights of a head; for HMM_CTX the fourth argument is the transition bias (or None)."""
    return sum_unit_logw(h, W_sum, r, bias=T_static if family == HMM_CTX else None)


def window_logprob(family: int, h, W_emit, W_sum, T_static, targets) -> np.ndarray:
    """log q(x_{t+1..t+n} | context) in nats for every position: [T]."""
    r = np.asarray(W_emit).shape[1]
    logphi = emission_logphi(h, W_emit)
    logw = head_logw(family, h, W_sum, T_static, r)
    return circuit_eval(family, logw, evidence(logphi, targets), T_static)


# ----------------------------------------------------------------------------------------------------
# ancestral sampling (Algorithm 1) from pre-generated uniforms
# ----------------------------------------------------------------------------------------------------
def inv_cdf(logp: np.ndarray, u: np.ndarray):
    """Rows of log-probabilities [M, c] and uniforms [M] -> (index [M], margin [M]).
    index = smallest j with u < p_0 + ... + p_j, or c-1 if rounding leaves none.
    margin = distance from u to the nearest interior CDF boundary (how close the draw is to flipping)."""
    cdf = np.cumsum(np.exp(logp), axis=-1)
    u = np.asarray(u, dtype=np.float64)
    idx = np.minimum((cdf <= u[:, None]).sum(axis=-1), logp.shape[-1] - 1)
    if logp.shape[-1] > 1:
        margin = np.abs(cdf[:, :-1] - u[:, None]).min(axis=-1)
    else:
        margin = np.full(u.shape, np.inf)
    return idx.astype(np.int64), margin


def sample_latents(family: int, logw: np.ndarray, T_static, wpp: int, u: np.ndarray, n: int):
    """Top-down draws at the sum units. logw [P, S, r]; u [P*wpp, 2n] (latent draws use columns 0..n-1:
    CP column 0; HMM column i for z_i; BTree column j for internal node j). Returns
    (unit [W, n]: the input unit selected for every token, margin [W]: smallest latent-draw margin)."""
    P, S, r = logw.shape
    W = P * wpp
    pos = np.repeat(np.arange(P), wpp)
    unit = np.zeros((W, n), dtype=np.int64)
    margin = np.full(W, np.inf)
    if family == CP:
        z, m = inv_cdf(logw[pos, 0, :], u[:, 0])
        unit[:] = z[:, None]
        margin = m
    elif family == HMM:
        logA = static_log_transitions(T_static)
        z, margin = inv_cdf(logw[pos, 0, :], u[:, 0])
        unit[:, 0] = z
        for i in range(1, n):
            z, m = inv_cdf(logA[i - 1][z, :], u[:, i])
            unit[:, i] = z
            margin = np.minimum(margin, m)
    elif family == HMM_CTX:
        z, margin = inv_cdf(logw[pos, 0, :], u[:, 0])
        unit[:, 0] = z
        for i in range(1, n):
            z, m = inv_cdf(logw[pos, 1 + (i - 1) * r + z, :], u[:, i])
            unit[:, i] = z
            margin = np.minimum(margin, m)
    elif family == BTREE:
        zs = np.zeros((W, n - 1), dtype=np.int64)
        zs[:, 0], margin = inv_cdf(logw[pos, 0, :], u[:, 0])
        for j in range(1, n - 1):
            parent = (j - 1) // 2
            zs[:, j], m = inv_cdf(logw[pos, 1 + (j - 1) * r + zs[:, parent], :], u[:, j])
            margin = np.minimum(margin, m)
        for i in range(n):
            unit[:, i] = zs[:, n // 2 - 1 + i // 2]
    else:
        raise ValueError(family)
    return unit, margin


def draft_sample(family: int, h, W_emit, W_sum, T_static, wpp: int, u: np.ndarray):
    """Algorithm 1 for wpp windows per position. Window w = p*wpp + j uses uniforms u[w]: latent draws in
    columns 0..n-1, the byte of token i in column n+i. Returns dict(bytes [W, n], logprob [W] = joint
    marginal log q of the drafted bytes, unit [W, n], margin [W] = smallest |u - CDF boundary| of any draw
    the window made)."""
    W_emit = np.asarray(W_emit)
    n, r, v, d = W_emit.shape
    logphi = emission_logphi(h, W_emit)                     # [P, n, r, v]
    logw = head_logw(family, h, W_sum, T_static, r)
    P = logphi.shape[0]
    pos = np.repeat(np.arange(P), wpp)
    unit, margin = sample_latents(family, logw, T_static, wpp, u, n)
    x = np.zeros((P * wpp, n), dtype=np.int64)
    for i in range(n):
        x[:, i], m = inv_cdf(logphi[pos, i, unit[:, i], :], u[:, n + i])
        margin = np.minimum(margin, m)
    g = evidence(logphi, x, pos)
    logprob = circuit_eval(family, logw[pos], g, T_static)
    return dict(bytes=x, logprob=logprob, unit=unit, margin=margin)


# ----------------------------------------------------------------------------------------------------
# prefix marginals and speculative acceptance (Algorithm 3)
# ----------------------------------------------------------------------------------------------------
def prefix_logprob(family: int, logw: np.ndarray, logphi: np.ndarray, T_static, x: np.ndarray,
                   pos: np.ndarray | None = None) -> np.ndarray:
    """log q(x_1..x_i | context) for i = 1..n (Algorithm 3, "compute marginals"): the joint with the bytes
    x_{i+1}..x_n summed out, which a smooth and decomposable circuit does by letting those input units output 1
    (App. B.1). Written as that definition: one masked evaluation per prefix length.  -> [W, n]."""
    x = np.asarray(x)
    W, n = x.shape
    lw = logw if pos is None else logw[pos]
    out = np.zeros((W, n))
    for i in range(n):
        masked = x.copy()
        masked[:, i + 1:] = -1
        out[:, i] = circuit_eval(family, lw, evidence(logphi, masked, pos), T_static)
    return out


def window_prefix_logprob(family: int, h, W_emit, W_sum, T_static, targets) -> np.ndarray:
    """Prefix log-marginals of the observed window at every position: [T, n]; column n-1 is the joint."""
    r = np.asarray(W_emit).shape[1]
    return prefix_logprob(family, head_logw(family, h, W_sum, T_static, r), emission_logphi(h, W_emit), T_static, targets)


def next_byte_logprob(family: int, logw: np.ndarray, logphi: np.ndarray, T_static, x: np.ndarray, s: np.ndarray,
                      pos: np.ndarray | None = None) -> np.ndarray:
    """log q(X_{s+1} = b | x_1..x_s, context) for every byte b: [W, v]. s[w] in [0, n) is the number of bytes
    already fixed in window w. By definition of the conditional: the marginal of (x_1..x_s, b) with everything
    after summed out, divided by the marginal of (x_1..x_s)."""
    x = np.asarray(x)
    W, n = x.shape
    v = logphi.shape[-1]
    lw = logw if pos is None else logw[pos]
    cols = np.arange(n)[None, :]
    base = np.where(cols < s[:, None], x, -1)
    denom = circuit_eval(family, lw, evidence(logphi, base, pos), T_static)
    out = np.zeros((W, v))
    for b in range(v):
        ext = np.where(cols == s[:, None], b, base)
        out[:, b] = circuit_eval(family, lw, evidence(logphi, ext, pos), T_static) - denom
    return out


def speculative_accept(prefix_lq: np.ndarray, x: np.ndarray, p: np.ndarray, u: np.ndarray, next_byte_fn):
    """The acceptance stage of Algorithm 3 for a batch of drafted windows.
      prefix_lq [W, n]   log q(x_1..x_i) of the draft, i = 1..n
      x         [W, n]   the drafted bytes
      p         [W, n+1, v]  target-model conditionals p(X_{t+i} | x_{<=t+i-1}) along the draft, i = 1..n+1
      u         [W, n+1] uniforms: column i is the alpha of the test on byte i+1; column n draws the last byte
      next_byte_fn(rows, s) -> [len(rows), v]  log q(X_{s+1} | x_1..x_s) for the given windows (needed only
                         where a byte was rejected)
    Steps, in the algorithm's order: s = 0; while s < n: the draft's conditional of byte s+1 is the ratio of
    consecutive prefix marginals (the first prefix marginal itself for s = 0); stop if alpha > p / q; else
    s += 1. Then one more byte: from the residual max(0, p - q) / Z if s < n, from p otherwise; both draws are
    inverse-CDF with the row's last uniform.
    Returns dict(accepted [W], next_byte [W], margin [W]): margin = how close any decision of the window was to
    flipping (min over the tests of |alpha - ratio| = margin_alpha, and the final draw's distance to a CDF
    boundary of the normalised distribution = margin_final); resid_mass [W] = Z of the residual (1 where all n
    bytes were accepted)."""
    x = np.asarray(x)
    W, n = x.shape
    v = p.shape[-1]
    p = np.asarray(p, dtype=np.float64)
    u = np.asarray(u, dtype=np.float64)
    accepted = np.zeros(W, dtype=np.int64)
    margin_alpha = np.full(W, np.inf)
    for w in range(W):
        s = 0
        while s < n:
            alpha = u[w, s]
            lq = prefix_lq[w, s] - (prefix_lq[w, s - 1] if s > 0 else 0.0)
            ratio = p[w, s, x[w, s]] / np.exp(lq)
            margin_alpha[w] = min(margin_alpha[w], abs(alpha - ratio))
            if alpha > ratio:
                break
            s += 1
        accepted[w] = s
    next_byte = np.zeros(W, dtype=np.int64)
    margin_final = np.full(W, np.inf)
    resid_mass = np.ones(W)
    rej = np.nonzero(accepted < n)[0]
    if len(rej):
        qn = np.exp(next_byte_fn(rej, accepted[rej]))
        m = np.maximum(0.0, p[rej, accepted[rej], :] - qn)
        resid_mass[rej] = m.sum(axis=-1)
        resid = m / m.sum(axis=-1, keepdims=True)
        idx, mg = inv_cdf(np.log(np.maximum(resid, 1e-300)), u[rej, n])
        next_byte[rej] = idx
        margin_final[rej] = mg
    full = np.nonzero(accepted == n)[0]
    if len(full):
        idx, mg = inv_cdf(np.log(np.maximum(p[full, n, :], 1e-300)), u[full, n])
        next_byte[full] = idx
        margin_final[full] = mg
    margin = np.minimum(margin_alpha, margin_final)
    return dict(accepted=accepted, next_byte=next_byte, margin=margin, margin_alpha=margin_alpha,
                margin_final=margin_final, resid_mass=resid_mass)


# ----------------------------------------------------------------------------------------------------
# training loss over overlapping windows (Eq. 6)
# ----------------------------------------------------------------------------------------------------
def composite_loss(prefix_lq: np.ndarray, targets: np.ndarray, num_sequences: int, gamma: float):
    """Eq. (6): L_j = -(1/N) sum_i (1/V_ij) sum_t log p(x_{t+j} | x_{<t+j}) and L = sum_j gamma^(j-1) L_j.
    prefix_lq [N*L, n] are the prefix log-marginals of every position's window (sequence-major rows); the
    conditional of slot j given the context and the window's earlier bytes is prefix[:, j] - prefix[:, j-1].
    A negative target is an invalid byte: it is left out of the sum and of the count V_ij (a slot of a sequence
    with no valid byte contributes nothing). Returns (L_j for every slot [n], L)."""
    pre = np.asarray(prefix_lq, dtype=np.float64)
    tg = np.asarray(targets)
    T, n = pre.shape
    N = num_sequences
    L = T // N
    cond = pre - np.concatenate([np.zeros((T, 1)), pre[:, :-1]], axis=1)
    slot = np.zeros(n)
    for j in range(n):
        acc = 0.0
        for i in range(N):
            rows = slice(i * L, (i + 1) * L)
            valid = tg[rows, j] >= 0
            V = int(valid.sum())
            if V:
                acc += cond[rows, j][valid].sum() / V
        slot[j] = -acc / N
    total = float(sum(gamma ** j * slot[j] for j in range(n)))
    return slot, total


# ----------------------------------------------------------------------------------------------------
# shared unembeddings with low-rank adaptors (App. G)
# ----------------------------------------------------------------------------------------------------
def lowrank_unembedding(W_base: np.ndarray, A: np.ndarray, B: np.ndarray) -> np.ndarray:
    """App. G, "Unembedding parameter sharing": the unembedding matrix of token i and component j is
    U[i, j] = W_base[i] + A[i, j] @ B[i, j], with W_base [n, v, d], A [n, r, v, k], B [n, r, k, d].
    Returns U [n, r, v, d]; written as the definition, one (i, j) at a time."""
    W_base = np.asarray(W_base, dtype=np.float64)
    A = np.asarray(A, dtype=np.float64)
    B = np.asarray(B, dtype=np.float64)
    n, r, v, k = A.shape
    d = B.shape[-1]
    U = np.empty((n, r, v, d))
    for i in range(n):
        for j in range(r):
            U[i, j] = W_base[i] + A[i, j] @ B[i, j]
    return U
