"""Pins of the oracle's shared-unembedding parametrisation (App. G, "Unembedding parameter sharing":
U_ij = W_i + A_ij B_ij with a rank-k adaptor per component)."""
import numpy as np

from oracle import mtpc_oracle as O
from oracle import mtpc_oracle_grad as OG


def _params(seed, n=2, r=3, v=5, d=4, k=2):
    rng = np.random.default_rng(seed)
    return rng.normal(size=(n, v, d)), rng.normal(size=(n, r, v, k)), rng.normal(size=(n, r, k, d))


def test_zero_adaptor_resumes_from_the_shared_matrix():
    """App. G: with every entry of B zero the head starts as the one that shares W_i across its components."""
    W, A, B = _params(0)
    U = O.lowrank_unembedding(W, A, np.zeros_like(B))
    for j in range(A.shape[1]):
        np.testing.assert_array_equal(U[:, j], W)


def test_adaptor_has_rank_k_and_is_per_component():
    W, A, B = _params(1, v=7, d=6, k=2)
    U = O.lowrank_unembedding(W, A, B)
    for i in range(U.shape[0]):
        for j in range(U.shape[1]):
            assert np.linalg.matrix_rank(U[i, j] - W[i]) == 2
    # a single entry, by the scalar formula: U[i, j, b, c] = W[i, b, c] + sum_q A[i, j, b, q] B[i, j, q, c]
    i, j, b, c = 1, 2, 4, 3
    want = W[i, b, c] + sum(A[i, j, b, q] * B[i, j, q, c] for q in range(2))
    assert abs(U[i, j, b, c] - want) < 1e-14
    # changing the adaptor of one component leaves the others alone
    A2 = A.copy()
    A2[0, 1] += 1.0
    U2 = O.lowrank_unembedding(W, A2, B)
    changed = np.abs(U2 - U).reshape(U.shape[0], U.shape[1], -1).max(axis=-1) > 0
    assert changed[0, 1] and changed.sum() == 1


def test_hand_example():
    """n = r = 1, v = d = 2, k = 1: U = W + a b^T with a = (1, 2), b = (3, -1)."""
    W = np.array([[[1.0, 0.0], [0.0, 1.0]]])
    A = np.array([[[[1.0], [2.0]]]])
    B = np.array([[[[3.0, -1.0]]]])
    np.testing.assert_array_equal(O.lowrank_unembedding(W, A, B)[0, 0], np.array([[4.0, -1.0], [6.0, -1.0]]))


def test_gradient_matches_finite_differences_of_the_numpy_definition():
    W, A, B = _params(2)
    rng = np.random.default_rng(3)
    dU = rng.normal(size=(2, 3, 5, 4))
    g = OG.lowrank_grad(W, A, B, dU)
    np.testing.assert_allclose(g["U"], O.lowrank_unembedding(W, A, B), atol=1e-13)
    f = lambda W_, A_, B_: float((O.lowrank_unembedding(W_, A_, B_) * dU).sum())
    eps = 1e-6
    for name, arr, pos in (("dW_base", W, 0), ("dA", A, 1), ("dB", B, 2)):
        for _ in range(12):
            idx = tuple(rng.integers(0, s) for s in arr.shape)
            args = [W.copy(), A.copy(), B.copy()]
            args[pos][idx] += eps
            up = f(*args)
            args[pos][idx] -= 2 * eps
            dn = f(*args)
            assert abs((up - dn) / (2 * eps) - g[name][idx]) < 1e-7, (name, idx)


def test_gradient_closed_forms():
    W, A, B = _params(4)
    dU = np.random.default_rng(5).normal(size=(2, 3, 5, 4))
    g = OG.lowrank_grad(W, A, B, dU)
    np.testing.assert_allclose(g["dW_base"], dU.sum(axis=1), atol=1e-13)   # the base matrix is shared by the r components
    g0 = OG.lowrank_grad(W, A, np.zeros_like(B), dU)
    assert np.abs(g0["dA"]).max() == 0.0                                   # at the App. G initialisation only B learns
    assert np.abs(g0["dB"]).max() > 0.0
