"""GPU parity of the shared-unembedding parametrisation (App. G: U_ij = W_i + A_ij B_ij): composition and the
gradient carried back to W, A, B, from the CUDA path (C ABI) against the fp64 oracle on the same seeded inputs.

Bar. The composed tensor is stored in bf16: the device rounds an fp32 sum of k + 1 terms of size <= 0.1 (error below
1e-7 absolute), so it must equal the oracle's value within half a bf16 spacing (at most 2^-8 relative) plus that slack,
and must be the exact bf16 rounding of the fp64 value on all but a small fraction of the entries (those that sit at a
rounding boundary). The gradients
are fp32 sums of at most max(v, d, r) products: 1e-5 of the tensor's largest magnitude."""
import numpy as np
import pytest
import torch

from oracle import mtpc_oracle as O
from oracle import mtpc_oracle_grad as OG
from paper_2511_11346_b200 import binding as B
from paper_2511_11346_b200 import inputs as I
from paper_2511_11346_b200.runner import DeviceHead, lowrank_backward, lowrank_compose, to_device_bf16

pytestmark = pytest.mark.gpu

SHAPES = [
    # n, r, v, d, k
    (1, 1, 16, 64, 1),
    (2, 3, 48, 100, 3),          # d not a multiple of the CTA width, odd k
    (3, 4, 320, 300, 8),
    (2, 2, 272, 520, 16),
    (1, 5, 33, 257, 9),          # ragged everywhere
    (2, 2, 64, 256, 64),         # the largest rank
]


def _device(x):
    return to_device_bf16(np.ascontiguousarray(x))


@pytest.mark.parametrize("n,r,v,d,k", SHAPES)
def test_compose_matches_the_definition(n, r, v, d, k):
    W, A, Bm = I.lowrank_parameters(n, r, v, d, k, seed=900 + n + r + v + d + k)
    got = lowrank_compose(_device(W), _device(A), _device(Bm)).float().cpu().numpy().astype(np.float64)
    ref = O.lowrank_unembedding(W, A, Bm)
    assert np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-7)
    exact = I.bf16_round(ref.astype(np.float32)).astype(np.float64)      # fp64 -> fp32 -> bf16, the value but for double rounding
    assert np.mean(got != exact) < 1e-3


def test_zero_adaptor_reproduces_the_shared_matrix_bit_for_bit():
    n, r, v, d, k = 2, 3, 48, 128, 4
    W, A, Bm = I.lowrank_parameters(n, r, v, d, k, seed=77, zero_B=True)
    got = lowrank_compose(_device(W), _device(A), _device(Bm)).float().cpu().numpy()
    for j in range(r):
        np.testing.assert_array_equal(got[:, j], W)


@pytest.mark.parametrize("n,r,v,d,k", SHAPES)
def test_backward_matches_the_gradient_oracle(n, r, v, d, k):
    W, A, Bm = I.lowrank_parameters(n, r, v, d, k, seed=300 + n + r + v + d + k)
    dU = np.random.default_rng(k + d).normal(size=(n, r, v, d)).astype(np.float32)
    dW, dA, dB = lowrank_backward(_device(A), _device(Bm), torch.from_numpy(dU).cuda())
    torch.cuda.synchronize()
    ref = OG.lowrank_grad(W, A, Bm, dU)
    for name, got, want in (("dW_base", dW, ref["dW_base"]), ("dA", dA, ref["dA"]), ("dB", dB, ref["dB"])):
        got = got.cpu().numpy().astype(np.float64)
        assert got.shape == want.shape
        assert np.abs(got - want).max() <= 1e-5 * np.abs(want).max(), name


@pytest.mark.parametrize("family", [I.CP, I.BTREE])
def test_head_on_composed_unembeddings_and_the_gradient_chain(family):
    """Compose on the device, run the head and its backward on the composed tensor, carry dW_emit back to W, A, B;
    the oracle does the same chain in fp64 on the bf16 rounding of its own composed tensor."""
    n, r, v, d, k, T = 4, 4, 64, 128, 4, 150
    shape = I.HeadShape(family, n, r, v, d)
    wl = I.make_workload("lowrank_chain", shape, T, seed=4242, weight_std=0.25)
    W, A, Bm = I.lowrank_parameters(n, r, v, d, k, seed=4243, weight_std=0.25, adaptor_std=0.2)
    U_q = I.bf16_round(O.lowrank_unembedding(W, A, Bm).astype(np.float32))
    dA_, dB_ = _device(A), _device(Bm)
    U_dev = lowrank_compose(_device(W), dA_, dB_)
    assert np.mean(U_dev.float().cpu().numpy() != U_q) < 1e-3
    wl.W_emit_q = U_q
    head = DeviceHead(wl)
    head.head.mtpc_destroy()
    head.W_emit = U_dev                                                   # the head under test runs on the device's own composition
    s = wl.shape
    head.head = B.MtpcHead(s.family, s.n, s.r, s.v, s.d, s.io_dtype, T, 1, head.W_emit, head.W_sum, head.T_static)
    weight = np.random.default_rng(5).normal(size=T).astype(np.float32)
    out = head.window_logprob_backward(torch.from_numpy(weight).cuda())
    assert head.head.mtpc_get_status() == 0
    ref = OG.window_logprob_grad(family, wl.hidden_q, U_q, wl.W_sum_q, None, wl.targets, weight)
    assert np.abs(out["logprob"].cpu().numpy() - ref["logprob"]).max() <= 2e-3
    dW, dA, dB = lowrank_backward(dA_, dB_, out["dW_emit"])
    chain = OG.lowrank_grad(W, A, Bm, ref["dW_emit"])
    for name, got, want in (("dW_base", dW, chain["dW_base"]), ("dA", dA, chain["dA"]), ("dB", dB, chain["dB"])):
        got = got.cpu().numpy().astype(np.float64)
        scale = np.abs(want).max()
        assert np.abs(got - want).max() <= 1e-2 * scale, name            # the bar of the head's own backward pass
        assert np.linalg.norm(got - want) <= 5e-3 * np.linalg.norm(want), name


def test_full_size_head_on_sampled_units():
    """The shape the benchmark times (the mixture head with n=8, r=16, v=320, d=4096; rank 16): whole units of the
    composed tensor and of the adaptor gradients, and one whole slot of the shared matrix's gradient, against the oracle
    run on those slices."""
    n, r, v, d, k = 8, 16, 320, 4096, 16
    W, A, Bm = I.lowrank_parameters(n, r, v, d, k, seed=97)
    dU = I.lowrank_upstream_gradient(n, r, v, d, seed=98)
    a_dev, b_dev = _device(A), _device(Bm)
    U = lowrank_compose(_device(W), a_dev, b_dev)
    dW, dA, dB = lowrank_backward(a_dev, b_dev, torch.from_numpy(dU).cuda())
    torch.cuda.synchronize()
    for (i, j) in [(0, 0), (3, 7), (7, 15)]:
        sl = (slice(i, i + 1), slice(j, j + 1))
        ref = OG.lowrank_grad(W[i:i + 1], A[sl], Bm[sl], dU[sl])
        got = U[i, j].float().cpu().numpy().astype(np.float64)
        assert np.all(np.abs(got - ref["U"][0, 0]) <= 2.0 ** -8 * np.abs(ref["U"][0, 0]) + 1e-7)
        exact = I.bf16_round(ref["U"][0, 0].astype(np.float32)).astype(np.float64)
        assert np.mean(got != exact) < 1e-3
        for name, dev, want in (("dA", dA[i, j], ref["dA"][0, 0]), ("dB", dB[i, j], ref["dB"][0, 0])):
            assert np.abs(dev.cpu().numpy().astype(np.float64) - want).max() <= 1e-5 * np.abs(want).max(), (name, i, j)
    i = 5
    ref = OG.lowrank_grad(W[i:i + 1], A[i:i + 1], Bm[i:i + 1], dU[i:i + 1])
    assert np.abs(dW[i].cpu().numpy().astype(np.float64) - ref["dW_base"][0]).max() <= 1e-5 * np.abs(ref["dW_base"]).max()


def test_argument_checks():
    n, r, v, d = 1, 1, 16, 64
    W, A, Bm = I.lowrank_parameters(n, r, v, d, 2, seed=1)
    a, b, w = _device(A), _device(Bm), _device(W)
    out = torch.empty((n, r, v, d), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.MtpcError) as e:
        B.mtpc_lowrank_compose(n, r, v, d, 65, w.data_ptr(), a.data_ptr(), b.data_ptr(), out.data_ptr())
    assert e.value.code == -3      # MTPC_ERR_UNSUPPORTED: rank above 64
    with pytest.raises(B.MtpcError) as e:
        B.mtpc_lowrank_compose(n, r, v, d, 0, w.data_ptr(), a.data_ptr(), b.data_ptr(), out.data_ptr())
    assert e.value.code == -2      # MTPC_ERR_SHAPE


# --------------------------------------------------------------------------- the factored head (no composed tensor)
FACTORED = [
    # family, n, r, v, vv, d, k, T
    (I.CP, 2, 4, 320, 0, 128, 16, 300),        # v = 320: the base in two 160-column halves, corrections in 96-column chunks
    (I.CP, 3, 16, 256, 0, 192, 16, 129),       # v = 256: one base box, 128-column chunks
    (I.HMM, 4, 8, 64, 0, 64, 32, 257),         # rank 32: two K steps per half
    (I.BTREE, 4, 4, 48, 44, 64, 16, 70),       # padded vocabulary, tree circuit
    (I.HMM_CTX, 3, 8, 320, 0, 128, 16, 200),   # contextual transitions: many sum tiles beside the factored projection
    (I.CP, 1, 1, 16, 0, 64, 16, 5),            # the smallest everything
    (I.CP, 2, 4, 480, 0, 64, 16, 140),         # three panels of 160 columns
    (I.HMM, 2, 4, 320, 306, 64, 16, 100),      # padded vocabulary, two panels, static transitions
    (I.CP, 1, 2, 1024, 1010, 64, 16, 40),      # eight panels of 128 columns
    (I.CP, 2, 4, 272, 268, 64, 16, 90),        # panels of 144 and 128 columns
    (I.CP, 1, 2, 1792, 0, 64, 16, 30),         # the widest unit: eight panels of 224 columns, one epilogue group, two-entry rings
    (I.HMM, 2, 4, 224, 0, 128, 32, 131),       # one panel of 224 columns, rank 32
]


def _factored_case(family, n, r, v, vv, d, k, T, seed):
    shape = I.HeadShape(family, n, r, v, d, v_valid=vv)
    wl = I.make_workload(f"lr_{family}_{v}_{k}", shape, T, seed=seed, weight_std=0.25)
    W, A, Bm = I.lowrank_parameters(n, r, v, d, k, seed=seed + 1, weight_std=0.25, adaptor_std=0.2)
    return wl, W, A, Bm


@pytest.mark.parametrize("family,n,r,v,vv,d,k,T", FACTORED)
def test_factored_head_matches_the_composed_definition(family, n, r, v, vv, d, k, T):
    """logit = W_i h + A_ij (B_ij h) evaluated without composing U: the window log-likelihood and the prefix marginals
    must equal the oracle's on U = W_i + A_ij B_ij (fp64, composed from the same bf16 parameters) within 2e-3."""
    wl, W, A, Bm = _factored_case(family, n, r, v, vv, d, k, T, seed=4100 + v + k + T)
    sym = vv or v
    U = O.lowrank_unembedding(W, A, Bm)[:, :, :sym, :]                     # the oracle never sees padding rows
    fam = wl.shape.family
    ref = O.window_logprob(fam, wl.hidden_q, U, wl.W_sum_q, wl.T_static, wl.targets)
    ctx = family == I.HMM_CTX
    W_sum = to_device_bf16(wl.W_sum_q)
    Ts = torch.from_numpy(np.ascontiguousarray(wl.T_static)).cuda() if wl.T_static is not None else None
    head = B.MtpcHead(B.MTPC_HMM if ctx else family, n, r, v, d, B.MTPC_BF16, T, 1, None, W_sum, Ts,
                      flags=B.MTPC_FLAG_HMM_CONTEXTUAL if ctx else 0, v_valid=vv, lowrank=(_device(W), _device(A), _device(Bm)))
    hidden = to_device_bf16(wl.hidden_q)
    t = wl.targets.copy()
    if T > 8 and n > 1:
        t[3, 1] = -1                                                       # a marginalised byte
        ref = O.window_logprob(fam, wl.hidden_q, U, wl.W_sum_q, wl.T_static, t)
    targets = torch.from_numpy(t).cuda()
    out = torch.empty(T, dtype=torch.float32, device="cuda")
    for _ in range(2):                                                     # twice: the accumulator ring wraps between calls
        head.mtpc_window_logprob(hidden, targets, out)
        assert head.mtpc_get_status() == 0
        err = np.abs(out.cpu().numpy() - ref).max()
        assert err <= 2e-3, err
    pre = torch.empty((T, n), dtype=torch.float32, device="cuda")
    head.mtpc_window_prefix_logprob(hidden, targets, pre)
    assert np.abs(pre[:, -1].cpu().numpy() - ref).max() <= 2e-3
    # what the factored head does not do is refused, not approximated: it drafts on the few-position path only
    # (tests/test_gpu_speculative.py checks those drafts), and has no backward pass
    # it drafts too, 128 positions at a time (tests/test_gpu_speculative.py checks drafts and acceptance); the backward call of a
    # head on a composed tensor is refused, not approximated
    u = wl.uniforms if wl.uniforms is not None else I.uniforms(I.BASE_SEED + 3, 5, (T, 2 * n))
    drafted = torch.empty((T, n), dtype=torch.int32, device="cuda")
    head.mtpc_draft_sample(hidden, 1, torch.from_numpy(np.ascontiguousarray(u[:T])).cuda(), drafted, out)
    assert head.mtpc_get_status() == 0
    d_ref = O.draft_sample(fam, wl.hidden_q, U, wl.W_sum_q, wl.T_static, 1, u[:T])
    differ = (drafted.cpu().numpy() != d_ref["bytes"]).any(axis=1)
    assert not (differ & (d_ref["margin"] >= 1e-6)).any()
    assert np.abs(out.cpu().numpy()[~differ] - d_ref["logprob"][~differ]).max() <= 2e-3
    with pytest.raises(B.MtpcError) as e:
        head.mtpc_window_logprob_backward(hidden, targets, torch.ones(T, device="cuda"), out, torch.empty((T, d), device="cuda"),
                                          torch.empty((n, r, v, d), device="cuda"), torch.empty((wl.W_sum_q.shape[0], d), device="cuda"),
                                          torch.empty((max(n - 1, 1), r, r), device="cuda"))
    assert e.value.code == -3
    head.mtpc_destroy()


def test_factored_head_agrees_with_the_dense_head_on_the_composed_tensor_and_refuses_other_ranks():
    family, n, r, v, d, k, T = I.CP, 2, 4, 320, 256, 16, 260
    wl, W, A, Bm = _factored_case(family, n, r, v, 0, d, k, T, seed=4999)
    Wd, Ad, Bd = _device(W), _device(A), _device(Bm)
    W_sum = to_device_bf16(wl.W_sum_q)
    hidden = to_device_bf16(wl.hidden_q)
    targets = torch.from_numpy(wl.targets).cuda()
    fact = B.MtpcHead(family, n, r, v, d, B.MTPC_BF16, T, 1, None, W_sum, None, lowrank=(Wd, Ad, Bd))
    U = lowrank_compose(Wd, Ad, Bd)                                        # bf16-rounded composition
    dense = B.MtpcHead(family, n, r, v, d, B.MTPC_BF16, T, 1, U, W_sum, None)
    a, b = torch.empty(T, device="cuda"), torch.empty(T, device="cuda")
    fact.mtpc_window_logprob(hidden, targets, a)
    dense.mtpc_window_logprob(hidden, targets, b)
    # the dense head computes on U rounded to bf16 (2^-9 relative per entry, d = 256 terms per logit): a looser agreement
    assert float((a - b).abs().max()) <= 5e-2
    exact = O.window_logprob(family, wl.hidden_q, O.lowrank_unembedding(W, A, Bm), wl.W_sum_q, None, wl.targets)
    assert np.abs(a.cpu().numpy() - exact).max() <= 2e-3
    assert np.abs(a.cpu().numpy() - exact).max() <= np.abs(b.cpu().numpy() - exact).max() + 1e-4
    fact.mtpc_destroy()
    dense.mtpc_destroy()
    cfg = B.MtpcConfig(family, n, r, v, d, B.MTPC_BF16, T, 1, 0, 0)
    import ctypes
    need = ctypes.c_size_t(0)
    assert B.lib().mtpc_lowrank_workspace_bytes(ctypes.byref(cfg), 8, ctypes.byref(need)) == -3      # rank not 16 or 32
    assert B.lib().mtpc_lowrank_workspace_bytes(ctypes.byref(cfg), 16, ctypes.byref(need)) == 0 and need.value > 0
    for bad_v in (40, 9616):        # 40: not a multiple of 16; 9616: more than eight panels
        big = B.MtpcConfig(family, n, r, bad_v, d, B.MTPC_BF16, T, 1, 0, 0)
        assert B.lib().mtpc_lowrank_workspace_bytes(ctypes.byref(big), 16, ctypes.byref(need)) == -3, bad_v


def test_a_wait_that_runs_out_in_the_factored_kernel_is_reported_and_the_head_recovers():
    """Both pipelines of the factored projection (base and corrections, each with its own producer and MMA issuer) give up
    at their first wait under a 50 ns limit: the status must say so, the context must stay usable, and the next call
    with the default limit must be right again."""
    family, n, r, v, d, k, T = I.CP, 3, 8, 320, 4096, 16, 400      # d = 4096: the first copies take longer than 64 polls
    wl, W, A, Bm = _factored_case(family, n, r, v, 0, d, k, T, seed=4500)
    head = B.MtpcHead(family, n, r, v, d, B.MTPC_BF16, T, 1, None, to_device_bf16(wl.W_sum_q), None,
                      lowrank=(_device(W), _device(A), _device(Bm)))
    hidden = to_device_bf16(wl.hidden_q)
    targets = torch.from_numpy(wl.targets).cuda()
    out = torch.empty(T, device="cuda")
    ref = O.window_logprob(family, wl.hidden_q, O.lowrank_unembedding(W, A, Bm), wl.W_sum_q, None, wl.targets)
    head.mtpc_window_logprob(hidden, targets, out)
    assert head.mtpc_get_status(with_code=True) == (B.MTPC_OK, 0)
    assert np.abs(out.cpu().numpy() - ref).max() <= 2e-3
    head.mtpc_debug_set_wait_limit_ns(50)
    head.mtpc_window_logprob(hidden, targets, out)            # gives up; outputs unspecified
    torch.cuda.synchronize()
    code, bits = head.mtpc_get_status(with_code=True)
    assert code == B.ERR_TIMEOUT and bits & B.STATUS_TIMEOUT
    head.mtpc_debug_set_wait_limit_ns(0)
    head.mtpc_window_logprob(hidden, targets, out)
    assert head.mtpc_get_status(with_code=True) == (B.MTPC_OK, 0)
    assert np.abs(out.cpu().numpy() - ref).max() <= 2e-3
    head.mtpc_destroy()


# --------------------------------------------------------------------------- training call of the factored head
def _check_tensor(name, got, ref, magnitude_sum, floor):
    """Entry by entry |got - ref| <= 2.2 * 2^-8 * (sum of the magnitudes of the products behind the entry) + floor: every
    product has at most two factors that the device rounded to bf16 (the logit gradient, and its sum over the components,
    its product with A, or the high half of B h); as a whole: relative L2 error below 1e-2."""
    got = got.cpu().numpy().astype(np.float64).reshape(ref.shape)
    assert np.isfinite(got).all(), name
    bound = 2.2 * 2.0 ** -8 * magnitude_sum.reshape(ref.shape) + floor
    excess = np.abs(got - ref) - bound
    worst = np.unravel_index(np.argmax(excess), excess.shape)
    assert excess[worst] <= 0, f"{name}: entry {worst} differs by {abs(got[worst] - ref[worst])}, bound {bound[worst]}"
    rel2 = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30)
    assert rel2 <= 1e-2 or np.abs(ref).max() < 100 * floor, f"{name}: relative L2 error {rel2}"
    return float((np.abs(got - ref) / bound).max()), rel2


@pytest.mark.parametrize("family,n,r,v,vv,d,k,T", [
    (I.CP, 2, 4, 320, 0, 128, 16, 300),        # two panels; v a multiple of 64
    (I.HMM, 4, 8, 64, 0, 64, 32, 257),         # rank 32, static transitions (dT_static)
    (I.BTREE, 4, 4, 48, 44, 64, 16, 70),       # padded vocabulary, v not a multiple of 64: the zero rows of the padded A
    (I.HMM_CTX, 3, 8, 320, 0, 128, 16, 200),   # contextual transitions: the sum units carry most of d hidden
    (I.CP, 2, 4, 272, 268, 64, 16, 90),        # ragged panels and a ragged K block per unit
    (I.CP, 1, 1, 16, 0, 64, 16, 5),
])
def test_factored_backward_is_the_chain_rule_through_the_composition(family, n, r, v, vv, d, k, T):
    """mtpc_lowrank_window_logprob_backward against the oracle: the gradient of sum_t weight[t] log q_t with respect to the
    exactly composed U (fp64), carried back to W_base, A and B by the oracle's reverse mode through U = W + A B."""
    wl, W, A, Bm = _factored_case(family, n, r, v, vv, d, k, T, seed=6100 + v + k + T)
    sym = vv or v
    fam = wl.shape.family
    U = O.lowrank_unembedding(W, A, Bm)[:, :, :sym, :]
    t = wl.targets.copy()
    if T > 8 and n > 1:
        t[3, 1] = -1
    weight = np.random.default_rng(T).normal(size=T).astype(np.float32)
    if T > 4:
        weight[2] = 0.0
    ref = OG.window_logprob_grad(fam, wl.hidden_q, U, wl.W_sum_q, wl.T_static, t, weight)
    dU = np.zeros((n, r, v, d))
    dU[:, :, :sym] = ref["dW_emit"]
    lr = OG.lowrank_grad(W, A, Bm, dU)
    ctx = family == I.HMM_CTX
    Ts = torch.from_numpy(np.ascontiguousarray(wl.T_static)).cuda() if wl.T_static is not None else None
    head = B.MtpcHead(B.MTPC_HMM if ctx else family, n, r, v, d, B.MTPC_BF16, T, 1, None, to_device_bf16(wl.W_sum_q), Ts,
                      flags=B.MTPC_FLAG_HMM_CONTEXTUAL if ctx else 0, v_valid=vv, lowrank=(_device(W), _device(A), _device(Bm)))
    f32 = dict(dtype=torch.float32, device="cuda")
    S = wl.W_sum_q.shape[0]
    out = dict(logprob=torch.empty(T, **f32), dh=torch.empty((T, d), **f32), dW_base=torch.empty((n, v, d), **f32),
               dA=torch.empty((n, r, v, k), **f32), dB=torch.empty((n, r, k, d), **f32), dW_sum=torch.empty((S, d), **f32),
               dT=torch.empty((max(n - 1, 1), r, r), **f32) if fam == I.HMM else None)
    hidden = to_device_bf16(wl.hidden_q)
    for _ in range(2):                       # twice: nothing of the first call may leak into the second
        head.mtpc_lowrank_window_logprob_backward(hidden, torch.from_numpy(t).cuda(), torch.from_numpy(weight).cuda(),
                                                  out["logprob"], out["dh"], out["dW_base"], out["dA"], out["dB"],
                                                  out["dW_sum"], out["dT"])
    assert head.mtpc_get_status() == 0
    assert np.abs(out["logprob"].cpu().numpy() - ref["logprob"]).max() <= 2e-3
    # magnitudes behind every entry, from the oracle's logit gradients
    lg = OG.window_logprob_logit_grad(fam, wl.hidden_q, U, wl.W_sum_q, wl.T_static, t, weight)
    g = np.zeros((T, n, r, v))
    g[..., :sym] = np.abs(lg["dlogit"]).reshape(T, n, r, sym)
    ds = np.abs(lg["dslog"]).reshape(T, -1)
    ah = np.abs(wl.hidden_q.astype(np.float64))
    aW, aA, aB = np.abs(W.astype(np.float64)), np.abs(A.astype(np.float64)), np.abs(Bm.astype(np.float64))
    gs = g.sum(axis=2)                                             # [T, n, v]
    gy = np.einsum("tijb,ijbq->tijq", g, aA)                       # [T, n, r, k]
    z = np.abs(np.einsum("ijqd,td->tijq", Bm.astype(np.float64), wl.hidden_q.astype(np.float64)))
    mags = dict(dh=np.einsum("tib,ibd->td", gs, aW) + np.einsum("tijq,ijqd->td", gy, aB) + ds @ np.abs(wl.W_sum_q.astype(np.float64)),
                dW_base=np.einsum("tib,td->ibd", gs, ah), dB=np.einsum("tijq,td->ijqd", gy, ah),
                dA=np.einsum("tijb,tijq->ijbq", g, z), dW_sum=ds.T @ ah)
    floor = 2e-5 * float(np.abs(weight).max()) * max(1.0, T ** 0.5)
    refs = dict(dh=ref["dh"], dW_base=lr["dW_base"], dA=lr["dA"], dB=lr["dB"], dW_sum=ref["dW_sum"])
    used = {name: _check_tensor(name, out[name], refs[name], mags[name], floor) for name in refs}
    if fam == I.HMM and n > 1:
        got = out["dT"][: n - 1].cpu().numpy().astype(np.float64)
        assert np.abs(got - ref["dT_static"]).max() <= 1e-2 * np.abs(ref["dT_static"]).max() + floor
    print(f"{wl.name}: share of the entry-wise bound used / relative L2: " + ", ".join(f"{n_} {u:.2f} / {l:.1e}" for n_, (u, l) in used.items()))
    # the padding rows of dA and dW_base receive no gradient
    if vv:
        assert float(out["dA"][:, :, vv:].abs().max()) <= floor and float(out["dW_base"][:, vv:].abs().max()) <= floor
    # the forward entry point still gives the same value
    fwd = torch.empty(T, **f32)
    head.mtpc_window_logprob(hidden, torch.from_numpy(t).cuda(), fwd)
    assert torch.equal(fwd, out["logprob"])
    head.mtpc_destroy()


def _whole_tensor(name, got, ref, floor):
    """Largest error below 1e-2 of the tensor's largest magnitude, relative L2 error below 1e-2 (two bf16-rounded factors
    per product)."""
    got = got.cpu().numpy().astype(np.float64).reshape(ref.shape)
    assert np.isfinite(got).all(), name
    scale = np.abs(ref).max()
    err = np.abs(got - ref).max()
    rel2 = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30)
    assert err <= 1e-2 * scale + floor, f"{name}: max error {err} against scale {scale}"
    assert rel2 <= 1e-2 or scale < 100 * floor, f"{name}: relative L2 error {rel2}"
    return err / max(scale, 1e-30), rel2


@pytest.mark.parametrize("family,n,r,v,d,k,N,L", [(I.CP, 4, 8, 320, 128, 16, 3, 50), (I.HMM, 8, 16, 64, 64, 16, 5, 33),
                                                   (I.HMM_CTX, 4, 8, 64, 64, 32, 4, 40), (I.BTREE, 8, 8, 32, 64, 16, 2, 140),
                                                   (I.HMM, 1, 4, 32, 64, 16, 2, 9)])
def test_eq6_loss_backward_on_a_factored_head(family, n, r, v, d, k, N, L):
    """The training loss of Eq. 6 and its gradients with respect to W_base, A and B, against reverse-mode differentiation of
    the definition on the exactly composed tensor, carried through U = W + A B. Windows run past the end of their sequences."""
    T = N * L
    wl, W, A, Bm = _factored_case(family, n, r, v, 0, d, k, T, seed=6400 + n + N + r)
    fam = wl.shape.family
    U = O.lowrank_unembedding(W, A, Bm)
    t = wl.targets.copy().reshape(N, L, n)
    for j in range(1, n):
        t[:, max(L - j, 0):, j] = -1
    if n > 1:
        t[0, :, n - 1] = -1
    t = t.reshape(T, n)
    gamma = 0.8
    ref = OG.composite_loss_grad(fam, wl.hidden_q, U, wl.W_sum_q, wl.T_static, t, N, gamma)
    lr = OG.lowrank_grad(W, A, Bm, ref["dW_emit"])
    ctx = family == I.HMM_CTX
    Ts = torch.from_numpy(np.ascontiguousarray(wl.T_static)).cuda() if wl.T_static is not None else None
    head = B.MtpcHead(B.MTPC_HMM if ctx else family, n, r, v, d, B.MTPC_BF16, T, 1, None, to_device_bf16(wl.W_sum_q), Ts,
                      flags=B.MTPC_FLAG_HMM_CONTEXTUAL if ctx else 0, lowrank=(_device(W), _device(A), _device(Bm)))
    f32 = dict(dtype=torch.float32, device="cuda")
    S = wl.W_sum_q.shape[0]
    slot, loss = torch.empty(n, **f32), torch.empty(1, **f32)
    out = dict(dh=torch.empty((T, d), **f32), dW_base=torch.empty((n, v, d), **f32), dA=torch.empty((n, r, v, k), **f32),
               dB=torch.empty((n, r, k, d), **f32), dW_sum=torch.empty((S, d), **f32))
    dT = torch.empty((max(n - 1, 1), r, r), **f32) if fam == I.HMM else None
    hidden = to_device_bf16(wl.hidden_q)
    td = torch.from_numpy(t).cuda()
    head.mtpc_lowrank_window_loss_backward(hidden, td, N, L, gamma, slot, loss, out["dh"], out["dW_base"], out["dA"], out["dB"],
                                           out["dW_sum"], dT)
    assert head.mtpc_get_status() == 0
    assert np.abs(slot.cpu().numpy() - ref["slot_loss"]).max() <= 2e-3
    assert abs(float(loss.cpu()[0]) - ref["loss"]) <= 2e-3 * n
    floor = 2e-5 / N * max(1.0, L ** 0.5)
    refs = dict(dh=ref["dh"], dW_base=lr["dW_base"], dA=lr["dA"], dB=lr["dB"], dW_sum=ref["dW_sum"])
    stats = {name: _whole_tensor(name, out[name], refs[name], floor) for name in refs}
    if fam == I.HMM and n > 1:
        stats["dT_static"] = _whole_tensor("dT_static", dT[: n - 1], ref["dT_static"], floor)
    print(f"{wl.name}: (max error / scale, relative L2): " + ", ".join(f"{n_} ({a:.1e}, {b:.1e})" for n_, (a, b) in stats.items()))
    # the forward-only entry point gives the same loss; the composed-tensor entry point refuses a factored head
    slot2, loss2 = torch.empty(n, **f32), torch.empty(1, **f32)
    head.mtpc_window_loss(hidden, td, N, L, gamma, slot2, loss2)
    assert torch.equal(slot, slot2) and torch.equal(loss, loss2)
    with pytest.raises(B.MtpcError) as e:
        head.mtpc_window_loss_backward(hidden, td, N, L, gamma, slot, loss, out["dh"], torch.empty((n, r, v, d), **f32), out["dW_sum"], dT)
    assert e.value.code == -3
    head.mtpc_destroy()


def test_factored_training_call_at_full_size_on_sampled_positions():
    """configs[1]'s shape, rank 16, the launch configuration the benchmark times (64 row tiles, 128 products per batched
    launch). The loss weights are non-zero on a seeded sample of positions, so every gradient is a sum over exactly those
    positions, which the oracle can afford; d hidden must vanish everywhere else. A second launch with every weight non-zero
    checks what holds at any size: the logit gradients of a unit sum to zero over its symbols, so dA summed over the symbols
    and dW_base summed over the symbols vanish."""
    wl = I.config_workload(1)
    s = wl.shape
    k = 16
    W, A, Bm = I.lowrank_parameters(s.n, s.r, s.v, s.d, k, seed=97)
    rng = np.random.default_rng(61)
    rows = np.unique(np.concatenate([[0, 127, 128, wl.T - 129, wl.T - 128, wl.T - 1], rng.choice(wl.T, 40, replace=False)]))
    weight = np.zeros(wl.T, dtype=np.float32)
    weight[rows] = rng.normal(size=len(rows)).astype(np.float32)
    U = O.lowrank_unembedding(W, A, Bm)
    ref = OG.window_logprob_grad(s.family, wl.hidden_q[rows], U, wl.W_sum_q, wl.T_static, wl.targets[rows], weight[rows])
    lr = OG.lowrank_grad(W, A, Bm, ref["dW_emit"])
    del U
    head = B.MtpcHead(s.family, s.n, s.r, s.v, s.d, B.MTPC_BF16, wl.T, 1, None, to_device_bf16(wl.W_sum_q), None,
                      lowrank=(_device(W), _device(A), _device(Bm)))
    f32 = dict(dtype=torch.float32, device="cuda")
    out = dict(logprob=torch.empty(wl.T, **f32), dh=torch.empty((wl.T, s.d), **f32), dW_base=torch.empty((s.n, s.v, s.d), **f32),
               dA=torch.empty((s.n, s.r, s.v, k), **f32), dB=torch.empty((s.n, s.r, k, s.d), **f32),
               dW_sum=torch.empty((wl.W_sum_q.shape[0], s.d), **f32))
    hidden = to_device_bf16(wl.hidden_q)
    targets = torch.from_numpy(wl.targets).cuda()
    call = lambda w: head.mtpc_lowrank_window_logprob_backward(hidden, targets, w, out["logprob"], out["dh"], out["dW_base"],
                                                               out["dA"], out["dB"], out["dW_sum"], None)
    call(torch.from_numpy(weight).cuda())
    assert head.mtpc_get_status() == 0
    floor = 2e-5 * float(np.abs(weight).max()) * len(rows) ** 0.5
    assert np.abs(out["logprob"].cpu().numpy()[rows] - ref["logprob"]).max() <= 2e-3
    got_dh = out["dh"].cpu().numpy()
    _whole_tensor("d_hidden", torch.from_numpy(got_dh[rows]), ref["dh"], floor)
    others = np.setdiff1d(np.arange(wl.T), rows)
    assert np.abs(got_dh[others]).max() == 0.0
    for name, want in (("dW_base", lr["dW_base"]), ("dA", lr["dA"]), ("dB", lr["dB"]), ("dW_sum", ref["dW_sum"])):
        _whole_tensor(name, out[name], want, floor)
    call(torch.full((wl.T,), -1.0 / wl.T, device="cuda"))
    assert head.mtpc_get_status() == 0
    dA, dWb = out["dA"], out["dW_base"]
    assert float(dA.abs().max()) > 0 and torch.isfinite(out["dh"]).all() and torch.isfinite(out["dB"]).all()
    # sum over the symbols b of g[t, i, j, b] = 0  =>  sum_b dW_base[i, b, :] = 0; dA[i, j, b, :] = sum_t g z sums to 0 over b
    assert float(dWb.sum(dim=1).abs().max()) <= 2e-2 * float(dWb.abs().max())
    assert float(dA.sum(dim=2).abs().max()) <= 2e-2 * float(dA.abs().max())
    head.mtpc_destroy()


@pytest.mark.parametrize("family,n,r,v,d,k,P,wpp", [
    (I.HMM, 4, 8, 48, 64, 16, 300, 1),         # one window per position: every (window, slot) forms its one unit's logits
    (I.BTREE, 4, 4, 32, 64, 32, 200, 1),
    (I.HMM_CTX, 3, 4, 320, 64, 16, 130, 1),    # two panels in the evidence pass
    (I.CP, 3, 8, 64, 64, 16, 150, 2),          # two windows per position: the few-position path, 128 positions at a time
])
def test_long_drafts_on_a_factored_head(family, n, r, v, d, k, P, wpp):
    """More positions than the few-position path takes (Algorithm 1 on a verification batch): bytes and log-probs against the
    oracle on the exactly composed tensor; refused draws keep their meaning (byte -1, log-prob NaN, status bit)."""
    wl = I.make_workload(f"lr_long_{family}_{n}_{r}", I.HeadShape(family, n, r, v, d), P, seed=6600 + n + r + v + P, wpp=wpp,
                         weight_std=0.25)
    W_, A, Bm = I.lowrank_parameters(n, r, v, d, k, seed=6700 + n + r, weight_std=0.25, adaptor_std=0.2)
    U = O.lowrank_unembedding(W_, A, Bm)
    fam = wl.shape.family
    dh = DeviceHead(wl, lowrank=(W_, A, Bm))
    u = wl.uniforms.copy()
    u[5, n + 1 if n > 1 else n] = 2.0          # a refused byte draw ...
    u[9, 0] = -1.0                             # ... and a refused latent draw
    out_bytes, out_lp = dh.draft_sample(uniforms=torch.from_numpy(u).cuda())
    assert dh.head.mtpc_get_status(with_code=True) == (B.MTPC_OK, B.STATUS_BAD_UNIFORM)
    gb, gl = out_bytes.cpu().numpy(), out_lp.cpu().numpy()
    assert gb[5, 1 if n > 1 else 0] == -1 and (gb[9] == -1).all() and np.isnan(gl[5]) and np.isnan(gl[9])
    ok = np.ones(len(gb), dtype=bool)
    ok[[5, 9]] = False
    ref = O.draft_sample(fam, wl.hidden_q, U, wl.W_sum_q, wl.T_static, wpp, wl.uniforms)
    differ = (gb != ref["bytes"]).any(axis=1) & ok
    assert not (differ & (ref["margin"] >= 1e-6)).any()
    same = ok & ~differ
    assert np.abs(gl[same] - ref["logprob"][same]).max() <= 2e-3
    # prefix marginals of the same draft
    b2, pre = dh.draft_sample_prefix()
    assert torch.equal(b2, dh.draft_sample()[0])
    want = O.prefix_logprob(fam, O.head_logw(fam, wl.hidden_q, wl.W_sum_q, wl.T_static, r), O.emission_logphi(wl.hidden_q, U),
                            wl.T_static, b2.cpu().numpy(), np.repeat(np.arange(P), wpp))
    assert np.abs(pre.cpu().numpy() - want).max() <= 2e-3
    if wpp > 1:                                # drafted 128 positions at a time: only the last chunk's logits remain
        W = P * wpp
        with pytest.raises(B.MtpcError) as e:
            dh.head.mtpc_speculative_accept(P, wpp, b2, pre, torch.zeros((W, n + 1, v), device="cuda"),
                                            torch.zeros((W, n + 1), device="cuda"), torch.empty(W, dtype=torch.int32, device="cuda"),
                                            torch.empty(W, dtype=torch.int32, device="cuda"))
        assert e.value.code == B.ERR_STATE
    dh.close()
