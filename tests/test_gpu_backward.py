"""GPU parity of the backward pass: gradients of sum_t weight[t] log q_t from the CUDA path (C ABI) against the fp64
gradient oracle on the same seeded inputs.

Bar. The forward value keeps the 2e-3 bar. The device rounds the gradient of the logits to bf16 (8 significant bits:
relative error at most 2^-8 per element) before the weight-sized GEMMs, which accumulate in fp32. Two checks per gradient tensor:
  - entry by entry: a gradient entry is a sum of products (dW[c, j] = sum_t dlogit[t, c] h[t, j], and so on); rounding
    one factor of every product to bf16 can move the sum by at most 2^-8 times the sum of the products' magnitudes, which
    the oracle gives (|dlogit|^T |h|). Every entry must lie within 1.1 x that bound (fp32 accumulation and the fp32
    circuit arithmetic take the rest) plus a floor for entries that are exactly zero in exact arithmetic;
  - as a whole: relative L2 error below 5e-3, largest error below 1e-2 of the tensor's largest magnitude."""
import numpy as np
import pytest
import torch

from oracle import mtpc_oracle_grad as og
from paper_2511_11346_b200 import inputs as I
from paper_2511_11346_b200.runner import DeviceHead

pytestmark = pytest.mark.gpu

SMALL = [
    # family, n, r, v, d, T
    (I.CP, 1, 1, 16, 64, 3),
    (I.CP, 3, 2, 48, 128, 129),
    (I.CP, 5, 4, 320, 192, 300),
    (I.CP, 2, 128, 16, 64, 37),
    (I.HMM, 1, 4, 32, 64, 7),
    (I.HMM, 6, 8, 64, 128, 257),
    (I.HMM, 4, 32, 320, 64, 64),
    (I.HMM, 3, 1, 16, 64, 3),
    (I.HMM_CTX, 6, 8, 64, 128, 257),
    (I.HMM_CTX, 4, 32, 320, 64, 64),
    (I.HMM_CTX, 3, 2, 16, 64, 5),
    (I.BTREE, 2, 4, 32, 64, 9),
    (I.BTREE, 4, 16, 256, 128, 130),
    (I.BTREE, 8, 32, 48, 64, 33),
    (I.BTREE, 16, 8, 32, 64, 70),
    (I.BTREE, 64, 2, 16, 64, 3),
    (I.BTREE, 64, 32, 16, 64, 9),          # long windows: fewer warps per CTA so that the messages still fit shared memory
    (I.HMM, 32, 16, 16, 64, 11),
    (I.HMM_CTX, 64, 32, 16, 64, 4),
]


def check(name, got, ref, floor):
    """floor: absolute slack for tensors that are exactly zero in exact arithmetic (e.g. a sum unit with one input,
    whose posterior minus prior is 1 - 1): fp32 rounding of order 1e-6 per position, times the weights."""
    got = got.cpu().numpy().astype(np.float64)
    scale = np.abs(ref).max()
    assert np.isfinite(got).all(), name
    err = np.abs(got - ref).max()
    rel2 = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30)
    assert err <= 1e-2 * scale + floor, f"{name}: max error {err} against scale {scale}"
    assert rel2 <= 5e-3 or scale < 100 * floor, f"{name}: relative L2 error {rel2}"
    return err / max(scale, 1e-30), rel2


BF16_UNIT_ROUNDOFF = 2.0 ** -8      # 8 significant bits, round to nearest


def check_entries(name, got, ref, magnitude_sum, floor):
    """|got - ref| <= 1.1 * 2^-8 * (sum of the magnitudes of the products behind the entry) + floor, entry by entry."""
    got = got.cpu().numpy().astype(np.float64).reshape(ref.shape)
    bound = 1.1 * BF16_UNIT_ROUNDOFF * magnitude_sum.reshape(ref.shape) + floor
    excess = np.abs(got - ref) - bound
    worst = np.unravel_index(np.argmax(excess), excess.shape)
    assert excess[worst] <= 0, (f"{name}: entry {worst} differs by {abs(got[worst] - ref[worst])}, bound {bound[worst]} "
                                f"(value {ref[worst]})")
    return float((np.abs(got - ref) / bound).max())


def entry_bounds(family, wl, targets, weight):
    """Sums of |products| behind every entry of dh, dW_emit and dW_sum, from the oracle's logit gradients."""
    s = wl.shape
    lg = og.window_logprob_logit_grad(family, wl.hidden_q, wl.W_emit_q, wl.W_sum_q, wl.T_static, targets, weight)
    T = wl.hidden_q.shape[0]
    vv = wl.W_emit_q.shape[2]
    dl = np.abs(lg["dlogit"]).reshape(T, s.n * s.r * vv)
    ds = np.abs(lg["dslog"]).reshape(T, -1)
    ah = np.abs(wl.hidden_q.astype(np.float64))
    aW = np.abs(wl.W_emit_q.astype(np.float64)).reshape(s.n * s.r * vv, s.d)
    aR = np.abs(wl.W_sum_q.astype(np.float64))
    return dict(dh=dl @ aW + ds @ aR, dW_emit=(dl.T @ ah).reshape(s.n, s.r, vv, s.d), dW_sum=ds.T @ ah)


@pytest.mark.parametrize("family,n,r,v,d,T", SMALL)
def test_backward_small_shapes(family, n, r, v, d, T):
    wl = I.make_workload(f"bwd_{family}_{n}_{r}_{v}", I.HeadShape(family, n, r, v, d), T, seed=5000 + 3 * n + r + v + T,
                         weight_std=0.25)
    t = wl.targets.copy()
    if T > 4 and n > 1:
        t[1, n // 2:] = -1                                  # marginalised bytes: no gradient through them
        t[2, 0] = -1
    rng = np.random.default_rng(T)
    weight = rng.normal(size=T).astype(np.float32)
    if T > 4:
        weight[3] = 0.0                                      # a masked position
    dh = DeviceHead(wl)
    out = dh.window_logprob_backward(torch.from_numpy(weight).cuda(), targets=torch.from_numpy(t).cuda())
    assert dh.head.mtpc_get_status() == 0
    ref = og.window_logprob_grad(family, wl.hidden_q, wl.W_emit_q, wl.W_sum_q, wl.T_static, t, weight)
    assert np.abs(out["logprob"].cpu().numpy() - ref["logprob"]).max() <= 2e-3
    floor = 2e-5 * float(np.abs(weight).max()) * max(1.0, T ** 0.5)
    stats = [check("d_hidden", out["dh"], ref["dh"], floor), check("dW_emit", out["dW_emit"], ref["dW_emit"], floor),
             check("dW_sum", out["dW_sum"], ref["dW_sum"], floor)]
    if family == I.HMM and n > 1:
        stats.append(check("dT_static", out["dT_static"][: n - 1], ref["dT_static"], floor))
    bounds = entry_bounds(family, wl, t, weight)
    used = [check_entries(k, out[k], ref[k], bounds[k], floor) for k in ("dh", "dW_emit", "dW_sum")]
    print(f"{wl.name}: (max error / scale, relative L2) per tensor: " + ", ".join(f"({a:.1e}, {b:.1e})" for a, b in stats)
          + "; largest share of the entry-wise bound used: " + ", ".join(f"{u:.2f}" for u in used))
    # the forward entry point still gives the same value after a backward call
    fwd = dh.window_logprob(targets=torch.from_numpy(t).cuda())
    assert torch.equal(fwd, out["logprob"])
    dh.close()


@pytest.mark.parametrize("idx,nsample", [(1, 48), (3, 24)])
def test_backward_full_size_configs_on_sampled_positions(idx, nsample):
    """Full-size launch (the configuration the benchmark times). The loss weights are non-zero on a seeded sample of
    positions only, so the weight gradients are sums over exactly those positions, which the oracle can afford; the
    gradient of the hidden states must vanish everywhere else. Properties that hold at any size are checked on a
    second launch with every weight non-zero: the logit gradients of an input unit sum to zero over the bytes, so
    dW_emit summed over the bytes of a unit is zero, and likewise dW_sum summed over the inputs of a sum unit."""
    wl = I.config_workload(idx)
    s = wl.shape
    rng = np.random.default_rng(60 + idx)
    rows = np.unique(np.concatenate([[0, 127, 128, wl.T - 129, wl.T - 128, wl.T - 1],
                                     rng.choice(wl.T, nsample, replace=False)]))
    weight = np.zeros(wl.T, dtype=np.float32)
    weight[rows] = rng.normal(size=len(rows)).astype(np.float32)
    dh = DeviceHead(wl)
    out = dh.window_logprob_backward(torch.from_numpy(weight).cuda())
    assert dh.head.mtpc_get_status() == 0
    ref = og.window_logprob_grad(s.family, wl.hidden_q[rows], wl.W_emit_q, wl.W_sum_q, wl.T_static, wl.targets[rows],
                                 weight[rows])
    floor = 2e-5 * float(np.abs(weight).max()) * len(rows) ** 0.5
    got_dh = out["dh"].cpu().numpy()
    assert np.abs(out["logprob"].cpu().numpy()[rows] - ref["logprob"]).max() <= 2e-3
    check("d_hidden", torch.from_numpy(got_dh[rows]), ref["dh"], floor)
    others = np.setdiff1d(np.arange(wl.T), rows)
    assert np.abs(got_dh[others]).max() == 0.0
    check("dW_emit", out["dW_emit"], ref["dW_emit"], floor)
    check("dW_sum", out["dW_sum"], ref["dW_sum"], floor)
    del ref
    # every position weighted: sums over the bytes of a unit / the inputs of a sum unit vanish
    weight_all = torch.full((wl.T,), -1.0 / wl.T, device="cuda")
    out = dh.window_logprob_backward(weight_all)
    assert dh.head.mtpc_get_status() == 0
    dW = out["dW_emit"]
    scale = float(dW.abs().max())
    assert scale > 0 and float(dW.sum(dim=2).abs().max()) <= 2e-2 * scale
    dR = out["dW_sum"].reshape(-1, s.r, s.d)
    assert float(dR.sum(dim=1).abs().max()) <= 2e-2 * float(dR.abs().max()) + 1e-9
    assert torch.isfinite(out["dh"]).all() and float(out["dh"].abs().max()) > 0
    dh.close()


@pytest.mark.parametrize("family,n,r,v,d,T", [(I.CP, 2, 2, 1024, 64, 130), (I.HMM, 2, 4, 2048, 64, 70),
                                               (I.BTREE, 4, 4, 4112, 64, 33), (I.CP, 1, 1, 32768, 64, 5)])
def test_large_vocabulary_heads_evaluate_train_and_draft(family, n, r, v, d, T):
    """More than 512 symbols: a unit's logits no longer fit tensor memory at once; the softmax runs online across the
    accumulator tiles (log-likelihood, prefix marginals, backward), and the draft streams a unit's tiles twice."""
    from oracle import mtpc_oracle as orc
    from paper_2511_11346_b200 import binding as B
    wl = I.make_workload(f"bigv_{family}_{v}", I.HeadShape(family, n, r, v, d), T, seed=7000 + v + T, wpp=1, weight_std=0.25)
    dh = DeviceHead(wl)
    got = dh.window_logprob().cpu().numpy()
    ref = orc.window_logprob(family, wl.hidden_q, wl.W_emit_q, wl.W_sum_q, wl.T_static, wl.targets)
    assert np.abs(got - ref).max() <= 2e-3
    pre = dh.window_prefix_logprob().cpu().numpy()
    assert np.abs(pre - orc.window_prefix_logprob(family, wl.hidden_q, wl.W_emit_q, wl.W_sum_q, wl.T_static, wl.targets)).max() <= 2e-3
    weight = np.random.default_rng(v).normal(size=T).astype(np.float32)
    out = dh.window_logprob_backward(torch.from_numpy(weight).cuda())
    assert dh.head.mtpc_get_status() == 0
    g = og.window_logprob_grad(family, wl.hidden_q, wl.W_emit_q, wl.W_sum_q, wl.T_static, wl.targets, weight)
    floor = 2e-5 * float(np.abs(weight).max()) * T ** 0.5
    check("d_hidden", out["dh"], g["dh"], floor)
    check("dW_emit", out["dW_emit"], g["dW_emit"], floor)
    check("dW_sum", out["dW_sum"], g["dW_sum"], floor)
    out_bytes, out_lp = dh.draft_sample(1)
    assert dh.head.mtpc_get_status() == 0
    d_ref = orc.draft_sample(family, wl.hidden_q, wl.W_emit_q, wl.W_sum_q, wl.T_static, 1, wl.uniforms)
    differ = (out_bytes.cpu().numpy() != d_ref["bytes"]).any(axis=1)
    assert not (differ & (d_ref["margin"] >= 1e-6)).any()
    assert np.abs(out_lp.cpu().numpy()[~differ] - d_ref["logprob"][~differ]).max() <= 2e-3
    dh.close()


def test_backward_refuses_what_does_not_fit_shared_memory():
    from paper_2511_11346_b200 import binding as B
    # static transitions: the per-CTA accumulator of the transition gradients alone is (n-1) r^2 floats = 258 KB here
    wl = I.make_workload("bwd_big", I.HeadShape(I.HMM, 64, 32, 16, 64), 4, seed=13, weight_std=0.3)
    dh = DeviceHead(wl)
    with pytest.raises(B.MtpcError) as e:
        dh.window_logprob_backward(torch.ones(4, device="cuda"))
    assert e.value.code == -3
    assert np.isfinite(dh.window_logprob().cpu().numpy()).all()      # the forward path is unaffected
    dh.close()


def test_backward_argument_checks():
    import ctypes
    from paper_2511_11346_b200 import binding as B
    wl = I.make_workload("bwd_args", I.HeadShape(I.HMM, 3, 4, 32, 64), 10, seed=12, weight_std=0.3)
    dh = DeviceHead(wl)
    lib = B.lib()
    need = ctypes.c_size_t(0)
    assert lib.mtpc_backward_workspace_bytes(ctypes.byref(dh.head.cfg), 10, ctypes.byref(need)) == 0 and need.value % 256 == 0
    assert lib.mtpc_backward_workspace_bytes(ctypes.byref(dh.head.cfg), 0, ctypes.byref(need)) == -2
    assert lib.mtpc_backward_workspace_bytes(None, 10, ctypes.byref(need)) == -1
    lib.mtpc_backward_workspace_bytes(ctypes.byref(dh.head.cfg), 10, ctypes.byref(need))
    s = wl.shape
    f32 = dict(dtype=torch.float32, device="cuda")
    h, t = dh.hidden_device(), torch.from_numpy(wl.targets).cuda()
    w = torch.ones(10, **f32)
    ws = torch.empty(need.value, dtype=torch.uint8, device="cuda")
    lp, dhid = torch.empty(10, **f32), torch.empty((10, s.d), **f32)
    dW, dR, dT = torch.empty((s.n, s.r, s.v, s.d), **f32), torch.empty((s.sum_rows, s.d), **f32), torch.empty((2, 4, 4), **f32)
    st = torch.cuda.current_stream().cuda_stream
    call = lambda **kw: lib.mtpc_window_logprob_backward(
        dh.head.handle, kw.get("h", h.data_ptr()), t.data_ptr(), kw.get("T", 10), w.data_ptr(), kw.get("ws", ws.data_ptr()),
        kw.get("wsb", need.value), lp.data_ptr(), dhid.data_ptr(), dW.data_ptr(), dR.data_ptr(), kw.get("dT", dT.data_ptr()), st)
    assert call() == 0
    assert call(T=0) == 0
    assert call(T=11) == -2                     # more positions than the head was created for
    assert call(h=None) == -1
    assert call(dT=None) == -1                  # a static HMM needs room for the transition gradients
    assert call(wsb=need.value - 256) == -4     # workspace too small
    assert call(ws=ws.data_ptr() + 8) == -4     # misaligned
    torch.cuda.synchronize()
    assert dh.head.mtpc_get_status() == 0
    dh.close()


@pytest.mark.parametrize("family,n,r,v,d,N,L", [(I.CP, 4, 8, 320, 128, 3, 50), (I.CP, 2, 128, 16, 64, 5, 7),
                                                 (I.HMM, 8, 16, 64, 64, 5, 33), (I.HMM, 1, 4, 32, 64, 2, 9),
                                                 (I.HMM_CTX, 4, 8, 64, 64, 4, 40), (I.BTREE, 8, 8, 32, 64, 2, 140),
                                                 (I.BTREE, 2, 4, 32, 64, 3, 11), (I.BTREE, 16, 16, 48, 64, 2, 40),
                                                 (I.HMM, 3, 1, 16, 64, 2, 5), (I.HMM, 16, 32, 32, 64, 2, 20),
                                                 (I.HMM, 5, 2, 16, 64, 3, 7), (I.HMM_CTX, 3, 2, 16, 64, 3, 7),
                                                 (I.HMM_CTX, 6, 32, 32, 64, 2, 17), (I.HMM_CTX, 1, 4, 32, 64, 2, 9)])
def test_eq6_loss_backward_matches_oracle(family, n, r, v, d, N, L):
    """The training loss of Eq. 6 and its gradients (mixture and tree: one circuit backward pass per prefix length,
    accumulated; HMM: every prefix is a forward message, one reverse sweep), against
    reverse-mode differentiation of the definition in float64. Windows run past the end of their sequences (masked
    tails), one sequence has no valid byte in the last slot."""
    wl = I.make_workload(f"l6_{family}_{n}_{r}", I.HeadShape(family, n, r, v, d), N * L, seed=6000 + n + N + r, weight_std=0.25)
    t = wl.targets.copy().reshape(N, L, n)
    for j in range(1, n):
        t[:, max(L - j, 0):, j] = -1
    if n > 1:
        t[0, :, n - 1] = -1
    t = t.reshape(N * L, n)
    gamma = 0.8
    dh = DeviceHead(wl)
    out = dh.window_loss_backward(N, L, gamma, targets=torch.from_numpy(t).cuda())
    assert dh.head.mtpc_get_status() == 0
    ref = og.composite_loss_grad(family, wl.hidden_q, wl.W_emit_q, wl.W_sum_q, wl.T_static, t, N, gamma)
    assert np.abs(out["slot_loss"].cpu().numpy() - ref["slot_loss"]).max() <= 2e-3
    assert abs(float(out["loss"].cpu()[0]) - ref["loss"]) <= 2e-3 * n
    floor = 2e-5 / N * max(1.0, L ** 0.5)
    stats = [check("d_hidden", out["dh"], ref["dh"], floor), check("dW_emit", out["dW_emit"], ref["dW_emit"], floor),
             check("dW_sum", out["dW_sum"], ref["dW_sum"], floor)]
    if family == I.HMM and n > 1:
        stats.append(check("dT_static", out["dT_static"][: n - 1], ref["dT_static"], floor))
    print(f"{wl.name}: (max error / scale, relative L2) per tensor: " + ", ".join(f"({a:.1e}, {b:.1e})" for a, b in stats))
    # same loss value as the forward-only entry point
    slot, loss = dh.window_loss(N, L, gamma, targets=torch.from_numpy(t).cuda())
    assert torch.equal(slot, out["slot_loss"]) and torch.equal(loss, out["loss"])
    dh.close()


def test_per_kernel_timing_of_the_training_calls():
    wl = I.make_workload("timing", I.HeadShape(I.BTREE, 4, 8, 32, 64), 40, seed=14, wpp=2, weight_std=0.3)
    dh = DeviceHead(wl)
    head = dh.head
    head.mtpc_set_timing(4)
    w = torch.ones(40, device="cuda")
    dh.window_logprob_backward(w)
    ph = head.mtpc_get_timing(0)
    assert len(ph) == 4 and all(p > 0 for p in ph)            # forward, circuit backward, logit gradients, GEMMs
    dh.window_loss_backward(4, 10, 0.8)
    ph = head.mtpc_get_timing(0)
    assert len(ph) == 4 and all(p > 0 for p in ph)            # forward+prefix+loss, the n circuit passes, projection, GEMMs
    assert len(head.mtpc_get_timing(1)) == 4                  # the call before is still in the ring
    b, pre = dh.draft_sample_prefix(2)
    assert len(head.mtpc_get_timing(0)) == 3                  # few-position draft: weight pass, per-slot kernel, circuit
    p = torch.from_numpy(I.target_rows(1, 1, (80, 5, 32))).cuda()
    u = torch.from_numpy(I.uniforms(1, 2, (80, 5))).cuda()
    dh.speculative_accept(40, 2, b, pre, p, u)
    assert len(head.mtpc_get_timing(0)) == 1
    head.mtpc_set_timing(0)
    assert head.mtpc_get_timing(0) == []
    assert dh.head.mtpc_get_status() == 0
    dh.close()


@pytest.mark.parametrize("family,io", [(I.HMM, I.BF16), (I.HMM_CTX, I.BF16), (I.CP, I.F32), (I.BTREE, I.BF16)])
def test_update_parameters_after_an_optimiser_step(family, io):
    """A training loop changes the parameters between calls: in place (bf16 heads read the weights where they are) or
    in new buffers. After mtpc_update_parameters the head computes on the new values - weights, static transitions
    or transition bias, fp32 weights re-rounded - and a draft made with the old ones can no longer be accepted."""
    n, r, v, d, T = 4, 8, 64, 128, 70
    old = I.make_workload("upd_old", I.HeadShape(family, n, r, v, d, io), T, seed=311, weight_std=0.25)
    new = I.make_workload("upd_new", I.HeadShape(family, n, r, v, d, io), T, seed=312, weight_std=0.25)
    dh = DeviceHead(old)
    from oracle import mtpc_oracle as O
    ref_old = O.window_logprob(family, old.hidden_q, old.W_emit_q, old.W_sum_q, old.T_static, old.targets)
    assert np.abs(dh.window_logprob().cpu().numpy() - ref_old).max() <= 2e-3
    fresh = DeviceHead(new)                                     # only to have the new parameters on the device
    h_new, t_new = fresh.hidden_device(), torch.from_numpy(new.targets).cuda()
    ref_new = O.window_logprob(family, new.hidden_q, new.W_emit_q, new.W_sum_q, new.T_static, new.targets)
    # (1) in place: overwrite the tensors the head was created on
    dh.W_emit.copy_(fresh.W_emit)
    dh.W_sum.copy_(fresh.W_sum)
    if dh.T_static is not None:
        dh.T_static.copy_(fresh.T_static)
    dh.head.mtpc_update_parameters(dh.W_emit, dh.W_sum, dh.T_static)
    assert np.abs(dh.window_logprob(hidden=h_new, targets=t_new).cpu().numpy() - ref_new).max() <= 2e-3
    # (2) other buffers: back to the old values, held in clones
    back = DeviceHead(old)
    dh.head.mtpc_update_parameters(back.W_emit, back.W_sum, back.T_static)
    assert np.abs(dh.window_logprob().cpu().numpy() - ref_old).max() <= 2e-3
    assert dh.head.mtpc_get_status() == 0
    # gradients follow the bound parameters too
    w = torch.full((T,), 1.0 / T, device="cuda")
    g = dh.window_logprob_backward(w)
    ref = og.window_logprob_grad(family, old.hidden_q, old.W_emit_q, old.W_sum_q, old.T_static, old.targets,
                                 np.full(T, 1.0 / T, dtype=np.float32))
    check("dW_emit after update", g["dW_emit"], ref["dW_emit"], 0.0)
    for x in (dh, fresh, back):
        x.close()


def test_update_parameters_forgets_the_draft():
    from paper_2511_11346_b200 import binding as B
    wl = I.make_workload("upd_draft", I.HeadShape(I.CP, 4, 8, 64, 128), 8, seed=77, wpp=4, weight_std=0.25)
    dh = DeviceHead(wl, max_wpp=4)
    bytes_, lq = dh.draft_sample_prefix(wpp=4)
    dh.head.mtpc_update_parameters(dh.W_emit, dh.W_sum, dh.T_static)
    p = torch.full((8 * 4, 5, 64), 1.0 / 64, device="cuda")
    u = torch.full((8 * 4, 5), 0.5, device="cuda")
    with pytest.raises(B.MtpcError) as e:
        dh.speculative_accept(8, 4, bytes_, lq, p, u)
    assert e.value.code == B.ERR_STATE
    dh.close()


@pytest.mark.parametrize("family", [I.CP, I.HMM, I.BTREE])
def test_gradient_descent_on_the_device_gradients_lowers_the_loss(family):
    """Ten plain SGD steps on the Eq. 6 loss with the gradients of mtpc_window_loss_backward (fp32 master weights kept by
    the test, rounded to bf16 into the head's buffers, mtpc_update_parameters after each step): the loss the device
    reports must fall at every step, and the fp64 oracle must agree with the last one."""
    from oracle import mtpc_oracle as O
    from paper_2511_11346_b200.runner import to_device_bf16
    n, r, v, d, N, L = 4, 4, 32, 64, 3, 40
    T = N * L
    wl = I.make_workload("sgd", I.HeadShape(family, n, r, v, d), T, seed=900 + family, target_kind="zipf", weight_std=0.1)
    dh = DeviceHead(wl)
    master = [dh.W_emit.float().clone(), dh.W_sum.float().clone(), None if dh.T_static is None else dh.T_static.clone()]
    gamma, lr = 0.8, 2.0
    losses = []
    for step in range(10):
        g = dh.window_loss_backward(N, L, gamma)
        losses.append(float(g["loss"].cpu()[0]))
        master[0] -= lr * g["dW_emit"]
        master[1] -= lr * g["dW_sum"]
        dh.W_emit.copy_(master[0].to(torch.bfloat16))
        dh.W_sum.copy_(master[1].to(torch.bfloat16))
        if master[2] is not None:
            master[2] -= lr * g["dT_static"]
            dh.T_static.copy_(master[2])
        dh.head.mtpc_update_parameters(dh.W_emit, dh.W_sum, dh.T_static)
    slot, loss = dh.window_loss(N, L, gamma)
    losses.append(float(loss.cpu()[0]))
    assert dh.head.mtpc_get_status() == 0
    assert all(b < a for a, b in zip(losses, losses[1:])), losses
    assert losses[-1] < 0.9 * losses[0], losses
    We = dh.W_emit.float().cpu().numpy().astype(np.float64)
    Ws = dh.W_sum.float().cpu().numpy().astype(np.float64)
    Ts = None if dh.T_static is None else dh.T_static.cpu().numpy().astype(np.float64)
    pre = O.window_prefix_logprob(family, wl.hidden_q, We, Ws, Ts, wl.targets)
    _, ref = O.composite_loss(pre, wl.targets, N, gamma)
    assert abs(losses[-1] - ref) <= 2e-3 * n, (losses[-1], ref)
    dh.close()
