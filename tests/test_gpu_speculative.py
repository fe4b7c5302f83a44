"""GPU parity of the prefix log-marginals, the acceptance stage of Algorithm 3 and the Eq. 6 loss: the CUDA path,
called through the C ABI, against the fp64 oracle on the same seeded inputs.

Bars. Prefix log-marginals and per-slot losses: 2e-3 absolute (the window log-prob bar). Acceptance: the number of
accepted bytes and the next byte are compared exactly for every window whose draft bytes agree with the oracle's and
whose decisions all lie outside a band around the oracle's decision boundaries; windows inside the band are
counted and printed. The bands follow from the arithmetic: the device's conditional q(x_i | ..) carries the fp32
error of two log-probs (<= 1e-4 each over n <= 16 slots), so an acceptance ratio <= 1 moves by < 2e-4; the residual
weights max(0, p - q) carry the same relative error of q, so the normalised residual CDF moves by < 1e-4 / Z."""
import numpy as np
import pytest
import torch

from oracle import mtpc_oracle as orc
from paper_2511_11346_b200 import binding as B
from paper_2511_11346_b200 import inputs as I
from paper_2511_11346_b200.runner import DeviceHead

pytestmark = pytest.mark.gpu

LOGPROB_TOL = 2e-3
BOUNDARY_BAND = 1e-6       # draft draws (as in test_gpu_parity.py)
OWN_ALPHA_BAND = 1e-5
ALPHA_BAND = 2e-4          # |alpha - p/q| of an acceptance test
FINAL_BAND = 1e-4          # distance of the last draw to a boundary of the residual CDF, times Z
FULL_BAND = 1e-5           # the same for a draw from a target row (both sides read the same fp32 row)


def oracle_params(wl, rows):
    logphi = orc.emission_logphi(wl.hidden_q[rows], wl.W_emit_q)
    logw = orc.head_logw(wl.shape.family, wl.hidden_q[rows], wl.W_sum_q, wl.T_static, wl.shape.r)
    return logphi, logw


# --------------------------------------------------------------------------- prefix log-marginals
SMALL = [
    # family, n, r, v, d, T
    (I.CP, 1, 1, 16, 64, 3),
    (I.CP, 5, 4, 320, 192, 140),
    (I.CP, 3, 128, 16, 64, 9),
    (I.HMM, 1, 4, 32, 64, 7),
    (I.HMM, 6, 8, 64, 128, 257),
    (I.HMM, 4, 32, 320, 64, 64),
    (I.HMM_CTX, 6, 8, 64, 128, 257),
    (I.HMM_CTX, 4, 32, 320, 64, 64),
    (I.BTREE, 2, 4, 32, 64, 9),
    (I.BTREE, 4, 16, 256, 128, 130),
    (I.BTREE, 8, 32, 48, 64, 33),
    (I.BTREE, 16, 8, 32, 64, 17),
    (I.BTREE, 64, 2, 16, 64, 3),
]


@pytest.mark.parametrize("family,n,r,v,d,T", SMALL)
def test_prefix_logprob_small_shapes(family, n, r, v, d, T):
    wl = I.make_workload(f"pre_{family}_{n}_{r}", I.HeadShape(family, n, r, v, d), T, seed=2000 + n + r + v + T,
                         weight_std=0.25)
    t = wl.targets.copy()
    if T > 4 and n > 1:
        t[1, n // 2:] = -1               # a masked tail (as at the end of a sequence)
        t[2, 0] = -1                     # a hole at the front
    dh = DeviceHead(wl)
    tt = torch.from_numpy(t).cuda()
    got = dh.window_prefix_logprob(targets=tt).cpu().numpy()
    joint = dh.window_logprob(targets=tt).cpu().numpy()
    assert dh.head.mtpc_get_status() == 0
    logphi, logw = oracle_params(wl, np.arange(T))
    ref = orc.prefix_logprob(family, logw, logphi, wl.T_static, t)
    assert got.shape == (T, n)
    assert np.abs(got - ref).max() <= LOGPROB_TOL
    assert np.abs(got[:, -1] - joint).max() <= 1e-4      # last column is the joint (another summation order)
    dh.close()


@pytest.mark.parametrize("idx,nsample", [(1, 96), (2, 96), (3, 48)])
def test_prefix_logprob_full_size_configs_on_sampled_positions(idx, nsample):
    wl = I.config_workload(idx)
    dh = DeviceHead(wl)
    rng = np.random.default_rng(40 + idx)
    rows = np.unique(np.concatenate([[0, 127, 128, wl.T - 129, wl.T - 128, wl.T - 1],
                                     rng.choice(wl.T, nsample, replace=False)]))
    got = dh.window_prefix_logprob().cpu().numpy()
    assert dh.head.mtpc_get_status() == 0 and np.isfinite(got).all()
    logphi, logw = oracle_params(wl, rows)
    ref = orc.prefix_logprob(wl.shape.family, logw, logphi, wl.T_static, wl.targets[rows])
    err = np.abs(got[rows] - ref).max()
    assert err <= LOGPROB_TOL, err
    assert (np.diff(got, axis=1) <= 1e-4).all()          # property at every position: prefixes only lose mass
    dh.close()


# --------------------------------------------------------------------------- draft -> acceptance
def target_rows_for(wl, W, bytes_o, logphi, logw, pos):
    """Target-model conditionals [W, n+1, v] fp32: Dirichlet rows; for every second window mixed half and half with
    the oracle's own conditional of the draft head along the oracle's draft (high acceptance), for every fourth
    window equal to it (everything accepted, up to rounding)."""
    s = wl.shape
    p = I.target_rows(I.BASE_SEED + 77, 9, (W, s.n + 1, s.v)).astype(np.float64)
    for i in range(s.n):
        qc = np.exp(orc.next_byte_logprob(s.family, logw, logphi, wl.T_static, bytes_o, np.full(W, i), pos))
        half = np.arange(W) % 2 == 0
        same = np.arange(W) % 4 == 0
        p[half, i, :] = 0.5 * p[half, i, :] + 0.5 * qc[half]
        p[same, i, :] = qc[same]
    return p.astype(np.float32)


def check_accept(wl, wpp, lowrank=None):
    """lowrank = (W_base, A, B): the device head keeps them factored; wl.W_emit_q must then be their exact composition."""
    s = wl.shape
    P, n = wl.T, s.n
    W = P * wpp
    rows = np.arange(P)
    pos = np.repeat(rows, wpp)
    dh = DeviceHead(wl, lowrank=lowrank)
    hidden_d = dh.hidden_device()            # kept alive: after a many-position draft the acceptance stage reads it again
    bytes_g, prefix_g = dh.draft_sample_prefix(wpp, hidden=hidden_d)
    assert dh.head.mtpc_get_status() == 0
    # oracle: its own draft, its own prefix marginals
    logphi, logw = oracle_params(wl, rows)
    d = orc.draft_sample(s.family, wl.hidden_q, wl.W_emit_q, wl.W_sum_q, wl.T_static, wpp, wl.uniforms)
    bytes_o = d["bytes"]
    gb = bytes_g.cpu().numpy()
    differ = (gb != bytes_o).any(axis=1)
    assert not (differ & (d["margin"] >= BOUNDARY_BAND)).any()
    # the device's prefix marginals of what it drafted
    want_prefix = orc.prefix_logprob(s.family, logw, logphi, wl.T_static, gb, pos)
    assert np.abs(prefix_g.cpu().numpy() - want_prefix).max() <= LOGPROB_TOL
    prefix_o = orc.prefix_logprob(s.family, logw, logphi, wl.T_static, bytes_o, pos)
    np.testing.assert_allclose(prefix_o[:, -1], d["logprob"], atol=1e-9)

    p = target_rows_for(wl, W, bytes_o, logphi, logw, pos)
    ua = I.uniforms(I.BASE_SEED + 78, 10, (W, n + 1))
    acc_g, next_g = dh.speculative_accept(P, wpp, bytes_g, prefix_g, torch.from_numpy(p).cuda(),
                                          torch.from_numpy(ua).cuda())
    assert dh.head.mtpc_get_status() == 0
    acc_g, next_g = acc_g.cpu().numpy(), next_g.cpu().numpy()
    ref = orc.speculative_accept(prefix_o, bytes_o, p, ua,
                                 lambda r_, s_: orc.next_byte_logprob(s.family, logw, logphi, wl.T_static,
                                                                      bytes_o[r_], s_, pos[r_]))
    assert acc_g.min() >= 0 and acc_g.max() <= n and next_g.min() >= 0 and next_g.max() < s.v
    near_final = np.where(ref["accepted"] == n, ref["margin_final"] < FULL_BAND,
                          ref["margin_final"] * ref["resid_mass"] < FINAL_BAND)
    near = (ref["margin_alpha"] < ALPHA_BAND) | near_final
    comparable = ~differ & ~near
    bad = comparable & ((acc_g != ref["accepted"]) | (next_g != ref["next_byte"]))
    hist = np.bincount(ref["accepted"], minlength=n + 1)
    print(f"{wl.name}: {W} windows, accepted-length histogram {hist.tolist()}, {int(differ.sum())} drafts differ near a "
          f"boundary, {int(near.sum())} windows inside a decision band, "
          f"{int(((acc_g != ref['accepted']) | (next_g != ref['next_byte'])).sum())} differ from the oracle")
    assert not bad.any(), (np.nonzero(bad)[0][:5], acc_g[bad][:5], ref["accepted"][bad][:5], next_g[bad][:5],
                           ref["next_byte"][bad][:5])
    # (with thousands of symbols the boundaries of the last draw's CDF lie closer together than its band is wide)
    assert comparable.sum() >= 0.9 * W or s.v > 512
    # The same decisions taken by the oracle from the DEVICE's own draft and prefix marginals: both sides then test
    # alpha against the same 32-bit numbers, the device as alpha * q > p in fp32, the oracle as alpha > p / q in fp64, so
    # the length of the accepted prefix must agree for every window whose closest test is further than 1e-5 from flipping
    # (two fp32 roundings of numbers below 1); only the last byte's draw keeps the wider band of the residual weights.
    own = orc.speculative_accept(prefix_g.cpu().numpy().astype(np.float64), gb, p, ua,
                                 lambda r_, s_: orc.next_byte_logprob(s.family, logw, logphi, wl.T_static, gb[r_], s_, pos[r_]))
    tight = own["margin_alpha"] >= OWN_ALPHA_BAND
    assert (acc_g[tight] == own["accepted"][tight]).all(), np.nonzero(tight & (acc_g != own["accepted"]))[0][:5]
    own_final = np.where(own["accepted"] == n, own["margin_final"] < FULL_BAND,
                         own["margin_final"] * own["resid_mass"] < FINAL_BAND)
    cmp_byte = tight & ~own_final
    assert (next_g[cmp_byte] == own["next_byte"][cmp_byte]).all()
    print(f"{wl.name}: against the oracle run on the device's own marginals: {int((~tight).sum())} of {W} windows within "
          f"{OWN_ALPHA_BAND} of flipping a test, {int((tight & own_final).sum())} more with the last draw inside its band")
    assert tight.sum() >= 0.98 * W
    if W >= 64:
        assert hist[n] > 0 and hist[:n].sum() > 0        # the case exercises full acceptance and rejection
    dh.close()


ACCEPT_SMALL = [
    # family, n, r, v, d, P, wpp
    (I.CP, 1, 2, 16, 64, 3, 4),
    (I.CP, 4, 8, 320, 128, 5, 16),
    (I.CP, 3, 32, 48, 64, 7, 8),
    (I.CP, 3, 64, 48, 64, 5, 16),          # more than 32 components: the mixture logits reach the kernels unnormalised
    (I.CP, 2, 128, 16, 64, 4, 16),
    (I.HMM, 1, 4, 32, 64, 2, 8),
    (I.HMM, 6, 8, 64, 128, 9, 8),
    (I.HMM, 4, 32, 512, 64, 3, 16),
    (I.HMM_CTX, 6, 8, 64, 128, 9, 8),
    (I.HMM_CTX, 4, 32, 512, 64, 3, 16),
    (I.BTREE, 2, 4, 32, 64, 9, 4),
    (I.BTREE, 4, 16, 256, 128, 6, 8),
    (I.BTREE, 8, 32, 48, 64, 5, 16),
    (I.BTREE, 16, 8, 32, 64, 128, 2),
    (I.CP, 2, 4, 1024, 64, 3, 4),          # vocabularies wider than 512 symbols
    (I.HMM, 2, 2, 4112, 64, 2, 8),
    # more than 128 positions: the many-position draft keeps no logits, the acceptance stage recomputes the slot it needs
    (I.CP, 3, 8, 64, 64, 150, 2),
    (I.HMM, 4, 8, 48, 64, 140, 1),
    (I.BTREE, 4, 4, 32, 64, 200, 1),
    (I.HMM_CTX, 3, 4, 320, 64, 130, 2),
    (I.CP, 2, 16, 320, 128, 300, 1),       # r v = 5120 logit columns per rejected window, 20 accumulator tiles per row tile
]


@pytest.mark.parametrize("family,n,r,v,d,P,wpp", ACCEPT_SMALL)
def test_accept_small_shapes(family, n, r, v, d, P, wpp):
    wl = I.make_workload(f"acc_{family}_{n}_{r}_{v}", I.HeadShape(family, n, r, v, d), P, seed=3000 + 5 * n + r + v + P,
                         wpp=wpp, weight_std=0.25)
    check_accept(wl, wpp)


@pytest.mark.parametrize("family,n,r,v,d,k,P,wpp", [
    (I.CP, 4, 8, 320, 128, 16, 5, 16),
    (I.HMM, 6, 8, 64, 128, 32, 9, 8),
    (I.BTREE, 4, 16, 256, 128, 16, 6, 8),
    (I.HMM_CTX, 4, 4, 48, 64, 16, 128, 2),     # the most positions the few-position path takes
    (I.CP, 2, 4, 1024, 64, 16, 3, 4),          # a vocabulary wider than 512 symbols
    # more than 128 positions, one window each: bytes drawn from the one selected unit, the rejected slot's logits formed
    # window by window from W_base h and B h
    (I.CP, 3, 8, 64, 64, 16, 150, 1),
    (I.HMM, 4, 8, 48, 64, 32, 140, 1),
    (I.BTREE, 4, 4, 32, 64, 16, 200, 1),
    (I.HMM_CTX, 3, 4, 320, 64, 16, 130, 1),
])
def test_draft_and_accept_on_a_factored_low_rank_head(family, n, r, v, d, k, P, wpp):
    """App. G's shared unembeddings kept factored (U_ij = W_i + A_ij B_ij never formed): the few-position draft streams
    W_base and B once, forms the logits from the two small products, and everything after is the dense head's path. Bytes,
    prefix marginals and acceptance decisions must be the oracle's on the exactly composed tensor."""
    wl = I.make_workload(f"lr_draft_{family}_{n}_{r}", I.HeadShape(family, n, r, v, d), P, seed=5200 + n + r + v + P,
                         wpp=wpp, weight_std=0.25)
    Wb, A, Bm = I.lowrank_parameters(n, r, v, d, k, seed=5300 + n + r, weight_std=0.25, adaptor_std=0.2)
    wl.W_emit_q = orc.lowrank_unembedding(Wb, A, Bm)       # fp64, exact: what the factored head computes on
    check_accept(wl, wpp, lowrank=(Wb, A, Bm))


@pytest.mark.parametrize("cell", [(I.CP, 8, 8), (I.CP, 16, 1), (I.HMM, 8, 64), (I.HMM, 16, 8)])
def test_accept_decode_cells(cell):
    fam, n, P = cell
    wl = I.config_workload(4, cell=cell)
    if P == 64:                                            # the oracle's conditionals are the cost: keep 8 positions
        wl = I.config_workload(4, cell=cell, T=8)
    check_accept(wl, wl.wpp)


def test_accept_needs_the_draft_state_and_flags_bad_inputs():
    wl = I.make_workload("acc_state", I.HeadShape(I.CP, 2, 4, 32, 64), 6, seed=31, wpp=2, weight_std=0.3)
    dh = DeviceHead(wl, max_positions=200)
    W, n, v = 12, 2, 32
    p = torch.from_numpy(I.target_rows(5, 1, (W, n + 1, v))).cuda()
    ua = torch.from_numpy(I.uniforms(5, 2, (W, n + 1))).cuda()
    b = torch.zeros((W, n), dtype=torch.int32, device="cuda")
    pre = torch.zeros((W, n), dtype=torch.float32, device="cuda")
    with pytest.raises(B.MtpcError) as e:                  # no draft yet
        dh.speculative_accept(6, 2, b, pre, p, ua)
    assert e.value.code == B.ERR_STATE
    bytes_g, prefix_g = dh.draft_sample_prefix(2)
    dh.speculative_accept(6, 2, bytes_g, prefix_g, p, ua)
    with pytest.raises(B.MtpcError) as e:                  # another P than the draft's
        dh.speculative_accept(5, 2, bytes_g, prefix_g, p, ua)
    assert e.value.code == B.ERR_STATE
    dh.window_logprob()                                    # overwrites the draft's sum-unit weights
    with pytest.raises(B.MtpcError) as e:
        dh.speculative_accept(6, 2, bytes_g, prefix_g, p, ua)
    assert e.value.code == B.ERR_STATE
    # more positions than were drafted (a many-position draft would have had to come first)
    with pytest.raises(B.MtpcError) as e:
        dh.speculative_accept(129, 1, bytes_g, prefix_g, p, ua)
    assert e.value.code == B.ERR_STATE
    # a uniform outside [0,1) and a byte outside [0,v): flagged, -1 / -1 for those windows only
    bytes_g, prefix_g = dh.draft_sample_prefix(2)
    ua2 = ua.clone()
    ua2[3, 1] = 1.5
    b2 = bytes_g.clone()
    b2[7, 0] = v
    acc, nxt = dh.speculative_accept(6, 2, b2, prefix_g, p, ua2)
    assert dh.head.mtpc_get_status() == (B.STATUS_BAD_UNIFORM | B.STATUS_BAD_TARGET)
    acc, nxt = acc.cpu().numpy(), nxt.cpu().numpy()
    assert acc[3] == -1 and nxt[3] == -1 and acc[7] == -1 and nxt[7] == -1
    keep = np.delete(np.arange(W), [3, 7])
    assert (acc[keep] >= 0).all() and (nxt[keep] >= 0).all()
    dh.close()


# --------------------------------------------------------------------------- Eq. 6
@pytest.mark.parametrize("family,n,r,v,d,N,L", [(I.CP, 4, 8, 320, 128, 3, 50), (I.HMM, 8, 16, 64, 64, 5, 33),
                                                 (I.BTREE, 8, 8, 32, 64, 2, 140), (I.CP, 2, 2, 16, 64, 300, 1),
                                                 (I.HMM_CTX, 4, 8, 64, 64, 4, 40)])
def test_window_loss_matches_oracle(family, n, r, v, d, N, L):
    wl = I.make_workload(f"loss_{family}", I.HeadShape(family, n, r, v, d), N * L, seed=4000 + n + N, weight_std=0.25)
    t = wl.targets.copy().reshape(N, L, n)
    for j in range(1, n):                                  # windows run past the end of their sequence
        t[:, max(L - j, 0):, j] = -1
    t[0, :, n - 1] = -1                                    # a sequence with no valid byte in the last slot
    t = t.reshape(N * L, n)
    dh = DeviceHead(wl)
    tt = torch.from_numpy(t).cuda()
    slot, loss = dh.window_loss(N, L, 0.8, targets=tt)
    slot2, loss2 = dh.window_loss(N, L, 0.8, targets=tt)
    assert torch.equal(slot, slot2) and torch.equal(loss, loss2)
    assert dh.head.mtpc_get_status() == 0
    logphi, logw = oracle_params(wl, np.arange(N * L))
    ref_slot, ref_loss = orc.composite_loss(orc.prefix_logprob(family, logw, logphi, wl.T_static, t), t, N, 0.8)
    assert np.abs(slot.cpu().numpy() - ref_slot).max() <= LOGPROB_TOL
    assert abs(float(loss.cpu()[0]) - ref_loss) <= LOGPROB_TOL * n
    dh.close()


# --------------------------------------------------------------------------- vocabulary not a multiple of 16
@pytest.mark.parametrize("family,n,r,v,vv,d,P,wpp", [(I.CP, 3, 4, 272, 268, 128, 6, 8), (I.HMM, 4, 8, 32, 17, 64, 5, 16),
                                                      (I.BTREE, 4, 4, 320, 305, 64, 4, 8), (I.HMM_CTX, 3, 4, 16, 1, 64, 3, 4)])
def test_padded_vocabulary_every_entry_point(family, n, r, v, vv, d, P, wpp):
    """v symbols per unit in memory, only the first vv exist (a byte-level Llama head has 268, stored as 272). The device
    gets weights whose padding rows hold noise; the oracle never sees them. Log-likelihood, prefix marginals, draft,
    acceptance and gradients must all ignore the padding."""
    from oracle import mtpc_oracle_grad as og
    shape = I.HeadShape(family, n, r, v, d, v_valid=vv)
    wl = I.make_workload(f"pad_{family}_{v}_{vv}", shape, P, seed=8000 + v + vv, wpp=wpp, weight_std=0.3)
    assert wl.W_emit_q.shape[2] == vv and wl.W_emit_dev_q.shape[2] == v and wl.targets.max() < vv
    dh = DeviceHead(wl)
    rows = np.arange(P)
    logphi, logw = oracle_params(wl, rows)
    assert logphi.shape[-1] == vv
    # log-likelihood and prefix marginals
    got = dh.window_logprob().cpu().numpy()
    assert np.abs(got - orc.window_logprob(family, wl.hidden_q, wl.W_emit_q, wl.W_sum_q, wl.T_static, wl.targets)).max() <= LOGPROB_TOL
    pre = dh.window_prefix_logprob().cpu().numpy()
    assert np.abs(pre - orc.prefix_logprob(family, logw, logphi, wl.T_static, wl.targets)).max() <= LOGPROB_TOL
    # draft: never a padding symbol, bytes as the oracle's
    bytes_g, prefix_g = dh.draft_sample_prefix(wpp)
    assert dh.head.mtpc_get_status() == 0
    gb = bytes_g.cpu().numpy()
    assert gb.min() >= 0 and gb.max() < vv
    dsm = orc.draft_sample(family, wl.hidden_q, wl.W_emit_q, wl.W_sum_q, wl.T_static, wpp, wl.uniforms)
    differ = (gb != dsm["bytes"]).any(axis=1)
    assert not (differ & (dsm["margin"] >= BOUNDARY_BAND)).any()
    pos = np.repeat(rows, wpp)
    assert np.abs(prefix_g.cpu().numpy() - orc.prefix_logprob(family, logw, logphi, wl.T_static, gb, pos)).max() <= LOGPROB_TOL
    # acceptance: target rows keep v entries on the device, the padding entries are ignored (filled with junk here)
    W = P * wpp
    p_valid = I.target_rows(99, 3, (W, n + 1, vv))
    p_dev = np.full((W, n + 1, v), 0.37, dtype=np.float32)
    p_dev[:, :, :vv] = p_valid
    ua = I.uniforms(99, 4, (W, n + 1))
    acc_g, next_g = dh.speculative_accept(P, wpp, bytes_g, prefix_g, torch.from_numpy(p_dev).cuda(), torch.from_numpy(ua).cuda())
    assert dh.head.mtpc_get_status() == 0
    bytes_o = dsm["bytes"]
    prefix_o = orc.prefix_logprob(family, logw, logphi, wl.T_static, bytes_o, pos)
    ref = orc.speculative_accept(prefix_o, bytes_o, p_valid.astype(np.float64), ua,
                                 lambda r_, s_: orc.next_byte_logprob(family, logw, logphi, wl.T_static, bytes_o[r_], s_, pos[r_]))
    near_final = np.where(ref["accepted"] == n, ref["margin_final"] < FULL_BAND, ref["margin_final"] * ref["resid_mass"] < FINAL_BAND)
    ok = ~differ & ~((ref["margin_alpha"] < ALPHA_BAND) | near_final)
    acc_g, next_g = acc_g.cpu().numpy(), next_g.cpu().numpy()
    assert next_g.max() < vv
    assert not (ok & ((acc_g != ref["accepted"]) | (next_g != ref["next_byte"]))).any()
    # gradients: nothing flows into the padding rows
    weight = np.random.default_rng(vv).normal(size=P).astype(np.float32)
    out = dh.window_logprob_backward(torch.from_numpy(weight).cuda())
    g = og.window_logprob_grad(family, wl.hidden_q, wl.W_emit_q, wl.W_sum_q, wl.T_static, wl.targets, weight)
    dW = out["dW_emit"].cpu().numpy()
    assert np.abs(dW[:, :, vv:, :]).max() == 0.0 if v > vv else True
    for name, got_t, want in (("dh", out["dh"].cpu().numpy(), g["dh"]), ("dW_emit", dW[:, :, :vv, :], g["dW_emit"]),
                              ("dW_sum", out["dW_sum"].cpu().numpy(), g["dW_sum"])):
        scale = np.abs(want).max()
        assert np.abs(got_t - want).max() <= 1e-2 * scale + 1e-4, name
    dh.close()


def test_argument_checks_of_prefix_loss_and_accept_calls():
    wl = I.make_workload("args2", I.HeadShape(I.CP, 2, 2, 16, 64), 6, seed=3, wpp=2)
    dh = DeviceHead(wl, max_positions=6, max_wpp=2)
    lib = B.lib()
    st = torch.cuda.current_stream().cuda_stream
    h = dh.hidden_device()
    t = torch.from_numpy(wl.targets).cuda()
    u = torch.from_numpy(wl.uniforms).cuda()
    f32 = dict(dtype=torch.float32, device="cuda")
    pre, slot, loss = torch.full((6, 2), 7.0, **f32), torch.empty(2, **f32), torch.empty(1, **f32)
    ob = torch.empty((12, 2), dtype=torch.int32, device="cuda")
    hd = dh.head.handle
    assert lib.mtpc_window_prefix_logprob(hd, h.data_ptr(), t.data_ptr(), 0, pre.data_ptr(), st) == 0
    torch.cuda.synchronize()
    assert (pre == 7.0).all()                                                          # T = 0 touches nothing
    assert lib.mtpc_window_prefix_logprob(hd, h.data_ptr(), t.data_ptr(), 7, pre.data_ptr(), st) == -2
    assert lib.mtpc_window_prefix_logprob(hd, h.data_ptr(), None, 6, pre.data_ptr(), st) == -1
    assert lib.mtpc_draft_sample_prefix(hd, h.data_ptr(), 6, 3, u.data_ptr(), ob.data_ptr(), pre.data_ptr(), st) == -2
    assert lib.mtpc_draft_sample_prefix(hd, h.data_ptr(), 6, 2, u.data_ptr(), None, pre.data_ptr(), st) == -1
    import ctypes
    g = ctypes.c_float(0.8)
    assert lib.mtpc_window_loss(hd, h.data_ptr(), t.data_ptr(), 3, 2, g, slot.data_ptr(), loss.data_ptr(), st) == 0
    assert lib.mtpc_window_loss(hd, h.data_ptr(), t.data_ptr(), 4, 2, g, slot.data_ptr(), loss.data_ptr(), st) == -2   # 8 > 6
    assert lib.mtpc_window_loss(hd, h.data_ptr(), t.data_ptr(), 0, 2, g, slot.data_ptr(), loss.data_ptr(), st) == -2
    assert lib.mtpc_window_loss(hd, h.data_ptr(), t.data_ptr(), 3, 2, g, None, loss.data_ptr(), st) == -1
    assert lib.mtpc_speculative_accept(hd, 6, 3, ob.data_ptr(), pre.data_ptr(), pre.data_ptr(), pre.data_ptr(), ob.data_ptr(),
                                       ob.data_ptr(), st) == -2
    assert lib.mtpc_speculative_accept(hd, 6, 2, None, pre.data_ptr(), pre.data_ptr(), pre.data_ptr(), ob.data_ptr(),
                                       ob.data_ptr(), st) == -1
    torch.cuda.synchronize()
    assert dh.head.mtpc_get_status() == 0
    dh.close()
