"""GPU tests of the library's housekeeping rather than of its arithmetic: heads of different shapes alive at the same
time, and the give-up path of the bounded waits inside the tensor-core kernels.

The waits are made to run out without breaking anything: a healthy call is given a time limit far below one memory
round trip (a test hook of the library), so its first wait for a TMA copy expires. The CTA must then raise the timeout
bit, wait for what it has in flight, free its tensor memory and return; the next call, with the normal limit, must be
correct again. Nothing is withheld from a kernel and no wait is unbounded."""
import numpy as np
import pytest
import torch

from oracle import mtpc_oracle as orc
from paper_2511_11346_b200 import binding as B
from paper_2511_11346_b200 import inputs as I
from paper_2511_11346_b200.runner import DeviceHead

pytestmark = pytest.mark.gpu

LOGPROB_TOL = 2e-3


def oracle_logprob(wl):
    return orc.window_logprob(wl.shape.family, wl.hidden_q, wl.W_emit_q, wl.W_sum_q, wl.T_static, wl.targets)


def test_heads_of_different_shapes_do_not_lower_each_others_shared_memory_limit():
    """The dynamic shared-memory limit is a property of a kernel, not of a head: a tree head with long windows (80 KB
    per CTA, 97 KB with prefix marginals) must keep working after a head with short windows, or the static entry
    point, has set the same kernels up for less."""
    big = I.make_workload("tree_n16", I.HeadShape(I.BTREE, 16, 32, 64, 64), 70, seed=41, weight_std=0.3)
    small = I.make_workload("tree_n4", I.HeadShape(I.BTREE, 4, 32, 64, 64), 50, seed=42, weight_std=0.3)
    hmm_big = I.make_workload("hmm_r32", I.HeadShape(I.HMM, 8, 32, 64, 64), 60, seed=43, weight_std=0.3)
    hmm_small = I.make_workload("hmm_r4", I.HeadShape(I.HMM, 3, 4, 64, 64), 40, seed=44, weight_std=0.3)
    heads = [(wl, DeviceHead(wl)) for wl in (big, hmm_big)]
    later = [(wl, DeviceHead(wl)) for wl in (small, hmm_small)]           # created while the first two are alive
    s = small.shape
    out = torch.empty(small.T, dtype=torch.float32, device="cuda")
    dsm = later[0][1]
    B.mtpc_window_logprob_static(s.family, s.n, s.r, s.v, s.d, dsm.W_emit, dsm.W_sum, None, dsm.hidden_device(),
                                 torch.from_numpy(small.targets).cuda(), out)
    torch.cuda.synchronize()
    assert np.abs(out.cpu().numpy() - oracle_logprob(small)).max() <= LOGPROB_TOL
    for wl, dh in heads + later:
        got = dh.window_logprob().cpu().numpy()
        assert dh.head.mtpc_get_status() == 0
        assert np.abs(got - oracle_logprob(wl)).max() <= LOGPROB_TOL, wl.name
        pre = dh.window_prefix_logprob().cpu().numpy()
        assert np.abs(pre[:, -1] - oracle_logprob(wl)).max() <= LOGPROB_TOL, wl.name
    # gradients of the long-window heads after the short ones ran theirs
    for wl, dh in later + heads:
        w = torch.full((wl.T,), -1.0 / wl.T, dtype=torch.float32, device="cuda")
        g = dh.window_logprob_backward(w)
        assert dh.head.mtpc_get_status() == 0
        assert np.abs(g["logprob"].cpu().numpy() - oracle_logprob(wl)).max() <= LOGPROB_TOL, wl.name
    for _, dh in heads + later:
        dh.close()


@pytest.mark.parametrize("family,n,r,v,d,T,wpp", [
    (I.CP, 3, 16, 320, 128, 700, 1),        # 6 m-tiles: three pairs; v = 320 tiles straddle units
    (I.HMM, 4, 8, 64, 192, 385, 2),         # odd number of m-tiles and a ragged last one: the last pair's second CTA is empty
    (I.BTREE, 8, 32, 256, 64, 290, 1),      # 193 sum units: several sum tiles
    (I.CP, 2, 4, 48, 64, 100, 3),           # a single m-tile run by a pair
])
def test_both_builds_of_the_projection_kernel_give_the_same_numbers(family, n, r, v, d, T, wpp):
    """Single CTAs (cta_group::1) and CTA pairs (cta_group::2) form the same products in the same order: log-probs,
    drafted bytes and gradients must agree bit for bit, and with the oracle."""
    wl = I.make_workload("variants", I.HeadShape(family, n, r, v, d), T, seed=300 + n + r, wpp=wpp, weight_std=0.25)
    dh = DeviceHead(wl)
    ref = oracle_logprob(wl)
    weight = torch.full((wl.T,), -1.0 / wl.T, dtype=torch.float32, device="cuda")
    results = []
    for variant in (1, 2):
        dh.head.mtpc_debug_set_projection_variant(variant)
        lp = dh.window_logprob().cpu().numpy()
        assert np.abs(lp - ref).max() <= LOGPROB_TOL, variant
        out_bytes, out_lp = dh.draft_sample()
        g = dh.window_logprob_backward(weight)
        assert dh.head.mtpc_get_status(with_code=True) == (B.MTPC_OK, 0)
        results.append((lp, out_bytes.cpu().numpy(), out_lp.cpu().numpy(), g["dh"].cpu().numpy(), g["dW_emit"].cpu().numpy()))
    for a, b in zip(*results):
        np.testing.assert_array_equal(a, b)
    d = orc.draft_sample(family, wl.hidden_q, wl.W_emit_q, wl.W_sum_q, wl.T_static, wl.wpp, wl.uniforms)
    differ = (results[0][1] != d["bytes"]).any(axis=1)
    assert not (differ & (d["margin"] >= 1e-6)).any()
    dh.close()


@pytest.mark.parametrize("family,n,r,v,d,T,wpp", [
    (I.CP, 3, 4, 320, 128, 2000, 1),        # 12 units, ~500 windows each: every unit spans several 128-row tiles
    (I.CP, 2, 64, 64, 64, 150, 1),          # 128 units for 300 draws: units with one window, units with none
    (I.HMM, 4, 8, 48, 64, 300, 2),          # two windows per position, padded-free odd vocabulary tile (48 columns)
    (I.BTREE, 8, 32, 256, 64, 290, 1),      # tree latents
    (I.HMM_CTX, 3, 16, 320, 64, 200, 1),    # contextual transitions; a unit's 320 columns in two accumulator tiles
])
def test_draws_sorted_by_unit_give_the_same_bytes(family, n, r, v, d, T, wpp):
    """Many-position draft (Algorithm 1): running every position against every unit, or sorting the (window, slot) pairs
    by the unit they sample from and multiplying each by that unit only, must return the same bytes and log-probs -
    the order in which windows are processed must not matter - and they must be the oracle's."""
    wl = I.make_workload("grouped", I.HeadShape(family, n, r, v, d), T, seed=500 + n + r, wpp=wpp, weight_std=0.25)
    dh = DeviceHead(wl)
    u = wl.uniforms.copy()
    u[5, n + 1] = 2.0                        # a refused byte draw ...
    u[9, 0] = -1.0                           # ... and a refused latent draw keep their meaning in both modes
    ud = torch.from_numpy(u).cuda()
    got = []
    for mode in (1, 2, 2):                   # the sorted pass twice: its internal row order differs from run to run
        dh.head.mtpc_debug_set_draft_grouping(mode)
        out_bytes, out_lp = dh.draft_sample(uniforms=ud)
        assert dh.head.mtpc_get_status(with_code=True) == (B.MTPC_OK, B.STATUS_BAD_UNIFORM)
        got.append((out_bytes.cpu().numpy(), out_lp.cpu().numpy()))
    for b, lp in got[1:]:
        np.testing.assert_array_equal(b, got[0][0])
        np.testing.assert_array_equal(lp, got[0][1])
    gb, gl = got[1]
    assert gb[5, 1] == -1 and (gb[9] == -1).all() and np.isnan(gl[5]) and np.isnan(gl[9])
    ok = np.ones(len(gb), dtype=bool)
    ok[[5, 9]] = False
    fam = wl.shape.family
    ref = orc.draft_sample(fam, wl.hidden_q, wl.W_emit_q, wl.W_sum_q, wl.T_static, wpp, wl.uniforms)
    differ = (gb != ref["bytes"]).any(axis=1) & ok
    assert not (differ & (ref["margin"] >= 1e-6)).any()
    same = ok & ~differ
    assert np.abs(gl[same] - ref["logprob"][same]).max() <= LOGPROB_TOL
    dh.close()


@pytest.mark.parametrize("path", ["logprob", "logprob_single_ctas", "draft_few", "draft_many", "draft_many_ungrouped", "backward"])
def test_a_wait_that_runs_out_is_reported_and_the_head_recovers(path):
    """Projection kernel (log-likelihood and sampling epilogues), the few-position draft kernel and the plain GEMMs of
    the backward pass: with a 50 ns limit the first wait for a copy gives up in every CTA."""
    T = {"logprob": 300, "logprob_single_ctas": 300, "draft_few": 8, "draft_many": 200, "draft_many_ungrouped": 200,
         "backward": 300}[path]
    wl = I.make_workload("timeout_" + path, I.HeadShape(I.HMM, 4, 8, 64, 4096), T, seed=77, wpp=2, weight_std=0.2)
    dh = DeviceHead(wl)
    weight = torch.full((wl.T,), -1.0 / wl.T, dtype=torch.float32, device="cuda")
    if path == "logprob_single_ctas":
        dh.head.mtpc_debug_set_projection_variant(1)      # the other paths pair their CTAs (more than one m-tile)
    if path == "draft_many_ungrouped":
        dh.head.mtpc_debug_set_draft_grouping(1)          # wpp = 2 against r = 8 units: sorted by unit otherwise

    def call():
        if path.startswith("logprob"):
            return dh.window_logprob()
        if path == "backward":
            return dh.window_logprob_backward(weight)["logprob"]
        return dh.draft_sample()[1]

    call()
    assert dh.head.mtpc_get_status(with_code=True) == (B.MTPC_OK, 0)
    dh.head.mtpc_debug_set_wait_limit_ns(50)
    call()                                                # gives up; outputs unspecified
    torch.cuda.synchronize()                              # the kernels returned: no hang, the context is alive
    code, bits = dh.head.mtpc_get_status(with_code=True)
    assert code == B.ERR_TIMEOUT and bits & B.STATUS_TIMEOUT
    assert "wait" in B.status_string(code)
    assert dh.head.mtpc_get_status(with_code=True) == (B.MTPC_OK, 0)      # reading cleared the word
    dh.head.mtpc_debug_set_wait_limit_ns(0)               # back to the default
    if path.startswith("logprob") or path == "backward":
        got = call().cpu().numpy()
        assert np.abs(got - oracle_logprob(wl)).max() <= LOGPROB_TOL
    else:
        out_bytes, out_lp = dh.draft_sample()
        ref = orc.draft_sample(wl.shape.family, wl.hidden_q, wl.W_emit_q, wl.W_sum_q, wl.T_static, wl.wpp, wl.uniforms)
        differ = (out_bytes.cpu().numpy() != ref["bytes"]).any(axis=1)
        assert not (differ & (ref["margin"] >= 1e-6)).any()
        same = ~differ
        assert np.abs(out_lp.cpu().numpy()[same] - ref["logprob"][same]).max() <= LOGPROB_TOL
    assert dh.head.mtpc_get_status(with_code=True) == (B.MTPC_OK, 0)
    dh.close()


@pytest.mark.parametrize("family,n,r,v,d,P,wpp", [
    (I.CP, 8, 16, 320, 256, 8, 16),         # few positions: weight pass, per-slot kernel and circuit as dependent launches
    (I.HMM, 4, 8, 64, 128, 5, 3),
    (I.BTREE, 8, 8, 64, 64, 200, 2),        # many positions: sorted draws, projection passes, circuit
])
def test_draft_and_acceptance_calls_can_be_captured_into_a_cuda_graph(family, n, r, v, d, P, wpp):
    """The calls only enqueue work on the caller's stream (no synchronisation, no allocation), so a serving loop may
    capture draft + acceptance once and replay the graph: the replay must return what the plain calls return, and they
    what the oracle returns."""
    wl = I.make_workload("graph", I.HeadShape(family, n, r, v, d), P, seed=900 + n + r, wpp=wpp, weight_std=0.25)
    dh = DeviceHead(wl)
    W = P * wpp
    hidden = dh.hidden_device()
    u = torch.from_numpy(wl.uniforms).cuda()
    tp = torch.from_numpy(I.target_rows(I.BASE_SEED + 5, 9, (W, n + 1, v))).cuda()
    ua = torch.from_numpy(I.uniforms(I.BASE_SEED + 6, 10, (W, n + 1))).cuda()

    targets = torch.from_numpy(wl.targets).cuda()

    def buffers():
        return (torch.zeros((W, n), dtype=torch.int32, device="cuda"), torch.zeros((W, n), dtype=torch.float32, device="cuda"),
                torch.zeros(W, dtype=torch.int32, device="cuda"), torch.zeros(W, dtype=torch.int32, device="cuda"),
                torch.zeros(P, dtype=torch.float32, device="cuda"), torch.zeros((P, n), dtype=torch.float32, device="cuda"))

    def cycle(ob, opre, oacc, onxt, lp, pre, stream=None):
        dh.head.mtpc_draft_sample_prefix(hidden, wpp, u, ob, opre, stream=stream)
        dh.head.mtpc_speculative_accept(P, wpp, ob, opre, tp, ua, oacc, onxt, stream=stream)
        dh.head.mtpc_window_logprob(hidden, targets, lp, stream=stream)           # the likelihood calls as well
        dh.head.mtpc_window_prefix_logprob(hidden, targets, pre, stream=stream)

    plain = buffers()
    cycle(*plain)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    replayed = buffers()
    with torch.cuda.stream(side):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            cycle(*replayed, stream=side)
        for t in replayed:
            t.zero_()
        graph.replay()
        graph.replay()
        side.synchronize()
    assert dh.head.mtpc_get_status(with_code=True) == (B.MTPC_OK, 0)
    for a, b in zip(plain, replayed):
        np.testing.assert_array_equal(a.cpu().numpy(), b.cpu().numpy())
    ref = orc.draft_sample(wl.shape.family, wl.hidden_q, wl.W_emit_q, wl.W_sum_q, wl.T_static, wpp, wl.uniforms)
    differ = (replayed[0].cpu().numpy() != ref["bytes"]).any(axis=1)
    assert not (differ & (ref["margin"] >= 1e-6)).any()
    assert np.abs(replayed[4].cpu().numpy() - oracle_logprob(wl)).max() <= LOGPROB_TOL
    assert np.abs(replayed[5].cpu().numpy()[:, -1] - oracle_logprob(wl)).max() <= LOGPROB_TOL
    del graph
    dh.close()
