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


@pytest.mark.parametrize("path", ["logprob", "draft_few", "draft_many", "backward"])
def test_a_wait_that_runs_out_is_reported_and_the_head_recovers(path):
    """Projection kernel (log-likelihood and sampling epilogues), the few-position draft kernel and the plain GEMMs of
    the backward pass: with a 50 ns limit the first wait for a copy gives up in every CTA."""
    T = {"logprob": 300, "draft_few": 8, "draft_many": 200, "backward": 300}[path]
    wl = I.make_workload("timeout_" + path, I.HeadShape(I.HMM, 4, 8, 64, 4096), T, seed=77, wpp=2, weight_std=0.2)
    dh = DeviceHead(wl)
    weight = torch.full((wl.T,), -1.0 / wl.T, dtype=torch.float32, device="cuda")

    def call():
        if path == "logprob":
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
    if path in ("logprob", "backward"):
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
