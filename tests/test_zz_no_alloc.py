"""mtpc_window_logprob_static: the window log-likelihood for callers that cannot allocate device memory (code
running inside another component's memory pool, or on a thread where a synchronising cudaMalloc is not
allowed). It takes no head and no workspace: its scratch is a static array inside the library.

The check: through the C ABI, its output must equal what mtpc_window_logprob gives on the same inputs (and what the
fp64 oracle gives), within the log-prob tolerance of the parity tests, on two calls in a row - the second on fewer positions and other targets,
so that whatever the first call left in the shared array would show if it were read. This file is collected last
on purpose: a run that stops at the first failure has then already run every other test."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import mtpc_oracle as orc
from paper_2511_11346_b200 import binding as B
from paper_2511_11346_b200 import inputs as I
from paper_2511_11346_b200.runner import DeviceHead

pytestmark = pytest.mark.gpu

LOGPROB_TOL = 2e-3


def static_logprob(dh, hidden, targets):
    s = dh.wl.shape
    out = torch.full((hidden.shape[0],), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.full((1,), 99, dtype=torch.int32, device="cuda")
    B.mtpc_window_logprob_static(s.family, s.n, s.r, s.v, s.d, dh.W_emit, dh.W_sum, dh.T_static, hidden, targets, out,
                                 status, v_valid=s.v_valid)
    torch.cuda.synchronize()
    return out.cpu().numpy(), int(status.item())


@pytest.mark.parametrize("family,n,r,v,d,T", [(I.CP, 5, 4, 320, 192, 300), (I.HMM, 6, 8, 64, 128, 257),
                                              (I.BTREE, 8, 16, 256, 128, 150)])
def test_static_scratch_call_matches_the_workspace_call_twice_in_a_row(family, n, r, v, d, T):
    wl = I.make_workload("noalloc", I.HeadShape(family, n, r, v, d, I.BF16), T, seed=900 + family, weight_std=0.25)
    dh = DeviceHead(wl)
    hidden = dh.hidden_device()
    targets = torch.from_numpy(wl.targets).cuda()
    want = dh.window_logprob(hidden, targets).cpu().numpy()
    assert dh.head.mtpc_get_status() == 0 and np.isfinite(want).all()

    got, status = static_logprob(dh, hidden, targets)
    assert status == 0
    assert np.abs(got - want).max() <= LOGPROB_TOL
    ref = orc.window_logprob(family, wl.hidden_q, wl.W_emit_q, wl.W_sum_q, wl.T_static, wl.targets)
    assert np.abs(got - ref).max() <= LOGPROB_TOL

    # second call: a ragged subset of the positions, shuffled targets with one byte marginalised and one bad
    T2 = T - 37
    t2 = wl.targets[::-1][:T2].copy()
    t2[3, 0] = -1
    t2[5, n - 1] = v
    hidden2 = hidden[:T2].contiguous()
    targets2 = torch.from_numpy(t2).cuda()
    want2 = dh.window_logprob(hidden2, targets2).cpu().numpy()
    assert dh.head.mtpc_get_status() == B.STATUS_BAD_TARGET
    got2, status2 = static_logprob(dh, hidden2, targets2)
    assert status2 == B.STATUS_BAD_TARGET
    assert np.isnan(got2[5]) and np.isnan(want2[5])
    keep = np.arange(T2) != 5
    assert np.abs(got2[keep] - want2[keep]).max() <= LOGPROB_TOL
    ref2 = orc.window_logprob(family, wl.hidden_q[:T2][keep], wl.W_emit_q, wl.W_sum_q, wl.T_static, t2[keep])
    assert np.abs(got2[keep] - ref2).max() <= LOGPROB_TOL
    dh.close()


def test_static_scratch_call_with_a_padded_vocabulary():
    # 44 symbols stored as 48 columns: the padding rows of W_emit hold large values that must carry no mass
    shape = I.HeadShape(I.CP, 3, 4, 48, 128, I.BF16, v_valid=44)
    wl = I.make_workload("noalloc_pad", shape, 140, seed=931, weight_std=0.25)
    dh = DeviceHead(wl)
    hidden = dh.hidden_device()
    targets = torch.from_numpy(wl.targets).cuda()
    want = dh.window_logprob(hidden, targets).cpu().numpy()
    ref = orc.window_logprob(I.CP, wl.hidden_q, wl.W_emit_q, wl.W_sum_q, wl.T_static, wl.targets)
    for _ in range(2):
        got, status = static_logprob(dh, hidden, targets)
        assert status == 0
        assert np.abs(got - want).max() <= LOGPROB_TOL and np.abs(got - ref).max() <= LOGPROB_TOL
    dh.close()


def test_static_scratch_call_refuses_what_does_not_fit_and_what_it_cannot_do():
    lib = B.lib()
    st = torch.cuda.current_stream().cuda_stream
    fake = ctypes.c_void_p(256)                    # never dereferenced: the size check comes first
    # BTree n=16 r=32 keeps 14368 + 512 fp32 per position: 16 MiB hold 281 positions, not 4096
    cfg = B.MtpcConfig(B.MTPC_BTREE, 16, 32, 256, 3072, B.MTPC_BF16, 1, 1, 0)
    assert lib.mtpc_window_logprob_static(ctypes.byref(cfg), fake, fake, None, fake, fake, 4096, fake, None, st) == B.ERR_STATIC_SCRATCH
    assert "static" in B.status_string(B.ERR_STATIC_SCRATCH)
    cfg32 = B.MtpcConfig(B.MTPC_CP, 2, 2, 16, 64, B.MTPC_F32, 1, 1, 0)
    assert lib.mtpc_window_logprob_static(ctypes.byref(cfg32), fake, fake, None, fake, fake, 4, fake, None, st) == -3
    cfg_ok = B.MtpcConfig(B.MTPC_CP, 2, 2, 16, 64, B.MTPC_BF16, 1, 1, 0)
    assert lib.mtpc_window_logprob_static(ctypes.byref(cfg_ok), fake, fake, None, fake, fake, 0, fake, None, st) == 0
    assert lib.mtpc_window_logprob_static(ctypes.byref(cfg_ok), None, fake, None, fake, fake, 4, fake, None, st) == -1
    assert lib.mtpc_window_logprob_static(None, fake, fake, None, fake, fake, 4, fake, None, st) == -1
