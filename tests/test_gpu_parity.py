"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same seeded inputs.

Bars: window log-probs within 2e-3 absolute; drafted bytes bit-exact for every window whose
draws all lie further than 1e-6 from an oracle CDF boundary (the others are counted and printed); draft
log-probs are checked for EVERY window against the oracle's joint of the bytes the GPU returned."""
import numpy as np
import pytest
import torch

from oracle import mtpc_oracle as orc
from paper_2511_11346_b200 import binding as B
from paper_2511_11346_b200 import inputs as I
from paper_2511_11346_b200.runner import DeviceHead

pytestmark = pytest.mark.gpu

LOGPROB_TOL = 2e-3
BOUNDARY_BAND = 1e-6


def oracle_logprob(wl, rows, targets=None):
    t = wl.targets[rows] if targets is None else targets
    return orc.window_logprob(wl.shape.family, wl.hidden_q[rows], wl.W_emit_q, wl.W_sum_q, wl.T_static, t)


def check_logprob(dh, wl, rows):
    got = dh.window_logprob().cpu().numpy()
    assert dh.head.mtpc_get_status() == 0
    assert np.isfinite(got).all()
    ref = oracle_logprob(wl, rows)
    err = np.abs(got[rows] - ref).max() if len(rows) else 0.0
    assert err <= LOGPROB_TOL, f"{wl.name}: max |log q - oracle| = {err}"
    return err


def check_draft(dh, wl, rows, wpp=None):
    wpp = wpp or wl.wpp
    n = wl.shape.n
    out_bytes, out_lp = dh.draft_sample(wpp)
    assert dh.head.mtpc_get_status() == 0
    gb, gl = out_bytes.cpu().numpy(), out_lp.cpu().numpy()
    assert gb.min() >= 0 and gb.max() < wl.shape.v
    wsel = (np.asarray(rows)[:, None] * wpp + np.arange(wpp)[None, :]).reshape(-1)
    ref = orc.draft_sample(wl.shape.family, wl.hidden_q[rows], wl.W_emit_q, wl.W_sum_q, wl.T_static, wpp,
                           wl.uniforms[wsel])
    mism = (gb[wsel] != ref["bytes"]).any(axis=1)
    near = ref["margin"] < BOUNDARY_BAND
    print(f"{wl.name}: {len(wsel)} windows, {int(near.sum())} with a draw within {BOUNDARY_BAND} of a CDF boundary, "
          f"{int(mism.sum())} differing from the oracle")
    assert not (mism & ~near).any(), f"bytes differ away from a boundary: margins {ref['margin'][mism & ~near]}"
    # joint log-prob of what the GPU actually drafted, all windows
    pos = np.repeat(np.arange(len(rows)), wpp)
    logphi = orc.emission_logphi(wl.hidden_q[rows], wl.W_emit_q)
    logw = orc.head_logw(wl.shape.family, wl.hidden_q[rows], wl.W_sum_q, wl.T_static, wl.shape.r)
    want = orc.circuit_eval(wl.shape.family, logw[pos], orc.evidence(logphi, gb[wsel], pos), wl.T_static)
    err = np.abs(gl[wsel] - want).max()
    assert err <= LOGPROB_TOL, f"{wl.name}: draft log-prob error {err}"
    return int(mism.sum()), int(near.sum())


# --------------------------------------------------------------------------- the five named workloads
def test_config0_cp_tiny_whole():
    wl = I.config_workload(0)
    dh = DeviceHead(wl)
    rows = np.arange(wl.T)
    check_logprob(dh, wl, rows)
    check_draft(dh, wl, rows)
    dh.close()


@pytest.mark.parametrize("idx,nsample", [(1, 256), (2, 256), (3, 128), (5, 128), (6, 256)])
def test_full_size_configs_on_sampled_positions(idx, nsample):
    """Full-size launch (the configuration the benchmark times); the oracle checks a seeded sample of
    positions, always including the first and last rows of the first and last 128-row tiles."""
    wl = I.config_workload(idx)
    dh = DeviceHead(wl)
    rng = np.random.default_rng(idx)
    rows = np.unique(np.concatenate([[0, 127, 128, wl.T - 129, wl.T - 128, wl.T - 1],
                                     rng.choice(wl.T, nsample, replace=False)]))
    check_logprob(dh, wl, rows)
    if wl.wpp:
        check_draft(dh, wl, rows)
    dh.close()


@pytest.mark.parametrize("cell", I.DECODE_CELLS)
def test_config4_decode_cells(cell):
    wl = I.config_workload(4, cell=cell)
    dh = DeviceHead(wl)
    rows = np.arange(wl.T) if wl.T <= 8 else np.sort(np.random.default_rng(4).choice(wl.T, 8, replace=False))
    check_draft(dh, wl, rows)
    dh.close()


# --------------------------------------------------------------------------- small, ragged, edge shapes
SMALL = [
    # family, n, r, v, d, T, wpp
    (I.CP, 1, 1, 16, 64, 1, 1),
    (I.CP, 3, 2, 48, 128, 129, 3),
    (I.CP, 5, 4, 320, 192, 300, 2),
    (I.CP, 2, 64, 32, 64, 37, 1),
    (I.CP, 2, 128, 16, 64, 5, 2),
    (I.CP, 2, 8, 512, 64, 131, 1),
    (I.HMM, 1, 4, 32, 64, 7, 2),
    (I.HMM, 6, 8, 64, 128, 257, 1),
    (I.HMM, 4, 32, 320, 64, 64, 16),
    (I.HMM, 3, 1, 16, 64, 3, 1),
    (I.HMM_CTX, 1, 4, 32, 64, 7, 2),
    (I.HMM_CTX, 6, 8, 64, 128, 257, 1),
    (I.HMM_CTX, 4, 32, 320, 64, 64, 16),
    (I.HMM_CTX, 3, 1, 16, 64, 3, 1),
    (I.HMM_CTX, 5, 16, 48, 64, 140, 3),
    (I.BTREE, 2, 4, 32, 64, 9, 2),
    (I.BTREE, 4, 16, 256, 128, 130, 1),
    (I.BTREE, 8, 32, 48, 64, 33, 4),
    (I.BTREE, 64, 2, 16, 64, 3, 1),
]


@pytest.mark.parametrize("family,n,r,v,d,T,wpp", SMALL)
def test_small_shapes_span_tiles_and_ragged_tails(family, n, r, v, d, T, wpp):
    shape = I.HeadShape(family, n, r, v, d, I.BF16)
    wl = I.make_workload(f"small_{family}_{n}_{r}_{v}", shape, T, seed=1000 + 7 * n + r + v + T, wpp=wpp,
                         weight_std=0.25)        # logits of order one even at small d
    dh = DeviceHead(wl)
    rows = np.arange(T)
    check_logprob(dh, wl, rows)
    check_draft(dh, wl, rows)
    dh.close()


@pytest.mark.parametrize("family,n,r,v,vv,d,T,wpp", [
    (I.CP, 2, 4, 1024, 0, 64, 6, 4),          # few positions: the per-slot kernel walks the unit 512 symbols at a time
    (I.HMM, 2, 2, 4112, 4100, 64, 5, 3),      # padded vocabulary, 4100 symbols stored as 4112
    (I.CP, 1, 2, 32768, 0, 64, 3, 4),         # a subword-sized vocabulary
    (I.CP, 2, 4, 1024, 0, 64, 200, 1),        # many positions: units streamed through tensor memory twice, draws sorted by unit
    (I.BTREE, 2, 2, 4112, 4100, 64, 150, 2),
    (I.HMM, 2, 2, 32768, 0, 64, 140, 1),
])
def test_drafting_from_vocabularies_wider_than_tensor_memory(family, n, r, v, vv, d, T, wpp):
    """More than 512 symbols per unit (App. G's subword case): log-likelihood, drafted bytes and draft log-probs against
    the oracle, on the few-position and on the many-position path."""
    wl = I.make_workload(f"widev_{v}_{T}", I.HeadShape(family, n, r, v, d, v_valid=vv), T, seed=2000 + v % 97 + T, wpp=wpp,
                         weight_std=0.25)
    dh = DeviceHead(wl)
    rows = np.arange(T)
    check_logprob(dh, wl, rows)
    check_draft(dh, wl, rows)
    dh.close()


def test_fp32_io_at_the_training_width():
    """fp32 hidden states and weights at d = 4096 (the library rounds them on the device), several m-tiles, ragged tail."""
    shape = I.HeadShape(I.CP, 2, 4, 320, 4096, I.F32)
    wl = I.make_workload("f32io_wide", shape, 300, seed=78, wpp=1)
    dh = DeviceHead(wl)
    rows = np.arange(wl.T)
    check_logprob(dh, wl, rows)
    check_draft(dh, wl, rows)
    dh.close()


def test_fp32_io_is_rounded_to_bf16_on_the_device():
    shape = I.HeadShape(I.HMM, 3, 4, 32, 128, I.F32)
    wl = I.make_workload("f32io", shape, 70, seed=77, wpp=2, weight_std=0.2)
    dh = DeviceHead(wl)
    check_logprob(dh, wl, np.arange(70))
    check_draft(dh, wl, np.arange(70))
    dh.close()


def test_masked_targets_marginalise_and_bad_targets_flag():
    shape = I.HeadShape(I.BTREE, 4, 8, 32, 64)
    wl = I.make_workload("mask", shape, 40, seed=5, weight_std=0.3)
    t = wl.targets.copy()
    t[0, :] = -1                      # everything summed out: log 1 = 0
    t[1, 2] = -1
    t[2, 0] = -5
    t[3, 1] = -1
    t[3, 3] = -1
    dh = DeviceHead(wl)
    got = dh.window_logprob(targets=torch.from_numpy(t).cuda()).cpu().numpy()
    assert dh.head.mtpc_get_status() == 0
    ref = oracle_logprob(wl, np.arange(40), t)
    assert np.abs(got - ref).max() <= LOGPROB_TOL
    assert abs(got[0]) <= 1e-4
    t[5, 1] = shape.v                 # out of range: NaN for that window only, status bit set
    got = dh.window_logprob(targets=torch.from_numpy(t).cuda()).cpu().numpy()
    assert dh.head.mtpc_get_status() == B.STATUS_BAD_TARGET
    assert np.isnan(got[5]) and np.isfinite(np.delete(got, 5)).all()
    assert dh.head.mtpc_get_status() == 0          # reading clears it
    dh.close()


def test_bad_uniform_is_flagged_not_sampled():
    shape = I.HeadShape(I.CP, 2, 4, 32, 64)
    wl = I.make_workload("badu", shape, 6, seed=6, wpp=2, weight_std=0.3)
    u = wl.uniforms.copy()
    u[3, 2 + 1] = 1.0                 # byte draw of slot 1, window 3
    u[7, 0] = -0.25                   # latent draw of window 7
    dh = DeviceHead(wl)
    out_bytes, out_lp = dh.draft_sample(uniforms=torch.from_numpy(u).cuda())
    assert dh.head.mtpc_get_status() == B.STATUS_BAD_UNIFORM
    gb, gl = out_bytes.cpu().numpy(), out_lp.cpu().numpy()
    assert gb[3, 1] == -1 and gb[3, 0] >= 0
    assert (gb[7] == -1).all()
    assert (np.delete(gb, [3, 7], axis=0) >= 0).all()
    # a window with a refused draw has no log-prob (NaN), the others are untouched
    assert np.isnan(gl[3]) and np.isnan(gl[7]) and np.isfinite(np.delete(gl, [3, 7])).all()
    dh.close()


def test_bad_uniform_many_position_path_gives_nan_logprob():
    shape = I.HeadShape(I.HMM, 4, 8, 64, 64)
    wl = I.make_workload("badu_many", shape, 150, seed=16, wpp=1, weight_std=0.3)     # 150 > 128 positions
    u = wl.uniforms.copy()
    u[20, 4 + 2] = 1.5                # byte draw of slot 2, window 20
    u[140, 1] = float("nan")          # latent draw of window 140
    dh = DeviceHead(wl)
    out_bytes, out_lp = dh.draft_sample(uniforms=torch.from_numpy(u).cuda())
    assert dh.head.mtpc_get_status() == B.STATUS_BAD_UNIFORM
    gb, gl = out_bytes.cpu().numpy(), out_lp.cpu().numpy()
    assert gb[20, 2] == -1 and (gb[140] == -1).all()
    assert np.isnan(gl[20]) and np.isnan(gl[140]) and np.isfinite(np.delete(gl, [20, 140])).all()
    dh.close()


def test_results_are_deterministic_and_host_calls_agree():
    wl = I.make_workload("det", I.HeadShape(I.HMM, 4, 8, 320, 256), 200, seed=11, wpp=3, weight_std=0.1)
    dh = DeviceHead(wl)
    a = dh.window_logprob().cpu().numpy()
    b = dh.window_logprob().cpu().numpy()
    np.testing.assert_array_equal(a, b)
    b1, l1 = dh.draft_sample()
    b2, l2 = dh.draft_sample()
    assert torch.equal(b1, b2) and torch.equal(l1, l2)
    # host-buffer entry points: same numbers, copies inside the call
    hh = dh.hidden_host()
    th = torch.from_numpy(wl.targets).pin_memory()
    oh = torch.empty(wl.T, dtype=torch.float32).pin_memory()
    dh.head.mtpc_window_logprob_host(hh, th, oh)
    np.testing.assert_array_equal(oh.numpy(), a)
    uh = torch.from_numpy(wl.uniforms).pin_memory()
    bh = torch.empty((wl.T * 3, 4), dtype=torch.int32).pin_memory()
    lh = torch.empty(wl.T * 3, dtype=torch.float32).pin_memory()
    dh.head.mtpc_draft_sample_host(hh, 3, uh, bh, lh)
    assert torch.equal(bh, b1.cpu()) and torch.equal(lh, l1.cpu())
    dh.close()


def test_call_limits_and_empty_calls():
    wl = I.make_workload("lim", I.HeadShape(I.CP, 2, 2, 16, 64), 4, seed=3, wpp=2)
    dh = DeviceHead(wl, max_positions=4, max_wpp=2)
    lib = B.lib()
    h = dh.hidden_device()
    t = torch.from_numpy(wl.targets).cuda()
    out = torch.full((4,), 7.0, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    assert lib.mtpc_window_logprob(dh.head.handle, h.data_ptr(), t.data_ptr(), 0, out.data_ptr(), st) == 0
    torch.cuda.synchronize()
    assert (out == 7.0).all()                                                         # T = 0 touches nothing
    assert lib.mtpc_window_logprob(dh.head.handle, h.data_ptr(), t.data_ptr(), 5, out.data_ptr(), st) == -2
    assert lib.mtpc_window_logprob(dh.head.handle, None, t.data_ptr(), 4, out.data_ptr(), st) == -1
    u = torch.from_numpy(wl.uniforms).cuda()
    ob = torch.empty((8, 2), dtype=torch.int32, device="cuda")
    assert lib.mtpc_draft_sample(dh.head.handle, h.data_ptr(), 4, 3, u.data_ptr(), ob.data_ptr(), out.data_ptr(), st) == -2
    assert lib.mtpc_draft_sample(dh.head.handle, h.data_ptr(), 4, 0, u.data_ptr(), ob.data_ptr(), out.data_ptr(), st) == -2
    # too small a workspace is refused at creation
    cfg = dh.head.cfg
    handle = __import__("ctypes").c_void_p(0)
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    code = lib.mtpc_create_head(__import__("ctypes").byref(cfg), dh.W_emit.data_ptr(), dh.W_sum.data_ptr(), None,
                                small.data_ptr(), 256, st, __import__("ctypes").byref(handle))
    assert code == -4
    assert dh.head.mtpc_launch_count() >= 0
    dh.close()


def test_max_windows_per_position():
    wl = I.make_workload("wpp64", I.HeadShape(I.CP, 2, 4, 32, 64), 3, seed=8, wpp=64, weight_std=0.3)
    dh = DeviceHead(wl)
    check_draft(dh, wl, np.arange(3))
    dh.close()


def test_chunked_host_call_equals_device_call():
    """The host-buffer entry point uploads and processes 2048 positions at a time; the results are those of one
    device-buffer call (same arithmetic per position), ragged last chunk included, twice in a row."""
    wl = I.make_workload("host_chunks", I.HeadShape(I.HMM, 4, 8, 320, 128), 5000, seed=91, weight_std=0.2)
    dh = DeviceHead(wl)
    dev = dh.window_logprob().cpu()
    hh = dh.hidden_host()
    th = torch.from_numpy(wl.targets).pin_memory()
    for _ in range(2):
        oh = torch.full((wl.T,), 7.0).pin_memory()
        dh.head.mtpc_window_logprob_host(hh, th, oh)
        assert torch.equal(oh, dev)
    assert dh.head.mtpc_get_status() == 0
    dh.close()
