"""The roofline arithmetic of bench.py against numbers worked out by hand (no GPU, no weights generated)."""
import types

import bench
from paper_2511_11346_b200 import inputs as I


def _fake(shape, T):
    return types.SimpleNamespace(shape=shape, T=T, name="fake", wpp=0)


def test_algorithmic_flops_of_the_mixture_training_head():
    # 2 d (n r v + S r) per position: 2 * 4096 * (8*16*320 + 1*16) = 335 675 392 FLOP, times 8192 positions
    wl = _fake(I.HeadShape(I.CP, 8, 16, 320, 4096), 8192)
    assert bench.algorithmic_flops(wl) == 2 * 4096 * (40960 + 16) * 8192 == 2749852811264


def test_algorithmic_flops_count_every_sum_unit_of_the_tree():
    # S = 1 + (n - 2) r = 449 sum units of r = 32 inputs
    wl = _fake(I.HeadShape(I.BTREE, 16, 32, 320, 4096), 4096)
    assert bench.algorithmic_flops(wl) == 2 * 4096 * (16 * 32 * 320 + 449 * 32) * 4096


def test_circuit_bytes():
    # the circuit kernel reads G [T, n, r] and log omega [T, S r] and writes [T], fp32
    wl = _fake(I.HeadShape(I.CP, 8, 16, 320, 4096), 8192)
    assert bench.circuit_bytes(wl) == 4 * 8192 * (128 + 16 + 1) == 4751360
    wl = _fake(I.HeadShape(I.HMM_CTX, 16, 32, 320, 4096), 8192)
    assert bench.circuit_bytes(wl) == 4 * 8192 * (512 + (1 + 15 * 32) * 32 + 1)


def test_workload_name_states_the_shape():
    wl = _fake(I.HeadShape(I.CP, 8, 16, 320, 4096), 8192)
    name = bench.workload_name(1, wl)
    for piece in ("T=8192", "d=4096", "n=8", "r=16", "v=320"):
        assert piece in name


def test_cpu_baseline_helper_runs_the_oracle_on_a_sample():
    wl = I.config_workload(0)
    rate, seconds = bench.oracle_positions_per_s(wl, 32, chunk=16)
    assert rate > 0 and seconds > 0 and abs(rate * seconds - 32) < 1e-6
    assert bench.host_threads() >= 1
