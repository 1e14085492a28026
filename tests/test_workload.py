"""The seeded input generator: deterministic, row-addressable, with the structure of VGGT activations (outlier channels, special-token rows)."""
import numpy as np

import workload


def test_rows_are_addressable_and_deterministic():
    spec = workload.block_specs(0)[0]
    full = spec.x_rows(0, 40)
    again = spec.x_rows(0, 40)
    part = spec.x_rows(17, 9)
    assert np.array_equal(full, again)
    assert np.array_equal(full[17:26], part)
    other = workload.block_specs(1)[0].x_rows(0, 40)
    assert not np.array_equal(full, other)


def test_special_rows_and_outlier_channels():
    spec = workload.block_specs(0)[0]
    x = workload.bf16_to_f32(spec.x_rows(0, 2 * workload.TOKENS_PER_FRAME)).astype(np.float64)
    g = spec.ch_gain()
    assert (g == workload.OUTLIER_GAIN).sum() == 8 and (g == 1).sum() == spec.K - 8
    rms_rows = np.sqrt((x[:, g == 1] ** 2).mean(axis=1))
    special = np.r_[0:5, workload.TOKENS_PER_FRAME:workload.TOKENS_PER_FRAME + 5]
    plain = np.setdiff1d(np.arange(x.shape[0]), special)
    assert np.all(rms_rows[special] > 80) and np.all(rms_rows[plain] < 1.3)   # special tokens of EVERY frame x100
    rms_cols = np.sqrt((x[plain] ** 2).mean(axis=0))
    assert np.all(rms_cols[g > 1] > 40) and np.all(rms_cols[g == 1] < 1.3)     # outlier channels x50


def test_distributions():
    fc2 = workload.block_specs(0)[3]
    assert fc2.K == 4096 and fc2.dist == workload.DIST_GELU
    x = workload.bf16_to_f32(fc2.x_rows(100, 64))
    assert x.min() > -0.3 * 50 and np.mean(x > 0) > 0.45 and abs(np.mean(x)) > 0.2     # GELU: bounded below, skewed
    t = workload.bf16_to_f32(workload.sweep_activations(0, 1024, 0, 256)).astype(np.float64)
    g = workload.outlier_gains(0, 2000 + 1024, 1024, 10)
    body = t[:, g == 1]
    kurt = np.mean(body ** 4) / np.mean(body ** 2) ** 2
    assert kurt > 6.0                                                                   # Student-t(3): heavy tails
    w = workload.bf16_to_f32(fc2.weight()).astype(np.float64)
    assert abs(w.std() - 0.02) < 5e-4 and abs(w.mean()) < 1e-4
    b = workload.bf16_to_f32(fc2.bias()).astype(np.float64)
    assert abs(b.std() - 0.01) < 1.5e-3
