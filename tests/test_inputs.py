"""Host-side checks of the seeded input generators (no attention arithmetic involved)."""
import numpy as np
import torch

from paper_2510_01450_b200 import inputs


def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(0)
    x = (rng.standard_normal(100000) * 10.0 ** rng.integers(-6, 6, 100000)).astype(np.float32)
    x[:4] = [0.0, -0.0, 1.00390625, 1.01171875]      # exact ties: round to even
    got = inputs.round_to_bf16(x)
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(got, want)


def test_workloads_are_seeded_and_shaped():
    w = inputs.CONFIGS[2].shrink(B=1, H=2, n=64)
    q, k, v = inputs.make_prefill(w)
    q2, k2, v2 = inputs.make_prefill(w)
    assert q.shape == (1, 2, 64, 64) and v.shape == (1, 2, 64, 64) and q.dtype == np.float32
    np.testing.assert_array_equal(q, q2)
    np.testing.assert_array_equal(v, v2)
    np.testing.assert_array_equal(q, inputs.round_to_bf16(q))        # already bf16 values
    assert abs(float(k.std()) * np.sqrt(64) - 1.0) < 0.1 and abs(float(v.std()) - 1.0) < 0.1
    w1 = inputs.CONFIGS[1]
    q1, k1, v1 = inputs.make_prefill(w1)
    assert q1.shape == (1, 1, 256, 16) and abs(float(v1.std()) * 4.0 - 1.0) < 0.1


def test_regression_recipe_structure():
    w = inputs.CONFIGS[3].shrink(B=1, H=1, n=1100)
    q, k, v = inputs.make_prefill(w)
    np.testing.assert_array_equal(q[0, 0, :-1], k[0, 0, 1:])          # query i is key i+1
    # inside one 512-token segment the values are a linear map of the keys plus 0.1-sigma noise
    for lo, hi in ((0, 512), (512, 1024)):
        A, res, *_ = np.linalg.lstsq(k[0, 0, lo:hi].astype(np.float64), v[0, 0, lo:hi].astype(np.float64), rcond=None)
        resid = v[0, 0, lo:hi] - k[0, 0, lo:hi] @ A
        assert 0.07 < resid.std() < 0.12
    # across a segment boundary one map does not fit
    A, *_ = np.linalg.lstsq(k[0, 0, 0:1024].astype(np.float64), v[0, 0, 0:1024].astype(np.float64), rcond=None)
    assert (v[0, 0, :1024] - k[0, 0, :1024] @ A).std() > 0.125   # signal std is 1/sqrt(d) = 0.125


def test_decode_workload_and_sharding():
    w = inputs.CONFIGS[5].shrink(B=5, H=2, n=96, len_min=10, len_max=96)
    q, kc, vc, lens = inputs.make_decode(w)
    assert q.shape == (5, 2, 64) and kc.shape == (5, 2, 96, 64) and lens.dtype == np.int32
    assert lens.min() >= 10 and lens.max() <= 96
    cover = []
    for r in range(3):
        lo, hi = inputs.shard_units(10, r, 3)
        cover += list(range(lo, hi))
    assert cover == list(range(10))
    rows = inputs.sample_rows(inputs.CONFIGS[2], per_head=8, heads=3, dense_below=16)
    assert rows.min() >= 0 and rows.max() < 32 * 1024 and len(np.unique(rows)) == len(rows)


def test_regression_targets_are_the_noise_free_next_values():
    # target_i = A_s q_i with s the segment of position i + 1 and q_i = k_{i+1}: equal to v_{i+1} minus its noise,
    # also across a segment boundary (bf16 rounding of v is the only other difference)
    w = inputs.CONFIGS[3].shrink(B=1, H=2, n=300, segment=64, dtype="f32")
    q, k, v = inputs.make_prefill(w)
    t = inputs.regression_targets(w)
    resid = (t[:, :, :-1] - v[:, :, 1:]) / inputs.REGRESSION_NOISE
    assert abs(resid.std() - 1.0) < 0.05 and abs(resid.mean()) < 0.05
    per_pos = np.abs(resid).max(axis=(0, 1, 3))
    assert per_pos.max() < 6.0            # no position (boundaries included) is off by more than noise
