"""Distortion of the CUDA path against what the paper states (Theorems 1-3, Section 3.2, Section 4.1):
properties that hold at any size, measured through tq_quantize_*, tq_dequantize and tq_score."""
import math
import os

import pytest

from paper_2504_19874_b200 import distortion

pytestmark = pytest.mark.gpu
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_values.txt")


def paper_values():
    vals = {}
    for line in open(GOLDEN):
        line = line.split("#")[0].split()
        if line:
            vals[line[0]] = [float(x) for x in line[1:]]
    return vals


@pytest.mark.parametrize("d", [1536, 200])
def test_distortion_levels_bounds_and_unbiasedness(d):
    pv = paper_values()
    r = distortion.measure(d=d, n=20000)
    for b in (1, 2, 3, 4):
        v = r[b]
        # Theorem 1 and the lower bound of Theorem 3; the printed values are rounded, hence the loose band
        assert 4.0 ** -b <= v["dmse"] <= pv["dmse_upper_const"][0] * 4.0 ** -b
        assert abs(v["dmse"] / pv["dmse_b1_b4"][b - 1] - 1) < 0.2
        # Theorem 2: error of the inner-product estimate for unit queries, and no bias
        assert 4.0 ** -b <= v["dprod_times_d"] <= pv["dprod_upper_const"][0] * 4.0 ** -b
        assert abs(v["dprod_times_d"] / pv["dprod_times_d_b1_b4"][b - 1] - 1) < 0.25
        assert abs(v["prod_bias"]) < 4 * v["prod_bias_sigma"]
        assert abs(v["prod_slope"] - 1) < 0.05
        # the error of the prod estimator does not grow with the inner product (Section 4.1)
        assert abs(v["prod_err_vs_ip_corr"]) < 0.05
    # Section 3.2: the mse reconstruction shrinks inner products, by 2/pi at one bit, less with more bits
    assert abs(r[1]["mse_estimator_slope"] - pv["mse_bias_b1"][0]) < 0.02
    assert r[1]["mse_estimator_slope"] < r[2]["mse_estimator_slope"] < r[3]["mse_estimator_slope"] < r[4]["mse_estimator_slope"] < 1
    # E||r||^2 of the prod residual = D_mse(b - 1): chain of Theorem 2's proof, D_prod = pi / (2 d) * D_mse(b - 1)
    for b in (2, 3, 4):
        assert abs(r[b]["dprod_times_d"] / (math.pi / 2 * r[b - 1]["dmse"]) - 1) < 0.12


def test_distortion_is_data_oblivious():
    """Same levels on the anisotropic, offset law of the embedding-like configurations (Section 1.1: the
    guarantees hold for worst-case inputs)."""
    iso = distortion.measure(d=1536, n=10000, isotropic=True)
    ani = distortion.measure(d=1536, n=10000, isotropic=False)
    for b in (1, 2, 3, 4):
        assert abs(ani[b]["dmse"] / iso[b]["dmse"] - 1) < 0.03
        assert abs(ani[b]["dprod_times_d"] / iso[b]["dprod_times_d"] - 1) < 0.15


def test_recall_grows_with_k_and_with_bits():
    """Recall 1@k of tq_topk against an exact fp32 scan (the measure of the paper's nearest-neighbour
    experiments) on synthetic embedding-like rows: monotone in k, better with more bits, complete by k = 64 at 4 bits."""
    rec = distortion.recall_1_at_k(d=1536, n=50000, nq=128)
    for b in (2, 4):
        vals = [rec[b][k] for k in sorted(rec[b])]
        assert all(x <= y + 1e-9 for x, y in zip(vals, vals[1:]))
    assert all(rec[4][k] >= rec[2][k] for k in rec[2])
    assert rec[4][1] >= 0.6 and rec[4][64] == 1.0 and rec[2][64] >= 0.95
