"""Length-aware batching simulator: the appendix metrics on cases small enough to work out by hand."""
import numpy as np
import pytest

from paper_2602_11812_b200 import inputs as gen
from paper_2602_11812_b200 import sjf_sim as sim


def test_hand_worked_example():
    true_len = np.array([10, 1, 9, 2])
    fcfs = sim.simulate_batches(true_len, np.arange(4), batch_size=2)
    # batches (10, 1) and (9, 2): allocated 2*10 + 2*9 = 38 for 22 useful slots
    assert fcfs.padding_ratio == pytest.approx((38 - 22) / 22)
    assert fcfs.total_time == 19 and fcfs.throughput == pytest.approx(4 / 19)
    assert fcfs.mean_jct == pytest.approx((10 + 1 + (10 + 9) + (10 + 2)) / 4)
    sjf = sim.simulate_batches(true_len, sim.sjf_order(true_len), batch_size=2)
    # batches (1, 2) and (9, 10): allocated 4 + 20 = 24
    assert sjf.padding_ratio == pytest.approx(2 / 22) and sjf.total_time == 12
    assert sjf.mean_jct == pytest.approx((1 + 2 + (2 + 9) + (2 + 10)) / 4)
    assert sim.mean_absolute_error([1, 2, 3], [2, 2, 5]) == pytest.approx(1.0)
    with pytest.raises(ValueError):
        sim.simulate_batches(true_len, np.array([0, 0, 1, 2]), 2)


def test_better_predictions_waste_less():
    # long-tailed true lengths; predictors of decreasing quality: exact, noisy, constant (= FCFS order)
    true_len = gen.lengths_lognormal(11, 512, 6.0, 1.0, 1, 8192)
    rng = np.random.default_rng(0)
    noisy = true_len * np.exp(rng.normal(0, 0.4, size=true_len.shape))
    res_exact = sim.compare_policies(true_len, true_len, 16)
    res_noisy = sim.compare_policies(true_len, noisy, 16)
    res_const = sim.compare_policies(true_len, np.full(512, 100.0), 16)
    assert res_exact["sjf_predicted"].padding_ratio == res_exact["sjf_oracle"].padding_ratio
    assert res_exact["sjf_oracle"].padding_ratio < res_noisy["sjf_predicted"].padding_ratio < res_const["sjf_predicted"].padding_ratio
    assert res_const["sjf_predicted"].padding_ratio == res_const["fcfs"].padding_ratio     # ties keep submission order
    assert res_noisy["sjf_predicted"].mean_jct < res_noisy["fcfs"].mean_jct
    assert res_noisy["sjf_predicted"].throughput > res_noisy["fcfs"].throughput
    assert res_exact["mae"] == 0 and res_noisy["mae"] > 0
    # batch size 1 never pads
    assert sim.simulate_batches(true_len, np.arange(512), 1).padding_ratio == 0
