"""The fit of the re-characterisation tool (host arithmetic only): synthetic timings whose best SM count follows a
known law of channel size and operation count must give that law back."""
import math

from paper_2011_05630_b200 import characterise as ch


def test_fit_recovers_a_planted_law():
    choices = list(range(1, 149))
    rows = []
    for c in (16, 32, 64, 128, 256, 512):
        for ops in (1e6, 1e7, 1e8, 1e9, 1e10):
            s_true = 3.0 * math.log2(c) + 4.0 * math.log2(ops) - 90.0
            s_true = min(max(round(s_true), 1), 148)
            # time falls as 1/S down to S = s_true and stays flat beyond it
            times = [1.0 / min(s, s_true) for s in choices]
            rows.append((c, ops, choices, times))
    kc, ko, k0, rms = ch.fit(rows, slack=0.0)
    assert abs(kc - 3.0) < 0.2 and abs(ko - 4.0) < 0.2 and abs(k0 + 90.0) < 4.0 and rms < 1.0


def test_sweep_is_bounded_and_covers_both_kernel_sizes():
    layers = list(ch.sweep_layers(quick=True))
    assert 10 < len(layers) < 60 and {k for _, _, _, k in layers} == {1, 3}
    assert all(2.0 * n * hw * hw * k * k * c * c <= 4e11 for n, hw, c, k in layers)


def test_critical_operation_count_of_a_saturating_curve():
    # throughput T(ops) = T_max * ops / (ops + o_half): 80 % of the best from ops = 4 * o_half on
    o_half, t_max = 1e7, 5e12
    single = [(o, o / (t_max * o / (o + o_half))) for o in (1e5, 1e6, 1e7, 3e7, 4.5e7, 1e8, 1e9, 1e10)]
    crit, best = ch.critical_ops(single, frac=0.8)
    assert crit == 4.5e7 and abs(best - t_max * 1e10 / (1e10 + o_half)) < 1e-3 * t_max
    crit, _ = ch.critical_ops(single, frac=0.5)
    assert crit == 1e7
