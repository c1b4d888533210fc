"""Plan helpers on top of the C ABI: default tuner constants for B200 and the strategies the
benchmark compares.  Everything here only marshals arguments; the tuner (Eq. 5 + Algorithm 1)
and the reduced brute-force search run inside the library."""
from __future__ import annotations

from . import binding as B

# Eq. 5 weights are the paper's; the affine map to an SM count is set so that the layers of the large workloads get the
# whole chip (the characterisation finds the best SM count flat below ~1e7 operations and 148 from ~1e8 on).  The critical
# operation count per SM is the one the characterisation reads off as the paper defines it (Sec. IV-C): a single SM's
# throughput stays within a fifth of its best (10 TFLOP/s) from 1.5e10 operations on (python -m ...characterise).
TUNER = dict(alpha=0.316, beta=0.659, kappa=12.0, kappa0=-60.0, op_critical=1.5e10)


def tuned_plan(net, n_layers, **over):
    p = dict(TUNER, **over)
    return B.net_autotune(net, n_layers, p["alpha"], p["beta"], p["kappa"], p["kappa0"], p["op_critical"],
                          s_max=0, legalise=1)


def sm_fractions(sms):
    """The paper's reduced core-count set {1,2,4,8,12,16,24,32}/32 scaled to this device."""
    return sorted({max(1, round(sms * f / 32)) for f in (1, 2, 4, 8, 12, 16, 24, 32)})


def ablation_plans(net, n_layers, sms, **over):
    """The execution strategies of the paper's ablation (Table 3), as (name, group_end, sm_count) with None for
    "to be searched": 1 no fusion on one SM; 2 no fusion, one network-wide SM count (the caller tries
    sm_fractions and keeps the best); 3 no fusion, every layer on its own Eq. 5 count; 4 everything fused that
    can be, all SMs; 5 Algorithm 1's blocks, all SMs; 6 Algorithm 1's blocks and SM counts.  Strategy 3 is
    Algorithm 1 with a vanishing critical operation count (every layer closes its own block), strategy 4 with an
    unreachable one and the hand-over through L2 allowed, so that a block closes only where no fused kernel can run the
    layers (a pooling or fully connected layer, sixteen layers reached) and not where fusing is estimated not to pay.
    The library's choice of hand-over is set back afterwards; setting it drops the net's current plan."""
    every = list(range(n_layers))
    per_layer = tuned_plan(net, n_layers, **dict(over, op_critical=1e-30))
    B.net_set_option(net, B.OPT_GROUP_KERNEL, 2)
    try:
        all_fused = tuned_plan(net, n_layers, **dict(over, op_critical=1e300))
    finally:
        B.net_set_option(net, B.OPT_GROUP_KERNEL, 0)
    tuned = tuned_plan(net, n_layers, **over)
    return [("1 no fusion, 1 SM", every, [1] * n_layers),
            ("2 no fusion, best fixed S", every, None),
            ("3 no fusion, per-layer S (Eq. 5)", per_layer[0], per_layer[1]),
            ("4 all fused, all SMs", all_fused[0], [sms] * len(all_fused[0])),
            ("5 Algorithm 1 blocks, all SMs", tuned[0], [sms] * len(tuned[0])),
            ("6 Algorithm 1 blocks and SM counts", tuned[0], tuned[1])]
